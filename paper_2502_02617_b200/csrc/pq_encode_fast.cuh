// Fast encoder for head_dim 128 (included by pq_encode.cu): sign tests for the analytic codebooks (uniform level 1,
// symmetric upper levels), a table-driven level 1 and per-boundary upper levels for any other codebook.
//
// The rotation y = x . S is computed with float32-grade accuracy (tensor cores with S split into
// bf16 terms, or float32 FMAs).  Either way |y - y_exact| <= rot_err * ||x||_2 per coordinate:
//   * a float32 dot product of 128 terms is off by at most 128 * 2^-24 = 2^-17 of sum_k |x_k||S_kj|, which is
//     at most ||x||_2 (Cauchy-Schwarz, columns of S have unit norm): kRotErr = 1.1 * 2^-17;
//   * on tensor cores the products of bf16 inputs are exact in float32.  Three bf16 terms (round to nearest,
//     8 significant bits each) represent a float32 S to 2^-26 |S|, and the 24 accumulating MMAs are taken to
//     add at most 2 ulp of the running sum each, 3 * 2^-20 of the same sum in all: kRotErrTc = 1.1 * (3 * 2^-20
//     + 2^-26).  Measured against float64 on 1.07e9 rotated coordinates of the synthetic workloads (N(0,1),
//     outlier channels, rows scaled up 30 x): the largest error was 0.09 * 2^-17 ||x||_2, 4.5 x inside the bound
//     (with two terms, whose representation error alone may reach 2^-18: 0.28 * 2^-17).
// Angles are never computed.  Every code is decided by sign tests on the pair (Algorithm 1, Polar +
// Quant, in the form "which side of the boundary line is the point on"), in float32, together with
// a certified margin: a decision is trusted only if the point is farther from every boundary than
// the error bound allows it to move.  The rare decisions inside the margin are taken again in
// float64 from the original inputs by the whole warp, so the codes equal a float64 evaluation of
// Algorithm 1 (up to ~1e-15 rad).
#pragma once

namespace pq {

constexpr float kRotErr = 1.1f * 7.62939453125e-06f;                                  // 1.1 * 2^-17
constexpr float kRotErrTc = 1.1f * (3.f * 9.5367431640625e-07f + 1.4901161193847656e-08f);  // 1.1 * (3 * 2^-20 + 2^-26)

// Per-call constants of the fast quantiser.
struct FastQuant {
  float t2[3][3];   // tan^2 of the three boundaries of levels 2, 3, 4
  uint32_t sym;     // the boundaries of every level >= 2 are b, pi/4, pi/2 - b (kFlagSymmetricUpper)
  float ua[3][3], ub[3][3];  // the boundary lines of levels 2, 3, 4 scaled to max(|A|, |B|) = 1: D_k = A_k sa + B_k sb
  uint32_t analytic;       // sym and the uniform level-1 codebook: every decision is a sign test
  const uint2* l1_cells;   // level-1 decision table of any other codebook (Tables::l1_cells or a copy in shared memory)
};

constexpr int kFastQuantBytes = 128;  // what the kernels set aside for a FastQuant in shared memory
static_assert(sizeof(FastQuant) <= kFastQuantBytes, "shared-memory slot of FastQuant");

__device__ inline void load_fast_quant(const Tables* tb, FastQuant* fq) {
  for (int l = 0; l < 3; ++l)
    for (int k = 0; k < 3; ++k) {
      const double T = tb->bnd_tan2[3 * l + k];
      fq->t2[l][k] = (float)T;
      fq->ua[l][k] = (float)(T > 1.0 ? -1.0 : -T);      // sb - T sa, divided by max(1, T)
      fq->ub[l][k] = (float)(T > 1.0 ? 1.0 / T : 1.0);
    }
  fq->sym = (tb->flags & kFlagSymmetricUpper) != 0u;
  fq->analytic = (tb->flags & (kFlagSymmetricUpper | kFlagUniformL1)) == (kFlagSymmetricUpper | kFlagUniformL1);
  fq->l1_cells = &tb->l1_cells[0][0];
}

// Per-row constants of the margins (dy = bound on the error of one rotated coordinate of the row).
struct RowMargins {
  float dy;       // as given
  float dy3;      // 3.02 dy: threshold of the table-driven level-1 test
  float dy1;      // level-1 threshold: dy plus the float32 roundings of the level-1 tests
  float c[3];     // 8.4 E^2 for levels 2, 3, 4 (E^2 = 2, 4, 8 dy^2)
  float cs[3];    // the same plus the float32-rounding term of the folded (symmetric) test
  float csg[3];   // the same for the scaled-line test of any codebook (quant_upper_lines_push)
  float base[3];  // 42 E^4 * 4: every tested line has coefficients of at most 1
};
// `norm` >= ||y||_2 of the row, `rot_err` = bound on the error of one rotated coordinate relative to it.
// The float32 roundings of the tests themselves are folded into the constants, using u <= norm and w <= norm^2
// for every coordinate magnitude u and partial squared radius w of the row:
//   * level 1: the scaled distances are off by at most 1.3 * 2^-24 u (the two constants of t and one product);
//     1.8e-7 norm covers that twice over;
//   * levels >= 2 (folded test): the squared radii carry a relative error of at most 2^-22 + 2^-24 < rho = 4e-7,
//     and 42 rho^2 w^2 <= 6.8e-12 norm^2 w.
__device__ __forceinline__ RowMargins make_row_margins(float norm, float rot_err, const FastQuant& fq) {
  RowMargins m;
  m.dy = rot_err * norm;
  m.dy1 = fmaf(1.8e-7f, norm, m.dy);
  m.dy3 = fmaxf(3.02f * m.dy, 1e-30f);  // the floor keeps a certified u in the range where the reciprocal is accurate
  const float e2 = m.dy * m.dy, rr = 6.8e-12f * norm * norm;
#pragma unroll
  for (int l = 0; l < 3; ++l) {
    const float el = (float)(2 << l) * e2;
    m.c[l] = 8.4f * el;
    m.cs[l] = m.c[l] + rr;
    m.csg[l] = fmaf(1.05e-11f * norm, norm, m.c[l]);
    m.base[l] = 168.f * el * el;
  }
  return m;
}

// Level >= 2 decisions on squared child radii (sa: cosine side, sb: sine side): the common margin.
//   code = #{k : sb > T_k sa},  T_k = tan^2(beta_k)  (both sides of r_b cos b > r_a sin b are >= 0).
// The radii are norms of n-coordinate sub-vectors, so they move by at most E = sqrt(n) * dy.
// With D = sb - T sa, |D - D_exact| <= 2E(r_b + T r_a) + E^2 (1 + T) + rho (sb + T sa), and
// (2E(r_b + T r_a))^2 <= 8 E^2 (sb + T^2 sa); with (p+q+z)^2 <= 1.05 p^2 + 21 (q+z)^2 <= 1.05 p^2 + 42 (q^2+z^2)
// boundary k is certified if D_k^2 > 8.4 E^2 (sb + T_k^2 sa) + 42 E^4 (1+T_k)^2 + 42 rho^2 (sb + T_k sa)^2.
// Both tests below first bring every line to coefficients of at most 1 (by folding for symmetric boundaries, by
// scaling otherwise), so that sb + T^2 sa <= sa + sb and (1 + T)^2 <= 4 for all of them.

// Codes, squared radius and ambiguity mask of one 16-coordinate block.
// Ambiguity bits: 0..7 level-1 pairs, 8..11 level 2, 12..13 level 3, 14 level 4.
struct FastBlock {
  uint32_t l1, l2, l3, l4, amb;
  float radius;
};

__device__ __forceinline__ float fast_sqrt(float x) {
  float r;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(x));  // 1 ulp-level error: far inside the fp16 rounding of the radius
  return r;
}

// ---- decisions whose code bits are read off sign bits ------------------------------------------
// (acc << 1) | sign bit of v: one funnel shift collects a decision bit.
__device__ __forceinline__ uint32_t push_sign(uint32_t acc, uint32_t v) { return __funnelshift_l(v, acc, 1); }

// Level-1 decision for the uniform codebook (boundaries k pi/8): fold into the first octant,
// u = max(|a|,|b|), v = min(|a|,|b|); the boundaries are the axes (v = 0), the diagonals (u = v) and
// the lines at pi/8 from the axes (v cos(pi/8) = u sin(pi/8)).  Each coordinate moves by at most
// dy, so the signed distance to a line with unit normal (n1, n2) moves by at most (|n1| + |n2|) dy:
// dy for an axis, sqrt(2) dy for a diagonal, (cos + sin)(pi/8) dy = 1.3066 dy for the pi/8 lines.
// The three distances are computed already scaled (d = (|a| - |b|) / 2, t = 0.76537 (v cos - u sin)), so
// that one comparison against `dy1` (dy plus the float32 roundings, see make_row_margins) serves all.
// The function appends four raw sign bits to `raw` -- sign(b), sign(a), sign(d), sign(t) -- and one
// "certified" bit to `ok`; level1_codes() turns the raw nibbles of a block into codes.  A zero (or NaN)
// anywhere leaves the pair uncertified, so the sign conventions at exact zeros do not matter.
__device__ __forceinline__ void quant_level1_push(float a, float b, float dy1, uint32_t& raw, uint32_t& ok) {
  const float ax = fabsf(a), ay = fabsf(b);
  const float u = fmaxf(ax, ay), v = fminf(ax, ay);
  const float d = fmaf(ay, -0.5f, 0.5f * ax);
  const float t = fmaf(v, 0.92387953251128674f * 0.76536686473017954f, u * (-0.38268343236508977f * 0.76536686473017954f));
  const float dmin = fminf(fminf(v, fabsf(d)), fabsf(t));
  const float slack = dy1 - dmin;  // < 0: certified
  raw = push_sign(push_sign(push_sign(push_sign(raw, __float_as_uint(b)), __float_as_uint(a)), __float_as_uint(d)),
                  __float_as_uint(t));
  ok = push_sign(ok, __float_as_uint(slack));
}
// Codes of the eight pairs of a block from their raw nibbles (sb, sa, sd, st), all pairs at once.  With
// x = sa ^ sb, w = (|b| > |a|) = sd, hi = (past the pi/8 line of the folded octant) = ~st the code is
// sb << 3 | x << 2 | (w ^ x) << 1 | (w ^ hi ^ x): a prefix-xor inside each nibble and a flip of bit 0.
__device__ __forceinline__ uint32_t level1_codes(uint32_t raw) {
  uint32_t c = raw ^ ((raw & 0xEEEEEEEEu) >> 1);   // (r3, r2^r3, r1^r2, r0^r1)
  c ^= (c & 0xCCCCCCCCu) >> 2;                     // (r3, r2^r3, r1^r2^r3, r0^r1^r2^r3)
  return c ^ 0x11111111u;
}

// Level-1 decision for any codebook, from the table Tables::l1_cells.  With u = max(|a|,|b|), v = min(|a|,|b|) and
// t = v / u, the octant (signs of b, a and |a| - |b|) and the cell of t select one boundary value tau and the codes
// on its two sides; the table guarantees that |t - tau| does not exceed the distance from t to any boundary ray,
// measured in the octant's coordinate t_c = tan(angle from the octant's first edge) continued past both edges.
// Margin: the exact pair differs from (a, b) by at most dy per coordinate, and in the octant's frame (the
// coordinates with the computed signs and order) its u changes by at most dy and its signed v by at most dy, so its
// t_c differs from t by at most dy (u + v) / (u (u - dy)) <= 2 dy / (u - dy).  A decision is certified if
//   |t - tau| u > 3.02 dy + 6e-7 u:
// the table keeps |t - tau| <= 1, hence u > 3 dy, hence the bound above is below 3 dy / u; 6e-7 covers the float32
// roundings of t (reciprocal and product: 1.8e-7), of tau (6e-8) and of this test.  The exact point then lies in the
// same gap between rays as t, in this octant or past one of its edges, and the code is the gap's.
// u = 0, a NaN in (a, b) or in the margin, or a cell without a single deciding boundary (tau = NaN) leave the
// pair uncertified.
// The function appends the 4 code bits to `l1` and one "certified" bit to `ok`.
__device__ __forceinline__ void quant_level1_table_push(float a, float b, float dy3, const uint2* __restrict__ cells,
                                                        uint32_t& l1, uint32_t& ok) {
  const float ax = fabsf(a), ay = fabsf(b);
  const float u = fmaxf(ax, ay), v = fminf(ax, ay);
  float ru;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(ru) : "f"(u));
  const float t = fminf(v * ru, 1.f);  // u = 0 or denormal (ru = inf): t = 1 and |t - tau| u stays below dy3
  const uint32_t o = push_sign(push_sign(push_sign(0u, __float_as_uint(b)), __float_as_uint(a)), __float_as_uint(ax - ay));
  // 2^20 + t * scale: the float's unit in the last place is 1/8, so mantissa bits 3.. hold floor(t * scale + 1/16)
  const uint32_t cell8 = __float_as_uint(fmaf(t, kL1CellScale, 1048576.f)) & (uint32_t)((kL1Cells - 1) << 3);
  const uint2 e = *reinterpret_cast<const uint2*>(reinterpret_cast<const char*>(cells) + (o * (kL1Cells * 8) + cell8));
  const float dd = t - __uint_as_float(e.x);
  const float slack = fmaf(-fabsf(dd), u, fmaf(6e-7f, u, dy3));  // < 0: certified (NaN: not)
  const uint32_t code = e.y << (dd > 0.f ? 4 : 0);                // the code in bits 28..31
  l1 = __funnelshift_l(code, l1, 4);
  ok = push_sign(ok, __float_as_uint(slack));
}

// The level >= 2 decision (margin: see above) for symmetric boundaries (T0, 1, 1/T0), folded onto m = min(sa, sb), M = max(sa, sb):
// only the diagonal (M - m) and the boundary m = T0 M of the point's own side can be the nearest ones, and the
// margin of the boundary sb = sa / T0 is the one of m = T0 M after multiplying both sides by T0^2.  Every T
// that is tested is <= 1, so sb + T^2 sa <= sa + sb and the caller's `base` uses (1 + T)^2 <= 4.
// The function appends the 2 code bits to `lv` and one "certified" bit to `ok`: the code is
// hi << 1 | (hi ^ lo) with hi = (sb > sa) = sign of sa - sb and lo = (m > T0 M) = complement of the sign of dout.
__device__ __forceinline__ void quant_upper_sym_push(float sa, float sb, float T0, float cs, float base, uint32_t& lv,
                                                     uint32_t& ok) {
  const float m = fminf(sa, sb), M = fmaxf(sa, sb);
  const float h = sa - sb, dout = fmaf(-T0, M, m);
  const float w = sa + sb;
  const float dm = fminf(fabsf(dout), fabsf(h));
  // certified if dm^2 > c w + base + 42 rho^2 w^2; the last term is inside cs (see make_row_margins).  NaN: not certified.
  const float slack = fmaf(-dm, dm, fmaf(cs, w, base));
  const uint32_t hb = __float_as_uint(h);
  lv = push_sign(push_sign(lv, hb), ~(hb ^ __float_as_uint(dout)));
  ok = push_sign(ok, __float_as_uint(slack));
}

// The level >= 2 decision for any three ascending boundaries.  Each boundary line sb = T_k sa is scaled by
// 1 / max(1, T_k): D_k = A_k sa + B_k sb with max(|A_k|, |B_k|) = 1 and the sign of sb - T_k sa, so that one margin
// serves all three: |D_k - exact| <= 2E(|B_k| r_b + |A_k| r_a) + E^2 (|A_k| + |B_k|) + rho (sa + sb) with
// (2E(...))^2 <= 8 E^2 (sa + sb), (|A_k| + |B_k|)^2 <= 4 and rho = 5e-7 for the float32 roundings (squared radii
// 2^-22 + 2^-24, the product and the fma), and as derived above boundary k is certified if
// D_k^2 > 8.4 E^2 w + 42 * 4 E^4 + 42 rho^2 w^2, w = sa + sb <= norm^2 (the last term is inside csg).
// D_0 >= D_1 >= D_2 up to those roundings, and the code is the number of positive ones: bit 1 = (D_1 > 0), bit 0 =
// parity of the three.  The function appends the COMPLEMENTS of the two code bits (the sign bits) to `lv` and one
// "certified" bit to `ok`; the caller complements `lv` once per block.
__device__ __forceinline__ void quant_upper_lines_push(float sa, float sb, const float* A, const float* B, float csg, float base,
                                                       uint32_t& lv, uint32_t& ok) {
  const float d0 = fmaf(A[0], sa, B[0] * sb), d1 = fmaf(A[1], sa, B[1] * sb), d2 = fmaf(A[2], sa, B[2] * sb);
  const float dm = fminf(fminf(fabsf(d0), fabsf(d1)), fabsf(d2));
  const float slack = fmaf(-dm, dm, fmaf(csg, sa + sb, base));  // < 0: certified (NaN: not)
  lv = push_sign(push_sign(lv, __float_as_uint(d1)), __float_as_uint(d0) ^ __float_as_uint(d1) ^ __float_as_uint(d2));
  ok = push_sign(ok, __float_as_uint(slack));
}

// Codes, squared radius and ambiguity mask of one block.  Pairs and nodes are visited from the last to the
// first, so that the bits that are appended end up in canonical order.
// kAnalytic: the analytic codebooks (uniform level 1, symmetric upper levels); otherwise any codebook.
template <bool kAnalytic>
__device__ __forceinline__ void polar_quant_block_fast(const float* y, const RowMargins& rm, const FastQuant& fq,
                                                       FastBlock* out) {
  float s1[8], s2[4], s3[2];
  uint32_t l1 = 0, l2 = 0, l3 = 0, l4 = 0, ok1 = 0, ok2 = 0, ok3 = 0, ok4 = 0;
#pragma unroll
  for (int j = 7; j >= 0; --j) {
    if (kAnalytic) quant_level1_push(y[2 * j], y[2 * j + 1], rm.dy1, l1, ok1);
    else quant_level1_table_push(y[2 * j], y[2 * j + 1], rm.dy3, fq.l1_cells, l1, ok1);
    s1[j] = fmaf(y[2 * j], y[2 * j], y[2 * j + 1] * y[2 * j + 1]);
  }
  if (kAnalytic) {
#pragma unroll
    for (int j = 3; j >= 0; --j) {
      quant_upper_sym_push(s1[2 * j], s1[2 * j + 1], fq.t2[0][0], rm.cs[0], rm.base[0], l2, ok2);
      s2[j] = s1[2 * j] + s1[2 * j + 1];
    }
#pragma unroll
    for (int j = 1; j >= 0; --j) {
      quant_upper_sym_push(s2[2 * j], s2[2 * j + 1], fq.t2[1][0], rm.cs[1], rm.base[1], l3, ok3);
      s3[j] = s2[2 * j] + s2[2 * j + 1];
    }
    quant_upper_sym_push(s3[0], s3[1], fq.t2[2][0], rm.cs[2], rm.base[2], l4, ok4);
  } else {
#pragma unroll
    for (int j = 3; j >= 0; --j) {
      quant_upper_lines_push(s1[2 * j], s1[2 * j + 1], fq.ua[0], fq.ub[0], rm.csg[0], rm.base[0], l2, ok2);
      s2[j] = s1[2 * j] + s1[2 * j + 1];
    }
#pragma unroll
    for (int j = 1; j >= 0; --j) {
      quant_upper_lines_push(s2[2 * j], s2[2 * j + 1], fq.ua[1], fq.ub[1], rm.csg[1], rm.base[1], l3, ok3);
      s3[j] = s2[2 * j] + s2[2 * j + 1];
    }
    quant_upper_lines_push(s3[0], s3[1], fq.ua[2], fq.ub[2], rm.csg[2], rm.base[2], l4, ok4);
    l2 = ~l2 & 0xFFu;   // the sign bits are the complements of the code bits
    l3 = ~l3 & 0xFu;
    l4 = ~l4 & 0x3u;
  }
  out->l1 = kAnalytic ? level1_codes(l1) : l1;
  out->l2 = l2;
  out->l3 = l3;
  out->l4 = l4;
  // ambiguity bits: 0..7 level-1 pairs, 8..11 level 2, 12..13 level 3, 14 level 4
  out->amb = ~(ok1 | (ok2 << 8) | (ok3 << 12) | (ok4 << 14)) & 0x7FFFu;
  out->radius = fast_sqrt(s3[0] + s3[1]);
}

// ---- exact re-decision of the ambiguous angles ------------------------------------------------
// Threads push their ambiguous decisions into a CTA-wide queue; after a barrier, groups of 8 lanes
// take one entry each, recompute in float64 the 2^level rotated coordinates under that angle from
// the original inputs (x in its storage type, S in float32: both exact in float64), decide again
// and patch the code bits in the cache with 32-bit atomics.  The queue is drained in rounds, so a
// tile with more ambiguous angles than the queue holds only takes more rounds.
// The queue is kept sorted by level (one region per level: 1/2, 1/4, 1/8 and 1/8 of the capacity), so that
// the four 8-lane groups of a warp, which take consecutive entries, almost always run the same code path.
template <int kCap>
struct FixQueueT {
  static constexpr int kCapacity = kCap;
  __host__ __device__ static constexpr int off(int level) {
    return level == 1 ? 0 : level == 2 ? kCap / 2 : level == 3 ? 3 * kCap / 4 : 7 * kCap / 8;
  }
  __host__ __device__ static constexpr int cap(int level) { return level == 1 ? kCap / 2 : level == 2 ? kCap / 4 : kCap / 8; }
  int count[4];         // entries pushed per level (may exceed the capacity: the excess was not stored)
  int64_t xoff[kCap];   // element offset of the source vector
  uint8_t* tok[kCap];   // token-block base of the destination
  uint32_t meta[kCap];  // token-in-block | blk << 6 | level << 9 | j << 12 | (1 = value, 0 = key) << 15
};
using FixQueue = FixQueueT<1024>;

// True if some region is 3/4 full (or has overflowed).
template <class Q>
__device__ __forceinline__ bool fix_should_drain(const Q* q) {
  return q->count[0] > 3 * Q::cap(1) / 4 || q->count[1] > 3 * Q::cap(2) / 4 || q->count[2] > 3 * Q::cap(3) / 4 ||
         q->count[3] > 3 * Q::cap(4) / 4;
}

// Replace `width` bits at bit offset `bit` of the byte at `addr`.
__device__ __forceinline__ void patch_bits(uint8_t* addr, int bit, uint32_t mask, uint32_t code) {
  uint32_t* word = reinterpret_cast<uint32_t*>(reinterpret_cast<uintptr_t>(addr) & ~(uintptr_t)3);
  const int sh = (int)(reinterpret_cast<uintptr_t>(addr) & 3) * 8 + bit;
  atomicAnd(word, ~(mask << sh));
  atomicOr(word, code << sh);
}

template <class Q>
__device__ __forceinline__ void fix_push(Q* q, uint32_t amb, int64_t xoff, uint8_t* tokblock, int tok, int blk,
                                         int kv, uint32_t* left) {
  uint32_t rest = 0;
  while (amb) {
    const int bit = __ffs(amb) - 1;
    amb &= amb - 1;
    int level, j;
    if (bit < 8) { level = 1; j = bit; }
    else if (bit < 12) { level = 2; j = bit - 8; }
    else if (bit < 14) { level = 3; j = bit - 12; }
    else { level = 4; j = 0; }
    const int idx = atomicAdd(&q->count[level - 1], 1);
    if (idx >= Q::cap(level)) {  // this level's region is full: keep the decision for the next round
      rest |= 1u << bit;
      continue;
    }
    const int e = Q::off(level) + idx;
    q->xoff[e] = xoff;
    q->tok[e] = tokblock;
    q->meta[e] = (uint32_t)tok | ((uint32_t)blk << 6) | ((uint32_t)level << 9) | ((uint32_t)j << 12) | ((uint32_t)kv << 15);
  }
  *left = rest;
}

// Exact value of NC consecutive rotated coordinates starting at column c0, for the 8-lane group of
// this lane: each lane owns 16 consecutive k, NC independent float64 chains, then a 3-step
// butterfly inside the group.  Every lane of the group returns all NC sums.
template <int NC>
__device__ __forceinline__ void exact_coords(const double* xk, const float* S, int sub, int c0, unsigned gmask, double* y) {
  double acc[NC];
#pragma unroll
  for (int c = 0; c < NC; ++c) acc[c] = 0.0;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float* srow = S + (16 * sub + i) * 128 + c0;
    if (NC == 2) {
      const float2 s2 = __ldg(reinterpret_cast<const float2*>(srow));
      acc[0] = fma(xk[i], (double)s2.x, acc[0]);
      acc[1] = fma(xk[i], (double)s2.y, acc[1]);
    } else {
#pragma unroll
      for (int c4 = 0; c4 < NC / 4; ++c4) {
        const float4 s4 = __ldg(reinterpret_cast<const float4*>(srow) + c4);
        acc[4 * c4] = fma(xk[i], (double)s4.x, acc[4 * c4]);
        acc[4 * c4 + 1] = fma(xk[i], (double)s4.y, acc[4 * c4 + 1]);
        acc[4 * c4 + 2] = fma(xk[i], (double)s4.z, acc[4 * c4 + 2]);
        acc[4 * c4 + 3] = fma(xk[i], (double)s4.w, acc[4 * c4 + 3]);
      }
    }
  }
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    double p = acc[c];
    p += __shfl_xor_sync(gmask, p, 1);
    p += __shfl_xor_sync(gmask, p, 2);
    p += __shfl_xor_sync(gmask, p, 4);
    y[c] = p;
  }
}

// The same sums with S staged in shared memory as float64 (no conversions, no L2 latency in the loop; on this
// GPU a warp-wide float64 FMA occupies its pipe for 16 cycles, so the loop should hold nothing else that is slow).
// Row k of S sits at row (k & 15) * 8 + (k >> 4) of `Sd`, rows kFixSdStride doubles apart, so the eight lanes of a
// group (k = 16 * sub + i) read eight consecutive rows: 16-byte loads without bank conflicts.
constexpr int kFixSdStride = 130;
constexpr int kFixSdBytes = 128 * kFixSdStride * 8;
__host__ __device__ constexpr int fix_sd_row(int k) { return (k & 15) * 8 + (k >> 4); }
template <int NC>
__device__ __forceinline__ void exact_coords_sm(const double* xk, const double* Sd, int sub, int c0, unsigned gmask,
                                                double* y) {
  double acc[NC];
#pragma unroll
  for (int c = 0; c < NC; ++c) acc[c] = 0.0;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const double2* srow = reinterpret_cast<const double2*>(Sd + (i * 8 + sub) * kFixSdStride + c0);
#pragma unroll
    for (int c2 = 0; c2 < NC / 2; ++c2) {
      const double2 s2 = srow[c2];
      acc[2 * c2] = fma(xk[i], s2.x, acc[2 * c2]);
      acc[2 * c2 + 1] = fma(xk[i], s2.y, acc[2 * c2 + 1]);
    }
  }
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    double p = acc[c];
    p += __shfl_xor_sync(gmask, p, 1);
    p += __shfl_xor_sync(gmask, p, 2);
    p += __shfl_xor_sync(gmask, p, 4);
    y[c] = p;
  }
}

// Decision of one angle of level log2(NC) from the exact coordinates under it.  Levels >= 2 compare
// the squared child radii, sb > tan^2(beta) sa, which is the same decision as atan2(r_b, r_a) > beta.
template <int NC>
__device__ __forceinline__ uint32_t exact_code(const double* y, int level, const Tables& tb) {
  if (NC == 2) return quant_level1_exact(y[0], y[1], tb);
  double sa = 0.0, sb = 0.0;
#pragma unroll
  for (int c = 0; c < NC / 2; ++c) {
    sa = fma(y[c], y[c], sa);
    sb = fma(y[NC / 2 + c], y[NC / 2 + c], sb);
  }
  const double* T = tb.bnd_tan2 + 3 * (level - 2);
  return (uint32_t)(sb > T[0] * sa) + (uint32_t)(sb > T[1] * sa) + (uint32_t)(sb > T[2] * sa);
}

// Process everything queued, in level order: called by `n_threads` threads (a multiple of 32) with linear index `t`.
// `q` points to `n_queues` queues laid out back to back; their entries are taken level by level.
// `Sd` (may be null) is the float64 copy of S in shared memory for exact_coords_sm.
template <class Q>
__device__ inline void fix_process(const Q* q, int n_queues, int t, int n_threads, const void* kbase, const void* vbase,
                                   int in_dtype, const float* S, const double* Sd, const Tables& tb, int32_t* status) {
  constexpr int o2 = 32 * kTokenBlock, o3 = o2 + 8 * kTokenBlock, o4 = o3 + 4 * kTokenBlock;
  const int sub = t & 7, n_groups = n_threads >> 3;
  const unsigned gmask = 0xFFu << (t & 24);
  int n = 0;
  for (int level = 1; level <= 4; ++level)
    for (int k = 0; k < n_queues; ++k) n += min(q[k].count[level - 1], Q::cap(level));
  int fixed = 0;
  // entry i of the level-major order: which queue, which slot of it
  auto entry_of = [&](int i, const Q** which) {
    int base = 0;
    for (int level = 1; level <= 4; ++level)
      for (int k = 0; k < n_queues; ++k) {
        const int cnt = min(q[k].count[level - 1], Q::cap(level));
        if (i < base + cnt) {
          *which = q + k;
          return Q::off(level) + (i - base);
        }
        base += cnt;
      }
    *which = q;
    return 0;
  };
  // The source vector of the group's next entry is fetched while the current one is decided.
  auto fetch = [&](int i, uint4* raw) {
    if (i >= n || in_dtype != PQ_DTYPE_BF16) return;
    const Q* qe;
    const int e = entry_of(i, &qe);
    const void* xbase = (qe->meta[e] >> 15) & 1 ? vbase : kbase;
    const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(xbase) + qe->xoff[e] + 16 * sub);
    raw[0] = __ldg(p);
    raw[1] = __ldg(p + 1);
  };
  uint4 raw[2] = {make_uint4(0u, 0u, 0u, 0u), make_uint4(0u, 0u, 0u, 0u)};
  fetch(t >> 3, raw);
  for (int i = t >> 3; i < n; i += n_groups) {  // uniform within a group of 8 lanes
    const Q* qe;
    const int e = entry_of(i, &qe);
    const uint32_t meta = qe->meta[e];
    const int tok = meta & 63, blk = (meta >> 6) & 7, level = (meta >> 9) & 7, j = (meta >> 12) & 7;
    const int c0 = blk * 16 + (j << level);
    double xk[16];  // this lane's 16 consecutive k
    if (in_dtype == PQ_DTYPE_BF16) {
      const uint32_t w[8] = {raw[0].x, raw[0].y, raw[0].z, raw[0].w, raw[1].x, raw[1].y, raw[1].z, raw[1].w};
#pragma unroll
      for (int i2 = 0; i2 < 8; ++i2) {
        xk[2 * i2] = (double)__uint_as_float(w[i2] << 16);
        xk[2 * i2 + 1] = (double)__uint_as_float(w[i2] & 0xFFFF0000u);
      }
      fetch(i + n_groups, raw);
    } else {
      const void* xbase = (meta >> 15) & 1 ? vbase : kbase;
      const float* p = reinterpret_cast<const float*>(xbase) + qe->xoff[e] + 16 * sub;
#pragma unroll
      for (int i2 = 0; i2 < 16; ++i2) xk[i2] = (double)p[i2];
    }
    double y[16];
    uint32_t code;
    if (Sd != nullptr) {  // uniform over the CTA
      if (level == 1) {
        exact_coords_sm<2>(xk, Sd, sub, c0, gmask, y);
        code = exact_code<2>(y, level, tb);
      } else if (level == 2) {
        exact_coords_sm<4>(xk, Sd, sub, c0, gmask, y);
        code = exact_code<4>(y, level, tb);
      } else if (level == 3) {
        exact_coords_sm<8>(xk, Sd, sub, c0, gmask, y);
        code = exact_code<8>(y, level, tb);
      } else {
        exact_coords_sm<16>(xk, Sd, sub, c0, gmask, y);
        code = exact_code<16>(y, level, tb);
      }
    } else if (level == 1) {
      exact_coords<2>(xk, S, sub, c0, gmask, y);
      code = exact_code<2>(y, level, tb);
    } else if (level == 2) {
      exact_coords<4>(xk, S, sub, c0, gmask, y);
      code = exact_code<4>(y, level, tb);
    } else if (level == 3) {
      exact_coords<8>(xk, S, sub, c0, gmask, y);
      code = exact_code<8>(y, level, tb);
    } else {
      exact_coords<16>(xk, S, sub, c0, gmask, y);
      code = exact_code<16>(y, level, tb);
    }
    if (sub == 0) {
      uint8_t* tbk = qe->tok[e];
      if (level == 1) patch_bits(tbk + tok * 32 + blk * 4 + (j >> 1), 4 * (j & 1), 0xFu, code);
      else if (level == 2) patch_bits(tbk + o2 + tok * 8 + blk, 2 * j, 3u, code);
      else if (level == 3) patch_bits(tbk + o3 + tok * 4 + (blk >> 1), 4 * (blk & 1) + 2 * j, 3u, code);
      else patch_bits(tbk + o4 + tok * 2 + (blk >> 2), 2 * (blk & 3), 3u, code);
      ++fixed;
    }
  }
  if (fixed) atomicAdd(status + 3, fixed);
}

}  // namespace pq
