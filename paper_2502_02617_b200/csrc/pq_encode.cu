// KV-cache encoder (Algorithm 1 lines 2 and 4 with fixed codebooks) and the append step.
#include <math_constants.h>

#include "pq_common.cuh"

namespace pq {

// Where the vectors of an encode call come from and go to.
struct EncodeArgs {
  const void* K;
  const void* V;
  int in_dtype;
  int64_t token_stride, head_stride;
  const int32_t* cu_seqlens;  // nullptr: one row per sequence (append)
  int batch;
  int total_tokens;
  int n_kv_heads;
  int head_dim;
  int capacity;
  const float* S;
  const Tables* tables;
  uint8_t* cache;
  const int32_t* cache_lens;
  int32_t* status;
  uint32_t debug;  // bit 0: test hook, the first bounded wait of CTA 0 of the tensor-core kernel reports failure
  // angle histograms (pq_angle_histograms) instead of codes: uint64 [4 levels][n_bins], added to
  unsigned long long* hist;
  int n_bins;
  Paging pg;  // where the cache's token-blocks live; `capacity` = pg.pages_per_seq * pg.page_tokens
};

__device__ inline float load_elem(const void* base, int dtype, int64_t idx) {
  if (dtype == PQ_DTYPE_BF16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(base)[idx]);
  return reinterpret_cast<const float*>(base)[idx];
}

// Sequence that owns packed row `row` (largest b with cu[b] <= row).
__device__ inline int find_sequence(const int32_t* cu, int batch, int row) {
  int lo = 0, hi = batch - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (cu[mid] <= row) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Destination of packed row `row`: sequence and cache position, or pos = -1 if the sequence
// would overflow the capacity (nothing of it is written).
template <bool kMayBePaged = true>
__device__ inline void row_destination(const EncodeArgs& a, int row, int* seq, int* pos) {
  int b, first, count;
  if (a.cu_seqlens == nullptr) {
    b = row; first = row; count = 1;
  } else {
    b = find_sequence(a.cu_seqlens, a.batch, row);
    first = a.cu_seqlens[b];
    count = a.cu_seqlens[b + 1] - first;
  }
  const int start = a.cache_lens[b];
  *seq = b;
  if (start < 0 || start + count > a.capacity) {
    set_status(a.status, PQ_ERR_CAPACITY);
    *pos = -1;
  } else {
    *pos = start + (row - first);
    // a page outside the pool: nothing of the row is written
    if (kMayBePaged && a.pg.table != nullptr && block_offset_paged(0, 0, a.pg.table, a.pg.page_tokens, a.pg.pages_per_seq, a.pg.n_pages, 0, b, 0, 0,
                                                    *pos) < 0) {
      set_status(a.status, PQ_ERR_INVALID_ARG);
      *pos = -1;
    }
  }
}

// Store the codes and radius of block `blk` of the token at `pos_in_block` of a token-block.
// Lanes of a warp that hold the nb blocks of one vector are consecutive and aligned, so the
// level-3 / level-4 bit fields of a token are merged with shuffles before the byte store.
__device__ inline void store_block(uint8_t* tb_base, const Layout& L, int tok, int blk, const BlockCodes& c,
                                   __half radius, bool valid) {
  const unsigned full = 0xffffffffu;
  // level 3: 4 bits per block, two blocks per byte
  uint32_t l3 = c.l3;
  if (L.nb >= 2) {
    const uint32_t other = __shfl_down_sync(full, l3, 1);
    l3 |= other << 4;
  }
  // level 4: 2 bits per block, four blocks per byte
  uint32_t l4 = c.l4;
  if (L.nb >= 2) l4 |= __shfl_down_sync(full, l4, 1) << 2;
  if (L.nb >= 4) l4 |= __shfl_down_sync(full, l4, 2) << 4;
  if (!valid) return;
  *reinterpret_cast<uint32_t*>(tb_base + tok * L.b1 + blk * 4) = c.l1;
  tb_base[L.o2 + tok * L.b2 + blk] = (uint8_t)c.l2;
  if (L.nb < 2 || (blk & 1) == 0) tb_base[L.o3 + tok * L.b3 + (blk >> 1)] = (uint8_t)l3;
  if (L.nb < 4 || (blk & 3) == 0) tb_base[L.o4 + tok * L.b4 + (blk >> 2)] = (uint8_t)l4;
  reinterpret_cast<__half*>(tb_base + L.orad + tok * L.br)[blk] = radius;
}

// ------------------------------------------------------------------------------------------
// Reference-precision encoder: everything in float64.  One CTA of 128 threads handles
// 16 * (128 / d) vectors: thread (group, j) forms coordinate j of y = x . S for the 16 vectors
// of its group, then every thread quantises one 16-coordinate block.
// A "vector" is (row, kv, head): index v = (row * 2 + kv) * n_kv_heads + head.
// ------------------------------------------------------------------------------------------
constexpr int kExactThreads = 128;
constexpr int kExactVecPerGroup = 16;

__global__ void __launch_bounds__(kExactThreads) encode_exact_kernel(EncodeArgs a) {
  extern __shared__ double smem_d[];
  const int d = a.head_dim;
  const int groups = kExactThreads / d;
  const int vec_per_cta = kExactVecPerGroup * groups;
  double* xs = smem_d;                     // [vec_per_cta][d]
  double* ys = smem_d + vec_per_cta * d;   // [vec_per_cta][d]
  const int64_t n_vec = (int64_t)a.total_tokens * 2 * a.n_kv_heads;
  const int64_t v0 = (int64_t)blockIdx.x * vec_per_cta;
  const int tid = threadIdx.x;
  const Layout L = make_layout(d, a.pg.page_tokens);

  int bad = 0;
  for (int i = tid; i < vec_per_cta * d; i += kExactThreads) {
    const int64_t v = v0 + i / d;
    double x = 0.0;
    if (v < n_vec) {
      const int head = (int)(v % a.n_kv_heads);
      const int kv = (int)((v / a.n_kv_heads) & 1);
      const int64_t row = v / (2 * a.n_kv_heads);
      const float f = load_elem(kv ? a.V : a.K, a.in_dtype, row * a.token_stride + head * a.head_stride + (i % d));
      if (!isfinite(f)) ++bad;
      x = (double)f;
    }
    xs[i] = x;
  }
  if (bad) {
    atomicAdd(a.status + 1, bad);
    set_status(a.status, PQ_ERR_NONFINITE);
  }
  __syncthreads();

  {
    const int grp = tid / d, j = tid % d;
    double acc[kExactVecPerGroup];
#pragma unroll
    for (int i = 0; i < kExactVecPerGroup; ++i) acc[i] = 0.0;
    const double* xg = xs + grp * kExactVecPerGroup * d;
    for (int k = 0; k < d; ++k) {
      const double s = (double)a.S[k * d + j];
#pragma unroll
      for (int i = 0; i < kExactVecPerGroup; ++i) acc[i] = fma(xg[i * d + k], s, acc[i]);
    }
#pragma unroll
    for (int i = 0; i < kExactVecPerGroup; ++i) ys[(grp * kExactVecPerGroup + i) * d + j] = acc[i];
  }
  __syncthreads();

  {
    const int nb = L.nb;
    const int lv = tid / nb, blk = tid % nb;  // local vector, block
    const int64_t v = v0 + lv;
    bool valid = v < n_vec;
    BlockCodes c = {0, 0, 0, 0};
    double radius = 0.0;
    int seq = 0, pos = -1, head = 0, kv = 0;
    if (valid) {
      head = (int)(v % a.n_kv_heads);
      kv = (int)((v / a.n_kv_heads) & 1);
      row_destination(a, (int)(v / (2 * a.n_kv_heads)), &seq, &pos);
      valid = pos >= 0;
    }
    if (valid) {
      double y[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) y[i] = ys[lv * d + blk * 16 + i];
      radius = polar_quant_block_exact(y, *a.tables, c);
      if (radius > 65504.0) {
        radius = 65504.0;
        atomicAdd(a.status + 2, 1);
      }
    }
    uint8_t* tb_base = a.cache + (valid ? block_offset(L, a.pg, a.n_kv_heads, seq, head, kv, pos) : 0);
    store_block(tb_base, L, valid ? pos % kTokenBlock : 0, blk, c, __double2half(radius), valid);
  }
}

}  // namespace pq
#include "pq_encode_fast.cuh"
namespace pq {

// ------------------------------------------------------------------------------------------
// head_dim 128, float32 rotation on the FMA pipe + the fast quantiser.  One CTA = 128 consecutive
// rows of one (K|V, head); thread (row, half) owns 64 rotated coordinates (4 blocks) of its row.
// ------------------------------------------------------------------------------------------
constexpr int kFfmaThreads = 256;
constexpr int kFfmaSmem = (128 * 129 + 2 * 128) * 4 + kFastQuantBytes + (int)sizeof(FixQueue);

// Write the four blocks [4*half, 4*half+4) of the token at `pos`.
__device__ __forceinline__ void store_half_token(uint8_t* tb, int tok, int half, const FastBlock* fb, int32_t* status) {
  constexpr int o2 = 32 * kTokenBlock, o3 = o2 + 8 * kTokenBlock, o4 = o3 + 4 * kTokenBlock, orad = o4 + 2 * kTokenBlock;
  *reinterpret_cast<uint4*>(tb + tok * 32 + half * 16) = make_uint4(fb[0].l1, fb[1].l1, fb[2].l1, fb[3].l1);
  *reinterpret_cast<uint32_t*>(tb + o2 + tok * 8 + half * 4) = fb[0].l2 | (fb[1].l2 << 8) | (fb[2].l2 << 16) | (fb[3].l2 << 24);
  *reinterpret_cast<uint16_t*>(tb + o3 + tok * 4 + half * 2) =
      (uint16_t)(fb[0].l3 | (fb[1].l3 << 4) | (fb[2].l3 << 8) | (fb[3].l3 << 12));
  tb[o4 + tok * 2 + half] = (uint8_t)(fb[0].l4 | (fb[1].l4 << 2) | (fb[2].l4 << 4) | (fb[3].l4 << 6));
  int sat = 0;
  __half r[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float v = fb[i].radius;
    if (v > 65504.f) { v = 65504.f; ++sat; }
    r[i] = __float2half_rn(v);
  }
  *reinterpret_cast<uint2*>(tb + orad + tok * 16 + half * 8) = *reinterpret_cast<uint2*>(r);
  if (sat) atomicAdd(status + 2, sat);
}

// Quantise and store the 4 blocks of (row, half) whose rotated coordinates are y[64]; ambiguous
// decisions go to the fix-up queue.  Returns the ambiguity bits that did not fit (4 x 15 bits).
__device__ __forceinline__ void quantise_and_store(const EncodeArgs& a, const FastQuant& fq, const float* y,
                                                   float row_norm, int row, int head, int kv, int half, bool valid,
                                                   FixQueue* q, uint32_t* left, int64_t* xoff_out, uint8_t** tb_out,
                                                   int* tok_out) {
  const RowMargins rm = make_row_margins(row_norm, kRotErr, fq);
  FastBlock fb[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (fq.analytic) polar_quant_block_fast<true>(y + 16 * i, rm, fq, &fb[i]);
    else polar_quant_block_fast<false>(y + 16 * i, rm, fq, &fb[i]);
    left[i] = 0u;
  }
  *tb_out = nullptr;
  if (!valid) return;
  int seq, pos;
  row_destination(a, row, &seq, &pos);
  if (pos < 0) return;
  const Layout L = make_layout(128, a.pg.page_tokens);
  uint8_t* tb = a.cache + block_offset(L, a.pg, a.n_kv_heads, seq, head, kv, pos);
  store_half_token(tb, pos % kTokenBlock, half, fb, a.status);
  *xoff_out = (int64_t)row * a.token_stride + (int64_t)head * a.head_stride;
  *tb_out = tb;
  *tok_out = pos % kTokenBlock;
#pragma unroll
  for (int i = 0; i < 4; ++i) left[i] = fb[i].amb;
}

// Named-barrier OR over `n_threads` threads (also a barrier).
__device__ __forceinline__ bool bar_or(int bar_id, int n_threads, bool v) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.or.pred p, %2, %3, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out)
      : "r"((uint32_t)v), "r"(bar_id), "r"(n_threads)
      : "memory");
  return out != 0;
}

// Drain the queue of ambiguous decisions: rounds of (barrier, process, barrier, reset, push what did
// not fit before).  All `n_threads` threads of named barrier `bar_id` call this together.
// `left` holds this thread's decisions that found the queue full: 15 bits per block, four blocks per
// word, starting at block `blk0`; it is all zero on return.
template <class Q, int kWords>
__device__ inline void fix_rounds(const EncodeArgs& a, Q* q, unsigned long long (&left)[kWords], int64_t xoff, uint8_t* tb,
                                  int tok, int blk0, int kv, int t, int n_threads, int bar_id,
                                  const double* Sd = nullptr) {
  for (int round = 0; round < 4096; ++round) {
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(n_threads) : "memory");
    fix_process(q, 1, t, n_threads, a.K, a.V, a.in_dtype, a.S, Sd, *a.tables, a.status);
    asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(n_threads) : "memory");
    if (t < 4) q->count[t] = 0;
    bool mine = false;
#pragma unroll
    for (int w = 0; w < kWords; ++w) mine = mine || left[w] != 0ull;
    const bool more = bar_or(bar_id, n_threads, mine);
    if (!more) break;
    if (mine && tb != nullptr) {
#pragma unroll
      for (int w = 0; w < kWords; ++w)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t bits = (uint32_t)(left[w] >> (15 * i)) & 0x7FFFu;
          if (bits) {
            uint32_t rest;
            fix_push(q, bits, xoff, tb, tok, blk0 + 4 * w + i, kv, &rest);
            left[w] = (left[w] & ~(0x7FFFull << (15 * i))) | ((unsigned long long)rest << (15 * i));
          }
        }
    }
  }
}

__global__ void __launch_bounds__(kFfmaThreads) encode_ffma_kernel(EncodeArgs a) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the length update may be set up (it waits for this grid)
  extern __shared__ __align__(16) float smem_f[];
  float* xT = smem_f;                  // [128 k][129]
  float* rowsq = smem_f + 128 * 129;   // [2][128]
  FastQuant* fq = reinterpret_cast<FastQuant*>(rowsq + 256);
  FixQueue* fixq = reinterpret_cast<FixQueue*>(rowsq + 256 + kFastQuantBytes / 4);
  const int tid = threadIdx.x, head = blockIdx.y, kv = blockIdx.z;
  const int row0 = blockIdx.x * 128;
  const void* xbase = kv ? a.V : a.K;
  int bad = 0;
  for (int idx = tid; idx < 128 * 128; idx += kFfmaThreads) {
    const int r = idx >> 7, k = idx & 127;
    float f = 0.f;
    if (row0 + r < a.total_tokens) {
      f = load_elem(xbase, a.in_dtype, (int64_t)(row0 + r) * a.token_stride + (int64_t)head * a.head_stride + k);
      if (!isfinite(f)) ++bad;
    }
    xT[k * 129 + r] = f;
  }
  if (bad) {
    atomicAdd(a.status + 1, bad);
    set_status(a.status, PQ_ERR_NONFINITE);
  }
  if (tid == 0) {
    load_fast_quant(a.tables, fq);
    fixq->count[0] = fixq->count[1] = fixq->count[2] = fixq->count[3] = 0;
  }
  __syncthreads();
  const int r = tid & 127, half = tid >> 7;
  float y[64];
#pragma unroll
  for (int i = 0; i < 64; ++i) y[i] = 0.f;
  const float4* S4 = reinterpret_cast<const float4*>(a.S) + half * 16;
  for (int k = 0; k < 128; ++k) {
    const float xv = xT[k * 129 + r];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float4 s = __ldg(S4 + k * 32 + i);
      y[4 * i] = fmaf(xv, s.x, y[4 * i]);
      y[4 * i + 1] = fmaf(xv, s.y, y[4 * i + 1]);
      y[4 * i + 2] = fmaf(xv, s.z, y[4 * i + 2]);
      y[4 * i + 3] = fmaf(xv, s.w, y[4 * i + 3]);
    }
  }
  float sq = 0.f;
#pragma unroll
  for (int i = 0; i < 64; ++i) sq = fmaf(y[i], y[i], sq);
  rowsq[half * 128 + r] = sq;
  __syncthreads();
  const float row_norm = sqrtf(rowsq[r] + rowsq[128 + r]) * 1.0001f;
  uint32_t left[4];
  int64_t xoff = 0;
  uint8_t* tb = nullptr;
  int tok = 0;
  quantise_and_store(a, *fq, y, row_norm, row0 + r, head, kv, half, row0 + r < a.total_tokens, fixq, left, &xoff,
                     &tb, &tok);
  unsigned long long leftbits[1] = {0ull};
  if (tb != nullptr) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t rest = 0;
      if (left[i]) fix_push(fixq, left[i], xoff, tb, tok, 4 * half + i, kv, &rest);
      leftbits[0] |= (unsigned long long)rest << (15 * i);
    }
  }
  fix_rounds(a, fixq, leftbits, xoff, tb, tok, 4 * half, kv, tid, kFfmaThreads, 1);
}

// ------------------------------------------------------------------------------------------
// Few vectors (append, short chunks), head_dim 128: one CTA of 128 threads per vector.  Thread j
// forms y_j in float32; eight threads quantise one block each with the certified sign tests; if
// any decision of the vector is ambiguous the CTA forms y again in float64 and those blocks are
// decided exactly.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) encode_vector_kernel(EncodeArgs a) {
  // a programmatic dependent of the kernel before it (which may have produced the vectors, or still reads the lengths):
  // nothing of the stream is read before the wait; the length update after this grid may be set up at once
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  __shared__ float xs[128];
  __shared__ float ys[128];
  __shared__ double yd[128];
  __shared__ float red[4];
  __shared__ uint32_t amb_blocks;   // bit b: block b has a decision that float32 cannot certify
  __shared__ FastQuant fq;
  const int j = threadIdx.x;
  const int64_t v = blockIdx.x;  // vector index: (row * 2 + kv) * n_kv_heads + head
  const int head = (int)(v % a.n_kv_heads), kv = (int)((v / a.n_kv_heads) & 1);
  const int row = (int)(v / (2 * a.n_kv_heads));
  const int64_t xoff = (int64_t)row * a.token_stride + (int64_t)head * a.head_stride;
  const float xv = load_elem(kv ? a.V : a.K, a.in_dtype, xoff + j);
  if (!isfinite(xv)) {
    atomicAdd(a.status + 1, 1);
    set_status(a.status, PQ_ERR_NONFINITE);
  }
  xs[j] = xv;
  if (j == 0) {
    load_fast_quant(a.tables, &fq);
    amb_blocks = 0u;
  }
  __syncthreads();
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
  for (int k = 0; k < 128; k += 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] = fmaf(xs[k + i], __ldg(a.S + (k + i) * 128 + j), acc[i]);
  }
  const float y = (acc[0] + acc[1]) + (acc[2] + acc[3]);
  ys[j] = y;
  float sq = y * y;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  if ((j & 31) == 0) red[j >> 5] = sq;
  __syncthreads();
  // four independent partial sums instead of one chain: the bound of a 128-term float32 dot product still holds
  const float norm = 1.0001f * sqrtf((red[0] + red[1]) + (red[2] + red[3]));
  FastBlock fb = {0u, 0u, 0u, 0u, 0u, 0.f};
  if (j < 8) {
    float yb[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) yb[i] = ys[16 * j + i];
    if (fq.analytic) polar_quant_block_fast<true>(yb, make_row_margins(norm, kRotErr, fq), fq, &fb);
    else polar_quant_block_fast<false>(yb, make_row_margins(norm, kRotErr, fq), fq, &fb);
  }
  if (fb.amb != 0u) atomicOr(&amb_blocks, 1u << j);
  if (__syncthreads_or(fb.amb != 0u)) {
    if ((amb_blocks >> (j >> 4)) & 1u) {   // only the coordinates of the blocks in question (half-warps: the float64 pipe is slow)
      double accd[4] = {0.0, 0.0, 0.0, 0.0};
      for (int k = 0; k < 128; k += 4) {
#pragma unroll
        for (int i = 0; i < 4; ++i) accd[i] = fma((double)xs[k + i], (double)__ldg(a.S + (k + i) * 128 + j), accd[i]);
      }
      yd[j] = (accd[0] + accd[1]) + (accd[2] + accd[3]);
    }
    __syncthreads();
    if (j < 8 && fb.amb != 0u) {
      double yb[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) yb[i] = yd[16 * j + i];
      BlockCodes c;
      fb.radius = (float)polar_quant_block_exact(yb, *a.tables, c);
      fb.l1 = c.l1; fb.l2 = c.l2; fb.l3 = c.l3; fb.l4 = c.l4;
      atomicAdd(a.status + 3, __popc(fb.amb));
    }
  }
  if (j >= 32) return;  // the first warp stores (lanes 0..7 hold the blocks)
  int seq = 0, pos = -1;
  if (j < 8) row_destination(a, row, &seq, &pos);
  const bool valid = j < 8 && pos >= 0;
  float rv = fb.radius;
  if (valid && rv > 65504.f) {
    rv = 65504.f;
    atomicAdd(a.status + 2, 1);
  }
  const Layout L = make_layout(128, a.pg.page_tokens);
  BlockCodes c = {fb.l1, fb.l2, fb.l3, fb.l4};
  uint8_t* tb = a.cache + (valid ? block_offset(L, a.pg, a.n_kv_heads, seq, head, kv, pos) : 0);
  store_block(tb, L, valid ? pos % kTokenBlock : 0, j & 7, c, __float2half_rn(rv), valid);
}

}  // namespace pq
#include "pq_hist.cuh"
#include "pq_encode_tc.cuh"
namespace pq {

// Angle histograms of any head_dim (multiple of 16, at most 128) and input type: 128 / head_dim vectors per CTA,
// thread = rotated coordinate in float32, then one thread per 16-block counts the block's 15 angles into the CTA's
// shared histogram.  The path of short inputs and of what the tensor-core kernel does not take.
constexpr int kHistSimpleThreads = 128;
__global__ void __launch_bounds__(kHistSimpleThreads) hist_simple_kernel(EncodeArgs a, int64_t n_vec, int vec_per_cta_step) {
  extern __shared__ uint32_t hist_s[];
  __shared__ float xs[128];
  __shared__ float ys[128];
  const int d = a.head_dim, per = 128 / d, j = threadIdx.x, vi = j / d, jj = j % d;
  for (int i = j; i < 4 * a.n_bins; i += kHistSimpleThreads) hist_s[i] = 0u;
  const float scale1 = (float)a.n_bins * 0.159154943091895336f, scale_up = (float)a.n_bins * 0.636619772367581343f;
  int bad = 0;
  for (int64_t v0 = (int64_t)blockIdx.x * per; v0 < n_vec; v0 += (int64_t)gridDim.x * per) {
    const int64_t v = v0 + vi;  // vector index: (row * 2 + kv) * n_kv_heads + head
    const bool valid = vi < per && v < n_vec;
    __syncthreads();
    if (valid) {
      const int head = (int)(v % a.n_kv_heads), kv = (int)((v / a.n_kv_heads) & 1);
      const int64_t row = v / (2 * a.n_kv_heads);
      xs[j] = load_elem(kv ? a.V : a.K, a.in_dtype, row * a.token_stride + (int64_t)head * a.head_stride + jj);
    }
    __syncthreads();
    if (valid) {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      for (int k = 0; k < d; k += 4)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[i] = fmaf(xs[vi * d + k + i], __ldg(a.S + (k + i) * d + jj), acc[i]);
      ys[j] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
    }
    __syncthreads();
    if (valid && (jj & 15) == 0) {
      float yb[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) yb[i] = ys[j + i];
      if (!hist_block(yb, hist_s, a.n_bins, scale1, scale_up)) ++bad;
    }
  }
  if (bad) {
    atomicAdd(a.status + 1, bad);
    set_status(a.status, PQ_ERR_NONFINITE);
  }
  __syncthreads();
  hist_flush(hist_s, 4 * a.n_bins, a.hist, j, kHistSimpleThreads);
}

// lens[b] += rows of sequence b (skipped for sequences that did not fit, or whose new positions reach a page outside
// the pool: rows of such a sequence that did land in good pages stay beyond its length).
__global__ void advance_lens_kernel(const int32_t* cu_seqlens, int batch, int capacity, Paging pg, int32_t* lens) {
  // This grid is launched ahead of time: wait for the encode grid (which reads the lengths) to complete.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  const int count = cu_seqlens ? cu_seqlens[b + 1] - cu_seqlens[b] : 1;
  const int start = lens[b];
  if (start < 0 || start + count > capacity || count <= 0) return;
  if (pg.table != nullptr)
    for (int p = start / pg.page_tokens; p <= (start + count - 1) / pg.page_tokens; ++p)
      if ((unsigned)pg.table[(int64_t)b * pg.pages_per_seq + p] >= (unsigned)pg.n_pages) return;
  lens[b] = start + count;
}

static int32_t check_common(int head_dim, int n_kv_heads, const void* S, const void* tables, const void* cache,
                            const void* lens, const void* status) {
  if (!(head_dim == 16 || head_dim == 32 || head_dim == 64 || head_dim == 128)) return PQ_ERR_UNSUPPORTED;
  if (n_kv_heads <= 0 || !S || !tables || !cache || !lens || !status) return PQ_ERR_INVALID_ARG;
  const uintptr_t bits = (uintptr_t)S | (uintptr_t)tables | (uintptr_t)cache;
  if (bits & 15) return PQ_ERR_ALIGNMENT;
  if (((uintptr_t)lens | (uintptr_t)status) & 3) return PQ_ERR_ALIGNMENT;
  return PQ_OK;
}

// The length update as a programmatic dependent launch of the encode kernel before it (which allows it with
// griddepcontrol.launch_dependents): set up while that grid runs, started when it has completed.
static int32_t launch_advance_lens(const EncodeArgs& a, int32_t* lens, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((a.batch + 127) / 128);
  cfg.blockDim = dim3(128);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, advance_lens_kernel, a.cu_seqlens, a.batch, a.capacity, a.pg, lens) != cudaSuccess) {
    cudaGetLastError();
    return PQ_ERR_CUDA;
  }
  return launch_status();
}

static int32_t launch_encode(EncodeArgs a, int32_t* lens, cudaStream_t stream) {
  if (a.total_tokens == 0) return PQ_OK;
  {
    const int32_t tc = try_launch_encode_tc(a, stream);
    if (tc < 0) return tc;
    if (tc == 1) return launch_advance_lens(a, lens, stream);
  }
  if (a.head_dim == 128 && a.total_tokens < 32) {
    const int64_t n_vec = (int64_t)a.total_tokens * 2 * a.n_kv_heads;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_vec);
    cfg.blockDim = dim3(128);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];   // may be set up while the kernel before it in the stream finishes (it waits inside)
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, encode_vector_kernel, a) != cudaSuccess) {
      cudaGetLastError();
      return PQ_ERR_CUDA;
    }
    return launch_advance_lens(a, lens, stream);
  }
  if (a.head_dim == 128 && a.total_tokens >= 32) {
    static DeviceMemo configured;
    if (configure_for_device(encode_ffma_kernel, kFfmaSmem, configured) == 0) return PQ_ERR_CUDA;
    dim3 grid((a.total_tokens + 127) / 128, a.n_kv_heads, 2);
    encode_ffma_kernel<<<grid, kFfmaThreads, kFfmaSmem, stream>>>(a);
    return launch_advance_lens(a, lens, stream);
  }
  const int groups = kExactThreads / a.head_dim;
  const int vec_per_cta = kExactVecPerGroup * groups;
  const int64_t n_vec = (int64_t)a.total_tokens * 2 * a.n_kv_heads;
  const int64_t grid = (n_vec + vec_per_cta - 1) / vec_per_cta;
  const size_t smem = (size_t)2 * vec_per_cta * a.head_dim * sizeof(double);
  encode_exact_kernel<<<(unsigned)grid, kExactThreads, smem, stream>>>(a);
  return launch_advance_lens(a, lens, stream);
}

}  // namespace pq

static int32_t encode_entry(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                            const void* K_dev, const void* V_dev, int32_t in_dtype, int64_t token_stride,
                            int64_t head_stride, const int32_t* cu_seqlens_dev, int32_t batch, int32_t total_tokens,
                            void* cache_dev, int32_t* cache_lens_dev, int32_t capacity, const pq::Paging& pg,
                            int32_t* status_dev, void* stream) {
  pq::NvtxRange nvtx_range("pq_encode_kv");
  int32_t st = pq::check_common(head_dim, n_kv_heads, S_dev, tables_dev, cache_dev, cache_lens_dev, status_dev);
  if (st != PQ_OK) return st;
  if (!K_dev || !V_dev || !cu_seqlens_dev || batch <= 0 || total_tokens < 0 || capacity <= 0) return PQ_ERR_INVALID_ARG;
  if (in_dtype != PQ_DTYPE_F32 && in_dtype != PQ_DTYPE_BF16) return PQ_ERR_UNSUPPORTED;
  if (token_stride < 0 || head_stride < 0) return PQ_ERR_INVALID_ARG;
  if ((int64_t)total_tokens * 2 * n_kv_heads >= (1ll << 31) * 16) return PQ_ERR_UNSUPPORTED;
  pq::EncodeArgs a;
  a.K = K_dev; a.V = V_dev; a.in_dtype = in_dtype;
  a.token_stride = token_stride; a.head_stride = head_stride;
  a.cu_seqlens = cu_seqlens_dev; a.batch = batch; a.total_tokens = total_tokens;
  a.n_kv_heads = n_kv_heads; a.head_dim = head_dim; a.capacity = capacity;
  a.S = S_dev; a.tables = reinterpret_cast<const pq::Tables*>(tables_dev);
  a.cache = reinterpret_cast<uint8_t*>(cache_dev); a.cache_lens = cache_lens_dev; a.status = status_dev;
  a.debug = 0u;
  a.hist = nullptr; a.n_bins = 0; a.pg = pg;
  return pq::launch_encode(a, cache_lens_dev, reinterpret_cast<cudaStream_t>(stream));
}

static int32_t append_entry(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                            const void* k_new_dev, const void* v_new_dev, int32_t in_dtype, int32_t batch,
                            void* cache_dev, int32_t* cache_lens_dev, int32_t capacity, const pq::Paging& pg,
                            int32_t* status_dev, void* stream) {
  pq::NvtxRange nvtx_range("pq_append_kv");
  int32_t st = pq::check_common(head_dim, n_kv_heads, S_dev, tables_dev, cache_dev, cache_lens_dev, status_dev);
  if (st != PQ_OK) return st;
  if (!k_new_dev || !v_new_dev || batch <= 0 || capacity <= 0) return PQ_ERR_INVALID_ARG;
  if (in_dtype != PQ_DTYPE_F32 && in_dtype != PQ_DTYPE_BF16) return PQ_ERR_UNSUPPORTED;
  pq::EncodeArgs a;
  a.K = k_new_dev; a.V = v_new_dev; a.in_dtype = in_dtype;
  a.token_stride = (int64_t)n_kv_heads * head_dim; a.head_stride = head_dim;
  a.cu_seqlens = nullptr; a.batch = batch; a.total_tokens = batch;
  a.n_kv_heads = n_kv_heads; a.head_dim = head_dim; a.capacity = capacity;
  a.S = S_dev; a.tables = reinterpret_cast<const pq::Tables*>(tables_dev);
  a.cache = reinterpret_cast<uint8_t*>(cache_dev); a.cache_lens = cache_lens_dev; a.status = status_dev;
  a.debug = 0u;
  a.hist = nullptr; a.n_bins = 0; a.pg = pg;
  return pq::launch_encode(a, cache_lens_dev, reinterpret_cast<cudaStream_t>(stream));
}

extern "C" {

int32_t pq_encode_kv(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                     const void* K_dev, const void* V_dev, int32_t in_dtype, int64_t token_stride,
                     int64_t head_stride, const int32_t* cu_seqlens_dev, int32_t batch, int32_t total_tokens,
                     void* cache_dev, int32_t* cache_lens_dev, int32_t capacity, int32_t* status_dev,
                     void* stream) {
  return encode_entry(head_dim, n_kv_heads, S_dev, tables_dev, K_dev, V_dev, in_dtype, token_stride, head_stride,
                      cu_seqlens_dev, batch, total_tokens, cache_dev, cache_lens_dev, capacity,
                      pq::contiguous_paging(capacity, batch), status_dev, stream);
}

int32_t pq_encode_kv_paged(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                           const void* K_dev, const void* V_dev, int32_t in_dtype, int64_t token_stride,
                           int64_t head_stride, const int32_t* cu_seqlens_dev, int32_t batch, int32_t total_tokens,
                           void* cache_dev, int32_t* cache_lens_dev, const pq_paging* paging, int32_t* status_dev,
                           void* stream) {
  pq::Paging pg;
  const int32_t st = pq::paging_from(paging, head_dim, &pg);
  if (st != PQ_OK) return st;
  return encode_entry(head_dim, n_kv_heads, S_dev, tables_dev, K_dev, V_dev, in_dtype, token_stride, head_stride,
                      cu_seqlens_dev, batch, total_tokens, cache_dev, cache_lens_dev, pg.page_tokens * pg.pages_per_seq, pg,
                      status_dev, stream);
}

int32_t pq_append_kv(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                     const void* k_new_dev, const void* v_new_dev, int32_t in_dtype, int32_t batch,
                     void* cache_dev, int32_t* cache_lens_dev, int32_t capacity, int32_t* status_dev,
                     void* stream) {
  return append_entry(head_dim, n_kv_heads, S_dev, tables_dev, k_new_dev, v_new_dev, in_dtype, batch, cache_dev,
                      cache_lens_dev, capacity, pq::contiguous_paging(capacity, batch), status_dev, stream);
}

int32_t pq_append_kv_paged(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                           const void* k_new_dev, const void* v_new_dev, int32_t in_dtype, int32_t batch,
                           void* cache_dev, int32_t* cache_lens_dev, const pq_paging* paging, int32_t* status_dev,
                           void* stream) {
  pq::Paging pg;
  const int32_t st = pq::paging_from(paging, head_dim, &pg);
  if (st != PQ_OK) return st;
  return append_entry(head_dim, n_kv_heads, S_dev, tables_dev, k_new_dev, v_new_dev, in_dtype, batch, cache_dev,
                      cache_lens_dev, pg.page_tokens * pg.pages_per_seq, pg, status_dev, stream);
}

int32_t pq_angle_histograms(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* K_dev,
                            const void* V_dev, int32_t in_dtype, int64_t token_stride, int64_t head_stride,
                            int32_t total_tokens, int32_t n_bins, uint64_t* hist_dev, int32_t* status_dev, void* stream) {
  if (!(head_dim == 16 || head_dim == 32 || head_dim == 64 || head_dim == 128)) return PQ_ERR_UNSUPPORTED;
  if (n_kv_heads <= 0 || !S_dev || !K_dev || !V_dev || !hist_dev || !status_dev || total_tokens < 0) return PQ_ERR_INVALID_ARG;
  if (n_bins < 16 || n_bins > PQ_HIST_MAX_BINS) return PQ_ERR_INVALID_ARG;
  if (in_dtype != PQ_DTYPE_F32 && in_dtype != PQ_DTYPE_BF16) return PQ_ERR_UNSUPPORTED;
  if (token_stride < 0 || head_stride < 0) return PQ_ERR_INVALID_ARG;
  if ((int64_t)total_tokens * 2 * n_kv_heads >= (1ll << 31) * 16) return PQ_ERR_UNSUPPORTED;
  if (((uintptr_t)S_dev & 15) || ((uintptr_t)hist_dev & 7)) return PQ_ERR_ALIGNMENT;
  if (total_tokens == 0) return PQ_OK;
  pq::EncodeArgs a;
  a.K = K_dev; a.V = V_dev; a.in_dtype = in_dtype;
  a.token_stride = token_stride; a.head_stride = head_stride;
  a.cu_seqlens = nullptr; a.batch = 0; a.total_tokens = total_tokens;
  a.n_kv_heads = n_kv_heads; a.head_dim = head_dim; a.capacity = 0;
  a.S = S_dev; a.tables = nullptr; a.cache = nullptr; a.cache_lens = nullptr; a.status = status_dev;
  a.debug = 0u;
  a.hist = reinterpret_cast<unsigned long long*>(hist_dev); a.n_bins = n_bins;
  a.pg = pq::contiguous_paging(0, 0);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const int32_t tc = pq::try_launch_hist_tc(a, s);
  if (tc < 0) return tc;
  if (tc == 1) return pq::launch_status();
  const int per = 128 / head_dim;
  const int64_t n_vec = (int64_t)total_tokens * 2 * n_kv_heads;
  const int64_t want = (n_vec + per - 1) / per;
  const int grid = (int)(want < 148 * 8 ? want : 148 * 8);
  pq::hist_simple_kernel<<<grid, pq::kHistSimpleThreads, (size_t)4 * n_bins * sizeof(uint32_t), s>>>(a, n_vec, per);
  return pq::launch_status();
}

}  // extern "C"
