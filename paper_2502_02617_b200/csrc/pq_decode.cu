// Decode attention over the packed cache (Eq. 3) and the inspection kernels.
#include <atomic>
#include <cmath>
#include <chrono>
#include <math_constants.h>

#include "pq_common.cuh"

namespace pq {

// ---- reading codes of (token, block) from a token-block held in global or shared memory ----
__device__ inline uint32_t get_l1(const uint8_t* tb, const Layout& L, int tok, int blk) {
  return *reinterpret_cast<const uint32_t*>(tb + tok * L.b1 + blk * 4);
}
__device__ inline uint32_t get_l2(const uint8_t* tb, const Layout& L, int tok, int blk) {
  return tb[L.o2 + tok * L.b2 + blk];
}
__device__ inline uint32_t get_l3(const uint8_t* tb, const Layout& L, int tok, int blk) {
  return (tb[L.o3 + tok * L.b3 + (blk >> 1)] >> (4 * (blk & 1))) & 0xFu;
}
__device__ inline uint32_t get_l4(const uint8_t* tb, const Layout& L, int tok, int blk) {
  return (tb[L.o4 + tok * L.b4 + (blk >> 2)] >> (2 * (blk & 3))) & 0x3u;
}
__device__ inline float get_radius(const uint8_t* tb, const Layout& L, int tok, int blk) {
  return __half2float(reinterpret_cast<const __half*>(tb + L.orad + tok * L.br)[blk]);
}

// DeQuant of one block in the rotated basis (Algorithm 1, DeQuant, without the final S^T):
// from the level-4 radius down, child 2j = parent * cos(theta), child 2j+1 = parent * sin(theta).
__device__ inline void decode_block(const uint8_t* tb, const Layout& L, int tok, int blk, const float* cen_cos,
                                    const float* cen_sin, float* y) {
  const uint32_t l1 = get_l1(tb, L, tok, blk), l2 = get_l2(tb, L, tok, blk);
  const uint32_t l3 = get_l3(tb, L, tok, blk), l4 = get_l4(tb, L, tok, blk);
  const float r = get_radius(tb, L, tok, blk);
  float r3[2], r2[4], r1[8];
  r3[0] = r * cen_cos[24 + l4];
  r3[1] = r * cen_sin[24 + l4];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const uint32_t c = (l3 >> (2 * j)) & 3u;
    r2[2 * j] = r3[j] * cen_cos[20 + c];
    r2[2 * j + 1] = r3[j] * cen_sin[20 + c];
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t c = (l2 >> (2 * j)) & 3u;
    r1[2 * j] = r2[j] * cen_cos[16 + c];
    r1[2 * j + 1] = r2[j] * cen_sin[16 + c];
  }
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t c = (l1 >> (4 * j)) & 15u;
    y[2 * j] = r1[j] * cen_cos[c];
    y[2 * j + 1] = r1[j] * cen_sin[c];
  }
}

// One rotated coordinate of one token.
__device__ inline float decode_coord(const uint8_t* tb, const Layout& L, int tok, int coord, const float* cen_cos,
                                     const float* cen_sin) {
  const int blk = coord >> 4, i = coord & 15;
  const uint32_t c1 = (get_l1(tb, L, tok, blk) >> (4 * (i >> 1))) & 15u;
  const uint32_t c2 = (get_l2(tb, L, tok, blk) >> (2 * (i >> 2))) & 3u;
  const uint32_t c3 = (get_l3(tb, L, tok, blk) >> (2 * (i >> 3))) & 3u;
  const uint32_t c4 = get_l4(tb, L, tok, blk);
  float v = get_radius(tb, L, tok, blk);
  v *= (i & 8) ? cen_sin[24 + c4] : cen_cos[24 + c4];
  v *= (i & 4) ? cen_sin[20 + c3] : cen_cos[20 + c3];
  v *= (i & 2) ? cen_sin[16 + c2] : cen_cos[16 + c2];
  v *= (i & 1) ? cen_sin[c1] : cen_cos[c1];
  return v;
}

// ---- workspace -----------------------------------------------------------------------------
constexpr int kFastMaxGridHost = 160;  // upper bound on the persistent kernel's grid (one CTA per SM)

struct Workspace {
  float* qrot;       // [B][Hq][d]      rotated queries times scale*log2(e)
  __half* qrot_h;    // the same rounded to fp16 (tensor-core operand of the fast kernel)
  __half* qrot_l;    // fp16 residual: qrot - qrot_h
  int32_t* tickets;  // [B][Hkv]
  float* ml;         // [slot][head in group][2]   slot = first slot of the unit + part
  float* o;          // [slot][head in group][d]
  int n_splits;      // parts per unit of the any-head_dim kernel (the head_dim-128 kernel decides on the device)
  int n_slots;
  int64_t bytes;
};

// Token splits per (sequence, kv head) for the any-head_dim kernel.
__host__ inline int choose_splits(int d, int batch, int n_kv_heads, int max_len) {
  const int units = batch * n_kv_heads;
  const int max_blocks = (max_len + kTokenBlock - 1) / kTokenBlock;
  int splits = (148 * 4 + units - 1) / units;
  if (splits > max_blocks) splits = max_blocks;
  if (splits < 1) splits = 1;
  if (splits > 256) splits = 256;
  return splits;
}

__host__ inline Workspace carve_workspace(void* base, int d, int batch, int n_q_heads, int n_kv_heads, int max_len) {
  Workspace w;
  w.n_splits = choose_splits(d, batch, n_kv_heads, max_len);
  auto align = [](int64_t x) { return (x + 255) & ~(int64_t)255; };
  int64_t off = 0;
  uint8_t* p = reinterpret_cast<uint8_t*>(base);
  w.qrot = reinterpret_cast<float*>(p + off);
  off = align(off + (int64_t)batch * n_q_heads * d * 4);
  w.qrot_h = reinterpret_cast<__half*>(p + off);
  off = align(off + (int64_t)batch * n_q_heads * d * 2);
  w.qrot_l = reinterpret_cast<__half*>(p + off);
  off = align(off + (int64_t)batch * n_q_heads * d * 2);
  w.tickets = reinterpret_cast<int32_t*>(p + off);
  off = align(off + (int64_t)batch * n_kv_heads * 8);  // 8 bytes per unit (the persistent kernel's tagged tickets)
  const int g = n_q_heads / n_kv_heads, units = batch * n_kv_heads;
  w.n_slots = (d == 128 && units <= 2048) ? units + kFastMaxGridHost : units * w.n_splits;
  w.ml = reinterpret_cast<float*>(p + off);
  off = align(off + (int64_t)w.n_slots * g * 2 * 4);
  w.o = reinterpret_cast<float*>(p + off);
  off = align(off + (int64_t)w.n_slots * g * d * 4);
  w.bytes = off;
  return w;
}


struct DecodeArgs {
  int d, n_q_heads, n_kv_heads, batch, capacity, io_dtype;
  int n_q;  // queries per sequence (1: decode).  `batch` counts (sequence, query) pairs: q and out are
            // [batch][n_q_heads][d] with pair p = sequence * n_q + query; `lens` and the cache are per sequence.
  float scale;
  uint32_t epoch;  // differs from call to call (top bit set): tags the split tickets of the persistent kernel
  uint32_t debug;  // test hooks.  bit 0: the first bounded wait of CTA 0 of the persistent kernel reports failure;
                   // bit 1: the MMA thread of CTA (0, 0, 0) of the tcgen05 multi-query kernel reports its wait for the
                   // third decoded block (the last one of a shorter sequence) as failed
  const float* S;
  const Tables* tables;
  const void* q;
  const uint8_t* cache;
  const int32_t* lens;
  void* out;
  float* lse;  // optional [batch][n_q_heads]: natural log of the softmax denominator (for merging partial attentions);
               // with it, a sequence of length 0 is not an error (zeros and -inf)
  int32_t* status;
  Workspace ws;
  Paging pg;  // where the cache's token-blocks live
  // Sequence of (sequence, query) pair p, and the cached tokens its query sees: query j of the n_q last positions of
  // a sequence attends to the tokens before and at its own position (Section 4: the i-th query sees i tokens).
  __device__ __forceinline__ int seq_of(int p) const { return n_q == 1 ? p : p / n_q; }
  __device__ __forceinline__ int visible_len(int p) const {
    if (n_q == 1) return lens[p];
    const int b = p / n_q, v = lens[b] - (n_q - 1 - (p - b * n_q));
    return v > 0 ? v : 0;
  }
};

// q' = (q . S) * scale * log2(e); also clears the split tickets.
__global__ void rotate_query_kernel(DecodeArgs a) {
  extern __shared__ float qs[];
  const int bh = blockIdx.x, j = threadIdx.x, d = a.d;
  const int64_t base = (int64_t)bh * d;
  if (a.io_dtype == PQ_DTYPE_BF16) qs[j] = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.q)[base + j]);
  else qs[j] = reinterpret_cast<const float*>(a.q)[base + j];
  __syncthreads();
  float acc = 0.f;
#pragma unroll 16
  for (int k = 0; k < d; ++k) acc = fmaf(qs[k], __ldg(a.S + k * d + j), acc);
  acc *= a.scale * 1.4426950408889634f;
  a.ws.qrot[base + j] = acc;
  const __half qh = __float2half_rn(acc);
  a.ws.qrot_h[base + j] = qh;
  a.ws.qrot_l[base + j] = __float2half_rn(acc - __half2float(qh));
  if (bh < a.batch * a.n_kv_heads && j == 0) a.ws.tickets[bh] = 0;
}

constexpr int kSimpleThreads = 128;

// Shared memory (floats) that combine_and_store needs.
__host__ __device__ inline int combine_smem_floats(int g, int d, int n_parts) { return ((2 * g * n_parts + g + 3) & ~3) + g * d; }

// Merge the `ns` partials (slots slot0 .. slot0 + ns - 1) of the `g` query heads of (b, kv head) in slot
// order, normalise, rotate back by S^T and store.  Runs in the last CTA that finishes for this
// (b, kv head); `sm` must hold combine_smem_floats(g, d, ns) floats.  Every phase issues its global
// loads side by side (the CTA that runs this is the last one still working on the unit).
__device__ void combine_and_store(const DecodeArgs& a, int b, int hk, int g, int slot0, int ns, float* sm) {
  const int d = a.d, tid = threadIdx.x, nthr = blockDim.x;
  float* w_sm = sm;                  // [g][ns] running maximum of split s for head h, then its weight
  float* l_sm = sm + g * ns;         // [g][ns] denominator of split s for head h
  float* linv_sm = l_sm + g * ns;    // [g]
  float* o_sm = sm + ((2 * g * ns + g + 3) & ~3);  // [g][d], 16-byte aligned
  const int64_t h0 = (int64_t)b * a.n_q_heads + hk * g;
  for (int idx = tid; idx < g * ns; idx += nthr) {
    const int h = idx / ns, s = idx - h * ns;
    const float2 ml = *reinterpret_cast<const float2*>(a.ws.ml + ((int64_t)(slot0 + s) * g + h) * 2);
    w_sm[idx] = ml.x;
    l_sm[idx] = ml.y;
  }
  __syncthreads();
  if (tid < g) {
    float M = -CUDART_INF_F;
    for (int s = 0; s < ns; ++s) M = fmaxf(M, w_sm[tid * ns + s]);
    float Lsum = 0.f;
    for (int s = 0; s < ns; ++s) {  // slot order
      const float ms = w_sm[tid * ns + s];
      const float w = ms == -CUDART_INF_F ? 0.f : exp2f(ms - M);
      w_sm[tid * ns + s] = w;
      Lsum += l_sm[tid * ns + s] * w;
    }
    linv_sm[tid] = Lsum > 0.f ? 1.f / Lsum : 0.f;
    // scores are kept in the log2 domain: sum_t exp(s_t) = 2^M * Lsum
    if (a.lse != nullptr) a.lse[h0 + tid] = Lsum > 0.f ? (M + log2f(Lsum)) * 0.693147180559945309f : -CUDART_INF_F;
  }
  __syncthreads();
  for (int idx = tid; idx < g * d; idx += nthr) {
    const int h = idx / d, j = idx - h * d;
    const float* op = a.ws.o + ((int64_t)slot0 * g + h) * d + j;
    float acc = 0.f;
#pragma unroll 4
    for (int s = 0; s < ns; ++s) acc = fmaf(op[(int64_t)s * g * d], w_sm[h * ns + s], acc);
    o_sm[idx] = acc * linv_sm[h];
  }
  __syncthreads();
  // x_hat_i = sum_j y_hat_j S[i][j]: a warp takes eight rows i at a time, lanes over j (coalesced), and
  // has the loads of all eight rows in flight before the first is used.
  const int lane = tid & 31, warp = tid >> 5, nwarps = nthr >> 5;
  constexpr int kRows = 8;
  for (int i0 = warp * kRows; i0 < d; i0 += nwarps * kRows) {
    float sv[kRows][4];
#pragma unroll
    for (int r = 0; r < kRows; ++r)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int j = lane + 32 * q;
        sv[r][q] = (i0 + r < d && j < d) ? __ldg(a.S + (int64_t)(i0 + r) * d + j) : 0.f;
      }
    for (int h = 0; h < g; ++h) {
      float ov[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) ov[q] = lane + 32 * q < d ? o_sm[h * d + lane + 32 * q] : 0.f;
      float v[kRows];
#pragma unroll
      for (int r = 0; r < kRows; ++r)
        v[r] = fmaf(ov[3], sv[r][3], fmaf(ov[2], sv[r][2], fmaf(ov[1], sv[r][1], ov[0] * sv[r][0])));
      // Sum over the 32 lanes: three halving exchanges leave lane L with row L >> 2 (summed over eight
      // lanes), two more finish it.  9 shuffles per head instead of 40; the order is fixed.
      float w4[4], w2[2];
      const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
#pragma unroll
      for (int k = 0; k < 4; ++k)
        w4[k] = (b4 ? v[k + 4] : v[k]) + __shfl_xor_sync(0xffffffffu, b4 ? v[k] : v[k + 4], 16);
#pragma unroll
      for (int k = 0; k < 2; ++k)
        w2[k] = (b3 ? w4[k + 2] : w4[k]) + __shfl_xor_sync(0xffffffffu, b3 ? w4[k] : w4[k + 2], 8);
      float t = (b2 ? w2[1] : w2[0]) + __shfl_xor_sync(0xffffffffu, b2 ? w2[0] : w2[1], 4);
      t += __shfl_xor_sync(0xffffffffu, t, 2);
      t += __shfl_xor_sync(0xffffffffu, t, 1);
      const int row = i0 + (lane >> 2);
      if ((lane & 3) == 0 && row < d) {
        const int64_t oidx = (h0 + h) * d + row;
        if (a.io_dtype == PQ_DTYPE_BF16) reinterpret_cast<__nv_bfloat16*>(a.out)[oidx] = __float2bfloat16(t);
        else reinterpret_cast<float*>(a.out)[oidx] = t;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Straightforward float32 kernel: one CTA per (token split, kv head, sequence); per token-block
// (1) stage the K and V blocks in shared memory, (2) a thread per token decodes the key and
// forms the scores of the group's query heads, (3) online softmax per head, (4) a thread per
// coordinate decodes the values and accumulates.  Serves every head_dim and group size.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSimpleThreads) decode_attention_simple_kernel(DecodeArgs a) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int d = a.d, g = a.n_q_heads / a.n_kv_heads;
  const Layout L = make_layout(d, a.pg.page_tokens);
  const int split = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  uint8_t* kblk = smem;
  uint8_t* vblk = smem + L.block_bytes;
  float* qs = reinterpret_cast<float*>(smem + 2 * L.block_bytes);  // [g][d]
  float* s_part = qs + g * d;                                      // [2][g][64]
  float* p_sm = s_part + 2 * g * kTokenBlock;                      // [g][64]
  float* corr_sm = p_sm + g * kTokenBlock;                         // [g]
  float* m_run = corr_sm + kMaxGroup;                              // [g]
  float* l_run = m_run + kMaxGroup;                                // [g]
  float* cen_cos = l_run + kMaxGroup;                              // [28]
  float* cen_sin = cen_cos + 32;                                   // [28]
  __shared__ int is_last;

  for (int i = tid; i < g * d; i += kSimpleThreads) qs[i] = a.ws.qrot[((int64_t)b * a.n_q_heads + hk * g) * d + i];
  if (tid < PQ_N_CENTROIDS) {
    cen_cos[tid] = a.tables->cen_cos[tid];
    cen_sin[tid] = a.tables->cen_sin[tid];
  }
  if (tid < g) {
    m_run[tid] = -CUDART_INF_F;
    l_run[tid] = 0.f;
  }
  float o_acc[kMaxGroup];
#pragma unroll
  for (int h = 0; h < kMaxGroup; ++h) o_acc[h] = 0.f;

  const int len = a.visible_len(b);
  const int nblk_total = len > 0 ? (len + kTokenBlock - 1) / kTokenBlock : 0;
  const int per = (nblk_total + a.ws.n_splits - 1) / a.ws.n_splits;
  const int j0 = split * per;
  const int j1 = min(nblk_total, j0 + per);
  const int seq = a.seq_of(b);
  __syncthreads();

  for (int jb = j0; jb < j1; ++jb) {
    {
      const uint4* src = reinterpret_cast<const uint4*>(a.cache + kv_block_pair_offset(L, a.pg, a.n_kv_heads, seq, hk, jb, a.status));
      uint4* dst = reinterpret_cast<uint4*>(smem);
      for (int i = tid; i < 2 * L.block_bytes / 16; i += kSimpleThreads) dst[i] = src[i];
    }
    __syncthreads();
    {  // scores
      const int tk = tid & 63, half = tid >> 6;
      float s[kMaxGroup];
#pragma unroll
      for (int h = 0; h < kMaxGroup; ++h) s[h] = 0.f;
      for (int blk = half; blk < L.nb; blk += 2) {
        float y[16];
        decode_block(kblk, L, tk, blk, cen_cos, cen_sin, y);
#pragma unroll
        for (int h = 0; h < kMaxGroup; ++h) {
          if (h < g) {
            const float* qh = qs + h * d + blk * 16;
            float acc = s[h];
#pragma unroll
            for (int i = 0; i < 16; ++i) acc = fmaf(qh[i], y[i], acc);
            s[h] = acc;
          }
        }
      }
#pragma unroll
      for (int h = 0; h < kMaxGroup; ++h)
        if (h < g) s_part[(half * g + h) * kTokenBlock + tk] = s[h];
    }
    __syncthreads();
    for (int h = warp; h < g; h += kSimpleThreads / 32) {  // online softmax, one warp per head
      float sv[2], mx = -CUDART_INF_F;
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const int tk = lane + 32 * t;
        const bool ok = jb * kTokenBlock + tk < len;
        sv[t] = ok ? s_part[h * kTokenBlock + tk] + s_part[(g + h) * kTokenBlock + tk] : -CUDART_INF_F;
        mx = fmaxf(mx, sv[t]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_old = m_run[h], m_new = fmaxf(m_old, mx);
      float sum = 0.f;
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const float p = sv[t] == -CUDART_INF_F ? 0.f : exp2f(sv[t] - m_new);
        p_sm[h * kTokenBlock + lane + 32 * t] = p;
        sum += p;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (lane == 0) {
        const float corr = m_old == -CUDART_INF_F ? 0.f : exp2f(m_old - m_new);
        corr_sm[h] = corr;
        m_run[h] = m_new;
        l_run[h] = l_run[h] * corr + sum;
      }
    }
    __syncthreads();
    if (tid < d) {  // values
#pragma unroll
      for (int h = 0; h < kMaxGroup; ++h)
        if (h < g) o_acc[h] *= corr_sm[h];
      const int n_valid = min(kTokenBlock, len - jb * kTokenBlock);  // stale bytes past len may decode to NaN
      for (int tk = 0; tk < n_valid; ++tk) {
        const float v = decode_coord(vblk, L, tk, tid, cen_cos, cen_sin);
#pragma unroll
        for (int h = 0; h < kMaxGroup; ++h)
          if (h < g) o_acc[h] = fmaf(p_sm[h * kTokenBlock + tk], v, o_acc[h]);
      }
    }
    __syncthreads();
  }

  // partials of this split
  const int slot0 = (b * a.n_kv_heads + hk) * a.ws.n_splits;
  for (int h = 0; h < g; ++h) {
    const int64_t idx = (int64_t)(slot0 + split) * g + h;
    if (tid == 0) {
      a.ws.ml[2 * idx] = m_run[h];
      a.ws.ml[2 * idx + 1] = l_run[h];
    }
    if (tid < d) a.ws.o[idx * d + tid] = o_acc[h];
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int t = atomicAdd(a.ws.tickets + b * a.n_kv_heads + hk, 1);
    is_last = (t == a.ws.n_splits - 1);
    if (is_last) a.ws.tickets[b * a.n_kv_heads + hk] = 0;  // leave no small counts behind in scratch that other calls reuse
    if (is_last && len <= 0 && a.lse == nullptr) set_status(a.status, PQ_ERR_EMPTY);
  }
  __syncthreads();
  if (is_last) {
    __threadfence();
    combine_and_store(a, b, hk, g, slot0, a.ws.n_splits, reinterpret_cast<float*>(smem));
  }
}

}  // namespace pq
#include "pq_decode_fast.cuh"
#include "pq_prefill.cuh"
#include "pq_prefill_tc.cuh"
namespace pq {

// ---- partial attentions: merge, and exact attention over an uncompressed window -----------------
// out = sum_p w_p out_p with w_p = exp(lse_p - lse) and lse = log sum_p exp(lse_p): the attention over the union of
// the token sets behind the parts (token shards on several GPUs; the packed cache and a 16-bit tail).
__global__ void merge_attention_kernel(int d, int64_t n_rows, int n_parts, const void* parts_out, int parts_dtype,
                                       const float* parts_lse, void* out, int out_dtype, float* lse_out, int32_t* status) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_rows * d) return;
  const int64_t row = idx / d;
  float mx = -CUDART_INF_F;
  for (int p = 0; p < n_parts; ++p) mx = fmaxf(mx, parts_lse[(int64_t)p * n_rows + row]);
  float acc = 0.f, wsum = 0.f;
  if (mx > -CUDART_INF_F) {
    for (int p = 0; p < n_parts; ++p) {   // part order: the result does not depend on the launch
      const float l = parts_lse[(int64_t)p * n_rows + row];
      if (l == -CUDART_INF_F) continue;   // a part without tokens (its output may hold anything)
      const float w = __expf(l - mx);
      const int64_t i = (int64_t)p * n_rows * d + idx;
      const float v = parts_dtype == PQ_DTYPE_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(parts_out)[i])
                                                   : reinterpret_cast<const float*>(parts_out)[i];
      acc = fmaf(w, v, acc);
      wsum += w;
    }
    acc /= wsum;
  } else if (idx == row * d) {
    set_status(status, PQ_ERR_EMPTY);
  }
  if (out_dtype == PQ_DTYPE_BF16) reinterpret_cast<__nv_bfloat16*>(out)[idx] = __float2bfloat16(acc);
  else reinterpret_cast<float*>(out)[idx] = acc;
  if (lse_out != nullptr && idx == row * d) lse_out[row] = mx > -CUDART_INF_F ? mx + __logf(wsum) : -CUDART_INF_F;
}

// Exact softmax attention (Eq. 2) of one query per sequence over an uncompressed window of keys and values (the
// tokens a serving loop keeps in 16 bits, Section 5.3's protocol for generated tokens).  One CTA per (kv head,
// sequence, split of the window's tokens); a CTA writes the partial attention of its tokens (part blockIdx.z of the
// output), to be merged by merge_attention_kernel.  Steps of kTailStage tokens (half as many for a float32 window): the
// key and value rows are copied to shared memory with coalesced 16-byte cp.async (all of a step's loads in flight at
// once), then scores by a thread per token (key rows 16 bytes apart modulo 128: conflict-free 16-byte reads), running
// maximum and denominator per head, then a thread per coordinate accumulates P . V.
constexpr int kTailThreads = 128, kTailStage = 64;
static_assert(2 * kTailStage <= kTailThreads, "two threads per staged token");
constexpr int kTailSmemMax = 80 * 1024;
__host__ __device__ inline int tail_stage_tokens(int kv_dtype) { return kv_dtype == PQ_DTYPE_BF16 ? kTailStage : kTailStage / 2; }
__host__ __device__ inline size_t tail_smem_bytes(int d, int g, int kv_dtype) {
  const int T = tail_stage_tokens(kv_dtype), row = d * (kv_dtype == PQ_DTYPE_BF16 ? 2 : 4);
  const int h = 4 * ((g + 3) / 4);
  return (size_t)4 * (h * d + h * kTailStage + 3 * kMaxGroup + 4) + (size_t)T * (row + 16) + (size_t)T * row;
}
struct TailArgs {
  int d, n_q_heads, n_kv_heads, io_dtype, kv_dtype, capacity, batch;
  float scale;
  const void* q;
  const void* k;
  const void* v;
  const int32_t* lens;
  void* out;
  float* lse;
  int32_t* status;
};
__device__ __forceinline__ float tail_elem(const void* p, int dtype, int64_t i) {
  return dtype == PQ_DTYPE_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i])
                                : reinterpret_cast<const float*>(p)[i];
}
// kHG = groups of four query heads per kv head (heads past the group read q' = 0 and are not stored).
template <int kHG>
__global__ void __launch_bounds__(kTailThreads) tail_attention_kernel(TailArgs a) {
  constexpr int kH = 4 * kHG;
  extern __shared__ float tsm[];
  const int d = a.d, g = a.n_q_heads / a.n_kv_heads, hk = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  float* qs = tsm;                       // [d][kH]: q' = q * scale * log2(e), the heads of a coordinate side by side
  float* sc = qs + kH * d;               // [kTailStage][kH]: scores, then probabilities, of a step
  float* m_sm = sc + kH * kTailStage;    // [kH] running maximum (log2 domain)
  float* l_sm = m_sm + kMaxGroup;        // [kH] running denominator
  float* corr_sm = l_sm + kMaxGroup;     // [kH]
  const int esz = a.kv_dtype == PQ_DTYPE_BF16 ? 2 : 4, row_bytes = d * esz, krow = row_bytes + 16;
  const int T = tail_stage_tokens(a.kv_dtype);
  uint8_t* ks = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(corr_sm + kMaxGroup) + 15) & ~(uintptr_t)15);   // [T][krow]
  uint8_t* vs = ks + (size_t)T * krow;                                                                          // [T][row_bytes]
  for (int i = tid; i < kH * d; i += kTailThreads) {
    const int c = i / kH, h = i - c * kH;
    qs[i] = h < g ? tail_elem(a.q, a.io_dtype, ((int64_t)b * a.n_q_heads + hk * g + h) * d + c) * a.scale * 1.4426950408889634f : 0.f;
  }
  if (tid < kH) {
    m_sm[tid] = -CUDART_INF_F;
    l_sm[tid] = 0.f;
  }
  int len_all = a.lens[b];
  len_all = len_all < 0 ? 0 : (len_all > a.capacity ? a.capacity : len_all);
  const int per = (len_all + (int)gridDim.z - 1) / (int)gridDim.z;
  const int t_begin = min(len_all, (int)blockIdx.z * per), len = min(len_all, t_begin + per) - t_begin;
  const int64_t part_rows = (int64_t)blockIdx.z * a.batch * a.n_q_heads;   // this split's part of out and lse
  float acc[kH];
#pragma unroll
  for (int h = 0; h < kH; ++h) acc[h] = 0.f;
  const uint32_t ks_s = (uint32_t)__cvta_generic_to_shared(ks), vs_s = (uint32_t)__cvta_generic_to_shared(vs);
  const int gr_shift = 31 - __clz(row_bytes >> 4);   // 16-byte pieces of a row: a power of two
  const int64_t row_stride = (int64_t)a.n_kv_heads * row_bytes;
  const int64_t base = (((int64_t)b * a.capacity + t_begin) * a.n_kv_heads + hk) * row_bytes;
  for (int c0 = 0; c0 < len; c0 += T) {
    const int n = min(T, len - c0);
    __syncthreads();   // the previous step's rows and probabilities have been used (first step: q', m, l are set)
    for (int i = tid; i < (n << gr_shift); i += kTailThreads) {
      const int t = i >> gr_shift, piece = i - (t << gr_shift);
      const int64_t off = base + (c0 + t) * row_stride + 16 * piece;
      pf_cp16(ks_s + t * krow + 16 * piece, reinterpret_cast<const uint8_t*>(a.k) + off);
      pf_cp16(vs_s + t * row_bytes + 16 * piece, reinterpret_cast<const uint8_t*>(a.v) + off);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    {   // scores: two threads per token, each over half of the coordinates (a stage holds at most 64 tokens)
      const int t = tid >> 1, i0 = (tid & 1) * (d >> 1);
      const uint8_t* row = ks + t * krow;
      float s[kH];
#pragma unroll
      for (int h = 0; h < kH; ++h) s[h] = 0.f;
#pragma unroll 2
      for (int i = i0; i < i0 + (d >> 1) && t < n; i += 8) {   // d is a multiple of 16
        float kv[8];
        if (a.kv_dtype == PQ_DTYPE_BF16) {
          const uint4 raw = *reinterpret_cast<const uint4*>(row + 2 * i);
          const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            kv[2 * e] = __uint_as_float(w[e] << 16);
            kv[2 * e + 1] = __uint_as_float(w[e] & 0xFFFF0000u);
          }
        } else {
          const float4 lo = *reinterpret_cast<const float4*>(row + 4 * i);
          const float4 hi = *reinterpret_cast<const float4*>(row + 4 * i + 16);
          kv[0] = lo.x; kv[1] = lo.y; kv[2] = lo.z; kv[3] = lo.w; kv[4] = hi.x; kv[5] = hi.y; kv[6] = hi.z; kv[7] = hi.w;
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
#pragma unroll
          for (int hg = 0; hg < kHG; ++hg) {   // one 16-byte broadcast read gives q' of four heads
            const float4 q4 = *reinterpret_cast<const float4*>(qs + (i + e) * kH + 4 * hg);
            s[4 * hg] = fmaf(q4.x, kv[e], s[4 * hg]);
            s[4 * hg + 1] = fmaf(q4.y, kv[e], s[4 * hg + 1]);
            s[4 * hg + 2] = fmaf(q4.z, kv[e], s[4 * hg + 2]);
            s[4 * hg + 3] = fmaf(q4.w, kv[e], s[4 * hg + 3]);
          }
        }
      }
#pragma unroll
      for (int h = 0; h < kH; ++h) s[h] += __shfl_xor_sync(0xffffffffu, s[h], 1);
      if (t < n && (tid & 1) == 0) {
#pragma unroll
        for (int hg = 0; hg < kHG; ++hg)
          *reinterpret_cast<float4*>(sc + t * kH + 4 * hg) = make_float4(s[4 * hg], s[4 * hg + 1], s[4 * hg + 2], s[4 * hg + 3]);
      }
    }
    __syncthreads();
    for (int h = warp; h < g; h += kTailThreads / 32) {   // a warp per head: maximum, probabilities, their sum
      float mx = -CUDART_INF_F;
      for (int t = lane; t < n; t += 32) mx = fmaxf(mx, sc[t * kH + h]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m_sm[h], mx);
      float sum = 0.f;
      for (int t = lane; t < n; t += 32) {
        const float p = exp2f(sc[t * kH + h] - m_new);
        sc[t * kH + h] = p;
        sum += p;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (lane == 0) {
        const float corr = exp2f(m_sm[h] - m_new);   // 0 on the first step
        corr_sm[h] = corr;
        l_sm[h] = l_sm[h] * corr + sum;
        m_sm[h] = m_new;
      }
    }
    __syncthreads();
    if (tid < d) {
#pragma unroll
      for (int h = 0; h < kH; ++h) acc[h] *= h < g ? corr_sm[h] : 0.f;
#pragma unroll 8
      for (int t = 0; t < n; ++t) {
        const float vv = a.kv_dtype == PQ_DTYPE_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(vs + t * row_bytes)[tid])
                                                     : reinterpret_cast<const float*>(vs + t * row_bytes)[tid];
#pragma unroll
        for (int hg = 0; hg < kHG; ++hg) {
          const float4 p4 = *reinterpret_cast<const float4*>(sc + t * kH + 4 * hg);
          acc[4 * hg] = fmaf(p4.x, vv, acc[4 * hg]);
          acc[4 * hg + 1] = fmaf(p4.y, vv, acc[4 * hg + 1]);
          acc[4 * hg + 2] = fmaf(p4.z, vv, acc[4 * hg + 2]);
          acc[4 * hg + 3] = fmaf(p4.w, vv, acc[4 * hg + 3]);
        }
      }
    }
  }
  __syncthreads();
  if (tid < d) {
#pragma unroll
    for (int h = 0; h < kH; ++h)
      if (h < g) {
        const float o = len > 0 ? acc[h] / l_sm[h] : 0.f;
        const int64_t oi = (part_rows + (int64_t)b * a.n_q_heads + hk * g + h) * d + tid;
        if (a.io_dtype == PQ_DTYPE_BF16) reinterpret_cast<__nv_bfloat16*>(a.out)[oi] = __float2bfloat16(o);
        else reinterpret_cast<float*>(a.out)[oi] = o;
      }
  }
  if (tid < g) {
    const int64_t li = part_rows + (int64_t)b * a.n_q_heads + hk * g + tid;
    if (a.lse != nullptr) a.lse[li] = len > 0 ? (m_sm[tid] + log2f(l_sm[tid])) * 0.693147180559945309f : -CUDART_INF_F;
    else if (len <= 0) set_status(a.status, PQ_ERR_EMPTY);
  }
}

// ---- inspection kernels ----------------------------------------------------------------------
__global__ void unpack_codes_kernel(int d, int n_kv_heads, const uint8_t* cache, int batch, Paging pg,
                                    int n_tokens, uint8_t* codes, __half* radii) {
  const Layout L = make_layout(d, pg.page_tokens);
  const int64_t n = (int64_t)batch * n_kv_heads * 2 * n_tokens;
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= n) return;
  const int tok = (int)(v % n_tokens);
  const int kv = (int)((v / n_tokens) & 1);
  const int h = (int)((v / (2 * (int64_t)n_tokens)) % n_kv_heads);
  const int b = (int)(v / (2 * (int64_t)n_tokens * n_kv_heads));
  const int64_t off = block_offset(L, pg, n_kv_heads, b, h, kv, tok);
  if (off < 0) return;  // a page outside the pool: the outputs of this token keep what they held
  const uint8_t* tb = cache + off;
  const int t = tok % kTokenBlock;
  const int n_codes = 15 * L.nb;
  uint8_t* out = codes + v * n_codes;
  for (int blk = 0; blk < L.nb; ++blk) {
    const uint32_t l1 = get_l1(tb, L, t, blk), l2 = get_l2(tb, L, t, blk);
    const uint32_t l3 = get_l3(tb, L, t, blk), l4 = get_l4(tb, L, t, blk);
    for (int j = 0; j < 8; ++j) out[blk * 8 + j] = (l1 >> (4 * j)) & 15u;
    for (int j = 0; j < 4; ++j) out[8 * L.nb + blk * 4 + j] = (l2 >> (2 * j)) & 3u;
    for (int j = 0; j < 2; ++j) out[12 * L.nb + blk * 2 + j] = (l3 >> (2 * j)) & 3u;
    out[14 * L.nb + blk] = l4;
    radii[v * L.nb + blk] = reinterpret_cast<const __half*>(tb + L.orad + t * L.br)[blk];
  }
}

__global__ void dequant_kernel(int d, int n_kv_heads, const float* S, const Tables* tables, const uint8_t* cache,
                               Paging pg, int n_tokens, float* x_hat) {
  extern __shared__ float ysm[];
  __shared__ float cc[32], cs[32];
  const Layout L = make_layout(d, pg.page_tokens);
  const int64_t v = blockIdx.x;
  const int j = threadIdx.x;
  for (int i = j; i < PQ_N_CENTROIDS; i += blockDim.x) {
    cc[i] = tables->cen_cos[i];
    cs[i] = tables->cen_sin[i];
  }
  __syncthreads();
  const int tok = (int)(v % n_tokens);
  const int kv = (int)((v / n_tokens) & 1);
  const int h = (int)((v / (2 * (int64_t)n_tokens)) % n_kv_heads);
  const int b = (int)(v / (2 * (int64_t)n_tokens * n_kv_heads));
  const int64_t off = block_offset(L, pg, n_kv_heads, b, h, kv, tok);
  if (off < 0) return;  // uniform over the CTA
  const uint8_t* tb = cache + off;
  if (d == 128) {
    // the fp16 arithmetic of the attention kernel's value path: u = rn(r * U), x = rn(u * t1)
    const int t = tok % kTokenBlock, blk = j >> 4, i = j & 15;
    const uint32_t c1 = (get_l1(tb, L, t, blk) >> (4 * (i >> 1))) & 15u;
    const uint32_t c2 = (get_l2(tb, L, t, blk) >> (2 * (i >> 2))) & 3u;
    const uint32_t c3 = (get_l3(tb, L, t, blk) >> (2 * (i >> 3))) & 3u;
    const uint32_t c4 = get_l4(tb, L, t, blk);
    const uint32_t up = tables->u_tab[i >> 2][c2 | (c3 << 2) | (c4 << 4)].x;
    const __half2 uh = *reinterpret_cast<const __half2*>(&up);
    const __half r = reinterpret_cast<const __half*>(tb + L.orad + t * L.br)[blk];
    const __half u = __hmul(r, (i & 2) ? __high2half(uh) : __low2half(uh));
    const __half2 t1 = *reinterpret_cast<const __half2*>(&tables->l1_hi[c1]);  // (cos, sin) of the centroid
    ysm[j] = __half2float(__hmul(u, (i & 1) ? __high2half(t1) : __low2half(t1)));
  } else {
    ysm[j] = decode_coord(tb, L, tok % kTokenBlock, j, cc, cs);
  }
  __syncthreads();
  float acc = 0.f;
  for (int k = 0; k < d; ++k) acc = fmaf(ysm[k], S[(int64_t)j * d + k], acc);
  x_hat[v * d + j] = acc;
}

}  // namespace pq

extern "C" {

int64_t pq_workspace_bytes(int32_t head_dim, int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t max_len) {
  if (!(head_dim == 16 || head_dim == 32 || head_dim == 64 || head_dim == 128)) return PQ_ERR_UNSUPPORTED;
  if (batch <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || max_len <= 0 || n_q_heads % n_kv_heads) return PQ_ERR_INVALID_ARG;
  return pq::carve_workspace(nullptr, head_dim, batch, n_q_heads, n_kv_heads, max_len).bytes;
}

static int32_t launch_attention(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                const void* tables_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                const int32_t* cache_lens_dev, int32_t batch, int32_t n_q, int32_t capacity, const pq::Paging& pg,
                                int32_t max_len, float scale, void* out_dev, void* workspace_dev, int32_t* status_dev,
                                void* stream, float* lse_dev = nullptr) {
  pq::NvtxRange nvtx_range("pq attention");
  if (!(head_dim == 16 || head_dim == 32 || head_dim == 64 || head_dim == 128)) return PQ_ERR_UNSUPPORTED;
  if (!S_dev || !tables_dev || !q_dev || !cache_dev || !cache_lens_dev || !out_dev || !workspace_dev || !status_dev)
    return PQ_ERR_INVALID_ARG;
  if (batch <= 0 || n_q <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || capacity <= 0 || max_len <= 0) return PQ_ERR_INVALID_ARG;
  if (n_q_heads % n_kv_heads) return PQ_ERR_INVALID_ARG;
  if (n_q_heads / n_kv_heads > pq::kMaxGroup) return PQ_ERR_UNSUPPORTED;
  if (io_dtype != PQ_DTYPE_F32 && io_dtype != PQ_DTYPE_BF16) return PQ_ERR_UNSUPPORTED;
  const uintptr_t bits = (uintptr_t)S_dev | (uintptr_t)tables_dev | (uintptr_t)q_dev | (uintptr_t)cache_dev |
                         (uintptr_t)out_dev | (uintptr_t)workspace_dev;
  if (bits & 15) return PQ_ERR_ALIGNMENT;
  const int64_t pairs = (int64_t)batch * n_q;  // (sequence, query) pairs: the kernels' batch
  if (pairs > 65535 || n_kv_heads > 65535) return PQ_ERR_UNSUPPORTED;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  pq::DecodeArgs a;
  a.d = head_dim; a.n_q_heads = n_q_heads; a.n_kv_heads = n_kv_heads; a.batch = (int)pairs; a.n_q = n_q; a.capacity = capacity;
  a.io_dtype = io_dtype; a.scale = scale; a.S = S_dev; a.tables = reinterpret_cast<const pq::Tables*>(tables_dev);
  a.q = q_dev; a.cache = reinterpret_cast<const uint8_t*>(cache_dev); a.lens = cache_lens_dev; a.out = out_dev;
  a.status = status_dev;
  a.lse = lse_dev;
  a.pg = pg;
  a.ws = pq::carve_workspace(workspace_dev, head_dim, (int)pairs, n_q_heads, n_kv_heads, max_len);
  const int g = n_q_heads / n_kv_heads;
  if (lse_dev != nullptr && n_q != 1) return PQ_ERR_UNSUPPORTED;
  // Chunks of 32 or more rows (queries x heads of a group), d = 128: the tcgen05 kernel (operands in shared memory,
  // accumulators in tensor memory) decodes every block once for all rows; below 128 rows it is taken when that is
  // estimated to be faster than one decode attention per query, which spreads over all SMs whatever the batch.
  // The register-fragment kernel is only reached through the test hook (it is the slower of the two at every size).
  const int rows = n_q * g;
  bool use_tc = false, use_fragment_kernel = false;
  int n_sm = 0, q_blocks = 0;
  bool pair = false;
  if (head_dim == 128 && rows >= 32) {
    static pq::DeviceMemo configured_pt, configured_pt2;
    n_sm = pq::configure_for_device(pq::prefill_tc_kernel<false>, pq::kPtSmTotal, configured_pt);
    if (n_sm == 0) return PQ_ERR_CUDA;
    if (pq::configure_for_device(pq::prefill_tc_kernel<true>, pq::kPtSmTotal, configured_pt2) == 0) return PQ_ERR_CUDA;
    const int qb_rows = pq::kPtRows / g;
    q_blocks = (n_q + qb_rows - 1) / qb_rows;
    // Two query blocks of one (kv head, sequence) per cluster: one 256-row MMA per step, each CTA decodes half of
    // every block.  An odd count is completed by a CTA without rows -- also a single block when the pairs still fit
    // on the device at once: the second CTA then only shares the decoding (the kernel is bound by it).
    pair = q_blocks >= 2 || 2 * (int64_t)n_kv_heads * batch <= n_sm;
    if (rows >= pq::kPfRows && pq::take_debug_wait_failure(3)) {
      use_fragment_kernel = true;
    } else if (rows >= pq::kPtRows) {
      use_tc = true;
    } else {
      // measured on B200: 1.25 us (pair) or 2.4 us per 64-token block and CTA; decode attention at 1.7 TB/s of packed bytes
      const double ctas = (double)n_kv_heads * batch * (pair ? 2.0 : 1.0);
      const double waves = std::ceil(ctas / n_sm);
      const double t_tc = waves * std::ceil(max_len / 64.0) * (pair ? 1.25 : 2.4) + 10.0;
      const double t_decode = (double)pairs * n_kv_heads * max_len * 124.0 / 1.7e6 + 10.0;
      use_tc = t_tc < t_decode || pairs * n_kv_heads > pq::kFastMaxUnits;
    }
  }
  if (use_tc) {
    a.epoch = 0u;
    a.debug = pq::take_debug_wait_failure(4) ? 2u : 0u;
    if (pair) {
      // Two query blocks of one (kv head, sequence) per cluster: one 256-row MMA per step, each CTA decodes half of
      // every block.  An odd count is completed by a CTA without rows -- also a single block when the pairs still fit
      // on the device at once: the second CTA then only shares the decoding (the kernel is bound by it).
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((q_blocks + 1) & ~1, n_kv_heads, batch);
      cfg.blockDim = dim3(pq::kPtThreads);
      cfg.dynamicSmemBytes = pq::kPtSmTotal;
      cfg.stream = st;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = 2;
      attr[0].val.clusterDim.y = 1;
      attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      if (cudaLaunchKernelEx(&cfg, pq::prefill_tc_kernel<true>, a, (int)n_q) != cudaSuccess) {
        cudaGetLastError();
        return PQ_ERR_CUDA;
      }
      return pq::launch_status();
    }
    dim3 grid(q_blocks, n_kv_heads, batch);
    pq::prefill_tc_kernel<false><<<grid, pq::kPtThreads, pq::kPtSmTotal, st>>>(a, n_q);
    return pq::launch_status();
  }
  if (use_fragment_kernel) {
    // decode each block of the cache once for 64 (query, head) rows, mma.sync on register fragments
    static pq::DeviceMemo configured_pf;
    if (pq::configure_for_device(pq::prefill_attention_kernel, pq::kPfTotal, configured_pf) == 0) return PQ_ERR_CUDA;
    const int qb_rows = pq::kPfRows / g;
    dim3 grid((n_q + qb_rows - 1) / qb_rows, n_kv_heads, batch);
    pq::prefill_attention_kernel<<<grid, pq::kPfThreads, pq::kPfTotal, st>>>(a, n_q);
    return pq::launch_status();
  }
  if (head_dim == 128 && pairs * n_kv_heads <= pq::kFastMaxUnits) {
    // One launch: the persistent kernel rotates the queries itself and needs no cleared tickets.
    // The tickets in the (uninitialised, possibly shared) scratch are tagged with a per-call number.  It starts
    // at a value drawn from the clock and the address space of this process, advances by an odd constant and
    // always has its top bit set, so it cannot equal a small integer that another kernel left in the same bytes.
    static std::atomic<uint32_t> call_epoch{[] {
      uint64_t x = (uint64_t)std::chrono::steady_clock::now().time_since_epoch().count() ^ (uint64_t)(uintptr_t)&launch_attention;
      x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
      x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
      return (uint32_t)(x ^ (x >> 31));
    }()};
    a.epoch = call_epoch.fetch_add(0x9E3779B1u, std::memory_order_relaxed) | 0x80000000u;
    a.debug = pq::take_debug_wait_failure(2) ? 1u : 0u;
    static pq::DeviceMemo configured[4];
    const bool paged = pg.table != nullptr;
    void (*kernel)(pq::DecodeArgs) =
        g <= 4 ? (paged ? pq::decode_attention_fast_kernel<1, true> : pq::decode_attention_fast_kernel<1, false>)
               : (paged ? pq::decode_attention_fast_kernel<2, true> : pq::decode_attention_fast_kernel<2, false>);
    const int n_sm = pq::configure_for_device(kernel, pq::kSmTotal, configured[(g <= 4 ? 0 : 1) + (paged ? 2 : 0)]);
    if (n_sm == 0) return PQ_ERR_CUDA;
    const int grid = n_sm < pq::kFastMaxGrid ? n_sm : pq::kFastMaxGrid;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(pq::kFastThreads);
    cfg.dynamicSmemBytes = pq::kSmTotal;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];   // may be set up while the kernel before it in the stream finishes (it waits inside)
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kernel, a) != cudaSuccess) {
      cudaGetLastError();
      return PQ_ERR_CUDA;
    }
    return pq::launch_status();
  }
  a.epoch = 0u;
  a.debug = 0u;
  pq::rotate_query_kernel<<<(unsigned)pairs * n_q_heads, head_dim, head_dim * sizeof(float), st>>>(a);
  const pq::Layout L = pq::make_layout(head_dim, pg.page_tokens);
  size_t smem = 2 * L.block_bytes + sizeof(float) * ((size_t)g * head_dim + 3 * g * pq::kTokenBlock +
                                                     3 * pq::kMaxGroup + 64);
  const size_t smem_combine = sizeof(float) * pq::combine_smem_floats(g, head_dim, a.ws.n_splits);
  if (smem < smem_combine) smem = smem_combine;
  dim3 grid(a.ws.n_splits, n_kv_heads, (unsigned)pairs);
  pq::decode_attention_simple_kernel<<<grid, pq::kSimpleThreads, smem, st>>>(a);
  return pq::launch_status();
}

int32_t pq_decode_attention(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                            const void* tables_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                            const int32_t* cache_lens_dev, int32_t batch, int32_t capacity, int32_t max_len,
                            float scale, void* out_dev, void* workspace_dev, int32_t* status_dev, void* stream) {
  return launch_attention(head_dim, n_q_heads, n_kv_heads, S_dev, tables_dev, q_dev, io_dtype, cache_dev, cache_lens_dev,
                          batch, 1, capacity, pq::contiguous_paging(capacity, batch), max_len, scale, out_dev, workspace_dev,
                          status_dev, stream);
}

int32_t pq_decode_attention_paged(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                  const void* tables_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                  const int32_t* cache_lens_dev, int32_t batch, const pq_paging* paging, int32_t max_len,
                                  float scale, void* out_dev, void* workspace_dev, int32_t* status_dev, void* stream) {
  pq::Paging pg;
  const int32_t st = pq::paging_from(paging, head_dim, &pg);
  if (st != PQ_OK) return st;
  return launch_attention(head_dim, n_q_heads, n_kv_heads, S_dev, tables_dev, q_dev, io_dtype, cache_dev, cache_lens_dev,
                          batch, 1, pg.page_tokens * pg.pages_per_seq, pg, max_len, scale, out_dev, workspace_dev, status_dev,
                          stream);
}

int32_t pq_multi_query_attention(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                 const void* tables_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                 const int32_t* cache_lens_dev, int32_t batch, int32_t n_q, int32_t capacity,
                                 int32_t max_len, float scale, void* out_dev, void* workspace_dev, int32_t* status_dev,
                                 void* stream) {
  return launch_attention(head_dim, n_q_heads, n_kv_heads, S_dev, tables_dev, q_dev, io_dtype, cache_dev, cache_lens_dev,
                          batch, n_q, capacity, pq::contiguous_paging(capacity, batch), max_len, scale, out_dev, workspace_dev,
                          status_dev, stream);
}

int32_t pq_multi_query_attention_paged(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                       const void* tables_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                       const int32_t* cache_lens_dev, int32_t batch, int32_t n_q, const pq_paging* paging,
                                       int32_t max_len, float scale, void* out_dev, void* workspace_dev,
                                       int32_t* status_dev, void* stream) {
  pq::Paging pg;
  const int32_t st = pq::paging_from(paging, head_dim, &pg);
  if (st != PQ_OK) return st;
  return launch_attention(head_dim, n_q_heads, n_kv_heads, S_dev, tables_dev, q_dev, io_dtype, cache_dev, cache_lens_dev,
                          batch, n_q, pg.page_tokens * pg.pages_per_seq, pg, max_len, scale, out_dev, workspace_dev, status_dev,
                          stream);
}

int32_t pq_decode_attention_lse(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                const void* tables_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                const int32_t* cache_lens_dev, int32_t batch, int32_t capacity, const pq_paging* paging,
                                int32_t max_len, float scale, void* out_dev, float* lse_dev, void* workspace_dev,
                                int32_t* status_dev, void* stream) {
  if (lse_dev == nullptr || ((uintptr_t)lse_dev & 3)) return lse_dev == nullptr ? PQ_ERR_INVALID_ARG : PQ_ERR_ALIGNMENT;
  pq::Paging pg = pq::contiguous_paging(capacity, batch);
  if (paging != nullptr) {
    const int32_t st = pq::paging_from(paging, head_dim, &pg);
    if (st != PQ_OK) return st;
    capacity = pg.page_tokens * pg.pages_per_seq;
  }
  return launch_attention(head_dim, n_q_heads, n_kv_heads, S_dev, tables_dev, q_dev, io_dtype, cache_dev, cache_lens_dev,
                          batch, 1, capacity, pg, max_len, scale, out_dev, workspace_dev, status_dev, stream, lse_dev);
}

int32_t pq_merge_attention(int32_t head_dim, int32_t n_q_heads, int32_t batch, int32_t n_parts, const void* parts_out_dev,
                           int32_t parts_dtype, const float* parts_lse_dev, void* out_dev, int32_t out_dtype,
                           float* lse_out_dev, int32_t* status_dev, void* stream) {
  if (head_dim <= 0 || n_q_heads <= 0 || batch <= 0 || n_parts <= 0 || n_parts > 1024) return PQ_ERR_INVALID_ARG;
  if (!parts_out_dev || !parts_lse_dev || !out_dev || !status_dev) return PQ_ERR_INVALID_ARG;
  if ((parts_dtype != PQ_DTYPE_F32 && parts_dtype != PQ_DTYPE_BF16) || (out_dtype != PQ_DTYPE_F32 && out_dtype != PQ_DTYPE_BF16))
    return PQ_ERR_UNSUPPORTED;
  const int64_t n_rows = (int64_t)batch * n_q_heads, n = n_rows * head_dim;
  if (n * n_parts >= (1ll << 40)) return PQ_ERR_UNSUPPORTED;
  pq::merge_attention_kernel<<<(unsigned)((n + 255) / 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      head_dim, n_rows, n_parts, parts_out_dev, parts_dtype, parts_lse_dev, out_dev, out_dtype, lse_out_dev, status_dev);
  return pq::launch_status();
}

int32_t pq_tail_attention(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const void* q_dev, int32_t io_dtype,
                          const void* k_tail_dev, const void* v_tail_dev, int32_t kv_dtype, const int32_t* tail_lens_dev,
                          int32_t batch, int32_t tail_capacity, int32_t n_splits, float scale, void* out_dev, float* lse_dev,
                          int32_t* status_dev, void* stream) {
  if (n_splits < 1 || n_splits > 1024 || (n_splits > 1 && lse_dev == nullptr)) return PQ_ERR_INVALID_ARG;
  if (((uintptr_t)k_tail_dev | (uintptr_t)v_tail_dev) & 15) return PQ_ERR_ALIGNMENT;
  if (!(head_dim == 16 || head_dim == 32 || head_dim == 64 || head_dim == 128)) return PQ_ERR_UNSUPPORTED;
  if (!q_dev || !k_tail_dev || !v_tail_dev || !tail_lens_dev || !out_dev || !status_dev) return PQ_ERR_INVALID_ARG;
  if (batch <= 0 || batch > 65535 || n_q_heads <= 0 || n_kv_heads <= 0 || tail_capacity <= 0 || n_q_heads % n_kv_heads)
    return PQ_ERR_INVALID_ARG;
  if (n_q_heads / n_kv_heads > pq::kMaxGroup) return PQ_ERR_UNSUPPORTED;
  if ((io_dtype != PQ_DTYPE_F32 && io_dtype != PQ_DTYPE_BF16) || (kv_dtype != PQ_DTYPE_F32 && kv_dtype != PQ_DTYPE_BF16))
    return PQ_ERR_UNSUPPORTED;
  pq::TailArgs a;
  a.d = head_dim; a.n_q_heads = n_q_heads; a.n_kv_heads = n_kv_heads; a.io_dtype = io_dtype; a.kv_dtype = kv_dtype;
  a.capacity = tail_capacity; a.batch = batch; a.scale = scale; a.q = q_dev; a.k = k_tail_dev; a.v = v_tail_dev; a.lens = tail_lens_dev;
  a.out = out_dev; a.lse = lse_dev; a.status = status_dev;
  const int g = n_q_heads / n_kv_heads;
  const size_t smem = pq::tail_smem_bytes(head_dim, g, kv_dtype);
  static pq::DeviceMemo configured1, configured2;
  if (smem > (size_t)pq::kTailSmemMax) return PQ_ERR_UNSUPPORTED;
  if (pq::configure_for_device(pq::tail_attention_kernel<1>, pq::kTailSmemMax, configured1) == 0) return PQ_ERR_CUDA;
  if (pq::configure_for_device(pq::tail_attention_kernel<2>, pq::kTailSmemMax, configured2) == 0) return PQ_ERR_CUDA;
  dim3 grid(n_kv_heads, batch, n_splits);
  if (g <= 4) pq::tail_attention_kernel<1><<<grid, pq::kTailThreads, smem, reinterpret_cast<cudaStream_t>(stream)>>>(a);
  else pq::tail_attention_kernel<2><<<grid, pq::kTailThreads, smem, reinterpret_cast<cudaStream_t>(stream)>>>(a);
  return pq::launch_status();
}

// ---- decode attention on the library's own scratch ---------------------------------------------
// Scratch for callers that cannot allocate: lives in every GPU context that loads the library.
// In host code the name below is only a handle; the device address comes from
// cudaGetSymbolAddress, once per device, and is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[PQ_STATIC_SCRATCH_BYTES];

int64_t pq_static_scratch_bytes(void) { return PQ_STATIC_SCRATCH_BYTES; }

int32_t pq_decode_attention_static(int32_t head_dim, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                   const void* tables_dev, const void* q_dev, int32_t io_dtype,
                                   const void* cache_dev, const int32_t* cache_lens_dev, int32_t batch,
                                   int32_t capacity, int32_t max_len, float scale, void* out_dev,
                                   int32_t* status_dev, void* stream) {
  const int64_t need = pq_workspace_bytes(head_dim, batch, n_q_heads, n_kv_heads, max_len);
  if (need < 0) return (int32_t)need;
  if (need > PQ_STATIC_SCRATCH_BYTES) return PQ_ERR_SCRATCH;
  static std::atomic<void*> scratch_of_device[pq::kMaxDevices];
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= pq::kMaxDevices) {
    pq::note_cuda_error(e == cudaSuccess ? cudaErrorInvalidDevice : e);
    return PQ_ERR_CUDA;
  }
  void* scratch = scratch_of_device[dev].load(std::memory_order_acquire);
  if (scratch == nullptr) {  // first call on this device (which is current): resolve the symbol
    e = cudaGetSymbolAddress(&scratch, g_static_scratch);
    if (e != cudaSuccess || scratch == nullptr) {
      pq::note_cuda_error(e == cudaSuccess ? cudaErrorInvalidSymbol : e);
      return PQ_ERR_CUDA;
    }
    scratch_of_device[dev].store(scratch, std::memory_order_release);
  }
  return pq_decode_attention(head_dim, n_q_heads, n_kv_heads, S_dev, tables_dev, q_dev, io_dtype, cache_dev,
                             cache_lens_dev, batch, capacity, max_len, scale, out_dev, scratch, status_dev, stream);
}

static int32_t unpack_entry(int32_t head_dim, int32_t n_kv_heads, const void* cache_dev, int32_t batch, int32_t capacity,
                            const pq::Paging& pg, int32_t n_tokens, uint8_t* codes_dev, void* radii_dev, void* stream) {
  if (!(head_dim == 16 || head_dim == 32 || head_dim == 64 || head_dim == 128)) return PQ_ERR_UNSUPPORTED;
  if (!cache_dev || !codes_dev || !radii_dev || batch <= 0 || n_kv_heads <= 0 || n_tokens <= 0 || n_tokens > capacity)
    return PQ_ERR_INVALID_ARG;
  const int64_t n = (int64_t)batch * n_kv_heads * 2 * n_tokens;
  pq::unpack_codes_kernel<<<(unsigned)((n + 127) / 128), 128, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      head_dim, n_kv_heads, reinterpret_cast<const uint8_t*>(cache_dev), batch, pg, n_tokens, codes_dev,
      reinterpret_cast<__half*>(radii_dev));
  return pq::launch_status();
}

int32_t pq_unpack_codes(int32_t head_dim, int32_t n_kv_heads, const void* cache_dev, int32_t batch, int32_t capacity,
                        int32_t n_tokens, uint8_t* codes_dev, void* radii_dev, void* stream) {
  return unpack_entry(head_dim, n_kv_heads, cache_dev, batch, capacity, pq::contiguous_paging(capacity, batch), n_tokens,
                      codes_dev, radii_dev, stream);
}

int32_t pq_unpack_codes_paged(int32_t head_dim, int32_t n_kv_heads, const void* cache_dev, int32_t batch,
                              const pq_paging* paging, int32_t n_tokens, uint8_t* codes_dev, void* radii_dev, void* stream) {
  pq::Paging pg;
  const int32_t st = pq::paging_from(paging, head_dim, &pg);
  if (st != PQ_OK) return st;
  return unpack_entry(head_dim, n_kv_heads, cache_dev, batch, pg.page_tokens * pg.pages_per_seq, pg, n_tokens, codes_dev,
                      radii_dev, stream);
}

static int32_t dequant_entry(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                             const void* cache_dev, int32_t batch, int32_t capacity, const pq::Paging& pg, int32_t n_tokens,
                             float* x_hat_dev, void* stream) {
  if (!(head_dim == 16 || head_dim == 32 || head_dim == 64 || head_dim == 128)) return PQ_ERR_UNSUPPORTED;
  if (!S_dev || !tables_dev || !cache_dev || !x_hat_dev || batch <= 0 || n_kv_heads <= 0 || n_tokens <= 0 ||
      n_tokens > capacity)
    return PQ_ERR_INVALID_ARG;
  const int64_t n = (int64_t)batch * n_kv_heads * 2 * n_tokens;
  if (n >= (1ll << 31)) return PQ_ERR_UNSUPPORTED;
  pq::dequant_kernel<<<(unsigned)n, head_dim, head_dim * sizeof(float), reinterpret_cast<cudaStream_t>(stream)>>>(
      head_dim, n_kv_heads, S_dev, reinterpret_cast<const pq::Tables*>(tables_dev),
      reinterpret_cast<const uint8_t*>(cache_dev), pg, n_tokens, x_hat_dev);
  return pq::launch_status();
}

int32_t pq_dequant_kv(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                      const void* cache_dev, int32_t batch, int32_t capacity, int32_t n_tokens, float* x_hat_dev,
                      void* stream) {
  return dequant_entry(head_dim, n_kv_heads, S_dev, tables_dev, cache_dev, batch, capacity,
                       pq::contiguous_paging(capacity, batch), n_tokens, x_hat_dev, stream);
}

int32_t pq_dequant_kv_paged(int32_t head_dim, int32_t n_kv_heads, const float* S_dev, const void* tables_dev,
                            const void* cache_dev, int32_t batch, const pq_paging* paging, int32_t n_tokens,
                            float* x_hat_dev, void* stream) {
  pq::Paging pg;
  const int32_t st = pq::paging_from(paging, head_dim, &pg);
  if (st != PQ_OK) return st;
  return dequant_entry(head_dim, n_kv_heads, S_dev, tables_dev, cache_dev, batch, pg.page_tokens * pg.pages_per_seq, pg,
                       n_tokens, x_hat_dev, stream);
}

}  // extern "C"
