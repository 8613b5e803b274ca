// Multi-query attention over the packed cache for head_dim 128 (included by pq_decode.cu): the last n_q
// positions of a sequence attend causally to the cached tokens (Eq. 2 / Eq. 3 for a chunk of queries).
//
// With many queries per sequence a decoded tile of the cache is reused by all of them, so the work is a
// dense contraction: one CTA takes 64 rows = (64 / g) queries x the g query heads of one kv head, loops over
// the 64-token blocks of the cache its queries may see, decodes a block once into shared memory (DeQuant of
// Algorithm 1 in float32, stored as fp16 value + fp16 residual for the keys, fp16 for the values) and runs
//   S = Q' K_hat^T (three MMAs per tile: hi*hi, lo*hi, hi*lo), online softmax, O += P V_hat
// on tensor cores (mma.sync m16n8k16 fed by ldmatrix; a warp owns 16 rows).  The queries are rotated by S
// once when the CTA starts (Q' = Q S * scale * log2 e, kept as fp16 value + residual) and the output by S^T
// once when it ends, as in decode attention.  There is no split over the tokens: the grid is
// (query blocks, kv heads, sequences), which fills the GPU for chunks of a prefill.
// This is the first implementation of the path.  The tcgen05 kernel (pq_prefill_tc.cuh) is faster at every size and
// takes every chunk this one could; the dispatch reaches this kernel only through the test hook, for chunks of 64
// rows and more, so that two independent implementations can be compared on the same inputs.
#pragma once

namespace pq {

constexpr int kPfThreads = 128;
constexpr int kPfRows = 64;                 // rows of a CTA: queries x heads of the group
constexpr int kPfStride = 136;              // halves per row of the fp16 tiles: 272 bytes, rows 16 bytes apart mod 128
constexpr int kPfTileBytes = 64 * kPfStride * 2;
constexpr int kPfQhi = 0, kPfQlo = kPfQhi + kPfTileBytes;
constexpr int kPfKhi = kPfQlo + kPfTileBytes, kPfKlo = kPfKhi + kPfTileBytes;   // also: q in float32 at the start, O at the end
constexpr int kPfV = kPfKlo + kPfTileBytes;
constexpr int kPfRaw = kPfV + kPfTileBytes;                                     // two packed (K block, V block) buffers
constexpr int kPfRawBytes = 2 * 62 * kTokenBlock;
constexpr int kPfTab = kPfRaw + 2 * kPfRawBytes;                                // cos / sin of the centroids
constexpr int kPfTotal = kPfTab + 256;
constexpr int kPfOStride = 132;             // floats per row of the output staging
static_assert(64 * 128 * 4 <= 2 * kPfTileBytes && 64 * kPfOStride * 4 <= 2 * kPfTileBytes, "float32 staging fits in the key tiles");

__device__ __forceinline__ void pf_ldsm4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void pf_ldsm4t(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void pf_cp16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

// acc[r] += sum_k x[r][k0 + k] * w[k], k = 0..3, for the 64 rows of a float32 tile in shared memory (row stride `ld` floats)
__device__ __forceinline__ void pf_rank4(float (&acc)[kPfRows], const float* x, int ld, int k0, float4 w) {
#pragma unroll
  for (int r = 0; r < kPfRows; ++r) {
    const float4 v = *reinterpret_cast<const float4*>(x + r * ld + k0);   // the same address in every thread: a broadcast
    acc[r] = fmaf(v.x, w.x, fmaf(v.y, w.y, fmaf(v.z, w.z, fmaf(v.w, w.w, acc[r]))));
  }
}

__global__ void __launch_bounds__(kPfThreads) prefill_attention_kernel(DecodeArgs a, int n_q) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gq = lane >> 2, cq = lane & 3;
  const int g = a.n_q_heads / a.n_kv_heads;
  const int qb_rows = kPfRows / g;                      // queries of a CTA
  const int q0 = blockIdx.x * qb_rows, hk = blockIdx.y, b = blockIdx.z;
  const int n_rows = min(qb_rows, n_q - q0) * g;        // rows in use; row r = (query q0 + r / g, head hk * g + r % g)
  const int len = a.lens[b];
  const uint32_t sb = smem_u32(smem);
  float* cen_cos = reinterpret_cast<float*>(smem + kPfTab);
  float* cen_sin = cen_cos + 32;
  if (tid < PQ_N_CENTROIDS) {
    cen_cos[tid] = a.tables->cen_cos[tid];
    cen_sin[tid] = a.tables->cen_sin[tid];
  }
  auto row_index = [&](int r) -> int64_t {               // offset of row r in q / out ([batch][n_q][n_q_heads][128])
    return (((int64_t)b * n_q + q0 + r / g) * a.n_q_heads + hk * g + r % g) * 128;
  };
  // ---- Q' = (Q S) * scale * log2(e) as fp16 value + residual
  {
    float* qs = reinterpret_cast<float*>(smem + kPfKhi);
    for (int i = tid; i < kPfRows * 128; i += kPfThreads) {
      const int r = i >> 7, k = i & 127;
      float v = 0.f;
      if (r < n_rows)
        v = a.io_dtype == PQ_DTYPE_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.q)[row_index(r) + k])
                                        : reinterpret_cast<const float*>(a.q)[row_index(r) + k];
      qs[i] = v;
    }
    __syncthreads();
    float acc[kPfRows];
#pragma unroll
    for (int r = 0; r < kPfRows; ++r) acc[r] = 0.f;
    for (int k0 = 0; k0 < 128; k0 += 4) {   // thread = column of S
      const float4 w = make_float4(__ldg(a.S + (k0 + 0) * 128 + tid), __ldg(a.S + (k0 + 1) * 128 + tid),
                                   __ldg(a.S + (k0 + 2) * 128 + tid), __ldg(a.S + (k0 + 3) * 128 + tid));
      pf_rank4(acc, qs, 128, k0, w);
    }
    __half* qhi = reinterpret_cast<__half*>(smem + kPfQhi);
    __half* qlo = reinterpret_cast<__half*>(smem + kPfQlo);
    const float f = a.scale * 1.4426950408889634f;
#pragma unroll
    for (int r = 0; r < kPfRows; ++r) {
      const float v = acc[r] * f;
      const __half h = __float2half_rn(v);
      qhi[r * kPfStride + tid] = h;
      qlo[r * kPfStride + tid] = __float2half_rn(v - __half2float(h));
    }
    __syncthreads();   // the float32 copy of q is dead: the key tiles may be written
  }
  // ---- which tokens each of this thread's two rows may see
  int vis[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int r = warp * 16 + gq + 8 * i;
    vis[i] = r < n_rows ? max(0, len - (n_q - 1 - (q0 + r / g))) : 0;
  }
  const int vis_cta = max(0, len - (n_q - 1 - (q0 + (n_rows - 1) / g)));   // the CTA's last query sees the most
  const int n_blocks = (vis_cta + kTokenBlock - 1) / kTokenBlock;
  const Layout L = make_layout(128, a.pg.page_tokens);
  auto fetch = [&](int jb) {  // packed K block and V block of token-block jb -> raw buffer jb & 1
    const uint8_t* src = a.cache + kv_block_pair_offset(L, a.pg, a.n_kv_heads, b, hk, jb, a.status);
    const uint32_t dst = sb + kPfRaw + (jb & 1) * kPfRawBytes;
    for (int i = tid; i < kPfRawBytes / 16; i += kPfThreads) pf_cp16(dst + 16 * i, src + 16 * i);
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  float oacc[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F}, l_run[2] = {0.f, 0.f};
  if (n_blocks > 0) fetch(0);
  for (int jb = 0; jb < n_blocks; ++jb) {
    if (jb + 1 < n_blocks) {
      fetch(jb + 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();   // the raw block has landed; the tiles of the previous block are no longer read
    // ---- DeQuant (Algorithm 1) of 64 tokens x 128 coordinates of K and V in the rotated basis: thread = (token, half)
    {
      const uint8_t* kraw = smem + kPfRaw + (jb & 1) * kPfRawBytes;
      const uint8_t* vraw = kraw + 62 * kTokenBlock;
      const int tok = tid & 63, half = tid >> 6;
      const bool live = jb * kTokenBlock + tok < len;   // stale bytes past the sequence end must not reach the MMAs
      __half* khi = reinterpret_cast<__half*>(smem + kPfKhi) + tok * kPfStride + half * 64;
      __half* klo = reinterpret_cast<__half*>(smem + kPfKlo) + tok * kPfStride + half * 64;
      __half* vhi = reinterpret_cast<__half*>(smem + kPfV) + tok * kPfStride + half * 64;
#pragma unroll 1
      for (int bi = 0; bi < 4; ++bi) {
        float y[16];
        __align__(16) __half h[16], lo[16];
        decode_block(kraw, L, tok, half * 4 + bi, cen_cos, cen_sin, y);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float v = live ? y[i] : 0.f;
          h[i] = __float2half_rn(v);
          lo[i] = __float2half_rn(v - __half2float(h[i]));
        }
        *reinterpret_cast<uint4*>(khi + bi * 16) = *reinterpret_cast<const uint4*>(h);
        *reinterpret_cast<uint4*>(khi + bi * 16 + 8) = *reinterpret_cast<const uint4*>(h + 8);
        *reinterpret_cast<uint4*>(klo + bi * 16) = *reinterpret_cast<const uint4*>(lo);
        *reinterpret_cast<uint4*>(klo + bi * 16 + 8) = *reinterpret_cast<const uint4*>(lo + 8);
        decode_block(vraw, L, tok, half * 4 + bi, cen_cos, cen_sin, y);
#pragma unroll
        for (int i = 0; i < 16; ++i) h[i] = __float2half_rn(live ? y[i] : 0.f);
        *reinterpret_cast<uint4*>(vhi + bi * 16) = *reinterpret_cast<const uint4*>(h);
        *reinterpret_cast<uint4*>(vhi + bi * 16 + 8) = *reinterpret_cast<const uint4*>(h + 8);
      }
    }
    __syncthreads();
    // ---- S = Q' K_hat^T for this warp's 16 rows x 64 tokens
    float sacc[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
    {
      const uint32_t a_off = (uint32_t)((warp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1)) * kPfStride + 8 * (lane >> 4)) * 2;
      const uint32_t b_off = (uint32_t)(((lane & 7) + 8 * (lane >> 4)) * kPfStride + 8 * ((lane >> 3) & 1)) * 2;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t ah[4], al[4];
        pf_ldsm4(sb + kPfQhi + a_off + ks * 32, ah);
        pf_ldsm4(sb + kPfQlo + a_off + ks * 32, al);
#pragma unroll
        for (int np = 0; np < 4; ++np) {   // two 8-token tiles at a time
          uint32_t bh[4], bl[4];
          pf_ldsm4(sb + kPfKhi + b_off + np * 16 * kPfStride * 2 + ks * 32, bh);
          pf_ldsm4(sb + kPfKlo + b_off + np * 16 * kPfStride * 2 + ks * 32, bl);
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            mma_16816(sacc[2 * np + t], al[0], al[1], al[2], al[3], bh[2 * t], bh[2 * t + 1]);   // small terms first
            mma_16816(sacc[2 * np + t], ah[0], ah[1], ah[2], ah[3], bl[2 * t], bl[2 * t + 1]);
            mma_16816(sacc[2 * np + t], ah[0], ah[1], ah[2], ah[3], bh[2 * t], bh[2 * t + 1]);
          }
        }
      }
    }
    // ---- causal mask and online softmax (log2 domain); a thread holds rows gq and gq + 8, tokens 8 nt + 2 cq + {0, 1}
    uint32_t pa[4][4];   // P as A fragments of the value MMAs: [16-token step][a0..a3]
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      float mx = -CUDART_INF_F;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int tok = jb * kTokenBlock + nt * 8 + 2 * cq + e;
          float& s = sacc[nt][2 * i + e];
          s = tok < vis[i] ? s : -CUDART_INF_F;
          mx = fmaxf(mx, s);
        }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run[i], mx);
      const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;       // nothing visible yet: every p is 0
      const float corr = fast_exp2(m_run[i] - m_use);                 // 0 while m_run is -inf
      m_run[i] = m_new;
      float sum = 0.f;
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const float p0 = fast_exp2(sacc[nt][2 * i] - m_use), p1 = fast_exp2(sacc[nt][2 * i + 1] - m_use);
        sum += p0 + p1;
        pa[nt >> 1][i + 2 * (nt & 1)] = as_u32(__floats2half2_rn(p0, p1));
      }
      l_run[i] = l_run[i] * corr + sum;
#pragma unroll
      for (int nt = 0; nt < 16; ++nt) {
        oacc[nt][2 * i] *= corr;
        oacc[nt][2 * i + 1] *= corr;
      }
    }
    // ---- O += P V_hat
    {
      const uint32_t v_off = (uint32_t)(((lane & 7) + 8 * ((lane >> 3) & 1)) * kPfStride + 8 * (lane >> 4)) * 2;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk)
#pragma unroll
        for (int np = 0; np < 8; ++np) {   // two 8-coordinate tiles at a time
          uint32_t bv[4];
          pf_ldsm4t(sb + kPfV + v_off + kk * 16 * kPfStride * 2 + np * 32, bv);
          mma_16816(oacc[2 * np], pa[kk][0], pa[kk][1], pa[kk][2], pa[kk][3], bv[0], bv[1]);
          mma_16816(oacc[2 * np + 1], pa[kk][0], pa[kk][1], pa[kk][2], pa[kk][3], bv[2], bv[3]);
        }
    }
  }
  // ---- normalise, un-rotate by S^T, store
  __syncthreads();
  float* osm = reinterpret_cast<float*>(smem + kPfKhi);
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    float l = l_run[i];
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    const float inv = l > 0.f ? 1.f / l : 0.f;
    const int r = warp * 16 + gq + 8 * i;
#pragma unroll
    for (int nt = 0; nt < 16; ++nt)
      *reinterpret_cast<float2*>(osm + r * kPfOStride + nt * 8 + 2 * cq) = make_float2(oacc[nt][2 * i] * inv, oacc[nt][2 * i + 1] * inv);
    if (cq == 0 && r < n_rows && l <= 0.f) set_status(a.status, PQ_ERR_EMPTY);   // a query that sees no token: zeros
  }
  __syncthreads();
  {
    float acc[kPfRows];
#pragma unroll
    for (int r = 0; r < kPfRows; ++r) acc[r] = 0.f;
    const float4* srow = reinterpret_cast<const float4*>(a.S + tid * 128);   // x_hat_i = sum_j y_hat_j S[i][j]: thread = i
    for (int j0 = 0; j0 < 128; j0 += 4) pf_rank4(acc, osm, kPfOStride, j0, __ldg(srow + (j0 >> 2)));
    for (int r = 0; r < n_rows; ++r) {
      const int64_t o = row_index(r) + tid;
      if (a.io_dtype == PQ_DTYPE_BF16) reinterpret_cast<__nv_bfloat16*>(a.out)[o] = __float2bfloat16(acc[r]);
      else reinterpret_cast<float*>(a.out)[o] = acc[r];
    }
  }
}

}  // namespace pq
