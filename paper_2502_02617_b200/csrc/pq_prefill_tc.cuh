// Multi-query attention over the packed cache on the 5th-generation tensor cores, head_dim 128 (included by
// pq_decode.cu).  Same computation as pq_prefill.cuh -- the last n_q positions of a sequence attend causally to the
// cached tokens (Eq. 2 / Eq. 3) -- for chunks that fill 128 rows = (128 / g) queries x the g query heads of a kv head.
//
// A CTA of sixteen warps owns 128 rows of one (kv head, sequence) and loops over the 64-token blocks its queries may
// see; two CTAs with consecutive query blocks run as a pair on one 256-row MMA (see prefill_tc_kernel):
//   * warps 4-14 ("decoders") copy the packed K and V block with cp.async, DeQuant it (Algorithm 1 by the table
//     lookups of the decode kernel: per 4-coordinate sub-block one entry for levels 4-2 and one for the two level-1
//     pairs, fp16 with error-free residuals) and write the tensor-core operands into shared memory as
//     128-byte-swizzled tiles of 64-coordinate rows: per coordinate half the fp16 values of the tokens followed by
//     their fp16 residuals (ONE K-major B operand: the contraction runs over the coordinates, the rows are
//     (value | residual, token)), and V_hat as fp16 values [token][64 coordinates] x two halves (an MN-major B
//     operand: the contraction runs over the tokens); four stages, so the decoders run ahead of the MMAs.
//     The lookups deliver coordinates (4s, 4s+2 | 4s+1, 4s+3); K_hat keeps that order and Q' is stored in the same
//     one (the contraction does not care), V_hat is put back in natural order by two byte permutes per sub-block;
//   * one thread of warp 15 issues the MMAs: [Q' K_hi^T | Q' K_lo^T] = (Q'lo + Q'hi) [K_hi | K_lo]^T (N = 128, eight
//     k-steps per term) into one of two 128-column accumulators in tensor memory, and O += P_j V_hat (N = 128, four
//     k-steps) into a 128-column accumulator.  The A operands live in tensor memory too (Q' hi and lo, written
//     once; P_j, written by the row owners), the B operands are read from shared memory by the tensor core itself:
//     no warp re-reads a tile (the register-fragment kernel spends 70 % of the shared-memory pipe on exactly that);
//   * warps 0-3 ("row owners": tensor-memory lane = row = thread) read the scores with tcgen05.ld, add the value and
//     residual halves, apply the causal mask and the online softmax in the log2 domain without any shuffle (a thread
//     owns its whole row), and write P_j in fp16 over the first columns of the accumulator the scores came from, as
//     the A operand of the value MMA.  The running maximum is updated lazily: only when a score exceeds it by more
//     than 8 is the output accumulator rescaled (tcgen05.ld / multiply / tcgen05.st by the row's owner, after the
//     previous value MMA has completed); otherwise p <= 2^8 stays well inside fp16.
// Q' = (Q S) * scale * log2(e) is formed once per CTA in float32 and kept as fp16 value + residual; the output is
// normalised and rotated back by S^T in float32 when the CTA ends.  All hand-offs are mbarriers (decoded stage
// full, scores full, P full, value MMA done = stage free); every wait is bounded, and a wait that gives up makes
// every role leave its loop, after which the CTA (the pair) drains its copies and MMAs, releases tensor memory and
// records PQ_ERR_TIMEOUT.
#pragma once

#include "pq_tc_common.cuh"

namespace pq {


constexpr int kPtThreads = 512;   // warps 0-3 row owners, 4-14 decoders, 15 the MMA issuer (registers are allocated per four warps)
constexpr int kPtDecoders = 352;
constexpr int kPtRawBufs = 3;
constexpr int kPtRows = 128;
constexpr int kPtStages = 4;                        // decoded (K_hat hi, K_hat lo, V_hat^T) blocks in flight
constexpr int kPtKBytes = 64 * 128 * 2;             // K_hat hi or lo of a block: two k-halves of 64 tokens x 128 bytes
constexpr int kPtVBytes = 64 * 128 * 2;             // V_hat of a block: two coordinate halves of 64 tokens x 128 bytes
constexpr int kPtStageBytes = 2 * kPtKBytes + kPtVBytes;
constexpr int kPtSmKv = 0;                          // the stages; also q, Q' at the start and O at the end
constexpr int kPtSmRaw = kPtSmKv + kPtStages * kPtStageBytes;   // three packed (K block, V block) buffers
constexpr int kPtSmTab = kPtSmRaw + kPtRawBufs * kPfRawBytes;   // u_tab[4][64], t1p_hi[256], t1p_lo[256] of Tables (8 bytes per entry)
constexpr int kPtSmBar = kPtSmTab + 6144;           // kv_full[S], pv_done[S], s_full[2], (unused)[2], p_full[2], p_free[2], drain
constexpr int kPtSmMisc = kPtSmBar + 16 * kPtStages + 80;   // tensor-memory base, abort flag
constexpr int kPtSmTotal = kPtSmMisc + 32 + 1024;   // + slack for 1024-byte alignment
constexpr int kPtOStride = 132;                     // floats per row of the output staging
constexpr int kPtQStride = 136;                     // halves per row of the Q' staging (rows 16 bytes apart mod 128)
// tensor-memory columns: two score accumulators of 128 (64 tokens x key value and residual; P_j, two fp16 per column,
// later takes the first 32 columns of the accumulator it came from), the output accumulator, Q' hi and lo
constexpr uint32_t kPtTmS = 0, kPtTmO = 256, kPtTmQhi = 384, kPtTmQlo = 448;
static_assert(kPtSmTotal <= 227 * 1024, "shared memory of one CTA");
static_assert(128 * kPtOStride * 4 <= kPtStages * kPtStageBytes, "float32 output staging fits in the stages");
static_assert(128 * 128 * 4 + 2 * 128 * kPtQStride * 2 <= kPtStages * kPtStageBytes, "q and Q' staging fit in the stages");
static_assert(kPtStageBytes % 1024 == 0, "swizzled tiles start on 1024-byte boundaries");

// acc[r] += sum_k x[r][k0 + k] * w[k] for 64 rows of a float32 tile in shared memory (the same address in every thread)
__device__ __forceinline__ void pt_rank4(float (&acc)[64], const float* x, int ld, int k0, float4 w) {
#pragma unroll
  for (int r = 0; r < 64; ++r) {
    const float4 v = *reinterpret_cast<const float4*>(x + r * ld + k0);
    acc[r] = fmaf(v.x, w.x, fmaf(v.y, w.y, fmaf(v.z, w.z, fmaf(v.w, w.w, acc[r]))));
  }
}

__device__ __forceinline__ void pt_sts128(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ void pt_sts16(uint32_t addr, __half v) {
  asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(__half_as_ushort(v)) : "memory");
}

__device__ __forceinline__ uint32_t pt_mapa(uint32_t addr, uint32_t cta_rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(cta_rank));
  return r;
}
__device__ __forceinline__ void pt_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrival on a barrier of the even CTA of the pair (`bar` = its shared::cluster address, from mapa).  What the arriving
// warp wrote before is read by its own SM's tensor core (operands in shared memory after fence.proxy.async, P in
// tensor memory after tcgen05.wait::st), which the even CTA's MMA triggers after it has seen the arrival.
__device__ __forceinline__ void pt_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}

// (a0, a1) + (b0, b1) as one packed float32 instruction
__device__ __forceinline__ void pt_add2(float a0, float a1, float b0, float b1, float& c0, float& c1) {
  asm("{\n\t.reg .b64 a, b, c;\n\t"
      "mov.b64 a, {%2, %3};\n\t"
      "mov.b64 b, {%4, %5};\n\t"
      "add.rn.f32x2 c, a, b;\n\t"
      "mov.b64 {%0, %1}, c;\n\t}"
      : "=f"(c0), "=f"(c1)
      : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}

// Named-barrier OR over `n_threads` threads (also a barrier).
__device__ __forceinline__ bool pt_bar_or(int bar_id, int n_threads, bool v) {
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

// kPair: the CTAs of two consecutive query blocks of one (kv head, sequence) form a cluster and run ONE 256-row MMA per
// step (cta_group::2, issued by a thread of the even CTA): every CTA keeps its own 128 rows of Q', S, P and O in its own
// tensor memory and supplies half of each B operand from its own shared memory -- the keys of 32 of the block's 64
// tokens, the values of 64 of the 128 coordinates -- so a CTA decodes half a block per block and no decoded data
// crosses between the CTAs.  The even CTA's barriers collect the arrivals of both CTAs' decoder and row-owner warps;
// its commits are multicast to both CTAs' barriers.
template <bool kPair>
__global__ void __launch_bounds__(kPtThreads, 1) prefill_tc_kernel(DecodeArgs a, int n_q) {
  extern __shared__ uint8_t pt_smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(pt_smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sb = tc_smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = a.n_q_heads / a.n_kv_heads;
  const int qb_rows = kPtRows / g;                      // queries of a CTA
  const int q0 = blockIdx.x * qb_rows, hk = blockIdx.y, b = blockIdx.z;
  const int n_rows = max(0, min(qb_rows, n_q - q0)) * g;   // rows in use; row r = (query q0 + r / g, head hk * g + r % g);
                                                           // none in the CTA that only completes a pair
  uint32_t crank = 0;
  if (kPair) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
  const bool leader = crank == 0;   // the CTA whose thread issues the MMAs and whose barriers collect the arrivals
  // Per-CTA shapes of the B operands: keys of kKTok tokens (two coordinate halves), values of 64 tokens x kVHalves x 64
  // coordinates.  A key tile holds, for each half of the coordinates, the fp16 values of the kKTok tokens followed by their residuals:
  // one B operand of 2 kKTok rows, so one MMA gives the products with both.
  constexpr int kKTok = kPair ? 32 : 64, kKLo = kKTok * 128, kKHalf = 2 * kKLo, kKTile = 2 * kKHalf, kVHalves = kPair ? 1 : 2;
  constexpr int kStage = kKTile + kVHalves * 8192;
  // columns of a score accumulator: tokens [32 c, 32 c + 32) times the values at kColHi(c), times the residuals at kColLo(c)
  // (a pair's accumulator columns follow the two CTAs' operand rows)
  auto col_hi = [](int c) -> uint32_t { return kPair ? 64u * c : 32u * c; };
  auto col_lo = [](int c) -> uint32_t { return kPair ? 64u * c + 32u : 64u + 32u * c; };
  // packed blocks in flight: the copy of block jb + kRawBufs - 1 starts when block jb is decoded.  A pair's stages are
  // half as large: its packed buffers follow them inside the stage area.
  constexpr int kRawBufs = kPair ? 6 : kPtRawBufs;
  constexpr int kSmRaw = kPair ? kPtSmKv + kPtStages * kStage : kPtSmRaw;
  static_assert(!kPair || kSmRaw + kRawBufs * kPfRawBytes <= kPtSmRaw, "a pair's packed buffers fit behind its stages");
  const int len = a.lens[b];
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kPtSmMisc + 4);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kPtSmMisc);
  uint2* tab = reinterpret_cast<uint2*>(smem + kPtSmTab);
  const uint32_t bar_kv = sb + kPtSmBar, bar_pv = bar_kv + 8 * kPtStages, bar_sfull = bar_pv + 8 * kPtStages,
                 bar_pfull = bar_sfull + 32, bar_pfree = bar_pfull + 16, bar_drain = bar_pfree + 16;
  auto row_index = [&](int r) -> int64_t {               // offset of row r in q / out ([batch][n_q][n_q_heads][128])
    return (((int64_t)b * n_q + q0 + r / g) * a.n_q_heads + hk * g + r % g) * 128;
  };
  if (tid == 0) {
    for (int i = 0; i < kPtStages; ++i) {
      tc_mbar_init(bar_kv + 8 * i, (kPair ? 2 : 1) * kPtDecoders / 32);   // one arrival per decoder warp (of both CTAs)
      tc_mbar_init(bar_pv + 8 * i, 1);                  // tcgen05.commit after the value MMA that read the stage
    }
    for (int i = 0; i < 2; ++i) {
      tc_mbar_init(bar_sfull + 8 * i, 1);   // tcgen05.commit
      tc_mbar_init(bar_pfull + 8 * i, kPair ? 8 : 4);
      tc_mbar_init(bar_pfree + 8 * i, 1);   // tcgen05.commit after the value MMA: the output accumulator holds the block
    }
    tc_mbar_init(bar_drain, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < 768; i += kPtThreads)
    tab[i] = i < 256 ? a.tables->u_tab[i >> 6][i & 63] : (i < 512 ? a.tables->t1p_hi[i - 256] : a.tables->t1p_lo[i - 512]);
  if (warp == 15) {   // in a pair: the same warp of both CTAs, the same destination offset
    if (kPair) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(sb + kPtSmMisc) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(sb + kPtSmMisc) : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  // ---- Q' = (Q S) * scale * log2(e) as fp16 value + residual (threads 0..255: column, half of the rows), staged in shared
  // memory and then written to tensor memory by the row owners (lane = row, two k values per column)
  __half* qhi_s = reinterpret_cast<__half*>(smem + kPtSmKv + 128 * 128 * 4);
  __half* qlo_s = qhi_s + 128 * kPtQStride;
  {
    float* qs = reinterpret_cast<float*>(smem + kPtSmKv);
    for (int i = tid; i < kPtRows * 128; i += kPtThreads) {
      const int r = i >> 7, k = i & 127;
      float v = 0.f;
      if (r < n_rows)
        v = a.io_dtype == PQ_DTYPE_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.q)[row_index(r) + k])
                                        : reinterpret_cast<const float*>(a.q)[row_index(r) + k];
      qs[i] = v;
    }
    __syncthreads();
    if (tid < 256) {
      const int j = tid & 127, rh = tid >> 7;
      float acc[64];
#pragma unroll
      for (int r = 0; r < 64; ++r) acc[r] = 0.f;
      for (int k0 = 0; k0 < 128; k0 += 4) {
        const float4 w = make_float4(__ldg(a.S + (k0 + 0) * 128 + j), __ldg(a.S + (k0 + 1) * 128 + j),
                                     __ldg(a.S + (k0 + 2) * 128 + j), __ldg(a.S + (k0 + 3) * 128 + j));
        pt_rank4(acc, qs + rh * 64 * 128, 128, k0, w);
      }
      const float f = a.scale * 1.4426950408889634f;
      // coordinate j sits at position (j & ~3) | (0, 2, 1, 3)[j & 3] of the contraction index: the order the decoders write
      const int jp = (j & ~3) | ((j & 1) << 1) | ((j >> 1) & 1);
#pragma unroll
      for (int r = 0; r < 64; ++r) {
        const int row = rh * 64 + r;
        const float v = acc[r] * f;
        const __half h = __float2half_rn(v);
        qhi_s[row * kPtQStride + jp] = h;
        qlo_s[row * kPtQStride + jp] = __float2half_rn(v - __half2float(h));
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();   // Q' is staged, tensor memory is allocated
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  if (warp < 4) {
    const uint32_t trow = tmem_base + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {   // hi columns 0..31, 32..63, then lo
      const uint4* src = reinterpret_cast<const uint4*>((c < 2 ? qhi_s : qlo_s) + tid * kPtQStride + 64 * (c & 1));
      uint32_t v[32];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint4 w = src[i];
        v[4 * i] = w.x; v[4 * i + 1] = w.y; v[4 * i + 2] = w.z; v[4 * i + 3] = w.w;
      }
      tc_st32u(trow + (c < 2 ? kPtTmQhi : kPtTmQlo) + 32 * (c & 1), v);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __syncthreads();   // Q' is in tensor memory; the staging is dead: the stages may be written
  if (kPair) pt_cluster_sync();   // both CTAs' barriers are initialised and both halves of Q' are in place
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  // the last query of the CTA (of the pair) sees the most
  const int q_last = min(n_q, ((kPair ? (int)(blockIdx.x | 1u) : (int)blockIdx.x) + 1) * qb_rows) - 1;
  const int vis_cta = max(0, len - (n_q - 1 - q_last));
  const int n_blocks = (vis_cta + kTokenBlock - 1) / kTokenBlock;
  // where this CTA's warps announce themselves: the barriers of the even CTA
  const uint32_t to_leader = kPair ? pt_mapa(sb, 0u) - sb : 0u;   // + a local shared address: that place in the even CTA (cluster window)
  const Layout L = make_layout(128, a.pg.page_tokens);

  float l_run = 0.f;   // row owners: denominator of this thread's row
  if (warp < 4) {
    // ================= row owners: softmax of row `tid` =================
    const int r = tid;
    const int vis = r < n_rows ? max(0, len - (n_q - 1 - (q0 + r / g))) : 0;
    const uint32_t trow = tmem_base + ((uint32_t)(warp * 32) << 16);
    float m_run = -CUDART_INF_F;
    const int vis_min = __reduce_min_sync(0xffffffffu, vis);
    for (int jb = 0; jb < n_blocks; ++jb) {
      const int t = jb & 1;
      const uint32_t ph = (uint32_t)(jb >> 1) & 1u;
      bool ok = __all_sync(0xffffffffu, tc_mbar_wait(bar_sfull + 8 * t, ph, abort_flag));
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float s[64];
#pragma unroll
      for (int c = 0; c < 2; ++c) {   // Q' K_hi^T + Q' K_lo^T
        float lo[32];
        tc_ld32(trow + t * 128 + col_hi(c), s + 32 * c);
        tc_ld32(trow + t * 128 + col_lo(c), lo);
#pragma unroll
        for (int i = 0; i < 32; i += 2) pt_add2(s[32 * c + i], s[32 * c + i + 1], lo[i], lo[i + 1], s[32 * c + i], s[32 * c + i + 1]);
      }
      // the causal mask touches only the last blocks of a row: one uniform test per warp skips it elsewhere
      if ((jb + 1) * kTokenBlock > vis_min) {
#pragma unroll
        for (int i = 0; i < 64; ++i) s[i] = jb * kTokenBlock + i < vis ? s[i] : -CUDART_INF_F;
      }
      float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};   // four chains: no 64-long dependency
#pragma unroll
      for (int i = 0; i < 64; i += 8) {
#pragma unroll
        for (int c = 0; c < 4; ++c) mx4[c] = fmaxf(mx4[c], fmaxf(s[i + 2 * c], s[i + 2 * c + 1]));
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      // lazy reference: move it only when some score exceeds it by more than 8 (p <= 2^8 otherwise)
      const bool grow = mx > m_run + 8.f || (m_run == -CUDART_INF_F && mx > -CUDART_INF_F);
      if (__any_sync(0xffffffffu, grow)) {
        const float m_new = grow ? mx : m_run;
        const float corr = m_run == -CUDART_INF_F ? 1.f : fast_exp2(m_run - m_new);   // nothing accumulated yet: nothing to scale
        if (jb > 0) {
          // the value MMAs up to block jb - 1 must have completed before the accumulator is touched
          ok = __all_sync(0xffffffffu, tc_mbar_wait(bar_pfree + 8 * ((jb - 1) & 1), (uint32_t)((jb - 1) >> 1) & 1u, abort_flag));
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            float o[32];
            tc_ld32(trow + kPtTmO + 32 * c, o);
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] *= corr;
            tc_st32(trow + kPtTmO + 32 * c, o);
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        }
        l_run *= corr;
        m_run = m_new;
      }
      const float m_use = m_run == -CUDART_INF_F ? 0.f : m_run;   // nothing visible yet: every p is 0
      // P_jb takes the first 32 columns of the accumulator it was computed from (all of it is in registers): the value
      // MMA of block jb - 2, which read them last, was issued before the score MMAs that s_full reported
      float sum8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {   // the store of the first half runs while the second half is computed
        uint32_t pw[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const int i = 32 * hf + 2 * e;
          float x0, x1;
          pt_add2(s[i], s[i + 1], -m_use, -m_use, x0, x1);
          const __half2 p2 = __floats2half2_rn(fast_exp2(x0), fast_exp2(x1));
          const float2 pf = __half22float2(p2);   // the denominator of what the MMA will see
          pt_add2(sum8[2 * (e & 3)], sum8[2 * (e & 3) + 1], pf.x, pf.y, sum8[2 * (e & 3)], sum8[2 * (e & 3) + 1]);
          pw[e] = as_u32(p2);
        }
        tc_st16u_nowait(trow + kPtTmS + 128 * t + 16 * hf, pw);
      }
      l_run += ((sum8[0] + sum8[1]) + (sum8[2] + sum8[3])) + ((sum8[4] + sum8[5]) + (sum8[6] + sum8[7]));
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        if (kPair) pt_arrive_cluster(bar_pfull + 8 * t + to_leader);
        else tc_mbar_arrive(bar_pfull + 8 * t);
      }
    }
  } else if (warp < 15) {
    // ================= decoders: packed block -> K_hat hi / lo, V_hat^T =================
    const int dt = tid - 128;
    auto fetch = [&](int jb) {  // packed K block and V block of token-block jb -> raw buffer jb % kRawBufs (one group per call)
      if (jb < n_blocks) {
        const uint8_t* src = a.cache + kv_block_pair_offset(L, a.pg, a.n_kv_heads, b, hk, jb, a.status);
        const uint32_t dst = sb + kSmRaw + (jb % kRawBufs) * kPfRawBytes;
        for (int i = dt; i < kPfRawBytes / 16; i += kPtDecoders) pf_cp16(dst + 16 * i, src + 16 * i);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    for (int i = 0; i < kRawBufs - 1; ++i) fetch(i);
    for (int jb = 0; jb < n_blocks; ++jb) {
      const int st = jb % kPtStages;
      asm volatile("cp.async.wait_group %0;" ::"n"(kRawBufs - 2) : "memory");   // this thread's part of block jb has landed
      // stage st is free once the value MMA of block jb - kPtStages has completed (it also covers that block's score MMAs)
      bool ok = true;
      if (jb >= kPtStages) ok = tc_mbar_wait(bar_pv + 8 * st, (uint32_t)(jb / kPtStages - 1) & 1u, abort_flag);
      // The raw block has landed for all decoder threads, and all of them have finished the previous block (the copy
      // that the next iteration starts goes into the buffer that block was read from); the decision to go on is
      // taken together.
      if (pt_bar_or(1, kPtDecoders, !ok)) break;
      fetch(jb + kRawBufs - 1);   // into the buffer of block jb - 1
      // all accesses below are shared-memory instructions on 32-bit addresses
      const uint32_t kraw = sb + kSmRaw + (jb % kRawBufs) * kPfRawBytes;
      const uint32_t stage = sb + kPtSmKv + st * kStage;
      const uint32_t utab = sb + kPtSmTab, t1hi = utab + 2048, t1lo = utab + 4096;
      // An item is one 16-byte chunk of an operand row: (K | V, 16-block, half of the block, token).  The 32 items of a
      // warp are 8 tokens x the 4 blocks of one coordinate half: the code words of a warp then sit in few shared-
      // memory rows (the level-1 plane is 32 bytes per token: 32 tokens with one block would be an 8-way bank
      // conflict, this is 2-way), and 8 lanes with one block and 8 tokens still store to 8 distinct swizzled
      // positions.  A CTA of a pair takes the keys of tokens 32 rank .. 32 rank + 31 and the values of blocks
      // 4 rank .. 4 rank + 3 (coordinates 64 rank .. 64 rank + 63) of all 64 tokens.
      constexpr int kItems = kPair ? 1024 : 2048;
#pragma unroll
      for (int item = dt; item < kItems; item += kPtDecoders) {
        const int iw = item >> 5;   // the warp's item group
        int kv, half, sp, tg;
        if (kPair) {
          kv = iw >> 4;
          if (kv == 0) { half = (iw >> 3) & 1; sp = (iw >> 2) & 1; tg = (iw & 3) + 4 * (int)crank; }
          else { half = (int)crank; sp = (iw >> 3) & 1; tg = iw & 7; }
        } else {
          kv = iw >> 5; half = (iw >> 4) & 1; sp = (iw >> 3) & 1; tg = iw & 7;
        }
        const int blk = 4 * half + (lane >> 3), tok = 8 * tg + (lane & 7), bi = blk & 3;
        const bool live = jb * kTokenBlock + tok < len;   // stale bytes past the sequence end must not reach the MMAs
        const uint32_t raw = kraw + kv * 62 * kTokenBlock;
        const uint32_t l1 = lds16(raw + tok * 32 + blk * 4 + sp * 2);               // the two level-1 bytes of this half
        const uint32_t c2 = lds8(raw + kO2 + tok * 8 + blk) >> (4 * sp);
        const uint32_t c3 = lds8(raw + kO3 + tok * 4 + (blk >> 1)) >> (4 * (blk & 1) + 2 * sp);
        const uint32_t c4 = (lds16(raw + kO4 + tok * 2) >> (2 * blk)) & 3u;
        const uint32_t rbits = live ? lds16(raw + kORad + tok * 16 + blk * 2) : 0u;
        const __half2 r2 = as_h2(rbits | (rbits << 16));
        const uint32_t c34 = ((c3 & 3u) << 2) | (c4 << 4);
        uint32_t hw[4], lw[4];
#pragma unroll
        for (int q = 0; q < 2; ++q) {   // sub-block 2 sp + q: coordinates 4 (2 sp + q) .. + 3 of the block
          const uint32_t iu = ((c2 >> (2 * q)) & 3u) | c34;
          const uint2 uu = lds64(utab + (uint32_t)(2 * sp + q) * 512u + iu * 8u);
          const uint32_t e = ((l1 >> (8 * q)) & 0xFFu) * 8u;
          const uint2 th = lds64(t1hi + e);
          const __half2 u_hi = __hmul2(r2, as_h2(uu.x));
          const __half2 xh = __hmul2(u_hi, as_h2(th.x)), yh = __hmul2(u_hi, as_h2(th.y));   // coordinates (4s, 4s+2), (4s+1, 4s+3)
          if (kv == 0) {
            // the key as an unevaluated sum hi + lo (fp16 fused multiply-adds return the exact residual of a product)
            const uint2 tl = lds64(t1lo + e);
            const __half2 u_lo = __hfma2(r2, as_h2(uu.y), __hfma2(r2, as_h2(uu.x), __hneg2(u_hi)));
            hw[2 * q] = as_u32(xh);
            hw[2 * q + 1] = as_u32(yh);
            lw[2 * q] = as_u32(__hfma2(u_hi, as_h2(tl.x), __hfma2(u_lo, as_h2(th.x), __hfma2(u_hi, as_h2(th.x), __hneg2(xh)))));
            lw[2 * q + 1] = as_u32(__hfma2(u_hi, as_h2(tl.y), __hfma2(u_lo, as_h2(th.y), __hfma2(u_hi, as_h2(th.y), __hneg2(yh)))));
          } else {
            // coordinates in natural order: (4s, 4s+1) = (x.lo, y.lo), (4s+2, 4s+3) = (x.hi, y.hi)
            hw[2 * q] = __byte_perm(as_u32(xh), as_u32(yh), 0x5410);
            hw[2 * q + 1] = __byte_perm(as_u32(xh), as_u32(yh), 0x7632);
          }
        }
        // chunk 2 bi + sp of the row's 64-coordinate half, swizzled by the row
        if (kv == 0) {
          const int row = tok & (kKTok - 1);
          const uint32_t dst = stage + half * kKHalf + row * 128 + (((2 * bi + sp) ^ (row & 7)) << 4);
          pt_sts128(dst, hw[0], hw[1], hw[2], hw[3]);
          pt_sts128(dst + kKLo, lw[0], lw[1], lw[2], lw[3]);
        } else {
          const uint32_t dst = stage + kKTile + (kPair ? 0 : half * 8192) + tok * 128 + (((2 * bi + sp) ^ (tok & 7)) << 4);
          pt_sts128(dst, hw[0], hw[1], hw[2], hw[3]);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) {
        if (kPair) pt_arrive_cluster(bar_kv + 8 * st + to_leader);
        else tc_mbar_arrive(bar_kv + 8 * st);
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  } else if (tid == 480 && leader) {
    // ================= MMA issuer =================
    // the value operand is MN-major: [token][coordinate] rows of 64 coordinates, the two coordinate halves 8192 bytes apart
    // (in a pair: one half per CTA)
    constexpr uint32_t kM = kPair ? 256 : 128;
    constexpr uint32_t idesc_qk = tc_idesc(false, kM, 128);   // 64 tokens x (value, residual)
    constexpr uint32_t idesc_pv = tc_idesc(false, kM, 128) | (1u << 16);
    auto mma = [&](uint32_t d, uint32_t a_t, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
      if (kPair) tc_mma_ts_pair(d, a_t, bdesc, idesc, acc);
      else tc_mma_ts(d, a_t, bdesc, idesc, acc);
    };
    auto commit = [&](uint32_t bar) {   // in a pair: arrives on both CTAs' barriers
      if (kPair) tc_commit_pair(bar);
      else tc_commit(bar);
    };
    uint64_t vdesc_hi = (uint64_t)(1024 >> 4) << 32;   // stride between groups of 8 tokens
    vdesc_hi |= (uint64_t)1 << 46;
    vdesc_hi |= (uint64_t)2 << 61;
    const uint32_t vdesc_lbo = (8192u >> 4) << 16;     // leading-dimension offset: the next 64 coordinates
    const uint64_t desc_hi = tc_smem_desc(0u) & 0xFFFFFFFF00000000ull;
    auto issue_pv = [&](int jb) -> bool {   // O (+)= P_jb V_hat_jb
      const int t = jb & 1, st = jb % kPtStages;
      if (!tc_mbar_wait(bar_pfull + 8 * t, (uint32_t)(jb >> 1) & 1u, abort_flag)) return false;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t v_lo = (((sb + kPtSmKv + st * kStage + kKTile) & 0x3FFFFu) >> 4) | vdesc_lbo;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk)   // 16 tokens = 8 columns of P = 16 rows of 128 bytes of V_hat per step
        mma(tmem_base + kPtTmO, tmem_base + kPtTmS + 128 * t + 8 * kk, vdesc_hi | (v_lo + 128 * kk), idesc_pv, (jb > 0 || kk > 0) ? 1u : 0u);
      commit(bar_pv + 8 * st);     // the stage is free
      commit(bar_pfree + 8 * t);   // the output accumulator holds block jb
      return true;
    };
    bool ok = true;
    for (int jb = 0; jb < n_blocks && ok; ++jb) {
      const int t = jb & 1;
      // The value MMA of the previous block frees its stage for the decoders: it goes first if its P is ready, so that
      // it does not queue behind this block's score MMAs; otherwise the score MMAs go first and keep the tensor
      // core busy while the softmax of the previous block finishes.
      bool pv_issued = jb == 0;
      if (!pv_issued && tc_mbar_test(bar_pfull + 8 * ((jb - 1) & 1), (uint32_t)((jb - 1) >> 1) & 1u)) {
        ok = issue_pv(jb - 1);
        pv_issued = true;
        if (!ok) break;
      }
      const int st = jb % kPtStages;
      ok = tc_mbar_wait(bar_kv + 8 * st, (uint32_t)(jb / kPtStages) & 1u, abort_flag);
      // accumulator t is free: its scores were read before P_{jb-2} was announced, and the value MMA that read
      // P_{jb-2} from its columns was issued in the previous iteration (MMAs of one thread execute in order)
      if (ok && (a.debug & 2u) && (blockIdx.x | blockIdx.y | blockIdx.z) == 0 && jb == min(2, n_blocks - 1)) {
        *abort_flag = 1;   // test hook: this wait counts as failed (what it waited for has arrived)
        ok = false;
      }
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t kb = (uint32_t)tc_smem_desc(sb + kPtSmKv + st * kStage);
      // [Q' K_hi^T | Q' K_lo^T] = (Q'lo + Q'hi) [K_hi | K_lo]^T, the small term first (its product with K_lo is
      // below float32 resolution and rides along); k-step ks: half ks >> 2, 32 bytes per step
#pragma unroll
      for (int term = 0; term < 2; ++term) {
        const uint32_t qa = tmem_base + (term == 0 ? kPtTmQlo : kPtTmQhi);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {   // 16 k values = 8 columns of Q' per step
          const uint32_t koff = (uint32_t)((ks >> 2) * kKHalf + (ks & 3) * 32) >> 4;
          mma(tmem_base + kPtTmS + t * 128, qa + 8 * ks, desc_hi | (kb + koff), idesc_qk, (term | ks) ? 1u : 0u);
        }
      }
      commit(bar_sfull + 8 * t);
      if (!pv_issued) ok = issue_pv(jb - 1);
    }
    if (ok && n_blocks > 0) ok = issue_pv(n_blocks - 1);
    if (n_blocks > 0) {
      // every MMA issued above has completed when this commit arrives (nothing was issued without blocks: no commit)
      commit(bar_drain);
      bool drained = false;
      for (int i = 0; i < (1 << 20) && !drained; ++i) {
        drained = tc_mbar_try(bar_drain, 0);
        if (!drained) __nanosleep(32);
      }
      if (!drained) *abort_flag = 1;
    }
    if (kPair && *abort_flag)   // tell the other CTA, whose warps wait for commits that will not come
      asm volatile("st.relaxed.cluster.shared::cluster.u32 [%0], %1;" ::"r"(sb + kPtSmMisc + 4 + (pt_mapa(sb, 1u) - sb)), "r"(1u) : "memory");
  } else if (kPair && tid == 480) {
    // the odd CTA of a pair: its operands are read until the even CTA's last commit arrives here too
    if (n_blocks > 0) {
      bool drained = false;
      for (int i = 0; i < kTcSpin && !drained && !*abort_flag; ++i) {
        drained = tc_mbar_try(bar_drain, 0);
        if (!drained) __nanosleep(64);
      }
      if (!drained) *abort_flag = 1;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();   // all MMAs have completed (the issuer waited for its last commit), the stages are idle
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const bool aborted = *abort_flag != 0;
  // ---- normalise, un-rotate by S^T, store
  float* osm = reinterpret_cast<float*>(smem + kPtSmKv);
  if (warp < 4) {
    const int r = tid;
    const float inv = (!aborted && l_run > 0.f) ? 1.f / l_run : 0.f;
    const uint32_t trow = tmem_base + ((uint32_t)(warp * 32) << 16);
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      float o[32];
      if (n_blocks > 0 && !aborted) {
        tc_ld32(trow + kPtTmO + 32 * c, o);
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) o[i] = 0.f;
      }
#pragma unroll
      for (int i = 0; i < 32; i += 4)
        *reinterpret_cast<float4*>(osm + r * kPtOStride + 32 * c + i) = make_float4(o[i] * inv, o[i + 1] * inv, o[i + 2] * inv, o[i + 3] * inv);
    }
    if (r < n_rows && l_run <= 0.f && !aborted) set_status(a.status, PQ_ERR_EMPTY);   // a query that sees no token: zeros
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  }
  __syncthreads();
  // In a pair neither CTA may release tensor memory or leave while the other may still arrive on its barriers or
  // have its operands read: both have drained here.
  if (kPair) pt_cluster_sync();
  if (warp == 15) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (kPair) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
  if (tid == 0 && aborted) set_status(a.status, PQ_ERR_TIMEOUT);
  if (tid < 256 && !aborted) {
    const int i = tid & 127, rh = tid >> 7;   // x_hat_i = sum_j y_hat_j S[i][j]: thread = i, half of the rows
    float acc[64];
#pragma unroll
    for (int r = 0; r < 64; ++r) acc[r] = 0.f;
    const float4* srow = reinterpret_cast<const float4*>(a.S + i * 128);
    for (int j0 = 0; j0 < 128; j0 += 4) pt_rank4(acc, osm + rh * 64 * kPtOStride, kPtOStride, j0, __ldg(srow + (j0 >> 2)));
#pragma unroll
    for (int r = 0; r < 64; ++r) {
      const int row = rh * 64 + r;
      if (row < n_rows) {
        const int64_t o = row_index(row) + i;
        if (a.io_dtype == PQ_DTYPE_BF16) reinterpret_cast<__nv_bfloat16*>(a.out)[o] = __float2bfloat16(acc[r]);
        else reinterpret_cast<float*>(a.out)[o] = acc[r];
      }
    }
  }
}

}  // namespace pq
