// Fast decode-attention kernel for head_dim 128 (included by pq_decode.cu).
//
// Persistent CTAs of 16 warps, each with a contiguous share of the (sequence, kv head) token streams.
// 128-token stages of the packed cache (K block, V block, K block, V block: one contiguous 15872-byte
// bulk copy) stream through a shared-memory ring.  The warps form two groups of 8 that take alternate
// stages; each group has two ring slots and one thread that issues its copies a stage ahead; each warp
// takes one 16-token tile of its group's stage.  (16 warps, not 17: the register file is split over
// four schedulers, and a fifth warp on one of them would cap every thread at 96 registers.)
//
// Per tile a warp
//   * decodes the keys of 16 tokens straight into mma.sync A fragments (fp16, rotated basis) with
//     shared-memory table lookups, and forms S = K_hat q'^T (tokens x heads) on tensor cores,
//   * runs the online softmax on the S fragment (log2 domain, fp32, lazily updated reference),
//   * decodes the values into A fragments (coordinates x (token, element of a decoded pair)) and
//     accumulates O^T += V_hat^T P on tensor cores (fp32 accumulators in registers).
// DeQuant (Algorithm 1) of one 16-coordinate block is a product tree r * t4 * t3 * t2 * t1.
// Levels 4..2 are folded into one table per 4-coordinate sub-block, level 1 is a half2 multiply:
//   u    [4][64][16] sub-block s, index c2_s | c3_(s>>1) << 2 | c4 << 4 -> the multipliers of the
//                    sub-block's two level-1 pairs as (half2 values, half2 rounding residuals)
//   t1hi [256][16]   index = one byte of level-1 codes (pair a = 2s | pair b = 2s+1 << 4) -> (cos a, cos b), (sin a, sin b)
//                    in fp16: the half2 (u_a, u_b) of the table above multiplies them element-wise
//   t1lo [256][16]   the fp16 rounding residuals of the same entries
// All are replicated 16 times so that every lane of a half-warp reads its own banks.
// Values use the fp16 parts only.  Keys feed the softmax exponent, where an fp16-rounded operand
// costs ~3x its relative error in the output, so they are decoded as an unevaluated sum hi + lo
// (error-free fp16 transformations with fused multiply-adds) and contracted with two MMAs.
#pragma once

namespace pq {

constexpr int kFastConsumerWarps = 16;
constexpr int kFastThreads = kFastConsumerWarps * 32;
constexpr int kStageTokens = 2 * kTokenBlock;       // 128
constexpr int kBlockBytes128 = 62 * kTokenBlock;    // 3968: one K or V token-block at d = 128
constexpr int kStageBytes = 4 * kBlockBytes128;     // 15872
constexpr int kStages = 4;                          // two per group of 8 warps
constexpr int kSpinLimit = 1 << 22;

// shared-memory map (bytes)
constexpr int kSmT1p = 0;                             // 256 * 16 * 8 = 32768
constexpr int kSmT1lo = kSmT1p + 256 * 16 * 8;        // 32768
constexpr int kSmU = kSmT1lo + 256 * 16 * 8;          // 4 * 64 * 16 * 8 = 32768
constexpr int kSmBar = kSmU + 4 * 64 * 16 * 8;        // full[4], empty[4] : 64
constexpr int kSmFlags = kSmBar + 64;                 // abort flag, is_last, n_segs, first_rank : 16
constexpr int kSmSegs = kSmFlags + 16;                // Segment[32] : 768
constexpr int kSmQ = kSmSegs + 768;                   // q (fp32) [8][128], q' fp16 value [8][128], q' fp16 residual [8][128] : 8192
constexpr int kSmRing = (kSmQ + 8192 + 127) / 128 * 128;
// after the main loop the ring is reused for the cross-warp merge: 16 warps x 8 heads x (kMrgStride + 2) floats
constexpr int kMrgStride = 136;  // floats per (warp, head) row of the merge buffer (136 = 128 + 8: heads 8 banks apart)
constexpr int kMergeBytes = 16 * 8 * kMrgStride * 4 + 16 * 8 * 2 * 4;  // also >= combine_smem_floats(8, 128, 160) * 4
constexpr int kSmUsed = kSmRing + (kStages * kStageBytes > kMergeBytes ? kStages * kStageBytes : kMergeBytes);
// The tables start on a 32 KB boundary of the shared window, so that a table address is the OR of
// disjoint bit fields (base | lane replica | index) and needs no addition; the launch asks for 32 KB
// of slack to place them.
constexpr int kSmAlign = 32768;
constexpr int kSmTotal = kSmUsed + kSmAlign;
static_assert(kSmT1p == 0 && kSmT1lo == 32768 && kSmU == 65536, "table addresses are formed with OR");
static_assert(kSmRing % 128 == 0, "ring must be 128-byte aligned");

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls (or as soon as another warp gave up) and raises
// the CTA's abort flag, so that a lost copy can never hang the GPU.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if (i > 64) {
      __nanosleep(64);
      if (*abort_flag) return false;
    }
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
template <int kOff>
__device__ __forceinline__ uint32_t lds32i(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(kOff));
  return v;
}
template <int kOff>
__device__ __forceinline__ uint2 lds64i(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2+%3];" : "=r"(v.x), "=r"(v.y) : "r"(addr), "n"(kOff));
  return v;
}
template <int kOff>
__device__ __forceinline__ uint32_t lds16i(uint32_t addr) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1+%2];" : "=h"(v) : "r"(addr), "n"(kOff));
  return v;
}
template <int kOff>
__device__ __forceinline__ uint32_t lds8i(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u8 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(kOff));
  return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t addr) {
  uint16_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds8(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}

// 2^x, x <= 0 or slightly above (ex2.approx: relative error 2^-22; 2^-inf = 0)
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
constexpr float kLazyMax = 8.f;

__device__ __forceinline__ __half2 as_h2(uint32_t v) { return *reinterpret_cast<__half2*>(&v); }
__device__ __forceinline__ uint32_t as_u32(__half2 v) { return *reinterpret_cast<uint32_t*>(&v); }

// D(16x8, f32) += A(16x16, f16, row) * B(16x8, f16, col)
__device__ __forceinline__ void mma_16816(float* d, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// D(16x8, f32) += A(16x8, f16, row) * B(8x8, f16, col)
__device__ __forceinline__ void mma_1688(float* d, uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(b0));
}

// Codes of one 16-coordinate block of one token, prepared for the table lookups.  Entry idx of the
// replicated u table of sub-block s sits at s * 8192 + idx * 128 with idx = c2_s | c3 << 2 | c4 << 4, i.e.
// c2_s -> address bits 7..8, c3 -> bits 9..10, c4 -> bits 11..12; `ub` = table base | lane replica has
// none of these bits set, so the address is an OR (the loads add s * 8192 as an immediate).
struct BlockRef {
  uint32_t l1;        // 8 level-1 codes, code j at bits [4j, 4j+4)
  uint32_t c2;        // 4 level-2 codes in bits 0..7 (higher bits are ignored)
  uint32_t hi0, hi1;  // ub | c4 | level-3 code of sub-blocks 0-1 / 2-3, in address position
  __half2 r2;         // the block radius in both halves
};
__device__ __forceinline__ BlockRef make_block_ref(uint32_t l1, uint32_t c2, uint32_t c3n, uint32_t c4_clean, __half2 r2,
                                                   uint32_t ub) {
  BlockRef b;
  const uint32_t a4 = c4_clean * 2048u + ub;
  b.l1 = l1;
  b.c2 = c2;
  b.hi0 = ((c3n << 9) & 0x600u) | a4;
  b.hi1 = ((c3n << 7) & 0x600u) | a4;
  b.r2 = r2;
  return b;
}
template <int kS>
__device__ __forceinline__ uint32_t u_address(const BlockRef& b) {
  return ((kS == 3 ? (b.c2 << 1) : (b.c2 << (7 - 2 * kS))) & 0x180u) | (kS < 2 ? b.hi0 : b.hi1);
}
template <int kS>
__device__ __forceinline__ uint32_t t1_address(uint32_t l1, uint32_t t1) {  // byte kS of l1 -> bits 7..14
  return ((kS == 0 ? (l1 << 7) : (l1 >> (8 * kS - 7))) & 0x7F80u) | t1;
}

// DeQuant (Algorithm 1) of sub-block kS (coordinates 4 kS .. 4 kS + 3, level-1 pairs a = 2 kS and
// b = 2 kS + 1) of a block in the rotated basis, fp16:  x = (x_a, x_b) = coordinates (4 kS, 4 kS + 2),
// y = (y_a, y_b) = coordinates (4 kS + 1, 4 kS + 3).  `t1` = level-1 table base | lane replica.
template <int kS>
__device__ __forceinline__ void sub_block_h2(const BlockRef& b, uint32_t t1, __half2& x, __half2& y) {
  const __half2 u = __hmul2(b.r2, as_h2(lds32i<kS * 8192>(u_address<kS>(b))));
  const uint2 e = lds64i<0>(t1_address<kS>(b.l1, t1));
  x = __hmul2(u, as_h2(e.x));
  y = __hmul2(u, as_h2(e.y));
}
// The same sub-block as an unevaluated sum hi + lo of fp16 values (about 21 significant bits):
//   u = r * (Uhi + Ulo)            u_hi = rn(r Uhi),  u_lo = fma(r, Uhi, -u_hi) + r Ulo
//   k = (u_hi + u_lo)(thi + tlo)   k_hi = rn(u_hi thi), k_lo = fma(u_hi, thi, -k_hi) + u_lo thi + u_hi tlo
// (fp16 fused multiply-adds return the exact rounding residual of a product).
template <int kS>
__device__ __forceinline__ void sub_block_hilo(const BlockRef& b, uint32_t t1, __half2& xh, __half2& yh, __half2& xl,
                                               __half2& yl) {
  const uint2 uu = lds64i<kS * 8192>(u_address<kS>(b));
  const __half2 u_hi = __hmul2(b.r2, as_h2(uu.x));
  const __half2 u_lo = __hfma2(b.r2, as_h2(uu.y), __hfma2(b.r2, as_h2(uu.x), __hneg2(u_hi)));
  const uint32_t ta = t1_address<kS>(b.l1, t1);
  const uint2 th = lds64i<0>(ta), tl = lds64i<kSmT1lo - kSmT1p>(ta);
  xh = __hmul2(u_hi, as_h2(th.x));
  yh = __hmul2(u_hi, as_h2(th.y));
  xl = __hfma2(u_hi, as_h2(tl.x), __hfma2(u_lo, as_h2(th.x), __hfma2(u_hi, as_h2(th.x), __hneg2(xh))));
  yl = __hfma2(u_hi, as_h2(tl.y), __hfma2(u_lo, as_h2(th.y), __hfma2(u_hi, as_h2(th.y), __hneg2(yh))));
}

// plane offsets of a d = 128 token-block
constexpr int kO2 = 32 * kTokenBlock, kO3 = kO2 + 8 * kTokenBlock, kO4 = kO3 + 4 * kTokenBlock,
              kORad = kO4 + 2 * kTokenBlock;

// Build the replicated shared-memory tables from `Tables`: entry e goes to 16 consecutive slots.
// All loads are issued before the stores so that their latencies overlap.
__device__ inline void build_fast_tables(uint8_t* smem, const Tables* tb) {
  const int tid = threadIdx.x;
  static_assert(kFastThreads == 512, "table fill assumes 512 threads");
  uint2 v[24];
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const int e = (tid + r * kFastThreads) >> 4;  // 0..255
    v[r] = tb->t1p_hi[e];
    v[8 + r] = tb->t1p_lo[e];
    v[16 + r] = tb->u_tab[e >> 6][e & 63];
  }
  uint2* t1hi = reinterpret_cast<uint2*>(smem + kSmT1p);
  uint2* t1lo = reinterpret_cast<uint2*>(smem + kSmT1lo);
  uint2* u = reinterpret_cast<uint2*>(smem + kSmU);
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const int i = tid + r * kFastThreads;
    t1hi[i] = v[r];
    t1lo[i] = v[8 + r];
    u[i] = v[16 + r];
  }
}

// Slots of split partials for the persistent kernel: every unit (sequence, kv head) has one slot
// per CTA that works on it; the slots of all units sum to at most units + grid size.
constexpr int kFastMaxGrid = 160;
constexpr int kFastMaxUnits = 2048;  // (sequence, kv head) units the persistent schedule handles
constexpr int kSegmentCost = 7;     // stages' worth of time a CTA spends on starting and finishing a unit
constexpr int kFastMaxSegs = 16;     // units of one CTA that are listed at a time
struct Segment {
  int unit, st0, st1, part, n_parts, slot0;
};

// kHG = groups of four query heads per kv head (1: up to 4 heads, 2: up to 8).
// kPaged: the cache lies behind a block table (the contiguous instantiation carries none of that code: the kernel
// sits at its register limit).
template <int kHG, bool kPaged>
__global__ void __launch_bounds__(kFastThreads, 1) decode_attention_fast_kernel(DecodeArgs a) {
  extern __shared__ __align__(128) uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((kSmAlign - (smem_u32(smem_raw) & (kSmAlign - 1))) & (kSmAlign - 1));
  const int g_heads = a.n_q_heads / a.n_kv_heads;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t sm_base = smem_u32(smem);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kSmFlags);
  int* is_last = reinterpret_cast<int*>(smem + kSmFlags) + 1;
  const int64_t head_bytes = make_layout(128, a.pg.page_tokens).head_bytes;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(sm_base + kSmBar + 8 * s, 1);                                  // full: producer + tx bytes
      mbar_init(sm_base + kSmBar + 8 * (kStages + s), kFastConsumerWarps / 2);  // empty: one arrive per warp of the group
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Launched as a programmatic dependent of the kernel before it in the stream: everything up to here may run
  // while that kernel finishes; its results (lengths, cache, queries, workspace) are read only after this wait.
  // The kernel after this one may be set up as soon as this grid has started.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  build_fast_tables(smem, a.tables);   // from the caller's tables, which no kernel writes
  asm volatile("griddepcontrol.wait;" ::: "memory");
  __syncthreads();

  // ---- persistent work split: the 128-token stages of all units, in unit order, are cut into
  // gridDim.x contiguous ranges of equal cost; a CTA's range may cover the end of one unit and the
  // start of the next, and a unit may be shared by several CTAs (its "parts").  Starting on another
  // unit costs a CTA about kSegmentCost stages (query rotation, refilling the ring, the merge), so
  // every unit is preceded by that many empty positions on the line that is cut.  Each thread works
  // out one unit; the units this CTA takes part in are consecutive among the non-empty ones and are
  // listed kFastMaxSegs at a time (a ragged batch -- one very long sequence and many short ones --
  // can give a CTA more than that; the split is then worked out again for the next batch of the list,
  // because its scratch lies in the ring).
  const int n_units = a.batch * a.n_kv_heads, G = gridDim.x, cta = blockIdx.x;
  int* u_nst = reinterpret_cast<int*>(smem + kSmRing);  // [n_units] stages; the ring is idle while the split is worked out
  int* u_parts = u_nst + kFastMaxUnits;                 // [n_units] CTAs that share the unit
  Segment* segs = reinterpret_cast<Segment*>(smem + kSmSegs);
  int* n_segs = reinterpret_cast<int*>(smem + kSmFlags) + 2;   // units of this CTA (all batches of the list)
  int* first_rank = reinterpret_cast<int*>(smem + kSmFlags) + 3;
  // Fills `segs` with the CTA's units number kFastMaxSegs * batch_no .. (counted among the CTA's own) and returns how many
  // units the CTA has in all.  Called by all threads.
  auto build_segments = [&](int batch_no) -> int {
    if (tid == 0) {
      *n_segs = 0;
      *first_rank = 0x7fffffff;
    }
    for (int u = tid; u < n_units; u += kFastThreads) {
      const int len_u = a.visible_len(u / a.n_kv_heads);
      u_nst[u] = len_u > 0 ? (len_u + kStageTokens - 1) / kStageTokens : 0;
    }
    __syncthreads();
    long long w_total = 0;
    for (int u = 0; u < n_units; ++u) w_total += u_nst[u] > 0 ? u_nst[u] + kSegmentCost : 0;
    const long long lo = cta * w_total / G, hi = (cta + 1) * w_total / G;
    // pass 1: parts of every unit; rank (among non-empty units) of the first unit of this CTA
    for (int u = tid; u < n_units; u += kFastThreads) {
      int parts = 0;
      if (u_nst[u] > 0) {
        long long start = kSegmentCost;  // position of the unit's first stage
        int rank = 0;
        for (int v = 0; v < u; ++v) {
          start += u_nst[v] > 0 ? u_nst[v] + kSegmentCost : 0;
          rank += u_nst[v] > 0;
        }
        const long long end = start + u_nst[u];
        const int c_first = (int)(((start + 1) * G + w_total - 1) / w_total) - 1;  // CTA whose range holds stage `start`
        const int c_last = (int)((end * G + w_total - 1) / w_total) - 1;           // ... stage `end - 1`
        parts = c_last - c_first + 1;
        if (cta >= c_first && cta <= c_last) {
          atomicAdd(n_segs, 1);
          atomicMin(first_rank, rank);
        }
      } else if (cta == 0 && batch_no == 0) {  // empty sequence: zeros, and the status says so
        const int b = u / a.n_kv_heads, hk = u - b * a.n_kv_heads;
        for (int i = 0; i < g_heads * 128; ++i) {
          const int64_t idx = ((int64_t)b * a.n_q_heads + hk * g_heads) * 128 + i;
          if (a.io_dtype == PQ_DTYPE_BF16) reinterpret_cast<__nv_bfloat16*>(a.out)[idx] = __float2bfloat16(0.f);
          else reinterpret_cast<float*>(a.out)[idx] = 0.f;
        }
        if (a.lse != nullptr)
          for (int h = 0; h < g_heads; ++h) a.lse[(int64_t)b * a.n_q_heads + hk * g_heads + h] = -CUDART_INF_F;
        else
          set_status(a.status, PQ_ERR_EMPTY);
      }
      u_parts[u] = parts;
    }
    __syncthreads();
    const int r0 = *first_rank + batch_no * kFastMaxSegs;  // this batch: ranks r0 .. r0 + kFastMaxSegs - 1
    // pass 2: the units of this batch, in unit order
    for (int u = tid; u < n_units; u += kFastThreads) {
      if (u_nst[u] == 0) continue;
      long long start = kSegmentCost;
      int rank = 0, slot = 0;
      for (int v = 0; v < u; ++v) {
        start += u_nst[v] > 0 ? u_nst[v] + kSegmentCost : 0;
        rank += u_nst[v] > 0;
        slot += u_parts[v];
      }
      const long long end = start + u_nst[u];
      const int c_first = (int)(((start + 1) * G + w_total - 1) / w_total) - 1;
      const int c_last = (int)((end * G + w_total - 1) / w_total) - 1;
      if (cta >= c_first && cta <= c_last && rank >= r0 && rank < r0 + kFastMaxSegs) {
        Segment& sgm = segs[rank - r0];
        sgm.unit = u;
        sgm.st0 = (int)((lo > start ? lo : start) - start);
        sgm.st1 = (int)((hi < end ? hi : end) - start);  // > st0: the CTA's range holds a stage of the unit
        sgm.part = cta - c_first;
        sgm.n_parts = u_parts[u];
        sgm.slot0 = slot;  // first partial slot of the unit
      }
    }
    __syncthreads();
    return *n_segs;
  };
  const int g = lane >> 2, c = lane & 3;
  const uint32_t rep = (lane & 15) * 8;
  const uint32_t ua = sm_base + kSmU + rep, t1a = sm_base + kSmT1p + rep;  // table base | lane replica
  const int wg = warp >> 3;  // group of 8 warps
  // Offsets, inside a token-block, of what this thread reads of its tile (16 tokens from token (warp & 3) * 16).
  // Keys: tokens g and g + 8, blocks 2c and 2c + 1.  Values: block g of tokens c, c + 4, c + 8, c + 12 (these are
  // rows 2c, 2c + 1, 2c + 8, 2c + 9 of the value MMA: with this order the four lanes of a quad read four
  // consecutive tokens and the loads are free of bank conflicts).
  const int tk_k = (warp & 3) * 16 + (lane >> 2), tk_v = (warp & 3) * 16 + (lane & 3);
  const uint32_t ok_l1 = tk_k * 32 + (lane & 3) * 8, ok_r = kORad + tk_k * 16 + (lane & 3) * 4;
  const uint32_t ok_c2 = kO2 + tk_k * 8 + (lane & 3) * 2, ok_c3 = kO3 + tk_k * 4 + (lane & 3), ok_c4 = kO4 + tk_k * 2;
  const uint32_t ov_l1 = tk_v * 32 + (lane >> 2) * 4, ov_r = kORad + tk_v * 16 + (lane >> 2) * 2;
  const uint32_t ov_c2 = kO2 + tk_v * 8 + (lane >> 2), ov_c3 = kO3 + tk_v * 4 + (lane >> 3), ov_c4 = kO4 + tk_v * 2;
  int gl0 = 0;               // stages this group has streamed so far (ring slot and barrier phase bookkeeping)

  int my_units = build_segments(0);
  for (int batch_no = 0; batch_no * kFastMaxSegs < my_units; ++batch_no) {
  if (batch_no > 0) my_units = build_segments(batch_no);
  const int my_segs = min(kFastMaxSegs, my_units - batch_no * kFastMaxSegs);
  for (int sg = 0; sg < my_segs; ++sg) {
    const int u = segs[sg].unit, st0 = segs[sg].st0, st1 = segs[sg].st1;
    const int n_parts = segs[sg].n_parts, unit_slot = segs[sg].slot0, c_first = cta - segs[sg].part;
    const int b = u / a.n_kv_heads, hk = u - b * a.n_kv_heads;
    const int len = a.visible_len(b);   // b counts (sequence, query) pairs: see DecodeArgs
    const int nblk_total = (len + kTokenBlock - 1) / kTokenBlock;
    const int seq = a.seq_of(b);
    const uint8_t* head_base = a.cache + ((int64_t)seq * a.n_kv_heads + hk) * head_bytes;  // of a contiguous cache

    // per-thread attention state
    // o_acc[hg][S][.]: head c + 4 hg, block g, coordinates 4S, 4S + 2, 4S + 1, 4S + 3 (see the value MMAs)
    float o_acc[kHG][4][4];
#pragma unroll
    for (int hg = 0; hg < kHG; ++hg)
#pragma unroll
      for (int i = 0; i < 4; ++i) o_acc[hg][i][0] = o_acc[hg][i][1] = o_acc[hg][i][2] = o_acc[hg][i][3] = 0.f;
    float m_run[kHG], l_run[kHG];  // of head c + 4 hg: reference (the same in the 8 lanes with this c), own share of the sum
#pragma unroll
    for (int hg = 0; hg < kHG; ++hg) {
      m_run[hg] = -CUDART_INF_F;
      l_run[hg] = 0.f;
    }

    // The two groups of 8 warps take alternate stages: group wg handles stages st0 + wg + 2 li and owns
    // ring slots 2 wg and 2 wg + 1.  Lane 0 of the group's first warp issues the group's copies, one
    // stage of its own ahead; it waits (bounded) until the group's 8 warps have released the slot.
    const int n_li = st1 - st0 > wg ? (st1 - st0 - wg + 1) >> 1 : 0;
    int issued = 0;
    auto issue_copy = [&](int li) -> bool {
      const int gl = gl0 + li, s = 2 * wg + (gl & 1);
      if (gl >= 2 && !mbar_wait(sm_base + kSmBar + 8 * (kStages + s), ((gl >> 1) - 1) & 1, abort_flag)) return false;
      const int st = st0 + wg + 2 * li;
      const int nblk = min(2, nblk_total - 2 * st);
      const uint32_t bytes = nblk * 2 * kBlockBytes128;
      mbar_expect_tx(sm_base + kSmBar + 8 * s, bytes);
      // a stage is two token-blocks, K | V | K | V, of one page (page_tokens is a multiple of 128)
      const uint8_t* src = head_base + (int64_t)st * kStageBytes;
      if (kPaged) {
        Layout Lp;  // the two fields the offset needs
        Lp.block_bytes = kBlockBytes128;
        Lp.head_bytes = head_bytes;
        src = a.cache + kv_block_pair_offset(Lp, a.pg, a.n_kv_heads, seq, hk, 2 * st, a.status);
      }
      bulk_load(sm_base + kSmRing + s * kStageBytes, src, bytes, sm_base + kSmBar + 8 * s);
      issued = li + 1;
      return true;
    };
    const bool producer = (tid & 255) == 0;
    if (producer && n_li > 0) issue_copy(0);
    __syncwarp();
    // q' = (q S) * scale * log2(e) for the unit's query heads, as an fp16 value plus an fp16 residual.
    // The first stages of the segment are already on their way while this runs.
    {
      float* q_in = reinterpret_cast<float*>(smem + kSmQ);
      __half* q_hi = reinterpret_cast<__half*>(smem + kSmQ + 4096);
      __half* q_lo = q_hi + 8 * 128;
      const int64_t q0 = ((int64_t)b * a.n_q_heads + hk * g_heads) * 128;
      for (int i = tid; i < g_heads * 128; i += kFastThreads)
        q_in[i] = a.io_dtype == PQ_DTYPE_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.q)[q0 + i])
                                              : reinterpret_cast<const float*>(a.q)[q0 + i];
      __syncthreads();
      for (int i = tid; i < g_heads * 128; i += kFastThreads) {
        const float* qrow = q_in + (i & ~127);
        const float* scol = a.S + (i & 127);
        float acc = 0.f;
#pragma unroll 32
        for (int k = 0; k < 128; ++k) acc = fmaf(qrow[k], __ldg(scol + k * 128), acc);
        acc *= a.scale * 1.4426950408889634f;
        const __half qh = __float2half_rn(acc);
        q_hi[i] = qh;
        q_lo[i] = __float2half_rn(acc - __half2float(qh));
      }
      __syncthreads();
    }
    // q' fragments, B operand (16 coords x 8 columns per k-step): column n = 2 h + part holds the fp16 value
    // (part 0) or the fp16 residual (part 1) of head h (+ 4 hg).  k-step ks covers, for thread c, sub-block
    // (ks & 3) of block 2c + (ks >> 2).
    uint32_t qb[kHG][8][2];
#pragma unroll
    for (int hg = 0; hg < kHG; ++hg) {
      const int h = (g >> 1) + 4 * hg;
      const uint2* qsrc = reinterpret_cast<const uint2*>(smem + kSmQ + 4096 + (g & 1) * 2048) + (h * 128 + 32 * c) / 4;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint2 v = make_uint2(0u, 0u);
        if (h < g_heads) v = qsrc[ks];
        // decoded keys come as (coord 0, coord 2), (coord 1, coord 3) of each sub-block: permute q' to match
        qb[hg][ks][0] = __byte_perm(v.x, v.y, 0x5410);
        qb[hg][ks][1] = __byte_perm(v.x, v.y, 0x7632);
      }
    }
    for (int li = 0; li < n_li; ++li) {
      const int gl = gl0 + li, s = 2 * wg + (gl & 1);
      const int st = st0 + wg + 2 * li;
      if (producer && li + 1 < n_li) issue_copy(li + 1);
      __syncwarp();
      if (!mbar_wait(sm_base + kSmBar + 8 * s, (gl >> 1) & 1, abort_flag)) break;
      if ((a.debug & 1u) && unit_slot == 0 && cta == c_first && li == 0 && warp == 0) {  // test hook: the first wait of the CTA
        // that starts the first non-empty unit is reported as failed
        *abort_flag = 1;
        break;
      }
      const int tile_tok0 = st * kStageTokens + (warp & 7) * 16;  // first token of this warp's 16-token tile
      if (tile_tok0 < len) {
        const uint32_t kblk = sm_base + kSmRing + s * kStageBytes + ((warp >> 2) & 1) * 2 * kBlockBytes128;
        const uint32_t vblk = kblk + kBlockBytes128;
        // ---- scores S (tokens x columns): A operand = keys of tokens g (rows 0..7) and g + 8 (rows 8..15),
        // decoded as hi + lo; one MMA with the hi parts and one with the lo parts per k-step.  Column 2c is
        // q_hi of head c, column 2c+1 its q_lo, so all four products of a (token, head) land in this thread.
        float sc[kHG][4], scl[kHG][4];
#pragma unroll
        for (int hg = 0; hg < kHG; ++hg)
#pragma unroll
          for (int i = 0; i < 4; ++i) sc[hg][i] = scl[hg][i] = 0.f;
        {
          const uint2 l1A = lds64i<0>(kblk + ok_l1), l1B = lds64i<8 * 32>(kblk + ok_l1);
          const uint32_t rrA = lds32i<0>(kblk + ok_r), rrB = lds32i<8 * 16>(kblk + ok_r);
          const uint32_t c2A = lds16i<0>(kblk + ok_c2), c2B = lds16i<8 * 8>(kblk + ok_c2);
          const uint32_t c3A = lds8i<0>(kblk + ok_c3), c3B = lds8i<8 * 4>(kblk + ok_c3);
          const uint32_t c4A = lds16i<0>(kblk + ok_c4) >> (4 * c), c4B = lds16i<8 * 2>(kblk + ok_c4) >> (4 * c);
#define PQ_KSTEP(H, S)                                                                                    \
  {                                                                                                       \
    __half2 xhA, yhA, xlA, ylA, xhB, yhB, xlB, ylB;                                                       \
    sub_block_hilo<S>(bA, t1a, xhA, yhA, xlA, ylA);                                                       \
    sub_block_hilo<S>(bB, t1a, xhB, yhB, xlB, ylB);                                                       \
    _Pragma("unroll") for (int hg = 0; hg < kHG; ++hg) {                                                  \
      mma_16816(scl[hg], as_u32(xlA), as_u32(xlB), as_u32(ylA), as_u32(ylB), qb[hg][4 * (H) + (S)][0],    \
                qb[hg][4 * (H) + (S)][1]);                                                                \
      mma_16816(sc[hg], as_u32(xhA), as_u32(xhB), as_u32(yhA), as_u32(yhB), qb[hg][4 * (H) + (S)][0],     \
                qb[hg][4 * (H) + (S)][1]);                                                                \
    }                                                                                                     \
  }
          {
            const BlockRef bA = make_block_ref(l1A.x, c2A, c3A, c4A & 3u, __low2half2(as_h2(rrA)), ua);
            const BlockRef bB = make_block_ref(l1B.x, c2B, c3B, c4B & 3u, __low2half2(as_h2(rrB)), ua);
            PQ_KSTEP(0, 0) PQ_KSTEP(0, 1) PQ_KSTEP(0, 2) PQ_KSTEP(0, 3)
          }
          {
            const BlockRef bA = make_block_ref(l1A.y, c2A >> 8, c3A >> 4, (c4A >> 2) & 3u, __high2half2(as_h2(rrA)), ua);
            const BlockRef bB = make_block_ref(l1B.y, c2B >> 8, c3B >> 4, (c4B >> 2) & 3u, __high2half2(as_h2(rrB)), ua);
            PQ_KSTEP(1, 0) PQ_KSTEP(1, 1) PQ_KSTEP(1, 2) PQ_KSTEP(1, 3)
          }
#undef PQ_KSTEP
        }
        // ---- online softmax: this thread holds head c (+ 4 hg) of tokens g and g + 8.  The reference m_run of a
        // head moves only when a score exceeds it by more than kLazyMax (log2 units), so p = 2^(s - m_run) stays
        // below 2^kLazyMax (fp16 holds it with its full relative precision) and the common tile needs neither
        // the reductions over tokens nor a rescaling; l_run is this thread's share of the denominator (its own
        // tokens), summed over the eight lanes of the head when the segment ends.
        const bool ok0 = tile_tok0 + g < len, ok1 = tile_tok0 + g + 8 < len;
        float s0[kHG], s1[kHG];
        bool over = false;
#pragma unroll
        for (int hg = 0; hg < kHG; ++hg) {
          s0[hg] = ok0 ? (scl[hg][0] + scl[hg][1]) + sc[hg][1] + sc[hg][0] : -CUDART_INF_F;  // small terms first
          s1[hg] = ok1 ? (scl[hg][2] + scl[hg][3]) + sc[hg][3] + sc[hg][2] : -CUDART_INF_F;
          over = over || fmaxf(s0[hg], s1[hg]) > m_run[hg] + kLazyMax;  // always on the first tile (m_run = -inf)
        }
        if (__any_sync(0xffffffffu, over)) {
          float corr[kHG];
#pragma unroll
          for (int hg = 0; hg < kHG; ++hg) {
            float mx = fmaxf(s0[hg], s1[hg]);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
            const float m_new = fmaxf(m_run[hg], mx);  // finite: token 0 of the tile is inside the sequence
            corr[hg] = fast_exp2(m_run[hg] - m_new);   // 0 on the first tile
            l_run[hg] *= corr[hg];
            m_run[hg] = m_new;
          }
#pragma unroll
          for (int hg = 0; hg < kHG; ++hg)  // the accumulators of this thread belong to its own head
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              o_acc[hg][i][0] *= corr[hg];
              o_acc[hg][i][1] *= corr[hg];
              o_acc[hg][i][2] *= corr[hg];
              o_acc[hg][i][3] *= corr[hg];
            }
        }
        uint32_t ph[kHG];   // (p of token g, p of token g + 8) in fp16
#pragma unroll
        for (int hg = 0; hg < kHG; ++hg) {
          const float p0 = fast_exp2(s0[hg] - m_run[hg]), p1 = fast_exp2(s1[hg] - m_run[hg]);
          l_run[hg] += p0 + p1;
          ph[hg] = as_u32(__floats2half2_rn(p0, p1));
        }
        // B operand of the value MMAs.  The contraction index is (token, which element of a decoded half2): rows
        // 2c, 2c+1 = token c (first MMA) or c + 8 (second), rows 2c+8, 2c+9 = token c + 4 or c + 12.  Column
        // n = 2h + e is head h restricted to element e: its entry is p in half e and zero in the other, so a
        // decoded half2 is an A register as it is and no column of the MMA is idle (4 heads x 2 elements).
        uint32_t pb[kHG][2][2];
#pragma unroll
        for (int hg = 0; hg < kHG; ++hg) {
          const int srcA = c * 4 + (g >> 1);  // lane that holds tokens c and c + 8 of head g >> 1
          const uint32_t uA = __shfl_sync(0xffffffffu, ph[hg], srcA), uB = __shfl_sync(0xffffffffu, ph[hg], srcA + 16);
          const uint32_t sel_lo = (g & 1) ? 0x1044u : 0x4410u, sel_hi = (g & 1) ? 0x3244u : 0x4432u;
          pb[hg][0][0] = __byte_perm(uA, 0u, sel_lo);
          pb[hg][0][1] = __byte_perm(uB, 0u, sel_lo);
          pb[hg][1][0] = __byte_perm(uA, 0u, sel_hi);
          pb[hg][1][1] = __byte_perm(uB, 0u, sel_hi);
        }
        // ---- values: block g of tokens c, c+4, c+8, c+12 -> O^T (coordinates x (head, element)) += V_hat^T P
        {
          BlockRef bv[4];
#define PQ_VLOAD(J)                                                                                          \
  {                                                                                                          \
    const uint32_t l1 = lds32i<4 * (J) * 32>(vblk + ov_l1);                                                  \
    uint32_t rr = lds16i<4 * (J) * 16>(vblk + ov_r);                                                         \
    const uint32_t c2 = lds8i<4 * (J) * 8>(vblk + ov_c2);                                                    \
    const uint32_t c3 = lds8i<4 * (J) * 4>(vblk + ov_c3) >> (4 * (g & 1));                                   \
    const uint32_t c4 = lds16i<4 * (J) * 2>(vblk + ov_c4) >> (2 * g);                                        \
    if (tile_tok0 + c + 4 * (J) >= len) rr = 0u; /* stale bytes past the sequence end stay out of the sums */ \
    bv[J] = make_block_ref(l1, c2, c3, c4 & 3u, as_h2(rr | (rr << 16)), ua);                                 \
  }
          PQ_VLOAD(0) PQ_VLOAD(1) PQ_VLOAD(2) PQ_VLOAD(3)
#undef PQ_VLOAD
#define PQ_VSTEP(S)                                                                                      \
  {                                                                                                      \
    __half2 x0, y0, x1, y1, x2, y2, x3, y3;                                                              \
    sub_block_h2<S>(bv[0], t1a, x0, y0);                                                                 \
    sub_block_h2<S>(bv[1], t1a, x1, y1);                                                                 \
    sub_block_h2<S>(bv[2], t1a, x2, y2);                                                                 \
    sub_block_h2<S>(bv[3], t1a, x3, y3);                                                                 \
    _Pragma("unroll") for (int hg = 0; hg < kHG; ++hg) {                                                 \
      mma_16816(o_acc[hg][S], as_u32(x0), as_u32(y0), as_u32(x1), as_u32(y1), pb[hg][0][0], pb[hg][0][1]); \
      mma_16816(o_acc[hg][S], as_u32(x2), as_u32(y2), as_u32(x3), as_u32(y3), pb[hg][1][0], pb[hg][1][1]); \
    }                                                                                                    \
  }
          PQ_VSTEP(0) PQ_VSTEP(1) PQ_VSTEP(2) PQ_VSTEP(3)
#undef PQ_VSTEP
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(sm_base + kSmBar + 8 * (kStages + s));
    }
    gl0 += n_li;
    __syncthreads();  // every copy that was consumed is done with; the rest is waited for below
    if (*abort_flag) {
      // gave up: let the copies still in flight land (bounded) before the ring is reused
      if (producer)
        for (int li = max(0, issued - 2); li < issued; ++li) {
          const int gl = gl0 - n_li + li;
          for (int i = 0; i < kSpinLimit && !mbar_try_wait(sm_base + kSmBar + 8 * (2 * wg + (gl & 1)), (gl >> 1) & 1); ++i)
            __nanosleep(64);
        }
      __syncthreads();
    }

    // ---- merge the 16 warps (fixed order), write this part's partial, last part combines the unit
    // Coordinate j of head h of warp w sits at (w * 8 + h) * kMrgStride + (j & 15) * 8 + (j >> 4): for a fixed
    // accumulator register the 32 lanes (block g, head c) then hit 32 different banks.
    float* mrg_o = reinterpret_cast<float*>(smem + kSmRing);          // [16 warps][8 heads][kMrgStride]
    float* mrg_ml = mrg_o + kFastConsumerWarps * 8 * kMrgStride;      // [16 warps][8 heads][2]
#pragma unroll
    for (int hg = 0; hg < kHG; ++hg) {  // the head's denominator: sum of the shares of its eight lanes
      l_run[hg] += __shfl_xor_sync(0xffffffffu, l_run[hg], 4);
      l_run[hg] += __shfl_xor_sync(0xffffffffu, l_run[hg], 8);
      l_run[hg] += __shfl_xor_sync(0xffffffffu, l_run[hg], 16);
    }
    if (g == 0) {
#pragma unroll
      for (int hg = 0; hg < kHG; ++hg) {
        mrg_ml[(warp * 8 + c + 4 * hg) * 2] = m_run[hg];
        mrg_ml[(warp * 8 + c + 4 * hg) * 2 + 1] = l_run[hg];
      }
      if (kHG == 1) {  // heads 4..7 do not exist: neutral entries
        mrg_ml[(warp * 8 + c + 4) * 2] = -CUDART_INF_F;
        mrg_ml[(warp * 8 + c + 4) * 2 + 1] = 0.f;
      }
    }
#pragma unroll
    for (int hg = 0; hg < kHG; ++hg)
      if (c + 4 * hg < g_heads) {
        float* o0 = mrg_o + (warp * 8 + c + 4 * hg) * kMrgStride + g;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          o0[(4 * i) * 8] = o_acc[hg][i][0];
          o0[(4 * i + 2) * 8] = o_acc[hg][i][1];
          o0[(4 * i + 1) * 8] = o_acc[hg][i][2];
          o0[(4 * i + 3) * 8] = o_acc[hg][i][3];
        }
      }
    __syncthreads();
    const int slot = unit_slot + (cta - c_first);
    for (int idx = tid; idx < g_heads * 128; idx += kFastThreads) {
      const int h = idx >> 7, j = idx & 127;
      float M = -CUDART_INF_F;
#pragma unroll
      for (int w = 0; w < kFastConsumerWarps; ++w) M = fmaxf(M, mrg_ml[(w * 8 + h) * 2]);
      float lsum = 0.f, acc = 0.f;
#pragma unroll
      for (int w = 0; w < kFastConsumerWarps; ++w) {
        const float mw = mrg_ml[(w * 8 + h) * 2];
        const float wgt = mw == -CUDART_INF_F ? 0.f : exp2f(mw - M);
        lsum += mrg_ml[(w * 8 + h) * 2 + 1] * wgt;
        acc += mrg_o[(w * 8 + h) * kMrgStride + (j & 15) * 8 + (j >> 4)] * wgt;
      }
      const int64_t pidx = (int64_t)slot * g_heads + h;
      a.ws.o[pidx * 128 + j] = acc;
      if (j == 0) {
        a.ws.ml[2 * pidx] = M;
        a.ws.ml[2 * pidx + 1] = lsum;
      }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      // Arrival count of the unit's parts.  The workspace is not assumed to start at zero: a ticket
      // holds (call epoch << 32 | arrivals), and a ticket of another epoch counts as zero arrivals.
      bool last = true;
      if (n_parts > 1) {
        unsigned long long* tk = reinterpret_cast<unsigned long long*>(a.ws.tickets) + u;
        unsigned long long cur = *reinterpret_cast<volatile unsigned long long*>(tk), want = 0ull;
        bool done = false;
        for (int i = 0; i < 4096 && !done; ++i) {  // every failed attempt is another part's success: <= n_parts rounds
          want = (uint32_t)(cur >> 32) == a.epoch ? cur + 1ull : ((unsigned long long)a.epoch << 32) | 1ull;
          const unsigned long long prev = atomicCAS(tk, cur, want);
          done = prev == cur;
          cur = prev;
        }
        if (!done) set_status(a.status, PQ_ERR_TIMEOUT);
        last = done && (int)(want & 0xffffffffull) == n_parts;
        if (last) *tk = 0ull;  // no other part of this call touches it any more
      }
      *is_last = last;
    }
    __syncthreads();
    if (*is_last) {
      __threadfence();
      combine_and_store(a, b, hk, g_heads, unit_slot, n_parts, reinterpret_cast<float*>(smem + kSmRing));
    }
    __syncthreads();  // the ring is free again for the next unit
  }
  }
  if (tid == 0 && *abort_flag) set_status(a.status, PQ_ERR_TIMEOUT);
}

}  // namespace pq
