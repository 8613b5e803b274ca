// Tensor-core encoder for head_dim 128, bf16 inputs (included by pq_encode.cu).
//
// Persistent CTAs (one per SM) loop over tiles of 128 rows x one (K|V, head).  Per tile
//   warp 0   (one lane): TMA loads of the x tile (two 64-column boxes, 128-byte swizzle) into a ring;
//   warp 1   (one lane): y = x . S on the 5th-generation tensor cores: S is split once per CTA into
//            two bf16 terms (S = S_hi + S_lo + O(2^-17)) kept in shared memory as the K-major B
//            operand; 2 terms x 8 k-steps of tcgen05.mma (M = 128 rows, N = 128, K = 16) accumulate
//            in float32 in tensor memory; two accumulators let the next tile's MMAs overlap the
//            current tile's epilogue;
//   warps 2-9: epilogue.  Tensor-memory lane = row, so a thread owns 64 consecutive rotated
//            coordinates (4 blocks) of one row: tcgen05.ld, sign-test quantiser with certified
//            margins, packed stores, queued float64 re-decision of the ambiguous angles.
// Every mbarrier wait is bounded; a wait that gives up raises the CTA's abort flag, all roles leave
// their loops, tensor memory is released and PQ_ERR_TIMEOUT is recorded.
#pragma once
#include <cuda.h>

namespace pq {

constexpr int kTcThreads = 320;
constexpr int kTcEpiThreads = 256;
constexpr int kTcStages = 3;
constexpr int kTcXBytes = 128 * 128 * 2;   // one x tile: 128 rows x 128 bf16
constexpr int kTcSBytes = 128 * 128 * 2;   // one bf16 term of S (B operand)
constexpr int kTcSmS = 0;                  // S_hi, S_lo
constexpr int kTcSmX = kTcSmS + 2 * kTcSBytes;
constexpr int kTcSmRowSq = kTcSmX + kTcStages * kTcXBytes;   // [2][128] float
constexpr int kTcSmFq = kTcSmRowSq + 1024;                   // FastQuant (36 B)
constexpr int kTcSmBar = kTcSmFq + 64;                       // full[3], empty[3], tfull[2], tempty[2]
constexpr int kTcSmMisc = kTcSmBar + 128;                    // tmem base, abort flag
constexpr int kTcSmFix = kTcSmMisc + 64;                     // FixQueue
constexpr int kTcSmTotal = kTcSmFix + (int)sizeof(FixQueue) + 1024;  // + slack for 1024-byte alignment
constexpr int kTcSpin = 1 << 22;

__device__ __forceinline__ uint32_t tc_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void tc_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool tc_mbar_try(uint32_t bar, uint32_t parity) {
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
__device__ __forceinline__ bool tc_mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (int i = 0; i < kTcSpin; ++i) {
    if (tc_mbar_try(bar, parity)) return true;
    if (i > 32) {
      __nanosleep(64);
      if (*abort_flag) return false;
    }
  }
  *abort_flag = 1;
  return false;
}

// K-major, 128-byte-swizzled shared-memory matrix descriptor (rows of 64 bf16 = 128 bytes, groups of
// 8 rows 1024 bytes apart).
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t addr) {
  uint64_t d = (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;            // leading byte offset (unused with 128-byte swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;  // stride byte offset: 8 rows
  d |= (uint64_t)1 << 46;            // descriptor version of this architecture
  d |= (uint64_t)2 << 61;            // 128-byte swizzle
  return d;
}
// kind::f16 instruction descriptor: D = f32, A = B = bf16, both K-major, N = 128, M = 128.
constexpr uint32_t kTcIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(kTcIdesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

struct TcMaps {
  CUtensorMap k, v;
};

__global__ void __launch_bounds__(kTcThreads, 1)
encode_tc_kernel(EncodeArgs a, const __grid_constant__ TcMaps maps, int n_row_tiles) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sb = tc_smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kTcSmMisc + 4);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kTcSmMisc);
  FastQuant* fq = reinterpret_cast<FastQuant*>(smem + kTcSmFq);
  FixQueue* fixq = reinterpret_cast<FixQueue*>(smem + kTcSmFix);
  float* rowsq = reinterpret_cast<float*>(smem + kTcSmRowSq);
  const uint32_t bar_full = sb + kTcSmBar, bar_empty = bar_full + 8 * kTcStages;
  const uint32_t bar_tfull = bar_empty + 8 * kTcStages, bar_tempty = bar_tfull + 16;
  const int n_tiles = n_row_tiles * 2 * a.n_kv_heads;

  // ---- set-up: barriers, tensor memory, S split into two bf16 terms in the B-operand layout
  if (tid == 0) {
    for (int s = 0; s < kTcStages; ++s) {
      tc_mbar_init(bar_full + 8 * s, 1);
      tc_mbar_init(bar_empty + 8 * s, 1);
    }
    for (int i = 0; i < 2; ++i) {
      tc_mbar_init(bar_tfull + 8 * i, 1);
      tc_mbar_init(bar_tempty + 8 * i, kTcEpiThreads / 32);
    }
    *abort_flag = 0;
    fixq->count = 0;
    load_fast_quant(a.tables, fq);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(sb + kTcSmMisc) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // B operand: B[n][k] = S[k][n]; two halves of 64 k; row n = 128 bytes, 16-byte chunk c stored at c ^ (n & 7).
  for (int idx = tid; idx < 128 * 128; idx += kTcThreads) {
    const int k = idx >> 7, n = idx & 127;  // consecutive threads read consecutive n: coalesced
    const float v = a.S[idx];
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
    const int half = k >> 6, kk = k & 63;
    const int off = half * 16384 + n * 128 + ((((kk >> 3) ^ (n & 7)) << 4) | ((kk & 7) << 1));
    *reinterpret_cast<__nv_bfloat16*>(smem + kTcSmS + off) = hi;
    *reinterpret_cast<__nv_bfloat16*>(smem + kTcSmS + kTcSBytes + off) = lo;
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the MMA unit
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int it = 0;
      for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
        const int s = it % kTcStages;
        if (it >= kTcStages && !tc_mbar_wait(bar_empty + 8 * s, ((it / kTcStages) - 1) & 1, abort_flag)) break;
        const int head = tile % a.n_kv_heads, kv = (tile / a.n_kv_heads) & 1, rt = tile / (2 * a.n_kv_heads);
        const CUtensorMap* map = kv ? &maps.v : &maps.k;
        const uint32_t dst = sb + kTcSmX + s * kTcXBytes, bar = bar_full + 8 * s;
        tc_mbar_expect_tx(bar, kTcXBytes);
#pragma unroll
        for (int h = 0; h < 2; ++h)
          asm volatile(
              "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
              ::"r"(dst + h * 16384), "l"(map), "r"(h * 64), "r"(head), "r"(rt * 128), "r"(bar)
              : "memory");
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int it = 0;
      for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
        const int s = it % kTcStages, acc = it & 1;
        if (!tc_mbar_wait(bar_full + 8 * s, (it / kTcStages) & 1, abort_flag)) break;
        if (it >= 2 && !tc_mbar_wait(bar_tempty + 8 * acc, ((it >> 1) - 1) & 1, abort_flag)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t xa = sb + kTcSmX + s * kTcXBytes;
        const uint32_t d = tmem_base + acc * 128;
        uint32_t accumulate = 0;
#pragma unroll
        for (int term = 0; term < 2; ++term)
#pragma unroll
          for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t ad = tc_smem_desc(xa + h * 16384 + ks * 32);
              const uint64_t bd = tc_smem_desc(sb + kTcSmS + term * kTcSBytes + h * 16384 + ks * 32);
              tc_mma(d, ad, bd, accumulate);
              accumulate = 1;
            }
        tc_commit(bar_empty + 8 * s);     // the x stage may be refilled once these MMAs have read it
        tc_commit(bar_tfull + 8 * acc);   // the accumulator is complete
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (8 warps)
    constexpr int o2 = 32 * kTokenBlock, o3 = o2 + 8 * kTokenBlock, o4 = o3 + 4 * kTokenBlock, orad = o4 + 2 * kTokenBlock;
    const int et = tid - 64;                       // 0..255
    const int quarter = warp & 3;                  // tensor-memory lanes this warp may read
    const int half = (warp - 2) >> 2;              // columns [64*half, 64*half + 64)
    const int r = quarter * 32 + lane;             // row of the tile
    const bool uniform = (a.tables->flags & kFlagUniformL1) != 0u;
    const Layout L = make_layout(128, a.capacity);
    int it = 0;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it) {
      const int acc = it & 1;
      const int head = tile % a.n_kv_heads, kv = (tile / a.n_kv_heads) & 1, rt = tile / (2 * a.n_kv_heads);
      // A wait that gives up must not leave the loop: the other epilogue warps may be past it and
      // would wait for this one at the named barriers.  The tile is skipped instead (warp-uniform).
      const bool ready = __all_sync(0xffffffffu, tc_mbar_wait(bar_tfull + 8 * acc, (it >> 1) & 1, abort_flag));
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * 128 + half * 64;
      // pass 1: squared norm of the row (its two halves are exchanged through shared memory)
      float sq = 0.f;
      if (ready) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
        for (int i = 0; i < 4; ++i) {
          float y[16];
          tc_ld16(taddr + 16 * i, y);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int c = 0; c < 16; ++c) sq = fmaf(y[c], y[c], sq);
        }
      }
      rowsq[half * 128 + r] = sq;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      const float dy = kRotErr * 1.0001f * sqrtf(rowsq[r] + rowsq[128 + r]);
      const int row = rt * 128 + r;
      uint8_t* tb = nullptr;
      int tok = 0;
      if (ready && row < a.total_tokens) {
        int seq, pos;
        row_destination(a, row, &seq, &pos);
        if (pos >= 0) {
          tb = a.cache + block_offset(L, a.n_kv_heads, seq, head, kv, pos);
          tok = pos % kTokenBlock;
        }
      }
      const int64_t xoff = (int64_t)row * a.token_stride + (int64_t)head * a.head_stride;
      // pass 2: one block at a time
      uint32_t l2acc = 0, l3acc = 0, l4acc = 0, sat = 0;
      unsigned long long racc = 0ull, leftbits = 0ull;
      if (ready) {
#pragma unroll 1
        for (int i = 0; i < 4; ++i) {
          float y[16];
          tc_ld16(taddr + 16 * i, y);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          FastBlock fb;
          polar_quant_block_fast(y, dy, *fq, &fb);
          if (!uniform) fb.amb |= 0xFFu;  // other level-1 codebooks: decide every level-1 angle exactly
          if (tb != nullptr) {
            *reinterpret_cast<uint32_t*>(tb + tok * 32 + half * 16 + 4 * i) = fb.l1;
            l2acc |= fb.l2 << (8 * i);
            l3acc |= fb.l3 << (4 * i);
            l4acc |= fb.l4 << (2 * i);
            float rv = fb.radius;
            if (rv > 65504.f) { rv = 65504.f; ++sat; }
            racc |= (unsigned long long)__half_as_ushort(__float2half_rn(rv)) << (16 * i);
            if (fb.amb) {
              uint32_t left;
              fix_push(fixq, fb.amb, xoff, tb, tok, 4 * half + i, kv, &left);
              leftbits |= (unsigned long long)left << (15 * i);  // queue full: pushed again by fix_rounds
            }
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) tc_mbar_arrive(bar_tempty + 8 * acc);  // this accumulator may be overwritten
      }
      if (tb != nullptr) {
        *reinterpret_cast<uint32_t*>(tb + o2 + tok * 8 + half * 4) = l2acc;
        *reinterpret_cast<uint16_t*>(tb + o3 + tok * 4 + half * 2) = (uint16_t)l3acc;
        tb[o4 + tok * 2 + half] = (uint8_t)l4acc;
        *reinterpret_cast<unsigned long long*>(tb + orad + tok * 16 + half * 8) = racc;
        if (sat) atomicAdd(a.status + 2, (int)sat);
      }
      // Exact re-decisions are batched over tiles: drain the queue when it is half full (a push that
      // did not fit leaves the counter above the capacity) or after the CTA's last tile.
      asm volatile("bar.sync 1, 256;" ::: "memory");
      const bool last_tile = tile + (int)gridDim.x >= n_tiles;
      if (fixq->count > kFixCap / 2 || last_tile)
        fix_rounds(a, fixq, leftbits, xoff, tb, tok, half, kv, et, kTcEpiThreads, 1);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem_base) : "memory");
  }
  if (tid == 0 && *abort_flag) set_status(a.status, PQ_ERR_TIMEOUT);
}

// Tensor maps for the K and V inputs ([tokens][heads][128] bf16 with element strides).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

static bool make_x_map(EncodeTiledFn fn, CUtensorMap* map, const void* base, int n_kv_heads, int total_tokens,
                       int64_t token_stride, int64_t head_stride) {
  const cuuint64_t dims[3] = {128, (cuuint64_t)n_kv_heads, (cuuint64_t)total_tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)head_stride * 2, (cuuint64_t)token_stride * 2};
  const cuuint32_t box[3] = {64, 1, 128};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Launch the tensor-core encoder if the inputs allow it.  Returns 1 if launched, 0 if not applicable,
// or a negative status.
static int32_t try_launch_encode_tc(const EncodeArgs& a, cudaStream_t stream) {
  if (a.head_dim != 128 || a.in_dtype != PQ_DTYPE_BF16 || a.total_tokens < 128) return 0;
  if ((a.token_stride & 7) || (a.head_stride & 7) || a.head_stride < 128 || a.token_stride < 128) return 0;
  if (((uintptr_t)a.K | (uintptr_t)a.V) & 15) return 0;
  if (a.n_kv_heads > 1 && a.head_stride * 2 >= ((int64_t)1 << 40)) return 0;
  EncodeTiledFn fn = get_encode_tiled();
  if (fn == nullptr) return 0;
  TcMaps maps;
  if (!make_x_map(fn, &maps.k, a.K, a.n_kv_heads, a.total_tokens, a.token_stride, a.head_stride)) return 0;
  if (!make_x_map(fn, &maps.v, a.V, a.n_kv_heads, a.total_tokens, a.token_stride, a.head_stride)) return 0;
  static int n_sm = 0;
  static bool configured = false;
  if (!configured) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(encode_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmTotal);
    if (e != cudaSuccess) {
      note_cuda_error(e);
      return PQ_ERR_CUDA;
    }
    configured = true;
  }
  const int n_row_tiles = (a.total_tokens + 127) / 128;
  const int n_tiles = n_row_tiles * 2 * a.n_kv_heads;
  const int grid = n_tiles < n_sm ? n_tiles : n_sm;
  encode_tc_kernel<<<grid, kTcThreads, kTcSmTotal, stream>>>(a, maps, n_row_tiles);
  return 1;
}

}  // namespace pq
