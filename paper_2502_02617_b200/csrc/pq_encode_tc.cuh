// Tensor-core encoder for head_dim 128, bf16 inputs (included by pq_encode.cu).
//
// Persistent CTAs (one per SM, 16 warps) loop over tiles of 128 rows x one (K|V, head).  Per tile
//   * TMA loads of the x tile (two 64-column boxes, 128-byte swizzle) into a 3-deep ring, issued by
//     one thread two tiles ahead;
//   * y = x . S on the 5th-generation tensor cores: S is split once per CTA into two bf16 terms
//     (S = S_hi + S_lo + O(2^-17)) kept in shared memory as the K-major B operand; 2 terms x 8
//     k-steps of tcgen05.mma (M = 128 rows, N = 128, K = 16) accumulate in float32 in tensor memory;
//     two accumulators, and the MMAs of tile i+1 are issued when the epilogue of tile i starts, so
//     they run under it.  Lane 0 of every warp issues one of the 16 MMAs, so that no warp is held up
//     by the batch (a warp that is late delays all 16 at the next barrier); since their order is then
//     free, every MMA accumulates and the epilogue clears the accumulator after reading it;
//   * epilogue on all 16 warps.  Tensor-memory lane = row, so a thread owns 32 consecutive rotated
//     coordinates (2 blocks) of one row: tcgen05.ld, sign-test quantiser with certified margins,
//     packed stores, queued float64 re-decision of the ambiguous angles.
// There are no dedicated producer / MMA warps: the register file is split over four schedulers, and
// a 17th warp would cap every thread at 96 registers (the quantiser then spills).  The issuing
// threads do not block in practice: what they wait for was completed a tile earlier.
// Every mbarrier wait is bounded; a wait that gives up raises the CTA's abort flag, the remaining
// tiles are skipped, tensor memory is released and PQ_ERR_TIMEOUT is recorded.
#pragma once
#include <cuda.h>

namespace pq {

constexpr int kTcThreads = 512;
constexpr int kTcEpiThreads = 512;
constexpr int kTcStages = 3;
constexpr int kTcXBytes = 128 * 128 * 2;   // one x tile: 128 rows x 128 bf16
constexpr int kTcSBytes = 128 * 128 * 2;   // one bf16 term of S (B operand)
constexpr int kTcSmS = 0;                  // S_hi, S_lo
constexpr int kTcSmX = kTcSmS + 2 * kTcSBytes;
constexpr int kTcSmRowSq = kTcSmX + kTcStages * kTcXBytes;   // [4][128] float, then [4][128] bytes of level-4 nibbles
constexpr int kTcSmFq = kTcSmRowSq + 2048 + 512;             // FastQuant (40 B)
constexpr int kTcSmBar = kTcSmFq + 64;                       // full[3], tfull[2]
constexpr int kTcSmMisc = kTcSmBar + 128;                    // tmem base, abort flag
constexpr int kTcSmFix = kTcSmMisc + 64;                     // FixQueue
constexpr int kTcSmTotal = kTcSmFix + (int)sizeof(FixQueue) + 1024;  // + slack for 1024-byte alignment
constexpr int kTcSpin = 1 << 22;
static_assert(kFixSdBytes <= kTcSmRowSq, "the float64 copy of S must fit in the operand buffers");

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
__device__ __forceinline__ bool tc_mbar_test(uint32_t bar, uint32_t parity) {  // non-blocking probe
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool tc_mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (tc_mbar_test(bar, parity)) return true;  // the usual case: completed a tile ago
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

__device__ __forceinline__ void tc_st16_zero(uint32_t taddr) {
  const uint32_t z = 0u;
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1,%1};" ::"r"(taddr), "r"(z)
      : "memory");
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
  uint8_t* l4s = reinterpret_cast<uint8_t*>(rowsq + 4 * 128);  // [4][128] level-4 codes of the row's column quarters
  const uint32_t bar_full = sb + kTcSmBar, bar_tfull = bar_full + 8 * kTcStages;
  const int n_tiles = n_row_tiles * 2 * a.n_kv_heads;

  // ---- set-up: barriers, tensor memory, S split into two bf16 terms in the B-operand layout
  if (tid == 0) {
    for (int s = 0; s < kTcStages; ++s) tc_mbar_init(bar_full + 8 * s, 1);
    for (int i = 0; i < 2; ++i) {
      tc_mbar_init(bar_tfull + 8 * i, kTcThreads / 32);   // one commit per warp
    }
    *abort_flag = 0;
    fixq->count[0] = fixq->count[1] = fixq->count[2] = fixq->count[3] = 0;
    load_fast_quant(a.tables, fq);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(sb + kTcSmMisc) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // B operand: B[n][k] = S[k][n]; two halves of 64 k; row n = 128 bytes, 16-byte chunk c stored at c ^ (n & 7).
  // A task is (row n, chunk of 8 consecutive k): 8 coalesced loads (lanes = consecutive n), one 16-byte store per term.
  for (int task = tid; task < 128 * 16; task += kTcThreads) {
    const int n = task & 127, oct = task >> 7;  // k = 8 * oct .. 8 * oct + 7
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float v0 = a.S[(8 * oct + 2 * i) * 128 + n], v1 = a.S[(8 * oct + 2 * i + 1) * 128 + n];
      const __nv_bfloat16 h0 = __float2bfloat16_rn(v0), h1 = __float2bfloat16_rn(v1);
      const __nv_bfloat16 l0 = __float2bfloat16_rn(v0 - __bfloat162float(h0));
      const __nv_bfloat16 l1 = __float2bfloat16_rn(v1 - __bfloat162float(h1));
      hi[i] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
      lo[i] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
    }
    const int half = oct >> 3, c = oct & 7;
    const int off = half * 16384 + n * 128 + ((c ^ (n & 7)) << 4);
    *reinterpret_cast<uint4*>(smem + kTcSmS + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    *reinterpret_cast<uint4*>(smem + kTcSmS + kTcSBytes + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the MMA unit
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  // Tile t = (row tile, K|V, head) with head fastest: t = head + n_kv_heads * hq, hq = 2 * row tile + kv.  A CTA's
  // tiles are gridDim.x apart; their coordinates are advanced without divisions.
  const int step_h = (int)gridDim.x % a.n_kv_heads, step_q = (int)gridDim.x / a.n_kv_heads;
  auto advance = [&](int& head, int& hq) {
    head += step_h;
    hq += step_q;
    if (head >= a.n_kv_heads) {
      head -= a.n_kv_heads;
      ++hq;
    }
  };
  // One thread issues the TMA loads of local tile `it` (tile blockIdx.x + it * gridDim.x = head + n_kv_heads * hq).
  int tma_issued = 0;  // local tiles whose copies this thread has issued (thread 0 only)
  auto issue_tma = [&](int it, int head, int hq) {
    const int tile = blockIdx.x + it * gridDim.x;
    if (tile >= n_tiles || *abort_flag) return;  // after a wait gave up nothing new is put in flight
    tma_issued = it + 1;
    const int s = it % kTcStages;
    // The stage is free: its previous tile (local tile it - 3) was multiplied before this thread passed the
    // wait for that tile's accumulator, two tiles ago.
    const int kv = hq & 1, rt = hq >> 1;
    const CUtensorMap* map = kv ? &maps.v : &maps.k;
    const uint32_t dst = sb + kTcSmX + s * kTcXBytes, bar = bar_full + 8 * s;
    tc_mbar_expect_tx(bar, kTcXBytes);
#pragma unroll
    for (int h = 0; h < 2; ++h)
      asm volatile(
          "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
          ::"r"(dst + h * 16384), "l"(map), "r"(h * 64), "r"(head), "r"(rt * 128), "r"(bar)
          : "memory");
  };
  // Lane 0 of every warp issues one of the 16 MMAs of local tile `it` into accumulator it & 1: issuer q takes
  // term q >> 3 of S, k-half (q >> 2) & 1 and k-step q & 3.  All MMAs accumulate (the accumulator is zero).
  // The accumulator is free: its previous tile was read and cleared by every warp before the CTA-wide barrier
  // that ended that tile, which this thread has passed.
  auto issue_mma = [&](int it, int q) {
    if (blockIdx.x + it * (int)gridDim.x >= n_tiles) return;
    const int s = it % kTcStages, acc = it & 1;
    if (!tc_mbar_wait(bar_full + 8 * s, (it / kTcStages) & 1, abort_flag)) return;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t off = ((q >> 2) & 1) * 16384 + (q & 3) * 32;
    tc_mma(tmem_base + acc * 128, tc_smem_desc(sb + kTcSmX + s * kTcXBytes + off),
           tc_smem_desc(sb + kTcSmS + (q >> 3) * kTcSBytes + off), 1u);
    tc_commit(bar_tfull + 8 * acc);   // this issuer's share of the accumulator is complete (and of the reads of the x stage)
  };
  // both accumulators start at zero
  {
    const uint32_t z = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (warp >> 2) * 32;
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j) tc_st16_zero(z + i * 128 + 16 * j);
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  }
  int head = (int)blockIdx.x % a.n_kv_heads, hq = (int)blockIdx.x / a.n_kv_heads;  // this tile
  int head2 = head, hq2 = hq;                                                      // the tile two ahead
  if (tid == 0) issue_tma(0, head2, hq2);
  advance(head2, hq2);
  if (tid == 0) issue_tma(1, head2, hq2);
  advance(head2, hq2);
  if (lane == 0) issue_mma(0, warp);
  __syncwarp();

  // ---- tile loop: all 16 warps are epilogue warps
  constexpr int o2 = 32 * kTokenBlock, o3 = o2 + 8 * kTokenBlock, o4 = o3 + 4 * kTokenBlock, orad = o4 + 2 * kTokenBlock;
  const int quarter = warp & 3;                  // tensor-memory lanes this warp may read
  const int cq = warp >> 2;                      // columns [32*cq, 32*cq + 32): blocks 2cq, 2cq+1
  const int r = quarter * 32 + lane;             // row of the tile
  const bool uniform = (a.tables->flags & kFlagUniformL1) != 0u;
  const bool sym = fq->sym != 0u;  // uniform over the grid
  const Layout L = make_layout(128, a.capacity);
  int rd_seq = 0, rd_first = 0, rd_count = 0, rd_start = -1;   // destination of the last row looked up
  int it = 0;
  for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++it, advance(head, hq)) {
    const int acc = it & 1;
    const int kv = hq & 1, rt = hq >> 1;
    // A wait that gives up must not leave the loop: the other warps may be past it and would wait
    // for this one at the named barriers.  The tile is skipped instead (warp-uniform).
    const bool ready = __all_sync(0xffffffffu, tc_mbar_wait(bar_tfull + 8 * acc, (it >> 1) & 1, abort_flag));
    // keep the pipeline fed: loads two tiles ahead, the next tile's MMAs under this tile's epilogue
    if (tid == 0) issue_tma(it + 2, head2, hq2);
    advance(head2, hq2);
    if (lane == 0) issue_mma(it + 1, warp);
    __syncwarp();
    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * 128 + cq * 32;
    // pass 1: the thread's 32 coordinates and their share of the row's squared norm (the four column
    // quarters of a row are exchanged through shared memory)
    float sq = 0.f;
    float y[32];
    if (ready) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      tc_ld16(taddr, y);
      tc_ld16(taddr + 16, y + 16);
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
      for (int c = 0; c < 32; ++c) sq = fmaf(y[c], y[c], sq);
    } else {
#pragma unroll
      for (int c = 0; c < 32; ++c) y[c] = 0.f;
    }
    rowsq[cq * 128 + r] = sq;
    // only the four warps that share these 32 rows exchange their parts of the norm
    asm volatile("bar.sync %0, 128;" ::"r"(2 + quarter) : "memory");
    const RowMargins rm = make_row_margins(
        kRotErr * 1.0001f * sqrtf((rowsq[r] + rowsq[128 + r]) + (rowsq[256 + r] + rowsq[384 + r])), *fq);
    const int row = rt * 128 + r;
    uint8_t* tb = nullptr;
    int tok = 0;
    if (ready && row < a.total_tokens) {
      int seq, pos;
      if (row >= rd_first && row < rd_first + rd_count) {  // same sequence as this thread's previous row
        seq = rd_seq;
        pos = rd_start < 0 ? -1 : rd_start + (row - rd_first);
      } else {
        row_destination(a, row, &seq, &pos);
        rd_seq = seq;
        rd_first = a.cu_seqlens ? a.cu_seqlens[seq] : row;
        rd_count = a.cu_seqlens ? a.cu_seqlens[seq + 1] - rd_first : 1;
        rd_start = pos < 0 ? -1 : pos - (row - rd_first);
      }
      if (pos >= 0) {
        tb = a.cache + block_offset(L, a.n_kv_heads, seq, head, kv, pos);
        tok = pos % kTokenBlock;
      }
    }
    const int64_t xoff = (int64_t)row * a.token_stride + (int64_t)head * a.head_stride;
    // pass 2: one block at a time
    uint32_t l2acc = 0, l3acc = 0, l4acc = 0, racc = 0, sat = 0;
    unsigned long long leftbits = 0ull;
    if (ready) {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        FastBlock fb;
        if (sym) polar_quant_block_fast<true>(y + 16 * i, rm, *fq, &fb);
        else polar_quant_block_fast<false>(y + 16 * i, rm, *fq, &fb);
        if (!uniform) fb.amb |= 0xFFu;  // other level-1 codebooks: decide every level-1 angle exactly
        if (tb != nullptr) {
          *reinterpret_cast<uint32_t*>(tb + tok * 32 + cq * 8 + 4 * i) = fb.l1;
          l2acc |= fb.l2 << (8 * i);
          l3acc |= fb.l3 << (4 * i);
          l4acc |= fb.l4 << (2 * i);
          float rv = fb.radius;
          if (rv > 65504.f) { rv = 65504.f; ++sat; }
          racc |= (uint32_t)__half_as_ushort(__float2half_rn(rv)) << (16 * i);
          if (fb.amb) {
            uint32_t left;
            fix_push(fixq, fb.amb, xoff, tb, tok, 2 * cq + i, kv, &left);
            leftbits |= (unsigned long long)left << (15 * i);  // queue full: pushed again by fix_rounds
          }
        }
      }
      tc_st16_zero(taddr);  // leave the accumulator cleared for the next tile that uses it
      tc_st16_zero(taddr + 16);
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    l4s[cq * 128 + r] = (uint8_t)l4acc;
    if (tb != nullptr) {
      *reinterpret_cast<uint16_t*>(tb + o2 + tok * 8 + cq * 2) = (uint16_t)l2acc;
      tb[o3 + tok * 4 + cq] = (uint8_t)l3acc;
      *reinterpret_cast<uint32_t*>(tb + orad + tok * 16 + cq * 4) = racc;
      if (sat) atomicAdd(a.status + 2, (int)sat);
    }
    asm volatile("bar.sync 1, 512;" ::: "memory");
    if (tb != nullptr && (cq & 1) == 0)  // level-4 codes of four blocks share a byte: two column quarters
      tb[o4 + tok * 2 + (cq >> 1)] = (uint8_t)(l4s[cq * 128 + r] | (l4s[(cq + 1) * 128 + r] << 4));
    // Exact re-decisions are batched over tiles: drain the queue when it is 3/4 full (a push that
    // did not fit leaves the counter above the capacity) or after the CTA's last tile.
    const bool last_tile = tile + (int)gridDim.x >= n_tiles;
    if (last_tile) {
      // The operand buffers are idle now (every MMA and copy of this CTA has completed): stage S there as
      // float64 so that the last, largest batch of re-decisions reads it from shared memory.
      asm volatile("bar.sync 1, 512;" ::: "memory");
      double* Sd = reinterpret_cast<double*>(smem + kTcSmS);
      for (int idx = tid; idx < 128 * 128; idx += kTcThreads) {
        const int k = idx >> 7, n = idx & 127;
        Sd[((k & 15) * 8 + (k >> 4)) * kFixSdStride + n] = (double)__ldg(a.S + idx);
      }
      fix_rounds(a, fixq, leftbits, xoff, tb, tok, 2 * cq, kv, tid, kTcEpiThreads, 1, Sd);
    } else if (fix_should_drain(fixq)) {
      fix_rounds(a, fixq, leftbits, xoff, tb, tok, 2 * cq, kv, tid, kTcEpiThreads, 1);
    }
  }
  if (*abort_flag && tid == 0) {
    // gave up somewhere: let the copies that are still in flight land (bounded) before the CTA and its
    // shared memory go away
    for (int t = max(0, tma_issued - kTcStages); t < tma_issued; ++t)
      for (int i = 0; i < (1 << 16) && !tc_mbar_try(bar_full + 8 * (t % kTcStages), (t / kTcStages) & 1); ++i)
        __nanosleep(64);
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
  static int configured[kMaxDevices] = {};
  const int n_sm = configure_for_device(encode_tc_kernel, kTcSmTotal, configured);
  if (n_sm == 0) return PQ_ERR_CUDA;
  const int n_row_tiles = (a.total_tokens + 127) / 128;
  const int n_tiles = n_row_tiles * 2 * a.n_kv_heads;
  const int grid = n_tiles < n_sm ? n_tiles : n_sm;
  encode_tc_kernel<<<grid, kTcThreads, kTcSmTotal, stream>>>(a, maps, n_row_tiles);
  return 1;
}

}  // namespace pq
