// Tensor-core encoder for head_dim 128, bf16 inputs (included by pq_encode.cu).
//
// Persistent CTAs (one per SM, 16 warps) loop over tiles of 128 rows x one (K|V, head).  The 16 warps form
// four groups ("slots") of four warps; a slot owns one of four 128-column accumulators in tensor memory
// and takes every fourth tile of the CTA.  Per tile
//   * TMA loads of the x tile (two 64-column boxes, 128-byte swizzle) into a 3-deep ring; the copy of
//     tile i+3 is issued as soon as the MMAs of tile i, which read the same ring stage, have completed;
//   * y = x . S on the 5th-generation tensor cores: S is split once per CTA into three bf16 terms (exact
//     for a float32 S) kept in shared memory as the K-major B operand; 3 terms x 8 k-steps of tcgen05.mma
//     (M = 128 rows, N = 128, K = 16) accumulate in float32 in the slot's accumulator.  One thread of the
//     slot issues them for the slot's next tile as soon as the current tile's last coordinates have been
//     read into registers, so the tensor work runs under the quantiser of the last two blocks (and the
//     other three slots are in their epilogues anyway);
//   * epilogue on the slot's four warps.  Tensor-memory lane = row and a warp may read its own quarter of
//     the lanes, so a thread owns one whole row (8 blocks): one pass over the accumulator for the row norm
//     (the certified margins need it), a second pass of tcgen05.ld of 32 coordinates at a time through the
//     sign-test quantiser, packed stores of whole plane entries of the token, queued float64 re-decision of
//     the ambiguous angles (one queue per slot; all 16 warps take them together after the CTA's last tile,
//     a slot drains alone only when its queue fills up).
// Per-row work (norm, margins, cache destination, stores) is paid once per 8 blocks, and the only
// synchronisation in the loop is two named barriers of the slot's 128 threads per tile.
// There are no dedicated producer / MMA warps: the register file is split over four schedulers, and
// a 17th warp would cap every thread at 96 registers (the quantiser then spills).
// Every mbarrier wait is bounded; a wait that gives up raises the CTA's abort flag, the remaining
// tiles are skipped (the loops keep their shape, so the named barriers stay consistent), copies in
// flight are drained, tensor memory is released and PQ_ERR_TIMEOUT is recorded.
#pragma once
#include <cuda.h>

#include "pq_tc_common.cuh"

namespace pq {

constexpr int kTcThreads = 512;
constexpr int kTcSlots = 4;                // accumulators in tensor memory = groups of four warps
constexpr int kTcSlotThreads = kTcThreads / kTcSlots;
constexpr int kTcStages = 3;               // x tiles in flight
constexpr int kTcTerms = 3;                // bf16 terms of S (exact for a float32 S)
constexpr int kTcXBytes = 128 * 128 * 2;   // one x tile: 128 rows x 128 bf16
constexpr int kTcSBytes = 128 * 128 * 2;   // one bf16 term of S (B operand)
using TcFixQueue = FixQueueT<256>;
constexpr int kTcSmS = 0;
constexpr int kTcSmX = kTcSmS + kTcTerms * kTcSBytes;
constexpr int kTcSmFq = kTcSmX + kTcStages * kTcXBytes;      // FastQuant
constexpr int kTcSmBar = kTcSmFq + kFastQuantBytes;                       // x_full[kTcStages], acc_full[kTcSlots]
constexpr int kTcSmMisc = kTcSmBar + 64;                     // tmem base, abort flag, copies issued per stage
constexpr int kTcSmFix = kTcSmMisc + 64;                     // one TcFixQueue per slot
constexpr int kTcSmL1 = kTcSmFix + kTcSlots * (int)sizeof(TcFixQueue);  // copy of Tables::l1_cells (codebooks other than the analytic ones)
constexpr int kTcSmTotal = kTcSmL1 + 8 * kL1Cells * 8 + 1024;             // + slack for 1024-byte alignment
static_assert(kTcTerms == 3, "kRotErrTc is the bound for three terms");
static_assert(sizeof(TcFixQueue) % 16 == 0, "queues are laid out back to back");
static_assert(kTcSmTotal <= 227 * 1024, "shared memory of one CTA");
static_assert(4 * PQ_HIST_MAX_BINS * 4 <= kTcSlots * (int)sizeof(TcFixQueue), "the histogram takes the queues' place");
static_assert(kFixSdBytes <= kTcSmFq, "the float64 copy of S must fit in the operand buffers");

struct TcMaps {
  CUtensorMap k, v;
};

// Non-finite elements among the 128 bf16 inputs of one vector (read again from global memory: only
// rows whose rotated norm is not finite get here).
__device__ inline int count_nonfinite_bf16(const void* base, int64_t xoff) {
  const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(base) + xoff);
  int bad = 0;
  for (int i = 0; i < 16; ++i) {
    const uint4 w = __ldg(p + i);
    const uint32_t v[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      bad += ((v[k] & 0x7F80u) == 0x7F80u);          // exponent all ones: Inf or NaN
      bad += ((v[k] & 0x7F800000u) == 0x7F800000u);
    }
  }
  return bad;
}

// kHist: the same pipeline up to the rotated coordinates in registers, which are then counted into the angle
// histograms (pq_hist.cuh) instead of being quantised; the shared memory of the re-decision queues holds the CTA's
// histogram (4 levels x n_bins 32-bit counters: a CTA would have to take 2^32 / 8192 tiles to overflow one).
// kPaged: the cache lies behind a block table (the other instantiations carry none of that code).
template <bool kHist, bool kPaged>
__global__ void __launch_bounds__(kTcThreads, 1)
encode_tc_kernel(EncodeArgs a, const __grid_constant__ TcMaps maps, int n_row_tiles) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sb = tc_smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // The kernel that advances the lengths may be set up now; it waits (griddepcontrol.wait) until this grid has
  // completed and its writes are visible, so only its launch latency is hidden.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int quarter = warp & 3;            // tensor-memory lanes this warp may read: rows 32 * quarter ..
  const int slot = warp >> 2;              // accumulator and tile sequence of this group of four warps
  const int st = quarter * 32 + lane;      // thread index inside the slot = row of the tile
  // The slot's issuing thread (TMA, MMAs).  The four warps of a slot sit on the four schedulers; the issuing threads
  // of the four slots are spread over them too, so that no scheduler carries all of that extra work (the other
  // warps of a slot would wait for the slow one at every barrier).
  const bool leader = quarter == slot && lane == 0;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kTcSmMisc + 4);
  volatile int* copies_issued = reinterpret_cast<volatile int*>(smem + kTcSmMisc + 8);  // [kTcStages]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kTcSmMisc);
  FastQuant* fq = reinterpret_cast<FastQuant*>(smem + kTcSmFq);
  TcFixQueue* fixq = reinterpret_cast<TcFixQueue*>(smem + kTcSmFix) + slot;
  const uint32_t bar_xfull = sb + kTcSmBar, bar_acc = bar_xfull + 8 * kTcStages;
  const int n_tiles = n_row_tiles * 2 * a.n_kv_heads;

  // Local tile `it` of this CTA is tile blockIdx.x + it * gridDim.x = head + n_kv_heads * (2 * row tile + kv); it
  // uses ring stage it % kTcStages and belongs to slot it % kTcSlots.
  // One thread issues the TMA loads of local tile `it`.  The caller knows that the stage is free: the MMAs of
  // local tile it - kTcStages, which read it, have completed.
  auto issue_tma = [&](int it) {
    const int tile = blockIdx.x + it * gridDim.x;
    if (tile >= n_tiles || *abort_flag) return;  // after a wait gave up nothing new is put in flight
    const int s = it % kTcStages;
    const int head = tile % a.n_kv_heads, hq = tile / a.n_kv_heads;
    const int kv = hq & 1, rt = hq >> 1;
    const CUtensorMap* map = kv ? &maps.v : &maps.k;
    const uint32_t dst = sb + kTcSmX + s * kTcXBytes, bar = bar_xfull + 8 * s;
    copies_issued[s] = copies_issued[s] + 1;
    tc_mbar_expect_tx(bar, kTcXBytes);
#pragma unroll
    for (int h = 0; h < 2; ++h)
      asm volatile(
          "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
          ::"r"(dst + h * 16384), "l"(map), "r"(h * 64), "r"(head), "r"(rt * 128), "r"(bar)
          : "memory");
  };

  // ---- set-up: barriers, first copies, tensor memory, S split into bf16 terms in the B-operand layout
  if (tid == 0) {
    for (int s = 0; s < kTcStages; ++s) {
      tc_mbar_init(bar_xfull + 8 * s, 1);
      copies_issued[s] = 0;
    }
    for (int i = 0; i < kTcSlots; ++i) tc_mbar_init(bar_acc + 8 * i, 1);   // one commit by the slot's issuing thread
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // Launched as a programmatic dependent of the kernel before it in the stream (which may have produced K and V):
    // its results are read only after this wait; the set-up around it overlaps that kernel's tail.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int it = 0; it < kTcStages; ++it) issue_tma(it);  // the first tiles arrive while S is split
    if (!kHist) {
      load_fast_quant(a.tables, fq);
      fq->l1_cells = reinterpret_cast<const uint2*>(smem + kTcSmL1);  // the copy made below
    }
  }
  uint32_t* hist_s = reinterpret_cast<uint32_t*>(smem + kTcSmFix);
  if (kHist) {
    for (int i = tid; i < 4 * a.n_bins; i += kTcThreads) hist_s[i] = 0u;
  } else {
    if (st < 4) fixq->count[st] = 0;
    if ((a.tables->flags & (kFlagSymmetricUpper | kFlagUniformL1)) != (kFlagSymmetricUpper | kFlagUniformL1)) {
      const uint2* src = &a.tables->l1_cells[0][0];
      uint2* dst = reinterpret_cast<uint2*>(smem + kTcSmL1);
      for (int i = tid; i < 8 * kL1Cells; i += kTcThreads) dst[i] = __ldg(src + i);
    }
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(sb + kTcSmMisc) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // B operand: B[n][k] = S[k][n]; two halves of 64 k; row n = 128 bytes, 16-byte chunk c stored at c ^ (n & 7).
  // A task is (row n, chunk of 8 consecutive k): 8 coalesced loads (lanes = consecutive n), one 16-byte store per
  // term.
  {
    constexpr int kTasks = 128 * 16 / kTcThreads;  // per thread
    float v[kTasks][8];
#pragma unroll
    for (int j = 0; j < kTasks; ++j) {             // all loads first: one round trip to L2 instead of kTasks
      const int task = tid + j * kTcThreads, n = task & 127, oct = task >> 7;
#pragma unroll
      for (int i = 0; i < 8; ++i) v[j][i] = __ldg(a.S + (8 * oct + i) * 128 + n);
    }
#pragma unroll
    for (int j = 0; j < kTasks; ++j) {
      const int task = tid + j * kTcThreads, n = task & 127, oct = task >> 7;  // k = 8 * oct .. 8 * oct + 7
      uint32_t term[kTcTerms][4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float v0 = v[j][2 * i], v1 = v[j][2 * i + 1];
#pragma unroll
        for (int t = 0; t < kTcTerms; ++t) {
          const __nv_bfloat16 h0 = __float2bfloat16_rn(v0), h1 = __float2bfloat16_rn(v1);
          term[t][i] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
          v0 -= __bfloat162float(h0);  // exact: the residual of a bf16 rounding fits float32
          v1 -= __bfloat162float(h1);
        }
      }
      const int half = oct >> 3, c = oct & 7;
      const int off = half * 16384 + n * 128 + ((c ^ (n & 7)) << 4);
#pragma unroll
      for (int t = 0; t < kTcTerms; ++t)
        *reinterpret_cast<uint4*>(smem + kTcSmS + t * kTcSBytes + off) = make_uint4(term[t][0], term[t][1], term[t][2], term[t][3]);
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the MMA unit
  asm volatile("griddepcontrol.wait;" ::: "memory");            // every thread reads lengths and writes the cache below
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  // The slot's issuing thread multiplies local tile `it` into the slot's accumulator.  The accumulator is free:
  // the slot's four warps have read the previous tile out of it before the barrier that precedes this call.
  // All MMAs of the tile come from this thread, in order: the first overwrites, the others accumulate.
  const uint64_t desc_hi = tc_smem_desc(0u) & 0xFFFFFFFF00000000ull;  // the address field is in the low word
  const uint32_t bdesc_lo = (uint32_t)tc_smem_desc(sb + kTcSmS);
  auto issue_mmas = [&](int it) {
    if (blockIdx.x + it * (int)gridDim.x >= n_tiles) return;
    const int s = it % kTcStages;
    // The copy of the tile is issued by another slot's thread (when the tile kTcStages back has been
    // multiplied).  A parity wait taken before that would be satisfied by the stage's previous phase, so
    // first wait (bounded) until the copy has been issued: the previous phase is complete by then.
    bool ok = false;
    for (int i = 0; i < kTcSpin && !ok; ++i) {
      ok = copies_issued[s] > it / kTcStages;
      if (!ok && i > 32) {
        __nanosleep(64);
        if (*abort_flag) break;
      }
    }
    if (!ok) *abort_flag = 1;
    ok = ok && tc_mbar_wait(bar_xfull + 8 * s, (it / kTcStages) & 1, abort_flag);
    if (ok && (a.debug & 1u) && blockIdx.x == 0 && it == 0) {  // test hook: report this wait as failed
      *abort_flag = 1;
      ok = false;
    }
    if (!ok) return;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t adesc_lo = (uint32_t)tc_smem_desc(sb + kTcSmX + s * kTcXBytes);
#pragma unroll
    for (int q = 0; q < 8 * kTcTerms; ++q) {
      const uint32_t off = ((q >> 2) & 1) * 16384 + (q & 3) * 32;  // k-half, k-step inside the 128-byte swizzled row
      tc_mma(tmem_base + slot * 128, desc_hi | (adesc_lo + (off >> 4)),
             desc_hi | (bdesc_lo + (((q >> 3) * kTcSBytes + off) >> 4)), q ? 1u : 0u);
    }
    tc_commit(bar_acc + 8 * slot);  // the accumulator is complete and the x stage has been read
  };

  // ---- tile loop of this slot
  constexpr int o2 = 32 * kTokenBlock, o3 = o2 + 8 * kTokenBlock, o4 = o3 + 4 * kTokenBlock, orad = o4 + 2 * kTokenBlock;
  const bool analytic = kHist || fq->analytic != 0u;  // uniform over the grid
  const float hist_scale1 = (float)a.n_bins * 0.159154943091895336f, hist_scale_up = (float)a.n_bins * 0.636619772367581343f;
  int hist_bad = 0;
  const Layout L = make_layout(128, a.pg.page_tokens);
  const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + slot * 128;
  const int slot_bar = 1 + slot;
  int rd_seq = 0, rd_first = 0, rd_count = 0, rd_start = -1;   // destination of the last row looked up
  if (leader) issue_mmas(slot);
  __syncwarp();
  for (int it = slot; blockIdx.x + it * (int)gridDim.x < n_tiles; it += kTcSlots) {
    const int tile = blockIdx.x + it * gridDim.x;
    const int head = tile % a.n_kv_heads, hq = tile / a.n_kv_heads;
    const int kv = hq & 1, rt = hq >> 1;
    // A wait that gives up must not leave the loop: the other warps of the slot would wait for this one at the
    // slot's barriers.  The tile is skipped instead (warp-uniform): it is quantised as zeros and not stored.
    const bool ready = __all_sync(0xffffffffu, tc_mbar_wait(bar_acc + 8 * slot, (it / kTcSlots) & 1, abort_flag));
    if (leader && ready) issue_tma(it + kTcStages);  // the stage of this tile is free again
    const int row = rt * 128 + st;
    const int64_t xoff = (int64_t)row * a.token_stride + (int64_t)head * a.head_stride;
    uint8_t* tb = nullptr;
    int tok = 0;
    unsigned long long left[2] = {0ull, 0ull};
    float y[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) y[i] = 0.f;
    if (kHist) {
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        if (ready) tc_ld32(taddr + 32 * c, y);
        if (c == 3) {  // as below: the accumulator is free for the slot's next tile
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          asm volatile("bar.sync %0, %1;" ::"r"(slot_bar), "n"(kTcSlotThreads) : "memory");
          if (leader) issue_mmas(it + kTcSlots);
          __syncwarp();
        }
        if (ready && row < a.total_tokens) {
          hist_bad += !hist_block(y, hist_s, a.n_bins, hist_scale1, hist_scale_up);
          hist_bad += !hist_block(y + 16, hist_s, a.n_bins, hist_scale1, hist_scale_up);
        }
      }
      continue;
    }
    // pass 1: squared norm of the row (four partial sums)
    float sq[4] = {0.f, 0.f, 0.f, 0.f};
    if (ready) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        tc_ld32(taddr + 32 * c, y);
#pragma unroll
        for (int i = 0; i < 32; ++i) sq[i & 3] = fmaf(y[i], y[i], sq[i & 3]);
      }
    }
    const float sqsum = (sq[0] + sq[1]) + (sq[2] + sq[3]);
    bool bad_row = false;
    if (!(sqsum < CUDART_INF_F) && row < a.total_tokens) {  // NaN or overflow: look at the inputs
      const int bad = count_nonfinite_bf16(kv ? a.V : a.K, xoff);
      if (bad) {
        atomicAdd(a.status + 1, bad);
        set_status(a.status, PQ_ERR_NONFINITE);
        bad_row = true;
      }
    }
    const RowMargins rm = make_row_margins(1.0001f * sqrtf(sqsum), kRotErrTc, *fq);
    if (ready && row < a.total_tokens) {
      int seq, pos;
      if (row >= rd_first && row < rd_first + rd_count) {  // same sequence as this thread's previous row
        seq = rd_seq;
        pos = rd_start < 0 ? -1 : rd_start + (row - rd_first);
      } else {
        row_destination<kPaged>(a, row, &seq, &pos);
        rd_seq = seq;
        rd_first = a.cu_seqlens ? a.cu_seqlens[seq] : row;
        rd_count = a.cu_seqlens ? a.cu_seqlens[seq + 1] - rd_first : 1;
        rd_start = pos < 0 ? -1 : pos - (row - rd_first);
      }
      if (pos >= 0) {
        tb = a.cache + (kPaged ? block_offset(L, a.pg, a.n_kv_heads, seq, head, kv, pos)
                               : block_offset(L, contiguous_paging(0, 0), a.n_kv_heads, seq, head, kv, pos));
        tok = pos % kTokenBlock;
      }
    }
    // pass 2: 32 coordinates (two blocks) at a time; the two blocks are quantised in one straight-line
    // piece of code (their instruction streams interleave), the rare queue pushes come after both
    uint32_t l2lo = 0, l2hi = 0, l3acc = 0, l4acc = 0, sat = 0;
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      if (ready) tc_ld32(taddr + 32 * c, y);
      if (c == 3) {
        // The last coordinates are in registers: the accumulator is free.  The slot's next tile is multiplied
        // while this one's last two blocks are quantised.
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("bar.sync %0, %1;" ::"r"(slot_bar), "n"(kTcSlotThreads) : "memory");
        if (leader) issue_mmas(it + kTcSlots);
        __syncwarp();
      }
      FastBlock fb0, fb1;
      if (analytic) {
        polar_quant_block_fast<true>(y, rm, *fq, &fb0);
        polar_quant_block_fast<true>(y + 16, rm, *fq, &fb1);
      } else {
        polar_quant_block_fast<false>(y, rm, *fq, &fb0);
        polar_quant_block_fast<false>(y + 16, rm, *fq, &fb1);
      }
      float r0 = fb0.radius, r1 = fb1.radius;
      sat += (r0 > 65504.f) + (r1 > 65504.f);
      r0 = fminf(r0, 65504.f);
      r1 = fminf(r1, 65504.f);
      uint32_t racc = (uint32_t)__half_as_ushort(__float2half_rn(r0)) | ((uint32_t)__half_as_ushort(__float2half_rn(r1)) << 16);
      const uint32_t l2c = fb0.l2 | (fb1.l2 << 8);
      l3acc |= (fb0.l3 | (fb1.l3 << 4)) << (8 * c);
      l4acc |= (fb0.l4 | (fb1.l4 << 2)) << (4 * c);
      if (c < 2) l2lo |= l2c << (16 * c);
      else l2hi |= l2c << (16 * (c - 2));
      uint32_t amb0 = fb0.amb, amb1 = fb1.amb;
      if (tb != nullptr) {
        if (bad_row) fb0.l1 = fb1.l1 = racc = amb0 = amb1 = 0u;
        *reinterpret_cast<uint2*>(tb + tok * 32 + c * 8) = make_uint2(fb0.l1, fb1.l1);
        *reinterpret_cast<uint32_t*>(tb + orad + tok * 16 + c * 4) = racc;
        if (amb0 | amb1) {
          uint32_t rest0 = 0, rest1 = 0;
          if (amb0) fix_push(fixq, amb0, xoff, tb, tok, 2 * c, kv, &rest0);
          if (amb1) fix_push(fixq, amb1, xoff, tb, tok, 2 * c + 1, kv, &rest1);
          // queue full: pushed again by fix_rounds
          left[c >> 1] |= ((unsigned long long)rest0 | ((unsigned long long)rest1 << 15)) << (30 * (c & 1));
        }
      }
    }
    if (tb != nullptr) {
      if (bad_row) l2lo = l2hi = l3acc = l4acc = sat = 0u;  // a row with non-finite inputs is stored as the zero vector
      *reinterpret_cast<uint2*>(tb + o2 + tok * 8) = make_uint2(l2lo, l2hi);
      *reinterpret_cast<uint32_t*>(tb + o3 + tok * 4) = l3acc;
      *reinterpret_cast<uint16_t*>(tb + o4 + tok * 2) = (uint16_t)l4acc;
      if (sat) atomicAdd(a.status + 2, (int)sat);
    }
    // End of the tile for the slot.  The barrier decides, for all 128 threads alike, whether the slot has to take
    // its queued exact re-decisions now: when a push did not fit or a region is 3/4 full.  Otherwise they wait
    // for the end of the CTA's work, where all 16 warps take them together (the float64 pipe is slow, and a slot
    // that drains alone holds up its own tiles for as long).
    const bool drain = bar_or(slot_bar, kTcSlotThreads, (left[0] | left[1]) != 0ull || fix_should_drain(fixq));
    if (drain) fix_rounds(a, fixq, left, xoff, tb, tok, 0, kv, st, kTcSlotThreads, slot_bar);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (kHist) {
    if (hist_bad) {
      atomicAdd(a.status + 1, hist_bad);
      set_status(a.status, PQ_ERR_NONFINITE);
    }
    hist_flush(hist_s, 4 * a.n_bins, a.hist, tid, kTcThreads);
  }
  // Every MMA and copy of this CTA has completed (each was waited for by its slot), so the operand buffers are
  // idle: put a float64 copy of S there (rows permuted, see fix_sd_row) for the queued exact re-decisions.
  double* Sd = reinterpret_cast<double*>(smem + kTcSmS);
  if (!kHist && !*abort_flag) {
    constexpr int kPer = 128 * 128 / kTcThreads;
    float sv[kPer];
#pragma unroll
    for (int j = 0; j < kPer; ++j) sv[j] = __ldg(a.S + tid + j * kTcThreads);
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
      const int idx = tid + j * kTcThreads;
      Sd[fix_sd_row(idx >> 7) * kFixSdStride + (idx & 127)] = (double)sv[j];
    }
    __syncthreads();
  }
  if (!kHist)
    fix_process(fixq - slot, kTcSlots, tid, kTcThreads, a.K, a.V, a.in_dtype, a.S, *abort_flag ? (const double*)nullptr : Sd,
                *a.tables, a.status);
  if (*abort_flag && tid < kTcStages && copies_issued[tid] > 0) {
    // gave up somewhere: let the copies that are still in flight land (bounded) before the CTA and its
    // shared memory go away
    for (int i = 0; i < (1 << 16) && !tc_mbar_try(bar_xfull + 8 * tid, (copies_issued[tid] - 1) & 1); ++i) __nanosleep(64);
  }
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
  if (tid == 0 && *abort_flag) set_status(a.status, PQ_ERR_TIMEOUT);
}

// Tensor maps for the K and V inputs ([tokens][heads][128] bf16 with element strides).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_tiled() {
  static const EncodeTiledFn fn = [] {  // looked up once per process (thread-safe initialisation)
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      return reinterpret_cast<EncodeTiledFn>(p);
    return static_cast<EncodeTiledFn>(nullptr);
  }();
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

// Launch the tensor-core encoder (or its histogram form) if the inputs allow it.  Returns 1 if launched, 0 if not
// applicable, or a negative status.
template <bool kHist, bool kPaged>
static int32_t try_launch_tc(const EncodeArgs& a, cudaStream_t stream) {
  if (a.head_dim != 128 || a.in_dtype != PQ_DTYPE_BF16 || a.total_tokens < 128) return 0;
  if ((a.token_stride & 7) || (a.head_stride & 7) || a.head_stride < 128 || a.token_stride < 128) return 0;
  if (((uintptr_t)a.K | (uintptr_t)a.V) & 15) return 0;
  if (a.n_kv_heads > 1 && a.head_stride * 2 >= ((int64_t)1 << 40)) return 0;
  EncodeTiledFn fn = get_encode_tiled();
  if (fn == nullptr) return 0;
  TcMaps maps;
  if (!make_x_map(fn, &maps.k, a.K, a.n_kv_heads, a.total_tokens, a.token_stride, a.head_stride)) return 0;
  if (!make_x_map(fn, &maps.v, a.V, a.n_kv_heads, a.total_tokens, a.token_stride, a.head_stride)) return 0;
  static DeviceMemo configured;  // one per instantiation
  const int n_sm = configure_for_device(encode_tc_kernel<kHist, kPaged>, kTcSmTotal, configured);
  if (n_sm == 0) return PQ_ERR_CUDA;
  const int n_row_tiles = (a.total_tokens + 127) / 128;
  const int n_tiles = n_row_tiles * 2 * a.n_kv_heads;
  const int grid = n_tiles < n_sm ? n_tiles : n_sm;
  EncodeArgs args = a;
  if (take_debug_wait_failure(1)) args.debug |= 1u;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = kTcSmTotal;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];   // may be set up while the kernel before it in the stream finishes (it waits inside)
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, encode_tc_kernel<kHist, kPaged>, args, maps, n_row_tiles) != cudaSuccess) {
    cudaGetLastError();
    return PQ_ERR_CUDA;
  }
  return 1;
}
static int32_t try_launch_encode_tc(const EncodeArgs& a, cudaStream_t stream) {
  return a.pg.table != nullptr ? try_launch_tc<false, true>(a, stream) : try_launch_tc<false, false>(a, stream);
}
static int32_t try_launch_hist_tc(const EncodeArgs& a, cudaStream_t stream) { return try_launch_tc<true, false>(a, stream); }

}  // namespace pq
