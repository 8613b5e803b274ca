// Shared definitions of the PolarQuant CUDA library: device tables, packed-cache layout,
// exact (float64) polar quantiser of one 16-coordinate block.
#pragma once
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include <nvtx3/nvToolsExt.h>

#include "../../include/polarquant.h"

namespace pq {

// NVTX range around a C-ABI call (shows the call in a timeline next to its kernels; a no-op without a profiler).
struct NvtxRange {
  explicit NvtxRange(const char* name) { nvtxRangePushA(name); }
  ~NvtxRange() { nvtxRangePop(); }
  NvtxRange(const NvtxRange&) = delete;
  NvtxRange& operator=(const NvtxRange&) = delete;
};


constexpr int kTokenBlock = 64;  // tokens per cache token-block
constexpr int kMaxGroup = 8;     // query heads per kv head that one thread block of an attention kernel handles
constexpr int kBlockDim = 16;    // coordinates per polar block (L = 4 levels)

// Offsets of each level inside the concatenated centroid / boundary arrays.
__host__ __device__ constexpr int cen_off(int level) { return level == 1 ? 0 : 16 + 4 * (level - 2); }
__host__ __device__ constexpr int bnd_off(int level) { return level == 1 ? 0 : 15 + 3 * (level - 2); }

constexpr int kL1Cells = 128;            // cells per octant of the level-1 decision table
constexpr float kL1CellScale = 127.93f;  // cell = floor(t * kL1CellScale + 1/16): t = 1 still falls in the last cell

// Compiled form of the codebooks (built on the host by pq_build_tables, copied verbatim to
// the device by the caller).
struct Tables {
  // Decision lines: angle psi = atan2(b, a) is above boundary beta iff
  // b cos(beta) - a sin(beta) > 0 (given the half-plane bookkeeping at level 1).
  double bnd[PQ_N_BOUNDARIES];
  double bnd_cos[PQ_N_BOUNDARIES];
  double bnd_sin[PQ_N_BOUNDARIES];
  float bnd_cosf[PQ_N_BOUNDARIES];
  float bnd_sinf[PQ_N_BOUNDARIES];
  int32_t bnd_upper[16];  // level 1: boundary k lies in [0, pi]
  int32_t n_upper;        // number of level-1 boundaries in [0, pi]
  uint32_t flags;         // bit 0: level-1 boundaries are exactly k*pi/8 (uniform codebook)
  // cos / sin of the centroids (Algorithm 1, DeQuant).
  float cen_cos[PQ_N_CENTROIDS];
  float cen_sin[PQ_N_CENTROIDS];
  // fp16 decode tables of the attention kernel.
  //   l1_hi[c], l1_lo[c] : (cos, sin) of level-1 centroid c as half2, split into the fp16 value and
  //                        the fp16 rounding residual (hi + lo carries ~22 bits)
  //   u_tab[s][i]        : sub-block s (0..3) of a block, i = c2 | c3 << 2 | c4 << 4: the product of
  //                        the level-4, level-3 and level-2 factors of the sub-block's two level-1
  //                        pairs, .x = half2 of the fp16 values, .y = half2 of the residuals
  uint32_t l1_hi[16];
  uint32_t l1_lo[16];
  uint2 u_tab[4][64];
  double bnd_tan2[9];  // tan^2 of the boundaries of levels 2, 3, 4 (decisions on squared radii)
  //   t1p_hi[e], t1p_lo[e] : e = one byte of level-1 codes (pair a | pair b << 4): .x = (cos a, cos b), .y = (sin a, sin b)
  //                          so that a half2 of the two pairs' multipliers multiplies element-wise
  uint2 t1p_hi[256];
  uint2 t1p_lo[256];
  uint32_t reserved[30];
  // Level-1 decision table for any codebook (see quant_level1_table_push): octant o = (b < 0) << 2 | (a < 0) << 1 |
  // (|b| > |a|), cell = position of t = min(|a|,|b|) / max(|a|,|b|) in [0, 1].  .x = float bits of tau, the
  // one boundary value of t the cell decides against (NaN: the cell cannot be decided by one comparison);
  // .y = code for t < tau in bits 28..31, code for t > tau in bits 24..27.
  uint2 l1_cells[8][kL1Cells];
};

constexpr uint32_t kFlagUniformL1 = 1u;
// bit 1: at every level >= 2 the boundaries are b, pi/4, pi/2 - b (tan^2: T, 1, 1/T to 1e-9 relative), as for
// every Lloyd-Max codebook of the symmetric densities of Lemma 2
constexpr uint32_t kFlagSymmetricUpper = 2u;

// ------------------------------------------------------------------------------------------
// Packed cache layout.
//
// cache = [sequence b][kv head h][token-block j][K | V] blocks of kTokenBlock tokens.
// One block holds five planes, each token-major:
//   L1   : 4*nb bytes per token, byte i = level-1 codes 2i (low nibble) and 2i+1 (high nibble)
//   L2   : nb bytes per token,   byte i = level-2 codes 4i .. 4i+3, two bits each, LSB first
//   L3   : max(1, nb/2) bytes,   same packing of the 2*nb level-3 codes
//   L4   : max(1, nb/4) bytes,   same packing of the nb level-4 codes
//   radii: nb fp16 values per token
// nb = head_dim / 16.  At head_dim 128 this is 32 + 8 + 4 + 2 + 16 = 62 bytes per token and
// every plane starts on a 16-byte boundary.  Each token owns whole bytes in every plane, so
// tokens can be written independently (append needs no read-modify-write).
// ------------------------------------------------------------------------------------------
struct Layout {
  int nb;                  // 16-blocks per vector
  int b1, b2, b3, b4, br;  // bytes per token in each plane
  int o2, o3, o4, orad;    // plane offsets inside a token-block (o1 = 0)
  int block_bytes;         // bytes of one token-block (K or V)
  int n_blocks_cap;        // token-blocks per sequence
  int64_t head_bytes;      // bytes of one (sequence, head): n_blocks_cap * 2 * block_bytes
};

__host__ __device__ inline Layout make_layout(int head_dim, int capacity) {
  Layout L;
  L.nb = head_dim / kBlockDim;
  L.b1 = 4 * L.nb;
  L.b2 = L.nb;
  L.b3 = L.nb >= 2 ? L.nb / 2 : 1;
  L.b4 = L.nb >= 4 ? L.nb / 4 : 1;
  L.br = 2 * L.nb;
  L.o2 = kTokenBlock * L.b1;
  L.o3 = L.o2 + kTokenBlock * L.b2;
  L.o4 = L.o3 + kTokenBlock * L.b3;
  L.orad = L.o4 + kTokenBlock * L.b4;
  L.block_bytes = L.orad + kTokenBlock * L.br;
  L.n_blocks_cap = (capacity + kTokenBlock - 1) / kTokenBlock;
  L.head_bytes = (int64_t)L.n_blocks_cap * 2 * L.block_bytes;
  return L;
}

// Where the token-blocks of a sequence live.  The cache is a pool of pages; a page holds `page_tokens` tokens of every
// kv head, head-major: [kv head][token-block of the page][K | V] (Layout::head_bytes per head, with the layout made
// for page_tokens).  Contiguous cache (table == nullptr): sequence b owns page b, of `capacity` tokens.  Paged cache:
// logical page p of sequence b is physical page table[b * pages_per_seq + p] of a pool of n_pages.
struct Paging {
  const int32_t* table;
  int page_tokens;    // multiple of kTokenBlock (of 128 at head_dim 128 for the persistent decode kernel) when paged
  int pages_per_seq;
  int n_pages;
};
__host__ __device__ inline Paging contiguous_paging(int capacity, int batch) {
  Paging pg;
  pg.table = nullptr; pg.page_tokens = capacity; pg.pages_per_seq = 1; pg.n_pages = batch;
  return pg;
}

// Start of head h's part of the page that holds position `pos` of sequence b; -1 if the table names a page outside
// the pool.
__device__ __forceinline__ int64_t head_page_offset(const Layout& L, const Paging& pg, int n_kv_heads, int b, int h, int pos) {
  int page = b;
  if (pg.table != nullptr) {
    page = __ldg(pg.table + (int64_t)b * pg.pages_per_seq + pos / pg.page_tokens);
    if ((unsigned)page >= (unsigned)pg.n_pages) return -1;
  }
  return ((int64_t)page * n_kv_heads + h) * L.head_bytes;
}
// Start of the token-block that holds position `pos` of (sequence b, head h), K (kv=0) or V (kv=1); -1: bad page.
__device__ __forceinline__ int64_t block_offset_paged(int block_bytes, int64_t head_bytes, const int32_t* table, int page_tokens,
                                                   int pages_per_seq, int n_pages, int n_kv_heads, int b, int h, int kv, int pos) {
  const int page = __ldg(table + (int64_t)b * pages_per_seq + pos / page_tokens);
  if ((unsigned)page >= (unsigned)n_pages) return -1;
  return ((int64_t)page * n_kv_heads + h) * head_bytes + ((int64_t)((pos % page_tokens) / kTokenBlock) * 2 + kv) * block_bytes;
}
__device__ __forceinline__ int64_t block_offset(const Layout& L, const Paging& pg, int n_kv_heads, int b, int h, int kv, int pos) {
  if (pg.table != nullptr)
    return block_offset_paged(L.block_bytes, L.head_bytes, pg.table, pg.page_tokens, pg.pages_per_seq, pg.n_pages, n_kv_heads, b,
                              h, kv, pos);
  return ((int64_t)b * n_kv_heads + h) * L.head_bytes + ((int64_t)(pos / kTokenBlock) * 2 + kv) * L.block_bytes;
}

// ------------------------------------------------------------------------------------------
// Codes of one 16-coordinate block in canonical order.
// ------------------------------------------------------------------------------------------
struct BlockCodes {
  uint32_t l1;  // 8 codes x 4 bits, code j at bits [4j, 4j+4)
  uint32_t l2;  // 4 codes x 2 bits, LSB first
  uint32_t l3;  // 2 codes x 2 bits
  uint32_t l4;  // 1 code  x 2 bits
};

// Level-1 code of the pair (a, b): number of interior boundaries below atan2(b, a) mod 2pi.
__device__ inline uint32_t quant_level1_exact(double a, double b, const Tables& tb) {
  const bool upper = !(b < 0.0);  // psi in [0, pi]; b == -0.0 counts as upper (psi = 0 or pi)
  uint32_t code = 0;
#pragma unroll
  for (int k = 0; k < 15; ++k) {
    const double cross = b * tb.bnd_cos[k] - a * tb.bnd_sin[k];
    const bool above = cross > 0.0;
    const bool bu = tb.bnd_upper[k] != 0;
    code += bu ? (upper ? above : true) : (upper ? false : above);
  }
  return code;
}

// Level >= 2 code of the pair of radii (a, b), both >= 0.
__device__ inline uint32_t quant_upper_exact(double a, double b, int level, const Tables& tb) {
  const int o = bnd_off(level);
  uint32_t code = 0;
#pragma unroll
  for (int k = 0; k < 3; ++k) code += (b * tb.bnd_cos[o + k] - a * tb.bnd_sin[o + k]) > 0.0;
  return code;
}

// Polar (Algorithm 1) + Quant of one block in float64.  Returns the level-4 radius.
__device__ inline double polar_quant_block_exact(const double* y, const Tables& tb, BlockCodes& c) {
  double r1[8], r2[4], r3[2];
  c.l1 = c.l2 = c.l3 = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    c.l1 |= quant_level1_exact(y[2 * j], y[2 * j + 1], tb) << (4 * j);
    r1[j] = hypot(y[2 * j], y[2 * j + 1]);
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    c.l2 |= quant_upper_exact(r1[2 * j], r1[2 * j + 1], 2, tb) << (2 * j);
    r2[j] = hypot(r1[2 * j], r1[2 * j + 1]);
  }
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    c.l3 |= quant_upper_exact(r2[2 * j], r2[2 * j + 1], 3, tb) << (2 * j);
    r3[j] = hypot(r2[2 * j], r2[2 * j + 1]);
  }
  c.l4 = quant_upper_exact(r3[0], r3[1], 4, tb);
  return hypot(r3[0], r3[1]);
}

// Host side: remember the CUDA error behind a PQ_ERR_CUDA return (see pq_last_cuda_error).
void note_cuda_error(cudaError_t e);
// Test hook (pq_debug_fail_next_wait): returns true once after the hook was armed for `which`
// (1 = tensor-core encoder, 2 = head_dim-128 decode attention) and disarms it.
bool take_debug_wait_failure(int which);
int32_t paging_from(const pq_paging* p, int head_dim, Paging* out);
inline int32_t launch_status() {
  const cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) return PQ_OK;
  note_cuda_error(e);
  return PQ_ERR_CUDA;
}

// One-time, per-device launch configuration of a kernel that needs more than 48 KB of dynamic shared
// memory: the attribute belongs to the (kernel, device) pair, so the memo is indexed by the current
// device. `state` is a zero-initialised array the caller keeps per kernel; an entry holds the device's
// SM count once the kernel is configured there (atomic: host threads may call into the library
// concurrently; two that race on a device both set the same attribute). Returns the SM count, or 0 with
// the CUDA error noted.
constexpr int kMaxDevices = 64;
using DeviceMemo = std::atomic<int>[kMaxDevices];
template <typename Kernel>
inline int configure_for_device(Kernel kernel, int smem_bytes, DeviceMemo& state) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess && (dev < 0 || dev >= kMaxDevices)) e = cudaErrorInvalidDevice;
  if (e != cudaSuccess) {
    note_cuda_error(e);
    return 0;
  }
  const int known = state[dev].load(std::memory_order_acquire);
  if (known > 0) return known;
  int n_sm = 0;
  e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e == cudaSuccess && n_sm <= 0) e = cudaErrorInvalidDevice;
  if (e != cudaSuccess) {
    note_cuda_error(e);
    return 0;
  }
  state[dev].store(n_sm, std::memory_order_release);
  return n_sm;
}

// Record the first error seen.
__device__ inline void set_status(int32_t* status, int32_t code) {
  if (status != nullptr) atomicCAS(status, 0, code);
}

// Readers: offset of the K block of token-block jb of (sequence b, head h); its V block follows it, and so does the
// next token-block of the same page.  A page outside the pool is reported and page 0 is read instead (the output
// for that sequence is then meaningless, but no address outside the cache is formed).
__device__ __forceinline__ int64_t kv_block_pair_offset(const Layout& L, const Paging& pg, int n_kv_heads, int b, int h, int jb,
                                                        int32_t* status) {
  if (pg.table == nullptr) return ((int64_t)b * n_kv_heads + h) * L.head_bytes + (int64_t)jb * 2 * L.block_bytes;
  int64_t off = block_offset_paged(L.block_bytes, L.head_bytes, pg.table, pg.page_tokens, pg.pages_per_seq, pg.n_pages, n_kv_heads,
                                   b, h, 0, jb * kTokenBlock);
  if (off < 0) {
    set_status(status, PQ_ERR_INVALID_ARG);
    off = (int64_t)h * L.head_bytes;
  }
  return off;
}

}  // namespace pq
