// General recursion depth and bit tables (Definition 1 and Algorithm 1 with any L <= log2 d levels and any bits per
// level; Section 4 counts b_FPN + (d - 1) b bits per vector for L = log2 d and b bits everywhere).  Plain kernels:
// float64 for the encoder (the codes are those of a float64 evaluation of Algorithm 1), float32 for attention; one
// thread block per vector, or per (sequence, kv head).  The tuned path of the other files is the L = 4, bits (4,2,2,2)
// case in its own layout; this one covers what the paper describes beyond it, at reference speed.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <math_constants.h>
#include <vector>

#include "pq_common.cuh"

namespace pq {

constexpr int kGenMaxLevels = PQ_GENERAL_MAX_LEVELS;
constexpr int kGenMaxBits = 6;
constexpr int kGenMaxDim = 256;
constexpr int kGenMaxCentroids = kGenMaxLevels << kGenMaxBits;

// A validated configuration with the derived sizes.  A row (one token of one head, K or V) holds, per level, the
// level's d / 2^l codes as one bit stream (code i at bits [i b, (i + 1) b), least significant first, padded to a
// byte), then padding to an even offset, then the d / 2^L block radii in fp16.  The cache is
// [sequence][kv head][K | V][token][row_bytes].
struct GenConfig {
  int d, L, nb, n_codes, n_cen, row_bytes, rad_off;
  int bits[kGenMaxLevels], cen_off[kGenMaxLevels], bnd_off[kGenMaxLevels], code_off[kGenMaxLevels], byte_off[kGenMaxLevels],
      level_bytes[kGenMaxLevels];
};

static int32_t make_gen_config(const pq_general_config* c, GenConfig* g) {
  if (c == nullptr) return PQ_ERR_INVALID_ARG;
  const int d = c->head_dim, L = c->n_levels;
  if (d < 2 || d > kGenMaxDim || (d & (d - 1)) || L < 1 || L > kGenMaxLevels || (1 << L) > d) return PQ_ERR_UNSUPPORTED;
  std::memset(g, 0, sizeof(*g));
  g->d = d; g->L = L; g->nb = d >> L; g->n_codes = d - g->nb;
  int cen = 0, bnd = 0, code = 0, byte = 0;
  for (int l = 0; l < L; ++l) {
    const int b = c->bits[l];
    if (b < 1 || b > kGenMaxBits) return PQ_ERR_UNSUPPORTED;
    g->bits[l] = b;
    g->cen_off[l] = cen; g->bnd_off[l] = bnd; g->code_off[l] = code; g->byte_off[l] = byte;
    g->level_bytes[l] = ((d >> (l + 1)) * b + 7) / 8;
    cen += 1 << b; bnd += (1 << b) - 1; code += d >> (l + 1); byte += g->level_bytes[l];
  }
  g->n_cen = cen;
  g->rad_off = (byte + 1) & ~1;
  g->row_bytes = g->rad_off + 2 * g->nb;
  return PQ_OK;
}

__host__ __device__ inline int64_t gen_row_offset(const GenConfig& g, int n_kv_heads, int capacity, int b, int h, int kv, int tok) {
  return ((((int64_t)b * n_kv_heads + h) * 2 + kv) * capacity + tok) * g.row_bytes;
}

// Code `idx` of level l (0-based) of a row.
__device__ __forceinline__ uint32_t gen_get_code(const uint8_t* row, const GenConfig& g, int l, int idx) {
  const int bit = idx * g.bits[l];
  const uint8_t* p = row + g.byte_off[l] + (bit >> 3);
  const uint32_t two = (uint32_t)p[0] | ((bit & 7) + g.bits[l] > 8 ? (uint32_t)p[1] << 8 : 0u);
  return (two >> (bit & 7)) & ((1u << g.bits[l]) - 1u);
}

// Rotated coordinate i of a row: the block radius times, level by level from the top, cos or sin of the centroid of
// the angle above coordinate i (Algorithm 1, DeQuant).
__device__ __forceinline__ float gen_decode_coord(const uint8_t* row, const GenConfig& g, int i, const float* cen_cos,
                                                  const float* cen_sin) {
  float v = __half2float(reinterpret_cast<const __half*>(row + g.rad_off)[i >> g.L]);
  for (int l = g.L - 1; l >= 0; --l) {
    const uint32_t code = gen_get_code(row, g, l, i >> (l + 1));
    v *= ((i >> l) & 1) ? cen_sin[g.cen_off[l] + code] : cen_cos[g.cen_off[l] + code];
  }
  return v;
}

struct GenEncodeArgs {
  GenConfig g;
  const void* K;
  const void* V;
  int in_dtype;
  int64_t token_stride, head_stride;
  const int32_t* cu_seqlens;
  int batch, total_tokens, n_kv_heads, capacity;
  const float* S;
  const double* boundaries;
  uint8_t* cache;
  const int32_t* lens;
  int32_t* status;
};

// One thread block of max(d, 32) threads per vector (row, K | V, head): y = x . S in float64, the polar tree level by
// level (thread j forms angle j of the level), codes = number of boundaries below the angle, then the bit streams.
__global__ void gen_encode_kernel(GenEncodeArgs a) {
  __shared__ double ra[kGenMaxDim], rb[kGenMaxDim];
  __shared__ uint8_t codes[kGenMaxDim];
  __shared__ int dest[2];
  const GenConfig& g = a.g;
  const int j = threadIdx.x, d = g.d;
  const int64_t v = blockIdx.x;
  const int head = (int)(v % a.n_kv_heads), kv = (int)((v / a.n_kv_heads) & 1);
  const int row = (int)(v / (2 * a.n_kv_heads));
  if (j == 0) {   // destination: the sequence that owns the row (largest b with cu[b] <= row) and its position
    int lo = 0, hi = a.batch - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (a.cu_seqlens[mid] <= row) lo = mid; else hi = mid - 1;
    }
    const int first = a.cu_seqlens[lo], count = a.cu_seqlens[lo + 1] - first, start = a.lens[lo];
    dest[0] = lo;
    dest[1] = (start < 0 || start + count > a.capacity) ? -1 : start + (row - first);
    if (dest[1] < 0) set_status(a.status, PQ_ERR_CAPACITY);
  }
  if (j < d) {
    const int64_t idx = (int64_t)row * a.token_stride + (int64_t)head * a.head_stride + j;
    const float x = a.in_dtype == PQ_DTYPE_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(kv ? a.V : a.K)[idx])
                                                : reinterpret_cast<const float*>(kv ? a.V : a.K)[idx];
    if (!isfinite(x)) {
      atomicAdd(a.status + 1, 1);
      set_status(a.status, PQ_ERR_NONFINITE);
    }
    ra[j] = (double)x;
  }
  __syncthreads();
  if (j < d) {
    double acc = 0.0;
    for (int k = 0; k < d; ++k) acc = fma(ra[k], (double)__ldg(a.S + (int64_t)k * d + j), acc);
    rb[j] = acc;
  }
  __syncthreads();
  double* src = rb;
  double* dst = ra;
  for (int l = 0; l < g.L; ++l) {
    const int n = d >> (l + 1);
    if (j < n) {
      const double x0 = src[2 * j], x1 = src[2 * j + 1];
      double psi = atan2(x1, x0);
      if (l == 0 && psi < 0.0) psi += 6.283185307179586476925286766559;
      const double* bnd = a.boundaries + g.bnd_off[l];
      int code = 0;
      for (int k = 0; k < (1 << g.bits[l]) - 1; ++k) code += psi > bnd[k];
      codes[g.code_off[l] + j] = (uint8_t)code;
      dst[j] = sqrt(x0 * x0 + x1 * x1);
    }
    __syncthreads();
    double* t = src; src = dst; dst = t;
  }
  const int pos = dest[1];
  if (pos < 0) return;
  uint8_t* out = a.cache + gen_row_offset(g, a.n_kv_heads, a.capacity, dest[0], head, kv, pos);
  for (int t = j; t < g.rad_off; t += blockDim.x) {   // byte t of the row: gather its bits
    int l = g.L - 1;
    while (l > 0 && t < g.byte_off[l]) --l;
    uint32_t byte = 0;
    if (t < g.byte_off[l] + g.level_bytes[l]) {
      const int b = g.bits[l], n = d >> (l + 1);
      for (int bit = 0; bit < 8; ++bit) {
        const int pos_bit = (t - g.byte_off[l]) * 8 + bit, idx = pos_bit / b;
        if (idx < n) byte |= (((uint32_t)codes[g.code_off[l] + idx] >> (pos_bit % b)) & 1u) << bit;
      }
    }
    out[t] = (uint8_t)byte;
  }
  if (j < g.nb) {
    double r = src[j];
    if (r > 65504.0) {
      r = 65504.0;
      atomicAdd(a.status + 2, 1);
    }
    reinterpret_cast<__half*>(out + g.rad_off)[j] = __double2half(r);
  }
}

__global__ void gen_advance_lens_kernel(const int32_t* cu_seqlens, int batch, int capacity, int32_t* lens) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  const int count = cu_seqlens[b + 1] - cu_seqlens[b], start = lens[b];
  if (start >= 0 && start + count <= capacity) lens[b] = start + count;
}

__global__ void gen_unpack_kernel(GenConfig g, int n_kv_heads, const uint8_t* cache, int batch, int capacity, int n_tokens,
                                  uint8_t* codes, __half* radii) {
  const int64_t n = (int64_t)batch * n_kv_heads * 2 * n_tokens;
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= n) return;
  const int tok = (int)(v % n_tokens), kv = (int)((v / n_tokens) & 1);
  const int h = (int)((v / (2 * (int64_t)n_tokens)) % n_kv_heads), b = (int)(v / (2 * (int64_t)n_tokens * n_kv_heads));
  const uint8_t* row = cache + gen_row_offset(g, n_kv_heads, capacity, b, h, kv, tok);
  for (int l = 0; l < g.L; ++l)
    for (int i = 0; i < (g.d >> (l + 1)); ++i) codes[v * g.n_codes + g.code_off[l] + i] = (uint8_t)gen_get_code(row, g, l, i);
  for (int i = 0; i < g.nb; ++i) radii[v * g.nb + i] = reinterpret_cast<const __half*>(row + g.rad_off)[i];
}

// DeQuant of one vector per thread block, including the final S^T.
__global__ void gen_dequant_kernel(GenConfig g, int n_kv_heads, const float* S, const double* centroids, const uint8_t* cache,
                                   int capacity, int n_tokens, float* x_hat) {
  __shared__ float cc[kGenMaxCentroids], cs[kGenMaxCentroids], ys[kGenMaxDim];
  const int j = threadIdx.x, d = g.d;
  for (int i = j; i < g.n_cen; i += blockDim.x) {
    cc[i] = (float)cos(centroids[i]);
    cs[i] = (float)sin(centroids[i]);
  }
  __syncthreads();
  const int64_t v = blockIdx.x;
  const int tok = (int)(v % n_tokens), kv = (int)((v / n_tokens) & 1);
  const int h = (int)((v / (2 * (int64_t)n_tokens)) % n_kv_heads), b = (int)(v / (2 * (int64_t)n_tokens * n_kv_heads));
  const uint8_t* row = cache + gen_row_offset(g, n_kv_heads, capacity, b, h, kv, tok);
  if (j < d) ys[j] = gen_decode_coord(row, g, j, cc, cs);
  __syncthreads();
  if (j < d) {
    float acc = 0.f;
    for (int k = 0; k < d; ++k) acc = fmaf(ys[k], __ldg(S + (int64_t)j * d + k), acc);
    x_hat[v * d + j] = acc;
  }
}

struct GenAttnArgs {
  GenConfig g;
  int n_q_heads, n_kv_heads, capacity, io_dtype;
  float scale;
  const float* S;
  const double* centroids;
  const void* q;
  const uint8_t* cache;
  const int32_t* lens;
  void* out;
  int32_t* status;
};

// Eq. 3, one thread block of 256 threads per (kv head, sequence): q' = q S once, then chunks of 256 tokens: a thread
// per token decodes the key coordinate by coordinate and forms the scores of the group's heads, a warp per head keeps
// the running maximum and denominator, a thread per coordinate decodes the values and accumulates P . V; the
// result is normalised and rotated back by S^T.
constexpr int kGenAttnThreads = 256;
__global__ void __launch_bounds__(kGenAttnThreads) gen_attention_kernel(GenAttnArgs a) {
  extern __shared__ float gsm[];
  const GenConfig& g = a.g;
  const int d = g.d, grp = a.n_q_heads / a.n_kv_heads, hk = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;
  float* cc = gsm;                          // [n_cen]
  float* cs = cc + g.n_cen;                 // [n_cen]
  float* qs = cs + g.n_cen;                 // [grp][d]  q' = q S * scale * log2(e); later the normalised output
  float* sc = qs + grp * d;                 // [grp][kGenAttnThreads]
  float* m_sm = sc + grp * kGenAttnThreads; // [grp]
  float* l_sm = m_sm + kMaxGroup;
  float* corr_sm = l_sm + kMaxGroup;
  float* qin = corr_sm + kMaxGroup;         // [grp][d] the queries as given
  for (int i = tid; i < g.n_cen; i += kGenAttnThreads) {
    cc[i] = (float)cos(a.centroids[i]);
    cs[i] = (float)sin(a.centroids[i]);
  }
  const int64_t q0 = ((int64_t)b * a.n_q_heads + hk * grp) * d;
  for (int i = tid; i < grp * d; i += kGenAttnThreads)
    qin[i] = a.io_dtype == PQ_DTYPE_BF16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.q)[q0 + i])
                                         : reinterpret_cast<const float*>(a.q)[q0 + i];
  if (tid < grp) {
    m_sm[tid] = -CUDART_INF_F;
    l_sm[tid] = 0.f;
  }
  __syncthreads();
  for (int i = tid; i < grp * d; i += kGenAttnThreads) {
    const int h = i / d, jj = i - h * d;
    float acc = 0.f;
    for (int k = 0; k < d; ++k) acc = fmaf(qin[h * d + k], __ldg(a.S + (int64_t)k * d + jj), acc);
    qs[i] = acc * a.scale * 1.4426950408889634f;
  }
  int len = a.lens[b];
  len = len < 0 ? 0 : (len > a.capacity ? a.capacity : len);
  float acc[kMaxGroup];
#pragma unroll
  for (int h = 0; h < kMaxGroup; ++h) acc[h] = 0.f;
  __syncthreads();
  const uint8_t* kbase = a.cache + gen_row_offset(g, a.n_kv_heads, a.capacity, b, hk, 0, 0);
  const uint8_t* vbase = a.cache + gen_row_offset(g, a.n_kv_heads, a.capacity, b, hk, 1, 0);
  for (int c0 = 0; c0 < len; c0 += kGenAttnThreads) {
    const int n = min(kGenAttnThreads, len - c0);
    if (tid < n) {
      const uint8_t* row = kbase + (int64_t)(c0 + tid) * g.row_bytes;
      float s[kMaxGroup];
#pragma unroll
      for (int h = 0; h < kMaxGroup; ++h) s[h] = 0.f;
      for (int i = 0; i < d; ++i) {
        const float kvv = gen_decode_coord(row, g, i, cc, cs);
#pragma unroll
        for (int h = 0; h < kMaxGroup; ++h)
          if (h < grp) s[h] = fmaf(qs[h * d + i], kvv, s[h]);
      }
#pragma unroll
      for (int h = 0; h < kMaxGroup; ++h)
        if (h < grp) sc[h * kGenAttnThreads + tid] = s[h];
    }
    __syncthreads();
    for (int h = warp; h < grp; h += kGenAttnThreads / 32) {
      float mx = -CUDART_INF_F;
      for (int t = lane; t < n; t += 32) mx = fmaxf(mx, sc[h * kGenAttnThreads + t]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_new = fmaxf(m_sm[h], mx);
      float sum = 0.f;
      for (int t = lane; t < n; t += 32) {
        const float p = exp2f(sc[h * kGenAttnThreads + t] - m_new);
        sc[h * kGenAttnThreads + t] = p;
        sum += p;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (lane == 0) {
        const float corr = exp2f(m_sm[h] - m_new);
        corr_sm[h] = corr;
        l_sm[h] = l_sm[h] * corr + sum;
        m_sm[h] = m_new;
      }
    }
    __syncthreads();
    if (tid < d) {
#pragma unroll
      for (int h = 0; h < kMaxGroup; ++h)
        if (h < grp) acc[h] *= corr_sm[h];
      for (int t = 0; t < n; ++t) {
        const float vv = gen_decode_coord(vbase + (int64_t)(c0 + t) * g.row_bytes, g, tid, cc, cs);
#pragma unroll
        for (int h = 0; h < kMaxGroup; ++h)
          if (h < grp) acc[h] = fmaf(sc[h * kGenAttnThreads + t], vv, acc[h]);
      }
    }
    __syncthreads();
  }
  if (tid < d) {
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h)
      if (h < grp) qs[h * d + tid] = len > 0 ? acc[h] / l_sm[h] : 0.f;
  }
  if (tid == 0 && len <= 0) set_status(a.status, PQ_ERR_EMPTY);
  __syncthreads();
  for (int i = tid; i < grp * d; i += kGenAttnThreads) {   // x_hat_j = sum_k y_hat_k S[j][k]
    const int h = i / d, jj = i - h * d;
    float o = 0.f;
    for (int k = 0; k < d; ++k) o = fmaf(qs[h * d + k], __ldg(a.S + (int64_t)jj * d + k), o);
    if (a.io_dtype == PQ_DTYPE_BF16) reinterpret_cast<__nv_bfloat16*>(a.out)[q0 + i] = __float2bfloat16(o);
    else reinterpret_cast<float*>(a.out)[q0 + i] = o;
  }
}

}  // namespace pq

namespace {
const double kPiG = 3.14159265358979323846264338327950288;
// Lloyd-Max centroids of the level's analytic density (Lemma 2) by Simpson quadrature; level is 1-based.
void gen_fit_level(int level, int n, double* theta, double* beta) {
  const double lo = 0.0, hi = level == 1 ? 2.0 * kPiG : 0.5 * kPiG;
  const int expo = (1 << (level - 1)) - 1;
  auto moments = [&](double a, double b, double* m0, double* m1) {
    const int panels = 2048;
    const double h = (b - a) / panels;
    double s0 = 0.0, s1 = 0.0;
    for (int i = 0; i <= panels; ++i) {
      const double p = a + h * i, w = (i == 0 || i == panels) ? 1.0 : ((i & 1) ? 4.0 : 2.0);
      const double f = level == 1 ? 1.0 : std::pow(std::sin(2.0 * p), expo);
      s0 += w * f;
      s1 += w * f * p;
    }
    *m0 = s0 * h / 3.0;
    *m1 = s1 * h / 3.0;
  };
  for (int k = 0; k < n; ++k) theta[k] = lo + (k + 0.5) * (hi - lo) / n;
  if (level > 1) {  // start inside the bulk of the density (it concentrates around pi/4 as the level grows)
    const double width = 4.0 / std::sqrt((double)(expo + 1));
    for (int k = 0; k < n; ++k) theta[k] = 0.25 * kPiG + (k + 0.5 - 0.5 * n) * std::fmin(hi / n, width / n);
  }
  for (int it = 0; it < 100000; ++it) {
    double delta = 0.0;
    for (int k = 0; k + 1 < n; ++k) beta[k] = 0.5 * (theta[k] + theta[k + 1]);
    for (int k = 0; k < n; ++k) {
      const double a = k == 0 ? lo : beta[k - 1], b = k == n - 1 ? hi : beta[k];
      double m0, m1;
      moments(a, b, &m0, &m1);
      const double t = m0 > 0.0 ? m1 / m0 : 0.5 * (a + b);
      delta = std::fmax(delta, std::fabs(t - theta[k]));
      theta[k] = t;
    }
    if (delta < 1e-14) break;
  }
  for (int k = 0; k + 1 < n; ++k) beta[k] = 0.5 * (theta[k] + theta[k + 1]);
}
}  // namespace

extern "C" {

int32_t pq_general_sizes(const pq_general_config* cfg, int32_t* n_centroids, int32_t* n_boundaries, int32_t* n_codes,
                         int32_t* n_radii, int32_t* row_bytes) {
  pq::GenConfig g;
  const int32_t st = pq::make_gen_config(cfg, &g);
  if (st != PQ_OK) return st;
  if (n_centroids) *n_centroids = g.n_cen;
  if (n_boundaries) *n_boundaries = g.n_cen - g.L;
  if (n_codes) *n_codes = g.n_codes;
  if (n_radii) *n_radii = g.nb;
  if (row_bytes) *row_bytes = g.row_bytes;
  return PQ_OK;
}

int32_t pq_general_fit_codebooks(const pq_general_config* cfg, double* centroids_host, double* boundaries_host) {
  pq::GenConfig g;
  const int32_t st = pq::make_gen_config(cfg, &g);
  if (st != PQ_OK) return st;
  if (centroids_host == nullptr || boundaries_host == nullptr) return PQ_ERR_INVALID_ARG;
  for (int l = 0; l < g.L; ++l) gen_fit_level(l + 1, 1 << g.bits[l], centroids_host + g.cen_off[l], boundaries_host + g.bnd_off[l]);
  return PQ_OK;
}

int64_t pq_general_cache_bytes(const pq_general_config* cfg, int32_t batch, int32_t n_kv_heads, int32_t capacity) {
  pq::GenConfig g;
  const int32_t st = pq::make_gen_config(cfg, &g);
  if (st != PQ_OK) return st;
  if (batch <= 0 || n_kv_heads <= 0 || capacity <= 0) return PQ_ERR_INVALID_ARG;
  return (int64_t)batch * n_kv_heads * 2 * capacity * g.row_bytes;
}

int32_t pq_general_encode_kv(const pq_general_config* cfg, int32_t n_kv_heads, const float* S_dev,
                             const double* boundaries_dev, const void* K_dev, const void* V_dev, int32_t in_dtype,
                             int64_t token_stride, int64_t head_stride, const int32_t* cu_seqlens_dev, int32_t batch,
                             int32_t total_tokens, void* cache_dev, int32_t* cache_lens_dev, int32_t capacity,
                             int32_t* status_dev, void* stream) {
  pq::GenEncodeArgs a;
  const int32_t st = pq::make_gen_config(cfg, &a.g);
  if (st != PQ_OK) return st;
  if (!S_dev || !boundaries_dev || !K_dev || !V_dev || !cu_seqlens_dev || !cache_dev || !cache_lens_dev || !status_dev)
    return PQ_ERR_INVALID_ARG;
  if (n_kv_heads <= 0 || batch <= 0 || total_tokens < 0 || capacity <= 0 || token_stride < 0 || head_stride < 0) return PQ_ERR_INVALID_ARG;
  if (in_dtype != PQ_DTYPE_F32 && in_dtype != PQ_DTYPE_BF16) return PQ_ERR_UNSUPPORTED;
  if ((int64_t)total_tokens * 2 * n_kv_heads >= (1ll << 31)) return PQ_ERR_UNSUPPORTED;
  if (((uintptr_t)boundaries_dev & 7) || ((uintptr_t)cache_dev & 1)) return PQ_ERR_ALIGNMENT;
  if (total_tokens == 0) return PQ_OK;
  a.K = K_dev; a.V = V_dev; a.in_dtype = in_dtype; a.token_stride = token_stride; a.head_stride = head_stride;
  a.cu_seqlens = cu_seqlens_dev; a.batch = batch; a.total_tokens = total_tokens; a.n_kv_heads = n_kv_heads; a.capacity = capacity;
  a.S = S_dev; a.boundaries = boundaries_dev; a.cache = reinterpret_cast<uint8_t*>(cache_dev); a.lens = cache_lens_dev;
  a.status = status_dev;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const unsigned n_vec = (unsigned)((int64_t)total_tokens * 2 * n_kv_heads);
  pq::gen_encode_kernel<<<n_vec, a.g.d < 32 ? 32 : a.g.d, 0, s>>>(a);
  pq::gen_advance_lens_kernel<<<(batch + 127) / 128, 128, 0, s>>>(cu_seqlens_dev, batch, capacity, cache_lens_dev);
  return pq::launch_status();
}

int32_t pq_general_decode_attention(const pq_general_config* cfg, int32_t n_q_heads, int32_t n_kv_heads, const float* S_dev,
                                    const double* centroids_dev, const void* q_dev, int32_t io_dtype, const void* cache_dev,
                                    const int32_t* cache_lens_dev, int32_t batch, int32_t capacity, float scale,
                                    void* out_dev, int32_t* status_dev, void* stream) {
  pq::GenAttnArgs a;
  const int32_t st = pq::make_gen_config(cfg, &a.g);
  if (st != PQ_OK) return st;
  if (!S_dev || !centroids_dev || !q_dev || !cache_dev || !cache_lens_dev || !out_dev || !status_dev) return PQ_ERR_INVALID_ARG;
  if (batch <= 0 || batch > 65535 || n_q_heads <= 0 || n_kv_heads <= 0 || capacity <= 0 || n_q_heads % n_kv_heads) return PQ_ERR_INVALID_ARG;
  if (n_q_heads / n_kv_heads > pq::kMaxGroup) return PQ_ERR_UNSUPPORTED;
  if (io_dtype != PQ_DTYPE_F32 && io_dtype != PQ_DTYPE_BF16) return PQ_ERR_UNSUPPORTED;
  if ((uintptr_t)centroids_dev & 7) return PQ_ERR_ALIGNMENT;
  a.n_q_heads = n_q_heads; a.n_kv_heads = n_kv_heads; a.capacity = capacity; a.io_dtype = io_dtype; a.scale = scale;
  a.S = S_dev; a.centroids = centroids_dev; a.q = q_dev; a.cache = reinterpret_cast<const uint8_t*>(cache_dev);
  a.lens = cache_lens_dev; a.out = out_dev; a.status = status_dev;
  const int grp = n_q_heads / n_kv_heads;
  const size_t smem = sizeof(float) * ((size_t)2 * a.g.n_cen + (size_t)2 * grp * a.g.d + (size_t)grp * pq::kGenAttnThreads +
                                      3 * pq::kMaxGroup);
  static pq::DeviceMemo configured;
  if (pq::configure_for_device(pq::gen_attention_kernel, 64 * 1024, configured) == 0) return PQ_ERR_CUDA;
  if (smem > 64 * 1024) return PQ_ERR_UNSUPPORTED;
  dim3 grid(n_kv_heads, batch);
  pq::gen_attention_kernel<<<grid, pq::kGenAttnThreads, smem, reinterpret_cast<cudaStream_t>(stream)>>>(a);
  return pq::launch_status();
}

int32_t pq_general_unpack_codes(const pq_general_config* cfg, int32_t n_kv_heads, const void* cache_dev, int32_t batch,
                                int32_t capacity, int32_t n_tokens, uint8_t* codes_dev, void* radii_dev, void* stream) {
  pq::GenConfig g;
  const int32_t st = pq::make_gen_config(cfg, &g);
  if (st != PQ_OK) return st;
  if (!cache_dev || !codes_dev || !radii_dev || batch <= 0 || n_kv_heads <= 0 || n_tokens <= 0 || n_tokens > capacity)
    return PQ_ERR_INVALID_ARG;
  const int64_t n = (int64_t)batch * n_kv_heads * 2 * n_tokens;
  pq::gen_unpack_kernel<<<(unsigned)((n + 127) / 128), 128, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      g, n_kv_heads, reinterpret_cast<const uint8_t*>(cache_dev), batch, capacity, n_tokens, codes_dev,
      reinterpret_cast<__half*>(radii_dev));
  return pq::launch_status();
}

int32_t pq_general_dequant_kv(const pq_general_config* cfg, int32_t n_kv_heads, const float* S_dev, const double* centroids_dev,
                              const void* cache_dev, int32_t batch, int32_t capacity, int32_t n_tokens, float* x_hat_dev,
                              void* stream) {
  pq::GenConfig g;
  const int32_t st = pq::make_gen_config(cfg, &g);
  if (st != PQ_OK) return st;
  if (!S_dev || !centroids_dev || !cache_dev || !x_hat_dev || batch <= 0 || n_kv_heads <= 0 || n_tokens <= 0 || n_tokens > capacity)
    return PQ_ERR_INVALID_ARG;
  const int64_t n = (int64_t)batch * n_kv_heads * 2 * n_tokens;
  if (n >= (1ll << 31)) return PQ_ERR_UNSUPPORTED;
  pq::gen_dequant_kernel<<<(unsigned)n, g.d < 32 ? 32 : g.d, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      g, n_kv_heads, S_dev, centroids_dev, reinterpret_cast<const uint8_t*>(cache_dev), capacity, n_tokens, x_hat_dev);
  return pq::launch_status();
}

}  // extern "C"
