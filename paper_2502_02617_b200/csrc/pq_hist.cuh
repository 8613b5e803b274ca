// Histograms of the observed angles (the sample the "online" codebook of Section 4.1 is clustered on); included by
// pq_encode.cu.  The angles of Algorithm 1's Polar are formed in float32 from the rotated coordinates and counted per
// level in n_bins bins of equal width over the level's range ([0, 2 pi) at level 1, [0, pi/2] above).  Against a
// float64 evaluation an angle within the float32 error of a bin edge (about 1e-5 rad) may fall in the neighbouring
// bin; the clustering sees a sample moved by less than a bin.
#pragma once

namespace pq {

constexpr int kHistMaxBins = PQ_HIST_MAX_BINS;

// atan(t) for t in [0, 1]: t * P(t^2), P of degree 5 fitted by least squares at Chebyshev nodes; the absolute error is
// below 2e-6 rad, a few thousandths of the narrowest bin.
__device__ __forceinline__ float hist_atan01(float t) {
  const float z = t * t;
  float p = -0.011465809307992458f;
  p = fmaf(p, z, 0.05195053294301033f);
  p = fmaf(p, z, -0.1157294437289238f);
  p = fmaf(p, z, 0.19323529303073883f);
  p = fmaf(p, z, -0.33256831765174866f);
  p = fmaf(p, z, 0.9999744892120361f);
  return p * t;
}

__device__ __forceinline__ float hist_rcp(float x) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

// Bin of atan2(b, a) in [0, 2 pi) (atan2(0, 0) = 0), `scale` = n_bins / (2 pi).
__device__ __forceinline__ int hist_bin_level1(float a, float b, float scale, int n_bins) {
  const float ax = fabsf(a), ay = fabsf(b);
  const float u = fmaxf(ax, ay), v = fminf(ax, ay);
  float phi = u > 0.f ? hist_atan01(fminf(v * hist_rcp(u), 1.f)) : 0.f;
  if (ay > ax) phi = 1.57079632679489662f - phi;
  if (a < 0.f) phi = 3.14159265358979324f - phi;
  if (b < 0.f) phi = 6.28318530717958648f - phi;
  return min((int)(phi * scale), n_bins - 1);
}

// Bin of atan2(sqrt(sb), sqrt(sa)) in [0, pi/2] from the squared radii, `scale` = n_bins / (pi/2).
__device__ __forceinline__ int hist_bin_upper(float sa, float sb, float scale, int n_bins) {
  const float M = fmaxf(sa, sb), m = fminf(sa, sb);
  float phi = M > 0.f ? hist_atan01(fminf(sqrtf(m * hist_rcp(M)), 1.f)) : 0.f;
  if (sb > sa) phi = 1.57079632679489662f - phi;
  return min((int)(phi * scale), n_bins - 1);
}

// Count the 15 angles of one 16-coordinate block into h[level - 1][bin] (shared or global 32-bit counters).
// A block with a non-finite coordinate (or an overflowing norm) is skipped and reported by the return value.
__device__ __forceinline__ bool hist_block(const float* y, uint32_t* h, int n_bins, float scale1, float scale_up) {
  float s1[8], s2[4], s3[2];
#pragma unroll
  for (int j = 0; j < 8; ++j) s1[j] = fmaf(y[2 * j], y[2 * j], y[2 * j + 1] * y[2 * j + 1]);
#pragma unroll
  for (int j = 0; j < 4; ++j) s2[j] = s1[2 * j] + s1[2 * j + 1];
  s3[0] = s2[0] + s2[1];
  s3[1] = s2[2] + s2[3];
  if (!(s3[0] + s3[1] < CUDART_INF_F)) return false;
  // all fifteen bins first (independent dependency chains that overlap), then the fifteen counts
  int bin[15];
#pragma unroll
  for (int j = 0; j < 8; ++j) bin[j] = hist_bin_level1(y[2 * j], y[2 * j + 1], scale1, n_bins);
#pragma unroll
  for (int j = 0; j < 4; ++j) bin[8 + j] = n_bins + hist_bin_upper(s1[2 * j], s1[2 * j + 1], scale_up, n_bins);
#pragma unroll
  for (int j = 0; j < 2; ++j) bin[12 + j] = 2 * n_bins + hist_bin_upper(s2[2 * j], s2[2 * j + 1], scale_up, n_bins);
  bin[14] = 3 * n_bins + hist_bin_upper(s3[0], s3[1], scale_up, n_bins);
#pragma unroll
  for (int j = 0; j < 15; ++j) atomicAdd(h + bin[j], 1u);
  return true;
}

// Add a CTA's 32-bit counters to the 64-bit histogram in global memory.
__device__ inline void hist_flush(const uint32_t* h, int n, unsigned long long* out, int tid, int n_threads) {
  for (int i = tid; i < n; i += n_threads)
    if (h[i]) atomicAdd(out + i, (unsigned long long)h[i]);
}

}  // namespace pq
