// Pieces shared by the selection kernels and the score kernel's fused tail: the block metric of
// Eq. 6 (and its entropy variant) computed by one warp, and the hash behind the random-order variant.
#pragma once
#include "common.cuh"

namespace tca {

enum { kMetricHHI = 0, kMetricEntropy = 1, kMetricRandom = 2 };

struct MetricOut {            // where a kernel leaves h_j; hkey == nullptr: do not compute it
  unsigned long long* hkey;   // [U][m] order-preserving keys of h
  double* h_out;              // optional [U][m]
  int m, b, mode;
  double alpha;
};

inline int metric_mode(const tca_params* prm) {
  if (prm->flags & TCA_FLAG_RANDOM_ORDER) return kMetricRandom;
  if (prm->flags & TCA_FLAG_ENTROPY_INDEX) return kMetricEntropy;
  return kMetricHHI;
}

#ifdef __CUDACC__

// SplitMix64 finaliser (Steele, Lea, Flood 2014).
__device__ __forceinline__ unsigned long long splitmix64(unsigned long long x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}
// Sort key in [0, 1) of block j of unit u for the random-order variant.
__device__ __forceinline__ double random_block_key(int seed, int u, int j) {
  const unsigned long long base =
      splitmix64((static_cast<unsigned long long>(static_cast<unsigned>(seed)) << 32) | static_cast<unsigned>(u));
  return double(splitmix64(base + static_cast<unsigned long long>(j)) >> 11) * 0x1.0p-53;
}

// h_j of Eq. 6 for the block whose b log-scores start at `ls` (global or shared memory), computed
// by one whole warp; every lane returns the value.  The concentration term is evaluated on
// s_i / max_i s_i (it does not change under a common factor), which never divides zero by zero.
//   kMetricHHI      1 - sum s^2 / (sum s)^2          (the paper's Herfindahl-Hirschman variant)
//   kMetricEntropy  -sum p ln p, p = s / sum s       (the ablation's block entropy)
__device__ __forceinline__ double block_metric_warp(const double* ls, int b, double alpha, int mode, int lane) {
  double v[4];
  double top = -1.0e308;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const int i = s * 32 + lane;
    v[s] = (i < b) ? ls[i] : -1.0e308;
    top = fmax(top, v[s]);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) top = fmax(top, shfl_xor_double(top, off));
  double se = 0.0, se2 = 0.0;   // se2: sum e^2 (HHI) or sum e * (log s - top) (entropy)
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const int i = s * 32 + lane;
    if (i < b) {
      const double e = double(expf(float(v[s] - top)));
      se += e;
      se2 += (mode == kMetricEntropy) ? (e > 0.0 ? e * (v[s] - top) : 0.0) : e * e;
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    se += shfl_xor_double(se, off);
    se2 += shfl_xor_double(se2, off);
  }
  const double mass = exp(top) * se;
  // entropy: -sum (e/se) (ln e - ln se) = ln se - (sum e ln e) / se
  const double conc = (mode == kMetricEntropy) ? log(se) - se2 / se : 1.0 - se2 / (se * se);
  return (1.0 - alpha) * mass + alpha * conc;
}

#endif  // __CUDACC__

}  // namespace tca
