// tca_score: token importance of Eq. 5 in the log domain.
//
// Pass 1 (score_logits_kernel) streams K once with 128-bit loads, 16 lanes per key row,
// accumulates the G dot products of a query group in fp64 (products of bf16 or fp32
// inputs are exact in fp64, so the logits are exact up to summation rounding), reduces
// across lanes with a transposing warp-shuffle butterfly (one exchange per output
// instead of four), writes the logits and a per-CTA (max, sum-exp) partial per head.
// Pass 2 (score_finalize_kernel) merges the partials into each head's log-sum-exp and
// turns logits into  log( (1/G) * sum_g softmax_g[j] ).
#include "common.cuh"

namespace tca {
namespace {

constexpr int kThreads = 256;
constexpr int kGroups = kThreads / 16;  // 16-lane groups per CTA, one key row each

template <int G>
struct ScoreCfg {
  static constexpr int R = (G == 1) ? 16 : (G == 2) ? 8 : 4;   // rows per lane group per step
  static constexpr int NV = R * G;                             // values reduced per step
  static constexpr int NB = (NV + 15) / 16;                    // 16-value butterflies
  static constexpr int NVP = NB * 16;
};

// Raw 16-lane row slice: EPL elements per lane.
template <typename T, int EPL>
struct RowSlice;
template <>
struct RowSlice<__nv_bfloat16, 8> {
  uint4 raw;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { raw = __ldcs(reinterpret_cast<const uint4*>(p)); }
  __device__ __forceinline__ void zero() { raw = make_uint4(0, 0, 0, 0); }
  __device__ __forceinline__ double get(int e) const {
    uint32_t w = (e < 2) ? raw.x : (e < 4) ? raw.y : (e < 6) ? raw.z : raw.w;
    return (e & 1) ? bf16_hi_to_double(w) : bf16_lo_to_double(w);
  }
};
template <>
struct RowSlice<__nv_bfloat16, 4> {
  uint2 raw;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { raw = __ldcs(reinterpret_cast<const uint2*>(p)); }
  __device__ __forceinline__ void zero() { raw = make_uint2(0, 0); }
  __device__ __forceinline__ double get(int e) const {
    uint32_t w = (e < 2) ? raw.x : raw.y;
    return (e & 1) ? bf16_hi_to_double(w) : bf16_lo_to_double(w);
  }
};
template <>
struct RowSlice<float, 4> {
  float4 raw;
  __device__ __forceinline__ void load(const float* p) { raw = __ldcs(reinterpret_cast<const float4*>(p)); }
  __device__ __forceinline__ void zero() { raw = make_float4(0, 0, 0, 0); }
  __device__ __forceinline__ double get(int e) const {
    return double(e == 0 ? raw.x : e == 1 ? raw.y : e == 2 ? raw.z : raw.w);
  }
};
template <>
struct RowSlice<float, 8> {
  float4 a, b;
  __device__ __forceinline__ void load(const float* p) {
    a = __ldcs(reinterpret_cast<const float4*>(p));
    b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
  }
  __device__ __forceinline__ void zero() { a = b = make_float4(0, 0, 0, 0); }
  __device__ __forceinline__ double get(int e) const {
    const float4& v = e < 4 ? a : b;
    int i = e & 3;
    return double(i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w);
  }
};

__device__ __forceinline__ double elt_to_double(float x) { return double(x); }
__device__ __forceinline__ double elt_to_double(__nv_bfloat16 x) { return double(__bfloat162float(x)); }

// Merge two (max, sum-exp) pairs; l == 0 marks "empty".  Symmetric in its operands, so
// two lanes that exchange their pairs end with identical results.
__device__ __forceinline__ void merge_ml(double& m, double& l, double m2, double l2) {
  if (l2 == 0.0) return;
  if (l == 0.0) { m = m2; l = l2; return; }
  double M = fmax(m, m2);
  double a = l * double(expf(float(m - M)));
  double b = l2 * double(expf(float(m2 - M)));
  l = a + b;
  m = M;
}

// Transposing butterfly over a 16-lane group: on entry every lane holds 16 partial sums
// (one per value index), on exit lane i holds the group total of value index i.
__device__ __forceinline__ double butterfly16(double (&v)[16], int lane16) {
  {
    const bool up = lane16 & 8;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      double send = up ? v[i] : v[i + 8];
      double keep = up ? v[i + 8] : v[i];
      v[i] = keep + shfl_xor_double(send, 8);
    }
  }
  {
    const bool up = lane16 & 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      double send = up ? v[i] : v[i + 4];
      double keep = up ? v[i + 4] : v[i];
      v[i] = keep + shfl_xor_double(send, 4);
    }
  }
  {
    const bool up = lane16 & 2;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      double send = up ? v[i] : v[i + 2];
      double keep = up ? v[i + 2] : v[i];
      v[i] = keep + shfl_xor_double(send, 2);
    }
  }
  {
    const bool up = lane16 & 1;
    double send = up ? v[0] : v[1];
    double keep = up ? v[1] : v[0];
    v[0] = keep + shfl_xor_double(send, 1);
  }
  return v[0];
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kThreads, 2)
score_logits_kernel(const T* __restrict__ q_last, const T* __restrict__ K, int64_t L, double sm_scale,
                    double* __restrict__ logits, double* __restrict__ partials, int n_chunks) {
  using Cfg = ScoreCfg<G>;
  constexpr int EPL = D / 16;
  constexpr int R = Cfg::R, NB = Cfg::NB;
  const int u = blockIdx.y;
  const int chunk = blockIdx.x;
  const int tid = threadIdx.x;
  const int lane16 = tid & 15;
  const int grp = tid >> 4;

  // this lane's slice of the G scaled queries
  double qd[G][EPL];
  {
    const T* qu = q_last + (size_t(u) * G) * D + lane16 * EPL;
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int e = 0; e < EPL; ++e) qd[g][e] = elt_to_double(qu[size_t(g) * D + e]) * sm_scale;
  }

  const T* Ku = K + size_t(u) * L * D + lane16 * EPL;
  double* logits_u = logits + size_t(u) * G * L;
  const int64_t row0 = int64_t(chunk) * kScoreChunkRows;
  const int64_t row_end = min(row0 + int64_t(kScoreChunkRows), L);

  double run_m[NB], run_l[NB];
#pragma unroll
  for (int i = 0; i < NB; ++i) { run_m[i] = 0.0; run_l[i] = 0.0; }

  for (int64_t base = row0; base < row_end; base += kGroups * R) {
    RowSlice<T, EPL> raw[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      int64_t row = base + r * kGroups + grp;
      if (row < row_end) raw[r].load(Ku + size_t(row) * D);
      else raw[r].zero();
    }
    double acc[Cfg::NVP];
#pragma unroll
    for (int i = 0; i < Cfg::NVP; ++i) acc[i] = 0.0;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        double kd = raw[r].get(e);
#pragma unroll
        for (int g = 0; g < G; ++g) acc[r * G + g] = fma(qd[g][e], kd, acc[r * G + g]);
      }
#pragma unroll
    for (int bf = 0; bf < NB; ++bf) {
      double part[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) part[i] = acc[bf * 16 + i];
      double x = butterfly16(part, lane16);
      int v = bf * 16 + lane16;
      int r = v / G, g = v - r * G;
      int64_t row = base + r * kGroups + grp;
      if (v < Cfg::NV && row < row_end) {
        logits_u[size_t(g) * L + row] = x;
        if (run_l[bf] == 0.0) { run_m[bf] = x; run_l[bf] = 1.0; }
        else if (x > run_m[bf]) { run_l[bf] = run_l[bf] * double(expf(float(run_m[bf] - x))) + 1.0; run_m[bf] = x; }
        else run_l[bf] += double(expf(float(x - run_m[bf])));
      }
    }
  }

  // CTA reduction of the per-lane (max, sum-exp): lanes with equal (bf, lane16) share a head.
  __shared__ double sm_m[NB][kThreads], sm_l[NB][kThreads];
  __shared__ double cls_m[Cfg::NVP], cls_l[Cfg::NVP];
#pragma unroll
  for (int bf = 0; bf < NB; ++bf) { sm_m[bf][tid] = run_m[bf]; sm_l[bf][tid] = run_l[bf]; }
  __syncthreads();
  if (tid < Cfg::NVP) {
    int bf = tid >> 4, l16 = tid & 15;
    double m = 0.0, l = 0.0;
    for (int gi = 0; gi < kGroups; ++gi) merge_ml(m, l, sm_m[bf][gi * 16 + l16], sm_l[bf][gi * 16 + l16]);
    cls_m[tid] = m;
    cls_l[tid] = l;
  }
  __syncthreads();
  if (tid < G) {
    double m = 0.0, l = 0.0;
    for (int v = tid; v < Cfg::NV; v += G) merge_ml(m, l, cls_m[v], cls_l[v]);
    double* p = partials + ((size_t(u) * n_chunks + chunk) * G + tid) * 2;
    p[0] = m;
    p[1] = l;
  }
}

template <int G>
__global__ void __launch_bounds__(kThreads)
score_finalize_kernel(const double* __restrict__ logits, const double* __restrict__ partials, int n_chunks,
                      int64_t L, double* __restrict__ logscore, int rows_per_cta) {
  const int u = blockIdx.y;
  const int tid = threadIdx.x;
  __shared__ double lse[G];
  // log-sum-exp of every head of the group from the per-chunk partials (warp g does head g)
  {
    const int warp = tid >> 5, lane = tid & 31;
    if (warp < G) {
      double m = 0.0, l = 0.0;
      for (int c = lane; c < n_chunks; c += 32) {
        const double* p = partials + ((size_t(u) * n_chunks + c) * G + warp) * 2;
        merge_ml(m, l, p[0], p[1]);
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        double m2 = shfl_xor_double(m, off), l2 = shfl_xor_double(l, off);
        merge_ml(m, l, m2, l2);
      }
      if (lane == 0) lse[warp] = m + log(l);
    }
  }
  __syncthreads();
  const double log_g = log(double(G));
  const double* lu = logits + size_t(u) * G * L;
  const int64_t j0 = int64_t(blockIdx.x) * rows_per_cta;
  const int64_t j1 = min(j0 + int64_t(rows_per_cta), L);
  for (int64_t j = j0 + tid; j < j1; j += kThreads) {
    double y[G];
    double top = -1.0e308;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      y[g] = lu[size_t(g) * L + j] - lse[g];
      top = fmax(top, y[g]);
    }
    if (G == 1) {
      logscore[size_t(u) * L + j] = y[0];
    } else {
      float sum = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) sum += expf(float(y[g] - top));
      logscore[size_t(u) * L + j] = top + double(logf(sum)) - log_g;
    }
  }
}

template <typename T, int D, int G>
int launch_score(const tca_params* prm, const void* q_last, const void* K, int64_t L, double* logscore,
                 const ScoreWs& ws, cudaStream_t stream) {
  const int U = prm->batch * prm->n_kv_heads;
  dim3 grid1(unsigned(ws.n_chunks), unsigned(U));
  score_logits_kernel<T, D, G><<<grid1, kThreads, 0, stream>>>(
      static_cast<const T*>(q_last), static_cast<const T*>(K), L, double(prm->sm_scale), ws.logits,
      ws.partials, int(ws.n_chunks));
  int st = check_launch();
  if (st != TCA_OK) return st;
  const int rows_per_cta = 1024;
  dim3 grid2(unsigned((L + rows_per_cta - 1) / rows_per_cta), unsigned(U));
  score_finalize_kernel<G><<<grid2, kThreads, 0, stream>>>(ws.logits, ws.partials, int(ws.n_chunks), L,
                                                           logscore, rows_per_cta);
  return check_launch();
}

template <typename T, int D>
int dispatch_group(int G, const tca_params* prm, const void* q_last, const void* K, int64_t L,
                   double* logscore, const ScoreWs& ws, cudaStream_t stream) {
  switch (G) {
    case 1: return launch_score<T, D, 1>(prm, q_last, K, L, logscore, ws, stream);
    case 2: return launch_score<T, D, 2>(prm, q_last, K, L, logscore, ws, stream);
    case 3: return launch_score<T, D, 3>(prm, q_last, K, L, logscore, ws, stream);
    case 4: return launch_score<T, D, 4>(prm, q_last, K, L, logscore, ws, stream);
    case 5: return launch_score<T, D, 5>(prm, q_last, K, L, logscore, ws, stream);
    case 6: return launch_score<T, D, 6>(prm, q_last, K, L, logscore, ws, stream);
    case 7: return launch_score<T, D, 7>(prm, q_last, K, L, logscore, ws, stream);
    case 8: return launch_score<T, D, 8>(prm, q_last, K, L, logscore, ws, stream);
    default: return TCA_ERR_UNSUPPORTED;
  }
}

}  // namespace
}  // namespace tca

using namespace tca;

extern "C" int tca_score(const tca_params* prm, const void* q_last, const void* K, int64_t L,
                         double* logscore, void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  TCA_CHECK_ARG(q_last && K && logscore && ws);
  TCA_CHECK_ARG(L >= 1 && L < (int64_t(1) << 31));
  TCA_CHECK_ARG(aligned(q_last, 16) && aligned(K, 16) && aligned(logscore, 8) && aligned(ws, 256));
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  TCA_CHECK_ARG(U <= 65535);
  ScoreWs lay = score_ws_layout(prm, L, ws);
  if (ws_bytes < lay.bytes) return TCA_ERR_WORKSPACE;
  const int G = prm->n_q_heads / prm->n_kv_heads;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (prm->dtype == TCA_BF16) {
    if (prm->head_dim == 128) return dispatch_group<__nv_bfloat16, 128>(G, prm, q_last, K, L, logscore, lay, s);
    return dispatch_group<__nv_bfloat16, 64>(G, prm, q_last, K, L, logscore, lay, s);
  }
  if (prm->head_dim == 128) return dispatch_group<float, 128>(G, prm, q_last, K, L, logscore, lay, s);
  return dispatch_group<float, 64>(G, prm, q_last, K, L, logscore, lay, s);
}
