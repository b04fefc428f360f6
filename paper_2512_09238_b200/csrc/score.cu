// tca_score: token importance of Eq. 5 in the log domain.
//
// Pass 1 (score_logits_kernel) streams K once with 128-bit loads and accumulates the G dot
// products of a query group in fp64 (products of bf16 or fp32 inputs are exact in fp64, so
// the logits are exact up to summation rounding: log-scores reach +-50, where fp32 has a
// 4e-6 ulp against the 1e-5 selection rule).  Four lanes share four key rows (4 x 4 register
// blocking, queries from shared memory), see the kernel.  Each CTA also leaves a
// (max, sum-exp) partial per head.
// Pass 2 (score_finalize_kernel) merges the partials into each head's log-sum-exp and
// turns logits into  log( (1/G) * sum_g softmax_g[j] ).  When asked to (tca_score_select), its
// CTAs, which each hold 1024 consecutive log-scores = whole blocks of b tokens, also form the
// block metric h_j of Eq. 6 for those blocks, so that the selection does not read the scores
// back for it.
#include "common.cuh"
#include "select_common.cuh"

namespace tca {
namespace {

constexpr int kThreads = 256;

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

// 16-byte chunk -> doubles
__device__ __forceinline__ void chunk_to_double(const uint4& w, double (&x)[8], __nv_bfloat16) {
  // one shift or mask and one hardware conversion per element: the conversion unit runs beside the
  // fp64 pipe, whereas placing the bits by integer arithmetic costs more issue slots than the
  // multiply-adds that use the value
  x[0] = double(bf16_lo(w.x)); x[1] = double(bf16_hi(w.x));
  x[2] = double(bf16_lo(w.y)); x[3] = double(bf16_hi(w.y));
  x[4] = double(bf16_lo(w.z)); x[5] = double(bf16_hi(w.z));
  x[6] = double(bf16_lo(w.w)); x[7] = double(bf16_hi(w.w));
}
__device__ __forceinline__ void chunk_to_double(const uint4& w, double (&x)[8], float) {
  x[0] = double(__uint_as_float(w.x)); x[1] = double(__uint_as_float(w.y));
  x[2] = double(__uint_as_float(w.z)); x[3] = double(__uint_as_float(w.w));
}

constexpr int kLogitThreads = 128;

// Register blocking 4 rows x 4 lanes: a group of four lanes owns four consecutive key rows;
// lane j takes the 16-byte chunks 4i + j of each of them.  A query value fetched from shared
// memory is then used for four rows (the 128 B/clk return path of shared loads, not the
// fp64 pipe, limits a one-row-per-thread layout), the sixteen accumulators per lane are
// independent chains, and the only cross-lane work is a two-step transposing exchange
// after which lane j holds row j of the group for all G heads.
template <typename T, int D, int G>
__global__ void __launch_bounds__(kLogitThreads)
score_logits_kernel(const T* __restrict__ q_last, const T* __restrict__ K, int64_t L, double sm_scale,
                    double* __restrict__ logits, double* __restrict__ partials, int n_chunks, int rows_per_cta) {
  constexpr int EPC = 16 / int(sizeof(T));          // elements per 16-byte chunk
  constexpr int kChunks = D / EPC;                  // chunks per row
  constexpr int kIters = kChunks / 4;               // chunks per lane
  constexpr int QS = EPC + 2;                       // padded query chunk (doubles): 4 chunks -> 4 bank groups
  constexpr int kWarps = kLogitThreads / 32;
  const int u = blockIdx.y, chunk = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int grp = lane >> 2, j = lane & 3;
  // Launched with programmatic dependent launch: the next kernel of the stream may be scheduled
  // now (it waits for this grid itself), and this grid waits for its predecessor before it
  // touches anything the predecessor may still be writing.
  pdl_launch_dependents();
  pdl_wait();

  __shared__ __align__(16) double qs[G][kChunks][QS];
  __shared__ double red_m[kWarps][G], red_l[kWarps][G];
  for (int i = tid; i < G * D; i += kLogitThreads) {
    const int g = i / D, d = i % D;
    qs[g][d / EPC][d % EPC] = elt_to_double(q_last[(size_t(u) * G) * D + i]) * sm_scale;
  }
  __syncthreads();

  const T* Ku = K + size_t(u) * L * D;
  double* logits_u = logits + size_t(u) * G * L;
  const int64_t row0 = int64_t(chunk) * rows_per_cta;
  const int64_t row_end = min(row0 + int64_t(rows_per_cta), L);
  double run_m[G], run_l[G];
#pragma unroll
  for (int g = 0; g < G; ++g) { run_m[g] = 0.0; run_l[g] = 0.0; }

  // The 16-byte pieces of the next step are requested before the current ones are used, so a
  // warp always has 64 bytes per lane in flight while its fp64 work runs.
  auto fetch = [&](int64_t base, int i, uint4 (&dst)[4]) {
    const int64_t r = base + grp * 4;
#pragma unroll
    for (int rr = 0; rr < 4; ++rr) {
      dst[rr] = make_uint4(0, 0, 0, 0);
      if (r + rr < row_end) dst[rr] = __ldcs(reinterpret_cast<const uint4*>(Ku + size_t(r + rr) * D) + (4 * i + j));
    }
  };
  uint4 raw[4];
  fetch(row0 + warp * 32, 0, raw);
  for (int64_t base = row0 + warp * 32; base < row_end; base += kWarps * 32) {
    const int64_t r0 = base + grp * 4;              // the group's four rows
    double acc[4][G];
#pragma unroll
    for (int rr = 0; rr < 4; ++rr)
#pragma unroll
      for (int g = 0; g < G; ++g) acc[rr][g] = 0.0;
#pragma unroll
    for (int i = 0; i < kIters; ++i) {
      const int c = 4 * i + j;
      uint4 nxt[4];
      if (i + 1 < kIters) fetch(base, i + 1, nxt);
      else fetch(base + kWarps * 32, 0, nxt);
#pragma unroll
      for (int e = 0; e < EPC; e += 2) {
        double2 qq[G];
#pragma unroll
        for (int g = 0; g < G; ++g) qq[g] = *reinterpret_cast<const double2*>(&qs[g][c][e]);
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) {
          double x[8];
          chunk_to_double(raw[rr], x, T());
#pragma unroll
          for (int g = 0; g < G; ++g) {
            acc[rr][g] = fma(qq[g].x, x[e], acc[rr][g]);
            acc[rr][g] = fma(qq[g].y, x[e + 1], acc[rr][g]);
          }
        }
      }
#pragma unroll
      for (int rr = 0; rr < 4; ++rr) raw[rr] = nxt[rr];
    }
    // transposing exchange over the four lanes of the group: lane j ends with row j, all heads
    double half2[2][G];
    {
      const bool up = j & 2;
#pragma unroll
      for (int rr = 0; rr < 2; ++rr)
#pragma unroll
        for (int g = 0; g < G; ++g) {
          const double send = up ? acc[rr][g] : acc[rr + 2][g];
          const double keep = up ? acc[rr + 2][g] : acc[rr][g];
          half2[rr][g] = keep + shfl_xor_double(send, 2);
        }
    }
    double xg[G];
    {
      const bool up = j & 1;
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const double send = up ? half2[0][g] : half2[1][g];
        const double keep = up ? half2[1][g] : half2[0][g];
        xg[g] = keep + shfl_xor_double(send, 1);
      }
    }
    const int64_t row = r0 + j;                     // = base + lane: coalesced stores
    if (row < row_end) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const double x = xg[g];
        logits_u[size_t(g) * L + row] = x;
        if (run_l[g] == 0.0) { run_m[g] = x; run_l[g] = 1.0; }
        else if (x > run_m[g]) { run_l[g] = run_l[g] * double(expf(float(run_m[g] - x))) + 1.0; run_m[g] = x; }
        else run_l[g] += double(expf(float(x - run_m[g])));
      }
    }
  }

  // merge the per-lane (max, sum-exp): lanes by shuffle, warps through shared memory
#pragma unroll
  for (int g = 0; g < G; ++g) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const double m2 = shfl_xor_double(run_m[g], off), l2 = shfl_xor_double(run_l[g], off);
      merge_ml(run_m[g], run_l[g], m2, l2);
    }
    if (lane == 0) { red_m[warp][g] = run_m[g]; red_l[warp][g] = run_l[g]; }
  }
  __syncthreads();
  if (tid < G) {
    double m = 0.0, l = 0.0;
    for (int w = 0; w < kWarps; ++w) merge_ml(m, l, red_m[w][tid], red_l[w][tid]);
    double* p = partials + ((size_t(u) * n_chunks + chunk) * G + tid) * 2;
    p[0] = m;
    p[1] = l;
  }
}

constexpr int kFinalizeRows = 1024;   // log-scores per CTA of the second pass: a multiple of every block size b <= 128

template <int G>
__global__ void __launch_bounds__(kThreads)
score_finalize_kernel(const double* __restrict__ logits, const double* __restrict__ partials, int n_chunks,
                      int64_t L, double* __restrict__ logscore, MetricOut mo) {
  const int u = blockIdx.y;
  const int tid = threadIdx.x;
  pdl_launch_dependents();   // see score_logits_kernel
  pdl_wait();
  __shared__ double lse[G];
  __shared__ double ls_s[kFinalizeRows];   // this CTA's log-scores, for the fused block metric
  // This thread's logits are requested first: they do not depend on the log-sum-exp, and the
  // sixteen loads then overlap each other and the merge of the partials below.
  constexpr int kPer = kFinalizeRows / kThreads;
  const double* lu = logits + size_t(u) * G * L;
  const int64_t j0 = int64_t(blockIdx.x) * kFinalizeRows;
  const int64_t j1 = min(j0 + int64_t(kFinalizeRows), L);
  double y[kPer][G];
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int64_t j = j0 + tid + i * kThreads;
#pragma unroll
    for (int g = 0; g < G; ++g) y[i][g] = (j < j1) ? __ldcs(lu + size_t(g) * L + j) : 0.0;
  }
  // log-sum-exp of every head of the group from the per-CTA partials (warp g does head g)
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
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int64_t j = j0 + tid + i * kThreads;
    if (j >= j1) break;
    double top = -1.0e308;
#pragma unroll
    for (int g = 0; g < G; ++g) {
      y[i][g] -= lse[g];
      top = fmax(top, y[i][g]);
    }
    double out;
    if (G == 1) {
      out = y[i][0];
    } else {
      float sum = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) sum += expf(float(y[i][g] - top));
      out = top + double(logf(sum)) - log_g;
    }
    logscore[size_t(u) * L + j] = out;
    ls_s[j - j0] = out;
  }
  if (mo.hkey == nullptr) return;
  // Fused tail: h_j for the blocks that lie in [j0, j1); blocks j >= m belong to the always-kept
  // tail and have no metric.  Same arithmetic as block_metric_kernel on the same doubles.
  __syncthreads();
  const int warp = tid >> 5, lane = tid & 31;
  const int jb0 = int(j0 / mo.b);
  for (int i = warp; i < kFinalizeRows / mo.b; i += kThreads / 32) {
    const int jb = jb0 + i;
    if (jb >= mo.m) break;
    const double h = block_metric_warp(ls_s + i * mo.b, mo.b, mo.alpha, mo.mode, lane);
    if (lane == 0) {
      mo.hkey[size_t(u) * mo.m + jb] = ordered_key(h);
      if (mo.h_out) mo.h_out[size_t(u) * mo.m + jb] = h;
    }
  }
}

template <typename T, int D, int G>
int launch_score(const tca_params* prm, const void* q_last, const void* K, int64_t L, double* logscore,
                 const ScoreWs& ws, const MetricOut& mo, cudaStream_t stream) {
  const int U = prm->batch * prm->n_kv_heads;
  // One wave: as many CTAs as the GPU holds at once (four per SM at 128 registers), each with an
  // equal share of its unit's rows, so that all of them start together and finish together; never
  // more parts than the workspace has partials for (one per kScoreChunkRows rows).
  const int64_t per_unit = std::max<int64_t>(1, std::min<int64_t>(ws.n_chunks, int64_t(4) * sm_count() / U));
  const int64_t rows_per_cta = ((L + per_unit - 1) / per_unit + 31) / 32 * 32;
  const int64_t n_parts = (L + rows_per_cta - 1) / rows_per_cta;
  dim3 grid1(static_cast<unsigned>(n_parts), static_cast<unsigned>(U));
  int st = launch_pdl(score_logits_kernel<T, D, G>, grid1, dim3(kLogitThreads), size_t(0), stream,
                      static_cast<const T*>(q_last), static_cast<const T*>(K), L, double(prm->sm_scale), ws.logits,
                      ws.partials, int(n_parts), int(rows_per_cta));
  if (st != TCA_OK) return st;
  dim3 grid2(unsigned((L + kFinalizeRows - 1) / kFinalizeRows), unsigned(U));
  return launch_pdl(score_finalize_kernel<G>, grid2, dim3(kThreads), size_t(0), stream,
                    static_cast<const double*>(ws.logits), static_cast<const double*>(ws.partials), int(n_parts), L,
                    logscore, mo);
}

template <typename T, int D>
int dispatch_group(int G, const tca_params* prm, const void* q_last, const void* K, int64_t L,
                   double* logscore, const ScoreWs& ws, const MetricOut& mo, cudaStream_t stream) {
  switch (G) {
    case 1: return launch_score<T, D, 1>(prm, q_last, K, L, logscore, ws, mo, stream);
    case 2: return launch_score<T, D, 2>(prm, q_last, K, L, logscore, ws, mo, stream);
    case 3: return launch_score<T, D, 3>(prm, q_last, K, L, logscore, ws, mo, stream);
    case 4: return launch_score<T, D, 4>(prm, q_last, K, L, logscore, ws, mo, stream);
    case 5: return launch_score<T, D, 5>(prm, q_last, K, L, logscore, ws, mo, stream);
    case 6: return launch_score<T, D, 6>(prm, q_last, K, L, logscore, ws, mo, stream);
    case 7: return launch_score<T, D, 7>(prm, q_last, K, L, logscore, ws, mo, stream);
    case 8: return launch_score<T, D, 8>(prm, q_last, K, L, logscore, ws, mo, stream);
    default: return TCA_ERR_UNSUPPORTED;
  }
}

}  // namespace

// tca_score proper; `fused.hkey != nullptr` also leaves the block metric of Eq. 6 there.
int score_impl(const tca_params* prm, const void* q_last, const void* K, int64_t L, double* logscore, void* ws,
               size_t ws_bytes, const MetricOut& fused, cudaStream_t s) {
  TCA_CHECK_ARG(q_last && K && logscore && ws);
  TCA_CHECK_ARG(L >= 1 && L < (int64_t(1) << 31));
  TCA_CHECK_ARG(aligned(q_last, 16) && aligned(K, 16) && aligned(logscore, 8) && aligned(ws, 256));
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  TCA_CHECK_ARG(U <= 65535);
  ScoreWs lay = score_ws_layout(prm, L, ws);
  if (ws_bytes < lay.bytes) return TCA_ERR_WORKSPACE;
  if (fused.hkey && kFinalizeRows % fused.b != 0) return TCA_ERR_UNSUPPORTED;
  const int G = prm->n_q_heads / prm->n_kv_heads;
  if (prm->dtype == TCA_BF16) {
    if (prm->head_dim == 128) return dispatch_group<__nv_bfloat16, 128>(G, prm, q_last, K, L, logscore, lay, fused, s);
    return dispatch_group<__nv_bfloat16, 64>(G, prm, q_last, K, L, logscore, lay, fused, s);
  }
  if (prm->head_dim == 128) return dispatch_group<float, 128>(G, prm, q_last, K, L, logscore, lay, fused, s);
  return dispatch_group<float, 64>(G, prm, q_last, K, L, logscore, lay, fused, s);
}

}  // namespace tca

using namespace tca;

extern "C" int tca_score(const tca_params* prm, const void* q_last, const void* K, int64_t L,
                         double* logscore, void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  const MetricOut none{nullptr, nullptr, 0, 1, 0, 0.0};
  return score_impl(prm, q_last, K, L, logscore, ws, ws_bytes, none, static_cast<cudaStream_t>(stream));
}
