// tca_select: core-context selection of Eqs. 6-8 (Algorithm 2, lines 2-6).
//
//   block_metric_kernel  one warp per block: h_j of Eq. 6 from log s, in fp64
//   block_rank_kernel    rank of every block in ascending (h, index) order by counting
//                        (8 threads per block over shared-memory tiles of keys),
//                        then t_j = Psi[rank_j] of Eq. 7
//   block_topt_kernel    one warp per block: the t_j largest scores by an MSB-first radix
//                        select on order-preserving 64-bit keys, ties to the lower
//                        position; survivors are written in ascending position at
//                        offset sum_{i<j} t_i, so the output needs no sort and no atomics
#include "common.cuh"

namespace tca {
namespace {

constexpr int kWarpsPerCta = 8;
constexpr int kMaxSelectHeads = 64;

struct BudgetCounts {
  int32_t cum[kMaxSelectHeads][8];  // cumulative n_k per KV head
};

__global__ void __launch_bounds__(kWarpsPerCta * 32)
block_metric_kernel(const double* __restrict__ logscore, int64_t L, int m, int b, double alpha,
                    unsigned long long* __restrict__ hkey, double* __restrict__ h_out) {
  const int u = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.x * kWarpsPerCta + warp;
  if (j >= m) return;
  const double* ls = logscore + size_t(u) * L + size_t(j) * b;
  double v[4];
  double top = -1.0e308;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    int i = s * 32 + lane;
    v[s] = (i < b) ? ls[i] : -1.0e308;
    top = fmax(top, v[s]);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) top = fmax(top, shfl_xor_double(top, off));
  double se = 0.0, se2 = 0.0;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    int i = s * 32 + lane;
    if (i < b) {
      double e = double(expf(float(v[s] - top)));
      se += e;
      se2 += e * e;
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    se += shfl_xor_double(se, off);
    se2 += shfl_xor_double(se2, off);
  }
  if (lane == 0) {
    double mass = exp(top) * se;
    double h = (1.0 - alpha) * mass + alpha * (1.0 - se2 / (se * se));
    hkey[size_t(u) * m + j] = ordered_key(h);
    if (h_out) h_out[size_t(u) * m + j] = h;
  }
}

constexpr int kRankThreads = 256, kRankParts = 8, kRankBlocks = kRankThreads / kRankParts;

// 32 blocks per CTA, 8 threads per block: thread (j, part) counts the keys i = part (mod 8)
// that sort before block j; the 8 counts are added with shuffles.
__global__ void __launch_bounds__(kRankThreads)
block_rank_kernel(const unsigned long long* __restrict__ hkey, int m, int n_kv_heads, int nK,
                  BudgetCounts counts, int32_t* __restrict__ t_ws, int32_t* __restrict__ t_out) {
  constexpr int kTile = 2048;
  __shared__ unsigned long long tile[kTile];
  const int u = blockIdx.y;
  const int part = threadIdx.x & (kRankParts - 1);
  const int j = blockIdx.x * kRankBlocks + (threadIdx.x >> 3);
  const unsigned long long* hk = hkey + size_t(u) * m;
  const unsigned long long mine = (j < m) ? hk[j] : 0ull;
  int rank = 0;
  for (int i0 = 0; i0 < m; i0 += kTile) {
    const int n = min(kTile, m - i0);
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += kRankThreads) tile[i] = hk[i0 + i];
    __syncthreads();
#pragma unroll 4
    for (int i = part; i < n; i += kRankParts) {
      const unsigned long long other = tile[i];
      rank += (other < mine) || (other == mine && (i0 + i) < j);
    }
  }
  rank += __shfl_xor_sync(0xffffffffu, rank, 1);
  rank += __shfl_xor_sync(0xffffffffu, rank, 2);
  rank += __shfl_xor_sync(0xffffffffu, rank, 4);
  if (j >= m || part != 0) return;
  const int h = u % n_kv_heads;
  int t = 1 << (nK - 1);
  for (int k = nK - 1; k >= 0; --k)
    if (rank < counts.cum[h][k]) t = 1 << k;
  t_ws[size_t(u) * m + j] = t;
  if (t_out) t_out[size_t(u) * m + j] = t;
}

__global__ void __launch_bounds__(kWarpsPerCta * 32)
block_topt_kernel(const double* __restrict__ logscore, int64_t L, int m, int b,
                  const int32_t* __restrict__ t_ws, const int64_t* __restrict__ offsets,
                  int32_t* __restrict__ idx) {
  const int u = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j0 = blockIdx.x * kWarpsPerCta;
  const int32_t* tu = t_ws + size_t(u) * m;

  // tokens kept by the blocks before this CTA's first block
  __shared__ int warp_sum[kWarpsPerCta];
  int part = 0;
  for (int i = threadIdx.x; i < j0; i += kWarpsPerCta * 32) part += tu[i];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
  if (lane == 0) warp_sum[warp] = part;
  __syncthreads();
  int out = 0;
#pragma unroll
  for (int i = 0; i < kWarpsPerCta; ++i) out += warp_sum[i];

  const int j = j0 + warp;
  if (j >= m) return;
  for (int i = j0; i < j; ++i) out += tu[i];
  const int t = tu[j];

  const double* ls = logscore + size_t(u) * L + size_t(j) * b;
  unsigned long long key[4];
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    int i = s * 32 + lane;
    key[s] = (i < b) ? ordered_key(ls[i]) : 0ull;
  }
  const unsigned keep = radix_select_top_t(key, b, t, lane);
  int32_t* dst = idx + offsets[u] + out;
  int before = 0;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const bool k = (keep >> s) & 1u;
    const unsigned bal = __ballot_sync(0xffffffffu, k);
    if (k) dst[before + __popc(bal & ((1u << lane) - 1u))] = j * b + s * 32 + lane;
    before += __popc(bal);
  }
}

}  // namespace
}  // namespace tca

using namespace tca;

extern "C" int tca_select(const tca_params* prm, const double* logscore, int64_t L, const int32_t* n_k,
                          int32_t nK, int32_t* idx, const int64_t* offsets_dev, double* h_out,
                          int32_t* t_out, void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  TCA_CHECK_ARG(logscore && n_k && offsets_dev && ws);
  TCA_CHECK_ARG(L >= 1 && L < (int64_t(1) << 31));
  TCA_CHECK_ARG(nK == num_counts(prm));
  TCA_CHECK_ARG(aligned(logscore, 8) && aligned(offsets_dev, 8) && aligned(ws, 256));
  if (prm->n_kv_heads > kMaxSelectHeads) return TCA_ERR_UNSUPPORTED;
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  TCA_CHECK_ARG(U <= 65535);
  const int64_t m = num_blocks(prm, L);
  BudgetCounts counts;
  bool any = false;
  for (int h = 0; h < prm->n_kv_heads; ++h) {
    int64_t run = 0;
    for (int k = 0; k < 8; ++k) {
      if (k < nK) {
        TCA_CHECK_ARG(n_k[h * nK + k] >= 0);
        run += n_k[h * nK + k];
        any |= n_k[h * nK + k] > 0;
      }
      counts.cum[h][k] = int32_t(run);
    }
    TCA_CHECK_ARG(run == m);  // Psi has exactly one entry per block
  }
  SelectWs lay = select_ws_layout(prm, L, ws);
  if (ws_bytes < lay.bytes) return TCA_ERR_WORKSPACE;
  if (m == 0) return TCA_OK;
  TCA_CHECK_ARG(idx != nullptr || !any);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const unsigned gx = unsigned((m + kWarpsPerCta - 1) / kWarpsPerCta);
  block_metric_kernel<<<dim3(gx, unsigned(U)), kWarpsPerCta * 32, 0, s>>>(
      logscore, L, int(m), prm->block, double(prm->alpha), lay.hkey, h_out);
  st = check_launch();
  if (st != TCA_OK) return st;
  block_rank_kernel<<<dim3(unsigned((m + kRankBlocks - 1) / kRankBlocks), unsigned(U)), kRankThreads, 0, s>>>(
      lay.hkey, int(m), prm->n_kv_heads, nK, counts, lay.t, t_out);
  st = check_launch();
  if (st != TCA_OK) return st;
  block_topt_kernel<<<dim3(gx, unsigned(U)), kWarpsPerCta * 32, 0, s>>>(logscore, L, int(m), prm->block,
                                                                         lay.t, offsets_dev, idx);
  return check_launch();
}
