// tca_select: core-context selection of Eqs. 6-8 (Algorithm 2, lines 2-6).
//
//   block_metric_kernel  one warp per block: h_j of Eq. 6 from log s, in fp64 (or the entropy
//                        variant, or the hash key of the random-order variant).  Skipped when
//                        the score kernel's tail has already produced h (tca_score_select).
//   block_rank_kernel    rank of every block in ascending (h, index) order by counting
//                        (8 threads per block over shared-memory tiles of keys),
//                        then t_j = Psi[rank_j] of Eq. 7
//   block_topt_kernel    one warp per block: the t_j largest scores by an MSB-first radix
//                        select on order-preserving 64-bit keys, ties to the lower
//                        position; survivors are written in ascending position at
//                        offset sum_{i<j} t_i, so the output needs no sort and no atomics
//   flat_topb_kernel     the flat variant: one CTA per unit finds the n_sel-th largest score of
//                        all candidates with an 8-bit-per-pass radix select, then writes the
//                        survivors in ascending position with a running block scan
#include "common.cuh"
#include "select_common.cuh"

namespace tca {

int score_impl(const tca_params* prm, const void* q_last, const void* K, int64_t L, double* logscore, void* ws,
               size_t ws_bytes, const MetricOut& fused, cudaStream_t stream);

namespace {

constexpr int kWarpsPerCta = 8;
constexpr int kMaxSelectHeads = 64;

struct BudgetCounts {
  int32_t cum[kMaxSelectHeads][8];  // cumulative n_k per KV head
};

__global__ void __launch_bounds__(kWarpsPerCta * 32)
block_metric_kernel(const double* __restrict__ logscore, int64_t L, int m, int b, double alpha, int mode, int seed,
                    unsigned long long* __restrict__ hkey, double* __restrict__ h_out) {
  const int u = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j = blockIdx.x * kWarpsPerCta + warp;
  pdl_launch_dependents();   // programmatic dependent launch: see score_logits_kernel
  pdl_wait();
  if (j >= m) return;
  double h;
  if (mode == kMetricRandom) h = random_block_key(seed, u, j);
  else h = block_metric_warp(logscore + size_t(u) * L + size_t(j) * b, b, alpha, mode, lane);
  if (lane == 0) {
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
  pdl_launch_dependents();
  pdl_wait();
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
                  int32_t* __restrict__ idx, int* __restrict__ status) {
  const int u = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j0 = blockIdx.x * kWarpsPerCta;
  const int32_t* tu = t_ws + size_t(u) * m;
  pdl_launch_dependents();
  pdl_wait();

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
  if constexpr (kDebugBounds) {
    // the count must fit the block and the output window of the unit
    const int64_t n_sel = offsets[u + 1] - offsets[u];
    if (t < 0 || t > b || out < 0 || int64_t(out) + t > n_sel) {
      if (lane == 0) report_bounds_ws(status, kBoundsBlockCount, (static_cast<long long>(j) << 32) | unsigned(t));
      return;
    }
  }

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

// ------------------------------------------------------------------ flat top-B (variant)
constexpr int kFlatThreads = 1024;

// Exclusive prefix of `flag` over the CTA's threads (thread order) plus the CTA total.
__device__ __forceinline__ int cta_exclusive_count(bool flag, int* warp_tot, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned bal = __ballot_sync(0xffffffffu, flag);
  __syncthreads();                                   // warp_tot may still be read from the previous call
  if (lane == 0) warp_tot[warp] = __popc(bal);
  __syncthreads();
  int before = 0, tot = 0;
  for (int w = 0; w < kFlatThreads / 32; ++w) {
    const int c = warp_tot[w];
    if (w < warp) before += c;
    tot += c;
  }
  total = tot;
  return before + __popc(bal & ((1u << lane) - 1u));
}

__global__ void __launch_bounds__(kFlatThreads)
flat_topb_kernel(const double* __restrict__ logscore, int64_t L, int64_t n_cand,
                 const int64_t* __restrict__ offsets, int32_t* __restrict__ idx) {
  const int u = blockIdx.x, tid = threadIdx.x;
  const double* ls = logscore + size_t(u) * L;
  pdl_launch_dependents();
  pdl_wait();
  const int64_t n_keep = offsets[u + 1] - offsets[u];
  if (n_keep <= 0) return;
  __shared__ unsigned hist[256];
  __shared__ unsigned long long s_prefix;
  __shared__ long long s_need;
  __shared__ int warp_tot[kFlatThreads / 32];
  // ---- the n_keep-th largest key, 8 bits per pass from the top; `need` = how many keys equal to
  // the decided prefix (so far) still have to be taken
  if (tid == 0) { s_prefix = 0ull; s_need = n_keep; }
  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    if (tid < 256) hist[tid] = 0u;
    __syncthreads();
    const unsigned long long prefix = s_prefix;
    for (int64_t i = tid; i < n_cand; i += kFlatThreads) {
      const unsigned long long k = ordered_key(ls[i]);
      if (pass == 0 || (k >> (shift + 8)) == prefix) atomicAdd(&hist[unsigned(k >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      long long need = s_need;
      int bin = 255;
      for (; bin > 0; --bin) {
        if (static_cast<long long>(hist[bin]) >= need) break;
        need -= hist[bin];
      }
      s_prefix = (prefix << 8) | static_cast<unsigned long long>(bin);
      s_need = need;
    }
    __syncthreads();
  }
  const unsigned long long thr = s_prefix;   // keys above it are all kept; `need_eq` of its equals, lowest positions first
  const long long need_eq = s_need;
  // ---- survivors in ascending position
  int32_t* dst = idx + offsets[u];
  long long out = 0, eq_seen = 0;
  for (int64_t c0 = 0; c0 < n_cand; c0 += kFlatThreads) {
    const int64_t i = c0 + tid;
    const unsigned long long k = (i < n_cand) ? ordered_key(ls[i]) : 0ull;
    const bool gt = (i < n_cand) && k > thr;
    const bool eq = (i < n_cand) && k == thr;
    int eq_tot, keep_tot;
    const int eq_before = cta_exclusive_count(eq, warp_tot, eq_tot);
    const bool keep = gt || (eq && eq_seen + eq_before < need_eq);
    const int keep_before = cta_exclusive_count(keep, warp_tot, keep_tot);
    if (keep && out + keep_before < n_keep) dst[out + keep_before] = int32_t(i);
    out += keep_tot;
    eq_seen += eq_tot;
  }
}

int select_impl(const tca_params* prm, const double* logscore, int64_t L, const int32_t* n_k, int32_t nK,
                int32_t* idx, const int64_t* offsets_dev, double* h_out, int32_t* t_out, const SelectWs& lay,
                bool metric_done, cudaStream_t s) {
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
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
  if (m == 0) return TCA_OK;
  TCA_CHECK_ARG(idx != nullptr || !any);
  if (prm->flags & TCA_FLAG_FLAT_TOPB) {
    return launch_pdl(flat_topb_kernel, dim3(unsigned(U)), dim3(kFlatThreads), size_t(0), s, logscore, L,
                      m * prm->block, offsets_dev, idx);
  }
  int st;
  const unsigned gx = unsigned((m + kWarpsPerCta - 1) / kWarpsPerCta);
  if (!metric_done) {
    st = launch_pdl(block_metric_kernel, dim3(gx, unsigned(U)), dim3(kWarpsPerCta * 32), size_t(0), s, logscore, L,
                    int(m), prm->block, double(prm->alpha), metric_mode(prm), prm->seed, lay.hkey, h_out);
    if (st != TCA_OK) return st;
  }
  st = launch_pdl(block_rank_kernel, dim3(unsigned((m + kRankBlocks - 1) / kRankBlocks), unsigned(U)),
                  dim3(kRankThreads), size_t(0), s, static_cast<const unsigned long long*>(lay.hkey), int(m),
                  prm->n_kv_heads, nK, counts, lay.t, t_out);
  if (st != TCA_OK) return st;
  return launch_pdl(block_topt_kernel, dim3(gx, unsigned(U)), dim3(kWarpsPerCta * 32), size_t(0), s, logscore, L,
                    int(m), prm->block, static_cast<const int32_t*>(lay.t), offsets_dev, idx, lay.status);
}

int check_select_args(const tca_params* prm, const double* logscore, int64_t L, const int32_t* n_k, int32_t nK,
                      const int64_t* offsets_dev, const void* ws) {
  TCA_CHECK_ARG(logscore && n_k && offsets_dev && ws);
  TCA_CHECK_ARG(L >= 1 && L < (int64_t(1) << 31));
  TCA_CHECK_ARG(nK == num_counts(prm));
  TCA_CHECK_ARG(aligned(logscore, 8) && aligned(offsets_dev, 8) && aligned(ws, 256));
  if (prm->n_kv_heads > kMaxSelectHeads) return TCA_ERR_UNSUPPORTED;
  TCA_CHECK_ARG(int64_t(prm->batch) * prm->n_kv_heads <= 65535);
  return TCA_OK;
}

}  // namespace
}  // namespace tca

using namespace tca;

extern "C" int tca_select(const tca_params* prm, const double* logscore, int64_t L, const int32_t* n_k,
                          int32_t nK, int32_t* idx, const int64_t* offsets_dev, double* h_out,
                          int32_t* t_out, void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  st = check_select_args(prm, logscore, L, n_k, nK, offsets_dev, ws);
  if (st != TCA_OK) return st;
  SelectWs lay = select_ws_layout(prm, L, ws);
  if (ws_bytes < lay.bytes) return TCA_ERR_WORKSPACE;
  return select_impl(prm, logscore, L, n_k, nK, idx, offsets_dev, h_out, t_out, lay, false,
                     static_cast<cudaStream_t>(stream));
}

extern "C" int tca_score_select(const tca_params* prm, const void* q_last, const void* K, int64_t L,
                                const int32_t* n_k, int32_t nK, double* logscore, int32_t* idx,
                                const int64_t* offsets_dev, double* h_out, int32_t* t_out, void* ws,
                                size_t ws_bytes, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  st = check_select_args(prm, logscore, L, n_k, nK, offsets_dev, ws);
  if (st != TCA_OK) return st;
  const size_t score_bytes = align_up(score_ws_layout(prm, L, nullptr).bytes, 256);
  SelectWs lay = select_ws_layout(prm, L, static_cast<char*>(ws) + score_bytes);
  if (ws_bytes < score_bytes + lay.bytes) return TCA_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t m = num_blocks(prm, L);
  // The score kernel's tail can form h only for the variants that derive it from the scores, and
  // only when a block never straddles two of its CTAs (b divides its 1024-token span: always).
  const int mode = metric_mode(prm);
  const bool fuse = m > 0 && mode != kMetricRandom && !(prm->flags & TCA_FLAG_FLAT_TOPB);
  MetricOut fused{fuse ? lay.hkey : nullptr, h_out, int(m), prm->block, mode, double(prm->alpha)};
  st = score_impl(prm, q_last, K, L, logscore, ws, score_bytes, fused, s);
  if (st != TCA_OK) return st;
  return select_impl(prm, logscore, L, n_k, nK, idx, offsets_dev, h_out, t_out, lay, fuse, s);
}
