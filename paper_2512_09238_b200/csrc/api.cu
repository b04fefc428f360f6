// Host-side pieces of the C ABI: validation, budget resolution (Eq. 7), workspace
// layouts, cache descriptor upload.
#include <cmath>
#include <cstring>
#include <mutex>
#include <vector>

#include "common.cuh"

namespace tca {

size_t prefill_tc_ws_bytes(const tca_params* prm);
size_t calib_ws_bytes(const tca_params* prm, int64_t L);

int check_params(const tca_params* prm) {
  TCA_CHECK_ARG(prm != nullptr);
  TCA_CHECK_ARG(prm->batch >= 1 && prm->n_kv_heads >= 1 && prm->n_q_heads >= 1);
  TCA_CHECK_ARG(prm->n_q_heads % prm->n_kv_heads == 0);
  TCA_CHECK_ARG(prm->window >= 0);
  TCA_CHECK_ARG(prm->alpha >= 0.f && prm->alpha <= 1.f);
  TCA_CHECK_ARG(prm->sm_scale > 0.f && std::isfinite(prm->sm_scale));
  constexpr int kKnownFlags = TCA_FLAG_PREFILL_SIMT | TCA_FLAG_ENTROPY_INDEX | TCA_FLAG_RANDOM_ORDER |
                              TCA_FLAG_FLAT_TOPB | TCA_FLAG_PREFILL_BAND_FIRST;
  TCA_CHECK_ARG((prm->flags & ~kKnownFlags) == 0);
  {   // at most one selection variant
    const int v = prm->flags & (TCA_FLAG_ENTROPY_INDEX | TCA_FLAG_RANDOM_ORDER | TCA_FLAG_FLAT_TOPB);
    TCA_CHECK_ARG((v & (v - 1)) == 0);
  }
  if (prm->dtype != TCA_F32 && prm->dtype != TCA_BF16) return TCA_ERR_UNSUPPORTED;
  if (prm->head_dim != 64 && prm->head_dim != 128) return TCA_ERR_UNSUPPORTED;
  if (!is_pow2(prm->block) || prm->block > kMaxBlock) return TCA_ERR_UNSUPPORTED;
  if (prm->n_q_heads / prm->n_kv_heads > kMaxGroup) return TCA_ERR_UNSUPPORTED;
  return TCA_OK;
}

namespace {
std::mutex g_device_mutex;
int g_sm_count[kMaxDevices] = {};
int64_t g_l2_bytes[kMaxDevices] = {};
}  // namespace

int sm_count() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  std::lock_guard<std::mutex> lock(g_device_mutex);
  if (g_sm_count[dev] == 0) {
    int n = 0;
    g_sm_count[dev] =
        (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) ? n : 148;
  }
  return g_sm_count[dev];
}

int64_t l2_bytes() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
  std::lock_guard<std::mutex> lock(g_device_mutex);
  if (g_l2_bytes[dev] == 0) {
    int n = 0;
    g_l2_bytes[dev] = (cudaDeviceGetAttribute(&n, cudaDevAttrL2CacheSize, dev) == cudaSuccess && n > 0) ? n : -1;
  }
  return g_l2_bytes[dev] > 0 ? g_l2_bytes[dev] : 0;
}

ScoreWs score_ws_layout(const tca_params* prm, int64_t L, void* ws) {
  ScoreWs w;
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  const int G = prm->n_q_heads / prm->n_kv_heads;
  w.n_chunks = (L + kScoreChunkRows - 1) / kScoreChunkRows;
  size_t logits_bytes = align_up(size_t(U) * G * L * sizeof(double), 256);
  size_t partial_bytes = align_up(size_t(U) * w.n_chunks * G * 2 * sizeof(double), 256);
  w.logits = reinterpret_cast<double*>(ws);
  w.partials = reinterpret_cast<double*>(reinterpret_cast<char*>(ws) + logits_bytes);
  w.bytes = logits_bytes + partial_bytes;
  return w;
}

SelectWs select_ws_layout(const tca_params* prm, int64_t L, void* ws) {
  SelectWs w;
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  const int64_t m = num_blocks(prm, L);
  size_t hkey_bytes = align_up(size_t(U) * (m > 0 ? m : 1) * sizeof(unsigned long long), 256);
  size_t t_bytes = align_up(size_t(U) * (m > 0 ? m : 1) * sizeof(int32_t), 256);
  char* base = reinterpret_cast<char*>(ws);
  w.status = reinterpret_cast<int*>(base);
  w.hkey = reinterpret_cast<unsigned long long*>(base + 256);
  w.t = reinterpret_cast<int32_t*>(base + 256 + hkey_bytes);
  w.bytes = 256 + hkey_bytes + t_bytes;
  return w;
}

DecodeWs decode_ws_layout(const tca_params* prm, int64_t rows_total, int64_t n_units, void* ws) {
  DecodeWs w;
  const int G = prm->n_q_heads / prm->n_kv_heads;
  // slices are at least kDecodeChunkRows long, plus one short slice per unit
  w.n_chunks_max = rows_total / kDecodeChunkRows + 2 * n_units + 1;
  w.status = reinterpret_cast<int*>(ws);
  w.partial = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + kDecodeHeaderBytes);
  w.bytes = kDecodeHeaderBytes + align_up(size_t(w.n_chunks_max) * G * (prm->head_dim + 2) * sizeof(float), 256);
  return w;
}

}  // namespace tca

using namespace tca;

extern "C" {

const char* tca_strerror(int status) {
  switch (status) {
    case TCA_OK: return "ok";
    case TCA_ERR_INVALID_ARG: return "invalid argument";
    case TCA_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case TCA_ERR_WORKSPACE: return "workspace too small";
    case TCA_ERR_CUDA: return "CUDA runtime error";
    case TCA_ERR_TIMEOUT: return "device-side wait timed out";
    case TCA_ERR_CAPACITY: return "cache capacity exceeded";
    case TCA_ERR_SCRATCH_LIMIT: return "problem exceeds the built-in scratch of the static entry point";
    case TCA_ERR_BOUNDS: return "index or offset out of range (range-checked build)";
    default: return "unknown status";
  }
}

int tca_version(void) { return 200; }

int tca_build_info(void) { return kDebugBounds ? TCA_BUILD_DEBUG_BOUNDS : 0; }

int tca_cache_status(const tca_cache_desc* c, void* stream, int64_t* detail) {
  TCA_CHECK_ARG(c && c->state && c->n_units >= 1);
  std::vector<int64_t> st(size_t(c->n_units) * TCA_STATE_WORDS);
  TCA_CHECK_CUDA(cudaMemcpyAsync(st.data(), c->state, st.size() * sizeof(int64_t), cudaMemcpyDeviceToHost,
                                 static_cast<cudaStream_t>(stream)));
  TCA_CHECK_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  for (int64_t u = 0; u < c->n_units; ++u) {
    const int64_t word = st[size_t(u) * TCA_STATE_WORDS + TCA_ST_RESERVED];
    if (word != 0) {
      if (detail) { detail[0] = u; detail[1] = int64_t(uint64_t(word) >> 56); detail[2] = word & 0x00FFFFFFFFFFFFFFll; }
      return TCA_ERR_BOUNDS;
    }
  }
  return TCA_OK;
}

int tca_budget_resolve(const double* p, int32_t n_kv_heads, int32_t nK, int64_t m,
                       int32_t* n_k, int64_t* n_sel, int32_t* tbar) {
  TCA_CHECK_ARG(p && n_k && n_sel && tbar);
  TCA_CHECK_ARG(n_kv_heads >= 1 && nK >= 1 && nK <= 8 && m >= 0 && m < (int64_t(1) << 30));
  for (int h = 0; h < n_kv_heads; ++h) {
    const double* ph = p + size_t(h) * nK;
    double sum = 0.0;
    for (int k = 0; k < nK; ++k) {
      TCA_CHECK_ARG(ph[k] >= 0.0 && std::isfinite(ph[k]));
      sum += ph[k];
    }
    TCA_CHECK_ARG(std::fabs(sum - 1.0) <= 1e-9);
  }
  for (int h = 0; h < n_kv_heads; ++h) {
    const double* ph = p + size_t(h) * nK;
    int32_t* nh = n_k + size_t(h) * nK;
    double frac[8];
    int64_t assigned = 0;
    double mean_keep = 0.0;
    for (int k = 0; k < nK; ++k) {
      double f = double(m) * ph[k];
      double fl = std::floor(f);
      nh[k] = int32_t(fl);
      frac[k] = f - fl;
      assigned += nh[k];
      mean_keep += double(int64_t(1) << k) * ph[k];
    }
    // hand the shortfall to the largest fractional parts, ties to the larger k
    for (int64_t left = m - assigned; left > 0; --left) {
      int best = -1;
      for (int k = nK - 1; k >= 0; --k)
        if (frac[k] >= 0.0 && (best < 0 || frac[k] > frac[best])) best = k;
      if (best < 0) return TCA_ERR_INVALID_ARG;
      nh[best] += 1;
      frac[best] = -1.0;
    }
    int64_t total = 0;
    for (int k = 0; k < nK; ++k) total += (int64_t(1) << k) * nh[k];
    n_sel[h] = total;
    tbar[h] = int32_t(std::floor(mean_keep));
  }
  return TCA_OK;
}

size_t tca_workspace_bytes(const tca_params* prm, int64_t L, int op) {
  if (check_params(prm) != TCA_OK || L < 1) return 0;
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  switch (op) {
    case TCA_OP_SCORE: return score_ws_layout(prm, L, nullptr).bytes;
    case TCA_OP_SELECT: return select_ws_layout(prm, L, nullptr).bytes;
    case TCA_OP_COMPACT: return 256;
    case TCA_OP_PREFILL: return align_up(prefill_tc_ws_bytes(prm), 256);
    case TCA_OP_DECODE: return decode_ws_layout(prm, L, U, nullptr).bytes;
    case TCA_OP_APPEND: return 256;
    case TCA_OP_CALIB: return prm->dtype == TCA_BF16 ? calib_ws_bytes(prm, L) : 0;
    case TCA_OP_SCORE_SELECT:
      return align_up(score_ws_layout(prm, L, nullptr).bytes, 256) + select_ws_layout(prm, L, nullptr).bytes;
    default: return 0;
  }
}

int tca_cache_init(const tca_params* prm, tca_cache_desc* c, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  TCA_CHECK_ARG(c && c->k && c->v && c->pos && c->state);
  TCA_CHECK_ARG(c->seg_start && c->global_cap && c->n_global && c->tail_head && c->n_tail &&
                c->seq_len && c->t_keep);
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  TCA_CHECK_ARG(c->n_units == U && c->tail_cap >= 1 && c->rows_total >= 1);
  TCA_CHECK_ARG(c->rows_total < (int64_t(1) << 31));
  TCA_CHECK_ARG(aligned(c->k, 16) && aligned(c->v, 16) && aligned(c->state, 8));
  for (int64_t u = 0; u < U; ++u) {
    TCA_CHECK_ARG(c->seg_start[u] >= 0 && c->global_cap[u] >= 0);
    TCA_CHECK_ARG(c->seg_start[u] + c->global_cap[u] + c->tail_cap <= c->rows_total);
    if (u > 0)
      TCA_CHECK_ARG(c->seg_start[u] >= c->seg_start[u - 1] + c->global_cap[u - 1] + c->tail_cap);
    TCA_CHECK_ARG(c->n_global[u] >= 0 && c->n_global[u] <= c->global_cap[u]);
    TCA_CHECK_ARG(c->n_tail[u] >= 0 && c->n_tail[u] <= c->tail_cap);
    TCA_CHECK_ARG(c->tail_head[u] >= 0 && c->tail_head[u] < c->tail_cap);
    TCA_CHECK_ARG(c->t_keep[u] >= 0 && c->t_keep[u] <= prm->block);
  }
  std::vector<int64_t> st_host(size_t(U) * TCA_STATE_WORDS, 0);
  for (int64_t u = 0; u < U; ++u) {
    int64_t* s = &st_host[size_t(u) * TCA_STATE_WORDS];
    s[TCA_ST_SEG_START] = c->seg_start[u];
    s[TCA_ST_GLOBAL_CAP] = c->global_cap[u];
    s[TCA_ST_N_GLOBAL] = c->n_global[u];
    s[TCA_ST_TAIL_HEAD] = c->tail_head[u];
    s[TCA_ST_N_TAIL] = c->n_tail[u];
    s[TCA_ST_SEQ_LEN] = c->seq_len[u];
    s[TCA_ST_T_KEEP] = c->t_keep[u];
  }
  // Unused rows must hold finite values: the tensor-pipe kernels multiply masked-out rows by
  // an exact zero weight, which only cancels finite numbers.
  const size_t cache_bytes = size_t(c->rows_total) * prm->head_dim * elt_size(prm->dtype);
  TCA_CHECK_CUDA(cudaMemsetAsync(c->k, 0, cache_bytes, static_cast<cudaStream_t>(stream)));
  TCA_CHECK_CUDA(cudaMemsetAsync(c->v, 0, cache_bytes, static_cast<cudaStream_t>(stream)));
  // pageable source: the runtime stages the bytes before returning, so the vector may die
  TCA_CHECK_CUDA(cudaMemcpyAsync(c->state, st_host.data(), st_host.size() * sizeof(int64_t),
                                 cudaMemcpyHostToDevice, static_cast<cudaStream_t>(stream)));
  return TCA_OK;
}

int tca_ws_status(const void* ws, void* stream) {
  TCA_CHECK_ARG(ws != nullptr);
  int32_t word = 0;
  TCA_CHECK_CUDA(cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost,
                                 static_cast<cudaStream_t>(stream)));
  TCA_CHECK_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  return word == 0 ? TCA_OK : (word == kStatusBounds ? TCA_ERR_BOUNDS : TCA_ERR_TIMEOUT);
}

}  // extern "C"
