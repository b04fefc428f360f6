// tca_attn_prefill / tca_attn_prefill_rows: entry points of the sparse causal prefill attention (Eq. 2).
// fp32 inputs run on the FP32 pipes; bf16 inputs run on the tcgen05 tensor-core kernel
// unless TCA_FLAG_PREFILL_SIMT asks for the FP32-pipe reference kernel.
#include "common.cuh"

namespace tca {
template <typename T, int D>
int launch_prefill_simt(const tca_params*, const void*, const void*, const void*, int64_t, int64_t, int64_t,
                        const tca_cache_desc*, void*, cudaStream_t);
template <int D>
int launch_prefill_tc(const tca_params*, const void*, const void*, const void*, int64_t, int64_t, int64_t,
                      const tca_cache_desc*, void*, void*, cudaStream_t);
template <int D>
int launch_prefill_tc_gather(const tca_params*, const void*, const void*, const void*, int64_t, int64_t, int64_t,
                             const int32_t*, const int64_t*, void*, void*, cudaStream_t);
}  // namespace tca

using namespace tca;

extern "C" int tca_attn_prefill_rows(const tca_params* prm, const void* Q, const void* K, const void* V, int64_t L,
                                     int64_t row_begin, int64_t row_end, const tca_cache_desc* c, void* O,
                                     void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  if (prm->window < 1) return TCA_ERR_UNSUPPORTED;  // a query always sees itself through its local subset
  TCA_CHECK_ARG(Q && K && V && c && O && ws);
  TCA_CHECK_ARG(c->k && c->v && c->pos && c->state);
  TCA_CHECK_ARG(L >= 1 && L < (int64_t(1) << 31));
  TCA_CHECK_ARG(row_begin >= 0 && row_begin < row_end && row_end <= L && row_begin % TCA_PREFILL_ROW_ALIGN == 0);
  TCA_CHECK_ARG(aligned(Q, 16) && aligned(K, 16) && aligned(V, 16) && aligned(O, 16) && aligned(ws, 256));
  TCA_CHECK_ARG(aligned(c->k, 16) && aligned(c->v, 16));
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  TCA_CHECK_ARG(c->n_units == U);
  TCA_CHECK_ARG(int64_t(prm->batch) * prm->n_q_heads <= 65535);
  if (ws_bytes < tca_workspace_bytes(prm, L, TCA_OP_PREFILL)) return TCA_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);   // word 0 of ws is the sticky status word: not cleared here
  if (prm->dtype == TCA_F32) {
    if (prm->head_dim == 128) return launch_prefill_simt<float, 128>(prm, Q, K, V, L, row_begin, row_end, c, O, s);
    return launch_prefill_simt<float, 64>(prm, Q, K, V, L, row_begin, row_end, c, O, s);
  }
  if (prm->flags & TCA_FLAG_PREFILL_SIMT) {
    if (prm->head_dim == 128) return launch_prefill_simt<__nv_bfloat16, 128>(prm, Q, K, V, L, row_begin, row_end, c, O, s);
    return launch_prefill_simt<__nv_bfloat16, 64>(prm, Q, K, V, L, row_begin, row_end, c, O, s);
  }
  TCA_CHECK_ARG(c->seg_start && c->n_global);
  if (prm->head_dim == 128) return launch_prefill_tc<128>(prm, Q, K, V, L, row_begin, row_end, c, O, ws, s);
  return launch_prefill_tc<64>(prm, Q, K, V, L, row_begin, row_end, c, O, ws, s);
}

extern "C" int tca_attn_prefill(const tca_params* prm, const void* Q, const void* K, const void* V, int64_t L,
                                const tca_cache_desc* c, void* O, void* ws, size_t ws_bytes, void* stream) {
  return tca_attn_prefill_rows(prm, Q, K, V, L, 0, L, c, O, ws, ws_bytes, stream);
}

// The prefill-only form: no cache, no compaction; the producer of the tensor-core kernel fetches
// the selected rows from K and V by index (Appendix C, "Memory Access Optimization").
extern "C" int tca_attn_prefill_gather(const tca_params* prm, const void* Q, const void* K, const void* V, int64_t L,
                                       int64_t row_begin, int64_t row_end, const int32_t* idx,
                                       const int64_t* offsets_dev, void* O, void* ws, size_t ws_bytes,
                                       void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  if (prm->window < 1) return TCA_ERR_UNSUPPORTED;
  if (prm->dtype != TCA_BF16 || (prm->flags & TCA_FLAG_PREFILL_SIMT)) return TCA_ERR_UNSUPPORTED;   // tensor-core kernel only
  TCA_CHECK_ARG(Q && K && V && idx && offsets_dev && O && ws);
  TCA_CHECK_ARG(L >= 1 && L < (int64_t(1) << 31));
  TCA_CHECK_ARG(row_begin >= 0 && row_begin < row_end && row_end <= L && row_begin % TCA_PREFILL_ROW_ALIGN == 0);
  TCA_CHECK_ARG(aligned(Q, 16) && aligned(K, 16) && aligned(V, 16) && aligned(O, 16) && aligned(ws, 256));
  TCA_CHECK_ARG(aligned(idx, 4) && aligned(offsets_dev, 8));
  TCA_CHECK_ARG(int64_t(prm->batch) * prm->n_q_heads <= 65535);
  if (ws_bytes < tca_workspace_bytes(prm, L, TCA_OP_PREFILL)) return TCA_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (prm->head_dim == 128)
    return launch_prefill_tc_gather<128>(prm, Q, K, V, L, row_begin, row_end, idx, offsets_dev, O, ws, s);
  return launch_prefill_tc_gather<64>(prm, Q, K, V, L, row_begin, row_end, idx, offsets_dev, O, ws, s);
}
