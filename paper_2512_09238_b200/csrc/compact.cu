// tca_compact_kv: gather the retained keys and values [K^G; K^L] of Eq. 2 into the
// per-unit segments of the flattened cache (Appendix C, "parallel tokens gathering" and
// "multi-head parallelization").  Every row is d*elt = 128..512 bytes, moved as 16-byte
// pieces with four independent loads in flight per thread; a row's pieces sit in
// adjacent lanes so both sides of the copy are fully coalesced per row.
#include "common.cuh"

namespace tca {
namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerCta = 256;

__global__ void __launch_bounds__(kThreads)
compact_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, int64_t L, int pieces_per_row,
               int64_t tail_begin, const int32_t* __restrict__ idx, const int64_t* __restrict__ offsets,
               uint4* __restrict__ Kc, uint4* __restrict__ Vc, int32_t* __restrict__ pos,
               int64_t* __restrict__ state, int64_t pos_begin, int64_t pos_end) {
  const int u = blockIdx.y;
  int64_t* st = state + size_t(u) * TCA_STATE_WORDS;
  // Programmatic dependent launch: the prefill that follows may be scheduled now and, in its
  // band-first order, work on the window band while this gather runs; this grid waits for the
  // selection before it reads the index set.
  pdl_launch_dependents();
  pdl_wait();
  const int64_t seg = st[TCA_ST_SEG_START];
  const int64_t gcap = st[TCA_ST_GLOBAL_CAP];
  const int64_t off = offsets[u];
  const int64_t n_sel = offsets[u + 1] - off;
  const int64_t n_tail = L - tail_begin;
  const int64_t n_rows = n_sel + n_tail;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    st[TCA_ST_N_GLOBAL] = n_sel;
    st[TCA_ST_TAIL_HEAD] = 0;
    st[TCA_ST_N_TAIL] = n_tail;
    st[TCA_ST_SEQ_LEN] = L;
  }
  const int64_t r0 = int64_t(blockIdx.x) * kRowsPerCta;
  if (r0 >= n_rows) return;
  const int64_t r1 = min(r0 + int64_t(kRowsPerCta), n_rows);
  const int64_t n_pieces = (r1 - r0) * pieces_per_row;
  const uint4* Ku = K + size_t(u) * L * pieces_per_row;
  const uint4* Vu = V + size_t(u) * L * pieces_per_row;
  const int shift = 31 - __clz(pieces_per_row);  // pieces_per_row is a power of two
  for (int64_t p0 = threadIdx.x; p0 < n_pieces; p0 += 4 * kThreads) {
    uint4 kv[4], vv[4];
    int64_t dst[4];
    int32_t src[4];
    bool lead[4], inr[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int64_t p = p0 + int64_t(i) * kThreads;
      dst[i] = -1;
      if (p < n_pieces) {
        const int64_t r = r0 + (p >> shift);
        const int piece = int(p & (pieces_per_row - 1));
        const int64_t s = (r < n_sel) ? int64_t(idx[off + r]) : tail_begin + (r - n_sel);
        const int64_t drow = (r < n_sel) ? seg + r : seg + gcap + (r - n_sel);
        if constexpr (kDebugBounds) {
          // a selected index must name a candidate token, and its row must fit the global region
          if (r < n_sel && (s < 0 || s >= tail_begin || r >= gcap)) {
            if (piece == 0) report_bounds_state(st, kBoundsSelectedIndex, s);
            continue;   // skip the access: dst[i] stays -1
          }
        }
        src[i] = int32_t(s);
        lead[i] = piece == 0;
        dst[i] = drow * pieces_per_row + piece;
        // a ranged call moves only the rows whose position it was given; positions are written by every call
        inr[i] = s >= pos_begin && s < pos_end;
        if (inr[i]) {
          kv[i] = __ldcs(Ku + s * pieces_per_row + piece);
          vv[i] = __ldcs(Vu + s * pieces_per_row + piece);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (dst[i] >= 0) {
        if (inr[i]) {
          Kc[dst[i]] = kv[i];
          Vc[dst[i]] = vv[i];
        }
        if (lead[i]) pos[dst[i] >> shift] = src[i];
      }
    }
  }
}

}  // namespace
}  // namespace tca

using namespace tca;

namespace tca {
namespace {
int compact_impl(const tca_params* prm, const void* K, const void* V, int64_t L, int64_t pos_begin, int64_t pos_end,
                 const int32_t* idx, const int64_t* offsets_dev, const int64_t* offsets_host, tca_cache_desc* c,
                 void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  TCA_CHECK_ARG(K && V && offsets_dev && offsets_host && c);
  TCA_CHECK_ARG(c->k && c->v && c->pos && c->state && c->seg_start && c->global_cap && c->n_global &&
                c->tail_head && c->n_tail && c->seq_len);
  TCA_CHECK_ARG(L >= 1 && L < (int64_t(1) << 31));
  TCA_CHECK_ARG(pos_begin >= 0 && pos_begin < pos_end && pos_end <= L);
  TCA_CHECK_ARG(aligned(K, 16) && aligned(V, 16) && aligned(c->k, 16) && aligned(c->v, 16));
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  TCA_CHECK_ARG(c->n_units == U && U <= 65535);
  const int64_t m = num_blocks(prm, L);
  const int64_t tail_begin = m * prm->block;
  const int64_t n_tail = L - tail_begin;
  int64_t max_rows = 0;
  TCA_CHECK_ARG(offsets_host[0] == 0);
  for (int64_t u = 0; u < U; ++u) {
    const int64_t n_sel = offsets_host[u + 1] - offsets_host[u];
    TCA_CHECK_ARG(n_sel >= 0 && n_sel <= tail_begin);
    if (n_sel > c->global_cap[u] || n_tail > c->tail_cap) return TCA_ERR_CAPACITY;
    max_rows = n_sel + n_tail > max_rows ? n_sel + n_tail : max_rows;
  }
  TCA_CHECK_ARG(idx != nullptr || offsets_host[U] == 0);
  const int pieces_per_row = int(prm->head_dim * elt_size(prm->dtype) / 16);
  if (max_rows == 0) max_rows = 1;  // still updates the device state
  dim3 grid(static_cast<unsigned>((max_rows + kRowsPerCta - 1) / kRowsPerCta), static_cast<unsigned>(U));
  st = launch_pdl(compact_kernel, grid, dim3(kThreads), size_t(0), static_cast<cudaStream_t>(stream),
                  static_cast<const uint4*>(K), static_cast<const uint4*>(V), L, pieces_per_row, tail_begin, idx,
                  offsets_dev, static_cast<uint4*>(c->k), static_cast<uint4*>(c->v), c->pos, c->state, pos_begin,
                  pos_end);
  if (st != TCA_OK) return st;
  for (int64_t u = 0; u < U; ++u) {
    c->n_global[u] = offsets_host[u + 1] - offsets_host[u];
    c->tail_head[u] = 0;
    c->n_tail[u] = n_tail;
    c->seq_len[u] = L;
  }
  return TCA_OK;
}
}  // namespace
}  // namespace tca

extern "C" int tca_compact_kv(const tca_params* prm, const void* K, const void* V, int64_t L,
                              const int32_t* idx, const int64_t* offsets_dev, const int64_t* offsets_host,
                              tca_cache_desc* c, void* stream) {
  return compact_impl(prm, K, V, L, 0, L >= 1 ? L : 1, idx, offsets_dev, offsets_host, c, stream);
}

// The rows whose position lies in [pos_begin, pos_end) only: for a caller whose K and V arrive in
// pieces.  Positions and state words are written by every call.
extern "C" int tca_compact_kv_range(const tca_params* prm, const void* K, const void* V, int64_t L,
                                    int64_t pos_begin, int64_t pos_end, const int32_t* idx,
                                    const int64_t* offsets_dev, const int64_t* offsets_host, tca_cache_desc* c,
                                    void* stream) {
  return compact_impl(prm, K, V, L, pos_begin, pos_end, idx, offsets_dev, offsets_host, c, stream);
}
