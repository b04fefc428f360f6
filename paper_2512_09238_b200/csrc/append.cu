// tca_cache_append: decode-time cache maintenance (Section 4.2, "Online Token Selection
// in Decoding Stage").  One CTA per unit: write the new key/value into the tail ring and,
// when the ring then holds window + block tokens, compress the block that leaves the
// window: score its b keys with the current query group (Eq. 5 restricted to the block,
// fp64), keep the top t_keep by the same radix select the prefill uses, and move those
// rows to the end of the global region in ascending position.
#include "common.cuh"
#include "rowslice.cuh"

namespace tca {
namespace {

constexpr int kThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kThreads)
cache_append_kernel(const T* __restrict__ k_new, const T* __restrict__ v_new, const T* __restrict__ q_cur,
                    T* __restrict__ Kc, T* __restrict__ Vc, int32_t* __restrict__ pos,
                    int64_t* __restrict__ state, int64_t tail_cap, int D, int G, int b, int window,
                    double sm_scale) {
  pdl_wait();                 // the previous step's kernels still read the cache and its state
  pdl_launch_dependents();
  const int u = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, lane16 = tid & 15, grp = tid >> 4;
  int64_t* st = state + size_t(u) * TCA_STATE_WORDS;
  // the new row is requested together with the state words (one trip to memory instead of two);
  // head_dim <= 128 < kThreads, so a thread holds at most one element of it
  T k_val = T(), v_val = T();
  if (tid < D) {
    k_val = k_new[size_t(u) * D + tid];
    v_val = v_new[size_t(u) * D + tid];
  }
  const int64_t seg = st[TCA_ST_SEG_START], gcap = st[TCA_ST_GLOBAL_CAP];
  const int64_t n_global = st[TCA_ST_N_GLOBAL], tail_head = st[TCA_ST_TAIL_HEAD];
  const int64_t n_tail = st[TCA_ST_N_TAIL], seq_len = st[TCA_ST_SEQ_LEN];
  const int t_keep = int(st[TCA_ST_T_KEEP]);
  const int64_t ring = seg + gcap;
  __syncthreads();  // every thread has read the state before anyone updates it

  if constexpr (kDebugBounds) {
    // the state words this kernel indexes with: ring position and fill, and room for a kept block
    const bool bad_ring = tail_head < 0 || tail_head >= tail_cap || n_tail < 0 || n_tail >= tail_cap;
    const bool bad_room = (n_tail + 1 >= int64_t(window) + b) && (t_keep < 0 || t_keep > b || n_global + t_keep > gcap);
    if (bad_ring || bad_room) {
      if (tid == 0) report_bounds_state(st, bad_ring ? kBoundsRingSlot : kBoundsGlobalRegion, bad_ring ? tail_head : n_global);
      return;
    }
  }
  // ---- append
  {
    const int64_t slot = (tail_head + n_tail) % tail_cap;
    if (tid < D) {
      Kc[(ring + slot) * D + tid] = k_val;
      Vc[(ring + slot) * D + tid] = v_val;
    }
    if (tid == 0) pos[ring + slot] = int32_t(seq_len);
  }
  const int64_t n_tail1 = n_tail + 1;
  const bool compress = n_tail1 >= int64_t(window) + b;
  if (!compress) {
    if (tid == 0) {
      st[TCA_ST_N_TAIL] = n_tail1;
      st[TCA_ST_SEQ_LEN] = seq_len + 1;
    }
    return;
  }
  __syncthreads();  // the appended row is visible to the CTA (it is in the block when w = 0)

  // ---- logits of the b oldest tail tokens against the G current queries, fp64
  __shared__ double xs[kMaxGroup][kMaxBlock];
  __shared__ double lse[kMaxGroup];
  __shared__ int kept_slot[kMaxBlock];
  const int EPL = D / 16;
  for (int i0 = 0; i0 < b; i0 += kThreads / 16) {  // uniform trip count: shuffles below need whole warps
    const int i = min(i0 + grp, b - 1);
    int64_t slot = tail_head + i;
    if (slot >= tail_cap) slot -= tail_cap;
    const T* krow = Kc + (ring + slot) * D + lane16 * EPL;
    for (int g = 0; g < G; ++g) {
      const T* qrow = q_cur + (size_t(u) * G + g) * D + lane16 * EPL;
      double acc = 0.0;
      for (int e = 0; e < EPL; ++e) acc = fma(double(elt_to_float(qrow[e])), double(elt_to_float(krow[e])), acc);
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) acc += shfl_xor_double(acc, off);
      if (lane16 == 0 && i0 + grp < b) xs[g][i] = acc * sm_scale;
    }
  }
  __syncthreads();
  if (warp < G) {  // log-sum-exp of head `warp` over the block
    double mx = -1.0e308;
    for (int i = lane; i < b; i += 32) mx = fmax(mx, xs[warp][i]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mx = fmax(mx, shfl_xor_double(mx, off));
    double sum = 0.0;
    for (int i = lane; i < b; i += 32) sum += exp(xs[warp][i] - mx);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) sum += shfl_xor_double(sum, off);
    if (lane == 0) lse[warp] = mx + log(sum);
  }
  __syncthreads();
  if (warp == 0) {
    unsigned long long key[4];
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const int i = s * 32 + lane;
      double score = -1.0e308;
      if (i < b) {
        if (G == 1) {
          score = xs[0][i] - lse[0];
        } else {
          double top = -1.0e308;
          for (int g = 0; g < G; ++g) top = fmax(top, xs[g][i] - lse[g]);
          double sum = 0.0;
          for (int g = 0; g < G; ++g) sum += exp(xs[g][i] - lse[g] - top);
          score = top + log(sum);
        }
      }
      key[s] = ordered_key(score);
    }
    const unsigned keep = radix_select_top_t(key, b, t_keep, lane);
    int before = 0;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const bool k = (keep >> s) & 1u;
      const unsigned bal = __ballot_sync(0xffffffffu, k);
      if (k) kept_slot[before + __popc(bal & ((1u << lane) - 1u))] = s * 32 + lane;
      before += __popc(bal);
    }
  }
  __syncthreads();
  // ---- move the kept rows to the end of the global region (ring and region are disjoint)
  for (int i = tid; i < t_keep * D; i += kThreads) {
    const int r = i / D, e = i - r * D;
    int64_t slot = tail_head + kept_slot[r];
    if (slot >= tail_cap) slot -= tail_cap;
    Kc[(seg + n_global + r) * D + e] = Kc[(ring + slot) * D + e];
    Vc[(seg + n_global + r) * D + e] = Vc[(ring + slot) * D + e];
    if (e == 0) pos[seg + n_global + r] = pos[ring + slot];
  }
  if (tid == 0) {
    st[TCA_ST_N_GLOBAL] = n_global + t_keep;
    st[TCA_ST_TAIL_HEAD] = (tail_head + b) % tail_cap;
    st[TCA_ST_N_TAIL] = n_tail1 - b;
    st[TCA_ST_SEQ_LEN] = seq_len + 1;
  }
}

}  // namespace
}  // namespace tca

using namespace tca;

extern "C" int tca_cache_append(const tca_params* prm, tca_cache_desc* c, const void* k_new, const void* v_new,
                                const void* q_cur, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  TCA_CHECK_ARG(c && k_new && v_new && q_cur);
  TCA_CHECK_ARG(c->k && c->v && c->pos && c->state && c->global_cap && c->n_global && c->tail_head &&
                c->n_tail && c->seq_len && c->t_keep);
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  TCA_CHECK_ARG(c->n_units == U);
  const int64_t full = int64_t(prm->window) + prm->block;
  if (c->tail_cap < full) return TCA_ERR_CAPACITY;
  for (int64_t u = 0; u < U; ++u) {
    TCA_CHECK_ARG(c->n_tail[u] < full);
    if (c->n_tail[u] + 1 >= full && c->n_global[u] + c->t_keep[u] > c->global_cap[u]) return TCA_ERR_CAPACITY;
    TCA_CHECK_ARG(c->seq_len[u] + 1 < (int64_t(1) << 31));
  }
  const int G = prm->n_q_heads / prm->n_kv_heads;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (prm->dtype == TCA_BF16) {
    using T = __nv_bfloat16;
    st = launch_pdl(cache_append_kernel<T>, dim3(unsigned(U)), dim3(kThreads), size_t(0), s,
                    static_cast<const T*>(k_new), static_cast<const T*>(v_new), static_cast<const T*>(q_cur),
                    static_cast<T*>(c->k), static_cast<T*>(c->v), c->pos, c->state, c->tail_cap, prm->head_dim, G,
                    prm->block, prm->window, double(prm->sm_scale));
  } else {
    using T = float;
    st = launch_pdl(cache_append_kernel<T>, dim3(unsigned(U)), dim3(kThreads), size_t(0), s,
                    static_cast<const T*>(k_new), static_cast<const T*>(v_new), static_cast<const T*>(q_cur),
                    static_cast<T*>(c->k), static_cast<T*>(c->v), c->pos, c->state, c->tail_cap, prm->head_dim, G,
                    prm->block, prm->window, double(prm->sm_scale));
  }
  if (st != TCA_OK) return st;
  for (int64_t u = 0; u < U; ++u) {
    c->n_tail[u] += 1;
    c->seq_len[u] += 1;
    if (c->n_tail[u] >= full) {
      c->n_global[u] += c->t_keep[u];
      c->tail_head[u] = (c->tail_head[u] + prm->block) % c->tail_cap;
      c->n_tail[u] -= prm->block;
    }
  }
  return TCA_OK;
}
