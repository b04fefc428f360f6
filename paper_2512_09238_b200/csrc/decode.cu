// tca_attn_decode: one query per head over the whole retained cache of its KV head
// (Eq. 2 at decode time; HBM-bound: every retained K and V row is read exactly once per
// step and shared by the G query heads of the group).
//
//   decode_split_kernel   CTA = (chunk of kDecodeChunkRows cache rows, unit).  Phase A
//                         streams the chunk's K rows (16 lanes x 16 B per row), forms the
//                         G logits per row with a transposing shuffle butterfly and parks
//                         them in shared memory; the chunk maximum and exp2 follow; phase B
//                         streams the V rows and accumulates p*V per lane slice.  Writes an
//                         un-normalised partial (acc, max, sum) per (chunk, query head).
//   decode_combine_kernel merges a unit's partials in chunk order (fixed order => bit-
//                         reproducible) and normalises.
#include <mutex>

#include "common.cuh"
#include "rowslice.cuh"

namespace tca {
namespace {

constexpr int kThreads = 256;
constexpr int kGroups = kThreads / 16;
constexpr int CH = kDecodeChunkRows;

template <int G>
struct DecCfg {
  static constexpr int R = (G == 1) ? 16 : (G == 2) ? 8 : 4;
  static constexpr int NV = R * G;
  static constexpr int NB = (NV + 15) / 16;
  static constexpr int NVP = NB * 16;
};

struct UnitView {
  int64_t seg, gcap, n_global, tail_head, n_tail, tail_cap;
  __device__ __forceinline__ int64_t len() const { return n_global + n_tail; }
  // logical row (global rows first, then the tail oldest-first) -> physical cache row
  __device__ __forceinline__ int64_t phys(int64_t r) const {
    if (r < n_global) return seg + r;
    int64_t slot = tail_head + (r - n_global);
    if (slot >= tail_cap) slot -= tail_cap;
    return seg + gcap + slot;
  }
};

__device__ __forceinline__ UnitView load_unit(const int64_t* state, int u, int64_t tail_cap) {
  const int64_t* st = state + size_t(u) * TCA_STATE_WORDS;
  UnitView v;
  v.seg = st[TCA_ST_SEG_START];
  v.gcap = st[TCA_ST_GLOBAL_CAP];
  v.n_global = st[TCA_ST_N_GLOBAL];
  v.tail_head = st[TCA_ST_TAIL_HEAD];
  v.n_tail = st[TCA_ST_N_TAIL];
  v.tail_cap = tail_cap;
  return v;
}

__device__ __forceinline__ int64_t partial_base(const UnitView& v, int u) {
  return v.seg / CH + 2 * int64_t(u);
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kThreads)
decode_split_kernel(const T* __restrict__ q, const T* __restrict__ Kc, const T* __restrict__ Vc,
                    const int64_t* __restrict__ state, int64_t tail_cap, float scale_log2e,
                    float* __restrict__ partial) {
  using Cfg = DecCfg<G>;
  constexpr int EPL = D / 16;
  constexpr int R = Cfg::R, NB = Cfg::NB;
  const int u = blockIdx.y;
  const int chunk = blockIdx.x;
  const UnitView uv = load_unit(state, u, tail_cap);
  const int64_t len = uv.len();
  const int64_t row0 = int64_t(chunk) * CH;
  if (row0 >= len) return;
  const int n_rows = int(min(int64_t(CH), len - row0));
  const int tid = threadIdx.x, lane16 = tid & 15, grp = tid >> 4, warp = tid >> 5;

  __shared__ float xs[CH][G];
  __shared__ float red[kThreads / 32][G][D];
  __shared__ float stat_m[G], stat_l[G];
  __shared__ float wred[kThreads / 32][G];

  float qf[G][EPL];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int e = 0; e < EPL; ++e)
      qf[g][e] = elt_to_float(q[(size_t(u) * G + g) * D + lane16 * EPL + e]) * scale_log2e;

  // ---- phase A: logits (in log2 units) of every row of the chunk
  for (int base = 0; base < CH; base += kGroups * R) {
    RowF<T, EPL> raw[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int lr = base + r * kGroups + grp;
      if (lr < n_rows) raw[r].load(Kc + size_t(uv.phys(row0 + lr)) * D + lane16 * EPL);
      else raw[r].zero();
    }
    float acc[Cfg::NVP];
#pragma unroll
    for (int i = 0; i < Cfg::NVP; ++i) acc[i] = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const float kf = raw[r].get(e);
#pragma unroll
        for (int g = 0; g < G; ++g) acc[r * G + g] = fmaf(qf[g][e], kf, acc[r * G + g]);
      }
#pragma unroll
    for (int bf = 0; bf < NB; ++bf) {
      float part[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) part[i] = acc[bf * 16 + i];
      const float x = butterfly16f(part, lane16);
      const int v = bf * 16 + lane16;
      const int r = v / G, g = v - r * G;
      const int lr = base + r * kGroups + grp;
      if (v < Cfg::NV && lr < CH) xs[lr][g] = (lr < n_rows) ? x : -INFINITY;
    }
  }
  __syncthreads();

  // ---- chunk maximum, exponentials and their sum, per query head (thread = row)
  {
    float xv[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      xv[g] = xs[tid][g];
      float mx = xv[g];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      if ((tid & 31) == 0) wred[warp][g] = mx;
    }
    __syncthreads();
    if (tid < G) {
      float mx = wred[0][tid];
      for (int w = 1; w < kThreads / 32; ++w) mx = fmaxf(mx, wred[w][tid]);
      stat_m[tid] = mx;
    }
    __syncthreads();
    float pv[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      pv[g] = exp2f(xv[g] - stat_m[g]);
      xs[tid][g] = pv[g];
      float sum = pv[g];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
      if ((tid & 31) == 0) wred[warp][g] = sum;
    }
    __syncthreads();
    if (tid < G) {
      float sum = 0.f;
      for (int w = 0; w < kThreads / 32; ++w) sum += wred[w][tid];
      stat_l[tid] = sum;
    }
  }
  __syncthreads();

  // ---- phase B: acc[g][e] += p[row][g] * V[row][e]
  float o[G][EPL];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[g][e] = 0.f;
  constexpr int RB = 4;
  for (int base = 0; base < n_rows; base += kGroups * RB) {
    RowF<T, EPL> raw[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      const int lr = base + r * kGroups + grp;
      if (lr < n_rows) raw[r].load(Vc + size_t(uv.phys(row0 + lr)) * D + lane16 * EPL);
      else raw[r].zero();
    }
#pragma unroll
    for (int r = 0; r < RB; ++r) {
      const int lr = min(base + r * kGroups + grp, CH - 1);
      float p[G];
#pragma unroll
      for (int g = 0; g < G; ++g) p[g] = xs[lr][g];
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const float vf = raw[r].get(e);
#pragma unroll
        for (int g = 0; g < G; ++g) o[g][e] = fmaf(p[g], vf, o[g][e]);
      }
    }
  }
  // the two 16-lane groups of a warp, then the warps, in a fixed order
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[g][e] += __shfl_xor_sync(0xffffffffu, o[g][e], 16);
  if ((tid & 31) < 16) {
#pragma unroll
    for (int g = 0; g < G; ++g)
#pragma unroll
      for (int e = 0; e < EPL; ++e) red[warp][g][lane16 * EPL + e] = o[g][e];
  }
  __syncthreads();
  float* out = partial + size_t(partial_base(uv, u) + chunk) * G * (D + 2);
  for (int i = tid; i < G * D; i += kThreads) {
    const int g = i / D, d = i - g * D;
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) sum += red[w][g][d];
    out[size_t(g) * (D + 2) + d] = sum;
  }
  if (tid < G) {
    out[size_t(tid) * (D + 2) + D] = stat_m[tid];
    out[size_t(tid) * (D + 2) + D + 1] = stat_l[tid];
  }
}

template <typename T, int D, int G>
__global__ void __launch_bounds__(kThreads)
decode_combine_kernel(const float* __restrict__ partial, const int64_t* __restrict__ state, int64_t tail_cap,
                      T* __restrict__ O) {
  constexpr int NCL = kThreads / D;  // chunk lanes
  const int g = blockIdx.x, u = blockIdx.y;
  const UnitView uv = load_unit(state, u, tail_cap);
  const int n_chunks = int((uv.len() + CH - 1) / CH);
  const float* base = partial + size_t(partial_base(uv, u)) * G * (D + 2) + size_t(g) * (D + 2);
  const size_t stride = size_t(G) * (D + 2);
  const int tid = threadIdx.x, d = tid % D, cl = tid / D;
  __shared__ float s_max[kThreads / 32];
  __shared__ float s_acc[NCL][D], s_l[NCL];

  float mx = -INFINITY;
  for (int c = tid; c < n_chunks; c += kThreads) mx = fmaxf(mx, base[c * stride + D]);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  if ((tid & 31) == 0) s_max[tid >> 5] = mx;
  __syncthreads();
  mx = s_max[0];
#pragma unroll
  for (int w = 1; w < kThreads / 32; ++w) mx = fmaxf(mx, s_max[w]);

  float acc = 0.f, l = 0.f;
  for (int c = cl; c < n_chunks; c += NCL) {
    const float* p = base + c * stride;
    const float w = exp2f(p[D] - mx);
    acc = fmaf(p[d], w, acc);
    l = fmaf(p[D + 1], w, l);
  }
  s_acc[cl][d] = acc;
  if (d == 0) s_l[cl] = l;
  __syncthreads();
  if (cl == 0) {
    float a = 0.f, ls = 0.f;
#pragma unroll
    for (int i = 0; i < NCL; ++i) { a += s_acc[i][d]; ls += s_l[i]; }
    store_elt(O + (size_t(u) * G + g) * D + d, n_chunks > 0 ? a / ls : 0.f);
  }
}

template <typename T, int D, int G>
int launch_decode(const tca_params* prm, const void* q, const tca_cache_desc* c, void* O, const DecodeWs& ws,
                  int64_t max_len, cudaStream_t stream) {
  const int U = prm->batch * prm->n_kv_heads;
  const float scale_log2e = prm->sm_scale * 1.4426950408889634f;
  dim3 grid(unsigned((max_len + CH - 1) / CH), unsigned(U));
  decode_split_kernel<T, D, G><<<grid, kThreads, 0, stream>>>(
      static_cast<const T*>(q), static_cast<const T*>(c->k), static_cast<const T*>(c->v), c->state,
      c->tail_cap, scale_log2e, ws.partial);
  int st = check_launch();
  if (st != TCA_OK) return st;
  decode_combine_kernel<T, D, G><<<dim3(G, unsigned(U)), kThreads, 0, stream>>>(ws.partial, c->state, c->tail_cap,
                                                                               static_cast<T*>(O));
  return check_launch();
}

template <typename T, int D>
int dispatch_group(int G, const tca_params* prm, const void* q, const tca_cache_desc* c, void* O,
                   const DecodeWs& ws, int64_t max_len, cudaStream_t s) {
  switch (G) {
    case 1: return launch_decode<T, D, 1>(prm, q, c, O, ws, max_len, s);
    case 2: return launch_decode<T, D, 2>(prm, q, c, O, ws, max_len, s);
    case 3: return launch_decode<T, D, 3>(prm, q, c, O, ws, max_len, s);
    case 4: return launch_decode<T, D, 4>(prm, q, c, O, ws, max_len, s);
    case 5: return launch_decode<T, D, 5>(prm, q, c, O, ws, max_len, s);
    case 6: return launch_decode<T, D, 6>(prm, q, c, O, ws, max_len, s);
    case 7: return launch_decode<T, D, 7>(prm, q, c, O, ws, max_len, s);
    case 8: return launch_decode<T, D, 8>(prm, q, c, O, ws, max_len, s);
    default: return TCA_ERR_UNSUPPORTED;
  }
}

}  // namespace
}  // namespace tca

using namespace tca;

extern "C" int tca_attn_decode(const tca_params* prm, const void* q, const tca_cache_desc* c, void* O,
                               void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  TCA_CHECK_ARG(q && c && O && ws);
  TCA_CHECK_ARG(c->k && c->v && c->state && c->n_global && c->n_tail);
  TCA_CHECK_ARG(aligned(q, 16) && aligned(O, 16) && aligned(ws, 256) && aligned(c->k, 16) && aligned(c->v, 16));
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  TCA_CHECK_ARG(c->n_units == U && U <= 65535);
  DecodeWs lay = decode_ws_layout(prm, c->rows_total, U, ws);
  if (ws_bytes < lay.bytes) return TCA_ERR_WORKSPACE;
  int64_t max_len = 0;
  for (int64_t u = 0; u < U; ++u) {
    const int64_t len = c->n_global[u] + c->n_tail[u];
    max_len = len > max_len ? len : max_len;
  }
  TCA_CHECK_ARG(max_len >= 1);
  const int G = prm->n_q_heads / prm->n_kv_heads;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (prm->dtype == TCA_BF16) {
    if (prm->head_dim == 128) return dispatch_group<__nv_bfloat16, 128>(G, prm, q, c, O, lay, max_len, s);
    return dispatch_group<__nv_bfloat16, 64>(G, prm, q, c, O, lay, max_len, s);
  }
  if (prm->head_dim == 128) return dispatch_group<float, 128>(G, prm, q, c, O, lay, max_len, s);
  return dispatch_group<float, 64>(G, prm, q, c, O, lay, max_len, s);
}

// ---------------------------------------------------------------------------------------
// Decode without any allocation: the split-KV partials live in a fixed array inside the
// library image instead of a caller-provided workspace.
namespace tca {
namespace {

constexpr size_t kStaticScratchBytes = size_t(TCA_DECODE_STATIC_SCRATCH_BYTES);
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_decode_scratch[kStaticScratchBytes];

std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of g_decode_scratch on the current device.  In host code the array's
// name is only a handle; the address a kernel can use comes from cudaGetSymbolAddress,
// looked up once per device with that device current.
int static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return TCA_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return TCA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_decode_scratch) != cudaSuccess || p == nullptr) return TCA_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return TCA_OK;
}

}  // namespace
}  // namespace tca

extern "C" int tca_attn_decode_static(const tca_params* prm, const void* q, const tca_cache_desc* c, void* O,
                                      void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  TCA_CHECK_ARG(q && c && O);
  TCA_CHECK_ARG(c->k && c->v && c->state && c->n_global && c->n_tail);
  TCA_CHECK_ARG(aligned(q, 16) && aligned(O, 16) && aligned(c->k, 16) && aligned(c->v, 16));
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  TCA_CHECK_ARG(c->n_units == U && U <= 65535);
  // same layout as the workspace variant; refuse what does not fit the built-in array
  DecodeWs lay = decode_ws_layout(prm, c->rows_total, U, nullptr);
  if (lay.bytes > kStaticScratchBytes) return TCA_ERR_SCRATCH_LIMIT;
  void* scratch = nullptr;
  st = static_scratch(&scratch);
  if (st != TCA_OK) return st;
  lay = decode_ws_layout(prm, c->rows_total, U, scratch);
  int64_t max_len = 0;
  for (int64_t u = 0; u < U; ++u) {
    const int64_t len = c->n_global[u] + c->n_tail[u];
    max_len = len > max_len ? len : max_len;
  }
  TCA_CHECK_ARG(max_len >= 1);
  const int G = prm->n_q_heads / prm->n_kv_heads;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (prm->dtype == TCA_BF16) {
    if (prm->head_dim == 128) return dispatch_group<__nv_bfloat16, 128>(G, prm, q, c, O, lay, max_len, s);
    return dispatch_group<__nv_bfloat16, 64>(G, prm, q, c, O, lay, max_len, s);
  }
  if (prm->head_dim == 128) return dispatch_group<float, 128>(G, prm, q, c, O, lay, max_len, s);
  return dispatch_group<float, 64>(G, prm, q, c, O, lay, max_len, s);
}
