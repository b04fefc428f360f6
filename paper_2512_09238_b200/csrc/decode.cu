// tca_attn_decode: one query per head over the whole retained cache of its KV head
// (Eq. 2 at decode time; HBM-bound: every retained K and V row is read exactly once per
// step and shared by the G query heads of the group).
//
//   decode_split_kernel   CTA = (slice of a unit's cache rows, unit); the rows of all units are cut
//                         into about two slices per SM.  A producer warp streams the slice's K and
//                         V rows through a shared-memory ring of 64-row tiles with 1-D bulk
//                         asynchronous copies (up to 96 KB in flight per CTA, independent of the
//                         consumers' registers).  Eight consumer warps work in rounds of 256 rows:
//                         K phase (G logits per row by a transposing shuffle butterfly, parked in
//                         shared memory), running maximum + exp2, V phase (p*V per lane slice).
//                         Writes one un-normalised partial (acc, max, sum) per (slice, query head).
//   decode_combine_kernel merges a unit's partials in slice order (fixed order => bit-
//                         reproducible) and normalises.
#include <mutex>

#include "bulk_ring.cuh"
#include "common.cuh"
#include "decode_common.cuh"
#include "rowslice.cuh"

namespace tca {

template <int D>
int launch_decode_mma(const tca_params*, const void*, const tca_cache_desc*, const DecodeWs&, int64_t, int,
                      cudaStream_t);

namespace {

constexpr int kConsumers = 256;              // 8 consumer warps
constexpr int kThreads = kConsumers + 32;    // + 1 producer warp
constexpr int kGroups = kConsumers / 16;     // 16-lane groups, one cache row each
constexpr int kTileRows = 64;                // rows per ring tile (4 per lane group)
constexpr int kSuperRows = 256;              // rows per softmax round (4 tiles)
constexpr int kRingBytes = 96 * 1024;

template <int G>
struct DecCfg {
  static constexpr int R = 4;                // rows per lane group per tile
  static constexpr int NV = R * G;
  static constexpr int NB = (NV + 15) / 16;
  static constexpr int NVP = NB * 16;
};

template <typename T, int D>
struct DecRing {
  static constexpr int kTileBytes = kTileRows * D * int(sizeof(T));
  static constexpr int kStages = kRingBytes / kTileBytes > 8 ? 8 : kRingBytes / kTileBytes;
  static constexpr int kSmemBytes = kStages * kTileBytes + 1024;
};

template <typename T, int D, int G>
__global__ void __maxnreg__(112)
decode_split_kernel(const T* __restrict__ q, const T* __restrict__ Kc, const T* __restrict__ Vc,
                    const int64_t* __restrict__ state, int64_t tail_cap, float scale_log2e, int target,
                    float* __restrict__ partial, int* __restrict__ status, int n_units) {
  using Cfg = DecCfg<G>;
  using Ring = DecRing<T, D>;
  constexpr int EPL = D / 16;
  constexpr int R = Cfg::R, NB = Cfg::NB;
  constexpr int kStages = Ring::kStages;
  pdl_wait();
  pdl_launch_dependents();
  __shared__ SliceId slice_slot;
  const SliceId slice = find_slice(state, n_units, target, tail_cap, &slice_slot);
  if (slice.u < 0) return;
  const int u = slice.u, part_idx = slice.part, np = slice.np;
  const UnitView uv = slice.uv;
  const int64_t len = uv.len();
  const int64_t row0 = slice_begin(len, np, part_idx);
  const int n_rows = int(slice_begin(len, np, part_idx + 1) - row0);
  const int n_super = (n_rows + kSuperRows - 1) / kSuperRows;
  const int tid = threadIdx.x, lane16 = tid & 15, grp = tid >> 4, warp = tid >> 5;
  const int base_slot = slice.base_slot;

  extern __shared__ uint8_t dec_smem_raw[];
  uint8_t* ring_buf = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(dec_smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ BulkRing<kStages> ring;
  __shared__ int abort_word;
  __shared__ float xs[kSuperRows][G];
  __shared__ float stat_m[G], stat_c[G], stat_l[G];
  __shared__ float wred[kConsumers / 32][G];
  volatile int* abort_flag = &abort_word;
  if (tid == 0) {
    ring.init(kConsumers / 32);   // one release per consumer warp
    abort_word = 0;
  }
  if (tid < G) { stat_m[tid] = -INFINITY; stat_l[tid] = 0.f; }
  __syncthreads();

  if (warp == kConsumers / 32) {
    // ------------------------------------------------------------- producer: K tiles then V tiles of every round
    if ((tid & 31) == 0) {
      int n = 0;
      for (int s = 0; s < n_super; ++s) {
        const int srow = s * kSuperRows;
        const int rows_here = min(kSuperRows, n_rows - srow);
        const int tiles = (rows_here + kTileRows - 1) / kTileRows;
        for (int kv = 0; kv < 2; ++kv) {
          const T* src = kv ? Vc : Kc;
          for (int k = 0; k < tiles; ++k, ++n) {
            const int trow = srow + k * kTileRows;
            const int cnt = min(kTileRows, n_rows - trow);
            if (!ring.acquire(n, uint32_t(cnt) * D * sizeof(T), abort_flag)) return;
            uint8_t* dst = ring_buf + (n % kStages) * Ring::kTileBytes;
            int done = 0;
            while (done < cnt) {   // at most three physically contiguous runs
              const int64_t r = row0 + trow + done;
              const int run = int(uv.run(r, cnt - done));
              if constexpr (kDebugBounds) {
                const int64_t y = uv.phys(r);
                if (run <= 0 || y < uv.seg || y + run > uv.seg + uv.gcap + uv.tail_cap) {
                  report_bounds_ws(status, kBoundsCacheRow, y);
                  *abort_flag = 1;   // the consumers leave their waits; nothing is copied
                  return;
                }
              }
              bulk_copy_g2s(dst + size_t(done) * D * sizeof(T), src + size_t(uv.phys(r)) * D,
                            uint32_t(run) * D * sizeof(T), &ring.full[n % kStages]);
              done += run;
            }
          }
        }
      }
    }
    return;
  }

  // --------------------------------------------------------------- consumers
  float qf[G][EPL];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int e = 0; e < EPL; ++e)
      qf[g][e] = elt_to_float(q[(size_t(u) * G + g) * D + lane16 * EPL + e]) * scale_log2e;
  float o[G][EPL];
#pragma unroll
  for (int g = 0; g < G; ++g)
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[g][e] = 0.f;

  int n = 0;
  bool ok = true;
  // A wait that gives up clears `ok`; the thread then skips the work but still walks the same
  // barriers as everybody else, so nobody is left waiting at a barrier.
  for (int s = 0; s < n_super; ++s) {
    const int srow = s * kSuperRows;
    const int rows_here = min(kSuperRows, n_rows - srow);
    const int tiles = (rows_here + kTileRows - 1) / kTileRows;
    // ---- phase A: logits (log2 units) of the round's rows
    for (int k = 0; k < tiles; ++k, ++n) {
      if (ok) ok = ring.wait_full(n, abort_flag);
      if (!ok) continue;
      const T* tile = reinterpret_cast<const T*>(ring_buf + (n % kStages) * Ring::kTileBytes);
      RowF<T, EPL> raw[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int tr = r * kGroups + grp;                   // row inside the tile
        if (k * kTileRows + tr < rows_here) raw[r].load_cached(tile + size_t(tr) * D + lane16 * EPL);
        else raw[r].zero();
      }
      __syncwarp();
      if ((tid & 31) == 0) ring.release(n);
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
        const int lr = k * kTileRows + r * kGroups + grp;
        if (v < Cfg::NV) xs[lr][g] = (lr < rows_here) ? x : -INFINITY;
      }
    }
    consumer_sync(kConsumers);
    // ---- running maximum, exponentials and their sum, per query head (thread = row)
    {
      const bool live = tid < tiles * kTileRows;
      float xv[G];
#pragma unroll
      for (int g = 0; g < G; ++g) {
        xv[g] = live ? xs[tid][g] : -INFINITY;
        float mx = xv[g];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
        if ((tid & 31) == 0) wred[warp][g] = mx;
      }
      consumer_sync(kConsumers);
      if (tid < G) {
        float mx = stat_m[tid];
        const float old = mx;
        for (int w = 0; w < kConsumers / 32; ++w) mx = fmaxf(mx, wred[w][tid]);
        stat_c[tid] = (old == -INFINITY) ? 0.f : exp2f(old - mx);
        stat_m[tid] = mx;
      }
      consumer_sync(kConsumers);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float pv = exp2f(xv[g] - stat_m[g]);
        if (live) xs[tid][g] = pv;
        float sum = pv;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if ((tid & 31) == 0) wred[warp][g] = sum;
      }
      consumer_sync(kConsumers);
      if (tid < G) {
        float sum = 0.f;
        for (int w = 0; w < kConsumers / 32; ++w) sum += wred[w][tid];
        stat_l[tid] = stat_l[tid] * stat_c[tid] + sum;
      }
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float c = stat_c[g];
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[g][e] *= c;
      }
    }
    // ---- phase B: acc[g][e] += p[row][g] * V[row][e]
    for (int k = 0; k < tiles; ++k, ++n) {
      if (ok) ok = ring.wait_full(n, abort_flag);
      if (!ok) continue;
      const T* tile = reinterpret_cast<const T*>(ring_buf + (n % kStages) * Ring::kTileBytes);
      RowF<T, EPL> raw[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int tr = r * kGroups + grp;
        if (k * kTileRows + tr < rows_here) raw[r].load_cached(tile + size_t(tr) * D + lane16 * EPL);
        else raw[r].zero();
      }
      __syncwarp();
      if ((tid & 31) == 0) ring.release(n);
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const int lr = k * kTileRows + r * kGroups + grp;
        float p[G];
#pragma unroll
        for (int g = 0; g < G; ++g) p[g] = (lr < rows_here) ? xs[lr][g] : 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
          const float vf = raw[r].get(e);
#pragma unroll
          for (int g = 0; g < G; ++g) o[g][e] = fmaf(p[g], vf, o[g][e]);
        }
      }
    }
    consumer_sync(kConsumers);   // xs is rewritten by the next round
  }
  if (*abort_flag) {   // uniform after the barrier above: some wait gave up, the result is not valid
    if (tid == 0) atomicCAS(status, 0, kStatusTimeout);   // keeps an earlier, more specific code
    return;
  }

  // the two 16-lane groups of a warp, then the warps, in a fixed order
  float(*red)[G][D] = reinterpret_cast<float(*)[G][D]>(ring_buf);   // the ring is drained: reuse it
  static_assert(sizeof(float) * (kConsumers / 32) * G * D <= size_t(Ring::kStages) * Ring::kTileBytes, "ring too small");
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
  consumer_sync(kConsumers);
  float* out = partial + size_t(base_slot + part_idx) * G * (D + 2);
  for (int i = tid; i < G * D; i += kConsumers) {
    const int g = i / D, d = i - g * D;
    float sum = 0.f;
#pragma unroll
    for (int w = 0; w < kConsumers / 32; ++w) sum += red[w][g][d];
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
                      int target, T* __restrict__ O) {
  constexpr int NW = kConsumers / 32;   // warp w merges partials w, w + NW, ...; a lane owns 4 outputs
  // The state words were written before the split kernel started (it triggered this launch only
  // after its own dependency wait had returned), so where this CTA's partials lie is worked out
  // while the split kernel is still streaming; only the partials themselves need the wait.
  const int g = blockIdx.x, u = blockIdx.y;
  const UnitView uv = load_unit(state, u, tail_cap);
  const int n_chunks = n_parts(uv.len(), target);
  const int base_slot = partial_base(state, u, target);
  pdl_wait();                 // the partials come from the split kernel
  pdl_launch_dependents();
  const int tid = threadIdx.x;
  if (tid >= kConsumers) return;
  const float* base = partial + size_t(base_slot) * G * (D + 2) + size_t(g) * (D + 2);
  const size_t stride = size_t(G) * (D + 2);
  const int warp = tid >> 5, lane = tid & 31;
  __shared__ float s_max[NW];
  __shared__ float s_acc[NW][D], s_l[NW];

  // One pass: warp w merges partials w, w + NW, ... with a running maximum (the loads do not
  // depend on it, so several partials are in flight), then the NW warp states are merged in
  // warp order.  Every partial holds at least one valid row, so its maximum is finite.
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  float l = 0.f, m = -INFINITY;
  const bool owns = lane * 4 < D;
#pragma unroll 4
  for (int c = warp; c < n_chunks; c += NW) {
    const float* p = base + c * stride;
    const float pm = p[D], pl = p[D + 1];
    float2 a = make_float2(0.f, 0.f), b = make_float2(0.f, 0.f);
    if (owns) {
      a = *reinterpret_cast<const float2*>(p + lane * 4);
      b = *reinterpret_cast<const float2*>(p + lane * 4 + 2);
    }
    const float m_new = fmaxf(m, pm);
    const float keep = exp2f(m - m_new);        // 0 for the first partial (m = -inf, m_new finite)
    const float w = exp2f(pm - m_new);
    l = fmaf(l, keep, pl * w);
    acc[0] = fmaf(acc[0], keep, a.x * w);
    acc[1] = fmaf(acc[1], keep, a.y * w);
    acc[2] = fmaf(acc[2], keep, b.x * w);
    acc[3] = fmaf(acc[3], keep, b.y * w);
    m = m_new;
  }
  if (owns) {
#pragma unroll
    for (int i = 0; i < 4; ++i) s_acc[warp][lane * 4 + i] = acc[i];
  }
  if (lane == 0) { s_l[warp] = l; s_max[warp] = m; }
  consumer_sync(kConsumers);
  if (tid < D) {
    float M = s_max[0];
#pragma unroll
    for (int w = 1; w < NW; ++w) M = fmaxf(M, s_max[w]);
    float a = 0.f, ls = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float wgt = (s_max[w] == -INFINITY) ? 0.f : exp2f(s_max[w] - M);   // a warp without partials
      a = fmaf(s_acc[w][tid], wgt, a);
      ls = fmaf(s_l[w], wgt, ls);
    }
    store_elt(O + (size_t(u) * G + g) * D + tid, n_chunks > 0 ? a / ls : 0.f);
  }
}

// Rows per CTA: enough CTAs for two per SM, at least one softmax round each.
inline int decode_target_rows(const tca_cache_desc* c, int64_t U, int ctas_per_sm, int64_t* n_slices_out) {
  int64_t total = 0, max_len = 0;
  for (int64_t u = 0; u < U; ++u) {
    const int64_t len = c->n_global[u] + c->n_tail[u];
    total += len;
    max_len = len > max_len ? len : max_len;
  }
  const int sms = sm_count();
  // Smallest slice length for which the slices of all units fit the resident CTAs in one
  // wave: with one slice more than that, the extra CTA starts only after another one ends.
  const int64_t slots = int64_t(ctas_per_sm) * sms;
  auto count = [&](int64_t target) {
    int64_t n = 0;
    for (int64_t u = 0; u < U; ++u) n += (c->n_global[u] + c->n_tail[u] + target - 1) / target;
    return n;
  };
  int64_t lo = (total + slots - 1) / slots, hi = max_len;
  if (lo < kSuperRows) lo = kSuperRows;
  if (hi < lo) hi = lo;
  if (count(lo) > slots) {
    while (lo < hi) {               // count() does not increase with target
      const int64_t mid = lo + (hi - lo) / 2;
      if (count(mid) <= slots) hi = mid; else lo = mid + 1;
    }
  }
  *n_slices_out = count(lo);   // CTAs of the attention kernel: one per slice
  return int(lo);
}

template <typename T, int D, int G>
int launch_decode(const tca_params* prm, const void* q, const tca_cache_desc* c, void* O, const DecodeWs& ws,
                  int64_t n_slices, int target, cudaStream_t stream) {
  using Ring = DecRing<T, D>;
  const int U = prm->batch * prm->n_kv_heads;
  const float scale_log2e = prm->sm_scale * 1.4426950408889634f;
  auto kern = decode_split_kernel<T, D, G>;
  TCA_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Ring::kSmemBytes));
  int st;
  if constexpr (sizeof(T) == 2) {
    st = launch_decode_mma<D>(prm, q, c, ws, n_slices, target, stream);   // tensor-pipe kernel for bf16
  } else {
    dim3 grid(static_cast<unsigned>(n_slices));   // one CTA per slice, none idle (see find_slice)
    kern<<<grid, kThreads, Ring::kSmemBytes, stream>>>(
        static_cast<const T*>(q), static_cast<const T*>(c->k), static_cast<const T*>(c->v), c->state,
        c->tail_cap, scale_log2e, target, ws.partial, ws.status, int(U));
    st = check_launch();
  }
  if (st != TCA_OK) return st;
  return launch_pdl(decode_combine_kernel<T, D, G>, dim3(G, unsigned(U)), dim3(kThreads), size_t(0), stream,
                    static_cast<const float*>(ws.partial), static_cast<const int64_t*>(c->state), c->tail_cap, target,
                    static_cast<T*>(O));
}

template <typename T, int D>
int dispatch_group(int G, const tca_params* prm, const void* q, const tca_cache_desc* c, void* O,
                   const DecodeWs& ws, int64_t n_slices, int target, cudaStream_t s) {
  switch (G) {
    case 1: return launch_decode<T, D, 1>(prm, q, c, O, ws, n_slices, target, s);
    case 2: return launch_decode<T, D, 2>(prm, q, c, O, ws, n_slices, target, s);
    case 3: return launch_decode<T, D, 3>(prm, q, c, O, ws, n_slices, target, s);
    case 4: return launch_decode<T, D, 4>(prm, q, c, O, ws, n_slices, target, s);
    case 5: return launch_decode<T, D, 5>(prm, q, c, O, ws, n_slices, target, s);
    case 6: return launch_decode<T, D, 6>(prm, q, c, O, ws, n_slices, target, s);
    case 7: return launch_decode<T, D, 7>(prm, q, c, O, ws, n_slices, target, s);
    case 8: return launch_decode<T, D, 8>(prm, q, c, O, ws, n_slices, target, s);
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
  int64_t n_slices = 0;
  const int target = decode_target_rows(c, U, prm->dtype == TCA_BF16 ? 1 : 2, &n_slices);
  TCA_CHECK_ARG(n_slices >= 1);
  const int G = prm->n_q_heads / prm->n_kv_heads;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (prm->dtype == TCA_BF16) {
    if (prm->head_dim == 128) return dispatch_group<__nv_bfloat16, 128>(G, prm, q, c, O, lay, n_slices, target, s);
    return dispatch_group<__nv_bfloat16, 64>(G, prm, q, c, O, lay, n_slices, target, s);
  }
  if (prm->head_dim == 128) return dispatch_group<float, 128>(G, prm, q, c, O, lay, n_slices, target, s);
  return dispatch_group<float, 64>(G, prm, q, c, O, lay, n_slices, target, s);
}

// ---------------------------------------------------------------------------------------
// Decode without any allocation: the split-KV partials live in a fixed array inside the
// library image instead of a caller-provided workspace.
namespace tca {
namespace {

constexpr size_t kStaticScratchBytes = size_t(TCA_DECODE_STATIC_SCRATCH_BYTES);

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
  int64_t n_slices = 0;
  const int target = decode_target_rows(c, U, prm->dtype == TCA_BF16 ? 1 : 2, &n_slices);
  TCA_CHECK_ARG(n_slices >= 1);
  const int G = prm->n_q_heads / prm->n_kv_heads;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (prm->dtype == TCA_BF16) {
    if (prm->head_dim == 128) return dispatch_group<__nv_bfloat16, 128>(G, prm, q, c, O, lay, n_slices, target, s);
    return dispatch_group<__nv_bfloat16, 64>(G, prm, q, c, O, lay, n_slices, target, s);
  }
  if (prm->head_dim == 128) return dispatch_group<float, 128>(G, prm, q, c, O, lay, n_slices, target, s);
  return dispatch_group<float, 64>(G, prm, q, c, O, lay, n_slices, target, s);
}

extern "C" int tca_decode_static_status(void* stream) {
  void* scratch = nullptr;
  int st = static_scratch(&scratch);
  if (st != TCA_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t word = 0;
  TCA_CHECK_CUDA(cudaMemcpyAsync(&word, scratch, sizeof(word), cudaMemcpyDeviceToHost, s));
  TCA_CHECK_CUDA(cudaStreamSynchronize(s));
  if (word == 0) return TCA_OK;
  TCA_CHECK_CUDA(cudaMemsetAsync(scratch, 0, sizeof(word), s));   // reported once: the word starts clean again
  TCA_CHECK_CUDA(cudaStreamSynchronize(s));
  return TCA_ERR_TIMEOUT;
}
