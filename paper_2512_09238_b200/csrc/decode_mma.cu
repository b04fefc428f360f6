// Split-KV decode for bf16 caches (Eq. 2, one query per head over the retained cache).
//
// The step is HBM-bound: 2 * d * 2 bytes per retained row and nothing else of size.  To
// keep the SMs out of the way the per-row arithmetic runs on the tensor pipe with
// mma.sync.m16n8k16 (the G <= 8 query heads of the group are the rows of a 16-row tile,
// padded with zeros): with one query token per head the tile is far too thin for
// tcgen05's 64-row minimum, and the warp-level MMA consumes bf16 straight from shared
// memory, which removes the conversion and FMA traffic that made a CUDA-core version
// issue-bound at a third of the bandwidth.
//
//   producer warp   streams 128-row K and V tiles of the CTA's slice through a shared-
//                   memory ring with TMA (2-D tensor map over the flattened cache,
//                   128-byte swizzle, no multicast); up to 192 KB in flight per SM.
//   8 consumer warps each own 16 rows of every tile and a private online softmax
//                   (max, sum, O[16 x d] accumulators in registers): S = Q K^T by
//                   ldmatrix + MMA, exp2, P reused as the A operand, O += P V by
//                   ldmatrix.trans + MMA.  No CTA-wide synchronisation per tile.
//   epilogue        the 8 private states are merged in warp order in shared memory and one
//                   un-normalised partial (acc, max, sum) per (slice, head) is written; the
//                   combine kernel of decode.cu merges slices in slice order.
#include <cuda.h>

#include <mutex>

#include "bulk_ring.cuh"
#include "common.cuh"
#include "decode_common.cuh"
#include "ptx_sm100.cuh"

namespace tca {
namespace {

constexpr int kMmaConsumers = 256;
constexpr int kMmaThreads = kMmaConsumers + 32;
constexpr int kMmaTileRows = 128;
// Part of the L2 that cache tiles are asked to stay in from one decode step to the next.  Measured
// at 229 MB of cache on a 126 MB L2: the step is fastest with 50-70 MB resident and no better than
// without hints from 115 MB up, so a little under half of the L2 is asked for.
constexpr double kL2Share = 0.45;
constexpr int kBoxBytes = kMmaTileRows * 128;   // 128 rows x 64 bf16

template <int D>
struct MmaRing {
  static constexpr int kTileBytes = (D / 64) * kBoxBytes;
  static constexpr int kStages = (192 * 1024) / kTileBytes > 8 ? 8 : (192 * 1024) / kTileBytes;
  static constexpr int kSmemBytes = kStages * kTileBytes + 1024;
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Byte offset of the 16-byte chunk (row, chunk16) inside a swizzled tile of D/64 boxes.
template <int D>
__device__ __forceinline__ uint32_t swz(int row, int chunk16) {
  const int box = chunk16 >> 3, c = chunk16 & 7;
  return uint32_t(box) * kBoxBytes + uint32_t(row) * 128u + (uint32_t(c ^ (row & 7)) << 4);
}

template <int D>
__global__ void __launch_bounds__(kMmaThreads, 1)
decode_mma_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                  const __nv_bfloat16* __restrict__ q, const int64_t* __restrict__ state, int64_t tail_cap,
                  int G, float scale_log2e, int target, float* __restrict__ partial, int* __restrict__ status,
                  int l2_keep, int n_units) {
  using Ring = MmaRing<D>;
  constexpr int kStages = Ring::kStages;
  constexpr int ND = D / 8;     // n8 tiles across the head dimension
  constexpr int KC = D / 16;    // k16 chunks across the head dimension
  extern __shared__ uint8_t dmma_smem_raw[];
  uint8_t* ring_buf = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(dmma_smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ BulkRing<kStages> ring;
  __shared__ int abort_word;
  __shared__ SliceId slice_slot;
  __shared__ float s_m[kMmaConsumers / 32][kMaxGroup], s_l[kMmaConsumers / 32][kMaxGroup];
  volatile int* abort_flag = &abort_word;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // Set-up that reads nothing the previous kernel wrote runs before the dependency wait.
  if (tid == 0) {
    ring.init(kMmaConsumers / 32);
    abort_word = 0;
    ptx::tma_prefetch_desc(&map_k);
    ptx::tma_prefetch_desc(&map_v);
  }
  __syncthreads();
  pdl_wait();                 // the cache state and rows come from the kernels before this one
  pdl_launch_dependents();
  const SliceId slice = find_slice(state, n_units, target, tail_cap, &slice_slot);
  if (slice.u < 0) return;
  const int u = slice.u, part_idx = slice.part, np = slice.np;
  const UnitView uv = slice.uv;
  const int64_t len = uv.len();
  const int64_t row0 = slice_begin(len, np, part_idx);
  const int n_rows = int(slice_begin(len, np, part_idx + 1) - row0);

  if (warp == kMmaConsumers / 32) {
    // ------------------------------------------------------------- producer
    if (lane == 0) {
      int n = 0, done = 0;
      // The cache is read again by the next step, and its rows stay where they are: l2_keep of every
      // 64 tiles (by address, hence the same ones every step) ask to stay in L2, the others to be
      // evicted first, so that the part of the cache that fits keeps being served from L2 instead of
      // the whole of it sweeping through.  The choice goes by the bit-reversed tile index, which
      // spreads the resident tiles evenly (every fourth tile for a quarter), so that every CTA's
      // slice holds the same share of them and the CTAs keep finishing together.
      const uint64_t pol_keep = ptx::l2_policy_evict_last(), pol_stream = ptx::l2_policy_evict_first();
      while (done < n_rows) {
        const int64_t r = row0 + done;
        const int cnt = int(min(int64_t(kMmaTileRows), uv.run(r, n_rows - done)));
        const int y = int(uv.phys(r));
        if constexpr (kDebugBounds) {
          // the tile must lie inside the unit's segment (the tensor map bounds the whole cache only)
          if (y < uv.seg || int64_t(y) + cnt > uv.seg + uv.gcap + uv.tail_cap) {
            report_bounds_ws(status, kBoundsCacheRow, y);
            *abort_flag = 1;   // the consumers leave their waits; nothing is copied
            return;
          }
        }
        for (int kv = 0; kv < 2; ++kv, ++n) {
          if (!ring.acquire(n, uint32_t(Ring::kTileBytes), abort_flag)) return;
          uint8_t* dst = ring_buf + (n % kStages) * Ring::kTileBytes;
          for (int box = 0; box < D / 64; ++box)
            ptx::tma_load_2d_hint(dst + box * kBoxBytes, kv ? &map_v : &map_k, box * 64, y, &ring.full[n % kStages],
                                  (int(__brev(unsigned(y >> 7)) >> 26) < l2_keep) ? pol_keep : pol_stream);
        }
        done += cnt;
      }
    }
    return;
  }

  // --------------------------------------------------------------- consumers
  const int base_slot = slice.base_slot;
  const int gq = lane >> 2, kq = (lane & 3) * 2;   // accumulator row (query head) and column pair
  // Q as the A operand, one k16 chunk of the head dimension per entry (rows >= G are zero)
  uint32_t qa[KC][2];
#pragma unroll
  for (int c = 0; c < KC; ++c) {
    qa[c][0] = qa[c][1] = 0u;
    if (gq < G) {
      const __nv_bfloat16* qp = q + (size_t(u) * G + gq) * D + c * 16 + kq;
      qa[c][0] = *reinterpret_cast<const uint32_t*>(qp);
      qa[c][1] = *reinterpret_cast<const uint32_t*>(qp + 8);
    }
  }
  float o[ND][4];
#pragma unroll
  for (int j = 0; j < ND; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
  float m_run = -INFINITY, l_run = 0.f;

  const uint32_t ring_base = ptx::smem_u32(ring_buf);
  // per-lane ldmatrix source rows/chunks
  const int ld_mi = lane >> 3, ld_rr = lane & 7;
  const int k_row = warp * 16 + (ld_mi >> 1) * 8 + ld_rr;   // K: matrices (keys lo, d lo) (keys lo, d hi) (keys hi, d lo) (keys hi, d hi)
  const int k_chunk = ld_mi & 1;
  const int v_row = warp * 16 + (ld_mi & 1) * 8 + ld_rr;    // V^T: (keys lo, d j) (keys hi, d j) (keys lo, d j+1) (keys hi, d j+1)
  const int v_chunk = ld_mi >> 1;

  int n = 0, done = 0;
  bool ok = true;
  while (done < n_rows) {
    const int64_t r = row0 + done;
    const int cnt = int(min(int64_t(kMmaTileRows), uv.run(r, n_rows - done)));
    const int my_rows = min(16, cnt - warp * 16);    // valid rows of this warp's 16 (may be <= 0)
    // ---- S = Q K^T for this warp's 16 keys: two n8 tiles
    float s[2][4];
#pragma unroll
    for (int t = 0; t < 2; ++t) s[t][0] = s[t][1] = s[t][2] = s[t][3] = 0.f;
    if (ok) ok = ring.wait_full(n, abort_flag);
    if (ok && my_rows > 0) {
      const uint32_t kt = ring_base + (n % kStages) * Ring::kTileBytes;
#pragma unroll
      for (int c = 0; c < KC; ++c) {
        uint32_t b[4];
        ldmatrix_x4(b, kt + swz<D>(k_row, c * 2 + k_chunk));
        const uint32_t a[4] = {qa[c][0], 0u, qa[c][1], 0u};
        mma_bf16(s[0], a, b[0], b[1]);
        mma_bf16(s[1], a, b[2], b[3]);
      }
    }
    __syncwarp();
    if (lane == 0) ring.release(n);
    ++n;
    // ---- online softmax on rows gq < G (columns kq, kq+1 of each n8 tile)
    uint32_t pa[4] = {0u, 0u, 0u, 0u};
    float corr = 1.f;
    if (my_rows > 0) {
      float x[4];
      float mx = -INFINITY;
#pragma unroll
      for (int t = 0; t < 2; ++t)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int key = t * 8 + kq + e;
          x[t * 2 + e] = (key < my_rows) ? s[t][e] * scale_log2e : -INFINITY;
          mx = fmaxf(mx, x[t * 2 + e]);
        }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run, mx);       // finite: key 0 of the warp's rows is valid
      corr = exp2f(m_run - m_new);                // 0 on the first tile
      float p[4], sum = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) { p[i] = exp2f(x[i] - m_new); sum += p[i]; }
      sum += __shfl_xor_sync(0xffffffffu, sum, 1);
      sum += __shfl_xor_sync(0xffffffffu, sum, 2);
      l_run = l_run * corr + sum;
      m_run = m_new;
      pa[0] = ptx::pack_bf16x2(p[0], p[1]);       // keys kq, kq+1
      pa[2] = ptx::pack_bf16x2(p[2], p[3]);       // keys 8+kq, 8+kq+1
    }
    // ---- O = O * corr + P V
    if (ok) ok = ring.wait_full(n, abort_flag);
    if (ok && my_rows > 0) {
      const uint32_t vt = ring_base + (n % kStages) * Ring::kTileBytes;
#pragma unroll
      for (int j = 0; j < ND; j += 2) {
        uint32_t b[4];
        ldmatrix_x4_trans(b, vt + swz<D>(v_row, j + v_chunk));
        o[j][0] *= corr; o[j][1] *= corr;
        o[j + 1][0] *= corr; o[j + 1][1] *= corr;
        mma_bf16(o[j], pa, b[0], b[1]);
        mma_bf16(o[j + 1], pa, b[2], b[3]);
      }
    }
    __syncwarp();
    if (lane == 0) ring.release(n);
    ++n;
    done += cnt;
  }

  // --------------------------------------------------------------- merge the 8 warp states, write the partial
  consumer_sync(kMmaConsumers);                     // the ring is drained: reuse it as scratch
  float* red = reinterpret_cast<float*>(ring_buf);  // [warp][G][D]
  if (gq < G) {
#pragma unroll
    for (int j = 0; j < ND; ++j) {
      red[(size_t(warp) * G + gq) * D + j * 8 + kq] = o[j][0];
      red[(size_t(warp) * G + gq) * D + j * 8 + kq + 1] = o[j][1];
    }
    if ((lane & 3) == 0) { s_m[warp][gq] = m_run; s_l[warp][gq] = l_run; }
  }
  consumer_sync(kMmaConsumers);
  if (*abort_flag) {
    if (tid == 0) atomicCAS(status, 0, kStatusTimeout);   // keeps an earlier, more specific code
    return;
  }
  float* out = partial + size_t(base_slot + part_idx) * G * (D + 2);
  for (int i = tid; i < G * D; i += kMmaConsumers) {
    const int g = i / D, d = i - g * D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kMmaConsumers / 32; ++w) M = fmaxf(M, s_m[w][g]);
    float acc = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < kMmaConsumers / 32; ++w) {
      const float wgt = (s_m[w][g] == -INFINITY) ? 0.f : exp2f(s_m[w][g] - M);
      acc = fmaf(red[(size_t(w) * G + g) * D + d], wgt, acc);
      l = fmaf(s_l[w][g], wgt, l);
    }
    out[size_t(g) * (D + 2) + d] = acc;
    if (d == 0) {
      out[size_t(g) * (D + 2) + D] = M;
      out[size_t(g) * (D + 2) + D + 1] = l;
    }
  }
}

// ------------------------------------------------------------------ host side: tensor maps over the cache
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct CachedMap {
  const void* base = nullptr;
  int64_t rows = 0;
  int D = 0;
  CUtensorMap map;
};
std::mutex g_map_mutex;
CachedMap g_maps[8];
int g_map_next = 0;

bool cache_map(const void* base, int64_t rows, int D, CUtensorMap* out) {
  std::lock_guard<std::mutex> lock(g_map_mutex);
  for (const CachedMap& m : g_maps)
    if (m.base == base && m.rows == rows && m.D == D) { *out = m.map; return true; }
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return false;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  CachedMap& slot = g_maps[g_map_next];
  g_map_next = (g_map_next + 1) % 8;
  cuuint64_t dims[2] = {cuuint64_t(D), cuuint64_t(rows)};
  cuuint64_t strides[1] = {cuuint64_t(D) * 2};
  cuuint32_t box[2] = {64, cuuint32_t(kMmaTileRows)};
  cuuint32_t estr[2] = {1, 1};
  if (fn(&slot.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
    slot.base = nullptr;
    return false;
  }
  slot.base = base;
  slot.rows = rows;
  slot.D = D;
  *out = slot.map;
  return true;
}

}  // namespace

template <int D>
int launch_decode_mma(const tca_params* prm, const void* q, const tca_cache_desc* c, const DecodeWs& ws,
                      int64_t n_slices, int target, cudaStream_t stream) {
  using Ring = MmaRing<D>;
  CUtensorMap mk, mv;
  if (!cache_map(c->k, c->rows_total, D, &mk) || !cache_map(c->v, c->rows_total, D, &mv)) return TCA_ERR_CUDA;
  const int U = prm->batch * prm->n_kv_heads;
  const int G = prm->n_q_heads / prm->n_kv_heads;
  // Share of the cache asked to stay in L2 between steps, in 64ths: what fits kL2Share of the L2.
  int64_t rows = 0;
  for (int u = 0; u < U; ++u) rows += c->n_global[u] + c->n_tail[u];
  const double cache_bytes = double(rows) * D * 2 * 2;            // K and V, bf16
  const double keep = cache_bytes > 0 ? kL2Share * double(l2_bytes()) / cache_bytes : 1.0;
  const int l2_keep = keep >= 1.0 ? 64 : int(keep * 64.0 + 0.5);
  auto kern = decode_mma_kernel<D>;
  TCA_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Ring::kSmemBytes));
  dim3 grid(static_cast<unsigned>(n_slices));   // one CTA per slice, none idle (see find_slice)
  return launch_pdl(kern, grid, dim3(kMmaThreads), size_t(Ring::kSmemBytes), stream, mk, mv,
                    static_cast<const __nv_bfloat16*>(q), static_cast<const int64_t*>(c->state), c->tail_cap, G,
                    prm->sm_scale * 1.4426950408889634f, target, ws.partial, ws.status, l2_keep, U);
}

template int launch_decode_mma<64>(const tca_params*, const void*, const tca_cache_desc*, const DecodeWs&, int64_t,
                                   int, cudaStream_t);
template int launch_decode_mma<128>(const tca_params*, const void*, const tca_cache_desc*, const DecodeWs&, int64_t,
                                    int, cudaStream_t);

}  // namespace tca
