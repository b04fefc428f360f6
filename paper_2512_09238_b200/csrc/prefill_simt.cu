// Sparse causal prefill attention (Eq. 2, Algorithm 2 line 7) on the FP32 pipes.
//
// This is the path for fp32 inputs, whose 1e-4 tolerance rules out bf16/tf32 tensor-core
// products, and the reference kernel the tensor-core path is cross-checked against.
// One CTA owns 64 consecutive queries of one query head and walks two key ranges with a
// single online softmax: (1) the unit's selected keys in the cache's global region whose
// position is below the tile's window start, (2) the contiguous band of original keys
// [c_lo, i_last].  Per query i the visible set is {pos < c_i} in (1) and {c_i <= j <= i}
// in (2), c_i = min(max(0, i - w + 1), m*b), so every key is counted exactly once.
#include "common.cuh"
#include "rowslice.cuh"

namespace tca {

constexpr int kPfBM = 64, kPfBN = 64, kPfThreads = 256;

template <int D>
struct PfSmem {
  static constexpr int LD = D + 4;      // padded row (floats)
  static constexpr int LDP = kPfBN + 4;
  static constexpr size_t bytes = sizeof(float) * (3 * size_t(kPfBM) * LD + size_t(kPfBM) * LDP) + 1024;
};

namespace {

// first index in pos[0, n) with pos[idx] >= bound (pos ascending)
__device__ __forceinline__ int lower_bound_pos(const int32_t* pos, int n, int64_t bound) {
  int lo = 0, hi = n;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (int64_t(pos[mid]) < bound) lo = mid + 1; else hi = mid;
  }
  return lo;
}

template <typename T, int D>
__device__ __forceinline__ void load_tile_rows(float* dst, const T* src_base, const int64_t row0, int n_valid,
                                               float scale, int tid) {
  constexpr int LD = PfSmem<D>::LD;
  constexpr int EPV = 16 / sizeof(T);           // elements per 16-byte vector
  constexpr int VPR = D / EPV;                  // vectors per row
  for (int i = tid; i < kPfBN * VPR; i += kPfThreads) {
    const int r = i / VPR, c = (i - r * VPR) * EPV;
    float vals[EPV];
    if (r < n_valid) {
      const uint4 raw = *reinterpret_cast<const uint4*>(src_base + (row0 + r) * D + c);
      if constexpr (sizeof(T) == 4) {
        vals[0] = __uint_as_float(raw.x); vals[1] = __uint_as_float(raw.y);
        vals[2] = __uint_as_float(raw.z); vals[3] = __uint_as_float(raw.w);
      } else {
        vals[0] = bf16_lo(raw.x); vals[1] = bf16_hi(raw.x); vals[2] = bf16_lo(raw.y); vals[3] = bf16_hi(raw.y);
        vals[4] = bf16_lo(raw.z); vals[5] = bf16_hi(raw.z); vals[6] = bf16_lo(raw.w); vals[7] = bf16_hi(raw.w);
      }
    } else {
#pragma unroll
      for (int e = 0; e < EPV; ++e) vals[e] = 0.f;
    }
#pragma unroll
    for (int e = 0; e < EPV; ++e) dst[r * LD + c + e] = vals[e] * scale;
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kPfThreads)
prefill_simt_kernel(const T* __restrict__ Q, const T* __restrict__ K, const T* __restrict__ V, int64_t L,
                    const T* __restrict__ Kc, const T* __restrict__ Vc, const int32_t* __restrict__ pos,
                    const int64_t* __restrict__ state, int n_q_heads, int n_kv_heads, int window, int64_t mb,
                    float scale_log2e, T* __restrict__ O, int tile0) {
  constexpr int LD = PfSmem<D>::LD, LDP = PfSmem<D>::LDP;
  constexpr int NC = D / 64;  // 4-wide output column chunks per thread
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;
  float* Ks = Qs + kPfBM * LD;
  float* Vs = Ks + kPfBN * LD;
  float* Ps = Vs + kPfBN * LD;
  __shared__ int s_n_vis;

  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int hq = blockIdx.y;
  const int n_tiles = gridDim.x;
  const int tile = tile0 + n_tiles - 1 - blockIdx.x;  // longest rows first
  const int seq = hq / n_q_heads;
  const int G = n_q_heads / n_kv_heads;
  const int u = seq * n_kv_heads + (hq % n_q_heads) / G;
  const int64_t i0 = int64_t(tile) * kPfBM;
  const int n_q = int(min(int64_t(kPfBM), L - i0));
  const int64_t i_last = i0 + n_q - 1;

  const int64_t* st = state + size_t(u) * TCA_STATE_WORDS;
  const int64_t seg = st[TCA_ST_SEG_START];
  const int n_global = int(st[TCA_ST_N_GLOBAL]);
  const int64_t c_lo = min(max(int64_t(0), i0 - window + 1), mb);
  const int64_t c_hi = min(max(int64_t(0), i_last - window + 1), mb);
  if (tid == 0) s_n_vis = lower_bound_pos(pos + seg, n_global, c_hi);

  load_tile_rows<T, D>(Qs, Q + size_t(hq) * L * D, i0, n_q, scale_log2e, tid);

  // per-thread rows ty + 16*i, their window starts and running softmax state
  int64_t c_row[4], i_row[4];
  float m_run[4], l_run[4];
  float o[4][NC][4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    i_row[i] = i0 + ty + 16 * i;
    c_row[i] = min(max(int64_t(0), i_row[i] - window + 1), mb);
    m_run[i] = -INFINITY;
    l_run[i] = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c)
#pragma unroll
      for (int e = 0; e < 4; ++e) o[i][c][e] = 0.f;
  }
  __syncthreads();
  const int n_vis = s_n_vis;
  const int n_gt = (n_vis + kPfBN - 1) / kPfBN;
  const int64_t band_len = i_last - c_lo + 1;
  const int n_bt = int((band_len + kPfBN - 1) / kPfBN);

  for (int t = 0; t < n_gt + n_bt; ++t) {
    const bool is_global = t < n_gt;
    int n_valid;
    int64_t key0;  // first cache row (global) or first position (band) of the tile
    if (is_global) {
      key0 = int64_t(t) * kPfBN;
      n_valid = min(kPfBN, n_vis - int(key0));
      load_tile_rows<T, D>(Ks, Kc + size_t(seg) * D, key0, n_valid, 1.f, tid);
      load_tile_rows<T, D>(Vs, Vc + size_t(seg) * D, key0, n_valid, 1.f, tid);
    } else {
      key0 = c_lo + int64_t(t - n_gt) * kPfBN;
      n_valid = int(min(int64_t(kPfBN), i_last + 1 - key0));
      load_tile_rows<T, D>(Ks, K + size_t(u) * L * D, key0, n_valid, 1.f, tid);
      load_tile_rows<T, D>(Vs, V + size_t(u) * L * D, key0, n_valid, 1.f, tid);
    }
    // positions of this thread's four key columns tx + 16*j
    int64_t pj[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = tx + 16 * j;
      if (col < n_valid) pj[j] = is_global ? int64_t(pos[seg + key0 + col]) : key0 + col;
      else pj[j] = -1;
    }
    __syncthreads();

    // S = Q K^T for rows ty+16i, cols tx+16j
    float s[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
#pragma unroll 4
    for (int d = 0; d < D; d += 4) {
      float4 qv[4], kv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) qv[i] = *reinterpret_cast<const float4*>(Qs + (ty + 16 * i) * LD + d);
#pragma unroll
      for (int j = 0; j < 4; ++j) kv[j] = *reinterpret_cast<const float4*>(Ks + (tx + 16 * j) * LD + d);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          s[i][j] = fmaf(qv[i].x, kv[j].x, s[i][j]);
          s[i][j] = fmaf(qv[i].y, kv[j].y, s[i][j]);
          s[i][j] = fmaf(qv[i].z, kv[j].z, s[i][j]);
          s[i][j] = fmaf(qv[i].w, kv[j].w, s[i][j]);
        }
    }
    // mask, online softmax (rows are shared by the 16 lanes tx = 0..15 of a half warp)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float mx = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        bool vis = pj[j] >= 0 && i_row[i] <= i_last;
        if (is_global) vis = vis && pj[j] < c_row[i];
        else vis = vis && pj[j] >= c_row[i] && pj[j] <= i_row[i];
        s[i][j] = vis ? s[i][j] : -INFINITY;
        mx = fmaxf(mx, s[i][j]);
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      const float m_new = fmaxf(m_run[i], mx);
      const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
      const float corr = exp2f(m_run[i] - m_use);  // exp2(-inf) = 0 on the first visible tile
      float sum = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float p = exp2f(s[i][j] - m_use);
        Ps[(ty + 16 * i) * LDP + tx + 16 * j] = p;
        sum += p;
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
      l_run[i] = l_run[i] * corr + sum;
      m_run[i] = m_new;
#pragma unroll
      for (int c = 0; c < NC; ++c)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[i][c][e] *= corr;
    }
    __syncthreads();
    // O += P V for rows ty+16i, cols tx*4 + 64*c
#pragma unroll 2
    for (int k = 0; k < kPfBN; k += 4) {
      float4 pv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) pv[i] = *reinterpret_cast<const float4*>(Ps + (ty + 16 * i) * LDP + k);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        float4 vv[NC];
#pragma unroll
        for (int c = 0; c < NC; ++c) vv[c] = *reinterpret_cast<const float4*>(Vs + (k + kk) * LD + tx * 4 + 64 * c);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float p = kk == 0 ? pv[i].x : kk == 1 ? pv[i].y : kk == 2 ? pv[i].z : pv[i].w;
#pragma unroll
          for (int c = 0; c < NC; ++c) {
            o[i][c][0] = fmaf(p, vv[c].x, o[i][c][0]);
            o[i][c][1] = fmaf(p, vv[c].y, o[i][c][1]);
            o[i][c][2] = fmaf(p, vv[c].z, o[i][c][2]);
            o[i][c][3] = fmaf(p, vv[c].w, o[i][c][3]);
          }
        }
      }
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (i_row[i] > i_last) continue;
    const float inv = 1.f / l_run[i];
    T* orow = O + (size_t(hq) * L + i_row[i]) * D;
#pragma unroll
    for (int c = 0; c < NC; ++c)
#pragma unroll
      for (int e = 0; e < 4; ++e) store_elt(orow + tx * 4 + 64 * c + e, o[i][c][e] * inv);
  }
}

}  // namespace

template <typename T, int D>
int launch_prefill_simt(const tca_params* prm, const void* Q, const void* K, const void* V, int64_t L,
                        int64_t row_begin, int64_t row_end, const tca_cache_desc* c, void* O, cudaStream_t stream) {
  auto kern = prefill_simt_kernel<T, D>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(PfSmem<D>::bytes)) !=
      cudaSuccess)
    return TCA_ERR_CUDA;
  const int64_t mb = num_blocks(prm, L) * prm->block;
  const int tile0 = int(row_begin / kPfBM);
  dim3 grid(unsigned((row_end - row_begin + kPfBM - 1) / kPfBM), unsigned(prm->batch * prm->n_q_heads));
  kern<<<grid, kPfThreads, PfSmem<D>::bytes, stream>>>(
      static_cast<const T*>(Q), static_cast<const T*>(K), static_cast<const T*>(V), L,
      static_cast<const T*>(c->k), static_cast<const T*>(c->v), c->pos, c->state, prm->n_q_heads,
      prm->n_kv_heads, prm->window, mb, prm->sm_scale * 1.4426950408889634f, static_cast<T*>(O), tile0);
  return check_launch();
}

template int launch_prefill_simt<float, 64>(const tca_params*, const void*, const void*, const void*, int64_t,
                                            int64_t, int64_t, const tca_cache_desc*, void*, cudaStream_t);
template int launch_prefill_simt<float, 128>(const tca_params*, const void*, const void*, const void*, int64_t,
                                             int64_t, int64_t, const tca_cache_desc*, void*, cudaStream_t);
template int launch_prefill_simt<__nv_bfloat16, 64>(const tca_params*, const void*, const void*, const void*,
                                                    int64_t, int64_t, int64_t, const tca_cache_desc*, void*,
                                                    cudaStream_t);
template int launch_prefill_simt<__nv_bfloat16, 128>(const tca_params*, const void*, const void*, const void*,
                                                     int64_t, int64_t, int64_t, const tca_cache_desc*, void*,
                                                     cudaStream_t);

}  // namespace tca
