// Sparse causal prefill attention (Eq. 2, Algorithm 2 line 7) on the 5th-generation tensor
// cores: tcgen05.mma with fp32 accumulators in TMEM, operands staged by TMA with 128-byte
// swizzle, online softmax on the CUDA cores, bf16 inputs.
//
// One CTA owns 128 consecutive query positions of TWO query heads of one GQA group (same
// KV head, same positions, hence the same key tiles and the same mask), which halves the
// K/V traffic per flop and lets the tensor pipe work on one head while the other head's
// softmax runs.  Key tiles (128 keys) come from two ranges under one online softmax:
//   (1) the unit's selected keys in the cache's global region with position < c_hi, read
//       through a per-unit tensor map whose bound is the region's length, and
//   (2) the contiguous band [c_lo, i_last] of the original K/V,
// with c_i = min(max(0, i - w + 1), m*b); row i sees columns {pos < c_i} of (1) and
// {c_i <= j <= i} of (2), so every key is counted once.  Only tiles that straddle one of
// those bounds evaluate a mask.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = MMA issuer, warps 2-5 /
// 6-9 = softmax of head 0 / head 1 (one thread per query row = one TMEM lane).
// TMEM (512 columns): S0 | S1 | O0 | O1; the bf16 P of a tile overwrites the first half of its
// S columns and feeds the PV product straight from TMEM.  Shared memory: Q0 Q1 | 5-slot K/V ring.
// Per tile the issuer runs  PV0(t) S0(t+1) PV1(t) S1(t+1)  so that S of one head is being
// computed while the other head's softmax is in flight; the whole issuer warp executes the
// loop and an elected lane's tcgen05 instructions take effect (see umma_ss_elect).  O stays
// in TMEM and is rescaled lazily: only when a row maximum grew by more than 2^8 since the last
// rescale.  The softmax arithmetic uses the packed fp32x2 forms (fma, add) and the three-input
// max, which halves its issue slots.  CTAs are ordered unit-major so that the CTAs resident
// at one time read the same one or two KV heads out of L2.
//
// Every mbarrier wait is bounded; a wait that gives up raises the status word of the
// workspace, lets outstanding copies land, frees TMEM and returns.
#include <cuda.h>

#include <vector>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "tensor_map.cuh"

namespace tca {
namespace {

constexpr int BM = 128, BN = 128;
constexpr int kThreads = 320;
constexpr int kRing = 5;
constexpr int kHalfBytes = 128 * 128;  // 128 rows x 128 bytes (64 bf16): one swizzled box
constexpr float kRescaleThreshold = 8.f;
constexpr int kPChunks = 1;   // column chunks in which P is handed to the PV GEMM (2 and 4 measured no faster)

template <int D>
struct TcCfg {
  static constexpr int NH = D / 64;                 // 64-element halves per row
  static constexpr int kQ = NH * kHalfBytes;        // one head's Q tile
  static constexpr int kKV = NH * kHalfBytes;       // one K or V tile
  static constexpr int offQ = 0;
  static constexpr int offKV = 2 * kQ;
  static constexpr int offBar = offKV + kRing * kKV;
  static constexpr int bytes = offBar + 256 + 1024;  // + barriers/scalars + alignment slack
  static constexpr uint32_t colP(int h) { return uint32_t(h) * 128u; }   // bf16 P overwrites the first half of S
  static constexpr uint32_t colS(int h) { return uint32_t(h) * 128u; }
  static constexpr uint32_t colO(int h) { return 256u + uint32_t(h) * uint32_t(D); }
};

enum { BAR_Q = 0, BAR_FULL = 1, BAR_EMPTY = BAR_FULL + kRing, BAR_S = BAR_EMPTY + kRing, BAR_P = BAR_S + 2,
       BAR_PV = BAR_P + 2 * kPChunks, N_BARS = BAR_PV + 2 };

struct TileGeom {
  int n_gt, nt;
  int64_t c_lo;
  __device__ __forceinline__ bool is_global(int t) const { return t < n_gt; }
  __device__ __forceinline__ int64_t first(int t) const {  // first cache row / first position
    return t < n_gt ? int64_t(t) * BN : c_lo + int64_t(t - n_gt) * BN;
  }
};

__device__ __forceinline__ int lower_bound_pos(const int32_t* pos, int n, int64_t bound) {
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (int64_t(pos[mid]) < bound) lo = mid + 1; else hi = mid;
  }
  return lo;
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const CUtensorMap* __restrict__ maps, const int32_t* __restrict__ pos,
                  const int64_t* __restrict__ state, int64_t L, int n_q_heads, int n_kv_heads, int window,
                  int64_t mb, float scale_log2e, __nv_bfloat16* __restrict__ O, int* __restrict__ status,
                  int n_qtiles, int pairs_per_unit, int tile0) {
  using Cfg = TcCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::offBar);
  static_assert(N_BARS <= 24, "barrier block");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 24);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* s_nvis = reinterpret_cast<int*>(tmem_slot + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = n_q_heads / n_kv_heads;
  // Unit-major order: the CTAs resident at any time share one or two KV heads, whose retained
  // rows and window band then stay in L2; within a unit the long rows go first.
  const int per_unit = n_qtiles * pairs_per_unit;
  const int u = int(blockIdx.x) / per_unit;
  const int rem = int(blockIdx.x) % per_unit;
  const int tile = tile0 + n_qtiles - 1 - rem / pairs_per_unit;
  const int pair = rem % pairs_per_unit;
  const int nh = min(2, G - 2 * pair);                          // heads handled here
  const int seq = u / n_kv_heads, kvh = u % n_kv_heads;
  const int hq0 = seq * n_q_heads + kvh * G + 2 * pair;         // first query head (flattened over batch)

  const int64_t i0 = int64_t(tile) * BM;
  const int64_t i_last = min(i0 + BM - 1, L - 1);
  const int64_t* st = state + size_t(u) * TCA_STATE_WORDS;
  const int64_t seg = st[TCA_ST_SEG_START];
  const int n_global = int(st[TCA_ST_N_GLOBAL]);
  const int64_t c_lo = min(max(int64_t(0), i0 - window + 1), mb);
  const int64_t c_hi = min(max(int64_t(0), i_last - window + 1), mb);

  if (tid == 0) {
    ptx::mbar_init(&bars[BAR_Q], 1);
    for (int i = 0; i < kRing; ++i) { ptx::mbar_init(&bars[BAR_FULL + i], 1); ptx::mbar_init(&bars[BAR_EMPTY + i], 1); }
    for (int h = 0; h < 2; ++h) {
      ptx::mbar_init(&bars[BAR_S + h], 1);
      for (int c = 0; c < kPChunks; ++c) ptx::mbar_init(&bars[BAR_P + h * kPChunks + c], 128);
      ptx::mbar_init(&bars[BAR_PV + h], 1);
    }
    ptx::fence_barrier_init();
    *abort_flag = (*reinterpret_cast<volatile int*>(status) != 0) ? 1 : 0;
    *s_nvis = lower_bound_pos(pos + seg, n_global, c_hi);
  }
  if (warp == 0) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  TileGeom geo;
  geo.n_gt = (*s_nvis + BN - 1) / BN;
  geo.c_lo = c_lo;
  geo.nt = geo.n_gt + int((i_last - c_lo + BN) / BN);
  const int nt = geo.nt;

  if (!*abort_flag) {
    if (warp == 0) {
      // ------------------------------------------------------------- TMA producer
      if (lane == 0) {
        ptx::mbar_arrive_expect_tx(&bars[BAR_Q], uint32_t(nh * Cfg::kQ));
        for (int h = 0; h < nh; ++h)
          for (int half = 0; half < Cfg::NH; ++half)
            ptx::tma_load_3d(smem + Cfg::offQ + h * Cfg::kQ + half * kHalfBytes, &maps[0], half * 64, int(i0),
                             hq0 + h, &bars[BAR_Q]);
        for (int n = 0; n < 2 * nt; ++n) {
          const int t = n >> 1, is_v = n & 1, slot = n % kRing;
          if (n >= kRing && !ptx::mbar_wait(&bars[BAR_EMPTY + slot], uint32_t(n / kRing - 1) & 1u, abort_flag)) break;
          ptx::mbar_arrive_expect_tx(&bars[BAR_FULL + slot], uint32_t(Cfg::kKV));
          uint8_t* dst = smem + Cfg::offKV + slot * Cfg::kKV;
          const int y = int(geo.first(t));
          for (int half = 0; half < Cfg::NH; ++half) {
            if (geo.is_global(t))
              ptx::tma_load_2d(dst + half * kHalfBytes, &maps[3 + 2 * u + is_v], half * 64, y, &bars[BAR_FULL + slot]);
            else
              ptx::tma_load_3d(dst + half * kHalfBytes, &maps[1 + is_v], half * 64, y, u, &bars[BAR_FULL + slot]);
          }
        }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------- MMA issuer
      // The whole warp runs this loop; one elected lane issues (see umma_ss_elect).  Waits are
      // made warp-uniform so that the warp stays converged for elect.sync.
      {
        constexpr uint32_t idescS = ptx::idesc_bf16(BM, BN, false);
        constexpr uint32_t idescPV = ptx::idesc_bf16(BM, D, true);
        const uint32_t q_base = ptx::smem_u32(smem + Cfg::offQ);
        const uint32_t kv_base = ptx::smem_u32(smem + Cfg::offKV);
        // Descriptors differ only in their 14-bit start-address field (bytes >> 4) and every
        // operand lives below 256 KB, so a k-step or a ring slot is one add on the low word.
        const uint64_t dq = ptx::smem_desc_sw128(q_base, 16, 1024);
        const uint64_t dk = ptx::smem_desc_sw128(kv_base, 16, 1024);           // K tile as K-major B
        const uint64_t dv = ptx::smem_desc_sw128(kv_base, kHalfBytes, 1024);   // V tile as MN-major B
        auto wait = [&](uint64_t* bar, uint32_t parity) -> bool {
          return __all_sync(0xffffffffu, ptx::mbar_wait(bar, parity, abort_flag));
        };
        auto issue_S = [&](int h, int slot) {
          const uint64_t a0 = dq + uint64_t(uint32_t(h * Cfg::kQ) >> 4);
          const uint64_t b0 = dk + uint64_t(uint32_t(slot * Cfg::kKV) >> 4);
          const uint32_t d = tmem_base + Cfg::colS(h);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (uint32_t(kk >> 2) * kHalfBytes + uint32_t(kk & 3) * 32u) >> 4;
            ptx::umma_ss_elect(d, a0 + off, b0 + off, idescS, kk > 0);
          }
        };
        // O += P V with P read from TMEM (it overwrote the first 64 columns of S as packed bf16):
        // the A operand costs no shared-memory bandwidth.
        // P arrives in kPChunks column chunks, each with its own barrier, so the first k-steps of
        // PV run while the softmax warps are still exponentiating the rest of the row.
        auto issue_PV = [&](int h, int slot, bool acc, uint32_t parity) -> bool {
          const uint64_t b0 = dv + uint64_t(uint32_t(slot * Cfg::kKV) >> 4);
          const uint32_t d = tmem_base + Cfg::colO(h);
          const uint32_t a = tmem_base + Cfg::colP(h);
          constexpr int kPer = BN / 16 / kPChunks;
#pragma unroll
          for (int c = 0; c < kPChunks; ++c) {
            if (!wait(&bars[BAR_P + h * kPChunks + c], parity)) return false;
            ptx::tc_fence_after();
#pragma unroll
            for (int k2 = 0; k2 < kPer; ++k2) {
              const int kk = c * kPer + k2;
              ptx::umma_ts_elect(d, a + uint32_t(kk * 8), b0 + uint32_t((kk * 2048) >> 4), idescPV,
                                 (acc || kk > 0) ? 1u : 0u);
            }
          }
          return true;
        };
        bool ok = wait(&bars[BAR_Q], 0) && wait(&bars[BAR_FULL + 0], 0);
        if (ok) {
          ptx::tc_fence_after();
          for (int h = 0; h < nh; ++h) { issue_S(h, 0); ptx::umma_commit_elect(&bars[BAR_S + h]); }
          ptx::umma_commit_elect(&bars[BAR_EMPTY + 0]);
        }
        for (int t = 0; t < nt && ok; ++t) {
          const int nV = 2 * t + 1, slotV = nV % kRing;
          const int nK = 2 * t + 2, slotK = nK % kRing;
          const bool more = t + 1 < nt;
          // everything a head's block needs is waited for first, then PV_h(t) and S_h(t+1) go to
          // the tensor pipe back to back and the commits follow: nothing sits between the two
          // products on the chain S -> softmax -> PV -> S
          ok = wait(&bars[BAR_FULL + slotV], uint32_t(nV / kRing) & 1u) &&
               (!more || wait(&bars[BAR_FULL + slotK], uint32_t(nK / kRing) & 1u));
          for (int h = 0; h < nh && ok; ++h) {
            ok = issue_PV(h, slotV, t > 0, uint32_t(t) & 1u);
            if (!ok) break;
            if (more) issue_S(h, slotK);
            ptx::umma_commit_elect(&bars[more ? BAR_S + h : BAR_PV + h]);   // S ready implies PV done
            if (h == nh - 1) {
              ptx::umma_commit_elect(&bars[BAR_EMPTY + slotV]);
              if (more) ptx::umma_commit_elect(&bars[BAR_EMPTY + slotK]);
            }
          }
        }
      }
    } else {
      // ------------------------------------------------------------- softmax, one row per thread
      const int h = (warp - 2) >> 2;
      if (h < nh) {
        const int quarter = warp & 3;                    // TMEM lanes this warp may touch
        const int row = quarter * 32 + lane;
        const int64_t i = i0 + row;
        const int64_t c_i = min(max(int64_t(0), i - window + 1), mb);
        const int nvis_i = lower_bound_pos(pos + seg, n_global, c_i);
        const uint32_t lane_addr = tmem_base + (uint32_t(quarter * 32) << 16);
        float m_run = -INFINITY, m_used = -INFINITY, l = 0.f;
        bool ok = true;
        for (int t = 0; t < nt; ++t) {
          int lo, hi;
          if (geo.is_global(t)) { lo = 0; hi = nvis_i - 1 - t * BN; }
          else {
            const int64_t p0 = geo.first(t);
            lo = int(max(int64_t(-1), c_i - p0));
            hi = int(min(int64_t(BN), i - p0));
          }
          const bool masked = __any_sync(0xffffffffu, lo > 0 || hi < BN - 1);
          ok = ptx::mbar_wait(&bars[BAR_S + h], uint32_t(t) & 1u, abort_flag);
          if (!ok) break;
          ptx::tc_fence_after();
          // the whole row of S (128 fp32) into registers with one wait
          uint32_t v[BN];
#pragma unroll
          for (int c = 0; c < BN / 32; ++c)
            ptx::tmem_ld32(lane_addr + Cfg::colS(h) + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[c * 32]));
          ptx::tc_wait_ld();
          if (masked) {   // a masked score is -inf: it loses every max and its exponential is exactly 0
#pragma unroll
            for (int k = 0; k < BN; ++k)
              if (k < lo || k > hi) v[k] = 0xff800000u;
          }
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int k = 0; k < BN; k += 8) {
            mx4[0] = ptx::max3(mx4[0], __uint_as_float(v[k]), __uint_as_float(v[k + 1]));
            mx4[1] = ptx::max3(mx4[1], __uint_as_float(v[k + 2]), __uint_as_float(v[k + 3]));
            mx4[2] = ptx::max3(mx4[2], __uint_as_float(v[k + 4]), __uint_as_float(v[k + 5]));
            mx4[3] = ptx::max3(mx4[3], __uint_as_float(v[k + 6]), __uint_as_float(v[k + 7]));
          }
          const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
          m_run = fmaxf(m_run, mx * scale_log2e);
          // lazy rescale of the accumulator (warp-uniform decision: TMEM access is warp-wide)
          if (__any_sync(0xffffffffu, m_run > m_used + kRescaleThreshold)) {
            const float alpha = (m_used == -INFINITY) ? 0.f : ptx::fast_exp2(m_used - m_run);
            if (t > 0) {
#pragma unroll 1
              for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                ptx::tmem_ld32(lane_addr + Cfg::colO(h) + c * 32, o);
                ptx::tc_wait_ld();
#pragma unroll
                for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * alpha);
                ptx::tmem_st32(lane_addr + Cfg::colO(h) + c * 32, o);
              }
              ptx::tc_wait_st();
            }
            l *= alpha;
            m_used = m_run;
          }
          // p = exp2(s*scale - m), row sum, packed bf16 P back into TMEM over the S columns
          const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
          const uint64_t scale2 = ptx::pack2(scale_log2e, scale_log2e);
          const uint64_t neg_m2 = ptx::pack2(neg_m, neg_m);
          uint64_t sum2[2] = {0ull, 0ull};
          constexpr int kPairs = BN / 2 / kPChunks;   // packed bf16 words per chunk
#pragma unroll
          for (int c = 0; c < kPChunks; ++c) {
#pragma unroll
            for (int jj = 0; jj < kPairs; ++jj) {
              const int j = c * kPairs + jj;
              float xl, xh;
              ptx::unpack2(ptx::fma2(ptx::pack2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), scale2, neg_m2),
                           xl, xh);
              const float el = ptx::fast_exp2(xl), eh = ptx::fast_exp2(xh);
              sum2[j & 1] = ptx::add2(sum2[j & 1], ptx::pack2(el, eh));
              v[j] = ptx::pack_bf16x2(el, eh);   // entry j is never read again (j <= 2j)
            }
            ptx::tmem_st<kPairs>(lane_addr + Cfg::colP(h) + c * kPairs, &v[c * kPairs]);
            ptx::tc_wait_st();
            ptx::tc_fence_before();
            ptx::mbar_arrive(&bars[BAR_P + h * kPChunks + c]);
          }
          {
            float s0, s1, s2, s3;
            ptx::unpack2(sum2[0], s0, s1);
            ptx::unpack2(sum2[1], s2, s3);
            l += (s0 + s1) + (s2 + s3);
          }
        }
        // epilogue: O / l -> bf16 -> global
        if (ok) ok = ptx::mbar_wait(&bars[BAR_PV + h], 0, abort_flag);   // committed once, after the last PV
        if (ok) {
          ptx::tc_fence_after();
          const float inv = 1.f / l;
          __nv_bfloat16* orow = O + (size_t(hq0 + h) * L + size_t(i)) * D;
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t v[32];
            ptx::tmem_ld32(lane_addr + Cfg::colO(h) + c * 32, v);
            ptx::tc_wait_ld();
            if (i <= i_last) {
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                uint4 w;
                w.x = ptx::pack_bf16x2(__uint_as_float(v[q * 8 + 0]) * inv, __uint_as_float(v[q * 8 + 1]) * inv);
                w.y = ptx::pack_bf16x2(__uint_as_float(v[q * 8 + 2]) * inv, __uint_as_float(v[q * 8 + 3]) * inv);
                w.z = ptx::pack_bf16x2(__uint_as_float(v[q * 8 + 4]) * inv, __uint_as_float(v[q * 8 + 5]) * inv);
                w.w = ptx::pack_bf16x2(__uint_as_float(v[q * 8 + 6]) * inv, __uint_as_float(v[q * 8 + 7]) * inv);
                *reinterpret_cast<uint4*>(orow + c * 32 + q * 8) = w;
              }
            }
          }
        }
      }
    }
  }

  // ------------------------------------------------------------- teardown
  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    ptx::abort_teardown(status, tid);   // status word, then time for copies in flight to land
  }
  if (warp == 0) ptx::tmem_dealloc(tmem_base, 512);
}

// ------------------------------------------------------------------ host side
}  // namespace

size_t prefill_tc_ws_bytes(const tca_params* prm) {
  const size_t U = size_t(prm->batch) * prm->n_kv_heads;
  return 256 + (3 + 2 * U) * sizeof(CUtensorMap);
}

template <int D>
int launch_prefill_tc(const tca_params* prm, const void* Q, const void* K, const void* V, int64_t L,
                      int64_t row_begin, int64_t row_end, const tca_cache_desc* c, void* O, void* ws,
                      cudaStream_t stream) {
  using Cfg = TcCfg<D>;
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  const int G = prm->n_q_heads / prm->n_kv_heads;
  std::vector<CUtensorMap> maps(3 + 2 * U);
  bool ok = encode_map(&maps[0], Q, D, L, int64_t(prm->batch) * prm->n_q_heads, L) &&
            encode_map(&maps[1], K, D, L, U, L) && encode_map(&maps[2], V, D, L, U, L);
  for (int64_t u = 0; u < U && ok; ++u) {
    const char* kb = static_cast<const char*>(c->k) + size_t(c->seg_start[u]) * D * 2;
    const char* vb = static_cast<const char*>(c->v) + size_t(c->seg_start[u]) * D * 2;
    ok = encode_map(&maps[3 + 2 * u], kb, D, c->n_global[u], 0, 0) &&
         encode_map(&maps[4 + 2 * u], vb, D, c->n_global[u], 0, 0);
  }
  if (!ok) return TCA_ERR_CUDA;
  CUtensorMap* maps_dev = reinterpret_cast<CUtensorMap*>(static_cast<char*>(ws) + 256);
  // pageable source: staged by the runtime before the call returns
  TCA_CHECK_CUDA(cudaMemcpyAsync(maps_dev, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice,
                                 stream));
  auto kern = prefill_tc_kernel<D>;
  TCA_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::bytes));
  const int tile0 = int(row_begin / BM);
  const int n_qtiles = int((row_end - row_begin + BM - 1) / BM);
  const int pairs = (G + 1) / 2;
  const int64_t n_ctas = int64_t(n_qtiles) * U * pairs;
  if (n_ctas >= (int64_t(1) << 31)) return TCA_ERR_UNSUPPORTED;
  const int64_t mb = num_blocks(prm, L) * prm->block;
  kern<<<unsigned(n_ctas), kThreads, Cfg::bytes, stream>>>(
      maps_dev, c->pos, c->state, L, prm->n_q_heads, prm->n_kv_heads, prm->window, mb,
      prm->sm_scale * 1.4426950408889634f, static_cast<__nv_bfloat16*>(O), static_cast<int*>(ws), n_qtiles, pairs, tile0);
  return check_launch();
}

template int launch_prefill_tc<64>(const tca_params*, const void*, const void*, const void*, int64_t, int64_t,
                                   int64_t, const tca_cache_desc*, void*, void*, cudaStream_t);
template int launch_prefill_tc<128>(const tca_params*, const void*, const void*, const void*, int64_t, int64_t,
                                    int64_t, const tca_cache_desc*, void*, void*, cudaStream_t);

}  // namespace tca
