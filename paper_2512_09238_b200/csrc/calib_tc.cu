// Offline calibration (Algorithm 1): the column means of the causal attention map that Eq. 4
// sums over a selected set, on the 5th-generation tensor cores.
//
//   c[k] = 1/(G (L-k)) * sum_g sum_{j >= k} exp2(q_{g,j}.k_k * scale*log2e - lse2_{g,j})
//
// Pass 1 computes the log-sum-exp of every query row (a tile of 128 queries stationary, the key
// tiles before it streamed).  Pass 2 keeps a tile of
// 128 keys stationary as the A operand and streams the query tiles at or after it as B:
// S^T = K_tile Q_tile^T lands in TMEM with one key per lane, and the thread that owns the
// lane exponentiates its 128 scores against the queries' log-sum-exps and adds them up.
// Nothing is multiplied by V and no running maximum is needed (every term is a probability).
//
// Warp roles (320 threads): warp 0 = TMA producer (the K tile once, then a ring of Q tiles,
// each followed by the 128 log-sum-exps of its rows), warp 1 = MMA issuer, warps 2-5 / 6-9 =
// the summing warps of chain 0 / chain 1.  The two chains work on two query heads of the
// group at the same query tile; a chain's S buffer is free again as soon as its 128 scores
// sit in registers, so the tensor pipe runs ahead of the exponentials, which are the limit
// (128 x 128 ex2 at 16 per clock = 1024 clocks per tile against 512 for the product).
// The heads of the group are taken pair after pair inside the CTA and the (L - k) rows of a
// column are visited in a fixed order, so the result is reproducible bit for bit.
//
// Every mbarrier wait is bounded; a wait that gives up raises the status word of the
// workspace, lets outstanding copies land, frees TMEM and returns.
#include <cuda.h>

#include <cmath>
#include <vector>

#include "bulk_ring.cuh"
#include "common.cuh"
#include "ptx_sm100.cuh"
#include "tensor_map.cuh"

namespace tca {

namespace {

constexpr int CT = 128;                  // keys per CTA and queries per tile
constexpr int kColThreads = 320;
constexpr int kQRing = 5;
constexpr int kColHalfBytes = 128 * 128;  // 128 rows x 128 bytes (64 bf16): one swizzled box

template <int D>
struct ColCfg {
  static constexpr int NH = D / 64;
  static constexpr int kTile = NH * kColHalfBytes;   // one K or Q tile
  static constexpr int kSlot = kTile + 1024;         // Q tile + the 128 negated log-sum-exps of its rows
  static constexpr int offK = 0;
  static constexpr int offRing = kTile;
  static constexpr int offBar = offRing + kQRing * kSlot;
  static constexpr int bytes = offBar + 256 + 1024;  // + barriers/scalars + alignment slack
};

enum { CB_K = 0, CB_FULL = 1, CB_EMPTY = CB_FULL + kQRing, CB_S = CB_EMPTY + kQRing, CB_FREE = CB_S + 2,
       CN_BARS = CB_FREE + 2 };

// ------------------------------------------------------------------ pass 1: row statistics
// For every query row of every head: minus the log2 of the causal softmax denominator in the
// units of the scaled scores, -(m + log2 sum_j exp2(s_j * scale - m)).  A tile of 128 queries
// of two heads of the group stays in shared memory as the A operands of two chains; the key
// tiles 0..qt stream through a ring and each feeds both chains (S_c = Q_c K_tile^T, one
// query per TMEM lane).  The lane's thread keeps a running reference maximum (moved only when
// a tile's maximum exceeds it by more than 2^8, the sum is rescaled then) and adds up the
// exponentials.  No V, no P, no O: a chain's S buffer is free once its scores are in registers.
template <int D>
struct RowCfg {
  static constexpr int NH = D / 64;
  static constexpr int kTile = NH * kColHalfBytes;   // one Q or K tile
  static constexpr int offQ = 0;                     // two Q tiles
  static constexpr int offRing = 2 * kTile;
  static constexpr int offBar = offRing + kQRing * kTile;
  static constexpr int bytes = offBar + 256 + 1024;
};

enum { RB_Q = 0, RB_QFREE = 1, RB_FULL = 2, RB_EMPTY = RB_FULL + kQRing, RB_S = RB_EMPTY + kQRing, RB_FREE = RB_S + 2,
       RN_BARS = RB_FREE + 2 };

template <int D>
__global__ void __launch_bounds__(kColThreads, 1)
calib_rowstats_kernel(const CUtensorMap* __restrict__ maps, float* __restrict__ neg_lse, int64_t lse_stride, int64_t L,
                      int n_q_heads, int n_kv_heads, float scale_log2e, int* __restrict__ status, int n_tiles) {
  using Cfg = RowCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::offBar);
  static_assert(RN_BARS <= 24, "barrier block");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 24);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = n_q_heads / n_kv_heads;
  const int u = int(blockIdx.x) / n_tiles;
  const int qt = n_tiles - 1 - int(blockIdx.x) % n_tiles;   // the longest rows go first
  const int seq = u / n_kv_heads, kvh = u % n_kv_heads;
  const int head0 = seq * n_q_heads + kvh * G;
  const int nk = qt + 1;                                     // key tiles 0 .. qt
  const int n_pairs = (G + 1) / 2;

  if (tid == 0) {
    ptx::mbar_init(&bars[RB_Q], 1);
    ptx::mbar_init(&bars[RB_QFREE], 1);
    for (int i = 0; i < kQRing; ++i) {
      ptx::mbar_init(&bars[RB_FULL + i], 1);
      ptx::mbar_init(&bars[RB_EMPTY + i], 1);
    }
    for (int c = 0; c < 2; ++c) {
      ptx::mbar_init(&bars[RB_S + c], 1);
      ptx::mbar_init(&bars[RB_FREE + c], 128);
    }
    ptx::fence_barrier_init();
    *abort_flag = (*reinterpret_cast<volatile int*>(status) != 0) ? 1 : 0;
  }
  if (warp == 0) {
    ptx::tmem_alloc(tmem_slot, 256);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (!*abort_flag) {
    if (warp == 0) {
      // ------------------------------------------------------------- TMA producer
      if (lane == 0) {
        int jj = 0;
        bool ok = true;
        for (int pair = 0; pair < n_pairs && ok; ++pair) {
          const int nh = min(2, G - 2 * pair);
          // the previous pair's products must have finished reading the Q tiles
          if (pair > 0 && !ptx::mbar_wait(&bars[RB_QFREE], uint32_t(pair - 1) & 1u, abort_flag)) break;
          ptx::mbar_arrive_expect_tx(&bars[RB_Q], uint32_t(nh * Cfg::kTile));
          for (int c = 0; c < nh; ++c)
            for (int half = 0; half < Cfg::NH; ++half)
              ptx::tma_load_3d(smem + Cfg::offQ + c * Cfg::kTile + half * kColHalfBytes, &maps[0], half * 64, qt * CT,
                               head0 + 2 * pair + c, &bars[RB_Q]);
          for (int kt = 0; kt < nk; ++kt, ++jj) {
            const int slot = jj % kQRing;
            if (jj >= kQRing && !ptx::mbar_wait(&bars[RB_EMPTY + slot], uint32_t(jj / kQRing - 1) & 1u, abort_flag)) {
              ok = false;
              break;
            }
            ptx::mbar_arrive_expect_tx(&bars[RB_FULL + slot], uint32_t(Cfg::kTile));
            for (int half = 0; half < Cfg::NH; ++half)
              ptx::tma_load_3d(smem + Cfg::offRing + slot * Cfg::kTile + half * kColHalfBytes, &maps[1], half * 64,
                               kt * CT, u, &bars[RB_FULL + slot]);
          }
        }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------- MMA issuer (whole warp, elected lane)
      {
        constexpr uint32_t idesc = ptx::idesc_bf16(CT, CT, false);
        const uint64_t dq = ptx::smem_desc_sw128(ptx::smem_u32(smem + Cfg::offQ), 16, 1024);      // queries as A
        const uint64_t dk = ptx::smem_desc_sw128(ptx::smem_u32(smem + Cfg::offRing), 16, 1024);   // keys as B
        auto wait = [&](uint64_t* bar, uint32_t parity) -> bool {
          return __all_sync(0xffffffffu, ptx::mbar_wait(bar, parity, abort_flag));
        };
        int jj = 0;
        uint32_t done[2] = {0u, 0u};
        bool ok = true;
        for (int pair = 0; pair < n_pairs && ok; ++pair) {
          const int nh = min(2, G - 2 * pair);
          ok = wait(&bars[RB_Q], uint32_t(pair) & 1u);
          for (int kt = 0; kt < nk && ok; ++kt, ++jj) {
            const int slot = jj % kQRing;
            ok = wait(&bars[RB_FULL + slot], uint32_t(jj / kQRing) & 1u);
            for (int c = 0; c < nh && ok; ++c) {
              ok = done[c] == 0 || wait(&bars[RB_FREE + c], (done[c] - 1) & 1u);
              if (!ok) break;
              ptx::tc_fence_after();
              const uint64_t a0 = dq + uint64_t(uint32_t(c * Cfg::kTile) >> 4);
              const uint64_t b0 = dk + uint64_t(uint32_t(slot * Cfg::kTile) >> 4);
              const uint32_t d = tmem_base + uint32_t(c) * CT;
#pragma unroll
              for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = (uint32_t(kk >> 2) * kColHalfBytes + uint32_t(kk & 3) * 32u) >> 4;
                ptx::umma_ss_elect(d, a0 + off, b0 + off, idesc, kk > 0);
              }
              ptx::umma_commit_elect(&bars[RB_S + c]);
              ++done[c];
            }
            if (ok) ptx::umma_commit_elect(&bars[RB_EMPTY + slot]);
          }
          if (ok) ptx::umma_commit_elect(&bars[RB_QFREE]);
        }
      }
    } else {
      // ------------------------------------------------------------- one query row per thread
      const int c = (warp - 2) >> 2;
      const int quarter = warp & 3;
      const int r = quarter * 32 + lane;
      const int64_t i = int64_t(qt) * CT + r;
      const uint32_t lane_addr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(c) * CT;
      const uint64_t scale2 = ptx::pack2(scale_log2e, scale_log2e);
      uint32_t done = 0;
      bool ok = true;
      for (int pair = 0; pair < n_pairs && ok; ++pair) {
        if (2 * pair + c >= G) break;                        // uniform for the chain's four warps
        float m_run = -INFINITY, m_used = -INFINITY, l = 0.f;
        for (int kt = 0; kt < nk; ++kt) {
          ok = __all_sync(0xffffffffu, ptx::mbar_wait(&bars[RB_S + c], done & 1u, abort_flag));
          if (!ok) break;
          ++done;
          ptx::tc_fence_after();
          uint32_t v[CT];
#pragma unroll
          for (int q4 = 0; q4 < CT / 32; ++q4)
            ptx::tmem_ld32(lane_addr + q4 * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[q4 * 32]));
          ptx::tc_wait_ld();
          ptx::tc_fence_before();
          ptx::mbar_arrive(&bars[RB_FREE + c]);              // the scores are in registers
          if (kt == qt) {                                     // diagonal tile: keys after the query are masked
#pragma unroll
            for (int k = 0; k < CT; ++k)
              if (k > r) v[k] = 0xff800000u;
          }
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int k = 0; k < CT; k += 8) {
            mx4[0] = ptx::max3(mx4[0], __uint_as_float(v[k]), __uint_as_float(v[k + 1]));
            mx4[1] = ptx::max3(mx4[1], __uint_as_float(v[k + 2]), __uint_as_float(v[k + 3]));
            mx4[2] = ptx::max3(mx4[2], __uint_as_float(v[k + 4]), __uint_as_float(v[k + 5]));
            mx4[3] = ptx::max3(mx4[3], __uint_as_float(v[k + 6]), __uint_as_float(v[k + 7]));
          }
          m_run = fmaxf(m_run, fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2e);
          if (m_run > m_used + 8.f) {                         // key 0 is visible to every row: m_run is finite
            l *= (m_used == -INFINITY) ? 0.f : ptx::fast_exp2(m_used - m_run);
            m_used = m_run;
          }
          const uint64_t neg_m2 = ptx::pack2(-m_used, -m_used);
          uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
          for (int j = 0; j < CT / 2; ++j) {
            float xl, xh;
            ptx::unpack2(ptx::fma2(ptx::pack2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), scale2, neg_m2),
                         xl, xh);
            sum2[j & 1] = ptx::add2(sum2[j & 1], ptx::pack2(ptx::fast_exp2(xl), ptx::fast_exp2(xh)));
          }
          float s0, s1, s2, s3;
          ptx::unpack2(sum2[0], s0, s1);
          ptx::unpack2(sum2[1], s2, s3);
          l += (s0 + s1) + (s2 + s3);
        }
        if (ok && i < L) neg_lse[size_t(head0 + 2 * pair + c) * lse_stride + size_t(i)] = -(m_used + log2f(l));
      }
    }
  }

  // ------------------------------------------------------------- teardown
  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    ptx::abort_teardown(status, tid);   // status word, then time for copies in flight to land
  }
  if (warp == 0) ptx::tmem_dealloc(tmem_base, 256);
}

// ------------------------------------------------------------------ pass 2: column sums
template <int D>
__global__ void __launch_bounds__(kColThreads, 1)
calib_colsum_kernel(const CUtensorMap* __restrict__ maps, const float* __restrict__ neg_lse, int64_t lse_stride,
                    int64_t L, int n_q_heads, int n_kv_heads, float scale_log2e, double* __restrict__ colmean,
                    int* __restrict__ status, int n_tiles) {
  using Cfg = ColCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::offBar);
  static_assert(CN_BARS <= 24, "barrier block");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 24);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = n_q_heads / n_kv_heads;
  // unit-major: the CTAs resident at one time stream the same query tiles of the same heads
  const int u = int(blockIdx.x) / n_tiles;
  const int kt = int(blockIdx.x) % n_tiles;          // ascending: the longest columns go first
  const int seq = u / n_kv_heads, kvh = u % n_kv_heads;
  const int head0 = seq * n_q_heads + kvh * G;       // first query head of the group (flattened over batch)
  const int nq = n_tiles - kt;                       // query tiles kt .. n_tiles-1
  const int n_pairs = (G + 1) / 2;
  const int n_items = n_pairs * nq;                  // item n: heads 2*(n / nq) + {0, 1}, query tile kt + n % nq
  double total = 0.0;                                // this thread's column sum (summing warps only)

  if (tid == 0) {
    ptx::mbar_init(&bars[CB_K], 1);
    for (int i = 0; i < kQRing; ++i) {
      ptx::mbar_init(&bars[CB_FULL + i], 1);
      ptx::mbar_init(&bars[CB_EMPTY + i], 1 + 4);    // the MMA that read the tile + the four warps that read its lse
    }
    for (int c = 0; c < 2; ++c) {
      ptx::mbar_init(&bars[CB_S + c], 1);
      ptx::mbar_init(&bars[CB_FREE + c], 128);
    }
    ptx::fence_barrier_init();
    *abort_flag = (*reinterpret_cast<volatile int*>(status) != 0) ? 1 : 0;
  }
  if (warp == 0) {
    ptx::tmem_alloc(tmem_slot, 256);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (!*abort_flag) {
    if (warp == 0) {
      // ------------------------------------------------------------- TMA producer
      if (lane == 0) {
        ptx::mbar_arrive_expect_tx(&bars[CB_K], uint32_t(Cfg::kTile));
        for (int half = 0; half < Cfg::NH; ++half)
          ptx::tma_load_3d(smem + Cfg::offK + half * kColHalfBytes, &maps[1], half * 64, kt * CT, u, &bars[CB_K]);
        int jj = 0;
        bool ok = true;
        for (int n = 0; n < n_items && ok; ++n) {
          const int pair = n / nq, qt = kt + n % nq;
          for (int c = 0; c < 2; ++c) {
            const int g = 2 * pair + c;
            if (g >= G) continue;
            const int slot = jj % kQRing;
            if (jj >= kQRing && !ptx::mbar_wait(&bars[CB_EMPTY + slot], uint32_t(jj / kQRing - 1) & 1u, abort_flag)) {
              ok = false;
              break;
            }
            ptx::mbar_arrive_expect_tx(&bars[CB_FULL + slot], uint32_t(Cfg::kTile + CT * 4));
            uint8_t* dst = smem + Cfg::offRing + slot * Cfg::kSlot;
            for (int half = 0; half < Cfg::NH; ++half)
              ptx::tma_load_3d(dst + half * kColHalfBytes, &maps[0], half * 64, qt * CT, head0 + g, &bars[CB_FULL + slot]);
            bulk_copy_g2s(dst + Cfg::kTile, neg_lse + size_t(head0 + g) * lse_stride + size_t(qt) * CT, CT * 4,
                          &bars[CB_FULL + slot]);
            ++jj;
          }
        }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------- MMA issuer (whole warp, elected lane)
      {
        constexpr uint32_t idesc = ptx::idesc_bf16(CT, CT, false);
        const uint64_t dk = ptx::smem_desc_sw128(ptx::smem_u32(smem + Cfg::offK), 16, 1024);        // keys as A
        const uint64_t dq = ptx::smem_desc_sw128(ptx::smem_u32(smem + Cfg::offRing), 16, 1024);     // queries as B
        auto wait = [&](uint64_t* bar, uint32_t parity) -> bool {
          return __all_sync(0xffffffffu, ptx::mbar_wait(bar, parity, abort_flag));
        };
        bool ok = wait(&bars[CB_K], 0);
        int jj = 0;
        uint32_t done[2] = {0u, 0u};                 // tiles issued so far per chain
        for (int n = 0; n < n_items && ok; ++n) {
          const int pair = n / nq;
          for (int c = 0; c < 2; ++c) {
            if (2 * pair + c >= G) continue;
            const int slot = jj % kQRing;
            ok = wait(&bars[CB_FULL + slot], uint32_t(jj / kQRing) & 1u) &&
                 (done[c] == 0 || wait(&bars[CB_FREE + c], (done[c] - 1) & 1u));
            if (!ok) break;
            ptx::tc_fence_after();
            const uint64_t b0 = dq + uint64_t(uint32_t(slot * Cfg::kSlot) >> 4);
            const uint32_t d = tmem_base + uint32_t(c) * CT;
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
              const uint32_t off = (uint32_t(kk >> 2) * kColHalfBytes + uint32_t(kk & 3) * 32u) >> 4;
              ptx::umma_ss_elect(d, dk + off, b0 + off, idesc, kk > 0);
            }
            ptx::umma_commit_elect(&bars[CB_S + c]);
            ptx::umma_commit_elect(&bars[CB_EMPTY + slot]);
            ++done[c];
            ++jj;
          }
        }
      }
    } else {
      // ------------------------------------------------------------- summing warps, one key per thread
      const int c = (warp - 2) >> 2;
      const int quarter = warp & 3;                    // TMEM lanes this warp may touch
      const int r = quarter * 32 + lane;
      const uint32_t lane_addr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(c) * CT;
      const uint64_t scale2 = ptx::pack2(scale_log2e, scale_log2e);
      uint32_t done = 0;
      int jj = 0;
      bool ok = true;
      for (int n = 0; n < n_items && ok; ++n) {
        const int pair = n / nq, qt = kt + n % nq;
        for (int cc = 0; cc < 2; ++cc) {
          if (2 * pair + cc >= G) continue;
          const int slot = jj % kQRing;
          const uint32_t full_parity = uint32_t(jj / kQRing) & 1u;
          ++jj;
          if (cc != c) continue;
          // the slot's own barrier first (it makes the copied lse values visible to this thread and
          // cannot run ahead: the slot is recycled only after this warp has released it), then S
          ok = ptx::mbar_wait(&bars[CB_FULL + slot], full_parity, abort_flag) &&
               ptx::mbar_wait(&bars[CB_S + c], done & 1u, abort_flag);
          if (!ok) break;
          ++done;
          ptx::tc_fence_after();
          uint32_t v[CT];
#pragma unroll
          for (int q4 = 0; q4 < CT / 32; ++q4)
            ptx::tmem_ld32(lane_addr + q4 * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[q4 * 32]));
          ptx::tc_wait_ld();
          ptx::tc_fence_before();
          ptx::mbar_arrive(&bars[CB_FREE + c]);        // the scores are in registers: S may be overwritten
          // p = exp2(s * scale - lse) for the 128 queries of the tile; the tile's data has landed
          // (the MMA that produced S waited for it), the lse values sit behind the Q tile
          const float2* nl = reinterpret_cast<const float2*>(smem + Cfg::offRing + slot * Cfg::kSlot + Cfg::kTile);
          const int lo = (qt == kt) ? r : 0;           // causal: query index >= key index
          const int hi = int(min(int64_t(CT), L - int64_t(qt) * CT));   // queries past L do not exist
          const bool masked = lo > 0 || hi < CT;
          uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
          for (int j = 0; j < CT / 2; ++j) {
            const float2 b = nl[j];
            float xl, xh;
            ptx::unpack2(ptx::fma2(ptx::pack2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), scale2,
                                   ptx::pack2(b.x, b.y)), xl, xh);
            float el = ptx::fast_exp2(xl), eh = ptx::fast_exp2(xh);
            if (masked) {
              if (2 * j < lo || 2 * j >= hi) el = 0.f;
              if (2 * j + 1 < lo || 2 * j + 1 >= hi) eh = 0.f;
            }
            sum2[j & 1] = ptx::add2(sum2[j & 1], ptx::pack2(el, eh));
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&bars[CB_EMPTY + slot]);   // this warp no longer reads the slot's lse
          float s0, s1, s2, s3;
          ptx::unpack2(sum2[0], s0, s1);
          ptx::unpack2(sum2[1], s2, s3);
          total += double((s0 + s1) + (s2 + s3));
        }
      }
    }
  }

  // ------------------------------------------------------------- teardown and result
  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    ptx::abort_teardown(status, tid);   // status word, then time for copies in flight to land
  } else {
    // every MMA has completed (each chain waited for its last S), so the K tile's shared memory
    // can carry chain 1's sums over to chain 0
    double* part = reinterpret_cast<double*>(smem + Cfg::offK);
    const int r = (warp & 3) * 32 + lane;
    if (warp >= 6) part[r] = total;
    __syncthreads();
    if (warp >= 2 && warp < 6) {
      const int64_t kidx = int64_t(kt) * CT + r;
      if (kidx < L) colmean[size_t(u) * L + kidx] = (total + part[r]) / (double(G) * double(L - kidx));
    }
  }
  if (warp == 0) ptx::tmem_dealloc(tmem_base, 256);
}


// a[u] of Eq. 4 as the share of the column means that the retained set holds: the unit's selected
// indices plus its always-kept tail [mb, L), over all L tokens (Section 4.3 counts the global and
// the local subset as retained).  One CTA per unit; strided partial sums and a fixed-shape tree,
// hence reproducible.
__global__ void __launch_bounds__(256)
calib_score_kernel(const double* __restrict__ colmean, int64_t L, int64_t mb, const int32_t* __restrict__ idx,
                   const int64_t* __restrict__ offsets, double* __restrict__ a_out) {
  const int u = blockIdx.x, tid = threadIdx.x;
  const double* c = colmean + size_t(u) * L;
  const int64_t i0 = offsets[u], i1 = offsets[u + 1];
  double num = 0.0, den = 0.0;
  for (int64_t i = i0 + tid; i < i1; i += 256) num += c[idx[i]];
  for (int64_t k = tid; k < L; k += 256) {
    const double v = c[k];
    den += v;
    if (k >= mb) num += v;
  }
  __shared__ double s_num[256], s_den[256];
  s_num[tid] = num;
  s_den[tid] = den;
  __syncthreads();
  for (int off = 128; off > 0; off >>= 1) {
    if (tid < off) { s_num[tid] += s_num[tid + off]; s_den[tid] += s_den[tid + off]; }
    __syncthreads();
  }
  if (tid == 0) a_out[u] = s_den[0] > 0.0 ? s_num[0] / s_den[0] : 1.0;
}

struct CalibWs {
  CUtensorMap* maps;    // Q and K, shared by both passes
  float* neg_lse;       // [batch * n_q_heads][Lp]
  int64_t Lp;
  size_t bytes;
};

CalibWs calib_ws_layout(const tca_params* prm, int64_t L, void* ws) {
  CalibWs w;
  char* p = static_cast<char*>(ws);
  size_t off = 256;     // word 0: status
  w.maps = reinterpret_cast<CUtensorMap*>(p + off);
  off += align_up(2 * sizeof(CUtensorMap), 256);
  w.Lp = (L + CT - 1) / CT * CT;
  w.neg_lse = reinterpret_cast<float*>(p + off);
  off += align_up(size_t(prm->batch) * prm->n_q_heads * size_t(w.Lp) * sizeof(float), 256);
  w.bytes = off;
  return w;
}

template <int D>
int launch_colmean(const tca_params* prm, const void* Q, const void* K, int64_t L, double* colmean, void* ws,
                   cudaStream_t stream) {
  const CalibWs w = calib_ws_layout(prm, L, ws);
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  const int64_t heads = int64_t(prm->batch) * prm->n_q_heads;
  CUtensorMap maps[2];
  if (!encode_map(&maps[0], Q, D, L, heads, L) || !encode_map(&maps[1], K, D, L, U, L)) return TCA_ERR_CUDA;
  // pageable source: staged by the runtime before the call returns
  TCA_CHECK_CUDA(cudaMemcpyAsync(w.maps, maps, sizeof(maps), cudaMemcpyHostToDevice, stream));
  const int n_tiles = int((L + CT - 1) / CT);
  const int64_t n_ctas = int64_t(n_tiles) * U;
  if (n_ctas >= (int64_t(1) << 31)) return TCA_ERR_UNSUPPORTED;
  const float scale_log2e = prm->sm_scale * 1.4426950408889634f;

  auto rows = calib_rowstats_kernel<D>;
  TCA_CHECK_CUDA(cudaFuncSetAttribute(rows, cudaFuncAttributeMaxDynamicSharedMemorySize, RowCfg<D>::bytes));
  rows<<<unsigned(n_ctas), kColThreads, RowCfg<D>::bytes, stream>>>(
      w.maps, w.neg_lse, w.Lp, L, prm->n_q_heads, prm->n_kv_heads, scale_log2e, static_cast<int*>(ws), n_tiles);
  int st = check_launch();
  if (st != TCA_OK) return st;

  auto cols = calib_colsum_kernel<D>;
  TCA_CHECK_CUDA(cudaFuncSetAttribute(cols, cudaFuncAttributeMaxDynamicSharedMemorySize, ColCfg<D>::bytes));
  cols<<<unsigned(n_ctas), kColThreads, ColCfg<D>::bytes, stream>>>(
      w.maps, w.neg_lse, w.Lp, L, prm->n_q_heads, prm->n_kv_heads, scale_log2e, colmean, static_cast<int*>(ws),
      n_tiles);
  return check_launch();
}

}  // namespace

size_t calib_ws_bytes(const tca_params* prm, int64_t L) { return calib_ws_layout(prm, L, nullptr).bytes; }

}  // namespace tca

using namespace tca;

extern "C" int tca_calib_colmean(const tca_params* prm, const void* Q, const void* K, int64_t L, double* colmean,
                                 void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  TCA_CHECK_ARG(Q && K && colmean && ws);
  TCA_CHECK_ARG(L >= 1 && L < (int64_t(1) << 31));
  TCA_CHECK_ARG(aligned(Q, 16) && aligned(K, 16) && aligned(colmean, 8) && aligned(ws, 256));
  if (prm->dtype != TCA_BF16) return TCA_ERR_UNSUPPORTED;
  TCA_CHECK_ARG(int64_t(prm->batch) * prm->n_q_heads <= 65535);
  if (ws_bytes < calib_ws_bytes(prm, L)) return TCA_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (prm->head_dim == 128) return launch_colmean<128>(prm, Q, K, L, colmean, ws, s);
  return launch_colmean<64>(prm, Q, K, L, colmean, ws, s);
}

extern "C" int tca_calib_score(const tca_params* prm, const double* colmean, int64_t L, const int32_t* idx,
                               const int64_t* offsets_dev, double* a_out, void* stream) {
  int st = check_params(prm);
  if (st != TCA_OK) return st;
  TCA_CHECK_ARG(colmean && offsets_dev && a_out && L >= 1);   // idx may be NULL when nothing is selected
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  const int64_t mb = num_blocks(prm, L) * prm->block;
  calib_score_kernel<<<unsigned(U), 256, 0, static_cast<cudaStream_t>(stream)>>>(colmean, L, mb, idx, offsets_dev,
                                                                                a_out);
  return check_launch();
}

extern "C" int tca_calib_choose(const double* a, const int64_t* sizes, int n_candidates, double tau) {
  if (!a || !sizes || n_candidates < 1) return TCA_ERR_INVALID_ARG;
  int best = -1;
  for (int i = 0; i < n_candidates; ++i)
    if (a[i] >= tau && (best < 0 || sizes[i] < sizes[best])) best = i;
  return best < 0 ? n_candidates - 1 : best;
}

extern "C" int tca_calib_candidates(int block, int n_candidates, double sigma, double* p_out) {
  if (block < 1 || (block & (block - 1)) != 0 || n_candidates < 2 || !(sigma > 0.0) || !p_out)
    return TCA_ERR_INVALID_ARG;
  int nK = 1;
  while ((1 << (nK - 1)) < block) ++nK;
  for (int i = 0; i < n_candidates; ++i) {
    // Eq. 3 with mu^i = log2(1 + (i - 1)(b - 1)/(M - 1)), i = 1..M
    const double mu = std::log2(1.0 + double(i) * double(block - 1) / double(n_candidates - 1));
    double sum = 0.0;
    for (int k = 0; k < nK; ++k) {
      const double x = double(k) - mu;               // log2 of the retain count 2^k, minus mu
      p_out[size_t(i) * nK + k] = std::exp(-x * x / (2.0 * sigma * sigma));
      sum += p_out[size_t(i) * nK + k];
    }
    for (int k = 0; k < nK; ++k) p_out[size_t(i) * nK + k] /= sum;
  }
  return TCA_OK;
}
