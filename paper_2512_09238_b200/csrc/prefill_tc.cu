// Sparse causal prefill attention (Eq. 2, Algorithm 2 line 7) on the 5th-generation tensor
// cores: tcgen05.mma with fp32 accumulators in TMEM, operands staged by TMA with 128-byte
// swizzle, online softmax on the CUDA cores, bf16 inputs.
//
// One CTA owns 128 consecutive query positions of TWO query heads of one GQA group (same
// KV head, same positions, hence the same key tiles and the same mask), which halves the
// K/V traffic per flop and lets the tensor pipe work on one head while the other head's
// softmax runs.  Key tiles (128 keys) come from two ranges under one online softmax:
//   (1) the unit's selected keys in the cache's global region with position < c_hi, and
//   (2) the contiguous band [c_lo, i_last] of the original K/V,
// with c_i = min(max(0, i - w + 1), m*b); row i sees columns {pos < c_i} of (1) and
// {c_i <= j <= i} of (2), so every key is counted once.  Only tiles that straddle one of
// those bounds evaluate a mask; a masked score is -inf and its weight an exact zero, so cache
// rows past the visible prefix only have to hold finite values.  The two ranges are walked
// global first (default) or band first (TCA_FLAG_PREFILL_BAND_FIRST).  The band needs nothing
// that score / select / compact produce, so in the band-first order the kernel, launched with
// programmatic dependent launch, starts on the band while those kernels are still running
// and waits for them (griddepcontrol.wait) only where it first touches the cache.
//
// Warp roles (384 threads = 3 warpgroups): warp 0 = TMA producer (one lane), warp 1 = MMA issuer,
// warp 2 = geometry of the global range (a warp-wide search at the start), warp 3 idle (when the
// selected rows are gathered from K and V instead of read from the cache: second producer);
// warps 4-7 / 8-11 = softmax of head 0 / head 1 (one thread per
// query row = one TMEM lane).  The first warpgroup hands most of its registers to the other two
// (setmaxnreg), so that a softmax thread can hold its row of 128 scores without spilling.
// TMEM (512 columns): S0 | S1 | O0 | O1; the bf16 P of a tile overwrites the first half of its
// S columns and feeds the PV product straight from TMEM.  Shared memory: Q0 Q1 | 5-slot K/V ring.
// Per tile the issuer runs  PV0(t) S0(t+1) PV1(t) S1(t+1)  so that S of one head is being
// computed while the other head's softmax is in flight; the whole issuer warp executes the
// loop and an elected lane's tcgen05 instructions take effect (see umma_ss_elect).
//
// Softmax of one tile, per thread: the 128 scores of the row come into registers with one wait;
// maximum; then the exponentials in eight groups of 16, each group's packed bf16 results stored to
// TMEM only after the next group's arithmetic has been issued, so the MUFU, which limits this
// phase (one ex2 per score is as many MUFU clocks as the two products of the tile are tensor
// clocks), is never left to drain.  P reaches the PV product in two parts (96 keys, then 32: the
// less is left to issue after the last announcement, the sooner the next S can follow), each
// announced by one arrival per warp.  O stays in TMEM and is rescaled lazily: only when a row
// maximum grew by more than 2^8 since the last rescale.
// CTAs are ordered unit-major so that the CTAs resident at one time read the same one or two
// KV heads out of L2.
//
// Every mbarrier wait is bounded; a wait that gives up raises the status word of the
// workspace, lets outstanding copies land, frees TMEM and returns.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "ptx_sm100.cuh"
#include "tensor_map.cuh"

namespace tca {
namespace {

constexpr int BM = 128, BN = 128;
constexpr int kThreads = 384;              // three warpgroups: producer + issuer, softmax of head 0, softmax of head 1
constexpr int kRegsLean = 88, kRegsSoftmax = 208;   // per-thread registers after the warpgroups trade them
constexpr int kRing = 5;                // K/V tiles in shared memory
constexpr int kPairs = 3;               // (V_t, K_t+1) barrier pairs that can be in flight
constexpr int kHalfBytes = 128 * 128;   // 128 rows x 128 bytes (64 bf16): one swizzled box
constexpr float kRescaleThreshold = 8.f;
constexpr int kPHalves = 2;             // P reaches the PV product in two parts
constexpr int kPSplit = 6;              // k-steps (16 keys each) in the first part: 96 keys, then 32

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

enum { BAR_Q = 0, BAR_K0_FULL = 1, BAR_K0_EMPTY = 2, BAR_GEO = 3, BAR_FULL = 4, BAR_EMPTY = BAR_FULL + kPairs,
       BAR_S = BAR_EMPTY + kPairs, BAR_P = BAR_S + 2, BAR_PV = BAR_P + 2 * kPHalves, N_BARS = BAR_PV + 2 };

// The two key ranges of a CTA in the order they are walked: n_a tiles of the first range, then
// n_b of the second.  Band first: a = band, b = global; otherwise a = global, b = band.
struct TileSeq {
  int n_a, n_b;
  bool band_first;
  int64_t c_lo;   // first position of the band
  int64_t seg;    // first cache row of the unit's global region
  __device__ __forceinline__ bool is_global(int t) const { return band_first ? t >= n_a : t < n_a; }
  __device__ __forceinline__ int index(int t) const { return t < n_a ? t : t - n_a; }   // within its range
  // global: first cache row of the tile; band: first position
  __device__ __forceinline__ int64_t first(int t) const {
    return is_global(t) ? seg + int64_t(index(t)) * BN : c_lo + int64_t(index(t)) * BN;
  }
};

__device__ __forceinline__ int lower_bound_pos(const int32_t* pos, int lo, int hi, int64_t bound) {
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (int64_t(pos[mid]) < bound) lo = mid + 1; else hi = mid;
  }
  return lo;
}
// The same search by a whole warp: 32 probes per round instead of one, so a range of 2^17 rows
// takes four dependent loads instead of seventeen.  Every lane returns the result.
__device__ __forceinline__ int lower_bound_pos_warp(const int32_t* pos, int lo, int hi, int64_t bound, int lane) {
  while (hi - lo > 32) {
    const int step = (hi - lo + 32) / 33;                     // 32 probes cut the range into 33 pieces
    const int idx = min(lo + (lane + 1) * step - 1, hi - 1);
    const unsigned below = __ballot_sync(0xffffffffu, int64_t(pos[idx]) < bound);   // monotone: a prefix of ones
    const int n = __popc(below);
    const int new_lo = (n == 0) ? lo : min(lo + n * step, hi);   // probe n-1 was below the bound: so is everything up to it
    const int new_hi = (n == 32) ? hi : min(lo + (n + 1) * step - 1, hi - 1);   // probe n was not: the answer is at or before it
    lo = new_lo;
    hi = max(new_hi, new_lo);
  }
  const int idx = lo + lane;
  const unsigned below = __ballot_sync(0xffffffffu, idx < hi && int64_t(pos[idx]) < bound);
  return lo + __popc(below);
}

// kGather: the selected keys are not read from a compacted cache but fetched from K and V
// themselves (Kraw, Vraw), row by row, by two producer warps with 16-byte asynchronous copies that
// they place into the swizzled tile themselves; `pos` is then the index set that the selection wrote,
// `state` its per-unit offsets, and map_ck / map_cv are not used.
template <int D, bool kGather>
__global__ void __launch_bounds__(kThreads, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_ck,
                  const __grid_constant__ CUtensorMap map_cv, const int32_t* __restrict__ pos,
                  const int64_t* __restrict__ state, int64_t L, int n_q_heads, int n_kv_heads, int window,
                  int64_t mb, float scale_log2e, __nv_bfloat16* __restrict__ O, int* __restrict__ status,
                  int n_qtiles, int pairs_per_unit, int tile0, int band_first,
                  const __nv_bfloat16* __restrict__ Kraw, const __nv_bfloat16* __restrict__ Vraw) {
  using Cfg = TcCfg<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + Cfg::offBar);
  static_assert(N_BARS <= 24, "barrier block");
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 24);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* s_geo = reinterpret_cast<volatile int*>(tmem_slot + 2);   // [0] visible rows at c_lo, [1] at c_hi

  pdl_launch_dependents();   // whatever follows in the stream may be scheduled; it waits for this grid itself
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
  const int64_t c_lo = min(max(int64_t(0), i0 - window + 1), mb);
  const int64_t c_hi = min(max(int64_t(0), i_last - window + 1), mb);
  const int n_band = int((i_last - c_lo + BN) / BN);            // >= 1: a query always sees itself

  if (tid == 0) {
    ptx::mbar_init(&bars[BAR_Q], 1);
    ptx::mbar_init(&bars[BAR_K0_FULL], kGather ? 32 : 1);   // gathering: every producer lane arrives
    ptx::mbar_init(&bars[BAR_K0_EMPTY], 1);
    ptx::mbar_init(&bars[BAR_GEO], 1);
    for (int i = 0; i < kPairs; ++i) {
      ptx::mbar_init(&bars[BAR_FULL + i], kGather ? 64 : 2);
      ptx::mbar_init(&bars[BAR_EMPTY + i], 1);
    }
    for (int h = 0; h < 2; ++h) {
      ptx::mbar_init(&bars[BAR_S + h], 1);
      for (int c = 0; c < kPHalves; ++c) ptx::mbar_init(&bars[BAR_P + h * kPHalves + c], 4);   // one arrival per warp
      ptx::mbar_init(&bars[BAR_PV + h], 1);
    }
    ptx::fence_barrier_init();
    // the status word is the caller's (no kernel of this stream writes it): readable before the dependency wait
    *abort_flag = (*reinterpret_cast<volatile int*>(status) != 0) ? 1 : 0;
    ptx::tma_prefetch_desc(&map_q);
    ptx::tma_prefetch_desc(&map_k);
    ptx::tma_prefetch_desc(&map_v);
  }
  if (warp == 0) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Q, K and V are the caller's inputs, but the kernels before this one in the stream (score,
  // select, compact, the previous row range) may still be running when this grid starts.  Q, K
  // and V are not written by any of them; the cache, its positions and its state words are.
  // Global-first order needs those at once; band-first order only after the band.
  if (!band_first) pdl_wait();

  // Everything about the global range comes from the geometry thread through BAR_GEO.
  TileSeq geo;
  geo.band_first = band_first != 0;
  geo.c_lo = c_lo;
  geo.seg = 0;
  geo.n_a = band_first ? n_band : 0;
  geo.n_b = band_first ? 0 : n_band;
  bool geo_known = false;
  // Blocks until the geometry thread has published, then fills in the global range.  Returns
  // false if the wait gave up.
  auto learn_geometry = [&]() -> bool {
    if (geo_known) return true;
    if (!ptx::mbar_wait(&bars[BAR_GEO], 0, abort_flag)) return false;
    pdl_wait();                                   // the cache rows read from here on are visible to this thread
    const int n_gt = (s_geo[1] + BN - 1) / BN;
    geo.seg = kGather ? state[u] : state[size_t(u) * TCA_STATE_WORDS + TCA_ST_SEG_START];
    if (geo.band_first) geo.n_b = n_gt; else geo.n_a = n_gt;
    geo_known = true;
    return true;
  };
  // The same for a whole warp that has to stay converged (elect.sync, warp-wide TMEM access, votes):
  // every lane leaves with the same answer.
  auto learn_geometry_warp = [&]() -> bool { return __all_sync(0xffffffffu, learn_geometry()); };

  // The two kinds of warpgroup part ways here for good, so that the compiler sees which code runs
  // under which register budget.
  if (warp < 4) {
    ptx::reg_dealloc<kRegsLean>();
    if (*abort_flag) {
      // a status word that was already set: do nothing
    } else if (warp == 2) {
      // ------------------------------------------------------------- geometry of the global range
      pdl_wait();
      const int64_t* st = state + size_t(u) * TCA_STATE_WORDS;
      const int64_t seg = kGather ? state[u] : st[TCA_ST_SEG_START];
      const int n_global = kGather ? int(state[u + 1] - state[u]) : int(st[TCA_ST_N_GLOBAL]);
      const int vis_lo = lower_bound_pos_warp(pos + seg, 0, n_global, c_lo, lane);
      const int vis_hi = lower_bound_pos_warp(pos + seg, vis_lo, n_global, c_hi, lane);
      if (lane == 0) {
        s_geo[0] = vis_lo;
        s_geo[1] = vis_hi;
        __threadfence_block();
        ptx::mbar_arrive(&bars[BAR_GEO]);
      }
    } else if (warp == 0 || (kGather && warp == 3)) {
      // ------------------------------------------------------------- producer
      // One lane of warp 0 issues the box loads.  Row gathers take a whole warp per tile (and one
      // warp cannot keep up with the tensor pipe), so when gathering warp 0 brings the K tiles and
      // warp 3 the V tiles; all their lanes walk the loop and every wait is made warp-uniform.
      const bool do_k = !kGather || warp == 0, do_v = !kGather || warp == 3;
      if (kGather || lane == 0) {
        auto pwait = [&](uint64_t* bar, uint32_t parity) -> bool {
          const bool r = ptx::mbar_wait(bar, parity, abort_flag);
          if constexpr (kGather) return __all_sync(0xffffffffu, r); else return r;
        };
        auto plearn = [&]() -> bool {
          if constexpr (kGather) return learn_geometry_warp(); else return learn_geometry();
        };
        if (lane == 0 && do_k) {
          ptx::mbar_arrive_expect_tx(&bars[BAR_Q], uint32_t(nh * Cfg::kQ));
          for (int h = 0; h < nh; ++h)
            for (int half = 0; half < Cfg::NH; ++half)
              ptx::tma_load_3d(smem + Cfg::offQ + h * Cfg::kQ + half * kHalfBytes, &map_q, half * 64, int(i0),
                               hq0 + h, &bars[BAR_Q]);
        }
        bool ok = band_first || plearn();
        // load n: n = 0 is K of tile 0; n = 2t+1 is V of tile t; n = 2t+2 is K of tile t+1.  V_t and
        // K_t+1 share the barrier pair t % kPairs (the issuer needs them together).
        for (int n = 0; ok; ++n) {
          const int is_v = n & 1;
          const int t = is_v ? (n - 1) >> 1 : n >> 1;          // the tile this load belongs to
          if (t >= geo.n_a && !geo_known) { ok = plearn(); if (!ok) break; }
          if (t >= geo.n_a + geo.n_b) {
            // past the last tile: the last pair holds V only, its barrier still expects two arrivals
            if (!is_v && t > 0 && do_k && (kGather || lane == 0)) ptx::mbar_arrive(&bars[BAR_FULL + (t - 1) % kPairs]);
            break;
          }
          if (is_v ? !do_v : !do_k) continue;                  // the other producer warp's tile
          // The row numbers of a gathered tile are requested before the wait for the ring slot, which
          // hides their latency.  Row r of the tile is the unit's selected key number index(t)*128 + r;
          // a tile that reaches past the keys visible to this query tile repeats the last visible one:
          // the mask gives those columns an exact zero weight, the row only has to be finite.
          const bool gathered = kGather && geo.is_global(t);
          int rows4[4] = {0, 0, 0, 0};
          if (gathered) {
            const int32_t* sel = pos + geo.seg;
            const int last = s_geo[1] - 1;                     // >= 0: there is at least one global tile
            const int first = geo.index(t) * BN + 4 * lane;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              int64_t p = sel[min(first + k, last)];
              if constexpr (kDebugBounds) {
                if (p < 0 || p >= mb) {                        // a selected index names a candidate token
                  report_bounds_ws(status, kBoundsSelectedIndex, p);
                  p = 0;
                }
              }
              rows4[k] = int(int64_t(u) * L + p);
            }
          }
          const int slot = n % kRing;
          if (n >= kRing) {                                    // the slot's previous tile must have been consumed
            const int r = n - kRing;
            if (r == 0) ok = pwait(&bars[BAR_K0_EMPTY], 0);
            else {
              const int tr = (r - 1) >> 1;
              ok = pwait(&bars[BAR_EMPTY + tr % kPairs], uint32_t(tr / kPairs) & 1u);
            }
            if (!ok) break;
          }
          uint64_t* full = (n == 0) ? &bars[BAR_K0_FULL] : &bars[BAR_FULL + ((n - 1) >> 1) % kPairs];
          uint8_t* dst = smem + Cfg::offKV + slot * Cfg::kKV;
          if (gathered) {
            // A lane copies its own four rows, 16 bytes at a time, to where the 128-byte swizzle wants
            // them: the chunk that lands at position j of the 128-byte shared-memory row r is chunk
            // j ^ (r & 7) of the source row.
            const uint8_t* gsrc = reinterpret_cast<const uint8_t*>(is_v ? Vraw : Kraw);
            const uint32_t dtile = ptx::smem_u32(dst);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int r = 4 * lane + k;
              const uint8_t* srow = gsrc + size_t(rows4[k]) * (D * 2);
              const uint32_t drow = dtile + uint32_t(r) * 128u;
              const int x = r & 7;
#pragma unroll
              for (int half = 0; half < Cfg::NH; ++half)
#pragma unroll
                for (int j = 0; j < 8; ++j)
                  ptx::cp_async_16(drow + uint32_t(half) * kHalfBytes + uint32_t(j) * 16u,
                                   srow + half * 128 + ((j ^ x) << 4));
            }
            ptx::cp_async_mbar_arrive_noinc(full);             // fires when this lane's copies have landed
          } else if (lane == 0) {
            ptx::mbar_arrive_expect_tx(full, uint32_t(Cfg::kKV));
            const int y = int(geo.first(t));
            for (int half = 0; half < Cfg::NH; ++half) {
              if (geo.is_global(t))
                ptx::tma_load_2d(dst + half * kHalfBytes, is_v ? &map_cv : &map_ck, half * 64, y, full);
              else
                ptx::tma_load_3d(dst + half * kHalfBytes, is_v ? &map_v : &map_k, half * 64, y, u, full);
            }
          } else if (kGather) {
            ptx::mbar_arrive(full);                            // a box load: the other lanes only make up the count
          }
        }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------- MMA issuer
      // The whole warp runs this loop; one elected lane issues (see umma_ss_elect).  Waits are
      // made warp-uniform so that the warp stays converged for elect.sync.
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
      // O += P V with P read from TMEM (packed bf16 over the first 64 columns of S): the A operand
      // costs no shared-memory bandwidth.  The first kPSplit k-steps go as soon as the first
      // part of P is announced, while the softmax warps still work on the rest.
      auto issue_PV = [&](int h, int slot, bool acc, uint32_t parity) -> bool {
        const uint64_t b0 = dv + uint64_t(uint32_t(slot * Cfg::kKV) >> 4);
        const uint32_t d = tmem_base + Cfg::colO(h);
        const uint32_t a = tmem_base + Cfg::colP(h);
#pragma unroll
        for (int c = 0; c < kPHalves; ++c) {
          if (!wait(&bars[BAR_P + h * kPHalves + c], parity)) return false;
          ptx::tc_fence_after();
#pragma unroll
          for (int kk = (c == 0 ? 0 : kPSplit); kk < (c == 0 ? kPSplit : BN / 16); ++kk) {
            ptx::umma_ts_elect(d, a + uint32_t(kk * 8), b0 + uint32_t((kk * 2048) >> 4), idescPV,
                               (acc || kk > 0) ? 1u : 0u);
          }
        }
        return true;
      };
      bool ok = (band_first || learn_geometry_warp()) && wait(&bars[BAR_Q], 0) && wait(&bars[BAR_K0_FULL], 0);
      if (ok) {
        ptx::tc_fence_after();
        for (int h = 0; h < nh; ++h) { issue_S(h, 0); ptx::umma_commit_elect(&bars[BAR_S + h]); }
        ptx::umma_commit_elect(&bars[BAR_K0_EMPTY]);
      }
      for (int t = 0; ok; ++t) {
        if (t + 1 >= geo.n_a && !geo_known) { ok = learn_geometry_warp(); if (!ok) break; }
        const int nt = geo.n_a + geo.n_b;
        if (t >= nt) break;
        const int slotV = (2 * t + 1) % kRing, slotK = (2 * t + 2) % kRing;
        const bool more = t + 1 < nt;
        // V of this tile and K of the next arrive under one barrier
        ok = wait(&bars[BAR_FULL + t % kPairs], uint32_t(t / kPairs) & 1u);
        for (int h = 0; h < nh && ok; ++h) {
          ok = issue_PV(h, slotV, t > 0, uint32_t(t) & 1u);
          if (!ok) break;
          if (more) issue_S(h, slotK);
          ptx::umma_commit_elect(&bars[more ? BAR_S + h : BAR_PV + h]);   // S ready implies PV done
          if (h == nh - 1) ptx::umma_commit_elect(&bars[BAR_EMPTY + t % kPairs]);
        }
      }
    }
  } else {
    ptx::reg_alloc<kRegsSoftmax>();
    {
      // ------------------------------------------------------------- softmax, one row per thread
      const int h = (warp - 4) >> 2;
      if (!*abort_flag && h < nh) {
        const int quarter = warp & 3;                    // TMEM lanes this warp may touch
        const int row = quarter * 32 + lane;
        const int64_t i = i0 + row;
        const int64_t c_i = min(max(int64_t(0), i - window + 1), mb);
        const int dc = int(c_i - c_lo), di = int(i - c_lo);   // window start and own position relative to the band
        const uint32_t lane_addr = tmem_base + (uint32_t(quarter * 32) << 16);
        const uint32_t s_addr = lane_addr + Cfg::colS(h);
        float m_run = -INFINITY, m_used = -INFINITY, l = 0.f;
        int nvis_i = 0;
        bool ok = band_first || learn_geometry_warp();
        bool have_nvis = false;
        const uint64_t scale2 = ptx::pack2(scale_log2e, scale_log2e);
        int t = 0;
        for (; ok; ++t) {
          if (t >= geo.n_a && !geo_known) { ok = learn_geometry_warp(); if (!ok) break; }
          if (t >= geo.n_a + geo.n_b) break;
          int lo, hi;
          if (geo.is_global(t)) {
            if (!have_nvis) {
              // rows of this tile see between s_geo[0] and s_geo[1] selected keys: search only there
              nvis_i = lower_bound_pos(pos + geo.seg, s_geo[0], s_geo[1], c_i);
              have_nvis = true;
            }
            lo = 0;
            hi = nvis_i - 1 - geo.index(t) * BN;
          } else {
            const int off = geo.index(t) * BN;             // tile start relative to the band's first position
            lo = max(-1, dc - off);
            hi = min(BN, di - off);
          }
          // Per lane, no vote: the branch it guards only rewrites registers, so lanes may diverge in
          // the few tiles that straddle a bound.
          const bool masked = lo > 0 || hi < BN - 1;
          ok = __all_sync(0xffffffffu, ptx::mbar_wait(&bars[BAR_S + h], uint32_t(t) & 1u, abort_flag));   // uniform: the warp leaves together
          if (!ok) break;
          ptx::tc_fence_after();
          // the whole row of S (128 fp32) into registers with one wait
          uint32_t v[BN];
#pragma unroll
          for (int c = 0; c < BN / 32; ++c)
            ptx::tmem_ld32(s_addr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&v[c * 32]));
          ptx::tc_wait_ld();
          if (masked) {   // a masked score is -inf: it loses every max and its exponential is exactly 0
#pragma unroll
            for (int k = 0; k < BN; ++k)
              if (k < lo || k > hi) v[k] = 0xff800000u;
          }
          float mx;
          {
            float mx8[8];
#pragma unroll
            for (int a = 0; a < 8; ++a) mx8[a] = fmaxf(__uint_as_float(v[2 * a]), __uint_as_float(v[2 * a + 1]));
#pragma unroll
            for (int k = 16; k < BN; k += 16)
#pragma unroll
              for (int a = 0; a < 8; ++a)
                mx8[a] = ptx::max3(mx8[a], __uint_as_float(v[k + 2 * a]), __uint_as_float(v[k + 2 * a + 1]));
            mx = fmaxf(fmaxf(ptx::max3(mx8[0], mx8[1], mx8[2]), ptx::max3(mx8[3], mx8[4], mx8[5])), fmaxf(mx8[6], mx8[7]));
          }
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
          // p = exp2(s*scale - m), row sum, packed bf16 P back into TMEM over the S columns.  Eight
          // groups of 16 scores; a group's store is issued only after the next group's arithmetic, so
          // that the store never waits for exponentials still in the MUFU and the MUFU never drains.
          const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used;
          const uint64_t neg_m2 = ptx::pack2(neg_m, neg_m);
          uint64_t sum2[2] = {0ull, 0ull};
#pragma unroll
          for (int g = 0; g < 8; ++g) {
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
              const int j = g * 8 + jj;
              float xl, xh;
              ptx::unpack2(ptx::fma2(ptx::pack2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])), scale2, neg_m2),
                           xl, xh);
              const float el = ptx::fast_exp2(xl), eh = ptx::fast_exp2(xh);
              sum2[j & 1] = ptx::add2(sum2[j & 1], ptx::pack2(el, eh));
              v[j] = ptx::pack_bf16x2(el, eh);   // entry j is never read again (j <= 2j)
            }
            if (g == kPSplit + 1) {   // groups 0 .. kPSplit-1 (the first 96 keys) were stored at least one group ago
              ptx::tc_wait_st();
              ptx::tc_fence_before();
              __syncwarp();
              if (lane == 0) ptx::mbar_arrive(&bars[BAR_P + h * kPHalves + 0]);
            }
            if (g >= 1) ptx::tmem_st8(lane_addr + Cfg::colP(h) + (g - 1) * 8, &v[(g - 1) * 8]);
          }
          ptx::tmem_st8(lane_addr + Cfg::colP(h) + 56, &v[56]);
          ptx::tc_wait_st();
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&bars[BAR_P + h * kPHalves + 1]);
          {
            float s0, s1, s2, s3;
            ptx::unpack2(sum2[0], s0, s1);
            ptx::unpack2(sum2[1], s2, s3);
            l += (s0 + s1) + (s2 + s3);
          }
        }
        // epilogue: O / l -> bf16 -> global
        if (ok) ok = __all_sync(0xffffffffu, ptx::mbar_wait(&bars[BAR_PV + h], 0, abort_flag));   // committed once, after the last PV
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
  pdl_wait();   // every thread has observed its predecessors before the grid can complete (keeps the chain ordered)
  ptx::tc_fence_before();
  __syncthreads();
  if (*abort_flag) ptx::abort_teardown(status, tid);   // status word, then time for copies in flight to land
  if (warp == 0) ptx::tmem_dealloc(tmem_base, 512);
}

// ------------------------------------------------------------------ host side
// Encoded tensor maps are kept in a small cache keyed by what they were encoded from: a prefill
// that comes as several row-range calls, or step after step over the same buffers, encodes them once.
struct MapKey {
  const void* base;
  int D;
  int64_t rows, heads;
  bool operator==(const MapKey& o) const { return base == o.base && D == o.D && rows == o.rows && heads == o.heads; }
};
struct MapEntry {
  MapKey key{nullptr, 0, 0, 0};
  CUtensorMap map;
};
std::mutex g_map_mutex;
MapEntry g_maps[16];
int g_map_next = 0;

bool cached_map(CUtensorMap* out, const void* base, int D, int64_t rows, int64_t heads) {
  const MapKey key{base, D, rows, heads};
  std::lock_guard<std::mutex> lock(g_map_mutex);
  for (const MapEntry& e : g_maps)
    if (e.key == key) { *out = e.map; return true; }
  MapEntry& slot = g_maps[g_map_next];
  g_map_next = (g_map_next + 1) % 16;
  slot.key = MapKey{nullptr, 0, 0, 0};
  if (!encode_map(&slot.map, base, D, rows, heads, rows)) return false;
  slot.key = key;
  *out = slot.map;
  return true;
}

}  // namespace

size_t prefill_tc_ws_bytes(const tca_params*) { return 256; }   // the status word

// The selected keys come either from the cache (c != nullptr) or, by row gathers, from K and V
// themselves (c == nullptr; idx and offsets_dev are what the selection wrote / was given).
template <int D, bool kGather>
int launch_prefill_tc_impl(const tca_params* prm, const void* Q, const void* K, const void* V, int64_t L,
                           int64_t row_begin, int64_t row_end, const tca_cache_desc* c, const int32_t* idx,
                           const int64_t* offsets_dev, void* O, void* ws, cudaStream_t stream) {
  using Cfg = TcCfg<D>;
  const int64_t U = int64_t(prm->batch) * prm->n_kv_heads;
  const int G = prm->n_q_heads / prm->n_kv_heads;
  CUtensorMap mq, mk, mv, mck, mcv;
  if (!cached_map(&mq, Q, D, L, int64_t(prm->batch) * prm->n_q_heads) || !cached_map(&mk, K, D, L, U) ||
      !cached_map(&mv, V, D, L, U))
    return TCA_ERR_CUDA;
  if constexpr (kGather) {
    if (U * L >= (int64_t(1) << 31)) return TCA_ERR_UNSUPPORTED;   // row numbers are 32-bit
    mck = mk;   // not used by the gathering kernel
    mcv = mv;
  } else {
    // The cache maps cover the whole flattened cache (rows past the end read as zero); a tile that
    // reaches past a unit's visible prefix reads other finite rows, which the mask turns into exact zeros.
    if (!cached_map(&mck, c->k, D, c->rows_total, 0) || !cached_map(&mcv, c->v, D, c->rows_total, 0))
      return TCA_ERR_CUDA;
  }
  auto kern = prefill_tc_kernel<D, kGather>;
  TCA_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::bytes));
  const int tile0 = int(row_begin / BM);
  const int n_qtiles = int((row_end - row_begin + BM - 1) / BM);
  const int pairs = (G + 1) / 2;
  const int64_t n_ctas = int64_t(n_qtiles) * U * pairs;
  if (n_ctas >= (int64_t(1) << 31)) return TCA_ERR_UNSUPPORTED;
  const int64_t mb = num_blocks(prm, L) * prm->block;
  const int32_t* pos = kGather ? idx : static_cast<const int32_t*>(c->pos);
  const int64_t* state = kGather ? offsets_dev : static_cast<const int64_t*>(c->state);
  return launch_pdl(kern, dim3(static_cast<unsigned>(n_ctas)), dim3(kThreads), size_t(Cfg::bytes), stream, mq, mk, mv,
                    mck, mcv, pos, state, L, prm->n_q_heads, prm->n_kv_heads, prm->window, mb,
                    prm->sm_scale * 1.4426950408889634f, static_cast<__nv_bfloat16*>(O), static_cast<int*>(ws),
                    n_qtiles, pairs, tile0, (prm->flags & TCA_FLAG_PREFILL_BAND_FIRST) ? 1 : 0,
                    static_cast<const __nv_bfloat16*>(K), static_cast<const __nv_bfloat16*>(V));
}

template <int D>
int launch_prefill_tc(const tca_params* prm, const void* Q, const void* K, const void* V, int64_t L,
                      int64_t row_begin, int64_t row_end, const tca_cache_desc* c, void* O, void* ws,
                      cudaStream_t stream) {
  return launch_prefill_tc_impl<D, false>(prm, Q, K, V, L, row_begin, row_end, c, nullptr, nullptr, O, ws, stream);
}
template <int D>
int launch_prefill_tc_gather(const tca_params* prm, const void* Q, const void* K, const void* V, int64_t L,
                             int64_t row_begin, int64_t row_end, const int32_t* idx, const int64_t* offsets_dev,
                             void* O, void* ws, cudaStream_t stream) {
  return launch_prefill_tc_impl<D, true>(prm, Q, K, V, L, row_begin, row_end, nullptr, idx, offsets_dev, O, ws,
                                         stream);
}

template int launch_prefill_tc<64>(const tca_params*, const void*, const void*, const void*, int64_t, int64_t,
                                   int64_t, const tca_cache_desc*, void*, void*, cudaStream_t);
template int launch_prefill_tc<128>(const tca_params*, const void*, const void*, const void*, int64_t, int64_t,
                                    int64_t, const tca_cache_desc*, void*, void*, cudaStream_t);

template int launch_prefill_tc_gather<64>(const tca_params*, const void*, const void*, const void*, int64_t, int64_t,
                                          int64_t, const int32_t*, const int64_t*, void*, void*, cudaStream_t);
template int launch_prefill_tc_gather<128>(const tca_params*, const void*, const void*, const void*, int64_t, int64_t,
                                           int64_t, const int32_t*, const int64_t*, void*, void*, cudaStream_t);

}  // namespace tca
