// Pieces shared by the decode kernels: the view of a unit's cache segment, the slicing of
// its rows over CTAs and the packing of the per-slice partial results.
#pragma once
#include "common.cuh"

namespace tca {

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
  // rows [r, r+n) are physically contiguous for the returned count (<= n)
  __device__ __forceinline__ int64_t run(int64_t r, int64_t n) const {
    if (r < n_global) return min(n, n_global - r);
    int64_t slot = tail_head + (r - n_global);
    if (slot >= tail_cap) slot -= tail_cap;
    return min(n, tail_cap - slot);
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

// CTAs of unit u: ceil(len / target).  Partials are packed unit after unit.  The unit's rows
// are dealt evenly: slice i covers [i*len/n, (i+1)*len/n), never empty and never longer than
// target, so no CTA carries a short remainder while the others carry full slices.
__device__ __forceinline__ int n_parts(int64_t len, int target) { return int((len + target - 1) / target); }
__device__ __forceinline__ int64_t slice_begin(int64_t len, int n, int i) { return (int64_t(i) * len) / n; }

// Sum of n_parts over the units before u.  Called by whole warps (all 32 lanes active); every
// lane returns the total.  It needs no CTA-wide barrier, so a producer warp can skip it.
__device__ __forceinline__ int partial_base(const int64_t* state, int u, int target) {
  int part = 0;
  for (int v = int(threadIdx.x & 31u); v < u; v += 32) {
    const int64_t* st = state + size_t(v) * TCA_STATE_WORDS;
    part += n_parts(st[TCA_ST_N_GLOBAL] + st[TCA_ST_N_TAIL], target);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
  return part;
}

// Which slice a CTA of the attention kernels works on.  blockIdx.x counts the slices of all units,
// unit after unit, and exactly as many CTAs are launched as there are slices: a CTA without work
// would still hold its SM until its dependency wait returns, and the slices behind it in launch
// order would start that much later (with a grid of units x longest-unit-slices, 124 of 272 CTAs
// were idle at the benchmark's mix of budgets and the last slices started 4-5 us late).
struct SliceId {
  int u;           // unit, -1 if blockIdx.x lies beyond the last slice
  int part;        // slice within the unit
  int np;          // slices of the unit
  int base_slot;   // slices of all earlier units = first partial slot of this unit
  UnitView uv;     // the unit's state words, fetched in the same trip to memory as the search
};
// Called by every thread of the CTA (it contains a CTA-wide barrier); warp 0 does the search, 32
// units per round with a warp scan.
__device__ __forceinline__ SliceId find_slice(const int64_t* state, int n_units, int target, int64_t tail_cap,
                                              SliceId* shared_slot) {
  if (threadIdx.x < 32) {
    const int lane = int(threadIdx.x), lin = int(blockIdx.x);
    int offset = 0;
    bool found = false;
    for (int v0 = 0; v0 < n_units && !found; v0 += 32) {
      const int v = v0 + lane;
      int npv = 0;
      UnitView mine{};
      if (v < n_units) {
        mine = load_unit(state, v, tail_cap);
        npv = n_parts(mine.len(), target);
      }
      int incl = npv;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
      }
      const unsigned hit = __ballot_sync(0xffffffffu, lin < offset + incl);
      if (hit) {
        const int l = __ffs(hit) - 1;
        const int excl = __shfl_sync(0xffffffffu, incl - npv, l), npl = __shfl_sync(0xffffffffu, npv, l);
        if (lane == l) *shared_slot = SliceId{v, lin - offset - excl, npl, offset + excl, mine};
        found = true;
      }
      offset += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (!found && lane == 0) shared_slot->u = -1;
  }
  __syncthreads();
  return *shared_slot;
}

}  // namespace tca
