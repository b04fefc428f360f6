// Shared declarations of the TCA-Attention kernels (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tca.h"

namespace tca {

constexpr int kStatusTimeout = 1;  // values of a workspace's status word
constexpr int kStatusBounds = 2;

// Range-checked build (-DTCA_DEBUG_BOUNDS): every index or offset that a kernel takes from memory
// (selected token indices, per-block counts, ring slots, cache rows) is compared with its range
// before it is used; an access that fails the test is skipped and the first failure is recorded
// where the host can read it (word 0 of the workspace, or the reserved state word of the unit for
// the calls that take no workspace).  Nothing traps.  In the normal build the checks compile away.
#ifdef TCA_DEBUG_BOUNDS
constexpr bool kDebugBounds = true;
#else
constexpr bool kDebugBounds = false;
#endif
enum { kBoundsSelectedIndex = 1, kBoundsBlockCount = 2, kBoundsRingSlot = 3, kBoundsCacheRow = 4,
       kBoundsGlobalRegion = 5 };
constexpr int kMaxGroup = 8;    // query heads per KV head
constexpr int kMaxBlock = 128;  // b

// ------------------------------------------------------------------ host-side checks
#define TCA_CHECK_ARG(cond) \
  do {                      \
    if (!(cond)) return TCA_ERR_INVALID_ARG; \
  } while (0)

#define TCA_CHECK_CUDA(expr)                      \
  do {                                            \
    cudaError_t _e = (expr);                      \
    if (_e != cudaSuccess) return TCA_ERR_CUDA;   \
  } while (0)

inline int check_launch() { return cudaGetLastError() == cudaSuccess ? TCA_OK : TCA_ERR_CUDA; }

inline bool is_pow2(int64_t x) { return x > 0 && (x & (x - 1)) == 0; }
inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Validates the hyper-parameters every entry point shares.
int check_params(const tca_params* prm);

inline int64_t num_blocks(const tca_params* prm, int64_t L) {
  return L > prm->window ? (L - prm->window) / prm->block : 0;
}
inline int num_counts(const tca_params* prm) {  // |{1, 2, 4, ..., b}|
  int n = 0;
  for (int b = prm->block; b; b >>= 1) ++n;
  return n;
}
inline size_t elt_size(int dtype) { return dtype == TCA_BF16 ? 2 : 4; }

// ------------------------------------------------------------------ workspace layouts
// score: logits [U][G][L] double, then partials [U][n_chunks][G][2] double.
constexpr int kScoreChunkRows = 1024;  // rows of K per CTA of the logit kernel
// Streaming multiprocessors of the current device, looked up once per device (api.cu).
constexpr int kMaxDevices = 64;
int sm_count();
int64_t l2_bytes();   // L2 cache size of the current device

struct ScoreWs {
  double* logits;
  double* partials;
  int64_t n_chunks;
  size_t bytes;
};
ScoreWs score_ws_layout(const tca_params* prm, int64_t L, void* ws);

// select: a 256-byte header (word 0: status, range-checked build), hkey [U][m] uint64, t [U][m] int32.
struct SelectWs {
  int* status;
  unsigned long long* hkey;
  int32_t* t;
  size_t bytes;
};
SelectWs select_ws_layout(const tca_params* prm, int64_t L, void* ws);

// decode: a 256-byte header (word 0: sticky error flag, set when a bounded wait gave up)
// followed by one partial (acc[d], max, sum) per (slice, query head of the group).
constexpr int kDecodeChunkRows = 256;  // smallest slice of cache rows one CTA takes
constexpr size_t kDecodeHeaderBytes = 256;
struct DecodeWs {
  int* status;
  float* partial;     // [n_chunks_max][G][d + 2]
  int64_t n_chunks_max;
  size_t bytes;
};
DecodeWs decode_ws_layout(const tca_params* prm, int64_t rows_total, int64_t n_units, void* ws);

// ------------------------------------------------------------------ device helpers
#ifdef __CUDACC__

// Programmatic dependent launch: a kernel launched with launch_pdl may start while its
// predecessor in the stream is still draining; pdl_wait() blocks until the predecessor has
// completed and its writes are visible, so it must come before the first dependent access.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }

template <typename... KArgs, typename... Args>
inline int launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...) == cudaSuccess ? TCA_OK : TCA_ERR_CUDA;
}

template <typename T>
struct Elt;
template <>
struct Elt<float> {
  static constexpr int kDtype = TCA_F32;
};
template <>
struct Elt<__nv_bfloat16> {
  static constexpr int kDtype = TCA_BF16;
};

// Record a failed range check in a workspace header: word 0 = kStatusBounds, word 1 = which check,
// bytes 8..15 = the offending value.  Only the first failure is kept.
__device__ __forceinline__ void report_bounds_ws(int* status, int which, long long value) {
  if (atomicCAS(status, 0, kStatusBounds) == 0) {
    status[1] = which;
    reinterpret_cast<long long*>(status)[1] = value;
  }
}
// The same for the calls without a workspace: the unit's reserved state word takes
// (which << 56) | (value & 2^56 - 1); zero means "no failure".
__device__ __forceinline__ void report_bounds_state(int64_t* unit_state, int which, long long value) {
  const unsigned long long word = (static_cast<unsigned long long>(which) << 56) |
                                  (static_cast<unsigned long long>(value) & 0x00FFFFFFFFFFFFFFull);
  atomicCAS(reinterpret_cast<unsigned long long*>(unit_state + TCA_ST_RESERVED), 0ull, word);
}

// Order-preserving map double -> uint64 (a < b  <=>  key(a) < key(b); -0 < +0).
__device__ __forceinline__ unsigned long long ordered_key(double x) {
  unsigned long long u = static_cast<unsigned long long>(__double_as_longlong(x));
  return (u & 0x8000000000000000ull) ? ~u : (u | 0x8000000000000000ull);
}

__device__ __forceinline__ float bf16_lo(uint32_t packed) { return __uint_as_float(packed << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t packed) { return __uint_as_float(packed & 0xFFFF0000u); }

__device__ __forceinline__ double shfl_xor_double(double v, int mask) {
  int lo = __double2loint(v), hi = __double2hiint(v);
  lo = __shfl_xor_sync(0xffffffffu, lo, mask);
  hi = __shfl_xor_sync(0xffffffffu, hi, mask);
  return __hiloint2double(hi, lo);
}
__device__ __forceinline__ double shfl_double(double v, int src) {
  int lo = __double2loint(v), hi = __double2hiint(v);
  lo = __shfl_sync(0xffffffffu, lo, src);
  hi = __shfl_sync(0xffffffffu, hi, src);
  return __hiloint2double(hi, lo);
}
__device__ __forceinline__ unsigned long long shfl_xor_u64(unsigned long long v, int mask) {
  return static_cast<unsigned long long>(
      __double_as_longlong(shfl_xor_double(__longlong_as_double(static_cast<long long>(v)), mask)));
}

// Top-t of up to 128 keys held 4 per lane by one warp: MSB-first radix select on the
// order-preserving 64-bit keys (radix 2, histogram = warp ballots), then ties at the
// threshold go to the lowest token index.  Token i lives in lane i % 32, slot i / 32.
// Returns per-slot keep flags as a 4-bit mask; `n_valid` tokens exist, t <= n_valid.
__device__ __forceinline__ unsigned radix_select_top_t(const unsigned long long (&key)[4], int n_valid,
                                                       int t, int lane) {
  unsigned alive = 0;
  unsigned long long k_or = 0ull, k_and = ~0ull;
#pragma unroll
  for (int s = 0; s < 4; ++s)
    if (s * 32 + lane < n_valid) {
      alive |= 1u << s;
      k_or |= key[s];
      k_and &= key[s];
    }
  // bits above the highest bit in which two keys differ cannot decide anything: skip them
  const unsigned or_hi = __reduce_or_sync(0xffffffffu, unsigned(k_or >> 32));
  const unsigned or_lo = __reduce_or_sync(0xffffffffu, unsigned(k_or));
  const unsigned and_hi = __reduce_and_sync(0xffffffffu, unsigned(k_and >> 32));
  const unsigned and_lo = __reduce_and_sync(0xffffffffu, unsigned(k_and));
  const unsigned long long diff = ((unsigned long long)(or_hi ^ and_hi) << 32) | (or_lo ^ and_lo);
  unsigned keep = 0;
  int need = t;
  int n_alive = n_valid;
  // Invariant: `need` more tokens must come from the alive set; all alive keys share the
  // bits above the current one.
  for (int bit = diff ? 63 - __clzll(diff) : -1; bit >= 0 && need > 0 && n_alive > need; --bit) {
    unsigned ones = 0;
    int n_ones = 0;
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      const bool one = ((alive >> s) & 1u) && ((key[s] >> bit) & 1ull);
      if (one) ones |= 1u << s;
      n_ones += __popc(__ballot_sync(0xffffffffu, one));
    }
    if (n_ones >= need) {
      alive = ones;              // the threshold has this bit set; zeros are out
      n_alive = n_ones;
    } else {
      keep |= ones;              // all ones are above the threshold
      need -= n_ones;
      alive &= ~ones;
      n_alive -= n_ones;
    }
  }
  // Whatever is still alive is either all kept (n_alive <= need) or a set of equal keys
  // of which the `need` lowest indices are kept.
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    bool a = (alive >> s) & 1u;
    unsigned bal = __ballot_sync(0xffffffffu, a);
    int before = __popc(bal & ((1u << lane) - 1u));
    if (a && before < need) keep |= 1u << s;
    need -= min(need, __popc(bal));
  }
  return keep;
}

#endif  // __CUDACC__

}  // namespace tca
