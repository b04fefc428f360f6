/*
 * tca.h -- C ABI of the B200-native hot path of TCA-Attention
 * (Training-free Context-adaptive Attention): score -> select -> compact ->
 * sparse attention (prefill, decode) -> append/compress while decoding.
 *
 * Conventions
 *   - Every pointer is labelled HOST or DEVICE.  All device buffers (inputs, outputs,
 *     cache, workspace) are allocated and freed by the caller; the library calls no
 *     allocator.  What it keeps between calls is limited to: the built-in scratch array of
 *     tca_attn_decode_static (and its per-device address), a small cache of encoded TMA
 *     tensor maps keyed by buffer address and shape, and per-device constants (SM count,
 *     L2 cache size).  The bf16 decode kernel asks the L2 to keep part of the cache it reads
 *     (eviction-priority hints on its loads; nothing is set on the device or the context).
 *   - Tensors are row-major with the head dimension contiguous:
 *       Q [batch, n_q_heads, L, head_dim]      K, V [batch, n_kv_heads, L, head_dim]
 *     A "unit" is one (sequence, KV head) pair, u = seq * n_kv_heads + kv_head; the G =
 *     n_q_heads / n_kv_heads query heads kv_head*G .. kv_head*G+G-1 share it.
 *   - Device work is enqueued on `stream` (a cudaStream_t passed as void*); no call
 *     synchronises the host except the three that read a status back (tca_ws_status,
 *     tca_cache_status, tca_decode_static_status).  Outputs are valid once the stream has
 *     been synchronised.
 *   - Status words.  Word 0 of the prefill, decode, select and calibration workspaces is a
 *     STICKY status word: zero it once after allocating (a zero-filled workspace is fine); a
 *     kernel sets it when one of its bounded device-side waits gives up (or, in the
 *     range-checked build, when an index is out of range) and nothing in the library clears
 *     it.  While it is set, the tensor-core kernels return at once without computing.  After
 *     a non-zero status, zero the whole workspace before using it again.
 *   - Return value: TCA_OK or a negative error.  Argument errors are detected on the
 *     host before anything is launched and leave every output untouched.  Unsupported
 *     shapes return TCA_ERR_UNSUPPORTED; nothing ever falls back to the CPU.
 *   - Identical inputs give bit-identical outputs (fixed split counts, fixed reduction
 *     order, no floating-point atomics).
 *   - Token positions are 0-based.
 */
#ifndef TCA_H_
#define TCA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  TCA_OK = 0,
  TCA_ERR_INVALID_ARG = -1, /* NULL / misaligned pointer, inconsistent sizes            */
  TCA_ERR_UNSUPPORTED = -2, /* shape or dtype outside what the kernels implement        */
  TCA_ERR_WORKSPACE = -3,   /* workspace smaller than tca_workspace_bytes() reports     */
  TCA_ERR_CUDA = -4,        /* a CUDA runtime call or a launch failed                   */
  TCA_ERR_TIMEOUT = -5,     /* a bounded device-side wait gave up (see tca_ws_status)   */
  TCA_ERR_CAPACITY = -6,    /* a cache region would overflow                            */
  TCA_ERR_SCRATCH_LIMIT = -7, /* problem larger than the built-in scratch of a *_static call */
  TCA_ERR_BOUNDS = -8        /* range-checked build only: an index or offset was out of range  */
};

enum { TCA_F32 = 0, TCA_BF16 = 1 };

/* tca_params.flags */
enum {
  /* run the prefill on the FP32 pipes even for bf16 inputs (the slow reference kernel the
   * tensor-core kernel is cross-checked against) */
  TCA_FLAG_PREFILL_SIMT = 1,
  /* Selection variants of the paper's ablations (appendix "Ablations on Concentration Index" and
   * "Effectiveness of Local-context Redundancy Metric") and a flat top-B; at most one of the three.
   * The paper names them without formulas; the definitions here are this library's reading.
   *   ENTROPY_INDEX  the concentration term of Eq. 6 becomes the block entropy
   *                  H_j = -sum_i p_i ln p_i, p_i = s_i / sum_{B_j} s  (in place of 1 - sum p_i^2)
   *   RANDOM_ORDER   blocks are ranked by a hash of (tca_params.seed, unit, block index) instead of
   *                  h_j: key = SplitMix64(SplitMix64(seed * 2^32 + unit) + j) >> 11, ascending,
   *                  ties to the lower block; h_out receives key * 2^-53
   *   FLAT_TOPB      no blocks: the n_sel = sum_k k * n_k highest-scoring tokens among the candidates
   *                  [0, m*b) are selected, ties to the lower position; h_out and t_out are not written */
  TCA_FLAG_ENTROPY_INDEX = 2,
  TCA_FLAG_RANDOM_ORDER = 4,
  TCA_FLAG_FLAT_TOPB = 8,
  /* prefill: walk each query tile's own window band before the selected keys (see tca_attn_prefill) */
  TCA_FLAG_PREFILL_BAND_FIRST = 16
};

enum {
  TCA_OP_SCORE = 0, TCA_OP_SELECT = 1, TCA_OP_COMPACT = 2,
  TCA_OP_PREFILL = 3, TCA_OP_DECODE = 4, TCA_OP_APPEND = 5, TCA_OP_CALIB = 6, TCA_OP_SCORE_SELECT = 7
};

/* Hyper-parameters of one attention layer (Algorithm 2, REQUIRE line). */
typedef struct tca_params {
  int32_t batch;      /* sequences                                                      */
  int32_t n_q_heads;  /* multiple of n_kv_heads, group size G <= 8                      */
  int32_t n_kv_heads;
  int32_t head_dim;   /* d_h: 64 or 128                                                 */
  int32_t block;      /* b: power of two, 1..128 (Section 4.1)                          */
  int32_t window;     /* w >= 0: local subset size (Section 4); the prefill needs w >= 1 */
  float alpha;        /* balance of Eq. 6, in [0, 1]                                    */
  float sm_scale;     /* 1/sqrt(d_h) of Eqs. 2 and 5                                    */
  int32_t dtype;      /* TCA_F32 or TCA_BF16: element type of Q, K, V, O and the cache  */
  int32_t flags;      /* 0, or TCA_FLAG_* bits                                          */
  int32_t seed;       /* TCA_FLAG_RANDOM_ORDER: seed of the block order; otherwise unused    */
} tca_params;

/* Number of int64 words per unit in tca_cache_desc.state. */
#define TCA_STATE_WORDS 8
enum {
  TCA_ST_SEG_START = 0,  /* first cache row of the unit's segment                       */
  TCA_ST_GLOBAL_CAP = 1, /* rows reserved for the global subset                         */
  TCA_ST_N_GLOBAL = 2,   /* rows of the global subset in use                            */
  TCA_ST_TAIL_HEAD = 3,  /* ring slot of the oldest tail token                          */
  TCA_ST_N_TAIL = 4,     /* tokens in the tail ring                                     */
  TCA_ST_SEQ_LEN = 5,    /* tokens seen so far = position of the next token             */
  TCA_ST_T_KEEP = 6,     /* tokens kept from a block compressed while decoding          */
  TCA_ST_RESERVED = 7
};

/*
 * The retained KV cache ([K^G; K^L] of Eq. 2 kept across decode steps, Section 4.2 last
 * paragraph).  All heads live in one flattened buffer with per-unit segments (the
 * variable-length multi-head layout of Appendix C).  A unit's segment is
 *     [ global region: global_cap rows | tail ring: tail_cap rows ]
 * The global region holds the selected tokens S in ascending position; the ring holds
 * the always-kept recent tokens, oldest at slot tail_head.
 *
 * The struct and its host arrays are owned by the caller and live in HOST memory; the
 * k/v/pos/state buffers are DEVICE memory.  The host arrays mirror the device state
 * words; lengths depend only on L, the number of appended tokens and the budget table,
 * never on data, so both sides advance in lock step and no call reads the device back.
 */
typedef struct tca_cache_desc {
  void* k;              /* DEVICE [rows_total, head_dim]                                */
  void* v;              /* DEVICE [rows_total, head_dim]                                */
  int32_t* pos;         /* DEVICE [rows_total]: original position of every row          */
  int64_t* state;       /* DEVICE [n_units * TCA_STATE_WORDS]                           */
  int64_t rows_total;
  int64_t n_units;      /* batch * n_kv_heads                                           */
  int64_t tail_cap;     /* ring capacity per unit; >= window + block for decoding       */
  int64_t* seg_start;   /* HOST [n_units]  set by the caller                            */
  int64_t* global_cap;  /* HOST [n_units]  set by the caller                            */
  int64_t* n_global;    /* HOST [n_units]  maintained by the library                    */
  int64_t* tail_head;   /* HOST [n_units]  maintained by the library                    */
  int64_t* n_tail;      /* HOST [n_units]  maintained by the library                    */
  int64_t* seq_len;     /* HOST [n_units]  maintained by the library                    */
  int64_t* t_keep;      /* HOST [n_units]  set by the caller (tbar of tca_budget_resolve)*/
} tca_cache_desc;

const char* tca_strerror(int status);
int tca_version(void);

/* Bit flags describing how the library was built. */
enum { TCA_BUILD_DEBUG_BOUNDS = 1 };
int tca_build_info(void);

/*
 * Budget map of Eq. 7 (Section 4.2), resolved on the host.
 *   p       HOST [n_kv_heads, nK] double: configuration over K = {1, 2, 4, ..., 2^(nK-1)};
 *           every row must be non-negative and sum to 1 within 1e-9.
 *   m       number of blocks, m = max(0, floor((L - window) / block)).
 *   n_k     HOST out [n_kv_heads, nK]: blocks that get retain count k.  floor(m * p_k) as
 *           in Eq. 7, then the shortfall m - sum_k floor(m p_k) is handed out one each to
 *           the largest fractional parts (ties to the larger k), so that Psi has exactly
 *           m entries.
 *   n_sel   HOST out [n_kv_heads]: size of the global subset, sum_k k * n_k.
 *   tbar    HOST out [n_kv_heads]: floor(sum_k k * p_k), the decode-time retain count.
 */
int tca_budget_resolve(const double* p, int32_t n_kv_heads, int32_t nK, int64_t m,
                       int32_t* n_k, int64_t* n_sel, int32_t* tbar);

/* Bytes of DEVICE workspace `op` needs for sequence length L (for TCA_OP_DECODE and
 * TCA_OP_APPEND, L is the total number of cache rows).  0 for an invalid request. */
size_t tca_workspace_bytes(const tca_params* prm, int64_t L, int op);

/*
 * Token importance, Eq. 5 / Algorithm 2 line 1:  s = softmax(q_L K^T * sm_scale) over all
 * L keys, per query head; the G distributions of a KV head's group are averaged.
 *   q_last    DEVICE [batch, n_q_heads, head_dim]   query of the last token
 *   K         DEVICE [batch, n_kv_heads, L, head_dim]
 *   logscore  DEVICE out [batch, n_kv_heads, L] double: log s (s itself underflows at
 *             long L).  Dot products are accumulated in fp64.
 *   ws        DEVICE workspace, tca_workspace_bytes(prm, L, TCA_OP_SCORE), 256-B aligned
 */
int tca_score(const tca_params* prm, const void* q_last, const void* K, int64_t L,
              double* logscore, void* ws, size_t ws_bytes, void* stream);

/*
 * Core-context selection, Eqs. 6-8 / Algorithm 2 lines 2-6, one selection per unit.
 * Blocks j < m of b tokens; h_j by Eq. 6; blocks ranked ascending by (h_j, j);
 * t_j = Psi[rank_j]; the t_j tokens of block j with the largest score are kept, ties to
 * the lower position.
 *   logscore     DEVICE [batch, n_kv_heads, L] double
 *   n_k          HOST [n_kv_heads, nK] from tca_budget_resolve (shared across the batch)
 *   idx          DEVICE out int32, flattened: unit u owns idx[offsets[u] .. offsets[u+1]),
 *                positions ascending
 *   offsets_dev  DEVICE [n_units + 1] int64: exclusive prefix of n_sel over units
 *   h_out        DEVICE out, optional (NULL to skip) [n_units, m] double
 *   t_out        DEVICE out, optional (NULL to skip) [n_units, m] int32
 */
int tca_select(const tca_params* prm, const double* logscore, int64_t L,
               const int32_t* n_k, int32_t nK, int32_t* idx, const int64_t* offsets_dev,
               double* h_out, int32_t* t_out, void* ws, size_t ws_bytes, void* stream);

/*
 * tca_score followed by tca_select in one call and fewer launches (Eqs. 5-8, Algorithm 2 lines
 * 1-6): the kernel that turns logits into log s also forms the block metric of Eq. 6 for the
 * blocks it holds, so the scores are not read back for it.  Arguments are those of the two calls;
 * ws is one workspace of tca_workspace_bytes(prm, L, TCA_OP_SCORE_SELECT) bytes.  logscore, idx,
 * h_out and t_out receive bit for bit what the two separate calls write.
 */
int tca_score_select(const tca_params* prm, const void* q_last, const void* K, int64_t L,
                     const int32_t* n_k, int32_t nK, double* logscore, int32_t* idx,
                     const int64_t* offsets_dev, double* h_out, int32_t* t_out,
                     void* ws, size_t ws_bytes, void* stream);

/* REQUIRED once after filling the descriptor and before any other call that takes it:
 * uploads the host mirror of `cache` (seg_start, global_cap, n_global, tail_head, n_tail,
 * seq_len, t_keep) into cache->state and zero-fills cache->k and cache->v.  The zero-fill is
 * not optional: the attention kernels multiply rows that are not in use by an exactly zero
 * weight, which cancels only finite values, so a cache that skips this call can turn
 * uninitialised memory into NaNs in the output without any error being reported. */
int tca_cache_init(const tca_params* prm, tca_cache_desc* cache, void* stream);

/*
 * Gather [K^G; K^L] (Eq. 2; "parallel tokens gathering", Appendix C): copy the rows of
 * the selected set S into each unit's global region and the always-kept tail [m*b, L)
 * into its ring, with their positions.  Sets n_global = n_sel, n_tail = L - m*b,
 * tail_head = 0, seq_len = L on both the host mirror and the device state.
 *   idx, offsets_dev  as written by / given to tca_select
 *   offsets_host      HOST [n_units + 1] copy of offsets_dev
 * TCA_ERR_CAPACITY if a unit's selection exceeds global_cap or its tail exceeds tail_cap.
 */
int tca_compact_kv(const tca_params* prm, const void* K, const void* V, int64_t L,
                   const int32_t* idx, const int64_t* offsets_dev, const int64_t* offsets_host,
                   tca_cache_desc* cache, void* stream);

/*
 * The same compaction for the retained rows whose position lies in [pos_begin, pos_end) only
 * (0 <= pos_begin < pos_end <= L, else TCA_ERR_INVALID_ARG), for a caller whose K and V arrive
 * in pieces: rows of K and V outside the range are not read.  Every call writes all positions
 * and the state words (they depend on the selection alone), so after the call for positions
 * [0, p) the cache serves tca_attn_prefill_rows for query rows below p; calls whose ranges cover
 * [0, L), in any order, leave the cache bit-identical to one tca_compact_kv.  Other arguments
 * and errors as tca_compact_kv.
 */
int tca_compact_kv_range(const tca_params* prm, const void* K, const void* V, int64_t L,
                         int64_t pos_begin, int64_t pos_end,
                         const int32_t* idx, const int64_t* offsets_dev, const int64_t* offsets_host,
                         tca_cache_desc* cache, void* stream);

/*
 * Sparse causal attention of the prefill, Eq. 2 / Algorithm 2 line 7.  Query i of a head
 * attends to {j <= i : j in S or j >= c_i}, c_i = min(max(0, i - w + 1), m*b): its own
 * last w keys (read from K, V) plus the selected keys before them (read from the cache's
 * global region); every key is counted once.  O has the shape of Q.
 *   ws   DEVICE workspace, tca_workspace_bytes(prm, L, TCA_OP_PREFILL); word 0 is the sticky
 *        status word (see Conventions), readable with tca_ws_status.
 * prm->window must be >= 1 (TCA_ERR_UNSUPPORTED otherwise): with w = 0 a query that is not
 * itself selected would attend to nothing, and Eq. 2 has no value for an empty key set.
 */
int tca_attn_prefill(const tca_params* prm, const void* Q, const void* K, const void* V,
                     int64_t L, const tca_cache_desc* cache, void* O,
                     void* ws, size_t ws_bytes, void* stream);

/*
 * The same attention (Eq. 2) for the query rows [row_begin, row_end) of every head only; the
 * other rows of O are not touched.  A row's result does not depend on which call computed it:
 * calls over a partition of [0, L) leave O bit-identical to one tca_attn_prefill call.  It
 * lets a caller whose Q arrives (or whose O leaves) in pieces overlap the transfers with the
 * arithmetic.  Q, K, V, O, L, cache and ws are those of tca_attn_prefill (Q and O are still
 * addressed as the full [batch, n_q_heads, L, d] arrays); row_begin must be a multiple of
 * TCA_PREFILL_ROW_ALIGN, 0 <= row_begin < row_end <= L, else TCA_ERR_INVALID_ARG.  Calls that
 * may run concurrently need a workspace each.
 */
#define TCA_PREFILL_ROW_ALIGN 128
int tca_attn_prefill_rows(const tca_params* prm, const void* Q, const void* K, const void* V,
                          int64_t L, int64_t row_begin, int64_t row_end,
                          const tca_cache_desc* cache, void* O,
                          void* ws, size_t ws_bytes, void* stream);

/*
 * The same attention (Eq. 2) without a cache: the selected keys are fetched from K and V
 * themselves, by index, inside the attention kernel (Appendix C, "Memory Access Optimization":
 * gathering fused into the consumer instead of a separate compaction pass).  For a caller that
 * only prefills, or that builds the decode cache later: no tca_compact_kv, no cache memory.
 * O is bit-identical to tca_compact_kv + tca_attn_prefill_rows over the same selection; the
 * call takes about 1.5 times as long as the prefill over a compacted cache (every block of the
 * grid gathers its rows again), so it pays only where the cache memory cannot be afforded.
 *   idx, offsets_dev  DEVICE, as written by / given to tca_select: unit u's selected positions
 *                     are idx[offsets_dev[u] .. offsets_dev[u+1]), ascending; not modified
 *   row_begin, row_end  as in tca_attn_prefill_rows ([0, L) for the whole prefill)
 *   ws                as in tca_attn_prefill (sticky status word in word 0)
 * bf16 only, on the tensor-core kernel (TCA_ERR_UNSUPPORTED for TCA_F32 or
 * TCA_FLAG_PREFILL_SIMT, and when batch * n_kv_heads * L >= 2^31: the row coordinates of a
 * gather are 32-bit).  TCA_FLAG_PREFILL_BAND_FIRST applies.  The index set is trusted to hold
 * candidate positions (< m*b); the range-checked build verifies it (TCA_ERR_BOUNDS in ws).
 */
int tca_attn_prefill_gather(const tca_params* prm, const void* Q, const void* K, const void* V,
                            int64_t L, int64_t row_begin, int64_t row_end,
                            const int32_t* idx, const int64_t* offsets_dev, void* O,
                            void* ws, size_t ws_bytes, void* stream);

/*
 * Offline calibration, Algorithm 1 and Eq. 4 (Section 4.1, "Cumulative-Score Configuration
 * Determination").  It produces the per-head configuration p* that the functions above take
 * as an input.  Three calls:
 *
 *   tca_calib_colmean  c[u][k] = mean over the causally visible rows j >= k (the non-zero
 *                      entries of column k) of A = softmax(Q K^T * sm_scale), averaged over
 *                      the G query heads of the KV head (the aggregation of tca_score).
 *                      Q DEVICE [batch, n_q_heads, L, d], K DEVICE [batch, n_kv_heads, L, d],
 *                      bf16 only (TCA_ERR_UNSUPPORTED otherwise); colmean DEVICE [U][L] doubles;
 *                      ws DEVICE, tca_workspace_bytes(prm, L, TCA_OP_CALIB), word 0 is a status
 *                      word readable with tca_ws_status.  prm->block and prm->window are not
 *                      used.  Cost: two dense causal passes over Q K^T (row log-sum-exps, then column sums).
 *   tca_calib_score    a[u] of Eq. 4 for the selection (idx, offsets_dev) that tca_select wrote
 *                      for one candidate: the column means summed over everything the method
 *                      retains (the selected tokens and the always-kept tail [m*b, L), the
 *                      S_total of Section 4.3), as a share of the sum over all L tokens.  A
 *                      100 % budget scores exactly 1 and 1 - a is the share that is dropped.
 *                      a_out DEVICE [U] doubles.
 *   tca_calib_choose   HOST: the index of the candidate with the fewest selected tokens among
 *                      those with a[i] >= tau (the lowest index on a tie); if none reaches tau,
 *                      n_candidates - 1.  a, sizes HOST arrays of n_candidates entries.
 *
 * The caller runs tca_score once, then for every candidate p^i: tca_budget_resolve,
 * tca_select, tca_calib_score; then tca_calib_choose per KV head.
 */
int tca_calib_colmean(const tca_params* prm, const void* Q, const void* K, int64_t L,
                      double* colmean, void* ws, size_t ws_bytes, void* stream);
int tca_calib_score(const tca_params* prm, const double* colmean, int64_t L,
                    const int32_t* idx, const int64_t* offsets_dev, double* a_out, void* stream);
int tca_calib_choose(const double* a, const int64_t* sizes, int n_candidates, double tau);

/*
 * HOST: the candidate configurations of Eq. 3 (log-Gaussian over the retain counts 1, 2, 4, ...,
 * block, centred at mu^i = log2(1 + (i-1)(block-1)/(M-1)), i = 1..M, fixed sigma).  p_out HOST
 * [n_candidates][log2(block)+1] doubles, every row sums to 1.  block must be a power of two,
 * n_candidates >= 2, sigma > 0, else TCA_ERR_INVALID_ARG.
 */
int tca_calib_candidates(int block, int n_candidates, double sigma, double* p_out);

/*
 * One decode step, Eq. 2 with a single query per head over the whole retained cache
 * (global region + tail ring) of its KV head.
 *   q  DEVICE [batch, n_q_heads, head_dim]     O  DEVICE out, same shape
 *   ws DEVICE workspace, tca_workspace_bytes(prm, cache->rows_total, TCA_OP_DECODE), zeroed
 *      once after allocating.  Word 0 is the sticky status word (tca_ws_status).  Every CTA
 *      leaves a partial result for its slice of a unit's rows in the workspace and a second,
 *      small kernel merges each unit's partials in slice order.  Calls that share a workspace
 *      must not overlap on the GPU.
 */
int tca_attn_decode(const tca_params* prm, const void* q, const tca_cache_desc* cache,
                    void* O, void* ws, size_t ws_bytes, void* stream);

/*
 * Append one token per sequence and compress when a block leaves the window (Section 4.2,
 * "Online Token Selection in Decoding Stage").  The token goes to the tail ring; if the
 * ring then holds window + block tokens, its oldest `block` tokens are scored with the
 * current query (Eq. 5 restricted to the block, averaged over the query group), the top
 * t_keep move to the end of the global region in ascending position and the rest are
 * dropped.  Call before tca_attn_decode of the same step.
 *   k_new, v_new  DEVICE [batch, n_kv_heads, head_dim]
 *   q_cur         DEVICE [batch, n_q_heads, head_dim]  query of the appended token
 * TCA_ERR_CAPACITY if the global region of a unit would overflow.
 */
int tca_cache_append(const tca_params* prm, tca_cache_desc* cache, const void* k_new,
                     const void* v_new, const void* q_cur, void* stream);

/* Size of the scratch array built into the library image for tca_attn_decode_static. */
#define TCA_DECODE_STATIC_SCRATCH_BYTES (16u << 20)

/*
 * tca_attn_decode for callers that must not allocate.  (The paper has no counterpart;
 * this is a deployment convenience.)  Some hosts of this library cannot hand it a
 * workspace: a plug-in inside a serving engine that has already claimed all device memory
 * for its own pool, a latency-critical loop in which cudaMalloc's implicit device-wide
 * synchronisation is not acceptable, or glue code that simply has no allocator at hand.
 * This variant computes exactly what tca_attn_decode computes, with the split-KV partial
 * results kept in a fixed TCA_DECODE_STATIC_SCRATCH_BYTES (16 MiB) array that is part of
 * the library image: every GPU that loads the library holds those 16 MiB until the
 * process exits, and the call performs no cudaMalloc, cudaFree or other allocation.
 *
 *   q, cache, O, stream   as for tca_attn_decode; inputs and outputs still belong to the
 *                         caller.
 *   Limit   the call needs what tca_workspace_bytes(prm, rows_total, TCA_OP_DECODE) reports:
 *             256 + roundup256((rows_total / 256 + 2 * n_units + 1) * G * (head_dim + 2) * 4)
 *           bytes (roundup256 = up to a multiple of 256; rows_total / 256 rounds down).  A
 *           cache for which that exceeds the array (about 2 million rows at G = 4,
 *           head_dim = 128) is refused with TCA_ERR_SCRATCH_LIMIT and nothing is launched.
 *           Use tca_attn_decode with a workspace of your own for larger caches.
 *   Set-up  the first call on each device looks up the array's device address (with that
 *           device current) and remembers it; make that first call outside any stream
 *           capture.
 *   Sharing every call on a device uses the same array, which keeps the previous call's
 *           contents.  Nothing in it has to be cleared by the caller: the status word is zero
 *           when the library is loaded and tca_decode_static_status clears it after reporting
 *           a failure, and each partial is written before it is read.  Two calls that overlap
 *           on the GPU (different streams, or different threads without ordering) race on
 *           the array and corrupt each other: serialise them.
 *   Errors  the status word of this variant lives inside the array, where tca_ws_status
 *           cannot reach it; tca_decode_static_status reads it instead.
 */
int tca_attn_decode_static(const tca_params* prm, const void* q, const tca_cache_desc* cache,
                           void* O, void* stream);

/* Synchronise `stream`, then report whether a bounded wait gave up in a tca_attn_decode_static
 * call on the current device since the last time this was asked: TCA_OK, or TCA_ERR_TIMEOUT (the
 * outputs of the calls since then are not valid).  After TCA_ERR_TIMEOUT the status word in the
 * array has been cleared and the entry point can be used again.  Performs no allocation.  (No
 * counterpart in the paper.) */
int tca_decode_static_status(void* stream);

/*
 * Range-checked build only (tca_build_info() & TCA_BUILD_DEBUG_BOUNDS; in the normal build this
 * always returns TCA_OK).  tca_compact_kv and tca_cache_append take no workspace, so their range
 * checks record a failure in the reserved state word of the unit concerned.  This call synchronises
 * `stream`, reads the state words back and returns TCA_ERR_BOUNDS for the first unit whose word is
 * set, with detail[0] = unit, detail[1] = which check (1 selected index, 2 block count, 3 ring
 * slot, 4 cache row, 5 global region full), detail[2] = the offending value; detail HOST [3],
 * optional.  The checked kernels skip the access that failed its test, so no build touches memory
 * outside the buffers it was given.  tca_cache_init clears the words.
 */
int tca_cache_status(const tca_cache_desc* cache, void* stream, int64_t* detail);

/* Synchronise `stream` and read the sticky status word at the start of a workspace: TCA_OK,
 * TCA_ERR_TIMEOUT if a bounded wait inside a kernel gave up, or (range-checked build)
 * TCA_ERR_BOUNDS if a kernel met an index or offset outside its range and skipped the access. */
int tca_ws_status(const void* ws, void* stream);

/*
 * Self-test of the abort path that every bounded device-side wait shares.  One small CTA with the
 * roles of the attention kernels (a warp that holds tensor memory, one waiter with a time limit,
 * waiters that watch the CTA's abort flag) waits on a barrier at which nothing ever arrives.  After
 * limit_ns the limited wait gives up, the other waiters leave on the flag, the CTA sets word 0 of
 * `ws` exactly as the production kernels do, frees its tensor memory and returns.  Nothing traps
 * and nothing waits without a limit.  Afterwards tca_ws_status(ws) is TCA_ERR_TIMEOUT.
 *   ws             DEVICE, at least 256 bytes, 256-byte aligned, word 0 zero on entry
 *   limit_ns       1000 .. 100000000 (1 us .. 100 ms), else TCA_ERR_INVALID_ARG
 *   waited_ns_dev  DEVICE out, optional: how long the limited wait actually lasted
 * (No counterpart in the paper: test support for the library's error handling.)
 */
int tca_selftest_wait_expiry(void* ws, uint64_t limit_ns, uint64_t* waited_ns_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TCA_H_ */
