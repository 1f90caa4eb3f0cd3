/*
 * lt_indexer.h -- C ABI of the fused DSA indexer top-k for NVIDIA B200 (sm_100a).
 *
 * The operation (paper Sec. 2, Eq. 1 and Sec. 3.1, Eq. 2): for every query row t
 * of a prefill chunk and every key s it may see,
 *
 *     I[t, s] = k_scale[s] * sum_{j<H} w[t, j] * ReLU( q[t, j, :] . k[s, :] )
 *
 * and the result is, per row, the exact top-k keys by I, ordered by (score
 * descending, key index ascending).  The T x N score matrix is never written
 * to memory: a sample of the keys fixes equal-width score bins, candidates are
 * gated against an online threshold bin while they are scored, only survivors
 * are written back, and an exact select runs on the survivors (paper Sec. 3.2:
 * sampling, filtering, threshold refresh, top-k selection).  Rows for which
 * that scheme cannot guarantee exactness are recomputed by an unfused exact
 * path, so the result is always the exact top-k of the library's own scores.
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller; the library
 *     never frees or keeps them.  Outputs are fully overwritten.
 *   - Layouts are dense row-major: q[T][H][D], w[T][H] (fp32), k[N][D],
 *     k_scale[N] (fp32), out_idx[T][topk] (int32), out_score[T][topk] (fp32).
 *     q, k, w, k_scale must be 16-byte aligned.
 *   - Row t stands at position causal_offset + t and sees keys
 *     0 .. causal_offset + t inclusive, clipped to [0, N).  causal_offset >= N-1
 *     disables masking.  Rows that see fewer than topk keys are padded with
 *     index -1 and score -inf.
 *   - Scores are computed from exact products of the stored values with fp32
 *     accumulation; -0.0 is returned as +0.0.  Inputs must be finite (no NaN /
 *     Inf, no e4m3 NaN codes) and k_scale >= 0; this is not checked.
 *   - A query-side fp8 scale is folded by the caller into w (w[t,j] *= q_scale[t]),
 *     which is exact because ReLU is positively homogeneous.
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work on it
 *     and never synchronise the host, except lt_read_status and the internal
 *     arena growth of the 13-argument lt_indexer_topk.  The calls that take a
 *     workspace can therefore be captured into a CUDA graph (stream capture)
 *     and replayed, once an eager call of the same kind has loaded the
 *     kernels; keep lt_set_profiling off while capturing.
 *   - Return value: LT_OK or a negative LT_ERR_* code detected on the host
 *     before anything is enqueued.  Conditions met on the device are recorded
 *     in a status word (LT_STATUS_* bits) inside the workspace; kernels never
 *     trap and every device-side wait is bounded.
 */
#ifndef LT_INDEXER_H_
#define LT_INDEXER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LT_VERSION 100

/* storage type of q and k */
#define LT_DTYPE_F32 0  /* float32                                   */
#define LT_DTYPE_BF16 1 /* bfloat16 bit patterns                     */
#define LT_DTYPE_E4M3 2 /* fp8 e4m3 ("fn") codes, k_scale required   */

/* return codes */
#define LT_OK 0
#define LT_ERR_INVALID_ARG (-1) /* null pointer, size <= 0, topk > N or > LT_MAX_TOPK, misaligned pointer */
#define LT_ERR_UNSUPPORTED (-2) /* dtype / shape the library has no path for                              */
#define LT_ERR_WORKSPACE (-3)   /* workspace missing, misaligned or too small                             */
#define LT_ERR_CUDA (-4)        /* a CUDA runtime call failed; see lt_last_cuda_error                     */
#define LT_ERR_TOO_LARGE (-5)   /* lt_indexer_topk_static: the problem does not fit the fixed scratch     */

/* bits of the device status word (lt_read_status, status[0]) */
#define LT_STATUS_TIMEOUT 1  /* a bounded device-side wait ran out; results are invalid   */
#define LT_STATUS_FALLBACK 2 /* some rows took the exact unfused fallback (informational) */
#define LT_STATUS_BOUNDS 4   /* a debug bounds check failed                               */

#define LT_MAX_TOPK 8192
#define LT_BINS 256 /* m, the number of equal-width score bins (paper Sec. 3.2, "Sampling") */

/* which implementation lt_indexer_topk_ex uses */
#define LT_PATH_AUTO 0    /* fused tensor-core path when the shape allows it, else generic */
#define LT_PATH_FUSED 1   /* fused tcgen05 path; LT_ERR_UNSUPPORTED if the shape does not fit */
#define LT_PATH_GENERIC 2 /* generic SIMT scoring + full-row select (any H, D, dtype)      */
#define LT_PATH_FUSED_ABS 3 /* fp8 only: an alternative fused tensor-core scan that evaluates Eq. 1 as
                               sum_h (w_h / 2) |x_h| + (1/2) (sum_h w_h q_h) . k (ReLU(x) = (x + |x|) / 2), the linear
                               term riding on the tensor core as five e4m3-split accumulator columns per query.
                               Exact like the default (its own scores, lt_indexer_scores with the same path, are
                               within the same tolerance of Eq. 1 and ranked bit-exactly), but slower as measured;
                               kept as a documented alternative.  LT_ERR_UNSUPPORTED for other dtypes / shapes     */

/*
 * Tunables.  None of them may change any output bit; they trade memory and speed.
 * A zero field means "default".
 */
typedef struct lt_tunables {
  int path;          /* LT_PATH_*                                                        */
  int cap_mult;      /* candidate buffer capacity per row = cap_mult * topk (12 k per row is the size
                        the paper reports in Sec. 4.2).  Default (0): max(12 topk, 16384) entries; an explicit
                        value is taken as given                                               */
  int sample_mult;   /* sample size k' = sample_mult * topk (paper Sec. 3.2: 3).  Default (0): max(3 topk,
                        min(8192, keys the sample is drawn from / 32)), but no more than 64 * (keys the
                        sample is drawn from) / topk, which is what the default sample_rank needs; an
                        explicit value is taken as given                                           */
  int segment_tiles; /* key tiles (128 keys each) per work item (default 256)            */
  int grid;          /* CTAs of the scan kernel (default: number of SMs)                 */
  int sample_rank;   /* initial gate = lower edge of the bin holding the sample's r-th largest
                        score.  0 (default): r = ceil(m + 5 sqrt(m) + 5) capped at topk, where
                        m = topk * k' / (keys the sample is drawn from) is the expected number of
                        sampled keys inside the true top-k; the sample then misjudges a row with
                        probability < 1e-6 (Poisson tail), and such a row is caught by the final
                        select (fewer than topk survivors) and redone by the exact fallback.
                        -1: r = topk, the paper's rule (Sec. 3.2 "Sampling"), which can never
                        misjudge but starts ~k'/r times looser.  > 0: r itself.              */
  int wait_limit_us; /* bound, in microseconds, of every device-side wait of the scan kernels (default 0 = 2 s).
                        A wait that runs out sets LT_STATUS_TIMEOUT, the kernel unwinds and returns; the
                        results of that call are invalid, the next call is unaffected               */
  int debug_flags;   /* LT_DEBUG_* test hooks, 0 in production                             */
} lt_tunables;

/* lt_tunables.debug_flags (no counterpart in the paper; used by the library's own tests) */
#define LT_DEBUG_SKIP_ONE_KTILE 1 /* the fused scan's first CTA never loads its first key tile: with a short
                                     wait_limit_us this exercises the bounded-wait timeout path without
                                     any fault (the call returns, status has LT_STATUS_TIMEOUT)        */

/*
 * Fused indexer top-k (paper Sec. 3.2; Eq. 1 + Eq. 2), 13-argument form.
 *   dtype is inferred: k_scale != NULL -> q, k are e4m3 codes; k_scale == NULL -> bf16.
 *   out_score may be NULL.  Uses a library-owned workspace, one per device, that grows on demand
 *   (growth waits for that device's earlier work once, then frees and reallocates); lt_shutdown
 *   frees them all.
 *   All calls of this form on one device share that workspace (counters, histograms, candidate
 *   buffers, fallback scratch), and each call clears the parts that must start at zero: two calls whose
 *   kernels may overlap on the GPU (different streams, or different host threads on different
 *   streams) race on it and return wrong results without any error - serialise them on one stream,
 *   or use lt_indexer_topk_ex with one workspace per stream.
 */
int lt_indexer_topk(const void* q, const float* w, const void* k, const float* k_scale,
                    int T, int N, int H, int D, int topk, int causal_offset,
                    int32_t* out_idx, float* out_score, void* stream);

/*
 * General form: explicit dtype, caller-owned workspace (device memory, 256-byte
 * aligned, at least lt_indexer_topk_workspace_bytes(...) bytes; its contents are
 * scratch), optional tunables (NULL = defaults).  fp32 inputs are reachable only
 * through this form.  The workspace also holds the status word.
 */
int lt_indexer_topk_ex(int dtype, const void* q, const float* w, const void* k, const float* k_scale,
                       int T, int N, int H, int D, int topk, int causal_offset,
                       int32_t* out_idx, float* out_score,
                       void* workspace, size_t workspace_bytes, const lt_tunables* tunables, void* stream);

/*
 * lt_indexer_topk_ex over a key matrix whose rows are k_pitch_elems elements apart (k_pitch_elems >= D,
 * the pitch a multiple of 16 bytes): a view of a wider cache, e.g. one D-wide field of a row that also
 * holds other data (paper Sec. 4.1 benchmarks the kernel on a serving engine's cache layout).  k_scale
 * stays dense, one float per key.  Same outputs as the dense layout, bit for bit; same workspace size;
 * fused tensor-core path only (LT_ERR_UNSUPPORTED otherwise).
 */
int lt_indexer_topk_strided(int dtype, const void* q, const float* w, const void* k, long long k_pitch_elems,
                            const float* k_scale, int T, int N, int H, int D, int topk, int causal_offset,
                            int32_t* out_idx, float* out_score,
                            void* workspace, size_t workspace_bytes, const lt_tunables* tunables, void* stream);

/* Bytes of workspace lt_indexer_topk_ex needs for this problem (0 on invalid arguments). */
size_t lt_indexer_topk_workspace_bytes(int dtype, int T, int N, int H, int D, int topk,
                                       const lt_tunables* tunables);

/*
 * Fused indexer top-k with a caller-provided sample (paper Sec. 3.2 "Sampling": for sparse attention
 * the sample of a chunk is the k' = 3k positions most frequent in the previous chunk's top-k, see
 * lt_topk_frequent).  Same outputs as lt_indexer_topk_ex, bit for bit, whatever the sample holds:
 * the sample only decides how tight the initial gate is.
 *   sample_idx  device, n_sample key positions (int32).  They should be distinct and visible to every
 *               row of the chunk (0 <= position <= causal_offset); the initial gate is then the bin of
 *               the topk-th largest sampled score, which can never misjudge (the sample is a subset of
 *               every row's keys).  Positions outside [0, N) are read as position 0; duplicates,
 *               positions past causal_offset or such replaced positions can at worst make the gate too
 *               tight for some rows, which the final select detects and the exact fallback redoes.
 *   n_sample    1 .. LT_MAX_SAMPLE.  Fewer than topk positions leave the gate open until the
 *               online refresh takes over.
 *   workspace   at least lt_indexer_topk_sampled_workspace_bytes(...) bytes.
 * lt_tunables.sample_mult is ignored; sample_rank > 0 overrides the rank, otherwise rank = topk.
 * On shapes the fused path does not support the sample is ignored.
 */
#define LT_MAX_SAMPLE 32768
int lt_indexer_topk_sampled(int dtype, const void* q, const float* w, const void* k, const float* k_scale,
                            int T, int N, int H, int D, int topk, int causal_offset,
                            const int32_t* sample_idx, int n_sample,
                            int32_t* out_idx, float* out_score,
                            void* workspace, size_t workspace_bytes, const lt_tunables* tunables, void* stream);
size_t lt_indexer_topk_sampled_workspace_bytes(int dtype, int T, int N, int H, int D, int topk, int n_sample,
                                               const lt_tunables* tunables);

/*
 * Fused indexer top-k over a PAGED key cache (serving layout; the paper's kernel reads the cache of its
 * serving engine, Sec. 4.1).  Keys live in a pool of pages of LT_PAGE_KEYS = 64 consecutive rows:
 *   k_pool        device, [pool_rows][D] (bf16 or e4m3), pool_rows a multiple of 64
 *   k_scale_pool  device, [pool_rows] fp32 (e4m3 only), indexed like k_pool
 *   page_table    device, n_pages int32: keys 64 j .. 64 j + 63 of the context are pool rows
 *                 64 page_table[j] .. 64 page_table[j] + 63; n_pages * 64 >= N; entries must be valid
 *                 page numbers (0 <= page_table[j] < pool_rows / 64)
 * Everything else as lt_indexer_topk_ex, and the outputs are bit-identical to lt_indexer_topk_ex on the
 * same keys laid out densely.  Only shapes of the tensor-core path (H = 64, D = 128, bf16 or e4m3);
 * LT_ERR_UNSUPPORTED otherwise.  workspace: lt_indexer_topk_paged_workspace_bytes(...) bytes (the sampled
 * keys are gathered into it: a strided view cannot reach a paged cache).
 */
#define LT_PAGE_KEYS 64
int lt_indexer_topk_paged(int dtype, const void* q, const float* w, const void* k_pool, const float* k_scale_pool,
                          const int32_t* page_table, int n_pages, long long pool_rows,
                          int T, int N, int H, int D, int topk, int causal_offset,
                          int32_t* out_idx, float* out_score,
                          void* workspace, size_t workspace_bytes, const lt_tunables* tunables, void* stream);
size_t lt_indexer_topk_paged_workspace_bytes(int dtype, int T, int N, int H, int D, int topk, const lt_tunables* tunables);

/*
 * The n_out positions that occur most often in a chunk's top-k index matrix (paper Sec. 3.2
 * "Sampling": the previous-chunk sampler), ordered by (count descending, position ascending);
 * positions that never occur (count 0) fill the tail in ascending order.
 *   idx        device, [T][topk] int32 as written by the top-k entry points; entries < 0 are padding
 *              and entries >= N are ignored
 *   out_pos    device, n_out int32;  out_count: device, n_out int32, or NULL
 *   n_out      1 .. min(N, LT_MAX_TOPK)
 *   workspace  device, 256-byte aligned, at least lt_topk_frequent_workspace_bytes(N) bytes (about 4 N)
 * Integer work only: the result is exact.  Enqueued on `stream`; no host synchronisation.
 */
int lt_topk_frequent(const int32_t* idx, int T, int topk, int N, int n_out, int32_t* out_pos, int32_t* out_count,
                     void* workspace, size_t workspace_bytes, void* stream);
size_t lt_topk_frequent_workspace_bytes(int N);

/*
 * k-NN (inner-product) variant: exact top-k of f(q, x) = q . x over a whole corpus for a batch of
 * queries (paper Sec. 3.1, Eq. 2; the retrieval workload of Sec. 4.1: 768-d embeddings, batches of 64
 * queries, k up to 8192, no causal mask).  Same method as the indexer path - strided sample, bins,
 * online threshold, filtered write-back, exact final select, exact fallback - with the scores coming
 * straight from the tensor cores (Sec. 3.2 "Filtering", first case), so the corpus is streamed from
 * HBM once per 64 queries.
 *   dtype       LT_DTYPE_BF16 only
 *   q           device, [T][D] bf16;  x: device, [N][D] bf16 (both 16-byte aligned, row-major, dense)
 *   D           a multiple of 64, at most 768;  topk: 1 .. min(N, LT_MAX_TOPK)
 *   out_idx     device, [T][topk] int32 in (score descending, index ascending) order; out_score: device,
 *               [T][topk] fp32 or NULL
 *   workspace   device, 256-byte aligned, at least lt_knn_topk_workspace_bytes(...) bytes; holds the
 *               status block (lt_read_status)
 * lt_knn_scores writes the dense scores of rows [row_begin, row_end) to out_scores[(t - row_begin) * N + s],
 * bit-identical to the scores lt_knn_topk ranks (debugging and parity).
 * Errors: LT_ERR_UNSUPPORTED for another dtype or D, LT_ERR_INVALID_ARG, LT_ERR_WORKSPACE, LT_ERR_CUDA.
 */
int lt_knn_topk(int dtype, const void* q, const void* x, int T, int N, int D, int topk,
                int32_t* out_idx, float* out_score,
                void* workspace, size_t workspace_bytes, const lt_tunables* tunables, void* stream);
size_t lt_knn_topk_workspace_bytes(int dtype, int T, int N, int D, int topk, const lt_tunables* tunables);
int lt_knn_scores(int dtype, const void* q, const void* x, int T, int N, int D,
                  int row_begin, int row_end, float* out_scores, void* stream);

/*
 * LiteDSA union list and membership masks (paper Sec. 3.3 "LiteDSA").  Rows are taken in consecutive
 * groups of `group` (the last group may be shorter).  For group g:
 *   union_pos[g][0 .. union_len[g])  the distinct positions selected by any row of the group, ascending
 *                                    (what a sweep of the group's bitmap yields); the rest of the
 *                                    group * topk slots is -1
 *   member_mask[t][s / 32] bit s % 32 = 1 iff union_pos[g(t)][s] is one of idx[t][:]
 * All pointers are device memory: idx [T][topk] int32 (entries < 0 or >= N are skipped), union_pos
 * [ceil(T / group)][group * topk] int32, union_len [ceil(T / group)] int32, member_mask
 * [T][ceil(group * topk / 32)] uint32.  1 <= group, group * topk <= 2^24.  Integer work only: the
 * result is exact.  The masked attention that consumes these is not part of this library.
 */
int lt_dsa_union_mask(const int32_t* idx, int T, int topk, int N, int group,
                      int32_t* union_pos, int32_t* union_len, uint32_t* member_mask, void* stream);

/*
 * Host-only helper (no GPU work): the sample plan the fused path would use for this problem.
 * plan3[0] = sample size k', plan3[1] = stride between sampled key positions (the sample is
 * positions 0, stride, 2 stride, ... of the keys every row of the chunk can see), plan3[2] = rank r
 * of the sampled score whose bin sets the initial gate (see lt_tunables.sample_rank).
 * Returns LT_OK or LT_ERR_INVALID_ARG.
 */
int lt_indexer_sample_plan(int N, int topk, int causal_offset, const lt_tunables* tunables, int plan3[3]);

/*
 * Dense scores of rows [row_begin, row_end) (Eq. 1), for debugging and parity:
 * out_scores[(t - row_begin) * N + s] = I[t, s] for visible keys, -inf otherwise.
 * The values are bit-identical to those lt_indexer_topk(_ex) ranks for the same
 * dtype and path.  dtype as in lt_indexer_topk_ex; path = LT_PATH_*.
 */
int lt_indexer_scores(int dtype, const void* q, const float* w, const void* k, const float* k_scale,
                      int T, int N, int H, int D, int causal_offset,
                      int row_begin, int row_end, float* out_scores, int path, void* stream);

/*
 * Unfused baseline (the decoupled design of paper Sec. 1: materialise scores, then
 * select): scores of `rows_per_pass` rows at a time are written to score_buf
 * (device, >= rows_per_pass * N * 4 bytes), each pass followed by a full-row radix
 * select.  Same outputs as lt_indexer_topk_ex.
 */
int lt_unfused_topk(int dtype, const void* q, const float* w, const void* k, const float* k_scale,
                    int T, int N, int H, int D, int topk, int causal_offset,
                    int32_t* out_idx, float* out_score,
                    float* score_buf, size_t score_buf_bytes, int path, void* stream);

/*
 * Exact indexer top-k for callers that must not allocate device memory.  (The paper has no
 * counterpart: this entry point exists for deployment reasons only.)
 *
 * Who needs it: a serving process that hands nearly all free HBM to its KV cache at start-up (the
 * paper's Sec. 1 budget leaves under 3 GB of headroom) cannot count on a later cudaMalloc to
 * succeed, and a caller in a latency-critical loop cannot afford the device-wide synchronisation a
 * cudaMalloc or cudaFree implies.  Such callers also often have no workspace of their own to lend.
 *
 * What it does: the same result as lt_indexer_topk_ex (same outputs, same ordering, same scores bit
 * for bit), computed by the decoupled path - dense scores of a few rows at a time, then a full-row
 * radix select - whose scratch is a fixed LT_STATIC_SCRATCH_BYTES array inside the library's device
 * image instead of a caller workspace.  Every GPU that loads the library holds that array until the
 * process exits.  The call itself performs no cudaMalloc, cudaFree or other allocating call; q, w,
 * k, k_scale, out_idx, out_score are the caller's device buffers as everywhere else.
 *
 * Limits and rules:
 *   - one score row must fit: N * 4 <= LT_STATIC_SCRATCH_BYTES - 256 (N <= 4,194,240), otherwise
 *     LT_ERR_TOO_LARGE is returned and nothing is enqueued; rows are processed
 *     floor((LT_STATIC_SCRATCH_BYTES - 256) / (4 N)) at a time, so large T x N problems run as many
 *     small passes and are slower than lt_indexer_topk_ex;
 *   - the first call on each device looks up the array's device address (cudaGetSymbolAddress);
 *     make that first call before any stream capture begins on that device;
 *   - all calls on a device share the one array, which keeps the previous call's contents (the call
 *     clears the status block it needs at zero and overwrites score rows before reading them):
 *     two calls whose kernels may overlap on the GPU (different streams, or different host threads
 *     on different streams) race on it - serialise them on one stream;
 *   - the status block lives in the fixed array too: read it with lt_read_status_static; device-side
 *     waits are bounded as in every other entry point.
 */
#define LT_STATIC_SCRATCH_BYTES (16u << 20)
int lt_indexer_topk_static(int dtype, const void* q, const float* w, const void* k, const float* k_scale,
                           int T, int N, int H, int D, int topk, int causal_offset,
                           int32_t* out_idx, float* out_score, void* stream);

/* Largest N lt_indexer_topk_static accepts: (LT_STATIC_SCRATCH_BYTES - 256) / 4 keys (no counterpart in the paper). */
int lt_indexer_topk_static_max_keys(void);

/*
 * Copies the 8-int status block of a workspace to host memory after synchronising
 * `stream`: [0] LT_STATUS_* bits, [1] rows that took the fallback, [2] largest
 * survivor count of any row, [3] total survivors (low 31 bits, saturating),
 * [4] rows whose candidate buffer overflowed, [5..7] reserved.
 * workspace == NULL reads the library-owned workspace of lt_indexer_topk.
 */
int lt_read_status(const void* workspace, int* status8_host, void* stream);
/* The same for the status block lt_indexer_topk_static keeps in the current device's fixed array. */
int lt_read_status_static(int* status8_host, void* stream);

/*
 * Test probe for the bounded waits (no counterpart in the paper): one warp waits, with the wait
 * every scan kernel uses, at most limit_us microseconds on a barrier nobody arrives at.  On return of
 * the kernel result2_device[0] = 0 (the wait gave up) and result2_device[1] = 1 (it raised the abort
 * flag its CTA would unwind on).  Nothing faults, traps or spins without bound.
 */
int lt_debug_wait_timeout(int limit_us, int* result2_device, void* stream);

/*
 * Measurement aid (no counterpart in the paper; used by the benchmark): a bare FP8 tensor-core stream.  One
 * launch of one CTA per SM; every CTA issues `iters` x 8 tcgen05.mma kind::f8f6f4 instructions of the scan's tile
 * shape (128 keys x 256 (query, head) columns x 32 bytes; 2 x 128 x 256 x 128 x 2 flops per SM and iteration) on
 * e4m3 operands that stay in shared memory: no TMA, no epilogue.  FLOPs of a launch = SMs x iters x 16,777,216.
 * What it sustains is the tensor ceiling of the board at the clocks and power it is granted, against which the
 * scan's roofline fraction can be read.
 *   pair           0: cta_group::1 (the scan's form).  1: CTA pairs, cta_group::2 with M = 256, each CTA holding
 *                  half of the second operand (an even number of CTAs is launched).
 *   iters          1 .. 2^24.
 *   status_device  DEVICE, one int the caller zeroed; LT_STATUS_TIMEOUT is OR-ed in if a bounded wait ran out.
 * Only enqueues on `stream`; returns LT_ERR_INVALID_ARG for bad arguments, LT_ERR_CUDA if the launch fails.
 */
int lt_debug_umma_stream(int pair, int iters, int* status_device, void* stream);

/*
 * Instrumentation (no counterpart in the paper; used by the benchmark).
 *   lt_launch_count     kernels this library has launched so far in this process.
 *   lt_set_profiling    when enabled, lt_indexer_topk(_ex) on the fused path records CUDA events on
 *                       the caller's stream between its phases (events are created on the first
 *                       enable for the current device).
 *   lt_read_phase_ms    synchronises `stream` and returns the device time in ms of the five phases
 *                       of the last profiled call: [0] sample scoring, [1] sample statistics,
 *                       [2] fused scan (score + filter), [3] final select, [4] exact fallback.
 */
unsigned long long lt_launch_count(void);
int lt_set_profiling(int enable);
int lt_read_phase_ms(float* ms5_host, void* stream);

const char* lt_strerror(int code);
int lt_last_cuda_error(void); /* the cudaError_t behind the last LT_ERR_CUDA of this thread */
int lt_version(void);
void lt_shutdown(void); /* frees the library-owned workspace */

#ifdef __cplusplus
}
#endif
#endif /* LT_INDEXER_H_ */
