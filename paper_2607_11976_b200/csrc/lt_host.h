// Host-side declarations shared by the library's translation units (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "lt_common.cuh"

namespace lt {

constexpr int kModeFilter = 0;
constexpr int kModeDump = 1;
constexpr int kRowsPerBlock = 8;     // query rows one scan CTA (and one k-NN fallback block) keeps resident
constexpr int kRowsPerBlockFp8 = 6;  // ... of the alternative fp8 scan (LT_PATH_FUSED_ABS, lt_scan_fp8.cu)
constexpr int kLinTerms = 5;         // e4m3 terms of the linear part of a query (alternative fp8 scan)
constexpr int kLinScaleStride = 8;   // floats per row of the linear-term scale table

// Parameters of the tensor-core scan kernel (lt_scan_mma.cu).
struct ScanParams {
  const float* w;          // [T][64]
  const float* k_scale;    // per key of the view, or null
  long long ks_stride;     // k_scale index of view key s is s * ks_stride
  int T;                   // rows of q / w
  int row_begin, row_end;  // rows handled by this launch (ignored when fb_list is set)
  int n_keys;              // keys in the view
  int causal_offset;       // row t sees view keys 0 .. causal_offset + t
  int skip_masked_tiles;   // 1: do not visit key tiles no row of the block can see
  int seg_tiles;           // key tiles per work item
  int topk;
  // filter mode
  float* thr;              // [T] gate: lower edge of the row's threshold bin (-inf = accept all)
  const float* smin;       // [T] sampled minimum score
  const float* width;      // [T] bin width
  unsigned int* tail;      // [T] survivors appended so far (may exceed cap)
  unsigned int* hist;      // [T][kBins]
  uint2* cand;             // [T][cap] (score bits, key index)
  int cap;
  // dump mode
  float* dump;             // dense scores
  long long dump_ld;       // row pitch of dump in floats
  // exact-fallback dump: blocks come from a device-side list, slot j of this round
  // is block fb_list[fb_round_base + j], its rows go to dump rows 8j .. 8j+7
  const int* fb_list;
  const int* fb_blocks;    // device counter: entries in fb_list
  int fb_round_base;
  int fb_slots;
  // paged key cache (null: keys are one dense matrix): logical page j of 64 keys is physical page page_table[j] of
  // the pool the key tensor map covers; k_scale is then indexed by physical row
  const int* page_table;
  int n_pages;
  long long pool_pages;    // pages of the pool behind page_table (bounds checks of the debug build)
  unsigned int wait_limit_us;  // bound of every device-side wait (0 is replaced by the default at launch)
  int debug_flags;         // LT_DEBUG_* test hooks (filter mode only)
  // alternative fp8 scan only: the linear part of Eq. 1 prepared by launch_lin_terms
  const void* lin_q;       // [T][kLinTerms][128] e4m3 codes
  const float* lin_scale;  // [T][kLinScaleStride], the first kLinTerms entries of a row are used
  Control* ctl;
};
constexpr int kPageKeys = 64;  // keys per page of a paged key cache

bool scan_mma_supported(int dtype, int H, int D);
// ---- lt_scan_fp8.cu: the alternative fp8 scan (|x| form of Eq. 1 with linear-term columns) ------------
// bytes of the linear-term operand rows / of the scale table of T query rows
inline size_t lin_q_bytes(int T) { return static_cast<size_t>(T) * kLinTerms * 128; }
inline size_t lin_scale_bytes(int T) { return static_cast<size_t>(T) * kLinScaleStride * 4; }
// pre-pass: q [T][64][128] e4m3, w [T][64] -> lin_q, lin_scale
cudaError_t launch_lin_terms(const void* q, const float* w, int T, void* lin_q, float* lin_scale, cudaStream_t stream);
cudaError_t launch_scan_fp8(int mode, const void* q, int T, const void* k, long long n_keys_view, long long key_pitch_elems,
                            const ScanParams& p, int grid, cudaStream_t stream);

// One warp waits, with the bounded wait every scan kernel uses, on a barrier nobody arrives at:
// result2[0] = what the wait returned (0 = gave up), result2[1] = the abort flag it left behind.
cudaError_t launch_wait_timeout_probe(unsigned int limit_us, int* result2, cudaStream_t stream);
// bare FP8 UMMA stream (measurement aid): grid CTAs, an even number when pair is set
cudaError_t launch_umma_stream(bool pair, int iters, int* status, int grid, cudaStream_t stream);

// q: [T][64][128]; k: view of n_keys_view rows whose pitch is key_pitch_elems elements.
cudaError_t launch_scan_mma(int dtype, int mode, const void* q, int T, const void* k, long long n_keys_view,
                            long long key_pitch_elems, const ScanParams& p, int grid, cudaStream_t stream);

// ---- lt_scan_knn.cu -------------------------------------------------------------------------
// Parameters of the tensor-core scan of the k-NN (inner-product) variant: bf16 queries [T][D], corpus view of
// n_keys rows, every row sees every key.
struct KnnScanParams {
  int T;                   // rows of q
  int row_begin, row_end;  // query rows handled by this launch
  int n_keys;              // corpus vectors in the view
  int D;                   // multiple of 64, at most 768
  int seg_tiles;           // corpus tiles (128 vectors) per work item
  int topk;
  // filter mode
  float* thr;              // [T] gate: lower edge of the row's threshold bin
  const float* smin;       // [T]
  const float* width;      // [T]
  unsigned int* tail;      // [T]
  unsigned int* hist;      // [T][kBins]
  uint2* cand;             // [T][cap]
  int cap;
  // dump mode
  float* dump;             // dense scores, row (t - row_begin)
  long long dump_ld;
  const unsigned int* fb_flag;  // fallback rounds: flag per block of 8 rows; the launch is a no-op if no block of its row range is flagged
  unsigned int wait_limit_us;   // bound of every device-side wait (0 is replaced by the default at launch)
  Control* ctl;
};
bool scan_knn_supported(int D);
cudaError_t launch_scan_knn(int mode, const void* q, int T, const void* x, long long n_keys_view, long long key_pitch_elems,
                            const KnnScanParams& p, int grid, cudaStream_t stream);

// ---- lt_select.cu ---------------------------------------------------------------------------
// Generic SIMT scoring (any H, D, dtype): dense scores of rows [row_begin, row_end), -inf where masked.
cudaError_t launch_simt_scores(int dtype, const void* q, const float* w, const void* k, const float* k_scale, int T, int N,
                               int H, int D, int causal_offset, int row_begin, int row_end, float* out, long long ld,
                               cudaStream_t stream);

// Sample statistics (paper Sec. 3.2 "Sampling"): per row min / max of the sampled scores, bin
// width, and the threshold edge of the bin holding the rank-th largest sampled score.
cudaError_t launch_sample_stats(const float* sample, int T, int n_sample, int rank, float* smin, float* width, float* thr,
                                cudaStream_t stream);

// Final selection from the candidate buffers (paper Sec. 3.2 "Top-k Selection"); rows that cannot
// be finished exactly are flagged and their block appended to the fallback list.
struct FinalSelectParams {
  const unsigned int* tail;
  const unsigned int* hist;
  const uint2* cand;
  const float* smin;
  const float* width;
  int cap, T, N, topk, causal_offset;
  int32_t* out_idx;
  float* out_score;
  unsigned char* row_flag;    // [T] 1 = needs the fallback
  unsigned int* block_flag;   // [ceil(T / rows_per_block)]
  int* fb_list;               // [ceil(T / rows_per_block)]
  int rows_per_block;         // rows of one fallback block (the scan kernel's query block)
  Control* ctl;
};
cudaError_t launch_final_select(const FinalSelectParams& p, cudaStream_t stream);

// Full-row exact select over dense scores.  Direct mode: block b handles row row_begin + b whose
// scores start at scores + b * ld.  Fallback mode (fb_list != null), R = rows_per_block: block b handles row
// fb_list[fb_round_base + b / R] * R + b % R if that row is flagged; scores at scores + b * ld.
struct SelectRowsParams {
  const float* scores;
  long long ld;
  int n_blocks;  // CTAs to launch
  int row_begin;
  int T, N, topk, causal_offset;
  int32_t* out_idx;
  float* out_score;
  const int* fb_list;
  const int* fb_blocks;
  int fb_round_base;
  int rows_per_block;
  const unsigned char* row_flag;
  Control* ctl;
};
cudaError_t launch_select_rows(const SelectRowsParams& p, cudaStream_t stream);

// ---- lt_sampler.cu --------------------------------------------------------------------------
// counts[p] += occurrences of p in idx[0..n) (entries outside [0, N) are skipped); counts must be zeroed.
cudaError_t launch_count_positions(const int32_t* idx, long long n, int N, unsigned int* counts, cudaStream_t stream);
// the n_out most frequent positions of counts[0..N), (count desc, position asc); max_count bounds every count; scratch: rank_scratch_bytes(n_out)
size_t rank_scratch_bytes(int n_out);
cudaError_t launch_rank_counts(const unsigned int* counts, int N, int n_out, unsigned long long max_count, void* scratch,
                               int32_t* out_pos, int32_t* out_count, cudaStream_t stream);
// dense copy of the key rows (row_bytes each, multiple of 16) and scales at the sampled positions (sample_idx, or
// j * stride when it is null); page_table (or null) translates positions to physical rows of a paged key cache
// (pool_rows and ctl serve the bounds-checking build: a translated row outside the pool is read as row 0 and flagged)
cudaError_t launch_gather_keys(const void* k, const float* k_scale, const int32_t* sample_idx, long long stride, int n_sample,
                               int N, int row_bytes, const int* page_table, long long pool_rows, Control* ctl, void* out_k,
                               float* out_scale, cudaStream_t stream);

// ---- lt_dsa_union.cu ------------------------------------------------------------------------
// LiteDSA union list + membership masks of consecutive groups of `group` rows (paper Sec. 3.3).
// union_pos [n_groups][group * topk] (-1 beyond union_len), mask [T][ceil(group * topk / 32)].
cudaError_t launch_dsa_union(const int32_t* idx, int T, int topk, int N, int group, int32_t* union_pos, int32_t* union_len,
                             uint32_t* mask, cudaStream_t stream);

}  // namespace lt
