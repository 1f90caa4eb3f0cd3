// C ABI of the indexer top-k library: argument checks, workspace layout, kernel sequencing.
#include <cuda_runtime.h>
#include <limits.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "../../include/lt_indexer.h"
#include "lt_common.cuh"
#include "lt_host.h"

namespace lt {
namespace {

thread_local int g_last_cuda_error = 0;

// ---- instrumentation: kernel-launch counter and optional per-phase CUDA events ---------------
std::atomic<unsigned long long> g_launches{0};
constexpr int kPhases = 5;  // sample scan, sample statistics, fused scan, final select, fallback
bool g_profiling = false;
cudaEvent_t g_events[kPhases + 1] = {nullptr};
int g_events_dev = -1;

void mark_phase(int i, cudaStream_t stream) {
  if (g_profiling && g_events[i] != nullptr) cudaEventRecord(g_events[i], stream);
}

#define LT_CUDA(expr)                                  \
  do {                                                 \
    cudaError_t e__ = (expr);                          \
    if (e__ != cudaSuccess) {                          \
      g_last_cuda_error = static_cast<int>(e__);       \
      return LT_ERR_CUDA;                              \
    }                                                  \
  } while (0)

#define LT_LAUNCH(expr) \
  do {                  \
    LT_CUDA(expr);      \
    ++g_launches;       \
  } while (0)

constexpr size_t kAlign = 256;
size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

constexpr size_t kFallbackScratchBudget = size_t(512) << 20;  // dense scores kept at once by the exact fallback
constexpr size_t kGenericScratchBudget = size_t(256) << 20;   // dense scores kept at once by the generic path

struct Tun {
  int path, cap_mult, sample_mult, segment_tiles, grid, sample_rank;
  bool sample_mult_given, cap_mult_given;
  unsigned int wait_limit_us;
  int debug_flags;
};
Tun resolve_tunables(const lt_tunables* t) {
  Tun r{LT_PATH_AUTO, 12, 3, 0, 0, 0, false, false, 0u, 0};
  if (t != nullptr) {
    r.path = t->path;
    if (t->cap_mult > 0) {
      r.cap_mult = t->cap_mult;
      r.cap_mult_given = true;
    }
    if (t->sample_mult > 0) {
      r.sample_mult = t->sample_mult;
      r.sample_mult_given = true;
    }
    if (t->segment_tiles > 0) r.segment_tiles = t->segment_tiles;
    if (t->grid > 0) r.grid = t->grid;
    r.sample_rank = t->sample_rank;
    if (t->wait_limit_us > 0) r.wait_limit_us = static_cast<unsigned int>(t->wait_limit_us);
    r.debug_flags = t->debug_flags;
  }
  return r;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_problem(int dtype, const void* q, const float* w, const void* k, const float* k_scale, int T, int N, int H, int D) {
  if (dtype != LT_DTYPE_F32 && dtype != LT_DTYPE_BF16 && dtype != LT_DTYPE_E4M3) return LT_ERR_UNSUPPORTED;
  if (q == nullptr || w == nullptr || k == nullptr) return LT_ERR_INVALID_ARG;
  if (dtype == LT_DTYPE_E4M3 && k_scale == nullptr) return LT_ERR_INVALID_ARG;
  if (T <= 0 || N <= 0 || H <= 0 || D <= 0) return LT_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(w) || !aligned16(k) || (k_scale != nullptr && !aligned16(k_scale))) return LT_ERR_INVALID_ARG;
  if (static_cast<size_t>(H) * D * 4 + 128 * (static_cast<size_t>(D) + 1) * 4 > 200 * 1024) return LT_ERR_UNSUPPORTED;
  return LT_OK;
}

bool use_fused(const Tun& tun, int dtype, int H, int D) {
  return tun.path != LT_PATH_GENERIC && scan_mma_supported(dtype, H, D);
}
// the alternative fp8 scan (|x| form with linear-term columns, 6-row query blocks) was asked for and applies
bool use_abs_form(const Tun& tun, int dtype, int H, int D) {
  return tun.path == LT_PATH_FUSED_ABS && dtype == LT_DTYPE_E4M3 && scan_mma_supported(dtype, H, D);
}

// ---- workspace layout ------------------------------------------------------------------------
struct Layout {
  bool fused;
  // zeroed region
  size_t ctl, tail, hist, row_flag, block_flag, zero_end;
  size_t smin, width, thr, fb_list, lin_q, lin_scale, sample, gather_k, gather_scale, cand, scratch, fb_base, total;
  int cap, n_sample, sample_stride, sample_rank, fb_slots, n_blocks, generic_rows;
  int rpb;        // rows of one scan block = rows of one fallback block
  bool abs_form;  // the alternative fp8 scan: linear-term rows live in the workspace
};

// n_given > 0: the caller provides that many sample positions (lt_indexer_topk_sampled); their keys are
// gathered into a dense buffer of the workspace (key_row_bytes each) and scored from there.
// gather_default: the default strided sample is gathered too (paged key cache: a strided view cannot reach it).
Layout make_layout(bool fused, int T, int N, int topk, int causal_offset, const Tun& tun, int n_given = 0,
                   int key_row_bytes = 0, bool gather_default = false, bool abs_form = false) {
  Layout L{};
  L.fused = fused;
  L.abs_form = fused && abs_form;
  L.rpb = L.abs_form ? kRowsPerBlockFp8 : kRowsPerBlock;
  size_t off = 0;
  L.ctl = off;
  off = align_up(off + sizeof(Control));
  if (!fused) {
    long long rows = static_cast<long long>(kGenericScratchBudget / (static_cast<size_t>(N) * 4));
    L.generic_rows = static_cast<int>(rows < 1 ? 1 : (rows > T ? T : rows));
    L.zero_end = off;
    L.scratch = off;
    off = align_up(off + static_cast<size_t>(L.generic_rows) * N * 4);
    L.total = off;
    return L;
  }
  L.n_blocks = (T + L.rpb - 1) / L.rpb;
  L.tail = off;
  off = align_up(off + static_cast<size_t>(T) * 4);
  L.hist = off;
  off = align_up(off + static_cast<size_t>(T) * kBins * 4);
  L.row_flag = off;
  off = align_up(off + static_cast<size_t>(T));
  L.block_flag = off;
  off = align_up(off + static_cast<size_t>(L.n_blocks) * 4);
  L.zero_end = off;
  L.smin = off;
  off = align_up(off + static_cast<size_t>(T) * 4);
  L.width = off;
  off = align_up(off + static_cast<size_t>(T) * 4);
  L.thr = off;
  off = align_up(off + static_cast<size_t>(T) * 4);
  L.fb_list = off;
  off = align_up(off + static_cast<size_t>(L.n_blocks) * 4);
  // alternative fp8 scan: operand rows and scales of the linear part of Eq. 1 (lt_scan_fp8.cu)
  L.lin_q = off;
  if (L.abs_form) off = align_up(off + lin_q_bytes(T));
  L.lin_scale = off;
  if (L.abs_form) off = align_up(off + lin_scale_bytes(T));
  // sample: keys every chunk row can see, i.e. positions 0 .. causal_offset, strided
  long long prefix = static_cast<long long>(causal_offset) + 1;
  if (prefix > N) prefix = N;
  if (prefix < 0) prefix = 0;
  long long want = static_cast<long long>(tun.sample_mult) * topk;
  if (tun.sample_rank == 0 && !tun.sample_mult_given && n_given == 0) {
    // With the rank scaled to the sampling fraction the sample only has to hold a few dozen of a row's top-k
    // keys: 64 expected ones (k' = 64 prefix / topk, rounded up to whole key tiles) already put the initial
    // gate within a factor 1.7 of the true k/N quantile.  Short contexts then pay for far fewer sampled
    // scores (65,536 keys, k = 2048: 2,048 instead of 6,144 per row).  A small k over a long context is the
    // opposite case: 3k keys hold less than one of the row's top-k, the gate starts orders of magnitude too
    // loose and the candidate buffers overflow, so the sample is at least 8,192 keys (6 % of a 1M-key scan
    // at most).
    // ... but no more than 1/32 of the keys it is drawn from: over a 64K context 8,192 samples would be an eighth
    // of the scan, while 2,048 still put a dozen top-k keys' worth of rank between the gate and the k-th score
    long long floor_n = prefix / 32;
    if (floor_n > 8192) floor_n = 8192;
    if (want < floor_n) want = floor_n;
    long long enough = (64 * prefix + topk - 1) / topk;
    enough = (enough + kTileKeys - 1) / kTileKeys * kTileKeys;
    if (enough < want) want = enough;
  }
  L.n_sample = static_cast<int>(want < prefix ? want : prefix);
  L.sample_stride = L.n_sample > 0 ? static_cast<int>(prefix / L.n_sample) : 1;
  if (n_given > 0) {
    L.n_sample = n_given;
    L.sample_stride = 1;
  }
  // Rank of the sampled score that sets the initial gate.  A row's true top-k holds about
  // m = topk * n_sample / prefix sampled keys (fewer for rows that see keys past the prefix); the gate
  // is too tight only if it holds at least `rank` of them, so rank = m + 5 sqrt(m) + 5 keeps that below
  // 1e-6 per row (Poisson tail), and the final select sends such a row to the exact fallback.
  if (tun.sample_rank > 0) {
    L.sample_rank = tun.sample_rank < topk ? tun.sample_rank : topk;
  } else if (tun.sample_rank < 0 || L.n_sample <= 0 || n_given > 0) {
    L.sample_rank = topk;  // the paper's rule; a caller-provided sample is not a uniform one
  } else {
    const double m = static_cast<double>(topk) * L.n_sample / static_cast<double>(prefix);
    const double r = ceil(m + 5.0 * sqrt(m) + 5.0);
    L.sample_rank = r < static_cast<double>(topk) ? static_cast<int>(r) : topk;
  }
  L.sample = off;
  off = align_up(off + static_cast<size_t>(T) * (L.n_sample > 0 ? L.n_sample : 1) * 4);
  const int gather_rows = n_given > 0 ? n_given : (gather_default ? L.n_sample : 0);
  L.gather_k = off;
  off = align_up(off + static_cast<size_t>(gather_rows) * key_row_bytes);
  L.gather_scale = off;
  off = align_up(off + static_cast<size_t>(gather_rows) * 4);
  long long cap = static_cast<long long>(tun.cap_mult) * topk;
  // the paper's 12k is sized for k = 2048; a small k leaves no slack for the looser gate a sample can give
  if (!tun.cap_mult_given && cap < 16384) cap = 16384;
  L.cap = static_cast<int>(cap > N ? N : cap);
  L.cand = off;
  off = align_up(off + static_cast<size_t>(T) * L.cap * 8);
  size_t slot_bytes = static_cast<size_t>(L.rpb) * N * 4;
  long long slots = static_cast<long long>(kFallbackScratchBudget / slot_bytes);
  const int own_slots = static_cast<int>(slots < 1 ? 1 : (slots > L.n_blocks ? L.n_blocks : slots));
  L.scratch = off;
  off = align_up(off + static_cast<size_t>(own_slots) * slot_bytes);
  // The candidate buffers are dead once the final select has run, and the fallback's dense rows are only written
  // after it: a fallback round uses the candidate region and the scratch behind it as one buffer, which makes the
  // rounds (two launches each, all of them enqueued whether or not a row is flagged) fewer.
  L.fb_base = L.cand;
  const size_t fb_total_slots = (off - L.cand) / slot_bytes;
  L.fb_slots = static_cast<int>(fb_total_slots > static_cast<size_t>(L.n_blocks) ? L.n_blocks : fb_total_slots);
  L.total = off;
  return L;
}

int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

int pick_seg_tiles(const Tun& tun, int n_keys, int n_blocks, int grid) {
  if (tun.segment_tiles > 0) return tun.segment_tiles;
  int n_tiles = (n_keys + kTileKeys - 1) / kTileKeys;
  int seg = 256;
  // at least two items per CTA, so that rows of different visible length even out; one per CTA for a chunk of one
  // or two row blocks, whose items all have the same length (measured: 84 instead of 102 us for 1 row over 2^20 keys)
  const long long want = (n_blocks <= 2 ? 1ll : 2ll) * grid;
  while (seg > 16 && static_cast<long long>(n_blocks) * ((n_tiles + seg - 1) / seg) < want) seg >>= 1;
  // Work items are dealt to the persistent CTAs round-robin, so the launch lasts as long as the CTA with the
  // most items: among the sizes from the one above down to 16 tiles, take the shortest such critical path (in key
  // tiles, plus a few tiles' worth of per-item start-up: the query block of an item is as large as four key tiles).
  // Matters for short chunks: 128 rows over 8192 tiles are 512 items of 256 tiles (4 rounds on 148 CTAs, the last
  // one half empty) or 592 items of 222 tiles.
  constexpr int kItemOverheadTiles = 4;
  long long best_cost = -1;
  int best = seg;
  for (int s = seg; s >= 16; --s) {
    const long long items = static_cast<long long>(n_blocks) * ((n_tiles + s - 1) / s);
    const long long rounds = (items + grid - 1) / grid;
    const long long cost = rounds * ((s < n_tiles ? s : n_tiles) + kItemOverheadTiles);
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best = s;
    }
  }
  return best;
}

// the default scan kernels, or the alternative fp8 scan, behind the same parameter block
cudaError_t launch_scan(bool abs_form, int dtype, int mode, const void* q, int T, const void* k, long long n_keys_view,
                        long long key_pitch_elems, const ScanParams& p, int grid, cudaStream_t stream) {
  if (abs_form) return launch_scan_fp8(mode, q, T, k, n_keys_view, key_pitch_elems, p, grid, stream);
  return launch_scan_mma(dtype, mode, q, T, k, n_keys_view, key_pitch_elems, p, grid, stream);
}

// Control block for entry points that have no workspace (lt_indexer_scores).
__device__ Control g_scores_ctl;

// ---- the generic path: dense scores of a few rows at a time, then a full-row select ----------
int run_unfused(int dtype, bool mma, const void* q, const float* w, const void* k, const float* k_scale, int T, int N, int H,
                int D, int topk, int causal_offset, int32_t* out_idx, float* out_score, float* scores, int rows_per_pass,
                Control* ctl, const Tun& tun, cudaStream_t stream) {
  const int grid = tun.grid > 0 ? tun.grid : sm_count();
  for (int r0 = 0; r0 < T; r0 += rows_per_pass) {
    const int r1 = (r0 + rows_per_pass < T) ? r0 + rows_per_pass : T;
    if (mma) {
      ScanParams p{};
      p.wait_limit_us = tun.wait_limit_us;
      p.w = w;
      p.k_scale = k_scale;
      p.ks_stride = 1;
      p.T = T;
      p.row_begin = r0;
      p.row_end = r1;
      p.n_keys = N;
      p.causal_offset = causal_offset;
      p.skip_masked_tiles = 0;
      p.seg_tiles = pick_seg_tiles(tun, N, (r1 - r0 + kRowsPerBlock - 1) / kRowsPerBlock, grid);
      p.topk = topk;
      p.dump = scores;
      p.dump_ld = N;
      p.ctl = ctl;
      LT_LAUNCH(launch_scan_mma(dtype, kModeDump, q, T, k, N, D, p, grid, stream));
    } else {
      LT_LAUNCH(launch_simt_scores(dtype, q, w, k, k_scale, T, N, H, D, causal_offset, r0, r1, scores, N, stream));
    }
    if (topk > 0) {
      SelectRowsParams sp{};
      sp.scores = scores;
      sp.ld = N;
      sp.n_blocks = r1 - r0;
      sp.row_begin = r0;
      sp.T = T;
      sp.N = N;
      sp.topk = topk;
      sp.causal_offset = causal_offset;
      sp.out_idx = out_idx;
      sp.out_score = out_score;
      sp.ctl = ctl;
      LT_LAUNCH(launch_select_rows(sp, stream));
    }
  }
  return LT_OK;
}

size_t elem_bytes(int dtype) { return dtype == LT_DTYPE_F32 ? 4 : (dtype == LT_DTYPE_BF16 ? 2 : 1); }

int topk_impl(int dtype, const void* q, const float* w, const void* k, const float* k_scale, int T, int N, int H, int D, int topk,
              int causal_offset, int32_t* out_idx, float* out_score, void* workspace, size_t workspace_bytes,
              const lt_tunables* tunables, cudaStream_t stream, const int32_t* sample_idx = nullptr, int n_given = 0,
              const int* page_table = nullptr, int n_pages = 0, long long pool_rows = 0, long long key_pitch_elems = 0) {
  int rc = check_problem(dtype, q, w, k, k_scale, T, N, H, D);
  if (rc != LT_OK) return rc;
  // distance between consecutive key rows in elements (a strided view of a wider cache); dense by default
  const long long key_pitch = key_pitch_elems > 0 ? key_pitch_elems : D;
  if (out_idx == nullptr || topk <= 0 || topk > N || topk > LT_MAX_TOPK) return LT_ERR_INVALID_ARG;
  const Tun tun = resolve_tunables(tunables);
  const bool fused = use_fused(tun, dtype, H, D);
  if ((tun.path == LT_PATH_FUSED || tun.path == LT_PATH_FUSED_ABS) && !fused) return LT_ERR_UNSUPPORTED;
  const int key_row_bytes = static_cast<int>(static_cast<size_t>(D) * elem_bytes(dtype));
  const bool paged = page_table != nullptr;
  if (paged && !fused) return LT_ERR_UNSUPPORTED;
  if (key_pitch != D && (!fused || paged || n_given > 0)) return LT_ERR_UNSUPPORTED;
  const bool abs_form = use_abs_form(tun, dtype, H, D);
  if (tun.path == LT_PATH_FUSED_ABS && !abs_form) return LT_ERR_UNSUPPORTED;
  const Layout L = make_layout(fused, T, N, topk, causal_offset, tun, n_given, key_row_bytes, paged, abs_form);
  const long long key_rows = paged ? pool_rows : N;  // rows the key tensor map covers
  if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) != 0 || workspace_bytes < L.total)
    return LT_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  Control* ctl = reinterpret_cast<Control*>(ws + L.ctl);
  LT_CUDA(cudaMemsetAsync(ws, 0, L.zero_end, stream));

  if (!fused) {
    return run_unfused(dtype, false, q, w, k, k_scale, T, N, H, D, topk, causal_offset, out_idx, out_score,
                       reinterpret_cast<float*>(ws + L.scratch), L.generic_rows, ctl, tun, stream);
  }

  const int grid = tun.grid > 0 ? tun.grid : sm_count();
  float* smin = reinterpret_cast<float*>(ws + L.smin);
  float* width = reinterpret_cast<float*>(ws + L.width);
  float* thr = reinterpret_cast<float*>(ws + L.thr);
  unsigned int* tail = reinterpret_cast<unsigned int*>(ws + L.tail);
  unsigned int* hist = reinterpret_cast<unsigned int*>(ws + L.hist);
  unsigned char* row_flag = ws + L.row_flag;
  unsigned int* block_flag = reinterpret_cast<unsigned int*>(ws + L.block_flag);
  int* fb_list = reinterpret_cast<int*>(ws + L.fb_list);
  float* sample = reinterpret_cast<float*>(ws + L.sample);
  uint2* cand = reinterpret_cast<uint2*>(ws + L.cand);
  float* scratch = reinterpret_cast<float*>(ws + L.fb_base);  // the fallback's dense rows (see make_layout)
  void* lin_q = abs_form ? ws + L.lin_q : nullptr;
  float* lin_scale = abs_form ? reinterpret_cast<float*>(ws + L.lin_scale) : nullptr;

  // 0. alternative fp8 scan: the linear part of Eq. 1 as extra operand rows of every query (used by all scans below)
  mark_phase(0, stream);
  if (abs_form) LT_LAUNCH(launch_lin_terms(q, w, T, lin_q, lin_scale, stream));

  // 1. sample phase: score n_sample strided keys of the common prefix with the same tensor-core path
  //    (or, with a caller-provided sample, a dense copy of the keys at the given positions)
  const void* sample_keys = k;
  const float* sample_scale = k_scale;
  long long sample_pitch = static_cast<long long>(L.sample_stride) * key_pitch;
  long long sample_ks_stride = L.sample_stride;
  if ((n_given > 0 || paged) && L.n_sample > 0) {
    LT_LAUNCH(launch_gather_keys(k, k_scale, n_given > 0 ? sample_idx : nullptr, L.sample_stride, L.n_sample, N, key_row_bytes,
                                 page_table, pool_rows, ctl, ws + L.gather_k, reinterpret_cast<float*>(ws + L.gather_scale),
                                 stream));
    sample_keys = ws + L.gather_k;
    if (k_scale != nullptr) sample_scale = reinterpret_cast<const float*>(ws + L.gather_scale);
    sample_pitch = D;
    sample_ks_stride = 1;
  }
  if (L.n_sample > 0) {
    ScanParams p{};
    p.wait_limit_us = tun.wait_limit_us;
    p.w = w;
    p.k_scale = sample_scale;
    p.ks_stride = sample_ks_stride;
    p.T = T;
    p.row_begin = 0;
    p.row_end = T;
    p.n_keys = L.n_sample;
    p.causal_offset = INT_MAX / 2;
    p.skip_masked_tiles = 0;
    p.seg_tiles = pick_seg_tiles(tun, L.n_sample, L.n_blocks, grid);
    p.topk = topk;
    p.dump = sample;
    p.dump_ld = L.n_sample;
    p.lin_q = lin_q;
    p.lin_scale = lin_scale;
    p.ctl = ctl;
    LT_LAUNCH(launch_scan(abs_form, dtype, kModeDump, q, T, sample_keys, L.n_sample, sample_pitch, p, grid, stream));
  }
  mark_phase(1, stream);
  LT_LAUNCH(launch_sample_stats(sample, T, L.n_sample, L.sample_rank, smin, width, thr, stream));
  mark_phase(2, stream);

  // 2. fused scan: score, gate, compact, count
  {
    ScanParams p{};
    p.wait_limit_us = tun.wait_limit_us;
    p.w = w;
    p.k_scale = k_scale;
    p.ks_stride = 1;
    p.T = T;
    p.row_begin = 0;
    p.row_end = T;
    p.n_keys = N;
    p.causal_offset = causal_offset;
    p.skip_masked_tiles = 1;
    p.seg_tiles = pick_seg_tiles(tun, N, L.n_blocks, grid);
    p.topk = topk;
    p.thr = thr;
    p.smin = smin;
    p.width = width;
    p.tail = tail;
    p.hist = hist;
    p.cand = cand;
    p.cap = L.cap;
    p.page_table = page_table;
    p.n_pages = n_pages;
    p.pool_pages = pool_rows / kPageKeys;
    p.debug_flags = tun.debug_flags;
    p.lin_q = lin_q;
    p.lin_scale = lin_scale;
    p.ctl = ctl;
    LT_LAUNCH(launch_scan(abs_form, dtype, kModeFilter, q, T, k, key_rows, key_pitch, p, grid, stream));
  }

  // 3. final select over the survivors; rows it cannot finish exactly are flagged
  mark_phase(3, stream);
  {
    FinalSelectParams p{};
    p.tail = tail;
    p.hist = hist;
    p.cand = cand;
    p.smin = smin;
    p.width = width;
    p.cap = L.cap;
    p.T = T;
    p.N = N;
    p.topk = topk;
    p.causal_offset = causal_offset;
    p.out_idx = out_idx;
    p.out_score = out_score;
    p.row_flag = row_flag;
    p.block_flag = block_flag;
    p.fb_list = fb_list;
    p.rows_per_block = L.rpb;
    p.ctl = ctl;
    LT_LAUNCH(launch_final_select(p, stream));
  }

  // 4. exact fallback for flagged rows.  The host does not know how many there are, so it
  // enqueues enough rounds for all blocks; rounds with nothing to do exit at once.
  mark_phase(4, stream);
  const int rounds = (L.n_blocks + L.fb_slots - 1) / L.fb_slots;
  for (int r = 0; r < rounds; ++r) {
    ScanParams p{};
    p.wait_limit_us = tun.wait_limit_us;
    p.w = w;
    p.k_scale = k_scale;
    p.ks_stride = 1;
    p.T = T;
    p.row_begin = 0;
    p.row_end = T;
    p.n_keys = N;
    p.causal_offset = causal_offset;
    p.skip_masked_tiles = 0;
    p.seg_tiles = pick_seg_tiles(tun, N, L.fb_slots, grid);
    p.topk = topk;
    p.dump = scratch;
    p.dump_ld = N;
    p.fb_list = fb_list;
    p.fb_blocks = &ctl->fb_blocks;
    p.fb_round_base = r * L.fb_slots;
    p.fb_slots = L.fb_slots;
    p.page_table = page_table;
    p.n_pages = n_pages;
    p.pool_pages = pool_rows / kPageKeys;
    p.lin_q = lin_q;
    p.lin_scale = lin_scale;
    p.ctl = ctl;
    LT_LAUNCH(launch_scan(abs_form, dtype, kModeDump, q, T, k, key_rows, key_pitch, p, grid, stream));
    SelectRowsParams sp{};
    sp.scores = scratch;
    sp.ld = N;
    sp.n_blocks = L.fb_slots * L.rpb;
    sp.rows_per_block = L.rpb;
    sp.T = T;
    sp.N = N;
    sp.topk = topk;
    sp.causal_offset = causal_offset;
    sp.out_idx = out_idx;
    sp.out_score = out_score;
    sp.fb_list = fb_list;
    sp.fb_blocks = &ctl->fb_blocks;
    sp.fb_round_base = r * L.fb_slots;
    sp.row_flag = row_flag;
    sp.ctl = ctl;
    LT_LAUNCH(launch_select_rows(sp, stream));
  }
  mark_phase(5, stream);
  return LT_OK;
}

// ---- fixed scratch of the allocation-free entry point -------------------------------------------
// Lives in the library's device image: every GPU whose context loads the library holds these
// 16 MiB until the process exits.  Layout: a 256-byte status block, then dense fp32 score rows.
constexpr size_t kStaticScratchBytes = LT_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address; the
// address each device gave the array is looked up once per device and cached here.
std::mutex g_static_mu;
void* g_static_ptr[64] = {nullptr};

int static_scratch_address(void** out) {
  int dev = 0;
  LT_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return LT_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (g_static_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    LT_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
    g_static_ptr[dev] = ptr;
  }
  *out = g_static_ptr[dev];
  return LT_OK;
}

// ---- library-owned workspace of the 13-argument entry point -----------------------------------
// One arena per device, grown on demand; g_arena_mu is held while a call's work is enqueued.
constexpr int kMaxDevices = 64;
std::mutex g_arena_mu;
void* g_arena[kMaxDevices] = {nullptr};
size_t g_arena_bytes[kMaxDevices] = {0};

}  // namespace
}  // namespace lt

using namespace lt;

extern "C" {

int lt_version(void) { return LT_VERSION; }

const char* lt_strerror(int code) {
  switch (code) {
    case LT_OK: return "ok";
    case LT_ERR_INVALID_ARG: return "invalid argument";
    case LT_ERR_UNSUPPORTED: return "unsupported dtype or shape";
    case LT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case LT_ERR_CUDA: return "CUDA runtime error";
    case LT_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of lt_indexer_topk_static (N * 4 bytes must fit in LT_STATIC_SCRATCH_BYTES - 256)";
    default: return "unknown error code";
  }
}

int lt_last_cuda_error(void) { return g_last_cuda_error; }

size_t lt_indexer_topk_workspace_bytes(int dtype, int T, int N, int H, int D, int topk, const lt_tunables* tunables) {
  if ((dtype != LT_DTYPE_F32 && dtype != LT_DTYPE_BF16 && dtype != LT_DTYPE_E4M3) || T <= 0 || N <= 0 || H <= 0 || D <= 0 ||
      topk <= 0 || topk > N || topk > LT_MAX_TOPK)
    return 0;
  const Tun tun = resolve_tunables(tunables);
  // the sample can never be larger with a different causal_offset than with the whole context visible
  return make_layout(use_fused(tun, dtype, H, D), T, N, topk, N - 1, tun, 0, 0, false, use_abs_form(tun, dtype, H, D)).total;
}

int lt_indexer_topk_sampled(int dtype, const void* q, const float* w, const void* k, const float* k_scale, int T, int N, int H,
                            int D, int topk, int causal_offset, const int32_t* sample_idx, int n_sample, int32_t* out_idx,
                            float* out_score, void* workspace, size_t workspace_bytes, const lt_tunables* tunables,
                            void* stream) {
  if (sample_idx == nullptr || n_sample <= 0 || n_sample > LT_MAX_SAMPLE) return LT_ERR_INVALID_ARG;
  return topk_impl(dtype, q, w, k, k_scale, T, N, H, D, topk, causal_offset, out_idx, out_score, workspace, workspace_bytes,
                   tunables, static_cast<cudaStream_t>(stream), sample_idx, n_sample);
}

size_t lt_indexer_topk_sampled_workspace_bytes(int dtype, int T, int N, int H, int D, int topk, int n_sample,
                                               const lt_tunables* tunables) {
  if ((dtype != LT_DTYPE_F32 && dtype != LT_DTYPE_BF16 && dtype != LT_DTYPE_E4M3) || T <= 0 || N <= 0 || H <= 0 || D <= 0 ||
      topk <= 0 || topk > N || topk > LT_MAX_TOPK || n_sample <= 0 || n_sample > LT_MAX_SAMPLE)
    return 0;
  const Tun tun = resolve_tunables(tunables);
  return make_layout(use_fused(tun, dtype, H, D), T, N, topk, N - 1, tun, n_sample,
                     static_cast<int>(static_cast<size_t>(D) * elem_bytes(dtype)), false, use_abs_form(tun, dtype, H, D)).total;
}

int lt_indexer_topk_paged(int dtype, const void* q, const float* w, const void* k_pool, const float* k_scale_pool,
                          const int32_t* page_table, int n_pages, long long pool_rows, int T, int N, int H, int D, int topk,
                          int causal_offset, int32_t* out_idx, float* out_score, void* workspace, size_t workspace_bytes,
                          const lt_tunables* tunables, void* stream) {
  if (page_table == nullptr || n_pages <= 0 || pool_rows <= 0 || pool_rows % kPageKeys != 0 ||
      static_cast<long long>(n_pages) * kPageKeys < N)
    return LT_ERR_INVALID_ARG;
  return topk_impl(dtype, q, w, k_pool, k_scale_pool, T, N, H, D, topk, causal_offset, out_idx, out_score, workspace,
                   workspace_bytes, tunables, static_cast<cudaStream_t>(stream), nullptr, 0, page_table, n_pages, pool_rows);
}

size_t lt_indexer_topk_paged_workspace_bytes(int dtype, int T, int N, int H, int D, int topk, const lt_tunables* tunables) {
  if ((dtype != LT_DTYPE_BF16 && dtype != LT_DTYPE_E4M3) || T <= 0 || N <= 0 || H <= 0 || D <= 0 || topk <= 0 || topk > N ||
      topk > LT_MAX_TOPK)
    return 0;
  const Tun tun = resolve_tunables(tunables);
  if (!use_fused(tun, dtype, H, D)) return 0;
  return make_layout(true, T, N, topk, N - 1, tun, 0, static_cast<int>(static_cast<size_t>(D) * elem_bytes(dtype)), true,
                     use_abs_form(tun, dtype, H, D)).total;
}

size_t lt_topk_frequent_workspace_bytes(int N) {
  if (N <= 0) return 0;
  return align_up(static_cast<size_t>(N) * 4) + align_up(rank_scratch_bytes(LT_MAX_TOPK));
}

int lt_topk_frequent(const int32_t* idx, int T, int topk, int N, int n_out, int32_t* out_pos, int32_t* out_count,
                     void* workspace, size_t workspace_bytes, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (idx == nullptr || out_pos == nullptr || T <= 0 || topk <= 0 || N <= 0 || n_out <= 0 || n_out > N || n_out > LT_MAX_TOPK ||
      T > (1 << 24))
    return LT_ERR_INVALID_ARG;
  if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) != 0 ||
      workspace_bytes < lt_topk_frequent_workspace_bytes(N))
    return LT_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  unsigned int* counts = reinterpret_cast<unsigned int*>(ws);
  void* scratch = ws + align_up(static_cast<size_t>(N) * 4);
  LT_CUDA(cudaMemsetAsync(counts, 0, static_cast<size_t>(N) * 4, stream));
  LT_LAUNCH(launch_count_positions(idx, static_cast<long long>(T) * topk, N, counts, stream));
  // rank the N (count, position) pairs with a grid-wide radix select and order the n_out winners; no position can
  // occur more often than there are entries
  LT_LAUNCH(launch_rank_counts(counts, N, n_out, static_cast<unsigned long long>(T) * topk, scratch, out_pos, out_count, stream));
  return LT_OK;
}

int lt_dsa_union_mask(const int32_t* idx, int T, int topk, int N, int group, int32_t* union_pos, int32_t* union_len,
                      uint32_t* member_mask, void* stream) {
  if (idx == nullptr || union_pos == nullptr || union_len == nullptr || member_mask == nullptr || T <= 0 || topk <= 0 || N <= 0 ||
      group <= 0 || static_cast<long long>(group) * topk > (1ll << 24))
    return LT_ERR_INVALID_ARG;
  LT_LAUNCH(launch_dsa_union(idx, T, topk, N, group, union_pos, union_len, member_mask, static_cast<cudaStream_t>(stream)));
  return LT_OK;
}

int lt_indexer_sample_plan(int N, int topk, int causal_offset, const lt_tunables* tunables, int plan3[3]) {
  if (plan3 == nullptr || N <= 0 || topk <= 0 || topk > N || topk > LT_MAX_TOPK) return LT_ERR_INVALID_ARG;
  const Layout L = make_layout(true, 1, N, topk, causal_offset, resolve_tunables(tunables));
  plan3[0] = L.n_sample;
  plan3[1] = L.sample_stride;
  plan3[2] = L.sample_rank;
  return LT_OK;
}

int lt_indexer_topk_ex(int dtype, const void* q, const float* w, const void* k, const float* k_scale, int T, int N, int H, int D,
                       int topk, int causal_offset, int32_t* out_idx, float* out_score, void* workspace, size_t workspace_bytes,
                       const lt_tunables* tunables, void* stream) {
  return topk_impl(dtype, q, w, k, k_scale, T, N, H, D, topk, causal_offset, out_idx, out_score, workspace, workspace_bytes,
                   tunables, static_cast<cudaStream_t>(stream));
}

int lt_indexer_topk_strided(int dtype, const void* q, const float* w, const void* k, long long k_pitch_elems,
                            const float* k_scale, int T, int N, int H, int D, int topk, int causal_offset, int32_t* out_idx,
                            float* out_score, void* workspace, size_t workspace_bytes, const lt_tunables* tunables,
                            void* stream) {
  if (k_pitch_elems < D) return LT_ERR_INVALID_ARG;
  // the tensor map wants row pitches that are multiples of 16 bytes
  if ((static_cast<size_t>(k_pitch_elems) * elem_bytes(dtype)) % 16 != 0) return LT_ERR_INVALID_ARG;
  return topk_impl(dtype, q, w, k, k_scale, T, N, H, D, topk, causal_offset, out_idx, out_score, workspace, workspace_bytes,
                   tunables, static_cast<cudaStream_t>(stream), nullptr, 0, nullptr, 0, 0, k_pitch_elems);
}

int lt_indexer_topk(const void* q, const float* w, const void* k, const float* k_scale, int T, int N, int H, int D, int topk,
                    int causal_offset, int32_t* out_idx, float* out_score, void* stream) {
  const int dtype = (k_scale != nullptr) ? LT_DTYPE_E4M3 : LT_DTYPE_BF16;
  int rc = check_problem(dtype, q, w, k, k_scale, T, N, H, D);
  if (rc != LT_OK) return rc;
  if (out_idx == nullptr || topk <= 0 || topk > N || topk > LT_MAX_TOPK) return LT_ERR_INVALID_ARG;
  const size_t need = lt_indexer_topk_workspace_bytes(dtype, T, N, H, D, topk, nullptr);
  if (need == 0) return LT_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_arena_mu);
  int dev = 0;
  LT_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return LT_ERR_UNSUPPORTED;
  if (g_arena[dev] == nullptr || g_arena_bytes[dev] < need) {
    if (g_arena[dev] != nullptr) {
      // earlier calls on this device may still be using the old arena: wait for them before it is freed
      LT_CUDA(cudaDeviceSynchronize());
      cudaFree(g_arena[dev]);
      g_arena[dev] = nullptr;
      g_arena_bytes[dev] = 0;
    }
    LT_CUDA(cudaMalloc(&g_arena[dev], need));
    g_arena_bytes[dev] = need;
  }
  return topk_impl(dtype, q, w, k, k_scale, T, N, H, D, topk, causal_offset, out_idx, out_score, g_arena[dev], g_arena_bytes[dev],
                   nullptr, static_cast<cudaStream_t>(stream));
}

int lt_indexer_scores(int dtype, const void* q, const float* w, const void* k, const float* k_scale, int T, int N, int H, int D,
                      int causal_offset, int row_begin, int row_end, float* out_scores, int path, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  int rc = check_problem(dtype, q, w, k, k_scale, T, N, H, D);
  if (rc != LT_OK) return rc;
  if (out_scores == nullptr || row_begin < 0 || row_end > T || row_begin > row_end) return LT_ERR_INVALID_ARG;
  if (row_begin == row_end) return LT_OK;
  Tun tun = resolve_tunables(nullptr);
  tun.path = path;
  const bool mma = use_fused(tun, dtype, H, D);
  if (path == LT_PATH_FUSED && !mma) return LT_ERR_UNSUPPORTED;
  Control* ctl = nullptr;
  LT_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&ctl), g_scores_ctl));
  // run_unfused with topk == 0 only dumps; rows are written straight to the caller's matrix
  const float* kk = k_scale;
  int rows = row_end - row_begin;
  const bool abs_form = use_abs_form(tun, dtype, H, D);
  if (path == LT_PATH_FUSED_ABS && !abs_form) return LT_ERR_UNSUPPORTED;
  if (mma) {
    // the scan kernel addresses dump rows relative to row_begin
    ScanParams p{};
    p.wait_limit_us = tun.wait_limit_us;
    const int grid = sm_count();
    void* lin = nullptr;
    if (abs_form) {
      // linear terms of all rows: a stream-ordered temporary (this entry point has no workspace)
      const size_t qb = align_up(lin_q_bytes(T));
      LT_CUDA(cudaMallocAsync(&lin, qb + lin_scale_bytes(T), stream));
      p.lin_q = lin;
      p.lin_scale = reinterpret_cast<float*>(static_cast<uint8_t*>(lin) + qb);
      LT_LAUNCH(launch_lin_terms(q, w, T, lin, const_cast<float*>(p.lin_scale), stream));
    }
    p.w = w;
    p.k_scale = kk;
    p.ks_stride = 1;
    p.T = T;
    p.row_begin = row_begin;
    p.row_end = row_end;
    p.n_keys = N;
    p.causal_offset = causal_offset;
    p.skip_masked_tiles = 0;
    const int rpb = abs_form ? kRowsPerBlockFp8 : kRowsPerBlock;
    p.seg_tiles = pick_seg_tiles(tun, N, (rows + rpb - 1) / rpb, grid);
    p.dump = out_scores;
    p.dump_ld = N;
    p.ctl = ctl;
    LT_LAUNCH(launch_scan(abs_form, dtype, kModeDump, q, T, k, N, D, p, grid, stream));
    if (lin != nullptr) LT_CUDA(cudaFreeAsync(lin, stream));
  } else {
    LT_LAUNCH(launch_simt_scores(dtype, q, w, k, kk, T, N, H, D, causal_offset, row_begin, row_end, out_scores, N, stream));
  }
  return LT_OK;
}

// ---- k-NN (inner-product) variant --------------------------------------------------------------
namespace {

int knn_check(int dtype, const void* q, const void* x, int T, int N, int D) {
  if (dtype != LT_DTYPE_BF16) return LT_ERR_UNSUPPORTED;
  if (q == nullptr || x == nullptr || T <= 0 || N <= 0 || D <= 0) return LT_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(x)) return LT_ERR_INVALID_ARG;
  if (!scan_knn_supported(D)) return LT_ERR_UNSUPPORTED;
  return LT_OK;
}

int knn_seg_tiles(const Tun& tun, int n_keys, int grid) {
  if (tun.segment_tiles > 0) return tun.segment_tiles;
  const int n_tiles = (n_keys + kTileKeys - 1) / kTileKeys;
  int seg = 32;
  while (seg > 2 && (n_tiles + seg - 1) / seg < 4 * grid) seg >>= 1;
  return seg;
}

}  // namespace

size_t lt_knn_topk_workspace_bytes(int dtype, int T, int N, int D, int topk, const lt_tunables* tunables) {
  if (dtype != LT_DTYPE_BF16 || T <= 0 || N <= 0 || !scan_knn_supported(D) || topk <= 0 || topk > N || topk > LT_MAX_TOPK) return 0;
  return make_layout(true, T, N, topk, N - 1, resolve_tunables(tunables)).total;
}

int lt_knn_scores(int dtype, const void* q, const void* x, int T, int N, int D, int row_begin, int row_end, float* out_scores,
                  void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  int rc = knn_check(dtype, q, x, T, N, D);
  if (rc != LT_OK) return rc;
  if (out_scores == nullptr || row_begin < 0 || row_end > T || row_begin > row_end) return LT_ERR_INVALID_ARG;
  if (row_begin == row_end) return LT_OK;
  Control* ctl = nullptr;
  LT_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&ctl), g_scores_ctl));
  const int grid = sm_count();
  KnnScanParams p{};
  p.T = T;
  p.row_begin = row_begin;
  p.row_end = row_end;
  p.n_keys = N;
  p.D = D;
  p.seg_tiles = knn_seg_tiles(resolve_tunables(nullptr), N, grid);
  p.dump = out_scores;
  p.dump_ld = N;
  p.ctl = ctl;
  LT_LAUNCH(launch_scan_knn(kModeDump, q, T, x, N, D, p, grid, stream));
  return LT_OK;
}

int lt_knn_topk(int dtype, const void* q, const void* x, int T, int N, int D, int topk, int32_t* out_idx, float* out_score,
                void* workspace, size_t workspace_bytes, const lt_tunables* tunables, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  int rc = knn_check(dtype, q, x, T, N, D);
  if (rc != LT_OK) return rc;
  if (out_idx == nullptr || topk <= 0 || topk > N || topk > LT_MAX_TOPK) return LT_ERR_INVALID_ARG;
  const Tun tun = resolve_tunables(tunables);
  const Layout L = make_layout(true, T, N, topk, N - 1, tun);  // every query sees the whole corpus
  if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) != 0 || workspace_bytes < L.total)
    return LT_ERR_WORKSPACE;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  Control* ctl = reinterpret_cast<Control*>(ws + L.ctl);
  LT_CUDA(cudaMemsetAsync(ws, 0, L.zero_end, stream));
  const int grid = tun.grid > 0 ? tun.grid : sm_count();
  float* smin = reinterpret_cast<float*>(ws + L.smin);
  float* width = reinterpret_cast<float*>(ws + L.width);
  float* thr = reinterpret_cast<float*>(ws + L.thr);
  unsigned int* tail = reinterpret_cast<unsigned int*>(ws + L.tail);
  unsigned int* hist = reinterpret_cast<unsigned int*>(ws + L.hist);
  unsigned char* row_flag = ws + L.row_flag;
  unsigned int* block_flag = reinterpret_cast<unsigned int*>(ws + L.block_flag);
  int* fb_list = reinterpret_cast<int*>(ws + L.fb_list);
  float* sample = reinterpret_cast<float*>(ws + L.sample);
  uint2* cand = reinterpret_cast<uint2*>(ws + L.cand);
  float* scratch = reinterpret_cast<float*>(ws + L.fb_base);  // the fallback's dense rows (see make_layout)

  // 1. sample phase (paper Sec. 3.2 "Sampling": k-NN needs no history-based sample; a strided subsample of
  //    the corpus is used here), scored by the same tensor-core kernel
  mark_phase(0, stream);
  if (L.n_sample > 0) {
    KnnScanParams p{};
    p.wait_limit_us = tun.wait_limit_us;
    p.T = T;
    p.row_begin = 0;
    p.row_end = T;
    p.n_keys = L.n_sample;
    p.D = D;
    p.seg_tiles = knn_seg_tiles(tun, L.n_sample, grid);
    p.dump = sample;
    p.dump_ld = L.n_sample;
    p.ctl = ctl;
    LT_LAUNCH(launch_scan_knn(kModeDump, q, T, x, L.n_sample, static_cast<long long>(L.sample_stride) * D, p, grid, stream));
  }
  mark_phase(1, stream);
  LT_LAUNCH(launch_sample_stats(sample, T, L.n_sample, L.sample_rank, smin, width, thr, stream));
  mark_phase(2, stream);

  // 2. fused scan: one pass over the corpus
  {
    KnnScanParams p{};
    p.wait_limit_us = tun.wait_limit_us;
    p.T = T;
    p.row_begin = 0;
    p.row_end = T;
    p.n_keys = N;
    p.D = D;
    p.seg_tiles = knn_seg_tiles(tun, N, grid);
    p.topk = topk;
    p.thr = thr;
    p.smin = smin;
    p.width = width;
    p.tail = tail;
    p.hist = hist;
    p.cand = cand;
    p.cap = L.cap;
    p.ctl = ctl;
    LT_LAUNCH(launch_scan_knn(kModeFilter, q, T, x, N, D, p, grid, stream));
  }

  // 3. final select; rows it cannot finish exactly are flagged
  mark_phase(3, stream);
  {
    FinalSelectParams p{};
    p.tail = tail;
    p.hist = hist;
    p.cand = cand;
    p.smin = smin;
    p.width = width;
    p.cap = L.cap;
    p.T = T;
    p.N = N;
    p.topk = topk;
    p.causal_offset = N;  // no causal mask
    p.out_idx = out_idx;
    p.out_score = out_score;
    p.row_flag = row_flag;
    p.block_flag = block_flag;
    p.fb_list = fb_list;
    p.rows_per_block = kRowsPerBlock;
    p.ctl = ctl;
    LT_LAUNCH(launch_final_select(p, stream));
  }

  // 4. exact fallback, as many rows at a time as the scratch holds (the corpus is streamed once per round
  //    however many rows are scored): dense scores of the round's rows (a launch in whose rows nobody was
  //    flagged returns at once), then the full-row select for the flagged rows
  mark_phase(4, stream);
  const int round_rows = L.fb_slots * kRowsPerBlock;
  for (int r0 = 0; r0 < T; r0 += round_rows) {
    const int r1 = r0 + round_rows < T ? r0 + round_rows : T;
    KnnScanParams p{};
    p.wait_limit_us = tun.wait_limit_us;
    p.T = T;
    p.row_begin = r0;
    p.row_end = r1;
    p.n_keys = N;
    p.D = D;
    p.seg_tiles = knn_seg_tiles(tun, N, grid);
    p.dump = scratch;
    p.dump_ld = N;
    p.fb_flag = block_flag;
    p.ctl = ctl;
    LT_LAUNCH(launch_scan_knn(kModeDump, q, T, x, N, D, p, grid, stream));
    SelectRowsParams sp{};
    sp.scores = scratch;
    sp.ld = N;
    sp.n_blocks = r1 - r0;
    sp.row_begin = r0;
    sp.T = T;
    sp.N = N;
    sp.topk = topk;
    sp.causal_offset = N;
    sp.out_idx = out_idx;
    sp.out_score = out_score;
    sp.row_flag = row_flag;
    sp.ctl = ctl;
    LT_LAUNCH(launch_select_rows(sp, stream));
  }
  mark_phase(5, stream);
  return LT_OK;
}

int lt_unfused_topk(int dtype, const void* q, const float* w, const void* k, const float* k_scale, int T, int N, int H, int D,
                    int topk, int causal_offset, int32_t* out_idx, float* out_score, float* score_buf, size_t score_buf_bytes,
                    int path, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  int rc = check_problem(dtype, q, w, k, k_scale, T, N, H, D);
  if (rc != LT_OK) return rc;
  if (out_idx == nullptr || topk <= 0 || topk > N || topk > LT_MAX_TOPK) return LT_ERR_INVALID_ARG;
  if (score_buf == nullptr || (reinterpret_cast<uintptr_t>(score_buf) & (kAlign - 1)) != 0) return LT_ERR_WORKSPACE;
  Tun tun = resolve_tunables(nullptr);
  tun.path = path;
  const bool mma = use_fused(tun, dtype, H, D);
  if (path == LT_PATH_FUSED && !mma) return LT_ERR_UNSUPPORTED;
  if (path == LT_PATH_FUSED_ABS) return LT_ERR_UNSUPPORTED;  // the decoupled baseline scores with the default kernels
  // the first 256 bytes of score_buf hold the status block (readable with lt_read_status)
  if (score_buf_bytes < kAlign + static_cast<size_t>(N) * 4) return LT_ERR_WORKSPACE;
  long long rows = static_cast<long long>((score_buf_bytes - kAlign) / (static_cast<size_t>(N) * 4));
  if (rows > T) rows = T;
  if (mma && rows >= kRowsPerBlock) rows -= rows % kRowsPerBlock;
  Control* ctl = reinterpret_cast<Control*>(score_buf);
  LT_CUDA(cudaMemsetAsync(ctl, 0, kAlign, stream));
  float* scores = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(score_buf) + kAlign);
  return run_unfused(dtype, mma, q, w, k, k_scale, T, N, H, D, topk, causal_offset, out_idx, out_score, scores,
                     static_cast<int>(rows), ctl, tun, stream);
}

int lt_indexer_topk_static(int dtype, const void* q, const float* w, const void* k, const float* k_scale, int T, int N, int H,
                           int D, int topk, int causal_offset, int32_t* out_idx, float* out_score, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  int rc = check_problem(dtype, q, w, k, k_scale, T, N, H, D);
  if (rc != LT_OK) return rc;
  if (out_idx == nullptr || topk <= 0 || topk > N || topk > LT_MAX_TOPK) return LT_ERR_INVALID_ARG;
  // one dense score row (N floats) must fit behind the status block
  if (static_cast<size_t>(N) * 4 > kStaticScratchBytes - kAlign) return LT_ERR_TOO_LARGE;
  void* base = nullptr;
  rc = static_scratch_address(&base);  // the first call on a device looks the address up
  if (rc != LT_OK) return rc;
  Tun tun = resolve_tunables(nullptr);
  const bool mma = use_fused(tun, dtype, H, D);
  long long rows = static_cast<long long>((kStaticScratchBytes - kAlign) / (static_cast<size_t>(N) * 4));
  if (rows > T) rows = T;
  if (mma && rows >= kRowsPerBlock) rows -= rows % kRowsPerBlock;
  // the array keeps whatever the previous call left: the status block must start at zero; the
  // score rows are fully rewritten before they are read
  Control* ctl = static_cast<Control*>(base);
  LT_CUDA(cudaMemsetAsync(ctl, 0, kAlign, stream));
  float* scores = reinterpret_cast<float*>(static_cast<unsigned char*>(base) + kAlign);
  return run_unfused(dtype, mma, q, w, k, k_scale, T, N, H, D, topk, causal_offset, out_idx, out_score, scores,
                     static_cast<int>(rows), ctl, tun, stream);
}

int lt_read_status(const void* workspace, int* status8_host, void* stream) {
  if (status8_host == nullptr) return LT_ERR_INVALID_ARG;
  const void* src = workspace;
  if (src == nullptr) {
    std::lock_guard<std::mutex> lock(g_arena_mu);
    int dev = 0;
    LT_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < kMaxDevices) src = g_arena[dev];
  }
  if (src == nullptr) return LT_ERR_WORKSPACE;
  LT_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  LT_CUDA(cudaMemcpy(status8_host, src, 8 * sizeof(int), cudaMemcpyDeviceToHost));
  return LT_OK;
}

int lt_indexer_topk_static_max_keys(void) { return static_cast<int>((kStaticScratchBytes - kAlign) / 4); }

int lt_read_status_static(int* status8_host, void* stream) {
  if (status8_host == nullptr) return LT_ERR_INVALID_ARG;
  void* base = nullptr;
  int rc = static_scratch_address(&base);
  if (rc != LT_OK) return rc;
  LT_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  LT_CUDA(cudaMemcpy(status8_host, base, 8 * sizeof(int), cudaMemcpyDeviceToHost));
  return LT_OK;
}

int lt_debug_wait_timeout(int limit_us, int* result2_device, void* stream) {
  if (limit_us <= 0 || result2_device == nullptr) return LT_ERR_INVALID_ARG;
  LT_LAUNCH(launch_wait_timeout_probe(static_cast<unsigned int>(limit_us), result2_device, static_cast<cudaStream_t>(stream)));
  return LT_OK;
}

int lt_debug_umma_stream(int pair, int iters, int* status_device, void* stream) {
  if (iters <= 0 || iters > (1 << 24) || status_device == nullptr) return LT_ERR_INVALID_ARG;
  int grid = sm_count();
  if (pair) grid &= ~1;
  if (grid <= 0) return LT_ERR_CUDA;
  LT_LAUNCH(launch_umma_stream(pair != 0, iters, status_device, grid, static_cast<cudaStream_t>(stream)));
  return LT_OK;
}

unsigned long long lt_launch_count(void) { return g_launches.load(); }

int lt_set_profiling(int enable) {
  if (enable) {
    int dev = 0;
    LT_CUDA(cudaGetDevice(&dev));
    if (g_events_dev != dev) {
      for (int i = 0; i <= kPhases; ++i) {
        if (g_events[i] != nullptr) cudaEventDestroy(g_events[i]);
        g_events[i] = nullptr;
        LT_CUDA(cudaEventCreate(&g_events[i]));
      }
      g_events_dev = dev;
    }
  }
  g_profiling = enable != 0;
  return LT_OK;
}

int lt_read_phase_ms(float* ms5_host, void* stream) {
  if (ms5_host == nullptr) return LT_ERR_INVALID_ARG;
  if (g_events_dev < 0) return LT_ERR_INVALID_ARG;
  LT_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  for (int i = 0; i < kPhases; ++i) LT_CUDA(cudaEventElapsedTime(&ms5_host[i], g_events[i], g_events[i + 1]));
  return LT_OK;
}

void lt_shutdown(void) {
  std::lock_guard<std::mutex> lock(g_arena_mu);
  int cur = 0;
  if (cudaGetDevice(&cur) != cudaSuccess) cur = -1;
  for (int dev = 0; dev < kMaxDevices; ++dev) {
    if (g_arena[dev] == nullptr) continue;
    // the arena belongs to `dev`: make it current, wait for its work, free
    if (cudaSetDevice(dev) == cudaSuccess) {
      cudaDeviceSynchronize();
      cudaFree(g_arena[dev]);
    }
    g_arena[dev] = nullptr;
    g_arena_bytes[dev] = 0;
  }
  if (cur >= 0) cudaSetDevice(cur);
}

}  // extern "C"
