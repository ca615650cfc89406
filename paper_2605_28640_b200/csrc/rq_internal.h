// Internal declarations shared by the library's translation units (host side).
// Not part of the public ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "rq.h"

namespace rq {

// ---- geometry of the prefill kernel ----
constexpr int kScanThreads = 512;  // threads per CTA

constexpr int kScanChannels = 32;   // channels of one prefill CTA (two per lane of a half-warp)
constexpr int kScanRunTokens = 8;   // consecutive positions that one half-warp of a prefill CTA owns in a tile

// ---- decode-side geometry ----
constexpr int kScoreWarps = 4;         // warps per scoring CTA, each with its own copy pipeline
constexpr int kScoreRingBytes = 64 * 1024;   // shared-memory ring of one scoring CTA (all warps): three CTAs per SM
constexpr int kAttendWarps = 4;        // warps per flash-decode CTA, each with its own copy pipeline
constexpr int kAttendRingBytes = 64 * 1024;  // shared-memory ring of one flash-decode CTA (all warps): three CTAs per SM
constexpr int kAttendMaxWarps = 2048;  // upper bound of the warps of a flash-decode grid
constexpr int kCtrStride = 64;         // int32 between the counters of two heads (256 bytes: different L2 lines)
constexpr int kTopkThreads = 1024;     // threads of the selection CTA
constexpr int64_t kTopkPrefetchBytes = 16ll << 20;   // selected pages the selection kernel sends towards L2, all heads together
constexpr int kSmallStepPages = 256;   // heads of up to this many pages are scored and selected by one CTA in one launch ...
constexpr int kSmallStepMinHeads = 16; // ... when there are at least this many heads to spread over the SMs
constexpr int kTopkMaxPerThread = 32;  // => at most 32768 pages per head
constexpr int kTargetSMs = 148;        // B200

// ---- the one-launch decode step (rq_step.cu) ----
constexpr int kStepMaxHeads = 256;     // the one-launch step serves at most this many (batch, head) pairs
constexpr int kStepBins = 2048;        // value buckets of a head's score histogram
constexpr int kStepCtrInts = 16;       // int32 per head and counter set (64 bytes)
constexpr int kTopkFastPages = 10240;  // heads of up to this many pages are selected from the scoring kernel's histogram,
constexpr int kTopkHistMinPages = 6144; // and of at least this many: below, counting the pages while scoring costs more than the selection saves

// ---- workspace carving (byte offsets, every region 256-byte aligned) ----
struct WorkspaceLayout {
    size_t status;    // int32[64]
    size_t tickets;   // int32[BH * kCtrStride]: per head, flash-decode ticket / slot / done counters (+0..2) and the scoring ticket counter (+3)
    size_t scores;    // float [BH][page_capacity]
    size_t sel;       // int32 [BH][max_budget]
    size_t partial;   // float [BH][slots per head][D + 4]: flash-decode partials
    size_t staging;   // 5 * [BH][D] elements of 4 bytes (host-call staging)
    size_t scan;      // kScanScratchBytes: the maps and entry states of the prefill's time chunks (few heads, long prompts)
    // the one-launch step (present when BH <= kStepMaxHeads, otherwise empty); everything from
    // `status` up to `scores` is cleared by rq_cache_reset, which is why these regions sit there
    size_t absmax;    // float [2][BH]: largest |stored key| of every head, two copies (read one, write the other)
    size_t step_ctr;  // int32 [2][BH][kStepCtrInts]: two sets of per-head counters, used by alternate steps
    size_t list;      // int2 [BH][max_budget]: page lists of the one-launch step, entries (page, step number)
    size_t hist;      // uint32 [BH][kStepBins]: score histogram of a head, all zero between steps
    size_t range;     // float2 [BH]: (lo, scale) of the bucket map the head's histogram was filled with
    size_t total;
};

WorkspaceLayout workspace_layout(const rq_config &c);

// ---- kernel launchers (defined in rq_scan.cu, rq_score.cu, rq_topk.cu, rq_attend.cu, rq_step.cu) ----
struct ScanArgs {
    const void *k, *v, *g;
    int64_t sb, st, sh;     // element strides of k, v, g
    void *kv, *meta;
    float *state;
    int B, H, D, S, dtype, gate_dtype;
    int64_t len0, T, page_cap;
    float *absmax;      // [2][BH] largest |stored key| per head, both copies brought up to date (NULL: not tracked)
    float *chunk_scratch;   // kScanScratchBytes of device memory for the time-chunked form (NULL: one chunk always)
};
constexpr size_t kScanScratchBytes = (size_t)2 << 20;
cudaError_t launch_scan(const ScanArgs &a, cudaStream_t s);

struct DecodeArgs {
    void *kv, *meta;
    float *state;
    int B, H, D, S, dtype, gate_dtype;
    int64_t len;        // tokens in the cache the kernel should see
    int64_t page_cap;
    int n_sink, n_local;
    int32_t *status;
    float *absmax;      // [2][BH] largest |stored key| per head (NULL: not tracked); copy `epoch & 1` is current
    int32_t epoch;      // number of the decode step (1, 2, ...); 0 outside decode steps
    int32_t poll_limit; // polls after which a device-side wait gives up
};
// a.len is the length the scores are for.  do_update: first append the token (k_t, v_t, g_t) as
// position a.len - 1 (state, cache row, newest page's bounds).  next: the scoring ticket counters
// (head h at next[h * kCtrStride]), zero at launch.
// Histogram of the scores for the selection that follows (NULL members: none is kept): every page
// that competes for the budget adds one to its value bucket; the bucket map of a head goes to range.
struct ScoreHist {
    uint32_t *hist;     // [BH][kStepBins], all zero at launch
    float2 *range;      // [BH] (lo, scale)
    int32_t *ctr_other; // [BH][kStepCtrInts]: the one-launch step's counters of the next step, cleared here
};
cudaError_t launch_score(const DecodeArgs &a, const void *q, const void *k_t, const void *v_t, const void *g_t,
                         float *scores, int32_t *next, int do_update, const ScoreHist &sh, int sm_count, cudaStream_t s);
// attend_ctr: the ticket counters of the streaming kernels (cleared here, one head per CTA)
// Short contexts: the work of launch_score and launch_topk in one launch, one CTA per head (at most
// kSmallStepPages pages per head).
cudaError_t launch_score_select(const DecodeArgs &a, const void *q, const void *k_t, const void *v_t, const void *g_t,
                                float *scores, int do_update, int budget, int32_t *idx, int idx_stride,
                                int32_t *attend_ctr, int prefetch, int32_t *ctr_other, cudaStream_t s);
// prefetch: the flash-decode kernel runs next, start moving the first selected pages into L2
// sh: the histogram the scoring kernel filled (NULL members: none).  With it, and
// kTopkHistMinPages to kTopkFastPages pages, the list comes out in no particular order; otherwise ascending.
cudaError_t launch_topk(const DecodeArgs &a, const float *scores, int budget, int32_t *idx,
                        int idx_stride, int32_t *attend_ctr, int prefetch, const ScoreHist &sh, cudaStream_t s);
// does launch_topk take the histogram path for this many pages per head?
bool topk_uses_hist(int64_t pages);
// per-head counters of the flash-decode kernel, kCtrStride int32 apart from head to head; all
// zero at launch
struct AttendCounters {
    int32_t *next;    // next tile ticket that the counter hands out
    int32_t *nslot;   // partial records handed out to sweeping warps
    int32_t *done;    // tiles whose partial has been written (low 20 bits) | CTA arrivals (high bits)
};
cudaError_t launch_attend(const DecodeArgs &a, const void *q, const int32_t *idx, int n_idx,
                          int idx_stride, float scale, float *partial, const AttendCounters &ctr, void *o,
                          int sm_count, cudaStream_t s);
// The whole decode step in one launch (rq_step.cu): append, scoring, selection, flash-decode and
// combine, the heads split into `waves` groups so that the selection of one group runs behind the
// streams of the others.  step_plan says whether the shape qualifies and with how many waves
// (0: use the separate kernels); list receives every head's pages in no particular order, every
// entry tagged with the step's number.
struct StepBuffers {
    float *scores;      // [BH][page_cap]
    int2 *list;         // [BH][list_stride]
    int list_stride;
    float *partial;     // [BH][slots][D + 4]
    int slots;
    int32_t *ctr;       // [2][BH][kStepCtrInts]
    uint32_t *hist;     // [BH][kStepBins]
};
int step_plan(const DecodeArgs &a, int budget, int sm_count, int forced_waves, int *grid_out);
cudaError_t launch_step(const DecodeArgs &a, const void *q, const void *k_t, const void *v_t, const void *g_t, int budget,
                        float scale, const StepBuffers &b, void *o, int waves, int grid, cudaStream_t s);
cudaError_t launch_sort_list32(const int32_t *sel, int sel_stride, int K, int P, int BH, int32_t *out, int out_stride,
                               cudaStream_t s);
// sel (any order, K valid entries per head) -> out ascending, tail -1
cudaError_t launch_sort_list(const int2 *sel, int sel_stride, int K, int P, int BH, int32_t *out, int out_stride,
                             cudaStream_t s);

// ---- SnapKV-style cache reduction (rq_snapkv.cu) ----
struct SnapArgs {
    const void *kv;     // the source cache
    int64_t page_cap, len;
    int B, H, D, S, dtype;
    const void *qw;     // [B][W][H][D] queries of the observation window
    int W;
    float scale;
    float *imp;         // [BH][len] importance of every position
    float2 *stats;      // [BH][tiles][64] per-tile row statistics
    float2 *rowstat;    // [BH][64] final row statistics
    int32_t *status;    // the cache's device status word (a wait that runs out is reported there)
};
size_t snap_scratch_bytes(int BH, int64_t len);
void snap_carve(void *scratch, int BH, int64_t len, float **imp, float2 **stats, float2 **rowstat);
cudaError_t launch_snap_scores(const SnapArgs &a, cudaStream_t s);
cudaError_t launch_snap_select(const float *imp, int BH, int64_t len, int window, int keep, int32_t *idx, cudaStream_t s);
cudaError_t launch_snap_compact(const void *skv, int64_t s_page_cap, void *dkv, void *dmeta, int64_t d_page_cap, int S, int D,
                                int dtype, const int32_t *idx, int keep, float *absmax, int BH, cudaStream_t s);

// ---- MoBA-style block-sparse prefill attention (rq_moba.cu) ----
struct MobaArgs {
    const void *kv;     // the cache the prompt was prefilled into
    int64_t page_cap, len;
    int B, H, D, S, dtype;
    const void *q;      // [B][len][H][D] queries of all prompt positions
    int block, K;       // block size in positions; blocks per query (first and own block included)
    float scale;
    float *means;       // [BH][blocks][D] block representatives
    int32_t *sel;       // [BH][len][K] chosen blocks of every query, ascending, -1 beyond
    void *o;            // [B][len][H][D]
    int32_t *status;    // the cache's device status word
};
size_t moba_scratch_bytes(int BH, int64_t len, int D, int block, int K);
void moba_carve(void *scratch, int BH, int64_t len, int D, int block, float **means, int32_t **sel);
cudaError_t launch_moba(const MobaArgs &a, cudaStream_t s);

// Grid of a streaming kernel for a number of work units spread evenly over `heads` heads: at
// most what the device holds at once, at least two units per warp, and a whole number of CTAs per
// head if that keeps at least 85 % of the CTAs (heads served by more CTAs than others would
// finish early); a grid that is not a multiple of the heads makes the kernels spread warps, not
// CTAs, over the heads.
int stream_grid(int64_t units, int heads, int resident_ctas, int warps_per_cta, int max_ctas);
// flash-decode grid for a number of tiles and the CTAs the device holds at once
int attend_grid(int64_t tiles, int heads, int resident_ctas);
// partial records a head can need when it has this many tiles
int attend_slots_per_head(int64_t tiles_per_head);
// SMs of the current device
int sm_count();

}  // namespace rq
