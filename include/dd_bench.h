/* dd_bench.h — instrumentation of the sparse decode library: timelines, load-only probes, counters and test
 * hooks used by the benchmark and the tests. None of these calls is a step of the method and none has a
 * counterpart in the paper; the method's boundary is dd.h. Same conventions as dd.h.
 */
#ifndef DD_BENCH_H_
#define DD_BENCH_H_

#include "dd.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Device address of ring slot `slot` (0 <= slot < D): lets a test read back what a gather wrote. */
int dd_slot_ptr(dd_ctx* ctx, int slot, void** dev_out);

/* ---- miss statistics --------------------------------------------------------------------------------- */

/* Synchronises, then reports how many pages were missing and how many were selected since the last reset. */
int dd_miss_stats(dd_ctx* ctx, unsigned long long* missing, unsigned long long* selected, int reset);

/* ---- timeline of the pipelined calls ------------------------------------------------------------------ */

/* dd_trace_begin arms a timeline of up to max_layer_steps calls of dd_decode_layer_step (it creates timing
 * events; no device memory). Every traced call records eight points, in microseconds since the first traced call:
 *   [0] the compute stream reaches the layer step (all earlier compute work done)
 *   [1] every transfer the layer needs is complete: attention starts ([1] - [0] = time the compute stream
 *       was stalled on the host link, plus the true-index selection and diff under miss correction)
 *   [2] attention done (buffer released)
 *   [3] end of the layer step on the compute stream (selection done or rejoined)
 *   [4] the gather this call enqueued (layer + ring depth) starts on the copy stream, its waits satisfied
 *   [5] that gather is complete
 *   [6] under miss correction: the fetch of this layer's missing pages starts on the urgent stream (the
 *       prefetch of the slot and the repair list are complete); -1 without miss correction
 *   [7] under miss correction: that fetch is complete; -1 without miss correction
 * dd_trace_end stops recording, synchronises and returns the number of traced calls; dd_trace_read copies
 * `count` rows of DD_TRACE_FIELDS floats starting at row `first` into host memory `out`. DD_ERR_STATE when no trace exists. */
#define DD_TRACE_FIELDS 8
int dd_trace_begin(dd_ctx* ctx, int max_layer_steps);
int dd_trace_end(dd_ctx* ctx, int* n_recorded);
int dd_trace_read(dd_ctx* ctx, int first, int count, float* out);

/* ---- measurement aids ------------------------------------------------------------------------------- */

/* Load-only twins of the two HBM-bound kernels: the same grid, the same walk over pages / landmark rows and the
 * same 16-byte fragment loads as dd_sparse_decode_attn (over ring slot `slot`) and as the fused selection
 * (over `landmarks`, dev bf16 [B][Hkv][P*R][d], with n_pages dev int32 [B]), but no arithmetic, no exchange and
 * no output. Their duration is what the memory system delivers for that launch shape and size; the benchmark
 * reports it next to the kernels' own times. dd_probe_select_loads needs the fused selection path
 * (DD_ERR_STATE otherwise). Asynchronous on `stream`. */
int dd_probe_attn_loads(dd_ctx* ctx, int slot, void* stream);
int dd_probe_select_loads(dd_ctx* ctx, const void* landmarks, const int* n_pages, void* stream);

/* ---- counters of the staged gather ---------------------------------------------------------------- */

/* Totals since the context was created (or since the last call with reset != 0) over all gathers issued in
 * DD_GATHER_STAGED mode; host-side counters, no synchronisation:
 *   out[0] gathers, out[1] copy-engine copies issued, out[2] bytes those copies moved over the host link,
 *   out[3] selected pages that went through the staging region, out[4] selected pages read by the zero-copy
 *   kernel, out[5] microseconds the host spent waiting for index sets, out[6] microseconds the host spent
 *   forming runs and issuing copies. */
#define DD_GATHER_STATS_FIELDS 7
int dd_gather_stats(dd_ctx* ctx, unsigned long long* out, int reset);

/* ---- test hooks ------------------------------------------------------------------------------------- */

/* The host's part of the staged gather without any CUDA call, so that it can be tested without a GPU. From the index
 * set idx (host int32 [B][Hkv][k]) it forms
 *   copies      [3 * n_copies] (source page = unit * P + page, first staging page, pages): runs of adjacent selected
 *               pages of at least min_run pages, or, with block_pages > 0, every aligned block of that many pages that
 *               holds a selected page (adjacent blocks merged into one copy)
 *   map         [n_staged] staged page -> slot item (unit * k + position), -1 for a page that was only fetched along
 *   stragglers  [n_stragglers] slot items left to the zero-copy kernel
 * n_pages (host int32 [B]) may be NULL; an index outside [0, min(n_pages[b], P)) is clamped as on the device and the
 * first one is reported in bad = {flag, value}. DD_ERR_INVALID_ARG when the plan does not fit staging_capacity pages or
 * max_copies copies. */
int dd_test_stage_plan(const int* idx, const int* n_pages, int batch, int n_kv_heads, int max_pages, int k_pages, int min_run,
                       int block_pages, long long staging_capacity, long long* copies, long long max_copies,
                       long long* n_copies, int* map, long long* n_staged, int* stragglers, long long* n_stragglers, int* bad);

/* Limit of the bounded device-side waits (the mbarrier waits of the bulk gather engine and of the streaming
 * attention kernel; default 2 s), and a way to make one run out without faulting anything: with
 * inflate_first_stage != 0 the first stage of block 0 of the bulk gather expects 16 bytes more than its copy
 * delivers, so its wait can never complete; the copy itself lands normally, the wait gives up after wait_seconds,
 * the block waits (bounded) for its other copies in flight and returns, and the device error word reports
 * DD_ERR_WAIT_EXPIRED. For tests of that error path only. */
int dd_set_bulk_wait(dd_ctx* ctx, double wait_seconds, int inflate_first_stage);

/* The cluster-size search of the fused selection kernel with the device queries replaced by a callback, so that
 * it can be tested without a GPU: returns the chosen blocks per (request, KV head), or 0 when no cluster size
 * fits (the two-kernel path is then used). fits(blocks, shared_bytes, user) returns how many clusters of that many
 * blocks with that much dynamic shared memory per block the device holds at once (0 = cannot run); a size whose
 * clusters are all resident (fits >= problems) is preferred. allow16 says whether 16-block
 * (non-portable) clusters may be tried. rows_per_page = landmarks per page, group = query heads per KV head;
 * ring_stages receives the depth of the scoring phase's shared-memory ring (tiles per warp), logits_global
 * whether the logits go to global scratch instead of shared memory. */
int dd_test_pick_cluster(int max_pages, int problems, int sm_count, int rows_per_page, int group, int allow16,
                         int (*fits)(int blocks, size_t shared_bytes, void* user), void* user, int* pages_per_block,
                         size_t* shared_bytes, int* ring_stages, int* logits_global);

/* Test hook, needs no GPU: the flat work split of the two TMA-fed attention kernels (kind 0: streaming kernel, two
 * blocks per SM; kind 1: tcgen05 kernel, one block per SM) for a launch of batch * n_kv_heads units of k_pages pages.
 * Block x owns the pages [x * pages_per_block, (x + 1) * pages_per_block) of the flat list; max_parts is the number of
 * partial results reserved per unit. Returns DD_OK or DD_ERR_INVALID_ARG. */
int dd_test_attn_split(int kind, int batch, int n_kv_heads, int k_pages, int sm_count, int* n_blocks, int* pages_per_block,
                       int* max_parts);

#ifdef __cplusplus
}
#endif
#endif  /* DD_BENCH_H_ */
