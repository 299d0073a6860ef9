/* dd.h — C ABI of the sparse decode hot path (DualDecoder, arxiv 2607.26475), B200 / sm_100a.
 *
 * Per layer and request: score the KV pages from the speculated token's query against
 * static GPU-resident page landmarks, pick a per-KV-head top-k set, gather those pages
 * from pinned host memory into a layer-scoped ring slot on a side stream, and run GQA
 * decode attention over the gathered set only.
 *
 * Conventions
 *   - every function returns int: DD_OK (0) or a negative DD_ERR_* code; nothing throws,
 *     aborts or traps. dd_last_error_message() gives the text of the last failure.
 *   - "dev" pointers are CUDA device pointers of the context's device; "host" pointers are
 *     ordinary host memory; "pinned" pointers are page-locked host memory the device can
 *     read (cudaHostAlloc / cudaHostRegister; torch pin_memory). Pageable host memory is
 *     rejected with DD_ERR_NOT_PINNED before any kernel is launched.
 *   - the caller owns every tensor and both streams. The library owns the context, its
 *     events, its scratch memory, its index tables and (unless supplied) the ring.
 *   - all kernel entry points are asynchronous on the stream they are given (or on the
 *     context's streams for the pipelined calls); dd_create, dd_destroy, dd_sync and
 *     dd_device_error synchronise.
 *   - timelines, probes, counters and test hooks live in dd_bench.h; they are not part of the method.
 *   - the scratch memory of a context is shared by its calls: calls of the same kind must
 *     be stream-ordered with respect to each other (the pipelined path does this itself).
 *   - tensors are dense, row-major in the index order written; bf16 tensors 16-byte aligned,
 *     int32 and fp32 arrays 4-byte aligned.
 *   - geometry supported by the kernels: head_dim 128, page_tokens 16,
 *     n_q_tokens * (n_q_heads / n_kv_heads) <= 8. Anything else is DD_ERR_INVALID_ARG.
 *
 * Notation: B requests, L layers, Hq query heads, Hkv KV heads, G = Hq/Hkv, d = head_dim,
 * T = page_tokens, P = max_pages, k = k_pages, Tq = n_q_tokens (token 0 = current output
 * token, token 1 = speculated token), D = ring_depth.
 */
#ifndef DD_H_
#define DD_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DD_OK                 0
#define DD_ERR_INVALID_ARG   (-1)
#define DD_ERR_NOT_PINNED    (-2)
#define DD_ERR_CUDA          (-3)
#define DD_ERR_TIMEOUT       (-4)
#define DD_ERR_INDEX_RANGE   (-5)   /* a page index outside [0, n_pages) reached a kernel; it was clamped */
#define DD_ERR_STATE         (-6)   /* call out of order (not bound, not primed, wrong step/layer) */
#define DD_ERR_WAIT_EXPIRED  (-7)   /* a bounded device-side wait gave up; the kernel returned early */

#define DD_GATHER_LOADS  0          /* zero-copy: warps read the pinned pages with 16-byte loads */
#define DD_GATHER_BULK   1          /* bulk-copy engine: pinned page -> shared memory -> slot (cp.async.bulk) */
#define DD_GATHER_STAGED 2          /* the device's copy engine moves runs of adjacent selected pages (or aligned
                                       blocks) into a staging region, an assembly kernel places them in the slot;
                                       short runs are read by the zero-copy kernel at the same time */

#define DD_ATTN_AUTO    0           /* the faster one as measured: the split-KV kernel */
#define DD_ATTN_SPLIT   1           /* split-KV kernel: grid (split, KV head, request), cluster merge */
#define DD_ATTN_STREAM  2           /* streaming kernel: equal runs of pages per block, TMA-fed shared-memory ring */
#define DD_ATTN_TC      3           /* the streaming split on tcgen05: tiles of 8 pages, accumulators in tensor memory */

#define DD_SELECT_AUTO         0    /* fused cluster kernel when the request fits, else the two-kernel path */
#define DD_SELECT_TWO_KERNELS  1    /* scoring kernel + top-k kernel with logits in global scratch */

typedef struct dd_ctx dd_ctx;

typedef struct dd_config {
  int n_layers;              /* L */
  int batch;                 /* B */
  int n_q_heads;             /* Hq */
  int n_kv_heads;            /* Hkv */
  int head_dim;              /* d, must be 128 */
  int page_tokens;           /* T, must be 16 */
  int max_pages;             /* P: pages per request in the landmark and host-store layouts */
  int k_pages;               /* k: selected pages per KV head (budget / T) */
  int forced_recent_pages;   /* last pages of every request that are always selected; counted inside k */
  int n_q_tokens;            /* Tq: 1 or 2 */
  int ring_depth;            /* D >= 2 (2 = the two-buffer scheme) */
  int gather_mode;           /* DD_GATHER_LOADS, DD_GATHER_BULK or DD_GATHER_STAGED */
  int gather_ctas;           /* thread blocks the gather may occupy; 0 = library default */
  int select_mode;           /* DD_SELECT_AUTO or DD_SELECT_TWO_KERNELS */
  int attn_splits;           /* blocks per (request, KV head) in attention, <= 64 or a multiple of 8 up to 512; 0 = automatic */
  void* compute_stream;      /* cudaStream_t used by the pipelined calls for attention and selection */
  void* copy_stream;         /* cudaStream_t used by the pipelined calls for the gather */
  void* ring_mem;            /* optional caller-owned ring of dd_ring_bytes(); NULL = library allocates */
  size_t ring_bytes;         /* size of ring_mem when supplied */
  int landmark_chunk_tokens; /* tokens summarised by one landmark: 0 or 16 = one per page; 8, 4, 2, 1 = several per page */
  int miss_correction;       /* 1: dd_decode_layer_step repairs prediction misses before attention (needs urgent_stream) */
  void* urgent_stream;       /* cudaStream_t, ideally of higher priority than copy_stream; used for the missing pages */
  void* select_stream;       /* optional cudaStream_t: the pipelined calls run the next-step selection there, concurrently
                                with attention (the two are independent); NULL = on the compute stream */
  int stage_min_run_pages;   /* DD_GATHER_STAGED: runs of at least this many adjacent selected pages go through the
                                copy engine, shorter ones through the zero-copy kernel; 0 = library default (8) */
  int stage_block_pages;     /* DD_GATHER_STAGED: 0 = copy exactly the selected runs; 2, 4, 8, 16 or 32 = copy every
                                aligned block of that many pages that holds a selected page (over-fetch, no stragglers) */
  int attn_mode;             /* DD_ATTN_AUTO, DD_ATTN_SPLIT, DD_ATTN_STREAM or DD_ATTN_TC (attn_splits applies to the split kernel) */
} dd_config;

/* ---- context ------------------------------------------------------------------------------- */

/* Validates the configuration, allocates events, scratch, the index tables [2][L][B][Hkv][k]
 * and (if ring_mem is NULL) the ring of D slots on the current device. DD_GATHER_STAGED adds a staging region of
 * one slot's size (times stage_block_pages with over-fetch), page-locked copies of the index tables and descriptor
 * buffers, and one library-owned stream for the zero-copy part of a gather. */
int dd_create(const dd_config* cfg, dd_ctx** out);
/* Waits for the context's streams (bounded, 10 s) and frees what dd_create allocated. */
int dd_destroy(dd_ctx* ctx);
/* Bytes of one ring slot [B][Hkv][2][k*T][d] bf16, of the whole ring (D slots) and of the
 * library's scratch for this configuration. 0 for an invalid configuration. */
size_t dd_slot_bytes(const dd_config* cfg);
size_t dd_ring_bytes(const dd_config* cfg);
size_t dd_scratch_bytes(const dd_config* cfg);
const char* dd_strerror(int code);
const char* dd_last_error_message(dd_ctx* ctx);
/* Synchronises the context's streams (bounded by timeout_s), then reads and clears the device
 * error word. *code is DD_OK, DD_ERR_INDEX_RANGE or DD_ERR_WAIT_EXPIRED; *detail is the
 * offending value (first bad index, or the id of the wait that gave up). */
int dd_device_error(dd_ctx* ctx, double timeout_s, int* code, int* detail);
/* The same error word without any synchronisation, enqueue or clearing: a kernel that reports an error also
 * writes it to a page-locked mirror the host can read at any time, so this call is safe between launches of a
 * running pipeline. It shows the first error reported since the last dd_device_error (which clears both copies);
 * an error of a kernel that has not run yet is not visible yet. */
int dd_last_device_error(dd_ctx* ctx, int* code, int* detail);
/* Host wait on both context streams with a deadline: DD_ERR_TIMEOUT instead of hanging. */
int dd_sync(dd_ctx* ctx, double timeout_s);

/* ---- set-up step ---------------------------------------------------------------------------- */

/* Landmarks of one layer (Sec. 2.2: adjacent KV entries are segmented into chunks with
 * compressed landmarks; Sec. 4.1: built before decoding and fixed afterwards). Here a
 * landmark is the mean of the valid keys of a page: fp32 sum in token order, fp32 divide,
 * round-to-nearest-even to bf16; a page with no valid token gets zeros.
 *   kv_layer   pinned or dev, bf16 [B][Hkv][P][2][T][d] ([..][0] = K, [..][1] = V)
 *   ctx_len    dev int32 [B], tokens per request
 *   landmarks  dev bf16 [B][Hkv][P][d], written
 * With landmark_chunk_tokens = c < 16 a page has R = 16/c landmarks, one per c consecutive tokens, and the
 * tensor is [B][Hkv][P*R][d] with the chunks of a page adjacent. */
int dd_build_landmarks(dd_ctx* ctx, const void* kv_layer, const int* ctx_len, void* landmarks, void* stream);

/* ---- the three kernels of the path ----------------------------------------------------------- */

/* Retrieval index of one layer (Sec. 2.2, Sec. 4.1: the index is determined by the token's
 * query and the GPU-resident landmarks; Sec. 4.1 "Retrieval index prediction": the speculated
 * token's query predicts the next step's index).
 *   s[h,p]     = <q[b,q_token,h,:], landmarks[b,h/G,p,:]> / sqrt(d)     for p < n_pages[b]
 *   score[g,p] = max over the G heads of group g of softmax_p(s[h,:])[p]
 * The last forced_recent_pages valid pages are always selected; the remaining k - forced are
 * the highest scores among the others; equal scores go to the lower page.
 *   q           dev bf16 [B][Tq][Hq][d]
 *   q_token     which token's query scores (1 = speculated; 0 when Tq == 1)
 *   landmarks   dev bf16 [B][Hkv][P][d] of this layer
 *   n_pages     dev int32 [B], valid pages per request; k <= n_pages[b] <= P is required
 *               (a violating request gets indices clamped into range and DD_ERR_INDEX_RANGE
 *               in the device error word)
 *   out_idx     dev int32 [B][Hkv][k], ascending page numbers, written
 *   out_scores  dev fp32 [B][Hkv][P] or NULL; score[g,p] for p < n_pages[b], written */
int dd_select_topk(dd_ctx* ctx, const void* q, int q_token, const void* landmarks, const int* n_pages,
                   int* out_idx, float* out_scores, void* stream);

/* The same selection when pages carry several landmarks (landmark_chunk_tokens < 16; the paper leaves the
 * chunk size open, Sec. 2.2): the soft-max of a head runs over the chunks that hold at least one token, and a
 * page's score is the maximum over the group's heads and over the page's chunks. landmarks is
 * [B][Hkv][P*R][d]; ctx_len (dev int32 [B]) tells which chunks exist. With one landmark per page it equals
 * dd_select_topk. dd_select_topk itself fails with DD_ERR_INVALID_ARG on a context with several chunks per page. */
int dd_select_topk_chunked(dd_ctx* ctx, const void* q, int q_token, const void* landmarks, const int* n_pages,
                           const int* ctx_len, int* out_idx, float* out_scores, void* stream);

/* Gather of the selected pages into a ring slot in attention layout (Sec. 5.3: predicted KV
 * entries are prefetched from host memory; Sec. 5.4 "GPU-side sparse KV assembly": the GPU
 * places them at their final attention layout). A bit copy:
 *   slot[b][g][0|1][j*T + i][:] = host_kv_layer[b][g][idx[b][g][j]][0|1][i][:]
 *   host_kv_layer  pinned (or dev) bf16 [B][Hkv][P][2][T][d] of this layer
 *   idx            dev int32 [B][Hkv][k]
 *   n_pages        dev int32 [B] or NULL; when given, idx outside [0, n_pages[b]) is clamped
 *                  and reported (otherwise checked against P)
 *   slot           ring slot number, 0 <= slot < D
 * With DD_GATHER_STAGED (the copy-engine form of Sec. 5.4: selected KV blocks are moved into a GPU staging
 * region and a GPU kernel compacts and reorders them into the attention layout) the host needs the index set:
 * this stand-alone call copies idx to the host and waits for `stream` before it issues the copies; the
 * pipelined calls copy every selected set to page-locked host memory right after its selection, a whole step
 * before it is needed. Index checks then happen on the host, with the same clamping and error code. */
int dd_gather_kv_from_host(dd_ctx* ctx, const void* host_kv_layer, const int* idx, const int* n_pages,
                           int slot, void* stream);

/* GQA decode attention of every query token over the gathered set only (Sec. 4.2, Sec. 5.4:
 * the attention kernel observes the layer's complete sparse KV set; Sec. 5.2: the output token
 * and the speculated token are computed in one call). bf16 inputs, fp32 accumulation, bf16 out.
 *   z[j,i]  = <q[b,t,h,:], Kslot[b,h/G,j*T+i,:]> / sqrt(d), dropped when idx[b,h/G,j]*T + i >= ctx_len[b]
 *   out[b,t,h,:] = sum softmax(z) * Vslot
 *   q        dev bf16 [B][Tq][Hq][d]
 *   idx      dev int32 [B][Hkv][k] (the set the slot was gathered with; used for the mask only)
 *   ctx_len  dev int32 [B]
 *   out      dev bf16 [B][Tq][Hq][d], written
 *   out_lse  dev fp32 [B][Tq][Hq] or NULL; natural-log sum of exp(z), written */
int dd_sparse_decode_attn(dd_ctx* ctx, const void* q, int slot, const int* idx, const int* ctx_len,
                          void* out, float* out_lse, void* stream);

/* ---- the pipelined layer step ---------------------------------------------------------------- */

/* Binds the per-layer tables used by dd_prime / dd_decode_layer_step.
 *   landmarks_per_layer  host array of L dev pointers, each bf16 [B][Hkv][P][d]
 *   host_kv_per_layer    host array of L pinned (or dev) pointers, each bf16 [B][Hkv][P][2][T][d]
 *   n_pages, ctx_len     dev int32 [B]
 * The arrays of pointers are copied; the tensors are not. */
int dd_bind(dd_ctx* ctx, const void* const* landmarks_per_layer, const void* const* host_kv_per_layer,
            const int* n_pages, const int* ctx_len);

/* Priming selection for every layer — the stand-in for the pre-decoding step that yields the
 * first speculated token (Sec. 5.2 "First speculative token initialization") — followed by the
 * gathers of layers 0..min(D,L)-1 of step 0 on the copy stream.
 *   q_init  dev bf16 [L][B][Hq][d] */
int dd_prime(dd_ctx* ctx, const void* q_init);

/* One layer of one decode step, in (step, layer) order starting at (0, 0) (Sec. 5.3 "Layer-aware
 * KV transfer overlapping": the transfer for layer i+2 starts when the attention of layer i is
 * done; Sec. 5.4 "Two-layer ping-pong buffering": the compute stream waits for the slot's
 * transfer-complete event, the copy stream waits for the slot's buffer-released event):
 *   compute stream: wait ready[slot(layer)] -> attention(step, layer) over the set selected one
 *                   step earlier -> record released[slot] -> selection from q's speculated token
 *                   -> index set of (step+1, layer)
 *   copy stream:    wait released[slot] (and the selection it depends on) -> gather of layer
 *                   layer+D of this step, or of layer layer+D-L of the next step
 * With a select_stream the selection runs there, next to the attention; the compute stream waits for it at the
 * end of the call, so that work enqueued on the compute stream after this call may reuse q as before.
 *   q    dev bf16 [B][Tq][Hq][d]
 *   out  dev bf16 [B][Tq][Hq][d], written */
int dd_decode_layer_step(dd_ctx* ctx, int step, int layer, const void* q, void* out);

/* One whole decode step from host buffers: copies the step's queries of all layers from pinned host memory to
 * the device, runs dd_decode_layer_step for layer 0..L-1, and copies the outputs back, all on the compute stream
 * (the KV pages come from the bound host store as always). Asynchronous: out_host is complete once the compute
 * stream has drained (dd_sync, or an event the caller records on that stream after the call).
 *   q_host    pinned bf16 [L][B][Tq][Hq][d], read when the copy executes
 *   out_host  pinned bf16 [L][B][Tq][Hq][d], written
 * The device staging for q and out is part of the context's scratch. Steps follow the same order rule as
 * dd_decode_layer_step (all layers of `step`, starting at step 0 after dd_prime). */
int dd_decode_step_host(dd_ctx* ctx, int step, const void* q_host, void* out_host);

/* ---- dual-token causal tail (Sec. 5.2 "Dual-token decoding") ----------------------------------------- */

/* The same attention with the step's own new KV entries appended: the output token and the speculated token
 * of a request are concatenated along the sequence, and the output token must not see the speculated token.
 * Query token t sees every valid gathered token and the new entries j <= t (itself and the tokens before it).
 *   k_new, v_new  dev bf16 [B][Tq][Hkv][d]: keys and values of the step's tokens (token 0 = output token)
 * Everything else as in dd_sparse_decode_attn / dd_decode_layer_step. out_lse includes the new entries. */
int dd_sparse_decode_attn_causal(dd_ctx* ctx, const void* q, int slot, const int* idx, const int* ctx_len,
                                 const void* k_new, const void* v_new, void* out, float* out_lse, void* stream);
int dd_decode_layer_step_causal(dd_ctx* ctx, int step, int layer, const void* q, const void* k_new,
                                const void* v_new, void* out);

/* Device address of the predicted index set [B][Hkv][k] prefetched for (step parity, layer). No copy. */
int dd_get_indices(dd_ctx* ctx, int step_parity, int layer, const int** dev_idx);

/* ---- miss correction (Sec. 5.3 "Prioritized missing KV transfer") --------------------------------- */

/* With dd_config.miss_correction = 1, dd_decode_layer_step first selects the TRUE index of the layer from
 * the current token (token 0 of q), compares it with the predicted set that was prefetched into the slot,
 * fetches the missing pages (true minus predicted) on urgent_stream into the buffer positions of the pages
 * the true set does not contain, and runs attention over the repaired slot — i.e. over the true set, so the
 * prediction no longer influences the result (Sec. 4.2). The selection for the next step runs on the
 * compute stream while the urgent transfer is in flight. The two calls below are that repair in pieces.
 *
 * dd_diff_indices: pred_idx, true_idx dev int32 [B][Hkv][k], both ascending. Writes merged_idx
 * (dev int32 [B][Hkv][k]): position j keeps pred_idx[j] when that page is in the true set, else takes the
 * next missing page in ascending order; as a set, merged_idx equals true_idx. Also fills the context's fix
 * list of ring slot `slot` and adds to the miss statistics. Asynchronous on `stream`. */
int dd_diff_indices(dd_ctx* ctx, const int* pred_idx, const int* true_idx, int slot, int* merged_idx, void* stream);
/* dd_fetch_missing_from_host: copies the pages on the fix list of `slot` (written by the last
 * dd_diff_indices for that slot, which must precede this call in stream order) from host_kv_layer
 * (pinned or dev, bf16 [B][Hkv][P][2][T][d]) into their positions of the slot. Asynchronous on `stream`. */
int dd_fetch_missing_from_host(dd_ctx* ctx, const void* host_kv_layer, int slot, void* stream);
/* Device address of the repaired page list [B][Hkv][k] of ring slot `slot` (valid after a corrected layer step). */
int dd_get_merged_indices(dd_ctx* ctx, int slot, const int** dev_idx);

/* ---- attention without any allocation ----------------------------------------------------------- */

/* (The paper has no counterpart of this call; it exists for integration.)
 * The same attention as dd_sparse_decode_attn, for callers that cannot allocate device memory and
 * therefore cannot own a dd_ctx (dd_create allocates): code that runs inside another framework's
 * memory plan, a process whose GPU memory is already fully handed to an arena, or a serving loop in
 * which an allocation's implicit device synchronisation is not acceptable. The split-merge scratch
 * lives in a fixed array of dd_static_scratch_capacity() bytes (8 MiB) inside the library image;
 * every GPU that loads the library holds that array until the process exits.
 *   - Nothing is allocated or freed: no cudaMalloc/cudaFree, no allocating library routine.
 *   - The caller passes the gathered slot itself (dev bf16 [B][Hkv][2][k*T][d]) instead of a ring
 *     slot number, and every other tensor as in dd_sparse_decode_attn.
 *   - n_splits is explicit (1 <= n_splits <= min(k_pages, 64)). B * Hkv * n_splits * 4160 bytes (plus 4 bytes
 *     per (request, KV head)) must fit the array; larger requests fail with DD_ERR_INVALID_ARG and a
 *     message that states both sizes. n_splits = 1 needs almost nothing.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress, with that
 *     device current) and remembers it; make that first call before any stream capture begins.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the call
 *     clears the arrival counters it needs on `stream` before the kernel. Two calls that overlap on the
 *     GPU (different streams, no ordering between them) race on the array and give wrong results:
 *     order them.
 *   - Every tensor pointer is checked on the host before anything is enqueued (cudaPointerGetAttributes,
 *     which allocates nothing): host memory or another device's memory gives DD_ERR_INVALID_ARG.
 * Asynchronous on `stream`. Returns DD_OK or DD_ERR_INVALID_ARG / DD_ERR_CUDA; the message is
 * available from dd_last_error_message(NULL) on the calling thread. */
size_t dd_static_scratch_capacity(void);
int dd_sparse_decode_attn_static(int batch, int n_q_heads, int n_kv_heads, int head_dim, int page_tokens,
                                 int k_pages, int n_q_tokens, int n_splits, const void* q, const void* slot,
                                 const int* idx, const int* ctx_len, void* out, float* out_lse, void* stream);

#ifdef __cplusplus
}
#endif
#endif  /* DD_H_ */
