// Host side of the C ABI: context life cycle, argument checks, and the layer-scoped ring with its
// event protocol (transfer-complete / buffer-released) driving the pipelined layer step.
#include <stdarg.h>
#include <string.h>

#include <chrono>
#include <new>
#include <thread>
#include <vector>

#include "dd_common.cuh"

int dd_select_setup(dd_ctx* ctx);
int dd_gather_setup(dd_ctx* ctx);

static thread_local char g_errmsg[512] = "";

int dd_fail(dd_ctx* ctx, int code, const char* fmt, ...) {
  char* dst = ctx ? ctx->errmsg : g_errmsg;
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(dst, 512, fmt, ap);
  va_end(ap);
  if (ctx) memcpy(g_errmsg, ctx->errmsg, 512);
  return code;
}

extern "C" const char* dd_strerror(int code) {
  switch (code) {
    case DD_OK: return "ok";
    case DD_ERR_INVALID_ARG: return "invalid argument";
    case DD_ERR_NOT_PINNED: return "host memory is not page-locked";
    case DD_ERR_CUDA: return "CUDA error";
    case DD_ERR_TIMEOUT: return "timed out";
    case DD_ERR_INDEX_RANGE: return "page index out of range (clamped)";
    case DD_ERR_STATE: return "call out of order";
    case DD_ERR_WAIT_EXPIRED: return "a bounded device-side wait expired";
    default: return "unknown error";
  }
}

extern "C" const char* dd_last_error_message(dd_ctx* ctx) { return ctx ? ctx->errmsg : g_errmsg; }

// ---------------------------------------------------------------------------------------------
// configuration
// ---------------------------------------------------------------------------------------------
static const char* dd_check_config(const dd_config* c) {
  if (!c) return "config is NULL";
  if (c->head_dim != DD_D) return "head_dim must be 128";
  if (c->page_tokens != DD_T) return "page_tokens must be 16";
  if (c->n_layers < 1 || c->batch < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1) return "sizes must be positive";
  if (c->n_q_heads % c->n_kv_heads) return "n_q_heads must be a multiple of n_kv_heads";
  if (c->n_q_tokens < 1 || c->n_q_tokens > 2) return "n_q_tokens must be 1 or 2";
  if (c->n_q_tokens * (c->n_q_heads / c->n_kv_heads) > 8) return "n_q_tokens * group size must be <= 8";
  if (c->max_pages < 1) return "max_pages must be positive";
  if (c->k_pages < 1 || c->k_pages > c->max_pages) return "need 1 <= k_pages <= max_pages";
  if (c->forced_recent_pages < 0 || c->forced_recent_pages > c->k_pages) return "need 0 <= forced_recent_pages <= k_pages";
  if (c->ring_depth < 2 || c->ring_depth > DD_MAX_RING) return "ring_depth must be in [2, 8]";
  if (c->gather_mode != DD_GATHER_LOADS && c->gather_mode != DD_GATHER_BULK && c->gather_mode != DD_GATHER_STAGED)
    return "unknown gather_mode";
  if (c->stage_min_run_pages < 0) return "stage_min_run_pages must be >= 0";
  {
    const int bp = c->stage_block_pages;
    if (bp != 0 && bp != 2 && bp != 4 && bp != 8 && bp != 16 && bp != 32) return "stage_block_pages must be 0, 2, 4, 8, 16 or 32";
  }
  if (c->select_mode != DD_SELECT_AUTO && c->select_mode != DD_SELECT_TWO_KERNELS) return "unknown select_mode";
  if (c->gather_ctas < 0 || c->attn_splits < 0) return "gather_ctas and attn_splits must be >= 0";
  if (c->miss_correction != 0 && c->miss_correction != 1) return "miss_correction must be 0 or 1";
  {
    const int ct = c->landmark_chunk_tokens;
    if (ct != 0 && ct != 16 && ct != 8 && ct != 4 && ct != 2 && ct != 1) return "landmark_chunk_tokens must be 0, 16, 8, 4, 2 or 1";
  }
  if (c->attn_mode != DD_ATTN_AUTO && c->attn_mode != DD_ATTN_SPLIT && c->attn_mode != DD_ATTN_STREAM &&
      c->attn_mode != DD_ATTN_TC)
    return "unknown attn_mode";
  if (c->attn_splits > 512) return "attn_splits must be <= 512";
  if (c->attn_splits > 64 && c->attn_splits % 8) return "attn_splits above 64 must be a multiple of 8";
  if ((long long)c->batch * c->n_kv_heads * c->k_pages > 0x7fffffffLL) return "too many selected pages";
  if ((long long)c->batch * c->n_kv_heads * c->max_pages > 0x7fffffffLL) return "too many pages";
  return nullptr;
}

// Blocks per (request, KV head) and how many of them form a thread-block cluster. Automatic choice: one
// wave of blocks (the attention kernel keeps four per SM resident), at least four pages (one per warp) in a
// split, clusters of up to eight blocks so that up to eight splits merge without touching global memory.
static int dd_resolve_splits(const dd_config* c, int sm_count, int* cluster_out) {
  int S = c->attn_splits, C = 1;
  if (S <= 0) {
    const int problems = c->batch * c->n_kv_heads;
    int target = (4 * sm_count) / problems;
    const int t_max = c->k_pages / 4 > 0 ? c->k_pages / 4 : 1;
    if (target > t_max) target = t_max;
    if (target < 1) target = 1;
    if (target >= 8) {
      int groups = target / 8;
      if (groups > 64) groups = 64;
      C = 8;
      S = 8 * groups;
    } else {
      C = target >= 4 ? 4 : (target >= 2 ? 2 : 1);
      S = C;
    }
  } else {
    if (S > c->k_pages) S = c->k_pages;
    C = (S % 8 == 0) ? 8 : (S % 4 == 0) ? 4 : (S % 2 == 0) ? 2 : 1;
  }
  if (cluster_out) *cluster_out = C;
  return S;
}

struct dd_sizes {
  size_t score_s, score_part, topk_keys, part_o, part_ml, ticket, idx_tab, err, idx_true, idx_merged, fix_stage, fix_list,
      fix_count, stats, stage;
  size_t total() const {
    return score_s + score_part + topk_keys + part_o + part_ml + ticket + idx_tab + err + idx_true + idx_merged +
           fix_stage + fix_list + fix_count + stats + 2 * stage;
  }
};

static size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

static dd_sizes dd_compute_sizes(const dd_config* c, int S, int sm_count) {
  dd_sizes z;
  const size_t B = c->batch, Hkv = c->n_kv_heads, Hq = c->n_q_heads, P = c->max_pages;
  const size_t G = Hq / Hkv, tiles = (P + DD_SCORE_TILE - 1) / DD_SCORE_TILE;
  const size_t Rr = c->landmark_chunk_tokens ? DD_T / c->landmark_chunk_tokens : 1;
  z.score_s = up256(2 * B * Hkv * P * Rr * G * 4);
  z.score_part = up256(B * Hq * tiles * 8);
  z.topk_keys = up256(B * Hkv * P * 4);
  {
    // partials of the split-KV kernel (S per unit) or of the streaming kernel (max_parts per unit), whichever is larger
    int nb = 0, ppb = 0, parts = 0, parts_tc = 0;
    dd_attn_stream_geometry(c, sm_count, &nb, &ppb, &parts);
    dd_attn_tc_geometry(c, sm_count, &nb, &ppb, &parts_tc);
    if (parts_tc > parts) parts = parts_tc;
    const size_t n_part = (size_t)(S > parts ? S : parts);
    z.part_o = up256(B * Hkv * n_part * 8 * DD_D * 4);
    z.part_ml = up256(B * Hkv * n_part * 8 * 8);
  }
  z.ticket = up256(B * Hkv * 4 + 4);               // arrival counters + one word the load-only probes may write
  z.idx_tab = up256((size_t)2 * c->n_layers * B * Hkv * c->k_pages * 4);
  z.err = 256;
  const size_t sel = B * Hkv * (size_t)c->k_pages, D = c->ring_depth;
  z.idx_true = up256(sel * 4);
  z.idx_merged = up256(D * sel * 4);
  z.fix_stage = up256(D * sel * 8);
  z.fix_list = up256(D * sel * 16);
  z.fix_count = 256;
  z.stats = 256;
  z.stage = up256((size_t)c->n_layers * B * c->n_q_tokens * Hq * DD_D * 2);
  return z;
}

static int dd_sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 148;
  return sms;
}

extern "C" size_t dd_slot_bytes(const dd_config* c) {
  if (dd_check_config(c)) return 0;
  return (size_t)c->batch * c->n_kv_heads * c->k_pages * DD_PAGE_BYTES;
}
extern "C" size_t dd_ring_bytes(const dd_config* c) { return dd_slot_bytes(c) * (c ? (size_t)c->ring_depth : 0); }
extern "C" size_t dd_scratch_bytes(const dd_config* c) {
  if (dd_check_config(c)) return 0;
  return dd_compute_sizes(c, dd_resolve_splits(c, dd_sm_count(), nullptr), dd_sm_count()).total();
}

// ---------------------------------------------------------------------------------------------
// life cycle
// ---------------------------------------------------------------------------------------------
static void dd_free_all(dd_ctx* ctx) {
  if (ctx->score_s) cudaFree(ctx->score_s);      // one allocation holds all the scratch
  if (ctx->own_ring && ctx->ring) cudaFree(ctx->ring);
  for (int i = 0; i < DD_MAX_RING; ++i) {
    if (ctx->ready[i]) cudaEventDestroy(ctx->ready[i]);
    if (ctx->released[i]) cudaEventDestroy(ctx->released[i]);
    if (ctx->fix_ready[i]) cudaEventDestroy(ctx->fix_ready[i]);
    if (ctx->urgent_done[i]) cudaEventDestroy(ctx->urgent_done[i]);
  }
  if (ctx->q_ready) cudaEventDestroy(ctx->q_ready);
  if (ctx->err_host) cudaFreeHost(ctx->err_host);
  if (ctx->idx_host) cudaFreeHost(ctx->idx_host);
  if (ctx->staging) cudaFree(ctx->staging);
  for (int i = 0; i < DD_STAGE_LISTS; ++i) {
    if (ctx->list_host[i]) cudaFreeHost(ctx->list_host[i]);
    if (ctx->list_free[i]) cudaEventDestroy(ctx->list_free[i]);
  }
  if (ctx->as_fence) cudaEventDestroy(ctx->as_fence);
  if (ctx->aux_fork) cudaEventDestroy(ctx->aux_fork);
  if (ctx->aux_join) cudaEventDestroy(ctx->aux_join);
  if (ctx->aux_stream) cudaStreamDestroy(ctx->aux_stream);
  if (ctx->idx_copied) {
    for (int l = 0; l < ctx->cfg.n_layers; ++l)
      if (ctx->idx_copied[l]) cudaEventDestroy(ctx->idx_copied[l]);
    delete[] ctx->idx_copied;
  }
  delete[] ctx->n_pages_host;
  delete[] ctx->copy_plan;
  delete[] ctx->host_kv_orig;
  if (ctx->sel_done) {
    for (int l = 0; l < ctx->cfg.n_layers; ++l)
      if (ctx->sel_done[l]) cudaEventDestroy(ctx->sel_done[l]);
    delete[] ctx->sel_done;
  }
  if (ctx->trace_ev) {
    for (int i = 0; i < ctx->trace_cap * DD_TRACE_FIELDS; ++i)
      if (ctx->trace_ev[i]) cudaEventDestroy(ctx->trace_ev[i]);
    delete[] ctx->trace_ev;
  }
  if (ctx->trace_origin) cudaEventDestroy(ctx->trace_origin);
  delete[] ctx->landmarks;
  delete[] ctx->host_kv;
  delete ctx;
}

extern "C" int dd_create(const dd_config* cfg, dd_ctx** out) {
  if (!out) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_create: out is NULL");
  *out = nullptr;
  if (const char* why = dd_check_config(cfg)) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_create: %s", why);
  if (cfg->miss_correction && !cfg->urgent_stream)
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_create: miss_correction needs an urgent_stream of its own");
  dd_ctx* ctx = new (std::nothrow) dd_ctx();
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_create: out of host memory");
  memset(ctx, 0, sizeof(*ctx));
  ctx->cfg = *cfg;
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e != cudaSuccess) {
    int rc = dd_fail(nullptr, DD_ERR_CUDA, "dd_create: no CUDA device: %s", cudaGetErrorString(e));
    delete ctx;
    return rc;
  }
  ctx->sm_count = dd_sm_count();
  ctx->G = cfg->n_q_heads / cfg->n_kv_heads;
  ctx->R = cfg->landmark_chunk_tokens ? DD_T / cfg->landmark_chunk_tokens : 1;
  ctx->n_rows = cfg->n_q_tokens * ctx->G;
  ctx->score_tiles = (cfg->max_pages + DD_SCORE_TILE - 1) / DD_SCORE_TILE;
  ctx->attn_splits = dd_resolve_splits(cfg, ctx->sm_count, &ctx->attn_cluster);
  ctx->slot_bytes = dd_slot_bytes(cfg);
  const dd_sizes z = dd_compute_sizes(cfg, ctx->attn_splits, ctx->sm_count);

#define DD_CREATE_TRY(expr)                                                                        \
  do {                                                                                             \
    cudaError_t e__ = (expr);                                                                      \
    if (e__ != cudaSuccess) {                                                                      \
      int rc__ = dd_fail(nullptr, DD_ERR_CUDA, "dd_create: %s: %s", #expr, cudaGetErrorString(e__)); \
      dd_free_all(ctx);                                                                            \
      return rc__;                                                                                 \
    }                                                                                              \
  } while (0)

  char* base = nullptr;
  DD_CREATE_TRY(cudaMalloc(&base, z.total()));
  ctx->score_s = (float*)base;                       base += z.score_s;
  ctx->score_part = (float2*)base;                   base += z.score_part;
  ctx->topk_keys = (uint32_t*)base;                  base += z.topk_keys;
  ctx->attn_part_o = (float*)base;                   base += z.part_o;
  ctx->attn_part_ml = (float2*)base;                 base += z.part_ml;
  ctx->attn_ticket = (unsigned int*)base;            base += z.ticket;
  ctx->idx_tab = (int*)base;                         base += z.idx_tab;
  ctx->err_word = (int*)base;                        base += z.err;
  ctx->idx_true = (int*)base;                        base += z.idx_true;
  ctx->idx_merged = (int*)base;                      base += z.idx_merged;
  ctx->fix_stage = (int2*)base;                      base += z.fix_stage;
  ctx->fix_list = (int4*)base;                       base += z.fix_list;
  ctx->fix_count = (unsigned int*)base;              base += z.fix_count;
  ctx->miss_stats = (unsigned long long*)base;       base += z.stats;
  ctx->stage_q = (__nv_bfloat16*)base;               base += z.stage;
  ctx->stage_out = (__nv_bfloat16*)base;
  DD_CREATE_TRY(cudaMemset(ctx->attn_ticket, 0, z.ticket));
  DD_CREATE_TRY(cudaMemset(ctx->idx_tab, 0, z.idx_tab));
  DD_CREATE_TRY(cudaMemset(ctx->err_word, 0, z.err));
  {
    // page-locked mirror of the error word; its device-visible address sits behind the two words
    DD_CREATE_TRY(cudaHostAlloc((void**)&ctx->err_host, 2 * sizeof(int), cudaHostAllocMapped));
    ctx->err_host[0] = ctx->err_host[1] = 0;
    void* mirror_dev = nullptr;
    DD_CREATE_TRY(cudaHostGetDevicePointer(&mirror_dev, ctx->err_host, 0));
    DD_CREATE_TRY(cudaMemcpy(ctx->err_word + 2, &mirror_dev, sizeof(void*), cudaMemcpyHostToDevice));
  }
  ctx->bulk_wait_ns = 2000000000ull;
  DD_CREATE_TRY(cudaMemset(ctx->fix_count, 0, z.fix_count));
  DD_CREATE_TRY(cudaMemset(ctx->miss_stats, 0, z.stats));
  if (cfg->ring_mem) {
    if (cfg->ring_bytes < dd_ring_bytes(cfg)) {
      int rc = dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_create: ring_mem holds %zu bytes, %zu needed", cfg->ring_bytes,
                       dd_ring_bytes(cfg));
      dd_free_all(ctx);
      return rc;
    }
    if (((uintptr_t)cfg->ring_mem) & 15) {
      int rc = dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_create: ring_mem must be 16-byte aligned");
      dd_free_all(ctx);
      return rc;
    }
    ctx->ring = (char*)cfg->ring_mem;
  } else {
    DD_CREATE_TRY(cudaMalloc(&ctx->ring, dd_ring_bytes(cfg)));
    ctx->own_ring = true;
  }
  for (int i = 0; i < cfg->ring_depth; ++i) {
    DD_CREATE_TRY(cudaEventCreateWithFlags(&ctx->ready[i], cudaEventDisableTiming));
    DD_CREATE_TRY(cudaEventCreateWithFlags(&ctx->released[i], cudaEventDisableTiming));
    DD_CREATE_TRY(cudaEventCreateWithFlags(&ctx->fix_ready[i], cudaEventDisableTiming));
    DD_CREATE_TRY(cudaEventCreateWithFlags(&ctx->urgent_done[i], cudaEventDisableTiming));
  }
  DD_CREATE_TRY(cudaEventCreateWithFlags(&ctx->q_ready, cudaEventDisableTiming));
  ctx->sel_done = new cudaEvent_t[cfg->n_layers]();
  for (int l = 0; l < cfg->n_layers; ++l)
    DD_CREATE_TRY(cudaEventCreateWithFlags(&ctx->sel_done[l], cudaEventDisableTiming));
  ctx->landmarks = new const void*[cfg->n_layers]();
  ctx->host_kv = new const void*[cfg->n_layers]();
  ctx->host_kv_orig = new const void*[cfg->n_layers]();
  if (cfg->gather_mode == DD_GATHER_STAGED) {
    const size_t total = (size_t)cfg->batch * cfg->n_kv_heads * cfg->k_pages;
    ctx->stage_min_run = cfg->stage_min_run_pages > 0 ? cfg->stage_min_run_pages : 8;
    ctx->stage_block = cfg->stage_block_pages;
    ctx->staging_pages = total * (size_t)(ctx->stage_block > 0 ? ctx->stage_block : 1);
    DD_CREATE_TRY(cudaMalloc(&ctx->staging, ctx->staging_pages * DD_PAGE_BYTES));
    DD_CREATE_TRY(cudaHostAlloc((void**)&ctx->idx_host, (size_t)2 * cfg->n_layers * total * sizeof(int), cudaHostAllocDefault));
    ctx->n_pages_host = new int[cfg->batch]();
    ctx->copy_plan = new long long[3 * total]();
    ctx->idx_copied = new cudaEvent_t[cfg->n_layers]();
    for (int l = 0; l < cfg->n_layers; ++l)
      DD_CREATE_TRY(cudaEventCreateWithFlags(&ctx->idx_copied[l], cudaEventDisableTiming));
    for (int i = 0; i < DD_STAGE_LISTS; ++i) {
      DD_CREATE_TRY(cudaHostAlloc((void**)&ctx->list_host[i], (ctx->staging_pages + total) * sizeof(int), cudaHostAllocMapped));
      void* dv = nullptr;
      DD_CREATE_TRY(cudaHostGetDevicePointer(&dv, ctx->list_host[i], 0));
      ctx->list_dev[i] = (const int*)dv;
      DD_CREATE_TRY(cudaEventCreateWithFlags(&ctx->list_free[i], cudaEventDisableTiming));
    }
    DD_CREATE_TRY(cudaStreamCreateWithFlags(&ctx->aux_stream, cudaStreamNonBlocking));
    DD_CREATE_TRY(cudaEventCreateWithFlags(&ctx->aux_fork, cudaEventDisableTiming));
    DD_CREATE_TRY(cudaEventCreateWithFlags(&ctx->aux_join, cudaEventDisableTiming));
  }
  int rc = dd_select_setup(ctx);
  if (rc == DD_OK) rc = dd_gather_setup(ctx);
  ctx->attn_stream = cfg->attn_mode == DD_ATTN_STREAM ? 1 : (cfg->attn_mode == DD_ATTN_TC ? 2 : 0);   // both opt-in
  if (rc == DD_OK && ctx->attn_stream == 1) rc = dd_attn_stream_setup(ctx);
  if (rc == DD_OK && ctx->attn_stream == 2) rc = dd_attn_tc_setup(ctx);
  if (rc == DD_OK && ctx->attn_stream && cudaEventCreate(&ctx->as_fence) != cudaSuccess) {
    snprintf(ctx->errmsg, sizeof(ctx->errmsg), "dd_create: cannot create the streaming kernel's fence event");
    rc = DD_ERR_CUDA;
  }
  if (rc != DD_OK) {
    memcpy(g_errmsg, ctx->errmsg, 512);
    dd_free_all(ctx);
    return rc;
  }
  DD_CREATE_TRY(cudaDeviceSynchronize());
#undef DD_CREATE_TRY
  *out = ctx;
  return DD_OK;
}

extern "C" int dd_sync(dd_ctx* ctx, double timeout_s) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sync: ctx is NULL");
  const auto deadline = std::chrono::steady_clock::now() + std::chrono::duration<double>(timeout_s);
  cudaStream_t streams[5] = {(cudaStream_t)ctx->cfg.compute_stream, (cudaStream_t)ctx->cfg.copy_stream, nullptr, nullptr,
                             nullptr};
  int n_streams = 2;
  if (ctx->aux_stream) streams[n_streams++] = ctx->aux_stream;
  if (ctx->cfg.miss_correction) streams[n_streams++] = (cudaStream_t)ctx->cfg.urgent_stream;
  if (ctx->cfg.select_stream) streams[n_streams++] = (cudaStream_t)ctx->cfg.select_stream;
  for (int i = 0; i < n_streams; ++i) {
    for (;;) {
      cudaError_t e = cudaStreamQuery(streams[i]);
      if (e == cudaSuccess) break;
      if (e != cudaErrorNotReady) return dd_fail(ctx, DD_ERR_CUDA, "dd_sync: %s", cudaGetErrorString(e));
      if (std::chrono::steady_clock::now() > deadline)
        return dd_fail(ctx, DD_ERR_TIMEOUT, "dd_sync: streams still busy after %.3f s", timeout_s);
      std::this_thread::sleep_for(std::chrono::microseconds(50));
    }
  }
  return DD_OK;
}

extern "C" int dd_destroy(dd_ctx* ctx) {
  if (!ctx) return DD_OK;
  int rc = dd_sync(ctx, 10.0);
  if (rc == DD_ERR_TIMEOUT) return rc;             // memory still in use by the device: leak rather than free
  dd_free_all(ctx);
  return DD_OK;
}

extern "C" int dd_device_error(dd_ctx* ctx, double timeout_s, int* code, int* detail) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_device_error: ctx is NULL");
  int rc = dd_sync(ctx, timeout_s);
  if (rc != DD_OK) return rc;
  int w[2] = {0, 0};
  DD_CUDA_TRY(ctx, cudaDeviceSynchronize());       // standalone calls may have used other streams
  DD_CUDA_TRY(ctx, cudaMemcpy(w, ctx->err_word, sizeof(w), cudaMemcpyDeviceToHost));
  DD_CUDA_TRY(ctx, cudaMemset(ctx->err_word, 0, sizeof(w)));
  if (w[0] == 0 && ctx->host_err[0] != 0) { w[0] = ctx->host_err[0]; w[1] = ctx->host_err[1]; }   // host-side index checks
  ctx->host_err[0] = ctx->host_err[1] = 0;
  ctx->err_host[0] = ctx->err_host[1] = 0;
  if (code) *code = w[0];
  if (detail) *detail = w[1];
  return DD_OK;
}

extern "C" int dd_last_device_error(dd_ctx* ctx, int* code, int* detail) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_last_device_error: ctx is NULL");
  const volatile int* m = ctx->err_host;
  int c = m[0], d = m[1];
  if (c == 0 && ctx->host_err[0] != 0) { c = ctx->host_err[0]; d = ctx->host_err[1]; }
  if (code) *code = c;
  if (detail) *detail = d;
  return DD_OK;
}

extern "C" int dd_slot_ptr(dd_ctx* ctx, int slot, void** dev_out) {
  if (!ctx || !dev_out) return dd_fail(ctx, DD_ERR_INVALID_ARG, "dd_slot_ptr: NULL argument");
  if (slot < 0 || slot >= ctx->cfg.ring_depth) return dd_fail(ctx, DD_ERR_INVALID_ARG, "dd_slot_ptr: slot %d of %d", slot, ctx->cfg.ring_depth);
  *dev_out = ctx->ring + (size_t)slot * ctx->slot_bytes;
  return DD_OK;
}

// ---------------------------------------------------------------------------------------------
// pointer checks
// ---------------------------------------------------------------------------------------------
// Device pointer of the context's device, aligned for its element type (16 bytes for bf16 tensors, which
// are read with 16-byte loads; 4 bytes for int32 / fp32 arrays), or failure.
static int dd_check_dev(dd_ctx* ctx, const void* p, const char* what, int align = 16) {
  if (!p) return dd_fail(ctx, DD_ERR_INVALID_ARG, "%s is NULL", what);
  if (((uintptr_t)p) & (uintptr_t)(align - 1)) return dd_fail(ctx, DD_ERR_INVALID_ARG, "%s is not %d-byte aligned", what, align);
  cudaPointerAttributes a;
  cudaError_t e = cudaPointerGetAttributes(&a, p);
  if (e != cudaSuccess) { cudaGetLastError(); return dd_fail(ctx, DD_ERR_INVALID_ARG, "%s: %s", what, cudaGetErrorString(e)); }
  if (a.type != cudaMemoryTypeDevice && a.type != cudaMemoryTypeManaged)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "%s is not device memory", what);
  if (a.type == cudaMemoryTypeDevice && a.device != ctx->device)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "%s lives on device %d, the context on %d", what, a.device, ctx->device);
  return DD_OK;
}

// Page-locked host memory (or device memory): returns the address the device uses.
static int dd_check_store(dd_ctx* ctx, const void* p, const char* what, const void** dev_visible) {
  if (!p) return dd_fail(ctx, DD_ERR_INVALID_ARG, "%s is NULL", what);
  if (((uintptr_t)p) & 15) return dd_fail(ctx, DD_ERR_INVALID_ARG, "%s is not 16-byte aligned", what);
  cudaPointerAttributes a;
  cudaError_t e = cudaPointerGetAttributes(&a, p);
  if (e != cudaSuccess) { cudaGetLastError(); return dd_fail(ctx, DD_ERR_INVALID_ARG, "%s: %s", what, cudaGetErrorString(e)); }
  if (a.type == cudaMemoryTypeUnregistered)
    return dd_fail(ctx, DD_ERR_NOT_PINNED, "%s is pageable host memory; page-lock it (cudaHostAlloc / cudaHostRegister)", what);
  if (a.type == cudaMemoryTypeHost) {
    if (!a.devicePointer) return dd_fail(ctx, DD_ERR_NOT_PINNED, "%s is page-locked but not mapped into the device", what);
    *dev_visible = a.devicePointer;
    return DD_OK;
  }
  if (a.type == cudaMemoryTypeDevice && a.device != ctx->device)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "%s lives on device %d, the context on %d", what, a.device, ctx->device);
  *dev_visible = p;
  return DD_OK;
}

#define DD_TRY(expr)             \
  do {                           \
    int rc__ = (expr);           \
    if (rc__ != DD_OK) return rc__; \
  } while (0)

// ---------------------------------------------------------------------------------------------
// stand-alone entry points
// ---------------------------------------------------------------------------------------------
extern "C" int dd_build_landmarks(dd_ctx* ctx, const void* kv_layer, const int* ctx_len, void* landmarks, void* stream) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_build_landmarks: ctx is NULL");
  const void* kv_dev = nullptr;
  DD_TRY(dd_check_store(ctx, kv_layer, "kv_layer", &kv_dev));
  DD_TRY(dd_check_dev(ctx, ctx_len, "ctx_len", 4));
  DD_TRY(dd_check_dev(ctx, landmarks, "landmarks"));
  return dd_launch_build_landmarks(ctx, kv_dev, ctx_len, landmarks, (cudaStream_t)stream);
}

extern "C" int dd_select_topk(dd_ctx* ctx, const void* q, int q_token, const void* landmarks, const int* n_pages,
                              int* out_idx, float* out_scores, void* stream) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_select_topk: ctx is NULL");
  if (q_token < 0 || q_token >= ctx->cfg.n_q_tokens)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "q_token %d outside [0, %d)", q_token, ctx->cfg.n_q_tokens);
  DD_TRY(dd_check_dev(ctx, q, "q"));
  DD_TRY(dd_check_dev(ctx, landmarks, "landmarks"));
  DD_TRY(dd_check_dev(ctx, n_pages, "n_pages", 4));
  DD_TRY(dd_check_dev(ctx, out_idx, "out_idx", 4));
  if (out_scores) DD_TRY(dd_check_dev(ctx, out_scores, "out_scores", 4));
  return dd_launch_select(ctx, q, q_token, ctx->cfg.n_q_tokens, landmarks, n_pages, out_idx, out_scores,
                          (cudaStream_t)stream);
}

extern "C" int dd_select_topk_chunked(dd_ctx* ctx, const void* q, int q_token, const void* landmarks, const int* n_pages,
                                      const int* ctx_len, int* out_idx, float* out_scores, void* stream) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_select_topk_chunked: ctx is NULL");
  if (q_token < 0 || q_token >= ctx->cfg.n_q_tokens)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "q_token %d outside [0, %d)", q_token, ctx->cfg.n_q_tokens);
  DD_TRY(dd_check_dev(ctx, q, "q"));
  DD_TRY(dd_check_dev(ctx, landmarks, "landmarks"));
  DD_TRY(dd_check_dev(ctx, n_pages, "n_pages", 4));
  DD_TRY(dd_check_dev(ctx, ctx_len, "ctx_len", 4));
  DD_TRY(dd_check_dev(ctx, out_idx, "out_idx", 4));
  if (out_scores) DD_TRY(dd_check_dev(ctx, out_scores, "out_scores", 4));
  return dd_launch_select(ctx, q, q_token, ctx->cfg.n_q_tokens, landmarks, n_pages, out_idx, out_scores,
                          (cudaStream_t)stream, ctx_len);
}

extern "C" int dd_gather_kv_from_host(dd_ctx* ctx, const void* host_kv_layer, const int* idx, const int* n_pages,
                                      int slot, void* stream) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_gather_kv_from_host: ctx is NULL");
  if (slot < 0 || slot >= ctx->cfg.ring_depth)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "slot %d outside [0, %d)", slot, ctx->cfg.ring_depth);
  const void* kv_dev = nullptr;
  DD_TRY(dd_check_store(ctx, host_kv_layer, "host_kv_layer", &kv_dev));
  DD_TRY(dd_check_dev(ctx, idx, "idx", 4));
  if (n_pages) DD_TRY(dd_check_dev(ctx, n_pages, "n_pages", 4));
  if (ctx->cfg.gather_mode == DD_GATHER_STAGED) {
    // the host forms the runs: bring the index set over and wait for it
    const size_t total = (size_t)ctx->cfg.batch * ctx->cfg.n_kv_heads * ctx->cfg.k_pages;
    std::vector<int> idx_h(total), np_h(n_pages ? ctx->cfg.batch : 0);
    DD_CUDA_TRY(ctx, cudaMemcpyAsync(idx_h.data(), idx, total * sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    if (n_pages)
      DD_CUDA_TRY(ctx, cudaMemcpyAsync(np_h.data(), n_pages, np_h.size() * sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    DD_CUDA_TRY(ctx, cudaStreamSynchronize((cudaStream_t)stream));
    return dd_launch_gather_staged(ctx, host_kv_layer, kv_dev, idx_h.data(), idx, n_pages ? np_h.data() : nullptr, n_pages,
                                   ctx->ring + (size_t)slot * ctx->slot_bytes, (cudaStream_t)stream);
  }
  return dd_launch_gather(ctx, kv_dev, idx, n_pages, ctx->ring + (size_t)slot * ctx->slot_bytes, (cudaStream_t)stream);
}

extern "C" int dd_sparse_decode_attn(dd_ctx* ctx, const void* q, int slot, const int* idx, const int* ctx_len,
                                     void* out, float* out_lse, void* stream) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn: ctx is NULL");
  if (slot < 0 || slot >= ctx->cfg.ring_depth)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "slot %d outside [0, %d)", slot, ctx->cfg.ring_depth);
  DD_TRY(dd_check_dev(ctx, q, "q"));
  DD_TRY(dd_check_dev(ctx, idx, "idx", 4));
  DD_TRY(dd_check_dev(ctx, ctx_len, "ctx_len", 4));
  DD_TRY(dd_check_dev(ctx, out, "out"));
  if (out_lse) DD_TRY(dd_check_dev(ctx, out_lse, "out_lse", 4));
  return dd_launch_attn(ctx, q, ctx->ring + (size_t)slot * ctx->slot_bytes, idx, ctx_len, out, out_lse,
                        (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------
// pipelined path
// ---------------------------------------------------------------------------------------------
extern "C" int dd_bind(dd_ctx* ctx, const void* const* landmarks_per_layer, const void* const* host_kv_per_layer,
                       const int* n_pages, const int* ctx_len) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_bind: ctx is NULL");
  if (!landmarks_per_layer || !host_kv_per_layer) return dd_fail(ctx, DD_ERR_INVALID_ARG, "dd_bind: table is NULL");
  ctx->bound = false;
  ctx->primed = false;
  for (int l = 0; l < ctx->cfg.n_layers; ++l) {
    DD_TRY(dd_check_dev(ctx, landmarks_per_layer[l], "landmarks_per_layer[l]"));
    const void* dv = nullptr;
    DD_TRY(dd_check_store(ctx, host_kv_per_layer[l], "host_kv_per_layer[l]", &dv));
    ctx->landmarks[l] = landmarks_per_layer[l];
    ctx->host_kv[l] = dv;
    ctx->host_kv_orig[l] = host_kv_per_layer[l];
  }
  DD_TRY(dd_check_dev(ctx, n_pages, "n_pages", 4));
  DD_TRY(dd_check_dev(ctx, ctx_len, "ctx_len", 4));
  ctx->n_pages = n_pages;
  ctx->ctx_len = ctx_len;
  if (ctx->n_pages_host)       // the staged gather checks indices on the host
    DD_CUDA_TRY(ctx, cudaMemcpy(ctx->n_pages_host, n_pages, ctx->cfg.batch * sizeof(int), cudaMemcpyDeviceToHost));
  ctx->bound = true;
  return DD_OK;
}

static int* dd_idx_of(dd_ctx* ctx, int parity, int layer) {
  const dd_config& c = ctx->cfg;
  return ctx->idx_tab + ((size_t)(parity & 1) * c.n_layers + layer) * c.batch * c.n_kv_heads * c.k_pages;
}

// What follows every selection of a set the pipeline will gather: in staged mode the set is copied to page-locked
// host memory on the stream that selected it; then the "selection done" event of the layer is recorded.
static int dd_after_select(dd_ctx* ctx, int parity, int layer, cudaStream_t st) {
  const dd_config& c = ctx->cfg;
  if (c.gather_mode == DD_GATHER_STAGED) {
    const size_t per_set = (size_t)c.batch * c.n_kv_heads * c.k_pages;
    DD_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->idx_host + ((size_t)(parity & 1) * c.n_layers + layer) * per_set,
                                     dd_idx_of(ctx, parity, layer), per_set * sizeof(int), cudaMemcpyDeviceToHost, st));
    DD_CUDA_TRY(ctx, cudaEventRecord(ctx->idx_copied[layer], st));
  }
  DD_CUDA_TRY(ctx, cudaEventRecord(ctx->sel_done[layer], st));
  return DD_OK;
}

// Gather number n = step * L + layer goes to slot n % D. It may start once the attention that last
// read the slot has released it and the selection that produced its index set is done.
static int dd_enqueue_gather(dd_ctx* ctx, long long n, cudaEvent_t ev_start = nullptr, cudaEvent_t ev_end = nullptr) {
  const dd_config& c = ctx->cfg;
  const int layer = (int)(n % c.n_layers), step = (int)(n / c.n_layers);
  const int slot = (int)(n % c.ring_depth);
  cudaStream_t xs = (cudaStream_t)c.copy_stream;
  if (ctx->released_recorded[slot]) DD_CUDA_TRY(ctx, cudaStreamWaitEvent(xs, ctx->released[slot], 0));
  DD_CUDA_TRY(ctx, cudaStreamWaitEvent(xs, ctx->sel_done[layer], 0));
  if (ev_start) DD_CUDA_TRY(ctx, cudaEventRecord(ev_start, xs));
  if (c.gather_mode == DD_GATHER_STAGED) {
    // the set was copied to the host right after its selection (normally a whole step ago)
    DD_TRY(dd_wait_index_copy(ctx, layer));
    const size_t per_set = (size_t)c.batch * c.n_kv_heads * c.k_pages;
    DD_TRY(dd_launch_gather_staged(ctx, ctx->host_kv_orig[layer], ctx->host_kv[layer],
                                   ctx->idx_host + ((size_t)(step & 1) * c.n_layers + layer) * per_set,
                                   dd_idx_of(ctx, step, layer), ctx->n_pages_host, ctx->n_pages,
                                   ctx->ring + (size_t)slot * ctx->slot_bytes, xs));
  } else {
    DD_TRY(dd_launch_gather(ctx, ctx->host_kv[layer], dd_idx_of(ctx, step, layer), ctx->n_pages,
                            ctx->ring + (size_t)slot * ctx->slot_bytes, xs));
  }
  if (ev_end) DD_CUDA_TRY(ctx, cudaEventRecord(ev_end, xs));
  DD_CUDA_TRY(ctx, cudaEventRecord(ctx->ready[slot], xs));
  return DD_OK;
}

extern "C" int dd_prime(dd_ctx* ctx, const void* q_init) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_prime: ctx is NULL");
  if (!ctx->bound) return dd_fail(ctx, DD_ERR_STATE, "dd_prime: call dd_bind first");
  DD_TRY(dd_check_dev(ctx, q_init, "q_init"));
  const dd_config& c = ctx->cfg;
  cudaStream_t cs = (cudaStream_t)c.compute_stream;
  // a restart must not overtake work of an earlier run that still uses the ring or the index tables
  DD_TRY(dd_sync(ctx, 30.0));
  const size_t q_layer = (size_t)c.batch * c.n_q_heads * DD_D;
  for (int l = 0; l < c.n_layers; ++l) {
    DD_TRY(dd_launch_select(ctx, (const __nv_bfloat16*)q_init + l * q_layer, 0, 1, ctx->landmarks[l], ctx->n_pages,
                            dd_idx_of(ctx, 0, l), nullptr, cs, ctx->ctx_len));
    DD_TRY(dd_after_select(ctx, 0, l, cs));
  }
  for (int i = 0; i < DD_MAX_RING; ++i) ctx->released_recorded[i] = false;
  const int ahead = c.ring_depth < c.n_layers ? c.ring_depth : c.n_layers;
  ctx->primed = false;
  for (long long n = 0; n < ahead; ++n) DD_TRY(dd_enqueue_gather(ctx, n));
  ctx->next_call = 0;
  ctx->in_flight = false;
  ctx->primed = true;
  return DD_OK;
}

static int dd_layer_step_body(dd_ctx* ctx, int step, int layer, const void* q, const void* k_new, const void* v_new,
                              void* out) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_decode_layer_step: ctx is NULL");
  if (!ctx->primed) return dd_fail(ctx, DD_ERR_STATE, "dd_decode_layer_step: call dd_bind and dd_prime first");
  const dd_config& c = ctx->cfg;
  if (layer < 0 || layer >= c.n_layers || step < 0) return dd_fail(ctx, DD_ERR_INVALID_ARG, "bad (step, layer) = (%d, %d)", step, layer);
  const long long n = (long long)step * c.n_layers + layer;
  if (n != ctx->next_call)
    return dd_fail(ctx, DD_ERR_STATE, "expected (step, layer) = (%lld, %lld), got (%d, %d)", ctx->next_call / c.n_layers,
                   ctx->next_call % c.n_layers, step, layer);
  DD_TRY(dd_check_dev(ctx, q, "q"));
  DD_TRY(dd_check_dev(ctx, out, "out"));
  if (k_new) DD_TRY(dd_check_dev(ctx, k_new, "k_new"));
  if (k_new) DD_TRY(dd_check_dev(ctx, v_new, "v_new"));
  cudaStream_t cs = (cudaStream_t)c.compute_stream;
  const int slot = (int)(n % c.ring_depth);
  ctx->in_flight = true;                         // from here on a failure leaves the ring protocol out of step
  cudaEvent_t* tr = nullptr;                     // this call's timeline events, when a trace is armed
  if (ctx->trace_on && ctx->trace_n < ctx->trace_cap) {
    tr = ctx->trace_ev + (size_t)ctx->trace_n * DD_TRACE_FIELDS;
    if (ctx->trace_n == 0) DD_CUDA_TRY(ctx, cudaEventRecord(ctx->trace_origin, cs));
    DD_CUDA_TRY(ctx, cudaEventRecord(tr[0], cs));
    ++ctx->trace_n;
  }

  const int spec_token = c.n_q_tokens - 1;
  const int* attn_idx = dd_idx_of(ctx, step, layer);
  // The selection of the next step's set is independent of this layer's attention. With a select stream it runs
  // there (the two-kernel path shares scratch with the true-index selection, so under correction only the fused
  // kernel may move); the compute stream rejoins it at the end of the call.
  cudaStream_t ss = (cudaStream_t)c.select_stream;
  const bool side_select = ss != nullptr && (!c.miss_correction || ctx->sel_cluster > 0);
  cudaStream_t sel_st = side_select ? ss : cs;
  if (side_select) {
    DD_CUDA_TRY(ctx, cudaEventRecord(ctx->q_ready, cs));
    DD_CUDA_TRY(ctx, cudaStreamWaitEvent(ss, ctx->q_ready, 0));
    DD_TRY(dd_launch_select(ctx, q, spec_token, c.n_q_tokens, ctx->landmarks[layer], ctx->n_pages,
                            dd_idx_of(ctx, step + 1, layer), nullptr, sel_st, ctx->ctx_len));
    DD_TRY(dd_after_select(ctx, step + 1, layer, sel_st));
  }
  if (c.miss_correction) {
    // true index from the current token, repair list, missing pages on the urgent stream; the selection for
    // the next step runs while that transfer is in flight
    cudaStream_t us = (cudaStream_t)c.urgent_stream;
    int* merged = ctx->idx_merged + (size_t)slot * c.batch * c.n_kv_heads * c.k_pages;
    DD_TRY(dd_launch_select(ctx, q, 0, c.n_q_tokens, ctx->landmarks[layer], ctx->n_pages, ctx->idx_true, nullptr, cs,
                            ctx->ctx_len));
    DD_TRY(dd_launch_diff(ctx, attn_idx, ctx->idx_true, slot, merged, cs));
    DD_CUDA_TRY(ctx, cudaEventRecord(ctx->fix_ready[slot], cs));
    DD_CUDA_TRY(ctx, cudaStreamWaitEvent(us, ctx->fix_ready[slot], 0));
    DD_CUDA_TRY(ctx, cudaStreamWaitEvent(us, ctx->ready[slot], 0));                  // the prefetch wrote the slot first
    if (tr) DD_CUDA_TRY(ctx, cudaEventRecord(tr[6], us));
    DD_TRY(dd_launch_gather_fix(ctx, ctx->host_kv[layer], slot, us));
    if (tr) DD_CUDA_TRY(ctx, cudaEventRecord(tr[7], us));
    DD_CUDA_TRY(ctx, cudaEventRecord(ctx->urgent_done[slot], us));
    if (!side_select) {
      DD_TRY(dd_launch_select(ctx, q, spec_token, c.n_q_tokens, ctx->landmarks[layer], ctx->n_pages,
                              dd_idx_of(ctx, step + 1, layer), nullptr, cs, ctx->ctx_len));
      DD_TRY(dd_after_select(ctx, step + 1, layer, cs));
    }
    DD_CUDA_TRY(ctx, cudaStreamWaitEvent(cs, ctx->ready[slot], 0));
    DD_CUDA_TRY(ctx, cudaStreamWaitEvent(cs, ctx->urgent_done[slot], 0));            // all transfers of the layer complete
    attn_idx = merged;
  } else {
    DD_CUDA_TRY(ctx, cudaStreamWaitEvent(cs, ctx->ready[slot], 0));                  // transfer complete
  }
  if (tr) DD_CUDA_TRY(ctx, cudaEventRecord(tr[1], cs));
  DD_TRY(dd_launch_attn(ctx, q, ctx->ring + (size_t)slot * ctx->slot_bytes, attn_idx, ctx->ctx_len, out, nullptr, cs,
                        k_new, v_new));
  if (tr) DD_CUDA_TRY(ctx, cudaEventRecord(tr[2], cs));
  // Measured: with the streaming kernel the layer period grows from 1318 to 1860 us when nothing but events
  // without timing follow the launch, and is back at 1318 us with one timing-enabled event recorded next to it
  // (before or after; it makes the stream take a completion timestamp). The split-KV kernel shows no such effect.
  else if (ctx->as_fence) DD_CUDA_TRY(ctx, cudaEventRecord(ctx->as_fence, cs));
  DD_CUDA_TRY(ctx, cudaEventRecord(ctx->released[slot], cs));                        // buffer released
  ctx->released_recorded[slot] = true;
  if (!c.miss_correction && !side_select) {
    DD_TRY(dd_launch_select(ctx, q, spec_token, c.n_q_tokens, ctx->landmarks[layer], ctx->n_pages,
                            dd_idx_of(ctx, step + 1, layer), nullptr, cs, ctx->ctx_len));
    DD_TRY(dd_after_select(ctx, step + 1, layer, cs));
  }
  if (side_select) DD_CUDA_TRY(ctx, cudaStreamWaitEvent(cs, ctx->sel_done[layer], 0));   // q may be reused after this call
  // the slot just released takes the gather `ahead` layers further on (index set known: it was
  // selected one step earlier, or just now when the ring is deeper than the model)
  if (tr) DD_CUDA_TRY(ctx, cudaEventRecord(tr[3], cs));
  const int ahead = c.ring_depth < c.n_layers ? c.ring_depth : c.n_layers;
  DD_TRY(dd_enqueue_gather(ctx, n + ahead, tr ? tr[4] : nullptr, tr ? tr[5] : nullptr));
  ctx->next_call = n + 1;
  ctx->in_flight = false;
  return DD_OK;
}

// A failure after the call began to enqueue work cannot be undone (events are recorded, index tables may be
// overwritten): the context then needs dd_prime again.
static int dd_layer_step_impl(dd_ctx* ctx, int step, int layer, const void* q, const void* k_new, const void* v_new,
                              void* out) {
  const int rc = dd_layer_step_body(ctx, step, layer, q, k_new, v_new, out);
  if (rc != DD_OK && ctx && ctx->in_flight) {
    ctx->primed = false;
    ctx->in_flight = false;
  }
  return rc;
}

extern "C" int dd_decode_layer_step(dd_ctx* ctx, int step, int layer, const void* q, void* out) {
  return dd_layer_step_impl(ctx, step, layer, q, nullptr, nullptr, out);
}

extern "C" int dd_decode_step_host(dd_ctx* ctx, int step, const void* q_host, void* out_host) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_decode_step_host: ctx is NULL");
  if (!ctx->primed) return dd_fail(ctx, DD_ERR_STATE, "dd_decode_step_host: call dd_bind and dd_prime first");
  const dd_config& c = ctx->cfg;
  for (int i = 0; i < 2; ++i) {                  // both host buffers must be page-locked: the copies are asynchronous
    const void* p = i == 0 ? q_host : (const void*)out_host;
    if (!p) return dd_fail(ctx, DD_ERR_INVALID_ARG, "dd_decode_step_host: host buffer is NULL");
    cudaPointerAttributes a;
    cudaError_t e = cudaPointerGetAttributes(&a, p);
    if (e != cudaSuccess) { cudaGetLastError(); return dd_fail(ctx, DD_ERR_INVALID_ARG, "%s", cudaGetErrorString(e)); }
    if (a.type != cudaMemoryTypeHost)
      return dd_fail(ctx, DD_ERR_NOT_PINNED, "dd_decode_step_host: %s must be page-locked host memory", i == 0 ? "q_host" : "out_host");
  }
  cudaStream_t cs = (cudaStream_t)c.compute_stream;
  const size_t per_layer = (size_t)c.batch * c.n_q_tokens * c.n_q_heads * DD_D;
  const size_t bytes = per_layer * c.n_layers * sizeof(__nv_bfloat16);
  if ((long long)step * c.n_layers != ctx->next_call)
    return dd_fail(ctx, DD_ERR_STATE, "expected step %lld, layer %lld next, got step %d", ctx->next_call / c.n_layers,
                   ctx->next_call % c.n_layers, step);
  // once the first copy is queued the step cannot be taken back: any later failure needs dd_prime again
  cudaError_t e = cudaMemcpyAsync(ctx->stage_q, q_host, bytes, cudaMemcpyHostToDevice, cs);
  int rc = e == cudaSuccess ? DD_OK : dd_fail(ctx, DD_ERR_CUDA, "cudaMemcpyAsync(q_host): %s", cudaGetErrorString(e));
  for (int l = 0; l < c.n_layers && rc == DD_OK; ++l)
    rc = dd_layer_step_impl(ctx, step, l, ctx->stage_q + l * per_layer, nullptr, nullptr, ctx->stage_out + l * per_layer);
  if (rc == DD_OK) {
    e = cudaMemcpyAsync(out_host, ctx->stage_out, bytes, cudaMemcpyDeviceToHost, cs);
    if (e != cudaSuccess) rc = dd_fail(ctx, DD_ERR_CUDA, "cudaMemcpyAsync(out_host): %s", cudaGetErrorString(e));
  }
  if (rc != DD_OK) ctx->primed = false;
  return rc;
}

extern "C" int dd_decode_layer_step_causal(dd_ctx* ctx, int step, int layer, const void* q, const void* k_new,
                                           const void* v_new, void* out) {
  if (!k_new || !v_new) return dd_fail(ctx, DD_ERR_INVALID_ARG, "dd_decode_layer_step_causal: k_new / v_new is NULL");
  return dd_layer_step_impl(ctx, step, layer, q, k_new, v_new, out);
}

extern "C" int dd_sparse_decode_attn_causal(dd_ctx* ctx, const void* q, int slot, const int* idx, const int* ctx_len,
                                            const void* k_new, const void* v_new, void* out, float* out_lse,
                                            void* stream) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_causal: ctx is NULL");
  if (slot < 0 || slot >= ctx->cfg.ring_depth)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "slot %d outside [0, %d)", slot, ctx->cfg.ring_depth);
  DD_TRY(dd_check_dev(ctx, q, "q"));
  DD_TRY(dd_check_dev(ctx, idx, "idx", 4));
  DD_TRY(dd_check_dev(ctx, ctx_len, "ctx_len", 4));
  DD_TRY(dd_check_dev(ctx, k_new, "k_new"));
  DD_TRY(dd_check_dev(ctx, v_new, "v_new"));
  DD_TRY(dd_check_dev(ctx, out, "out"));
  if (out_lse) DD_TRY(dd_check_dev(ctx, out_lse, "out_lse", 4));
  return dd_launch_attn(ctx, q, ctx->ring + (size_t)slot * ctx->slot_bytes, idx, ctx_len, out, out_lse,
                        (cudaStream_t)stream, k_new, v_new);
}

extern "C" int dd_get_indices(dd_ctx* ctx, int step_parity, int layer, const int** dev_idx) {
  if (!ctx || !dev_idx) return dd_fail(ctx, DD_ERR_INVALID_ARG, "dd_get_indices: NULL argument");
  if (layer < 0 || layer >= ctx->cfg.n_layers) return dd_fail(ctx, DD_ERR_INVALID_ARG, "layer %d outside [0, %d)", layer, ctx->cfg.n_layers);
  *dev_idx = dd_idx_of(ctx, step_parity, layer);
  return DD_OK;
}

extern "C" int dd_diff_indices(dd_ctx* ctx, const int* pred_idx, const int* true_idx, int slot, int* merged_idx,
                               void* stream) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_diff_indices: ctx is NULL");
  if (slot < 0 || slot >= ctx->cfg.ring_depth)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "slot %d outside [0, %d)", slot, ctx->cfg.ring_depth);
  DD_TRY(dd_check_dev(ctx, pred_idx, "pred_idx", 4));
  DD_TRY(dd_check_dev(ctx, true_idx, "true_idx", 4));
  DD_TRY(dd_check_dev(ctx, merged_idx, "merged_idx", 4));
  return dd_launch_diff(ctx, pred_idx, true_idx, slot, merged_idx, (cudaStream_t)stream);
}

extern "C" int dd_fetch_missing_from_host(dd_ctx* ctx, const void* host_kv_layer, int slot, void* stream) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_fetch_missing_from_host: ctx is NULL");
  if (slot < 0 || slot >= ctx->cfg.ring_depth)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "slot %d outside [0, %d)", slot, ctx->cfg.ring_depth);
  const void* kv_dev = nullptr;
  DD_TRY(dd_check_store(ctx, host_kv_layer, "host_kv_layer", &kv_dev));
  return dd_launch_gather_fix(ctx, kv_dev, slot, (cudaStream_t)stream);
}

extern "C" int dd_get_merged_indices(dd_ctx* ctx, int slot, const int** dev_idx) {
  if (!ctx || !dev_idx) return dd_fail(ctx, DD_ERR_INVALID_ARG, "dd_get_merged_indices: NULL argument");
  if (slot < 0 || slot >= ctx->cfg.ring_depth)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "slot %d outside [0, %d)", slot, ctx->cfg.ring_depth);
  *dev_idx = ctx->idx_merged + (size_t)slot * ctx->cfg.batch * ctx->cfg.n_kv_heads * ctx->cfg.k_pages;
  return DD_OK;
}

extern "C" int dd_miss_stats(dd_ctx* ctx, unsigned long long* missing, unsigned long long* selected, int reset) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_miss_stats: ctx is NULL");
  DD_TRY(dd_sync(ctx, 60.0));
  DD_CUDA_TRY(ctx, cudaDeviceSynchronize());
  unsigned long long w[2] = {0, 0};
  DD_CUDA_TRY(ctx, cudaMemcpy(w, ctx->miss_stats, sizeof(w), cudaMemcpyDeviceToHost));
  if (reset) DD_CUDA_TRY(ctx, cudaMemset(ctx->miss_stats, 0, sizeof(w)));
  if (missing) *missing = w[0];
  if (selected) *selected = w[1];
  return DD_OK;
}

extern "C" int dd_probe_attn_loads(dd_ctx* ctx, int slot, void* stream) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_probe_attn_loads: ctx is NULL");
  if (slot < 0 || slot >= ctx->cfg.ring_depth)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "slot %d outside [0, %d)", slot, ctx->cfg.ring_depth);
  return dd_launch_attn_loads_only(ctx, ctx->ring + (size_t)slot * ctx->slot_bytes, (cudaStream_t)stream);
}

extern "C" int dd_probe_select_loads(dd_ctx* ctx, const void* landmarks, const int* n_pages, void* stream) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_probe_select_loads: ctx is NULL");
  DD_TRY(dd_check_dev(ctx, landmarks, "landmarks"));
  DD_TRY(dd_check_dev(ctx, n_pages, "n_pages", 4));
  return dd_launch_select_loads_only(ctx, landmarks, n_pages, (cudaStream_t)stream);
}

extern "C" int dd_trace_begin(dd_ctx* ctx, int max_layer_steps) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_trace_begin: ctx is NULL");
  if (max_layer_steps < 1 || max_layer_steps > (1 << 20)) return dd_fail(ctx, DD_ERR_INVALID_ARG, "max_layer_steps out of range");
  DD_TRY(dd_sync(ctx, 60.0));
  if (ctx->trace_ev) {
    for (int i = 0; i < ctx->trace_cap * DD_TRACE_FIELDS; ++i)
      if (ctx->trace_ev[i]) cudaEventDestroy(ctx->trace_ev[i]);
    delete[] ctx->trace_ev;
    ctx->trace_ev = nullptr;
  }
  if (!ctx->trace_origin) DD_CUDA_TRY(ctx, cudaEventCreate(&ctx->trace_origin));
  ctx->trace_cap = max_layer_steps;
  ctx->trace_n = 0;
  ctx->trace_ev = new cudaEvent_t[(size_t)max_layer_steps * DD_TRACE_FIELDS]();
  for (int i = 0; i < max_layer_steps * DD_TRACE_FIELDS; ++i) DD_CUDA_TRY(ctx, cudaEventCreate(&ctx->trace_ev[i]));
  ctx->trace_on = true;
  return DD_OK;
}

extern "C" int dd_trace_end(dd_ctx* ctx, int* n_recorded) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_trace_end: ctx is NULL");
  if (!ctx->trace_ev) return dd_fail(ctx, DD_ERR_STATE, "dd_trace_end: no trace was begun");
  ctx->trace_on = false;
  DD_TRY(dd_sync(ctx, 120.0));
  if (n_recorded) *n_recorded = ctx->trace_n;
  return DD_OK;
}

extern "C" int dd_trace_read(dd_ctx* ctx, int first, int count, float* out) {
  if (!ctx || !out) return dd_fail(ctx, DD_ERR_INVALID_ARG, "dd_trace_read: NULL argument");
  if (!ctx->trace_ev || ctx->trace_on) return dd_fail(ctx, DD_ERR_STATE, "dd_trace_read: end the trace first");
  if (first < 0 || count < 0 || first + count > ctx->trace_n)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "rows [%d, %d) outside the %d traced calls", first, first + count, ctx->trace_n);
  for (int i = 0; i < count; ++i) {
    for (int f = 0; f < DD_TRACE_FIELDS; ++f) {
      float ms = 0.f;
      if (f >= 6 && !ctx->cfg.miss_correction) {   // urgent-stream points exist under miss correction only
        out[(size_t)i * DD_TRACE_FIELDS + f] = -1.f;
        continue;
      }
      DD_CUDA_TRY(ctx, cudaEventElapsedTime(&ms, ctx->trace_origin, ctx->trace_ev[(size_t)(first + i) * DD_TRACE_FIELDS + f]));
      out[(size_t)i * DD_TRACE_FIELDS + f] = ms * 1e3f;
    }
  }
  return DD_OK;
}

extern "C" int dd_gather_stats(dd_ctx* ctx, unsigned long long* out, int reset) {
  if (!ctx || !out) return dd_fail(ctx, DD_ERR_INVALID_ARG, "dd_gather_stats: NULL argument");
  for (int i = 0; i < DD_GATHER_STATS_FIELDS; ++i) out[i] = ctx->gstats[i];
  if (reset) memset(ctx->gstats, 0, sizeof(ctx->gstats));
  return DD_OK;
}

extern "C" int dd_set_bulk_wait(dd_ctx* ctx, double wait_seconds, int inflate_first_stage) {
  if (!ctx) return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_set_bulk_wait: ctx is NULL");
  if (!(wait_seconds > 0.0) || wait_seconds > 60.0) return dd_fail(ctx, DD_ERR_INVALID_ARG, "wait_seconds must be in (0, 60]");
  ctx->bulk_wait_ns = (unsigned long long)(wait_seconds * 1e9);
  ctx->bulk_inflate = inflate_first_stage ? 1 : 0;
  return DD_OK;
}
