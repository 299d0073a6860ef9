// Gather of the selected KV pages from pinned host memory into a ring slot in attention layout.
//
// A page is 8 KiB contiguous in the host store (4 KiB of K followed by 4 KiB of V); in the slot the K
// halves of a (request, KV head) are contiguous, followed by the V halves. The copy is bitwise.
//
// DD_GATHER_LOADS: one warp per page, sixteen 16-byte loads per lane issued back to back (8 KiB of
// reads in flight per warp across the host link), then sixteen stores.
// DD_GATHER_BULK: one thread per block drives the bulk-copy engine: page -> shared memory ring
// (cp.async.bulk with mbarrier completion) -> two bulk stores into the slot. Every wait is bounded.
// DD_GATHER_STAGED: the host, which holds a copy of the index set, forms runs of adjacent selected pages and
// lets the device's copy engine move each long run with one asynchronous copy into a staging region; an
// assembly kernel places the staged pages in the slot, and the short runs are read by the zero-copy kernel on
// a second stream at the same time.
#include <chrono>
#include <vector>

#include "dd_common.cuh"

__device__ __forceinline__ int dd_checked_page(const int* idx, const int* n_pages, int item, int b, int P,
                                               int* err_word) {
  int p = idx[item];
  int limit = P;
  if (n_pages) {
    const int np = n_pages[b];
    limit = np < P ? np : P;
  }
  if (p < 0 || p >= limit) {
    dd_report(err_word, DD_ERR_INDEX_RANGE, p);
    p = p < 0 ? 0 : (limit > 0 ? limit - 1 : 0);
  }
  return p;
}

__global__ void __launch_bounds__(256) dd_gather_loads_kernel(const char* __restrict__ kv,
                                                              const int* __restrict__ idx,
                                                              const int* __restrict__ n_pages,
                                                              char* __restrict__ slot, int Hkv, int P, int k,
                                                              int total, int* err_word) {
  const int lane = threadIdx.x & 31;
  const int warps_per_block = blockDim.x >> 5;
  const int n_warps = gridDim.x * warps_per_block;
  // consecutive pages go to different blocks so that every SM in use has work from the start
  for (int item = (threadIdx.x >> 5) * gridDim.x + blockIdx.x; item < total; item += n_warps) {
    const int j = item % k;
    const int bg = item / k;
    const int p = dd_checked_page(idx, n_pages, item, bg / Hkv, P, err_word);
    const char* src = kv + ((size_t)bg * P + p) * DD_PAGE_BYTES + lane * 16;
    char* dst_k = slot + ((size_t)bg * 2 * k + j) * DD_HALF_PAGE_BYTES + lane * 16;
    char* dst_v = dst_k + (size_t)k * DD_HALF_PAGE_BYTES;
    uint4 r[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) r[i] = dd_ld_stream(src + i * 512);
#pragma unroll
    for (int i = 0; i < 8; ++i) dd_st_v4(dst_k + i * 512, r[i]);
#pragma unroll
    for (int i = 0; i < 8; ++i) dd_st_v4(dst_v + i * 512, r[8 + i]);
  }
}

// ------------------------------------------------------------------------------------------------
// Bulk-copy engine variant
// ------------------------------------------------------------------------------------------------
constexpr int BULK_STAGES = 16;                       // 16 x 8 KiB = 128 KiB of shared memory per block

__device__ __forceinline__ uint32_t dd_smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long dd_globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ bool dd_mbar_wait_bounded(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
  const unsigned long long t0 = dd_globaltimer();
  for (unsigned it = 0;; ++it) {
    if ((it & 63u) == 63u && dd_globaltimer() - t0 > limit_ns) return false;
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
}

__global__ void __launch_bounds__(32) dd_gather_bulk_kernel(const char* __restrict__ kv, const int* __restrict__ idx,
                                                            const int* __restrict__ n_pages, char* __restrict__ slot,
                                                            int Hkv, int P, int k, int total, int* err_word,
                                                            unsigned long long wait_ns, int inflate) {
  extern __shared__ __align__(128) unsigned char stage_mem[];     // BULK_STAGES pages
  __shared__ __align__(8) unsigned long long full_bar[BULK_STAGES];
  if (threadIdx.x != 0) return;                       // one thread drives the engine; no block-wide barrier is used

  const int n_mine = blockIdx.x < total ? (total - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  for (int s = 0; s < BULK_STAGES; ++s)
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(dd_smem_addr(&full_bar[s])));
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");

  auto issue_load = [&](int n) {                      // n-th page of this block -> stage n % BULK_STAGES
    const int item = blockIdx.x + n * gridDim.x;
    const int bg = item / k;
    const int p = dd_checked_page(idx, n_pages, item, bg / Hkv, P, err_word);
    const char* src = kv + ((size_t)bg * P + p) * DD_PAGE_BYTES;
    const int s = n % BULK_STAGES;
    const uint32_t bar = dd_smem_addr(&full_bar[s]);
    const uint32_t dst = dd_smem_addr(stage_mem + (size_t)s * DD_PAGE_BYTES);
    // test hook: the first stage of block 0 may be told to expect more bytes than its copy delivers
    const uint32_t expect = (uint32_t)DD_PAGE_BYTES + ((inflate && n == 0 && blockIdx.x == 0) ? 16u : 0u);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(expect) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"((uint32_t)DD_PAGE_BYTES), "r"(bar)
                 : "memory");
  };

  int issued = 0;
  for (; issued < n_mine && issued < BULK_STAGES - 1; ++issued) issue_load(issued);

  bool ok = true;
  int n = 0;
  for (; n < n_mine; ++n) {
    const int s = n % BULK_STAGES;
    if (!dd_mbar_wait_bounded(dd_smem_addr(&full_bar[s]), (uint32_t)((n / BULK_STAGES) & 1), wait_ns)) { ok = false; break; }
    const int item = blockIdx.x + n * gridDim.x;
    const int j = item % k, bg = item / k;
    char* dst_k = slot + ((size_t)bg * 2 * k + j) * DD_HALF_PAGE_BYTES;
    char* dst_v = dst_k + (size_t)k * DD_HALF_PAGE_BYTES;
    const uint32_t src = dd_smem_addr(stage_mem + (size_t)s * DD_PAGE_BYTES);
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst_k), "r"(src),
                 "r"((uint32_t)DD_HALF_PAGE_BYTES)
                 : "memory");
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst_v),
                 "r"(src + DD_HALF_PAGE_BYTES), "r"((uint32_t)DD_HALF_PAGE_BYTES)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    if (issued < n_mine) {
      // the stage the next load lands in was last read by the stores of page n-1: all but the newest
      // store group must have finished reading shared memory
      asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      issue_load(issued);
      ++issued;
    }
  }
  if (!ok) {
    dd_report(err_word, DD_ERR_WAIT_EXPIRED, 1);
    // loads already issued may still land in shared memory: give each one more bounded wait before leaving
    for (int m = n + 1; m < issued; ++m)
      dd_mbar_wait_bounded(dd_smem_addr(&full_bar[m % BULK_STAGES]), (uint32_t)((m / BULK_STAGES) & 1), wait_ns);
  }
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");       // stores complete before the block retires
}

int dd_launch_gather(dd_ctx* ctx, const void* kv_dev, const int* idx, const int* n_pages, char* slot, cudaStream_t st) {
  const dd_config& c = ctx->cfg;
  const int total = c.batch * c.n_kv_heads * c.k_pages;
  if (c.gather_mode == DD_GATHER_BULK) {
    int ctas = c.gather_ctas > 0 ? c.gather_ctas : 16;
    if (ctas > total) ctas = total;
    dd_gather_bulk_kernel<<<ctas, 32, BULK_STAGES * DD_PAGE_BYTES, st>>>((const char*)kv_dev, idx, n_pages, slot,
                                                                         c.n_kv_heads, c.max_pages, c.k_pages, total,
                                                                         ctx->err_word, ctx->bulk_wait_ns,
                                                                         ctx->bulk_inflate);
  } else {
    int ctas = c.gather_ctas > 0 ? c.gather_ctas : 16;
    const int max_ctas = (total + 7) / 8;
    if (ctas > max_ctas) ctas = max_ctas;
    dd_gather_loads_kernel<<<ctas, 256, 0, st>>>((const char*)kv_dev, idx, n_pages, slot, c.n_kv_heads, c.max_pages,
                                                 c.k_pages, total, ctx->err_word);
  }
  DD_CUDA_TRY(ctx, cudaGetLastError());
  return DD_OK;
}

// ------------------------------------------------------------------------------------------------
// Staged variant: copy engine -> staging region -> assembly kernel; short runs by zero-copy loads
// ------------------------------------------------------------------------------------------------
// The zero-copy kernel over a list of slot items (item = unit * k + position) instead of all of them.
__global__ void __launch_bounds__(256) dd_gather_list_kernel(const char* __restrict__ kv, const int* __restrict__ idx,
                                                             const int* __restrict__ n_pages,
                                                             const int* __restrict__ items, int n_items,
                                                             char* __restrict__ slot, int Hkv, int P, int k,
                                                             int* err_word) {
  const int lane = threadIdx.x & 31;
  const int n_warps = gridDim.x * (blockDim.x >> 5);
  for (int i = (threadIdx.x >> 5) * gridDim.x + blockIdx.x; i < n_items; i += n_warps) {
    const int item = items[i];
    const int j = item % k;
    const int bg = item / k;
    const int p = dd_checked_page(idx, n_pages, item, bg / Hkv, P, err_word);
    const char* src = kv + ((size_t)bg * P + p) * DD_PAGE_BYTES + lane * 16;
    char* dst_k = slot + ((size_t)bg * 2 * k + j) * DD_HALF_PAGE_BYTES + lane * 16;
    char* dst_v = dst_k + (size_t)k * DD_HALF_PAGE_BYTES;
    uint4 r[16];
#pragma unroll
    for (int q = 0; q < 16; ++q) r[q] = dd_ld_stream(src + q * 512);
#pragma unroll
    for (int q = 0; q < 8; ++q) dd_st_v4(dst_k + q * 512, r[q]);
#pragma unroll
    for (int q = 0; q < 8; ++q) dd_st_v4(dst_v + q * 512, r[8 + q]);
  }
}

// Assembly: staged page s (8 KiB: K half, V half) goes to slot item map[s]; map[s] < 0 marks a page that was
// only fetched because it shares an aligned block with a selected one.
__global__ void __launch_bounds__(256) dd_assemble_kernel(const char* __restrict__ staging, const int* __restrict__ map,
                                                          int n_staged, char* __restrict__ slot, int k) {
  const int lane = threadIdx.x & 31;
  const int n_warps = gridDim.x * (blockDim.x >> 5);
  for (int s = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); s < n_staged; s += n_warps) {
    const int item = map[s];
    if (item < 0) continue;
    const int j = item % k;
    const int bg = item / k;
    const char* src = staging + (size_t)s * DD_PAGE_BYTES + lane * 16;
    char* dst_k = slot + ((size_t)bg * 2 * k + j) * DD_HALF_PAGE_BYTES + lane * 16;
    char* dst_v = dst_k + (size_t)k * DD_HALF_PAGE_BYTES;
    uint4 r[16];
#pragma unroll
    for (int q = 0; q < 16; ++q) r[q] = dd_ld_stream(src + q * 512);
#pragma unroll
    for (int q = 0; q < 8; ++q) dd_st_v4(dst_k + q * 512, r[q]);
#pragma unroll
    for (int q = 0; q < 8; ++q) dd_st_v4(dst_v + q * 512, r[8 + q]);
  }
}

// Host wait on an event with a deadline (the staged gather's only blocking points).
static int dd_wait_event(dd_ctx* ctx, cudaEvent_t ev, double seconds, const char* what) {
  const auto deadline = std::chrono::steady_clock::now() + std::chrono::duration<double>(seconds);
  for (;;) {
    const cudaError_t e = cudaEventQuery(ev);
    if (e == cudaSuccess) return DD_OK;
    if (e != cudaErrorNotReady) return dd_fail(ctx, DD_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    if (std::chrono::steady_clock::now() > deadline)
      return dd_fail(ctx, DD_ERR_TIMEOUT, "%s: not complete after %.1f s", what, seconds);
  }
}

int dd_wait_index_copy(dd_ctx* ctx, int layer) {
  const auto t0 = std::chrono::steady_clock::now();
  const int rc = dd_wait_event(ctx, ctx->idx_copied[layer], 30.0, "staged gather: copy of the index set to the host");
  ctx->gstats[5] += (unsigned long long)std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - t0).count();
  return rc;
}

// The host's part of the staged gather, free of any CUDA call so that it can be tested without a GPU: from the index
// set [units][k] form the copy-engine copies (runs of adjacent selected pages of at least min_run pages, or, with
// block_pages > 0, every aligned block of that many pages that holds a selected page, adjacent blocks merged), the map
// staged page -> slot item (-1 for a page that was only fetched along), and the list of slot items left to the
// zero-copy kernel. A copy is three numbers: source page (unit * P + page), first staging page, pages. Indices outside
// [0, limit) are clamped like on the device and the first one is reported in bad[2] = {flag, value}.
extern "C" int dd_test_stage_plan(const int* idx, const int* n_pages, int batch, int n_kv_heads, int max_pages, int k_pages,
                                  int min_run, int block_pages, long long staging_capacity, long long* copies,
                                  long long max_copies, long long* n_copies_out, int* map, long long* n_staged_out,
                                  int* stragglers, long long* n_stragglers_out, int* bad) {
  if (!idx || !copies || !map || !stragglers || !n_copies_out || !n_staged_out || !n_stragglers_out || batch < 1 ||
      n_kv_heads < 1 || max_pages < 1 || k_pages < 1 || min_run < 1 || block_pages < 0)
    return DD_ERR_INVALID_ARG;
  const int Hkv = n_kv_heads, P = max_pages, k = k_pages, Bp = block_pages;
  const int units = batch * Hkv;
  long long n_staged = 0, n_strag = 0, n_copies = 0;
  for (int bg = 0; bg < units; ++bg) {
    int limit = P;
    if (n_pages) limit = n_pages[bg / Hkv] < P ? n_pages[bg / Hkv] : P;
    const int* row = idx + (size_t)bg * k;
    auto page_of = [&](int j) {
      int p = row[j];
      if (p < 0 || p >= limit) {
        if (bad && bad[0] == 0) { bad[0] = 1; bad[1] = p; }
        p = p < 0 ? 0 : (limit > 0 ? limit - 1 : 0);
      }
      return p;
    };
    int j = 0;
    while (j < k) {
      const int p = page_of(j);
      int jj = j + 1, page0, n_pages_copy;
      if (Bp > 0) {
        // aligned blocks: extend over the selected pages that fall into this block or the one right after the last
        int blk_end = p / Bp;
        while (jj < k) {
          const int bj = page_of(jj) / Bp;
          if (bj < blk_end || bj > blk_end + 1 || page_of(jj) <= page_of(jj - 1)) break;
          blk_end = bj;
          ++jj;
        }
        page0 = (p / Bp) * Bp;
        const int page1 = (blk_end + 1) * Bp < P ? (blk_end + 1) * Bp : P;
        n_pages_copy = page1 - page0;
      } else {
        while (jj < k && page_of(jj) == p + (jj - j)) ++jj;
        page0 = p;
        n_pages_copy = jj - j;
        if (n_pages_copy < min_run) {
          for (int x = j; x < jj; ++x) stragglers[n_strag++] = bg * k + x;
          j = jj;
          continue;
        }
      }
      if (n_staged + n_pages_copy > staging_capacity || n_copies >= max_copies) return DD_ERR_INVALID_ARG;
      for (int x = 0; x < n_pages_copy; ++x) map[n_staged + x] = -1;
      for (int x = j; x < jj; ++x) map[n_staged + page_of(x) - page0] = bg * k + x;
      copies[3 * n_copies + 0] = (long long)bg * P + page0;
      copies[3 * n_copies + 1] = n_staged;
      copies[3 * n_copies + 2] = n_pages_copy;
      ++n_copies;
      n_staged += n_pages_copy;
      j = jj;
    }
  }
  *n_copies_out = n_copies;
  *n_staged_out = n_staged;
  *n_stragglers_out = n_strag;
  return DD_OK;
}

int dd_launch_gather_staged(dd_ctx* ctx, const void* kv_src, const void* kv_dev, const int* idx_h, const int* idx_dev,
                            const int* n_pages_h, const int* n_pages_dev, char* slot, cudaStream_t st) {
  const dd_config& c = ctx->cfg;
  const int Hkv = c.n_kv_heads, P = c.max_pages, k = c.k_pages;
  const long long total = (long long)c.batch * Hkv * k;
  const int li = (int)(ctx->list_next % DD_STAGE_LISTS);
  if (ctx->list_used[li]) {
    const auto tw = std::chrono::steady_clock::now();
    const int rc = dd_wait_event(ctx, ctx->list_free[li], 30.0, "staged gather: descriptor buffer still in use");
    ctx->gstats[5] += (unsigned long long)std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - tw).count();
    if (rc != DD_OK) return rc;
  }
  const auto t0 = std::chrono::steady_clock::now();
  int* map = ctx->list_host[li];
  int* strag = map + ctx->staging_pages;
  long long n_staged = 0, n_strag = 0, n_copies = 0;
  int bad[2] = {0, 0};
  if (dd_test_stage_plan(idx_h, n_pages_h, c.batch, Hkv, P, k, ctx->stage_min_run, ctx->stage_block,
                         (long long)ctx->staging_pages, ctx->copy_plan, total, &n_copies, map, &n_staged, strag, &n_strag,
                         bad) != DD_OK)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "staged gather: staging region too small (index set not ascending?)");
  if (bad[0] && ctx->host_err[0] == 0) { ctx->host_err[0] = DD_ERR_INDEX_RANGE; ctx->host_err[1] = bad[1]; }
  DD_CUDA_TRY(ctx, cudaEventRecord(ctx->aux_fork, st));          // the short runs may start when the copies may
  const char* src_base = (const char*)kv_src;
  unsigned long long sel_staged = (unsigned long long)(total - n_strag);
  for (long long i = 0; i < n_copies; ++i) {
    const long long* cp = ctx->copy_plan + 3 * i;
    DD_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->staging + (size_t)cp[1] * DD_PAGE_BYTES, src_base + (size_t)cp[0] * DD_PAGE_BYTES,
                                     (size_t)cp[2] * DD_PAGE_BYTES, cudaMemcpyDefault, st));
  }
  if (n_strag > 0) {
    int ctas = c.gather_ctas > 0 ? c.gather_ctas : 16;
    const int max_ctas = (int)((n_strag + 7) / 8);
    if (ctas > max_ctas) ctas = max_ctas;
    DD_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->aux_stream, ctx->aux_fork, 0));
    dd_gather_list_kernel<<<ctas, 256, 0, ctx->aux_stream>>>((const char*)kv_dev, idx_dev, n_pages_dev,
                                                             ctx->list_dev[li] + ctx->staging_pages, (int)n_strag, slot, Hkv, P,
                                                             k, ctx->err_word);
    DD_CUDA_TRY(ctx, cudaGetLastError());
    DD_CUDA_TRY(ctx, cudaEventRecord(ctx->aux_join, ctx->aux_stream));
  }
  if (n_staged > 0) {
    int blocks = (int)((n_staged + 7) / 8);
    if (blocks > 4 * ctx->sm_count) blocks = 4 * ctx->sm_count;
    dd_assemble_kernel<<<blocks, 256, 0, st>>>(ctx->staging, ctx->list_dev[li], (int)n_staged, slot, k);
    DD_CUDA_TRY(ctx, cudaGetLastError());
  }
  if (n_strag > 0) DD_CUDA_TRY(ctx, cudaStreamWaitEvent(st, ctx->aux_join, 0));
  DD_CUDA_TRY(ctx, cudaEventRecord(ctx->list_free[li], st));
  ctx->list_used[li] = true;
  ++ctx->list_next;
  ctx->gstats[0] += 1;
  ctx->gstats[1] += (unsigned long long)n_copies;
  ctx->gstats[2] += (unsigned long long)n_staged * DD_PAGE_BYTES;
  ctx->gstats[3] += sel_staged;
  ctx->gstats[4] += (unsigned long long)n_strag;
  ctx->gstats[6] += (unsigned long long)std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - t0).count();
  return DD_OK;
}

int dd_gather_setup(dd_ctx* ctx) {
  DD_CUDA_TRY(ctx, cudaFuncSetAttribute(dd_gather_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        BULK_STAGES * DD_PAGE_BYTES));
  return DD_OK;
}
