// Gather of the selected KV pages from pinned host memory into a ring slot in attention layout.
//
// A page is 8 KiB contiguous in the host store (4 KiB of K followed by 4 KiB of V); in the slot the K
// halves of a (request, KV head) are contiguous, followed by the V halves. The copy is bitwise.
//
// DD_GATHER_LOADS: one warp per page, sixteen 16-byte loads per lane issued back to back (8 KiB of
// reads in flight per warp across the host link), then sixteen stores.
// DD_GATHER_BULK: one thread per block drives the bulk-copy engine: page -> shared memory ring
// (cp.async.bulk with mbarrier completion) -> two bulk stores into the slot. Every wait is bounded.
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
constexpr unsigned long long BULK_WAIT_NS = 2000000000ull;   // a wait gives up after two seconds

__device__ __forceinline__ uint32_t dd_smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long dd_globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ bool dd_mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  const unsigned long long t0 = dd_globaltimer();
  for (unsigned it = 0;; ++it) {
    if ((it & 63u) == 63u && dd_globaltimer() - t0 > BULK_WAIT_NS) return false;
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
                                                            int Hkv, int P, int k, int total, int* err_word) {
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
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)DD_PAGE_BYTES)
                 : "memory");
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
    if (!dd_mbar_wait_bounded(dd_smem_addr(&full_bar[s]), (uint32_t)((n / BULK_STAGES) & 1))) { ok = false; break; }
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
      dd_mbar_wait_bounded(dd_smem_addr(&full_bar[m % BULK_STAGES]), (uint32_t)((m / BULK_STAGES) & 1));
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
                                                                         ctx->err_word);
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

int dd_gather_setup(dd_ctx* ctx) {
  DD_CUDA_TRY(ctx, cudaFuncSetAttribute(dd_gather_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        BULK_STAGES * DD_PAGE_BYTES));
  return DD_OK;
}
