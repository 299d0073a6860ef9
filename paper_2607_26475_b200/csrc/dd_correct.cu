// Miss correction: once the true index of a layer is known, the pages the prediction missed are fetched
// on the urgent stream into the buffer positions of the pages the true set does not want.
//
// dd_diff_kernel (one warp per (request, KV head)) compares the two ascending page lists by binary search,
// pairs the m-th missing page with the m-th victim position, writes the repaired page list of the slot and
// appends (unit, position, page) to a compact fix list. dd_gather_fix_kernel copies the listed pages from
// the pinned store, one warp per page, exactly like the prefetch gather.
#include "dd_common.cuh"

__device__ __forceinline__ bool dd_sorted_contains(const int* __restrict__ a, int n, int v) {
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (a[mid] < v) lo = mid + 1;
    else hi = mid;
  }
  return lo < n && a[lo] == v;
}

__global__ void __launch_bounds__(128) dd_diff_kernel(const int* __restrict__ pred, const int* __restrict__ truth,
                                                      int* __restrict__ merged, int2* __restrict__ stage,
                                                      int4* __restrict__ fix_list, unsigned int* __restrict__ fix_count,
                                                      unsigned long long* __restrict__ stats, int k, int n_units) {
  const int lane = threadIdx.x & 31;
  const int u = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (u >= n_units) return;
  const int* p_u = pred + (size_t)u * k;
  const int* t_u = truth + (size_t)u * k;
  int* m_u = merged + (size_t)u * k;
  int2* s_u = stage + (size_t)u * k;
  const unsigned lt = (1u << lane) - 1u;
  // victims: positions whose predicted page is not in the true set (ascending position)
  int n_vic = 0;
  for (int j0 = 0; j0 < k; j0 += 32) {
    const int j = j0 + lane;
    int page = 0;
    bool vic = false;
    if (j < k) {
      page = p_u[j];
      m_u[j] = page;
      vic = !dd_sorted_contains(t_u, k, page);
    }
    const unsigned b = __ballot_sync(0xffffffffu, vic);
    if (vic) s_u[n_vic + __popc(b & lt)].x = j;
    n_vic += __popc(b);
  }
  // missing: true pages the prediction does not hold (ascending page)
  int n_mis = 0;
  for (int i0 = 0; i0 < k; i0 += 32) {
    const int i = i0 + lane;
    int page = 0;
    bool mis = false;
    if (i < k) {
      page = t_u[i];
      mis = !dd_sorted_contains(p_u, k, page);
    }
    const unsigned b = __ballot_sync(0xffffffffu, mis);
    if (mis) s_u[n_mis + __popc(b & lt)].y = page;
    n_mis += __popc(b);
  }
  __syncwarp();
  const int n_fix = n_vic < n_mis ? n_vic : n_mis;    // equal when both lists hold k distinct pages
  unsigned base = 0;
  if (lane == 0) {
    base = atomicAdd(fix_count, (unsigned)n_fix);
    atomicAdd(&stats[0], (unsigned long long)n_fix);
    atomicAdd(&stats[1], (unsigned long long)k);
  }
  base = __shfl_sync(0xffffffffu, base, 0);
  for (int m = lane; m < n_fix; m += 32) {
    const int2 f = s_u[m];
    m_u[f.x] = f.y;
    fix_list[base + m] = make_int4(u, f.x, f.y, 0);
  }
}

__global__ void __launch_bounds__(256) dd_gather_fix_kernel(const char* __restrict__ kv, const int4* __restrict__ fix_list,
                                                            const unsigned int* __restrict__ fix_count,
                                                            char* __restrict__ slot, int P, int k, int* err_word) {
  const int lane = threadIdx.x & 31;
  const int n_warps = gridDim.x * (blockDim.x >> 5);
  const int total = (int)*fix_count;
  for (int i = (threadIdx.x >> 5) * gridDim.x + blockIdx.x; i < total; i += n_warps) {
    const int4 f = fix_list[i];
    int page = f.z;
    if (page < 0 || page >= P) {
      dd_report(err_word, DD_ERR_INDEX_RANGE, page);
      page = page < 0 ? 0 : P - 1;
    }
    const char* src = kv + ((size_t)f.x * P + page) * DD_PAGE_BYTES + lane * 16;
    char* dst_k = slot + ((size_t)f.x * 2 * k + f.y) * DD_HALF_PAGE_BYTES + lane * 16;
    char* dst_v = dst_k + (size_t)k * DD_HALF_PAGE_BYTES;
    uint4 r[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) r[j] = dd_ld_stream(src + j * 512);
#pragma unroll
    for (int j = 0; j < 8; ++j) dd_st_v4(dst_k + j * 512, r[j]);
#pragma unroll
    for (int j = 0; j < 8; ++j) dd_st_v4(dst_v + j * 512, r[8 + j]);
  }
}

int dd_launch_diff(dd_ctx* ctx, const int* pred, const int* truth, int slot, int* merged, cudaStream_t st) {
  const dd_config& c = ctx->cfg;
  const int n_units = c.batch * c.n_kv_heads;
  const size_t per_slot = (size_t)n_units * c.k_pages;
  DD_CUDA_TRY(ctx, cudaMemsetAsync(ctx->fix_count + slot, 0, sizeof(unsigned int), st));
  dd_diff_kernel<<<(n_units + 3) / 4, 128, 0, st>>>(pred, truth, merged, ctx->fix_stage + slot * per_slot,
                                                    ctx->fix_list + slot * per_slot, ctx->fix_count + slot,
                                                    ctx->miss_stats, c.k_pages, n_units);
  DD_CUDA_TRY(ctx, cudaGetLastError());
  return DD_OK;
}

int dd_launch_gather_fix(dd_ctx* ctx, const void* kv_dev, int slot, cudaStream_t st) {
  const dd_config& c = ctx->cfg;
  const size_t per_slot = (size_t)c.batch * c.n_kv_heads * c.k_pages;
  const int ctas = c.gather_ctas > 0 ? c.gather_ctas : 16;
  dd_gather_fix_kernel<<<ctas, 256, 0, st>>>((const char*)kv_dev, ctx->fix_list + slot * per_slot, ctx->fix_count + slot,
                                             ctx->ring + (size_t)slot * ctx->slot_bytes, c.max_pages, c.k_pages,
                                             ctx->err_word);
  DD_CUDA_TRY(ctx, cudaGetLastError());
  return DD_OK;
}
