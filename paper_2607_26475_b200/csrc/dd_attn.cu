// GQA decode attention over the gathered set of a ring slot.
//
// Work is split flash-decoding style: grid (split, KV head, request), 4 warps per block, each warp
// walks pages of its split with a running soft-max; the block merges its warps, and the last block of
// a (request, KV head) to arrive merges the splits (arrival counter, no waiting).
//
// Both products run on warp-level bf16 MMAs in their transposed form, so that the up-to-8 query rows
// that share a KV head (Tq tokens x G heads) are the N = 8 columns and nothing is padded:
//   S^T[token, n] = K[token, :] . q[n, :]        A = K page (16 tokens x 128), B = q^T
//   O^T[d, n]    += V^T[d, token] P^T[token, n]   A = V^T (16 channels x 16 tokens), B = P^T
// K and V are read straight from global memory into MMA fragments with 16-byte loads:
//   * for S^T the 128 channels may be summed in any order, so a thread feeds k-slots {2t,2t+1,2t+8,2t+9}
//     of two consecutive k-steps with 8 consecutive channels of its token row (one load);
//   * for O^T the rows of the MMA (channels) may be assigned freely, so a thread takes 8 consecutive
//     channels of tokens 2t, 2t+1, 2t+8, 2t+9 and pairs neighbouring tokens with byte permutes;
//   * P^T goes from accumulator layout to B-operand layout with one 8x8 matrix transpose per half page.
#include <cooperative_groups.h>

#include "dd_common.cuh"


constexpr int ATTN_WARPS = 4;
constexpr int ATTN_THREADS = ATTN_WARPS * 32;
constexpr int ATTN_ROWS = 8;       // query rows per KV head the MMA shape carries
constexpr int ATTN_MAX_SPLITS = 64;
constexpr int ATTN_MAX_CLUSTER = 8;
constexpr int ATTN_OPAD = 9;       // row pitch (floats) of the per-warp O^T staging: conflict-free reads, 2-way writes

__device__ __forceinline__ uint32_t dd_movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

__device__ __forceinline__ uint32_t dd_pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// K rows gl and gl+8 of a page: channels [32kk + 8t, +8) for kk = 0..3
__device__ __forceinline__ void dd_load_k(const char* kp, int gl, int t, uint4 (&klo)[4], uint4 (&khi)[4]) {
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    klo[kk] = dd_ld_stream(kp + gl * DD_ROW_BYTES + (kk * 4 + t) * 16);
    khi[kk] = dd_ld_stream(kp + (gl + 8) * DD_ROW_BYTES + (kk * 4 + t) * 16);
  }
}

// V tokens 2t, 2t+1, 2t+8, 2t+9 of a page: channels [8gl, 8gl+8) and [64+8gl, 64+8gl+8)
__device__ __forceinline__ void dd_load_v(const char* vp, int gl, int t, uint4 (&v)[4][2]) {
#pragma unroll
  for (int tk = 0; tk < 4; ++tk) {
    const int tok = 2 * t + (tk & 1) + (tk >> 1) * 8;
#pragma unroll
    for (int c = 0; c < 2; ++c) v[tk][c] = dd_ld_stream(vp + tok * DD_ROW_BYTES + (c * 64 + gl * 8) * 2);
  }
}

__device__ __forceinline__ uint32_t dd_word(const uint4& v, int w) {
  return w == 0 ? v.x : (w == 1 ? v.y : (w == 2 ? v.z : v.w));
}

// Grid (n_splits, KV head, request), launched with thread-block clusters of `cluster` blocks along x
// (n_splits = cluster * n_groups). The blocks of a cluster merge through distributed shared memory;
// when a (request, KV head) has several clusters, each publishes a partial to global scratch and the
// last one to arrive merges them (arrival counter, no waiting).
__global__ void __launch_bounds__(ATTN_THREADS, 4) dd_attn_kernel(
    const __nv_bfloat16* __restrict__ q, const char* __restrict__ slot, const int* __restrict__ idx,
    const int* __restrict__ ctx_len, __nv_bfloat16* __restrict__ out, float* __restrict__ out_lse,
    float* __restrict__ part_o, float2* __restrict__ part_ml, unsigned int* __restrict__ ticket, int Hkv, int G, int Tq,
    int k, int n_splits, int pages_per_split, int cluster, const __nv_bfloat16* __restrict__ k_new,
    const __nv_bfloat16* __restrict__ v_new) {
  const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gl = lane >> 2, t = lane & 3;
  const int Hq = Hkv * G;
  const int n_rows = Tq * G;
  const size_t bg = (size_t)b * Hkv + g;

  __shared__ float sm_o[ATTN_WARPS][DD_D][ATTN_OPAD];   // per-warp O^T, [channel][row]
  __shared__ float2 sm_ml[ATTN_WARPS][ATTN_ROWS];
  __shared__ float sm_scale[ATTN_WARPS][ATTN_ROWS];
  // what the blocks of the cluster send each other: block r owns the channels [r*128/C, (r+1)*128/C) and receives
  // every block's partial of them, [source block][row][channel of the slice], plus every block's (max, sum)
  __shared__ float recv_o[ATTN_ROWS * DD_D];
  __shared__ float2 recv_ml[ATTN_MAX_CLUSTER][ATTN_ROWS];
  __shared__ float2 blk_ml[ATTN_ROWS];
  __shared__ int sm_last;

  dd_grid_dependency_wait();
  // arrives now, waits just before the first write into a peer's shared memory: by then every block has started
  if (cluster > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  // B operand of S^T: column n = gl is query row (token n / G, head g*G + n % G)
  uint4 qf[4];
  if (gl < n_rows) {
    const int tq = gl / G, hh = gl - tq * G;
    const uint4* qrow =
        reinterpret_cast<const uint4*>(q + (((size_t)b * Tq + tq) * Hq + g * G + hh) * DD_D);
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) qf[kk] = __ldg(qrow + kk * 4 + t);
  } else {
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) qf[kk] = make_uint4(0u, 0u, 0u, 0u);
  }

  const char* kbase = slot + bg * 2 * (size_t)k * DD_HALF_PAGE_BYTES;
  const char* vbase = kbase + (size_t)k * DD_HALF_PAGE_BYTES;
  const int* idx_bg = idx + bg * k;
  const int n_ctx = ctx_len[b];
  const float scale_log2 = rsqrtf((float)DD_D) * 1.4426950408889634f;

  float o[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY};   // columns n = 2t, 2t+1, log2 domain
  float l_run[2] = {0.f, 0.f};               // partial over this lane's tokens

  uint4 klo[4], khi[4], v[4][2];

  // S^T = K q^T for the page held in klo / khi, scaled to the log2 domain
  auto qk = [&](float (&acc)[4]) {
    acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      dd_mma_bf16(acc, klo[kk].x, khi[kk].x, klo[kk].y, khi[kk].y, qf[kk].x, qf[kk].y);
      dd_mma_bf16(acc, klo[kk].z, khi[kk].z, klo[kk].w, khi[kk].w, qf[kk].z, qf[kk].w);
    }
    // acc[0], acc[1]: token gl, columns 2t, 2t+1; acc[2], acc[3]: token gl+8
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] *= scale_log2;
  };
  // running soft-max per column, then O^T += V^T P^T with the page held in v
  auto softmax_pv = [&](float (&acc)[4]) {
    float alpha[2], pr[4];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      float pm = fmaxf(acc[c], acc[2 + c]);
      pm = fmaxf(pm, __shfl_xor_sync(0xffffffffu, pm, 4));
      pm = fmaxf(pm, __shfl_xor_sync(0xffffffffu, pm, 8));
      pm = fmaxf(pm, __shfl_xor_sync(0xffffffffu, pm, 16));
      const float mn = fmaxf(m_run[c], pm);
      if (mn == -INFINITY) {
        alpha[c] = 1.f; pr[c] = 0.f; pr[2 + c] = 0.f;
      } else {
        alpha[c] = exp2f(m_run[c] - mn);
        pr[c] = exp2f(acc[c] - mn);
        pr[2 + c] = exp2f(acc[2 + c] - mn);
      }
      l_run[c] = l_run[c] * alpha[c] + pr[c] + pr[2 + c];
      m_run[c] = mn;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      o[i][0] *= alpha[0]; o[i][1] *= alpha[1]; o[i][2] *= alpha[0]; o[i][3] *= alpha[1];
    }
    // P^T as the B operand: tokens {2t, 2t+1} and {2t+8, 2t+9} of column gl
    const uint32_t pb0 = dd_movmatrix_trans(dd_pack_bf16(pr[0], pr[1]));
    const uint32_t pb1 = dd_movmatrix_trans(dd_pack_bf16(pr[2], pr[3]));
    // MMA tile i has rows gl -> channel 8gl+i and gl+8 -> channel 64+8gl+i
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int w = i >> 1;
      const uint32_t sel = (i & 1) ? 0x7632u : 0x5410u;
      const uint32_t a0 = __byte_perm(dd_word(v[0][0], w), dd_word(v[1][0], w), sel);
      const uint32_t a1 = __byte_perm(dd_word(v[0][1], w), dd_word(v[1][1], w), sel);
      const uint32_t a2 = __byte_perm(dd_word(v[2][0], w), dd_word(v[3][0], w), sel);
      const uint32_t a3 = __byte_perm(dd_word(v[2][1], w), dd_word(v[3][1], w), sel);
      dd_mma_bf16(o[i], a0, a1, a2, a3, pb0, pb1);
    }
  };

  // ---- the step's own new KV entries (dual-token causal tail): one extra "page" whose tokens 0..Tq-1 are the
  // new entries; query token t sees the entries j <= t. Taken by the first warp of the first split.
  if (k_new != nullptr && split == 0 && warp == 0) {
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      klo[kk] = gl < Tq ? __ldg(reinterpret_cast<const uint4*>(k_new + (((size_t)b * Tq + gl) * Hkv + g) * DD_D) + kk * 4 + t)
                        : zero;
      khi[kk] = zero;
    }
#pragma unroll
    for (int tk = 0; tk < 4; ++tk) {
      const int tok = 2 * t + (tk & 1) + (tk >> 1) * 8;
#pragma unroll
      for (int c = 0; c < 2; ++c)
        v[tk][c] = tok < Tq ? __ldg(reinterpret_cast<const uint4*>(v_new + (((size_t)b * Tq + tok) * Hkv + g) * DD_D +
                                                                  c * 64 + gl * 8))
                            : zero;
    }
    float acc[4];
    qk(acc);
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const int n = 2 * t + c;                   // query row: token n / G
      const bool visible = gl < Tq && n < n_rows && gl <= n / G;
      if (!visible) acc[c] = -INFINITY;
      acc[2 + c] = -INFINITY;
    }
    softmax_pv(acc);
  }

  const int p_begin = split * pages_per_split;
  const int p_end = min(k, p_begin + pages_per_split);
  int j = p_begin + warp;
  int page = 0;
  if (j < p_end) {
    dd_load_k(kbase + (size_t)j * DD_HALF_PAGE_BYTES, gl, t, klo, khi);
    dd_load_v(vbase + (size_t)j * DD_HALF_PAGE_BYTES, gl, t, v);
    page = idx_bg[j];
  }
  while (j < p_end) {
    const int jn = j + ATTN_WARPS;
    const bool has_next = jn < p_end;
    float acc[4];
    qk(acc);
    // the K fragments are consumed: the next page's K goes into the same registers while this page finishes
    if (has_next) dd_load_k(kbase + (size_t)jn * DD_HALF_PAGE_BYTES, gl, t, klo, khi);
    const int page_next = has_next ? idx_bg[jn] : 0;
    if (page * DD_T + DD_T > n_ctx) {            // only the last page of a request can be partial
      if (page * DD_T + gl >= n_ctx) acc[0] = acc[1] = -INFINITY;
      if (page * DD_T + gl + 8 >= n_ctx) acc[2] = acc[3] = -INFINITY;
    }
    softmax_pv(acc);
    if (has_next) dd_load_v(vbase + (size_t)jn * DD_HALF_PAGE_BYTES, gl, t, v);
    page = page_next;
    j = jn;
  }
  // l over the 8 row groups of the warp
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    l_run[c] += __shfl_xor_sync(0xffffffffu, l_run[c], 4);
    l_run[c] += __shfl_xor_sync(0xffffffffu, l_run[c], 8);
    l_run[c] += __shfl_xor_sync(0xffffffffu, l_run[c], 16);
  }
  // ---- merge the warps of the block
  if (gl == 0) {
    sm_ml[warp][2 * t] = make_float2(m_run[0], l_run[0]);
    sm_ml[warp][2 * t + 1] = make_float2(m_run[1], l_run[1]);
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    sm_o[warp][8 * gl + i][2 * t] = o[i][0];
    sm_o[warp][8 * gl + i][2 * t + 1] = o[i][1];
    sm_o[warp][64 + 8 * gl + i][2 * t] = o[i][2];
    sm_o[warp][64 + 8 * gl + i][2 * t + 1] = o[i][3];
  }
  __syncthreads();
  if (threadIdx.x < ATTN_ROWS) {
    const int n = threadIdx.x;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < ATTN_WARPS; ++w) M = fmaxf(M, sm_ml[w][n].x);
    float L = 0.f;
#pragma unroll
    for (int w = 0; w < ATTN_WARPS; ++w) {
      const float sc = (M == -INFINITY) ? 0.f : exp2f(sm_ml[w][n].x - M);
      sm_scale[w][n] = sc;
      L += sm_ml[w][n].y * sc;
    }
    blk_ml[n] = make_float2(M, L);
  }
  __syncthreads();
  const int d = threadIdx.x;                     // one channel per thread, all rows
  float ob[ATTN_ROWS];
#pragma unroll
  for (int n = 0; n < ATTN_ROWS; ++n) {
    float a = 0.f;
#pragma unroll
    for (int w = 0; w < ATTN_WARPS; ++w) a += sm_o[w][d][n] * sm_scale[w][n];
    ob[n] = a;
  }

  if (n_splits == 1) {
#pragma unroll
    for (int n = 0; n < ATTN_ROWS; ++n) {
      if (n < n_rows) {
        const int tq = n / G, hh = n - tq * G;
        const float2 ml = blk_ml[n];
        const size_t row = ((size_t)b * Tq + tq) * Hq + g * G + hh;
        out[row * DD_D + d] = __float2bfloat16_rn(ml.y > 0.f ? ob[n] / ml.y : 0.f);
        if (out_lse && d == 0) out_lse[row] = (ml.x + log2f(ml.y)) * 0.6931471805599453f;
      }
    }
    return;
  }

  const int n_groups = n_splits / cluster;       // clusters per (request, KV head)
  const int group = split / cluster;
  if (cluster > 1) {
    // ---- merge the blocks of the cluster through distributed shared memory. Every block sends the slice of its
    // partial that block r owns into r's receive buffer (remote stores, nobody waits for an answer), one cluster
    // barrier makes them visible, and every block reduces its slice from its own shared memory. Nothing remote is
    // touched after the barrier, so a block may leave as soon as it is done.
    namespace cg = cooperative_groups;
    cg::cluster_group cl = cg::this_cluster();
    const int rank = (int)cl.block_rank();
    const int ch = DD_D / cluster;               // channels per block
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");   // pairs with the arrive at the top
    {
      const int r = d / ch, dd = d - r * ch;
      float* dst = cl.map_shared_rank(recv_o, r) + (size_t)rank * ATTN_ROWS * ch + dd;
#pragma unroll
      for (int n = 0; n < ATTN_ROWS; ++n) dst[n * ch] = ob[n];
      if (d < ATTN_ROWS * cluster) {
        const int rr = d / ATTN_ROWS, n = d - rr * ATTN_ROWS;
        *cl.map_shared_rank(&recv_ml[rank][n], rr) = blk_ml[n];
      }
    }
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    for (int e = threadIdx.x; e < ATTN_ROWS * ch; e += ATTN_THREADS) {
      const int n = e / ch, dd = e - n * ch;
      float ms[ATTN_MAX_CLUSTER], ls[ATTN_MAX_CLUSTER], os[ATTN_MAX_CLUSTER];
      float M = -INFINITY;
#pragma unroll
      for (int r = 0; r < ATTN_MAX_CLUSTER; ++r) {
        if (r < cluster) {
          const float2 ml = recv_ml[r][n];
          ms[r] = ml.x; ls[r] = ml.y;
          os[r] = recv_o[(r * ATTN_ROWS + n) * ch + dd];
          M = fmaxf(M, ml.x);
        }
      }
      float L = 0.f, a = 0.f;
#pragma unroll
      for (int r = 0; r < ATTN_MAX_CLUSTER; ++r) {
        if (r < cluster) {
          const float sc = (ms[r] == -INFINITY) ? 0.f : exp2f(ms[r] - M);
          L += ls[r] * sc;
          a += os[r] * sc;
        }
      }
      const int dg = rank * ch + dd;             // channel of the head
      if (n_groups == 1) {
        if (n < n_rows) {
          const int tq = n / G, hh = n - tq * G;
          const size_t row = ((size_t)b * Tq + tq) * Hq + g * G + hh;
          out[row * DD_D + dg] = __float2bfloat16_rn(L > 0.f ? a / L : 0.f);
          if (out_lse && dg == 0) out_lse[row] = (M + log2f(L)) * 0.6931471805599453f;
        }
      } else {
        part_o[((bg * n_groups + group) * ATTN_ROWS + n) * DD_D + dg] = a;
        if (dg == 0) part_ml[(bg * n_groups + group) * ATTN_ROWS + n] = make_float2(M, L);
      }
    }
    if (n_groups == 1) return;
    // several clusters per unit: the ticket below must follow every block's partial stores
    __threadfence();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (rank != 0) return;
  } else {
    // ---- one block per cluster: publish the block's partial directly
    float* po = part_o + ((bg * n_groups + group) * ATTN_ROWS) * DD_D;
#pragma unroll
    for (int n = 0; n < ATTN_ROWS; ++n) po[n * DD_D + d] = ob[n];
    if (d < ATTN_ROWS) part_ml[(bg * n_groups + group) * ATTN_ROWS + d] = blk_ml[d];
    __threadfence();
    __syncthreads();
  }

  // ---- several clusters: the last one to arrive merges the partials
  if (threadIdx.x == 0) {
    const unsigned prev = atomicAdd(&ticket[bg], 1u);
    sm_last = (prev == (unsigned)(n_groups - 1));
  }
  __syncthreads();
  if (!sm_last) return;
  __threadfence();
  if (threadIdx.x == 0) ticket[bg] = 0u;         // ready for the next launch
  // scale of every (group, row) and the row sums: warp w takes rows w and w+4, lanes take groups
  float2* sm_lm = &sm_ml[0][0];                  // reused: [row] -> (max, sum)
  float* sm_sc = &sm_o[0][0][0];                 // reused: [group][row] scale, n_groups <= ATTN_MAX_SPLITS
  for (int n = warp; n < ATTN_ROWS; n += ATTN_WARPS) {
    const float2* pml = part_ml + bg * n_groups * ATTN_ROWS + n;
    float ms[ATTN_MAX_SPLITS / 32], ls[ATTN_MAX_SPLITS / 32];
    float M = -INFINITY;
#pragma unroll
    for (int i = 0; i < ATTN_MAX_SPLITS / 32; ++i) {
      const int sp = lane + 32 * i;
      ms[i] = sp < n_groups ? __ldcg(&pml[sp * ATTN_ROWS].x) : -INFINITY;
      ls[i] = sp < n_groups ? __ldcg(&pml[sp * ATTN_ROWS].y) : 0.f;
      M = fmaxf(M, ms[i]);
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
    float L = 0.f;
#pragma unroll
    for (int i = 0; i < ATTN_MAX_SPLITS / 32; ++i) {
      const int sp = lane + 32 * i;
      const float sc = (ms[i] == -INFINITY) ? 0.f : exp2f(ms[i] - M);
      if (sp < n_groups) sm_sc[sp * ATTN_ROWS + n] = sc;
      L += ls[i] * sc;
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) L += __shfl_xor_sync(0xffffffffu, L, off);
    if (lane == 0) sm_lm[n] = make_float2(M, L);
  }
  __syncthreads();
  // every thread owns one channel of all rows; the loads of a group are independent of each other
  float a[ATTN_ROWS];
#pragma unroll
  for (int n = 0; n < ATTN_ROWS; ++n) a[n] = 0.f;
  const float* po = part_o + bg * n_groups * ATTN_ROWS * DD_D + d;
#pragma unroll 4
  for (int sp = 0; sp < n_groups; ++sp) {
#pragma unroll
    for (int n = 0; n < ATTN_ROWS; ++n) a[n] += __ldcg(po + (sp * ATTN_ROWS + n) * DD_D) * sm_sc[sp * ATTN_ROWS + n];
  }
#pragma unroll
  for (int n = 0; n < ATTN_ROWS; ++n) {
    if (n < n_rows) {
      const float2 ml = sm_lm[n];
      const int tq = n / G, hh = n - tq * G;
      const size_t row = ((size_t)b * Tq + tq) * Hq + g * G + hh;
      out[row * DD_D + d] = __float2bfloat16_rn(ml.y > 0.f ? a[n] / ml.y : 0.f);
      if (out_lse && d == 0) out_lse[row] = (ml.x + log2f(ml.y)) * 0.6931471805599453f;
    }
  }
}

// Launch with clusters of `cluster` blocks along x (1 = no cluster attribute needed).
static cudaError_t dd_attn_launch_raw(cudaStream_t st, int batch, int Hkv, int G, int Tq, int k, int n_splits,
                                      int cluster, const void* q, const char* slot, const int* idx, const int* ctx_len,
                                      void* out, float* out_lse, float* part_o, float2* part_ml, unsigned int* ticket,
                                      const void* k_new = nullptr, const void* v_new = nullptr) {
  const int pps = (k + n_splits - 1) / n_splits;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_splits, Hkv, batch);
  cfg.blockDim = dim3(ATTN_THREADS);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  dd_pdl_attr(&attr[0]);
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = cluster > 1 ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, dd_attn_kernel, (const __nv_bfloat16*)q, slot, idx, ctx_len, (__nv_bfloat16*)out,
                            out_lse, part_o, part_ml, ticket, Hkv, G, Tq, k, n_splits, pps, cluster,
                            (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new);
}

int dd_launch_attn(dd_ctx* ctx, const void* q, const char* slot, const int* idx, const int* ctx_len, void* out,
                   float* out_lse, cudaStream_t st, const void* k_new, const void* v_new) {
  const dd_config& c = ctx->cfg;
  if (ctx->attn_stream == 2)  // every slot of the ring has its tensor maps
    return dd_launch_attn_tc(ctx, q, (int)((size_t)(slot - ctx->ring) / ctx->slot_bytes), idx, ctx_len, out, out_lse, st,
                             k_new, v_new);
  if (ctx->attn_stream)
    return dd_launch_attn_stream(ctx, q, (int)((size_t)(slot - ctx->ring) / ctx->slot_bytes), idx, ctx_len, out, out_lse, st,
                                 k_new, v_new, false);
  DD_CUDA_TRY(ctx, dd_attn_launch_raw(st, c.batch, c.n_kv_heads, ctx->G, c.n_q_tokens, c.k_pages, ctx->attn_splits,
                                      ctx->attn_cluster, q, slot, idx, ctx_len, out, out_lse, ctx->attn_part_o,
                                      ctx->attn_part_ml, ctx->attn_ticket, k_new, v_new));
  return DD_OK;
}

// ------------------------------------------------------------------------------------------------
// Measurement aid: the attention kernel's loads and nothing else (same grid, same page walk, same fragment
// addresses, no arithmetic, no merge). Its duration is what the memory system delivers for this launch shape.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(ATTN_THREADS, 4) dd_attn_loads_only_kernel(const char* __restrict__ slot, int Hkv, int k,
                                                                             int pages_per_split,
                                                                             unsigned int* __restrict__ sink) {
  const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gl = lane >> 2, t = lane & 3;
  const size_t bg = (size_t)b * Hkv + g;
  const char* kbase = slot + bg * 2 * (size_t)k * DD_HALF_PAGE_BYTES;
  const char* vbase = kbase + (size_t)k * DD_HALF_PAGE_BYTES;
  const int p_begin = split * pages_per_split;
  const int p_end = min(k, p_begin + pages_per_split);
  dd_grid_dependency_wait();
  unsigned int acc = 0;
  for (int j = p_begin + warp; j < p_end; j += ATTN_WARPS) {
    uint4 klo[4], khi[4], v[4][2];
    dd_load_k(kbase + (size_t)j * DD_HALF_PAGE_BYTES, gl, t, klo, khi);
    dd_load_v(vbase + (size_t)j * DD_HALF_PAGE_BYTES, gl, t, v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc ^= klo[i].x ^ klo[i].y ^ klo[i].z ^ klo[i].w ^ khi[i].x ^ khi[i].y ^ khi[i].z ^ khi[i].w;
      acc ^= v[i][0].x ^ v[i][0].y ^ v[i][0].z ^ v[i][0].w ^ v[i][1].x ^ v[i][1].y ^ v[i][1].z ^ v[i][1].w;
    }
  }
  if (acc == 0x9E3779B9u) sink[0] = acc;        // keeps the loads alive; practically never true
}

int dd_launch_attn_loads_only(dd_ctx* ctx, const char* slot, cudaStream_t st) {
  const dd_config& c = ctx->cfg;
  if (ctx->attn_stream == 1)
    return dd_launch_attn_stream(ctx, nullptr, (int)((size_t)(slot - ctx->ring) / ctx->slot_bytes), nullptr, nullptr, nullptr,
                                 nullptr, st, nullptr, nullptr, true);
  const int S = ctx->attn_splits;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(S, c.n_kv_heads, c.batch);
  cfg.blockDim = dim3(ATTN_THREADS);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  dd_pdl_attr(&attr[0]);                         // launched the way the kernel it stands in for is
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  DD_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, dd_attn_loads_only_kernel, slot, c.n_kv_heads, c.k_pages, (c.k_pages + S - 1) / S,
                                      ctx->attn_ticket + c.batch * c.n_kv_heads));
  return DD_OK;
}

// ------------------------------------------------------------------------------------------------
// Allocation-free variant of the attention entry point.
//
// Some callers must not allocate device memory: code running between other libraries' memory pools,
// a plug-in that was handed every byte it may touch, a process that has already given the whole GPU
// to an arena allocator, or a latency-critical loop where an allocation (which can synchronise the
// device) is not acceptable. A dd_ctx cannot serve them, because dd_create allocates the split-merge
// scratch. This entry point keeps that scratch in a fixed array inside the library image instead.
//
// The array's name below is only a host-side handle in host code: passing it to a kernel would hand
// the kernel a host address. Its device address is looked up once per device with
// cudaGetSymbolAddress (by the first call on that device) and that address is what the kernel gets.
// ------------------------------------------------------------------------------------------------
#include <mutex>

constexpr size_t DD_STATIC_SCRATCH_BYTES = (size_t)8 << 20;   // held by every GPU that loads the library
static __device__ __align__(256) unsigned char dd_static_scratch[DD_STATIC_SCRATCH_BYTES];

constexpr int DD_STATIC_MAX_DEVICES = 64;
static unsigned char* g_static_scratch_addr[DD_STATIC_MAX_DEVICES];   // device address per device, 0 = not set up
static std::mutex g_static_scratch_mutex;

static size_t dd_static_need(int batch, int n_kv_heads, int n_splits, size_t* off_ml, size_t* off_ticket) {
  const size_t bg = (size_t)batch * n_kv_heads;
  const size_t part_o = (bg * n_splits * ATTN_ROWS * DD_D * sizeof(float) + 255) & ~(size_t)255;
  const size_t part_ml = (bg * n_splits * ATTN_ROWS * sizeof(float2) + 255) & ~(size_t)255;
  const size_t ticket = (bg * sizeof(unsigned int) + 255) & ~(size_t)255;
  if (off_ml) *off_ml = part_o;
  if (off_ticket) *off_ticket = part_o + part_ml;
  return part_o + part_ml + ticket;
}

extern "C" size_t dd_static_scratch_capacity(void) { return DD_STATIC_SCRATCH_BYTES; }

// Host-side pointer check of the context-free entry point: device (or managed) memory of the current device,
// aligned for its element type. cudaPointerGetAttributes allocates nothing.
static int dd_static_check_dev(const void* p, const char* what, int align, int dev) {
  if (((uintptr_t)p) & (uintptr_t)(align - 1))
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_static: %s is not %d-byte aligned", what, align);
  cudaPointerAttributes a;
  const cudaError_t e = cudaPointerGetAttributes(&a, p);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_static: %s: %s", what, cudaGetErrorString(e));
  }
  if (a.type != cudaMemoryTypeDevice && a.type != cudaMemoryTypeManaged)
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_static: %s is not device memory", what);
  if (a.type == cudaMemoryTypeDevice && a.device != dev)
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_static: %s lives on device %d, the current device is %d",
                   what, a.device, dev);
  return DD_OK;
}

extern "C" int dd_sparse_decode_attn_static(int batch, int n_q_heads, int n_kv_heads, int head_dim, int page_tokens,
                                            int k_pages, int n_q_tokens, int n_splits, const void* q,
                                            const void* slot, const int* idx, const int* ctx_len, void* out,
                                            float* out_lse, void* stream) {
  if (head_dim != DD_D || page_tokens != DD_T)
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_static: head_dim must be 128 and page_tokens 16");
  if (batch < 1 || n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads || k_pages < 1 || n_q_tokens < 1 ||
      n_q_tokens > 2 || n_q_tokens * (n_q_heads / n_kv_heads) > ATTN_ROWS)
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_static: unsupported geometry");
  if (n_splits < 1 || n_splits > k_pages || n_splits > ATTN_MAX_SPLITS)
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_static: need 1 <= n_splits <= min(k_pages, 64)");
  if (!q || !slot || !idx || !ctx_len || !out)
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_static: NULL tensor");
  if ((((uintptr_t)q) | ((uintptr_t)slot) | ((uintptr_t)out)) & 15)
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_static: bf16 tensors must be 16-byte aligned");
  size_t off_ml = 0, off_ticket = 0;
  const size_t need = dd_static_need(batch, n_kv_heads, n_splits, &off_ml, &off_ticket);
  if (need > DD_STATIC_SCRATCH_BYTES)
    return dd_fail(nullptr, DD_ERR_INVALID_ARG,
                   "dd_sparse_decode_attn_static: batch %d x kv heads %d x splits %d needs %zu bytes of scratch, the "
                   "built-in array holds %zu; use fewer splits or a dd_ctx",
                   batch, n_kv_heads, n_splits, need, (size_t)DD_STATIC_SCRATCH_BYTES);
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return dd_fail(nullptr, DD_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= DD_STATIC_MAX_DEVICES)
    return dd_fail(nullptr, DD_ERR_INVALID_ARG, "dd_sparse_decode_attn_static: device ordinal %d not supported", dev);
  {
    int rc;
    if ((rc = dd_static_check_dev(q, "q", 16, dev)) != DD_OK) return rc;
    if ((rc = dd_static_check_dev(slot, "slot", 16, dev)) != DD_OK) return rc;
    if ((rc = dd_static_check_dev(idx, "idx", 4, dev)) != DD_OK) return rc;
    if ((rc = dd_static_check_dev(ctx_len, "ctx_len", 4, dev)) != DD_OK) return rc;
    if ((rc = dd_static_check_dev(out, "out", 16, dev)) != DD_OK) return rc;
    if (out_lse && (rc = dd_static_check_dev(out_lse, "out_lse", 4, dev)) != DD_OK) return rc;
  }
  unsigned char* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_addr[dev]) {
      // once per device, with that device current: the device address of this device's copy of the array
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, dd_static_scratch);
      if (e != cudaSuccess || !p)
        return dd_fail(nullptr, DD_ERR_CUDA, "cudaGetSymbolAddress(dd_static_scratch): %s", cudaGetErrorString(e));
      g_static_scratch_addr[dev] = (unsigned char*)p;
    }
    base = g_static_scratch_addr[dev];
  }
  cudaStream_t st = (cudaStream_t)stream;
  unsigned int* ticket = (unsigned int*)(base + off_ticket);
  // the array keeps whatever the previous call (or an interrupted one) left: the arrival counters must start at zero
  e = cudaMemsetAsync(ticket, 0, (size_t)batch * n_kv_heads * sizeof(unsigned int), st);
  if (e != cudaSuccess) return dd_fail(nullptr, DD_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
  e = dd_attn_launch_raw(st, batch, n_kv_heads, n_q_heads / n_kv_heads, n_q_tokens, k_pages, n_splits, 1, q,
                         (const char*)slot, idx, ctx_len, out, out_lse, (float*)base, (float2*)(base + off_ml), ticket);
  if (e != cudaSuccess) return dd_fail(nullptr, DD_ERR_CUDA, "dd_attn_kernel launch: %s", cudaGetErrorString(e));
  return DD_OK;
}
