// Landmark build (set-up), page scoring and per-KV-head top-k selection.
//
// Scoring streams the landmarks of a layer once from HBM: the 16 landmarks of a tile are the M rows
// of a warp-level bf16 MMA, the G query heads that share the KV head are its N columns. The top-k
// kernel turns the per-head logits into log-probabilities with the per-head log-sum-exp, takes the
// group maximum, and finds the k-th largest by an MSB-first radix select on order-preserving keys,
// followed by an ordered compaction that emits ascending page numbers.
#include <cooperative_groups.h>

#include "dd_common.cuh"

// ------------------------------------------------------------------------------------------------
// Landmarks: mean of the valid keys of a chunk (a page, or 1/R of a page), fp32 sum in token order, fp32
// divide, RNE to bf16. One warp per chunk; a lane owns 4 consecutive channels.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) dd_landmark_kernel(const __nv_bfloat16* __restrict__ kv,
                                                          const int* __restrict__ ctx_len,
                                                          __nv_bfloat16* __restrict__ lm, int Hkv, int P, int R,
                                                          long long n_chunks_total) {
  const int lane = threadIdx.x & 31;
  const int c = DD_T / R;                        // tokens per chunk
  long long chunk = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long stride = (long long)gridDim.x * (blockDim.x >> 5);
  for (; chunk < n_chunks_total; chunk += stride) {
    const long long page = chunk / R;
    const int r = (int)(chunk - page * R);
    const int p = (int)(page % P);
    const int b = (int)(page / ((long long)P * Hkv));
    int cnt = ctx_len[b] - (p * DD_T + r * c);
    cnt = cnt > c ? c : cnt;
    const __nv_bfloat16* src = kv + page * (2 * DD_T * DD_D) + (size_t)r * c * DD_D + lane * 4;   // K half comes first
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    for (int i = 0; i < cnt; ++i) {
      uint2 w = *reinterpret_cast<const uint2*>(src + i * DD_D);
      __nv_bfloat162 lo = *reinterpret_cast<__nv_bfloat162*>(&w.x);
      __nv_bfloat162 hi = *reinterpret_cast<__nv_bfloat162*>(&w.y);
      a0 = __fadd_rn(a0, __low2float(lo));
      a1 = __fadd_rn(a1, __high2float(lo));
      a2 = __fadd_rn(a2, __low2float(hi));
      a3 = __fadd_rn(a3, __high2float(hi));
    }
    uint2 o = make_uint2(0u, 0u);
    if (cnt > 0) {
      const float n = (float)cnt;
      __nv_bfloat162 lo = __floats2bfloat162_rn(__fdiv_rn(a0, n), __fdiv_rn(a1, n));
      __nv_bfloat162 hi = __floats2bfloat162_rn(__fdiv_rn(a2, n), __fdiv_rn(a3, n));
      o.x = *reinterpret_cast<uint32_t*>(&lo);
      o.y = *reinterpret_cast<uint32_t*>(&hi);
    }
    *reinterpret_cast<uint2*>(lm + chunk * DD_D + lane * 4) = o;
  }
}

int dd_launch_build_landmarks(dd_ctx* ctx, const void* kv_dev, const int* ctx_len, void* landmarks, cudaStream_t st) {
  const dd_config& c = ctx->cfg;
  const long long total = (long long)c.batch * c.n_kv_heads * c.max_pages * ctx->R;
  const int warps_per_block = 8;
  long long blocks = (total + warps_per_block - 1) / warps_per_block;
  const long long cap = (long long)ctx->sm_count * 16;
  if (blocks > cap) blocks = cap;
  dd_landmark_kernel<<<(unsigned)blocks, warps_per_block * 32, 0, st>>>(
      (const __nv_bfloat16*)kv_dev, ctx_len, (__nv_bfloat16*)landmarks, c.n_kv_heads, c.max_pages, ctx->R, total);
  DD_CUDA_TRY(ctx, cudaGetLastError());
  return DD_OK;
}

// ------------------------------------------------------------------------------------------------
// Scoring. Grid (tile, KV head, request); 4 warps; each warp scores two 16-page MMA tiles.
//
// Fragment trick: the dot product does not care in which order the 128 channels are summed, so a
// thread feeds the MMA's k-slots {2t, 2t+1, 2t+8, 2t+9} of two consecutive k-steps with the eight
// consecutive channels [32*kk + 8t, 32*kk + 8t + 8) of its row — one 16-byte load — and the query
// fragment uses the same assignment. The four threads of a row then read 64 contiguous bytes.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) dd_score_kernel(const __nv_bfloat16* __restrict__ q, int q_req_stride,
                                                       int q_token_off, const __nv_bfloat16* __restrict__ lm,
                                                       const int* __restrict__ n_pages, float* __restrict__ s_out,
                                                       float2* __restrict__ part, int P, int G, int Hkv,
                                                       int n_tiles) {
  const int tile = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gl = lane >> 2, t = lane & 3;
  const int Hq = Hkv * G;
  int np = n_pages[b];
  np = np > P ? P : np;
  const int p_base = tile * DD_SCORE_TILE;

  __shared__ float2 red[4][8];

  float m_run[2] = {-INFINITY, -INFINITY};   // heads 2t, 2t+1
  float l_run[2] = {0.f, 0.f};

  if (p_base < np) {
    // query fragments: column n = gl is head g*G + gl
    uint4 qf[4];
    if (gl < G) {
      const uint4* qrow = reinterpret_cast<const uint4*>(q + (size_t)b * q_req_stride + q_token_off +
                                                         (size_t)(g * G + gl) * DD_D);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) qf[kk] = __ldg(qrow + kk * 4 + t);
    } else {
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) qf[kk] = make_uint4(0u, 0u, 0u, 0u);
    }
    const __nv_bfloat16* lm_bg = lm + (size_t)(b * Hkv + g) * P * DD_D;
    uint4 lo[2][4], hi[2][4];
    int prow[2][2];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      const int p0 = p_base + (warp * 2 + mt) * 16;
      prow[mt][0] = p0 + gl;
      prow[mt][1] = p0 + gl + 8;
      const int pa = prow[mt][0] < P ? prow[mt][0] : P - 1;   // stay inside the tensor; result discarded
      const int pb = prow[mt][1] < P ? prow[mt][1] : P - 1;
      const uint4* ra = reinterpret_cast<const uint4*>(lm_bg + (size_t)pa * DD_D);
      const uint4* rb = reinterpret_cast<const uint4*>(lm_bg + (size_t)pb * DD_D);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        lo[mt][kk] = dd_ld_stream(ra + kk * 4 + t);
        hi[mt][kk] = dd_ld_stream(rb + kk * 4 + t);
      }
    }
    const float scale = rsqrtf((float)DD_D);
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        dd_mma_bf16(acc, lo[mt][kk].x, hi[mt][kk].x, lo[mt][kk].y, hi[mt][kk].y, qf[kk].x, qf[kk].y);
        dd_mma_bf16(acc, lo[mt][kk].z, hi[mt][kk].z, lo[mt][kk].w, hi[mt][kk].w, qf[kk].z, qf[kk].w);
      }
      // acc[0], acc[1]: page prow[mt][0], heads 2t, 2t+1; acc[2], acc[3]: page prow[mt][1]
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int p = prow[mt][r];
        if (p < np) {
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const int h = 2 * t + c;
            if (h < G) {
              const float v = acc[2 * r + c] * scale;
              s_out[((size_t)(b * Hkv + g) * P + p) * G + h] = v;
              const float mn = fmaxf(m_run[c], v);
              l_run[c] = l_run[c] * expf(m_run[c] - mn) + expf(v - mn);
              m_run[c] = mn;
            }
          }
        }
      }
    }
  }
  // reduce (m, l) over the 8 row groups of the warp, then over the 4 warps
#pragma unroll
  for (int c = 0; c < 2; ++c) {
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m_run[c], off);
      const float l2 = __shfl_xor_sync(0xffffffffu, l_run[c], off);
      dd_ml_merge(m_run[c], l_run[c], m2, l2, false);
    }
  }
  if (gl == 0) {
    red[warp][2 * t] = make_float2(m_run[0], l_run[0]);
    red[warp][2 * t + 1] = make_float2(m_run[1], l_run[1]);
  }
  __syncthreads();
  if (threadIdx.x < G) {
    float m = red[0][threadIdx.x].x, l = red[0][threadIdx.x].y;
#pragma unroll
    for (int w = 1; w < 4; ++w) dd_ml_merge(m, l, red[w][threadIdx.x].x, red[w][threadIdx.x].y, false);
    part[((size_t)b * Hq + g * G + threadIdx.x) * n_tiles + tile] = make_float2(m, l);
  }
}

// ------------------------------------------------------------------------------------------------
// Top-k of one (request, KV head) per thread block.
// ------------------------------------------------------------------------------------------------
constexpr int TOPK_THREADS = 1024;
constexpr int TOPK_SMEM_KEYS = 16384;          // requests up to this many pages keep their keys in shared memory
constexpr int RADIX_BITS = 11;
constexpr int RADIX_BINS = 1 << RADIX_BITS;

// fp32 -> uint32 with the same order
__device__ __forceinline__ uint32_t dd_orderable(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive prefix sum over the 1024 threads of the block; `total` is returned to every thread.
__device__ __forceinline__ unsigned dd_block_scan_excl(unsigned v, unsigned* warp_tot, unsigned& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned inc = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned n = __shfl_up_sync(0xffffffffu, inc, off);
    if (lane >= off) inc += n;
  }
  __syncthreads();                               // warp_tot may still be read from the previous scan
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  unsigned wt = warp_tot[lane];                  // 32 warps
  unsigned winc = wt;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned n = __shfl_up_sync(0xffffffffu, winc, off);
    if (lane >= off) winc += n;
  }
  total = __shfl_sync(0xffffffffu, winc, 31);
  const unsigned wexcl = __shfl_sync(0xffffffffu, winc - wt, warp);
  return wexcl + inc - v;
}

__global__ void __launch_bounds__(TOPK_THREADS) dd_topk_kernel(
    const float* __restrict__ s, const float2* __restrict__ part, const int* __restrict__ n_pages,
    uint32_t* __restrict__ gkeys, int* __restrict__ out_idx, float* __restrict__ out_scores, int P, int G, int Hkv,
    int n_tiles, int k, int forced, int* err_word) {
  extern __shared__ uint32_t smem_keys[];
  __shared__ unsigned hist[RADIX_BINS];
  __shared__ unsigned warp_tot[32];
  __shared__ float lse_s[8];
  __shared__ unsigned sh_min, sh_max, sh_bin, sh_above;

  const int g = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Hq = Hkv * G;
  const size_t bg = (size_t)b * Hkv + g;
  int np = n_pages[b];
  if (np > P || np < k) {
    if (tid == 0) dd_report(err_word, DD_ERR_INDEX_RANGE, np);
    np = np > P ? P : (np < 0 ? 0 : np);
  }
  const int k_eff = k < np ? k : np;
  const int forced_eff = forced < k_eff ? forced : k_eff;
  const int n_free = np - forced_eff;            // pages [n_free, np) are forced
  const int k_free = k_eff - forced_eff;
  int* out = out_idx + bg * k;
  if (tid == 0) { sh_min = 0xFFFFFFFFu; sh_max = 0u; }

  // 1. log-sum-exp of every head of the group from the per-tile partials
  if (warp < G) {
    const int tiles = (np + DD_SCORE_TILE - 1) / DD_SCORE_TILE;
    const float2* pp = part + ((size_t)b * Hq + g * G + warp) * n_tiles;
    float m = -INFINITY, l = 0.f;
    for (int i = lane; i < tiles; i += 32) {
      const float2 v = pp[i];
      dd_ml_merge(m, l, v.x, v.y, false);
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
      const float l2 = __shfl_xor_sync(0xffffffffu, l, off);
      dd_ml_merge(m, l, m2, l2, false);
    }
    if (lane == 0) lse_s[warp] = m + logf(l);
  }
  __syncthreads();

  // 2. keys: group maximum of the log-probabilities, order-preserving integer form
  uint32_t* keys = (np <= TOPK_SMEM_KEYS) ? smem_keys : gkeys + bg * P;
  {
    float lse[8];
#pragma unroll
    for (int h = 0; h < 8; ++h) lse[h] = h < G ? lse_s[h] : 0.f;
    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
    const float* sp = s + bg * (size_t)P * G;
    for (int p = tid; p < np; p += TOPK_THREADS) {
      float c = -INFINITY;
#pragma unroll
      for (int h = 0; h < 8; ++h)
        if (h < G) c = fmaxf(c, sp[(size_t)p * G + h] - lse[h]);
      if (out_scores) out_scores[bg * P + p] = expf(c);
      uint32_t key = dd_orderable(c);
      if (p >= n_free) key = 0xFFFFFFFFu;
      else { kmin = min(kmin, key); kmax = max(kmax, key); }
      keys[p] = key;
    }
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) { atomicMin(&sh_min, kmin); atomicMax(&sh_max, kmax); }
  }
  __syncthreads();

  // 3. radix select of the k_free-th largest key among the non-forced pages
  uint32_t thr = 0xFFFFFFFFu;
  unsigned k_rem = 0;
  if (k_free > 0) {
    const uint32_t kmin = sh_min;
    const uint32_t range = sh_max - kmin;
    const int nbits = 32 - __clz(range);
    unsigned long long prefix = 0;
    k_rem = (unsigned)k_free;
    int hi = nbits;                              // unresolved bits of (key - min); digits are cut from the top
    while (hi > 0) {
      const int width = hi < RADIX_BITS ? hi : RADIX_BITS;
      const int shift = hi - width;
      for (int i = tid; i < RADIX_BINS; i += TOPK_THREADS) hist[i] = 0u;
      __syncthreads();
      for (int p = tid; p < n_free; p += TOPK_THREADS) {
        const unsigned long long rel = (unsigned long long)(keys[p] - kmin);
        if ((rel >> hi) == prefix) atomicAdd(&hist[(unsigned)(rel >> shift) & ((1u << width) - 1u)], 1u);
      }
      __syncthreads();
      // thread i owns bins 2047-2i and 2046-2i; scan from the top bin downwards
      const unsigned h_hi = hist[RADIX_BINS - 1 - 2 * tid], h_lo = hist[RADIX_BINS - 2 - 2 * tid];
      unsigned total;
      const unsigned above = dd_block_scan_excl(h_hi + h_lo, warp_tot, total);
      if (above < k_rem && k_rem <= above + h_hi + h_lo) {
        if (above + h_hi >= k_rem) { sh_bin = RADIX_BINS - 1 - 2 * tid; sh_above = above; }
        else { sh_bin = RADIX_BINS - 2 - 2 * tid; sh_above = above + h_hi; }
      }
      __syncthreads();
      prefix = (prefix << width) | sh_bin;
      k_rem -= sh_above;
      hi = shift;
      __syncthreads();
    }
    thr = kmin + (uint32_t)prefix;               // k_rem of the keys equal to thr are still to be taken
  }

  // 4. ordered compaction: ascending page numbers; equal keys are taken from the lowest page up
  unsigned base_gt = 0, base_eq = 0;
  for (int c0 = 0; c0 < np; c0 += TOPK_THREADS) {
    const int p = c0 + tid;
    unsigned gt = 0, eq = 0;
    if (p < np) {
      const uint32_t key = keys[p];
      if (p >= n_free || key > thr) gt = 1;
      else if (key == thr) eq = 1;
    }
    unsigned total;
    const unsigned ex = dd_block_scan_excl(gt | (eq << 16), warp_tot, total);
    const unsigned eq_before = base_eq + (ex >> 16);
    if (gt || (eq && eq_before < k_rem)) {
      const unsigned pos = base_gt + (ex & 0xFFFFu) + min(eq_before, k_rem);
      if (pos < (unsigned)k) out[pos] = p;
    }
    base_gt += total & 0xFFFFu;
    base_eq += total >> 16;
  }
  // precondition k <= n_pages violated: pad with the last valid page so that later stages stay in range
  for (int j = k_eff + tid; j < k; j += TOPK_THREADS) out[j] = np > 0 ? np - 1 : 0;
}

// ------------------------------------------------------------------------------------------------
// Fused selection: one thread-block cluster per (request, KV head).
//
// Block `rank` of the cluster scores the pages [rank*ppc, (rank+1)*ppc) and keeps their logits in its own
// shared memory; what the blocks must agree on is published in shared memory and read by the peers through
// distributed shared memory after a cluster barrier:
//   barrier 1   per-head (max, sum exp, min) of every block's logits  -> log-sum-exp of the request and a range
//               [lo, hi] that certainly holds every key (key = max over heads of logit - lse, so
//               max_h(min_h - lse_h) <= key <= max_h(max_h - lse_h)): no separate min / max exchange
//   barrier 2   per radix pass (11-bit digits cut from the top of key - lo), the sums of 8-bin groups; the 8 bins
//               of the group where the count crosses k are then read directly
//   barrier 3   the few keys that share the leading digits with the k-th largest, and how many local keys lie
//               above them -> every block ranks the candidates (the k-th largest key) and derives every other
//               block's contribution, i.e. its own output offset, without a further exchange
//   barrier 4   nobody leaves while a peer may still read its shared memory (arrive after the last remote read,
//               wait at the very end)
// Nothing but the landmarks is read from global memory, and nothing but the index set is written.
// ------------------------------------------------------------------------------------------------
namespace cg = cooperative_groups;

constexpr int SEL_THREADS = 256;
constexpr int SEL_WARPS = SEL_THREADS / 32;
constexpr int SEL_CAND_MAX = 256;          // keys sharing a radix prefix that are ranked directly
constexpr int SEL_MAX_SMEM = 200 * 1024;   // dynamic shared memory the fused kernel may be launched with
constexpr int SEL_MAX_CLUSTER = 16;

__device__ __forceinline__ void dd_cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void dd_cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void dd_cluster_sync() { dd_cluster_arrive(); dd_cluster_wait(); }

// Exclusive prefix sum over the 256 threads of the block; `total` is returned to every thread.
__device__ __forceinline__ unsigned dd_scan256_excl(unsigned v, unsigned* warp_tot, unsigned& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned inc = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned n = __shfl_up_sync(0xffffffffu, inc, off);
    if (lane >= off) inc += n;
  }
  __syncthreads();
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  const unsigned wt = lane < SEL_WARPS ? warp_tot[lane] : 0u;
  unsigned winc = wt;
#pragma unroll
  for (int off = 1; off < SEL_WARPS; off <<= 1) {
    const unsigned n = __shfl_up_sync(0xffffffffu, winc, off);
    if (lane >= off) winc += n;
  }
  total = __shfl_sync(0xffffffffu, winc, SEL_WARPS - 1);
  const unsigned wexcl = __shfl_sync(0xffffffffu, winc - wt, warp);
  return wexcl + inc - v;
}

// What a block publishes for its peers.
struct dd_sel_pub {
  float m[8], l[8];            // per head of the group: reference and sum of exp(s - reference) over this block's logits
  float mn[8], mx[8];          // smallest and largest logit
  unsigned above;              // local pages certainly selected: forced ones and keys above the candidates' digits
  unsigned eq;                 // local keys equal to the threshold when the digits resolve it exactly
  unsigned cand_n;             // local candidate keys listed in cand[]
  uint32_t cand[SEL_CAND_MAX];
};

// 16-byte asynchronous copy global -> shared memory (bypasses registers and L1), and its group bookkeeping.
__device__ __forceinline__ void dd_cp_async16(void* smem, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem) : "memory");
}
__device__ __forceinline__ void dd_cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void dd_cp_async_wait_pending(int n) {   // at most n groups still in flight (n <= 3)
  if (n >= 3) asm volatile("cp.async.wait_group 3;" ::: "memory");
  else if (n == 2) asm volatile("cp.async.wait_group 2;" ::: "memory");
  else if (n == 1) asm volatile("cp.async.wait_group 1;" ::: "memory");
  else asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// Fragments of one 16-row tile of landmarks: rows gl and gl + 8, channels [32kk + 8t, +8) for kk = 0..3.
struct dd_sel_frag {
  uint4 lo[4], hi[4];
};

__device__ __forceinline__ void dd_sel_load_tile(dd_sel_frag& f, const __nv_bfloat16* lm_bg, int row0, int row_max, int gl,
                                                 int t) {
  const int pa = min(row0 + gl, row_max);                 // stay inside the tensor; rows past the end are discarded later
  const int pb = min(row0 + gl + 8, row_max);
  const uint4* ra = reinterpret_cast<const uint4*>(lm_bg + (size_t)pa * DD_D);
  const uint4* rb = reinterpret_cast<const uint4*>(lm_bg + (size_t)pb * DD_D);
#pragma unroll
  for (int kk = 0; kk < 4; ++kk) {
    f.lo[kk] = dd_ld_stream(ra + kk * 4 + t);
    f.hi[kk] = dd_ld_stream(rb + kk * 4 + t);
  }
}

__global__ void __launch_bounds__(SEL_THREADS, 2) dd_select_fused_kernel(
    const __nv_bfloat16* __restrict__ q, int q_req_stride, int q_token_off, const __nv_bfloat16* __restrict__ lm,
    const int* __restrict__ n_pages, int* __restrict__ out_idx, float* __restrict__ out_scores, int P, int G, int Hkv,
    int k, int forced, int ppc, int* err_word, int R, const int* __restrict__ ctx_len, int ring_stages, float* __restrict__ s_glob) {
  extern __shared__ __align__(16) unsigned char sel_smem[];
  // logits [ppc * R][G] of this block's rows: in shared memory when they leave room for a deep ring, otherwise in
  // the context's global scratch (written and re-read by this block only; it stays in L2)
  float* s_sm = s_glob ? s_glob + ((size_t)(blockIdx.z * Hkv + blockIdx.y) * P + (size_t)blockIdx.x * ppc) * R * G
                       : reinterpret_cast<float*>(sel_smem);
  // the landmark ring of the scoring phase shares its memory with the keys and histograms of the later phases
  uint4* ring = reinterpret_cast<uint4*>(sel_smem + (s_glob ? 0 : (size_t)ppc * R * G * 4));   // [warp][stage][8][32] x 16 B
  uint32_t* keys = reinterpret_cast<uint32_t*>(ring);                                   // [ppc] key of every local page
  unsigned* hist = reinterpret_cast<unsigned*>(keys + ppc);                             // [2][RADIX_BINS]
  __shared__ dd_sel_pub pub;
  __shared__ unsigned grp[2][SEL_THREADS];
  __shared__ float red_m[SEL_WARPS][8], red_l[SEL_WARPS][8], red_mn[SEL_WARPS][8], red_mx[SEL_WARPS][8];
  __shared__ float pull_m[SEL_MAX_CLUSTER][8], pull_l[SEL_MAX_CLUSTER][8], pull_mn[SEL_MAX_CLUSTER][8], pull_mx[SEL_MAX_CLUSTER][8];
  __shared__ float lse_s[8], lo_s[8], hi_s[8];
  __shared__ unsigned warp_tot[SEL_WARPS];
  __shared__ unsigned warp_gt[SEL_WARPS], warp_eq[SEL_WARPS];
  __shared__ unsigned sh_above, sh_grp, sh_thr, sh_base_gt, sh_base_eq;
  __shared__ unsigned cnt8[8];
  __shared__ unsigned peer_above[SEL_MAX_CLUSTER], peer_eq[SEL_MAX_CLUSTER], peer_cand[SEL_MAX_CLUSTER];
  __shared__ uint32_t all_c[SEL_CAND_MAX];

  cg::cluster_group cl = cg::this_cluster();
  const int C = (int)cl.num_blocks();
  const int rank = (int)cl.block_rank();
  const int g = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int gl = lane >> 2, t = lane & 3;
  const size_t bg = (size_t)b * Hkv + g;
  dd_grid_dependency_wait();
  int np = n_pages[b];
  if (np > P || np < k) {
    if (tid == 0 && rank == 0) dd_report(err_word, DD_ERR_INDEX_RANGE, np);
    np = np > P ? P : (np < 0 ? 0 : np);
  }
  const int k_eff = k < np ? k : np;
  const int forced_eff = forced < k_eff ? forced : k_eff;
  const int n_free = np - forced_eff;            // pages [n_free, np) are forced
  const int k_free = k_eff - forced_eff;
  const int p_lo = rank * ppc;
  const int n_local = max(0, min(np, p_lo + ppc) - p_lo);
  // landmark rows (chunks) of this block: with R chunks per page only the chunks that hold a token exist
  int n_rows_req = np * R;
  if (R > 1) n_rows_req = min(n_rows_req, (ctx_len[b] + DD_T / R - 1) / (DD_T / R));
  const int n_local_rows = max(0, min(n_rows_req, (p_lo + ppc) * R) - p_lo * R);
  if (tid == 0) { pub.above = 0u; pub.eq = 0u; pub.cand_n = 0u; sh_base_gt = 0u; sh_base_eq = 0u; }

  // ---- A. logits of this block's rows, kept in shared memory. 16 landmarks are the M rows of a bf16 MMA, the G heads
  // its N columns (same fragment trick as dd_score_kernel). Every lane copies the fragments it will use itself with
  // 16-byte asynchronous copies into a private ring in shared memory (ring_stages tiles deep per warp), so that
  // several tiles per warp are in flight whatever the register allocation; no lane reads another lane's bytes.
  float m_run[2] = {-INFINITY, -INFINITY};       // heads 2t, 2t+1: reference of the running sum
  float l_run[2] = {0.f, 0.f};
  float mn_run[2] = {INFINITY, INFINITY}, mx_run[2] = {-INFINITY, -INFINITY};   // smallest and largest logit
  {
    uint4 qf[4];
    if (gl < G) {
      const uint4* qrow = reinterpret_cast<const uint4*>(q + (size_t)b * q_req_stride + q_token_off +
                                                         (size_t)(g * G + gl) * DD_D);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) qf[kk] = __ldg(qrow + kk * 4 + t);
    } else {
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) qf[kk] = make_uint4(0u, 0u, 0u, 0u);
    }
    const __nv_bfloat16* lm_bg = lm + bg * (size_t)P * R * DD_D;
    const float scale = rsqrtf((float)DD_D);
    const int row_lo = p_lo * R, row_max = P * R - 1;
    const int n_tiles = (n_local_rows + 15) >> 4;
    auto consume = [&](const dd_sel_frag& f, int tile) {
      // two independent accumulator chains halve the latency of the dependent MMAs
      float acc[4] = {0.f, 0.f, 0.f, 0.f}, acc2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        dd_mma_bf16(acc, f.lo[kk].x, f.hi[kk].x, f.lo[kk].y, f.hi[kk].y, qf[kk].x, qf[kk].y);
        dd_mma_bf16(acc2, f.lo[kk].z, f.hi[kk].z, f.lo[kk].w, f.hi[kk].w, qf[kk].z, qf[kk].w);
      }
      // acc[0], acc[1]: row gl, heads 2t, 2t+1; acc[2], acc[3]: row gl + 8
      const int r0 = tile * 16 + gl, r1 = r0 + 8;
      const bool ok0 = r0 < n_local_rows, ok1 = r1 < n_local_rows;
      if (G == 4) {
        // one 16-byte store per row instead of four 4-byte ones: lanes t = 0 and t = 1 of a row group swap halves,
        // t = 0 then holds all four heads of row gl, t = 1 those of row gl + 8
        const float a0 = (acc[0] + acc2[0]) * scale, a1 = (acc[1] + acc2[1]) * scale;      // row gl,     heads 2t, 2t+1
        const float b0 = (acc[2] + acc2[2]) * scale, b1 = (acc[3] + acc2[3]) * scale;      // row gl + 8, heads 2t, 2t+1
        const float x0 = __shfl_xor_sync(0xffffffffu, t == 0 ? b0 : a0, 1);
        const float x1 = __shfl_xor_sync(0xffffffffu, t == 0 ? b1 : a1, 1);
        if (t == 0 && ok0) *reinterpret_cast<float4*>(s_sm + (size_t)r0 * 4) = make_float4(a0, a1, x0, x1);
        if (t == 1 && ok1) *reinterpret_cast<float4*>(s_sm + (size_t)r1 * 4) = make_float4(x0, x1, b0, b1);
      }
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int h = 2 * t + c;
        if (h < G && ok0) {
          const float v0 = (acc[c] + acc2[c]) * scale;
          const float v1 = ok1 ? (acc[2 + c] + acc2[2 + c]) * scale : v0;
          if (G != 4) {
            s_sm[(size_t)r0 * G + h] = v0;
            if (ok1) s_sm[(size_t)r1 * G + h] = v1;
          }
          const float vmax = fmaxf(v0, v1);
          mx_run[c] = fmaxf(mx_run[c], vmax);
          mn_run[c] = fminf(mn_run[c], fminf(v0, v1));
          // running sum of exp(v - m_run): the reference m_run moves only when a value exceeds it by a wide margin
          // (any reference gives the same log-sum-exp as long as nothing overflows)
          if (vmax > m_run[c] + 40.f) {
            l_run[c] *= __expf(m_run[c] - vmax);
            m_run[c] = vmax;
          }
          l_run[c] += __expf(v0 - m_run[c]) + (ok1 ? __expf(v1 - m_run[c]) : 0.f);
        }
      }
    };
    uint4* my_ring = ring + (size_t)warp * ring_stages * 256 + lane;   // [stage][8][32] of this warp, this lane's column
    auto issue = [&](int tile, int slot) {                 // always commits a group, possibly an empty one
      if (tile < n_tiles) {
        const int pa = min(row_lo + tile * 16 + gl, row_max);   // stay inside the tensor; rows past the end are discarded
        const int pb = min(row_lo + tile * 16 + gl + 8, row_max);
        const uint4* ra = reinterpret_cast<const uint4*>(lm_bg + (size_t)pa * DD_D) + t;
        const uint4* rb = reinterpret_cast<const uint4*>(lm_bg + (size_t)pb * DD_D) + t;
        uint4* dst = my_ring + slot * 256;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          dd_cp_async16(dst + kk * 32, ra + kk * 4);
          dd_cp_async16(dst + (4 + kk) * 32, rb + kk * 4);
        }
      }
      dd_cp_async_commit();
    };
    const int ahead = ring_stages - 1;                     // tiles in flight per warp
    for (int s = 0; s < ahead; ++s) issue(warp + s * SEL_WARPS, s);
    int slot = 0, slot_issue = ahead;
    for (int tile = warp; tile < n_tiles; tile += SEL_WARPS) {
      issue(tile + ahead * SEL_WARPS, slot_issue);
      dd_cp_async_wait_pending(ahead);                     // the oldest group, this tile, has landed
      dd_sel_frag f;
      const uint4* src = my_ring + slot * 256;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        f.lo[kk] = src[kk * 32];
        f.hi[kk] = src[(4 + kk) * 32];
      }
      consume(f, tile);
      slot = slot + 1 == ring_stages ? 0 : slot + 1;
      slot_issue = slot_issue + 1 == ring_stages ? 0 : slot_issue + 1;
    }
    dd_cp_async_wait_pending(0);
  }
#pragma unroll
  for (int c = 0; c < 2; ++c) {
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m_run[c], off);
      const float l2 = __shfl_xor_sync(0xffffffffu, l_run[c], off);
      dd_ml_merge(m_run[c], l_run[c], m2, l2, false);
      mn_run[c] = fminf(mn_run[c], __shfl_xor_sync(0xffffffffu, mn_run[c], off));
      mx_run[c] = fmaxf(mx_run[c], __shfl_xor_sync(0xffffffffu, mx_run[c], off));
    }
  }
  if (gl == 0) {
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      red_m[warp][2 * t + c] = m_run[c];
      red_l[warp][2 * t + c] = l_run[c];
      red_mn[warp][2 * t + c] = mn_run[c];
      red_mx[warp][2 * t + c] = mx_run[c];
    }
  }
  __syncthreads();                               // every warp is done with its ring: the memory becomes keys + histograms
  for (int i = tid; i < 2 * RADIX_BINS; i += SEL_THREADS) hist[i] = 0u;
  if (tid < 8) {
    float m = red_m[0][tid], l = red_l[0][tid], mn = red_mn[0][tid], mx = red_mx[0][tid];
#pragma unroll
    for (int w = 1; w < SEL_WARPS; ++w) {
      dd_ml_merge(m, l, red_m[w][tid], red_l[w][tid], false);
      mn = fminf(mn, red_mn[w][tid]);
      mx = fmaxf(mx, red_mx[w][tid]);
    }
    pub.m[tid] = m;
    pub.l[tid] = l;
    pub.mn[tid] = mn;
    pub.mx[tid] = mx;
  }
  // ---- B. log-sum-exp of the whole request and the key range, from every block's partials
  dd_cluster_sync();
  if (tid < C * 8) {                             // one thread per (peer, head): all remote reads are in flight at once
    const int r = tid >> 3, h = tid & 7;
    const dd_sel_pub* pr = cl.map_shared_rank(&pub, r);
    pull_m[r][h] = pr->m[h];
    pull_l[r][h] = pr->l[h];
    pull_mn[r][h] = pr->mn[h];
    pull_mx[r][h] = pr->mx[h];
  }
  __syncthreads();
  if (tid < G) {
    float m = -INFINITY, l = 0.f, mn = INFINITY, mx = -INFINITY;
    for (int r = 0; r < C; ++r) {
      dd_ml_merge(m, l, pull_m[r][tid], pull_l[r][tid], false);
      mn = fminf(mn, pull_mn[r][tid]);
      mx = fmaxf(mx, pull_mx[r][tid]);
    }
    const float lse = m + logf(l);
    lse_s[tid] = lse;
    lo_s[tid] = mn - lse;
    hi_s[tid] = mx - lse;
  }
  __syncthreads();
  // ---- C. keys: group maximum of the log-probabilities (a page takes the best of its existing chunks) in
  // order-preserving integer form, and the first histogram over the leading digits of key - lo
  uint32_t klo, khi;
  {
    float lo = -INFINITY, hi = -INFINITY;
    for (int h = 0; h < G; ++h) { lo = fmaxf(lo, lo_s[h]); hi = fmaxf(hi, hi_s[h]); }
    klo = dd_orderable(lo);
    khi = dd_orderable(hi);
  }
  const int n_free_local = max(0, min(n_free, p_lo + ppc) - p_lo);     // local pages that take part in the select
  const int nbits = khi > klo ? 32 - __clz(khi - klo) : 0;
  int hi_bits = nbits;                           // bits of (key - lo) not resolved yet; digits are cut from the top
  {
    float lse[8];
#pragma unroll
    for (int h = 0; h < 8; ++h) lse[h] = h < G ? lse_s[h] : 0.f;
    const int width = hi_bits < RADIX_BITS ? hi_bits : RADIX_BITS;
    const int shift = hi_bits - width;
    auto finish = [&](int pl, float c) {
      const int p = p_lo + pl;
      if (out_scores) out_scores[bg * P + p] = expf(c);
      uint32_t key = dd_orderable(c);
      key = key < klo ? klo : (key > khi ? khi : key);                  // the range holds every key; keep the digits safe
      if (p >= n_free) key = 0xFFFFFFFFu;
      else if (width > 0) atomicAdd(&hist[(key - klo) >> shift], 1u);
      keys[pl] = key;
    };
    if (G == 4 && R == 1) {
      // the common shape: one 16-byte read per page, four pages per thread in flight (the logits may sit in L2)
      for (int base = tid; base < n_local; base += 4 * SEL_THREADS) {
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int pl = base + u * SEL_THREADS;
          v[u] = pl < n_local ? *reinterpret_cast<const float4*>(s_sm + (size_t)pl * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int pl = base + u * SEL_THREADS;
          if (pl < n_local)
            finish(pl, fmaxf(fmaxf(v[u].x - lse[0], v[u].y - lse[1]), fmaxf(v[u].z - lse[2], v[u].w - lse[3])));
        }
      }
    } else {
      for (int pl = tid; pl < n_local; pl += SEL_THREADS) {
        float c = -INFINITY;
        for (int r = 0; r < R; ++r) {
          if (pl * R + r < n_local_rows) {
#pragma unroll
            for (int h = 0; h < 8; ++h)
              if (h < G) c = fmaxf(c, s_sm[((size_t)pl * R + r) * G + h] - lse[h]);
          }
        }
        finish(pl, c);
      }
    }
  }

  // ---- D. the k_free-th largest key. MSB-first radix passes on (key - lo); a pass exchanges only the sums of 8-bin
  // groups and reads the 8 bins of the group where the count crosses k. It ends when the digits are exhausted or
  // the crossing bin holds few keys.
  unsigned long long prefix = 0;
  unsigned k_rem = (unsigned)k_free;
  int shift = hi_bits;                           // bits below the resolved prefix
  unsigned above_acc = 0;                        // this thread's share of the local keys above the chosen bins
  unsigned eq_local = (unsigned)n_free_local;    // local keys equal to the threshold when the digits resolve it exactly
  if (k_free > 0) {
    for (int pass = 0; shift > 0; ++pass) {
      const int width = shift < RADIX_BITS ? shift : RADIX_BITS;
      const int nshift = shift - width;
      unsigned* h = hist + (pass & 1) * RADIX_BINS;                     // double-buffered: peers may still read the other
      unsigned* gp = grp[pass & 1];
      if (pass > 0) {
        for (int i = tid; i < RADIX_BINS; i += SEL_THREADS) h[i] = 0u;
        __syncthreads();
        for (int pl = tid; pl < n_free_local; pl += SEL_THREADS) {
          const unsigned long long rel = (unsigned long long)(keys[pl] - klo);
          if ((rel >> shift) == prefix) atomicAdd(&h[(unsigned)(rel >> nshift) & ((1u << width) - 1u)], 1u);
        }
      }
      __syncthreads();
      {                                           // thread i owns the 8 bins [2047-8i-7, 2047-8i]
        unsigned sum8 = 0;
#pragma unroll
        for (int jb = 0; jb < 8; ++jb) sum8 += h[RADIX_BINS - 1 - 8 * tid - jb];
        gp[tid] = sum8;
      }
      dd_cluster_sync();
      unsigned tot = 0;
      for (int r = 0; r < C; ++r) tot += cl.map_shared_rank(gp, r)[tid];
      unsigned total;
      const unsigned above = dd_scan256_excl(tot, warp_tot, total);      // groups are scanned from the top bin down
      if (above < k_rem && k_rem <= above + tot) { sh_grp = (unsigned)tid; sh_above = above; }
      __syncthreads();
      const int gsel = (int)sh_grp;
      if (tid < 8) {
        unsigned c8 = 0;
        for (int r = 0; r < C; ++r) c8 += cl.map_shared_rank(h, r)[RADIX_BINS - 1 - 8 * gsel - tid];
        cnt8[tid] = c8;
      }
      __syncthreads();
      unsigned ab = sh_above, bin = 0, bin_cnt = 0;  // every thread walks the 8 bins itself
#pragma unroll
      for (int jb = 0; jb < 8; ++jb) {
        const unsigned c8 = cnt8[jb];
        if (bin_cnt == 0 && ab < k_rem && k_rem <= ab + c8) { bin = RADIX_BINS - 1 - 8 * gsel - jb; bin_cnt = c8; }
        if (bin_cnt == 0) ab += c8;
      }
      prefix = (prefix << width) | bin;
      k_rem -= ab;                                // keys in higher bins are all selected
      shift = nshift;
#pragma unroll
      for (int jb = 0; jb < 8; ++jb) {            // local keys in higher bins of this pass, counted from the histogram
        const unsigned b8 = RADIX_BINS - 1 - 8 * tid - jb;
        if (b8 > bin) above_acc += h[b8];
      }
      eq_local = h[bin];
      __syncthreads();                            // sh_grp, sh_above and cnt8 are rewritten by the next pass
      if (bin_cnt <= (unsigned)SEL_CAND_MAX) break;
    }
  }

  // ---- E. publish what the peers need to finish: how many local pages are certainly selected (forced pages and
  // the keys above the chosen bins, already counted from the histograms), and the local keys that share the prefix
  // (listed when digits remain, only counted when the prefix is the whole key)
  {
    above_acc = __reduce_add_sync(0xffffffffu, above_acc);
    if (lane == 0 && above_acc) atomicAdd(&pub.above, above_acc);
    if (tid == 0) {
      atomicAdd(&pub.above, (unsigned)(n_local - n_free_local));        // forced pages of this block
      if (k_free > 0 && shift == 0) pub.eq = eq_local;
    }
    if (k_free > 0 && shift > 0) {
      for (int pl = tid; pl < n_free_local; pl += SEL_THREADS) {
        const uint32_t key = keys[pl];
        if (((unsigned long long)(key - klo) >> shift) == prefix) {
          const unsigned slot = atomicAdd(&pub.cand_n, 1u);
          if (slot < (unsigned)SEL_CAND_MAX) pub.cand[slot] = key;
        }
      }
    }
  }
  dd_cluster_sync();
  // ---- F. every block derives the threshold and its own output offsets
  if (tid < C) {
    const dd_sel_pub* pr = cl.map_shared_rank(&pub, tid);
    peer_above[tid] = pr->above;
    peer_eq[tid] = pr->eq;
    peer_cand[tid] = min(pr->cand_n, (unsigned)SEL_CAND_MAX);
  }
  __syncthreads();
  uint32_t thr = 0xFFFFFFFFu;
  unsigned base_gt = 0, base_eq = 0;
  for (int r = 0; r < rank; ++r) base_gt += peer_above[r];
  if (k_free > 0 && shift == 0) {
    thr = klo + (uint32_t)prefix;                 // k_rem of the keys equal to thr are still to be taken
    for (int r = 0; r < rank; ++r) base_eq += peer_eq[r];
  } else if (k_free > 0) {
    unsigned n_all = 0, n_mine_from = 0;          // candidates of all blocks, in block order
    for (int r = 0; r < C; ++r) {
      if (r == rank) n_mine_from = n_all;
      const uint32_t* cr = cl.map_shared_rank(&pub, r)->cand;
      const unsigned n_r = peer_cand[r];
      for (unsigned i = tid; i < n_r; i += SEL_THREADS) all_c[n_all + i] = cr[i];
      n_all += n_r;
    }
    __syncthreads();
    for (unsigned i = tid; i < n_all; i += SEL_THREADS) {
      const uint32_t v = all_c[i];
      unsigned gtc = 0, gec = 0;
      for (unsigned j = 0; j < n_all; ++j) {
        const uint32_t u = all_c[j];
        gtc += u > v;
        gec += u >= v;
      }
      if (gtc < k_rem && k_rem <= gec) { sh_thr = v; sh_above = gtc; }   // equal candidates write equal values
    }
    __syncthreads();
    thr = sh_thr;
    k_rem -= sh_above;
    // candidates of lower blocks above / equal to the threshold
    unsigned c_gt = 0, c_eq = 0;
    for (unsigned i = tid; i < n_mine_from; i += SEL_THREADS) {
      c_gt += all_c[i] > thr;
      c_eq += all_c[i] == thr;
    }
    c_gt = __reduce_add_sync(0xffffffffu, c_gt);
    c_eq = __reduce_add_sync(0xffffffffu, c_eq);
    if (lane == 0) {
      if (c_gt) atomicAdd(&sh_base_gt, c_gt);
      if (c_eq) atomicAdd(&sh_base_eq, c_eq);
    }
    __syncthreads();
    base_gt += sh_base_gt;
    base_eq += sh_base_eq;
  }
  dd_cluster_arrive();                           // last remote read done: peers may leave
  // ---- G. ordered compaction of this block's pages: a warp owns a contiguous segment and walks it 32 pages at a
  // time; ascending page numbers, equal keys are taken from the lowest page up
  {
    const int seg = (((n_local + SEL_WARPS - 1) / SEL_WARPS) + 31) & ~31;
    const int s0 = min(n_local, warp * seg), s1 = min(n_local, s0 + seg);
    const unsigned lt = (1u << lane) - 1u;
    unsigned n_gt = 0, n_eq = 0;
    for (int base = s0; base < s1; base += 32) {
      const int pl = base + lane;
      bool gt = false, eq = false;
      if (pl < s1) {
        const uint32_t key = keys[pl];
        gt = p_lo + pl >= n_free || key > thr;
        eq = !gt && key == thr;
      }
      n_gt += __popc(__ballot_sync(0xffffffffu, gt));
      n_eq += __popc(__ballot_sync(0xffffffffu, eq));
    }
    if (lane == 0) { warp_gt[warp] = n_gt; warp_eq[warp] = n_eq; }
    __syncthreads();
    unsigned run_gt = base_gt, run_eq = base_eq;
    for (int w = 0; w < warp; ++w) { run_gt += warp_gt[w]; run_eq += warp_eq[w]; }
    int* out = out_idx + bg * k;
    for (int base = s0; base < s1; base += 32) {
      const int pl = base + lane;
      bool gt = false, eq = false;
      if (pl < s1) {
        const uint32_t key = keys[pl];
        gt = p_lo + pl >= n_free || key > thr;
        eq = !gt && key == thr;
      }
      const unsigned bgt = __ballot_sync(0xffffffffu, gt), beq = __ballot_sync(0xffffffffu, eq);
      const unsigned gt_before = run_gt + __popc(bgt & lt);
      const unsigned eq_before = run_eq + __popc(beq & lt);
      if (gt || (eq && eq_before < k_rem)) {
        const unsigned pos = gt_before + min(eq_before, k_rem);
        if (pos < (unsigned)k) out[pos] = p_lo + pl;
      }
      run_gt += __popc(bgt);
      run_eq += __popc(beq);
    }
    if (rank == 0)                               // precondition k <= n_pages violated: pad with the last valid page
      for (int j = k_eff + tid; j < k; j += SEL_THREADS) out[j] = np > 0 ? np - 1 : 0;
  }
  dd_cluster_wait();                             // nobody leaves while its shared memory may still be read
}

// ------------------------------------------------------------------------------------------------
// Measurement aid: the fused selection kernel's landmark loads and nothing else (same grid and block shape,
// same rows per block, same fragment addresses; no arithmetic, no exchange).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(SEL_THREADS, 2) dd_select_loads_only_kernel(const __nv_bfloat16* __restrict__ lm,
                                                                              const int* __restrict__ n_pages, int P,
                                                                              int Hkv, int ppc, int R, int ring_stages,
                                                                              unsigned int* __restrict__ sink) {
  extern __shared__ __align__(16) unsigned char sel_smem[];
  const int rank = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gl = lane >> 2, t = lane & 3;
  const size_t bg = (size_t)b * Hkv + g;
  dd_grid_dependency_wait();
  const int np = min(n_pages[b], P);
  const int row_lo = rank * ppc * R, row_max = P * R - 1;
  const int n_local_rows = max(0, min(np * R, row_lo + ppc * R) - row_lo);
  const int n_tiles = (n_local_rows + 15) >> 4;
  const __nv_bfloat16* lm_bg = lm + bg * (size_t)P * R * DD_D;
  uint4* my_ring = reinterpret_cast<uint4*>(sel_smem) + (size_t)warp * ring_stages * 256 + lane;
  unsigned int acc = 0;
  auto issue = [&](int tile, int slot) {
    if (tile < n_tiles) {
      const int pa = min(row_lo + tile * 16 + gl, row_max);
      const int pb = min(row_lo + tile * 16 + gl + 8, row_max);
      const uint4* ra = reinterpret_cast<const uint4*>(lm_bg + (size_t)pa * DD_D) + t;
      const uint4* rb = reinterpret_cast<const uint4*>(lm_bg + (size_t)pb * DD_D) + t;
      uint4* dst = my_ring + slot * 256;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        dd_cp_async16(dst + kk * 32, ra + kk * 4);
        dd_cp_async16(dst + (4 + kk) * 32, rb + kk * 4);
      }
    }
    dd_cp_async_commit();
  };
  const int ahead = ring_stages - 1;
  for (int s = 0; s < ahead; ++s) issue(warp + s * SEL_WARPS, s);
  int slot = 0, slot_issue = ahead;
  for (int tile = warp; tile < n_tiles; tile += SEL_WARPS) {
    issue(tile + ahead * SEL_WARPS, slot_issue);
    dd_cp_async_wait_pending(ahead);
    const uint4* src = my_ring + slot * 256;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint4 v = src[i * 32];
      acc ^= v.x ^ v.y ^ v.z ^ v.w;
    }
    slot = slot + 1 == ring_stages ? 0 : slot + 1;
    slot_issue = slot_issue + 1 == ring_stages ? 0 : slot_issue + 1;
  }
  dd_cp_async_wait_pending(0);
  if (acc == 0x9E3779B9u) sink[0] = acc;        // keeps the loads alive; practically never true
}

int dd_launch_select_loads_only(dd_ctx* ctx, const void* landmarks, const int* n_pages, cudaStream_t st) {
  const dd_config& c = ctx->cfg;
  if (ctx->sel_cluster <= 0) return dd_fail(ctx, DD_ERR_STATE, "the load-only probe follows the fused selection kernel");
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctx->sel_cluster, c.n_kv_heads, c.batch);
  cfg.blockDim = dim3(SEL_THREADS);
  cfg.dynamicSmemBytes = ctx->sel_smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  dd_pdl_attr(&attr[0]);                         // launched the way the kernel it stands in for is
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  DD_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, dd_select_loads_only_kernel, (const __nv_bfloat16*)landmarks, n_pages,
                                      c.max_pages, c.n_kv_heads, ctx->sel_ppc, ctx->R, ctx->sel_stages,
                                      ctx->attn_ticket + c.batch * c.n_kv_heads));
  return DD_OK;
}

int dd_launch_select(dd_ctx* ctx, const void* q, int q_token, int q_tokens_in_tensor, const void* landmarks,
                     const int* n_pages, int* out_idx, float* out_scores, cudaStream_t st, const int* ctx_len) {
  const dd_config& c = ctx->cfg;
  const int G = ctx->G;
  if (ctx->R > 1 && !ctx_len) return dd_fail(ctx, DD_ERR_INVALID_ARG, "finer landmarks need ctx_len for the selection");
  if (ctx->sel_cluster > 0) {
    // logits in global scratch: the selection stream of the pipelined path has a buffer of its own, because a
    // selection there may run next to one on the compute stream
    float* s_glob = nullptr;
    if (ctx->sel_logits_global) {
      const size_t per_buf = (size_t)c.batch * c.n_kv_heads * c.max_pages * ctx->R * G;
      s_glob = ctx->score_s + ((c.select_stream && st == (cudaStream_t)c.select_stream) ? per_buf : 0);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctx->sel_cluster, c.n_kv_heads, c.batch);
    cfg.blockDim = dim3(SEL_THREADS);
    cfg.dynamicSmemBytes = ctx->sel_smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ctx->sel_cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    dd_pdl_attr(&attr[1]);
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    DD_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, dd_select_fused_kernel, (const __nv_bfloat16*)q,
                                        q_tokens_in_tensor * c.n_q_heads * DD_D, q_token * c.n_q_heads * DD_D,
                                        (const __nv_bfloat16*)landmarks, n_pages, out_idx, out_scores, c.max_pages, G,
                                        c.n_kv_heads, c.k_pages, c.forced_recent_pages, ctx->sel_ppc, ctx->err_word,
                                        ctx->R, ctx_len, ctx->sel_stages, s_glob));
    return DD_OK;
  }
  dim3 sgrid(ctx->score_tiles, c.n_kv_heads, c.batch);
  dd_score_kernel<<<sgrid, 128, 0, st>>>((const __nv_bfloat16*)q, q_tokens_in_tensor * c.n_q_heads * DD_D,
                                         q_token * c.n_q_heads * DD_D, (const __nv_bfloat16*)landmarks, n_pages,
                                         ctx->score_s, ctx->score_part, c.max_pages, G, c.n_kv_heads,
                                         ctx->score_tiles);
  DD_CUDA_TRY(ctx, cudaGetLastError());
  dim3 tgrid(c.n_kv_heads, c.batch);
  dd_topk_kernel<<<tgrid, TOPK_THREADS, TOPK_SMEM_KEYS * sizeof(uint32_t), st>>>(
      ctx->score_s, ctx->score_part, n_pages, ctx->topk_keys, out_idx, out_scores, c.max_pages, G, c.n_kv_heads,
      ctx->score_tiles, c.k_pages, c.forced_recent_pages, ctx->err_word);
  DD_CUDA_TRY(ctx, cudaGetLastError());
  return DD_OK;
}

// Picks the cluster size of the fused selection: a power of two such that all clusters are resident at once
// (two blocks per SM), every block has at least 32 pages, and a block's share of the logits fits in shared
// memory. Up to 8 blocks, 16 for very long requests. 0 = not possible, use the two-kernel path.
// The search walks a fixed candidate list exactly once, so it always terminates; `fits` answers whether clusters of that shape can be resident on the device.
// Shared memory of one block: the logits of its rows (unless they live in global scratch), then the larger of the
// scoring ring (one 4 KiB tile per warp and stage) and the keys + two histograms that take its place afterwards.
static size_t dd_select_smem(int ppc, int rows_per_page, int group, int stages, bool logits_in_smem) {
  const size_t ring = (size_t)SEL_WARPS * stages * 4096, later = (size_t)ppc * 4 + 2 * RADIX_BINS * 4;
  return (logits_in_smem ? (size_t)ppc * rows_per_page * group * 4 : 0) + (ring > later ? ring : later);
}

// Block shape of the fused selection for one cluster size: every block is sized so that two fit on an SM (the device
// holds about half as many clusters otherwise). The logits stay in shared memory when a ring of two tiles per warp
// still fits next to them; else they go to global scratch.
static void dd_select_shape(int max_pages, int C, int rows_per_page, int group, int* ppc_out, int* stages_out,
                            int* logits_global_out, size_t* smem_out) {
  const size_t budget = (size_t)112 * 1024;
  int ppc = (max_pages + C - 1) / C;
  ppc = (ppc + 31) & ~31;                                  // whole pairs of MMA tiles
  const bool in_smem = dd_select_smem(ppc, rows_per_page, group, 2, true) <= budget;
  const int stages = 2;                                    // measured: deeper rings buy nothing, larger blocks launch slower
  *ppc_out = ppc;
  *stages_out = stages;
  *logits_global_out = in_smem ? 0 : 1;
  *smem_out = dd_select_smem(ppc, rows_per_page, group, stages, in_smem);
}

extern "C" int dd_test_pick_cluster(int max_pages, int problems, int sm_count, int rows_per_page, int group, int allow16,
                                    int (*fits)(int blocks, size_t shared_bytes, void* user), void* user,
                                    int* pages_per_block, size_t* shared_bytes, int* ring_stages, int* logits_global) {
  if (max_pages < 1 || problems < 1 || sm_count < 1 || rows_per_page < 1 || group < 1 || !fits) return 0;
  const int c_max = (max_pages >= 32768 && allow16) ? 16 : 8;
  int start = 1;
  while (start * 2 <= c_max && (long long)start * 2 * problems <= 2LL * sm_count && max_pages / (start * 2) >= 32) start *= 2;
  // candidates: the preferred size, every larger one, then the smaller ones (fewer, larger blocks)
  int cand[16], n_cand = 0;
  for (int C = start; C <= c_max; C *= 2) cand[n_cand++] = C;
  for (int C = start / 2; C >= 1; C /= 2) cand[n_cand++] = C;
  // first choice: a size of which the device holds all clusters at once; else any size that can run at all
  for (int need_all = 1; need_all >= 0; --need_all) {
    for (int i = 0; i < n_cand; ++i) {
      const int C = cand[i];
      int ppc, stages, lg;
      size_t smem;
      dd_select_shape(max_pages, C, rows_per_page, group, &ppc, &stages, &lg, &smem);
      if (smem > (size_t)SEL_MAX_SMEM) continue;           // too long for this cluster size
      if (fits(C, smem, user) < (need_all ? problems : 1)) continue;
      if (pages_per_block) *pages_per_block = ppc;
      if (shared_bytes) *shared_bytes = smem;
      if (ring_stages) *ring_stages = stages;
      if (logits_global) *logits_global = lg;
      return C;
    }
  }
  return 0;
}

// How many clusters of C blocks with `smem` bytes of dynamic shared memory can be resident at once (0 on error).
static int dd_select_resident_clusters(const dd_ctx* ctx, int C, size_t smem) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(C, ctx->cfg.n_kv_heads, ctx->cfg.batch);
  cfg.blockDim = dim3(SEL_THREADS);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n_clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&n_clusters, dd_select_fused_kernel, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n_clusters;
}

static int dd_select_cluster_fits(int C, size_t smem, void* user) {
  return dd_select_resident_clusters((const dd_ctx*)user, C, smem);
}

static int dd_select_pick_cluster(dd_ctx* ctx, int* ppc_out, int* smem_out) {
  const dd_config& c = ctx->cfg;
  // function attributes are per process, not per context: always ask for the largest the kernel may use
  if (cudaFuncSetAttribute(dd_select_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SEL_MAX_SMEM) !=
      cudaSuccess) { cudaGetLastError(); return 0; }
  const bool big_ok = cudaFuncSetAttribute(dd_select_fused_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed,
                                           1) == cudaSuccess;
  if (!big_ok) cudaGetLastError();
  size_t smem = 0;
  const int C = dd_test_pick_cluster(c.max_pages, c.batch * c.n_kv_heads, ctx->sm_count, ctx->R, ctx->G, big_ok ? 1 : 0,
                                     dd_select_cluster_fits, ctx, ppc_out, &smem, &ctx->sel_stages, &ctx->sel_logits_global);
  *smem_out = (int)smem;
  return C;
}

int dd_select_setup(dd_ctx* ctx) {
  DD_CUDA_TRY(ctx, cudaFuncSetAttribute(dd_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)(TOPK_SMEM_KEYS * sizeof(uint32_t))));
  DD_CUDA_TRY(ctx, cudaFuncSetAttribute(dd_select_loads_only_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        SEL_MAX_SMEM));
  ctx->sel_cluster = 0;
  if (ctx->cfg.select_mode != DD_SELECT_TWO_KERNELS)
    ctx->sel_cluster = dd_select_pick_cluster(ctx, &ctx->sel_ppc, &ctx->sel_smem_bytes);
  if (ctx->R > 1 && ctx->sel_cluster == 0)
    return dd_fail(ctx, DD_ERR_INVALID_ARG, "finer landmarks are supported by the fused selection kernel only, and "
                   "this request length does not fit it");
  return DD_OK;
}
