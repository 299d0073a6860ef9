// GQA decode attention over the gathered set of a ring slot on the fifth-generation tensor cores.
//
// Same work split as the streaming kernel (the slot is one flat list of pages, cut into equal runs, one run per
// block, units that are cut across blocks are merged by the last block to arrive), one block per SM. Inside a
// block the pages of a unit are taken in tiles of eight (128 tokens):
//   warp 4, one thread   TMA: the tile's K and V rows into a three-deep shared-memory ring, 128-byte swizzle, one
//                        [64 channels x 128 rows] box per (K | V, channel half); partial tiles page by page
//   warps 5 and 6, one   tcgen05.mma, accumulators in tensor memory (an issuing thread per product: issuing costs
//   thread each          40-70 ns per instruction whatever its size, the tensor pipe itself is busy 2% of the time):
//                          S^T[128 tokens x 16] = K[128 x 128] . q^T          (A = K tile, K-major; B = q, rows 8..15 zero)
//                          O^T[128 channels x 16] += V^T[128 x 16 tokens] . P^T   per page (A = V, MN-major; B = P)
//   warps 0-3            one thread per token of the tile: S from tensor memory, running soft-max over tiles, P
//                        (bf16) into shared memory as the next B operand; S and P are double-buffered, O is rescaled
//                        in tensor memory only when a row's reference maximum moves by more than 2^8; at the end of a
//                        unit's pages thread d owns channel d of O
// The up-to-8 query rows of a KV head are the N columns (padded to 16, the smallest N for M = 128). All waits on
// mbarriers are bounded; a wait that gives up sets the device error word and the block runs out without waiting
// again, frees its tensor memory and returns.
#include <cuda.h>

#include "dd_common.cuh"

constexpr int TC_EPI = 4;                              // soft-max / epilogue warps = 128 tensor-memory lanes
constexpr int TC_THREADS = (TC_EPI + 3) * 32;           // + TMA warp, S^T issuer, O^T issuer
constexpr int TC_TILE_PAGES = 8;
constexpr int TC_TILE_TOKENS = TC_TILE_PAGES * DD_T;   // 128
constexpr int TC_HALF_BYTES = TC_TILE_TOKENS * 128;    // one (K | V, channel half) of a tile: 128 rows of 128 B
constexpr int TC_TILE_BYTES = 4 * TC_HALF_BYTES;       // 64 KiB: K ch 0-63, K ch 64-127, V ch 0-63, V ch 64-127
constexpr int TC_STAGES = 3;
constexpr int TC_N = 16;                               // N of both products (8 query rows, padded)
constexpr int TC_B_BYTES = TC_N * 128 * 2;             // q operand: 16 rows x 128 channels; P operand: 16 rows x 128 tokens
constexpr int TC_ROWS = 8;
constexpr int TC_MAX_PARTS = 64;
constexpr int TC_SMEM_BYTES = TC_STAGES * TC_TILE_BYTES + 4 * TC_B_BYTES + 1024;   // ring, two q buffers, two P buffers
constexpr int TC_TMEM_COLS = 64;                       // S^T of even / odd tiles in columns 0..15 / 16..31, O^T in 32..47
constexpr float TC_LAZY = 8.f;                         // a row's reference maximum moves only when exceeded by 2^8

__device__ __forceinline__ uint32_t tc_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long tc_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait for a phase of an mbarrier. Returns at once when another thread of the block already gave up.
__device__ __forceinline__ bool tc_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned long long limit_ns) {
  unsigned long long t0 = 0;
  for (unsigned it = 0;; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    if (*abort_flag) return false;
    if ((it & 31u) == 31u) {
      const unsigned long long now = tc_timer();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) { *abort_flag = 1; return false; }
    }
  }
}

__device__ __forceinline__ void tc_tma_box(uint32_t dst, const CUtensorMap* tmap, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(tmap), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

// Shared-memory matrix descriptor of tcgen05.mma: start address, leading and stride byte offsets in 16-byte units,
// descriptor version 1, swizzle mode in the top bits (0: none, 2: 128 bytes).
__device__ __forceinline__ uint64_t tc_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t swizzle) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | ((uint64_t)swizzle << 61);
}

// Instruction descriptor, kind::f16: D = f32, A = B = bf16, majorness of A (0: K-major, 1: MN-major), B K-major.
__host__ __device__ constexpr uint32_t tc_idesc(int M, int N, int a_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// The mbarrier gets one arrival when every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_ld8(uint32_t taddr, float (&v)[8]) {
  uint32_t r[8];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tc_st8(uint32_t taddr, const float (&v)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr),
               "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
               "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7]))
               : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_arrive(uint32_t bar) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); }
__device__ __forceinline__ void tc_epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ float tc_warp_max(float v) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
  return r;
}
// A load the compiler may not move: issued where it stands, so that its latency runs under the work that follows.
__device__ __forceinline__ int tc_ld_idx(const int* p) {
  int v;
  asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
// Every lane holds the same n values v[0..n): lane i < n gets v[i] (a chain of selects; a loop of `if (lane == i)`
// stores costs 0.6 us for eight values, measured).
template <int N>
__device__ __forceinline__ float tc_pick(const float (&v)[N], int lane) {
  float mine = v[0];
#pragma unroll
  for (int i = 1; i < N; ++i) mine = lane == i ? v[i] : mine;
  return mine;
}
__device__ __forceinline__ float tc_ex2(float x) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

// The tiles of a block's run in order: unit by unit (a segment = the pages of one unit inside the run), eight pages at
// a time. All three roles walk the same sequence.
struct tc_iter {
  int f, f1, k, u, j0, seg_n, tp, seg_no, tile_no;
  __device__ void start(int f0_, int f1_, int k_) {
    f = f0_; f1 = f1_; k = k_; seg_no = 0; tile_no = 0; tp = 0;
    segment();
  }
  __device__ void segment() {
    if (f < f1) { u = f / k; j0 = f - u * k; seg_n = min(f1 - f, k - j0); }
  }
  __device__ bool valid() const { return f < f1; }
  __device__ int np() const { return min(TC_TILE_PAGES, seg_n - tp); }
  __device__ bool first() const { return tp == 0; }
  __device__ bool last() const { return tp + TC_TILE_PAGES >= seg_n; }
  __device__ void next() {
    tp += TC_TILE_PAGES; ++tile_no;
    if (tp >= seg_n) { f += seg_n; ++seg_no; tp = 0; segment(); }
  }
};

// Grid: n_blocks blocks of TC_THREADS threads; block x owns the pages [x * ppb, min(total, (x + 1) * ppb)) of the
// flat list (unit u = page / k, position j = page % k). part_o / part_ml hold max_parts partials per unit.
// map_tile: boxes of 64 channels x 128 rows; map_page: boxes of 64 channels x 16 rows; both with the 128-byte swizzle.
__global__ void __launch_bounds__(TC_THREADS, 1) dd_attn_tc_kernel(
    const __grid_constant__ CUtensorMap map_tile, const __grid_constant__ CUtensorMap map_page,
    const __nv_bfloat16* __restrict__ q, const int* __restrict__ idx, const int* __restrict__ ctx_len,
    __nv_bfloat16* __restrict__ out, float* __restrict__ out_lse, float* __restrict__ part_o, float2* __restrict__ part_ml,
    unsigned int* __restrict__ ticket, int Hkv, int G, int Tq, int k, int total_pages, int ppb, int max_parts,
    const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new, int* err_word,
    unsigned long long wait_ns) {
  extern __shared__ unsigned char tc_dyn[];
  __shared__ __align__(8) unsigned long long full_bar[TC_STAGES];
  __shared__ __align__(8) unsigned long long empty_bar[TC_STAGES];
  __shared__ __align__(8) unsigned long long s_full_bar[2], p_ready_bar[2], pv_done_bar[2], q_bar[2];
  __shared__ uint32_t tmem_base_s;
  __shared__ float red_a[2][TC_EPI][TC_ROWS], red_b[TC_EPI][TC_ROWS];
  __shared__ float tail_s[TC_EPI][2 * TC_ROWS];
  __shared__ float2 sm_lm[TC_ROWS];
  __shared__ float sm_sc[TC_MAX_PARTS * TC_ROWS];
  __shared__ int sm_last;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t ring = (tc_smem(tc_dyn) + 1023u) & ~1023u;          // swizzled tiles want 1 KiB alignment
  const uint32_t q_smem = ring + TC_STAGES * TC_TILE_BYTES;
  const uint32_t p_smem = q_smem + 2 * TC_B_BYTES;
  const int f0 = blockIdx.x * ppb;
  const int f1 = min(total_pages, f0 + ppb);

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < TC_STAGES; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tc_smem(&full_bar[s])));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tc_smem(&empty_bar[s])));
    }
    for (int i = 0; i < 2; ++i) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tc_smem(&s_full_bar[i])));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tc_smem(&pv_done_bar[i])));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 128;" ::"r"(tc_smem(&p_ready_bar[i])));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 128;" ::"r"(tc_smem(&q_bar[i])));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp < TC_EPI) {
    // both B operands start as zeros: their rows 8..15 are never written again
    for (int i = threadIdx.x; i < 4 * TC_B_BYTES / 16; i += TC_EPI * 32)
      asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(q_smem + i * 16), "r"(0u) : "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == TC_EPI + 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem(&tmem_base_s)),
                 "r"((uint32_t)TC_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_s;
  volatile int* abort_p = &abort_flag;
  dd_grid_dependency_wait();

  if (warp == TC_EPI) {
    // ---- producer: one thread keeps the ring of tiles full
    if (lane == 0) {
      int tile_no = 0, issued = 0;
      bool ok = true;
      for (int f = f0; f < f1 && ok;) {
        const int u = f / k, j0 = f - u * k;
        const int seg_n = min(f1 - f, k - j0);
        for (int tp = 0; tp < seg_n && ok; tp += TC_TILE_PAGES, ++tile_no) {
          const int np = min(TC_TILE_PAGES, seg_n - tp);
          const int s = tile_no % TC_STAGES, round = tile_no / TC_STAGES;
          if (round > 0 && !tc_wait(tc_smem(&empty_bar[s]), (uint32_t)((round - 1) & 1), abort_p, wait_ns)) { ok = false; break; }
          const int row_k = (u * 2 * k + j0 + tp) * DD_T, row_v = row_k + k * DD_T;
          const uint32_t bar = tc_smem(&full_bar[s]);
          const uint32_t dst = ring + (uint32_t)s * TC_TILE_BYTES;
          asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)(np * DD_PAGE_BYTES)) : "memory");
          if (np == TC_TILE_PAGES) {
            tc_tma_box(dst, &map_tile, 0, row_k, bar);
            tc_tma_box(dst + TC_HALF_BYTES, &map_tile, 64, row_k, bar);
            tc_tma_box(dst + 2 * TC_HALF_BYTES, &map_tile, 0, row_v, bar);
            tc_tma_box(dst + 3 * TC_HALF_BYTES, &map_tile, 64, row_v, bar);
          } else {
            for (int p = 0; p < np; ++p) {
              tc_tma_box(dst + p * 2048, &map_page, 0, row_k + p * DD_T, bar);
              tc_tma_box(dst + TC_HALF_BYTES + p * 2048, &map_page, 64, row_k + p * DD_T, bar);
              tc_tma_box(dst + 2 * TC_HALF_BYTES + p * 2048, &map_page, 0, row_v + p * DD_T, bar);
              tc_tma_box(dst + 3 * TC_HALF_BYTES + p * 2048, &map_page, 64, row_v + p * DD_T, bar);
            }
          }
          issued = tile_no + 1;
        }
        f += seg_n;
      }
      // every copy this thread issued must have landed before the block may retire: wait (bounded, whatever the
      // abort flag says) for the last use of every stage
      for (int i = max(0, issued - TC_STAGES); i < issued; ++i) {
        const uint32_t bar = tc_smem(&full_bar[i % TC_STAGES]);
        const unsigned long long t0 = tc_timer();
        for (unsigned it = 0;; ++it) {
          uint32_t done;
          asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                       : "=r"(done) : "r"(bar), "r"((uint32_t)((i / TC_STAGES) & 1)) : "memory");
          if (done) break;
          if ((it & 31u) == 31u && tc_timer() - t0 > wait_ns) { *abort_p = 1; break; }
        }
      }
      if (*abort_p) dd_report(err_word, DD_ERR_WAIT_EXPIRED, 4);
    }
    __syncwarp();
  } else if (warp == TC_EPI + 1) {
    // ---- one thread issues S^T = K q^T. Issuing costs 40-70 ns per tcgen05.mma whatever its size (measured), so the
    // two products have an issuing thread each. S^T of tile t goes to buffer t % 2 as soon as the soft-max of tile
    // t - 2 has read it, also across a unit boundary (the q operand of unit s sits in buffer s % 2, written a unit ahead).
    if (lane == 0) {
      constexpr uint32_t IDESC_QK = tc_idesc(128, TC_N, 0);
      tc_iter it;
      for (it.start(f0, f1, k); it.valid(); it.next()) {
        const int t = it.tile_no, s = t % TC_STAGES, round = t / TC_STAGES;
        if (it.first() && !tc_wait(tc_smem(&q_bar[it.seg_no & 1]), (uint32_t)((it.seg_no >> 1) & 1), abort_p, wait_ns)) break;
        if (t >= 2 && !tc_wait(tc_smem(&p_ready_bar[t & 1]), (uint32_t)(((t - 2) >> 1) & 1), abort_p, wait_ns)) break;
        if (!tc_wait(tc_smem(&full_bar[s]), (uint32_t)(round & 1), abort_p, wait_ns)) break;
        tc_fence_after();
        const uint32_t stage = ring + (uint32_t)s * TC_TILE_BYTES;
        const uint32_t qb = q_smem + (it.seg_no & 1) * TC_B_BYTES;
#pragma unroll
        for (int kk = 0; kk < DD_D / 16; ++kk) {
          const uint64_t a = tc_desc(stage + (kk >> 2) * TC_HALF_BYTES + (kk & 3) * 32, 16, 1024, 2);
          const uint64_t bq = tc_desc(qb + kk * 512, 256, 128, 0);
          tc_mma(tmem_base + (t & 1) * TC_N, a, bq, IDESC_QK, kk > 0 ? 1u : 0u);
        }
        tc_commit(tc_smem(&s_full_bar[t & 1]));
      }
    }
    __syncwarp();
  } else if (warp == TC_EPI + 2) {
    // ---- one thread issues O^T += V^T P^T, page by page, and releases the tile's ring stage (its S^T product was
    // complete before the soft-max that produced this P could start)
    if (lane == 0) {
      constexpr uint32_t IDESC_PV = tc_idesc(128, TC_N, 1);
      const uint32_t tmem_o = tmem_base + 2 * TC_N;
      tc_iter it;
      for (it.start(f0, f1, k); it.valid(); it.next()) {
        const int t = it.tile_no, s = t % TC_STAGES, round = t / TC_STAGES, np = it.np();
        if (!tc_wait(tc_smem(&full_bar[s]), (uint32_t)(round & 1), abort_p, wait_ns)) break;
        if (!tc_wait(tc_smem(&p_ready_bar[t & 1]), (uint32_t)((t >> 1) & 1), abort_p, wait_ns)) break;
        tc_fence_after();
        const uint32_t stage = ring + (uint32_t)s * TC_TILE_BYTES;
#pragma unroll
        for (int p = 0; p < TC_TILE_PAGES; ++p) {
          if (p >= np) break;
          const uint64_t a = tc_desc(stage + 2 * TC_HALF_BYTES + p * 2048, TC_HALF_BYTES, 1024, 2);
          const uint64_t bp = tc_desc(p_smem + (t & 1) * TC_B_BYTES + p * 512, 256, 128, 0);
          tc_mma(tmem_o, a, bp, IDESC_PV, (it.first() && p == 0) ? 0u : 1u);
        }
        tc_commit(tc_smem(&empty_bar[s]));
        tc_commit(tc_smem(&pv_done_bar[t & 1]));
      }
    }
    __syncwarp();
  } else {
    // ---- soft-max and epilogue: thread = token of the tile (lane of S^T), later channel of O^T
    const int Hq = Hkv * G;
    const int n_rows = Tq * G;
    const float scale_log2 = rsqrtf((float)DD_D) * 1.4426950408889634f;
    const int d = threadIdx.x;
    const int pg = d >> 4, tk = d & 15;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const uint32_t tmem_o = tmem_base + lane_base + 2 * TC_N;
    const uint32_t p_dst = p_smem + pg * 512 + (tk >> 3) * 256 + (tk & 7) * 2;      // + buffer * TC_B_BYTES + n * 16
    // A wait that gives up is not acted upon here: the abort flag makes every later wait return at once, and all 128
    // threads keep the same control flow through the named barriers (the results are then garbage and the error word says so).
    // q of unit `uu` as the B operand of S^T: [16 rows][128 channels] in 8 x 16-byte core matrices, rows 8..15 zero.
    // Unit s of the run uses buffer s % 2 and is written while unit s - 1 is being worked on: the buffer's previous
    // user, unit s - 2, is complete by then.
    auto write_q = [&](int uu, int sn) {
      const int bb = uu / Hkv, gg = uu - bb * Hkv;
      const uint32_t qb = q_smem + (sn & 1) * TC_B_BYTES;
      for (int i = d; i < TC_N * 16; i += TC_EPI * 32) {
        const int n = i >> 4, c = i & 15;
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (n < n_rows) {
          const int tq = n / G, hh = n - tq * G;
          val = __ldg(reinterpret_cast<const uint4*>(q + (((size_t)bb * Tq + tq) * Hq + gg * G + hh) * DD_D) + c);
        }
        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(qb + c * 256 + (n >> 3) * 128 + (n & 7) * 16),
                     "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w)
                     : "memory");
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      tc_arrive(tc_smem(&q_bar[sn & 1]));
    };
    int tile_no = 0, seg_no = 0;
    if (f0 < f1) write_q(f0 / k, 0);
    for (int f = f0; f < f1; ++seg_no) {
      const int u = f / k, j0 = f - u * k;
      const int seg_n = min(f1 - f, k - j0);
      const int b = u / Hkv, g = u - b * Hkv;
      const size_t bg = (size_t)u;
      if (f + seg_n < f1) write_q(u + 1, seg_no + 1);
      const int* idx_bg = idx + bg * k;
      const int n_ctx = ctx_len[b];
      float m_used[TC_ROWS], l_part[TC_ROWS];
#pragma unroll
      for (int n = 0; n < TC_ROWS; ++n) { m_used[n] = -INFINITY; l_part[n] = 0.f; }

      int page_next = pg < seg_n ? tc_ld_idx(idx_bg + j0 + pg) : 0;
      for (int tp = 0; tp < seg_n; tp += TC_TILE_PAGES, ++tile_no) {
        const int np = min(TC_TILE_PAGES, seg_n - tp);
        const bool in_tile = pg < np;
        const int page = page_next;
        page_next = tp + TC_TILE_PAGES + pg < seg_n ? tc_ld_idx(idx_bg + j0 + tp + TC_TILE_PAGES + pg) : 0;   // in flight during this tile
        const bool valid = in_tile && page * DD_T + tk < n_ctx;
        tc_wait(tc_smem(&s_full_bar[tile_no & 1]), (uint32_t)((tile_no >> 1) & 1), abort_p, wait_ns);
        tc_fence_after();
        float s[TC_ROWS];
        tc_ld8(tmem_base + lane_base + (tile_no & 1) * TC_N, s);
        float tmax[TC_ROWS];
#pragma unroll
        for (int n = 0; n < TC_ROWS; ++n) {
          s[n] = valid ? s[n] * scale_log2 : -INFINITY;
          tmax[n] = tc_warp_max(s[n]);
        }
        float (*red)[TC_ROWS] = red_a[tile_no & 1];           // two buffers: one barrier per tile is enough
        {
          const float mine = tc_pick(tmax, lane);             // every lane holds all eight maxima: lane n publishes row n
          if (lane < TC_ROWS) red[warp][lane] = mine;
        }
        tc_epi_sync();
        // A row's reference moves only when the tile's maximum exceeds it by more than 2^TC_LAZY (or it is the unit's
        // first finite one): P then stays below 2^TC_LAZY, sums are fp32, and O is rescaled a few times per unit at most.
        float alpha[TC_ROWS];
        bool moved = false;
#pragma unroll
        for (int n = 0; n < TC_ROWS; ++n) {
          const float tm = fmaxf(fmaxf(red[0][n], red[1][n]), fmaxf(red[2][n], red[3][n]));
          alpha[n] = 1.f;
          if (tm > m_used[n] + TC_LAZY) {            // also the first finite maximum (m_used = -inf)
            alpha[n] = tc_ex2(m_used[n] - tm);       // 0 when m_used was -inf
            m_used[n] = tm;
            moved = true;
          }
          const float p = (m_used[n] == -INFINITY) ? 0.f : tc_ex2(s[n] - m_used[n]);
          l_part[n] = l_part[n] * alpha[n] + p;
          s[n] = p;
        }
        // the P buffer of this tile was last read by the tile two back
        if (tile_no > 1) tc_wait(tc_smem(&pv_done_bar[tile_no & 1]), (uint32_t)(((tile_no - 2) >> 1) & 1), abort_p, wait_ns);
#pragma unroll
        for (int n = 0; n < TC_ROWS; ++n) {
          const __nv_bfloat16 pb = __float2bfloat16_rn(s[n]);
          asm volatile("st.shared.b16 [%0], %1;" ::"r"(p_dst + (tile_no & 1) * TC_B_BYTES + n * 16),
                       "h"(*reinterpret_cast<const unsigned short*>(&pb))
                       : "memory");
        }
        if (tp > 0 && moved) {                       // uniform over the block: every thread holds the same references
          tc_wait(tc_smem(&pv_done_bar[(tile_no - 1) & 1]), (uint32_t)(((tile_no - 1) >> 1) & 1), abort_p, wait_ns);
          tc_fence_after();
          float o[TC_ROWS];
          tc_ld8(tmem_o, o);
#pragma unroll
          for (int n = 0; n < TC_ROWS; ++n) o[n] *= alpha[n];
          tc_st8(tmem_o, o);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        tc_fence_before();
        tc_arrive(tc_smem(&p_ready_bar[tile_no & 1]));
      }
      f += seg_n;

      // ---- the unit's pages held by this block are done: O^T from tensor memory, row sums over the tokens
      tc_wait(tc_smem(&pv_done_bar[(tile_no - 1) & 1]), (uint32_t)(((tile_no - 1) >> 1) & 1), abort_p, wait_ns);
      tc_fence_after();
      float ob[TC_ROWS];
      tc_ld8(tmem_o, ob);
      tc_fence_before();
      float L[TC_ROWS];
#pragma unroll
      for (int n = 0; n < TC_ROWS; ++n) {
        float v = l_part[n];
#pragma unroll
        for (int off = 16; off; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        L[n] = v;
      }
      {
        const float mine = tc_pick(L, lane);
        if (lane < TC_ROWS) red_b[warp][lane] = mine;
      }
      tc_epi_sync();
#pragma unroll
      for (int n = 0; n < TC_ROWS; ++n) L[n] = (red_b[0][n] + red_b[1][n]) + (red_b[2][n] + red_b[3][n]);

      if (k_new != nullptr && j0 == 0) {
        // the step's own new KV entries (dual-token causal tail): query token t sees the entries j <= t. Thread d
        // holds channel d: the dot products are block sums, the values go straight into this thread's channel.
        float part[2 * TC_ROWS];
#pragma unroll
        for (int n = 0; n < TC_ROWS; ++n) {
          float qv = 0.f;
          if (n < n_rows) {
            const int tq = n / G, hh = n - tq * G;
            qv = __bfloat162float(q[(((size_t)b * Tq + tq) * Hq + g * G + hh) * DD_D + d]);
          }
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            float v = (j < Tq) ? qv * __bfloat162float(k_new[(((size_t)b * Tq + j) * Hkv + g) * DD_D + d]) : 0.f;
#pragma unroll
            for (int off = 16; off; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            part[2 * n + j] = v;
          }
        }
        {
          const float mine = tc_pick(part, lane);
          if (lane < 2 * TC_ROWS) tail_s[warp][lane] = mine;
        }
        tc_epi_sync();
        float vn[2];
#pragma unroll
        for (int j = 0; j < 2; ++j)
          vn[j] = (j < Tq) ? __bfloat162float(v_new[(((size_t)b * Tq + j) * Hkv + g) * DD_D + d]) : 0.f;
#pragma unroll
        for (int n = 0; n < TC_ROWS; ++n) {
          if (n < n_rows) {
            const int tq = n / G;
            float sj[2], M = m_used[n];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              sj[j] = (j <= tq && j < Tq)
                          ? ((tail_s[0][2 * n + j] + tail_s[1][2 * n + j]) + (tail_s[2][2 * n + j] + tail_s[3][2 * n + j])) * scale_log2
                          : -INFINITY;
              M = fmaxf(M, sj[j]);
            }
            const float sc = exp2f(m_used[n] - M);   // M is finite: entry 0 is visible to every row
            float a = ob[n] * sc, l = L[n] * sc;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
              const float p = exp2f(sj[j] - M);
              a += p * vn[j];
              l += p;
            }
            ob[n] = a; L[n] = l; m_used[n] = M;
          }
        }
      }

      // which blocks hold pages of this unit
      const int b_first = (u * k) / ppb, b_last = ((u + 1) * k - 1) / ppb;
      const int n_parts = b_last - b_first + 1;
      if (n_parts == 1) {
#pragma unroll
        for (int n = 0; n < TC_ROWS; ++n) {
          if (n < n_rows) {
            const int tq = n / G, hh = n - tq * G;
            const size_t row = ((size_t)b * Tq + tq) * Hq + g * G + hh;
            out[row * DD_D + d] = __float2bfloat16_rn(L[n] > 0.f ? ob[n] / L[n] : 0.f);
            if (out_lse && d == 0) out_lse[row] = (m_used[n] + log2f(L[n])) * 0.6931471805599453f;
          }
        }
        tc_epi_sync();                               // the staging arrays are rewritten by the next unit
        continue;
      }
      {
        const int part = (int)blockIdx.x - b_first;
        float* po = part_o + ((bg * max_parts + part) * TC_ROWS) * DD_D;
#pragma unroll
        for (int n = 0; n < TC_ROWS; ++n) po[n * DD_D + d] = ob[n];
        if (d < TC_ROWS) {
          float mv = -INFINITY, lv = 0.f;
#pragma unroll
          for (int n = 0; n < TC_ROWS; ++n)
            if (n == d) { mv = m_used[n]; lv = L[n]; }
          part_ml[(bg * max_parts + part) * TC_ROWS + d] = make_float2(mv, lv);
        }
        __threadfence();
      }
      tc_epi_sync();
      if (threadIdx.x == 0) {
        const unsigned prev = atomicAdd(&ticket[bg], 1u);
        sm_last = (prev == (unsigned)(n_parts - 1));
      }
      tc_epi_sync();
      if (sm_last) {
        // ---- the last block of the unit to arrive merges the partials
        __threadfence();
        if (threadIdx.x == 0) ticket[bg] = 0u;           // ready for the next launch
        for (int n = warp; n < TC_ROWS; n += TC_EPI) {
          const float2* pml = part_ml + bg * max_parts * TC_ROWS + n;
          float ms[TC_MAX_PARTS / 32], ls[TC_MAX_PARTS / 32];
          float M = -INFINITY;
#pragma unroll
          for (int i = 0; i < TC_MAX_PARTS / 32; ++i) {
            const int sp = lane + 32 * i;
            ms[i] = sp < n_parts ? __ldcg(&pml[sp * TC_ROWS].x) : -INFINITY;
            ls[i] = sp < n_parts ? __ldcg(&pml[sp * TC_ROWS].y) : 0.f;
            M = fmaxf(M, ms[i]);
          }
#pragma unroll
          for (int off = 16; off; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
          float Ls = 0.f;
#pragma unroll
          for (int i = 0; i < TC_MAX_PARTS / 32; ++i) {
            const int sp = lane + 32 * i;
            const float sc = (ms[i] == -INFINITY) ? 0.f : exp2f(ms[i] - M);
            if (sp < n_parts) sm_sc[sp * TC_ROWS + n] = sc;
            Ls += ls[i] * sc;
          }
#pragma unroll
          for (int off = 16; off; off >>= 1) Ls += __shfl_xor_sync(0xffffffffu, Ls, off);
          if (lane == 0) sm_lm[n] = make_float2(M, Ls);
        }
        tc_epi_sync();
        float a[TC_ROWS];
#pragma unroll
        for (int n = 0; n < TC_ROWS; ++n) a[n] = 0.f;
        const float* po = part_o + bg * max_parts * TC_ROWS * DD_D + d;
#pragma unroll 4
        for (int sp = 0; sp < n_parts; ++sp) {
#pragma unroll
          for (int n = 0; n < TC_ROWS; ++n) a[n] += __ldcg(po + (sp * TC_ROWS + n) * DD_D) * sm_sc[sp * TC_ROWS + n];
        }
#pragma unroll
        for (int n = 0; n < TC_ROWS; ++n) {
          if (n < n_rows) {
            const float2 ml = sm_lm[n];
            const int tq = n / G, hh = n - tq * G;
            const size_t row = ((size_t)b * Tq + tq) * Hq + g * G + hh;
            out[row * DD_D + d] = __float2bfloat16_rn(ml.y > 0.f ? a[n] / ml.y : 0.f);
            if (out_lse && d == 0) out_lse[row] = (ml.x + log2f(ml.y)) * 0.6931471805599453f;
          }
        }
      }
      tc_epi_sync();                                     // the staging arrays are rewritten by the next unit
    }
    if (threadIdx.x == 0 && *abort_p) dd_report(err_word, DD_ERR_WAIT_EXPIRED, 5);
  }

  // ---- everybody is done with tensor memory: free it
  tc_fence_before();
  __syncthreads();
  if (warp == TC_EPI + 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TC_TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
// Blocks, pages per block and partials per unit: one block per SM when there is enough work (at least one tile per
// block), and never more than TC_MAX_PARTS blocks per unit.
void dd_attn_tc_geometry(const dd_config* c, int sm_count, int* n_blocks, int* ppb_out, int* max_parts_out) {
  const long long total = (long long)c->batch * c->n_kv_heads * c->k_pages;
  long long nb = sm_count;
  if (nb > (total + TC_TILE_PAGES - 1) / TC_TILE_PAGES) nb = (total + TC_TILE_PAGES - 1) / TC_TILE_PAGES;
  if (nb < 1) nb = 1;
  long long ppb = (total + nb - 1) / nb;
  while ((c->k_pages - 1) / ppb + 2 > TC_MAX_PARTS) ++ppb;
  nb = (total + ppb - 1) / ppb;
  *n_blocks = (int)nb;
  *ppb_out = (int)ppb;
  *max_parts_out = (int)((c->k_pages - 1) / ppb + 2);
}

int dd_attn_tc_setup(dd_ctx* ctx) {
  DD_CUDA_TRY(ctx, cudaFuncSetAttribute(dd_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_BYTES));
  dd_attn_tc_geometry(&ctx->cfg, ctx->sm_count, &ctx->as_blocks, &ctx->as_ppb, &ctx->as_max_parts);
  for (int s = 0; s < ctx->cfg.ring_depth; ++s) {
    const void* slot = ctx->ring + (size_t)s * ctx->slot_bytes;
    int rc = dd_attn_stream_make_map(ctx, slot, &ctx->as_tmap[s], DD_T);
    if (rc == DD_OK) rc = dd_attn_stream_make_map(ctx, slot, &ctx->tc_tmap[s], TC_TILE_TOKENS);
    if (rc != DD_OK) return rc;
  }
  return DD_OK;
}

int dd_launch_attn_tc(dd_ctx* ctx, const void* q, int slot, const int* idx, const int* ctx_len, void* out, float* out_lse,
                      cudaStream_t st, const void* k_new, const void* v_new) {
  const dd_config& c = ctx->cfg;
  const int total = c.batch * c.n_kv_heads * c.k_pages;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctx->as_blocks);
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = TC_SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  dd_pdl_attr(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  DD_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, dd_attn_tc_kernel, *reinterpret_cast<const CUtensorMap*>(&ctx->tc_tmap[slot]),
                                      *reinterpret_cast<const CUtensorMap*>(&ctx->as_tmap[slot]), (const __nv_bfloat16*)q, idx,
                                      ctx_len, (__nv_bfloat16*)out, out_lse, ctx->attn_part_o, ctx->attn_part_ml,
                                      ctx->attn_ticket, c.n_kv_heads, ctx->G, c.n_q_tokens, c.k_pages, total, ctx->as_ppb,
                                      ctx->as_max_parts, (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new,
                                      ctx->err_word, ctx->bulk_wait_ns));
  return DD_OK;
}

extern "C" int dd_test_attn_split(int kind, int batch, int n_kv_heads, int k_pages, int sm_count, int* n_blocks,
                                  int* pages_per_block, int* max_parts) {
  if ((kind != 0 && kind != 1) || batch < 1 || n_kv_heads < 1 || k_pages < 1 || sm_count < 1 || !n_blocks || !pages_per_block ||
      !max_parts)
    return DD_ERR_INVALID_ARG;
  dd_config c = {};
  c.batch = batch; c.n_kv_heads = n_kv_heads; c.k_pages = k_pages;
  if (kind == 0) dd_attn_stream_geometry(&c, sm_count, n_blocks, pages_per_block, max_parts);
  else dd_attn_tc_geometry(&c, sm_count, n_blocks, pages_per_block, max_parts);
  return DD_OK;
}
