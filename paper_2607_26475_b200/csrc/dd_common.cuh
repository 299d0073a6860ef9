// Shared declarations of the CUDA sources: the context, error plumbing and small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "../../include/dd.h"
#include "../../include/dd_bench.h"

constexpr int DD_D = 128;          // head_dim the kernels are written for
constexpr int DD_T = 16;           // tokens per page
constexpr int DD_ROW_BYTES = DD_D * 2;
constexpr int DD_HALF_PAGE_BYTES = DD_T * DD_ROW_BYTES;   // K (or V) part of a page: 4 KiB
constexpr int DD_PAGE_BYTES = 2 * DD_HALF_PAGE_BYTES;     // 8 KiB
constexpr int DD_MAX_RING = 8;
constexpr int DD_SCORE_TILE = 128; // pages scored by one thread block
constexpr int DD_STAGE_LISTS = 8;  // page-locked descriptor buffers of the staged gather (host may run this far ahead)

struct dd_ctx {
  dd_config cfg;
  int device;
  int sm_count;
  int G;                 // query heads per KV head
  int R;                 // landmark chunks per page (1 = one landmark per page)
  int n_rows;            // Tq * G query rows that share one KV head
  int score_tiles;       // ceil(P / DD_SCORE_TILE)
  int attn_splits;       // resolved blocks per (request, KV head)
  int attn_cluster;      // blocks per thread-block cluster (divides attn_splits)
  int attn_stream;       // which attention kernel serves the context's calls: 0 split-KV, 1 streaming, 2 tcgen05
  cudaEvent_t as_fence;  // timing-enabled event recorded behind the streaming kernel inside the layer step (see dd_api.cu)
  int as_blocks, as_ppb, as_max_parts;   // streaming kernel: grid, pages per block, partials per unit
  struct alignas(64) { unsigned char bytes[128]; } as_tmap[DD_MAX_RING];   // tensor map of every ring slot, page boxes
  struct alignas(64) { unsigned char bytes[128]; } tc_tmap[DD_MAX_RING];   // the same with boxes of a tile (128 rows)
  int sel_cluster;       // blocks per cluster of the fused selection kernel; 0 = two-kernel path
  int sel_ppc;           // pages per block of the fused selection
  int sel_smem_bytes;
  int sel_stages;        // tiles per warp in the scoring ring of the fused selection
  int sel_logits_global; // 1: the fused selection keeps its logits in score_s (two buffers) instead of shared memory
  size_t slot_bytes;
  // scratch (device)
  float* score_s;        // [2][B][Hkv][P*R][G] scaled logits (second buffer: selections on the selection stream)
  float2* score_part;    // [B][Hq][score_tiles] per-tile (max, sum exp)
  uint32_t* topk_keys;   // [B][Hkv][P] order-preserving keys when a request does not fit shared memory
  float* attn_part_o;    // [B][Hkv][S][8][128] unnormalised partial outputs
  float2* attn_part_ml;  // [B][Hkv][S][8] (max, sum) in the log2 domain
  unsigned int* attn_ticket;  // [B*Hkv] arrival counters, zero between launches
  int* idx_tab;          // [2][L][B][Hkv][k]
  int* err_word;         // [0] code, [1] detail, [2..3] device-visible address of err_host
  int* err_host;         // page-locked mirror [2] that reporting kernels also write (read without synchronising)
  int host_err[2];       // errors found by host-side index checks (staged gather)
  __nv_bfloat16* stage_q;    // [L][B][Tq][Hq][d] device staging of dd_decode_step_host
  __nv_bfloat16* stage_out;  // [L][B][Tq][Hq][d]
  // miss correction
  int* idx_true;         // [B][Hkv][k] true index of the layer being corrected
  int* idx_merged;       // [D][B][Hkv][k] page held by every position of a slot after the repair
  int2* fix_stage;       // [D][B][Hkv][k] per-unit (victim position, missing page) before pairing
  int4* fix_list;        // [D][B*Hkv*k] compact (unit, position, page, 0)
  unsigned int* fix_count;          // [D]
  unsigned long long* miss_stats;   // [2]: missing pages, selected pages
  char* ring;
  bool own_ring;
  // events of the pipelined path
  cudaEvent_t ready[DD_MAX_RING];
  cudaEvent_t released[DD_MAX_RING];
  bool released_recorded[DD_MAX_RING];
  cudaEvent_t* sel_done;  // [L]
  cudaEvent_t q_ready;    // start of a layer step on the compute stream (the select stream starts from it)
  cudaEvent_t fix_ready[DD_MAX_RING];    // fix list of the slot written (compute stream)
  cudaEvent_t urgent_done[DD_MAX_RING];  // missing pages of the slot fetched (urgent stream)
  // bound tables
  const void** landmarks;  // [L]
  const void** host_kv;    // [L] device-visible addresses
  const void** host_kv_orig;  // [L] the pointers as given to dd_bind (sources of copy-engine copies)
  const int* n_pages;
  const int* ctx_len;
  bool bound, primed;
  long long next_call;     // step * L + layer expected by dd_decode_layer_step
  bool in_flight;          // a pipelined call has begun to enqueue work (a failure now needs dd_prime again)
  // bulk gather engine: limit of its bounded waits, and the test hook that makes one run out
  unsigned long long bulk_wait_ns;
  int bulk_inflate;
  // staged gather (DD_GATHER_STAGED)
  int stage_min_run, stage_block;
  int* idx_host;           // page-locked [2][L][B*Hkv*k]: every selected set, copied right after its selection
  cudaEvent_t* idx_copied; // [L] that copy is complete
  int* n_pages_host;       // [B]
  char* staging;           // device landing zone of the copy engine, staging_pages pages of 8 KiB
  size_t staging_pages;
  int* list_host[DD_STAGE_LISTS];   // page-locked: [staging_pages] staged page -> slot item (or -1), then [B*Hkv*k] straggler items
  const int* list_dev[DD_STAGE_LISTS];
  cudaEvent_t list_free[DD_STAGE_LISTS];
  bool list_used[DD_STAGE_LISTS];
  long long list_next;
  long long* copy_plan;    // [3 * B*Hkv*k] (source page, staging page, pages) of the gather being issued
  cudaStream_t aux_stream; // library-owned: the zero-copy kernel of the short runs, next to the copy engine
  cudaEvent_t aux_fork, aux_join;
  unsigned long long gstats[DD_GATHER_STATS_FIELDS];
  // optional timeline of the pipelined calls: DD_TRACE_FIELDS timing events per layer step
  cudaEvent_t* trace_ev;
  cudaEvent_t trace_origin;
  int trace_cap, trace_n;
  bool trace_on;
  char errmsg[512];
};

int dd_fail(dd_ctx* ctx, int code, const char* fmt, ...);
#define DD_CUDA_TRY(ctx, expr)                                                                  \
  do {                                                                                          \
    cudaError_t e__ = (expr);                                                                   \
    if (e__ != cudaSuccess) return dd_fail((ctx), DD_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)

// Programmatic dependent launch (sm_90+): a kernel launched with dd_pdl_attr() may be scheduled while the previous
// kernel of its stream is still draining (its blocks become resident as that kernel's blocks leave). Such a kernel
// calls dd_grid_dependency_wait() before its first access to global memory: the wait returns once every earlier
// kernel of the stream has completed and its writes are visible, so the ordering a stream gives is unchanged. Our
// kernels never signal their dependents early: measured, an early signal packs the next launch's blocks onto the SMs
// that free up first and slows it. Saves 1.5-2 us per launch behind another kernel (B200, events around 40 launches).
#ifdef __CUDACC__
__device__ __forceinline__ void dd_grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif
static inline void dd_pdl_attr(cudaLaunchAttribute* a) {
  a->id = cudaLaunchAttributeProgrammaticStreamSerialization;
  a->val.programmaticStreamSerializationAllowed = 1;
}

// Launchers implemented next to their kernels; all asynchronous on `st`.
int dd_launch_build_landmarks(dd_ctx* ctx, const void* kv_dev, const int* ctx_len, void* landmarks, cudaStream_t st);
int dd_launch_select(dd_ctx* ctx, const void* q, int q_token, int q_tokens_in_tensor, const void* landmarks,
                     const int* n_pages, int* out_idx, float* out_scores, cudaStream_t st, const int* ctx_len = nullptr);
int dd_launch_gather(dd_ctx* ctx, const void* kv_dev, const int* idx, const int* n_pages, char* slot, cudaStream_t st);
// Staged gather of one layer: idx_h is the index set on the host (already complete), kv_src the store as given by
// the caller; copies run on `st`, the short runs on the context's auxiliary stream (joined into `st` before return).
int dd_launch_gather_staged(dd_ctx* ctx, const void* kv_src, const void* kv_dev, const int* idx_h, const int* idx_dev,
                            const int* n_pages_h, const int* n_pages_dev, char* slot, cudaStream_t st);
int dd_wait_index_copy(dd_ctx* ctx, int layer);   // host wait (bounded) until layer's newest index set is on the host
int dd_launch_attn(dd_ctx* ctx, const void* q, const char* slot, const int* idx, const int* ctx_len, void* out,
                   float* out_lse, cudaStream_t st, const void* k_new = nullptr, const void* v_new = nullptr);
int dd_launch_attn_loads_only(dd_ctx* ctx, const char* slot, cudaStream_t st);
void dd_attn_stream_geometry(const dd_config* c, int sm_count, int* n_blocks, int* ppb, int* max_parts);
int dd_attn_stream_setup(dd_ctx* ctx);
int dd_attn_stream_make_map(dd_ctx* ctx, const void* slot, void* map_out, int box_rows);
void dd_attn_tc_geometry(const dd_config* c, int sm_count, int* n_blocks, int* ppb, int* max_parts);
int dd_attn_tc_setup(dd_ctx* ctx);
int dd_launch_attn_tc(dd_ctx* ctx, const void* q, int slot, const int* idx, const int* ctx_len, void* out, float* out_lse,
                      cudaStream_t st, const void* k_new, const void* v_new);
int dd_launch_attn_stream(dd_ctx* ctx, const void* q, int slot, const int* idx, const int* ctx_len, void* out,
                          float* out_lse, cudaStream_t st, const void* k_new, const void* v_new, bool probe);
int dd_launch_select_loads_only(dd_ctx* ctx, const void* landmarks, const int* n_pages, cudaStream_t st);
int dd_launch_diff(dd_ctx* ctx, const int* pred, const int* truth, int slot, int* merged, cudaStream_t st);
int dd_launch_gather_fix(dd_ctx* ctx, const void* kv_dev, int slot, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------
#ifdef __CUDACC__

// First error wins; later ones are dropped. Never traps. The winner also writes the page-locked mirror whose
// address the host stored behind the two words.
__device__ __forceinline__ void dd_report(int* err_word, int code, int detail) {
  if (atomicCAS(err_word, 0, code) == 0) {
    err_word[1] = detail;
    volatile int* mirror = *reinterpret_cast<int* volatile*>(err_word + 2);
    if (mirror) {
      mirror[1] = detail;
      __threadfence_system();
      mirror[0] = code;
    }
  }
}

// 16-byte read-only load that does not allocate in L1 (every byte on this path is used once per block).
__device__ __forceinline__ uint4 dd_ld_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// 16-byte store. Kept as volatile asm so that the compiler cannot sink it between the loads of a
// batch: all loads of a batch are in flight before the first store waits on one.
__device__ __forceinline__ void dd_st_v4(void* p, const uint4& v) {
  asm volatile("st.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void dd_mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                            uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// (m, l) pairs of a running soft-max: l counts exp(x - m). Safe when either side is empty (m = -inf).
__device__ __forceinline__ void dd_ml_merge(float& m, float& l, float m2, float l2, bool base2) {
  float mn = fmaxf(m, m2);
  if (mn == -INFINITY) { l = 0.f; return; }
  float a = base2 ? exp2f(m - mn) : expf(m - mn);
  float b = base2 ? exp2f(m2 - mn) : expf(m2 - mn);
  l = l * a + l2 * b;
  m = mn;
}

#endif  // __CUDACC__
