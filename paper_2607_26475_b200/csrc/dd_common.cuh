// Shared declarations of the CUDA sources: the context, error plumbing and small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "../../include/dd.h"

constexpr int DD_D = 128;          // head_dim the kernels are written for
constexpr int DD_T = 16;           // tokens per page
constexpr int DD_ROW_BYTES = DD_D * 2;
constexpr int DD_HALF_PAGE_BYTES = DD_T * DD_ROW_BYTES;   // K (or V) part of a page: 4 KiB
constexpr int DD_PAGE_BYTES = 2 * DD_HALF_PAGE_BYTES;     // 8 KiB
constexpr int DD_MAX_RING = 8;
constexpr int DD_SCORE_TILE = 128; // pages scored by one thread block

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
  int sel_cluster;       // blocks per cluster of the fused selection kernel; 0 = two-kernel path
  int sel_ppc;           // pages per block of the fused selection
  int sel_smem_bytes;
  size_t slot_bytes;
  // scratch (device)
  float* score_s;        // [B][Hkv][P][G] scaled logits
  float2* score_part;    // [B][Hq][score_tiles] per-tile (max, sum exp)
  uint32_t* topk_keys;   // [B][Hkv][P] order-preserving keys when a request does not fit shared memory
  float* attn_part_o;    // [B][Hkv][S][8][128] unnormalised partial outputs
  float2* attn_part_ml;  // [B][Hkv][S][8] (max, sum) in the log2 domain
  unsigned int* attn_ticket;  // [B*Hkv] arrival counters, zero between launches
  int* idx_tab;          // [2][L][B][Hkv][k]
  int* err_word;         // [2]: code, detail
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
  const int* n_pages;
  const int* ctx_len;
  bool bound, primed;
  long long next_call;     // step * L + layer expected by dd_decode_layer_step
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

// Launchers implemented next to their kernels; all asynchronous on `st`.
int dd_launch_build_landmarks(dd_ctx* ctx, const void* kv_dev, const int* ctx_len, void* landmarks, cudaStream_t st);
int dd_launch_select(dd_ctx* ctx, const void* q, int q_token, int q_tokens_in_tensor, const void* landmarks,
                     const int* n_pages, int* out_idx, float* out_scores, cudaStream_t st, const int* ctx_len = nullptr);
int dd_launch_gather(dd_ctx* ctx, const void* kv_dev, const int* idx, const int* n_pages, char* slot, cudaStream_t st);
int dd_launch_attn(dd_ctx* ctx, const void* q, const char* slot, const int* idx, const int* ctx_len, void* out,
                   float* out_lse, cudaStream_t st, const void* k_new = nullptr, const void* v_new = nullptr);
int dd_launch_attn_loads_only(dd_ctx* ctx, const char* slot, cudaStream_t st);
int dd_launch_select_loads_only(dd_ctx* ctx, const void* landmarks, const int* n_pages, cudaStream_t st);
int dd_launch_diff(dd_ctx* ctx, const int* pred, const int* truth, int slot, int* merged, cudaStream_t st);
int dd_launch_gather_fix(dd_ctx* ctx, const void* kv_dev, int slot, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------
#ifdef __CUDACC__

// First error wins; later ones are dropped. Never traps.
__device__ __forceinline__ void dd_report(int* err_word, int code, int detail) {
  if (atomicCAS(err_word, 0, code) == 0) err_word[1] = detail;
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

// Optional per-block timeline for tuning (compile with -DDD_TRACE; never in the shipped library): mark i of
// block (x, y, z) is the global nanosecond timer when thread 0 passed it; <name>_read copies the table out.
#ifdef DD_TRACE
#define DD_TRACE_DECLARE(name)                                                                       \
  __device__ unsigned long long name[1 << 16][8];                                                    \
  extern "C" int name##_read(unsigned long long* host, size_t bytes) {                               \
    return (int)cudaMemcpyFromSymbol(host, name, bytes);                                             \
  }
#define DD_TRACE_MARK_IN(name, i)                                                                    \
  do {                                                                                               \
    if (threadIdx.x == 0) {                                                                          \
      unsigned long long t__;                                                                        \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t__));                                        \
      name[(blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x][i] = t__;                 \
    }                                                                                                \
  } while (0)
#else
#define DD_TRACE_DECLARE(name)
#define DD_TRACE_MARK_IN(name, i)
#endif

#endif  // __CUDACC__
