/* A caller written in plain C: no torch, no C++ — only include/dd.h and the CUDA runtime for memory.
 * Builds landmarks, selects, gathers from pinned memory and attends; checks what can be checked without a
 * reference implementation: indices ascending and in range, the slot a bit copy of the selected pages, and
 * attention over constant values returning that constant. Exit code 0 = all checks passed. */
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "dd.h"
#include "dd_bench.h"   /* dd_slot_ptr: reads back what the gather wrote */

#define CHECK_DD(expr)                                                                          \
  do {                                                                                          \
    int rc__ = (expr);                                                                          \
    if (rc__ != DD_OK) {                                                                        \
      fprintf(stderr, "%s -> %d (%s): %s\n", #expr, rc__, dd_strerror(rc__), dd_last_error_message(ctx)); \
      return 1;                                                                                 \
    }                                                                                           \
  } while (0)
#define CHECK_CUDA(expr)                                                        \
  do {                                                                          \
    cudaError_t e__ = (expr);                                                   \
    if (e__ != cudaSuccess) {                                                   \
      fprintf(stderr, "%s -> %s\n", #expr, cudaGetErrorString(e__));            \
      return 1;                                                                 \
    }                                                                           \
  } while (0)

static uint16_t bf16_of(float f) {             /* truncation is fine for test data */
  uint32_t u;
  memcpy(&u, &f, 4);
  return (uint16_t)(u >> 16);
}

int main(void) {
  enum { B = 1, HKV = 2, HQ = 8, D = 128, T = 16, P = 64, K = 8, TQ = 2 };
  dd_ctx* ctx = NULL;
  dd_config cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.n_layers = 1; cfg.batch = B; cfg.n_q_heads = HQ; cfg.n_kv_heads = HKV; cfg.head_dim = D; cfg.page_tokens = T;
  cfg.max_pages = P; cfg.k_pages = K; cfg.n_q_tokens = TQ; cfg.ring_depth = 2;
  cudaStream_t s1, s2;
  CHECK_CUDA(cudaStreamCreate(&s1));
  CHECK_CUDA(cudaStreamCreate(&s2));
  cfg.compute_stream = s1; cfg.copy_stream = s2;
  CHECK_DD(dd_create(&cfg, &ctx));

  const size_t page_elems = 2 * T * D, store_elems = (size_t)B * HKV * P * page_elems;
  uint16_t* store = NULL;
  CHECK_CUDA(cudaHostAlloc((void**)&store, store_elems * 2, cudaHostAllocPortable | cudaHostAllocMapped));
  uint32_t lcg = 12345u;
  const float vconst = 0.75f;
  for (size_t pg = 0; pg < (size_t)B * HKV * P; ++pg) {
    for (int i = 0; i < T * D; ++i) {          /* keys: pseudo-random in [-1, 1) */
      lcg = lcg * 1664525u + 1013904223u;
      store[pg * page_elems + i] = bf16_of((float)(lcg >> 8) / 8388608.0f - 1.0f);
    }
    for (int i = 0; i < T * D; ++i) store[pg * page_elems + T * D + i] = bf16_of(vconst);   /* values: constant */
  }
  int h_ctx[B] = {P * T - 5}, h_np[B] = {P};
  int *d_ctx, *d_np, *d_idx;
  uint16_t *d_lm, *d_q, *d_out;
  CHECK_CUDA(cudaMalloc((void**)&d_ctx, sizeof(h_ctx)));
  CHECK_CUDA(cudaMalloc((void**)&d_np, sizeof(h_np)));
  CHECK_CUDA(cudaMalloc((void**)&d_idx, sizeof(int) * B * HKV * K));
  CHECK_CUDA(cudaMalloc((void**)&d_lm, (size_t)B * HKV * P * D * 2));
  CHECK_CUDA(cudaMalloc((void**)&d_q, (size_t)B * TQ * HQ * D * 2));
  CHECK_CUDA(cudaMalloc((void**)&d_out, (size_t)B * TQ * HQ * D * 2));
  CHECK_CUDA(cudaMemcpy(d_ctx, h_ctx, sizeof(h_ctx), cudaMemcpyHostToDevice));
  CHECK_CUDA(cudaMemcpy(d_np, h_np, sizeof(h_np), cudaMemcpyHostToDevice));
  uint16_t h_q[B * TQ * HQ * D];
  for (int i = 0; i < B * TQ * HQ * D; ++i) {
    lcg = lcg * 1664525u + 1013904223u;
    h_q[i] = bf16_of((float)(lcg >> 8) / 8388608.0f - 1.0f);
  }
  CHECK_CUDA(cudaMemcpy(d_q, h_q, sizeof(h_q), cudaMemcpyHostToDevice));

  CHECK_DD(dd_build_landmarks(ctx, store, d_ctx, d_lm, s1));
  CHECK_DD(dd_select_topk(ctx, d_q, 1, d_lm, d_np, d_idx, NULL, s1));
  CHECK_DD(dd_gather_kv_from_host(ctx, store, d_idx, d_np, 0, s1));
  CHECK_DD(dd_sparse_decode_attn(ctx, d_q, 0, d_idx, d_ctx, d_out, NULL, s1));
  int code = -1, detail = -1;
  CHECK_DD(dd_device_error(ctx, 30.0, &code, &detail));
  if (code != DD_OK) { fprintf(stderr, "device error %d (%d)\n", code, detail); return 1; }

  int h_idx[B * HKV * K];
  CHECK_CUDA(cudaMemcpy(h_idx, d_idx, sizeof(h_idx), cudaMemcpyDeviceToHost));
  for (int u = 0; u < B * HKV; ++u)
    for (int j = 0; j < K; ++j) {
      const int p = h_idx[u * K + j];
      if (p < 0 || p >= P || (j > 0 && p <= h_idx[u * K + j - 1])) { fprintf(stderr, "bad index set\n"); return 1; }
    }
  void* slot_dev = NULL;
  CHECK_DD(dd_slot_ptr(ctx, 0, &slot_dev));
  const size_t slot_bytes = dd_slot_bytes(&cfg);
  if (slot_bytes != (size_t)B * HKV * K * page_elems * 2) { fprintf(stderr, "slot size\n"); return 1; }
  uint16_t* slot = (uint16_t*)malloc(slot_bytes);
  CHECK_CUDA(cudaMemcpy(slot, slot_dev, slot_bytes, cudaMemcpyDeviceToHost));
  for (int u = 0; u < B * HKV; ++u)
    for (int j = 0; j < K; ++j) {
      const uint16_t* src = store + ((size_t)u * P + h_idx[u * K + j]) * page_elems;
      const uint16_t* dk = slot + ((size_t)u * 2 * K + j) * T * D;
      const uint16_t* dv = dk + (size_t)K * T * D;
      if (memcmp(dk, src, T * D * 2) || memcmp(dv, src + T * D, T * D * 2)) { fprintf(stderr, "slot is not a bit copy\n"); return 1; }
    }
  uint16_t h_out[B * TQ * HQ * D];
  CHECK_CUDA(cudaMemcpy(h_out, d_out, sizeof(h_out), cudaMemcpyDeviceToHost));
  for (int i = 0; i < B * TQ * HQ * D; ++i)
    if (h_out[i] != bf16_of(vconst)) { fprintf(stderr, "attention over constant values gave %04x at %d\n", h_out[i], i); return 1; }

  /* pageable memory must be refused before anything is launched */
  uint16_t* pageable = (uint16_t*)malloc(store_elems * 2);
  if (dd_gather_kv_from_host(ctx, pageable, d_idx, d_np, 0, s1) != DD_ERR_NOT_PINNED) { fprintf(stderr, "pageable memory accepted\n"); return 1; }
  free(pageable);
  free(slot);
  CHECK_DD(dd_destroy(ctx));
  cudaFreeHost(store);
  printf("C ABI OK: select -> gather -> attention from plain C\n");
  return 0;
}
