/* A plain C consumer of the kb library: device memory through the CUDA runtime's C API, the
 * gate through kb_screen, records read back and checked.  Built and run by
 * tests/test_gpu_c_abi.py.  Three float candidates of N elements: an exact copy, a copy with
 * one element off by 0.5 at index 12345, a copy with a NaN at index 7. */
#include <cuda_runtime_api.h>
#include <math.h>
#include <stdio.h>
#include <string.h>
#include <stdlib.h>

#include "kb.h"

#define CHECK(x)                                               \
  do {                                                         \
    if ((x) != 0) {                                            \
      fprintf(stderr, "failed at line %d: %s\n", __LINE__, #x); \
      return 1;                                                \
    }                                                          \
  } while (0)

int main(void) {
  const uint64_t N = 3u * 4096u * 40u + 17u;
  float* h = (float*)malloc(N * sizeof(float));
  float *d_ref = 0, *d_c[3] = {0, 0, 0};
  kb_screen_result* d_out = 0;
  kb_screen_result out[3];
  kb_ctx* ctx = 0;
  kb_status dev_status = KB_OK;
  uint64_t i;
  int k;
  if (!h) return 1;
  for (i = 0; i < N; ++i) h[i] = (float)((i * 2654435761u) % 1000u) / 250.0f - 2.0f;
  CHECK(cudaMalloc((void**)&d_ref, N * sizeof(float)));
  CHECK(cudaMemcpy(d_ref, h, N * sizeof(float), cudaMemcpyHostToDevice));
  for (k = 0; k < 3; ++k) {
    float saved = 0.0f;
    uint64_t at = k == 1 ? 12345u : 7u;
    if (k > 0) {
      saved = h[at];
      h[at] = k == 1 ? saved + 0.5f : NAN;
    }
    CHECK(cudaMalloc((void**)&d_c[k], N * sizeof(float)));
    CHECK(cudaMemcpy(d_c[k], h, N * sizeof(float), cudaMemcpyHostToDevice));
    if (k > 0) h[at] = saved;
  }
  CHECK(cudaMalloc((void**)&d_out, sizeof out));
  CHECK(kb_ctx_create(0, &ctx));
  {
    const void* cands[3];
    cands[0] = d_c[0];
    cands[1] = d_c[1];
    cands[2] = d_c[2];
    CHECK(kb_screen(ctx, d_ref, cands, 3, N, KB_F32, 1e-3f, 1e-3f, 0, d_out, 0));
  }
  CHECK(kb_ctx_poll(ctx, 0, &dev_status));
  CHECK(dev_status);
  CHECK(cudaMemcpy(out, d_out, sizeof out, cudaMemcpyDeviceToHost));
  if (!(out[0].pass == 1 && out[0].mismatch_count == 0 && out[0].argmax_idx == 0 && out[0].max_abs_err == 0.0f)) {
    fprintf(stderr, "candidate 0: unexpected record\n");
    return 2;
  }
  if (!(out[1].pass == 0 && out[1].mismatch_count == 1 && out[1].argmax_idx == 12345 && out[1].max_abs_err == 0.5f)) {
    fprintf(stderr, "candidate 1: unexpected record\n");
    return 3;
  }
  if (!(out[2].pass == 0 && out[2].mismatch_count == 1 && out[2].nan_count == 1 && out[2].argmax_idx == 0)) {
    fprintf(stderr, "candidate 2: unexpected record\n");
    return 4;
  }
  /* the same tensors in two parts cut on a tile boundary, merged: the same records */
  {
    const uint64_t cut = 4096u * 50u;
    const uint64_t first[2] = {0u, cut};
    kb_screen_result *d_parts = 0, *d_merged = 0;
    kb_screen_result merged[3];
    const void* lo[3];
    const void* hi[3];
    CHECK(cudaMalloc((void**)&d_parts, 2 * sizeof out));
    CHECK(cudaMalloc((void**)&d_merged, sizeof out));
    for (k = 0; k < 3; ++k) {
      lo[k] = d_c[k];
      hi[k] = d_c[k] + cut;
    }
    CHECK(kb_screen(ctx, d_ref, lo, 3, cut, KB_F32, 1e-3f, 1e-3f, 0, d_parts, 0));
    CHECK(kb_screen(ctx, d_ref + cut, hi, 3, N - cut, KB_F32, 1e-3f, 1e-3f, 0, d_parts + 3, 0));
    CHECK(kb_merge_ranges(ctx, d_parts, 2, 3, first, d_merged, 0));
    CHECK(kb_ctx_poll(ctx, 0, &dev_status));
    CHECK(dev_status);
    CHECK(cudaMemcpy(merged, d_merged, sizeof merged, cudaMemcpyDeviceToHost));
    if (memcmp(merged, out, sizeof out) != 0) {
      fprintf(stderr, "merged parts differ from the whole range\n");
      return 5;
    }
    cudaFree(d_parts);
    cudaFree(d_merged);
  }
  CHECK(kb_ctx_destroy(ctx));
  printf("ok\n");
  return 0;
}
