/*
 * A plain C99 caller of libssa (no Python, no torch): reads one small problem
 * from a file, runs ssa_spans_to_index + ssa_decode_attn_sparse and
 * ssa_decode_attn_dense through the C ABI with memory from cudaMalloc, and
 * writes the results to a file.  Used by tests/test_gpu_c_client.py, which
 * prepares the input and checks the output against the oracle.
 *
 * Input file (little endian): int32 B, H, D, T, dtype (0 f16 / 1 bf16),
 * index_stride, n_spans; int32 ctx_lens[B]; int32 span_offsets[B+1];
 * int32 spans[2*n_spans]; uint16 q[B*H*D]; uint16 k[B*H*T*D]; uint16 v[B*H*T*D].
 * Output file: int32 counts[B]; int32 index[B*index_stride]; uint32 status;
 * float out_sparse[B*H*D]; float lse_sparse[B*H]; float out_dense[B*H*D].
 */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "ssa.h"

#define CHECK_CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { \
  fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_)); return 3; } } while (0)
#define CHECK_SSA(x) do { int32_t s_ = (x); if (s_ != SSA_OK) { \
  fprintf(stderr, "%s: %s\n", #x, ssa_status_string(s_)); return 4; } } while (0)

static void* upload(const void* host, size_t bytes) {
  void* dev = NULL;
  if (cudaMalloc(&dev, bytes ? bytes : 16) != cudaSuccess) return NULL;
  if (bytes && cudaMemcpy(dev, host, bytes, cudaMemcpyHostToDevice) != cudaSuccess) return NULL;
  return dev;
}

int main(int argc, char** argv) {
  if (argc != 3) { fprintf(stderr, "usage: %s input output\n", argv[0]); return 2; }
  FILE* f = fopen(argv[1], "rb");
  if (!f) { perror(argv[1]); return 2; }
  int32_t hdr[7];
  if (fread(hdr, sizeof(int32_t), 7, f) != 7) return 2;
  const int32_t B = hdr[0], H = hdr[1], D = hdr[2], T = hdr[3], dtype = hdr[4], stride = hdr[5], n_spans = hdr[6];
  const size_t nq = (size_t)B * H * D, nkv = (size_t)B * H * T * D;
  int32_t* ctx = malloc(sizeof(int32_t) * B);
  int32_t* offs = malloc(sizeof(int32_t) * (B + 1));
  int32_t* spans = malloc(sizeof(int32_t) * 2 * (n_spans ? n_spans : 1));
  uint16_t* q = malloc(2 * nq);
  uint16_t* k = malloc(2 * nkv);
  uint16_t* v = malloc(2 * nkv);
  if (!ctx || !offs || !spans || !q || !k || !v) return 2;
  if (fread(ctx, 4, B, f) != (size_t)B || fread(offs, 4, B + 1, f) != (size_t)B + 1 ||
      fread(spans, 4, 2 * (size_t)n_spans, f) != 2 * (size_t)n_spans || fread(q, 2, nq, f) != nq ||
      fread(k, 2, nkv, f) != nkv || fread(v, 2, nkv, f) != nkv)
    return 2;
  fclose(f);

  void* d_ctx = upload(ctx, 4 * (size_t)B);
  void* d_offs = upload(offs, 4 * ((size_t)B + 1));
  void* d_spans = upload(spans, 8 * (size_t)(n_spans ? n_spans : 1));
  void* d_q = upload(q, 2 * nq);
  void* d_k = upload(k, 2 * nkv);
  void* d_v = upload(v, 2 * nkv);
  void *d_index = NULL, *d_counts = NULL, *d_status = NULL, *d_out = NULL, *d_lse = NULL, *d_ws = NULL;
  if (!d_ctx || !d_offs || !d_spans || !d_q || !d_k || !d_v) return 3;
  CHECK_CUDA(cudaMalloc(&d_index, 4 * (size_t)B * stride));
  CHECK_CUDA(cudaMalloc(&d_counts, 4 * (size_t)B));
  CHECK_CUDA(cudaMalloc(&d_status, 4));
  CHECK_CUDA(cudaMemset(d_status, 0, 4));
  CHECK_CUDA(cudaMalloc(&d_out, 4 * nq));
  CHECK_CUDA(cudaMalloc(&d_lse, 4 * (size_t)B * H));

  ssa_attn_desc desc;
  memset(&desc, 0, sizeof desc);
  desc.B = B; desc.H = H; desc.H_kv = H; desc.D = D; desc.max_ctx = T;
  desc.kv_dtype = dtype ? SSA_BF16 : SSA_F16;
  desc.out_dtype = SSA_F32;
  desc.scale = 0.0f;                                   /* 1 / sqrt(D) */
  desc.q_stride_b = (int64_t)H * D; desc.q_stride_h = D;
  desc.k_stride_b = (int64_t)H * T * D; desc.k_stride_h = (int64_t)T * D; desc.k_stride_t = D;
  desc.v_stride_b = desc.k_stride_b; desc.v_stride_h = desc.k_stride_h; desc.v_stride_t = D;
  desc.o_stride_b = (int64_t)H * D; desc.o_stride_h = D;

  size_t ws_bytes = ssa_decode_workspace_bytes(&desc, stride);
  const size_t ws_dense = ssa_decode_workspace_bytes(&desc, T);
  if (ws_dense > ws_bytes) ws_bytes = ws_dense;
  if (ws_bytes == 0) { fprintf(stderr, "descriptor rejected\n"); return 4; }
  CHECK_CUDA(cudaMalloc(&d_ws, ws_bytes));

  float* out_sparse = malloc(4 * nq);
  float* lse = malloc(4 * (size_t)B * H);
  float* out_dense = malloc(4 * nq);
  int32_t* counts = malloc(4 * (size_t)B);
  int32_t* index = malloc(4 * (size_t)B * stride);
  uint32_t status = 0;
  if (!out_sparse || !lse || !out_dense || !counts || !index) return 2;

  CHECK_SSA(ssa_spans_to_index(d_offs, d_spans, d_ctx, B, d_index, stride, d_counts, d_status, NULL));
  CHECK_SSA(ssa_decode_attn_sparse(&desc, d_q, d_k, d_v, d_ctx, d_index, stride, d_counts, stride, d_out, d_lse,
                                   d_ws, ws_bytes, d_status, NULL));
  CHECK_CUDA(cudaDeviceSynchronize());
  CHECK_CUDA(cudaMemcpy(out_sparse, d_out, 4 * nq, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(lse, d_lse, 4 * (size_t)B * H, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(counts, d_counts, 4 * (size_t)B, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(index, d_index, 4 * (size_t)B * stride, cudaMemcpyDeviceToHost));
  CHECK_SSA(ssa_decode_attn_dense(&desc, d_q, d_k, d_v, d_ctx, d_out, d_lse, d_ws, ws_bytes, d_status, NULL));
  CHECK_CUDA(cudaDeviceSynchronize());
  CHECK_CUDA(cudaMemcpy(out_dense, d_out, 4 * nq, cudaMemcpyDeviceToHost));
  CHECK_CUDA(cudaMemcpy(&status, d_status, 4, cudaMemcpyDeviceToHost));

  f = fopen(argv[2], "wb");
  if (!f) { perror(argv[2]); return 2; }
  fwrite(counts, 4, B, f);
  fwrite(index, 4, (size_t)B * stride, f);
  fwrite(&status, 4, 1, f);
  fwrite(out_sparse, 4, nq, f);
  fwrite(lse, 4, (size_t)B * H, f);
  fwrite(out_dense, 4, nq, f);
  fclose(f);
  printf("libssa version %d, %llu kernels launched\n", ssa_version(), (unsigned long long)ssa_launch_count());
  return 0;
}
