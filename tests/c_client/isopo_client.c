/* A caller of the library written in plain C: no Python, no PyTorch.  It reads one layer problem from a file,
 * runs the three calls of the per-layer path (K_ij = <G_i, G_j>; (K + lambda I) c = A, Sec. 3; dW = sum_i c_i G_i)
 * on device buffers it allocates itself with the CUDA runtime, and writes K, c and dW to another file.
 *
 * Input file (little endian):  int64 T, d_in, d_out, B, path;  double lambda;  int64 off[B+1];
 *                              float32 X[T*d_in], dY[T*d_out], A[B]
 * Output file:                 int32 info;  float32 K[B*B], c[B], dW[d_out*d_in]
 * Exit code 0 on success; otherwise the failing call and the library's message are printed to stderr. */
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include <cuda_runtime_api.h>

#include "isopo.h"

#define CUDA_TRY(call)                                                                   \
  do {                                                                                   \
    cudaError_t e_ = (call);                                                             \
    if (e_ != cudaSuccess) {                                                             \
      fprintf(stderr, "%s: %s\n", #call, cudaGetErrorString(e_));                        \
      return 2;                                                                          \
    }                                                                                    \
  } while (0)
#define ISOPO_TRY(call)                                                                  \
  do {                                                                                   \
    isopo_status s_ = (call);                                                            \
    if (s_ != ISOPO_OK) {                                                                \
      fprintf(stderr, "%s: %s (%s)\n", #call, isopo_status_string(s_), isopo_last_cuda_error()); \
      return 3;                                                                          \
    }                                                                                    \
  } while (0)

static int read_exact(FILE* f, void* dst, size_t bytes) { return fread(dst, 1, bytes, f) == bytes ? 0 : 1; }

int main(int argc, char** argv) {
  int64_t hdr[5];
  double lambda;
  int64_t* off;
  float *X, *dY, *A, *K, *c, *dW;
  float *dX, *ddY, *dA, *dK, *dc, *ddW;
  void *ws, *ws_raw;
  int32_t* dinfo;
  int32_t info = 0;
  size_t ws_bytes, nX, nY, nW;
  int64_t T;
  int d_in, d_out, B;
  isopo_path path;
  FILE* f;
  if (argc != 3) {
    fprintf(stderr, "usage: %s problem.bin result.bin\n", argv[0]);
    return 1;
  }
  f = fopen(argv[1], "rb");
  if (!f || read_exact(f, hdr, sizeof hdr) || read_exact(f, &lambda, sizeof lambda)) return 1;
  T = hdr[0]; d_in = (int)hdr[1]; d_out = (int)hdr[2]; B = (int)hdr[3]; path = (isopo_path)hdr[4];
  nX = (size_t)T * (size_t)d_in; nY = (size_t)T * (size_t)d_out; nW = (size_t)d_in * (size_t)d_out;
  off = (int64_t*)malloc(sizeof(int64_t) * (size_t)(B + 1));
  X = (float*)malloc(sizeof(float) * nX);
  dY = (float*)malloc(sizeof(float) * nY);
  A = (float*)malloc(sizeof(float) * (size_t)B);
  K = (float*)malloc(sizeof(float) * (size_t)B * (size_t)B);
  c = (float*)malloc(sizeof(float) * (size_t)B);
  dW = (float*)malloc(sizeof(float) * nW);
  if (!off || !X || !dY || !A || !K || !c || !dW) return 1;
  if (read_exact(f, off, sizeof(int64_t) * (size_t)(B + 1)) || read_exact(f, X, sizeof(float) * nX) ||
      read_exact(f, dY, sizeof(float) * nY) || read_exact(f, A, sizeof(float) * (size_t)B))
    return 1;
  fclose(f);

  ws_bytes = isopo_workspace_bytes(ISOPO_F32, T, d_in, d_out, B, path);
  if (ws_bytes == 0) {
    fprintf(stderr, "isopo_workspace_bytes: invalid sizes\n");
    return 3;
  }
  CUDA_TRY(cudaMalloc((void**)&dX, sizeof(float) * nX));
  CUDA_TRY(cudaMalloc((void**)&ddY, sizeof(float) * nY));
  CUDA_TRY(cudaMalloc((void**)&dA, sizeof(float) * (size_t)B));
  CUDA_TRY(cudaMalloc((void**)&dK, sizeof(float) * (size_t)B * (size_t)B));
  CUDA_TRY(cudaMalloc((void**)&dc, sizeof(float) * (size_t)B));
  CUDA_TRY(cudaMalloc((void**)&ddW, sizeof(float) * nW));
  /* the workspace must start on a 1024-byte boundary; cudaMalloc promises 256: allocate 1024 more and round up */
  CUDA_TRY(cudaMalloc(&ws_raw, ws_bytes + 1024));
  ws = (void*)(((uintptr_t)ws_raw + 1023u) & ~(uintptr_t)1023u);
  CUDA_TRY(cudaMalloc((void**)&dinfo, sizeof(int32_t)));
  CUDA_TRY(cudaMemcpy(dX, X, sizeof(float) * nX, cudaMemcpyHostToDevice));
  CUDA_TRY(cudaMemcpy(ddY, dY, sizeof(float) * nY, cudaMemcpyHostToDevice));
  CUDA_TRY(cudaMemcpy(dA, A, sizeof(float) * (size_t)B, cudaMemcpyHostToDevice));
  CUDA_TRY(cudaMemset(dinfo, 0, sizeof(int32_t)));

  /* the three calls, on the default stream */
  ISOPO_TRY(isopo_layer_gram(dX, ddY, ISOPO_F32, T, d_in, d_out, off, B, path, dK, ws, ws_bytes, dinfo, NULL));
  ISOPO_TRY(isopo_transform_advantages(dK, dA, B, ISOPO_VAR_INTERACTING, (float)lambda, NULL, dc, dinfo, NULL));
  ISOPO_TRY(isopo_weight_grad(dX, ddY, ISOPO_F32, T, d_in, d_out, dc, off, B, path, ddW, 0.0f, ws, ws_bytes, dinfo, NULL));
  CUDA_TRY(cudaDeviceSynchronize());

  CUDA_TRY(cudaMemcpy(&info, dinfo, sizeof(int32_t), cudaMemcpyDeviceToHost));
  CUDA_TRY(cudaMemcpy(K, dK, sizeof(float) * (size_t)B * (size_t)B, cudaMemcpyDeviceToHost));
  CUDA_TRY(cudaMemcpy(c, dc, sizeof(float) * (size_t)B, cudaMemcpyDeviceToHost));
  CUDA_TRY(cudaMemcpy(dW, ddW, sizeof(float) * nW, cudaMemcpyDeviceToHost));
  f = fopen(argv[2], "wb");
  if (!f) return 1;
  fwrite(&info, sizeof info, 1, f);
  fwrite(K, sizeof(float), (size_t)B * (size_t)B, f);
  fwrite(c, sizeof(float), (size_t)B, f);
  fwrite(dW, sizeof(float), nW, f);
  fclose(f);
  cudaFree(dX); cudaFree(ddY); cudaFree(dA); cudaFree(dK); cudaFree(dc); cudaFree(ddW); cudaFree(ws_raw); cudaFree(dinfo);
  free(off); free(X); free(dY); free(A); free(K); free(c); free(dW);
  return 0;
}
