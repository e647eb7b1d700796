// fp32 GEMM for CERB_F32 models: out[M][N] = X[M][K] . W[N][K]^T with plain FMA arithmetic
// (tensor cores would round the operands to tf32, which the fp32 contract does not allow).
#include "cerb_internal.cuh"

namespace cerb {

constexpr int TM = 64, TN = 64, TK = 16;

__global__ void __launch_bounds__(256) gemm_f32_kernel(const float* __restrict__ X, const float* __restrict__ W,
                                                       float* __restrict__ out, int M, int N, int K) {
  __shared__ float sx[TK][TM + 4];
  __shared__ float sw[TK][TN + 4];
  griddep_wait();
  griddep_launch();
  int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
  int tx = threadIdx.x % 16, ty = threadIdx.x / 16;     // tx -> n, ty -> m
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += TK) {
    for (int i = threadIdx.x; i < TM * TK; i += 256) {
      int r = i / TK, kk = i % TK;
      int m = m0 + r, k = k0 + kk;
      sx[kk][r] = (m < M && k < K) ? X[(size_t)m * K + k] : 0.f;
      int nn = n0 + r;
      sw[kk][r] = (nn < N && k < K) ? W[(size_t)nn * K + k] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = sx[kk][ty * 4 + i]; b[i] = sw[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  for (int i = 0; i < 4; ++i) {
    int m = m0 + ty * 4 + i;
    if (m >= M) continue;
    for (int j = 0; j < 4; ++j) {
      int nn = n0 + tx * 4 + j;
      if (nn < N) out[(size_t)m * N + nn] = acc[i][j];
    }
  }
}

int launch_gemm_f32(cerb_ctx* c, const float* X, const float* W, float* out, int M, int N, int K, cudaStream_t st) {
  dim3 grid((N + TN - 1) / TN, (M + TM - 1) / TM);
  launch_pdl(gemm_f32_kernel, grid, dim3(256), 0, st, X, W, out, M, N, K);
  CERB_LAUNCH_CHECK(c);
  return CERB_OK;
}

}  // namespace cerb
