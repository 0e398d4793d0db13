// CUDA-core GEMM out = A W^T (+ bias, activation, residual): the float32 path of the
// library and the validation path for the tensor-core kernel.  64x64 tile, 4x4 per thread,
// fp32 FMA accumulation in a fixed order (no TF32).
#include "common.cuh"
#include "kernels.h"

namespace zo {

template <typename T>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T* __restrict__ A, int lda, const T* __restrict__ W, int M, int N, int K,
                 void* out, int ldo, int out_f32, const T* __restrict__ bias,
                 const T* res, int ldr, int res_mod, int act) {
  __shared__ float As[16][64 + 4];
  __shared__ float Ws[16][64 + 4];
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int k0 = 0; k0 < K; k0 += 16) {
    for (int i = tid; i < 64 * 16; i += 256) {
      const int r = i >> 4, kk = i & 15;
      const int gm = m0 + r, gn = n0 + r, gk = k0 + kk;
      As[kk][r] = (gm < M && gk < K) ? to_f(A[(size_t)gm * lda + gk]) : 0.f;
      Ws[kk][r] = (gn < N && gk < K) ? to_f(W[(size_t)gn * K + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) w[j] = Ws[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
    const int rr = res_mod > 0 ? gm % res_mod : gm;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      float v = acc[i][j];
      if (bias) v += to_f(bias[gn]);
      if (act == ACT_RELU) v = fmaxf(v, 0.f);
      if (res) v += to_f(res[(size_t)rr * ldr + gn]);
      if (out_f32) ((float*)out)[(size_t)gm * ldo + gn] = v;
      else ((T*)out)[(size_t)gm * ldo + gn] = from_f<T>(v);
    }
  }
}

void launch_gemm_simt(cudaStream_t st, int bf, const GemmDesc& G) {
  if (G.M <= 0 || G.N <= 0) return;
  dim3 grid((G.N + 63) / 64, (G.M + 63) / 64);
  if (bf)
    gemm_simt_kernel<bf16><<<grid, 256, 0, st>>>((const bf16*)G.A, G.lda, (const bf16*)G.W, G.M, G.N,
                                                 G.K, G.out, G.ldo, G.out_f32, (const bf16*)G.bias,
                                                 (const bf16*)G.res, G.ldr, G.res_mod, G.act);
  else
    gemm_simt_kernel<float><<<grid, 256, 0, st>>>((const float*)G.A, G.lda, (const float*)G.W, G.M,
                                                  G.N, G.K, G.out, G.ldo, 1, (const float*)G.bias,
                                                  (const float*)G.res, G.ldr, G.res_mod, G.act);
}

}  // namespace zo
