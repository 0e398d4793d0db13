// Shared device helpers: element types, Philox4x32-10 perturbation stream, reductions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace zo {

typedef __nv_bfloat16 bf16;

// Bits of the device status word (deferred errors, read back by zo_losses).
enum : uint32_t {
  ST_TIMEOUT = 1u,      // a bounded mbarrier wait ran out inside a kernel
  ST_NONFINITE = 2u,    // a replica loss is NaN/Inf
  ST_BAD_LABELS = 4u,   // more labelled positions than max_labelled, or label out of range
  ST_BAD_TOKEN = 8u,    // token id outside [0, vocab)
  ST_PEER_FAULT = 16u   // sharded step: another device published a fault with its losses
};

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(bf16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float x) { return __float2bfloat16_rn(x); }

// ---------------------------------------------------------------------------------------
// Perturbation stream (Algorithm 1: z_i ~ N(0, I) "using s_i"; seed trick).
// Philox4x32-10 as published (Salmon et al., SC'11): ten rounds of two 32x32->64
// multiplies, key bumped by the Weyl constants between rounds.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), hi1 = __umulhi(0xCD9E8D57u, c.z);
    const uint32_t lo0 = 0xD2511F53u * c.x, lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}

// Raw words of block `blk` (elements 4*blk .. 4*blk+3) of tensor `tensor`, query `query`.
__device__ __forceinline__ uint4 z_words(uint64_t seed, uint32_t tensor, uint32_t query,
                                         uint32_t blk) {
  return philox4x32_10(make_uint4(blk, tensor, query, 0u),
                       make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
}

__device__ __forceinline__ float u01(uint32_t x) {
  return ((float)(x >> 9) + 0.5f) * 1.1920928955078125e-07f;  // 2^-23, exact in fp32
}

// Box-Muller on the word pairs (0,1) and (2,3): rho = sqrt(-2 ln u_a), phi = 2 pi u_b.
__device__ __forceinline__ float4 z_normals(uint4 w) {
  float4 z;
  float s, c;
  float rho = sqrtf(-2.0f * logf(u01(w.x)));
  sincospif(2.0f * u01(w.y), &s, &c);
  z.x = rho * c;
  z.y = rho * s;
  rho = sqrtf(-2.0f * logf(u01(w.z)));
  sincospif(2.0f * u01(w.w), &s, &c);
  z.z = rho * c;
  z.w = rho * s;
  return z;
}

__device__ __forceinline__ float4 z_block(uint64_t seed, uint32_t tensor, uint32_t query,
                                          uint32_t blk) {
  return z_normals(z_words(seed, tensor, query, blk));
}

// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// Block-wide sum; `red` is shared scratch of >= 32 floats.  All threads get the result.
__device__ __forceinline__ float block_sum(float v, float* red) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  v = (lane < nw) ? red[lane] : 0.0f;
  return warp_sum(v);
}
__device__ __forceinline__ float block_max(float v, float* red) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_max(v);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  v = (lane < nw) ? red[lane] : -INFINITY;
  return warp_max(v);
}

__device__ __forceinline__ double block_sum_d(double v, double* red) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  v = (lane < nw) ? red[lane] : 0.0;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

}  // namespace zo
