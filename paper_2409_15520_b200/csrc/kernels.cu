// Bandwidth-bound and small kernels of the perturbed forward, the losses and the update.
#include "common.cuh"
#include "kernels.h"
#include "lora_operand.cuh"

namespace zo {

// =========================================================================================
// Embedding (+ learned positions) on the SHARED token block only: the n replicas of the
// batch are identical up to the first MP-LoRA layer ("n copies of the input batch"), so
// this is computed once.  Pad rows (t >= T) are zero-filled.
// =========================================================================================
template <typename T>
__global__ void embed_kernel(const int32_t* __restrict__ tokens, const T* __restrict__ tok_emb,
                             const T* __restrict__ pos_emb, T* __restrict__ out, int Tn, SeqLayout sl,
                             int d, int vocab, uint32_t* status) {
  const int t = blockIdx.x;
  T* o = out + (size_t)t * d;
  if (t >= Tn) {
    for (int c = threadIdx.x; c < d; c += blockDim.x) o[c] = from_f<T>(0.f);
    return;
  }
  int id = tokens[t];
  if (id < 0 || id >= vocab) {
    if (threadIdx.x == 0) atomicOr(status, ST_BAD_TOKEN);
    id = 0;
  }
  const T* e = tok_emb + (size_t)id * d;
  const T* p = pos_emb ? pos_emb + (size_t)(sl.pos ? sl.pos[t] : t % sl.S) * d : nullptr;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float v = to_f(e[c]);
    if (p) v += to_f(p[c]);
    o[c] = from_f<T>(v);
  }
}

void launch_embed(cudaStream_t st, int bf, const int32_t* tokens, const void* tok_emb,
                  const void* pos_emb, void* out, int T, int Tp, SeqLayout sl, int d, int vocab,
                  uint32_t* status) {
  if (bf)
    embed_kernel<bf16><<<Tp, 128, 0, st>>>(tokens, (const bf16*)tok_emb, (const bf16*)pos_emb,
                                           (bf16*)out, T, sl, d, vocab, status);
  else
    embed_kernel<float><<<Tp, 128, 0, st>>>(tokens, (const float*)tok_emb, (const float*)pos_emb,
                                            (float*)out, T, sl, d, vocab, status);
}

// =========================================================================================
// LayerNorm / RMSNorm, one block per row, fp32 statistics (two-pass variance).
// =========================================================================================
template <typename T>
__global__ void norm_kernel(int kind, const T* __restrict__ x, T* __restrict__ out,
                            const T* __restrict__ g, const T* __restrict__ b, int d, float eps,
                            const int32_t* __restrict__ lab_idx, int EP, int Tp) {
  __shared__ float red[32];
  const int row = blockIdx.x;
  long long src = row;
  if (lab_idx) {
    const int n = row / EP, j = row % EP;
    const int li = lab_idx[j];
    src = li < 0 ? -1 : (long long)n * Tp + li;
  }
  T* o = out + (size_t)row * d;
  if (src < 0) {
    for (int c = threadIdx.x; c < d; c += blockDim.x) o[c] = from_f<T>(0.f);
    return;
  }
  const T* xr = x + (size_t)src * d;
  float s = 0.f;
  if (kind == 0) {
    for (int c = threadIdx.x; c < d; c += blockDim.x) s += to_f(xr[c]);
    const float mu = block_sum(s, red) / d;
    float v = 0.f;
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
      const float t = to_f(xr[c]) - mu;
      v += t * t;
    }
    const float rstd = rsqrtf(block_sum(v, red) / d + eps);
    for (int c = threadIdx.x; c < d; c += blockDim.x)
      o[c] = from_f<T>((to_f(xr[c]) - mu) * rstd * to_f(g[c]) + (b ? to_f(b[c]) : 0.f));
  } else {
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
      const float t = to_f(xr[c]);
      s += t * t;
    }
    const float rstd = rsqrtf(block_sum(s, red) / d + eps);
    for (int c = threadIdx.x; c < d; c += blockDim.x)
      o[c] = from_f<T>(to_f(xr[c]) * rstd * to_f(g[c]));
  }
}

// One block per row: 16-byte accesses, the row is read once and kept packed in registers (NV vectors
// per thread), one shared-memory exchange per reduction.  Few registers per thread, so many rows are
// in flight per SM.  KIND 0 = LayerNorm, 1 = RMSNorm (compiled apart: the kernel is close to its issue
// limit, so the RMS path carries no mean or bias arithmetic).  Requires d % VEC == 0 and d <= TPB * VEC * NV with TPB = blockDim.x <= 256.
template <typename T, int NV, int KIND>
__global__ void __launch_bounds__(256)
norm_vec_kernel(const T* __restrict__ x, T* __restrict__ out, const T* __restrict__ g,
                const T* __restrict__ b, int d, float eps, const int32_t* __restrict__ lab_idx,
                int EP, int Tp) {
  constexpr int VEC = 16 / sizeof(T);
  __shared__ float red[2][8];
  const int row = blockIdx.x, tpb = blockDim.x, nw = tpb >> 5;
  long long src = row;
  if (lab_idx) {
    const int n = row / EP, j = row % EP;
    const int li = lab_idx[j];
    src = li < 0 ? -1 : (long long)n * Tp + li;
  }
  T* o = out + (size_t)row * d;
  const int nvec = d / VEC;
  if (src < 0) {
    for (int v = threadIdx.x; v < nvec; v += tpb)
      *reinterpret_cast<uint4*>(o + v * VEC) = make_uint4(0, 0, 0, 0);
    return;
  }
  const T* xr = x + (size_t)src * d;
  uint4 raw[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int v = threadIdx.x + i * tpb;
    raw[i] = v < nvec ? *reinterpret_cast<const uint4*>(xr + v * VEC) : make_uint4(0, 0, 0, 0);
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const T* e = reinterpret_cast<const T*>(&raw[i]);
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      const float t = to_f(e[j]);
      s += KIND == 0 ? t : t * t;
    }
  }
  // block sum: one exchange through shared memory, every thread adds the warp partials itself
  auto all_sum = [&](float v, float* r) {
    v = warp_sum(v);
    if ((threadIdx.x & 31) == 0) r[threadIdx.x >> 5] = v;
    __syncthreads();
    float tot = 0.f;
    for (int w = 0; w < nw; ++w) tot += r[w];
    return tot;
  };
  s = all_sum(s, red[0]);
  float mu = 0.f, rstd;
  if (KIND == 0) {
    mu = s / d;
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      if (threadIdx.x + i * tpb < nvec) {
        const T* e = reinterpret_cast<const T*>(&raw[i]);
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
          const float t = to_f(e[j]) - mu;
          q += t * t;
        }
      }
    }
    rstd = rsqrtf(all_sum(q, red[1]) / d + eps);
  } else {
    rstd = rsqrtf(s / d + eps);
  }
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int v = threadIdx.x + i * tpb;
    if (v < nvec) {
      const uint4 graw = *reinterpret_cast<const uint4*>(g + v * VEC);
      const T* ge = reinterpret_cast<const T*>(&graw);
      uint4 braw = make_uint4(0, 0, 0, 0);
      if (KIND == 0 && b) braw = *reinterpret_cast<const uint4*>(b + v * VEC);
      const T* be = reinterpret_cast<const T*>(&braw);
      const T* e = reinterpret_cast<const T*>(&raw[i]);
      uint4 oraw;
      T* oe = reinterpret_cast<T*>(&oraw);
#pragma unroll
      for (int j = 0; j < VEC; ++j) {
        if (KIND == 0) oe[j] = from_f<T>((to_f(e[j]) - mu) * rstd * to_f(ge[j]) + (b ? to_f(be[j]) : 0.f));
        else oe[j] = from_f<T>(to_f(e[j]) * rstd * to_f(ge[j]));
      }
      *reinterpret_cast<uint4*>(o + v * VEC) = oraw;
    }
  }
}

// Packed fp32 pairs (sm_100: one instruction multiplies two floats) for the bf16 RMSNorm, which is bound
// by instruction issue: a bf16 pair widens to an fp32 pair with two logic operations.
__device__ __forceinline__ unsigned long long f2_from_bf2(uint32_t w) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(w << 16), "r"(w & 0xFFFF0000u));
  return r;
}
__device__ __forceinline__ unsigned long long f2_mul(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ unsigned long long f2_fma(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint32_t bf2_from_f2(unsigned long long a) {
  uint32_t lo, hi, r;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(a));
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(__uint_as_float(hi)), "f"(__uint_as_float(lo)));
  return r;
}

// One warp per row, four rows per block: the row is read once (16-byte accesses, all issued before the
// first use), kept packed in registers (NV vectors per lane), reduced with shuffles only: no barrier and
// no shared memory.  Default for bf16 rows of up to 4096 elements (NV = 16: 153 registers, 12 rows of
// 8 KB in flight per SM).  Against one block per row, CUDA events inside the step: d = 4096 -6 %,
// d = 2048 -19 %, d = 768 -11 %.  KIND 0 = LayerNorm, 1 = RMSNorm.  Requires d % VEC == 0, d <= 32*VEC*NV.
template <typename T, int NV, int KIND>
__global__ void __launch_bounds__(128)
norm_warp_kernel(const T* __restrict__ x, T* __restrict__ out, const T* __restrict__ g,
                 const T* __restrict__ b, int rows, int d, float eps,
                 const int32_t* __restrict__ lab_idx, int EP, int Tp) {
  constexpr int VEC = 16 / sizeof(T);
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * 4 + (threadIdx.x >> 5);
  if (row >= rows) return;
  long long src = row;
  if (lab_idx) {
    const int n = row / EP, j = row % EP;
    const int li = lab_idx[j];
    src = li < 0 ? -1 : (long long)n * Tp + li;
  }
  T* o = out + (size_t)row * d;
  const int nvec = d / VEC;
  if (src < 0) {
    for (int v = lane; v < nvec; v += 32) *reinterpret_cast<uint4*>(o + v * VEC) = make_uint4(0, 0, 0, 0);
    return;
  }
  const T* xr = x + (size_t)src * d;
  uint4 raw[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int v = lane + 32 * i;
    raw[i] = v < nvec ? *reinterpret_cast<const uint4*>(xr + v * VEC) : make_uint4(0, 0, 0, 0);
  }
  if constexpr (sizeof(T) == 2) {
    // bf16 rows on packed fp32 pairs: per element the same products and roundings as the scalar form below
    // ((x - mean) * rstd, then * g + b fused); the sums run in two interleaved chains
    auto hsum = [](unsigned long long a) {
      float s0, s1;
      asm("mov.b64 {%0, %1}, %2;" : "=f"(s0), "=f"(s1) : "l"(a));
      return s0 + s1;
    };
    auto dup = [](float a) {
      unsigned long long r;
      asm("mov.b64 %0, {%1, %1};" : "=l"(r) : "f"(a));
      return r;
    };
    // every sweep widens the packed row again: carrying the widened copy from one sweep to the next would
    // cost 8 registers per vector, and the rows in flight per SM with them
    auto forget = [&]() {
#pragma unroll
      for (int i = 0; i < NV; ++i)
        asm volatile("" : "+r"(raw[i].x), "+r"(raw[i].y), "+r"(raw[i].z), "+r"(raw[i].w));
    };
    unsigned long long acc = 0ull;
    const unsigned long long one2 = dup(1.f);
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const unsigned long long t = f2_from_bf2(w[j]);
        acc = KIND == 0 ? f2_fma(t, one2, acc) : f2_fma(t, t, acc);       // vectors past the row are zero
      }
    }
    forget();
    float mu = 0.f, rs;
    if (KIND == 0) {
      mu = warp_sum(hsum(acc)) / d;
      const unsigned long long nmu2 = dup(-mu);
      unsigned long long q2 = 0ull;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        if (lane + 32 * i < nvec) {
          const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const unsigned long long t = f2_fma(f2_from_bf2(w[j]), one2, nmu2);
            q2 = f2_fma(t, t, q2);
          }
        }
      }
      forget();
      rs = rsqrtf(warp_sum(hsum(q2)) / d + eps);
    } else {
      rs = rsqrtf(warp_sum(hsum(acc)) / d + eps);
    }
    const unsigned long long rs2 = dup(rs), nmu2 = dup(-mu);
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int v = lane + 32 * i;
      if (v < nvec) {
        const uint4 graw = *reinterpret_cast<const uint4*>(g + v * VEC);
        uint4 braw = make_uint4(0, 0, 0, 0);
        if (KIND == 0 && b) braw = *reinterpret_cast<const uint4*>(b + v * VEC);
        const uint32_t w[4] = {raw[i].x, raw[i].y, raw[i].z, raw[i].w};
        const uint32_t gw[4] = {graw.x, graw.y, graw.z, graw.w};
        const uint32_t bw[4] = {braw.x, braw.y, braw.z, braw.w};
        uint32_t ow[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          unsigned long long t = f2_from_bf2(w[j]);
          if (KIND == 0) t = f2_fma(t, one2, nmu2);
          t = f2_mul(t, rs2);
          t = KIND == 0 ? f2_fma(t, f2_from_bf2(gw[j]), f2_from_bf2(bw[j])) : f2_mul(t, f2_from_bf2(gw[j]));
          ow[j] = bf2_from_f2(t);
        }
        *reinterpret_cast<uint4*>(o + v * VEC) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
      }
    }
    return;
  }
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const T* e = reinterpret_cast<const T*>(&raw[i]);
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
      const float t = to_f(e[j]);
      s += KIND == 0 ? t : t * t;
    }
  }
  s = warp_sum(s);
  float mu = 0.f, rstd;
  if (KIND == 0) {
    mu = s / d;
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      if (lane + 32 * i < nvec) {
        const T* e = reinterpret_cast<const T*>(&raw[i]);
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
          const float t = to_f(e[j]) - mu;
          q += t * t;
        }
      }
    }
    rstd = rsqrtf(warp_sum(q) / d + eps);
  } else {
    rstd = rsqrtf(s / d + eps);
  }
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int v = lane + 32 * i;
    if (v < nvec) {
      const uint4 graw = *reinterpret_cast<const uint4*>(g + v * VEC);
      const T* ge = reinterpret_cast<const T*>(&graw);
      uint4 braw = make_uint4(0, 0, 0, 0);
      if (KIND == 0 && b) braw = *reinterpret_cast<const uint4*>(b + v * VEC);
      const T* be = reinterpret_cast<const T*>(&braw);
      const T* e = reinterpret_cast<const T*>(&raw[i]);
      uint4 oraw;
      T* oe = reinterpret_cast<T*>(&oraw);
#pragma unroll
      for (int j = 0; j < VEC; ++j)
        oe[j] = from_f<T>((to_f(e[j]) - mu) * rstd * to_f(ge[j]) + ((KIND == 0 && b) ? to_f(be[j]) : 0.f));
      *reinterpret_cast<uint4*>(o + v * VEC) = oraw;
    }
  }
}

template <typename T>
static void norm_dispatch(cudaStream_t st, int kind, const void* x, void* out, const void* g,
                          const void* b, int rows, int d, float eps, const int32_t* lab_idx, int EP,
                          int Tp) {
  constexpr int VEC = 16 / sizeof(T);
  const bool aligned = (((uintptr_t)x | (uintptr_t)out | (uintptr_t)g | (uintptr_t)b) & 15) == 0;
  const int nvec = d / VEC;
  if (aligned && d % VEC == 0 && nvec <= (sizeof(T) == 2 ? 512 : 64)) {
    // one warp per row, four rows per block (bf16: up to 4096 elements; fp32: up to 256)
    const int nv = (nvec + 31) / 32;
    const int grid = (rows + 3) / 4;
#define ZO_NW(NV)                                                                                              \
  do {                                                                                                         \
    if (kind == 0)                                                                                             \
      norm_warp_kernel<T, NV, 0><<<grid, 128, 0, st>>>((const T*)x, (T*)out, (const T*)g, (const T*)b, rows, d, eps, lab_idx, EP, Tp); \
    else                                                                                                       \
      norm_warp_kernel<T, NV, 1><<<grid, 128, 0, st>>>((const T*)x, (T*)out, (const T*)g, (const T*)b, rows, d, eps, lab_idx, EP, Tp); \
  } while (0)
    if (nv <= 1) ZO_NW(1);
    else if (nv == 2) ZO_NW(2);
    else if (nv <= 4) ZO_NW(4);
    else if (nv <= 8) ZO_NW(8);
    else ZO_NW(16);
#undef ZO_NW
    return;
  }
  if (aligned && d % VEC == 0 && nvec <= 256 * 4) {
    // two vectors per thread up to 256 threads, then more vectors per thread
    int th = ((nvec + 1) / 2 + 31) / 32 * 32;
    if (th > 256) th = 256;
    const int nv = (nvec + th - 1) / th;
#define ZO_NV(NV)                                                                                              \
  do {                                                                                                         \
    if (kind == 0)                                                                                             \
      norm_vec_kernel<T, NV, 0><<<rows, th, 0, st>>>((const T*)x, (T*)out, (const T*)g, (const T*)b, d, eps, lab_idx, EP, Tp); \
    else                                                                                                       \
      norm_vec_kernel<T, NV, 1><<<rows, th, 0, st>>>((const T*)x, (T*)out, (const T*)g, (const T*)b, d, eps, lab_idx, EP, Tp); \
  } while (0)
    if (nv <= 1) ZO_NV(1);
    else if (nv == 2) ZO_NV(2);
    else if (nv == 3) ZO_NV(3);
    else ZO_NV(4);
#undef ZO_NV
    return;
  }
  const int th = d >= 2048 ? 256 : 128;
  norm_kernel<T><<<rows, th, 0, st>>>(kind, (const T*)x, (T*)out, (const T*)g, (const T*)b, d, eps, lab_idx, EP, Tp);
}

void launch_norm(cudaStream_t st, int bf, int kind, const void* x, void* out, const void* g,
                 const void* b, int rows, int d, float eps, const int32_t* lab_idx, int EP,
                 int Tp) {
  if (rows <= 0) return;
  if (bf) norm_dispatch<bf16>(st, kind, x, out, g, b, rows, d, eps, lab_idx, EP, Tp);
  else norm_dispatch<float>(st, kind, x, out, g, b, rows, d, eps, lab_idx, EP, Tp);
}

// =========================================================================================
// LoRA down-projection U = X A^T (A shared by all replicas, frozen): [rows,K] x [J,K]^T.
// 32 rows per block, K streamed through shared memory in chunks of 32.
// =========================================================================================
constexpr int LD_MAXJ = 192;  // 3 targets x rank 64
template <typename T>
__global__ void __launch_bounds__(256)
lora_down_kernel(const T* __restrict__ X, int ldx, const T* __restrict__ A,
                 float* __restrict__ U, int rows, int K, int J) {
  extern __shared__ float sm[];
  float* Xs = sm;              // [32][33]
  float* As = sm + 32 * 33;    // [J][33]
  const int tid = threadIdx.x, r = tid >> 3, cg = tid & 7;
  const int row0 = blockIdx.x * 32;
  float acc[LD_MAXJ / 8];
#pragma unroll
  for (int i = 0; i < LD_MAXJ / 8; ++i) acc[i] = 0.f;
  for (int k0 = 0; k0 < K; k0 += 32) {
    for (int i = tid; i < 32 * 32; i += 256) {
      const int rr = i >> 5, kk = i & 31;
      const int gr = row0 + rr, gk = k0 + kk;
      Xs[rr * 33 + kk] = (gr < rows && gk < K) ? to_f(X[(size_t)gr * ldx + gk]) : 0.f;
    }
    for (int i = tid; i < J * 32; i += 256) {
      const int jj = i >> 5, kk = i & 31;
      const int gk = k0 + kk;
      As[jj * 33 + kk] = gk < K ? to_f(A[(size_t)jj * K + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int kk = 0; kk < 32; ++kk) {
      const float xv = Xs[r * 33 + kk];
#pragma unroll
      for (int i = 0; i < LD_MAXJ / 8; ++i) {
        const int j = cg + 8 * i;
        if (j < J) acc[i] = fmaf(xv, As[j * 33 + kk], acc[i]);
      }
    }
    __syncthreads();
  }
  const int gr = row0 + r;
  if (gr < rows) {
#pragma unroll
    for (int i = 0; i < LD_MAXJ / 8; ++i) {
      const int j = cg + 8 * i;
      if (j < J) U[(size_t)gr * J + j] = acc[i];
    }
  }
}

void launch_lora_down(cudaStream_t st, int bf, const void* X, int ldx, const void* A, float* U,
                      int rows, int K, int J) {
  if (rows <= 0 || J <= 0) return;
  const size_t smem = (size_t)(32 * 33 + J * 33) * sizeof(float);
  const int grid = (rows + 31) / 32;
  if (bf)
    lora_down_kernel<bf16><<<grid, 256, smem, st>>>((const bf16*)X, ldx, (const bf16*)A, U, rows, K, J);
  else
    lora_down_kernel<float><<<grid, 256, smem, st>>>((const float*)X, ldx, (const float*)A, U, rows, K, J);
}

// =========================================================================================
// MP-LoRA low-rank term applied to a base product:
//   out[n, t, c] = base[(shared ? t : n*Tp + t), c]
//                + s * sum_k U[.., slot*r + k] * (B[slot,k,c'] + k_n eps z)
// z regenerated from the seed in registers (never stored).  Each thread owns 4 consecutive
// columns (= one Philox block per rank index) and LA_ROWS rows of one replica.
// =========================================================================================
constexpr int LA_ROWS = 64, LA_COLS = 128;
template <typename T>
__global__ void __launch_bounds__(256)
lora_apply_kernel(const T* base, int ldb, int base_shared, T* out, int ldo, int Tn, LoraDesc L,
                  int /*nsec*/) {
  extern __shared__ float sB[];                       // [r][LA_COLS]: s * (B + k eps z) of this tile
  const int n = blockIdx.z;
  const int tiles_per_sec = (L.width + LA_COLS - 1) / LA_COLS;   // tiles never straddle two sections
  const int sec = blockIdx.x / tiles_per_sec, cc_t = (blockIdx.x - sec * tiles_per_sec) * LA_COLS;
  const int col_t = sec * L.width + cc_t;             // first column of the tile
  const int t0 = blockIdx.y * LA_ROWS;
  const int slot = L.slot_of_sec[sec];                // uniform over the block
  const int Tp = L.rows_per_replica;
  const int ncols = min(LA_COLS, L.width - cc_t);
  if (slot >= 0) {
    const int rid = L.rep_base + L.rep_stride * n;    // replica id within the step
    for (int i = threadIdx.x; i < L.r * (LA_COLS / 4); i += blockDim.x) {
      const int k = i / (LA_COLS / 4), c4 = (i % (LA_COLS / 4)) * 4;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (c4 < ncols) {
        v = lora_replica_b(L, slot, (size_t)k * L.width + cc_t + c4, rid);
        v.x *= L.scale; v.y *= L.scale; v.z *= L.scale; v.w *= L.scale;
      }
      *reinterpret_cast<float4*>(sB + k * LA_COLS + c4) = v;
    }
    __syncthreads();
  }
  const int c4 = (threadIdx.x & 31) * 4;
  if (c4 >= ncols) return;
  for (int i = threadIdx.x >> 5; i < LA_ROWS; i += 8) {
    const int t = t0 + i;
    if (t >= Tn) break;
    const size_t brow = base_shared ? (size_t)t : (size_t)n * Tp + t;
    const T* bp = base + brow * ldb + col_t + c4;
    float a0 = to_f(bp[0]), a1 = to_f(bp[1]), a2 = to_f(bp[2]), a3 = to_f(bp[3]);
    if (slot >= 0) {
      const float* up = L.U + brow * L.ldu + slot * L.r;
      for (int k = 0; k < L.r; ++k) {
        const float u = up[k];
        const float4 bv = *reinterpret_cast<const float4*>(sB + k * LA_COLS + c4);
        a0 = fmaf(u, bv.x, a0); a1 = fmaf(u, bv.y, a1);
        a2 = fmaf(u, bv.z, a2); a3 = fmaf(u, bv.w, a3);
      }
    }
    T* op = out + ((size_t)n * Tp + t) * ldo + col_t + c4;
    op[0] = from_f<T>(a0); op[1] = from_f<T>(a1); op[2] = from_f<T>(a2); op[3] = from_f<T>(a3);
  }
}

void launch_lora_apply(cudaStream_t st, int bf, const void* base, int ldb, int base_shared,
                       void* out, int ldo, int n, int T, const LoraDesc& L, int nsec) {
  if (n <= 0 || T <= 0) return;
  const int tiles_per_sec = (L.width + LA_COLS - 1) / LA_COLS;
  dim3 grid(nsec * tiles_per_sec, (T + LA_ROWS - 1) / LA_ROWS, n);
  const size_t smem = (size_t)L.r * LA_COLS * sizeof(float);
  if (bf)
    lora_apply_kernel<bf16><<<grid, 256, smem, st>>>((const bf16*)base, ldb, base_shared, (bf16*)out, ldo, T, L, nsec);
  else
    lora_apply_kernel<float><<<grid, 256, smem, st>>>((const float*)base, ldb, base_shared, (float*)out, ldo, T, L, nsec);
}

// =========================================================================================
// RoPE (rotate-half pairing (j, j + dh/2)); table of cos/sin built once in fp64.
// =========================================================================================
__global__ void rope_table_kernel(float* tab, int max_seq, int half, double theta) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= max_seq * half) return;
  const int s = i / half, j = i % half;
  const double inv = pow(theta, -2.0 * (double)j / (double)(2 * half));
  const double a = (double)s * inv;
  tab[(size_t)s * 2 * half + j] = (float)cos(a);          // row s: cos[0..half) then sin[0..half)
  tab[(size_t)s * 2 * half + half + j] = (float)sin(a);
}
void launch_rope_table(cudaStream_t st, float* tab, int max_seq, int dh, float theta) {
  const int n = max_seq * (dh / 2);
  rope_table_kernel<<<(n + 255) / 256, 256, 0, st>>>(tab, max_seq, dh / 2, (double)theta);
}

// In place on the q and k sections of the fused [rows, 3d] buffer.  Each thread rotates VEC
// consecutive pairs (16-byte accesses).
template <typename T>
__global__ void rope_kernel(T* __restrict__ qkv, long long total, int Tp, SeqLayout sl, int d, int H,
                            const float* __restrict__ tab) {
  constexpr int VEC = 16 / sizeof(T);
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int half = d / H / 2;
  const int vph = half / VEC;                         // vectors per half head
  const int j = (int)(i % vph) * VEC;
  long long rest = i / vph;
  const int h = (int)(rest % H);
  rest /= H;
  const int which = (int)(rest % 2);                  // 0 = q, 1 = k
  const long long row = rest / 2;
  const int s = sl.pos ? sl.pos[row % Tp] : (int)((row % Tp) % sl.S);
  const float* cs = tab + (size_t)s * 2 * half + j;   // row s: cos[0..half) then sin[0..half)
  T* p = qkv + (size_t)row * 3 * d + (size_t)which * d + h * 2 * half + j;
  uint4 lo = *reinterpret_cast<const uint4*>(p), hi = *reinterpret_cast<const uint4*>(p + half);
  T* e1 = reinterpret_cast<T*>(&lo);
  T* e2 = reinterpret_cast<T*>(&hi);
#pragma unroll
  for (int k = 0; k < VEC; ++k) {
    const float c = cs[k], sn = cs[half + k];
    const float x1 = to_f(e1[k]), x2 = to_f(e2[k]);
    e1[k] = from_f<T>(x1 * c - x2 * sn);
    e2[k] = from_f<T>(x2 * c + x1 * sn);
  }
  *reinterpret_cast<uint4*>(p) = lo;
  *reinterpret_cast<uint4*>(p + half) = hi;
}
// Scalar variant for head dimensions whose half is not a multiple of the vector width.
template <typename T>
__global__ void rope_scalar_kernel(T* __restrict__ qkv, long long total, int Tp, SeqLayout sl, int d, int H,
                                   const float* __restrict__ tab) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int half = d / H / 2;
  const int j = (int)(i % half);
  long long rest = i / half;
  const int h = (int)(rest % H);
  rest /= H;
  const int which = (int)(rest % 2);
  const long long row = rest / 2;
  const int s = sl.pos ? sl.pos[row % Tp] : (int)((row % Tp) % sl.S);
  const float c = tab[(size_t)s * 2 * half + j], sn = tab[(size_t)s * 2 * half + half + j];
  T* p = qkv + (size_t)row * 3 * d + (size_t)which * d + h * 2 * half + j;
  const float x1 = to_f(p[0]), x2 = to_f(p[half]);
  p[0] = from_f<T>(x1 * c - x2 * sn);
  p[half] = from_f<T>(x2 * c + x1 * sn);
}
template <typename T>
static void rope_dispatch(cudaStream_t st, void* qkv, int rows, int Tp, SeqLayout sl, int d, int H,
                          const float* tab) {
  constexpr int VEC = 16 / sizeof(T);
  const int half = d / H / 2;
  if (half % VEC == 0 && d % VEC == 0 && ((uintptr_t)qkv & 15) == 0) {
    const long long total = (long long)rows * 2 * H * (half / VEC);
    if (total > 0)
      rope_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>((T*)qkv, total, Tp, sl, d, H, tab);
  } else {
    const long long total = (long long)rows * 2 * H * half;
    if (total > 0)
      rope_scalar_kernel<T><<<(unsigned)((total + 255) / 256), 256, 0, st>>>((T*)qkv, total, Tp, sl, d, H, tab);
  }
}
void launch_rope(cudaStream_t st, int bf, void* qkv, int rows, int Tp, SeqLayout sl, int d, int H,
                 const float* tab) {
  if (bf) rope_dispatch<bf16>(st, qkv, rows, Tp, sl, d, H, tab);
  else rope_dispatch<float>(st, qkv, rows, Tp, sl, d, H, tab);
}

// =========================================================================================
// Causal attention on CUDA cores (validation / fp32 path): one block per
// (64-query tile, head, sequence).  Scores of the tile against all visible keys are kept in
// shared memory (S <= 512), then a row softmax, then P V.
// =========================================================================================
template <typename T, int DH>
__global__ void __launch_bounds__(256)
attention_simt_kernel(const T* __restrict__ qkv, T* __restrict__ ctx, SeqLayout sl, int Tp,
                      int d) {
  extern __shared__ float sm[];
  constexpr int LDQ = DH + 1;
  const int Sp = (sl.S + 63) & ~63;              // row pitch of the score tile (longest sequence)
  float* Qs = sm;                 // [64][LDQ]
  float* Ks = Qs + 64 * LDQ;      // [64][LDQ]  (K tile, later V tile)
  float* Ss = Ks + 64 * LDQ;      // [64][Sp + 1]
  const int LDS = Sp + 1;
  const int q0 = blockIdx.x * 64, h = blockIdx.y, sq = blockIdx.z;
  const int n = sq / sl.E, b = sq % sl.E;
  const int S = sl.len(b);                          // this sequence's length
  if (q0 >= S) return;
  const size_t row_base = (size_t)n * Tp + (size_t)sl.start(b);
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const float scale = rsqrtf((float)DH);
  const int ld = 3 * d;

  for (int i = tid; i < 64 * DH; i += 256) {
    const int r = i / DH, c = i % DH;
    const int s = q0 + r;
    Qs[r * LDQ + c] = s < S ? to_f(qkv[(row_base + s) * ld + h * DH + c]) : 0.f;
  }
  const int kend = min(S, q0 + 64);  // keys visible to this query tile
  for (int k0 = 0; k0 < kend; k0 += 64) {
    __syncthreads();
    for (int i = tid; i < 64 * DH; i += 256) {
      const int r = i / DH, c = i % DH;
      const int s = k0 + r;
      Ks[r * LDQ + c] = s < S ? to_f(qkv[(row_base + s) * ld + d + h * DH + c]) : 0.f;
    }
    __syncthreads();
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 8
    for (int c = 0; c < DH; ++c) {
      float qv[4], kv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) qv[i] = Qs[(ty * 4 + i) * LDQ + c];
#pragma unroll
      for (int j = 0; j < 4; ++j) kv[j] = Ks[(tx * 4 + j) * LDQ + c];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(qv[i], kv[j], acc[i][j]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) Ss[(ty * 4 + i) * LDS + k0 + tx * 4 + j] = acc[i][j] * scale;
  }
  __syncthreads();
  // row softmax over keys 0..q (causal), one warp per row
  const int warp = tid >> 5, lane = tid & 31;
  for (int r = warp; r < 64; r += 8) {
    const int s = q0 + r;
    const int lim = min(s, S - 1) + 1;  // number of visible keys
    float* p = Ss + r * LDS;
    float m = -INFINITY;
    for (int k = lane; k < lim; k += 32) m = fmaxf(m, p[k]);
    m = warp_max(m);
    float sum = 0.f;
    for (int k = lane; k < lim; k += 32) {
      const float e = expf(p[k] - m);
      p[k] = e;
      sum += e;
    }
    sum = warp_sum(sum);
    const float inv = 1.f / sum;
    for (int k = lane; k < Sp; k += 32) p[k] = k < lim ? p[k] * inv : 0.f;
  }
  // O = P V
  constexpr int NC = DH / 16;
  float o[4][NC];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < NC; ++j) o[i][j] = 0.f;
  for (int k0 = 0; k0 < kend; k0 += 64) {
    __syncthreads();
    for (int i = tid; i < 64 * DH; i += 256) {
      const int r = i / DH, c = i % DH;
      const int s = k0 + r;
      Ks[r * LDQ + c] = s < S ? to_f(qkv[(row_base + s) * ld + 2 * d + h * DH + c]) : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int k = 0; k < 64; ++k) {
      float pv[4], vv[NC];
#pragma unroll
      for (int i = 0; i < 4; ++i) pv[i] = Ss[(ty * 4 + i) * LDS + k0 + k];
#pragma unroll
      for (int j = 0; j < NC; ++j) vv[j] = Ks[k * LDQ + tx + 16 * j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < NC; ++j) o[i][j] = fmaf(pv[i], vv[j], o[i][j]);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int s = q0 + ty * 4 + i;
    if (s < S) {
#pragma unroll
      for (int j = 0; j < NC; ++j)
        ctx[(row_base + s) * d + h * DH + tx + 16 * j] = from_f<T>(o[i][j]);
    }
  }
}

template <typename T, int DH>
static void attention_simt_launch(cudaStream_t st, const void* qkv, void* ctx, int n, SeqLayout sl,
                                  int Tp, int d, int H) {
  const int S = sl.S, E = sl.E;
  const int Sp = (S + 63) & ~63;
  const size_t smem = (size_t)(2 * 64 * (DH + 1) + 64 * (Sp + 1)) * sizeof(float);
  cudaFuncSetAttribute(attention_simt_kernel<T, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       (int)smem);
  dim3 grid((S + 63) / 64, H, n * E);
  attention_simt_kernel<T, DH><<<grid, 256, smem, st>>>((const T*)qkv, (T*)ctx, sl, Tp, d);
}

void launch_attention_simt(cudaStream_t st, int bf, const void* qkv, void* ctx, int n, SeqLayout sl,
                           int Tp, int d, int H) {
  const int dh = d / H;
#define ZO_ATT(DH)                                                             \
  if (dh == DH) {                                                              \
    if (bf) attention_simt_launch<bf16, DH>(st, qkv, ctx, n, sl, Tp, d, H);    \
    else attention_simt_launch<float, DH>(st, qkv, ctx, n, sl, Tp, d, H);      \
    return;                                                                    \
  }
  ZO_ATT(16) ZO_ATT(32) ZO_ATT(64) ZO_ATT(128)
#undef ZO_ATT
}

// =========================================================================================
// SwiGLU on an unfused [rows, 2*ffn] gate|up buffer.
// =========================================================================================
template <typename T>
__global__ void swiglu_kernel(const T* __restrict__ gu, T* __restrict__ out, long long total,
                              int ffn) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const long long row = i / ffn;
  const int c = (int)(i % ffn);
  const float g = to_f(gu[row * 2 * ffn + c]), u = to_f(gu[row * 2 * ffn + ffn + c]);
  out[i] = from_f<T>(g / (1.f + expf(-g)) * u);
}
void launch_swiglu(cudaStream_t st, int bf, const void* gu, void* out, int rows, int ffn) {
  const long long total = (long long)rows * ffn;
  if (total <= 0) return;
  const unsigned grid = (unsigned)((total + 255) / 256);
  if (bf) swiglu_kernel<bf16><<<grid, 256, 0, st>>>((const bf16*)gu, (bf16*)out, total, ffn);
  else swiglu_kernel<float><<<grid, 256, 0, st>>>((const float*)gu, (float*)out, total, ffn);
}

// =========================================================================================
// Packed variable-length batch: position of every packed row inside its sequence.
__global__ void varlen_index_kernel(const int32_t* __restrict__ cu, int E, int Tn, int Tp, int max_len,
                                    int32_t* __restrict__ pos, uint32_t* status) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= Tp) return;
  if (t >= Tn) { pos[t] = 0; return; }
  int lo = 0, hi = E;                               // largest b with cu[b] <= t
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu[mid] <= t) lo = mid; else hi = mid;
  }
  const int p = t - cu[lo];
  const int len = cu[lo + 1] - cu[lo];
  if (p < 0 || len < 1 || len > max_len || p >= len || cu[0] != 0 || cu[E] != Tn) {
    atomicOr(status, ST_BAD_LABELS);
    pos[t] = 0;
    return;
  }
  pos[t] = p;
}
void launch_varlen_index(cudaStream_t st, const int32_t* cu, int E, int T, int Tp, int max_len, int32_t* pos,
                         uint32_t* status) {
  varlen_index_kernel<<<(Tp + 255) / 256, 256, 0, st>>>(cu, E, T, Tp, max_len, pos, status);
}

// Labelled positions of each sequence, in order: lab_idx[b*P + p] = b*S + s (or -1),
// lab_val = the label there.  One thread per sequence (S is small).
// =========================================================================================
__global__ void label_scan_kernel(const int32_t* __restrict__ labels, SeqLayout sl, int P,
                                  int n_classes, int32_t* lab_idx, int32_t* lab_val,
                                  int32_t* lab_cnt, uint32_t* status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= sl.E) return;
  const int start = sl.start(b);
  const int S = sl.len(b);
  int cnt = 0;
  for (int s = 0; s < S; ++s) {
    const int v = labels[start + s];
    if (v < 0) continue;
    if (v >= n_classes || cnt >= P) {
      atomicOr(status, ST_BAD_LABELS);
      continue;
    }
    lab_idx[b * P + cnt] = start + s;
    lab_val[b * P + cnt] = v;
    ++cnt;
  }
  lab_cnt[b] = cnt;
  for (; cnt < P; ++cnt) {
    lab_idx[b * P + cnt] = -1;
    lab_val[b * P + cnt] = -1;
  }
}
void launch_label_scan(cudaStream_t st, const int32_t* labels, SeqLayout sl, int P, int n_classes,
                       int32_t* lab_idx, int32_t* lab_val, int32_t* lab_cnt, uint32_t* status) {
  label_scan_kernel<<<(sl.E + 63) / 64, 64, 0, st>>>(labels, sl, P, n_classes, lab_idx, lab_val,
                                                  lab_cnt, status);
}

// =========================================================================================
// Fused log-softmax / label pick over the whole vocabulary, one block per labelled row:
// row_loss = logsumexp(logits) - logits[label].
// The row is read once: every thread keeps a running (max, sum of exp relative to that max) over
// 16-byte loads, four of them in flight, and the block merges the 256 pairs at the end.  The
// logits are streamed (read exactly once, by this kernel), so the loads bypass L1 allocation.
// =========================================================================================
__device__ __forceinline__ void lse_push4(float& m, float& s, const float4 v) {
  const float mx = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
  if (mx > m) {                       // first chunk: m = -inf, s = 0, expf(-inf) = 0
    s *= expf(m - mx);
    m = mx;
  }
  s += (expf(v.x - m) + expf(v.y - m)) + (expf(v.z - m) + expf(v.w - m));
}
__global__ void __launch_bounds__(256)
ce_rows_kernel(const float* __restrict__ logits, int ldl, int V, const int32_t* __restrict__ lab_val, int EP,
               double* __restrict__ row_loss) {
  __shared__ float red[32];
  const int row = blockIdx.x;
  const int lab = lab_val[row % EP];
  if (lab < 0) {
    if (threadIdx.x == 0) row_loss[row] = 0.0;
    return;
  }
  const float* p = logits + (size_t)row * ldl;
  float m = -INFINITY, s = 0.f;
  // the vector path is taken for all rows or for none, so that a row's sum order (and with it the
  // last bits of its loss) does not depend on where the row sits in the array
  if ((((uintptr_t)logits) & 15) == 0 && (ldl & 3) == 0) {
    const float4* p4 = reinterpret_cast<const float4*>(p);
    const int n4 = V >> 2;
    int c = threadIdx.x;
    for (; c + 3 * 256 < n4; c += 4 * 256) {
      const float4 a = __ldcs(p4 + c), b = __ldcs(p4 + c + 256);
      const float4 d = __ldcs(p4 + c + 512), e = __ldcs(p4 + c + 768);
      lse_push4(m, s, a);
      lse_push4(m, s, b);
      lse_push4(m, s, d);
      lse_push4(m, s, e);
    }
    for (; c < n4; c += 256) lse_push4(m, s, __ldcs(p4 + c));
    for (int t = (n4 << 2) + threadIdx.x; t < V; t += 256) {      // V % 4 leftovers
      const float v = p[t];
      if (v > m) { s *= expf(m - v); m = v; }
      s += expf(v - m);
    }
  } else {
    for (int t = threadIdx.x; t < V; t += 256) {
      const float v = p[t];
      if (v > m) { s *= expf(m - v); m = v; }
      s += expf(v - m);
    }
  }
  const float mb = block_max(m, red);
  // a thread that saw no element has m = -inf, s = 0: expf(-inf) = 0 keeps it out (mb is finite
  // unless the whole row is -inf or holds a NaN, which the replica mean reports as non-finite)
  const float sb = block_sum(m == -INFINITY ? 0.f : s * expf(m - mb), red);
  if (threadIdx.x == 0) row_loss[row] = ((double)mb - (double)p[lab]) + log((double)sb);
}
void launch_ce_rows(cudaStream_t st, const float* logits, int ldl, int V, const int32_t* lab_val,
                    int EP, int rows, double* row_loss) {
  if (rows <= 0) return;
  ce_rows_kernel<<<rows, 256, 0, st>>>(logits, ldl, V, lab_val, EP, row_loss);
}

// Second half of the fused cross-entropy head: one warp per labelled row merges the (max, sum) pairs of
// the row's column tiles.  Lane l folds pairs l, l + 32, ... in index order, then the lanes are folded by
// a fixed butterfly: the order, and with it every bit of the result, is the same from run to run.
__global__ void __launch_bounds__(256)
ce_merge_kernel(const float2* __restrict__ part, int ppr, const float* __restrict__ logit,
                const int32_t* __restrict__ lab_val, int EP, int rows, double* __restrict__ row_loss) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= rows) return;
  if (lab_val[row % EP] < 0) {
    if (lane == 0) row_loss[row] = 0.0;
    return;
  }
  const float2* p = part + (size_t)row * ppr;
  double m = -INFINITY, s = 0.0;
  auto fold = [&](double m2, double s2) {
    if (m2 == -INFINITY) return;                 // an empty share
    if (m2 > m) { s = s * exp(m - m2) + s2; m = m2; }   // (first pair: m = -inf, s = 0)
    else s += s2 * exp(m2 - m);
  };
  for (int i = lane; i < ppr; i += 32) {
    const float2 v = p[i];
    fold((double)v.x, (double)v.y);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const double m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
    // both partners must end with the same bits: fold the pair in lane order, whichever side this is
    double ma = (lane & o) ? m2 : m, sa = (lane & o) ? s2 : s;
    const double mb = (lane & o) ? m : m2, sb = (lane & o) ? s : s2;
    if (mb != -INFINITY) {
      if (mb > ma) { sa = sa * exp(ma - mb) + sb; ma = mb; }
      else sa += sb * exp(mb - ma);
    }
    m = ma; s = sa;
  }
  if (lane == 0) row_loss[row] = (m - (double)logit[row]) + log(s);
}
void launch_ce_merge(cudaStream_t st, const void* ce_part, int parts_per_row, const float* ce_logit,
                     const int32_t* lab_val, int EP, int rows, double* row_loss) {
  if (rows <= 0) return;
  ce_merge_kernel<<<(rows + 7) / 8, 256, 0, st>>>((const float2*)ce_part, parts_per_row, ce_logit, lab_val, EP, rows, row_loss);
}

// Two-way softmax over the two label-word logits at the labelled (final) position.
template <typename T>
__global__ void label_word_rows_kernel(const T* __restrict__ xh, const T* __restrict__ head,
                                       int d, int w0, int w1, const int32_t* __restrict__ lab_val,
                                       int EP, double* __restrict__ row_loss) {
  __shared__ float red[32];
  const int row = blockIdx.x;
  const int cls = lab_val[row % EP];
  if (cls < 0) {
    if (threadIdx.x == 0) row_loss[row] = 0.0;
    return;
  }
  const T* x = xh + (size_t)row * d;
  const T* h0 = head + (size_t)w0 * d;
  const T* h1 = head + (size_t)w1 * d;
  float a = 0.f, b = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const float xv = to_f(x[c]);
    a = fmaf(xv, to_f(h0[c]), a);
    b = fmaf(xv, to_f(h1[c]), b);
  }
  a = block_sum(a, red);
  b = block_sum(b, red);
  if (threadIdx.x == 0) {
    const double da = a, db = b, m = fmax(da, db);
    const double lse = m + log(exp(da - m) + exp(db - m));
    row_loss[row] = lse - (cls == 0 ? da : db);
  }
}
void launch_label_word_rows(cudaStream_t st, int bf, const void* xh, const void* head, int d,
                            int w0, int w1, const int32_t* lab_val, int EP, int rows,
                            double* row_loss) {
  if (rows <= 0) return;
  if (bf)
    label_word_rows_kernel<bf16><<<rows, 128, 0, st>>>((const bf16*)xh, (const bf16*)head, d, w0, w1, lab_val, EP, row_loss);
  else
    label_word_rows_kernel<float><<<rows, 128, 0, st>>>((const float*)xh, (const float*)head, d, w0, w1, lab_val, EP, row_loss);
}

// Mean squared error of one output row against its target (ZO_ARCH_LINEAR).
template <typename T>
__global__ void mse_rows_kernel(const T* __restrict__ Y, const float* __restrict__ target, int Tn,
                                int Tp, int k_out, double* __restrict__ row_loss) {
  __shared__ double red[32];
  const int t = blockIdx.x, n = blockIdx.y;
  const T* y = Y + ((size_t)n * Tp + t) * k_out;
  const float* g = target + (size_t)t * k_out;
  double s = 0.0;
  for (int c = threadIdx.x; c < k_out; c += blockDim.x) {
    const double dlt = (double)to_f(y[c]) - (double)g[c];
    s = fma(dlt, dlt, s);
  }
  s = block_sum_d(s, red);
  if (threadIdx.x == 0) row_loss[(size_t)n * Tn + t] = s / (double)k_out;
}
void launch_mse_rows(cudaStream_t st, int bf, const void* Y, const float* target, int n, int T,
                     int Tp, int k_out, double* row_loss) {
  if (n <= 0 || T <= 0) return;
  dim3 grid(T, n);
  if (bf) mse_rows_kernel<bf16><<<grid, 128, 0, st>>>((const bf16*)Y, target, T, Tp, k_out, row_loss);
  else mse_rows_kernel<float><<<grid, 128, 0, st>>>((const float*)Y, target, T, Tp, k_out, row_loss);
}

// =========================================================================================
// Per-replica mean over its valid rows: fixed order, fp64 accumulation (Algorithm 1: the
// loss of a path is the mean over the labelled positions of the batch).
// =========================================================================================
__global__ void replica_mean_kernel(const double* __restrict__ row_loss,
                                    const int32_t* __restrict__ lab_val, int rows, int rep_base,
                                    int rep_stride, double* __restrict__ rows_out,
                                    float* __restrict__ losses, double* __restrict__ losses_d,
                                    uint32_t* status) {
  __shared__ double sd[256];
  __shared__ int sc[256];
  const int n = blockIdx.x;
  const int rid = rep_base + rep_stride * n;     // replica id within the step
  double s = 0.0;
  int c = 0;
  for (int i = threadIdx.x; i < rows; i += 256) {
    const double v = row_loss[(size_t)n * rows + i];
    rows_out[(size_t)rid * rows + i] = v;
    if (!lab_val || lab_val[i] >= 0) {
      s += v;
      ++c;
    }
  }
  sd[threadIdx.x] = s;
  sc[threadIdx.x] = c;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if (threadIdx.x < o) {
      sd[threadIdx.x] += sd[threadIdx.x + o];
      sc[threadIdx.x] += sc[threadIdx.x + o];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double ld = sc[0] > 0 ? sd[0] / (double)sc[0] : 0.0;
    const float l = (float)ld;
    losses[rid] = l;
    losses_d[rid] = ld;
    if (!isfinite(l)) atomicOr(status, ST_NONFINITE);
  }
}
void launch_replica_mean(cudaStream_t st, const double* row_loss, const int32_t* lab_val, int n,
                         int rows_per_replica, int rep_base, int rep_stride, double* rows_out,
                         float* losses, double* losses_d, uint32_t* status) {
  if (n <= 0) return;
  replica_mean_kernel<<<n, 256, 0, st>>>(row_loss, lab_val, rows_per_replica, rep_base, rep_stride,
                                         rows_out, losses, losses_d, status);
}

// =========================================================================================
// Projected gradients and ZO-SGD update (Algorithm 1): g_i = (l+ - l-) / (2 eps);
// B <- B - eta (1/q) sum_i g_i z_i with z_i regenerated from the same seed.  Only the
// master copy is written.  Each thread owns one Philox block (4 consecutive elements).
// =========================================================================================
constexpr int UPD_MAXQ = 64;
__global__ void zo_update_kernel(UpdateDesc D, const double* __restrict__ losses,
                                 float* __restrict__ g_out, int q, float eps, float lr,
                                 uint64_t seed, const uint32_t* __restrict__ status, int write_g) {
  __shared__ float gs[UPD_MAXQ];
  const bool live = eps > 0.f;
  for (int i = threadIdx.x; i < q; i += blockDim.x)
    gs[i] = live ? (float)((losses[2 * i] - losses[2 * i + 1]) / (2.0 * (double)eps)) : 0.f;
  __syncthreads();
  if (write_g && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0)
    for (int i = threadIdx.x; i < q; i += blockDim.x) g_out[i] = gs[i];
  if (!live || lr == 0.f || *status != 0u) return;
  const long long blk = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long e = blk * 4;
  if (e >= D.elems_per_slot) return;
  const int slot = blockIdx.y, li = blockIdx.z;
  float* Bp = D.B[li] + (size_t)slot * D.elems_per_slot + e;
  const uint32_t tensor = D.tensor_base[li] + slot;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
  for (int i = 0; i < q; ++i) {
    const float4 z = z_block(seed, tensor, (uint32_t)i, (uint32_t)blk);
    const float gi = gs[i];
    a0 = fmaf(gi, z.x, a0);
    a1 = fmaf(gi, z.y, a1);
    a2 = fmaf(gi, z.z, a2);
    a3 = fmaf(gi, z.w, a3);
  }
  const float sc = lr / (float)q;
  const long long left = D.elems_per_slot - e;
  if (left >= 4) {
    float4 b = *reinterpret_cast<float4*>(Bp);
    b.x -= sc * a0; b.y -= sc * a1; b.z -= sc * a2; b.w -= sc * a3;
    *reinterpret_cast<float4*>(Bp) = b;
  } else {
    const float a[4] = {a0, a1, a2, a3};
    for (int j = 0; j < left; ++j) Bp[j] -= sc * a[j];
  }
}
// After the losses of other devices' queries have been written into the fp64 array: the fp32 copy
// that zo_losses reads, and the finiteness check the local reduction did for its own entries.
__global__ void losses_refresh_kernel(const double* __restrict__ losses_d, float* __restrict__ losses,
                                      int n, const double* __restrict__ fault_slot, uint32_t* status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  // a fault on any device of a sharded step blocks the update on every device (all see the same slot)
  if (i == 0 && fault_slot && *fault_slot != 0.0) atomicOr(status, ST_PEER_FAULT);
  if (i >= n) return;
  const float l = (float)losses_d[i];
  losses[i] = l;
  if (!isfinite(l)) atomicOr(status, ST_NONFINITE);
}
void launch_losses_refresh(cudaStream_t st, const double* losses_d, float* losses, int n,
                           const double* fault_slot, uint32_t* status) {
  losses_refresh_kernel<<<(n + 63) / 64, 64, 0, st>>>(losses_d, losses, n, fault_slot, status);
}
__global__ void fault_publish_kernel(const uint32_t* __restrict__ status, double* __restrict__ fault_slot) {
  *fault_slot = *status != 0u ? 1.0 : 0.0;
}
void launch_fault_publish(cudaStream_t st, const uint32_t* status, double* fault_slot) {
  fault_publish_kernel<<<1, 1, 0, st>>>(status, fault_slot);
}

// =========================================================================================
// Stored-pair form of the trainable tensors (Algorithm 2, "Mobile MP-LoRA", q = 1): B[0] = B + eps z
// and B[1] = B - eps z live in memory.  At the start of a forward pass the previous step's update and
// the new perturbation are applied to both, in the algorithm's order of operations:
//   diff = (B[0] - B[1]) / 2;  update = eta g diff / eps;  z = eps randn;
//   B[0] = B[0] - diff - update + z;  B[1] = B[1] + diff - update - z.
// g is the previous step's projected gradient (device pointer, or a value).  draw = 0 leaves z = 0:
// both tensors end at the updated master copy.
// =========================================================================================
__global__ void pair_update_kernel(UpdateDesc D, long long pair_stride, const float* __restrict__ g_dev,
                                   float g_val, float eps, float lr, uint64_t seed, int draw) {
  const long long blk = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long e = blk * 4;
  if (e >= D.elems_per_slot) return;
  const int slot = blockIdx.y, li = blockIdx.z;
  const float g = g_dev ? *g_dev : g_val;
  float* p0 = D.B[li] + (size_t)slot * D.elems_per_slot + e;
  float* p1 = p0 + pair_stride;
  float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
  if (draw) {
    const float4 n4 = z_block(seed, D.tensor_base[li] + slot, 0u, (uint32_t)blk);
    z = make_float4(eps * n4.x, eps * n4.y, eps * n4.z, eps * n4.w);
  }
  const float zz[4] = {z.x, z.y, z.z, z.w};
  const long long left = D.elems_per_slot - e;
  for (int j = 0; j < 4 && j < left; ++j) {
    const float b0 = p0[j], b1 = p1[j];
    const float diff = (b0 - b1) / 2.f;
    const float update = lr * g * diff / eps;
    p0[j] = b0 - diff - update + zz[j];
    p1[j] = b1 + diff - update - zz[j];
  }
}
void launch_pair_update(cudaStream_t st, const UpdateDesc& D, long long pair_stride, const float* g_dev,
                        float g_val, float eps, float lr, uint64_t seed, int draw) {
  const long long blks = (D.elems_per_slot + 3) / 4;
  if (blks <= 0 || D.count <= 0 || D.n_slots <= 0) return;
  dim3 grid((unsigned)((blks + 127) / 128), D.n_slots, D.count);
  pair_update_kernel<<<grid, 128, 0, st>>>(D, pair_stride, g_dev, g_val, eps, lr, seed, draw);
}
// Projected gradient of a stored-pair step, kept on the device for the next step's forward:
// g = (l0 - l1) / (2 eps), or 0 when the step faulted (its update is then a no-op).
__global__ void pair_g_kernel(const double* __restrict__ losses, float* __restrict__ g, float eps,
                              const uint32_t* __restrict__ status) {
  const float v = (float)((losses[0] - losses[1]) / (2.0 * (double)eps));
  g[0] = (*status == 0u && isfinite(v)) ? v : 0.f;
}
void launch_pair_g(cudaStream_t st, const double* losses, float* g, float eps, const uint32_t* status) {
  pair_g_kernel<<<1, 1, 0, st>>>(losses, g, eps, status);
}

void launch_zo_update(cudaStream_t st, const UpdateDesc& D, const double* losses, float* g, int q,
                      float eps, float lr, uint64_t seed, const uint32_t* status, int write_g) {
  const long long blks = (D.elems_per_slot + 3) / 4;
  // a model without adapted projections still gets its g[] written by one (idle) block
  dim3 grid((unsigned)(blks > 0 ? (blks + 127) / 128 : 1), D.n_slots > 0 ? D.n_slots : 1, D.count > 0 ? D.count : 1);
  zo_update_kernel<<<grid, 128, 0, st>>>(D, losses, g, q, eps, lr, seed, status, write_g);
}

// =========================================================================================
// Weight-only dequantisation, once per forward pass for all replicas (appendix "MobiZO with
// weight-only quantization").  16 elements per thread; one fp32 product, one rounding.
// =========================================================================================
__constant__ float c_nf4[16] = {-1.0f, -0.6961928009986877f, -0.5250730514526367f, -0.39491748809814453f,
                                -0.28444138169288635f, -0.18477343022823334f, -0.09105003625154495f, 0.0f,
                                0.07958029955625534f, 0.16093020141124725f, 0.24611230194568634f,
                                0.33791524171829224f, 0.44070982933044434f, 0.5626170039176941f,
                                0.7229568362236023f, 1.0f};
template <typename T>
__global__ void dequant_kernel(int fmt, const uint8_t* __restrict__ codes, const float* __restrict__ scale,
                               T* __restrict__ out, long long total16, int K) {
  // the 16 levels go to shared memory: lanes look up different codes, which constant memory serialises
  __shared__ float tab[16];
  if (threadIdx.x < 16) tab[threadIdx.x] = c_nf4[threadIdx.x];
  __syncthreads();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // group of 16 elements
  if (i >= total16) return;
  const long long e0 = i * 16;
  const long long row = e0 / K;
  const int col = (int)(e0 - row * K);
  float w[16];
  if (fmt == 1) {
    const uint4 raw = *reinterpret_cast<const uint4*>(codes + e0);
    const int8_t* c = reinterpret_cast<const int8_t*>(&raw);
    const float s = scale[row];
#pragma unroll
    for (int j = 0; j < 16; ++j) w[j] = (float)c[j] * s;
  } else {
    const uint2 raw = *reinterpret_cast<const uint2*>(codes + e0 / 2);
    const uint8_t* c = reinterpret_cast<const uint8_t*>(&raw);
    const float s = scale[row * (K / 64) + col / 64];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      w[2 * j] = tab[c[j] >> 4] * s;
      w[2 * j + 1] = tab[c[j] & 15] * s;
    }
  }
  __align__(16) T o[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) o[j] = from_f<T>(w[j]);
  uint4* dst = reinterpret_cast<uint4*>(out + e0);
  const uint4* srcv = reinterpret_cast<const uint4*>(o);
#pragma unroll
  for (int j = 0; j < (int)(16 * sizeof(T) / 16); ++j) dst[j] = srcv[j];
}
void launch_dequant(cudaStream_t st, int bf, int fmt, const void* codes, const float* scale, void* out,
                    int rows, int K) {
  const long long total16 = (long long)rows * K / 16;
  if (total16 <= 0) return;
  const unsigned grid = (unsigned)((total16 + 255) / 256);
  if (bf) dequant_kernel<bf16><<<grid, 256, 0, st>>>(fmt, (const uint8_t*)codes, scale, (bf16*)out, total16, K);
  else dequant_kernel<float><<<grid, 256, 0, st>>>(fmt, (const uint8_t*)codes, scale, (float*)out, total16, K);
}

__global__ void perturbation_kernel(uint64_t seed, uint32_t tensor, uint32_t query, long long n,
                                    uint32_t* u32, float* z) {
  const long long blk = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long e = blk * 4;
  if (e >= n) return;
  const uint4 w = z_words(seed, tensor, query, (uint32_t)blk);
  const float4 zn = z_normals(w);
  const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
  const float zz[4] = {zn.x, zn.y, zn.z, zn.w};
  for (int j = 0; j < 4 && e + j < n; ++j) {
    if (u32) u32[e + j] = ww[j];
    if (z) z[e + j] = zz[j];
  }
}
void launch_perturbation(cudaStream_t st, uint64_t seed, uint32_t tensor, uint32_t query,
                         long long n, uint32_t* u32, float* z) {
  if (n <= 0) return;
  const long long blks = (n + 3) / 4;
  perturbation_kernel<<<(unsigned)((blks + 127) / 128), 128, 0, st>>>(seed, tensor, query, n, u32, z);
}

}  // namespace zo
