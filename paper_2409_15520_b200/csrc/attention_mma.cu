// Causal attention for the bf16 path: softmax(Q K^T / sqrt(dh) + causal) V over the n*E
// sequences of the replicated batch, with the rotary embedding of q and k applied while the
// tiles are staged in shared memory (no separate pass over the activations).
//
// One CTA (4 warps) per (64-query tile, head, sequence); each warp owns 16 query rows.
// K/V tiles of 64 keys; scores and P V on warp-level tensor-core MMAs (m16n8k16, bf16 in,
// fp32 accumulate) with an online softmax; fully masked key tiles are skipped.  Attention is
// ~1 % of the step's flops, so this kernel only has to stay off the critical path.
#include "common.cuh"
#include "kernels.h"

namespace zo {
namespace {

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                        uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                          uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                         uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void unpack8f(const uint4 v, float* f) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ uint4 pack8f(const float* f) {
  return make_uint4(pack2(f[0], f[1]), pack2(f[2], f[3]), pack2(f[4], f[5]), pack2(f[6], f[7]));
}

// Stage a [64][DH] tile (rows s0.., columns col0.. of qkv) into shared memory, rotating the
// pairs (j, j + DH/2) by the position's angle when ROT is set.  Rows >= S are zero-filled.
template <int DH, bool ROT>
__device__ __forceinline__ void stage_tile(bf16* dst, const bf16* __restrict__ qkv, size_t row_base,
                                           int ld, int col0, int s0, int S,
                                           const float* __restrict__ rope) {
  constexpr int LDS = DH + 8;
  constexpr int HALF = DH / 2;
  if (ROT) {
    constexpr int VPR = HALF / 8;                     // 16-byte vectors per half row
    for (int i = threadIdx.x; i < 64 * VPR; i += 128) {
      const int r = i / VPR, j0 = (i % VPR) * 8;
      const int s = s0 + r;
      uint4 lo = make_uint4(0, 0, 0, 0), hi = lo;
      if (s < S) {
        const bf16* p = qkv + (row_base + s) * (size_t)ld + col0 + j0;
        float x1[8], x2[8], y1[8], y2[8];
        unpack8f(*reinterpret_cast<const uint4*>(p), x1);
        unpack8f(*reinterpret_cast<const uint4*>(p + HALF), x2);
        const float* cs = rope + (size_t)s * DH + j0;  // [s][cos 0..HALF) | sin 0..HALF)]
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float c = cs[j], sn = cs[HALF + j];
          y1[j] = x1[j] * c - x2[j] * sn;
          y2[j] = x2[j] * c + x1[j] * sn;
        }
        lo = pack8f(y1);
        hi = pack8f(y2);
      }
      *reinterpret_cast<uint4*>(dst + r * LDS + j0) = lo;
      *reinterpret_cast<uint4*>(dst + r * LDS + HALF + j0) = hi;
    }
  } else {
    constexpr int VPR = DH / 8;
    for (int i = threadIdx.x; i < 64 * VPR; i += 128) {
      const int r = i / VPR, j0 = (i % VPR) * 8;
      const int s = s0 + r;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (s < S) v = *reinterpret_cast<const uint4*>(qkv + (row_base + s) * (size_t)ld + col0 + j0);
      *reinterpret_cast<uint4*>(dst + r * LDS + j0) = v;
    }
  }
}

template <int DH, bool ROPE>
__global__ void __launch_bounds__(128)
attention_mma_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ ctx, int E, int S, int Tp,
                     int d, const float* __restrict__ rope) {
  extern __shared__ __align__(16) uint8_t sm_raw[];
  constexpr int LDS = DH + 8;
  bf16* Qs = reinterpret_cast<bf16*>(sm_raw);
  bf16* Ks = Qs + 64 * LDS;
  bf16* Vs = Ks + 64 * LDS;
  const int qt = gridDim.x - 1 - blockIdx.x;          // longest tiles first
  const int q0 = qt * 64, h = blockIdx.y, sq = blockIdx.z;
  const int n = sq / E, b = sq % E;
  const size_t row_base = (size_t)n * Tp + (size_t)b * S;
  const int ld = 3 * d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;

  stage_tile<DH, ROPE>(Qs, qkv, row_base, ld, h * DH, q0, S, rope);
  __syncthreads();
  // Q fragments of this warp's 16 rows stay in registers for the whole kernel
  uint32_t qf[DH / 16][4];
  {
    const int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
    const int c = (lane >> 4) * 8;
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk)
      ldsm_x4((uint32_t)__cvta_generic_to_shared(Qs + r * LDS + kk * 16 + c), qf[kk][0], qf[kk][1],
              qf[kk][2], qf[kk][3]);
  }
  float o[DH / 8][4];
#pragma unroll
  for (int j = 0; j < DH / 8; ++j)
#pragma unroll
    for (int i = 0; i < 4; ++i) o[j][i] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const float sl2 = rsqrtf((float)DH) * 1.4426950408889634f;   // 1/sqrt(dh) * log2(e)
  const int qrow0 = q0 + warp * 16 + g;                         // this thread's rows: qrow0, qrow0+8

  const int kend = min(S, q0 + 64);
  for (int k0 = 0; k0 < kend; k0 += 64) {
    __syncthreads();                                            // previous tile fully consumed
    stage_tile<DH, ROPE>(Ks, qkv, row_base, ld, d + h * DH, k0, S, rope);
    stage_tile<DH, false>(Vs, qkv, row_base, ld, 2 * d + h * DH, k0, S, rope);
    __syncthreads();
    // scores S = Q K^T for 16 rows x 64 keys
    float sc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) sc[j][i] = 0.f;
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
#pragma unroll
      for (int jp = 0; jp < 4; ++jp) {                          // two 8-key tiles per ldmatrix
        uint32_t b0, b1, b2, b3;
        const int key = jp * 16 + (lane & 7) + (lane >> 4) * 8;
        const int c = kk * 16 + ((lane >> 3) & 1) * 8;
        ldsm_x4((uint32_t)__cvta_generic_to_shared(Ks + key * LDS + c), b0, b1, b2, b3);
        mma_bf16(sc[2 * jp], qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3], b0, b1);
        mma_bf16(sc[2 * jp + 1], qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3], b2, b3);
      }
    }
    // causal / length mask (only the diagonal tile and a ragged last tile need it)
    const bool need_mask = (k0 + 64 > q0) || (k0 + 64 > S);
    if (need_mask) {
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int key = k0 + 8 * j + 2 * t + (i & 1);
          const int qr = qrow0 + (i >> 1) * 8;
          if (key > qr || key >= S) sc[j][i] = -INFINITY;
        }
    }
    // online softmax for rows g (i = 0,1) and g + 8 (i = 2,3)
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      mx[0] = fmaxf(mx[0], fmaxf(sc[j][0], sc[j][1]));
      mx[1] = fmaxf(mx[1], fmaxf(sc[j][2], sc[j][3]));
    }
    float corr[2], mnew[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
      mnew[r] = fmaxf(m_run[r], mx[r]);
      // key 0 is visible to every valid query, so mnew is finite from the first tile on
      corr[r] = (m_run[r] == -INFINITY) ? 0.f : exp2f((m_run[r] - mnew[r]) * sl2);
      m_run[r] = mnew[r];
    }
    float ls[2] = {0.f, 0.f};
    uint32_t pf[4][4];                                          // P as A fragments (16 keys each)
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float p0 = exp2f((sc[j][0] - mnew[0]) * sl2), p1 = exp2f((sc[j][1] - mnew[0]) * sl2);
      const float p2 = exp2f((sc[j][2] - mnew[1]) * sl2), p3 = exp2f((sc[j][3] - mnew[1]) * sl2);
      ls[0] += p0 + p1;
      ls[1] += p2 + p3;
      pf[j >> 1][(j & 1) * 2 + 0] = pack2(p0, p1);
      pf[j >> 1][(j & 1) * 2 + 1] = pack2(p2, p3);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) l_run[r] = l_run[r] * corr[r] + ls[r];
#pragma unroll
    for (int j = 0; j < DH / 8; ++j) {
      o[j][0] *= corr[0]; o[j][1] *= corr[0];
      o[j][2] *= corr[1]; o[j][3] *= corr[1];
    }
    // O += P V
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {                            // 16 keys per step
#pragma unroll
      for (int jp = 0; jp < DH / 16; ++jp) {                    // two 8-column tiles per ldmatrix
        uint32_t b0, b1, b2, b3;
        const int key = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
        const int c = jp * 16 + (lane >> 4) * 8;
        ldsm_x4_t((uint32_t)__cvta_generic_to_shared(Vs + key * LDS + c), b0, b1, b2, b3);
        mma_bf16(o[2 * jp], pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], b0, b1);
        mma_bf16(o[2 * jp + 1], pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], b2, b3);
      }
    }
  }
  // normalise and store
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int s = qrow0 + r * 8;
    if (s >= S) continue;
    const float inv = 1.f / l_run[r];
    bf16* op = ctx + (row_base + s) * (size_t)d + h * DH + 2 * t;
#pragma unroll
    for (int j = 0; j < DH / 8; ++j)
      *reinterpret_cast<uint32_t*>(op + 8 * j) = pack2(o[j][2 * r] * inv, o[j][2 * r + 1] * inv);
  }
}

template <int DH, bool ROPE>
void launch_t(cudaStream_t st, const void* qkv, void* ctx, int n, int E, int S, int Tp, int d, int H,
              const float* rope) {
  const size_t smem = (size_t)3 * 64 * (DH + 8) * sizeof(bf16);
  cudaFuncSetAttribute(attention_mma_kernel<DH, ROPE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                       (int)smem);
  dim3 grid((S + 63) / 64, H, n * E);
  attention_mma_kernel<DH, ROPE><<<grid, 128, smem, st>>>((const bf16*)qkv, (bf16*)ctx, E, S, Tp, d, rope);
}

}  // namespace

bool attention_mma_supported(int dh) { return dh == 64 || dh == 128; }

void launch_attention_mma(cudaStream_t st, const void* qkv, void* ctx, int n, int E, int S, int Tp,
                          int d, int H, const float* rope) {
  const int dh = d / H;
  if (dh == 64) {
    if (rope) launch_t<64, true>(st, qkv, ctx, n, E, S, Tp, d, H, rope);
    else launch_t<64, false>(st, qkv, ctx, n, E, S, Tp, d, H, rope);
  } else if (dh == 128) {
    if (rope) launch_t<128, true>(st, qkv, ctx, n, E, S, Tp, d, H, rope);
    else launch_t<128, false>(st, qkv, ctx, n, E, S, Tp, d, H, rope);
  }
}

}  // namespace zo
