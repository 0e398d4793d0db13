// Causal attention for the bf16 path: softmax(Q K^T / sqrt(dh) + causal) V over the n*E
// sequences of the replicated batch (q and k already carry their rotary embedding).
//
// One CTA (4 warps) per (64-query tile, head, sequence); each warp owns 16 query rows.
// K/V tiles of 64 keys stream through cp.async with one buffer each: the next K tile is fetched
// under the softmax and P V of the current one, the next V tile under the next Q K^T, which keeps
// shared memory at three tiles (three CTAs per SM); scores and P V on
// warp-level tensor-core MMAs (m16n8k16, bf16 in, fp32 accumulate) with an online softmax;
// fully masked key tiles are skipped.  Attention is
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

// Asynchronously stage a [64][DH] tile (rows s0.., columns col0.. of qkv) into shared memory.
// Rows >= S are zero-filled (zero-size source).
template <int DH>
__device__ __forceinline__ void stage_tile_async(bf16* dst, const bf16* __restrict__ qkv,
                                                 size_t row_base, int ld, int col0, int s0, int S) {
  constexpr int LDS = DH + 8;
  constexpr int VPR = DH / 8;                          // 16-byte vectors per row
  for (int i = threadIdx.x; i < 64 * VPR; i += 128) {
    const int r = i / VPR, j0 = (i % VPR) * 8;
    const int s = s0 + r;
    const bf16* src = qkv + (row_base + min(s, S - 1)) * (size_t)ld + col0 + j0;
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst + r * LDS + j0);
    const int bytes = s < S ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
  }
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

template <int DH>
__global__ void __launch_bounds__(128, 3)
attention_mma_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ ctx, SeqLayout sl, int Tp,
                     int d) {
  extern __shared__ __align__(16) uint8_t sm_raw[];
  constexpr int LDS = DH + 8;
  bf16* Qs = reinterpret_cast<bf16*>(sm_raw);
  bf16* Ks = Qs + 64 * LDS;
  bf16* Vs = Ks + 64 * LDS;
  const int qt = gridDim.x - 1 - blockIdx.x;          // longest tiles first
  const int q0 = qt * 64, h = blockIdx.y, sq = blockIdx.z;
  const int n = sq / sl.E, b = sq % sl.E;
  const int S = sl.len(b);                                        // this sequence's length
  if (q0 >= S) return;                                            // uniform over the CTA
  const size_t row_base = (size_t)n * Tp + (size_t)sl.start(b);
  const int ld = 3 * d;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;

  const int kend = min(S, q0 + 64);
  const int n_kt = (kend + 63) / 64;
  stage_tile_async<DH>(Qs, qkv, row_base, ld, h * DH, q0, S);
  stage_tile_async<DH>(Ks, qkv, row_base, ld, d + h * DH, 0, S);
  cp_commit();
  stage_tile_async<DH>(Vs, qkv, row_base, ld, 2 * d + h * DH, 0, S);
  cp_commit();
  cp_wait<1>();                                        // Q and K tile 0 have landed (V may be in flight)
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

  for (int kt = 0; kt < n_kt; ++kt) {
    const int k0 = kt * 64;
    const bool more = kt + 1 < n_kt;
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
    __syncthreads();                                            // every warp is done with this K tile
    if (more) {                                                 // next K tile streams in under the rest
      stage_tile_async<DH>(Ks, qkv, row_base, ld, d + h * DH, k0 + 64, S);
      cp_commit();
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
    // O += P V (the V tile was requested one phase earlier)
    if (more) cp_wait<1>(); else cp_wait<0>();
    __syncthreads();
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
    __syncthreads();                                            // every warp is done with this V tile
    if (more) {
      stage_tile_async<DH>(Vs, qkv, row_base, ld, 2 * d + h * DH, k0 + 64, S);
      cp_commit();
      cp_wait<1>();                                             // the next K tile has landed
      __syncthreads();
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

template <int DH>
void launch_t(cudaStream_t st, const void* qkv, void* ctx, int n, SeqLayout sl, int Tp, int d, int H) {
  const int S = sl.S, E = sl.E;
  const size_t smem = (size_t)3 * 64 * (DH + 8) * sizeof(bf16);
  cudaFuncSetAttribute(attention_mma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  dim3 grid((S + 63) / 64, H, n * E);
  attention_mma_kernel<DH><<<grid, 128, smem, st>>>((const bf16*)qkv, (bf16*)ctx, sl, Tp, d);
}

}  // namespace

bool attention_mma_supported(int dh) { return dh == 64 || dh == 128; }

void launch_attention_mma(cudaStream_t st, const void* qkv, void* ctx, int n, SeqLayout sl, int Tp,
                          int d, int H) {
  const int dh = d / H;
  if (dh == 64) launch_t<64>(st, qkv, ctx, n, sl, Tp, d, H);
  else if (dh == 128) launch_t<128>(st, qkv, ctx, n, sl, Tp, d, H);
}

}  // namespace zo
