// Causal attention for the bf16 path: softmax(Q K^T / sqrt(dh) + causal) V over the n*E
// sequences of the replicated batch (q and k already carry their rotary embedding).
//
// One CTA (8 warps) per (128-query tile, head, sequence); each warp owns 16 query rows.
// K/V stream through cp.async in 64-key tiles with two buffers: the first two tiles are requested
// together with Q before any arithmetic, so a sequence of up to 128 tokens is read exactly once with
// all of its loads in flight at the same time, and longer ones prefetch tile kt+2 while tile kt+1 is
// consumed.  Scores and P V run on warp-level tensor-core MMAs (m16n8k16, bf16 in, fp32 accumulate)
// with an online softmax; a warp skips the key tiles that are fully masked for its rows.  The
// normalised output goes through the warp's own (no longer
// needed) Q rows in shared memory so that global stores are 16 bytes per lane on contiguous row segments.  Attention is ~1 % of the step's flops: the kernel
// is bound by reading q, k, v and writing the context once.
#include "kernels.h"
#include "mma.cuh"

namespace zo {
namespace {

// Asynchronously stage a [ROWS][DH] tile (rows s0.., columns col0.. of the sequence whose first row
// is seq) into shared memory: every thread copies one 16-byte column slot of ROWS*DH/2048 rows.
// Rows >= S are zero-filled (zero-size source).
template <int DH, int ROWS>
__device__ __forceinline__ void stage_tile_async(bf16* dst, const bf16* __restrict__ seq, int ld,
                                                 int col0, int s0, int S) {
  constexpr int LDS = DH + 8;
  constexpr int VPR = DH / 8;                          // 16-byte vectors per row
  constexpr int RSTEP = 256 / VPR;                     // rows covered by one pass of the CTA
  const int r0 = threadIdx.x / VPR, j0 = (threadIdx.x % VPR) * 8;
  const bf16* src0 = seq + col0 + j0;                  // row 0 of the sequence: always readable
  const uint32_t d0 = (uint32_t)__cvta_generic_to_shared(dst + r0 * LDS + j0);
#pragma unroll
  for (int k = 0; k < ROWS / RSTEP; ++k) {
    const int s = s0 + r0 + k * RSTEP;
    const bool ok = s < S;
    cp_async16(d0 + k * RSTEP * LDS * 2, ok ? src0 + (size_t)s * ld : src0, ok ? 16 : 0);
  }
}

// 2^x on the special-function unit (2^-inf = 0).
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int DH>
__global__ void __launch_bounds__(256, 2)
attention_mma_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ ctx, SeqLayout sl, int Tp,
                     int d) {
  extern __shared__ __align__(16) uint8_t sm_raw[];
  constexpr int LDS = DH + 8;
  constexpr int TILE = 64 * LDS;                       // elements of one 64-key K or V tile
  bf16* Qs = reinterpret_cast<bf16*>(sm_raw);          // [128][LDS]
  bf16* Ks = Qs + 128 * LDS;                           // [2][64][LDS]
  bf16* Vs = Ks + 2 * TILE;                            // [2][64][LDS]
  const int qt = gridDim.x - 1 - blockIdx.x;          // longest tiles first
  const int q0 = qt * 128, h = blockIdx.y, sq = blockIdx.z;
  const int n = sq / sl.E, b = sq % sl.E;
  const int S = sl.len(b);                                        // this sequence's length
  if (q0 >= S) return;                                            // uniform over the CTA
  const size_t row_base = (size_t)n * Tp + (size_t)sl.start(b);
  const int ld = 3 * d;
  const bf16* seq = qkv + row_base * ld;                          // first row of this sequence
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;

  const int kend = min(S, q0 + 128);
  const int n_kt = (kend + 63) / 64;
  // one cp.async group per key tile (K and V together); group 0 also carries Q
  stage_tile_async<DH, 128>(Qs, seq, ld, h * DH, q0, S);
  stage_tile_async<DH, 64>(Ks, seq, ld, d + h * DH, 0, S);
  stage_tile_async<DH, 64>(Vs, seq, ld, 2 * d + h * DH, 0, S);
  cp_commit();
  if (n_kt > 1) {
    stage_tile_async<DH, 64>(Ks + TILE, seq, ld, d + h * DH, 64, S);
    stage_tile_async<DH, 64>(Vs + TILE, seq, ld, 2 * d + h * DH, 64, S);
  }
  cp_commit();                                         // (possibly empty: keeps the group count uniform)

  float o[DH / 8][4];
#pragma unroll
  for (int j = 0; j < DH / 8; ++j)
#pragma unroll
    for (int i = 0; i < 4; ++i) o[j][i] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  const float sl2 = rsqrtf((float)DH) * 1.4426950408889634f;   // 1/sqrt(dh) * log2(e)
  const int wrow0 = q0 + warp * 16;                             // first query row of this warp
  const int qrow0 = wrow0 + g;                                  // this thread's rows: qrow0, qrow0+8
  const uint32_t q_addr = (uint32_t)__cvta_generic_to_shared(
      Qs + (warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LDS + (lane >> 4) * 8);

  for (int kt = 0; kt < n_kt; ++kt) {
    const int k0 = kt * 64;
    const bf16* Kt = Ks + (kt & 1) * TILE;
    const bf16* Vt = Vs + (kt & 1) * TILE;
    cp_wait<1>();                                               // tile kt (and Q) has landed
    __syncthreads();
    // keys of this tile that some row of the warp may attend to, and rows that exist at all
    if (k0 <= wrow0 + 15 && wrow0 < S) {
      // scores S = Q K^T for 16 rows x 64 keys
      float sc[8][4];
#pragma unroll
      for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) sc[j][i] = 0.f;
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk) {
        uint32_t a0, a1, a2, a3;
        ldsm_x4(q_addr + kk * 32, a0, a1, a2, a3);
#pragma unroll
        for (int jp = 0; jp < 4; ++jp) {                          // two 8-key tiles per ldmatrix
          uint32_t b0, b1, b2, b3;
          const int key = jp * 16 + (lane & 7) + (lane >> 4) * 8;
          const int c = kk * 16 + ((lane >> 3) & 1) * 8;
          ldsm_x4((uint32_t)__cvta_generic_to_shared(Kt + key * LDS + c), b0, b1, b2, b3);
          mma_bf16(sc[2 * jp], a0, a1, a2, a3, b0, b1);
          mma_bf16(sc[2 * jp + 1], a0, a1, a2, a3, b2, b3);
        }
      }
      // causal / length mask (only tiles that reach past the warp's first row or the sequence end)
      const bool need_mask = (k0 + 64 > wrow0) || (k0 + 64 > S);
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
        // key 0 is visible to every query, so mnew is finite from the first tile on
        corr[r] = ex2((m_run[r] - mnew[r]) * sl2);
        m_run[r] = mnew[r];
      }
      const float nm[2] = {-mnew[0] * sl2, -mnew[1] * sl2};
      float ls[2] = {0.f, 0.f};
      uint32_t pf[4][4];                                          // P as A fragments (16 keys each)
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float p0 = ex2(fmaf(sc[j][0], sl2, nm[0])), p1 = ex2(fmaf(sc[j][1], sl2, nm[0]));
        const float p2 = ex2(fmaf(sc[j][2], sl2, nm[1])), p3 = ex2(fmaf(sc[j][3], sl2, nm[1]));
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
          ldsm_x4_t((uint32_t)__cvta_generic_to_shared(Vt + key * LDS + c), b0, b1, b2, b3);
          mma_bf16(o[2 * jp], pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], b0, b1);
          mma_bf16(o[2 * jp + 1], pf[kk][0], pf[kk][1], pf[kk][2], pf[kk][3], b2, b3);
        }
      }
    }
    if (kt + 2 < n_kt) {                                        // uniform over the CTA
      __syncthreads();                                          // every warp is done with this buffer
      stage_tile_async<DH, 64>(Ks + (kt & 1) * TILE, seq, ld, d + h * DH, k0 + 128, S);
      stage_tile_async<DH, 64>(Vs + (kt & 1) * TILE, seq, ld, 2 * d + h * DH, k0 + 128, S);
    }
    cp_commit();
  }
  cp_wait<0>();
  if (wrow0 >= S) return;                                       // no barrier follows
  // normalise, stage the warp's 16 rows in its own Q rows, store 16 bytes per lane
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xffffffffu, l_run[r], 2);
  }
  bf16* Ow = Qs + warp * 16 * LDS;
  __syncwarp();
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const float inv = 1.f / l_run[r];
    bf16* op = Ow + (g + r * 8) * LDS + 2 * t;
#pragma unroll
    for (int j = 0; j < DH / 8; ++j)
      *reinterpret_cast<uint32_t*>(op + 8 * j) = pack2(o[j][2 * r] * inv, o[j][2 * r + 1] * inv);
  }
  __syncwarp();
  constexpr int VPR = DH / 8, RPI = 32 / VPR;                   // lanes per row, rows per store instruction
#pragma unroll
  for (int i = 0; i < 16 / RPI; ++i) {
    const int r = i * RPI + lane / VPR, c = (lane % VPR) * 8;
    const int s = wrow0 + r;
    if (s < S)
      *reinterpret_cast<uint4*>(ctx + (row_base + s) * (size_t)d + h * DH + c) =
          *reinterpret_cast<const uint4*>(Ow + r * LDS + c);
  }
}

template <int DH>
void launch_t(cudaStream_t st, const void* qkv, void* ctx, int n, SeqLayout sl, int Tp, int d, int H) {
  const int S = sl.S, E = sl.E;
  const size_t smem = (size_t)(128 + 4 * 64) * (DH + 8) * sizeof(bf16);
  cudaFuncSetAttribute(attention_mma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  dim3 grid((S + 127) / 128, H, n * E);
  attention_mma_kernel<DH><<<grid, 256, smem, st>>>((const bf16*)qkv, (bf16*)ctx, sl, Tp, d);
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
