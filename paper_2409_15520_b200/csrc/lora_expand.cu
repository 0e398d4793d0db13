// Shared-input MP-LoRA expansion for the bf16 path (first perturbed layer, Eq. 6 with X^(n) = X):
//   out[n, t, :] = base[t, :] + s * U[t, :] (B + k_n eps z_{n/2})      for the n replicas of a pass,
// where base = X W^T (+ bias) and U = X A^T were computed once on the shared rows.  The op writes
// n*T*k_out outputs from T*k_out inputs: it is bound by the output stream, so everything is arranged
// for full-line accesses.  One CTA owns a (replica, 128-column tile) pair, generates that pair's
// operand [s B ; s k eps z] (bf16, rank index along K) once, and sweeps row tiles of 128 tokens.
// Inside a tile every warp runs a private pipeline on its 16 rows: the base rows arrive through
// cp.async (double-buffered, one tile ahead), the rank-2r product [U|U] x operand runs on warp-level
// tensor-core MMAs (m16n8k16, fp32 accumulate), the sum is rounded once to bf16 and leaves through
// shared memory as 16 bytes per lane on contiguous row segments.  Sections that carry
// no adapter are copied through the same pipeline.
#include "kernels.h"
#include "lora_operand.cuh"
#include "mma.cuh"

namespace zo {
namespace {

constexpr int XT = 128;                 // rows and columns of one tile
constexpr int LDC = XT + 8;             // pitch of a staged base/output tile (elements)

template <int KT>                       // K extent of the generated operand (>= 2r, multiple of 16)
__global__ void __launch_bounds__(256, 2)
lora_expand_kernel(const bf16* __restrict__ base, int ldb, bf16* __restrict__ out, int ldo, int T,
                   LoraDesc L, int tiles_per_cta) {
  constexpr int LDB = KT + 8;
  extern __shared__ __align__(16) uint8_t sm_raw[];
  bf16* Bs = reinterpret_cast<bf16*>(sm_raw);          // [XT columns][LDB]: operand, K contiguous
  bf16* Cs = Bs + XT * LDB;                            // [2][XT rows][LDC]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int col0 = blockIdx.x * XT;
  const int sec = col0 / L.width, cs = col0 - sec * L.width;
  const int slot = sec == 0 ? L.slot_of_sec[0] : (sec == 1 ? L.slot_of_sec[1] : L.slot_of_sec[2]);   // uniform over the CTA
  const int n = blockIdx.y;
  const int Tp = L.rows_per_replica, r = L.r;
  const int ntile = (T + XT - 1) / XT;
  const int tile0 = blockIdx.z * tiles_per_cta, tile1 = min(ntile, tile0 + tiles_per_cta);
  if (tile0 >= tile1) return;

  // Every warp runs its own pipeline over its 16 rows of each row tile: it stages those rows itself,
  // so after the operand is built no CTA-wide barrier is needed.
  bf16* Cw0 = Cs + warp * 16 * LDC;                    // the warp's rows in buffer 0 (buffer 1: + XT * LDC)
  auto stage_base = [&](int tile, int buf) {
    const int wrow0 = tile * XT + warp * 16;
    const int j0 = (lane & 15) * 8;
    const bf16* src0 = base + col0 + j0;
    const uint32_t d0 = (uint32_t)__cvta_generic_to_shared(Cw0 + buf * XT * LDC + (lane >> 4) * LDC + j0);
#pragma unroll
    for (int k = 0; k < 8; ++k) {                      // two rows of 256 bytes per pass
      const int row = wrow0 + 2 * k + (lane >> 4);
      const bool ok = row < T;
      cp_async16(d0 + 2 * k * LDC * 2, ok ? src0 + (size_t)row * ldb : src0, ok ? 16 : 0);
    }
  };
  stage_base(tile0, 0);
  cp_commit();

  if (slot >= 0) {
    // operand of this (replica, column tile): K index k holds s B[k, col], K index r + k holds
    // s k_n eps z[k, col]; the rest of the K extent is zero
    for (int i = threadIdx.x; i < XT * LDB / 8; i += 256) reinterpret_cast<uint4*>(Bs)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    const int rid = L.rep_base + L.rep_stride * n;     // replica id within the step
    for (int i = threadIdx.x; i < r * (XT / 4); i += 256) {
      const int k = i / (XT / 4), c4 = (i % (XT / 4)) * 4;
      float4 b, z;
      lora_operand(L, slot, (size_t)k * L.width + cs + c4, rid, b, z);
      const float bb[4] = {b.x, b.y, b.z, b.w}, zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        Bs[(c4 + j) * LDB + k] = __float2bfloat16_rn(bb[j] * L.scale);
        Bs[(c4 + j) * LDB + r + k] = __float2bfloat16_rn(zz[j] * L.scale);
      }
    }
    __syncthreads();                                   // operand complete: the only CTA-wide hand-over
  }

  // A = [U | U | 0] of the warp's 16 rows of a tile, rounded to bf16 as it is loaded (fragment order of
  // the m16n8k16 A operand).  Short operands are fetched one tile ahead.
  constexpr int NKS = KT / 16;
  constexpr bool PREFETCH_A = KT <= 32;
  auto load_a = [&](int tile, uint32_t (&af)[NKS][4]) {
    const int ra = tile * XT + warp * 16 + g, rb = ra + 8;
    const float* ua = L.U + (size_t)min(ra, T - 1) * L.ldu + slot * r;
    const float* ub = L.U + (size_t)min(rb, T - 1) * L.ldu + slot * r;
    auto aval = [&](const float* u, bool ok, int kk) -> float {
      return (ok && kk < 2 * r) ? u[kk < r ? kk : kk - r] : 0.f;
    };
#pragma unroll
    for (int ks = 0; ks < NKS; ++ks) {
      const int k0 = ks * 16 + 2 * t;
      af[ks][0] = pack2(aval(ua, ra < T, k0), aval(ua, ra < T, k0 + 1));
      af[ks][1] = pack2(aval(ub, rb < T, k0), aval(ub, rb < T, k0 + 1));
      af[ks][2] = pack2(aval(ua, ra < T, k0 + 8), aval(ua, ra < T, k0 + 9));
      af[ks][3] = pack2(aval(ub, rb < T, k0 + 8), aval(ub, rb < T, k0 + 9));
    }
  };
  uint32_t af[NKS][4];
  if (slot >= 0 && PREFETCH_A) load_a(tile0, af);

  for (int tile = tile0; tile < tile1; ++tile) {
    const int buf = (tile - tile0) & 1;
    __syncwarp();                                      // every lane is done with the other buffer
    if (tile + 1 < tile1) stage_base(tile + 1, buf ^ 1);
    cp_commit();                                       // (possibly empty: keeps the group count uniform)
    const int wrow0 = tile * XT + warp * 16;           // first token row of this warp
    float acc[XT / 8][4];
#pragma unroll
    for (int j = 0; j < XT / 8; ++j)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;
    if (slot >= 0 && wrow0 < T) {
      if (!PREFETCH_A) load_a(tile, af);
#pragma unroll
      for (int ks = 0; ks < NKS; ++ks) {
        if (ks * 16 >= 2 * r) break;                   // nothing but zeros from here on
#pragma unroll
        for (int jp = 0; jp < XT / 16; ++jp) {          // two 8-column tiles per ldmatrix
          uint32_t b0, b1, b2, b3;
          const int col = jp * 16 + (lane & 7) + (lane >> 4) * 8;
          const int c = ks * 16 + ((lane >> 3) & 1) * 8;
          ldsm_x4((uint32_t)__cvta_generic_to_shared(Bs + col * LDB + c), b0, b1, b2, b3);
          mma_bf16(acc[2 * jp], af[ks][0], af[ks][1], af[ks][2], af[ks][3], b0, b1);
          mma_bf16(acc[2 * jp + 1], af[ks][0], af[ks][1], af[ks][2], af[ks][3], b2, b3);
        }
      }
      if (PREFETCH_A && tile + 1 < tile1) load_a(tile + 1, af);   // lands under the stores below
    }
    cp_wait<1>();                                      // this lane's share of the tile's base rows has landed
    __syncwarp();                                      // ... and so has every other lane's
    if (wrow0 >= T) continue;
    bf16* Cw = Cw0 + buf * XT * LDC;
    if (slot >= 0) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        bf16* cp = Cw + (g + h * 8) * LDC + 2 * t;
#pragma unroll
        for (int j = 0; j < XT / 8; ++j) {
          const uint32_t w = *reinterpret_cast<const uint32_t*>(cp + 8 * j);
          const float b0 = __uint_as_float(w << 16), b1 = __uint_as_float(w & 0xFFFF0000u);
          *reinterpret_cast<uint32_t*>(cp + 8 * j) = pack2(acc[j][2 * h] + b0, acc[j][2 * h + 1] + b1);
        }
      }
      __syncwarp();
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {                      // two rows of 256 bytes per store instruction
      const int rr = 2 * i + (lane >> 4), c = (lane & 15) * 8;
      const int row = wrow0 + rr;
      if (row < T)
        *reinterpret_cast<uint4*>(out + ((size_t)n * Tp + row) * ldo + col0 + c) =
            *reinterpret_cast<const uint4*>(Cw + rr * LDC + c);
    }
  }
  cp_wait<0>();
}

template <int KT>
void launch_t(cudaStream_t st, const void* base, int ldb, void* out, int ldo, int n, int T,
              const LoraDesc& L, int nsec, int n_sms) {
  const size_t smem = (size_t)(XT * (KT + 8) + 2 * XT * LDC) * sizeof(bf16);
  cudaFuncSetAttribute(lora_expand_kernel<KT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  const int ctiles = nsec * L.width / XT, ntile = (T + XT - 1) / XT;
  // enough CTAs for a few waves; beyond that, longer row sweeps amortise the generated operand
  int z = (4 * n_sms + ctiles * n - 1) / (ctiles * n);
  z = z < 1 ? 1 : (z > ntile ? ntile : z);
  const int per = (ntile + z - 1) / z;
  z = (ntile + per - 1) / per;
  dim3 grid(ctiles, n, z);
  lora_expand_kernel<KT><<<grid, 256, smem, st>>>((const bf16*)base, ldb, (bf16*)out, ldo, T, L, per);
}

}  // namespace

bool lora_expand_supported(const void* base, int ldb, const void* out, int ldo, const LoraDesc& L) {
  return L.width % XT == 0 && L.r >= 1 && L.r <= 64 && ldb % 8 == 0 && ldo % 8 == 0 &&
         (((uintptr_t)base | (uintptr_t)out | (uintptr_t)L.B) & 15) == 0;
}

void launch_lora_expand(cudaStream_t st, const void* base, int ldb, void* out, int ldo, int n, int T,
                        const LoraDesc& L, int nsec, int n_sms) {
  if (n <= 0 || T <= 0) return;
  if (L.r <= 8) launch_t<16>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms);
  else if (L.r <= 16) launch_t<32>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms);
  else if (L.r <= 32) launch_t<64>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms);
  else launch_t<128>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms);
}

}  // namespace zo
