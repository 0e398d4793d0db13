// Shared-input MP-LoRA expansion for the bf16 path (first perturbed layer, Eq. 6 with X^(n) = X):
//   out[n, t, :] = base[t, :] + s * U[t, :] (B + k_n eps z_{n/2})      for the n replicas of a pass,
// where base = X W^T (+ bias) and U = X A^T were computed once on the shared rows.  The op writes
// n*T*k_out outputs from T*k_out inputs: it is bound by the output stream.  One CTA owns a (replica,
// 128-column tile) pair, generates that pair's operand [s B ; s k eps z] (bf16, rank index along K) once
// and sweeps row tiles of 128 tokens; the rank-2r product [U|U] x operand runs on warp-level tensor-core
// MMAs (m16n8k16, fp32 accumulate) and the sum is rounded once to bf16.  Replicas are the fastest grid
// dimension: the CTAs that expand one base tile run together and the tile comes from DRAM once.
// Sections that carry no adapter are copied through the same pipeline.  Two forms:
//   * rank <= 16 (lora_expand_tma_kernel): tiles move by bulk tensor copies in both directions, so the
//     load/store pipe carries one ldmatrix and one stmatrix per 16 x 16 block and nothing else;
//   * rank 17 .. 64 (lora_expand_kernel): every warp stages its 16 rows with cp.async (double-buffered, one
//     tile ahead) and writes 16 bytes per lane on contiguous row segments.
#include "kernels.h"
#include "lora_operand.cuh"
#include "mma.cuh"
#include "tcgen05.cuh"

namespace zo {
namespace {

constexpr int XT = 128;                 // rows and columns of one tile
constexpr int LDC = XT + 8;             // pitch of a staged base/output tile (elements)

// Row tiles one CTA sweeps.  Two CTAs fit an SM, so the grid runs in waves of 2 n_sms CTAs; a (replica,
// column tile) pair swept whole by one CTA leaves the last wave mostly empty at the usual shapes
// (672 pairs on 296 places: 2.3 waves).  The sweep is cut into equal parts: the longest part (the
// generated operand is amortised over it) whose waves are at least 93 % full, else the fullest cut.
int tiles_per_cta(int pairs, int ntile, int n_sms) {
  const long long wave = 2LL * n_sms;
  int best = ntile;
  double best_eff = 0.0;
  for (int z = 1; z <= ntile; ++z) {
    const int per = (ntile + z - 1) / z, parts = (ntile + per - 1) / per;
    const long long waves = ((long long)pairs * parts + wave - 1) / wave;
    const double eff = (double)pairs * ntile / (double)wave / ((double)per * (double)waves);
    if (eff >= 0.93) return per;
    if (eff > best_eff) {
      best_eff = eff;
      best = per;
    }
  }
  return best;
}

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
  const int col0 = blockIdx.y * XT;
  const int sec = col0 / L.width, cs = col0 - sec * L.width;
  const int slot = sec == 0 ? L.slot_of_sec[0] : (sec == 1 ? L.slot_of_sec[1] : L.slot_of_sec[2]);   // uniform over the CTA
  const int n = blockIdx.x;   // replicas of one base tile are neighbours in launch order: the tile comes from DRAM once
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


// ---- rank <= 16: bulk-tensor form ------------------------------------------------------------------
// The same operation with the tile traffic taken off the load/store pipe.  A warp owns 32 rows x 64
// columns of each 128 x 128 tile (one 4 KB box, 128-byte swizzle) and runs a private pipeline on it:
// a bulk tensor load brings the base rows (rows beyond T arrive as zeros), the warp reads them once in
// accumulator-fragment order (ldmatrix), adds the rank-2r product [U|U] x operand (m16n8k16, fp32
// accumulate, operand fragments held in registers for the whole sweep), rounds once to bf16, writes
// the block back in place (stmatrix) and hands the box to a bulk tensor store (rows beyond T of the
// replica are clipped by the 3-D map).  Three boxes per warp: one being loaded, one in work, one being
// stored.  Waits on the load barriers are bounded.
constexpr int WR = 32, WC = 64;         // rows and columns of a warp's box
constexpr int NBOX = 3;
constexpr uint32_t BOX_BYTES = WR * WC * 2;

struct ExpandCtrl {
  unsigned long long full[8][NBOX];
  unsigned long long wait_ns;
  uint32_t abort_flag;
};

template <int KT, bool DUP>          // DUP: 2r == KT, the two halves of [U|U] are the same registers
__global__ void __launch_bounds__(256, 2)
lora_expand_tma_kernel(const __grid_constant__ CUtensorMap base_map, const __grid_constant__ CUtensorMap out_map,
                       int T, LoraDesc L, int tiles_per_cta, unsigned long long wait_ns, uint32_t* status) {
  constexpr int LDB = KT + 8;
  constexpr int NKS = KT / 16;
  extern __shared__ uint8_t sm_dyn[];
  uint8_t* boxes = sm_dyn + ((1024u - (tc::smem_u32(sm_dyn) & 1023u)) & 1023u);   // [8 warps][NBOX][4 KB], 1024-byte aligned
  bf16* Bs = reinterpret_cast<bf16*>(boxes + 8 * NBOX * BOX_BYTES);   // [XT columns][LDB]: operand, K contiguous
  ExpandCtrl* ctl = reinterpret_cast<ExpandCtrl*>(Bs + XT * LDB);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int wr0 = (warp >> 1) * WR, wc0 = (warp & 1) * WC;
  const int col0 = blockIdx.y * XT;
  const int sec = col0 / L.width, cs = col0 - sec * L.width;
  const int slot = sec == 0 ? L.slot_of_sec[0] : (sec == 1 ? L.slot_of_sec[1] : L.slot_of_sec[2]);
  const int n = blockIdx.x;   // replicas of one base tile are neighbours in launch order: the tile comes from DRAM once
  const int r = L.r;
  const int ntile = (T + XT - 1) / XT;
  const int tile0 = blockIdx.z * tiles_per_cta;
  // the warp's last tile is the last one whose first row of the warp's share exists
  const int tile1 = min(min(ntile, tile0 + tiles_per_cta), (T - wr0 + XT - 1) / XT);

  const uint32_t box0 = tc::smem_u32(boxes + (size_t)warp * NBOX * BOX_BYTES);
  const uint32_t bar0 = tc::smem_u32(&ctl->full[warp][0]);
  if (threadIdx.x == 0) {
    ctl->wait_ns = wait_ns;
    ctl->abort_flag = 0u;
  }
  if (lane == 0) {
#pragma unroll
    for (int b = 0; b < NBOX; ++b) tc::mbar_init(bar0 + 8 * b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (tile0 < tile1) {
      tc::mbar_expect_tx(bar0, BOX_BYTES);
      tc::tma_load_2d(box0, &base_map, col0 + wc0, tile0 * XT + wr0, bar0);
    }
  }

  if (slot >= 0) {
    // operand of this (replica, column tile): K index k holds s B[k, col], K index r + k holds
    // s k_n eps z[k, col]; the rest of the K extent is zero
    for (int i = threadIdx.x; i < XT * LDB / 8; i += 256) reinterpret_cast<uint4*>(Bs)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    const int rid = L.rep_base + L.rep_stride * n;
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
  }
  __syncthreads();                                     // operand and control words complete
  if (tile0 >= tile1) return;

  // operand fragments of the warp's 64 columns: [k-step][pair of 8-column tiles] -> {b0, b1 | b0, b1}
  uint32_t bfrag[NKS][WC / 16][4];
  if (slot >= 0) {
#pragma unroll
    for (int ks = 0; ks < NKS; ++ks)
#pragma unroll
      for (int jp = 0; jp < WC / 16; ++jp) {
        const int col = wc0 + jp * 16 + (lane & 7) + (lane >> 4) * 8;
        const int c = ks * 16 + ((lane >> 3) & 1) * 8;
        ldsm_x4(tc::smem_u32(Bs + col * LDB + c), bfrag[ks][jp][0], bfrag[ks][jp][1], bfrag[ks][jp][2],
                bfrag[ks][jp][3]);
      }
  }

  // A = [U | U | 0] of the warp's two 16-row blocks in the fragment order of the m16n8k16 A operand.
  // With 2r == KT every fragment register is one aligned pair of U (rows g and g + 8, columns 2t and
  // 8 + 2t of each 16-wide group; the second half of the K extent repeats the first), fetched one tile
  // ahead as raw fp32 pairs and rounded to bf16 when its tile comes up.  Other ranks gather by element.
  // Rows beyond T repeat row T - 1: their outputs are clipped by the store.
  constexpr int NU = KT / 8;                           // distinct fragment registers of a 16-row block
  float2 raw[2][DUP ? NU : 1];
  auto fetch_u = [&](int tile) {
#pragma unroll
    for (int mb = 0; mb < 2; ++mb) {
      const int ra = tile * XT + wr0 + mb * 16 + g;
      const float* ua = L.U + (size_t)min(ra, T - 1) * L.ldu + slot * r + 2 * t;
      const float* ub = L.U + (size_t)min(ra + 8, T - 1) * L.ldu + slot * r + 2 * t;
#pragma unroll
      for (int j = 0; j < NU / 2; ++j) {
        raw[mb][2 * j] = *reinterpret_cast<const float2*>(ua + 8 * j);
        raw[mb][2 * j + 1] = *reinterpret_cast<const float2*>(ub + 8 * j);
      }
    }
  };
  auto load_a = [&](int tile, int mb, uint32_t (&af)[NKS][4]) {
    const int ra = tile * XT + wr0 + mb * 16 + g, rb = ra + 8;
    const float* ua = L.U + (size_t)min(ra, T - 1) * L.ldu + slot * r;
    const float* ub = L.U + (size_t)min(rb, T - 1) * L.ldu + slot * r;
    auto aval = [&](const float* u, int kk) -> float { return kk < 2 * r ? u[kk < r ? kk : kk - r] : 0.f; };
#pragma unroll
    for (int ks = 0; ks < NKS; ++ks) {
      const int k0 = ks * 16 + 2 * t;
      af[ks][0] = pack2(aval(ua, k0), aval(ua, k0 + 1));
      af[ks][1] = pack2(aval(ub, k0), aval(ub, k0 + 1));
      af[ks][2] = pack2(aval(ua, k0 + 8), aval(ua, k0 + 9));
      af[ks][3] = pack2(aval(ub, k0 + 8), aval(ub, k0 + 9));
    }
  };
  if (DUP && slot >= 0) fetch_u(tile0);

  // lane's 16-byte cell of a 16 x 16 block at (row block mb, column pair jp) inside a swizzled box:
  // row = mb*16 + (lane & 15), 16-byte chunk = 2 jp + (lane >> 4), chunk index XORed with row & 7
  const int lrow = lane & 15, lchunk = lane >> 4;
  int b = 0;                                           // box of the current tile
  uint32_t ph = 0;                                     // its barrier phase
  for (int tile = tile0; tile < tile1; ++tile) {
    const int nb = b + 1 == NBOX ? 0 : b + 1;
    if (lane == 0 && tile + 1 < tile1) {
      tc::tma_store_wait_read<1>();                    // the store that last used box nb (two tiles back) has read it
      tc::mbar_expect_tx(bar0 + 8 * nb, BOX_BYTES);
      tc::tma_load_2d(box0 + nb * BOX_BYTES, &base_map, col0 + wc0, (tile + 1) * XT + wr0, bar0 + 8 * nb);
    }
    uint32_t af[2][NKS][4];
    if (slot >= 0) {
      if constexpr (DUP) {
#pragma unroll
        for (int mb = 0; mb < 2; ++mb)
#pragma unroll
          for (int ks = 0; ks < NKS; ++ks)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 v = raw[mb][(ks * 4 + i) % NU];
              af[mb][ks][i] = pack2(v.x, v.y);
            }
        if (tile + 1 < tile1) fetch_u(tile + 1);       // in flight under this tile's arithmetic
      } else {
        load_a(tile, 0, af[0]);
        load_a(tile, 1, af[1]);
      }
    }
    if (!tc::mbar_wait_bounded(bar0 + 8 * b, ph, &ctl->abort_flag, &ctl->wait_ns, status)) break;
    const uint32_t box = box0 + b * BOX_BYTES;
    if (slot >= 0) {
#pragma unroll
      for (int mb = 0; mb < 2; ++mb) {
#pragma unroll
        for (int jp = 0; jp < WC / 16; ++jp) {
          const int row = mb * 16 + lrow;
          const uint32_t caddr = box + row * 128 + (((2 * jp + lchunk) ^ (row & 7)) << 4);
          uint32_t c0, c1, c2, c3;
          ldsm_x4(caddr, c0, c1, c2, c3);
          float a0[4] = {__uint_as_float(c0 << 16), __uint_as_float(c0 & 0xFFFF0000u),
                         __uint_as_float(c1 << 16), __uint_as_float(c1 & 0xFFFF0000u)};
          float a1[4] = {__uint_as_float(c2 << 16), __uint_as_float(c2 & 0xFFFF0000u),
                         __uint_as_float(c3 << 16), __uint_as_float(c3 & 0xFFFF0000u)};
#pragma unroll
          for (int ks = 0; ks < NKS; ++ks) {
            if (ks * 16 >= 2 * r) break;               // nothing but zeros from here on
            mma_bf16(a0, af[mb][ks][0], af[mb][ks][1], af[mb][ks][2], af[mb][ks][3], bfrag[ks][jp][0],
                     bfrag[ks][jp][1]);
            mma_bf16(a1, af[mb][ks][0], af[mb][ks][1], af[mb][ks][2], af[mb][ks][3], bfrag[ks][jp][2],
                     bfrag[ks][jp][3]);
          }
          stsm_x4(caddr, pack2(a0[0], a0[1]), pack2(a0[2], a0[3]), pack2(a1[0], a1[1]), pack2(a1[2], a1[3]));
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the block as the bulk store will read it
    }
    __syncwarp();
    if (lane == 0) {
      tc::tma_store_3d(&out_map, col0 + wc0, tile * XT + wr0, n, box);
      tc::tma_store_commit();
    }
    if (nb == 0) ph ^= 1u;
    b = nb;
  }
  if (lane == 0) tc::tma_store_wait_read<0>();         // shared memory stays until the last store has read it
}

template <int KT, bool DUP>
int launch_tma(cudaStream_t st, const void* base, int ldb, void* out, int ldo, int n, int T, const LoraDesc& L,
               int nsec, int n_sms, unsigned long long wait_ns, uint32_t* status) {
  const uint64_t ncols = (uint64_t)nsec * L.width;
  CUtensorMap bm, om;
  {
    const uint64_t dims[2] = {ncols, (uint64_t)T}, strides[1] = {(uint64_t)ldb * 2};
    const uint32_t box[2] = {WC, WR};
    if (tc_make_map_bf16_nd(&bm, base, 2, dims, strides, box)) return 1;
  }
  {
    const uint64_t dims[3] = {ncols, (uint64_t)T, (uint64_t)n};
    const uint64_t strides[2] = {(uint64_t)ldo * 2, (uint64_t)L.rows_per_replica * ldo * 2};
    const uint32_t box[3] = {WC, WR, 1};
    if (tc_make_map_bf16_nd(&om, out, 3, dims, strides, box)) return 1;
  }
  const size_t smem = 8 * NBOX * BOX_BYTES + (size_t)XT * (KT + 8) * sizeof(bf16) + sizeof(ExpandCtrl) + 1024;
  cudaFuncSetAttribute(lora_expand_tma_kernel<KT, DUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  const int ctiles = (int)(ncols / XT), ntile = (T + XT - 1) / XT;
  const int per = tiles_per_cta(ctiles * n, ntile, n_sms);
  dim3 grid(n, ctiles, (ntile + per - 1) / per);
  lora_expand_tma_kernel<KT, DUP><<<grid, 256, smem, st>>>(bm, om, T, L, per, wait_ns, status);
  return 0;
}

template <int KT>
void launch_t(cudaStream_t st, const void* base, int ldb, void* out, int ldo, int n, int T,
              const LoraDesc& L, int nsec, int n_sms) {
  const size_t smem = (size_t)(XT * (KT + 8) + 2 * XT * LDC) * sizeof(bf16);
  cudaFuncSetAttribute(lora_expand_kernel<KT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  const int ctiles = nsec * L.width / XT, ntile = (T + XT - 1) / XT;
  const int per = tiles_per_cta(ctiles * n, ntile, n_sms);
  dim3 grid(n, ctiles, (ntile + per - 1) / per);
  lora_expand_kernel<KT><<<grid, 256, smem, st>>>((const bf16*)base, ldb, (bf16*)out, ldo, T, L, per);
}

}  // namespace

bool lora_expand_supported(const void* base, int ldb, const void* out, int ldo, const LoraDesc& L) {
  return L.width % XT == 0 && L.r >= 1 && L.r <= 64 && ldb % 8 == 0 && ldo % 8 == 0 &&
         (((uintptr_t)base | (uintptr_t)out | (uintptr_t)L.B) & 15) == 0;
}

void launch_lora_expand(cudaStream_t st, const void* base, int ldb, void* out, int ldo, int n, int T,
                        const LoraDesc& L, int nsec, int n_sms, uint32_t* status) {
  if (n <= 0 || T <= 0) return;
  if (L.r <= 16 && status != nullptr) {                // bulk-tensor form; the form below if a map cannot be made
    int e;
    if (L.r == 8) e = launch_tma<16, true>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms, 2000000000ull, status);
    else if (L.r == 16) e = launch_tma<32, true>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms, 2000000000ull, status);
    else if (L.r < 8) e = launch_tma<16, false>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms, 2000000000ull, status);
    else e = launch_tma<32, false>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms, 2000000000ull, status);
    if (e == 0) return;
  }
  if (L.r <= 8) launch_t<16>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms);
  else if (L.r <= 16) launch_t<32>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms);
  else if (L.r <= 32) launch_t<64>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms);
  else launch_t<128>(st, base, ldb, out, ldo, n, T, L, nsec, n_sms);
}

}  // namespace zo
