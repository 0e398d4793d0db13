// bf16 tensor-core GEMM for sm_100a:  out = A W^T with fused epilogues.
//
//   * operands staged by TMA (cp.async.bulk.tensor, 128-byte swizzle, no multicast) through a
//     4-deep shared-memory ring, one elected thread issues tcgen05.mma (128 x 256 x 16 per
//     instruction), fp32 accumulators live in tensor memory, two accumulator buffers so the
//     epilogue of tile i overlaps the main loop of tile i+1; persistent CTAs, one per SM.
//   * epilogue (8 warps, two per tensor-memory lane quarter, tcgen05.ld): bias, ReLU, residual add, SiLU(gate)*up, float or
//     bfloat16 output, and the MP-LoRA term of the paper's layer equation
//         Y_n = X_n W + s * U_n (B + k_n eps z_i)
//     with z_i regenerated from the Philox seed inside the epilogue (never in HBM).  Every
//     128-row tile lies inside one replica, so the perturbed B columns of the tile are built
//     once in shared memory and reused by its 128 rows.
//   * Tensor-core form of the MP-LoRA term (rank <= 32, sections that are a multiple of the
//     256-column tile, single-CTA variant): the term becomes one extra 64-deep k-block of the
//     same accumulator.  Its A operand is a bf16 copy of U laid out [U | U] (written by the
//     down-projection's epilogue, loaded by TMA), its B operand [s B ; s k eps z] is generated
//     by the epilogue warps straight into shared memory in the swizzled K-major layout the MMA
//     expects, one tile ahead.  Keeping B and k eps z in separate K ranges keeps the
//     perturbation's resolution in bf16 whatever the magnitude of B.  Otherwise the term is
//     added on CUDA cores in the epilogue from fp32 U and fp32 (B + k eps z).
//   * PAIR variant: two CTAs of a cluster work on one 256 x 256 tile with tcgen05.mma.cta_group::2 -
//     each CTA stages its own 128 rows of A and its 128-row half of the weight tile, so the L2
//     traffic per flop drops by a third; 6 stages.  The leader CTA issues the MMAs and releases
//     stages/accumulators in both CTAs with multicast commits; the peer's TMA completes on the
//     leader's barrier.  The one-block LoRA form rides along (each CTA generates the operand rows
//     it stages; the peer's epilogue warps arrive on the leader's barrier).  It keeps the tensor
//     pipe busier per clock; under the 1 kW power cap of the largest shapes that only lowers the
//     clock, so the host takes it for mid-size launches only (launch_gemm_tc).
//   * split K for small batches (far fewer tiles than SMs, cost = the stream of weights): a first
//     launch computes one K range of a tile per CTA and stores fp32 parts, a second launch of the
//     same template sums them in K order and runs the fused epilogue; no CTA waits for another.
//   * every mbarrier wait is bounded; on expiry the kernel raises ST_TIMEOUT in the status
//     word, drains its copies and MMAs, frees its tensor memory and returns.
#include <cuda.h>

#include <atomic>
#include <mutex>

#include "common.cuh"
#include "kernels.h"
#include "lora_operand.cuh"
#include "tcgen05.cuh"

namespace zo {

namespace tc {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int MAX_STAGES = 9;                   // narrow-output launches with a 32-row weight box: nine stages of 20 KiB
constexpr uint32_t A_BYTES = BM * BK * 2;       // 16 KiB
constexpr uint32_t BOX_BYTES = 128 * BK * 2;    // one 128-row box of the weight tile, 16 KiB
template <bool PAIR> struct Cfg {
  static constexpr int STAGES = PAIR ? 6 : 4;
  static constexpr uint32_t B_BYTES = PAIR ? BOX_BYTES : 2 * BOX_BYTES;   // per CTA
  static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr uint32_t TX_BYTES = PAIR ? 2 * STAGE_BYTES : STAGE_BYTES;  // per full barrier
};
constexpr int LORA_MAXR = 64;
constexpr uint32_t LORA_BUF_FLOATS = LORA_MAXR * 32;  // one 32-column chunk of s*(B + k eps z)
constexpr uint32_t TMEM_COLS = 512;
constexpr int EP_WARPS = 8;                     // two per tensor-memory lane quarter, alternating chunks
constexpr int EP_THREADS = EP_WARPS * 32;
constexpr int THREADS = 64 + EP_THREADS;        // warp 0: TMA, warp 1: MMA, warps 2-9: epilogue
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

struct Ctrl {
  unsigned long long full[MAX_STAGES], empty[MAX_STAGES], tfull[2], tempty[2], drain, lfull;
  unsigned long long rawfull[2], rawempty[2];   // ring of quantised-code groups (kernels that decode weights)
  unsigned long long wait_ns;       // limit of every bounded wait of this CTA
  uint32_t tmem_base;
  volatile uint32_t abort;
  volatile uint32_t ep_go;
};
constexpr uint32_t SLAB_BYTES = BN * BK * 2;     // generated B operand of the LoRA k-block (aliases the fp32 staging)
constexpr size_t SMEM_BYTES = 1024 + 4 * 49152 + SLAB_BYTES + sizeof(Ctrl);  // both variants: 192 KiB of stages
constexpr size_t SMEM_BYTES_SUM = 1024 + SLAB_BYTES + sizeof(Ctrl);          // summing launch of split K: no ring

struct Params {
  int M, N, K;              // N: accumulator columns (swiglu: d_ffn, the number of OUTPUT columns)
  void* out; int ldo; int out_f32;
  const bf16* bias;
  const bf16* res; int ldr; int res_mod;
  int act, swiglu;
  const float* rope_tab;    // non-null: rotate q and k (columns < rope_cols) in the epilogue
  int rope_cols, rope_dh, rope_s, rope_tp;
  const int32_t* rope_pos;  // packed variable-length rows: position of row (m % rope_tp), else null
  int group_m;              // 128-row tiles per raster group
  int has_lora;
  int slab;                 // 1: the LoRA term is one or two extra k-blocks on the tensor cores
  int kslot, khalf;         // K extent of one slot in the packed bf16 U, offset of its second copy
  bf16* pack_out; int pack_ld;  // down-projection: also write the packed bf16 U here (or null)
  int pack_r;
  LoraDesc L;
  uint32_t* status;
  int n_half;               // 1: at most 128 output columns in all: one weight box per stage, MMAs of N = bbox
  int bbox;                 // rows of that box (32, 64 or 128: the smallest that holds N): a down-projection is a
                            // stream of activations, and the bytes not spent on weight rows are stages in flight
  int ksplit;               // > 1: the K range of every tile is cut into ksplit units of work
  float4* part;             // ksplit > 1: fp32 partial accumulators, [unit][64 column quads][128 rows]
  // Cross-entropy head: instead of storing the tile, every thread folds the logits of its row into a
  // running (max, sum of exp) pair and stores one pair per (row, column tile, sibling warp); the label's
  // logit is stored by the thread that holds its column.  The logits never reach memory.
  float2* ce_part;          // [M][tiles_n][2] or null
  float* ce_logit;          // [M]
  const int32_t* ce_label;  // label of row m = ce_label[m % ce_ep] (< 0: row not in the loss)
  int ce_ep;
  // Weight-only quantised B operand decoded inside the kernel (small batches: the GEMM is a stream of
  // weights, and a weight is then read once, as codes): 0 = bf16 weights through TMA, 1 = int8 codes with one
  // scale per row, 2 = NF4 codes (two per byte, blocks of 64 along K) with one absmax per row and k-block.
  int wfmt;
  const uint8_t* wq;
  const float* wscale;
  unsigned long long wait_ns;   // limit of the bounded waits (WAIT_LIMIT_NS unless a failure-detection test shortens it)
  int withhold;             // failure-detection test: CTA 0 never delivers the second k-block of its first tile
};

// The 16 levels of the 4-bit NormalFloat format (Dettmers et al., "QLoRA"): normal quantiles scaled to [-1, 1].
__constant__ float c_nf4_levels[16] = {-1.0f, -0.6961928009986877f, -0.5250730514526367f, -0.39491748809814453f,
                                       -0.28444138169288635f, -0.18477343022823334f, -0.09105003625154495f, 0.0f,
                                       0.07958029955625534f, 0.16093020141124725f, 0.24611230194568634f,
                                       0.33791524171829224f, 0.44070982933044434f, 0.5626170039176941f,
                                       0.7229568362236023f, 1.0f};

// Bounded wait of this kernel's roles (limit and abort flag live in the CTA's control block).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, Ctrl* c, uint32_t* status) {
  return mbar_wait_bounded(bar, parity, &c->abort, &c->wait_ns, status);
}
__device__ __forceinline__ void ep_bar() { asm volatile("bar.sync 1, %0;" ::"n"(EP_THREADS) : "memory"); }
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 256.
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                           ((uint32_t)(BM >> 4) << 24);
// The pair instruction spans both CTAs: M = 256.
// The same with N = 32, 64 or 128 (launches with at most 128 output columns, e.g. the LoRA down-projection).
__device__ __forceinline__ constexpr uint32_t idesc_n(uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}
constexpr uint32_t IDESC_PAIR = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                                ((uint32_t)((2 * BM) >> 4) << 24);

// Tile raster: groups of GROUP_M row tiles sweep all column tiles, so a wave of CTAs shares
// both a few weight panels and a bounded set of activation panels in L2.
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int GROUP_M, int& tm,
                                            int& tn) {
  const int per_group = GROUP_M * tiles_n;
  const int g = tile / per_group, r = tile - g * per_group;
  const int gm0 = g * GROUP_M;
  const int gsz = min(GROUP_M, tiles_m - gm0);
  tn = r / gsz;
  tm = gm0 + (r - tn * gsz);
}

// Columns of perturbed B staged per generation phase: as many as fit the 16 KiB staging area,
// a multiple of 32, at most one tile.
__device__ __forceinline__ int lora_phase_cols(int r) {
  const int g = ((int)(2 * LORA_BUF_FLOATS) / r) & ~31;
  return g > 256 ? 256 : g;
}
// Up to 16 consecutive floats of a U row (zero-padded), issued back to back.
__device__ __forceinline__ void load_u16(const float* p, int left, bool vec, float (&u)[16]) {
  if (vec && left >= 16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float4 t = reinterpret_cast<const float4*>(p)[i];
      u[4 * i] = t.x; u[4 * i + 1] = t.y; u[4 * i + 2] = t.z; u[4 * i + 3] = t.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) u[i] = i < left ? p[i] : 0.f;
  }
}

// Slab mode: the LoRA slot of the tile whose first output column is n0 (-1: not adapted).
__device__ __forceinline__ int tile_slot(const Params& P, int n0) {
  return P.slab ? P.L.slot_of_sec[n0 / P.L.width] : -1;
}

// Position in the operand ring: stage and phase advance by counting, so the per-k-block path of the
// producer, the MMA issuer and the decode warps carries no division (the stage count is a run-time value).
struct RingPos {
  uint32_t s = 0, ph = 0;
  __device__ __forceinline__ void advance(uint32_t stages) {
    if (++s == stages) { s = 0; ph ^= 1u; }
  }
};

// SPLIT 0: every CTA (pair) computes whole tiles.  Split K, for launches with far fewer tiles than SMs
// whose cost is the stream of weights (small batches), takes two launches of this kernel: SPLIT 1
// computes one K range of a tile per unit of work and stores the fp32 accumulator to scratch; SPLIT 2
// runs no MMA at all: its CTAs take a quarter of a tile's column chunks each, sum the parts in K order
// (so the result does not depend on timing) and run the same fused epilogue as SPLIT 0.
constexpr int FIN_GROUPS = 4;
// WQ: the B operand is decoded inside the kernel from weight-only quantised codes (instantiated apart so
// that the decode path costs the bf16 kernels no registers).
// CE: the cross-entropy head (epilogue folds the logits instead of storing them); also its own instantiation.
template <bool PAIR, int SPLIT, bool WQ = false, bool CE = false>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmU, const Params P) {
  // ring depth: one stage is given up when the LoRA term needs two generated k-blocks (rank > 32);
  // narrow-output launches stage one weight box, so the same 192 KiB hold six stages of 32 KiB
  const bool narrow = !PAIR && P.n_half;
  // (the kernels that decode quantised weights keep two stages: the other two hold the ring of raw codes)
  const int STAGES = PAIR ? Cfg<PAIR>::STAGES
                          : (narrow && !WQ ? (P.bbox == 32 ? 9 : (P.bbox == 64 ? 8 : 6))
                                           : Cfg<PAIR>::STAGES - (P.slab && P.kslot > 64 ? 1 : 0) - (WQ ? 2 : 0));
  const uint32_t STAGE_BYTES = narrow && !WQ ? A_BYTES + (uint32_t)P.bbox * 128u : Cfg<PAIR>::STAGE_BYTES;
  constexpr int TILE_M = PAIR ? 2 * BM : BM;           // rows of one scheduled tile
  const int GROUP_M = PAIR ? (P.group_m + 1) / 2 : P.group_m;   // row tiles of a raster group
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  // the summing launch of split K stages nothing: its shared memory starts at the LoRA staging area
  float* lbuf = (float*)(smem + (SPLIT == 2 ? 0 : STAGES * STAGE_BYTES));
  Ctrl* ctrl = (Ctrl*)(smem + (SPLIT == 2 ? 0 : Cfg<PAIR>::STAGES * Cfg<PAIR>::STAGE_BYTES) + SLAB_BYTES);
  // quantised weights: two slots of raw codes (a group of k-blocks: 256 rows x 128 bytes each) behind the slab area
  constexpr uint32_t RAW_BYTES = 2 * BOX_BYTES;
  uint8_t* raw_ring = smem + STAGES * STAGE_BYTES + (P.kslot > 64 ? 2 : 1) * SLAB_BYTES;
  const uint32_t tiles_base = smem_u32(smem);
  const uint32_t rank = PAIR ? cluster_rank() : 0u;    // 0 = leader of the pair
  const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int n_units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (P.M + TILE_M - 1) / TILE_M;
  const int ncol_tile = P.swiglu ? 128 : BN;          // output columns covered by one tile
  const int tiles_n = (P.N + ncol_tile - 1) / ncol_tile;
  const int num_tiles = tiles_m * tiles_n;
  const int num_kb = (P.K + BK - 1) / BK;
  // Work schedule of this CTA (pair): units unit, unit + n_units, ...  A unit is a tile of the grouped
  // raster, or with split K one of the ksplit K ranges of a tile.
  const int ksplit = SPLIT ? P.ksplit : 1;
  const int t_first = unit, t_step = n_units, t_end = num_tiles * ksplit;
  auto coords = [&](int t, int& tm, int& tn) { tile_coords(t / ksplit, tiles_m, tiles_n, GROUP_M, tm, tn); };
  auto kb_range = [&](int t, int& ks, int& kb0, int& kb1) {
    ks = t % ksplit;
    kb0 = (int)((long long)ks * num_kb / ksplit);
    kb1 = (int)((long long)(ks + 1) * num_kb / ksplit);
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_STAGES; ++s) {
      // a quantised B operand is written into the stage by the eight decode warps, who arrive too
      mbar_init(smem_u32(&ctrl->full[s]), WQ ? 1 + EP_WARPS : 1);
      mbar_init(smem_u32(&ctrl->empty[s]), 1);
    }

    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&ctrl->tfull[a]), 1);
      mbar_init(smem_u32(&ctrl->tempty[a]), PAIR ? 2 * EP_WARPS : EP_WARPS);
    }
    if (WQ) {
      for (int r = 0; r < 2; ++r) {
        mbar_init(smem_u32(&ctrl->rawfull[r]), 1);
        mbar_init(smem_u32(&ctrl->rawempty[r]), EP_WARPS);
      }
    }
    mbar_init(smem_u32(&ctrl->drain), 1);
    mbar_init(smem_u32(&ctrl->lfull), PAIR ? 2 * EP_WARPS : EP_WARPS);
    ctrl->abort = 0u;
    ctrl->ep_go = 0u;
    ctrl->wait_ns = P.wait_ns;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1 && SPLIT != 2) {
    if (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                       smem_u32(&ctrl->tmem_base)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                       smem_u32(&ctrl->tmem_base)),
                   "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync();                            // the peer's barriers are initialised too
  tc_fence_after();
  const uint32_t tmem_base = ctrl->tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0 && SPLIT != 2) {
      uint32_t issued = 0;
      RingPos rp;
      bool ok = true, withheld = false;
      for (int tile = t_first; tile < t_end && ok && !withheld; tile += t_step) {
        int tm, tn;
        coords(tile, tm, tn);
        const int m0 = tm * TILE_M + (int)rank * BM;
        const int brow0 = tn * ncol_tile;
        const int brow1 = P.swiglu ? P.N + brow0 : brow0 + 128;
        int ks, kb0, kb1;
        kb_range(tile, ks, kb0, kb1);
        for (int kb = kb0; kb < kb1; ++kb, ++issued, rp.advance(STAGES)) {
          // failure-detection test: this producer goes silent (nothing armed, nothing in flight), so the
          // MMA warp's wait for the stage runs out and the CTA takes its abort path
          if (!PAIR && P.withhold && blockIdx.x == 0 && issued == (kb1 - kb0 > 1 ? 1u : 0u)) { withheld = true; break; }
          const uint32_t s = rp.s, ph = rp.ph;
          if (!mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, ctrl, P.status)) { ok = false; break; }
          const uint32_t bar = smem_u32(&ctrl->full[s]);
          const uint32_t sa = tiles_base + s * STAGE_BYTES;
          if (PAIR) {
            // the leader's barrier collects the bytes of both CTAs
            if (rank == 0) mbar_expect_tx(bar, Cfg<PAIR>::TX_BYTES);
            tma_load_2d_pair(sa, &tmA, kb * BK, m0, bar);
            tma_load_2d_pair(sa + A_BYTES, &tmB, kb * BK, rank == 0 ? brow0 : brow1, bar);
          } else if (WQ) {
            mbar_expect_tx(bar, A_BYTES);            // the B operand of the stage comes from the decode warps
            tma_load_2d(sa, &tmA, kb * BK, m0, bar);
          } else {
            mbar_expect_tx(bar, P.n_half ? A_BYTES + (uint32_t)P.bbox * 128u : Cfg<PAIR>::TX_BYTES);
            tma_load_2d(sa, &tmA, kb * BK, m0, bar);
            tma_load_2d(sa + A_BYTES, &tmB, kb * BK, brow0, bar);
            if (!P.n_half) tma_load_2d(sa + A_BYTES + BOX_BYTES, &tmB, kb * BK, brow1, bar);
          }
        }
        const int lslot = ks != 0 ? -1 : tile_slot(P, brow0);   // the LoRA block rides with the first K range
        for (int lkb = 0; ok && !withheld && lslot >= 0 && lkb < P.kslot / BK; ++lkb, ++issued, rp.advance(STAGES)) {
          // LoRA k-blocks: only the A operand (packed U) travels through the ring
          const uint32_t s = rp.s, ph = rp.ph;
          if (!mbar_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u, ctrl, P.status)) { ok = false; break; }
          const uint32_t bar = smem_u32(&ctrl->full[s]);
          if (PAIR) {
            if (rank == 0) mbar_expect_tx(bar, 2 * A_BYTES);     // each CTA brings the U rows of its half
            tma_load_2d_pair(tiles_base + s * STAGE_BYTES, &tmU, lslot * P.kslot + lkb * BK, m0, bar);
          } else {
            mbar_expect_tx(bar, A_BYTES);
            tma_load_2d(tiles_base + s * STAGE_BYTES, &tmU, lslot * P.kslot + lkb * BK, m0, bar);
          }
        }
        if (!ok) break;
      }
      if (!ok && (!PAIR || rank == 0)) {
        // abort: let the copies already issued land before the CTA goes away
        const uint32_t lo = issued > STAGES ? issued - STAGES : 0u;
        for (uint32_t i = lo; i < issued; ++i)
          mbar_wait_drain(smem_u32(&ctrl->full[i % STAGES]), (i / STAGES) & 1u);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && rank == 0 && SPLIT != 2) {
      uint32_t titer = 0, ltiles = 0;
      RingPos rp;
      const uint32_t idesc_main = PAIR ? IDESC_PAIR : (P.n_half ? idesc_n((uint32_t)P.bbox) : IDESC);
      bool ok = true;
      for (int tile = t_first; tile < t_end && ok; tile += t_step, ++titer) {
        const uint32_t a = titer & 1u, aph = (titer >> 1) & 1u;
        if (!mbar_wait(smem_u32(&ctrl->tempty[a]), aph ^ 1u, ctrl, P.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * BN;
        int ks, kb0, kb1;
        kb_range(tile, ks, kb0, kb1);
        for (int kb = kb0; kb < kb1; ++kb, rp.advance(STAGES)) {
          const uint32_t s = rp.s, ph = rp.ph;
          if (!mbar_wait(smem_u32(&ctrl->full[s]), ph, ctrl, P.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = tiles_base + s * STAGE_BYTES;
          const uint64_t ad = smem_desc(sa), bd = smem_desc(sa + A_BYTES);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            if (PAIR)
              tc_mma_pair(d_tmem, ad + (uint64_t)(2 * k), bd + (uint64_t)(2 * k), idesc_main,
                          (uint32_t)(((kb - kb0) | k) != 0));
            else
              tc_mma(d_tmem, ad + (uint64_t)(2 * k), bd + (uint64_t)(2 * k), idesc_main,
                     (uint32_t)(((kb - kb0) | k) != 0));
          }
          // frees the stage (in both CTAs of a pair) once these MMAs retire
          if (PAIR) tc_commit_pair(smem_u32(&ctrl->empty[s]));
          else tc_commit(smem_u32(&ctrl->empty[s]));
        }
        if (ok) {
          int tm, tn;
          coords(tile, tm, tn);
          if (ks == 0 && tile_slot(P, tn * ncol_tile) >= 0) {
            for (int lkb = 0; lkb < P.kslot / BK; ++lkb, rp.advance(STAGES)) {
              const uint32_t s = rp.s, ph = rp.ph;
              if (!mbar_wait(smem_u32(&ctrl->full[s]), ph, ctrl, P.status) ||
                  (lkb == 0 && !mbar_wait(smem_u32(&ctrl->lfull), ltiles & 1u, ctrl, P.status))) { ok = false; break; }
              tc_fence_after();
              const uint64_t ad = smem_desc(tiles_base + s * STAGE_BYTES);
              const uint64_t bd = smem_desc(tiles_base + STAGES * STAGE_BYTES + lkb * SLAB_BYTES);
#pragma unroll
              for (int k = 0; k < BK / 16; ++k) {
                if (PAIR) tc_mma_pair(d_tmem, ad + (uint64_t)(2 * k), bd + (uint64_t)(2 * k), IDESC_PAIR, 1u);
                else tc_mma(d_tmem, ad + (uint64_t)(2 * k), bd + (uint64_t)(2 * k), IDESC, 1u);
              }
              if (PAIR) tc_commit_pair(smem_u32(&ctrl->empty[s]));
              else tc_commit(smem_u32(&ctrl->empty[s]));
            }
            if (!ok) break;
            ++ltiles;
          }
        }
        if (ok) {
          if (PAIR) tc_commit_pair(smem_u32(&ctrl->tfull[a]));
          else tc_commit(smem_u32(&ctrl->tfull[a]));
        }
      }
      if (!ok) {
        // wait for the MMAs already issued (a pair's instructions are tracked by the pair form of the commit)
        if (PAIR) tc_commit_pair(smem_u32(&ctrl->drain));
        else tc_commit(smem_u32(&ctrl->drain));
        mbar_wait_drain(smem_u32(&ctrl->drain), 0u);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int wq = warp & 3;                       // tensor-memory lane quarter of this warp
    const int et = threadIdx.x - 64;               // 0..EP_THREADS-1
    const int half = (warp - 2) >> 2;              // which of the quarter's two warps: even or odd chunks
    const bool out_vec_ok = ((uintptr_t)P.out & 15) == 0 && (P.ldo % (P.out_f32 ? 4 : 8)) == 0;
    // a lane reads and writes its own row, so an access instruction touches 32 rows whatever its width:
    // 32-byte accesses (whole sectors) halve the number of such instructions of a bf16 tile
    const bool out_wide_ok = !P.out_f32 && ((uintptr_t)P.out & 31) == 0 && P.ldo % 16 == 0;
    const bool res_wide_ok = ((uintptr_t)P.res & 31) == 0 && P.ldr % 16 == 0;
    const bool out_f32_wide_ok = P.out_f32 && ((uintptr_t)P.out & 31) == 0 && P.ldo % 8 == 0;
    const bool pack_wide_ok = ((uintptr_t)P.pack_out & 31) == 0 && P.pack_ld % 16 == 0 && P.kslot % 16 == 0 &&
                              P.khalf % 16 == 0 && P.N % 8 == 0;
    const bool res_vec_ok = ((uintptr_t)P.res & 15) == 0 && (P.ldr % 8) == 0;
    const bool bias_vec_ok = ((uintptr_t)P.bias & 15) == 0;   // col0 is a multiple of 32 elements
    uint8_t* slab = smem + (SPLIT == 2 ? 0 : STAGES * STAGE_BYTES);
    // Slab mode: build the B operand [s B ; s k eps z] of a tile's LoRA k-block: 256 rows (output
    // columns) x 64 K-elements, K-major with the 128-byte swizzle.  Rank index k sits at K = k
    // (B part) and K = khalf + k (perturbation part); all other K positions stay zero.
    auto gen_slab = [&](int g_tile) {
      int tm, tn;
      coords(g_tile, tm, tn);
      const int n0g = tn * ncol_tile;
      const int slot = tile_slot(P, n0g);
      if (slot < 0 || g_tile % ksplit != 0) return;  // uniform over the CTA (same decision as the MMA warp's)
      const int sec = n0g / P.L.width, cs = n0g - sec * P.L.width;
      const int repg = P.L.rep_base + P.L.rep_stride * ((tm * TILE_M) / P.L.rows_per_replica);
      const int kgroups = (P.L.r + 7) / 8;
      constexpr int CQ = PAIR ? 32 : 64;               // column quads of the operand rows this CTA holds
      // the operand is generated by the four epilogue warps that share no scheduler with the TMA producer
      // (warp 0) and the MMA issuer (warp 1): the Philox / Box-Muller bursts then cost those two no issue
      // slots, and their waits sit on the latency chain of the operand ring
      const int gen_i = (warp & 2) ? ((warp >> 2) & 1) * 64 + (warp & 1) * 32 + lane : -1;   // warps 2, 3, 6, 7
      for (int unit_i = gen_i; unit_i >= 0 && unit_i < CQ * kgroups; unit_i += EP_THREADS / 2) {
        const int c4l = (unit_i % CQ) * 4, k0 = (unit_i / CQ) * 8;
        const int c4 = c4l + (PAIR ? (int)rank * 128 : 0);       // column inside the 256-column tile
        float bb[8][4], zz[8][4];
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const int k = k0 + kk;
          float4 b = make_float4(0.f, 0.f, 0.f, 0.f), z = b;
          if (k < P.L.r) lora_operand(P.L, slot, (size_t)k * P.L.width + cs + c4, repg, b, z);
          bb[kk][0] = b.x * P.L.scale; bb[kk][1] = b.y * P.L.scale; bb[kk][2] = b.z * P.L.scale; bb[kk][3] = b.w * P.L.scale;
          zz[kk][0] = z.x * P.L.scale; zz[kk][1] = z.y * P.L.scale; zz[kk][2] = z.z * P.L.scale; zz[kk][3] = z.w * P.L.scale;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int n = c4l + j;                      // row of this CTA's operand tile = output column
          const uint4 vb = make_uint4(pack_bf16(bb[0][j], bb[1][j]), pack_bf16(bb[2][j], bb[3][j]),
                                      pack_bf16(bb[4][j], bb[5][j]), pack_bf16(bb[6][j], bb[7][j]));
          const uint4 vz = make_uint4(pack_bf16(zz[0][j], zz[1][j]), pack_bf16(zz[2][j], zz[3][j]),
                                      pack_bf16(zz[4][j], zz[5][j]), pack_bf16(zz[6][j], zz[7][j]));
          // 16-byte chunk index along K; K >= 64 lives in the second generated k-block
          const int cb = k0 >> 3, pz = P.khalf + k0, cz = (pz & 63) >> 3;
          *reinterpret_cast<uint4*>(slab + n * 128 + ((cb ^ (n & 7)) << 4)) = vb;
          *reinterpret_cast<uint4*>(slab + (pz >> 6) * SLAB_BYTES + n * 128 + ((cz ^ (n & 7)) << 4)) = vz;
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the tensor core
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_leader(smem_u32(&ctrl->lfull));        // the leader's MMA warp waits for both halves
        else mbar_arrive(smem_u32(&ctrl->lfull));
      }
    };
    if (P.slab && SPLIT != 2) {
      for (int i = et; i < (int)(SLAB_BYTES / 16) * (P.kslot / BK); i += EP_THREADS)
        reinterpret_cast<uint4*>(slab)[i] = make_uint4(0, 0, 0, 0);
      ep_bar();
    }
    if (P.slab && SPLIT != 2 && t_first < t_end) gen_slab(t_first);
    // Quantised weights: these warps are the producer of the B operand.  The codes of a GROUP of k-blocks
    // (128 bytes of every one of the tile's 256 weight rows: 4 k-blocks of NF4, 2 of int8) are brought
    // into a two-slot ring in shared memory by bulk tensor copies (issued by the first decode warp, one
    // group ahead), so the weight stream moves in full lines with many bytes in flight.  Thread `et`
    // owns row `et` of the operand tile (= one output column): it reads the row's codes from the slot and
    // writes each k-block as eight 16-byte chunks of bf16 into the stage, in the swizzled K-major layout
    // of the TMA path.  One fp32 product and one rounding per weight, as the stand-alone decoder does.
    // The warps run independently (each polls the barriers itself, one lane per warp).
    RingPos dq;                                      // ring position (mirrors the TMA producer's)
    uint32_t rgroups = 0;                            // code groups consumed so far (slot and phase of the ring)
    bool dq_ok = true;                               // this warp's waits so far succeeded
    auto warp_wait = [&](uint32_t bar, uint32_t parity) -> bool {   // one lane waits, all lanes learn the outcome
      uint32_t ok = 1u;
      if (lane == 0) ok = mbar_wait(bar, parity, ctrl, P.status) ? 1u : 0u;
      return __shfl_sync(0xffffffffu, ok, 0) != 0u;
    };
    auto decode_unit = [&](int d_tile) {
      if constexpr (!WQ) return;
      int tm, tn, ks, kb0, kb1;
      coords(d_tile, tm, tn);
      kb_range(d_tile, ks, kb0, kb1);
      const int brow0 = tn * ncol_tile;
      const int brow1 = P.swiglu ? P.N + brow0 : brow0 + 128;
      const int wrow = et < 128 ? brow0 + et : brow1 + (et - 128);
      const bool live = (P.swiglu ? (brow0 + (et & 127)) < P.N : wrow < P.N) && !(P.n_half && et >= 128);
      const int nkb_all = P.K / BK;
      const bool nf4 = P.wfmt == 2;
      const int DQ_G = nf4 ? 4 : 2;                  // k-blocks per 128-byte group of a row's codes
      const float* srow = P.wscale + (nf4 ? (size_t)wrow * nkb_all : (size_t)wrow);
      const float rscale = (!nf4 && live) ? srow[0] : 0.f;
      // group `gr` of this CTA's sequence -> ring slot gr & 1; its codes start at k-block g0
      auto issue_group = [&](uint32_t gr, int g0) -> bool {       // first decode warp only
        const uint32_t slot = gr & 1u, ph = (gr >> 1) & 1u;
        if (!warp_wait(smem_u32(&ctrl->rawempty[slot]), ph ^ 1u)) return false;
        if (lane == 0) {
          const uint32_t bar = smem_u32(&ctrl->rawfull[slot]);
          const uint32_t dst = smem_u32(raw_ring + slot * RAW_BYTES);
          const int xb = g0 * (nf4 ? 32 : 64);                    // byte offset inside a weight row
          mbar_expect_tx(bar, P.n_half ? BOX_BYTES : RAW_BYTES);
          tma_load_2d(dst, &tmB, xb, brow0, bar);
          if (!P.n_half) tma_load_2d(dst + BOX_BYTES, &tmB, xb, brow1, bar);
        }
        return true;
      };
      float csc[4] = {0.f, 0.f, 0.f, 0.f}, nsc[4] = {0.f, 0.f, 0.f, 0.f};
      auto load_scales = [&](int g0, float (&sc)[4]) {
#pragma unroll
        for (int j = 0; j < 4; ++j) sc[j] = (nf4 && live && g0 + j < kb1) ? __ldg(srow + g0 + j) : 0.f;
      };
      if (warp == 2) dq_ok = issue_group(rgroups, kb0);
      load_scales(kb0, csc);
      for (int g0 = kb0; g0 < kb1 && dq_ok; g0 += DQ_G, ++rgroups) {
        if (g0 + DQ_G < kb1) {
          if (warp == 2) dq_ok = issue_group(rgroups + 1, g0 + DQ_G);
          load_scales(g0 + DQ_G, nsc);
          if (!dq_ok) break;
        }
        const uint32_t slot = rgroups & 1u;
        if (!warp_wait(smem_u32(&ctrl->rawfull[slot]), (rgroups >> 1) & 1u)) { dq_ok = false; break; }
        // this thread's 128 code bytes of the group, chunk c16 at its swizzled place
        const uint8_t* rrow = raw_ring + slot * RAW_BYTES + (et >> 7) * BOX_BYTES + (et & 127) * 128;
#pragma unroll
        for (int gi = 0; gi < 4; ++gi) {
          const int kb = g0 + gi;
          if (gi < DQ_G && kb < kb1 && dq_ok) {       // uniform over the warp
            const uint32_t s = dq.s, ph = dq.ph;
            dq_ok = warp_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u);
            if (dq_ok) {
              uint8_t* brow = smem + s * STAGE_BYTES + A_BYTES + et * 128;
              if (!(P.n_half && et >= 128)) {
                if (nf4) {
                  // The 16 possible values of this (row, k-block), level x scale rounded to bf16 exactly as
                  // the stand-alone decode rounds them, held as byte planes in registers: lo[m] / hi[m] are
                  // the low / high bytes of entries 4m .. 4m + 3.  A weight is then two byte selections
                  // (no table in shared memory, no multiply per weight).
                  const float sc = csc[gi];
                  uint32_t lo[4], hi[4];
#pragma unroll
                  for (int m = 0; m < 4; ++m) {
                    const uint32_t t0 = pack_bf16(c_nf4_levels[4 * m] * sc, c_nf4_levels[4 * m + 1] * sc);
                    const uint32_t t1 = pack_bf16(c_nf4_levels[4 * m + 2] * sc, c_nf4_levels[4 * m + 3] * sc);
                    lo[m] = __byte_perm(t0, t1, 0x6420);
                    hi[m] = __byte_perm(t0, t1, 0x7531);
                  }
#pragma unroll
                  for (int h = 0; h < 2; ++h) {       // 16 code bytes = 32 weights = 4 output chunks
                    const uint4 q4 = *reinterpret_cast<const uint4*>(rrow + (((2 * gi + h) ^ (et & 7)) << 4));
                    const uint32_t cw[4] = {q4.x, q4.y, q4.z, q4.w};
                    uint32_t o[16];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {     // one code word = 8 weights = one output chunk
                      // byte b of the word: element 2b in the high nibble, 2b + 1 in the low one, so the four
                      // nibbles of a 16-bit half are elements 1, 0, 3, 2.  Selector a picks entry (code & 7)
                      // of either half of the table, selector b then takes the half that bit 3 names.
                      const uint32_t a32 = cw[i] & 0x77777777u;
                      const uint32_t b32 = ((cw[i] >> 1) & 0x44444444u) | 0x32103210u;
#pragma unroll
                      for (int hh = 0; hh < 2; ++hh) {
                        const uint32_t a = hh ? a32 >> 16 : a32, b = hh ? b32 >> 16 : b32;
                        const uint32_t l = __byte_perm(__byte_perm(lo[0], lo[1], a), __byte_perm(lo[2], lo[3], a), b);
                        const uint32_t u = __byte_perm(__byte_perm(hi[0], hi[1], a), __byte_perm(hi[2], hi[3], a), b);
                        o[4 * i + 2 * hh] = __byte_perm(l, u, 0x4051);        // elements 0 | 1
                        o[4 * i + 2 * hh + 1] = __byte_perm(l, u, 0x6273);    // elements 2 | 3
                      }
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                      *reinterpret_cast<uint4*>(brow + (((4 * h + c) ^ (et & 7)) << 4)) =
                          make_uint4(o[4 * c], o[4 * c + 1], o[4 * c + 2], o[4 * c + 3]);
                  }
                } else {
#pragma unroll
                  for (int h = 0; h < 4; ++h) {       // 16 code bytes = 16 weights = 2 output chunks
                    const uint4 q4 = *reinterpret_cast<const uint4*>(rrow + (((4 * gi + h) ^ (et & 7)) << 4));
                    const uint32_t cw[4] = {q4.x, q4.y, q4.z, q4.w};
                    float w[16];
                    // int8 -> float without a conversion instruction: byte b ^ 0x80 placed in the low mantissa
                    // byte of 2^23 is the float 8388608 + (b + 128), so subtracting 8388736 leaves b exactly
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                      const uint32_t bits = __byte_perm(cw[i >> 2] ^ 0x80808080u, 0x4B000000u, 0x7650 + (i & 3));
                      w[i] = (__uint_as_float(bits) - 8388736.f) * rscale;
                    }
#pragma unroll
                    for (int c = 0; c < 2; ++c)
                      *reinterpret_cast<uint4*>(brow + (((2 * h + c) ^ (et & 7)) << 4)) =
                          make_uint4(pack_bf16(w[8 * c], w[8 * c + 1]), pack_bf16(w[8 * c + 2], w[8 * c + 3]),
                                     pack_bf16(w[8 * c + 4], w[8 * c + 5]), pack_bf16(w[8 * c + 6], w[8 * c + 7]));
                  }
                }
              }
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the tensor core
              __syncwarp();
              if (lane == 0) mbar_arrive(smem_u32(&ctrl->full[s]));
              dq.advance(STAGES);
            }
          }
        }
        // done with the slot (on the abort path nobody refills it)
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->rawempty[slot]));
#pragma unroll
        for (int j = 0; j < 4; ++j) csc[j] = nsc[j];
      }
      // the LoRA k-blocks of the unit bring only their A operand through the ring: arrive for the stage
      if (ks == 0 && tile_slot(P, brow0) >= 0) {
        for (int lkb = 0; lkb < P.kslot / BK && dq_ok; ++lkb) {
          const uint32_t s = dq.s, ph = dq.ph;
          dq_ok = warp_wait(smem_u32(&ctrl->empty[s]), ph ^ 1u);
          if (dq_ok) {
            if (lane == 0) mbar_arrive(smem_u32(&ctrl->full[s]));
            dq.advance(STAGES);
          }
        }
      }
    };
    constexpr bool wq_mode = WQ;
    uint32_t titer = 0;
    // iteration space: the units of this CTA; in the summing launch (tile, chunk group) pairs
    const int e_first = SPLIT == 2 ? (int)blockIdx.x : t_first;
    const int e_step = SPLIT == 2 ? (int)gridDim.x : t_step;
    const int e_end = SPLIT == 2 ? num_tiles * FIN_GROUPS : t_end;
    for (int it = e_first; it < e_end; it += e_step, ++titer) {
      const int tile = SPLIT == 2 ? (it / FIN_GROUPS) * ksplit : it;   // (summing launch: first unit of the tile)
      const int grp = SPLIT == 2 ? it % FIN_GROUPS : -1;
      const uint32_t a = titer & 1u, aph = (titer >> 1) & 1u;
      if constexpr (WQ) {
        // this unit's operands first: its LoRA operand (the first unit's was built above; the slab is free
        // again because the previous unit's accumulator has been waited for), then its decoded weights
        // (a warp whose wait ran out stops decoding; the CTA-wide decision to leave is taken at the wait
        // for the accumulator below, where one thread sees the abort flag for all)
        if (P.slab && titer > 0) gen_slab(tile);
        decode_unit(tile);
      }
      if (SPLIT != 2) {
        if (et == 0) ctrl->ep_go = mbar_wait(smem_u32(&ctrl->tfull[a]), aph, ctrl, P.status) ? 1u : 0u;
        ep_bar();
        const bool go = ctrl->ep_go != 0u;
        ep_bar();                                    // ep_go may be rewritten after this point
        if (!go) break;
        tc_fence_after();
        // this tile's MMAs have retired, so the slab is free: build the next tile's operand first
        if (P.slab && !wq_mode && tile + t_step < t_end) gen_slab(tile + t_step);
      }
      int tm, tn;
      coords(tile, tm, tn);
      const int m0 = tm * TILE_M + (int)rank * BM, n0 = tn * ncol_tile;
      const int row = m0 + wq * 32 + lane;
      const bool row_ok = row < P.M;
      const uint32_t taddr = tmem_base + ((uint32_t)(wq * 32) << 16) + a * BN;
      constexpr bool split = SPLIT != 0;
      if (SPLIT == 1) {
        // deliver this unit's partial accumulator (the chunks that hold output columns; lanes = rows are
        // contiguous in the scratch layout, so every access is a full 512-byte segment) and hand the
        // accumulator buffer back
        float4* pu = P.part + (size_t)tile * 64 * 128 + wq * 32 + lane;
        const int cvalid = P.swiglu ? 8 : min(8, (P.N - n0 + 31) / 32);   // chunks that hold output columns
        for (int c = half; c < cvalid; c += 2) {
          uint32_t v[32];
          tc_ld32(taddr + c * 32, v);
          tc_ld_wait();
#pragma unroll
          for (int j4 = 0; j4 < 8; ++j4)
            pu[(size_t)(c * 8 + j4) * 128] =
                make_float4(__uint_as_float(v[4 * j4]), __uint_as_float(v[4 * j4 + 1]),
                            __uint_as_float(v[4 * j4 + 2]), __uint_as_float(v[4 * j4 + 3]));
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->tempty[a]));
        continue;
      }
      // accumulator chunk `cchunk` (32 columns) of this thread's row: from tensor memory, or the sum of
      // the tile's parts
      auto load_acc = [&](int cchunk, uint32_t (&v)[32]) {
        if (!split) {
          tc_ld32(taddr + cchunk * 32, v);
          return;
        }
        const float4* pp = P.part + (size_t)tile * 64 * 128 + (size_t)cchunk * 8 * 128 + wq * 32 + lane;
        float sacc[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) sacc[j] = 0.f;
        // two parts per round: the loads of a round are all in flight before the first add, and the
        // adds stay in K order
        for (int s2 = 0; s2 < ksplit; s2 += 2, pp += 2 * 64 * 128) {
          const bool two = s2 + 1 < ksplit;
          float4 t0[8], t1[8];
#pragma unroll
          for (int j4 = 0; j4 < 8; ++j4) t0[j4] = __ldcg(pp + j4 * 128);
#pragma unroll
          for (int j4 = 0; j4 < 8; ++j4) t1[j4] = two ? __ldcg(pp + 64 * 128 + j4 * 128) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int j4 = 0; j4 < 8; ++j4) {
            sacc[4 * j4] += t0[j4].x; sacc[4 * j4 + 1] += t0[j4].y; sacc[4 * j4 + 2] += t0[j4].z; sacc[4 * j4 + 3] += t0[j4].w;
          }
          if (two) {
#pragma unroll
            for (int j4 = 0; j4 < 8; ++j4) {
              sacc[4 * j4] += t1[j4].x; sacc[4 * j4 + 1] += t1[j4].y; sacc[4 * j4 + 2] += t1[j4].z; sacc[4 * j4 + 3] += t1[j4].w;
            }
          }
        }
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(sacc[j]);
      };
      const int rrow = P.res ? (P.res_mod > 0 ? row % P.res_mod : row) : 0;
      // the rotary table row of this thread's token, once per tile (two divisions by run-time values)
      const float* rope_row = nullptr;
      if (P.rope_tab && row_ok)
        rope_row = P.rope_tab + (size_t)(P.rope_pos ? P.rope_pos[row % P.rope_tp] : (row % P.rope_tp) % P.rope_s) * P.rope_dh;
      // per-tile LoRA constants: all rows of the tile belong to one replica
      const int rep = P.has_lora ? P.L.rep_base + P.L.rep_stride * (m0 / P.L.rows_per_replica) : 0;
      const float* urow = P.has_lora ? P.L.U + (size_t)min(row, P.M - 1) * P.L.ldu : nullptr;
      const bool u_vec = P.has_lora && (P.L.ldu % 4 == 0) && (P.L.r % 4 == 0) && (((uintptr_t)P.L.U & 15) == 0);
      const int nchunk = ncol_tile / 32;
      const int po = P.rope_tab ? (P.rope_dh >> 6) : 0;          // 128 -> 2, 64 -> 1, <= 32 -> 0 (same chunk)
      const int pshift = po == 1 ? 1 : 0;                      // keep both chunks of a pair with one warp
      // The perturbed B columns are staged G columns at a time (the whole 256-column tile for
      // rank <= 16): one generation phase, two barriers, then barrier-free chunks.
      const int G = P.has_lora ? lora_phase_cols(P.L.r) : 256;
      const int cpp = G / 32;                      // chunks per generation phase
      // residual add (before any rotation: the rotary embedding applies to the finished projection)
      auto add_res = [&](int col0, float (&f)[32]) {
        if (!P.res) return;
        const bool full_chunk = col0 + 32 <= P.N;
        const bf16* rp = P.res + (size_t)rrow * P.ldr + col0;
        if (full_chunk && res_wide_ok) {
#pragma unroll
          for (int j16 = 0; j16 < 2; ++j16) {
            uint32_t w[8];
            asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                         : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                         : "l"(rp + 16 * j16));
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              f[16 * j16 + 2 * j] += __uint_as_float(w[j] << 16);
              f[16 * j16 + 2 * j + 1] += __uint_as_float(w[j] & 0xFFFF0000u);
            }
          }
        } else if (full_chunk && res_vec_ok) {
#pragma unroll
          for (int j8 = 0; j8 < 4; ++j8) {
            float t[8];
            unpack8(*reinterpret_cast<const uint4*>(rp + 8 * j8), t);
#pragma unroll
            for (int j = 0; j < 8; ++j) f[8 * j8 + j] += t[j];
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (col0 + j < P.N) f[j] += to_f(rp[j]);
        }
      };
      // store of one 32-column chunk of this thread's row
      auto emit = [&](int col0, float (&f)[32]) {
        const bool full_chunk = col0 + 32 <= P.N;
        // 16-byte vector accesses need the row pitch (and base) to keep rows 16-byte aligned
        const bool vec_out = full_chunk && out_vec_ok;
        if (P.out_f32) {
          float* op = (float*)P.out + (size_t)row * P.ldo + col0;
          if (full_chunk && out_f32_wide_ok) {
#pragma unroll
            for (int j8 = 0; j8 < 4; ++j8)
              asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(op + 8 * j8), "f"(f[8 * j8]),
                           "f"(f[8 * j8 + 1]), "f"(f[8 * j8 + 2]), "f"(f[8 * j8 + 3]), "f"(f[8 * j8 + 4]), "f"(f[8 * j8 + 5]),
                           "f"(f[8 * j8 + 6]), "f"(f[8 * j8 + 7])
                           : "memory");
          } else if (vec_out) {
#pragma unroll
            for (int j4 = 0; j4 < 8; ++j4)
              *reinterpret_cast<float4*>(op + 4 * j4) =
                  make_float4(f[4 * j4], f[4 * j4 + 1], f[4 * j4 + 2], f[4 * j4 + 3]);
          } else {
            #pragma unroll
            for (int j = 0; j < 32; ++j)
              if (col0 + j < P.N) op[j] = f[j];
          }
        } else {
          bf16* op = (bf16*)P.out + (size_t)row * P.ldo + col0;
          if (full_chunk && out_wide_ok) {
#pragma unroll
            for (int j16 = 0; j16 < 2; ++j16) {
              uint32_t o[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) o[j] = pack_bf16(f[16 * j16 + 2 * j], f[16 * j16 + 2 * j + 1]);
              asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(op + 16 * j16), "r"(o[0]), "r"(o[1]),
                           "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7])
                           : "memory");
            }
          } else if (vec_out) {
#pragma unroll
            for (int j8 = 0; j8 < 4; ++j8)
              *reinterpret_cast<uint4*>(op + 8 * j8) =
                  make_uint4(pack_bf16(f[8 * j8], f[8 * j8 + 1]), pack_bf16(f[8 * j8 + 2], f[8 * j8 + 3]),
                             pack_bf16(f[8 * j8 + 4], f[8 * j8 + 5]), pack_bf16(f[8 * j8 + 6], f[8 * j8 + 7]));
          } else {
            #pragma unroll
            for (int j = 0; j < 32; ++j)
              if (col0 + j < P.N) op[j] = __float2bfloat16_rn(f[j]);
          }
        }
      };
      float ce_m = -INFINITY, ce_s = 0.f;          // cross-entropy head: this thread's share of the tile
      int ce_lab = -1;
      if constexpr (CE) ce_lab = row_ok ? P.ce_label[row % P.ce_ep] : -1;
      for (int c = 0; c < nchunk; ++c) {
        const int col0 = n0 + c * 32;
        if (col0 >= P.N) break;
        int lslot = -1;
        float u[16];
        if (P.has_lora && !P.slab && !P.swiglu) {
          if (c % cpp == 0) {
            bool any = false;
            for (int cc = c; cc < c + cpp && cc < nchunk; ++cc) {
              const int col = n0 + cc * 32;
              any = any || (col < P.N && P.L.slot_of_sec[col / P.L.width] >= 0);
            }
            if (any) {                             // uniform over the CTA
              ep_bar();                            // everyone is done with the previous phase
              const int g4 = G / 4;
              for (int idx = et; idx < P.L.r * g4; idx += EP_THREADS) {
                const int k = idx / g4, c4 = (idx - k * g4) * 4;
                const int col = col0 + c4;
                float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
                if (col < P.N) {
                  const int sec = col / P.L.width;
                  const int slot = P.L.slot_of_sec[sec];
                  if (slot >= 0) {
                    b = lora_replica_b(P.L, slot, (size_t)k * P.L.width + (col - sec * P.L.width), rep);
                    b.x *= P.L.scale; b.y *= P.L.scale; b.z *= P.L.scale; b.w *= P.L.scale;
                  }
                }
                *reinterpret_cast<float4*>(lbuf + k * G + c4) = b;
              }
              ep_bar();
            }
          }
          if (((c >> pshift) & 1) != half) continue;   // the sibling warp's chunk
          lslot = P.L.slot_of_sec[col0 / P.L.width];
          if (lslot >= 0) load_u16(urow + lslot * P.L.r, P.L.r, u_vec, u);
        } else if (((c >> pshift) & 1) != half) {
          continue;
        }
        // summing launch: this CTA owns a quarter of the chunks (a rotary pair stays together)
        if (SPLIT == 2 && (po == 2 ? (c & 1) + 2 * (c >> 2) : (c >> 1)) != grp) continue;
        // rotary embedding fused here: the pair (j, j + dh/2) of a head sits po chunks apart
        const bool rope_here = P.rope_tab != nullptr && col0 < P.rope_cols;
        if (rope_here && po > 0 && (c % (2 * po)) >= po) continue;   // done with its low partner
        uint32_t v[32];
        load_acc(c, v);
        float f[32];
        if (P.swiglu) {
          uint32_t up[32];
          load_acc(4 + c, up);
          tc_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            float g = __uint_as_float(v[j]), u = __uint_as_float(up[j]);
            if (P.bias && col0 + j < P.N) {
              g += to_f(P.bias[col0 + j]);
              u += to_f(P.bias[P.N + col0 + j]);
            }
            // SiLU(g) * u with the approximate reciprocal (two ulp, far below the bf16 rounding of the
            // result): an IEEE division is about ten instructions per element on the warps that share their
            // schedulers with the copy producer and the MMA issuer.  g -> -inf: 1 + e^-g overflows to inf,
            // the quotient is -0, which is the limit
            f[j] = __fdividef(g, 1.f + __expf(-g)) * u;
          }
        } else {
          tc_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) f[j] = __uint_as_float(v[j]);
          if (lslot >= 0) {
            // f += U[row, :] * (s (B + k eps z))[:, chunk]; 16 rank indices at a time, the first 16
            // values of U were requested before the accumulator load
            const float* lb = lbuf + (c % cpp) * 32;
            for (int kb = 0; kb < P.L.r; kb += 16) {
              if (kb) load_u16(urow + lslot * P.L.r + kb, P.L.r - kb, u_vec, u);
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                if (kb + i < P.L.r) {
                  const float4* b4 = reinterpret_cast<const float4*>(lb + (kb + i) * G);
#pragma unroll
                  for (int j4 = 0; j4 < 8; ++j4) {
                    const float4 b = b4[j4];
                    f[4 * j4 + 0] = fmaf(u[i], b.x, f[4 * j4 + 0]);
                    f[4 * j4 + 1] = fmaf(u[i], b.y, f[4 * j4 + 1]);
                    f[4 * j4 + 2] = fmaf(u[i], b.z, f[4 * j4 + 2]);
                    f[4 * j4 + 3] = fmaf(u[i], b.w, f[4 * j4 + 3]);
                  }
                }
              }
            }
          }
          if (P.bias) {
            if (col0 + 32 <= P.N && bias_vec_ok) {
              // the chunk's 32 bias values as four 16-byte loads (every lane reads the same addresses)
#pragma unroll
              for (int j8 = 0; j8 < 4; ++j8) {
                float t[8];
                unpack8(__ldg(reinterpret_cast<const uint4*>(P.bias + col0 + 8 * j8)), t);
#pragma unroll
                for (int j = 0; j < 8; ++j) f[8 * j8 + j] += t[j];
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col0 + j < P.N) f[j] += to_f(P.bias[col0 + j]);
            }
          }
          if (P.act == ACT_RELU) {
#pragma unroll
            for (int j = 0; j < 32; ++j) f[j] = fmaxf(f[j], 0.f);
          }
        }
        float f2[32];
        const bool have2 = rope_here && po > 0;
        if (have2) {
          uint32_t v2[32];
          load_acc(c + po, v2);
          tc_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            f2[j] = __uint_as_float(v2[j]);
            if (P.bias) f2[j] += to_f(P.bias[col0 + po * 32 + j]);
          }
        }
        if (!row_ok) continue;
        if constexpr (CE) {
          float cm = -INFINITY;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (col0 + j < P.N) cm = fmaxf(cm, f[j]);
          if (cm > ce_m) {                           // first chunk: ce_m = -inf, ce_s = 0, expf(-inf) = 0
            ce_s *= expf(ce_m - cm);
            ce_m = cm;
          }
          float add = 0.f;
#pragma unroll
          for (int j = 0; j < 32; ++j)
            if (col0 + j < P.N) add += expf(f[j] - ce_m);
          ce_s += add;
          if (ce_lab >= col0 && ce_lab < col0 + 32) {
            float lv = 0.f;
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (col0 + j == ce_lab) lv = f[j];
            P.ce_logit[row] = lv;
          }
          continue;
        }
        add_res(col0, f);
        if (have2) add_res(col0 + po * 32, f2);
        if (rope_here) {
          const int dh = P.rope_dh, hd = dh >> 1;
          const float* cs = rope_row;                  // cos[0..hd) | sin[0..hd) of this row's position
          if (po > 0) {
            const int h0 = col0 & (dh - 1);            // head-local index of this chunk's first column (< hd); dh is 64 or 128 here
            // every lane reads the table row of its own position: 32-byte loads, for the same reason as the stores
#pragma unroll
            for (int j8 = 0; j8 < 4; ++j8) {
              float cc[8], ss[8];
              asm volatile("ld.global.nc.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                           : "=f"(cc[0]), "=f"(cc[1]), "=f"(cc[2]), "=f"(cc[3]), "=f"(cc[4]), "=f"(cc[5]), "=f"(cc[6]), "=f"(cc[7])
                           : "l"(cs + h0 + 8 * j8));
              asm volatile("ld.global.nc.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                           : "=f"(ss[0]), "=f"(ss[1]), "=f"(ss[2]), "=f"(ss[3]), "=f"(ss[4]), "=f"(ss[5]), "=f"(ss[6]), "=f"(ss[7])
                           : "l"(cs + hd + h0 + 8 * j8));
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const float x1 = f[8 * j8 + j], x2 = f2[8 * j8 + j];
                f[8 * j8 + j] = x1 * cc[j] - x2 * ss[j];
                f2[8 * j8 + j] = x2 * cc[j] + x1 * ss[j];
              }
            }
          } else if (dh == 32) {                       // both halves inside this chunk
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float x1 = f[j], x2 = f[j + 16], cc = cs[j], sn = cs[16 + j];
              f[j] = x1 * cc - x2 * sn;
              f[j + 16] = x2 * cc + x1 * sn;
            }
          } else {                                     // dh = 16: two heads inside this chunk
#pragma unroll
            for (int hh = 0; hh < 2; ++hh)
#pragma unroll
              for (int j = 0; j < 8; ++j) {
                const float x1 = f[16 * hh + j], x2 = f[16 * hh + j + 8], cc = cs[j], sn = cs[8 + j];
                f[16 * hh + j] = x1 * cc - x2 * sn;
                f[16 * hh + j + 8] = x2 * cc + x1 * sn;
              }
          }
        }
        if (P.pack_out) {
          // bf16 copy of U for the tensor-core LoRA k-block: rank index k of slot t goes to
          // K = t*kslot + k and again to K = t*kslot + khalf + k
          bf16* pr = P.pack_out + (size_t)row * P.pack_ld;
          if (P.pack_r == 16 && pack_wide_ok) {
            // a slot's 16 values are one 32-byte run, written at K = t*kslot and again at K = t*kslot + khalf
#pragma unroll
            for (int u = 0; u < 2; ++u) {
              if (col0 + 16 * u + 16 <= P.N) {
                uint32_t o[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) o[j] = pack_bf16(f[16 * u + 2 * j], f[16 * u + 2 * j + 1]);
                bf16* dst = pr + (col0 / 16 + u) * P.kslot;
                asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst), "r"(o[0]), "r"(o[1]), "r"(o[2]),
                             "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7])
                             : "memory");
                asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst + P.khalf), "r"(o[0]), "r"(o[1]),
                             "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7])
                             : "memory");
              }
            }
          } else if (P.pack_r == 8 && pack_wide_ok) {
            // rank 8: 16-byte runs
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              if (col0 + 8 * u + 8 <= P.N) {
                const uint4 o = make_uint4(pack_bf16(f[8 * u], f[8 * u + 1]), pack_bf16(f[8 * u + 2], f[8 * u + 3]),
                                           pack_bf16(f[8 * u + 4], f[8 * u + 5]), pack_bf16(f[8 * u + 6], f[8 * u + 7]));
                bf16* dst = pr + (col0 / 8 + u) * P.kslot;
                *reinterpret_cast<uint4*>(dst) = o;
                *reinterpret_cast<uint4*>(dst + P.khalf) = o;
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int col = col0 + j;
              if (col < P.N) {
                const int t = col / P.pack_r, k = col - t * P.pack_r;
                const bf16 hv = __float2bfloat16_rn(f[j]);
                pr[t * P.kslot + k] = hv;
                pr[t * P.kslot + P.khalf + k] = hv;
              }
            }
          }
        }
        emit(col0, f);
        if (have2) emit(col0 + po * 32, f2);
      }
      if constexpr (CE)
        if (row_ok) P.ce_part[((size_t)row * tiles_n + tn) * 2 + half] = make_float2(ce_m, ce_s);
      // accumulator buffer drained: hand it back to the MMA warp (split K did so when it delivered)
      tc_fence_before();
      __syncwarp();
      if (lane == 0 && !split) {
        if (PAIR) mbar_arrive_leader(smem_u32(&ctrl->tempty[a]));   // the leader waits for both CTAs
        else mbar_arrive(smem_u32(&ctrl->tempty[a]));
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (PAIR) cluster_sync();      // neither CTA leaves while the other may still signal or write into it
  if (warp == 1 && SPLIT != 2) {
    __syncwarp();
    tc_fence_after();
    if (PAIR)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                   "r"(TMEM_COLS)
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base),
                   "r"(TMEM_COLS)
                   : "memory");
  }
}

}  // namespace tc

// ---------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

// Per-device set-up (the opt-in to large dynamic shared memory is a per-device attribute of each
// kernel, and the number of co-resident CTA pairs is a property of the device): done once per
// device ordinal, with that device current, under a mutex so that host threads may race into it.
constexpr int kMaxDevices = 64;
static std::mutex g_setup_mutex;
static std::atomic<bool> g_dev_ready[kMaxDevices];
static int g_max_clusters[kMaxDevices];   // co-resident CTA pairs, 0 = not yet asked

static int current_device(int* dev) {
  const cudaError_t e = cudaGetDevice(dev);
  if (e != cudaSuccess) return (int)e;
  return (*dev < 0 || *dev >= kMaxDevices) ? (int)cudaErrorInvalidDevice : 0;
}

int gemm_tc_init() {
  int dev = 0;
  if (const int e = current_device(&dev)) return e;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    const cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) return e ? (int)e : 999;
    g_encode = (EncodeTiledFn)fn;
  }
  if (g_dev_ready[dev].load(std::memory_order_relaxed)) return 0;
  cudaError_t e = cudaFuncSetAttribute(tc::gemm_tc_kernel<false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)tc::SMEM_BYTES);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::gemm_tc_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tc::SMEM_BYTES);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::gemm_tc_kernel<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tc::SMEM_BYTES);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::gemm_tc_kernel<true, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tc::SMEM_BYTES);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::gemm_tc_kernel<false, 0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tc::SMEM_BYTES);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::gemm_tc_kernel<false, 1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tc::SMEM_BYTES);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::gemm_tc_kernel<false, 0, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tc::SMEM_BYTES);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(tc::gemm_tc_kernel<true, 0, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tc::SMEM_BYTES);
  if (e == cudaSuccess) g_dev_ready[dev].store(true, std::memory_order_release);
  return (int)e;
}

// 2-D bf16 tensor map: rows x K (K contiguous), box 128 rows x 64 columns, 128-byte swizzle;
// out-of-range elements read as zero.
static int make_map(CUtensorMap* m, const void* ptr, uint64_t K, uint64_t rows, uint64_t pitch_elems,
                    uint32_t box_rows = 128u) {
  const cuuint64_t dims[2] = {K, rows};
  const cuuint64_t strides[1] = {pitch_elems * 2};
  const cuuint32_t box[2] = {(cuuint32_t)tc::BK, box_rows};
  const cuuint32_t es[2] = {1u, 1u};
  return (int)g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides,
                       box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

int tc_make_map_bf16(CUtensorMap* m, const void* ptr, uint64_t K, uint64_t rows, uint64_t pitch_elems) {
  if (!g_encode) {
    const int e = gemm_tc_init();
    if (e) return e;
  }
  return make_map(m, ptr, K, rows, pitch_elems);
}

int tc_make_map_bf16_nd(CUtensorMap* m, const void* ptr, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                        const uint32_t* box) {
  if (!g_encode) {
    const int e = gemm_tc_init();
    if (e) return e;
  }
  cuuint64_t d[3], st[2];
  cuuint32_t b[3], es[3] = {1u, 1u, 1u};
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) st[i] = strides_bytes[i];
  return (int)g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(ptr), d, st, b, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// 2-D byte tensor map over quantised codes: rows x row_bytes, box 128 rows x 128 bytes, 128-byte swizzle.
static int make_code_map(CUtensorMap* m, const void* ptr, uint64_t row_bytes, uint64_t rows) {
  const cuuint64_t dims[2] = {row_bytes, rows};
  const cuuint64_t strides[1] = {row_bytes};
  const cuuint32_t box[2] = {128u, 128u};
  const cuuint32_t es[2] = {1u, 1u};
  return (int)g_encode(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, es,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

int launch_gemm_tc(cudaStream_t st, const GemmDesc& G, uint32_t* status, int n_sms) {
  if (G.M <= 0 || G.N <= 0) return 0;
  if (G.K <= 0) return (int)cudaErrorInvalidValue;   // every tile needs at least one base k-block
  int dev = 0;
  if (const int de = current_device(&dev)) return de;
  if (!g_dev_ready[dev].load(std::memory_order_acquire)) {
    const int ie = gemm_tc_init();
    if (ie) return ie;
  }
  CUtensorMap tmA, tmB;
  int e = make_map(&tmA, G.A, (uint64_t)G.K, (uint64_t)G.M, (uint64_t)G.lda);
  if (e) return 10000 + e;
  if (G.wfmt) {
    // codes are decoded inside the kernel; only whole k-blocks, one thread block per tile
    if (!G.wq || !G.wscale || G.K % tc::BK != 0) return (int)cudaErrorInvalidValue;
    e = make_code_map(&tmB, G.wq, (uint64_t)(G.wfmt == 2 ? G.K / 2 : G.K), (uint64_t)G.N);
    if (e) return 10000 + e;
  } else {
    e = make_map(&tmB, G.W, (uint64_t)G.K, (uint64_t)G.N, (uint64_t)G.K);
    if (e) return 10000 + e;
  }
  tc::Params P;
  P.M = G.M;
  P.N = G.swiglu ? G.N / 2 : G.N;
  P.K = G.K;
  P.out = G.out; P.ldo = G.ldo; P.out_f32 = G.out_f32;
  P.bias = (const bf16*)G.bias;
  P.res = (const bf16*)G.res; P.ldr = G.ldr; P.res_mod = G.res_mod;
  P.act = G.act; P.swiglu = G.swiglu;
  P.has_lora = G.lora ? 1 : 0;
  if (G.lora) P.L = *G.lora; else P.L = LoraDesc{};
  P.slab = (G.lora && G.lora_slab) ? 1 : 0;
  P.kslot = G.kslot; P.khalf = G.khalf;
  P.pack_out = (bf16*)G.pack_out; P.pack_ld = G.pack_ld; P.pack_r = G.pack_r;
  CUtensorMap tmU = tmA;
  P.group_m = G.group_m > 0 ? G.group_m : 16;
  if (G.rope_tab && ((uintptr_t)G.rope_tab & 31) != 0) return (int)cudaErrorMisalignedAddress;   // 32-byte table loads
  P.rope_tab = G.rope_tab; P.rope_cols = G.rope_cols; P.rope_dh = G.rope_dh; P.rope_s = G.rope_s; P.rope_tp = G.rope_tp; P.rope_pos = G.rope_pos;
  if (P.slab) {
    e = make_map(&tmU, G.pack_u, (uint64_t)G.pack_ld, (uint64_t)G.M, (uint64_t)G.pack_ld);
    if (e) return 10000 + e;
  }
  P.status = status;
  P.ksplit = 1; P.part = nullptr;
  P.wfmt = G.wfmt; P.wq = (const uint8_t*)G.wq; P.wscale = G.wscale;
  P.ce_part = (float2*)G.ce_part; P.ce_logit = G.ce_logit; P.ce_label = G.ce_label; P.ce_ep = G.ce_ep;
  if (G.ce_part && (G.wfmt || G.swiglu || G.lora || G.rope_tab || !G.ce_logit || !G.ce_label || G.ce_ep < 1))
    return (int)cudaErrorInvalidValue;
  P.wait_ns = G.test_wait_ns ? G.test_wait_ns : tc::WAIT_LIMIT_NS;
  P.withhold = G.test_wait_ns ? 1 : 0;
  const int tiles_n = (P.N + (G.swiglu ? 128 : tc::BN) - 1) / (G.swiglu ? 128 : tc::BN);
  const long long tiles2 = (long long)((P.M + 2 * tc::BM - 1) / (2 * tc::BM)) * tiles_n;   // 256-row tiles
  int max_clusters = 0;                              // co-resident CTA pairs on this device
  if (G.cta_pair) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    max_clusters = g_max_clusters[dev];
  }
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(tc::THREADS); cfg.dynamicSmemBytes = tc::SMEM_BYTES; cfg.stream = st;
  cfg.attrs = attr; cfg.numAttrs = 1;
  if (G.cta_pair && max_clusters == 0) {
    cfg.gridDim = dim3(2 * (n_sms / 2));
    int mc = 0;
    if (cudaOccupancyMaxActiveClusters(&mc, tc::gemm_tc_kernel<true, 0>, &cfg) != cudaSuccess || mc < 1) {
      cudaGetLastError();
      mc = n_sms / 2;
    }
    max_clusters = mc < n_sms / 2 ? mc : n_sms / 2;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    g_max_clusters[dev] = max_clusters;
  }
  // cta_pair 1: pairs wherever the kernel allows; 2: pairs for the launches they were measured faster on:
  // no low-rank term or its one-block tensor-core form (below), at least
  // eight waves of 256-row tiles (the coarser tiles then cost no tail), and at most 3 TFLOP in the launch.
  // The last bound separates the two regimes measured: at the OPT-1.3B shape (launches of 0.5-2.2 TFLOP,
  // board below its power limit) pairs keep the tensor pipe 83 % busy against 70 % and the step gains
  // 5 %; at the Llama-2-7B shape (4-24 TFLOP per launch, board at its 1 kW limit) the pair kernel's higher
  // duty cycle only pulls the clock down, for every kernel of the step, and the step loses 3.5 %.
  // A low-rank term rides along in the pair kernel only as the one-block tensor-core form, whose generated
  // operand serves both 128-row halves of a tile: a replica must then be a whole number of 256-row tiles.
  const bool pair_slab_ok = P.slab && P.kslot == tc::BK && P.L.rows_per_replica % (2 * tc::BM) == 0;
  // (a down-projection that also packs bf16 U always runs single-CTA)
  const bool pair = P.M > tc::BM && !G.pack_out && !P.withhold && !G.wfmt &&
                    (G.cta_pair == 1 || (G.cta_pair == 2 && (!G.lora || pair_slab_ok) && P.N >= tc::BN &&
                                         tiles2 >= 8LL * max_clusters &&
                                         2.0 * (double)G.M * (double)G.N * (double)G.K <= 3.0e12));
  P.n_half = (!pair && !G.swiglu && !P.slab && P.N <= 128) ? 1 : 0;
  P.bbox = 128;
  if (P.n_half && !G.wfmt && P.N <= 64) {
    // a narrow product streams its activations: the smallest weight box leaves the most stages in flight
    P.bbox = P.N <= 32 ? 32 : 64;
    e = make_map(&tmB, G.W, (uint64_t)G.K, (uint64_t)G.N, (uint64_t)G.K, (uint32_t)P.bbox);
    if (e) return 10000 + e;
  }
  if (pair) {
    // pairs of CTAs (clusters of 2) on 256-row tiles
    const int pairs = (int)(tiles2 < max_clusters ? tiles2 : max_clusters);
    cfg.gridDim = dim3(2 * pairs);
    if (!pair_slab_ok) P.slab = 0;
    if (G.ce_part) return (int)cudaLaunchKernelEx(&cfg, tc::gemm_tc_kernel<true, 0, false, true>, tmA, tmB, tmU, P);
    return (int)cudaLaunchKernelEx(&cfg, tc::gemm_tc_kernel<true, 0>, tmA, tmB, tmU, P);
  }
  const int tiles_m = (P.M + tc::BM - 1) / tc::BM;
  const long long tiles = (long long)tiles_m * tiles_n;
  // At most 256 rows, few tiles and a long K (the small-batch regime: the GEMM is a stream of weights):
  // cut K so that the units of work cover the SMs, at least four k-blocks per unit.  Larger launches
  // are never split, so their sums do not depend on the batch shape.
  const int num_kb = (G.K + tc::BK - 1) / tc::BK;
  const int unit_cap = n_sms < G.split_units ? n_sms : G.split_units;
  if (G.split_ws && !G.ce_part && tiles_m <= 2 && tiles * 3 <= unit_cap && num_kb >= 8) {
    int ks = (int)(unit_cap / tiles);
    if (ks > num_kb / 4) ks = num_kb / 4;
    if (G.split_cap > 0 && ks > G.split_cap) ks = G.split_cap;
    if (ks >= 2) { P.ksplit = ks; P.part = (float4*)G.split_ws; }
  }
  const long long units = tiles * P.ksplit;
  const int grid = (int)(units < n_sms ? units : n_sms);
  if (P.ksplit > 1) {
    if (G.wfmt) tc::gemm_tc_kernel<false, 1, true><<<grid, tc::THREADS, tc::SMEM_BYTES, st>>>(tmA, tmB, tmU, P);
    else tc::gemm_tc_kernel<false, 1><<<grid, tc::THREADS, tc::SMEM_BYTES, st>>>(tmA, tmB, tmU, P);
    const long long fin = tiles * tc::FIN_GROUPS;
    tc::gemm_tc_kernel<false, 2><<<(int)(fin < n_sms ? fin : n_sms), tc::THREADS, tc::SMEM_BYTES_SUM, st>>>(tmA, tmB, tmU, P);
    if (G.extra_launches) ++*G.extra_launches;
  } else if (G.wfmt)
    tc::gemm_tc_kernel<false, 0, true><<<grid, tc::THREADS, tc::SMEM_BYTES, st>>>(tmA, tmB, tmU, P);
  else if (G.ce_part)
    tc::gemm_tc_kernel<false, 0, false, true><<<grid, tc::THREADS, tc::SMEM_BYTES, st>>>(tmA, tmB, tmU, P);
  else
    tc::gemm_tc_kernel<false, 0><<<grid, tc::THREADS, tc::SMEM_BYTES, st>>>(tmA, tmB, tmU, P);
  return (int)cudaGetLastError();
}

}  // namespace zo
