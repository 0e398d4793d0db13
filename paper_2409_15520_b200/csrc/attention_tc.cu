// Causal attention on the Blackwell tensor cores for sequences of up to 256 tokens (bf16, head_dim 64
// or 128): softmax(Q K^T / sqrt(dh) + causal) V over the n*E sequences of the replicated batch (q and
// k already carry their rotary embedding).  Attention is ~1 % of the step's flops; the kernel's job is
// to read q, k, v once, write the context once, and keep those streams in flight.
//
//   * persistent CTAs, one per SM; a job is one (sequence, head).  Warp 0 is the copy engine's
//     producer (cp.async.bulk.tensor boxes of 128 rows x 64 columns, 128-byte swizzle, no multicast),
//     warp 1 issues tcgen05.mma, warps 2-9 are two threads per query row (softmax and output), each taking
//     one half of every 64-key chunk of the row's P (one of the two takes the row maximum, the other writes the output); pieces that the causal mask blanks for a whole warp are skipped,
//     and the next piece is requested from tensor memory while the current one is worked on.
//   * a sequence of <= 256 tokens is at most two query tiles and two key tiles, so the scores of a
//     whole query tile fit in tensor memory (128 + 256 columns for the two tiles): the row maximum is
//     exact, nothing is ever rescaled.  S = Q K^T (both operands K-major), the row threads read S twice
//     with tcgen05.ld (maximum, then exponentials), write P in bf16 into a two-slot ring of 64-key
//     chunks in the K-major swizzled layout, and O += P V runs with V as an MN-major operand (V sits in
//     shared memory as the copy engine delivers it: key rows, head_dim contiguous).
//   * the loads of job j+1 overlap the arithmetic of job j: Q and K are free as soon as both score
//     products have retired (early in the job), V when the last P V product has.
//   * every wait is bounded; on expiry the CTA raises ST_TIMEOUT, drains its copies and MMAs, frees its
//     tensor memory and returns.
#include <math.h>

#include <atomic>

#include "kernels.h"
#include "tcgen05.cuh"

namespace zo {
namespace atc {

using namespace tc;

constexpr int SM_WARPS = 8;                        // softmax / output warps: two per tensor-memory lane quarter
constexpr int THREADS = 64 + 32 * SM_WARPS;
constexpr uint32_t BOX = 128 * 128;                 // one 128-row x 64-column bf16 box, 16 KiB
constexpr uint32_t TMEM_COLS = 512;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;

struct Ctrl {
  unsigned long long qk_full, qk_empty, v_full, v_empty, s_full[2], s_empty[2], p_full[2], p_empty[2], o_full, o_empty,
      drain;
  unsigned long long wait_ns;                       // limit of every bounded wait
  uint32_t tmem_base;
  volatile uint32_t abort;
  unsigned long long pair[4];                       // meeting point of the two warps of a lane quarter
  float xmax[2][128];                               // row maxima of the two threads of a row, exchanged both ways
  float xsum[128];                                  // row sum of the odd-chunk thread, handed to the even-chunk one
};
static_assert(sizeof(Ctrl) <= 2048 - 128, "control block must fit beside 224 KiB of tiles");

template <int DH> struct Lay {
  static constexpr int KB = DH / 64;                // 64-column boxes per head
  static constexpr uint32_t Q_OFF = 0;              // [query tile][box][128 rows x 128 B]
  static constexpr uint32_t K_OFF = 2 * KB * BOX;   // [box][256 key rows x 128 B]
  static constexpr uint32_t V_OFF = K_OFF + 2 * KB * BOX;
  static constexpr uint32_t P_OFF = V_OFF + 2 * KB * BOX;   // two chunks of [128 rows x 64 keys]
  static constexpr uint32_t DATA = P_OFF + 2 * BOX;
  static constexpr size_t SMEM = 1024 + DATA + sizeof(Ctrl);
};

struct Params {
  bf16* ctx;
  SeqLayout sl;
  int n, Tp, d, H;
  float scale_log2e;                                // log2(e) / sqrt(dh)
  uint32_t* status;
};

// bf16 x bf16 -> fp32, M = 128; B K-major or MN-major
__host__ __device__ constexpr uint32_t idesc(int n, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn ? (1u << 16) : 0u) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}
// MN-major operand, 128-byte swizzle: 64 elements contiguous along MN, rows (K) 128 B apart, groups of
// eight rows 1024 B apart (stride offset), the next 64 elements along MN `lbo_bytes` further (leading offset)
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr, uint32_t lbo_bytes) {
  uint64_t dsc = 0;
  dsc |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  dsc |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  dsc |= (uint64_t)(1024u >> 4) << 32;
  dsc |= (uint64_t)1 << 46;
  dsc |= (uint64_t)2 << 61;
  return dsc;
}
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int DH>
__global__ void __launch_bounds__(THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tm, const Params P) {
  using L = Lay<DH>;
  constexpr int KB = L::KB;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  Ctrl* ctrl = (Ctrl*)(smem + L::DATA);
  const uint32_t base = smem_u32(smem);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_jobs = P.n * P.sl.E * P.H;

  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&ctrl->qk_full), 1);
    mbar_init(smem_u32(&ctrl->qk_empty), 1);
    mbar_init(smem_u32(&ctrl->v_full), 1);
    mbar_init(smem_u32(&ctrl->v_empty), 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&ctrl->s_full[i]), 1);
      mbar_init(smem_u32(&ctrl->s_empty[i]), SM_WARPS);
      mbar_init(smem_u32(&ctrl->p_full[i]), SM_WARPS);
      mbar_init(smem_u32(&ctrl->p_empty[i]), 1);
    }
    mbar_init(smem_u32(&ctrl->o_full), 1);
    mbar_init(smem_u32(&ctrl->o_empty), SM_WARPS / 2);
    mbar_init(smem_u32(&ctrl->drain), 1);
    for (int i = 0; i < 4; ++i) mbar_init(smem_u32(&ctrl->pair[i]), 2);
    ctrl->abort = 0u;
    ctrl->wait_ns = WAIT_LIMIT_NS;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctrl->tmem_base)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctrl->tmem_base;
  auto wait = [&](unsigned long long* bar, uint32_t parity) {
    return mbar_wait_bounded(smem_u32(bar), parity, &ctrl->abort, &ctrl->wait_ns, P.status);
  };
  // job -> (first row of the sequence in the replicated buffer, its length, head)
  auto job_of = [&](int job, size_t& row_base, int& S_len, int& h) {
    const int sq = job / P.H;
    h = job - sq * P.H;
    const int rep = sq / P.sl.E, b = sq - rep * P.sl.E;
    row_base = (size_t)rep * P.Tp + (size_t)P.sl.start(b);
    S_len = min(P.sl.len(b), 256);
  };

  if (warp == 0) {
    // ---------------------------------------------------------------- copy producer
    if (lane == 0) {
      uint32_t it = 0, qk_issued = 0, v_issued = 0;
      bool ok = true;
      for (int job = blockIdx.x; job < n_jobs && ok; job += gridDim.x) {
        size_t row_base; int S_len, h;
        job_of(job, row_base, S_len, h);
        if (S_len <= 0) continue;
        const int nqt = (S_len + 127) >> 7;
        const int y0 = (int)row_base;
        if (!wait(&ctrl->qk_empty, (it & 1u) ^ 1u)) { ok = false; break; }
        {
          const uint32_t bar = smem_u32(&ctrl->qk_full);
          mbar_expect_tx(bar, (uint32_t)(2 * nqt * KB) * BOX);
          for (int t = 0; t < nqt; ++t)
            for (int kb = 0; kb < KB; ++kb) {
              tma_load_2d(base + L::Q_OFF + (t * KB + kb) * BOX, &tm, h * DH + kb * 64, y0 + t * 128, bar);
              tma_load_2d(base + L::K_OFF + kb * 2 * BOX + t * BOX, &tm, P.d + h * DH + kb * 64, y0 + t * 128, bar);
            }
          ++qk_issued;
        }
        if (!wait(&ctrl->v_empty, (it & 1u) ^ 1u)) { ok = false; break; }
        {
          const uint32_t bar = smem_u32(&ctrl->v_full);
          mbar_expect_tx(bar, (uint32_t)(nqt * KB) * BOX);
          for (int t = 0; t < nqt; ++t)
            for (int kb = 0; kb < KB; ++kb)
              tma_load_2d(base + L::V_OFF + kb * 2 * BOX + t * BOX, &tm, 2 * P.d + h * DH + kb * 64, y0 + t * 128, bar);
          ++v_issued;
        }
        ++it;
      }
      if (!ok) {
        // abort: let the copies already issued land before the CTA goes away (a phase that completed
        // long ago answers at once)
        if (qk_issued) mbar_wait_drain(smem_u32(&ctrl->qk_full), (qk_issued - 1u) & 1u);
        if (v_issued) mbar_wait_drain(smem_u32(&ctrl->v_full), (v_issued - 1u) & 1u);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      uint32_t it = 0, us[2] = {0u, 0u}, pc = 0, oc = 0;
      bool ok = true;
      bool s0_ahead = false;                         // S_0 of the job about to start was already issued (hoisted)
      // S_t = Q_t K^T of the job whose tiles are in shared memory, keys 0 .. 128 (t + 1) - 1 (causal: later
      // keys are never needed); the caller has seen qk_full and s_empty[t]
      auto issue_scores = [&](int t) {
        tc_fence_after();
        const uint32_t dcol = tmem + (t == 0 ? 0u : 128u);
        for (int kb = 0; kb < KB; ++kb) {
          const uint64_t ad = smem_desc(base + L::Q_OFF + (t * KB + kb) * BOX);
          const uint64_t bd = smem_desc(base + L::K_OFF + kb * 2 * BOX);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc_mma(dcol, ad + (uint64_t)(2 * k), bd + (uint64_t)(2 * k), t == 0 ? idesc(128, false) : idesc(256, false),
                   (uint32_t)((kb | k) != 0));
        }
        tc_commit(smem_u32(&ctrl->s_full[t]));
        ++us[t];
      };
      // next job of this CTA with a non-empty sequence (n_jobs if none)
      auto next_job = [&](int job) {
        for (job += gridDim.x; job < n_jobs; job += gridDim.x) {
          size_t rb; int sl_, h_;
          job_of(job, rb, sl_, h_);
          if (sl_ > 0) return job;
        }
        return n_jobs;
      };
      for (int job = blockIdx.x; job < n_jobs && ok; job += gridDim.x) {
        size_t row_base; int S_len, h;
        job_of(job, row_base, S_len, h);
        if (S_len <= 0) continue;
        const int nqt = (S_len + 127) >> 7;
        if (!s0_ahead) {
          if (!wait(&ctrl->qk_full, it & 1u) || !wait(&ctrl->s_empty[0], (us[0] & 1u) ^ 1u)) { ok = false; break; }
          issue_scores(0);
        }
        s0_ahead = false;
        if (nqt > 1) {
          if (!wait(&ctrl->s_empty[1], (us[1] & 1u) ^ 1u)) { ok = false; break; }
          issue_scores(1);
        }
        tc_commit(smem_u32(&ctrl->qk_empty));        // Q and K may be overwritten once both products retire
        if (!wait(&ctrl->v_full, it & 1u)) { ok = false; break; }
        const int nj = next_job(job);
        for (int t = 0; t < nqt && ok; ++t) {
          const int kend = min(S_len, (t + 1) * 128), nch = (kend + 63) >> 6;
          if (!wait(&ctrl->o_empty, (oc & 1u) ^ 1u)) { ok = false; break; }
          tc_fence_after();
          for (int c = 0; c < nch; ++c, ++pc) {
            const uint32_t slot = pc & 1u;
            if (!wait(&ctrl->p_full[slot], (pc >> 1) & 1u)) { ok = false; break; }
            tc_fence_after();
            const uint64_t ad = smem_desc(base + L::P_OFF + slot * BOX);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              // V rows (keys) 64 c + 16 k ..: MN-major operand, the second 64 columns of a 128-wide head 32 KiB on
              const uint64_t bd = smem_desc_mn(base + L::V_OFF + (uint32_t)(c * 64 + k * 16) * 128u, 2 * BOX);
              tc_mma(tmem + 384u, ad + (uint64_t)(2 * k), bd, idesc(DH, true), (uint32_t)((c | k) != 0));
            }
            tc_commit(smem_u32(&ctrl->p_empty[slot]));
          }
          if (!ok) break;
          tc_commit(smem_u32(&ctrl->o_full));
          ++oc;
          // the next job's first score product, as soon as its tiles have landed and this job's S_0 has been
          // read (never waited for here: the remaining P V work of this job must not queue behind a load)
          if (t == 0 && !s0_ahead && nj < n_jobs && mbar_test(smem_u32(&ctrl->qk_full), (it + 1u) & 1u) &&
              mbar_test(smem_u32(&ctrl->s_empty[0]), (us[0] & 1u) ^ 1u)) {
            issue_scores(0);
            s0_ahead = true;
          }
        }
        if (!ok) break;
        tc_commit(smem_u32(&ctrl->v_empty));
        ++it;
      }
      if (!ok) {
        tc_commit(smem_u32(&ctrl->drain));           // wait for the MMAs already issued
        mbar_wait_drain(smem_u32(&ctrl->drain), 0u);
      }
    }
  } else {
    // ---------------------------------------------------------------- two threads per query row
    const int wq = warp & 3;                         // tensor-memory lane quarter of this warp
    const int half = (warp - 2) >> 2;                // which of the row's two threads: even or odd 32-column chunks
    const int r = wq * 32 + lane;                    // row of the query tile
    const uint32_t lane_base = tmem + ((uint32_t)(wq * 32) << 16);
    uint32_t us[2] = {0u, 0u}, pc = 0, oc = 0;
    bool ok = true;
    // one lane waits, the warp learns the outcome
    auto warp_wait = [&](unsigned long long* bar, uint32_t parity) -> bool {
      uint32_t good = 1u;
      if (lane == 0)
        good = mbar_wait_bounded<1>(smem_u32(bar), parity, &ctrl->abort, &ctrl->wait_ns, P.status) ? 1u : 0u;
      return __shfl_sync(0xffffffffu, good, 0) != 0u;
    };
    // the two warps of a lane quarter meet (bounded like every other wait: false once the CTA is aborting)
    uint32_t n_meet = 0;
    auto pair_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctrl->pair[wq]));
      return warp_wait(&ctrl->pair[wq], n_meet++ & 1u);
    };
    for (int job = blockIdx.x; job < n_jobs && ok; job += gridDim.x) {
      size_t row_base; int S_len, h;
      job_of(job, row_base, S_len, h);
      if (S_len <= 0) continue;
      const int nqt = (S_len + 127) >> 7;
      for (int t = 0; t < nqt && ok; ++t) {
        const int qpos = t * 128 + r;
        const int kend = min(S_len, (t + 1) * 128), nch = (kend + 63) >> 6;
        const uint32_t scol = lane_base + (t == 0 ? 0u : 128u);
        if (!warp_wait(&ctrl->s_full[t], us[t] & 1u)) { ok = false; break; }
        ++us[t];
        tc_fence_after();
        // key k counts for this row when k <= qpos (causal) and k < S_len (rows past the end of the
        // sequence in the loaded tiles belong to other sequences)
        const int klim = min(qpos, S_len - 1);
        const int klim_lo = min(t * 128 + wq * 32, S_len - 1);        // smallest and largest limit in this warp
        const int klim_hi = min(t * 128 + wq * 32 + 31, S_len - 1);
        // this thread owns the 32-column pieces j of the row with j % 2 == half: one half of every 64-key
        // chunk.  A piece is needed unless the causal mask blanks it for the whole warp (then so are all
        // later ones).  The loops are kept rolled: ten warps in four roles share one instruction cache.
        // (four independent running maxima / sums: a single chain of 32 dependent operations would leave the
        // two warps of a scheduler waiting on arithmetic latency)
        // The row maximum is taken by the odd-half thread of the row alone, over all pieces: the even-half warps
        // are still writing the previous tile's output when the scores of this tile arrive, and the odd-half
        // warps would only wait for them.
        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        for (int j = 0; half && j < 2 * nch; j += 2) {    // two pieces per round trip to tensor memory
          if (j * 32 > klim_hi) break;
          const bool two = (j + 1) * 32 <= klim_hi;
          uint32_t v[32], w[32];
          tc_ld32(scol + j * 32, v);
          if (two) tc_ld32(scol + (j + 1) * 32, w);
          tc_ld_wait();
          const int lim = klim - j * 32;             // elements 0 .. lim of the piece count (>= 31: all of them)
          // a piece that lies below the diagonal for every row of the warp needs no mask (most pieces do)
          if (klim_lo - j * 32 >= 31) {
#pragma unroll
            for (int i = 0; i < 32; ++i) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(v[i]));
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) m4[i & 3] = fmaxf(m4[i & 3], i <= lim ? __uint_as_float(v[i]) : -INFINITY);
          }
          if (two) {
            if (klim_lo - j * 32 >= 63) {
#pragma unroll
              for (int i = 0; i < 32; ++i) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(w[i]));
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                m4[i & 3] = fmaxf(m4[i & 3], i + 32 <= lim ? __uint_as_float(w[i]) : -INFINITY);
            }
          }
        }
        float m = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
        if (half) ctrl->xmax[1][r] = m;
        if (!pair_sync()) { ok = false; break; }
        if (!half) m = ctrl->xmax[1][r];             // (key 0 counts for every row: the maximum is finite)
        const float ms = m * P.scale_log2e;
        float l4[4] = {0.f, 0.f, 0.f, 0.f};
        for (int c = 0; c < nch && ok; ++c, ++pc) {
          const uint32_t slot = pc & 1u;
          uint8_t* prow = smem + L::P_OFF + slot * BOX + r * 128;
          const int j = 2 * c + half;                // this thread's half of the 64-key chunk
          uint32_t pk[16];                           // P of the piece, bf16 pairs
          if (j * 32 > klim_hi) {
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = 0u;
          } else {
            uint32_t v[32];
            tc_ld32(scol + j * 32, v);
            tc_ld_wait();
            const int lim = klim - j * 32;
            if (klim_lo - j * 32 >= 31) {             // unmasked piece
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const float p0 = ex2f(fmaf(__uint_as_float(v[i]), P.scale_log2e, -ms));
                const float p1 = ex2f(fmaf(__uint_as_float(v[i + 1]), P.scale_log2e, -ms));
                l4[(i >> 1) & 3] += p0 + p1;
                pk[i >> 1] = pack_bf16(p0, p1);
              }
            } else {
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                const float p0 = i <= lim ? ex2f(fmaf(__uint_as_float(v[i]), P.scale_log2e, -ms)) : 0.f;
                const float p1 = i + 1 <= lim ? ex2f(fmaf(__uint_as_float(v[i + 1]), P.scale_log2e, -ms)) : 0.f;
                l4[(i >> 1) & 3] += p0 + p1;
                pk[i >> 1] = pack_bf16(p0, p1);
              }
            }
          }
          // the slot is needed only now: the piece's arithmetic ran under the P V product that still read it
          if (!warp_wait(&ctrl->p_empty[slot], ((pc >> 1) & 1u) ^ 1u)) { ok = false; break; }
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4)             // 16-byte chunk half*4 + q4 of the row's 128 bytes: 8 keys per chunk
            *reinterpret_cast<uint4*>(prow + (((half * 4 + q4) ^ (r & 7)) << 4)) =
                make_uint4(pk[4 * q4], pk[4 * q4 + 1], pk[4 * q4 + 2], pk[4 * q4 + 3]);
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // visible to the tensor core
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&ctrl->p_full[slot]));
        }
        if (!ok) break;
        // scores consumed: the next job's product for this tile may overwrite them
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->s_empty[t]));
        // the even-chunk thread of a row writes the row's output; its partner hands over its share of the sum
        // (this meeting also orders the tile's reads of xmax before the next tile's writes)
        float l = (l4[0] + l4[1]) + (l4[2] + l4[3]);
        if (half) ctrl->xsum[r] = l;
        if (!pair_sync()) { ok = false; break; }
        if (half) continue;
        l += ctrl->xsum[r];
        if (!warp_wait(&ctrl->o_full, oc & 1u)) { ok = false; break; }
        ++oc;
        tc_fence_after();
        const float inv = 1.f / l;
        bf16* orow = P.ctx + (row_base + (size_t)qpos) * P.d + h * DH;
#pragma unroll
        for (int j = 0; j < DH / 64; ++j) {
          uint32_t v0[32], v1[32];
          tc_ld32(lane_base + 384u + j * 64, v0);
          tc_ld32(lane_base + 384u + j * 64 + 32, v1);
          tc_ld_wait();
          if (qpos < S_len) {
            // a lane writes its own row, so a store instruction touches 32 rows whatever its width: 32-byte
            // stores (whole sectors) halve the number of such instructions
#pragma unroll
            for (int q8 = 0; q8 < 4; ++q8) {
              const uint32_t* v = q8 < 2 ? v0 + 16 * q8 : v1 + 16 * (q8 - 2);
              uint32_t o[8];
#pragma unroll
              for (int i = 0; i < 8; ++i)
                o[i] = pack_bf16(__uint_as_float(v[2 * i]) * inv, __uint_as_float(v[2 * i + 1]) * inv);
              asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(orow + j * 64 + q8 * 16),
                           "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]), "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7])
                           : "memory");
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctrl->o_empty));
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace atc

// ---------------------------------------------------------------------------------- host side
bool attention_tc_supported(int dh, int max_len) { return (dh == 64 || dh == 128) && max_len <= 256; }

template <int DH>
static int launch_t(cudaStream_t st, const CUtensorMap& tm, const atc::Params& P, int n_sms, int n_jobs) {
  static std::atomic<unsigned long long> ready{0};   // bit per device ordinal: shared-memory opt-in done
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return (int)e;
  if (dev < 0 || dev >= 64) return (int)cudaErrorInvalidDevice;
  if (!(ready.load(std::memory_order_acquire) >> dev & 1ull)) {
    e = cudaFuncSetAttribute(atc::attention_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)atc::Lay<DH>::SMEM);
    if (e != cudaSuccess) return (int)e;
    ready.fetch_or(1ull << dev, std::memory_order_release);
  }
  const int grid = n_jobs < n_sms ? n_jobs : n_sms;
  atc::attention_tc_kernel<DH><<<grid, atc::THREADS, atc::Lay<DH>::SMEM, st>>>(tm, P);
  return (int)cudaGetLastError();
}

int launch_attention_tc(cudaStream_t st, const void* qkv, void* ctx, int n, SeqLayout sl, int Tp, int d, int H,
                        uint32_t* status, int n_sms) {
  const int dh = d / H;
  const int n_jobs = n * sl.E * H;
  if (n_jobs <= 0) return 0;
  if ((reinterpret_cast<uintptr_t>(ctx) & 31) != 0 || d % 16 != 0) return (int)cudaErrorMisalignedAddress;   // 32-byte output stores
  CUtensorMap tm;
  // rows of the replicated q|k|v buffer x 3d columns; boxes of 128 rows x 64 columns, 128-byte swizzle
  const int me = tc_make_map_bf16(&tm, qkv, (uint64_t)3 * d, (uint64_t)n * Tp, (uint64_t)3 * d);
  if (me) return 10000 + me;
  atc::Params P;
  P.ctx = (bf16*)ctx; P.sl = sl; P.n = n; P.Tp = Tp; P.d = d; P.H = H;
  P.scale_log2e = 1.4426950408889634f / sqrtf((float)dh);
  P.status = status;
  return dh == 64 ? launch_t<64>(st, tm, P, n_sms, n_jobs) : launch_t<128>(st, tm, P, n_sms, n_jobs);
}

}  // namespace zo
