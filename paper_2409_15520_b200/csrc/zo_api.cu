// C ABI of the library: argument checks, workspace partition and the per-step launch plan.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <vector>

#include "../../include/zo.h"
#include "common.cuh"
#include "kernels.h"

using namespace zo;

namespace {

// text of the last zo_init failure of the calling thread (zo_last_error(NULL))
thread_local char g_init_error[256] = "";

constexpr int ZO_MAX_Q = 32;            // largest q a context accepts; sizes the per-step pass lists
constexpr int MAX_PASSES = 2 * ZO_MAX_Q;  // the sequential schedule cuts a step into 2q passes

struct Plan {  // byte offsets into the workspace
  size_t h0, x0, qkv0, h, x, qkv, a, gu, U, rope, lab_idx, lab_val, lab_cnt, tok_stage, lab_stage,
      xh, logits, ce_part, ce_logit, rowloss, rowloss_pass, losses, losses_d, g, status, ub, wdq, pos, split_ws, total;
};

inline size_t up(size_t v, size_t a) { return (v + a - 1) / a * a; }
constexpr int SPLIT_UNITS = 160;   // units of split-K work the scratch can hold (>= SMs of the device in use)

inline int n_targets(const zo_config& c) {
  return ((c.lora_targets >> 0) & 1) + ((c.lora_targets >> 1) & 1) + ((c.lora_targets >> 2) & 1);
}
// Full-vocabulary loss without the logits round trip: the head GEMM's epilogue reduces its tile to
// (max, sum of exp) pairs.  Tensor-core path only; ZO_FLAG_CE_LOGITS keeps the stored-logits form.
inline bool fused_ce(const zo_config& c) {
  return c.loss_kind == ZO_LOSS_CE_FULL_VOCAB && c.precision == ZO_BF16 &&
         !(c.flags & (ZO_FLAG_SIMT_GEMM | ZO_FLAG_CE_LOGITS));
}
inline size_t ce_parts_per_row(const zo_config& c) { return 2 * (((size_t)c.vocab + 255) / 256); }
inline int row_pad(const zo_config& c) { return c.precision == ZO_BF16 ? 128 : 1; }
// Queries a context runs in one step: all of them, or at most max_shard_q when it only ever runs shards.
inline int run_q(const zo_config& c) { return c.max_shard_q > 0 ? c.max_shard_q : c.max_q; }

// Returns ZO_OK or the reason the configuration cannot be run.
zo_status check_config(const zo_config* c, char* err, size_t errn) {
#define BAD(code, ...)                 \
  do {                                 \
    snprintf(err, errn, __VA_ARGS__);  \
    return code;                       \
  } while (0)
  if (!c) BAD(ZO_ERR_INVALID_ARG, "config is NULL");
  if (c->struct_size != sizeof(zo_config))
    BAD(ZO_ERR_INVALID_ARG, "struct_size %u != %zu", c->struct_size, sizeof(zo_config));
  if (c->arch < ZO_ARCH_LINEAR || c->arch > ZO_ARCH_LLAMA) BAD(ZO_ERR_INVALID_ARG, "bad arch");
  if (c->precision != ZO_FP32 && c->precision != ZO_BF16) BAD(ZO_ERR_INVALID_ARG, "bad precision");
  if (c->loss_kind < ZO_LOSS_MSE || c->loss_kind > ZO_LOSS_CE_LABEL_WORDS)
    BAD(ZO_ERR_INVALID_ARG, "bad loss_kind");
  if (c->lora_rank < 1 || c->lora_rank > 64) BAD(ZO_ERR_INVALID_ARG, "lora_rank must be 1..64");
  if (c->max_q < 1 || c->max_q > ZO_MAX_Q) BAD(ZO_ERR_INVALID_ARG, "max_q must be 1..32");
  if (c->max_shard_q < 0 || c->max_shard_q > c->max_q) BAD(ZO_ERR_INVALID_ARG, "max_shard_q must be 0..max_q");
  if (c->max_E < 1 || c->max_seq < 1) BAD(ZO_ERR_INVALID_ARG, "max_E and max_seq must be >= 1");
  if (c->d_model < 1) BAD(ZO_ERR_INVALID_ARG, "d_model must be >= 1");
  if (!isfinite(c->lora_scale)) BAD(ZO_ERR_INVALID_ARG, "lora_scale not finite");
  const bool bf = c->precision == ZO_BF16;
  if (c->weight_format < ZO_W_NATIVE || c->weight_format > ZO_W_NF4) BAD(ZO_ERR_INVALID_ARG, "bad weight_format");
  if (c->arch == ZO_ARCH_LINEAR) {
    if (c->weight_format != ZO_W_NATIVE) BAD(ZO_ERR_UNSUPPORTED, "quantised weights are for decoders");
    if (c->loss_kind != ZO_LOSS_MSE) BAD(ZO_ERR_INVALID_ARG, "ZO_ARCH_LINEAR requires ZO_LOSS_MSE");
    if (c->d_out < 1) BAD(ZO_ERR_INVALID_ARG, "d_out must be >= 1");
    if (c->d_out % 4) BAD(ZO_ERR_UNSUPPORTED, "d_out must be a multiple of 4");
    if (bf && (c->d_model % 8 || c->d_out % 8))
      BAD(ZO_ERR_UNSUPPORTED, "bf16 needs d_model and d_out to be multiples of 8");
    return ZO_OK;
  }
  if (c->loss_kind == ZO_LOSS_MSE) BAD(ZO_ERR_INVALID_ARG, "decoders need a cross-entropy loss");
  if (c->n_layers < 1 || c->n_heads < 1 || c->d_ffn < 1 || c->vocab < 2 || c->max_labelled < 1)
    BAD(ZO_ERR_INVALID_ARG, "n_layers, n_heads, d_ffn, vocab, max_labelled must be positive");
  if (c->lora_targets & ~7u) BAD(ZO_ERR_INVALID_ARG, "unknown lora_targets bits");
  if (c->d_model % c->n_heads) BAD(ZO_ERR_UNSUPPORTED, "d_model %% n_heads != 0");
  const int dh = c->d_model / c->n_heads;
  if (dh != 16 && dh != 32 && dh != 64 && dh != 128)
    BAD(ZO_ERR_UNSUPPORTED, "head_dim %d not in {16,32,64,128}", dh);
  if (c->max_seq > 512) BAD(ZO_ERR_UNSUPPORTED, "max_seq > 512");
  if (c->d_model % 4) BAD(ZO_ERR_UNSUPPORTED, "d_model must be a multiple of 4");
  if (bf && (c->d_model % 8 || c->d_ffn % 8))
    BAD(ZO_ERR_UNSUPPORTED, "bf16 needs d_model and d_ffn to be multiples of 8");
  if (c->loss_kind == ZO_LOSS_CE_LABEL_WORDS)
    for (int i = 0; i < 2; ++i)
      if (c->label_words[i] < 0 || c->label_words[i] >= c->vocab)
        BAD(ZO_ERR_INVALID_ARG, "label word out of the vocabulary");
  if (c->weight_format != ZO_W_NATIVE && (c->d_model % 64 || c->d_ffn % 64))
    BAD(ZO_ERR_UNSUPPORTED, "quantised weights need d_model and d_ffn to be multiples of 64");
  if (!(c->norm_eps > 0.f)) BAD(ZO_ERR_INVALID_ARG, "norm_eps must be > 0");
  if (c->arch == ZO_ARCH_LLAMA && !(c->rope_theta > 1.f)) BAD(ZO_ERR_INVALID_ARG, "rope_theta must be > 1");
  return ZO_OK;
#undef BAD
}

Plan make_plan(const zo_config& c) {
  Plan p;
  memset(&p, 0, sizeof(p));
  const size_t es = c.precision == ZO_BF16 ? 2 : 4;
  const size_t n = 2 * (size_t)c.max_q;                 // replicas of a whole step (loss arrays)
  const size_t na = 2 * (size_t)run_q(c);               // replicas this context ever runs in one step
  const size_t Tm = (size_t)c.max_E * c.max_seq;
  const size_t Tp = up(Tm, row_pad(c));
  const size_t Mp = na * Tp;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off += up(bytes, 256);
    return o;
  };
  const bool unfused_mlp = c.precision == ZO_FP32 || (c.flags & ZO_FLAG_SIMT_GEMM);
  if (c.arch == ZO_ARCH_LINEAR) {
    p.U = take(Tp * c.lora_rank * 4);
    p.qkv0 = take(Tp * c.d_out * es);                 // base product X W^T
    p.qkv = take(Mp * c.d_out * es);                  // Y[n]
    p.tok_stage = take(Tm * c.d_model * es);          // host-variant staging of X
    p.lab_stage = take(Tm * c.d_out * 4);             // and of the targets
    p.rowloss = take(n * Tm * 8);
    p.rowloss_pass = take(na * Tm * 8);
  } else {
    const size_t d = c.d_model, f = c.d_ffn, J = (size_t)n_targets(c) * c.lora_rank;
    const size_t P = c.max_labelled, Mh = na * c.max_E * P;
    p.h0 = take(Tp * d * es);
    p.x0 = take(Tp * d * es);
    p.qkv0 = take(Tp * 3 * d * es);
    p.h = take(Mp * d * es);
    p.x = take(Mp * d * es);
    p.qkv = take(Mp * 3 * d * es);
    p.a = take(Mp * f * es);
    if (c.arch == ZO_ARCH_LLAMA && unfused_mlp) p.gu = take(Mp * 2 * f * es);
    p.U = take(Mp * (J ? J : 1) * 4);
    if (c.precision == ZO_BF16) p.ub = take(Mp * (size_t)(n_targets(c) ? n_targets(c) : 1) * (c.lora_rank > 32 ? 128 : 64) * 2);  // packed bf16 U
    if (c.arch == ZO_ARCH_LLAMA) p.rope = take((size_t)c.max_seq * (d / c.n_heads) * 4);
    p.lab_idx = take(c.max_E * P * 4);
    p.lab_val = take(c.max_E * P * 4);
    p.lab_cnt = take(c.max_E * 4);
    p.tok_stage = take(Tm * 4);
    p.lab_stage = take(Tm * 4);
    p.pos = take(Tp * 4);
    p.xh = take(Mh * d * es);
    if (fused_ce(c)) {
      p.ce_part = take(Mh * ce_parts_per_row(c) * 8);
      p.ce_logit = take(Mh * 4);
    } else if (c.loss_kind == ZO_LOSS_CE_FULL_VOCAB) {
      p.logits = take(Mh * (size_t)c.vocab * 4);
    }
    p.rowloss = take(n * c.max_E * P * 8);
    p.rowloss_pass = take(Mh * 8);
    if (c.weight_format != ZO_W_NATIVE) {   // one dequantised weight at a time
      size_t big = 3 * d * d;
      const size_t f1 = (c.arch == ZO_ARCH_LLAMA ? 2 : 1) * f * d;
      if (f1 > big) big = f1;
      p.wdq = take(big * es);
    }
  }
  p.losses = take(n * 4);
  p.losses_d = take((n + 1) * 8);   // 2 max_q losses + the fault slot of a sharded step
  p.g = take((size_t)c.max_q * 4);
  p.status = take(256);
  if (c.precision == ZO_BF16) {             // split-K scratch of the tensor-core GEMM (small batches)
    p.split_ws = take((size_t)SPLIT_UNITS * 128 * 256 * 4);
  }
  p.total = off;
  return p;
}

}  // namespace

enum { PC_GEMM_TC = 0, PC_GEMM_SIMT, PC_ATTN, PC_NORM, PC_LORA_DOWN, PC_LORA_APPLY, PC_ROPE,
       PC_SWIGLU, PC_LOSS, PC_UPDATE, PC_MISC, PC_GEMM_QKV, PC_GEMM_O, PC_GEMM_FC1, PC_GEMM_FC2,
       PC_GEMM_HEAD, PC_DEQUANT, PC_COUNT };
static_assert(PC_COUNT == ZO_PROFILE_CLASSES, "profile classes out of sync with zo.h");

struct ProfRec { int cat; double flops; cudaEvent_t e0, e1; };

struct zo_ctx {
  int prof_on;
  std::vector<ProfRec>* prof;      // records of the launches since the last read
  std::vector<cudaEvent_t>* evpool; // events free for reuse
  zo_config cfg;
  Plan plan;
  uint8_t* ws;
  cudaStream_t st;
  int bf, n_sms, nt;
  int slot_of_sec[3];
  int launches;
  int stepped, last_q, last_E, last_S;
  int schedule;
  int shard_begin, shard_count;    // queries this context computes in a step (count 0 = all of them)
  unsigned long long test_wait_ns; // failure-detection test aid (zo_test_expire_wait), 0 = off
  int pair_mode;                   // the running step uses the stored +/- pair of Algorithm 2 (lora->B[l] = the pair)
  char err[256];
  template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
};

namespace {

// Brackets one launch with CUDA events on the context's stream when profiling is on.
struct ProfScope {
  zo_ctx* c;
  ProfRec r;
  bool live;
  ProfScope(zo_ctx* ctx, int cat, double flops) : c(ctx), live(false) {
    if (!c || !c->prof_on) return;
    r.cat = cat; r.flops = flops; r.e0 = r.e1 = nullptr;
    for (cudaEvent_t* e : {&r.e0, &r.e1}) {
      if (!c->evpool->empty()) { *e = c->evpool->back(); c->evpool->pop_back(); }
      else if (cudaEventCreate(e) != cudaSuccess) { *e = nullptr; }
    }
    if (!r.e0 || !r.e1) return;
    live = cudaEventRecord(r.e0, c->st) == cudaSuccess;
  }
  ~ProfScope() {
    if (!live) return;
    if (cudaEventRecord(r.e1, c->st) == cudaSuccess) c->prof->push_back(r);
  }
};
#define PROF(cat, flops, call)      \
  do {                              \
    ProfScope ps_(c, cat, flops);   \
    call;                           \
    ++c->launches;                  \
  } while (0)

zo_status fail(zo_ctx* c, zo_status s, const char* fmt, const char* a = "") {
  snprintf(c->err, sizeof(c->err), fmt, a);
  return s;
}

// GEMM dispatch: tensor-core kernel for bf16 unless the validation flag asks otherwise.
zo_status run_gemm(zo_ctx* c, cudaStream_t st, int bf, uint32_t flags, const GemmDesc& G,
                   uint32_t* status, int n_sms, int* launches, char* err, size_t errn) {
  const bool tcore = bf && !(flags & ZO_FLAG_SIMT_GEMM);
  ProfScope ps(c, tcore ? (G.prof_class ? G.prof_class : PC_GEMM_TC) : PC_GEMM_SIMT,
               2.0 * G.M * (double)G.N * G.K);
  if (tcore) {
    GemmDesc Gt = G;
    Gt.cta_pair = (flags & ZO_FLAG_GEMM_PAIR) ? 1 : ((flags & ZO_FLAG_GEMM_SINGLE) ? 0 : 2);
    Gt.group_m = (int)((flags >> 8) & 0xFF);     // diagnostic: raster group override in bits 8..15
    Gt.split_cap = (int)((flags >> 16) & 0x1F);  // diagnostic: bound on the split-K factor in bits 16..20
    Gt.test_wait_ns = c ? c->test_wait_ns : ((flags & ZO_FLAG_TEST_EXPIRE_WAIT) ? 1000000ull : 0ull);
    if (c && c->plan.split_ws) {
      Gt.split_ws = c->at<float>(c->plan.split_ws); Gt.split_units = SPLIT_UNITS; Gt.extra_launches = launches;
    }
    const int e = launch_gemm_tc(st, Gt, status, n_sms);
    if (e) {
      snprintf(err, errn, "tensor-core GEMM launch failed (code %d: %s)", e,
               e < 10000 ? cudaGetErrorString((cudaError_t)e) : "tensor-map encode");
      return ZO_ERR_CUDA;
    }
  } else {
    launch_gemm_simt(st, bf, G);
  }
  ++*launches;
  return ZO_OK;
}

// Down-projection U = X A^T (fp32 out): on the tensor cores for bf16 operands (it only has to
// read X once; the MMA work is small), on CUDA cores otherwise.
zo_status run_lora_down(zo_ctx* c, cudaStream_t st, int bf, uint32_t flags, const void* X, int ldx,
                        const void* A, float* U, int rows, int K, int J, uint32_t* status, int n_sms,
                        int* launches, char* err, size_t errn, void* pack_out = nullptr, int pack_ld = 0,
                        int pack_r = 0, int kslot = 64) {
  if (bf && !(flags & ZO_FLAG_SIMT_GEMM) && K % 8 == 0 && ldx % 8 == 0) {
    GemmDesc G{};
    G.A = X; G.lda = ldx; G.W = A; G.M = rows; G.N = J; G.K = K; G.out = U; G.ldo = J; G.out_f32 = 1;
    G.cta_pair = (flags & ZO_FLAG_GEMM_PAIR) ? 1 : 0;
    G.pack_out = pack_out; G.pack_ld = pack_ld; G.pack_r = pack_r; G.kslot = kslot; G.khalf = kslot / 2;
    if (c && c->plan.split_ws) {
      G.split_ws = c->at<float>(c->plan.split_ws); G.split_units = SPLIT_UNITS; G.extra_launches = launches;
    }
    G.split_cap = (int)((flags >> 16) & 0x1F);
    ProfScope ps(c, PC_LORA_DOWN, 2.0 * rows * (double)J * K);
    const int e = launch_gemm_tc(st, G, status, n_sms);
    if (e) {
      snprintf(err, errn, "tensor-core down-projection launch failed (code %d)", e);
      return ZO_ERR_CUDA;
    }
  } else {
    ProfScope ps(c, PC_LORA_DOWN, 2.0 * rows * (double)J * K);
    launch_lora_down(st, bf, X, ldx, A, U, rows, K, J);
  }
  ++*launches;
  return ZO_OK;
}

// The forward passes a step is cut into.  Pass p covers the replicas base + stride * j, j < count.
struct Pass { int base, stride, count; };
inline int make_passes(int schedule, int q, Pass* out) {   // out holds up to 2q entries
  int np = 0;
  switch (schedule) {
    case ZO_SCHEDULE_OUTER_ONLY:   // all +eps replicas, then all -eps replicas
      out[np++] = Pass{0, 2, q};
      out[np++] = Pass{1, 2, q};
      break;
    case ZO_SCHEDULE_INNER_ONLY:   // the +/- pair of one query at a time
      for (int i = 0; i < q; ++i) out[np++] = Pass{2 * i, 1, 2};
      break;
    case ZO_SCHEDULE_SEQUENTIAL:   // one perturbed forward at a time
      for (int n = 0; n < 2 * q; ++n) out[np++] = Pass{n, 1, 1};
      break;
    default:                       // everything in one pass
      out[np++] = Pass{0, 1, 2 * q};
  }
  return np;
}

// Passes of a step on this context: with a query shard set, only the replicas of the queries
// [shard_begin, shard_begin + shard_count) are run, at their positions in the whole step.
inline int step_passes(const zo_ctx* c, int q, Pass* out) {
  if (c->shard_count == 0) return make_passes(c->schedule, q, out);
  const int np = make_passes(c->schedule, c->shard_count, out);
  for (int i = 0; i < np; ++i) out[i].base += 2 * c->shard_begin;
  return np;
}

// Can the MP-LoRA term ride in the tensor-core GEMM's epilogue?
inline bool fused_lora_ok(int bf, uint32_t flags, int Tp, int width) {
  return bf && !(flags & ZO_FLAG_SIMT_GEMM) && Tp % 128 == 0 && width % 32 == 0;
}
// ... and as extra k-blocks on the tensor cores?  (rank <= 64; every 256-column tile inside one
// section.  The CTA-pair kernel shares the generated operand between the two 128-row halves of its
// 256-row tile, so there a replica must be a whole number of such tiles, and only the one-block
// form, rank <= 32, is built.)
inline bool slab_lora_ok(int bf, uint32_t flags, int Tp, int width, int r) {
  if (!fused_lora_ok(bf, flags, Tp, width) || (flags & ZO_FLAG_LORA_EPILOGUE) || width % 256 != 0 || r > 64)
    return false;
  return !(flags & ZO_FLAG_GEMM_PAIR) || (Tp % 256 == 0 && r <= 32);
}

// Projected gradients g_i from the step's 2q fp64 losses and the ZO-SGD update of every B tensor
// (Algorithm 1, last line of the step).
void enqueue_update(zo_ctx* c, const zo_lora* lora, uint64_t seed, int q, float eps, float lr) {
  const zo_config& cf = c->cfg;
  cudaStream_t st = c->st;
  const uint32_t* status = c->at<uint32_t>(c->plan.status);
  const double* losses_d = c->at<double>(c->plan.losses_d);
  float* g = c->at<float>(c->plan.g);
  const int r = cf.lora_rank;
  if (cf.arch == ZO_ARCH_LINEAR) {
    UpdateDesc D{};
    D.B[0] = lora->B[0]; D.tensor_base[0] = 0; D.count = 1; D.n_slots = 1;
    D.elems_per_slot = (long long)r * cf.d_out;
    PROF(PC_UPDATE, 0.0, launch_zo_update(st, D, losses_d, g, q, eps, lr, seed, status, 1));
    return;
  }
  const int nt = c->nt, J = nt * r;
  if (J == 0) {
    UpdateDesc D{};
    D.count = 0; D.n_slots = 0; D.elems_per_slot = 0;
    PROF(PC_UPDATE, 0.0, launch_zo_update(st, D, losses_d, g, q, eps, 0.f, seed, status, 1));
  }
  for (int l0 = 0; l0 < cf.n_layers && J; l0 += UpdateDesc::MAX_T) {
    UpdateDesc D{};
    D.count = cf.n_layers - l0 < UpdateDesc::MAX_T ? cf.n_layers - l0 : UpdateDesc::MAX_T;
    D.n_slots = nt;
    D.elems_per_slot = (long long)r * cf.d_model;
    for (int i = 0; i < D.count; ++i) {
      D.B[i] = lora->B[l0 + i];
      D.tensor_base[i] = (uint32_t)((l0 + i) * nt);
    }
    PROF(PC_UPDATE, 0.0, launch_zo_update(st, D, losses_d, g, q, eps, lr, seed, status, l0 == 0));
  }
}

// End of a step: projected gradients and ZO-SGD update of every B tensor; a sharded step stops at its
// losses and publishes whether this device saw a fault in the slot that is exchanged with them.
void finish_step(zo_ctx* c, const zo_lora* lora, uint64_t seed, int q, float eps, float lr) {
  if (c->pair_mode) {   // Algorithm 2: g stays on the device as the next forward pass's input; no update here
    PROF(PC_UPDATE, 0.0, launch_pair_g(c->st, c->at<double>(c->plan.losses_d), c->at<float>(c->plan.g), eps,
                                       c->at<uint32_t>(c->plan.status)));
    return;
  }
  if (c->shard_count == 0) {
    enqueue_update(c, lora, seed, q, eps, lr);
    return;
  }
  PROF(PC_LOSS, 0.0, launch_fault_publish(c->st, c->at<uint32_t>(c->plan.status),
                                          c->at<double>(c->plan.losses_d) + 2 * c->cfg.max_q));
}

zo_status step_linear(zo_ctx* c, const zo_weights* w, const zo_lora* lora, const void* X,
                      const void* target, int T, uint64_t seed, int q, float eps, float lr) {
  const zo_config& cf = c->cfg;
  const int bf = c->bf, r = cf.lora_rank, ki = cf.d_model, ko = cf.d_out;
  const double es = bf ? 2.0 : 4.0;            // bytes per activation element (profile bookkeeping)
  const int Tp = (int)up(T, row_pad(cf));
  cudaStream_t st = c->st;
  uint32_t* status = c->at<uint32_t>(c->plan.status);
  float* U = c->at<float>(c->plan.U);
  void* base = c->at<uint8_t>(c->plan.qkv0);
  void* Y = c->at<uint8_t>(c->plan.qkv);
  double* rowloss = c->at<double>(c->plan.rowloss);
  double* rowloss_pass = c->at<double>(c->plan.rowloss_pass);
  float* losses = c->at<float>(c->plan.losses);
  double* losses_d = c->at<double>(c->plan.losses_d);
  Pass passes[MAX_PASSES];
  const int n_pass = step_passes(c, q, passes);
  for (int pi = 0; pi < n_pass; ++pi) {
  const Pass ps = passes[pi];
  const int n = ps.count;
  zo_status s = run_lora_down(c, st, bf, cf.flags, X, ki, lora->A[0], U, T, ki, r, status, c->n_sms,
                              &c->launches, c->err, sizeof(c->err));
  if (s) return s;
  GemmDesc G{};
  G.A = X; G.lda = ki; G.W = w->linear_w; G.M = T; G.N = ko; G.K = ki;
  G.out = base; G.ldo = ko; G.bias = w->linear_bias;
  s = run_gemm(c, st, bf, cf.flags, G, status, c->n_sms, &c->launches, c->err, sizeof(c->err));
  if (s) return s;
  LoraDesc L{};
  L.U = U; L.ldu = r; L.B = lora->B[0]; L.r = r; L.width = ko;
  L.B1 = c->pair_mode ? L.B + (size_t)r * ko : nullptr;
  L.slot_of_sec[0] = 0; L.slot_of_sec[1] = L.slot_of_sec[2] = -1;
  L.scale = cf.lora_scale; L.eps = eps; L.seed = seed; L.tensor_base = 0; L.rows_per_replica = Tp;
  L.rep_base = ps.base; L.rep_stride = ps.stride;
  if (bf && !(cf.flags & ZO_FLAG_SIMT_GEMM) && lora_expand_supported(base, ko, Y, ko, L)) {
    PROF(PC_LORA_APPLY, es * T * ko * (n + 1), launch_lora_expand(st, base, ko, Y, ko, n, T, L, 1, c->n_sms, status));
  } else {
    PROF(PC_LORA_APPLY, es * T * ko * (n + 1), launch_lora_apply(st, bf, base, ko, 1, Y, ko, n, T, L, 1));
  }
  PROF(PC_LOSS, 0.0, launch_mse_rows(st, bf, Y, (const float*)target, n, T, Tp, ko, rowloss_pass));
  PROF(PC_LOSS, 0.0, launch_replica_mean(st, rowloss_pass, nullptr, n, T, ps.base, ps.stride, rowloss, losses, losses_d, status));
  }
  finish_step(c, lora, seed, q, eps, lr);
  return ZO_OK;
}

zo_status step_decoder(zo_ctx* c, const zo_weights* w, const zo_lora* lora, const int32_t* tokens,
                       const int32_t* labels, int E, int S, uint64_t seed, int q, float eps,
                       float lr, const int32_t* cu = nullptr, int total_tokens = 0) {
  const zo_config& cf = c->cfg;
  const int bf = c->bf, r = cf.lora_rank, d = cf.d_model, f = cf.d_ffn, H = cf.n_heads;
  const double es = bf ? 2.0 : 4.0;            // bytes per activation element (profile bookkeeping)
  // packed variable-length batch: T = all tokens, S = longest allowed sequence
  const int T = cu ? total_tokens : E * S, Tp = (int)up(T, row_pad(cf));
  const int nt = c->nt, J = nt * r;
  const bool opt = cf.arch == ZO_ARCH_OPT;
  const int nkind = opt ? 0 : 1;
  const bool unfused_mlp = !bf || (cf.flags & ZO_FLAG_SIMT_GEMM);
  cudaStream_t st = c->st;
  uint32_t* status = c->at<uint32_t>(c->plan.status);
  void *h0 = c->at<uint8_t>(c->plan.h0), *x0 = c->at<uint8_t>(c->plan.x0);
  void *qkv0 = c->at<uint8_t>(c->plan.qkv0), *h = c->at<uint8_t>(c->plan.h);
  void *x = c->at<uint8_t>(c->plan.x), *qkv = c->at<uint8_t>(c->plan.qkv);
  void *a = c->at<uint8_t>(c->plan.a), *gu = c->at<uint8_t>(c->plan.gu);
  float* U = c->at<float>(c->plan.U);
  const float* rope = c->at<float>(c->plan.rope);
  int32_t *lab_idx = c->at<int32_t>(c->plan.lab_idx), *lab_val = c->at<int32_t>(c->plan.lab_val);
  int32_t* lab_cnt = c->at<int32_t>(c->plan.lab_cnt);
  double* rowloss = c->at<double>(c->plan.rowloss);
  double* rowloss_pass = c->at<double>(c->plan.rowloss_pass);
  float* losses = c->at<float>(c->plan.losses);
  double* losses_d = c->at<double>(c->plan.losses_d);
  zo_status s;
#define GEMM(G)                                                                                  \
  do {                                                                                           \
    s = run_gemm(c, st, bf, cf.flags, G, status, c->n_sms, &c->launches, c->err, sizeof(c->err)); \
    if (s) return s;                                                                             \
  } while (0)

  const int P = cf.max_labelled, EP = E * P;
  const int n_classes = cf.loss_kind == ZO_LOSS_CE_LABEL_WORDS ? 2 : cf.vocab;
  SeqLayout sl{E, S, cu, nullptr, T};
  if (cu) {
    int32_t* pos = c->at<int32_t>(c->plan.pos);
    PROF(PC_MISC, 0.0, launch_varlen_index(st, cu, E, T, Tp, S, pos, status));
    sl.pos = pos;
  }
  PROF(PC_MISC, 0.0, launch_label_scan(st, labels, sl, P, n_classes, lab_idx, lab_val, lab_cnt, status));

  Pass passes[MAX_PASSES];
  const int n_pass = step_passes(c, q, passes);
  for (int pi = 0; pi < n_pass; ++pi) {
  const Pass ps = passes[pi];
  const int n = ps.count, M = n * Tp;          // replicas and token rows of this forward pass
  // shared prefix: embedding on the T shared tokens, once for all replicas of the pass
  PROF(PC_MISC, 0.0, launch_embed(st, bf, tokens, w->tok_emb, opt ? w->pos_emb : nullptr, h0, T, Tp, sl, d, cf.vocab, status));

  for (int l = 0; l < cf.n_layers; ++l) {
    const zo_layer_weights& W = w->layers[l];
    const bool first = l == 0;
    const int rows = first ? Tp : M;           // layer 0 still works on the shared block
    void* hin = first ? h0 : h;
    void* xn = first ? x0 : x;
    PROF(PC_NORM, 2.0 * es * rows * d, launch_norm(st, bf, nkind, hin, xn, W.norm1_g, W.norm1_b, rows, d, cf.norm_eps, nullptr, 0, 0));
    LoraDesc L{};
    L.U = U; L.ldu = J; L.B = J ? lora->B[l] : nullptr; L.r = r; L.width = d;
    L.B1 = (J && c->pair_mode) ? L.B + (size_t)nt * r * d : nullptr;
    for (int j = 0; j < 3; ++j) L.slot_of_sec[j] = c->slot_of_sec[j];
    L.scale = cf.lora_scale; L.eps = eps; L.seed = seed; L.tensor_base = (uint32_t)(l * nt);
    L.rows_per_replica = Tp;
    L.rep_base = ps.base; L.rep_stride = ps.stride;
    const bool slab = J && slab_lora_ok(bf, cf.flags, Tp, d, r);
    const int kslot = r > 32 ? 128 : 64;       // K extent of one slot of the packed bf16 U
    void* ub = c->at<uint8_t>(c->plan.ub);
    if (J) {
      s = run_lora_down(c, st, bf, cf.flags, xn, d, lora->A[l], U, rows, d, J, status, c->n_sms,
                        &c->launches, c->err, sizeof(c->err), (slab && !first) ? ub : nullptr, nt * kslot, r, kslot);
      if (s) return s;
    }
    // Quantised storage.  Default: each weight is decoded once per forward pass into scratch, right before
    // its GEMM, for all replicas of the pass (large launches reuse every weight tile hundreds of times).
    // ZO_FLAG_DEQUANT_FUSED: launches of at most 256 rows (small batches: the GEMM is a stream of weights)
    // decode the codes inside the tensor-core kernel's operand producer instead, so a weight is read once, as
    // codes, and never written back.
    const bool tcore = bf && !(cf.flags & ZO_FLAG_SIMT_GEMM);
    void* wdq = c->at<uint8_t>(c->plan.wdq);
    auto set_weight = [&](GemmDesc& D, const void* wq, const float* sc, int n_rows, int k_in) {
      if (cf.weight_format == ZO_W_NATIVE) { D.W = wq; return; }
      if (tcore && D.M <= 256 && (cf.flags & ZO_FLAG_DEQUANT_FUSED)) {
        D.W = nullptr; D.wfmt = cf.weight_format; D.wq = wq; D.wscale = sc;
        return;
      }
      PROF(PC_DEQUANT, 0.0, launch_dequant(st, bf, cf.weight_format, wq, sc, wdq, n_rows, k_in));
      D.W = wdq;
    };
    // The rotary embedding rides in the epilogue of whichever tensor-core GEMM writes q|k|v last.
    bool rope_done = opt;
    auto with_rope = [&](GemmDesc& D) {
      D.rope_tab = rope; D.rope_cols = 2 * d; D.rope_dh = d / H; D.rope_s = S; D.rope_tp = Tp; D.rope_pos = sl.pos;
      rope_done = true;
    };
    GemmDesc G{};
    G.A = xn; G.lda = d; G.M = rows; G.N = 3 * d; G.K = d; G.bias = W.b_qkv;
    set_weight(G, W.w_qkv, W.s_qkv, 3 * d, d);
    G.prof_class = PC_GEMM_QKV;
    if (first) {
      // first perturbed layer: one base product on the shared block, expanded to 2q outputs
      G.out = qkv0; G.ldo = 3 * d;
      GEMM(G);
      if (tcore && lora_expand_supported(qkv0, 3 * d, qkv, 3 * d, L)) {
        // expansion to the 2q outputs of the pass: bound by the output stream, full-line stores
        PROF(PC_LORA_APPLY, es * T * 3 * d * (n + 1), launch_lora_expand(st, qkv0, 3 * d, qkv, 3 * d, n, T, L, 3, c->n_sms, status));
      } else {
        PROF(PC_LORA_APPLY, es * T * 3 * d * (n + 1), launch_lora_apply(st, bf, qkv0, 3 * d, 1, qkv, 3 * d, n, T, L, 3));
      }
    } else if (J && fused_lora_ok(bf, cf.flags, Tp, d)) {
      G.out = qkv; G.ldo = 3 * d; G.lora = &L;
      if (slab) { G.lora_slab = 1; G.pack_u = ub; G.pack_ld = nt * kslot; G.pack_r = r; G.kslot = kslot; G.khalf = kslot / 2; }
      if (slab && !opt) with_rope(G);
      GEMM(G);
    } else {
      G.out = qkv; G.ldo = 3 * d;
      if (!J && tcore && !opt) with_rope(G);
      GEMM(G);
      if (J) { PROF(PC_LORA_APPLY, 0.0, launch_lora_apply(st, bf, qkv, 3 * d, 0, qkv, 3 * d, n, T, L, 3)); }
    }
    if (!rope_done) { PROF(PC_ROPE, 4.0 * es * M * d, launch_rope(st, bf, qkv, M, Tp, sl, d, H, rope)); }   // q and k, read and written
    if (tcore && !(cf.flags & ZO_FLAG_ATTN_WARP_MMA) && attention_tc_supported(d / H, S)) {
      int ae = 0;
      PROF(PC_ATTN, 4.0 * es * M * d, ae = launch_attention_tc(st, qkv, x, n, sl, Tp, d, H, status, c->n_sms));
      if (ae) {
        snprintf(c->err, sizeof(c->err), "tensor-core attention launch failed (code %d)", ae);
        return ZO_ERR_CUDA;
      }
    } else if (bf && !(cf.flags & ZO_FLAG_SIMT_GEMM) && attention_mma_supported(d / H)) {
      PROF(PC_ATTN, 4.0 * es * M * d, launch_attention_mma(st, qkv, x, n, sl, Tp, d, H));
    } else {
      PROF(PC_ATTN, 4.0 * es * M * d, launch_attention_simt(st, bf, qkv, x, n, sl, Tp, d, H));
    }
    GemmDesc O{};
    O.A = x; O.lda = d; O.M = M; O.N = d; O.K = d; O.out = h; O.ldo = d;
    set_weight(O, W.w_o, W.s_o, d, d);
    O.bias = W.b_o; O.res = hin; O.ldr = d; O.res_mod = first ? Tp : 0; O.prof_class = PC_GEMM_O;
    GEMM(O);
    PROF(PC_NORM, 2.0 * es * M * d, launch_norm(st, bf, nkind, h, x, W.norm2_g, W.norm2_b, M, d, cf.norm_eps, nullptr, 0, 0));
    GemmDesc F1{};
    F1.A = x; F1.lda = d; F1.M = M; F1.K = d; F1.bias = W.b_fc1; F1.prof_class = PC_GEMM_FC1;
    set_weight(F1, W.w_fc1, W.s_fc1, opt ? f : 2 * f, d);
    if (opt) {
      F1.N = f; F1.out = a; F1.ldo = f; F1.act = ACT_RELU;
      GEMM(F1);
    } else if (unfused_mlp) {
      F1.N = 2 * f; F1.out = gu; F1.ldo = 2 * f;
      GEMM(F1);
      PROF(PC_SWIGLU, 0.0, launch_swiglu(st, bf, gu, a, M, f));
    } else {
      F1.N = 2 * f; F1.out = a; F1.ldo = f; F1.swiglu = 1;
      GEMM(F1);
    }
    GemmDesc F2{};
    F2.A = a; F2.lda = f; F2.M = M; F2.N = d; F2.K = f; F2.out = h; F2.ldo = d;
    set_weight(F2, W.w_fc2, W.s_fc2, d, f);
    F2.bias = W.b_fc2; F2.res = h; F2.ldr = d; F2.prof_class = PC_GEMM_FC2;
    GEMM(F2);
  }

  // per-replica loss on the labelled rows only
  const int Mh = n * EP;
  void* xh = c->at<uint8_t>(c->plan.xh);
  PROF(PC_NORM, 2.0 * es * Mh * d, launch_norm(st, bf, nkind, h, xh, w->final_norm_g, w->final_norm_b, Mh, d, cf.norm_eps, lab_idx, EP, Tp));
  const void* head = cf.tie_lm_head ? w->tok_emb : w->lm_head;
  if (fused_ce(cf)) {
    // LM head and log-softmax in one pass: the logits stay in tensor memory and registers
    GemmDesc Hd{};
    Hd.A = xh; Hd.lda = d; Hd.W = head; Hd.M = Mh; Hd.N = cf.vocab; Hd.K = d; Hd.prof_class = PC_GEMM_HEAD;
    Hd.ce_part = c->at<uint8_t>(c->plan.ce_part); Hd.ce_logit = c->at<float>(c->plan.ce_logit);
    Hd.ce_label = lab_val; Hd.ce_ep = EP;
    GEMM(Hd);
    PROF(PC_LOSS, 0.0, launch_ce_merge(st, Hd.ce_part, (int)ce_parts_per_row(cf), Hd.ce_logit, lab_val, EP, Mh, rowloss_pass));
  } else if (cf.loss_kind == ZO_LOSS_CE_FULL_VOCAB) {
    float* logits = c->at<float>(c->plan.logits);
    GemmDesc Hd{};
    Hd.A = xh; Hd.lda = d; Hd.W = head; Hd.M = Mh; Hd.N = cf.vocab; Hd.K = d;
    Hd.out = logits; Hd.ldo = cf.vocab; Hd.out_f32 = 1; Hd.prof_class = PC_GEMM_HEAD;
    GEMM(Hd);
    PROF(PC_LOSS, 0.0, launch_ce_rows(st, logits, cf.vocab, cf.vocab, lab_val, EP, Mh, rowloss_pass));
  } else {
    PROF(PC_LOSS, 0.0, launch_label_word_rows(st, bf, xh, head, d, cf.label_words[0], cf.label_words[1], lab_val, EP, Mh, rowloss_pass));
  }
  PROF(PC_LOSS, 0.0, launch_replica_mean(st, rowloss_pass, lab_val, n, EP, ps.base, ps.stride, rowloss, losses, losses_d, status));
  }  // passes

  finish_step(c, lora, seed, q, eps, lr);
#undef GEMM
  return ZO_OK;
}

zo_status check_step_args(zo_ctx* c, const zo_weights* w, const zo_lora* lora, const void* tokens,
                          const void* labels, int E, int S, int q, float eps, float lr) {
  if (!c) return ZO_ERR_INVALID_ARG;
  const zo_config& cf = c->cfg;
  if (!w || !lora || !tokens || !labels) return fail(c, ZO_ERR_INVALID_ARG, "null argument");
  if (q < 1 || q > cf.max_q) return fail(c, ZO_ERR_INVALID_ARG, "q outside 1..max_q");
  if (E < 1 || E > cf.max_E) return fail(c, ZO_ERR_INVALID_ARG, "E outside 1..max_E");
  if (S < 1 || S > cf.max_seq) return fail(c, ZO_ERR_INVALID_ARG, "S outside 1..max_seq");
  if (!(eps >= 0.f) || !isfinite(eps)) return fail(c, ZO_ERR_INVALID_ARG, "eps must be finite and >= 0");
  if (!isfinite(lr)) return fail(c, ZO_ERR_INVALID_ARG, "lr must be finite");
  if (!lora->A || !lora->B) return fail(c, ZO_ERR_INVALID_ARG, "lora pointer arrays are NULL");
  if (cf.arch == ZO_ARCH_LINEAR) {
    if (!w->linear_w || !lora->A[0] || !lora->B[0]) return fail(c, ZO_ERR_INVALID_ARG, "null linear tensor");
    return ZO_OK;
  }
  if (!w->tok_emb || !w->final_norm_g || !w->layers) return fail(c, ZO_ERR_INVALID_ARG, "null model tensor");
  if (cf.arch == ZO_ARCH_OPT && (!w->pos_emb || !w->final_norm_b))
    return fail(c, ZO_ERR_INVALID_ARG, "OPT needs pos_emb and final_norm_b");
  if (!cf.tie_lm_head && !w->lm_head) return fail(c, ZO_ERR_INVALID_ARG, "lm_head is NULL");
  for (int l = 0; l < cf.n_layers; ++l) {
    const zo_layer_weights& W = w->layers[l];
    if (!W.norm1_g || !W.w_qkv || !W.w_o || !W.norm2_g || !W.w_fc1 || !W.w_fc2)
      return fail(c, ZO_ERR_INVALID_ARG, "null layer tensor");
    if (cf.arch == ZO_ARCH_OPT && (!W.norm1_b || !W.b_qkv || !W.b_o || !W.norm2_b || !W.b_fc1 || !W.b_fc2))
      return fail(c, ZO_ERR_INVALID_ARG, "OPT layers need every bias");
    if (c->nt && (!lora->A[l] || !lora->B[l])) return fail(c, ZO_ERR_INVALID_ARG, "null LoRA tensor");
    if (cf.weight_format != ZO_W_NATIVE && (!W.s_qkv || !W.s_o || !W.s_fc1 || !W.s_fc2))
      return fail(c, ZO_ERR_INVALID_ARG, "quantised weights need their scales");
  }
  return ZO_OK;
}

// Start of every step: launch counter and device status word cleared; a sharded step also zeroes
// the fp64 loss array so that the entries of the other shards' queries read 0 until the exchange.
zo_status begin_step(zo_ctx* c, int q) {
  c->launches = 0;
  if (c->shard_count && c->shard_begin + c->shard_count > q)
    return fail(c, ZO_ERR_INVALID_ARG, "query shard reaches past q");
  if ((c->shard_count ? c->shard_count : q) > run_q(c->cfg))
    return fail(c, ZO_ERR_INVALID_ARG, "more queries in one step than max_shard_q sized the workspace for");
  cudaError_t e = cudaMemsetAsync(c->at<uint32_t>(c->plan.status), 0, 4, c->st);
  if (e == cudaSuccess) {   // a sharded step zeroes the whole loss array; the fault slot is cleared by every step
    double* ld = c->at<double>(c->plan.losses_d);
    const size_t n = (size_t)2 * c->cfg.max_q;
    e = c->shard_count ? cudaMemsetAsync(ld, 0, (n + 1) * 8, c->st) : cudaMemsetAsync(ld + n, 0, 8, c->st);
  }
  if (e != cudaSuccess) return fail(c, ZO_ERR_CUDA, "cudaMemsetAsync: %s", cudaGetErrorString(e));
  return ZO_OK;
}

zo_status do_step(zo_ctx* c, const zo_weights* w, const zo_lora* lora, const void* tokens,
                  const void* labels, int E, int S, uint64_t seed, int q, float eps, float lr) {
  zo_status s = begin_step(c, q);
  if (s) return s;
  cudaError_t e;
  if (c->cfg.arch == ZO_ARCH_LINEAR)
    s = step_linear(c, w, lora, tokens, labels, E * S, seed, q, eps, lr);
  else
    s = step_decoder(c, w, lora, (const int32_t*)tokens, (const int32_t*)labels, E, S, seed, q, eps, lr);
  if (s) return s;
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(c, ZO_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  c->stepped = 1; c->last_q = q; c->last_E = E; c->last_S = S;
  return ZO_OK;
}

}  // namespace

extern "C" {

size_t zo_workspace_bytes(const zo_config* cfg) {
  char err[256];
  if (check_config(cfg, err, sizeof(err)) != ZO_OK) return 0;
  return make_plan(*cfg).total;
}

zo_status zo_init(const zo_config* cfg, void* workspace, size_t workspace_bytes, void* cuda_stream,
                  zo_ctx** out) {
  if (!out) { snprintf(g_init_error, sizeof(g_init_error), "out is NULL"); return ZO_ERR_INVALID_ARG; }
  *out = nullptr;
  zo_status s = check_config(cfg, g_init_error, sizeof(g_init_error));
  if (s) return s;
  const Plan plan = make_plan(*cfg);
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < plan.total) {
    snprintf(g_init_error, sizeof(g_init_error), "workspace NULL, misaligned or smaller than %zu bytes", plan.total);
    return ZO_ERR_WORKSPACE;
  }
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  int major = 0;
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (e != cudaSuccess) {
    snprintf(g_init_error, sizeof(g_init_error), "no usable CUDA device: %s", cudaGetErrorString(e));
    return ZO_ERR_CUDA;
  }
  if (major != 10) {
    snprintf(g_init_error, sizeof(g_init_error), "device compute capability %d.x: built for sm_100a only", major);
    return ZO_ERR_UNSUPPORTED;
  }
  if (cfg->precision == ZO_BF16 && !(cfg->flags & ZO_FLAG_SIMT_GEMM)) {
    const int ge = gemm_tc_init();
    if (ge) {
      snprintf(g_init_error, sizeof(g_init_error), "tensor-core GEMM set-up failed (%d)", ge);
      return ZO_ERR_CUDA;
    }
  }
  zo_ctx* c = new (std::nothrow) zo_ctx();   // value-initialised: every field zero
  if (c) {
    c->prof = new (std::nothrow) std::vector<ProfRec>();
    c->evpool = new (std::nothrow) std::vector<cudaEvent_t>();
  }
  if (!c || !c->prof || !c->evpool) {
    snprintf(g_init_error, sizeof(g_init_error), "out of host memory");
    zo_free(c);
    return ZO_ERR_CUDA;
  }
  c->cfg = *cfg; c->plan = plan; c->ws = (uint8_t*)workspace; c->st = (cudaStream_t)cuda_stream;
  c->bf = cfg->precision == ZO_BF16; c->n_sms = sms;
  c->nt = cfg->arch == ZO_ARCH_LINEAR ? 1 : n_targets(*cfg);
  int slot = 0;
  for (int j = 0; j < 3; ++j) c->slot_of_sec[j] = ((cfg->lora_targets >> j) & 1) ? slot++ : -1;
  // a defined (finite) start for pad rows, which kernels carry along but never mix into real rows
  e = cudaMemsetAsync(workspace, 0, plan.total, c->st);
  if (e == cudaSuccess && cfg->arch == ZO_ARCH_LLAMA) {
    launch_rope_table(c->st, c->at<float>(plan.rope), cfg->max_seq, cfg->d_model / cfg->n_heads, cfg->rope_theta);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) {
    snprintf(g_init_error, sizeof(g_init_error), "workspace set-up: %s", cudaGetErrorString(e));
    zo_free(c);
    return ZO_ERR_CUDA;
  }
  *out = c;
  return ZO_OK;
}

zo_status zo_step(zo_ctx* ctx, const zo_weights* weights, const zo_lora* lora, const void* tokens,
                  const void* labels, int32_t E, int32_t S, uint64_t seed, int32_t q, float eps,
                  float lr) {
  zo_status s = check_step_args(ctx, weights, lora, tokens, labels, E, S, q, eps, lr);
  if (s) return s;
  return do_step(ctx, weights, lora, tokens, labels, E, S, seed, q, eps, lr);
}

zo_status zo_step_varlen(zo_ctx* ctx, const zo_weights* weights, const zo_lora* lora, const int32_t* tokens,
                         const int32_t* labels, const int32_t* cu_seqlens, int32_t E, int32_t total_tokens,
                         int32_t max_len, uint64_t seed, int32_t q, float eps, float lr) {
  zo_status s = check_step_args(ctx, weights, lora, tokens, labels, E, max_len, q, eps, lr);
  if (s) return s;
  if (ctx->cfg.arch == ZO_ARCH_LINEAR) return fail(ctx, ZO_ERR_UNSUPPORTED, "variable-length batches are for decoders");
  if (!cu_seqlens) return fail(ctx, ZO_ERR_INVALID_ARG, "cu_seqlens is NULL");
  if (total_tokens < E || (long long)total_tokens > (long long)E * max_len ||
      (long long)total_tokens > (long long)ctx->cfg.max_E * ctx->cfg.max_seq)
    return fail(ctx, ZO_ERR_INVALID_ARG, "total_tokens outside E .. E*max_len");
  s = begin_step(ctx, q);
  if (s) return s;
  s = step_decoder(ctx, weights, lora, tokens, labels, E, max_len, seed, q, eps, lr, cu_seqlens, total_tokens);
  if (s) return s;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ctx, ZO_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  ctx->stepped = 1; ctx->last_q = q; ctx->last_E = E; ctx->last_S = max_len;
  return ZO_OK;
}

zo_status zo_step_host(zo_ctx* ctx, const zo_weights* weights, const zo_lora* lora,
                       const void* host_tokens, const void* host_labels, int32_t E, int32_t S,
                       uint64_t seed, int32_t q, float eps, float lr) {
  zo_status s = check_step_args(ctx, weights, lora, host_tokens, host_labels, E, S, q, eps, lr);
  if (s) return s;
  const zo_config& cf = ctx->cfg;
  const size_t T = (size_t)E * S;
  size_t tb, lb;
  if (cf.arch == ZO_ARCH_LINEAR) {
    tb = T * cf.d_model * (ctx->bf ? 2 : 4);
    lb = T * cf.d_out * 4;
  } else {
    tb = lb = T * 4;
  }
  void* dt = ctx->at<uint8_t>(ctx->plan.tok_stage);
  void* dl = ctx->at<uint8_t>(ctx->plan.lab_stage);
  cudaError_t e = cudaMemcpyAsync(dt, host_tokens, tb, cudaMemcpyHostToDevice, ctx->st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(dl, host_labels, lb, cudaMemcpyHostToDevice, ctx->st);
  if (e != cudaSuccess) return fail(ctx, ZO_ERR_CUDA, "host-to-device copy: %s", cudaGetErrorString(e));
  return do_step(ctx, weights, lora, dt, dl, E, S, seed, q, eps, lr);
}

zo_status zo_losses(zo_ctx* ctx, float* host_losses, float* host_g) {
  if (!ctx) return ZO_ERR_INVALID_ARG;
  if (!host_losses) return fail(ctx, ZO_ERR_INVALID_ARG, "host_losses is NULL");
  if (!ctx->stepped) return fail(ctx, ZO_ERR_STATE, "zo_losses before any zo_step");
  uint32_t st = 0;
  cudaError_t e = cudaMemcpyAsync(host_losses, ctx->at<float>(ctx->plan.losses), (size_t)2 * ctx->last_q * 4,
                                  cudaMemcpyDeviceToHost, ctx->st);
  if (e == cudaSuccess && host_g)
    e = cudaMemcpyAsync(host_g, ctx->at<float>(ctx->plan.g), (size_t)ctx->last_q * 4, cudaMemcpyDeviceToHost, ctx->st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(&st, ctx->at<uint32_t>(ctx->plan.status), 4, cudaMemcpyDeviceToHost, ctx->st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->st);
  if (e != cudaSuccess) return fail(ctx, ZO_ERR_CUDA, "zo_losses: %s", cudaGetErrorString(e));
  if (st & ST_TIMEOUT) return fail(ctx, ZO_ERR_TIMEOUT, "a bounded device-side wait ran out");
  if (st & (ST_BAD_LABELS | ST_BAD_TOKEN))
    return fail(ctx, ZO_ERR_INVALID_ARG, "token id or label out of range, or too many labelled positions");
  if (st & ST_NONFINITE) return fail(ctx, ZO_ERR_NONFINITE, "a replica loss is not finite; B left untouched");
  if (st & ST_PEER_FAULT)
    return fail(ctx, ZO_ERR_STATE, "another device of the sharded step reported a fault; no device applied the update");
  return ZO_OK;
}

zo_status zo_row_losses(zo_ctx* ctx, float* host_rows, int32_t* host_n_rows) {
  if (!ctx) return ZO_ERR_INVALID_ARG;
  if (!host_n_rows) return fail(ctx, ZO_ERR_INVALID_ARG, "host_n_rows is NULL");
  if (!ctx->stepped) return fail(ctx, ZO_ERR_STATE, "zo_row_losses before any zo_step");
  const int rows = ctx->cfg.arch == ZO_ARCH_LINEAR ? ctx->last_E * ctx->last_S
                                                   : ctx->last_E * ctx->cfg.max_labelled;
  *host_n_rows = rows;
  if (!host_rows) return ZO_OK;
  const size_t cnt = (size_t)2 * ctx->last_q * rows;
  double* tmp = new (std::nothrow) double[cnt];
  if (!tmp) return fail(ctx, ZO_ERR_CUDA, "out of host memory");
  cudaError_t e = cudaMemcpyAsync(tmp, ctx->at<double>(ctx->plan.rowloss), cnt * 8, cudaMemcpyDeviceToHost, ctx->st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->st);
  if (e == cudaSuccess)
    for (size_t i = 0; i < cnt; ++i) host_rows[i] = (float)tmp[i];
  delete[] tmp;
  if (e != cudaSuccess) return fail(ctx, ZO_ERR_CUDA, "zo_row_losses: %s", cudaGetErrorString(e));
  return ZO_OK;
}

int32_t zo_launch_count(const zo_ctx* ctx) { return ctx ? ctx->launches : 0; }

zo_status zo_set_schedule(zo_ctx* ctx, int32_t schedule) {
  if (!ctx) return ZO_ERR_INVALID_ARG;
  if (schedule < ZO_SCHEDULE_FULL || schedule > ZO_SCHEDULE_SEQUENTIAL)
    return fail(ctx, ZO_ERR_INVALID_ARG, "unknown schedule");
  ctx->schedule = schedule;
  return ZO_OK;
}

zo_status zo_test_expire_wait(zo_ctx* ctx, uint64_t wait_limit_ns) {
  if (!ctx) return ZO_ERR_INVALID_ARG;
  if (wait_limit_ns > 2000000000ull) return fail(ctx, ZO_ERR_INVALID_ARG, "wait limit above the regular 2 s");
  ctx->test_wait_ns = wait_limit_ns;
  return ZO_OK;
}

zo_status zo_set_query_shard(zo_ctx* ctx, int32_t q_begin, int32_t q_count) {
  if (!ctx) return ZO_ERR_INVALID_ARG;
  if (q_begin < 0 || q_count < 0 || (q_count == 0 && q_begin != 0) || q_begin + q_count > ctx->cfg.max_q)
    return fail(ctx, ZO_ERR_INVALID_ARG, "query shard outside 0..max_q");
  ctx->shard_begin = q_begin;
  ctx->shard_count = q_count;
  return ZO_OK;
}

zo_status zo_loss_buffer(zo_ctx* ctx, double** dev_losses, int32_t* host_capacity) {
  if (!ctx) return ZO_ERR_INVALID_ARG;
  if (!dev_losses) return fail(ctx, ZO_ERR_INVALID_ARG, "dev_losses is NULL");
  *dev_losses = ctx->at<double>(ctx->plan.losses_d);
  if (host_capacity) *host_capacity = 2 * ctx->cfg.max_q + 1;
  return ZO_OK;
}

zo_status zo_apply_update(zo_ctx* ctx, const zo_lora* lora, uint64_t seed, int32_t q, float eps, float lr) {
  if (!ctx) return ZO_ERR_INVALID_ARG;
  if (!lora || !lora->B) return fail(ctx, ZO_ERR_INVALID_ARG, "lora is NULL");
  if (!ctx->stepped) return fail(ctx, ZO_ERR_STATE, "zo_apply_update before any zo_step");
  if (q != ctx->last_q) return fail(ctx, ZO_ERR_INVALID_ARG, "q differs from the step's");
  if (!(eps >= 0.f) || !isfinite(eps) || !isfinite(lr)) return fail(ctx, ZO_ERR_INVALID_ARG, "eps or lr not finite");
  const int n_b = ctx->cfg.arch == ZO_ARCH_LINEAR ? 1 : (ctx->nt ? ctx->cfg.n_layers : 0);
  for (int l = 0; l < n_b; ++l)
    if (!lora->B[l]) return fail(ctx, ZO_ERR_INVALID_ARG, "null LoRA tensor");
  zo_ctx* c = ctx;
  PROF(PC_LOSS, 0.0, launch_losses_refresh(ctx->st, ctx->at<double>(ctx->plan.losses_d), ctx->at<float>(ctx->plan.losses),
                                           2 * q, ctx->at<double>(ctx->plan.losses_d) + 2 * ctx->cfg.max_q,
                                           ctx->at<uint32_t>(ctx->plan.status)));
  enqueue_update(ctx, lora, seed, q, eps, lr);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(ctx, ZO_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  return ZO_OK;
}

void zo_free(zo_ctx* ctx) {
  if (!ctx) return;
  if (ctx->prof) {
    for (ProfRec& r : *ctx->prof) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
    delete ctx->prof;
  }
  if (ctx->evpool) {
    for (cudaEvent_t e : *ctx->evpool) cudaEventDestroy(e);
    delete ctx->evpool;
  }
  delete ctx;
}

zo_status zo_profile_enable(zo_ctx* ctx, int32_t on) {
  if (!ctx || !ctx->prof || !ctx->evpool) return ZO_ERR_INVALID_ARG;
  ctx->prof_on = on ? 1 : 0;
  return ZO_OK;
}

zo_status zo_profile_read(zo_ctx* ctx, double* host_ms, double* host_flops, int32_t* host_launches) {
  if (!ctx || !host_ms || !host_flops || !host_launches) return ZO_ERR_INVALID_ARG;
  for (int i = 0; i < PC_COUNT; ++i) { host_ms[i] = 0.0; host_flops[i] = 0.0; host_launches[i] = 0; }
  cudaError_t e = cudaStreamSynchronize(ctx->st);
  if (e != cudaSuccess) return fail(ctx, ZO_ERR_CUDA, "zo_profile_read: %s", cudaGetErrorString(e));
  for (ProfRec& r : *ctx->prof) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.e0, r.e1) == cudaSuccess) {
      host_ms[r.cat] += ms; host_flops[r.cat] += r.flops; ++host_launches[r.cat];
    }
    ctx->evpool->push_back(r.e0);
    ctx->evpool->push_back(r.e1);
  }
  ctx->prof->clear();
  return ZO_OK;
}

const char* zo_last_error(const zo_ctx* ctx) { return ctx ? ctx->err : g_init_error; }

zo_status zo_dequantize(void* cuda_stream, int32_t weight_format, int32_t precision, const void* codes,
                        const float* scale, void* out, int32_t rows, int32_t k_in) {
  if (!codes || !scale || !out || rows < 1 || k_in < 1) return ZO_ERR_INVALID_ARG;
  if (weight_format != ZO_W_INT8 && weight_format != ZO_W_NF4) return ZO_ERR_INVALID_ARG;
  if (precision != ZO_FP32 && precision != ZO_BF16) return ZO_ERR_INVALID_ARG;
  if (k_in % (weight_format == ZO_W_NF4 ? 64 : 16)) return ZO_ERR_UNSUPPORTED;
  launch_dequant((cudaStream_t)cuda_stream, precision == ZO_BF16, weight_format, codes, scale, out, rows, k_in);
  return cudaGetLastError() == cudaSuccess ? ZO_OK : ZO_ERR_CUDA;
}

zo_status zo_perturbation(void* cuda_stream, uint64_t seed, uint32_t tensor_id, uint32_t query,
                          int64_t n, uint32_t* dev_u32, float* dev_z) {
  if (n < 0 || (n > 0 && !dev_u32 && !dev_z)) return ZO_ERR_INVALID_ARG;
  if (n > ((int64_t)1 << 34)) return ZO_ERR_INVALID_ARG;   // block index must fit 32 bits
  launch_perturbation((cudaStream_t)cuda_stream, seed, tensor_id, query, n, dev_u32, dev_z);
  return cudaGetLastError() == cudaSuccess ? ZO_OK : ZO_ERR_CUDA;
}

size_t zo_mp_lora_scratch_bytes(int32_t precision, int32_t T, int32_t k_in, int32_t k_out, int32_t r,
                                int32_t q, int32_t x_replicated) {
  if (T < 1 || k_in < 1 || k_out < 1 || r < 1 || q < 1) return 0;
  const size_t es = precision == ZO_BF16 ? 2 : 4;
  const size_t rows = x_replicated ? (size_t)2 * q * T : (size_t)T;
  size_t b = 256 + up(rows * r * 4, 256);
  if (!x_replicated) b += up((size_t)T * k_out * es, 256);
  if (precision == ZO_BF16) b += up(rows * 128 * 2, 256);       // packed bf16 U of the tensor-core LoRA blocks
  return b;
}

}  // extern "C"

// The layer with either storage form of B: B1 == null is the master-copy form (z regenerated), otherwise
// (B, B1) is a stored pair and q must be 1.
static zo_status mp_lora_linear_impl(void* cuda_stream, int32_t precision, const void* X, const void* W,
                            const void* bias, const void* A, const float* B, const float* B1, void* Y, int32_t T,
                            int32_t k_in, int32_t k_out, int32_t r, float scale, uint64_t seed,
                            uint32_t tensor_id, int32_t q, float eps, int32_t x_replicated,
                            void* scratch, size_t scratch_bytes, uint32_t flags) {
  if (!X || !W || !A || !B || !Y || !scratch) return ZO_ERR_INVALID_ARG;
  if (precision != ZO_FP32 && precision != ZO_BF16) return ZO_ERR_INVALID_ARG;
  if (T < 1 || k_in < 1 || k_out < 1 || r < 1 || r > 64 || q < 1 || q > ZO_MAX_Q || !(eps >= 0.f))
    return ZO_ERR_INVALID_ARG;
  const int bf = precision == ZO_BF16;
  if (k_out % 4) return ZO_ERR_UNSUPPORTED;
  if (bf && (k_in % 8 || k_out % 8)) return ZO_ERR_UNSUPPORTED;
  if (bf && x_replicated && T % 128) return ZO_ERR_UNSUPPORTED;
  const size_t need = zo_mp_lora_scratch_bytes(precision, T, k_in, k_out, r, q, x_replicated);
  if (((uintptr_t)scratch & 255) || scratch_bytes < need) return ZO_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return ZO_ERR_CUDA;
  const int n = 2 * q;
  const size_t rows = x_replicated ? (size_t)n * T : (size_t)T;
  uint8_t* sp = (uint8_t*)scratch;
  uint32_t* status = (uint32_t*)sp;
  float* U = (float*)(sp + 256);
  void* base = sp + 256 + up(rows * r * 4, 256);   // shared input: base product X W^T
  void* pack = (uint8_t*)base + (x_replicated ? 0 : up((size_t)T * k_out * (bf ? 2 : 4), 256));
  if (cudaMemsetAsync(status, 0, 4, st) != cudaSuccess) return ZO_ERR_CUDA;
  LoraDesc L{};
  L.U = U; L.ldu = r; L.B = B; L.B1 = B1; L.r = r; L.width = k_out;
  L.slot_of_sec[0] = 0; L.slot_of_sec[1] = L.slot_of_sec[2] = -1;
  L.scale = scale; L.eps = eps; L.seed = seed; L.tensor_base = tensor_id; L.rows_per_replica = T;
  L.rep_base = 0; L.rep_stride = 1;
  const bool slab = x_replicated && slab_lora_ok(bf, flags, T, k_out, r);
  const int kslot = r > 32 ? 128 : 64;
  if (slab && cudaMemsetAsync(pack, 0, rows * kslot * 2, st) != cudaSuccess) return ZO_ERR_CUDA;
  int launches = 0;
  char err[128];
  zo_status s = run_lora_down(nullptr, st, bf, flags, X, k_in, A, U, (int)rows, k_in, r, status, sms,
                              &launches, err, sizeof(err), slab ? pack : nullptr, kslot, r, kslot);
  if (s) return s;
  GemmDesc G{};
  G.A = X; G.lda = k_in; G.W = W; G.M = (int)rows; G.N = k_out; G.K = k_in; G.bias = bias;
  G.ldo = k_out;
  if (!x_replicated) {
    G.out = base;
    s = run_gemm(nullptr, st, bf, flags, G, status, sms, &launches, err, sizeof(err));
    if (s) return s;
    if (bf && !(flags & ZO_FLAG_SIMT_GEMM) && lora_expand_supported(base, k_out, Y, k_out, L)) {
      launch_lora_expand(st, base, k_out, Y, k_out, n, T, L, 1, sms, status);
    } else {
      launch_lora_apply(st, bf, base, k_out, 1, Y, k_out, n, T, L, 1);
    }
  } else if (fused_lora_ok(bf, flags, T, k_out)) {
    G.out = Y; G.lora = &L;
    if (slab) { G.lora_slab = 1; G.pack_u = pack; G.pack_ld = kslot; G.pack_r = r; G.kslot = kslot; G.khalf = kslot / 2; }
    s = run_gemm(nullptr, st, bf, flags, G, status, sms, &launches, err, sizeof(err));
    if (s) return s;
  } else {
    G.out = Y;
    s = run_gemm(nullptr, st, bf, flags, G, status, sms, &launches, err, sizeof(err));
    if (s) return s;
    launch_lora_apply(st, bf, Y, k_out, 0, Y, k_out, n, T, L, 1);
  }
  return cudaGetLastError() == cudaSuccess ? ZO_OK : ZO_ERR_CUDA;
}

extern "C" {

zo_status zo_mp_lora_linear(void* cuda_stream, int32_t precision, const void* X, const void* W,
                            const void* bias, const void* A, const float* B, void* Y, int32_t T,
                            int32_t k_in, int32_t k_out, int32_t r, float scale, uint64_t seed,
                            uint32_t tensor_id, int32_t q, float eps, int32_t x_replicated,
                            void* scratch, size_t scratch_bytes, uint32_t flags) {
  return mp_lora_linear_impl(cuda_stream, precision, X, W, bias, A, B, nullptr, Y, T, k_in, k_out, r, scale, seed,
                             tensor_id, q, eps, x_replicated, scratch, scratch_bytes, flags);
}

zo_status zo_mp_lora_linear_pair(void* cuda_stream, int32_t precision, const void* X, const void* W,
                                 const void* bias, const void* A, float* B_pair, void* Y, int32_t T,
                                 int32_t k_in, int32_t k_out, int32_t r, float scale, uint64_t seed,
                                 uint32_t tensor_id, float g_prev, float eps, float lr, int32_t x_replicated,
                                 void* scratch, size_t scratch_bytes, uint32_t flags) {
  if (!B_pair || r < 1 || k_out < 1 || !(eps > 0.f) || !isfinite(eps) || !isfinite(lr) || !isfinite(g_prev))
    return ZO_ERR_INVALID_ARG;
  if (k_out % 4) return ZO_ERR_UNSUPPORTED;
  // lines 2-6 of Algorithm 2 on the stored pair, then the layer on the pair as it then stands
  UpdateDesc D{};
  D.B[0] = B_pair; D.tensor_base[0] = tensor_id; D.count = 1; D.n_slots = 1;
  D.elems_per_slot = (long long)r * k_out;
  launch_pair_update((cudaStream_t)cuda_stream, D, D.elems_per_slot, nullptr, g_prev, eps, lr, seed, 1);
  return mp_lora_linear_impl(cuda_stream, precision, X, W, bias, A, B_pair, B_pair + (size_t)r * k_out, Y, T, k_in,
                             k_out, r, scale, seed, tensor_id, 1, eps, x_replicated, scratch, scratch_bytes, flags);
}

}  // extern "C"

namespace {

// Previous update and (draw != 0) new perturbation applied to every stored pair of the model.
void enqueue_pair_update(zo_ctx* c, const zo_lora_pair* pair, uint64_t seed, const float* dev_g_prev, float eps,
                         float lr, int draw) {
  const zo_config& cf = c->cfg;
  const int r = cf.lora_rank;
  if (cf.arch == ZO_ARCH_LINEAR) {
    UpdateDesc D{};
    D.B[0] = pair->B_pair[0]; D.tensor_base[0] = 0; D.count = 1; D.n_slots = 1;
    D.elems_per_slot = (long long)r * cf.d_out;
    PROF(PC_UPDATE, 0.0, launch_pair_update(c->st, D, D.elems_per_slot, dev_g_prev, 0.f, eps, lr, seed, draw));
    return;
  }
  const int nt = c->nt;
  for (int l0 = 0; l0 < cf.n_layers && nt; l0 += UpdateDesc::MAX_T) {
    UpdateDesc D{};
    D.count = cf.n_layers - l0 < UpdateDesc::MAX_T ? cf.n_layers - l0 : UpdateDesc::MAX_T;
    D.n_slots = nt;
    D.elems_per_slot = (long long)r * cf.d_model;
    for (int i = 0; i < D.count; ++i) {
      D.B[i] = pair->B_pair[l0 + i];
      D.tensor_base[i] = (uint32_t)((l0 + i) * nt);
    }
    PROF(PC_UPDATE, 0.0, launch_pair_update(c->st, D, (long long)nt * D.elems_per_slot, dev_g_prev, 0.f, eps, lr,
                                            seed, draw));
  }
}

zo_status check_pair_args(zo_ctx* c, const zo_lora_pair* pair, float eps, float lr) {
  if (!c) return ZO_ERR_INVALID_ARG;
  if (!pair || !pair->A || !pair->B_pair) return fail(c, ZO_ERR_INVALID_ARG, "lora pair is NULL");
  if (!(eps > 0.f) || !isfinite(eps)) return fail(c, ZO_ERR_INVALID_ARG, "the stored-pair step needs eps > 0");
  if (!isfinite(lr)) return fail(c, ZO_ERR_INVALID_ARG, "lr must be finite");
  if (c->shard_count) return fail(c, ZO_ERR_STATE, "the stored-pair step has one query: switch query sharding off");
  const int n_b = c->cfg.arch == ZO_ARCH_LINEAR ? 1 : (c->nt ? c->cfg.n_layers : 0);
  for (int l = 0; l < n_b; ++l)
    if (!pair->B_pair[l]) return fail(c, ZO_ERR_INVALID_ARG, "null LoRA pair tensor");
  return ZO_OK;
}

}  // namespace

extern "C" {

zo_status zo_step_pair(zo_ctx* ctx, const zo_weights* weights, const zo_lora_pair* pair, const void* tokens,
                       const void* labels, int32_t E, int32_t S, uint64_t seed, const float* dev_g_prev,
                       float eps, float lr) {
  zo_status s = check_pair_args(ctx, pair, eps, lr);
  if (s) return s;
  const zo_lora view{pair->A, pair->B_pair};          // B[l] of the view = B[0] of the pair; B[1] follows it
  s = check_step_args(ctx, weights, &view, tokens, labels, E, S, 1, eps, lr);
  if (s) return s;
  s = begin_step(ctx, 1);
  if (s) return s;
  zo_ctx* c = ctx;
  enqueue_pair_update(c, pair, seed, dev_g_prev, eps, lr, 1);
  c->pair_mode = 1;
  if (c->cfg.arch == ZO_ARCH_LINEAR)
    s = step_linear(c, weights, &view, tokens, labels, E * S, seed, 1, eps, 0.f);
  else
    s = step_decoder(c, weights, &view, (const int32_t*)tokens, (const int32_t*)labels, E, S, seed, 1, eps, 0.f);
  c->pair_mode = 0;
  if (s) return s;
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(c, ZO_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  c->stepped = 1; c->last_q = 1; c->last_E = E; c->last_S = S;
  return ZO_OK;
}

zo_status zo_pair_collapse(zo_ctx* ctx, const zo_lora_pair* pair, const float* dev_g_prev, float eps, float lr) {
  const zo_status s = check_pair_args(ctx, pair, eps, lr);
  if (s) return s;
  zo_ctx* c = ctx;
  enqueue_pair_update(c, pair, 0, dev_g_prev, eps, lr, 0);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return fail(c, ZO_ERR_CUDA, "kernel launch: %s", cudaGetErrorString(e));
  return ZO_OK;
}

zo_status zo_g_buffer(zo_ctx* ctx, float** dev_g, int32_t* host_capacity) {
  if (!ctx) return ZO_ERR_INVALID_ARG;
  if (!dev_g) return fail(ctx, ZO_ERR_INVALID_ARG, "dev_g is NULL");
  *dev_g = ctx->at<float>(ctx->plan.g);
  if (host_capacity) *host_capacity = ctx->cfg.max_q;
  return ZO_OK;
}

}  // extern "C"
