// Host-side launchers of the CUDA kernels (internal to the library).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace zo {

// Where the per-replica low-rank term s * U (B + k eps z) comes from.
struct LoraDesc {
  const float* U;        // [rows, ldu] fp32 down-projections X A^T, row-indexed like the X operand
  int ldu;
  const float* B;        // [n_slots, r, width] fp32 master copy of this layer (stored pair: B[0] = B + eps z)
  const float* B1;       // null, or the second tensor of a stored pair (B[1] = B - eps z): replica n then uses
                         // the stored B[n & 1] and nothing is regenerated (Algorithm 2, q = 1)
  int r;
  int width;             // k_out of one section
  int slot_of_sec[3];    // output columns [j*width, (j+1)*width) -> slot, or -1 (not adapted)
  float scale, eps;
  uint64_t seed;
  uint32_t tensor_base;  // tensor_id of slot 0
  int rows_per_replica;  // rows of one replica in the (padded) activation layout
  int rep_base, rep_stride;  // replica id of the j-th replica in the buffers = rep_base + rep_stride * j
};

enum { ACT_NONE = 0, ACT_RELU = 1 };

// How the T token rows of one replica split into sequences.  Fixed length: E sequences of S rows
// (cu = pos = null).  Packed variable length: sequence b is rows cu[b] .. cu[b+1]-1, S is the longest
// allowed length, pos[t] the position of packed row t inside its sequence.
struct SeqLayout {
  int E, S;
  const int32_t* cu;
  const int32_t* pos;
  int T;   // token rows of one replica (bounds every cu-derived index)
  // first row and length of sequence b, clamped so that a malformed cu cannot index outside the batch
  __host__ __device__ int start(int b) const {
    if (!cu) return b * S;
    const int s0 = cu[b];
    return s0 < 0 ? 0 : (s0 > T ? T : s0);
  }
  __host__ __device__ int len(int b) const {
    if (!cu) return S;
    const int s0 = start(b);
    int l = cu[b + 1] - s0;
    if (l > S) l = S;
    if (l > T - s0) l = T - s0;
    return l < 0 ? 0 : l;
  }
};

struct GemmDesc {
  const void* A; int lda;       // [M, K] activations
  const void* W;                // [N, K] weights (K contiguous)
  int M, N, K;
  void* out; int ldo;           // [M, N]  (swiglu: [M, N/2])
  int out_f32;                  // 1: float output regardless of the operand type
  const void* bias;             // [N] or null
  const void* res; int ldr;     // residual rows (row % res_mod when res_mod > 0) or null
  int res_mod;
  int act;
  int swiglu;                   // 1: W = [gate rows | up rows] (N = 2 * d_ffn), out = silu(g)*u
  const LoraDesc* lora;         // null: plain GEMM
  int lora_slab;                // 1: the LoRA term runs as an extra tensor-core k-block fed from pack_u
  const void* pack_u;           // bf16 [M, pack_ld]: per slot [U | U] in kslot columns (second copy at khalf)
  void* pack_out;               // down-projection: write that packed copy here (bf16 [M, pack_ld]) or null
  int pack_ld, pack_r, kslot, khalf;
  const float* rope_tab;        // tensor-core kernel: rotate columns < rope_cols (q, k) in the epilogue; table
                                // rows cos[0..dh/2) | sin[0..dh/2); position of row m = (m % rope_tp) % rope_s
  int rope_cols, rope_dh, rope_s, rope_tp;
  const int32_t* rope_pos;      // packed variable-length rows: position of row (m % rope_tp), else null
  int group_m;                  // 128-row tiles per raster group of the tensor-core kernel (0 = default 16)
  int prof_class;               // profiling class of this launch (0: generic tensor-core GEMM)
  int cta_pair;                 // CTA pairs (cta_group::2) on 256-row tiles: 0 never, 1 wherever possible, 2 where measured faster (large launches without a low-rank term)
  float* split_ws;              // split-K scratch of the tensor-core kernel: split_units * 32768 floats, or null
  int split_units;
  int* extra_launches;          // incremented when the GEMM took a second launch (split K), or null
  int split_cap;                // > 0: upper bound on the number of K ranges per tile (1 = never split)
  void* ce_part;                // tensor-core kernel, cross-entropy head: non-null = store no output; per (row, 256-column tile,
                                // sibling warp) one float2 (max, sum of exp(logit - max)) into ce_part [M][ceil(N/256)][2] ...
  float* ce_logit;              // ... and the label's logit of every row whose label is >= 0 into ce_logit [M]
  const int32_t* ce_label;      // label of row m = ce_label[m % ce_ep]
  int ce_ep;
  int wfmt;                     // tensor-core kernel: 0 = W holds bf16 weights; 1 / 2 = W is unused and the B operand is decoded
  const void* wq;               // inside the kernel from int8 / NF4 codes [N, K] / [N, K/2] ...
  const float* wscale;          // ... and their float32 scales [N] / [N, K/64] (K % 64 == 0; at most 256 rows M)
  unsigned long long test_wait_ns;  // failure-detection tests only; > 0: the launch runs single-CTA, its bounded waits give
                                // up after this many ns, and CTA 0 withholds one k-block so that a wait does run out
};

// --- elementwise / reduction kernels (bf = 1: bfloat16 tensors, 0: float) -------------------
void launch_embed(cudaStream_t st, int bf, const int32_t* tokens, const void* tok_emb,
                  const void* pos_emb, void* out, int T, int Tp, SeqLayout sl, int d, int vocab,
                  uint32_t* status);
// Row norm. kind 0 = LayerNorm (gain, bias), 1 = RMSNorm (gain).  When lab_idx != null the
// source row of output row (n, j) with j < EP is n*Tp + lab_idx[j] (negative: zero row).
void launch_norm(cudaStream_t st, int bf, int kind, const void* x, void* out, const void* g,
                 const void* b, int rows, int d, float eps, const int32_t* lab_idx, int EP,
                 int Tp);
void launch_lora_down(cudaStream_t st, int bf, const void* X, int ldx, const void* A, float* U,
                      int rows, int K, int J);
void launch_lora_apply(cudaStream_t st, int bf, const void* base, int ldb, int base_shared,
                       void* out, int ldo, int n, int T, const LoraDesc& L, int nsec);
// Shared-input expansion on the bf16 path: out[j, t, :] = base[t, :] + s U[t, :] (B + k eps z) for the n
// replicas of a pass (base and U on the T shared rows; out rows j * rows_per_replica + t), written with
// full-line stores.  Supported when every section is a multiple of 128 columns, r <= 64 and rows are
// 16-byte aligned.  Rank <= 16 moves its tiles with bulk tensor copies, whose bounded waits report to
// the device status word.
bool lora_expand_supported(const void* base, int ldb, const void* out, int ldo, const LoraDesc& L);
void launch_lora_expand(cudaStream_t st, const void* base, int ldb, void* out, int ldo, int n, int T,
                        const LoraDesc& L, int nsec, int n_sms, uint32_t* status);
void launch_rope_table(cudaStream_t st, float* tab, int max_seq, int dh, float theta);
void launch_rope(cudaStream_t st, int bf, void* qkv, int rows, int Tp, SeqLayout sl, int d, int H,
                 const float* tab);
void launch_attention_simt(cudaStream_t st, int bf, const void* qkv, void* ctx, int n, SeqLayout sl,
                           int Tp, int d, int H);
// Tensor-core causal attention for bf16 with head_dim 64 or 128 (q, k already rotated).
bool attention_mma_supported(int dh);
void launch_attention_mma(cudaStream_t st, const void* qkv, void* ctx, int n, SeqLayout sl, int Tp,
                          int d, int H);
// Causal attention on tcgen05 tensor cores (bf16, head_dim 64 or 128, sequences of at most 256 tokens).
// Returns a CUDA error code (0 = ok).
bool attention_tc_supported(int dh, int max_len);
int launch_attention_tc(cudaStream_t st, const void* qkv, void* ctx, int n, SeqLayout sl, int Tp, int d, int H,
                        uint32_t* status, int n_sms);
void launch_swiglu(cudaStream_t st, int bf, const void* gu, void* out, int rows, int ffn);
// Positions of packed rows: pos[t] = t - cu[b] for the sequence b that holds row t (0 for pad rows);
// flags sequences longer than max_len or a non-monotone cu.
void launch_varlen_index(cudaStream_t st, const int32_t* cu, int E, int T, int Tp, int max_len, int32_t* pos,
                         uint32_t* status);
void launch_label_scan(cudaStream_t st, const int32_t* labels, SeqLayout sl, int P, int n_classes,
                       int32_t* lab_idx, int32_t* lab_val, int32_t* lab_cnt, uint32_t* status);
void launch_ce_rows(cudaStream_t st, const float* logits, int ldl, int V, const int32_t* lab_val,
                    int EP, int rows, double* row_loss);
// Row losses from the partial (max, sum) pairs the cross-entropy head GEMM left: pairs merged in a fixed
// order in fp64, loss = max + log(sum) - label logit (0 for rows whose label is < 0).
void launch_ce_merge(cudaStream_t st, const void* ce_part, int parts_per_row, const float* ce_logit,
                     const int32_t* lab_val, int EP, int rows, double* row_loss);
void launch_label_word_rows(cudaStream_t st, int bf, const void* xh, const void* head, int d,
                            int w0, int w1, const int32_t* lab_val, int EP, int rows,
                            double* row_loss);
void launch_mse_rows(cudaStream_t st, int bf, const void* Y, const float* target, int n, int T,
                     int Tp, int k_out, double* row_loss);
// losses[n] = mean of the valid rows of replica n (fixed order, fp64 accumulation); the fp64
// copy feeds the projected gradients, whose loss difference would drown in fp32 rounding.
// The j-th replica of the pass is replica rep_base + rep_stride * j of the step: its mean goes to
// losses[that id] and its rows are copied to rows_out[that id] (the per-step row-loss table).
void launch_replica_mean(cudaStream_t st, const double* row_loss, const int32_t* lab_val, int n,
                         int rows_per_replica, int rep_base, int rep_stride, double* rows_out,
                         float* losses, double* losses_d, uint32_t* status);

struct UpdateDesc {
  enum { MAX_T = 96 };
  float* B[MAX_T];       // tensors updated by this launch (one per layer)
  uint32_t tensor_base[MAX_T];
  int count;
  int n_slots;
  long long elems_per_slot;  // r * width
};
// g_i = (l_{2i} - l_{2i+1}) / (2 eps); B <- B - (lr/q) sum_i g_i z_i  (skipped if *status != 0
// or lr == 0).  With write_g, block 0 also stores g[0..q).
void launch_zo_update(cudaStream_t st, const UpdateDesc& D, const double* losses, float* g, int q,
                      float eps, float lr, uint64_t seed, const uint32_t* status, int write_g);
// After the exchange of a sharded step: fp32 copy of the completed loss array, finiteness check, and the
// fault slot (sum over devices of 0/1 flags) folded into the local status word.
// Stored-pair form (Algorithm 2): D.B[i] points at B[0] of tensor group i, B[1] lies pair_stride floats
// further.  Applies the previous step's update (g from g_dev if non-null, else g_val) and, with draw != 0,
// the new perturbation eps z of query 0 to both tensors.
void launch_pair_update(cudaStream_t st, const UpdateDesc& D, long long pair_stride, const float* g_dev,
                        float g_val, float eps, float lr, uint64_t seed, int draw);
// g[0] = (losses[0] - losses[1]) / (2 eps), or 0 when the status word is set.
void launch_pair_g(cudaStream_t st, const double* losses, float* g, float eps, const uint32_t* status);
void launch_losses_refresh(cudaStream_t st, const double* losses_d, float* losses, int n,
                           const double* fault_slot, uint32_t* status);
// End of a sharded step: *fault_slot = 1.0 when this device's status word is non-zero, else 0.0.
void launch_fault_publish(cudaStream_t st, const uint32_t* status, double* fault_slot);
void launch_perturbation(cudaStream_t st, uint64_t seed, uint32_t tensor, uint32_t query,
                         long long n, uint32_t* u32, float* z);

// Weight-only dequantisation (fmt 1 = int8 per-row scale, 2 = NF4 with 64-element blocks) to T.
void launch_dequant(cudaStream_t st, int bf, int fmt, const void* codes, const float* scale, void* out,
                    int rows, int K);

// --- GEMMs ---------------------------------------------------------------------------------
void launch_gemm_simt(cudaStream_t st, int bf, const GemmDesc& G);
// bf16 tensor-core GEMM (tcgen05 + TMEM + TMA).  Returns a CUDA error code (0 = ok).
int launch_gemm_tc(cudaStream_t st, const GemmDesc& G, uint32_t* status, int n_sms);
int gemm_tc_init();  // resolves the driver entry point for tensor-map encoding; 0 = ok

}  // namespace zo
