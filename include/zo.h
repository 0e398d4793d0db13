/*
 * zo.h - C ABI of the parallelised zeroth-order (MobiZO-style) gradient estimator
 *        for NVIDIA B200 (sm_100a).
 *
 * One zo_step is one iteration of the paper's Algorithm 1 ("MobiZO Algorithm"):
 * the q queries (outer loop) and the +/- pair of each query (inner loop) are
 * folded into ONE forward pass over n = 2q replicas of the shared batch through
 * Multi-Perturbed LoRA layers ("MP-LoRA" paragraph: Y = X W + (X A) (.) B^(n), W and
 * A shared, only B perturbed per path), followed by the 2q losses, the q
 * projected gradients g_i = (l+ - l-) / (2 eps) and the ZO-SGD update
 * B <- B - lr * (1/q) * sum_i g_i z_i of the trainable LoRA B tensors.
 * The perturbations z_i are never stored: they are regenerated from the seed
 * wherever they are needed (seed trick, Background section).
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its name starts with `host_`.
 *     The structs zo_config, zo_weights, zo_lora and the pointer arrays inside
 *     them live in HOST memory and are read during the call only.
 *   - The library allocates no device memory: the caller passes a workspace of
 *     zo_workspace_bytes() bytes (256-byte aligned) that must stay valid until
 *     zo_free(), and owns every tensor and the CUDA stream.
 *   - Frozen tensors and activations are float32 (ZO_FP32) or bfloat16
 *     (ZO_BF16); the trainable B tensors are always float32 ("master copy").
 *   - Layouts are row-major.  Weights are stored [k_out, k_in] (the paper's W
 *     transposed), LoRA A as [r, k_in] (the paper's A transposed), LoRA B as
 *     [r, k_out].
 *   - Replica order: n = 2*i + 0 carries +eps*z_i, n = 2*i + 1 carries -eps*z_i
 *     (the B[0] / B[1] order of the paper's Algorithm 2).
 *   - Perturbation stream: Philox4x32-10, key = (seed low, seed high), counter =
 *     (e >> 2, tensor_id, i, 0), element e (row-major index in B) reads output
 *     word e & 3; word x -> u = ((x >> 9) + 0.5) * 2^-23; words (0,1) and (2,3)
 *     are Box-Muller pairs (sqrt(-2 ln u_a) * {cos, sin}(2 pi u_b)).
 *     tensor_id = layer * n_targets + slot, slots numbering the adapted
 *     sections (q, k, v) in ascending order; 0 for ZO_ARCH_LINEAR.
 *   - Every entry point returns a zo_status; nothing throws, aborts or traps.
 *     There is no CPU fallback: without a CUDA device the calls fail with
 *     ZO_ERR_CUDA.
 */
#ifndef ZO_H_
#define ZO_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ZO_API __attribute__((visibility("default")))
#else
#define ZO_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum zo_status {
  ZO_OK = 0,
  ZO_ERR_INVALID_ARG = 1, /* null pointer, size out of the configured range, bad enum      */
  ZO_ERR_UNSUPPORTED = 2, /* shape the kernels do not cover (see zo_init)                   */
  ZO_ERR_WORKSPACE = 3,   /* workspace too small or misaligned                              */
  ZO_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed (text in zo_last_error)    */
  ZO_ERR_TIMEOUT = 5,     /* a bounded device-side wait ran out; the step's results are void */
  ZO_ERR_NONFINITE = 6,   /* a loss came out NaN/Inf; B was left untouched                  */
  ZO_ERR_STATE = 7        /* call order (e.g. zo_losses before any zo_step)                 */
} zo_status;

enum { ZO_ARCH_LINEAR = 0, ZO_ARCH_OPT = 1, ZO_ARCH_LLAMA = 2 };
enum { ZO_FP32 = 0, ZO_BF16 = 1 };
enum { ZO_LOSS_MSE = 0, ZO_LOSS_CE_FULL_VOCAB = 1, ZO_LOSS_CE_LABEL_WORDS = 2 };
enum { ZO_TARGET_Q = 1, ZO_TARGET_K = 2, ZO_TARGET_V = 4 };
/* Storage of the four frozen linear weights of a decoder block (w_qkv, w_o, w_fc1, w_fc2), after the
 * paper's appendix "MobiZO with weight-only quantization" (Q-LoRA style): stored low-bit, dequantised
 * to the compute type once per forward pass, i.e. once per step for all 2q replicas (ZO_FLAG_DEQUANT_FUSED:
 * small bfloat16 launches decode inside the GEMM's operand producer instead).
 *   ZO_W_NATIVE  element type of `precision`
 *   ZO_W_INT8    int8 codes [k_out, k_in] + float32 scale [k_out]:      w = code * scale[row]
 *   ZO_W_NF4     4-bit NormalFloat codes, two per byte (even element in the high nibble), uint8
 *                [k_out, k_in/2] + float32 absmax [k_out, k_in/64]:     w = level[code] * absmax[row, col/64]
 * The dequantised value is rounded once to the compute type. */
enum { ZO_W_NATIVE = 0, ZO_W_INT8 = 1, ZO_W_NF4 = 2 };
/* flags: ZO_FLAG_SIMT_GEMM routes every bf16 GEMM (and attention) through the plain
 * CUDA-core validation kernels instead of the tensor-core ones (cross-checking only). */
enum { ZO_FLAG_SIMT_GEMM = 1,
       /* Tensor-core GEMM tile shape.  Default: CTA pairs (tcgen05 cta_group::2) on 256-row tiles for
        * launches that have at least eight waves of such tiles and at most 3 TFLOP, and either no
        * low-rank term or its one-block tensor-core form (projections and MLP at mid-size shapes:
        * each CTA stages half of the weight tile, which cuts the L2 traffic per flop by a third);
        * one CTA per 128-row tile for everything else (at the largest shapes the board sits at its
        * power limit and pairs only lower the clock).
        * ZO_FLAG_GEMM_PAIR: pairs wherever the kernel allows (the low-rank term then runs in the
        * epilogue unless rank <= 32 and a replica is a multiple of 256 rows).
        * ZO_FLAG_GEMM_SINGLE: never pairs.
        * A/B switches: the two tile shapes accumulate in the same order, so results are
        * bit-identical when the low-rank term takes the same form in both and no launch is split
        * along K. */
       ZO_FLAG_GEMM_PAIR = 2,
       ZO_FLAG_GEMM_SINGLE = 8,
       /* ZO_FLAG_LORA_EPILOGUE: the MP-LoRA term is always added on CUDA cores in the GEMM epilogue
        * from fp32 U and fp32 (B + k eps z), never as the extra tensor-core k-block (which rounds
        * U, B and k eps z to bfloat16).  A/B switch. */
       ZO_FLAG_LORA_EPILOGUE = 4,
       /* ZO_FLAG_DEQUANT_FUSED: bfloat16 GEMM launches of at most 256 rows decode quantised weights inside
        * the tensor-core kernel's operand producer (codes brought to shared memory by bulk tensor copies,
        * decoded by the epilogue warps straight into the MMA's operand stage; a weight is read once, as
        * codes, and nothing is written back) instead of decoding every weight into scratch before its GEMM.
        * Same bf16 operands, same accumulation order: both forms compute the same bits.  Off by default:
        * with eight decode warps per SM the in-kernel form is slower on B200 than decode-then-GEMM. */
       ZO_FLAG_DEQUANT_FUSED = 16,
       /* ZO_FLAG_ATTN_WARP_MMA: bfloat16 attention always runs the warp-level (mma.sync) kernel.  Default for
        * head_dim 64 / 128 and sequences of at most 256 tokens: the tcgen05 kernel (scores and P V on the
        * fifth-generation tensor cores with tensor-memory accumulators, q / k / v brought in by bulk tensor
        * copies).  A/B switch. */
       ZO_FLAG_ATTN_WARP_MMA = 64,
       /* ZO_FLAG_CE_LOGITS: the full-vocabulary loss stores float32 logits [2q*E*max_labelled, vocab] in the
        * workspace and reduces them in a second kernel.  Default in bfloat16 mode: the LM-head GEMM's epilogue
        * folds its tile of logits into (max, sum of exp) pairs and the logits never reach memory.  Checker /
        * A/B switch; the two forms differ in summation order only. */
       ZO_FLAG_CE_LOGITS = 32,
       /* ZO_FLAG_TEST_EXPIRE_WAIT (zo_mp_lora_linear only; contexts use zo_test_expire_wait): failure-
        * detection test aid, see zo_test_expire_wait. */
       ZO_FLAG_TEST_EXPIRE_WAIT = 1 << 24 };
/* Bits 8..15 of flags, when non-zero, override the tensor-core GEMM's raster group (128-row tiles that
 * sweep the weight panels together; default 16).  Tuning aid; results do not depend on it.
 * Bits 16..20, when non-zero, bound the number of K ranges the tensor-core GEMM cuts a tile into when a
 * launch has fewer tiles than SMs (small batches; 1 = never split).  Tuning aid; the sum order, and
 * with it the last bits of the result, depends on the number of ranges, not on the run. */

typedef struct zo_ctx zo_ctx; /* opaque; owned by the library; released by zo_free */

/* Model and limits; plain data, versioned by struct_size (= sizeof(zo_config)). */
typedef struct zo_config {
  uint32_t struct_size;
  int32_t arch;      /* ZO_ARCH_*                                                   */
  int32_t precision; /* ZO_FP32 | ZO_BF16                                           */
  int32_t loss_kind; /* ZO_LOSS_*; ZO_ARCH_LINEAR requires ZO_LOSS_MSE              */
  int32_t n_layers;  /* decoder blocks (1 for ZO_ARCH_LINEAR)                       */
  int32_t d_model;   /* hidden size; ZO_ARCH_LINEAR: k_in                           */
  int32_t d_out;     /* ZO_ARCH_LINEAR only: k_out                                  */
  int32_t n_heads;
  int32_t d_ffn;
  int32_t vocab;
  int32_t max_seq;      /* largest S; also rows of the learned position table (OPT) */
  int32_t lora_rank;    /* r, 1..64                                                  */
  float lora_scale;     /* multiplies the low-rank term; 1.0 = the layer equation as printed */
  uint32_t lora_targets; /* ZO_TARGET_* mask over the fused q|k|v projection          */
  int32_t label_words[2]; /* ZO_LOSS_CE_LABEL_WORDS: the two vocabulary rows          */
  int32_t max_q;        /* largest q (n = 2q replicas), <= 32                        */
  int32_t max_E;        /* largest number of sequences in the shared batch           */
  int32_t max_labelled; /* largest number of labelled positions per sequence         */
  float norm_eps;
  float rope_theta;
  int32_t tie_lm_head; /* 1: LM head = token embedding                               */
  uint32_t flags;
  int32_t weight_format; /* ZO_W_*; quantised formats need k_in % 64 == 0 (NF4) and decoders   */
  int32_t max_shard_q;   /* 0, or the largest number of queries this context runs in ONE step when it only
                          * ever runs query shards (zo_set_query_shard): the activation workspace is then
                          * sized for 2 * max_shard_q replicas instead of 2 * max_q, so a device's memory
                          * shrinks with the number of devices.  Steps with more queries are rejected. */
} zo_config;

/* Frozen tensors of one decoder block (device pointers; element type per precision).
 * OPT: LayerNorm gains+biases, biases on every linear, w_fc1 [d_ffn, d], ReLU.
 * Llama: RMSNorm gains only (bias pointers NULL), w_fc1 [2*d_ffn, d] = gate rows
 * followed by up rows, SiLU(gate)*up, rotate-half RoPE on q and k. */
typedef struct zo_layer_weights {
  const void* norm1_g; const void* norm1_b;
  const void* w_qkv;   const void* b_qkv;  /* [3d, d], [3d]: q rows, k rows, v rows */
  const void* w_o;     const void* b_o;    /* [d, d], [d]   */
  const void* norm2_g; const void* norm2_b;
  const void* w_fc1;   const void* b_fc1;
  const void* w_fc2;   const void* b_fc2;  /* [d, d_ffn], [d] */
  /* ZO_W_INT8 / ZO_W_NF4 only: float32 scales of the four weights above (else NULL) */
  const float* s_qkv; const float* s_o; const float* s_fc1; const float* s_fc2;
} zo_layer_weights;

typedef struct zo_weights {
  const void* tok_emb;      /* [vocab, d]                                            */
  const void* pos_emb;      /* [max_seq, d] learned positions (OPT) or NULL          */
  const void* lm_head;      /* [vocab, d]; ignored when tie_lm_head                  */
  const void* final_norm_g; const void* final_norm_b;
  const zo_layer_weights* layers; /* HOST array [n_layers]                           */
  const void* linear_w;     /* ZO_ARCH_LINEAR: W [d_out, d_model]                    */
  const void* linear_bias;  /* ZO_ARCH_LINEAR: [d_out] or NULL                       */
} zo_weights;

/* LoRA tensors: HOST arrays of n_layers device pointers.
 * A[l]: [n_targets * r, d_model] frozen (LoRA-FA), shared by all replicas.
 * B[l]: float32 [n_targets, r, k_out]; the master copy, UPDATED IN PLACE by zo_step. */
typedef struct zo_lora {
  const void* const* A;
  float* const* B;
} zo_lora;

/* Bytes of device workspace zo_init needs for this configuration (0 on a bad config). */
ZO_API size_t zo_workspace_bytes(const zo_config* cfg);

/* Set-up of the inputs Algorithm 1 lists before its loop (model, loss kind, bounds on q and the batch):
 * validates cfg, partitions the workspace, creates the context.  `cuda_stream` is a
 * cudaStream_t (NULL = legacy default stream) on which every later call enqueues.
 * Several devices in one process: call with the context's device current, here and in every later call
 * on the context; per-device set-up of the kernels is done on first use and host threads may call in
 * concurrently (one context is still one thread's at a time).
 * Unsupported (ZO_ERR_UNSUPPORTED): d_model % n_heads != 0; head_dim not in
 * {16, 32, 64, 128}; max_seq > 512; (r * k_out) % 4 != 0; ZO_BF16 with d_model, d_ffn or
 * d_out not a multiple of 8 (16-byte row pitch needed by the tensor-memory-accelerator loads). */
ZO_API zo_status zo_init(const zo_config* cfg, void* workspace, size_t workspace_bytes,
                  void* cuda_stream, zo_ctx** out);

/* One step of Algorithm 1 on the shared batch.  Asynchronous: enqueues kernels on
 * the context's stream and returns; never synchronises.
 *   tokens : int32 [E, S] token ids        (ZO_ARCH_LINEAR: X [E*S, d_model], element type per precision)
 *   labels : int32 [E, S]; <0 = position not in the loss.  ZO_LOSS_CE_FULL_VOCAB: the
 *            vocabulary id to predict at that position.  ZO_LOSS_CE_LABEL_WORDS: class id
 *            0/1 (index into label_words).  At most max_labelled entries >= 0 per sequence.
 *            (ZO_ARCH_LINEAR: float32 targets [E*S, d_out].)
 *   seed, q, eps, lr : Algorithm 1's s (s_i = (seed, i)), q, epsilon, eta.
 *   eps == 0  : losses only; g = 0 and B untouched.
 *   lr  == 0  : losses and g; B untouched (times the perturbed forward alone).
 * Errors: ZO_ERR_INVALID_ARG for null pointers, q < 1, q > max_q, E < 1, E > max_E,
 * S < 1, S > max_seq, eps < 0 or non-finite scalars.  Device-side problems
 * (ZO_ERR_TIMEOUT, ZO_ERR_NONFINITE, too many labelled positions = ZO_ERR_INVALID_ARG)
 * are reported by the next zo_losses. */
ZO_API zo_status zo_step(zo_ctx* ctx, const zo_weights* weights, const zo_lora* lora,
                  const void* tokens, const void* labels, int32_t E, int32_t S,
                  uint64_t seed, int32_t q, float eps, float lr);

/* The same step on a PACKED variable-length batch (no padding rows at all: the paper's second
 * argument for small E is less padding; here there is none).  Decoders only.
 *   tokens, labels : int32 [total_tokens], the E sequences back to back
 *   cu_seqlens     : int32 [E + 1] device array, cu[0] = 0, cu[b+1] - cu[b] = length of sequence b
 *                    (1 .. max_len), cu[E] = total_tokens
 *   max_len        : upper bound of the lengths, <= max_seq; total_tokens <= max_E * max_seq
 * Positions (learned or rotary) restart at 0 in every sequence; attention is causal inside a
 * sequence; labels as in zo_step.  A malformed cu_seqlens is reported by zo_losses as
 * ZO_ERR_INVALID_ARG. */
ZO_API zo_status zo_step_varlen(zo_ctx* ctx, const zo_weights* weights, const zo_lora* lora,
                                const int32_t* tokens, const int32_t* labels, const int32_t* cu_seqlens,
                                int32_t E, int32_t total_tokens, int32_t max_len, uint64_t seed,
                                int32_t q, float eps, float lr);

/* Same step with tokens and labels in HOST memory (pinned or pageable): they are
 * copied to the device on the context's stream first.  The host buffers must stay
 * untouched until the stream has passed the copy (e.g. until zo_losses returns). */
ZO_API zo_status zo_step_host(zo_ctx* ctx, const zo_weights* weights, const zo_lora* lora,
                       const void* host_tokens, const void* host_labels, int32_t E, int32_t S,
                       uint64_t seed, int32_t q, float eps, float lr);

/* The outputs of Algorithm 1's inner and outer loops: synchronises the stream and copies out the last
 * step's 2q losses l^(k) of the perturbed parameters theta_l + k eps z_i (replica order n = 2i + {0: +,
 * 1: -}) and, if host_g != NULL, its q projected gradients g_i = (l^(+1) - l^(-1)) / (2 eps), the
 * scalars Algorithm 1 stores next to the seeds.  Returns the step's deferred status. */
ZO_API zo_status zo_losses(zo_ctx* ctx, float* host_losses, float* host_g);

/* Diagnostics: per labelled-row losses of the last step, [2q][rows] with rows in
 * (sequence, labelled slot) order, max_labelled slots per sequence (unused slots are 0);
 * *host_n_rows receives rows per replica.  host_rows may be NULL to query the count.
 * ZO_ARCH_LINEAR: one value per token row (mean over k_out).  Synchronises the stream. */
ZO_API zo_status zo_row_losses(zo_ctx* ctx, float* host_rows, int32_t* host_n_rows);

/* How a step is cut into forward passes (the paper's ablation of its two parallelisations; only the
 * cost of a step depends on it.  Results are bit-identical across schedules as long as no GEMM of the
 * pass is small enough to be split along K, i.e. has at most 256 rows and at most a third as many
 * 128x256 tiles as the device has SMs; a split launch sums its K ranges in a fixed order that depends on the number of
 * ranges, so there the schedules agree to fp32 summation order.  Every pass of one step has the same
 * shape, so the + and - losses of a query always see the same summation order.  flags bits 16..20 = 1
 * switch the split off):
 *   ZO_SCHEDULE_FULL        one pass over all 2q replicas (outer and inner loop in parallel; default)
 *   ZO_SCHEDULE_OUTER_ONLY  two passes of q replicas: every +eps path, then every -eps path
 *   ZO_SCHEDULE_INNER_ONLY  q passes of 2 replicas: the +/- pair of one query at a time
 *   ZO_SCHEDULE_SEQUENTIAL  2q passes of one replica: the order of forward passes of sequential
 *                           MeZO with LoRA-FA (appendix "MeZO with q>1"), without its in-place
 *                           parameter sweeps since the perturbed copy is formed on the fly. */
enum { ZO_SCHEDULE_FULL = 0, ZO_SCHEDULE_OUTER_ONLY = 1, ZO_SCHEDULE_INNER_ONLY = 2,
       ZO_SCHEDULE_SEQUENTIAL = 3 };
ZO_API zo_status zo_set_schedule(zo_ctx* ctx, int32_t schedule);

/* Replica sharding over several devices.  The 2q replicas of a step are independent forward passes
 * (Algorithm 1: every query i has its own seed s_i and its own pair of losses), so a step can be
 * spread over devices that each hold the frozen weights and a copy of the trainable B tensors:
 * device k runs the queries [q_begin, q_begin + q_count) of the step, the devices exchange the 2q
 * loss scalars, and every device regenerates all z_i and applies the same update to its copy of B.
 * No parameter or activation ever crosses between devices.
 *
 *   zo_set_query_shard(ctx, q_begin, q_count)
 *       From now on zo_step / zo_step_host / zo_step_varlen run only the replicas 2*q_begin ..
 *       2*(q_begin + q_count) - 1 of the q-query step they are given (same seed, same replica
 *       numbering, so the perturbations are those of the whole step), write their losses at those
 *       positions of the loss array, zero the other positions and stop there: no g, no update
 *       (lr is ignored).  q_begin + q_count must not exceed the step's q (ZO_ERR_INVALID_ARG
 *       from the step otherwise).  q_count = 0 (with q_begin = 0) switches sharding off.  The
 *       schedule set by zo_set_schedule applies inside the shard.
 *   zo_loss_buffer(ctx, &dev_losses, &capacity)
 *       Device address of the step's float64 loss array (inside the caller's workspace):
 *       `capacity` = 2*max_q + 1 entries, the losses in replica order followed by one fault slot.
 *       After a sharded step it holds this shard's losses, zeros at every other loss, and in the
 *       fault slot 1.0 if this device's status word is set (bounded wait ran out, bad token or
 *       label, non-finite loss), else 0.0.  A sum over devices of the WHOLE array (one all-reduce
 *       of 2*max_q + 1 doubles; exact, since every loss has one non-zero contributor) completes
 *       the losses and tells every device whether any device faulted.  The exchange itself is the
 *       caller's: enqueue it on the context's stream, or order it with the stream by events.
 *   zo_apply_update(ctx, lora, seed, q, eps, lr)
 *       g_i = (l_{2i} - l_{2i+1}) / (2 eps) from the loss array as it then stands, and
 *       B <- B - lr (1/q) sum_i g_i z_i on this device's B.  Asynchronous on the context's stream.
 *       A non-finite loss from any device, or a non-zero fault slot, leaves B untouched on every
 *       device (all see the same array), so the copies of B cannot drift apart; zo_losses
 *       afterwards returns all 2q losses and g and the deferred status: the device's own fault if
 *       it had one, ZO_ERR_STATE when only another device did.
 *       Also valid after an unsharded step with lr = 0 (apply the step later).
 * If only the 2q losses are exchanged (fault slot left out), a device-side fault on ONE device skips
 * that device's update only: check zo_losses on every device before the next step.  zo_row_losses
 * after a sharded step holds this shard's rows only. */
ZO_API zo_status zo_set_query_shard(zo_ctx* ctx, int32_t q_begin, int32_t q_count);
ZO_API zo_status zo_loss_buffer(zo_ctx* ctx, double** dev_losses, int32_t* host_capacity);
ZO_API zo_status zo_apply_update(zo_ctx* ctx, const zo_lora* lora, uint64_t seed, int32_t q,
                                 float eps, float lr);

/* ---------------------------------------------------------------------------------------------------
 * The step in the form of the paper's Algorithm 2 ("Mobile MP-LoRA Module", q = 1).
 *
 * Algorithm 2 keeps, per trainable tensor, the two perturbed copies B[0] = B + eps z and B[1] = B - eps z
 * in memory instead of the master copy, takes the projected gradient g of the PREVIOUS step as an input
 * of the forward pass, and does inside that pass:
 *     diff = (B[0] - B[1]) / 2;  update = eta g diff / eps;  z = eps randn_like(B[0]);
 *     B[0] = B[0] - diff - update + z;  B[1] = B[1] + diff - update - z;
 *     output = x W + bmm(x A, B)
 * so that nothing but forward passes ever runs: the previous update and the new perturbation ride in
 * the forward pass, and no host round trip separates two steps.
 *
 *   zo_lora_pair.B_pair[l] : float32 [2, n_targets, r, k_out] of layer l, B[0] then B[1]; UPDATED IN
 *       PLACE by every zo_step_pair.  Before the first step both halves hold the same B (diff = 0).
 *   zo_step_pair(ctx, weights, pair, tokens, labels, E, S, seed, dev_g_prev, eps, lr)
 *       One step: applies the lines above to every pair of the model (z = eps * the normals of
 *       (seed, tensor, query 0), the stream of zo_step), runs the forward pass of the two replicas on
 *       the stored pair, and leaves the two losses and g = (l0 - l1) / (2 eps) on the device.
 *       dev_g_prev: DEVICE pointer to the previous step's g (the buffer zo_g_buffer returns, which
 *       this call overwrites at its end, or any device float), or NULL for g = 0 (first step).
 *       Asynchronous; steps can be enqueued back to back without reading anything back.  A step that
 *       faults on the device (status word set) leaves g = 0, so the next step's update is a no-op.
 *       eps must be > 0.  zo_losses returns the two losses and g as after zo_step with q = 1.
 *       The mean (B[0] + B[1]) / 2 after the call is the master copy BEFORE this step's own update
 *       (which the next call applies): it equals the B that zo_step would hold at the same point.
 *   zo_pair_collapse(ctx, pair, dev_g_prev, eps, lr)
 *       Applies the pending update without a new perturbation: B[0] = B[1] = the updated master copy
 *       (to finish a run, or to hand the tensors to zo_step).
 *   zo_g_buffer(ctx, &dev_g, &capacity)
 *       Device address of the context's projected gradients (float32 [max_q]; entry 0 after a pair step).
 *   zo_mp_lora_linear_pair(...)
 *       The module of Algorithm 2 on its own: the lines above on one stored pair (g_prev by value),
 *       then Y[n] = X[n or shared] W^T + bias + scale (X A^T) B[n], n = 0, 1.  Arguments as
 *       zo_mp_lora_linear with q = 1; B_pair is float32 [2, r, k_out], updated in place. */
typedef struct zo_lora_pair {
  const void* const* A;      /* HOST array [n_layers] of device pointers, as zo_lora.A */
  float* const* B_pair;      /* HOST array [n_layers] of device pointers to [2, n_targets, r, k_out] */
} zo_lora_pair;
ZO_API zo_status zo_step_pair(zo_ctx* ctx, const zo_weights* weights, const zo_lora_pair* pair,
                              const void* tokens, const void* labels, int32_t E, int32_t S, uint64_t seed,
                              const float* dev_g_prev, float eps, float lr);
ZO_API zo_status zo_pair_collapse(zo_ctx* ctx, const zo_lora_pair* pair, const float* dev_g_prev, float eps,
                                  float lr);
ZO_API zo_status zo_g_buffer(zo_ctx* ctx, float** dev_g, int32_t* host_capacity);
ZO_API zo_status zo_mp_lora_linear_pair(void* cuda_stream, int32_t precision, const void* X, const void* W,
                                        const void* bias, const void* A, float* B_pair, void* Y, int32_t T,
                                        int32_t k_in, int32_t k_out, int32_t r, float scale, uint64_t seed,
                                        uint32_t tensor_id, float g_prev, float eps, float lr,
                                        int32_t x_replicated, void* scratch, size_t scratch_bytes,
                                        uint32_t flags);

/* Failure-detection test aid; off (0) by default and in every measured run.  Every device-side wait of
 * the tensor-core GEMM (on a shared-memory barrier that a copy or a tensor-core instruction completes) is
 * bounded: when it runs out, the thread block raises the time-out bit of the status word, lets the copies
 * and tensor-core instructions it has issued finish, frees its tensor memory and returns, and zo_losses
 * reports ZO_ERR_TIMEOUT with B untouched.  Nothing in a correct run makes a wait run out, so this call
 * arranges it without faulting anything: while wait_limit_ns > 0, every tensor-core GEMM launch of the
 * context runs one thread block per tile, gives up its waits after wait_limit_ns (<= 2e9), and the copy
 * engine of thread block 0 goes silent after its first k-block (nothing armed, nothing in flight), so
 * that block's tensor-core warp waits for a stage that never arrives.  wait_limit_ns = 0 restores
 * normal operation; the context, the stream and the device stay usable throughout. */
ZO_API zo_status zo_test_expire_wait(zo_ctx* ctx, uint64_t wait_limit_ns);

/* Number of kernels the last zo_step enqueued. */
ZO_API int32_t zo_launch_count(const zo_ctx* ctx);

/* Profiling aid.  While enabled, every kernel launch of zo_step is bracketed by CUDA events
 * on the context's stream.  zo_profile_read synchronises the stream and returns, per kernel
 * class, the summed device time in ms, the summed algorithmic work and the number of launches
 * since the previous read.  Work is flops 2*M*N*K for the GEMM classes and LORA_DOWN, and bytes that
 * must cross HBM (inputs read once, outputs written once) for ATTENTION, NORM, LORA_APPLY and ROPE;
 * 0 for the rest.  Arrays of ZO_PROFILE_CLASSES.
 * Decoder GEMMs are booked under their own classes (QKV, O, FC1, FC2, HEAD); ZO_PROF_GEMM_TC
 * holds the tensor-core GEMMs of ZO_ARCH_LINEAR. */
enum { ZO_PROF_GEMM_TC = 0, ZO_PROF_GEMM_SIMT, ZO_PROF_ATTENTION, ZO_PROF_NORM, ZO_PROF_LORA_DOWN,
       ZO_PROF_LORA_APPLY, ZO_PROF_ROPE, ZO_PROF_SWIGLU, ZO_PROF_LOSS, ZO_PROF_UPDATE,
       ZO_PROF_MISC, ZO_PROF_GEMM_QKV, ZO_PROF_GEMM_O, ZO_PROF_GEMM_FC1, ZO_PROF_GEMM_FC2,
       ZO_PROF_GEMM_HEAD, ZO_PROF_DEQUANT, ZO_PROFILE_CLASSES };
ZO_API zo_status zo_profile_enable(zo_ctx* ctx, int32_t on);
ZO_API zo_status zo_profile_read(zo_ctx* ctx, double* host_ms, double* host_flops,
                                 int32_t* host_launches);

ZO_API void zo_free(zo_ctx* ctx);
ZO_API const char* zo_last_error(const zo_ctx* ctx); /* ctx may be NULL: last zo_init failure of the calling thread */

/* The perturbation stream itself (Algorithm 1: z_i from s_i), for bit-level checks:
 * writes the first n raw 32-bit words (dev_u32, may be NULL) and normals (dev_z, may be
 * NULL) of tensor `tensor_id`, query `query`.  Asynchronous on `cuda_stream`. */
ZO_API zo_status zo_perturbation(void* cuda_stream, uint64_t seed, uint32_t tensor_id, uint32_t query,
                          int64_t n, uint32_t* dev_u32, float* dev_z);

/* The weight decoder on its own (for bit-level checks): out [rows, k_in] in the element type of
 * `precision` from codes and scales in the given ZO_W_INT8 / ZO_W_NF4 format.  Asynchronous. */
ZO_API zo_status zo_dequantize(void* cuda_stream, int32_t weight_format, int32_t precision,
                               const void* codes, const float* scale, void* out, int32_t rows,
                               int32_t k_in);

/* The MP-LoRA linear on its own ("MP-LoRA" paragraph, layer equation):
 *   Y[n] = X[n or shared] W^T + bias + scale * (X A^T) (B + k_n eps z_{n>>1}),  n < 2q.
 * x_replicated = 0: X is [T, k_in], the base product is computed once and expanded to the
 * 2q outputs (first perturbed layer of a model); 1: X is [2q*T, k_in] (every later layer).
 * Y is [2q, T, k_out].  `precision` selects float32 or bfloat16 for X, W, bias, A and Y.
 * `scratch` needs zo_mp_lora_scratch_bytes() bytes (256-byte aligned).  bfloat16 requires
 * k_in % 8 == 0, k_out % 8 == 0 and, for replicated input, T % 128 == 0.
 * Asynchronous on `cuda_stream`. */
ZO_API size_t zo_mp_lora_scratch_bytes(int32_t precision, int32_t T, int32_t k_in, int32_t k_out,
                                int32_t r, int32_t q, int32_t x_replicated);
ZO_API zo_status zo_mp_lora_linear(void* cuda_stream, int32_t precision, const void* X, const void* W,
                            const void* bias, const void* A, const float* B, void* Y,
                            int32_t T, int32_t k_in, int32_t k_out, int32_t r, float scale,
                            uint64_t seed, uint32_t tensor_id, int32_t q, float eps,
                            int32_t x_replicated, void* scratch, size_t scratch_bytes,
                            uint32_t flags);

/* zo_mp_lora_linear without any caller-provided scratch (the paper has no counterpart: this is
 * a packaging variant of the entry point above, same arithmetic, same results).
 *
 * For callers that cannot allocate device memory where they need the layer: code hosted inside
 * a framework whose allocator owns the device budget, plug-ins that receive only their input and
 * output buffers, and loops where an allocation would stall the device.  The scratch lives in a
 * fixed array of ZO_STATIC_SCRATCH_BYTES inside the library's device image; every GPU that loads
 * the library holds those bytes until the process exits.  The call allocates nothing (no
 * cudaMalloc, cudaFree or allocating library routine); X, W, bias, A, B and Y are still the
 * caller's buffers.
 *   - Problems whose zo_mp_lora_scratch_bytes() exceeds ZO_STATIC_SCRATCH_BYTES are rejected
 *     with ZO_ERR_WORKSPACE; nothing is launched.
 *   - The first call on each device looks up the array's device address (a host-side step);
 *     make that first call before starting any stream capture on that device.
 *   - All calls on a device share the one array, which keeps the previous call's contents; what
 *     must start at zero is cleared by every call.  Two calls that overlap on the GPU (different
 *     streams, no ordering between them) race on it: order them, or use zo_mp_lora_linear with
 *     separate scratch buffers. */
#define ZO_STATIC_SCRATCH_BYTES (16u << 20)
ZO_API zo_status zo_mp_lora_linear_static(void* cuda_stream, int32_t precision, const void* X,
                                          const void* W, const void* bias, const void* A,
                                          const float* B, void* Y, int32_t T, int32_t k_in,
                                          int32_t k_out, int32_t r, float scale, uint64_t seed,
                                          uint32_t tensor_id, int32_t q, float eps,
                                          int32_t x_replicated, uint32_t flags);
/* Deferred device-side status of the calls made so far through zo_mp_lora_linear_static on the
 * current device: the call itself only enqueues work, and its status word lives inside the fixed
 * array, out of the caller's reach.  Copies that word to *host_status on `cuda_stream` (use the
 * stream of the call) and waits for the stream; allocates nothing.  Returns ZO_ERR_TIMEOUT when a
 * bounded device-side wait ran out (Y is then void), ZO_OK otherwise.  The word is cleared by the
 * next zo_mp_lora_linear_static call. */
ZO_API zo_status zo_mp_lora_linear_static_status(void* cuda_stream, uint32_t* host_status);

#ifdef __cplusplus
}
#endif
#endif /* ZO_H_ */
