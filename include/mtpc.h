/*
 * mtpc.h - C ABI of the B200 (sm_100a) MtPC head: the probabilistic-circuit multi-byte prediction head of
 * "MtPC" (arXiv 2511.11346).
 *
 * For every context position the head maps the LLM hidden state h (the paper's e_t) to a circuit over the
 * next n bytes (Sec. 3.3: phi = softmax(W_ij e_t) for the input units, omega = softmax(R_i e_t) for the sum
 * units) and then either
 *   - evaluates the exact joint log-likelihood of n observed bytes (Eq. 1 through Eq. CP / HMM / BTree), or
 *   - draws n-byte draft windows by ancestral sampling (App. B.2, Algorithm 1) and returns their joint
 *     log-probability (the quantity Algorithm 3 needs for verification).
 *
 * Conventions
 *   - All indices are 0-based. Window slot i in [0,n), unit k in [0,r), byte b in [0,v).
 *   - "dev" = device (HBM) pointer, "host" = host pointer. Every device buffer is allocated and owned by the
 *     caller and must stay valid until the work that uses it has finished on the stream. The library
 *     allocates no device memory: all scratch lives in the caller's workspace.
 *   - Calls enqueue work on the given CUDA stream (a cudaStream_t passed as void*) and return without
 *     waiting, except where stated. A head must not be used from two streams at once: its workspace is shared.
 *     mtpc_window_logprob, mtpc_window_prefix_logprob, the two draft calls and mtpc_speculative_accept do nothing
 *     else (no synchronisation, no allocation, nothing read back), so they may be recorded into a CUDA graph by
 *     stream capture and replayed; the pointers they were given are then fixed for the life of the graph. With the
 *     timing ring switched on (mtpc_set_timing) a call also records events and is not meant for capture.
 *   - Return value: MTPC_OK (0) or a negative MTPC_ERR_* code. Nothing throws or aborts across this ABI and
 *     the device code never traps: data errors only the device can see (target >= v, uniform outside [0,1),
 *     a bounded wait that ran out) set bits in a device status word, read with mtpc_get_status, and put
 *     NaN / -1 in the affected outputs.
 *   - There is no CPU fallback: without a CUDA device every compute call returns MTPC_ERR_CUDA.
 */
#ifndef MTPC_H_
#define MTPC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mtpc_head mtpc_head; /* opaque; created by mtpc_create_head, freed by mtpc_destroy */

/* Circuit family (Sec. 3.2). The fully factorised head (Eq. FF) is MTPC_CP with r = 1. */
enum { MTPC_CP = 0, MTPC_HMM = 1, MTPC_BTREE = 2 };
/* dtype of the hidden states and of the weight buffers handed to the library. Arithmetic is always
 * bf16 x bf16 -> fp32 on the tensor cores; MTPC_F32 inputs are rounded to bf16 (nearest-even) first. */
enum { MTPC_F32 = 0, MTPC_BF16 = 1 };

enum {
  MTPC_OK = 0,
  MTPC_ERR_NULL = -1,        /* a required pointer is NULL                                            */
  MTPC_ERR_SHAPE = -2,       /* a size is out of range (T > max_positions, n < 1, ...)                */
  MTPC_ERR_UNSUPPORTED = -3, /* a valid request this version does not implement (see mtpc_config)     */
  MTPC_ERR_WORKSPACE = -4,   /* workspace too small or misaligned                                     */
  MTPC_ERR_CUDA = -5,        /* a CUDA runtime/driver call failed (includes: no device)               */
  MTPC_ERR_TIMEOUT = -6,     /* mtpc_get_status: a device-side bounded wait gave up                   */
  MTPC_ERR_STATIC_SCRATCH = -7, /* mtpc_window_logprob_static: the call needs more than the built-in array */
  MTPC_ERR_STATE = -8        /* mtpc_speculative_accept without a matching draft call before it         */
};

/* mtpc_config.flags */
enum {
  MTPC_FLAG_HMM_CONTEXTUAL = 1u /* MTPC_HMM only: the transitions depend on the hidden state (App. H), see below */
};

/* Bits of the device status word. */
enum {
  MTPC_STATUS_BAD_TARGET = 1u,  /* a target >= v was seen; that window's log-prob is NaN               */
  MTPC_STATUS_BAD_UNIFORM = 2u, /* a uniform outside [0,1) was seen; that draw returned -1 and the log-prob
                                   (or the prefix log-marginals from that byte on) of its window is NaN */
  MTPC_STATUS_TIMEOUT = 4u      /* a bounded barrier wait expired; the outputs of that call are invalid */
};

typedef struct {
  int32_t family;              /* MTPC_CP | MTPC_HMM | MTPC_BTREE                                      */
  int32_t n;                   /* window length. BTREE: a power of two >= 2                            */
  int32_t r;                   /* units per layer (mixture components / hidden states): a power of two,
                                  <= 128 for CP, <= 32 for HMM and BTREE                               */
  int32_t v;                   /* vocabulary: a multiple of 16, any size the n*r*v <= 2^30 limit admits (a unit of
                                  up to 512 symbols is sampled out of tensor memory in one go; wider units are
                                  streamed through it twice and, on more than 128 positions, always with the
                                  draws sorted by unit). v = 272 and the like (no split into equal 16-aligned
                                  tiles of <= 256 columns) draft on up to 128 positions per call only              */
  int32_t d;                   /* hidden size: a multiple of 64                                        */
  int32_t io_dtype;            /* MTPC_F32 | MTPC_BF16: dtype of hidden, W_emit and W_sum              */
  int32_t max_positions;       /* upper bound on T (log-prob) and P (draft) per call                   */
  int32_t max_windows_per_pos; /* upper bound on wpp (>= 1; <= 64)                                     */
  uint32_t flags;              /* 0 or MTPC_FLAG_HMM_CONTEXTUAL                                        */
  int32_t v_valid;             /* 0, or the number of symbols that exist when the vocabulary is not a
                                  multiple of 16 (v - 16 < v_valid <= v; a byte-level Llama has 268: v = 272):
                                  every unit of W_emit keeps v rows, the last v - v_valid of them are padding
                                  whose values are ignored (logit -inf: no mass, never sampled, no gradient);
                                  targets and bytes are < v_valid; target_probs rows keep v entries          */
} mtpc_config;

/* Bytes of device workspace a head with this configuration needs (a multiple of 256). */
int mtpc_workspace_bytes(const mtpc_config* cfg, size_t* out_bytes);

/*
 * Build a head (Sec. 3.3). Enqueues, on `stream`, the one-off preparation (bf16 rounding of F32 weights into
 * the workspace; log-softmax of the static HMM transition logits) and encodes the TMA descriptors.
 *   W_emit   dev [n, r, v, d] io_dtype, row-major: the unembedding tensor W of Sec. 3.3; row ((i*r+k)*v+b).
 *   W_sum    dev [S*r, d] io_dtype: the sum-unit projection R of Sec. 3.3. CP: S=1, the mixture logits
 *            (W_mix). HMM: S=1, the initial-state logits (W_init). BTREE: S = 1+(n-2)*r; rows [0,r) are the
 *            root's weights; for internal node j >= 1 (heap order: root 0, children 2j+1, 2j+2; node
 *            n/2-1+m owns tokens 2m and 2m+1) row r + (j-1)*r*r + a*r + b is the logit of
 *            z_j = b given z_parent(j) = a (softmax over b).
 *   T_static dev [n-1, r, r] fp32, HMM only (else NULL): logit of z_i = b given z_{i-1} = a at
 *            [i-1, a, b], softmax over b (Eq. HMM with input-independent transitions, App. H).
 *            With MTPC_FLAG_HMM_CONTEXTUAL (App. H, "contextual, inhomogeneous"; the paper's best HMM): the
 *            transitions come from the hidden state. W_sum then has S = 1+(n-1)*r sum units: rows [0,r) the
 *            initial-state logits, row r + ((i-1)*r + a)*r + b the logit of z_i = b given z_{i-1} = a, and
 *            T_static is the bias added to those logits before the softmax (the term that allows the identity
 *            initialisation), or NULL for no bias. The bias is copied into the workspace at creation.
 *   workspace dev, 256-byte aligned, >= mtpc_workspace_bytes(cfg); owned by the caller, used by every call
 *            on this head, and must outlive it. With MTPC_BF16 the head keeps the W_emit / W_sum pointers
 *            (they must outlive it too); with MTPC_F32 it keeps rounded copies in the workspace.
 */
int mtpc_create_head(const mtpc_config* cfg, const void* W_emit, const void* W_sum, const float* T_static,
                     void* workspace, size_t workspace_bytes, void* stream, mtpc_head** out);

/*
 * After the parameters have changed (an optimiser step between two training calls): rebinds the head to W_emit,
 * W_sum and T_static, which may be the buffers it was created on, updated in place, or others of the same shapes.
 * With MTPC_BF16 the kernels read W_emit / W_sum in place, so only what creation derived from the parameters is
 * redone: the log-softmax of the static HMM transitions or the copy of the contextual transition bias, the tensor
 * maps, and with MTPC_F32 the rounded copies of the weights. Arguments and ownership as for mtpc_create_head; the
 * work is enqueued on `stream`, which must also order it after the calls that still use the old parameters. The
 * logits a draft call left in the workspace are forgotten (mtpc_speculative_accept then needs a new draft).
 * MTPC_ERR_NULL for a missing pointer (T_static is required exactly where creation requires it).
 */
int mtpc_update_parameters(mtpc_head* head, const void* W_emit, const void* W_sum, const float* T_static, void* stream);

/*
 * Window log-likelihood (Eq. 1 evaluated through Eq. CP / Eq. HMM / Eq. BTree):
 *   out_logprob[t] = log q(x_{t,0..n-1} | h_t), natural log, for t in [0,T).
 *   hidden  dev [T, d] io_dtype, row-major.
 *   targets dev [T, n] int32. A negative target marginalises that byte (App. B.1: any subset of the
 *           variables can be summed out in one pass); a target >= v sets MTPC_STATUS_BAD_TARGET and yields NaN.
 *   T       0 <= T <= max_positions (T == 0 is a no-op).
 *   out_logprob dev [T] fp32.
 * The [T, n, r, v] logit tensor is never written to memory: the GEMM epilogue reduces it on chip.
 */
int mtpc_window_logprob(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t T,
                        float* out_logprob, void* stream);

/*
 * Draft sampling (App. B.2, Algorithm 1) of wpp windows for each of P positions, then the joint log-prob of
 * every drafted window (latents summed out), as speculative verification needs (Algorithm 3).
 *   hidden   dev [P, d] io_dtype.
 *   uniforms dev [P*wpp, 2n] fp32 in [0,1). Window w = p*wpp + j uses row w: columns 0..n-1 drive the latent
 *            draws (CP: column 0; HMM: column i for z_i; BTREE: column j for internal node j, column n-1
 *            unused), column n+i drives the byte of slot i. Every categorical draw is inverse-CDF: the
 *            smallest index j with u < p_0 + ... + p_j (the last index if rounding leaves none).
 *   out_bytes   dev [P*wpp, n] int32.
 *   out_logprob dev [P*wpp] fp32, natural log.
 *   1 <= wpp <= max_windows_per_pos, 0 <= P <= max_positions.
 */
int mtpc_draft_sample(mtpc_head* head, const void* hidden, int32_t P, int32_t wpp, const float* uniforms,
                      int32_t* out_bytes, float* out_logprob, void* stream);

/*
 * Prefix log-marginals (Algorithm 3, "compute marginals"; also the per-slot terms of Eq. 6):
 *   out_prefix_logprob[t, i] = log q(x_{t,0..i} | h_t), the joint with the bytes after slot i summed out, which a
 *   smooth and decomposable circuit gives in one pass (App. B.1). Column n-1 equals mtpc_window_logprob's output.
 *   CP: log-sum-exp over the components of the first i+1 slots; HMM: log-sum-exp of the forward message alpha_i;
 *   BTree: the subtrees right of token i evaluate to one, only the path from its owner to the root is re-evaluated.
 * mtpc_window_prefix_logprob: arguments as mtpc_window_logprob, out_prefix_logprob dev [T, n] fp32.
 * mtpc_draft_sample_prefix:   arguments as mtpc_draft_sample, out_prefix_logprob dev [P*wpp, n] fp32 for the
 *                             drafted windows (what the acceptance stage consumes).
 */
int mtpc_window_prefix_logprob(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t T,
                               float* out_prefix_logprob, void* stream);
int mtpc_draft_sample_prefix(mtpc_head* head, const void* hidden, int32_t P, int32_t wpp, const float* uniforms,
                             int32_t* out_bytes, float* out_prefix_logprob, void* stream);

/*
 * Acceptance stage of speculative sampling (Algorithm 3, from "determine the number of accepted tokens" to the
 * last byte), for the P*wpp windows of the head's most recent draft. The target model's conditionals are an input:
 * the LLM that produces them is outside this library.
 *   draft_bytes     dev [W, n] int32, W = P*wpp: the drafted windows (as written by mtpc_draft_sample*).
 *   prefix_logprob  dev [W, n] fp32: their prefix log-marginals (as written by mtpc_draft_sample_prefix).
 *   target_probs    dev [W, n+1, v] fp32: row i is p(X_{t+i+1} | context, draft bytes 0..i-1), probabilities.
 *   accept_uniforms dev [W, n+1] fp32 in [0,1): column i is the alpha of the test on byte i; column n draws the
 *                   last byte.
 *   out_accepted    dev [W] int32: s in [0, n], the number of accepted draft bytes: byte i is accepted while
 *                   alpha_i <= p(x_i) / q(x_i | x_0..x_{i-1}), q being the ratio of consecutive prefix marginals.
 *   out_next_byte   dev [W] int32: the byte that follows the accepted ones: drawn from target row n if s = n, else
 *                   from the residual max(0, p - q(. | x_0..x_{s-1})) / Z with p = target row s. Inverse-CDF draws
 *                   as in mtpc_draft_sample. (With zero residual mass, which exact arithmetic excludes after a
 *                   rejection, the last byte v-1 is returned.)
 * The conditional q(. | x_0..x_{s-1}) is a mixture of the r input units of slot s whose weights are the posterior of
 * the latent that owns the slot; it is evaluated from what the draft call left in the workspace. Hence:
 *   - the call must follow mtpc_draft_sample / mtpc_draft_sample_prefix on this head with the same P and wpp, with no
 *     other call on the head in between, else MTPC_ERR_STATE;
 *   - a draft of P <= 128 positions (decode-time batches) leaves every logit of those positions: one kernel;
 *   - a draft of more positions (a verification batch) leaves only the evidence of the drafted bytes. The call then
 *     runs the tests, sorts the rejected windows by the slot of their first rejected byte, recomputes that slot's
 *     r*v logits for them in one projection pass over staged hidden states, and draws. It reads the hidden states the
 *     DRAFT call was given (bf16 heads: the caller's buffer, which must still hold them); heads created for at most 128
 *     positions have no scratch for this (MTPC_ERR_UNSUPPORTED).
 * A uniform outside [0,1) or a draft byte outside [0,v) sets the status bit and yields -1 / -1 for that window.
 */
int mtpc_speculative_accept(mtpc_head* head, int32_t P, int32_t wpp, const int32_t* draft_bytes,
                            const float* prefix_logprob, const float* target_probs, const float* accept_uniforms,
                            int32_t* out_accepted, int32_t* out_next_byte, void* stream);

/*
 * Training loss over overlapping windows (Eq. 6): num_sequences sequences of sequence_length positions each
 * (T = num_sequences * sequence_length rows of hidden / targets, sequence-major).
 *   out_slot_loss[j] = L_j = -(1/N) sum_i (1/V_ij) sum_t log q(x_{t,j} | h_t, x_{t,0..j-1}),
 *   out_loss[0]      = sum_j gamma^j L_j   (j from 0; the paper's gamma^(j-1) with j from 1),
 * where the conditional is the difference of consecutive prefix log-marginals, a negative target marks an invalid
 * (masked, marginalised) byte and V_ij counts the valid targets of slot j in sequence i (a slot with none
 * contributes 0). Forward value only. out_slot_loss dev [n] fp32, out_loss dev [1] fp32. The reduction order is
 * fixed: the same inputs give the same bits.
 */
int mtpc_window_loss(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t num_sequences,
                     int32_t sequence_length, float gamma, float* out_slot_loss, float* out_loss, void* stream);

/*
 * Backward pass of the window log-likelihood (training, Sec. 4.1): gradients of
 *     L = sum_t weight[t] * log q(x_{t,0..n-1} | h_t)
 * through the circuit (Eq. CP / Eq. HMM / Eq. BTree), the softmaxes of Sec. 3.3 and the two projections.
 * (weight[t] = -1/T gives the mean negative log-likelihood; a zero weight masks a position.)
 *   hidden, targets, T   as for mtpc_window_logprob (a negative target is a marginalised byte: no gradient).
 *   weight        dev [T] fp32.
 *   bwd_workspace dev, 256-byte aligned, >= mtpc_backward_workspace_bytes(cfg, T): holds the units' log-sum-exps and
 *                 posteriors, the fp32 emission logits the forward pass keeps for the backward pass (T * n*r*v * 4
 *                 bytes) and their bf16 gradient (half as many bytes again). The weights and hidden states are read
 *                 where they lie (no transposed copies). Caller-owned, used only during the call's work.
 *   out_logprob   dev [T] fp32 or NULL: the forward value.
 *   d_hidden      dev [T, d] fp32;  dW_emit dev [n, r, v, d] fp32;  dW_sum dev [S*r, d] fp32: overwritten, not
 *                 accumulated.
 *   dT_static     dev [n-1, r, r] fp32: gradient of the static transition logits (MTPC_HMM without the contextual
 *                 flag; required there, ignored otherwise). With MTPC_FLAG_HMM_CONTEXTUAL the gradient of the bias is the
 *                 column sum of the transition-logit gradients and is not returned separately.
 * Long windows: the circuit backward kernels keep the messages of every step / node of a window in shared memory and use
 * fewer warps per CTA as n*r grows; a static HMM whose (n-1)*r*r transition-gradient accumulator does not fit beside them
 * (n = 64 with r = 32) returns MTPC_ERR_UNSUPPORTED.
 * Arithmetic: posteriors in fp32; the logit gradients are rounded to bf16 (the operand type of the tensor cores) before
 * the three weight-sized GEMMs, fp32 accumulation. dT_static is accumulated with atomic adds (order not fixed).
 */
/*
 * mtpc_window_loss_backward: the training loss of Eq. 6 (as mtpc_window_loss: per-slot conditionals, valid-token
 * normalisation V_ij, discount gamma^j) AND its gradients, for num_sequences sequences of sequence_length positions.
 * Eq. 6 is linear in the prefix log-marginals, L = sum_t sum_j coeff[t, j] log q(x_{t,0..j}), with
 * coeff[t, j] = c[t, j] - c[t, j+1], c[t, j] = -gamma^j / (N V_ij) for a valid target and 0 otherwise; the call runs one
 * circuit backward pass per prefix length j+1 (later bytes summed out), accumulates the posteriors in fp32, and then
 * shares the projection-sized work (logit gradients, the three GEMMs) with mtpc_window_logprob_backward. Same workspace
 * (mtpc_backward_workspace_bytes with T = num_sequences * sequence_length), same outputs, same arithmetic notes.
 */
int mtpc_backward_workspace_bytes(const mtpc_config* cfg, int32_t T, size_t* out_bytes);
int mtpc_window_logprob_backward(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t T,
                                 const float* weight, void* bwd_workspace, size_t bwd_workspace_bytes,
                                 float* out_logprob, float* d_hidden, float* dW_emit, float* dW_sum, float* dT_static,
                                 void* stream);
int mtpc_window_loss_backward(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t num_sequences,
                              int32_t sequence_length, float gamma, void* bwd_workspace, size_t bwd_workspace_bytes,
                              float* out_slot_loss, float* out_loss, float* d_hidden, float* dW_emit, float* dW_sum,
                              float* dT_static, void* stream);

/*
 * Low-rank-adapted unembeddings (App. G, "Unembedding parameter sharing"): U[i, j] = W_base[i] + A[i, j] B[i, j], one
 * base matrix per token slot shared by its r components plus a rank-k adaptor per component. The head computes on the
 * composed tensor; these two calls convert between the shared parameters and it. They need no head.
 *   W_base  device [n, v, d] bf16      A  device [n, r, v, k] bf16      B  device [n, r, k, d] bf16   (row-major)
 * mtpc_lowrank_compose writes W_emit_out, device [n, r, v, d] bf16 = round-to-nearest of the fp32 sum: the W_emit of
 * mtpc_create_head. A bf16 head reads that buffer in place, so composing into it again after an optimiser step is
 * all a training loop needs (plus mtpc_update_parameters where T_static changed too).
 * mtpc_lowrank_backward takes the gradient of the composed tensor, dW_emit device [n, r, v, d] fp32 (as written by
 * the backward calls above), and OVERWRITES
 *   dW_base [n, v, d] = sum_j dW_emit[i, j],  dA [n, r, v, k] = dW_emit[i, j] B[i, j]^T,  dB [n, r, k, d] = A[i, j]^T dW_emit[i, j]
 * (device fp32, caller-owned). 1 <= k <= 64 (MTPC_ERR_UNSUPPORTED beyond); v <= 65535 and n r <= 65535
 * (MTPC_ERR_SHAPE). Any d works; with d a multiple of 4 and 16-byte aligned pointers the kernels use vector accesses.
 * Asynchronous on `stream`.
 */
int mtpc_lowrank_compose(int32_t n, int32_t r, int32_t v, int32_t d, int32_t k, const void* W_base, const void* A,
                         const void* B, void* W_emit_out, void* stream);
int mtpc_lowrank_backward(int32_t n, int32_t r, int32_t v, int32_t d, int32_t k, const void* A, const void* B,
                          const float* dW_emit, float* dW_base, float* dA, float* dB, void* stream);

/*
 * A head that keeps the shared unembeddings of App. G FACTORED: the emission logits are evaluated as
 *   logit[t, i, j, :] = W_base[i] h_t + A[i, j] (B[i, j] h_t)
 * without ever forming the composed [n, r, v, d] tensor: one contraction over d per slot (shared by its r components), a
 * small one for z = B h, and a rank-k correction per component, 2 d (n v + n r k) + 4 n r v k FLOPs per position instead
 * of 2 d n r v. z is handed to the tensor cores as two bf16 halves (z = hi + lo), so the result differs from exact
 * arithmetic on the bf16 parameters only by fp32 accumulation (no rounding of a composed U to bf16).
 *   cfg, W_sum, T_static, workspace, stream, out: as mtpc_create_head; cfg->io_dtype must be MTPC_BF16.
 *   k        the adaptors' rank: 16 or 32 (MTPC_ERR_UNSUPPORTED otherwise). v must be a multiple of 16 that splits into
 *            at most eight panels of at most 224 columns (a panel's two accumulators and the correction slots share the
 *            512 columns of tensor memory): every such v up to 1792; MTPC_ERR_UNSUPPORTED otherwise.
 *   W_base   dev [n, v, d] bf16;  A dev [n, r, v, k] bf16;  B dev [n, r, k, d] bf16: caller-owned, read in place, must
 *            outlive the head (after an optimiser step no call is needed unless W_sum / T_static moved:
 *            mtpc_update_parameters with W_emit = NULL then).
 *   workspace >= mtpc_lowrank_workspace_bytes(cfg, k): the dense head's workspace plus z = B h as two bf16 halves, a copy
 *            of A in the layout the kernel reads (remade on every call, so A is always read as it is then) and, for
 *            v > 224, the per-panel partial log-sum-exps.
 * Such a head serves mtpc_window_logprob, mtpc_window_prefix_logprob, mtpc_window_loss, mtpc_window_logprob_host,
 * mtpc_draft_sample, mtpc_draft_sample_prefix and mtpc_speculative_accept: up to 128 positions, the draft's weight pass
 * streams W_base and B (n v + n r k rows) instead of n r v composed rows and the logits are formed from the two small
 * products; longer drafts with one window per position and v <= 512 form, per (window, slot), the logits of the one unit
 * the latent draw selected, and the acceptance stage after them forms the rejected slot's logits the same way; other
 * long drafts run 128 positions at a time and keep no logits (mtpc_speculative_accept then returns MTPC_ERR_STATE). Its training calls are mtpc_lowrank_window_logprob_backward and
 * mtpc_lowrank_window_loss_backward (below); mtpc_window_logprob_backward and mtpc_window_loss_backward return
 * MTPC_ERR_UNSUPPORTED on it (they produce the gradient of a composed tensor: mtpc_lowrank_compose + mtpc_create_head,
 * carried back by mtpc_lowrank_backward).
 */
int mtpc_lowrank_workspace_bytes(const mtpc_config* cfg, int32_t k, size_t* out_bytes);

/*
 * Training call of a factored head (App. G): out_logprob[t] = log q(targets[t]) as mtpc_window_logprob, and the gradients
 * of sum_t weight[t] out_logprob[t] with respect to the hidden states and to the parameters the head was built on, without
 * the [n, r, v, d] gradient of a composed tensor ever existing: with g = d / d logit [T, n r v],
 *   dW_base[i] = (sum_j g_ij)^T h,   dA[i,j] = g_ij^T (B[i,j] h),   dB[i,j] = (g_ij A[i,j])^T h,
 *   d_hidden   = sum_i (sum_j g_ij) W_base[i] + sum_ij (g_ij A[i,j]) B[i,j] + the sum units' part.
 *   hidden, targets, T, weight, out_logprob, d_hidden [T, d], dW_sum, dT_static: as mtpc_window_logprob_backward.
 *   dW_base dev [n, v, d] fp32;  dA dev [n, r, v, k] fp32;  dB dev [n, r, k, d] fp32: OVERWRITTEN.
 *   bwd_workspace  dev, 256-byte aligned, >= mtpc_lowrank_backward_workspace_bytes(cfg, k, T): the kept logits
 *                  [T, n r v] fp32, their gradients in bf16, and the small operands derived from them.
 * g is rounded to bf16 before the tensor cores contract it (as in mtpc_window_logprob_backward), dA uses the bf16 high
 * half of B h. MTPC_ERR_STATE on a head that was not created by mtpc_create_head_lowrank. Asynchronous on `stream`.
 */
int mtpc_lowrank_backward_workspace_bytes(const mtpc_config* cfg, int32_t k, int32_t T, size_t* out_bytes);
int mtpc_lowrank_window_logprob_backward(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t T,
                                         const float* weight, void* bwd_workspace, size_t bwd_workspace_bytes,
                                         float* out_logprob, float* d_hidden, float* dW_base, float* dA, float* dB,
                                         float* dW_sum, float* dT_static, void* stream);
/*
 * The training loss of Eq. 6 and its gradients on a factored head: arguments as mtpc_window_loss_backward, with dW_base, dA,
 * dB (as above) in place of dW_emit; the same workspace size as mtpc_lowrank_window_logprob_backward for
 * T = num_sequences * sequence_length.
 */
int mtpc_lowrank_window_loss_backward(mtpc_head* head, const void* hidden, const int32_t* targets, int32_t num_sequences,
                                      int32_t sequence_length, float gamma, void* bwd_workspace, size_t bwd_workspace_bytes,
                                      float* out_slot_loss, float* out_loss, float* d_hidden, float* dW_base, float* dA,
                                      float* dB, float* dW_sum, float* dT_static, void* stream);
int mtpc_create_head_lowrank(const mtpc_config* cfg, int32_t k, const void* W_base, const void* A, const void* B,
                             const void* W_sum, const float* T_static, void* workspace, size_t workspace_bytes,
                             void* stream, mtpc_head** out);

/*
 * Host-buffer variants: same results, but hidden / targets / uniforms are HOST pointers (pinned memory for
 * full copy speed) and the outputs are written to HOST buffers. The copies to and from the device go through
 * staging areas in the workspace; the call returns after the stream has been synchronised, so the outputs are
 * ready on return. mtpc_window_logprob_host uploads and processes 2048 positions at a time: the uploads run on a
 * second stream the head owns, ordered after the work already on `stream`, so that all but the first are hidden
 * behind the kernels (with per-kernel timing on, every chunk is recorded as a call of its own).
 */
int mtpc_window_logprob_host(mtpc_head* head, const void* hidden_host, const int32_t* targets_host, int32_t T,
                             float* out_logprob_host, void* stream);
int mtpc_draft_sample_host(mtpc_head* head, const void* hidden_host, int32_t P, int32_t wpp,
                           const float* uniforms_host, int32_t* out_bytes_host, float* out_logprob_host,
                           void* stream);

/*
 * Read and clear the device status word. Synchronises `stream` first. *out_flags receives the MTPC_STATUS_*
 * bits; returns MTPC_ERR_TIMEOUT if MTPC_STATUS_TIMEOUT is set, MTPC_ERR_CUDA on a CUDA error, else MTPC_OK.
 */
int mtpc_get_status(mtpc_head* head, void* stream, uint32_t* out_flags);

/*
 * Per-kernel device timing (CUDA events recorded on the call's stream around each launch). Off by default.
 * mtpc_set_timing(head, ring): keep the events of the `ring` most recent calls (0 <= ring <= 4096; 0 = off;
 * changing it discards what was recorded). mtpc_get_timing(head, calls_back, ...) synchronises on the events
 * of the call made `calls_back` calls ago (0 = the most recent) and writes up to `capacity` phase durations
 * in milliseconds, *out_count = number of phases that call had:
 *   mtpc_window_logprob: [0] projection GEMM + fused epilogue, [1] circuit evaluation.
 *   mtpc_window_prefix_logprob, mtpc_window_loss: as mtpc_window_logprob (the loss reduction is not timed).
 *   mtpc_speculative_accept: [0] the acceptance kernel.
 *   mtpc_window_logprob_backward: [0] forward projection, [1] circuit backward, [2] gradient of the logits,
 *                        [3] the three plain GEMMs.
 *   mtpc_window_loss_backward: [0] forward projection + prefix marginals + loss, [1] circuit backward (mixture:
 *                        one pass per prefix length; tree: the same passes in one launch; HMM: one reverse sweep),
 *                        [2] and [3] as above.
 *   mtpc_draft_sample, mtpc_draft_sample_prefix:   P <= 128 positions: [0] one pass over all weights (logits of every unit),
 *                        [1] per-slot latent + byte draws and evidence, [2] circuit evaluation.
 *                        Otherwise: [0] sum-unit GEMM, [1] latent sampling, [2] byte draws (GEMM + inverse-CDF
 *                        epilogue; when the draws are sorted by unit: the sort, the staging copy and that GEMM),
 *                        [3] GEMM + gather epilogue on the drafted bytes, [4] circuit evaluation.
 */
int mtpc_set_timing(mtpc_head* head, int32_t ring);
int mtpc_get_timing(mtpc_head* head, int32_t calls_back, float* out_ms, int32_t capacity, int32_t* out_count);

/* Number of kernels the library launched on behalf of this head since creation (preparation included). */
int mtpc_launch_count(mtpc_head* head, uint64_t* out_count);

/*
 * Test hook, not part of the method (no passage of the paper): sets the time limit of the pipeline waits inside
 * the tensor-core kernels of this head (waits on shared-memory barriers for a TMA copy, an MMA batch or a free
 * accumulator). The default is 1 s, far beyond any healthy wait; limit_ns == 0 restores it. With a limit shorter
 * than a memory round trip a healthy call gives up: the CTA that saw the wait expire raises MTPC_STATUS_TIMEOUT,
 * waits (up to the fixed 1 s) for its copies and MMAs in flight, frees its tensor memory and returns, the
 * outputs of that call are unspecified and the next mtpc_get_status returns MTPC_ERR_TIMEOUT. That is how the tests
 * exercise the give-up path without withholding anything from a kernel. Host-side only; takes effect at the next call.
 */
int mtpc_debug_set_wait_limit_ns(mtpc_head* head, uint64_t limit_ns);

/*
 * Test and measurement hook (no passage of the paper): which build of the projection kernel this head launches.
 * 0 (default): chosen per launch; 1: every CTA works alone (tcgen05 cta_group::1); 2: clusters of two CTAs share every
 * MMA (cta_group::2), MTPC_ERR_UNSUPPORTED if the device cannot hold such a cluster. The results are the same numbers
 * either way (same products, same order of accumulation); the tests run both.
 */
int mtpc_debug_set_projection_variant(mtpc_head* head, int32_t variant);

/*
 * Test and measurement hook (no passage of the paper): how mtpc_draft_sample on more than 128 positions runs the byte
 * draws of Algorithm 1. 0 (default): chosen per call; 1: one pass of every position against every input unit;
 * 2: the (window, slot) pairs are first sorted by the unit they sample from, and each is multiplied by that unit only
 * (MTPC_ERR_UNSUPPORTED if the head was created for at most 128 positions). Same uniforms, same bytes either way.
 */
int mtpc_debug_set_draft_grouping(mtpc_head* head, int32_t mode);

/*
 * Window log-likelihood without any allocation (the paper has no counterpart: this is a packaging variant of
 * mtpc_window_logprob, same arithmetic, same kernels, same results).
 *
 * Who needs it: code that must not, or cannot, allocate device memory at the point where it wants a
 * log-likelihood - a plug-in running inside somebody else's memory pool, a callback on a serving thread that
 * is forbidden to call cudaMalloc because that call synchronises the device, a process whose memory budget was
 * handed out in full at start-up. mtpc_window_logprob asks such callers for a workspace they have no way to
 * obtain. This entry point needs neither a head nor a workspace: its scratch (a status word, the
 * log-softmaxed HMM transitions, G [T, n, r] and log omega [T, S*r], all fp32) lives in one static device array
 * of MTPC_STATIC_SCRATCH_BYTES that is part of the library image. Every GPU that loads the library therefore
 * holds those bytes until the process exits, whether or not this function is ever called. It calls no
 * cudaMalloc / cudaFree and no allocating library routine.
 *
 *   cfg        family, n, r, v, v_valid, d as for mtpc_create_head (v_valid: a padded vocabulary, 0 = none);
 *              io_dtype must be MTPC_BF16 and flags 0 (MTPC_ERR_UNSUPPORTED otherwise: fp32 inputs would need a
 *              rounded copy of the weights, contextual transitions a copy of their bias); max_positions,
 *              max_windows_per_pos are ignored.
 *   W_emit, W_sum, T_static, hidden, targets, out_logprob: dev, exactly as for mtpc_create_head and
 *              mtpc_window_logprob; all caller-owned, read or written only by the work this call enqueues.
 *   out_status dev uint32 or NULL: receives this call's MTPC_STATUS_* bits (stream-ordered, like the outputs).
 *   T          T == 0 is a no-op. If 256 + 4*(n-1)*r*r (HMM) + 4*T*n*r + 4*T*S*r bytes (each term rounded up
 *              to 256) exceed MTPC_STATIC_SCRATCH_BYTES the call returns MTPC_ERR_STATIC_SCRATCH and
 *              enqueues nothing; split the positions over several calls then.
 *
 * First call on a device: it looks up the array's device address (once per device, with that device current)
 * and may make the CUDA runtime load the library's kernels. Make that first call outside any stream capture.
 * All calls on one device share the one array, and the array keeps the previous call's contents; the call
 * clears the part that has to start at zero (the status word) itself. Two calls whose work overlaps on the
 * GPU (different streams, or different threads without ordering) race on the array: order them on one stream
 * or with events. Asynchronous like mtpc_window_logprob: the outputs are ready when `stream` reaches them.
 */
#define MTPC_STATIC_SCRATCH_BYTES (16u << 20) /* 16 MiB: configs up to T*(n*r + S*r) = 4.19 M fp32 entries */
int mtpc_window_logprob_static(const mtpc_config* cfg, const void* W_emit, const void* W_sum,
                               const float* T_static, const void* hidden, const int32_t* targets, int32_t T,
                               float* out_logprob, uint32_t* out_status, void* stream);

/* Frees the host-side object (the workspace and the weights stay the caller's). Synchronises nothing. */
int mtpc_destroy(mtpc_head* head);

/* Static, NUL-terminated description of a return code. */
const char* mtpc_status_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* MTPC_H_ */
