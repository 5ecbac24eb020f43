/*
 * pipemare.h -- C ABI of the B200 (sm_100a) PipeMare hot path.
 *
 * One GPU emulates a P-stage asynchronous pipeline.  Each call of pm_step is one
 * pipeline tick: every stage runs one forward with the weights it holds now, one
 * backward for the microbatch that entered it tau_fwd updates ago (against the
 * discrepancy-corrected weights of T2), and one weight update with the
 * rescheduled step size of T1.  All arithmetic runs in CUDA kernels; this
 * interface only carries pointers and sizes.
 *
 * Conventions
 *   - "device" pointers are CUDA device memory owned by the caller.  The library
 *     never allocates or frees device memory; it borrows the pointers for the
 *     lifetime of the context.  "host" pointers are ordinary host memory, read
 *     during the call unless stated otherwise.
 *   - Work is enqueued on the CUDA stream given at initialisation and returns
 *     before it completes, except pm_get_losses and pm_get_bookkeeping, which
 *     synchronise that stream.
 *   - Every function returns a pm_status; nothing throws or aborts.  After an
 *     error pm_last_error(ctx) gives a readable message.
 *   - Stages are numbered 1..P in the paper and 0..P-1 in array arguments here.
 *   - One microbatch per update (N = 1 in the notation of Section 2.1) unless pm_config.n_micro says otherwise.
 *
 * Two loop orders compute the same recurrence (pm_config.loop_order):
 *   PM_TICK_MAJOR  the pipeline as it would run on P devices: every call of pm_step is one tick in which all
 *                  stages work side by side on different microbatches; each stage holds ONE version of its
 *                  weights and a ring of the activations of its microbatches in flight (depth tau_fwd + 1, so
 *                  the rings grow with P^2: Appendix A.1).
 *   PM_MB_MAJOR    the form in which Section 2.1 states the method: every call of pm_step takes one microbatch
 *                  through all stages forward, then backward, then applies the update; each stage keeps a queue
 *                  of its last tau_fwd + 1 weight versions (the forward operands) and activations of one
 *                  microbatch only.  Memory grows with sum_i tau_fwd,i * |w_i| instead of P^2 activations, any
 *                  tau_fwd,i >= 0 is accepted (all zero = synchronous training), and no drain ticks exist.
 */
#ifndef PIPEMARE_H
#define PIPEMARE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pm_ctx pm_ctx;

typedef enum {
  PM_OK = 0,
  PM_ERR_INVALID_ARG = 1,   /* null pointer, negative size, unknown enum value            */
  PM_ERR_SHAPE = 2,         /* dimensions the kernels cannot take (see pm_init_stages)    */
  PM_ERR_STATE = 3,         /* phase calls out of order                                   */
  PM_ERR_NOMEM = 4,         /* ring or workspace too small; message states the need       */
  PM_ERR_UNSUPPORTED = 5,   /* valid request that is not built                            */
  PM_ERR_CUDA = 6,          /* a CUDA runtime call failed; message carries its text       */
  PM_ERR_TIMEOUT = 7        /* a bounded device-side wait expired                         */
} pm_status;

enum { PM_F32 = 0, PM_BF16 = 1 };                 /* GEMM operand type; state is always fp32 */
enum { PM_SGDM = 0, PM_ADAM = 1 };
enum { PM_ACT_NONE = 0, PM_ACT_RELU = 1, PM_ACT_GELU = 2 };   /* GELU = exact erf form      */
enum { PM_OP_LINEAR = 0, PM_OP_EMBED = 1, PM_OP_LAYERNORM = 2, PM_OP_ATTENTION = 3, PM_OP_SKIP_OUT = 4,
       PM_OP_RESIDUAL = 5, PM_OP_CROSS_ATTENTION = 6 };
/* pm_op_desc.flags */
enum { PM_OPF_CAUSAL = 1,          /* ATTENTION: keys after the query position are masked                        */
       PM_OPF_FROM_MEMORY = 2,     /* LAYERNORM: normalises the memory (see RESIDUAL) instead of the main input; the
                                      stage's Linear reads that, the main input goes to the post-op               */
       PM_OPF_SECOND_STREAM = 4,   /* EMBED: embeds the second token stream (the decoder input)                   */
       PM_OPF_EMIT_MEMORY = 8,     /* RESIDUAL: the stage's output is the memory (the encoder output); the next
                                      stage must start with EMBED | PM_OPF_SECOND_STREAM                          */
       PM_OPF_SKIP_TWO = 16 };     /* SKIP_OUT: the skip tensor goes to the stage two positions on                */
enum { PM_LOSS_MSE = 0, PM_LOSS_CE = 1 };
enum { PM_TICK_MAJOR = 0, PM_MB_MAJOR = 1 };      /* pm_config.loop_order */

/* Alignment, in elements, of every stage slice and of every tensor inside it. */
#define PM_ALIGN_ELEMS 64
#define PM_MAX_LINEARS 4       /* Linear ops per stage                                    */
#define PM_MAX_STAGES 1024

/* One operator of a stage.  A stage is  [EMBED | LAYERNORM]  LINEAR{1..PM_MAX_LINEARS}  [ATTENTION | SKIP_OUT |
 * RESIDUAL]  (with a pre- or post-op exactly one LINEAR).
 *   LINEAR     y = act(x W^T + b), W is [n_out, n_in] row-major, b is [n_out].
 *   EMBED      x = table[id] * sqrt(n_out) + sinusoidal position; table is [n_in = vocabulary, n_out = width, a
 *              multiple of four];
 *              the stage's input is int32 token ids: the first stage embeds the first stream; a later stage with
 *              PM_OPF_SECOND_STREAM (the first stage of a decoder) embeds the second and ignores the previous
 *              stage's output.  seq_len gives the position period.
 *   LAYERNORM  over the last dimension (n_in = n_out = width), eps 1e-5, biased variance; parameters gain, bias.
 *   ATTENTION  splits the Linear's output [T, 3d] into q, k, v; softmax(q k^T / sqrt(d / n_heads)) v per head and
 *              per sequence of seq_len rows (T a multiple of seq_len; seq_len <= 128, or seq_len = 256 with
 *              PM_BF16 and heads of width 64, else PM_ERR_UNSUPPORTED); the stage hands o [T, d]
 *              and, as a skip tensor, the Linear's input to the next stage, which must end in RESIDUAL.
 *   SKIP_OUT   hands the Linear's input on as a skip tensor next to its output; next stage must end in RESIDUAL.
 *   RESIDUAL   adds the skip tensor it was sent to the Linear's output.
 *   CROSS_ATTENTION  the stage starts with LAYERNORM | PM_OPF_FROM_MEMORY; the Linear's output [T, 2d] is k, v, the
 *              stage's main input [T, d] is q; attention of q over k, v per head and sequence (source and target
 *              sequences have the same length seq_len); o [T, d] goes to the next stage.  A skip tensor sent with
 *              PM_OPF_SKIP_TWO by the previous stage passes over this one.  The gradients the memory receives
 *              from the cross-attention stages are added in descending stage order (Section 2.1 fixes no order).
 * Where the backward pass reads a parameter value it reads the T2-corrected one (Section 3.2): the Linear
 * matrix in the input-gradient product and the LayerNorm gain.  Nothing else is read in the backward pass. */
typedef struct {
  int32_t kind;            /* PM_OP_* */
  int32_t n_in, n_out;
  int32_t act;             /* PM_ACT_* (LINEAR) */
  int32_t n_heads;         /* ATTENTION, CROSS_ATTENTION */
  int32_t seq_len;         /* ATTENTION, CROSS_ATTENTION, EMBED */
  int32_t flags;           /* PM_OPF_* */
} pm_op_desc;

/* One pipeline stage (Section 2.1).  Copied during pm_init_stages.
 * tau_fwd / tau_bkwd: number of updates between the forward / backward read of this
 * stage's weights and the update that uses the resulting gradient.  PipeMare
 * (Table 1) has tau_fwd = 2(P-i)+1 and tau_bkwd = 0, which is the only delay
 * pattern the tick schedule (PM_TICK_MAJOR) realises; PM_MB_MAJOR takes any
 * tau_fwd >= 0 with tau_bkwd = 0, or tau_bkwd = tau_fwd for EVERY stage: weight
 * stashing (Section 2.2), the backward pass of a microbatch reads the queued version
 * its forward read (weights in the operand type, LayerNorm gain in fp32), there is no
 * discrepancy and T2 corrects nothing; other values are PM_ERR_UNSUPPORTED.
 * param_offset / param_count: this stage's slice of the flat arenas, in elements;
 * both multiples of PM_ALIGN_ELEMS.  Inside the slice each op's W and then b start
 * at the next multiple of PM_ALIGN_ELEMS (pm_op_param_offsets gives the numbers). */
typedef struct {
  int32_t tau_fwd, tau_bkwd;
  int32_t n_ops;
  const pm_op_desc* ops;   /* host */
  uint64_t param_offset, param_count;
} pm_stage_desc;

/* Hyper-parameters.
 * T1 (Section 3.1, Eq. 2): step size of stage i at its update k is
 *   alpha_base(k) / tau_fwd,i ^ p_k,  p_k = 1 - min(k / t1_K, 1).
 * T2 (Section 3.2): backward reads w - (tau_fwd - tau_bkwd) * delta, and
 *   delta <- gamma delta + (1 - gamma)(w_new - w_old), gamma = t2_D ^ (1/(tau_fwd - tau_bkwd)).
 * Optimiser: momentum SGD in the form of Appendix B.3 (v <- beta1 v - alpha g; w <- w + v)
 * or bias-corrected Adam without weight decay.
 * alpha_base(k) = alpha_by_step[min(k, alpha_len-1)] if alpha_by_step != NULL (host array,
 * copied at initialisation), else alpha_const. */
typedef struct {
  int32_t n_stages;        /* P */
  int32_t microbatch;      /* rows T of every activation matrix */
  int32_t compute_dtype;   /* PM_F32 | PM_BF16 */
  int32_t optimizer;       /* PM_SGDM | PM_ADAM */
  int32_t loss;            /* PM_LOSS_MSE: mean over all T*out entries of (y - target)^2;
                              PM_LOSS_CE: mean over the T rows of logsumexp(logits) - logits[target], logits =
                              the last Linear's fp32 output (last stage: one Linear, activation none, no post-op) */
  float beta1, beta2, eps;
  int32_t t1_enable;
  int64_t t1_K;
  int32_t t2_enable;
  double t2_D;
  double alpha_const;
  const double* alpha_by_step;   /* host, may be NULL */
  int64_t alpha_len;
  int64_t loss_log_capacity;     /* losses kept on the device (a ring); 0 = default 4096 */
  int32_t loop_order;            /* PM_TICK_MAJOR | PM_MB_MAJOR (see the top of this file) */
  int32_t entry_period;          /* E, PM_TICK_MAJOR only; 0 or 1: a microbatch enters at every tick.  E > 1: one enters every
                                    E ticks (pm_forward takes inputs at ticks 0, E, 2E, ... and NULL between, PM_ERR_STATE
                                    otherwise), so a stage holds floor(tau_fwd / E) + 1 microbatches' activations instead of
                                    tau_fwd + 1, and reads the weight version Table 1's delay names, max(0, a - tau_fwd), from a
                                    queue of tau_fwd + 1 versions as in PM_MB_MAJOR: the recurrence is unchanged, only the
                                    schedule on the GPU is sparser (activation memory / E, weight queues added).  N microbatches
                                    need (N - 1) E + 2P ticks.  Not combined with pm_set_warmup. */
  int32_t n_micro;               /* N of Section 2.1: microbatches per update; 0 or 1 = one.  N > 1 needs PM_MB_MAJOR
                                    (else PM_ERR_UNSUPPORTED): calls t = 0, 1, ... of pm_step belong to update u = t / N;
                                    tau_fwd counts updates (Table 1: ceil((2(P-i)+1)/N)), every microbatch of a minibatch
                                    reads weight version max(0, u - tau_fwd,i); the minibatch loss is the mean of its N
                                    microbatch losses, so dL/dy carries the factor 1/N and the N parameter gradients are
                                    added in the grad arena in call order; pm_update applies update u after the N-th call
                                    and is a no-op before.  The step-size schedule, the T1 annealing and Adam's bias
                                    correction count updates. */
  int32_t recompute_segment;     /* S: PipeMare Recompute (Appendix A.2, Appendix D); 0 = none (also when S >= n_stages).  S > 0
                                    needs PM_MB_MAJOR (else PM_ERR_UNSUPPORTED).  Stages [kS, (k+1)S) form segment k.  The
                                    forward pass and the loss are unchanged; before a segment's backward pass its stages run
                                    forward once more from what the forward pass left at the segment's inputs (main input, skip
                                    tensors and memory that cross the segment's boundary), reading the weights
                                    w_{u - tau_recomp,i}, and the backward pass takes every stashed activation from that
                                    recomputation.  tau_recomp,i = min(tau_fwd,i, ceil((2(S - j) + 1) / N)) for the j-th stage
                                    (1-based) of its segment: inside a segment the recomputation precedes the backward pass
                                    like the forward pass of an S-stage pipeline.  The last segment's backward follows its
                                    forward at that very distance and is not recomputed (tau_recomp = tau_fwd).  With
                                    t2_enable the recomputation reads w_v - (tau_fwd - tau_recomp) delta_v, v = u -
                                    tau_recomp (T2 for recompute, with the accumulator as it stood with version v): the update
                                    that produces version v also writes that copy, in the operand type, into tau_recomp + 1
                                    further slots of the stage's version queue (counted by pm_query_bytes). */
  int32_t fuse_update;           /* 1: the weight-gradient GEMM of a Linear applies the update of its matrix in its epilogue,
                                    while dW is still on chip (same arithmetic per element, bit for bit; dW of Linear matrices
                                    is then NOT written to arenas.grad).  The weight-gradient GEMMs move from pm_backward to
                                    pm_update, whose update kernel covers the remaining parameters (biases, LayerNorm
                                    parameters, embedding tables).  Needs PM_BF16, one Linear per stage, n_micro <= 1,
                                    entry_period <= 1 and recompute_segment = 0, else PM_ERR_UNSUPPORTED.  0: off. */
  int32_t stochastic_tau_max;    /* > 0: the stage-wise stochastic delay model of Appendix E instead of the pipeline's fixed delays:
                                      w_{i,t+1} = w_{i,t} - alpha [grad f_{t-tau_i}(w_{t-tau_i})]_i,   tau_i drawn per step and stage.
                                    Every microbatch runs forward and backward on the current weights of all stages; the
                                    gradients of the last stochastic_tau_max + 1 microbatches are kept (a ring of that many
                                    copies of the grad arena, counted by pm_query_bytes), and at step t stage i applies its slice
                                    of the gradient of microbatch t - tau_i, tau_i from pm_set_delays (0 <= tau_i <=
                                    stochastic_tau_max); while t - tau_i < 0 the stage is left alone.  A stage's update index
                                    (step-size schedule, T1 annealing, Adam's bias correction) counts the updates it has applied;
                                    pm_stage_desc.tau_fwd is the delay T1 divides by (the mean of the stage's distribution),
                                    tau_bkwd must be 0 and T2 has nothing to correct.  Needs PM_MB_MAJOR, n_micro <= 1,
                                    recompute_segment = 0, fuse_update = 0, else PM_ERR_UNSUPPORTED.  0: off. */
  int32_t materialize_backward;  /* 0 (default): the T2-corrected backward weights w - tau delta exist only inside the dgrad
                                    kernel, formed while the operand is loaded; no second copy of the weights is kept.
                                    1: the update that produces version v also writes bf16(w_v - tau delta_v) (fp32 with
                                    PM_F32) into one more slot of the stage's version queue, and the backward pass of the next
                                    step reads that copy: dgrad becomes a plain GEMM.  The same bits in every result (the
                                    correction is the same fp32 subtraction and product, rounded once), + one operand-type copy
                                    of the parameters in memory and 2 B per parameter of update traffic, less dgrad time.
                                    Needs PM_MB_MAJOR, recompute_segment = 0, stochastic_tau_max = 0, fuse_update = 0 and
                                    tau_bkwd = 0, else PM_ERR_UNSUPPORTED. */
} pm_config;

/* Flat state arenas, device, `count` elements each.  w: master weights; m: momentum /
 * Adam first moment; s: Adam second moment (may be NULL for SGD); delta: T2
 * accumulator; grad: gradient of the current tick (written by the backward phase);
 * w_lp: bfloat16 copy of w kept by the update kernel (may be NULL when
 * compute_dtype is PM_F32).  All 256-byte aligned. */
typedef struct {
  float* w;
  float* m;
  float* s;
  float* delta;
  float* grad;
  uint16_t* w_lp;
  uint64_t count;
} pm_arenas;

/* ---- parameter layout (host arithmetic only) ------------------------------------------ */

/* Number of elements a stage with these ops occupies in the arenas (padded). */
pm_status pm_stage_param_count(const pm_op_desc* ops, int32_t n_ops, uint64_t* count);
/* Offsets of op `op`'s two parameter tensors relative to the stage's param_offset: LINEAR (W, b);
 * LAYERNORM (gain, bias); EMBED (table, unused).  Ops without parameters give PM_ERR_INVALID_ARG. */
pm_status pm_op_param_offsets(const pm_op_desc* ops, int32_t n_ops, int32_t op,
                              uint64_t* w_off, uint64_t* b_off);

/* ---- pipeline context ------------------------------------------------------------------ */

/* Bytes the caller must provide: state_bytes = all arenas together (fp32 w, m, [s,] delta,
 * grad [+ bf16 copy]); ring_bytes = the per-stage delay rings of in-flight activations
 * (Section 2 / Appendix A: depth grows with 2(P-i)+1) or, for PM_MB_MAJOR, the activations of one
 * microbatch plus the per-stage queues of weight versions ((tau_fwd,i + 1) copies of the stage's
 * parameters in the GEMM operand type, and of its biases and LayerNorm parameters in fp32);
 * workspace_bytes = gradient mailboxes, per-stage scratch, target ring, loss log and tables. */
pm_status pm_query_bytes(const pm_config* cfg, const pm_stage_desc* stages,
                         uint64_t* state_bytes, uint64_t* ring_bytes, uint64_t* workspace_bytes);

/* Build a context.  The arenas must already hold the initial weights (w, and w_lp = bf16(w)
 * for PM_BF16), zero m/s/delta.  ring and workspace are device buffers of at least the
 * queried sizes, 256-byte aligned; the library zero-fills neither (contents are written
 * before they are read).  `stream` is a cudaStream_t passed as void*.
 * PM_ERR_SHAPE: stage i's first n_in differs from stage i-1's last n_out; for PM_BF16 a
 * dimension that is not a multiple of 8. */
pm_status pm_init_stages(pm_ctx** out, const pm_config* cfg, const pm_stage_desc* stages,
                         const pm_arenas* arenas, void* ring, uint64_t ring_bytes,
                         void* workspace, uint64_t workspace_bytes, void* stream);

/* Synchronous warm-up before PipeMare ("PipeMareW", Section 4: a number of epochs of the synchronous baseline with
 * the standard learning rate, then PipeMare).  Call once, before the first tick; n_microbatches >= 0 (0 = none,
 * the default).  The first n_microbatches microbatches then enter 2P ticks apart instead of one per tick, so
 * that the pipeline holds one microbatch at a time: each of them runs forward and backward on the same weights
 * and is applied before the next one enters, which is synchronous training with one microbatch per update.
 * Their updates use the base step size as it is (no T1 division), their backward passes no T2 correction, and
 * delta is left at zero.  For those microbatches pm_forward takes inputs at ticks 0, 2P, 4P, ... and NULL at the
 * ticks between (PM_ERR_STATE otherwise); from tick 2P * n_microbatches on the pipeline runs as described below,
 * with the T1 annealing counted from that point and the base step-size table and Adam's bias correction counted
 * from the first microbatch.  PM_ERR_STATE if a tick has already run.
 * PM_MB_MAJOR: the first n_microbatches calls of pm_step read the live weights in the forward pass too (the same
 * synchronous steps, without idle ticks); everything else as above. */
pm_status pm_set_warmup(pm_ctx* ctx, int64_t n_microbatches);

/* One tick = pm_forward, pm_backward, pm_update in this order (pm_step does all three).
 * inputs/targets (device) belong to the microbatch that enters the pipeline at this tick:
 * inputs is [T, n_in of stage 1] (float for PM_F32, bfloat16 for PM_BF16), or [T] int32 token ids when
 * stage 1 starts with EMBED ([2][T]: first stream, then second stream, when a stage embeds the second
 * stream); targets is [T, n_out of stage P] float (PM_LOSS_MSE) or [T] int32 class ids
 * (PM_LOSS_CE).  Both are copied before the call returns control to the
 * stream order, so the caller may overwrite them after any later call on the same stream.
 * Pass NULL for both to drain: N microbatches need N + 2P - 1 ticks (plus 2P - 1 ticks for each warm-up
 * microbatch, see pm_set_warmup).
 *
 * Tick s (0-based): stage i (1-based) runs the forward of microbatch s-(i-1) and the
 * backward and update of microbatch s-(2P-i).  Hence its forward for microbatch a reads
 * weight version max(0, a - tau_fwd,i) and its backward reads version a (Section 2.1 with
 * PipeMare's delays).
 *
 * PM_MB_MAJOR: one call of pm_step (or pm_forward, pm_backward, pm_update in this order) processes microbatch t
 * completely: pm_forward takes it through stages 1..P, stage i reading weight version max(0, t - tau_fwd,i) from
 * its queue; pm_backward computes the loss and walks stages P..1 against the live weights (version t, T2-corrected)
 * and forms every weight gradient; pm_update applies update t to all stages and pushes version t + 1 into the
 * queues.  inputs and targets must be given at every call (there is nothing to drain: NULL is PM_ERR_INVALID_ARG);
 * after N calls every stage has applied N updates.  In this order the w_lp arena is read once, at
 * initialisation (version 0); the live bf16 copy is the newest slot of the queue. */
pm_status pm_forward(pm_ctx* ctx, const void* inputs, const void* targets);
pm_status pm_backward(pm_ctx* ctx);
pm_status pm_update(pm_ctx* ctx);
pm_status pm_step(pm_ctx* ctx, const void* inputs, const void* targets);

/* Stochastic delay model (pm_config.stochastic_tau_max > 0): the delays of the NEXT step, one per stage (host array of
 * n_stages entries, copied during the call), each in [0, stochastic_tau_max], else PM_ERR_INVALID_ARG.  They stay in force
 * until the next call; before the first call every delay is 0.  PM_ERR_STATE outside that model. */
pm_status pm_set_delays(pm_ctx* ctx, const int32_t* delays);

/* Per-stage record of the last completed tick, written by the device kernels, for the
 * delay-bookkeeping check.  out[0..7] = forward microbatch (-1 if idle), weight version
 * the forward read, backward microbatch (-1 if idle), weight version the backward read,
 * updates applied so far, forward ring slot, backward ring slot, tick.  Synchronises.
 * PM_MB_MAJOR: the record of the last completed microbatch (both passes of every stage are active); out[7] is
 * that microbatch's index, out[5] the slot of the weight-version queue the forward read; with recompute_segment > 0
 * out[6] is the weight version the recomputation read; with stochastic_tau_max > 0 out[6] is the microbatch whose gradient
 * the stage applied in the last step (-1: none) and out[1] = out[3] the updates it had applied when the step began. */
pm_status pm_get_bookkeeping(pm_ctx* ctx, int32_t stage, int64_t* out8);

/* Copy losses of microbatches first_mb .. first_mb+n-1 to host_out.  The loss of microbatch
 * t is the one computed from its (stale) forward weights.  Synchronises.  PM_ERR_INVALID_ARG
 * if a requested microbatch has not finished or has left the device log. */
pm_status pm_get_losses(pm_ctx* ctx, float* host_out, int64_t first_mb, int64_t n);

/* Number of CUDA kernels this context has enqueued since pm_init_stages (for launch accounting). */
uint64_t pm_launch_count(pm_ctx* ctx);

/* Self-test of the failure path of the tensor-core kernels (PM_BF16 contexts).  Every wait of those kernels on a
 * barrier is bounded (about one second); when one expires the kernel records a code in a status word, stops, and
 * the next synchronising call returns PM_ERR_TIMEOUT.  This call exercises exactly that path without disturbing
 * anything: a one-thread kernel (no tensor memory, no copy in flight) waits with the given limit, in SM cycles, on
 * a barrier on which nothing arrives.  It synchronises the stream, returns PM_ERR_TIMEOUT when the expiry was
 * recorded and reported as designed (anything else is a defect), and clears the record, so the context stays
 * usable.  Use a small limit (a few million cycles = milliseconds). */
pm_status pm_selftest_wait_timeout(pm_ctx* ctx, int64_t limit_cycles);

/* Optional timing of the tick's kernels by class, with CUDA events recorded on the context's stream around each
 * launch (up to 8192 launches between reads; later ones are not recorded).  pm_profile_read synchronises the
 * stream, writes the summed milliseconds and the number of timed launches per class (arrays of PM_PROF_CLASSES
 * entries) and clears the record. */
enum { PM_PROF_SCHEDULE = 0, PM_PROF_INGEST, PM_PROF_PRE_FWD, PM_PROF_GEMM_FWD, PM_PROF_ATTN_FWD, PM_PROF_POST_FWD,
       PM_PROF_LOSS, PM_PROF_ATTN_BWD, PM_PROF_ACT_BWD, PM_PROF_WGRAD, PM_PROF_DGRAD, PM_PROF_PRE_BWD, PM_PROF_UPDATE,
       PM_PROF_CLASSES };
pm_status pm_profile_enable(pm_ctx* ctx, int32_t on);
pm_status pm_profile_read(pm_ctx* ctx, float* ms_by_class, int64_t* launches_by_class);

const char* pm_last_error(pm_ctx* ctx);   /* never NULL; ctx may be NULL (global message) */
void pm_destroy(pm_ctx* ctx);

/* ---- the fused update on its own ---------------------------------------------------------- */

/* One fused PipeMare update (T1 step size, momentum or Adam, T2 accumulator refresh,
 * bf16 copy) over the flat arenas of n_stages stages, every stage at update index k.
 * stage_offsets / stage_counts (host, elements, offsets multiples of PM_ALIGN_ELEMS)
 * delimit the slices; elements between a slice's end and the next offset are padding
 * and must hold zeros.  tau_fwd / tau_bkwd: host arrays.  From cfg the optimiser,
 * betas, eps, T1/T2 settings and alpha are read.  `workspace` is a device buffer of at
 * least pm_update_flat_workspace_bytes(n_stages) bytes that receives the stage table.
 * Asynchronous on `stream`.  PM_ERR_INVALID_ARG for alpha_by_step with alpha_len < 1;
 * PM_ERR_NOMEM for a slice that does not fit the arenas. */
uint64_t pm_update_flat_workspace_bytes(int32_t n_stages);
pm_status pm_update_flat(const pm_arenas* arenas, const uint64_t* stage_offsets,
                         const uint64_t* stage_counts, const int32_t* tau_fwd,
                         const int32_t* tau_bkwd, int32_t n_stages, const pm_config* cfg,
                         int64_t k, void* workspace, uint64_t workspace_bytes, void* stream);

/* The same update for callers that cannot allocate device memory (the paper has no counterpart;
 * this is a deployment convenience).  Who needs it: code running under a framework whose caching
 * allocator already owns the device, real-time loops that must not allocate after start-up, and
 * plug-ins that receive tensors but no allocator -- none of them can produce the `workspace`
 * pm_update_flat asks for.  Here the stage table lives in a fixed array inside the library
 * (about 35 KB on every GPU that loads the library, held until the process exits), so the call
 * takes only the arenas.  Arguments and results are those of pm_update_flat.
 *   - At most pm_update_flat_static_max_stages() (= 256) stages; more is PM_ERR_NOMEM with a
 *     message that says so.  pm_update_flat_static_last_error() returns the message (per thread).
 *   - Neither this call nor anything it uses calls cudaMalloc, cudaFree or an allocating library
 *     routine; host staging is a fixed per-thread buffer.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside any CUDA stream capture.
 *   - All calls on a device share the one array, and it keeps the previous call's contents; each
 *     call rewrites the whole table, counters included, before its kernels read it.  Two calls
 *     whose GPU work overlaps (different streams, or threads racing on one device) would
 *     overwrite each other's table: issue them on one stream or serialise them. */
int32_t pm_update_flat_static_max_stages(void);
const char* pm_update_flat_static_last_error(void);
pm_status pm_update_flat_static(const pm_arenas* arenas, const uint64_t* stage_offsets,
                                const uint64_t* stage_counts, const int32_t* tau_fwd,
                                const int32_t* tau_bkwd, int32_t n_stages, const pm_config* cfg,
                                int64_t k, void* stream);

const char* pm_status_string(pm_status s);

#ifdef __cplusplus
}
#endif
#endif /* PIPEMARE_H */
