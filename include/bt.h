/*
 * bt -- FP32 GPT-2 training step for NVIDIA B200 (sm_100a), C ABI.
 *
 * The library runs the forward pass, the backward pass and the AdamW update of a
 * decoder-only pre-LayerNorm transformer with tied embeddings (the paper's evaluation
 * model: architecture-figure caption and hyper-parameter table of Section 5; step
 * structure of Algorithm 1: forward, cross-entropy against the target, backward,
 * optimizer step).  Every step of the path runs in hand-written CUDA kernels; there is
 * no CPU fallback.
 *
 * Conventions that hold for every entry point
 * -------------------------------------------
 * Memory    All array arguments are DEVICE pointers unless the name starts with `h_`
 *           (host).  The caller owns every buffer, including the model workspace and
 *           any `scratch` argument; the library allocates no device memory.  Device
 *           pointers must be 16-byte aligned.  Arrays are row-major FP32 unless
 *           declared int32.
 * Streams   `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *           stream).  Calls enqueue work and return; only calls with a non-NULL host
 *           output pointer (h_loss, h_grad_norm) synchronise the stream.
 * Errors    Every call returns a bt_status.  Arguments are validated on the host
 *           before any launch; nothing is thrown or aborted.  bt_last_error() returns
 *           a thread-local description of the last failure.  Kernels that wait on
 *           hardware barriers bound every wait; a wait that runs out sets a device
 *           error word that the next synchronising call reports as
 *           BT_ERR_DEVICE_TIMEOUT.  An error word is reported once and then cleared.
 * Split     The tensor-core GEMMs compute FP32 products as three TF32 products
 *           (a_hi*b_hi + a_hi*b_lo + a_lo*b_hi, FP32 accumulate).  Operands are therefore
 *           stored as two FP32 planes, `hi` = the value rounded to the nearest TF32 number
 *           (low 13 mantissa bits zero) and `lo` = value - hi (exact).  A "split" array of R x C values is
 *           [2][R][C]: plane 0 = hi, plane 1 = lo.  Kernels that produce GEMM operands
 *           can write the split form directly.
 * Tokens    Token and target ids must lie in [0, vocab_size).  No kernel ever indexes
 *           with an id outside that range: such an id is treated as id 0 and its
 *           position is recorded in a device error word, which the next synchronising
 *           call of the model (h_loss, h_grad_norm, bt_get_loss) reports as
 *           BT_ERR_INVALID_ARG.  Entry points that receive the ids in HOST memory
 *           (bt_train_step_host, the loader) check them before anything is enqueued.
 *           With BT_FLAG_DEBUG in the configuration, or BT_DEBUG=1 in the environment,
 *           bt_forward, bt_backward and bt_adamw_step synchronise before returning and
 *           report any device error at the call that caused it.
 */
#ifndef BT_H_
#define BT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define BT_API __attribute__((visibility("default")))
#else
#define BT_API
#endif

typedef struct bt_model bt_model; /* opaque host object */

typedef enum {
    BT_OK = 0,
    BT_ERR_INVALID_ARG = 1,    /* null / misaligned pointer, bad size, bad configuration */
    BT_ERR_UNSUPPORTED = 2,    /* valid request the compiled kernels do not cover */
    BT_ERR_OOM = 3,            /* workspace or scratch too small */
    BT_ERR_CUDA = 4,           /* a CUDA runtime / driver call failed */
    BT_ERR_DEVICE_TIMEOUT = 5, /* a bounded device-side wait ran out */
    BT_ERR_NOT_FOUND = 6       /* unknown tensor / activation name */
} bt_status;

/* Model configuration ("layers / d_model / heads / seq_len / vocab").  The MLP width is
 * 4 * d_model.  padded_vocab_size >= vocab_size is the number of rows of the tied
 * embedding / LM-head matrix; the softmax and the loss run over all padded columns. */
typedef struct {
    int32_t n_layers, d_model, n_heads, seq_len, vocab_size, padded_vocab_size, max_batch;
    uint32_t flags;
} bt_config;

enum {
    BT_FLAG_GELU_TANH = 1u,  /* tanh-form GELU instead of the exact erf form */
    BT_FLAG_GEMM_SIMT = 2u,  /* plain FP32 FMA GEMM (bring-up reference) instead of tcgen05 */
    BT_FLAG_ATTN_SIMT = 4u,  /* plain FP32 FMA attention (bring-up reference) */
    BT_FLAG_GEMM_PAIR = 8u,  /* per-op GEMM calls: 256-row tiles on CTA pairs wherever M >= 256 */
    BT_FLAG_GEMM_SINGLE = 16u, /* per-op GEMM calls: 128-row tiles on single CTAs only (default: planner) */
    BT_FLAG_DEBUG = 32u,      /* every step call synchronises and reports device errors (ids, waits) itself */
    BT_FLAG_RECOMPUTE_LN = 64u, /* do not keep the LayerNorm outputs of every layer (2 x 8 B per token and feature):
                                  the backward pass re-runs the LayerNorm forward from the saved input and statistics
                                  before the two weight-gradient products that read them (same bits, about 1 % more time) */
    BT_FLAG_LOGITS_IN_PLACE = 128u, /* the hi plane of the logit gradient is written over the logits (4 B per token and
                                  vocabulary entry less); the "logits" activation is then unavailable.  padded_vocab <= 51200 */
    BT_FLAG_RECOMPUTE_GELU = 256u /* do not keep the GELU output planes of every layer (8 B per token and MLP feature):
                                  the backward pass forms them again from the kept pre-activation (same bits, about 2 % more time) */
};

/* AdamW hyper-parameters (hyper-parameter table, "Optimization" column).  grad_clip <= 0
 * disables global-norm clipping. */
typedef struct {
    float lr, beta1, beta2, eps, weight_decay, grad_clip;
} bt_adamw_config;

/* ----------------------------------------------------------------------------------
 * Model lifetime
 * -------------------------------------------------------------------------------- */

/* Bytes of device workspace a model of this configuration needs (parameters, gradients,
 * both moments, split weight copies, activations for max_batch sequences, scratch).
 * Returns 0 for an invalid configuration. */
BT_API size_t bt_workspace_bytes(const bt_config* cfg);
/* The same total by section (the paper's Evaluation reports the memory footprint beside the
 * throughput): part 0 parameters + gradients + both moments, 1 TF32 hi/lo planes of the weights in
 * both orientations, 2 gradient accumulator of the micro-step loop and small tables, 3 activations
 * kept for the backward pass (max_batch sequences), 4 logits, their gradient planes and per-row
 * losses, 5 backward temporaries reused by every layer, 6 scratch (split-K partial sums, reduction
 * partials, id staging, embedding table).  The seven parts add up to bt_workspace_bytes; 0 for an
 * invalid configuration or part. */
BT_API size_t bt_workspace_part_bytes(const bt_config* cfg, int32_t part);

/* Builds the host-side model over a caller-allocated device workspace of at least
 * bt_workspace_bytes(cfg) bytes, 256-byte aligned.  Moments and the step counter start
 * at zero; parameters are NOT initialised (load them through bt_tensor_ptr, or call
 * bt_model_init).  All later calls on the model enqueue on `stream`.
 * Errors: BT_ERR_INVALID_ARG (bad cfg: d_model % n_heads, d_model % 32, head_dim not in
 * {16,32,64,128}, padded_vocab % 32, seq_len or max_batch < 1, ...), BT_ERR_OOM. */
BT_API bt_status bt_model_create(const bt_config* cfg, void* d_workspace, size_t workspace_bytes,
                                 void* stream, bt_model** out);

/* Frees the host object only; the workspace stays with the caller. */
BT_API void bt_model_destroy(bt_model* m);

/* Fills the parameters on the device with the paper's initialisation (hyper-parameter
 * table: weight std 0.02, residual projections 0.02/sqrt(2*n_layers); biases 0, LayerNorm
 * gain 1 / shift 0) from a counter-based generator, and zeroes moments and step counter.
 * Meant for benchmarks; parity tests load explicit arrays instead. */
BT_API bt_status bt_model_init(bt_model* m, uint64_t seed);

/* Parameter registry.  Order: wte [Vp,C], wpe [T,C], then per block l: h{l}.ln1.g, h{l}.ln1.b,
 * h{l}.attn.qkv.w [3C,C], h{l}.attn.qkv.b, h{l}.attn.proj.w [C,C], h{l}.attn.proj.b, h{l}.ln2.g,
 * h{l}.ln2.b, h{l}.mlp.fc.w [4C,C], h{l}.mlp.fc.b, h{l}.mlp.proj.w [C,4C], h{l}.mlp.proj.b, then
 * lnf.g, lnf.b.  Weights are [out,in] row-major.  `decay` is 1 for the two-dimensional
 * tensors (weight decay applies), 0 otherwise.  The LM head is wte (tied). */
BT_API int32_t bt_num_tensors(const bt_model* m);
BT_API bt_status bt_tensor_info(const bt_model* m, int32_t index, const char** name, int64_t* numel,
                                int32_t* decay);
/* kind: 0 parameter, 1 gradient, 2 first moment, 3 second moment.  The pointer addresses
 * `numel` floats inside the workspace and stays valid for the model's lifetime. */
BT_API bt_status bt_tensor_ptr(bt_model* m, const char* name, int32_t kind, float** d_ptr);

/* Activations of the last forward/backward, for tests: per-layer "x", "qkv" (raw; written only
 * when head_dim is neither 64 nor 128 or a reference-kernel flag is set), "x1", "h" (the MLP
 * pre-activation; without BT_FLAG_RECOMPUTE_GELU and BT_FLAG_GEMM_SIMT the array holds GELU'(h),
 * all the backward pass needs of it),
 * "ln1.mean", "ln1.rstd", "ln2.mean", "ln2.rstd", "lse"; split per-layer "qkv_split", "a", "o", "m", "g"
 * (pointer to the hi plane; lo plane follows at +numel); global "xL", "logits", "losses",
 * split "xf", "dlogits".  `numel` (nullable) receives the element count of one plane for
 * the current batch. */
BT_API bt_status bt_activation_ptr(bt_model* m, const char* name, int32_t layer, float** d_ptr,
                                   int64_t* numel);

/* Optimizer step counter t (number of AdamW updates applied so far). */
BT_API int64_t bt_get_step(const bt_model* m);
BT_API bt_status bt_set_step(bt_model* m, int64_t t);

/* ----------------------------------------------------------------------------------
 * The training step (Algorithm 1, loop body: forward + loss, backward, optimizer step)
 * -------------------------------------------------------------------------------- */

/* Forward pass and mean cross-entropy of B sequences: d_tokens, d_targets are int32
 * [B, seq_len].  If h_loss is non-NULL the stream is synchronised and the loss written. */
BT_API bt_status bt_forward(bt_model* m, const int32_t* d_tokens, const int32_t* d_targets, int32_t B,
                            float* h_loss);

/* Gradient of the last bt_forward's loss with respect to every parameter (overwrites the
 * gradient tensors). */
BT_API bt_status bt_backward(bt_model* m);

/* Global-norm clip (scale = min(1, clip / (norm + 1e-6))) followed by one AdamW update of
 * every tensor in a single launch: p <- p (1 - lr wd [decay]); m, v moment updates on the
 * clipped gradient; p <- p - lr mhat / (sqrt(vhat) + eps), t incremented first (t = 1 on
 * the first call).  h_grad_norm (nullable) receives the unclipped norm (synchronises). */
BT_API bt_status bt_adamw_step(bt_model* m, const bt_adamw_config* opt, float* h_grad_norm);

/* bt_forward + bt_backward + bt_adamw_step. */
BT_API bt_status bt_train_step(bt_model* m, const int32_t* d_tokens, const int32_t* d_targets, int32_t B,
                               const bt_adamw_config* opt, float* h_loss);

/* Same step with HOST token / target buffers (int32 [B, seq_len], pinned for a truly
 * asynchronous copy): the ids are checked against [0, vocab_size) on the host
 * (BT_ERR_INVALID_ARG names the first offender; nothing is enqueued), then copied into the
 * workspace on the model's stream. */
BT_API bt_status bt_train_step_host(bt_model* m, const int32_t* h_tokens, const int32_t* h_targets,
                                    int32_t B, const bt_adamw_config* opt, float* h_loss);

/* Gradient accumulation (Algorithm 1: grad_accum_steps micro-steps, then one optimizer step).
 * bt_micro_step runs bt_forward + bt_backward on micro-batch micro_index of n_micro equally
 * sized micro-batches and folds its gradient, weighted 1/n_micro, into an accumulator inside
 * the workspace; after the call with micro_index == n_micro - 1 the gradient tensors hold the
 * gradient of the mean loss over all n_micro * B sequences and the loss word holds that mean
 * (reading: the paper does not say how micro-batch losses are weighted; the mean over the global
 * batch is the definition that makes the result independent of the split).  Call the micro-steps
 * in order 0 .. n_micro - 1, then bt_adamw_step.  h_loss (nullable, synchronises): this
 * micro-batch's loss, on the last micro-step the mean over all of them. */
BT_API bt_status bt_micro_step(bt_model* m, const int32_t* d_tokens, const int32_t* d_targets, int32_t B,
                               int32_t micro_index, int32_t n_micro, float* h_loss);

/* n_micro micro-steps over d_tokens / d_targets of shape [n_micro * B, seq_len] (device),
 * then bt_adamw_step; h_loss (nullable) receives the mean loss. */
BT_API bt_status bt_train_step_accum(bt_model* m, const int32_t* d_tokens, const int32_t* d_targets, int32_t B,
                                     int32_t n_micro, const bt_adamw_config* opt, float* h_loss);

/* ----------------------------------------------------------------------------------
 * Data-parallel gradient exchange (Distributed Execution, "Data-Parallel Orchestration",
 * Algorithm 1 "Distributed Data Parallel Training Step")
 * --------------------------------------------------------------------------------
 * Every rank holds a replica and its own batch rows; on the synchronising micro-step the
 * gradients are averaged over the ranks in buckets, each bucket as soon as the backward pass has
 * finished it, on a second stream, ordered against the compute stream by events only (the host
 * never blocks), and the optimizer step waits for the last bucket.
 *
 * The gradients of a model lie in ONE flat arena in registry order and the backward pass finishes
 * them in the reverse of that order, so a bucket is a contiguous range of the arena and is reduced
 * in place: there is no copy into bucket memory and no scatter back.  bt_ddp_plan_* is the host-only
 * part -- which range each bucket covers, which tensors it waits for, and the in-order launch gate
 * -- usable (and tested) without a GPU:
 *   bt_ddp_plan_create    buckets for `cfg` under a cap of bucket_cap_bytes (the paper uses 25 MB):
 *                         tensors are taken in gradient-ready order (last registry entry first) and
 *                         a bucket is closed when the next tensor would exceed the cap; a tensor
 *                         larger than the cap is cut into equal ranges under the cap.  Bucket 0 is ready first.
 *   bt_ddp_plan_bucket    range (offset and count, in floats, inside the arena) of bucket b and the
 *                         number of tensors it waits for.
 *   bt_ddp_plan_tensor    arena offset and padded length of registry tensor i (every tensor starts
 *                         on a multiple of 1024 floats; the padding is zero and stays zero).
 *   bt_ddp_plan_reset     before a backward pass: every bucket pending again, next bucket = 0.
 *   bt_ddp_plan_mark_ready  "the gradient of tensor i is final" (the hook of Algorithm 1): returns
 *                         how many buckets may be launched NOW, in order, and writes their indices
 *                         to `launch` (room for bt_ddp_plan_num_buckets entries).  A bucket is
 *                         launched only after all buckets before it, whatever order the marks
 *                         arrive in; marking a tensor twice is an error (-1).
 * bt_ddp_attach connects a model to an all-reduce: during bt_backward the library marks tensors
 * ready as the kernels that finish them are enqueued; for every released bucket it records an
 * event on the model's stream, makes `comm_stream` wait for it and calls
 *     fn(user, d_grads + offset, count, bucket, comm_stream)
 * which must ENQUEUE on comm_stream an in-place all-reduce of `count` floats that leaves the
 * AVERAGE over the ranks (for example ncclAllReduce with ncclAvg), must not block the host, and
 * returns 0 on success.  After the last bucket the model's stream is made to wait for
 * comm_stream, so bt_adamw_step sees the averaged gradients.  With bt_micro_step /
 * bt_train_step_accum only the last micro-step exchanges gradients (the others run without any
 * communication), and its accumulation is folded in bucket by bucket so that the exchange still
 * overlaps the backward pass.  The loss every rank reports stays its own.  Start every rank from
 * the same parameters (bt_arena_ptr gives the parameter arena as one range to broadcast).
 * bt_ddp_detach returns the model to single-replica operation. */
typedef struct bt_ddp_plan bt_ddp_plan;
typedef int32_t (*bt_allreduce_fn)(void* user, float* d_buf, int64_t count, int32_t bucket, void* comm_stream);
BT_API bt_status bt_ddp_plan_create(const bt_config* cfg, int64_t bucket_cap_bytes, bt_ddp_plan** out);
BT_API void bt_ddp_plan_destroy(bt_ddp_plan* plan);
BT_API int32_t bt_ddp_plan_num_buckets(const bt_ddp_plan* plan);
BT_API bt_status bt_ddp_plan_bucket(const bt_ddp_plan* plan, int32_t b, int64_t* offset, int64_t* count,
                                    int32_t* n_tensors);
BT_API bt_status bt_ddp_plan_tensor(const bt_ddp_plan* plan, int32_t tensor, int64_t* offset, int64_t* padded_len);
BT_API void bt_ddp_plan_reset(bt_ddp_plan* plan);
BT_API int32_t bt_ddp_plan_mark_ready(bt_ddp_plan* plan, int32_t tensor, int32_t* launch);
BT_API bt_status bt_ddp_attach(bt_model* m, int64_t bucket_cap_bytes, bt_allreduce_fn fn, void* user,
                               void* comm_stream);
BT_API bt_status bt_ddp_detach(bt_model* m);
/* The four flat arenas (kind: 0 parameters, 1 gradients, 2 / 3 moments): device pointer and length
 * in floats, padding included. */
BT_API bt_status bt_arena_ptr(bt_model* m, int32_t kind, float** d_ptr, int64_t* count);

/* Learning rate of optimizer step `step` (1-based) from the hyper-parameter table's max / min
 * learning rate, warmup steps and training steps.  Reading (the paper gives the four numbers, not
 * the curve): linear warmup max_lr * step / warmup_steps, then a half cosine from max_lr at
 * step = warmup_steps to min_lr at step = max_steps, min_lr afterwards.  Host arithmetic only. */
typedef struct {
    float max_lr, min_lr;
    int32_t warmup_steps, max_steps;
} bt_lr_schedule;
BT_API float bt_lr_at(const bt_lr_schedule* s, int64_t step);

/* Prefetching batch production (Implementation, "Data Loader", Algorithm 2 "Double-Buffered Batch
 * Production").  The token stream is a list of shards (host int32 arrays the caller keeps alive,
 * e.g. memory-mapped files).  The algorithm fixes which windows a rank sees: rank r of `world`
 * starts at position B*T*r of shard 0; each batch is the window [pos, pos + B*T) as tokens and
 * [pos + 1, pos + B*T + 1) as targets; pos advances by B*T*world; the next shard is opened when
 * fewer than B*T*world + 1 tokens remain after the advance.  Every shard must hold at least
 * B*T*world + 1 tokens.  Here that sequence is computed in closed form (a rank takes
 * max(1, floor((len - 1 - B*T*r) / (B*T*world))) windows from a shard of `len` tokens), and the
 * two buffers of the algorithm are a ring of n_slots slots (2 <= n_slots <= 8; 2 is the paper's
 * double buffering) with one "copy landed" and one "consumer done" event per slot:
 *   d_buffers: device, n_slots * 2 * B*T int32 (tokens and targets of every slot), caller-owned;
 *   h_pinned:  page-locked host memory of the same size, or NULL: then windows are copied straight
 *              from the shards, synchronously, with identical results;
 *   vocab_size: if > 0, every id is checked against [0, vocab_size) while it is staged; a window
 *              with an id outside makes the staging call return BT_ERR_INVALID_ARG (shard and
 *              position in bt_last_error()) and the loader unusable; 0 = unchecked;
 *   compute_stream: the stream the consumer (bt_train_step ...) runs on.
 * bt_loader_next hands out the oldest filled slot: device pointers to its tokens and targets and
 * the slot number; the compute stream is made to wait for the slot's copy.  The first call stages
 * all n_slots slots.  The pointers stay valid until the slot is released.
 * bt_loader_release(slot): call it after the LAST kernel that reads the slot has been enqueued on
 * the compute stream.  It records the slot's "consumer done" event there and immediately stages
 * the next window into the slot on the loader's own stream, which waits for that event: a slot is
 * never overwritten before its readers have finished, however far the host runs ahead, and the host
 * never rewrites a staging buffer before the copy out of it has run.  With every slot lent out and
 * none released, bt_loader_next returns BT_ERR_INVALID_ARG.
 * bt_loader_plan is the window sequence alone (host only): the shard index and position of the
 * first n_batches windows. */
typedef struct bt_loader bt_loader;
BT_API bt_status bt_loader_plan(const int64_t* shard_lens, int32_t n_shards, int32_t B, int32_t T, int32_t rank,
                                int32_t world, int32_t n_batches, int32_t* out_shard, int64_t* out_pos);
BT_API bt_status bt_loader_create(const int32_t* const* shards, const int64_t* shard_lens, int32_t n_shards,
                                  int32_t B, int32_t T, int32_t rank, int32_t world, int32_t vocab_size,
                                  int32_t n_slots, int32_t* d_buffers, int32_t* h_pinned, void* compute_stream,
                                  bt_loader** out);
BT_API bt_status bt_loader_next(bt_loader* loader, const int32_t** d_tokens, const int32_t** d_targets,
                                int32_t* slot);
BT_API bt_status bt_loader_release(bt_loader* loader, int32_t slot);
BT_API void bt_loader_destroy(bt_loader* loader);

/* Position of the first id outside [0, vocab_size) in a HOST array of n ids, -1 if all are valid,
 * -2 for bad arguments.  Host arithmetic only (what bt_train_step_host and the loader run). */
BT_API int64_t bt_first_invalid_id(const int32_t* h_ids, int64_t n, int32_t vocab_size);

/* Self-test of the error path of the bounded device-side waits (the paper's fault-handling layer
 * is an operations subsystem; this covers only the library's own promise that a kernel never
 * waits forever).  One warp runs the library's barrier wait, with limit_ms (0 < limit_ms <= 1000)
 * as its limit, on a barrier nothing arrives at -- no copy or tensor-memory operation is in
 * flight, the kernel returns normally -- and the call returns what the next synchronising call
 * of a real step would: BT_ERR_DEVICE_TIMEOUT (bt_last_error() names code 900).  The model stays
 * usable.  Synchronises the stream. */
BT_API bt_status bt_selftest_bounded_wait(bt_model* m, float limit_ms);

/* Measurement aid (Appendix "Hardware and Benchmarking Methodology" asks for measured, not
 * nominal, peaks): n_ctas CTAs each issue `iters` tcgen05.mma.kind::tf32 instructions of
 * M = 128, N = 256, K = 8 (operands in shared memory, two alternating accumulators) and store the
 * SM clocks from first issue to last completion in d_clocks[cta] (device int64, -1 if the bounded
 * completion wait ran out, which also sets *d_err (device int32, zeroed by the caller) to 901).
 * 262,144 MACs per instruction / (clocks / iters) is the dense TF32 rate of one SM in MAC per
 * clock; times 2 x SMs x SM clock it is the TF32 peak, and a third of that the 3xTF32 peak the
 * GEMM roofline is scaled with.  Asynchronous; one CTA per SM when n_ctas <= the SM count. */
BT_API bt_status bt_probe_tf32_mma_rate(int32_t n_ctas, int32_t iters, int64_t* d_clocks, int32_t* d_err,
                                        void* stream);

/* The same kind of measurement for the ISSUE rate: in each of n_ctas CTAs, `issuers` threads (1-4,
 * in different warps) each issue `iters` MMAs of M = 128, N = n (64, 128 or 256), K = 8 with the A
 * operand in shared memory or (a_in_tmem, n <= 128) in tensor memory; d_clocks[4 * cta + i] (device
 * int64, 4 * n_ctas entries) receives thread i's clocks from its first issue to the completion of
 * its last MMA (-1 and *d_err = 902 if the bounded wait ran out).  max_i clocks / (iters x issuers)
 * is the cost of one MMA with that many issuing threads: the attention kernels' division of their
 * products among issuing threads rests on it (Appendix "Hardware and Benchmarking Methodology").
 * Asynchronous. */
BT_API bt_status bt_probe_mma_issue_rate(int32_t n, int32_t a_in_tmem, int32_t issuers, int32_t n_ctas, int32_t iters,
                                         int64_t* d_clocks, int32_t* d_err, void* stream);

/* Synchronises and reads the loss of the last forward. */
BT_API bt_status bt_get_loss(bt_model* m, float* h_loss);

/* Number of kernels the library has launched on behalf of this model since creation. */
BT_API int64_t bt_launch_count(const bt_model* m);

BT_API const char* bt_last_error(void);

/* Optional per-kernel timing of the step (the paper's profiler module reports exact
 * kernel-level timings).  While enabled, every launch group of bt_forward / bt_backward /
 * bt_adamw_step is bracketed by two CUDA events on the model's stream and tagged with a
 * category and its algorithmic FLOPs and bytes.  bt_profile_enable synchronises and clears the
 * records; bt_profile_read synchronises and returns, for one category, the summed event time
 * in milliseconds, the number of launch groups, and their summed algorithmic FLOPs and bytes
 * (any output may be NULL).  Events are host objects; no device memory is allocated. */
BT_API bt_status bt_profile_enable(bt_model* m, int32_t on);
BT_API int32_t bt_profile_num_categories(void);
BT_API const char* bt_profile_category_name(int32_t category);
BT_API bt_status bt_profile_read(bt_model* m, int32_t category, double* ms_total, int64_t* launches, double* flops,
                                 double* bytes);

/* ----------------------------------------------------------------------------------
 * Per-operation entry points (the kernels of the step, one at a time, for tests and
 * micro-benchmarks).  Optional outputs may be NULL.  `*_split` outputs are [2][rows][cols].
 * -------------------------------------------------------------------------------- */

/* x[n,:] = wte[tok[n],:] + wpe[n mod T,:], one IEEE single-precision add per element
 * (Evaluation, GPT-2 architecture figure: token embedding plus learned position embedding feed the
 * first decoder block).  wte has V rows; an id outside [0, V) is read as id 0 and its position + 1
 * is stored in *d_bad (device int32, nullable, zeroed by the caller; first writer wins). */
BT_API bt_status bt_op_embedding_fwd(const int32_t* tok, const float* wte, const float* wpe, int64_t N,
                                     int32_t T, int32_t C, int32_t V, float* x, int32_t* d_bad, void* stream);

/* Backward of the above (Evaluation, GPT-2 architecture figure caption: the embeddings are
 * weight-tied, so the gradient of the tied matrix is the LM-head part plus this scatter-add):
 * dwte[tok[n],:] += dx[n,:] summed in ascending n; dwpe[t,:] = sum_b dx[b*T+t,:].
 * dwte (V rows) is accumulated into (the tied LM-head gradient is already there), dwpe is
 * overwritten.  Deterministic and free of atomics: positions are grouped by id inside chunks of
 * 128 positions, one partial row per (chunk, id) is written to scratch, and the partial rows of an
 * id are added in chunk order.  Ids outside [0, V) count as id 0 (as in the forward).
 * scratch: device, bt_op_embedding_bwd_scratch_bytes(N, C, V) bytes, 256-byte aligned, caller-owned,
 * contents irrelevant on entry.  N % T == 0, N <= 2^24. */
BT_API size_t bt_op_embedding_bwd_scratch_bytes(int64_t N, int32_t C, int32_t V);
BT_API bt_status bt_op_embedding_bwd(const int32_t* tok, const float* dx, int64_t N, int32_t T, int32_t C,
                                     int32_t V, float* dwte, float* dwpe, void* scratch, size_t scratch_bytes,
                                     void* stream);

/* LayerNorm forward (Kernel Design and Optimization: the memory-bound kernels, reductions kept
 * inside a warp; Appendix "Performance Benchmarks", LayerNorm Forward):
 * y = gamma * (x - mean) * rstd + beta over the C features of each of N rows; biased
 * variance, eps = 1e-5.  C % 4 == 0. */
BT_API bt_status bt_op_layernorm_fwd(const float* x, const float* gamma, const float* beta, int64_t N,
                                     int32_t C, float* y, float* y_split, float* mean, float* rstd,
                                     void* stream);

/* LayerNorm backward (Appendix "Performance Benchmarks", LayerNorm Backward; the residual add is
 * the pre-normalised block's skip connection of the GPT-2 architecture figure):
 * dx = rstd * (dxhat - mean_c dxhat - xhat * mean_c(dxhat * xhat)) [+ dres], dxhat = dy * gamma;
 * dgamma = sum_n dy * xhat, dbeta = sum_n dy (overwritten, fixed summation order). */
BT_API size_t bt_op_layernorm_bwd_scratch_bytes(int64_t N, int32_t C);
BT_API bt_status bt_op_layernorm_bwd(const float* dy, const float* x, const float* gamma, const float* mean,
                                     const float* rstd, const float* dres, int64_t N, int32_t C, float* dx,
                                     float* dx_split, float* dgamma, float* dbeta, void* scratch,
                                     size_t scratch_bytes, void* stream);
/* The same, plus dx_colsum[C] (device) = the column sums of the dx written (residual included):
 * in the pre-normalised decoder block (Evaluation, GPT-2 architecture figure caption) that dx is
 * the gradient at a residual-stream position, so its
 * column sums are the bias gradient of the projection that wrote to that position.  Same scratch. */
BT_API bt_status bt_op_layernorm_bwd_colsum(const float* dy, const float* x, const float* gamma, const float* mean,
                                            const float* rstd, const float* dres, int64_t N, int32_t C, float* dx,
                                            float* dx_split, float* dgamma, float* dbeta, float* dx_colsum,
                                            void* scratch, size_t scratch_bytes, void* stream);

/* Dense FP32 GEMM with 3xTF32 split accumulation on the tensor cores (Implementation, "Native
 * GEMM Library": one library serves the QKV, attention-output and MLP projections in all forward
 * and backward layouts, including the irregular weight-gradient shapes):  D[M,N] = op(A) op(B) (+ bias[N]) (+ residual[M,N]).
 *   BT_GEMM_NT: A [M,K], B [N,K]   (forward:  Y  = X W^T)
 *   BT_GEMM_NN: A [M,K], B [K,N]   (backward: dX = dY W)
 *   BT_GEMM_TN: A [K,M], B [K,N]   (backward: dW = dY^T X)
 * M, N, K multiples of 4 (NN/TN: the contiguous extents multiples of 32).
 * flags: BT_FLAG_GEMM_SIMT selects the FP32 FMA reference kernel; BT_FLAG_GEMM_PAIR / BT_FLAG_GEMM_SINGLE
 * pin the tensor-core tile (256 rows on a CTA pair / 128 rows on one CTA) instead of letting the
 * wave-model planner choose. */
enum { BT_GEMM_NT = 0, BT_GEMM_NN = 1, BT_GEMM_TN = 2 };

/* x_split[0][i] = hi(x[i]), x_split[1][i] = lo(x[i]) for n values (n % 4 == 0).  The paper has no
 * counterpart: this is the operand format of the 3xTF32 products above. */
BT_API bt_status bt_op_split(const float* x, int64_t n, float* x_split, void* stream);

/* The GEMM as the training step calls it: operands already stored as hi/lo planes
 * (A_split is [2][rows_A][cols_A], B_split likewise).  Asynchronous; `scratch` (256-byte
 * aligned, bt_op_gemm_split_scratch_bytes() bytes) holds split-K partial sums and the device
 * error word that bt_op_gemm_check reads (it synchronises the stream and returns
 * BT_ERR_DEVICE_TIMEOUT if a bounded wait inside the kernel ran out). */
BT_API size_t bt_op_gemm_split_scratch_bytes(void);
BT_API bt_status bt_op_gemm_split(int32_t layout, int64_t M, int64_t N, int64_t K, const float* A_split,
                                  const float* B_split, float* D, const float* bias, const float* residual,
                                  void* scratch, size_t scratch_bytes, uint32_t flags, void* stream);
/* The same, and D_act_split [2][M][N] (device) receives the TF32 hi/lo planes of act(D) from the
 * same epilogue: act 0 = D itself, 1 = GELU(D) in the erf form, 2 = the tanh form; 3 / 4 = as
 * 1 / 2, and D receives GELU'(output) instead of the output (tensor-core kernels only).  The
 * training step uses 3 / 4 for the MLP up-projection (the GELU feed-forward sublayer of the GPT-2
 * architecture figure: g = GELU(h), h = m Wfc^T + b, is the next GEMM's operand, and GELU'(h) is
 * all the backward pass needs of h), 1 / 2 where h itself is needed again. */
BT_API bt_status bt_op_gemm_split_act(int32_t layout, int64_t M, int64_t N, int64_t K, const float* A_split,
                                      const float* B_split, float* D, float* D_act_split, int32_t act,
                                      const float* bias, const float* residual, void* scratch,
                                      size_t scratch_bytes, uint32_t flags, void* stream);
BT_API bt_status bt_op_gemm_check(const void* scratch, void* stream);
/* What the wave-model planner chooses for a product of these sizes (host arithmetic, no launch; the
 * "Native GEMM Library" passage: tiles "tuned for highly irregular, low-parallelism gradient shapes").
 * epilogue != 0: a bias or residual is applied, which rules out a K split of all tiles.  out7 (host) =
 * {tile width, 1 if 256-row tiles on CTA pairs, K splits over all tiles, tail tiles, K ranges per
 * tail tile, k-blocks per range, group height of the tile raster}.  A tail split (entries 3-5 non-zero)
 * cuts only the tiles of the last, partly filled round along K and adds a small reduction pass.  The
 * raster walks groups of `group height` row tiles, inside a group row tiles fastest, then column tiles:
 * the tiles in flight at one time share their A and B tiles through L2, and the height is chosen so that
 * an operand larger than L2 is not fetched from HBM once per tile column (or row).  The answer is the
 * one for the per-op calls, whose partial-sum buffer has a fixed size; a model sizes its own buffer so
 * that the LM head's two backward products can always be cut along K, and may therefore split where
 * this call reports none. */
BT_API bt_status bt_op_gemm_plan(int64_t M, int64_t N, int64_t K, int32_t epilogue, uint32_t flags, int32_t* out7);
/* The input-gradient product of the MLP down-projection with the GELU backward in its epilogue
 * (Kernel Design, fused element-wise epilogues; Appendix B "GELU Backward"): with dy_split
 * [2][M][K] (hi/lo planes of the gradient at the projection's output), w_split [2][K][N] (the
 * projection's weight, [out, in] = [K, N]) and h [M][N] (the pre-activation kept by the forward),
 *   dh_split [2][M][N] = hi/lo planes of (dy . W) o GELU'(h)     (form 0: erf form, 1: tanh form,
 *                         2: `h` already holds GELU'(h), as bt_op_gemm_split_act with act 3 / 4 leaves it)
 *   colsum [N]          = the column sums of that product over the M rows, added per 32-row
 *                         group in row order (the bias gradient of the up-projection).
 * All pointers device, 16-byte aligned; N a multiple of 32, M and K multiples of 4.  `scratch`
 * (256-byte aligned, bt_op_gemm_gelu_bwd_scratch_bytes(M, N) bytes) holds the group sums and the
 * error word bt_op_gemm_check reads.  Asynchronous.  flags as for bt_op_gemm_split
 * (BT_FLAG_GEMM_SIMT is not supported here: BT_ERR_UNSUPPORTED). */
BT_API size_t bt_op_gemm_gelu_bwd_scratch_bytes(int64_t M, int64_t N);
BT_API bt_status bt_op_gemm_gelu_bwd(int64_t M, int64_t N, int64_t K, const float* dy_split, const float* w_split,
                                     const float* h, int32_t form, float* dh_split, float* colsum,
                                     void* scratch, size_t scratch_bytes, uint32_t flags, void* stream);

/* Convenience form on raw FP32 operands: bt_op_split of A and B into `scratch`, then
 * bt_op_gemm_split, then bt_op_gemm_check (synchronises). */
BT_API size_t bt_op_gemm_scratch_bytes(int32_t layout, int64_t M, int64_t N, int64_t K);
BT_API bt_status bt_op_gemm(int32_t layout, int64_t M, int64_t N, int64_t K, const float* A, const float* B,
                            float* D, const float* bias, const float* residual, void* scratch,
                            size_t scratch_bytes, uint32_t flags, void* stream);

/* Attention forward (Kernel Design and Optimization: the compute-bound kernels, tensor cores with
 * on-chip reuse of the score tiles; Appendix "Performance Benchmarks", Attention Forward, Causal=1).
 * Causal multi-head self-attention over fused qkv [B*T, 3C] (columns q | k | v, head h at
 * columns h*d..(h+1)*d-1 of each part): o = softmax(q k^T / sqrt(d) + causal mask) v,
 * lse [B,H,T] = log of the softmax normaliser.  d = C/H in {16, 32, 64, 128}.
 * qkv_split (nullable) is the same array as hi/lo planes [2][B*T][3C]; when it is given and d is
 * 64 or 128 the tcgen05 kernels run (TMA-fed, scores and probabilities in tensor memory;
 * synchronises to report a device timeout), otherwise the warp-MMA kernel (d <= 64) or the FMA
 * kernel (d = 128) runs on the raw array.  One of qkv, qkv_split may be NULL. */
BT_API bt_status bt_op_attention_fwd(const float* qkv, const float* qkv_split, int32_t B, int32_t T, int32_t C,
                                     int32_t H, float* o, float* o_split, float* lse, uint32_t flags, void* stream);

/* Attention backward (Appendix "Performance Benchmarks", Attention Backward, Causal=1), with
 * recomputed probabilities: dV = P^T do, dP = do V^T,
 * dS = P o (dP - rowsum(do o o)), dq = dS k / sqrt(d), dk = dS^T q / sqrt(d).
 * scratch: B*H*T floats.  qkv and d_o may be given raw and/or as hi/lo planes (qkv_split
 * [2][B*T][3C], d_o_split [2][B*T][C]); with both split inputs, d = 64 or 128 and only dqkv_split
 * requested (dqkv NULL) the tcgen05 kernels run (they synchronise to report a device timeout),
 * otherwise the warp-MMA kernels run on the raw arrays, which must then be given. */
BT_API bt_status bt_op_attention_bwd(const float* qkv, const float* qkv_split, const float* o, const float* lse,
                                     const float* d_o, const float* d_o_split, int32_t B, int32_t T, int32_t C,
                                     int32_t H, float* dqkv, float* dqkv_split, void* scratch, size_t scratch_bytes,
                                     uint32_t flags, void* stream);

/* GELU forward (Appendix "Performance Benchmarks", GELU Forward; Kernel Design and Optimization:
 * 128-bit accesses, one pass, no lossy approximation): y = GELU(x) in the exact erf form (or the
 * tanh form), n % 4 == 0. */
BT_API bt_status bt_op_gelu_fwd(const float* x, int64_t n, int32_t tanh_form, float* y, float* y_split,
                                void* stream);
/* GELU backward (Appendix "Performance Benchmarks", GELU Backward): dx = dy * GELU'(x). */
BT_API bt_status bt_op_gelu_bwd(const float* x, const float* dy, int64_t n, int32_t tanh_form, float* dx,
                                float* dx_split, void* stream);

/* The same dx for x, dy of shape [N, C] (device), plus colsum[C] (device) = the column sums of
 * dx: the bias gradient of the linear layer that produced x (the MLP up-projection of the GELU
 * feed-forward sublayer; Appendix "Performance Benchmarks", Reduce Sum Kernel, is the paper's
 * stand-alone form of that sum), taken in the pass that writes dx.  scratch: device,
 * bt_op_colsum_scratch_bytes(N, C) bytes, caller-owned.  C % 4 == 0; summation order fixed. */
BT_API bt_status bt_op_gelu_bwd_colsum(const float* x, const float* dy, int64_t N, int32_t C, int32_t tanh_form,
                                       float* dx, float* dx_split, float* colsum, void* scratch,
                                       size_t scratch_bytes, void* stream);

/* Fused softmax cross-entropy over all Vp columns (Appendix "Performance Benchmarks", Sparse
 * Cross-Entropy Loss Forward and Backward, here one kernel; Algorithm 1's "cross-entropy against
 * target"): losses[n] = logsumexp(logits[n,:]) - logits[n, y_n]; dlogits = (softmax - onehot) *
 * inv_count; loss_mean (1 float) = inv_count * sum_n losses[n] in fixed order.  Vp % 4 == 0.
 * A target outside [0, Vp) counts as class 0 and its row + 1 is stored in *d_bad (device int32,
 * nullable, zeroed by the caller; first writer wins).  dlogits (raw) and dlogits_split (hi plane,
 * then lo plane, N * Vp floats each) are both optional; for Vp <= 51,200 (rows held in registers)
 * logits may be the hi plane of dlogits_split itself: the gradient then overwrites the logits. */
BT_API bt_status bt_op_softmax_xent(const float* logits, const int32_t* targets, int64_t N, int32_t Vp,
                                    float inv_count, float* losses, float* loss_mean, float* dlogits,
                                    float* dlogits_split, int32_t* d_bad, void* stream);

/* Column sums (Appendix "Performance Benchmarks", Reduce Sum Kernel; in the step: the bias
 * gradients): out[c] = sum_n x[n,c], fixed summation order. */
BT_API size_t bt_op_colsum_scratch_bytes(int64_t N, int32_t C);
BT_API bt_status bt_op_colsum(const float* x, int64_t N, int32_t C, float* out, void* scratch,
                              size_t scratch_bytes, void* stream);

/* Column sums for callers that cannot provide scratch memory.  (The paper has no counterpart;
 * this entry point exists for integration.)  Some hosts of this library may not allocate device
 * memory at the point of the call: a serving process whose device memory was handed out in full
 * at start-up, a real-time control loop where cudaMalloc's implicit device synchronisation is
 * forbidden, a plug-in that is only given its input and output buffers.  For them the partial
 * sums live in a fixed array inside the library image: 98,304 floats (384 KB) that every GPU
 * loading the library holds until the process exits.  The call allocates nothing (no cudaMalloc,
 * cudaFree or allocating library routine) and returns BT_ERR_UNSUPPORTED when
 * bt_op_colsum_scratch_bytes(N, C) exceeds that size (C > 98,304).
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current) and caches it; that lookup may make the CUDA runtime load the library's
 * device code onto the device, so make that first call at start-up, before any stream capture.
 * Every call on a device shares the one array and overwrites the part it uses, so calls that
 * may overlap on the GPU (different streams, no ordering between them) race; keep them on one
 * stream or order them with events.  Same result as bt_op_colsum, bit for bit. */
BT_API size_t bt_op_colsum_static_max_floats(void);
BT_API bt_status bt_op_colsum_static(const float* x, int64_t N, int32_t C, float* out, void* stream);

/* Global gradient norm and clip factor (hyper-parameter table: "Gradient clip 1.0"; a reduce-sum
 * over the whole gradient arena): out[0] = sqrt(sum g^2), out[1] = clip > 0 ?
 * min(1, clip / (out[0] + 1e-6)) : 1. */
BT_API size_t bt_op_grad_norm_scratch_bytes(int64_t n);
BT_API bt_status bt_op_grad_norm(const float* g, int64_t n, float clip, float* out2, void* scratch,
                                 size_t scratch_bytes, void* stream);

/* One AdamW update at step t >= 1 of n_tensors tensors in one launch (Implementation,
 * "Horizontal Tensor Fusion": the multi-tensor optimizer; Appendix "Performance Benchmarks", AdamW
 * Optimizer Kernel).  h_p/h_g/h_m/h_v are HOST arrays of device
 * pointers, h_numel/h_decay host arrays; d_scale (nullable) is a device float multiplying
 * every gradient (the clip factor).  n_tensors <= 64 per call. */
BT_API bt_status bt_op_adamw_multi(int32_t n_tensors, float* const* h_p, const float* const* h_g,
                                   float* const* h_m, float* const* h_v, const int64_t* h_numel,
                                   const int32_t* h_decay, const bt_adamw_config* opt, int64_t t,
                                   const float* d_scale, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BT_H_ */
