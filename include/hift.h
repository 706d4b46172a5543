/*
 * hift.h -- C ABI of the B200 hierarchical fine-tuning (HiFT) training step.
 *
 * One context = one model on one GPU.  A call to hift_step() performs one
 * iteration of the paper's Algorithm 1: select the active group (steps c-g),
 * full forward pass (h), move that group's optimizer state to the GPU (i),
 * back-propagate only as far down as the group and form weight gradients only
 * inside it (the "Backpropagation" step), update the group with the chosen
 * optimizer, clear gradients, move the state back to host memory (k), and
 * advance the learning-rate schedule once every full cycle of groups (final
 * branch of Algorithm 1).  Only the active group's parameters change
 * (Eq. 2-3: the binary mask beta_i).
 *
 * Conventions
 *   - "dev" pointers are CUDA device pointers on the context's GPU, "host"
 *     pointers are ordinary host memory.  The caller owns every buffer it
 *     passes in; the library never frees or keeps them past the call.
 *   - Everything the context allocates (device and pinned host memory) is
 *     released by hift_destroy().
 *   - Every function returns a hift_status (or a plain value for getters);
 *     nothing aborts, throws, or traps on the device.
 *   - A context is not thread-safe.  Work is issued on the CUDA stream given to
 *     hift_create() plus copy streams the context owns.
 *   - Row-major everywhere.  Linear weights are [out_features, in_features].
 */
#ifndef HIFT_H_
#define HIFT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hift_ctx hift_ctx;

typedef enum {
  HIFT_OK = 0,
  HIFT_ERR_CFG = 1,          /* invalid or unsupported configuration / argument      */
  HIFT_ERR_OOM_DEVICE = 2,   /* cudaMalloc failed                                    */
  HIFT_ERR_OOM_PINNED = 3,   /* pinned host allocation failed                        */
  HIFT_ERR_INPUT = 4,        /* token id or label out of range, NULL pointer         */
  HIFT_ERR_NONFINITE = 5,    /* the loss of the step was NaN/Inf (no update was made)*/
  HIFT_ERR_TIMEOUT = 6,      /* a bounded device-side wait gave up (no update made)  */
  HIFT_ERR_CUDA = 7,         /* any other CUDA runtime/driver error                  */
  HIFT_ERR_CAPACITY = 8      /* size exceeds the library's built-in scratch capacity */
} hift_status;

/* Model description.  Units (the paper's "layers", Section "Hierarchical
 * Training": the embedding is the bottom layer, the head the top layer):
 * unit 0 = all embeddings, units 1..n_blocks = transformer blocks,
 * unit n_blocks+1 = head (final norm + LM matrix, or classifier). */
typedef struct {
  int32_t arch;        /* 0 pre-LN causal decoder (GELU, learned positions)
                          1 post-LN bidirectional encoder + classifier on token 0
                          2 LLaMA-style (RMSNorm, RoPE, SwiGLU, no biases)          */
  int32_t n_blocks, d_model, n_heads, d_ffn, vocab;
  int32_t max_pos;     /* rows of the learned position table (arch 0,1)            */
  int32_t n_classes;   /* arch 1 only                                              */
  int32_t causal;      /* 1: attention masks keys after the query                  */
  int32_t tie_head;    /* 1: LM head shares tok_emb; the matrix belongs to unit 0  */
  int32_t dtype;       /* 0: fp32 params+activations; 1: bf16 with fp32 master     */
  int32_t batch, seq;  /* fixed per context                                        */
  double  norm_eps, rope_base;
  double  dropout;     /* probability p in [0, 1) of dropping an element at the outputs of each block's
                          attention projection and feed-forward network (before the residual addition)
                          and at the embedding output; kept values are scaled by 1/(1-p); 0 = none.
                          The paper fine-tunes with the models' usual dropout without describing it.   */
  uint64_t dropout_seed; /* the mask is Philox4x32-10(key = seed, counter = (element / 4, site, step)),
                          word element % 4, kept iff word >= floor(p 2^32); site 0 = embedding,
                          1 + 2 i = block i attention output, 2 + 2 i = its feed-forward output;
                          step = t.  Reproducible from (seed, t) alone, also across checkpoints.     */
  double  attn_dropout; /* probability in [0, 1) of dropping an attention probability, after the softmax and
                          before the product with V (kept ones scaled by 1/(1-p)); 0 = none.  Same seed;
                          site 1000 + i for block i; the probabilities are numbered ((b H + h) S + q) S' + k
                          with S' = seq rounded up to a multiple of 4.  The tensor-core (tcgen05) and the
                          CUDA-core attention kernels apply it; the warp-level fallback kernels do not, so a
                          bf16 launch they would have taken goes to the CUDA-core kernels.            */
} hift_model_cfg;

/* Grouping and order (paper: Notation paragraph; Algorithm 1 "UpdateStrategy"). */
typedef struct {
  int32_t layers_per_group;  /* m: consecutive units per group, last group short   */
  int32_t split_emb_head;    /* 1: embedding | blocks in chunks of m | head        */
  int32_t order;             /* 0 bottom2up, 1 top2down, 2 random (shuffled once)  */
  uint64_t order_seed;       /* seed of the one-time shuffle                       */
  const int32_t *group_sizes;/* host; NULL = the uniform rule above.  Otherwise n_group_sizes counts of
                                consecutive units per group, bottom first, each >= 1, summing to
                                n_blocks + 2 (groups of unequal size: the paper's grouping is uniform,
                                this is the same fixed partition with the chunk lengths chosen by the
                                caller); read during hift_create only, not kept            */
  int32_t n_group_sizes;
  int32_t literal_queue;     /* 1: Algorithm 1, steps c-d, taken literally: a queue of the n units in the strategy's
                                order (random: shuffled once); every step pops m units from its head and appends
                                them to its tail.  When m divides n this is the fixed partition above.  When it does
                                not, the sets drift: a set can wrap around (top and bottom units together) and a unit
                                is trained ceil- or floor-many times per pass; every unit then keeps its own master,
                                state and update count, a step trains a SET of units (hift_num_sets() distinct sets,
                                set id = step mod that; hift_active_group() returns the set id and hift_set_units()
                                its units), and the learning rate still moves every k = floor(n/m) + 1 steps
                                (hift_num_groups()).  State paging uses one slot in this mode (sets share units).
                                Not with group_sizes, split_emb_head or sharded state.                            */
} hift_group_cfg;

/* Optimizer P and schedule eta_t of Algorithm 1's "Require" list; state residency
 * per its steps i and k ("MoveOptimizerState2GPU/2CPU") and the adapted mixed
 * precision of Section "Mixing Precision" (only the active group's fp32 master
 * is on the GPU). */
typedef struct {
  int32_t kind;              /* 0 AdamW, 1 AdaGrad, 2 SGD with momentum, 3 plain SGD
                                (no optimizer state: only the fp32 master, if any, is paged),
                                4 Adafactor (factored second moment: rows + cols floats of state per
                                matrix; `lr` caps the relative step, `eps` is its epsilon_1;
                                epsilon_2 = 1e-3, clipping d = 1, decay exponent -0.8, no momentum) */
  int32_t sched;             /* 0 constant, 1 linear: warm-up, then decay to 0     */
  int32_t total_cycles;      /* horizon C of the linear schedule, in cycles        */
  int32_t offload_state;     /* 1: inactive groups' master+state in pinned host    */
  int32_t prefetch_groups;   /* state slots on the GPU beyond the first, 0..3 (each the size of the largest
                                group's paged state).  0: one slot, upload issued after the forward pass
                                (the paper's order).  1: two slots, upload at the start of the group's
                                own step, overlapped with the previous write-back.  p >= 2: p + 1 slots,
                                the uploads of the next p - 1 steps' groups are issued ahead (the order
                                is known), so transfers stream across steps and a step no longer lasts
                                at least one transfer.  Residency rule of Algorithm 1 steps i/k kept:
                                only the active group and groups whose transfer is in flight are on
                                the GPU.  Same bits in every mode.                                   */
  int32_t recompute;         /* 1: frozen blocks above the active group keep only their input during the
                                forward pass; what their backward (dX) needs is recomputed block by block in
                                the backward pass.  Same bits, less HBM (the paper's concern), one extra
                                forward of those blocks per step.  0: keep (default)                */
  int32_t warmup_cycles;     /* W (sched 1; the warm-up the paper's hyper-parameter tables list, counted in
                                cycles because the rate moves once per cycle): cycle c < W runs at
                                lr*c/W, cycle c >= W at lr*max(0, (C-c)/(C-W)); 0 = none             */
  int32_t shard_rank;        /* data-parallel ranks may split the optimizer state (ZeRO stage 1): with   */
  int32_t shard_world;       /* shard_world = W > 1 this context holds fp32 master and state (device     */
                             /* slots, pinned blobs, paging) only for piece shard_rank of every group's  */
                             /* span (W contiguous pieces of whole 128-element lines, hift_shard_range), */
                             /* and hift_step_end / hift_step_finish update only that piece; the caller  */
                             /* reduces each piece of the gradient to its owner before, and broadcasts   */
                             /* each piece of the updated parameters (hift_param_view) from its owner    */
                             /* after.  The update is element-wise, so the pieces together are exactly   */
                             /* the unsharded update.  0 or 1 = off.  Not with Adafactor (its statistics */
                             /* span rows and columns); checkpoints are refused while sharded; outside   */
                             /* its piece hift_get_param returns the model value, hift_get_state zeros.  */
  int32_t grad_bf16;         /* 1: the active group's gradient is kept in bf16: the weight-gradient GEMMs store  */
                             /* bf16 from their fp32 accumulators, the other gradient producers round once, the   */
                             /* optimizer reads bf16; half the gradient buffer, half the exchange volume of a     */
                             /* data-parallel step, 2 bytes per element less optimizer traffic.  One rounding of  */
                             /* 2^-9 relative per gradient element (within the 2e-2 gradient tolerance; the       */
                             /* update given that gradient is exact as before).  bf16 models with AdamW, AdaGrad, */
                             /* SGD-momentum or SGD only.  0: fp32 gradients.                                     */
  double lr, beta1, beta2, eps, weight_decay, momentum;
} hift_opt_cfg;

/* Build a context.  `cuda_stream` is a cudaStream_t (NULL = default stream).
 * Parameters start as zeros; fill them with hift_set_param() or
 * hift_init_synthetic().  Fails with HIFT_ERR_OOM_* and leaves *out NULL if the
 * device or pinned memory cannot be had (everything allocated so far is released).
 * One process drives one GPU: the tensor-core kernels' time-out flag, the SM count and the
 * driver entry point for tensor maps are looked up once per process, for the device that
 * was current at the first call; contexts on two different GPUs in one process are not
 * supported (several contexts on the same GPU are).
 * batch * seq <= 65536 tokens a step (HIFT_ERR_CFG beyond it). */
hift_status hift_create(const hift_model_cfg *model, const hift_group_cfg *groups,
                        const hift_opt_cfg *opt, void *cuda_stream, hift_ctx **out);
void hift_destroy(hift_ctx *ctx);

/* One iteration of Algorithm 1 on the group hift_active_group() names.
 * tokens_dev: int32 [batch, seq].  labels_dev: int32 [batch, seq] (arch 0, 2;
 * -1 = position ignored) or int32 [batch] (arch 1).  The mean cross-entropy of
 * the batch, computed before the update, is written to *loss_host.  Returns
 * after the loss is on the host; state write-back may still be in flight.
 * A step that fails changes nothing: when a bounded device-side wait gave up
 * (HIFT_ERR_TIMEOUT), a token id or label was out of range (HIFT_ERR_INPUT; the
 * id is clamped on the device so that the pass itself stays in bounds) or the
 * loss is not finite (HIFT_ERR_NONFINITE), the optimizer kernels see the
 * failure on the device and store nothing, so every parameter, master value and
 * optimizer-state value of every group keeps its bits, the group's update
 * count and t do not advance, and the next call trains the same group again.
 * (Gradients that overflow while the loss stays finite are not detected.) */
hift_status hift_step(hift_ctx *ctx, const int32_t *tokens_dev, const int32_t *labels_dev,
                      float *loss_host);
/* Same, with the batch in host memory (validated on the host, then copied to
 * the GPU inside the call; invalid input is rejected before anything runs). */
hift_status hift_step_host(hift_ctx *ctx, const int32_t *tokens_host, const int32_t *labels_host,
                           float *loss_host);

/* Batches of unequal length, padded on the right to `seq` (what fine-tuning on the paper's tasks feeds a
 * model; the paper does not discuss it): lens_host[b] in [1, seq] is the number of real tokens of batch
 * entry b.  From the next step on, attention lets every query of entry b see keys 0 .. lens_host[b]-1 only
 * (on top of the causal mask, if any); NULL switches the table off again.  Padded positions still run
 * through the model; the caller keeps them out of the loss with label -1 (arch 0, 2; arch 1 reads
 * token 0 only), and then no gradient flows through them.  The table is copied during the call.
 * HIFT_ERR_INPUT if a length is out of range. */
hift_status hift_set_key_lengths(hift_ctx *ctx, const int32_t *lens_host);

/* The same step in two halves, for data-parallel training (several contexts, one per GPU, each
 * on its shard of the batch; the paper's method itself is single-device).  hift_step_begin runs
 * the forward pass and the truncated backward pass and returns the loss; the active group's flat
 * fp32 gradient (its tensors in layout order, zero in the alignment gaps) is then exposed by
 * hift_grad_view as a device pointer the caller may reduce over ranks and scale (1/k of the
 * volume a full-parameter step would exchange); hift_step_end applies the optimizer to the group,
 * starts the state write-back and advances t.  Work the caller enqueued on the stream given to
 * hift_create is ordered before the update.  begin/end must alternate; hift_step in between is
 * refused with HIFT_ERR_CFG.  A hift_step_begin that fails leaves no update pending.
 * hift_step_abort drops a pending update instead of applying it (t does not advance): what
 * every rank calls when any rank's first half failed, so that replicas stay identical. */
hift_status hift_step_begin(hift_ctx *ctx, const int32_t *tokens_dev, const int32_t *labels_dev,
                            float *loss_host);
hift_status hift_grad_view(hift_ctx *ctx, void **grad_dev, size_t *n);   /* n elements of hift_grad_elem_bytes() each */
int32_t     hift_grad_elem_bytes(const hift_ctx *ctx);                    /* 4: fp32 gradients, 2: bf16 (grad_bf16) */
hift_status hift_step_end(hift_ctx *ctx);
hift_status hift_step_abort(hift_ctx *ctx);

/* The exchange overlapped with the backward pass.  The truncated backward pass finishes the group's
 * gradient from the top of its flat span downwards (the last block's down projection first, the lowest
 * unit's first norm last), so the tail of the buffer can be reduced over the ranks while the head is
 * still being computed: with one all-reduce per chunk this hides all but the last chunk's exchange
 * behind the remaining dX / dW GEMMs.
 *   hift_step_begin_async  enqueues forward + truncated backward and returns without waiting;
 *   hift_grad_num_chunks / hift_grad_chunk  list the chunks of hift_grad_view's buffer in the order
 *       they become final (offset and length in elements; together they tile the span exactly once;
 *       each at least the size set by hift_set_grad_chunk_bytes, default 32 MiB, except the last);
 *   hift_grad_chunk_wait   makes `cuda_stream` (the caller's communication stream) wait until chunk
 *       i is final; waiting for the last chunk also covers the step's gate word;
 *   hift_gate_view         device address of the step's gate word (int32): 0 = the update goes ahead,
 *       otherwise a positive code of what failed.  Ranks reduce it with MAX next to the last chunk,
 *       so that all of them call the update off when one of them failed;
 *   hift_step_finish       = hift_step_end that also returns the loss: orders itself after the work
 *       enqueued on the stream given to hift_create (make that stream wait for the communication
 *       stream first), applies the optimizer, starts the write-back, waits for the step and returns
 *       its status.  A rank whose own pass was fine but whose gate word a peer raised returns the
 *       peer's failure.
 * The chunk plan itself is host logic; hift_plan_grad_chunks runs it on a caller-given tensor list
 * (ascending offsets) and completion order without touching a GPU: chunk_off / chunk_n receive the
 * chunks, chunk_after[i] the index into completion_order after which chunk i is final.  Returns the
 * number of chunks, or -1 (bad arguments, max_chunks too small). */
hift_status hift_step_begin_async(hift_ctx *ctx, const int32_t *tokens_dev, const int32_t *labels_dev);
int32_t     hift_grad_num_chunks(const hift_ctx *ctx);
hift_status hift_grad_chunk(const hift_ctx *ctx, int32_t i, size_t *offset, size_t *n);
hift_status hift_grad_chunk_wait(hift_ctx *ctx, int32_t i, void *cuda_stream);
hift_status hift_gate_view(hift_ctx *ctx, int32_t **gate_dev);
hift_status hift_set_grad_chunk_bytes(hift_ctx *ctx, size_t bytes);
/* Sharded optimizer state (hift_opt_cfg.shard_world): the piece of group g's flat span that `rank` holds, as
 * offset and length in elements of hift_grad_view / hift_param_view; and the parameters of the group trained
 * by the step in flight (or the last one) as the forward pass reads them (bf16: elem_bytes 2, or fp32: 4),
 * a device pointer to the group's whole span, for the exchange of the updated pieces. */
hift_status hift_shard_range(const hift_ctx *ctx, int32_t g, int32_t rank, size_t *offset, size_t *n);
hift_status hift_param_view(hift_ctx *ctx, void **param_dev, size_t *n, int32_t *elem_bytes);
hift_status hift_step_finish(hift_ctx *ctx, float *loss_host);
int32_t     hift_plan_grad_chunks(const size_t *offsets, const size_t *sizes, int32_t n_tensors, size_t span_elems,
                                  const int32_t *completion_order, int32_t n_completed, size_t min_chunk_elems,
                                  size_t *chunk_off, size_t *chunk_n, int32_t *chunk_after, int32_t max_chunks);

int32_t hift_active_group(const hift_ctx *ctx);   /* group the NEXT hift_step trains */
int32_t hift_num_groups(const hift_ctx *ctx);     /* k: steps per learning-rate cycle */
int32_t hift_num_sets(const hift_ctx *ctx);       /* distinct sets of units the schedule trains (= k unless the queue drifts) */
/* Units of set `set_id` (ascending) into units_out[0 .. cap); *n_units receives their number. */
hift_status hift_set_units(const hift_ctx *ctx, int32_t set_id, int32_t *units_out, int32_t cap, int32_t *n_units);
int64_t hift_step_count(const hift_ctx *ctx);     /* t, steps taken so far           */
double  hift_current_lr(const hift_ctx *ctx);     /* lr the NEXT step will use       */
/* Units of group (set) g: writes the first and last unit id (inclusive); HIFT_ERR_CFG for a set of the drifting
 * queue that is not an interval of units (use hift_set_units). */
hift_status hift_group_units(const hift_ctx *ctx, int32_t g, int32_t *unit_lo, int32_t *unit_hi);
/* Force the group trained by the next steps (depth sweeps); -1 restores the schedule. */
hift_status hift_force_group(hift_ctx *ctx, int32_t g);
/* The same for a list: the next steps train groups[0], groups[1], ..., groups[n-1], groups[0], ...
 * (host array, copied; n = 0 restores the schedule; a forced single group takes precedence).  Unlike
 * a group forced step by step, the list is known ahead, so look-ahead paging works on it: what a
 * benchmark uses to time an even sample of the cycle.  t, the learning rate and the update counts
 * advance as always. */
hift_status hift_force_sequence(hift_ctx *ctx, const int32_t *groups, int32_t n);

/* High-water mark, in bytes, of all device memory the context holds. */
size_t hift_peak_hbm_bytes(const hift_ctx *ctx);
/* Bytes of pinned host memory the context holds. */
size_t hift_pinned_host_bytes(const hift_ctx *ctx);

/* ---- parameter / gradient access (tests and checkpoints) ---------------- */
int32_t hift_num_tensors(const hift_ctx *ctx);
/* name_out: at least 64 bytes.  A vector has rows = 1. */
hift_status hift_tensor_info(const hift_ctx *ctx, int32_t tensor, char *name_out,
                             int32_t *unit, int64_t *rows, int64_t *cols);
/* fp32 master values of one tensor, host memory, `n` = rows*cols elements.
 * set: also refreshes the bf16 model copy (round to nearest even). */
hift_status hift_set_param(hift_ctx *ctx, int32_t tensor, const float *src_host, size_t n);
hift_status hift_get_param(hift_ctx *ctx, int32_t tensor, float *dst_host, size_t n);
/* The value the forward pass reads (bf16 widened to fp32, or the fp32 itself). */
hift_status hift_get_model_param(hift_ctx *ctx, int32_t tensor, float *dst_host, size_t n);
/* Optimizer state `which` (0: first moment / accumulator / momentum, 1: second moment). */
hift_status hift_get_state(hift_ctx *ctx, int32_t tensor, int32_t which, float *dst_host, size_t n);
/* Adafactor only: which = 0 the row statistics R [rows] (for a vector, rows = 1: its second
 * moment V [cols]), which = 1 the column statistics C [cols]. */
hift_status hift_get_factored_state(hift_ctx *ctx, int32_t tensor, int32_t which, float *dst_host, size_t n);
/* fp32 gradient of a tensor of the group trained by the LAST step. */
hift_status hift_get_grad(hift_ctx *ctx, int32_t tensor, float *dst_host, size_t n);
/* Fill every parameter on the device: matrices N(0, std^2) from a counter-based
 * hash of (seed, element index), gains 1, biases 0; optimizer state zero. */
hift_status hift_init_synthetic(hift_ctx *ctx, uint64_t seed, double std);

/* Weights from a file in the library's container format ("HIFTWTS1": magic[8], uint32 n, then n records of
 * { char name[64]; uint32 dtype (0 fp32, 1 bf16); uint64 rows, cols; rows*cols elements }, names and shapes
 * as hift_tensor_info reports them).  Each record goes through hift_set_param (fp32 master and bf16 model
 * copy; optimizer state is left alone).  strict != 0: every tensor of the model must be in the file.
 * *n_loaded (may be NULL) receives the number of tensors set.  HIFT_ERR_INPUT for a missing / short /
 * foreign file, an unknown or repeated tensor, a wrong shape; tensors set before the error stay set.
 * The package's weights.py writes this format and converts safetensors checkpoints with the public
 * LLaMA / GPT-2 / RoBERTa tensor names into it. */
hift_status hift_load_weights(hift_ctx *ctx, const char *path, int32_t strict, int32_t *n_loaded);

/* Checkpoint: the whole training state is the fp32 master (or fp32 parameters), the optimizer
 * state and update count of every group (which Algorithm 1 keeps on the host between a group's
 * turns anyway), and the step counter t; the group order follows from the configuration.
 * hift_load needs a context created with the same configuration (HIFT_ERR_CFG otherwise) and
 * rebuilds the bf16 model copy.  A missing / short / foreign file gives HIFT_ERR_INPUT. */
hift_status hift_save(hift_ctx *ctx, const char *path);
hift_status hift_load(hift_ctx *ctx, const char *path);

/* ---- instrumentation ------------------------------------------------------ */
/* Kernel classes for hift_profile(). */
enum { HIFT_K_GEMM_FWD = 0, HIFT_K_GEMM_DX = 1, HIFT_K_GEMM_DW = 2, HIFT_K_ATTN_FWD = 3,
       HIFT_K_ATTN_BWD = 4, HIFT_K_NORM = 5, HIFT_K_ELEMWISE = 6, HIFT_K_CE = 7,
       HIFT_K_EMBED = 8, HIFT_K_OPT = 9, HIFT_K_REDUCE = 10, HIFT_K_NUM = 11 };
/* on=1: bracket every kernel launch of the following steps with CUDA events on
 * the launching stream and accumulate per class; on=0 stops.  Resets counters. */
hift_status hift_profile_enable(hift_ctx *ctx, int32_t on);
/* Accumulated since enable: launches, device milliseconds and algorithmic work
 * (flops for GEMM/attention classes, bytes for the others). */
hift_status hift_profile(hift_ctx *ctx, int32_t kernel_class, int64_t *launches,
                         double *millis, double *work);
/* Kernel launches issued by the last hift_step (all classes). */
int64_t hift_last_step_launches(const hift_ctx *ctx);
/* Bytes paged host->device and device->host by the last step. */
hift_status hift_last_step_paging(const hift_ctx *ctx, size_t *h2d_bytes, size_t *d2h_bytes);

/* Device timeline of the last step's state paging (Algorithm 1 steps i and k), in milliseconds
 * after the step's first kernel: [0] H2D begin, [1] H2D end (of the upload that made the group
 * resident: negative when an earlier step issued it ahead), [2] optimizer reaches its wait
 * for the state, [3] wait over, [4] D2H begin, [5] D2H end.  NaN where there is nothing to
 * report (offload off).  Waits for the copies to finish. */
hift_status hift_last_step_timeline(hift_ctx *ctx, double *ms6);

/* The tensor-core GEMM bounds every device-side wait; a wait that gives up records a code in a
 * device flag, after which every tensor-core GEMM launch returns at once and hift_step reports
 * HIFT_ERR_TIMEOUT.  This call reads the flag (set_value < 0) or overwrites it first
 * (set_value >= 0; 0 clears it, which is how a caller resumes after a time-out, and a non-zero
 * value lets a test walk the time-out path without stalling anything).  Returns the flag, or -1
 * if the tensor-core path is unavailable.  Synchronises the device. */
int32_t hift_tc_error_flag(int32_t set_value);

/* Code-path switches for tests and A/B timing; every one defaults to 1, the fast path.  which = 0: CTA-pair
 * tiles in the tensor-core GEMM (0 = one CTA per tile); 1: programmatic dependent launch (0 = plain stream
 * order); 2: tcgen05 attention forward, 3: tcgen05 attention backward (0 = the warp-level mma.sync kernels).
 * value >= 0 sets the switch, value < 0 only reads it; returns the previous value, or -1 for an unknown
 * switch.  Process-wide, consulted at every launch, not thread-safe.  Results do not depend on switches 0
 * and 1 (same bits); 2 and 3 select kernels with a different summation order.
 * Two more, for fault-path tests that need no faulting GPU: which = 4: the value-th pinned host allocation
 * from now on (0 = the next one) fails as if the host were out of pinned memory, once (value -1 = off),
 * so that hift_create's HIFT_ERR_OOM_PINNED path and its clean-up run; which = 5: contexts created while it
 * is 1 run in checked mode: every slice of the activation arena is followed by a 256-byte guard region that
 * each step paints before its first kernel, and hift_check_arena() counts the regions a step wrote into. */
int32_t hift_test_switch(int32_t which, int32_t value);
/* Checked mode only (-1 otherwise): guard regions of the last step's arena plan that no longer hold their
 * pattern (0 = no kernel wrote past the end of its buffer), and how many regions there are. */
int64_t hift_check_arena(hift_ctx *ctx);
int64_t hift_arena_guard_count(const hift_ctx *ctx);

/* ---- the group-local fused optimizer on caller-owned flat buffers --------
 * One streaming pass over n elements (the update Algorithm 1 applies to the
 * active group once "UpdateOptimizerParameter" has pointed P at theta_s).  All
 * pointers are device pointers, 16-byte aligned.  master/grad/s0/s1 are fp32;
 * s1 is used by AdamW only (may be NULL otherwise), s0 by all but plain SGD
 * (kind 3; may be NULL there); param_bf16 may be NULL
 * (fp32 configs).  tau >= 1 is the number of updates this group has had,
 * including this one (bias correction).  Launches on `cuda_stream`, does not
 * synchronise. */
hift_status hift_opt_step(int32_t kind, size_t n, void *param_bf16_dev, float *master_dev,
                          const float *grad_dev, float *s0_dev, float *s1_dev,
                          double lr, double beta1, double beta2, double eps,
                          double weight_decay, double momentum, int64_t tau,
                          void *cuda_stream);

/* Adafactor (one of the optimizers the paper profiles, without formulas; built in the form
 * torch.optim.Adafactor uses for Shazeer & Stern 2018, Algorithms 4-5: epsilon_1 is a lower clamp on the
 * factored second-moment estimate and on the root of it, not a term added to the squared gradient)
 * on one caller-owned tensor [rows, cols] (rows = 1: a vector, unfactored).
 * master/grad: fp32 [rows*cols]; state: fp32, R[rows] | C[cols] for a matrix, V[cols] for a
 * vector; scratch: fp32, 2*rows + 64*cols + 8 floats; param_bf16 may be NULL.  tau >= 1 as in
 * hift_opt_step.  Launches several small kernels on `cuda_stream`; does not synchronise. */
hift_status hift_adafactor_step(int64_t rows, int64_t cols, void *param_bf16_dev, float *master_dev,
                                const float *grad_dev, float *state_dev, float *scratch_dev,
                                double lr, double eps1, double weight_decay, int64_t tau, void *cuda_stream);

/* ---- single kernels on caller-owned device buffers (per-kernel parity) ----
 * These are the pieces of Algorithm 1's "ForwardPropagation"/"Backpropagation"
 * steps.  dtype 0: fp32 operands, 1: bf16 operands.  All launch on `cuda_stream`
 * and do not synchronise. */
/* form 0: y[M,N]  = x[M,K] * w[N,K]^T (+ bias[N]);             out has operand type
 * form 1: dx[M,K] = dy[M,N] * w[N,K];                          out has operand type
 * form 2: dw[N,K] = dy[M,N]^T * x[M,K];                        out is fp32
 * residual_dev (forms 0,1; optional): fp32 [M, out cols]; when given the output
 * is fp32 too (the residual stream is kept in fp32).
 * `path`: 0 = pick automatically, 1 = force the CUDA-core kernel, 2 = force the
 * tcgen05 tensor-core kernel (bf16 only; HIFT_ERR_CFG if the shape is not eligible). */
hift_status hift_k_linear(int32_t form, int32_t dtype, int32_t path, int64_t M, int64_t N, int64_t K,
                          const void *a_dev, const void *b_dev, void *out_dev,
                          const void *bias_dev, const float *residual_dev, void *cuda_stream);
/* qkv[T,3d] (q|k|v column blocks, head h at columns h*d_h) -> o[T,d], lse[B,H,S] fp32.
 * key_lens_dev: int32 [batch] or NULL; entry b attends to keys 0 .. key_lens[b]-1 only (values are
 * clamped to [1, seq] on the device). */
hift_status hift_k_attention_fwd(int32_t dtype, int32_t batch, int32_t seq, int32_t n_heads,
                                 int32_t d_head, int32_t causal, const void *qkv_dev, void *o_dev,
                                 float *lse_dev, const int32_t *key_lens_dev, void *cuda_stream);
/* -> dqkv[T,3d]; dsum_dev is fp32 scratch of batch*seq*n_heads elements.  Rows of dk, dv at padded
 * keys are written as zeros. */
hift_status hift_k_attention_bwd(int32_t dtype, int32_t batch, int32_t seq, int32_t n_heads,
                                 int32_t d_head, int32_t causal, const void *qkv_dev,
                                 const void *o_dev, const float *lse_dev, const void *do_dev,
                                 void *dqkv_dev, float *dsum_dev, const int32_t *key_lens_dev,
                                 void *cuda_stream);
/* The same two with dropout on the probabilities (hift_model_cfg.attn_dropout): rate p in [0, 1), the generator's
 * seed, site and step as the step would pass them (site 1000 + block, step t).  p = 0 is the plain kernel. */
hift_status hift_k_attention_fwd_drop(int32_t dtype, int32_t batch, int32_t seq, int32_t n_heads,
                                      int32_t d_head, int32_t causal, const void *qkv_dev, void *o_dev,
                                      float *lse_dev, const int32_t *key_lens_dev, double p, uint64_t seed,
                                      int32_t site, int64_t step, void *cuda_stream);
hift_status hift_k_attention_bwd_drop(int32_t dtype, int32_t batch, int32_t seq, int32_t n_heads,
                                      int32_t d_head, int32_t causal, const void *qkv_dev,
                                      const void *o_dev, const float *lse_dev, const void *do_dev,
                                      void *dqkv_dev, float *dsum_dev, const int32_t *key_lens_dev, double p,
                                      uint64_t seed, int32_t site, int64_t step, void *cuda_stream);
/* Rotary models (RoPE on q and k, as in the LLaMA-shaped configuration the paper profiles) on the
 * tensor-core path: the rotation is fused into the epilogue of the qkv projection, and this hook
 * exposes exactly that kernel: out[M,N] = rope(x[M,K] w[N,K]^T + bias) on columns [0, rope_cols),
 * plain beyond.  cs_dev: fp32 [seq, d_head/2] cosines followed by [seq, d_head/2] sines of
 * angle(pos, j) = pos * base^(-2j/d_head); pair (j, j + d_head/2); row r has position r mod seq.
 * HIFT_ERR_CFG when the fused kernel does not apply (d_head != 128, operands not 16-byte aligned,
 * N or rope_cols not a multiple of 128). */
hift_status hift_k_linear_rope(int64_t M, int64_t N, int64_t K, const void *a_dev, const void *b_dev, void *out_dev,
                               const void *bias_dev, const float *cs_dev, int32_t seq, int32_t d_head,
                               int64_t rope_cols, void *cuda_stream);
/* SwiGLU blocks on the tensor-core path: the gate | up projection (w[2f, K]: f gate rows, then f up rows) and
 * the activation are one kernel.  s_dev[M, f] = silu(gate) * up (bf16); gu_dev[M, 2f] receives the two
 * pre-activations, or may be NULL when nothing will read them (blocks below the active group keep no
 * activations).  HIFT_ERR_CFG when the fused kernel does not apply (f not a multiple of 128, M < 128,
 * operands not 16-byte aligned). */
hift_status hift_k_linear_swiglu(int64_t M, int64_t f, int64_t K, const void *a_dev, const void *b_dev, void *gu_dev,
                                 void *s_dev, const void *bias_dev, void *cuda_stream);
/* ... and its backward: dgu_dev[M, 2f] = swiglu_bwd(dy[M,N] w[N,f]; gu_dev[M, 2f]), i.e. the dX product of the
 * down projection (w is the down matrix [N = d_model, f]) with the activation's backward applied in
 * its epilogue: d gate in columns [0, f), d up in [f, 2f).  HIFT_ERR_CFG when the fused kernel does not
 * apply (f not a multiple of 32, M < 128, operands not 16-byte aligned). */
hift_status hift_k_linear_dx_swiglu_bwd(int64_t M, int64_t N, int64_t f, const void *dy_dev, const void *w_dev,
                                        const void *gu_dev, void *dgu_dev, void *cuda_stream);
/* GELU blocks (the GPT-2- and RoBERTa-shaped configurations), same two fusions:
 *   hift_k_linear_gelu       : pre_dev[M,N] = x[M,K] w[N,K]^T + bias (may be NULL when not needed), act_dev[M,N] = gelu(pre)
 *   hift_k_linear_dx_gelu_bwd: da_dev[M,f] = (dy[M,N] w[N,f]) * gelu'(pre_dev[M,f])
 * exact (erf) GELU; HIFT_ERR_CFG when the fused kernel does not apply (output width not a multiple of 32, M < 128,
 * operands not 16-byte aligned). */
hift_status hift_k_linear_gelu(int64_t M, int64_t N, int64_t K, const void *a_dev, const void *b_dev, void *pre_dev,
                               void *act_dev, const void *bias_dev, void *cuda_stream);
hift_status hift_k_linear_dx_gelu_bwd(int64_t M, int64_t N, int64_t f, const void *dy_dev, const void *w_dev,
                                      const void *pre_dev, void *da_dev, void *cuda_stream);
/* kind 0 LayerNorm (gain, bias), 1 RMSNorm (gain).  x is the fp32 residual stream in every
 * dtype; gain/bias/y have the operand type.  stats: fp32 [2*rows] (mean|rstd). */
hift_status hift_k_norm_fwd(int32_t dtype, int32_t kind, int64_t rows, int64_t cols, double eps,
                            const float *x_dev, const void *gain_dev, const void *bias_dev,
                            void *y_dev, float *stats_dev, void *cuda_stream);
/* dx = norm_bwd(dy) (+ add).  dy and gain have the operand type; x, add and dx are fp32
 * (residual stream and its gradient).  dx may be NULL (skipped).  dgain/dbias fp32 [cols]
 * may be NULL (skipped); partial_dev: fp32 scratch of 2*64*cols elements, needed when
 * dgain != NULL. */
hift_status hift_k_norm_bwd(int32_t dtype, int32_t kind, int64_t rows, int64_t cols,
                            const void *dy_dev, const float *x_dev, const float *stats_dev,
                            const void *gain_dev, const float *add_dev, float *dx_dev,
                            float *dgain_dev, float *dbias_dev, float *partial_dev,
                            void *cuda_stream);
/* The paper has no counterpart for this entry point; it exists for callers that must not
 * allocate.  It computes exactly what hift_k_norm_bwd computes (same kernels, same summation
 * order, same results), but takes no `partial_dev` argument: the column-reduction scratch lives
 * in a fixed array that is part of the library image (4 MiB of device memory per GPU that loads
 * the library, held until the process exits).  Nothing is allocated or freed, on the host or on
 * the device, by this call: no cudaMalloc, no cudaFree, no allocating library routine.  That is
 * what code needs which runs where the allocator is off limits - inside a memory pool whose
 * budget is already committed, in a latency-critical loop that cannot afford an allocator's
 * implicit synchronisation, or in a host process that was handed its buffers by someone else
 * and has no allocator of its own for this device.
 *   - cols must be <= HIFT_STATIC_SCRATCH_MAX_COLS, else HIFT_ERR_CAPACITY (nothing is launched).
 *   - The first call on each device looks up the device address of the array (with that
 *     device current).  Make that first call before starting any stream capture.  The address is
 *     kept for the life of the process: it does not survive a cudaDeviceReset of that device.
 *   - dy, x, stats and gain must not be NULL when dx or dgain is requested (HIFT_ERR_INPUT;
 *     hift_k_norm_bwd checks the same).
 *   - All calls on one GPU share the one array, which keeps whatever the previous call left.
 *     Every word a call reads it has written earlier in the same call, so stale contents
 *     are harmless and nothing needs clearing; but two calls that overlap on the GPU (different
 *     streams, or different host threads) race on it.  Serialise them.
 * Inputs and outputs are the caller's, as for hift_k_norm_bwd. */
#define HIFT_STATIC_SCRATCH_MAX_COLS 8192
hift_status hift_k_norm_bwd_static(int32_t dtype, int32_t kind, int64_t rows, int64_t cols,
                                   const void *dy_dev, const float *x_dev, const float *stats_dev,
                                   const void *gain_dev, const float *add_dev, float *dx_dev,
                                   float *dgain_dev, float *dbias_dev, void *cuda_stream);

/* Softmax cross-entropy over rows of logits[rows, ld] (columns >= vocab are
 * padding).  Overwrites logits with d loss / d logits.  loss_dev: 4 fp32 words,
 * [0] = mean loss over rows with label >= 0, [1] = that row count (int32 bits),
 * [2] = 1 (int32) if a label was >= vocab.  rowloss_dev: fp32 scratch [rows]. */
hift_status hift_k_cross_entropy(int32_t dtype, int64_t rows, int64_t vocab, int64_t ld,
                                 void *logits_dev, const int32_t *labels_dev, float *rowloss_dev,
                                 float *loss_dev, void *cuda_stream);

const char *hift_strerror(hift_status s);

#ifdef __cplusplus
}
#endif
#endif /* HIFT_H_ */
