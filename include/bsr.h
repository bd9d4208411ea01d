/*
 * bsr.h -- C ABI of the Block Selective Reprogramming (BSR) fine-tuning step for Vision
 * Transformers on NVIDIA B200 (sm_100a).
 *
 * The calls follow the paper's statement of the method (arXiv 2405.10951, Section 4.1 and
 * Fig. 2): a pre-trained ViT of which only chosen blocks and the classification head train,
 * with tokens dropped at designated blocks by the classification token's attention (Eq. 6).
 *
 * Conventions for every function
 *   - returns a bsr_status (0 = BSR_OK, negative = error); never throws, aborts or traps;
 *   - "dev" pointers are device (global-memory) addresses valid on the current CUDA device,
 *     "host" pointers are ordinary host addresses; nothing here takes a framework type;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream);
 *   - the library allocates no device memory: weights, optimiser state, saved activations and
 *     scratch are carved from the single workspace block the caller hands to bsr_create, and
 *     the caller keeps ownership of that block and of every input and output buffer;
 *   - bsr_train_step / bsr_eval_forward only enqueue work on `stream` and do not synchronise;
 *     results are in device memory once the stream reaches that point;
 *   - tensors are dense row-major; linear weights are [out_features, in_features].
 *
 * Parameter names (bsr_set_param / bsr_get_tensor), L = dim, F = mlp_hidden:
 *   patch_embed.weight [L, C*P*P] (input flattened as channel, row, column), patch_embed.bias [L],
 *   cls_token [L], pos_embed [N+1, L],
 *   blocks.<l>.norm1.weight|bias [L], blocks.<l>.attn.qkv.weight [3L, L] (rows: all Q heads, all K
 *   heads, all V heads), blocks.<l>.attn.qkv.bias [3L], blocks.<l>.attn.proj.weight [L, L], .bias [L],
 *   blocks.<l>.norm2.weight|bias [L], blocks.<l>.mlp.fc1.weight [F, L], .bias [F],
 *   blocks.<l>.mlp.fc2.weight [L, F], .bias [L],
 *   MoE blocks instead of mlp.*: blocks.<l>.moe.gate.weight [tasks, E, L], moe.fc1.weight [E, F, L],
 *   moe.fc1.bias [E, F], moe.fc2.weight [E, L, F], moe.fc2.bias [E, L],
 *   norm.weight|bias [L], head.<t>.weight [classes_t, L], head.<t>.bias [classes_t].
 */
#ifndef BSR_H_
#define BSR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  BSR_OK = 0,
  BSR_ERR_INVALID_ARG = -1,         /* null pointer, bad dimension, unknown name, batch > max_batch */
  BSR_ERR_UNSUPPORTED = -2,         /* valid request this build does not implement */
  BSR_ERR_WORKSPACE_TOO_SMALL = -3,
  BSR_ERR_CUDA = -4,                /* a CUDA runtime/driver call failed; see bsr_last_error */
  BSR_ERR_DEVICE_TIMEOUT = -5,      /* a bounded device-side wait gave up (reported by bsr_sync_status) */
  BSR_ERR_NONFINITE = -6,           /* loss was not finite (reported by bsr_sync_status) */
  BSR_ERR_MEMORY_GUARD = -7,        /* a guard word between two workspace slices was overwritten (bsr_sync_status) */
  BSR_ERR_DEVICE_CHECK = -8         /* an index check of the checked build (-DBSR_DEBUG) failed (bsr_sync_status) */
} bsr_status;

enum { BSR_DTYPE_FP32 = 0, BSR_DTYPE_BF16 = 1 };
/* What becomes of the dropped tokens (Section 4.1: "fused"): nothing, one extra token sum_j s_j x'_j weighted by the
 * head-mean scores, or that sum divided by sum_j s_j (the weighted mean). */
enum { BSR_FUSE_NONE = 0, BSR_FUSE_WEIGHTED_SUM = 1, BSR_FUSE_WEIGHTED_MEAN = 2 };
enum { BSR_OPT_ADAMW = 0, BSR_OPT_SGD = 1 };
enum { BSR_MAX_DROPS = 8, BSR_MAX_TASKS = 4, BSR_MAX_DEPTH = 32 };

/* Model dimensions (Section 3.1: N patches + 1 classification token, embedding length L, H heads). */
typedef struct {
  int32_t image_size, patch_size, in_chans;
  int32_t dim, heads, depth, mlp_hidden;
  int32_t num_tasks, num_classes[BSR_MAX_TASKS];
  int32_t moe_experts, moe_top_k;   /* 0 = dense FFN everywhere */
  uint32_t moe_block_mask;          /* bit l set: block l's FFN is an MoE layer (Section 5.2) */
  int32_t dtype;                    /* BSR_DTYPE_*: storage type of weights and activations */
  float ln_eps;
} bsr_dims;

/* The BSR configuration (Section 4.1, Fig. 2): which blocks train, where and how many tokens drop.  Any set of
 * blocks may train (e.g. the paper's 4th, 8th and 12th): frozen blocks after the earliest trainable one pass the
 * gradient on and get no parameter gradient (Eq. 2, Eq. 8); blocks before it run forward only and keep nothing. */
typedef struct {
  bsr_dims dims;
  uint32_t trainable_mask;          /* bit l set: block l trains; head and final LayerNorm always train */
  int32_t n_drop;                   /* number of token drop locations */
  int32_t drop_block[BSR_MAX_DROPS];/* 0-based block index of each location, strictly ascending */
  int32_t keep_num[BSR_MAX_DROPS];  /* keep rate of the location = keep_num / keep_den (1 - drop rate) */
  int32_t keep_den[BSR_MAX_DROPS];
  int32_t fuse_mode;                /* BSR_FUSE_* */
  float lr, beta1, beta2, eps, weight_decay;   /* AdamW (Section 5, training hyper-parameters) */
  int32_t max_batch;
  /* Optimiser (Section 5: AdamW for the DeiT-S runs, SGD for the ViT-B and MoE runs).  BSR_OPT_SGD is SGD with
   * momentum: d = g + weight_decay p (matrices only), buf <- momentum buf + d, p <- p - lr buf, buf starting at
   * zero; the buffer is read under the name "adam_m/<param>" and "adam_v/<param>" stays zero. */
  int32_t optimizer;                /* BSR_OPT_* */
  float momentum;
  /* 8-bit floating point in the gradient-free prefix (Conclusions: quantisation is orthogonal to BSR and can be added
   * on top).  1: in every dense block before the earliest trainable one, the two linear layers fed by a LayerNorm
   * (QKV and the first FFN layer) multiply E4M3 operands on the tensor cores: each LayerNorm output row and each weight
   * row is scaled so that its largest magnitude maps to 448 and rounded to nearest-even, the accumulation is float32,
   * the product is rescaled before the bias.  Those blocks carry no gradient, so nothing else changes.  bf16 models
   * with dim a multiple of 16; 0 (the default) keeps every layer in bf16. */
  int32_t frozen_fp8;
} bsr_config;

/* HBM footprint of a created handle, in bytes. */
typedef struct {
  uint64_t workspace_bytes;         /* whole workspace */
  uint64_t weight_bytes;            /* weights in the storage dtype (all blocks) */
  uint64_t master_bytes;            /* fp32 master copy of trainable parameters */
  uint64_t optimizer_bytes;         /* AdamW first and second moments */
  uint64_t grad_bytes;              /* fp32 gradients of trainable parameters */
  uint64_t saved_activation_bytes;  /* activations kept for backward: trainable blocks only, at max_batch */
  uint64_t scratch_bytes;           /* forward/backward scratch shared by all blocks */
  uint64_t paper_activation_bytes;  /* the same blocks in the paper's fp32 accounting (Table 1), at max_batch */
  uint64_t trainable_params;
  uint64_t block_saved_bytes[BSR_MAX_DEPTH]; /* per block, its share of saved_activation_bytes (0 before the earliest
                                               trainable block); the earliest one also holds the fp32 input of the path */
} bsr_footprint;

typedef struct bsr_handle bsr_handle;

/* Token schedule implied by a configuration (Section 4.1: K from the drop rate; Section 4.3,
 * Discussion 3: the MHSA of a drop location sees all incoming tokens, its FFN the reduced set).
 * Host-only.  Writes, for each block l < depth, the tokens entering its MHSA (tokens_attn[l]), the
 * tokens entering its FFN (tokens_ffn[l]) and K (keep[l], or -1 if l is not a drop location), with
 * K = ceil(keep_num * M / keep_den) clamped to [1, M], M = incoming tokens minus the classification
 * token.  Arrays are host memory of `depth` int32 each, owned by the caller. */
int32_t bsr_token_schedule(const bsr_config* cfg_host, int32_t* tokens_attn_host, int32_t* tokens_ffn_host,
                           int32_t* keep_host);

/* Size of the workspace bsr_create needs for this configuration.  Host-only. */
int32_t bsr_workspace_bytes(const bsr_config* cfg_host, size_t* bytes_host);

/* Creates the step engine (Fig. 2).  `workspace_dev` must be 256-byte aligned device memory of at
 * least bsr_workspace_bytes() bytes and must outlive the handle.  Validates the configuration
 * (BSR_ERR_INVALID_ARG), rejects what is not built (BSR_ERR_UNSUPPORTED: MoE layers outside bf16 or with
 * dim / mlp_hidden not multiples of 64), zeroes optimiser state and sets the step counter to 0.  Parameters are
 * undefined until set with bsr_set_param.  On failure *out_host is NULL. */
int32_t bsr_create(const bsr_config* cfg_host, void* workspace_dev, size_t bytes, bsr_handle** out_host);

int32_t bsr_destroy(bsr_handle* h);

/* Static, human-readable description of the last error on this handle (or of the last failed
 * handle-less call when h is NULL).  Never NULL; valid until the next call on the same handle. */
const char* bsr_last_error(const bsr_handle* h);

/* Loads one parameter ("pre-trained weights", Section 5).  `src` holds `count` values of type `src_dtype`
 * (BSR_DTYPE_FP32: float32; BSR_DTYPE_BF16: bfloat16 bit patterns) in device memory (src_is_device != 0) or in host
 * memory (src_is_device == 0); they are converted to the storage dtype (and widened into the fp32 master for trainable
 * tensors) on `stream`.  `count` must equal the tensor's element count.  A host source is first copied into a staging
 * area of the workspace: pageable memory may be released when the call returns, pinned memory only once `stream` has
 * reached this point; all parameter loads of a handle must be issued on one stream (they share the staging area). */
int32_t bsr_set_param(bsr_handle* h, const char* name, const void* src, size_t count, int32_t src_dtype, int32_t src_is_device,
                      void* stream);

/* Reads a tensor as float32 into device memory `dst_dev` (capacity `count` elements, which must
 * equal the tensor's size) on `stream`.  Names: a parameter name (the fp32 master if it trains,
 * else the stored weight widened), "grad/<param>", "adam_m/<param>", "adam_v/<param>" (trainable
 * parameters only), "logits" ([max_batch, max classes], rows of the last step; classes a task does
 * not have hold -inf), "loss" (1 element), "scores/<l>" (Eq. 6: the head-mean classification-token attention of the
 * last step at the drop location in block l, [max_batch, M], rows of images beyond the last batch undefined),
 * "fp8/blocks.<l>.attn.qkv.weight" / "fp8/blocks.<l>.mlp.fc1.weight" (frozen_fp8: the E4M3 copy of that prefix weight
 * scaled back to float), "moe_experts/<l>" (the experts chosen by block l's router in the last step, [tokens routed, top_k] as floats,
 * best first; the last block routes only the classification rows; `count` may be any prefix of the record). */
int32_t bsr_get_tensor(bsr_handle* h, const char* name, float* dst_dev, size_t count, void* stream);

/* Learning rate for the next steps (the cosine schedule of Section 5 lives in the caller). */
int32_t bsr_set_lr(bsr_handle* h, float lr);
/* Number of optimiser steps already taken (for bias correction when resuming). */
int32_t bsr_set_step(bsr_handle* h, int64_t steps_done);

/* One BSR fine-tuning step (Fig. 2; Section 4.1; Eq. 2-5 and Eq. 8 for the backward pass): forward
 * through the frozen blocks without saving activations, token selection and fusion at the drop
 * locations, forward + backward of the trainable blocks and head, AdamW on their parameters.
 *   images_dev   [batch, in_chans, image_size, image_size] in the storage dtype (fp32 or bf16 bits)
 *   labels_dev   [batch] int32, each in [0, num_classes[task])
 *   task_ids_dev [batch] int32, or NULL when num_tasks == 1
 *   loss_dev_out 1 float32: mean cross-entropy of the batch before the update
 *   kept_idx_dev_out  optional (may be NULL): int32, concatenated over drop locations i, each
 *                [batch, K_i]: positions (0-based, among the M non-classification tokens entering
 *                that location, ascending) of the tokens kept for each image.
 * batch must be in [1, max_batch]. */
int32_t bsr_train_step(bsr_handle* h, const void* images_dev, const int32_t* labels_dev,
                       const int32_t* task_ids_dev, int32_t batch, void* stream,
                       float* loss_dev_out, int32_t* kept_idx_dev_out);

/* A run of n_steps fine-tuning steps with the cosine learning-rate decay of Section 5 (training hyper-parameters)
 * evaluated on the device: step t of the whole training (t counts optimiser steps from 0, continuing from the handle's
 * step counter) uses lr(t) = lr_min + (lr_max - lr_min) (1 + cos(pi t / total_steps)) / 2, held at lr_min from
 * t = total_steps on.  The step counter, the learning rate, the bias corrections and the position in the input arrays
 * live in device memory and every step is one replay of the same captured graph (when `stream` can be captured, as
 * for bsr_train_step), so the host supplies no scalars between steps.
 *   images_dev   [n_steps, batch, in_chans, image_size, image_size] in the storage dtype: a fresh batch per step
 *                (batch * in_chans * image_size^2 elements must be a multiple of 16 bytes)
 *   labels_dev   [n_steps, batch] int32;  task_ids_dev [n_steps, batch] int32 or NULL when num_tasks == 1
 *   loss_dev_out [n_steps] float32: the mean cross-entropy of every step before its update
 *   kept_idx_dev_out  optional, laid out as for bsr_train_step: the kept positions of the LAST step
 * Afterwards bsr_set_lr's value is the schedule's learning rate of the last step taken. */
typedef struct {
  float lr_max, lr_min;
  int64_t total_steps;
} bsr_lr_schedule;
int32_t bsr_train_steps(bsr_handle* h, const void* images_dev, const int32_t* labels_dev, const int32_t* task_ids_dev,
                        int32_t batch, int32_t n_steps, const bsr_lr_schedule* schedule_host, void* stream,
                        float* loss_dev_out, int32_t* kept_idx_dev_out);

/* Data-parallel training over several GPUs (one process and one handle per GPU, each with its share of the batch):
 * bsr_train_step in two halves with the caller's gradient exchange between them.  The images of a batch are independent
 * up to the batch-mean loss, so the only coupling between the shares is the mean of their gradients:
 *   bsr_forward_backward  forward, loss and backward of this GPU's share; the gradients of the local mean loss are
 *                         left in the gradient buffer, nothing is updated (arguments as for bsr_train_step);
 *   bsr_grad_buffer       the gradient buffer: `count` float32 values holding every trainable tensor (each padded to
 *                         a multiple of 64 values, padding zero).  Average it over the GPUs in place on the same
 *                         stream -- one all-reduce (NCCL over NVLink), equal shares assumed -- and every GPU holds
 *                         the gradient of the global batch mean;
 *   bsr_optimizer_step    AdamW / SGD on the buffer as it stands, with the bias corrections of the next step; advances
 *                         the step counter.
 * On one GPU the three calls equal bsr_train_step bit for bit.  The library itself never communicates. */
int32_t bsr_forward_backward(bsr_handle* h, const void* images_dev, const int32_t* labels_dev, const int32_t* task_ids_dev,
                             int32_t batch, void* stream, float* loss_dev_out, int32_t* kept_idx_dev_out);
int32_t bsr_grad_buffer(bsr_handle* h, float** grads_dev_out_host, size_t* count_out_host);
int32_t bsr_optimizer_step(bsr_handle* h, void* stream);

/* bsr_train_step fed from and read back into HOST memory (the same step; Fig. 2).  images_host, labels_host and
 * task_ids_host are copied into one of two staging slots inside the workspace on a copy stream the library owns, so
 * that the copy for this step overlaps the kernels of the previous one; the step runs on `stream`; the loss (and, if
 * kept_idx_host_out is not NULL, the kept positions) are copied back to host memory on `stream`.  Nothing is
 * synchronised: loss_host_out is valid once `stream` has reached the end of this call's work.  Use pinned host memory
 * for the overlap; with pinned memory the input buffers must stay untouched until then as well.  Layouts as for
 * bsr_train_step. */
int32_t bsr_train_step_host(bsr_handle* h, const void* images_host, const int32_t* labels_host, const int32_t* task_ids_host,
                            int32_t batch, void* stream, float* loss_host_out, int32_t* kept_idx_host_out);

/* Inference with the same token dropping (Section 2: unlike other on-device methods the dropping
 * also speeds up inference).  logits_dev_out: [batch, max classes] float32. */
int32_t bsr_eval_forward(bsr_handle* h, const void* images_dev, const int32_t* task_ids_dev, int32_t batch,
                         void* stream, float* logits_dev_out, int32_t* kept_idx_dev_out);

/* Memory report (Section 3.2, Table 1: activations dominate training memory). Host-only. */
int32_t bsr_get_footprint(const bsr_handle* h, bsr_footprint* out_host);

/* Checks the guard words that follow every slice of the workspace (weights, optimiser state, each saved activation,
 * each scratch buffer), synchronises `stream` and reads the device status word: BSR_OK, BSR_ERR_DEVICE_TIMEOUT if a
 * bounded wait in a kernel expired, BSR_ERR_MEMORY_GUARD if a kernel wrote past the end of its slice,
 * BSR_ERR_DEVICE_CHECK if an index check of the checked build failed, BSR_ERR_NONFINITE if the last loss was not
 * finite.  Clears the status word (an overwritten guard stays overwritten and is reported again). */
int32_t bsr_sync_status(bsr_handle* h, void* stream);

/* Diagnostic of the failure path (no counterpart in the paper).  Every device-side wait of the tensor-core kernels
 * is bounded; when one expires the CTA raises a status bit, frees its tensor memory and returns, and the next
 * bsr_sync_status reports BSR_ERR_DEVICE_TIMEOUT with the context still usable.  This call runs exactly that path on
 * purpose: it enqueues one CTA that waits, for at most limit_ns nanoseconds (1e3 .. 1e8), on a barrier nothing ever
 * arrives at.  Nothing faults and nothing hangs; the following bsr_sync_status returns BSR_ERR_DEVICE_TIMEOUT and
 * clears the status word.  bf16 handles only. */
int32_t bsr_selftest_wait_expiry(bsr_handle* h, uint64_t limit_ns, void* stream);

/* Which kernels run the dense contractions and attention of a bf16 handle (no counterpart in the paper):
 * 0 = the FP32-FMA kernels of the fp32 configuration (slow; a cross-check), 1 = tcgen05 kernels with one CTA per
 * tile (the default), 2 = as 1 but GEMMs with more than 128 rows run on CTA pairs (cta_group::2). */
int32_t bsr_set_gemm_mode(bsr_handle* h, int32_t mode);

/* bsr_train_step replays a captured CUDA graph of its ~200 launches when `stream` can be captured (any stream but
 * the legacy default stream, and not one the caller is capturing) -- the first call with a given set of pointers
 * and batch captures it, later calls with the same arguments replay it.  The key of a captured graph is (images,
 * labels, task ids, loss and kept-index pointers, batch, kernel mode); the handle keeps the eight most recently
 * used graphs, so an input pipeline should rotate through at most eight sets of buffers (bsr_profile.graph_captures
 * counts captures: it stops growing once a pipeline fits).  on = 0 turns this off (every call enqueues its kernels
 * one by one); the results are identical.  No counterpart in the paper. */
int32_t bsr_set_graph_mode(bsr_handle* h, int32_t on);

/* Measurement support (no counterpart in the paper).  bsr_profile_enable resets the counters; with
 * time_gemms != 0 every tensor-core GEMM launch of the following steps is bracketed by a pair of CUDA
 * events on the launching stream (host objects; this slows the step slightly, so timed throughput is
 * taken with it off).  bsr_profile_read synchronises `stream` and reports, since the last enable: kernels
 * launched by the library (host count, whole process), and for the timed GEMMs their number, their
 * algorithmic FLOPs (2 m n k each) and the sum of their durations in milliseconds. */
typedef struct {
  uint64_t kernel_launches;
  uint64_t gemm_launches;
  double gemm_flops;
  double gemm_ms;
  uint64_t graph_captures;          /* training-step graphs captured by this handle since it was created */
} bsr_profile;
int32_t bsr_profile_enable(bsr_handle* h, int32_t time_gemms);
int32_t bsr_profile_read(bsr_handle* h, void* stream, bsr_profile* out_host);
/* Per-launch view of the same timed GEMMs, in launch order: writes up to `capacity` entries of FLOPs and
 * milliseconds into host arrays and the number of timed launches into *count_out_host. */
int32_t bsr_profile_launches(bsr_handle* h, void* stream, int32_t capacity, double* flops_out_host, float* ms_out_host,
                             int32_t* count_out_host);

/* ---- stand-alone forms of the paper-specific token kernels (no handle) ---------------------- */

/* Token importance and top-K (Eq. 6; Section 4.1).  p_dev [batch, heads, m] float32: for every
 * head the classification token's attention probabilities to the m other tokens.  Computes
 * s[b, j] = (p[b,0,j] + ... + p[b,heads-1,j]) / heads in float32, summed in head order, and keeps
 * the k largest per image (equal scores: lower index first).
 *   scores_dev_out  [batch, m] float32
 *   kept_dev_out    [batch, k] int32 ascending;  dropped_dev_out [batch, m-k] int32 ascending
 * 1 <= k <= m <= 4096. */
int32_t bsr_token_select(const float* p_dev, int32_t batch, int32_t heads, int32_t m, int32_t k,
                         float* scores_dev_out, int32_t* kept_dev_out, int32_t* dropped_dev_out, void* stream);

/* Compaction between MHSA and FFN (Section 4.1: kept tokens preserved, the others fused).
 * x_dev [batch, 1+m, dim] in `dtype`; out_dev [batch, 1+k+f, dim] with f = 1 when
 * fuse_mode != BSR_FUSE_NONE and k < m, else 0.  Row 0 is copied, rows 1..k are the kept
 * rows in the order of kept_dev, the last row is sum_j scores[b, j] * x[b, 1+j] over dropped j
 * (float32 accumulation in a fixed order), divided by sum_j scores[b, j] for BSR_FUSE_WEIGHTED_MEAN.
 * dim * sizeof(dtype) must be a multiple of 16. */
int32_t bsr_gather_fuse(const void* x_dev, int32_t dtype, int32_t batch, int32_t m, int32_t dim, int32_t k,
                        const int32_t* kept_dev, const int32_t* dropped_dev, const float* scores_dev,
                        int32_t fuse_mode, void* out_dev, void* stream);

/* ---- stand-alone forms of the dense kernels, for unit checks against the oracle ------------- */

/* y = act(x W^T + bias) + residual (FFN / projection layers of Section 3.1).  x [m, k], w [n, k],
 * y [m, n], residual [m, n] or NULL, bias [n] float32 or NULL; x, w, y, residual in `dtype`;
 * act_gelu != 0 applies the exact GELU.  use_tensor_cores != 0 selects the tcgen05 kernel (bf16 only). */
int32_t bsr_linear_forward(const void* x_dev, const void* w_dev, const float* bias_dev, const void* residual_dev,
                           void* y_dev, int32_t m, int32_t n, int32_t k, int32_t dtype, int32_t act_gelu,
                           int32_t use_tensor_cores, void* stream);

/* The same product with both operands rounded to E4M3 row by row, as the 8-bit prefix computes it (frozen_fp8):
 * y = act((x_q W_q^T) * sx * sw + bias), x_q[r] = round_e4m3(x[r] / sx[r]), sx[r] = max|x[r]| / 448, likewise for the rows
 * of W.  x [m, k], w [n, k], y [m, n] bf16, bias [n] float32 or NULL; k a multiple of 16, n of 8.  scratch_dev: at
 * least m*k + n*k + 4*(m + n) + 1024 bytes of device memory for the quantised copies and their scales. */
int32_t bsr_linear_forward_e4m3(const void* x_dev, const void* w_dev, const float* bias_dev, void* y_dev, int32_t m, int32_t n,
                                int32_t k, int32_t act_gelu, void* scratch_dev, size_t scratch_bytes, void* stream);

/* Backward of y = x W^T: dx = dy W (Eq. 2: needs only the weights) and dw = dy^T x (Eq. 4: needs the stored
 * input).  x [m, k], w [n, k], dy [m, n], dx [m, k] in `dtype`; dw [n, k] float32.  With
 * use_tensor_cores != 0 (bf16, m, n, k multiples of 8) the operands are read in place through
 * transposing shared-memory descriptors; workspace_dev (float32, may be NULL) lets a long
 * reduction over m be split and summed in a fixed order. */
int32_t bsr_linear_backward(const void* x_dev, const void* w_dev, const void* dy_dev, void* dx_dev, float* dw_dev,
                            int32_t m, int32_t n, int32_t k, int32_t dtype, int32_t use_tensor_cores,
                            float* workspace_dev, size_t workspace_floats, void* stream);

/* The same backward pass for callers that cannot allocate device memory (the paper has no counterpart:
 * this is a property of the library, not of the method).  Such callers exist: a trainer on a device whose
 * memory was divided up once at start-up, a plug-in inside an application that owns all device memory
 * through its own pool, a latency-critical loop that must not pay cudaMalloc's device-wide synchronisation.
 * The split-reduction scratch that bsr_linear_backward takes from its caller is here a fixed array of
 * BSR_STATIC_SCRATCH_BYTES inside the library image; every GPU that loads the library holds it until the
 * process exits.  bf16 only; x [m, k], w [n, k], dy [m, n], dx [m, k] bf16, dw [n, k] float32, all device
 * memory owned by the caller; m, n, k multiples of 8.  n * k must not exceed BSR_STATIC_SCRATCH_BYTES / 8
 * elements, otherwise BSR_ERR_WORKSPACE_TOO_SMALL is returned and nothing runs.  The call allocates and
 * frees nothing.  The first call on each device looks up the array's device address (with that device
 * current) and should therefore come before any stream capture; where the CUDA runtime loads device code lazily,
 * that first call is also when the device image with the array is loaded and its bytes are taken.  All calls on a device share the one
 * array: each call fully rewrites the part it reads, so nothing needs clearing between calls, but two
 * calls whose kernels overlap on the GPU (different streams) race on it -- keep them on one stream or
 * order them with events.  Errors are described by bsr_static_last_error(). */
#define BSR_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
int32_t bsr_linear_backward_static(const void* x_dev, const void* w_dev, const void* dy_dev, void* dx_dev, float* dw_dev,
                                   int32_t m, int32_t n, int32_t k, void* stream);
const char* bsr_static_last_error(void);

/* Multi-head self-attention, Eq. 1, on packed projections.  qkv_dev [batch, t, 3, heads, d] in
 * `dtype`; out_dev [batch, t, heads*d]; cls_prob_dev_out optional [batch, heads, t-1] float32: the
 * classification token's row of the attention map without its own column; lse_dev_out optional
 * [batch, heads, t] float32: log of the softmax denominator of every row (natural logarithm, of the scaled scores),
 * which bsr_attention_backward reads.  d must be 64 or less and a multiple of 8.  use_tensor_cores != 0 selects the
 * tcgen05 kernels (bf16, d = 64).  All buffers are caller-owned device memory. */
int32_t bsr_attention_forward(const void* qkv_dev, int32_t dtype, int32_t batch, int32_t t, int32_t heads,
                              int32_t d, void* out_dev, float* cls_prob_dev_out, float* lse_dev_out,
                              int32_t use_tensor_cores, void* stream);

/* Backward of Eq. 1 (the attention part of Eq. 3): from dout_dev [batch, t, heads*d], the gradient at the attention
 * output, to dqkv_dev_out [batch, t, 3, heads, d], the gradient at the packed projections; both in `dtype`.  The
 * attention map is recomputed from qkv_dev and lse_dev (as written by bsr_attention_forward).  score_grad_dev optional
 * [batch, t-1] float32: a gradient arriving at the head-mean classification scores of Eq. 6 (from the fused token);
 * every head's classification row receives 1/heads of it.  delta_scratch_dev: batch*heads*t floats of caller-owned
 * scratch (used by the kernels without tensor cores; may be null when use_tensor_cores != 0).  use_tensor_cores != 0
 * selects the tcgen05 kernels (bf16, d = 64, t <= 256) and fails with BSR_ERR_UNSUPPORTED outside their range. */
int32_t bsr_attention_backward(const void* qkv_dev, const void* dout_dev, const float* lse_dev, const float* score_grad_dev,
                               int32_t dtype, int32_t batch, int32_t t, int32_t heads, int32_t d, void* dqkv_dev_out,
                               float* delta_scratch_dev, int32_t use_tensor_cores, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BSR_H_ */
