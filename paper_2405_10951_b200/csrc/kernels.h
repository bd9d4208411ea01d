// Host-side launchers of the BSR kernels.  Every launcher enqueues on ctx.stream and returns;
// pointers are device addresses; `dtype` selects the storage type of activations and matrices
// (0 = float, 1 = bf16); LayerNorm parameters, biases, statistics, scores and gradients of
// parameters are always float.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

namespace bsr {

// Optional timing of the tensor-core GEMM launches: each launch is bracketed by a pair of CUDA events on the
// launching stream (events are host objects; no device memory is involved).
struct GemmProfile {
  bool on = false;
  std::vector<cudaEvent_t> events;   // pairs
  size_t used = 0;
  double flops = 0.0;
  std::vector<double> launch_flops;
  void begin(cudaStream_t s, double f) {
    if (used + 2 > events.size()) {
      size_t old = events.size();
      events.resize(old + 512);
      for (size_t i = old; i < events.size(); ++i) cudaEventCreate(&events[i]);
    }
    cudaEventRecord(events[used], s);
    flops += f;
    launch_flops.push_back(f);
  }
  void end(cudaStream_t s) {
    cudaEventRecord(events[used + 1], s);
    used += 2;
  }
};

// Reductions whose results only the optimiser reads (split sums of weight gradients, partial sums of LayerNorm
// parameter gradients and of bias gradients) need not sit on the chain of the backward pass: they are enqueued on a
// second stream that forks from the main one and is joined before the buffer they read is written again, and before
// the update.  Inside a stream capture the fork and the joins become edges of the graph.
struct SideLane {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr;
  cudaEvent_t done[3] = {nullptr, nullptr, nullptr};   // 0: LayerNorm partials, 1: column-sum partials, 2: split-k workspace
  bool pending[3] = {false, false, false};
};

struct Ctx {
  cudaStream_t stream;
  int dtype;        // 0 fp32, 1 bf16
  int* status;      // device status word (may be null for the stand-alone entry points)
  int sm_count;
  int use_tc;       // bf16 only: dense contractions on the tcgen05 kernels
  float* split_ws = nullptr;       // scratch for split-k partial sums (optional)
  size_t split_ws_floats = 0;
  GemmProfile* prof = nullptr;
  SideLane* side = nullptr;        // optional second lane for optimiser-only reductions
};

// The main stream is about to rewrite buffer `which`: wait for the side reduction that may still read it.
inline void side_join(const Ctx& c, int which) {
  if (c.side != nullptr && c.side->pending[which]) {
    cudaStreamWaitEvent(c.stream, c.side->done[which], 0);
    c.side->pending[which] = false;
  }
}
inline void side_join_all(const Ctx& c) {
  for (int w = 0; w < 3; ++w) side_join(c, w);
}
// Stream for a reduction of buffer `which`: the side lane, made to wait for everything enqueued on the main stream so far
// (the main stream itself when there is no side lane).  side_end marks the reduction as in flight.
inline cudaStream_t side_begin(const Ctx& c) {
  if (c.side == nullptr) return c.stream;
  cudaEventRecord(c.side->fork, c.stream);
  cudaStreamWaitEvent(c.side->stream, c.side->fork, 0);
  return c.side->stream;
}
inline void side_end(const Ctx& c, int which) {
  if (c.side == nullptr) return;
  cudaEventRecord(c.side->done[which], c.side->stream);
  c.side->pending[which] = true;
}

inline size_t dtype_size(int dtype) { return dtype == 0 ? 4 : 2; }

// ---- embedding --------------------------------------------------------------------------------
// img_offset (optional, device): element offset of the images from `images`, read when the kernel runs.
void patchify(const Ctx& c, const void* images, void* patches, int B, int C, int S, int P, const long long* img_offset = nullptr);
void assemble_tokens(const Ctx& c, const void* emb, const float* cls, const float* pos, float* x, int B, int N, int D);

// ---- LayerNorm (the residual stream is float in every configuration) ----------------------------
// y[r] = LN(x[r]) * g + b for `rows` rows of length D; row r of x starts at x + r * x_stride elements.
// y takes the storage dtype unless y_is_float.  mean/rstd (optional) receive the row statistics.
void layernorm_fwd(const Ctx& c, const float* x, long x_stride, const float* g, const float* b, void* y, int y_is_float,
                   float* mean, float* rstd, int rows, int D, float eps);
// dx[r] = dres[r] + LN'(dy[r]) (float; rows dx_stride apart); dx_copy (optional, bf16 configurations) receives
// the same rows in the storage dtype.  Partial sums of dgamma/dbeta go to `partials` ([2][groups][D]) and are
// reduced in a fixed order; with dx_colsum the column sums of dx (a bias gradient of the layer that produced the
// normalised input's predecessor) come out of the same pass ([3][groups][D] partials).  dx may be null (only parameter gradients wanted); dres may be null.
// dy is in the storage dtype, or float [rows, D] when dy_is_float (head path).
void layernorm_bwd(const Ctx& c, const void* dy, int dy_is_float, const float* x, long x_stride, const float* mean,
                   const float* rstd, const float* g, const float* dres, float* dx, long dx_stride, void* dx_copy,
                   float* partials, float* dgamma, float* dbeta, int rows, int D, float* dx_colsum = nullptr);
int layernorm_bwd_groups(const Ctx& c, int rows);

// ---- column sums (bias gradients) -------------------------------------------------------------
void colsum(const Ctx& c, const void* x, int rows, int cols, float* partials, float* out);
int colsum_groups(int rows);

// ---- dense contractions -----------------------------------------------------------------------
// C[m, n] = epilogue(sum_k A(m, k) * B(n, k)).  A(m,k) = A[m * a_rs + k * a_cs], B alike.
// Expert grouping of a contraction (MoE layer).  mode 0: none.  mode 1: every 128-row tile of A / C belongs to one
// expert (tile_expert[tile], -1 = unused tile) whose slice of the stacked weights and biases is used.  mode 2:
// weight gradients, one output matrix per expert, reduced over that expert's row segment (seg_start[e] ..
// seg_start[e+1], multiples of 128).
struct GemmGroup {
  const int* tile_expert = nullptr;
  const int* seg_start = nullptr;
  int mode = 0;
  int b_stride = 0;
  int bias_stride = 0;
  long c_stride = 0;
};

struct GemmEpilogue {
  const float* bias = nullptr;      // [n]
  const void* residual = nullptr;   // [m, n] in the output type, added last
  int act = 0;                      // 0 none, 1 GELU (pre-activation optionally stored), 2 multiply by GELU'(aux_in)
  void* aux_out = nullptr;          // act 1: pre-activation [m, n], output type; act 2 (optional): GELU(aux_in) [m, n], storage type
  const void* aux_in = nullptr;     // act 2: pre-activation [m, n], storage type
};
void gemm(const Ctx& c, const void* A, long a_rs, long a_cs, const void* B, long b_rs, long b_cs, void* C,
          int out_is_float, int m, int n, int k, const GemmEpilogue& e);
// True when the tcgen05 kernel can take this problem (bf16, both operands contiguous along k, aligned).
bool gemm_tc_supported(int m, int n, int k);
int gemm_tc(const Ctx& c, const void* A, const void* B, void* C, int out_is_float, int m, int n, int k,
            const GemmEpilogue& e);
// E4M3 operands (one byte per element, k contiguous), one float scale per row of A and per row of B; bf16 output.
// e: bias, GELU (act 1) and the stored pre-activation; no residual.  k a multiple of 16, n of 8.
int gemm_tc_e4m3(const Ctx& c, const void* Aq, const float* a_scale, const void* Bq, const float* b_scale, void* C, int m, int n,
                 int k, const GemmEpilogue& e);
// Rows of x [rows, cols] (bf16) to E4M3 with scale[r] = max|row| / 448 (1 for a zero row): q = round(x / scale).
void quantize_rows_e4m3(const Ctx& c, const void* x, int rows, int cols, void* q, float* scale);
// q * scale back to float (for inspection).
void dequantize_rows_e4m3(const Ctx& c, const void* q, const float* scale, int rows, int cols, float* out);
// LayerNorm forward with the normalised row written as E4M3 and its scale (max|y| / 448) beside it.
void layernorm_fwd_e4m3(const Ctx& c, const float* x, long x_stride, const float* g, const float* b, void* yq, float* y_scale,
                        int rows, int D, float eps);
// Same with operand strides as in gemm(); each operand contiguous along k or along its own index.  A problem
// with few output tiles and a long k (weight gradients) is split along k into split_ws and reduced in order.
int gemm_tc_strided(const Ctx& c, const void* A, long a_rs, long a_cs, const void* B, long b_rs, long b_cs, void* C,
                    int out_is_float, int m, int n, int k, const GemmEpilogue& e, float* split_ws, size_t split_ws_floats);

// C[rows_cap, n] = epilogue(A[rows_cap, k] . W_e) with W_e the expert's slice of stacked weights: Bst [E*n, k]
// (b_mn = 0, forward) or [E*k, n] (b_mn = 1, input gradient: C = A W_e).  bf16 operands, bf16 or float output; e.bias stacked [E*n].
int gemm_tc_grouped_rows(const Ctx& c, const void* A, const void* Bst, int b_mn, void* C, int out_is_float, int rows_cap, int n, int k,
                         int experts, const int* tile_expert, const GemmEpilogue& e);
// dW[e][m, n] = sum over rows r of expert e's segment of dY[r, m] * X[r, n]  (float out).
int gemm_tc_grouped_wgrad(const Ctx& c, const void* dY, const void* X, float* dW, int rows_cap, int m, int n, int experts,
                          const int* seg_start);
// The same on CTA pairs (tcgen05 cta_group::2, 256 x 256 tiles); preferred when m > 128.
int gemm_tc2_strided(const Ctx& c, const void* A, long a_rs, long a_cs, const void* B, long b_rs, long b_cs, void* C,
                     int out_is_float, int m, int n, int k, const GemmEpilogue& e, float* split_ws, size_t split_ws_floats);
void splitk_reduce(cudaStream_t s, const float* partial, float* out, size_t n, int splits);
// Diagnostic: one CTA whose bounded wait expires after limit_ns and which then tears down as the GEMM kernels do.
void wait_expiry_selftest(const Ctx& c, unsigned long long limit_ns);

// ---- attention --------------------------------------------------------------------------------
// qkv [B, T, 3, H, d]; out [B, T, H*d]; lse (optional) [B, H, T] natural-log sum of exponentials of the
// scaled scores; cls_prob (optional) [B, H, T-1].
// tcgen05 kernels (bf16, head dimension 64); return non-zero when they do not take the problem.
int attention_fwd_tc(const Ctx& c, const void* qkv, void* out, float* lse, float* cls_prob, int B, int T, int H, int d);
int attention_bwd_tc(const Ctx& c, const void* qkv, const void* dout, const float* lse, const float* cls_extra, void* dqkv,
                     int B, int T, int H, int d);
int attention_fwd(const Ctx& c, const void* qkv, void* out, float* lse, float* cls_prob, int B, int T, int H, int d);
// dqkv from dout; delta scratch [B, H, T]; cls_extra (optional) [B, T-1]: gradient arriving at the head-mean
// score of each non-classification token (zero for kept tokens); cls_prob needed with it.
int attention_bwd(const Ctx& c, const void* qkv, const void* out, const void* dout, const float* lse, float* delta,
                  const float* cls_extra, void* dqkv, int B, int T, int H, int d);

// The classification row alone (last block: only that row of the block's output is ever read).  out_cls / dout_cls
// [B, H*d]: attention output of query 0 and its gradient; dqkv [B, T, 3, H, d] is written in full (rows of dQ other
// than the first are zero).  Return non-zero when the problem does not fit (more than 1024 tokens, a head dimension above 64 or not a multiple of 8).
int attention_cls_fwd(const Ctx& c, const void* qkv, void* out_cls, int B, int T, int H, int d);
int attention_cls_bwd(const Ctx& c, const void* qkv, const void* dout_cls, void* dqkv, int B, int T, int H, int d);

// ---- token selection --------------------------------------------------------------------------
void token_select(cudaStream_t s, const float* p, int B, int H, int M, int k, float* scores, int* kept, int* dropped);
void gather_fuse(const Ctx& c, const void* x, int B, int M, int D, int k, const int* kept, const int* dropped,
                 const float* scores, int fuse, void* out);
// Backward of the compaction: dx [B, 1+M, D] from dout [B, 1+k+f, D]; escore [B, M] = gradient arriving at the fusion
// weight of each dropped token (<g_fused, x_j> for the weighted sum), 0 for kept ones.  fuse: 0 none, 1 weighted sum,
// 2 weighted mean (needs fwd_out, the forward pass's compacted tensor [B, 1+k+1, D] float, for the fused row).
// dx_copy (optional): the same rows in bf16 for the GEMMs that consume them (float streams only).
void gather_fuse_bwd(const Ctx& c, const void* dout, const void* x, int B, int M, int D, int k, const int* kept,
                     const int* dropped, const float* scores, int fuse, void* dx, void* dx_copy, float* escore, const void* fwd_out);

// ---- head, loss, optimiser --------------------------------------------------------------------
// logits[b, c] = xn[b] . W_task(b)[c] + bias; classes beyond the task's count get -inf.
struct HeadDesc {
  int num_tasks, cmax, D;
  int ncls[4];
  const void* w[4];       // storage dtype [ncls, D]
  const float* bias[4];
  float* dw[4];           // gradients (float)
  float* db[4];
};
void head_fwd(const Ctx& c, const HeadDesc& h, const float* xn, const int* task_ids, float* logits, int B);
void cross_entropy(const Ctx& c, const HeadDesc& h, const float* logits, const int* labels, const int* task_ids,
                   float* per_image, float* dlogits, float* loss, int B);
void head_bwd(const Ctx& c, const HeadDesc& h, const float* xn, const float* dlogits, const int* task_ids, float* dxn, int B);

struct AdamChunk { uint32_t offset; uint32_t count; int64_t shadow; uint32_t decay; uint32_t pad; };
// scalars (device): learning rate, 1 - beta1^t, 1 - beta2^t of the step being taken.
void adamw(const Ctx& c, const AdamChunk* chunks, int nchunks, float* master, const float* grad, float* m, float* v,
           void* shadow_base, const float* scalars, float b1, float b2, float eps, float wd);
// SGD with momentum (buf starts at zero): buf <- mu buf + (g + wd p on decayed tensors), p <- p - lr buf; lr from scalars[0].
void sgd_momentum(const Ctx& c, const AdamChunk* chunks, int nchunks, float* master, const float* grad, float* buf,
                  void* shadow_base, const float* scalars, float mu, float wd);
void set_scalars(cudaStream_t s, float* dst, float a, float b, float c3);

// Device-resident state of a run of steps with a cosine learning-rate schedule (Section 5).
struct LoopState {
  long long step_done;       // optimiser steps taken before the current one
  long long total_steps;     // length of the schedule
  long long image_stride;    // elements between the images of successive steps
  long long image_offset;    // element offset of the current step's images
  float lr_max, lr_min, beta1, beta2;
  int i, n;                  // index of the current step within the call, steps of the call
};
void loop_init(cudaStream_t s, LoopState* st, long long step_done, long long total, long long image_stride, float lr_max, float lr_min,
               float b1, float b2, int n);
// Start of a step: learning rate and bias corrections of this step into scalars[0..2], this step's labels and task
// ids into the staging arrays, the image offset into the state.
void loop_begin(cudaStream_t s, LoopState* st, float* scalars, const int* labels, const int* tasks, int* lab_stage, int* task_stage, int batch);
// End of a step: loss_out[i] = loss, counters advance.
void loop_end(cudaStream_t s, LoopState* st, const float* loss, float* loss_out);

// dst row r = src row r (row_bytes a multiple of 16), independent pitches: gathers / scatters token rows.
void copy_rows(cudaStream_t s, const void* src, long src_pitch_bytes, void* dst, long dst_pitch_bytes, int rows, int row_bytes);

// ---- mixture of experts (routing, grouping, combination; the expert MLPs are grouped GEMMs) -----------------------
struct MoeBufs {
  int* eidx;          // [M, K] chosen experts per token, best first
  float* ew;          // [M, K] their weights (softmax over the chosen gate logits)
  int* pos;           // [M, K] row of each (token, slot) in the expert-ordered buffers
  int* row_token;     // [rows_cap] token of each row, -1 for padding
  float* row_w;       // [rows_cap] weight of each row
  int* seg_start;     // [E + 1] first row of each expert's segment (multiples of 128)
  int* tile_expert;   // [rows_cap / 128] expert of each 128-row tile, -1 beyond the last segment
  int* blk_counts;    // [blocks, E]
  int* blk_off;       // [blocks, E]
  void* xg;           // [rows_cap, D] gathered expert inputs
  void* zg;           // [rows_cap, F] FC1 pre-activation (kept by trainable blocks)
  void* hg;           // [rows_cap, F] GELU output
  float* og;          // [rows_cap, D] expert outputs (float: they are summed into the residual stream)
};
int moe_rows_cap(int M, int E, int K);
int moe_blocks(int M);
// y [M, D]: routes every token, builds the segment tables and gathers the expert inputs into b.xg.  logits (optional):
// the gate logits of all tasks, [M, logit_stride] with task t's experts at columns t E .. t E + E - 1, formed beforehand
// (y times the transposed gate matrices); without them the kernel forms each token's own task's logits itself.
void moe_route(const Ctx& c, const MoeBufs& b, const void* y, const void* wg, const int* task_ids, int tokens_per_image, int M,
               int D, int E, int K, int num_tasks, const float* logits = nullptr, int logit_stride = 0);
void moe_combine(const Ctx& c, const MoeBufs& b, const float* res, float* out, int M, int D, int K);
void moe_combine_bwd(const Ctx& c, const MoeBufs& b, const float* dout, void* dog, float* dw, int M, int D, int E, int K);
void moe_seg_colsum(const Ctx& c, const MoeBufs& b, const void* x, int cols, int E, float* out);
void moe_gate_bwd(const Ctx& c, const MoeBufs& b, const void* dxg, const float* dw, const void* wg, const int* task_ids,
                  int tokens_per_image, int tasks, int M, int D, int E, int K, void* dy, float* dsel_row, float* dwg);

// ---- guard words between workspace slices ------------------------------------------------------
// table[i]: byte offset from base of guard i (words 32-bit values each).  guards_write fills them with `word`;
// guards_check raises STATUS_GUARD in *status when any word differs.
void guards_write(cudaStream_t s, char* base, const unsigned long long* table, int n, int words, uint32_t word);
void guards_check(cudaStream_t s, const char* base, const unsigned long long* table, int n, int words, uint32_t word, int* status);

// ---- conversions ------------------------------------------------------------------------------
void convert_from_float(const Ctx& c, const float* src, void* dst, size_t n);   // float -> storage dtype
void convert_to_float(const Ctx& c, const void* src, float* dst, size_t n);     // storage dtype -> float
void fill_float(cudaStream_t s, float* dst, float v, size_t n);
void convert_int_to_float(cudaStream_t s, const int* src, float* dst, size_t n);

}  // namespace bsr
