// Mixture-of-experts FFN (paper Section 5.2): a task-dependent router picks the top-k of E expert MLPs per
// token and adds their outputs, weighted by a softmax over the selected gate logits.  These are the routing,
// grouping and combination kernels; the expert MLPs themselves run as expert-grouped tcgen05 GEMMs.
//
// Grouping.  Every (token, slot) pair becomes one row of an expert-ordered buffer: expert e owns rows
// seg_start[e] .. seg_start[e] + count[e], padded with empty rows to a multiple of 128 so that a GEMM tile never
// mixes experts.  Within an expert rows keep token order, and every reduction runs in row order: results do not
// depend on scheduling.
#include "common.cuh"
#include "kernels.h"

namespace bsr {

constexpr int MOE_BLOCK_TOKENS = 128;
constexpr int MOE_MAX_E = 32;
constexpr int MOE_MAX_K = 4;

// ---- routing: gate logits, top-k (ties -> lower expert id), softmax over the selected logits -------------------
constexpr int MOE_ROUTE_WARPS = 8;
constexpr int MOE_ROUTE_TOKENS = 16;
static_assert(MOE_BLOCK_TOKENS % MOE_ROUTE_TOKENS == 0, "a routing block must not straddle two counting groups");
template <typename T>
__global__ void __launch_bounds__(MOE_ROUTE_WARPS * 32)
moe_route_kernel(const T* __restrict__ y, const T* __restrict__ wg, const float* __restrict__ logits, int logit_stride,
                 const int* __restrict__ task_ids, int tokens_per_image, int M, int D, int E, int K, int gate_elems_in_smem,
                 int* __restrict__ eidx, float* __restrict__ ew, int* __restrict__ blk_counts) {
  // A block takes MOE_ROUTE_TOKENS consecutive tokens (a divisor of MOE_BLOCK_TOKENS, so all of them fall into one
  // counting group), a warp one token at a time.  Expert by expert the lanes multiply 16-byte pieces of the token's row
  // of y (coalesced; from L1 after the first expert) with the same pieces of the gate row -- the gate matrices of all
  // tasks are staged in shared memory when they are small -- and the partial dot products are summed over the lanes
  // in a fixed (butterfly) order; lane e keeps logit e.  The top k then come from k warp-wide maxima (among equal
  // logits the lowest expert id, found with a ballot).  Few registers, so many tokens are in flight per SM: the work
  // per token is a chain of dependent loads.  The per-group expert counts (zeroed before the launch) are integer sums.
  // When `logits` is given (row stride logit_stride, the E logits of task t at column t E), the products were formed
  // by a GEMM over all tasks' gates beforehand and lane e just reads its logit.
  extern __shared__ __align__(16) unsigned char route_smem[];
  __shared__ int counts[MOE_MAX_E];
  constexpr int N = Pack<T>::N;
  if (threadIdx.x < MOE_MAX_E) counts[threadIdx.x] = 0;
  const T* gates = wg;
  if (logits == nullptr && gate_elems_in_smem > 0) {
    T* sg = reinterpret_cast<T*>(route_smem);
    for (int i = threadIdx.x * N; i < gate_elems_in_smem; i += blockDim.x * N)
      *reinterpret_cast<uint4*>(sg + i) = *reinterpret_cast<const uint4*>(wg + i);
    gates = sg;
  }
  __syncthreads();
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int chunks = D / N;
  const uint32_t all = (E >= 32) ? 0xffffffffu : ((1u << E) - 1u);
  for (int t = warp; t < MOE_ROUTE_TOKENS; t += MOE_ROUTE_WARPS) {
    int tok = blockIdx.x * MOE_ROUTE_TOKENS + t;
    if (tok >= M) break;
    int task = task_ids ? task_ids[tok / tokens_per_image] : 0;
    const T* yr = y + (size_t)tok * D;
    const T* gt = gates + (size_t)task * E * D;
    float logit = -INFINITY;                      // lane e: logit of expert e
    if (logits != nullptr) {
      if (lane < E) logit = logits[(size_t)tok * logit_stride + task * E + lane];
    } else
#pragma unroll 4
    for (int e = 0; e < E; ++e) {
      float acc = 0.f;
      for (int ch = lane; ch < chunks; ch += 32) {
        float yv[N], wv[N];
        load16(yr + ch * N, yv);
        load16(gt + (size_t)e * D + ch * N, wv);
#pragma unroll
        for (int j = 0; j < N; ++j) acc = fmaf(yv[j], wv[j], acc);
      }
      acc = warp_sum(acc);
      if (lane == e) logit = acc;
    }
    float sel[MOE_MAX_K];
    int sid[MOE_MAX_K];
    uint32_t taken = 0;
#pragma unroll
    for (int i = 0; i < MOE_MAX_K; ++i) {
      if (i < K) {
        bool open = lane < E && !((taken >> lane) & 1u);
        float best = warp_max(open ? logit : -INFINITY);
        uint32_t at = __ballot_sync(0xffffffffu, open && logit == best);
        if (at == 0) at = all & ~taken;             // nothing compares equal (a NaN among the logits): lowest open id
        int bi = __ffs(at) - 1;                     // the lowest id wins among equals
        sel[i] = __shfl_sync(0xffffffffu, logit, bi);
        sid[i] = bi;
        taken |= 1u << bi;
      }
    }
    if (lane == 0) {
      float den = 0.f;
#pragma unroll
      for (int i = 0; i < MOE_MAX_K; ++i)
        if (i < K) den += expf(sel[i] - sel[0]);
#pragma unroll
      for (int i = 0; i < MOE_MAX_K; ++i) {
        if (i < K) {
          eidx[(size_t)tok * K + i] = sid[i];
          ew[(size_t)tok * K + i] = expf(sel[i] - sel[0]) / den;
          atomicAdd(&counts[sid[i]], 1);            // integer counts: order-independent
        }
      }
    }
  }
  __syncthreads();
  if (threadIdx.x < E && counts[threadIdx.x] != 0)
    atomicAdd(&blk_counts[(size_t)(blockIdx.x * MOE_ROUTE_TOKENS / MOE_BLOCK_TOKENS) * E + threadIdx.x], counts[threadIdx.x]);
}

// ---- segment table and row assignment in one kernel ---------------------------------------------------------------
// A block per group of MOE_BLOCK_TOKENS tokens.  Every block sums the per-group expert counts itself (a few KB): the
// totals give the start of every expert's segment (padded to 128 rows), the counts of the groups before its own give
// its place inside each segment.  Then the position of every (token, slot) inside its expert's segment, in token order.
// Block 0 also publishes the segment starts and the expert of every 128-row tile for the grouped GEMMs.
__global__ void __launch_bounds__(256)
moe_assign_kernel(const int* __restrict__ eidx, const float* __restrict__ ew, const int* __restrict__ blk_counts, int nblk,
                  int tiles_cap, int M, int E, int K, int* __restrict__ seg_start, int* __restrict__ tile_expert,
                  int* __restrict__ pos, int* __restrict__ row_token, float* __restrict__ row_w) {
  __shared__ int total[MOE_MAX_E];
  __shared__ int before[MOE_MAX_E];
  __shared__ int start[MOE_MAX_E + 1];
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int e = warp; e < E; e += 8) {
    int all = 0, pre = 0;
    for (int g = lane; g < nblk; g += 32) {
      int cnt = blk_counts[(size_t)g * E + e];
      all += cnt;
      if (g < (int)blockIdx.x) pre += cnt;
    }
    all = warp_sum_int(all);
    pre = warp_sum_int(pre);
    if (lane == 0) { total[e] = all; before[e] = pre; }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int s = 0;
    for (int i = 0; i < E; ++i) {
      start[i] = s;
      s += (total[i] + 127) & ~127;
    }
    start[E] = s;
  }
  __syncthreads();
  if (blockIdx.x == 0) {
    for (int i = threadIdx.x; i <= E; i += blockDim.x) seg_start[i] = start[i];
    for (int t = threadIdx.x; t < tiles_cap; t += blockDim.x) {
      int row = t * 128, ex = -1;
      for (int i = 0; i < E; ++i)
        if (row >= start[i] && row < start[i + 1]) ex = i;
      tile_expert[t] = ex;
    }
  }
  int t0 = blockIdx.x * MOE_BLOCK_TOKENS;
  int n_entries = min(MOE_BLOCK_TOKENS, M - t0) * K;
  uint32_t lt = (1u << lane) - 1u;
  for (int e = warp; e < E; e += 8) {
    int base = start[e] + before[e];
    int run = 0;
    for (int i0 = 0; i0 < n_entries; i0 += 32) {
      int i = i0 + lane;
      bool hit = i < n_entries && eidx[(size_t)t0 * K + i] == e;
      uint32_t m = __ballot_sync(0xffffffffu, hit);
      if (hit) {
        int r = base + run + __popc(m & lt);
        pos[(size_t)t0 * K + i] = r;
        row_token[r] = t0 + i / K;
        row_w[r] = ew[(size_t)t0 * K + i];
      }
      run += __popc(m);
    }
  }
}

// ---- gather the expert inputs: xg[r] = y[row_token[r]], empty rows are zero ---------------------------------------
template <typename T>
__global__ void moe_gather_kernel(const T* __restrict__ y, const int* __restrict__ row_token, const int* __restrict__ seg_start,
                                  int E, int D, T* __restrict__ xg, int rows_cap, int M, int* status) {
  constexpr int N = Pack<T>::N;
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= rows_cap || warp >= seg_start[E]) return;
  int tok = row_token[warp];
  if (!BSR_CHECK(tok < M, status)) return;
  for (int ch = lane; ch < D / N; ch += 32) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (tok >= 0) v = *reinterpret_cast<const uint4*>(y + (size_t)tok * D + ch * N);
    *reinterpret_cast<uint4*>(xg + (size_t)warp * D + ch * N) = v;
  }
}

// ---- combine: out[t] = res[t] + sum_slot w_slot * og[pos(t, slot)]  (float residual stream) ------------------------
__global__ void moe_combine_kernel(const float* __restrict__ og, const int* __restrict__ pos, const float* __restrict__ ew,
                                   const float* __restrict__ res, float* __restrict__ out, int M, int D, int K) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= M) return;
  for (int ch = lane; ch < D / 4; ch += 32) {
    float acc[4];
    load16(res + (size_t)warp * D + ch * 4, acc);
    for (int s = 0; s < K; ++s) {
      float w = ew[(size_t)warp * K + s];
      float v[4];
      load16(og + (size_t)pos[(size_t)warp * K + s] * D + ch * 4, v);
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[j] = fmaf(w, v[j], acc[j]);
    }
    store16(out + (size_t)warp * D + ch * 4, acc);
  }
}

// ---- backward of the combination: dog[r] = w_r * dout[token_r]; dw[r] = <dout[token_r], og[r]> ------------------
template <typename T>
__global__ void moe_combine_bwd_kernel(const float* __restrict__ dout, const float* __restrict__ og, const int* __restrict__ row_token,
                                       const float* __restrict__ row_w, const int* __restrict__ seg_start, int E, int D,
                                       T* __restrict__ dog, float* __restrict__ dw, int rows_cap) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= rows_cap || warp >= seg_start[E]) return;
  int tok = row_token[warp];
  float w = tok >= 0 ? row_w[warp] : 0.f;
  float dot = 0.f;
  for (int ch = lane; ch < D / 4; ch += 32) {
    float g[4] = {0.f, 0.f, 0.f, 0.f}, o[4], r[4];
    if (tok >= 0) {
      load16(dout + (size_t)tok * D + ch * 4, g);
      load16(og + (size_t)warp * D + ch * 4, o);
#pragma unroll
      for (int j = 0; j < 4; ++j) dot = fmaf(g[j], o[j], dot);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) r[j] = w * g[j];
    store4(dog + (size_t)warp * D + ch * 4, r);
  }
  dot = warp_sum(dot);
  if (lane == 0) dw[warp] = dot;
}

// ---- per-expert column sums (bias gradients): out[e][col] = sum over the expert's rows of x[r][col] -----------------
template <typename T>
__global__ void __launch_bounds__(256)
moe_seg_colsum_kernel(const T* __restrict__ x, const int* __restrict__ seg_start, int cols, float* __restrict__ out) {
  constexpr int N = Pack<T>::N;
  __shared__ float sm[8][32 * N];
  int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  int e = blockIdx.y;
  int col0 = (blockIdx.x * 32 + tx) * N;
  float acc[N];
#pragma unroll
  for (int j = 0; j < N; ++j) acc[j] = 0.f;
  if (col0 < cols) {
    for (int r = seg_start[e] + ty; r < seg_start[e + 1]; r += 8) {
      float v[N];
      load16(x + (size_t)r * cols + col0, v);
#pragma unroll
      for (int j = 0; j < N; ++j) acc[j] += v[j];
    }
  }
#pragma unroll
  for (int j = 0; j < N; ++j) sm[ty][tx * N + j] = acc[j];
  __syncthreads();
  for (int c = threadIdx.x; c < 32 * N; c += blockDim.x) {
    int col = blockIdx.x * 32 * N + c;
    if (col < cols) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) s += sm[w][c];
      out[(size_t)e * cols + col] = s;
    }
  }
}

// ---- gate backward, token side: d(selected logits) and the gradient of the layer input -----------------------------
//   dsel_s = w_s (dw_s - sum_u w_u dw_u);  dy[t] = sum_s dxg[pos_s] + sum_s dsel_s Wg[task][e_s]
template <typename T>
__global__ void moe_gate_bwd_kernel(const T* __restrict__ dxg, const float* __restrict__ dw, const int* __restrict__ pos,
                                    const int* __restrict__ eidx, const float* __restrict__ ew, const T* __restrict__ wg,
                                    const int* __restrict__ task_ids, int tokens_per_image, int M, int D, int E, int K,
                                    T* __restrict__ dy, float* __restrict__ dsel_row) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= M) return;
  int task = task_ids ? task_ids[warp / tokens_per_image] : 0;
  float w[MOE_MAX_K], d[MOE_MAX_K];
  int p[MOE_MAX_K], ex[MOE_MAX_K];
  float mean = 0.f;
  for (int s = 0; s < K; ++s) {
    p[s] = pos[(size_t)warp * K + s];
    ex[s] = eidx[(size_t)warp * K + s];
    w[s] = ew[(size_t)warp * K + s];
    d[s] = dw[p[s]];
    mean = fmaf(w[s], d[s], mean);
  }
  for (int s = 0; s < K; ++s) {
    d[s] = w[s] * (d[s] - mean);
    if (lane == 0) dsel_row[p[s]] = d[s];
  }
  for (int ch = lane; ch < D / 4; ch += 32) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int s = 0; s < K; ++s) {
      float v[4], g[4];
      load4(dxg + (size_t)p[s] * D + ch * 4, v);
      load4(wg + ((size_t)task * E + ex[s]) * D + ch * 4, g);
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[j] += v[j] + d[s] * g[j];
    }
    store4(dy + (size_t)warp * D + ch * 4, acc);
  }
}

// ---- gate backward, weight side: dWg[task][e] = sum over expert e's rows of that task of dsel[r] * xg[r] --------------
template <typename T>
__global__ void __launch_bounds__(256)
moe_gate_wgrad_kernel(const T* __restrict__ xg, const float* __restrict__ dsel_row, const int* __restrict__ row_token,
                      const int* __restrict__ seg_start, const int* __restrict__ task_ids, int tokens_per_image, int D, int E,
                      float* __restrict__ dwg) {
  constexpr int N = Pack<T>::N;
  __shared__ float sm[8][32 * N];
  int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  int e = blockIdx.y, task = blockIdx.z;
  int col0 = (blockIdx.x * 32 + tx) * N;
  float acc[N];
#pragma unroll
  for (int j = 0; j < N; ++j) acc[j] = 0.f;
  if (col0 < D) {
    for (int r = seg_start[e] + ty; r < seg_start[e + 1]; r += 8) {
      int tok = row_token[r];
      if (tok < 0) continue;
      int tk = task_ids ? task_ids[tok / tokens_per_image] : 0;
      if (tk != task) continue;
      float c = dsel_row[r];
      float v[N];
      load16(xg + (size_t)r * D + col0, v);
#pragma unroll
      for (int j = 0; j < N; ++j) acc[j] = fmaf(c, v[j], acc[j]);
    }
  }
#pragma unroll
  for (int j = 0; j < N; ++j) sm[ty][tx * N + j] = acc[j];
  __syncthreads();
  for (int c = threadIdx.x; c < 32 * N; c += blockDim.x) {
    int col = blockIdx.x * 32 * N + c;
    if (col < D) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) s += sm[w][c];
      dwg[((size_t)task * E + e) * D + col] = s;
    }
  }
}

// =================================================================================================
// launchers
// =================================================================================================
int moe_rows_cap(int M, int E, int K) { return ((M * K + E * 127) + 127) & ~127; }
int moe_blocks(int M) { return ceil_div(M, MOE_BLOCK_TOKENS); }

void moe_route(const Ctx& c, const MoeBufs& b, const void* y, const void* wg, const int* task_ids, int tokens_per_image, int M,
               int D, int E, int K, int num_tasks, const float* logits, int logit_stride) {
  int nblk = moe_blocks(M);
  int rows_cap = moe_rows_cap(M, E, K);
  note_launch(3);
  size_t es = c.dtype == 0 ? 4 : 2;
  size_t gate_elems = (size_t)(num_tasks < 1 ? 1 : num_tasks) * E * D;
  size_t smem = gate_elems * es;
  if (smem > 16 * 1024 || logits != nullptr) { smem = 0; gate_elems = 0; }       // not worth staging for 16 tokens: the gates are read through L1 instead
  static SmemLimit lim[2];
  int rblk = ceil_div(M, MOE_ROUTE_TOKENS);
  cudaMemsetAsync(b.blk_counts, 0, (size_t)nblk * E * sizeof(int), c.stream);
  if (c.dtype == 0) {
    ensure_smem(lim[0], moe_route_kernel<float>, smem);
    moe_route_kernel<float><<<rblk, MOE_ROUTE_WARPS * 32, smem, c.stream>>>((const float*)y, (const float*)wg, logits, logit_stride, task_ids, tokens_per_image, M, D, E, K,
                                                                        (int)gate_elems, b.eidx, b.ew, b.blk_counts);
  } else {
    ensure_smem(lim[1], moe_route_kernel<bf16>, smem);
    moe_route_kernel<bf16><<<rblk, MOE_ROUTE_WARPS * 32, smem, c.stream>>>((const bf16*)y, (const bf16*)wg, logits, logit_stride, task_ids, tokens_per_image, M, D, E, K,
                                                                       (int)gate_elems, b.eidx, b.ew, b.blk_counts);
  }
  cudaMemsetAsync(b.row_token, 0xFF, (size_t)rows_cap * sizeof(int), c.stream);
  moe_assign_kernel<<<nblk, 256, 0, c.stream>>>(b.eidx, b.ew, b.blk_counts, nblk, rows_cap / 128, M, E, K, b.seg_start, b.tile_expert,
                                                b.pos, b.row_token, b.row_w);
  int blocks = ceil_div((long)rows_cap * 32, 256);
  if (c.dtype == 0) moe_gather_kernel<float><<<blocks, 256, 0, c.stream>>>((const float*)y, b.row_token, b.seg_start, E, D, (float*)b.xg, rows_cap, M, c.status);
  else moe_gather_kernel<bf16><<<blocks, 256, 0, c.stream>>>((const bf16*)y, b.row_token, b.seg_start, E, D, (bf16*)b.xg, rows_cap, M, c.status);
}

void moe_combine(const Ctx& c, const MoeBufs& b, const float* res, float* out, int M, int D, int K) {
  note_launch(1);
  int blocks = ceil_div((long)M * 32, 256);
  moe_combine_kernel<<<blocks, 256, 0, c.stream>>>(b.og, b.pos, b.ew, res, out, M, D, K);
}

void moe_combine_bwd(const Ctx& c, const MoeBufs& b, const float* dout, void* dog, float* dw, int M, int D, int E, int K) {
  note_launch(1);
  int rows_cap = moe_rows_cap(M, E, K);
  int blocks = ceil_div((long)rows_cap * 32, 256);
  if (c.dtype == 0)
    moe_combine_bwd_kernel<float><<<blocks, 256, 0, c.stream>>>(dout, b.og, b.row_token, b.row_w, b.seg_start, E, D, (float*)dog, dw, rows_cap);
  else
    moe_combine_bwd_kernel<bf16><<<blocks, 256, 0, c.stream>>>(dout, b.og, b.row_token, b.row_w, b.seg_start, E, D, (bf16*)dog, dw, rows_cap);
}

void moe_seg_colsum(const Ctx& c, const MoeBufs& b, const void* x, int cols, int E, float* out) {
  note_launch(1);
  if (c.dtype == 0) moe_seg_colsum_kernel<float><<<dim3(ceil_div(cols, 128), E), 256, 0, c.stream>>>((const float*)x, b.seg_start, cols, out);
  else moe_seg_colsum_kernel<bf16><<<dim3(ceil_div(cols, 256), E), 256, 0, c.stream>>>((const bf16*)x, b.seg_start, cols, out);
}

void moe_gate_bwd(const Ctx& c, const MoeBufs& b, const void* dxg, const float* dw, const void* wg, const int* task_ids,
                  int tokens_per_image, int tasks, int M, int D, int E, int K, void* dy, float* dsel_row, float* dwg) {
  note_launch(2);
  int blocks = ceil_div((long)M * 32, 256);
  if (c.dtype == 0) {
    moe_gate_bwd_kernel<float><<<blocks, 256, 0, c.stream>>>((const float*)dxg, dw, b.pos, b.eidx, b.ew, (const float*)wg, task_ids, tokens_per_image, M, D, E, K, (float*)dy, dsel_row);
    if (dwg != nullptr) moe_gate_wgrad_kernel<float><<<dim3(ceil_div(D, 128), E, tasks), 256, 0, c.stream>>>((const float*)b.xg, dsel_row, b.row_token, b.seg_start, task_ids, tokens_per_image, D, E, dwg);
  } else {
    moe_gate_bwd_kernel<bf16><<<blocks, 256, 0, c.stream>>>((const bf16*)dxg, dw, b.pos, b.eidx, b.ew, (const bf16*)wg, task_ids, tokens_per_image, M, D, E, K, (bf16*)dy, dsel_row);
    if (dwg != nullptr) moe_gate_wgrad_kernel<bf16><<<dim3(ceil_div(D, 256), E, tasks), 256, 0, c.stream>>>((const bf16*)b.xg, dsel_row, b.row_token, b.seg_start, task_ids, tokens_per_image, D, E, dwg);
  }
}

}  // namespace bsr
