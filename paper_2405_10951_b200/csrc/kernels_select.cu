// Token importance, per-image top-K and the compaction between MHSA and FFN (paper Section 4.1, Eq. 6).
#include "common.cuh"
#include "kernels.h"

namespace bsr {

// Monotone map float -> uint32 (larger float, larger key).
__device__ __forceinline__ uint32_t ordered_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// One warp per image.  Scores are the head mean of the classification token's attention row, summed in
// head order and divided by H in float.  The K-th largest key is found bit by bit (largest t with
// count(key >= t) >= K); ties at the threshold go to the lower index; both index lists come out ascending.
constexpr int SEL_WARPS = 4;

__global__ void token_select_kernel(const float* __restrict__ p, int B, int H, int M, int k,
                                    float* __restrict__ scores, int* __restrict__ kept, int* __restrict__ dropped) {
  extern __shared__ uint32_t keys_all[];
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int b = blockIdx.x * SEL_WARPS + warp;
  if (b >= B) return;
  uint32_t* keys = keys_all + (size_t)warp * M;
  const float* pb = p + (size_t)b * H * M;
  for (int j = lane; j < M; j += 32) {
    float acc = pb[j];
    for (int h = 1; h < H; ++h) acc = acc + pb[(size_t)h * M + j];
    float s = acc / (float)H;
    scores[(size_t)b * M + j] = s;
    keys[j] = ordered_key(s);
  }
  __syncwarp();
  uint32_t t = 0;
  for (int bit = 31; bit >= 0; --bit) {
    uint32_t cand = t | (1u << bit);
    int cnt = 0;
    for (int j = lane; j < M; j += 32) cnt += (keys[j] >= cand) ? 1 : 0;
    cnt = warp_sum_int(cnt);
    if (cnt >= k) t = cand;
  }
  int gt = 0;
  for (int j = lane; j < M; j += 32) gt += (keys[j] > t) ? 1 : 0;
  gt = warp_sum_int(gt);
  int need_eq = k - gt;                 // how many of the keys equal to t are kept (lowest indices first)
  int n_kept = 0, n_drop = 0, eq_seen = 0;
  uint32_t lt_mask = (1u << lane) - 1u;
  for (int base = 0; base < M; base += 32) {
    int j = base + lane;
    bool valid = j < M;
    uint32_t key = valid ? keys[j] : 0u;
    bool is_eq = valid && key == t;
    uint32_t eq_mask = __ballot_sync(0xffffffffu, is_eq);
    int eq_rank = eq_seen + __popc(eq_mask & lt_mask);
    bool keep = valid && (key > t || (is_eq && eq_rank < need_eq));
    uint32_t keep_mask = __ballot_sync(0xffffffffu, keep);
    uint32_t drop_mask = __ballot_sync(0xffffffffu, valid && !keep);
    if (keep) kept[(size_t)b * k + n_kept + __popc(keep_mask & lt_mask)] = j;
    else if (valid) dropped[(size_t)b * (M - k) + n_drop + __popc(drop_mask & lt_mask)] = j;
    n_kept += __popc(keep_mask);
    n_drop += __popc(drop_mask);
    eq_seen += __popc(eq_mask);
  }
}

// Same selection with the keys of one image held in registers (IPL per lane, M <= 32 * IPL): the 32 threshold
// steps are register compares and one warp reduction each.  Element j lives in lane j % 32, slot j / 32, so a
// slot is a run of 32 consecutive tokens and ballots give positions in token order.
template <int IPL>
__global__ void __launch_bounds__(SEL_WARPS * 32)
token_select_reg_kernel(const float* __restrict__ p, int B, int H, int M, int k, float* __restrict__ scores,
                        int* __restrict__ kept, int* __restrict__ dropped) {
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int b = blockIdx.x * SEL_WARPS + warp;
  if (b >= B) return;
  const float* pb = p + (size_t)b * H * M;
  uint32_t key[IPL];
  float acc[IPL];
  // head sum in head order per token; the IPL loads of one head are independent, so many are in flight
#pragma unroll
  for (int i = 0; i < IPL; ++i) acc[i] = (i * 32 + lane < M) ? pb[i * 32 + lane] : 0.f;
  // heads in groups of four: the loads of a group are all issued before its (ordered) additions
  int h = 1;
  for (; h + 4 <= H; h += 4) {
    float v[4][IPL];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const float* ph = pb + (size_t)(h + u) * M;
#pragma unroll
      for (int i = 0; i < IPL; ++i) v[u][i] = (i * 32 + lane < M) ? ph[i * 32 + lane] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
#pragma unroll
      for (int i = 0; i < IPL; ++i) acc[i] = acc[i] + v[u][i];
    }
  }
  for (; h < H; ++h) {
    const float* ph = pb + (size_t)h * M;
#pragma unroll
    for (int i = 0; i < IPL; ++i)
      if (i * 32 + lane < M) acc[i] = acc[i] + ph[i * 32 + lane];
  }
#pragma unroll
  for (int i = 0; i < IPL; ++i) {
    int j = i * 32 + lane;
    key[i] = 0u;
    if (j < M) {
      float s = acc[i] / (float)H;
      scores[(size_t)b * M + j] = s;
      key[i] = ordered_key(s);
    }
  }
  // keys of absent elements are 0, below every real key (a real key has its top bit set unless the score is negative;
  // scores are probabilities), and they are excluded by index below anyway
  uint32_t t = 0;
  for (int bit = 31; bit >= 0; --bit) {
    uint32_t cand = t | (1u << bit);
    int cnt = 0;
#pragma unroll
    for (int i = 0; i < IPL; ++i) cnt += (i * 32 + lane < M && key[i] >= cand) ? 1 : 0;
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if (cnt >= k) t = cand;
  }
  int gt = 0;
#pragma unroll
  for (int i = 0; i < IPL; ++i) gt += (i * 32 + lane < M && key[i] > t) ? 1 : 0;
  gt = __reduce_add_sync(0xffffffffu, gt);
  int need_eq = k - gt;
  int n_kept = 0, n_drop = 0, eq_seen = 0;
  uint32_t lt_mask = (1u << lane) - 1u;
#pragma unroll
  for (int i = 0; i < IPL; ++i) {
    int j = i * 32 + lane;
    if (i * 32 >= M) break;
    bool valid = j < M;
    bool is_eq = valid && key[i] == t;
    uint32_t eq_mask = __ballot_sync(0xffffffffu, is_eq);
    int eq_rank = eq_seen + __popc(eq_mask & lt_mask);
    bool keep = valid && (key[i] > t || (is_eq && eq_rank < need_eq));
    uint32_t keep_mask = __ballot_sync(0xffffffffu, keep);
    uint32_t drop_mask = __ballot_sync(0xffffffffu, valid && !keep);
    if (keep) kept[(size_t)b * k + n_kept + __popc(keep_mask & lt_mask)] = j;
    else if (valid) dropped[(size_t)b * (M - k) + n_drop + __popc(drop_mask & lt_mask)] = j;
    n_kept += __popc(keep_mask);
    n_drop += __popc(drop_mask);
    eq_seen += __popc(eq_mask);
  }
}

void token_select(cudaStream_t s, const float* p, int B, int H, int M, int k, float* scores, int* kept, int* dropped) {
  note_launch(1);
  int blocks = ceil_div(B, SEL_WARPS), threads = SEL_WARPS * 32;
  if (M <= 256) { token_select_reg_kernel<8><<<blocks, threads, 0, s>>>(p, B, H, M, k, scores, kept, dropped); return; }
  if (M <= 640) { token_select_reg_kernel<20><<<blocks, threads, 0, s>>>(p, B, H, M, k, scores, kept, dropped); return; }
  size_t smem = (size_t)SEL_WARPS * M * sizeof(uint32_t);
  if (smem > 48 * 1024) cudaFuncSetAttribute(token_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  token_select_kernel<<<blocks, threads, smem, s>>>(p, B, H, M, k, scores, kept, dropped);
}

// ------------------------------------------------------------------------------------------------
// Compaction.  grid = (B, copy_splits + fuse_slices), 256 threads.
//   blockIdx.y <  copy_splits : copies the classification row and a share of the kept rows (16-byte vectors);
//   blockIdx.y >= copy_splits : builds a column slice of the fused token, sum over dropped j of s_j * x_j,
//                               row lanes accumulate in float and are combined through shared memory in lane order.
// ------------------------------------------------------------------------------------------------
constexpr int GF_THREADS = 256;
constexpr int GF_SLICE_CHUNKS = 32;     // 16-byte chunks per fused-token column slice
constexpr int GF_ROWLANES = GF_THREADS / GF_SLICE_CHUNKS;

template <typename T>
__global__ void gather_fuse_kernel(const T* __restrict__ x, int M, int D, int k, const int* __restrict__ kept,
                                   const int* __restrict__ dropped, const float* __restrict__ scores, int fuse,
                                   T* __restrict__ out, int copy_splits, int* status) {
  constexpr int N = Pack<T>::N;
  int b = blockIdx.x;
  int chunks = D / N;
  int t_out = 1 + k + (fuse ? 1 : 0);
  const T* xb = x + (size_t)b * (1 + M) * D;
  T* ob = out + (size_t)b * t_out * D;
  if ((int)blockIdx.y < copy_splits) {
    int rows = 1 + k;
    int per = (rows + copy_splits - 1) / copy_splits;
    int r0 = blockIdx.y * per, r1 = min(rows, r0 + per);
    int total = (r1 - r0) * chunks;
    for (int i = threadIdx.x; i < total; i += GF_THREADS) {
      int r = r0 + i / chunks, ch = i % chunks;
      int src = (r == 0) ? 0 : 1 + kept[(size_t)b * k + (r - 1)];
      if (!BSR_CHECK(src >= 0 && src <= M, status)) continue;
      uint4 v = *reinterpret_cast<const uint4*>(xb + (size_t)src * D + ch * N);
      *reinterpret_cast<uint4*>(ob + (size_t)r * D + ch * N) = v;
    }
    return;
  }
  __shared__ float sm[GF_ROWLANES][GF_SLICE_CHUNKS * N];
  __shared__ float weight_sum;
  int slice = blockIdx.y - copy_splits;
  int cs = threadIdx.x % GF_SLICE_CHUNKS, rl = threadIdx.x / GF_SLICE_CHUNKS;
  int ch = slice * GF_SLICE_CHUNKS + cs;
  float acc[N];
#pragma unroll
  for (int j = 0; j < N; ++j) acc[j] = 0.f;
  int nd = M - k;
  if (fuse == 2 && threadIdx.x < 32) {        // weighted mean: the sum of the dropped tokens' weights, in a fixed order
    float ws = 0.f;
    for (int i = threadIdx.x; i < nd; i += 32) ws += scores[(size_t)b * M + dropped[(size_t)b * nd + i]];
    ws = warp_sum(ws);
    if (threadIdx.x == 0) weight_sum = ws;
  }
  if (ch < chunks) {
    for (int i = rl; i < nd; i += GF_ROWLANES) {
      int j = dropped[(size_t)b * nd + i];
      if (!BSR_CHECK(j >= 0 && j < M, status)) continue;
      float w = scores[(size_t)b * M + j];
      float v[N];
      load16(xb + (size_t)(1 + j) * D + ch * N, v);
#pragma unroll
      for (int e = 0; e < N; ++e) acc[e] += w * v[e];
    }
  }
#pragma unroll
  for (int e = 0; e < N; ++e) sm[rl][cs * N + e] = acc[e];
  __syncthreads();
  if (rl == 0 && ch < chunks) {
    float o[N];
#pragma unroll
    for (int e = 0; e < N; ++e) {
      float s = 0.f;
#pragma unroll
      for (int r = 0; r < GF_ROWLANES; ++r) s += sm[r][cs * N + e];
      o[e] = fuse == 2 ? s / weight_sum : s;
    }
    store16(ob + (size_t)(1 + k) * D + ch * N, o);
  }
}

void gather_fuse(const Ctx& c, const void* x, int B, int M, int D, int k, const int* kept, const int* dropped,
                 const float* scores, int fuse, void* out) {
  note_launch(1);
  int n = (c.dtype == 0) ? 4 : 8;
  int chunks = D / n;
  int do_fuse = ((fuse == 1 || fuse == 2) && k < M) ? fuse : 0;          // 1: weighted sum, 2: weighted mean
  int fuse_slices = do_fuse ? ceil_div(chunks, GF_SLICE_CHUNKS) : 0;
  int sms = c.sm_count > 0 ? c.sm_count : 148;
  int copy_splits = ceil_div(4L * sms, B);            // about four blocks per SM in total
  if (copy_splits < 1) copy_splits = 1;
  if (copy_splits > 1 + k) copy_splits = 1 + k;
  dim3 grid(B, copy_splits + fuse_slices);
  if (c.dtype == 0)
    gather_fuse_kernel<float><<<grid, GF_THREADS, 0, c.stream>>>((const float*)x, M, D, k, kept, dropped, scores, do_fuse, (float*)out, copy_splits, c.status);
  else
    gather_fuse_kernel<bf16><<<grid, GF_THREADS, 0, c.stream>>>((const bf16*)x, M, D, k, kept, dropped, scores, do_fuse, (bf16*)out, copy_splits, c.status);
}

// Backward of the compaction, one warp per input row (the index sets are constants, the fusion weights are
// differentiated):  dx_0 = g_0;  dx_{kept_i} = g_{1+i};  dx_j = s_j g_f and e_j = <g_f, x_j> for dropped j.
// Weighted mean (fuse == 2, f = sum_j s_j x_j / S, S = sum_j s_j): dx_j = (s_j / S) g_f, e_j = (<g_f, x_j> - <g_f, f>) / S
// with f read from the forward pass's compacted tensor `fwd_out`.
// Rows are float (residual stream); dx_copy optionally receives the same rows in bf16.
__global__ void gather_fuse_bwd_kernel(const float* __restrict__ dout, const float* __restrict__ x, int B, int M, int D, int k,
                                       const int* __restrict__ kept, const int* __restrict__ dropped,
                                       const float* __restrict__ scores, int fuse, float* __restrict__ dx,
                                       bf16* __restrict__ dx_copy, float* __restrict__ escore, const float* __restrict__ fwd_out,
                                       int* status) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= B * (1 + M)) return;
  int b = warp / (1 + M), e = warp % (1 + M);
  int chunks = D / 4;
  int t_out = 1 + k + (fuse ? 1 : 0);
  const float* gb = dout + (size_t)b * t_out * D;
  size_t ob = (size_t)b * (1 + M) * D;
  if (e <= k) {                         // classification row or a kept row: plain copy
    int dst = (e == 0) ? 0 : 1 + kept[(size_t)b * k + (e - 1)];
    if (!BSR_CHECK(dst >= 0 && dst <= M, status)) return;
    for (int ch = lane; ch < chunks; ch += 32) {
      float v[4];
      load16(gb + (size_t)e * D + ch * 4, v);
      store16(dx + ob + (size_t)dst * D + ch * 4, v);
      if (dx_copy != nullptr) store4(dx_copy + ob + (size_t)dst * D + ch * 4, v);
    }
    if (e > 0 && lane == 0) escore[(size_t)b * M + (dst - 1)] = 0.f;
    return;
  }
  int j = dropped[(size_t)b * (M - k) + (e - 1 - k)];
  if (!BSR_CHECK(j >= 0 && j < M, status)) return;
  float w = fuse ? scores[(size_t)b * M + j] : 0.f;
  const float* gf = gb + (size_t)(1 + k) * D;
  const float* xr = x + ob + (size_t)(1 + j) * D;
  float inv_sum = 1.f, dot_f = 0.f;
  if (fuse == 2) {
    int nd = M - k;
    float ws = 0.f;
    for (int i = lane; i < nd; i += 32) ws += scores[(size_t)b * M + dropped[(size_t)b * nd + i]];
    inv_sum = 1.0f / warp_sum(ws);
    const float* fr = fwd_out + ((size_t)b * t_out + 1 + k) * D;
    for (int ch = lane; ch < chunks; ch += 32) {
      float g[4], fv[4];
      load16(gf + ch * 4, g);
      load16(fr + ch * 4, fv);
#pragma unroll
      for (int i = 0; i < 4; ++i) dot_f += g[i] * fv[i];
    }
    dot_f = warp_sum(dot_f);
    w *= inv_sum;
  }
  float dot = 0.f;
  for (int ch = lane; ch < chunks; ch += 32) {
    float g[4], o[4];
    if (fuse) {
      float xv[4];
      load16(gf + ch * 4, g);
      load16(xr + ch * 4, xv);
#pragma unroll
      for (int i = 0; i < 4; ++i) { dot += g[i] * xv[i]; o[i] = w * g[i]; }
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) o[i] = 0.f;
    }
    store16(dx + ob + (size_t)(1 + j) * D + ch * 4, o);
    if (dx_copy != nullptr) store4(dx_copy + ob + (size_t)(1 + j) * D + ch * 4, o);
  }
  dot = warp_sum(dot);
  if (lane == 0) escore[(size_t)b * M + j] = fuse == 2 ? (dot - dot_f) * inv_sum : dot;
}

void gather_fuse_bwd(const Ctx& c, const void* dout, const void* x, int B, int M, int D, int k, const int* kept,
                     const int* dropped, const float* scores, int fuse, void* dx, void* dx_copy, float* escore, const void* fwd_out) {
  note_launch(1);
  int do_fuse = ((fuse == 1 || fuse == 2) && k < M) ? fuse : 0;
  int threads = 256, blocks = ceil_div((long)B * (1 + M) * 32, threads);
  gather_fuse_bwd_kernel<<<blocks, threads, 0, c.stream>>>((const float*)dout, (const float*)x, B, M, D, k, kept, dropped, scores,
                                                           do_fuse, (float*)dx, (bf16*)dx_copy, escore, (const float*)fwd_out, c.status);
}

}  // namespace bsr
