// Multi-head self-attention (paper Eq. 1) forward and backward in FP32 arithmetic, one warp per
// query (or key) row with the head's K/V (or Q/dO) resident in shared memory.  Used by the fp32
// configuration, and by bf16 problems until the tensor-core attention takes them.
//
// Layout: qkv [B, T, 3, H, d], out/dout [B, T, H*d], lse/delta [B, H, T], cls_prob [B, H, T-1].
// The forward kernel also emits the classification token's attention row (Eq. 6: the token
// importance scores), and the backward kernels accept a gradient arriving at that row.
#include "common.cuh"
#include "kernels.h"

namespace bsr {

constexpr int AT_WARPS = 8;
constexpr int AT_MAXD = 64;

template <typename T> struct Row;
template <> struct Row<float> {
  __device__ static int stride(int d) { return d + 1; }
  __device__ static float dot(const float* q, const float* row, int d) {
    float s = 0.f;
    for (int i = 0; i < d; ++i) s = fmaf(q[i], row[i], s);
    return s;
  }
  // the two feature indices a lane owns
  __device__ static int dim0(int lane) { return lane; }
  __device__ static int dim1(int lane) { return lane + 32; }
  __device__ static void pair(const float* row, int lane, int d, float& a, float& b) {
    a = (lane < d) ? row[lane] : 0.f;
    b = (lane + 32 < d) ? row[lane + 32] : 0.f;
  }
  __device__ static void fill(float* row, const float* src, int d, int lane) {
    for (int i = lane; i < d; i += 32) row[i] = src[i];
  }
};
template <> struct Row<bf16> {
  __device__ static int stride(int d) { return d + 2; }
  __device__ static float dot(const float* q, const bf16* row, int d) {
    const __nv_bfloat162* r2 = reinterpret_cast<const __nv_bfloat162*>(row);
    float s = 0.f;
    for (int i = 0; i < d / 2; ++i) {
      float2 v = __bfloat1622float2(r2[i]);
      s = fmaf(q[2 * i], v.x, s);
      s = fmaf(q[2 * i + 1], v.y, s);
    }
    return s;
  }
  __device__ static int dim0(int lane) { return 2 * lane; }
  __device__ static int dim1(int lane) { return 2 * lane + 1; }
  __device__ static void pair(const bf16* row, int lane, int d, float& a, float& b) {
    if (2 * lane < d) {
      float2 v = __bfloat1622float2(reinterpret_cast<const __nv_bfloat162*>(row)[lane]);
      a = v.x; b = v.y;
    } else { a = 0.f; b = 0.f; }
  }
  __device__ static void fill(bf16* row, const bf16* src, int d, int lane) {
    for (int i = lane; i < d / 2; i += 32)
      reinterpret_cast<__nv_bfloat162*>(row)[i] = reinterpret_cast<const __nv_bfloat162*>(src)[i];
  }
};

// Copies [T, d] rows of one (image, head, which) slice of qkv (or of a [B, T, H*d] tensor) into padded smem rows.
template <typename T>
__device__ void stage_rows(T* dst, const T* src, long src_row_stride, int T_, int d) {
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  int rs = Row<T>::stride(d);
  for (int t = warp; t < T_; t += nw) Row<T>::fill(dst + (size_t)t * rs, src + (size_t)t * src_row_stride, d, lane);
}

// ---------------------------------------------------------------------------------------------
// forward
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(AT_WARPS * 32)
attn_fwd_kernel(const T* __restrict__ qkv, T* __restrict__ out, float* __restrict__ lse, float* __restrict__ cls_prob,
                int B, int T_, int H, int d, int qsplit) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  int rs = Row<T>::stride(d);
  T* Ks = reinterpret_cast<T*>(smem_raw);
  T* Vs = Ks + (size_t)T_ * rs;
  float* Ps = reinterpret_cast<float*>(Vs + (size_t)T_ * rs);     // [AT_WARPS][T_]
  float* Qs = Ps + (size_t)AT_WARPS * T_;                          // [AT_WARPS][AT_MAXD]
  int bh = blockIdx.x, b = bh / H, h = bh % H;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  long tok_stride = 3L * H * d;
  const T* base = qkv + (size_t)b * T_ * tok_stride + (size_t)h * d;
  stage_rows<T>(Ks, base + (size_t)H * d, tok_stride, T_, d);
  stage_rows<T>(Vs, base + 2 * (size_t)H * d, tok_stride, T_, d);
  __syncthreads();
  float scale = rsqrtf((float)d);
  float* P = Ps + (size_t)warp * T_;
  float* q = Qs + warp * AT_MAXD;
  for (int i = blockIdx.y * AT_WARPS + warp; i < T_; i += qsplit * AT_WARPS) {
    const T* qrow = base + (size_t)i * tok_stride;
    for (int dd = lane; dd < d; dd += 32) q[dd] = to_f(qrow[dd]) * scale;
    __syncwarp();
    float mx = -INFINITY;
    for (int j = lane; j < T_; j += 32) {
      float s = Row<T>::dot(q, Ks + (size_t)j * rs, d);
      P[j] = s;
      mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    float sum = 0.f;
    for (int j = lane; j < T_; j += 32) {
      float e = expf(P[j] - mx);
      P[j] = e;
      sum += e;
    }
    sum = warp_sum(sum);
    float inv = 1.0f / sum;
    __syncwarp();
    float o0 = 0.f, o1 = 0.f;
    for (int j = 0; j < T_; ++j) {
      float a, c2;
      Row<T>::pair(Vs + (size_t)j * rs, lane, d, a, c2);
      float pj = P[j];
      o0 = fmaf(pj, a, o0);
      o1 = fmaf(pj, c2, o1);
    }
    T* orow = out + ((size_t)b * T_ + i) * H * d + (size_t)h * d;
    int d0 = Row<T>::dim0(lane), d1 = Row<T>::dim1(lane);
    if (d0 < d) orow[d0] = from_f<T>(o0 * inv);
    if (d1 < d) orow[d1] = from_f<T>(o1 * inv);
    if (lse != nullptr && lane == 0) lse[((size_t)b * H + h) * T_ + i] = mx + logf(sum);
    if (i == 0 && cls_prob != nullptr) {
      float* cp = cls_prob + ((size_t)b * H + h) * (T_ - 1);
      for (int j = 1 + lane; j < T_; j += 32) cp[j - 1] = P[j] * inv;
    }
    __syncwarp();
  }
}

// ---------------------------------------------------------------------------------------------
// backward, part 1: one warp per query row -> delta_i and dQ_i
//   P_ij = exp(s_ij - lse_i); dP_ij = dO_i . V_j (+ extra_j / H on the classification row);
//   delta_i = sum_j P_ij dP_ij; dS_ij = P_ij (dP_ij - delta_i); dQ_i = scale * sum_j dS_ij K_j
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(AT_WARPS * 32)
attn_bwd_dq_kernel(const T* __restrict__ qkv, const T* __restrict__ dout, const float* __restrict__ lse,
                   float* __restrict__ delta, const float* __restrict__ cls_extra, T* __restrict__ dqkv,
                   int B, int T_, int H, int d, int qsplit) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  int rs = Row<T>::stride(d);
  T* Ks = reinterpret_cast<T*>(smem_raw);
  T* Vs = Ks + (size_t)T_ * rs;
  float* Ps = reinterpret_cast<float*>(Vs + (size_t)T_ * rs);
  float* Qs = Ps + (size_t)AT_WARPS * T_;                          // [AT_WARPS][2][AT_MAXD]: q and dO
  int bh = blockIdx.x, b = bh / H, h = bh % H;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  long tok_stride = 3L * H * d;
  const T* base = qkv + (size_t)b * T_ * tok_stride + (size_t)h * d;
  stage_rows<T>(Ks, base + (size_t)H * d, tok_stride, T_, d);
  stage_rows<T>(Vs, base + 2 * (size_t)H * d, tok_stride, T_, d);
  __syncthreads();
  float scale = rsqrtf((float)d);
  float invH = 1.0f / (float)H;
  float* P = Ps + (size_t)warp * T_;
  float* q = Qs + warp * 2 * AT_MAXD;
  float* g = q + AT_MAXD;
  for (int i = blockIdx.y * AT_WARPS + warp; i < T_; i += qsplit * AT_WARPS) {
    const T* qrow = base + (size_t)i * tok_stride;
    const T* grow = dout + ((size_t)b * T_ + i) * H * d + (size_t)h * d;
    for (int dd = lane; dd < d; dd += 32) { q[dd] = to_f(qrow[dd]) * scale; g[dd] = to_f(grow[dd]); }
    __syncwarp();
    float l = lse[((size_t)b * H + h) * T_ + i];
    float dl = 0.f;
    for (int j = lane; j < T_; j += 32) {
      float p = expf(Row<T>::dot(q, Ks + (size_t)j * rs, d) - l);
      float dp = Row<T>::dot(g, Vs + (size_t)j * rs, d);
      if (cls_extra != nullptr && i == 0 && j > 0) dp += cls_extra[(size_t)b * (T_ - 1) + (j - 1)] * invH;
      dl += p * dp;
      P[j] = p;
      // dS needs delta: keep dP in the upper half of the pass by recomputing below
    }
    dl = warp_sum(dl);
    for (int j = lane; j < T_; j += 32) {
      float dp = Row<T>::dot(g, Vs + (size_t)j * rs, d);
      if (cls_extra != nullptr && i == 0 && j > 0) dp += cls_extra[(size_t)b * (T_ - 1) + (j - 1)] * invH;
      P[j] = P[j] * (dp - dl);
    }
    __syncwarp();
    float a0 = 0.f, a1 = 0.f;
    for (int j = 0; j < T_; ++j) {
      float x0, x1;
      Row<T>::pair(Ks + (size_t)j * rs, lane, d, x0, x1);
      float ds = P[j];
      a0 = fmaf(ds, x0, a0);
      a1 = fmaf(ds, x1, a1);
    }
    T* drow = dqkv + ((size_t)b * T_ + i) * tok_stride + (size_t)h * d;
    int d0 = Row<T>::dim0(lane), d1 = Row<T>::dim1(lane);
    if (d0 < d) drow[d0] = from_f<T>(a0 * scale);
    if (d1 < d) drow[d1] = from_f<T>(a1 * scale);
    if (lane == 0) delta[((size_t)b * H + h) * T_ + i] = dl;
    __syncwarp();
  }
}

// ---------------------------------------------------------------------------------------------
// backward, part 2: one warp per key row -> dK_j and dV_j
//   dV_j = sum_i P_ij dO_i;  dK_j = scale * sum_i dS_ij Q_i
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(AT_WARPS * 32)
attn_bwd_dkv_kernel(const T* __restrict__ qkv, const T* __restrict__ dout, const float* __restrict__ lse,
                    const float* __restrict__ delta, const float* __restrict__ cls_extra, T* __restrict__ dqkv,
                    int B, int T_, int H, int d, int ksplit) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  int rs = Row<T>::stride(d);
  T* Qs = reinterpret_cast<T*>(smem_raw);
  T* Gs = Qs + (size_t)T_ * rs;
  float* Ps = reinterpret_cast<float*>(Gs + (size_t)T_ * rs);     // [AT_WARPS][2][T_]: P and dS
  float* Ls = Ps + (size_t)AT_WARPS * 2 * T_;                      // lse [T_]
  float* Ds = Ls + T_;                                             // delta [T_]
  float* KVs = Ds + T_;                                            // [AT_WARPS][2][AT_MAXD]: k_j and v_j
  int bh = blockIdx.x, b = bh / H, h = bh % H;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  long tok_stride = 3L * H * d;
  const T* base = qkv + (size_t)b * T_ * tok_stride + (size_t)h * d;
  stage_rows<T>(Qs, base, tok_stride, T_, d);
  stage_rows<T>(Gs, dout + (size_t)b * T_ * H * d + (size_t)h * d, (long)H * d, T_, d);
  for (int i = threadIdx.x; i < T_; i += blockDim.x) {
    Ls[i] = lse[((size_t)b * H + h) * T_ + i];
    Ds[i] = delta[((size_t)b * H + h) * T_ + i];
  }
  __syncthreads();
  float scale = rsqrtf((float)d);
  float invH = 1.0f / (float)H;
  float* P = Ps + (size_t)warp * 2 * T_;
  float* dS = P + T_;
  float* kk = KVs + warp * 2 * AT_MAXD;
  float* vv = kk + AT_MAXD;
  for (int j = blockIdx.y * AT_WARPS + warp; j < T_; j += ksplit * AT_WARPS) {
    const T* krow = base + (size_t)j * tok_stride + (size_t)H * d;
    const T* vrow = krow + (size_t)H * d;
    for (int dd = lane; dd < d; dd += 32) { kk[dd] = to_f(krow[dd]) * scale; vv[dd] = to_f(vrow[dd]); }
    __syncwarp();
    for (int i = lane; i < T_; i += 32) {
      float p = expf(Row<T>::dot(kk, Qs + (size_t)i * rs, d) - Ls[i]);
      float dp = Row<T>::dot(vv, Gs + (size_t)i * rs, d);
      if (cls_extra != nullptr && i == 0 && j > 0) dp += cls_extra[(size_t)b * (T_ - 1) + (j - 1)] * invH;
      P[i] = p;
      dS[i] = p * (dp - Ds[i]);
    }
    __syncwarp();
    float v0 = 0.f, v1 = 0.f, k0 = 0.f, k1 = 0.f;
    for (int i = 0; i < T_; ++i) {
      float g0, g1, q0, q1;
      Row<T>::pair(Gs + (size_t)i * rs, lane, d, g0, g1);
      Row<T>::pair(Qs + (size_t)i * rs, lane, d, q0, q1);
      float p = P[i], ds = dS[i];
      v0 = fmaf(p, g0, v0); v1 = fmaf(p, g1, v1);
      k0 = fmaf(ds, q0, k0); k1 = fmaf(ds, q1, k1);
    }
    T* dk = dqkv + ((size_t)b * T_ + j) * tok_stride + (size_t)H * d + (size_t)h * d;
    T* dv = dk + (size_t)H * d;
    int d0 = Row<T>::dim0(lane), d1 = Row<T>::dim1(lane);
    if (d0 < d) { dk[d0] = from_f<T>(k0 * scale); dv[d0] = from_f<T>(v0); }
    if (d1 < d) { dk[d1] = from_f<T>(k1 * scale); dv[d1] = from_f<T>(v1); }
    __syncwarp();
  }
}

static int split_for(const Ctx& c, int bh, int T_) {
  int sms = c.sm_count > 0 ? c.sm_count : 148;
  int s = ceil_div(2L * sms, bh);
  int cap = ceil_div(T_, AT_WARPS);
  if (s > cap) s = cap;
  return s < 1 ? 1 : s;
}

template <typename T>
static int launch_fwd(const Ctx& c, const void* qkv, void* out, float* lse, float* cls_prob, int B, int T_, int H, int d) {
  size_t rs = d + (sizeof(T) == 2 ? 2 : 1);
  size_t smem = 2 * (size_t)T_ * rs * sizeof(T) + ((size_t)AT_WARPS * T_ + AT_WARPS * AT_MAXD) * sizeof(float);
  if (smem > 227 * 1024) return -2;
  static SmemLimit lim;
  if (!ensure_smem(lim, attn_fwd_kernel<T>, smem)) return -3;
  int qs = split_for(c, B * H, T_);
  dim3 grid(B * H, qs);
  note_launch(1);
  attn_fwd_kernel<T><<<grid, AT_WARPS * 32, smem, c.stream>>>((const T*)qkv, (T*)out, lse, cls_prob, B, T_, H, d, qs);
  return 0;
}

int attention_fwd(const Ctx& c, const void* qkv, void* out, float* lse, float* cls_prob, int B, int T_, int H, int d) {
  if (c.dtype == 1 && c.use_tc && attention_fwd_tc(c, qkv, out, lse, cls_prob, B, T_, H, d) == 0) return 0;
  if (d > AT_MAXD || (d % 8) != 0) return -2;
  return c.dtype == 0 ? launch_fwd<float>(c, qkv, out, lse, cls_prob, B, T_, H, d)
                      : launch_fwd<bf16>(c, qkv, out, lse, cls_prob, B, T_, H, d);
}

template <typename T>
static int launch_bwd(const Ctx& c, const void* qkv, const void* dout, const float* lse, float* delta,
                      const float* cls_extra, void* dqkv, int B, int T_, int H, int d) {
  size_t rs = d + (sizeof(T) == 2 ? 2 : 1);
  size_t smem1 = 2 * (size_t)T_ * rs * sizeof(T) + ((size_t)AT_WARPS * T_ + AT_WARPS * 2 * AT_MAXD) * sizeof(float);
  size_t smem2 = 2 * (size_t)T_ * rs * sizeof(T) + ((size_t)AT_WARPS * 2 * T_ + 2 * (size_t)T_ + AT_WARPS * 2 * AT_MAXD) * sizeof(float);
  if (smem1 > 227 * 1024 || smem2 > 227 * 1024) return -2;
  static SmemLimit lim1, lim2;
  if (!ensure_smem(lim1, attn_bwd_dq_kernel<T>, smem1) || !ensure_smem(lim2, attn_bwd_dkv_kernel<T>, smem2)) return -3;
  int qs = split_for(c, B * H, T_);
  dim3 grid(B * H, qs);
  note_launch(2);
  attn_bwd_dq_kernel<T><<<grid, AT_WARPS * 32, smem1, c.stream>>>((const T*)qkv, (const T*)dout, lse, delta, cls_extra, (T*)dqkv, B, T_, H, d, qs);
  attn_bwd_dkv_kernel<T><<<grid, AT_WARPS * 32, smem2, c.stream>>>((const T*)qkv, (const T*)dout, lse, delta, cls_extra, (T*)dqkv, B, T_, H, d, qs);
  return 0;
}

int attention_bwd(const Ctx& c, const void* qkv, const void* out, const void* dout, const float* lse, float* delta,
                  const float* cls_extra, void* dqkv, int B, int T_, int H, int d) {
  (void)out;
  if (c.dtype == 1 && c.use_tc && attention_bwd_tc(c, qkv, dout, lse, cls_extra, dqkv, B, T_, H, d) == 0) return 0;
  if (d > AT_MAXD || (d % 8) != 0) return -2;
  return c.dtype == 0 ? launch_bwd<float>(c, qkv, dout, lse, delta, cls_extra, dqkv, B, T_, H, d)
                      : launch_bwd<bf16>(c, qkv, dout, lse, delta, cls_extra, dqkv, B, T_, H, d);
}


// ---------------------------------------------------------------------------------------------
// Classification row only.  In the last block nothing but the classification token's output is ever read (the head
// takes row 0), so its attention reduces to one query per (image, head): o_0 = sum_j p_j v_j with p = softmax(q_0 K^T
// / sqrt(d)) (Eq. 1, first row), and in the backward pass only that row carries a gradient: dV_j = p_j dO_0,
// dS_j = p_j (dO_0 . v_j - sum_i p_i dO_0 . v_i), dK_j = dS_j q_0 / sqrt(d), dQ_0 = sum_j dS_j k_j / sqrt(d), every
// other row of dQ is zero.  One block per (image, head); the probabilities are recomputed in the backward kernel.
// ---------------------------------------------------------------------------------------------
constexpr int ATC_WARPS = 4;
constexpr int ATC_THREADS = ATC_WARPS * 32;
constexpr int ATC_MAXKEYS = 1024;                // scores of one row in shared memory

template <typename T> __device__ __forceinline__ float2 ld_pair(const T* p);
template <> __device__ __forceinline__ float2 ld_pair<float>(const float* p) { return *reinterpret_cast<const float2*>(p); }
template <> __device__ __forceinline__ float2 ld_pair<bf16>(const bf16* p) { return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p)); }
template <typename T> __device__ __forceinline__ void st_pair(T* p, float a, float b);
template <> __device__ __forceinline__ void st_pair<float>(float* p, float a, float b) { *reinterpret_cast<float2*>(p) = make_float2(a, b); }
template <> __device__ __forceinline__ void st_pair<bf16>(bf16* p, float a, float b) { *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(a, b); }

// One thread, one key: dot product of the key's (or value's) d entries with a vector in shared memory, 16 bytes a load.
template <typename T>
__device__ __forceinline__ float row_dot(const T* row, const float* vec, int d) {
  constexpr int N = Pack<T>::N;
  float s = 0.f;
  for (int e = 0; e < d; e += N) {
    float kv[N];
    load16(row + e, kv);
#pragma unroll
    for (int i = 0; i < N; i += 4) {
      float4 v = *reinterpret_cast<const float4*>(vec + e + i);
      s = fmaf(v.x, kv[i], s); s = fmaf(v.y, kv[i + 1], s); s = fmaf(v.z, kv[i + 2], s); s = fmaf(v.w, kv[i + 3], s);
    }
  }
  return s;
}

// Block-wide maximum / sum over ATC_WARPS warps, combined in warp order; red holds ATC_WARPS floats.
__device__ __forceinline__ float cls_block_max(float v, float* red) {
  v = warp_max(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = red[0];
#pragma unroll
  for (int w = 1; w < ATC_WARPS; ++w) r = fmaxf(r, red[w]);
  __syncthreads();
  return r;
}
__device__ __forceinline__ float cls_block_sum(float v, float* red) {
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = red[0];
#pragma unroll
  for (int w = 1; w < ATC_WARPS; ++w) r += red[w];
  __syncthreads();
  return r;
}

// Softmax row of the classification query of one (image, head) into sp[0..T): the block's threads stride the keys.
template <typename T>
__device__ __forceinline__ void cls_row_probs(const T* kbase, long row_stride, const float* qs, int T_, int d, float scale,
                                              float* sp, float* red) {
  float mx = -INFINITY;
  for (int j = threadIdx.x; j < T_; j += ATC_THREADS) {
    float s = row_dot<T>(kbase + (long)j * row_stride, qs, d) * scale;
    sp[j] = s;
    mx = fmaxf(mx, s);
  }
  mx = cls_block_max(mx, red);
  float sum = 0.f;
  for (int j = threadIdx.x; j < T_; j += ATC_THREADS) {
    float e = expf(sp[j] - mx);
    sp[j] = e;
    sum += e;
  }
  float inv = 1.0f / cls_block_sum(sum, red);
  for (int j = threadIdx.x; j < T_; j += ATC_THREADS) sp[j] *= inv;
  __syncthreads();
}

// One block of ATC_WARPS warps per (image, head).  Scores: a thread per key.  Weighted sums over the keys: warp w takes
// keys w, w + ATC_WARPS, ... with the lanes across the features (whole rows, coalesced), and the warps' partial sums are
// combined through shared memory in warp order.
template <typename T>
__global__ void __launch_bounds__(ATC_THREADS)
attn_cls_fwd_kernel(const T* __restrict__ qkv, T* __restrict__ out_cls, int B, int T_, int H, int d) {
  __shared__ __align__(16) float qs[AT_MAXD];
  __shared__ float part[ATC_WARPS][AT_MAXD];
  __shared__ float red[ATC_WARPS];
  __shared__ float sp[ATC_MAXKEYS];
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int pair = blockIdx.x;
  int b = pair / H, h = pair % H;
  long row_stride = 3L * H * d;
  const T* base = qkv + (long)b * T_ * row_stride + (long)h * d;
  if (warp == 0 && 2 * lane < d) {
    float2 q = ld_pair<T>(base + 2 * lane);
    qs[2 * lane] = q.x; qs[2 * lane + 1] = q.y;
  }
  __syncthreads();
  cls_row_probs<T>(base + (long)H * d, row_stride, qs, T_, d, rsqrtf((float)d), sp, red);
  // o_0 = sum_j p_j v_j: every lane owns two feature indices; this warp's keys in order
  float o0 = 0.f, o1 = 0.f;
  const T* vbase = base + 2L * H * d;
  if (2 * lane < d) {
#pragma unroll 4
    for (int j = warp; j < T_; j += ATC_WARPS) {
      float2 v = ld_pair<T>(vbase + (long)j * row_stride + 2 * lane);
      float pj = sp[j];
      o0 = fmaf(pj, v.x, o0); o1 = fmaf(pj, v.y, o1);
    }
    part[warp][2 * lane] = o0; part[warp][2 * lane + 1] = o1;
  }
  __syncthreads();
  if (warp == 0 && 2 * lane < d) {
    float a0 = 0.f, a1 = 0.f;
#pragma unroll
    for (int w = 0; w < ATC_WARPS; ++w) { a0 += part[w][2 * lane]; a1 += part[w][2 * lane + 1]; }
    st_pair<T>(out_cls + (long)b * H * d + (long)h * d + 2 * lane, a0, a1);
  }
}

template <typename T>
__global__ void __launch_bounds__(ATC_THREADS)
attn_cls_bwd_kernel(const T* __restrict__ qkv, const T* __restrict__ dout_cls, T* __restrict__ dqkv, int B, int T_, int H, int d) {
  __shared__ __align__(16) float qs[AT_MAXD];
  __shared__ __align__(16) float gs[AT_MAXD];
  __shared__ float part[ATC_WARPS][AT_MAXD];
  __shared__ float red[ATC_WARPS];
  __shared__ float sp[ATC_MAXKEYS], sd[ATC_MAXKEYS];
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int pair = blockIdx.x;
  int b = pair / H, h = pair % H;
  long row_stride = 3L * H * d;
  const T* base = qkv + (long)b * T_ * row_stride + (long)h * d;
  T* dbase = dqkv + (long)b * T_ * row_stride + (long)h * d;
  float q0 = 0.f, q1 = 0.f, g0 = 0.f, g1 = 0.f;
  if (2 * lane < d) {
    float2 q = ld_pair<T>(base + 2 * lane);
    float2 g = ld_pair<T>(dout_cls + (long)b * H * d + (long)h * d + 2 * lane);
    q0 = q.x; q1 = q.y; g0 = g.x; g1 = g.y;
    if (warp == 0) {
      qs[2 * lane] = q0; qs[2 * lane + 1] = q1;
      gs[2 * lane] = g0; gs[2 * lane + 1] = g1;
    }
  }
  __syncthreads();
  float scale = rsqrtf((float)d);
  cls_row_probs<T>(base + (long)H * d, row_stride, qs, T_, d, scale, sp, red);
  // dP_j = dO_0 . v_j (a thread per key), delta = sum_j p_j dP_j
  const T* vbase = base + 2L * H * d;
  float delta = 0.f;
  for (int j = threadIdx.x; j < T_; j += ATC_THREADS) {
    float dp = row_dot<T>(vbase + (long)j * row_stride, gs, d);
    sd[j] = dp;
    delta = fmaf(sp[j], dp, delta);
  }
  delta = cls_block_sum(delta, red);
  for (int j = threadIdx.x; j < T_; j += ATC_THREADS) sd[j] = sp[j] * (sd[j] - delta) * scale;      // dS_j / sqrt(d)
  __syncthreads();
  // rows of this warp's keys: dV_j = p_j dO_0, dK_j = dS_j q_0 / sqrt(d), dQ_j = 0 for j > 0; dQ_0 = sum_j dS_j k_j / sqrt(d)
  float dq0 = 0.f, dq1 = 0.f;
  const T* kbase = base + (long)H * d;
  if (2 * lane < d) {
#pragma unroll 4
    for (int j = warp; j < T_; j += ATC_WARPS) {
      float pj = sp[j], dsj = sd[j];
      float2 k = ld_pair<T>(kbase + (long)j * row_stride + 2 * lane);
      dq0 = fmaf(dsj, k.x, dq0); dq1 = fmaf(dsj, k.y, dq1);
      T* drow = dbase + (long)j * row_stride + 2 * lane;
      st_pair<T>(drow + (long)H * d, dsj * q0, dsj * q1);
      st_pair<T>(drow + 2L * H * d, pj * g0, pj * g1);
      if (j > 0) st_pair<T>(drow, 0.f, 0.f);
    }
    part[warp][2 * lane] = dq0; part[warp][2 * lane + 1] = dq1;
  }
  __syncthreads();
  if (warp == 0 && 2 * lane < d) {
    float a0 = 0.f, a1 = 0.f;
#pragma unroll
    for (int w = 0; w < ATC_WARPS; ++w) { a0 += part[w][2 * lane]; a1 += part[w][2 * lane + 1]; }
    st_pair<T>(dbase + 2 * lane, a0, a1);
  }
}

template <typename T>
static int launch_cls(const Ctx& c, bool bwd, const void* qkv, const void* io_cls, void* dqkv, int B, int T_, int H, int d) {
  if (d > AT_MAXD || (d % 8) != 0 || T_ < 1 || T_ > ATC_MAXKEYS) return -2;
  int blocks = B * H;
  note_launch(1);
  if (bwd) attn_cls_bwd_kernel<T><<<blocks, ATC_THREADS, 0, c.stream>>>((const T*)qkv, (const T*)io_cls, (T*)dqkv, B, T_, H, d);
  else attn_cls_fwd_kernel<T><<<blocks, ATC_THREADS, 0, c.stream>>>((const T*)qkv, (T*)const_cast<void*>(io_cls), B, T_, H, d);
  return 0;
}

int attention_cls_fwd(const Ctx& c, const void* qkv, void* out_cls, int B, int T_, int H, int d) {
  return c.dtype == 0 ? launch_cls<float>(c, false, qkv, out_cls, nullptr, B, T_, H, d) : launch_cls<bf16>(c, false, qkv, out_cls, nullptr, B, T_, H, d);
}
int attention_cls_bwd(const Ctx& c, const void* qkv, const void* dout_cls, void* dqkv, int B, int T_, int H, int d) {
  return c.dtype == 0 ? launch_cls<float>(c, true, qkv, dout_cls, dqkv, B, T_, H, d) : launch_cls<bf16>(c, true, qkv, dout_cls, dqkv, B, T_, H, d);
}

}  // namespace bsr
