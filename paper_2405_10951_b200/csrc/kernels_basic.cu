// Bandwidth-bound kernels of the BSR step: patch extraction, token assembly, LayerNorm forward and
// backward, column sums, head/loss, AdamW, conversions.  All reductions run in a fixed order.
#include "common.cuh"
#include "kernels.h"

namespace bsr {

long g_kernel_launches = 0;

// ------------------------------------------------------------------------------------------------
// Patch extraction (Section 3.1: the image is partitioned into N patches).  Output row = one patch
// flattened as (channel, row in patch, column in patch).
// ------------------------------------------------------------------------------------------------
// img_offset (optional): element offset of this step's images from `img`, read from device memory (multi-step loop).
template <typename T>
__global__ void patchify_kernel(const T* __restrict__ img, T* __restrict__ out, int B, int C, int S, int P, long total,
                                const long long* __restrict__ img_offset) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  if (img_offset != nullptr) img += *img_offset;
  int g = S / P;
  int px = (int)(i % P); long r = i / P;
  int py = (int)(r % P); r /= P;
  int ch = (int)(r % C); r /= C;
  int gx = (int)(r % g); r /= g;
  int gy = (int)(r % g); r /= g;
  int b = (int)r;
  out[i] = img[(((long)b * C + ch) * S + (gy * P + py)) * S + gx * P + px];
}

// Same copy in 16-byte units (P * sizeof(T) a multiple of 16): a patch row is P/E units.
template <typename T>
__global__ void patchify_vec_kernel(const T* __restrict__ img, T* __restrict__ out, int B, int C, int S, int P, long units,
                                    const long long* __restrict__ img_offset) {
  constexpr int E = 16 / sizeof(T);
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= units) return;
  if (img_offset != nullptr) img += *img_offset;
  int g = S / P, upr = P / E;
  int ux = (int)(i % upr); long r = i / upr;
  int py = (int)(r % P); r /= P;
  int ch = (int)(r % C); r /= C;
  int gx = (int)(r % g); r /= g;
  int gy = (int)(r % g); r /= g;
  int b = (int)r;
  const T* src = img + (((long)b * C + ch) * S + (gy * P + py)) * S + gx * P + ux * E;
  *reinterpret_cast<uint4*>(out + i * E) = *reinterpret_cast<const uint4*>(src);
}

void patchify(const Ctx& c, const void* images, void* patches, int B, int C, int S, int P, const long long* img_offset) {
  note_launch(1);
  int g = S / P;
  long total = (long)B * g * g * C * P * P;
  int threads = 256;
  size_t es = dtype_size(c.dtype);
  // with an offset read on the device, every step's images must be 16-byte aligned: one image holds C*S*S elements
  bool vec = (P * es) % 16 == 0 && (((uintptr_t)images | (uintptr_t)patches) & 15) == 0 &&
             (img_offset == nullptr || ((long)C * S * S * (long)es) % 16 == 0);
  if (vec) {
    long units = total * (long)es / 16;
    int blocks = ceil_div(units, threads);
    if (c.dtype == 0) patchify_vec_kernel<float><<<blocks, threads, 0, c.stream>>>((const float*)images, (float*)patches, B, C, S, P, units, img_offset);
    else patchify_vec_kernel<bf16><<<blocks, threads, 0, c.stream>>>((const bf16*)images, (bf16*)patches, B, C, S, P, units, img_offset);
    return;
  }
  int blocks = ceil_div(total, threads);
  if (c.dtype == 0)
    patchify_kernel<float><<<blocks, threads, 0, c.stream>>>((const float*)images, (float*)patches, B, C, S, P, total, img_offset);
  else
    patchify_kernel<bf16><<<blocks, threads, 0, c.stream>>>((const bf16*)images, (bf16*)patches, B, C, S, P, total, img_offset);
}

// x[b, 0] = cls + pos[0];  x[b, 1 + n] = emb[b, n] + pos[1 + n]   (classification token and positional embedding);
// four columns per thread (D % 4 == 0).
template <typename T>
__global__ void assemble_kernel(const T* __restrict__ emb, const float* __restrict__ cls, const float* __restrict__ pos,
                                float* __restrict__ x, int B, int N, int D, long total4) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total4) return;
  int d4 = D / 4;
  int d = (int)(i % d4) * 4; long r = i / d4;
  int t = (int)(r % (N + 1));
  int b = (int)(r / (N + 1));
  float v[4], p[4];
  if (t == 0) load16(cls + d, v);
  else load4(emb + ((long)b * N + (t - 1)) * D + d, v);
  load16(pos + (long)t * D + d, p);
#pragma unroll
  for (int j = 0; j < 4; ++j) v[j] += p[j];
  store16(x + i * 4, v);
}

void assemble_tokens(const Ctx& c, const void* emb, const float* cls, const float* pos, float* x, int B, int N, int D) {
  note_launch(1);
  long total4 = (long)B * (N + 1) * D / 4;
  int threads = 256, blocks = ceil_div(total4, threads);
  if (c.dtype == 0)
    assemble_kernel<float><<<blocks, threads, 0, c.stream>>>((const float*)emb, cls, pos, x, B, N, D, total4);
  else
    assemble_kernel<bf16><<<blocks, threads, 0, c.stream>>>((const bf16*)emb, cls, pos, x, B, N, D, total4);
}

// ------------------------------------------------------------------------------------------------
// LayerNorm.  The residual stream x is float in every configuration (only the small block updates
// would survive bf16 rounding of the stream poorly); the normalised output feeds a GEMM and takes
// the storage dtype.  One warp per row, the row held in registers (D <= 1024, D % 4 == 0).
// ------------------------------------------------------------------------------------------------
// NCH = 16-byte chunks of the row each lane holds (D <= 128 * NCH); instantiated for 2, 3, 4, 6 and 8.

template <typename TY, int NCH>
__global__ void layernorm_fwd_kernel(const float* __restrict__ x, long x_stride, const float* __restrict__ g,
                                     const float* __restrict__ b, TY* __restrict__ y, float* __restrict__ mean,
                                     float* __restrict__ rstd, int rows, int D, float eps) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  int lane = threadIdx.x & 31;
  if (warp >= rows) return;
  const float* xr = x + (long)warp * x_stride;
  int chunks = D / 4;
  float v[(NCH * 4)];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    int ch = lane + i * 32;
    if (ch < chunks) {
      load16(xr + ch * 4, v + i * 4);
#pragma unroll
      for (int j = 0; j < 4; ++j) sum += v[i * 4 + j];
    }
  }
  float mu = warp_sum(sum) / (float)D;
  float sq = 0.f;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    int ch = lane + i * 32;
    if (ch < chunks) {
#pragma unroll
      for (int j = 0; j < 4; ++j) { float t = v[i * 4 + j] - mu; sq += t * t; }
    }
  }
  float rs = rsqrtf(warp_sum(sq) / (float)D + eps);
  if (lane == 0) {
    if (mean) mean[warp] = mu;
    if (rstd) rstd[warp] = rs;
  }
  TY* yr = y + (long)warp * D;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    int ch = lane + i * 32;
    if (ch < chunks) {
      float4 gg = *reinterpret_cast<const float4*>(g + ch * 4), bb = *reinterpret_cast<const float4*>(b + ch * 4);
      float o[4];
      o[0] = (v[i * 4 + 0] - mu) * rs * gg.x + bb.x;
      o[1] = (v[i * 4 + 1] - mu) * rs * gg.y + bb.y;
      o[2] = (v[i * 4 + 2] - mu) * rs * gg.z + bb.z;
      o[3] = (v[i * 4 + 3] - mu) * rs * gg.w + bb.w;
      store4(yr + ch * 4, o);
    }
  }
}

template <typename TY>
static void launch_ln_fwd(const Ctx& c, const float* x, long x_stride, const float* g, const float* b, TY* y, float* mean,
                          float* rstd, int rows, int D, float eps) {
  int threads = 256;
  int blocks = ceil_div((long)rows * 32, threads);
  int nch = ceil_div(D, 128);
#define BSR_LN_FWD(N) layernorm_fwd_kernel<TY, N><<<blocks, threads, 0, c.stream>>>(x, x_stride, g, b, y, mean, rstd, rows, D, eps)
  if (nch <= 2) BSR_LN_FWD(2); else if (nch == 3) BSR_LN_FWD(3); else if (nch == 4) BSR_LN_FWD(4); else if (nch <= 6) BSR_LN_FWD(6); else BSR_LN_FWD(8);
#undef BSR_LN_FWD
}

void layernorm_fwd(const Ctx& c, const float* x, long x_stride, const float* g, const float* b, void* y, int y_is_float,
                   float* mean, float* rstd, int rows, int D, float eps) {
  note_launch(1);
  if (c.dtype == 0 || y_is_float) launch_ln_fwd<float>(c, x, x_stride, g, b, (float*)y, mean, rstd, rows, D, eps);
  else launch_ln_fwd<bf16>(c, x, x_stride, g, b, (bf16*)y, mean, rstd, rows, D, eps);
}

// ------------------------------------------------------------------------------------------------
// E4M3 (8-bit floating point: 1 sign, 4 exponent, 3 mantissa bits, largest magnitude 448) rows with one scale each.
// ------------------------------------------------------------------------------------------------
// Two floats to two E4M3 bytes, round to nearest even, saturating; a in the low byte.
__device__ __forceinline__ uint16_t to_e4m3x2(float a, float b) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(b), "f"(a));
  return r;
}
__device__ __forceinline__ uint32_t to_e4m3x4(const float* v, float s) {
  return (uint32_t)to_e4m3x2(__fdiv_rn(v[0], s), __fdiv_rn(v[1], s)) | ((uint32_t)to_e4m3x2(__fdiv_rn(v[2], s), __fdiv_rn(v[3], s)) << 16);
}
__device__ __forceinline__ float e4m3_scale(float amax) { return amax > 0.f ? __fdiv_rn(amax, 448.0f) : 1.0f; }

// One warp per row (cols % 4 == 0): scale = max|row| / 448, q = round(x / scale).
__global__ void quantize_rows_e4m3_kernel(const bf16* __restrict__ x, int rows, int cols, uint8_t* __restrict__ q, float* __restrict__ scale) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= rows) return;
  const bf16* xr = x + (size_t)warp * cols;
  float amax = 0.f;
  for (int ch = lane; ch < cols / 4; ch += 32) {
    float v[4];
    load4(xr + ch * 4, v);
#pragma unroll
    for (int j = 0; j < 4; ++j) amax = fmaxf(amax, fabsf(v[j]));
  }
  amax = warp_max(amax);
  float s = e4m3_scale(amax);
  if (lane == 0) scale[warp] = s;
  uint32_t* qr = reinterpret_cast<uint32_t*>(q + (size_t)warp * cols);
  for (int ch = lane; ch < cols / 4; ch += 32) {
    float v[4];
    load4(xr + ch * 4, v);
    qr[ch] = to_e4m3x4(v, s);
  }
}
void quantize_rows_e4m3(const Ctx& c, const void* x, int rows, int cols, void* q, float* scale) {
  note_launch(1);
  quantize_rows_e4m3_kernel<<<ceil_div((long)rows * 32, 256), 256, 0, c.stream>>>((const bf16*)x, rows, cols, (uint8_t*)q, scale);
}

// E4M3 byte to float: sign, exponent (bias 7) and mantissa unpacked by hand (subnormals: exponent field 0).
__device__ __forceinline__ float from_e4m3(uint8_t b) {
  int e = (b >> 3) & 15, m = b & 7;
  float v = e == 0 ? (float)m * 0.001953125f : ldexpf(1.0f + (float)m * 0.125f, e - 7);
  return (b & 0x80) ? -v : v;
}
__global__ void dequantize_rows_e4m3_kernel(const uint8_t* __restrict__ q, const float* __restrict__ scale, int rows, int cols,
                                            float* __restrict__ out) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (size_t)rows * cols) return;
  out[i] = from_e4m3(q[i]) * scale[i / cols];
}
void dequantize_rows_e4m3(const Ctx& c, const void* q, const float* scale, int rows, int cols, float* out) {
  note_launch(1);
  dequantize_rows_e4m3_kernel<<<ceil_div((long)rows * cols, 256), 256, 0, c.stream>>>((const uint8_t*)q, scale, rows, cols, out);
}

// LayerNorm forward whose output row goes out as E4M3 with scale max|y| / 448: the row is already in the warp's
// registers, so the quantisation costs one more warp reduction and halves the bytes written.
template <int NCH>
__global__ void layernorm_fwd_e4m3_kernel(const float* __restrict__ x, long x_stride, const float* __restrict__ g,
                                          const float* __restrict__ b, uint8_t* __restrict__ yq, float* __restrict__ y_scale,
                                          int rows, int D, float eps) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  int lane = threadIdx.x & 31;
  if (warp >= rows) return;
  const float* xr = x + (long)warp * x_stride;
  int chunks = D / 4;
  float v[(NCH * 4)];
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    int ch = lane + i * 32;
    if (ch < chunks) {
      load16(xr + ch * 4, v + i * 4);
#pragma unroll
      for (int j = 0; j < 4; ++j) sum += v[i * 4 + j];
    }
  }
  float mu = warp_sum(sum) / (float)D;
  float sq = 0.f;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    int ch = lane + i * 32;
    if (ch < chunks) {
#pragma unroll
      for (int j = 0; j < 4; ++j) { float t = v[i * 4 + j] - mu; sq += t * t; }
    }
  }
  float rs = rsqrtf(warp_sum(sq) / (float)D + eps);
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    int ch = lane + i * 32;
    if (ch < chunks) {
      float4 gg = *reinterpret_cast<const float4*>(g + ch * 4), bb = *reinterpret_cast<const float4*>(b + ch * 4);
      v[i * 4 + 0] = (v[i * 4 + 0] - mu) * rs * gg.x + bb.x;
      v[i * 4 + 1] = (v[i * 4 + 1] - mu) * rs * gg.y + bb.y;
      v[i * 4 + 2] = (v[i * 4 + 2] - mu) * rs * gg.z + bb.z;
      v[i * 4 + 3] = (v[i * 4 + 3] - mu) * rs * gg.w + bb.w;
#pragma unroll
      for (int j = 0; j < 4; ++j) amax = fmaxf(amax, fabsf(v[i * 4 + j]));
    }
  }
  amax = warp_max(amax);
  float s = e4m3_scale(amax);
  if (lane == 0) y_scale[warp] = s;
  uint32_t* qr = reinterpret_cast<uint32_t*>(yq + (size_t)warp * D);
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    int ch = lane + i * 32;
    if (ch < chunks) qr[ch] = to_e4m3x4(v + i * 4, s);
  }
}
void layernorm_fwd_e4m3(const Ctx& c, const float* x, long x_stride, const float* g, const float* b, void* yq, float* y_scale,
                        int rows, int D, float eps) {
  note_launch(1);
  int threads = 256;
  int blocks = ceil_div((long)rows * 32, threads);
  int nch = ceil_div(D, 128);
#define BSR_LN_Q(N) layernorm_fwd_e4m3_kernel<N><<<blocks, threads, 0, c.stream>>>(x, x_stride, g, b, (uint8_t*)yq, y_scale, rows, D, eps)
  if (nch <= 2) BSR_LN_Q(2); else if (nch == 3) BSR_LN_Q(3); else if (nch == 4) BSR_LN_Q(4); else if (nch <= 6) BSR_LN_Q(6); else BSR_LN_Q(8);
#undef BSR_LN_Q
}

// Backward.  Each block owns rows blockIdx.x*8 + warp, stepping by gridDim.x*8; every lane accumulates the
// dgamma/dbeta contributions of its columns, warps are combined through shared memory in warp order, and the
// block's sums go to partials[0][block][col] (dgamma) and partials[1][block][col] (dbeta).
// dx (float, the gradient of the residual stream) = dres + LN'(dy); dx_copy receives the same values in the
// storage dtype for the GEMMs that consume them.
constexpr int LNB_WARPS = 8;

template <typename TDY, typename TC, int NCH>
__global__ void __launch_bounds__(256, 2) layernorm_bwd_kernel(const TDY* __restrict__ dy, const float* __restrict__ x, long x_stride,
                                     const float* __restrict__ mean, const float* __restrict__ rstd,
                                     const float* __restrict__ g, const float* __restrict__ dres, float* __restrict__ dx,
                                     long dx_stride, TC* __restrict__ dx_copy, float* __restrict__ partials, int rows, int D, int nsum) {
  extern __shared__ float sm[];   // [LNB_WARPS][nsum][D]: dgamma, dbeta and (nsum == 3) the column sums of dx
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int chunks = D / 4;
  // The warp's partial sums for the scale and shift gradients live in its slice of shared memory (each lane owns
  // its columns), which leaves the registers for a whole row of x, dy and the residual gradient in flight at once.
  float* mine = sm + (size_t)warp * nsum * D;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    int ch = lane + i * 32;
    if (ch < chunks) {
      *reinterpret_cast<float4*>(mine + ch * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
      *reinterpret_cast<float4*>(mine + D + ch * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
      if (nsum == 3) *reinterpret_cast<float4*>(mine + 2 * D + ch * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  for (int r = blockIdx.x * LNB_WARPS + warp; r < rows; r += gridDim.x * LNB_WARPS) {
    const float* xr = x + (long)r * x_stride;
    const TDY* dyr = dy + (long)r * D;
    float mu = mean[r], rs = rstd[r];
    float xh[(NCH * 4)], dh[(NCH * 4)], o[(NCH * 4)];
#pragma unroll
    for (int i = 0; i < NCH; ++i) {                      // all loads of the row first
      int ch = lane + i * 32;
      if (ch < chunks) {
        load16(xr + ch * 4, xh + i * 4);
        load4(dyr + ch * 4, dh + i * 4);
        if (dx != nullptr && dres != nullptr) load16(dres + (long)r * D + ch * 4, o + i * 4);
        else {
#pragma unroll
          for (int j = 0; j < 4; ++j) o[i * 4 + j] = 0.f;
        }
      }
    }
    float s1 = 0.f, s2 = 0.f;
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
      int ch = lane + i * 32;
      if (ch < chunks) {
        float4 gg = *reinterpret_cast<const float4*>(g + ch * 4);
        float gv[4] = {gg.x, gg.y, gg.z, gg.w};
        float4 pg = *reinterpret_cast<const float4*>(mine + ch * 4);
        float4 pb = *reinterpret_cast<const float4*>(mine + D + ch * 4);
        float pgv[4] = {pg.x, pg.y, pg.z, pg.w}, pbv[4] = {pb.x, pb.y, pb.z, pb.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float d = dh[i * 4 + j];
          float h = (xh[i * 4 + j] - mu) * rs;
          xh[i * 4 + j] = h;
          pgv[j] += d * h;
          pbv[j] += d;
          float dxh = d * gv[j];
          dh[i * 4 + j] = dxh;
          s1 += dxh;
          s2 += dxh * h;
        }
        *reinterpret_cast<float4*>(mine + ch * 4) = make_float4(pgv[0], pgv[1], pgv[2], pgv[3]);
        *reinterpret_cast<float4*>(mine + D + ch * 4) = make_float4(pbv[0], pbv[1], pbv[2], pbv[3]);
      }
    }
    s1 = warp_sum(s1) / (float)D;
    s2 = warp_sum(s2) / (float)D;
    if (dx != nullptr) {
      float* dxr = dx + (long)r * dx_stride;
#pragma unroll
      for (int i = 0; i < NCH; ++i) {
        int ch = lane + i * 32;
        if (ch < chunks) {
#pragma unroll
          for (int j = 0; j < 4; ++j) o[i * 4 + j] += rs * (dh[i * 4 + j] - s1 - xh[i * 4 + j] * s2);
          store16(dxr + ch * 4, o + i * 4);
          if (dx_copy != nullptr) store4(dx_copy + (long)r * dx_stride + ch * 4, o + i * 4);
          if (nsum == 3) {
            float4 ps = *reinterpret_cast<const float4*>(mine + 2 * D + ch * 4);
            ps.x += o[i * 4]; ps.y += o[i * 4 + 1]; ps.z += o[i * 4 + 2]; ps.w += o[i * 4 + 3];
            *reinterpret_cast<float4*>(mine + 2 * D + ch * 4) = ps;
          }
        }
      }
    }
  }
  __syncthreads();
  for (int col = threadIdx.x; col < nsum * D; col += blockDim.x) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < LNB_WARPS; ++w) s += sm[(size_t)w * nsum * D + col];
    int which = col / D, cc = col % D;
    partials[((size_t)which * gridDim.x + blockIdx.x) * D + cc] = s;
  }
}

// out_y[col] = sum over groups of partials[y][group][col] for y = blockIdx.y (one or two outputs per launch).
// 16 lanes stride the groups and are combined through shared memory in lane order: the result is deterministic.
__global__ void reduce_partials_kernel(const float* __restrict__ partials, int groups, int cols, float* __restrict__ out0,
                                       float* __restrict__ out1, float* __restrict__ out2 = nullptr) {
  __shared__ float sm[16][17];
  int cx = threadIdx.x & 15, gy = threadIdx.x >> 4;
  int col = blockIdx.x * 16 + cx;
  const float* p = partials + (size_t)blockIdx.y * groups * cols;
  float s = 0.f;
  if (col < cols)
    for (int g = gy; g < groups; g += 16) s += p[(size_t)g * cols + col];
  sm[gy][cx] = s;
  __syncthreads();
  if (gy == 0 && col < cols) {
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) t += sm[i][cx];
    float* out = blockIdx.y == 0 ? out0 : (blockIdx.y == 1 ? out1 : out2);
    if (out != nullptr) out[col] = t;
  }
}

int layernorm_bwd_groups(const Ctx& c, int rows) {
  int want = ceil_div(rows, LNB_WARPS);
  int cap = c.sm_count > 0 ? 2 * c.sm_count : 296;
  return want < cap ? (want < 1 ? 1 : want) : cap;
}

template <typename TDY, typename TC>
static void launch_ln_bwd(const Ctx& c, int groups, size_t smem, const void* dy, const float* x, long x_stride, const float* mean,
                          const float* rstd, const float* g, const float* dres, float* dx, long dx_stride, void* dx_copy,
                          float* partials, int rows, int D, int nsum) {
  int nch = ceil_div(D, 128);
#define BSR_LN_BWD(N)                                                                                                   \
  do {                                                                                                                  \
    static SmemLimit lim;                                                                                               \
    ensure_smem(lim, layernorm_bwd_kernel<TDY, TC, N>, smem);                                                           \
    layernorm_bwd_kernel<TDY, TC, N><<<groups, LNB_WARPS * 32, smem, c.stream>>>((const TDY*)dy, x, x_stride, mean, rstd, g, dres, \
                                                                                 dx, dx_stride, (TC*)dx_copy, partials, rows, D, nsum); \
  } while (0)
  if (nch <= 2) BSR_LN_BWD(2); else if (nch == 3) BSR_LN_BWD(3); else if (nch == 4) BSR_LN_BWD(4); else if (nch <= 6) BSR_LN_BWD(6); else BSR_LN_BWD(8);
#undef BSR_LN_BWD
}

void layernorm_bwd(const Ctx& c, const void* dy, int dy_is_float, const float* x, long x_stride, const float* mean,
                   const float* rstd, const float* g, const float* dres, float* dx, long dx_stride, void* dx_copy,
                   float* partials, float* dgamma, float* dbeta, int rows, int D, float* dx_colsum) {
  note_launch(2);
  int groups = layernorm_bwd_groups(c, rows);
  int nsum = (dx_colsum != nullptr && dx != nullptr) ? 3 : 2;
  size_t smem = (size_t)LNB_WARPS * nsum * D * sizeof(float);
  side_join(c, 0);                                                     // the previous reduction has read the partials
  if (c.dtype == 0)
    launch_ln_bwd<float, float>(c, groups, smem, dy, x, x_stride, mean, rstd, g, dres, dx, dx_stride, nullptr, partials, rows, D, nsum);
  else if (dy_is_float)
    launch_ln_bwd<float, bf16>(c, groups, smem, dy, x, x_stride, mean, rstd, g, dres, dx, dx_stride, dx_copy, partials, rows, D, nsum);
  else
    launch_ln_bwd<bf16, bf16>(c, groups, smem, dy, x, x_stride, mean, rstd, g, dres, dx, dx_stride, dx_copy, partials, rows, D, nsum);
  if (dgamma == nullptr && nsum == 2) return;                          // a frozen block in the gradient path: only dx is wanted
  dim3 grid(ceil_div(D, 16), nsum);
  cudaStream_t rs = side_begin(c);                                     // only the optimiser reads these sums
  reduce_partials_kernel<<<grid, 256, 0, rs>>>(partials, groups, D, dgamma, dbeta, nsum == 3 ? dx_colsum : nullptr);
  side_end(c, 0);
}

// ------------------------------------------------------------------------------------------------
// Column sums (bias gradients): two stages, fixed order.
// ------------------------------------------------------------------------------------------------
constexpr int CS_ROWLANES = 8;
constexpr int CS_GROUPS = 64;

template <typename T>
__global__ void colsum_kernel(const T* __restrict__ x, int rows, int cols, float* __restrict__ partials) {
  constexpr int N = Pack<T>::N;
  __shared__ float sm[CS_ROWLANES][32 * N];
  int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  int col0 = (blockIdx.x * 32 + tx) * N;
  float acc[N];
#pragma unroll
  for (int j = 0; j < N; ++j) acc[j] = 0.f;
  if (col0 < cols) {
    // four rows per trip: their loads are independent and issued together, the additions keep the row order
    const int step = gridDim.y * CS_ROWLANES;
    int r = blockIdx.y * CS_ROWLANES + ty;
    for (; r + 3 * step < rows; r += 4 * step) {
      float v[4][N];
#pragma unroll
      for (int u = 0; u < 4; ++u) load16(x + (long)(r + u * step) * cols + col0, v[u]);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
#pragma unroll
        for (int j = 0; j < N; ++j) acc[j] += v[u][j];
      }
    }
    for (; r < rows; r += step) {
      float v[N];
      load16(x + (long)r * cols + col0, v);
#pragma unroll
      for (int j = 0; j < N; ++j) acc[j] += v[j];
    }
  }
#pragma unroll
  for (int j = 0; j < N; ++j) sm[ty][tx * N + j] = acc[j];
  __syncthreads();
  for (int cidx = threadIdx.x; cidx < 32 * N; cidx += blockDim.x) {
    int col = blockIdx.x * 32 * N + cidx;
    if (col < cols) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < CS_ROWLANES; ++w) s += sm[w][cidx];
      partials[(size_t)blockIdx.y * cols + col] = s;
    }
  }
}

int colsum_groups(int rows) {
  int want = ceil_div(rows, CS_ROWLANES);
  return want < CS_GROUPS ? (want < 1 ? 1 : want) : CS_GROUPS;
}

void colsum(const Ctx& c, const void* x, int rows, int cols, float* partials, float* out) {
  note_launch(2);
  int groups = colsum_groups(rows);
  int threads = CS_ROWLANES * 32;
  side_join(c, 1);
  if (c.dtype == 0) {
    dim3 grid(ceil_div(cols, 32 * 4), groups);
    colsum_kernel<float><<<grid, threads, 0, c.stream>>>((const float*)x, rows, cols, partials);
  } else {
    dim3 grid(ceil_div(cols, 32 * 8), groups);
    colsum_kernel<bf16><<<grid, threads, 0, c.stream>>>((const bf16*)x, rows, cols, partials);
  }
  cudaStream_t rs = side_begin(c);
  reduce_partials_kernel<<<dim3(ceil_div(cols, 16), 1), 256, 0, rs>>>(partials, groups, cols, out, out);
  side_end(c, 1);
}

// ------------------------------------------------------------------------------------------------
// Classification head on the normalised classification token, cross-entropy, head backward.
// ------------------------------------------------------------------------------------------------
struct HeadDev {
  int num_tasks, cmax, D;
  int ncls[4];
  const void* w[4];
  const float* bias[4];
  float* dw[4];
  float* db[4];
};

template <typename T>
__global__ void head_fwd_kernel(HeadDev h, const float* __restrict__ xn, const int* __restrict__ task_ids,
                                float* __restrict__ logits, int B) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= B * h.cmax) return;
  int b = warp / h.cmax, cls = warp % h.cmax;
  int t = task_ids ? task_ids[b] : 0;
  if (cls >= h.ncls[t]) {
    if (lane == 0) logits[warp] = -INFINITY;
    return;
  }
  const T* w = (const T*)h.w[t] + (size_t)cls * h.D;
  const float* xr = xn + (size_t)b * h.D;
  float s = 0.f;
  for (int d = lane; d < h.D; d += 32) s += xr[d] * to_f(w[d]);
  s = warp_sum(s);
  if (lane == 0) logits[warp] = s + h.bias[t][cls];
}

static HeadDev to_dev(const HeadDesc& h) {
  HeadDev d;
  d.num_tasks = h.num_tasks; d.cmax = h.cmax; d.D = h.D;
  for (int i = 0; i < 4; ++i) { d.ncls[i] = h.ncls[i]; d.w[i] = h.w[i]; d.bias[i] = h.bias[i]; d.dw[i] = h.dw[i]; d.db[i] = h.db[i]; }
  return d;
}

void head_fwd(const Ctx& c, const HeadDesc& h, const float* xn, const int* task_ids, float* logits, int B) {
  note_launch(1);
  int threads = 256, blocks = ceil_div((long)B * h.cmax * 32, threads);
  if (c.dtype == 0) head_fwd_kernel<float><<<blocks, threads, 0, c.stream>>>(to_dev(h), xn, task_ids, logits, B);
  else head_fwd_kernel<bf16><<<blocks, threads, 0, c.stream>>>(to_dev(h), xn, task_ids, logits, B);
}

// One warp per image: loss_b = logsumexp(logits) - logits[label]; dlogits = (softmax - onehot) / B.
__global__ void cross_entropy_kernel(HeadDev h, const float* __restrict__ logits, const int* __restrict__ labels,
                                     const int* __restrict__ task_ids, float* __restrict__ per_image,
                                     float* __restrict__ dlogits, int B, int* status) {
  int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= B) return;
  int t = task_ids ? task_ids[warp] : 0;
  // labels and task ids come from the caller: in every build a value outside its range raises STATUS_CHECK and is
  // clamped, instead of indexing outside the logits
  if (t < 0 || t >= h.num_tasks) {
    if (lane == 0 && status != nullptr) atomicOr(status, STATUS_CHECK);
    t = 0;
  }
  int n = h.ncls[t];
  const float* lr = logits + (size_t)warp * h.cmax;
  float mx = -INFINITY;
  for (int i = lane; i < n; i += 32) mx = fmaxf(mx, lr[i]);
  mx = warp_max(mx);
  float se = 0.f;
  for (int i = lane; i < n; i += 32) se += expf(lr[i] - mx);
  se = warp_sum(se);
  int label = labels[warp];
  if (label < 0 || label >= n) {
    if (lane == 0 && status != nullptr) atomicOr(status, STATUS_CHECK);
    label = 0;
  }
  float inv = 1.0f / se, invB = 1.0f / (float)B;
  for (int i = lane; i < h.cmax; i += 32) {
    float g = 0.f;
    if (i < n) g = (expf(lr[i] - mx) * inv - (i == label ? 1.f : 0.f)) * invB;
    dlogits[(size_t)warp * h.cmax + i] = g;
  }
  if (lane == 0) per_image[warp] = logf(se) + mx - lr[label];
}

// Single warp: mean of the per-image losses, lanes stride the images, fixed order.
__global__ void loss_reduce_kernel(const float* __restrict__ per_image, int B, float* __restrict__ loss, int* status) {
  int lane = threadIdx.x;
  float s = 0.f;
  for (int i = lane; i < B; i += 32) s += per_image[i];
  s = warp_sum(s);
  if (lane == 0) {
    float l = s / (float)B;
    *loss = l;
    if (status != nullptr && !isfinite(l)) atomicOr(status, STATUS_NONFINITE);
  }
}

void cross_entropy(const Ctx& c, const HeadDesc& h, const float* logits, const int* labels, const int* task_ids,
                   float* per_image, float* dlogits, float* loss, int B) {
  note_launch(2);
  int threads = 128, blocks = ceil_div((long)B * 32, threads);
  cross_entropy_kernel<<<blocks, threads, 0, c.stream>>>(to_dev(h), logits, labels, task_ids, per_image, dlogits, B, c.status);
  loss_reduce_kernel<<<1, 32, 0, c.stream>>>(per_image, B, loss, c.status);
}

// dW_t[c, d] = sum_b [task(b) = t] dlogits[b, c] xn[b, d];  db_t[c] = sum_b [..] dlogits[b, c]
__global__ void head_wgrad_kernel(HeadDev h, const float* __restrict__ xn, const float* __restrict__ dlogits,
                                  const int* __restrict__ task_ids, int B, int t) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  int n = h.ncls[t];
  if (i >= n * (h.D + 1)) return;
  int cls = i / (h.D + 1), d = i % (h.D + 1);
  // branch-free and unrolled: the loads of eight images are in flight together; the sum still runs in image order
  float s = 0.f;
#pragma unroll 8
  for (int b = 0; b < B; ++b) {
    int tb = task_ids ? task_ids[b] : 0;
    float g = (tb == t) ? dlogits[(size_t)b * h.cmax + cls] : 0.f;
    float x = (d < h.D) ? xn[(size_t)b * h.D + d] : 1.f;
    s = fmaf(g, x, s);
  }
  if (d < h.D) h.dw[t][(size_t)cls * h.D + d] = s;
  else h.db[t][cls] = s;
}

template <typename T>
__global__ void head_dgrad_kernel(HeadDev h, const float* __restrict__ dlogits, const int* __restrict__ task_ids,
                                  float* __restrict__ dxn, int B) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= B * h.D) return;
  int b = i / h.D, d = i % h.D;
  int t = task_ids ? task_ids[b] : 0;
  const T* w = (const T*)h.w[t];
  float s = 0.f;
  for (int cidx = 0; cidx < h.ncls[t]; ++cidx) s += dlogits[(size_t)b * h.cmax + cidx] * to_f(w[(size_t)cidx * h.D + d]);
  dxn[i] = s;
}

void head_bwd(const Ctx& c, const HeadDesc& h, const float* xn, const float* dlogits, const int* task_ids, float* dxn, int B) {
  note_launch(h.num_tasks + 1);
  HeadDev hd = to_dev(h);
  for (int t = 0; t < h.num_tasks; ++t) {
    int total = h.ncls[t] * (h.D + 1);
    head_wgrad_kernel<<<ceil_div(total, 128), 128, 0, c.stream>>>(hd, xn, dlogits, task_ids, B, t);
  }
  int total = B * h.D;
  if (c.dtype == 0) head_dgrad_kernel<float><<<ceil_div(total, 128), 128, 0, c.stream>>>(hd, dlogits, task_ids, dxn, B);
  else head_dgrad_kernel<bf16><<<ceil_div(total, 128), 128, 0, c.stream>>>(hd, dlogits, task_ids, dxn, B);
}

// ------------------------------------------------------------------------------------------------
// AdamW over the flat trainable-parameter buffers (Section 5: DeiT-S is trained with AdamW).
//   m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;  p <- p - lr * (m/bc1) / (sqrt(v/bc2) + eps) - lr * wd * p
// One block per chunk; a chunk never straddles two tensors.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void adamw_kernel(const AdamChunk* __restrict__ chunks, float* __restrict__ master,
                             const float* __restrict__ grad, float* __restrict__ m, float* __restrict__ v,
                             T* __restrict__ shadow_base, const float* __restrict__ scalars, float b1, float b2, float eps,
                             float wd) {
  // step-dependent scalars live in device memory so that a captured graph of the step stays valid: lr, 1-b1^t, 1-b2^t
  float lr = scalars[0], bc1 = scalars[1], bc2 = scalars[2];
  AdamChunk ch = chunks[blockIdx.x];
  float decay = ch.decay ? lr * wd : 0.f;
  for (uint32_t i = threadIdx.x; i < ch.count; i += blockDim.x) {
    size_t idx = (size_t)ch.offset + i;
    float g = grad[idx];
    float p = master[idx];
    float mm = b1 * m[idx] + (1.f - b1) * g;
    float vv = b2 * v[idx] + (1.f - b2) * g * g;
    m[idx] = mm;
    v[idx] = vv;
    float np = p - lr * (mm / bc1) / (sqrtf(vv / bc2) + eps) - decay * p;
    master[idx] = np;
    if (ch.shadow >= 0) shadow_base[ch.shadow + i] = from_f<T>(np);
  }
}

// SGD with momentum on the same chunk table: buf <- mu buf + (g + wd p), p <- p - lr buf.
template <typename T>
__global__ void sgd_kernel(const AdamChunk* __restrict__ chunks, float* __restrict__ master, const float* __restrict__ grad,
                           float* __restrict__ buf, T* __restrict__ shadow_base, const float* __restrict__ scalars, float mu,
                           float wd) {
  float lr = scalars[0];
  AdamChunk ch = chunks[blockIdx.x];
  float decay = ch.decay ? wd : 0.f;
  for (uint32_t i = threadIdx.x; i < ch.count; i += blockDim.x) {
    size_t idx = (size_t)ch.offset + i;
    float p = master[idx];
    float b = mu * buf[idx] + (grad[idx] + decay * p);
    buf[idx] = b;
    float np = p - lr * b;
    master[idx] = np;
    if (ch.shadow >= 0) shadow_base[ch.shadow + i] = from_f<T>(np);
  }
}

void sgd_momentum(const Ctx& c, const AdamChunk* chunks, int nchunks, float* master, const float* grad, float* buf,
                  void* shadow_base, const float* scalars, float mu, float wd) {
  if (nchunks <= 0) return;
  note_launch(1);
  if (c.dtype == 0)
    sgd_kernel<float><<<nchunks, 256, 0, c.stream>>>(chunks, master, grad, buf, (float*)shadow_base, scalars, mu, wd);
  else
    sgd_kernel<bf16><<<nchunks, 256, 0, c.stream>>>(chunks, master, grad, buf, (bf16*)shadow_base, scalars, mu, wd);
}

// ------------------------------------------------------------------------------------------------
// Multi-step loop (Section 5: cosine learning-rate decay).  The state lives in device memory; each step's graph reads
// it, so a run of steps needs no host scalars: lr(t) = lr_min + (lr_max - lr_min) (1 + cos(pi t / total)) / 2 for the
// t-th step overall (t from 0, held at lr_min from t = total on), bias corrections 1 - beta^(t+1).
// ------------------------------------------------------------------------------------------------
__global__ void loop_init_kernel(LoopState* st, long long step_done, long long total, long long image_stride, float lr_max,
                                 float lr_min, float b1, float b2, int n) {
  st->step_done = step_done; st->total_steps = total; st->image_stride = image_stride; st->image_offset = 0;
  st->lr_max = lr_max; st->lr_min = lr_min; st->beta1 = b1; st->beta2 = b2; st->i = 0; st->n = n;
}
__global__ void loop_begin_kernel(LoopState* st, float* scalars, const int* __restrict__ labels, const int* __restrict__ tasks,
                                  int* __restrict__ lab_stage, int* __restrict__ task_stage, int batch) {
  int i = st->i;
  for (int j = threadIdx.x; j < batch; j += blockDim.x) {
    lab_stage[j] = labels[(long)i * batch + j];
    if (tasks != nullptr) task_stage[j] = tasks[(long)i * batch + j];
  }
  if (threadIdx.x == 0) {
    long long t = st->step_done;
    double frac = st->total_steps > 0 ? (double)(t < st->total_steps ? t : st->total_steps) / (double)st->total_steps : 1.0;
    double lr = (double)st->lr_min + 0.5 * ((double)st->lr_max - (double)st->lr_min) * (1.0 + cos(3.14159265358979323846 * frac));
    scalars[0] = (float)lr;
    scalars[1] = (float)(1.0 - pow((double)st->beta1, (double)(t + 1)));
    scalars[2] = (float)(1.0 - pow((double)st->beta2, (double)(t + 1)));
    st->image_offset = (long long)i * st->image_stride;
  }
}
__global__ void loop_end_kernel(LoopState* st, const float* __restrict__ loss, float* __restrict__ loss_out) {
  loss_out[st->i] = *loss;
  st->i += 1;
  st->step_done += 1;
}
void loop_init(cudaStream_t s, LoopState* st, long long step_done, long long total, long long image_stride, float lr_max, float lr_min,
               float b1, float b2, int n) {
  note_launch(1);
  loop_init_kernel<<<1, 1, 0, s>>>(st, step_done, total, image_stride, lr_max, lr_min, b1, b2, n);
}
void loop_begin(cudaStream_t s, LoopState* st, float* scalars, const int* labels, const int* tasks, int* lab_stage, int* task_stage, int batch) {
  note_launch(1);
  loop_begin_kernel<<<1, 256, 0, s>>>(st, scalars, labels, tasks, lab_stage, task_stage, batch);
}
void loop_end(cudaStream_t s, LoopState* st, const float* loss, float* loss_out) {
  note_launch(1);
  loop_end_kernel<<<1, 1, 0, s>>>(st, loss, loss_out);
}

// Guard words after every workspace slice: one warp per guard.
__global__ void guards_write_kernel(char* base, const unsigned long long* __restrict__ table, int n, int words, uint32_t word) {
  int g = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (g >= n) return;
  uint32_t* p = reinterpret_cast<uint32_t*>(base + table[g]);
  for (int i = lane; i < words; i += 32) p[i] = word;
}
__global__ void guards_check_kernel(const char* base, const unsigned long long* __restrict__ table, int n, int words, uint32_t word,
                                    int* status) {
  int g = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (g >= n) return;
  const uint32_t* p = reinterpret_cast<const uint32_t*>(base + table[g]);
  bool bad = false;
  for (int i = lane; i < words; i += 32) bad |= p[i] != word;
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, STATUS_GUARD);
}
void guards_write(cudaStream_t s, char* base, const unsigned long long* table, int n, int words, uint32_t word) {
  note_launch(1);
  guards_write_kernel<<<ceil_div((long)n * 32, 256), 256, 0, s>>>(base, table, n, words, word);
}
void guards_check(cudaStream_t s, const char* base, const unsigned long long* table, int n, int words, uint32_t word, int* status) {
  note_launch(1);
  guards_check_kernel<<<ceil_div((long)n * 32, 256), 256, 0, s>>>(base, table, n, words, word, status);
}

__global__ void set_scalars_kernel(float* dst, float a, float b, float c3) {
  dst[0] = a; dst[1] = b; dst[2] = c3;
}
void set_scalars(cudaStream_t s, float* dst, float a, float b, float c3) {
  note_launch(1);
  set_scalars_kernel<<<1, 1, 0, s>>>(dst, a, b, c3);
}

void adamw(const Ctx& c, const AdamChunk* chunks, int nchunks, float* master, const float* grad, float* m, float* v,
           void* shadow_base, const float* scalars, float b1, float b2, float eps, float wd) {
  if (nchunks <= 0) return;
  note_launch(1);
  if (c.dtype == 0)
    adamw_kernel<float><<<nchunks, 256, 0, c.stream>>>(chunks, master, grad, m, v, (float*)shadow_base, scalars, b1, b2, eps, wd);
  else
    adamw_kernel<bf16><<<nchunks, 256, 0, c.stream>>>(chunks, master, grad, m, v, (bf16*)shadow_base, scalars, b1, b2, eps, wd);
}

// ------------------------------------------------------------------------------------------------
// Strided row copy in 16-byte units: dst[r] = src[r] for rows of row_bytes, each side with its own row pitch.
// Gathers the classification rows of a [B, T, D] tensor into [B, D] and scatters them back.
// ------------------------------------------------------------------------------------------------
__global__ void copy_rows_kernel(const char* __restrict__ src, long src_pitch, char* __restrict__ dst, long dst_pitch, int rows,
                                 int units) {
  long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long)rows * units) return;
  int r = (int)(i / units), u = (int)(i % units);
  *reinterpret_cast<uint4*>(dst + (long)r * dst_pitch + u * 16L) = *reinterpret_cast<const uint4*>(src + (long)r * src_pitch + u * 16L);
}

void copy_rows(cudaStream_t st, const void* src, long src_pitch_bytes, void* dst, long dst_pitch_bytes, int rows, int row_bytes) {
  note_launch(1);
  int units = row_bytes / 16;
  long total = (long)rows * units;
  copy_rows_kernel<<<ceil_div(total, 256), 256, 0, st>>>((const char*)src, src_pitch_bytes, (char*)dst, dst_pitch_bytes, rows, units);
}

// ------------------------------------------------------------------------------------------------
// Conversions
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void from_float_kernel(const float* __restrict__ s, T* __restrict__ d, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) d[i] = from_f<T>(s[i]);
}
template <typename T>
__global__ void to_float_kernel(const T* __restrict__ s, float* __restrict__ d, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) d[i] = to_f(s[i]);
}
__global__ void fill_kernel(float* d, float v, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) d[i] = v;
}

void convert_from_float(const Ctx& c, const float* src, void* dst, size_t n) {
  note_launch(1);
  if (n == 0) return;
  int blocks = ceil_div((long)n, 256);
  if (c.dtype == 0) from_float_kernel<float><<<blocks, 256, 0, c.stream>>>(src, (float*)dst, n);
  else from_float_kernel<bf16><<<blocks, 256, 0, c.stream>>>(src, (bf16*)dst, n);
}
void convert_to_float(const Ctx& c, const void* src, float* dst, size_t n) {
  note_launch(1);
  if (n == 0) return;
  int blocks = ceil_div((long)n, 256);
  if (c.dtype == 0) to_float_kernel<float><<<blocks, 256, 0, c.stream>>>((const float*)src, dst, n);
  else to_float_kernel<bf16><<<blocks, 256, 0, c.stream>>>((const bf16*)src, dst, n);
}
__global__ void int_to_float_kernel(const int* s, float* d, size_t n) {
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) d[i] = (float)s[i];
}
void convert_int_to_float(cudaStream_t st, const int* src, float* dst, size_t n) {
  if (n == 0) return;
  note_launch(1);
  int_to_float_kernel<<<ceil_div((long)n, 256), 256, 0, st>>>(src, dst, n);
}
void fill_float(cudaStream_t s, float* dst, float v, size_t n) {
  note_launch(1);
  if (n == 0) return;
  fill_kernel<<<ceil_div((long)n, 256), 256, 0, s>>>(dst, v, n);
}

}  // namespace bsr
