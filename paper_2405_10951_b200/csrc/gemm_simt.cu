// FP32-FMA dense contraction with arbitrary operand strides.  It is the contraction of the fp32
// configuration (TF32 tensor-core math cannot hold a 1e-4 relative tolerance) and the fall-back for
// bf16 problems the tcgen05 kernel does not take (tiny or unaligned shapes).
#include "common.cuh"
#include "kernels.h"

namespace bsr {

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16, SG_THREADS = 256;

template <typename T, typename TC>
__global__ void __launch_bounds__(SG_THREADS)
gemm_simt_kernel(const T* __restrict__ A, long a_rs, long a_cs, const T* __restrict__ B, long b_rs, long b_cs,
                 TC* __restrict__ C, int M, int N, int K, const float* __restrict__ bias, const TC* __restrict__ residual,
                 int act, TC* __restrict__ aux_out, const T* __restrict__ aux_in) {
  __shared__ float As[SG_BK][SG_BM + 4];
  __shared__ float Bs[SG_BK][SG_BN + 4];
  int tid = threadIdx.x;
  int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  int tx = tid % 16, ty = tid / 16;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  bool a_kmajor = (a_cs == 1), b_kmajor = (b_cs == 1);
  for (int k0 = 0; k0 < K; k0 += SG_BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int idx = tid + i * SG_THREADS;
      int r, kk;
      if (a_kmajor) { r = idx / SG_BK; kk = idx % SG_BK; } else { r = idx % SG_BM; kk = idx / SG_BM; }
      int gm = m0 + r, gk = k0 + kk;
      As[kk][r] = (gm < M && gk < K) ? to_f(A[(long)gm * a_rs + (long)gk * a_cs]) : 0.f;
      if (b_kmajor) { r = idx / SG_BK; kk = idx % SG_BK; } else { r = idx % SG_BN; kk = idx / SG_BN; }
      int gn = n0 + r;
      gk = k0 + kk;
      Bs[kk][r] = (gn < N && gk < K) ? to_f(B[(long)gn * b_rs + (long)gk * b_cs]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < SG_BK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      size_t o = (size_t)gm * N + gn;
      float v = acc[i][j];
      if (bias != nullptr) v += bias[gn];
      if (act == 1) {
        if (aux_out != nullptr) aux_out[o] = from_f<TC>(v);
        v = gelu_f(v);
      } else if (act == 2) {
        float z = to_f(aux_in[o]);
        v *= gelu_grad_f(z);
        if (aux_out != nullptr) reinterpret_cast<T*>(aux_out)[o] = from_f<T>(gelu_f(z));     // GELU(z), storage type
      }
      if (residual != nullptr) v += to_f(residual[o]);
      C[o] = from_f<TC>(v);
    }
  }
}

void gemm(const Ctx& c, const void* A, long a_rs, long a_cs, const void* B, long b_rs, long b_cs, void* C,
          int out_is_float, int m, int n, int k, const GemmEpilogue& e) {
  if (m <= 0 || n <= 0) return;
  if (c.dtype == 1 && c.use_tc && gemm_tc_supported(m, n, k)) {
    if (c.use_tc >= 2 && m > 128 &&
        gemm_tc2_strided(c, A, a_rs, a_cs, B, b_rs, b_cs, C, out_is_float, m, n, k, e, c.split_ws, c.split_ws_floats) == 0) return;
    if (gemm_tc_strided(c, A, a_rs, a_cs, B, b_rs, b_cs, C, out_is_float, m, n, k, e, c.split_ws, c.split_ws_floats) == 0) return;
  }
  dim3 grid(ceil_div(n, SG_BN), ceil_div(m, SG_BM));
  note_launch(1);
  if (c.dtype == 0) {
    gemm_simt_kernel<float, float><<<grid, SG_THREADS, 0, c.stream>>>(
        (const float*)A, a_rs, a_cs, (const float*)B, b_rs, b_cs, (float*)C, m, n, k, e.bias, (const float*)e.residual,
        e.act, (float*)e.aux_out, (const float*)e.aux_in);
  } else if (out_is_float) {
    gemm_simt_kernel<bf16, float><<<grid, SG_THREADS, 0, c.stream>>>(
        (const bf16*)A, a_rs, a_cs, (const bf16*)B, b_rs, b_cs, (float*)C, m, n, k, e.bias, (const float*)e.residual,
        e.act, (float*)e.aux_out, (const bf16*)e.aux_in);
  } else {
    gemm_simt_kernel<bf16, bf16><<<grid, SG_THREADS, 0, c.stream>>>(
        (const bf16*)A, a_rs, a_cs, (const bf16*)B, b_rs, b_cs, (bf16*)C, m, n, k, e.bias, (const bf16*)e.residual,
        e.act, (bf16*)e.aux_out, (const bf16*)e.aux_in);
  }
}

}  // namespace bsr
