// Epilogue of the tcgen05 GEMM kernels: a warp turns 32 rows x 32 columns of fp32 accumulators (lane = row) into
// outputs with bias, GELU, GELU-derivative and residual options, moving data to and from global memory through a
// swizzled staging buffer so that every global access is row-contiguous.
#pragma once

#include "common.cuh"

namespace bsr {
namespace tc {

struct Epi {
  const float* bias = nullptr;
  const void* residual = nullptr;
  void* aux_out = nullptr;
  const void* aux_in = nullptr;
  int act = 0;
  // operands quantised with one scale per row of A and per row of B (8-bit floating point): the accumulator of
  // (row, col) is multiplied by row_scale[row] * col_scale[col] before the bias
  const float* row_scale = nullptr;
  const float* col_scale = nullptr;
};

// Two fp32 lanes per instruction (fma.rn.f32x2 and friends): halves the issue slots of the polynomial below.
__device__ __forceinline__ uint64_t pack2(float a, float b) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t r, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(r)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ uint64_t dup2(float a) { return pack2(a, a); }

// Phi(z) - 1/2 = z * q(z^2) with q a polynomial of degree 8 fitted to erf in double precision on |z| <= 4:
// |error of Phi| < 3e-5 everywhere (4e-6 inside the interval), no special-function unit involved.  Returns
// q(min(z^2, 16)) for two values: beyond |z| = 4 the product z * q(16) leaves [-1/2, 1/2], so that adding 1/2 with
// saturation pins Phi to 0 or 1.  Used where the result is rounded to bf16 (resolution 4e-3 relative).
__device__ __forceinline__ void phi_slope2(float u0, float u1, float& q0, float& q1) {
  uint64_t u = pack2(fminf(u0, 16.0f), fminf(u1, 16.0f));
  uint64_t q = dup2(8.065214468500059e-11f);
  q = fma2(q, u, dup2(-7.004623547857136e-09f));
  q = fma2(q, u, dup2(2.716460869578441e-07f));
  q = fma2(q, u, dup2(-6.295422281255014e-06f));
  q = fma2(q, u, dup2(9.891138324746862e-05f));
  q = fma2(q, u, dup2(-0.001133936457335949f));
  q = fma2(q, u, dup2(0.009877507574856281f));
  q = fma2(q, u, dup2(-0.0664106160402298f));
  q = fma2(q, u, dup2(0.3989226818084717f));
  unpack2(q, q0, q1);
}
// z <- GELU(z) = z * Phi(z), two values.
__device__ __forceinline__ void gelu_fast2(float& z0, float& z1) {
  float u0, u1, q0, q1;
  uint64_t z = pack2(z0, z1);
  unpack2(mul2(z, z), u0, u1);
  phi_slope2(u0, u1, q0, q1);
  z0 *= __saturatef(fmaf(z0, q0, 0.5f));
  z1 *= __saturatef(fmaf(z1, q1, 0.5f));
}
// g <- g * GELU'(z), two values: GELU'(z) = Phi(z) + z * phi(z), with the density phi(z) = exp(-z^2 / 2) / sqrt(2 pi)
// from one exponential of the unclamped square.
__device__ __forceinline__ void gelu_grad_mul2(float& g0, float& g1, float z0, float z1) {
  float u0, u1, q0, q1, d0, d1, e0, e1;
  uint64_t z = pack2(z0, z1);
  unpack2(mul2(z, z), u0, u1);
  phi_slope2(u0, u1, q0, q1);
  const float kh = -0.5f * 1.4426950408889634f;          // exp(-u / 2) = 2^(kh u)
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(u0 * kh));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(u1 * kh));
  unpack2(mul2(z, dup2(0.39894228040143268f)), d0, d1);
  g0 *= fmaf(d0, e0, __saturatef(fmaf(z0, q0, 0.5f)));
  g1 *= fmaf(d1, e1, __saturatef(fmaf(z1, q1, 0.5f)));
}

// The same, also returning h = GELU(z) = z * Phi(z) (the second FFN layer's input, recomputed in the backward pass
// instead of being kept since the forward pass).
__device__ __forceinline__ void gelu_grad_mul2h(float& g0, float& g1, float z0, float z1, float& h0, float& h1) {
  float u0, u1, q0, q1, d0, d1, e0, e1;
  uint64_t z = pack2(z0, z1);
  unpack2(mul2(z, z), u0, u1);
  phi_slope2(u0, u1, q0, q1);
  const float kh = -0.5f * 1.4426950408889634f;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(u0 * kh));
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(u1 * kh));
  unpack2(mul2(z, dup2(0.39894228040143268f)), d0, d1);
  float p0 = __saturatef(fmaf(z0, q0, 0.5f)), p1 = __saturatef(fmaf(z1, q1, 0.5f));
  h0 = z0 * p0; h1 = z1 * p1;
  g0 *= fmaf(d0, e0, p0);
  g1 *= fmaf(d1, e1, p1);
}

// 16-byte global load of data that is read once (residual stream, stored pre-activations).
template <typename T>
__device__ __forceinline__ uint4 ld_stream(const T* p) {
  uint4 x;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(x.x), "=r"(x.y), "=r"(x.z), "=r"(x.w) : "l"(p));
  return x;
}

// A warp moves a 32-row x 32-column chunk between registers (lane = row, v[32] = the row's columns) and global
// memory through its staging buffer, so that the global accesses are row-contiguous: each instruction touches a
// few full rows instead of one 16-byte piece of 32 different rows.
template <typename T>
struct ChunkIO {
  static constexpr int E = 16 / sizeof(T);          // elements per 16-byte unit
  static constexpr int UNITS = 32 / E;               // units per chunk row: 4 (bf16) or 8 (float)
  static constexpr int ROWS_PER_PASS = 32 / UNITS;
  __device__ static uint32_t slot(int r, int u) { return (uint32_t)(r * 128 + ((u ^ (r & 7)) << 4)); }

  // All global loads are issued before the first shared-memory store: the staging pointer may alias anything as
  // far as the compiler knows, so a load placed after a store could not be moved ahead of it.
  __device__ static void load(const T* g, int ld, int row0, int col0, int M, int N, unsigned char* st, int lane, float* v) {
    uint4 x[UNITS];
#pragma unroll
    for (int i = 0; i < UNITS; ++i) {
      int r = i * ROWS_PER_PASS + lane / UNITS, u = lane % UNITS;
      int col = col0 + u * E;
      x[i] = make_uint4(0, 0, 0, 0);
      if (row0 + r < M && col < N) x[i] = ld_stream(g + (size_t)(row0 + r) * ld + col);
    }
#pragma unroll
    for (int i = 0; i < UNITS; ++i) {
      int r = i * ROWS_PER_PASS + lane / UNITS, u = lane % UNITS;
      *reinterpret_cast<uint4*>(st + slot(r, u)) = x[i];
    }
    __syncwarp();
#pragma unroll
    for (int u = 0; u < UNITS; ++u) {
      uint4 y = *reinterpret_cast<const uint4*>(st + slot(lane, u));
      unpack(y, v + u * E);
    }
    __syncwarp();
  }
  __device__ static void store(T* g, int ld, int row0, int col0, int M, int N, unsigned char* st, int lane, const float* v) {
#pragma unroll
    for (int u = 0; u < UNITS; ++u) *reinterpret_cast<uint4*>(st + slot(lane, u)) = pack(v + u * E);
    __syncwarp();
    uint4 x[UNITS];
#pragma unroll
    for (int i = 0; i < UNITS; ++i) {
      int r = i * ROWS_PER_PASS + lane / UNITS, u = lane % UNITS;
      x[i] = *reinterpret_cast<const uint4*>(st + slot(r, u));
    }
#pragma unroll
    for (int i = 0; i < UNITS; ++i) {
      int r = i * ROWS_PER_PASS + lane / UNITS, u = lane % UNITS;
      int col = col0 + u * E;
      if (row0 + r < M && col < N) *reinterpret_cast<uint4*>(g + (size_t)(row0 + r) * ld + col) = x[i];
    }
    __syncwarp();
  }
  __device__ static void unpack(const uint4& x, float* f);
  __device__ static uint4 pack(const float* f);
};
template <> __device__ __forceinline__ void ChunkIO<float>::unpack(const uint4& x, float* f) {
  f[0] = __uint_as_float(x.x); f[1] = __uint_as_float(x.y); f[2] = __uint_as_float(x.z); f[3] = __uint_as_float(x.w);
}
template <> __device__ __forceinline__ uint4 ChunkIO<float>::pack(const float* f) {
  return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
template <> __device__ __forceinline__ void ChunkIO<bf16>::unpack(const uint4& x, float* f) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&x);
#pragma unroll
  for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
}
template <> __device__ __forceinline__ uint4 ChunkIO<bf16>::pack(const float* f) {
  uint4 x;
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&x);
#pragma unroll
  for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  return x;
}

// v[j]: accumulator of (row0 + lane, col0 + j).  All lanes of the warp take part (row0, col0 are warp-uniform).
// zpre: the chunk of the stored pre-activation for act == 2, already in this lane's row order (or null: loaded here).
template <typename TOut>
__device__ __forceinline__ void epilogue_chunk(const uint32_t* r, const Epi& ep, TOut* Cs, int M, int N, int row0, int col0,
                                               unsigned char* st, int lane, const float* zpre = nullptr) {
  if (row0 < M && col0 < N) {
    float v[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
    if (ep.row_scale != nullptr) {
      float rs = row0 + lane < M ? __ldg(ep.row_scale + row0 + lane) : 0.f;
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        if (col0 + g * 4 < N) {
          float4 cs = __ldg(reinterpret_cast<const float4*>(ep.col_scale + col0 + g * 4));
          v[g * 4 + 0] *= rs * cs.x; v[g * 4 + 1] *= rs * cs.y; v[g * 4 + 2] *= rs * cs.z; v[g * 4 + 3] *= rs * cs.w;
        }
      }
    }
    if (ep.bias != nullptr) {
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        if (col0 + g * 4 < N) {
          float4 bb = __ldg(reinterpret_cast<const float4*>(ep.bias + col0 + g * 4));
          v[g * 4 + 0] += bb.x; v[g * 4 + 1] += bb.y; v[g * 4 + 2] += bb.z; v[g * 4 + 3] += bb.w;
        }
      }
    }
    if (ep.act == 1) {
      if (ep.aux_out != nullptr) ChunkIO<TOut>::store((TOut*)ep.aux_out, N, row0, col0, M, N, st, lane, v);
#pragma unroll
      for (int j = 0; j < 32; j += 2) gelu_fast2(v[j], v[j + 1]);
    } else if (ep.act == 2) {
      float z[32];
      if (zpre != nullptr) {
#pragma unroll
        for (int j = 0; j < 32; ++j) z[j] = zpre[j];
      } else {
        ChunkIO<bf16>::load((const bf16*)ep.aux_in, N, row0, col0, M, N, st, lane, z);
      }
      if (ep.aux_out != nullptr) {          // GELU(z) recomputed for the weight gradient of the second FFN layer
#pragma unroll
        for (int j = 0; j < 32; j += 2) gelu_grad_mul2h(v[j], v[j + 1], z[j], z[j + 1], z[j], z[j + 1]);
        ChunkIO<bf16>::store((bf16*)ep.aux_out, N, row0, col0, M, N, st, lane, z);
      } else {
#pragma unroll
        for (int j = 0; j < 32; j += 2) gelu_grad_mul2(v[j], v[j + 1], z[j], z[j + 1]);
      }
    }
    if (ep.residual != nullptr) {
      float rr[32];
      ChunkIO<TOut>::load((const TOut*)ep.residual, N, row0, col0, M, N, st, lane, rr);
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] += rr[j];
    }
    ChunkIO<TOut>::store(Cs, N, row0, col0, M, N, st, lane, v);
  }
}


// ---- float outputs without activation (projection, second FFN layer, weight gradients) ----------------------------
// The accumulators are transposed once, through the staging buffer, into the row-contiguous order in which global
// memory is read and written; bias and residual are added in that order, so the residual needs no staging at all and
// its loads (issued by chunk_issue a chunk ahead, the first of a tile before the tile's accumulator is complete) stay
// in flight while the tensor-memory read and the transposition proceed.
__device__ __forceinline__ void chunk_issue(const float* g, int ld, int row0, int col0, int M, int N, int lane, uint4* x) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    int r = i * 4 + lane / 8, col = col0 + (lane % 8) * 4;
    x[i] = make_uint4(0, 0, 0, 0);
    if (row0 + r < M && col < N) x[i] = ld_stream(g + (size_t)(row0 + r) * ld + col);
  }
}
__device__ __forceinline__ void epilogue_chunk_f32(const uint32_t* r, const float* bias, float* Cs, int M, int N, int row0, int col0,
                                                   unsigned char* st, int lane, const uint4* xres, bool has_res) {
  if (row0 < M && col0 < N) {
    using IO = ChunkIO<float>;
#pragma unroll
    for (int u = 0; u < 8; ++u)
      *reinterpret_cast<uint4*>(st + IO::slot(lane, u)) = make_uint4(r[4 * u], r[4 * u + 1], r[4 * u + 2], r[4 * u + 3]);
    __syncwarp();
    int u = lane % 8, col = col0 + u * 4;
    float4 bb = make_float4(0.f, 0.f, 0.f, 0.f);
    if (bias != nullptr && col < N) bb = __ldg(reinterpret_cast<const float4*>(bias + col));
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      int rr = i * 4 + lane / 8;
      uint4 a = *reinterpret_cast<const uint4*>(st + IO::slot(rr, u));
      float4 v = make_float4(__uint_as_float(a.x) + bb.x, __uint_as_float(a.y) + bb.y, __uint_as_float(a.z) + bb.z, __uint_as_float(a.w) + bb.w);
      if (has_res) {
        v.x += __uint_as_float(xres[i].x); v.y += __uint_as_float(xres[i].y); v.z += __uint_as_float(xres[i].z); v.w += __uint_as_float(xres[i].w);
      }
      if (row0 + rr < M && col < N) *reinterpret_cast<float4*>(Cs + (size_t)(row0 + rr) * N + col) = v;
    }
    __syncwarp();
  }
}

// Stored pre-activation chunk (bf16) fetched ahead of use: four 16-byte units per lane in row-contiguous order, later
// turned into this lane's row through the staging buffer.
__device__ __forceinline__ void chunk_issue(const bf16* g, int ld, int row0, int col0, int M, int N, int lane, uint4* x) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int r = i * 8 + lane / 4, col = col0 + (lane % 4) * 8;
    x[i] = make_uint4(0, 0, 0, 0);
    if (row0 + r < M && col < N) x[i] = ld_stream(g + (size_t)(row0 + r) * ld + col);
  }
}
__device__ __forceinline__ void chunk_land_bf16(const uint4* x, unsigned char* st, int lane, float* v) {
  using IO = ChunkIO<bf16>;
#pragma unroll
  for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(st + IO::slot(i * 8 + lane / 4, lane % 4)) = x[i];
  __syncwarp();
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    uint4 y = *reinterpret_cast<const uint4*>(st + IO::slot(lane, u));
    IO::unpack(y, v + u * 8);
  }
  __syncwarp();
}

// ---- the same with the auxiliary input (residual, or the stored pre-activation) prefetched one chunk ahead ----
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// Starts the copy of a 32 x 32 chunk of g into the staging buffer `st` (shared address `st_addr`); out-of-range
// units are zero-filled.
template <typename T>
__device__ __forceinline__ void chunk_prefetch(const T* g, int ld, int row0, int col0, int M, int N, uint32_t st_addr, int lane) {
  using IO = ChunkIO<T>;
#pragma unroll
  for (int i = 0; i < IO::UNITS; ++i) {
    int r = i * IO::ROWS_PER_PASS + lane / IO::UNITS, u = lane % IO::UNITS;
    int col = col0 + u * IO::E;
    bool in = row0 + r < M && col < N;
    const T* src = in ? g + (size_t)(row0 + r) * ld + col : g;
    cp_async16(st_addr + IO::slot(r, u), src, in ? 16u : 0u);
  }
  cp_async_commit();
}
template <typename T>
__device__ __forceinline__ void chunk_take(unsigned char* st, int lane, float* v) {
  using IO = ChunkIO<T>;
  cp_async_wait_all();
  __syncwarp();
#pragma unroll
  for (int u = 0; u < IO::UNITS; ++u) {
    uint4 x = *reinterpret_cast<const uint4*>(st + IO::slot(lane, u));
    IO::unpack(x, v + u * IO::E);
  }
  __syncwarp();
}

// One warp's share of a tile: `nchunks` chunks of 32 columns starting at column colbase, accumulators at
// taddr0 + 32 * chunk.  st_in / st_out: two staging buffers of this warp.
template <typename TOut, typename LoadTmem>
__device__ __forceinline__ void epilogue_warp_tile(LoadTmem load_tmem, const Epi& ep, TOut* Cs, int M, int N, int row0, int colbase,
                                                   int nchunks, unsigned char* st_in, uint32_t st_in_addr, unsigned char* st_out,
                                                   int lane, bool prefetched_first) {
  bool pre_res = ep.residual != nullptr;
  bool pre_aux = !pre_res && ep.act == 2;
  for (int cc = 0; cc < nchunks; ++cc) {
    int col0 = colbase + cc * 32;
    uint32_t r[32];
    load_tmem(cc, r);
    bool live = row0 < M && col0 < N;                       // warp-uniform
    if (!live) continue;
    if (cc == 0 && !prefetched_first) {
      if (pre_res) chunk_prefetch<TOut>((const TOut*)ep.residual, N, row0, col0, M, N, st_in_addr, lane);
      else if (pre_aux) chunk_prefetch<bf16>((const bf16*)ep.aux_in, N, row0, col0, M, N, st_in_addr, lane);
    }
    float v[32], a[32];
    if (pre_res) chunk_take<TOut>(st_in, lane, a);
    else if (pre_aux) chunk_take<bf16>(st_in, lane, a);
    if (cc + 1 < nchunks && col0 + 32 < N) {                // next chunk's auxiliary input, overlapped with this chunk's work
      if (pre_res) chunk_prefetch<TOut>((const TOut*)ep.residual, N, row0, col0 + 32, M, N, st_in_addr, lane);
      else if (pre_aux) chunk_prefetch<bf16>((const bf16*)ep.aux_in, N, row0, col0 + 32, M, N, st_in_addr, lane);
    }
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
    if (ep.bias != nullptr) {
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        if (col0 + g * 4 < N) {
          float4 bb = __ldg(reinterpret_cast<const float4*>(ep.bias + col0 + g * 4));
          v[g * 4 + 0] += bb.x; v[g * 4 + 1] += bb.y; v[g * 4 + 2] += bb.z; v[g * 4 + 3] += bb.w;
        }
      }
    }
    if (ep.act == 1) {
      if (ep.aux_out != nullptr) ChunkIO<TOut>::store((TOut*)ep.aux_out, N, row0, col0, M, N, st_out, lane, v);
#pragma unroll
      for (int j = 0; j < 32; j += 2) gelu_fast2(v[j], v[j + 1]);
    } else if (ep.act == 2) {
      if (!pre_aux) ChunkIO<bf16>::load((const bf16*)ep.aux_in, N, row0, col0, M, N, st_out, lane, a);
      if (ep.aux_out != nullptr) {
#pragma unroll
        for (int j = 0; j < 32; j += 2) gelu_grad_mul2h(v[j], v[j + 1], a[j], a[j + 1], a[j], a[j + 1]);
        ChunkIO<bf16>::store((bf16*)ep.aux_out, N, row0, col0, M, N, st_out, lane, a);
      } else {
#pragma unroll
        for (int j = 0; j < 32; j += 2) gelu_grad_mul2(v[j], v[j + 1], a[j], a[j + 1]);
      }
    }
    if (pre_res) {
#pragma unroll
      for (int j = 0; j < 32; ++j) v[j] += a[j];
    }
    ChunkIO<TOut>::store(Cs, N, row0, col0, M, N, st_out, lane, v);
  }
}

}  // namespace tc
}  // namespace bsr
