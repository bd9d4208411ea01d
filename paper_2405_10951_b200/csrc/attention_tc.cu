// Multi-head self-attention (paper Eq. 1) on the tcgen05 tensor cores for bf16, head dimension 64.
//
// Forward (T <= 256 keys): a persistent, warp-specialised kernel (see attn_fwd_ws_kernel): TMA loads Q, K, V tiles of
//   the packed projections [B*T, 3*H*64] into 128-byte-swizzled shared memory; S = Q K^T goes to tensor memory; a
//   thread owns (half of) a query row: row maximum, exp2, row sum in float from tcgen05.ld; the probabilities go back
//   into tensor memory as bf16 and O = P V reads them from there; the epilogue scales by 1 / row sum.
//   The classification token's row (query 0) is also written out as probabilities: these are the token
//   importance scores of Eq. 6.
// Rows and keys beyond T inside a tile belong to the next image (or are zero-filled past the tensor's end):
// keys are masked in the softmax, rows are computed and never stored.
#include "common.cuh"
#include "kernels.h"
#include "tc_ptx.cuh"

namespace bsr {
namespace tc {

constexpr int AT_D = 64;
constexpr int AT_BOX = 64;                       // rows per TMA box
constexpr int AT_BOX_BYTES = AT_BOX * AT_D * 2;  // 8 KB
constexpr int AT_QROWS = 128;
constexpr int AT_MAXKEYS = 256;
constexpr float AT_LONG_SLACK = 8.0f;             // binary orders the row maximum may exceed the reference before a rescale
constexpr int AT_LONG_MAXBLK = 64;                // key blocks of the longest sequence the kernel takes
constexpr int AT_LONG_KB = 64;                   // keys per block of the kernel for longer sequences (four CTAs per SM)

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Byte offset of element (row, key) in a probability tile stored as 64-key chunks of [128 rows x 128 bytes],
// 16-byte units XOR-swizzled with the row (the layout TMA produces for a 128-byte-swizzled operand tile).
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float ex2_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t p_offset(int row, int key8) {   // key8: index of a group of 8 keys
  int chunk = key8 >> 3, unit = key8 & 7;
  return (uint32_t)(chunk * (AT_QROWS * 128) + row * 128 + ((unit ^ (row & 7)) << 4));
}

// ------------------------------------------------------------------------------------------------
// Forward for T <= 256, persistent and warp-specialised: one CTA per SM walks (image, head) pairs.
//   loader warp : TMA (one lane): K and V of a pair into a ring of slots, each 128-query tile of Q into another
//                 ring, running ahead of the tensor core as far as the slots allow;
//   NBUF softmax groups, one per accumulator buffer in tensor memory, each working on every NBUF-th tile.  A group's
//                 first thread also issues the group's MMAs: S = Q K^T for the group's next tile as soon as the
//                 previous O has been read, and O = P V as soon as the group has written P.  A thread owns (half
//                 of) a query row: row maximum and exp2 from tcgen05.ld, probabilities packed to bf16 and written
//                 back with tcgen05.st over the S columns already consumed (P never goes through shared memory,
//                 the second MMA reads it from tensor memory), then O scaled by the row sum and stored.
// NBUF is 4, 3 or 2 for up to 128, 160 or 256 keys; with two groups a group has eight warps, two per lane quarter
// splitting the keys (and the output columns).  Accumulator buffer layout (columns): S at 0 .. tpad-1 (fp32), P (bf16
// pairs) over S columns its writer has already consumed, O in the last 64 columns of the buffer, beyond P.
// ------------------------------------------------------------------------------------------------
constexpr int WS_QSLOTS = 3;
constexpr int WS_Q_BYTES = 2 * AT_BOX_BYTES;
constexpr int WS_MAXBUF = 4, WS_MAXKV = 6;

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void group_sync(int id, int threads) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory"); }
// mbar_wait that gives up at once when another role already has: after a failure the groups keep walking their
// tiles (their named barriers need every thread) and every further wait must return quickly.
__device__ __forceinline__ bool mbar_wait_q(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  if (*abort_flag) return false;
  return mbar_wait(bar, parity, abort_flag);
}

template <int NBUF>
__global__ void __launch_bounds__((NBUF == 2 ? 19 : 4 * NBUF + 3) * 32, 1)
attn_fwd_ws_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kv, bf16* __restrict__ out,
                   float* __restrict__ lse, float* __restrict__ cls_prob, int B, int T, int H, int kvslots, int* status) {
  constexpr int GW = NBUF == 2 ? 8 : 4;                         // warps per softmax group
  constexpr int GT = GW * 32;
  constexpr uint32_t BUF_COLS = NBUF == 2 ? 256u : (NBUF == 3 ? 160u : 128u);
  constexpr uint32_t O_COL = BUF_COLS - 64u;                                 // 192, 96, 64
  extern __shared__ unsigned char smem_dyn[];
  uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const int tpad = (T + 15) & ~15;
  const int nqt = (T + AT_QROWS - 1) / AT_QROWS;
  const uint32_t kv_bytes = tpad * 128;                          // one of K, V: tpad rows of 64 bf16
  const uint32_t sQ = base, sKV = sQ + WS_QSLOTS * WS_Q_BYTES;
  const uint32_t tail = sKV + kvslots * 2 * kv_bytes;
  float* cls_buf = reinterpret_cast<float*>(base_ptr + (tail - base));     // [NBUF][AT_MAXKEYS]
  float* red = cls_buf + WS_MAXBUF * AT_MAXKEYS;                            // [NBUF][max, sum][2 halves][128 rows]
  const uint32_t bars = tail + (WS_MAXBUF * AT_MAXKEYS + WS_MAXBUF * 4 * AT_QROWS) * 4;
  auto q_full = [&](int s) { return bars + 8u * s; };
  auto q_empty = [&](int s) { return bars + 8u * (4 + s); };
  auto kv_full = [&](int s) { return bars + 8u * (8 + s); };
  auto kv_empty = [&](int s) { return bars + 8u * (16 + s); };
  auto s_full = [&](int b) { return bars + 8u * (24 + b); };
  auto o_full = [&](int b) { return bars + 8u * (28 + b); };
  auto p_full = [&](int b) { return bars + 8u * (32 + b); };
  auto t_empty = [&](int b) { return bars + 8u * (36 + b); };
  auto token = [&](int b) { return bars + 8u * (40 + b); };
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int pairs = B * H;
  constexpr int LOADER = NBUF * GW;                             // then the two MMA issuer warps

  if (tid == 0) {
    abort_flag = 0;
    for (int s = 0; s < WS_QSLOTS; ++s) { mbar_init(q_full(s), 1); mbar_init(q_empty(s), 1); }
    for (int s = 0; s < WS_MAXKV; ++s) { mbar_init(kv_full(s), 1); mbar_init(kv_empty(s), nqt); }
    for (int b = 0; b < WS_MAXBUF; ++b) {
      mbar_init(s_full(b), 1); mbar_init(o_full(b), 1); mbar_init(p_full(b), GW); mbar_init(t_empty(b), GW); mbar_init(token(b), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == LOADER) {
    tmem_alloc(smem_u32(&tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  volatile int* abortp = &abort_flag;

  if (warp == LOADER) {
    // ------------------------------- TMA loader ---------------------------------
    if (lane == 0) {
      int i = 0, n = 0;
      bool ok = true;
      for (int bh = blockIdx.x; bh < pairs && ok; bh += gridDim.x, ++n) {
        int b = bh / H, h = bh % H, row0 = b * T;
        int ks = n % kvslots;
        if (!mbar_wait(kv_empty(ks), ((n / kvslots) & 1) ^ 1u, abortp)) { ok = false; break; }
        mbar_expect_tx(kv_full(ks), 2 * kv_bytes);
        uint32_t sK = sKV + ks * 2 * kv_bytes, sV = sK + kv_bytes;
        tma_load_2d(sK, &map_kv, kv_full(ks), (H + h) * AT_D, row0);
        tma_load_2d(sV, &map_kv, kv_full(ks), (2 * H + h) * AT_D, row0);
        for (int qt = 0; qt < nqt; ++qt, ++i) {
          int qs = i % WS_QSLOTS;
          if (!mbar_wait(q_empty(qs), ((i / WS_QSLOTS) & 1) ^ 1u, abortp)) { ok = false; break; }
          mbar_expect_tx(q_full(qs), WS_Q_BYTES);
          tma_load_2d(sQ + qs * WS_Q_BYTES, &map_q, q_full(qs), h * AT_D, row0 + qt * AT_QROWS);
        }
      }
      if (!ok) {                      // copies already issued still land: give them a bounded time before the CTA leaves
        unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 1000000ull) {}
      }
    }
  } else if (warp == LOADER + 1) {
    // ------------------------------- S = Q K^T issuer ---------------------------
    if (lane == 0) {
      const uint32_t idesc_s = make_idesc_mn(AT_QROWS, tpad, false, false);
      int i = 0, n = 0;
      bool ok = true;
      for (int bh = blockIdx.x; bh < pairs && ok; bh += gridDim.x, ++n) {
        int ks = n % kvslots;
        for (int qt = 0; qt < nqt; ++qt, ++i) {
          int qs = i % WS_QSLOTS, buf = i % NBUF;
          if (qt == 0 && !mbar_wait(kv_full(ks), (n / kvslots) & 1, abortp)) { ok = false; break; }
          if (!mbar_wait(q_full(qs), (i / WS_QSLOTS) & 1, abortp)) { ok = false; break; }
          if (!mbar_wait(t_empty(buf), ((i / NBUF) & 1) ^ 1u, abortp)) { ok = false; break; }
          tc_fence_after();
          uint32_t sq = sQ + qs * WS_Q_BYTES, sK = sKV + ks * 2 * kv_bytes;
#pragma unroll
          for (int k = 0; k < AT_D / 16; ++k)
            umma_bf16(tmem + buf * BUF_COLS, make_desc(sq + k * 32, 16, 1024), make_desc(sK + k * 32, 16, 1024), idesc_s, k > 0 ? 1u : 0u);
          umma_commit(s_full(buf));
          umma_commit(q_empty(qs));
        }
      }
    }
  } else if (warp == LOADER + 2) {
    // ------------------------------- O = P V issuer -----------------------------
    if (lane == 0) {
      const uint32_t idesc_o = make_idesc_mn(AT_QROWS, AT_D, false, true);
      const int ksteps = tpad / 16;
      const int chs2 = ((((T + 31) >> 5) + 1) >> 1) * 2;       // first 16-key step of the second half's probabilities
      int i = 0, n = 0;
      bool ok = true;
      for (int bh = blockIdx.x; bh < pairs && ok; bh += gridDim.x, ++n) {
        int ks = n % kvslots;
        for (int qt = 0; qt < nqt; ++qt, ++i) {
          int pb = i % NBUF;
          if (!mbar_wait(p_full(pb), (i / NBUF) & 1, abortp)) { ok = false; break; }
          tc_fence_after();
          uint32_t tb = tmem + pb * BUF_COLS;
          uint32_t sV = sKV + ks * 2 * kv_bytes + kv_bytes;
          for (int k = 0; k < ksteps; ++k)
            umma_bf16_ts(tb + O_COL, tb + 8 * k + ((GW == 8 && k >= chs2) ? 8 * chs2 : 0), make_desc(sV + k * (16 * 128), 8192, 1024),
                         idesc_o, k > 0 ? 1u : 0u);
          umma_commit(o_full(pb));
          umma_commit(kv_empty(ks));
        }
      }
    }
  } else {
    // ------------------------------- softmax groups -----------------------------
    const int g = warp / GW, gw = warp % GW;
    const int quarter = gw & 3, half = gw >> 2;            // half: which part of the keys / output columns (eight-warp groups)
    const bool leader = (gw == 0 && lane == 0);
    const int row = quarter * 32 + lane;
    const float c = 0.125f * 1.4426950408889634f;          // 1/sqrt(64) * log2(e)
    const uint32_t tbuf = tmem + g * BUF_COLS;
    const uint32_t trow = tbuf + ((uint32_t)(quarter * 32) << 16);
    const int nchunk = (T + 31) >> 5;
    const int ch0 = (GW == 8 && half == 1) ? (nchunk + 1) >> 1 : 0;
    const int ch1 = (GW == 8 && half == 0) ? (nchunk + 1) >> 1 : nchunk;
    // An eight-warp group writes the second half's probabilities over the S columns that half itself has consumed
    // (the first half may still be reading its own): chunk ch >= chs lands 16 * chs columns further right.
    const int chs = (nchunk + 1) >> 1;
    const uint32_t p_shift = (GW == 8 && half == 1) ? 16u * chs : 0u;
    float* cbuf = cls_buf + g * AT_MAXKEYS;
    float* rmax = red + g * 4 * AT_QROWS;                  // [2][128]
    float* rsum = rmax + 2 * AT_QROWS;                     // [2][128]
    bool ok = true;
    // tile i of this CTA: pair n = i / nqt (bh = blockIdx.x + n * gridDim.x), query tile qt = i % nqt
    const int my_pairs = blockIdx.x < pairs ? (pairs - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int items = my_pairs * nqt;
    int use = 0;
    for (int i = g; i < items; i += NBUF, ++use) {
      const int n = i / nqt, qt = i - n * nqt;
      const int bh = blockIdx.x + n * gridDim.x;
      const int b = bh / H, h = bh - b * H;
      const uint32_t par = use & 1;
      const int q0 = qt * AT_QROWS;
      const bool live = q0 + quarter * 32 < T;           // warp-uniform: a quarter whose rows all lie past T does no work
      ok = mbar_wait_q(s_full(g), par, abortp) && ok;
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      float mx = -INFINITY, sum = 0.f;
      const bool cls_row = (q0 == 0 && row == 0 && cls_prob != nullptr);
      if (live) {
        for (int ch = ch0; ch < ch1; ++ch) {
          uint32_t r[32];
          tmem_ld32(trow + ch * 32, r);
          tmem_ld_wait();
          if (ch * 32 + 32 <= T) {
#pragma unroll
            for (int j = 0; j < 32; j += 2) mx = fmax3(mx, __uint_as_float(r[j]), __uint_as_float(r[j + 1]));
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j)
              if (ch * 32 + j < T) mx = fmaxf(mx, __uint_as_float(r[j]));
          }
        }
      }
      if (GW == 8) {
        rmax[half * AT_QROWS + row] = mx;
        group_sync(1 + g, GT);
        mx = fmaxf(rmax[row], rmax[AT_QROWS + row]);
      }
      // With two groups the exponentials of successive tiles take turns (the special-function unit is shared), so
      // that one group's exponentials overlap the other's tensor-core and load/store phases instead of colliding
      // with its exponentials.  Three or four groups drift apart by themselves.
      if (NBUF == 2 && i > 0) {
        ok = mbar_wait_q(token(g), (g == 0 ? use - 1 : use) & 1, abortp) && ok;
        ok = __all_sync(0xffffffffu, ok);
      }
      if (live) {
        const float mc = mx * c;
        for (int ch = ch0; ch < ch1; ++ch) {
          uint32_t r[32];
          tmem_ld32(trow + ch * 32, r);
          tmem_ld_wait();
          float p[32];
          if (ch * 32 + 32 <= T) {
#pragma unroll
            for (int j = 0; j < 32; ++j) p[j] = ex2_fast(fmaf(__uint_as_float(r[j]), c, -mc));
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) p[j] = (ch * 32 + j < T) ? ex2_fast(fmaf(__uint_as_float(r[j]), c, -mc)) : 0.f;
          }
          float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
          for (int j = 0; j < 32; j += 4) { s0 += p[j]; s1 += p[j + 1]; s2 += p[j + 2]; s3 += p[j + 3]; }
          sum += (s0 + s1) + (s2 + s3);
          if (cls_row) {
#pragma unroll
            for (int j = 0; j < 32; ++j) cbuf[ch * 32 + j] = p[j];
          }
          uint32_t pk[16];
#pragma unroll
          for (int j = 0; j < 16; ++j) pk[j] = pack_bf16x2(p[2 * j], p[2 * j + 1]);
          tmem_st16(trow + ch * 16 + p_shift, pk);
        }
        tmem_st_wait();
      }
      if (GW == 8) rsum[half * AT_QROWS + row] = sum;
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full(g));             // P of this warp's rows and keys is in tensor memory
      if (GW == 8) group_sync(1 + g, GT);                // partial sums and the classification row are in shared memory
      else __syncwarp();
      if (NBUF == 2 && leader) mbar_arrive(token((g + 1) % NBUF));
      if (GW == 8) sum = rsum[row] + rsum[AT_QROWS + row];
      const float inv = 1.0f / sum;
      const int q = q0 + row;
      if (live && q < T && half == 0 && lse != nullptr) lse[((size_t)b * H + h) * T + q] = mx * 0.125f + logf(sum);
      if (q0 == 0 && gw == 0 && cls_prob != nullptr) {        // this warp holds query 0 in lane 0
        float s_inv = __shfl_sync(0xffffffffu, inv, 0);
        float* cp = cls_prob + ((size_t)b * H + h) * (T - 1);
        for (int j = 1 + lane; j < T; j += 32) cp[j - 1] = cbuf[j] * s_inv;
      }
      ok = mbar_wait_q(o_full(g), par, abortp) && ok;
      ok = __all_sync(0xffffffffu, ok);
      tc_fence_after();
      constexpr int NH = GW == 8 ? 1 : 2;                // 32-column halves of O this thread reads
      if (live) {
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) {
          uint32_t ro[32];
          tmem_ld32(trow + O_COL + (half + hh) * 32, ro);
          tmem_ld_wait();
          if (q < T && ok) {
            bf16* orow = out + ((size_t)b * T + q) * H * AT_D + (size_t)h * AT_D + (half + hh) * 32;
#pragma unroll
            for (int gq = 0; gq < 4; ++gq) {
              float v[8];
#pragma unroll
              for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(ro[gq * 8 + j]) * inv;
              store16(orow + gq * 8, v);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(t_empty(g));            // O has been read: the buffer may take the next S
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == LOADER) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && abort_flag && status != nullptr) atomicOr(status, STATUS_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------
// Forward for longer sequences (T > 256): the keys are walked once in blocks of AT_LONG_KB.  Per block S = Q K^T
// goes into tensor memory, each thread reads its row, forms P = exp(S - m) against the row's reference maximum m,
// sums P as it goes and hands P (bf16, through shared memory) to the second product, which adds P V into a separate
// set of tensor-memory columns; the output is divided by the sum at the end.  m follows the running maximum only in
// jumps of more than AT_LONG_SLACK binary orders, at which the accumulator is rescaled in place (rare after the first
// block), so that almost every block costs one product, one exponential per score and one more product.  The
// classification row's probabilities are written out block by block against the m of the moment and brought onto the
// final scale by its warp at the end.  One CTA per (image, head, 128 queries), one block in flight, several CTAs per SM.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
attn_fwd_tc_long_kernel(const __grid_constant__ CUtensorMap map_qkv, bf16* __restrict__ out, float* __restrict__ lse,
                        float* __restrict__ cls_prob, int B, int T, int H, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  constexpr int KB = AT_LONG_KB;                         // keys per block
  constexpr uint32_t KV_BYTES = KB * 128;                // 16 KB
  uint32_t sQ = base, sK = sQ + 2 * AT_BOX_BYTES, sV = sK + KV_BYTES, sP = sV + KV_BYTES;
  uint32_t bars = sP + (KB / 64) * (AT_QROWS * 128);
  unsigned char* pP = base_ptr + (sP - base);
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  int tid = threadIdx.x, warp = tid >> 5;
  int bh = blockIdx.y, b = bh / H, h = bh % H;
  int q0 = blockIdx.x * AT_QROWS;
  uint32_t tma_bar = bars, mma_bar = bars + 8;
  if (tid == 0) {
    abort_flag = 0;
    mbar_init(tma_bar, 1);
    mbar_init(mma_bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&tmem_slot), 2 * KB);           // S in the first KB columns, O behind it: several CTAs share an SM
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem = tmem_slot;
  constexpr uint32_t C_O = KB;
  volatile int* abortp = &abort_flag;
  const float c = 0.125f * 1.4426950408889634f;
  uint32_t trow = tmem + ((uint32_t)(warp * 32) << 16);
  int nblk = (T + KB - 1) / KB;
  int row0 = b * T;
  uint32_t tma_phase = 0, mma_phase = 0;
  bool ok = true;
  float mx = -INFINITY, sum = 0.f;
  bool cls_row = (q0 == 0 && tid == 0 && cls_prob != nullptr);
  bool cls_warp = (q0 == 0 && warp == 0 && cls_prob != nullptr);
  __shared__ float cls_m[AT_LONG_MAXBLK];               // reference maximum of the classification row, block by block

  for (int kb = 0; kb < nblk && ok; ++kb) {
    int k0 = kb * KB;
    int keys = min(KB, T - k0);
    int kpad = (keys + 15) & ~15;
    int nbox = (kpad + AT_BOX - 1) / AT_BOX;
    if (tid == 0) {
      int boxes = 2 * nbox + (kb == 0 ? 2 : 0);
      mbar_expect_tx(tma_bar, boxes * AT_BOX_BYTES);
      if (kb == 0)
        for (int j = 0; j < 2; ++j) tma_load_2d(sQ + j * AT_BOX_BYTES, &map_qkv, tma_bar, h * AT_D, row0 + q0 + j * AT_BOX);
      for (int j = 0; j < nbox; ++j) {
        tma_load_2d(sK + j * AT_BOX_BYTES, &map_qkv, tma_bar, (H + h) * AT_D, row0 + k0 + j * AT_BOX);
        tma_load_2d(sV + j * AT_BOX_BYTES, &map_qkv, tma_bar, (2 * H + h) * AT_D, row0 + k0 + j * AT_BOX);
      }
      ok = mbar_wait(tma_bar, tma_phase, abortp);
      if (ok) {
        tc_fence_after();
        uint32_t idesc = make_idesc_mn(AT_QROWS, kpad, false, false);
#pragma unroll
        for (int k = 0; k < AT_D / 16; ++k)
          umma_bf16(tmem, make_desc(sQ + k * 32, 16, 1024), make_desc(sK + k * 32, 16, 1024), idesc, k > 0 ? 1u : 0u);
        umma_commit(mma_bar);
      }
    }
    tma_phase ^= 1u;
    ok = mbar_wait(mma_bar, mma_phase, abortp);
    mma_phase ^= 1u;
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    if (!ok) break;
    // the block's maximum of this thread's query row (the scores are read again below: cheaper than holding them)
    float bm = -INFINITY;
#pragma unroll
    for (int ch = 0; ch < KB / 32; ++ch) {
      uint32_t r[32];
      tmem_ld32(trow + ch * 32, r);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (ch * 32 + j < keys) bm = fmaxf(bm, __uint_as_float(r[j]));
    }
    // The reference maximum of a row moves only when the block's maximum exceeds it by more than AT_LONG_SLACK in the
    // exponent (the probabilities then stay below 2^AT_LONG_SLACK, harmless in bf16 and in the fp32 sum); when it
    // moves, the accumulated output and sum of that row are scaled down.  The decision is taken per warp, because the
    // accumulator is read and written with warp-wide instructions; rows that do not move scale by one.
    if (kb == 0) {
      mx = bm;
    } else {
      bool grow = (bm - mx) * c > AT_LONG_SLACK;
      if (__any_sync(0xffffffffu, grow)) {
        float nm = grow ? bm : mx;
        float f = ex2_fast((mx - nm) * c);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          uint32_t r[32];
          tmem_ld32(trow + C_O + half * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * f);
          tmem_st16(trow + C_O + half * 32, r);
          tmem_st16(trow + C_O + half * 32 + 16, r + 16);
        }
        tmem_st_wait();
        sum *= f;
        mx = nm;
      }
    }
    if (cls_row) cls_m[kb] = mx;
    float mc = mx * c;
#pragma unroll
    for (int ch = 0; ch < KB / 32; ++ch) {
      uint32_t r[32];
      tmem_ld32(trow + ch * 32, r);
      tmem_ld_wait();
      float p[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        float e = ex2_fast(fmaf(__uint_as_float(r[j]), c, -mc));
        p[j] = (ch * 32 + j < keys) ? e : 0.f;
        sum += p[j];
      }
      if (cls_row) {                  // relative to this block's reference maximum; put on the final scale below
        float* cp = cls_prob + ((size_t)b * H + h) * (T - 1);
        for (int j = 0; j < 32; ++j) {
          int key = k0 + ch * 32 + j;
          if (key >= 1 && key < T) cp[key - 1] = p[j];
        }
      }
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        int key8 = ch * 4 + g;
        if (key8 * 8 < nbox * AT_BOX) {
          uint4 v;
          __nv_bfloat162* hh = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
          for (int i = 0; i < 4; ++i) hh[i] = __floats2bfloat162_rn(p[g * 8 + 2 * i], p[g * 8 + 2 * i + 1]);
          *reinterpret_cast<uint4*>(pP + p_offset(tid, key8)) = v;
        }
      }
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (tid == 0) {
      uint32_t idesc = make_idesc_mn(AT_QROWS, AT_D, false, true);
      for (int k = 0; k < kpad / 16; ++k)
        umma_bf16(tmem + C_O, make_desc(sP + (k >> 2) * (AT_QROWS * 128) + (k & 3) * 32, 16, 1024),
                  make_desc(sV + k * (16 * 128), 8192, 1024), idesc, (kb > 0 || k > 0) ? 1u : 0u);
      umma_commit(mma_bar);
    }
    ok = mbar_wait(mma_bar, mma_phase, abortp);      // P, K and V of this block are free again; O is complete
    mma_phase ^= 1u;
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
  }
  if (ok && cls_warp) {
    // the classification row's probabilities: from each block's reference maximum to the final one, over the row sum
    float fm = __shfl_sync(0xffffffffu, mx, 0), fs = __shfl_sync(0xffffffffu, sum, 0);
    float inv0 = 1.0f / fs;
    __syncwarp();
    float* cp = cls_prob + ((size_t)b * H + h) * (T - 1);
    for (int key = 1 + (tid & 31); key < T; key += 32)
      cp[key - 1] *= ex2_fast((cls_m[key / KB] - fm) * c) * inv0;
  }
  int q = q0 + tid;
  if (ok) {
    float inv = 1.0f / sum;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t r[32];
      tmem_ld32(trow + C_O + half * 32, r);
      tmem_ld_wait();
      if (q < T) {
        bf16* orow = out + ((size_t)b * T + q) * H * AT_D + (size_t)h * AT_D + half * 32;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
          float v[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(r[g * 8 + j]) * inv;
          store16(orow + g * 8, v);
        }
      }
    }
    if (q < T && lse != nullptr) lse[((size_t)b * H + h) * T + q] = mx * 0.125f + logf(sum);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 2 * AT_LONG_KB);
  }
  if (tid == 0 && abort_flag && status != nullptr) atomicOr(status, STATUS_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------
// Backward (T <= 128): one CTA of 128 threads per (image, head).  With P = exp(S - lse):
//   dP = dO V^T;  delta_i = sum_j P_ij dP_ij;  dS = P * (dP - delta) / sqrt(d)
//   dQ = dS K;  dK = dS^T Q;  dV = P^T dO                      (chain rule through Eq. 1, cf. Eq. 3)
// S and dP are two MMA groups into tensor memory; each thread owns one query row and writes P and dS as
// bf16 operand tiles into shared memory; the three products then read those tiles K-major (dQ) or through
// transposing descriptors (dK, dV), so nothing is transposed by hand.  A gradient arriving at the head-mean
// score of token j (cls_extra[b, j-1], from the fused token) is added to dP of the classification row.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256, 2)
attn_bwd_tc_kernel(const __grid_constant__ CUtensorMap map_qkv, const __grid_constant__ CUtensorMap map_do,
                   const float* __restrict__ lse, const float* __restrict__ cls_extra, bf16* __restrict__ dqkv,
                   int B, int T, int H, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  constexpr uint32_t TILE = 2 * AT_BOX_BYTES;            // 128 rows x 128 bytes
  int tpad = (T + 15) & ~15;
  // P and dS hold tpad query rows per 64-key chunk; dS starts in V's space (V is dead once dP = dO V^T is done).
  uint32_t CH = (uint32_t)tpad * 128u;
  uint32_t sQ = base, sK = sQ + TILE, sG = sK + TILE, sV = sG + TILE, sS = sV;
  uint32_t sP = sV + (2 * CH > TILE ? 2 * CH : TILE);
  uint32_t red_off = sP + 2 * CH + (3 * CH < 16384u ? 16384u - 3 * CH : 0u);   // slack: MMA row extent past tpad stays in bounds
  float* red = reinterpret_cast<float*>(base_ptr + (red_off - base));        // [2][128]: the halves' shares of delta
  float* exs = red + 2 * AT_QROWS;                                             // [128]: classification-row score gradients / H
  uint32_t bars = red_off + 3 * AT_QROWS * 4;
  unsigned char* pP = base_ptr + (sP - base);
  unsigned char* pS = base_ptr + (sS - base);
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  // 256 threads: warps w and w + 4 share the TMEM lane quarter w & 3 (query rows 32 * (w & 3) ..) and split the
  // keys (chunks 0-1 and 2-3 of 32) and later the output columns between them.
  int tid = threadIdx.x, warp = tid >> 5;
  int row = tid & 127, half = tid >> 7;
  int bh = blockIdx.x, b = bh / H, h = bh % H;
  uint32_t tma_bar = bars, mma_bar = bars + 8, mma2_bar = bars + 16;
  if (tid == 0) {
    abort_flag = 0;
    mbar_init(tma_bar, 1);
    mbar_init(mma_bar, 1);
    mbar_init(mma2_bar, 3);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&tmem_slot), 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem = tmem_slot;
  // dQ, dK, dV reuse the columns of S and dP, which are dead once P and dS sit in shared memory
  constexpr uint32_t C_S = 0, C_DP = 128, C_DQ = 0, C_DK = 64, C_DV = 128;
  volatile int* abortp = &abort_flag;
  bool ok = true;
  if (tid == 0) {
    mbar_expect_tx(tma_bar, 4 * TILE);
    int row0 = b * T;
    for (int j = 0; j < 2; ++j) {
      tma_load_2d(sQ + j * AT_BOX_BYTES, &map_qkv, tma_bar, h * AT_D, row0 + j * AT_BOX);
      tma_load_2d(sK + j * AT_BOX_BYTES, &map_qkv, tma_bar, (H + h) * AT_D, row0 + j * AT_BOX);
      tma_load_2d(sV + j * AT_BOX_BYTES, &map_qkv, tma_bar, (2 * H + h) * AT_D, row0 + j * AT_BOX);
      tma_load_2d(sG + j * AT_BOX_BYTES, &map_do, tma_bar, h * AT_D, row0 + j * AT_BOX);
    }
  }
  // inputs that do not come through TMA are fetched while the tiles are on their way
  const bool valid_row = row < T;
  const float l2 = valid_row ? lse[((size_t)b * H + h) * T + row] * 1.4426950408889634f : 0.f;
  const bool has_extra = cls_extra != nullptr;
  if (half == 0) exs[row] = (has_extra && row >= 1 && row < T) ? cls_extra[(size_t)b * (T - 1) + row - 1] * (1.0f / (float)H) : 0.f;
  __syncthreads();
  if (tid == 0) {
    ok = mbar_wait(tma_bar, 0, abortp);
    if (ok) {
      tc_fence_after();
      uint32_t idesc = make_idesc_mn(AT_QROWS, tpad, false, false);
#pragma unroll
      for (int k = 0; k < AT_D / 16; ++k)
        umma_bf16(tmem + C_S, make_desc(sQ + k * 32, 16, 1024), make_desc(sK + k * 32, 16, 1024), idesc, k > 0 ? 1u : 0u);
#pragma unroll
      for (int k = 0; k < AT_D / 16; ++k)
        umma_bf16(tmem + C_DP, make_desc(sG + k * 32, 16, 1024), make_desc(sV + k * 32, 16, 1024), idesc, k > 0 ? 1u : 0u);
      umma_commit(mma_bar);
    }
  }
  ok = mbar_wait(mma_bar, 0, abortp);
  ok = __all_sync(0xffffffffu, ok);
  tc_fence_after();

  const float c = 0.125f * 1.4426950408889634f;
  uint32_t trow = tmem + ((uint32_t)((warp & 3) * 32) << 16);
  const bool extra_row = (row == 0 && has_extra);
  float delta = 0.f;
  // tcgen05.ld is warp-collective: every lane issues it, rows past T only skip the arithmetic.  Keys are taken 16 at
  // a time (two loads of 16 columns) to keep the live registers of a step few.
  if (ok) {
    for (int kk = 4 * half; kk < 4 * half + 4 && kk * 16 < T; ++kk) {
      uint32_t rs[16], rp[16];
      tmem_ld16(trow + C_S + kk * 16, rs);
      tmem_ld16(trow + C_DP + kk * 16, rp);
      tmem_ld_wait();
      if (valid_row) {
        float d0 = 0.f, d1 = 0.f;
#pragma unroll
        for (int j = 0; j < 16; j += 2) {
          int key = kk * 16 + j;
          float p0 = key < T ? ex2_fast(fmaf(__uint_as_float(rs[j]), c, -l2)) : 0.f;
          float p1 = key + 1 < T ? ex2_fast(fmaf(__uint_as_float(rs[j + 1]), c, -l2)) : 0.f;
          float e0 = __uint_as_float(rp[j]), e1 = __uint_as_float(rp[j + 1]);
          if (extra_row) { e0 += exs[key]; e1 += exs[key + 1]; }
          d0 = fmaf(p0, e0, d0);
          d1 = fmaf(p1, e1, d1);
        }
        delta += d0 + d1;
      }
    }
  }
  red[half * AT_QROWS + row] = delta;          // every thread reaches this barrier, whatever the waits returned
  __syncthreads();
  delta = red[row] + red[AT_QROWS + row];
  if (ok) {
    for (int kk = 4 * half; kk < 4 * half + 4; ++kk) {
      float p[16], ds[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) { p[j] = 0.f; ds[j] = 0.f; }
      if (kk * 16 < T) {
        uint32_t rs[16], rp[16];
        tmem_ld16(trow + C_S + kk * 16, rs);
        tmem_ld16(trow + C_DP + kk * 16, rp);
        tmem_ld_wait();
        if (valid_row) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            int key = kk * 16 + j;
            float pv = key < T ? ex2_fast(fmaf(__uint_as_float(rs[j]), c, -l2)) : 0.f;
            float dp = __uint_as_float(rp[j]);
            if (extra_row) dp += exs[key];
            p[j] = pv;
            ds[j] = pv * (dp - delta) * 0.125f;
          }
        }
      }
#pragma unroll
      for (int g = 0; g < 2; ++g) {
        uint4 vp, vs;
        __nv_bfloat162* hp = reinterpret_cast<__nv_bfloat162*>(&vp);
        __nv_bfloat162* hs = reinterpret_cast<__nv_bfloat162*>(&vs);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          hp[i] = __floats2bfloat162_rn(p[g * 8 + 2 * i], p[g * 8 + 2 * i + 1]);
          hs[i] = __floats2bfloat162_rn(ds[g * 8 + 2 * i], ds[g * 8 + 2 * i + 1]);
        }
        if (row < tpad) {
          int key8 = kk * 2 + g;
          uint32_t off = (uint32_t)(key8 >> 3) * CH + (uint32_t)row * 128u + (uint32_t)(((key8 & 7) ^ (row & 7)) << 4);
          *reinterpret_cast<uint4*>(pP + off) = vp;
          *reinterpret_cast<uint4*>(pS + off) = vs;
        }
      }
    }
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  ok = ok && !abort_flag;
  // dQ, dK and dV are issued by three different threads (lane 0 of warps 0, 1, 2), each committing to the same barrier
  if (ok && (tid & 31) == 0 && warp < 3) {
    if (warp == 0) {
      // dQ = dS K: A = dS (contiguous along keys), B = K read with keys as the reduction index
      uint32_t id_q = make_idesc_mn(AT_QROWS, AT_D, false, true);
      for (int k = 0; k < tpad / 16; ++k)
        umma_bf16(tmem + C_DQ, make_desc(sS + (k >> 2) * CH + (k & 3) * 32, 16, 1024), make_desc(sK + k * 2048, 8192, 1024), id_q,
                  k > 0 ? 1u : 0u);
    } else {
      // dK = dS^T Q and dV = P^T dO: both operands read with queries as the reduction index
      uint32_t id_t = make_idesc_mn(AT_QROWS, AT_D, true, true);
      uint32_t sa = warp == 1 ? sS : sP, sb = warp == 1 ? sQ : sG, cd = warp == 1 ? C_DK : C_DV;
      for (int k = 0; k < tpad / 16; ++k)
        umma_bf16(tmem + cd, make_desc(sa + k * 2048, CH, 1024), make_desc(sb + k * 2048, 8192, 1024), id_t, k > 0 ? 1u : 0u);
    }
    umma_commit(mma2_bar);
  }
  if (ok) ok = mbar_wait(mma2_bar, 0, abortp);
  ok = __all_sync(0xffffffffu, ok);
  tc_fence_after();
  if (ok) {
    const uint32_t cols[3] = {C_DQ, C_DK, C_DV};
#pragma unroll
    for (int which = 0; which < 3; ++which) {
      {
        uint32_t r[32];
        tmem_ld32(trow + cols[which] + half * 32, r);
        tmem_ld_wait();
        if (valid_row) {
          bf16* drow = dqkv + (((size_t)b * T + row) * 3 + which) * H * AT_D + (size_t)h * AT_D + half * 32;
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(r[g * 8 + j]);
            store16(drow + g * 8, v);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
  if (tid == 0 && abort_flag && status != nullptr) atomicOr(status, STATUS_TIMEOUT);
}

// ------------------------------------------------------------------------------------------------
// Backward for 128 < T <= 256: one CTA of 256 threads per (image, head), queries and keys in two tiles of 128.
// The formulas are those of the kernel above; what changes is that delta_i = sum_j P_ij dP_ij runs over both key
// tiles, so a first sweep (one step per query tile, both key tiles at once) forms S and dP only to accumulate delta, and a
// second sweep (key tile outer, query tile inner) forms them again, writes P and dS as bf16 operand tiles and issues
// the three products: dQ_i accumulates over the key tiles, dK_j and dV_j over the query tiles, all in tensor memory
// (S 128 + dP 128 + dQ 2 x 64 + dK 64 + dV 64 = 512 columns: one CTA per SM).  No step leaves the loop early: after a
// wait that expired the remaining steps only keep the barriers in step.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256, 1)
attn_bwd_tc256_kernel(const __grid_constant__ CUtensorMap map_qkv, const __grid_constant__ CUtensorMap map_do,
                      const float* __restrict__ lse, const float* __restrict__ cls_extra, bf16* __restrict__ dqkv,
                      int B, int T, int H, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  constexpr uint32_t TILE = 2 * AT_BOX_BYTES;            // 128 rows x 128 bytes
  constexpr uint32_t CH = TILE;                          // one 64-key chunk of a P / dS tile: 128 query rows x 128 bytes
  uint32_t sQ = base, sK = sQ + 2 * TILE, sG = sK + 2 * TILE, sV = sG + 2 * TILE, sP = sV + 2 * TILE, sS = sP + 2 * TILE;
  uint32_t arrays = sS + 2 * TILE;
  float* sdelta = reinterpret_cast<float*>(base_ptr + (arrays - base));     // [256] delta of every query row
  float* sl2 = sdelta + 256;                                                 // [256] log-sum-exp in binary orders
  float* exs = sl2 + 256;                                                    // [256] classification-row score gradients / H
  float* red = exs + 256;                                                    // [2][128] the halves' shares of delta
  uint32_t bars = arrays + 4 * 256 * 4;
  unsigned char* pP = base_ptr + (sP - base);
  unsigned char* pS = base_ptr + (sS - base);
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  int tid = threadIdx.x, warp = tid >> 5;
  int rowl = tid & 127, half = tid >> 7;
  int bh = blockIdx.x, b = bh / H, h = bh % H;
  uint32_t tma_bar = bars, mma_bar = bars + 8, mma2_bar = bars + 16;
  if (tid == 0) {
    abort_flag = 0;
    mbar_init(tma_bar, 1);
    mbar_init(mma_bar, 1);
    mbar_init(mma2_bar, 3);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(&tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem = tmem_slot;
  constexpr uint32_t C_S = 0, C_DP = 128, C_DQ = 256, C_DK = 384, C_DV = 448;
  volatile int* abortp = &abort_flag;
  const int tpad = (T + 15) & ~15;
  const int row0 = b * T;
  if (tid == 0) {
    mbar_expect_tx(tma_bar, 8 * TILE);
    for (int j = 0; j < 4; ++j) {                        // rows past the image: the next image's, or zero fill; never used
      tma_load_2d(sQ + j * AT_BOX_BYTES, &map_qkv, tma_bar, h * AT_D, row0 + j * AT_BOX);
      tma_load_2d(sK + j * AT_BOX_BYTES, &map_qkv, tma_bar, (H + h) * AT_D, row0 + j * AT_BOX);
      tma_load_2d(sV + j * AT_BOX_BYTES, &map_qkv, tma_bar, (2 * H + h) * AT_D, row0 + j * AT_BOX);
      tma_load_2d(sG + j * AT_BOX_BYTES, &map_do, tma_bar, h * AT_D, row0 + j * AT_BOX);
    }
  }
  const bool has_extra = cls_extra != nullptr;
  sl2[tid] = tid < T ? lse[((size_t)b * H + h) * T + tid] * 1.4426950408889634f : 0.f;
  exs[tid] = (has_extra && tid >= 1 && tid < T) ? cls_extra[(size_t)b * (T - 1) + tid - 1] * (1.0f / (float)H) : 0.f;
  __syncthreads();
  bool ok = true;
  if (tid == 0) ok = mbar_wait(tma_bar, 0, abortp);
  const float c = 0.125f * 1.4426950408889634f;
  const uint32_t trow = tmem + ((uint32_t)((warp & 3) * 32) << 16);
  uint32_t ph1 = 0, ph2 = 0;

  // S = Q_i K_j^T and dP = dO_i V_j^T into tensor memory; everyone waits for them
  auto scores = [&](int i, int j) {
    tc_fence_before();
    __syncthreads();                       // the previous step's reads of S / dP (and of the operand tiles) are over
    tc_fence_after();
    if (tid == 0 && ok && !abort_flag) {
      int kpad = min(128, tpad - 128 * j);
      uint32_t idesc = make_idesc_mn(AT_QROWS, kpad, false, false);
      uint32_t q = sQ + i * TILE, k_ = sK + j * TILE, g = sG + i * TILE, v = sV + j * TILE;
#pragma unroll
      for (int k = 0; k < AT_D / 16; ++k)
        umma_bf16(tmem + C_S, make_desc(q + k * 32, 16, 1024), make_desc(k_ + k * 32, 16, 1024), idesc, k > 0 ? 1u : 0u);
#pragma unroll
      for (int k = 0; k < AT_D / 16; ++k)
        umma_bf16(tmem + C_DP, make_desc(g + k * 32, 16, 1024), make_desc(v + k * 32, 16, 1024), idesc, k > 0 ? 1u : 0u);
      umma_commit(mma_bar);
    }
    bool w = mbar_wait(mma_bar, ph1, abortp);
    ph1 ^= 1u;
    ok = __all_sync(0xffffffffu, ok && w);
    tc_fence_after();
  };

  // S and dP of query tile i against BOTH key tiles at once: the second pair lands in the columns that hold dQ, dK, dV
  // later (free during the first sweep), so the sweep takes one product group and one wait per query tile
  auto scores_both = [&](int i) {
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (tid == 0 && ok && !abort_flag) {
      uint32_t q = sQ + i * TILE, g = sG + i * TILE;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        int kpad = min(128, tpad - 128 * j);
        uint32_t idesc = make_idesc_mn(AT_QROWS, kpad, false, false);
        uint32_t k_ = sK + j * TILE, v = sV + j * TILE;
#pragma unroll
        for (int k = 0; k < AT_D / 16; ++k)
          umma_bf16(tmem + 256 * j + C_S, make_desc(q + k * 32, 16, 1024), make_desc(k_ + k * 32, 16, 1024), idesc, k > 0 ? 1u : 0u);
#pragma unroll
        for (int k = 0; k < AT_D / 16; ++k)
          umma_bf16(tmem + 256 * j + C_DP, make_desc(g + k * 32, 16, 1024), make_desc(v + k * 32, 16, 1024), idesc, k > 0 ? 1u : 0u);
      }
      umma_commit(mma_bar);
    }
    bool w = mbar_wait(mma_bar, ph1, abortp);
    ph1 ^= 1u;
    ok = __all_sync(0xffffffffu, ok && w);
    tc_fence_after();
  };

  // ---- first sweep: delta of every query row ----
  for (int i = 0; i < 2; ++i) {
    const int row = i * 128 + rowl;
    const bool valid_row = row < T;
    const bool extra_row = (row == 0 && has_extra);
    const float l2 = sl2[row];
    float dacc = 0.f;
    scores_both(i);
    for (int j = 0; j < 2; ++j) {
      const int kbase = j * 128;
      const int kvalid = min(128, T - kbase);
      if (ok) {
        for (int kk = 4 * half; kk < 4 * half + 4 && kk * 16 < kvalid; ++kk) {
          uint32_t rs[16], rp[16];
          tmem_ld16(trow + 256 * j + C_S + kk * 16, rs);
          tmem_ld16(trow + 256 * j + C_DP + kk * 16, rp);
          tmem_ld_wait();
          if (valid_row) {
            float d0 = 0.f, d1 = 0.f;
#pragma unroll
            for (int jj = 0; jj < 16; jj += 2) {
              int key = kbase + kk * 16 + jj;
              float p0 = key < T ? ex2_fast(fmaf(__uint_as_float(rs[jj]), c, -l2)) : 0.f;
              float p1 = key + 1 < T ? ex2_fast(fmaf(__uint_as_float(rs[jj + 1]), c, -l2)) : 0.f;
              float e0 = __uint_as_float(rp[jj]), e1 = __uint_as_float(rp[jj + 1]);
              if (extra_row) { e0 += exs[key]; e1 += exs[key + 1]; }
              d0 = fmaf(p0, e0, d0);
              d1 = fmaf(p1, e1, d1);
            }
            dacc += d0 + d1;
          }
        }
      }
    }
    red[half * AT_QROWS + rowl] = dacc;
    __syncthreads();
    if (half == 0) sdelta[row] = red[rowl] + red[AT_QROWS + rowl];
  }

  // ---- second sweep: P and dS tiles, the three products ----
  auto store_rows = [&](uint32_t col, int which, int row) {      // 64 accumulator columns of `row` -> dqkv[.., which, h, :]
    uint32_t r[32];
    tmem_ld32(trow + col + half * 32, r);
    tmem_ld_wait();
    if (row < T) {
      bf16* drow = dqkv + (((size_t)b * T + row) * 3 + which) * H * AT_D + (size_t)h * AT_D + half * 32;
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        float v[8];
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) v[jj] = __uint_as_float(r[g * 8 + jj]);
        store16(drow + g * 8, v);
      }
    }
  };
  for (int j = 0; j < 2; ++j) {
    const int kbase = j * 128;
    const int kvalid = min(128, T - kbase);
    const int kpad = min(128, tpad - kbase);
    for (int i = 0; i < 2; ++i) {
      scores(i, j);                          // its leading barrier also orders the delta written above before its use
      const int row = i * 128 + rowl;
      const bool valid_row = row < T;
      const bool extra_row = (row == 0 && has_extra);
      const float l2 = sl2[row];
      const float delta = sdelta[row];
      const int qpad = min(128, tpad - 128 * i);
      if (ok) {
        for (int kk = 4 * half; kk < 4 * half + 4; ++kk) {
          float p[16], ds[16];
#pragma unroll
          for (int jj = 0; jj < 16; ++jj) { p[jj] = 0.f; ds[jj] = 0.f; }
          if (kk * 16 < kvalid) {
            uint32_t rs[16], rp[16];
            tmem_ld16(trow + C_S + kk * 16, rs);
            tmem_ld16(trow + C_DP + kk * 16, rp);
            tmem_ld_wait();
            if (valid_row) {
#pragma unroll
              for (int jj = 0; jj < 16; ++jj) {
                int key = kbase + kk * 16 + jj;
                float pv = key < T ? ex2_fast(fmaf(__uint_as_float(rs[jj]), c, -l2)) : 0.f;
                float dp = __uint_as_float(rp[jj]);
                if (extra_row) dp += exs[key];
                p[jj] = pv;
                ds[jj] = pv * (dp - delta) * 0.125f;
              }
            }
          }
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            uint4 vp, vs;
            __nv_bfloat162* hp = reinterpret_cast<__nv_bfloat162*>(&vp);
            __nv_bfloat162* hs = reinterpret_cast<__nv_bfloat162*>(&vs);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              hp[e] = __floats2bfloat162_rn(p[g * 8 + 2 * e], p[g * 8 + 2 * e + 1]);
              hs[e] = __floats2bfloat162_rn(ds[g * 8 + 2 * e], ds[g * 8 + 2 * e + 1]);
            }
            int key8 = kk * 2 + g;
            uint32_t off = (uint32_t)(key8 >> 3) * CH + (uint32_t)rowl * 128u + (uint32_t)(((key8 & 7) ^ (rowl & 7)) << 4);
            *reinterpret_cast<uint4*>(pP + off) = vp;
            *reinterpret_cast<uint4*>(pS + off) = vs;
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      tc_fence_after();
      // dQ_i, dK_j and dV_j are issued by lane 0 of warps 0, 1, 2, each committing to the same barrier
      if ((tid & 31) == 0 && warp < 3) {
        if (ok && !abort_flag) {
          if (warp == 0) {
            uint32_t id_q = make_idesc_mn(AT_QROWS, AT_D, false, true);
            for (int k = 0; k < kpad / 16; ++k)
              umma_bf16(tmem + C_DQ + 64 * i, make_desc(sS + (k >> 2) * CH + (k & 3) * 32, 16, 1024),
                        make_desc(sK + j * TILE + k * 2048, 8192, 1024), id_q, (j > 0 || k > 0) ? 1u : 0u);
          } else {
            uint32_t id_t = make_idesc_mn(AT_QROWS, AT_D, true, true);
            uint32_t sa = warp == 1 ? sS : sP, sb = (warp == 1 ? sQ : sG) + i * TILE, cd = warp == 1 ? C_DK : C_DV;
            for (int k = 0; k < qpad / 16; ++k)
              umma_bf16(tmem + cd, make_desc(sa + k * 2048, CH, 1024), make_desc(sb + k * 2048, 8192, 1024), id_t,
                        (i > 0 || k > 0) ? 1u : 0u);
          }
          umma_commit(mma2_bar);
        }
      }
      bool w = ok && mbar_wait(mma2_bar, ph2, abortp);   // the products are done: P, dS, S and dP may be overwritten
      ph2 ^= 1u;
      ok = __all_sync(0xffffffffu, w);
      tc_fence_after();
    }
    if (ok) {
      store_rows(C_DK, 1, kbase + rowl);
      store_rows(C_DV, 2, kbase + rowl);
    }
  }
  if (ok) {
    store_rows(C_DQ, 0, rowl);
    store_rows(C_DQ + 64, 0, 128 + rowl);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && abort_flag && status != nullptr) atomicOr(status, STATUS_TIMEOUT);
}

}  // namespace tc

// Returns 0 when the tensor-core kernel took the problem, non-zero when the caller must use another kernel.
int attention_fwd_tc(const Ctx& c, const void* qkv, void* out, float* lse, float* cls_prob, int B, int T, int H, int d) {
  using namespace tc;
  if (c.dtype != 1 || d != AT_D || T < 1 || T > AT_LONG_KB * AT_LONG_MAXBLK) return -1;
  if (((uintptr_t)qkv & 15) || ((uintptr_t)out & 15)) return -1;
  CUtensorMap map;
  if (!make_map(&map, qkv, (uint64_t)3 * H * d, (uint64_t)B * T, (uint64_t)3 * H * d, AT_BOX)) return -2;
  if (T > AT_MAXKEYS) {
    size_t smem_l = 1024 + 2 * (size_t)AT_BOX_BYTES + 2 * (size_t)AT_LONG_KB * 128 + (AT_LONG_KB / 64) * (size_t)(AT_QROWS * 128) + 64;
    static SmemLimit lim_l;
    if (!ensure_smem(lim_l, attn_fwd_tc_long_kernel, smem_l)) return -3;
    dim3 grid_l((T + AT_QROWS - 1) / AT_QROWS, B * H);
    note_launch(1);
    attn_fwd_tc_long_kernel<<<grid_l, 128, smem_l, c.stream>>>(map, (bf16*)out, lse, cls_prob, B, T, H, c.status);
    return 0;
  }
  int tpad = (T + 15) & ~15;
  CUtensorMap map_q, map_kv;
  if (!make_map(&map_q, qkv, (uint64_t)3 * H * d, (uint64_t)B * T, (uint64_t)3 * H * d, AT_QROWS)) return -2;
  if (!make_map(&map_kv, qkv, (uint64_t)3 * H * d, (uint64_t)B * T, (uint64_t)3 * H * d, tpad)) return -2;
  int nbuf = tpad <= 128 ? 4 : (tpad <= 160 ? 3 : 2);
  size_t fixed = 1024 + (size_t)WS_QSLOTS * WS_Q_BYTES + (WS_MAXBUF * AT_MAXKEYS + WS_MAXBUF * 4 * AT_QROWS) * 4 + 44 * 8 + 64;
  size_t slot = (size_t)2 * tpad * 128;
  int kvslots = (int)((227 * 1024 - fixed) / slot);
  if (kvslots > WS_MAXKV) kvslots = WS_MAXKV;
  if (kvslots < 2) return -1;
  size_t smem = fixed + kvslots * slot;
  int sms = c.sm_count > 0 ? c.sm_count : 148;
  int grid = B * H < sms ? B * H : sms;
  static SmemLimit lim[5];
  auto launch = [&](auto kern, int threads) -> int {
    if (!ensure_smem(lim[nbuf], kern, smem)) return -3;
    note_launch(1);
    kern<<<grid, threads, smem, c.stream>>>(map_q, map_kv, (bf16*)out, lse, cls_prob, B, T, H, kvslots, c.status);
    return 0;
  };
  if (nbuf == 4) return launch(attn_fwd_ws_kernel<4>, 19 * 32);
  if (nbuf == 3) return launch(attn_fwd_ws_kernel<3>, 15 * 32);
  return launch(attn_fwd_ws_kernel<2>, 19 * 32);
}

}  // namespace bsr

namespace bsr {

int attention_bwd_tc(const Ctx& c, const void* qkv, const void* dout, const float* lse, const float* cls_extra, void* dqkv,
                     int B, int T, int H, int d) {
  using namespace tc;
  if (c.dtype != 1 || d != AT_D || T > 2 * AT_QROWS || T < 1) return -1;
  if (((uintptr_t)qkv & 15) || ((uintptr_t)dout & 15) || ((uintptr_t)dqkv & 15)) return -1;
  CUtensorMap mq, mg;
  if (!make_map(&mq, qkv, (uint64_t)3 * H * d, (uint64_t)B * T, (uint64_t)3 * H * d, AT_BOX)) return -2;
  if (!make_map(&mg, dout, (uint64_t)H * d, (uint64_t)B * T, (uint64_t)H * d, AT_BOX)) return -2;
  if (T > AT_QROWS) {                      // two tiles of queries and keys
    size_t smem2 = 1024 + 12 * 2 * (size_t)AT_BOX_BYTES + 4 * 256 * 4 + 64;
    static SmemLimit lim2;
    if (!ensure_smem(lim2, attn_bwd_tc256_kernel, smem2)) return -3;
    note_launch(1);
    attn_bwd_tc256_kernel<<<B * H, 256, smem2, c.stream>>>(mq, mg, lse, cls_extra, (bf16*)dqkv, B, T, H, c.status);
    return 0;
  }
  size_t tile = 2 * (size_t)AT_BOX_BYTES, ch = (size_t)((T + 15) & ~15) * 128;
  size_t smem = 1024 + 3 * tile + (2 * ch > tile ? 2 * ch : tile) + 2 * ch + (3 * ch < 16384 ? 16384 - 3 * ch : 0) + 3 * AT_QROWS * 4 + 64;
  static SmemLimit lim;
  if (!ensure_smem(lim, attn_bwd_tc_kernel, smem)) return -3;
  note_launch(1);
  attn_bwd_tc_kernel<<<B * H, 256, smem, c.stream>>>(mq, mg, lse, cls_extra, (bf16*)dqkv, B, T, H, c.status);
  return 0;
}

}  // namespace bsr
