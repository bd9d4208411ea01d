// bf16 dense contraction on the 5th-generation tensor cores (sm_100a): TMA -> 128B-swizzled shared
// memory ring -> tcgen05.mma accumulating fp32 in tensor memory -> tcgen05.ld epilogue.
//
//   C[m, n] = epilogue( sum_k A(m, k) * B(n, k) )
//
// Each operand may be contiguous along k ("K-major", the forward layers: activations [m, k] and
// weights [n, k]) or along its own index ("MN-major": the weight in the input-gradient product
// dX = dY W, and both operands of the weight-gradient product dW = dY^T X, Eq. 2 and Eq. 4 of the
// paper).  No operand is transposed in memory; the shared-memory descriptors say how to read it.
//
// Kernel shape: persistent, one CTA per SM, 128 x 256 output tiles, k in slabs of 64.  Tiles are walked with the
// column index fastest, so that the CTAs running at one time share rows of A and find them in L2.
//   warp 0      : TMA producer (one lane)
//   warp 1      : tensor-memory allocation, MMA issue (one lane)
//   warps 2..9  : epilogue, two warps per TMEM lane quarter; chunks of 32 x 32 outputs go through a staging
//                 buffer so that global loads and stores are row-contiguous; two accumulator buffers of 256
//                 columns let the epilogue of one tile overlap the main loop of the next.
// Every wait is bounded: on expiry the CTA raises STATUS_TIMEOUT in the status word, gives the
// copies it issued time to land, frees its tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"
#include "tc_ptx.cuh"
#include "tc_epilogue.cuh"

namespace bsr {

namespace tc {

constexpr int BM = 128, BN_MAX = 256, BK = 64;       // tile width BN is 256, or 192 where that wastes less of the last wave
constexpr int STAGES = 4;
constexpr int UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2;
constexpr int STAGE_BYTES_MAX = A_BYTES + BN_MAX * BK * 2;
constexpr int EPI_WARPS = 8;                     // two warps per TMEM lane quarter, each takes half of the columns
constexpr int STAGING_BYTES = 32 * 128;          // per epilogue warp: 32 rows x 128 bytes, 16-byte units XOR-swizzled
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES_MAX + EPI_WARPS * STAGING_BYTES + 1024 /*alignment slack*/ + 128 /*barriers*/;
constexpr int THREADS = 64 + EPI_WARPS * 32;
constexpr uint32_t TMEM_COLS = 512;

// Instruction descriptor: D = f32, A = B = bf16, M = 128, N = bn, operand majors as given.
__host__ __device__ constexpr uint32_t make_idesc(bool a_mn, bool b_mn, int bn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

// One unit of work of the persistent loop, decoded identically by the three roles.
struct Work {
  int mt, nt, kb0, kb1, b_off, bias_off;
  size_t c_off;
  bool active;
};
__device__ __forceinline__ Work decode_work(int w, int tiles_m, int tiles_n, int total_kb, int kb_per_split, const GemmGroup& g,
                                            size_t mn) {
  Work k;
  k.nt = w % tiles_n;
  k.mt = (w / tiles_n) % tiles_m;
  int sp = w / (tiles_m * tiles_n);
  k.b_off = 0; k.bias_off = 0; k.active = true;
  if (g.mode == 0) {                       // plain (optionally split along k)
    k.kb0 = sp * kb_per_split;
    k.kb1 = min(total_kb, k.kb0 + kb_per_split);
    k.c_off = (size_t)sp * mn;
  } else if (g.mode == 1) {                // rows grouped by expert: the tile's expert picks the weight slice
    int e = g.tile_expert[k.mt];
    k.active = e >= 0;
    k.kb0 = 0; k.kb1 = total_kb;
    k.b_off = e * g.b_stride;
    k.bias_off = e * g.bias_stride;
    k.c_off = 0;
  } else {                                 // weight gradients per expert: reduce over the expert's row segment
    k.kb0 = g.seg_start[sp] / BK;
    k.kb1 = g.seg_start[sp + 1] / BK;
    k.c_off = (size_t)sp * (size_t)g.c_stride;
  }
  return k;
}

// FP8: both operands are E4M3 bytes, K-major; a k-slab is still 128 bytes of every row, i.e. 128 elements instead of
// 64, and the MMA consumes 32 elements per instruction, so the staging and the descriptors are those of the bf16 kernel.
template <bool A_MN, bool B_MN, typename TOut, int BN, bool FP8 = false>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, TOut* __restrict__ C,
               int M, int N, int K, Epi ep, int tiles_m, int tiles_n, int splits, int kb_per_split, GemmGroup grp, int* status) {
  constexpr int B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
  constexpr int HALF_CHUNKS = BN / 64;               // 32-column chunks per epilogue warp
  extern __shared__ unsigned char smem_dyn[];
  uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  uint32_t staging0 = base + STAGES * STAGE_BYTES;
  uint32_t bars = staging0 + EPI_WARPS * STAGING_BYTES;   // full[STAGES], empty[STAGES], tfull[2], tempty[2]
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int BKE = FP8 ? 2 * BK : BK;             // elements of k per slab (128 bytes of a K-major row)
  static_assert(!FP8 || (!A_MN && !B_MN), "8-bit operands are read along k");
  int total_kb = (K + BKE - 1) / BKE;
  int work_items = tiles_m * tiles_n * splits;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), EPI_WARPS); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&tmem_base_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  uint32_t tmem_base = tmem_base_slot;
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    // ------------------------------- TMA producer -------------------------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int armed = 0;
      bool ok = true;
      for (int w = blockIdx.x; w < work_items && ok; w += gridDim.x) {
        Work wk = decode_work(w, tiles_m, tiles_n, total_kb, kb_per_split, grp, (size_t)M * N);
        if (!wk.active) continue;
        int nt = wk.nt, mt = wk.mt;
        for (int kb = wk.kb0; kb < wk.kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abortp)) { ok = false; break; }
          mbar_expect_tx(full_bar(stage), STAGE_BYTES);
          uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
          if (!A_MN) {
            tma_load_2d(sa, &map_a, full_bar(stage), kb * BKE, mt * BM);
          } else {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) tma_load_2d(sa + j * (BK * 128), &map_a, full_bar(stage), mt * BM + j * 64, kb * BK);
          }
          if (!B_MN) {
            tma_load_2d(sb, &map_b, full_bar(stage), kb * BKE, nt * BN + wk.b_off);
          } else {
#pragma unroll
            for (int j = 0; j < BN / 64; ++j) tma_load_2d(sb + j * (BK * 128), &map_b, full_bar(stage), nt * BN + j * 64, kb * BK + wk.b_off);
          }
          ++armed;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && armed > 0) {
        // copies already issued still land in shared memory: give them a bounded time before the CTA leaves
        unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 1000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer ---------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = FP8 ? make_idesc_e4m3(BM, BN) : make_idesc(A_MN, B_MN, BN);
      // k step of 16 inside a stage: 32 bytes along a K-major row, 16 rows of 128 bytes for an MN-major operand
      constexpr uint32_t A_KSTEP = (A_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4, B_KSTEP = (B_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
      const uint64_t desc_a0 = A_MN ? make_desc(base, BK * 128, 1024) : make_desc(base, 16, 1024);
      const uint64_t desc_b0 = B_MN ? make_desc(base + A_BYTES, BK * 128, 1024) : make_desc(base + A_BYTES, 16, 1024);
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int w = blockIdx.x; w < work_items && ok; w += gridDim.x) {
        Work wk = decode_work(w, tiles_m, tiles_n, total_kb, kb_per_split, grp, (size_t)M * N);
        if (!wk.active) continue;
        int kb0 = wk.kb0, kb1 = wk.kb1;
        int buf = local & 1;
        if (!mbar_wait(tempty_bar(buf), ((local >> 1) & 1) ^ 1u, abortp)) { ok = false; break; }
        tc_fence_after();
        uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abortp)) { ok = false; break; }
          tc_fence_after();
          // descriptors of this stage: only the 16-byte-unit address field (low bits) moves with the stage and the k step
          uint64_t da = desc_a0 + (uint64_t)((stage * STAGE_BYTES) >> 4), db = desc_b0 + (uint64_t)((stage * STAGE_BYTES) >> 4);
          if (FP8) {
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k)       // four steps of 32 bytes along k, as for bf16
              umma_e4m3(d_tmem, da + (uint64_t)(k * A_KSTEP), db + (uint64_t)(k * B_KSTEP), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          } else {
            umma_bf16(d_tmem, da, db, idesc, kb > kb0 ? 1u : 0u);
#pragma unroll
            for (int k = 1; k < BK / UMMA_K; ++k)
              umma_bf16_acc(d_tmem, da + (uint64_t)(k * A_KSTEP), db + (uint64_t)(k * B_KSTEP), idesc);
          }
          umma_commit(empty_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(tfull_bar(buf));
        ++local;
      }
    }
  } else {
    // ------------------------------- epilogue -----------------------------------
    int ew = warp - 2;                      // 0..7
    int quarter = warp & 3;                 // TMEM lanes 32*quarter .. 32*quarter+31 (fixed by the warp's rank)
    int chalf = ew >> 2;                    // which half of the tile's columns
    unsigned char* st = smem_dyn + (staging0 - smem_u32(smem_dyn)) + ew * STAGING_BYTES;
    int local = 0;
    bool ok = true;
    for (int w = blockIdx.x; w < work_items && ok; w += gridDim.x) {
      Work wk = decode_work(w, tiles_m, tiles_n, total_kb, kb_per_split, grp, (size_t)M * N);
      if (!wk.active) continue;
      int nt = wk.nt, mt = wk.mt;
      int buf = local & 1;
      Epi epw = ep;
      if (epw.bias != nullptr) epw.bias += wk.bias_off;
      bool empty = wk.kb0 >= wk.kb1;          // an expert without tokens: its gradient tile is zero
      int row0 = mt * BM + quarter * 32;
      TOut* Cs = C + wk.c_off;
      // float outputs without activation take the single-transposition path; their residual is fetched a chunk ahead
      const bool f32_path = sizeof(TOut) == 4 && epw.act == 0 && epw.aux_out == nullptr;
      const bool has_res = f32_path && epw.residual != nullptr;
      // the stored pre-activation of the GELU derivative is fetched a chunk ahead as well
      const bool pre_z = sizeof(TOut) == 2 && epw.act == 2;       // (bf16 outputs: dz of the FFN backward)
      uint4 xn[8];
      if (has_res) chunk_issue((const float*)epw.residual, N, row0, nt * BN + chalf * HALF_CHUNKS * 32, M, N, lane, xn);
      if (pre_z) chunk_issue((const bf16*)epw.aux_in, N, row0, nt * BN + chalf * HALF_CHUNKS * 32, M, N, lane, xn);
      ok = mbar_wait(tfull_bar(buf), (local >> 1) & 1, abortp);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      if (f32_path) {
#pragma unroll
        for (int cc = 0; cc < HALF_CHUNKS; ++cc) {
          int cchunk = chalf * HALF_CHUNKS + cc;
          uint4 xc[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) xc[i] = xn[i];
          if (has_res && cc + 1 < HALF_CHUNKS) chunk_issue((const float*)epw.residual, N, row0, nt * BN + (cchunk + 1) * 32, M, N, lane, xn);
          uint32_t r[32];
          uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + cchunk * 32);
          tmem_ld32(taddr, r);
          tmem_ld_wait();
          if (empty) {
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = 0u;
          }
          epilogue_chunk_f32(r, epw.bias, (float*)Cs, M, N, row0, nt * BN + cchunk * 32, st, lane, xc, has_res);
        }
      } else {
#pragma unroll 1
      for (int cc = 0; cc < HALF_CHUNKS; ++cc) {
        int cchunk = chalf * HALF_CHUNKS + cc;
        float z[sizeof(TOut) == 2 ? 32 : 1];
        if (sizeof(TOut) == 2 && pre_z) {
          chunk_land_bf16(xn, st, lane, z);
          if (cc + 1 < HALF_CHUNKS) chunk_issue((const bf16*)epw.aux_in, N, row0, nt * BN + (cchunk + 1) * 32, M, N, lane, xn);
        }
        uint32_t r[32];
        uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + cchunk * 32);
        tmem_ld32(taddr, r);
        tmem_ld_wait();
        if (empty) {
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = 0u;
        }
        epilogue_chunk<TOut>(r, epw, Cs, M, N, row0, nt * BN + cchunk * 32, st, lane, pre_z ? z : nullptr);
      }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(buf));
      ++local;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && abort_flag && status != nullptr) atomicOr(status, STATUS_TIMEOUT);
}

// Diagnostic: the give-up path of the bounded waits, run on purpose.  One CTA allocates tensor memory as the GEMM does,
// waits on an mbarrier that nothing ever arrives at, gives up after limit_ns, frees its tensor memory, raises
// STATUS_TIMEOUT and returns -- the same teardown the kernels above perform when a wait of theirs expires.
__global__ void wait_expiry_kernel(int* status, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar_storage;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  uint32_t bar = smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  tmem_alloc(smem_u32(&tmem_slot), 32);
  tmem_relinquish();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (threadIdx.x == 0) mbar_wait_ns(bar, 0, &abort_flag, limit_ns);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  tmem_dealloc(tmem_slot, 32);
  if (threadIdx.x == 0 && abort_flag && status != nullptr) atomicOr(status, STATUS_TIMEOUT);
}

// out[i] = sum over splits of partial[s][i], ascending s.
__global__ void splitk_reduce_kernel(const float* __restrict__ partial, float* __restrict__ out, size_t n, int splits) {
  size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= n) return;
  float4 acc = *reinterpret_cast<const float4*>(partial + i);
  for (int s = 1; s < splits; ++s) {
    float4 v = *reinterpret_cast<const float4*>(partial + (size_t)s * n + i);
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
  }
  *reinterpret_cast<float4*>(out + i) = acc;
}

// The same reduction followed by the epilogue the GEMM kernel would have applied (bias, GELU with optional copy of the
// pre-activation, GELU derivative of a stored pre-activation, residual), for products whose few tiles are split along k.
template <typename TOut>
__global__ void splitk_reduce_epi_kernel(const float* __restrict__ partial, TOut* __restrict__ out, int m, int n, int splits, Epi ep) {
  size_t total = (size_t)m * n;
  size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= total) return;
  float4 a4 = *reinterpret_cast<const float4*>(partial + i);
  for (int s = 1; s < splits; ++s) {
    float4 v = *reinterpret_cast<const float4*>(partial + (size_t)s * total + i);
    a4.x += v.x; a4.y += v.y; a4.z += v.z; a4.w += v.w;
  }
  float v[4] = {a4.x, a4.y, a4.z, a4.w};
  int col = (int)(i % (size_t)n);                    // n is a multiple of 4: the four values share a row
  if (ep.bias != nullptr) {
    float4 bb = *reinterpret_cast<const float4*>(ep.bias + col);
    v[0] += bb.x; v[1] += bb.y; v[2] += bb.z; v[3] += bb.w;
  }
  if (ep.act == 1) {
    if (ep.aux_out != nullptr) store4(reinterpret_cast<TOut*>(ep.aux_out) + i, v);
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = gelu_f(v[j]);
  } else if (ep.act == 2) {
    float z[4];
    load4(reinterpret_cast<const bf16*>(ep.aux_in) + i, z);
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] *= gelu_grad_f(z[j]);
    if (ep.aux_out != nullptr) {            // GELU(z), recomputed for the weight gradient that follows
#pragma unroll
      for (int j = 0; j < 4; ++j) z[j] = gelu_f(z[j]);
      store4(reinterpret_cast<bf16*>(ep.aux_out) + i, z);
    }
  }
  if (ep.residual != nullptr) {
    float r[4];
    load4(reinterpret_cast<const TOut*>(ep.residual) + i, r);
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] += r[j];
  }
  store4(out + i, v);
}

static EncodeFn lookup_encode_fn() {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
    return (EncodeFn)p;
  return nullptr;
}

EncodeFn encode_fn() {
  static EncodeFn fn = lookup_encode_fn();      // initialised once, thread-safe
  return fn;
}

// 2-D bf16 tensor map: `inner` contiguous elements per row, `outer` rows `ld` elements apart, box {64, box_outer}.
bool make_map(CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t outer, uint64_t ld, uint32_t box_outer) {
  EncodeFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {64, box_outer};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_map_u8(CUtensorMap* map, const void* ptr, uint64_t inner, uint64_t outer, uint64_t ld, uint32_t box_outer) {
  EncodeFn fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld};
  cuuint32_t box[2] = {128, box_outer};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool A_MN, bool B_MN, typename TOut, int BN = BN_MAX, bool FP8 = false>
static int launch(const Ctx& c, const CUtensorMap& ma, const CUtensorMap& mb, void* C, int m, int n, int k, const Epi& ep,
                  int tiles_m, int tiles_n, int splits, int kb_per_split, const GemmGroup& grp) {
  auto kern = gemm_tc_kernel<A_MN, B_MN, TOut, BN, FP8>;
  static SmemLimit lim;
  if (!ensure_smem(lim, kern, SMEM_BYTES)) return -3;
  int work = tiles_m * tiles_n * splits;
  int sms = c.sm_count > 0 ? c.sm_count : 148;
  int grid = work < sms ? work : sms;
  note_launch(1);
  kern<<<grid, THREADS, SMEM_BYTES, c.stream>>>(ma, mb, (TOut*)C, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, grp, c.status);
  return 0;
}

}  // namespace tc

void wait_expiry_selftest(const Ctx& c, unsigned long long limit_ns) {
  note_launch(1);
  tc::wait_expiry_kernel<<<1, 32, 0, c.stream>>>(c.status, limit_ns);
}

void splitk_reduce(cudaStream_t s, const float* partial, float* out, size_t n, int splits) {
  note_launch(1);
  tc::splitk_reduce_kernel<<<ceil_div((long)(n / 4), 256), 256, 0, s>>>(partial, out, n, splits);
}

bool gemm_tc_supported(int m, int n, int k) { return m >= 1 && n >= 8 && k >= 8 && (n % 8) == 0 && (k % 8) == 0; }

// Strides as in gemm(): A(m,k) = A[m*a_rs + k*a_cs].  One of (a_rs, a_cs) must be 1, likewise for B.
int gemm_tc_strided(const Ctx& c, const void* A, long a_rs, long a_cs, const void* B, long b_rs, long b_cs, void* C,
                    int out_is_float, int m, int n, int k, const GemmEpilogue& e, float* split_ws, size_t split_ws_floats) {
  using namespace tc;
  bool a_mn = (a_cs != 1), b_mn = (b_cs != 1);
  if (a_mn && a_rs != 1) return -1;
  if (b_mn && b_rs != 1) return -1;
  long lda = a_mn ? a_cs : a_rs, ldb = b_mn ? b_cs : b_rs;
  if ((lda % 8) != 0 || (ldb % 8) != 0 || ((uintptr_t)A & 15) || ((uintptr_t)B & 15) || ((uintptr_t)C & 15)) return -1;
  if ((n % 8) != 0) return -1;
  if (a_mn && (m % 8) != 0) return -1;
  if (a_mn && !b_mn) return -1;                 // combination not instantiated
  CUtensorMap ma, mb;
  bool ok = a_mn ? make_map(&ma, A, (uint64_t)m, (uint64_t)k, (uint64_t)lda, BK) : make_map(&ma, A, (uint64_t)k, (uint64_t)m, (uint64_t)lda, BM);
  int sms = c.sm_count > 0 ? c.sm_count : 148;
  // Tile width: 192 columns instead of 256 where the narrower tiles fill the SMs' last wave better (a persistent CTA
  // per SM walks ceil(tiles / SMs) tiles; the time goes with that count times the tile width).  Not for operand A
  // read along m (weight gradients: those are split along k instead).
  int bn = BN_MAX;
  if (!a_mn) {
    long w256 = (long)ceil_div(ceil_div(m, BM) * ceil_div(n, 256), sms) * 256, w192 = (long)ceil_div(ceil_div(m, BM) * ceil_div(n, 192), sms) * 192;
    if (w192 < w256) bn = 192;
  }
  ok = ok && (b_mn ? make_map(&mb, B, (uint64_t)n, (uint64_t)k, (uint64_t)ldb, BK) : make_map(&mb, B, (uint64_t)k, (uint64_t)n, (uint64_t)ldb, bn));
  if (!ok) return -2;
  int tiles_m = ceil_div(m, BM), tiles_n = ceil_div(n, bn);
  int total_kb = ceil_div(k, BK);
  int splits = 1;
  bool plain = e.bias == nullptr && e.residual == nullptr && e.act == 0;
  // split along k: weight gradients (plain float outputs) and the few-row products of the classification-only tail,
  // whose epilogue then runs in the reduction
  if (split_ws != nullptr && tiles_m * tiles_n * 2 <= sms && total_kb >= 8 && ((out_is_float && plain) || (m <= 256 && (n % 4) == 0))) {
    splits = sms / (tiles_m * tiles_n);
    if (splits > total_kb / 4) splits = total_kb / 4;
    if (splits > 16) splits = 16;
    while (splits > 1 && (size_t)splits * m * n > split_ws_floats) --splits;
    if (splits < 1) splits = 1;
  }
  int kb_per_split = ceil_div(total_kb, splits);
  splits = ceil_div(total_kb, kb_per_split);
  Epi ep_full;
  ep_full.bias = e.bias; ep_full.residual = e.residual; ep_full.aux_out = e.aux_out; ep_full.aux_in = e.aux_in; ep_full.act = e.act;
  // split products write plain float partials; their epilogue runs in the reduction
  const bool deferred = splits > 1 && !(out_is_float && plain);
  Epi ep = ep_full;
  if (splits > 1) { ep.bias = nullptr; ep.residual = nullptr; ep.aux_out = nullptr; ep.aux_in = nullptr; ep.act = 0; }
  const int final_is_float = out_is_float;
  if (splits > 1) out_is_float = 1;
  void* dst = (splits > 1) ? (void*)split_ws : C;
  if (splits > 1) side_join(c, 2);         // the previous split sum has read the workspace
  if (c.prof != nullptr && c.prof->on) c.prof->begin(c.stream, 2.0 * m * n * (double)k);
  int rc;
  GemmGroup gg;
  if (bn == 192) {
    if (out_is_float) rc = b_mn ? launch<false, true, float, 192>(c, ma, mb, dst, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, gg)
                                : launch<false, false, float, 192>(c, ma, mb, dst, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, gg);
    else rc = b_mn ? launch<false, true, bf16, 192>(c, ma, mb, dst, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, gg)
                   : launch<false, false, bf16, 192>(c, ma, mb, dst, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, gg);
  } else if (out_is_float) {
    if (a_mn) rc = launch<true, true, float>(c, ma, mb, dst, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, gg);
    else if (b_mn) rc = launch<false, true, float>(c, ma, mb, dst, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, gg);
    else rc = launch<false, false, float>(c, ma, mb, dst, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, gg);
  } else {
    if (a_mn) rc = launch<true, true, bf16>(c, ma, mb, dst, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, gg);
    else if (b_mn) rc = launch<false, true, bf16>(c, ma, mb, dst, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, gg);
    else rc = launch<false, false, bf16>(c, ma, mb, dst, m, n, k, ep, tiles_m, tiles_n, splits, kb_per_split, gg);
  }
  if (rc != 0) return rc;
  if (splits > 1) {
    size_t total = (size_t)m * n;
    if (!deferred) {                       // a weight gradient: only the optimiser reads the sum
      splitk_reduce(side_begin(c), split_ws, (float*)C, total, splits);
      side_end(c, 2);
    } else {
      note_launch(1);
      int blocks = ceil_div((long)(total / 4), 256);
      if (final_is_float) splitk_reduce_epi_kernel<float><<<blocks, 256, 0, c.stream>>>(split_ws, (float*)C, m, n, splits, ep_full);
      else splitk_reduce_epi_kernel<bf16><<<blocks, 256, 0, c.stream>>>(split_ws, (bf16*)C, m, n, splits, ep_full);
    }
  }
  if (c.prof != nullptr && c.prof->on) c.prof->end(c.stream);
  return 0;
}

// Expert-grouped contractions of the MoE layer (paper Section 5.2); see kernels.h.
int gemm_tc_grouped_rows(const Ctx& c, const void* A, const void* Bst, int b_mn, void* C, int out_is_float, int rows_cap, int n, int k,
                         int experts, const int* tile_expert, const GemmEpilogue& e) {
  using namespace tc;
  if ((n % 8) || (k % 8) || (rows_cap % BM) || ((uintptr_t)A & 15) || ((uintptr_t)Bst & 15) || ((uintptr_t)C & 15)) return -1;
  if (b_mn && (k % BK)) return -1;             // a k-slab must not straddle two experts' weights
  CUtensorMap ma, mb;
  bool ok = make_map(&ma, A, (uint64_t)k, (uint64_t)rows_cap, (uint64_t)k, BM);
  ok = ok && (b_mn ? make_map(&mb, Bst, (uint64_t)n, (uint64_t)experts * k, (uint64_t)n, BK)
                   : make_map(&mb, Bst, (uint64_t)k, (uint64_t)experts * n, (uint64_t)k, BN_MAX));
  if (!ok) return -2;
  GemmGroup g;
  g.mode = 1;
  g.tile_expert = tile_expert;
  g.b_stride = b_mn ? k : n;
  g.bias_stride = n;
  Epi ep;
  ep.bias = e.bias; ep.residual = e.residual; ep.aux_out = e.aux_out; ep.aux_in = e.aux_in; ep.act = e.act;
  int tiles_m = rows_cap / BM, tiles_n = ceil_div(n, BN_MAX);
  if (c.prof != nullptr && c.prof->on) c.prof->begin(c.stream, 2.0 * rows_cap * n * (double)k);
  int rc;
  if (out_is_float)
    rc = b_mn ? launch<false, true, float>(c, ma, mb, C, rows_cap, n, k, ep, tiles_m, tiles_n, 1, ceil_div(k, BK), g)
              : launch<false, false, float>(c, ma, mb, C, rows_cap, n, k, ep, tiles_m, tiles_n, 1, ceil_div(k, BK), g);
  else
    rc = b_mn ? launch<false, true, bf16>(c, ma, mb, C, rows_cap, n, k, ep, tiles_m, tiles_n, 1, ceil_div(k, BK), g)
              : launch<false, false, bf16>(c, ma, mb, C, rows_cap, n, k, ep, tiles_m, tiles_n, 1, ceil_div(k, BK), g);
  if (c.prof != nullptr && c.prof->on) c.prof->end(c.stream);
  return rc;
}

int gemm_tc_grouped_wgrad(const Ctx& c, const void* dY, const void* X, float* dW, int rows_cap, int m, int n, int experts,
                          const int* seg_start) {
  using namespace tc;
  if ((m % 8) || (n % 8) || (rows_cap % BM) || ((uintptr_t)dY & 15) || ((uintptr_t)X & 15) || ((uintptr_t)dW & 15)) return -1;
  CUtensorMap ma, mb;
  if (!make_map(&ma, dY, (uint64_t)m, (uint64_t)rows_cap, (uint64_t)m, BK) || !make_map(&mb, X, (uint64_t)n, (uint64_t)rows_cap, (uint64_t)n, BK)) return -2;
  GemmGroup g;
  g.mode = 2;
  g.seg_start = seg_start;
  g.c_stride = (long)m * n;
  Epi ep;
  ep.bias = nullptr; ep.residual = nullptr; ep.aux_out = nullptr; ep.aux_in = nullptr; ep.act = 0;
  if (c.prof != nullptr && c.prof->on) c.prof->begin(c.stream, 2.0 * rows_cap * n * (double)m);
  int rc = launch<true, true, float>(c, ma, mb, dW, m, n, rows_cap, ep, ceil_div(m, BM), ceil_div(n, BN_MAX), experts, 0, g);
  if (c.prof != nullptr && c.prof->on) c.prof->end(c.stream);
  return rc;
}

// C[m, n] (bf16) = epilogue(a_scale[row] * b_scale[col] * sum_k Aq(m, k) * Bq(n, k)): E4M3 operands, one byte each, k contiguous.
int gemm_tc_e4m3(const Ctx& c, const void* Aq, const float* a_scale, const void* Bq, const float* b_scale, void* C, int m, int n,
                 int k, const GemmEpilogue& e) {
  using namespace tc;
  if ((k % 16) != 0 || (n % 8) != 0 || ((uintptr_t)Aq & 15) || ((uintptr_t)Bq & 15) || ((uintptr_t)C & 15)) return -1;
  if (a_scale == nullptr || b_scale == nullptr || e.residual != nullptr || e.act == 2) return -1;
  int sms = c.sm_count > 0 ? c.sm_count : 148;
  int bn = BN_MAX;
  long w256 = (long)ceil_div(ceil_div(m, BM) * ceil_div(n, 256), sms) * 256, w192 = (long)ceil_div(ceil_div(m, BM) * ceil_div(n, 192), sms) * 192;
  if (w192 < w256) bn = 192;
  CUtensorMap ma, mb;
  if (!make_map_u8(&ma, Aq, (uint64_t)k, (uint64_t)m, (uint64_t)k, BM) || !make_map_u8(&mb, Bq, (uint64_t)k, (uint64_t)n, (uint64_t)k, bn)) return -2;
  Epi ep;
  ep.bias = e.bias; ep.aux_out = e.aux_out; ep.act = e.act; ep.row_scale = a_scale; ep.col_scale = b_scale;
  int tiles_m = ceil_div(m, BM), tiles_n = ceil_div(n, bn);
  int total_kb = ceil_div(k, 2 * BK);
  GemmGroup gg;
  if (c.prof != nullptr && c.prof->on) c.prof->begin(c.stream, 2.0 * m * n * (double)k);
  int rc = bn == 192 ? launch<false, false, bf16, 192, true>(c, ma, mb, C, m, n, k, ep, tiles_m, tiles_n, 1, total_kb, gg)
                     : launch<false, false, bf16, 256, true>(c, ma, mb, C, m, n, k, ep, tiles_m, tiles_n, 1, total_kb, gg);
  if (c.prof != nullptr && c.prof->on) c.prof->end(c.stream);
  return rc;
}

int gemm_tc(const Ctx& c, const void* A, const void* B, void* C, int out_is_float, int m, int n, int k, const GemmEpilogue& e) {
  return gemm_tc_strided(c, A, k, 1, B, k, 1, C, out_is_float, m, n, k, e, nullptr, 0);
}

}  // namespace bsr
