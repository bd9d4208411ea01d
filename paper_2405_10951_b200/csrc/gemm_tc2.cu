// bf16 GEMM on CTA pairs: tcgen05.mma cta_group::2 with a 256 x 256 accumulator tile spread over the tensor
// memory of two SMs.  Same contract as the single-CTA kernel (operand majors, epilogues, split-k), but each SM
// stages only its own 128 rows of A and its own 128 columns' worth of B per k-slab (32 KB instead of 48 KB
// for the same number of multiply-accumulates), which is what the per-SM shared-memory fill rate limits.
//
// Cluster of two CTAs, persistent, one cluster per SM pair:
//   warp 0 (both CTAs) : TMA producer; every copy signals the full barrier of the leader CTA (rank 0)
//   warp 1 (leader)    : issues the MMAs; its commits arrive on the empty / accumulator-full barriers of both CTAs
//   warps 2..9 (both)  : epilogue of the CTA's own 128 rows; they release the accumulator on the leader's barrier
// Five-stage ring of 32 KB per CTA; the epilogue prefetches residual / pre-activation chunks with cp.async.  Waits are bounded as in the single-CTA kernel.
#include <cuda.h>

#include "common.cuh"
#include "kernels.h"
#include "tc_ptx.cuh"
#include "tc_epilogue.cuh"

namespace bsr {
namespace tc2 {

using namespace tc;

constexpr int BM = 128;                   // rows per CTA (256 per pair)
constexpr int BN = 256;                   // columns per pair tile; each CTA stages BN/2 of B
constexpr int BK = 64;
constexpr int STAGES = 5;
constexpr int UMMA_K = 16;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = (BN / 2) * BK * 2;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;      // 32 KB
constexpr int EPI_WARPS = 8;
constexpr int STAGING_BYTES = 32 * 128;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 2 * EPI_WARPS * STAGING_BYTES + 1024 + 256;
constexpr int THREADS = 64 + EPI_WARPS * 32;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t PEER_MASK = 0xFEFFFFFFu;         // clears the CTA-rank bit of a shared address: the even CTA of the pair

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrives (once the MMAs issued so far have completed) on the barrier at the same offset in both CTAs of the pair.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
               "h"(mask)
               : "memory");
}
// Arrive on the barrier at the same offset in the leader CTA's shared memory.
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(remote) : "r"(bar));
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}

template <bool A_MN, bool B_MN, typename TOut>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, TOut* __restrict__ C,
                int M, int N, int K, Epi ep, int pairs_m, int tiles_n, int splits, int kb_per_split, int* status) {
  extern __shared__ unsigned char smem_dyn[];
  uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  uint32_t staging0 = base + STAGES * STAGE_BYTES;
  uint32_t bars = staging0 + 2 * EPI_WARPS * STAGING_BYTES;   // full[STAGES], empty[STAGES], tfull[2], tempty[2]
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  uint32_t rank = cluster_rank();
  bool leader = rank == 0;
  int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  int total_kb = (K + BK - 1) / BK;
  int work_items = pairs_m * tiles_n * splits;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 2 * EPI_WARPS); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&tmem_base_slot), TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();                       // barriers of both CTAs exist before anyone signals them
  tc_fence_after();
  uint32_t tmem_base = tmem_base_slot;
  volatile int* abortp = &abort_flag;

  if (warp == 0) {
    // ------------------------------- TMA producer (both CTAs) -------------------------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int armed = 0;
      bool ok = true;
      for (int w = cluster_id; w < work_items && ok; w += n_clusters) {
        int nt = w % tiles_n, pm = (w / tiles_n) % pairs_m, sp = w / (pairs_m * tiles_n);
        int kb0 = sp * kb_per_split, kb1 = min(total_kb, kb0 + kb_per_split);
        int m0 = pm * (2 * BM) + (int)rank * BM;          // this CTA's rows of A
        int n0 = nt * BN + (int)rank * (BN / 2);          // this CTA's share of B
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abortp)) { ok = false; break; }
          uint32_t fb = full_bar(stage) & PEER_MASK;      // the leader's barrier collects both CTAs' bytes
          if (leader) mbar_expect_tx(full_bar(stage), 2 * STAGE_BYTES);
          uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
          if (!A_MN) {
            tma_load_2d_pair(sa, &map_a, fb, kb * BK, m0);
          } else {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) tma_load_2d_pair(sa + j * (BK * 128), &map_a, fb, m0 + j * 64, kb * BK);
          }
          if (!B_MN) {
            tma_load_2d_pair(sb, &map_b, fb, kb * BK, n0);
          } else {
#pragma unroll
            for (int j = 0; j < BN / 128; ++j) tma_load_2d_pair(sb + j * (BK * 128), &map_b, fb, n0 + j * 64, kb * BK);
          }
          ++armed;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && armed > 0) {
        unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 1000000ull) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer (leader CTA only) ---------------------------
    if (lane == 0 && leader) {
      constexpr uint32_t idesc = make_idesc_mn(2 * BM, BN, A_MN, B_MN);
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int w = cluster_id; w < work_items && ok; w += n_clusters, ++local) {
        int sp = w / (pairs_m * tiles_n);
        int kb0 = sp * kb_per_split, kb1 = min(total_kb, kb0 + kb_per_split);
        int buf = local & 1;
        if (!mbar_wait(tempty_bar(buf), ((local >> 1) & 1) ^ 1u, abortp)) { ok = false; break; }
        tc_fence_after();
        uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abortp)) { ok = false; break; }
          tc_fence_after();
          uint32_t sa = base + stage * STAGE_BYTES, sb = sa + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            uint64_t da = A_MN ? make_desc(sa + k * (UMMA_K * 128), BK * 128, 1024) : make_desc(sa + k * (UMMA_K * 2), 16, 1024);
            uint64_t db = B_MN ? make_desc(sb + k * (UMMA_K * 128), BK * 128, 1024) : make_desc(sb + k * (UMMA_K * 2), 16, 1024);
            umma_bf16_pair(d_tmem, da, db, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          }
          umma_commit_pair(empty_bar(stage));
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit_pair(tfull_bar(buf));
      }
    }
  } else {
    // ------------------------------- epilogue (both CTAs, own rows) --------------------------
    int ew = warp - 2;
    int quarter = warp & 3;
    int chalf = ew >> 2;
    uint32_t st_in_addr = staging0 + (2 * ew) * STAGING_BYTES;
    unsigned char* st_in = smem_dyn + (st_in_addr - smem_u32(smem_dyn));
    unsigned char* st_out = st_in + STAGING_BYTES;
    int local = 0;
    bool ok = true;
    for (int w = cluster_id; w < work_items && ok; w += n_clusters, ++local) {
      int nt = w % tiles_n, pm = (w / tiles_n) % pairs_m, sp = w / (pairs_m * tiles_n);
      int buf = local & 1;
      ok = mbar_wait(tfull_bar(buf), (local >> 1) & 1, abortp);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      int row0 = pm * (2 * BM) + (int)rank * BM + quarter * 32;
      TOut* Cs = C + (size_t)sp * M * N;
      uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + chalf * 128);
      auto load_tmem = [&](int cc, uint32_t* r) {
        tmem_ld32(taddr0 + cc * 32, r);
        tmem_ld_wait();
      };
      epilogue_warp_tile<TOut>(load_tmem, ep, Cs, M, N, row0, nt * BN + chalf * 128, 4, st_in, st_in_addr, st_out, lane, false);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(tempty_bar(buf));
    }
  }
  tc_fence_before();
  __syncwarp();
  cluster_sync_all();                       // neither CTA leaves while the other may still touch its memory
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0 && abort_flag && status != nullptr) atomicOr(status, STATUS_TIMEOUT);
}

template <bool A_MN, bool B_MN, typename TOut>
static int launch(const Ctx& c, const CUtensorMap& ma, const CUtensorMap& mb, void* C, int m, int n, int k, const Epi& ep,
                  int pairs_m, int tiles_n, int splits, int kb_per_split) {
  auto kern = gemm_tc2_kernel<A_MN, B_MN, TOut>;
  static SmemLimit lim;
  if (!ensure_smem(lim, kern, SMEM_BYTES)) return -3;
  int work = pairs_m * tiles_n * splits;
  int sms = c.sm_count > 0 ? c.sm_count : 148;
  int clusters = work < sms / 2 ? work : sms / 2;
  note_launch(1);
  kern<<<2 * clusters, THREADS, SMEM_BYTES, c.stream>>>(ma, mb, (TOut*)C, m, n, k, ep, pairs_m, tiles_n, splits, kb_per_split, c.status);
  return 0;
}

}  // namespace tc2

// Same contract as gemm_tc_strided, on CTA pairs.  Returns non-zero when the problem is not taken.
int gemm_tc2_strided(const Ctx& c, const void* A, long a_rs, long a_cs, const void* B, long b_rs, long b_cs, void* C,
                     int out_is_float, int m, int n, int k, const GemmEpilogue& e, float* split_ws, size_t split_ws_floats) {
  using namespace tc2;
  bool a_mn = (a_cs != 1), b_mn = (b_cs != 1);
  if (a_mn && a_rs != 1) return -1;
  if (b_mn && b_rs != 1) return -1;
  long lda = a_mn ? a_cs : a_rs, ldb = b_mn ? b_cs : b_rs;
  if ((lda % 8) != 0 || (ldb % 8) != 0 || ((uintptr_t)A & 15) || ((uintptr_t)B & 15) || ((uintptr_t)C & 15)) return -1;
  if ((n % 8) != 0) return -1;
  if (a_mn && (m % 8) != 0) return -1;
  if (a_mn && !b_mn) return -1;
  CUtensorMap ma, mb;
  bool ok = a_mn ? tc::make_map(&ma, A, (uint64_t)m, (uint64_t)k, (uint64_t)lda, BK) : tc::make_map(&ma, A, (uint64_t)k, (uint64_t)m, (uint64_t)lda, BM);
  ok = ok && (b_mn ? tc::make_map(&mb, B, (uint64_t)n, (uint64_t)k, (uint64_t)ldb, BK) : tc::make_map(&mb, B, (uint64_t)k, (uint64_t)n, (uint64_t)ldb, BN / 2));
  if (!ok) return -2;
  int pairs_m = ceil_div(m, 2 * BM), tiles_n = ceil_div(n, BN);
  int total_kb = ceil_div(k, BK);
  int splits = 1;
  bool plain = e.bias == nullptr && e.residual == nullptr && e.act == 0;
  int clusters = (c.sm_count > 0 ? c.sm_count : 148) / 2;
  if (out_is_float && plain && split_ws != nullptr && pairs_m * tiles_n * 2 <= clusters && total_kb >= 8) {
    splits = clusters / (pairs_m * tiles_n);
    if (splits > total_kb / 4) splits = total_kb / 4;
    if (splits > 16) splits = 16;
    while (splits > 1 && (size_t)splits * m * n > split_ws_floats) --splits;
    if (splits < 1) splits = 1;
  }
  int kb_per_split = ceil_div(total_kb, splits);
  splits = ceil_div(total_kb, kb_per_split);
  tc::Epi ep;
  ep.bias = e.bias; ep.residual = e.residual; ep.aux_out = e.aux_out; ep.aux_in = e.aux_in; ep.act = e.act;
  void* dst = (splits > 1) ? (void*)split_ws : C;
  if (c.prof != nullptr && c.prof->on) c.prof->begin(c.stream, 2.0 * m * n * (double)k);
  int rc;
  if (out_is_float) {
    if (a_mn) rc = launch<true, true, float>(c, ma, mb, dst, m, n, k, ep, pairs_m, tiles_n, splits, kb_per_split);
    else if (b_mn) rc = launch<false, true, float>(c, ma, mb, dst, m, n, k, ep, pairs_m, tiles_n, splits, kb_per_split);
    else rc = launch<false, false, float>(c, ma, mb, dst, m, n, k, ep, pairs_m, tiles_n, splits, kb_per_split);
  } else {
    if (a_mn) rc = launch<true, true, bf16>(c, ma, mb, dst, m, n, k, ep, pairs_m, tiles_n, splits, kb_per_split);
    else if (b_mn) rc = launch<false, true, bf16>(c, ma, mb, dst, m, n, k, ep, pairs_m, tiles_n, splits, kb_per_split);
    else rc = launch<false, false, bf16>(c, ma, mb, dst, m, n, k, ep, pairs_m, tiles_n, splits, kb_per_split);
  }
  if (rc != 0) return rc;
  if (splits > 1) {
    size_t total = (size_t)m * n;
    splitk_reduce(c.stream, split_ws, (float*)C, total, splits);
  }
  if (c.prof != nullptr && c.prof->on) c.prof->end(c.stream);
  return 0;
}

}  // namespace bsr
