// The prefill-regime GEMM on CTA pairs (tcgen05 cta_group::2): one 256 x 256 output tile per pair of SMs.
//
// k_umma_gemm with 128 x 256 tiles is bound by the operand traffic into an SM (48 KB per 64-wide k-block against
// ~620 cycles of MMA).  Here the two CTAs of a cluster each load their own 128 rows of A and one half (128 rows) of
// the 256-wide weight tile, 32 KB per k-block, and the leader CTA's MMA thread issues 256 x 256 x 16 instructions that
// read both CTAs' shared memory and write each CTA's 128 accumulator rows into that CTA's tensor memory.
//
// Barriers: full[s] lives in the leader (rank 0) and counts both CTAs' TMA transactions; empty[s] and accfull[b] exist
// in both CTAs and are signalled by the leader's tcgen05.commit with the cluster multicast mask; accempty[b] lives in
// the leader and collects one arrival per CTA's epilogue.  Work items, epilogues and all bounded-wait / error
// behaviour are those of k_umma_gemm; the row tile of an item covers 256 rows.
#pragma once
#include "umma_gemm.cuh"

namespace snlp {

constexpr int kU2BN = 256;                                   // output columns of a pair's tile
constexpr int kU2ABytes = kUmmaBM * kUmmaBK * 2;             // this CTA's 128 rows of A: 16 KB per stage
constexpr int kU2BBytes = (kU2BN / 2) * kUmmaBK * 2;         // this CTA's half of the weight tile: 16 KB per stage
constexpr int kU2Stage = 8 * 4096;                           // epilogue staging, as in k_umma_gemm
constexpr int kU2Stages = (kUmmaSmemBudget - kU2Stage - 1024 - 512) / (kU2ABytes + kU2BBytes);
constexpr int kU2Smem = kU2Stages * (kU2ABytes + kU2BBytes) + kU2Stage + 1024 + 512;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
}
// TMA load into this CTA's shared memory whose bytes are counted on an mbarrier that may sit in the peer CTA
__device__ __forceinline__ void tma_load_3d_pair(void *dst, const CUtensorMap *tm, uint32_t bar_cluster, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(tm), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t *slot, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on the mbarrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(smem_u32(bar)),
               "h"((uint16_t)3)
               : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// grid = 2 * min(items, #SMs / 2) CTAs in clusters of 2, 320 threads, dynamic shared memory kU2Smem.
// tmA: 3-D map over A {K, M, nl}, box {64, 128, 1}; tmB: 3-D map over the stacked weights {K, N, L}, box {64, 128, 1}.
// p.Mt counts 256-row tiles.
template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kUmmaThreads, 1)
    k_umma_gemm2(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, UmmaParams p) {
  constexpr int BN = kU2BN;
  extern __shared__ unsigned char umma2_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)umma2_smem_raw + 1023) & ~(uintptr_t)1023);
  constexpr int S = kU2Stages;
  unsigned char *sA = smem;                                // [S][128 x 128 B]
  unsigned char *sB = smem + (size_t)S * kU2ABytes;        // [S][128 x 128 B]
  float *outs = reinterpret_cast<float *>(sB + (size_t)S * kU2BBytes);
  uint64_t *full = reinterpret_cast<uint64_t *>(reinterpret_cast<unsigned char *>(outs) + kU2Stage);
  uint64_t *empty = full + S;
  uint64_t *accfull = empty + S, *accempty = accfull + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(accempty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = (int)blockIdx.x >> 1, npairs = (int)gridDim.x >> 1;
  const int nkb1 = p.kslice / kUmmaBK;
  const int nkb = nkb1 * p.kfuse;
  const int n_items = p.Mt * p.Nt * p.ksplit * p.nl;
  const int my_items = pair < n_items ? (n_items - 1 - pair) / npairs + 1 : 0;
  constexpr uint32_t kTmemCols = 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(&full[s], 2);    // used in the leader only: one arrive.expect_tx per CTA
      mbar_init(&empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&accfull[i], 1);
      mbar_init(&accempty[i], 2);  // used in the leader only: one arrival per CTA's epilogue
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // the peer's barriers are initialised before anything is signalled across
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

#define SNLP_DECODE_ITEM2(i)                                      \
  const int it_ = pair + (i) * npairs;                            \
  const int m_tile = it_ % p.Mt;                                  \
  const int n_tile = (it_ / p.Mt) % p.Nt;                         \
  const int ks = (it_ / (p.Mt * p.Nt)) % p.ksplit;                \
  const int li_ = it_ / (p.Mt * p.Nt * p.ksplit);                 \
  const int la = p.a_share > 1 ? (li_ / p.a_share) * p.a_share : li_ * p.kfuse; \
  const int l = li_ * p.kfuse;

  if (warp == 0) {
    if (lane == 0) {
      int g = 0, issued = 0;
      bool ok = true;
      for (int i = 0; i < my_items && ok; ++i) {
        SNLP_DECODE_ITEM2(i)
        for (int kb = 0; kb < nkb; ++kb, ++g) {
          const int s = g % S;
          ok = mbar_wait(&empty[s], ((g / S) & 1) ^ 1u, abort_flag, p.err);
          if (!ok) break;
          const uint32_t lead_full = mapa_rank(smem_u32(&full[s]), 0);
          mbar_expect_tx_cluster(lead_full, kU2ABytes + kU2BBytes);
          const int j = kb / nkb1, k0 = ks * p.kslice + (kb % nkb1) * kUmmaBK;
          tma_load_3d_pair(sA + (size_t)s * kU2ABytes, &tmA, lead_full, k0, m_tile * 2 * kUmmaBM + (int)rank * kUmmaBM, la + j);
          tma_load_3d_pair(sB + (size_t)s * kU2BBytes, &tmB, lead_full, k0, n_tile * BN + (int)rank * (BN / 2), p.l0 + l + j);
          issued = g + 1;
        }
      }
      (void)issued;
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(2 * kUmmaBM, BN);
      int g = 0;
      bool ok = true;
      for (int i = 0; i < my_items && ok; ++i) {
        const int b = i & 1;
        ok = mbar_wait(&accempty[b], ((i >> 1) & 1) ^ 1u, abort_flag, p.err);
        if (!ok) break;
        tc_fence_after();
        const uint32_t dcol = tmem_base + b * BN;
        for (int kb = 0; kb < nkb; ++kb, ++g) {
          const int s = g % S;
          ok = mbar_wait(&full[s], (g / S) & 1, abort_flag, p.err);
          if (!ok) break;
          tc_fence_after();
          const uint64_t da = umma_desc_sw128(smem_u32(sA + (size_t)s * kU2ABytes));
          const uint64_t db = umma_desc_sw128(smem_u32(sB + (size_t)s * kU2BBytes));
#pragma unroll
          for (int k = 0; k < kUmmaBK / 16; ++k) umma_bf16_pair(dcol, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
          umma_commit_pair(&empty[s]);
        }
        if (ok) umma_commit_pair(&accfull[b]);
      }
    }
  } else {
    const int et = threadIdx.x - 64, ew = et >> 5, grp = ew >> 2;
    const int quarter = warp & 3;
    for (int i = 0; i < my_items; ++i) {
      SNLP_DECODE_ITEM2(i)
      const int b = i & 1;
      const int row0 = m_tile * 2 * kUmmaBM + (int)rank * kUmmaBM;
      if (EPI == UEPI_RESID) {
        const int prow = row0 + quarter * 32 + lane;
        if (prow < p.M) {
          const float *px = p.xm + (size_t)l * p.xm_ls + (size_t)prow * p.N + (size_t)n_tile * BN + grp * (BN / 2);
#pragma unroll
          for (int c = 0; c < BN / 64; ++c) asm volatile("prefetch.global.L2 [%0];" ::"l"(px + c * 32));
        }
      }
      if (!epi_all(mbar_wait(&accfull[b], (i >> 1) & 1, abort_flag, p.err))) break;
      tc_fence_after();
      const uint32_t tbase = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * BN;
      umma_epilogue_rows<BN, EPI>(p, tbase, row0 + quarter * 32 + lane, n_tile, ks, l, la, grp, reinterpret_cast<float4 *>(outs) + ew * 256);
      tc_fence_before();
      epi_bar_sync();
      if (et == 0) mbar_arrive_cluster(mapa_rank(smem_u32(&accempty[b]), 0));
    }
  }
#undef SNLP_DECODE_ITEM2
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // the leader's MMAs read the peer's shared memory and signal its barriers: leave together
  if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
}

}  // namespace snlp
