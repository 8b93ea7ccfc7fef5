// Decode-regime layer-batched product (at most 16 rows per layer) on the 5th-generation tensor cores:
//   D[l][m][n] = sum_k A[l][m][k] * W[l][n][k]      A = activations [nl][M<=16][K] bf16, W = stacked weights [L][N][K] bf16
// The launch is bound by streaming W from HBM once, so the work is cut by BYTES, not by tiles:
//   * a tile = BN output columns of one layer; its reduction is cut into fixed SLICES of `kslice_kb` 64-element
//     k-blocks.  The slice length depends on the projection's shape only -- never on how many layers a launch
//     covers, on BN or on the grid -- and a tile's result is DEFINED as (((s_0 + s_1) + s_2) + ...) with every slice
//     s_i accumulated from zero in tensor memory.  A single-layer launch of the sequential path and a launch over
//     all layers of a sweep therefore produce the same bits, whichever CTA computes which slice.
//   * the (tile, slice) units of the launch, slice index fastest, are dealt to the CTAs (one per SM) as contiguous
//     ranges of equal length, so every SM streams the same number of bytes (+- one slice).
//   * a CTA that holds slice 0 of a tile adds its consecutive slices of that tile in shared memory; if it holds all
//     of them it runs the fused epilogue itself.  Otherwise the pieces go to a scratch area -- the holder of slice 0
//     writes its running sum, the others their slices one by one -- and whoever arrives last (a counter per split
//     tile, which it leaves at zero) adds them in slice order and runs the epilogue.  No CTA ever waits for another.
// TMA ring, MMA issue, tensor-memory double buffering, the bounded waits and the fused epilogues are those of
// k_umma_gemm (umma_gemm.cuh); the weights stay the 256-wide (or 128-wide) operand and the tokens a 16-row box.
#pragma once
#include "umma_gemm.cuh"

namespace snlp {

constexpr int kGemvMaxSlices = 40;   // most slices a tile may have (sizes the scratch area: [#CTAs][slices][rows][256] floats)

// The CTA that holds unit u when U units are dealt to G CTAs as ranges [c*U/G, (c+1)*U/G).
__host__ __device__ inline int gemv_owner(long long u, long long U, int G) { return (int)(((u + 1) * G + U - 1) / U) - 1; }

// k-blocks per slice for a reduction of nkb1 k-blocks per layer with kfuse layers chained into one tile: the smallest
// divisor of nkb1 that is >= 2 and leaves at most 20 slices per layer and kGemvMaxSlices per tile.
inline int gemv_kslice_kb(int nkb1, int kfuse) {
  for (int d = 1; d <= nkb1; ++d) {
    if (nkb1 % d) continue;
    if (d < 2 && nkb1 > 1) continue;
    const int s1 = nkb1 / d;
    if (s1 <= 20 && s1 * kfuse <= kGemvMaxSlices) return d;
  }
  return nkb1;
}

// grid = min(units, #SMs), 320 threads, dynamic shared memory UmmaCfg<BN, 16>::kSmem.
// p.ksplit = slices per layer's reduction, p.kslice = elements per slice; p.partial / p.tile_counters: scratch as above.
template <int BN, int EPI>
__global__ void __launch_bounds__(kUmmaThreads, 1) k_umma_gemv(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                                                              UmmaParams p) {
  using Cfg = UmmaCfg<BN, 16>;
  extern __shared__ unsigned char umma_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)umma_smem_raw + 1023) & ~(uintptr_t)1023);
  const int S = p.nstages;
  unsigned char *sA = smem;                                   // [S][16 x 128 B]; the A descriptor reads 128 rows from a slot
  unsigned char *sB = smem + (size_t)S * Cfg::kABytes;        // [S][BN x 128 B]   (>= 16 KB, so those reads stay in bounds)
  float *outs = reinterpret_cast<float *>(sB + (size_t)S * Cfg::kBBytes);   // [16][BN + 1]
  uint64_t *full = reinterpret_cast<uint64_t *>(reinterpret_cast<unsigned char *>(outs) + Cfg::kOuts);
  uint64_t *empty = full + S;
  uint64_t *accfull = empty + S, *accempty = accfull + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(accempty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  int *s_last = const_cast<int *>(abort_flag) + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int skb = p.kslice / kUmmaBK;                 // k-blocks per slice
  const int kst = p.ksplit * p.kfuse;                 // slices per tile
  const long long U = (long long)p.Nt * p.nl * kst;   // units of the launch
  const int G = (int)gridDim.x;
  const int u_begin = (int)((long long)blockIdx.x * U / G), u_end = (int)((long long)(blockIdx.x + 1) * U / G);
  const int my_units = u_end - u_begin;
  constexpr uint32_t kTmemCols = 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < S; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&accfull[i], 1);
      mbar_init(&accempty[i], 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // unit -> (tile, slice); tile -> (column tile, layer item); slice -> (layer inside a K-concatenated chunk, K offset)
#define SNLP_DECODE_UNIT(i)                                                                                   \
  const int u_ = u_begin + (i);                                                                               \
  const int tile = u_ / kst, sl = u_ % kst;                                                                   \
  const int n_tile = tile % p.Nt, li_ = tile / p.Nt;                                                          \
  const int la = p.a_share > 1 ? (li_ / p.a_share) * p.a_share : li_ * p.kfuse; /* A rows' layer slot */      \
  const int l = li_ * p.kfuse;                                                   /* output / weight layer slot */ \
  const int jl = sl / p.ksplit, k0 = (sl % p.ksplit) * p.kslice;

  if (warp == 0) {
    if (lane == 0) {
      int g = 0, issued = 0;
      bool ok = true;
      for (int i = 0; i < my_units && ok; ++i) {
        SNLP_DECODE_UNIT(i)
        for (int kb = 0; kb < skb; ++kb, ++g) {
          const int s = g % S;
          ok = mbar_wait(&empty[s], ((g / S) & 1) ^ 1u, abort_flag, p.err);
          if (!ok) break;
          mbar_expect_tx(&full[s], Cfg::kABytes + Cfg::kBBytes);
          tma_load_3d(sA + (size_t)s * Cfg::kABytes, &tmA, &full[s], k0 + kb * kUmmaBK, 0, la + jl);
          tma_load_3d(sB + (size_t)s * Cfg::kBBytes, &tmB, &full[s], k0 + kb * kUmmaBK, n_tile * BN, p.l0 + l + jl);
          issued = g + 1;
        }
      }
      if (*abort_flag) {
        // let the copies still in flight land before the CTA's shared memory is handed on
        const int first = issued > S ? issued - S : 0;
        for (int q = first; q < issued; ++q) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(&full[q % S], (q / S) & 1) && global_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kUmmaBM, BN);
      int g = 0;
      bool ok = true;
      for (int i = 0; i < my_units && ok; ++i) {
        const int b = i & 1;
        ok = mbar_wait(&accempty[b], ((i >> 1) & 1) ^ 1u, abort_flag, p.err);
        if (!ok) break;
        tc_fence_after();
        const uint32_t dcol = tmem_base + b * BN;
        for (int kb = 0; kb < skb; ++kb, ++g) {
          const int s = g % S;
          ok = mbar_wait(&full[s], (g / S) & 1, abort_flag, p.err);
          if (!ok) break;
          tc_fence_after();
          const uint64_t da = umma_desc_sw128(smem_u32(sA + (size_t)s * Cfg::kABytes));
          const uint64_t db = umma_desc_sw128(smem_u32(sB + (size_t)s * Cfg::kBBytes));
#pragma unroll
          for (int k = 0; k < kUmmaBK / 16; ++k)  // 16 bf16 = 32 bytes = 2 descriptor address units per step
            umma_bf16(dcol, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
          umma_commit(&empty[s]);
        }
        if (ok) umma_commit(&accfull[b]);
      }
    }
  } else {
    const int et = threadIdx.x - 64, ew = et >> 5, grp = ew >> 2;   // two warp groups share the columns
    const int quarter = warp & 3;  // tensor-memory lanes this warp may read: 32*quarter .. +31
    const int nelem = p.M * BN;    // fp32 values of one piece in the scratch area
    for (int i = 0; i < my_units; ++i) {
      SNLP_DECODE_UNIT(i)
      (void)jl; (void)k0;
      const int b = i & 1;
      const int t0u = tile * kst;                       // first unit of the tile
      const bool own0 = t0u >= u_begin;                 // this CTA holds slice 0: it keeps a running sum of its slices
      const int seg_end = (t0u + kst < u_end ? t0u + kst : u_end);   // one past this CTA's last unit of the tile
      const bool add = own0 && sl > 0;
      const bool last_of_piece = own0 ? (u_ == seg_end - 1) : true;
      if (!epi_all(mbar_wait(&accfull[b], (i >> 1) & 1, abort_flag, p.err))) break;
      tc_fence_after();
      const uint32_t tbase = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * BN;
      if (quarter == 0) {  // the token rows live in lanes 0..15; each group's quarter-0 warp moves half the columns
#pragma unroll 1
        for (int c = grp * (BN / 64); c < (grp + 1) * (BN / 64); ++c) {
          uint32_t r[32];
          tmem_ld32(tbase + c * 32, r);
          if (lane < 16) {
            float *o = outs + lane * (BN + 1) + c * 32;
            if (add) {
#pragma unroll
              for (int j = 0; j < 32; ++j) o[j] = o[j] + __uint_as_float(r[j]);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) o[j] = __uint_as_float(r[j]);
            }
          }
        }
      }
      tc_fence_before();
      epi_bar_sync();
      if (et == 0) mbar_arrive(&accempty[b]);
      if (!last_of_piece) continue;
      bool finish = own0 && sl == kst - 1;   // every slice of the tile went through this CTA
      if (!finish) {
        // a split tile: its pieces meet in the scratch region of the CTA that holds slice 0
        const int c0 = own0 ? (int)blockIdx.x : gemv_owner(t0u, U, G);
        const int c0_end = (int)((long long)(c0 + 1) * U / G);
        const int npre = (c0_end < t0u + kst ? c0_end : t0u + kst) - t0u;    // slices inside the running sum (slot 0)
        float *reg = p.partial + (size_t)c0 * kst * nelem;
        float *dst = reg + (size_t)(own0 ? 0 : sl) * nelem;
        for (int e = et; e < nelem; e += kUmmaEpiThreads) dst[e] = outs[(e / BN) * (BN + 1) + (e % BN)];
        __threadfence();
        epi_bar_sync();
        if (et == 0) *s_last = atomicAdd(&p.tile_counters[c0], 1u) == (unsigned)(kst - npre) ? 1 : 0;   // 1 + (kst - npre) pieces
        epi_bar_sync();
        if (*s_last) {
          __threadfence();
          for (int e = et; e < nelem; e += kUmmaEpiThreads) {
            float acc = __ldcg(reg + e);
            for (int q = npre; q < kst; ++q) acc = acc + __ldcg(reg + (size_t)q * nelem + e);   // slice order
            outs[(e / BN) * (BN + 1) + (e % BN)] = acc;
          }
          if (et == 0) p.tile_counters[c0] = 0u;
          epi_bar_sync();
          finish = true;
        }
      }
      if (finish) umma_epilogue_small<BN, EPI>(p, outs, ew, lane, n_tile, 0, l, la);
      epi_bar_sync();  // outs is reused by the next unit
    }
    if (EPI == UEPI_LMHEAD && (p.argmax != nullptr || p.argmax_pp != nullptr)) {
      // Greedy token: every CTA counts itself in once its units are done (also after a wait that ran out, so that the
      // counter always returns to zero); the last one merges the tiles' maxima.
      __threadfence();
      epi_bar_sync();
      if (et == 0) *s_last = atomicAdd(p.lm_counter, 1u) == gridDim.x - 1 ? 1 : 0;
      epi_bar_sync();
      if (*s_last) {
        __threadfence();
        int32_t *amax = p.argmax_pp != nullptr ? *p.argmax_pp : p.argmax;
        for (int tok = ew; tok < p.M; tok += 8) {
          float bv = -INFINITY;
          int bi = 0x7fffffff;
          for (int j = lane; j < p.Nt; j += 32) {
            const float v = __ldcg(&p.pm_val[(size_t)tok * p.Nt + j]);
            const int ix = __ldcg(&p.pm_idx[(size_t)tok * p.Nt + j]);
            if (v > bv || (v == bv && ix < bi)) { bv = v; bi = ix; }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
          if (lane == 0) amax[tok] = (unsigned)bi < (unsigned)p.N ? bi : 0;
        }
        if (et == 0) {
          if (p.bump != nullptr) *p.bump += 1;
          *p.lm_counter = 0u;
        }
      }
    }
  }
#undef SNLP_DECODE_UNIT
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace snlp
