// Decode-regime products that follow one another (attention out-projection -> MLP up -> MLP down) as ONE persistent
// kernel: the phases are separated by grid-wide barriers instead of kernel boundaries, and the weight stream never
// stops at them.  A phase's weight tiles depend on nothing the kernel computes, so the producer of every CTA keeps
// requesting the next phase's weights while the previous phase's epilogues are still running elsewhere (CTAs that have
// no item in a phase -- 48 of 148 in the out-projection of a sweep -- start on the next phase's weights at once); only
// the activation tiles of a phase wait for its barrier.  What this removes is the drain and ramp-up of the memory system
// around every kernel boundary.  Items, tiles, accumulation order and epilogues are exactly those of k_umma_gemm (one
// launch per product), so the results are the same bits.
//
// Grid barrier: one counter in global memory, zero on entry.  Every CTA adds one when its epilogues of a phase are
// complete (after a device-scope fence); a CTA without items in a phase adds its one as soon as that phase is open.
// Phase ph opens when the counter reaches ph * #CTAs.  The CTA whose arrival completes the last phase puts the counter
// back to zero.  The kernel needs all its CTAs resident
// (one per SM): it is launched cooperatively.  All waits are bounded as in k_umma_gemm.
#pragma once
#include "decode.cuh"
#include "umma_gemm.cuh"

namespace snlp {

constexpr int kChainMax = 3;

struct ChainParams {
  CUtensorMap tmA[kChainMax], tmB[kChainMax];   // per phase: activations {64, M, K / 64, layers}, box {64, 16, kbox, 1}; weights {64, N, K / 64, L}, box {64, BN, kbox, 1}
  UmmaParams p[kChainMax];
  int epi[kChainMax];                           // UEPI_* of the phase
  int nphase;
  int kbox;                                     // k-blocks per bulk-tensor copy, the same in every phase (the ring is shared)
  unsigned *bar;                                // grid-barrier counter
  // Optional first step: merge the split-KV partials the decode attention left behind (k_attn_decode with merge_here = 0)
  // into the bf16 attention output that phase 0 reads.  comb_rows = layers x sequences x heads x queries (0 = no such step).
  const float *comb_part; __nv_bfloat16 *comb_out; size_t comb_o_ls;
  int comb_rows, comb_nchunk, comb_Tq, comb_BH, comb_H, comb_d;
};

__device__ __forceinline__ unsigned ld_acquire_gpu(const unsigned *p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Wait (bounded) until the grid-barrier counter has reached `target`.
__device__ __forceinline__ bool chain_wait(const unsigned *bar, unsigned target, volatile int *abort_flag, int *err) {
  if (ld_acquire_gpu(bar) >= target) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 0;; ++it) {
    if (ld_acquire_gpu(bar) >= target) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(err, 1);
        return false;
      }
    }
  }
}

// pre_o / pre_u: the inputs of the out-projection's and the MLP-up epilogue, fetched before the accumulator wait -- the
// former come from earlier launches, the latter from the previous phase of this launch, so they are fetched once the phase
// is known to be open.
template <int BN>
__device__ __forceinline__ void chain_epilogue(int epi, const UmmaParams &p, const float *outs, int ew, int lane, int n_tile, int ks, int l, int ls,
                                               const SmallPre<BN, UEPI_RESID> &pre_o, const SmallPre<BN, UEPI_RELU2_BF16> &pre_u) {
  switch (epi) {
    case UEPI_F32: {
      SmallPre<BN, UEPI_F32> q;
      umma_epilogue_small_pre<BN, UEPI_F32>(p, ew, lane, n_tile, l, ls, q);
      umma_epilogue_small<BN, UEPI_F32>(p, outs, ew, lane, n_tile, ks, l, ls, q);
      break;
    }
    case UEPI_RELU2_BF16: umma_epilogue_small<BN, UEPI_RELU2_BF16>(p, outs, ew, lane, n_tile, ks, l, ls, pre_u); break;
    case UEPI_RESID: umma_epilogue_small<BN, UEPI_RESID>(p, outs, ew, lane, n_tile, ks, l, ls, pre_o); break;
    default: break;
  }
}

// grid = #SMs (cooperative), 320 threads, dynamic shared memory UmmaCfg<BN, 16>::kSmem.  Every phase has M <= 16 rows.
template <int BN>
__global__ void __launch_bounds__(kUmmaThreads, 1) k_umma_chain(const __grid_constant__ ChainParams cp) {
  using Cfg = UmmaCfg<BN, 16>;
  extern __shared__ unsigned char umma_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)umma_smem_raw + 1023) & ~(uintptr_t)1023);
  constexpr int S = Cfg::kStages;
  unsigned char *sA = smem;                                   // [S][16 x 128 B]; the A descriptor reads 64 rows from a slot
  unsigned char *sB = smem + (size_t)S * Cfg::kABytes;        // [S][BN x 128 B]
  float *outs = reinterpret_cast<float *>(sB + (size_t)S * Cfg::kBBytes);
  uint64_t *full = reinterpret_cast<uint64_t *>(reinterpret_cast<unsigned char *>(outs) + Cfg::kOuts);
  uint64_t *empty = full + S;
  uint64_t *accfull = empty + S, *accempty = accfull + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(accempty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = (int)gridDim.x;
  const int pre = cp.comb_rows > 0 ? 1 : 0;   // barriers before phase 0
  int *err = cp.p[0].err;
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

  // items of phase ph that this CTA runs: it_ = blockIdx.x + i * G, i < my_items
#define SNLP_CHAIN_PHASE(ph)                                                                 \
  const UmmaParams &p = cp.p[ph];                                                            \
  const int nkb1 = p.kslice / kUmmaBK, nkb = nkb1 * p.kfuse;                                 \
  const int n_items = p.Nt * p.ksplit * p.nl;                                                \
  const int my_items = (int)blockIdx.x < n_items ? (n_items - 1 - (int)blockIdx.x) / G + 1 : 0;
#define SNLP_CHAIN_ITEM(i)                                                                   \
  const int it_ = (int)blockIdx.x + (i) * G;                                                 \
  const int n_tile = it_ % p.Nt;                                                             \
  const int ks = (it_ / p.Nt) % p.ksplit;                                                    \
  const int li_ = it_ / (p.Nt * p.ksplit);                                                   \
  const int la = p.a_share > 1 ? (li_ / p.a_share) * p.a_share : li_ * p.kfuse;              \
  const int l = li_ * p.kfuse;

  if (warp == 0) {
    if (lane == 0) {
      int g = 0, issued = 0;
      bool ok = true;
      for (int ph = 0; ph < cp.nphase && ok; ++ph) {
        SNLP_CHAIN_PHASE(ph)
        (void)nkb;
        // The activation tiles of this phase may only be requested once the phase is open; its weight tiles go out at
        // once.  pend_*: the stages of this phase whose activation tile is still to be requested (at most S of them:
        // a stage cannot be reused before the product that reads it has run, and that needs its activations).
        bool open = ph == 0 && pre == 0;
        int pend_from = g;
        int pend_k0[S], pend_la[S];
        const unsigned target = (unsigned)(ph + pre) * (unsigned)G;
        const int kbox = cp.kbox;   // k-blocks per request (the same in every phase): kbox consecutive ring slots, signalled on the first one's barrier, handed back on the last one's
        auto flush = [&]() {
          asm volatile("fence.proxy.async;" ::: "memory");   // the other CTAs' stores, seen through the barrier, before the bulk copies that read them
          for (int q = pend_from; q < g; q += kbox)
            tma_load_4d(sA + (size_t)(q % S) * Cfg::kABytes, &cp.tmA[ph], &full[q % S], 0, 0, pend_k0[q % S] / kUmmaBK, pend_la[q % S]);
          pend_from = g;
        };
        for (int i = 0; i < my_items && ok; ++i) {
          SNLP_CHAIN_ITEM(i)
          for (int kb = 0; kb < nkb && ok; kb += kbox, g += kbox) {
            if (!open) {
              if (g - pend_from >= S) { ok = chain_wait(cp.bar, target, abort_flag, err); open = ok; if (ok) flush(); }
              else if (ld_acquire_gpu(cp.bar) >= target) { open = true; flush(); }
              if (!ok) break;
            }
            const int s = g % S;
            ok = mbar_wait(&empty[s + kbox - 1], ((g / S) & 1) ^ 1u, abort_flag, err);
            if (!ok) break;
            mbar_expect_tx(&full[s], (Cfg::kABytes + Cfg::kBBytes) * kbox);
            const int j = kb / nkb1, k0 = ks * p.kslice + (kb % nkb1) * kUmmaBK;   // j: layer inside a K-concatenated chunk
            tma_load_4d(sB + (size_t)s * Cfg::kBBytes, &cp.tmB[ph], &full[s], 0, n_tile * BN, k0 / kUmmaBK, p.l0 + l + j);
            if (open) tma_load_4d(sA + (size_t)s * Cfg::kABytes, &cp.tmA[ph], &full[s], 0, 0, k0 / kUmmaBK, la + j);
            else { pend_k0[s] = k0; pend_la[s] = la + j; }
            issued = g + kbox;
          }
        }
        if (ok && !open && pend_from < g) { ok = chain_wait(cp.bar, target, abort_flag, err); if (ok) flush(); }
      }
      if (*abort_flag) {
        // let the copies still in flight land before the CTA's shared memory is handed on (stages whose activation
        // tile was never requested cannot complete: their wait runs into its limit)
        const int first = issued > S ? issued - S : 0;
        for (int q = first; q < issued; q += cp.kbox) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(&full[q % S], (q / S) & 1) && global_ns() - t0 < kWaitLimitNs / 16) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(64, BN);
      int g = 0, n = 0;   // stages / items so far, over all phases
      bool ok = true;
      for (int ph = 0; ph < cp.nphase && ok; ++ph) {
        SNLP_CHAIN_PHASE(ph)
        (void)nkb1;
        for (int i = 0; i < my_items && ok; ++i, ++n) {
          const int b = n & 1;
          ok = mbar_wait(&accempty[b], ((n >> 1) & 1) ^ 1u, abort_flag, err);
          if (!ok) break;
          tc_fence_after();
          const uint32_t dcol = tmem_base + b * BN;
          for (int kb = 0; kb < nkb; kb += cp.kbox, g += cp.kbox) {   // one wait and one commit per request
            const int s = g % S;
            ok = mbar_wait(&full[s], (g / S) & 1, abort_flag, err);
            if (!ok) break;
            tc_fence_after();
            uint64_t da = umma_desc_sw128(smem_u32(sA + (size_t)s * Cfg::kABytes));
            uint64_t db = umma_desc_sw128(smem_u32(sB + (size_t)s * Cfg::kBBytes));
            for (int q = 0; q < cp.kbox; ++q, da += Cfg::kABytes >> 4, db += Cfg::kBBytes >> 4) {
#pragma unroll
              for (int k = 0; k < kUmmaBK / 16; ++k) umma_bf16(dcol, da + 2 * k, db + 2 * k, idesc, (kb | q | k) != 0);
            }
            umma_commit(&empty[s + cp.kbox - 1]);
          }
          if (ok) umma_commit(&accfull[b]);
        }
      }
    }
  } else {
    const int et = threadIdx.x - 64, ew = et >> 5, grp = ew >> 2;   // two warp groups share the columns
    const int quarter = warp & 3;
    int n = 0;
    bool alive = true;
    if (pre) {
      // merge the attention's chunk partials: one output row (128 head features) per group of four warps at a time
      const int grp4 = et >> 7, e = et & 127;
      for (int r = (int)blockIdx.x + G * grp4; r < cp.comb_rows; r += 2 * G) {
        const int t = r % cp.comb_Tq, pair = r / cp.comb_Tq, bh = pair % cp.comb_BH, l = pair / cp.comb_BH;
        const int b = bh / cp.comb_H, h = bh % cp.comb_H;
        const float v = attn_merge_row(cp.comb_part + (size_t)r * cp.comb_nchunk * kAttnPartStride, cp.comb_nchunk, e);
        cp.comb_out[(size_t)l * cp.comb_o_ls + (size_t)(b * cp.comb_Tq + t) * cp.comb_d + h * 128 + e] = __float2bfloat16_rn(v);
      }
      __threadfence();
      epi_bar_sync();
      if (et == 0) atomicAdd(cp.bar, 1u);
    }
    for (int ph = 0; ph < cp.nphase; ++ph) {
      SNLP_CHAIN_PHASE(ph)
      (void)nkb;
      for (int i = 0; i < my_items && alive; ++i, ++n) {
        SNLP_CHAIN_ITEM(i)
        const int b = n & 1;
        SmallPre<BN, UEPI_RESID> pre_o;
        SmallPre<BN, UEPI_RELU2_BF16> pre_u;
        if (cp.epi[ph] == UEPI_RESID) {
          umma_epilogue_small_pre<BN, UEPI_RESID>(p, ew, lane, n_tile, l, la, pre_o);
        } else if (cp.epi[ph] == UEPI_RELU2_BF16) {
          if (i == 0 && ph + pre > 0) {   // the row scales are the previous phase's results: wait until this phase is open
            bool open_ = true;
            if (et == 0) open_ = chain_wait(cp.bar, (unsigned)(ph + pre) * (unsigned)G, abort_flag, err);
            if (!epi_all(open_)) { alive = false; break; }
          }
          umma_epilogue_small_pre<BN, UEPI_RELU2_BF16>(p, ew, lane, n_tile, l, la, pre_u);
        }
        if (!epi_all(mbar_wait(&accfull[b], (n >> 1) & 1, abort_flag, err))) { alive = false; break; }
        tc_fence_after();
        const uint32_t tbase = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * BN;
        if (quarter == 0) {  // the token rows live in lanes 0..15; each group's quarter-0 warp moves half the columns
#pragma unroll 1
          for (int c = grp * (BN / 64); c < (grp + 1) * (BN / 64); ++c) {
            uint32_t r[32];
            tmem_ld32(tbase + c * 32, r);
            if (lane < 16) {
#pragma unroll
              for (int j = 0; j < 32; ++j) outs[lane * (BN + 1) + c * 32 + j] = __uint_as_float(r[j]);
            }
          }
        }
        tc_fence_before();
        epi_bar_sync();
        if (et == 0) mbar_arrive(&accempty[b]);
        chain_epilogue<BN>(cp.epi[ph], p, outs, ew, lane, n_tile, ks, l, la, pre_o, pre_u);
        epi_bar_sync();  // outs is reused by the next item
      }
      // This CTA's part of the phase is complete: publish its results and count it in.  A CTA counts itself into phase
      // ph only once that phase is open (with items of its own that is implied; without, it waits here), so that the
      // counter's value / #CTAs is always the number of completed phases.
      __threadfence();
      epi_bar_sync();
      if (et == 0) {
        if (ph + pre > 0 && my_items == 0 && alive) chain_wait(cp.bar, (unsigned)(ph + pre) * (unsigned)G, abort_flag, err);
        const unsigned old = atomicAdd(cp.bar, 1u);
        if (old == (unsigned)(cp.nphase + pre) * (unsigned)G - 1u) *cp.bar = 0u;   // the last arrival of the last phase: nobody polls any more
      }
    }
  }
#undef SNLP_CHAIN_PHASE
#undef SNLP_CHAIN_ITEM
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace snlp
