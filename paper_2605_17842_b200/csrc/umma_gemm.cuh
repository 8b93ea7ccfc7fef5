// Prefill-regime layer-batched GEMM on the 5th-generation tensor cores (sm_100a):
//   D[l][m][n] = sum_k A[l][m][k] * B[l][n][k]     A = activations [L][M][K] bf16, B = weights [L][N][K] bf16
// One CTA computes a 128 x BN tile of one layer.  Operand tiles (128 x 64 and BN x 64 bf16, 128-byte
// swizzle) are brought into a shared-memory ring by TMA (one elected thread), a second elected thread
// issues tcgen05.mma (UMMA 128 x BN x 16, fp32 accumulator in tensor memory) and releases ring slots with
// tcgen05.commit; four epilogue warps read the accumulator back with tcgen05.ld and apply the fused
// epilogue.  Every wait on an mbarrier is bounded: on expiry the kernel raises a flag in global memory,
// lets its copies in flight land, frees its tensor memory and returns.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace snlp {

// Epilogues.  The A operand of the QKV and MLP-up products is the *un-normalised* bf16 branch input; its
// RMSNorm is a per-row scalar, so it is applied to the accumulator row here (sum of squares of the row =
// sum of `nparts` partials written by the producing kernel, in fixed order).
//   UEPI_F32         c = acc
//   UEPI_RELU2_BF16  z = bf16(relu(rstd_row * acc)^2)                      (rstd_row = 1 if ssq == nullptr)
//   UEPI_QKV         per 128-wide head: y = rstd_row * acc; q,k: rotary + RMSNorm over the head; q -> q buffer,
//                    k,v -> the layer's key/value store at the row's position
//   UEPI_RESID       u = xm + kappa_l * acc;  a = acc (fp32, for the correction), ub = bf16(u), and the partial
//                    sum of u^2 over this CTA's BN columns -> ssq_out[l][n_tile][row]
enum { UEPI_F32 = 0, UEPI_RELU2_BF16 = 1, UEPI_QKV = 2, UEPI_RESID = 3 };

struct UmmaParams {
  int M, N, K;             // rows, columns, reduction length of one layer's product
  float *c;                // UEPI_F32 / UEPI_RESID: [nl][M][N] fp32
  __nv_bfloat16 *z;        // UEPI_RELU2_BF16: [nl][M][N] bf16;  UEPI_RESID: ub [nl][M][N] bf16
  size_t out_ls;           // layer stride of the outputs above (elements)
  int *err;                // device flag set to 1 when a bounded wait expires
  // row scale (UEPI_QKV, UEPI_RELU2_BF16)
  const float *ssq; int nparts; float eps;   // [nl][nparts][M] partial sums of squares of the A rows
  // UEPI_QKV
  __nv_bfloat16 *q; size_t q_ls;
  __nv_bfloat16 *kc, *vc; size_t kv_ls, kv_bs;
  int T, d; const int *pos_base; const float2 *rope; float qk_eps;
  // UEPI_RESID
  const float *xm; size_t xm_ls; const HcCoef *coef; float *ssq_out;   // ssq_out [nl][N/BN][M]
};

constexpr int kUmmaThreads = 192;   // warp 0: TMA, warp 1: MMA + TMEM allocation, warps 2-5: epilogue
constexpr int kUmmaBM = 128;
constexpr int kUmmaBK = 64;         // 64 bf16 = one 128-byte swizzle row
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.b32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises *abort_flag / *err) if the phase has not completed in time or
// another thread of the CTA has already given up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, int *err) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(err, 1);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *tm, uint64_t *bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t *slot, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 operands, fp32 accumulator; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive on an mbarrier once all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns of tensor memory -> 32 registers per thread (thread i = lane i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor for a K-major operand tile stored as rows of 128 bytes with the
// 128-byte swizzle (what TMA writes): 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);  // start address / 16
  d |= (uint64_t)1 << 16;                        // leading byte offset / 16 (not used by swizzled K-major tiles)
  d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset / 16: next 8-row group
  d |= (uint64_t)1 << 46;                        // descriptor version of sm_100
  d |= (uint64_t)2 << 61;                        // layout type: 128-byte swizzle
  return d;
}

// Instruction descriptor: D fp32, A and B bf16, both K-major, M x N tile.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

template <int BN>
struct UmmaCfg {
  static constexpr int kStages = BN == 256 ? 4 : 6;
  static constexpr int kABytes = kUmmaBM * kUmmaBK * 2;
  static constexpr int kBBytes = BN * kUmmaBK * 2;
  static constexpr int kSmem = kStages * (kABytes + kBBytes) + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// grid (N/BN, ceil(M/128), nl), 192 threads, dynamic shared memory UmmaCfg<BN>::kSmem.
// tmA: 3-D map over A {K, M, nl}, box {64, 128, 1}; tmB: 3-D map over B {K, N, nl}, box {64, BN, 1}; both
// bf16, 128-byte swizzle, out-of-range rows read as zero.
template <int BN, int EPI>
__global__ void __launch_bounds__(kUmmaThreads) k_umma_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                                                           UmmaParams p) {
  using Cfg = UmmaCfg<BN>;
  extern __shared__ unsigned char umma_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)umma_smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char *sA = smem;
  unsigned char *sB = smem + Cfg::kStages * Cfg::kABytes;
  uint64_t *full = reinterpret_cast<uint64_t *>(sB + Cfg::kStages * Cfg::kBBytes);
  uint64_t *empty = full + Cfg::kStages;
  uint64_t *accbar = empty + Cfg::kStages;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(accbar + 1);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tile = blockIdx.x, m_tile = blockIdx.y, l = blockIdx.z;
  const int nkb = p.K / kUmmaBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 1);
    }
    mbar_init(accbar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int kb = 0; kb < nkb; ++kb) {
        const int s = kb % Cfg::kStages;
        const uint32_t ph = (kb / Cfg::kStages) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag, p.err)) break;
        mbar_expect_tx(&full[s], Cfg::kABytes + Cfg::kBBytes);
        tma_load_3d(sA + s * Cfg::kABytes, &tmA, &full[s], kb * kUmmaBK, m_tile * kUmmaBM, l);
        tma_load_3d(sB + s * Cfg::kBBytes, &tmB, &full[s], kb * kUmmaBK, n_tile * BN, l);
        issued = kb + 1;
      }
      if (*abort_flag) {
        // let the copies still in flight land before the CTA's shared memory is handed on
        const int first = issued > Cfg::kStages ? issued - Cfg::kStages : 0;
        for (int kb = first; kb < issued; ++kb) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(&full[kb % Cfg::kStages], (kb / Cfg::kStages) & 1) && global_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kUmmaBM, BN);
      bool ok = true;
      for (int kb = 0; kb < nkb && ok; ++kb) {
        const int s = kb % Cfg::kStages;
        const uint32_t ph = (kb / Cfg::kStages) & 1;
        ok = mbar_wait(&full[s], ph, abort_flag, p.err);
        if (!ok) break;
        tc_fence_after();
        const uint64_t da = umma_desc_sw128(smem_u32(sA + s * Cfg::kABytes));
        const uint64_t db = umma_desc_sw128(smem_u32(sB + s * Cfg::kBBytes));
#pragma unroll
        for (int k = 0; k < kUmmaBK / 16; ++k)  // 16 bf16 = 32 bytes = 2 descriptor address units per step
          umma_bf16(tmem_base, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
        umma_commit(&empty[s]);
      }
      if (ok) umma_commit(accbar);
    }
  } else {
    const bool ok = mbar_wait(accbar, 0, abort_flag, p.err);
    tc_fence_after();
    if (ok) {
      const int quarter = warp & 3;  // tensor-memory lanes this warp may read: 32*quarter .. +31
      const int row = m_tile * kUmmaBM + quarter * 32 + lane;
      const bool live = row < p.M;
      const uint32_t tbase = tmem_base + ((uint32_t)(quarter * 32) << 16);
      float rstd = 1.f;
      if ((EPI == UEPI_QKV || EPI == UEPI_RELU2_BF16) && p.ssq != nullptr && live) {
        float ss = 0.f;
        for (int i = 0; i < p.nparts; ++i) ss += p.ssq[((size_t)l * p.nparts + i) * p.M + row];
        rstd = rsqrtf(ss / (float)p.K + p.eps);
      }
      if (EPI == UEPI_F32 || EPI == UEPI_RELU2_BF16) {
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(tbase + c * 32, r);
          if (live) {
            const size_t off = (size_t)l * p.out_ls + (size_t)row * p.N + (size_t)n_tile * BN + c * 32;
            if (EPI == UEPI_F32) {
              float4 *dst = reinterpret_cast<float4 *>(p.c + off);
#pragma unroll
              for (int j = 0; j < 8; ++j)
                dst[j] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                                     __uint_as_float(r[4 * j + 3]));
            } else {
              uint4 *dst = reinterpret_cast<uint4 *>(p.z + off);
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                uint32_t w[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                  const float a = fmaxf(__uint_as_float(r[8 * j + 2 * q]) * rstd, 0.f);
                  const float b = fmaxf(__uint_as_float(r[8 * j + 2 * q + 1]) * rstd, 0.f);
                  __nv_bfloat162 v = __floats2bfloat162_rn(a * a, b * b);
                  w[q] = *reinterpret_cast<uint32_t *>(&v);
                }
                dst[j] = make_uint4(w[0], w[1], w[2], w[3]);
              }
            }
          }
        }
      } else if (EPI == UEPI_RESID) {
        const float kappa = p.coef[l].kappa;
        float ss = 0.f;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(tbase + c * 32, r);
          if (live) {
            const size_t col = (size_t)n_tile * BN + c * 32;
            const size_t off = (size_t)l * p.out_ls + (size_t)row * p.N + col;
            const float4 *xs = reinterpret_cast<const float4 *>(p.xm + (size_t)l * p.xm_ls + (size_t)row * p.N + col);
            float4 *adst = reinterpret_cast<float4 *>(p.c + off);
            uint4 *udst = reinterpret_cast<uint4 *>(p.z + off);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              uint32_t w[4];
#pragma unroll
              for (int q = 0; q < 2; ++q) {
                const float4 x = xs[2 * j + q];
                const float a0 = __uint_as_float(r[8 * j + 4 * q]), a1 = __uint_as_float(r[8 * j + 4 * q + 1]);
                const float a2 = __uint_as_float(r[8 * j + 4 * q + 2]), a3 = __uint_as_float(r[8 * j + 4 * q + 3]);
                adst[2 * j + q] = make_float4(a0, a1, a2, a3);
                const float u0 = fmaf(kappa, a0, x.x), u1 = fmaf(kappa, a1, x.y), u2 = fmaf(kappa, a2, x.z), u3 = fmaf(kappa, a3, x.w);
                ss += u0 * u0 + u1 * u1 + u2 * u2 + u3 * u3;
                __nv_bfloat162 v0 = __floats2bfloat162_rn(u0, u1), v1 = __floats2bfloat162_rn(u2, u3);
                w[2 * q] = *reinterpret_cast<uint32_t *>(&v0);
                w[2 * q + 1] = *reinterpret_cast<uint32_t *>(&v1);
              }
              udst[j] = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
        if (live) p.ssq_out[((size_t)l * gridDim.x + n_tile) * p.M + row] = ss;
      } else {  // UEPI_QKV
        const int Tn = p.T, b = live ? row / Tn : 0, pos = *p.pos_base + (live ? row % Tn : 0);
#pragma unroll 1
        for (int hh = 0; hh < BN / 128; ++hh) {
          const int n = n_tile * BN + hh * 128, kind = n / p.d, hcol = n % p.d;
          const uint32_t tcol = tbase + hh * 128;
          __nv_bfloat16 *dst;
          if (kind == 0) dst = p.q + (size_t)l * p.q_ls + (size_t)row * p.d + hcol;
          else dst = (kind == 1 ? p.kc : p.vc) + (size_t)l * p.kv_ls + (size_t)b * p.kv_bs + (size_t)pos * p.d + hcol;
          if (kind == 2) {
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              uint32_t r[32];
              tmem_ld32(tcol + c * 32, r);
              if (live) {
                uint4 *o = reinterpret_cast<uint4 *>(dst + c * 32);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  uint32_t w[4];
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(r[8 * j + 2 * q]) * rstd, __uint_as_float(r[8 * j + 2 * q + 1]) * rstd);
                    w[q] = *reinterpret_cast<uint32_t *>(&v);
                  }
                  o[j] = make_uint4(w[0], w[1], w[2], w[3]);
                }
              }
            }
          } else {
            float ss = 0.f;  // rotation preserves the norm, so the head's sum of squares can be taken before it
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              uint32_t r[32];
              tmem_ld32(tcol + c * 32, r);
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float v = __uint_as_float(r[j]) * rstd;
                ss = fmaf(v, v, ss);
              }
            }
            const float rn = rsqrtf(ss * (1.f / 128.f) + p.qk_eps) * rstd;
            const float2 *cs = p.rope + (size_t)pos * 64;
#pragma unroll 1
            for (int c = 0; c < 2; ++c) {
              uint32_t lo[32], hi[32];
              tmem_ld32(tcol + c * 32, lo);
              tmem_ld32(tcol + 64 + c * 32, hi);
              if (live) {
                uint4 *o1 = reinterpret_cast<uint4 *>(dst + c * 32), *o2 = reinterpret_cast<uint4 *>(dst + 64 + c * 32);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  uint32_t w1[4], w2[4];
#pragma unroll
                  for (int q = 0; q < 4; ++q) {
                    const int i0 = 8 * j + 2 * q;
                    const float2 ca = cs[c * 32 + i0], cb = cs[c * 32 + i0 + 1];
                    const float xa1 = __uint_as_float(lo[i0]) * rn, xa2 = __uint_as_float(hi[i0]) * rn;
                    const float xb1 = __uint_as_float(lo[i0 + 1]) * rn, xb2 = __uint_as_float(hi[i0 + 1]) * rn;
                    __nv_bfloat162 y1 = __floats2bfloat162_rn(xa1 * ca.x - xa2 * ca.y, xb1 * cb.x - xb2 * cb.y);
                    __nv_bfloat162 y2 = __floats2bfloat162_rn(xa1 * ca.y + xa2 * ca.x, xb1 * cb.y + xb2 * cb.x);
                    w1[q] = *reinterpret_cast<uint32_t *>(&y1);
                    w2[q] = *reinterpret_cast<uint32_t *>(&y2);
                  }
                  o1[j] = make_uint4(w1[0], w1[1], w1[2], w1[3]);
                  o2[j] = make_uint4(w2[0], w2[1], w2[2], w2[3]);
                }
              }
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, BN);
}

// ---- host side: tensor maps -----------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 3-D bf16 map over [layers][rows][K] (K innermost), box {64, box_rows, 1}, 128-byte swizzle.
inline bool make_tmap_bf16(EncodeTiledFn fn, CUtensorMap *tm, const void *base, uint64_t K, uint64_t rows, uint64_t layers,
                           uint64_t layer_stride_elems, uint32_t box_rows) {
  cuuint64_t dims[3] = {K, rows, layers};
  cuuint64_t strides[2] = {K * 2, layer_stride_elems * 2};
  cuuint32_t box[3] = {(cuuint32_t)kUmmaBK, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace snlp
