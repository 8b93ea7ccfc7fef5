// Layer-batched grouped GEMM on the 5th-generation tensor cores (sm_100a), used by both regimes:
//   D[l][m][n] = sum_k A[l][m][k] * W[l][n][k]     A = activations [nl][M][K] bf16, W = stacked weights [L][N][K] bf16
// Persistent CTAs (one per SM) walk (row tile, column tile, K split, layer) items.  Operand tiles -- AM x 64
// activations and BN x 64 weights, 128-byte swizzle -- are brought into a shared-memory ring by TMA (one
// elected thread) that keeps running across item boundaries; a second elected thread issues tcgen05.mma
// (UMMA 128 x BN x 16 -- 64 x BN x 16 in the decode regime --, fp32 accumulators in tensor memory, two accumulators so the epilogue of one item
// overlaps the main loop of the next) and releases ring slots with tcgen05.commit; four epilogue warps read
// the accumulator back with tcgen05.ld and apply the fused epilogue.
//   AM = 128: prefill regime, one accumulator row per epilogue thread.
//   AM = 16 : decode regime (<= 16 rows).  The weights stay the 256-wide operand: a 64 x 256 x 16 instruction takes the
//             tensor pipe 128 cycles and covers 8 KB of weights (as many cycles as the 128-row form -- the time goes with
//             the columns -- but half the multiply-adds, which shows under the board's power cap; a 128-wide one takes
//             64 cycles for 4 KB, and the issuing thread spends 55-100 cycles per instruction of any shape), and the token
//             box is only 16 rows high (rows 16..63 of the A operand are whatever follows in shared memory and land in
//             accumulator rows nobody reads).  The kernel is then bound by the weight stream from HBM; the accumulator is
//             transposed through shared memory so all 256 epilogue threads work.
// Every wait on an mbarrier is bounded: on expiry the kernel raises a flag in global memory, lets its
// copies in flight land, frees its tensor memory and returns.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace snlp {

// Epilogues.  The A operand of the QKV, MLP-up and LM-head products is the *un-normalised* bf16 branch input;
// its RMSNorm is a per-row scalar, so it is applied to the accumulator row here (sum of squares of the row =
// sum of `nparts` partials written by the producing kernel, in fixed order).
//   UEPI_F32         c[ks] = acc                                           (K-split partial sums)
//   UEPI_RELU2_BF16  z = bf16(relu(rstd_row * acc)^2)
//   UEPI_QKV         per 128-wide head: y = rstd_row * acc; q,k: rotary + RMSNorm over the head; q -> q buffer,
//                    k,v -> the layer's key/value store at the row's position
//   UEPI_RESID       u = xm + kappa_l * acc;  c = acc (fp32, for the correction), z = bf16(u), and the partial
//                    sum of u^2 over this tile's BN columns -> ssq_out[l][n_tile][row]
//   UEPI_LMHEAD      v = rstd_row * acc; optional logits; per-tile argmax -> pm_val/pm_idx[row][n_tile]   (AM = 16 only)
enum { UEPI_F32 = 0, UEPI_RELU2_BF16 = 1, UEPI_QKV = 2, UEPI_RESID = 3, UEPI_LMHEAD = 4 };

struct UmmaParams {
  int M, N, K;             // rows, columns, reduction length of one layer's product
  int kslice, ksplit;      // K split: kslice = K / ksplit (a multiple of 64)
  int Mt, Nt, nl, l0;      // row tiles, column tiles, layers of the launch; l0 = first layer's coordinate in the weight map
  int nstages;             // ring depth
  // Fused chunks (several layers reading one input, App. C.3).  a_share > 1: the `nl` items' layers are grouped in
  // chunks of a_share and every layer of a chunk reads the A rows (and their sums of squares) of the chunk's first
  // layer -- the column-concatenated form (QKV, MLP up).  kfuse > 1: an item is a chunk; its reduction runs over the
  // kfuse layers' A rows and weights in turn and accumulates into one output -- the K-concatenated form
  // (attention out-projection, MLP down); outputs and epilogue inputs are indexed by the chunk's first layer.
  int a_share, kfuse;
  // Decode regime: k-blocks fetched by one bulk-tensor copy (1, 2 or 4; divides kslice / 64 and the ring depth).  One
  // thread requests the copies and one issues the products; each spends several hundred cycles per ring step whatever
  // the step's size (~590 per copy request, ~500 per k-block of four products with its barrier wait and commit), which
  // caps a CTA streaming 128-wide tiles one k-block at a time at ~55 GB/s.  With boxes of several k-blocks there is one
  // request, one wait and one commit per box.
  int kbox;
  float *c;                // UEPI_F32 / UEPI_RESID: [ksplit][nl][M][N] fp32
  __nv_bfloat16 *z;        // UEPI_RELU2_BF16: [nl][M][N] bf16;  UEPI_RESID: bf16(u) [nl][M][N]
  size_t out_ls, out_ss;   // layer / split stride of the outputs above (elements)
  int *err;                // device flag set to 1 when a bounded wait expires
  const float *ssq; int nparts; float eps;   // row scale: [nl][nparts][M] partial sums of squares of the A rows
  __nv_bfloat16 *q; size_t q_ls;             // UEPI_QKV
  __nv_bfloat16 *kc, *vc; size_t kv_ls, kv_bs;
  int T, d; const int *pos_base; const float2 *rope; float qk_eps;
  const float2 *rope_t; int rope_ld;  // rope transposed [hd/2][rope_ld], read by the prefill-regime epilogue (thread = row)
  const float *xm; size_t xm_ls; const HcCoef *coef; float *ssq_out;   // UEPI_RESID; ssq_out [nl][partials][M]
  float *logits; float *pm_val; int *pm_idx;                            // UEPI_LMHEAD
  // UEPI_LMHEAD, optional: the CTA that finishes last merges the per-tile maxima into argmax[M] (ties -> lowest
  // index) and then adds one to *bump (nullable).  lm_counter: zero on entry, left zero.
  // argmax_pp (nullable): the address of argmax is read from a device slot instead (replayed decode graphs).
  int32_t *argmax; int *bump; unsigned *lm_counter; int32_t *const *argmax_pp;
};

constexpr int kUmmaThreads = 320;   // warp 0: TMA, warp 1: MMA + TMEM allocation, warps 2-9: epilogue (two per TMEM lane quarter)
constexpr int kUmmaEpiThreads = 256;
constexpr int kUmmaBM = 128;
constexpr int kUmmaBK = 64;         // 64 bf16 = one 128-byte swizzle row
constexpr int kUmmaSmemBudget = 227 * 1024;  // the most one CTA may take
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
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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

__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *tm, uint64_t *bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(tm), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
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

// The same load without the wait: several loads may be in flight before one tmem_wait_ld().
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Barrier over the 256 epilogue threads (named barrier 1), plain and with an AND-reduced predicate: after a
// bounded wait every thread learns whether all of them got through, so they leave the item loop together.
__device__ __forceinline__ void epi_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ bool epi_all(bool v) {
  uint32_t out;
  asm volatile("{\n .reg .pred p, q;\n setp.ne.b32 q, %1, 0;\n bar.red.and.pred p, 1, 256, q;\n selp.b32 %0, 1, 0, p;\n}"
               : "=r"(out)
               : "r"((uint32_t)v)
               : "memory");
  return out != 0;
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

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

template <int BN, int AM>
struct UmmaCfg {
  static constexpr int kABytes = AM * kUmmaBK * 2;
  static constexpr int kBBytes = BN * kUmmaBK * 2;
  // decode regime: the transposed accumulator outs[16][BN+1]; prefill regime: one 32 x 32 fp32 staging tile per epilogue warp
  static constexpr int kOuts = AM == 16 ? 16 * (BN + 1) * 4 : 8 * 4096;
  static constexpr int kFixed = kOuts + 1024 /*alignment slack*/ + 512 /*barriers*/;
  static constexpr int kStagesMax = (kUmmaSmemBudget - kFixed) / (kABytes + kBBytes);
  // decode regime: a whole number of the largest boxes (4 k-blocks at BN = 128, 2 at BN = 256)
  static constexpr int kStages = AM == 16 ? (BN == 128 ? (kStagesMax / 4) * 4 : (kStagesMax / 2) * 2) : (kStagesMax > 10 ? 10 : kStagesMax);
  static constexpr int kSmem = kStages * (kABytes + kBBytes) + kFixed;
};

// ---- epilogue of the prefill regime: thread = accumulator row ----------------------------------------
// grp = 0/1: which half of the tile's columns (or which head of a 256-wide QKV tile) this warp owns.
template <int BN, int EPI>
__device__ __forceinline__ void umma_epilogue_rows(const UmmaParams &p, uint32_t tbase, int row, int n_tile, int ks, int l, int ls, int grp,
                                                   float4 *stg) {
  const bool live = row < p.M;
  float rstd = 1.f;
  if ((EPI == UEPI_QKV || EPI == UEPI_RELU2_BF16) && p.ssq != nullptr && live) {
    float ss = 0.f;
    for (int i = 0; i < p.nparts; ++i) ss += p.ssq[((size_t)ls * p.nparts + i) * p.M + row];
    rstd = rsqrtf(ss / (float)p.K + p.eps);
  }
  constexpr int kHalf = BN / 64;  // 32-column chunks per warp group
  if (EPI == UEPI_F32 || EPI == UEPI_RELU2_BF16) {
    // Each 32 x 32 chunk goes through the warp's staging tile (float4 slots XOR-swizzled by row, conflict-free both
    // ways) and is stored with 8 lanes per row, 4 rows per instruction: whole 128-byte (fp32) or 64-byte (bf16) runs
    // instead of 16 bytes per row.
    const int lane = threadIdx.x & 31, row0 = row - lane, rsub = lane >> 3, c4 = lane & 7;
#pragma unroll 1
    for (int c = grp * kHalf; c < (grp + 1) * kHalf; ++c) {
      uint32_t r[32];
      tmem_ld32(tbase + c * 32, r);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        float4 v = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
        if (EPI == UEPI_RELU2_BF16) {   // the row scale belongs to this thread's row: apply it before the transposition
          v.x = fmaxf(v.x * rstd, 0.f); v.y = fmaxf(v.y * rstd, 0.f); v.z = fmaxf(v.z * rstd, 0.f); v.w = fmaxf(v.w * rstd, 0.f);
          v.x *= v.x; v.y *= v.y; v.z *= v.z; v.w *= v.w;
        }
        stg[lane * 8 + (j ^ (lane & 7))] = v;
      }
      __syncwarp();
      const size_t col = (size_t)n_tile * BN + c * 32 + c4 * 4;
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int rr = it * 4 + rsub, grow = row0 + rr;
        if (grow < p.M) {
          const float4 v = stg[rr * 8 + (c4 ^ (rr & 7))];
          const size_t off = (size_t)l * p.out_ls + (size_t)grow * p.N + col;
          if (EPI == UEPI_F32) *reinterpret_cast<float4 *>(p.c + (size_t)ks * p.out_ss + off) = v;
          else *reinterpret_cast<uint2 *>(p.z + off) = make_uint2(pack_bf16x2(v.x, v.y), pack_bf16x2(v.z, v.w));
        }
      }
      __syncwarp();
    }
  } else if (EPI == UEPI_RESID) {
    // Ten bytes move per accumulator element here (x read, a and u written), so the accesses must be whole lines:
    // each 32 x 32 chunk goes through the warp's staging tile (float4 slots XOR-swizzled by row, conflict-free
    // both ways) and is then handled with 8 lanes per row, 4 rows per instruction.
    const float kappa = p.coef[l].kappa;
    const int lane = threadIdx.x & 31, row0 = row - lane, rsub = lane >> 3, c4 = lane & 7;
    float ss[8];
#pragma unroll
    for (int it = 0; it < 8; ++it) ss[it] = 0.f;
    // The residual-stream values of a chunk are fetched before anything of it is stored, and one chunk ahead:
    // interleaved with the stores they would be issued one at a time (the compiler must assume that a store may
    // alias the next load), which leaves the epilogue waiting on eight DRAM latencies per chunk.
    float4 xv[8], xn[8];
    auto load_x = [&](int c, float4 (&dst)[8]) {
      const size_t col = (size_t)n_tile * BN + c * 32 + c4 * 4;
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int grow = row0 + it * 4 + rsub;
        dst[it] = grow < p.M ? __ldg(reinterpret_cast<const float4 *>(p.xm + (size_t)l * p.xm_ls + (size_t)grow * p.N + col))
                             : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    };
    load_x(grp * kHalf, xn);
#pragma unroll 1
    for (int c = grp * kHalf; c < (grp + 1) * kHalf; ++c) {
#pragma unroll
      for (int it = 0; it < 8; ++it) xv[it] = xn[it];
      if (c + 1 < (grp + 1) * kHalf) load_x(c + 1, xn);
      uint32_t r[32];
      tmem_ld32(tbase + c * 32, r);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        stg[lane * 8 + (j ^ (lane & 7))] = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]), __uint_as_float(r[4 * j + 2]),
                                                       __uint_as_float(r[4 * j + 3]));
      __syncwarp();
      const size_t col = (size_t)n_tile * BN + c * 32 + c4 * 4;
#pragma unroll
      for (int it = 0; it < 8; ++it) {
        const int rr = it * 4 + rsub, grow = row0 + rr;
        if (grow < p.M) {
          const float4 a = stg[rr * 8 + (c4 ^ (rr & 7))];
          const size_t off = (size_t)l * p.out_ls + (size_t)grow * p.N + col;
          const float4 x = xv[it];
          *reinterpret_cast<float4 *>(p.c + off) = a;
          const float u0 = fmaf(kappa, a.x, x.x), u1 = fmaf(kappa, a.y, x.y), u2 = fmaf(kappa, a.z, x.z), u3 = fmaf(kappa, a.w, x.w);
          ss[it] += u0 * u0 + u1 * u1 + u2 * u2 + u3 * u3;
          *reinterpret_cast<uint2 *>(p.z + off) = make_uint2(pack_bf16x2(u0, u1), pack_bf16x2(u2, u3));
        }
      }
      __syncwarp();
    }
#pragma unroll
    for (int it = 0; it < 8; ++it) {  // the 8 lanes of a row hold its partial sums
      float v = ss[it];
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      v += __shfl_xor_sync(0xffffffffu, v, 2);
      v += __shfl_xor_sync(0xffffffffu, v, 4);
      const int grow = row0 + it * 4 + rsub;
      if (c4 == 0 && grow < p.M) p.ssq_out[(((size_t)l * p.Nt + n_tile) * 2 + grp) * p.M + grow] = v;
    }
  } else if (EPI == UEPI_QKV) {
    const int Tn = p.T, b = live ? row / Tn : 0, pos = *p.pos_base + (live ? row % Tn : 0);
#pragma unroll 1
    for (int hh = grp; hh < BN / 128; hh += 2) {   // a 256-wide tile holds two heads, one per warp group
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
              for (int q = 0; q < 4; ++q) w[q] = pack_bf16x2(__uint_as_float(r[8 * j + 2 * q]) * rstd, __uint_as_float(r[8 * j + 2 * q + 1]) * rstd);
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
        const float2 *cs = p.rope_t + pos;  // lanes hold consecutive positions: every table read is one coalesced line
        const size_t cld = (size_t)p.rope_ld;
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
                const float2 ca = __ldg(cs + (c * 32 + i0) * cld), cb = __ldg(cs + (c * 32 + i0 + 1) * cld);
                const float xa1 = __uint_as_float(lo[i0]) * rn, xa2 = __uint_as_float(hi[i0]) * rn;
                const float xb1 = __uint_as_float(lo[i0 + 1]) * rn, xb2 = __uint_as_float(hi[i0 + 1]) * rn;
                w1[q] = pack_bf16x2(xa1 * ca.x - xa2 * ca.y, xb1 * cb.x - xb2 * cb.y);
                w2[q] = pack_bf16x2(xa1 * ca.y + xa2 * ca.x, xb1 * cb.y + xb2 * cb.x);
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

// ---- epilogue of the decode regime: accumulator rows (tokens) already transposed into outs[16][BN+1] ----
// What an item's epilogue reads from global memory besides its accumulator (a warp serves tokens ew and ew + 8): row
// scales, the residual-stream values, the rotation-table entries.  Fetched by umma_epilogue_small_pre, which a kernel may
// call before it waits for the accumulator when those values come from an earlier launch, so that the round trip is
// over when the products are (the last item's epilogue of a launch or phase is on the critical path).
template <int BN, int EPI>
struct SmallPre {
  float rstd[2];
  float xv[2][EPI == UEPI_RESID ? BN / 32 : 1];
  float kappa;
  float2 c0[2], c1[2];
  int pos[2];
};

template <int BN, int EPI>
__device__ __forceinline__ void umma_epilogue_small_pre(const UmmaParams &p, int ew, int lane, int n_tile, int l, int ls, SmallPre<BN, EPI> &q) {
#pragma unroll
  for (int tt = 0; tt < 2; ++tt) {
    const int tok = ew + 8 * tt;
    q.rstd[tt] = 1.f;
    if (tok < p.M) {
      if ((EPI == UEPI_QKV || EPI == UEPI_RELU2_BF16 || EPI == UEPI_LMHEAD) && p.ssq != nullptr) {
        float ss = 0.f;
        for (int i = 0; i < p.nparts; ++i) ss += p.ssq[((size_t)ls * p.nparts + i) * p.M + tok];
        q.rstd[tt] = rsqrtf(ss / (float)p.K + p.eps);
      }
      if (EPI == UEPI_RESID) {
        const float *xs = p.xm + (size_t)l * p.xm_ls + (size_t)tok * p.N + (size_t)n_tile * BN;
#pragma unroll
        for (int j = 0; j < BN / 32; ++j) q.xv[tt][EPI == UEPI_RESID ? j : 0] = xs[lane + 32 * j];
      }
      if (EPI == UEPI_QKV) {
        const int pos = *p.pos_base + (tok % p.T);
        q.pos[tt] = pos;
        q.c0[tt] = p.rope[(size_t)pos * 64 + lane];
        q.c1[tt] = p.rope[(size_t)pos * 64 + lane + 32];
      }
    }
  }
  if (EPI == UEPI_RESID) q.kappa = p.coef[l].kappa;
}

// ew = epilogue warp 0..7, lane; one warp per token, lanes across the tile's columns.
template <int BN, int EPI>
__device__ __forceinline__ void umma_epilogue_small(const UmmaParams &p, const float *outs, int ew, int lane, int n_tile, int ks, int l, int ls,
                                                    const SmallPre<BN, EPI> &q) {
#pragma unroll
  for (int tt = 0; tt < 2; ++tt) {
    const int tok = ew + 8 * tt;
    if (tok >= p.M) break;
    const float *y = outs + tok * (BN + 1);
    const float rstd = q.rstd[tt];
    const size_t n0 = (size_t)n_tile * BN;
    if (EPI == UEPI_F32) {
      float *dst = p.c + (size_t)ks * p.out_ss + (size_t)l * p.out_ls + (size_t)tok * p.N + n0;
#pragma unroll
      for (int j = 0; j < BN / 32; ++j) dst[lane + 32 * j] = y[lane + 32 * j];
    } else if (EPI == UEPI_RELU2_BF16) {
      __nv_bfloat16 *dst = p.z + (size_t)l * p.out_ls + (size_t)tok * p.N + n0;
#pragma unroll
      for (int j = 0; j < BN / 32; ++j) {
        const float v = fmaxf(y[lane + 32 * j] * rstd, 0.f);
        dst[lane + 32 * j] = __float2bfloat16_rn(v * v);
      }
    } else if (EPI == UEPI_RESID) {
      const float kappa = q.kappa;
      float *adst = p.c + (size_t)l * p.out_ls + (size_t)tok * p.N + n0;
      __nv_bfloat16 *udst = p.z + (size_t)l * p.out_ls + (size_t)tok * p.N + n0;
      // (the residual-stream values were all fetched before: loads left between the stores below would be issued one at
      // a time, one memory round trip each, and this epilogue is on the path between two phases of a chained launch)
      const float *xv = q.xv[tt];
      // one partial sum of u^2 per 128 columns, so that 128- and 256-wide tiles leave the same numbers behind
#pragma unroll
      for (int h = 0; h < BN / 128; ++h) {
        float ss = 0.f;
#pragma unroll
        for (int j = 4 * h; j < 4 * h + 4; ++j) {
          const float a = y[lane + 32 * j];
          const float u = fmaf(kappa, a, xv[EPI == UEPI_RESID ? j : 0]);
          adst[lane + 32 * j] = a;
          udst[lane + 32 * j] = __float2bfloat16_rn(u);
          ss = fmaf(u, u, ss);
        }
        ss = warp_sum(ss);
        if (lane == 0) p.ssq_out[((size_t)l * p.Nt * (BN / 128) + n_tile * (BN / 128) + h) * p.M + tok] = ss;
      }
    } else if (EPI == UEPI_QKV) {
      const int b = tok / p.T, pos = q.pos[tt];
      // (the rotation-table entries of this position serve every head of the tile and were fetched before anything is
      // stored: a load that follows a store is not issued ahead of it)
      const float2 c0 = q.c0[tt], c1 = q.c1[tt];
#pragma unroll
      for (int hh = 0; hh < BN / 128; ++hh) {
        const int n = (int)n0 + hh * 128, kind = n / p.d, hcol = n % p.d;
        const float *yh = y + hh * 128;
        __nv_bfloat16 *dst;
        if (kind == 0) dst = p.q + (size_t)l * p.q_ls + (size_t)tok * p.d + hcol;
        else dst = (kind == 1 ? p.kc : p.vc) + (size_t)l * p.kv_ls + (size_t)b * p.kv_bs + (size_t)pos * p.d + hcol;
        if (kind == 2) {
#pragma unroll
          for (int j = 0; j < 4; ++j) dst[lane + 32 * j] = __float2bfloat16_rn(yh[lane + 32 * j] * rstd);
        } else {
          const float a1 = yh[lane] * rstd, a2 = yh[lane + 64] * rstd, b1 = yh[lane + 32] * rstd, b2 = yh[lane + 96] * rstd;
          const float ya1 = a1 * c0.x - a2 * c0.y, ya2 = a1 * c0.y + a2 * c0.x;
          const float yb1 = b1 * c1.x - b2 * c1.y, yb2 = b1 * c1.y + b2 * c1.x;
          const float ss = warp_sum(ya1 * ya1 + ya2 * ya2 + yb1 * yb1 + yb2 * yb2);
          const float rn = rsqrtf(ss * (1.f / 128.f) + p.qk_eps);
          dst[lane] = __float2bfloat16_rn(ya1 * rn);
          dst[lane + 64] = __float2bfloat16_rn(ya2 * rn);
          dst[lane + 32] = __float2bfloat16_rn(yb1 * rn);
          dst[lane + 96] = __float2bfloat16_rn(yb2 * rn);
        }
      }
    } else {  // UEPI_LMHEAD
      float bv = -INFINITY;
      int bi = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < BN / 32; ++j) {
        const int cidx = lane + 32 * j;
        const float v = y[cidx] * rstd;
        if (p.logits) p.logits[(size_t)tok * p.N + n0 + cidx] = v;
        if (v > bv) { bv = v; bi = (int)n0 + cidx; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      if (lane == 0) { p.pm_val[(size_t)tok * p.Nt + n_tile] = bv; p.pm_idx[(size_t)tok * p.Nt + n_tile] = bi; }
    }
  }
}

// grid = min(items, #SMs), 320 threads, dynamic shared memory UmmaCfg<BN, AM>::kSmem.
// tmA: 3-D map over A {K, M, nl}, box {64, AM, 1}; tmB: 3-D map over the stacked weights {K, N, L}, box {64, BN, 1};
// both bf16, 128-byte swizzle, rows outside the tensor read as zero.
template <int BN, int AM, int EPI>
__global__ void __launch_bounds__(kUmmaThreads, 1) k_umma_gemm(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                                                              UmmaParams p) {
  using Cfg = UmmaCfg<BN, AM>;
  extern __shared__ unsigned char umma_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)umma_smem_raw + 1023) & ~(uintptr_t)1023);
  const int S = p.nstages;
  unsigned char *sA = smem;                                   // [S][AM x 128 B]; the A descriptor reads 128 (decode regime: 64) rows from a slot
  unsigned char *sB = smem + (size_t)S * Cfg::kABytes;        // [S][BN x 128 B]   (>= 14 KB, so those reads stay in bounds)
  float *outs = reinterpret_cast<float *>(sB + (size_t)S * Cfg::kBBytes);
  uint64_t *full = reinterpret_cast<uint64_t *>(reinterpret_cast<unsigned char *>(outs) + Cfg::kOuts);
  uint64_t *empty = full + S;
  uint64_t *accfull = empty + S, *accempty = accfull + 2;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(accempty + 2);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nkb1 = p.kslice / kUmmaBK;      // k-blocks of one layer's K slice
  const int nkb = nkb1 * p.kfuse;           // k-blocks of one item
  const int n_items = p.Mt * p.Nt * p.ksplit * p.nl;
  const int my_items = (int)blockIdx.x < n_items ? (n_items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  constexpr uint32_t kTmemCols = 2 * BN;

  // item -> (row tile, column tile, K split, layer); row tiles fastest so that concurrent CTAs share a weight tile
#define SNLP_DECODE_ITEM(i)                                       \
  const int it_ = (int)blockIdx.x + (i) * (int)gridDim.x;         \
  const int m_tile = it_ % p.Mt;                                  \
  const int n_tile = (it_ / p.Mt) % p.Nt;                         \
  const int ks = (it_ / (p.Mt * p.Nt)) % p.ksplit;                \
  const int li_ = it_ / (p.Mt * p.Nt * p.ksplit);                 /* layer (or chunk) of the launch */ \
  const int la = p.a_share > 1 ? (li_ / p.a_share) * p.a_share : li_ * p.kfuse; /* A rows' layer slot */ \
  const int l = li_ * p.kfuse;                                    /* output / weight layer slot */

  // (decode regime: a request covers kbox consecutive k-blocks = kbox consecutive ring slots; it is signalled on the
  // first slot's barrier and handed back on the last slot's)
  const int kbox = AM == 16 ? p.kbox : 1;
  auto load_a = [&](int s, int k0, int m_tile, int layer) {
    if (AM == 16) tma_load_4d(sA + (size_t)s * Cfg::kABytes, &tmA, &full[s], 0, 0, k0 / kUmmaBK, layer);
    else tma_load_3d(sA + (size_t)s * Cfg::kABytes, &tmA, &full[s], k0, m_tile * kUmmaBM, layer);
  };
  auto load_b = [&](int s, int k0, int n_tile, int layer) {
    if (AM == 16) tma_load_4d(sB + (size_t)s * Cfg::kBBytes, &tmB, &full[s], 0, n_tile * BN, k0 / kUmmaBK, layer);
    else tma_load_3d(sB + (size_t)s * Cfg::kBBytes, &tmB, &full[s], k0, n_tile * BN, layer);
  };
  const int total_kb = my_items * nkb, npre = total_kb < S ? total_kb : S;   // the first ring-ful of k-blocks

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
    // The weight tiles of the first ring-ful of k-blocks depend on nothing -- not on the tensor-memory allocation the
    // rest of the CTA is waiting for below, not on an earlier kernel of the stream: this thread, which is also the
    // producer, requests them at once (under a programmatic dependent launch they stream in while the previous kernel
    // is still finishing).  The activation tiles of the same stages follow behind the dependency wait.
    for (int i = 0, gp = 0; gp < npre; ++i) {
      SNLP_DECODE_ITEM(i)
      (void)m_tile; (void)la;
      for (int kb = 0; kb < nkb && gp < npre; kb += kbox, gp += kbox) {
        const int j = kb / nkb1, k0 = ks * p.kslice + (kb % nkb1) * kUmmaBK;
        mbar_expect_tx(&full[gp], (Cfg::kABytes + Cfg::kBBytes) * kbox);   // the stages are empty: first use
        load_b(gp, k0, n_tile, p.l0 + l + j);
      }
    }
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Everything up to here, and the weight tiles requested above, depend on no earlier kernel of the stream.
  if (!(warp == 0 && lane == 0)) pdl_wait();

  if (warp == 0) {
    if (lane == 0) {
      int g = 0, issued = 0;
      bool ok = true;
      pdl_wait();
      for (int i = 0, gp = 0; gp < npre; ++i) {   // the activation tiles of the stages whose weights are already on their way
        SNLP_DECODE_ITEM(i)
        (void)n_tile; (void)l;
        for (int kb = 0; kb < nkb && gp < npre; kb += kbox, gp += kbox) {
          const int j = kb / nkb1, k0 = ks * p.kslice + (kb % nkb1) * kUmmaBK;
          load_a(gp, k0, m_tile, la + j);
        }
      }
      issued = npre;
      for (int i = npre / nkb; i < my_items && ok; ++i) {
        SNLP_DECODE_ITEM(i)
        for (int kb = (i == npre / nkb ? npre % nkb : 0); kb < nkb; kb += kbox) {
          g = i * nkb + kb;
          const int s = g % S;
          ok = mbar_wait(&empty[s + kbox - 1], ((g / S) & 1) ^ 1u, abort_flag, p.err);
          if (!ok) break;
          mbar_expect_tx(&full[s], (Cfg::kABytes + Cfg::kBBytes) * kbox);
          const int j = kb / nkb1, k0 = ks * p.kslice + (kb % nkb1) * kUmmaBK;   // j: layer inside a K-concatenated chunk
          load_a(s, k0, m_tile, la + j);
          load_b(s, k0, n_tile, p.l0 + l + j);
          issued = g + kbox;
        }
      }
      // every load of this CTA has been requested: what is left is its tail, so the next kernel of the stream may be
      // scheduled onto the SMs as they free up (it waits for this kernel to complete before it reads any result)
      pdl_trigger();
      if (*abort_flag) {
        // let the copies still in flight land before the CTA's shared memory is handed on
        const int first = issued > S ? issued - S : 0;
        for (int q = first; q < issued; q += kbox) {
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(&full[q % S], (q / S) & 1) && global_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(AM == 16 ? 64 : kUmmaBM, BN);
      int g = 0;
      bool ok = true;
      for (int i = 0; i < my_items && ok; ++i) {
        const int b = i & 1;
        ok = mbar_wait(&accempty[b], ((i >> 1) & 1) ^ 1u, abort_flag, p.err);
        if (!ok) break;
        tc_fence_after();
        const uint32_t dcol = tmem_base + b * BN;
        for (int kb = 0; kb < nkb; kb += kbox, g += kbox) {   // one wait and one commit per request
          const int s = g % S;
          ok = mbar_wait(&full[s], (g / S) & 1, abort_flag, p.err);
          if (!ok) break;
          tc_fence_after();
          uint64_t da = umma_desc_sw128(smem_u32(sA + (size_t)s * Cfg::kABytes));
          uint64_t db = umma_desc_sw128(smem_u32(sB + (size_t)s * Cfg::kBBytes));
          for (int q = 0; q < kbox; ++q, da += Cfg::kABytes >> 4, db += Cfg::kBBytes >> 4) {
#pragma unroll
            for (int k = 0; k < kUmmaBK / 16; ++k)  // 16 bf16 = 32 bytes = 2 descriptor address units per step
              umma_bf16(dcol, da + 2 * k, db + 2 * k, idesc, (kb | q | k) != 0);
          }
          umma_commit(&empty[s + kbox - 1]);
        }
        if (ok) umma_commit(&accfull[b]);
      }
    }
  } else {
    const int et = threadIdx.x - 64, ew = et >> 5, grp = ew >> 2;   // two warp groups share the columns
    const int quarter = warp & 3;  // tensor-memory lanes this warp may read: 32*quarter .. +31
    for (int i = 0; i < my_items; ++i) {
      SNLP_DECODE_ITEM(i)
      const int b = i & 1;
      if (EPI == UEPI_RESID && AM == kUmmaBM) {
        // While the tile's products are still being accumulated, pull the residual-stream lines this warp will add
        // into L2 (one 128-byte line per row and 32-column chunk), so the epilogue's reads do not wait on DRAM.
        const int prow = m_tile * kUmmaBM + quarter * 32 + lane;
        if (prow < p.M) {
          const float *px = p.xm + (size_t)l * p.xm_ls + (size_t)prow * p.N + (size_t)n_tile * BN + grp * (BN / 2);
#pragma unroll
          for (int c = 0; c < BN / 64; ++c) asm volatile("prefetch.global.L2 [%0];" ::"l"(px + c * 32));
        }
      }
      SmallPre<BN, EPI> pre;
      if (AM != kUmmaBM) umma_epilogue_small_pre<BN, EPI>(p, ew, lane, n_tile, l, la, pre);   // every input is an earlier launch's
      if (!epi_all(mbar_wait(&accfull[b], (i >> 1) & 1, abort_flag, p.err))) break;
      tc_fence_after();
      const uint32_t tbase = tmem_base + ((uint32_t)(quarter * 32) << 16) + b * BN;
      if (AM == kUmmaBM) {
        umma_epilogue_rows<BN, EPI>(p, tbase, m_tile * kUmmaBM + quarter * 32 + lane, n_tile, ks, l, la, grp,
                                    reinterpret_cast<float4 *>(outs) + ew * 256);
        tc_fence_before();
        epi_bar_sync();
        if (et == 0) mbar_arrive(&accempty[b]);
      } else {
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
        umma_epilogue_small<BN, EPI>(p, outs, ew, lane, n_tile, ks, l, la, pre);
        epi_bar_sync();  // outs is reused by the next item
      }
    }
    if (EPI == UEPI_LMHEAD && AM != kUmmaBM && (p.argmax != nullptr || p.argmax_pp != nullptr)) {
      // Greedy token: every CTA counts itself in once its partial maxima are out (also after a wait that ran out,
      // so that the counter always returns to zero); the last one merges the tiles.
      int *s_last = reinterpret_cast<int *>(outs);
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
          if (lane == 0) {
            amax[tok] = (unsigned)bi < (unsigned)p.N ? bi : 0;
            __threadfence_system();   // the token buffer may be mapped host memory that the host is watching
          }
        }
        if (et == 0) {
          if (p.bump != nullptr) *p.bump += 1;
          *p.lm_counter = 0u;
        }
      }
    }
  }
#undef SNLP_DECODE_ITEM
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
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

// 4-D bf16 map over the same [layers][rows][K] array with K split into k-blocks: dims {64, rows, K / 64, layers}, box
// {64, box_rows, kbox, 1}: one copy brings kbox consecutive k-blocks of box_rows rows, each laid out like a {64, box_rows} box
// of the 3-D map, one after the other.
inline bool make_tmap_bf16_kb(EncodeTiledFn fn, CUtensorMap *tm, const void *base, uint64_t K, uint64_t rows, uint64_t layers,
                              uint64_t layer_stride_elems, uint32_t box_rows, uint32_t kbox) {
  cuuint64_t dims[4] = {(cuuint64_t)kUmmaBK, rows, K / kUmmaBK, layers};
  cuuint64_t strides[3] = {K * 2, (cuuint64_t)kUmmaBK * 2, layer_stride_elems * 2};
  cuuint32_t box[4] = {(cuuint32_t)kUmmaBK, box_rows, kbox, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace snlp
