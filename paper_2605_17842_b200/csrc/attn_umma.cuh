// Causal attention of the prefill regime on the 5th-generation tensor cores (head_dim 128, bf16).
//
// One work item = 128 consecutive query positions of one (layer, sequence, head); persistent CTAs (one per SM) walk
// the items, longest first.  Per 128-key tile:   S = Q K^T  (tcgen05.mma, 128 x 128 x 128, accumulator in tensor
// memory)  ->  softmax warps (thread = query row: no cross-thread reductions) read S, keep the running maximum and
// denominator, write P = exp2(S - max) as bf16 back into tensor memory over the scores they came from  ->
// O_tile = P V (tcgen05.mma with the A operand in tensor memory, V read as an MN-major operand straight from the
// [key][head_dim] tile TMA delivers), accumulated over the item's tiles in tensor memory.  The exponent uses a
// reference maximum per row that is only raised when a tile's maximum exceeds it by more than 2^8; then (rarely after
// the first tiles) the row's accumulator and denominator are rescaled in place, between two P V products.  The result
// O / l does not depend on the reference.  S/P are double-buffered by tile and O by item in tensor memory (4 x 128
// columns), K and V tiles in two-slot TMA rings, so the tensor pipe computes tile j+1's scores while tile j's
// probabilities are formed.  The MMAs of one issuing thread execute in order, so S_{j+2} (issued after P_j V_j)
// cannot overwrite P_j early.
//
// Roles: warp 0 = TMA producer, warp 1 = MMA issuer + tensor-memory owner, warps 4-11 = softmax: two warps per
// tensor-memory lane quarter, one for keys 0..63 of a tile (and head dims 0..63 of the output), one for keys 64..127
// (head dims 64..127); the two halves of a row exchange their maxima through shared memory once per tile.  The
// roles are aligned to warp groups so that setmaxnreg can hand the registers the first group does not need to the
// softmax groups (scores and accumulator of a row half live in registers).
// Every mbarrier wait is bounded (see mbar_wait); on a timeout the CTA raises the error flag, leaves its loops and
// frees its tensor memory.
#pragma once
#include "umma_gemm.cuh"

namespace snlp {

constexpr int kFuThreads = 384;   // warp group 0: TMA producer, MMA issuer (+ two idle warps); warp groups 1, 2: softmax
constexpr int kFuTile = 128;                         // query rows per item, keys per tile
constexpr int kFuPanel = kFuTile * 64 * 2;           // one [128 rows][64 bf16] swizzled panel: 16 KB
constexpr int kFuTileBytes = 2 * kFuPanel;           // a [128][128] bf16 tile = two panels
constexpr int kFuKSlots = 2;                         // key-tile ring (values: 2 slots, queries: 2 slots)
constexpr int kFuSmem = (4 + kFuKSlots) * kFuTileBytes + 1024 + 256 + 2 * 1024;  // Q x2, K, V x2 + alignment slack + barriers + row exchange

struct FaUmmaParams {
  int T, H, BH, nq, n_items;   // nq = ceil(T / 128) query tiles per sequence; n_items = nq * BH * layers
  const int *pos_base;         // device: absolute position of query 0
  int *err;
};

// Shared-memory descriptor of an MN-major operand: rows of 128 bytes = 64 consecutive MN elements of one K index,
// 128-byte swizzle; the next 8 K indices are 1024 bytes on, the next 64 MN elements `mn_stride` bytes on.
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t smem_addr, uint32_t mn_stride) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(mn_stride >> 4) << 16;   // leading byte offset: next swizzle atom along MN
  d |= (uint64_t)(1024 >> 4) << 32;        // stride byte offset: next group of 8 K indices
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// D[tmem] (+)= A[tmem] * B[smem]: the A operand (128 rows x 16 bf16, two per 32-bit column) read from tensor memory.
__device__ __forceinline__ void umma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// 32 registers per thread -> 32 lanes x 32 consecutive 32-bit columns of tensor memory (thread i = lane i); waits for completion.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
      "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
      "r"(r[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// shared -> global tile store (rows or columns outside the tensor are clipped), tracked by the thread's bulk group
__device__ __forceinline__ void tma_store_4d(const CUtensorMap *tm, const void *src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(tm), "r"(smem_u32(src)), "r"(c0),
               "r"(c1), "r"(c2), "r"(c3)
               : "memory");
}
__device__ __forceinline__ void tma_store_commit_and_wait_read() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// item -> (layer, sequence*head, query tile).  The query tiles of one (layer, sequence, head) are neighbours in the
// item order, so the CTAs that run at the same time share their key / value tiles through L2 (longest-first order
// would stream the whole key / value store once per query-tile index).  The tile index is rotated by the pair index,
// which spreads short and long items evenly over the round-robin assignment to CTAs.
#define SNLP_FA_ITEM(i)                                                  \
  const int it_ = (int)blockIdx.x + (i) * (int)gridDim.x;                \
  const int pair_ = it_ / p.nq;                                          \
  const int qt = (it_ % p.nq + pair_) % p.nq;                            \
  const int l = pair_ / p.BH, bh = pair_ % p.BH;                         \
  const int b = bh / p.H, h = bh % p.H;                                  \
  const int q_hi = (qt + 1) * kFuTile < p.T ? (qt + 1) * kFuTile : p.T;  \
  const int ntile = (pos0 + q_hi - 1) / kFuTile + 1;

// tmQ: 3-D map over q {d, B*T, layers}, box {64, 128, 1}; tmK / tmV: 4-D maps over the key / value stores
// {d, rows per sequence, B, layers}, box {64, 128, 1, 1}; tmO: the same form over the output {d, T, B, layers} (so that a
// ragged last query tile is clipped at its own sequence); all bf16 with the 128-byte swizzle, out-of-range rows read 0.
__global__ void __launch_bounds__(kFuThreads, 1) k_attn_umma(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                                                             const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                                                             FaUmmaParams p, int nl) {
  extern __shared__ unsigned char fa_smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)fa_smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char *sQ = smem, *sK = smem + 2 * kFuTileBytes, *sV = smem + (2 + kFuKSlots) * kFuTileBytes;
  uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (4 + kFuKSlots) * kFuTileBytes);
  uint64_t *q_full = bars, *q_empty = bars + 2, *k_full = bars + 4, *k_empty = bars + 7, *v_full = bars + 10, *v_empty = bars + 12;
  uint64_t *s_full = bars + 14, *p_full = bars + 16, *pv_done = bars + 18, *o_empty = bars + 19, *st_full = bars + 21;
  uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 23);
  volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
  float *xch = reinterpret_cast<float *>(smem + (4 + kFuKSlots) * kFuTileBytes + 256);   // [2 tile parities][2 halves][128 rows]: row maxima; slot 0 also carries the denominators at the end of an item

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int pos0 = *p.pos_base;
  const int my_items = (int)blockIdx.x < p.n_items ? (p.n_items - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
  constexpr uint32_t kTmemCols = 512;   // S x2 by tile (columns 0..255; P overwrites the first 64 columns of its S), O x2 by item (256..511)

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&q_full[s], 1); mbar_init(&q_empty[s], 2);   // emptied by the last score product and by the output store
      mbar_init(&st_full[s], 8);
      mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
      mbar_init(&s_full[s], 1); mbar_init(&p_full[s], 8);
      mbar_init(&o_empty[s], 8);
    }
    mbar_init(pv_done, 1);
    for (int s = 0; s < kFuKSlots; ++s) { mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish();
  }
  if (warp == 0 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmQ) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmK) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmV) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmO) : "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp < 4) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      bool ok = true;
      uint32_t gk = 0, gv = 0;   // key / value tiles issued so far (ring positions); keys run one tile ahead of values
      auto load_v = [&](int j, int b, int h, int l) -> bool {
        const int s = gv & 1;
        if (!mbar_wait(&v_empty[s], ((gv >> 1) & 1) ^ 1u, abort_flag, p.err)) return false;
        mbar_expect_tx(&v_full[s], kFuTileBytes);
        tma_load_4d(sV + s * kFuTileBytes, &tmV, &v_full[s], h * 128, j * kFuTile, b, l);
        tma_load_4d(sV + s * kFuTileBytes + kFuPanel, &tmV, &v_full[s], h * 128 + 64, j * kFuTile, b, l);
        ++gv;
        return true;
      };
      for (int i = 0; i < my_items && ok; ++i) {
        SNLP_FA_ITEM(i)
        const int qs = i & 1;
        ok = mbar_wait(&q_empty[qs], ((i >> 1) & 1) ^ 1u, abort_flag, p.err);
        if (!ok) break;
        mbar_expect_tx(&q_full[qs], kFuTileBytes);
        tma_load_3d(sQ + qs * kFuTileBytes, &tmQ, &q_full[qs], h * 128, b * p.T + qt * kFuTile, l);
        tma_load_3d(sQ + qs * kFuTileBytes + kFuPanel, &tmQ, &q_full[qs], h * 128 + 64, b * p.T + qt * kFuTile, l);
        for (int j = 0; j < ntile && ok; ++j, ++gk) {
          const int s = gk % kFuKSlots;
          ok = mbar_wait(&k_empty[s], ((gk / kFuKSlots) & 1) ^ 1u, abort_flag, p.err);
          if (!ok) break;
          mbar_expect_tx(&k_full[s], kFuTileBytes);
          tma_load_4d(sK + s * kFuTileBytes, &tmK, &k_full[s], h * 128, j * kFuTile, b, l);
          tma_load_4d(sK + s * kFuTileBytes + kFuPanel, &tmK, &k_full[s], h * 128 + 64, j * kFuTile, b, l);
          if (j >= 1) ok = load_v(j - 1, b, h, l);
        }
        if (ok) ok = load_v(ntile - 1, b, h, l);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc_s = umma_idesc_bf16(kFuTile, kFuTile);                // Q, K both K-major
      constexpr uint32_t idesc_o = umma_idesc_bf16(kFuTile, kFuTile) | (1u << 16);   // P K-major, V MN-major
      bool ok = true;
      uint32_t gs = 0, gp = 0;   // score tiles / PV tiles issued so far
      // The tiles of all items form one stream: the scores of tile t+1 are issued before P V of tile t, across item
      // boundaries too, so the softmax warps find the next item's first scores ready when they finish an item.
      bool pend = false, pend_first = false;   // a P V product waiting to be issued; is it the first of its item?
      int pend_item = 0;
      auto issue_pv = [&]() -> bool {
        const int s = gp & 1;
        bool w = mbar_wait(&v_full[s], (gp >> 1) & 1, abort_flag, p.err);
        w = w && mbar_wait(&p_full[s], (gp >> 1) & 1, abort_flag, p.err);
        if (pend_first) w = w && mbar_wait(&o_empty[pend_item & 1], ((pend_item >> 1) & 1) ^ 1u, abort_flag, p.err);   // item - 2 has been read out
        if (!w) return false;
        tc_fence_after();
        const uint32_t dcol = tmem_base + 2 * kFuTile + (pend_item & 1) * kFuTile;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {   // 16 keys per step = 8 packed columns of P
          const uint64_t db = umma_desc_sw128_mn(smem_u32(sV + s * kFuTileBytes + kk * 16 * 128), kFuPanel);
          umma_bf16_ta(dcol, tmem_base + s * kFuTile + kk * 8, db, idesc_o, !pend_first || kk != 0);
        }
        umma_commit(&v_empty[s]);
        umma_commit(pv_done);
        ++gp;
        pend = false;
        return true;
      };
      for (int i = 0; i < my_items && ok; ++i) {
        SNLP_FA_ITEM(i)
        (void)l; (void)b; (void)h; (void)qt;
        const int qs = i & 1;
        // do not hold the previous item's last P V back for a query tile that has not arrived yet
        if (pend && !mbar_try_wait(&q_full[qs], (i >> 1) & 1)) ok = issue_pv();
        if (ok) ok = mbar_wait(&q_full[qs], (i >> 1) & 1, abort_flag, p.err);
        if (!ok) break;
        for (int j = 0; j < ntile && ok; ++j) {
          {   // S_j = Q K_j^T
            const int s = gs & 1, ks = gs % kFuKSlots;
            // buffer s last held P of tile gs-2, whose P V product this thread has already issued
            ok = mbar_wait(&k_full[ks], (gs / kFuKSlots) & 1, abort_flag, p.err);
            if (!ok) break;
            tc_fence_after();
            const uint32_t dcol = tmem_base + s * kFuTile;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint64_t da = umma_desc_sw128(smem_u32(sQ + qs * kFuTileBytes + (kk >> 2) * kFuPanel)) + 2 * (kk & 3);
              const uint64_t db = umma_desc_sw128(smem_u32(sK + ks * kFuTileBytes + (kk >> 2) * kFuPanel)) + 2 * (kk & 3);
              umma_bf16(dcol, da, db, idesc_s, kk != 0);
            }
            umma_commit(&k_empty[ks]);
            umma_commit(&s_full[s]);
            if (j == ntile - 1) umma_commit(&q_empty[qs]);
            ++gs;
          }
          if (pend) ok = issue_pv();
          pend = true;
          pend_first = j == 0;
          pend_item = i;
        }
      }
      if (ok && pend) ok = issue_pv();
    }
  } else if (warp == 2) {
    // ---------------- output store: the finished tile, staged by the softmax warps in the item's query buffer ----------------
    if (lane == 0) {
      for (int i = 0; i < my_items; ++i) {
        SNLP_FA_ITEM(i)
        (void)ntile;
        const int qs = i & 1;
        if (!mbar_wait(&st_full[qs], (i >> 1) & 1, abort_flag, p.err)) break;
        tma_store_4d(&tmO, sQ + qs * kFuTileBytes, h * 128, qt * kFuTile, b, l);
        tma_store_4d(&tmO, sQ + qs * kFuTileBytes + kFuPanel, h * 128 + 64, qt * kFuTile, b, l);
        tma_store_commit_and_wait_read();
        mbar_arrive(&q_empty[qs]);
      }
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    // ---------------- softmax / accumulation: thread = (query row, half of the keys / head dims) ----------------
    const int quarter = warp & 3, row = quarter * 32 + lane, hf = (warp - 4) >> 2;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const float sl2 = 0.08838834764831845f * 1.4426950408889634f;   // 1/sqrt(128) * log2(e)
    bool ok = true;
    uint32_t g = 0;   // key tiles processed so far
    for (int i = 0; i < my_items; ++i) {
      SNLP_FA_ITEM(i)
      (void)l; (void)b; (void)h;
      const int t = qt * kFuTile + row;           // query position inside the sequence
      const int vis = pos0 + t;                   // last visible key
      float m = -INFINITY, lsum = 0.f;   // reference maximum (scaled, log2 domain) and denominator of this row half
      const uint32_t ocol = tmem_base + lane_base + 2 * kFuTile + (i & 1) * kFuTile + hf * 64;
      bool all_ok = true;
      for (int j = 0; j < ntile; ++j, ++g) {
        const int s = g & 1;
        float *mx_slot = xch + (g & 1) * 256;
        uint32_t sv[64];
        float alpha = 1.f, m_use = 0.f;
        const bool masked = j * kFuTile + kFuTile - 1 > pos0 + qt * kFuTile;   // some (row, key) of this tile is in the future
        const int k0 = j * kFuTile + hf * 64;
        if (ok) ok = mbar_wait(&s_full[s], (g >> 1) & 1, abort_flag, p.err);
        ok = __all_sync(0xffffffffu, ok);   // keep the warp together for the warp-wide tensor-memory accesses
        if (ok) {
          tc_fence_after();
          const uint32_t scol = tmem_base + lane_base + s * kFuTile + hf * 64;
          tmem_ld32_nowait(scol, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
          tmem_ld32_nowait(scol + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
          tmem_wait_ld();
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four independent chains
          if (masked) {
#pragma unroll
            for (int e = 0; e < 64; ++e) {
              const float v = k0 + e <= vis ? __uint_as_float(sv[e]) : -INFINITY;
              sv[e] = __float_as_uint(v);
              mx4[e & 3] = fmaxf(mx4[e & 3], v);
            }
          } else {
#pragma unroll
            for (int e = 0; e < 64; ++e) mx4[e & 3] = fmaxf(mx4[e & 3], __uint_as_float(sv[e]));
          }
          mx_slot[hf * 128 + row] = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        }
        all_ok = epi_all(ok);   // also the barrier of the exchange
        if (!all_ok) break;
        {
          // raise the row's reference only when this tile's maximum is more than 2^8 above it (both halves of the row
          // take the same decision from the same numbers)
          const float mx = fmaxf(mx_slot[row], mx_slot[128 + row]) * sl2;
          if (mx > m + 8.f) {
            alpha = fast_exp2(m - mx);   // m = -inf -> 0
            m = mx;
          }
          m_use = m == -INFINITY ? 0.f : m;   // a row with no visible key yet: all probabilities 0
        }
        {
          // P over the scores: this thread's 64 keys become 32 packed columns (hf * 32 ..) of its lane; every thread of
          // the row's two halves has its scores in registers by now (the exchange above was a barrier)
          float rs4[4] = {0.f, 0.f, 0.f, 0.f};
          uint32_t w[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float p0 = fast_exp2(fmaf(__uint_as_float(sv[2 * e]), sl2, -m_use));       // exp2(-inf) = 0 for masked keys
            const float p1 = fast_exp2(fmaf(__uint_as_float(sv[2 * e + 1]), sl2, -m_use));
            rs4[e & 3] += p0 + p1;
            w[e] = pack_bf16x2(p0, p1);
          }
          lsum = fmaf(lsum, alpha, (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]));
          // the previous tile's P V must have left the accumulator (and P's buffer) before either is touched
          if (j >= 1) ok = __all_sync(0xffffffffu, mbar_wait(pv_done, (g - 1) & 1, abort_flag, p.err));
          if (ok) {
            tc_fence_after();
            if (j >= 1 && __any_sync(0xffffffffu, alpha != 1.f)) {   // rescale this warp's rows of the accumulator in place
#pragma unroll 1
              for (int c = 0; c < 2; ++c) {
                uint32_t r[32];
                tmem_ld32(ocol + c * 32, r);
#pragma unroll
                for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                tmem_st32(ocol + c * 32, r);
              }
            }
            tmem_st32(tmem_base + lane_base + s * kFuTile + hf * 32, w);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_full[s]);
          }
        }
      }
      if (!all_ok) break;
      if (ok) ok = mbar_wait(pv_done, (g - 1) & 1, abort_flag, p.err);
      ok = __all_sync(0xffffffffu, ok);
      // denominators of the two halves of a row add up (both ran on the same sequence of reference maxima)
      float *l_slot = xch;   // free: the wait above returns only after every warp has read the last tile's maxima and stored its P
      l_slot[hf * 128 + row] = lsum;
      if (!epi_all(ok)) break;
      const float inv = 1.f / (l_slot[row] + l_slot[128 + row]);
      epi_bar_sync();   // l_slot is rewritten by the next item's first exchange
      {
        tc_fence_after();
        uint32_t r0[32], r1[32];
        tmem_ld32_nowait(ocol, r0);
        tmem_ld32_nowait(ocol + 32, r1);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&o_empty[i & 1]);
        // normalised row half -> the item's (no longer needed) query buffer, in the layout of a swizzled TMA box:
        // panel hf, row `row`, 16-byte chunks XOR-ed with the row
        unsigned char *srow = sQ + (i & 1) * kFuTileBytes + hf * kFuPanel + row * 128;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) w[e] = pack_bf16x2(__uint_as_float(r0[8 * q + 2 * e]) * inv, __uint_as_float(r0[8 * q + 2 * e + 1]) * inv);
          *reinterpret_cast<uint4 *>(srow + ((q ^ (row & 7)) * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) w[e] = pack_bf16x2(__uint_as_float(r1[8 * q + 2 * e]) * inv, __uint_as_float(r1[8 * q + 2 * e + 1]) * inv);
          *reinterpret_cast<uint4 *>(srow + (((4 + q) ^ (row & 7)) * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&st_full[i & 1]);
      }
    }
  }
#undef SNLP_FA_ITEM
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// 4-D bf16 map over a key / value store [layers][B][rows][d] (d innermost), box {64, 128, 1, 1}, 128-byte swizzle.
inline bool make_tmap_kv(EncodeTiledFn fn, CUtensorMap *tm, const void *base, uint64_t d, uint64_t rows, uint64_t B, uint64_t layers,
                         uint64_t batch_stride_elems, uint64_t layer_stride_elems) {
  cuuint64_t dims[4] = {d, rows, B, layers};
  cuuint64_t strides[3] = {d * 2, batch_stride_elems * 2, layer_stride_elems * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)kFuTile, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace snlp
