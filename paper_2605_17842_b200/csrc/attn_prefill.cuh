// Prefill-regime causal attention (bf16, head_dim 128) over the (query tile, sequence x head, layer) grid.
// One CTA = 64 query rows of one (layer, sequence, head); 4 warps x 16 rows.  Keys/values are walked in
// 64-row tiles, double-buffered in shared memory with cp.async; S = Q K^T and O += P V run on
// mma.sync m16n8k16 with fragments fetched by ldmatrix from XOR-swizzled tiles; the softmax is online, in
// fp32, with the probabilities fed to the second product straight from the accumulator registers.
// Query row t of the call sits at absolute position *pos_base + t and sees keys 0 .. *pos_base + t of the
// layer's own key/value store (so a chunked prefill against a cache uses the same kernel).
#pragma once
#include "common.cuh"

namespace snlp {

constexpr int kFaRows = 64;   // query rows per CTA
constexpr int kFaKeys = 64;   // keys per tile
constexpr int kFaSmem = (kFaRows + 4 * kFaKeys) * 128 * 2;  // Q + 2 x (K, V) tiles

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void *p) {
  const uint32_t s = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(s));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], const void *p) {
  const uint32_t s = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(s));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

// Tile element (row, 16-byte chunk c of 16) lives at chunk (c ^ (row & 7)) of its 256-byte row.
__device__ __forceinline__ __nv_bfloat16 *tile_ptr(__nv_bfloat16 *tile, int row, int chunk) {
  return tile + row * 128 + ((chunk ^ (row & 7)) << 3);
}

// Copy rows [r0, r0+64) of a [rows][d] matrix slice (128 columns starting at `src`) into a swizzled tile.
__device__ __forceinline__ void load_tile_async(__nv_bfloat16 *tile, const __nv_bfloat16 *src, size_t row_stride, int r0, int rows_valid) {
  for (int i = threadIdx.x; i < 64 * 16; i += 128) {
    const int r = i >> 4, c = i & 15;
    const bool ok = r0 + r < rows_valid;
    cp_async16(tile_ptr(tile, r, c), src + (size_t)(ok ? r0 + r : 0) * row_stride + c * 8, ok);
  }
}

// grid (ceil(T/64), B*H, nl), 128 threads, dynamic shared memory kFaSmem.
static __global__ void __launch_bounds__(128) k_attn_prefill(const __nv_bfloat16 *__restrict__ q, size_t q_ls,
                                                             const __nv_bfloat16 *__restrict__ kc, const __nv_bfloat16 *__restrict__ vc,
                                                             size_t kv_ls, size_t kv_bs, __nv_bfloat16 *__restrict__ out, size_t o_ls, int T,
                                                             int H, const int *__restrict__ pos_base) {
  extern __shared__ __align__(128) unsigned char fa_smem[];
  __nv_bfloat16 *sQ = reinterpret_cast<__nv_bfloat16 *>(fa_smem);
  __nv_bfloat16 *sK = sQ + kFaRows * 128;          // [2][64][128]
  __nv_bfloat16 *sV = sK + 2 * kFaKeys * 128;      // [2][64][128]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t4 = lane & 3;
  const int qt = gridDim.x - 1 - blockIdx.x /* longest tiles first */, bh = blockIdx.y, l = blockIdx.z, b = bh / H, h = bh % H, d = H * 128;
  const int pos0 = *pos_base, t0 = qt * kFaRows;
  const int n_keys = pos0 + T;                                              // valid rows of the key/value store
  const int last_q = (t0 + kFaRows - 1 < T ? t0 + kFaRows - 1 : T - 1);
  const int nkt = (pos0 + last_q) / kFaKeys + 1;                            // key tiles this query tile can see

  const __nv_bfloat16 *qsrc = q + (size_t)l * q_ls + (size_t)(b * T) * d + h * 128;
  const __nv_bfloat16 *ksrc = kc + (size_t)l * kv_ls + (size_t)b * kv_bs + h * 128;
  const __nv_bfloat16 *vsrc = vc + (size_t)l * kv_ls + (size_t)b * kv_bs + h * 128;
  load_tile_async(sQ, qsrc, d, t0, T);
  load_tile_async(sK, ksrc, d, 0, n_keys);
  load_tile_async(sV, vsrc, d, 0, n_keys);
  cp_async_commit();

  float o[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
  const float sl2 = 0.08838834764831845f * 1.4426950408889634f;  // 1/sqrt(128) * log2(e)
  const int qpos0 = pos0 + t0 + warp * 16 + g, qpos1 = qpos0 + 8;           // positions of this thread's two rows
  uint32_t qf[8][4];

  for (int j = 0; j < nkt; ++j) {
    const int buf = j & 1;
    cp_async_wait<0>();
    __syncthreads();
    if (j + 1 < nkt) {
      load_tile_async(sK + (buf ^ 1) * kFaKeys * 128, ksrc, d, (j + 1) * kFaKeys, n_keys);
      load_tile_async(sV + (buf ^ 1) * kFaKeys * 128, vsrc, d, (j + 1) * kFaKeys, n_keys);
      cp_async_commit();
    }
    if (j == 0) {
#pragma unroll
      for (int kk = 0; kk < 8; ++kk)
        ldsm_x4(qf[kk], tile_ptr(sQ, warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, kk * 2 + (lane >> 4)));
    }
    __nv_bfloat16 *tK = sK + buf * kFaKeys * 128, *tV = sV + buf * kFaKeys * 128;
    // ---- S = Q K^T (16 x 64 per warp) ----------------------------------------------------------
    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t kf[4];
        ldsm_x4(kf, tile_ptr(tK, np * 16 + (lane >> 4) * 8 + (lane & 7), kk * 2 + ((lane >> 3) & 1)));
        mma16816(s[2 * np], qf[kk], kf[0], kf[1]);
        mma16816(s[2 * np + 1], qf[kk], kf[2], kf[3]);
      }
    }
    // ---- scale, causal mask, online softmax ------------------------------------------------------
    const int key0 = j * kFaKeys;
    float mx0 = mrow[0], mx1 = mrow[1];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int key = key0 + nt * 8 + 2 * t4;
      s[nt][0] = key <= qpos0 ? s[nt][0] * sl2 : -INFINITY;
      s[nt][1] = key + 1 <= qpos0 ? s[nt][1] * sl2 : -INFINITY;
      s[nt][2] = key <= qpos1 ? s[nt][2] * sl2 : -INFINITY;
      s[nt][3] = key + 1 <= qpos1 ? s[nt][3] * sl2 : -INFINITY;
      mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
      mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float base0 = mx0 == -INFINITY ? 0.f : mx0, base1 = mx1 == -INFINITY ? 0.f : mx1;
    const float c0 = exp2f(mrow[0] - base0), c1 = exp2f(mrow[1] - base1);  // exp2(-inf) = 0 on the first tile
    mrow[0] = mx0;
    mrow[1] = mx1;
    float ps0 = 0.f, ps1 = 0.f;
    uint32_t pf[4][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const float p0 = exp2f(s[nt][0] - base0), p1 = exp2f(s[nt][1] - base0);
      const float p2 = exp2f(s[nt][2] - base1), p3 = exp2f(s[nt][3] - base1);
      ps0 += p0 + p1;
      ps1 += p2 + p3;
      pf[nt >> 1][(nt & 1) * 2] = pack2_bf16(p0, p1);
      pf[nt >> 1][(nt & 1) * 2 + 1] = pack2_bf16(p2, p3);
    }
    lrow[0] = lrow[0] * c0 + ps0;
    lrow[1] = lrow[1] * c1 + ps1;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      o[i][0] *= c0; o[i][1] *= c0;
      o[i][2] *= c1; o[i][3] *= c1;
    }
    // ---- O += P V (16 x 128 per warp) --------------------------------------------------------------
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
      for (int np = 0; np < 8; ++np) {
        uint32_t vf[4];
        ldsm_x4_trans(vf, tile_ptr(tV, kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7), np * 2 + (lane >> 4)));
        mma16816(o[2 * np], pf[kk], vf[0], vf[1]);
        mma16816(o[2 * np + 1], pf[kk], vf[2], vf[3]);
      }
    }
  }
  // ---- normalise and store ---------------------------------------------------------------------------
  float l0 = lrow[0], l1 = lrow[1];
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
  const int r0 = t0 + warp * 16 + g, r1 = r0 + 8;
  __nv_bfloat16 *obase = out + (size_t)l * o_ls + (size_t)(b * T) * d + h * 128;
#pragma unroll
  for (int nt = 0; nt < 16; ++nt) {
    const int col = nt * 8 + 2 * t4;
    if (r0 < T) *reinterpret_cast<uint32_t *>(obase + (size_t)r0 * d + col) = pack2_bf16(o[nt][0] * i0, o[nt][1] * i0);
    if (r1 < T) *reinterpret_cast<uint32_t *>(obase + (size_t)r1 * d + col) = pack2_bf16(o[nt][2] * i1, o[nt][3] * i1);
  }
}

}  // namespace snlp
