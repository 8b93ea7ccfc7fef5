// Decode-regime kernels (at most 16 rows per layer, bf16 operands, head_dim 128): the sweep is bound by
// streaming every layer's weights and keys/values from HBM once.
//
//  k_gemv_mma   layer-batched weight-streaming "GEMV": y[l][tok][n] = sum_k x[l][tok][k] W[l][n][k].
//               The weights are the 16-row MMA operand (read once, 16-byte loads straight from global
//               memory into the fragment registers), the <= 16 tokens are the 8-wide operand staged in
//               shared memory, so the ALU cost is independent of the token count and a token's result
//               does not depend on how many other tokens are in the call (batch invariance).
//               Fused prologues: RMSNorm of the fp32 input row, residual add of the attention branch.
//               Fused epilogues: rotary + QK-norm + KV-cache append; ReLU^2 + bf16 cast; per-tile argmax.
//  k_attn_decode / k_attn_combine   split-KV causal attention over the (chunk, batch x head, layer) grid.
#pragma once
#include "common.cuh"

namespace snlp {

enum { PRO_BF16 = 0, PRO_NORM = 1, PRO_RESID_NORM = 2 };
enum { EPI_PARTIAL = 0, EPI_QKV = 1, EPI_RELU2 = 2, EPI_LMHEAD = 3 };

struct GemvParams {
  const __nv_bfloat16 *W; size_t w_ls;  // [nl][N][Kd]
  int N, Kd, kslice, M;
  // prologue
  const __nv_bfloat16 *xb; size_t xb_ls;            // PRO_BF16: [nl][M][Kd]
  const float *xf; size_t xf_ls, xf_rs; int nsum;   // PRO_NORM / PRO_RESID_NORM: fp32 rows (sum of nsum streams)
  const float *ap; size_t ap_ls, ap_ss; int ap_splits;  // PRO_RESID_NORM: attention-branch partials [S][nl][M][Kd]
  const HcCoef *coef;                               // indexed by blockIdx.z (already offset to the first layer)
  float eps;
  // epilogue
  float *out; size_t out_ls, out_ss;                // EPI_PARTIAL: [ksplit][nl][M][N]
  __nv_bfloat16 *zout; size_t z_ls;                 // EPI_RELU2:   [nl][M][N]
  __nv_bfloat16 *q; size_t q_ls;                    // EPI_QKV
  __nv_bfloat16 *kc, *vc; size_t kv_ls, kv_bs;
  int T, H; const int *pos_base; const float2 *rope; float qk_eps;
  float *logits; float *pm_val; int *pm_idx; int ntile;  // EPI_LMHEAD: logits [M][N] nullable, partial argmax [M][ntile]
};

__device__ __forceinline__ uint4 ldg_stream(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

constexpr int kGemvThreads = 256;
constexpr int kGemvRows = 128;   // weight rows per CTA: 8 warps x 16
constexpr int kGemvPad = 32;     // bf16 elements of padding per staged token row (64 B: conflict-free 16 B reads)
constexpr int kGemvUnroll = 8;   // 32-wide k steps kept in flight per thread (16 x 16 B loads)

// grid (N/128, ksplit, nl), 256 threads.  NT = number of 8-token tiles (1 or 2).
// Dynamic shared memory: NT*8*(kslice+32) bf16 + NT*8*129 floats + 16 floats.
template <int NT, int PRO, int EPI>
__global__ void __launch_bounds__(kGemvThreads) k_gemv_mma(GemvParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int xstride = p.kslice + kGemvPad;
  __nv_bfloat16 *xs = reinterpret_cast<__nv_bfloat16 *>(smem_raw);
  float *outs = reinterpret_cast<float *>(smem_raw + (size_t)NT * 8 * xstride * sizeof(__nv_bfloat16));
  float *rstd = outs + NT * 8 * (kGemvRows + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, ks = blockIdx.y, l = blockIdx.z;
  const int kbase = ks * p.kslice;
  const int g = lane >> 2, t = lane & 3;

  // ---- prologue: stage the token operand as bf16 ------------------------------------------------
  if (PRO == PRO_BF16) {
    const int vec_per_row = p.kslice >> 3;
    for (int i = tid; i < NT * 8 * vec_per_row; i += kGemvThreads) {
      const int tok = i / vec_per_row, v = i % vec_per_row;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (tok < p.M) val = *reinterpret_cast<const uint4 *>(p.xb + (size_t)l * p.xb_ls + (size_t)tok * p.Kd + kbase + v * 8);
      *reinterpret_cast<uint4 *>(xs + (size_t)tok * xstride + v * 8) = val;
    }
    if (tid < NT * 8) rstd[tid] = 1.f;
  } else {
    // one warp per token; kslice == Kd here
    for (int tok = warp; tok < NT * 8; tok += kGemvThreads / 32) {
      float ss = 0.f;
      if (tok < p.M) {
        const float *x = p.xf + (size_t)l * p.xf_ls + (size_t)tok * p.xf_rs;
        const float kappa = PRO == PRO_RESID_NORM ? p.coef[l].kappa : 0.f;
        for (int j = lane * 4; j < p.Kd; j += 128) {
          float4 v = *reinterpret_cast<const float4 *>(x + j);
          for (int s = 1; s < p.nsum; ++s) {
            const float4 w = *reinterpret_cast<const float4 *>(x + (size_t)s * p.Kd + j);
            v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
          }
          if (PRO == PRO_RESID_NORM) {
            const float *a = p.ap + (size_t)l * p.ap_ls + (size_t)tok * p.Kd + j;
            float4 as = *reinterpret_cast<const float4 *>(a);
            for (int s = 1; s < p.ap_splits; ++s) {
              const float4 w = *reinterpret_cast<const float4 *>(a + (size_t)s * p.ap_ss);
              as.x += w.x; as.y += w.y; as.z += w.z; as.w += w.w;
            }
            v.x += kappa * as.x; v.y += kappa * as.y; v.z += kappa * as.z; v.w += kappa * as.w;
          }
          ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
          uint2 pk = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
          *reinterpret_cast<uint2 *>(xs + (size_t)tok * xstride + j) = pk;
        }
        ss = warp_sum(ss);
        if (lane == 0) rstd[tok] = rsqrtf(ss / (float)p.Kd + p.eps);
      } else {
        for (int j = lane * 4; j < p.Kd; j += 128) *reinterpret_cast<uint2 *>(xs + (size_t)tok * xstride + j) = make_uint2(0, 0);
        if (lane == 0) rstd[tok] = 0.f;
      }
    }
  }
  __syncthreads();

  // ---- main loop: stream 16 weight rows per warp -------------------------------------------------
  float acc[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
  const int r0 = tile * kGemvRows + warp * 16;
  const __nv_bfloat16 *w0 = p.W + (size_t)l * p.w_ls + (size_t)(r0 + g) * p.Kd + kbase + t * 8;
  const __nv_bfloat16 *w1 = w0 + (size_t)8 * p.Kd;
  const __nv_bfloat16 *x0 = xs + (size_t)g * xstride + t * 8;
  for (int kk = 0; kk < p.kslice; kk += 32 * kGemvUnroll) {
    uint4 wa[kGemvUnroll], wb[kGemvUnroll];
#pragma unroll
    for (int u = 0; u < kGemvUnroll; ++u) {
      const int k = kk + 32 * u;
      if (k < p.kslice) {
        wa[u] = ldg_stream(w0 + k);
        wb[u] = ldg_stream(w1 + k);
      }
    }
#pragma unroll
    for (int u = 0; u < kGemvUnroll; ++u) {
      const int k = kk + 32 * u;
      if (k < p.kslice) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const uint4 xv = *reinterpret_cast<const uint4 *>(x0 + (size_t)nt * 8 * xstride + k);
          mma_bf16_16816(acc[nt], wa[u].x, wb[u].x, wa[u].y, wb[u].y, xv.x, xv.y);
          mma_bf16_16816(acc[nt], wa[u].z, wb[u].z, wa[u].w, wb[u].w, xv.z, xv.w);
        }
      }
    }
  }
  // accumulator (row g / g+8, token 2t / 2t+1) -> outs[token][row in tile]
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const int tk = nt * 8 + 2 * t, rr = warp * 16 + g;
    outs[(tk) * (kGemvRows + 1) + rr] = acc[nt][0];
    outs[(tk + 1) * (kGemvRows + 1) + rr] = acc[nt][1];
    outs[(tk) * (kGemvRows + 1) + rr + 8] = acc[nt][2];
    outs[(tk + 1) * (kGemvRows + 1) + rr + 8] = acc[nt][3];
  }
  __syncthreads();

  // ---- epilogues -----------------------------------------------------------------------------------
  const int n0 = tile * kGemvRows;
  if (EPI == EPI_PARTIAL) {
    for (int i = tid; i < p.M * kGemvRows; i += kGemvThreads) {
      const int tok = i >> 7, r = i & 127;
      p.out[(size_t)ks * p.out_ss + (size_t)l * p.out_ls + (size_t)tok * p.N + n0 + r] = outs[tok * (kGemvRows + 1) + r] * rstd[tok];
    }
  } else if (EPI == EPI_RELU2) {
    for (int i = tid; i < p.M * kGemvRows; i += kGemvThreads) {
      const int tok = i >> 7, r = i & 127;
      const float v = fmaxf(outs[tok * (kGemvRows + 1) + r] * rstd[tok], 0.f);
      p.zout[(size_t)l * p.z_ls + (size_t)tok * p.N + n0 + r] = __float2bfloat16_rn(v * v);
    }
  } else if (EPI == EPI_QKV) {
    // the tile is exactly one 128-wide head of q, k or v
    const int kind = tile / p.H, head = tile % p.H, d = p.H * 128;
    for (int tok = warp; tok < p.M; tok += kGemvThreads / 32) {
      const int b = tok / p.T, pos = *p.pos_base + (tok % p.T);
      const float *y = outs + tok * (kGemvRows + 1);
      const float rs = rstd[tok];
      __nv_bfloat16 *dst;
      if (kind == 0) dst = p.q + (size_t)l * p.q_ls + (size_t)tok * d + head * 128;
      else dst = (kind == 1 ? p.kc : p.vc) + (size_t)l * p.kv_ls + (size_t)b * p.kv_bs + (size_t)pos * d + head * 128;
      if (kind == 2) {
#pragma unroll
        for (int j = 0; j < 4; ++j) dst[lane + 32 * j] = __float2bfloat16_rn(y[lane + 32 * j] * rs);
      } else {
        const float2 c0 = p.rope[(size_t)pos * 64 + lane], c1 = p.rope[(size_t)pos * 64 + lane + 32];
        const float a1 = y[lane] * rs, a2 = y[lane + 64] * rs, b1 = y[lane + 32] * rs, b2 = y[lane + 96] * rs;
        const float ya1 = a1 * c0.x - a2 * c0.y, ya2 = a1 * c0.y + a2 * c0.x;
        const float yb1 = b1 * c1.x - b2 * c1.y, yb2 = b1 * c1.y + b2 * c1.x;
        const float ss = warp_sum(ya1 * ya1 + ya2 * ya2 + yb1 * yb1 + yb2 * yb2);
        const float r = rsqrtf(ss * (1.f / 128.f) + p.qk_eps);
        dst[lane] = __float2bfloat16_rn(ya1 * r);
        dst[lane + 64] = __float2bfloat16_rn(ya2 * r);
        dst[lane + 32] = __float2bfloat16_rn(yb1 * r);
        dst[lane + 96] = __float2bfloat16_rn(yb2 * r);
      }
    }
  } else {  // EPI_LMHEAD
    for (int tok = warp; tok < p.M; tok += kGemvThreads / 32) {
      const float *y = outs + tok * (kGemvRows + 1);
      const float rs = rstd[tok];
      float bv = -INFINITY;
      int bi = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int r = lane + 32 * j;
        const float v = y[r] * rs;
        if (p.logits) p.logits[(size_t)tok * p.N + n0 + r] = v;
        if (v > bv) { bv = v; bi = n0 + r; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
      }
      if (lane == 0) { p.pm_val[(size_t)tok * p.ntile + tile] = bv; p.pm_idx[(size_t)tok * p.ntile + tile] = bi; }
    }
  }
}

// Final argmax over the per-tile partials (ties -> lowest index).  One block per token.
// bump (nullable): a device counter incremented by one once per launch (the cache position after a decode step).
static __global__ void k_argmax_tiles(const float *__restrict__ pm_val, const int *__restrict__ pm_idx, int ntile, int32_t *__restrict__ out,
                                      int *__restrict__ bump = nullptr) {
  __shared__ float sv[32];
  __shared__ int si[32];
  const int tok = blockIdx.x;
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  for (int j = threadIdx.x; j < ntile; j += blockDim.x) {
    const float v = pm_val[(size_t)tok * ntile + j];
    const int ix = pm_idx[(size_t)tok * ntile + j];
    if (v > bv || (v == bv && ix < bi)) { bv = v; bi = ix; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (lane == 0) { sv[w] = bv; si[w] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int nw = (blockDim.x + 31) >> 5;
    for (int i = 1; i < nw; ++i)
      if (sv[i] > bv || (sv[i] == bv && si[i] < bi)) { bv = sv[i]; bi = si[i]; }
    out[tok] = bi == 0x7fffffff ? 0 : bi;
    if (bump != nullptr && tok == 0) *bump += 1;
  }
}

// ---------------------------------------------------------------------------------------------------
// Split-KV causal attention for <= 16 query rows per sequence.  A CTA owns one chunk of `csub` x 64
// consecutive key positions of one (layer, sequence, head) and walks it in 64-key sub-blocks with an
// online softmax; its 8 half-warps take interleaved keys and every lane holds 8 of the 128 head
// features (one 16-byte load per key row, K and V of a sub-block issued together).  The last CTA of a
// (layer, sequence, head) to finish merges the chunk partials in chunk order and writes the bf16
// output, so no second launch is needed; arrival order does not change the result.  Chunk boundaries
// are fixed multiples of the chunk length and a query's result never depends on the other queries in
// the call (batch invariance: a T = 1 decode step and a T = 9 verify block give identical rows).
// part: [(l*BH + bh)*Tq + t][nchunk][132] = 128 un-normalised outputs, running max, denominator.
constexpr int kAttnPartStride = 132;
constexpr int kAttnSub = 64;

static __global__ void __launch_bounds__(128, 4) k_attn_decode(const __nv_bfloat16 *__restrict__ q, size_t q_ls,
                                                        const __nv_bfloat16 *__restrict__ kc, const __nv_bfloat16 *__restrict__ vc,
                                                        size_t kv_ls, size_t kv_bs, float *__restrict__ part,
                                                        unsigned *__restrict__ counters, __nv_bfloat16 *__restrict__ out,
                                                        size_t o_ls, int Tq, int H, const int *__restrict__ pos_base, int csub) {
  __shared__ float qs[16][128];
  __shared__ float hacc[8][128];
  __shared__ float hm[8], hl[8];
  __shared__ bool s_last;
  const int chunk = blockIdx.x, nchunk = gridDim.x, bh = blockIdx.y, l = blockIdx.z;
  const int b = bh / H, h = bh % H, d = H * 128;
  const int pos0 = *pos_base, kbeg = chunk * csub * kAttnSub;
  const int tid = threadIdx.x, hw = tid >> 4, li = tid & 15;
  const float scale = 0.08838834764831845f;  // 1/sqrt(128)
  for (int i = tid; i < Tq * 128; i += 128) {
    const int t = i >> 7, e = i & 127;
    qs[t][e] = __bfloat162float(q[(size_t)l * q_ls + (size_t)(b * Tq + t) * d + h * 128 + e]) * scale;
  }
  __syncthreads();
  const __nv_bfloat16 *kp = kc + (size_t)l * kv_ls + (size_t)b * kv_bs + h * 128 + li * 8;
  const __nv_bfloat16 *vp = vc + (size_t)l * kv_ls + (size_t)b * kv_bs + h * 128 + li * 8;
  float *pbase = part + (size_t)((size_t)l * gridDim.y + bh) * Tq * nchunk * kAttnPartStride;
  for (int t = 0; t < Tq; ++t) {
    const int pos_q = pos0 + t;
    float *dst = pbase + ((size_t)t * nchunk + chunk) * kAttnPartStride;
    if (kbeg > pos_q) {  // whole chunk is in this query's future
      dst[tid] = 0.f;
      if (tid == 0) { dst[128] = -INFINITY; dst[129] = 0.f; }
      continue;
    }
    // query features and the output accumulator as fp32 pairs: the dot products and the value accumulation run on the
    // packed fp32 pipe (the kernel is limited by instruction issue as much as by bandwidth)
    unsigned long long qv2[4], acc2[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      qv2[i] = pk2(qs[t][li * 8 + 2 * i], qs[t][li * 8 + 2 * i + 1]);
      acc2[i] = pk2(0.f, 0.f);
    }
    float mrun = -INFINITY, lrun = 0.f;
    // The chunk is walked in 32-key mini-blocks (4 keys per half-warp), software-pipelined through two register
    // buffers: the loads of the next mini-block are in flight while the current one is reduced.
    constexpr int JM = 4;
    auto load_mb = [&](uint4 (&kr)[JM], uint4 (&vr)[JM], int base) {
#pragma unroll
      for (int j = 0; j < JM; ++j) {
        const int key = base + hw + 8 * j;
        const bool ok = key <= pos_q;
        kr[j] = ok ? ldg_stream(kp + (size_t)key * d) : make_uint4(0, 0, 0, 0);
        vr[j] = ok ? ldg_stream(vp + (size_t)key * d) : make_uint4(0, 0, 0, 0);
      }
    };
    auto reduce_mb = [&](const uint4 (&kr)[JM], const uint4 (&vr)[JM], int base) {
      float s[JM];
      float mloc = -INFINITY;
#pragma unroll
      for (int j = 0; j < JM; ++j) {
        const int key = base + hw + 8 * j;
        const __nv_bfloat162 *k2 = reinterpret_cast<const __nv_bfloat162 *>(&kr[j]);
        unsigned long long d2 = pk2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(k2[i]);
          d2 = fma2(qv2[i], pk2(f.x, f.y), d2);
        }
        float dlo, dhi;
        upk2(d2, dlo, dhi);
        float dot = dlo + dhi;
        dot += __shfl_xor_sync(0xffffffffu, dot, 8);
        dot += __shfl_xor_sync(0xffffffffu, dot, 4);
        dot += __shfl_xor_sync(0xffffffffu, dot, 2);
        dot += __shfl_xor_sync(0xffffffffu, dot, 1);
        s[j] = key <= pos_q ? dot : -INFINITY;
        mloc = fmaxf(mloc, s[j]);
      }
      if (mloc == -INFINITY) return;  // none of this half-warp's keys of the mini-block is visible
      const float mnew = fmaxf(mrun, mloc);
      const float resc = mrun == -INFINITY ? 0.f : __expf(mrun - mnew);
      lrun *= resc;
#pragma unroll
      for (int i = 0; i < 4; ++i) acc2[i] = mul2(acc2[i], pk2(resc, resc));
#pragma unroll
      for (int j = 0; j < JM; ++j) {
        const float pj = s[j] == -INFINITY ? 0.f : __expf(s[j] - mnew);
        lrun += pj;
        const __nv_bfloat162 *v2 = reinterpret_cast<const __nv_bfloat162 *>(&vr[j]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 f = __bfloat1622float2(v2[i]);
          acc2[i] = fma2(pk2(pj, pj), pk2(f.x, f.y), acc2[i]);
        }
      }
      mrun = mnew;
    };
    {
      const int vis = (pos_q - kbeg) / 32 + 1;                         // mini-blocks with at least one visible key
      const int nmb = vis < csub * (kAttnSub / 32) ? vis : csub * (kAttnSub / 32);
      uint4 ka[JM], va[JM], kb2[JM], vb2[JM];
      load_mb(ka, va, kbeg);
      for (int mb = 0; mb < nmb; mb += 2) {
        if (mb + 1 < nmb) load_mb(kb2, vb2, kbeg + (mb + 1) * 32);
        reduce_mb(ka, va, kbeg + mb * 32);
        if (mb + 1 < nmb) {
          if (mb + 2 < nmb) load_mb(ka, va, kbeg + (mb + 2) * 32);
          reduce_mb(kb2, vb2, kbeg + (mb + 1) * 32);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) upk2(acc2[i], hacc[hw][li * 8 + 2 * i], hacc[hw][li * 8 + 2 * i + 1]);
    if (li == 0) { hm[hw] = mrun; hl[hw] = lrun; }
    __syncthreads();
    {  // merge the 8 half-warps in index order
      float M = hm[0];
#pragma unroll
      for (int j = 1; j < 8; ++j) M = fmaxf(M, hm[j]);
      float o = 0.f, den = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float w = hm[j] == -INFINITY ? 0.f : __expf(hm[j] - M);
        o = fmaf(w, hacc[j][tid], o);
        den = fmaf(w, hl[j], den);
      }
      dst[tid] = o;
      if (tid == 0) { dst[128] = M; dst[129] = den; }
    }
    __syncthreads();
  }
  // ---- last CTA of this (layer, sequence, head) merges the chunks in chunk order --------------------
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(&counters[(size_t)l * gridDim.y + bh], 1u) == (unsigned)nchunk - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int t = 0; t < Tq; ++t) {
    const float *src = pbase + (size_t)t * nchunk * kAttnPartStride;
    float M = -INFINITY;
    for (int c = 0; c < nchunk; ++c) M = fmaxf(M, __ldcg(src + (size_t)c * kAttnPartStride + 128));
    float o = 0.f, den = 0.f;
    for (int c = 0; c < nchunk; ++c) {
      const float mc = __ldcg(src + (size_t)c * kAttnPartStride + 128);
      const float w = mc == -INFINITY ? 0.f : __expf(mc - M);
      o = fmaf(w, __ldcg(src + (size_t)c * kAttnPartStride + tid), o);
      den = fmaf(w, __ldcg(src + (size_t)c * kAttnPartStride + 129), den);
    }
    out[(size_t)l * o_ls + (size_t)(b * Tq + t) * d + h * 128 + tid] = __float2bfloat16_rn(o / den);
  }
  if (tid == 0) counters[(size_t)l * gridDim.y + bh] = 0u;
}

}  // namespace snlp
