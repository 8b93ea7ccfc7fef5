// Decode-regime attention (at most 16 query rows per sequence, bf16 operands, head_dim 128): split-KV causal
// attention over the (chunk, batch x head, layer) grid; a sweep streams every layer's keys/values from HBM once.
#pragma once
#include "common.cuh"

namespace snlp {

__device__ __forceinline__ uint4 ldg_stream(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
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

// One output row from the chunk partials of its (layer, sequence, head, query): the chunks are merged in chunk order.
// src: [nchunk][kAttnPartStride]; e = the head feature this thread produces.  Used by k_attn_decode's last-arriver
// merge and by the chained launch that follows the attention, so both give the same bits.
__device__ __forceinline__ float attn_merge_row(const float *src, int nchunk, int e) {
  constexpr int NC = 16;
  if (nchunk <= NC) {
    // every operand requested before the first is used: one memory round trip instead of two (same arithmetic, same order)
    float mc[NC], oc[NC], dc[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      if (c < nchunk) {
        mc[c] = __ldcg(src + (size_t)c * kAttnPartStride + 128);
        oc[c] = __ldcg(src + (size_t)c * kAttnPartStride + e);
        dc[c] = __ldcg(src + (size_t)c * kAttnPartStride + 129);
      }
    }
    float M = -INFINITY;
#pragma unroll
    for (int c = 0; c < NC; ++c)
      if (c < nchunk) M = fmaxf(M, mc[c]);
    float o = 0.f, den = 0.f;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      if (c < nchunk) {
        const float w = mc[c] == -INFINITY ? 0.f : __expf(mc[c] - M);
        o = fmaf(w, oc[c], o);
        den = fmaf(w, dc[c], den);
      }
    }
    return o / den;
  }
  float M = -INFINITY;
  for (int c = 0; c < nchunk; ++c) M = fmaxf(M, __ldcg(src + (size_t)c * kAttnPartStride + 128));
  float o = 0.f, den = 0.f;
  for (int c = 0; c < nchunk; ++c) {
    const float mc = __ldcg(src + (size_t)c * kAttnPartStride + 128);
    const float w = mc == -INFINITY ? 0.f : __expf(mc - M);
    o = fmaf(w, __ldcg(src + (size_t)c * kAttnPartStride + e), o);
    den = fmaf(w, __ldcg(src + (size_t)c * kAttnPartStride + 129), den);
  }
  return o / den;
}

// merge_here == 0: the CTAs only leave their chunk partials behind (the kernel that follows merges them); no fence, no
// arrival counter, no tail.
static __global__ void __launch_bounds__(128, 4) k_attn_decode(const __nv_bfloat16 *__restrict__ q, size_t q_ls,
                                                        const __nv_bfloat16 *__restrict__ kc, const __nv_bfloat16 *__restrict__ vc,
                                                        size_t kv_ls, size_t kv_bs, float *__restrict__ part,
                                                        unsigned *__restrict__ counters, __nv_bfloat16 *__restrict__ out,
                                                        size_t o_ls, int Tq, int H, const int *__restrict__ pos_base, int csub, int merge_here) {
  __shared__ float qs[16][128];
  __shared__ float hacc[8][128];
  __shared__ float hm[8], hl[8];
  __shared__ bool s_last;
  pdl_wait();
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
  pdl_trigger();   // the chunk has been streamed: only the merge is left
  if (!merge_here) return;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = atomicAdd(&counters[(size_t)l * gridDim.y + bh], 1u) == (unsigned)nchunk - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int t = 0; t < Tq; ++t) {
    const float *src = pbase + (size_t)t * nchunk * kAttnPartStride;
    out[(size_t)l * o_ls + (size_t)(b * Tq + t) * d + h * 128 + tid] = __float2bfloat16_rn(attn_merge_row(src, nchunk, tid));
  }
  if (tid == 0) counters[(size_t)l * gridDim.y + bh] = 0u;
}

}  // namespace snlp
