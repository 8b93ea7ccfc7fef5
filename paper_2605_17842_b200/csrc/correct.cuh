// Fused structured correction along the layer axis (Alg. 2 lines 8-10, Eq. 5), one coalesced pass
// over the trace: per (row, 4-column) thread a serial loop over the layers of the range; no
// dependency between threads along L.  Also produces the residual norms of Eq. (2) and, for mHC
// models, the two pre-mapped branch inputs of every layer for the next sweep.
#pragma once
#include "common.cuh"

namespace snlp {

struct CorrParams {
  float *trace;      // [L+1][M][n][d], updated in place for states l0+1 .. l0+nl
  const float *a;    // [a_splits][L][M][d] attention-branch outputs (partial sums over splits)
  const float *m;    // [m_splits][L][M][d] MLP-branch outputs
  size_t a_ss, m_ss; // split strides (elements)
  int a_splits, m_splits;
  int l0, nl, L;     // nl steps starting at state l0
  int lstep;         // layers per step: 1, or the number of fused layers of a chunk (states l0, l0+lstep, ...)
  int M, d;
  int mode;          // SNLP_MODE_*
  int skip_next;     // 1: no sweep follows, so the next sweep's branch inputs (xa, xm, xb, ssq_x) are not produced (k_correct only)
  int implicit_old;  // 1: the states after l0 have not been materialised yet and all equal state l0 (first pass after Alg. 2 line 5)
  const HcCoef *coef;
  float *xa, *xm;    // [L][M][d] pre-mapped inputs for the next sweep (n > 1 only); xa nullable (not needed where xb is read)
  __nv_bfloat16 *xb; // nullable: [L+1][M][d] bf16 copy of the next sweep's attention-branch input (h_l, or pa_l . x_l);
                     //           slot L = the LM-head input (sum of the streams of the last state)
  float *ssq_x;      //           [L+1][d/128][M] its row sums of squares, one partial per 128 columns
  float *partial;    // [nl][2][gridDim.x] scratch for the norms (nullable => no norms); k_correct_small: [blocks][nl][2]
  float *resnorm;    // [L][2] (entries l0 .. l0+nl-1 written)
  unsigned *counter; // zero on entry, left zero on exit
};

// float4 arithmetic on the packed fp32 pipe (two IEEE operations per instruction: same bits as the scalar forms, half
// the issue slots; the correction is issue-limited for n > 1 streams)
__device__ __forceinline__ float4 f4_add(float4 a, float4 b) {
  unsigned long long d0, d1;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d0) : "l"(pk2(a.x, a.y)), "l"(pk2(b.x, b.y)));
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d1) : "l"(pk2(a.z, a.w)), "l"(pk2(b.z, b.w)));
  float4 r;
  upk2(d0, r.x, r.y);
  upk2(d1, r.z, r.w);
  return r;
}
__device__ __forceinline__ float4 f4_sub(float4 a, float4 b) {
  unsigned long long d0, d1;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d0) : "l"(pk2(a.x, a.y)), "l"(pk2(b.x, b.y)));
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d1) : "l"(pk2(a.z, a.w)), "l"(pk2(b.z, b.w)));
  float4 r;
  upk2(d0, r.x, r.y);
  upk2(d1, r.z, r.w);
  return r;
}
__device__ __forceinline__ float4 f4_fma(float s, float4 a, float4 b) {
  unsigned long long d0, d1;
  const unsigned long long ss = pk2(s, s);
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d0) : "l"(ss), "l"(pk2(a.x, a.y)), "l"(pk2(b.x, b.y)));
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d1) : "l"(ss), "l"(pk2(a.z, a.w)), "l"(pk2(b.z, b.w)));
  float4 r;
  upk2(d0, r.x, r.y);
  upk2(d1, r.z, r.w);
  return r;
}
__device__ __forceinline__ float4 f4_scale(float s, float4 a) {
  unsigned long long d0, d1;
  const unsigned long long ss = pk2(s, s);
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d0) : "l"(ss), "l"(pk2(a.x, a.y)));
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d1) : "l"(ss), "l"(pk2(a.z, a.w)));
  float4 r;
  upk2(d0, r.x, r.y);
  upk2(d1, r.z, r.w);
  return r;
}
// explicit fused multiply-adds: the same bits in every kernel that takes a row's sum of squares, whatever the compiler
// would otherwise contract
__device__ __forceinline__ float f4_sq(float4 a) { return fmaf(a.w, a.w, fmaf(a.z, a.z, fmaf(a.y, a.y, a.x * a.x))); }

// Depth of the operand ring of k_correct (steps in flight per thread) and its shared-memory size.
__host__ __device__ constexpr int corr_depth(int ns) { return ns <= 1 ? 4 : (ns <= 4 ? 3 : 2); }
// floats per step of the staged mixing coefficients (A, c^a, c^m, next pre-maps), rounded up to whole float4
__host__ __device__ constexpr int corr_coef_stride(int ns) { return (ns * (ns + 4) + 3) / 4 * 4; }
__host__ __device__ constexpr size_t corr_ring_bytes(int ns, int threads) { return (size_t)corr_depth(ns) * (2 + ns) * threads * sizeof(float4); }

// NS = number of residual streams (compile time so the per-thread state stays in registers).
// The kernel is bound by HBM bandwidth and each thread's loop over the layers is a chain of dependent steps, so the
// operands of the next corr_depth(NS)-1 steps are kept in flight with cp.async into a per-thread ring in shared memory
// (a thread only ever reads its own slots, so no block barrier is involved).  With K-split branch outputs (a_splits or
// m_splits > 1) the operands are summed from global memory directly, one step ahead.
// Dynamic shared memory: corr_ring_bytes(NS, blockDim.x) + [warps][nl][2] floats (with norms) + [nl][corr_coef_stride(NS)] floats (NS > 1).
// NATIVE: the surrogate is the block's own affine map (IDN on a single stream, HCN on n streams), known at compile time.
template <int NS, bool NATIVE>
__global__ void __launch_bounds__(256, NS == 1 ? 4 : 2) k_correct(CorrParams p) {
  extern __shared__ float4 s_ring[];  // [depth][2 + NS][blockDim.x]
  constexpr int D = corr_depth(NS);
  float *s_norm = reinterpret_cast<float *>(s_ring + (size_t)D * (2 + NS) * blockDim.x);  // [warps][nl][2] (only with norms)
  const int d4 = p.d >> 2;
  const size_t total = (size_t)p.M * d4;
  const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const bool active = idx < total;
  const size_t row = active ? idx / d4 : 0;
  const int c4 = active ? (int)(idx % d4) : 0;
  const size_t Md4 = (size_t)p.M * d4;             // float4 per [M][d] plane
  const size_t state4 = Md4 * NS;                  // float4 per trace state
  const float4 *a4 = reinterpret_cast<const float4 *>(p.a);
  const float4 *m4 = reinterpret_cast<const float4 *>(p.m);
  float4 *tr4 = reinterpret_cast<float4 *>(p.trace);
  const size_t bm_off = row * d4 + c4;             // offset inside an [M][d] plane
  const size_t st_off = row * NS * d4 + c4;        // offset of stream 0 inside a state
  const bool native = NATIVE;  // direct form == the block itself
  const bool want_norm = p.partial != nullptr;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
  const bool ring = p.a_splits == 1 && p.m_splits == 1;
  const bool need_old = (want_norm || !native) && !p.implicit_old;   // the old next state enters only the residual norm and the surrogate forms
  // Mixing coefficients of every step in shared memory, [nl][kCoefStride]: A, c^a, c^m of the step's layer, then the
  // pre-maps of the layer after it (zero past the last layer).  Read back as broadcast vector loads: per step a
  // thread would otherwise issue one global load per coefficient.
  constexpr int kCoefStride = corr_coef_stride(NS);
  float *s_coef = s_norm + (want_norm ? (size_t)nwarp * p.nl * 2 : 0);
  if (NS > 1) {
    for (int idx = threadIdx.x; idx < p.nl * kCoefStride; idx += blockDim.x) {
      const int i = idx / kCoefStride, j = idx % kCoefStride;
      const int l = p.l0 + i * p.lstep, ln = l + p.lstep;
      float v = 0.f;
      if (j < NS * NS) v = p.coef[l].A[j];
      else if (j < NS * NS + NS) v = p.coef[l].ca[j - NS * NS];
      else if (j < NS * NS + 2 * NS) v = p.coef[l].cm[j - NS * NS - NS];
      else if (j < NS * NS + 3 * NS) v = ln < p.L ? p.coef[ln].pa[j - NS * NS - 2 * NS] : 0.f;
      else if (j < NS * NS + 4 * NS) v = ln < p.L ? p.coef[ln].pmra[j - NS * NS - 3 * NS] : 0.f;
      s_coef[idx] = v;
    }
    __syncthreads();
  }

  float4 oldp[NS], newp[NS];
  // operands of one step: branch outputs and the old next state
  float4 av_n, mv_n, oldn_n[NS];
  auto fetch = [&](int i, float4 &av, float4 &mv, float4 (&on)[NS]) {
    const int l = p.l0 + i * p.lstep, ln = l + p.lstep;
    av = a4[(size_t)l * Md4 + bm_off];
    for (int q = 1; q < p.a_splits; ++q) av = f4_add(av, a4[(size_t)q * (p.a_ss >> 2) + (size_t)l * Md4 + bm_off]);
    mv = m4[(size_t)l * Md4 + bm_off];
    for (int q = 1; q < p.m_splits; ++q) mv = f4_add(mv, m4[(size_t)q * (p.m_ss >> 2) + (size_t)l * Md4 + bm_off]);
#pragma unroll
    for (int r = 0; r < NS; ++r) on[r] = need_old ? tr4[(size_t)ln * state4 + st_off + (size_t)r * d4] : make_float4(0.f, 0.f, 0.f, 0.f);
  };
  auto slot = [&](int i, int k) { return s_ring + ((size_t)(i % D) * (2 + NS) + k) * blockDim.x + threadIdx.x; };
  auto issue = [&](int i) {  // start the copies of step i's operands into ring slot i % D
    if (active && i < p.nl) {
      const int l = p.l0 + i * p.lstep, ln = l + p.lstep;
      cp_async16(slot(i, 0), a4 + (size_t)l * Md4 + bm_off, true);
      cp_async16(slot(i, 1), m4 + (size_t)l * Md4 + bm_off, true);
      if (need_old) {
#pragma unroll
        for (int r = 0; r < NS; ++r) cp_async16(slot(i, 2 + r), tr4 + (size_t)ln * state4 + st_off + (size_t)r * d4, true);
      }
    }
    cp_async_commit();  // one group per step, empty or not, so the wait below can count groups
  };
  if (active) {
#pragma unroll
    for (int s = 0; s < NS; ++s) oldp[s] = newp[s] = tr4[(size_t)p.l0 * state4 + st_off + (size_t)s * d4];
    if (!ring && p.nl > 0) fetch(0, av_n, mv_n, oldn_n);
  }
  if (ring) {
#pragma unroll
    for (int i = 0; i < D - 1; ++i) issue(i);
  }
  for (int i = 0; i < p.nl; ++i) {
    const int l = p.l0 + i * p.lstep, ln = l + p.lstep;  // this step maps state l to state ln
    float rs = 0.f, hs = 0.f, xs = 0.f;
    if (ring) {
      issue(i + D - 1);       // its slot was read in the previous iteration
      cp_async_wait<D - 1>();  // step i's group has landed
      if (active) {
        av_n = *slot(i, 0);
        mv_n = *slot(i, 1);
#pragma unroll
        for (int r = 0; r < NS; ++r) oldn_n[r] = need_old ? *slot(i, 2 + r) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    if (active) {
      const float4 av = av_n, mv = mv_n;
      // this step's coefficients into registers once
      float cA[NS * NS], cca[NS], ccm[NS], cpa[NS], cpm[NS];
      if (NS > 1) {
        const float *sc = s_coef + (size_t)i * kCoefStride;
        if (NS % 4 == 0) {
          const float4 *sc4 = reinterpret_cast<const float4 *>(sc);
#pragma unroll
          for (int k = 0; k < NS * NS / 4; ++k) { const float4 t = sc4[k]; cA[4 * k] = t.x; cA[4 * k + 1] = t.y; cA[4 * k + 2] = t.z; cA[4 * k + 3] = t.w; }
#pragma unroll
          for (int k = 0; k < NS / 4; ++k) {
            const float4 t0 = sc4[NS * NS / 4 + k], t1 = sc4[NS * NS / 4 + NS / 4 + k], t2 = sc4[NS * NS / 4 + 2 * (NS / 4) + k], t3 = sc4[NS * NS / 4 + 3 * (NS / 4) + k];
            cca[4 * k] = t0.x; cca[4 * k + 1] = t0.y; cca[4 * k + 2] = t0.z; cca[4 * k + 3] = t0.w;
            ccm[4 * k] = t1.x; ccm[4 * k + 1] = t1.y; ccm[4 * k + 2] = t1.z; ccm[4 * k + 3] = t1.w;
            cpa[4 * k] = t2.x; cpa[4 * k + 1] = t2.y; cpa[4 * k + 2] = t2.z; cpa[4 * k + 3] = t2.w;
            cpm[4 * k] = t3.x; cpm[4 * k + 1] = t3.y; cpm[4 * k + 2] = t3.z; cpm[4 * k + 3] = t3.w;
          }
        } else {
#pragma unroll
          for (int k = 0; k < NS * NS; ++k) cA[k] = sc[k];
#pragma unroll
          for (int k = 0; k < NS; ++k) {
            cca[k] = sc[NS * NS + k];
            ccm[k] = sc[NS * NS + NS + k];
            cpa[k] = sc[NS * NS + 2 * NS + k];
            cpm[k] = sc[NS * NS + 3 * NS + k];
          }
        }
      }
      float4 oldn[NS], newn[NS], tilde[NS];
#pragma unroll
      for (int r = 0; r < NS; ++r) oldn[r] = p.implicit_old ? oldp[r] : oldn_n[r];   // implicit: every old state is the first one
      if (!ring && i + 1 < p.nl) fetch(i + 1, av_n, mv_n, oldn_n);  // the next step's loads overlap this step's arithmetic and stores
#pragma unroll
      for (int r = 0; r < NS; ++r) {
        if (NS == 1) {
          tilde[r] = f4_add(f4_add(oldp[0], av), mv);  // F_l(h_l^k) = (h + a) + m
        } else {
          float4 t = f4_scale(cA[r * NS], oldp[0]);
#pragma unroll
          for (int s = 1; s < NS; ++s) t = f4_fma(cA[r * NS + s], oldp[s], t);
          tilde[r] = f4_fma(ccm[r], mv, f4_fma(cca[r], av, t));
        }
      }
#pragma unroll
      for (int r = 0; r < NS; ++r) {
        if (!NATIVE && p.mode == 2) {
          newn[r] = tilde[r];                                        // A = 0
        } else if (NATIVE) {
          if (NS == 1) {
            newn[r] = f4_add(f4_add(newp[0], av), mv);               // prefix sum over depth
          } else {
            float4 t = f4_scale(cA[r * NS], newp[0]);
#pragma unroll
            for (int s = 1; s < NS; ++s) t = f4_fma(cA[r * NS + s], newp[s], t);
            newn[r] = f4_fma(ccm[r], mv, f4_fma(cca[r], av, t));   // affine scan with A_l
          }
        } else {
          newn[r] = f4_add(tilde[r], f4_sub(newp[r], oldp[r]));      // identity surrogate on n streams
        }
        const float4 rr = f4_sub(tilde[r], oldn[r]);
        rs += f4_sq(rr);
        hs += f4_sq(oldn[r]);
        tr4[(size_t)ln * state4 + st_off + (size_t)r * d4] = newn[r];
      }
      float4 nxt = newn[0];  // the next layer's attention-branch input
      if (NS > 1 && ln < p.L && !p.skip_next) {
        float4 sa = f4_scale(cpa[0], newn[0]), sm = f4_scale(cpm[0], newn[0]);
#pragma unroll
        for (int s = 1; s < NS; ++s) {
          sa = f4_fma(cpa[s], newn[s], sa);
          sm = f4_fma(cpm[s], newn[s], sm);
        }
        if (p.xa != nullptr) reinterpret_cast<float4 *>(p.xa)[(size_t)ln * Md4 + bm_off] = sa;
        reinterpret_cast<float4 *>(p.xm)[(size_t)ln * Md4 + bm_off] = sm;
        nxt = sa;
      }
      if (NS > 1 && ln == p.L) {  // after the last block: the LM head reads the sum of the streams
#pragma unroll
        for (int s = 1; s < NS; ++s) nxt = f4_add(nxt, newn[s]);
      }
      if (p.xb != nullptr && !p.skip_next) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(nxt.x, nxt.y), hi = __floats2bfloat162_rn(nxt.z, nxt.w);
        uint2 pk = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
        reinterpret_cast<uint2 *>(p.xb)[(size_t)ln * Md4 + bm_off] = pk;
        xs = f4_sq(nxt);
      }
#pragma unroll
      for (int r = 0; r < NS; ++r) { oldp[r] = oldn[r]; newp[r] = newn[r]; }
    }
    if (p.xb != nullptr && !p.skip_next) {
      // d is a multiple of 128 here, so the 32 lanes of a warp hold 128 consecutive columns of one row
      xs = warp_sum(xs);
      if (lane == 0 && active) p.ssq_x[((size_t)ln * (d4 >> 5) + (c4 >> 5)) * p.M + row] = xs;
    }
    if (want_norm) {
      // both sums in one butterfly: the upper half-warp hands its residual part to the lower one and takes the
      // state part in return, then each half reduces one quantity (lane 0: sum r^2, lane 16: sum h^2)
      const bool up = (lane & 16) != 0;
      float keep = up ? hs : rs;
      keep += __shfl_xor_sync(0xffffffffu, up ? rs : hs, 16);
      keep += __shfl_xor_sync(0xffffffffu, keep, 8);
      keep += __shfl_xor_sync(0xffffffffu, keep, 4);
      keep += __shfl_xor_sync(0xffffffffu, keep, 2);
      keep += __shfl_xor_sync(0xffffffffu, keep, 1);
      if ((lane & 15) == 0) s_norm[(warp * p.nl + i) * 2 + (up ? 1 : 0)] = keep;
    }
  }
  if (!want_norm) return;
  __syncthreads();
  for (int i = threadIdx.x; i < p.nl * 2; i += blockDim.x) {
    float s = 0.f;
    for (int w = 0; w < nwarp; ++w) s += s_norm[w * p.nl * 2 + i];
    p.partial[(size_t)i * gridDim.x + blockIdx.x] = s;  // [nl * 2][blocks]
  }
  __threadfence();
  __syncthreads();
  __shared__ bool last;
  if (threadIdx.x == 0) last = (atomicAdd(p.counter, 1u) == gridDim.x - 1);
  __syncthreads();
  if (!last) return;
  __threadfence();
  // The last block adds the per-block partials in a fixed order: one warp per output, its lanes striding over the
  // blocks, then a butterfly.  (One thread per output walking all blocks kept a single SM busy for tens of
  // microseconds after every other block had left.)
  for (int i = warp; i < p.nl * 2; i += nwarp) {
    double s = 0.0;
    for (unsigned b = lane; b < gridDim.x; b += 32) s += (double)__ldcg(&p.partial[(size_t)i * gridDim.x + b]);
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) p.resnorm[(size_t)(p.l0 + (i >> 1) * p.lstep) * 2 + (i & 1)] = (float)s;
  }
  if (threadIdx.x == 0) *p.counter = 0u;
}


// Branch inputs of layers l0 .. l0+nl-1 from the current trace, for the tensor-core path: xb = bf16 of the
// attention-branch input (h_l, or pa_l . x_l for mHC), its per-128-column sums of squares, and for mHC the
// fp32 MLP pre-map xm = pmra_l . x_l.  Used before the first sweep; afterwards k_correct keeps them current.
// grid (M, nl), d/4 threads (d a multiple of 128).
template <int NS>
__global__ void k_prep_rows(const float *__restrict__ trace, int l0, int M, int d, const HcCoef *__restrict__ coef,
                            __nv_bfloat16 *__restrict__ xb, float *__restrict__ ssq_x, float *__restrict__ xm) {
  pdl_trigger();
  pdl_wait();
  const int d4 = d >> 2, c4 = threadIdx.x, l = l0 + blockIdx.y;
  const size_t row = blockIdx.x, Md4 = (size_t)M * d4;
  const float4 *x = reinterpret_cast<const float4 *>(trace) + (size_t)l * Md4 * NS + row * NS * d4 + c4;
  float4 v = x[0];
  if (NS > 1) {
    const HcCoef &c = coef[l];
    float4 sa = f4_scale(c.pa[0], v), sm = f4_scale(c.pmra[0], v);
#pragma unroll
    for (int s = 1; s < NS; ++s) {
      const float4 xv = x[(size_t)s * d4];
      sa = f4_fma(c.pa[s], xv, sa);
      sm = f4_fma(c.pmra[s], xv, sm);
    }
    reinterpret_cast<float4 *>(xm)[(size_t)l * Md4 + row * d4 + c4] = sm;
    v = sa;
  }
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  reinterpret_cast<uint2 *>(xb)[(size_t)l * Md4 + row * d4 + c4] = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
  const float ss = warp_sum(f4_sq(v));
  if ((threadIdx.x & 31) == 0) ssq_x[((size_t)l * (d4 >> 5) + (c4 >> 5)) * M + row] = ss;
}

// Alg. 2 line 5 fused with the first branch inputs: every state l0+1 .. L starts as a copy of state l0, and layers
// l0 .. L-1 get their bf16 attention-branch input, its sums of squares and (mHC) the fp32 MLP pre-map, all from one read
// of the row.  Same values as k_bcast_trace followed by k_prep_rows.  grid (M), d/4 threads (d a multiple of 128).
// write_trace == 0 leaves the copies out: the first pass then reads state l0 wherever it needs a later state.
// ids != nullptr: state l0 itself is the embedding of the row's token (replicated into every stream) and is written
// here too, so that a decode step needs no separate embedding kernel.
template <int NS>
__global__ void k_init_rows(float *__restrict__ trace, int l0, int L, int M, int d, const HcCoef *__restrict__ coef,
                            __nv_bfloat16 *__restrict__ xb, float *__restrict__ ssq_x, float *__restrict__ xm, int write_trace,
                            const int32_t *__restrict__ ids = nullptr, const __nv_bfloat16 *__restrict__ table = nullptr, int vocab = 0,
                            const int32_t *const *__restrict__ ids_pp = nullptr) {
  pdl_trigger();
  pdl_wait();
  if (ids_pp != nullptr) ids = *ids_pp;   // the ids' address is read from a device slot (replayed decode graphs)
  const int d4 = d >> 2, c4 = threadIdx.x;
  const size_t row = blockIdx.x, Md4 = (size_t)M * d4;
  float4 *tr4 = reinterpret_cast<float4 *>(trace);
  float4 x[NS];
  if (ids != nullptr) {
    int id = ids[row];
    id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);
    const uint2 e = reinterpret_cast<const uint2 *>(table + (size_t)id * d)[c4];
    const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&e.x)), hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&e.y));
#pragma unroll
    for (int s = 0; s < NS; ++s) {
      x[s] = make_float4(lo.x, lo.y, hi.x, hi.y);
      tr4[(size_t)l0 * Md4 * NS + row * NS * d4 + (size_t)s * d4 + c4] = x[s];
    }
  } else {
#pragma unroll
    for (int s = 0; s < NS; ++s) x[s] = tr4[(size_t)l0 * Md4 * NS + row * NS * d4 + (size_t)s * d4 + c4];
  }
  float4 v = x[0];
  uint2 pk = make_uint2(0, 0);
  float ss = 0.f;
  for (int l = l0; l < L; ++l) {
    if (write_trace) {
#pragma unroll
      for (int s = 0; s < NS; ++s) tr4[(size_t)(l + 1) * Md4 * NS + row * NS * d4 + (size_t)s * d4 + c4] = x[s];
    }
    if (NS > 1) {
      const HcCoef &c = coef[l];
      float4 sa = f4_scale(c.pa[0], x[0]), sm = f4_scale(c.pmra[0], x[0]);
#pragma unroll
      for (int s = 1; s < NS; ++s) {
        sa = f4_fma(c.pa[s], x[s], sa);
        sm = f4_fma(c.pmra[s], x[s], sm);
      }
      reinterpret_cast<float4 *>(xm)[(size_t)l * Md4 + row * d4 + c4] = sm;
      v = sa;
    }
    if (NS > 1 || l == l0) {   // single stream: the same input for every layer
      __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
      pk = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
      ss = warp_sum(f4_sq(v));
    }
    reinterpret_cast<uint2 *>(xb)[(size_t)l * Md4 + row * d4 + c4] = pk;
    if ((threadIdx.x & 31) == 0) ssq_x[((size_t)l * (d4 >> 5) + (c4 >> 5)) * M + row] = ss;
  }
}

// LM-head input from arbitrary hidden-state rows: xb = bf16(sum of the NS streams), per-128-column sums of squares.
// grid (rows), d/4 threads.
__global__ void k_prep_lm(const float *__restrict__ h, size_t row_stride, int nsum, int rows, int d, __nv_bfloat16 *__restrict__ xb,
                          float *__restrict__ ssq) {
  const int d4 = d >> 2, c4 = threadIdx.x;
  const size_t row = blockIdx.x;
  const float4 *x = reinterpret_cast<const float4 *>(h + row * row_stride) + c4;
  float4 v = x[0];
  for (int s = 1; s < nsum; ++s) v = f4_add(v, x[(size_t)s * d4]);
  __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  reinterpret_cast<uint2 *>(xb)[row * d4 + c4] = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
  const float ss = warp_sum(f4_sq(v));
  if ((threadIdx.x & 31) == 0) ssq[(size_t)(c4 >> 5) * rows + row] = ss;
}

// Latency-oriented variant for the decode regime (a handful of rows): the per-thread loop over
// layers above serialises ~7 dependent-latency loads per layer, which dominates when there are too
// few threads to hide it.  Here a block owns 32 float4 columns of one row; its 16 warps first fetch
// every layer's branch outputs (with up to four K-split partial sums each) and old states into shared memory (two
// layers per warp at a time, all loads issued before the first is consumed), then warp 0 runs the serial recurrence
// out of shared memory, keeping the per-layer sums of squares per lane; afterwards all warps reduce those, so the
// serial loop carries no shuffles.  Same arithmetic, same summation order as k_correct.
// grid (d/128, M), 512 threads; dynamic shared memory nl*32*(2+NS) float4 + nl*2 floats + nl*3*32 floats.
constexpr int kCorrSmallWarps = 16;
template <int NS>
__global__ void __launch_bounds__(32 * kCorrSmallWarps) k_correct_small(CorrParams p) {
  extern __shared__ float4 s_buf[];
  pdl_trigger();   // a few CTAs on a few SMs: the next kernel may move in beside it at once and fetch its first weights
  pdl_wait();
  const int d4 = p.d >> 2;
  const int c = threadIdx.x & 31, ll = threadIdx.x >> 5;
  const int c4 = blockIdx.x * 32 + c;
  const size_t row = blockIdx.y;
  const bool active = c4 < d4;
  const size_t Md4 = (size_t)p.M * d4, state4 = Md4 * NS;
  const float4 *a4 = reinterpret_cast<const float4 *>(p.a);
  const float4 *m4 = reinterpret_cast<const float4 *>(p.m);
  float4 *tr4 = reinterpret_cast<float4 *>(p.trace);
  const size_t bm_off = row * d4 + c4, st_off = row * NS * d4 + c4;
  float4 *sa = s_buf, *sm = s_buf + (size_t)p.nl * 32, *so = s_buf + (size_t)p.nl * 64;  // so: [nl][NS][32]
  float *snorm = reinterpret_cast<float *>(s_buf + (size_t)p.nl * 32 * (2 + NS));          // [nl][2]
  float *sred = snorm + (size_t)p.nl * 2;                                                  // [nl][3][32]: per-lane xs, rs, hs
  const bool want_norm = p.partial != nullptr;
  float4 first[NS];  // warp 0: the state the recurrence starts from
  if (active) {
    if (ll == 0) {
#pragma unroll
      for (int s = 0; s < NS; ++s) first[s] = tr4[(size_t)p.l0 * state4 + st_off + (size_t)s * d4];
    }
#pragma unroll 1
    for (int i0 = ll; i0 < p.nl; i0 += 2 * kCorrSmallWarps) {
      // every load of two steps (K-split partial sums included) is issued before the first is consumed
      float4 av[2], mv[2], aq[2][3], mq[2][3], ov[2][NS];
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int i = i0 + kCorrSmallWarps * k;
        if (i < p.nl) {
          const int l = p.l0 + i * p.lstep, ln = l + p.lstep;  // this step maps state l to state ln
          av[k] = a4[(size_t)l * Md4 + bm_off];
          mv[k] = m4[(size_t)l * Md4 + bm_off];
#pragma unroll
          for (int q = 1; q < 4; ++q) {
            if (q < p.a_splits) aq[k][q - 1] = a4[(size_t)q * (p.a_ss >> 2) + (size_t)l * Md4 + bm_off];
            if (q < p.m_splits) mq[k][q - 1] = m4[(size_t)q * (p.m_ss >> 2) + (size_t)l * Md4 + bm_off];
          }
#pragma unroll
          for (int r = 0; r < NS; ++r) ov[k][r] = tr4[(size_t)(p.implicit_old ? p.l0 : ln) * state4 + st_off + (size_t)r * d4];
        }
      }
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const int i = i0 + kCorrSmallWarps * k;
        if (i < p.nl) {
#pragma unroll
          for (int q = 1; q < 4; ++q) {  // partial sums are added in slice order
            if (q < p.a_splits) av[k] = f4_add(av[k], aq[k][q - 1]);
            if (q < p.m_splits) mv[k] = f4_add(mv[k], mq[k][q - 1]);
          }
          const int l = p.l0 + i * p.lstep;
          for (int q = 4; q < p.a_splits; ++q) av[k] = f4_add(av[k], a4[(size_t)q * (p.a_ss >> 2) + (size_t)l * Md4 + bm_off]);
          for (int q = 4; q < p.m_splits; ++q) mv[k] = f4_add(mv[k], m4[(size_t)q * (p.m_ss >> 2) + (size_t)l * Md4 + bm_off]);
          sa[i * 32 + c] = av[k];
          sm[i * 32 + c] = mv[k];
#pragma unroll
          for (int r = 0; r < NS; ++r) so[(i * NS + r) * 32 + c] = ov[k][r];
        }
      }
    }
  }
  __syncthreads();
  if (ll == 0) {
    const bool native = (NS == 1) ? (p.mode != 2) : (p.mode == 1);
    float4 oldp[NS], newp[NS];
    if (active) {
#pragma unroll
      for (int s = 0; s < NS; ++s) oldp[s] = newp[s] = first[s];
    }
    for (int i = 0; i < p.nl; ++i) {
      const int l = p.l0 + i * p.lstep, ln = l + p.lstep;  // this step maps state l to state ln
      float rs = 0.f, hs = 0.f, xs = 0.f;
      if (active) {
        const float4 av = sa[i * 32 + c], mv = sm[i * 32 + c];
        const HcCoef &cf = p.coef[l];
        float4 oldn[NS], newn[NS], tilde[NS];
#pragma unroll
        for (int r = 0; r < NS; ++r) {
          oldn[r] = so[(i * NS + r) * 32 + c];
          if (NS == 1) {
            tilde[r] = f4_add(f4_add(oldp[0], av), mv);
          } else {
            float4 t = f4_scale(cf.A[r * NS], oldp[0]);
#pragma unroll
            for (int s = 1; s < NS; ++s) t = f4_fma(cf.A[r * NS + s], oldp[s], t);
            tilde[r] = f4_fma(cf.cm[r], mv, f4_fma(cf.ca[r], av, t));
          }
        }
#pragma unroll
        for (int r = 0; r < NS; ++r) {
          if (p.mode == 2) {
            newn[r] = tilde[r];
          } else if (native) {
            if (NS == 1) {
              newn[r] = f4_add(f4_add(newp[0], av), mv);
            } else {
              float4 t = f4_scale(cf.A[r * NS], newp[0]);
#pragma unroll
              for (int s = 1; s < NS; ++s) t = f4_fma(cf.A[r * NS + s], newp[s], t);
              newn[r] = f4_fma(cf.cm[r], mv, f4_fma(cf.ca[r], av, t));
            }
          } else {
            newn[r] = f4_add(tilde[r], f4_sub(newp[r], oldp[r]));
          }
          const float4 rr = f4_sub(tilde[r], oldn[r]);
          rs += f4_sq(rr);
          hs += f4_sq(oldn[r]);
          tr4[(size_t)ln * state4 + st_off + (size_t)r * d4] = newn[r];
        }
        float4 nxt = newn[0];
        if (NS > 1 && ln < p.L) {
          const HcCoef &cn = p.coef[ln];
          float4 xa = f4_scale(cn.pa[0], newn[0]), xm = f4_scale(cn.pmra[0], newn[0]);
#pragma unroll
          for (int s = 1; s < NS; ++s) {
            xa = f4_fma(cn.pa[s], newn[s], xa);
            xm = f4_fma(cn.pmra[s], newn[s], xm);
          }
          if (p.xa != nullptr) reinterpret_cast<float4 *>(p.xa)[(size_t)ln * Md4 + bm_off] = xa;
          reinterpret_cast<float4 *>(p.xm)[(size_t)ln * Md4 + bm_off] = xm;
          nxt = xa;
        }
        if (NS > 1 && ln == p.L) {
#pragma unroll
          for (int s = 1; s < NS; ++s) nxt = f4_add(nxt, newn[s]);
        }
        if (p.xb != nullptr) {
          __nv_bfloat162 lo = __floats2bfloat162_rn(nxt.x, nxt.y), hi = __floats2bfloat162_rn(nxt.z, nxt.w);
          reinterpret_cast<uint2 *>(p.xb)[(size_t)ln * Md4 + bm_off] = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
          xs = f4_sq(nxt);
        }
#pragma unroll
        for (int r = 0; r < NS; ++r) { oldp[r] = oldn[r]; newp[r] = newn[r]; }
      }
      sred[(i * 3 + 0) * 32 + c] = xs;
      sred[(i * 3 + 1) * 32 + c] = rs;
      sred[(i * 3 + 2) * 32 + c] = hs;
    }
  }
  __syncthreads();
  // every warp reduces the sums of some steps (this block's 32 lanes hold 128 consecutive columns of the row: partial blockIdx.x)
  for (int i = ll; i < p.nl; i += kCorrSmallWarps) {
    const int ln = p.l0 + (i + 1) * p.lstep;
    if (p.xb != nullptr) {
      const float xs = warp_sum(sred[(i * 3 + 0) * 32 + c]);
      if (c == 0) p.ssq_x[((size_t)ln * gridDim.x + blockIdx.x) * p.M + row] = xs;
    }
    if (want_norm) {
      const float rs = warp_sum(sred[(i * 3 + 1) * 32 + c]), hs = warp_sum(sred[(i * 3 + 2) * 32 + c]);
      if (c == 0) { snorm[i * 2] = rs; snorm[i * 2 + 1] = hs; }
    }
  }
  if (!want_norm) return;
  __syncthreads();
  if (ll != 0) return;
  // warp 0 only from here on
  const unsigned nblk = gridDim.x * gridDim.y, blk = blockIdx.y * gridDim.x + blockIdx.x;
  for (int i = c; i < p.nl * 2; i += 32) p.partial[(size_t)blk * p.nl * 2 + i] = snorm[i];
  __threadfence();
  __syncwarp();
  unsigned ticket = 0;
  if (c == 0) ticket = atomicAdd(p.counter, 1u);
  ticket = __shfl_sync(0xffffffffu, ticket, 0);
  if (ticket != nblk - 1) return;
  __threadfence();
  for (int i = c; i < p.nl * 2; i += 32) {
    double s = 0.0;
    for (unsigned b = 0; b < nblk; ++b) s += (double)__ldcg(&p.partial[(size_t)b * p.nl * 2 + i]);
    p.resnorm[(size_t)(p.l0 + (i >> 1) * p.lstep) * 2 + (i & 1)] = (float)s;
  }
  __syncwarp();
  if (c == 0) *p.counter = 0u;
}

}  // namespace snlp
