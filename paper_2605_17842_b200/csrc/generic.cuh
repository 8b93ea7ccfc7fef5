// Generic SIMT kernels: any shape, fp32 or bf16 operands, fp32 arithmetic.  They are the fp32-mode
// path (true FFMA, no TF32) and cover every shape the specialised kernels do not.
#pragma once
#include "common.cuh"

namespace snlp {

// ---------------------------------------------------------------------------------------------
// h_0 = Embed(ids): one block per row; the embedding row is replicated into each stream.
template <typename T>
__global__ void k_embed(const int32_t *__restrict__ ids, const T *__restrict__ table, float *__restrict__ h0,
                        int d, int n, int vocab, const int32_t *const *__restrict__ ids_pp = nullptr) {
  const int row = blockIdx.x;
  if (ids_pp != nullptr) ids = *ids_pp;   // the ids' address is read from a device slot (replayed decode graphs)
  int id = ids[row];
  id = id < 0 ? 0 : (id >= vocab ? vocab - 1 : id);
  const T *src = table + (size_t)id * d;
  float *dst = h0 + (size_t)row * n * d;
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    const float v = to_f<T>(src[j]);
    for (int s = 0; s < n; ++s) dst[(size_t)s * d + j] = v;
  }
}

// trace[l] = h0 for l = 0..L ("h0" initialisation of Alg. 2, line 5).  float4 granularity.
__global__ void k_bcast_trace(const float4 *__restrict__ h0, float4 *__restrict__ trace, size_t n4, int L1) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  const float4 v = h0[i];
  for (int l = 0; l < L1; ++l) trace[(size_t)l * n4 + i] = v;
}

// ---------------------------------------------------------------------------------------------
// dst[l][row][:] = T( RMSNorm( sum_{s<nsum} src[l][row][s][:] ) ).  grid (rows, nl).
template <typename T>
__global__ void k_rmsnorm_cast(const float *__restrict__ src, size_t src_ls, size_t src_rs, int nsum, T *__restrict__ dst,
                               size_t dst_ls, int d, float eps) {
  __shared__ float red[32];
  const float *x = src + (size_t)blockIdx.y * src_ls + (size_t)blockIdx.x * src_rs;
  T *y = dst + (size_t)blockIdx.y * dst_ls + (size_t)blockIdx.x * d;
  float ss = 0.f;
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float v = 0.f;
    for (int s = 0; s < nsum; ++s) v += x[(size_t)s * d + j];
    ss += v * v;
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)d + eps);
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float v = 0.f;
    for (int s = 0; s < nsum; ++s) v += x[(size_t)s * d + j];
    y[j] = from_f<T>(v * r);
  }
}

// u = xm + kappa_l * sum_p a[p];  un = T(RMSNorm(u)).  grid (rows, nl).
template <typename T>
__global__ void k_resid_rmsnorm_cast(const float *__restrict__ xm, size_t xm_ls, size_t xm_rs, const float *__restrict__ a,
                                     size_t a_ls, int a_splits, size_t a_ss, const HcCoef *__restrict__ coef, int l0,
                                     T *__restrict__ un, size_t un_ls, int d, float eps) {
  __shared__ float red[32];
  const int l = blockIdx.y, row = blockIdx.x;
  const float kappa = coef[l0 + l].kappa;
  const float *x = xm + (size_t)l * xm_ls + (size_t)row * xm_rs;
  const float *av = a + (size_t)l * a_ls + (size_t)row * d;
  T *y = un + (size_t)l * un_ls + (size_t)row * d;
  float ss = 0.f;
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float as = 0.f;
    for (int p = 0; p < a_splits; ++p) as += av[(size_t)p * a_ss + j];
    const float v = x[j] + kappa * as;
    ss += v * v;
  }
  ss = block_sum(ss, red);
  const float r = rsqrtf(ss / (float)d + eps);
  for (int j = threadIdx.x; j < d; j += blockDim.x) {
    float as = 0.f;
    for (int p = 0; p < a_splits; ++p) as += av[(size_t)p * a_ss + j];
    const float v = x[j] + kappa * as;
    y[j] = from_f<T>(v * r);
  }
}

// z = T(relu(y)^2), elementwise.
template <typename T>
__global__ void k_relu2_cast(const float *__restrict__ y, T *__restrict__ z, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    const float v = fmaxf(y[i], 0.f);
    z[i] = from_f<T>(v * v);
  }
}

// ---------------------------------------------------------------------------------------------
// C[l][M][N] (fp32) = A[l][M][K] * W[l][N][K]^T, both operands K-innermost.  64x64x16 tiles,
// 256 threads, 4x4 outputs per thread, plain FFMA.  grid (ceil(N/64), ceil(M/64), nl).
template <typename T>
__global__ void __launch_bounds__(256) k_gemm_nt(const T *__restrict__ A, size_t a_ls, const T *__restrict__ W, size_t w_ls,
                                                 float *__restrict__ C, size_t c_ls, int M, int N, int K) {
  __shared__ float As[16][64 + 4];
  __shared__ float Ws[16][64 + 4];
  const T *Ab = A + (size_t)blockIdx.z * a_ls;
  const T *Wb = W + (size_t)blockIdx.z * w_ls;
  float *Cb = C + (size_t)blockIdx.z * c_ls;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  const int lr = threadIdx.x >> 2;        // 0..63: tile row loaded by this thread
  const int lk = (threadIdx.x & 3) * 4;   // 0,4,8,12: k offset
  for (int k0 = 0; k0 < K; k0 += 16) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int k = k0 + lk + j;
      const int am = m0 + lr, wn = n0 + lr;
      As[lk + j][lr] = (am < M && k < K) ? to_f<T>(Ab[(size_t)am * K + k]) : 0.f;
      Ws[lk + j][lr] = (wn < N && k < K) ? to_f<T>(Wb[(size_t)wn * K + k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int i = 0; i < 4; ++i) w[i] = Ws[k][tx * 4 + i];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < N) Cb[(size_t)m * N + n] = acc[i][j];
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Rotary + QK-norm + scatter.  Reads raw projections qkv[l][row][3d]; writes q[l][row][d] and the
// layer's key/value slots at position *pos_base + (row % T) of sequence row / T.
// grid (rows, 3H, nl), 128 threads.  rope_cs[pos][hd/2] holds (cos, sin) pairs.
template <typename T>
__global__ void k_rope_qknorm_store(const float *__restrict__ qkv, size_t qkv_ls, T *__restrict__ q, size_t q_ls,
                                    T *__restrict__ kc, T *__restrict__ vc, size_t kv_ls, size_t kv_bs, int Tlen, int H,
                                    int hd, const int *__restrict__ pos_base, const float2 *__restrict__ rope_cs, float eps) {
  __shared__ float red[32];
  const int row = blockIdx.x, hh = blockIdx.y, l = blockIdx.z;
  const int d = H * hd, kind = hh / H, head = hh % H, half = hd >> 1;
  const int b = row / Tlen, pos = *pos_base + (row % Tlen);
  const float *src = qkv + (size_t)l * qkv_ls + (size_t)row * 3 * d + (size_t)kind * d + (size_t)head * hd;
  if (kind == 2) {
    T *dst = vc + (size_t)l * kv_ls + (size_t)b * kv_bs + (size_t)pos * d + (size_t)head * hd;
    for (int i = threadIdx.x; i < hd; i += blockDim.x) dst[i] = from_f<T>(src[i]);
    return;
  }
  T *dst = kind == 0 ? q + (size_t)l * q_ls + (size_t)row * d + (size_t)head * hd
                     : kc + (size_t)l * kv_ls + (size_t)b * kv_bs + (size_t)pos * d + (size_t)head * hd;
  // hd <= 256 and blockDim = 128, so each thread owns at most one rotary pair
  float y1 = 0.f, y2 = 0.f;
  const int i = threadIdx.x;
  if (i < half) {
    const float2 cs = rope_cs[(size_t)pos * half + i];
    const float x1 = src[i], x2 = src[i + half];
    y1 = x1 * cs.x - x2 * cs.y;
    y2 = x1 * cs.y + x2 * cs.x;
  }
  const float ss = block_sum(y1 * y1 + y2 * y2, red);
  const float r = rsqrtf(ss / (float)hd + eps);
  if (i < half) {
    dst[i] = from_f<T>(y1 * r);
    dst[i + half] = from_f<T>(y2 * r);
  }
}

// ---------------------------------------------------------------------------------------------
// Causal attention, one warp per (row, head): online softmax over keys 0 .. pos(row) of the layer's
// own key/value store.  grid (ceil(rows*H/4), nl), 128 threads.  head_dim <= 256.
template <typename T>
__global__ void k_attn_generic(const T *__restrict__ q, size_t q_ls, const T *__restrict__ kc, const T *__restrict__ vc,
                               size_t kv_ls, size_t kv_bs, T *__restrict__ out, size_t o_ls, int rows, int Tlen, int H, int hd,
                               const int *__restrict__ pos_base) {
  const int wid = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31, l = blockIdx.y;
  if (wid >= rows * H) return;
  const int row = wid / H, head = wid % H, d = H * hd;
  const int b = row / Tlen, pos = *pos_base + (row % Tlen);
  const T *qp = q + (size_t)l * q_ls + (size_t)row * d + (size_t)head * hd;
  const T *kp = kc + (size_t)l * kv_ls + (size_t)b * kv_bs + (size_t)head * hd;
  const T *vp = vc + (size_t)l * kv_ls + (size_t)b * kv_bs + (size_t)head * hd;
  float qr[8], acc[8];
  const float scale = rsqrtf((float)hd);
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int e = lane + 32 * j;
    qr[j] = e < hd ? to_f<T>(qp[e]) * scale : 0.f;
    acc[j] = 0.f;
  }
  float mx = -INFINITY, den = 0.f;
  for (int s = 0; s <= pos; ++s) {
    const T *kr = kp + (size_t)s * d;
    float dot = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int e = lane + 32 * j;
      if (e < hd) dot = fmaf(qr[j], to_f<T>(kr[e]), dot);
    }
    dot = warp_sum(dot);
    const float mn = fmaxf(mx, dot);
    const float c = __expf(mx - mn), p = __expf(dot - mn);
    den = den * c + p;
    const T *vr = vp + (size_t)s * d;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int e = lane + 32 * j;
      if (e < hd) acc[j] = fmaf(p, to_f<T>(vr[e]), acc[j] * c);
    }
    mx = mn;
  }
  T *op = out + (size_t)l * o_ls + (size_t)row * d + (size_t)head * hd;
  const float inv = 1.f / den;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int e = lane + 32 * j;
    if (e < hd) op[e] = from_f<T>(acc[j] * inv);
  }
}

// ---------------------------------------------------------------------------------------------
// Per-row argmax over `vocab` logits, ties to the lowest index.  One block per row.
// out_pp (nullable): the output's address is read from a device slot and `out_off` added (replayed decode graphs).
__global__ void k_argmax_rows(const float *__restrict__ logits, int vocab, int32_t *__restrict__ out, int32_t *const *__restrict__ out_pp = nullptr,
                              int out_off = 0) {
  if (out_pp != nullptr) out = *out_pp + out_off;
  __shared__ float sv[32];
  __shared__ int si[32];
  const float *x = logits + (size_t)blockIdx.x * vocab;
  float bv = -INFINITY;
  int bi = 0x7fffffff;
  for (int j = threadIdx.x; j < vocab; j += blockDim.x) {
    const float v = x[j];
    if (v > bv || (v == bv && j < bi)) { bv = v; bi = j; }
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
    out[blockIdx.x] = bi == 0x7fffffff ? 0 : bi;
    __threadfence_system();   // the token buffer may be mapped host memory that the host is watching
  }
}

// Stream pre-maps for mHC models: xa[l] = pa_l . x_l, xm[l] = pmra_l . x_l for l in [l0, l0+nl).
// grid (ceil(M*d/256), nl).
__global__ void k_premix(const float *__restrict__ trace, size_t t_ls, int n, int d, size_t Md, const HcCoef *__restrict__ coef,
                         int l0, float *__restrict__ xa, float *__restrict__ xm, size_t x_ls) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= Md) return;
  const int l = l0 + blockIdx.y;
  const size_t row = i / d, j = i % d;
  const float *x = trace + (size_t)l * t_ls + row * n * d + j;
  const HcCoef &c = coef[l];
  float sa = 0.f, sm = 0.f;
  for (int s = 0; s < n; ++s) {
    const float v = x[(size_t)s * d];
    sa = fmaf(c.pa[s], v, sa);
    sm = fmaf(c.pmra[s], v, sm);
  }
  xa[(size_t)l * x_ls + i] = sa;
  xm[(size_t)l * x_ls + i] = sm;
}

// Small helpers for the decoding policies -------------------------------------------------------
__global__ void k_set_int(int *p, int v) { *p = v; }
__global__ void k_add_int(int *p, int v) { *p += v; }
__global__ void k_copy_int(int *dst, const int *src) { *dst = *src; }
// The device slot through which replayed decode graphs find the caller's token buffers.
__global__ void k_set_ptrs(const void **slot, const void *a, const void *b) { slot[0] = a; slot[1] = b; }

// Greedy acceptance (Sec. 5.1): n = longest prefix with draft[i] == y[i]; emit drafts[0..n), y[n].
__global__ void k_accept(const int32_t *__restrict__ drafts, const int32_t *__restrict__ y, int block, int32_t *emitted,
                         int32_t *n_emitted, int32_t *n_accepted, int32_t *last_tok, int *pos, const int *len0_p) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  const int len0 = *len0_p;   // cache length when the round began (kept on the device: the host need not know it)
  int n = 0;
  while (n < block && drafts[n] == y[n]) ++n;
  for (int i = 0; i < n; ++i) emitted[i] = drafts[i];
  emitted[n] = y[n];
  for (int i = n + 1; i <= block; ++i) emitted[i] = -1;
  *n_emitted = n + 1;
  *n_accepted = n;
  *last_tok = y[n];
  *pos = len0 + n + 1;
}

}  // namespace snlp
