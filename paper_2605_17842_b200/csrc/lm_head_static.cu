// snlp_lm_head_greedy_static: the greedy LM head (stream sum -> RMSNorm -> vocabulary projection ->
// argmax) for callers that must not allocate device memory.  It computes what snlp_lm_head computes,
// restricted to the argmax, with kernels of its own: a register-fed mma.sync weight-streaming product
// (k_gemv_lmhead, below) instead of the handle-bound tcgen05 kernel, so the order in which a logit's terms
// are added differs from snlp_lm_head's and the two may pick different tokens at near-ties.  The per-tile
// argmax partials live in a fixed array that is part of the loaded library image instead of in a
// cudaMalloc'd workspace, and no model handle is involved.
#include "../../include/snlp.h"

#include <cstdio>
#include <mutex>

#include "common.cuh"

using namespace snlp;

namespace snlp {
void set_last_error(const char *msg);  // defined next to snlp_last_error()
}

namespace {

struct GemvParams {
  const __nv_bfloat16 *W;   // [N][Kd] bf16 head weights
  int N, Kd, M;             // vocabulary, model width, rows (<= 16)
  const float *xf; size_t xf_rs; int nsum;   // fp32 rows, row stride (elements), streams summed per row
  float eps;
  float *pm_val; int *pm_idx; int ntile;     // partial argmax [M][ntile]
};

__device__ __forceinline__ uint4 ldg_stream16(const void *p) {
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

// Weight-streaming product of one 128-row tile of the head with <= 16 token rows, then the tile's argmax per row.
// The weights are the 16-row MMA operand (read once, 16-byte loads straight from global memory into the fragment
// registers); the tokens -- stream sum, bf16, staged in shared memory -- are the 8-wide operand; the RMSNorm of a
// row is a scalar applied to its logits.  grid (N/128), 256 threads.  NT = number of 8-token tiles (1 or 2).
// Dynamic shared memory: NT*8*(Kd+32) bf16 + NT*8*129 floats + 16 floats.
template <int NT>
__global__ void __launch_bounds__(kGemvThreads) k_gemv_lmhead(GemvParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int xstride = p.Kd + kGemvPad;
  __nv_bfloat16 *xs = reinterpret_cast<__nv_bfloat16 *>(smem_raw);
  float *outs = reinterpret_cast<float *>(smem_raw + (size_t)NT * 8 * xstride * sizeof(__nv_bfloat16));
  float *rstd = outs + NT * 8 * (kGemvRows + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x;
  const int g = lane >> 2, t = lane & 3;

  // one warp per token: stream sum, sum of squares, bf16 copy
  for (int tok = warp; tok < NT * 8; tok += kGemvThreads / 32) {
    float ss = 0.f;
    if (tok < p.M) {
      const float *x = p.xf + (size_t)tok * p.xf_rs;
      for (int j = lane * 4; j < p.Kd; j += 128) {
        float4 v = *reinterpret_cast<const float4 *>(x + j);
        for (int s = 1; s < p.nsum; ++s) {
          const float4 w = *reinterpret_cast<const float4 *>(x + (size_t)s * p.Kd + j);
          v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
        }
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        *reinterpret_cast<uint2 *>(xs + (size_t)tok * xstride + j) = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
      }
      ss = warp_sum(ss);
      if (lane == 0) rstd[tok] = rsqrtf(ss / (float)p.Kd + p.eps);
    } else {
      for (int j = lane * 4; j < p.Kd; j += 128) *reinterpret_cast<uint2 *>(xs + (size_t)tok * xstride + j) = make_uint2(0, 0);
      if (lane == 0) rstd[tok] = 0.f;
    }
  }
  __syncthreads();

  float acc[NT][4];
#pragma unroll
  for (int i = 0; i < NT; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
  const int r0 = tile * kGemvRows + warp * 16;
  const __nv_bfloat16 *w0 = p.W + (size_t)(r0 + g) * p.Kd + t * 8;
  const __nv_bfloat16 *w1 = w0 + (size_t)8 * p.Kd;
  const __nv_bfloat16 *x0 = xs + (size_t)g * xstride + t * 8;
  for (int kk = 0; kk < p.Kd; kk += 32 * kGemvUnroll) {
    uint4 wa[kGemvUnroll], wb[kGemvUnroll];
#pragma unroll
    for (int u = 0; u < kGemvUnroll; ++u) {
      const int k = kk + 32 * u;
      if (k < p.Kd) {
        wa[u] = ldg_stream16(w0 + k);
        wb[u] = ldg_stream16(w1 + k);
      }
    }
#pragma unroll
    for (int u = 0; u < kGemvUnroll; ++u) {
      const int k = kk + 32 * u;
      if (k < p.Kd) {
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

  const int n0 = tile * kGemvRows;
  for (int tok = warp; tok < p.M; tok += kGemvThreads / 32) {
    const float *y = outs + tok * (kGemvRows + 1);
    const float rs = rstd[tok];
    float bv = -INFINITY;
    int bi = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = lane + 32 * j;
      const float v = y[r] * rs;
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

// Final argmax over the per-tile partials (ties -> lowest index).  One block per token.
__global__ void k_argmax_tiles(const float *__restrict__ pm_val, const int *__restrict__ pm_idx, int ntile, int32_t *__restrict__ out) {
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
  }
}

constexpr int kMaxRows = 16;                                 // rows per call
constexpr int kMaxVocab = SNLP_STATIC_LM_HEAD_MAX_VOCAB;     // vocabulary entries
constexpr int kMaxDModel = SNLP_STATIC_LM_HEAD_MAX_D_MODEL;  // bounded by the staged token rows in shared memory
constexpr int kMaxTiles = kMaxVocab / kGemvRows;
constexpr int kMaxDevices = 64;

// Per-tile (best value, best index) pairs: kMaxRows x kMaxTiles floats followed by as many ints, 256 KiB
// in total.  Every GPU that loads this library carries its own copy until the process exits.
constexpr size_t kSlots = (size_t)kMaxRows * kMaxTiles;
constexpr size_t kScratchBytes = kSlots * (sizeof(float) + sizeof(int));
static __device__ __align__(256) unsigned char g_lm_head_scratch[kScratchBytes];

// In host code `g_lm_head_scratch` only names the symbol; the device address has to be asked for, once
// per device, while that device is current.
std::mutex g_mu;
unsigned char *g_scratch_ptr[kMaxDevices] = {};
bool g_ready[kMaxDevices] = {};
thread_local char g_msg[256];

int setup_device(int dev) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_ready[dev]) return SNLP_OK;
  void *ptr = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&ptr, g_lm_head_scratch);
  if (e != cudaSuccess) {
    snprintf(g_msg, sizeof g_msg, "snlp_lm_head_greedy_static: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
    set_last_error(g_msg);
    return SNLP_ERR_CUDA;
  }
  const int smem = 200 * 1024;
  e = cudaFuncSetAttribute(k_gemv_lmhead<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemv_lmhead<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) {
    snprintf(g_msg, sizeof g_msg, "snlp_lm_head_greedy_static: cudaFuncSetAttribute failed: %s", cudaGetErrorString(e));
    set_last_error(g_msg);
    return SNLP_ERR_CUDA;
  }
  g_scratch_ptr[dev] = static_cast<unsigned char *>(ptr);
  g_ready[dev] = true;
  return SNLP_OK;
}

int reject(int code, const char *msg) {
  snprintf(g_msg, sizeof g_msg, "%s", msg);
  set_last_error(g_msg);
  return code;
}

}  // namespace

extern "C" int snlp_lm_head_greedy_static(const float *hL, const void *lm_head_bf16, int rows, int n_streams, int d_model, int vocab,
                                          float rms_eps, int32_t *argmax, void *stream) {
  g_msg[0] = 0;
  if (!hL || !lm_head_bf16 || !argmax) return reject(SNLP_ERR_ARG, "snlp_lm_head_greedy_static: NULL pointer");
  // the kernels read hL and the head with 16-byte loads: a view at an odd offset must be turned away here, a
  // misaligned access on the device would cost the caller its CUDA context
  if ((uintptr_t)hL % 16 || (uintptr_t)lm_head_bf16 % 16 || (uintptr_t)argmax % 4)
    return reject(SNLP_ERR_ARG, "snlp_lm_head_greedy_static: hL and lm_head_bf16 must be 16-byte aligned, argmax 4-byte aligned");
  if (rows < 1 || n_streams < 1 || n_streams > kMaxStreams || d_model < 1 || vocab < 1) {
    snprintf(g_msg, sizeof g_msg, "snlp_lm_head_greedy_static: sizes must be positive (n_streams <= %d)", kMaxStreams);
    set_last_error(g_msg);
    return SNLP_ERR_ARG;
  }
  if (rows > kMaxRows || vocab > kMaxVocab || d_model > kMaxDModel) {
    snprintf(g_msg, sizeof g_msg,
             "snlp_lm_head_greedy_static: rows=%d vocab=%d d_model=%d exceed the fixed scratch (limits: %d rows, vocab %d, d_model %d)",
             rows, vocab, d_model, kMaxRows, kMaxVocab, kMaxDModel);
    set_last_error(g_msg);
    return SNLP_ERR_SHAPE;
  }
  if (vocab % kGemvRows || d_model % 32) {
    snprintf(g_msg, sizeof g_msg, "snlp_lm_head_greedy_static: vocab must be a multiple of %d and d_model of 32", kGemvRows);
    set_last_error(g_msg);
    return SNLP_ERR_UNSUPPORTED;
  }
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return reject(SNLP_ERR_CUDA, "snlp_lm_head_greedy_static: cudaGetDevice failed or device index out of range");
  int rc = setup_device(dev);
  if (rc != SNLP_OK) return rc;
  float *sc_val = reinterpret_cast<float *>(g_scratch_ptr[dev]);
  int *sc_idx = reinterpret_cast<int *>(g_scratch_ptr[dev] + kSlots * sizeof(float));
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  GemvParams p{};
  p.W = static_cast<const __nv_bfloat16 *>(lm_head_bf16);
  p.N = vocab;
  p.Kd = d_model;
  p.M = rows;
  p.xf = hL;
  p.xf_rs = (size_t)n_streams * d_model;
  p.nsum = n_streams;
  p.eps = rms_eps;
  p.pm_val = sc_val;
  p.pm_idx = sc_idx;
  p.ntile = vocab / kGemvRows;
  // Nothing in the scratch has to start at zero: every (row, tile) slot read by the final reduction is
  // written by this call's first kernel.  Slots beyond rows x ntile keep whatever an earlier call left.
  const int NT = rows <= 8 ? 1 : 2;
  const size_t sm = (size_t)NT * 8 * (p.Kd + kGemvPad) * 2 + (size_t)NT * 8 * (kGemvRows + 1) * 4 + 16 * 4;
  dim3 grid(vocab / kGemvRows, 1, 1);
  if (NT == 1) k_gemv_lmhead<1><<<grid, kGemvThreads, sm, st>>>(p);
  else k_gemv_lmhead<2><<<grid, kGemvThreads, sm, st>>>(p);
  k_argmax_tiles<<<rows, 256, 0, st>>>(sc_val, sc_idx, p.ntile, argmax);
  e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(g_msg, sizeof g_msg, "snlp_lm_head_greedy_static: kernel launch failed: %s", cudaGetErrorString(e));
    set_last_error(g_msg);
    return SNLP_ERR_CUDA;
  }
  return SNLP_OK;
}
