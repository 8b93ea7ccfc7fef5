// Shared device helpers and internal types of libsnlp (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace snlp {

constexpr int kMaxStreams = 8;

// Per-layer stream-mixing coefficients derived on the host (in double) from the mHC maps of
// App. C.2.  With x' = Ra x + Qa a and x_next = Rm x' + Qm m the block is affine in (x, a, m):
//   x_next = A x + ca * a + cm * m,  A = Rm Ra (the HCN surrogate, Eq. 8), ca = Rm Qa, cm = Qm;
// the attention branch reads pa . x (pa = Pa) and the MLP branch reads Pm . x' = pmra . x + kappa a
// with pmra = Pm Ra and kappa = Pm . Qa.  For a residual model (n = 1) every entry is 1.
struct HcCoef {
  float A[kMaxStreams * kMaxStreams];
  float ca[kMaxStreams];
  float cm[kMaxStreams];
  float pa[kMaxStreams];
  float pmra[kMaxStreams];
  float kappa;
  float pad[3];
};

template <typename T>
__device__ __forceinline__ float to_f(T v);
template <>
__device__ __forceinline__ float to_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__device__ __forceinline__ T from_f(float v);
template <>
__device__ __forceinline__ float from_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Deterministic block-wide sum (fixed order: lanes by butterfly, warps in index order).
// `red` must hold at least 32 floats of shared memory.  All threads get the result.
__device__ __forceinline__ float block_sum(float v, float *red) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) red[w] = v;
  __syncthreads();
  float s = 0.f;
  for (int i = 0; i < nw; ++i) s += red[i];
  return s;
}

// Two fp32 values in one 64-bit register for the packed fp32 pipe (add / mul / fma .f32x2: two IEEE operations per
// instruction, bit-identical to the scalar forms).
__device__ __forceinline__ unsigned long long pk2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void upk2(unsigned long long v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long mul2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// 16-byte asynchronous global -> shared copy (L2 only); valid == false zero-fills the destination instead.
__device__ __forceinline__ void cp_async16(void *smem, const void *gmem, bool valid) {
  const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
  const int sz = valid ? 16 : 0;  // src-size 0 => the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Programmatic dependent launch.  A kernel launched with the programmatic-serialisation attribute may start while the
// kernel before it in the stream is still running; pdl_wait() returns once that kernel (and, by induction, every
// earlier one) has completed and its writes are visible, so everything a kernel does before it must depend on nothing
// an earlier kernel of the stream writes (set-up, weight prefetch).  pdl_trigger() lets the NEXT kernel of the stream be
// scheduled as soon as every CTA of this grid has issued it (or exited).  Both are no-ops in a normal launch.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

}  // namespace snlp
