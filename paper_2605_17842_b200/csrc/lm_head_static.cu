// snlp_lm_head_greedy_static: the greedy LM head (stream sum -> RMSNorm -> vocabulary projection ->
// argmax) for callers that must not allocate device memory.  It runs the same weight-streaming kernel
// as snlp_lm_head, but the per-tile argmax partials live in a fixed array that is part of the loaded
// library image instead of in a cudaMalloc'd workspace, and no model handle is involved.
#include "../../include/snlp.h"

#include <cstdio>
#include <mutex>

#include "decode.cuh"

using namespace snlp;

namespace snlp {
void set_last_error(const char *msg);  // defined next to snlp_last_error()
}

namespace {

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
  e = cudaFuncSetAttribute(k_gemv_mma<1, PRO_NORM, EPI_LMHEAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_gemv_mma<2, PRO_NORM, EPI_LMHEAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) {
    snprintf(g_msg, sizeof g_msg, "snlp_lm_head_greedy_static: cudaFuncSetAttribute failed: %s", cudaGetErrorString(e));
    set_last_error(g_msg);
    return SNLP_ERR_CUDA;
  }
  g_scratch_ptr[dev] = static_cast<unsigned char *>(ptr);
  g_ready[dev] = true;
  return SNLP_OK;
}

}  // namespace

extern "C" int snlp_lm_head_greedy_static(const float *hL, const void *lm_head_bf16, int rows, int n_streams, int d_model, int vocab,
                                          float rms_eps, int32_t *argmax, void *stream) {
  g_msg[0] = 0;
  if (!hL || !lm_head_bf16 || !argmax) {
    snprintf(g_msg, sizeof g_msg, "snlp_lm_head_greedy_static: NULL pointer");
    set_last_error(g_msg);
    return SNLP_ERR_ARG;
  }
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
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    snprintf(g_msg, sizeof g_msg, "snlp_lm_head_greedy_static: cudaGetDevice failed or device index out of range");
    set_last_error(g_msg);
    return SNLP_ERR_CUDA;
  }
  int rc = setup_device(dev);
  if (rc != SNLP_OK) return rc;
  float *sc_val = reinterpret_cast<float *>(g_scratch_ptr[dev]);
  int *sc_idx = reinterpret_cast<int *>(g_scratch_ptr[dev] + kSlots * sizeof(float));
  cudaStream_t st = static_cast<cudaStream_t>(stream);

  GemvParams p{};
  p.W = static_cast<const __nv_bfloat16 *>(lm_head_bf16);
  p.w_ls = 0;
  p.N = vocab;
  p.Kd = d_model;
  p.kslice = d_model;
  p.M = rows;
  p.xf = hL;
  p.xf_ls = 0;
  p.xf_rs = (size_t)n_streams * d_model;
  p.nsum = n_streams;
  p.eps = rms_eps;
  p.logits = nullptr;
  p.pm_val = sc_val;
  p.pm_idx = sc_idx;
  p.ntile = vocab / kGemvRows;
  // Nothing in the scratch has to start at zero: every (row, tile) slot read by the final reduction is
  // written by this call's first kernel.  Slots beyond rows x ntile keep whatever an earlier call left.
  const int NT = rows <= 8 ? 1 : 2;
  const size_t sm = (size_t)NT * 8 * (p.kslice + kGemvPad) * 2 + (size_t)NT * 8 * (kGemvRows + 1) * 4 + 16 * 4;
  dim3 grid(vocab / kGemvRows, 1, 1);
  if (NT == 1) k_gemv_mma<1, PRO_NORM, EPI_LMHEAD><<<grid, kGemvThreads, sm, st>>>(p);
  else k_gemv_mma<2, PRO_NORM, EPI_LMHEAD><<<grid, kGemvThreads, sm, st>>>(p);
  k_argmax_tiles<<<rows, 256, 0, st>>>(sc_val, sc_idx, p.ntile, argmax);
  e = cudaGetLastError();
  if (e != cudaSuccess) {
    snprintf(g_msg, sizeof g_msg, "snlp_lm_head_greedy_static: kernel launch failed: %s", cudaGetErrorString(e));
    set_last_error(g_msg);
    return SNLP_ERR_CUDA;
  }
  return SNLP_OK;
}
