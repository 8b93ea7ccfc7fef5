// libsnlp: host side of the C ABI declared in include/snlp.h -- handles, workspace, launch sequences.
// Every arithmetic step of the path runs in the CUDA kernels of generic.cuh / decode.cuh / correct.cuh.
#include "../../include/snlp.h"

#include <algorithm>
#include <atomic>
#include <chrono>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <numeric>
#include <string>
#include <tuple>
#include <vector>

#include "common.cuh"
#include "correct.cuh"
#include "decode.cuh"
#include "generic.cuh"
#include "umma_gemm.cuh"
#include "umma_gemm2.cuh"
#include "umma_chain.cuh"
#include "attn_umma.cuh"

using namespace snlp;

// ------------------------------------------------------------------------------------------------
// errors
static thread_local std::string g_err;

static int fail(int code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  g_err = buf;
  return code;
}

#define CU(call)                                                                                     \
  do {                                                                                               \
    cudaError_t e_ = (call);                                                                         \
    if (e_ != cudaSuccess) return fail(SNLP_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

#define TRY(call)            \
  do {                       \
    int r_ = (call);         \
    if (r_ != SNLP_OK) return r_; \
  } while (0)

extern "C" const char *snlp_last_error(void) { return g_err.c_str(); }

namespace snlp {
void set_last_error(const char *msg) { g_err = msg; }  // for the library's other translation units
}

// ------------------------------------------------------------------------------------------------
// handles
constexpr size_t kCorrExtraSmem = 32768;   // k_correct: shared memory beyond the operand ring (norm partials, staged coefficients)
constexpr int kMaxSplits = 4;    // K-splits of the partial-sum GEMV outputs
constexpr int kDecodeRows = 16;  // largest row count served by the decode-regime kernels
constexpr size_t kCorrSmallSmem = 160 * 1024;

// A captured decode step.  The token buffers are not part of the key: the step's kernels find them through the
// handle's device slot (tok_slot), so one graph serves every caller buffer.
struct GraphKey {
  int B, K, mode, prefix, init, fuse, nchunk;
  const void *res;
  const void *kv;
  bool operator<(const GraphKey &o) const {
    return std::tie(B, K, mode, prefix, init, fuse, nchunk, res, kv) < std::tie(o.B, o.K, o.mode, o.prefix, o.init, o.fuse, o.nchunk, o.res, o.kv);
  }
};
struct GraphEntry { cudaGraphExec_t exec; int64_t nodes; };
struct PendingTime { int cls; cudaEvent_t e0, e1; };
// TMA maps over one stacked weight array: boxes {64, BN, 1} and (for CTA pairs) {64, 128, 1}; for the decode regime
// td128[i] / td256[i] with boxes of 2^i k-blocks of 128 / 256 rows (those that divide nkb1, the k-blocks one decode-regime
// item reduces over; td256 only when BN == 256).
struct WMap { CUtensorMap tm, tm_half, td128[3], td256[2]; int BN, nkb1; };
enum { KC_QKV = 0, KC_ATTN, KC_OPROJ, KC_UP, KC_DOWN, KC_CORRECT, KC_LMHEAD, KC_OTHER, KC_COUNT };
static_assert(KC_COUNT == SNLP_NUM_KERNEL_CLASSES, "kernel class count");

struct snlp_model {
  snlp_config cfg{};
  int device = 0;
  bool loaded = false;
  size_t esz = 4;  // operand element size
  // weights
  void *embed = nullptr, *lm_head = nullptr, *wqkv = nullptr, *wo = nullptr, *wup = nullptr, *wdn = nullptr;
  HcCoef *coef = nullptr;
  float2 *rope = nullptr;    // [max_ctx][hd/2] (cos, sin)
  float2 *rope_t = nullptr;  // the same table transposed, [hd/2][max_ctx]: coalesced when the lanes of a warp hold consecutive positions
  // workspace (R = max_rows)
  float *trace = nullptr, *xa = nullptr, *xm = nullptr, *qkv_raw = nullptr, *a = nullptr, *y_raw = nullptr, *mb = nullptr;
  void *ub = nullptr;
  float *ssq_x = nullptr, *ssq_u = nullptr, *ssq_lm = nullptr;
  void *xn = nullptr, *q = nullptr, *att = nullptr, *z = nullptr, *sk = nullptr, *sv = nullptr, *xlm = nullptr;
  float *attn_part = nullptr, *corr_part = nullptr, *logits = nullptr, *pm_val = nullptr;
  int *pm_idx = nullptr;
  unsigned *counter = nullptr, *attn_counters = nullptr;
  int *zero = nullptr;
  unsigned *lm_counter = nullptr;   // arrival counter of the LM-head launch (zero between launches)
  unsigned *chain_bar = nullptr;    // grid-barrier counter of the chained decode-regime products (zero between launches)
  int32_t *spec = nullptr;  // [2 * (max_rows + 1)] ids / verifier tokens for draft-and-verify
  int32_t *tok_pin = nullptr, *tok_dev = nullptr;   // [2][max_batch] mapped pinned host memory (tokens in, tokens out) and its device address (snlp_decode_step_host)
  int logit_rows = 0;
  std::vector<void *> allocs;
  // flags / stats
  int use_graphs = 1, force_generic = 0, timing = 0, use_pdl = 1, use_chain = 1;
  bool pdl_now = false;   // launches issued right now carry the programmatic-serialisation attribute (layer-by-layer execution only)
  std::vector<PendingTime> pending;
  std::vector<cudaEvent_t> free_events;
  double class_ms[KC_COUNT] = {};
  int64_t class_launches[KC_COUNT] = {};
  int64_t launches = 0;
  bool capturing = false;
  int64_t cap_nodes = 0;
  std::map<GraphKey, GraphEntry> graphs;
  std::vector<snlp_kv *> caches;  // live KV caches of this model (orphaned, not freed, by snlp_destroy)
  WMap w_qkv, w_o, w_up, w_dn, w_lm;
  bool have_wmaps = false;
  int n_sm = 148;
  EncodeTiledFn encode_tiled = nullptr;  // cuTensorMapEncodeTiled, looked up through the runtime
  int *dev_err = nullptr;                // raised by a kernel whose bounded wait expired
  int last_rows = 0;                     // rows of the forward whose states the internal trace holds (snlp_copy_trace)
  const void **tok_slot = nullptr;       // device: addresses of the decode step's {tok_in, tok_out}, read by its kernels
  const void *slot_in = nullptr, *slot_out = nullptr;   // what tok_slot holds, in the order the calls were issued
  int64_t graph_captures = 0;            // decode graphs captured so far
  cudaStream_t cap_stream = nullptr;  // capture target: graphs are recorded here and replayed on the caller's stream
};

struct snlp_kv {
  snlp_model *m = nullptr;
  int B = 0, max_ctx = 0;
  // The cache length lives on the device (pos[0]); the host mirrors it.  After an asynchronous draft-and-verify
  // round only an upper bound is known here (len_known == false, len_hi) until snlp_kv_len reads the device value.
  int len = 0, len_hi = 0;
  bool len_known = true;
  void *k = nullptr, *v = nullptr;
  int *pos = nullptr;   // device int[4]: [0] the length, [1] the length saved at the start of a draft-and-verify round
};

// a forward call's geometry and key/value store
struct Fwd {
  int M, B, T;
  void *kc, *vc;
  size_t kv_ls, kv_bs;  // elements
  const int *pos;       // device: first position of this call
  int pos_hi;           // host copy of *pos
  int kv_rows;          // rows per sequence in the key / value store
  const int32_t *embed_ids = nullptr;   // non-NULL: state 0 is the embedding of these tokens and has not been written yet
  const int32_t *const *embed_ids_pp = nullptr;   // the same, with the tokens' address read from a device slot
  bool last_pass = false;   // no sweep follows this correction: it need not prepare the next sweep's branch inputs
  int implicit_state = -1;  // >= 0: states after this one are not materialised yet and equal it (first pass after Alg. 2 line 5)
  cudaStream_t st;
};

static inline void count(snlp_model *m, int n = 1) {
  if (m->capturing) m->cap_nodes += n;
  else m->launches += n;
}

static int pick_ksplit(int K, int want);

// Optional device timing of every launch, by kernel class (CUDA events on the launching stream).
struct TimedLaunch {
  snlp_model *m;
  cudaStream_t st;
  int cls;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  TimedLaunch(snlp_model *m_, cudaStream_t st_, int cls_) : m(m_), st(st_), cls(cls_) {
    if (!m->timing || m->capturing || m->pending.size() >= 200000) return;
    if (m->free_events.size() >= 2) {
      e0 = m->free_events.back(); m->free_events.pop_back();
      e1 = m->free_events.back(); m->free_events.pop_back();
    } else if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
      e0 = e1 = nullptr;
      return;
    }
    cudaEventRecord(e0, st);
  }
  ~TimedLaunch() {
    if (e0) {
      cudaEventRecord(e1, st);
      m->pending.push_back({cls, e0, e1});
    }
    count(m);
  }
};

#define KLAUNCH(m, st, cls, ...)     \
  do {                               \
    {                                \
      TimedLaunch tl_(m, st, cls);   \
      __VA_ARGS__;                   \
    }                                \
    LAUNCH_CHECK();                  \
  } while (0)

#define LAUNCH_CHECK()                                                                              \
  do {                                                                                              \
    cudaError_t e_ = cudaGetLastError();                                                            \
    if (e_ != cudaSuccess) return fail(SNLP_ERR_CUDA, "kernel launch failed (%s:%d): %s", __FILE__, __LINE__, cudaGetErrorString(e_)); \
  } while (0)

// Launch with the programmatic-serialisation attribute (see pdl_wait / pdl_trigger in common.cuh): the kernel may be
// scheduled while the one before it in the stream is still finishing.  Works the same under stream capture (the
// dependency becomes a programmatic edge of the graph).  pdl == false: an ordinary launch.
template <typename... KArgs, typename... Args>
static void launch_pdl(bool pdl, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = pdl ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);   // a failure is picked up by the cudaGetLastError() that follows every launch
}

template <typename P>
static int dalloc(snlp_model *m, P **p, size_t bytes) {
  void *q = nullptr;
  if (bytes == 0) bytes = 16;
  cudaError_t e = cudaMalloc(&q, bytes);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(SNLP_ERR_OOM, "cudaMalloc of %zu bytes failed: %s", bytes, cudaGetErrorString(e));
  }
  m->allocs.push_back(q);
  *p = reinterpret_cast<P *>(q);
  return SNLP_OK;
}

static int init_kernel_attributes();
static bool fused_prefill_ok(const snlp_model *m, int M);
static bool fast_decode_ok(const snlp_model *m, int M);
static bool umma_path_ok(const snlp_model *m);

// 64-key sub-blocks per split-KV chunk of the decode-regime attention.  It depends only on the number of
// (sequence, head) pairs -- not on the context length, the number of query rows or how many layers one
// launch covers -- so a decode step, the verifier block of self-speculative decoding, a sequential pass and
// a layer-parallel sweep all merge their keys in the same order (K = L sweeps then reproduce the
// sequential result bit for bit).
static int attn_csub(int pairs) { return pairs < 32 ? 4 : 8; }

extern "C" int snlp_create(const snlp_config *cfg, snlp_model **out) {
  if (!cfg || !out) return fail(SNLP_ERR_ARG, "snlp_create: NULL argument");
  const snlp_config &c = *cfg;
  if (c.n_layer < 1 || c.d_model < 1 || c.n_head < 1 || c.head_dim < 2 || c.d_ff < 1 || c.vocab < 1 || c.max_rows < 1 ||
      c.max_batch < 1 || c.max_ctx < 1)
    return fail(SNLP_ERR_ARG, "snlp_create: sizes must be positive");
  if (c.n_head * c.head_dim != c.d_model) return fail(SNLP_ERR_ARG, "snlp_create: n_head*head_dim != d_model");
  if (c.head_dim % 2 || c.head_dim > 256) return fail(SNLP_ERR_ARG, "snlp_create: head_dim must be even and <= 256");
  if (c.d_model % 4) return fail(SNLP_ERR_ARG, "snlp_create: d_model must be a multiple of 4");
  if (c.n_streams < 1 || c.n_streams > kMaxStreams) return fail(SNLP_ERR_ARG, "snlp_create: n_streams must be in 1..8");
  if (c.dtype != SNLP_DTYPE_FP32 && c.dtype != SNLP_DTYPE_BF16) return fail(SNLP_ERR_ARG, "snlp_create: unknown dtype");
  if (c.max_batch > c.max_rows) return fail(SNLP_ERR_ARG, "snlp_create: max_batch > max_rows");
  snlp_model *m = new (std::nothrow) snlp_model;
  if (!m) return fail(SNLP_ERR_OOM, "snlp_create: host allocation failed");
  m->cfg = c;
  m->esz = c.dtype == SNLP_DTYPE_BF16 ? 2 : 4;
  cudaError_t e = cudaGetDevice(&m->device);
  if (e != cudaSuccess) {
    delete m;
    return fail(SNLP_ERR_CUDA, "cudaGetDevice failed: %s", cudaGetErrorString(e));
  }
  const size_t L = c.n_layer, d = c.d_model, ff = c.d_ff, V = c.vocab, n = c.n_streams, R = c.max_rows, es = m->esz;
  int rc = SNLP_OK;
  auto A = [&](auto **p, size_t bytes) { if (rc == SNLP_OK) rc = dalloc(m, p, bytes); };
  A(&m->embed, V * d * es);
  A(&m->lm_head, V * d * es);
  A(&m->wqkv, L * 3 * d * d * es);
  A(&m->wo, L * d * d * es);
  A(&m->wup, L * ff * d * es);
  A(&m->wdn, L * d * ff * es);
  A(&m->coef, L * sizeof(HcCoef));
  A(&m->rope, (size_t)c.max_ctx * (c.head_dim / 2) * sizeof(float2));
  A(&m->rope_t, (size_t)c.max_ctx * (c.head_dim / 2) * sizeof(float2));
  A(&m->trace, (L + 1) * R * n * d * 4);
  if (n > 1) {
    A(&m->xa, L * R * d * 4);
    A(&m->xm, L * R * d * 4);
  }
  A(&m->qkv_raw, L * R * 3 * d * 4);
  // the decode-regime kernels write up to kMaxSplits partial sums for at most kDecodeRows rows
  const size_t split_rows = std::max<size_t>(R, (size_t)kMaxSplits * std::min<size_t>(R, kDecodeRows));
  A(&m->a, L * split_rows * d * 4);
  A(&m->y_raw, L * R * ff * 4);
  A(&m->mb, L * split_rows * d * 4);
  A(&m->xn, (L + 1) * R * d * es);
  if (c.dtype == SNLP_DTYPE_BF16 && d % 128 == 0) {
    A(&m->ub, L * R * d * es);
    A(&m->ssq_x, (L + 1) * (d / 128) * R * 4);
    A(&m->ssq_u, L * 2 * (d / 128) * R * 4);
    A(&m->ssq_lm, (size_t)(d / 128) * kDecodeRows * 4);
  }
  A(&m->q, L * R * d * es);
  A(&m->att, L * R * d * es);
  A(&m->z, L * R * ff * es);
  A(&m->sk, L * R * d * es);
  A(&m->sv, L * R * d * es);
  A(&m->xlm, R * d * es);
  const size_t nchunk_max = ((size_t)c.max_ctx + kAttnSub - 1) / kAttnSub;
  A(&m->attn_part, L * (size_t)kDecodeRows * c.n_head * nchunk_max * kAttnPartStride * 4);
  // partial norms: one slot per block of k_correct (256 threads over R x d/4) or of k_correct_small ((d/128) x rows, rows <= 16)
  const size_t corr_blocks = std::max<size_t>((R * (d / 4) + 255) / 256, (size_t)((d + 127) / 128) * kDecodeRows);
  A(&m->corr_part, corr_blocks * L * 2 * 4);
  m->logit_rows = (int)(R < 64 ? R : 64);
  A(&m->logits, (size_t)m->logit_rows * V * 4);
  A(&m->pm_val, (size_t)kDecodeRows * ((V + 127) / 128) * 4);
  A(&m->pm_idx, (size_t)kDecodeRows * ((V + 127) / 128) * 4);
  A(&m->counter, 16);
  A(&m->dev_err, 16);
  A(&m->attn_counters, L * (size_t)kDecodeRows * c.n_head * 4);
  A(&m->zero, 16);
  A(&m->lm_counter, 16);
  A(&m->chain_bar, 16);
  A(&m->spec, 2 * (R + 1) * 4);
  A(&m->tok_slot, 2 * sizeof(void *));
  if (rc == SNLP_OK && (cudaHostAlloc((void **)&m->tok_pin, (size_t)2 * c.max_batch * 4, cudaHostAllocMapped) != cudaSuccess ||
                        cudaHostGetDevicePointer((void **)&m->tok_dev, m->tok_pin, 0) != cudaSuccess)) {
    cudaGetLastError();
    rc = fail(SNLP_ERR_OOM, "cudaHostAlloc of the token staging buffer failed");
  }
  if (rc == SNLP_OK) {
    if (cudaMemset(m->dev_err, 0, 16) != cudaSuccess || cudaMemset(m->attn_counters, 0, L * (size_t)kDecodeRows * c.n_head * 4) != cudaSuccess || cudaMemset(m->counter, 0, 16) != cudaSuccess || cudaMemset(m->zero, 0, 16) != cudaSuccess || cudaMemset(m->lm_counter, 0, 16) != cudaSuccess || cudaMemset(m->chain_bar, 0, 16) != cudaSuccess)
      rc = fail(SNLP_ERR_CUDA, "cudaMemset failed");
  }
  if (rc == SNLP_OK) {
    // rotary table in double on the host: (cos, sin)(pos * base^(-2i/hd))
    const int half = c.head_dim / 2;
    std::vector<float2> tab((size_t)c.max_ctx * half);
    for (int pos = 0; pos < c.max_ctx; ++pos)
      for (int i = 0; i < half; ++i) {
        const double ang = (double)pos * std::pow((double)c.rope_base, -2.0 * i / c.head_dim);
        tab[(size_t)pos * half + i] = make_float2((float)std::cos(ang), (float)std::sin(ang));
      }
    std::vector<float2> tab_t(tab.size());
    for (int pos = 0; pos < c.max_ctx; ++pos)
      for (int i = 0; i < half; ++i) tab_t[(size_t)i * c.max_ctx + pos] = tab[(size_t)pos * half + i];
    if (cudaMemcpy(m->rope, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(m->rope_t, tab_t.data(), tab_t.size() * sizeof(float2), cudaMemcpyHostToDevice) != cudaSuccess)
      rc = fail(SNLP_ERR_CUDA, "rotary table upload failed");
  }
  if (rc == SNLP_OK) rc = init_kernel_attributes();
  if (rc == SNLP_OK) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, m->device) == cudaSuccess) m->n_sm = prop.multiProcessorCount;
  }
  if (rc == SNLP_OK) {
    cudaDriverEntryPointQueryResult qres;
    void *fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
      m->encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
    else
      cudaGetLastError();  // without it the tensor-core GEMM is not used
  }
  if (rc == SNLP_OK && cudaStreamCreateWithFlags(&m->cap_stream, cudaStreamNonBlocking) != cudaSuccess)
    rc = fail(SNLP_ERR_CUDA, "cudaStreamCreateWithFlags failed");
  if (rc != SNLP_OK) {
    for (void *p : m->allocs) cudaFree(p);
    if (m->tok_pin) cudaFreeHost(m->tok_pin);
    delete m;
    return rc;
  }
  *out = m;
  return SNLP_OK;
}

extern "C" int snlp_destroy(snlp_model *m) {
  if (!m) return fail(SNLP_ERR_ARG, "snlp_destroy: NULL handle");
  cudaDeviceSynchronize();
  for (snlp_kv *kv : m->caches) kv->m = nullptr;  // their memory stays valid until snlp_kv_destroy
  for (auto &g : m->graphs) cudaGraphExecDestroy(g.second.exec);
  if (m->cap_stream) cudaStreamDestroy(m->cap_stream);
  for (const PendingTime &t : m->pending) { cudaEventDestroy(t.e0); cudaEventDestroy(t.e1); }
  for (cudaEvent_t e : m->free_events) cudaEventDestroy(e);
  for (void *p : m->allocs) cudaFree(p);
  if (m->tok_pin) cudaFreeHost(m->tok_pin);
  delete m;
  return SNLP_OK;
}

extern "C" int snlp_load_weights(snlp_model *m, const snlp_weights *w) {
  if (!m || !w) return fail(SNLP_ERR_ARG, "snlp_load_weights: NULL argument");
  if (!w->embed || !w->lm_head || !w->wqkv || !w->wo || !w->wup || !w->wdn)
    return fail(SNLP_ERR_ARG, "snlp_load_weights: NULL weight array");
  const snlp_config &c = m->cfg;
  const int n = c.n_streams;
  if (n > 1 && (!w->hc_res_attn || !w->hc_res_mlp || !w->hc_pre_attn || !w->hc_pre_mlp || !w->hc_post_attn || !w->hc_post_mlp))
    return fail(SNLP_ERR_ARG, "snlp_load_weights: n_streams > 1 needs all hc_* arrays");
  const size_t L = c.n_layer, d = c.d_model, ff = c.d_ff, V = c.vocab, es = m->esz;
  CU(cudaMemcpy(m->embed, w->embed, V * d * es, cudaMemcpyHostToDevice));
  CU(cudaMemcpy(m->lm_head, w->lm_head, V * d * es, cudaMemcpyHostToDevice));
  CU(cudaMemcpy(m->wqkv, w->wqkv, L * 3 * d * d * es, cudaMemcpyHostToDevice));
  CU(cudaMemcpy(m->wo, w->wo, L * d * d * es, cudaMemcpyHostToDevice));
  CU(cudaMemcpy(m->wup, w->wup, L * ff * d * es, cudaMemcpyHostToDevice));
  CU(cudaMemcpy(m->wdn, w->wdn, L * d * ff * es, cudaMemcpyHostToDevice));
  std::vector<HcCoef> co(L);
  for (size_t l = 0; l < L; ++l) {
    HcCoef &h = co[l];
    std::memset(&h, 0, sizeof h);
    if (n == 1) {
      h.A[0] = h.ca[0] = h.cm[0] = h.pa[0] = h.pmra[0] = 1.f;
      h.kappa = 1.f;
      continue;
    }
    const float *Ra = w->hc_res_attn + l * n * n, *Rm = w->hc_res_mlp + l * n * n;
    const float *Pa = w->hc_pre_attn + l * n, *Pm = w->hc_pre_mlp + l * n;
    const float *Qa = w->hc_post_attn + l * n, *Qm = w->hc_post_mlp + l * n;
    double kappa = 0.0;
    for (int r = 0; r < n; ++r) {
      double ca = 0.0, pm = 0.0;
      for (int s = 0; s < n; ++s) {
        double acc = 0.0;
        for (int q = 0; q < n; ++q) acc += (double)Rm[r * n + q] * (double)Ra[q * n + s];
        h.A[r * n + s] = (float)acc;       // A = Rm Ra
        ca += (double)Rm[r * n + s] * (double)Qa[s];
        pm += (double)Pm[s] * (double)Ra[s * n + r];  // (Pm Ra)[r]
      }
      h.ca[r] = (float)ca;
      h.cm[r] = Qm[r];
      h.pa[r] = Pa[r];
      h.pmra[r] = (float)pm;
      kappa += (double)Pm[r] * (double)Qa[r];
    }
    h.kappa = (float)kappa;
  }
  CU(cudaMemcpy(m->coef, co.data(), L * sizeof(HcCoef), cudaMemcpyHostToDevice));
  m->have_wmaps = false;
  if (m->encode_tiled && c.dtype == SNLP_DTYPE_BF16 && d % 128 == 0 && ff % 128 == 0 && V % 128 == 0) {
    // kslice: the K range one decode-regime item reduces over (K, or a K-split slice of it)
    auto mk = [&](WMap &w, const void *base, uint64_t K, uint64_t N, uint64_t layers, uint64_t kslice) {
      w.BN = N % 256 == 0 ? 256 : 128;
      w.nkb1 = (int)(kslice / kUmmaBK);
      bool ok = make_tmap_bf16(m->encode_tiled, &w.tm, base, K, N, layers, N * K, w.BN) &&
                make_tmap_bf16(m->encode_tiled, &w.tm_half, base, K, N, layers, N * K, 128);
      for (int i = 0; i < 3 && ok; ++i)
        if (w.nkb1 % (1 << i) == 0) ok = make_tmap_bf16_kb(m->encode_tiled, &w.td128[i], base, K, N, layers, N * K, 128, 1u << i);
      for (int i = 0; i < 2 && ok; ++i)
        if (w.BN == 256 && w.nkb1 % (1 << i) == 0) ok = make_tmap_bf16_kb(m->encode_tiled, &w.td256[i], base, K, N, layers, N * K, 256, 1u << i);
      return ok;
    };
    const uint64_t dn_slice = ff / pick_ksplit(ff, kMaxSplits);
    m->have_wmaps = mk(m->w_qkv, m->wqkv, d, 3 * d, L, d) && mk(m->w_o, m->wo, d, d, L, d) && mk(m->w_up, m->wup, d, ff, L, d) &&
                    mk(m->w_dn, m->wdn, ff, d, L, dn_slice) && mk(m->w_lm, m->lm_head, d, V, 1, d);
  }
  m->loaded = true;
  return SNLP_OK;
}

extern "C" int snlp_set_flag(snlp_model *m, int flag, int value) {
  if (!m) return fail(SNLP_ERR_ARG, "snlp_set_flag: NULL handle");
  if (flag == 0) m->use_graphs = value != 0;
  else if (flag == 1) m->force_generic = value != 0;
  else if (flag == 2) m->timing = value != 0;
  else if (flag == 4) {
    if (m->use_pdl != (value != 0)) {   // captured decode steps carry the launch attributes they were recorded with
      CU(cudaDeviceSynchronize());
      for (auto &g : m->graphs) cudaGraphExecDestroy(g.second.exec);
      m->graphs.clear();
    }
    m->use_pdl = value != 0;
  }
  else if (flag == 5) {
    if (m->use_chain != (value != 0)) {   // captured decode steps were recorded with the other launch sequence
      CU(cudaDeviceSynchronize());
      for (auto &g : m->graphs) cudaGraphExecDestroy(g.second.exec);
      m->graphs.clear();
    }
    m->use_chain = value != 0;
  }
  else if (flag == 3) {   // host-side injection of the error word a kernel raises when a bounded wait expires
    const int v = value != 0;
    CU(cudaDeviceSynchronize());
    CU(cudaMemcpy(m->dev_err, &v, sizeof v, cudaMemcpyHostToDevice));
  }
  else return fail(SNLP_ERR_ARG, "snlp_set_flag: unknown flag %d", flag);
  return SNLP_OK;
}

static int drain_times(snlp_model *m) {
  for (const PendingTime &t : m->pending) {
    CU(cudaEventSynchronize(t.e1));
    float ms = 0.f;
    CU(cudaEventElapsedTime(&ms, t.e0, t.e1));
    m->class_ms[t.cls] += ms;
    m->class_launches[t.cls] += 1;
    m->free_events.push_back(t.e0);
    m->free_events.push_back(t.e1);
  }
  m->pending.clear();
  return SNLP_OK;
}

extern "C" int snlp_kernel_times(snlp_model *m, double *ms, int64_t *launches, int reset) {
  if (!m || !ms || !launches) return fail(SNLP_ERR_ARG, "snlp_kernel_times: NULL argument");
  TRY(drain_times(m));
  for (int i = 0; i < KC_COUNT; ++i) {
    ms[i] = m->class_ms[i];
    launches[i] = m->class_launches[i];
    if (reset) { m->class_ms[i] = 0.0; m->class_launches[i] = 0; }
  }
  return SNLP_OK;
}

extern "C" int snlp_device_status(snlp_model *m, void *stream) {
  if (!m) return fail(SNLP_ERR_ARG, "snlp_device_status: NULL handle");
  int flag = 0;
  CU(cudaStreamSynchronize((cudaStream_t)stream));
  CU(cudaMemcpy(&flag, m->dev_err, sizeof flag, cudaMemcpyDeviceToHost));
  if (flag) {
    cudaMemset(m->dev_err, 0, sizeof flag);
    // a kernel that gave up may have left arrival counters part-way: bring them back to zero for the calls that follow
    cudaMemset(m->lm_counter, 0, 16);
    cudaMemset(m->chain_bar, 0, 16);
    cudaMemset(m->counter, 0, 16);
    cudaMemset(m->attn_counters, 0, (size_t)m->cfg.n_layer * kDecodeRows * m->cfg.n_head * 4);
    return fail(SNLP_ERR_TIMEOUT, "a device-side bounded wait expired; results of the calls since the last check are invalid");
  }
  return SNLP_OK;
}

extern "C" int snlp_launch_count(const snlp_model *m, int64_t *count_out) {
  if (!m || !count_out) return fail(SNLP_ERR_ARG, "snlp_launch_count: NULL argument");
  *count_out = m->launches;
  return SNLP_OK;
}

// ------------------------------------------------------------------------------------------------
// launch sequences
template <typename T>
static int gemm(snlp_model *m, cudaStream_t st, int cls, const T *A, size_t a_ls, const T *W, size_t w_ls, float *C, size_t c_ls, int M,
                int N, int K, int nl) {
  dim3 grid((N + 63) / 64, (M + 63) / 64, nl);
  KLAUNCH(m, st, cls, k_gemm_nt<T><<<grid, 256, 0, st>>>(A, a_ls, W, w_ls, C, c_ls, M, N, K));
  return SNLP_OK;
}

// The structured correction over `nsteps` steps of `lstep` layers starting at state l0 (lstep > 1: fused chunks).
// a/m: branch outputs at the first layer slot of every step, each the sum of `*_splits` arrays `*_ss` elements apart.
static int correct(snlp_model *m, const Fwd &f, int l0, int nsteps, int lstep, int mode, int a_splits, size_t a_ss, int m_splits, size_t m_ss,
                   float *resnorm) {
  const int nl = nsteps;
  const snlp_config &c = m->cfg;
  CorrParams p{};
  p.trace = m->trace;
  p.a = m->a;
  p.m = m->mb;
  p.a_ss = a_ss;
  p.m_ss = m_ss;
  p.lstep = lstep;
  p.a_splits = a_splits;
  p.m_splits = m_splits;
  p.l0 = l0;
  p.nl = nl;
  p.L = c.n_layer;
  p.M = f.M;
  p.d = c.d_model;
  p.mode = mode;
  p.implicit_old = f.implicit_state >= 0 ? 1 : 0;
  p.skip_next = f.last_pass && f.M > kDecodeRows ? 1 : 0;   // the decode regime's LM head reads slot L of xb
  p.coef = m->coef;
  p.xa = umma_path_ok(m) ? nullptr : m->xa;   // the tensor-core path reads the bf16 copy xb instead
  p.xm = m->xm;
  p.xb = umma_path_ok(m) ? (__nv_bfloat16 *)m->xn : nullptr;
  p.ssq_x = m->ssq_x;
  p.partial = resnorm ? m->corr_part : nullptr;
  p.resnorm = resnorm;
  p.counter = m->counter;
  const size_t total = (size_t)f.M * (c.d_model / 4);
  const int threads = 256;
  const unsigned blocks = (unsigned)((total + threads - 1) / threads);
  const size_t sm = corr_ring_bytes(c.n_streams, threads) + (resnorm ? (size_t)(threads / 32) * nl * 2 * sizeof(float) : 0) +
                    (c.n_streams > 1 ? (size_t)nl * corr_coef_stride(c.n_streams) * sizeof(float) : 0);
  if (sm > corr_ring_bytes(c.n_streams, threads) + kCorrExtraSmem) return fail(SNLP_ERR_UNSUPPORTED, "correction: too many layers in one range");
  const size_t sm_small = (size_t)nl * 32 * (2 + c.n_streams) * sizeof(float4) + (size_t)nl * 2 * sizeof(float) + (size_t)nl * 3 * 32 * sizeof(float);
  if (f.M <= kDecodeRows && c.n_streams <= 4 && sm_small <= kCorrSmallSmem) {
    dim3 grid((c.d_model / 4 + 31) / 32, f.M);
    TimedLaunch tl_(m, f.st, KC_CORRECT);
    switch (c.n_streams) {
#define CASE(NS) case NS: launch_pdl(m->pdl_now, k_correct_small<NS>, grid, dim3(32 * kCorrSmallWarps), sm_small, f.st, p); break;
      CASE(1) CASE(2) CASE(3) CASE(4)
#undef CASE
    }
  } else {
    TimedLaunch tl_(m, f.st, KC_CORRECT);
    const bool native = c.n_streams == 1 ? mode != SNLP_MODE_NOCORR : mode == SNLP_MODE_HCN;
    switch (c.n_streams) {
#define CASE(NS) case NS: if (native) k_correct<NS, true><<<blocks, threads, sm, f.st>>>(p); else k_correct<NS, false><<<blocks, threads, sm, f.st>>>(p); break;
      CASE(1) CASE(2) CASE(3) CASE(4) CASE(5) CASE(6) CASE(7) CASE(8)
#undef CASE
    }
  }
  LAUNCH_CHECK();
  return SNLP_OK;
}

// Blocks l0 .. l0+nl-1 (branch outputs a, m; the correction is separate).  fuse == 1: each block on its own current
// input state.  fuse > 1: fused chunks (App. C.3): the layers of a chunk read the chunk's input; the per-layer
// attention outputs a[l] are summed by the consumer (a_splits = fuse), likewise the MLP outputs.
template <typename T>
static int blocks_generic(snlp_model *m, const Fwd &f, int l0, int nl, int fuse) {
  const snlp_config &c = m->cfg;
  const int M = f.M, d = c.d_model, ff = c.d_ff, H = c.n_head, hd = c.head_dim, n = c.n_streams;
  const size_t Md = (size_t)M * d;
  cudaStream_t st = f.st;
  // g layers per launch group, all reading the group's first state when fused
  const int g = fuse > 1 ? fuse : nl;
  for (int h0 = l0; h0 < l0 + nl; h0 += g) {
    const float *xa_src = n == 1 ? m->trace + h0 * Md : m->xa + h0 * Md;
    const float *xm_src = n == 1 ? m->trace + h0 * Md : m->xm + h0 * Md;
    T *xn = (T *)m->xn + h0 * Md, *q = (T *)m->q + h0 * Md, *att = (T *)m->att + h0 * Md;
    T *z = (T *)m->z + (size_t)h0 * M * ff;
    float *qkv = m->qkv_raw + (size_t)h0 * M * 3 * d, *a = m->a + h0 * Md, *y = m->y_raw + (size_t)h0 * M * ff, *mb = m->mb + h0 * Md;
    T *kc = (T *)f.kc + (size_t)h0 * f.kv_ls, *vc = (T *)f.vc + (size_t)h0 * f.kv_ls;
    const int nin = fuse > 1 ? 1 : g;             // distinct input states of the group
    const size_t in_ls = fuse > 1 ? 0 : Md;       // layer stride of the (possibly shared) GEMM input
    KLAUNCH(m, st, KC_OTHER, k_rmsnorm_cast<T><<<dim3(M, nin), 256, 0, st>>>(xa_src, Md, (size_t)d, 1, xn, Md, d, c.rms_eps));
    TRY(gemm<T>(m, st, KC_QKV, xn, in_ls, (const T *)m->wqkv + (size_t)h0 * 3 * d * d, (size_t)3 * d * d, qkv, (size_t)M * 3 * d, M, 3 * d, d, g));
    KLAUNCH(m, st, KC_OTHER, k_rope_qknorm_store<T><<<dim3(M, 3 * H, g), 128, 0, st>>>(qkv, (size_t)M * 3 * d, q, Md, kc, vc, f.kv_ls, f.kv_bs, f.T, H, hd, f.pos,
                                                               m->rope, c.rms_eps));
    KLAUNCH(m, st, KC_ATTN, k_attn_generic<T><<<dim3((M * H + 3) / 4, g), 128, 0, st>>>(q, Md, kc, vc, f.kv_ls, f.kv_bs, att, Md, M, f.T, H, hd, f.pos));
    TRY(gemm<T>(m, st, KC_OPROJ, att, Md, (const T *)m->wo + (size_t)h0 * d * d, (size_t)d * d, a, Md, M, d, d, g));
    KLAUNCH(m, st, KC_OTHER, k_resid_rmsnorm_cast<T><<<dim3(M, nin), 256, 0, st>>>(xm_src, Md, (size_t)d, a, Md, fuse > 1 ? fuse : 1, Md, m->coef, h0, xn, Md, d,
                                                                c.rms_eps));
    TRY(gemm<T>(m, st, KC_UP, xn, in_ls, (const T *)m->wup + (size_t)h0 * ff * d, (size_t)ff * d, y, (size_t)M * ff, M, ff, d, g));
    {
      const size_t tot = (size_t)g * M * ff;
      KLAUNCH(m, st, KC_OTHER, k_relu2_cast<T><<<(unsigned)((tot + 255) / 256), 256, 0, st>>>(y, z, tot));
    }
    TRY(gemm<T>(m, st, KC_DOWN, z, (size_t)M * ff, (const T *)m->wdn + (size_t)h0 * d * ff, (size_t)d * ff, mb, Md, M, d, ff, g));
  }
  return SNLP_OK;
}

// The tensor-core path (both regimes): bf16, head_dim 128, dims in whole 128-column tiles, weight maps built.
static bool umma_path_ok(const snlp_model *m) {
  const snlp_config &c = m->cfg;
  return m->have_wmaps && !m->force_generic && c.dtype == SNLP_DTYPE_BF16 && c.head_dim == 128 && c.d_model % 128 == 0 &&
         c.d_ff % 128 == 0 && c.d_model <= 4096;
}
static bool fused_prefill_ok(const snlp_model *m, int M) { return umma_path_ok(m) && M > kDecodeRows; }
static bool fast_decode_ok(const snlp_model *m, int M) { return umma_path_ok(m) && M <= kDecodeRows; }

// Largest K split <= want whose slices are whole 64-element k-blocks.
static int pick_ksplit(int K, int want) {
  for (int s = want; s > 1; --s)
    if (K % s == 0 && (K / s) % kUmmaBK == 0) return s;
  return 1;
}

template <int BN, int AM, int EPI>
static cudaError_t umma_attr() {
  return cudaFuncSetAttribute(k_umma_gemm<BN, AM, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, UmmaCfg<BN, AM>::kSmem);
}
template <int EPI>
static cudaError_t umma_attr_all() {
  cudaError_t e = umma_attr<128, 128, EPI>();
  if (e == cudaSuccess) e = umma_attr<256, 128, EPI>();
  if (e == cudaSuccess) e = umma_attr<128, 16, EPI>();
  if (e == cudaSuccess) e = umma_attr<256, 16, EPI>();
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_umma_gemm2<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kU2Smem);
  return e;
}

// Column width of a decode-regime launch.  A launch that does not occupy every SM (a sequential step's single layer: 5-20
// items) lasts as long as one item.  The column tiling does not touch the numbers (every output column is its own dot
// product), so a launch whose 128-wide items still fit one round over the SMs takes those: twice the CTAs, half the bytes
// each.  Beyond that the 256-wide tile is the faster one (the thread that issues the products spends 55-100 cycles per
// instruction of any width, so 128-wide tiles, 4 KB of weights per instruction, stream at roughly half the rate per CTA).
// The out-projection's partial sums of squares are per 128 columns in this regime, whatever the tile width.
static int decode_bn(const snlp_model *m, const WMap &w, int N, int ksplit, int nl) {
  return (w.BN == 256 && (N / 128) * ksplit * nl <= m->n_sm) ? 128 : w.BN;
}

// A product ready to be launched: C[l] = A[l] (M x K bf16, activations) * W[l0 + l]^T (N x K bf16, stacked weights), nl
// layers, `ksplit` K slices.
struct GemmLaunch {
  CUtensorMap ta;
  const CUtensorMap *tmw;
  UmmaParams p;
  int bn, grid;
  bool small, pairs;
};

// k-blocks per bulk-tensor copy of a decode-regime product whose items reduce over nkb1 k-blocks: as many as divide it,
// up to 64 KB of weights per copy
static int best_kbox(int bn, int nkb1) {
  if (bn == 128 && nkb1 % 4 == 0) return 4;
  return nkb1 % 2 == 0 ? 2 : 1;
}

// bn_force: 0 = choose the column width; 128 / 256 = use that one (decode regime; the phases of a chained launch share it,
// and the box depth kbox_force)
static int umma_prepare(snlp_model *m, GemmLaunch &g, int epi, const __nv_bfloat16 *A, size_t a_ls, const WMap &w, int l0, UmmaParams p, int M, int N,
                        int K, int ksplit, int nl, int bn_force = 0, int kbox_force = 0) {
  const bool small = M <= kDecodeRows;
  if (epi == UEPI_LMHEAD && !small) return fail(SNLP_ERR_UNSUPPORTED, "LM-head epilogue needs <= %d rows", kDecodeRows);
  if (p.a_share < 1) p.a_share = 1;
  if (p.kfuse < 1) p.kfuse = 1;
  if (!small && !make_tmap_bf16(m->encode_tiled, &g.ta, A, K, M, (uint64_t)nl * p.kfuse, a_ls ? a_ls : (size_t)M * K, kUmmaBM))
    return fail(SNLP_ERR_CUDA, "cuTensorMapEncodeTiled failed (M=%d K=%d)", M, K);
  p.kbox = 1;
  p.M = M; p.N = N; p.K = K; p.ksplit = ksplit; p.kslice = K / ksplit;
  p.Mt = small ? 1 : (M + kUmmaBM - 1) / kUmmaBM; p.Nt = N / w.BN; p.nl = nl; p.l0 = l0; p.err = m->dev_err;
  g.small = small;
  g.pairs = !small && w.BN == 256 && M > kUmmaBM && epi != UEPI_LMHEAD;
  if (g.pairs) {
    // prefill regime with more than one row tile: 256 x 256 tiles on CTA pairs (same results, less operand traffic per SM)
    p.Mt = (M + 2 * kUmmaBM - 1) / (2 * kUmmaBM);
    p.nstages = kU2Stages;
    const int items2 = p.Mt * p.Nt * ksplit * nl, pairs = items2 < m->n_sm / 2 ? items2 : m->n_sm / 2;
    g.bn = 256; g.grid = 2 * pairs; g.tmw = &w.tm_half; g.p = p;
    return SNLP_OK;
  }
  int bn = w.BN;
  if (small) {
    bn = bn_force ? bn_force : decode_bn(m, w, N, ksplit, nl);
    if (K / ksplit / kUmmaBK != w.nkb1) return fail(SNLP_ERR_UNSUPPORTED, "decode-regime product: K slice %d does not match the weight maps", K / ksplit);
    p.kbox = kbox_force ? kbox_force : best_kbox(bn, w.nkb1);
    const int ki = p.kbox == 4 ? 2 : p.kbox == 2 ? 1 : 0;
    g.tmw = bn == 256 ? &w.td256[ki] : &w.td128[ki];
    if (!make_tmap_bf16_kb(m->encode_tiled, &g.ta, A, K, M, (uint64_t)nl * p.kfuse, a_ls ? a_ls : (size_t)M * K, 16, p.kbox))
      return fail(SNLP_ERR_CUDA, "cuTensorMapEncodeTiled failed (M=%d K=%d)", M, K);
  } else {
    g.tmw = bn == w.BN ? &w.tm : &w.tm_half;
  }
  p.Nt = N / bn;
  const int items = p.Mt * p.Nt * ksplit * nl;
  g.bn = bn; g.grid = items < m->n_sm ? items : m->n_sm;
  g.p = p;
  return SNLP_OK;
}

template <int EPI>
static int umma_gemm(snlp_model *m, cudaStream_t st, int cls, const __nv_bfloat16 *A, size_t a_ls, const WMap &w, int l0, UmmaParams p,
                     int M, int N, int K, int ksplit, int nl) {
  GemmLaunch g;
  TRY(umma_prepare(m, g, EPI, A, a_ls, w, l0, p, M, N, K, ksplit, nl));
  if (g.pairs) {
    KLAUNCH(m, st, cls, k_umma_gemm2<EPI><<<g.grid, kUmmaThreads, kU2Smem, st>>>(g.ta, *g.tmw, g.p));
    return SNLP_OK;
  }
  const bool pdl_ = m->pdl_now;
#define SNLP_UMMA_LAUNCH(BN_, AM_)                                                                                                   \
  do {                                                                                                                               \
    g.p.nstages = UmmaCfg<BN_, AM_>::kStages;                                                                                        \
    KLAUNCH(m, st, cls, launch_pdl(pdl_, k_umma_gemm<BN_, AM_, EPI>, dim3(g.grid), dim3(kUmmaThreads), UmmaCfg<BN_, AM_>::kSmem, st, g.ta, *g.tmw, g.p)); \
  } while (0)
  if (g.bn == 256) {
    if (g.small) SNLP_UMMA_LAUNCH(256, 16);
    else if (EPI != UEPI_LMHEAD) SNLP_UMMA_LAUNCH(256, 128);
  } else {
    if (g.small) SNLP_UMMA_LAUNCH(128, 16);
    else if (EPI != UEPI_LMHEAD) SNLP_UMMA_LAUNCH(128, 128);
  }
#undef SNLP_UMMA_LAUNCH
  return SNLP_OK;
}

// Decode regime: the three products that follow the attention -- out-projection, MLP up, MLP down -- as one cooperative
// launch whose phases are separated by grid barriers (umma_chain.cuh).  Same items and epilogues as three launches.
static int umma_chain3(snlp_model *m, cudaStream_t st, GemmLaunch (&g)[3], const int (&epi)[3], ChainParams &cp) {
  cp.nphase = 3;
  cp.bar = m->chain_bar;
  for (int i = 0; i < 3; ++i) {
    cp.tmA[i] = g[i].ta; cp.tmB[i] = *g[i].tmw; cp.p[i] = g[i].p; cp.epi[i] = epi[i];
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(m->n_sm); cfg.blockDim = dim3(kUmmaThreads); cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;   // every CTA must be resident: they wait for one another at the phase barriers
  attr[0].val.cooperative = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  if (g[0].bn == 256) {
    cfg.dynamicSmemBytes = UmmaCfg<256, 16>::kSmem;
    KLAUNCH(m, st, KC_UP, cudaLaunchKernelEx(&cfg, k_umma_chain<256>, cp));
  } else {
    cfg.dynamicSmemBytes = UmmaCfg<128, 16>::kSmem;
    KLAUNCH(m, st, KC_UP, cudaLaunchKernelEx(&cfg, k_umma_chain<128>, cp));
  }
  return SNLP_OK;
}

// The blocks of layers l0 .. l0+nl-1 on the tensor-core path: five launches whatever nl (the correction is the sixth).
// The four projections run on k_umma_gemm with the rest of the block fused into their epilogues (row RMSNorm
// as a scale, rotary + QK-norm + KV store, residual add + sum of squares, ReLU^2); the bf16 branch inputs
// xb/ssq_x of the range must be current (prep_rows, or the previous correction).
static int down_splits(const snlp_model *m, int M);

static int blocks_umma(snlp_model *m, const Fwd &f, int l0, int nl, int fuse) {
  typedef __nv_bfloat16 T;
  const snlp_config &c = m->cfg;
  const int M = f.M, d = c.d_model, ff = c.d_ff, H = c.n_head, n = c.n_streams, P = d / 128, L = c.n_layer;
  const bool small = M <= kDecodeRows;
  const size_t Md = (size_t)M * d;
  cudaStream_t st = f.st;
  // residual stream read by the out-projection epilogue: h_l (single stream; before the first correction every h_l is
  // still the one materialised state), or the fp32 MLP pre-map (mHC)
  const bool implicit = n == 1 && f.implicit_state >= 0;
  const float *xm_src = n == 1 ? m->trace + (implicit ? f.implicit_state : l0) * Md : m->xm + l0 * Md;
  T *xb = (T *)m->xn + l0 * Md, *ub = (T *)m->ub + l0 * Md, *q = (T *)m->q + l0 * Md, *att = (T *)m->att + l0 * Md;
  T *z = (T *)m->z + (size_t)l0 * M * ff;
  float *a = m->a + l0 * Md, *mb = m->mb + l0 * Md;
  T *kc = (T *)f.kc + (size_t)l0 * f.kv_ls, *vc = (T *)f.vc + (size_t)l0 * f.kv_ls;
  const int Pu = small ? d / 128 : 2 * (d / m->w_o.BN);  // partials of sum u^2: one per 128 columns (decode regime), two per column tile of the out-projection
  const int sd = down_splits(m, M);
  const bool chained = small && m->use_chain;   // the three products after the attention as one launch, which also merges the attention's chunk partials
  int comb_nchunk = 0;
  bool comb = false;
  {
    UmmaParams p{};
    p.ssq = m->ssq_x + (size_t)l0 * P * M; p.nparts = P; p.eps = c.rms_eps;
    p.q = q; p.q_ls = Md; p.kc = kc; p.vc = vc; p.kv_ls = f.kv_ls; p.kv_bs = f.kv_bs;
    p.T = f.T; p.d = d; p.pos_base = f.pos; p.rope = m->rope; p.rope_t = m->rope_t; p.rope_ld = c.max_ctx; p.qk_eps = c.rms_eps;
    p.a_share = fuse;
    TRY(umma_gemm<UEPI_QKV>(m, st, KC_QKV, xb, Md, m->w_qkv, l0, p, M, 3 * d, d, 1, nl));
  }
  if (small) {
    const int csub = attn_csub(f.B * H);
    const int nchunk = (f.pos_hi + f.T - 1) / (csub * kAttnSub) + 1;
    // Where the chunk partials are merged.  In the attention kernel itself the CTA that arrives last at its (layer,
    // sequence, head) merges them, which puts a device-scope fence and an atomic round trip at the end of every CTA; with
    // only a few waves of CTAs (a batch-1 sweep: ~3) that tail is a fifth of the launch, and the chained launch that
    // follows merges them instead (measured: attention 46.6 -> 40.5 us, chained launch 105 -> 108 us).  With many waves
    // (batch 8) or a single layer the tail is hidden or the chain's extra step costs as much: merged in place.  The same
    // function merges in both places: no bit depends on the choice.
    comb = chained && nl > 1 && (long long)nchunk * f.B * H * nl <= 16LL * m->n_sm;
    KLAUNCH(m, st, KC_ATTN, launch_pdl(m->pdl_now, k_attn_decode, dim3(nchunk, f.B * H, nl), dim3(128), 0, st, (const __nv_bfloat16 *)q, Md, (const __nv_bfloat16 *)kc,
                                       (const __nv_bfloat16 *)vc, f.kv_ls, f.kv_bs, m->attn_part, m->attn_counters, att, Md, f.T, H, f.pos, csub,
                                       comb ? 0 : 1));
    comb_nchunk = nchunk;
  } else {
    // tensor-core attention: 128-query items over the (layer, sequence, head, query tile) grid, persistent CTAs
    CUtensorMap tq, tk, tv, to;
    if (!make_tmap_bf16(m->encode_tiled, &tq, q, d, M, nl, Md, kFuTile) ||
        !make_tmap_kv(m->encode_tiled, &tk, kc, d, f.kv_rows, f.B, nl, f.kv_bs, f.kv_ls) ||
        !make_tmap_kv(m->encode_tiled, &tv, vc, d, f.kv_rows, f.B, nl, f.kv_bs, f.kv_ls) ||
        !make_tmap_kv(m->encode_tiled, &to, att, d, f.T, f.B, nl, (size_t)f.T * d, Md))
      return fail(SNLP_ERR_CUDA, "cuTensorMapEncodeTiled failed for the attention operands");
    FaUmmaParams ap{};
    ap.T = f.T; ap.H = H; ap.BH = f.B * H; ap.nq = (f.T + kFuTile - 1) / kFuTile;
    ap.n_items = ap.nq * ap.BH * nl; ap.pos_base = f.pos; ap.err = m->dev_err;
    const int grid = ap.n_items < m->n_sm ? ap.n_items : m->n_sm;
    KLAUNCH(m, st, KC_ATTN, k_attn_umma<<<grid, kFuThreads, kFuSmem, st>>>(tq, tk, tv, to, ap, nl));
  }
  UmmaParams po{}, pu{}, pd{};
  po.c = a; po.z = ub; po.out_ls = Md;
  po.xm = xm_src; po.xm_ls = implicit ? 0 : Md; po.coef = m->coef + l0; po.ssq_out = m->ssq_u + (size_t)l0 * Pu * M;
  po.kfuse = fuse;   // a chunk's out-projections are one product over the concatenated attention outputs
  pu.z = z; pu.out_ls = (size_t)M * ff;
  pu.ssq = m->ssq_u + (size_t)l0 * Pu * M; pu.nparts = Pu; pu.eps = c.rms_eps;
  pu.a_share = fuse;
  pd.c = mb; pd.out_ls = Md; pd.out_ss = (size_t)L * Md;
  pd.kfuse = fuse;
  if (chained) {
    // one cooperative launch for the three products; a common column width: 256 as soon as one of them wants it
    const int b0 = decode_bn(m, m->w_o, d, 1, nl / fuse), b1 = decode_bn(m, m->w_up, ff, 1, nl), b2 = decode_bn(m, m->w_dn, d, sd, nl / fuse);
    const bool all256 = m->w_o.BN == 256 && m->w_up.BN == 256 && m->w_dn.BN == 256;
    const int bn = (all256 && (b0 == 256 || b1 == 256 || b2 == 256)) ? 256 : 128;
    // ... and a common box depth: the three products share the ring
    const int kbox = best_kbox(bn, std::gcd(std::gcd(m->w_o.nkb1, m->w_up.nkb1), m->w_dn.nkb1));
    GemmLaunch g[3];
    TRY(umma_prepare(m, g[0], UEPI_RESID, att, Md, m->w_o, l0, po, M, d, d, 1, nl / fuse, bn, kbox));
    TRY(umma_prepare(m, g[1], UEPI_RELU2_BF16, ub, Md, m->w_up, l0, pu, M, ff, d, 1, nl, bn, kbox));
    TRY(umma_prepare(m, g[2], UEPI_F32, z, (size_t)M * ff, m->w_dn, l0, pd, M, d, ff, sd, nl / fuse, bn, kbox));
    const int epi[3] = {UEPI_RESID, UEPI_RELU2_BF16, UEPI_F32};
    ChainParams cp{};
    cp.kbox = kbox;
    cp.comb_part = m->attn_part; cp.comb_out = att; cp.comb_o_ls = Md;
    cp.comb_rows = comb ? nl * f.B * H * f.T : 0; cp.comb_nchunk = comb_nchunk; cp.comb_Tq = f.T; cp.comb_BH = f.B * H; cp.comb_H = H; cp.comb_d = d;
    TRY(umma_chain3(m, st, g, epi, cp));
    return SNLP_OK;
  }
  TRY(umma_gemm<UEPI_RESID>(m, st, KC_OPROJ, att, Md, m->w_o, l0, po, M, d, d, 1, nl / fuse));
  TRY(umma_gemm<UEPI_RELU2_BF16>(m, st, KC_UP, ub, Md, m->w_up, l0, pu, M, ff, d, 1, nl));
  TRY(umma_gemm<UEPI_F32>(m, st, KC_DOWN, z, (size_t)M * ff, m->w_dn, l0, pd, M, d, ff, sd, nl / fuse));
  return SNLP_OK;
}

// K split of the decode-regime down-projection (its reduction is the longest); it does not depend on how many
// layers a launch covers, so sequential execution and layer-parallel sweeps add the partial sums in the same order.
static int down_splits(const snlp_model *m, int M) {
  return (umma_path_ok(m) && M <= kDecodeRows) ? pick_ksplit(m->cfg.d_ff, kMaxSplits) : 1;
}

// bf16 branch inputs of layers l0 .. l0+nl-1 for blocks_umma (and the fp32 MLP pre-map of mHC models)
static int prep_rows(snlp_model *m, const Fwd &f, int l0, int nl) {
  const snlp_config &c = m->cfg;
  dim3 grid(f.M, nl);
  const int threads = c.d_model / 4;
  switch (c.n_streams) {
#define CASE(NS) case NS: KLAUNCH(m, f.st, KC_OTHER, launch_pdl(m->pdl_now, k_prep_rows<NS>, grid, dim3(threads), 0, f.st, (const float *)m->trace, l0, f.M, c.d_model, (const HcCoef *)m->coef, (__nv_bfloat16 *)m->xn, m->ssq_x, m->xm)); break;
    CASE(1) CASE(2) CASE(3) CASE(4) CASE(5) CASE(6) CASE(7) CASE(8)
#undef CASE
  }
  return SNLP_OK;
}

static int init_kernel_attributes() {
  CU(umma_attr_all<UEPI_F32>());
  CU(umma_attr_all<UEPI_RELU2_BF16>());
  CU(umma_attr_all<UEPI_QKV>());
  CU(umma_attr_all<UEPI_RESID>());
  CU((umma_attr<128, 16, UEPI_LMHEAD>()));
  CU((umma_attr<256, 16, UEPI_LMHEAD>()));
  CU(cudaFuncSetAttribute(k_umma_chain<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, UmmaCfg<128, 16>::kSmem));
  CU(cudaFuncSetAttribute(k_umma_chain<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, UmmaCfg<256, 16>::kSmem));
  CU(cudaFuncSetAttribute(k_attn_umma, cudaFuncAttributeMaxDynamicSharedMemorySize, kFuSmem));
#define ATTR(NS) CU(cudaFuncSetAttribute(k_correct<NS, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(corr_ring_bytes(NS, 256) + kCorrExtraSmem))); \
  CU(cudaFuncSetAttribute(k_correct<NS, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(corr_ring_bytes(NS, 256) + kCorrExtraSmem)));
  ATTR(1) ATTR(2) ATTR(3) ATTR(4) ATTR(5) ATTR(6) ATTR(7) ATTR(8)
#undef ATTR
  CU(cudaFuncSetAttribute(k_correct_small<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCorrSmallSmem));
  CU(cudaFuncSetAttribute(k_correct_small<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCorrSmallSmem));
  CU(cudaFuncSetAttribute(k_correct_small<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCorrSmallSmem));
  CU(cudaFuncSetAttribute(k_correct_small<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kCorrSmallSmem));
  return SNLP_OK;
}

static int run_blocks(snlp_model *m, const Fwd &f, int l0, int nl, int fuse = 1) {
  if (umma_path_ok(m)) return blocks_umma(m, f, l0, nl, fuse);
  if (m->cfg.dtype == SNLP_DTYPE_BF16) return blocks_generic<__nv_bfloat16>(m, f, l0, nl, fuse);
  return blocks_generic<float>(m, f, l0, nl, fuse);
}

// The correction over layers l0 .. l0+nl-1 in steps of `fuse` layers, on the branch outputs run_blocks left.
static int correct_range(snlp_model *m, const Fwd &f, int l0, int nl, int fuse, int mode, float *resnorm) {
  const size_t Md = (size_t)f.M * m->cfg.d_model;
  if (umma_path_ok(m))  // a, m at the chunk's first layer slot; m possibly in K-split partials
    return correct(m, f, l0, nl / fuse, fuse, mode, 1, 0, down_splits(m, f.M), (size_t)m->cfg.n_layer * Md, resnorm);
  return correct(m, f, l0, nl / fuse, fuse, mode, fuse, Md, fuse, Md, resnorm);  // per-layer outputs, summed here
}

static int native_mode(const snlp_model *m) { return m->cfg.n_streams > 1 ? SNLP_MODE_HCN : SNLP_MODE_IDN; }

static int premix(snlp_model *m, const Fwd &f, int l0, int nl) {
  const snlp_config &c = m->cfg;
  if (c.n_streams == 1) return SNLP_OK;
  const size_t Md = (size_t)f.M * c.d_model;
  KLAUNCH(m, f.st, KC_OTHER, k_premix<<<dim3((unsigned)((Md + 255) / 256), nl), 256, 0, f.st>>>(m->trace, Md * c.n_streams, c.n_streams, c.d_model, Md, m->coef, l0,
                                                                    m->xa, m->xm, Md));
  return SNLP_OK;
}

static int check_solver(const snlp_model *m, const snlp_solver &sol, const char *who) {
  const int L = m->cfg.n_layer;
  if (sol.mode < SNLP_MODE_IDN || sol.mode > SNLP_MODE_SEQUENTIAL) return fail(SNLP_ERR_ARG, "%s: unknown mode %d", who, sol.mode);
  if (sol.K < 0) return fail(SNLP_ERR_ARG, "%s: K must be >= 0 (got %d)", who, sol.K);
  if (sol.prefix < 0 || sol.prefix > L) return fail(SNLP_ERR_ARG, "%s: prefix must be in 0..%d (got %d)", who, L, sol.prefix);
  if (sol.init != SNLP_INIT_H0 && sol.init != SNLP_INIT_FWD) return fail(SNLP_ERR_ARG, "%s: unknown init %d", who, sol.init);
  if (sol.fuse < 1) return fail(SNLP_ERR_ARG, "%s: fuse must be >= 1 (got %d)", who, sol.fuse);
  if (sol.fuse > 1) {
    if (m->cfg.n_streams != 1) return fail(SNLP_ERR_UNSUPPORTED, "%s: fused chunks need a single-stream model", who);
    if ((L - sol.prefix) % sol.fuse) return fail(SNLP_ERR_ARG, "%s: suffix length %d is not a multiple of fuse = %d", who, L - sol.prefix, sol.fuse);
    if (sol.mode == SNLP_MODE_HCN) return fail(SNLP_ERR_ARG, "%s: fused chunks use the identity surrogate (mode IDN or NOCORR)", who);
  }
  return SNLP_OK;
}

static int embed_impl(snlp_model *m, cudaStream_t st, const int32_t *ids, int rows, float *h0, const int32_t *const *ids_pp = nullptr);

// General Alg. 2 over the internal trace (trace[0] must hold h_0, or f.embed_ids the tokens it is the embedding of): sequential prefix, initialisation, K sweeps over the
// suffix in chunks of `fuse` fused layers (Eq. 5 for fuse = 1, Eq. 11 otherwise).
static int solve(snlp_model *m, const Fwd &f, const snlp_solver &sol, float *resnorm_out) {
  const snlp_config &c = m->cfg;
  const int L = c.n_layer, F = sol.fuse;
  const bool seq = sol.mode == SNLP_MODE_SEQUENTIAL;
  const int S = (seq && F == 1) ? L : sol.prefix;
  // a decode step hands over token ids instead of state 0: the initialisation kernel embeds them itself where it runs
  // on state 0; every other path needs the embedding first
  const bool have_ids = f.embed_ids != nullptr || f.embed_ids_pp != nullptr;
  const bool fused_embed = have_ids && umma_path_ok(m) && S == 0 && !seq;
  if (have_ids && !fused_embed) TRY(embed_impl(m, f.st, f.embed_ids, f.M, m->trace, f.embed_ids_pp));
  if (resnorm_out && sol.K > 0 && !seq) CU(cudaMemsetAsync(resnorm_out, 0, (size_t)sol.K * L * 2 * sizeof(float), f.st));
  // Layer-by-layer execution is a chain of short kernels on a few SMs each: there a kernel is launched with the
  // programmatic-serialisation attribute, so that it is scheduled while its predecessor finishes and requests its
  // first weight tiles before it waits for that kernel's results (measured: 4-5 % of a sequential decode step).  The
  // launches of a sweep fill the GPU; they gain nothing from it (measured: 2-8 % slower) and are launched normally.
  struct PdlScope {
    snlp_model *m;
    PdlScope(snlp_model *m_, int rows) : m(m_) { m->pdl_now = m->use_pdl != 0 && rows <= kDecodeRows; }   // decode regime only
    ~PdlScope() { m->pdl_now = false; }
  };
  if (S > 0) {  // Alg. 2 lines 2-4
    PdlScope pdl(m, f.M);
    if (umma_path_ok(m)) TRY(prep_rows(m, f, 0, 1));
    else TRY(premix(m, f, 0, 1));
    for (int l = 0; l < S; ++l) {
      TRY(run_blocks(m, f, l, 1));
      TRY(correct_range(m, f, l, 1, 1, native_mode(m), nullptr));
    }
  }
  if (S == L) return SNLP_OK;
  if (seq) {  // sequential execution of the fused model: chunk after chunk
    PdlScope pdl(m, f.M);
    if (umma_path_ok(m)) TRY(prep_rows(m, f, S, 1));
    for (int h = S; h < L; h += F) {
      TRY(run_blocks(m, f, h, F, F));
      TRY(correct_range(m, f, h, F, F, SNLP_MODE_IDN, nullptr));
    }
    return SNLP_OK;
  }
  // Alg. 2 line 5: every suffix state starts at h_S
  if (umma_path_ok(m)) {
    switch (c.n_streams) {   // one kernel: the copies and the layers' first branch inputs
#define CASE(NS) case NS: KLAUNCH(m, f.st, KC_OTHER, launch_pdl(m->pdl_now, k_init_rows<NS>, dim3(f.M), dim3(c.d_model / 4), 0, f.st, m->trace, S, L, f.M, c.d_model, (const HcCoef *)m->coef, (__nv_bfloat16 *)m->xn, m->ssq_x, m->xm, 0, fused_embed ? f.embed_ids : (const int32_t *)nullptr, (const __nv_bfloat16 *)m->embed, c.vocab, fused_embed ? f.embed_ids_pp : (const int32_t *const *)nullptr)); break;
      CASE(1) CASE(2) CASE(3) CASE(4) CASE(5) CASE(6) CASE(7) CASE(8)
#undef CASE
    }
  } else {
    const size_t n4 = (size_t)f.M * c.n_streams * c.d_model / 4;
    KLAUNCH(m, f.st, KC_OTHER, k_bcast_trace<<<(unsigned)((n4 + 255) / 256), 256, 0, f.st>>>(reinterpret_cast<const float4 *>(m->trace) + (size_t)S * n4,
                                                                 reinterpret_cast<float4 *>(m->trace) + (size_t)(S + 1) * n4, n4, L - S));
    TRY(premix(m, f, S, L - S));
  }
  int exact = S;  // states 0..exact equal the sequential trace (of the fused model when F > 1)
  // On the tensor-core path the copies of h_S are not written: the first pass reads h_S itself wherever it needs a later
  // state, and its correction writes every state for the first time.
  Fwd first = f;
  if (umma_path_ok(m)) first.implicit_state = S;
  bool fresh = true;
  if (umma_path_ok(m) && sol.K == 0 && sol.init != SNLP_INIT_FWD) {   // nothing will write the states: materialise them after all
    const size_t n4 = (size_t)f.M * c.n_streams * c.d_model / 4;
    KLAUNCH(m, f.st, KC_OTHER, k_bcast_trace<<<(unsigned)((n4 + 255) / 256), 256, 0, f.st>>>(reinterpret_cast<const float4 *>(m->trace) + (size_t)S * n4,
                                                                 reinterpret_cast<float4 *>(m->trace) + (size_t)(S + 1) * n4, n4, L - S));
  }
  if (sol.init == SNLP_INIT_FWD) {
    // one batched evaluation of every suffix chunk on h_S; with A = 0 the correction just stores F(h_S)
    TRY(run_blocks(m, first, S, L - S, F));
    TRY(correct_range(m, first, S, L - S, F, SNLP_MODE_NOCORR, nullptr));
    exact = S + F;
    fresh = false;
  }
  for (int k = 0; k < sol.K; ++k) {
    // Exactness-aware trimming: entering this sweep the states 0..exact already equal the sequential trace (Newton
    // on a block lower-bidiagonal system), so chunks before `exact` would reproduce, bit for bit, the branch
    // outputs they wrote in the previous pass.  Only chunks from `exact` on are evaluated; the correction still runs
    // over the whole suffix on the stored branch outputs, so trace, residual norms and next inputs are unchanged.
    const int b0 = exact < L ? exact : L;
    Fwd fk = fresh ? first : f;
    fk.last_pass = k == sol.K - 1;
    if (b0 < L) TRY(run_blocks(m, fk, b0, L - b0, F));
    TRY(correct_range(m, fk, S, L - S, F, sol.mode, resnorm_out ? resnorm_out + (size_t)k * L * 2 : nullptr));
    fresh = false;
    exact += F;
  }
  return SNLP_OK;
}

static int sequential(snlp_model *m, const Fwd &f) {
  snlp_solver sol{0, SNLP_MODE_SEQUENTIAL, m->cfg.n_layer, SNLP_INIT_H0, 1};
  return solve(m, f, sol, nullptr);
}

static int parallel(snlp_model *m, const Fwd &f, int K, int mode, float *resnorm_out) {
  snlp_solver sol{K, mode, 0, SNLP_INIT_H0, 1};
  return solve(m, f, sol, resnorm_out);
}

// LMHead on `rows` hidden states.  pre_xb / pre_ssq: the bf16 stream-summed rows and their sums of squares if the
// caller already has them (slot L of the branch-input buffers after a decode-regime forward), else NULL.
static int lm_head_impl(snlp_model *m, cudaStream_t st, const float *hL, size_t row_stride, int rows, float *logits, int32_t *argmax,
                        const __nv_bfloat16 *pre_xb = nullptr, const float *pre_ssq = nullptr, int *bump = nullptr,
                        int32_t *const *argmax_pp = nullptr) {
  const bool want_argmax = argmax != nullptr || argmax_pp != nullptr;
  const snlp_config &c = m->cfg;
  const int d = c.d_model, V = c.vocab, n = c.n_streams;
  if (umma_path_ok(m) && rows <= kDecodeRows) {
    const int P = d / 128;
    if (!pre_xb) {
      KLAUNCH(m, st, KC_LMHEAD, k_prep_lm<<<rows, d / 4, 0, st>>>(hL, row_stride, n, rows, d, (__nv_bfloat16 *)m->xlm, m->ssq_lm));
      pre_xb = (const __nv_bfloat16 *)m->xlm;
      pre_ssq = m->ssq_lm;
    }
    UmmaParams p{};
    p.ssq = pre_ssq; p.nparts = P; p.eps = c.rms_eps;
    p.logits = logits; p.pm_val = m->pm_val; p.pm_idx = m->pm_idx;
    p.argmax = argmax; p.argmax_pp = argmax_pp; p.bump = want_argmax ? bump : nullptr; p.lm_counter = m->lm_counter;   // the last CTA merges the tiles' maxima
    TRY(umma_gemm<UEPI_LMHEAD>(m, st, KC_LMHEAD, pre_xb, 0, m->w_lm, 0, p, rows, V, d, 1, 1));
    if (!want_argmax && bump) KLAUNCH(m, st, KC_OTHER, k_add_int<<<1, 1, 0, st>>>(bump, 1));
    return SNLP_OK;
  }
  for (int r0 = 0; r0 < rows; r0 += m->logit_rows) {
    const int nr = rows - r0 < m->logit_rows ? rows - r0 : m->logit_rows;
    float *lg = logits ? logits + (size_t)r0 * V : m->logits;
    const float *src = hL + (size_t)r0 * row_stride;
    if (c.dtype == SNLP_DTYPE_BF16) {
      typedef __nv_bfloat16 T;
      KLAUNCH(m, st, KC_OTHER, k_rmsnorm_cast<T><<<dim3(nr, 1), 256, 0, st>>>(src, 0, row_stride, n, (T *)m->xlm, 0, d, c.rms_eps));
      TRY(gemm<T>(m, st, KC_LMHEAD, (const T *)m->xlm, 0, (const T *)m->lm_head, 0, lg, 0, nr, V, d, 1));
    } else {
      typedef float T;
      KLAUNCH(m, st, KC_OTHER, k_rmsnorm_cast<T><<<dim3(nr, 1), 256, 0, st>>>(src, 0, row_stride, n, (T *)m->xlm, 0, d, c.rms_eps));
      TRY(gemm<T>(m, st, KC_LMHEAD, (const T *)m->xlm, 0, (const T *)m->lm_head, 0, lg, 0, nr, V, d, 1));
    }
    if (want_argmax) {
      KLAUNCH(m, st, KC_LMHEAD, k_argmax_rows<<<nr, 256, 0, st>>>(lg, V, argmax ? argmax + r0 : nullptr, argmax_pp, r0));
    }
  }
  return SNLP_OK;
}

static int embed_impl(snlp_model *m, cudaStream_t st, const int32_t *ids, int rows, float *h0, const int32_t *const *ids_pp) {
  const snlp_config &c = m->cfg;
  if (c.dtype == SNLP_DTYPE_BF16)
    KLAUNCH(m, st, KC_OTHER, k_embed<__nv_bfloat16><<<rows, 128, 0, st>>>(ids, (const __nv_bfloat16 *)m->embed, h0, c.d_model, c.n_streams, c.vocab, ids_pp));
  else
    KLAUNCH(m, st, KC_OTHER, k_embed<float><<<rows, 128, 0, st>>>(ids, (const float *)m->embed, h0, c.d_model, c.n_streams, c.vocab, ids_pp));
  return SNLP_OK;
}

// ------------------------------------------------------------------------------------------------
// public entry points
static int check_model(const snlp_model *m, const char *who) {
  if (!m) return fail(SNLP_ERR_ARG, "%s: NULL model handle", who);
  if (!m->loaded) return fail(SNLP_ERR_STATE, "%s: weights not loaded", who);
  return SNLP_OK;
}

// The kernels read and write hidden states with 16-byte accesses; a misaligned pointer is turned away on the host.
static int check_align16(const void *h0, const void *trace_out, const char *who) {
  if ((uintptr_t)h0 % 16 || (uintptr_t)trace_out % 16) return fail(SNLP_ERR_ARG, "%s: hidden-state pointers must be 16-byte aligned", who);
  return SNLP_OK;
}

static int check_shape(const snlp_model *m, int B, int T, const char *who) {
  if (B < 1 || T < 1) return fail(SNLP_ERR_ARG, "%s: B and T must be >= 1", who);
  const snlp_config &c = m->cfg;
  if ((int64_t)B * T > c.max_rows) return fail(SNLP_ERR_SHAPE, "%s: B*T = %lld exceeds max_rows = %d", who, (long long)B * T, c.max_rows);
  if (B > c.max_batch) return fail(SNLP_ERR_SHAPE, "%s: B = %d exceeds max_batch = %d", who, B, c.max_batch);
  if (T > c.max_ctx) return fail(SNLP_ERR_SHAPE, "%s: T = %d exceeds max_ctx = %d", who, T, c.max_ctx);
  return SNLP_OK;
}

extern "C" int snlp_embed(snlp_model *m, const int32_t *ids, int B, int T, float *h0, void *stream) {
  TRY(check_model(m, "snlp_embed"));
  if (!ids || !h0) return fail(SNLP_ERR_ARG, "snlp_embed: NULL pointer");
  if ((uintptr_t)ids % 4 || (uintptr_t)h0 % 16) return fail(SNLP_ERR_ARG, "snlp_embed: ids must be 4-byte aligned, h0 16-byte aligned");
  TRY(check_shape(m, B, T, "snlp_embed"));
  return embed_impl(m, (cudaStream_t)stream, ids, B * T, h0);
}

static Fwd scratch_fwd(snlp_model *m, int B, int T, cudaStream_t st) {
  Fwd f{};
  f.M = B * T; f.B = B; f.T = T;
  f.kc = m->sk; f.vc = m->sv;
  f.kv_bs = (size_t)T * m->cfg.d_model;
  f.kv_ls = (size_t)B * f.kv_bs;
  f.kv_rows = T;
  f.pos = m->zero; f.pos_hi = 0; f.st = st;
  return f;
}

extern "C" int snlp_forward_sequential(snlp_model *m, const float *h0, int B, int T, float *trace_out, void *stream) {
  TRY(check_model(m, "snlp_forward_sequential"));
  if (!h0) return fail(SNLP_ERR_ARG, "snlp_forward_sequential: NULL h0");
  TRY(check_align16(h0, trace_out, "snlp_forward_sequential"));
  TRY(check_shape(m, B, T, "snlp_forward_sequential"));
  cudaStream_t st = (cudaStream_t)stream;
  const size_t state = (size_t)B * T * m->cfg.n_streams * m->cfg.d_model;
  CU(cudaMemcpyAsync(m->trace, h0, state * 4, cudaMemcpyDeviceToDevice, st));
  Fwd f = scratch_fwd(m, B, T, st);
  TRY(sequential(m, f));
  m->last_rows = B * T;
  if (trace_out) CU(cudaMemcpyAsync(trace_out, m->trace, (m->cfg.n_layer + 1) * state * 4, cudaMemcpyDeviceToDevice, st));
  return SNLP_OK;
}

static int check_mode(int mode, const char *who) {
  if (mode != SNLP_MODE_IDN && mode != SNLP_MODE_HCN && mode != SNLP_MODE_NOCORR) return fail(SNLP_ERR_ARG, "%s: unknown mode %d", who, mode);
  return SNLP_OK;
}

extern "C" int snlp_forward_parallel(snlp_model *m, const float *h0, int B, int T, int K, int mode, float *trace_out, float *resnorm_out,
                                     void *stream) {
  TRY(check_model(m, "snlp_forward_parallel"));
  if (!h0) return fail(SNLP_ERR_ARG, "snlp_forward_parallel: NULL h0");
  TRY(check_align16(h0, trace_out, "snlp_forward_parallel"));
  if (resnorm_out && (uintptr_t)resnorm_out % 4) return fail(SNLP_ERR_ARG, "snlp_forward_parallel: resnorm_out must be 4-byte aligned");
  if (K < 1) return fail(SNLP_ERR_ARG, "snlp_forward_parallel: K must be >= 1 (got %d)", K);
  TRY(check_mode(mode, "snlp_forward_parallel"));
  TRY(check_shape(m, B, T, "snlp_forward_parallel"));
  cudaStream_t st = (cudaStream_t)stream;
  const size_t state = (size_t)B * T * m->cfg.n_streams * m->cfg.d_model;
  CU(cudaMemcpyAsync(m->trace, h0, state * 4, cudaMemcpyDeviceToDevice, st));
  Fwd f = scratch_fwd(m, B, T, st);
  TRY(parallel(m, f, K, mode, resnorm_out));
  m->last_rows = B * T;
  if (trace_out) CU(cudaMemcpyAsync(trace_out, m->trace, (m->cfg.n_layer + 1) * state * 4, cudaMemcpyDeviceToDevice, st));
  return SNLP_OK;
}

extern "C" int snlp_forward_solver(snlp_model *m, const float *h0, int B, int T, const snlp_solver *solver, float *trace_out,
                                   float *resnorm_out, void *stream) {
  TRY(check_model(m, "snlp_forward_solver"));
  if (!h0 || !solver) return fail(SNLP_ERR_ARG, "snlp_forward_solver: NULL pointer");
  TRY(check_align16(h0, trace_out, "snlp_forward_solver"));
  TRY(check_solver(m, *solver, "snlp_forward_solver"));
  TRY(check_shape(m, B, T, "snlp_forward_solver"));
  cudaStream_t st = (cudaStream_t)stream;
  const size_t state = (size_t)B * T * m->cfg.n_streams * m->cfg.d_model;
  CU(cudaMemcpyAsync(m->trace, h0, state * 4, cudaMemcpyDeviceToDevice, st));
  Fwd f = scratch_fwd(m, B, T, st);
  TRY(solve(m, f, *solver, resnorm_out));
  m->last_rows = B * T;
  if (trace_out) CU(cudaMemcpyAsync(trace_out, m->trace, (m->cfg.n_layer + 1) * state * 4, cudaMemcpyDeviceToDevice, st));
  return SNLP_OK;
}

extern "C" int snlp_lm_head(snlp_model *m, const float *hL, int rows, float *logits, int32_t *argmax, void *stream) {
  TRY(check_model(m, "snlp_lm_head"));
  if (!hL || (!logits && !argmax)) return fail(SNLP_ERR_ARG, "snlp_lm_head: NULL pointer");
  if ((uintptr_t)hL % 16 || (uintptr_t)logits % 4 || (uintptr_t)argmax % 4) return fail(SNLP_ERR_ARG, "snlp_lm_head: hL must be 16-byte aligned, logits and argmax 4-byte aligned");
  if (rows < 1) return fail(SNLP_ERR_ARG, "snlp_lm_head: rows must be >= 1");
  if (rows > m->cfg.max_rows) return fail(SNLP_ERR_SHAPE, "snlp_lm_head: rows = %d exceeds max_rows = %d", rows, m->cfg.max_rows);
  return lm_head_impl(m, (cudaStream_t)stream, hL, (size_t)m->cfg.n_streams * m->cfg.d_model, rows, logits, argmax);
}

extern "C" int snlp_copy_trace(snlp_model *m, int rows, float *trace_out, void *stream) {
  TRY(check_model(m, "snlp_copy_trace"));
  if (!trace_out) return fail(SNLP_ERR_ARG, "snlp_copy_trace: NULL trace_out");
  if ((uintptr_t)trace_out % 16) return fail(SNLP_ERR_ARG, "snlp_copy_trace: trace_out must be 16-byte aligned");
  if (m->last_rows == 0) return fail(SNLP_ERR_STATE, "snlp_copy_trace: no forward, prefill or decode call has run on this handle yet");
  if (rows != m->last_rows) return fail(SNLP_ERR_SHAPE, "snlp_copy_trace: rows = %d but the last call ran %d rows", rows, m->last_rows);
  const size_t bytes = (size_t)(m->cfg.n_layer + 1) * rows * m->cfg.n_streams * m->cfg.d_model * sizeof(float);
  CU(cudaMemcpyAsync(trace_out, m->trace, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
  return SNLP_OK;
}

extern "C" int snlp_kv_create(snlp_model *m, int B, int max_ctx, snlp_kv **out) {
  if (!m || !out) return fail(SNLP_ERR_ARG, "snlp_kv_create: NULL argument");
  if (B < 1 || max_ctx < 1) return fail(SNLP_ERR_ARG, "snlp_kv_create: B and max_ctx must be >= 1");
  if (B > m->cfg.max_batch) return fail(SNLP_ERR_SHAPE, "snlp_kv_create: B = %d exceeds max_batch = %d", B, m->cfg.max_batch);
  if (max_ctx > m->cfg.max_ctx) return fail(SNLP_ERR_SHAPE, "snlp_kv_create: max_ctx = %d exceeds the model's %d", max_ctx, m->cfg.max_ctx);
  snlp_kv *kv = new (std::nothrow) snlp_kv;
  if (!kv) return fail(SNLP_ERR_OOM, "snlp_kv_create: host allocation failed");
  kv->m = m; kv->B = B; kv->max_ctx = max_ctx;
  const size_t bytes = (size_t)m->cfg.n_layer * B * max_ctx * m->cfg.d_model * m->esz;
  if (cudaMalloc(&kv->k, bytes) != cudaSuccess || cudaMalloc(&kv->v, bytes) != cudaSuccess || cudaMalloc(&kv->pos, 16) != cudaSuccess) {
    cudaGetLastError();
    cudaFree(kv->k); cudaFree(kv->v); cudaFree(kv->pos);
    delete kv;
    return fail(SNLP_ERR_OOM, "snlp_kv_create: cudaMalloc of 2 x %zu bytes failed", bytes);
  }
  if (cudaMemset(kv->k, 0, bytes) != cudaSuccess || cudaMemset(kv->v, 0, bytes) != cudaSuccess || cudaMemset(kv->pos, 0, 16) != cudaSuccess) {
    cudaFree(kv->k); cudaFree(kv->v); cudaFree(kv->pos);
    delete kv;
    return fail(SNLP_ERR_CUDA, "snlp_kv_create: cudaMemset failed");
  }
  m->caches.push_back(kv);
  *out = kv;
  return SNLP_OK;
}

extern "C" int snlp_kv_destroy(snlp_kv *kv) {
  if (!kv) return fail(SNLP_ERR_ARG, "snlp_kv_destroy: NULL handle");
  cudaDeviceSynchronize();
  if (kv->m) {  // the model is still alive: drop the graphs captured against this cache (they hold its pointers)
    for (auto it = kv->m->graphs.begin(); it != kv->m->graphs.end();) {
      if (it->first.kv == kv) { cudaGraphExecDestroy(it->second.exec); it = kv->m->graphs.erase(it); }
      else ++it;
    }
    kv->m->caches.erase(std::remove(kv->m->caches.begin(), kv->m->caches.end(), kv), kv->m->caches.end());
  }
  cudaFree(kv->k); cudaFree(kv->v); cudaFree(kv->pos);
  delete kv;
  return SNLP_OK;
}

// Make the host's mirror of the cache length exact again (it is only an upper bound after an asynchronous
// draft-and-verify round): wait for the device and read the length it holds.
static int kv_resolve(snlp_kv *kv) {
  if (kv->len_known) return SNLP_OK;
  CU(cudaDeviceSynchronize());
  int len = 0;
  CU(cudaMemcpy(&len, kv->pos, sizeof len, cudaMemcpyDeviceToHost));
  kv->len = kv->len_hi = len;
  kv->len_known = true;
  return SNLP_OK;
}

// Room for `need` more positions?  Decided on the host's upper bound; when that bound is not exact and says no,
// the exact length is fetched first.
static int kv_room(snlp_kv *kv, int need, const char *who) {
  if (kv->len_hi + need > kv->max_ctx && !kv->len_known) TRY(kv_resolve(kv));
  if (kv->len_hi + need > kv->max_ctx)
    return fail(SNLP_ERR_SHAPE, "%s: cache length %d + %d exceeds max_ctx %d", who, kv->len_hi, need, kv->max_ctx);
  return SNLP_OK;
}

static void kv_advance(snlp_kv *kv, int n) {
  kv->len_hi += n;
  if (kv->len_known) kv->len = kv->len_hi;
}

extern "C" int snlp_kv_len(snlp_kv *kv, int32_t *len) {
  if (!kv || !len) return fail(SNLP_ERR_ARG, "snlp_kv_len: NULL argument");
  TRY(kv_resolve(kv));
  *len = kv->len;
  return SNLP_OK;
}

extern "C" int snlp_kv_truncate(snlp_kv *kv, int new_len, void *stream) {
  if (!kv) return fail(SNLP_ERR_ARG, "snlp_kv_truncate: NULL handle");
  if (!kv->m) return fail(SNLP_ERR_STATE, "snlp_kv_truncate: the model of this cache has been destroyed");
  TRY(kv_resolve(kv));
  if (new_len < 0 || new_len > kv->len) return fail(SNLP_ERR_ARG, "snlp_kv_truncate: new_len = %d outside 0..%d", new_len, kv->len);
  KLAUNCH(kv->m, (cudaStream_t)stream, KC_OTHER, k_set_int<<<1, 1, 0, (cudaStream_t)stream>>>(kv->pos, new_len));
  kv->len = kv->len_hi = new_len;
  return SNLP_OK;
}

// Geometry of a forward over T new positions per sequence against the cache.  pos_hi (which only sizes the split-KV
// grid of the decode-regime attention) is the host's upper bound of the length: chunks that lie wholly beyond the
// true length contribute exact zeros to the merge, so an overestimate changes no output bit.
static Fwd kv_fwd(snlp_model *m, snlp_kv *kv, int T, cudaStream_t st) {
  Fwd f{};
  f.M = kv->B * T; f.B = kv->B; f.T = T;
  f.kc = kv->k; f.vc = kv->v;
  f.kv_bs = (size_t)kv->max_ctx * m->cfg.d_model;
  f.kv_ls = (size_t)kv->B * f.kv_bs;
  f.kv_rows = kv->max_ctx;
  f.pos = kv->pos; f.pos_hi = kv->len_hi; f.st = st;
  return f;
}

__global__ void k_gather_ids(const int32_t *__restrict__ ids, int32_t *__restrict__ out, int B, int Tc, int T, int t0) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < B * Tc) out[i] = ids[(size_t)(i / Tc) * T + t0 + (i % Tc)];
}

extern "C" int snlp_prefill(snlp_model *m, snlp_kv *kv, const int32_t *ids, int B, int T, int32_t *last_argmax, void *stream) {
  TRY(check_model(m, "snlp_prefill"));
  if (!kv || !ids) return fail(SNLP_ERR_ARG, "snlp_prefill: NULL pointer");
  if (kv->m != m) return fail(SNLP_ERR_ARG, "snlp_prefill: cache belongs to another model");
  if (B < 1 || T < 1) return fail(SNLP_ERR_ARG, "snlp_prefill: B and T must be >= 1");
  if (B != kv->B) return fail(SNLP_ERR_SHAPE, "snlp_prefill: B = %d but the cache holds %d sequences", B, kv->B);
  TRY(kv_room(kv, T, "snlp_prefill"));
  cudaStream_t st = (cudaStream_t)stream;
  const snlp_config &c = m->cfg;
  const int tc_max = c.max_rows / B;
  if (tc_max < 1) return fail(SNLP_ERR_SHAPE, "snlp_prefill: B exceeds max_rows");
  const size_t nd = (size_t)c.n_streams * c.d_model;
  int Tc = 0;
  for (int t0 = 0; t0 < T; t0 += Tc) {
    Tc = T - t0 < tc_max ? T - t0 : tc_max;
    KLAUNCH(m, st, KC_OTHER, k_gather_ids<<<(B * Tc + 255) / 256, 256, 0, st>>>(ids, m->spec, B, Tc, T, t0));
    TRY(embed_impl(m, st, m->spec, B * Tc, m->trace));
    Fwd f = kv_fwd(m, kv, Tc, st);
    TRY(sequential(m, f));
    KLAUNCH(m, st, KC_OTHER, k_add_int<<<1, 1, 0, st>>>(kv->pos, Tc));
    kv_advance(kv, Tc);
    m->last_rows = B * Tc;
  }
  if (last_argmax) {
    const float *hL = m->trace + (size_t)c.n_layer * B * Tc * nd + (size_t)(Tc - 1) * nd;
    TRY(lm_head_impl(m, st, hL, (size_t)Tc * nd, B, nullptr, last_argmax));
  }
  return SNLP_OK;
}

// greedy tokens of all `rows` rows of the forward that just ran (rows <= 16)
// bump (nullable): device counter to advance by one after the tokens are out (done by the LM-head kernel itself on the tensor-core path)
static int lm_head_tail(snlp_model *m, cudaStream_t st, int rows, int32_t *argmax, int *bump = nullptr, int32_t *const *argmax_pp = nullptr) {
  const snlp_config &c = m->cfg;
  const size_t nd = (size_t)c.n_streams * c.d_model, L = c.n_layer;
  if (umma_path_ok(m) && rows <= kDecodeRows)  // the correction left the LM-head input in slot L of xb / ssq_x
    return lm_head_impl(m, st, nullptr, 0, rows, nullptr, argmax, (const __nv_bfloat16 *)m->xn + L * rows * c.d_model,
                        m->ssq_x + L * (c.d_model / 128) * rows, bump, argmax_pp);
  TRY(lm_head_impl(m, st, m->trace + L * rows * nd, nd, rows, nullptr, argmax, nullptr, nullptr, nullptr, argmax_pp));
  if (bump) KLAUNCH(m, st, KC_OTHER, k_add_int<<<1, 1, 0, st>>>(bump, 1));
  return SNLP_OK;
}

// Enqueue one decode step (no graph handling, no host-side length update).  The step reads its input tokens and
// writes its output tokens through the handle's device slot, so the launches -- and a graph captured from them --
// do not depend on where the caller keeps its tokens.
static int decode_launches(snlp_model *m, snlp_kv *kv, const snlp_solver &sol, float *resnorm_out, cudaStream_t st) {
  Fwd f = kv_fwd(m, kv, 1, st);
  f.embed_ids_pp = (const int32_t *const *)m->tok_slot;
  TRY(solve(m, f, sol, resnorm_out));
  TRY(lm_head_tail(m, st, kv->B, nullptr, kv->pos, (int32_t *const *)(m->tok_slot + 1)));   // also advances the cache position
  return SNLP_OK;
}

static int decode_step_impl(snlp_model *m, snlp_kv *kv, const int32_t *tok_in, const snlp_solver &sol, int32_t *tok_out, float *resnorm_out,
                            cudaStream_t st) {
  if (m->slot_in != tok_in || m->slot_out != tok_out) {   // point the slot at this call's buffers (stream-ordered)
    KLAUNCH(m, st, KC_OTHER, k_set_ptrs<<<1, 1, 0, st>>>(m->tok_slot, tok_in, tok_out));
    m->slot_in = tok_in;
    m->slot_out = tok_out;
  }
  m->last_rows = kv->B;
  if (!m->use_graphs || m->timing) {
    TRY(decode_launches(m, kv, sol, resnorm_out, st));
    kv_advance(kv, 1);
    return SNLP_OK;
  }
  const bool fast = fast_decode_ok(m, kv->B);
  const int chunk_len = attn_csub(kv->B * m->cfg.n_head) * kAttnSub;
  GraphKey key{kv->B, sol.K, sol.mode, sol.prefix, sol.init, sol.fuse, fast ? kv->len_hi / chunk_len + 1 : 0, resnorm_out, kv};
  auto it = m->graphs.find(key);
  if (it == m->graphs.end()) {
    if (m->graphs.size() >= 256) {
      for (auto &g : m->graphs) cudaGraphExecDestroy(g.second.exec);
      m->graphs.clear();
    }
    cudaGraph_t graph = nullptr;
    CU(cudaStreamBeginCapture(m->cap_stream, cudaStreamCaptureModeThreadLocal));
    m->capturing = true;
    m->cap_nodes = 0;
    const int rc = decode_launches(m, kv, sol, resnorm_out, m->cap_stream);
    m->capturing = false;
    cudaError_t e = cudaStreamEndCapture(m->cap_stream, &graph);
    if (rc != SNLP_OK) {
      if (graph) cudaGraphDestroy(graph);
      return rc;
    }
    if (e != cudaSuccess) return fail(SNLP_ERR_CUDA, "cudaStreamEndCapture failed: %s", cudaGetErrorString(e));
    GraphEntry ge{};
    ge.nodes = m->cap_nodes;
    e = cudaGraphInstantiate(&ge.exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) return fail(SNLP_ERR_CUDA, "cudaGraphInstantiate failed: %s", cudaGetErrorString(e));
    it = m->graphs.emplace(key, ge).first;
    m->graph_captures += 1;
  }
  CU(cudaGraphLaunch(it->second.exec, st));
  m->launches += it->second.nodes;
  kv_advance(kv, 1);
  return SNLP_OK;
}

static int check_token_ptrs(const int32_t *tok_in, const int32_t *tok_out, const char *who) {
  if (!tok_in || !tok_out) return fail(SNLP_ERR_ARG, "%s: NULL pointer", who);
  if ((uintptr_t)tok_in % 4 || (uintptr_t)tok_out % 4) return fail(SNLP_ERR_ARG, "%s: token pointers must be 4-byte aligned", who);
  return SNLP_OK;
}

extern "C" int snlp_decode_step(snlp_model *m, snlp_kv *kv, const int32_t *tok_in, int K, int mode, int32_t *tok_out, float *resnorm_out,
                                void *stream) {
  TRY(check_model(m, "snlp_decode_step"));
  if (!kv) return fail(SNLP_ERR_ARG, "snlp_decode_step: NULL pointer");
  TRY(check_token_ptrs(tok_in, tok_out, "snlp_decode_step"));
  if (kv->m != m) return fail(SNLP_ERR_ARG, "snlp_decode_step: cache belongs to another model");
  if (K < 0) return fail(SNLP_ERR_ARG, "snlp_decode_step: K must be >= 0 (got %d)", K);
  TRY(check_mode(mode, "snlp_decode_step"));
  TRY(kv_room(kv, 1, "snlp_decode_step"));
  const snlp_solver sol = K == 0 ? snlp_solver{0, SNLP_MODE_SEQUENTIAL, m->cfg.n_layer, SNLP_INIT_H0, 1} : snlp_solver{K, mode, 0, SNLP_INIT_H0, 1};
  return decode_step_impl(m, kv, tok_in, sol, tok_out, K > 0 ? resnorm_out : nullptr, (cudaStream_t)stream);
}

extern "C" int snlp_decode_step_host(snlp_model *m, snlp_kv *kv, const int32_t *tok_in_host, int K, int mode, int32_t *tok_out_host, void *stream) {
  TRY(check_model(m, "snlp_decode_step_host"));
  if (!kv || !tok_in_host || !tok_out_host) return fail(SNLP_ERR_ARG, "snlp_decode_step_host: NULL pointer");
  if (kv->m != m) return fail(SNLP_ERR_ARG, "snlp_decode_step_host: cache belongs to another model");
  // The step's kernels read the tokens from, and write the next ones to, mapped pinned host memory: the embedding
  // gather fetches B ids across the bus and the LM-head kernel posts B ids back, with no copy operations around the graph.
  const size_t bytes = (size_t)kv->B * sizeof(int32_t);
  memcpy(m->tok_pin, tok_in_host, bytes);
  // The host does not go through the stream's completion machinery (tens of microseconds of wake-up latency) to learn
  // that the step is done: it marks the output slots with a value no token can take and watches them until the step's
  // last kernel has stored every token (the stores travel straight over the bus).  If they do not arrive within a
  // generous limit -- an error in the step, a device that is busy with other work -- it falls back to synchronising.
  volatile int32_t *out = m->tok_pin + m->cfg.max_batch;
  constexpr int32_t kNoToken = INT32_MIN;
  for (int i = 0; i < kv->B; ++i) out[i] = kNoToken;
  TRY(snlp_decode_step(m, kv, m->tok_dev, K, mode, m->tok_dev + m->cfg.max_batch, nullptr, stream));
  bool seen = false;
  const auto t0 = std::chrono::steady_clock::now();
  for (uint32_t it = 0; !seen; ++it) {
    seen = true;
    for (int i = 0; i < kv->B; ++i) seen = seen && out[i] != kNoToken;
    if (seen) break;
    __builtin_ia32_pause();
    if ((it & 1023u) == 1023u && std::chrono::steady_clock::now() - t0 > std::chrono::milliseconds(50)) break;
  }
  if (!seen) CU(cudaStreamSynchronize((cudaStream_t)stream));
  std::atomic_thread_fence(std::memory_order_acquire);
  memcpy(tok_out_host, m->tok_pin + m->cfg.max_batch, bytes);
  return SNLP_OK;
}

extern "C" int snlp_decode_step_solver(snlp_model *m, snlp_kv *kv, const int32_t *tok_in, const snlp_solver *solver, int32_t *tok_out,
                                       float *resnorm_out, void *stream) {
  TRY(check_model(m, "snlp_decode_step_solver"));
  if (!kv || !solver) return fail(SNLP_ERR_ARG, "snlp_decode_step_solver: NULL pointer");
  TRY(check_token_ptrs(tok_in, tok_out, "snlp_decode_step_solver"));
  if (kv->m != m) return fail(SNLP_ERR_ARG, "snlp_decode_step_solver: cache belongs to another model");
  TRY(check_solver(m, *solver, "snlp_decode_step_solver"));
  TRY(kv_room(kv, 1, "snlp_decode_step_solver"));
  return decode_step_impl(m, kv, tok_in, *solver, tok_out, solver->K > 0 ? resnorm_out : nullptr, (cudaStream_t)stream);
}

// One draft-and-verify round, everything enqueued on the stream; the round's first position and the number of accepted
// drafts stay on the device.  On return the host knows the cache length only up to len_hi (every draft accepted).
static int draft_and_verify_launches(snlp_model *m, snlp_kv *kv, int32_t *last_tok, int block, int K, int mode, int32_t *emitted,
                                     int32_t *n_emitted, int32_t *n_accepted, cudaStream_t st, const char *who) {
  TRY(check_model(m, who));
  if (!kv || !last_tok || !emitted || !n_emitted || !n_accepted) return fail(SNLP_ERR_ARG, "%s: NULL pointer", who);
  if ((uintptr_t)last_tok % 4 || (uintptr_t)emitted % 4 || (uintptr_t)n_emitted % 4 || (uintptr_t)n_accepted % 4)
    return fail(SNLP_ERR_ARG, "%s: int32 pointers must be 4-byte aligned", who);
  if (kv->m != m) return fail(SNLP_ERR_ARG, "%s: cache belongs to another model", who);
  if (block < 1) return fail(SNLP_ERR_ARG, "%s: block must be >= 1", who);
  if (K < 1) return fail(SNLP_ERR_ARG, "%s: K must be >= 1", who);
  TRY(check_mode(mode, who));
  if (kv->B != 1) return fail(SNLP_ERR_SHAPE, "%s: batch must be 1 (cache holds %d)", who, kv->B);
  if (block + 1 > m->cfg.max_rows) return fail(SNLP_ERR_SHAPE, "%s: block+1 exceeds max_rows", who);
  TRY(kv_room(kv, block + 1, who));
  const snlp_config &c = m->cfg;
  const int hi0 = kv->len_hi;
  int32_t *ids = m->spec;                          // [block+1]: last_tok, x_1..x_block
  int32_t *y = m->spec + (c.max_rows + 1);         // [block+1]: verifier tokens
  CU(cudaMemcpyAsync(ids, last_tok, 4, cudaMemcpyDeviceToDevice, st));
  KLAUNCH(m, st, KC_OTHER, k_copy_int<<<1, 1, 0, st>>>(kv->pos + 1, kv->pos));   // remember where the round began
  const snlp_solver draft{K, mode, 0, SNLP_INIT_H0, 1};
  for (int i = 0; i < block; ++i) TRY(decode_step_impl(m, kv, ids + i, draft, ids + i + 1, nullptr, st));
  KLAUNCH(m, st, KC_OTHER, k_copy_int<<<1, 1, 0, st>>>(kv->pos, kv->pos + 1));   // back to the round's first position
  kv->len_hi = hi0;
  if (kv->len_known) kv->len = hi0;
  TRY(embed_impl(m, st, ids, block + 1, m->trace));
  Fwd f = kv_fwd(m, kv, block + 1, st);
  f.pos_hi = hi0;
  TRY(sequential(m, f));
  m->last_rows = block + 1;
  TRY(lm_head_tail(m, st, block + 1, y));
  KLAUNCH(m, st, KC_OTHER, k_accept<<<1, 32, 0, st>>>(ids + 1, y, block, emitted, n_emitted, n_accepted, last_tok, kv->pos, kv->pos + 1));
  kv->len_hi = hi0 + block + 1;   // the most the round can have kept
  kv->len_known = false;
  return SNLP_OK;
}

extern "C" int snlp_draft_and_verify_async(snlp_model *m, snlp_kv *kv, int32_t *last_tok, int block, int K, int mode, int32_t *emitted,
                                           int32_t *n_emitted, int32_t *n_accepted, void *stream) {
  return draft_and_verify_launches(m, kv, last_tok, block, K, mode, emitted, n_emitted, n_accepted, (cudaStream_t)stream,
                                   "snlp_draft_and_verify_async");
}

extern "C" int snlp_draft_and_verify(snlp_model *m, snlp_kv *kv, int32_t *last_tok, int block, int K, int mode, int32_t *emitted,
                                     int32_t *n_emitted, int32_t *n_accepted, void *stream) {
  TRY(draft_and_verify_launches(m, kv, last_tok, block, K, mode, emitted, n_emitted, n_accepted, (cudaStream_t)stream, "snlp_draft_and_verify"));
  int len = 0;   // the convenience form: wait for the round and bring the cache length back to the host
  CU(cudaMemcpyAsync(&len, kv->pos, sizeof len, cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  CU(cudaStreamSynchronize((cudaStream_t)stream));
  kv->len = kv->len_hi = len;
  kv->len_known = true;
  return SNLP_OK;
}

extern "C" int snlp_graph_count(const snlp_model *m, int64_t *captured) {
  if (!m || !captured) return fail(SNLP_ERR_ARG, "snlp_graph_count: NULL argument");
  *captured = m->graph_captures;
  return SNLP_OK;
}
