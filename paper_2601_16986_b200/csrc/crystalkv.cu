// C ABI of the Crystal-KV decode hot path (see include/crystalkv.h).  Host code only
// validates, keeps the per-layer clocks and launches; every step of the path runs in the
// kernels of attn_kernel.cuh, lrfu_kernel.cuh and aux_kernels.cuh.
//
// Stream plan of a tracked decode step of layer l: the attention kernel runs on the caller's
// stream (so `out` is ready in stream order), the LRFU kernel of the same layer on an
// internal stream behind an event, which lets it overlap the attention kernel of the next
// layer.  Before an attention kernel reuses a scratch set, or touches a layer whose LRFU
// kernel of the previous step may still run, the caller's stream waits on that kernel's
// event.  Everything else (prefill, reallocation, inspection) first joins the internal stream.
#include "../../include/crystalkv.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "attn_kernel.cuh"
#include "aux_kernels.cuh"
#include "lrfu_kernel.cuh"
#include "plan.cuh"

using namespace ckv;

struct crystalkv {
  crystalkv_config_t cfg;
  int G = 0, U = 0, units = 0, cap = 0, num_sms = 0, grid = 0;
  size_t smem = 0;
  long long pages_per_seq = 0;
  State st{};
  std::vector<Plan> plans;         // per layer: the launch plan of its next attention kernel
  Plan* d_plans = nullptr;
  int* done_ctr = nullptr;
  // scratch: logits and merged (m, l) per cycled set (the LRFU kernel reads them while later
  // attention kernels run), partials and tickets alternate between two (attention kernels do
  // not overlap one another's compute), pbar is only touched by kernels that run one at a time
  float* sc_logits[NSETS] = {};
  float* sc_mfin[NSETS] = {};
  float* sc_partials[2] = {};
  int* sc_ticket[2] = {};
  float* sc_pbar[2] = {};          // one per internal stream
  int* piece_ctr = nullptr;
  int cap_s = 0, pmax = 0;
  long long nA = 0;                // attention launches so far
  std::vector<int> t_layer;        // per layer: time of the last step
  // LRFU launches are numbered; launch k uses scratch set k % NSETS and event k % EV_RING
  static constexpr int EV_RING = 32;
  // two internal streams taken in turn: the LRFU kernels of consecutive layers do not depend on
  // one another, so the second may fill SM room as the first one's CTAs finish
  cudaStream_t side[2] = {};
  cudaEvent_t evA[EV_RING] = {}, evF[EV_RING] = {};
  long long kF = 0, joined = -1;
  std::vector<long long> lastF;    // per layer: number of its latest LRFU launch, -1 = none
  int prev_layer = -1;             // layer of the launch pair issued last, -1 after any other call
  int stage = CRYSTALKV_STAGE_THINK;
  int answer_steps = 0;
  long long* Asum = nullptr;
  // host I/O: HOST_RING staging sets; inputs go up on one internal stream and results come
  // down on another, so the copies of other layers run beside the attention kernels
  static constexpr int HOST_RING = 64;
  __nv_bfloat16 *dq[HOST_RING] = {}, *dk[HOST_RING] = {}, *dv[HOST_RING] = {}, *dout[HOST_RING] = {};
  cudaStream_t copy_in = nullptr, copy_out = nullptr;
  cudaEvent_t evIn[HOST_RING] = {}, evUse[HOST_RING] = {}, evOut[HOST_RING] = {};
  long long outJoined = -1;   // newest host step whose copy back the caller's stream has waited for
  long long nHost = 0;             // host-buffer steps so far
  __nv_bfloat16* dummy_out = nullptr;
  int* io_rec = nullptr;           // staging for export / import of one head: records, rows, count
  unsigned char* io_rows = nullptr;
  int* io_n = nullptr;
  float* tab = nullptr;
  std::vector<void*> allocs;
  std::string err;
  bool cuda_dead = false;
};

namespace {

thread_local std::string g_create_err;
constexpr int MAX_DEVICES = 64;   // device ordinals this library keeps per-device state for

int fail(crystalkv_t* h, int code, const std::string& msg) {
  if (h) h->err = msg;
  return code;
}

// An error that only says "not while this stream is being captured" leaves the context and the
// handle intact; every other CUDA error is sticky for the handle.
bool capture_refusal(cudaError_t e) {
  return e >= cudaErrorStreamCaptureUnsupported && e <= cudaErrorStreamCaptureWrongThread;
}

#define CK(h, call)                                                                      \
  do {                                                                                   \
    cudaError_t e_ = (call);                                                             \
    if (e_ != cudaSuccess) {                                                             \
      if ((h) && !capture_refusal(e_)) (h)->cuda_dead = true;                            \
      return fail((h), CRYSTALKV_ECUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); \
    }                                                                                    \
  } while (0)

// Makes the handle's device current for the duration of a call and puts the caller's back.
struct DeviceScope {
  int prev = -1;
  cudaError_t err = cudaSuccess;
  explicit DeviceScope(int dev) {
    int cur = -1;
    err = cudaGetDevice(&cur);
    if (err == cudaSuccess && cur != dev) {
      err = cudaSetDevice(dev);
      if (err == cudaSuccess) prev = cur;
    }
  }
  ~DeviceScope() {
    if (prev >= 0) cudaSetDevice(prev);
  }
  DeviceScope(const DeviceScope&) = delete;
  DeviceScope& operator=(const DeviceScope&) = delete;
};
#define ON_DEVICE(h)                       \
  DeviceScope dev_scope_((h)->cfg.device); \
  CK((h), dev_scope_.err)

template <typename T>
int dalloc(crystalkv_t* h, T** p, size_t count) {
  void* q = nullptr;
  cudaError_t e = cudaMalloc(&q, std::max<size_t>(count, 1) * sizeof(T));
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(h, e == cudaErrorMemoryAllocation ? CRYSTALKV_ENOMEM : CRYSTALKV_ECUDA,
                std::string("cudaMalloc: ") + cudaGetErrorString(e));
  }
  h->allocs.push_back(q);
  *p = static_cast<T*>(q);
  return CRYSTALKV_OK;
}

__global__ void init_free_stack_kernel(int* stack, int* top, long long pages_per_seq, int batch) {
  const long long total = pages_per_seq * batch;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const long long r = i % pages_per_seq;
    stack[i] = (int)(pages_per_seq - 1 - r);   // popping from the top hands out ascending page ids
  }
  if (blockIdx.x == 0)
    for (int b = threadIdx.x; b < batch; b += blockDim.x) top[b] = (int)pages_per_seq;
}

__global__ void fill_int_kernel(int* p, long long n, int v) {
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
    p[i] = v;
}

template <int G>
cudaError_t launch_lrfu(const DecodeParams& p, int grid, cudaStream_t s) {
  // the same shared-memory carve-out as the attention kernel, so that CTAs of both can be
  // resident on one SM at the same time
  // (function attributes are kept per device)
  static std::atomic<bool> prepared[MAX_DEVICES] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
  if (!prepared[dev].load(std::memory_order_acquire)) {
    e = cudaFuncSetAttribute(lrfu_kernel<G>, cudaFuncAttributePreferredSharedMemoryCarveout,
                             (int)cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    prepared[dev].store(true, std::memory_order_release);
  }
  lrfu_kernel<G><<<grid, NT, 0, s>>>(p);
  return cudaGetLastError();
}

cudaError_t lrfu_dispatch(int G, const DecodeParams& p, int grid, cudaStream_t s) {
  switch (G) {
    case 1: return launch_lrfu<1>(p, grid, s);
    case 2: return launch_lrfu<2>(p, grid, s);
    case 3: return launch_lrfu<3>(p, grid, s);
    case 4: return launch_lrfu<4>(p, grid, s);
    case 5: return launch_lrfu<5>(p, grid, s);
    case 6: return launch_lrfu<6>(p, grid, s);
    case 7: return launch_lrfu<7>(p, grid, s);
    case 8: return launch_lrfu<8>(p, grid, s);
  }
  return cudaErrorInvalidValue;
}

int validate(const crystalkv_config_t* c, std::string& why) {
  if (!c) { why = "cfg is NULL"; return CRYSTALKV_EINVAL; }
  if (c->head_dim != HD) { why = "head_dim must be 128"; return CRYSTALKV_EINVAL; }
  if (c->dtype != CRYSTALKV_BF16) { why = "dtype must be CRYSTALKV_BF16"; return CRYSTALKV_EINVAL; }
  if (c->n_layers < 1 || c->n_kv_heads < 1 || c->batch < 1) { why = "n_layers, n_kv_heads, batch must be >= 1"; return CRYSTALKV_EINVAL; }
  if (c->n_q_heads < c->n_kv_heads || c->n_q_heads % c->n_kv_heads) { why = "n_q_heads must be a multiple of n_kv_heads"; return CRYSTALKV_EINVAL; }
  if (c->n_q_heads / c->n_kv_heads > 8) { why = "group size above 8"; return CRYSTALKV_EINVAL; }
  if ((long long)c->batch * c->n_kv_heads > MAX_UNITS_PER_CALL) { why = "batch * n_kv_heads above 2048"; return CRYSTALKV_EINVAL; }
  if (c->mode != CRYSTALKV_MODE_EVICT && c->mode != CRYSTALKV_MODE_FULLKV) { why = "bad mode"; return CRYSTALKV_EINVAL; }
  if (c->max_context < 2) { why = "max_context must be >= 2"; return CRYSTALKV_EINVAL; }
  if (c->mode == CRYSTALKV_MODE_EVICT && c->budget_per_head < 1) { why = "budget_per_head must be >= 1"; return CRYSTALKV_EINVAL; }
  if (c->min_budget < 0 || c->max_budget < 0 || c->max_answer_tokens < 0) { why = "negative budget bound"; return CRYSTALKV_EINVAL; }
  if (c->max_budget && c->max_budget < c->budget_per_head) { why = "max_budget below budget_per_head"; return CRYSTALKV_EINVAL; }
  if (c->min_budget > c->budget_per_head) { why = "min_budget above budget_per_head"; return CRYSTALKV_EINVAL; }
  if (c->top_p < 0.f || c->top_p > 1.f) { why = "top_p outside (0, 1]"; return CRYSTALKV_EINVAL; }
  if (c->lambda > 1.f) { why = "lambda above 1"; return CRYSTALKV_EINVAL; }
  if (c->sm_scale < 0.f) { why = "negative sm_scale"; return CRYSTALKV_EINVAL; }
  if (c->device < 0 || c->device >= MAX_DEVICES) { why = "device ordinal outside [0, 64)"; return CRYSTALKV_EINVAL; }
  if (c->evict_every < 0 || c->evict_every > 4096) { why = "evict_every outside [0, 4096]"; return CRYSTALKV_EINVAL; }
  if (c->literal_return != 0 && c->literal_return != 1) { why = "literal_return must be 0 or 1"; return CRYSTALKV_EINVAL; }
  if (!(c->budget_ratio >= 0.f) || c->budget_ratio > 1.f) { why = "budget_ratio outside [0, 1]"; return CRYSTALKV_EINVAL; }
  return CRYSTALKV_OK;
}

// Ratio budgets: the average budget per head after `tokens` tokens, floor(r * tokens) in fp64 from
// the fp32 ratio, kept within [max(1, min_budget), budget_per_head].
int ratio_budget(const crystalkv_config_t& c, int tokens) {
  long long b = (long long)std::floor((double)c.budget_ratio * (double)tokens);
  b = std::max<long long>(b, std::max(1, c.min_budget));
  b = std::min<long long>(b, c.budget_per_head);
  return (int)b;
}

// Sets the budget of every head of one layer.
__global__ void fill_layer_budget_kernel(State st, int layer, int v) {
  const int u = blockIdx.x * blockDim.x + threadIdx.x;
  if (u < st.batch * st.H) st.budget[((u / st.H) * st.L + layer) * st.H + (u % st.H)] = v;
}

int check_layer(crystalkv_t* h, int layer) {
  if (!h) return CRYSTALKV_EINVAL;
  if (h->cuda_dead) return fail(h, CRYSTALKV_ECUDA, "an earlier CUDA error is sticky for this handle");
  if (layer < 0 || layer >= h->cfg.n_layers) return fail(h, CRYSTALKV_EINVAL, "layer out of range");
  return CRYSTALKV_OK;
}

int check_unit(crystalkv_t* h, int layer, int seq, int head) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  if (seq < 0 || seq >= h->cfg.batch || head < 0 || head >= h->cfg.n_kv_heads)
    return fail(h, CRYSTALKV_EINVAL, "seq or kv_head out of range");
  return CRYSTALKV_OK;
}

DecodeParams make_params(crystalkv_t* h, int layer) {
  DecodeParams p{};
  p.st = h->st;
  p.plan = h->plans[layer];
  p.done_ctr = h->done_ctr;   // (launch_step picks the internal stream's own)
  p.sc.cap_s = h->cap_s;
  p.sc.pmax = h->pmax;
  p.sc.pbar = h->sc_pbar[0];
  p.sc.partials = h->sc_partials[h->nA & 1];
  p.sc.ticket = h->sc_ticket[h->nA & 1];
  p.sc.logits = h->sc_logits[0];
  p.sc.mfin = h->sc_mfin[0];
  h->nA++;
  p.layer = layer;
  p.G = h->G;
  p.scale = h->cfg.sm_scale;
  p.scale_log2 = h->cfg.sm_scale * 1.44269504088896340736f;
  p.top_p = h->cfg.top_p;
  p.evict_every = h->cfg.evict_every;
  p.literal = h->cfg.literal_return;
  p.plan_append = -1;
  p.plan_warps = h->grid * NW;
  p.plan_grid = h->grid;
  return p;
}

// Writes the launch plans of `count` layers from their heads' current lengths, on `s`.
int replan(crystalkv_t* h, int layer0, int count, int append, int n_limit, cudaStream_t s) {
  plan_kernel<<<count, NT, 0, s>>>(h->st, h->d_plans, layer0, append, n_limit, h->grid * NW, h->grid);
  CK(h, cudaGetLastError());
  return CRYSTALKV_OK;
}

// Makes `s` wait for every LRFU kernel launched so far.
int join_side(crystalkv_t* h, cudaStream_t s) {
  h->prev_layer = -1;
  if (h->kF > 0) CK(h, cudaStreamWaitEvent(s, h->evF[(h->kF - 1) % crystalkv::EV_RING], 0));
  if (h->kF > 1) CK(h, cudaStreamWaitEvent(s, h->evF[(h->kF - 2) % crystalkv::EV_RING], 0));   // the other internal stream
  h->joined = h->kF - 1;
  if (h->nHost > 0) CK(h, cudaStreamWaitEvent(s, h->evOut[(h->nHost - 1) % crystalkv::HOST_RING], 0));   // copies back run in order
  return CRYSTALKV_OK;
}

// One attention launch on `s` and its follow-up (Algorithm 1 when it runs, the heads' new lengths
// and the layer's next plan) on the internal stream.
// chain: this launch scores the same, unchanged lists as the layer's previous launch (a window of
// prompt queries): its attention kernel need not wait for that launch's LRFU kernel, only its own
// LRFU kernel must run behind it.
int launch_step(crystalkv_t* h, DecodeParams& p, int layer, cudaStream_t s, bool chain = false) {
  const bool track = true;   // every launch has a follow-up that uses a scratch set
  const long long k = h->kF;
  if (track) {
    // launch k reuses the scratch of launch k - NSETS and continues the state its layer's
    // previous LRFU launch wrote; each internal stream runs in order, so the events of two
    // consecutive launches cover everything before them
    // A wait on the caller's stream costs several microseconds (the attention kernel behind it
    // no longer starts early), so one wait covers as many launches as the sets allow: it targets
    // the newest LRFU launch that has had two attention kernels' time to finish.
    const long long need = chain ? k - NSETS : std::max(k - NSETS, h->lastF[layer]);
    if (need >= 0 && need > h->joined) {
      const long long target = std::max(need, k - 3);
      CK(h, cudaStreamWaitEvent(s, h->evF[target % crystalkv::EV_RING], 0));
      if (target > 0) CK(h, cudaStreamWaitEvent(s, h->evF[(target - 1) % crystalkv::EV_RING], 0));   // the other internal stream
      h->joined = target;
    }
    p.sc.logits = h->sc_logits[k % NSETS];
    p.sc.mfin = h->sc_mfin[k % NSETS];
  }
  // The attention kernel may start while the kernel ahead of it still runs: it first fills its
  // pipeline from the cache and waits for that kernel before it touches the call's inputs.
  // That is only sound if the kernel ahead cannot be writing this layer's lists, which holds
  // when it is the attention kernel of another layer.
  p.early = (h->prev_layer >= 0 && h->prev_layer != layer) ? 1 : 0;
  {
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(h->grid);
    lc.blockDim = dim3(NT);
    lc.dynamicSmemBytes = h->smem;
    lc.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    CK(h, cudaLaunchKernelEx(&lc, attn_kernel, p));
  }
  h->prev_layer = layer;
  if (track) {
    const int si = (int)(k & 1);
    cudaEvent_t ea = h->evA[k % crystalkv::EV_RING];
    p.sc.pbar = h->sc_pbar[si];
    p.done_ctr = h->done_ctr + 2 * si;
    CK(h, cudaEventRecord(ea, s));
    CK(h, cudaStreamWaitEvent(h->side[si], ea, 0));
    if (chain && k > 0) CK(h, cudaStreamWaitEvent(h->side[si], h->evF[(k - 1) % crystalkv::EV_RING], 0));   // (the other internal stream)
    CK(h, lrfu_dispatch(h->G, p, h->U, h->side[si]));
    CK(h, cudaEventRecord(h->evF[k % crystalkv::EV_RING], h->side[si]));
    h->lastF[layer] = k;
    h->kF = k + 1;
  }
  return CRYSTALKV_OK;
}

}  // namespace

extern "C" {

const char* crystalkv_strerror(int code) {
  switch (code) {
    case CRYSTALKV_OK: return "ok";
    case CRYSTALKV_EINVAL: return "invalid argument";
    case CRYSTALKV_ESTATE: return "call out of order or capacity exhausted";
    case CRYSTALKV_ENOMEM: return "device allocation failed";
    case CRYSTALKV_ECUDA: return "CUDA runtime error";
    case CRYSTALKV_ECHECK: return "device-side consistency check failed";
  }
  return "unknown error";
}

const char* crystalkv_last_error(crystalkv_t* h) { return h ? h->err.c_str() : g_create_err.c_str(); }

int crystalkv_destroy(crystalkv_t* h) {
  if (!h) return CRYSTALKV_OK;
  DeviceScope scope(h->cfg.device);
  cudaDeviceSynchronize();
  for (cudaStream_t x : h->side)
    if (x) cudaStreamDestroy(x);
  if (h->copy_in) cudaStreamDestroy(h->copy_in);
  if (h->copy_out) cudaStreamDestroy(h->copy_out);
  for (int i = 0; i < crystalkv::HOST_RING; ++i) {
    if (h->evIn[i]) cudaEventDestroy(h->evIn[i]);
    if (h->evUse[i]) cudaEventDestroy(h->evUse[i]);
    if (h->evOut[i]) cudaEventDestroy(h->evOut[i]);
  }
  for (cudaEvent_t e : h->evA)
    if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : h->evF)
    if (e) cudaEventDestroy(e);
  for (void* p : h->allocs) cudaFree(p);
  delete h;
  return CRYSTALKV_OK;
}

int crystalkv_create(const crystalkv_config_t* cfg, crystalkv_t** out) {
  std::string why;
  int rc = validate(cfg, why);
  if (rc) { g_create_err = why; return rc; }
  if (!out) { g_create_err = "out is NULL"; return CRYSTALKV_EINVAL; }
  crystalkv_t* h = new (std::nothrow) crystalkv();
  if (!h) return CRYSTALKV_ENOMEM;
  h->cfg = *cfg;
  crystalkv_config_t& c = h->cfg;
  if (c.top_p == 0.f) c.top_p = 0.9f;
  if (c.lambda < 0.f) c.lambda = 0.6f;
  if (c.sm_scale == 0.f) c.sm_scale = (float)(1.0 / std::sqrt((double)c.head_dim));
  if (c.min_budget == 0) c.min_budget = std::min(c.budget_per_head, std::max(16, c.budget_per_head / 8));
  if (c.max_budget == 0) c.max_budget = 4 * c.budget_per_head;
  if (c.evict_every < 1) c.evict_every = 1;
  const bool evict = c.mode == CRYSTALKV_MODE_EVICT;
  h->G = c.n_q_heads / c.n_kv_heads;
  h->U = c.batch * c.n_kv_heads;
  h->units = h->U * c.n_layers;
  // list positions per head: entries up to the largest budget plus those that arrive before the
  // next eviction and the answer-stage tail, plus the place of the next arrival; FullKV keeps
  // every token.  Whole pages of 16.
  h->cap = evict ? c.max_budget + c.evict_every + c.max_answer_tokens + 1 : c.max_context + 1;
  h->cap = (h->cap + GRP - 1) / GRP * GRP;
  // pages per sequence: the entries all heads may hold together (B_total, what arrives before an
  // eviction, the answer tail, the hole), and one page per head for lists that end inside a page
  {
    const long long N = (long long)c.n_layers * c.n_kv_heads;
    const long long per_head = evict ? (long long)c.budget_per_head + c.evict_every + c.max_answer_tokens + 1
                                     : (long long)c.max_context + 1;
    h->pages_per_seq = (N * per_head + GRP - 1) / GRP + N;
  }
  if (h->pages_per_seq > 0x7fffffffLL) { g_create_err = "more than 2^31 pages per sequence"; delete h; return CRYSTALKV_EINVAL; }

#define CREATE_FAIL(code_)                    \
  do {                                        \
    int c_ = (code_);                         \
    g_create_err = h->err;                    \
    crystalkv_destroy(h);                     \
    return c_;                                \
  } while (0)
#define CKC(call)                                                              \
  do {                                                                         \
    cudaError_t e_ = (call);                                                   \
    if (e_ != cudaSuccess) {                                                   \
      h->err = std::string(#call) + ": " + cudaGetErrorString(e_);             \
      CREATE_FAIL(CRYSTALKV_ECUDA);                                            \
    }                                                                          \
  } while (0)
#define DA(ptr, count)                                   \
  do {                                                   \
    int r_ = dalloc(h, ptr, (size_t)(count));            \
    if (r_) CREATE_FAIL(r_);                             \
  } while (0)

  DeviceScope scope(c.device);
  CKC(scope.err);
  cudaDeviceProp prop;
  CKC(cudaGetDeviceProperties(&prop, c.device));
  h->num_sms = prop.multiProcessorCount;
  // ring stages, one mbarrier per stage, every warp's queue of fetched pieces: the same for every
  // handle (the attribute belongs to the function, so no handle may lower it under another)
  h->smem = RING_BYTES + NW * STAGES * 8 + NW * FIFO * sizeof(int);
  int bps = 0;
  CKC(cudaFuncSetAttribute(attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->smem));
  // The largest shared-memory carve-out, although the ring alone would fit a smaller one: the CTAs
  // of the LRFU kernel have to find room beside an attention CTA on the same SM.
  CKC(cudaFuncSetAttribute(attn_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared));
  CKC(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, attn_kernel, NT, h->smem));
  if (bps < 1) { h->err = "attention kernel does not fit on an SM"; CREATE_FAIL(CRYSTALKV_ECUDA); }
  h->grid = h->num_sms * bps;
  {
    // The LRFU kernels run at the highest stream priority: the attention kernel of the layer after
    // next is already queued when one of them becomes ready (it was released early and waits for
    // shared memory), and at equal priority its CTAs, which cannot be placed yet, are served first.
    int least = 0, greatest = 0;
    CKC(cudaDeviceGetStreamPriorityRange(&least, &greatest));
    for (cudaStream_t& x : h->side) CKC(cudaStreamCreateWithPriority(&x, cudaStreamNonBlocking, greatest));
  }
  CKC(cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking));
  CKC(cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking));
  for (int i = 0; i < crystalkv::HOST_RING; ++i) {
    CKC(cudaEventCreateWithFlags(&h->evIn[i], cudaEventDisableTiming));
    CKC(cudaEventCreateWithFlags(&h->evUse[i], cudaEventDisableTiming));
    CKC(cudaEventCreateWithFlags(&h->evOut[i], cudaEventDisableTiming));
  }
  for (cudaEvent_t& e : h->evA) CKC(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  for (cudaEvent_t& e : h->evF) CKC(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));

  State& st = h->st;
  st.batch = c.batch; st.L = c.n_layers; st.H = c.n_kv_heads; st.cap = h->cap; st.capg = h->cap / GRP;
  st.pages_per_seq = h->pages_per_seq;
  DA(&st.pool, (size_t)c.batch * h->pages_per_seq * PAGE_BYTES);
  DA(&st.free_stack, (size_t)c.batch * h->pages_per_seq);
  DA(&st.free_top, c.batch);
  DA(&st.ptab, (size_t)h->units * st.capg);
  DA(&st.meta_pos, (size_t)h->units * h->cap);
  DA(&st.meta_tau, (size_t)h->units * h->cap);
  DA(&st.meta_crf, (size_t)h->units * h->cap);
  DA(&st.n_cur, h->units);
  DA(&st.hole, h->units);
  DA(&st.npages, h->units);
  DA(&st.budget, h->units);
  // launch plans, one per layer: at most one piece per warp and one more per head
  {
    const int nWarps = h->grid * NW, pd_cap = nWarps + h->U;
    int4* desc = nullptr; int4* wr = nullptr; int *npc = nullptr, *gpl = nullptr, *hdr = nullptr;
    DA(&desc, (size_t)c.n_layers * pd_cap);
    DA(&wr, (size_t)c.n_layers * nWarps);
    DA(&npc, (size_t)c.n_layers * h->U);
    DA(&gpl, (size_t)c.n_layers * h->U);
    DA(&hdr, (size_t)c.n_layers * 4);
    CKC(cudaMemset(hdr, 0, (size_t)c.n_layers * 4 * sizeof(int)));
    h->plans.resize(c.n_layers);
    for (int l = 0; l < c.n_layers; ++l)
      h->plans[l] = Plan{desc + (size_t)l * pd_cap, wr + (size_t)l * nWarps, npc + (size_t)l * h->U, gpl + (size_t)l * h->U,
                         hdr + (size_t)l * 4};
    DA(&h->d_plans, c.n_layers);
    CKC(cudaMemcpy(h->d_plans, h->plans.data(), (size_t)c.n_layers * sizeof(Plan), cudaMemcpyHostToDevice));
    DA(&h->done_ctr, 4);   // per internal stream: finished CTAs of its running LRFU kernel; whether the layer's plan went stale
    CKC(cudaMemset(h->done_ctr, 0, 4 * sizeof(int)));
  }
  DA(&h->tab, (size_t)c.max_context + 1);
  st.tab = h->tab;
  DA(&st.errword, 1);
  DA(&st.counters, 4);
  DA(&h->Asum, h->units);
  const int capgroups = (h->cap + GRP - 1) / GRP;
  h->cap_s = evict ? h->cap : 4;   // whole 128-byte lines of logit rows per unit (cap is a multiple of 16)
  h->pmax = capgroups / GMIN + 2;
  for (int i = 0; i < NSETS; ++i) {
    DA(&h->sc_logits[i], (size_t)h->U * h->cap_s * QH);
    DA(&h->sc_mfin[i], (size_t)h->U * 2 * QH);
  }
  for (int i = 0; i < 2; ++i) {
    DA(&h->sc_partials[i], (size_t)h->U * h->pmax * (16 + h->G * HD));
    DA(&h->sc_ticket[i], h->U);
    CKC(cudaMemset(h->sc_ticket[i], 0, (size_t)h->U * sizeof(int)));
  }
  for (int i = 0; i < 2; ++i) DA(&h->sc_pbar[i], (size_t)h->U * h->cap_s);
  DA(&h->piece_ctr, 4);
  CKC(cudaMemset(h->piece_ctr, 0, 4 * sizeof(int)));
  const size_t qn = (size_t)c.batch * c.n_q_heads * HD, kn = (size_t)c.batch * c.n_kv_heads * HD;
  for (int i = 0; i < crystalkv::HOST_RING; ++i) { DA(&h->dq[i], qn); DA(&h->dout[i], qn); DA(&h->dk[i], kn); DA(&h->dv[i], kn); }
  DA(&h->dummy_out, qn);
  DA(&h->io_rec, (size_t)3 * h->cap);
  DA(&h->io_rows, (size_t)2 * h->cap * ROW_BYTES);
  DA(&h->io_n, 1);

  // lambda^D as fp32 from an fp64 pow; pow(0, 0) = 1 keeps same-step hits when lambda = 0
  {
    std::vector<float> tab((size_t)c.max_context + 1);
    for (int D = 0; D <= c.max_context; ++D) tab[D] = (float)std::pow((double)c.lambda, (double)D);
    CKC(cudaMemcpy(h->tab, tab.data(), tab.size() * sizeof(float), cudaMemcpyHostToDevice));
  }
  init_free_stack_kernel<<<1024, 256>>>(st.free_stack, st.free_top, h->pages_per_seq, c.batch);
  fill_int_kernel<<<256, 256>>>(st.budget, h->units, c.budget_per_head);
  CKC(cudaMemset(st.n_cur, 0, (size_t)h->units * sizeof(int)));
  CKC(cudaMemset(st.hole, 0, (size_t)h->units * sizeof(int)));
  CKC(cudaMemset(st.npages, 0, (size_t)h->units * sizeof(int)));
  CKC(cudaMemset(st.errword, 0, sizeof(int)));
  CKC(cudaMemset(st.counters, 0, 4 * sizeof(unsigned long long)));
  CKC(cudaGetLastError());
  CKC(cudaDeviceSynchronize());
  h->t_layer.assign(c.n_layers, -1);
  h->lastF.assign(c.n_layers, -1);
  *out = h;
  return CRYSTALKV_OK;
#undef CREATE_FAIL
#undef CKC
#undef DA
}

int crystalkv_set_stage(crystalkv_t* h, int stage) {
  if (!h) return CRYSTALKV_EINVAL;
  if (stage != CRYSTALKV_STAGE_THINK && stage != CRYSTALKV_STAGE_ANSWER) return fail(h, CRYSTALKV_EINVAL, "bad stage");
  if (stage == CRYSTALKV_STAGE_THINK && h->answer_steps > 0)
    return fail(h, CRYSTALKV_ESTATE, "answer tokens were appended; the think stage cannot resume");
  ON_DEVICE(h);
  if (stage != h->stage)   // no LRFU kernel is left behind the switch
    for (cudaStream_t x : h->side) CK(h, cudaStreamSynchronize(x));
  h->prev_layer = -1;
  h->stage = stage;
  return CRYSTALKV_OK;
}

int crystalkv_time(crystalkv_t* h, int layer) {
  if (!h || layer < 0 || layer >= h->cfg.n_layers) return -1;
  return h->t_layer[layer];
}

// Prompt insertion and the Algorithm 1 passes that seed CRF/tau: one pass with the last query
// (W = 0) or a replay of the last W queries, each over the tokens up to its own.
static int prefill_common(crystalkv_t* h, int layer, const void* k, const void* v, const void* q,
                          int P, int W, void* out_window, void* stream) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  if (!k || !v || !q) return fail(h, CRYSTALKV_EINVAL, "null tensor");
  const crystalkv_config_t& c = h->cfg;
  const bool evict = c.mode == CRYSTALKV_MODE_EVICT;
  if (P < 1) return fail(h, CRYSTALKV_EINVAL, "P must be >= 1");
  // A prompt beyond the budget is scored from the caller's tensors and only its survivors are
  // stored; with an observation window the whole prompt must fit the pool for a moment (the
  // window's attention outputs need the values).
  const bool score_first = evict && W == 0 && P > (c.budget_ratio > 0.f ? ratio_budget(c, P) : c.budget_per_head);
  if (evict && !score_first && P > c.budget_per_head + c.max_answer_tokens)
    return fail(h, CRYSTALKV_EINVAL, "prompt with an observation window longer than budget_per_head + max_answer_tokens");
  if (evict && P + 1 > h->cap) return fail(h, CRYSTALKV_EINVAL, "prompt longer than the heads' list capacity (max_budget + evict_every + max_answer_tokens)");
  if (P >= c.max_context) return fail(h, CRYSTALKV_EINVAL, "prompt reaches max_context");
  if (h->t_layer[layer] >= 0) return fail(h, CRYSTALKV_ESTATE, "layer already prefilled");
  ON_DEVICE(h);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  rc = join_side(h, s);   // the insertion takes pages; no LRFU kernel may take or return any meanwhile
  if (rc) return rc;
  if (evict && c.budget_ratio > 0.f) {   // the prompt's share of the context
    fill_layer_budget_kernel<<<(h->U + NT - 1) / NT, NT, 0, s>>>(h->st, layer, ratio_budget(c, P));
    CK(h, cudaGetLastError());
  }
  if (score_first) {
    // Algorithm 1 with the last query over metadata and logits only; every kernel on `s`, which has
    // joined the internal stream, so any scratch set is free
    DecodeParams p = make_params(h, layer);
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.t = P - 1;
    p.append = 0; p.track = 1; p.release = 1; p.rows_absent = 1; p.plan_append = 1;
    prefill_score_kernel<<<h->U, NT, 0, s>>>(h->st, p.sc, layer, static_cast<const __nv_bfloat16*>(k), p.q, P, h->G,
                                             p.scale, p.scale_log2);
    CK(h, cudaGetLastError());
    CK(h, lrfu_dispatch(h->G, p, h->U, s));
    prefill_rows_kernel<<<h->U, NT, 0, s>>>(h->st, layer, static_cast<const __nv_bfloat16*>(k),
                                            static_cast<const __nv_bfloat16*>(v), P);
    CK(h, cudaGetLastError());
    h->prev_layer = -1;
    h->t_layer[layer] = P - 1;
    return CRYSTALKV_OK;
  }
  prefill_insert_kernel<<<h->U, NT, 0, s>>>(h->st, layer, static_cast<const __nv_bfloat16*>(k),
                                            static_cast<const __nv_bfloat16*>(v), P, W > 0 ? 1 : 0);
  CK(h, cudaGetLastError());
  if (evict) {
    const int passes = W > 0 ? W : 1;
    const size_t qn = (size_t)c.batch * c.n_q_heads * HD;
    int planned_groups = -1;
    for (int i = 0; i < passes; ++i) {
      // Algorithm 1 with the query of token t: steps 1-3 for every query, step 4 (down to the
      // budget, emptied pages back to the free list) after the last one
      const int t = P - passes + i;
      const bool last = i == passes - 1;
      // a scoring pass over the first t + 1 entries; a plan serves the passes that follow it until
      // their heads are two groups longer (pieces take their bounds from the lengths at launch)
      const int groups = (t + 1 + GRP - 1) / GRP;
      const bool planned = planned_groups < 0 || groups >= planned_groups + 2;
      if (planned) {
        rc = replan(h, layer, 1, 0, last ? 0 : t + 1, s);
        if (rc) return rc;
        planned_groups = groups;
      }
      DecodeParams p = make_params(h, layer);
      p.q = static_cast<const __nv_bfloat16*>(q) + (size_t)i * qn;
      p.k_new = p.v_new = nullptr;
      p.out = out_window ? static_cast<__nv_bfloat16*>(out_window) + (size_t)i * qn : h->dummy_out;
      p.t = t;
      p.append = 0; p.track = 1; p.release = 1;
      if (!last) { p.n_limit = t + 1; p.hold = 1; }
      else p.plan_append = 1;   // the layer's first decode step
      h->prev_layer = -1;       // the plan kernel ahead writes what the attention kernel reads at once
      rc = launch_step(h, p, layer, s, i > 0);
      if (rc) return rc;
    }
    rc = join_side(h, s);
    if (rc) return rc;
  } else {
    rc = replan(h, layer, 1, 1, 0, s);
    if (rc) return rc;
    h->prev_layer = -1;
  }
  h->t_layer[layer] = P - 1;
  return CRYSTALKV_OK;
}

int crystalkv_prefill(crystalkv_t* h, int layer, const void* k, const void* v, const void* q_last,
                      int P, void* stream) {
  return prefill_common(h, layer, k, v, q_last, P, 0, nullptr, stream);
}

int crystalkv_prefill_window(crystalkv_t* h, int layer, const void* k, const void* v,
                             const void* q_window, int P, int W, void* out_window, void* stream) {
  if (h && (W < 1 || W > P)) return fail(h, CRYSTALKV_EINVAL, "W must be in [1, P]");
  return prefill_common(h, layer, k, v, q_window, P, W, out_window, stream);
}

int crystalkv_decode_step(crystalkv_t* h, int layer, const void* q, const void* k_new,
                          const void* v_new, void* out, void* stream) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  if (!q || !k_new || !v_new || !out) return fail(h, CRYSTALKV_EINVAL, "null tensor");
  const crystalkv_config_t& c = h->cfg;
  if (h->t_layer[layer] < 0) return fail(h, CRYSTALKV_ESTATE, "decode before prefill");
  const int t = h->t_layer[layer] + 1;
  ON_DEVICE(h);
  if (t >= c.max_context) return fail(h, CRYSTALKV_ESTATE, "max_context reached");
  const bool track = c.mode == CRYSTALKV_MODE_EVICT && h->stage == CRYSTALKV_STAGE_THINK;
  if (c.mode == CRYSTALKV_MODE_EVICT && h->stage == CRYSTALKV_STAGE_ANSWER) {
    // every layer appends once per answer token; count tokens by layer 0's clock
    const int used = h->answer_steps / c.n_layers;
    if (used >= c.max_answer_tokens) return fail(h, CRYSTALKV_ESTATE, "max_answer_tokens reached");
  }
  DecodeParams p = make_params(h, layer);
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k_new = static_cast<const __nv_bfloat16*>(k_new);
  p.v_new = static_cast<const __nv_bfloat16*>(v_new);
  p.out = static_cast<__nv_bfloat16*>(out);
  p.t = t;
  p.append = 1; p.track = track ? 1 : 0; p.release = 0;
  p.plan_append = 1;
  rc = launch_step(h, p, layer, static_cast<cudaStream_t>(stream));
  if (rc) return rc;
  h->t_layer[layer] = t;
  if (!track && c.mode == CRYSTALKV_MODE_EVICT) h->answer_steps++;
  return CRYSTALKV_OK;
}

int crystalkv_decode_step_host(crystalkv_t* h, int layer, const void* q_host, const void* k_new_host,
                               const void* v_new_host, void* out_host, void* stream) {
  int rc = check_layer(h, layer);
  if (rc) return rc;
  if (!q_host || !k_new_host || !v_new_host || !out_host) return fail(h, CRYSTALKV_EINVAL, "null tensor");
  ON_DEVICE(h);
  const crystalkv_config_t& c = h->cfg;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t qb = (size_t)c.batch * c.n_q_heads * HD * 2, kb = (size_t)c.batch * c.n_kv_heads * HD * 2;
  if (h->t_layer[layer] < 0) return fail(h, CRYSTALKV_ESTATE, "decode before prefill");
  // Staging set j was last used HOST_RING host steps ago.  Page-locked inputs that the GPU can
  // address are fetched by one small kernel in the caller's stream; anything else (pageable
  // memory, 16-byte misalignment) goes up by three copies on the copy-in stream, for which the
  // caller's stream then waits.  The result comes down on the copy-out stream behind the
  // attention kernel.
  const int j = (int)(h->nHost % crystalkv::HOST_RING);
  const void* dev_view[3] = {nullptr, nullptr, nullptr};
  const void* host_in[3] = {q_host, k_new_host, v_new_host};
  bool mapped = true;
  for (int i = 0; i < 3 && mapped; ++i) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host_in[i]) != cudaSuccess) { cudaGetLastError(); mapped = false; break; }
    mapped = at.type == cudaMemoryTypeHost && at.devicePointer != nullptr &&
             (reinterpret_cast<uintptr_t>(at.devicePointer) & 15) == 0;
    dev_view[i] = at.devicePointer;
  }
  if (mapped) {
    // The set's staged inputs were read by an attention kernel HOST_RING launches back in this
    // stream, which is complete before this kernel may start.  Its result buffer must have been
    // copied down as well; a wait in the caller's stream costs several microseconds, so one wait
    // on a much newer copy covers the steps until the ring comes round again.
    const long long n = h->nHost;
    if (n >= crystalkv::HOST_RING && n - crystalkv::HOST_RING > h->outJoined) {
      const long long target = n - 4;   // a copy that has long run by the time the stream gets here
      CK(h, cudaStreamWaitEvent(s, h->evOut[target % crystalkv::HOST_RING], 0));
      h->outJoined = target;
    }
    const int nq = (int)(qb / 16), nk = (int)(kb / 16);
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3((nq + 2 * nk + NT - 1) / NT);
    lc.blockDim = dim3(NT);
    lc.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    CK(h, cudaLaunchKernelEx(&lc, stage_in_kernel, reinterpret_cast<uint4*>(h->dq[j]), reinterpret_cast<uint4*>(h->dk[j]),
                             reinterpret_cast<uint4*>(h->dv[j]), static_cast<const uint4*>(dev_view[0]),
                             static_cast<const uint4*>(dev_view[1]), static_cast<const uint4*>(dev_view[2]), nq, nk));
  } else {
    // the copy back of the step that used the set before ran behind that step's attention
    // kernel, so its event covers both
    if (h->nHost >= crystalkv::HOST_RING) CK(h, cudaStreamWaitEvent(h->copy_in, h->evOut[j], 0));
    CK(h, cudaMemcpyAsync(h->dq[j], q_host, qb, cudaMemcpyHostToDevice, h->copy_in));
    CK(h, cudaMemcpyAsync(h->dk[j], k_new_host, kb, cudaMemcpyHostToDevice, h->copy_in));
    CK(h, cudaMemcpyAsync(h->dv[j], v_new_host, kb, cudaMemcpyHostToDevice, h->copy_in));
    CK(h, cudaEventRecord(h->evIn[j], h->copy_in));
    CK(h, cudaStreamWaitEvent(s, h->evIn[j], 0));
  }
  rc = crystalkv_decode_step(h, layer, h->dq[j], h->dk[j], h->dv[j], h->dout[j], stream);
  if (rc) return rc;
  CK(h, cudaEventRecord(h->evUse[j], s));
  CK(h, cudaStreamWaitEvent(h->copy_out, h->evUse[j], 0));
  CK(h, cudaMemcpyAsync(out_host, h->dout[j], qb, cudaMemcpyDeviceToHost, h->copy_out));
  CK(h, cudaEventRecord(h->evOut[j], h->copy_out));
  h->nHost++;
  return CRYSTALKV_OK;
}

int crystalkv_rebudget(crystalkv_t* h, void* stream) {
  if (!h) return CRYSTALKV_EINVAL;
  if (h->cuda_dead) return fail(h, CRYSTALKV_ECUDA, "an earlier CUDA error is sticky for this handle");
  const crystalkv_config_t& c = h->cfg;
  if (c.mode != CRYSTALKV_MODE_EVICT) return fail(h, CRYSTALKV_ESTATE, "rebudget in FullKV mode");
  ON_DEVICE(h);
  const int t_last = h->t_layer[0];
  if (t_last < 0) return fail(h, CRYSTALKV_ESTATE, "rebudget before prefill");
  for (int l = 1; l < c.n_layers; ++l)
    if (h->t_layer[l] != t_last) return fail(h, CRYSTALKV_ESTATE, "layers are at different time steps");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (int jr = join_side(h, s)) return jr;
  crf_sum_kernel<<<h->units, NT, 0, s>>>(h->st, t_last, h->Asum);
  CK(h, cudaGetLastError());
  const int N = c.n_layers * c.n_kv_heads;
  const size_t sm = (size_t)N * (3 * sizeof(double) + sizeof(long long) + 2 * sizeof(int)) + (size_t)c.n_layers * 2 * sizeof(double);
  if (sm > 48 * 1024) CK(h, cudaFuncSetAttribute(alg2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm));
  const long long B_total = (long long)(c.budget_ratio > 0.f ? ratio_budget(c, t_last + 1) : c.budget_per_head) * N;
  alg2_kernel<<<c.batch, NT, sm, s>>>(h->Asum, h->st.budget, c.n_layers, c.n_kv_heads, B_total, c.min_budget, c.max_budget);
  CK(h, cudaGetLastError());
  for (int l = 0; l < c.n_layers; ++l) {
    shrink_kernel<<<h->U, NT, 0, s>>>(h->st, l, t_last, reinterpret_cast<int*>(h->sc_pbar[0]), h->cap_s);
    CK(h, cudaGetLastError());
  }
  // heads changed length: every layer's next decode step needs a new plan
  return replan(h, 0, c.n_layers, 1, 0, s);
}

int crystalkv_set_budget(crystalkv_t* h, int layer, int seq, int kv_head, int32_t budget, void* stream) {
  int rc = check_unit(h, layer, seq, kv_head);
  if (rc) return rc;
  const crystalkv_config_t& c = h->cfg;
  if (c.mode != CRYSTALKV_MODE_EVICT) return fail(h, CRYSTALKV_ESTATE, "set_budget in FullKV mode");
  if (budget < 1 || budget > c.max_budget) return fail(h, CRYSTALKV_EINVAL, "budget outside [1, max_budget]");
  ON_DEVICE(h);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (int jr = join_side(h, s)) return jr;
  const int uid = (seq * c.n_layers + layer) * c.n_kv_heads + kv_head;
  CK(h, cudaMemcpyAsync(h->st.budget + uid, &budget, sizeof(int), cudaMemcpyHostToDevice, s));
  CK(h, cudaStreamSynchronize(s));
  if (h->t_layer[layer] >= 0) {
    shrink_kernel<<<h->U, NT, 0, s>>>(h->st, layer, h->t_layer[layer], reinterpret_cast<int*>(h->sc_pbar[0]), h->cap_s);
    CK(h, cudaGetLastError());
    return replan(h, layer, 1, 1, 0, s);
  }
  return CRYSTALKV_OK;
}

int crystalkv_get_budgets(crystalkv_t* h, int32_t* out_host, void* stream) {
  if (!h || !out_host) return fail(h, CRYSTALKV_EINVAL, "null argument");
  ON_DEVICE(h);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (int jr = join_side(h, s)) return jr;
  CK(h, cudaMemcpyAsync(out_host, h->st.budget, (size_t)h->units * sizeof(int), cudaMemcpyDeviceToHost, s));
  CK(h, cudaStreamSynchronize(s));
  return CRYSTALKV_OK;
}

// Copies one head's entries to the host, sorted by token position: records and, if asked for, rows.
static int fetch_unit(crystalkv_t* h, int layer, int seq, int kv_head, std::vector<int32_t>& rec,
                      std::vector<unsigned char>* krows, std::vector<unsigned char>* vrows, cudaStream_t s) {
  const crystalkv_config_t& c = h->cfg;
  if (int jr = join_side(h, s)) return jr;
  const int uid = (seq * c.n_layers + layer) * c.n_kv_heads + kv_head;
  export_unit_kernel<<<1, NT, 0, s>>>(h->st, uid, seq, h->io_rec, krows ? h->io_rows : nullptr,
                                      krows ? h->io_rows + (size_t)h->cap * ROW_BYTES : nullptr, h->io_n);
  CK(h, cudaGetLastError());
  int n = 0;
  CK(h, cudaMemcpyAsync(&n, h->io_n, sizeof(int), cudaMemcpyDeviceToHost, s));
  CK(h, cudaStreamSynchronize(s));
  std::vector<int32_t> raw((size_t)3 * n);
  std::vector<unsigned char> kr, vr;
  CK(h, cudaMemcpyAsync(raw.data(), h->io_rec, raw.size() * 4, cudaMemcpyDeviceToHost, s));
  if (krows) {
    kr.resize((size_t)n * ROW_BYTES); vr.resize((size_t)n * ROW_BYTES);
    CK(h, cudaMemcpyAsync(kr.data(), h->io_rows, kr.size(), cudaMemcpyDeviceToHost, s));
    CK(h, cudaMemcpyAsync(vr.data(), h->io_rows + (size_t)h->cap * ROW_BYTES, vr.size(), cudaMemcpyDeviceToHost, s));
  }
  CK(h, cudaStreamSynchronize(s));
  std::vector<int> idx(n);
  for (int i = 0; i < n; ++i) idx[i] = i;
  std::sort(idx.begin(), idx.end(), [&](int a, int b) { return raw[3 * a] < raw[3 * b]; });
  rec.resize((size_t)3 * n);
  if (krows) { krows->resize((size_t)n * ROW_BYTES); vrows->resize((size_t)n * ROW_BYTES); }
  for (int i = 0; i < n; ++i) {
    std::memcpy(&rec[3 * i], &raw[3 * idx[i]], 12);
    if (krows) {
      std::memcpy(krows->data() + (size_t)i * ROW_BYTES, kr.data() + (size_t)idx[i] * ROW_BYTES, ROW_BYTES);
      std::memcpy(vrows->data() + (size_t)i * ROW_BYTES, vr.data() + (size_t)idx[i] * ROW_BYTES, ROW_BYTES);
    }
  }
  return CRYSTALKV_OK;
}

int crystalkv_export_state(crystalkv_t* h, int layer, int seq, int kv_head, int32_t* host_buf,
                           int32_t cap, int32_t* n_out, void* stream) {
  int rc = check_unit(h, layer, seq, kv_head);
  if (rc) return rc;
  if (!host_buf || !n_out) return fail(h, CRYSTALKV_EINVAL, "null argument");
  ON_DEVICE(h);
  std::vector<int32_t> rec;
  rc = fetch_unit(h, layer, seq, kv_head, rec, nullptr, nullptr, static_cast<cudaStream_t>(stream));
  if (rc) return rc;
  const int n = (int)(rec.size() / 3);
  *n_out = n;
  if (n > cap) return fail(h, CRYSTALKV_ESTATE, "buffer too small");
  std::memcpy(host_buf, rec.data(), rec.size() * 4);
  return CRYSTALKV_OK;
}

int crystalkv_export_kv(crystalkv_t* h, int layer, int seq, int kv_head, void* k_rows_host, void* v_rows_host,
                        int32_t cap, int32_t* n_out, void* stream) {
  int rc = check_unit(h, layer, seq, kv_head);
  if (rc) return rc;
  if (!k_rows_host || !v_rows_host || !n_out) return fail(h, CRYSTALKV_EINVAL, "null argument");
  ON_DEVICE(h);
  std::vector<int32_t> rec;
  std::vector<unsigned char> kr, vr;
  rc = fetch_unit(h, layer, seq, kv_head, rec, &kr, &vr, static_cast<cudaStream_t>(stream));
  if (rc) return rc;
  const int n = (int)(rec.size() / 3);
  *n_out = n;
  if (n > cap) return fail(h, CRYSTALKV_ESTATE, "buffer too small");
  std::memcpy(k_rows_host, kr.data(), kr.size());
  std::memcpy(v_rows_host, vr.data(), vr.size());
  return CRYSTALKV_OK;
}

int crystalkv_get_retained(crystalkv_t* h, int layer, int seq, int kv_head, int32_t* pos_out_host,
                           int32_t cap, int32_t* n_out, void* stream) {
  int rc = check_unit(h, layer, seq, kv_head);
  if (rc) return rc;
  if (!pos_out_host || !n_out) return fail(h, CRYSTALKV_EINVAL, "null argument");
  ON_DEVICE(h);
  std::vector<int32_t> rec;
  rc = fetch_unit(h, layer, seq, kv_head, rec, nullptr, nullptr, static_cast<cudaStream_t>(stream));
  if (rc) return rc;
  const int n = (int)(rec.size() / 3);
  *n_out = n;
  if (n > cap) return fail(h, CRYSTALKV_ESTATE, "buffer too small");
  for (int i = 0; i < n; ++i) pos_out_host[i] = rec[3 * i];
  return CRYSTALKV_OK;
}

int crystalkv_import_state(crystalkv_t* h, int layer, int seq, int kv_head, const int32_t* host_buf,
                           int32_t n_rec, const void* k_rows_host, const void* v_rows_host, int32_t budget,
                           int32_t t, void* stream) {
  int rc = check_unit(h, layer, seq, kv_head);
  if (rc) return rc;
  if (!host_buf || !k_rows_host || !v_rows_host) return fail(h, CRYSTALKV_EINVAL, "null argument");
  const crystalkv_config_t& c = h->cfg;
  if (n_rec < 1 || n_rec + 1 > h->cap) return fail(h, CRYSTALKV_EINVAL, "entry count outside [1, list capacity)");
  if (budget < 0 || (c.mode == CRYSTALKV_MODE_EVICT && budget > c.max_budget)) return fail(h, CRYSTALKV_EINVAL, "budget outside [0, max_budget]");
  if (t < 0 || t >= c.max_context) return fail(h, CRYSTALKV_EINVAL, "time outside [0, max_context)");
  if (h->t_layer[layer] >= 0 && h->t_layer[layer] != t) return fail(h, CRYSTALKV_ESTATE, "the layer is at another time step");
  for (int i = 0; i < n_rec; ++i)
    if (host_buf[3 * i] < 0 || host_buf[3 * i] > t || host_buf[3 * i + 2] < 0 || host_buf[3 * i + 2] > t)
      return fail(h, CRYSTALKV_EINVAL, "a record's position or last hit time lies after the layer's time");
  ON_DEVICE(h);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (int jr = join_side(h, s)) return jr;
  const int uid = (seq * c.n_layers + layer) * c.n_kv_heads + kv_head;
  CK(h, cudaMemcpyAsync(h->io_rec, host_buf, (size_t)n_rec * 12, cudaMemcpyHostToDevice, s));
  CK(h, cudaMemcpyAsync(h->io_rows, k_rows_host, (size_t)n_rec * ROW_BYTES, cudaMemcpyHostToDevice, s));
  CK(h, cudaMemcpyAsync(h->io_rows + (size_t)h->cap * ROW_BYTES, v_rows_host, (size_t)n_rec * ROW_BYTES, cudaMemcpyHostToDevice, s));
  int b = budget;
  if (b == 0) {
    CK(h, cudaMemcpyAsync(&b, h->st.budget + uid, sizeof(int), cudaMemcpyDeviceToHost, s));
    CK(h, cudaStreamSynchronize(s));
  }
  import_unit_kernel<<<1, NT, 0, s>>>(h->st, uid, seq, h->io_rec, h->io_rows, h->io_rows + (size_t)h->cap * ROW_BYTES, n_rec, b);
  CK(h, cudaGetLastError());
  CK(h, cudaStreamSynchronize(s));   // the host buffers and the staging area are free again
  h->t_layer[layer] = t;
  h->prev_layer = -1;
  return replan(h, layer, 1, 1, 0, s);
}

int crystalkv_get_counters(crystalkv_t* h, uint64_t* entries_attended, uint64_t* hits,
                           uint64_t* evictions, void* stream) {
  if (!h) return CRYSTALKV_EINVAL;
  ON_DEVICE(h);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (int jr = join_side(h, s)) return jr;
  unsigned long long v[4];
  CK(h, cudaMemcpyAsync(v, h->st.counters, sizeof(v), cudaMemcpyDeviceToHost, s));
  CK(h, cudaStreamSynchronize(s));
  if (entries_attended) *entries_attended = v[0];
  if (hits) *hits = v[1];
  if (evictions) *evictions = v[2];
  return CRYSTALKV_OK;
}

int crystalkv_validate(crystalkv_t* h, void* stream) {
  if (!h) return CRYSTALKV_EINVAL;
  if (h->cuda_dead) return fail(h, CRYSTALKV_ECUDA, "an earlier CUDA error is sticky for this handle");
  const crystalkv_config_t& c = h->cfg;
  for (int l = 0; l < c.n_layers; ++l)
    if (h->t_layer[l] < 0) return fail(h, CRYSTALKV_ESTATE, "validate before every layer is prefilled");
  ON_DEVICE(h);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (int jr = join_side(h, s)) return jr;
  const long long total = (long long)c.batch * h->pages_per_seq;
  int* seen = nullptr;
  CK(h, cudaMalloc(&seen, (size_t)(total + 2) * sizeof(int)));
  cudaError_t e = cudaMemsetAsync(seen, 0, (size_t)(total + 2) * sizeof(int), s);
  if (e == cudaSuccess) {
    mark_free_kernel<<<dim3(256, c.batch), 256, 0, s>>>(h->st, seen);
    for (int l = 0; l < c.n_layers; ++l)
      mark_owned_kernel<<<h->U, 128, 0, s>>>(h->st, l, seen);
    count_bad_kernel<<<1024, 256, 0, s>>>(seen, total, seen + total + 1);
    e = cudaGetLastError();
  }
  int res[2] = {0, 0};
  if (e == cudaSuccess) e = cudaMemcpyAsync(res, seen + total, 2 * sizeof(int), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  cudaFree(seen);
  CK(h, e);
  if (res[0] || res[1])
    return fail(h, CRYSTALKV_ECHECK, "page ownership broken: " + std::to_string(res[0]) + " ids or counts out of range, " +
                                         std::to_string(res[1]) + " pages not owned exactly once");
  return CRYSTALKV_OK;
}

// ---- the page-ownership check for callers that cannot allocate device memory
// The per-page counters live in this file-scope device array instead of a temporary from
// cudaMalloc.  Every GPU that loads the library holds the array (512 KB) until the process exits.
constexpr long long STATIC_SEEN_PAGES = 1ll << 17;
static __device__ __align__(256) int g_seen_static[STATIC_SEEN_PAGES + 2];
constexpr int STATIC_MAX_DEVICES = 64;
static int* g_seen_addr[STATIC_MAX_DEVICES] = {};   // device address of the array, per device ordinal
static std::mutex g_seen_mu;                        // guards the look-up above

int crystalkv_validate_static(crystalkv_t* h, int32_t* counts_out_host, void* stream) {
  if (!h) return CRYSTALKV_EINVAL;
  if (h->cuda_dead) return fail(h, CRYSTALKV_ECUDA, "an earlier CUDA error is sticky for this handle");
  const crystalkv_config_t& c = h->cfg;
  for (int l = 0; l < c.n_layers; ++l)
    if (h->t_layer[l] < 0) return fail(h, CRYSTALKV_ESTATE, "validate before every layer is prefilled");
  const long long total = (long long)c.batch * h->pages_per_seq;
  if (total > STATIC_SEEN_PAGES)
    return fail(h, CRYSTALKV_EINVAL,
                "crystalkv_validate_static: the handle has " + std::to_string(total) + " pool pages, the built-in "
                "scratch covers " + std::to_string(STATIC_SEEN_PAGES) + "; use crystalkv_validate");
  if (c.device >= STATIC_MAX_DEVICES) return fail(h, CRYSTALKV_EINVAL, "crystalkv_validate_static: device ordinal above 63");
  ON_DEVICE(h);
  int* seen = nullptr;
  {
    // In host code the array's name is only a handle for the runtime; its device address has
    // to be asked for, once per device and with that device current.
    std::lock_guard<std::mutex> lock(g_seen_mu);
    if (!g_seen_addr[c.device]) {
      int* addr = nullptr;
      CK(h, cudaGetSymbolAddress(reinterpret_cast<void**>(&addr), g_seen_static));
      g_seen_addr[c.device] = addr;
    }
    seen = g_seen_addr[c.device];
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (int jr = join_side(h, s)) return jr;
  // the array keeps what the last call left: everything this call reads starts from zero
  CK(h, cudaMemsetAsync(seen, 0, (size_t)(total + 2) * sizeof(int), s));
  mark_free_kernel<<<dim3(256, c.batch), 256, 0, s>>>(h->st, seen);
  for (int l = 0; l < c.n_layers; ++l)
    mark_owned_kernel<<<h->U, 128, 0, s>>>(h->st, l, seen);
  count_bad_kernel<<<1024, 256, 0, s>>>(seen, total, seen + total + 1);
  CK(h, cudaGetLastError());
  int res[2] = {0, 0};
  CK(h, cudaMemcpyAsync(res, seen + total, 2 * sizeof(int), cudaMemcpyDeviceToHost, s));
  CK(h, cudaStreamSynchronize(s));
  if (counts_out_host) { counts_out_host[0] = res[0]; counts_out_host[1] = res[1]; }
  if (res[0] || res[1])
    return fail(h, CRYSTALKV_ECHECK, "page ownership broken: " + std::to_string(res[0]) + " ids or counts out of range, " +
                                         std::to_string(res[1]) + " pages not owned exactly once");
  return CRYSTALKV_OK;
}

int crystalkv_debug_set_page(crystalkv_t* h, int layer, int seq, int kv_head, int32_t index, int32_t page, void* stream) {
  int rc = check_unit(h, layer, seq, kv_head);
  if (rc) return rc;
  if (index < 0 || index >= h->st.capg || page < 0 || page >= h->pages_per_seq)
    return fail(h, CRYSTALKV_EINVAL, "page table index or page id out of range");
  ON_DEVICE(h);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (int jr = join_side(h, s)) return jr;
  const int uid = (seq * h->cfg.n_layers + layer) * h->cfg.n_kv_heads + kv_head;
  CK(h, cudaMemcpyAsync(h->st.ptab + (size_t)uid * h->st.capg + index, &page, sizeof(int), cudaMemcpyHostToDevice, s));
  CK(h, cudaStreamSynchronize(s));
  return CRYSTALKV_OK;
}

int crystalkv_debug_ctas_needed(int32_t whole_ctas, const int32_t* runs_by_length) {
  if (!runs_by_length || whole_ctas < 0) return CRYSTALKV_EINVAL;
  int cnt[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  for (int s = 1; s < 8; ++s) {
    if (runs_by_length[s] < 0) return CRYSTALKV_EINVAL;
    cnt[s] = runs_by_length[s];
  }
  return ctas_needed(whole_ctas, cnt);
}

int crystalkv_debug_get_plan(crystalkv_t* h, int layer, int32_t* hdr_host, int32_t* wrange_host, int32_t warps_cap,
                             int32_t* desc_host, int32_t pieces_cap, void* stream) {
  if (!h) return CRYSTALKV_EINVAL;
  if (h->cuda_dead) return fail(h, CRYSTALKV_ECUDA, "an earlier CUDA error is sticky for this handle");
  if (layer < 0 || layer >= h->cfg.n_layers || !hdr_host || !wrange_host || !desc_host)
    return fail(h, CRYSTALKV_EINVAL, "layer out of range or a NULL output");
  const int nWarps = h->grid * NW;
  if (warps_cap < nWarps || pieces_cap < nWarps + h->U) return fail(h, CRYSTALKV_EINVAL, "output arrays too small for the plan");
  ON_DEVICE(h);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (int jr = join_side(h, s)) return jr;
  const Plan& pl = h->plans[layer];
  CK(h, cudaMemcpyAsync(hdr_host, pl.hdr, 4 * sizeof(int), cudaMemcpyDeviceToHost, s));
  std::vector<int4> wr((size_t)nWarps);
  CK(h, cudaMemcpyAsync(wr.data(), pl.wrange, (size_t)nWarps * sizeof(int4), cudaMemcpyDeviceToHost, s));
  CK(h, cudaMemcpyAsync(desc_host, pl.desc, (size_t)(nWarps + h->U) * sizeof(int4), cudaMemcpyDeviceToHost, s));
  CK(h, cudaStreamSynchronize(s));
  for (int w = 0; w < nWarps; ++w) { wrange_host[2 * w] = wr[w].x; wrange_host[2 * w + 1] = wr[w].y; }
  return CRYSTALKV_OK;
}

int crystalkv_join(crystalkv_t* h, void* stream) {
  if (!h) return CRYSTALKV_EINVAL;
  if (h->cuda_dead) return fail(h, CRYSTALKV_ECUDA, "an earlier CUDA error is sticky for this handle");
  ON_DEVICE(h);
  return join_side(h, static_cast<cudaStream_t>(stream));
}

int crystalkv_check(crystalkv_t* h, void* stream) {
  if (!h) return CRYSTALKV_EINVAL;
  ON_DEVICE(h);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (int jr = join_side(h, s)) return jr;
  int w = 0;
  CK(h, cudaMemcpyAsync(&w, h->st.errword, sizeof(int), cudaMemcpyDeviceToHost, s));
  CK(h, cudaStreamSynchronize(s));
  if (w == 0) return CRYSTALKV_OK;
  CK(h, cudaMemsetAsync(h->st.errword, 0, sizeof(int), s));
  std::string msg = "device error word:";
  if (w & ERR_FREE_UNDERFLOW) msg += " free page list underflow;";
  if (w & ERR_OVER_EVICT) msg += " head further over its budget than the eviction period in a decode step;";
  if (w & ERR_CAPACITY) msg += " head list capacity exceeded;";
  if (w & ERR_NUCLEUS) msg += " top-p boundary not found;";
  if (w & ERR_COPY_TIMEOUT) msg += " a bulk copy into shared memory timed out;";
  if (w & ERR_PLAN) msg += " a layer's launch plan did not fit the launch (or a head was empty);";
  return fail(h, CRYSTALKV_ECHECK, msg);
}

}  // extern "C"
