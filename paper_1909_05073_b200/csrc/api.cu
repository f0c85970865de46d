// C ABI entry points: argument checks, kernel selection, layer stacks.
#include <cstring>
#include <cstdlib>
#include <mutex>
#include <new>
#include <vector>

#include "pconv_internal.h"
#ifdef PCONV_DEV
#include "pconv_dev.h"
#endif

using namespace pconv;

int pconv::device_sm_count() {
  constexpr int kMaxDev = 64, kDefault = 148;
  static int cached[kMaxDev] = {0};
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) {
    cudaGetLastError();
    return kDefault;
  }
  int v = cached[dev];
  if (v > 0) return v;
  if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) {
    cudaGetLastError();
    return kDefault;
  }
  cached[dev] = v;
  return v;
}

extern "C" const char* pconv_status_str(pconv_status s) {
  switch (s) {
    case PCONV_OK: return "ok";
    case PCONV_ERR_NULL: return "required pointer is NULL";
    case PCONV_ERR_SHAPE: return "bad shape or stride";
    case PCONV_ERR_PATTERN_SET: return "bad pattern set";
    case PCONV_ERR_KERNEL_NOT_IN_SET: return "a kernel fits no pattern of the set";
    case PCONV_ERR_RANGE: return "non-finite weight or fp16 overflow";
    case PCONV_ERR_UNSUPPORTED: return "unsupported storage type or flag";
    case PCONV_ERR_ALIGN: return "misaligned device pointer";
    case PCONV_ERR_ALLOC: return "allocation failed";
    case PCONV_ERR_CUDA: return "CUDA error";
    case PCONV_ERR_DEVICE_TIMEOUT: return "a kernel abandoned a bounded wait";
    case PCONV_ERR_WORKSPACE: return "shape needs more scratch memory than this entry point has";
  }
  return "unknown status";
}

// What a caller pinned for the tiled kernel: rows per lane (0 = the planner chooses) and the
// bulk-copy staging.
static int rows_mode(unsigned flags) {
  return ((flags & PCONV_ROWS8) ? 8 : (flags & PCONV_ROWS4) ? 4 : 0) | ((flags & PCONV_STAGE_BULK) ? pconv::kPinBulk : 0);
}

// Scratch a forward of this shape may use, whichever kernel takes it.  rmode: the rows per lane
// the caller pins for the tiled kernel (0 = the planner's choice), -1 = whatever it may pin.
static size_t workspace_need(const pconv::DeviceLayer& L, int n, int h_in, int w_in, int rmode) {
  size_t need = tensor_workspace_bytes(L, n, h_in, w_in);
  for (int r = 0; r <= 8; r += 4)
    for (int bulk = 0; bulk <= pconv::kPinBulk; bulk += pconv::kPinBulk) {
      if (rmode >= 0 && (r | bulk) != rmode) continue;
      const size_t a = tiled_workspace_bytes(L, n, h_in, w_in, r | bulk);
      if (a > need) need = a;
    }
  return need;
}

extern "C" pconv_status pconv_workspace_bytes(const pconv_handle* h, int n, int h_in, int w_in,
                                              size_t* bytes) {
  if (!h || !bytes) return PCONV_ERR_NULL;
  if (n < 0 || h_in <= 0 || w_in <= 0) return PCONV_ERR_SHAPE;
  // (whichever kernel a forward of this shape may take)
  *bytes = 0;
  if (n > 0) {
    *bytes = workspace_need(h->d, n, h_in, w_in, -1);
  }
  return PCONV_OK;
}

extern "C" pconv_status pconv_plan(const pconv_handle* h, int n, int h_in, int w_in, unsigned flags,
                                   int with_workspace, pconv_plan_t* plan) {
  if (!h || !plan) return PCONV_ERR_NULL;
  if (n <= 0 || h_in <= 0 || w_in <= 0) return PCONV_ERR_SHAPE;
  std::memset(plan, 0, sizeof(*plan));
  if (!tiled_plan(h->d, n, h_in, w_in, (flags & PCONV_KERNEL_GENERIC_TAPS) != 0, with_workspace != 0,
                  rows_mode(flags), plan))
    return PCONV_ERR_UNSUPPORTED;
  plan->tensor_path = tensor_preferred(h->d, n, h_in, w_in) ? 1 : 0;
  return PCONV_OK;
}

extern "C" pconv_status pconv_plan_shape(int c_out, int c_in, long long kept_kernels, int stride,
                                         int storage, int n_patterns_canonical, int n, int h_in,
                                         int w_in, unsigned flags, int with_workspace,
                                         pconv_plan_t* plan) {
  if (!plan) return PCONV_ERR_NULL;
  if (c_out <= 0 || c_in <= 0 || kept_kernels < 0 || n <= 0 || h_in <= 0 || w_in <= 0) return PCONV_ERR_SHAPE;
  if ((stride != 1 && stride != 2) || (storage != PCONV_F32 && storage != PCONV_F16)) return PCONV_ERR_UNSUPPORTED;
  pconv::DeviceLayer L;
  std::memset(&L, 0, sizeof(L));
  L.c_out = c_out;
  L.c_in = c_in;
  L.stride = stride;
  L.storage = storage;
  L.n_groups = (c_out + pconv::kGroup - 1) / pconv::kGroup;
  L.n_chunks = (c_in + pconv::kChunk - 1) / pconv::kChunk;
  L.n_kept = kept_kernels;
  L.wide_codes = n_patterns_canonical ? 0 : 1;
  L.codes_s = reinterpret_cast<const uint8_t*>(&L);   // only tested for presence by the planner
  std::memset(plan, 0, sizeof(*plan));
  if (!tiled_plan(L, n, h_in, w_in, (flags & PCONV_KERNEL_GENERIC_TAPS) != 0, with_workspace != 0,
                  rows_mode(flags), plan))
    return PCONV_ERR_UNSUPPORTED;
  return PCONV_OK;
}

extern "C" pconv_status pconv_forward(const pconv_handle* h, const void* x, const float* bias,
                                      void* y, int n, int h_in, int w_in, unsigned flags,
                                      void* stream_v) {
  return pconv_forward_ws(h, x, bias, y, n, h_in, w_in, flags, nullptr, 0, stream_v);
}

// The forward behind every entry point.  `status_dev` != nullptr makes the kernels record an
// abandoned wait there instead of in the handle's own status block (a stack collects the status
// of all its layers in one word).
static pconv_status forward_impl(const pconv_handle* h, const void* x, const float* bias, void* y,
                                 int n, int h_in, int w_in, unsigned flags, void* ws,
                                 size_t ws_bytes, void* stream_v, int* status_dev);

extern "C" pconv_status pconv_forward_ws(const pconv_handle* h, const void* x, const float* bias,
                                         void* y, int n, int h_in, int w_in, unsigned flags,
                                         void* ws, size_t ws_bytes, void* stream_v) {
  return forward_impl(h, x, bias, y, n, h_in, w_in, flags, ws, ws_bytes, stream_v, nullptr);
}

static pconv_status forward_impl(const pconv_handle* h, const void* x, const float* bias, void* y,
                                 int n, int h_in, int w_in, unsigned flags, void* ws,
                                 size_t ws_bytes, void* stream_v, int* status_dev) {
  if (!h || !x || !y) return PCONV_ERR_NULL;
  if (n < 0 || h_in <= 0 || w_in <= 0) return PCONV_ERR_SHAPE;
  const unsigned known =
      PCONV_RELU | PCONV_POOL2X2 | PCONV_REPRODUCIBLE | PCONV_CHAIN | PCONV_KERNEL_SIMPLE | PCONV_KERNEL_TILED |
      PCONV_KERNEL_GENERIC_TAPS | PCONV_KERNEL_TENSOR | PCONV_ROWS4 | PCONV_ROWS8 | PCONV_CLUSTER |
      PCONV_STAGE_BULK;
  if (flags & ~known) return PCONV_ERR_UNSUPPORTED;
  if ((flags & PCONV_ROWS4) && (flags & PCONV_ROWS8)) return PCONV_ERR_UNSUPPORTED;
  const int rmode = rows_mode(flags);
  const bool cluster = (flags & PCONV_CLUSTER) != 0;
  const unsigned sel = flags & (PCONV_KERNEL_SIMPLE | PCONV_KERNEL_TILED | PCONV_KERNEL_GENERIC_TAPS |
                                PCONV_KERNEL_TENSOR);
  if (sel & (sel - 1)) return PCONV_ERR_UNSUPPORTED;  // at most one selection bit
  if (((uintptr_t)x | (uintptr_t)y) & 15u) return PCONV_ERR_ALIGN;
  if (bias && ((uintptr_t)bias & 3u)) return PCONV_ERR_ALIGN;
  if (ws && ((uintptr_t)ws & 255u)) return PCONV_ERR_ALIGN;
  if (n == 0) return PCONV_OK;
  DeviceLayer L = h->d;
  if (status_dev) L.err = status_dev;
  {  // x and y must not overlap
    const size_t es = (L.storage == PCONV_F16) ? 2 : 4;
    const int ho = (h_in - 1) / L.stride + 1, wo = (w_in - 1) / L.stride + 1;
    const char* xb = (const char*)x;
    const char* yb = (const char*)y;
    const bool pooled = flags & PCONV_POOL2X2;
    if (pooled && (ho < 2 || wo < 2)) return PCONV_ERR_SHAPE;
    const size_t xs = (size_t)n * L.c_in * h_in * w_in * es;
    const size_t ys = (size_t)n * L.c_out * (pooled ? ho / 2 : ho) * (pooled ? wo / 2 : wo) * es;
    if (xb < yb + ys && yb < xb + xs) return PCONV_ERR_SHAPE;
  }
  cudaStream_t stream = (cudaStream_t)stream_v;
  const bool relu = flags & PCONV_RELU;
  const bool pool = flags & PCONV_POOL2X2;
  const bool repro = flags & PCONV_REPRODUCIBLE;
  cudaError_t e;
  if (pool && (sel == PCONV_KERNEL_SIMPLE || !tiled_supported(L, n, h_in, w_in)))
    return PCONV_ERR_UNSUPPORTED;  // only the tiled kernels fuse the pool
  if (sel == PCONV_KERNEL_TENSOR) {
    if (pool || !tensor_supported(L, n, h_in, w_in)) return PCONV_ERR_UNSUPPORTED;
    e = launch_tensor(L, x, bias, y, n, h_in, w_in, relu, repro ? nullptr : ws, ws_bytes, stream);
  } else if (sel == 0 && !pool && tensor_preferred(L, n, h_in, w_in)) {
    e = launch_tensor(L, x, bias, y, n, h_in, w_in, relu, repro ? nullptr : ws, ws_bytes, stream);
  } else if (sel == PCONV_KERNEL_SIMPLE) {
    e = launch_simple(L, x, bias, y, n, h_in, w_in, relu, stream);
  } else if (sel == PCONV_KERNEL_TILED || sel == PCONV_KERNEL_GENERIC_TAPS) {
    if (!tiled_supported(L, n, h_in, w_in)) return PCONV_ERR_UNSUPPORTED;
    const bool generic = (sel == PCONV_KERNEL_GENERIC_TAPS);
    if ((rmode & pconv::kPinRowsMask) == 8 && (generic || L.wide_codes || !L.codes_s)) return PCONV_ERR_UNSUPPORTED;
    e = launch_tiled(L, x, bias, y, n, h_in, w_in, relu, pool, repro, generic, rmode, cluster, ws, ws_bytes, stream);
  } else if (tiled_supported(L, n, h_in, w_in)) {
    if ((rmode & pconv::kPinRowsMask) == 8 && (L.wide_codes || !L.codes_s)) return PCONV_ERR_UNSUPPORTED;
    e = launch_tiled(L, x, bias, y, n, h_in, w_in, relu, pool, repro, false, rmode, cluster, ws, ws_bytes, stream);
  } else {
    e = launch_simple(L, x, bias, y, n, h_in, w_in, relu, stream);
  }
  if (e != cudaSuccess) return PCONV_ERR_CUDA;
  return PCONV_OK;
}

// ---- the entry point that allocates nothing --------------------------------------------------------
// Scratch for callers that cannot call cudaMalloc: a fixed array in this library's device image.
// In host code the name below is only a handle for the runtime, not a device address; the address
// every kernel needs is fetched per device with cudaGetSymbolAddress and cached.
static __device__ __align__(256) unsigned char g_static_ws[PCONV_STATIC_WS_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_ws_mutex;
void* g_static_ws_ptr[kMaxDevices] = {nullptr};

// Device address of g_static_ws on the current device (looked up once per device), or nullptr.
void* static_ws_address() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return nullptr;
  }
  std::lock_guard<std::mutex> lock(g_static_ws_mutex);
  if (!g_static_ws_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    g_static_ws_ptr[dev] = p;
  }
  return g_static_ws_ptr[dev];
}
}  // namespace

extern "C" pconv_status pconv_forward_static_ws(const pconv_handle* h, const void* x,
                                                const float* bias, void* y, int n, int h_in,
                                                int w_in, unsigned flags, void* stream_v) {
  if (!h || !x || !y) return PCONV_ERR_NULL;
  if (n < 0 || h_in <= 0 || w_in <= 0) return PCONV_ERR_SHAPE;
  if (n == 0) return PCONV_OK;
  const size_t need = workspace_need(h->d, n, h_in, w_in, rows_mode(flags));
  if (need > (size_t)PCONV_STATIC_WS_BYTES) return PCONV_ERR_WORKSPACE;
  if (need == 0)  // this shape is never split: no scratch involved
    return pconv_forward_ws(h, x, bias, y, n, h_in, w_in, flags, nullptr, 0, stream_v);
  void* ws = static_ws_address();
  if (!ws) return PCONV_ERR_CUDA;
  // the array keeps whatever the last call left (normally zeros, but not after an aborted launch)
  if (cudaMemsetAsync(ws, 0, need, (cudaStream_t)stream_v) != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  return pconv_forward_ws(h, x, bias, y, n, h_in, w_in, flags, ws, need, stream_v);
}

extern "C" pconv_status pconv_maxpool2x2(const void* x, void* y, int n, int c, int h, int w,
                                         int storage, void* stream) {
  if (!x || !y) return PCONV_ERR_NULL;
  if (n < 0 || c <= 0 || h < 2 || w < 2) return PCONV_ERR_SHAPE;
  if (storage != PCONV_F32 && storage != PCONV_F16) return PCONV_ERR_UNSUPPORTED;
  if (launch_maxpool(x, y, n, c, h, w, storage, (cudaStream_t)stream) != cudaSuccess)
    return PCONV_ERR_CUDA;
  return PCONV_OK;
}

extern "C" pconv_status pconv_device_status(const pconv_handle* h, int* where) {
  if (!h) return PCONV_ERR_NULL;
  int v = 0;
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(&v, h->d.err, 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  if (v) {
    if (where) *where = v;
    return PCONV_ERR_DEVICE_TIMEOUT;
  }
  return PCONV_OK;
}

#ifdef PCONV_DEV
extern "C" pconv_status pconv_trace_read(const pconv_handle* h, unsigned long long* words, int n_words) {
  if (!h || !words) return PCONV_ERR_NULL;
  if (n_words < 0 || n_words > pconv::kTraceWords) return PCONV_ERR_SHAPE;
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(words, pconv::trace_words(h->d), (size_t)n_words * 8, cudaMemcpyDeviceToHost) !=
          cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  return PCONV_OK;
}

extern "C" pconv_status pconv_dev_withhold(int chunk, unsigned spin_limit) {
  if (pconv::dev_set_withhold(chunk, spin_limit) != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  return PCONV_OK;
}

extern "C" pconv_status pconv_dev_clear_status(const pconv_handle* h) {
  if (!h) return PCONV_ERR_NULL;
  if (cudaDeviceSynchronize() != cudaSuccess || cudaMemset(h->d.err, 0, 4) != cudaSuccess ||
      cudaDeviceSynchronize() != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  return PCONV_OK;
}
#endif

// ---- stacks ---------------------------------------------------------------------------------------

struct pconv_stack {
  int n_layers, n, h, w, storage;
  unsigned flags;
  const pconv_handle** layers;
  const float** bias;
  unsigned char* pool;
  int out_c, out_h, out_w;
  size_t in_bytes, out_bytes, act_bytes;
  void* act[2];   // ping-pong activations
  void* io[2];    // device input / output used by the host entry point
  void* ws;       // channel-split workspace shared by the layers (kept zeroed between launches)
  size_t ws_bytes;
  int* status_dev;   // status block of every launch of this stack (word 0: first abandoned wait)
  int* status_host;  // pinned copy of word 0, read back by the host entry point
  // a captured forward (pconv_stack_capture) and the buffers it was captured for
  cudaGraphExec_t graph_exec;
  const void* graph_x;
  void* graph_y;
  cudaGraphExec_t host_exec;   // the host entry point's own graph (io[0] -> io[1])
  bool host_graph_failed;      // its capture was tried and is not possible on the stream given
  // chains: runs of consecutive layers that one persistent kernel executes (batch-1 stacks, where
  // every layer is a single wave of CTAs and launch, set-up and first-data latencies dominate)
  struct Chain {
    int begin, end;            // layers [begin, end)
    void* table_host;          // the chain kernel's per-layer table, and its device copy
    void* table_dev;
    std::vector<void*> mid;    // outputs of the chain's inner layers (never reused inside the launch)
  };
  std::vector<Chain>* chains;
  unsigned int* sync_dev;      // the chain kernel's two counters (zero between launches)
};

extern "C" void pconv_stack_free(pconv_stack* s) {
  if (!s) return;
  for (int i = 0; i < 2; ++i) {
    if (s->act[i]) cudaFree(s->act[i]);
    if (s->io[i]) cudaFree(s->io[i]);
  }
  if (s->ws) cudaFree(s->ws);
  if (s->chains) {
    for (pconv_stack::Chain& c : *s->chains) {
      std::free(c.table_host);
      if (c.table_dev) cudaFree(c.table_dev);
      for (void* m : c.mid)
        if (m) cudaFree(m);
    }
    delete s->chains;
  }
  if (s->sync_dev) cudaFree(s->sync_dev);
  if (s->status_dev) cudaFree(s->status_dev);
  if (s->status_host) cudaFreeHost(s->status_host);
  if (s->graph_exec) cudaGraphExecDestroy(s->graph_exec);
  if (s->host_exec) cudaGraphExecDestroy(s->host_exec);
  delete[] s->layers;
  delete[] s->bias;
  delete[] s->pool;
  delete s;
}

// Finds the runs of consecutive layers that a chain kernel can execute, builds their tables and
// inner buffers, and allocates the workspace (the layers' and the chains' largest need).
static bool build_chains(pconv_stack* s) {
  s->chains = new (std::nothrow) std::vector<pconv_stack::Chain>();
  if (!s->chains) return false;
  const unsigned sel_bits = PCONV_KERNEL_SIMPLE | PCONV_KERNEL_TILED | PCONV_KERNEL_GENERIC_TAPS | PCONV_KERNEL_TENSOR;
  const size_t es = (s->storage == PCONV_F16) ? 2 : 4;
  if ((s->flags & PCONV_CHAIN) && !(s->flags & (sel_bits | PCONV_REPRODUCIBLE))) {
    // shapes of every layer's input and output
    std::vector<int> hi(s->n_layers), wi(s->n_layers);
    int ch = s->h, cw = s->w;
    std::vector<bool> ok(s->n_layers, false);
    for (int i = 0; i < s->n_layers; ++i) {
      const pconv::DeviceLayer& L = s->layers[i]->d;
      hi[i] = ch;
      wi[i] = cw;
      ok[i] = pconv::chain_layer_ok(L, s->n, ch, cw, s->pool[i] != 0, nullptr) &&
              !pconv::tensor_preferred(L, s->n, ch, cw);
      ch = (ch - 1) / L.stride + 1;
      cw = (cw - 1) / L.stride + 1;
      if (s->pool[i]) {
        ch /= 2;
        cw /= 2;
      }
    }
    for (int b = 0; b < s->n_layers;) {
      int e = b;
      while (e < s->n_layers && ok[e] && e - b < 16) ++e;
      if (e - b < 2) {
        b = e > b ? e : b + 1;
        continue;
      }
      pconv_stack::Chain c;
      c.begin = b;
      c.end = e;
      c.table_dev = nullptr;
      c.table_host = std::malloc(pconv::chain_table_bytes(e - b));
      if (!c.table_host) return false;
      s->chains->push_back(c);
      pconv_stack::Chain& cc = s->chains->back();
      const void* x = nullptr;     // the chain's input: given at launch
      for (int i = b; i < e; ++i) {
        const pconv::DeviceLayer& L = s->layers[i]->d;
        int ho = hi[i], wo = wi[i];
        if (s->pool[i]) {
          ho /= 2;
          wo /= 2;
        }
        void* y = nullptr;         // the chain's output: given at launch
        if (i + 1 < e) {
          if (cudaMalloc(&y, (size_t)s->n * L.c_out * ho * wo * es) != cudaSuccess) return false;
          cc.mid.push_back(y);
        }
        if (!pconv::chain_fill(cc.table_host, i - b, L, x, s->bias[i], y, s->n, hi[i], wi[i],
                               (s->flags & PCONV_RELU) != 0, s->pool[i] != 0, s->status_dev))
          return false;
        x = y;
      }
      const size_t tb = pconv::chain_table_bytes(e - b);
      if (cudaMalloc(&cc.table_dev, tb) != cudaSuccess ||
          cudaMemcpy(cc.table_dev, cc.table_host, tb, cudaMemcpyHostToDevice) != cudaSuccess)
        return false;
      const size_t wsb = pconv::chain_workspace_bytes(cc.table_host, e - b);
      if (wsb > s->ws_bytes) s->ws_bytes = wsb;
      b = e;
    }
  }
  if (s->ws_bytes) {
    if (cudaMalloc(&s->ws, s->ws_bytes) != cudaSuccess || cudaMemset(s->ws, 0, s->ws_bytes) != cudaSuccess)
      return false;
  }
  if (!s->chains->empty()) {
    if (cudaMalloc((void**)&s->sync_dev, 256) != cudaSuccess || cudaMemset(s->sync_dev, 0, 256) != cudaSuccess)
      return false;
  }
  return true;
}

extern "C" pconv_status pconv_stack_create(const pconv_handle* const* layers,
                                           const float* const* bias_dev,
                                           const unsigned char* pool_after, int n_layers, int n,
                                           int h, int w, unsigned flags, pconv_stack** out) {
  if (!layers || !out) return PCONV_ERR_NULL;
  if (n_layers <= 0 || n <= 0 || h <= 0 || w <= 0) return PCONV_ERR_SHAPE;
  for (int i = 0; i < n_layers; ++i)
    if (!layers[i]) return PCONV_ERR_NULL;
  pconv_stack* s = new (std::nothrow) pconv_stack();
  if (!s) return PCONV_ERR_ALLOC;
  std::memset(s, 0, sizeof(*s));
  s->layers = new (std::nothrow) const pconv_handle*[n_layers];
  s->bias = new (std::nothrow) const float*[n_layers];
  s->pool = new (std::nothrow) unsigned char[n_layers];
  if (!s->layers || !s->bias || !s->pool) {
    pconv_stack_free(s);
    return PCONV_ERR_ALLOC;
  }
  s->n_layers = n_layers;
  s->n = n;
  s->h = h;
  s->w = w;
  s->flags = flags;
  s->storage = layers[0]->d.storage;
  const size_t es = (s->storage == PCONV_F16) ? 2 : 4;
  int ch = h, cw = w, cc = layers[0]->d.c_in;
  size_t max_act = 0;
  s->in_bytes = (size_t)n * cc * h * w * es;
  for (int i = 0; i < n_layers; ++i) {
    const pconv::DeviceLayer& L = layers[i]->d;
    s->layers[i] = layers[i];
    s->bias[i] = bias_dev ? bias_dev[i] : nullptr;
    s->pool[i] = pool_after ? pool_after[i] : 0;
    if (L.storage != s->storage || L.c_in != cc) {
      pconv_stack_free(s);
      return PCONV_ERR_SHAPE;
    }
    const size_t wsb = tiled_workspace_bytes(L, n, ch, cw, rows_mode(flags)), wsd = tensor_workspace_bytes(L, n, ch, cw);
    if (wsb > s->ws_bytes) s->ws_bytes = wsb;
    if (wsd > s->ws_bytes) s->ws_bytes = wsd;
    ch = (ch - 1) / L.stride + 1;
    cw = (cw - 1) / L.stride + 1;
    cc = L.c_out;
    const size_t bytes = (size_t)n * cc * ch * cw * es;
    if (bytes > max_act) max_act = bytes;
    if (s->pool[i]) {
      if (ch < 2 || cw < 2) {
        pconv_stack_free(s);
        return PCONV_ERR_SHAPE;
      }
      ch /= 2;
      cw /= 2;
    }
  }
  s->out_c = cc;
  s->out_h = ch;
  s->out_w = cw;
  s->out_bytes = (size_t)n * cc * ch * cw * es;
  s->act_bytes = max_act;
  cudaError_t e = cudaMalloc(&s->act[0], max_act);
  if (e == cudaSuccess) e = cudaMalloc(&s->act[1], max_act);
  if (e == cudaSuccess) e = cudaMalloc(&s->io[0], s->in_bytes);
  if (e == cudaSuccess) e = cudaMalloc(&s->io[1], s->out_bytes);
  if (e == cudaSuccess) e = cudaMalloc(&s->status_dev, pconv::kStatusBlockBytes);
  if (e == cudaSuccess) e = cudaMemset(s->status_dev, 0, pconv::kStatusBlockBytes);
  if (e == cudaSuccess) e = cudaMallocHost(&s->status_host, sizeof(int));
  if (e == cudaSuccess) *s->status_host = 0;
  if (e == cudaSuccess && !build_chains(s)) e = cudaErrorMemoryAllocation;
  if (e != cudaSuccess) {
    cudaGetLastError();
    pconv_stack_free(s);
    return PCONV_ERR_ALLOC;
  }
  *out = s;
  return PCONV_OK;
}

extern "C" pconv_status pconv_stack_out_shape(const pconv_stack* s, int* n, int* c, int* h,
                                              int* w) {
  if (!s) return PCONV_ERR_NULL;
  if (n) *n = s->n;
  if (c) *c = s->out_c;
  if (h) *h = s->out_h;
  if (w) *w = s->out_w;
  return PCONV_OK;
}

extern "C" pconv_status pconv_stack_launches(const pconv_stack* s, int* launches) {
  if (!s || !launches) return PCONV_ERR_NULL;
  int n = 0, ch = s->h, cw = s->w;
  for (int i = 0; i < s->n_layers; ++i) {
    const pconv_stack::Chain* chain = nullptr;
    if (s->chains)
      for (const pconv_stack::Chain& c : *s->chains)
        if (c.begin == i) chain = &c;
    const int last = chain ? chain->end : i + 1;
    ++n;
    for (int k = i; k < last; ++k) {
      const pconv::DeviceLayer& L = s->layers[k]->d;
      const unsigned sel_bits = PCONV_KERNEL_SIMPLE | PCONV_KERNEL_TILED | PCONV_KERNEL_GENERIC_TAPS | PCONV_KERNEL_TENSOR;
      const bool tensor = (s->flags & PCONV_KERNEL_TENSOR) ||
                          (!(s->flags & sel_bits) && pconv::tensor_preferred(L, s->n, ch, cw));
      const bool fuse = s->pool[k] && !(s->flags & PCONV_KERNEL_SIMPLE) && !tensor &&
                        pconv::tiled_supported(L, s->n, ch, cw);
      if (!chain && s->pool[k] && !fuse) ++n;      // a max-pool kernel of its own
      ch = (ch - 1) / L.stride + 1;
      cw = (cw - 1) / L.stride + 1;
      if (s->pool[k]) {
        ch /= 2;
        cw /= 2;
      }
    }
    i = last - 1;
  }
  *launches = n;
  return PCONV_OK;
}

extern "C" pconv_status pconv_stack_forward(pconv_stack* s, const void* x, void* y, void* stream) {
  if (!s || !x || !y) return PCONV_ERR_NULL;
  const void* cur = x;
  int ch = s->h, cw = s->w, which = 0;
  for (int i = 0; i < s->n_layers; ++i) {
    const pconv_stack::Chain* chain = nullptr;
    if (s->chains)
      for (const pconv_stack::Chain& c : *s->chains)
        if (c.begin == i) chain = &c;
    if (chain) {   // layers [begin, end) in one persistent launch
      void* dst = (chain->end == s->n_layers) ? y : s->act[which];
      if (pconv::launch_chain(chain->table_dev, chain->table_host, chain->end - chain->begin, cur, dst, s->ws,
                              s->ws_bytes, s->sync_dev, (cudaStream_t)stream) != cudaSuccess) {
        cudaGetLastError();
        return PCONV_ERR_CUDA;
      }
      for (int k = chain->begin; k < chain->end; ++k) {
        const int st = s->layers[k]->d.stride;
        ch = (ch - 1) / st + 1;
        cw = (cw - 1) / st + 1;
        if (s->pool[k]) {
          ch /= 2;
          cw /= 2;
        }
      }
      cur = dst;
      which ^= 1;
      i = chain->end - 1;
      continue;
    }
    const pconv::DeviceLayer& L = s->layers[i]->d;
    // a pool that follows the layer is fused into the layer's epilogue when a tiled kernel runs it
    // (not when the layer takes the dense tensor-core kernel, which has no pooled epilogue: the
    // plain max-pool kernel follows it)
    const unsigned sel_bits = PCONV_KERNEL_SIMPLE | PCONV_KERNEL_TILED | PCONV_KERNEL_GENERIC_TAPS | PCONV_KERNEL_TENSOR;
    const bool tensor = (s->flags & PCONV_KERNEL_TENSOR) ||
                        (!(s->flags & sel_bits) && pconv::tensor_preferred(L, s->n, ch, cw));
    const bool fuse = s->pool[i] && !(s->flags & PCONV_KERNEL_SIMPLE) && !tensor &&
                      pconv::tiled_supported(L, s->n, ch, cw);
    const bool last_op = (i == s->n_layers - 1) && (!s->pool[i] || fuse);
    void* dst = last_op ? y : s->act[which];
    pconv_status st = forward_impl(s->layers[i], cur, s->bias[i], dst, s->n, ch, cw,
                                   s->flags | (fuse ? PCONV_POOL2X2 : 0u), s->ws, s->ws_bytes, stream,
                                   s->status_dev);
    if (st != PCONV_OK) return st;
    ch = (ch - 1) / L.stride + 1;
    cw = (cw - 1) / L.stride + 1;
    cur = dst;
    which ^= 1;
    if (fuse) {
      ch /= 2;
      cw /= 2;
    } else if (s->pool[i]) {
      void* pd = (i == s->n_layers - 1) ? y : s->act[which];
      st = pconv_maxpool2x2(cur, pd, s->n, L.c_out, ch, cw, s->storage, stream);
      if (st != PCONV_OK) return st;
      ch /= 2;
      cw /= 2;
      cur = pd;
      which ^= 1;
    }
  }
  return PCONV_OK;
}

static pconv_status capture_forward(pconv_stack* s, const void* x, void* y, void* stream_v,
                                    cudaGraphExec_t* exec) {
  cudaStream_t stream = (cudaStream_t)stream_v;
  if (*exec) {
    cudaGraphExecDestroy(*exec);
    *exec = nullptr;
  }
  // the legacy default stream cannot be captured
  if (stream == nullptr || stream == cudaStreamLegacy) return PCONV_ERR_UNSUPPORTED;
  if (cudaStreamBeginCapture(stream, cudaStreamCaptureModeRelaxed) != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  const pconv_status st = pconv_stack_forward(s, x, y, stream_v);
  cudaGraph_t graph = nullptr;
  const cudaError_t e = cudaStreamEndCapture(stream, &graph);
  if (st != PCONV_OK || e != cudaSuccess || !graph) {
    cudaGetLastError();
    if (graph) cudaGraphDestroy(graph);
    return st != PCONV_OK ? st : PCONV_ERR_CUDA;
  }
  const cudaError_t ei = cudaGraphInstantiate(exec, graph, 0);
  cudaGraphDestroy(graph);
  if (ei != cudaSuccess) {
    cudaGetLastError();
    *exec = nullptr;
    return PCONV_ERR_CUDA;
  }
  return PCONV_OK;
}

extern "C" pconv_status pconv_stack_capture(pconv_stack* s, const void* x, void* y, void* stream_v) {
  if (!s || !x || !y) return PCONV_ERR_NULL;
  const pconv_status st = capture_forward(s, x, y, stream_v, &s->graph_exec);
  s->graph_x = st == PCONV_OK ? x : nullptr;
  s->graph_y = st == PCONV_OK ? y : nullptr;
  return st;
}

extern "C" pconv_status pconv_stack_replay(pconv_stack* s, void* stream_v) {
  if (!s) return PCONV_ERR_NULL;
  if (!s->graph_exec) return PCONV_ERR_UNSUPPORTED;
  if (cudaGraphLaunch(s->graph_exec, (cudaStream_t)stream_v) != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  return PCONV_OK;
}

extern "C" pconv_status pconv_stack_forward_host(pconv_stack* s, const void* x_host, void* y_host,
                                                 void* stream_v) {
  if (!s || !x_host || !y_host) return PCONV_ERR_NULL;
  cudaStream_t stream = (cudaStream_t)stream_v;
  // the device part always runs on the stack's own input / output buffers: replay it from a graph
  // captured on first use where the stream allows capture
  if (!s->host_exec && !s->host_graph_failed &&
      capture_forward(s, s->io[0], s->io[1], stream_v, &s->host_exec) != PCONV_OK)
    s->host_graph_failed = true;
  const bool replay = s->host_exec != nullptr;
  if (cudaMemcpyAsync(s->io[0], x_host, s->in_bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  pconv_status st = PCONV_OK;
  if (replay) {
    if (cudaGraphLaunch(s->host_exec, stream) != cudaSuccess) {
      cudaGetLastError();
      st = PCONV_ERR_CUDA;
    }
  } else {
    st = pconv_stack_forward(s, s->io[0], s->io[1], stream_v);
  }
  if (st != PCONV_OK) return st;
  if (cudaMemcpyAsync(y_host, s->io[1], s->out_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaMemcpyAsync(s->status_host, s->status_dev, sizeof(int), cudaMemcpyDeviceToHost, stream) !=
          cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  // a layer that abandoned a bounded wait wrote no valid output: say so instead of handing it on
  return *s->status_host ? PCONV_ERR_DEVICE_TIMEOUT : PCONV_OK;
}

extern "C" pconv_status pconv_stack_status(pconv_stack* s, int* where) {
  if (!s) return PCONV_ERR_NULL;
  int v = 0;
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(&v, s->status_dev, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  if (!v) return PCONV_OK;
  if (where) *where = v;
  // the abandoned launch may have left partial sums and tickets in the workspace
  if (cudaMemset(s->status_dev, 0, sizeof(int)) != cudaSuccess ||
      (s->ws && cudaMemset(s->ws, 0, s->ws_bytes) != cudaSuccess) ||
      (s->sync_dev && cudaMemset(s->sync_dev, 0, 256) != cudaSuccess) ||
      cudaDeviceSynchronize() != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  *s->status_host = 0;
  return PCONV_ERR_DEVICE_TIMEOUT;
}
