// Projection of dense 3x3 kernels onto the PCONV constraint set (pattern per kernel + a keep rate
// over kernels): what turns trained weights into weights that pconv_pack accepts.  Three steps, all
// on the device: per kernel the pattern that retains the largest sum of squares; the k-th largest
// retained sum by a four-pass radix select on the bits of the (non-negative) fp32 sums; masking.
#include <cstring>

#include "pconv_internal.h"

namespace pconv {
namespace {

constexpr int kThreads = 256;

struct PatternSet {
  int n;
  uint16_t mask[PCONV_MAX_PATTERNS];
};

// Retained sum of squares under every pattern; the first maximum wins.  Separate multiply and add
// in ascending tap order: the decision must not depend on how the compiler contracts the sum.
// (Staging a block's 2304 floats through shared memory for coalesced accesses measured slower.)
__global__ void __launch_bounds__(kThreads) score_kernel(const float* __restrict__ w, long long n,
                                                         PatternSet ps, float* __restrict__ best,
                                                         signed char* __restrict__ pid) {
  const long long i = blockIdx.x * (long long)kThreads + threadIdx.x;
  if (i >= n) return;
  float sq[9];
#pragma unroll
  for (int t = 0; t < 9; ++t) {
    const float v = w[i * 9 + t];
    sq[t] = __fmul_rn(v, v);
  }
  float top = -1.f;
  int arg = 0;
  for (int p = 0; p < ps.n; ++p) {
    float s = 0.f;
#pragma unroll
    for (int t = 0; t < 9; ++t)
      if (ps.mask[p] >> t & 1) s = __fadd_rn(s, sq[t]);
    if (s > top) {
      top = s;
      arg = p;
    }
  }
  best[i] = top;
  pid[i] = (signed char)arg;
}

// One pass of the radix select: histogram of byte `shift / 8` of the values whose higher bytes
// equal those of `state->prefix`.
struct SelectState {
  unsigned int prefix;        // the bytes of the threshold found so far (higher bytes)
  unsigned int remaining;     // rank (from the top, 1-based) still to be found inside the prefix
  unsigned int hist[256];
};

__global__ void __launch_bounds__(kThreads) hist_kernel(const float* __restrict__ best, long long n,
                                                        int shift, SelectState* st) {
  __shared__ unsigned int h[256];
  h[threadIdx.x] = 0;
  __syncthreads();
  const unsigned int prefix = st->prefix;
  const unsigned int high_mask = shift == 24 ? 0u : 0xFFFFFFFFu << (shift + 8);
  for (long long i = blockIdx.x * (long long)kThreads + threadIdx.x; i < n;
       i += (long long)gridDim.x * kThreads) {
    const unsigned int b = __float_as_uint(best[i]);
    if ((b & high_mask) == (prefix & high_mask)) atomicAdd(&h[(b >> shift) & 255u], 1u);
  }
  __syncthreads();
  if (h[threadIdx.x]) atomicAdd(&st->hist[threadIdx.x], h[threadIdx.x]);
}

// Picks the byte whose bucket holds the wanted rank, counting from the largest byte down.
__global__ void pick_kernel(int shift, SelectState* st) {
  if (threadIdx.x != 0) return;
  unsigned int remaining = st->remaining;
  int b = 255;
  for (; b > 0; --b) {
    if (st->hist[b] >= remaining) break;
    remaining -= st->hist[b];
  }
  st->prefix |= (unsigned int)b << shift;
  st->remaining = remaining;
  for (int i = 0; i < 256; ++i) st->hist[i] = 0;
}

// `out` may be `w` itself (in-place use), so neither pointer is declared restrict and a thread
// reads its kernel's nine taps before it writes any of them.
__global__ void __launch_bounds__(kThreads) mask_kernel(const float* w, long long n, PatternSet ps,
                                                        const float* __restrict__ best,
                                                        const SelectState* __restrict__ st, int keep_none,
                                                        float* out, signed char* __restrict__ pid) {
  const long long i = blockIdx.x * (long long)kThreads + threadIdx.x;
  if (i >= n) return;
  float v[9];
#pragma unroll
  for (int t = 0; t < 9; ++t) v[t] = w[i * 9 + t];
  const bool kept = !keep_none && __float_as_uint(best[i]) >= st->prefix;   // ties with the k-th stay
  const unsigned int m = kept ? ps.mask[pid[i]] : 0u;
#pragma unroll
  for (int t = 0; t < 9; ++t) out[i * 9 + t] = (m >> t & 1u) ? v[t] : 0.f;
  if (!kept) pid[i] = -1;
}

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace
}  // namespace pconv

using namespace pconv;

extern "C" pconv_status pconv_project_workspace_bytes(long long n_kernels, size_t* bytes) {
  if (!bytes) return PCONV_ERR_NULL;
  if (n_kernels < 0) return PCONV_ERR_SHAPE;
  *bytes = align256((size_t)n_kernels * 4) + align256(sizeof(SelectState));
  return PCONV_OK;
}

extern "C" pconv_status pconv_project(const float* w_dev, long long n_kernels,
                                      const uint16_t* patterns, int n_patterns, double keep,
                                      float* w_out_dev, signed char* pattern_id_dev, void* ws_dev,
                                      size_t ws_bytes, void* stream_v) {
  if (!w_dev || !patterns || !w_out_dev || !pattern_id_dev || !ws_dev) return PCONV_ERR_NULL;
  if (n_kernels < 0 || !(keep >= 0.0 && keep <= 1.0)) return PCONV_ERR_SHAPE;
  if (n_patterns < 1 || n_patterns > PCONV_MAX_PATTERNS) return PCONV_ERR_PATTERN_SET;
  PatternSet ps;
  std::memset(&ps, 0, sizeof(ps));
  ps.n = n_patterns;
  for (int p = 0; p < n_patterns; ++p) {
    if (patterns[p] >= 512 || __builtin_popcount(patterns[p]) != 4) return PCONV_ERR_PATTERN_SET;
    for (int q = 0; q < p; ++q)
      if (patterns[q] == patterns[p]) return PCONV_ERR_PATTERN_SET;
    ps.mask[p] = patterns[p];
  }
  size_t need = 0;
  pconv_project_workspace_bytes(n_kernels, &need);
  if (ws_bytes < need) return PCONV_ERR_WORKSPACE;
  if (((uintptr_t)ws_dev & 255u) || ((uintptr_t)w_dev & 3u) || ((uintptr_t)w_out_dev & 3u)) return PCONV_ERR_ALIGN;
  if (n_kernels == 0) return PCONV_OK;
  cudaStream_t stream = (cudaStream_t)stream_v;
  float* best = (float*)ws_dev;
  SelectState* st = (SelectState*)((char*)ws_dev + align256((size_t)n_kernels * 4));
  long long k = (long long)(keep * (double)n_kernels + 0.5);
  if (k > n_kernels) k = n_kernels;
  const int keep_none = k == 0;
  SelectState init;
  std::memset(&init, 0, sizeof(init));
  init.remaining = (unsigned int)(k > 0 ? k : 1);
  if (n_kernels > 0xFFFFFFFFll) return PCONV_ERR_SHAPE;
  if (cudaMemcpyAsync(st, &init, sizeof(init), cudaMemcpyHostToDevice, stream) != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  const long long blocks = (n_kernels + kThreads - 1) / kThreads;
  if (blocks > 0x7FFFFFFF) return PCONV_ERR_SHAPE;
  score_kernel<<<(unsigned)blocks, kThreads, 0, stream>>>(w_dev, n_kernels, ps, best, pattern_id_dev);
  const long long hist_max = (long long)device_sm_count() * 8;
  const unsigned hist_blocks = (unsigned)(blocks < hist_max ? blocks : hist_max);
  for (int shift = 24; shift >= 0; shift -= 8) {
    hist_kernel<<<hist_blocks, kThreads, 0, stream>>>(best, n_kernels, shift, st);
    pick_kernel<<<1, 32, 0, stream>>>(shift, st);
  }
  mask_kernel<<<(unsigned)blocks, kThreads, 0, stream>>>(w_dev, n_kernels, ps, best, st, keep_none,
                                                         w_out_dev, pattern_id_dev);
  if (cudaGetLastError() != cudaSuccess) return PCONV_ERR_CUDA;
  return PCONV_OK;
}
