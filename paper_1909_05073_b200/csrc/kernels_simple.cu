// Plain kernels: a one-thread-per-output pattern-sparse convolution that walks the per-filter
// kernel list (kept as the in-library cross-check and as the path for shapes the tiled kernel
// does not take), and the 2x2 max-pool between VGG blocks.
#include <cuda_fp16.h>

#include "pconv_internal.h"

namespace pconv {
namespace {

template <typename T>
__device__ __forceinline__ float ldx(const T* p);
template <>
__device__ __forceinline__ float ldx<float>(const float* p) { return __ldg(p); }
template <>
__device__ __forceinline__ float ldx<__half>(const __half* p) { return __half2float(__ldg(p)); }
__device__ __forceinline__ void stx(float* p, float v) { *p = v; }
__device__ __forceinline__ void stx(__half* p, float v) { *p = __float2half_rn(v); }

template <typename T>
__global__ void __launch_bounds__(256) simple_kernel(DeviceLayer L, const T* __restrict__ x,
                                                     const float* __restrict__ bias,
                                                     T* __restrict__ y, int h, int w, int h_out,
                                                     int w_out, int relu) {
  const int o = blockIdx.y;
  const int n = blockIdx.z;
  const int pix = blockIdx.x * blockDim.x + threadIdx.x;
  if (pix >= h_out * w_out) return;
  const int i = pix / w_out, j = pix - i * w_out;
  const int r0 = i * L.stride - 1, q0 = j * L.stride - 1;
  const T* xn = x + (size_t)n * L.c_in * h * w;
  float acc = 0.f;
  const int beg = L.row_ptr[o], end = L.row_ptr[o + 1];
  for (int k = beg; k < end; ++k) {
    const uint32_t idx = __ldg(L.csr_idx + k);
    const int c = idx & 0xFFFF;
    const unsigned mask = idx >> 16;
    const float4 wv = __ldg(reinterpret_cast<const float4*>(L.csr_val) + k);
    const float wk[4] = {wv.x, wv.y, wv.z, wv.w};
    const T* xc = xn + (size_t)c * h * w;
    int s = 0;
#pragma unroll
    for (int t = 0; t < 9; ++t) {
      if (mask >> t & 1) {
        const int r = r0 + t / 3, q = q0 + t % 3;
        if (r >= 0 && r < h && q >= 0 && q < w) acc = fmaf(wk[s], ldx(xc + (size_t)r * w + q), acc);
        ++s;
      }
    }
  }
  if (bias) acc += __ldg(bias + o);
  if (relu) acc = fmaxf(acc, 0.f);
  stx(y + (((size_t)n * L.c_out + o) * h_out + i) * w_out + j, acc);
}

template <typename T>
__global__ void __launch_bounds__(256) maxpool_kernel(const T* __restrict__ x, T* __restrict__ y,
                                                      long long total, int h, int w, int h_out,
                                                      int w_out) {
  // started early under programmatic stream serialisation: let the next kernel do the same, and
  // wait for the producer of x
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < total;
       e += (long long)gridDim.x * blockDim.x) {
    const int j = (int)(e % w_out);
    const long long t = e / w_out;
    const int i = (int)(t % h_out);
    const long long plane = t / h_out;
    const T* p = x + ((size_t)plane * h + 2 * i) * w + 2 * j;
    const float a = ldx(p), b = ldx(p + 1), c = ldx(p + w), d = ldx(p + w + 1);
    stx(y + e, fmaxf(fmaxf(a, b), fmaxf(c, d)));
  }
}

}  // namespace

cudaError_t launch_simple(const DeviceLayer& L, const void* x, const float* bias, void* y, int n,
                          int h, int w, bool relu, cudaStream_t stream) {
  const int h_out = (h - 1) / L.stride + 1, w_out = (w - 1) / L.stride + 1;
  // grid.y / grid.z are limited to 65535: walk the batch in slices if needed
  const int zmax = 65535;
  if (L.c_out > 65535) return cudaErrorInvalidValue;
  for (int n0 = 0; n0 < n; n0 += zmax) {
    const int nb = (n - n0 < zmax) ? (n - n0) : zmax;
    dim3 grid((h_out * w_out + 255) / 256, L.c_out, nb);
    if (L.storage == PCONV_F16) {
      const __half* xs = (const __half*)x + (size_t)n0 * L.c_in * h * w;
      __half* ys = (__half*)y + (size_t)n0 * L.c_out * h_out * w_out;
      simple_kernel<__half><<<grid, 256, 0, stream>>>(L, xs, bias, ys, h, w, h_out, w_out, relu);
    } else {
      const float* xs = (const float*)x + (size_t)n0 * L.c_in * h * w;
      float* ys = (float*)y + (size_t)n0 * L.c_out * h_out * w_out;
      simple_kernel<float><<<grid, 256, 0, stream>>>(L, xs, bias, ys, h, w, h_out, w_out, relu);
    }
  }
  return cudaGetLastError();
}

cudaError_t launch_maxpool(const void* x, void* y, int n, int c, int h, int w, int storage,
                           cudaStream_t stream) {
  const int h_out = h / 2, w_out = w / 2;
  const long long total = (long long)n * c * h_out * w_out;
  if (total == 0) return cudaSuccess;
  long long blocks = (total + 255) / 256;
  const long long max_blocks = (long long)device_sm_count() * 16;
  if (blocks > max_blocks) blocks = max_blocks;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks, 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (storage == PCONV_F16)
    return cudaLaunchKernelEx(&cfg, maxpool_kernel<__half>, (const __half*)x, (__half*)y, total, h, w,
                              h_out, w_out);
  return cudaLaunchKernelEx(&cfg, maxpool_kernel<float>, (const float*)x, (float*)y, total, h, w, h_out,
                            w_out);
}

}  // namespace pconv
