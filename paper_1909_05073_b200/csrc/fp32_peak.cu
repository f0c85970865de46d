// Stand-alone measurement of the FP32 multiply-add peak that the tiled kernel's roofline is
// quoted against, and of what an FMA costs the instruction scheduler:
//   * scalar fma.rn.f32 and packed fma.rn.f32x2 from registers only (the peak);
//   * the same with K independent integer instructions (lop3 on eight separate registers) issued
//     per FMA instruction, K = 1/4 .. 2: if the packed FMA takes one issue slot and two pipe
//     cycles, one other instruction per packed FMA is free; if it blocks the issue port for two
//     cycles, every other instruction adds its full cycle.
// Build and run (build.py: build_peak()):  nvcc -arch=sm_100a -O3 -o fp32_peak fp32_peak.cu && ./fp32_peak
// It is a measuring tool, not part of libpconv.so.
#include <cuda_runtime.h>

#include <cstdio>

typedef unsigned long long u64;

// MODE 0: scalar FFMA, 1: FFMA2.  OTHER_NUM / OTHER_DEN integer instructions per FMA instruction.
template <int MODE, int OTHER_NUM, int OTHER_DEN>
__global__ void __launch_bounds__(1024) peak_kernel(float* out, int iters, float a, float b,
                                                    long long* cycles) {
  unsigned x[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = threadIdx.x * (i + 3);
  float acc[32];
  u64 acc2[16];
#pragma unroll
  for (int i = 0; i < 32; ++i) acc[i] = (float)(i + threadIdx.x);
#pragma unroll
  for (int i = 0; i < 16; ++i)
    acc2[i] = ((u64)__float_as_uint(i + 1.f) << 32) | __float_as_uint((float)threadIdx.x);
  const u64 aa = ((u64)__float_as_uint(a) << 32) | __float_as_uint(a);
  const u64 bb = ((u64)__float_as_uint(b) << 32) | __float_as_uint(b);
  const long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
    int owed = 0, xi = 0;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
#pragma unroll
      for (int i = 0; i < (MODE == 0 ? 32 : 16); ++i) {
        if (MODE == 0) asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(acc[i]) : "f"(a), "f"(b));
        else asm volatile("fma.rn.f32x2 %0, %0, %1, %2;" : "+l"(acc2[i]) : "l"(aa), "l"(bb));
        owed += OTHER_NUM;
        while (owed >= OTHER_DEN) {   // resolved at compile time (everything is unrolled)
          asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[xi & 7]) : "r"(it), "r"(i + r));
          owed -= OTHER_DEN;
          ++xi;
        }
      }
    }
  }
  const long long t1 = clock64();
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) s += (float)x[i];
  if (MODE == 0) {
#pragma unroll
    for (int i = 0; i < 32; ++i) s += acc[i];
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i)
      s += __uint_as_float((unsigned)acc2[i]) + __uint_as_float((unsigned)(acc2[i] >> 32));
  }
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
  if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
}

template <int MODE, int NUM, int DEN>
void run(const char* name, int block, int sms) {
  const int iters = 4000;
  float* out;
  long long* cyc;
  cudaMalloc(&out, sizeof(float) * sms * block);
  cudaMalloc(&cyc, sizeof(long long) * sms);
  peak_kernel<MODE, NUM, DEN><<<sms, block>>>(out, 10, 0.999f, 0.001f, cyc);
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  float best = 1e9f;
  for (int rep = 0; rep < 3; ++rep) {
    cudaEventRecord(e0);
    peak_kernel<MODE, NUM, DEN><<<sms, block>>>(out, iters, 0.999f, 0.001f, cyc);
    cudaEventRecord(e1);
    cudaEventSynchronize(e1);
    float ms;
    cudaEventElapsedTime(&ms, e0, e1);
    if (ms < best) best = ms;
  }
  long long c0 = 0;
  cudaMemcpy(&c0, cyc, 8, cudaMemcpyDeviceToHost);
  const double fma = (double)sms * block * iters * 4 * 32;   // lane-level multiply-adds
  const double inst_per_warp = (double)iters * 4 * (MODE == 0 ? 32 : 16) * (1.0 + (double)NUM / DEN);
  const double warps_per_sched = block / 128.0;
  printf("%-34s block %4d  %7.3f ms  %6.2f TFLOP/s  %6.1f FMA/clk/SM  %5.3f issue slots used per cycle  (%s)\n",
         name, block, best, 2 * fma / (best * 1e-3) / 1e12, (double)block * iters * 4 * 32 / (double)c0,
         inst_per_warp * warps_per_sched / (double)c0, cudaGetErrorString(cudaGetLastError()));
  cudaFree(out);
  cudaFree(cyc);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
}

int main() {
  cudaDeviceProp p;
  if (cudaGetDeviceProperties(&p, 0) != cudaSuccess) {
    printf("no CUDA device\n");
    return 1;
  }
  const int sms = p.multiProcessorCount;
  printf("%s, %d SMs, max SM clock %d kHz; nominal FP32 peak %.2f TFLOP/s (SMs x 128 lanes x 2 x clock)\n",
         p.name, sms, p.clockRate, sms * 128 * 2.0 * p.clockRate * 1e3 / 1e12);
  for (int block : {512, 1024}) {
    run<0, 0, 1>("fma.f32", block, sms);
    run<1, 0, 1>("fma.f32x2", block, sms);
    run<0, 1, 4>("fma.f32   + 1/4 lop3 per fma", block, sms);
    run<0, 1, 1>("fma.f32   + 1 lop3 per fma", block, sms);
    run<1, 1, 4>("fma.f32x2 + 1/4 lop3 per fma", block, sms);
    run<1, 1, 2>("fma.f32x2 + 1/2 lop3 per fma", block, sms);
    run<1, 1, 1>("fma.f32x2 + 1 lop3 per fma", block, sms);
    run<1, 3, 2>("fma.f32x2 + 3/2 lop3 per fma", block, sms);
    run<1, 2, 1>("fma.f32x2 + 2 lop3 per fma", block, sms);
    run<1, 3, 1>("fma.f32x2 + 3 lop3 per fma", block, sms);
  }
  return 0;
}
