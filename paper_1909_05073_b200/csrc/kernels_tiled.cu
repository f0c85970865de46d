// Tiled pattern-sparse 3x3 convolution for sm_100a.
//
// One CTA = 8 consumer warps + 4 producer warps (warp-specialised, setmaxnreg re-balances the
// register file).  The consumer warps form a (wy x ng) grid: ng filter groups of 16 filters that
// share the staged input, wy independent sets of pixel sub-tiles.  Lanes are pixels: a lane owns a
// column of 4 output rows in each of two sub-tiles ("A" and "B"), and the two are interleaved as
// float2 in shared memory so that every multiply-add is a packed fma.rn.f32x2 (one issue slot per
// two FMAs) on naturally aligned register pairs:  acc[g][k].{A,B} += {w,w} * win[row][col].{A,B}.
//
// Per input channel a lane loads its register window once (6x3 float2 at stride 1, 9x3 at stride 2)
// and reuses it for every surviving kernel of the warp's 16 filters on that channel.  Which kernels
// survive, for which filter slot and with which pattern, is a byte-code stream written by the
// packer: the warp-uniform `switch` lands in a straight-line body specialised on (filter slot,
// pattern), so accumulator and window registers are indexed at compile time, exactly 4 taps are
// executed per kernel and no lane diverges.  Pruned kernels cost nothing.
//
// Producer warps stage, per chunk of 8 input channels, the halo'd sub-tiles (zero-filled outside
// the image, converted from fp16 when the storage type is fp16) and the chunk's weight records
// (duplicated to {w,w} pairs) and codes, through a ring of shared-memory stages guarded by
// full/empty mbarriers.  Every wait is bounded; a wait that runs out records its id in the
// layer's status word and the warp leaves.
#include <cuda_fp16.h>

#include "pconv_internal.h"

namespace pconv {
namespace {

typedef unsigned long long u64;

constexpr int kConsumerWarps = 8;
constexpr int kProducerWarps = 4;
constexpr int kThreads = 32 * (kConsumerWarps + kProducerWarps);
constexpr int kMaxStages = 4;
constexpr int kWSlot = kMaxBlockKernels * 32;  // bytes per (group, stage): {w0,w0,w1,w1,w2,w2,w3,w3}
constexpr int kCodeSlot = 288;                 // bytes per (group, stage)
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int kSmemLimit = 227 * 1024;

struct SubTile {
  int n, y0, x0, valid;  // image, first output row / column, inside the batch?
};

struct Geo {
  int n, h, w, h_out, w_out;
  int tw, sw, tx, ty, q_total;
  int wys, wy, ng;       // warp grid: warp -> (warp % wys, warp / wys); rows >= wy are idle
  int pairs;             // sub-tile pairs per CTA = wy * sw
  int rows, pitch, substride, chan_stride;  // float2 units
  int stages, x_stage_bytes, stage_bytes, tab_off, stage_off;
  int relu, is_half;
};

// ---- PTX helpers ----------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void ffma2(u64& d, u64 a, u64 b) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}
__device__ __forceinline__ u64 lds64(uint32_t addr) {
  u64 v;
  asm volatile("ld.shared.b64 %0, [%1];" : "=l"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void lds128(u64& a, u64& b, uint32_t addr) {
  asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(a), "=l"(b) : "r"(addr));
}
__device__ __forceinline__ uint32_t lds_u8(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void sts64f(uint32_t addr, float a, float b) {
  asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void sts128f(uint32_t addr, float a, float b, float c, float d) {
  asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
               : "memory");
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
  asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false (and the wait id recorded) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* err, int id) {
  for (uint32_t it = 0; it < kSpinLimit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  atomicCAS(err, 0, id);
  return false;
}

// ---- compile-time tap tables ------------------------------------------------------------------------
__host__ __device__ constexpr int nth_set_bit(unsigned mask, int n) {
  int seen = 0;
  for (int t = 0; t < 9; ++t)
    if (mask >> t & 1) {
      if (seen == n) return t;
      ++seen;
    }
  return 0;
}

template <int S>
struct Win {
  static constexpr int kRows = (S == 1) ? 6 : 9;
};

// One surviving kernel, specialised on its mask and filter slot: taps 0,1, refill their weight
// registers with the next record, taps 2,3, refill (the refills complete under the other half's
// FMAs and under the next dispatch).
template <unsigned MASK, int S, int G>
__device__ __forceinline__ void kernel_body(u64 (&acc)[kGroup][4], const u64 (&win)[Win<S>::kRows][3],
                                            u64& w0, u64& w1, u64& w2, u64& w3, uint32_t& wp) {
  constexpr int t0 = nth_set_bit(MASK, 0), t1 = nth_set_bit(MASK, 1);
  constexpr int t2 = nth_set_bit(MASK, 2), t3 = nth_set_bit(MASK, 3);
#pragma unroll
  for (int k = 0; k < 4; ++k) ffma2(acc[G][k], win[S * k + t0 / 3][t0 % 3], w0);
#pragma unroll
  for (int k = 0; k < 4; ++k) ffma2(acc[G][k], win[S * k + t1 / 3][t1 % 3], w1);
  lds128(w0, w1, wp);
#pragma unroll
  for (int k = 0; k < 4; ++k) ffma2(acc[G][k], win[S * k + t2 / 3][t2 % 3], w2);
#pragma unroll
  for (int k = 0; k < 4; ++k) ffma2(acc[G][k], win[S * k + t3 / 3][t3 % 3], w3);
  lds128(w2, w3, wp + 16);
  wp += 32;
}

// Any 4-of-9 mask, taken at run time: nine warp-uniform tests, a weight load per taken tap.
template <int S, int G>
__device__ __forceinline__ void kernel_body_generic(u64 (&acc)[kGroup][4],
                                                    const u64 (&win)[Win<S>::kRows][3],
                                                    uint32_t mask, uint32_t& wp) {
#pragma unroll
  for (int t = 0; t < 9; ++t) {
    if (mask >> t & 1) {
      const u64 wv = lds64(wp);
      wp += 8;
#pragma unroll
      for (int k = 0; k < 4; ++k) ffma2(acc[G][k], win[S * k + t / 3][t % 3], wv);
    }
  }
}

template <int S>
__device__ __forceinline__ void load_window(u64 (&win)[Win<S>::kRows][3], uint32_t xptr,
                                            uint32_t pitch_b, uint32_t off_mid, uint32_t off_right) {
#pragma unroll
  for (int r = 0; r < Win<S>::kRows; ++r) {
    const uint32_t a = xptr + r * pitch_b;
    win[r][0] = lds64(a);
    win[r][1] = lds64(a + off_mid);
    win[r][2] = lds64(a + off_right);
  }
}

#define PC_CASE(G, P)                                                               \
  case (G * 8 + P):                                                                  \
    kernel_body<kCanonMasks[P], S, G>(acc, win, w0, w1, w2, w3, wp);                 \
    break;
#define PC_CASES(G) \
  PC_CASE(G, 0) PC_CASE(G, 1) PC_CASE(G, 2) PC_CASE(G, 3) PC_CASE(G, 4) PC_CASE(G, 5) PC_CASE(G, 6) PC_CASE(G, 7)
#define PG_CASE(G)                                          \
  case G:                                                   \
    kernel_body_generic<S, G>(acc, win, code & 0x1FFu, wp); \
    break;

template <typename T>
__device__ __forceinline__ float ldg_f(const T* p);
template <>
__device__ __forceinline__ float ldg_f<float>(const float* p) { return __ldg(p); }
template <>
__device__ __forceinline__ float ldg_f<__half>(const __half* p) { return __half2float(__ldg(p)); }

// ---- producer: stage one chunk -----------------------------------------------------------------------
template <int S, bool GENERIC, typename T>
__device__ __forceinline__ void produce_chunk(const DeviceLayer& L, const Geo& g, const T* __restrict__ x,
                                              const SubTile* tab, uint32_t stage_base, int k, int pw,
                                              int lane) {
  const int c0 = k * kChunk;
  const int nc = min(kChunk, L.c_in - c0);
  const size_t hw = (size_t)g.h * g.w;
  const int n_rows = g.pairs * g.rows;
  for (int row = pw; row < n_rows; row += kProducerWarps) {
    const int p = row / g.rows, r = row - p * g.rows;
    const SubTile A = tab[2 * p], B = tab[2 * p + 1];
    const int iyA = A.y0 * S - 1 + r, iyB = B.y0 * S - 1 + r;
    const bool vA = A.valid && iyA >= 0 && iyA < g.h;
    const bool vB = B.valid && iyB >= 0 && iyB < g.h;
    const T* pa = x + ((size_t)A.n * L.c_in + c0) * hw + (size_t)(vA ? iyA : 0) * g.w;
    const T* pb = x + ((size_t)B.n * L.c_in + c0) * hw + (size_t)(vB ? iyB : 0) * g.w;
    const uint32_t dst_row = stage_base + (uint32_t)((p * g.substride + r * g.pitch) * 8);
    for (int i = lane; i < g.pitch; i += 32) {
      int dx;  // input column relative to the sub-tile's first output column (in input units)
      if (S == 1) dx = i - 1;
      else dx = (i <= g.tw) ? (2 * i - 1) : (2 * (i - g.tw - 1));
      const int ixA = A.x0 * S + dx, ixB = B.x0 * S + dx;
      const bool okA = vA && ixA >= 0 && ixA < g.w;
      const bool okB = vB && ixB >= 0 && ixB < g.w;
      float va[kChunk], vb[kChunk];
#pragma unroll
      for (int cc = 0; cc < kChunk; ++cc) {
        va[cc] = (okA && cc < nc) ? ldg_f(pa + cc * hw + ixA) : 0.f;
        vb[cc] = (okB && cc < nc) ? ldg_f(pb + cc * hw + ixB) : 0.f;
      }
      const uint32_t dst = dst_row + (uint32_t)i * 8;
#pragma unroll
      for (int cc = 0; cc < kChunk; ++cc) sts64f(dst + (uint32_t)(cc * g.chan_stride) * 8, va[cc], vb[cc]);
    }
  }
  // weight records and codes of the CTA's groups
  const int ptid = pw * 32 + lane;
  const uint32_t wbase = stage_base + g.x_stage_bytes;
  const uint32_t cbase = wbase + g.ng * kWSlot;
  for (int j = 0; j < g.ng; ++j) {
    const int gi = blockIdx.y * g.ng + j;
    const uint32_t cdst = cbase + j * kCodeSlot;
    if (gi >= L.n_groups) {
      if (ptid == 0) sts32(cdst, GENERIC ? 0x40004000u : 0xFFFFFFFFu);
      continue;
    }
    const uint4 b0 = __ldg(reinterpret_cast<const uint4*>(L.blocks + (size_t)gi * L.n_chunks + k));
    const uint4 b1 = __ldg(reinterpret_cast<const uint4*>(L.blocks + (size_t)gi * L.n_chunks + k) + 1);
    const uint32_t w_off = b0.x, n_k = b0.y;
    const uint32_t c_off = GENERIC ? b1.x : b0.z, c_len = GENERIC ? b1.y : b0.w;
    if ((uint32_t)ptid < n_k) {
      float4 v;
      if (sizeof(T) == 4) {
        v = __ldg(reinterpret_cast<const float4*>(L.wvals) + w_off + ptid);
      } else {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(L.wvals) + w_off + ptid);
        const __half2 lo = *reinterpret_cast<const __half2*>(&raw.x);
        const __half2 hi = *reinterpret_cast<const __half2*>(&raw.y);
        v = make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
      }
      const uint32_t wd = wbase + j * kWSlot + ptid * 32;
      sts128f(wd, v.x, v.x, v.y, v.y);
      sts128f(wd + 16, v.z, v.z, v.w, v.w);
    }
    const uint32_t n_words = (c_len + 3) >> 2;
    const uint8_t* codes = GENERIC ? L.codes_g : L.codes_s;
    if ((uint32_t)ptid < n_words)
      sts32(cdst + ptid * 4, __ldg(reinterpret_cast<const uint32_t*>(codes + c_off) + ptid));
  }
}

template <int S, bool GENERIC>
__global__ void __launch_bounds__(kThreads, 1)
tiled_kernel(const DeviceLayer L, const Geo g, const void* __restrict__ x,
             const float* __restrict__ bias, void* __restrict__ y) {
  extern __shared__ __align__(16) unsigned char smem[];
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  SubTile* tab = reinterpret_cast<SubTile*>(smem + g.tab_off);

  if (tid == 0) {
    for (int s = 0; s < g.stages; ++s) {
      mbar_init(sbase + 8 * s, kProducerWarps);
      mbar_init(sbase + 8 * (kMaxStages + s), kConsumerWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < 2 * g.pairs; i += kThreads) {
    const long long q = (long long)blockIdx.x * (2 * g.pairs) + i;
    SubTile t;
    t.valid = q < g.q_total;
    const int qq = t.valid ? (int)q : 0;
    const int per_img = g.tx * g.ty;
    t.n = qq / per_img;
    const int rem = qq - t.n * per_img;
    const int tyi = rem / g.tx;
    t.y0 = tyi * 4;
    t.x0 = (rem - tyi * g.tx) * g.tw;
    tab[i] = t;
  }
  __syncthreads();

  if (warp >= kConsumerWarps) {
    // ===================================== producer warps =====================================
    asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
    const int pw = warp - kConsumerWarps;
    for (int k = 0; k < L.n_chunks; ++k) {
      const int s = k % g.stages, it = k / g.stages;
      if (it > 0 && !mbar_wait(sbase + 8 * (kMaxStages + s), (it - 1) & 1, L.err, 1)) return;
      const uint32_t stage_base = sbase + g.stage_off + s * g.stage_bytes;
      if (g.is_half)
        produce_chunk<S, GENERIC, __half>(L, g, (const __half*)x, tab, stage_base, k, pw, lane);
      else
        produce_chunk<S, GENERIC, float>(L, g, (const float*)x, tab, stage_base, k, pw, lane);
      __syncwarp();
      if (lane == 0) mbar_arrive(sbase + 8 * s);
    }
    return;
  }

  // ======================================= consumer warps =======================================
  asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
  const int wyi = warp % g.wys, wgi = warp / g.wys;
  const int gi = blockIdx.y * g.ng + wgi;
  const bool active = (wyi < g.wy) && (gi < L.n_groups);
  const int slot = wyi * g.sw + lane / g.tw;  // sub-tile pair of this lane
  const int col = lane % g.tw;
  const uint32_t pitch_b = g.pitch * 8;
  const uint32_t off_mid = (S == 1) ? 8u : (uint32_t)(g.tw + 1) * 8u;
  const uint32_t off_right = (S == 1) ? 16u : 8u;
  const uint32_t chan_b = (uint32_t)g.chan_stride * 8u;
  const uint32_t lane_off = (uint32_t)(slot * g.substride + col) * 8u;

  u64 acc[kGroup][4];
#pragma unroll
  for (int a = 0; a < kGroup; ++a)
#pragma unroll
    for (int k = 0; k < 4; ++k) acc[a][k] = 0ull;

  for (int k = 0; k < L.n_chunks; ++k) {
    const int s = k % g.stages;
    if (!mbar_wait(sbase + 8 * s, (k / g.stages) & 1, L.err, 2)) return;
    if (active) {
      const uint32_t stage_base = sbase + g.stage_off + s * g.stage_bytes;
      uint32_t xptr = stage_base + lane_off - chan_b;  // one channel before the chunk
      uint32_t wp = stage_base + g.x_stage_bytes + wgi * kWSlot;
      uint32_t cp = stage_base + g.x_stage_bytes + g.ng * kWSlot + wgi * kCodeSlot;
      u64 win[Win<S>::kRows][3];
#pragma unroll
      for (int r = 0; r < Win<S>::kRows; ++r) win[r][0] = win[r][1] = win[r][2] = 0ull;
      if (!GENERIC) {
        u64 w0, w1, w2, w3;
        lds128(w0, w1, wp);
        lds128(w2, w3, wp + 16);
        wp += 32;
        uint32_t code = lds_u8(cp);
        ++cp;
        for (;;) {
          const uint32_t next = lds_u8(cp);
          ++cp;
          switch (code) {
            PC_CASES(0) PC_CASES(1) PC_CASES(2) PC_CASES(3) PC_CASES(4) PC_CASES(5) PC_CASES(6) PC_CASES(7)
            PC_CASES(8) PC_CASES(9) PC_CASES(10) PC_CASES(11) PC_CASES(12) PC_CASES(13) PC_CASES(14) PC_CASES(15)
            case 128: case 129: case 130: case 131: case 132: case 133: case 134: case 135:
              xptr += (code - 127u) * chan_b;
              load_window<S>(win, xptr, pitch_b, off_mid, off_right);
              break;
            default:
              goto chunk_done;
          }
          code = next;
        }
      } else {
        for (;;) {
          const uint32_t code = lds_u16(cp);
          cp += 2;
          if (code & (uint32_t)kGenEnd) break;
          if (code & (uint32_t)kGenNext) {
            xptr += ((code & 0xFFu) + 1u) * chan_b;
            load_window<S>(win, xptr, pitch_b, off_mid, off_right);
            continue;
          }
          switch (code >> 9) {
            PG_CASE(0) PG_CASE(1) PG_CASE(2) PG_CASE(3) PG_CASE(4) PG_CASE(5) PG_CASE(6) PG_CASE(7)
            PG_CASE(8) PG_CASE(9) PG_CASE(10) PG_CASE(11) PG_CASE(12) PG_CASE(13) PG_CASE(14) PG_CASE(15)
            default: break;
          }
        }
      }
    }
  chunk_done:
    __syncwarp();
    if (lane == 0) mbar_arrive(sbase + 8 * (kMaxStages + s));
  }

  // ---- epilogue: bias, ReLU, store at the original filter index ----------------------------------
  if (!active) return;
  const SubTile A = tab[2 * slot], B = tab[2 * slot + 1];
  const int ox_a = A.x0 + col, ox_b = B.x0 + col;
  const bool col_a = A.valid && ox_a < g.w_out, col_b = B.valid && ox_b < g.w_out;
  const size_t plane = (size_t)g.h_out * g.w_out;
#pragma unroll
  for (int a = 0; a < kGroup; ++a) {
    const int o = __ldg(L.perm + gi * kGroup + a);
    if (o < 0) continue;
    const float bv = bias ? __ldg(bias + o) : 0.f;
    const size_t base_a = ((size_t)A.n * L.c_out + o) * plane;
    const size_t base_b = ((size_t)B.n * L.c_out + o) * plane;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float va = __uint_as_float((uint32_t)acc[a][k]) + bv;
      float vb = __uint_as_float((uint32_t)(acc[a][k] >> 32)) + bv;
      if (g.relu) {
        va = fmaxf(va, 0.f);
        vb = fmaxf(vb, 0.f);
      }
      const int ya = A.y0 + k, yb = B.y0 + k;
      if (g.is_half) {
        __half* yh = (__half*)y;
        if (col_a && ya < g.h_out) yh[base_a + (size_t)ya * g.w_out + ox_a] = __float2half_rn(va);
        if (col_b && yb < g.h_out) yh[base_b + (size_t)yb * g.w_out + ox_b] = __float2half_rn(vb);
      } else {
        float* yf = (float*)y;
        if (col_a && ya < g.h_out) yf[base_a + (size_t)ya * g.w_out + ox_a] = va;
        if (col_b && yb < g.h_out) yf[base_b + (size_t)yb * g.w_out + ox_b] = vb;
      }
    }
  }
}

bool make_geo(const DeviceLayer& L, int n, int h, int w, Geo* out) {
  Geo g;
  g.n = n;
  g.h = h;
  g.w = w;
  g.h_out = (h - 1) / L.stride + 1;
  g.w_out = (w - 1) / L.stride + 1;
  g.tw = 32;
  while (g.tw > 2 && g.tw / 2 >= g.w_out) g.tw /= 2;
  g.sw = 32 / g.tw;
  g.tx = (g.w_out + g.tw - 1) / g.tw;
  g.ty = (g.h_out + 3) / 4;
  const long long q = (long long)n * g.tx * g.ty;
  if (q > 0x7FFFFFFF) return false;
  g.q_total = (int)q;
  g.ng = (L.n_groups >= 3) ? 4 : L.n_groups;
  g.wys = kConsumerWarps / g.ng;
  g.wy = g.wys;
  g.rows = (L.stride == 1) ? 6 : 9;
  g.pitch = (L.stride == 1) ? (g.tw + 2) : (2 * g.tw + 1);
  g.substride = g.rows * g.pitch;
  if (g.tw < 16)  // spread the sub-tiles of a half-warp over distinct banks
    while (g.substride % 16 != g.tw % 16) ++g.substride;
  g.tab_off = 8 * 2 * kMaxStages;
  for (;;) {
    g.pairs = g.wy * g.sw;
    g.chan_stride = g.pairs * g.substride;
    g.x_stage_bytes = kChunk * g.chan_stride * 8;
    g.stage_bytes = (g.x_stage_bytes + g.ng * (kWSlot + kCodeSlot) + 15) & ~15;
    g.stage_off = (g.tab_off + 2 * g.pairs * (int)sizeof(SubTile) + 15) & ~15;
    g.stages = (kSmemLimit - g.stage_off) / g.stage_bytes;
    if (g.stages > kMaxStages) g.stages = kMaxStages;
    if (g.stages >= 2 || g.wy == 1) break;
    g.wy /= 2;
  }
  if (g.stages < 2) return false;
  if (g.stages > L.n_chunks) g.stages = (L.n_chunks < 1) ? 1 : L.n_chunks;
  g.relu = 0;
  g.is_half = (L.storage == PCONV_F16);
  *out = g;
  return true;
}

template <int S, bool GENERIC>
cudaError_t launch_one(const DeviceLayer& L, const Geo& g, const void* x, const float* bias, void* y,
                       cudaStream_t stream) {
  const int smem = g.stage_off + g.stages * g.stage_bytes;
  cudaError_t e = cudaFuncSetAttribute(tiled_kernel<S, GENERIC>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
  if (e != cudaSuccess) return e;
  const long long ctas_x = ((long long)g.q_total + 2 * g.pairs - 1) / (2 * g.pairs);
  const int ctas_y = (L.n_groups + g.ng - 1) / g.ng;
  if (ctas_x > 0x7FFFFFFF || ctas_y > 65535) return cudaErrorInvalidValue;
  dim3 grid((unsigned)ctas_x, (unsigned)ctas_y);
  tiled_kernel<S, GENERIC><<<grid, kThreads, smem, stream>>>(L, g, x, bias, y);
  return cudaGetLastError();
}

}  // namespace

bool tiled_supported(const DeviceLayer& L, int n, int h, int w) {
  Geo g;
  if (n <= 0 || h <= 0 || w <= 0) return false;
  if ((L.n_groups + 3) / 4 > 65535) return false;
  return make_geo(L, n, h, w, &g);
}

cudaError_t launch_tiled(const DeviceLayer& L, const void* x, const float* bias, void* y, int n, int h,
                         int w, bool relu, bool generic_taps, cudaStream_t stream) {
  Geo g;
  if (!make_geo(L, n, h, w, &g)) return cudaErrorInvalidValue;
  g.relu = relu ? 1 : 0;
  if (!generic_taps && !L.codes_s) generic_taps = true;
  if (L.stride == 1)
    return generic_taps ? launch_one<1, true>(L, g, x, bias, y, stream)
                        : launch_one<1, false>(L, g, x, bias, y, stream);
  return generic_taps ? launch_one<2, true>(L, g, x, bias, y, stream)
                      : launch_one<2, false>(L, g, x, bias, y, stream);
}

}  // namespace pconv
