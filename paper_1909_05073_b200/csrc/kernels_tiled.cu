// Tiled pattern-sparse 3x3 convolution for sm_100a.
//
// One CTA = consumer warps + 4 producer warps (warp-specialised), one CTA per SM.  Lanes are pixels:
// a lane owns a column of 4 output rows in each of two sub-tiles ("A" and "B"), and the two are
// interleaved as float2 in shared memory so that every multiply-add is a packed fma.rn.f32x2 (one
// issue slot per two FMAs) on naturally aligned register pairs:
//     acc[slot][k].{A,B} += {w,w} * win[row][col].{A,B}.
// A consumer warp works for one unit = (256 pixels, a group of 16 filters).  Per input channel a
// lane loads its register window once (6x3 float2 at stride 1, 9x3 at stride 2) and reuses it for
// every surviving kernel of the unit's 16 filters on that channel.  Which kernels survive, for which
// filter slot and with which pattern, is a code stream written by the packer; pruned kernels cost
// nothing and no lane ever diverges.
//
// Consumer variants (template parameters GENERIC, WIDE):
//  * Tensor-Memory accumulators (GENERIC = false): 16 consumer warps.  TMEM is addressed at run
//    time, so the filter slot is data, not code: a warp-uniform indexed jump selects a straight-line
//    body specialised on the 4-tap mask only, which reads the slot's 8 accumulator columns, runs 16
//    packed FMAs and writes them back (gen_dispatch.py).  WIDE = false: the eight canonical masks,
//    one-byte codes; WIDE = true: a body for each of the 126 masks, two-byte codes.
//    zs = 1, 2 or 4 warps of one TMEM lane quadrant may share a unit: they draw the chunks of the
//    channel range from a counter, accumulate in their own columns, and add the column sets up
//    before the epilogue.  The channel range can also be split across CTAs (grid.z), with fp32
//    atomics into a workspace and per-warp tickets that elect who finishes each part of a tile.
//    Template parameter R (canonical masks only): a lane owns R = 4 or 8 output rows per sub-tile.
//    R = 8: eight consumer warps with 256 TMEM columns each, a unit is 512 pixels and a decoded
//    kernel runs 32 packed FMAs; measured 3-10 % faster where a warp owns a unit's whole channel
//    range (large batches) and slower where channels are split (only two warps share a TMEM lane
//    quadrant), so the planner takes it for unsplit plans only.
//  * run-time masks (GENERIC = true): 8 consumer warps with register accumulators, a switch on the
//    filter slot and nine warp-uniform tap tests per kernel (384 threads leave 168 registers each,
//    which the accumulators fit); a slower cross-check of the generated bodies.
//
// Producer warps stage, per chunk of 8 input channels, the halo'd sub-tiles (zero-filled outside
// the image; fp16 storage goes through a raw ring and is widened from shared memory) and the
// chunk's weight records and codes, through a ring of shared-memory stages guarded by full/empty
// mbarriers.  Every wait is bounded; a wait that runs out records its id in the layer's status word
// and the warp stops working but still reaches every barrier and the common exit, where the TMEM
// allocation is released.  Launches use programmatic stream serialisation: set-up runs while the
// previous kernel finishes, and griddepcontrol.wait precedes the first access to activations.
#include <cuda_fp16.h>

#include <cstring>
#include <map>
#include <mutex>
#include <tuple>
#include <type_traits>
#ifdef PCONV_DEV
#include <cstdlib>
#endif

#include "pconv_internal.h"

namespace pconv {
namespace {

typedef unsigned long long u64;

constexpr int kProducerWarps = 4;
// R = output rows per lane and sub-tile: 4 (16 consumer warps with 128 TMEM columns each) or 8
// (8 consumer warps with 256 columns each: twice the packed FMAs per decoded kernel).
__host__ __device__ constexpr int consumer_warps(bool generic, int R = 4) { return (generic || R == 8) ? 8 : 16; }
__host__ __device__ constexpr int cta_threads(bool generic, int R = 4) {
  return 32 * (consumer_warps(generic, R) + kProducerWarps);
}
constexpr int kMaxConsumerWarps = 16;
constexpr int kTmemCols = 512;  // whole TMEM of the SM: 16 warps x 16 slots x 8 columns (8 x 16 x 16)
constexpr int kMaxStages = 8;
constexpr int kMaxCoop = 4;   // chunks whose x the consumer warps copy at the start of a launch
constexpr int kWSlot = kMaxBlockKernels * 16 + 16;  // bytes per (group, stage): 4 fp32 per kernel
constexpr int kCodeSlot = 400;                 // bytes per (group, stage): <= 24 records of 7 wide codes
constexpr int kWRawSlot = kMaxBlockKernels * 8;  // fp16 weight records of one (group, chunk)
constexpr int kRawStages = 3;
constexpr uint32_t kSpinLimit = 1u << 20;
// A waiting warp is suspended by the hardware for up to this long per try (it is woken when the
// phase completes), so that waiting warps leave the issue slots to the warps that have work.
constexpr uint32_t kWaitHintNs = 200;
constexpr int kSmemLimit = 227 * 1024;

struct SubTile {
  int n, y0, x0, valid;  // image, first output row / column, inside the batch?
};

struct Geo {
  int n, h, w, h_out, w_out;
  int tw, sw, tx, ty, q_total;
  int zs;                // consumer warps that share one (pixel set, filter group) and split its channels
  int wys, wy, ng;       // warp grid: unit -> (unit % wys, unit / wys); rows >= wy are idle
  int pairs;             // sub-tile pairs per CTA = wy * sw
  int rpl;               // output rows per lane and sub-tile (4 or 8)
  int rows, pitch;       // staged rows and columns of one sub-tile
  int colstride;         // bytes between staged columns (rows are contiguous float2)
  int substride, chan_stride;  // bytes per (sub-tile pair, channel) and per channel
  int stages, x_stage_bytes, stage_bytes, tab_off, desc_off, stage_off;
  // fp16 storage with an even image width: raw copies of the chunk (fp16, row-major, fetched with
  // cp.async) wait in a ring of raw_stages slots until the producers widen them into a stage
  int raw_stages, raw_off, raw_slot, raw_pitch, raw_x_bytes;
  // how a chunk reaches the raw ring: 0 = no raw ring (element-wise cp.async or loads straight into
  // the stage), 1 = fp16 element pairs by cp.async, 2 / 3 = fp32 rows / plane spans by bulk copies
  // (raw_sub = bytes per (sub-tile, channel) of a raw slot); raw_want = the mode the shape allows
  int raw_mode, raw_want, raw_sub;
  int ks, cps;           // channel splits (grid.z) and chunks per split
  int relu, is_half;
  int pool, h_y, w_y;     // fused 2x2 max-pool: y holds [h_y][w_y] = [h_out/2][w_out/2] maps
  int fixed_turns;        // 1 = the warps of a unit take the chunks in a fixed order (reproducible sums)
  int cluster;            // 1 = the ks CTAs of a tile form a thread-block cluster and add their partial
                          // sums up through distributed shared memory (no workspace, no tickets)
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
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
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
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// The mbarrier receives one arrival from this thread once all its earlier cp.async have landed.
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
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
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kWaitHintNs)
      : "memory");
  return ok != 0;
}
#ifdef PCONV_DEV
// Development build only (pconv_dev_withhold): the number of tries of every bounded wait, and the
// chunk for which one producer thread leaves out its arrival (-1 = none).
__device__ unsigned int g_dev_spin_limit = kSpinLimit;
__device__ int g_dev_withhold_chunk = -1;
#define PCONV_SPIN_LIMIT g_dev_spin_limit
#define PCONV_WITHHELD(kk, ptid) (g_dev_withhold_chunk == (kk) && (ptid) == 0)
#else
#define PCONV_SPIN_LIMIT kSpinLimit
#define PCONV_WITHHELD(kk, ptid) false
#endif

// Bounded wait: false (and the wait id recorded) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* err, int id) {
  const uint32_t limit = PCONV_SPIN_LIMIT;
  for (uint32_t it = 0; it < limit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  atomicCAS(err, 0, id);
  return false;
}

// Built with -DPCONV_DEV (build.py: build(dev=True) -> libpconv_dev.so) the kernel leaves
// timestamps in the trace words of the handle's status block (pconv_trace_read):
//   0 start, 1 set-up done, 2 warp 0's first chunk landed, 3 loop end, 4 partial sums issued (split only;
//   cluster form: partial sums in shared memory, before the cluster's first barrier),
//   5 epilogue end, 6 after the CTA's last barrier -- thread 0 of CTA (0,0,0), globaltimer ns;
//   7 end, 8 start, 9 loop end, 10 partial sums issued -- latest over all CTAs;
//   11 / 12 cycles warp 0 of CTA (0,0,0) spent waiting for chunks / working on them, 13 its chunks.
#ifdef PCONV_DEV
#define PCONV_MARK(i)                                                         \
  if (threadIdx.x == 0 && bp.x == 0 && bp.y == 0 && bp.z == 0) { \
    unsigned long long t_;                                                    \
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                    \
    trace_words(L)[i] = t_;                                                   \
  }
#define PCONV_MARK_MAX(i)                                                     \
  if (threadIdx.x == 0) {                                                     \
    unsigned long long t_;                                                    \
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                    \
    atomicMax(trace_words(L) + i, t_);                                        \
  }
#else
#define PCONV_MARK(i)
#define PCONV_MARK_MAX(i)
#endif

template <int S, int R = 4>
struct Win {
  static constexpr int kRows = S * (R - 1) + 3;   // input rows under R output rows
};

// The specialised dispatch loop of one (warp, chunk): generated PTX (see gen_dispatch.py); the
// accumulators stay in TMEM at `tq` (+ 8 columns per filter slot).
template <int S, int R>
__device__ __forceinline__ void dispatch_chunk(uint32_t cp, uint32_t wp, uint32_t xptr,
                                               uint32_t chan_b, uint32_t col_b, uint32_t off_mid,
                                               uint32_t tq, uint32_t entry_code) {
  if constexpr (S == 1 && R == 4) {
    asm volatile(
#include "dispatch_s1.inc"
        :
        : "r"(cp), "r"(wp), "r"(xptr), "r"(chan_b), "r"(col_b), "r"(off_mid), "r"(tq), "r"(entry_code)
        : "memory");
  } else if constexpr (S == 2 && R == 4) {
    asm volatile(
#include "dispatch_s2.inc"
        :
        : "r"(cp), "r"(wp), "r"(xptr), "r"(chan_b), "r"(col_b), "r"(off_mid), "r"(tq), "r"(entry_code)
        : "memory");
  } else if constexpr (S == 1) {
    asm volatile(
#include "dispatch_s1t.inc"
        :
        : "r"(cp), "r"(wp), "r"(xptr), "r"(chan_b), "r"(col_b), "r"(off_mid), "r"(tq), "r"(entry_code)
        : "memory");
  } else {
    asm volatile(
#include "dispatch_s2t.inc"
        :
        : "r"(cp), "r"(wp), "r"(xptr), "r"(chan_b), "r"(col_b), "r"(off_mid), "r"(tq), "r"(entry_code)
        : "memory");
  }
}
// The same loop for wide codes (a body for every 4-of-9 mask); only the kernel instantiations for
// non-canonical pattern sets contain it, so the canonical kernels stay compact.
template <int S>
__device__ __forceinline__ void dispatch_chunk_wide(uint32_t cp, uint32_t wp, uint32_t xptr,
                                                 uint32_t chan_b, uint32_t col_b, uint32_t off_mid,
                                                 uint32_t tq, uint32_t entry_code) {
  if (S == 1) {
    asm volatile(
#include "dispatch_s1w.inc"
        :
        : "r"(cp), "r"(wp), "r"(xptr), "r"(chan_b), "r"(col_b), "r"(off_mid), "r"(tq), "r"(entry_code)
        : "memory");
  } else {
    asm volatile(
#include "dispatch_s2w.inc"
        :
        : "r"(cp), "r"(wp), "r"(xptr), "r"(chan_b), "r"(col_b), "r"(off_mid), "r"(tq), "r"(entry_code)
        : "memory");
  }
}

__device__ __forceinline__ void tmem_ld8_nowait(uint32_t* r, uint32_t taddr) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]),
                 "=r"(r[7])
               : "r"(taddr));
}
// The NV = 8 or 16 columns of one filter slot.
template <int NV>
__device__ __forceinline__ void tmem_ld_slot_nowait(uint32_t (&r)[NV], uint32_t taddr) {
  tmem_ld8_nowait(r, taddr);
  if constexpr (NV == 16) tmem_ld8_nowait(r + 8, taddr + 8);
}
__device__ __forceinline__ void tmem_st8_zero(uint32_t taddr) {
  const uint32_t z = 0;
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%1,%1,%1,%1,%1,%1,%1};" ::"r"(taddr), "r"(z)
               : "memory");
}

// Any 4-of-9 mask, taken at run time: nine warp-uniform tests, a weight load per taken tap.
template <int S, int G>
__device__ __forceinline__ void kernel_body_generic(u64 (&acc)[kGroup][4],
                                                    const u64 (&win)[Win<S>::kRows][3],
                                                    uint32_t mask, uint32_t& wp) {
#pragma unroll
  for (int t = 0; t < 9; ++t) {
    if (mask >> t & 1) {
      const uint32_t w1 = lds32(wp);
      const u64 wv = ((u64)w1 << 32) | w1;
      wp += 4;
#pragma unroll
      for (int k = 0; k < 4; ++k) ffma2(acc[G][k], win[S * k + t / 3][t % 3], wv);
    }
  }
}

template <int S>
__device__ __forceinline__ void load_window(u64 (&win)[Win<S>::kRows][3], uint32_t xptr,
                                            uint32_t off_mid, uint32_t off_right) {
#pragma unroll
  for (int r = 0; r < Win<S>::kRows; ++r) {
    win[r][0] = lds64(xptr + r * 8);
    win[r][1] = lds64(xptr + off_mid + r * 8);
    win[r][2] = lds64(xptr + off_right + r * 8);
  }
}

#define PG_CASE(G)                                          \
  case G:                                                   \
    kernel_body_generic<S, G>(acc, win, code & 0x1FFu, wp); \
    break;
#define PG_CASES8(B) PG_CASE(B + 0) PG_CASE(B + 1) PG_CASE(B + 2) PG_CASE(B + 3) PG_CASE(B + 4) PG_CASE(B + 5) PG_CASE(B + 6) PG_CASE(B + 7)

// ---- producer: stage one chunk -----------------------------------------------------------------------
// Input columns staged for row element i of a sub-tile, relative to its first output column
// (stride 1: i-1; stride 2: the odd columns 2i-1 first, then the even columns).
template <int S>
__device__ __forceinline__ int staged_dx(int i, int tw) {
  if (S == 1) return i - 1;
  return (i <= tw) ? (2 * i - 1) : (2 * (i - tw - 1));
}

// One staged element = one (sub-tile pair, row, column) position of the halo'd tile, holding the
// A and the B pixel.  Elements are dealt to the 128 producer threads in flat order, so narrow
// sub-tiles keep all lanes busy.
struct StagedElem {
  long long off_a, off_b;   // element offsets into x for channel c0 of the chunk, or -1
  uint32_t dst;             // byte offset inside the channel's staged block
};
template <int S, int R>
__device__ __forceinline__ StagedElem staged_elem(const DeviceLayer& L, const Geo& g,
                                                  const SubTile* tab, int e, int c0) {
  constexpr int kRows = Win<S, R>::kRows;
  const int q = e / g.pitch, i = e - q * g.pitch;   // q = pair * rows + row
  const int p = q / kRows, r = q - p * kRows;
  const SubTile A = tab[2 * p], B = tab[2 * p + 1];
  const int dx = staged_dx<S>(i, g.tw);
  const int iyA = A.y0 * S - 1 + r, iyB = B.y0 * S - 1 + r;
  const int ixA = A.x0 * S + dx, ixB = B.x0 * S + dx;
  const long long hw = (long long)g.h * g.w;
  StagedElem se;
  se.off_a = (A.valid && iyA >= 0 && iyA < g.h && ixA >= 0 && ixA < g.w)
                 ? ((long long)A.n * L.c_in + c0) * hw + (long long)iyA * g.w + ixA : -1;
  se.off_b = (B.valid && iyB >= 0 && iyB < g.h && ixB >= 0 && ixB < g.w)
                 ? ((long long)B.n * L.c_in + c0) * hw + (long long)iyB * g.w + ixB : -1;
  se.dst = (uint32_t)(p * g.substride + i * g.colstride + r * 8);
  return se;
}

// A producer thread's staged elements are the same in every chunk (only the channel moves), so up
// to kPreElems of them are worked out once, for channel 0, and kept in registers; threads of wider
// tiles work the rest out per chunk.  dst == kSkipElem marks a slot past the tile's last element.
constexpr int kPreElems = 4;
constexpr uint32_t kSkipElem = 0xFFFFFFFFu;
constexpr int kProducerThreads = 32 * kProducerWarps;

template <int S, int R>
__device__ __forceinline__ void precompute_elems(StagedElem (&pre)[kPreElems], const DeviceLayer& L,
                                                 const Geo& g, const SubTile* tab, int ptid) {
  const int n_elem = g.pairs * g.rows * g.pitch;
#pragma unroll
  for (int i = 0; i < kPreElems; ++i) {
    const int e = ptid + i * kProducerThreads;
    if (e < n_elem) {
      pre[i] = staged_elem<S, R>(L, g, tab, e, 0);
    } else {
      pre[i].off_a = pre[i].off_b = -1;
      pre[i].dst = kSkipElem;
    }
  }
}

// The weight records and codes of the CTA's groups for chunk kk of its range.
__device__ __forceinline__ void stage_blocks_async(const DeviceLayer& L, const Geo& g, const uint4* desc,
                                                   const uint8_t* codes, uint32_t stage_base, int kk,
                                                   int ptid) {
  const uint32_t wbase = stage_base + g.x_stage_bytes;
  const uint32_t cbase = wbase + g.ng * kWSlot;
  for (int j = 0; j < g.ng; ++j) {
    const uint4 d = desc[2 * (j * g.cps + kk)];  // {w_off, n_k, code_off, code_len}
    if ((uint32_t)ptid < d.y)
      cp_async16(wbase + j * kWSlot + ptid * 16,
                 reinterpret_cast<const float*>(L.wvals) + (size_t)(d.x + ptid) * 4);
    if ((uint32_t)ptid * 16 < d.w) cp_async16(cbase + j * kCodeSlot + ptid * 16, codes + d.z + ptid * 16);
  }
}

// The same for fp16 storage: the values are widened on the way (loaded, converted, stored).  All
// groups' loads are issued before the first store, so a chunk costs two round trips, not 2 x ng.
__device__ __forceinline__ void stage_blocks_half(const DeviceLayer& L, const Geo& g, const uint4* desc,
                                                  const uint8_t* codes, uint32_t stage_base, int kk,
                                                  int ptid) {
  constexpr int kMaxNg = 16;
  const uint32_t wbase = stage_base + g.x_stage_bytes;
  const uint32_t cbase = wbase + g.ng * kWSlot;
  // codes need no conversion: asynchronous copies, issued first and waited for at the end (the
  // caller's plain barrier arrival does not cover them)
  for (int j = 0; j < g.ng; ++j) {
    const uint4 d = desc[2 * (j * g.cps + kk)];
    if ((uint32_t)ptid * 16 < d.w) cp_async16(cbase + j * kCodeSlot + ptid * 16, codes + d.z + ptid * 16);
  }
  uint2 raw[kMaxNg];
#pragma unroll
  for (int j = 0; j < kMaxNg; ++j) {
    raw[j] = make_uint2(0u, 0u);
    if (j < g.ng) {
      const uint4 d = desc[2 * (j * g.cps + kk)];
      if ((uint32_t)ptid < d.y) raw[j] = __ldg(reinterpret_cast<const uint2*>(L.wvals) + d.x + ptid);
    }
  }
#pragma unroll
  for (int j = 0; j < kMaxNg; ++j) {
    if (j < g.ng) {
      const __half2 lo = *reinterpret_cast<const __half2*>(&raw[j].x);
      const __half2 hi = *reinterpret_cast<const __half2*>(&raw[j].y);
      sts128f(wbase + j * kWSlot + ptid * 16, __low2float(lo), __high2float(lo), __low2float(hi),
              __high2float(hi));
    }
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
}

// fp32 storage: everything is fetched with cp.async (zero-fill outside the image), so the producer
// never waits for data and several chunks are in flight; each thread's arrival on the stage's full
// barrier fires when its own copies have landed.
template <int S, int R>
__device__ __forceinline__ void produce_chunk_async(const DeviceLayer& L, const Geo& g,
                                                    const float* __restrict__ x, const SubTile* tab,
                                                    const StagedElem (&pre)[kPreElems], const uint4* desc,
                                                    const uint8_t* codes, uint32_t stage_base, int k, int kk,
                                                    int ptid, bool with_x, bool with_blocks) {
  const int c0 = k * kChunk;
  const int nc = min(kChunk, L.c_in - c0);
  const size_t hw = (size_t)g.h * g.w;
  const int n_elem = with_x ? g.pairs * g.rows * g.pitch : 0;
  const uint32_t chan_b = (uint32_t)g.chan_stride;
  auto copy_elem = [&](const StagedElem& se, size_t chan_off) {
    const float* sa = se.off_a >= 0 ? x + se.off_a + chan_off : x;
    const float* sb = se.off_b >= 0 ? x + se.off_b + chan_off : x;
    const size_t step_a = se.off_a >= 0 ? hw : 0, step_b = se.off_b >= 0 ? hw : 0;
    const uint32_t na = se.off_a >= 0 ? 4u : 0u, nb = se.off_b >= 0 ? 4u : 0u;
    uint32_t dst = stage_base + se.dst;
    if (nc == kChunk) {   // a whole chunk: straight-line copies
#pragma unroll
      for (int cc = 0; cc < kChunk; ++cc) {
        cp_async4(dst + cc * chan_b, sa + cc * step_a, na);
        cp_async4(dst + cc * chan_b + 4, sb + cc * step_b, nb);
      }
    } else {
      for (int cc = 0; cc < nc; ++cc) {
        cp_async4(dst, sa, na);
        cp_async4(dst + 4, sb, nb);
        sa += step_a;
        sb += step_b;
        dst += chan_b;
      }
    }
  };
  if (with_x) {
#pragma unroll
    for (int i = 0; i < kPreElems; ++i)
      if (pre[i].dst != kSkipElem) copy_elem(pre[i], (size_t)c0 * hw);
  }
  for (int e = ptid + kPreElems * kProducerThreads; e < n_elem; e += kProducerThreads)
    copy_elem(staged_elem<S, R>(L, g, tab, e, c0), 0);
  if (with_blocks) stage_blocks_async(L, g, desc, codes, stage_base, kk, ptid);
}

// The x part of one chunk copied by `n_threads` threads (thread `t` of them): used by the
// consumer warps, which have nothing else to do yet, for the first chunks of a launch.  A warp can
// keep only a few cp.async in flight, so twenty warps fill a chunk several times faster than the
// four producer warps.
template <int S, int R>
__device__ __forceinline__ void fill_chunk_x(const DeviceLayer& L, const Geo& g, const float* __restrict__ x,
                                             const SubTile* tab, uint32_t stage_base, int k, int t,
                                             int n_threads) {
  const int c0 = k * kChunk;
  const int nc = min(kChunk, L.c_in - c0);
  const size_t hw = (size_t)g.h * g.w;
  const int n_elem = g.pairs * g.rows * g.pitch;
  const uint32_t chan_b = (uint32_t)g.chan_stride;
  for (int e = t; e < n_elem; e += n_threads) {
    const StagedElem se = staged_elem<S, R>(L, g, tab, e, c0);
    const float* sa = se.off_a >= 0 ? x + se.off_a : x;
    const float* sb = se.off_b >= 0 ? x + se.off_b : x;
    const size_t step_a = se.off_a >= 0 ? hw : 0, step_b = se.off_b >= 0 ? hw : 0;
    const uint32_t na = se.off_a >= 0 ? 4u : 0u, nb = se.off_b >= 0 ? 4u : 0u;
    uint32_t dst = stage_base + se.dst;
    for (int cc = 0; cc < nc; ++cc) {
      cp_async4(dst, sa, na);
      cp_async4(dst + 4, sb, nb);
      sa += step_a;
      sb += step_b;
      dst += chan_b;
    }
  }
}

// ---- fp16 storage, even image width: raw ring ----------------------------------------------------
// A chunk is first copied as it is (fp16, each sub-tile row-major with a two-column margin so that
// every 4-byte unit starts on an even column and lies wholly inside or outside the image) into a
// slot of the raw ring with cp.async -- no registers held, several chunks in flight -- together
// with its fp16 weight records and its codes.  When the copies have landed the producer warps widen
// the slot into a stage (shared memory to shared memory) in the layout the consumers read.

// Byte offsets of a staged element's A and B halves inside a raw slot (channel 0) and of its
// place in the stage, in the fields of a StagedElem (off_a, off_b, dst).
template <int S, int R>
__device__ __forceinline__ StagedElem raw_elem(const Geo& g, int e) {
  constexpr int kRows = Win<S, R>::kRows;
  const int q = e / g.pitch, i = e - q * g.pitch;   // q = pair * rows + row
  const int p = q / kRows, r = q - p * kRows;
  const int hidx = staged_dx<S>(i, g.tw) + 2;        // column inside the raw row
  const int row_b = g.raw_pitch * 2;
  StagedElem se;
  se.off_a = ((long long)(2 * p) * kChunk * kRows + r) * row_b + hidx * 2;
  se.off_b = ((long long)(2 * p + 1) * kChunk * kRows + r) * row_b + hidx * 2;
  se.dst = (uint32_t)(p * g.substride + i * g.colstride + r * 8);
  return se;
}

template <int S, int R>
__device__ __forceinline__ void issue_raw(const DeviceLayer& L, const Geo& g, const __half* __restrict__ x,
                                          const SubTile* tab, const uint4* desc, const uint8_t* codes,
                                          uint32_t raw_base, int k, int kk, int ptid) {
  constexpr int kRows = Win<S, R>::kRows;
  const int c0 = k * kChunk;
  const int nc = min(kChunk, L.c_in - c0);
  const size_t hw = (size_t)g.h * g.w;
  const int units_row = g.raw_pitch / 2;
  const int n_units = g.pairs * 2 * kRows * units_row;
  const uint32_t chan_b = (uint32_t)(kRows * g.raw_pitch * 2);
  for (int v = ptid; v < n_units; v += kProducerThreads) {
    const int q = v / units_row, u = v - q * units_row;   // q = sub-tile * rows + row
    const int ps = q / kRows, r = q - ps * kRows;
    const SubTile T = tab[ps];
    const int iy = T.y0 * S - 1 + r, ix = T.x0 * S - 2 + 2 * u;
    const bool in = T.valid && iy >= 0 && iy < g.h && ix >= 0 && ix < g.w;
    const __half* src = in ? x + (((size_t)T.n * L.c_in + c0) * g.h + iy) * g.w + ix : x;
    const size_t step = in ? hw : 0;
    uint32_t dst = raw_base + (uint32_t)((ps * kChunk * kRows + r) * g.raw_pitch * 2 + u * 4);
    for (int cc = 0; cc < kChunk; ++cc) {
      cp_async4(dst, src, (in && cc < nc) ? 4u : 0u);
      src += step;
      dst += chan_b;
    }
  }
  const uint32_t wbase = raw_base + g.raw_x_bytes;
  const uint32_t cbase = wbase + g.ng * kWRawSlot;
  for (int j = 0; j < g.ng; ++j) {
    const uint4 d = desc[2 * (j * g.cps + kk)];
    if ((uint32_t)ptid < d.y)
      asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(wbase + j * kWRawSlot + ptid * 8),
                   "l"(reinterpret_cast<const uint2*>(L.wvals) + d.x + ptid)
                   : "memory");
    if ((uint32_t)ptid * 16 < d.w) cp_async16(cbase + j * kCodeSlot + ptid * 16, codes + d.z + ptid * 16);
  }
}

template <int S, int R>
__device__ __forceinline__ void widen_raw(const Geo& g, const StagedElem (&pre)[kPreElems],
                                          const uint4* desc, uint32_t raw_base, uint32_t stage_base,
                                          int kk, int ptid) {
  constexpr int kRows = Win<S, R>::kRows;
  const int n_elem = g.pairs * g.rows * g.pitch;
  const uint32_t raw_chan = (uint32_t)(kRows * g.raw_pitch * 2);
  auto widen = [&](const StagedElem& se) {
    uint32_t va[kChunk], vb[kChunk];
#pragma unroll
    for (int cc = 0; cc < kChunk; ++cc) {
      va[cc] = lds_u16(raw_base + (uint32_t)se.off_a + cc * raw_chan);
      vb[cc] = lds_u16(raw_base + (uint32_t)se.off_b + cc * raw_chan);
    }
#pragma unroll
    for (int cc = 0; cc < kChunk; ++cc) {
      const uint32_t pk = va[cc] | (vb[cc] << 16);
      const __half2 h = *reinterpret_cast<const __half2*>(&pk);
      sts64f(stage_base + se.dst + (uint32_t)(cc * g.chan_stride), __low2float(h), __high2float(h));
    }
  };
#pragma unroll
  for (int i = 0; i < kPreElems; ++i)
    if (pre[i].dst != kSkipElem) widen(pre[i]);
  for (int e = ptid + kPreElems * kProducerThreads; e < n_elem; e += kProducerThreads) widen(raw_elem<S, R>(g, e));
  const uint32_t rw = raw_base + g.raw_x_bytes, rc = rw + g.ng * kWRawSlot;
  const uint32_t wbase = stage_base + g.x_stage_bytes, cbase = wbase + g.ng * kWSlot;
  for (int j = 0; j < g.ng; ++j) {
    const uint4 d = desc[2 * (j * g.cps + kk)];
    if ((uint32_t)ptid < d.y) {
      const u64 raw = lds64(rw + j * kWRawSlot + ptid * 8);
      const uint32_t lo32 = (uint32_t)raw, hi32 = (uint32_t)(raw >> 32);
      const __half2 lo = *reinterpret_cast<const __half2*>(&lo32);
      const __half2 hi = *reinterpret_cast<const __half2*>(&hi32);
      sts128f(wbase + j * kWSlot + ptid * 16, __low2float(lo), __high2float(lo), __low2float(hi),
              __high2float(hi));
    }
    if ((uint32_t)ptid * 16 < d.w) {
      uint32_t c0, c1, c2, c3;
      asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                   : "=r"(c0), "=r"(c1), "=r"(c2), "=r"(c3)
                   : "r"(rc + j * kCodeSlot + ptid * 16));
      asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(cbase + j * kCodeSlot + ptid * 16),
                   "r"(c0), "r"(c1), "r"(c2), "r"(c3)
                   : "memory");
    }
  }
}

// The producers' loop of the raw-ring path.  Every producer thread passes through every named
// barrier of every chunk, also after a bounded wait ran out (it then does no more work), so the
// barrier counts always match.
template <int S, int R>
__device__ __forceinline__ void produce_raw_stream(const DeviceLayer& L, const Geo& g,
                                                   const __half* __restrict__ x, const SubTile* tab,
                                                   const StagedElem (&pre)[kPreElems], const uint4* desc,
                                                   const uint8_t* codes, uint32_t sbase, int k0, int nk,
                                                   int ptid) {
  const int RS = g.raw_stages;
  bool ok = true;
  auto raw_base = [&](int kk) { return sbase + g.raw_off + (kk % RS) * g.raw_slot; };
  auto producers_sync = [] { asm volatile("bar.sync 2, %0;" ::"n"(kProducerThreads) : "memory"); };
  // one cp.async group per chunk (empty past the last chunk), RS - 1 chunks ahead of the one being
  // widened, so "all but the newest RS - 1 groups" is exactly "chunk kk has landed"
  for (int j = 0; j < RS - 1; ++j) {
    if (j < nk) issue_raw<S, R>(L, g, x, tab, desc, codes, raw_base(j), k0 + j, j, ptid);
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  for (int kk = 0; kk < nk; ++kk) {
    const int ahead = kk + RS - 1;
    if (ok && ahead < nk) issue_raw<S, R>(L, g, x, tab, desc, codes, raw_base(ahead), k0 + ahead, ahead, ptid);
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (RS >= 3) asm volatile("cp.async.wait_group 2;" ::: "memory");
    else if (RS == 2) asm volatile("cp.async.wait_group 1;" ::: "memory");
    else asm volatile("cp.async.wait_group 0;" ::: "memory");
    producers_sync();   // everybody's copies of chunk kk have landed
    const int s = kk % g.stages, it = kk / g.stages;
    if (ok && it > 0) ok = mbar_wait(sbase + 8 * (kMaxStages + s), (it - 1) & 1, L.err, 1);
    if (ok) {
      widen_raw<S, R>(g, pre, desc, raw_base(kk), sbase + g.stage_off + s * g.stage_bytes, kk, ptid);
      if (!PCONV_WITHHELD(kk, ptid)) mbar_arrive(sbase + 8 * s);
    }
    producers_sync();   // the raw slot may be overwritten
  }
}

// ---- fp32 storage: bulk copies into the raw ring -----------------------------------------------------
// Where the rows (or whole planes) of the input start on 16-byte boundaries, a chunk is fetched by
// the copy engine instead of by element-wise cp.async: cp.async.bulk (no tensor map, this CTA's own
// shared memory, no multicast) brings, per sub-tile and channel, either its rows (raw_mode 2:
// image wider than a sub-tile, width a multiple of 4; a raw row starts 4 columns left of the
// sub-tile so that every copy is aligned) or one contiguous span of the plane (raw_mode 3:
// sub-tile as wide as the image, plane size a multiple of 4 elements), and the chunk's weight
// records and codes, all completing on the raw slot's mbarrier.  The producer warps then build the
// stage from the raw slot (shared memory to shared memory): the {A,B}-interleaved column-major
// tile, with zeros for everything outside the image -- the copies carry no padding.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void sts64u(uint32_t addr, uint32_t a, uint32_t b) {
  asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(addr), "r"(a), "r"(b) : "memory");
}
// First element of the plane that a sub-tile's span holds (raw_mode 3): its first input row,
// rounded down to a multiple of 4 elements.
template <int S>
__device__ __forceinline__ int span_origin(const Geo& g, const SubTile& T) {
  const int iy0 = T.y0 * S - 1;
  return (iy0 > 0 ? iy0 * g.w : 0) & ~3;
}

// Byte offsets of a staged element's A and B sources inside a raw slot (channel 0 of the chunk),
// or -1 where the element lies outside the image or the batch (the stage gets a zero there).
template <int S, int R>
__device__ __forceinline__ StagedElem bulk_elem(const Geo& g, const SubTile* tab, int e) {
  constexpr int kRows = Win<S, R>::kRows;
  const int q = e / g.pitch, i = e - q * g.pitch;   // q = pair * rows + row
  const int p = q / kRows, r = q - p * kRows;
  const int dx = staged_dx<S>(i, g.tw);
  auto src = [&](int sub) -> long long {
    const SubTile T = tab[sub];
    const int iy = T.y0 * S - 1 + r, ix = T.x0 * S + dx;
    if (!T.valid || iy < 0 || iy >= g.h || ix < 0 || ix >= g.w) return -1;
    const int idx = (g.raw_mode == 2) ? r * g.raw_pitch + dx + 4 : iy * g.w + ix - span_origin<S>(g, T);
    return (long long)sub * kChunk * g.raw_sub + (long long)idx * 4;
  };
  StagedElem se;
  se.off_a = src(2 * p);
  se.off_b = src(2 * p + 1);
  se.dst = (uint32_t)(p * g.substride + i * g.colstride + r * 8);
  return se;
}

// This thread's share of the copies of chunk k (kk-th of the CTA) into the raw slot at raw_base;
// it then arrives on the slot's barrier with the bytes it asked for.
template <int S, int R>
__device__ __forceinline__ void issue_bulk(const DeviceLayer& L, const Geo& g, const float* __restrict__ x,
                                           const SubTile* tab, const uint4* desc, const uint8_t* codes,
                                           uint32_t raw_base, uint32_t bar, int k, int kk, int ptid) {
  constexpr int kRows = Win<S, R>::kRows;
  const int c0 = k * kChunk;
  const int nc = min(kChunk, L.c_in - c0);
  const size_t hw = (size_t)g.h * g.w;
  uint32_t bytes = 0;
  if (g.raw_mode == 2) {
    const int n_copy = g.pairs * 2 * kChunk * kRows;
    for (int v = ptid; v < n_copy; v += kProducerThreads) {
      const int t = v / kRows, r = v - t * kRows;
      const int sub = t / kChunk, cc = t - sub * kChunk;
      const SubTile T = tab[sub];
      const int iy = T.y0 * S - 1 + r;
      if (!T.valid || cc >= nc || iy < 0 || iy >= g.h) continue;
      const int xo = T.x0 * S - 4;                       // column of the raw row's first element
      const int xs = xo > 0 ? xo : 0;
      const int xe = min(g.w, xo + g.raw_pitch);
      if (xe <= xs) continue;
      const uint32_t nb = (uint32_t)(xe - xs) * 4u;
      bulk_copy_g2s(raw_base + (uint32_t)((sub * kChunk + cc) * g.raw_sub + (r * g.raw_pitch + xs - xo) * 4),
                    x + ((size_t)T.n * L.c_in + c0 + cc) * hw + (size_t)iy * g.w + xs, nb, bar);
      bytes += nb;
    }
  } else {
    const int n_copy = g.pairs * 2 * kChunk;
    for (int v = ptid; v < n_copy; v += kProducerThreads) {
      const int sub = v / kChunk, cc = v - sub * kChunk;
      const SubTile T = tab[sub];
      if (!T.valid || cc >= nc) continue;
      const int fo = span_origin<S>(g, T);
      const int last_row = min(g.h, T.y0 * S - 1 + kRows);
      const int fe = min((int)hw, (last_row * g.w + 3) & ~3);
      if (fe <= fo) continue;
      const uint32_t nb = (uint32_t)(fe - fo) * 4u;
      bulk_copy_g2s(raw_base + (uint32_t)((sub * kChunk + cc) * g.raw_sub),
                    x + ((size_t)T.n * L.c_in + c0 + cc) * hw + fo, nb, bar);
      bytes += nb;
    }
  }
  // the chunk's weight records and codes, one copy each per filter group
  const uint32_t wbase = raw_base + g.raw_x_bytes;
  const uint32_t cbase = wbase + g.ng * kWSlot;
  for (int v = ptid; v < 2 * g.ng; v += kProducerThreads) {
    const int j = v >> 1;
    const uint4 d = desc[2 * (j * g.cps + kk)];   // {w_off, n_k, code_off, code_len}
    if (v & 1) {
      const uint32_t nb = (d.w + 15u) & ~15u;
      if (nb) {
        bulk_copy_g2s(cbase + j * kCodeSlot, codes + d.z, nb, bar);
        bytes += nb;
      }
    } else if (d.y) {
      bulk_copy_g2s(wbase + j * kWSlot, reinterpret_cast<const float*>(L.wvals) + (size_t)d.x * 4, d.y * 16u, bar);
      bytes += d.y * 16u;
    }
  }
  mbar_arrive_expect_tx(bar, bytes);
}

// Raw slot -> stage: the interleaved tile (zeros outside the image), the weight records, the codes.
template <int S, int R>
__device__ __forceinline__ void widen_bulk(const Geo& g, const SubTile* tab, const StagedElem (&pre)[kPreElems],
                                           const uint4* desc, uint32_t raw_base, uint32_t stage_base,
                                           int kk, int ptid) {
  const int n_elem = g.pairs * g.rows * g.pitch;
  const uint32_t raw_chan = (uint32_t)g.raw_sub;
  auto widen = [&](const StagedElem& se) {
    uint32_t va[kChunk], vb[kChunk];
#pragma unroll
    for (int cc = 0; cc < kChunk; ++cc) {
      va[cc] = se.off_a >= 0 ? lds32(raw_base + (uint32_t)se.off_a + cc * raw_chan) : 0u;
      vb[cc] = se.off_b >= 0 ? lds32(raw_base + (uint32_t)se.off_b + cc * raw_chan) : 0u;
    }
#pragma unroll
    for (int cc = 0; cc < kChunk; ++cc)
      sts64u(stage_base + se.dst + (uint32_t)(cc * g.chan_stride), va[cc], vb[cc]);
  };
#pragma unroll
  for (int i = 0; i < kPreElems; ++i)
    if (pre[i].dst != kSkipElem) widen(pre[i]);
  for (int e = ptid + kPreElems * kProducerThreads; e < n_elem; e += kProducerThreads)
    widen(bulk_elem<S, R>(g, tab, e));
  const uint32_t rw = raw_base + g.raw_x_bytes, rc = rw + g.ng * kWSlot;
  const uint32_t wbase = stage_base + g.x_stage_bytes, cbase = wbase + g.ng * kWSlot;
  auto copy16 = [](uint32_t dst, uint32_t src) {
    uint32_t c0, c1, c2, c3;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(c0), "=r"(c1), "=r"(c2), "=r"(c3) : "r"(src));
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
  };
  for (int j = 0; j < g.ng; ++j) {
    const uint4 d = desc[2 * (j * g.cps + kk)];
    if ((uint32_t)ptid < d.y) copy16(wbase + j * kWSlot + ptid * 16, rw + j * kWSlot + ptid * 16);
    if ((uint32_t)ptid * 16 < d.w) copy16(cbase + j * kCodeSlot + ptid * 16, rc + j * kCodeSlot + ptid * 16);
  }
}

// The producers' loop of the bulk-copy path: the copies of a chunk are issued raw_stages - 1 chunks
// ahead of the chunk being turned into a stage.  Every wait is bounded (id 4: a raw slot's copies).
template <int S, int R>
__device__ __forceinline__ void produce_bulk_stream(const DeviceLayer& L, const Geo& g,
                                                    const float* __restrict__ x, const SubTile* tab,
                                                    const StagedElem (&pre)[kPreElems], const uint4* desc,
                                                    const uint8_t* codes, uint32_t sbase, uint32_t raw_bar0,
                                                    int k0, int nk, int ptid) {
  const int RS = g.raw_stages;
  bool ok = true;
  auto raw_base = [&](int kk) { return sbase + g.raw_off + (kk % RS) * g.raw_slot; };
  auto raw_bar = [&](int kk) { return raw_bar0 + 8u * (uint32_t)(kk % RS); };
  auto producers_sync = [] { asm volatile("bar.sync 2, %0;" ::"n"(kProducerThreads) : "memory"); };
  for (int j = 0; j < RS - 1; ++j)
    if (j < nk) issue_bulk<S, R>(L, g, x, tab, desc, codes, raw_base(j), raw_bar(j), k0 + j, j, ptid);
  for (int kk = 0; kk < nk; ++kk) {
    const int ahead = kk + RS - 1;
    if (ok && ahead < nk)
      issue_bulk<S, R>(L, g, x, tab, desc, codes, raw_base(ahead), raw_bar(ahead), k0 + ahead, ahead, ptid);
    if (ok) ok = mbar_wait(raw_bar(kk), (kk / RS) & 1, L.err, 4);
    const int s = kk % g.stages, it = kk / g.stages;
    if (ok && it > 0) ok = mbar_wait(sbase + 8 * (kMaxStages + s), (it - 1) & 1, L.err, 1);
    if (ok) {
      widen_bulk<S, R>(g, tab, pre, desc, raw_base(kk), sbase + g.stage_off + s * g.stage_bytes, kk, ptid);
      if (!PCONV_WITHHELD(kk, ptid)) mbar_arrive(sbase + 8 * s);
    }
    producers_sync();   // everybody has read the raw slot: the copy engine may overwrite it
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
}

// fp16 storage: loads, converts to fp32 and stores (the interleaved fp32 layout cannot be produced
// by an asynchronous copy of 2-byte elements).  The loads of a batch (two staged elements x 8
// channels x {A,B}) are issued before the previous batch is converted and stored, across chunk
// boundaries too, so a thread always has loads in flight; the ring slot is only waited for when a
// chunk's first store is due.  Returns false if a bounded wait ran out.
struct HalfBatch {
  uint32_t raw[2][kChunk];   // {A, B} halves of one staged element and channel
  uint32_t dst[2];           // byte offset in the channel's staged block, kSkipElem = none
};

template <int S, int R>
__device__ __forceinline__ bool produce_half_stream(const DeviceLayer& L, const Geo& g,
                                                    const __half* __restrict__ x, const SubTile* tab,
                                                    const StagedElem (&pre)[kPreElems], const uint4* desc,
                                                    const uint8_t* codes, uint32_t sbase, int k0, int nk,
                                                    int n_early, int ptid) {
  const size_t hw = (size_t)g.h * g.w;
  const int n_elem = g.pairs * g.rows * g.pitch;
  const int nb = ((n_elem + kProducerThreads - 1) / kProducerThreads + 1) / 2;  // batches per chunk
  const unsigned short* xs = reinterpret_cast<const unsigned short*>(x);
  auto issue = [&](HalfBatch& bt, int kk, int b) {
    const int c0 = (k0 + kk) * kChunk;
    const int nc = min(kChunk, L.c_in - c0);
    const size_t chan_off = (size_t)c0 * hw;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int i = 2 * b + u, e = ptid + i * kProducerThreads;
      StagedElem se;
      se.off_a = se.off_b = -1;
      se.dst = kSkipElem;
      if (e < n_elem) {
        if (i < kPreElems) {
#pragma unroll
          for (int j = 0; j < kPreElems; ++j)   // static indices keep `pre` in registers
            if (i == j) se = pre[j];
        } else {
          se = staged_elem<S, R>(L, g, tab, e, 0);
        }
      }
      bt.dst[u] = se.dst;
#pragma unroll
      for (int cc = 0; cc < kChunk; ++cc) {
        const uint32_t va = (se.off_a >= 0 && cc < nc) ? (uint32_t)__ldg(xs + se.off_a + chan_off + cc * hw) : 0u;
        const uint32_t vb = (se.off_b >= 0 && cc < nc) ? (uint32_t)__ldg(xs + se.off_b + chan_off + cc * hw) : 0u;
        bt.raw[u][cc] = va | (vb << 16);
      }
    }
  };
  auto store = [&](const HalfBatch& bt, uint32_t stage_base) {
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      if (bt.dst[u] == kSkipElem) continue;
#pragma unroll
      for (int cc = 0; cc < kChunk; ++cc) {
        const __half2 h = *reinterpret_cast<const __half2*>(&bt.raw[u][cc]);
        sts64f(stage_base + bt.dst[u] + (uint32_t)(cc * g.chan_stride), __low2float(h), __high2float(h));
      }
    }
  };
  HalfBatch cur, nxt;
  issue(cur, 0, 0);
  for (int kk = 0; kk < nk; ++kk) {
    const int s = kk % g.stages, it = kk / g.stages;
    const uint32_t stage_base = sbase + g.stage_off + s * g.stage_bytes;
    for (int b = 0; b < nb; ++b) {
      const bool last = b + 1 == nb;
      const int kk2 = last ? kk + 1 : kk, b2 = last ? 0 : b + 1;
      if (kk2 < nk) issue(nxt, kk2, b2);
      if (b == 0 && it > 0 && !mbar_wait(sbase + 8 * (kMaxStages + s), (it - 1) & 1, L.err, 1)) return false;
      store(cur, stage_base);
      cur = nxt;
    }
    if (kk >= n_early) stage_blocks_half(L, g, desc, codes, stage_base, kk, ptid);
    if (!PCONV_WITHHELD(kk, ptid)) mbar_arrive(sbase + 8 * s);
  }
  return true;
}


// Where a lane's outputs go: the element offsets (inside filter 0's plane of the A / B image) of
// row 0 of its two pixels, and which of the 2 R outputs lie inside the image and the batch
// (bit 2k = A row k, bit 2k+1 = B row k).  Rows are w_out elements apart.
struct LaneOut {
  long long base_a, base_b;
  uint32_t mask;
};
template <int R>
__device__ __forceinline__ LaneOut lane_outputs(const DeviceLayer& L, const Geo& g, const SubTile* tab,
                                                int slot, int col) {
  const SubTile A = tab[2 * slot], B = tab[2 * slot + 1];
  const int ox_a = A.x0 + col, ox_b = B.x0 + col;
  const bool col_a = A.valid && ox_a < g.w_out, col_b = B.valid && ox_b < g.w_out;
  const long long plane = (long long)g.h_out * g.w_out;
  LaneOut r;
  r.base_a = (long long)A.n * L.c_out * plane + (long long)A.y0 * g.w_out + ox_a;
  r.base_b = (long long)B.n * L.c_out * plane + (long long)B.y0 * g.w_out + ox_b;
  r.mask = 0;
#pragma unroll
  for (int k = 0; k < R; ++k) {
    if (col_a && A.y0 + k < g.h_out) r.mask |= 1u << (2 * k);
    if (col_b && B.y0 + k < g.h_out) r.mask |= 2u << (2 * k);
  }
  return r;
}

// The same for the pooled output: a lane in an even column writes, for each of its two pixels,
// the R / 2 pooled rows that its R conv rows give (bit 2j / 2j+1 = A / B pooled row j); rows are
// w_y elements apart.  A pooled position inside the pooled map has all four of its sources inside
// the conv map, so no source needs masking.
template <int R>
__device__ __forceinline__ LaneOut lane_outputs_pooled(const DeviceLayer& L, const Geo& g,
                                                       const SubTile* tab, int slot, int col) {
  const SubTile A = tab[2 * slot], B = tab[2 * slot + 1];
  const int px_a = (A.x0 + col) >> 1, px_b = (B.x0 + col) >> 1;
  const bool even = (col & 1) == 0;
  const bool col_a = even && A.valid && px_a < g.w_y, col_b = even && B.valid && px_b < g.w_y;
  const long long plane = (long long)g.h_y * g.w_y;
  LaneOut r;
  r.base_a = (long long)A.n * L.c_out * plane + (long long)(A.y0 >> 1) * g.w_y + px_a;
  r.base_b = (long long)B.n * L.c_out * plane + (long long)(B.y0 >> 1) * g.w_y + px_b;
  r.mask = 0;
#pragma unroll
  for (int k = 0; k < R / 2; ++k) {
    if (col_a && (A.y0 >> 1) + k < g.h_y) r.mask |= 1u << (2 * k);
    if (col_b && (B.y0 >> 1) + k < g.h_y) r.mask |= 2u << (2 * k);
  }
  return r;
}

template <bool HALF, bool RELU>
__device__ __forceinline__ void store_out(void* __restrict__ y, long long i, float v) {
  if (RELU) v = fmaxf(v, 0.f);
  if (HALF)
    ((__half*)y)[i] = __float2half_rn(v);
  else
    ((float*)y)[i] = v;
}

// Calls f with the storage type and the activation as compile-time flags.
template <class F>
__device__ __forceinline__ void with_flags(const Geo& g, F f) {
  if (g.is_half) {
    if (g.relu) f(std::true_type(), std::true_type()); else f(std::true_type(), std::false_type());
  } else {
    if (g.relu) f(std::false_type(), std::true_type()); else f(std::false_type(), std::false_type());
  }
}

__device__ __forceinline__ void red_add_v4(float* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("red.global.v4.f32.add [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(__uint_as_float(a)),
               "f"(__uint_as_float(b)), "f"(__uint_as_float(c)), "f"(__uint_as_float(d))
               : "memory");
}

// ---- thread-block clusters: the CTAs that share an output tile ---------------------------------------
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// The address, in the cluster's shared-memory window, of `addr` (a shared::cta address) in CTA `rank`.
__device__ __forceinline__ uint32_t cluster_map(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float4 ld_cluster_v4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "r"(addr));
  return v;
}

// The 2 R outputs of one filter slot.  MODE 0: y = act(v + bias); MODE 1: workspace += v, where
// `ws` points at this lane's 2 R floats of the slot in the warp's part of the workspace (the
// workspace is laid out for the warps that write and read it, not like y: [tile][warp][slot]
// [lane][2 R], so that a lane's partial sums go out as 16-byte reductions and come back as
// 16-byte loads; lanes and rows outside the image carry zeros or garbage that nobody uses).
template <int R, int MODE, bool HALF, bool RELU>
__device__ __forceinline__ void emit_slot(const Geo& g, const LaneOut& lo, void* __restrict__ y,
                                          float* __restrict__ ws, long long fbase, float bv,
                                          const uint32_t (&v)[2 * R]) {
  if (MODE == 1) {
#pragma unroll
    for (int i = 0; i < 2 * R; i += 4) red_add_v4(ws + i, v[i], v[i + 1], v[i + 2], v[i + 3]);
    return;
  }
  if (MODE == 2) {   // `ws` is a generic pointer into this CTA's shared memory (same layout)
#pragma unroll
    for (int i = 0; i < 2 * R; i += 4)
      *reinterpret_cast<uint4*>(ws + i) = make_uint4(v[i], v[i + 1], v[i + 2], v[i + 3]);
    return;
  }
  const long long ia = fbase + lo.base_a, ib = fbase + lo.base_b;
#pragma unroll
  for (int k = 0; k < R; ++k) {
    const int row = k * g.w_out;
    if (lo.mask >> (2 * k) & 1u) store_out<HALF, RELU>(y, ia + row, __uint_as_float(v[2 * k]) + bv);
    if (lo.mask >> (2 * k + 1) & 1u) store_out<HALF, RELU>(y, ib + row, __uint_as_float(v[2 * k + 1]) + bv);
  }
}

// 2x2 max over a slot's 2 R values (rows pairwise inside the lane, columns with the neighbour
// lane), bias and activation after the max (both are monotone), stored by the even lane.  Must be
// called by the whole warp.
template <int R, bool HALF, bool RELU>
__device__ __forceinline__ void emit_slot_pooled(const Geo& g, const LaneOut& lp, void* __restrict__ y,
                                                 long long fbase, float bv, const float (&v)[2 * R]) {
  float m[R];
#pragma unroll
  for (int j = 0; j < R / 2; ++j) {
    m[2 * j] = fmaxf(v[4 * j], v[4 * j + 2]);
    m[2 * j + 1] = fmaxf(v[4 * j + 1], v[4 * j + 3]);
  }
#pragma unroll
  for (int i = 0; i < R; ++i) m[i] = fmaxf(m[i], __shfl_xor_sync(0xffffffffu, m[i], 1));
  const long long ia = fbase + lp.base_a, ib = fbase + lp.base_b;
#pragma unroll
  for (int j = 0; j < R / 2; ++j) {
    if (lp.mask >> (2 * j) & 1u) store_out<HALF, RELU>(y, ia + j * g.w_y, m[2 * j] + bv);
    if (lp.mask >> (2 * j + 1) & 1u) store_out<HALF, RELU>(y, ib + j * g.w_y, m[2 * j + 1] + bv);
  }
}

// Which accumulators a consumer warp writes out: filter slots [a0, a1) of the `zs` column sets
// that start at TMEM address `t0` (16 slots x 2 R columns apart), summed.  zs = 1: the warp's own 16 slots.
struct OutRange {
  uint32_t t0;
  int zs, a0, a1;
};

// 16 / R filter slots of a lane's accumulators, summed over the warps that split the channels.
template <int R>
__device__ __forceinline__ void tmem_sum_slots(uint32_t (&v)[16 / R][2 * R], const OutRange& r, int a) {
  constexpr int kB = 16 / R, kNV = 2 * R;
#pragma unroll
  for (int b = 0; b < kB; ++b) tmem_ld_slot_nowait<kNV>(v[b], r.t0 + (a + b) * kNV);
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll 1
  for (int j = 1; j < r.zs; ++j) {
    uint32_t t[kB][kNV];
#pragma unroll
    for (int b = 0; b < kB; ++b) tmem_ld_slot_nowait<kNV>(t[b], r.t0 + j * (kGroup * kNV) + (a + b) * kNV);
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int b = 0; b < kB; ++b)
#pragma unroll
      for (int e = 0; e < kNV; ++e)
        v[b][e] = __float_as_uint(__uint_as_float(v[b][e]) + __uint_as_float(t[b][e]));
  }
}

// Outputs of one consumer warp (filter slots x R rows x {A,B} per lane).  `my_o` / `my_b` hold, in
// lane a < 16, the original filter index and the bias of slot a (loaded at kernel start).
template <int R, bool GENERIC, int MODE, bool HALF, bool RELU>
__device__ __forceinline__ void write_outputs(const Geo& g, const LaneOut& lo, const LaneOut& lp,
                                              void* __restrict__ y, float* __restrict__ ws,
                                              const u64 (&acc)[GENERIC ? kGroup : 1][4],
                                              const OutRange& r, int my_o, float my_b) {
  constexpr int kNV = 2 * R;
  const long long plane = (long long)g.h_out * g.w_out;
  const long long plane_y = (long long)g.h_y * g.w_y;
  // one filter slot: plain stores / atomics, or the fused 2x2 max-pool (warp-uniform choice)
  auto emit = [&](int o, float bv, const uint32_t (&v)[kNV]) {
    if (MODE == 0 && g.pool) {
      float f[kNV];
#pragma unroll
      for (int e = 0; e < kNV; ++e) f[e] = __uint_as_float(v[e]);
      emit_slot_pooled<R, HALF, RELU>(g, lp, y, (long long)o * plane_y, bv, f);
    } else {
      emit_slot<R, MODE, HALF, RELU>(g, lo, y, ws, (long long)o * plane, bv, v);
    }
  };
  // MODE 1 / 2: `ws` is the lane's first float of the warp's first slot (r.a0); slots are 32 x 2 R floats apart
  auto emit_ws = [&](int a, const uint32_t (&v)[kNV]) {
    emit_slot<R, MODE, false, false>(g, lo, y, ws + (size_t)(a - r.a0) * (32 * kNV), 0, 0.f, v);
  };
  if constexpr (GENERIC) {
    static_assert(!GENERIC || R == 4, "register accumulators hold 4 rows");
#pragma unroll
    for (int a = 0; a < kGroup; ++a) {
      uint32_t v[kNV];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        v[2 * k] = (uint32_t)acc[a][k];
        v[2 * k + 1] = (uint32_t)(acc[a][k] >> 32);
      }
      const int o = __shfl_sync(0xffffffffu, my_o, a);
      const float bv = __shfl_sync(0xffffffffu, my_b, a);
      if (o >= 0) emit(o, bv, v);
    }
  } else {
    constexpr int kB = 16 / R;
#pragma unroll 1
    for (int a = r.a0; a < r.a1; a += kB) {  // run-time TMEM addresses: several slots per round trip
      uint32_t v[kB][kNV];
      tmem_sum_slots<R>(v, r, a);
#pragma unroll
      for (int b = 0; b < kB; ++b) {
        const int o = __shfl_sync(0xffffffffu, my_o, a + b);
        const float bv = __shfl_sync(0xffffffffu, my_b, a + b);
        if (o >= 0) {
          if (MODE != 0) emit_ws(a + b, v[b]);
          else emit(o, bv, v[b]);
        }
      }
    }
  }
}

// The last split to finish a warp's part of an output tile: workspace -> y, leaving the workspace
// zeroed.  `ws` is the lane's first float of the warp's first slot (a_begin); a slot's 2 R sums
// come back as 16-byte loads, 16 / R slots (eight loads per lane) in flight at once.
template <int R, bool HALF, bool RELU>
__device__ __forceinline__ void finalize_outputs(const Geo& g, const LaneOut& lo, const LaneOut& lp,
                                                 void* __restrict__ y, float* __restrict__ ws,
                                                 int a_begin, int a_end, int my_o, float my_b) {
  const long long plane = (long long)g.h_out * g.w_out;
  const long long plane_y = (long long)g.h_y * g.w_y;
  constexpr int kBatch = 16 / R, kNV = 2 * R;
#pragma unroll 1
  for (int a0 = a_begin; a0 < a_end; a0 += kBatch) {
    float v[kBatch][kNV];
    int fo[kBatch];
    float bv[kBatch];
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      fo[b] = __shfl_sync(0xffffffffu, my_o, a0 + b);
      bv[b] = __shfl_sync(0xffffffffu, my_b, a0 + b);
      float4* p = reinterpret_cast<float4*>(ws + (size_t)(a0 + b - a_begin) * (32 * kNV));
#pragma unroll
      for (int i = 0; i < kNV / 4; ++i) {
        const float4 q = (fo[b] < 0) ? make_float4(0.f, 0.f, 0.f, 0.f) : __ldcg(p + i);
        v[b][4 * i] = q.x; v[b][4 * i + 1] = q.y; v[b][4 * i + 2] = q.z; v[b][4 * i + 3] = q.w;
      }
    }
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      if (fo[b] < 0) continue;
      float4* p = reinterpret_cast<float4*>(ws + (size_t)(a0 + b - a_begin) * (32 * kNV));
#pragma unroll
      for (int i = 0; i < kNV / 4; ++i) p[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (g.pool) {
        emit_slot_pooled<R, HALF, RELU>(g, lp, y, (long long)fo[b] * plane_y, bv[b], v[b]);
        continue;
      }
      const long long fb = (long long)fo[b] * plane;
      const long long ia = fb + lo.base_a, ib = fb + lo.base_b;
#pragma unroll
      for (int k = 0; k < R; ++k) {
        const int row = k * g.w_out;
        if (lo.mask >> (2 * k) & 1u) store_out<HALF, RELU>(y, ia + row, v[b][2 * k] + bv[b]);
        if (lo.mask >> (2 * k + 1) & 1u) store_out<HALF, RELU>(y, ib + row, v[b][2 * k + 1] + bv[b]);
      }
    }
  }
}

// Cluster form of the channel split: every CTA of a tile's cluster leaves the partial sums of its
// warps in its own shared memory at `part` ([warp][slot][lane][2 R], the workspace layout); the
// slot parts of the tile are dealt to the cluster's warps (part sp -> rank sp % ks, warp
// sp / ks % CW), and a warp adds a part up over the ranks in rank order -- so the sums do not
// depend on timing -- through distributed shared memory, applies bias / ReLU (pools) and writes y.
constexpr int kMaxClusterParts = 4;   // slot parts a warp may be dealt: CW * 16 / zs parts over ks * CW warps, ks >= 2, zs >= 2
struct ClusterPart {
  int sp, o;       // slot part (-1 = none) and the original filter index of its slot (-1 = padding)
  float bv;        // the filter's bias
  int slot2;       // sub-tile pair of this lane in the part's pixel set
};
// What a warp will add up, worked out (and its filter indices and biases fetched) before the
// CTAs meet, while the slower warps still compute.
template <int R, int CW>
__device__ __forceinline__ void cluster_parts(ClusterPart (&cp)[kMaxClusterParts], const DeviceLayer& L,
                                              const Geo& g, const float* __restrict__ bias, int group0,
                                              int rank, int warp, int lane) {
  const int zs = g.zs, spw = kGroup / zs, n_sp = CW * spw;
#pragma unroll
  for (int i = 0; i < kMaxClusterParts; ++i) {
    const int sp = rank + g.ks * (warp + CW * i);
    cp[i].sp = -1;
    cp[i].o = -1;
    cp[i].bv = 0.f;
    cp[i].slot2 = 0;
    if (sp >= n_sp) continue;
    const int w2 = sp / spw, j = sp - w2 * spw;        // the warp that holds this part in every rank
    int unit2 = w2, z2 = 0;
    if (zs > 1) {
      z2 = (w2 >> 2) % zs;
      unit2 = (w2 & 3) + 4 * ((w2 >> 2) / zs);
    }
    const int wyi2 = unit2 % g.wys, gi2 = group0 + unit2 / g.wys;
    if (wyi2 >= g.wy || gi2 >= L.n_groups) continue;
    cp[i].sp = sp;
    cp[i].o = __ldg(L.perm + gi2 * kGroup + z2 * spw + j);
    cp[i].slot2 = wyi2 * g.sw + lane / g.tw;
  }
#pragma unroll
  for (int i = 0; i < kMaxClusterParts; ++i)
    if (cp[i].o >= 0 && bias) cp[i].bv = __ldg(bias + cp[i].o);
}

template <int R, bool HALF, bool RELU>
__device__ __forceinline__ void cluster_reduce_emit(const DeviceLayer& L, const Geo& g, const SubTile* tab,
                                                    void* __restrict__ y, uint32_t part,
                                                    const ClusterPart (&cp)[kMaxClusterParts], int lane) {
  constexpr int kNV = 2 * R;
  const long long plane = (long long)g.h_out * g.w_out;
  const long long plane_y = (long long)g.h_y * g.w_y;
#pragma unroll
  for (int i = 0; i < kMaxClusterParts; ++i) {
    if (cp[i].o < 0) continue;
    const uint32_t off = part + (uint32_t)((cp[i].sp * 32 + lane) * kNV * 4);
    float v[kNV];
#pragma unroll
    for (int e = 0; e < kNV; ++e) v[e] = 0.f;
#pragma unroll 4
    for (int q = 0; q < g.ks; ++q) {
      const uint32_t ra = cluster_map(off, (uint32_t)q);
#pragma unroll
      for (int k = 0; k < kNV; k += 4) {
        const float4 t = ld_cluster_v4(ra + k * 4);
        v[k] += t.x; v[k + 1] += t.y; v[k + 2] += t.z; v[k + 3] += t.w;
      }
    }
    const int col = lane % g.tw;
    if (g.pool) {
      const LaneOut lp = lane_outputs_pooled<R>(L, g, tab, cp[i].slot2, col);
      emit_slot_pooled<R, HALF, RELU>(g, lp, y, (long long)cp[i].o * plane_y, cp[i].bv, v);
    } else {
      const LaneOut lo = lane_outputs<R>(L, g, tab, cp[i].slot2, col);
      uint32_t u[kNV];
#pragma unroll
      for (int e = 0; e < kNV; ++e) u[e] = __float_as_uint(v[e]);
      emit_slot<R, 0, HALF, RELU>(g, lo, y, nullptr, (long long)cp[i].o * plane, cp[i].bv, u);
    }
  }
}

// Where a CTA stands in a layer's grid (a chain kernel gives every layer its own virtual grid).
struct BlockPos {
  int x, y, z, gx;
};
// A layer inside a chain kernel (several layers of a stack in one persistent launch, one CTA per
// SM): Tensor Memory is allocated once by the chain kernel and kept across layers; a CTA that has
// finished its part of a layer counts itself in `sync` and goes on to the next layer's set-up
// and weight blocks at once, and waits for `target` arrivals -- every CTA's part of the previous
// layer -- only where a stand-alone kernel waits for the previous kernel of the stream.
struct ChainCtx {
  unsigned int* sync;     // nullptr: a stand-alone launch of one layer
  unsigned int target;    // 0: the chain's first layer (waits for the previous kernel instead)
  int own_tmem;           // 1: the body allocates and releases Tensor Memory (stand-alone launch)
  int reinit;             // 1: the CTA's barriers were used by an earlier layer: invalidate them first
};
constexpr uint32_t kGridSpinLimit = 1u << 21;

// What a role does before it first touches activations, workspace or tickets: wait for the
// previous kernel of the stream or, inside a chain, for the previous layer.  Bounded: false (and
// wait id 9 recorded) if the other CTAs never arrive.
__device__ __forceinline__ bool dependency_wait(const ChainCtx& cc, int lane, int warp, unsigned char* smem,
                                                int* err) {
  if (cc.sync == nullptr || cc.target == 0) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    return true;
  }
  // One warp of the CTA polls the grid's counter (every warp of every CTA polling the same word
  // kept the arrivals themselves waiting); the others watch a word in shared memory that it sets.
  volatile uint32_t* seen_s = reinterpret_cast<volatile uint32_t*>(smem + 8 * 2 * kMaxStages + 4);
  uint32_t ok = 1;
  if (lane == 0) {
    uint32_t it = 0, seen = 0;
    if (warp == 0) {
      for (;;) {
        asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(cc.sync) : "memory");
        if (seen >= cc.target) break;
        if (++it > kGridSpinLimit) {
          atomicCAS(err, 0, 9);
          ok = 0;
          seen = 0xFFFFFFFFu;      // releases the CTA's other warps, which then find the status set
          break;
        }
        __nanosleep(100);
      }
      // acquire once, after the count has been seen (an acquiring load in the polling loop costs
      // the SM an L1 invalidation per try), then tell the CTA's other warps
      asm volatile("fence.acq_rel.gpu;" ::: "memory");
      *seen_s = seen;
    } else {
      for (;;) {
        seen = *seen_s;
        if (seen >= cc.target) break;
        if (++it > (kGridSpinLimit << 2)) {
          atomicCAS(err, 0, 9);
          break;
        }
        __nanosleep(40);
      }
      if (seen == 0xFFFFFFFFu || seen < cc.target) ok = 0;
      asm volatile("fence.acq_rel.cta;" ::: "memory");   // order this warp's reads after the flag's value
    }
  }
  ok = __shfl_sync(0xffffffffu, ok, 0);
  return ok != 0;
}

template <int S, bool GENERIC, bool WIDE, int R>
__device__ __forceinline__ void tiled_body(const DeviceLayer& L, const Geo& g, const void* __restrict__ x,
                                           const float* __restrict__ bias, void* __restrict__ y,
                                           float* __restrict__ ws, int* __restrict__ counters,
                                           unsigned char* smem, const BlockPos bp, const ChainCtx cc) {
  static_assert(R == 4 || (R == 8 && !GENERIC && !WIDE), "8 rows per lane: canonical TMEM bodies only");
  constexpr int kCW = consumer_warps(GENERIC, R);
  constexpr int kThreads = cta_threads(GENERIC, R);
  constexpr int kNV = 2 * R;              // TMEM columns of one filter slot
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31;
  // broadcast from lane 0: tells the compiler that everything derived from it is warp-uniform
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  SubTile* tab = reinterpret_cast<SubTile*>(smem + g.tab_off);
  volatile uint32_t* tmem_base_s = reinterpret_cast<volatile uint32_t*>(smem + 8 * 2 * kMaxStages);
  int* unit_ctr = reinterpret_cast<int*>(smem + 8 * 2 * kMaxStages + 16);  // next chunk of each unit

  PCONV_MARK(0)
  PCONV_MARK_MAX(8)
  // The next kernel of the stream may start its own set-up while this one runs (it waits for this
  // grid to finish before it touches activations, see below).
  if (cc.own_tmem) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid < kCW) unit_ctr[tid] = 0;
  const uint32_t coop_bar = sbase + 8 * 2 * kMaxStages + 16 + 64;   // kMaxCoop barriers
  const uint32_t raw_bar0 = coop_bar + 8 * kMaxCoop;                // kRawStages barriers (bulk copies of a raw slot)
  if (tid == 0) {
    // every barrier is initialised, used or not, so that a chain's next layer may invalidate
    // and initialise them all again (its ring may be deeper)
    if (cc.reinit)
      for (int j = 0; j < 2 * kMaxStages + 2 + 8 + kMaxCoop + kRawStages; ++j)
        if (j < 2 * kMaxStages || j >= 2 * kMaxStages + 10)
          asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(sbase + 8 * j) : "memory");
    for (int j = 0; j < kMaxCoop; ++j) mbar_init(coop_bar + 8 * j, 32 * kCW);
    for (int j = 0; j < kRawStages; ++j) mbar_init(raw_bar0 + 8 * j, kProducerThreads);
    for (int s = 0; s < kMaxStages; ++s) {
      mbar_init(sbase + 8 * s, 32 * kProducerWarps);
      mbar_init(sbase + 8 * (kMaxStages + s), kCW / (GENERIC ? 1 : g.zs));
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (!GENERIC && warp == 0 && cc.own_tmem) {  // the whole TMEM of this SM (one CTA per SM by shared-memory use)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32((const void*)tmem_base_s)),
                 "n"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int i = tid; i < 2 * g.pairs; i += kThreads) {
    const long long q = (long long)bp.x * (2 * g.pairs) + i;
    SubTile t;
    t.valid = q < g.q_total;
    const int qq = t.valid ? (int)q : 0;
    const int per_img = g.tx * g.ty;
    t.n = qq / per_img;
    const int rem = qq - t.n * per_img;
    const int tyi = rem / g.tx;
    t.y0 = tyi * R;
    t.x0 = (rem - tyi * g.tx) * g.tw;
    tab[i] = t;
  }
  const int k0 = bp.z * g.cps;                             // this CTA's chunk range
  const int nk = min(L.n_chunks, k0 + g.cps) - k0;
  // Block descriptors of the CTA's groups and chunks, two 16-byte words each:
  // {first kernel record, records, code offset, code bytes}, {-, -, first channel, -}.
  uint4* desc = reinterpret_cast<uint4*>(smem + g.desc_off);
  for (int i = tid; i < g.ng * g.cps; i += kThreads) {
    const int j = i / g.cps, kk = i - j * g.cps;
    const int gj = bp.y * g.ng + j;
    uint4 d0 = make_uint4(0u, 0u, 0u, 0u), d1 = d0;
    if (gj < L.n_groups && kk < nk) {
      const uint4* src = reinterpret_cast<const uint4*>(L.blocks + (size_t)gj * L.n_chunks + k0 + kk);
      const uint4 b0 = __ldg(src), b1 = __ldg(src + 1);
      d0 = GENERIC ? make_uint4(b0.x, b0.y, b1.x, b1.y) : b0;
      d1 = b1;
    }
    desc[2 * i] = d0;
    desc[2 * i + 1] = d1;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  // Everything above reads only the packed layer.  When launched with programmatic stream
  // serialisation the kernel has started before the previous one in the stream finished: each
  // role waits for it (griddepcontrol.wait) below, after what it can do from the packed layer
  // alone and before x or the bias is read and y, workspace or tickets are written.
  PCONV_MARK(1)
  const uint32_t tmem_base = GENERIC ? 0u : *tmem_base_s;

  // Consumer-warp coordinates (meaningless for producer warps).  zs warps of one TMEM lane
  // quadrant form a unit: they work on the same pixels and filter group and take the chunks in
  // turn, each with accumulators in its own 16 x 2 R TMEM columns.
  const int zs = GENERIC ? 1 : g.zs;
  int unit = warp, z = 0;
  if (zs > 1) {
    z = (warp >> 2) % zs;
    unit = (warp & 3) + 4 * ((warp >> 2) / zs);
  }
  const int wyi = unit % g.wys, wgi = unit / g.wys;
  const int gi = bp.y * g.ng + wgi;
  const bool active = (wyi < g.wy) && (gi < L.n_groups);
  const int slot = wyi * g.sw + lane / g.tw;  // sub-tile pair of this lane
  const int col = lane % g.tw;
  const uint32_t col_b = (uint32_t)g.colstride;
  const uint32_t off_mid = (S == 1) ? col_b : (uint32_t)(g.tw + 1) * col_b;  // window column 1
  const uint32_t off_right = (S == 1) ? 2 * col_b : col_b;                   // window column 2
  const uint32_t chan_b = (uint32_t)g.chan_stride;
  const uint32_t lane_off = (uint32_t)(slot * g.substride) + (uint32_t)col * col_b;
  // TMEM: a warp reaches the 32 lanes of its quadrant (warp % 4); the 4 (R = 4) or 2 (R = 8) warps
  // of a quadrant take 128 or 256 columns each = 16 filter slots x (R rows x {A,B}).
  const uint32_t tquad = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16);
  const uint32_t tq = tquad + (uint32_t)((warp >> 2) * (kGroup * kNV));

  // lane a < 16 keeps the original filter index and bias of slot a for the epilogue
  int my_o = -1;
  float my_b = 0.f;
  if (warp < kCW && active && lane < kGroup) my_o = __ldg(L.perm + gi * kGroup + lane);
  u64 acc[GENERIC ? kGroup : 1][4];
  bool ok = true;
  // fp32 element-wise staging: the consumer warps copy the x part of the first chunks themselves
  // (one per warp of a unit), the producers only their weight blocks
  const int n_coop = (!g.is_half && g.raw_stages == 0) ? min(min(zs, g.stages), min(nk, kMaxCoop)) : 0;

  if (warp >= kCW) {
    // ===================================== producer warps =====================================
    const int ptid = (warp - kCW) * 32 + lane;
    const uint8_t* codes = GENERIC ? L.codes_g : L.codes_s;
    StagedElem pre[kPreElems];
    if (g.raw_mode >= 2) {
      const int n_elem = g.pairs * g.rows * g.pitch;
#pragma unroll
      for (int i = 0; i < kPreElems; ++i) {
        const int e = ptid + i * kProducerThreads;
        pre[i] = bulk_elem<S, R>(g, tab, e < n_elem ? e : 0);
        if (e >= n_elem) pre[i].dst = kSkipElem;
      }
      if (dependency_wait(cc, lane, warp, smem, L.err))
        produce_bulk_stream<S, R>(L, g, (const float*)x, tab, pre, desc, codes, sbase, raw_bar0, k0, nk, ptid);
    } else if (g.raw_stages > 0) {
      const int n_elem = g.pairs * g.rows * g.pitch;
#pragma unroll
      for (int i = 0; i < kPreElems; ++i) {
        const int e = ptid + i * kProducerThreads;
        pre[i] = raw_elem<S, R>(g, e < n_elem ? e : 0);
        if (e >= n_elem) pre[i].dst = kSkipElem;
      }
      if (dependency_wait(cc, lane, warp, smem, L.err))
        produce_raw_stream<S, R>(L, g, (const __half*)x, tab, pre, desc, codes, sbase, k0, nk, ptid);
    } else {
      precompute_elems<S, R>(pre, L, g, tab, ptid);
      // the weight records and codes of the first ring-full of chunks do not depend on the previous
      // kernel: fetch them while it finishes
      const int n_early = min(g.stages, nk);
      for (int kk = 0; kk < n_early; ++kk) {
        const uint32_t stage_base = sbase + g.stage_off + kk * g.stage_bytes;
        if (g.is_half) stage_blocks_half(L, g, desc, codes, stage_base, kk, ptid);
        else stage_blocks_async(L, g, desc, codes, stage_base, kk, ptid);
        // chunks whose x the consumers copy are complete, for the producers, once their blocks have
        // landed: arrive now, so that the barrier does not also wait for the later chunks' blocks
        if (kk < n_coop && !PCONV_WITHHELD(kk, ptid)) cp_async_arrive(sbase + 8 * kk);
      }
      if (!dependency_wait(cc, lane, warp, smem, L.err)) {
        // the previous layer never completed: nothing more is staged, the consumers give up too
      } else if (g.is_half) {
        produce_half_stream<S, R>(L, g, (const __half*)x, tab, pre, desc, codes, sbase, k0, nk, n_early, ptid);
      } else {
        for (int kk = n_coop; kk < nk; ++kk) {
          const int s = kk % g.stages, it = kk / g.stages;
          if (it > 0 && !mbar_wait(sbase + 8 * (kMaxStages + s), (it - 1) & 1, L.err, 1)) break;
          const uint32_t stage_base = sbase + g.stage_off + s * g.stage_bytes;
          produce_chunk_async<S, R>(L, g, (const float*)x, tab, pre, desc, codes, stage_base, k0 + kk, kk, ptid,
                                 true, kk >= n_early);
          if (!PCONV_WITHHELD(kk, ptid)) cp_async_arrive(sbase + 8 * s);
        }
      }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
  } else {
    // ===================================== consumer warps =====================================
    if constexpr (GENERIC) {
#pragma unroll
      for (int a = 0; a < kGroup; ++a)
#pragma unroll
        for (int k = 0; k < 4; ++k) acc[a][k] = 0ull;
    } else {
      for (int a = 0; a < kGroup * kNV; a += 8) tmem_st8_zero(tq + a);
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    ok = dependency_wait(cc, lane, warp, smem, L.err);
    // (each consumer thread arrives on the chunk's own barrier when its copies for that chunk
    // have landed; a warp waits for that barrier as well as for the producers' before the chunk)
    for (int kk = 0; ok && kk < n_coop; ++kk) {
      fill_chunk_x<S, R>(L, g, (const float*)x, tab, sbase + g.stage_off + kk * g.stage_bytes, k0 + kk,
                      warp * 32 + lane, 32 * kCW);
      cp_async_arrive(coop_bar + 8 * kk);
    }
    if (bias && my_o >= 0) my_b = __ldg(bias + my_o);

#ifdef PCONV_DEV
    long long t_wait = 0, t_work = 0;
#endif
    // The warps of a unit draw the chunks from the unit's counter, so a warp that got a heavier
    // chunk (or started later) simply takes fewer -- or, when reproducible sums are asked for,
    // take them in turn (warp z: chunks z, z + zs, ...; the ring depth is then a multiple of zs,
    // so a slot always comes back to the same warps).
    int next_kk = 0;
    while (ok) {
      int kk = next_kk++;
      if (zs > 1) {
        if (g.fixed_turns) {
          kk = z + kk * zs;
        } else {
          if (lane == 0) kk = atomicAdd(unit_ctr + unit, 1);
          kk = __shfl_sync(0xffffffffu, kk, 0);
        }
      }
      if (kk >= nk) break;
      const int s = kk % g.stages;
#ifdef PCONV_DEV
      const long long tc0 = clock64();
#endif
      ok = mbar_wait(sbase + 8 * s, (kk / g.stages) & 1, L.err, 2);
      if (ok && kk < n_coop) ok = mbar_wait(coop_bar + 8 * kk, 0, L.err, 3);
      if (!ok) break;
#ifdef PCONV_DEV
      const long long tc1 = clock64();
#endif
      if (next_kk == 1) { PCONV_MARK(2) }   // this warp's first chunk has landed
      if (active) {
        const uint32_t stage_base = sbase + g.stage_off + s * g.stage_bytes;
        uint32_t xptr = stage_base + lane_off - chan_b;  // one channel before the chunk
        uint32_t wp = stage_base + g.x_stage_bytes + wgi * kWSlot;
        uint32_t cp = stage_base + g.x_stage_bytes + g.ng * kWSlot + wgi * kCodeSlot;
        if constexpr (!GENERIC) {
          const uint4 d0 = desc[2 * (wgi * g.cps + kk)], d1 = desc[2 * (wgi * g.cps + kk) + 1];
          if (d0.y) {  // the block has kernels: enter at its first channel
            if constexpr (WIDE) dispatch_chunk_wide<S>(cp, wp, xptr, chan_b, col_b, off_mid, tq, (d1.z + 1u) << 8);
            else dispatch_chunk<S, R>(cp, wp, xptr, chan_b, col_b, off_mid, tq, (d1.z + 1u) << 4);
          }
        } else {
          u64 win[Win<S>::kRows][3];
#pragma unroll
          for (int r = 0; r < Win<S>::kRows; ++r) win[r][0] = win[r][1] = win[r][2] = 0ull;
          for (;;) {
            const uint32_t code = lds_u16(cp);
            cp += 2;
            if (code & (uint32_t)kGenEnd) break;
            if (code & (uint32_t)kGenNext) {
              xptr += ((code & 0xFFu) + 1u) * chan_b;
              load_window<S>(win, xptr, off_mid, off_right);
              continue;
            }
            switch (code >> 9) {
              PG_CASES8(0) PG_CASES8(8)
              default: break;
            }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(sbase + 8 * (kMaxStages + s));
      __syncwarp();
#ifdef PCONV_DEV
      t_wait += tc1 - tc0;
      t_work += clock64() - tc1;
#endif
    }
#ifdef PCONV_DEV
    if (threadIdx.x == 0 && bp.x == 0 && bp.y == 0 && bp.z == 0) {
      trace_words(L)[11] = (unsigned long long)t_wait;
      trace_words(L)[12] = (unsigned long long)t_work;
      trace_words(L)[13] = (unsigned long long)nk;
    }
#endif

    PCONV_MARK(3)
    PCONV_MARK_MAX(9)
    // ---- epilogue: final values straight to y, or partial sums into the workspace --------------
    OutRange orng;
    orng.t0 = tq;
    orng.zs = 1;
    orng.a0 = 0;
    orng.a1 = kGroup;
    if constexpr (!GENERIC) {
      if (zs > 1) {
        // The warps of a unit hold partial sums over the chunks they drew in their own TMEM columns
        // of the same lanes; once all have finished, each adds up and writes 16 / zs filter slots.
        // (a barrier of the unit's own zs warps: units do not wait for one another)
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("bar.sync %0, %1;" ::"r"(3 + unit), "r"(32 * zs) : "memory");
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        orng.t0 = tquad + (uint32_t)(((warp >> 2) - z) * (kGroup * kNV));
        orng.zs = zs;
        orng.a0 = z * (kGroup / zs);
        orng.a1 = orng.a0 + kGroup / zs;
      }
    }
    if (!GENERIC && g.cluster) {
      // the partial sums overwrite the staging ring: wait until every consumer warp of the CTA has
      // left its loop (all chunks consumed, so the producers' copies have all landed too)
      asm volatile("bar.sync 1, %0;" ::"n"(32 * kCW) : "memory");
    }
    if (active && ok) {
      const LaneOut lo = lane_outputs<R>(L, g, tab, slot, col);
      const LaneOut lp = g.pool ? lane_outputs_pooled<R>(L, g, tab, slot, col) : lo;
      bool split = false;
      if constexpr (!GENERIC) split = g.ks > 1;
      if (!split) {
        with_flags(g, [&](auto half, auto relu) {
          write_outputs<R, GENERIC, 0, decltype(half)::value, decltype(relu)::value>(g, lo, lp, y, ws, acc,
                                                                                      orng, my_o, my_b);
        });
      } else if (g.cluster) {
        // cluster form: the warp's partial sums go to this CTA's shared memory (the staging ring is
        // free: every consumer warp has passed the barrier above), in the workspace layout
        const int spw = kGroup / (GENERIC ? 1 : g.zs);
        float* part = reinterpret_cast<float*>(smem + g.stage_off) + ((size_t)(warp * spw) * 32 + lane) * kNV;
        write_outputs<R, GENERIC, 2, false, false>(g, lo, lp, y, part, acc, orng, my_o, my_b);
      } else {
        // this lane's floats in the warp's part of the tile's workspace: [tile][warp][slot][lane][2 R]
        const int spw = kGroup / (GENERIC ? 1 : g.zs);   // slots a warp writes out
        float* wsl = ws + ((((size_t)bp.y * bp.gx + bp.x) * kCW + warp) * spw * 32 + lane) * kNV;
        write_outputs<R, GENERIC, 1, false, false>(g, lo, lp, y, wsl, acc, orng, my_o, my_b);
        PCONV_MARK(4)
        PCONV_MARK_MAX(10)
        // Every warp owns the same part of the output tile in each of the ks splits, and takes a
        // ticket for that part once its partial sums are visible.  The warp that draws the last
        // ticket turns the summed partials into the layer's output and leaves workspace and
        // ticket zeroed for the next launch; nobody waits for anybody, and the finishing work of a
        // tile spreads over the CTAs that share it.
        // (one release-acquire atomic by lane 0 after the warp has synchronised: the release covers
        // the whole warp's partial sums, the acquire orders the last arriver's reads after every
        // other split's release)
        __syncwarp();
        int* ticket = counters + ((size_t)bp.y * bp.gx + bp.x) * kCW + warp;
        int t = 0;
        if (lane == 0) {
          asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(t) : "l"(ticket) : "memory");
          if (t == g.ks - 1) *ticket = 0;
        }
        t = __shfl_sync(0xffffffffu, t, 0);
        __syncwarp();
        if (t == g.ks - 1) {
          with_flags(g, [&](auto half, auto relu) {
            finalize_outputs<R, decltype(half)::value, decltype(relu)::value>(g, lo, lp, y, wsl, orng.a0,
                                                                             orng.a1, my_o, my_b);
          });
        }
      }
    }
    PCONV_MARK(5)
  }

  // ---- cluster form of the channel split: all warps of all CTAs of the tile meet twice ------------
  if constexpr (!GENERIC) {
    if (g.cluster) {
      ClusterPart cparts[kMaxClusterParts];
      if (warp < kCW) cluster_parts<R, kCW>(cparts, L, g, bias, bp.y * g.ng, bp.z, warp, lane);
      PCONV_MARK(4)
      PCONV_MARK_MAX(10)
      cluster_sync_all();          // every CTA's partial sums are in its shared memory
      if (warp < kCW) {
        with_flags(g, [&](auto half, auto relu) {
          cluster_reduce_emit<R, decltype(half)::value, decltype(relu)::value>(
              L, g, tab, y, sbase + (uint32_t)g.stage_off, cparts, lane);
        });
      }
      PCONV_MARK(5)
      cluster_sync_all();          // nobody leaves while a peer may still read its shared memory
    }
  }

  // ---- common exit: every warp arrives here, then the TMEM columns are handed back ---------------
  if constexpr (!GENERIC) {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    PCONV_MARK(6)
    if (warp == 0 && cc.own_tmem)
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "n"(kTmemCols)
                   : "memory");
  }
  PCONV_MARK_MAX(7)
}

template <int S, bool GENERIC, bool WIDE, int R>
__global__ void __launch_bounds__(cta_threads(GENERIC, R), 1)
tiled_kernel(const DeviceLayer L, const Geo g, const void* __restrict__ x,
             const float* __restrict__ bias, void* __restrict__ y, float* __restrict__ ws,
             int* __restrict__ counters) {
  extern __shared__ __align__(16) unsigned char smem[];
  BlockPos bp;
  bp.x = (int)blockIdx.x;
  bp.y = (int)blockIdx.y;
  bp.z = (int)blockIdx.z;
  bp.gx = (int)gridDim.x;
  ChainCtx cc;
  cc.sync = nullptr;
  cc.target = 0;
  cc.own_tmem = 1;
  cc.reinit = 0;
  tiled_body<S, GENERIC, WIDE, R>(L, g, x, bias, y, ws, counters, smem, bp, cc);
}

// One layer of a chain, as the chain kernel reads it from device memory.
struct ChainLayer {
  DeviceLayer L;
  Geo g;
  const void* x;
  const float* bias;
  void* y;
  int gx, gy, gz;     // the layer's own grid: CTA c works at (c % gx, c / gx % gy, c / (gx * gy)) if c < gx * gy * gz
  int pad;
};

// Several consecutive layers of a stack in one persistent launch (canonical pattern sets, stride
// 1; one CTA per SM, every layer's grid no larger than the launch's).  `sync` = {arrivals,
// CTAs that have left}: both zero before the launch and zero again after it.
__global__ void __launch_bounds__(cta_threads(false), 1)
tiled_chain_kernel(const ChainLayer* __restrict__ layers, int n_layers, const void* __restrict__ x_first,
                   void* __restrict__ y_last, float* __restrict__ ws, int* __restrict__ counters,
                   unsigned int* __restrict__ sync) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int n_ctas = (int)gridDim.x;
  const int cta = (int)blockIdx.x;
  const int warp = __shfl_sync(0xffffffffu, (int)threadIdx.x >> 5, 0);
  volatile uint32_t* tmem_base_s = reinterpret_cast<volatile uint32_t*>(smem + 8 * 2 * kMaxStages);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (warp == 0) {   // the whole TMEM of this SM, kept for every layer of the chain
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32((const void*)tmem_base_s)),
                 "n"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (threadIdx.x == 0) *reinterpret_cast<volatile uint32_t*>(smem + 8 * 2 * kMaxStages + 4) = 0u;
  bool used = false;     // this CTA's barriers have been initialised by an earlier layer
  for (int li = 0; li < n_layers; ++li) {
    // (read in place: a private copy of the layer's 400 bytes cost registers all through the body)
    const ChainLayer& cl = layers[li];
    const void* xl = (li == 0) ? x_first : cl.x;              // the chain's input and output are the caller's
    void* yl = (li == n_layers - 1) ? y_last : cl.y;
    ChainCtx cc;
    cc.sync = sync;
    cc.target = (unsigned int)li * (unsigned int)n_ctas;
    cc.own_tmem = 0;
    cc.reinit = used ? 1 : 0;
    if (cta < cl.gx * cl.gy * cl.gz) {     // (a CTA outside a layer's grid only counts itself in)
      BlockPos bp;
      bp.gx = cl.gx;
      bp.x = cta % cl.gx;
      bp.y = (cta / cl.gx) % cl.gy;
      bp.z = cta / (cl.gx * cl.gy);
      tiled_body<1, false, false, 4>(cl.L, cl.g, xl, cl.bias, yl, ws, counters, smem, bp, cc);
      used = true;
    } else if (warp == 0) {
      // (in step with the others all the same: its arrival for this layer must not be counted
      // before the previous layer is complete)
      dependency_wait(cc, (int)threadIdx.x & 31, 0, smem, cl.L.err);
    }
    if (threadIdx.x == 0 && li + 1 < n_layers) {   // this CTA's part of the layer is complete and visible
      __threadfence();
      atomicAdd(sync, 1u);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(*tmem_base_s), "n"(kTmemCols)
                 : "memory");
  if (threadIdx.x == 0) {                 // the last CTA to leave puts the counters back to zero
    __threadfence();
    if (atomicAdd(sync + 1, 1u) == (unsigned int)n_ctas - 1u) {
      sync[0] = 0u;
      sync[1] = 0u;
    }
  }
}

// Places descriptors, the raw ring (if any) and the stages for `cps` chunks per CTA, and picks the
// ring depth; false if nothing fits.
int pick_stages(int fit, int zs, int cps);
bool place_stages(Geo* g, int n_chunks_total, int cps, int raw_mode, int stride) {
  g->stage_off = g->desc_off + g->ng * cps * 32;
  g->raw_stages = 0;
  g->raw_mode = 0;
  g->raw_off = g->stage_off;
  g->raw_slot = g->raw_pitch = g->raw_x_bytes = g->raw_sub = 0;
  if (raw_mode == 1) {
    g->raw_pitch = (stride == 1) ? g->tw + 4 : 2 * g->tw + 2;   // halves per raw row (even)
    g->raw_x_bytes = g->pairs * 2 * kChunk * g->rows * g->raw_pitch * 2;
    g->raw_slot = (g->raw_x_bytes + g->ng * (kWRawSlot + kCodeSlot) + 15) & ~15;
  } else if (raw_mode == 2) {
    g->raw_pitch = (stride == 1) ? g->tw + 8 : 2 * g->tw + 8;   // floats per raw row: from 4 columns left of the sub-tile
    g->raw_sub = g->rows * g->raw_pitch * 4;
  } else if (raw_mode == 3) {
    g->raw_sub = ((g->rows * g->w + 8 + 3) & ~3) * 4;           // the rows' span of the plane and its alignment slack
  }
  if (raw_mode >= 2) {
    g->raw_x_bytes = g->pairs * 2 * kChunk * g->raw_sub;
    g->raw_slot = (g->raw_x_bytes + g->ng * (kWSlot + kCodeSlot) + 15) & ~15;
  }
  if (raw_mode) {
    g->raw_mode = raw_mode;
    g->raw_stages = kRawStages < cps ? kRawStages : cps;
    if (raw_mode >= 2 && g->raw_stages > 2) g->raw_stages = 2;   // (fp32 slots are twice the size)
    g->stage_off += g->raw_stages * g->raw_slot;
  }
  (void)n_chunks_total;
  g->stages = pick_stages((kSmemLimit - g->stage_off) / g->stage_bytes, g->zs, cps);
  if (g->stages < 1 && raw_mode) return place_stages(g, n_chunks_total, cps, 0, stride);
  return g->stages >= 1;
}

// Depth of the staging ring when `fit` stages fit in shared memory (0 = the geometry is not
// usable).  The zs warps of a unit work on different chunks at the same time, so the ring holds at
// least zs (then a warp that draws chunk k knows that chunk k - stages has been consumed, which
// makes waiting on a slot's barrier by phase parity safe), and twice zs when it fits: one set of
// chunks being worked on, one in flight.
int pick_stages(int fit, int zs, int cps) {
  int s = fit < 4 * (zs > 1 ? zs / 2 : 1) ? fit : 4 * (zs > 1 ? zs / 2 : 1);  // 4, 4, 8 for zs = 1, 2, 4
  if (s > cps) s = cps;
  if (s == cps) return s;
  return s >= (zs == 1 ? 2 : zs) ? s : 0;
}

// Geometry for `zs` consumer warps per unit, R output rows per lane and no channel split across CTAs.
template <bool GENERIC>
bool geo_for(const DeviceLayer& L, int n, int h, int w, int zs, int R, bool bulk, Geo* out) {
  // the warps of a unit add up column sets of the same TMEM lanes: they sit in one lane quadrant,
  // which holds a quarter of the consumer warps
  if (zs > consumer_warps(GENERIC, R) / 4) return false;
  const int units = consumer_warps(GENERIC, R) / zs;
  Geo g;
  g.rpl = R;
  g.n = n;
  g.h = h;
  g.w = w;
  g.zs = zs;
  g.h_out = (h - 1) / L.stride + 1;
  g.w_out = (w - 1) / L.stride + 1;
  g.tw = 32;
  while (g.tw > 2 && g.tw / 2 >= g.w_out) g.tw /= 2;
  g.sw = 32 / g.tw;
  g.tx = (g.w_out + g.tw - 1) / g.tw;
  g.ty = (g.h_out + R - 1) / R;
  const long long q = (long long)n * g.tx * g.ty;
  if (q > 0x7FFFFFFF) return false;
  g.q_total = (int)q;
  // Filter groups per CTA (ng) x pixel sets (wy) = units.  Wide ng shares the staged input among
  // more filters; when the whole batch has few sub-tiles, pixel sets are traded for groups.
  int ng_max = 1;
  while (ng_max < units && ng_max < L.n_groups) ng_max *= 2;
  const int ng_pref = GENERIC ? 4 : 8;
  g.ng = ng_max < ng_pref ? ng_max : ng_pref;
  g.wys = units / g.ng;
  const long long pairs_needed = (q + 1) / 2;
  while (g.ng < ng_max && (long long)(g.wys / 2) * g.sw >= pairs_needed) {
    g.ng *= 2;
    g.wys /= 2;
  }
  g.wy = g.wys;
  {  // warp rows beyond the batch's sub-tiles stay idle and are not staged
    const long long need = (pairs_needed + g.sw - 1) / g.sw;
    if (need < g.wy) g.wy = need < 1 ? 1 : (int)need;
  }
  g.rows = L.stride * (R - 1) + 3;
  g.pitch = (L.stride == 1) ? (g.tw + 2) : (2 * g.tw + 1);
  // The staged tile is column-major: the rows of a column are contiguous float2, so a lane's
  // window column comes in 16-byte loads.  48 B (80 B at stride 2; 80 B and 144 B with 8 rows per
  // lane) between columns keeps the 8 lanes of a quarter-warp on distinct 16-byte bank groups;
  // narrower sub-tiles are offset so that the sub-tiles sharing a quarter-warp do not collide.
  g.colstride = (g.rows * 8 + 15) & ~15;
  g.substride = g.pitch * g.colstride;
  if (g.tw == 4) while (g.substride % 128 != 64) g.substride += 16;
  if (g.tw == 2) while (g.substride % 128 != 32) g.substride += 16;
  // barriers, TMEM base word, unit counters, first-chunk barriers, raw-slot barriers
  g.tab_off = 8 * 2 * kMaxStages + 16 + 64 + 8 * kMaxCoop + 8 * (kRawStages + 1);
  if (L.n_chunks > 512) return false;   // descriptor table budget (c_in <= 4096)
  g.ks = 1;
  g.cps = L.n_chunks;
  // how chunks are fetched: fp16 pairs by cp.async where rows start on 4-byte boundaries; fp32, when
  // asked for, by bulk copies where plane spans (sub-tile as wide as the image) or rows start on
  // 16-byte boundaries (measured slower than element-wise cp.async: see PCONV_STAGE_BULK)
  g.raw_want = 0;
  if (L.storage == PCONV_F16) {
    if (w % 2 == 0) g.raw_want = 1;
  } else if (bulk && g.tx == 1 && ((long long)h * w) % 4 == 0) {
    g.raw_want = 3;
  } else if (bulk && g.tx > 1 && w % 4 == 0) {
    g.raw_want = 2;
  }
  for (;;) {
    g.pairs = g.wy * g.sw;
    g.chan_stride = g.pairs * g.substride;
    g.x_stage_bytes = kChunk * g.chan_stride;
    g.stage_bytes = (g.x_stage_bytes + g.ng * (kWSlot + kCodeSlot) + 15) & ~15;
    g.desc_off = (g.tab_off + 2 * g.pairs * (int)sizeof(SubTile) + 15) & ~15;
    if (place_stages(&g, L.n_chunks, g.cps, g.raw_want, L.stride)) break;
    if (g.wy > 1) {
      g.wy /= 2;          // fewer pixel sets (the other warp rows idle)
    } else if (g.ng > 1) {
      g.ng /= 2;          // fewer filter groups per CTA
      g.wys = units / g.ng;
    } else {
      break;
    }
  }
  if (g.stages < 1) return false;
  g.relu = 0;
  g.fixed_turns = 0;
  g.cluster = 0;
  g.pool = 0;
  g.h_y = g.h_out;
  g.w_y = g.w_out;
  g.is_half = (L.storage == PCONV_F16);
  *out = g;
  return true;
}

long long geo_tiles(const DeviceLayer& L, const Geo& g) {
  return (((long long)g.q_total + 2 * g.pairs - 1) / (2 * g.pairs)) * ((L.n_groups + g.ng - 1) / g.ng);
}

// Cuts the chunk range of a geometry in ks parts (grid.z).
void set_split(const DeviceLayer& L, Geo* g, int ks) {
  if (ks < 1) ks = 1;
  if (ks > L.n_chunks) ks = L.n_chunks;
  g->cps = (L.n_chunks + ks - 1) / ks;
  g->ks = (L.n_chunks + g->cps - 1) / g->cps;
  if (!place_stages(g, L.n_chunks, g->cps, g->raw_want, L.stride)) g->stages = 0;
}

// Estimated duration of a launch in units of one kernel (4 taps on a warp's 256 pixels, about
// 0.17 us), from measurements of batch-1 and small-map layers: a CTA pays a fixed start (first
// chunk in flight) and an epilogue that shrinks with the warps sharing a unit; a chunk takes the
// consumers its kernels plus a fixed part, and the four producer warps a time that grows with the
// staged elements (measured 0.5 us + 4 ns per element), zs chunks being consumed at a time; CTAs
// run in waves of one per SM; a channel split across CTAs adds the atomic traffic of every CTA's
// tile and its draining.
constexpr double kTallKernelTime = 0.93;
double geo_cost(const DeviceLayer& L, const Geo& g) {
  const double k_unit = (double)L.n_kept / (L.n_groups > 0 ? L.n_groups : 1);  // kernels of one group
  const double per_chunk = 1.5;                                                // barrier, entry, exit
  const int turns = (g.cps + g.zs - 1) / g.zs;                                 // chunks per warp
  // (with 8 rows per lane a warp's kernel covers 512 pixels and its scheduler serves two warps
  // instead of four: measured per-warp time per kernel relative to the 4-row form, on layers
  // with one warp per unit)
  const double k_time = (g.rpl == 8) ? kTallKernelTime : 1.0;
  const double consume = k_time * k_unit / L.n_chunks + per_chunk;
  const double produce = 3.0 + 0.024 * (g.pairs * g.rows * g.pitch);
  const double chunk = consume > g.zs * produce ? consume : g.zs * produce;
  const double loop = turns * chunk;
  const double fixed = 28.0 + 17.0 / g.zs;
  const long long ctas = geo_tiles(L, g) * g.ks;
  const int sms = device_sm_count();
  const double waves = (double)((ctas + sms - 1) / sms);
  return waves * (fixed + loop) + (g.ks > 1 ? 100.0 / g.zs : 0.0);
}

// The geometry of a launch.  `pin` = what the caller pinned: the rows per lane (4, 8 or 0 = by the
// estimate; 8 needs one-byte codes), | kPinBulk = fp32 chunks by bulk copies.  Canonical pattern
// sets choose the rows per lane, how the consumer warps are used (zs = 1, 2 or 4
// warps per unit) and, when a workspace is available, whether the channel range is also split
// across CTAs, by the estimate above.
template <bool GENERIC>
bool make_geo(const DeviceLayer& L, int n, int h, int w, bool allow_split, int pin, Geo* out) {
  const int rmode = pin & kPinRowsMask;
  const bool bulk = (pin & kPinBulk) != 0;
  if (GENERIC) return geo_for<true>(L, n, h, w, 1, 4, bulk, out);
  bool found = false;
  double best = 0.0;
#ifdef PCONV_DEV
  const char* force_zs = getenv("PCONV_FORCE_ZS");
  const char* force_ks = getenv("PCONV_FORCE_KS");
#endif
  for (int R = 4; R <= 8; R *= 2) {
    if (rmode && rmode != R) continue;
    if (R == 8 && L.wide_codes) continue;
    // Left to itself the planner takes 8 rows per lane only where the 4-row form already runs one
    // warp per unit on the whole channel range (large batches): measured 3-10 % faster there, and
    // slower wherever channels are split (a TMEM lane quadrant then holds two warps, not four).
    if (R == 8 && !rmode && found && (out->zs != 1 || out->ks != 1)) continue;
    for (int zs = 1; zs <= 4; zs *= 2) {
      if (R == 8 && !rmode && zs != 1) continue;
      Geo g;
#ifdef PCONV_DEV
      if (force_zs && atoi(force_zs) != zs) continue;
#endif
      if (!geo_for<false>(L, n, h, w, zs, R, bulk, &g)) continue;
#ifdef PCONV_DEV
      if (force_ks && allow_split) {
        set_split(L, &g, atoi(force_ks));
        if (g.stages < 1) continue;
        *out = g;
        return true;
      }
#endif
      for (int pass = 0; pass < 2; ++pass) {
        Geo c = g;
        if (pass == 1) {
          if (!allow_split || (R == 8 && !rmode)) break;
          const long long tiles = geo_tiles(L, g);
          const long long ks = device_sm_count() / tiles;   // fill one wave
          if (ks < 2) break;
          set_split(L, &c, (int)ks);
          if (c.ks < 2 || c.stages < 1) break;
        }
        const double cost = geo_cost(L, c);
        if (!found || cost < best) {
          found = true;
          best = cost;
          *out = c;
        }
      }
    }
  }
  return found;
}

template <int S, bool GENERIC, bool WIDE, int R>
cudaError_t launch_one(const DeviceLayer& L, Geo g, const void* x, const float* bias, void* y, float* ws,
                       int* counters, cudaStream_t stream) {
  int smem = g.stage_off + g.stages * g.stage_bytes;
  // the TMEM variant must be alone on its SM (it takes all 512 columns): make sure two CTAs can
  // never be co-resident by asking for more than half of the shared memory
  if (!GENERIC && smem < 120 * 1024) smem = 120 * 1024;
  cudaError_t e = cudaFuncSetAttribute(tiled_kernel<S, GENERIC, WIDE, R>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
  if (e != cudaSuccess) return e;
  const long long ctas_x = ((long long)g.q_total + 2 * g.pairs - 1) / (2 * g.pairs);
  const int ctas_y = (L.n_groups + g.ng - 1) / g.ng;
  if (ctas_x > 0x7FFFFFFF || ctas_y > 65535 || g.ks > 65535) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)ctas_x, (unsigned)ctas_y, (unsigned)g.ks);
  cfg.blockDim = dim3(cta_threads(GENERIC, R), 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (g.cluster) {
    // The ks CTAs of a tile as one thread-block cluster.  More than 8 CTAs per cluster is beyond
    // the portable size: allowed per kernel, and taken only if all the launch's clusters can be
    // resident at once (a cluster needs its SMs inside one GPC); otherwise, and on any error here,
    // the launch falls back to the workspace form.
    bool ok = true;
    if (g.ks > 8)
      ok = cudaFuncSetAttribute(tiled_kernel<S, GENERIC, WIDE, R>, cudaFuncAttributeNonPortableClusterSizeAllowed,
                                1) == cudaSuccess;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = (unsigned)g.ks;
    cfg.numAttrs = 2;
    int n_clusters = 0;
    if (ok) {
      // (asked once per kernel, shared-memory size, cluster size and device: the answer does not change)
      static std::mutex mu;
      static std::map<std::tuple<int, int, int>, int> known;
      int dev = 0;
      ok = cudaGetDevice(&dev) == cudaSuccess;
      if (ok) {
        std::lock_guard<std::mutex> lock(mu);
        const auto key = std::make_tuple(dev, smem, g.ks);
        const auto it = known.find(key);
        if (it != known.end()) {
          n_clusters = it->second;
        } else {
          ok = cudaOccupancyMaxActiveClusters(&n_clusters, tiled_kernel<S, GENERIC, WIDE, R>, &cfg) == cudaSuccess;
          if (ok) known[key] = n_clusters;
        }
      }
    }
    if (ok) ok = (long long)n_clusters >= ctas_x * ctas_y;
    if (!ok) {
      (void)cudaGetLastError();
      if (!ws) return cudaErrorInvalidValue;   // (launch_tiled only asks for a cluster with a workspace to fall back on)
      g.cluster = 0;
      cfg.numAttrs = 1;
    }
  }
  return cudaLaunchKernelEx(&cfg, tiled_kernel<S, GENERIC, WIDE, R>, L, g, x, bias, y, ws, counters);
}


}  // namespace

bool tiled_supported(const DeviceLayer& L, int n, int h, int w) {
  Geo g;
  if (n <= 0 || h <= 0 || w <= 0) return false;
  if (L.n_groups > 65535) return false;
  return make_geo<true>(L, n, h, w, false, 4, &g) && make_geo<false>(L, n, h, w, false, 4, &g);
}

// Workspace of the channel-split path: the partial sums of every (tile, consumer warp, filter slot
// the warp writes out, lane) as 8 floats -- the layout of the warps that add to it and read it
// back, not y's --, then one ticket per (tile, consumer warp); 0 if this shape is never split.
size_t split_sums_bytes(const DeviceLayer& L, const Geo& g) {
  return (size_t)geo_tiles(L, g) * consumer_warps(false, g.rpl) * (kGroup / g.zs) * 32 * (2 * g.rpl) * sizeof(float);
}
// `rmode`: rows per lane the launch will be asked for (4, 8, 0 = the planner's choice).
size_t tiled_workspace_bytes(const DeviceLayer& L, int n, int h, int w, int rmode) {
  Geo g;
  if (!L.codes_s || !make_geo<false>(L, n, h, w, true, rmode, &g) || g.ks <= 1) return 0;
  const size_t ctas = (size_t)geo_tiles(L, g);
  return ((split_sums_bytes(L, g) + 255) & ~(size_t)255) +
         ((ctas * kMaxConsumerWarps * 4 + 255) & ~(size_t)255);
}

// The launch geometry launch_tiled would use (see pconv_plan_t).
bool tiled_plan(const DeviceLayer& L, int n, int h, int w, bool generic_taps, bool with_workspace,
                int rmode, pconv_plan_t* out) {
  if (!generic_taps && !L.codes_s) generic_taps = true;
  Geo g;
  if (!(generic_taps ? make_geo<true>(L, n, h, w, false, 4, &g)
                     : make_geo<false>(L, n, h, w, with_workspace, rmode, &g)))
    return false;
  out->generic_taps = generic_taps ? 1 : 0;
  out->rows_per_lane = g.rpl;
  out->staging = g.raw_mode;
  out->warps_per_unit = g.zs;
  out->channel_splits = g.ks;
  out->groups_per_cta = g.ng;
  out->pixel_sets = g.wy;
  out->tile_width = g.tw;
  out->stages = g.stages;
  out->ctas = geo_tiles(L, g) * g.ks;
  out->smem_bytes = g.stage_off + g.stages * g.stage_bytes;
  return true;
}

cudaError_t launch_tiled(const DeviceLayer& L, const void* x, const float* bias, void* y, int n, int h,
                         int w, bool relu, bool pool, bool reproducible, bool generic_taps, int rmode,
                         bool allow_cluster, void* ws, size_t ws_bytes, cudaStream_t stream) {
  if (!generic_taps && !L.codes_s) generic_taps = true;
  if ((rmode & kPinRowsMask) == 8 && (generic_taps || L.wide_codes)) return cudaErrorInvalidValue;
  Geo g;
  const size_t need = generic_taps ? 0 : tiled_workspace_bytes(L, n, h, w, rmode);
  const bool split = !reproducible && need > 0 && ws && ws_bytes >= need;
  if (!(generic_taps ? make_geo<true>(L, n, h, w, false, 4 | (rmode & kPinBulk), &g)
                     : make_geo<false>(L, n, h, w, split, rmode, &g)))
    return cudaErrorInvalidValue;
  g.relu = relu ? 1 : 0;
  if (reproducible && g.zs > 1) {
    g.fixed_turns = 1;
    if (g.stages < g.cps) g.stages = g.stages / g.zs * g.zs;   // >= zs by pick_stages
    if (g.stages < 1) return cudaErrorInvalidValue;
  }
  if (pool) {
    if (g.h_out < 2 || g.w_out < 2) return cudaErrorInvalidValue;
    g.pool = 1;
    g.h_y = g.h_out / 2;
    g.w_y = g.w_out / 2;
  }
  float* wsf = nullptr;
  int* counters = nullptr;
  if (g.ks > 1) {
    wsf = (float*)ws;
    counters = (int*)((char*)ws + ((split_sums_bytes(L, g) + 255) & ~(size_t)255));
    // The CTAs that share a tile add their partial sums up through distributed shared memory when
    // they can form one cluster (at most 16 CTAs) and a CTA's partial sums fit the staging ring;
    // the workspace stays untouched then.
    const size_t part_bytes = (size_t)consumer_warps(false, g.rpl) * (kGroup / g.zs) * 32 * (2 * g.rpl) * sizeof(float);
    const int parts_per_warp = (kGroup / g.zs + g.ks - 1) / g.ks;
    g.cluster = (allow_cluster && g.ks <= 16 && parts_per_warp <= kMaxClusterParts &&
                 part_bytes <= (size_t)g.stages * g.stage_bytes) ? 1 : 0;
  }
  const bool wide = L.wide_codes != 0;
  if (L.stride == 1) {
    if (generic_taps) return launch_one<1, true, false, 4>(L, g, x, bias, y, wsf, counters, stream);
    if (wide) return launch_one<1, false, true, 4>(L, g, x, bias, y, wsf, counters, stream);
    return g.rpl == 8 ? launch_one<1, false, false, 8>(L, g, x, bias, y, wsf, counters, stream)
                      : launch_one<1, false, false, 4>(L, g, x, bias, y, wsf, counters, stream);
  }
  if (generic_taps) return launch_one<2, true, false, 4>(L, g, x, bias, y, wsf, counters, stream);
  if (wide) return launch_one<2, false, true, 4>(L, g, x, bias, y, wsf, counters, stream);
  return g.rpl == 8 ? launch_one<2, false, false, 8>(L, g, x, bias, y, wsf, counters, stream)
                    : launch_one<2, false, false, 4>(L, g, x, bias, y, wsf, counters, stream);
}

// ---- chains ---------------------------------------------------------------------------------------
// Whether a layer may be part of a chain kernel for this input shape: fp32 or fp16 storage with
// stride 1 and a canonical pattern set (the chain kernel is one instantiation), and a launch plan
// of at most one CTA per SM.  *ctas / *ws_bytes (optional) receive the plan's CTA count and
// workspace need.
bool chain_layer_ok(const DeviceLayer& L, int n, int h, int w, bool pool, long long* ctas) {
  if (!L.codes_s || L.wide_codes || L.stride != 1) return false;
  Geo g;
  if (!make_geo<false>(L, n, h, w, true, 4, &g)) return false;   // (the chain kernel is the 4-row form)
  if (pool && (g.h_out < 2 || g.w_out < 2)) return false;
  const long long c = geo_tiles(L, g) * g.ks;
  if (ctas) *ctas = c;
  return c <= device_sm_count();
}

size_t chain_table_bytes(int n_layers) { return (size_t)n_layers * sizeof(ChainLayer); }

// Fills entry `index` of a chain's table (HOST memory, `table` has chain_table_bytes(n) bytes):
// the layer, its geometry for this input shape (with the channel split the workspace allows) and
// its buffers (x / y of the chain's first / last layer are given at launch).
bool chain_fill(void* table, int index, const DeviceLayer& L, const void* x, const float* bias, void* y, int n,
                int h, int w, bool relu, bool pool, int* status_dev) {
  ChainLayer& cl = reinterpret_cast<ChainLayer*>(table)[index];
  std::memset(&cl, 0, sizeof(cl));
  cl.L = L;
  if (status_dev) cl.L.err = status_dev;
  if (!make_geo<false>(L, n, h, w, true, 4, &cl.g)) return false;
  cl.g.relu = relu ? 1 : 0;
  if (pool) {
    cl.g.pool = 1;
    cl.g.h_y = cl.g.h_out / 2;
    cl.g.w_y = cl.g.w_out / 2;
  }
  cl.x = x;
  cl.bias = bias;
  cl.y = y;
  cl.gx = (int)(((long long)cl.g.q_total + 2 * cl.g.pairs - 1) / (2 * cl.g.pairs));
  cl.gy = (L.n_groups + cl.g.ng - 1) / cl.g.ng;
  cl.gz = cl.g.ks;
  return true;
}

// Workspace a chain needs: the largest split layer's sums, then tickets for one grid of CTAs.
size_t chain_workspace_bytes(const void* table_host, int n_layers) {
  const ChainLayer* t = reinterpret_cast<const ChainLayer*>(table_host);
  size_t sums_max = 0;
  for (int i = 0; i < n_layers; ++i)
    if (t[i].g.ks > 1) {
      const size_t need = split_sums_bytes(t[i].L, t[i].g);
      if (need > sums_max) sums_max = need;
    }
  if (!sums_max) return 0;
  return ((sums_max + 255) & ~(size_t)255) + (((size_t)device_sm_count() * kMaxConsumerWarps * 4 + 255) & ~(size_t)255);
}

// Launches a chain: `table_dev` is the DEVICE copy of a filled table, `table_host` the host one
// (for the launch geometry); ws = the stack's channel-split workspace (sums, tickets), sync = two
// zeroed counters.
cudaError_t launch_chain(const void* table_dev, const void* table_host, int n_layers, const void* x_first,
                         void* y_last, void* ws, size_t ws_bytes, unsigned int* sync, cudaStream_t stream) {
  const ChainLayer* t = reinterpret_cast<const ChainLayer*>(table_host);
  long long ctas = 0;
  int smem = 0;
  size_t sums_max = 0;
  for (int i = 0; i < n_layers; ++i) {
    const long long c = (long long)t[i].gx * t[i].gy * t[i].gz;
    if (c > ctas) ctas = c;
    const int sm = t[i].g.stage_off + t[i].g.stages * t[i].g.stage_bytes;
    if (sm > smem) smem = sm;
    if (t[i].g.ks > 1) {
      const size_t need = split_sums_bytes(t[i].L, t[i].g);
      if (need > sums_max) sums_max = need;
    }
  }
  if (ctas < 1 || ctas > device_sm_count()) return cudaErrorInvalidValue;
  // every layer of the chain finds its tickets behind the largest layer's sums
  const size_t tick_off = (sums_max + 255) & ~(size_t)255;
  if (sums_max && (!ws || ws_bytes < tick_off + (size_t)device_sm_count() * kMaxConsumerWarps * 4))
    return cudaErrorInvalidValue;
  if (smem < 120 * 1024) smem = 120 * 1024;
  cudaError_t e = cudaFuncSetAttribute(tiled_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)ctas, 1, 1);
  cfg.blockDim = dim3(cta_threads(false), 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, tiled_chain_kernel, reinterpret_cast<const ChainLayer*>(table_dev), n_layers,
                            x_first, y_last, (float*)ws, (int*)((char*)ws + tick_off), sync);
}

#ifdef PCONV_DEV
cudaError_t dev_set_withhold(int chunk, unsigned spin_limit) {
  const unsigned limit = chunk < 0 ? kSpinLimit : (spin_limit ? spin_limit : 1u);
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_dev_spin_limit, &limit, sizeof(limit));
  if (e == cudaSuccess) e = cudaMemcpyToSymbol(g_dev_withhold_chunk, &chunk, sizeof(chunk));
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  return e;
}
#endif

}  // namespace pconv
