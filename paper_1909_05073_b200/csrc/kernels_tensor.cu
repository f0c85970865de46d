// Dense regrouping on the tensor cores (fp16 storage, stride 1): the layer as an implicit GEMM
// over zero-inserted weights, D[pixel, filter] = sum over (tap, channel) of A_tap[pixel, channel] *
// W_tap[channel, filter], on tcgen05.mma with the accumulators in Tensor Memory.
//
// Why this exists beside the pattern-sparse kernel: with fp16 operands every product is exact in
// the fp32 accumulator, so the zero-inserted contraction computes the same sums; it does
// 9 / (4 x keep) times the multiply-adds, but the tensor pipe is ~30 times faster than the FP32
// pipe, so for fp16 storage it wins at every keep rate the benchmark configurations use.
//
// Mapping.  An MMA tile is 128 pixels (TMEM lanes) x n_t filters (TMEM columns), K = 16 channels
// per instruction, nine instructions (taps) per 16 channels.
//  * Pixels.  The batch is laid out as one tall virtual strip: images (or, for maps narrower than
//    8, rows of 8 / cell-width images side by side) stacked vertically with ONE separator row
//    between consecutive images.  A tile is r = 128 / tw consecutive strip rows x tw columns.  The
//    separator row is the zero padding below one image and above the next, so a vertical tap
//    shift is the same strip shifted by one row for every pixel of the tile; outputs computed for
//    separator rows and padding columns are thrown away (h / (h + 1) of the rows are useful).
//  * A operand (activations), pixel-major ("MN-major") canonical layout without swizzle: a core
//    matrix is 8 channels x 8 consecutive pixels (8 rows of 16 bytes).  Per stage (16 channels)
//    the producers build three copies of the halo'd tile, one per horizontal tap offset (the
//    shifted copies are made in registers from one 16-byte load plus two neighbours); the rows of
//    a copy are contiguous, so the vertical tap offset is just the descriptor's start address
//    moved by one row of core matrices.  Nothing is ever im2col'ed in global memory.
//  * B operand (weights): the packer writes, per (filter tile, 16-channel step), the nine
//    zero-inserted [n_t x 16] fp16 matrices already in the K-major canonical core-matrix order; a
//    stage's 9 x n_t x 32 bytes arrive with one bulk copy (cp.async.bulk, no tensor map, no
//    multicast) that completes on the stage's mbarrier.
//  * Warp roles: warps 0-3 epilogue (warp q reads TMEM lanes 32q..32q+31: bias, ReLU, fp16
//    convert, store to NCHW), warp 4 issues the MMAs (one thread) and owns the TMEM allocation,
//    warps 5-12 are the A producers, in two groups that take alternate stages so that one group's
//    global loads are in flight while the other converts and stores.  Two accumulator buffers
//    (2 x n_t columns) let the epilogue of a tile overlap the next tile's MMAs.  CTAs are
//    persistent: tile t of a CTA is blockIdx.x + t * gridDim.x.
//  * Every wait is bounded; a wait that runs out records its id (20-25) in the layer's status word,
//    the role stops working, and all roles meet at the common exit where TMEM is released.
#include <cuda_fp16.h>

#include "pconv_internal.h"

namespace pconv {
namespace {

typedef unsigned long long u64;

constexpr int kEpiWarps = 4;
constexpr int kMmaWarp = 4;
constexpr int kProdWarp0 = 5;
constexpr int kProdGroups = 2;
constexpr int kProdWarpsPerGroup = 4;
constexpr int kProdThreadsPerGroup = 32 * kProdWarpsPerGroup;
constexpr int kTensorThreads = 32 * (kProdWarp0 + kProdGroups * kProdWarpsPerGroup);
constexpr int kMaxTStages = 6;
constexpr int kMaxTasks = 4;              // A tasks of one producer thread per stage
constexpr uint32_t kTSpinLimit = 1u << 20;
constexpr uint32_t kTWaitHintNs = 200;
constexpr int kTSmemLimit = 227 * 1024;

struct TGeo {
  int n, h, w, c_in, c_out;
  int hp;            // strip period: h + 1 (image rows + one separator row)
  int wc;            // cell width: w rounded up to a multiple of 8, or to 1, 2, 4 for w < 8
  int cpr;           // cells (images) side by side in a strip row
  int tw, r;         // tile: r strip rows x tw columns, r * tw = 128
  int tiles_x;       // column tiles of the virtual width cpr * wc
  long long strip_rows, tiles_y;
  int n_t, n_tiles_n, k_steps;
  int stages, a_copy_bytes, a_lbo, row_bytes, b_bytes, stage_bytes, stage_off;
  int relu;
  long long total_tiles;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kTWaitHintNs)
      : "memory");
  return ok != 0;
}
// Bounded wait: false (and the wait id recorded) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* err, int id) {
  for (uint32_t it = 0; it < kTSpinLimit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  atomicCAS(err, 0, id);
  return false;
}
// 1-D bulk copy global -> shared (this CTA's own shared memory; no multicast), completing `bytes`
// on the mbarrier.  Addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// Shared-memory matrix descriptor, no swizzle: start address, leading-dimension and stride byte
// offsets in 16-byte units, descriptor version 1.
__device__ __forceinline__ u64 smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (u64)((addr & 0x3FFFFu) >> 4) | ((u64)(lbo_bytes >> 4) << 16) | ((u64)(sbo_bytes >> 4) << 32) |
         (1ull << 46);
}
// D[tmem] (+)= A[smem] * B[smem], 128 x n_t x 16, fp16 operands, fp32 accumulate; one thread issues.
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, u64 a_desc, u64 b_desc, uint32_t idesc,
                                         uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The mbarrier receives one arrival when all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t (&v)[16], uint32_t taddr) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// One A task = (halo row, 8-channel block, column group of 8 pixels, channel within the block): 16
// bytes of each of the three horizontally shifted copies.  What depends on the tile only is kept
// per task: the element offset of the group's first pixel for channel `ch` of step 0 (-1: the
// whole group is padding), the same for the pixel left of the group and right of it, and for
// narrow maps the per-pixel data.
struct ATask {
  long long off;        // element offset of pixel 0 of the group (channel `ch` of k-step 0), or -1
  uint32_t dst;         // byte offset inside a copy
  int ch;               // channel inside the 16-channel step
  uint32_t flags;       // bit 0: left neighbour exists, bit 1: right neighbour exists
};

// The strip row a tile row maps to: image group and row inside it, or invalid (separator / outside).
__device__ __forceinline__ bool strip_row(const TGeo& g, long long s, long long* group, int* row) {
  if (s < 0 || s >= g.strip_rows) return false;
  const long long gi = s / g.hp;
  const int lr = (int)(s - gi * g.hp);
  *group = gi;
  *row = lr;
  return lr < g.h;
}

template <bool RELU>
__device__ __forceinline__ void store_col(__half* y, long long idx, float v) {
  if (RELU) v = fmaxf(v, 0.f);
  y[idx] = __float2half_rn(v);
}

__global__ void __launch_bounds__(kTensorThreads, 1)
tensor_kernel(const DeviceLayer L, const TGeo g, const __half* __restrict__ x,
              const float* __restrict__ bias, __half* __restrict__ y) {
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  // barriers: full[s], empty[s] (s < stages), acc_full[2], acc_empty[2]; then the TMEM base word
  const uint32_t bar_full = sbase, bar_empty = sbase + 8 * kMaxTStages;
  const uint32_t bar_accf = sbase + 16 * kMaxTStages, bar_acce = bar_accf + 16;
  volatile uint32_t* tmem_base_s = reinterpret_cast<volatile uint32_t*>(smem + 16 * kMaxTStages + 32);
  const uint32_t tmem_cols = (uint32_t)(2 * g.n_t);   // 128 or 256: a power of two >= 32

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) {
    for (int s = 0; s < g.stages; ++s) {
      mbar_init(bar_full + 8 * s, kProdThreadsPerGroup + 1);   // a group's threads + the bulk copy's issuer
      mbar_init(bar_empty + 8 * s, 1);                         // one tcgen05.commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_accf + 8 * b, 1);
      mbar_init(bar_acce + 8 * b, 32 * kEpiWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32((const void*)tmem_base_s)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_base_s;
  // the previous kernel of the stream must have finished before x is read or y written
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const long long my_tiles = (g.total_tiles > blockIdx.x)
                                 ? (g.total_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  const uint32_t row_b = (uint32_t)g.row_bytes;     // bytes of one tile row of core matrices
  const size_t hw = (size_t)g.h * g.w;

  if (warp == kMmaWarp) {
    // ======================================= MMA issuer =======================================
    if (lane == 0) {
      // instruction descriptor: D fp32, A and B fp16, A pixel-major (MN-major), B K-major, N, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 15) | ((uint32_t)(g.n_t >> 3) << 17) | ((128u >> 4) << 24);
      const uint32_t b_lbo = (uint32_t)(g.n_t / 8) * 128u;
      long long it = 0;
      bool ok = true;
      for (long long ti = 0; ti < my_tiles && ok; ++ti) {
        const int buf = (int)(ti & 1);
        const uint32_t use = (uint32_t)(ti >> 1);
        ok = mbar_wait(bar_acce + 8 * buf, (use & 1u) ^ 1u, L.err, 20);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * g.n_t);
        for (int ks = 0; ks < g.k_steps; ++ks, ++it) {
          const int s = (int)(it % g.stages);
          ok = mbar_wait(bar_full + 8 * s, (uint32_t)((it / g.stages) & 1), L.err, 21);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a0 = sbase + g.stage_off + s * g.stage_bytes;
          const uint32_t b0 = a0 + 3 * g.a_copy_bytes;
#pragma unroll
          for (int t = 0; t < 9; ++t) {
            const int u = t / 3, v = t - 3 * u;
            const u64 ad = smem_desc(a0 + v * g.a_copy_bytes + u * row_b, (uint32_t)g.a_lbo, 128u);
            const u64 bd = smem_desc(b0 + t * (g.n_t * 32), b_lbo, 128u);
            umma_f16(d_tmem, ad, bd, idesc, (ks > 0 || t > 0) ? 1u : 0u);
          }
          umma_commit(bar_empty + 8 * s);          // the stage may be refilled once these MMAs are done
        }
        if (ok) umma_commit(bar_accf + 8 * buf);   // the tile's accumulator is complete
      }
    }
    __syncwarp();
  } else if (warp >= kProdWarp0) {
    // ======================================= A producers ======================================
    const int group = (warp - kProdWarp0) / kProdWarpsPerGroup;
    const int gt = (warp - kProdWarp0 - group * kProdWarpsPerGroup) * 32 + lane;
    const int cgs = g.tw / 8;
    const int n_tasks = (g.r + 2) * 2 * cgs * 8;
    const unsigned short* xs = reinterpret_cast<const unsigned short*>(x);
    const bool fast = (g.w % 8) == 0;          // rows are 16-byte aligned: one vector load per task
    bool ok = true;
    long long it = 0;                          // global stage counter (all tiles of this CTA)
    for (long long ti = 0; ti < my_tiles && ok; ++ti) {
      const long long tile = blockIdx.x + ti * gridDim.x;
      const long long mt = tile / g.n_tiles_n;
      const int nt = (int)(tile - mt * g.n_tiles_n);
      const long long ty = mt / g.tiles_x;
      const int tx = (int)(mt - ty * g.tiles_x);
      ATask task[kMaxTasks];
#pragma unroll
      for (int q = 0; q < kMaxTasks; ++q) {
        const int t = gt + q * kProdThreadsPerGroup;
        task[q].off = -1;
        task[q].dst = 0xFFFFFFFFu;
        task[q].ch = 0;
        task[q].flags = 0;
        if (t < n_tasks) {
          const int c8 = t & 7;
          int rest = t >> 3;
          const int cg = rest % cgs;
          rest /= cgs;
          const int kb = rest & 1, hr = rest >> 1;
          task[q].ch = kb * 8 + c8;
          task[q].dst = (uint32_t)(kb * g.a_lbo + hr * (int)row_b + cg * 128 + c8 * 16);
          long long gi;
          int lr;
          const int vx = tx * g.tw + cg * 8;        // virtual column of the group's first pixel
          if (strip_row(g, ty * g.r + hr - 1, &gi, &lr) && g.wc >= 8) {
            const long long n_img = gi;             // one image per strip row
            if (n_img < g.n && vx < g.w) {
              task[q].off = ((n_img * g.c_in + task[q].ch) * g.h + lr) * (long long)g.w + vx;
              task[q].flags = (vx > 0 ? 1u : 0u) | (vx + 8 < g.w ? 2u : 0u);
            }
          } else if (g.wc < 8 && strip_row(g, ty * g.r + hr - 1, &gi, &lr)) {
            // narrow maps: the 8 pixels are 8 / wc images side by side; `off` addresses the first
            task[q].off = ((gi * g.cpr + vx / g.wc) * (long long)g.c_in + task[q].ch) * g.h * (long long)g.w +
                          (long long)lr * g.w;
            task[q].flags = 4u;
          }
        }
      }
      for (int ks = 0; ks < g.k_steps && ok; ++ks, ++it) {
        if ((it & 1) != group) continue;           // the other group's stage
        const int s = (int)(it % g.stages);
        ok = mbar_wait(bar_empty + 8 * s, (uint32_t)(((it / g.stages) & 1) ^ 1), L.err, 22);
        if (!ok) break;
        const uint32_t a0 = sbase + g.stage_off + s * g.stage_bytes;
        if (gt == 0) {   // the stage's weights: one bulk copy, counted on the same barrier
          mbar_arrive_expect_tx(bar_full + 8 * s, (uint32_t)g.b_bytes);
          bulk_copy_g2s(a0 + 3 * g.a_copy_bytes,
                        reinterpret_cast<const char*>(L.wdense) + ((size_t)nt * g.k_steps + ks) * g.b_bytes,
                        (uint32_t)g.b_bytes, bar_full + 8 * s);
        }
        const int c_base = ks * 16;
        // loads of all tasks first, then shifts and stores
        uint4 v[kMaxTasks];
        uint32_t lft[kMaxTasks], rgt[kMaxTasks];
#pragma unroll
        for (int q = 0; q < kMaxTasks; ++q) {
          v[q] = make_uint4(0u, 0u, 0u, 0u);
          lft[q] = rgt[q] = 0u;
          if (task[q].dst == 0xFFFFFFFFu || task[q].off < 0) continue;
          const int c = c_base + task[q].ch;
          if (c >= g.c_in) continue;
          const unsigned short* p = xs + task[q].off + (size_t)c_base * hw;
          if (task[q].flags & 4u) {
            // narrow maps: pixel q8 belongs to image (q8 / wc) of the row, column q8 % wc
            uint32_t e[8];
            const long long img0 = task[q].off / ((long long)g.c_in * (long long)hw);
#pragma unroll
            for (int q8 = 0; q8 < 8; ++q8) {
              const int cell = q8 / g.wc, xin = q8 - cell * g.wc;
              e[q8] = (xin < g.w && img0 + cell < g.n)
                          ? (uint32_t)__ldg(p + (size_t)cell * g.c_in * hw + xin) : 0u;
            }
            v[q] = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
          } else if (fast) {
            v[q] = __ldg(reinterpret_cast<const uint4*>(p));
            if (task[q].flags & 1u) lft[q] = (uint32_t)__ldg(p - 1);
            if (task[q].flags & 2u) rgt[q] = (uint32_t)__ldg(p + 8);
          } else {
            const int vx = (int)((task[q].off) % g.w);   // column of pixel 0 (off = ... * w + vx)
            uint32_t e[8];
#pragma unroll
            for (int q8 = 0; q8 < 8; ++q8) e[q8] = (vx + q8 < g.w) ? (uint32_t)__ldg(p + q8) : 0u;
            v[q] = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
            if (task[q].flags & 1u) lft[q] = (uint32_t)__ldg(p - 1);
            if (task[q].flags & 2u) rgt[q] = (uint32_t)__ldg(p + 8);
          }
        }
#pragma unroll
        for (int q = 0; q < kMaxTasks; ++q) {
          if (task[q].dst == 0xFFFFFFFFu) continue;
          const uint4 c = v[q];
          // copy 0: pixel p holds input column p - 1;  copy 2: column p + 1
          uint4 m1, p1;
          m1.x = __funnelshift_l(lft[q] << 16, c.x, 16);
          m1.y = __funnelshift_l(c.x, c.y, 16);
          m1.z = __funnelshift_l(c.y, c.z, 16);
          m1.w = __funnelshift_l(c.z, c.w, 16);
          p1.x = __funnelshift_r(c.x, c.y, 16);
          p1.y = __funnelshift_r(c.y, c.z, 16);
          p1.z = __funnelshift_r(c.z, c.w, 16);
          p1.w = __funnelshift_r(c.w, rgt[q], 16);
          if (task[q].flags & 4u) {
            // narrow maps: no pixel may see across its image's edge
            uint32_t zm[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};   // keep masks, copy 0
            uint32_t zp[4] = {0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu};   // copy 2
#pragma unroll
            for (int q8 = 0; q8 < 8; ++q8) {
              const int xin = q8 % g.wc;
              const uint32_t half_mask = (q8 & 1) ? 0x0000FFFFu : 0xFFFF0000u;   // what stays when this half is cleared
              if (xin == 0) zm[q8 >> 1] &= half_mask;
              if (xin + 1 >= g.w) zp[q8 >> 1] &= half_mask;
            }
            m1.x &= zm[0]; m1.y &= zm[1]; m1.z &= zm[2]; m1.w &= zm[3];
            p1.x &= zp[0]; p1.y &= zp[1]; p1.z &= zp[2]; p1.w &= zp[3];
          }
          const uint32_t d = a0 + task[q].dst;
          sts128(d, m1.x, m1.y, m1.z, m1.w);
          sts128(d + g.a_copy_bytes, c.x, c.y, c.z, c.w);
          sts128(d + 2 * g.a_copy_bytes, p1.x, p1.y, p1.z, p1.w);
        }
        // generic-proxy stores must be visible to the tensor core's (async proxy) reads
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mbar_arrive(bar_full + 8 * s);
      }
    }
  } else {
    // ======================================= epilogue =========================================
    const int q = warp;                       // TMEM lane quadrant
    const int m = 32 * q + lane;              // pixel of the tile
    const int tr = m / g.tw, tc = m - tr * g.tw;
    bool ok = true;
    for (long long ti = 0; ti < my_tiles && ok; ++ti) {
      const long long tile = blockIdx.x + ti * gridDim.x;
      const long long mt = tile / g.n_tiles_n;
      const int nt = (int)(tile - mt * g.n_tiles_n);
      const long long ty = mt / g.tiles_x;
      const int tx = (int)(mt - ty * g.tiles_x);
      const int buf = (int)(ti & 1);
      const uint32_t use = (uint32_t)(ti >> 1);
      long long gi = 0;
      int lr = 0;
      bool valid = strip_row(g, ty * g.r + tr, &gi, &lr);
      const int vcol = tx * g.tw + tc;
      const int cell = vcol / g.wc, xin = vcol - cell * g.wc;
      const long long n_img = gi * g.cpr + cell;
      valid = valid && xin < g.w && cell < g.cpr && n_img < g.n;
      const long long base = valid ? (n_img * g.c_out * (long long)g.h + lr) * g.w + xin : 0;
      ok = mbar_wait(bar_accf + 8 * buf, use & 1u, L.err, 23);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * g.n_t);
      for (int j0 = 0; j0 < g.n_t; j0 += 16) {
        const int o0 = nt * g.n_t + j0;
        if (o0 >= g.c_out) break;               // padding filters of the last tile (warp-uniform)
        uint32_t acc[16];
        tmem_ld16(acc, taddr + (uint32_t)j0);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int o = o0 + j;
          if (o < g.c_out && valid) {
            const float bv = bias ? __ldg(bias + o) : 0.f;
            const float val = __uint_as_float(acc[j]) + bv;
            if (g.relu) store_col<true>(y, base + (long long)o * (long long)hw, val);
            else store_col<false>(y, base + (long long)o * (long long)hw, val);
          }
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(bar_acce + 8 * buf);
    }
  }

  // ---- common exit ----------------------------------------------------------------------------
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kMmaWarp)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols)
                 : "memory");
}

bool tensor_geo(const DeviceLayer& L, int n, int h, int w, TGeo* out) {
  if (!L.wdense || L.dense_nt <= 0 || L.stride != 1 || L.storage != PCONV_F16) return false;
  TGeo g;
  g.n = n;
  g.h = h;
  g.w = w;
  g.c_in = L.c_in;
  g.c_out = L.c_out;
  g.hp = h + 1;
  if (w >= 8) {
    g.wc = (w + 7) / 8 * 8;
    g.cpr = 1;
  } else {
    g.wc = w <= 1 ? 1 : (w <= 2 ? 2 : (w <= 4 ? 4 : 8));
    g.cpr = 8 / g.wc;
  }
  const int vw = g.wc * g.cpr;
  // Tile width: a power of two from 8 to 32.  32 columns are 64 contiguous bytes per row and
  // channel (whole sectors), and four rows of halo'd height 6 keep the re-read of halo rows at 1.5;
  // wider maps take several column tiles, the horizontal neighbours come from the image itself.
  g.tw = 8;
  while (g.tw < vw && g.tw < 32) g.tw *= 2;
  g.r = 128 / g.tw;
  g.tiles_x = (vw + g.tw - 1) / g.tw;
  g.strip_rows = ((long long)n + g.cpr - 1) / g.cpr * g.hp;
  g.tiles_y = (g.strip_rows + g.r - 1) / g.r;
  g.n_t = L.dense_nt;
  g.n_tiles_n = (L.c_out + g.n_t - 1) / g.n_t;
  g.k_steps = (L.c_in + 15) / 16;
  g.row_bytes = (g.tw / 8) * 128;
  g.a_lbo = (g.r + 2) * g.row_bytes;
  g.a_copy_bytes = 2 * g.a_lbo;
  g.b_bytes = 9 * g.n_t * 32;
  g.stage_bytes = 3 * g.a_copy_bytes + g.b_bytes;
  g.stage_off = 256;
  g.stages = (kTSmemLimit - g.stage_off) / g.stage_bytes;
  if (g.stages > kMaxTStages) g.stages = kMaxTStages;
  if (g.stages & 1) --g.stages;            // the two producer groups take alternate stages
  if (g.stages < 2) return false;
  if ((g.r + 2) * 2 * (g.tw / 8) * 8 > kMaxTasks * kProdThreadsPerGroup) return false;
  g.relu = 0;
  g.total_tiles = g.tiles_y * g.tiles_x * g.n_tiles_n;
  if (g.tiles_y * g.tiles_x > 0x7FFFFFFFll) return false;
  *out = g;
  return true;
}

}  // namespace

bool tensor_supported(const DeviceLayer& L, int n, int h, int w) {
  TGeo g;
  return n > 0 && h > 0 && w > 0 && tensor_geo(L, n, h, w, &g);
}

// Whether the dense tensor-core path is expected to beat the pattern-sparse kernel: it needs
// enough tiles to occupy the device (it has no channel split), and the zero-inserted contraction
// (9 / (4 x keep) times the surviving multiply-adds, at roughly a third of the tensor peak) must be
// cheaper than the surviving multiply-adds at the ~20 % of the FP32 peak the sparse kernel reaches.
bool tensor_preferred(const DeviceLayer& L, int n, int h, int w) {
  TGeo g;
  if (!tensor_geo(L, n, h, w, &g)) return false;
  if (g.total_tiles < device_sm_count() / 2) return false;
  const double dense = 2.0 * 9.0 * (double)L.c_in * (double)g.n_tiles_n * g.n_t;   // per pixel
  const double sparse = 8.0 * (double)L.n_kept;
  return dense / (0.33 * 2250e12) < sparse / (0.2 * 74.45e12);
}

cudaError_t launch_tensor(const DeviceLayer& L, const void* x, const float* bias, void* y, int n, int h,
                          int w, bool relu, cudaStream_t stream) {
  TGeo g;
  if (!tensor_geo(L, n, h, w, &g)) return cudaErrorInvalidValue;
  g.relu = relu ? 1 : 0;
  const int smem = g.stage_off + g.stages * g.stage_bytes;
  cudaError_t e = cudaFuncSetAttribute(tensor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTSmemLimit);
  if (e != cudaSuccess) return e;
  const long long sms = device_sm_count();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(g.total_tiles < sms ? g.total_tiles : sms), 1, 1);
  cfg.blockDim = dim3(kTensorThreads, 1, 1);
  // more than half of an SM's shared memory: one CTA per SM, whatever the stage count
  cfg.dynamicSmemBytes = (size_t)(smem < 120 * 1024 ? 120 * 1024 : smem);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, tensor_kernel, L, g, (const __half*)x, bias, (__half*)y);
}

}  // namespace pconv
