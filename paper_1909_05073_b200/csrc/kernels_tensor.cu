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
//    step's weights arrive as three bulk copies of three taps each (cp.async.bulk, no tensor map,
//    no multicast), each completing on the mbarrier of its own sub-stage of the weight ring.
//  * Warp roles: warps 0-3 epilogue (warp q reads TMEM lanes 32q..32q+31, adds the bias, applies
//    ReLU, converts to fp16 and stages the tile in shared memory as [filter][pixel]; the 128
//    threads then copy it out in 16-byte pieces, a filter's 8 consecutive pixels each -- the
//    first version stored 2 bytes per lane and column straight from the registers and spent more
//    time in its epilogue than in its MMAs), warp 4 issues the MMAs and owns the TMEM allocation
//    (the whole warp runs the issue loop and waits, elect.sync picks the lane that issues, so the
//    loop stays warp-uniform), warps 5-12 are the A producers (each thread keeps the loads of the next two stages in
//    flight in two register sets while it shifts and stores the current one), warp 13 streams
//    the weights through a ring of their own (three taps per bulk copy).  Two accumulator buffers
//    (2 x n_t columns) let the epilogue of a tile overlap the next tile's MMAs.  CTAs are
//    persistent: item t of a CTA is blockIdx.x + t * gridDim.x.
//  * Weight reuse.  The nine taps make the weight operand of a step (9 x n_t x 16 values) six
//    times larger than the activations it meets (128 pixels x 16 channels, halo included), and
//    measured on the first version -- one pixel tile per weight stage -- the L2-to-SM traffic of
//    the weight stream held the tensor pipe at 23 %.  A work item is therefore mt = 1, 2 or 4
//    vertically adjacent pixel tiles (one halo'd strip of mt * r + 2 rows) that share every weight
//    stage: mt accumulators of n_t columns each.  mt * n_t <= 256 leaves room for two accumulator
//    sets; with 512 columns in use the epilogue of an item is not overlapped.
//  * Every wait is bounded; a wait that runs out records its id (20-25) in the layer's status word,
//    the role stops working, and all roles meet at the common exit where TMEM is released.
//  * The kernel is compiled once per input layout (template parameter MODE): rows of a multiple of
//    8 pixels (one aligned 16-byte load per task), other widths of 8 and more (element-wise), and
//    the narrow maps with 4, 2 and 1 or 3 columns.  The producers' inner loop is instruction-bound
//    (a task is one load, eight funnel shifts and three 16-byte stores), so everything that does
//    not depend on the channel step is worked out once per item.
#include <cuda_fp16.h>

#include "pconv_internal.h"

namespace pconv {
namespace {

typedef unsigned long long u64;

constexpr int kEpiWarps = 4;
constexpr int kMmaWarp = 4;
constexpr int kProdWarp0 = 5;
constexpr int kProdWarps = 8;
constexpr int kProdThreads = 32 * kProdWarps;
constexpr int kBWarp = kProdWarp0 + kProdWarps;   // warp 13: streams the weights
constexpr int kTensorThreads = 32 * (kBWarp + 1);
constexpr int kMaxAStages = 6;            // ring of activation stages (one 16-channel step each)
constexpr int kMaxBStages = 16;           // ring of weight sub-stages (three taps of a step each)
constexpr int kTHeaderBytes = 512;        // barriers and the TMEM base word
constexpr int kMaxTasks = 5;              // A tasks of one producer thread per stage (18 rows x 64 / 256)
constexpr uint32_t kTSpinLimit = 1u << 20;
constexpr uint32_t kTWaitHintNs = 200;
constexpr int kTSmemLimit = 227 * 1024;

struct TGeo {
  int n, h, w, c_in, c_out;
  int hp;            // strip period: h + 1 (image rows + one separator row)
  int wc;            // cell width: w rounded up to a multiple of 8, or to 1, 2, 4 for w < 8
  int cpr;           // cells (images) side by side in a strip row
  int tw, r;         // tile: r strip rows x tw columns, r * tw = 128
  int mt, n_buf;     // pixel tiles per work item (stacked vertically); accumulator sets (1 or 2)
  int rows_a;        // staged rows of an item: mt * r + 2
  int tiles_x;       // column tiles of the virtual width cpr * wc
  int strip_rows, tiles_y;   // strip rows of the batch; items along the strip
  int n_t, n_tiles_n, k_steps;
  int ksplit, kpp;   // parts the channel steps of an item are cut in (1 = none), steps per part
  int a_stages, b_stages;  // ring depths
  int b_resident;          // 1: the layer's whole weight operand fits the ring and is loaded once per CTA
  int a_copy_bytes, a_lbo, row_bytes, a_stage_bytes, a_off;
  int b_bytes, b_sub_bytes, b_off;   // weights of a step (nine taps) / of a sub-stage (three taps)
  int out_off, bias_off;   // the epilogue's staging tile [n_t / 2][128][2] fp16 and the tile's bias [n_t] fp32
  int relu;
  long long total_items;   // tiles_y * tiles_x * n_tiles_n * ksplit
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
// True in exactly one lane of the (converged) warp.  The MMA and weight-stream warps run their
// loops with all 32 lanes, so that addresses and descriptors stay warp-uniform (the tensor-core
// instructions take them from uniform registers), and only the issuing instruction is elected.
__device__ __forceinline__ bool elect_one() {
  uint32_t p;
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "elect.sync _|P, 0xFFFFFFFF;\n\t"
      "selp.u32 %0, 1, 0, P;\n\t}"
      : "=r"(p));
  return p != 0;
}
// The mbarrier receives one arrival when all MMAs issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}

// Development build: CTA 0 leaves, in the layer's trace words, the cycles its roles spent waiting
// and working (0 whole kernel; MMA warp: 1 waiting for free accumulators, 2 for activations, 3 for
// weights, 4 issuing; producers' thread 0: 5 waiting for a free stage, 6 issuing loads, 7 shifting
// and storing; weight stream: 8 waiting for a free sub-stage; epilogue thread 0: 9 waiting for
// accumulators, 10 working).
#ifdef PCONV_DEV
#define T_NOW() clock64()
#define T_ADD(i, t0) do { if (blockIdx.x == 0) tw_[i] += clock64() - (t0); } while (0)
#define T_DECL long long tw_[14] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}
#define T_FLUSH(lo, hi) do { if (blockIdx.x == 0) for (int i_ = (lo); i_ <= (hi); ++i_) trace_words(L)[i_] = (unsigned long long)tw_[i_]; } while (0)
#else
#define T_NOW() 0ll
#define T_ADD(i, t0) do { (void)(t0); } while (0)
#define T_DECL
#define T_FLUSH(lo, hi)
#endif

// Input layouts the kernel is compiled for.
enum { kModeW8 = 0,   // w a multiple of 8: a task is one aligned 16-byte load (+ two neighbours)
       kModeWX = 1,   // any other w >= 5: element-wise loads and stores
       kModeN4 = 2,   // w = 4: two images side by side, 8-byte rows
       kModeN2 = 3,   // w = 2: four images side by side, 4-byte rows
       kModeNX = 4 }; // w = 1 or 3: element-wise, 8 or 2 images side by side

// One A task = (staged row, 8-channel block, column group of 8 pixels, channel within the block):
// 16 bytes of each of the three horizontally shifted copies.  Task t of a stage decodes as
// t = ((row * 2 + block) * (tw / 8) + group) * 8 + channel, so that the 32 lanes of a warp write
// 512 contiguous bytes.

// The image group and row of strip row s, or false for a separator row / outside the strip.
__device__ __forceinline__ bool strip_row(const TGeo& g, int s, int* group, int* row) {
  if (s < 0 || s >= g.strip_rows) return false;
  const int gi = s / g.hp;
  const int lr = s - gi * g.hp;
  *group = gi;
  *row = lr;
  return lr < g.h;
}

__device__ __forceinline__ uint32_t ldg_u16(const unsigned short* p) { return (uint32_t)__ldg(p); }
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// Barrier of the 128 epilogue threads that also tells whether `v` holds for all of them (so that a
// bounded wait that ran out for some of them makes all of them leave together).
__device__ __forceinline__ bool epi_all(bool v) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "bar.red.and.pred p, 1, 128, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)v)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ uint4 lds_v4(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 32 accumulator columns of this warp's 32 lanes; the registers are valid after tmem_ld_wait().
__device__ __forceinline__ void tmem_ld32_issue(uint32_t (&v)[32], uint32_t taddr) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr));
}

// The 8 pixels of one task (one channel, one staged row, one column group) as four packed fp16
// pairs, and the pixels left and right of the group (0 where there is none).  `p` addresses the
// group's first pixel; `aux` is what the item set-up left for the task: in the wide layouts bit 0 /
// bit 1 = a left / right neighbour exists and bits 8.. = the first pixel's column, in the narrow
// ones the number of the group's images that lie inside the batch.
template <int MODE>
__device__ __forceinline__ void load_task(const TGeo& g, const unsigned short* p, uint32_t aux, size_t img,
                                          uint4* v, uint32_t* lft, uint32_t* rgt) {
  *lft = *rgt = 0u;
  if (MODE == kModeW8) {
    *v = __ldg(reinterpret_cast<const uint4*>(p));
    if (aux & 1u) *lft = ldg_u16(p - 1);
    if (aux & 2u) *rgt = ldg_u16(p + 8);
  } else if (MODE == kModeWX) {
    const int vx = (int)(aux >> 8);
    uint32_t e[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) e[i] = (vx + i < g.w) ? ldg_u16(p + i) : 0u;
    *v = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
    if (aux & 1u) *lft = ldg_u16(p - 1);
    if (aux & 2u) *rgt = ldg_u16(p + 8);
  } else if (MODE == kModeN4) {
    uint2 a = make_uint2(0u, 0u), b = a;
    if (aux > 0) a = __ldg(reinterpret_cast<const uint2*>(p));
    if (aux > 1) b = __ldg(reinterpret_cast<const uint2*>(p + img));
    *v = make_uint4(a.x, a.y, b.x, b.y);
  } else if (MODE == kModeN2) {
    uint32_t e[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if ((uint32_t)i < aux) e[i] = __ldg(reinterpret_cast<const uint32_t*>(p + i * img));
    *v = make_uint4(e[0], e[1], e[2], e[3]);
  } else {
    uint32_t e[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int cell = g.wc == 1 ? i : i >> 2;      // w = 1: eight images; w = 3: two cells of four
      const int xin = i - cell * g.wc;
      e[i] = ((uint32_t)cell < aux && xin < g.w) ? ldg_u16(p + cell * img + xin) : 0u;
    }
    *v = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16), e[6] | (e[7] << 16));
  }
}

// A work item: pixel tiles (ty, tx), filter tile nt, and -- when the channel steps are cut in
// `ksplit` parts that different CTAs take -- the first step k0 of its part; mn numbers the
// (pixel, filter) tile whatever the part.
struct TItem {
  int ty, tx, nt, k0;
  long long mn;
};
__device__ __forceinline__ TItem decode_item(const TGeo& g, long long item) {
  TItem it;
  const int kp = (int)(item % g.ksplit);
  it.mn = item / g.ksplit;
  const int mti = (int)(it.mn / g.n_tiles_n);
  it.nt = (int)(it.mn - (long long)mti * g.n_tiles_n);
  it.ty = mti / g.tiles_x;
  it.tx = mti - it.ty * g.tiles_x;
  it.k0 = kp * g.kpp;
  return it;
}

__device__ __forceinline__ void red_add_v4(float* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("red.global.v4.f32.add [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(__uint_as_float(a)),
               "f"(__uint_as_float(b)), "f"(__uint_as_float(c)), "f"(__uint_as_float(d))
               : "memory");
}

template <int MODE>
__global__ void __launch_bounds__(kTensorThreads, 1)
tensor_kernel(const DeviceLayer L, const TGeo g, const __half* __restrict__ x,
              const float* __restrict__ bias, __half* __restrict__ y, float* __restrict__ ws,
              int* __restrict__ tickets) {
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  // barriers: a_full / a_empty per activation stage, b_full / b_empty per weight sub-stage,
  // acc_full[2], acc_empty[2]; then the TMEM base word
  const uint32_t bar_afull = sbase, bar_aempty = sbase + 8 * kMaxAStages;
  const uint32_t bar_bfull = sbase + 16 * kMaxAStages, bar_bempty = bar_bfull + 8 * kMaxBStages;
  const uint32_t bar_accf = bar_bempty + 8 * kMaxBStages, bar_acce = bar_accf + 16;
  volatile uint32_t* tmem_base_s = reinterpret_cast<volatile uint32_t*>(smem + 16 * (kMaxAStages + kMaxBStages) + 32);
  const int acc_cols = g.mt * g.n_t;                          // columns of one accumulator set
  const uint32_t tmem_cols = (uint32_t)(g.n_buf * acc_cols);  // 64 .. 512, a power of two

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) {
    for (int s = 0; s < g.a_stages; ++s) {
      mbar_init(bar_afull + 8 * s, kProdThreads);              // every producer thread
      mbar_init(bar_aempty + 8 * s, 1);                        // one tcgen05.commit
    }
    for (int s = 0; s < g.b_stages; ++s) {
      mbar_init(bar_bfull + 8 * s, 1);                         // the bulk copy's issuer (+ its bytes)
      mbar_init(bar_bempty + 8 * s, 1);                        // one tcgen05.commit
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

  const int my_items = (g.total_items > (long long)blockIdx.x)
                           ? (int)((g.total_items - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;
  const uint32_t row_b = (uint32_t)g.row_bytes;     // bytes of one staged row of core matrices
  const size_t hw = (size_t)g.h * g.w;

  if (warp == kMmaWarp) {
    // ======================================= MMA issuer =======================================
    {
      // instruction descriptor: D fp32, A and B fp16, A pixel-major (MN-major), B K-major, N, M = 128
      const uint32_t idesc = (1u << 4) | (1u << 15) | ((uint32_t)(g.n_t >> 3) << 17) | ((128u >> 4) << 24);
      // descriptors of a stage differ in the start address only: bits 0-13 of the low word, in
      // 16-byte units (shared memory is below 256 KB, so adding an offset never carries out)
      const u64 a_desc0 = smem_desc(0u, (uint32_t)g.a_lbo, 128u);
      const u64 b_desc0 = smem_desc(0u, (uint32_t)(g.n_t / 8) * 128u, 128u);
      const uint32_t copy16 = (uint32_t)g.a_copy_bytes >> 4, row16 = row_b >> 4;
      const uint32_t tap16 = (uint32_t)(g.n_t * 32) >> 4;
      long long ita = 0, itb = 0;    // activation stages and weight sub-stages consumed so far
      bool ok = true;
      T_DECL;
      const long long t_start = T_NOW();
      for (int ti = 0; ti < my_items && ok; ++ti) {
        const int buf = ti % g.n_buf;
        const uint32_t use = (uint32_t)(ti / g.n_buf);
        long long t0 = T_NOW();
        ok = mbar_wait(bar_acce + 8 * buf, (use & 1u) ^ 1u, L.err, 20);
        T_ADD(1, t0);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * acc_cols);
        for (int ks = 0; ks < g.kpp && ok; ++ks, ++ita) {
          const int sa = (int)(ita % g.a_stages);
          t0 = T_NOW();
          ok = mbar_wait(bar_afull + 8 * sa, (uint32_t)((ita / g.a_stages) & 1), L.err, 21);
          T_ADD(2, t0);
          if (!ok) break;
          const u64 a_st = a_desc0 + ((sbase + g.a_off + sa * g.a_stage_bytes) >> 4);
          for (int u = 0; u < 3; ++u, ++itb) {    // the three taps of kernel row u
            const int sb = g.b_resident ? ks * 3 + u : (int)(itb % g.b_stages);
            t0 = T_NOW();
            ok = mbar_wait(bar_bfull + 8 * sb, g.b_resident ? 0u : (uint32_t)((itb / g.b_stages) & 1), L.err, 24);
            T_ADD(3, t0);
            if (!ok) break;
            t0 = T_NOW();
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const u64 b_st = b_desc0 + ((sbase + g.b_off + sb * g.b_sub_bytes) >> 4);
            for (int j = 0; j < g.mt; ++j) {      // the item's pixel tiles share the weights
              const u64 a_tile = a_st + (uint32_t)(j * g.r + u) * row16;
#pragma unroll
              for (int v = 0; v < 3; ++v)
                if (elect_one())
                  umma_f16(d_tmem + (uint32_t)(j * g.n_t), a_tile + v * copy16, b_st + v * tap16, idesc,
                           (ks > 0 || u > 0 || v > 0) ? 1u : 0u);
            }
            // the sub-stage may be refilled once these MMAs are done
            if (!g.b_resident && elect_one()) umma_commit(bar_bempty + 8 * sb);
            T_ADD(4, t0);
          }
          if (ok && elect_one()) umma_commit(bar_aempty + 8 * sa);
        }
        if (ok && elect_one()) umma_commit(bar_accf + 8 * buf);   // the item's accumulators are complete
      }
      T_ADD(0, t_start);
      if (lane == 0) T_FLUSH(0, 4);
    }
    __syncwarp();
  } else if (warp >= kProdWarp0 && warp < kBWarp) {
    // ======================================= A producers ======================================
    const int gt = (warp - kProdWarp0) * 32 + lane;                  // 0..255
    const int cg_shift = g.tw == 32 ? 2 : (g.tw == 16 ? 1 : 0);      // log2(column groups of a row)
    const int n_tasks = g.rows_a << (4 + cg_shift);                 // rows x 2 blocks x groups x 8 channels
    const unsigned short* xs = reinterpret_cast<const unsigned short*>(x);
    const size_t img = (size_t)g.c_in * hw;    // elements of one image
    const size_t step = 16 * hw;               // elements between channel steps
    // what depends on the task only: its place in a copy
    uint32_t dst[kMaxTasks];
#pragma unroll
    for (int q = 0; q < kMaxTasks; ++q) {
      const int t = gt + q * kProdThreads;
      const int c8 = t & 7, cg = (t >> 3) & ((1 << cg_shift) - 1);
      const int kb = (t >> (3 + cg_shift)) & 1, hr = t >> (4 + cg_shift);
      dst[q] = (uint32_t)(kb * g.a_lbo) + (uint32_t)hr * row_b + (uint32_t)(cg * 128 + c8 * 16);
    }
    // keep-masks of the shifted copies on narrow maps: no pixel may see across its image's edge
    // (copy 0 shows the left neighbour: cleared where the pixel is a row's first; copy 2 the right
    // neighbour: cleared where the pixel is the row's last); even / odd = words 0, 2 / 1, 3
    uint32_t zm_even = 0xFFFFFFFFu, zm_odd = 0xFFFFFFFFu, zp_even = 0xFFFFFFFFu, zp_odd = 0xFFFFFFFFu;
    if (MODE == kModeN4 || (MODE == kModeNX && g.wc == 4)) {
      zm_even = 0xFFFF0000u;                                   // pixels 0 and 4 start a row
      zp_odd = (g.w == 4) ? 0x0000FFFFu : 0xFFFF0000u;         // pixels 3, 7 (w = 4) or 2, 6 (w = 3) end one
    } else if (MODE == kModeN2) {
      zm_even = zm_odd = 0xFFFF0000u;                          // even pixels start a row, odd ones end it
      zp_even = zp_odd = 0x0000FFFFu;
    } else if (MODE == kModeNX) {                              // w = 1: no neighbours at all
      zm_even = zm_odd = zp_even = zp_odd = 0u;
    }
    // A thread's loads run two stages ahead of its stores, in two register sets: global-memory
    // latency is then covered by two stage periods, whatever the ring still has free.
    struct RegSet {
      uint4 v[kMaxTasks];
      uint32_t lft[kMaxTasks], rgt[kMaxTasks];
    };
    RegSet set0, set1;
    const unsigned short* src[kMaxTasks];   // of the item being loaded: a task's 8 pixels at step 0 (null = padding)
    uint32_t aux[kMaxTasks];
    int l_k0 = 0;                           // first channel step of the item being loaded
    auto setup_item = [&](int ti) {
      const TItem wi = decode_item(g, blockIdx.x + (long long)ti * gridDim.x);
      const int ty = wi.ty, tx = wi.tx;
      l_k0 = wi.k0;
#pragma unroll
      for (int q = 0; q < kMaxTasks; ++q) {
        const int t = gt + q * kProdThreads;
        src[q] = nullptr;
        aux[q] = 0u;
        if (t < n_tasks) {
          const int c8 = t & 7, cg = (t >> 3) & ((1 << cg_shift) - 1);
          const int kb = (t >> (3 + cg_shift)) & 1, hr = t >> (4 + cg_shift);
          const int ch = kb * 8 + c8;
          int gi, lr;
          if (strip_row(g, ty * (g.mt * g.r) + hr - 1, &gi, &lr)) {
            if (MODE == kModeW8 || MODE == kModeWX) {   // one image per strip row
              const int vx = tx * g.tw + cg * 8;        // column of the group's first pixel
              if (vx < g.w) {
                src[q] = xs + (((size_t)gi * g.c_in + ch) * g.h + lr) * (size_t)g.w + vx;
                aux[q] = (vx > 0 ? 1u : 0u) | (vx + 8 < g.w ? 2u : 0u) | ((uint32_t)vx << 8);
              }
            } else {                                    // 8 / wc images side by side: the first one
              src[q] = xs + (((size_t)gi * g.cpr * g.c_in + ch) * g.h + lr) * (size_t)g.w;
              aux[q] = (uint32_t)min(g.cpr, g.n - gi * g.cpr);
            }
          }
        }
      }
    };
    // (l_ti, l_ks): the next stage to load; loading past the last stage does nothing
    int l_ti = 0, l_ks = 0;
    if (my_items > 0) setup_item(0);
    auto load_next = [&](RegSet& rs) {
#pragma unroll
      for (int q = 0; q < kMaxTasks; ++q) {
        rs.v[q] = make_uint4(0u, 0u, 0u, 0u);
        rs.lft[q] = rs.rgt[q] = 0u;
      }
      if (l_ti >= my_items) return;
      // channels beyond c_in (last step of a layer whose depth is no multiple of 16) are zeros
      const int ch_limit = g.c_in - (l_k0 + l_ks) * 16;
      const size_t chan_off = (size_t)(l_k0 + l_ks) * step;
#pragma unroll
      for (int q = 0; q < kMaxTasks; ++q) {
        if (src[q] == nullptr) continue;
        if (ch_limit < 16) {
          const int t = gt + q * kProdThreads;
          if (((((t >> (3 + cg_shift)) & 1) << 3) | (t & 7)) >= ch_limit) continue;
        }
        load_task<MODE>(g, src[q] + chan_off, aux[q], img, &rs.v[q], &rs.lft[q], &rs.rgt[q]);
      }
      if (++l_ks == g.kpp) {
        l_ks = 0;
        if (++l_ti < my_items) setup_item(l_ti);
      }
    };
    const uint32_t copy_b = (uint32_t)g.a_copy_bytes;
    const long long n_stages = (long long)my_items * g.kpp;
    T_DECL;
    auto store_stage = [&](const RegSet& rs, long long it) -> bool {
      const int s = (int)(it % g.a_stages);
      long long t0 = T_NOW();
      const bool got = mbar_wait(bar_aempty + 8 * s, (uint32_t)(((it / g.a_stages) & 1) ^ 1), L.err, 22);
      T_ADD(5, t0);
      if (!got) return false;
      t0 = T_NOW();
      const uint32_t a0 = sbase + g.a_off + s * g.a_stage_bytes;
#pragma unroll
      for (int q = 0; q < kMaxTasks; ++q) {
        if (gt + q * kProdThreads >= n_tasks) continue;
        const uint4 c = rs.v[q];
        // copy 0: pixel p holds input column p - 1;  copy 2: column p + 1
        uint4 m1, p1;
        m1.x = __funnelshift_l(rs.lft[q] << 16, c.x, 16);
        m1.y = __funnelshift_l(c.x, c.y, 16);
        m1.z = __funnelshift_l(c.y, c.z, 16);
        m1.w = __funnelshift_l(c.z, c.w, 16);
        p1.x = __funnelshift_r(c.x, c.y, 16);
        p1.y = __funnelshift_r(c.y, c.z, 16);
        p1.z = __funnelshift_r(c.z, c.w, 16);
        p1.w = __funnelshift_r(c.w, rs.rgt[q], 16);
        if (MODE >= kModeN4) {
          m1.x &= zm_even; m1.y &= zm_odd; m1.z &= zm_even; m1.w &= zm_odd;
          p1.x &= zp_even; p1.y &= zp_odd; p1.z &= zp_even; p1.w &= zp_odd;
        }
        const uint32_t d = a0 + dst[q];
        sts128(d, m1.x, m1.y, m1.z, m1.w);
        sts128(d + copy_b, c.x, c.y, c.z, c.w);
        sts128(d + 2 * copy_b, p1.x, p1.y, p1.z, p1.w);
      }
      // generic-proxy stores must be visible to the tensor core's (async proxy) reads
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(bar_afull + 8 * s);
      T_ADD(7, t0);
      return true;
    };
    load_next(set0);
    load_next(set1);
    for (long long it = 0; it < n_stages; it += 2) {
      if (!store_stage(set0, it)) break;
      long long t0 = T_NOW();
      load_next(set0);
      T_ADD(6, t0);
      if (it + 1 >= n_stages) break;
      if (!store_stage(set1, it + 1)) break;
      t0 = T_NOW();
      load_next(set1);
      T_ADD(6, t0);
    }
    if (gt == 0) T_FLUSH(5, 7);
  } else if (warp == kBWarp) {
    // ======================================= weight stream ====================================
    // One thread: per (item, step, kernel row) one bulk copy of three taps' [n_t x 16] matrices
    // into the next free sub-stage, as far ahead of the MMAs as the ring allows.
    {
      bool ok = true;
      long long itb = 0;
      T_DECL;
      for (int ti = 0; ti < (g.b_resident ? min(my_items, 1) : my_items) && ok; ++ti) {
        const TItem wi = decode_item(g, blockIdx.x + (long long)ti * gridDim.x);
        const char* wsrc = reinterpret_cast<const char*>(L.wdense) +
                           ((size_t)wi.nt * g.k_steps + wi.k0) * g.b_bytes;
        for (int ks = 0; ks < g.kpp && ok; ++ks) {
          for (int u = 0; u < 3; ++u, ++itb) {
            const int sb = (int)(itb % g.b_stages);
            const long long t0 = T_NOW();
            ok = mbar_wait(bar_bempty + 8 * sb, (uint32_t)(((itb / g.b_stages) & 1) ^ 1), L.err, 25);
            T_ADD(8, t0);
            if (!ok) break;
            if (elect_one()) {
              mbar_arrive_expect_tx(bar_bfull + 8 * sb, (uint32_t)g.b_sub_bytes);
              bulk_copy_g2s(sbase + g.b_off + sb * g.b_sub_bytes,
                            wsrc + (size_t)ks * g.b_bytes + (size_t)u * g.b_sub_bytes,
                            (uint32_t)g.b_sub_bytes, bar_bfull + 8 * sb);
            }
          }
        }
      }
      if (lane == 0) T_FLUSH(8, 8);
    }
    __syncwarp();
  } else {
    // ======================================= epilogue =========================================
    // Accumulators (lane = pixel, column = filter) -> bias, ReLU, fp16 -> shared memory as
    // [filter][pixel] -> 16-byte pieces (8 consecutive pixels of a filter) to y.
    const int q = warp;                       // TMEM lane quadrant
    const int m = 32 * q + lane;              // this lane's pixel of a tile
    const int et = tid;                       // 0..127
    const uint32_t out_s = sbase + (uint32_t)g.out_off;       // [n_t / 2][128] pairs of fp16
    // copy-out: this thread always handles pixel group pg (8 pixels) of filter pairs f0, f0 + 8, ...
    const int pg = et & 15, f0 = et >> 4;
    const int ctr = (pg * 8) / g.tw, ctc = (pg * 8) - ctr * g.tw;   // the group's tile row / first column
    bool ok = true;
    T_DECL;
    for (int ti = 0; ti < my_items && ok; ++ti) {
      const TItem wi = decode_item(g, blockIdx.x + (long long)ti * gridDim.x);
      const int nt = wi.nt, ty = wi.ty, tx = wi.tx;
      const int buf = ti % g.n_buf;
      const uint32_t use = (uint32_t)(ti / g.n_buf);
      const int o_base = nt * g.n_t;
      long long t0 = T_NOW();
      const int n_f = min(g.n_t, g.c_out - o_base);            // real filters of this tile
      epi_sync();                                              // the previous item's bias is no longer read
      if (et < g.n_t)
        reinterpret_cast<float*>(smem + g.bias_off)[et] = (bias && et < n_f) ? __ldg(bias + o_base + et) : 0.f;
      ok = mbar_wait(bar_accf + 8 * buf, use & 1u, L.err, 23);
      ok = epi_all(ok);                                        // bias staged; all leave together if a wait ran out
      T_ADD(9, t0);
      if (!ok) break;
      t0 = T_NOW();
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // Channel steps cut in parts: every part adds its accumulators to the (pixel, filter) tile's
      // fp32 sums in the workspace ([tile j][filter / 4][pixel][4]: a lane's four consecutive
      // filters are one 16-byte reduction) and takes a ticket; the part that draws the last one
      // reads the sums back -- instead of Tensor Memory -- and finishes the tile as usual,
      // leaving sums and ticket zeroed.
      float* wsb = nullptr;
      bool finish = true;
      if (g.ksplit > 1) {
        wsb = ws + (size_t)wi.mn * ((size_t)g.mt * g.n_t * 128);
        for (int j = 0; j < g.mt; ++j) {
          const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * acc_cols + j * g.n_t);
          for (int j0 = 0; j0 < n_f; j0 += 32) {
            uint32_t acc[32];
            tmem_ld32_issue(acc, taddr + (uint32_t)j0);
            tmem_ld_wait();
            float* pw = wsb + (((size_t)j * (g.n_t / 4) + (j0 >> 2)) * 128 + m) * 4;
#pragma unroll
            for (int i = 0; i < 8; ++i)
              red_add_v4(pw + (size_t)i * 512, acc[4 * i], acc[4 * i + 1], acc[4 * i + 2], acc[4 * i + 3]);
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        mbar_arrive(bar_acce + 8 * buf);                       // the accumulators have been read
        __threadfence();
        epi_sync();
        volatile int* last_s = reinterpret_cast<volatile int*>(smem + 16 * (kMaxAStages + kMaxBStages) + 36);
        if (et == 0) {
          const int t = atomicAdd(tickets + wi.mn, 1);
          if (t == g.ksplit - 1) tickets[wi.mn] = 0;
          *last_s = (t == g.ksplit - 1) ? 1 : 0;
        }
        epi_sync();
        finish = *last_s != 0;
        if (finish) __threadfence();
      }
      for (int j = 0; finish && j < g.mt; ++j) {
        long long t1 = T_NOW();
        const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(buf * acc_cols + j * g.n_t);
        // Two adjacent filters of a pixel are converted together (the packed fp16 conversion runs
        // at full rate, the scalar one at a quarter of it: it alone took longer than the MMAs of
        // a tile) and staged as one 32-bit word: [filter pair][pixel].  Plain shared-memory
        // accesses, not asm: the compiler may overlap the columns.  The TMEM load of the next 32
        // columns is in flight while the current ones are converted.
        auto stage_block = [&](const uint32_t (&acc)[32], int j0) {
          // (the 32 bias values first: a load after a store to shared memory could not be moved up)
          const float4* bias_p = reinterpret_cast<const float4*>(smem + g.bias_off + 4 * j0);
          float bv[32];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float4 b4 = bias_p[i];
            bv[4 * i] = b4.x;
            bv[4 * i + 1] = b4.y;
            bv[4 * i + 2] = b4.z;
            bv[4 * i + 3] = b4.w;
          }
          __half2* out_p = reinterpret_cast<__half2*>(smem + g.out_off) + (size_t)(j0 >> 1) * 128 + m;
#pragma unroll
          for (int jj = 0; jj < 32; jj += 2) {
            float v0 = __uint_as_float(acc[jj]) + bv[jj];
            float v1 = __uint_as_float(acc[jj + 1]) + bv[jj + 1];
            if (g.relu) {
              v0 = fmaxf(v0, 0.f);
              v1 = fmaxf(v1, 0.f);
            }
            out_p[(jj >> 1) * 128] = __floats2half2_rn(v0, v1);
          }
        };
        uint32_t acc0[32], acc1[32];
        if (g.ksplit > 1) {
          for (int j0 = 0; j0 < n_f; j0 += 32) {
            float4* pw = reinterpret_cast<float4*>(wsb + (((size_t)j * (g.n_t / 4) + (j0 >> 2)) * 128 + m) * 4);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float4 f4 = __ldcg(pw + (size_t)i * 128);
              acc0[4 * i] = __float_as_uint(f4.x);
              acc0[4 * i + 1] = __float_as_uint(f4.y);
              acc0[4 * i + 2] = __float_as_uint(f4.z);
              acc0[4 * i + 3] = __float_as_uint(f4.w);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) pw[(size_t)i * 128] = make_float4(0.f, 0.f, 0.f, 0.f);
            stage_block(acc0, j0);
          }
        } else {
          tmem_ld32_issue(acc0, taddr);
          tmem_ld_wait();
          for (int j0 = 0; j0 < n_f; j0 += 64) {
            if (j0 + 32 < n_f) tmem_ld32_issue(acc1, taddr + (uint32_t)(j0 + 32));
            stage_block(acc0, j0);
            tmem_ld_wait();
            if (j0 + 32 < n_f) {
              if (j0 + 64 < n_f) tmem_ld32_issue(acc0, taddr + (uint32_t)(j0 + 64));
              stage_block(acc1, j0 + 32);
              tmem_ld_wait();
            }
          }
          if (j == g.mt - 1) {   // the accumulators have been read: the MMA warp may reuse them
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(bar_acce + 8 * buf);
          }
        }
        T_ADD(11, t1);
        t1 = T_NOW();
        epi_sync();                                            // the tile is staged
        T_ADD(12, t1);
        t1 = T_NOW();
        // where this thread's pixel group goes
        int gi = 0, lr = 0;
        const bool row_ok = strip_row(g, (ty * g.mt + j) * g.r + ctr, &gi, &lr);
        const int vx = tx * g.tw + ctc;
        bool grp_ok = row_ok;
        __half* dstp = y;
        int cells = 0;
        if (MODE == kModeW8 || MODE == kModeWX) {
          grp_ok = grp_ok && vx < g.w;
          if (grp_ok) dstp = y + (((size_t)gi * g.c_out + o_base) * g.h + lr) * (size_t)g.w + vx;
        } else if (grp_ok) {
          // narrow maps: the group is 8 / wc images side by side, w pixels of each are real
          cells = min(g.cpr, g.n - gi * g.cpr);
          dstp = y + (((size_t)gi * g.cpr * g.c_out + o_base) * g.h + lr) * (size_t)g.w;
        }
        if (grp_ok) {
          const int npx = min(8, g.w - vx);                    // kModeWX: real pixels of the group
          const size_t oimg = (size_t)g.c_out * hw;
          for (int fp = f0; 2 * fp < n_f; fp += 8) {
            // 8 pixels x {filter 2 fp, filter 2 fp + 1} -> 8 pixels of each filter
            const uint4 a = lds_v4(out_s + (uint32_t)(fp * 512 + pg * 32));
            const uint4 b = lds_v4(out_s + (uint32_t)(fp * 512 + pg * 32 + 16));
            uint4 vv[2];
            vv[0] = make_uint4(__byte_perm(a.x, a.y, 0x5410), __byte_perm(a.z, a.w, 0x5410),
                               __byte_perm(b.x, b.y, 0x5410), __byte_perm(b.z, b.w, 0x5410));
            vv[1] = make_uint4(__byte_perm(a.x, a.y, 0x7632), __byte_perm(a.z, a.w, 0x7632),
                               __byte_perm(b.x, b.y, 0x7632), __byte_perm(b.z, b.w, 0x7632));
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int f = 2 * fp + e;
              if (f >= n_f) break;
              __half* dp = dstp + (size_t)f * hw;
              const uint32_t wds[4] = {vv[e].x, vv[e].y, vv[e].z, vv[e].w};
              if (MODE == kModeW8) {
                *reinterpret_cast<uint4*>(dp) = vv[e];
              } else if (MODE == kModeWX) {
#pragma unroll
                for (int i = 0; i < 8; ++i)
                  if (i < npx) reinterpret_cast<unsigned short*>(dp)[i] = (unsigned short)(wds[i >> 1] >> (16 * (i & 1)));
              } else if (MODE == kModeN4) {
                if (cells > 0) *reinterpret_cast<uint2*>(dp) = make_uint2(wds[0], wds[1]);
                if (cells > 1) *reinterpret_cast<uint2*>(dp + oimg) = make_uint2(wds[2], wds[3]);
              } else if (MODE == kModeN2) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                  if (i < cells) *reinterpret_cast<uint32_t*>(dp + i * oimg) = wds[i];
              } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  const int cell = g.wc == 1 ? i : i >> 2;
                  const int xin = i - cell * g.wc;
                  if (cell < cells && xin < g.w)
                    reinterpret_cast<unsigned short*>(dp + cell * oimg)[xin] =
                        (unsigned short)(wds[i >> 1] >> (16 * (i & 1)));
                }
              }
            }
          }
        }
        T_ADD(13, t1);
        epi_sync();                                            // staging buffer free again
      }
      T_ADD(10, t0);
    }
    if (et == 0) T_FLUSH(9, 13);
  }

  // ---- common exit ----------------------------------------------------------------------------
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kMmaWarp)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols)
                 : "memory");
}

// Geometry of a launch with mt pixel tiles per work item; false if it does not fit.
bool tensor_geo_mt(const DeviceLayer& L, int n, int h, int w, int mt, int ksplit, TGeo* out) {
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
  // channel (whole sectors); wider maps take several column tiles, the horizontal neighbours
  // come from the image itself.
  g.tw = 8;
  while (g.tw < vw && g.tw < 32) g.tw *= 2;
  g.r = 128 / g.tw;
  g.tiles_x = (vw + g.tw - 1) / g.tw;
  const long long strip = ((long long)n + g.cpr - 1) / g.cpr * g.hp;
  if (strip > 0x3FFFFFFF) return false;
  g.strip_rows = (int)strip;
  g.n_t = L.dense_nt;
  if (mt * g.n_t > 512) return false;
  g.mt = mt;
  g.n_buf = (2 * mt * g.n_t <= 512) ? 2 : 1;
  g.rows_a = mt * g.r + 2;
  g.tiles_y = (g.strip_rows + mt * g.r - 1) / (mt * g.r);
  g.n_tiles_n = (L.c_out + g.n_t - 1) / g.n_t;
  g.k_steps = (L.c_in + 15) / 16;
  if (ksplit < 1 || g.k_steps % ksplit != 0) return false;
  g.ksplit = ksplit;
  g.kpp = g.k_steps / ksplit;
  g.row_bytes = (g.tw / 8) * 128;
  g.a_lbo = g.rows_a * g.row_bytes;
  g.a_copy_bytes = 2 * g.a_lbo;
  g.b_bytes = 9 * g.n_t * 32;
  g.b_sub_bytes = 3 * g.n_t * 32;
  g.a_stage_bytes = 3 * g.a_copy_bytes;
  // Shared memory: barriers, activation ring, weight ring, the epilogue's staging tile and bias.
  // The producers keep two stages of loads in registers, so three activation stages are enough;
  // the weight ring takes what is left (what matters is how many steps of MMAs it covers: a
  // sub-stage comes back only after its MMAs have completed and a copy from L2 has landed, about
  // 2 us, while a step of one tile is 0.3 us of MMAs), and what the weight ring cannot use goes
  // back to the activations.
  const int epi_bytes = g.n_t * 256 + g.n_t * 4;
  const int avail = kTSmemLimit - kTHeaderBytes - epi_bytes;
  g.a_stages = (3 * g.a_stage_bytes + 6 * g.b_sub_bytes <= avail) ? 3 : 2;
  g.b_stages = (avail - g.a_stages * g.a_stage_bytes) / g.b_sub_bytes;
  if (g.b_stages > kMaxBStages) g.b_stages = kMaxBStages;
  if (g.b_stages < 3) return false;
  // a layer with one filter tile whose weights all fit keeps them: nothing is streamed again
  g.b_resident = 0;
  if (ksplit == 1 && g.n_tiles_n == 1 && 3 * g.k_steps <= kMaxBStages &&
      2 * g.a_stage_bytes + 3 * g.k_steps * g.b_sub_bytes <= avail) {
    g.b_resident = 1;
    g.b_stages = 3 * g.k_steps;
    g.a_stages = 2;
  }
  while (g.a_stages < kMaxAStages &&
         (g.a_stages + 1) * g.a_stage_bytes + g.b_stages * g.b_sub_bytes <= avail)
    ++g.a_stages;
  g.a_off = kTHeaderBytes;
  g.b_off = g.a_off + g.a_stages * g.a_stage_bytes;
  g.out_off = g.b_off + g.b_stages * g.b_sub_bytes;
  g.bias_off = g.out_off + g.n_t * 256;
  if (g.rows_a * 2 * (g.tw / 8) * 8 > kMaxTasks * kProdThreads) return false;
  g.relu = 0;
  g.total_items = (long long)g.tiles_y * g.tiles_x * g.n_tiles_n * ksplit;
  *out = g;
  return true;
}

// The launch geometry: pixel tiles per item chosen by an estimate of the launch's duration in
// units of one MMA (128 x n_t x 16): a CTA runs ceil(items / SMs) items one after the other; a step
// of an item issues 9 * mt MMAs and cannot be shorter than the hand-over of a stage between the
// producers, the weight stream and the MMA warp (measured: about eighteen MMAs' time per step when
// the step itself is shorter: the rings then cover less than the time a stage takes to come back); an item ends with the epilogue of its mt tiles, overlapped with the next item's steps
// only if two accumulator sets fit.
bool tensor_geo(const DeviceLayer& L, int n, int h, int w, bool allow_split, TGeo* out) {
  const long long sms = device_sm_count();
  bool found = false;
  double best = 0.0;
  for (int mt = 4; mt >= 1; mt /= 2) {
    TGeo g;
    if (!tensor_geo_mt(L, n, h, w, mt, 1, &g)) continue;
    const double waves = (double)((g.total_items + sms - 1) / sms);
    const double step = 9.0 * mt > 18.0 ? 9.0 * mt : 18.0;
    const double epilogue = 6.0 * mt;
    const double cost = waves * (g.k_steps * step + (g.n_buf == 1 || waves == 1.0 ? epilogue : 0.0)) + epilogue;
    if (!found || cost < best) {
      found = true;
      best = cost;
      *out = g;
    }
  }
  // Too few tiles for the device even one by one (small maps, deep layers): cut the channel steps
  // in parts that different CTAs take; the parts meet in an fp32 workspace (see the epilogue).
  if (found && allow_split && out->mt == 1 && 2 * out->total_items <= sms) {
    int ksplit = 1;
    for (int d = 2; d <= 8; ++d)
      if (out->k_steps % d == 0 && out->k_steps / d >= 4 && out->total_items * d <= sms) ksplit = d;
    TGeo g;
    if (ksplit > 1 && tensor_geo_mt(L, n, h, w, 1, ksplit, &g)) *out = g;
  }
  return found;
}

// Workspace of a split launch: fp32 sums of every (pixel, filter) tile, then a ticket per tile.
size_t tensor_sums_bytes(const TGeo& g) {
  return (size_t)(g.total_items / g.ksplit) * g.mt * g.n_t * 128 * sizeof(float);
}

}  // namespace

bool tensor_supported(const DeviceLayer& L, int n, int h, int w) {
  TGeo g;
  return n > 0 && h > 0 && w > 0 && tensor_geo(L, n, h, w, false, &g);
}

size_t tensor_workspace_bytes(const DeviceLayer& L, int n, int h, int w) {
  TGeo g;
  if (n <= 0 || h <= 0 || w <= 0 || !tensor_geo(L, n, h, w, true, &g) || g.ksplit <= 1) return 0;
  return ((tensor_sums_bytes(g) + 255) & ~(size_t)255) +
         (((size_t)(g.total_items / g.ksplit) * sizeof(int) + 255) & ~(size_t)255);
}

// Whether the dense tensor-core path is expected to beat the pattern-sparse kernel: it needs
// enough pixel tiles to occupy a fair part of the device (it has no channel split), and the
// zero-inserted contraction over the padded shape (channels to 16, filters to the tile) at the
// fifth of the tensor peak this kernel reaches must be cheaper than the surviving multiply-adds at
// the fifth of the FP32 peak the sparse kernel reaches.  (Measured on the CIFAR-shaped stack at
// batch 256: faster on every layer but the 3-channel first one, which this rule leaves to the
// sparse kernel.)
bool tensor_preferred(const DeviceLayer& L, int n, int h, int w) {
  TGeo g;
  if (!tensor_geo(L, n, h, w, false, &g)) return false;
  if (g.total_items * g.mt < device_sm_count() / 4) return false;
  const double dense = 2.0 * 9.0 * (16.0 * g.k_steps) * ((double)g.n_tiles_n * g.n_t);   // per pixel
  const double sparse = 8.0 * (double)L.n_kept;
  return dense / (0.2 * 2250e12) < sparse / (0.2 * 74.45e12);
}

template <int MODE>
cudaError_t launch_tensor_mode(const DeviceLayer& L, const TGeo& g, const void* x, const float* bias, void* y,
                               float* ws, int* tickets, cudaStream_t stream) {
  const int smem = g.bias_off + g.n_t * 4;
  cudaError_t e = cudaFuncSetAttribute(tensor_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kTSmemLimit);
  if (e != cudaSuccess) return e;
  const long long sms = device_sm_count();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(g.total_items < sms ? g.total_items : sms), 1, 1);
  cfg.blockDim = dim3(kTensorThreads, 1, 1);
  // more than half of an SM's shared memory: one CTA per SM, whatever the stage count
  cfg.dynamicSmemBytes = (size_t)(smem < 120 * 1024 ? 120 * 1024 : smem);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, tensor_kernel<MODE>, L, g, (const __half*)x, bias, (__half*)y, ws, tickets);
}

cudaError_t launch_tensor(const DeviceLayer& L, const void* x, const float* bias, void* y, int n, int h,
                          int w, bool relu, void* ws, size_t ws_bytes, cudaStream_t stream) {
  TGeo g;
  const size_t need = ws ? tensor_workspace_bytes(L, n, h, w) : 0;
  const bool split = need > 0 && ws_bytes >= need;
  if (!tensor_geo(L, n, h, w, split, &g)) return cudaErrorInvalidValue;
  g.relu = relu ? 1 : 0;
  float* sums = nullptr;
  int* tickets = nullptr;
  if (g.ksplit > 1) {
    sums = (float*)ws;
    tickets = (int*)((char*)ws + ((tensor_sums_bytes(g) + 255) & ~(size_t)255));
  }
  if (w >= 8 && w % 8 == 0) return launch_tensor_mode<kModeW8>(L, g, x, bias, y, sums, tickets, stream);
  if (w >= 5) return launch_tensor_mode<kModeWX>(L, g, x, bias, y, sums, tickets, stream);
  if (w == 4) return launch_tensor_mode<kModeN4>(L, g, x, bias, y, sums, tickets, stream);
  if (w == 2) return launch_tensor_mode<kModeN2>(L, g, x, bias, y, sums, tickets, stream);
  return launch_tensor_mode<kModeNX>(L, g, x, bias, y, sums, tickets, stream);
}

}  // namespace pconv
