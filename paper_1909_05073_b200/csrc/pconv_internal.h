// Internal declarations shared by the packer, the C ABI and the kernels (product code only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/pconv.h"

namespace pconv {

constexpr int kGroup = 16;         // filters per group (accumulator slots of one consumer warp)
constexpr int kChunk = 8;          // input channels per pipeline stage
constexpr int kMaxBlockKernels = kGroup * kChunk;

// Specialised code stream (the tiled kernel with Tensor-Memory accumulators).  A (group, chunk) block
// is a sequence of 16-byte records; a record is a run of kernel codes closed by one terminator.
// Nothing precedes a block's first kernel: the block descriptor names its channel, and the kernel
// loads that channel's window before it reads the first record.
//
// Narrow codes (one byte, 15 kernels to a record) -- pattern sets inside the canonical eight:
//   low nibble 0..7   kernel: canonical pattern id; high nibble = filter slot
//   low nibble 8      terminator: advance (high nibble, 0..8) channels inside the chunk, load that
//                     channel's window and continue with the next record
//   9                 terminator: end of the block (also fills unused bytes)
constexpr int kCodeNext = 8;
constexpr int kCodeEnd = 9;
constexpr int kCodesPerRecord = 16;
// Wide codes (two bytes, 7 kernels to a record) -- any other set of 4-of-9 masks:
//   low byte 0        terminator: advance (high byte, 0..8) channels, load that channel's window
//                     and continue with the next record
//   low byte 1        terminator: end of the block (also fills unused entries)
//   low byte 2        terminator: the channel's kernels continue in the next record
//   low byte 3..128   kernel: kWideBody0 + index of the body for its mask (body_index()); high
//                     byte = filter slot
constexpr int kWideAdv = 0;
constexpr int kWideEnd = 1;
constexpr int kWideCont = 2;
constexpr int kWideBody0 = 3;
constexpr int kWideCodesPerRecord = 8;
// Generic code stream (two bytes per entry) -- any 4-of-9 mask.
//   (g << 9) | mask   kernel with run-time mask;   0x2000 | (adv-1)   advance;   0x4000   end
constexpr int kGenNext = 0x2000;
constexpr int kGenEnd = 0x4000;

// The eight masks whose bodies come first, in canonical order (bit 3u+v); the bodies of all other
// masks with four bits follow in ascending order of the mask (the generated dispatch code
// enumerates them the same way).
constexpr uint16_t kCanonMasks[8] = {0x03A, 0x09A, 0x0B8, 0x0B2, 0x01B, 0x036, 0x0D8, 0x1B0};
inline int body_index(uint16_t mask) {
  for (int q = 0; q < 8; ++q)
    if (kCanonMasks[q] == mask) return q;
  int idx = 8;
  for (int m = 0; m < 512; ++m) {
    if (__builtin_popcount(m) != 4) continue;
    bool canon = false;
    for (int q = 0; q < 8; ++q) canon = canon || kCanonMasks[q] == m;
    if (canon) continue;
    if (m == mask) return idx;
    ++idx;
  }
  return -1;
}

struct BlockDesc {      // one per (group, chunk); 32 bytes
  uint32_t w_off;       // first kernel record of the block in the value stream
  uint32_t n_k;         // kernel records in the block (<= kMaxBlockKernels)
  uint32_t cs_off;      // byte offset of the specialised codes (16-byte aligned)
  uint32_t cs_len;      // specialised code bytes including the end code
  uint32_t cg_off;      // byte offset of the generic codes (16-byte aligned)
  uint32_t cg_len;      // generic code bytes including the end code
  uint32_t first_ch;    // channel (inside the chunk) of the block's first kernel
  uint32_t pad0;
};

struct DeviceLayer {         // device pointers of one packed layer (passed to kernels by value)
  // per-filter lists in original filter order (simple kernel)
  const int* row_ptr;        // [c_out + 1]
  const uint32_t* csr_idx;   // channel | mask << 16
  const float* csr_val;      // 4 floats per kernel
  // grouped / chunked streams (tiled kernel)
  const BlockDesc* blocks;   // [n_groups][n_chunks]
  const void* wvals;         // 4 values per kernel: fp32 (16 B) or fp16 (8 B)
  const uint8_t* codes_s;    // specialised codes (narrow or wide, see wide_codes)
  const uint8_t* codes_g;    // generic codes
  const int* perm;           // [n_groups * kGroup] original filter index or -1
  int* err;                  // device status block: word 0 = status (0 = fine), then trace words
  int c_out, c_in, stride, storage, n_groups, n_chunks;
  int wide_codes;            // 0 = narrow codes (canonical set), 1 = wide codes
  long long n_kept;          // surviving kernels of the layer
  // zero-inserted dense fp16 weights for the tensor-core path (fp16 storage, stride 1; else null):
  // per (filter tile of dense_nt, 16-channel step) nine [dense_nt x 16] matrices in the K-major
  // core-matrix order of tcgen05 shared-memory descriptors: [tap][k half][filter / 8][filter % 8][k % 8]
  const void* wdense;
  int dense_nt;
};

// Status block: one status word, one pad word, kTraceWords 64-bit trace words (written only by
// builds with -DPCONV_DEV).
constexpr int kTraceWords = 14;
constexpr int kStatusBlockBytes = 8 + 8 * kTraceWords;
__host__ __device__ inline unsigned long long* trace_words(const DeviceLayer& L) {
  return reinterpret_cast<unsigned long long*>(L.err + 2);
}

}  // namespace pconv

struct pconv_handle {
  pconv::DeviceLayer d;
  int device;
  int n_patterns;
  uint16_t patterns[PCONV_MAX_PATTERNS];
  int body_id[PCONV_MAX_PATTERNS];   // body index of each pattern
  bool canonical;                    // every pattern is one of the canonical eight
  pconv_stats_t stats;
  long long n_kept;
  size_t wvals_bytes, codes_s_bytes, codes_g_bytes;
  void* dev_block;                   // the single device allocation
  size_t dev_bytes;
};

namespace pconv {
// Streaming multiprocessors of the current device (cudaDevAttrMultiProcessorCount, looked up once
// per device).  Without a usable device -- the planner also runs on machines that have none -- the
// count of the part this library is written for (B200: 148).
int device_sm_count();
// kernels (defined in the .cu files); all asynchronous on `stream`
cudaError_t launch_simple(const DeviceLayer& L, const void* x, const float* bias, void* y, int n,
                          int h, int w, bool relu, cudaStream_t stream);
cudaError_t launch_tiled(const DeviceLayer& L, const void* x, const float* bias, void* y, int n,
                         int h, int w, bool relu, bool pool, bool reproducible, bool generic_taps,
                         int rmode, bool allow_cluster, void* ws, size_t ws_bytes, cudaStream_t stream);
cudaError_t launch_tensor(const DeviceLayer& L, const void* x, const float* bias, void* y, int n,
                          int h, int w, bool relu, void* ws, size_t ws_bytes, cudaStream_t stream);
size_t tensor_workspace_bytes(const DeviceLayer& L, int n, int h, int w);
bool tensor_supported(const DeviceLayer& L, int n, int h, int w);
bool tensor_preferred(const DeviceLayer& L, int n, int h, int w);
// rmode: what the caller pinned for the tiled kernel: output rows per lane (4, 8, or 0 = the planner
// chooses) | kPinBulk (fp32 chunks fetched by bulk copies into a raw ring)
constexpr int kPinRowsMask = 0xff;
constexpr int kPinBulk = 0x100;
size_t tiled_workspace_bytes(const DeviceLayer& L, int n, int h, int w, int rmode);
bool tiled_supported(const DeviceLayer& L, int n, int h, int w);
bool tiled_plan(const DeviceLayer& L, int n, int h, int w, bool generic_taps, bool with_workspace,
                int rmode, pconv_plan_t* out);
#ifdef PCONV_DEV
cudaError_t dev_set_withhold(int chunk, unsigned spin_limit);   // see pconv_dev.h
#endif
// chains: several consecutive layers of a stack in one persistent launch (kernels_tiled.cu)
bool chain_layer_ok(const DeviceLayer& L, int n, int h, int w, bool pool, long long* ctas);
size_t chain_table_bytes(int n_layers);
bool chain_fill(void* table_host, int index, const DeviceLayer& L, const void* x, const float* bias, void* y,
                int n, int h, int w, bool relu, bool pool, int* status_dev);
size_t chain_workspace_bytes(const void* table_host, int n_layers);
cudaError_t launch_chain(const void* table_dev, const void* table_host, int n_layers, const void* x_first,
                         void* y_last, void* ws, size_t ws_bytes, unsigned int* sync, cudaStream_t stream);
cudaError_t launch_maxpool(const void* x, void* y, int n, int c, int h, int w, int storage,
                           cudaStream_t stream);
}  // namespace pconv
