// Host-side packer: pattern-set validation, per-kernel classification ("layerwise information
// extraction"), filter grouping balanced by surviving-kernel count and same-pattern ordering
// inside a block ("filter kernel reorder"), and emission of the compressed value / code streams.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <memory>
#include <new>
#include <numeric>

#include "pconv_internal.h"

namespace pconv {
namespace {

inline int popcount9(unsigned m) { return __builtin_popcount(m & 0x1FFu); }

// fp32 -> fp16 bits, round to nearest even; returns false on overflow to infinity.
bool float_to_half_rne(float f, uint16_t* out) {
  uint32_t x;
  std::memcpy(&x, &f, 4);
  const uint32_t sign = (x >> 16) & 0x8000u;
  const uint32_t absx = x & 0x7FFFFFFFu;
  if (absx >= 0x7F800000u) return false;  // caller rejects NaN/Inf earlier
  uint32_t h;
  if (absx >= 0x38800000u) {              // normal half range (>= 2^-14)
    const uint32_t mant = absx & 0x7FFFFFu;
    const uint32_t exp = (absx >> 23) - 112;           // rebias 127 -> 15
    h = (exp << 10) | (mant >> 13);
    const uint32_t rem = mant & 0x1FFFu;
    if (rem > 0x1000u || (rem == 0x1000u && (h & 1u))) ++h;  // may carry into the exponent
    if (h >= 0x7C00u) return false;
  } else if (absx >= 0x33000000u) {       // subnormal half: h = round(value * 2^24)
    const uint32_t drop = 126 - (absx >> 23);          // 14..24 low bits of the 24-bit mantissa
    const uint32_t mant = (absx & 0x7FFFFFu) | 0x800000u;
    h = mant >> drop;
    const uint32_t rem = mant & ((1u << drop) - 1u);
    const uint32_t half = 1u << (drop - 1);
    if (rem > half || (rem == half && (h & 1u))) ++h;
  } else {
    h = 0;
  }
  *out = (uint16_t)(sign | h);
  return true;
}

float half_to_float(uint16_t h) {
  const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  const uint32_t exp = (h >> 10) & 0x1Fu;
  const uint32_t mant = h & 0x3FFu;
  uint32_t x;
  if (exp == 0) {
    if (mant == 0) {
      x = sign;
    } else {
      float v = std::ldexp((float)mant, -24);
      std::memcpy(&x, &v, 4);
      x |= sign;
    }
  } else if (exp == 31) {
    x = sign | 0x7F800000u | (mant << 13);
  } else {
    x = sign | ((exp + 112) << 23) | (mant << 13);
  }
  float f;
  std::memcpy(&f, &x, 4);
  return f;
}

struct KernelRec {
  int c;        // input channel
  int pid;      // pattern id in the caller's set
  float v[4];   // values at the mask's set bits, ascending bit order (fp16-rounded if F16)
  uint16_t hv[4];
};

}  // namespace
}  // namespace pconv

using namespace pconv;

extern "C" pconv_status pconv_pack(const float* w, int c_out, int c_in, const uint16_t* patterns,
                                   int n_patterns, int stride, int storage, unsigned flags,
                                   void* stream_v, pconv_handle** out, int* bad_o, int* bad_c) {
  if (!w || !patterns || !out) return PCONV_ERR_NULL;
  if (c_out <= 0 || c_in <= 0 || c_in > 65535 || c_out > (1 << 24)) return PCONV_ERR_SHAPE;
  if (stride != 1 && stride != 2) return PCONV_ERR_SHAPE;
  if (storage != PCONV_F32 && storage != PCONV_F16) return PCONV_ERR_UNSUPPORTED;
  if (flags & ~(unsigned)PCONV_STRICT4) return PCONV_ERR_UNSUPPORTED;
  if (n_patterns < 1 || n_patterns > PCONV_MAX_PATTERNS) return PCONV_ERR_PATTERN_SET;
  for (int p = 0; p < n_patterns; ++p) {
    if (patterns[p] > 0x1FFu || popcount9(patterns[p]) != 4) return PCONV_ERR_PATTERN_SET;
    for (int q = 0; q < p; ++q)
      if (patterns[q] == patterns[p]) return PCONV_ERR_PATTERN_SET;
  }
  cudaStream_t stream = (cudaStream_t)stream_v;

  try {
    // ---- classification -----------------------------------------------------------------
    std::vector<std::vector<KernelRec>> per_filter(c_out);
    long long n_kept = 0;
    long long per_pattern[PCONV_MAX_PATTERNS] = {0};
    for (int o = 0; o < c_out; ++o) {
      for (int c = 0; c < c_in; ++c) {
        const float* k = w + ((size_t)o * c_in + c) * 9;
        unsigned support = 0;
        for (int t = 0; t < 9; ++t) {
          if (!std::isfinite(k[t])) {
            if (bad_o) *bad_o = o;
            if (bad_c) *bad_c = c;
            return PCONV_ERR_RANGE;
          }
          if (k[t] != 0.0f) support |= 1u << t;
        }
        if (!support) continue;
        if ((flags & PCONV_STRICT4) && popcount9(support) != 4) {
          if (bad_o) *bad_o = o;
          if (bad_c) *bad_c = c;
          return PCONV_ERR_KERNEL_NOT_IN_SET;
        }
        int pid = -1;
        for (int p = 0; p < n_patterns; ++p)
          if ((support & ~(unsigned)patterns[p]) == 0) {
            pid = p;
            break;
          }
        if (pid < 0) {
          if (bad_o) *bad_o = o;
          if (bad_c) *bad_c = c;
          return PCONV_ERR_KERNEL_NOT_IN_SET;
        }
        KernelRec r;
        r.c = c;
        r.pid = pid;
        int s = 0;
        for (int t = 0; t < 9; ++t)
          if (patterns[pid] >> t & 1) {
            float v = k[t];
            uint16_t hv = 0;
            if (storage == PCONV_F16) {
              if (!float_to_half_rne(v, &hv)) {
                if (bad_o) *bad_o = o;
                if (bad_c) *bad_c = c;
                return PCONV_ERR_RANGE;
              }
              v = half_to_float(hv);
            }
            r.v[s] = v;
            r.hv[s] = hv;
            ++s;
          }
        per_filter[o].push_back(r);
        ++n_kept;
        ++per_pattern[pid];
      }
    }

    // owned here until the pack has succeeded: an allocation failure further down (the vectors
    // below can throw) must not leak the handle
    std::unique_ptr<pconv_handle> owner(new pconv_handle());
    pconv_handle* h = owner.get();
    std::memset(h, 0, sizeof(*h));
    h->n_patterns = n_patterns;
    h->canonical = true;
    for (int p = 0; p < n_patterns; ++p) {
      h->patterns[p] = patterns[p];
      h->body_id[p] = body_index(patterns[p]);
      if (h->body_id[p] >= 8) h->canonical = false;
    }
    h->n_kept = n_kept;

    // ---- per-filter lists in original order (simple kernel, unpack cross-check) -----------
    std::vector<int> row_ptr(c_out + 1, 0);
    std::vector<uint32_t> csr_idx;
    std::vector<float> csr_val;
    csr_idx.reserve(n_kept);
    csr_val.reserve(4 * n_kept);
    for (int o = 0; o < c_out; ++o) {
      for (const KernelRec& r : per_filter[o]) {
        csr_idx.push_back((uint32_t)r.c | ((uint32_t)patterns[r.pid] << 16));
        csr_val.insert(csr_val.end(), r.v, r.v + 4);
      }
      row_ptr[o + 1] = (int)csr_idx.size();
    }

    // ---- filter grouping: sort by surviving-kernel count, deal in snake order ----------------
    const int n_groups = (c_out + kGroup - 1) / kGroup;
    const int n_chunks = (c_in + kChunk - 1) / kChunk;
    std::vector<int> order(c_out);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
      return per_filter[a].size() > per_filter[b].size();
    });
    std::vector<int> perm((size_t)n_groups * kGroup, -1);
    std::vector<int> fill(n_groups, 0);
    for (int i = 0; i < c_out; ++i) {
      const int round = i / n_groups, pos = i % n_groups;
      const int g = (round & 1) ? (n_groups - 1 - pos) : pos;
      perm[(size_t)g * kGroup + fill[g]++] = order[i];
    }

    // ---- emit blocks ---------------------------------------------------------------------------
    std::vector<BlockDesc> blocks((size_t)n_groups * n_chunks);
    std::vector<uint8_t> codes_s, codes_g;
    std::vector<float> wv32;
    std::vector<uint16_t> wv16;
    long long max_gk = 0, min_gk = -1;
    struct Item { int c, canon_or_pid, slot; const KernelRec* r; };
    std::vector<Item> items;
    std::vector<size_t> cursor(c_out, 0);
    for (int g = 0; g < n_groups; ++g) {
      long long gk = 0;
      for (int s = 0; s < kGroup; ++s) {
        const int o = perm[(size_t)g * kGroup + s];
        if (o >= 0) { gk += (long long)per_filter[o].size(); cursor[o] = 0; }
      }
      max_gk = std::max(max_gk, gk);
      min_gk = (min_gk < 0) ? gk : std::min(min_gk, gk);
      for (int k = 0; k < n_chunks; ++k) {
        const int c0 = k * kChunk, c1 = std::min(c_in, c0 + kChunk);
        items.clear();
        for (int s = 0; s < kGroup; ++s) {
          const int o = perm[(size_t)g * kGroup + s];
          if (o < 0) continue;
          const std::vector<KernelRec>& v = per_filter[o];
          size_t& cur = cursor[o];
          while (cur < v.size() && v[cur].c < c1) {
            items.push_back({v[cur].c, v[cur].pid, s, &v[cur]});
            ++cur;
          }
        }
        // channel-major; inside a channel, same-pattern kernels adjacent, then by slot
        std::stable_sort(items.begin(), items.end(), [](const Item& a, const Item& b) {
          if (a.c != b.c) return a.c < b.c;
          if (a.canon_or_pid != b.canon_or_pid) return a.canon_or_pid < b.canon_or_pid;
          return a.slot < b.slot;
        });
        BlockDesc& bd = blocks[(size_t)g * n_chunks + k];
        std::memset(&bd, 0, sizeof(bd));
        bd.w_off = (uint32_t)((storage == PCONV_F16 ? wv16.size() : wv32.size()) / 4);
        bd.n_k = (uint32_t)items.size();
        while (codes_g.size() % 16) codes_g.push_back(0);
        bd.cs_off = (uint32_t)codes_s.size();
        bd.cg_off = (uint32_t)codes_g.size();
        // Specialised stream: 16-byte records, each a run of kernel codes closed by a terminator
        // (advance to another channel's window, or end); the kernel reads a record with one load.
        // Nothing precedes the first kernel: the descriptor names its channel (`first_ch`).
        // Canonical sets use one-byte codes (15 to a record), any other set two-byte codes (7 to a
        // record) that can name every mask's body.
        const bool wide = !h->canonical;
        const int per_record = wide ? kWideCodesPerRecord : kCodesPerRecord;
        std::vector<uint16_t> rec;
        auto close_record = [&](uint16_t terminator) {
          rec.push_back(terminator);
          while ((int)rec.size() < per_record) rec.push_back((uint16_t)(wide ? kWideEnd : kCodeEnd));
          for (uint16_t c : rec) {
            codes_s.push_back((uint8_t)(c & 0xFF));
            if (wide) codes_s.push_back((uint8_t)(c >> 8));
          }
          rec.clear();
        };
        bd.first_ch = items.empty() ? 0u : (uint32_t)(items.front().c - c0);
        int pos_s = -1;      // channel whose window the specialised stream has loaded (-1: none yet)
        int pos_g = c0 - 1;  // the same for the generic stream
        for (const Item& it : items) {
          if (it.c != pos_g) {
            const int adv = it.c - pos_g;  // 1..kChunk
            const uint16_t cg = (uint16_t)(kGenNext | (adv - 1));
            codes_g.push_back((uint8_t)(cg & 0xFF));
            codes_g.push_back((uint8_t)(cg >> 8));
            pos_g = it.c;
          }
          if (it.c != pos_s) {
            if (pos_s >= 0)
              close_record(wide ? (uint16_t)(((it.c - pos_s) << 8) | kWideAdv)
                                : (uint16_t)(((it.c - pos_s) << 4) | kCodeNext));
            pos_s = it.c;
          }
          if ((int)rec.size() == per_record - 1)   // same channel, next record
            close_record((uint16_t)(wide ? kWideCont : kCodeNext));
          rec.push_back(wide ? (uint16_t)((it.slot << 8) | (kWideBody0 + h->body_id[it.r->pid]))
                             : (uint16_t)((it.slot << 4) | h->body_id[it.r->pid]));
          const uint16_t cg = (uint16_t)((it.slot << 9) | patterns[it.r->pid]);
          codes_g.push_back((uint8_t)(cg & 0xFF));
          codes_g.push_back((uint8_t)(cg >> 8));
          if (storage == PCONV_F16)
            wv16.insert(wv16.end(), it.r->hv, it.r->hv + 4);
          else
            wv32.insert(wv32.end(), it.r->v, it.r->v + 4);
        }
        close_record((uint16_t)(wide ? kWideEnd : kCodeEnd));
        codes_g.push_back((uint8_t)(kGenEnd & 0xFF));
        codes_g.push_back((uint8_t)(kGenEnd >> 8));
        bd.cs_len = (uint32_t)codes_s.size() - bd.cs_off;
        bd.cg_len = (uint32_t)codes_g.size() - bd.cg_off;
      }
    }
    // slack so that a staged block may be read in whole 16-byte pieces
    for (int i = 0; i < 32; ++i) { codes_s.push_back(0); codes_s.push_back(0); codes_g.push_back(0); }
    for (int i = 0; i < 8; ++i) { wv32.push_back(0.f); wv16.push_back(0); }

    // ---- zero-inserted dense weights for the tensor-core path (fp16 storage, stride 1) ----------
    // Filters in original order, tiles of 64 (layers of up to 64 filters) or 128; channels padded to
    // a multiple of 16 with zeros.  Left out for layers whose dense form would exceed 64 MB.
    std::vector<uint16_t> wdense;
    int dense_nt = 0;
    if (storage == PCONV_F16 && stride == 1) {
      const int nt = c_out <= 64 ? 64 : 128;
      const size_t n_tiles = (size_t)(c_out + nt - 1) / nt, k_steps = (size_t)(c_in + 15) / 16;
      const size_t halves = n_tiles * k_steps * 9 * nt * 16;
      if (halves * 2 <= ((size_t)64 << 20)) {
        dense_nt = nt;
        wdense.assign(halves, 0);
        for (int o = 0; o < c_out; ++o) {
          const size_t tile = (size_t)o / nt, on = (size_t)o % nt;
          for (const KernelRec& r : per_filter[o]) {
            const size_t ks = (size_t)r.c / 16, kc = (size_t)r.c % 16;
            int s = 0;
            for (int t = 0; t < 9; ++t) {
              if (!(patterns[r.pid] >> t & 1)) continue;
              const size_t idx = ((((tile * k_steps + ks) * 9 + t) * 2 + kc / 8) * (nt / 8) + on / 8) * 64 +
                                 (on % 8) * 8 + kc % 8;
              wdense[idx] = r.hv[s++];
            }
          }
        }
      }
    }

    // ---- one device allocation, sub-buffers 256-byte aligned ------------------------------------
    struct Part { const void* src; size_t bytes; size_t off; };
    auto align256 = [](size_t v) { return (v + 255) & ~(size_t)255; };
    Part parts[10];
    int np = 0;
    size_t total = 0;
    auto add = [&](const void* src, size_t bytes) {
      parts[np] = {src, bytes, total};
      total += align256(std::max<size_t>(bytes, 4));
      return np++;
    };
    const int i_rp = add(row_ptr.data(), row_ptr.size() * 4);
    const int i_ci = add(csr_idx.data(), csr_idx.size() * 4);
    const int i_cv = add(csr_val.data(), csr_val.size() * 4);
    const int i_bl = add(blocks.data(), blocks.size() * sizeof(BlockDesc));
    const int i_wv = (storage == PCONV_F16) ? add(wv16.data(), wv16.size() * 2)
                                            : add(wv32.data(), wv32.size() * 4);
    const int i_cs = add(codes_s.data(), codes_s.size());
    const int i_cg = add(codes_g.data(), codes_g.size());
    const int i_pm = add(perm.data(), perm.size() * 4);
    const std::vector<unsigned char> zero_block(kStatusBlockBytes, 0);
    const int i_er = add(zero_block.data(), zero_block.size());
    const int i_wd = dense_nt ? add(wdense.data(), wdense.size() * 2) : -1;

    char* dev = nullptr;
    if (cudaMalloc((void**)&dev, total) != cudaSuccess) {
      cudaGetLastError();
      return PCONV_ERR_ALLOC;
    }
    cudaError_t e = cudaSuccess;
    for (int i = 0; i < np && e == cudaSuccess; ++i)
      if (parts[i].bytes)
        e = cudaMemcpyAsync(dev + parts[i].off, parts[i].src, parts[i].bytes,
                            cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) {
      cudaGetLastError();
      cudaFree(dev);
      return PCONV_ERR_CUDA;
    }
    cudaGetDevice(&h->device);
    h->dev_block = dev;
    h->dev_bytes = total;
    h->wvals_bytes = parts[i_wv].bytes;
    h->codes_s_bytes = parts[i_cs].bytes;
    h->codes_g_bytes = parts[i_cg].bytes;
    DeviceLayer& d = h->d;
    d.row_ptr = (const int*)(dev + parts[i_rp].off);
    d.csr_idx = (const uint32_t*)(dev + parts[i_ci].off);
    d.csr_val = (const float*)(dev + parts[i_cv].off);
    d.blocks = (const BlockDesc*)(dev + parts[i_bl].off);
    d.wvals = dev + parts[i_wv].off;
    d.codes_s = (const uint8_t*)(dev + parts[i_cs].off);
    d.wide_codes = h->canonical ? 0 : 1;
    d.codes_g = (const uint8_t*)(dev + parts[i_cg].off);
    d.perm = (const int*)(dev + parts[i_pm].off);
    d.err = (int*)(dev + parts[i_er].off);
    d.wdense = i_wd >= 0 ? dev + parts[i_wd].off : nullptr;
    d.dense_nt = dense_nt;
    d.c_out = c_out;
    d.c_in = c_in;
    d.stride = stride;
    d.storage = storage;
    d.n_groups = n_groups;
    d.n_chunks = n_chunks;
    d.n_kept = n_kept;

    pconv_stats_t& st = h->stats;
    st.c_out = c_out;
    st.c_in = c_in;
    st.stride = stride;
    st.storage = storage;
    st.n_patterns = n_patterns;
    st.kept_kernels = n_kept;
    for (int p = 0; p < PCONV_MAX_PATTERNS; ++p) st.per_pattern[p] = per_pattern[p];
    st.min_per_filter = c_in + 1;
    st.max_per_filter = 0;
    for (int o = 0; o < c_out; ++o) {
      st.min_per_filter = std::min(st.min_per_filter, (int)per_filter[o].size());
      st.max_per_filter = std::max(st.max_per_filter, (int)per_filter[o].size());
    }
    st.n_groups = n_groups;
    st.group_size = kGroup;
    st.max_group_kernels = max_gk;
    st.min_group_kernels = min_gk < 0 ? 0 : min_gk;
    st.packed_bytes = (long long)total;
    st.canonical_patterns = h->canonical ? 1 : 0;
    *out = owner.release();
    return PCONV_OK;
  } catch (const std::bad_alloc&) {
    return PCONV_ERR_ALLOC;
  }
}

extern "C" void pconv_free(pconv_handle* h) {
  if (!h) return;
  if (h->dev_block) cudaFree(h->dev_block);
  delete h;
}

extern "C" pconv_status pconv_stats(const pconv_handle* h, pconv_stats_t* out) {
  if (!h || !out) return PCONV_ERR_NULL;
  *out = h->stats;
  return PCONV_OK;
}

extern "C" pconv_status pconv_filter_order(const pconv_handle* h, int* perm_out) {
  if (!h || !perm_out) return PCONV_ERR_NULL;
  const size_t n = (size_t)h->d.n_groups * kGroup;
  if (cudaMemcpy(perm_out, h->d.perm, n * 4, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return PCONV_ERR_CUDA;
  }
  return PCONV_OK;
}

// Decodes the grouped/chunked device streams (the generic code stream carries the masks) and
// cross-checks them against the per-filter lists; both are downloaded from the device.
extern "C" pconv_status pconv_unpack(const pconv_handle* h, float* w_out) {
  if (!h || !w_out) return PCONV_ERR_NULL;
  const DeviceLayer& d = h->d;
  try {
    const size_t nb = (size_t)d.n_groups * d.n_chunks;
    std::vector<BlockDesc> blocks(nb);
    std::vector<uint8_t> codes(h->codes_g_bytes);
    std::vector<uint8_t> wraw(h->wvals_bytes);
    std::vector<int> perm((size_t)d.n_groups * kGroup);
    std::vector<int> row_ptr(d.c_out + 1);
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess)
      e = cudaMemcpy(blocks.data(), d.blocks, nb * sizeof(BlockDesc), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess)
      e = cudaMemcpy(codes.data(), d.codes_g, codes.size(), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && !wraw.empty())
      e = cudaMemcpy(wraw.data(), d.wvals, wraw.size(), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess)
      e = cudaMemcpy(perm.data(), d.perm, perm.size() * 4, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess)
      e = cudaMemcpy(row_ptr.data(), d.row_ptr, row_ptr.size() * 4, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return PCONV_ERR_CUDA;
    }
    std::memset(w_out, 0, (size_t)d.c_out * d.c_in * 9 * sizeof(float));
    long long decoded = 0;
    for (int g = 0; g < d.n_groups; ++g)
      for (int k = 0; k < d.n_chunks; ++k) {
        const BlockDesc& bd = blocks[(size_t)g * d.n_chunks + k];
        int c = k * kChunk - 1;
        size_t rec = bd.w_off;
        for (uint32_t i = 0; i + 1 < bd.cg_len + 1; i += 2) {
          const uint16_t code = (uint16_t)(codes[bd.cg_off + i] | (codes[bd.cg_off + i + 1] << 8));
          if (code & kGenEnd) break;
          if (code & kGenNext) {
            c += (code & 0xFF) + 1;
            continue;
          }
          const int slot = code >> 9;
          const unsigned mask = code & 0x1FFu;
          const int o = perm[(size_t)g * kGroup + slot];
          if (o < 0 || c < 0 || c >= d.c_in) return PCONV_ERR_CUDA;
          float* k9 = w_out + ((size_t)o * d.c_in + c) * 9;
          int s = 0;
          for (int t = 0; t < 9; ++t)
            if (mask >> t & 1) {
              float v;
              if (d.storage == PCONV_F16) {
                uint16_t hv;
                std::memcpy(&hv, wraw.data() + (rec * 4 + s) * 2, 2);
                v = half_to_float(hv);
              } else {
                std::memcpy(&v, wraw.data() + (rec * 4 + s) * 4, 4);
              }
              k9[t] = v;
              ++s;
            }
          ++rec;
          ++decoded;
        }
      }
    if (decoded != h->n_kept || row_ptr[d.c_out] != (int)h->n_kept) return PCONV_ERR_CUDA;
    return PCONV_OK;
  } catch (const std::bad_alloc&) {
    return PCONV_ERR_ALLOC;
  }
}
