// Graded single-query decode attention (paper Sec. 3.7: dequantisation inside the online-softmax
// loop, all KV heads of a layer in one launch, split-context partials reduced separately).
//
// Work split: every warp owns a contiguous, byte-balanced range of one stream's items (closed
// blocks of any level, the exact tail block, groups of exact residual rows) and keeps its own
// online-softmax state for the g <= 8 query heads of the KV head (one read of the KV bytes serves
// the whole GQA group, Sec. 3.1).  Warps never wait on each other: each one runs a private
// double-buffered cp.async pipeline (global -> shared, 16 B per lane, 512 B per instruction) and
// reads back only what it staged, so there are no block-level barriers and no spin waits.
//
// Math: S^T[tokens x heads] = K[tokens x ch] Q^T and O^T[ch x heads] += V^T[ch x tokens] P^T on
// mma.m16n8k16 with the query heads as the n = 8 dimension.  Quantised codes are stored in
// A-fragment order (gkv_layout.cuh), unpacked with the fp16 magic-number trick (0x6400 | code),
// dequantised with one hfma2 per pair and fed to f16 MMAs; exact rows go through ldmatrix and
// bf16 MMAs with P split into hi + lo bf16 parts so that its rounding stays below 2^-16.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gkv_internal.h"

namespace gkv {
namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr float kNegInf = -__builtin_huge_valf();

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&a)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&a)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
               : "r"(addr));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t lop3_and_or(uint32_t x, uint32_t mask, uint32_t orv) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;\n" : "=r"(r) : "r"(x), "r"(mask), "r"(orv));   // (x & mask) | orv
  return r;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;\n" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}
__device__ __forceinline__ uint32_t h2_as_u32(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u32_as_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16lo_to_f32(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// Unpack the four A registers of one MMA from packed codes and dequantise them:
// a0,a1 use (scA, zrA), a2,a3 use (scB, zrB).  `w` is the 32-bit word holding the pairs and
// `odd` tells (for 2-bit codes) whether the MMA index is odd (pairs 4..7 of the word).
template <int BITS>
__device__ __forceinline__ void unpack_dequant(uint32_t w0, uint32_t w1, bool odd, __half2 scA, __half2 zrA,
                                               __half2 scB, __half2 zrB, uint32_t (&a)[4]) {
  constexpr uint32_t kMagic = 0x64006400u;   // half2(1024, 1024)
  __half2 c0, c1, c2, c3;
  if constexpr (BITS == 8) {
    // w0 = pairs (a0, a1), w1 = pairs (a2, a3); pair pos 0: bytes 0/2, pos 1: bytes 1/3;
    // selector 5 picks the 0x64 byte of the magic word as the high byte of each half
    const __half2 k1024 = __float2half2_rn(1024.f);
    c0 = __hsub2(u32_as_h2(prmt(w0, kMagic, 0x5250u)), k1024);
    c1 = __hsub2(u32_as_h2(prmt(w0, kMagic, 0x5351u)), k1024);
    c2 = __hsub2(u32_as_h2(prmt(w1, kMagic, 0x5250u)), k1024);
    c3 = __hsub2(u32_as_h2(prmt(w1, kMagic, 0x5351u)), k1024);
  } else if constexpr (BITS == 4) {
    // w0 holds the four pairs: pos p at bits 4p / 16 + 4p
    const __half2 k1024 = __float2half2_rn(1024.f);
    const __half2 k16th = __float2half2_rn(0.0625f), km64 = __float2half2_rn(-64.f);
    const uint32_t hi = w0 >> 8;
    c0 = __hsub2(u32_as_h2(lop3_and_or(w0, 0x000F000Fu, kMagic)), k1024);
    c1 = __hfma2(u32_as_h2(lop3_and_or(w0, 0x00F000F0u, kMagic)), k16th, km64);
    c2 = __hsub2(u32_as_h2(lop3_and_or(hi, 0x000F000Fu, kMagic)), k1024);
    c3 = __hfma2(u32_as_h2(lop3_and_or(hi, 0x00F000F0u, kMagic)), k16th, km64);
  } else {
    // 2-bit: the word holds eight pairs; an odd MMA index uses pairs 4..7 (bits 8.. / 24..)
    const uint32_t v = odd ? (w0 >> 8) : w0;
    c0 = __hsub2(u32_as_h2(lop3_and_or(v, 0x00030003u, kMagic)), __float2half2_rn(1024.f));
    c1 = __hfma2(u32_as_h2(lop3_and_or(v, 0x000C000Cu, kMagic)), __float2half2_rn(0.25f), __float2half2_rn(-256.f));
    c2 = __hfma2(u32_as_h2(lop3_and_or(v, 0x00300030u, kMagic)), __float2half2_rn(0.0625f), __float2half2_rn(-64.f));
    c3 = __hfma2(u32_as_h2(lop3_and_or(v, 0x00C000C0u, kMagic)), __float2half2_rn(0.015625f), __float2half2_rn(-16.f));
  }
  a[0] = h2_as_u32(__hfma2(c0, scA, zrA));
  a[1] = h2_as_u32(__hfma2(c1, scA, zrA));
  a[2] = h2_as_u32(__hfma2(c2, scB, zrB));
  a[3] = h2_as_u32(__hfma2(c3, scB, zrB));
}

// Fetch the code word(s) of MMA index s from a lane's preloaded chunk(s) of a tile.
template <int BITS>
struct TileCodes {
  // 8-bit: 16 words (4 chunks); 4-bit: 8 words (2 chunks); 2-bit: 4 words (1 chunk)
  static constexpr int kChunks = BITS / 2;
  uint4 ch[kChunks];
  __device__ __forceinline__ void load(const uint8_t* tile_codes, int lane) {
#pragma unroll
    for (int j = 0; j < kChunks; ++j) ch[j] = *reinterpret_cast<const uint4*>(tile_codes + (j * 32 + lane) * 16);
  }
  __device__ __forceinline__ uint32_t word(int w) const {
    const uint4& c = ch[w >> 2];
    switch (w & 3) {
      case 0: return c.x;
      case 1: return c.y;
      case 2: return c.z;
      default: return c.w;
    }
  }
};

struct SoftmaxState {
  float m0, m1;        // running max (log2 domain) of heads 2*c4, 2*c4+1
  float l0, l1;        // lane-partial sums of exp2 (reduced over the r lanes at the end)
  float o[8][4];       // O^T accumulators: tile u rows (16u + r, 16u + 8 + r) x heads (2c4, 2c4+1)
};

// Online-softmax update for NT token tiles.  On entry S holds raw dot products; bias is additive
// in the log2 domain (0, -inf for masked tokens, log2(count) for centroid rows).  On exit S holds
// the probabilities relative to the new running max.
template <int NT>
__device__ __forceinline__ void softmax_update(float (&S)[NT][4], const float (&bias)[NT][2], float scale_log2,
                                               SoftmaxState& st) {
  float mx0 = kNegInf, mx1 = kNegInf;
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    S[t][0] = fmaf(S[t][0], scale_log2, bias[t][0]);
    S[t][1] = fmaf(S[t][1], scale_log2, bias[t][0]);
    S[t][2] = fmaf(S[t][2], scale_log2, bias[t][1]);
    S[t][3] = fmaf(S[t][3], scale_log2, bias[t][1]);
    mx0 = fmaxf(mx0, fmaxf(S[t][0], S[t][2]));
    mx1 = fmaxf(mx1, fmaxf(S[t][1], S[t][3]));
  }
#pragma unroll
  for (int d = 4; d <= 16; d <<= 1) {
    mx0 = fmaxf(mx0, __shfl_xor_sync(kFull, mx0, d));
    mx1 = fmaxf(mx1, __shfl_xor_sync(kFull, mx1, d));
  }
  const float mn0 = fmaxf(st.m0, mx0), mn1 = fmaxf(st.m1, mx1);
  const float ms0 = (mn0 == kNegInf) ? 0.f : mn0, ms1 = (mn1 == kNegInf) ? 0.f : mn1;
  const float al0 = exp2f(st.m0 - ms0), al1 = exp2f(st.m1 - ms1);
  st.m0 = mn0;
  st.m1 = mn1;
  st.l0 *= al0;
  st.l1 *= al1;
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    st.o[u][0] *= al0;
    st.o[u][1] *= al1;
    st.o[u][2] *= al0;
    st.o[u][3] *= al1;
  }
#pragma unroll
  for (int t = 0; t < NT; ++t) {
    S[t][0] = exp2f(S[t][0] - ms0);
    S[t][1] = exp2f(S[t][1] - ms1);
    S[t][2] = exp2f(S[t][2] - ms0);
    S[t][3] = exp2f(S[t][3] - ms1);
  }
}

// P^T B-fragments in fp16 for one tile; accumulates the rounded probabilities into l.
__device__ __forceinline__ void make_p_f16(const float (&S)[4], uint32_t (&pf)[2], SoftmaxState& st) {
  const __half2 h01 = __floats2half2_rn(S[0], S[1]);
  const __half2 h23 = __floats2half2_rn(S[2], S[3]);
  st.l0 += __low2float(h01) + __low2float(h23);
  st.l1 += __high2float(h01) + __high2float(h23);
  pf[0] = movmatrix_trans(h2_as_u32(h01));
  pf[1] = movmatrix_trans(h2_as_u32(h23));
}
// P^T B-fragments as bf16 hi + lo parts (p = hi + lo to ~2^-17).
__device__ __forceinline__ void make_p_bf16(const float (&S)[4], uint32_t (&pf)[4], SoftmaxState& st) {
  const uint32_t hi01 = pack_bf16x2(S[0], S[1]), hi23 = pack_bf16x2(S[2], S[3]);
  const uint32_t lo01 = pack_bf16x2(S[0] - bf16lo_to_f32(hi01), S[1] - bf16hi_to_f32(hi01));
  const uint32_t lo23 = pack_bf16x2(S[2] - bf16lo_to_f32(hi23), S[3] - bf16hi_to_f32(hi23));
  st.l0 += S[0] + S[2];
  st.l1 += S[1] + S[3];
  pf[0] = movmatrix_trans(hi01);
  pf[1] = movmatrix_trans(hi23);
  pf[2] = movmatrix_trans(lo01);
  pf[3] = movmatrix_trans(lo23);
}

// ---- item cursor ---------------------------------------------------------------------------
enum StepKind : int { kRowsK = 0, kRowsV = 1, kQ8K = 2, kQ8V = 3, kQ4 = 4, kQ2 = 5 };
enum RowSrc : int { kSrcBlock = 0, kSrcCentroid = 1, kSrcResidual = 2 };

struct Cursor {
  int item;          // full mode: item index; sparse mode: position in the warp's page range
  int sub;           // step inside the item
  int nsub;          // steps of the item
  int adv;           // items consumed when the item is done (centroid runs consume several)
  int level;         // 16 / 8 / 4 / 2 / 1, or 17 for a residual group
  int ntok;          // valid rows (row sources) or 64
  int tmask;         // 4-bit mask of active 16-token tiles
  uint32_t off256;
  uint64_t resmask;
};

struct WarpCtx {
  const DecodeParams* p;
  const TableEntry* table;   // this stream's table
  int lane;
  int item_end;              // full mode: one past the last item; sparse: one past the last page position
  int stream;
  bool sparse, has_tail;
  int page_lo;               // sparse: first page position
  uint32_t stage[kStages];   // shared-memory addresses of the stages
  const uint8_t* stage_ptr[kStages];
};

__device__ __forceinline__ int popc4(int m) { return __popc(m & 15); }

// Set up cursor fields for item index `it` (full mode).  Returns false when past the end.
__device__ __forceinline__ bool load_item_full(const WarpCtx& w, int it, Cursor& c) {
  const DecodeParams& p = *w.p;
  while (true) {
    if (it >= w.item_end) return false;
    c.item = it;
    c.sub = 0;
    c.adv = 1;
    if (it <= p.n_closed) {
      const TableEntry e = w.table[it];
      c.off256 = e.off256;
      c.resmask = e.resmask;
      c.level = static_cast<int>(e.level);
      c.tmask = 15;
      c.ntok = kBlock;
      if (it == p.n_closed) {           // tail block: exact rows, n_tail of them
        c.level = 16;
        c.ntok = p.n_tail;
        const int nt = (p.n_tail + 15) >> 4;
        c.tmask = (1 << nt) - 1;
        if (nt == 0) { ++it; continue; }
      }
      switch (c.level) {
        case 16: c.nsub = 2 * popc4(c.tmask); break;
        case 8: c.nsub = 4; break;
        case 4: c.nsub = 2; break;
        case 2: c.nsub = 1; break;
        default: {   // centroid run: up to 16 consecutive centroid blocks inside this warp's range
          int run = 1;
          const int lim = min(min(w.item_end, p.n_closed) - it, 16);
          while (run < lim && w.table[it + run].level == 1u) ++run;
          c.adv = run;
          c.ntok = run;
          c.nsub = 2;
          c.level = 1;
        }
      }
      return true;
    }
    // residual group j: rows [16 j, 16 j + 16) of the stream's residual pool
    const int j = it - p.n_closed - 1;
    const int n_res = p.res_count ? p.res_count[w.stream] : 0;
    const int rows = min(16, n_res - 16 * j);
    if (rows <= 0) return false;
    c.level = 17;
    c.ntok = rows;
    c.nsub = 2;
    c.tmask = 1;
    c.off256 = p.res_off256[w.stream] + 2u * 16u * static_cast<uint32_t>(j);   // 512 B per row = 2 units
    c.resmask = 0;
    return true;
  }
}

// Sparse mode: position `pos` in the warp's slice of the ascending page list; pages that fall in
// the same block are merged into one visit.  Position item_end stands for the tail block.
__device__ __forceinline__ bool load_item_sparse(const WarpCtx& w, int pos, Cursor& c) {
  const DecodeParams& p = *w.p;
  const int tiles_per_page = p.page_tokens >> 4;
  const int pages_per_block = kBlock / p.page_tokens;
  if (pos < w.item_end) {
    const int32_t* list = p.page_idx + static_cast<size_t>(w.stream) * p.n_sel;
    const int page = list[pos];
    const int blk = page / pages_per_block;
    int mask = ((1 << tiles_per_page) - 1) << (tiles_per_page * (page % pages_per_block));
    int adv = 1;
    while (pos + adv < w.item_end) {
      const int pg = list[pos + adv];
      if (pg / pages_per_block != blk) break;
      mask |= ((1 << tiles_per_page) - 1) << (tiles_per_page * (pg % pages_per_block));
      ++adv;
    }
    const TableEntry e = w.table[blk];
    c.item = pos;
    c.sub = 0;
    c.adv = adv;
    c.off256 = e.off256;
    c.resmask = 0;
    c.level = static_cast<int>(e.level);
    c.tmask = mask;
    c.ntok = kBlock;
    switch (c.level) {
      case 16: c.nsub = 2 * popc4(mask); break;
      case 8: c.nsub = 2 * (((mask & 3) != 0) + ((mask & 12) != 0)); break;
      case 4: c.nsub = ((mask & 3) != 0) + ((mask & 12) != 0); break;
      case 2: c.nsub = 1; break;
      default: c.nsub = 2; c.ntok = 1; break;     // a single centroid row weighted by the selected tokens
    }
    return true;
  }
  if (pos == w.item_end && w.has_tail && p.n_tail > 0) {
    const TableEntry e = w.table[p.n_closed];
    c.item = pos;
    c.sub = 0;
    c.adv = 1;
    c.off256 = e.off256;
    c.resmask = 0;
    c.level = 16;
    c.ntok = p.n_tail;
    const int nt = (p.n_tail + 15) >> 4;
    c.tmask = (1 << nt) - 1;
    c.nsub = 2 * nt;
    return true;
  }
  return false;
}

__device__ __forceinline__ bool load_item(const WarpCtx& w, int it, Cursor& c) {
  return w.sparse ? load_item_sparse(w, it, c) : load_item_full(w, it, c);
}
__device__ __forceinline__ bool advance(const WarpCtx& w, Cursor& c) {
  if (++c.sub < c.nsub) return true;
  return load_item(w, c.item + c.adv, c);
}

// k-th set bit (0-based) of a 4-bit mask
__device__ __forceinline__ int nth_set_bit(int mask, int k) {
  int idx = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (mask & (1 << i)) {
      if (k == 0) idx = i;
      --k;
    }
  }
  return idx;
}
// For quantised levels in sparse mode: which half does step `sub` address (levels 8 and 4)?
__device__ __forceinline__ int half_of_step(const Cursor& c, int idx) {
  // idx-th active half
  const bool h0 = (c.tmask & 3) != 0;
  return (idx == 0) ? (h0 ? 0 : 1) : 1;
}

// Contiguous copy of `bytes` (multiple of 512) from global to a stage offset.
__device__ __forceinline__ void copy_span(uint32_t sdst, const uint8_t* gsrc, int bytes, int lane) {
  for (int o = lane * 16; o < bytes; o += 512) cp_async16(sdst + o, gsrc + o, 16);
}

// Issue the loads of the cursor's current step into stage `sidx`.
__device__ __forceinline__ void issue_step(const WarpCtx& w, const Cursor& c, int sidx) {
  const DecodeParams& p = *w.p;
  const uint32_t sdst = w.stage[sidx];
  const int lane = w.lane;
  if (c.level == 16 || c.level == 1 || c.level == 17) {
    // 16 rows of 256 B, row r chunk q stored at r*256 + ((q ^ (r & 7)) << 4)
    const bool is_v = (c.sub & 1) != 0;
    const uint8_t* base;
    size_t row_stride;
    int row0 = 0, nrows;
    if (c.level == 16) {
      const int tile = nth_set_bit(c.tmask, c.sub >> 1);
      base = p.arena + static_cast<size_t>(c.off256) * 256 + (is_v ? kBlock * kRowBytes : 0);
      row_stride = kRowBytes;
      row0 = tile * 16;
      nrows = min(16, c.ntok - row0);
    } else if (c.level == 17) {
      base = p.arena + static_cast<size_t>(c.off256) * 256 + (is_v ? kRowBytes : 0);
      row_stride = 2 * kRowBytes;
      nrows = c.ntok;
    } else {
      base = nullptr;   // centroid rows live in separate slots
      row_stride = 0;
      nrows = c.ntok;
    }
    // per-row source pointer for centroid runs: lane r < nrows looks up block (item + r)
    const uint8_t* myrow = p.arena;
    if (c.level == 1) {
      if (lane < nrows) {
        const int blk = w.sparse ? (p.page_idx[static_cast<size_t>(w.stream) * p.n_sel + c.item] /
                                    (kBlock / p.page_tokens))
                                 : (c.item + lane);
        myrow = p.arena + static_cast<size_t>(w.table[blk].off256) * 256 + (is_v ? kRowBytes : 0);
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int row = 2 * j + (lane >> 4), q = lane & 15;
      const uint8_t* src;
      if (c.level == 1) {
        const unsigned long long ptr = __shfl_sync(kFull, reinterpret_cast<unsigned long long>(myrow), row);
        src = reinterpret_cast<const uint8_t*>(ptr);
      } else {
        src = base + static_cast<size_t>(row0 + row) * row_stride;
      }
      const bool valid = row < nrows;
      cp_async16(sdst + row * 256 + ((q ^ (row & 7)) << 4), valid ? (src + q * 16) : p.arena, valid ? 16 : 0);
    }
    return;
  }
  const int bits = c.level;
  const int cb = code_bytes_per_tile(bits);
  const uint8_t* slot = p.arena + static_cast<size_t>(c.off256) * 256;
  if (c.tmask == 15) {
    // full block: every step is one contiguous span of the slot
    if (bits == 8) {
      const int half = c.sub >> 1;
      const uint8_t* hb = slot + half * half_bytes(8);
      if ((c.sub & 1) == 0) copy_span(sdst, hb, 512 + 2 * cb, lane);
      else copy_span(sdst, hb + 512 + 2 * cb, 512 + 2 * cb, lane);
    } else if (bits == 4) {
      copy_span(sdst, slot + c.sub * half_bytes(4), half_bytes(4), lane);
    } else {
      copy_span(sdst, slot, 2 * half_bytes(2), lane);
    }
    return;
  }
  // sparse visit: copy only the pieces of the selected tiles (same stage offsets as a full copy)
  if (bits == 8) {
    const int half = half_of_step(c, c.sub >> 1);
    const int tm = (c.tmask >> (2 * half)) & 3;
    const uint8_t* hb = slot + half * half_bytes(8);
    if ((c.sub & 1) == 0) {
      copy_span(sdst, hb, 512, lane);
      for (int t = 0; t < 2; ++t)
        if (tm & (1 << t)) copy_span(sdst + 512 + t * cb, hb + off_kc(8, t), cb, lane);
    } else {
      const int vbase = 512 + 2 * cb;
      for (int t = 0; t < 2; ++t)
        if (tm & (1 << t)) {
          if (lane < 16) cp_async16(sdst + t * 256 + lane * 16, hb + off_vp(8, t) + lane * 16, 16);
          copy_span(sdst + 512 + t * cb, hb + off_vc(8, t), cb, lane);
        }
      (void)vbase;
    }
  } else {
    const int nh = (bits == 4) ? 1 : 2;
    for (int hh = 0; hh < nh; ++hh) {
      const int half = (bits == 4) ? half_of_step(c, c.sub) : hh;
      const int tm = (c.tmask >> (2 * half)) & 3;
      if (tm == 0) continue;
      const uint8_t* hb = slot + half * half_bytes(bits);
      const uint32_t sd = sdst + ((bits == 4) ? 0 : hh * half_bytes(2));
      copy_span(sd, hb, 512, lane);
      for (int t = 0; t < 2; ++t)
        if (tm & (1 << t)) {
          copy_span(sd + off_kc(bits, t), hb + off_kc(bits, t), cb, lane);
          if (lane < 16) cp_async16(sd + off_vp(bits, t) + lane * 16, hb + off_vp(bits, t) + lane * 16, 16);
          copy_span(sd + off_vc(bits, t), hb + off_vc(bits, t), cb, lane);
        }
    }
  }
}

// ---- compute ---------------------------------------------------------------------------------
// QK^T of the active tiles of one half from staged key params + codes.
template <int BITS>
__device__ __forceinline__ void qk_half(const uint8_t* kp, const uint8_t* kc0, const uint8_t* kc1, int tm,
                                        const uint32_t (&qh)[16], int lane, float (&S)[2][4]) {
  const int c4 = lane & 3;
  TileCodes<BITS> t0, t1;
  if (tm & 1) t0.load(kc0, lane);
  if (tm & 2) t1.load(kc1, lane);
#pragma unroll
  for (int s = 0; s < 8; ++s) {
    const uint4 pr = *reinterpret_cast<const uint4*>(kp + (s * 4 + c4) * 16);
    const __half2 scA = u32_as_h2(pr.x), zrA = u32_as_h2(pr.y), scB = u32_as_h2(pr.z), zrB = u32_as_h2(pr.w);
    uint32_t a[4];
    if (tm & 1) {
      if constexpr (BITS == 8) unpack_dequant<8>(t0.word(2 * s), t0.word(2 * s + 1), false, scA, zrA, scB, zrB, a);
      else if constexpr (BITS == 4) unpack_dequant<4>(t0.word(s), 0u, false, scA, zrA, scB, zrB, a);
      else unpack_dequant<2>(t0.word(s >> 1), 0u, (s & 1) != 0, scA, zrA, scB, zrB, a);
      mma_f16(S[0], a, qh[2 * s], qh[2 * s + 1]);
    }
    if (tm & 2) {
      if constexpr (BITS == 8) unpack_dequant<8>(t1.word(2 * s), t1.word(2 * s + 1), false, scA, zrA, scB, zrB, a);
      else if constexpr (BITS == 4) unpack_dequant<4>(t1.word(s), 0u, false, scA, zrA, scB, zrB, a);
      else unpack_dequant<2>(t1.word(s >> 1), 0u, (s & 1) != 0, scA, zrA, scB, zrB, a);
      mma_f16(S[1], a, qh[2 * s], qh[2 * s + 1]);
    }
  }
}

// O^T += V^T P^T for the active tiles of one half from staged value params + codes.
template <int BITS>
__device__ __forceinline__ void pv_half(const uint8_t* vp0, const uint8_t* vp1, const uint8_t* vc0,
                                        const uint8_t* vc1, int tm, const uint32_t (&pf)[2][2], int lane,
                                        SoftmaxState& st) {
  const int c4 = lane & 3;
  TileCodes<BITS> t0, t1;
  if (tm & 1) t0.load(vc0, lane);
  if (tm & 2) t1.load(vc1, lane);
#pragma unroll
  for (int grp = 0; grp < 4; ++grp) {
    uint4 pr0 = make_uint4(0, 0, 0, 0), pr1 = make_uint4(0, 0, 0, 0);
    if (tm & 1) pr0 = *reinterpret_cast<const uint4*>(vp0 + (grp * 4 + c4) * 16);
    if (tm & 2) pr1 = *reinterpret_cast<const uint4*>(vp1 + (grp * 4 + c4) * 16);
#pragma unroll
    for (int uu = 0; uu < 2; ++uu) {
      const int u = 2 * grp + uu;
      uint32_t a[4];
      if (tm & 1) {
        const __half2 scA = u32_as_h2(pr0.x), zrA = u32_as_h2(pr0.y), scB = u32_as_h2(pr0.z), zrB = u32_as_h2(pr0.w);
        if constexpr (BITS == 8) unpack_dequant<8>(t0.word(2 * u), t0.word(2 * u + 1), false, scA, zrA, scB, zrB, a);
        else if constexpr (BITS == 4) unpack_dequant<4>(t0.word(u), 0u, false, scA, zrA, scB, zrB, a);
        else unpack_dequant<2>(t0.word(u >> 1), 0u, (u & 1) != 0, scA, zrA, scB, zrB, a);
        mma_f16(st.o[u], a, pf[0][0], pf[0][1]);
      }
      if (tm & 2) {
        const __half2 scA = u32_as_h2(pr1.x), zrA = u32_as_h2(pr1.y), scB = u32_as_h2(pr1.z), zrB = u32_as_h2(pr1.w);
        if constexpr (BITS == 8) unpack_dequant<8>(t1.word(2 * u), t1.word(2 * u + 1), false, scA, zrA, scB, zrB, a);
        else if constexpr (BITS == 4) unpack_dequant<4>(t1.word(u), 0u, false, scA, zrA, scB, zrB, a);
        else unpack_dequant<2>(t1.word(u >> 1), 0u, (u & 1) != 0, scA, zrA, scB, zrB, a);
        mma_f16(st.o[u], a, pf[1][0], pf[1][1]);
      }
    }
  }
}

// Token validity bias of a half for the lane's rows: tokens 32*half + 16*t + r (+8).
__device__ __forceinline__ void half_bias(uint64_t resmask, int half, int tm, int lane, float (&bias)[2][2]) {
  const int r = lane >> 2;
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int tok = 32 * half + 16 * t + r;
    const bool on = (tm >> t) & 1;
    bias[t][0] = (on && !((resmask >> tok) & 1ull)) ? 0.f : kNegInf;
    bias[t][1] = (on && !((resmask >> (tok + 8)) & 1ull)) ? 0.f : kNegInf;
  }
}

template <int BITS>
__device__ __forceinline__ void qk_softmax_half(const uint8_t* half_k, int half, int tm, uint64_t resmask,
                                                const uint32_t (&qh)[16], int lane, float scale_log2,
                                                SoftmaxState& st, uint32_t (&pf)[2][2]) {
  constexpr int cb = 256 * BITS;
  float S[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
  qk_half<BITS>(half_k, half_k + 512, half_k + 512 + cb, tm, qh, lane, S);
  float bias[2][2];
  half_bias(resmask, half, tm, lane, bias);
  softmax_update<2>(S, bias, scale_log2, st);
  make_p_f16(S[0], pf[0], st);
  make_p_f16(S[1], pf[1], st);
}

// Process a staged step.  pf carries P fragments from a key step to the following value step.
__device__ __forceinline__ void compute_step(const WarpCtx& w, const Cursor& c, int sidx, const uint32_t (&qb)[16],
                                             const uint32_t (&qh)[16], SoftmaxState& st, uint32_t (&pf)[4]) {
  const DecodeParams& p = *w.p;
  const int lane = w.lane;
  const uint8_t* sp = w.stage_ptr[sidx];
  const uint32_t sa = w.stage[sidx];
  if (c.level == 16 || c.level == 1 || c.level == 17) {
    if ((c.sub & 1) == 0) {
      // key rows: S^T = K Q^T
      float S[1][4] = {{0.f, 0.f, 0.f, 0.f}};
      const int mi = lane >> 3;
      const int row = (lane & 7) + (mi & 1) * 8;
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        uint32_t a[4];
        const int q = 2 * s + (mi >> 1);
        ldmatrix_x4(a, sa + row * 256 + ((q ^ (row & 7)) << 4));
        mma_bf16(S[0], a, qb[2 * s], qb[2 * s + 1]);
      }
      // validity / weight of the lane's rows r and r + 8
      const int r = lane >> 2;
      float bias[1][2];
      if (c.level == 16) {
        const int tile = nth_set_bit(c.tmask, c.sub >> 1);
        const int t0 = tile * 16 + r;
        bias[0][0] = (t0 < c.ntok && !((c.resmask >> t0) & 1ull)) ? 0.f : kNegInf;
        bias[0][1] = (t0 + 8 < c.ntok && !((c.resmask >> (t0 + 8)) & 1ull)) ? 0.f : kNegInf;
      } else if (c.level == 17) {
        bias[0][0] = (r < c.ntok) ? 0.f : kNegInf;
        bias[0][1] = (r + 8 < c.ntok) ? 0.f : kNegInf;
      } else {
        // centroid rows: each stands for the block's readable tokens -> add log2(count)
        float myb = kNegInf;
        if (lane < c.ntok) {
          int cnt;
          if (w.sparse) cnt = 16 * popc4(c.tmask);
          else cnt = kBlock - __popcll(w.table[c.item + lane].resmask);
          myb = cnt > 0 ? log2f(static_cast<float>(cnt)) : kNegInf;
        }
        bias[0][0] = __shfl_sync(kFull, myb, r);
        bias[0][1] = __shfl_sync(kFull, myb, r + 8);
      }
      softmax_update<1>(S, bias, p.scale_log2, st);
      make_p_bf16(S[0], pf, st);
    } else {
      // value rows: O^T += V^T P^T with P = hi + lo
      const int mi = lane >> 3;
      const int row = (lane & 7) + (mi >> 1) * 8;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        uint32_t a[4];
        const int q = 2 * u + (mi & 1);
        ldmatrix_x4_trans(a, sa + row * 256 + ((q ^ (row & 7)) << 4));
        mma_bf16(st.o[u], a, pf[0], pf[1]);
        mma_bf16(st.o[u], a, pf[2], pf[3]);
      }
    }
    return;
  }
  uint32_t (&pf2)[2][2] = *reinterpret_cast<uint32_t (*)[2][2]>(&pf);
  if (c.level == 8) {
    const int half = (c.tmask == 15) ? (c.sub >> 1) : half_of_step(c, c.sub >> 1);
    const int tm = (c.tmask >> (2 * half)) & 3;
    if ((c.sub & 1) == 0) {
      qk_softmax_half<8>(sp, half, tm, c.resmask, qh, lane, p.scale_log2, st, pf2);
    } else {
      pv_half<8>(sp, sp + 256, sp + 512, sp + 512 + 2048, tm, pf2, lane, st);
    }
  } else if (c.level == 4) {
    const int half = (c.tmask == 15) ? c.sub : half_of_step(c, c.sub);
    const int tm = (c.tmask >> (2 * half)) & 3;
    qk_softmax_half<4>(sp, half, tm, c.resmask, qh, lane, p.scale_log2, st, pf2);
    pv_half<4>(sp + off_vp(4, 0), sp + off_vp(4, 1), sp + off_vc(4, 0), sp + off_vc(4, 1), tm, pf2, lane, st);
  } else {
#pragma unroll 1
    for (int half = 0; half < 2; ++half) {
      const int tm = (c.tmask >> (2 * half)) & 3;
      if (tm == 0) continue;
      const uint8_t* hb = sp + half * half_bytes(2);
      qk_softmax_half<2>(hb, half, tm, c.resmask, qh, lane, p.scale_log2, st, pf2);
      pv_half<2>(hb + off_vp(2, 0), hb + off_vp(2, 1), hb + off_vc(2, 0), hb + off_vc(2, 1), tm, pf2, lane, st);
    }
  }
}

__global__ void __launch_bounds__(kDecodeWarps * 32, 2) decode_kernel(const __grid_constant__ DecodeParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gw = blockIdx.x * kDecodeWarps + warp;
  if (gw >= p.n_warps) return;

  WarpCtx w;
  w.p = &p;
  w.lane = lane;
  w.sparse = p.page_idx != nullptr;
  int partial_row, first;
  if (!w.sparse) {
    const WarpDesc wd = p.warps[gw];
    if (wd.stream < 0) return;
    w.stream = wd.stream;
    w.item_end = wd.item_end;
    w.has_tail = false;
    first = wd.item_begin;
    partial_row = wd.partial;
  } else {
    const int wps = p.warps_per_stream;
    w.stream = gw / wps;
    const int wi = gw - w.stream * wps;
    first = static_cast<int>((static_cast<long long>(wi) * p.n_sel) / wps);
    w.item_end = static_cast<int>((static_cast<long long>(wi + 1) * p.n_sel) / wps);
    w.has_tail = (wi == wps - 1);
    partial_row = gw;
  }
  w.table = p.table + static_cast<size_t>(w.stream) * p.table_stride;
  uint8_t* sbase = smem + warp * (kStages * kStageBytes);
#pragma unroll
  for (int s = 0; s < kStages; ++s) {
    w.stage_ptr[s] = sbase + s * kStageBytes;
    w.stage[s] = smem_u32(sbase + s * kStageBytes);
  }

  // Query fragments: B operand Q^T[16 channels x 8 heads]; lane (r, c4) holds head r, channels
  // 16 s + 2 c4 (+1) and 16 s + 8 + 2 c4 (+1), in bf16 (exact rows) and fp16 (quantised tiers).
  const int r = lane >> 2, c4 = lane & 3;
  uint32_t qb[16], qh[16];
  {
    const int b = w.stream / p.n_kv_heads, kvh = w.stream - b * p.n_kv_heads;
    const int n_q_heads = p.n_kv_heads * p.group;
    const uint16_t* qrow = p.q + (static_cast<size_t>(b) * n_q_heads + static_cast<size_t>(kvh) * p.group + r) * kD;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      uint32_t v0 = 0, v1 = 0;
      if (r < p.group) {
        v0 = *reinterpret_cast<const uint32_t*>(qrow + 16 * s + 2 * c4);
        v1 = *reinterpret_cast<const uint32_t*>(qrow + 16 * s + 8 + 2 * c4);
      }
      qb[2 * s] = v0;
      qb[2 * s + 1] = v1;
      qh[2 * s] = h2_as_u32(__floats2half2_rn(bf16lo_to_f32(v0), bf16hi_to_f32(v0)));
      qh[2 * s + 1] = h2_as_u32(__floats2half2_rn(bf16lo_to_f32(v1), bf16hi_to_f32(v1)));
    }
  }

  SoftmaxState st;
  st.m0 = st.m1 = kNegInf;
  st.l0 = st.l1 = 0.f;
#pragma unroll
  for (int u = 0; u < 8; ++u) st.o[u][0] = st.o[u][1] = st.o[u][2] = st.o[u][3] = 0.f;
  uint32_t pf[4] = {0, 0, 0, 0};

  Cursor cur;
  bool have = load_item(w, first, cur);
  int sidx = 0;
  if (have) {
    issue_step(w, cur, 0);
    cp_async_commit();
  }
  while (have) {
    Cursor nxt = cur;
    const bool more = advance(w, nxt);
    if (more) issue_step(w, nxt, sidx ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncwarp();
    compute_step(w, cur, sidx, qb, qh, st, pf);
    __syncwarp();
    cur = nxt;
    have = more;
    sidx ^= 1;
  }
  cp_async_wait<0>();

  // lane-partial sums -> per-head sums (reduce over the 8 r lanes that share c4)
#pragma unroll
  for (int d = 4; d <= 16; d <<= 1) {
    st.l0 += __shfl_xor_sync(kFull, st.l0, d);
    st.l1 += __shfl_xor_sync(kFull, st.l1, d);
  }
  float* out = p.partial + static_cast<size_t>(partial_row) * kPartialFloats;
  const int h0 = 2 * c4, h1 = 2 * c4 + 1;
  if (r == 0) {
    if (h0 < p.group) { out[h0 * (kD + 2)] = st.m0; out[h0 * (kD + 2) + 1] = st.l0; }
    if (h1 < p.group) { out[h1 * (kD + 2)] = st.m1; out[h1 * (kD + 2) + 1] = st.l1; }
  }
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const int ch = 16 * u + r;
    if (h0 < p.group) {
      out[h0 * (kD + 2) + 2 + ch] = st.o[u][0];
      out[h0 * (kD + 2) + 2 + ch + 8] = st.o[u][2];
    }
    if (h1 < p.group) {
      out[h1 * (kD + 2) + 2 + ch] = st.o[u][1];
      out[h1 * (kD + 2) + 2 + ch + 8] = st.o[u][3];
    }
  }
}

// Merge the partials of one (stream, query head): fixed ascending order, so results are
// reproducible run to run.
__global__ void __launch_bounds__(kD) combine_kernel(const __grid_constant__ CombineParams p) {
  const int stream = blockIdx.x, h = blockIdx.y, c = threadIdx.x;
  int begin, end;
  if (p.parts) {
    begin = p.parts[stream].begin;
    end = p.parts[stream].end;
  } else {
    begin = stream * p.warps_per_stream;
    end = begin + p.warps_per_stream;
  }
  float M = kNegInf;
  for (int i = begin; i < end; ++i) M = fmaxf(M, p.partial[static_cast<size_t>(i) * kPartialFloats + h * (kD + 2)]);
  float L = 0.f, acc = 0.f;
  for (int i = begin; i < end; ++i) {
    const float* row = p.partial + static_cast<size_t>(i) * kPartialFloats + h * (kD + 2);
    const float m = row[0];
    if (m == kNegInf) continue;
    const float wgt = exp2f(m - M);
    L = fmaf(wgt, row[1], L);
    acc = fmaf(wgt, row[2 + c], acc);
  }
  const int b = stream / p.n_kv_heads, kvh = stream - b * p.n_kv_heads;
  const size_t hq = static_cast<size_t>(b) * p.n_kv_heads * p.group + static_cast<size_t>(kvh) * p.group + h;
  p.out[hq * kD + c] = (L > 0.f) ? acc / L : 0.f;
  if (p.lse && c == 0) p.lse[hq] = (L > 0.f) ? (M + log2f(L)) * 0.6931471805599453f : kNegInf;
}

}  // namespace

size_t decode_smem_bytes() { return static_cast<size_t>(kDecodeWarps) * kStages * kStageBytes; }

cudaError_t launch_decode(const DecodeParams& p, int n_ctas, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(decode_smem_bytes()));
    if (e != cudaSuccess) return e;
    configured = true;
  }
  if (n_ctas <= 0) return cudaSuccess;
  decode_kernel<<<n_ctas, kDecodeWarps * 32, decode_smem_bytes(), st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_combine(const CombineParams& p, int n_streams, cudaStream_t st) {
  combine_kernel<<<dim3(n_streams, p.group), kD, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace gkv
