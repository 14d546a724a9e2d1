// Graded single-query decode attention (paper Sec. 3.7: dequantisation inside the online-softmax
// loop, all KV heads of a layer in one launch, split-context partials merged in the same launch).
//
// Work split: the host cuts every stream into units (a block, half of a quantised block, a run of
// centroid blocks, the tail, a group of exact residual rows) and deals them longest-first to the
// stream's warps; a warp walks its unit list and keeps its own online-softmax state for the g <= 8
// query heads of the KV head (one read of the KV bytes serves the whole GQA group, Sec. 3.1).
// Warps never wait on each other: each one runs a private double-buffered pipeline of TMA bulk
// copies (cp.async.bulk global -> shared, completion on a per-warp mbarrier) and consumes only what
// it staged; every mbarrier wait is bounded.
//
// Math: S^T[tokens x heads] = K[tokens x ch] Q^T and O^T[ch x heads] += V^T[ch x tokens] P^T on
// mma.m16n8k16 with the query heads as the n = 8 dimension.  Quantised codes are stored in
// A-fragment order (gkv_layout.cuh) and become A operands by masking: a code in the mantissa of an
// fp16 with a zero exponent field is the number code * 2^(p - 24), bias-free.  Scales are folded into the
// B operands (q' = q * s_k per 32-token key group, P' = p * s_v per 32-channel value group); zero
// points are handled by extra MMAs (A = zero-point pattern) instead of per-value arithmetic, the
// powers of two of the code fields in fp32 after the key MMAs and in P' before the value MMAs.
//
// Precision: every B operand that carries a rounded product or probability is a pair hi + lo of
// fp16 (bf16 for exact rows) numbers, hi = rn(x), lo = rn(x - hi), so that the operand is good to
// ~2^-22 and the fp32 accumulators decide the error.  A warp serves at most four query heads: the
// n = 8 dimension holds (hi, lo) column pairs, column 2 j the hi part and column 2 j + 1 the lo part of
// head j, so one MMA does both and a lane finds the two halves of its head side by side in its
// accumulator registers.  A KV head with 5..8 query heads is read as two such head groups.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstdio>

#include "gkv_internal.h"

namespace gkv {
namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr float kNegInf = -__builtin_huge_valf();
constexpr int kRowPitch = kRowBytes + 16;       // staged exact rows: 272 B pitch -> conflict-free ldmatrix
constexpr int kWaitSpins = 1 << 20;             // bound of every mbarrier wait (each poll may sleep up to the hint)
constexpr uint32_t kWaitHintNs = 2000;          // suspend-time hint of one mbarrier poll, nanoseconds

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
// 16-byte asynchronous copy; src_bytes = 0 writes zeros instead
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// the mbarrier gets one more pending arrival now, delivered when this thread's copies above are done
__device__ __forceinline__ void cp_async_mbar_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.shared::cta.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(kWaitHintNs)
      : "memory");
  return ok != 0;
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
  asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
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

// ---- code unpack: the four A registers of MMA index s as bias-free fp16 numbers --------------------
// A code that sits at mantissa bit p of an fp16 whose exponent field is zero is the number
// code * 2^(p - 24): masking the packed word is a complete conversion, there is no bias to cancel in the
// accumulators afterwards and no precision is lost to one.  The fields of a word are read where they are
// (one shift per word brings the second pair of fields down), so p differs between the fields:
//   keys    (field = A register a: rows r / r + 8 of the MMA for a & 1 = 0 / 1): the two row classes of an
//           MMA come out with the weights 2^-24 and 2^(p1 - 24) (KScale), evened out in fp32 after it;
//   values  (fields ordered by token half, gkv_layout.cuh): registers 0, 1 (tokens 0-7 of the tile) at
//           p = 0, registers 2, 3 (tokens 8-15) at p1; P' is multiplied by 2^(4 - p) (VScale), so that
//           every product carries the common factor 2^-20, which the exact rows put into P and the final
//           row takes out again.
template <int BITS>
struct KScale;                     // 2^(24 - p) of the rows r (lo) and r + 8 (hi)
template <>
struct KScale<8> {
  static constexpr float lo = 16777216.f, hi = 16777216.f;
};
template <>
struct KScale<4> {
  static constexpr float lo = 16777216.f, hi = 1048576.f;
};
template <>
struct KScale<2> {
  static constexpr float lo = 16777216.f, hi = 4194304.f;
};
template <int BITS>
struct VScale;                     // 2^(4 - p) of the tokens 0-7 (lo) and 8-15 (hi) of a tile
template <>
struct VScale<8> {
  static constexpr float lo = 16.f, hi = 16.f;
};
template <>
struct VScale<4> {
  static constexpr float lo = 16.f, hi = 1.f;
};
template <>
struct VScale<2> {
  static constexpr float lo = 16.f, hi = 4.f;
};
constexpr float kVUnit = 1.f / 1048576.f;         // 2^-20: weight of a value product in the accumulators
constexpr float kVUnitInv = 1048576.f;

// Words of one lane for MMA indices [s0, s0 + NS): 8-bit 2 words per s, 4-bit 1, 2-bit 1 per 2.
// Keys: field f of a word belongs to register f.  Values: fields 0, 1 / 2, 3 belong to registers 0, 2 / 1, 3.
template <int BITS, bool IS_V>
__device__ __forceinline__ void unpack(const uint32_t* w, int s_local, uint32_t (&a)[4]) {
  constexpr int i1 = IS_V ? 2 : 1, i2 = IS_V ? 1 : 2;      // registers of fields 1 and 2
  if constexpr (BITS == 8) {
    const uint32_t w0 = w[2 * s_local], w1 = w[2 * s_local + 1];
    a[0] = prmt(w0, 0u, 0x4240u);
    a[1] = prmt(w0, 0u, 0x4341u);
    a[2] = prmt(w1, 0u, 0x4240u);
    a[3] = prmt(w1, 0u, 0x4341u);
  } else if constexpr (BITS == 4) {
    // fields at bits 0, 4, 8, 12 of each 16-bit half
    const uint32_t v0 = w[s_local], v1 = v0 >> 8;
    a[0] = v0 & 0x000F000Fu;
    a[i1] = v0 & 0x00F000F0u;
    a[i2] = v1 & 0x000F000Fu;
    a[3] = v1 & 0x00F000F0u;
  } else {
    // even s: fields at bits 0, 2, 8, 10; odd s: 4 further
    const uint32_t x = w[s_local >> 1];
    const uint32_t v0 = (s_local & 1) ? (x >> 4) : x, v1 = (s_local & 1) ? (x >> 12) : (x >> 8);
    a[0] = v0 & 0x00030003u;
    a[i1] = v0 & 0x000C000Cu;
    a[i2] = v1 & 0x00030003u;
    a[3] = v1 & 0x000C000Cu;
  }
}

__device__ __forceinline__ float fast_exp2(float x);

// Lane (r, c4) = (lane / 4, lane % 4).  Accumulator side: the lane owns head c4 of the warp's head
// group: columns 2 c4 (hi) and 2 c4 + 1 (lo), rows r and r + 8.  B-fragment side: the lane holds column
// r, i.e. the hi (r even) or lo (r odd) part of head r / 2.
struct SoftmaxState {
  float m;             // running max (log2 domain) of head c4
  float l;             // lane-partial sum of exp2 (reduced over the r lanes at the end)
  float o[8][4];       // O^T accumulators: tile u rows (16u + r, 16u + 8 + r) x (hi, lo) columns of head c4
  float zc;            // value zero-point term: row = 32-channel group (lanes r < 4), head c4
};
__device__ __forceinline__ bool lo_part_lane(int lane) { return (lane & 4) != 0; }

// Online-softmax update for N logits of the lane's head (log2 domain, bias already added: 0, -inf
// for masked tokens, log2(count) for centroid rows).  On exit x holds the probabilities relative to the
// new running max.
template <int N>
__device__ __forceinline__ void softmax_update(float (&x)[N], SoftmaxState& st) {
  float mx = x[0];
#pragma unroll
  for (int i = 1; i < N; ++i) mx = fmaxf(mx, x[i]);
#pragma unroll
  for (int d = 4; d <= 16; d <<= 1) mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, d));
  const float mn = fmaxf(st.m, mx);
  const float ms = (mn == kNegInf) ? 0.f : mn;
  if (__any_sync(kFull, mn != st.m)) {
    const float al = fast_exp2(st.m - ms);
    st.m = mn;
    st.l *= al;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      st.o[u][0] *= al;
      st.o[u][1] *= al;
      st.o[u][2] *= al;
      st.o[u][3] *= al;
    }
    st.zc *= al;
  }
#pragma unroll
  for (int i = 0; i < N; ++i) x[i] = fast_exp2(x[i] - ms);
}

// x * y of two fp16 pairs as hi + lo: hi = rn(x y), lo = x y - hi (exact: the product has 22 bits)
__device__ __forceinline__ void hmul2_split(uint32_t x, uint32_t y, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __hmul2(u32_as_h2(x), u32_as_h2(y));
  hi = h2_as_u32(h);
  lo = h2_as_u32(__hfma2(u32_as_h2(x), u32_as_h2(y), __hneg2(h)));
}
// (xh + xl) * y as hi + lo, with xl a small correction of xh
__device__ __forceinline__ void hmul2_split(uint32_t xh, uint32_t xl, uint32_t y, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __hmul2(u32_as_h2(xh), u32_as_h2(y));
  const __half2 e = __hfma2(u32_as_h2(xh), u32_as_h2(y), __hneg2(h));
  hi = h2_as_u32(h);
  lo = h2_as_u32(__hfma2(u32_as_h2(xl), u32_as_h2(y), e));
}

// P^T B-fragments of one 16-token tile from the probabilities of the lane's rows r (pa) and r + 8 (pb):
// fp16 hi + lo parts (p = hi + lo to ~2^-22) placed in the (hi, lo) columns of the head and
// transposed.  pf = {tokens 0-7, tokens 8-15} of the lane's column: hi part (r even) or lo part (r odd).
// The unrounded probabilities go into l.
__device__ __forceinline__ void make_p_f16(float pa, float pb, uint32_t (&pf)[2], SoftmaxState& st) {
  const __half2 hh = __floats2half2_rn(pa, pb);
  const __half2 ll = __floats2half2_rn(pa - __low2float(hh), pb - __high2float(hh));
  st.l += pa + pb;
  pf[0] = movmatrix_trans(prmt(h2_as_u32(hh), h2_as_u32(ll), 0x5410u));    // (hi, lo) of row r
  pf[1] = movmatrix_trans(prmt(h2_as_u32(hh), h2_as_u32(ll), 0x7632u));    // (hi, lo) of row r + 8
}
// The same with bf16 parts (p = hi + lo to ~2^-17) for the exact rows, in the accumulators' unit 2^-18.
__device__ __forceinline__ void make_p_bf16(float pa, float pb, uint32_t (&pf)[2], SoftmaxState& st) {
  st.l += pa + pb;
  pa *= kVUnit;
  pb *= kVUnit;
  const uint32_t hh = pack_bf16x2(pa, pb);
  const uint32_t ll = pack_bf16x2(pa - bf16lo_to_f32(hh), pb - bf16hi_to_f32(hh));
  pf[0] = movmatrix_trans(prmt(hh, ll, 0x5410u));
  pf[1] = movmatrix_trans(prmt(hh, ll, 0x7632u));
}

// ---- item cursor ---------------------------------------------------------------------------
struct Cursor {
  int item;          // dense: position in the warp's unit list; sparse: position in its slice of the page list
  int first;         // dense: first item (block index) of the unit
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
  int item_end;              // dense: one past the last item; sparse: one past the last page position
  int stream;                // the (sequence, KV head) stream whose cache is read
  int sparse_rank;           // page-list reads: this warp's number among the warps of its head group
  int head0;                 // first query head (within the KV head's group) of the warp's head group
  bool has_tail;
  uint32_t stage0;           // shared-memory address of stage 0 (stage s at + s * kStageBytes)
  const uint8_t* stage_ptr0; // the same as a generic pointer
  uint32_t bar0;             // mbarrier of stage 0 (stage s at + 8 s)
  uint32_t qb_addr;          // this lane's bf16 query fragments in shared memory (16 words)
  uint32_t qh_addr;          // the same in fp16
  // dense mode: this warp's unit list and the prefetched entry of the unit after the current one
  const uint32_t* units;     // unit = first item | 16-token tile mask << 20 | run length << 24
  uint32_t pf_unit;
  uint4 pf_entry;
  int pf_pos;
};

__device__ __forceinline__ int popc4(int m) { return __popc(m & 15); }

// Unit at list position `pos` and the table entry of its first item; the pair for pos + 1 is
// requested right away so that its two dependent loads are in flight while this unit is processed.
__device__ __forceinline__ void unit_at(WarpCtx& w, int pos, uint32_t* unit, TableEntry* e) {
  uint32_t u;
  uint4 raw;
  if (pos == w.pf_pos) {
    u = w.pf_unit;
    raw = w.pf_entry;
  } else {
    u = w.units[pos];
    raw = *reinterpret_cast<const uint4*>(w.table + min(static_cast<int>(u & kUnitItemMask), w.p->n_closed));
  }
  if (pos + 1 < w.item_end) {
    w.pf_unit = w.units[pos + 1];
    w.pf_entry = *reinterpret_cast<const uint4*>(w.table + min(static_cast<int>(w.pf_unit & kUnitItemMask), w.p->n_closed));
    w.pf_pos = pos + 1;
  }
  *unit = u;
  e->off256 = raw.x;
  e->level = raw.y;
  e->resmask = (static_cast<uint64_t>(raw.w) << 32) | raw.z;
}

// Dense mode: set up the cursor for position `pos` of the warp's unit list (c.item holds the
// position, c.adv = 1).  Returns false when past the end.
__device__ __forceinline__ bool load_item_dense(WarpCtx& w, int pos, Cursor& c) {
  const DecodeParams& p = *w.p;
  while (true) {
    if (pos >= w.item_end) return false;
    uint32_t unit;
    TableEntry e;
    unit_at(w, pos, &unit, &e);
    const int it = static_cast<int>(unit & kUnitItemMask), run = static_cast<int>(unit >> 24);
    const int mask = static_cast<int>(unit >> 20) & 15;      // 16-token tiles of the block this unit covers
    c.item = pos;
    c.first = it;
    c.sub = 0;
    c.adv = 1;
    if (it <= p.n_closed) {
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
        if (nt == 0) {
          ++pos;
          continue;
        }
      }
      if (it < p.n_closed && c.level == 16) c.tmask = mask;
      // a unit may cover one half of a quantised block (tile mask 3 or 12): steps [sub, nsub)
      const int lo = (mask & 3) ? 0 : 1, hi = (mask & 12) ? 2 : 1;
      switch (c.level) {
        case 16: c.nsub = 2 * popc4(c.tmask); break;
        case 8: c.sub = 2 * lo; c.nsub = 2 * hi; break;
        case 4: c.sub = lo; c.nsub = hi; break;
        case 2: c.sub = lo; c.nsub = hi; break;
        default:     // run of up to 16 consecutive centroid blocks (merged by the host)
          c.ntok = run;
          c.nsub = 2;
          c.level = 1;
      }
      return true;
    }
    // residual group j: rows [16 j, 16 j + 16) of the stream's residual pool
    const int j = it - p.n_closed - 1;
    const int n_res = p.res_count ? p.res_count[w.stream] : 0;
    const int rows = min(16, n_res - 16 * j);
    if (rows <= 0) {
      ++pos;
      continue;
    }
    c.level = 17;
    c.ntok = rows;
    c.nsub = 2;
    c.tmask = 1;
    c.off256 = p.res_off256[w.stream] + 32u * static_cast<uint32_t>(j);   // 16 rows x 512 B = 32 units
    c.resmask = 0;
    return true;
  }
}

// Sparse mode: position `pos` in the warp's slice of the ascending page list; pages that fall in
// the same block are merged into one visit.  Position item_end stands for the tail block.  The list
// is the caller's memory: an entry outside [0, closed pages) is skipped (nothing is read through it)
// and raises kStatusInternal, which the next gkv_bits_report returns as GKV_ERR_BAD_STATE.
__device__ __forceinline__ bool load_item_sparse(WarpCtx& w, int pos, Cursor& c) {
  const DecodeParams& p = *w.p;
  const int tiles_per_page = p.page_tokens >> 4;
  const int pages_per_block = kBlock / p.page_tokens;
  const int n_pages = p.n_closed * pages_per_block;
  const int32_t* list = p.page_idx + static_cast<size_t>(w.stream) * p.n_sel;
  while (pos < w.item_end) {
    const int page = list[pos];
    if (page < 0 || page >= n_pages) {
      if (w.lane == 0) atomicOr(p.status, kStatusInternal);
      ++pos;
      continue;
    }
    const int blk = page / pages_per_block;
    int mask = ((1 << tiles_per_page) - 1) << (tiles_per_page * (page % pages_per_block));
    int adv = 1;
    while (pos + adv < w.item_end) {
      const int pg = list[pos + adv];
      if (pg < 0 || pg >= n_pages || pg / pages_per_block != blk) break;
      mask |= ((1 << tiles_per_page) - 1) << (tiles_per_page * (pg % pages_per_block));
      ++adv;
    }
    const TableEntry e = w.table[blk];
    c.item = pos;
    c.first = page;              // the visit's first page (the centroid gather looks its block up again)
    c.sub = 0;
    c.adv = adv;
    c.off256 = e.off256;
    c.resmask = e.resmask;       // tokens served from the residual pool: their stored copies are masked
    c.level = static_cast<int>(e.level);
    c.tmask = mask;
    c.ntok = kBlock;
    switch (c.level) {
      case 16: c.nsub = 2 * popc4(mask); break;
      case 8: c.nsub = 2 * (((mask & 3) != 0) + ((mask & 12) != 0)); break;
      case 4:
      case 2: c.nsub = ((mask & 3) != 0) + ((mask & 12) != 0); break;
      default: c.nsub = 2; c.ntok = 1; break;     // a single centroid row weighted by the selected tokens
    }
    return true;
  }
  // pos == item_end (also after skipped entries): the tail
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
  // Positions past the tail: the stream's groups of 16 exact residual rows, dealt round-robin to
  // its warps.  Which rows of a group count (those whose page is listed) is decided when the
  // group is computed.
  const int n_res = p.res_count ? p.res_count[w.stream] : 0;
  const int n_groups = (n_res + 15) >> 4;
  const int k = max(pos - w.item_end - 1, 0);
  const int j = w.sparse_rank + k * p.warps_per_stream;
  if (j >= n_groups) return false;
  c.item = w.item_end + 1 + k;
  c.first = p.n_closed + 1 + j;
  c.sub = 0;
  c.adv = 1;
  c.level = 17;
  c.ntok = min(16, n_res - 16 * j);
  c.nsub = 2;
  c.tmask = 1;
  c.off256 = p.res_off256[w.stream] + 32u * static_cast<uint32_t>(j);
  c.resmask = 0;
  return true;
}

// Page-list reads: is the page of token `tok` in the stream's ascending list?
__device__ __forceinline__ bool page_listed(const DecodeParams& p, int stream, int tok) {
  const int32_t* list = p.page_idx + static_cast<size_t>(stream) * p.n_sel;
  const int page = tok / p.page_tokens;
  int lo = 0, hi = p.n_sel;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (list[mid] < page) lo = mid + 1;
    else hi = mid;
  }
  return lo < p.n_sel && list[lo] == page;
}

template <bool SPARSE>
__device__ __forceinline__ bool load_item(WarpCtx& w, int it, Cursor& c) {
  if constexpr (SPARSE) return load_item_sparse(w, it, c);
  else return load_item_dense(w, it, c);
}
template <bool SPARSE>
__device__ __forceinline__ bool advance(WarpCtx& w, Cursor& c) {
  if (++c.sub < c.nsub) return true;
  return load_item<SPARSE>(w, c.item + c.adv, c);
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
// idx-th half that has an active tile (levels 8 and 4, sparse visits)
__device__ __forceinline__ int half_of_step(const Cursor& c, int idx) {
  const bool h0 = (c.tmask & 3) != 0;
  return (idx == 0) ? (h0 ? 0 : 1) : 1;
}

// Issue the TMA bulk copies of the cursor's current step into stage `sidx`.  The warp must have
// finished reading that stage (callers __syncwarp() before).
template <bool SPARSE>
__device__ __forceinline__ void issue_step(const WarpCtx& w, const Cursor& c, int sidx) {
  const DecodeParams& p = *w.p;
  const uint32_t sdst = w.stage0 + sidx * kStageBytes, bar = w.bar0 + sidx * 8;
  const int lane = w.lane;
  if (c.level == 16 || c.level == 17) {
    // 16 rows of 256 B at a regular stride, staged at a 272-byte pitch: 256 16-byte pieces, eight per
    // lane (piece q = lane + 32 i is row q / 16, column q % 16).  Rows past the end are written as
    // zeros so that 0 * garbage never produces a NaN.  The warp's copies complete the barrier
    // phase through one tracked arrival per lane plus the plain arrival that matches the
    // barrier's count of one.
    const bool is_v = (c.sub & 1) != 0;
    const int row0 = lane >> 4, col = lane & 15;
    const uint8_t* g = p.arena + static_cast<size_t>(c.off256) * 256 + col * 16;
    const uint32_t d = sdst + row0 * kRowPitch + col * 16;
    if (c.level == 16) {
      const int tile = nth_set_bit(c.tmask, c.sub >> 1);
      const int nrows = c.ntok - tile * 16;
      g += (is_v ? kBlock * kRowBytes : 0) + static_cast<size_t>(tile * 16 + row0) * kRowBytes;
#pragma unroll
      for (int i = 0; i < 8; ++i) cp_async16(d + i * 2 * kRowPitch, g + i * 2 * kRowBytes, (row0 + 2 * i < nrows) ? 16u : 0u);
    } else {
      g += (is_v ? kRowBytes : 0) + static_cast<size_t>(row0) * 2 * kRowBytes;
#pragma unroll
      for (int i = 0; i < 8; ++i) cp_async16(d + i * 2 * kRowPitch, g + i * 4 * kRowBytes, (row0 + 2 * i < c.ntok) ? 16u : 0u);
    }
    cp_async_mbar_arrive(bar);
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
    return;
  }
  if (c.level == 1) {
    // up to 16 centroid rows gathered from their blocks; one bulk copy per row
    const bool is_v = (c.sub & 1) != 0;
    const uint8_t* src = nullptr;
    const int nrows = c.ntok;
    if (lane < nrows) {
      int blk;
      if constexpr (SPARSE) blk = c.first / (kBlock / p.page_tokens);      // c.first = the visit's (range-checked) first page
      else blk = c.first + lane;
      src = p.arena + static_cast<size_t>(w.table[blk].off256) * 256 + (is_v ? kRowBytes : 0);
    }
    if (lane == 0) mbar_expect_tx(bar, static_cast<uint32_t>(nrows) * kRowBytes);
    __syncwarp();
    if (lane < nrows) {
      bulk_g2s(sdst + lane * kRowPitch, src, kRowBytes, bar);
    } else if (lane < 16) {
      uint4* z = reinterpret_cast<uint4*>(const_cast<uint8_t*>(w.stage_ptr0) + sidx * kStageBytes + lane * kRowPitch);
#pragma unroll
      for (int i = 0; i < kRowBytes / 16; ++i) z[i] = make_uint4(0, 0, 0, 0);
    }
    return;
  }
  const int bits = c.level;
  const int cb = code_bytes_per_tile(bits);
  const uint8_t* slot = p.arena + static_cast<size_t>(c.off256) * 256;
  if (!SPARSE || c.tmask == 15) {
    // full block: every step is one contiguous span of the slot, all steps of a level alike
    // (8-bit: key part and value part of each half, 4608 B; 4- and 2-bit: one half)
    const uint32_t bytes = (bits == 8) ? 512 + 2 * 2048 : (bits == 4 ? half_bytes(4) : half_bytes(2));
    const uint8_t* src = slot + c.sub * bytes;
    if (lane == 0) {
      mbar_expect_tx(bar, bytes);
      bulk_g2s(sdst, src, bytes, bar);
    }
    return;
  }
  if (lane != 0) return;
  // sparse visit: copy only the pieces of the selected tiles (same stage offsets as a full copy)
  if (bits == 8) {
    const int half = half_of_step(c, c.sub >> 1);
    const int tm = (c.tmask >> (2 * half)) & 3;
    const uint8_t* hb = slot + half * half_bytes(8);
    const int nt = popc4(tm);
    if ((c.sub & 1) == 0) {
      mbar_expect_tx(bar, 512 + nt * cb);
      bulk_g2s(sdst, hb, 512, bar);
      for (int t = 0; t < 2; ++t)
        if (tm & (1 << t)) bulk_g2s(sdst + 512 + t * cb, hb + off_kc(8, t), cb, bar);
    } else {
      mbar_expect_tx(bar, nt * (256 + cb));
      for (int t = 0; t < 2; ++t)
        if (tm & (1 << t)) {
          bulk_g2s(sdst + t * 256, hb + off_vp(8, t), 256, bar);
          bulk_g2s(sdst + 512 + t * cb, hb + off_vc(8, t), cb, bar);
        }
    }
  } else {
    const int half = half_of_step(c, c.sub);
    const int tm = (c.tmask >> (2 * half)) & 3;
    const uint8_t* hb = slot + half * half_bytes(bits);
    mbar_expect_tx(bar, 512 + popc4(tm) * (2 * cb + 256));
    bulk_g2s(sdst, hb, 512, bar);
    for (int t = 0; t < 2; ++t)
      if (tm & (1 << t)) {
        bulk_g2s(sdst + off_kc(bits, t), hb + off_kc(bits, t), cb, bar);
        bulk_g2s(sdst + off_vp(bits, t), hb + off_vp(bits, t), 256, bar);
        bulk_g2s(sdst + off_vc(bits, t), hb + off_vc(bits, t), cb, bar);
      }
  }
}

// ---- compute ---------------------------------------------------------------------------------
__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
// D = A B (no accumulator input: the first MMA of a chain)
__device__ __forceinline__ void mma_f16_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}

// Code words of MMA indices (2 j, 2 j + 1) of one lane: 8-bit 4 words, 4-bit 2 words, 2-bit 1 word.
template <int BITS>
__device__ __forceinline__ void load_words(uint32_t codes, int j, int lane, uint32_t (&w)[BITS / 2]) {
  constexpr int kW = BITS / 2;
  const uint32_t a = codes + ((j * kW >> 2) * 32 + lane) * 16 + ((j * kW) & 3) * 4;
  if constexpr (BITS == 8) {
    const uint4 v = lds128(a);
    w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
  } else if constexpr (BITS == 4) {
    const uint2 v = lds64(a);
    w[0] = v.x; w[1] = v.y;
  } else {
    w[0] = lds32(a);
  }
}

// Logits of the active tiles of one half (32 tokens): S = scale * (q . k~) + token bias, with
// k~ = s * code + z.  Data MMAs use A = code * 2^(p - 24) and B = q' = q * s (hi and lo columns); an MMA with
// A = zero points and B = q gives sum q z.  All arguments that address shared memory are 32-bit addresses.
// Channel slab j (MMA indices 2 j and 2 j + 1) of qk_half; FIRST starts the accumulation chains.
template <int BITS, bool FULL, bool FIRST>
__device__ __forceinline__ void qk_slab(uint32_t kp, uint32_t kc0, int j, int tm, uint32_t qh_addr, int lane,
                                        float (&zd)[4], float (&S)[2][4]) {
  constexpr int cb = 256 * BITS;
  constexpr int kW = BITS / 2;
  uint32_t w0[kW], w1[kW];
  if (FULL || (tm & 1)) load_words<BITS>(kc0, j, lane, w0);
  if (FULL || (tm & 2)) load_words<BITS>(kc0 + cb, j, lane, w1);
  // zero points and scales of the slab's two MMA indices: {s0: c0 c1, s1: c0 c1, s0: c2 c3, s1: c2 c3}
  const uint4 zp = lds128(kp + j * 128), sp = lds128(kp + j * 128 + 16);
  {
    // sum q z of both MMA indices in one MMA: rows r carry the zero points of index s0, rows r + 8 those of
    // s1; the hi column of a head carries the query slice of s0, its lo column that of s1.  The wanted
    // products sit in the accumulator registers 0 (row r, hi column) and 3 (row r + 8, lo column).
    const uint2 qz = lds64(qh_addr + j * 512 + (lo_part_lane(lane) ? 256 : 0));
    if (FIRST) mma_f16_first(zd, zp.x, zp.y, zp.z, zp.w, qz.x, qz.y);
    else mma_f16(zd, zp.x, zp.y, zp.z, zp.w, qz.x, qz.y);
  }
#pragma unroll
  for (int ss = 0; ss < 2; ++ss) {
    const uint2 q = lds64(qh_addr + j * 512 + ss * 256);
    uint32_t q0, q1, q0l, q1l;
    hmul2_split(q.x, ss ? sp.y : sp.x, q0, q0l);
    hmul2_split(q.y, ss ? sp.w : sp.z, q1, q1l);
    if (lo_part_lane(lane)) {
      q0 = q0l;
      q1 = q1l;
    }
    uint32_t a[4];
    if (FULL || (tm & 1)) {
      unpack<BITS, false>(w0, ss, a);
      if (FIRST && ss == 0) mma_f16_first(S[0], a[0], a[1], a[2], a[3], q0, q1);
      else mma_f16(S[0], a[0], a[1], a[2], a[3], q0, q1);
    }
    if (FULL || (tm & 2)) {
      unpack<BITS, false>(w1, ss, a);
      if (FIRST && ss == 0) mma_f16_first(S[1], a[0], a[1], a[2], a[3], q0, q1);
      else mma_f16(S[1], a[0], a[1], a[2], a[3], q0, q1);
    }
  }
}

// x = the four logits of the lane's head: tile 0 rows r, r + 8, tile 1 rows r, r + 8.
template <int BITS, bool FULL>
__device__ __forceinline__ void qk_half(uint32_t kp, uint32_t kc0, int tm, uint32_t qh_addr, int lane, float scale_log2,
                                        uint64_t resmask, int half, float (&x)[4]) {
  const int c4 = lane & 3, r = lane >> 2;
  // sum_c q_c z_c = zd[0] + zd[3] (exact products, see qk_slab)
  float zd[4];
  float S[2][4];
  kp += c4 * 32;
  qk_slab<BITS, FULL, true>(kp, kc0, 0, tm, qh_addr, lane, zd, S);
#pragma unroll
  for (int j = 1; j < 4; ++j) qk_slab<BITS, FULL, false>(kp, kc0, j, tm, qh_addr, lane, zd, S);
  // rows r and rows r + 8 carry the weights of their code fields (KScale)
  const float k_lo = KScale<BITS>::lo * scale_log2, k_hi = KScale<BITS>::hi * scale_log2, zs = (zd[0] + zd[3]) * scale_log2;
  const uint32_t rm = static_cast<uint32_t>(resmask >> (32 * half));            // this half's 32 tokens
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const bool on = FULL || ((tm >> t) & 1);
    const int tok = 16 * t + r;
    const float v_lo = on ? fmaf(S[t][0] + S[t][1], k_lo, zs) : kNegInf;
    const float v_hi = on ? fmaf(S[t][2] + S[t][3], k_hi, zs) : kNegInf;
    x[2 * t] = ((rm >> tok) & 1u) ? kNegInf : v_lo;
    x[2 * t + 1] = ((rm >> (tok + 8)) & 1u) ? kNegInf : v_hi;
  }
}

// O^T += V~^T P^T for the active tiles of one half, v~ = s * code + z per (token, 32-channel group).
// pf holds the fp16 P^T fragments of the two tiles (hi / lo columns); tile t has its parameters at
// vp + 256 t and its codes at vc + 256 BITS t.  The data MMAs accumulate code * P' (bias-free codes,
// see unpack) straight into O; the zero points go through one MMA per tile into zc.
// The loop over the two tiles is kept rolled (see qk_half).
template <int BITS, bool FULL>
__device__ __forceinline__ void pv_half(uint32_t vp, uint32_t vc, int tm, const uint32_t (&pf)[2][2], int lane,
                                        SoftmaxState& st) {
  constexpr int cb = 256 * BITS;
  const int c4 = lane & 3, r = lane >> 2;
  const bool lo_lane = lo_part_lane(lane);
  float tz[4] = {0.f, 0.f, 0.f, 0.f};   // rows g < 4: sum_tok p z[tok][g] (rows 8 + g: sum_tok p s[tok][g], not used)
  const __half2 f_lo = __float2half2_rn(VScale<BITS>::lo), f_hi = __float2half2_rn(VScale<BITS>::hi);
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    if (!FULL && !((tm >> t) & 1)) continue;
    const uint32_t m0 = t ? pf[1][0] : pf[0][0], m1 = t ? pf[1][1] : pf[0][1];
    // the hi parts, also in the lanes that hold a lo column (their partner is the lane 4 below)
    const uint32_t h0 = __shfl_sync(kFull, m0, lane & ~4), h1 = __shfl_sync(kFull, m1, lane & ~4);
    const uint32_t vpt = vp + t * 256, vct = vc + t * cb;
    // per-lane scales of its token pairs, all four groups: {sA, sB} x 4
    const uint4 x = lds128(vpt + c4 * 32), y = lds128(vpt + c4 * 32 + 16);
    uint2 z = make_uint2(0, 0), sg = make_uint2(0, 0);
    if (r < 4) {
      z = lds64(vpt + 128 + (r * 4 + c4) * 8);
      sg = lds64(vpt + c4 * 32 + r * 8);
    }
    mma_f16(tz, z.x, sg.x, z.y, sg.y, m0, m1);
    const uint32_t sc[8] = {x.x, x.y, x.z, x.w, y.x, y.y, y.z, y.w};
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      // the scales in the accumulators' unit: tokens 0-7 (sA) and 8-15 (sB) of the tile
      const uint32_t sa = h2_as_u32(__hmul2(u32_as_h2(sc[2 * g]), f_lo));
      const uint32_t sb = VScale<BITS>::hi == 1.f ? sc[2 * g + 1] : h2_as_u32(__hmul2(u32_as_h2(sc[2 * g + 1]), f_hi));
      uint32_t p0, p1, p0l, p1l;
      hmul2_split(h0, m0, sa, p0, p0l);        // (m0, m1 are the lo parts where p0l, p1l are used)
      hmul2_split(h1, m1, sb, p1, p1l);
      if (lo_lane) {
        p0 = p0l;
        p1 = p1l;
      }
      uint32_t wd[BITS / 2];
      uint32_t a[4];
      load_words<BITS>(vct, g, lane, wd);
      unpack<BITS, true>(wd, 0, a);
      mma_f16(st.o[2 * g], a[0], a[1], a[2], a[3], p0, p1);
      unpack<BITS, true>(wd, 1, a);
      mma_f16(st.o[2 * g + 1], a[0], a[1], a[2], a[3], p0, p1);
    }
  }
  st.zc += tz[0] + tz[1];
}

template <int BITS, bool FULL>
__device__ __forceinline__ void qk_softmax_half(uint32_t half_k, int half, int tm, uint64_t resmask, uint32_t qh_addr,
                                                int lane, float scale_log2, SoftmaxState& st,
                                                uint32_t (&pf)[2][2]) {
  float x[4];
  qk_half<BITS, FULL>(half_k, half_k + 512, tm, qh_addr, lane, scale_log2, resmask, half, x);
  softmax_update<4>(x, st);
  make_p_f16(x[0], x[1], pf[0], st);
  make_p_f16(x[2], x[3], pf[1], st);
}

// Process a staged step.  pf carries P fragments from a key step to the following value step.
template <bool SPARSE, bool MASS>
__device__ __forceinline__ void compute_step(const WarpCtx& w, const Cursor& c, int sidx,
                                             SoftmaxState& st, uint32_t (&pf)[4]) {
  const DecodeParams& p = *w.p;
  const int lane = w.lane;
  const uint32_t sa = w.stage0 + sidx * kStageBytes;
  if (c.level == 16 || c.level == 1 || c.level == 17) {
    uint32_t (&pfx)[2] = *reinterpret_cast<uint32_t (*)[2]>(&pf);
    if ((c.sub & 1) == 0) {
      // key rows: S^T = K Q^T (bf16 x bf16 products are exact; the hi and lo columns of a head both
      // hold its query, so the two accumulator columns are equal)
      float S[4] = {0.f, 0.f, 0.f, 0.f};
      const int mi = lane >> 3;
      const uint32_t base = sa + ((lane & 7) + (mi & 1) * 8) * kRowPitch + (mi >> 1) * 16;
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        uint32_t a[4];
        ldmatrix_x4(a, base + s * 32);
        const uint2 b = lds64(w.qb_addr + s * 256);
        mma_bf16(S, a, b.x, b.y);
      }
      // validity / weight of the lane's rows r and r + 8
      const int r = lane >> 2;
      float b_lo, b_hi;
      if (c.level == 16) {
        const int tile = nth_set_bit(c.tmask, c.sub >> 1);
        const int t0 = tile * 16 + r;
        b_lo = (t0 < c.ntok && !((c.resmask >> t0) & 1ull)) ? 0.f : kNegInf;
        b_hi = (t0 + 8 < c.ntok && !((c.resmask >> (t0 + 8)) & 1ull)) ? 0.f : kNegInf;
      } else if (c.level == 17) {
        bool on_lo = r < c.ntok, on_hi = r + 8 < c.ntok;
        if constexpr (SPARSE) {
          // a residual row counts only when the page of its token is listed (Sec. 3.5: every token of
          // a page that is not selected is masked, exact or not)
          const int32_t* ri = p.res_idx + static_cast<size_t>(w.stream) * p.res_cap + 16 * (c.first - p.n_closed - 1);
          on_lo = on_lo && page_listed(p, w.stream, ri[r]);
          on_hi = on_hi && page_listed(p, w.stream, ri[r + 8]);
        }
        b_lo = on_lo ? 0.f : kNegInf;
        b_hi = on_hi ? 0.f : kNegInf;
      } else {
        // centroid rows: each stands for the block's readable tokens -> add log2(count)
        float myb = kNegInf;
        if (lane < c.ntok) {
          int cnt;
          if constexpr (SPARSE) {
            // tokens of the selected pages that are not served from the residual pool
            uint64_t sel = 0;
#pragma unroll
            for (int t4 = 0; t4 < 4; ++t4)
              if ((c.tmask >> t4) & 1) sel |= 0xffffull << (16 * t4);
            cnt = __popcll(sel & ~c.resmask);
          } else {
            cnt = kBlock - __popcll(w.table[c.first + lane].resmask);
          }
          myb = cnt > 0 ? log2f(static_cast<float>(cnt)) : kNegInf;
        }
        b_lo = __shfl_sync(kFull, myb, r);
        b_hi = __shfl_sync(kFull, myb, r + 8);
      }
      float x[2] = {fmaf(S[0], p.scale_log2, b_lo), fmaf(S[2], p.scale_log2, b_hi)};
      softmax_update<2>(x, st);
      if constexpr (MASS) {
        // centroid rows stand for whole blocks and residual rows belong to the block of their token:
        // their weights are recorded row by row (relative to the running max, which goes with them)
        if (c.level != 16) {
          const int head = w.head0 + (lane & 3);
          float2* dst = (c.level == 1)
                            ? p.mass_raw + (static_cast<size_t>(w.stream) * p.mass_stride + c.first) * kMaxHeadsPerKv
                            : p.res_raw + (static_cast<size_t>(w.stream) * p.res_cap + 16 * (c.first - p.n_closed - 1)) * kMaxHeadsPerKv;
          if (r < c.ntok) dst[r * kMaxHeadsPerKv + head] = make_float2(st.m, x[0]);
          if (r + 8 < c.ntok) dst[(r + 8) * kMaxHeadsPerKv + head] = make_float2(st.m, x[1]);
        }
      }
      make_p_bf16(x[0], x[1], pfx, st);
    } else {
      // value rows: O^T += V^T P^T with P = hi + lo in the head's two columns
      const int mi = lane >> 3;
      const uint32_t base = sa + ((lane & 7) + (mi >> 1) * 8) * kRowPitch + (mi & 1) * 16;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        uint32_t a[4];
        ldmatrix_x4_trans(a, base + u * 32);
        mma_bf16(st.o[u], a, pfx[0], pfx[1]);
      }
    }
    return;
  }
  uint32_t (&pf2)[2][2] = *reinterpret_cast<uint32_t (*)[2][2]>(&pf);
  constexpr bool FULL = !SPARSE;
  const uint32_t qh = w.qh_addr;
  if (c.level == 8) {
    const int half = FULL ? (c.sub >> 1) : ((c.tmask == 15) ? (c.sub >> 1) : half_of_step(c, c.sub >> 1));
    const int tm = (c.tmask >> (2 * half)) & 3;
    if ((c.sub & 1) == 0) qk_softmax_half<8, FULL>(sa, half, tm, c.resmask, qh, lane, p.scale_log2, st, pf2);
    else pv_half<8, FULL>(sa, sa + 512, tm, pf2, lane, st);
  } else {
    const int half = FULL ? c.sub : ((c.tmask == 15) ? c.sub : half_of_step(c, c.sub));
    const int tm = (c.tmask >> (2 * half)) & 3;
    if (c.level == 4) {
      qk_softmax_half<4, FULL>(sa, half, tm, c.resmask, qh, lane, p.scale_log2, st, pf2);
      pv_half<4, FULL>(sa + off_vp(4, 0), sa + off_vc(4, 0), tm, pf2, lane, st);
    } else {
      qk_softmax_half<2, FULL>(sa, half, tm, c.resmask, qh, lane, p.scale_log2, st, pf2);
      pv_half<2, FULL>(sa + off_vp(2, 0), sa + off_vc(2, 0), tm, pf2, lane, st);
    }
  }
}

template <bool SPARSE, bool MASS>
__global__ void __launch_bounds__(kDecodeWarps * 32, kDecodeCtasPerSm) decode_kernel(const __grid_constant__ DecodeParams p) {
  static_assert(!(SPARSE && MASS), "block masses are observed by full reads only");
  extern __shared__ __align__(128) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gw = blockIdx.x * kDecodeWarps + warp;

  WarpCtx w;
  w.p = &p;
  w.lane = lane;
  w.units = p.units;
  w.pf_pos = -1;
  w.pf_unit = 0;
  w.pf_entry = make_uint4(0, 0, 0, 0);
  w.stream = -1;
  w.head0 = 0;
  w.sparse_rank = 0;
  w.item_end = 0;
  w.has_tail = false;
  // A warp works for one head group: up to four query heads of one KV head.  Head group hg of stream s
  // has the index s * head_groups + hg; partial rows, ranges of rows and tickets go by that index.
  int hgroup = -1, partial_row = 0, first = 0;
  if (gw < p.n_warps) {
    if constexpr (!SPARSE) {
      const WarpDesc wd = p.warps[gw];
      hgroup = wd.stream;
      w.item_end = wd.item_end;
      first = wd.item_begin;
      partial_row = wd.partial;
    } else {
      const int wps = p.warps_per_stream;
      hgroup = gw / wps;
      const int wi = gw - hgroup * wps;
      first = static_cast<int>((static_cast<long long>(wi) * p.n_sel) / wps);
      w.item_end = static_cast<int>((static_cast<long long>(wi + 1) * p.n_sel) / wps);
      w.has_tail = (wi == wps - 1);
      w.sparse_rank = wi;
      partial_row = blockIdx.x;      // whole CTAs per head group: one partial row per CTA
    }
  }
  // per-warp (head group, partial row) for the merge at the end
  int* s_group = reinterpret_cast<int*>(smem + kDecodeWarps * (kStages * kStageBytes + kStages * 8 + 2 * 2048));
  if (lane == 0) {
    s_group[warp] = hgroup;
    s_group[kDecodeWarps + warp] = partial_row;
  }
  if (hgroup >= 0) {
  w.stream = hgroup / p.head_groups;
  w.head0 = kHeadsPerWarp * (hgroup - w.stream * p.head_groups);
  w.table = p.table + static_cast<size_t>(w.stream) * p.table_stride;
  uint8_t* sbase = smem + warp * (kStages * kStageBytes);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kDecodeWarps * kStages * kStageBytes) + warp * kStages;
  uint8_t* qb_smem = smem + kDecodeWarps * (kStages * kStageBytes + kStages * 8) + warp * 2048;
  w.stage_ptr0 = sbase;
  w.stage0 = smem_u32(sbase);
  w.bar0 = smem_u32(bars);
  w.qb_addr = smem_u32(qb_smem) + lane * 8;       // word pair s at + 256 s (conflict-free 8-byte accesses)
  w.qh_addr = w.qb_addr + kDecodeWarps * 2048;
  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < kStages; ++s) mbar_init(w.bar0 + 8 * s, 1);
    fence_proxy_async();
  }
  __syncwarp();
  // The start of a launch is a chain of dependent look-ups (work list -> block table -> bytes):
  // the first unit word is asked for here, its table entry right after the wait below, so that both
  // are on their way while the query is staged.  unit_at() picks them up as its prefetched pair.
  if constexpr (!SPARSE) {
    if (first < w.item_end) w.pf_unit = w.units[first];
  }
  // Launched with programmatic stream serialisation: what is above (descriptor fetch, barrier
  // set-up, the first word of the host-written work list) may overlap the tail of the previous
  // kernel in the stream.  Nothing that a previous kernel may have written (the block table, the
  // query, appended rows, partial rows, tickets) is touched before this wait, which returns once
  // that kernel has completed and its writes are visible.
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  if constexpr (!SPARSE) {
    if (first < w.item_end) {
      w.pf_entry = *reinterpret_cast<const uint4*>(w.table + min(static_cast<int>(w.pf_unit & kUnitItemMask), p.n_closed));
      w.pf_pos = first;
    }
  }

  // Query fragments: B operand Q^T[16 channels x 8 columns]; lane (r, c4) holds column r = the hi
  // (r even) or lo (r odd) column of head r / 2 of the head group, channels 16 s + 2 c4 (+1) and
  // 16 s + 8 + 2 c4 (+1), in bf16 (exact rows) and fp16 (quantised tiers).  Both columns of a head
  // hold its query; the parts of the scaled query are formed per key group.
  const int r = lane >> 2, c4 = lane & 3;
  {
    const int b = w.stream / p.n_kv_heads, kvh = w.stream - b * p.n_kv_heads;
    const int n_q_heads = p.n_kv_heads * p.group;
    const int head = w.head0 + (r >> 1);
    const uint16_t* qrow = p.q + (static_cast<size_t>(b) * n_q_heads + static_cast<size_t>(kvh) * p.group + head) * kD;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
      uint32_t v0 = 0, v1 = 0;
      if (head < p.group) {
        v0 = *reinterpret_cast<const uint32_t*>(qrow + 16 * s + 2 * c4);
        v1 = *reinterpret_cast<const uint32_t*>(qrow + 16 * s + 8 + 2 * c4);
      }
      asm volatile("st.shared.v2.u32 [%0], {%1,%2};\n" ::"r"(w.qb_addr + s * 256), "r"(v0), "r"(v1) : "memory");
      const uint32_t h0 = h2_as_u32(__floats2half2_rn(bf16lo_to_f32(v0), bf16hi_to_f32(v0)));
      const uint32_t h1 = h2_as_u32(__floats2half2_rn(bf16lo_to_f32(v1), bf16hi_to_f32(v1)));
      asm volatile("st.shared.v2.u32 [%0], {%1,%2};\n" ::"r"(w.qh_addr + s * 256), "r"(h0), "r"(h1) : "memory");
    }
  }
  __syncwarp();

  SoftmaxState st;
  st.m = kNegInf;
  st.l = 0.f;
#pragma unroll
  for (int u = 0; u < 8; ++u) st.o[u][0] = st.o[u][1] = st.o[u][2] = st.o[u][3] = 0.f;
  st.zc = 0.f;
  uint32_t pf[4] = {0, 0, 0, 0};

  // Software pipeline over steps: while step k is computed, step k + 1 is in flight.  The loop
  // starts on an empty pseudo-unit (level 0) so that the cursor and copy code exists once.
  Cursor cur;
  cur.item = first - 1;
  cur.first = 0;
  cur.sub = 0;
  cur.nsub = 1;
  cur.adv = 1;
  cur.level = 0;
  cur.ntok = 0;
  cur.tmask = 0;
  cur.off256 = 0;
  cur.resmask = 0;
  bool have = true;
  int sidx = 1;
  uint32_t phase = 0;             // bit s = parity to wait for on stage s
  bool failed = false;
  float mass_l = 0.f, mass_m = kNegInf;     // (l, m) when the current block began
  while (have) {
    Cursor nxt = cur;
    const bool more = advance<SPARSE>(w, nxt);
    if (more) issue_step<SPARSE>(w, nxt, sidx ^ 1);
    if (cur.level != 0) {
      // bounded wait for this step's bytes
      int spins = 0;
      while (!mbar_try_wait(w.bar0 + 8 * sidx, (phase >> sidx) & 1u)) {
        if (++spins > kWaitSpins) {
          failed = true;
          break;
        }
      }
      if (__any_sync(kFull, failed)) break;
      phase ^= 1u << sidx;
      if constexpr (MASS) {
        if (cur.sub == 0) {
          mass_l = st.l;
          mass_m = st.m;
        }
      }
      compute_step<SPARSE, MASS>(w, cur, sidx, st, pf);
      if constexpr (MASS) {
        // A block (or the partial block) is done: what it added to the lane's running sum is the
        // sum now minus the sum at its start brought to the current max.
        if (cur.sub == cur.nsub - 1 && cur.level != 1 && cur.level != 17) {
          float d0 = st.l - ((mass_m == kNegInf) ? 0.f : mass_l * fast_exp2(mass_m - st.m));
#pragma unroll
          for (int d = 4; d <= 16; d <<= 1) d0 += __shfl_xor_sync(kFull, d0, d);
          if (lane < 4)
            p.mass_raw[(static_cast<size_t>(w.stream) * p.mass_stride + cur.first) * kMaxHeadsPerKv + w.head0 + lane] =
                make_float2(st.m, fmaxf(d0, 0.f));
        }
      }
      __syncwarp();
    }
    cur = nxt;
    have = more;
    sidx ^= 1;
  }
  if (failed) {
    // a copy never completed: flag it and publish an empty partial (the host reports BAD_STATE)
    if (lane == 0) atomicOr(p.status, kStatusInternal);
    st.m = kNegInf;
    st.l = 0.f;
  }

  // lane-partial sum -> the head's sum (reduce over the 8 r lanes that share c4)
#pragma unroll
  for (int d = 4; d <= 16; d <<= 1) st.l += __shfl_xor_sync(kFull, st.l, d);
  // the warp's partial row goes to its own (now idle) stage memory: hi + lo columns added, plus the
  // value zero-point term (row g of zc, held by lane 4 g + c4, belongs to channels [32 g, 32 g + 32))
  float* out = reinterpret_cast<float*>(sbase) + c4 * (kD + 2);
  if (r == 0) {
    out[0] = st.m;
    out[1] = st.l;
  }
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const float z = __shfl_sync(kFull, st.zc, 4 * (u >> 1) + c4);
    out[2 + 16 * u + r] = fmaf(st.o[u][0] + st.o[u][1], kVUnitInv, z);
    out[2 + 16 * u + 8 + r] = fmaf(st.o[u][2] + st.o[u][3], kVUnitInv, z);
  }
  }   // hgroup >= 0

  // Merge the rows of the CTA's warps that share a stream (they are neighbours) into one global
  // partial row per (CTA, stream), in warp order; every warp of the CTA arrives here exactly once.
  __syncthreads();
  constexpr int kRowFloats = kStages * kStageBytes / 4;     // distance between two warps' rows
  const float* rows = reinterpret_cast<const float*>(smem);
  int gb = 0;
#pragma unroll 1
  while (gb < kDecodeWarps) {
    const int sid = s_group[gb];
    int ge = gb + 1;
#pragma unroll 1
    while (ge < kDecodeWarps && s_group[ge] == sid) ++ge;
    if (sid >= 0) {
      const int sid_stream = sid / p.head_groups, sid_head0 = kHeadsPerWarp * (sid - sid_stream * p.head_groups);
      const int n_heads = min(kHeadsPerWarp, p.group - sid_head0);
      const int n_pair = n_heads * ((kD + 2) / 2);
      float* dst = p.partial + static_cast<size_t>(s_group[kDecodeWarps + gb]) * kPartialFloats;
      // the stream's range of partial rows, asked for now and needed when the ticket is taken
      // (sparse mode: a stream's CTAs are neighbours, one partial row each, row = CTA index)
      int row_begin = 0, row_end = 0;
      if (threadIdx.x == 0) {
        const int per = p.warps_per_stream / kDecodeWarps;
        row_begin = sid * per;
        row_end = row_begin + per;
        if (p.parts) {
          const StreamParts sp = p.parts[sid];
          row_begin = sp.begin;
          row_end = sp.end;
        }
      }
      // an element is a pair of floats of the row: (m, l) of a head, or two of its channels
#pragma unroll 1
      for (int e = threadIdx.x; e < n_pair; e += kDecodeWarps * 32) {
        const int h = e / ((kD + 2) / 2), j = e - h * ((kD + 2) / 2);
        // one pass in warp order: running maximum M and the sums relative to it (the loads of the
        // rows do not depend on one another; only the short rescaling chain is serial)
        const float* col = rows + h * (kD + 2);
        float M = kNegInf, acc0 = 0.f, acc1 = 0.f;
#pragma unroll 2
        for (int i = gb; i < ge; ++i) {
          const float m = col[i * kRowFloats];
          const float2 v = *reinterpret_cast<const float2*>(col + i * kRowFloats + 2 * j);
          const float Mn = fmaxf(M, m);
          const float a = (M == kNegInf) ? 0.f : fast_exp2(M - Mn), bwt = (m == kNegInf) ? 0.f : fast_exp2(m - Mn);
          acc0 = fmaf(acc0, a, v.x * bwt);
          acc1 = fmaf(acc1, a, v.y * bwt);
          M = Mn;
        }
        *reinterpret_cast<float2*>(dst + h * (kD + 2) + 2 * j) = make_float2(j == 0 ? M : acc0, acc1);
      }
      // The CTA that delivers the stream's last row normalises and writes the output: rows are
      // published with a fence before the ticket is taken, and read back through L2.  Nobody
      // waits for anybody; the order of summation is the row order, whichever CTA does it.
      __threadfence();
      __syncthreads();
      if (threadIdx.x == 0) {
        const int begin = row_begin, end = row_end;
        const int n = end - begin;
        bool is_last = true;
        if (n > 1) {
          is_last = atomicAdd(&p.tickets[sid], 1) == n - 1;
          if (is_last) p.tickets[sid] = 0;        // ready for the next launch
        }
        s_group[2 * kDecodeWarps] = is_last ? begin : -1;
        s_group[2 * kDecodeWarps + 1] = end;
      }
      __syncthreads();
      const int begin = s_group[2 * kDecodeWarps], end = s_group[2 * kDecodeWarps + 1];
      if (begin >= 0) {
        __threadfence();
        const int b = sid_stream / p.n_kv_heads, kvh = sid_stream - b * p.n_kv_heads;
        // a thread takes two neighbouring channels of a head and one half of the rows; the second half's
        // aggregate joins the first's through shared memory (warp 0's stage memory behind its row), so
        // the order of summation stays fixed whichever CTA does it
        float4* s_half = reinterpret_cast<float4*>(smem + 5120);
        const int e = threadIdx.x & 255, part = threadIdx.x >> 8;
        const int n = end - begin, n0 = (n + 1) >> 1;
        const bool on = e < n_heads * (kD / 2);
        const int h = e / (kD / 2), ch = 2 * (e - h * (kD / 2));
        float M = kNegInf, L = 0.f, acc0 = 0.f, acc1 = 0.f;
        if (on) {
          const int i0 = part ? n0 : 0, i1 = part ? n : n0;
          const float* col = p.partial + static_cast<size_t>(begin) * kPartialFloats + h * (kD + 2);
          // one pass in row order (rounds of independent loads; only the short rescaling chain is serial)
#pragma unroll 8
          for (int i = i0; i < i1; ++i) {
            const float* row = col + static_cast<size_t>(i) * kPartialFloats;
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(row));
            const float2 v = __ldcg(reinterpret_cast<const float2*>(row + 2 + ch));
            const float Mn = fmaxf(M, ml.x);
            const float a = (M == kNegInf) ? 0.f : exp2f(M - Mn), bwt = (ml.x == kNegInf) ? 0.f : exp2f(ml.x - Mn);
            L = fmaf(L, a, ml.y * bwt);
            acc0 = fmaf(acc0, a, v.x * bwt);
            acc1 = fmaf(acc1, a, v.y * bwt);
            M = Mn;
          }
          if (part) s_half[e] = make_float4(M, L, acc0, acc1);
        }
        __syncthreads();
        if (on && part == 0) {
          const float4 o2 = s_half[e];
          const float Mn = fmaxf(M, o2.x);
          const float a = (M == kNegInf) ? 0.f : exp2f(M - Mn), bwt = (o2.x == kNegInf) ? 0.f : exp2f(o2.x - Mn);
          L = fmaf(L, a, o2.y * bwt);
          acc0 = fmaf(acc0, a, o2.z * bwt);
          acc1 = fmaf(acc1, a, o2.w * bwt);
          M = Mn;
          const size_t hq = static_cast<size_t>(b) * p.n_kv_heads * p.group + static_cast<size_t>(kvh) * p.group + sid_head0 + h;
          *reinterpret_cast<float2*>(p.out + hq * kD + ch) = (L > 0.f) ? make_float2(acc0 / L, acc1 / L) : make_float2(0.f, 0.f);
          if (p.lse && ch == 0) p.lse[hq] = (L > 0.f) ? (M + log2f(L)) * 0.6931471805599453f : kNegInf;
          if constexpr (MASS) {
            if (ch == 0) p.lse2[hq] = (L > 0.f) ? M + log2f(L) : kNegInf;
          }
        }
      }
      __syncthreads();
    }
    gb = ge;
  }
}

}  // namespace

size_t decode_smem_bytes() {
  // per warp: pipeline stages, their mbarriers, and the bf16 query fragments (2 KiB)
  return static_cast<size_t>(kDecodeWarps) * (kStages * kStageBytes + kStages * sizeof(uint64_t) + 2 * 2048 + 2 * sizeof(int)) + 2 * sizeof(int);
}

cudaError_t launch_decode(const DecodeParams& p, int n_ctas, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    const int bytes = static_cast<int>(decode_smem_bytes());
    cudaError_t e = cudaFuncSetAttribute(decode_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(decode_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(decode_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  if (n_ctas <= 0) return cudaSuccess;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_ctas);
  cfg.blockDim = dim3(kDecodeWarps * 32);
  cfg.dynamicSmemBytes = decode_smem_bytes();
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (p.page_idx) return cudaLaunchKernelEx(&cfg, decode_kernel<true, false>, p);
  if (p.mass_raw) return cudaLaunchKernelEx(&cfg, decode_kernel<false, true>, p);
  return cudaLaunchKernelEx(&cfg, decode_kernel<false, false>, p);
}

namespace {
// One thread per (stream, item).  Residual rows are ascending in token index, so the rows of a
// block are one run found by bisection; everything is summed in a fixed order.
__global__ void mass_finish_kernel(const MassFinishParams p) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= p.n_streams * p.n_items) return;
  const int s = idx / p.n_items, b = idx - s * p.n_items;
  const float* lse2 = p.lse2 + static_cast<size_t>(s) * p.group;
  const float2* raw = p.mass_raw + (static_cast<size_t>(s) * p.mass_stride + b) * kMaxHeadsPerKv;
  float a = 0.f;
  for (int h = 0; h < p.group; ++h) {
    const float2 v = raw[h];
    if (v.y > 0.f && lse2[h] != -INFINITY) a += v.y * exp2f(v.x - lse2[h]);
  }
  const int n_res = p.res_count ? p.res_count[s] : 0;
  if (n_res > 0) {
    const int32_t* ri = p.res_idx + static_cast<size_t>(s) * p.res_cap;
    int lo = 0, hi = n_res;
    while (lo < hi) {                                  // first row with token >= 64 b
      const int mid = (lo + hi) >> 1;
      if (ri[mid] < b * kBlock) lo = mid + 1;
      else hi = mid;
    }
    for (int i = lo; i < n_res && ri[i] < (b + 1) * kBlock; ++i) {
      const float2* rr = p.res_raw + (static_cast<size_t>(s) * p.res_cap + i) * kMaxHeadsPerKv;
      for (int h = 0; h < p.group; ++h) {
        const float2 v = rr[h];
        if (v.y > 0.f && lse2[h] != -INFINITY) a += v.y * exp2f(v.x - lse2[h]);
      }
    }
  }
  a /= static_cast<float>(p.group);
  float* e = p.ema + static_cast<size_t>(s) * p.mass_stride + b;
  *e = fmaf(0.9f, *e, 0.1f * a);
  if (p.observed) p.observed[idx] = a;
}
}  // namespace

namespace {
// One CTA of 128 threads per query head.  Every sum is taken in a fixed order (a thread's items in
// ascending order, then a tree over the threads), so the certificate is reproducible bit for bit.
__global__ void __launch_bounds__(128) certificate_kernel(const CertificateParams p) {
  __shared__ float red[4][128];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int s = blockIdx.x / p.group, h = blockIdx.x - s * p.group;
  const int hq = s * p.group + h;
  // |q|
  const float qc = __uint_as_float(static_cast<uint32_t>(p.q[static_cast<size_t>(hq) * kD + tid]) << 16);
  red[0][tid] = qc * qc;
  __syncthreads();
  for (int w = 64; w > 0; w >>= 1) {
    if (tid < w) red[0][tid] += red[0][tid + w];
    __syncthreads();
  }
  const float qn = sqrtf(red[0][0]);
  __syncthreads();
  const float lse2 = p.lse2[hq];
  const int n_items = p.n_closed + (p.n_tail > 0 ? 1 : 0);
  float first = 0.f, mp = 0.f, mm = 0.f, vmax = 0.f;
  for (int b = tid; b < n_items; b += 128) {
    const float2 v = p.mass_raw[(static_cast<size_t>(s) * p.mass_stride + b) * kMaxHeadsPerKv + h];
    const float a = (v.y > 0.f && lse2 != -INFINITY) ? v.y * exp2f(v.x - lse2) : 0.f;
    if (b < p.n_closed) {
      const float4 e = p.err[static_cast<size_t>(s) * p.err_stride + b];
      const float eps = p.scale * qn * e.x;
      first = fmaf(a, e.y, first);
      mp = fmaf(a, expf(eps), mp);
      mm = fmaf(a, expf(-eps), mm);
      vmax = fmaxf(vmax, e.z);
    } else {                                    // the partial block is exact
      mp += a;
      mm += a;
    }
  }
  const int n_res = p.res_count ? p.res_count[s] : 0;
  for (int i = tid; i < n_res; i += 128) {      // residual rows are exact
    const float2 v = p.res_raw[(static_cast<size_t>(s) * p.res_cap + i) * kMaxHeadsPerKv + h];
    const float a = (v.y > 0.f && lse2 != -INFINITY) ? v.y * exp2f(v.x - lse2) : 0.f;
    mp += a;
    mm += a;
  }
  if (p.n_tail > 0) {                           // value rows of the partial block
    const TableEntry te = p.table[static_cast<size_t>(s) * p.table_stride + p.n_closed];
    const uint16_t* vrows = reinterpret_cast<const uint16_t*>(p.arena + static_cast<size_t>(te.off256) * 256) + kBlock * kD;
    for (int t = warp; t < p.n_tail; t += 4) {
      const uint2 raw = *reinterpret_cast<const uint2*>(vrows + t * kD + 4 * lane);
      const float x0 = __uint_as_float(raw.x << 16), x1 = __uint_as_float(raw.x & 0xffff0000u);
      const float x2 = __uint_as_float(raw.y << 16), x3 = __uint_as_float(raw.y & 0xffff0000u);
      float n2 = fmaf(x0, x0, fmaf(x1, x1, fmaf(x2, x2, x3 * x3)));
      for (int d = 1; d <= 16; d <<= 1) n2 += __shfl_xor_sync(kFull, n2, d);
      vmax = fmaxf(vmax, sqrtf(n2));
    }
  }
  red[0][tid] = first;
  red[1][tid] = mp;
  red[2][tid] = mm;
  red[3][tid] = vmax;
  __syncthreads();
  for (int w = 64; w > 0; w >>= 1) {
    if (tid < w) {
      red[0][tid] += red[0][tid + w];
      red[1][tid] += red[1][tid + w];
      red[2][tid] += red[2][tid + w];
      red[3][tid] = fmaxf(red[3][tid], red[3][tid + w]);
    }
    __syncthreads();
  }
  if (tid == 0) {
    const float Mp = red[1][0], Mm = red[2][0];
    float second = 0.f;
    if (Mm > 0.f && Mp > 0.f) second = fminf(2.f, fmaxf(0.f, Mp / Mm - Mm / Mp));
    p.out[hq] = red[0][0] + second * red[3][0];
  }
}
}  // namespace

cudaError_t launch_certificate(const CertificateParams& p, cudaStream_t st) {
  const int n = p.n_streams * p.group;
  if (n <= 0) return cudaSuccess;
  certificate_kernel<<<n, 128, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_mass_finish(const MassFinishParams& p, cudaStream_t st) {
  const int n = p.n_streams * p.n_items;
  if (n <= 0) return cudaSuccess;
  mass_finish_kernel<<<(n + 255) / 256, 256, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace gkv
