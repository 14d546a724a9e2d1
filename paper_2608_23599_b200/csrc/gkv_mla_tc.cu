// Decode attention for latent-attention (MLA) streams on the 5th-generation tensor cores
// (Sec. 3.1 read path applied to a 576-wide latent row that is key and value at once).
//
// A quantised latent row is k~[c] = s[c] * code[c] + z[c] with one (s, z) pair per channel and
// half block (32 tokens, Sec. 3.2).  fp16 operands hold 11 bits, too few for k~ itself, for the
// query times a scale and for the probabilities, so nothing rounded ever becomes an operand:
//   * the tile holds the integers code - mid (exact in fp16); exact and centroid rows are bf16 values
//     (exact in fp16) with s = 1, z = 0;
//   * the scales go into the query: Q'[half][head][c] = q[head][c] * s[half][c] as an fp16 pair
//     hi + lo, so S[64 tokens x (2 halves x (hi | lo) x 16 heads)] = T Q'^T in one MMA chain and a
//     token takes the 32 columns of its own half; sum_c q[c] (z[c] + mid s[c]) is added per (half, head);
//   * O^T[512 x 16] += V~^T P^T runs per half block on the same tile (read MN-major) with P as an
//     fp16 pair hi + lo (N = 32), into a per-half accumulator in tensor memory; four warps read it out,
//     apply s[c] and z[c] in fp32 and add it to the running O^T (also in tensor memory), together with
//     the rescaling of the online softmax.
// One CTA per SM walks a contiguous range of one stream's blocks.  Nine warps convert packed
// blocks (read straight from global memory, prefetched into L2 by a helper warp) into the
// 128-byte-swizzled tile [9 panels of 64 channels][64 tokens][128 B] and prepare Q'; one warp
// issues tcgen05.mma; four warps run the softmax and the read-out.  Tiles are double-buffered.
// Every wait is bounded; on a time-out the CTA raises kStatusInternal and publishes an empty
// partial.  Partials of the CTAs of a stream are merged by mla_combine_kernel in CTA order.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <type_traits>

#include "gkv_internal.h"
#include "gkv_layout.cuh"
#include "gkv_mla.h"

namespace gkv {
namespace {

constexpr int kTcConvertWarps = 9;                     // 288 threads = 72 chunks x 4 token groups
constexpr int kTcFirstConvertWarp = 8;                 // warps 0-3: softmax + read-out, warps 4-7: read-out
constexpr int kTcMmaWarp = 17;
constexpr int kTcThreads = 18 * 32;
constexpr int kTcReadTiles0 = 0;                       // channel tiles (of 128) read out by warps 0-3 beside the softmax; warps 4-7 take the rest
constexpr int kTcPanelBytes = 64 * 128;                // 64 rows x 64 channels fp16
constexpr int kTcTileBytes = 9 * kTcPanelBytes;        // 73728: 64 rows x 576 channels
constexpr int kTcPBytes = 2 * 64 * 32;                 // P: hi block and lo block, each 64 tokens x 16 heads fp16
// shared-memory map (offsets from a 1024-byte aligned base)
constexpr int kOffTile = 0;
constexpr int kOffQp = 2 * kTcTileBytes;               // 147456: Q' of one block, laid out like a tile (row = column of S)
constexpr int kOffP = kOffQp + kTcTileBytes;           // 221184
constexpr int kOffMisc = kOffP + kTcPBytes;            // 225280
#ifdef GKV_MLA_PROF
constexpr int kTcSmem = kOffMisc + 5120 + 1024 + 128;
#else
constexpr int kTcSmem = kOffMisc + 5120 + 1024;        // + misc + alignment slack = 231424
#endif
// misc: mbarriers (128 B) | tmem base @128 | abort flag @132 | bias[2][64] floats @256 |
//       head maxima [2][4 warps][16] @768 | row sums [4][16] @1280 | key constants [2 tiles][2 halves][16] @1536 |
//       probability sums per warp [2 tiles][4][16] @1792 | parts of the key constants [2][2][9 warps][16] @2304 |
//       rescale factors [2][16] + flag [2] @4608
constexpr int kMiscTmem = 128, kMiscAbort = 132, kMiscBias = 256, kMiscMax = 768, kMiscSum = 1280;
constexpr int kMiscConst = 1536;                       // [2][2][16] floats = 256 B
constexpr int kMiscHalfSum = 1792;                     // [2 tiles][4 warps][16] floats = 512 B: probability sums per warp
constexpr int kMiscConstPart = 2304;                   // [2][2][9][16] floats = 2304 B, ends at 4608
constexpr int kMiscAlpha = 4608;                       // [2][16] floats, then [2] ints (1 = rescale): ends at 4744
constexpr int kMiscHalfSum2 = 4864;                    // [2 tiles][2 halves][16] floats = 256 B: sums per half block
enum { kBarKtFull = 0, kBarQpFull = 2, kBarSFull = 4, kBarPFull = 6, kBarPvDone = 7, kBarRFree = 9, kBarHsFull = 10 };
constexpr int kTcWaitSpins = 1 << 20;
constexpr float kNegInfT = -INFINITY;
constexpr uint32_t kFullT = 0xffffffffu;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemS = 0;                         // S[2]: 64 columns each
constexpr uint32_t kTmemR = 128;                       // per-half accumulators: [2 halves][4 channel tiles][32 columns]
constexpr uint32_t kTmemO = 384;                       // running O^T: [4 channel tiles][16 heads]
constexpr int kPrefetchAhead = 6;                      // tiles the L2 prefetch runs ahead of the key MMAs
constexpr float kRescaleSlack = 8.f;                   // keep a stale running max while logits stay within 2^8 of it

#ifdef GKV_MLA_PROF
// development aid: cycles per role and phase, kept in shared memory by one lane per role
__device__ unsigned long long g_prof[148 * 32];
#define PROF_DECL(basei) uint32_t* const pbase = prof_sm + (basei); uint32_t pt0 = clock()
#define PROF_LAP(i) do { const uint32_t pt1 = clock(); if (prof_lane) pbase[i] += pt1 - pt0; pt0 = pt1; } while (0)
#else
#define PROF_DECL(basei)
#define PROF_LAP(i)
#endif

__device__ __forceinline__ uint32_t t_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void t_bar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void t_fence_async() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void t_bar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool t_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(200)
      : "memory");
  return ok != 0;
}
// Bounded wait; a time-out raises the CTA's abort flag, which every other waiter also watches.  A
// waiting thread backs off between polls: the polls of eighteen warps otherwise take a third of the
// SM's issue slots from the warps that work.
__device__ __forceinline__ bool t_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  int spins = 0;
  while (!t_try_wait(bar, parity)) {
    __nanosleep(spins < 4 ? 64 : 256);
    if (++spins > kTcWaitSpins || *abort_flag) {
      *abort_flag = 1;
      return false;
    }
  }
  return true;
}
// Wait of a whole warp role (n threads on named barrier `id`): the role's first warp polls the
// mbarrier, the others block on the named barrier and spend no issue slots; the outcome (false after a
// time-out or an abort) reaches every thread through the barrier's reduction, so the role leaves its
// loop as one.
__device__ __forceinline__ bool t_role_sync(int id, int n, bool ok_in) {
  const uint32_t ok = ok_in ? 1u : 0u;
  uint32_t all;
  asm volatile(
      "{\n"
      ".reg .pred pi, po;\n"
      "setp.ne.u32 pi, %1, 0;\n"
      "bar.red.and.pred po, %2, %3, pi;\n"
      "selp.u32 %0, 1, 0, po;\n"
      "}\n"
      : "=r"(all)
      : "r"(ok), "r"(id), "r"(n)
      : "memory");
  return all != 0;
}
__device__ __forceinline__ bool t_wait_role(bool leader, uint32_t bar, uint32_t parity, int id, int n, volatile int* abort_flag) {
  bool ok = true;
  if (leader) ok = t_wait(bar, parity, abort_flag);
  return t_role_sync(id, n, ok);
}
__device__ __forceinline__ void t_sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ uint32_t t_prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;\n" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}
__device__ __forceinline__ __half2 t_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }
__device__ __forceinline__ uint32_t t_u(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ float t_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// ---- tensor memory and tcgen05 -----------------------------------------------------------------
__device__ __forceinline__ void t_tmem_alloc(uint32_t smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_dst), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void t_tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void t_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void t_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
// Issued by a whole (converged) warp; one elected lane executes the instruction, so the operands
// stay warp-uniform and the loop around it runs on the uniform datapath.
__device__ __forceinline__ void t_mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p, e;\n"
      "elect.sync _|e, 0xffffffff;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "@e tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// legacy warp-level MMA (m16n8k16, fp16 operands, fp32 accumulators) for the small key-constant products
__device__ __forceinline__ void t_mma_sync_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void t_commit(uint32_t bar) {
  asm volatile(
      "{\n"
      ".reg .pred e;\n"
      "elect.sync _|e, 0xffffffff;\n"
      "@e tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n"
      "}\n" ::"r"(bar)
      : "memory");
}
__device__ __forceinline__ void t_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// the same without the wait: several loads may be in flight; t_wait_ld() before the first use
__device__ __forceinline__ void t_ld16_async(uint32_t taddr, float (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
      : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]), "=f"(v[8]),
        "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15])
      : "r"(taddr));
}
__device__ __forceinline__ void t_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void t_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};\n" ::"r"(taddr),
      "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
      "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
      "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
      "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
}

// Shared-memory matrix descriptor (Blackwell version bit set), 128-byte swizzle unless told otherwise.
// Strides in bytes.
__device__ __forceinline__ uint64_t t_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint64_t layout = 2) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr >> 4) & 0x3fffu);
  d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3fffu) << 32;
  d |= 1ull << 46;                 // descriptor version
  d |= layout << 61;               // 2 = SWIZZLE_128B, 6 = SWIZZLE_32B
  return d;
}
// Instruction descriptor for kind::f16 with fp16 operands and an fp32 accumulator.
__host__ __device__ constexpr uint32_t t_idesc(int m, int n, bool a_mn_major, bool b_mn_major = false) {
  return (1u << 4) | (static_cast<uint32_t>(a_mn_major) << 15) | (static_cast<uint32_t>(b_mn_major) << 16) |
         (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(m >> 4) << 24);
}

// ---- tiles -------------------------------------------------------------------------------------
// (tc_next is called by whole, converged warps: the centroid run is found with warp ballots.)
// A tile is up to 64 rows of the score matrix: one quantised block, one exact block (or the tail),
// or up to 64 neighbouring centroid blocks (one row each, weighted by log2(64) on the logit).
struct TcTile {
  int kind;        // 0 quantised, 1 exact rows, 2 centroid rows
  int level;       // 8 / 4 for kind 0
  int item, adv;   // first block and number of blocks covered
  int nrows;       // valid rows
  int nstages;     // raw stages: 2 halves (kind 0) or groups of 16 rows
  uint32_t off256;
};

// `e` is the caller's copy of table[it] (it fetches the next one while a tile is being worked on).
__device__ __forceinline__ bool tc_next(const MlaDecodeParams& p, const TableEntry* table, int item_end, int it, const TableEntry e,
                                     TcTile& t) {
  if (it >= item_end) return false;
  t.item = it;
  t.adv = 1;
  t.off256 = e.off256;
  t.level = static_cast<int>(e.level);
  if (it == p.n_closed) {                 // the tail: exact rows, the last item of the stream
    if (p.n_tail == 0) return false;
    t.kind = 1;
    t.nrows = p.n_tail;
    t.nstages = (t.nrows + 15) >> 4;
    return true;
  }
  if (t.level == 16) {
    t.kind = 1;
    t.nrows = kBlock;
    t.nstages = 4;
  } else if (t.level == 1) {
    // length of the run of centroid blocks, up to 64: two look-ups per lane, then ballots
    const int lim = min(min(item_end, p.n_closed) - it, 64);
    const int ln = static_cast<int>(threadIdx.x & 31);
    const bool c0 = ln < lim && table[it + ln].level == 1u;
    const bool c1 = ln + 32 < lim && table[it + 32 + ln].level == 1u;
    const uint32_t b0 = __ballot_sync(0xffffffffu, c0), b1 = __ballot_sync(0xffffffffu, c1);
    int run = __ffs(~b0) - 1;                   // first lane that is not a centroid block (-1: none)
    if (run < 0) {
      run = 32 + __ffs(~b1) - 1;
      if (__ffs(~b1) == 0) run = 64;
    }
    t.kind = 2;
    t.adv = run;
    t.nrows = run;
    t.nstages = (run + 15) >> 4;
  } else {
    t.kind = 0;
    t.nrows = kBlock;
    t.nstages = 2;
  }
  return true;
}

// table[it] for the iterator, clamped to the stream's last entry (the tail)
__device__ __forceinline__ TableEntry tc_entry(const MlaDecodeParams& p, const TableEntry* table, int it) {
  return table[min(it, p.n_closed)];
}

// address of the 16-byte piece (row, chunk j of 8 channels) inside a swizzled tile
__device__ __forceinline__ uint32_t tc_tile_addr(uint32_t tile, int row, int j) {
  return tile + (j >> 3) * kTcPanelBytes + row * 128 + ((((j & 7) ^ (row & 7))) << 4);
}
__device__ __forceinline__ uint32_t tc_bf2_to_h2(uint32_t u) {
  return t_u(__floats2half2_rn(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u)));
}
// Streaming loads bypass L1: what little of it the shared-memory carve-out leaves is kept for the
// threads' stack slots.
__device__ __forceinline__ uint4 t_ldg128(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint2 t_ldg64(const void* p) {
  uint2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t t_ldg32(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];\n" : "=r"(v) : "l"(p));
  return v;
}

// A code in the mantissa of an fp16 with a zero exponent field is the number code * 2^(b - 24), b the
// code's lowest bit: no bias to take out again.  8-bit codes sit at b = 0; 4-bit codes at b = 0
// (channels with (c & 2) == 0) or b = 4.  The logits of a quantised tile therefore come out of the
// tensor cores scaled by 2^-24 (8 bits) or 2^-20 (4 bits, whose b = 0 channels get 16 s in Q'), and a
// value channel by 2^(b - 24).
__device__ __forceinline__ float tc_logit_scale(const int kind, const int level) {
  return kind != 0 ? 1.f : (level == 8 ? 16777216.f : 1048576.f);
}

// A quantised block -> the tile as the codes themselves (scaled by a power of two).  Thread = (chunk j of 8 channels, 8
// tokens of each half); the packed codes come straight from global memory (a token's chunk is 8
// bytes at 8 bits, 4 bytes at 4 bits).  The loads are issued a tile ahead (tc_load_half).
__device__ __forceinline__ void tc_load_half(const uint8_t* slot, int bits, int half, int j, int tg, uint2 (&w)[8]) {
  const int row = kMlaChunks * bits;
  const uint8_t* codes = slot + static_cast<size_t>(half) * mla_half_bytes(bits) + mla_kp_bytes() + static_cast<size_t>(8 * tg) * row + j * bits;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    if (bits == 8) w[i] = t_ldg64(codes + i * row);
    else w[i] = make_uint2(t_ldg32(codes + i * row), 0u);
  }
}
template <int BITS>
__device__ __forceinline__ void tc_store_block(const uint2 (&w)[2][8], uint32_t tile, int j, int tg) {
  const uint32_t jx = (j & 7) << 4;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const uint32_t out = tile + (j >> 3) * kTcPanelBytes + (32 * half + 8 * tg) * 128;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      uint32_t x0, x1, x2, x3;
      if constexpr (BITS == 4) {
        const uint32_t v = w[half][i].x >> 8;
        x0 = w[half][i].x & 0x000F000Fu;      // channels 0, 1: b = 0
        x1 = w[half][i].x & 0x00F000F0u;      // channels 2, 3: b = 4
        x2 = v & 0x000F000Fu;
        x3 = v & 0x00F000F0u;
      } else {
        x0 = t_prmt(w[half][i].x, 0u, 0x4240u);
        x1 = t_prmt(w[half][i].x, 0u, 0x4341u);
        x2 = t_prmt(w[half][i].y, 0u, 0x4240u);
        x3 = t_prmt(w[half][i].y, 0u, 0x4341u);
      }
      // rows 32 half + 8 tg + i: row & 7 = i, so the swizzled 16-byte slot is (j & 7) ^ i
      t_sts128(out + i * 128 + (jx ^ (i << 4)), x0, x1, x2, x3);
    }
  }
}

// bf16 rows -> fp16 rows of the tile (exact for the magnitudes a cache holds).  Thread = (chunk j, rows
// 16 rg .. 16 rg + 15); rows >= n become zeros.  CENTROID: row r is the centroid row of block item + r.
template <bool CENTROID>
__device__ __forceinline__ void tc_convert_rows(const MlaDecodeParams& p, const TableEntry* table, const TcTile& t, uint32_t tile, int j,
                                                int rg) {
  const uint8_t* slot = p.arena + static_cast<size_t>(t.off256) * 256;
#pragma unroll 4
  for (int i = 0; i < 16; ++i) {
    const int r = 16 * rg + i;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r < t.nrows) {
      const uint8_t* row = CENTROID ? p.arena + static_cast<size_t>(table[t.item + r].off256) * 256 : slot + static_cast<size_t>(r) * kMlaRowBytes;
      v = t_ldg128(row + j * 16);
      v.x = tc_bf2_to_h2(v.x);
      v.y = tc_bf2_to_h2(v.y);
      v.z = tc_bf2_to_h2(v.z);
      v.w = tc_bf2_to_h2(v.w);
    }
    t_sts128(tc_tile_addr(tile, r, j), v.x, v.y, v.z, v.w);
  }
}

// ---- kernel ------------------------------------------------------------------------------------
// Warp roles: 0-3 softmax + read-out of the first channel tile, 4-7 read-out of the other three
// (warp w owns tensor-memory lanes 32 (w % 4) .. + 31), 8-16 conversion and Q', 17 tensor-core issue.

// Read-out of the accumulators of tile `pt` (number pn) for the channel tiles [i0, i1): O^T *= alpha
// when this tile moved the running max (O^T holds the tiles before it), then per half block
// O^T <- O^T + s[c] R[c] + z'[c] sum_t p.  A thread owns channel 128 i + lt of every channel tile i (its
// tensor-memory lane lt).  hs = [2 halves][16 heads] sums of the tile's probabilities.
__device__ __forceinline__ bool tc_read_out(const MlaDecodeParams& p, const TcTile& pt, int pn, int i0, int i1, bool scale,
                                            const float* alpha_sm, const float* hs, uint32_t tlane, int lt, uint32_t bar_pv,
                                            bool leader, int role_bar, volatile int* abort_flag
#ifdef GKV_MLA_PROF
                                            , uint32_t* prof_sm
#endif
) {
  // scale and zero point of this thread's channels in both halves (asked for before the wait)
  const float unscale = (pt.level == 4 && (lt & 2)) ? 1048576.f : 16777216.f;      // 2^(24 - b) of the thread's channels
  const uint8_t* slot = p.arena + static_cast<size_t>(pt.off256) * 256;
  __half sch[4][2], zph[4][2];
  if (pt.kind == 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (i < i0 || i >= i1) continue;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const __half* prm = reinterpret_cast<const __half*>(slot + static_cast<size_t>(hf) * mla_half_bytes(pt.level));
        sch[i][hf] = __ldg(prm + 128 * i + lt);
        zph[i][hf] = __ldg(prm + kMlaZeroOff + 128 * i + lt);
      }
    }
  }
#ifdef GKV_MLA_PROF
  const uint32_t rw0 = clock();
#endif
  const bool ok = t_wait_role(leader, bar_pv, (pn >> 1) & 1, role_bar, 128, abort_flag);
#ifdef GKV_MLA_PROF
  if (threadIdx.x == 128) prof_sm[20] += clock() - rw0;
#endif
  t_fence_after();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (i < i0 || i >= i1) continue;
    float o[16], r[16], rl[16];
    if (pn > 0) {
      t_ld16_async(tlane + kTmemO + 16 * i, o);
    } else {
#pragma unroll
      for (int h = 0; h < 16; ++h) o[h] = 0.f;
    }
    t_ld16_async(tlane + kTmemR + 32 * i, r);
    t_ld16_async(tlane + kTmemR + 32 * i + 16, rl);
    t_wait_ld();
    if (scale) {
#pragma unroll
      for (int h4 = 0; h4 < 4; ++h4) {
        const float4 a = reinterpret_cast<const float4*>(alpha_sm)[h4];
        o[4 * h4] *= a.x;
        o[4 * h4 + 1] *= a.y;
        o[4 * h4 + 2] *= a.z;
        o[4 * h4 + 3] *= a.w;
      }
    }
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      float sc = 1.f, zp = 0.f;
      if (pt.kind == 0) {
        sc = __half2float(sch[i][hf]) * unscale;
        zp = __half2float(zph[i][hf]);
      }
#pragma unroll
      for (int h4 = 0; h4 < 4; ++h4) {
        const float4 w = reinterpret_cast<const float4*>(hs)[hf * 4 + h4];
        o[4 * h4] = fmaf(sc, r[4 * h4] + rl[4 * h4], fmaf(zp, w.x, o[4 * h4]));
        o[4 * h4 + 1] = fmaf(sc, r[4 * h4 + 1] + rl[4 * h4 + 1], fmaf(zp, w.y, o[4 * h4 + 1]));
        o[4 * h4 + 2] = fmaf(sc, r[4 * h4 + 2] + rl[4 * h4 + 2], fmaf(zp, w.z, o[4 * h4 + 2]));
        o[4 * h4 + 3] = fmaf(sc, r[4 * h4 + 3] + rl[4 * h4 + 3], fmaf(zp, w.w, o[4 * h4 + 3]));
      }
      if (hf == 0) {                                    // the second half's accumulators
        t_ld16_async(tlane + kTmemR + 128 + 32 * i, r);
        t_ld16_async(tlane + kTmemR + 128 + 32 * i + 16, rl);
        t_wait_ld();
      }
    }
    t_st16(tlane + kTmemO + 16 * i, o);
  }
  t_fence_before();
  return ok;
}

__global__ void __launch_bounds__(kTcThreads, 1) mla_tc_decode_kernel(const __grid_constant__ MlaDecodeParams p) {
  extern __shared__ uint8_t tsm_raw[];
  const WarpDesc cd = p.ctas[blockIdx.x];
  if (cd.stream < 0) return;                               // uniform for the CTA
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const uint32_t base = (t_u32(tsm_raw) + 1023u) & ~1023u;
  uint8_t* gbase = tsm_raw + (base - t_u32(tsm_raw));
  const uint32_t misc = base + kOffMisc;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + kOffMisc + kMiscAbort);
  float* bias_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscBias);            // [2][64]
  float* max_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscMax);              // [2][4][16]
  float* sum_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscSum);              // [4][16]
  float* const_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscConst);          // [2][2][16]
  float* hsum_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscHalfSum);         // [2][4][16]
  float* cpart_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscConstPart);      // [2][2][9][16]
  float* alpha_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscAlpha);          // [2][16]
  float* hsum2_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscHalfSum2);       // [2][2][16]
  volatile int* need_sm = reinterpret_cast<volatile int*>(gbase + kOffMisc + kMiscAlpha + 128);   // [2]
#ifdef GKV_MLA_PROF
  uint32_t* prof_sm = reinterpret_cast<uint32_t*>(gbase + kOffMisc + 5120);
  const bool prof_lane = (lane == 0) && (warp == 0 || warp == 4 || warp == kTcFirstConvertWarp || warp == kTcMmaWarp);
  if (tid < 32) prof_sm[tid] = 0;
#endif
  const TableEntry* table = p.table + static_cast<size_t>(cd.stream) * p.table_stride;
  auto bar = [&](int which, int i) { return misc + 8u * static_cast<uint32_t>(which + i); };

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      t_bar_init(bar(kBarKtFull, i), kTcConvertWarps);
      t_bar_init(bar(kBarSFull, i), 1);
      t_bar_init(bar(kBarQpFull, i), kTcConvertWarps);
      t_bar_init(bar(kBarPvDone, i), 1);
      t_bar_init(bar(kBarHsFull, i), 4);
    }
    t_bar_init(bar(kBarPFull, 0), 4);
    t_bar_init(bar(kBarRFree, 0), kTcReadTiles0 > 0 ? 8 : 4);
    *abort_flag = 0;
    t_fence_async();
  }
  if (warp == 0) t_tmem_alloc(misc + kMiscTmem, kTmemCols);
  t_fence_before();
  __syncthreads();
  t_fence_after();
  const uint32_t tmem = __shfl_sync(kFullT, *reinterpret_cast<volatile uint32_t*>(gbase + kOffMisc + kMiscTmem), 0);
  const uint16_t* qg = p.q + static_cast<size_t>(cd.stream) * kMlaHeads * kMlaDk;

  if (warp == kTcMmaWarp) {
    // ---------------- tensor-core issue (whole warp, one elected lane per instruction) ----------------
    constexpr uint32_t kIdQK = t_idesc(64, 64, false), kIdPV = t_idesc(128, 32, true, true);
    // descriptors differ only in the start-address field (16-byte units in the low word)
    const uint64_t dq = t_desc(base + kOffQp, 16, 1024);
    // P: hi block | lo block, each [64 tokens][16 heads] fp16 with the heads contiguous (MN-major),
    // 32-byte swizzle, 8-token groups of 256 B; the lo block is the second 16 columns (2048 B further)
    const uint64_t dp = t_desc(base + kOffP, 2048, 256, 6);
    auto issue_qk = [&](int tg) {
      const int b = tg & 1;
      const uint64_t da = t_desc(base + kOffTile + b * kTcTileBytes, 16, 1024);
      const uint32_t d = tmem + kTmemS + 64 * b;
      // (the loops stay rolled: the issue warp's code competes with the working warps for the instruction cache)
#pragma unroll 1
      for (int pn = 0; pn < 9; ++pn) {
        const uint32_t o16 = static_cast<uint32_t>(pn * kTcPanelBytes) >> 4;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) t_mma_f16(d, da + o16 + 2 * kk, dq + o16 + 2 * kk, kIdQK, (pn | kk) != 0);
      }
      t_commit(bar(kBarSFull, b));
    };
    auto issue_pv = [&](int tg) {
      const int b = tg & 1;
      const uint64_t da = t_desc(base + kOffTile + b * kTcTileBytes, kTcPanelBytes, 1024);
#pragma unroll 1
      for (int hi = 0; hi < 8; ++hi) {
        const int half = hi >> 2, i = hi & 3;
        const uint32_t oa = static_cast<uint32_t>(2 * i * kTcPanelBytes + 2 * half * 2048) >> 4, ob = static_cast<uint32_t>(2 * half * 512) >> 4;
        const uint32_t d = tmem + kTmemR + 128 * half + 32 * i;
        t_mma_f16(d, da + oa, dp + ob, kIdPV, 0);
        t_mma_f16(d, da + oa + (2048 >> 4), dp + ob + (512 >> 4), kIdPV, 1);
      }
      t_commit(bar(kBarPvDone, b));
    };
    // packed bytes of a tile that is about to be converted: ask for them in L2
    auto prefetch = [&](const TcTile& t) {
      if (t.kind != 2 && lane == 0) {
        const uint8_t* slot = p.arena + static_cast<size_t>(t.off256) * 256;
        const uint32_t bytes = t.kind == 0 ? 2u * static_cast<uint32_t>(mla_half_bytes(t.level)) : static_cast<uint32_t>(t.nrows) * kMlaRowBytes;
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(slot), "r"(bytes) : "memory");
      }
    };
    // Event-driven order: the value MMAs of tile pv go out as soon as its P is there (and the
    // accumulators of tile pv - 1 have been read out), the key MMAs of tile qk as soon as its tile and
    // its Q' are there (qk runs at most two tiles ahead of pv: S and the tile buffers are double).
    TcTile t;
    int it = cd.item_begin;
    TableEntry pre = tc_entry(p, table, it);
    bool more_tiles = tc_next(p, table, cd.item_end, it, pre, t);
    pre = tc_entry(p, table, t.item + t.adv);
    int qk = 0, pv = 0, n_known = more_tiles ? 1 : 0;      // tiles [0, n_known) exist so far
    // a second walk over the tiles runs kPrefetchAhead tiles in front and asks for their bytes in L2
    TcTile tp;
    int itp = cd.item_begin;
    TableEntry prep = tc_entry(p, table, itp);
    bool more_pf = true;
    auto prefetch_step = [&]() {
      if (!more_pf) return;
      more_pf = tc_next(p, table, cd.item_end, itp, prep, tp);
      if (more_pf) {
        prefetch(tp);
        itp = tp.item + tp.adv;
        prep = tc_entry(p, table, itp);
      }
    };
#pragma unroll 1
    for (int i = 0; i < kPrefetchAhead; ++i) prefetch_step();
    bool ok = true;
    int spins = 0;
    PROF_DECL(24);
    while (ok && (pv < n_known || more_tiles)) {
      bool progress = false;
      if (qk < n_known && qk < pv + 2) {
        const bool ready = __all_sync(kFullT, t_try_wait(bar(kBarKtFull, qk & 1), (qk >> 1) & 1) && t_try_wait(bar(kBarQpFull, qk & 1), (qk >> 1) & 1));
        if (ready) {
          t_fence_after();
          PROF_LAP(0);
          issue_qk(qk);
          PROF_LAP(1);
          ++qk;
          it = t.item + t.adv;
          more_tiles = tc_next(p, table, cd.item_end, it, pre, t);
          if (more_tiles) {
            ++n_known;
            pre = tc_entry(p, table, t.item + t.adv);
          }
          prefetch_step();
          progress = true;
        }
      }
      if (pv < qk) {
        const bool ready = __all_sync(kFullT, t_try_wait(bar(kBarPFull, 0), pv & 1) && (pv == 0 || t_try_wait(bar(kBarRFree, 0), (pv - 1) & 1)));
        if (ready) {
          t_fence_after();
          PROF_LAP(0);
          issue_pv(pv);
          PROF_LAP(2);
          ++pv;
          progress = true;
        }
      }
      if (progress) {
        spins = 0;
      } else {
        __nanosleep(128);
        if (++spins > kTcWaitSpins || *abort_flag) {
          *abort_flag = 1;
          ok = false;
        }
      }
      ok = __all_sync(kFullT, ok);
    }
  } else if (warp >= kTcFirstConvertWarp) {
    // ---------------- conversion of blocks into tiles, and Q' ----------------
    const int dt = tid - kTcFirstConvertWarp * 32;          // 0 .. 287
    const int dj = dt % kMlaChunks, dg = dt / kMlaChunks;   // tile conversion: chunk of 8 channels, token group
    // Q' and the key constants: warp cw owns the panel of 64 channels cw; lane (n, c4) = (lane / 4, lane % 4)
    // holds the heads n and n + 8 on the 16 channels 64 cw + 16 c4 .. + 15 (chunks qj0 and qj0 + 1) as fp16
    // pairs.  That is at once the B-fragment layout of mma.m16n8k16 for a contraction over the panel's
    // channels taken in the order "k-step ks, index k = 2 c4 + e (+ 8)  <->  channel 16 c4 + 4 ks + e (+ 2)":
    // the key constants sum_c q[c] z[c] come from eight legacy MMAs per warp (A rows 0, 1 = the zero points of
    // the two half blocks), and the same registers times the scales give the Q' rows.
    const int cw = warp - kTcFirstConvertWarp;
    const int qn = lane >> 2, qc4 = lane & 3;
    const int qj0 = 8 * cw + 2 * qc4;
    uint32_t qf[2][8];                                      // [head n + 8 t][channel pair i of the lane's 16 channels]
#pragma unroll
    for (int tq = 0; tq < 2; ++tq) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const uint4 v = t_ldg128(qg + (qn + 8 * tq) * kMlaDk + 8 * (qj0 + e));
        qf[tq][4 * e + 0] = tc_bf2_to_h2(v.x);
        qf[tq][4 * e + 1] = tc_bf2_to_h2(v.y);
        qf[tq][4 * e + 2] = tc_bf2_to_h2(v.z);
        qf[tq][4 * e + 3] = tc_bf2_to_h2(v.w);
      }
    }
    // The packed codes of a tile's quantised block (w) and the scales and zero points of the
    // thread's Q' chunk (svh, zvh) are asked for one tile ahead: the codes of the next tile as soon as
    // this tile is stored, its parameters once this tile's Q' is written.
    TcTile t, tn;
    int tg = 0;
    bool ok = true;
    uint2 w[2][8];
    uint4 svh[2][2], zvh[2];        // scales [half][chunk of the lane]; zero points of half (n & 1), both chunks
    auto load_params = [&](const TcTile& x) {
      const uint8_t* slot = p.arena + static_cast<size_t>(x.off256) * 256;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const uint8_t* prm = slot + static_cast<size_t>(half) * mla_half_bytes(x.level);
        svh[half][0] = t_ldg128(prm + 16 * qj0);
        svh[half][1] = t_ldg128(prm + 16 * qj0 + 16);
      }
      const uint8_t* zp = slot + static_cast<size_t>(qn & 1) * mla_half_bytes(x.level) + 2 * kMlaZeroOff + 16 * qj0;
      zvh[0] = t_ldg128(zp);
      zvh[1] = t_ldg128(zp + 16);
    };
    TableEntry pre = tc_entry(p, table, cd.item_begin);
    bool have = tc_next(p, table, cd.item_end, cd.item_begin, pre, t);
    if (have && t.kind == 0) {
      tc_load_half(p.arena + static_cast<size_t>(t.off256) * 256, t.level, 0, dj, dg, w[0]);
      tc_load_half(p.arena + static_cast<size_t>(t.off256) * 256, t.level, 1, dj, dg, w[1]);
      load_params(t);
    }
    if (have) pre = tc_entry(p, table, t.item + t.adv);
    PROF_DECL(0);
    while (ok && have) {
      const int b = tg & 1;
      const uint32_t tile = base + kOffTile + b * kTcTileBytes;
      const bool have_n = tc_next(p, table, cd.item_end, t.item + t.adv, pre, tn);
      if (have_n) pre = tc_entry(p, table, tn.item + tn.adv);
      PROF_LAP(0);
      // the tile buffer is free once the value MMAs of tile tg - 2 are done
      if (tg >= 2) ok = t_wait_role(cw == 0, bar(kBarPvDone, b), ((tg - 2) >> 1) & 1, 2, kTcConvertWarps * 32, abort_flag);
      if (!ok) break;
      PROF_LAP(1);
      if (dt < 64) bias_sm[b * 64 + dt] = dt < t.nrows ? (t.kind == 2 ? 6.0f : 0.f) : kNegInfT;   // log2(64) per centroid row
      if (t.kind == 0) {
        if (t.level == 8) tc_store_block<8>(w, tile, dj, dg);
        else tc_store_block<4>(w, tile, dj, dg);
      } else if (t.kind == 1) {
        tc_convert_rows<false>(p, table, t, tile, dj, dg);
      } else {
        tc_convert_rows<true>(p, table, t, tile, dj, dg);
      }
      PROF_LAP(2);
      t_fence_async();
      __syncwarp();
      if (lane == 0) t_bar_arrive(bar(kBarKtFull, b));
      PROF_LAP(3);
      // Key constants sum_c q[c] z[c] per (half, head) over the warp's panel: D[half][head] = Z Q^T on the
      // legacy tensor-core path (products of two fp16 numbers are exact, the sums are fp32).  Row r of A is
      // the zero-point row of half r & 1 (only rows 0 and 1 are read back), so the lanes 0-3 end up with
      // half 0 and the lanes 4-7 with half 1, heads 2 c4, 2 c4 + 1 (+ 8).  Formed before the wait for the
      // Q' buffer.
      {
        float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
        if (t.kind == 0) {
          const uint32_t zr[8] = {zvh[0].x, zvh[0].y, zvh[0].z, zvh[0].w, zvh[1].x, zvh[1].y, zvh[1].z, zvh[1].w};
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            t_mma_sync_f16(c0, zr[2 * ks], zr[2 * ks], zr[2 * ks + 1], zr[2 * ks + 1], qf[0][2 * ks], qf[0][2 * ks + 1]);
            t_mma_sync_f16(c1, zr[2 * ks], zr[2 * ks], zr[2 * ks + 1], zr[2 * ks + 1], qf[1][2 * ks], qf[1][2 * ks + 1]);
          }
        }
        if (lane < 8) {
          float* dst = cpart_sm + ((b * 2 + qn) * kTcConvertWarps + cw) * 16 + 2 * qc4;
          *reinterpret_cast<float2*>(dst) = make_float2(c0[0], c0[1]);
          *reinterpret_cast<float2*>(dst + 8) = make_float2(c1[0], c1[1]);
        }
      }
      // the next tile's codes: the first half block now, the second once this tile's Q' is written (the
      // registers they need are free by then)
      if (have_n && tn.kind == 0) tc_load_half(p.arena + static_cast<size_t>(tn.off256) * 256, tn.level, 0, dj, dg, w[0]);
      PROF_LAP(4);
      // the Q' buffer is free once the key MMAs of tile tg - 1 are done
      if (tg >= 1) ok = t_wait_role(cw == 0, bar(kBarSFull, (tg - 1) & 1), ((tg - 1) >> 1) & 1, 2, kTcConvertWarps * 32, abort_flag);
      if (!ok) break;
      PROF_LAP(5);
      const uint32_t qp = base + kOffQp;
      const bool quant = t.kind == 0;
      const __half2 f16 = __float2half2_rn((quant && t.level == 4) ? 16.f : 1.f);     // the b = 0 channel pairs of a 4-bit chunk
#pragma unroll
      for (int half = 0; half < 2; ++half) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          uint32_t sw[4] = {svh[half][e].x, svh[half][e].y, svh[half][e].z, svh[half][e].w};
          if (!quant) sw[0] = sw[1] = sw[2] = sw[3] = 0x3C003C00u;                      // exact and centroid rows: scale 1
          sw[0] = t_u(__hmul2(t_h2(sw[0]), f16));
          sw[2] = t_u(__hmul2(t_h2(sw[2]), f16));
#pragma unroll
          for (int tq = 0; tq < 2; ++tq) {
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const __half2 h = __hmul2(t_h2(qf[tq][4 * e + i]), t_h2(sw[i]));
              hi[i] = t_u(h);
              lo[i] = t_u(__hfma2(t_h2(qf[tq][4 * e + i]), t_h2(sw[i]), __hneg2(h)));
            }
            const int row = 32 * half + qn + 8 * tq;          // column of S: half, (hi | lo), head
            t_sts128(tc_tile_addr(qp, row, qj0 + e), hi[0], hi[1], hi[2], hi[3]);
            t_sts128(tc_tile_addr(qp, row + 16, qj0 + e), lo[0], lo[1], lo[2], lo[3]);
          }
        }
      }
      t_fence_async();
      __syncwarp();
      PROF_LAP(6);
      if (lane == 0) t_bar_arrive(bar(kBarQpFull, b));
      if (have_n && tn.kind == 0) {
        tc_load_half(p.arena + static_cast<size_t>(tn.off256) * 256, tn.level, 1, dj, dg, w[1]);
        load_params(tn);
      }
      t = tn;
      have = have_n;
      ++tg;
      PROF_LAP(7);
    }
  } else if (warp >= 4) {
    // ---------------- read-out of the channel tiles [kTcReadTiles0, 4) (warps 4-7) ----------------
    const int lt = tid - 128;                               // tensor-memory lane
    const uint32_t tlane = tmem + (static_cast<uint32_t>(32 * (warp - 4)) << 16);
    TcTile t;
    int it = cd.item_begin, ts = 0;
    bool ok = true;
    TableEntry pre = tc_entry(p, table, it);
    PROF_DECL(16);
    while (ok && tc_next(p, table, cd.item_end, it, pre, t)) {
      pre = tc_entry(p, table, t.item + t.adv);
      PROF_LAP(0);
      // what the softmax of tile ts published: the sums of its probabilities and whether it moved the running max
      ok = t_wait_role(warp == 4, bar(kBarHsFull, ts & 1), (ts >> 1) & 1, 3, 128, abort_flag) && ok;
      PROF_LAP(1);
      ok = tc_read_out(p, t, ts, kTcReadTiles0, 4, need_sm[ts & 1] != 0, alpha_sm + (ts & 1) * 16, hsum2_sm + (ts & 1) * 32, tlane, lt,
                       bar(kBarPvDone, ts & 1), warp == 4, 3, abort_flag
#ifdef GKV_MLA_PROF
                       , prof_sm
#endif
                       ) && ok;
      __syncwarp();
      if (lane == 0) t_bar_arrive(bar(kBarRFree, 0));
      it = t.item + t.adv;
      ++ts;
      PROF_LAP(2);
    }
  } else {
    // ---------------- softmax, read-out of the first channel tiles (warps 0-3) and the result ----------------
    float m_run[16], l_part[16];
#pragma unroll
    for (int h = 0; h < 16; ++h) {
      m_run[h] = kNegInfT;
      l_part[h] = 0.f;
    }
    const uint32_t tlane = tmem + (static_cast<uint32_t>(32 * warp) << 16);
    const int half = warp >> 1;                             // the half block of this warp's 16 token rows
    bool ok = true;
    TcTile t;
    int it = cd.item_begin, ts = 0, xph = 0;                // xph: exchanges done so far (phase of the exchange buffers)
    TableEntry pre = tc_entry(p, table, it);
    PROF_DECL(8);
    while (tc_next(p, table, cd.item_end, it, pre, t)) {
      pre = tc_entry(p, table, t.item + t.adv);
      const int b = ts & 1;
      PROF_LAP(0);
      {
        // warp 0 waits for the parts of the key constants (written before Q' is published), adds the
        // nine parts per (half, head) in a fixed order, then waits for the logits; the role barrier
        // releases the other three warps and publishes the constants to them
        bool okl = true;
        if (warp == 0) {
          okl = t_wait(bar(kBarQpFull, b), (ts >> 1) & 1, abort_flag);
          const float* cp = cpart_sm + ((b * 2 + (tid >> 4)) * kTcConvertWarps) * 16 + (tid & 15);
          float c = 0.f;
#pragma unroll
          for (int w9 = 0; w9 < kTcConvertWarps; ++w9) c += cp[w9 * 16];
          const_sm[b * 32 + tid] = t.kind == 0 ? c : 0.f;
          okl = t_wait(bar(kBarSFull, b), (ts >> 1) & 1, abort_flag) && okl;
        }
        ok = t_role_sync(1, 128, okl) && ok;
      }
      PROF_LAP(1);
      t_fence_after();
      float s[16], sl[16];
      t_ld16_async(tlane + kTmemS + 64 * b + 32 * half, s);
      t_ld16_async(tlane + kTmemS + 64 * b + 32 * half + 16, sl);
      t_wait_ld();
      const int row = 16 * warp + (lane & 15);
      const float bs = (lane < 16) ? bias_sm[b * 64 + row] : kNegInfT;
      const float ks = tc_logit_scale(t.kind, t.level);
      // Common case: no logit of the tile exceeds its head's running max by more than the slack;
      // then the (stale) max stays and nothing is reduced.  The four warps agree through one flag
      // exchange; only when a flag is up are the head maxima reduced and the sums rescaled.
      bool mine = false;
#pragma unroll
      for (int h = 0; h < 16; ++h) {
        s[h] = (bs == kNegInfT) ? kNegInfT : fmaf(fmaf(s[h] + sl[h], ks, const_sm[b * 32 + half * 16 + h]), p.scale_log2, bs);
        mine |= s[h] > m_run[h] + kRescaleSlack;            // also true for the first finite logit (max = -inf)
      }
      uint32_t need_u;
      asm volatile(
          "{\n"
          ".reg .pred pi, po;\n"
          "setp.ne.u32 pi, %1, 0;\n"
          "bar.red.or.pred po, 1, 128, pi;\n"
          "selp.u32 %0, 1, 0, po;\n"
          "}\n"
          : "=r"(need_u)
          : "r"(static_cast<uint32_t>(mine))
          : "memory");
      const bool need = need_u != 0;
      if (need) {                                           // uniform over the 128 softmax threads
        float mx[16];
#pragma unroll
        for (int h = 0; h < 16; ++h) mx[h] = s[h];
#pragma unroll
        for (int d = 8; d >= 1; d >>= 1)
#pragma unroll
          for (int h = 0; h < 16; ++h) mx[h] = fmaxf(mx[h], __shfl_xor_sync(kFullT, mx[h], d));
        float* mbuf = max_sm + (xph & 1) * 64;
        if (lane == 0) {
#pragma unroll
          for (int h = 0; h < 16; ++h) mbuf[warp * 16 + h] = mx[h];
        }
        asm volatile("bar.sync 1, 128;\n" ::: "memory");
#pragma unroll
        for (int h = 0; h < 16; ++h) {
          const float bm = fmaxf(fmaxf(mbuf[h], mbuf[16 + h]), fmaxf(mbuf[32 + h], mbuf[48 + h]));
          const float mn = fmaxf(m_run[h], bm);
          const float al = (m_run[h] == kNegInfT) ? 0.f : t_ex2(m_run[h] - mn);
          m_run[h] = mn;
          l_part[h] *= al;
          if (tid == 0) alpha_sm[b * 16 + h] = al;          // what O^T (tiles before this one) is rescaled by
        }
        ++xph;
      }
      if (tid == 0) need_sm[b] = need ? 1 : 0;
      // probabilities relative to the (possibly stale) running max as fp16 pairs hi + lo; the
      // unrounded value is what is summed
      float pr[16];
#pragma unroll
      for (int h = 0; h < 16; ++h) {
        pr[h] = (lane < 16 && s[h] != kNegInfT) ? t_ex2(s[h] - m_run[h]) : 0.f;
        l_part[h] += pr[h];
      }
      // the P buffer is free once the value MMAs of the tile before are done
      PROF_LAP(2);
      if (ts > 0) ok = t_wait_role(warp == 0, bar(kBarPvDone, (ts - 1) & 1), ((ts - 1) >> 1) & 1, 1, 128, abort_flag) && ok;
      PROF_LAP(3);
      if (lane < 16) {
        uint32_t pk[8], pl[8];
#pragma unroll
        for (int h = 0; h < 16; h += 2) {
          const __half2 ph = __floats2half2_rn(pr[h], pr[h + 1]);
          pk[h >> 1] = t_u(ph);
          pl[h >> 1] = t_u(__floats2half2_rn(pr[h] - __low2float(ph), pr[h + 1] - __high2float(ph)));
        }
        // row of 16 heads (32 B) of token `row`; 32-byte swizzle: the 16-byte halves swap on bit 7
        const uint32_t prow = base + kOffP + row * 32;
        const uint32_t sw = ((row >> 2) & 1) << 4;
        t_sts128(prow + sw, pk[0], pk[1], pk[2], pk[3]);
        t_sts128(prow + (sw ^ 16), pk[4], pk[5], pk[6], pk[7]);
        t_sts128(prow + 2048 + sw, pl[0], pl[1], pl[2], pl[3]);
        t_sts128(prow + 2048 + (sw ^ 16), pl[4], pl[5], pl[6], pl[7]);
      }
      // sums of the warp's 16 rows per head (for the zero-point term of the read-out), fixed order
      // (reduce-scatter: after the step with distance d a lane keeps the heads whose bit d equals
      // its own, so lane j < 16 ends with the sum of head j; lanes 16-31 hold zeros)
#pragma unroll
      for (int d = 8; d >= 1; d >>= 1) {
        const bool up = (lane & d) != 0;
#pragma unroll
        for (int h = 0; h < d; ++h) {
          const float give = up ? pr[h] : pr[h + d], keep = up ? pr[h + d] : pr[h];
          pr[h] = keep + __shfl_xor_sync(kFullT, give, d);
        }
      }
      if (lane < 16) hsum_sm[b * 64 + warp * 16 + lane] = pr[0];
      t_fence_async();
      t_fence_before();
      __syncwarp();
      if (lane == 0) t_bar_arrive(bar(kBarPFull, 0));
      // the sums of the tile per half block: the two warps of a half added in a fixed order
      asm volatile("bar.sync 1, 128;\n" ::: "memory");
      if (tid < 32) hsum2_sm[b * 32 + tid] = hsum_sm[b * 64 + (tid >> 4) * 32 + (tid & 15)] + hsum_sm[b * 64 + (tid >> 4) * 32 + 16 + (tid & 15)];
      __syncwarp();
      if (lane == 0) t_bar_arrive(bar(kBarHsFull, b));
      if (kTcReadTiles0 > 0) {
        asm volatile("bar.sync 1, 128;\n" ::: "memory");                  // the sums are complete
        ok = tc_read_out(p, t, ts, 0, kTcReadTiles0, need, alpha_sm + b * 16, hsum2_sm + b * 32, tlane, tid, bar(kBarPvDone, b), warp == 0, 1, abort_flag
#ifdef GKV_MLA_PROF
                       , prof_sm
#endif
                       ) && ok;
        __syncwarp();
        if (lane == 0) t_bar_arrive(bar(kBarRFree, 0));
      }
      it = t.item + t.adv;
      ++ts;
      PROF_LAP(4);
    }
#ifdef GKV_MLA_PROF
    if (tid == 0) prof_sm[13] += ts;
#endif
    // ---------------- result ----------------
    float* out = p.partial + static_cast<size_t>(cd.partial) * kMlaPartialFloats;
#pragma unroll
    for (int d = 8; d >= 1; d >>= 1)
#pragma unroll
      for (int h = 0; h < 16; ++h) l_part[h] += __shfl_xor_sync(kFullT, l_part[h], d);
    if (lane == 0) {
#pragma unroll
      for (int h = 0; h < 16; ++h) sum_sm[warp * 16 + h] = l_part[h];
    }
    asm volatile("bar.sync 1, 128;\n" ::: "memory");
    const bool good = __all_sync(kFullT, ok && ts > 0 && !*abort_flag);
    if (warp == 0 && lane == 0) {
#pragma unroll
      for (int h = 0; h < 16; ++h) {
        out[h * (kMlaDv + 2)] = good ? m_run[h] : kNegInfT;
        out[h * (kMlaDv + 2) + 1] = good ? sum_sm[h] + sum_sm[16 + h] + sum_sm[32 + h] + sum_sm[48 + h] : 0.f;
      }
    }
  }
  // the running O^T is complete once every read-out warp is here
  t_fence_before();
  __syncthreads();
  t_fence_after();
  if (warp < 4) {
    const uint32_t tlane = tmem + (static_cast<uint32_t>(32 * warp) << 16);
    float* out = p.partial + static_cast<size_t>(cd.partial) * kMlaPartialFloats;
    const bool good = !*abort_flag;
#pragma unroll 1
    for (int i = 0; i < 4; ++i) {
      float o[16];
      if (good) {
        t_ld16(tlane + kTmemO + 16 * i, o);
      } else {
#pragma unroll
        for (int h = 0; h < 16; ++h) o[h] = 0.f;
      }
      const int ch = 128 * i + 32 * warp + lane;
#pragma unroll
      for (int h = 0; h < 16; ++h) out[h * (kMlaDv + 2) + 2 + ch] = o[h];
    }
  }
  t_fence_before();
  __syncthreads();
#ifdef GKV_MLA_PROF
  if (tid < 32) g_prof[blockIdx.x * 32 + tid] += prof_sm[tid];
#endif
  if (tid == 0 && *abort_flag) atomicOr(p.status, kStatusInternal);
  if (warp == 0) t_tmem_dealloc(tmem, kTmemCols);
}

// Merge the partial rows of a stream's CTAs.  One block per (stream, head, slice of 64 value
// channels); its 512 threads are 8 row groups x 64 channels, row group g sums rows g, g + 8, ...
// in that order and the 8 sums are added in group order, so the result is bitwise reproducible.
constexpr int kCombSlice = 64, kCombGroups = 8, kCombThreads = kCombSlice * kCombGroups;
__global__ void __launch_bounds__(kCombThreads) mla_combine_kernel(const float* partial, const StreamParts* parts, float* out,
                                                                   float* lse) {
  __shared__ float sm_m[kCombThreads], sm_w[kCombThreads], sm_acc[kCombGroups][kCombSlice];
  const int stream = blockIdx.x, h = blockIdx.y, slice = blockIdx.z, tid = threadIdx.x;
  const int c = tid % kCombSlice, g = tid / kCombSlice;
  const int begin = parts[stream].begin, end = parts[stream].end;
  const float* base = partial + h * (kMlaDv + 2);
  // pass 1: the maximum of the rows' maxima (one row per thread, then a shared-memory sweep)
  float M = kNegInfT;
  for (int c0 = begin; c0 < end; c0 += kCombThreads) {
    const int n = min(kCombThreads, end - c0);
    __syncthreads();
    sm_m[tid] = tid < n ? __ldcg(base + static_cast<size_t>(c0 + tid) * kMlaPartialFloats) : kNegInfT;
    __syncthreads();
#pragma unroll 8
    for (int i = 0; i < n; ++i) M = fmaxf(M, sm_m[i]);
  }
  // pass 2: weights per row in shared memory, then every thread sums its channel over its rows
  float L = 0.f, acc = 0.f;
  for (int c0 = begin; c0 < end; c0 += kCombThreads) {
    const int n = min(kCombThreads, end - c0);
    __syncthreads();
    if (tid < n) {
      const float* row = base + static_cast<size_t>(c0 + tid) * kMlaPartialFloats;
      const float m = __ldcg(row);
      const float w = (m == kNegInfT) ? 0.f : exp2f(m - M);
      sm_w[tid] = w;
      sm_m[tid] = w * __ldcg(row + 1);
    }
    __syncthreads();
    const float* col = base + static_cast<size_t>(c0) * kMlaPartialFloats + 2 + slice * kCombSlice + c;
#pragma unroll 8
    for (int i = g; i < n; i += kCombGroups) acc = fmaf(sm_w[i], __ldcg(col + static_cast<size_t>(i) * kMlaPartialFloats), acc);
    if (g == 0 && c == 0)
      for (int i = 0; i < n; ++i) L += sm_m[i];
  }
  sm_acc[g][c] = acc;
  __syncthreads();
  if (g == 0) {
    if (c == 0) sm_m[0] = L;
  }
  __syncthreads();
  L = sm_m[0];
  if (g == 0) {
    float tot = 0.f;
#pragma unroll
    for (int k = 0; k < kCombGroups; ++k) tot += sm_acc[k][c];
    const size_t hq = static_cast<size_t>(stream) * kMlaHeads + h;
    out[hq * kMlaDv + slice * kCombSlice + c] = (L > 0.f) ? tot / L : 0.f;
    if (lse && slice == 0 && c == 0) lse[hq] = (L > 0.f) ? (M + log2f(L)) * 0.6931471805599453f : kNegInfT;
  }
}

}  // namespace

cudaError_t launch_mla_decode(const MlaDecodeParams& p, int n_ctas, const StreamParts* parts, int n_streams, float* out,
                              float* lse, cudaStream_t st) {
  if (n_ctas <= 0) return cudaSuccess;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(mla_tc_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  mla_tc_decode_kernel<<<n_ctas, kTcThreads, kTcSmem, st>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  mla_combine_kernel<<<dim3(n_streams, kMlaHeads, kMlaDv / kCombSlice), kCombThreads, 0, st>>>(p.partial, parts, out, lse);
  return cudaGetLastError();
}

}  // namespace gkv

#ifdef GKV_MLA_PROF
extern "C" __attribute__((visibility("default"))) void gkv_x_prof_read(unsigned long long* buf, int reset) {
  if (reset) {
    static unsigned long long z[148 * 32];
    cudaMemcpyToSymbol(gkv::g_prof, z, sizeof(z));
  } else {
    cudaMemcpyFromSymbol(buf, gkv::g_prof, sizeof(unsigned long long) * 148 * 32);
  }
}
#endif
