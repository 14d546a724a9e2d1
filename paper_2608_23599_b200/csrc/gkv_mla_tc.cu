// Decode attention for latent-attention (MLA) streams on the 5th-generation tensor cores
// (Sec. 3.1 read path applied to a 576-wide latent row that is key and value at once).
//
// One CTA per SM walks a contiguous range of one stream's blocks.  Per 64-token tile:
//   1. a producer thread stages the packed block (TMA bulk copies, two raw stages, mbarriers);
//   2. nine warps dequantise it to fp16 (k~ = s * code + z, rounded once) into a 128-byte-swizzled
//      shared-memory tile [9 panels of 64 channels][64 tokens][128 B];
//   3. one thread issues tcgen05.mma: S[64 tokens x 16 heads] = K~ Q^T (A = the tile, K-major;
//      B = the query, K-major; accumulator in tensor memory);
//   4. four warps read S from tensor memory, run the online softmax and write P (fp16) to shared
//      memory;
//   5. the same thread issues O^T[512 channels x 16 heads] += V~^T P^T with A = the same tile read
//      MN-major (channels are contiguous), four accumulators of 128 channels in tensor memory.
// Tiles are double-buffered, so the dequantisation of tile i + 1 overlaps the tensor-core work of
// tile i.  Every wait is bounded; on a time-out the CTA raises kStatusInternal and publishes an
// empty partial.  Partials of the CTAs of a stream are merged by mla_combine_kernel in CTA order.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "gkv_internal.h"
#include "gkv_layout.cuh"
#include "gkv_mla.h"

namespace gkv {
namespace {

constexpr int kTcDequantWarps = 9;                     // 288 threads = 72 chunks x 4 token groups
constexpr int kTcFirstDequantWarp = 4;                 // warps 0-3 run the softmax
constexpr int kTcProducerWarp = 13, kTcMmaWarp = 14;
constexpr int kTcThreads = 15 * 32;
constexpr int kTcPanelBytes = 64 * 128;                // 64 tokens x 64 channels fp16
constexpr int kTcTileBytes = 9 * kTcPanelBytes;        // 73728
constexpr int kTcQBytes = 9 * 16 * 128;                // 16 heads x 576 channels fp16, 9 panels
constexpr int kTcPBytes = 16 * 128;                    // 16 heads x 64 tokens fp16
constexpr int kTcRawBytes = 20736;                     // int8 half = 2304 + 32 x 576; 16 exact rows = 18432
// shared-memory map (offsets from a 1024-byte aligned base)
constexpr int kOffTile = 0;
constexpr int kOffQ = 2 * kTcTileBytes;                // 147456
constexpr int kOffP = kOffQ + kTcQBytes;               // 165888
constexpr int kOffRaw = kOffP + 2 * kTcPBytes;         // 169984
constexpr int kOffMisc = kOffRaw + 2 * kTcRawBytes;    // 211456
constexpr int kTcSmem = kOffMisc + 2048 + 1024;        // + misc + alignment slack
// misc: 16 mbarriers (128 B) | tmem base (4 B) @128 | abort flag @132 | bias[2][64] floats @256 |
//       head maxima [2][4 warps][16] floats @768, rescale flags [2][4] ints @1280 | row sums [4][16] @1344
constexpr int kMiscTmem = 128, kMiscAbort = 132, kMiscBias = 256, kMiscMax = 768, kMiscSum = 1344;
enum { kBarRawFull = 0, kBarRawEmpty = 2, kBarKtFull = 4, kBarSFull = 6, kBarPFull = 8, kBarPvDone = 10, kBarMax = 12, kBarSum = 14 };
constexpr int kTcWaitSpins = 1 << 20;
constexpr float kNegInfT = -INFINITY;
constexpr uint32_t kFullT = 0xffffffffu;
constexpr uint32_t kTmemCols = 128;                    // S[2] at columns 0 / 16, O^T tiles at 32 + 16 i
constexpr uint32_t kTmemS = 0, kTmemO = 32;
constexpr float kRescaleSlack = 8.f;                   // keep a stale running max while logits stay within 2^8 of it

__device__ __forceinline__ uint32_t t_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void t_bar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void t_fence_async() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void t_bar_expect(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void t_bar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void t_bulk(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
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
      : "r"(bar), "r"(parity), "r"(2000)
      : "memory");
  return ok != 0;
}
// Bounded wait; a time-out raises the CTA's abort flag, which every other waiter also watches.
__device__ __forceinline__ bool t_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  int spins = 0;
  while (!t_try_wait(bar, parity)) {
    if (++spins > kTcWaitSpins || *abort_flag) {
      *abort_flag = 1;
      return false;
    }
  }
  return true;
}
// the same for a whole warp: the outcome is made uniform (lanes poll on their own)
__device__ __forceinline__ bool t_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return __all_sync(kFullT, t_wait(bar, parity, abort_flag));
}
__device__ __forceinline__ uint4 t_lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 t_lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t t_lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ void t_sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ uint32_t t_lop_ao(uint32_t x, uint32_t mask, uint32_t orv) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;\n" : "=r"(r) : "r"(x), "r"(mask), "r"(orv));
  return r;
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
__device__ __noinline__ bool tc_next(const MlaDecodeParams& p, const TableEntry* table, int item_end, int it, const TableEntry e,
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

// producer warp: copies of stage s of tile t into raw buffer `raw`.  Lane 0 posts the byte count
// and issues the contiguous copies; the rows of a centroid gather are issued by lanes 0-15, one
// row each, so that their table look-ups run in parallel.
__device__ __forceinline__ void tc_issue(const MlaDecodeParams& p, const TableEntry* table, const TcTile& t, int s, uint32_t raw,
                                         uint32_t bar, int lane) {
  const uint8_t* slot = p.arena + static_cast<size_t>(t.off256) * 256;
  if (t.kind == 0) {
    if (lane == 0) {
      const uint32_t bytes = static_cast<uint32_t>(mla_half_bytes(t.level));
      t_bar_expect(bar, bytes);
      t_bulk(raw, slot + static_cast<size_t>(s) * bytes, bytes, bar);
    }
  } else if (t.kind == 1) {
    if (lane == 0) {
      const int n = min(16, t.nrows - 16 * s);
      t_bar_expect(bar, static_cast<uint32_t>(n) * kMlaRowBytes);
      t_bulk(raw, slot + static_cast<size_t>(16 * s) * kMlaRowBytes, static_cast<uint32_t>(n) * kMlaRowBytes, bar);
    }
  } else {
    const int n = min(16, t.nrows - 16 * s);
    const uint8_t* src = nullptr;
    if (lane < n) src = p.arena + static_cast<size_t>(table[t.item + 16 * s + lane].off256) * 256;
    if (lane == 0) t_bar_expect(bar, static_cast<uint32_t>(n) * kMlaRowBytes);
    __syncwarp();
    if (lane < n) t_bulk(raw + lane * kMlaRowBytes, src, kMlaRowBytes, bar);
  }
  __syncwarp();
}

// address of the 16-byte piece (row, chunk j of 8 channels) inside a swizzled tile
__device__ __forceinline__ uint32_t tc_tile_addr(uint32_t tile, int row, int j) {
  return tile + (j >> 3) * kTcPanelBytes + row * 128 + ((((j & 7) ^ (row & 7))) << 4);
}

// dequantise one half (32 tokens) of a quantised block: thread = (chunk j, 8 tokens)
template <int BITS>
__device__ __forceinline__ void tc_dequant_half(uint32_t raw, uint32_t tile, int half, int j, int tg) {
  const uint4 sv = t_lds128(raw + j * 16), zv = t_lds128(raw + kMlaZeroOff * 2 + j * 16);
  const __half2 s0 = t_h2(sv.x), s1 = t_h2(sv.y), s2 = t_h2(sv.z), s3 = t_h2(sv.w);
  const __half2 z0 = t_h2(zv.x), z1 = t_h2(zv.y), z2 = t_h2(zv.z), z3 = t_h2(zv.w);
  const uint32_t codes = raw + mla_kp_bytes() + j * BITS + tg * 8 * (kMlaChunks * BITS);
  // rows 32 half + 8 tg + i: row & 7 = i, so the swizzled 16-byte slot is (j & 7) ^ i
  const uint32_t out = tile + (j >> 3) * kTcPanelBytes + (32 * half + 8 * tg) * 128;
  const uint32_t jx = (j & 7) << 4;
  const __half2 b0 = __float2half2_rn(1024.f), b1 = __float2half2_rn(BITS == 4 ? 64.f : 1024.f);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    uint32_t x0, x1, x2, x3;
    if constexpr (BITS == 4) {
      const uint32_t w = t_lds32(codes + i * (kMlaChunks * 4));
      const uint32_t v = w >> 8;
      x0 = t_lop_ao(w, 0x000F000Fu, 0x64006400u);      // 1024 + code (channels 0, 1)
      x1 = t_lop_ao(w, 0x00F000F0u, 0x54005400u);      // 64 + code   (channels 2, 3)
      x2 = t_lop_ao(v, 0x000F000Fu, 0x64006400u);
      x3 = t_lop_ao(v, 0x00F000F0u, 0x54005400u);
    } else {
      const uint2 w = t_lds64(codes + i * (kMlaChunks * 8));
      x0 = t_prmt(w.x, 0x64006400u, 0x5250u);
      x1 = t_prmt(w.x, 0x64006400u, 0x5351u);
      x2 = t_prmt(w.y, 0x64006400u, 0x5250u);
      x3 = t_prmt(w.y, 0x64006400u, 0x5351u);
    }
    // code = x - bias exactly; k~ = code * s + z with one rounding
    const uint32_t y0 = t_u(__hfma2(__hsub2(t_h2(x0), b0), s0, z0));
    const uint32_t y1 = t_u(__hfma2(__hsub2(t_h2(x1), b1), s1, z1));
    const uint32_t y2 = t_u(__hfma2(__hsub2(t_h2(x2), b0), s2, z2));
    const uint32_t y3 = t_u(__hfma2(__hsub2(t_h2(x3), b1), s3, z3));
    t_sts128(out + i * 128 + (jx ^ (i << 4)), y0, y1, y2, y3);
  }
}

__device__ __forceinline__ uint32_t tc_bf2_to_h2(uint32_t u) {
  return t_u(__floats2half2_rn(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u)));
}
// 16 bf16 rows of a raw stage -> fp16 rows [16 q, 16 q + 16) of the tile; rows >= n become zeros
__device__ __forceinline__ void tc_rows_quarter(uint32_t raw, uint32_t tile, int q, int n, int tid) {
  const int j = tid % kMlaChunks, rg = tid / kMlaChunks;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = rg * 4 + i;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (r < n) {
      v = t_lds128(raw + r * kMlaRowBytes + j * 16);
      v.x = tc_bf2_to_h2(v.x);
      v.y = tc_bf2_to_h2(v.y);
      v.z = tc_bf2_to_h2(v.z);
      v.w = tc_bf2_to_h2(v.w);
    }
    t_sts128(tc_tile_addr(tile, 16 * q + r, j), v.x, v.y, v.z, v.w);
  }
}

// ---- kernel ------------------------------------------------------------------------------------
// Warp roles: 0-3 softmax (warp w owns tensor-memory lanes 32 w .. 32 w + 31), 4-12 dequantisation,
// 13 producer, 14 tensor-core issue.
__global__ void __launch_bounds__(kTcThreads, 1) mla_tc_decode_kernel(const __grid_constant__ MlaDecodeParams p) {
  extern __shared__ uint8_t tsm_raw[];
  const WarpDesc cd = p.ctas[blockIdx.x];
  if (cd.stream < 0) return;                               // uniform for the CTA
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
  const uint32_t base = (t_u32(tsm_raw) + 1023u) & ~1023u;
  uint8_t* gbase = tsm_raw + (base - t_u32(tsm_raw));
  const uint32_t misc = base + kOffMisc;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + kOffMisc + kMiscAbort);
  float* bias_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscBias);      // [2][64]
  float* max_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscMax);        // [2][4][16]
  float* sum_sm = reinterpret_cast<float*>(gbase + kOffMisc + kMiscSum);        // [4][16]
  const TableEntry* table = p.table + static_cast<size_t>(cd.stream) * p.table_stride;
  auto bar = [&](int which, int i) { return misc + 8u * static_cast<uint32_t>(which + i); };

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      t_bar_init(bar(kBarRawFull, i), 1);
      t_bar_init(bar(kBarRawEmpty, i), kTcDequantWarps);
      t_bar_init(bar(kBarKtFull, i), kTcDequantWarps);
      t_bar_init(bar(kBarSFull, i), 1);
      t_bar_init(bar(kBarPFull, i), 4);
      t_bar_init(bar(kBarPvDone, i), 1);
      t_bar_init(bar(kBarMax, i), 4);
    }
    t_bar_init(bar(kBarSum, 0), 4);
    *abort_flag = 0;
    t_fence_async();
  }
  if (warp == 0) t_tmem_alloc(misc + kMiscTmem, kTmemCols);
  // query -> fp16, K-major swizzled panels [9][16 heads][128 B]
  {
    const uint16_t* q = p.q + static_cast<size_t>(cd.stream) * kMlaHeads * kMlaDk;
    for (int i = tid; i < kMlaHeads * kMlaChunks; i += kTcThreads) {
      const int h = i / kMlaChunks, j = i % kMlaChunks;
      const uint4 v = *reinterpret_cast<const uint4*>(q + h * kMlaDk + 8 * j);
      const uint32_t dst = base + kOffQ + (j >> 3) * (16 * 128) + h * 128 + ((((j & 7) ^ (h & 7))) << 4);
      t_sts128(dst, tc_bf2_to_h2(v.x), tc_bf2_to_h2(v.y), tc_bf2_to_h2(v.z), tc_bf2_to_h2(v.w));
    }
  }
  t_fence_async();
  t_fence_before();
  __syncthreads();
  t_fence_after();
  const uint32_t tmem = __shfl_sync(kFullT, *reinterpret_cast<volatile uint32_t*>(gbase + kOffMisc + kMiscTmem), 0);

  if (warp == kTcProducerWarp) {
    // ---------------- producer: raw stages (lane 0 drives; lanes 0-15 share a centroid gather) ----------------
    TcTile t;
    int it = cd.item_begin, sg = 0;
    bool ok = true;
    TableEntry pre = tc_entry(p, table, it);
    while (ok && tc_next(p, table, cd.item_end, it, pre, t)) {
      pre = tc_entry(p, table, t.item + t.adv);
      for (int s = 0; s < t.nstages && ok; ++s, ++sg) {
        const int b = sg & 1;
        ok = t_wait_warp(bar(kBarRawEmpty, b), ((sg >> 1) & 1) ^ 1, abort_flag);        // fresh barriers pass
        if (ok) tc_issue(p, table, t, s, base + kOffRaw + b * kTcRawBytes, bar(kBarRawFull, b), lane);
      }
      it = t.item + t.adv;
    }
  } else if (warp == kTcMmaWarp) {
    // ---------------- tensor-core issue (whole warp, one elected lane per instruction) ----------------
    {
      constexpr uint32_t kIdQK = t_idesc(64, 16, false), kIdPV = t_idesc(128, 16, true, true);
      // descriptors differ only in the start-address field (16-byte units in the low word)
      const uint64_t dq = t_desc(base + kOffQ, 16, 1024);
      auto issue_qk = [&](int tg) {
        const int b = tg & 1;
        const uint64_t da = t_desc(base + kOffTile + b * kTcTileBytes, 16, 1024);
        const uint32_t d = tmem + kTmemS + 16 * b;
#pragma unroll
        for (int pn = 0; pn < 9; ++pn)
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            t_mma_f16(d, da + ((pn * kTcPanelBytes + kk * 32) >> 4), dq + ((pn * 2048 + kk * 32) >> 4), kIdQK, (pn | kk) != 0);
        t_commit(bar(kBarSFull, b));
      };
      auto issue_pv = [&](int tg) {
        const int b = tg & 1;
        const uint64_t da = t_desc(base + kOffTile + b * kTcTileBytes, kTcPanelBytes, 1024);
        // P: [64 tokens][16 heads] fp16, heads contiguous (MN-major), 32-byte swizzle, 8-token groups of 256 B
        const uint64_t dp = t_desc(base + kOffP + b * kTcPBytes, 256, 256, 6);
        const uint32_t first = tg != 0;
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int kk = 0; kk < 4; ++kk)
            t_mma_f16(tmem + kTmemO + 16 * i, da + ((2 * i * kTcPanelBytes + kk * 2048) >> 4), dp + ((kk * 512) >> 4), kIdPV,
                      kk != 0 ? 1u : first);
        t_commit(bar(kBarPvDone, b));
      };
      // Event-driven order: the value MMAs of tile pv go out as soon as its P is there, the key MMAs
      // of tile qk as soon as its tile is there (qk runs at most two tiles ahead of pv: S and the
      // tile buffers are double).  n_tiles is not known in advance: the iterator tells.
      TcTile t;
      int it = cd.item_begin;
      TableEntry pre = tc_entry(p, table, it);
      bool more_tiles = tc_next(p, table, cd.item_end, it, pre, t);
      pre = tc_entry(p, table, t.item + t.adv);
      int qk = 0, pv = 0, n_known = more_tiles ? 1 : 0;      // tiles [0, n_known) exist so far
      bool ok = true;
      int spins = 0;
      while (ok && (pv < n_known || more_tiles)) {
        bool progress = false;
        // key MMAs of tile qk: S[qk & 1] is free once the softmax of tile qk - 2 has published its P
        if (qk < n_known && qk < pv + 2) {
          const bool ready = __all_sync(kFullT, t_try_wait(bar(kBarKtFull, qk & 1), (qk >> 1) & 1));
          if (ready) {
            t_fence_after();
            issue_qk(qk);
            ++qk;
            // look one tile further
            it = t.item + t.adv;
            more_tiles = tc_next(p, table, cd.item_end, it, pre, t);
            if (more_tiles) {
              ++n_known;
              pre = tc_entry(p, table, t.item + t.adv);
            }
            progress = true;
          }
        }
        if (pv < qk) {
          const bool ready = __all_sync(kFullT, t_try_wait(bar(kBarPFull, pv & 1), (pv >> 1) & 1));
          if (ready) {
            t_fence_after();
            issue_pv(pv);
            ++pv;
            progress = true;
          }
        }
        if (progress) spins = 0;
        else if (++spins > kTcWaitSpins || *abort_flag) {
          *abort_flag = 1;
          ok = false;
        }
        ok = __all_sync(kFullT, ok);
      }
    }
  } else if (warp >= kTcFirstDequantWarp) {
    // ---------------- dequantisation ----------------
    const int dt = tid - kTcFirstDequantWarp * 32;          // 0 .. 287
    const int dj = dt % kMlaChunks, dg = dt / kMlaChunks;   // chunk of 8 channels, token group
    TcTile t;
    int it = cd.item_begin, tg = 0, sg = 0;
    bool ok = true;
    TableEntry pre = tc_entry(p, table, it);
    while (ok && tc_next(p, table, cd.item_end, it, pre, t)) {
      pre = tc_entry(p, table, t.item + t.adv);
      const int b = tg & 1;
      const uint32_t tile = base + kOffTile + b * kTcTileBytes;
      // the tile buffer is free once the value MMAs of tile tg - 2 are done
      if (tg >= 2) ok = t_wait_warp(bar(kBarPvDone, b), ((tg - 2) >> 1) & 1, abort_flag);
      if (!ok) break;
      if (dt < 64) bias_sm[b * 64 + dt] = dt < t.nrows ? (t.kind == 2 ? 6.0f : 0.f) : kNegInfT;   // log2(64) per centroid row
      const int nq = (t.kind == 0) ? 2 : 4;
      for (int s = 0; s < nq && ok; ++s) {
        if (s < t.nstages) {
          const int rb = sg & 1;
          ok = t_wait_warp(bar(kBarRawFull, rb), (sg >> 1) & 1, abort_flag);
          if (!ok) break;
          const uint32_t raw = base + kOffRaw + rb * kTcRawBytes;
          if (t.kind == 0) {
            if (t.level == 8) tc_dequant_half<8>(raw, tile, s, dj, dg);
            else tc_dequant_half<4>(raw, tile, s, dj, dg);
          } else {
            tc_rows_quarter(raw, tile, s, min(16, t.nrows - 16 * s), dt);
          }
          __syncwarp();
          if (lane == 0) t_bar_arrive(bar(kBarRawEmpty, rb));
          ++sg;
        } else {
          tc_rows_quarter(0, tile, s, 0, dt);               // rows past the data: zeros
        }
      }
      if (!ok) break;
      t_fence_async();
      __syncwarp();
      if (lane == 0) t_bar_arrive(bar(kBarKtFull, b));
      it = t.item + t.adv;
      ++tg;
    }
  } else {
    // ---------------- softmax (warps 0-3) and the result ----------------
    float m_run[16], l_part[16];
#pragma unroll
    for (int h = 0; h < 16; ++h) {
      m_run[h] = kNegInfT;
      l_part[h] = 0.f;
    }
    TcTile t;
    int it = cd.item_begin, ts = 0, xph = 0;                // xph: exchanges done so far (phase of the exchange barrier)
    bool ok = true;
    const uint32_t tlane = tmem + (static_cast<uint32_t>(32 * warp) << 16);
    TableEntry pre = tc_entry(p, table, it);
    while (tc_next(p, table, cd.item_end, it, pre, t)) {
      pre = tc_entry(p, table, t.item + t.adv);
      const int b = ts & 1;
      ok = t_wait_warp(bar(kBarSFull, b), (ts >> 1) & 1, abort_flag) && ok;
      t_fence_after();
      float s[16];
      t_ld16(tlane + kTmemS + 16 * b, s);
      const int row = 16 * warp + (lane & 15);
      const float bs = (lane < 16) ? bias_sm[b * 64 + row] : kNegInfT;
      // Common case: no logit of the tile exceeds its head's running max by more than the slack;
      // then the (stale) max stays and nothing is reduced.  The four warps agree through one flag
      // exchange; only when a flag is up are the head maxima reduced and O rescaled.
      bool mine = false;
#pragma unroll
      for (int h = 0; h < 16; ++h) {
        s[h] = (bs == kNegInfT) ? kNegInfT : fmaf(s[h], p.scale_log2, bs);
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
        float alpha[16];
#pragma unroll
        for (int h = 0; h < 16; ++h) {
          const float bm = fmaxf(fmaxf(mbuf[h], mbuf[16 + h]), fmaxf(mbuf[32 + h], mbuf[48 + h]));
          const float mn = fmaxf(m_run[h], bm);
          alpha[h] = (m_run[h] == kNegInfT) ? 0.f : t_ex2(m_run[h] - mn);
          m_run[h] = mn;
          l_part[h] *= alpha[h];
        }
        ++xph;
        if (ts > 0) {                                       // O holds the tiles before ts: rescale it
          ok = t_wait_warp(bar(kBarPvDone, (ts - 1) & 1), ((ts - 1) >> 1) & 1, abort_flag) && ok;
          t_fence_after();
#pragma unroll 1
          for (int i = 0; i < 4; ++i) {
            float o[16];
            t_ld16(tlane + kTmemO + 16 * i, o);
#pragma unroll
            for (int h = 0; h < 16; ++h) o[h] *= alpha[h];
            t_st16(tlane + kTmemO + 16 * i, o);
          }
        }
      }
      // probabilities relative to the (possibly stale) running max; the rounded value is what is summed
      if (lane < 16) {
        uint32_t pk[8];
#pragma unroll
        for (int h = 0; h < 16; h += 2) {
          const float p0 = (s[h] == kNegInfT) ? 0.f : t_ex2(s[h] - m_run[h]);
          const float p1 = (s[h + 1] == kNegInfT) ? 0.f : t_ex2(s[h + 1] - m_run[h + 1]);
          const __half2 ph = __floats2half2_rn(p0, p1);
          l_part[h] += __low2float(ph);
          l_part[h + 1] += __high2float(ph);
          pk[h >> 1] = t_u(ph);
        }
        // row of 16 heads (32 B) of token `row`; 32-byte swizzle: the 16-byte halves swap on bit 7
        const uint32_t prow = base + kOffP + b * kTcPBytes + row * 32;
        const uint32_t sw = ((row >> 2) & 1) << 4;
        t_sts128(prow + sw, pk[0], pk[1], pk[2], pk[3]);
        t_sts128(prow + (sw ^ 16), pk[4], pk[5], pk[6], pk[7]);
      }
      t_fence_async();
      t_fence_before();
      __syncwarp();
      if (lane == 0) t_bar_arrive(bar(kBarPFull, b));
      it = t.item + t.adv;
      ++ts;
    }
    // ---------------- result ----------------
    float* out = p.partial + static_cast<size_t>(cd.partial) * kMlaPartialFloats;
    if (ts > 0) ok = t_wait_warp(bar(kBarPvDone, (ts - 1) & 1), ((ts - 1) >> 1) & 1, abort_flag) && ok;
    t_fence_after();
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
