// Decode attention for latent-attention (MLA) streams (Sec. 3.1 read path applied to a 576-wide
// latent row that is key and value at once), on warp-level tensor-core instructions with the
// running output in tensor memory.
//
// A quantised latent row is k~[c] = s[c] * code[c] + z[c] with one (s, z) pair per channel and
// half block (32 tokens, Sec. 3.2).  Nothing rounded ever becomes a tensor-core operand:
//   * codes are used as they are stored: a code in the mantissa of an fp16 with a zero exponent
//     field is the number code * 2^(b - 24), b its lowest bit (8-bit codes b = 0; 4-bit codes b = 0
//     or 4), taken out of the packed words with byte permutes and masks only;
//   * keys, heads along the MMA rows: S^T[16 heads x 32 tokens] = Q'^T K^T.  The scales go into the
//     query, Q'[c][head] = q[c][head] * s[c] as an fp16 pair hi + lo (the product of an 8-bit and an
//     11-bit mantissa has 19 bits), formed in registers once per half block: a lane's query registers
//     (heads g and g + 8, its four channels of the slab) times the scales are the A fragment, the code
//     registers the B fragments of the four 8-token groups.  sum_c q[c] z[c] is one more MMA per
//     channel slab with the unscaled query as A and the zero points in every column of B;
//   * values: O^T[512 x 16] += V~^T P^T reads the same packed codes a second time with tokens along k
//     and channels along m; the probabilities are an fp16 pair hi + lo; the per-channel scale and the
//     zero point (times the half block's probability sum) are applied in fp32 to the half block's
//     accumulator before it is added to the running O^T;
//   * exact rows, the tail and centroid rows (one row per block, +log2(64) on the logit) are bf16
//     operands of bf16 MMAs, the probabilities a bf16 pair hi + lo.
//
// Work split: a CTA is four groups of four warps ("quads").  A quad walks its own contiguous range
// of the stream's blocks in units of one half block (quantised) or 16 rows (exact, tail, centroid
// runs); a unit is staged by one bulk copy (or one per row) into the quad's two-stage ring.  Inside
// a quad warp w owns the value channels [128 w, 128 w + 128) and the rope channels
// [512 + 16 w, 512 + 16 w + 16): it computes the partial logits of its 144 channels for all tokens
// and heads of the unit, the four partials are exchanged through shared memory (added in warp
// order, so all four warps hold the same logits bit for bit), every warp runs the same online
// softmax, and then accumulates its own 128 rows of O^T.  A lane group g = lane / 4 owns the 16
// channels 128 w + 16 g .. + 15: M-tile mu of the value MMAs has row g = channel 2 mu and row
// g + 8 = channel 2 mu + 1 of them, for every kind of unit.
//
// Tensor memory holds what 128 registers per thread cannot: a warp's piece of the running O^T (64
// fp32 per thread; the eight of an M-tile are loaded before its MMAs and stored after its update)
// and the bf16 query fragments of its nine channel slabs for the row units.  Each warp touches only
// its own columns of its own lane quarter, so no tensor-memory access needs a barrier.
//
// At the end the quads' (m, l, O^T) are merged in shared memory into the CTA's partial row; the
// partial rows of a stream's CTAs are merged by mla_combine_kernel in CTA order.  Every wait is
// bounded; on a time-out the CTA raises kStatusInternal and publishes an empty partial.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "gkv_internal.h"
#include "gkv_layout.cuh"
#include "gkv_mla.h"

namespace gkv {
namespace {

constexpr int kMThreads = kMlaQuads * 128;
constexpr int kMStageBytes = 20736;                    // one 8-bit half block: params 2304 + 32 x 576
constexpr int kMStages = 2;
constexpr int kMRowPitch = kMlaRowBytes + 16;          // bf16 rows staged at this pitch (conflict-free ldmatrix)
constexpr int kMQPitch = 2 * kMlaRowBytes + 16;        // a head pair's row of the fp16 query: (q[g][c c+1], q[g + 8][c c+1]) per channel pair
constexpr int kMXBytes = 4 * 4 * 32 * 16;              // exchange buffer [warp][token group][lane] x 16 B = 8192
constexpr int kMOffQ16 = 0;
constexpr int kMOffQuad = 8 * kMQPitch;                // 18560
constexpr int kMQuadBytes = kMStages * kMStageBytes + kMXBytes + 64;   // stages | exchange | mbarriers
constexpr int kMOffFlag = kMOffQuad + kMlaQuads * kMQuadBytes;
constexpr int kMSmem = kMOffFlag + 16;                 // abort flag, tensor-memory base
constexpr uint32_t kMTmemCols = 512;                   // per warp 64 columns of O^T and 36 of bf16 query fragments, four warps per lane quarter
constexpr uint32_t kMTmemQ = 256;                      // first column of the query fragments
constexpr int kMOutPitch = kMlaDv + 2;                 // floats per head row of a quad's result in shared memory
constexpr int kMWaitSpins = 1 << 22;
constexpr float kMNegInf = -INFINITY;
constexpr float kMSlack = 8.f;                         // keep a stale running max while logits stay within 2^8 of it
constexpr uint32_t kMFull = 0xffffffffu;
static_assert(kMStageBytes >= 16 * kMRowPitch, "a stage holds 16 staged rows");
static_assert(kMStages * kMStageBytes >= kMlaHeads * kMOutPitch * 4 + 128, "a quad's result fits its stages");

// ---- PTX helpers -------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t m_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void m_bar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void m_fence_async() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void m_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void m_bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ bool m_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// bounded wait; false after kMWaitSpins failed polls
__device__ __forceinline__ bool m_wait(uint32_t bar, uint32_t parity) {
  for (int i = 0; i < kMWaitSpins; ++i) {
    if (m_try_wait(bar, parity)) return true;
    if (i > 64) __nanosleep(64);
  }
  return false;
}
__device__ __forceinline__ void m_quad_sync(int quad) { asm volatile("bar.sync %0, 128;\n" ::"r"(quad + 1) : "memory"); }
__device__ __forceinline__ uint4 m_lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 m_lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t m_lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ float4 m_ldsf4(uint32_t a) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void m_stsf4(uint32_t a, float x, float y, float z, float w) {
  asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};\n" ::"r"(a), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
__device__ __forceinline__ void m_stsf(uint32_t a, float v) { asm volatile("st.shared.f32 [%0], %1;\n" ::"r"(a), "f"(v) : "memory"); }
__device__ __forceinline__ void m_stsf2(uint32_t a, float x, float y) {
  asm volatile("st.shared.v2.f32 [%0], {%1,%2};\n" ::"r"(a), "f"(x), "f"(y) : "memory");
}
__device__ __forceinline__ void m_sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ uint32_t m_prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;\n" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}
__device__ __forceinline__ float m_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ __half2 m_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }
__device__ __forceinline__ uint32_t m_u(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ uint32_t m_ubf(__nv_bfloat162 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ void m_mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// D = A B (no accumulator input: the first MMA of a chain)
__device__ __forceinline__ void m_mma_f16_first(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
      : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ void m_mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void m_ldmatrix4(uint32_t a, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
// ---- tensor memory as the home of the running O^T (64 fp32 per thread: column 8 mu + 4 hg + i of the thread's lane) ----
__device__ __forceinline__ void m_tmem_alloc(uint32_t smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_dst), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void m_tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void m_tfence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void m_tfence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
// eight columns of the thread's lane; m_twait_ld() before the first use
__device__ __forceinline__ void m_tld8(uint32_t taddr, float (&v)[2][4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n"
               : "=f"(v[0][0]), "=f"(v[0][1]), "=f"(v[0][2]), "=f"(v[0][3]), "=f"(v[1][0]), "=f"(v[1][1]), "=f"(v[1][2]), "=f"(v[1][3])
               : "r"(taddr));
}
__device__ __forceinline__ void m_tld4(uint32_t taddr, uint32_t (&v)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(taddr));
}
__device__ __forceinline__ void m_tst4(uint32_t taddr, const uint32_t (&v)[4]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]) : "memory");
}
__device__ __forceinline__ void m_twait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ void m_tst8(uint32_t taddr, const float (&v)[2][4]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};\n" ::"r"(taddr), "f"(v[0][0]), "f"(v[0][1]),
               "f"(v[0][2]), "f"(v[0][3]), "f"(v[1][0]), "f"(v[1][1]), "f"(v[1][2]), "f"(v[1][3])
               : "memory");
}
__device__ __forceinline__ void m_twait_st() { asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ uint32_t m_ldg32(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.u32 %0, [%1];\n" : "=r"(v) : "l"(p));
  return v;
}

// q * s as an fp16 pair: hi = the rounded product, lo = the exact remainder
__device__ __forceinline__ void m_split(uint32_t q, uint32_t s, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __hmul2(m_h2(q), m_h2(s));
  hi = m_u(h);
  lo = m_u(__hfma2(m_h2(q), m_h2(s), __hneg2(h)));
}
__device__ __forceinline__ uint32_t m_bf2_to_h2(uint32_t u) {
  return m_u(__floats2half2_rn(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u)));
}
// 4-bit field n of both 16-bit halves of a packed word, left where it is (weight 2^(4 (n & 1)))
template <int N>
__device__ __forceinline__ uint32_t m_fld4(uint32_t w) {
  const uint32_t v = (N & 2) ? (w >> 8) : w;
  return v & ((N & 1) ? 0x00F000F0u : 0x000F000Fu);
}
__device__ __forceinline__ float m_h2f(uint32_t pair, int hi) {
  return hi ? __high2float(m_h2(pair)) : __low2float(m_h2(pair));
}

// ---- units -------------------------------------------------------------------------------------
// A quad's range of blocks is walked in units: one half block of a quantised block (kind 0), 16 rows
// of an exact block or of the tail (kind 1), or a run of up to 16 neighbouring centroid blocks, one
// row each (kind 2).  (m_load is called by whole, converged warps: the run is found with a ballot.)
struct MWalk {
  int it;                // item (block index; n_closed = the tail)
  uint32_t meta;         // sub | nsub << 4 | kind << 8 | level << 12 | run << 20 | nrows << 25
  uint32_t off256;
  __device__ __forceinline__ int sub() const { return static_cast<int>(meta & 15u); }        // unit inside the item
  __device__ __forceinline__ int nsub() const { return static_cast<int>((meta >> 4) & 15u); }
  __device__ __forceinline__ int kind() const { return static_cast<int>((meta >> 8) & 15u); }
  __device__ __forceinline__ int level() const { return static_cast<int>((meta >> 12) & 255u); }
  __device__ __forceinline__ int run() const { return static_cast<int>((meta >> 20) & 31u); }   // blocks the item covers
  __device__ __forceinline__ int nrows() const { return static_cast<int>(meta >> 25); }         // rows of the item (kind 1) or run (kind 2)
};
__device__ __forceinline__ uint32_t m_meta(int nsub, int kind, int level, int run, int nrows) {
  return static_cast<uint32_t>(nsub) << 4 | static_cast<uint32_t>(kind) << 8 | static_cast<uint32_t>(level) << 12 |
         static_cast<uint32_t>(run) << 20 | static_cast<uint32_t>(nrows) << 25;
}

__device__ __forceinline__ bool m_load(const MlaDecodeParams& p, const TableEntry* table, int item_end, MWalk& w) {
  if (w.it >= item_end) return false;
  const TableEntry e = table[min(w.it, p.n_closed)];
  w.off256 = e.off256;
  const int level = static_cast<int>(e.level);
  if (w.it == p.n_closed) {                        // the tail: exact rows, the last item of the stream
    if (p.n_tail == 0) return false;
    w.meta = m_meta((p.n_tail + 15) >> 4, 1, 16, 1, p.n_tail);
    return true;
  }
  if (level == 16) {
    w.meta = m_meta(4, 1, 16, 1, kBlock);
  } else if (level == 1) {
    const int lim = min(min(item_end, p.n_closed) - w.it, 16);
    const int ln = static_cast<int>(threadIdx.x & 31);
    const bool c = ln < lim && table[w.it + ln].level == 1u;
    const uint32_t b = __ballot_sync(kMFull, c);
    const int run = __ffs(~b) - 1;                 // first lane that is not a centroid block (lanes >= 16 never are)
    w.meta = m_meta(1, 2, 1, run, run);
  } else {
    w.meta = m_meta(2, 0, level, 1, kBlock);
  }
  return true;
}
__device__ __forceinline__ bool m_advance(const MlaDecodeParams& p, const TableEntry* table, int item_end, MWalk& w) {
  ++w.meta;                                        // sub + 1 (never carries: nsub <= 4)
  if (w.sub() < w.nsub()) return true;
  w.it += w.run();
  return m_load(p, table, item_end, w);
}
// valid rows of the current unit of a walk of kind 1 or 2
__device__ __forceinline__ int m_unit_rows(const MWalk& w) { return min(16, w.nrows() - 16 * w.sub()); }

// Start the copies of a unit into a stage (one warp, converged).  Rows past the end of a row unit
// are written as zeros so that 0 * garbage never produces a NaN.
__device__ __forceinline__ void m_issue(const MlaDecodeParams& p, const TableEntry* table, const MWalk& w, uint32_t st, uint32_t bar,
                                        int lane) {
  if (w.kind() == 0) {
    if (lane == 0) {
      const uint32_t bytes = static_cast<uint32_t>(mla_half_bytes(w.level()));
      m_expect_tx(bar, bytes);
      m_bulk_g2s(st, p.arena + static_cast<size_t>(w.off256) * 256 + static_cast<size_t>(w.sub()) * bytes, bytes, bar);
    }
    return;
  }
  const int n = m_unit_rows(w);
  if (lane == 0) m_expect_tx(bar, static_cast<uint32_t>(n) * kMlaRowBytes);
  __syncwarp();
  if (lane < n) {
    const uint8_t* src = (w.kind() == 2) ? p.arena + static_cast<size_t>(table[w.it + lane].off256) * 256
                                       : p.arena + static_cast<size_t>(w.off256) * 256 + static_cast<size_t>(16 * w.sub() + lane) * kMlaRowBytes;
    m_bulk_g2s(st + lane * kMRowPitch, src, kMlaRowBytes, bar);
  }
  if (n < 16) {
    for (int idx = lane; idx < (16 - n) * (kMlaRowBytes / 16); idx += 32) {
      const int r = n + idx / (kMlaRowBytes / 16), piece = idx % (kMlaRowBytes / 16);
      m_sts128(st + r * kMRowPitch + piece * 16, 0u, 0u, 0u, 0u);
    }
    m_fence_async();
  }
}

// ---- softmax -------------------------------------------------------------------------------------
// The four warps' partial logits -> this lane's share of the unit's probabilities.  A lane holds, for
// the heads g and g + 8, the tokens 16 ks + 8 j + 2 c4 + e: the B-fragment layout of the value MMAs.
// The running maximum may stay stale by up to kMSlack (then nothing is rescaled); when it moves, the
// running sums and O^T are rescaled.  Outputs: the probabilities as a pair hi + lo (fp16 or bf16) and
// the unit's probability sums of the heads 2 c4 + e (+ 8 hg), the columns of the lane's O^T registers.
template <int NKS, bool BF16>
__device__ __forceinline__ void m_softmax(uint32_t xb, int lane, float scale_log2, float bias, int nvalid, uint32_t ot,
                                          float (&m_run)[2], float (&l_run)[2], uint32_t (&ph)[2][NKS][2], uint32_t (&pl)[2][NKS][2],
                                          float (&psc)[2][2]) {
  const int c4 = lane & 3;
  // token group j4 (tokens 8 j4 .. 8 j4 + 7) of every warp's partial is one 16-byte piece per lane:
  // heads g (x, y) and g + 8 (z, w), tokens 8 j4 + 2 c4, + 1
  float x[2][NKS][2][2];
  float mloc[2] = {kMNegInf, kMNegInf};
#pragma unroll
  for (int j4 = 0; j4 < 2 * NKS; ++j4) {
    const uint32_t a = xb + (j4 * 32 + lane) * 16;
    float4 acc = m_ldsf4(a);
#pragma unroll
    for (int w = 1; w < 4; ++w) {
      const float4 v = m_ldsf4(a + w * 4 * 32 * 16);
      acc.x += v.x;
      acc.y += v.y;
      acc.z += v.z;
      acc.w += v.w;
    }
    const int tok = 8 * j4 + 2 * c4;
    const int ks = j4 >> 1, j = j4 & 1;
    x[0][ks][j][0] = tok < nvalid ? fmaf(acc.x, scale_log2, bias) : kMNegInf;
    x[0][ks][j][1] = tok + 1 < nvalid ? fmaf(acc.y, scale_log2, bias) : kMNegInf;
    x[1][ks][j][0] = tok < nvalid ? fmaf(acc.z, scale_log2, bias) : kMNegInf;
    x[1][ks][j][1] = tok + 1 < nvalid ? fmaf(acc.w, scale_log2, bias) : kMNegInf;
    mloc[0] = fmaxf(mloc[0], fmaxf(x[0][ks][j][0], x[0][ks][j][1]));
    mloc[1] = fmaxf(mloc[1], fmaxf(x[1][ks][j][0], x[1][ks][j][1]));
  }
#pragma unroll
  for (int hg = 0; hg < 2; ++hg) {
    mloc[hg] = fmaxf(mloc[hg], __shfl_xor_sync(kMFull, mloc[hg], 1));
    mloc[hg] = fmaxf(mloc[hg], __shfl_xor_sync(kMFull, mloc[hg], 2));
  }
  const bool mine = mloc[0] > m_run[0] + kMSlack || mloc[1] > m_run[1] + kMSlack;   // also the first finite logit (max = -inf)
  if (__any_sync(kMFull, mine)) {
    float al[2];
#pragma unroll
    for (int hg = 0; hg < 2; ++hg) {
      const float mn = fmaxf(m_run[hg], mloc[hg]);
      al[hg] = (m_run[hg] == kMNegInf) ? 0.f : m_ex2(m_run[hg] - mn);
      m_run[hg] = mn;
      l_run[hg] *= al[hg];
    }
    // the factors of the heads 2 c4 + e + 8 hg sit in the lanes whose g is 2 c4 + e
    float ac[2][2];
#pragma unroll
    for (int hg = 0; hg < 2; ++hg)
#pragma unroll
      for (int e = 0; e < 2; ++e) ac[hg][e] = __shfl_sync(kMFull, al[hg], 4 * (2 * c4 + e));
#pragma unroll 2
    for (int mu = 0; mu < 8; ++mu) {
      float o[2][4];
      m_tld8(ot + 8 * mu, o);
      m_twait_ld();
#pragma unroll
      for (int hg = 0; hg < 2; ++hg)
#pragma unroll
        for (int i = 0; i < 4; ++i) o[hg][i] *= ac[hg][i & 1];
      m_tst8(ot + 8 * mu, o);
    }
    m_twait_st();
  }
  float ps[2];
#pragma unroll
  for (int hg = 0; hg < 2; ++hg) {
    ps[hg] = 0.f;
#pragma unroll
    for (int ks = 0; ks < NKS; ++ks) {
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const float p0 = x[hg][ks][j][0] == kMNegInf ? 0.f : m_ex2(x[hg][ks][j][0] - m_run[hg]);
        const float p1 = x[hg][ks][j][1] == kMNegInf ? 0.f : m_ex2(x[hg][ks][j][1] - m_run[hg]);
        ps[hg] += p0 + p1;
        if constexpr (BF16) {
          const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
          ph[hg][ks][j] = m_ubf(h);
          pl[hg][ks][j] = m_ubf(__floats2bfloat162_rn(p0 - __low2float(h), p1 - __high2float(h)));
        } else {
          const __half2 h = __floats2half2_rn(p0, p1);
          ph[hg][ks][j] = m_u(h);
          pl[hg][ks][j] = m_u(__floats2half2_rn(p0 - __low2float(h), p1 - __high2float(h)));
        }
      }
    }
    l_run[hg] += ps[hg];
    ps[hg] += __shfl_xor_sync(kMFull, ps[hg], 1);
    ps[hg] += __shfl_xor_sync(kMFull, ps[hg], 2);
  }
#pragma unroll
  for (int hg = 0; hg < 2; ++hg)
#pragma unroll
    for (int e = 0; e < 2; ++e) psc[hg][e] = __shfl_sync(kMFull, ps[hg], 4 * (2 * c4 + e));
}

// ---- a quantised half block ---------------------------------------------------------------------
// Key MMAs of one channel slab (16 channels = the four lanes' four channels each), heads along the rows:
// S^T[head][token] += Q'^T K^T.  qa = the query entries (q[g][k0 k0+1], q[g + 8][k0 k0+1], q[g][k1 k1+1],
// q[g + 8][k1 k1+1]) of the lane's channel pairs k0 = 2 c4 and k1 = 2 c4 + 8: times the scales (s0, s1) they are
// the A fragment of Q'^T, as they are the A fragment of Q^T for sum_c q[c] z[c] (zero points (z0, z1) in
// every column of B; Zt[0] / Zt[2] = the sums of the heads g / g + 8).  a[mt] = the code registers of the
// two 16-token tiles (tokens g and g + 8, channel pairs k0 and k1): B fragments of the four 8-token groups.
template <bool FIRST>
__device__ __forceinline__ void m_slab(const uint32_t (&a)[2][4], uint32_t s0, uint32_t s1, uint32_t z0, uint32_t z1, const uint32_t (&qa)[4],
                                       float (&S)[4][4], float (&Zt)[4]) {
  uint32_t h[4], l[4];
  m_split(qa[0], s0, h[0], l[0]);
  m_split(qa[1], s0, h[1], l[1]);
  m_split(qa[2], s1, h[2], l[2]);
  m_split(qa[3], s1, h[3], l[3]);
  if (FIRST) m_mma_f16_first(Zt, qa[0], qa[1], qa[2], qa[3], z0, z1);
  else m_mma_f16(Zt, qa[0], qa[1], qa[2], qa[3], z0, z1);
  // four accumulator chains; the two MMAs of a chain are kept four apart
#pragma unroll
  for (int j4 = 0; j4 < 4; ++j4) {
    if (FIRST) m_mma_f16_first(S[j4], h[0], h[1], h[2], h[3], a[j4 >> 1][j4 & 1], a[j4 >> 1][(j4 & 1) + 2]);
    else m_mma_f16(S[j4], h[0], h[1], h[2], h[3], a[j4 >> 1][j4 & 1], a[j4 >> 1][(j4 & 1) + 2]);
  }
#pragma unroll
  for (int j4 = 0; j4 < 4; ++j4) m_mma_f16(S[j4], l[0], l[1], l[2], l[3], a[j4 >> 1][j4 & 1], a[j4 >> 1][(j4 & 1) + 2]);
}

template <int BITS>
__device__ __forceinline__ void m_unit_quant(uint32_t st, uint32_t q16, uint32_t xb, int quad, int wq, int g, int c4, float scale_log2,
                                             uint32_t ot, float (&m_run)[2], float (&l_run)[2]) {
  constexpr int RB = kMlaChunks * BITS;                    // bytes per token row of codes
  const uint32_t codes = st + mla_kp_bytes();
  const uint32_t zbase = st + 2 * kMlaZeroOff;
  const uint32_t x16 = 0x4C004C00u;                        // fp16 pair (16, 16)
  const uint32_t qrow = q16 + g * kMQPitch;                // (q[g], q[g + 8]) interleaved per channel pair
  float S[4][4], Zt[4];
  // ---- keys: four steps of 32 value channels (8 per lane = two slabs), then the rope slab ----
  // A slab takes four neighbouring channels of the lane: 8-bit word sl (bytes c0 c2 c1 c3); 4-bit fields 2 sl
  // (b = 0: weight 2^-24, its scale is taken times 16) and 2 sl + 1 (b = 4: weight 2^-20).
#pragma unroll
  for (int step = 0; step < 4; ++step) {
    const int cb = 128 * wq + 32 * step + 8 * c4;          // the lane's 8 channels
    uint32_t w[4][2];
#pragma unroll
    for (int tt = 0; tt < 4; ++tt) {
      if constexpr (BITS == 8) {
        const uint2 v = m_lds64(codes + (g + 8 * tt) * RB + cb);
        w[tt][0] = v.x;
        w[tt][1] = v.y;
      } else {
        w[tt][0] = m_lds32(codes + (g + 8 * tt) * RB + (cb >> 1));
        w[tt][1] = 0u;
      }
    }
    const uint4 s4 = m_lds128(st + 2 * cb), z4 = m_lds128(zbase + 2 * cb);
    const uint4 q4a = m_lds128(qrow + 4 * cb), q4b = m_lds128(qrow + 4 * cb + 16);
    const uint32_t sr[4] = {s4.x, s4.y, s4.z, s4.w}, zr[4] = {z4.x, z4.y, z4.z, z4.w};
    const uint32_t qr[2][4] = {{q4a.x, q4a.y, q4a.z, q4a.w}, {q4b.x, q4b.y, q4b.z, q4b.w}};
#pragma unroll
    for (int sl = 0; sl < 2; ++sl) {
      uint32_t s0 = sr[2 * sl];
      if (BITS == 4) s0 = m_u(__hmul2(m_h2(s0), m_h2(x16)));
      uint32_t a[2][4];
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        if constexpr (BITS == 8) {
          a[mt][0] = m_prmt(w[2 * mt][sl], 0u, 0x4240u);
          a[mt][1] = m_prmt(w[2 * mt + 1][sl], 0u, 0x4240u);
          a[mt][2] = m_prmt(w[2 * mt][sl], 0u, 0x4341u);
          a[mt][3] = m_prmt(w[2 * mt + 1][sl], 0u, 0x4341u);
        } else {
          a[mt][0] = sl ? m_fld4<2>(w[2 * mt][0]) : m_fld4<0>(w[2 * mt][0]);
          a[mt][1] = sl ? m_fld4<2>(w[2 * mt + 1][0]) : m_fld4<0>(w[2 * mt + 1][0]);
          a[mt][2] = sl ? m_fld4<3>(w[2 * mt][0]) : m_fld4<1>(w[2 * mt][0]);
          a[mt][3] = sl ? m_fld4<3>(w[2 * mt + 1][0]) : m_fld4<1>(w[2 * mt + 1][0]);
        }
      }
      if (step == 0 && sl == 0) m_slab<true>(a, s0, sr[2 * sl + 1], zr[2 * sl], zr[2 * sl + 1], qr[sl], S, Zt);
      else m_slab<false>(a, s0, sr[2 * sl + 1], zr[2 * sl], zr[2 * sl + 1], qr[sl], S, Zt);
    }
  }
  {
    // the rope slab: 16 channels of the warp, four per lane
    uint32_t a[2][4], s0, s1, z0, z1, qa[4];
    int cb;
    if constexpr (BITS == 8) {
      cb = kMlaDv + 16 * wq + 4 * c4;
      uint32_t w[4];
#pragma unroll
      for (int tt = 0; tt < 4; ++tt) w[tt] = m_lds32(codes + (g + 8 * tt) * RB + cb);
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        a[mt][0] = m_prmt(w[2 * mt], 0u, 0x4240u);
        a[mt][1] = m_prmt(w[2 * mt + 1], 0u, 0x4240u);
        a[mt][2] = m_prmt(w[2 * mt], 0u, 0x4341u);
        a[mt][3] = m_prmt(w[2 * mt + 1], 0u, 0x4341u);
      }
    } else {
      // the lane's word is chunk c4 / 2 of the warp's two; its fields 2 (c4 & 1) and 2 (c4 & 1) + 1
      cb = kMlaDv + 16 * wq + 8 * (c4 >> 1) + 4 * (c4 & 1);
      uint32_t w[4];
#pragma unroll
      for (int tt = 0; tt < 4; ++tt) {
        w[tt] = m_lds32(codes + (g + 8 * tt) * RB + ((kMlaDv + 16 * wq + 8 * (c4 >> 1)) >> 1));
        if (c4 & 1) w[tt] >>= 8;
      }
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        a[mt][0] = w[2 * mt] & 0x000F000Fu;
        a[mt][1] = w[2 * mt + 1] & 0x000F000Fu;
        a[mt][2] = w[2 * mt] & 0x00F000F0u;
        a[mt][3] = w[2 * mt + 1] & 0x00F000F0u;
      }
    }
    const uint2 s2 = m_lds64(st + 2 * cb), z2 = m_lds64(zbase + 2 * cb);
    const uint4 q4 = m_lds128(qrow + 4 * cb);
    s0 = BITS == 4 ? m_u(__hmul2(m_h2(s2.x), m_h2(x16))) : s2.x;
    s1 = s2.y; z0 = z2.x; z1 = z2.y;
    qa[0] = q4.x; qa[1] = q4.y; qa[2] = q4.z; qa[3] = q4.w;
    m_slab<false>(a, s0, s1, z0, z1, qa, S, Zt);
  }
  // partial logits of the warp's channels -> the exchange buffer [warp][token group][lane]: heads g and
  // g + 8, tokens 8 j4 + 2 c4, + 1
  {
    const float ks = BITS == 8 ? 16777216.f : 1048576.f;
    const int lane = 4 * g + c4;
#pragma unroll
    for (int j4 = 0; j4 < 4; ++j4)
      m_stsf4(xb + ((wq * 4 + j4) * 32 + lane) * 16, fmaf(S[j4][0], ks, Zt[0]), fmaf(S[j4][1], ks, Zt[0]), fmaf(S[j4][2], ks, Zt[2]),
              fmaf(S[j4][3], ks, Zt[2]));
  }
  m_quad_sync(quad);
  uint32_t ph[2][2][2], pl[2][2][2];
  float psc[2][2];
  m_softmax<2, false>(xb, 4 * g + c4, scale_log2, 0.f, 32, ot, m_run, l_run, ph, pl, psc);
  // ---- values: the warp's 128 channels, 16 per lane group; two passes of four M-tiles ----
#pragma unroll
  for (int hp = 0; hp < 2; ++hp) {
    const int cv = 128 * wq + 16 * g + 8 * hp;               // channels of this pass
    uint32_t w[2][4][2];                                     // [k-step][token 2 c4, 2 c4 + 1, 2 c4 + 8, 2 c4 + 9][word]
#pragma unroll
    for (int ks = 0; ks < 2; ++ks)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int tok = 16 * ks + 2 * c4 + (i & 1) + 8 * (i >> 1);
        if constexpr (BITS == 8) {
          const uint2 v = m_lds64(codes + tok * RB + cv);
          w[ks][i][0] = v.x;
          w[ks][i][1] = v.y;
        } else {
          w[ks][i][0] = m_lds32(codes + tok * RB + (cv >> 1));
          w[ks][i][1] = 0u;
        }
      }
    const uint4 s4 = m_lds128(st + 2 * cv), z4 = m_lds128(zbase + 2 * cv);
    const uint32_t sr[4] = {s4.x, s4.y, s4.z, s4.w}, zr[4] = {z4.x, z4.y, z4.z, z4.w};
    uint32_t lo01[2], hi01[2], lo23[2], hi23[2];             // 4-bit: the token pairs' low and high halves
    if constexpr (BITS == 4) {
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        lo01[ks] = m_prmt(w[ks][0][0], w[ks][1][0], 0x5410u);
        hi01[ks] = m_prmt(w[ks][0][0], w[ks][1][0], 0x7632u);
        lo23[ks] = m_prmt(w[ks][2][0], w[ks][3][0], 0x5410u);
        hi23[ks] = m_prmt(w[ks][2][0], w[ks][3][0], 0x7632u);
      }
    }
#pragma unroll
    for (int m4 = 0; m4 < 4; ++m4) {
      // M-tile mu = 4 hp + m4: row g = channel cv + 2 m4, row g + 8 = channel cv + 2 m4 + 1
      const int mu = 4 * hp + m4;
      float T[2][4], o[2][4];
      m_tld8(ot + 8 * mu, o);                                // this M-tile's rows of O^T, asked for before the MMAs
#pragma unroll
      for (int ks = 0; ks < 2; ++ks) {
        uint32_t a0, a1, a2, a3;
        if constexpr (BITS == 8) {
          // word m4 / 2 holds the channels 4 (m4 / 2) + (0, 2, 1, 3); the pair 2 (m4 & 1), 2 (m4 & 1) + 1 sits in the
          // bytes (m4 & 1) and (m4 & 1) + 2
          const uint32_t sel = (m4 & 1) ? 0x7531u : 0x6420u;
          const uint32_t y01 = m_prmt(w[ks][0][m4 >> 1], w[ks][1][m4 >> 1], sel);
          const uint32_t y23 = m_prmt(w[ks][2][m4 >> 1], w[ks][3][m4 >> 1], sel);
          a0 = m_prmt(y01, 0u, 0x4240u);
          a1 = m_prmt(y01, 0u, 0x4341u);
          a2 = m_prmt(y23, 0u, 0x4240u);
          a3 = m_prmt(y23, 0u, 0x4341u);
        } else {
          a0 = m4 == 0 ? m_fld4<0>(lo01[ks]) : (m4 == 1 ? m_fld4<1>(lo01[ks]) : (m4 == 2 ? m_fld4<2>(lo01[ks]) : m_fld4<3>(lo01[ks])));
          a1 = m4 == 0 ? m_fld4<0>(hi01[ks]) : (m4 == 1 ? m_fld4<1>(hi01[ks]) : (m4 == 2 ? m_fld4<2>(hi01[ks]) : m_fld4<3>(hi01[ks])));
          a2 = m4 == 0 ? m_fld4<0>(lo23[ks]) : (m4 == 1 ? m_fld4<1>(lo23[ks]) : (m4 == 2 ? m_fld4<2>(lo23[ks]) : m_fld4<3>(lo23[ks])));
          a3 = m4 == 0 ? m_fld4<0>(hi23[ks]) : (m4 == 1 ? m_fld4<1>(hi23[ks]) : (m4 == 2 ? m_fld4<2>(hi23[ks]) : m_fld4<3>(hi23[ks])));
        }
#pragma unroll
        for (int hg = 0; hg < 2; ++hg) {
          if (ks == 0) m_mma_f16_first(T[hg], a0, a1, a2, a3, ph[hg][ks][0], ph[hg][ks][1]);
          else m_mma_f16(T[hg], a0, a1, a2, a3, ph[hg][ks][0], ph[hg][ks][1]);
        }
#pragma unroll
        for (int hg = 0; hg < 2; ++hg) m_mma_f16(T[hg], a0, a1, a2, a3, pl[hg][ks][0], pl[hg][ks][1]);
      }
      const float un = (BITS == 4 && (m4 & 1)) ? 1048576.f : 16777216.f;   // 2^(24 - b)
      const float sa = m_h2f(sr[m4], 0) * un, sb = m_h2f(sr[m4], 1) * un;
      const float za = m_h2f(zr[m4], 0), zb = m_h2f(zr[m4], 1);
      m_twait_ld();
#pragma unroll
      for (int hg = 0; hg < 2; ++hg) {
        o[hg][0] = fmaf(T[hg][0], sa, fmaf(za, psc[hg][0], o[hg][0]));
        o[hg][1] = fmaf(T[hg][1], sa, fmaf(za, psc[hg][1], o[hg][1]));
        o[hg][2] = fmaf(T[hg][2], sb, fmaf(zb, psc[hg][0], o[hg][2]));
        o[hg][3] = fmaf(T[hg][3], sb, fmaf(zb, psc[hg][1], o[hg][3]));
      }
      m_tst8(ot + 8 * mu, o);
    }
  }
  m_twait_st();
}

// ---- 16 bf16 rows (an exact tile, the tail, a run of centroid rows) ---------------------------------
__device__ __forceinline__ void m_unit_rows16(uint32_t st, uint32_t qt, uint32_t xb, int quad, int wq, int lane, float scale_log2,
                                              float bias, int nvalid, uint32_t ot, float (&m_run)[2], float (&l_run)[2]) {
  const int g = lane >> 2, c4 = lane & 3;
  // keys, heads along the rows: the A fragment is the query (bf16), the ldmatrix registers are the B fragments
  // of the two 8-token groups
  float S[2][4];
#pragma unroll
  for (int j4 = 0; j4 < 2; ++j4)
#pragma unroll
    for (int i = 0; i < 4; ++i) S[j4][i] = 0.f;
  const uint32_t arow = st + (lane & 15) * kMRowPitch + 16 * (lane >> 4);
  // (the bf16 query fragments of the warp's nine slabs wait in tensor memory)
  uint32_t qa[9][4];
#pragma unroll
  for (int sl = 0; sl < 9; ++sl) m_tld4(qt + 4 * sl, qa[sl]);
  m_twait_ld();
#pragma unroll
  for (int sl = 0; sl < 9; ++sl) {
    const int ch0 = sl < 8 ? 128 * wq + 16 * sl : kMlaDv + 16 * wq;
    uint32_t a[4];
    m_ldmatrix4(arow + 2 * ch0, a);
    m_mma_bf16(S[0], qa[sl][0], qa[sl][1], qa[sl][2], qa[sl][3], a[0], a[2]);
    m_mma_bf16(S[1], qa[sl][0], qa[sl][1], qa[sl][2], qa[sl][3], a[1], a[3]);
  }
#pragma unroll
  for (int j4 = 0; j4 < 2; ++j4) m_stsf4(xb + ((wq * 4 + j4) * 32 + lane) * 16, S[j4][0], S[j4][1], S[j4][2], S[j4][3]);
  m_quad_sync(quad);
  uint32_t ph[2][1][2], pl[2][1][2];
  float psc[2][2];
  m_softmax<1, true>(xb, lane, scale_log2, bias, nvalid, ot, m_run, l_run, ph, pl, psc);
  // values: channel pairs (2 mu, 2 mu + 1) of the lane group's 16 channels from the tokens 2 c4, 2 c4 + 1, 2 c4 + 8, 2 c4 + 9
#pragma unroll
  for (int hp = 0; hp < 2; ++hp) {
    uint32_t w[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int tok = 2 * c4 + (i & 1) + 8 * (i >> 1);
      const uint4 v = m_lds128(st + tok * kMRowPitch + 2 * (128 * wq + 16 * g + 8 * hp));
      w[i][0] = v.x; w[i][1] = v.y; w[i][2] = v.z; w[i][3] = v.w;
    }
#pragma unroll
    for (int m4 = 0; m4 < 4; ++m4) {
      const int mu = 4 * hp + m4;
      const uint32_t a0 = m_prmt(w[0][m4], w[1][m4], 0x5410u), a1 = m_prmt(w[0][m4], w[1][m4], 0x7632u);
      const uint32_t a2 = m_prmt(w[2][m4], w[3][m4], 0x5410u), a3 = m_prmt(w[2][m4], w[3][m4], 0x7632u);
      float o[2][4];
      m_tld8(ot + 8 * mu, o);
      m_twait_ld();
#pragma unroll
      for (int hg = 0; hg < 2; ++hg) {
        m_mma_bf16(o[hg], a0, a1, a2, a3, ph[hg][0][0], ph[hg][0][1]);
        m_mma_bf16(o[hg], a0, a1, a2, a3, pl[hg][0][0], pl[hg][0][1]);
      }
      m_tst8(ot + 8 * mu, o);
    }
  }
  m_twait_st();
}

// ---- kernel --------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kMThreads, 1) mla_decode_kernel(const __grid_constant__ MlaDecodeParams p) {
  extern __shared__ __align__(128) uint8_t msm[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int quad = warp >> 2, wq = warp & 3, g = lane >> 2, c4 = lane & 3;
  const WarpDesc cd = p.ctas[blockIdx.x * kMlaQuads + quad];
  if (p.ctas[blockIdx.x * kMlaQuads].stream < 0) return;        // uniform for the CTA
  const uint32_t base = m_u32(msm);
  const uint32_t q16 = base + kMOffQ16;
  const uint32_t qd = base + kMOffQuad + quad * kMQuadBytes;
  const uint32_t xb = qd + kMStages * kMStageBytes, bars = xb + kMXBytes;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(msm + kMOffFlag);
  const TableEntry* table = p.table + static_cast<size_t>(cd.stream) * p.table_stride;
  const uint16_t* qg = p.q + static_cast<size_t>(cd.stream) * kMlaHeads * kMlaDk;

  // (launched with programmatic stream serialisation as well: nothing above reads what an earlier kernel of the
  // stream may have written; the table, the query and the cache are touched after this wait)
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  if (tid == 0) *abort_flag = 0;
  if (wq == 0 && lane == 0) {
    m_bar_init(bars, 1);
    m_bar_init(bars + 8, 1);
    m_fence_async();
  }
  if (warp == 0) m_tmem_alloc(base + kMOffFlag + 4, kMTmemCols);
  {
    // the query as fp16 (exact for the magnitudes a query has), the heads g and g + 8 interleaved per channel pair
    for (int idx = tid; idx < 8 * kMlaChunks; idx += kMThreads) {
      const int hp = idx / kMlaChunks, piece = idx % kMlaChunks;
      const uint4 v0 = *reinterpret_cast<const uint4*>(qg + hp * kMlaDk + 8 * piece);
      const uint4 v1 = *reinterpret_cast<const uint4*>(qg + (hp + 8) * kMlaDk + 8 * piece);
      const uint32_t d = hp * kMQPitch + 32 * piece;
      m_sts128(q16 + d, m_bf2_to_h2(v0.x), m_bf2_to_h2(v1.x), m_bf2_to_h2(v0.y), m_bf2_to_h2(v1.y));
      m_sts128(q16 + d + 16, m_bf2_to_h2(v0.z), m_bf2_to_h2(v1.z), m_bf2_to_h2(v0.w), m_bf2_to_h2(v1.w));
    }
  }
  m_tfence_before();
  __syncthreads();
  m_tfence_after();
  // this warp's 64 columns of its lane quarter: the running O^T, zero to begin with
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(msm + kMOffFlag + 4);
  const uint32_t ot = tmem + (static_cast<uint32_t>(32 * wq) << 16) + 64u * static_cast<uint32_t>(quad);
  {
    const float zero[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
    for (int mu = 0; mu < 8; ++mu) m_tst8(ot + 8 * mu, zero);
    m_twait_st();
  }
  // the bf16 query as the A fragments of the warp's nine channel slabs (rows = heads g and g + 8), for the units of
  // exact and centroid rows
  const uint32_t qt = tmem + (static_cast<uint32_t>(32 * wq) << 16) + kMTmemQ + 36u * static_cast<uint32_t>(quad);
  {
    const uint16_t* qa = qg + g * kMlaDk + 2 * c4;
#pragma unroll 3
    for (int sl = 0; sl < 9; ++sl) {
      const int ch0 = sl < 8 ? 128 * wq + 16 * sl : kMlaDv + 16 * wq;
      const uint32_t f[4] = {m_ldg32(qa + ch0), m_ldg32(qa + 8 * kMlaDk + ch0), m_ldg32(qa + ch0 + 8), m_ldg32(qa + 8 * kMlaDk + ch0 + 8)};
      m_tst4(qt + 4 * sl, f);
    }
    m_twait_st();
  }
  float m_run[2] = {kMNegInf, kMNegInf}, l_run[2] = {0.f, 0.f};

  MWalk wc, wl;
  wc.it = cd.item_begin;
  bool have_c = m_load(p, table, cd.item_end, wc);
  wl = wc;
  bool have_l = have_c;
  // the first two units' copies
#pragma unroll 1
  for (int i = 0; i < kMStages; ++i) {
    if (have_l) {
      if (wq == 0) m_issue(p, table, wl, qd + i * kMStageBytes, bars + 8 * i, lane);
      have_l = m_advance(p, table, cd.item_end, wl);
    }
  }
  int k = 0;
#pragma unroll 1
  while (have_c) {
    const int s = k & 1;
    const uint32_t st = qd + s * kMStageBytes;
    // after a time-out nothing waits any more: the remaining units run through on whatever the stages hold
    if (!*abort_flag && !m_wait(bars + 8 * s, (k >> 1) & 1)) *abort_flag = 1;
    if (wc.kind() == 0) {
      if (wc.level() == 8) m_unit_quant<8>(st, q16, xb, quad, wq, g, c4, p.scale_log2, ot, m_run, l_run);
      else m_unit_quant<4>(st, q16, xb, quad, wq, g, c4, p.scale_log2, ot, m_run, l_run);
    } else {
      m_unit_rows16(st, qt, xb, quad, wq, lane, p.scale_log2, wc.kind() == 2 ? 6.0f : 0.f, m_unit_rows(wc), ot, m_run, l_run);
    }
    // the stage and the exchange buffer are free once all four warps are here
    m_quad_sync(quad);
    if (have_l) {
      if (wq == 0) m_issue(p, table, wl, st, bars + 8 * s, lane);
      have_l = m_advance(p, table, cd.item_end, wl);
    }
    have_c = m_advance(p, table, cd.item_end, wc);
    ++k;
  }

  // ---- the quad's result into its (now idle) stages: O^T as [head][channel], then m and l ----
  {
    float l[2];
#pragma unroll
    for (int hg = 0; hg < 2; ++hg) {
      l[hg] = l_run[hg] + __shfl_xor_sync(kMFull, l_run[hg], 1);
      l[hg] += __shfl_xor_sync(kMFull, l[hg], 2);
    }
#pragma unroll 2
    for (int mu = 0; mu < 8; ++mu) {
      float o[2][4];
      m_tld8(ot + 8 * mu, o);
      m_twait_ld();
#pragma unroll
      for (int hg = 0; hg < 2; ++hg)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int head = 8 * hg + 2 * c4 + e, ch = 128 * wq + 16 * g + 2 * mu;
          m_stsf2(qd + (head * kMOutPitch + ch) * 4, o[hg][e], o[hg][e + 2]);
        }
    }
    if (wq == 0 && c4 == 0) {
#pragma unroll
      for (int hg = 0; hg < 2; ++hg) {
        m_stsf(qd + (kMlaHeads * kMOutPitch + g + 8 * hg) * 4, m_run[hg]);
        m_stsf(qd + (kMlaHeads * kMOutPitch + 16 + g + 8 * hg) * 4, l[hg]);
      }
    }
  }
  __syncthreads();
  // ---- merge of the quads in quad order -> the CTA's partial row ----
  {
    const bool good = !*abort_flag;
    float* out = p.partial + static_cast<size_t>(cd.partial) * kMlaPartialFloats;
    const float* sm = reinterpret_cast<const float*>(msm + kMOffQuad);
    constexpr int kQF = kMQuadBytes / 4;                      // floats between two quads' results
    for (int idx = tid; idx < kMlaHeads * kMlaDv; idx += kMThreads) {
      const int head = idx / kMlaDv, ch = idx % kMlaDv;
      float M = kMNegInf;
#pragma unroll
      for (int qn = 0; qn < kMlaQuads; ++qn) M = fmaxf(M, sm[qn * kQF + kMlaHeads * kMOutPitch + head]);
      float acc = 0.f, L = 0.f;
#pragma unroll
      for (int qn = 0; qn < kMlaQuads; ++qn) {
        const float mq = sm[qn * kQF + kMlaHeads * kMOutPitch + head];
        const float wgt = (mq == kMNegInf) ? 0.f : exp2f(mq - M);
        acc = fmaf(wgt, sm[qn * kQF + head * kMOutPitch + ch], acc);
        L = fmaf(wgt, sm[qn * kQF + kMlaHeads * kMOutPitch + 16 + head], L);
      }
      out[head * (kMlaDv + 2) + 2 + ch] = good ? acc : 0.f;
      if (ch == 0) {
        out[head * (kMlaDv + 2)] = good ? M : kMNegInf;
        out[head * (kMlaDv + 2) + 1] = good ? L : 0.f;
      }
    }
  }
  if (tid == 0 && *abort_flag) atomicOr(p.status, kStatusInternal);
  m_tfence_before();
  __syncthreads();
  if (warp == 0) m_tmem_dealloc(tmem, kMTmemCols);
}

// Merge the partial rows of a stream's CTAs.  One block per (stream, head, slice of 64 value
// channels); its 512 threads are 8 row groups x 64 channels, row group g sums rows g, g + 8, ...
// in that order and the 8 sums are added in group order, so the result is bitwise reproducible.
constexpr int kCombSlice = 64, kCombGroups = 8, kCombThreads = kCombSlice * kCombGroups;
__global__ void __launch_bounds__(kCombThreads) mla_combine_kernel(const float* partial, const StreamParts* parts, float* out,
                                                                   float* lse) {
  __shared__ float sm_m[kCombThreads], sm_w[kCombThreads], sm_acc[kCombGroups][kCombSlice];
  // launched with programmatic stream serialisation: the launch overlaps the decode kernel's tail, the
  // partial rows are touched only after that kernel has completed
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  const int stream = blockIdx.x, h = blockIdx.y, slice = blockIdx.z, tid = threadIdx.x;
  const int c = tid % kCombSlice, g = tid / kCombSlice;
  const int begin = parts[stream].begin, end = parts[stream].end;
  const float* base = partial + h * (kMlaDv + 2);
  // pass 1: the maximum of the rows' maxima (one row per thread, then a shared-memory sweep)
  float M = kMNegInf;
  for (int c0 = begin; c0 < end; c0 += kCombThreads) {
    const int n = min(kCombThreads, end - c0);
    __syncthreads();
    sm_m[tid] = tid < n ? __ldcg(base + static_cast<size_t>(c0 + tid) * kMlaPartialFloats) : kMNegInf;
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
      const float w = (m == kMNegInf) ? 0.f : exp2f(m - M);
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
    if (lse && slice == 0 && c == 0) lse[hq] = (L > 0.f) ? (M + log2f(L)) * 0.6931471805599453f : kMNegInf;
  }
}

}  // namespace

cudaError_t launch_mla_decode(const MlaDecodeParams& p, int n_ctas, const StreamParts* parts, int n_streams, float* out,
                              float* lse, cudaStream_t st) {
  if (n_ctas <= 0) return cudaSuccess;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(mla_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMSmem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_ctas);
  cfg.blockDim = dim3(kMThreads);
  cfg.dynamicSmemBytes = kMSmem;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, mla_decode_kernel, p);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cc = {};
  cc.gridDim = dim3(n_streams, kMlaHeads, kMlaDv / kCombSlice);
  cc.blockDim = dim3(kCombThreads);
  cc.stream = st;
  cc.attrs = attr;
  cc.numAttrs = 1;
  return cudaLaunchKernelEx(&cc, mla_combine_kernel, static_cast<const float*>(p.partial), parts, out, lse);
}

}  // namespace gkv
