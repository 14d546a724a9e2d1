// Latent-attention (MLA) streams: one 576-wide row per token (512 latent + 64 rope channels),
// 16 query heads on one stream, values = channels [0, 512) of the same row.  The row is stored
// once on the precision ladder with the key rule (groups of 32 tokens x 1 channel, paper
// Sec. 3.2) and read twice by the attention kernel: as K (contraction over the 576 channels) and
// as V (contraction over tokens) - from one staged copy, so every byte crosses HBM once.
//
// decode: one CTA of 8 warps owns a contiguous range of blocks.  Per step (32 quantised tokens or
// 16 exact rows) the 36 sixteen-channel slices of the key contraction are split over the warps,
// the partial logits are summed through shared memory, every warp runs the same online softmax,
// and warp w accumulates value channels [64 w, 64 w + 64) for all 16 heads.  The value role
// transposes the unpacked 8x8 code fragments in registers (movmatrix); its per-channel scale is
// applied to the accumulator after the MMA, the code bias / centre and the zero points are taken
// out with two small MMAs on P.  Staging is a double-buffered TMA bulk-copy pipeline on per-stage
// mbarriers with bounded waits.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gkv_internal.h"
#include "gkv_mla.h"

namespace gkv {
namespace {

constexpr unsigned kFullM = 0xffffffffu;
constexpr float kNegInfM = -__builtin_huge_valf();
constexpr int kMlaWarps = 8;
constexpr int kMlaRowPitch = kMlaRowBytes + 16;                         // 1168: conflict-free ldmatrix
constexpr int kMlaStageBytes = 2 * 1152 * 8 + 2304;                     // int8 half = 20736 (>= 16 x 1168)
constexpr int kMlaQBytes = kMlaKSteps * 2 * 32 * 8;                     // one B-fragment image of q: 18432
constexpr int kMlaXchgBytes = kMlaWarps * 2 * 2 * 32 * 16;              // partial logits: 16384
constexpr int kMlaSmem = 2 * kMlaStageBytes + 2 * kMlaQBytes + kMlaXchgBytes + 64;
constexpr uint32_t kOnes = 0x3C003C00u;
constexpr int kMlaWaitSpins = 1 << 20;

__device__ __forceinline__ uint32_t s_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void m_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void m_fence() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void m_expect(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void m_bulk(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ bool m_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(2000u)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint4 l128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 l64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t l32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ float4 l128f(uint32_t a) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ void s128f(uint32_t a, float x, float y, float z, float w) {
  asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};\n" ::"r"(a), "f"(x), "f"(y), "f"(z), "f"(w) : "memory");
}
__device__ __forceinline__ void ldsm4(uint32_t (&a)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t (&a)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3])
               : "r"(addr));
}
__device__ __forceinline__ uint32_t movt(uint32_t x) {
  uint32_t y;
  asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}
__device__ __forceinline__ void mma_h(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                      uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_b(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t lop_ao(uint32_t x, uint32_t mask, uint32_t orv) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;\n" : "=r"(r) : "r"(x), "r"(mask), "r"(orv));
  return r;
}
__device__ __forceinline__ uint32_t prm(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;\n" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}
__device__ __forceinline__ uint32_t hmul2u(uint32_t a, uint32_t b) {
  __half2 r = __hmul2(*reinterpret_cast<__half2*>(&a), *reinterpret_cast<__half2*>(&b));
  return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float h_lo(uint32_t u) { return __half2float(__ushort_as_half(static_cast<unsigned short>(u & 0xffffu))); }
__device__ __forceinline__ float h_hi(uint32_t u) { return __half2float(__ushort_as_half(static_cast<unsigned short>(u >> 16))); }
__device__ __forceinline__ uint32_t bf2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bflo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bfhi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ float bfbits(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }
__device__ __forceinline__ uint16_t f2bf(float x) {
  __nv_bfloat16 h = __float2bfloat16_rn(x);
  return *reinterpret_cast<uint16_t*>(&h);
}
__device__ __forceinline__ uint16_t f2h_sat(float x) {
  x = fminf(fmaxf(x, -65504.f), 65504.f);
  __half h = __float2half_rn(x);
  return *reinterpret_cast<uint16_t*>(&h);
}
__device__ __forceinline__ float hbits(uint16_t b) { return __half2float(*reinterpret_cast<__half*>(&b)); }

// Code biases of the K-role fragments (rows r / rows r + 8) and the centre used on the value side.
template <int BITS>
struct MB;
template <>
struct MB<8> {
  static constexpr float lo = 1024.f, hi = 1024.f, mid = 127.5f, vmid = 128.f;
  static constexpr uint32_t clo = 0x64806480u, chi = 0x64806480u;      // half2(1152): bias + vmid
};
template <>
struct MB<4> {
  static constexpr float lo = 256.f, hi = 16.f, mid = 7.5f, vmid = 7.5f;
  static constexpr uint32_t clo = 0x5C1E5C1Eu, chi = 0x4DE04DE0u;      // half2(263.5), half2(23.5)
};

template <int BITS>
__device__ __forceinline__ void unpack_k(uint32_t w0, uint32_t w1, uint32_t (&a)[4]) {
  if constexpr (BITS == 8) {
    constexpr uint32_t kMagic = 0x64006400u;
    a[0] = prm(w0, kMagic, 0x5250u);
    a[1] = prm(w0, kMagic, 0x5351u);
    a[2] = prm(w1, kMagic, 0x5250u);
    a[3] = prm(w1, kMagic, 0x5351u);
  } else {
    const uint32_t v0 = w0 << 2, v1 = w0 >> 6;
    a[0] = lop_ao(v0, 0x003C003Cu, 0x5C005C00u);
    a[1] = lop_ao(v0, 0x03C003C0u, 0x4C004C00u);
    a[2] = lop_ao(v1, 0x003C003Cu, 0x5C005C00u);
    a[3] = lop_ao(v1, 0x03C003C0u, 0x4C004C00u);
  }
}

// ---------------------------------------------------------------------------------------------
// encode / requantise one block [64][576] (key rule only), centroid, exact rows
// ---------------------------------------------------------------------------------------------
constexpr int kMTileLd = kMlaDk + 1;

__device__ __forceinline__ int mla_read_code(const uint8_t* slot, int bits, int tok, int ch) {
  int tile, lane, s, a, hlf;
  k_coord(tok, ch, &tile, &lane, &s, &a, &hlf);
  int boff, bit;
  mla_code_pos(bits, lane, s, a, hlf, &boff, &bit);
  const uint8_t* region = slot + (tile >> 1) * mla_half_bytes(bits) + mla_kp_bytes() + (tile & 1) * mla_code_bytes_per_tile(bits);
  const uint32_t w = *reinterpret_cast<const uint32_t*>(region + boff);
  return static_cast<int>((w >> bit) & ((1u << bits) - 1u));
}

__global__ void __launch_bounds__(256) mla_encode_kernel(const __grid_constant__ MlaEncodeParams p) {
  extern __shared__ __align__(16) uint8_t esm[];
  float* tile = reinterpret_cast<float*>(esm);                              // [64][577]
  uint8_t* codes = esm + kBlock * kMTileLd * sizeof(float);                 // [64][576]
  const int tid = threadIdx.x;
  for (int j = blockIdx.x; j < p.n_jobs; j += gridDim.x) {
    const EncodeJob job = p.jobs[j];
    uint8_t* dst = p.arena + static_cast<size_t>(job.dst_off256) * 256;
    const int L = job.dst_level;
    __syncthreads();
    // ---- current reconstruction of the block in fp32 ----
    if (job.src_level == 0) {
      const uint16_t* in = p.k_in + (static_cast<size_t>(job.stream) * p.n_tok + static_cast<size_t>(job.block) * kBlock) * kMlaDk;
      for (int i = tid; i < kBlock * kMlaDk; i += blockDim.x) tile[(i / kMlaDk) * kMTileLd + i % kMlaDk] = bfbits(in[i]);
    } else {
      const uint8_t* slot = p.arena + static_cast<size_t>(job.src_off256) * 256;
      if (job.src_level == 16) {
        const uint16_t* rows = reinterpret_cast<const uint16_t*>(slot);
        for (int i = tid; i < kBlock * kMlaDk; i += blockDim.x) tile[(i / kMlaDk) * kMTileLd + i % kMlaDk] = bfbits(rows[i]);
      } else {
        const int bits = job.src_level;
        for (int i = tid; i < kBlock * kMlaDk; i += blockDim.x) {
          const int t = i / kMlaDk, c = i % kMlaDk;
          const int code = mla_read_code(slot, bits, t, c);
          const uint16_t* kp = reinterpret_cast<const uint16_t*>(slot + (t >> 5) * mla_half_bytes(bits));
          const int idx = kp_index(c);
          tile[t * kMTileLd + c] = __fmaf_rn(static_cast<float>(code), hbits(kp[idx]), hbits(kp[idx + 2]));
        }
      }
    }
    __syncthreads();
    if (L == 16) {
      uint16_t* rows = reinterpret_cast<uint16_t*>(dst);
      for (int i = tid; i < kBlock * kMlaDk; i += blockDim.x) rows[i] = f2bf(tile[(i / kMlaDk) * kMTileLd + i % kMlaDk]);
    } else if (L == 1) {
      for (int c = tid; c < kMlaDk; c += blockDim.x) {
        float acc = 0.f;
        for (int t = 0; t < kBlock; ++t) acc = __fadd_rn(acc, tile[t * kMTileLd + c]);
        reinterpret_cast<uint16_t*>(dst)[c] = f2bf(__fmul_rn(acc, 1.0f / kBlock));
      }
    } else {
      const float qmax = static_cast<float>((1 << L) - 1);
      bool range = false;
      for (int g = tid; g < 2 * kMlaDk; g += blockDim.x) {
        const int half = g / kMlaDk, c = g % kMlaDk;
        float mn = tile[(32 * half) * kMTileLd + c], mx = mn;
        for (int t = 1; t < kGroup; ++t) {
          const float x = tile[(32 * half + t) * kMTileLd + c];
          mn = fminf(mn, x);
          mx = fmaxf(mx, x);
        }
        const float s_raw = __fdiv_rn(__fsub_rn(mx, mn), qmax);
        range |= fabsf(s_raw) > 65504.f || fabsf(mn) > 65504.f;
        const uint16_t sb = f2h_sat(s_raw), zb = f2h_sat(mn);
        const float s32 = hbits(sb), z32 = hbits(zb);
        const float inv = s32 > 0.f ? __fdiv_rn(1.f, s32) : 0.f;
        for (int t = 0; t < kGroup; ++t) {
          const float v = __fmul_rn(__fsub_rn(tile[(32 * half + t) * kMTileLd + c], z32), inv);
          codes[(32 * half + t) * kMlaDk + c] = static_cast<uint8_t>(fminf(fmaxf(rintf(v), 0.f), qmax));
        }
        uint16_t* kp = reinterpret_cast<uint16_t*>(dst + half * mla_half_bytes(L));
        const int idx = kp_index(c);
        kp[idx] = sb;
        kp[idx + 2] = zb;
      }
      if (range) atomicOr(p.status, kStatusRange);
      __syncthreads();
      // pack fragment-ordered words: 4 tiles x 32 lanes x (9 L) words
      const int wpl = 9 * L;
      for (int i = tid; i < 4 * 32 * wpl; i += blockDim.x) {
        const int w = i % wpl, lane = (i / wpl) & 31, tl = i / (wpl * 32);
        const int r = lane >> 2, c4 = lane & 3;
        uint32_t word = 0;
        const int s0 = (L == 8) ? (w >> 1) : w;
        for (int a = 0; a < 4; ++a)
          for (int hlf = 0; hlf < 2; ++hlf) {
            int boff, bit;
            mla_code_pos(L, lane, s0, a, hlf, &boff, &bit);
            if (boff != (w * 32 + lane) * 4) continue;
            const int tok = 16 * tl + r + 8 * (a & 1);
            const int ch = 16 * s0 + 8 * (a >> 1) + 2 * c4 + hlf;
            word |= static_cast<uint32_t>(codes[tok * kMlaDk + ch]) << bit;
          }
        uint8_t* region = dst + (tl >> 1) * mla_half_bytes(L) + mla_kp_bytes() + (tl & 1) * mla_code_bytes_per_tile(L);
        *reinterpret_cast<uint32_t*>(region + (w * 32 + lane) * 4) = word;
      }
    }
  }
}

__global__ void __launch_bounds__(288) mla_append_rows_kernel(uint8_t* arena, const TableEntry* table, int table_stride,
                                                              int tail_index, const uint16_t* k_in, int n_tok,
                                                              int first_tok, int dst_row0) {
  const int stream = blockIdx.x, row = blockIdx.y;
  const TableEntry e = table[static_cast<size_t>(stream) * table_stride + tail_index];
  const uint32_t* src = reinterpret_cast<const uint32_t*>(k_in + (static_cast<size_t>(stream) * n_tok + first_tok + row) * kMlaDk);
  uint32_t* dst = reinterpret_cast<uint32_t*>(arena + static_cast<size_t>(e.off256) * 256 +
                                              static_cast<size_t>(dst_row0 + row) * kMlaRowBytes);
  dst[threadIdx.x] = src[threadIdx.x];
}

__global__ void __launch_bounds__(256) mla_export_kernel(const uint8_t* arena, uint32_t off256, int level, uint8_t* codes,
                                                         uint16_t* scale, uint16_t* zero, uint16_t* rows) {
  const uint8_t* slot = arena + static_cast<size_t>(off256) * 256;
  const int tid = threadIdx.x;
  if (level == 16) {
    for (int i = tid; i < kBlock * kMlaDk; i += blockDim.x) rows[i] = reinterpret_cast<const uint16_t*>(slot)[i];
    return;
  }
  if (level == 1) {
    for (int i = tid; i < kMlaDk; i += blockDim.x) rows[i] = reinterpret_cast<const uint16_t*>(slot)[i];
    return;
  }
  for (int i = tid; i < kBlock * kMlaDk; i += blockDim.x) codes[i] = static_cast<uint8_t>(mla_read_code(slot, level, i / kMlaDk, i % kMlaDk));
  for (int g = tid; g < 2 * kMlaDk; g += blockDim.x) {
    const int half = g / kMlaDk, c = g % kMlaDk;
    const uint16_t* kp = reinterpret_cast<const uint16_t*>(slot + half * mla_half_bytes(level));
    scale[g] = kp[kp_index(c)];
    zero[g] = kp[kp_index(c) + 2];
  }
}

// ---------------------------------------------------------------------------------------------
// decode
// ---------------------------------------------------------------------------------------------
struct MState {
  float m[2][2];       // running max (log2) of heads {8 n + 2 c4, 8 n + 2 c4 + 1}
  float l[2][2];       // lane-partial sums
  float o[4][2][4];    // channels 64 w + 16 u + {r, r + 8} x heads of n-tile n
};

// online softmax over NT tiles for both head tiles; S in / P out
template <int NT>
__device__ __forceinline__ void m_softmax(float (&S)[2][2][4], MState& st) {
#pragma unroll
  for (int n = 0; n < 2; ++n) {
    float mx0 = kNegInfM, mx1 = kNegInfM;
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      mx0 = fmaxf(mx0, fmaxf(S[t][n][0], S[t][n][2]));
      mx1 = fmaxf(mx1, fmaxf(S[t][n][1], S[t][n][3]));
    }
#pragma unroll
    for (int d = 4; d <= 16; d <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(kFullM, mx0, d));
      mx1 = fmaxf(mx1, __shfl_xor_sync(kFullM, mx1, d));
    }
    const float mn0 = fmaxf(st.m[n][0], mx0), mn1 = fmaxf(st.m[n][1], mx1);
    const float ms0 = (mn0 == kNegInfM) ? 0.f : mn0, ms1 = (mn1 == kNegInfM) ? 0.f : mn1;
    if (__any_sync(kFullM, mn0 != st.m[n][0] || mn1 != st.m[n][1])) {
      const float al0 = ex2(st.m[n][0] - ms0), al1 = ex2(st.m[n][1] - ms1);
      st.m[n][0] = mn0;
      st.m[n][1] = mn1;
      st.l[n][0] *= al0;
      st.l[n][1] *= al1;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        st.o[u][n][0] *= al0;
        st.o[u][n][1] *= al1;
        st.o[u][n][2] *= al0;
        st.o[u][n][3] *= al1;
      }
    }
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      S[t][n][0] = ex2(S[t][n][0] - ms0);
      S[t][n][1] = ex2(S[t][n][1] - ms1);
      S[t][n][2] = ex2(S[t][n][2] - ms0);
      S[t][n][3] = ex2(S[t][n][3] - ms1);
    }
  }
}

// sum the 8 warps' partial logits (fixed order) and write them back into S
template <int NT>
__device__ __forceinline__ void m_exchange(float (&S)[2][2][4], uint32_t xchg, int warp, int lane) {
#pragma unroll
  for (int t = 0; t < NT; ++t)
#pragma unroll
    for (int n = 0; n < 2; ++n)
      s128f(xchg + (((warp * 2 + t) * 2 + n) * 32 + lane) * 16, S[t][n][0], S[t][n][1], S[t][n][2], S[t][n][3]);
  __syncthreads();
#pragma unroll
  for (int t = 0; t < NT; ++t)
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int w = 0; w < kMlaWarps; ++w) {
        const float4 v = l128f(xchg + (((w * 2 + t) * 2 + n) * 32 + lane) * 16);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
      }
      S[t][n][0] = acc.x; S[t][n][1] = acc.y; S[t][n][2] = acc.z; S[t][n][3] = acc.w;
    }
}

__device__ __forceinline__ void m_kstep_range(int warp, int* kb, int* ke) {
  // 36 sixteen-channel slices over 8 warps: 5,5,5,5,4,4,4,4
  *kb = warp < 4 ? 5 * warp : 20 + 4 * (warp - 4);
  *ke = *kb + (warp < 4 ? 5 : 4);
}

// One quantised half (32 tokens) staged at `stg`: [params 2304][codes tile 0][codes tile 1].
template <int BITS>
__device__ __forceinline__ void m_quant_half(uint32_t stg, uint32_t qh, uint32_t xchg, int warp, int lane,
                                             float scale_log2, MState& st) {
  const int c4 = lane & 3, r = lane >> 2;
  constexpr int kCb = 1152 * BITS;
  const uint32_t kp = stg, kc0 = stg + 2304, kc1 = stg + 2304 + kCb;
  int kb, ke;
  m_kstep_range(warp, &kb, &ke);
  float S[2][2][4];
  float zd[2][4], qe[2][4];
#pragma unroll
  for (int t = 0; t < 2; ++t)
#pragma unroll
    for (int n = 0; n < 2; ++n) S[t][n][0] = S[t][n][1] = S[t][n][2] = S[t][n][3] = 0.f;
#pragma unroll
  for (int n = 0; n < 2; ++n) {
    zd[n][0] = zd[n][1] = zd[n][2] = zd[n][3] = 0.f;
    qe[n][0] = qe[n][1] = qe[n][2] = qe[n][3] = 0.f;
  }
  for (int s = kb; s < ke; ++s) {
    const uint4 pr = l128(kp + (s * 4 + c4) * 16);          // s01, z01, s23, z23
    uint32_t a0[4], a1[4];
    if constexpr (BITS == 8) {
      unpack_k<8>(l32(kc0 + ((2 * s) * 32 + lane) * 4), l32(kc0 + ((2 * s + 1) * 32 + lane) * 4), a0);
      unpack_k<8>(l32(kc1 + ((2 * s) * 32 + lane) * 4), l32(kc1 + ((2 * s + 1) * 32 + lane) * 4), a1);
    } else {
      unpack_k<4>(l32(kc0 + (s * 32 + lane) * 4), 0u, a0);
      unpack_k<4>(l32(kc1 + (s * 32 + lane) * 4), 0u, a1);
    }
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      const uint2 q = l64(qh + ((s * 2 + n) * 32 + lane) * 8);
      const uint32_t q0 = hmul2u(q.x, pr.x), q1 = hmul2u(q.y, pr.z);
      mma_h(zd[n], pr.y, pr.x, pr.w, pr.z, q.x, q.y);       // rows r: sum q z, rows r + 8: sum q s
      mma_h(qe[n], kOnes, kOnes, kOnes, kOnes, q0, q1);     // sum q'
      mma_h(S[0][n], a0[0], a0[1], a0[2], a0[3], q0, q1);
      mma_h(S[1][n], a1[0], a1[1], a1[2], a1[3], q0, q1);
    }
  }
#pragma unroll
  for (int n = 0; n < 2; ++n) {
    const float z0 = fmaf(MB<BITS>::mid, zd[n][2], zd[n][0]), z1 = fmaf(MB<BITS>::mid, zd[n][3], zd[n][1]);
    const float cl0 = z0 - (MB<BITS>::lo + MB<BITS>::mid) * qe[n][0], cl1 = z1 - (MB<BITS>::lo + MB<BITS>::mid) * qe[n][1];
    const float ch0 = z0 - (MB<BITS>::hi + MB<BITS>::mid) * qe[n][0], ch1 = z1 - (MB<BITS>::hi + MB<BITS>::mid) * qe[n][1];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      S[t][n][0] += cl0; S[t][n][1] += cl1; S[t][n][2] += ch0; S[t][n][3] += ch1;
    }
  }
  m_exchange<2>(S, xchg, warp, lane);
#pragma unroll
  for (int t = 0; t < 2; ++t)
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) S[t][n][i] *= scale_log2;
  m_softmax<2>(S, st);
  // fp16 P^T fragments
  uint32_t pf[2][2][2];
#pragma unroll
  for (int t = 0; t < 2; ++t)
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      const __half2 h01 = __floats2half2_rn(S[t][n][0], S[t][n][1]), h23 = __floats2half2_rn(S[t][n][2], S[t][n][3]);
      st.l[n][0] += __low2float(h01) + __low2float(h23);
      st.l[n][1] += __high2float(h01) + __high2float(h23);
      pf[t][n][0] = movt(*reinterpret_cast<const uint32_t*>(&h01));
      pf[t][n][1] = movt(*reinterpret_cast<const uint32_t*>(&h23));
    }
  // value role: channels 64 w + 16 u .. of the same codes, transposed in registers
  float corr[2][4], psum[2][4];
#pragma unroll
  for (int n = 0; n < 2; ++n) {
    corr[n][0] = corr[n][1] = corr[n][2] = corr[n][3] = 0.f;
    psum[n][0] = psum[n][1] = psum[n][2] = psum[n][3] = 0.f;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      mma_h(corr[n], MB<BITS>::clo, MB<BITS>::clo, MB<BITS>::chi, MB<BITS>::chi, pf[t][n][0], pf[t][n][1]);
      mma_h(psum[n], kOnes, kOnes, kOnes, kOnes, pf[t][n][0], pf[t][n][1]);
    }
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int s = 4 * warp + u;                              // the MMA index that holds these 16 channels
    float acc[2][4];
#pragma unroll
    for (int n = 0; n < 2; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const uint32_t kc = t ? kc1 : kc0;
      uint32_t a[4];
      if constexpr (BITS == 8) unpack_k<8>(l32(kc + ((2 * s) * 32 + lane) * 4), l32(kc + ((2 * s + 1) * 32 + lane) * 4), a);
      else unpack_k<4>(l32(kc + (s * 32 + lane) * 4), 0u, a);
      const uint32_t v0 = movt(a[0]), v1 = movt(a[2]), v2 = movt(a[1]), v3 = movt(a[3]);
#pragma unroll
      for (int n = 0; n < 2; ++n) mma_h(acc[n], v0, v1, v2, v3, pf[t][n][0], pf[t][n][1]);
    }
    // per-channel scale and zero of rows (16 s + r) and (16 s + 8 + r)
    const uint32_t rec = kp + (s * 4 + ((r & 7) >> 1)) * 16;
    const uint32_t lo_s = l32(rec + 0), lo_z = l32(rec + 4), hi_s = l32(rec + 8), hi_z = l32(rec + 12);
    const bool odd = r & 1;
    const float s_lo = odd ? h_hi(lo_s) : h_lo(lo_s), z_lo = odd ? h_hi(lo_z) : h_lo(lo_z);
    const float s_hi = odd ? h_hi(hi_s) : h_lo(hi_s), z_hi = odd ? h_hi(hi_z) : h_lo(hi_z);
    const float zm_lo = fmaf(MB<BITS>::vmid, s_lo, z_lo), zm_hi = fmaf(MB<BITS>::vmid, s_hi, z_hi);
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      st.o[u][n][0] = fmaf(s_lo, acc[n][0] - corr[n][0], fmaf(zm_lo, psum[n][0], st.o[u][n][0]));
      st.o[u][n][1] = fmaf(s_lo, acc[n][1] - corr[n][1], fmaf(zm_lo, psum[n][1], st.o[u][n][1]));
      st.o[u][n][2] = fmaf(s_hi, acc[n][2] - corr[n][0], fmaf(zm_hi, psum[n][0], st.o[u][n][2]));
      st.o[u][n][3] = fmaf(s_hi, acc[n][3] - corr[n][1], fmaf(zm_hi, psum[n][1], st.o[u][n][3]));
    }
  }
}

// Sixteen exact bf16 rows staged at `stg` with pitch kMlaRowPitch.  bias_lo / bias_hi: additive
// log2-domain terms of the lane's rows r and r + 8 (0, -inf, or log2(count) for centroid rows).
__device__ __forceinline__ void m_rows_tile(uint32_t stg, uint32_t qb, uint32_t xchg, int warp, int lane,
                                            float scale_log2, float bias_lo, float bias_hi, MState& st) {
  int kb, ke;
  m_kstep_range(warp, &kb, &ke);
  float S[2][2][4];
#pragma unroll
  for (int t = 0; t < 2; ++t)
#pragma unroll
    for (int n = 0; n < 2; ++n) S[t][n][0] = S[t][n][1] = S[t][n][2] = S[t][n][3] = 0.f;
  const int mi = lane >> 3;
  const uint32_t kbase = stg + ((lane & 7) + (mi & 1) * 8) * kMlaRowPitch + (mi >> 1) * 16;
  for (int s = kb; s < ke; ++s) {
    uint32_t a[4];
    ldsm4(a, kbase + s * 32);
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      const uint2 q = l64(qb + ((s * 2 + n) * 32 + lane) * 8);
      mma_b(S[0][n], a, q.x, q.y);
    }
  }
  m_exchange<1>(S, xchg, warp, lane);
#pragma unroll
  for (int n = 0; n < 2; ++n) {
    S[0][n][0] = fmaf(S[0][n][0], scale_log2, bias_lo);
    S[0][n][1] = fmaf(S[0][n][1], scale_log2, bias_lo);
    S[0][n][2] = fmaf(S[0][n][2], scale_log2, bias_hi);
    S[0][n][3] = fmaf(S[0][n][3], scale_log2, bias_hi);
  }
  m_softmax<1>(S, st);
  uint32_t ph[2][2], pl[2][2];
#pragma unroll
  for (int n = 0; n < 2; ++n) {
    const uint32_t hi01 = bf2(S[0][n][0], S[0][n][1]), hi23 = bf2(S[0][n][2], S[0][n][3]);
    const uint32_t lo01 = bf2(S[0][n][0] - bflo(hi01), S[0][n][1] - bfhi(hi01));
    const uint32_t lo23 = bf2(S[0][n][2] - bflo(hi23), S[0][n][3] - bfhi(hi23));
    st.l[n][0] += S[0][n][0] + S[0][n][2];
    st.l[n][1] += S[0][n][1] + S[0][n][3];
    ph[n][0] = movt(hi01); ph[n][1] = movt(hi23);
    pl[n][0] = movt(lo01); pl[n][1] = movt(lo23);
  }
  const uint32_t vbase = stg + ((lane & 7) + (mi >> 1) * 8) * kMlaRowPitch + (mi & 1) * 16;
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    uint32_t a[4];
    ldsm4t(a, vbase + (4 * warp + u) * 32);
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      mma_b(st.o[u][n], a, ph[n][0], ph[n][1]);
      mma_b(st.o[u][n], a, pl[n][0], pl[n][1]);
    }
  }
}

struct MCursor {
  int item, sub, nsub, adv, level, ntok;
  uint32_t off256;
};

__device__ __forceinline__ bool m_load_item(const MlaDecodeParams& p, const TableEntry* table, int item_end, int it,
                                            MCursor& c) {
  while (true) {
    if (it >= item_end) return false;
    c.item = it;
    c.sub = 0;
    c.adv = 1;
    const TableEntry e = table[it];
    c.off256 = e.off256;
    c.level = static_cast<int>(e.level);
    c.ntok = kBlock;
    if (it == p.n_closed) {
      c.level = 16;
      c.ntok = p.n_tail;
      if (p.n_tail == 0) return false;       // the tail is the last item
    }
    if (c.level == 16) c.nsub = (c.ntok + 15) >> 4;
    else if (c.level == 1) {
      int run = 1;
      const int lim = min(min(item_end, p.n_closed) - it, 16);
      while (run < lim && table[it + run].level == 1u) ++run;
      c.adv = run;
      c.ntok = run;
      c.nsub = 1;
    } else c.nsub = 2;
    return true;
  }
}
__device__ __forceinline__ bool m_advance(const MlaDecodeParams& p, const TableEntry* table, int item_end, MCursor& c) {
  if (++c.sub < c.nsub) return true;
  return m_load_item(p, table, item_end, c.item + c.adv, c);
}

// issue the copies of the cursor's step (threads 0..15 take part)
__device__ __forceinline__ void m_issue(const MlaDecodeParams& p, const TableEntry* table, const MCursor& c, uint32_t stg,
                                        uint32_t bar, uint8_t* stg_ptr) {
  const int tid = threadIdx.x;
  if (c.level == 16 || c.level == 1) {
    const int nrows = c.level == 16 ? min(16, c.ntok - 16 * c.sub) : c.ntok;
    if (tid == 0) m_expect(bar, static_cast<uint32_t>(nrows) * kMlaRowBytes);
    __syncwarp();
    if (tid < 16) {
      if (tid < nrows) {
        const uint8_t* src = c.level == 16
                                 ? p.arena + static_cast<size_t>(c.off256) * 256 + static_cast<size_t>(16 * c.sub + tid) * kMlaRowBytes
                                 : p.arena + static_cast<size_t>(table[c.item + tid].off256) * 256;
        m_bulk(stg + tid * kMlaRowPitch, src, kMlaRowBytes, bar);
      } else {
        uint4* z = reinterpret_cast<uint4*>(stg_ptr + tid * kMlaRowPitch);
        for (int i = 0; i < kMlaRowBytes / 16; ++i) z[i] = make_uint4(0, 0, 0, 0);
      }
    }
    return;
  }
  if (tid == 0) {
    const uint32_t bytes = mla_half_bytes(c.level);
    m_expect(bar, bytes);
    m_bulk(stg, p.arena + static_cast<size_t>(c.off256) * 256 + static_cast<size_t>(c.sub) * bytes, bytes, bar);
  }
}

__global__ void __launch_bounds__(kMlaWarps * 32, 2) mla_decode_kernel(const __grid_constant__ MlaDecodeParams p) {
  extern __shared__ __align__(128) uint8_t msm[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WarpDesc cd = p.ctas[blockIdx.x];
  if (cd.stream < 0) return;
  const TableEntry* table = p.table + static_cast<size_t>(cd.stream) * p.table_stride;
  uint8_t* stage_ptr = msm;
  const uint32_t stage0 = s_u32(msm);
  const uint32_t qh = stage0 + 2 * kMlaStageBytes, qb = qh + kMlaQBytes, xchg = qb + kMlaQBytes;
  const uint32_t bar0 = xchg + kMlaXchgBytes;
  if (threadIdx.x == 0) {
    m_init(bar0, 1);
    m_init(bar0 + 8, 1);
    m_fence();
  }
  // query B-fragments for both head tiles: image [s][n][lane] of {channels 16s+2c4(+1) | 16s+8+2c4(+1)} of head 8n+r
  {
    const uint16_t* q = p.q + static_cast<size_t>(cd.stream) * kMlaHeads * kMlaDk;
    for (int i = threadIdx.x; i < kMlaKSteps * 2 * 32; i += blockDim.x) {
      const int ln = i & 31, n = (i >> 5) & 1, s = i >> 6;
      const int rr = ln >> 2, cc = ln & 3;
      const uint16_t* row = q + (8 * n + rr) * kMlaDk + 16 * s + 2 * cc;
      const uint32_t v0 = *reinterpret_cast<const uint32_t*>(row), v1 = *reinterpret_cast<const uint32_t*>(row + 8);
      const __half2 h0 = __floats2half2_rn(bflo(v0), bfhi(v0)), h1 = __floats2half2_rn(bflo(v1), bfhi(v1));
      uint2* dq = reinterpret_cast<uint2*>(msm + 2 * kMlaStageBytes) + i;
      uint2* db = reinterpret_cast<uint2*>(msm + 2 * kMlaStageBytes + kMlaQBytes) + i;
      *dq = make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
      *db = make_uint2(v0, v1);
    }
  }
  __syncthreads();

  MState st;
#pragma unroll
  for (int n = 0; n < 2; ++n) {
    st.m[n][0] = st.m[n][1] = kNegInfM;
    st.l[n][0] = st.l[n][1] = 0.f;
#pragma unroll
    for (int u = 0; u < 4; ++u) st.o[u][n][0] = st.o[u][n][1] = st.o[u][n][2] = st.o[u][n][3] = 0.f;
  }

  MCursor cur;
  bool have = m_load_item(p, table, cd.item_end, cd.item_begin, cur);
  int sidx = 0;
  uint32_t phase = 0;
  bool failed = false;
  if (have && warp == 0) m_issue(p, table, cur, stage0, bar0, stage_ptr);
  while (have) {
    MCursor nxt = cur;
    const bool more = m_advance(p, table, cd.item_end, nxt);
    if (more && warp == 0)
      m_issue(p, table, nxt, stage0 + (sidx ^ 1) * kMlaStageBytes, bar0 + 8 * (sidx ^ 1), stage_ptr + (sidx ^ 1) * kMlaStageBytes);
    int spins = 0;
    while (!m_try_wait(bar0 + 8 * sidx, (phase >> sidx) & 1u)) {
      if (++spins > kMlaWaitSpins) {
        failed = true;
        break;
      }
    }
    if (__syncthreads_or(failed)) {
      failed = true;
      break;
    }
    phase ^= 1u << sidx;
    const uint32_t stg = stage0 + sidx * kMlaStageBytes;
    if (cur.level == 16 || cur.level == 1) {
      const int r = lane >> 2;
      float b_lo, b_hi;
      if (cur.level == 16) {
        const int t0 = 16 * cur.sub + r;
        b_lo = t0 < cur.ntok ? 0.f : kNegInfM;
        b_hi = t0 + 8 < cur.ntok ? 0.f : kNegInfM;
      } else {
        b_lo = r < cur.ntok ? 6.0f : kNegInfM;          // log2(64): a centroid row stands for 64 tokens
        b_hi = r + 8 < cur.ntok ? 6.0f : kNegInfM;
      }
      m_rows_tile(stg, qb, xchg, warp, lane, p.scale_log2, b_lo, b_hi, st);
    } else if (cur.level == 8) {
      m_quant_half<8>(stg, qh, xchg, warp, lane, p.scale_log2, st);
    } else {
      m_quant_half<4>(stg, qh, xchg, warp, lane, p.scale_log2, st);
    }
    __syncthreads();
    cur = nxt;
    have = more;
    sidx ^= 1;
  }
  if (failed) {
    if (threadIdx.x == 0) atomicOr(p.status, kStatusInternal);
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      st.m[n][0] = st.m[n][1] = kNegInfM;
      st.l[n][0] = st.l[n][1] = 0.f;
    }
  }
  // partial row: [16 heads][m, l, o[512]]
#pragma unroll
  for (int n = 0; n < 2; ++n)
#pragma unroll
    for (int d = 4; d <= 16; d <<= 1) {
      st.l[n][0] += __shfl_xor_sync(kFullM, st.l[n][0], d);
      st.l[n][1] += __shfl_xor_sync(kFullM, st.l[n][1], d);
    }
  float* out = p.partial + static_cast<size_t>(cd.partial) * kMlaPartialFloats;
  const int r = lane >> 2, c4 = lane & 3;
#pragma unroll
  for (int n = 0; n < 2; ++n) {
    const int h0 = 8 * n + 2 * c4, h1 = h0 + 1;
    if (warp == 0 && r == 0) {
      out[h0 * (kMlaDv + 2)] = st.m[n][0];
      out[h0 * (kMlaDv + 2) + 1] = st.l[n][0];
      out[h1 * (kMlaDv + 2)] = st.m[n][1];
      out[h1 * (kMlaDv + 2) + 1] = st.l[n][1];
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int ch = 64 * warp + 16 * u + r;
      out[h0 * (kMlaDv + 2) + 2 + ch] = st.o[u][n][0];
      out[h1 * (kMlaDv + 2) + 2 + ch] = st.o[u][n][1];
      out[h0 * (kMlaDv + 2) + 2 + ch + 8] = st.o[u][n][2];
      out[h1 * (kMlaDv + 2) + 2 + ch + 8] = st.o[u][n][3];
    }
  }
}

__global__ void __launch_bounds__(kMlaDv) mla_combine_kernel(const float* partial, const StreamParts* parts, float* out,
                                                             float* lse) {
  __shared__ float sm_w[128], sm_l[128];
  const int stream = blockIdx.x, h = blockIdx.y, c = threadIdx.x;
  const int begin = parts[stream].begin, end = parts[stream].end;
  const float* base = partial + h * (kMlaDv + 2);
  float M = kNegInfM;
  for (int i = begin; i < end; ++i) M = fmaxf(M, __ldcg(base + static_cast<size_t>(i) * kMlaPartialFloats));
  float L = 0.f, acc = 0.f;
  for (int c0 = begin; c0 < end; c0 += 128) {
    const int n = min(128, end - c0);
    __syncthreads();
    if (c < n) {
      const float* row = base + static_cast<size_t>(c0 + c) * kMlaPartialFloats;
      const float m = __ldcg(row);
      const float w = (m == kNegInfM) ? 0.f : exp2f(m - M);
      sm_w[c] = w;
      sm_l[c] = w * __ldcg(row + 1);
    }
    __syncthreads();
    const float* col = base + static_cast<size_t>(c0) * kMlaPartialFloats + 2 + c;
#pragma unroll 4
    for (int i = 0; i < n; ++i) {
      L += sm_l[i];
      acc = fmaf(sm_w[i], __ldcg(col + static_cast<size_t>(i) * kMlaPartialFloats), acc);
    }
  }
  const size_t hq = static_cast<size_t>(stream) * kMlaHeads + h;
  out[hq * kMlaDv + c] = (L > 0.f) ? acc / L : 0.f;
  if (lse && c == 0) lse[hq] = (L > 0.f) ? (M + log2f(L)) * 0.6931471805599453f : kNegInfM;
}

}  // namespace

cudaError_t launch_mla_encode(const MlaEncodeParams& p, cudaStream_t st) {
  if (p.n_jobs <= 0) return cudaSuccess;
  const size_t smem = kBlock * kMTileLd * sizeof(float) + kBlock * kMlaDk;
  cudaError_t e = cudaFuncSetAttribute(mla_encode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  const int grid = p.n_jobs < 148 * 8 ? p.n_jobs : 148 * 8;
  mla_encode_kernel<<<grid, 256, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_mla_append_rows(uint8_t* arena, const TableEntry* table, int table_stride, int tail_index, int n_streams,
                                   const uint16_t* k_in, int n_tok, int first_tok, int n_rows, int dst_row0, cudaStream_t st) {
  if (n_rows <= 0) return cudaSuccess;
  mla_append_rows_kernel<<<dim3(n_streams, n_rows), kMlaDk / 2, 0, st>>>(arena, table, table_stride, tail_index, k_in, n_tok,
                                                                         first_tok, dst_row0);
  return cudaGetLastError();
}

cudaError_t launch_mla_export(const uint8_t* arena, uint32_t off256, int level, uint8_t* codes, uint16_t* scale,
                              uint16_t* zero, uint16_t* rows, cudaStream_t st) {
  mla_export_kernel<<<1, 256, 0, st>>>(arena, off256, level, codes, scale, zero, rows);
  return cudaGetLastError();
}

cudaError_t launch_mla_decode(const MlaDecodeParams& p, int n_ctas, const StreamParts* parts, int n_streams, float* out,
                              float* lse, cudaStream_t st) {
  if (n_ctas <= 0) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(mla_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMlaSmem);
  if (e != cudaSuccess) return e;
  mla_decode_kernel<<<n_ctas, kMlaWarps * 32, kMlaSmem, st>>>(p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  mla_combine_kernel<<<dim3(n_streams, kMlaHeads), kMlaDv, 0, st>>>(p.partial, parts, out, lse);
  return cudaGetLastError();
}

}  // namespace gkv
