// Bulk ingest: every closed block of a prompt goes from its bf16 rows straight to its planned
// rung of the ladder (paper Sec. 3.2: exact rows, b-bit codes with fp16 scale / zero per group of
// 32, or the block centroid), one launch for the whole layer.
//
// The arithmetic of every stored bit is the one of the block encoder used for demotions:
//   s = fp16((max - min) / (2^b - 1)), z = fp16(min) (saturating), code = clamp(rint((x - z) * (1 / s)), 0, 2^b - 1)
//   centroid = bf16(sequential fp32 sum over the 64 tokens * 1/64)
// (clamping before the rounding gives the same integer: both bounds are integers).  What differs
// is how the work is laid out.  The packed codes are stored in the order of the attention
// kernel's tensor-core fragments, so the block is read from shared memory with ldmatrix, which
// hands every lane exactly the values whose codes it has to pack: keys as the A fragment of a
// [16 tokens x 16 channels] tile, values as the A fragment of the transposed tile.  A lane then
// builds its 32-bit code words in registers and stores them with 8- or 16-byte stores; nothing is
// exchanged through shared memory except the per-token error sums of the two key warps that share
// a token.  Group minima / maxima are taken on packed bf16 pairs (exact) with three shuffles over
// the eight lanes that share a group; the division for scale and reciprocal is done once per
// group by one lane and handed to the others.
//
// One CTA (8 warps: 4 for keys, 4 for values) per block; the next block's 32 KB of rows are in
// flight (cp.async, second buffer) while the current one is encoded.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gkv_internal.h"

namespace gkv {
namespace {

constexpr int kInRow = kRowBytes + 16;            // padded shared-memory row: ldmatrix without bank conflicts
constexpr int kInTensor = kBlock * kInRow;        // 17408
constexpr int kInBuf = 2 * kInTensor;             // keys, values
constexpr int kInThreads = 256;
constexpr int kInSmem = 2 * kInBuf + (256 + 128 + 16) * static_cast<int>(sizeof(float));
constexpr float kMagic = 12582912.f;              // 1.5 * 2^23: x + kMagic rounds x to an integer (ties to even)
constexpr uint32_t kMagicBits = 0x4B400000u;
constexpr uint32_t kFullI = 0xffffffffu;

__device__ __forceinline__ uint32_t i_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void i_cp16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void i_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
__device__ __forceinline__ void i_wait_all() { asm volatile("cp.async.wait_group 0;\n" ::: "memory"); }
__device__ __forceinline__ void i_ldm4(uint32_t a, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(a));
}
__device__ __forceinline__ void i_ldm4t(uint32_t a, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(a));
}
__device__ __forceinline__ float i_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float i_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ uint32_t i_min2(uint32_t a, uint32_t b) {
  const __nv_bfloat162 r = __hmin2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
  return *reinterpret_cast<const uint32_t*>(&r);
}
__device__ __forceinline__ uint32_t i_max2(uint32_t a, uint32_t b) {
  const __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
  return *reinterpret_cast<const uint32_t*>(&r);
}
__device__ __forceinline__ uint16_t i_fp16_sat(float x) {
  x = fminf(fmaxf(x, -65504.f), 65504.f);
  const __half h = __float2half_rn(x);
  return *reinterpret_cast<const uint16_t*>(&h);
}
__device__ __forceinline__ float i_fp16_f32(uint16_t b) { return __half2float(*reinterpret_cast<const __half*>(&b)); }
__device__ __forceinline__ uint16_t i_bf16(float x) {
  const __nv_bfloat16 h = __float2bfloat16_rn(x);
  return *reinterpret_cast<const uint16_t*>(&h);
}

// scale, zero point and reciprocal of one group from its minimum and maximum
struct GroupParams {
  float s, z, inv;
  uint16_t s_bits, z_bits;
  bool range;
};
template <int BITS>
__device__ __forceinline__ GroupParams i_params(float mn, float mx) {
  constexpr float qmax = static_cast<float>((1 << BITS) - 1);
  const float s_raw = __fdiv_rn(__fsub_rn(mx, mn), qmax);
  GroupParams g;
  g.range = fabsf(s_raw) > 65504.f || fabsf(mn) > 65504.f;
  g.s_bits = i_fp16_sat(s_raw);
  g.z_bits = i_fp16_sat(mn);
  g.s = i_fp16_f32(g.s_bits);
  g.z = i_fp16_f32(g.z_bits);
  g.inv = g.s > 0.f ? __fdiv_rn(1.f, g.s) : 0.f;
  return g;
}

// bit position of code (slice s, register a, half hlf) inside its 32-bit word
template <int BITS>
__device__ __forceinline__ constexpr int i_bit(int s, int a, int hlf) {
  return BITS == 8 ? 8 * (a & 1) + 16 * hlf : (BITS == 4 ? 4 * a + 16 * hlf : 4 * (s & 1) + 2 * (a & 1) + 8 * (a >> 1) + 16 * hlf);
}

// Quantise the two values of a register (low half: params 0, high half: params 1), add the codes to
// `word` at bit positions b0 / b1 (the magic constant is taken off by the caller, once per word) and
// add the squared reconstruction errors to e0 / e1.
template <int BITS>
__device__ __forceinline__ void i_quant2(uint32_t x, float s0, float z0, float inv0, float s1, float z1, float inv1, int b0,
                                         int b1, uint32_t& word, float& e0, float& e1) {
  constexpr float qmax = static_cast<float>((1 << BITS) - 1);
  const float x0 = i_lo(x), x1 = i_hi(x);
  const float r0 = __fadd_rn(fminf(fmaxf(__fmul_rn(__fsub_rn(x0, z0), inv0), 0.f), qmax), kMagic);
  const float r1 = __fadd_rn(fminf(fmaxf(__fmul_rn(__fsub_rn(x1, z1), inv1), 0.f), qmax), kMagic);
  word += (__float_as_uint(r0) << b0) + (__float_as_uint(r1) << b1);
  const float d0 = x0 - __fmaf_rn(r0 - kMagic, s0, z0), d1 = x1 - __fmaf_rn(r1 - kMagic, s1, z1);
  e0 = fmaf(d0, d0, e0);
  e1 = fmaf(d1, d1, e1);
}

// Keys of one half (32 tokens) x 64 channels: x[tile of the half][slice][a].  Groups are 32 tokens of
// one channel: the lane's registers (tile, a & 1) and the eight lanes of a column (r = lane >> 2).
// Pair k = 2 * slice + (a >> 1) names the lane's two channels 16 s + 8 (a >> 1) + 2 c4 + {0, 1}.
// e[tile][a & 1][0 / 1]: squared error of token 16 tile + 8 (a & 1) + r over the lane's channels;
// the two halves of a pair are summed at the end.
template <int BITS>
__device__ __forceinline__ bool ingest_keys(const uint32_t (&x)[2][4][4], uint8_t* half_base, int chh, int lane, float (&e)[2][2]) {
  const int r = lane >> 2, c4 = lane & 3;
  uint32_t mn[8], mx[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int sl = k >> 1, ah = k & 1;
    mn[k] = i_min2(i_min2(x[0][sl][2 * ah], x[0][sl][2 * ah + 1]), i_min2(x[1][sl][2 * ah], x[1][sl][2 * ah + 1]));
    mx[k] = i_max2(i_max2(x[0][sl][2 * ah], x[0][sl][2 * ah + 1]), i_max2(x[1][sl][2 * ah], x[1][sl][2 * ah + 1]));
#pragma unroll
    for (int d = 4; d <= 16; d <<= 1) {
      mn[k] = i_min2(mn[k], __shfl_xor_sync(kFullI, mn[k], d));
      mx[k] = i_max2(mx[k], __shfl_xor_sync(kFullI, mx[k], d));
    }
  }
  // lane r works out the parameters of pair r
  uint32_t my_mn = mn[0], my_mx = mx[0];
#pragma unroll
  for (int k = 1; k < 8; ++k) {
    if (r == k) {
      my_mn = mn[k];
      my_mx = mx[k];
    }
  }
  const GroupParams g0 = i_params<BITS>(i_lo(my_mn), i_lo(my_mx)), g1 = i_params<BITS>(i_hi(my_mn), i_hi(my_mx));
  {
    // record [slice][c4] = {scale c0, scale c1, zero c0, zero c1, scale c0 + 8, scale c1 + 8, zero c0 + 8, zero c1 + 8}
    const int s_glob = 4 * chh + (r >> 1);
    uint2 rec;
    rec.x = static_cast<uint32_t>(g0.s_bits) | (static_cast<uint32_t>(g1.s_bits) << 16);
    rec.y = static_cast<uint32_t>(g0.z_bits) | (static_cast<uint32_t>(g1.z_bits) << 16);
    *reinterpret_cast<uint2*>(half_base + off_kp() + (s_glob * 4 + c4) * 16 + (r & 1) * 8) = rec;
  }
  float e00 = 0.f, e01 = 0.f, e10 = 0.f, e11 = 0.f;      // [tile][a & 1], low halves
  float f00 = 0.f, f01 = 0.f, f10 = 0.f, f11 = 0.f;      // high halves
  uint32_t w[2][4];
#pragma unroll
  for (int t = 0; t < 2; ++t)
#pragma unroll
    for (int i = 0; i < 4; ++i) w[t][i] = 0u;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int sl = k >> 1, ah = k & 1, src = 4 * k + c4;
    const float s0 = __shfl_sync(kFullI, g0.s, src), z0 = __shfl_sync(kFullI, g0.z, src), v0 = __shfl_sync(kFullI, g0.inv, src);
    const float s1 = __shfl_sync(kFullI, g1.s, src), z1 = __shfl_sync(kFullI, g1.z, src), v1 = __shfl_sync(kFullI, g1.inv, src);
    // word index inside the lane's words of a tile: 8 bits: 2 sl + ah (8 words), 4 bits: sl (4), 2 bits: sl >> 1 (2)
    const int wi = BITS == 8 ? (2 * sl + ah) & 3 : (BITS == 4 ? sl : sl >> 1);
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      i_quant2<BITS>(x[t][sl][2 * ah], s0, z0, v0, s1, z1, v1, i_bit<BITS>(sl, 2 * ah, 0), i_bit<BITS>(sl, 2 * ah, 1), w[t][wi],
                     t == 0 ? e00 : e10, t == 0 ? f00 : f10);
      i_quant2<BITS>(x[t][sl][2 * ah + 1], s0, z0, v0, s1, z1, v1, i_bit<BITS>(sl, 2 * ah + 1, 0), i_bit<BITS>(sl, 2 * ah + 1, 1),
                     w[t][wi], t == 0 ? e01 : e11, t == 0 ? f01 : f11);
    }
    // a group of words is complete: take the magic constants off and store
    const bool flush = BITS == 8 ? (k & 3) == 3 : k == 7;
    if (flush) {
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        uint8_t* codes = half_base + off_kc(BITS, t);
        if (BITS == 8) {
#pragma unroll
          for (int i = 0; i < 4; ++i) w[t][i] -= kMagicBits * 0x01010101u;
          const int chunk = 2 * chh + (k >> 2);
          *reinterpret_cast<uint4*>(codes + (chunk * 32 + lane) * 16) = make_uint4(w[t][0], w[t][1], w[t][2], w[t][3]);
#pragma unroll
          for (int i = 0; i < 4; ++i) w[t][i] = 0u;
        } else if (BITS == 4) {
#pragma unroll
          for (int i = 0; i < 4; ++i) w[t][i] -= kMagicBits * 0x11111111u;
          *reinterpret_cast<uint4*>(codes + (chh * 32 + lane) * 16) = make_uint4(w[t][0], w[t][1], w[t][2], w[t][3]);
        } else {
#pragma unroll
          for (int i = 0; i < 2; ++i) w[t][i] -= kMagicBits * 0x55555555u;
          *reinterpret_cast<uint2*>(codes + lane * 16 + chh * 8) = make_uint2(w[t][0], w[t][1]);
        }
      }
    }
  }
  e[0][0] = e00 + f00;
  e[0][1] = e01 + f01;
  e[1][0] = e10 + f10;
  e[1][1] = e11 + f11;
  return g0.range || g1.range;
}

// Values of one tile (16 tokens) x 128 channels: x[slice][a], channel 16 s + r + 8 (a & 1), token
// 8 (a >> 1) + 2 c4 + {0, 1}.  Groups are 32 channels of one token: slices 2 g and 2 g + 1, a & 1 and the
// eight lanes r.  Pair k = 2 g + (a >> 1) names the lane's tokens 8 (a >> 1) + 2 c4 + {0, 1} in group g.
// e[a >> 1][0 / 1]: squared error of token 8 (a >> 1) + 2 c4 + {0, 1} over the lane's channels.
template <int BITS>
__device__ __forceinline__ bool ingest_values(const uint32_t (&x)[8][4], uint8_t* vp, uint8_t* codes, int lane, float (&e)[2][2]) {
  const int r = lane >> 2, c4 = lane & 3;
  uint32_t mn[8], mx[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int g = k >> 1, ah = k & 1;
    mn[k] = i_min2(i_min2(x[2 * g][2 * ah], x[2 * g][2 * ah + 1]), i_min2(x[2 * g + 1][2 * ah], x[2 * g + 1][2 * ah + 1]));
    mx[k] = i_max2(i_max2(x[2 * g][2 * ah], x[2 * g][2 * ah + 1]), i_max2(x[2 * g + 1][2 * ah], x[2 * g + 1][2 * ah + 1]));
#pragma unroll
    for (int d = 4; d <= 16; d <<= 1) {
      mn[k] = i_min2(mn[k], __shfl_xor_sync(kFullI, mn[k], d));
      mx[k] = i_max2(mx[k], __shfl_xor_sync(kFullI, mx[k], d));
    }
  }
  uint32_t my_mn = mn[0], my_mx = mx[0];
#pragma unroll
  for (int k = 1; k < 8; ++k) {
    if (r == k) {
      my_mn = mn[k];
      my_mx = mx[k];
    }
  }
  const GroupParams g0 = i_params<BITS>(i_lo(my_mn), i_lo(my_mx)), g1 = i_params<BITS>(i_hi(my_mn), i_hi(my_mx));
  {
    // scales [c4][group] = {tA0, tA1, tB0, tB1}, zeros [group][c4] likewise at fp16 index 64; pair r = (group, a >> 1)
    const int g = r >> 1, ah = r & 1;
    uint16_t* p16 = reinterpret_cast<uint16_t*>(vp);
    *reinterpret_cast<uint32_t*>(p16 + (c4 * 4 + g) * 4 + ah * 2) = static_cast<uint32_t>(g0.s_bits) | (static_cast<uint32_t>(g1.s_bits) << 16);
    *reinterpret_cast<uint32_t*>(p16 + 64 + (g * 4 + c4) * 4 + ah * 2) = static_cast<uint32_t>(g0.z_bits) | (static_cast<uint32_t>(g1.z_bits) << 16);
  }
  float e0 = 0.f, e1 = 0.f, e2 = 0.f, e3 = 0.f;      // [a >> 1][hlf]
  uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int g = k >> 1, ah = k & 1, src = 4 * k + c4;
    const float s0 = __shfl_sync(kFullI, g0.s, src), z0 = __shfl_sync(kFullI, g0.z, src), v0 = __shfl_sync(kFullI, g0.inv, src);
    const float s1 = __shfl_sync(kFullI, g1.s, src), z1 = __shfl_sync(kFullI, g1.z, src), v1 = __shfl_sync(kFullI, g1.inv, src);
#pragma unroll
    for (int ss = 0; ss < 2; ++ss) {
      const int s = 2 * g + ss;
      // word of (s, a): 8 bits: 2 s + ah, 4 bits: s, 2 bits: s >> 1; index inside the 16-byte chunk being filled
      const int wi = BITS == 8 ? (2 * s + ah) & 3 : (BITS == 4 ? s & 3 : s >> 1);
#pragma unroll
      for (int al = 0; al < 2; ++al)
        i_quant2<BITS>(x[s][2 * ah + al], s0, z0, v0, s1, z1, v1, i_bit<BITS>(s, 2 * ah + al, 0), i_bit<BITS>(s, 2 * ah + al, 1), w[wi],
                       ah == 0 ? e0 : e2, ah == 0 ? e1 : e3);
    }
    const bool flush = BITS == 8 ? ah == 1 : (BITS == 4 ? (k & 3) == 3 : k == 7);
    if (flush) {
      constexpr uint32_t kOff = BITS == 8 ? 0x01010101u : (BITS == 4 ? 0x11111111u : 0x55555555u);
#pragma unroll
      for (int i = 0; i < 4; ++i) w[i] -= kMagicBits * kOff;
      const int chunk = BITS == 8 ? g : (BITS == 4 ? g >> 1 : 0);
      *reinterpret_cast<uint4*>(codes + (chunk * 32 + lane) * 16) = make_uint4(w[0], w[1], w[2], w[3]);
#pragma unroll
      for (int i = 0; i < 4; ++i) w[i] = 0u;
    }
  }
  e[0][0] = e0;
  e[0][1] = e1;
  e[1][0] = e2;
  e[1][1] = e3;
  return g0.range || g1.range;
}

__global__ void __launch_bounds__(kInThreads, 3) ingest_kernel(const __grid_constant__ EncodeParams p) {
  extern __shared__ __align__(16) uint8_t ism[];
  float* cen = reinterpret_cast<float*>(ism + 2 * kInBuf);      // [2][128] centroid of keys, of values
  float* kd2 = cen + 256;                                       // [2 channel halves][64 tokens]
  float* red = kd2 + 128;                                       // [4 value warps][2]: max error, max norm (squared)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int r = lane >> 2, c4 = lane & 3;
  const uint32_t sbase = i_u32(ism);
  const size_t row_stride = static_cast<size_t>(p.n_kv_heads) * kD;      // elements between two tokens of a stream

  auto stage = [&](int item, int buf) {
    const EncodeJob job = p.jobs[item];
    const int b = job.stream / p.n_kv_heads, kvh = job.stream - b * p.n_kv_heads;
    const size_t first = (static_cast<size_t>(b) * p.n_tok + static_cast<size_t>(job.block) * kBlock) * row_stride + static_cast<size_t>(kvh) * kD;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int q = tid + kInThreads * i;
      const int tensor = q >> 10, row = (q >> 4) & 63, col = q & 15;
      const uint16_t* src = (tensor ? p.v_in : p.k_in) + first + static_cast<size_t>(row) * row_stride + col * 8;
      i_cp16(sbase + buf * kInBuf + tensor * kInTensor + row * kInRow + col * 16, src);
    }
  };

  int item = blockIdx.x, buf = 0;
  if (item < p.n_jobs) stage(item, 0);
  i_commit();
  for (; item < p.n_jobs; item += gridDim.x, buf ^= 1) {
    const EncodeJob job = p.jobs[item];
    i_wait_all();
    __syncthreads();                       // the block's rows are there; nobody still reads the other buffer
    if (item + static_cast<int>(gridDim.x) < p.n_jobs) stage(item + gridDim.x, buf ^ 1);
    i_commit();

    uint8_t* dst = p.arena + static_cast<size_t>(job.dst_off256) * 256;
    const int L = job.dst_level;
    const uint8_t* tile_g = ism + buf * kInBuf;
    const uint32_t tile_s = sbase + buf * kInBuf;

    if (L == 16) {
      // exact rows: keys, then values, row-major
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int q = tid + kInThreads * i;
        const int tensor = q >> 10, row = (q >> 4) & 63, col = q & 15;
        *reinterpret_cast<uint4*>(dst + tensor * (kBlock * kRowBytes) + row * kRowBytes + col * 16) =
            *reinterpret_cast<const uint4*>(tile_g + tensor * kInTensor + row * kInRow + col * 16);
      }
    } else if (L == 1) {
      // centroid: sequential sum over the tokens per channel (thread = tensor, channel)
      const int tensor = tid >> 7, c = tid & (kD - 1);
      const uint16_t* col = reinterpret_cast<const uint16_t*>(tile_g + tensor * kInTensor) + c;
      float acc = 0.f;
#pragma unroll 16
      for (int t = 0; t < kBlock; ++t) acc = __fadd_rn(acc, __uint_as_float(static_cast<uint32_t>(col[t * (kInRow / 2)]) << 16));
      const uint16_t cb = i_bf16(__fmul_rn(acc, 1.0f / kBlock));
      reinterpret_cast<uint16_t*>(dst + tensor * kRowBytes)[c] = cb;
      cen[tid] = __uint_as_float(static_cast<uint32_t>(cb) << 16);
      __syncthreads();
    }

    bool range = false;
    if (warp < 4) {
      // ---- keys: warp = (half of the block, half of the channels) ----
      const int half = warp >> 1, chh = warp & 1;
      float e[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
      if (L != 16) {
        uint32_t x[2][4][4];
        const int mi = lane >> 3;
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
          for (int sl = 0; sl < 4; ++sl)
            i_ldm4(tile_s + (32 * half + 16 * t + (mi & 1) * 8 + (lane & 7)) * kInRow + (64 * chh + 16 * sl + (mi >> 1) * 8) * 2, x[t][sl]);
        uint8_t* half_base = dst + half * half_bytes(L);
        if (L == 8) range = ingest_keys<8>(x, half_base, chh, lane, e);
        else if (L == 4) range = ingest_keys<4>(x, half_base, chh, lane, e);
        else if (L == 2) range = ingest_keys<2>(x, half_base, chh, lane, e);
        else {
          // distance from the centroid
#pragma unroll
          for (int sl = 0; sl < 4; ++sl)
#pragma unroll
            for (int ah = 0; ah < 2; ++ah) {
              const float2 cc = *reinterpret_cast<const float2*>(cen + 64 * chh + 16 * sl + 8 * ah + 2 * c4);
#pragma unroll
              for (int t = 0; t < 2; ++t)
#pragma unroll
                for (int al = 0; al < 2; ++al) {
                  const float d0 = i_lo(x[t][sl][2 * ah + al]) - cc.x, d1 = i_hi(x[t][sl][2 * ah + al]) - cc.y;
                  e[t][al] = fmaf(d0, d0, e[t][al]);
                  e[t][al] = fmaf(d1, d1, e[t][al]);
                }
            }
        }
      }
      // a token's sum over this warp's 64 channels: add the four lanes of its row
#pragma unroll
      for (int t = 0; t < 2; ++t)
#pragma unroll
        for (int al = 0; al < 2; ++al) {
          float v = e[t][al];
          v += __shfl_xor_sync(kFullI, v, 1);
          v += __shfl_xor_sync(kFullI, v, 2);
          if (c4 == 0) kd2[chh * kBlock + 32 * half + 16 * t + 8 * al + r] = v;
        }
    } else {
      // ---- values: warp = 16-token tile ----
      const int tile = warp - 4;
      uint32_t x[8][4];
      const int mi = lane >> 3;
#pragma unroll
      for (int s = 0; s < 8; ++s)
        i_ldm4t(tile_s + kInTensor + (16 * tile + (mi >> 1) * 8 + (lane & 7)) * kInRow + (16 * s + (mi & 1) * 8) * 2, x[s]);
      float e[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
      if (L != 16 && L != 1) {
        uint8_t* hb = dst + (tile >> 1) * half_bytes(L);
        uint8_t* vp = hb + off_vp(L, tile & 1);
        uint8_t* codes = hb + off_vc(L, tile & 1);
        if (L == 8) range = ingest_values<8>(x, vp, codes, lane, e);
        else if (L == 4) range = ingest_values<4>(x, vp, codes, lane, e);
        else range = ingest_values<2>(x, vp, codes, lane, e);
      } else if (L == 1) {
#pragma unroll
        for (int s = 0; s < 8; ++s)
#pragma unroll
          for (int al = 0; al < 2; ++al) {
            const float cc = cen[kD + 16 * s + r + 8 * al];
#pragma unroll
            for (int ah = 0; ah < 2; ++ah) {
              const float d0 = i_lo(x[s][2 * ah + al]) - cc, d1 = i_hi(x[s][2 * ah + al]) - cc;
              e[ah][0] = fmaf(d0, d0, e[ah][0]);
              e[ah][1] = fmaf(d1, d1, e[ah][1]);
            }
          }
      }
      // squared norms of the original value rows, same token layout
      float n[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
      for (int s = 0; s < 8; ++s)
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          const float x0 = i_lo(x[s][a]), x1 = i_hi(x[s][a]);
          n[a >> 1][0] = fmaf(x0, x0, n[a >> 1][0]);
          n[a >> 1][1] = fmaf(x1, x1, n[a >> 1][1]);
        }
      // a token's sums over all channels: add the eight lanes r; then the largest token of the tile
      float em = 0.f, nm = 0.f;
#pragma unroll
      for (int ah = 0; ah < 2; ++ah)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float v = e[ah][h], w = n[ah][h];
#pragma unroll
          for (int d = 4; d <= 16; d <<= 1) {
            v += __shfl_xor_sync(kFullI, v, d);
            w += __shfl_xor_sync(kFullI, w, d);
          }
          em = fmaxf(em, v);
          nm = fmaxf(nm, w);
        }
#pragma unroll
      for (int d = 1; d <= 2; d <<= 1) {
        em = fmaxf(em, __shfl_xor_sync(kFullI, em, d));
        nm = fmaxf(nm, __shfl_xor_sync(kFullI, nm, d));
      }
      if (lane == 0) {
        red[2 * tile] = em;
        red[2 * tile + 1] = nm;
      }
    }
    if (range) atomicOr(p.status, kStatusRange);
    __syncthreads();
    if (warp == 0 && p.err) {
      // bound on |k - k^| (largest token), on |v - v^|, and the largest |v| of the block
      float km = fmaxf(kd2[lane] + kd2[kBlock + lane], kd2[32 + lane] + kd2[kBlock + 32 + lane]);
#pragma unroll
      for (int d = 1; d <= 16; d <<= 1) km = fmaxf(km, __shfl_xor_sync(kFullI, km, d));
      if (lane == 0) {
        const float vm = fmaxf(fmaxf(red[0], red[2]), fmaxf(red[4], red[6]));
        const float nm = fmaxf(fmaxf(red[1], red[3]), fmaxf(red[5], red[7]));
        p.err[static_cast<size_t>(job.stream) * p.err_stride + job.block] = make_float4(sqrtf(km), sqrtf(vm), sqrtf(nm), 0.f);
      }
    }
  }
}

}  // namespace

// All jobs read the bf16 input rows (src_level == 0).
cudaError_t launch_ingest(const EncodeParams& p, cudaStream_t st) {
  if (p.n_jobs <= 0) return cudaSuccess;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(ingest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kInSmem);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int grid = p.n_jobs < 148 * 3 ? p.n_jobs : 148 * 3;
  ingest_kernel<<<grid, kInThreads, kInSmem, st>>>(p);
  return cudaGetLastError();
}

}  // namespace gkv
