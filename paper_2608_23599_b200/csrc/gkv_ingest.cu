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
#include "gkv_mla.h"

namespace gkv {
namespace {

constexpr int kInRow = kRowBytes + 16;            // padded shared-memory row: ldmatrix without bank conflicts
constexpr int kInTensor = kBlock * kInRow;        // 17408
constexpr int kInBuf = 2 * kInTensor;             // keys, values
constexpr int kInThreads = 256;
constexpr int kInSmem = 2 * kInBuf + (256 + 128 + 16) * static_cast<int>(sizeof(float)) + 8 * 32 * 16;   // + the warps' group parameters
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

// bit position of code (slice s, register a, half hlf) inside its 32-bit word (value codes: the fields
// of registers 1 and 2 change places, see gkv_layout.cuh)
template <int BITS>
__device__ __forceinline__ constexpr int i_bit(int s, int a, int hlf) {
  return BITS == 8 ? 8 * (a & 1) + 16 * hlf : (BITS == 4 ? 4 * a + 16 * hlf : 4 * (s & 1) + 2 * (a & 1) + 8 * (a >> 1) + 16 * hlf);
}
template <int BITS>
__device__ __forceinline__ constexpr int i_bit_v(int s, int a, int hlf) {
  return i_bit<BITS>(s, BITS == 8 ? a : ((a >> 1) | ((a & 1) << 1)), hlf);
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

// Parameters of a group as the warp keeps them in shared memory between its two passes:
// {scale | zero << 16 (fp16 bits), reciprocal} of the low and of the high half of a register pair.
__device__ __forceinline__ uint4 i_pack_params(const GroupParams& g0, const GroupParams& g1) {
  return make_uint4(static_cast<uint32_t>(g0.s_bits) | (static_cast<uint32_t>(g0.z_bits) << 16), __float_as_uint(g0.inv),
                    static_cast<uint32_t>(g1.s_bits) | (static_cast<uint32_t>(g1.z_bits) << 16), __float_as_uint(g1.inv));
}
__device__ __forceinline__ float i_h_lo(uint32_t u) { return __half2float(__ushort_as_half(static_cast<unsigned short>(u & 0xffffu))); }
__device__ __forceinline__ float i_h_hi(uint32_t u) { return __half2float(__ushort_as_half(static_cast<unsigned short>(u >> 16))); }

// Keys of one half (32 tokens) x 64 channels.  ldmatrix hands a lane, per 16-token tile and slice of
// 16 channels, registers a = 0..3: token 8 (a & 1) + r, channels 16 s + 8 (a >> 1) + 2 c4 + {0, 1}
// (r = lane >> 2, c4 = lane & 3).  Groups are 32 tokens of one channel: the lane's registers
// (tile, a & 1) and the eight lanes r.  Pair k = 2 * slice + (a >> 1) names the lane's two channels.
// Pass 1 finds the extremes of every pair, lane r works out the parameters of pair r; pass 2 reads
// the rows again, quantises and stores whole words.  Both passes are rolled loops over the slices
// (the code of all rungs together has to stay inside the instruction cache).
// e[tile][a & 1]: squared error of token 16 tile + 8 (a & 1) + r summed over the lane's channels.
template <int BITS>
__device__ __forceinline__ bool ingest_keys(uint32_t tile_k, uint8_t* half_base, int half, int chh, int lane, uint4* prm, float (&e)[2][2]) {
  const int r = lane >> 2, c4 = lane & 3, mi = lane >> 3;
  const uint32_t ld = tile_k + (32 * half + (mi & 1) * 8 + (lane & 7)) * kInRow + (64 * chh + (mi >> 1) * 8) * 2;
  uint32_t my_mn = 0u, my_mx = 0u;
#pragma unroll 1
  for (int sl = 0; sl < 4; ++sl) {
    uint32_t x0[4], x1[4];
    i_ldm4(ld + sl * 32, x0);
    i_ldm4(ld + 16 * kInRow + sl * 32, x1);
#pragma unroll
    for (int ah = 0; ah < 2; ++ah) {
      uint32_t mn = i_min2(i_min2(x0[2 * ah], x0[2 * ah + 1]), i_min2(x1[2 * ah], x1[2 * ah + 1]));
      uint32_t mx = i_max2(i_max2(x0[2 * ah], x0[2 * ah + 1]), i_max2(x1[2 * ah], x1[2 * ah + 1]));
#pragma unroll
      for (int d = 4; d <= 16; d <<= 1) {
        mn = i_min2(mn, __shfl_xor_sync(kFullI, mn, d));
        mx = i_max2(mx, __shfl_xor_sync(kFullI, mx, d));
      }
      if (r == 2 * sl + ah) {
        my_mn = mn;
        my_mx = mx;
      }
    }
  }
  const GroupParams g0 = i_params<BITS>(i_lo(my_mn), i_lo(my_mx)), g1 = i_params<BITS>(i_hi(my_mn), i_hi(my_mx));
  {
    // per (slab, c4) a record of zero points and one of scales, each {s0: c0 c1, s1: c0 c1, s0: c2 c3, s1: c2 c3}
    // (gkv_layout.cuh); this lane holds the pair (c0, c1) or (c2, c3) (r & 1) of MMA index s_glob
    const int s_glob = 4 * chh + (r >> 1);
    uint32_t* rec = reinterpret_cast<uint32_t*>(half_base + off_kp() + ((s_glob >> 1) * 4 + c4) * 32) + (r & 1) * 2 + (s_glob & 1);
    rec[0] = static_cast<uint32_t>(g0.z_bits) | (static_cast<uint32_t>(g1.z_bits) << 16);
    rec[4] = static_cast<uint32_t>(g0.s_bits) | (static_cast<uint32_t>(g1.s_bits) << 16);
  }
  prm[r * 4 + c4] = i_pack_params(g0, g1);
  __syncwarp();
  constexpr int SL = BITS == 2 ? 2 : 1;             // slices that fill whole words
  constexpr uint32_t kOff = BITS == 8 ? 0x01010101u : (BITS == 4 ? 0x11111111u : 0x55555555u);
  float e00 = 0.f, e01 = 0.f, e10 = 0.f, e11 = 0.f, f00 = 0.f, f01 = 0.f, f10 = 0.f, f11 = 0.f;
#pragma unroll 1
  for (int u = 0; u < 4 / SL; ++u) {
    uint32_t w[2][2] = {{0u, 0u}, {0u, 0u}};        // [tile][word]: 8 bits: one word per a >> 1; else one word
#pragma unroll
    for (int ss = 0; ss < SL; ++ss) {
      const int sl = u * SL + ss;
      uint32_t x[2][4];
      i_ldm4(ld + sl * 32, x[0]);
      i_ldm4(ld + 16 * kInRow + sl * 32, x[1]);
#pragma unroll
      for (int ah = 0; ah < 2; ++ah) {
        const uint4 P = prm[(2 * sl + ah) * 4 + c4];
        const float s0 = i_h_lo(P.x), z0 = i_h_hi(P.x), v0 = __uint_as_float(P.y);
        const float s1 = i_h_lo(P.z), z1 = i_h_hi(P.z), v1 = __uint_as_float(P.w);
        const int wi = BITS == 8 ? ah : 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          i_quant2<BITS>(x[t][2 * ah], s0, z0, v0, s1, z1, v1, i_bit<BITS>(ss, 2 * ah, 0), i_bit<BITS>(ss, 2 * ah, 1), w[t][wi],
                         t == 0 ? e00 : e10, t == 0 ? f00 : f10);
          i_quant2<BITS>(x[t][2 * ah + 1], s0, z0, v0, s1, z1, v1, i_bit<BITS>(ss, 2 * ah + 1, 0), i_bit<BITS>(ss, 2 * ah + 1, 1),
                         w[t][wi], t == 0 ? e01 : e11, t == 0 ? f01 : f11);
        }
      }
    }
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      uint8_t* codes = half_base + off_kc(BITS, t);
      if (BITS == 8) {          // words 8 chh + 2 u + {0, 1}
        *reinterpret_cast<uint2*>(codes + ((2 * chh + (u >> 1)) * 32 + lane) * 16 + (u & 1) * 8) =
            make_uint2(w[t][0] - kMagicBits * kOff, w[t][1] - kMagicBits * kOff);
      } else if (BITS == 4) {   // word 4 chh + u
        *reinterpret_cast<uint32_t*>(codes + (chh * 32 + lane) * 16 + u * 4) = w[t][0] - kMagicBits * kOff;
      } else {                  // word 2 chh + u
        *reinterpret_cast<uint32_t*>(codes + lane * 16 + chh * 8 + u * 4) = w[t][0] - kMagicBits * kOff;
      }
    }
  }
  e[0][0] = e00 + f00;
  e[0][1] = e01 + f01;
  e[1][0] = e10 + f10;
  e[1][1] = e11 + f11;
  return g0.range || g1.range;
}

// Values of one tile (16 tokens) x 128 channels.  ldmatrix.trans hands a lane, per slice of 16
// channels, registers a = 0..3: channel 16 s + r + 8 (a & 1), tokens 8 (a >> 1) + 2 c4 + {0, 1}.  Groups
// are 32 channels of one token: slices 2 g and 2 g + 1, a & 1 and the eight lanes r.  Pair
// k = 2 g + (a >> 1) names the lane's two tokens in group g.
// e[a >> 1][0 / 1], n[a >> 1][0 / 1]: squared error / squared norm of token 8 (a >> 1) + 2 c4 + {0, 1}
// summed over the lane's channels.
template <int BITS>
__device__ __forceinline__ bool ingest_values(uint32_t ld, uint8_t* vp, uint8_t* codes, int lane, uint4* prm, float (&e)[2][2],
                                              float (&n)[2][2]) {
  const int r = lane >> 2, c4 = lane & 3;
  uint32_t my_mn = 0u, my_mx = 0u;
#pragma unroll 1
  for (int g = 0; g < 4; ++g) {
    uint32_t x0[4], x1[4];
    i_ldm4t(ld + g * 64, x0);
    i_ldm4t(ld + g * 64 + 32, x1);
#pragma unroll
    for (int ah = 0; ah < 2; ++ah) {
      uint32_t mn = i_min2(i_min2(x0[2 * ah], x0[2 * ah + 1]), i_min2(x1[2 * ah], x1[2 * ah + 1]));
      uint32_t mx = i_max2(i_max2(x0[2 * ah], x0[2 * ah + 1]), i_max2(x1[2 * ah], x1[2 * ah + 1]));
#pragma unroll
      for (int d = 4; d <= 16; d <<= 1) {
        mn = i_min2(mn, __shfl_xor_sync(kFullI, mn, d));
        mx = i_max2(mx, __shfl_xor_sync(kFullI, mx, d));
      }
      if (r == 2 * g + ah) {
        my_mn = mn;
        my_mx = mx;
      }
    }
  }
  const GroupParams g0 = i_params<BITS>(i_lo(my_mn), i_lo(my_mx)), g1 = i_params<BITS>(i_hi(my_mn), i_hi(my_mx));
  {
    // scales [c4][group] = {tA0, tA1, tB0, tB1}, zeros [group][c4] likewise from fp16 index 64; pair r = (group, a >> 1)
    const int g = r >> 1, ah = r & 1;
    uint16_t* p16 = reinterpret_cast<uint16_t*>(vp);
    *reinterpret_cast<uint32_t*>(p16 + (c4 * 4 + g) * 4 + ah * 2) = static_cast<uint32_t>(g0.s_bits) | (static_cast<uint32_t>(g1.s_bits) << 16);
    *reinterpret_cast<uint32_t*>(p16 + 64 + (g * 4 + c4) * 4 + ah * 2) = static_cast<uint32_t>(g0.z_bits) | (static_cast<uint32_t>(g1.z_bits) << 16);
  }
  prm[r * 4 + c4] = i_pack_params(g0, g1);
  __syncwarp();
  constexpr uint32_t kOff = BITS == 8 ? 0x01010101u : (BITS == 4 ? 0x11111111u : 0x55555555u);
  float e0 = 0.f, e1 = 0.f, e2 = 0.f, e3 = 0.f, n0 = 0.f, n1 = 0.f, n2 = 0.f, n3 = 0.f;
#pragma unroll 1
  for (int g = 0; g < 4; ++g) {
    uint32_t x[2][4];
    i_ldm4t(ld + g * 64, x[0]);
    i_ldm4t(ld + g * 64 + 32, x[1]);
    uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int ah = 0; ah < 2; ++ah) {
      const uint4 P = prm[(2 * g + ah) * 4 + c4];
      const float s0 = i_h_lo(P.x), z0 = i_h_hi(P.x), v0 = __uint_as_float(P.y);
      const float s1 = i_h_lo(P.z), z1 = i_h_hi(P.z), v1 = __uint_as_float(P.w);
#pragma unroll
      for (int ss = 0; ss < 2; ++ss) {
        // word of (slice 2 g + ss, a): 8 bits: 4 g + 2 ss + (a >> 1), 4 bits: 2 g + ss, 2 bits: g
        const int wi = BITS == 8 ? 2 * ss + ah : (BITS == 4 ? ss : 0);
#pragma unroll
        for (int al = 0; al < 2; ++al) {
          const uint32_t xv = x[ss][2 * ah + al];
          i_quant2<BITS>(xv, s0, z0, v0, s1, z1, v1, i_bit_v<BITS>(ss, 2 * ah + al, 0), i_bit_v<BITS>(ss, 2 * ah + al, 1), w[wi],
                         ah == 0 ? e0 : e2, ah == 0 ? e1 : e3);
          const float x0f = i_lo(xv), x1f = i_hi(xv);
          if (ah == 0) {
            n0 = fmaf(x0f, x0f, n0);
            n1 = fmaf(x1f, x1f, n1);
          } else {
            n2 = fmaf(x0f, x0f, n2);
            n3 = fmaf(x1f, x1f, n3);
          }
        }
      }
    }
    if (BITS == 8) {
      *reinterpret_cast<uint4*>(codes + (g * 32 + lane) * 16) =
          make_uint4(w[0] - kMagicBits * kOff, w[1] - kMagicBits * kOff, w[2] - kMagicBits * kOff, w[3] - kMagicBits * kOff);
    } else if (BITS == 4) {
      *reinterpret_cast<uint2*>(codes + ((g >> 1) * 32 + lane) * 16 + (g & 1) * 8) = make_uint2(w[0] - kMagicBits * kOff, w[1] - kMagicBits * kOff);
    } else {
      *reinterpret_cast<uint32_t*>(codes + lane * 16 + g * 4) = w[0] - kMagicBits * kOff;
    }
  }
  e[0][0] = e0;
  e[0][1] = e1;
  e[1][0] = e2;
  e[1][1] = e3;
  n[0][0] = n0;
  n[0][1] = n1;
  n[1][0] = n2;
  n[1][1] = n3;
  return g0.range || g1.range || g0.s > v_scale_limit(BITS) || g1.s > v_scale_limit(BITS);
}

__global__ void __launch_bounds__(kInThreads, 3) ingest_kernel(const __grid_constant__ EncodeParams p) {
  extern __shared__ __align__(16) uint8_t ism[];
  float* cen = reinterpret_cast<float*>(ism + 2 * kInBuf);      // [2][128] centroid of keys, of values
  float* kd2 = cen + 256;                                       // [2 channel halves][64 tokens]
  float* red = kd2 + 128;                                       // [4 value warps][2]: max error, max norm (squared)
  uint4* prm_all = reinterpret_cast<uint4*>(red + 16);          // [8 warps][8 pairs][4 lanes c4]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int r = lane >> 2, c4 = lane & 3, mi = lane >> 3;
  uint4* prm = prm_all + warp * 32;
  const uint32_t sbase = i_u32(ism);
  const size_t row_stride = static_cast<size_t>(p.n_kv_heads) * kD;      // elements between two tokens of a stream

  // work item -> (stream, block, slot, level): from the job list, or counted off in the order
  // (sequence, block, KV head) with slot and level taken from the block table
  auto job_of = [&](int item) -> EncodeJob {
    if (p.jobs) return p.jobs[item];
    const int per_seq = p.n_blocks * p.n_kv_heads;
    const int sq = item / per_seq, rem = item - sq * per_seq;
    EncodeJob job;
    job.block = rem / p.n_kv_heads;
    job.stream = (p.first_seq + sq) * p.n_kv_heads + (rem - job.block * p.n_kv_heads);
    const TableEntry te = p.table[static_cast<size_t>(job.stream) * p.table_stride + job.block];
    job.src_off256 = 0;
    job.dst_off256 = te.off256;
    job.src_level = 0;
    job.dst_level = static_cast<int16_t>(te.level);
    job.pad = 0;
    return job;
  };
  auto stage = [&](int item, int buf) {
    const EncodeJob job = job_of(item);
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
    const EncodeJob job = job_of(item);
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
      uint8_t* half_base = dst + half * half_bytes(L);
      if (L == 8) range = ingest_keys<8>(tile_s, half_base, half, chh, lane, prm, e);
      else if (L == 4) range = ingest_keys<4>(tile_s, half_base, half, chh, lane, prm, e);
      else if (L == 2) range = ingest_keys<2>(tile_s, half_base, half, chh, lane, prm, e);
      else if (L == 1) {
        // distance from the centroid
        const uint32_t ld = tile_s + (32 * half + (mi & 1) * 8 + (lane & 7)) * kInRow + (64 * chh + (mi >> 1) * 8) * 2;
#pragma unroll 1
        for (int sl = 0; sl < 4; ++sl) {
          uint32_t x[2][4];
          i_ldm4(ld + sl * 32, x[0]);
          i_ldm4(ld + 16 * kInRow + sl * 32, x[1]);
#pragma unroll
          for (int ah = 0; ah < 2; ++ah) {
            const float2 cc = *reinterpret_cast<const float2*>(cen + 64 * chh + 16 * sl + 8 * ah + 2 * c4);
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
              for (int al = 0; al < 2; ++al) {
                const float d0 = i_lo(x[t][2 * ah + al]) - cc.x, d1 = i_hi(x[t][2 * ah + al]) - cc.y;
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
      const uint32_t ld = tile_s + kInTensor + (16 * tile + (mi >> 1) * 8 + (lane & 7)) * kInRow + ((mi & 1) * 8) * 2;
      float e[2][2] = {{0.f, 0.f}, {0.f, 0.f}}, n[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
      if (L != 16 && L != 1) {
        uint8_t* hb = dst + (tile >> 1) * half_bytes(L);
        uint8_t* vp = hb + off_vp(L, tile & 1);
        uint8_t* codes = hb + off_vc(L, tile & 1);
        if (L == 8) range = ingest_values<8>(ld, vp, codes, lane, prm, e, n);
        else if (L == 4) range = ingest_values<4>(ld, vp, codes, lane, prm, e, n);
        else range = ingest_values<2>(ld, vp, codes, lane, prm, e, n);
      } else {
        // squared norms of the rows; for a centroid block also the distance from the centroid
#pragma unroll 1
        for (int s = 0; s < 8; ++s) {
          uint32_t x[4];
          i_ldm4t(ld + s * 32, x);
#pragma unroll
          for (int al = 0; al < 2; ++al) {
            const float cc = L == 1 ? cen[kD + 16 * s + r + 8 * al] : 0.f;
#pragma unroll
            for (int ah = 0; ah < 2; ++ah) {
              const float x0 = i_lo(x[2 * ah + al]), x1 = i_hi(x[2 * ah + al]);
              n[ah][0] = fmaf(x0, x0, n[ah][0]);
              n[ah][1] = fmaf(x1, x1, n[ah][1]);
              if (L == 1) {
                const float d0 = x0 - cc, d1 = x1 - cc;
                e[ah][0] = fmaf(d0, d0, e[ah][0]);
                e[ah][1] = fmaf(d1, d1, e[ah][1]);
              }
            }
          }
        }
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

// ---- latent-attention (MLA) streams -------------------------------------------------------------
// One 576-wide row per token, quantised with the key rule (groups of 32 tokens of one channel);
// codes are stored row-major, a chunk of 8 neighbouring channels of a token per 32-bit word (4 bits)
// or pair of words (8 bits).  Thread = (half of the block, chunk): it owns the 8 groups of its
// chunk, so nothing is exchanged between threads.  The block (73.7 KB, contiguous in the input) is
// staged in shared memory with 16-byte cp.async copies; three CTAs per SM take turns loading and
// encoding.
constexpr int kMlaInThreads = 160;                       // 144 = 2 halves x 72 chunks work on quantised blocks
constexpr int kMlaInTile = kBlock * kMlaRowBytes;         // 73728

// code of x as an integer in the low mantissa bits of (clamped value + 1.5 * 2^23)
template <int BITS>
__device__ __forceinline__ uint32_t i_code(float x, float z, float inv) {
  constexpr float qmax = static_cast<float>((1 << BITS) - 1);
  return __float_as_uint(__fadd_rn(fminf(fmaxf(__fmul_rn(__fsub_rn(x, z), inv), 0.f), qmax), kMagic));
}

template <int BITS>
__device__ __forceinline__ bool mla_ingest_quant(const uint8_t* tile, uint8_t* dst, int tid) {
  const int half = tid / kMlaChunks, j = tid - half * kMlaChunks;
  const uint8_t* rows = tile + (32 * half) * kMlaRowBytes + j * 16;
  uint4 mn = *reinterpret_cast<const uint4*>(rows), mx = mn;
#pragma unroll 4
  for (int t = 1; t < kGroup; ++t) {
    const uint4 v = *reinterpret_cast<const uint4*>(rows + t * kMlaRowBytes);
    mn.x = i_min2(mn.x, v.x);
    mn.y = i_min2(mn.y, v.y);
    mn.z = i_min2(mn.z, v.z);
    mn.w = i_min2(mn.w, v.w);
    mx.x = i_max2(mx.x, v.x);
    mx.y = i_max2(mx.y, v.y);
    mx.z = i_max2(mx.z, v.z);
    mx.w = i_max2(mx.w, v.w);
  }
  const uint32_t mnr[4] = {mn.x, mn.y, mn.z, mn.w}, mxr[4] = {mx.x, mx.y, mx.z, mx.w};
  float z[8], inv[8];
  uint32_t sb[4], zb[4];
  bool range = false;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const GroupParams g0 = i_params<BITS>(i_lo(mnr[i]), i_lo(mxr[i])), g1 = i_params<BITS>(i_hi(mnr[i]), i_hi(mxr[i]));
    z[2 * i] = g0.z;
    z[2 * i + 1] = g1.z;
    inv[2 * i] = g0.inv;
    inv[2 * i + 1] = g1.inv;
    sb[i] = static_cast<uint32_t>(g0.s_bits) | (static_cast<uint32_t>(g1.s_bits) << 16);
    zb[i] = static_cast<uint32_t>(g0.z_bits) | (static_cast<uint32_t>(g1.z_bits) << 16);
    range |= g0.range || g1.range;
  }
  uint8_t* hb = dst + half * mla_half_bytes(BITS);
  // parameters: the 576 fp16 scales, then the 576 fp16 zero points; chunk j owns piece j of each
  *reinterpret_cast<uint4*>(hb + j * 16) = make_uint4(sb[0], sb[1], sb[2], sb[3]);
  *reinterpret_cast<uint4*>(hb + kMlaZeroOff * 2 + j * 16) = make_uint4(zb[0], zb[1], zb[2], zb[3]);
  uint8_t* codes = hb + mla_kp_bytes() + j * BITS;
#pragma unroll 2
  for (int t = 0; t < kGroup; ++t) {
    const uint4 v = *reinterpret_cast<const uint4*>(rows + t * kMlaRowBytes);
    const uint32_t u0 = i_code<BITS>(i_lo(v.x), z[0], inv[0]), u1 = i_code<BITS>(i_hi(v.x), z[1], inv[1]);
    const uint32_t u2 = i_code<BITS>(i_lo(v.y), z[2], inv[2]), u3 = i_code<BITS>(i_hi(v.y), z[3], inv[3]);
    const uint32_t u4 = i_code<BITS>(i_lo(v.z), z[4], inv[4]), u5 = i_code<BITS>(i_hi(v.z), z[5], inv[5]);
    const uint32_t u6 = i_code<BITS>(i_lo(v.w), z[6], inv[6]), u7 = i_code<BITS>(i_hi(v.w), z[7], inv[7]);
    if (BITS == 8) {
      // channel c of a word's four sits at byte ((c & 3) >> 1) + 2 (c & 1)
      const uint32_t w0 = u0 + (u2 << 8) + (u1 << 16) + (u3 << 24) - kMagicBits * 0x01010101u;
      const uint32_t w1 = u4 + (u6 << 8) + (u5 << 16) + (u7 << 24) - kMagicBits * 0x01010101u;
      *reinterpret_cast<uint2*>(codes + t * mla_code_row_bytes(8)) = make_uint2(w0, w1);
    } else {
      // channel c sits at bit 4 (c >> 1) + 16 (c & 1)
      const uint32_t w0 = u0 + (u2 << 4) + (u4 << 8) + (u6 << 12) + (u1 << 16) + (u3 << 20) + (u5 << 24) + (u7 << 28) -
                          kMagicBits * 0x11111111u;
      *reinterpret_cast<uint32_t*>(codes + t * mla_code_row_bytes(4)) = w0;
    }
  }
  return range;
}

__global__ void __launch_bounds__(kMlaInThreads, 3) mla_ingest_kernel(const __grid_constant__ MlaEncodeParams p) {
  extern __shared__ __align__(16) uint8_t msm[];
  const int tid = threadIdx.x;
  const uint32_t sbase = i_u32(msm);
  constexpr int kChunks = kMlaInTile / 16;               // 4608
  for (int item = blockIdx.x; item < p.n_jobs; item += gridDim.x) {
    const EncodeJob job = p.jobs[item];
    const uint8_t* src = reinterpret_cast<const uint8_t*>(
        p.k_in + (static_cast<size_t>(job.stream) * p.n_tok + static_cast<size_t>(job.block) * kBlock) * kMlaDk);
    __syncthreads();                                     // everybody is done with the previous block
    for (int q = tid; q < kChunks; q += kMlaInThreads) i_cp16(sbase + q * 16, src + q * 16);
    i_commit();
    i_wait_all();
    __syncthreads();
    uint8_t* dst = p.arena + static_cast<size_t>(job.dst_off256) * 256;
    const int L = job.dst_level;
    if (L == 16) {
      for (int q = tid; q < kChunks; q += kMlaInThreads)
        *reinterpret_cast<uint4*>(dst + q * 16) = *reinterpret_cast<const uint4*>(msm + q * 16);
    } else if (L == 1) {
      for (int c = tid; c < kMlaDk; c += kMlaInThreads) {
        const uint16_t* col = reinterpret_cast<const uint16_t*>(msm) + c;
        float acc = 0.f;
#pragma unroll 16
        for (int t = 0; t < kBlock; ++t) acc = __fadd_rn(acc, __uint_as_float(static_cast<uint32_t>(col[t * kMlaDk]) << 16));
        reinterpret_cast<uint16_t*>(dst)[c] = i_bf16(__fmul_rn(acc, 1.0f / kBlock));
      }
    } else if (tid < 2 * kMlaChunks) {
      const bool range = L == 8 ? mla_ingest_quant<8>(msm, dst, tid) : mla_ingest_quant<4>(msm, dst, tid);
      if (range) atomicOr(p.status, kStatusRange);
    }
  }
}

}  // namespace

// All jobs read the bf16 input rows (src_level == 0); without a job list the work is counted off the block table.
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

namespace gkv {
// Bulk ingest of latent-attention rows: every job reads the bf16 input (src_level == 0), rows 16-byte aligned.
cudaError_t launch_mla_ingest(const MlaEncodeParams& p, cudaStream_t st) {
  if (p.n_jobs <= 0) return cudaSuccess;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(mla_ingest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMlaInTile);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int grid = p.n_jobs < 148 * 3 ? p.n_jobs : 148 * 3;
  mla_ingest_kernel<<<grid, kMlaInThreads, kMlaInTile, st>>>(p);
  return cudaGetLastError();
}
}  // namespace gkv
