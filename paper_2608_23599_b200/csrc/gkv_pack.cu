// Block encode / requantise / statistics kernels (paper Sec. 3.2 ladder and monotone demotion,
// Sec. 3.4 residual score, Sec. 3.5 boxes).  Everything that decides a stored bit follows one
// written evaluation order in IEEE fp32 (fp64 for the residual score) with explicit
// round-to-nearest intrinsics, so results do not depend on compiler contraction:
//   quantise a group to b bits:  s = fp16((max - min) / (2^b - 1)), z = fp16(min) (saturating),
//                                code = clamp(rint((x - z) * (1 / s)), 0, 2^b - 1), s == 0 -> code 0
//   dequantise:                  x^ = fma(code, s, z)
//   centroid:                    sequential sum over the 64 tokens, times 1/64, rounded to bf16
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gkv_internal.h"

namespace gkv {
namespace {

constexpr int kTileLd = kD + 1;   // padded fp32 tile row

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }
__device__ __forceinline__ uint16_t f32_to_bf16_bits(float x) {
  __nv_bfloat16 h = __float2bfloat16_rn(x);
  return *reinterpret_cast<uint16_t*>(&h);
}
__device__ __forceinline__ uint16_t f32_to_fp16_bits_sat(float x) {
  x = fminf(fmaxf(x, -65504.f), 65504.f);
  __half h = __float2half_rn(x);
  return *reinterpret_cast<uint16_t*>(&h);
}
__device__ __forceinline__ float fp16_bits_to_f32(uint16_t b) {
  __half h = *reinterpret_cast<__half*>(&b);
  return __half2float(h);
}

// Read code (tok, ch) of a quantised tensor from its slot half/tile regions.
__device__ __forceinline__ int read_code(const uint8_t* slot, int bits, bool is_v, int tok, int ch) {
  int tile, lane, s, a, hlf;
  if (is_v) v_coord(tok, ch, &tile, &lane, &s, &a, &hlf);
  else k_coord(tok, ch, &tile, &lane, &s, &a, &hlf);
  int boff, bit;
  code_pos(bits, is_v, lane, s, a, hlf, &boff, &bit);
  const int half = tile >> 1, t = tile & 1;
  const uint8_t* region = slot + half * half_bytes(bits) + (is_v ? off_vc(bits, t) : off_kc(bits, t));
  const uint32_t w = *reinterpret_cast<const uint32_t*>(region + boff);
  return static_cast<int>((w >> bit) & ((1u << bits) - 1u));
}

// Fill an fp32 tile [64][kTileLd] with the block's current reconstruction.
__device__ void load_tile(float* tile, const uint8_t* arena, const EncodeParams& p, const EncodeJob& job, bool is_v) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  if (job.src_level == 0) {
    const uint16_t* in = is_v ? p.v_in : p.k_in;
    const int b = job.stream / p.n_kv_heads, kvh = job.stream - b * p.n_kv_heads;
    for (int i = tid; i < kBlock * kD; i += nthr) {
      const int t = i >> 7, c = i & (kD - 1);
      const size_t tok = static_cast<size_t>(b) * p.n_tok + static_cast<size_t>(job.block) * kBlock + t;
      tile[t * kTileLd + c] = bf16_bits_to_f32(in[(tok * p.n_kv_heads + kvh) * kD + c]);
    }
    return;
  }
  const uint8_t* slot = arena + static_cast<size_t>(job.src_off256) * 256;
  if (job.src_level == 16) {
    const uint16_t* rows = reinterpret_cast<const uint16_t*>(slot + (is_v ? kBlock * kRowBytes : 0));
    for (int i = tid; i < kBlock * kD; i += nthr) tile[(i >> 7) * kTileLd + (i & (kD - 1))] = bf16_bits_to_f32(rows[i]);
    return;
  }
  const int bits = job.src_level;
  for (int i = tid; i < kBlock * kD; i += nthr) {
    const int t = i >> 7, c = i & (kD - 1);
    const int code = read_code(slot, bits, is_v, t, c);
    const uint8_t* hb = slot + (t >> 5) * half_bytes(bits);
    float s, z;
    if (!is_v) {
      const uint16_t* kp = reinterpret_cast<const uint16_t*>(hb + off_kp());
      const int idx = kp_index(c);
      s = fp16_bits_to_f32(kp[idx]);
      z = fp16_bits_to_f32(kp[kp_zero_index(c)]);
    } else {
      const uint16_t* vp = reinterpret_cast<const uint16_t*>(hb + off_vp(bits, (t >> 4) & 1));
      s = fp16_bits_to_f32(vp[vp_scale_index(t & 15, c >> 5)]);
      z = fp16_bits_to_f32(vp[vp_zero_index(t & 15, c >> 5)]);
    }
    tile[t * kTileLd + c] = __fmaf_rn(static_cast<float>(code), s, z);
  }
}

// Quantise one group of 32 values read with a stride; writes codes through `put`.
struct QuantOut {
  uint16_t s_bits, z_bits;
  bool range;
};
__device__ __forceinline__ QuantOut quant_params(float mn, float mx, int bits) {
  const float qmax = static_cast<float>((1 << bits) - 1);
  const float s_raw = __fdiv_rn(__fsub_rn(mx, mn), qmax);
  QuantOut o;
  o.range = fabsf(s_raw) > 65504.f || fabsf(mn) > 65504.f;
  o.s_bits = f32_to_fp16_bits_sat(s_raw);
  o.z_bits = f32_to_fp16_bits_sat(mn);
  return o;
}
__device__ __forceinline__ uint8_t quant_code(float x, float s32, float z32, float inv, float qmax) {
  const float t = __fmul_rn(__fsub_rn(x, z32), inv);
  const float c = fminf(fmaxf(rintf(t), 0.f), qmax);
  return static_cast<uint8_t>(c);
}

// Pack the logical codes [64][128] (shared) of one tensor into the slot's fragment-ordered words.
__device__ void pack_codes(uint8_t* slot, const uint8_t* codes, int bits, bool is_v) {
  const int words_per_lane = 2 * bits;           // 64 codes of `bits` bits per lane and tile
  const int total = 4 * 32 * words_per_lane;
  for (int i = threadIdx.x; i < total; i += blockDim.x) {
    const int w = i % words_per_lane;
    const int lane = (i / words_per_lane) & 31;
    const int tile = i / (words_per_lane * 32);
    const int r = lane >> 2, c4 = lane & 3;
    uint32_t word = 0;
    // the 32 / bits codes (s, a, hlf) that live in word w of this lane (the inverse of code_pos)
    const int per = 32 / bits;
    for (int q = 0; q < per; ++q) {
      int s, a, hlf;
      if (bits == 8) {
        s = w >> 1;
        a = ((w & 1) << 1) | (q & 1);
        hlf = q >> 1;
      } else if (bits == 4) {
        s = w;
        a = q & 3;
        hlf = q >> 2;
      } else {
        s = 2 * w + (q & 1);
        a = (q >> 1) & 3;
        hlf = q >> 3;
      }
      int boff, bit;
      code_pos(bits, is_v, lane, s, a, hlf, &boff, &bit);
      int tok, ch;
      if (!is_v) {
        tok = 16 * tile + r + 8 * (a & 1);
        ch = 16 * s + 8 * (a >> 1) + 2 * c4 + hlf;
      } else {
        ch = 16 * s + r + 8 * (a & 1);
        tok = 16 * tile + 8 * (a >> 1) + 2 * c4 + hlf;
      }
      word |= static_cast<uint32_t>(codes[tok * kD + ch]) << bit;
    }
    const int half = tile >> 1, t = tile & 1;
    uint8_t* region = slot + half * half_bytes(bits) + (is_v ? off_vc(bits, t) : off_kc(bits, t));
    *reinterpret_cast<uint32_t*>(region + ((w >> 2) * 32 + lane) * 16 + (w & 3) * 4) = word;
  }
}

__global__ void __launch_bounds__(256) encode_kernel(const __grid_constant__ EncodeParams p) {
  extern __shared__ __align__(16) uint8_t esm[];
  float* tile = reinterpret_cast<float*>(esm);                       // [64][kTileLd]
  uint8_t* codes = esm + kBlock * kTileLd * sizeof(float);           // [64][128]
  float* ps = reinterpret_cast<float*>(codes + kBlock * kD);         // [256] scales (or the centroid row) of the tensor
  float* pz = ps + 256;                                              // [256] zero points
  float* red = pz + 256;                                             // [16] per-warp maxima
  const int tid = threadIdx.x;
  // a work item is one tensor (keys or values) of one job: the two halves of a job are independent
  // (separate regions of the slot, separate components of the error bounds) and run in different CTAs
  for (int item = blockIdx.x; item < 2 * p.n_jobs; item += gridDim.x) {
    const EncodeJob job = p.jobs[item >> 1];
    uint8_t* dst = p.arena + static_cast<size_t>(job.dst_off256) * 256;
    const int L = job.dst_level;
    const bool from_original = job.src_level == 0 || job.src_level == 16;
    float* bound_out = p.err ? reinterpret_cast<float*>(p.err + static_cast<size_t>(job.stream) * p.err_stride + job.block) : nullptr;
    float4 bound = make_float4(0.f, 0.f, 0.f, 0.f);
    if (p.err && !from_original && tid == 0) bound = *reinterpret_cast<const float4*>(bound_out);
    {
      const int tensor = item & 1;
      const bool is_v = tensor == 1;
      __syncthreads();
      load_tile(tile, p.arena, p, job, is_v);
      __syncthreads();
      if (L == 16) {
        uint16_t* rows = reinterpret_cast<uint16_t*>(dst + (is_v ? kBlock * kRowBytes : 0));
        for (int i = tid; i < kBlock * kD; i += blockDim.x)
          rows[i] = f32_to_bf16_bits(tile[(i >> 7) * kTileLd + (i & (kD - 1))]);
      } else if (L == 1) {
        if (tid < kD) {
          float acc = 0.f;
          for (int t = 0; t < kBlock; ++t) acc = __fadd_rn(acc, tile[t * kTileLd + tid]);
          uint16_t* row = reinterpret_cast<uint16_t*>(dst + (is_v ? kRowBytes : 0));
          const uint16_t cb = f32_to_bf16_bits(__fmul_rn(acc, 1.0f / kBlock));
          row[tid] = cb;
          ps[tid] = bf16_bits_to_f32(cb);
        }
      } else {
        const float qmax = static_cast<float>((1 << L) - 1);
        bool range = false;
        if (!is_v) {
          // keys: group = 32 tokens x 1 channel; thread = (half, channel)
          const int half = tid >> 7, c = tid & (kD - 1);
          float mn = tile[(32 * half) * kTileLd + c], mx = mn;
          for (int t = 1; t < kGroup; ++t) {
            const float x = tile[(32 * half + t) * kTileLd + c];
            mn = fminf(mn, x);
            mx = fmaxf(mx, x);
          }
          const QuantOut q = quant_params(mn, mx, L);
          range = q.range;
          const float s32 = fp16_bits_to_f32(q.s_bits), z32 = fp16_bits_to_f32(q.z_bits);
          const float inv = s32 > 0.f ? __fdiv_rn(1.f, s32) : 0.f;
          for (int t = 0; t < kGroup; ++t)
            codes[(32 * half + t) * kD + c] = quant_code(tile[(32 * half + t) * kTileLd + c], s32, z32, inv, qmax);
          uint16_t* kp = reinterpret_cast<uint16_t*>(dst + half * half_bytes(L) + off_kp());
          const int idx = kp_index(c);
          kp[idx] = q.s_bits;
          kp[kp_zero_index(c)] = q.z_bits;
          ps[tid] = s32;                 // index = half * 128 + channel
          pz[tid] = z32;
        } else {
          // values: group = 1 token x 32 channels; thread = (token, group)
          const int t = tid >> 2, g = tid & 3;
          float mn = tile[t * kTileLd + 32 * g], mx = mn;
          for (int c = 1; c < kGroup; ++c) {
            const float x = tile[t * kTileLd + 32 * g + c];
            mn = fminf(mn, x);
            mx = fmaxf(mx, x);
          }
          const QuantOut q = quant_params(mn, mx, L);
          const float s32 = fp16_bits_to_f32(q.s_bits), z32 = fp16_bits_to_f32(q.z_bits);
          range = q.range || s32 > v_scale_limit(L);
          const float inv = s32 > 0.f ? __fdiv_rn(1.f, s32) : 0.f;
          for (int c = 0; c < kGroup; ++c)
            codes[t * kD + 32 * g + c] = quant_code(tile[t * kTileLd + 32 * g + c], s32, z32, inv, qmax);
          uint16_t* vp = reinterpret_cast<uint16_t*>(dst + (t >> 5) * half_bytes(L) + off_vp(L, (t >> 4) & 1));
          vp[vp_scale_index(t & 15, g)] = q.s_bits;
          vp[vp_zero_index(t & 15, g)] = q.z_bits;
          ps[tid] = s32;                 // index = token * 4 + group
          pz[tid] = z32;
        }
        if (range) atomicOr(p.status, kStatusRange);
        __syncthreads();
        pack_codes(dst, codes, L, is_v);
      }
      if (p.err) {
        // Distance of the new representation from what it was made of: per token the 2-norm over
        // the channels (thread = token x 32-channel quarter, fixed summation order), then the
        // largest token.  The bound against the original rows grows by it (triangle inequality);
        // for a block made from its original rows it is the distance itself.
        __syncthreads();
        const int t = tid >> 2, g = tid & 3;
        float d2 = 0.f, n2 = 0.f;
        for (int c = 32 * g; c < 32 * g + 32; ++c) {
          const float x = tile[t * kTileLd + c];
          float xh = x;
          if (L == 1) xh = ps[c];
          else if (L != 16) {
            const int pi = is_v ? t * 4 + g : (t >> 5) * kD + c;
            xh = __fmaf_rn(static_cast<float>(codes[t * kD + c]), ps[pi], pz[pi]);
          }
          const float d = x - xh;
          d2 = fmaf(d, d, d2);
          n2 = fmaf(x, x, n2);
        }
        d2 += __shfl_xor_sync(0xffffffffu, d2, 1);
        d2 += __shfl_xor_sync(0xffffffffu, d2, 2);
        n2 += __shfl_xor_sync(0xffffffffu, n2, 1);
        n2 += __shfl_xor_sync(0xffffffffu, n2, 2);
#pragma unroll
        for (int s = 4; s <= 16; s <<= 1) {
          d2 = fmaxf(d2, __shfl_xor_sync(0xffffffffu, d2, s));
          n2 = fmaxf(n2, __shfl_xor_sync(0xffffffffu, n2, s));
        }
        if ((tid & 31) == 0) {
          red[tid >> 5] = d2;
          red[8 + (tid >> 5)] = n2;
        }
        __syncthreads();
        if (tid == 0) {
          float dm = red[0], nm = red[8];
          for (int w = 1; w < 8; ++w) {
            dm = fmaxf(dm, red[w]);
            nm = fmaxf(nm, red[8 + w]);
          }
          if (!is_v) bound.x += sqrtf(dm);
          else {
            bound.y += sqrtf(dm);
            if (from_original) bound.z = sqrtf(nm);
          }
        }
      }
    }
    if (p.err && tid == 0) {
      if ((item & 1) == 0) {
        bound_out[0] = bound.x;            // keys: x
      } else {
        bound_out[1] = bound.y;            // values: y, z; w stays 0
        bound_out[2] = bound.z;
        bound_out[3] = 0.f;
      }
    }
    if (p.table && tid == 0 && (item & 1) == 0) {
      TableEntry* te = p.table + static_cast<size_t>(job.stream) * p.table_stride + job.block;
      te->off256 = job.dst_off256;
      te->level = static_cast<uint32_t>(job.dst_level);
    }
  }
}

// Per closed block: exact per-page key boxes (min/max of the unquantised bf16 keys), the block's
// largest per-channel key range (allocator's range proxy) and its attention mass (sequential sum).
__global__ void __launch_bounds__(kD) stats_kernel(const __grid_constant__ StatsParams p) {
  const int bi = blockIdx.x, stream = blockIdx.y, c = threadIdx.x;
  const int block = p.first_block + bi;
  const int b = stream / p.n_kv_heads, kvh = stream - b * p.n_kv_heads;
  const uint16_t* rows;
  size_t row_stride;
  if (p.k_in) {
    rows = p.k_in + ((static_cast<size_t>(b) * p.n_tok + static_cast<size_t>(block) * kBlock) * p.n_kv_heads + kvh) * kD;
    row_stride = static_cast<size_t>(p.n_kv_heads) * kD;
  } else {
    const TableEntry e = p.table[static_cast<size_t>(stream) * p.table_stride + block];
    rows = reinterpret_cast<const uint16_t*>(p.arena + static_cast<size_t>(e.off256) * 256);
    row_stride = kD;
  }
  float bmn = 0.f, bmx = 0.f;
  const int page = p.page_tokens > 0 ? p.page_tokens : kBlock;
  // The block's 64 values of this channel are fetched 16 at a time (independent loads, issued
  // together) and folded into the running page minimum / maximum; a page is 16, 32 or 64 tokens.
  uint16_t lo_b = 0, hi_b = 0;
  float lo = 0.f, hi = 0.f;
#pragma unroll 1
  for (int t0 = 0; t0 < kBlock; t0 += 16) {
    uint16_t xb[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) xb[i] = rows[static_cast<size_t>(t0 + i) * row_stride + c];
    if (t0 % page == 0) {
      lo_b = hi_b = xb[0];
      lo = hi = bf16_bits_to_f32(xb[0]);
    }
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float x = bf16_bits_to_f32(xb[i]);
      if (x < lo) { lo = x; lo_b = xb[i]; }
      if (x > hi) { hi = x; hi_b = xb[i]; }
    }
    if ((t0 + 16) % page == 0) {                       // the page is complete
      const int p0 = t0 + 16 - page;
      if (p.page_tokens > 0) {
        const int pg = block * (kBlock / page) + p0 / page;
        uint16_t* bx = p.boxes + (static_cast<size_t>(stream) * kD + c) * 2 * p.box_stride;
        bx[pg] = lo_b;
        bx[p.box_stride + pg] = hi_b;
      }
      if (p0 == 0) { bmn = lo; bmx = hi; }
      else { bmn = fminf(bmn, lo); bmx = fmaxf(bmx, hi); }
    }
  }
  if (p.block_range) {
    __shared__ float red[kD];
    red[c] = __fsub_rn(bmx, bmn);
    __syncthreads();
    for (int s = kD / 2; s > 0; s >>= 1) {
      if (c < s) red[c] = fmaxf(red[c], red[c + s]);
      __syncthreads();
    }
    if (c == 0) p.block_range[static_cast<size_t>(stream) * (p.stat_stride ? p.stat_stride : p.n_blocks) + p.stat_base + bi] = red[0];
  }
  if (p.block_mass && c == 0) {
    const float* m = p.token_mass + static_cast<size_t>(stream) * p.n_tok + static_cast<size_t>(block) * kBlock;
    float acc = 0.f;
    for (int t = 0; t < kBlock; ++t) acc = __fadd_rn(acc, m[t]);
    p.block_mass[static_cast<size_t>(stream) * (p.stat_stride ? p.stat_stride : p.n_blocks) + p.stat_base + bi] = acc;
  }
  if (p.err && !p.k_in) {
    // a block that closes in place (exact rows): no error yet, largest value-row norm for the
    // certificate.  Warp w takes tokens w, w + 4, ...; a lane sums four channels.
    __shared__ float vred[kD / 32];
    const uint16_t* vrows = rows + kBlock * kD;
    const int warp = c >> 5, lane = c & 31;
    float best = 0.f;
    for (int t = warp; t < kBlock; t += kD / 32) {
      const uint2 raw = *reinterpret_cast<const uint2*>(vrows + t * kD + 4 * lane);
      const float x0 = bf16_bits_to_f32(static_cast<uint16_t>(raw.x & 0xffffu)), x1 = bf16_bits_to_f32(static_cast<uint16_t>(raw.x >> 16));
      const float x2 = bf16_bits_to_f32(static_cast<uint16_t>(raw.y & 0xffffu)), x3 = bf16_bits_to_f32(static_cast<uint16_t>(raw.y >> 16));
      float n2 = fmaf(x0, x0, fmaf(x1, x1, fmaf(x2, x2, x3 * x3)));
      for (int s = 1; s <= 16; s <<= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, s);
      best = fmaxf(best, n2);
    }
    if (lane == 0) vred[warp] = best;
    __syncthreads();
    if (c == 0) {
      float m = vred[0];
      for (int w = 1; w < kD / 32; ++w) m = fmaxf(m, vred[w]);
      p.err[static_cast<size_t>(stream) * p.err_stride + block] = make_float4(0.f, 0.f, sqrtf(m), 0.f);
    }
  }
}

// Copy token rows [first_tok, first_tok + n_rows) of the input into rows dst_row0.. of every
// stream's tail slot (exact tier, natural row-major layout).
__global__ void __launch_bounds__(128) append_rows_kernel(uint8_t* arena, const TableEntry* table, int table_stride,
                                                          int tail_index, int n_kv_heads, const uint16_t* k_in,
                                                          const uint16_t* v_in, int n_tok, int first_tok,
                                                          int dst_row0) {
  const int stream = blockIdx.x, row = blockIdx.y;
  const int b = stream / n_kv_heads, kvh = stream - b * n_kv_heads;
  const TableEntry e = table[static_cast<size_t>(stream) * table_stride + tail_index];
  uint8_t* slot = arena + static_cast<size_t>(e.off256) * 256;
  const bool is_v = threadIdx.x >= 64;
  const int i = threadIdx.x & 63;
  const uint16_t* in = is_v ? v_in : k_in;
  const uint32_t* src = reinterpret_cast<const uint32_t*>(
      in + ((static_cast<size_t>(b) * n_tok + first_tok + row) * n_kv_heads + kvh) * kD);
  uint32_t* dst = reinterpret_cast<uint32_t*>(slot + (is_v ? kBlock * kRowBytes : 0) +
                                              static_cast<size_t>(dst_row0 + row) * kRowBytes);
  // launched with programmatic stream serialisation: the address set-up above overlaps the tail
  // of the previous kernel; the new rows are read, and the slot written, only after it completed
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  dst[i] = src[i];
}

// Residual score per token (Sec. 3.4): mass * || v - value centroid of its block ||^2, with the
// centroid taken by the sequential-sum rule on the original values; fp64 sequential in channels.
__global__ void __launch_bounds__(kD) residual_score_kernel(const uint16_t* v_in, const float* token_mass,
                                                            const int8_t* levels, int levels_stride,
                                                            int n_sink_blocks, int n_kv_heads, int n_tok,
                                                            float* scores) {
  const int block = blockIdx.x, stream = blockIdx.y, tid = threadIdx.x;
  const int b = stream / n_kv_heads, kvh = stream - b * n_kv_heads;
  float* out = scores + static_cast<size_t>(stream) * n_tok + static_cast<size_t>(block) * kBlock;
  const int level = levels[static_cast<size_t>(stream) * levels_stride + block];
  if (block < n_sink_blocks || level == 16) {
    if (tid < kBlock) out[tid] = -__builtin_huge_valf();
    return;
  }
  __shared__ double cen[kD];
  __shared__ uint16_t vals[kBlock][kD + 2];
  const uint16_t* rows = v_in + ((static_cast<size_t>(b) * n_tok + static_cast<size_t>(block) * kBlock) * n_kv_heads + kvh) * kD;
  const size_t row_stride = static_cast<size_t>(n_kv_heads) * kD;
  float acc = 0.f;
  for (int t = 0; t < kBlock; ++t) {
    const uint16_t xb = rows[t * row_stride + tid];
    vals[t][tid] = xb;
    acc = __fadd_rn(acc, bf16_bits_to_f32(xb));
  }
  cen[tid] = static_cast<double>(bf16_bits_to_f32(f32_to_bf16_bits(__fmul_rn(acc, 1.0f / kBlock))));
  __syncthreads();
  if (tid < kBlock) {
    double err = 0.0;
    for (int c = 0; c < kD; ++c) {
      const double d = __dsub_rn(static_cast<double>(bf16_bits_to_f32(vals[tid][c])), cen[c]);
      err = __dadd_rn(err, __dmul_rn(d, d));
    }
    const double m = static_cast<double>(token_mass[static_cast<size_t>(stream) * n_tok + static_cast<size_t>(block) * kBlock + tid]);
    out[tid] = __double2float_rn(__dmul_rn(m, err));
  }
}

// Copy the selected residual tokens' exact K and V rows into the stream's residual pool
// (row j: [K row 256 B | V row 256 B]).
__global__ void __launch_bounds__(128) residual_gather_kernel(uint8_t* arena, const uint16_t* k_in,
                                                              const uint16_t* v_in, int n_tok, int n_kv_heads,
                                                              const int32_t* idx, int idx_stride,
                                                              const int32_t* count, const uint32_t* res_off256) {
  const int j = blockIdx.x, stream = blockIdx.y;
  if (j >= count[stream]) return;
  const int b = stream / n_kv_heads, kvh = stream - b * n_kv_heads;
  const int tok = idx[static_cast<size_t>(stream) * idx_stride + j];
  const bool is_v = threadIdx.x >= 64;
  const int i = threadIdx.x & 63;
  const uint16_t* in = is_v ? v_in : k_in;
  const uint32_t* src = reinterpret_cast<const uint32_t*>(in + ((static_cast<size_t>(b) * n_tok + tok) * n_kv_heads + kvh) * kD);
  uint32_t* dst = reinterpret_cast<uint32_t*>(arena + static_cast<size_t>(res_off256[stream]) * 256 +
                                              static_cast<size_t>(j) * 2 * kRowBytes + (is_v ? kRowBytes : 0));
  dst[i] = src[i];
}

// Parity helper: logical view of one tensor of one slot.
__global__ void __launch_bounds__(256) export_kernel(const uint8_t* arena, uint32_t off256, int level, int which,
                                                     uint8_t* codes, uint16_t* scale, uint16_t* zero, uint16_t* rows) {
  const uint8_t* slot = arena + static_cast<size_t>(off256) * 256;
  const bool is_v = which == 1;
  const int tid = threadIdx.x;
  if (level == 16) {
    const uint16_t* src = reinterpret_cast<const uint16_t*>(slot + (is_v ? kBlock * kRowBytes : 0));
    for (int i = tid; i < kBlock * kD; i += blockDim.x) rows[i] = src[i];
    return;
  }
  if (level == 1) {
    const uint16_t* src = reinterpret_cast<const uint16_t*>(slot + (is_v ? kRowBytes : 0));
    if (tid < kD) rows[tid] = src[tid];
    return;
  }
  for (int i = tid; i < kBlock * kD; i += blockDim.x) codes[i] = static_cast<uint8_t>(read_code(slot, level, is_v, i >> 7, i & (kD - 1)));
  if (!is_v) {
    // [2][128]
    const int half = tid >> 7, c = tid & (kD - 1);
    const uint16_t* kp = reinterpret_cast<const uint16_t*>(slot + half * half_bytes(level) + off_kp());
    scale[half * kD + c] = kp[kp_index(c)];
    zero[half * kD + c] = kp[kp_zero_index(c)];
  } else {
    // [64][4]
    const int t = tid >> 2, g = tid & 3;
    const uint16_t* vp = reinterpret_cast<const uint16_t*>(slot + (t >> 5) * half_bytes(level) + off_vp(level, (t >> 4) & 1));
    scale[t * 4 + g] = vp[vp_scale_index(t & 15, g)];
    zero[t * 4 + g] = vp[vp_zero_index(t & 15, g)];
  }
}

}  // namespace

cudaError_t launch_encode(const EncodeParams& p, cudaStream_t st) {
  if (p.n_jobs <= 0) return cudaSuccess;
  const size_t smem = kBlock * kTileLd * sizeof(float) + kBlock * kD + (256 + 256 + 16) * sizeof(float);
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(encode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int grid = 2 * p.n_jobs < 148 * 16 ? 2 * p.n_jobs : 148 * 16;
  encode_kernel<<<grid, 256, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_stats(const StatsParams& p, cudaStream_t st) {
  if (p.n_blocks <= 0) return cudaSuccess;
  stats_kernel<<<dim3(p.n_blocks, p.n_streams), kD, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_append_rows(uint8_t* arena, const TableEntry* table, int table_stride, int tail_index,
                               int n_streams, int n_kv_heads, const uint16_t* k_in, const uint16_t* v_in,
                               int n_tok, int first_tok, int n_rows, int dst_row0, cudaStream_t st) {
  if (n_rows <= 0) return cudaSuccess;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_streams, n_rows);
  cfg.blockDim = dim3(128);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, append_rows_kernel, arena, table, table_stride, tail_index, n_kv_heads, k_in, v_in, n_tok,
                            first_tok, dst_row0);
}

cudaError_t launch_residual_scores(const uint16_t* v_in, const float* token_mass, const int8_t* levels,
                                   int levels_stride, int n_sink_blocks, int n_streams, int n_kv_heads, int n_tok,
                                   int n_closed, float* scores, cudaStream_t st) {
  if (n_closed <= 0) return cudaSuccess;
  residual_score_kernel<<<dim3(n_closed, n_streams), kD, 0, st>>>(v_in, token_mass, levels, levels_stride,
                                                                  n_sink_blocks, n_kv_heads, n_tok, scores);
  return cudaGetLastError();
}

cudaError_t launch_residual_gather(uint8_t* arena, const uint16_t* k_in, const uint16_t* v_in, int n_tok,
                                   int n_kv_heads, const int32_t* idx, int idx_stride, const int32_t* count,
                                   const uint32_t* res_off256, int max_count, int n_streams, cudaStream_t st) {
  if (max_count <= 0) return cudaSuccess;
  residual_gather_kernel<<<dim3(max_count, n_streams), 128, 0, st>>>(arena, k_in, v_in, n_tok, n_kv_heads, idx,
                                                                     idx_stride, count, res_off256);
  return cudaGetLastError();
}

cudaError_t launch_export_block(const uint8_t* arena, uint32_t off256, int level, int which, uint8_t* codes,
                                uint16_t* scale, uint16_t* zero, uint16_t* rows, cudaStream_t st) {
  export_kernel<<<1, 256, 0, st>>>(arena, off256, level, which, codes, scale, zero, rows);
  return cudaGetLastError();
}

}  // namespace gkv
