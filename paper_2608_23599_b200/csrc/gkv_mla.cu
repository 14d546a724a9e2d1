// Latent-attention (MLA) streams: one 576-wide row per token (512 latent + 64 rope channels),
// 16 query heads on one stream, values = channels [0, 512) of the same row.  The row is stored
// once on the precision ladder with the key rule (groups of 32 tokens x 1 channel, paper
// Sec. 3.2) and read twice by the attention kernel: as K (contraction over the 576 channels) and
// as V (contraction over tokens) - from one staged copy, so every byte crosses HBM once.
// This file holds the write side (encode / requantise, tail append) and the parity export; the
// read side is gkv_mla_tc.cu.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "gkv_internal.h"
#include "gkv_mla.h"

namespace gkv {
namespace {

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

// ---------------------------------------------------------------------------------------------
// encode / requantise one block [64][576] (key rule only), centroid, exact rows
// ---------------------------------------------------------------------------------------------
constexpr int kMTileLd = kMlaDk + 1;

__device__ __forceinline__ int mla_read_code(const uint8_t* slot, int bits, int tok, int ch) {
  int boff, bit;
  mla_code_pos(bits, tok & 31, ch, &boff, &bit);
  const uint8_t* region = slot + (tok >> 5) * mla_half_bytes(bits) + mla_kp_bytes();
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
          const int idx = mla_kp_index(c);
          tile[t * kMTileLd + c] = __fmaf_rn(static_cast<float>(code), hbits(kp[idx]), hbits(kp[idx + kMlaZeroOff]));
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
        const int idx = mla_kp_index(c);
        kp[idx] = sb;
        kp[idx + kMlaZeroOff] = zb;
      }
      if (range) atomicOr(p.status, kStatusRange);
      __syncthreads();
      // pack the chunk words: 64 tokens x 72 chunks x (L / 4) words
      const int wpc = L / 4;
      for (int i = tid; i < kBlock * kMlaChunks * wpc; i += blockDim.x) {
        const int w = i % wpc, j = (i / wpc) % kMlaChunks, tok = i / (wpc * kMlaChunks);
        uint32_t word = 0;
        int boff0 = 0;
        for (int c = (L == 8 ? 4 * w : 0); c < (L == 8 ? 4 * w + 4 : 8); ++c) {
          int boff, bit;
          mla_code_pos(L, tok & 31, 8 * j + c, &boff, &bit);
          boff0 = boff;
          word |= static_cast<uint32_t>(codes[tok * kMlaDk + 8 * j + c]) << bit;
        }
        *reinterpret_cast<uint32_t*>(dst + (tok >> 5) * mla_half_bytes(L) + mla_kp_bytes() + boff0) = word;
      }
    }
  }
}

__global__ void __launch_bounds__(288) mla_append_rows_kernel(uint8_t* arena, const TableEntry* table, int table_stride,
                                                              int tail_index, const uint16_t* k_in, int n_tok,
                                                              int first_tok, int dst_row0) {
  // launched with programmatic stream serialisation: returns once the previous kernel of the stream has
  // completed (the launch itself overlaps that kernel's tail)
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
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
    scale[g] = kp[mla_kp_index(c)];
    zero[g] = kp[mla_kp_index(c) + kMlaZeroOff];
  }
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
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_streams, n_rows);
  cfg.blockDim = dim3(kMlaDk / 2);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, mla_append_rows_kernel, arena, table, table_stride, tail_index, k_in, n_tok, first_tok, dst_row0);
}

cudaError_t launch_mla_export(const uint8_t* arena, uint32_t off256, int level, uint8_t* codes, uint16_t* scale,
                              uint16_t* zero, uint16_t* rows, cudaStream_t st) {
  mla_export_kernel<<<1, 256, 0, st>>>(arena, off256, level, codes, scale, zero, rows);
  return cudaGetLastError();
}

}  // namespace gkv
