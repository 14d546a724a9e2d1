// Compressed-Quest page scorer and top-k selection (paper Sec. 3.5), also used for the exact
// residual's top fraction (Sec. 3.4).
//
// Score of a page for one query head: acc <- fma(q_d, q_d >= 0 ? max_d : min_d, acc) for
// d = 0..127 in order, fp32.  q_d and the box bounds are bf16, so every product is exact in fp32
// and the fma rounds exactly like "exact product, then add": the order of d is the only thing
// that fixes the bits.  Boxes are stored channel-major ([stream][channel][min|max][page]) so a
// warp's loads run along pages and coalesce.
//
// Selection: k largest scores, ties to the lower index, emitted in ascending index order
// (radix select on an order-preserving key, then an ordered compaction).
#include "gkv_internal.h"

namespace gkv {
namespace {

constexpr float kNegInfQ = -__builtin_huge_valf();

__global__ void __launch_bounds__(128) quest_score_kernel(const uint16_t* __restrict__ boxes, int box_stride,
                                                          int n_pages, const uint16_t* __restrict__ q,
                                                          int n_kv_heads, int group, int reduce,
                                                          float* __restrict__ scores, int score_stride) {
  __shared__ float qs[kMaxHeadsPerKv][kD];
  const int stream = blockIdx.y;
  const int b = stream / n_kv_heads, kvh = stream - b * n_kv_heads;
  for (int i = threadIdx.x; i < group * kD; i += blockDim.x) {
    const int h = i / kD, d = i - h * kD;
    const uint16_t bits = q[(static_cast<size_t>(b) * n_kv_heads * group + static_cast<size_t>(kvh) * group + h) * kD + d];
    qs[h][d] = __uint_as_float(static_cast<uint32_t>(bits) << 16);
  }
  __syncthreads();
  const int p0 = (blockIdx.x * blockDim.x + threadIdx.x) * 2;     // two pages per thread (one 32-bit load)
  if (p0 >= n_pages) return;
  float acc[kMaxHeadsPerKv][2];
#pragma unroll
  for (int h = 0; h < kMaxHeadsPerKv; ++h) acc[h][0] = acc[h][1] = 0.f;
  const uint16_t* base = boxes + static_cast<size_t>(stream) * kD * 2 * box_stride + p0;
#pragma unroll 8
  for (int d = 0; d < kD; ++d) {
    const uint32_t lo2 = *reinterpret_cast<const uint32_t*>(base + static_cast<size_t>(2 * d) * box_stride);
    const uint32_t hi2 = *reinterpret_cast<const uint32_t*>(base + static_cast<size_t>(2 * d + 1) * box_stride);
    const float lo_a = __uint_as_float(lo2 << 16), lo_b = __uint_as_float(lo2 & 0xffff0000u);
    const float hi_a = __uint_as_float(hi2 << 16), hi_b = __uint_as_float(hi2 & 0xffff0000u);
#pragma unroll
    for (int h = 0; h < kMaxHeadsPerKv; ++h) {
      if (h < group) {
        const float qv = qs[h][d];
        const bool pos = qv >= 0.f;
        acc[h][0] = __fmaf_rn(qv, pos ? hi_a : lo_a, acc[h][0]);
        acc[h][1] = __fmaf_rn(qv, pos ? hi_b : lo_b, acc[h][1]);
      }
    }
  }
  float s0 = acc[0][0], s1 = acc[0][1];
  for (int h = 1; h < group; ++h) {
    if (reduce == 0) {
      s0 = fmaxf(s0, acc[h][0]);
      s1 = fmaxf(s1, acc[h][1]);
    } else {
      s0 = __fadd_rn(s0, acc[h][0]);
      s1 = __fadd_rn(s1, acc[h][1]);
    }
  }
  float* out = scores + static_cast<size_t>(stream) * score_stride;
  out[p0] = s0;
  if (p0 + 1 < n_pages) out[p0 + 1] = s1;
}

// Order-preserving key: larger score <-> larger key; -0 and +0 map to the same key.
__device__ __forceinline__ uint32_t score_key(float s) {
  const uint32_t f = __float_as_uint(s + 0.0f);
  return (f & 0x80000000u) ? ~f : (f | 0x80000000u);
}

constexpr int kTopkThreads = 1024;

__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const float* __restrict__ scores, int score_stride,
                                                            int n, const int32_t* __restrict__ k_per_stream,
                                                            int k_uniform, int32_t* __restrict__ idx_out,
                                                            int idx_stride) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_remaining;
  __shared__ uint32_t warp_sel[32], warp_eq[32];
  __shared__ uint32_t base_sel, base_eq;
  const int stream = blockIdx.x, tid = threadIdx.x;
  const float* sc = scores + static_cast<size_t>(stream) * score_stride;
  int32_t* out = idx_out + static_cast<size_t>(stream) * idx_stride;
  int k = k_per_stream ? k_per_stream[stream] : k_uniform;
  if (k > n) k = n;
  if (k <= 0) return;
  if (tid == 0) {
    s_prefix = 0;
    s_remaining = static_cast<uint32_t>(k);
  }
  // radix select, most significant byte first: find the key of the k-th largest score
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < 256; i += kTopkThreads) hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t pmask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    for (int i = tid; i < n; i += kTopkThreads) {
      const uint32_t key = score_key(sc[i]);
      if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      uint32_t rem = s_remaining;
      int d = 255;
      for (; d > 0; --d) {
        if (hist[d] >= rem) break;
        rem -= hist[d];
      }
      s_prefix = prefix | (static_cast<uint32_t>(d) << shift);
      s_remaining = rem;
    }
    __syncthreads();
  }
  const uint32_t thr = s_prefix;          // key of the k-th largest
  const uint32_t need_eq = s_remaining;   // how many elements equal to thr are taken (lowest indices)
  if (tid == 0) {
    base_sel = 0;
    base_eq = 0;
  }
  __syncthreads();
  // ordered compaction in index order
  const int lane = tid & 31, wid = tid >> 5;
  for (int i0 = 0; i0 < n; i0 += kTopkThreads) {
    const int i = i0 + tid;
    uint32_t key = 0;
    bool gt = false, eq = false;
    if (i < n) {
      key = score_key(sc[i]);
      gt = key > thr;
      eq = key == thr;
    }
    // rank of this element among the equal ones (exclusive, in index order)
    const uint32_t eq_ballot = __ballot_sync(0xffffffffu, eq);
    const uint32_t eq_before_w = __popc(eq_ballot & ((1u << lane) - 1u));
    if (lane == 0) warp_eq[wid] = __popc(eq_ballot);
    __syncthreads();
    uint32_t eq_before = base_eq + eq_before_w;
    for (int w2 = 0; w2 < wid; ++w2) eq_before += warp_eq[w2];
    const bool take = gt || (eq && eq_before < need_eq);
    const uint32_t sel_ballot = __ballot_sync(0xffffffffu, take);
    const uint32_t sel_before_w = __popc(sel_ballot & ((1u << lane) - 1u));
    if (lane == 0) warp_sel[wid] = __popc(sel_ballot);
    __syncthreads();
    uint32_t pos = base_sel + sel_before_w;
    for (int w2 = 0; w2 < wid; ++w2) pos += warp_sel[w2];
    if (take && pos < static_cast<uint32_t>(k)) out[pos] = i;
    __syncthreads();
    if (tid == 0) {
      uint32_t te = 0, ts = 0;
      for (int w2 = 0; w2 < 32; ++w2) {
        te += warp_eq[w2];
        ts += warp_sel[w2];
      }
      base_eq += te;
      base_sel += ts;
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t launch_quest_scores(const uint16_t* boxes, int box_stride, int n_pages, const uint16_t* q,
                                int n_streams, int n_kv_heads, int group, int reduce, float* scores,
                                int score_stride, cudaStream_t st) {
  if (n_pages <= 0) return cudaSuccess;
  const int threads = 128;
  const int per_cta = threads * 2;
  quest_score_kernel<<<dim3((n_pages + per_cta - 1) / per_cta, n_streams), threads, 0, st>>>(
      boxes, box_stride, n_pages, q, n_kv_heads, group, reduce, scores, score_stride);
  return cudaGetLastError();
}

cudaError_t launch_topk(const float* scores, int score_stride, int n, const int32_t* k_per_stream, int k_uniform,
                        int32_t* idx_out, int idx_stride, int n_streams, cudaStream_t st) {
  if (n <= 0 || n_streams <= 0) return cudaSuccess;
  topk_kernel<<<n_streams, kTopkThreads, 0, st>>>(scores, score_stride, n, k_per_stream, k_uniform, idx_out,
                                                   idx_stride);
  return cudaGetLastError();
}

}  // namespace gkv
