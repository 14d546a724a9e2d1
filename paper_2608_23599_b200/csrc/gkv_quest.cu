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

// One CTA scores kQPages consecutive pages of one stream.  The 256 box rows of the stream (channel x
// min|max, kQPages * 2 bytes of each) are streamed through shared memory in chunks of kQRows rows
// with 16-byte cp.async copies, kQStages chunks in flight, so that the loads are wide, contiguous
// and deep while every thread still adds its pages' channels strictly in order.
constexpr int kQThreads = 128, kQPages = kQThreads;          // one page per thread
constexpr int kQRows = 32;                                   // rows per chunk = 16 channels x (min, max)
constexpr int kQStages = 4;
constexpr int kQRowBytes = kQPages * 2;                      // 256
constexpr int kQChunkBytes = kQRows * kQRowBytes;            // 8 KiB
constexpr int kQPieces = kQRowBytes / 16;                    // 16-byte pieces per row
constexpr int kQChunks = 2 * kD / kQRows;                    // 8

__device__ __forceinline__ void q_cp_async16(uint32_t dst, const void* src, bool on) {
  const uint32_t n = on ? 16u : 0u;                          // 0 source bytes: the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(n) : "memory");
}

// GROUP = query heads per KV head, a compile-time bound: a run-time bound would leave the unused
// heads' instructions in the loop, predicated off but still issued.
template <int GROUP>
__global__ void __launch_bounds__(kQThreads) quest_score_kernel(const uint16_t* __restrict__ boxes, int box_stride,
                                                                int n_pages, const uint16_t* __restrict__ q,
                                                                int n_kv_heads, int reduce,
                                                                float* __restrict__ scores, int score_stride) {
  constexpr int group = GROUP;
  // launched with programmatic stream serialisation: returns once the previous kernel of the stream
  // has completed (the launch itself overlaps that kernel's tail)
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  extern __shared__ __align__(16) uint8_t qsm[];
  float (*qs)[kD] = reinterpret_cast<float (*)[kD]>(qsm + kQStages * kQChunkBytes);       // [8][128]
  const int stream = blockIdx.y, tid = threadIdx.x;
  const int b = stream / n_kv_heads, kvh = stream - b * n_kv_heads;
  const int page0 = blockIdx.x * kQPages;
  const uint16_t* rows = boxes + static_cast<size_t>(stream) * kD * 2 * box_stride + page0;
  const uint32_t stage0 = static_cast<uint32_t>(__cvta_generic_to_shared(qsm));
  // chunk c -> stage c % kQStages: row r of the chunk is box row c * kQRows + r; a row is 32 pieces
  // of 16 bytes (8 pages); pieces that start beyond the row's end (box_stride) are zero-filled
  auto issue = [&](int c) {
    const uint32_t dst = stage0 + (c % kQStages) * kQChunkBytes;
#pragma unroll
    for (int i = 0; i < kQRows * kQPieces / kQThreads; ++i) {
      const int piece = tid + i * kQThreads, r = piece / kQPieces, col = piece % kQPieces;
      const bool on = page0 + 8 * col < box_stride;
      q_cp_async16(dst + r * kQRowBytes + col * 16, rows + static_cast<size_t>(c * kQRows + r) * box_stride + (on ? 8 * col : 0), on);
    }
    asm volatile("cp.async.commit_group;\n" ::: "memory");
  };
#pragma unroll
  for (int c = 0; c < kQStages - 1; ++c) issue(c);
  for (int i = tid; i < group * kD; i += kQThreads) {
    const int h = i / kD, d = i - h * kD;
    const uint16_t bits = q[(static_cast<size_t>(b) * n_kv_heads * group + static_cast<size_t>(kvh) * group + h) * kD + d];
    qs[h][d] = __uint_as_float(static_cast<uint32_t>(bits) << 16);
  }
  float acc[GROUP];
#pragma unroll
  for (int h = 0; h < GROUP; ++h) acc[h] = 0.f;
#pragma unroll 1
  for (int c = 0; c < kQChunks; ++c) {
    if (c + kQStages - 1 < kQChunks) issue(c + kQStages - 1);
    else asm volatile("cp.async.commit_group;\n" ::: "memory");          // keeps the group count uniform
    asm volatile("cp.async.wait_group %0;\n" ::"n"(kQStages - 1) : "memory");
    __syncthreads();                                   // chunk c (and, the first time, the query) is visible to all
    const uint8_t* st = qsm + (c % kQStages) * kQChunkBytes + tid * 2;
#pragma unroll
    for (int i = 0; i < kQRows / 2; ++i) {
      const float lo = __uint_as_float(static_cast<uint32_t>(*reinterpret_cast<const uint16_t*>(st + (2 * i) * kQRowBytes)) << 16);
      const float hi = __uint_as_float(static_cast<uint32_t>(*reinterpret_cast<const uint16_t*>(st + (2 * i + 1) * kQRowBytes)) << 16);
      const int d = c * (kQRows / 2) + i;
#pragma unroll
      for (int h = 0; h < GROUP; ++h) {
        const float qv = qs[h][d];
        acc[h] = __fmaf_rn(qv, qv >= 0.f ? hi : lo, acc[h]);
      }
    }
    __syncthreads();                                   // the stage may be refilled
  }
  const int p0 = page0 + tid;
  if (p0 >= n_pages) return;
  float s0 = acc[0];
#pragma unroll
  for (int h = 1; h < GROUP; ++h) s0 = (reduce == 0) ? fmaxf(s0, acc[h]) : __fadd_rn(s0, acc[h]);
  scores[static_cast<size_t>(stream) * score_stride + p0] = s0;
}

// Order-preserving key: larger score <-> larger key; -0 and +0 map to the same key.
__device__ __forceinline__ uint32_t score_key(float s) {
  const uint32_t f = __float_as_uint(s + 0.0f);
  return (f & 0x80000000u) ? ~f : (f | 0x80000000u);
}

constexpr int kTopkThreads = 1024;

// KEEP: n <= 4 * kTopkThreads, every thread keeps the keys of its (up to four) elements in registers
// instead of reading the scores again in every pass.
template <bool KEEP>
__global__ void __launch_bounds__(kTopkThreads) topk_kernel(const float* __restrict__ scores, int score_stride,
                                                            int n, const int32_t* __restrict__ k_per_stream,
                                                            int k_uniform, int32_t* __restrict__ idx_out,
                                                            int idx_stride) {
  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_prefix, s_remaining;
  __shared__ uint32_t warp_sel[32], warp_eq[32];
  __shared__ uint32_t base_sel, base_eq;
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
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
  uint32_t kreg[4] = {0u, 0u, 0u, 0u};
  if (KEEP) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = tid + j * kTopkThreads;
      if (i < n) kreg[j] = score_key(sc[i]);
    }
  }
  // radix select, most significant byte first: find the key of the k-th largest score
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < 256; i += kTopkThreads) hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const uint32_t pmask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    if (KEEP) {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (tid + j * kTopkThreads < n && (kreg[j] & pmask) == prefix) atomicAdd(&hist[(kreg[j] >> shift) & 255u], 1u);
    } else {
      for (int i = tid; i < n; i += kTopkThreads) {
        const uint32_t key = score_key(sc[i]);
        if ((key & pmask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
      }
    }
    __syncthreads();
    // The digit of the k-th largest is the t with c[t] >= rem > c[t + 1], c[t] = sum_{j >= t} hist[j].
    // Warp 0: lane l owns bins 255 - 8 l .. 248 - 8 l (from the top), a shuffle scan joins the lanes.
    if (tid < 32) {
      const uint32_t rem = s_remaining;
      uint32_t own[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        own[j] = hist[255 - 8 * tid - j];
        tot += own[j];
      }
      uint32_t incl = tot;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
        if (tid >= d) incl += up;
      }
      uint32_t above = incl - tot;                  // count in bins above this lane's eight
      if (above < rem && incl >= rem) {             // exactly one lane
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (above < rem && above + own[j] >= rem) {
            s_prefix = prefix | (static_cast<uint32_t>(255 - 8 * tid - j) << shift);
            s_remaining = rem - above;
            above = rem;                            // done: no later bin matches
          } else {
            above += own[j];
          }
        }
      }
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
#pragma unroll 1
  for (int i0 = 0, j = 0; i0 < n; i0 += kTopkThreads, ++j) {
    const int i = i0 + tid;
    uint32_t key = 0;
    bool gt = false, eq = false;
    if (i < n) {
      if (KEEP) key = j == 0 ? kreg[0] : (j == 1 ? kreg[1] : (j == 2 ? kreg[2] : kreg[3]));
      else key = score_key(sc[i]);
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
  const size_t smem = kQStages * kQChunkBytes + kMaxHeadsPerKv * kD * sizeof(float);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((n_pages + kQPages - 1) / kQPages, n_streams);
  cfg.blockDim = dim3(kQThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaSuccess;
#define GKV_QUEST_CASE(G)                                                                                                \
  case G: {                                                                                                              \
    static bool configured = false;                                                                                      \
    if (!configured) {                                                                                                   \
      e = cudaFuncSetAttribute(quest_score_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)); \
      if (e != cudaSuccess) return e;                                                                                    \
      configured = true;                                                                                                 \
    }                                                                                                                    \
    e = cudaLaunchKernelEx(&cfg, quest_score_kernel<G>, boxes, box_stride, n_pages, q, n_kv_heads, reduce, scores,       \
                           score_stride);                                                                                \
    break;                                                                                                               \
  }
  switch (group) {
    GKV_QUEST_CASE(1)
    GKV_QUEST_CASE(2)
    GKV_QUEST_CASE(3)
    GKV_QUEST_CASE(4)
    GKV_QUEST_CASE(5)
    GKV_QUEST_CASE(6)
    GKV_QUEST_CASE(7)
    GKV_QUEST_CASE(8)
    default: return cudaErrorInvalidValue;
  }
#undef GKV_QUEST_CASE
  return e;
}

cudaError_t launch_topk(const float* scores, int score_stride, int n, const int32_t* k_per_stream, int k_uniform,
                        int32_t* idx_out, int idx_stride, int n_streams, cudaStream_t st) {
  if (n <= 0 || n_streams <= 0) return cudaSuccess;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_streams);
  cfg.blockDim = dim3(kTopkThreads);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (n <= 4 * kTopkThreads)
    return cudaLaunchKernelEx(&cfg, topk_kernel<true>, scores, score_stride, n, k_per_stream, k_uniform, idx_out, idx_stride);
  return cudaLaunchKernelEx(&cfg, topk_kernel<false>, scores, score_stride, n, k_per_stream, k_uniform, idx_out, idx_stride);
}

}  // namespace gkv
