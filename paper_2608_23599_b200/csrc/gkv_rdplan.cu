// RD allocator on the device (Sec. 3.3): the level plan of every stream from its block masses m_b and
// range proxies e_b, the same plan the host allocator makes from the same numbers, bit for bit.
//
// "b bits suffice for block b iff y_b = m_b e_b <= tau (2^b - 1)"; levels snap up to the ladder
// (y <= tau: centroid, <= 3 tau: 2 bits, <= 15 tau: 4, <= 255 tau: 8, else exact); pinned blocks (attention
// sinks, the recent window) stay exact; no level rises above the block's present one (Sec. 3.2) nor, with
// the age constraint, above that of any younger unpinned block.  tau is the smallest of the
// breakpoints {0} u {y_b / k : k in 1, 3, 15, 255} whose plan fits the bit budget.  The bit count never
// increases with tau, so the breakpoints are sorted and bisected; every test is a parallel pass over
// the blocks (thresholds, a suffix minimum for the age constraint, a sum of block sizes).  All
// arithmetic on y and tau is IEEE binary64 (exact products of two fp32, correctly rounded divisions),
// which is what makes the plan independent of who computes it.
//
// One CTA per stream.  Shared memory: the padded breakpoint array (a power of two of doubles), y, and
// the working levels.
#include <cuda_runtime.h>

#include <cstdint>

#include "gkv_internal.h"
#include "gkv_layout.cuh"

namespace gkv {
namespace {

constexpr int kPlanThreads = 256;

__device__ __forceinline__ unsigned long long plan_block_bits(int level, unsigned long long nval_tok) {
  if (level == 16) return 16ull * kBlock * nval_tok;
  if (level == 1) return 16ull * nval_tok;
  return static_cast<unsigned long long>(level) * kBlock * nval_tok + (kBlock * nval_tok / kGroup) * 32ull;
}

// Levels of the plan for threshold tau into lv[] (shared) and the plan's bits (returned to every thread).
// Thread t owns the blocks [t * per, min(n, (t + 1) * per)).
__device__ unsigned long long plan_for_tau(const RdPlanParams& p, const double* y, const TableEntry* table, int n, int per, double tau,
                                           int8_t* lv, int* s_min, unsigned long long* s_bits) {
  const int t = threadIdx.x;
  const int b0 = min(n, t * per), b1 = min(n, b0 + per);
  const int recent = p.retire_after / kBlock;
  const double t3 = tau * 3.0, t15 = tau * 15.0, t255 = tau * 255.0;
  // thresholds, pins and "never above the present level"; the chunk's minimum over unpinned blocks
  int cmin = 127;
  for (int b = b0; b < b1; ++b) {
    const double yb = y[b];
    int L = yb <= tau ? 1 : (yb <= t3 ? 2 : (yb <= t15 ? 4 : (yb <= t255 ? 8 : 16)));
    const bool pinned = b < p.n_sink_blocks || (n - 1 - b) < recent;
    if (pinned) L = 16;
    if (p.use_prev) {
      const int prev = static_cast<int>(table[b].level);
      if (prev < L) L = prev;
    }
    lv[b] = static_cast<int8_t>(L);
    if (!pinned) cmin = min(cmin, L);
  }
  unsigned long long bits = 0;
  if (p.monotone) {
    // level of a block <- minimum over the unpinned blocks at or after it (younger ones have higher
    // indices): the chunks' minima are combined by a suffix scan over the threads
    s_min[t] = cmin;
    __syncthreads();
    int after = 127;                               // minimum over the chunks after this one
    for (int u = t + 1; u < kPlanThreads; ++u) after = min(after, s_min[u]);
    __syncthreads();
    int run = after;
    for (int b = b1 - 1; b >= b0; --b) {
      const bool pinned = b < p.n_sink_blocks || (n - 1 - b) < recent;
      if (!pinned) {
        run = min(run, static_cast<int>(lv[b]));
        lv[b] = static_cast<int8_t>(run);
      }
      bits += plan_block_bits(lv[b], p.nval_tok);
    }
  } else {
    for (int b = b0; b < b1; ++b) bits += plan_block_bits(lv[b], p.nval_tok);
  }
  // sum over the CTA (integers: any order)
  for (int d = 16; d >= 1; d >>= 1) bits += __shfl_xor_sync(0xffffffffu, bits, d);
  if ((t & 31) == 0) s_bits[t >> 5] = bits;
  __syncthreads();
  unsigned long long total = 0;
  for (int w = 0; w < kPlanThreads / 32; ++w) total += s_bits[w];
  __syncthreads();
  return total;
}

__global__ void __launch_bounds__(kPlanThreads) rd_plan_kernel(const RdPlanParams p) {
  extern __shared__ __align__(16) unsigned char plan_sm[];
  __shared__ int s_min[kPlanThreads];
  __shared__ unsigned long long s_bits[kPlanThreads / 32];
  const int s = blockIdx.x, t = threadIdx.x, n = p.n;
  double* cand = reinterpret_cast<double*>(plan_sm);                 // [m_pad]
  double* y = cand + p.m_pad;                                        // [n]
  int8_t* lv = reinterpret_cast<int8_t*>(y + n);                     // [n]
  const float* mass = p.mass + static_cast<size_t>(s) * p.mass_stride;
  const float* range = p.range + static_cast<size_t>(s) * p.range_stride;
  const TableEntry* table = p.table + static_cast<size_t>(s) * p.table_stride;
  const int m = 4 * n + 1;
  for (int b = t; b < n; b += kPlanThreads) {
    const double yb = static_cast<double>(mass[b]) * static_cast<double>(range[b]);
    y[b] = yb;
    cand[4 * b + 1] = yb;
    cand[4 * b + 2] = yb / 3.0;
    cand[4 * b + 3] = yb / 15.0;
    cand[4 * b + 4] = yb / 255.0;
  }
  if (t == 0) cand[0] = 0.0;
  for (int i = m + t; i < p.m_pad; i += kPlanThreads) cand[i] = __longlong_as_double(0x7ff0000000000000ll);   // +inf padding
  __syncthreads();
  // bitonic sort, ascending
  for (int k = 2; k <= p.m_pad; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int i = t; i < p.m_pad; i += kPlanThreads) {
        const int l = i ^ j;
        if (l > i) {
          const double a = cand[i], b = cand[l];
          const bool up = (i & k) == 0;
          if ((a > b) == up) {
            cand[i] = b;
            cand[l] = a;
          }
        }
      }
      __syncthreads();
    }
  }
  // the smallest feasible breakpoint (duplicates do not matter: equal values give equal plans)
  const int per = (n + kPlanThreads - 1) / kPlanThreads;
  const unsigned long long budget = p.budget_bits >= p.tail_bits ? p.budget_bits - p.tail_bits : 0ull;
  const bool any_room = p.budget_bits >= p.tail_bits;
  int lo = 0, hi = m;
  while (lo < hi) {                                                  // uniform for the CTA
    const int mid = (lo + hi) >> 1;
    const unsigned long long bits = plan_for_tau(p, y, table, n, per, cand[mid], lv, s_min, s_bits);
    if (any_room && bits <= budget) hi = mid;
    else lo = mid + 1;
  }
  const bool miss = lo == m;
  if (miss) lo = m - 1;
  plan_for_tau(p, y, table, n, per, cand[lo], lv, s_min, s_bits);
  __syncthreads();
  int8_t* out = p.levels_out + static_cast<size_t>(s) * p.out_stride;
  for (int b = t; b < n; b += kPlanThreads) out[b] = lv[b];
  if (t == 0 && miss) atomicOr(p.miss_flag, 1u);
}

}  // namespace

size_t rd_plan_smem_bytes(int n, int* m_pad_out) {
  int m_pad = 1;
  while (m_pad < 4 * n + 1) m_pad <<= 1;
  if (m_pad_out) *m_pad_out = m_pad;
  return static_cast<size_t>(m_pad) * sizeof(double) + static_cast<size_t>(n) * sizeof(double) + static_cast<size_t>(n) + 16;
}

cudaError_t launch_rd_plan(const RdPlanParams& p, int n_streams, cudaStream_t st) {
  const size_t bytes = rd_plan_smem_bytes(p.n, nullptr);
  static size_t configured = 0;
  if (bytes > 48 * 1024 && bytes > configured) {
    cudaError_t e = cudaFuncSetAttribute(rd_plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
    if (e != cudaSuccess) return e;
    configured = bytes;
  }
  rd_plan_kernel<<<n_streams, kPlanThreads, bytes, st>>>(p);
  return cudaGetLastError();
}

}  // namespace gkv
