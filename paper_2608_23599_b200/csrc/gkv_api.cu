// Host side of the graded KV-cache library: arena layout, slot allocator, ladder policies and the
// extern "C" entry points declared in include/gkv.h.  All tensor work is done by the kernels in
// gkv_decode.cu / gkv_pack.cu / gkv_quest.cu; this file only decides *which* block sits on which
// rung (paper Sec. 3.2-3.3), where it lives in the arena, and which warp reads what.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <mutex>
#include <numeric>
#include <thread>
#include <vector>

#include "../../include/gkv.h"
#include "gkv_internal.h"
#include "gkv_mla.h"

using namespace gkv;

namespace {

constexpr int kTargetWarps = 148 * kDecodeCtasPerSm * kDecodeWarps;   // one resident wave of CTAs
// Page-list reads: a stream's pages are split over whole CTAs, as many as fill the GPU once (at most 8)
int sparse_ctas_per_stream(int n_streams) { return std::max(1, std::min(8, 148 / std::max(n_streams, 1))); }
constexpr size_t kMinWarpCost = 1000;     // do not split below about one block per warp

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int level_index(int level) { return level == 16 ? 0 : level == 8 ? 1 : level == 4 ? 2 : level == 2 ? 3 : 4; }
constexpr int kLevels[5] = {16, 8, 4, 2, 1};
// Logical bits of one closed block (codes + fp16 scale/zero per group of 32, or one centroid row
// per tensor, or exact rows); nval_tok = values per token (d_k + d_v, or d_k when V aliases K).
inline uint64_t block_bits(int level, uint64_t nval_tok) {
  if (level == 16) return 16ull * kBlock * nval_tok;
  if (level == 1) return 16ull * nval_tok;
  return static_cast<uint64_t>(level) * kBlock * nval_tok + (kBlock * nval_tok / kGroup) * 32ull;
}

// Segregated free lists over one heap of 256-byte units.  Slots are freed and reallocated by
// size class; when the bump region is exhausted a larger free slot is split.
struct SlotHeap {
  uint32_t begin = 0, end = 0, bump = 0;
  uint32_t units[5] = {0, 0, 0, 0, 0};          // slot size per level (16, 8, 4, 2, 1) in 256-byte units
  std::vector<uint32_t> free_list[5];
  uint32_t slot_units(int level) const { return units[level_index(level)]; }
  bool alloc(int level, uint32_t* off) {
    const int ci = level_index(level);
    if (!free_list[ci].empty()) {
      *off = free_list[ci].back();
      free_list[ci].pop_back();
      return true;
    }
    const uint32_t need = slot_units(level);
    if (bump + need <= end) {
      *off = bump;
      bump += need;
      return true;
    }
    for (int cj = ci - 1; cj >= 0; --cj) {      // split a larger free slot
      if (free_list[cj].empty()) continue;
      const uint32_t base = free_list[cj].back();
      free_list[cj].pop_back();
      uint32_t rest_off = base + need, rest = slot_units(kLevels[cj]) - need;
      *off = base;
      for (int ck = 0; ck < 5 && rest > 0; ++ck) {
        const uint32_t u = slot_units(kLevels[ck]);
        while (rest >= u) {
          free_list[ck].push_back(rest_off);
          rest_off += u;
          rest -= u;
        }
      }
      return true;
    }
    return false;
  }
  void release(int level, uint32_t off) { free_list[level_index(level)].push_back(off); }
};

struct LayerState {
  int n_closed = 0, n_tail = 0;
  bool has_tail_slot = false;
  std::vector<int8_t> level;            // [n_streams][max_blocks]
  TableEntry* table_h = nullptr;        // pinned [n_streams][table_stride]
  WarpDesc* warps_h = nullptr;          // pinned [max_warps]
  uint32_t* units_h = nullptr;          // pinned [n_streams][unit_stride]
  int n_units = 0;
  StreamParts* parts_h = nullptr;       // pinned [n_streams * head_groups]
  uint32_t* res_off_h = nullptr;        // pinned [n_streams]
  int32_t* res_count_h = nullptr;       // pinned [n_streams]
  std::vector<std::vector<int32_t>> res_idx;
  bool desc_dirty = true;
  bool desc_split = false;              // the work lists hold sub-block units (never for observing calls)
  bool desc_allow_split = false;        // what the lists were built with
  int n_warps = 0;
  cudaEvent_t ev = nullptr;             // last upload from this layer's pinned table / residual mirrors
  cudaEvent_t ev_desc = nullptr;        // last upload from its pinned work lists (warps, units, parts)
  // device regions
  TableEntry* table_d = nullptr;
  WarpDesc* warps_d = nullptr;
  uint32_t* units_d = nullptr;
  StreamParts* parts_d = nullptr;
  uint32_t* res_off_d = nullptr;
  int32_t* res_count_d = nullptr;
  int32_t* res_idx_d = nullptr;         // [n_streams][res_cap]
  float* ema_d = nullptr;               // running block mass m_b [n_streams][max_blocks + 1] (Sec. 3.1)
  float* range_d = nullptr;             // RD policy: range proxy e_b of every closed block [n_streams][max_blocks]
  float4* err_d = nullptr;              // error bounds of every closed block for the certificate [n_streams][max_blocks]
  uint16_t* boxes_d = nullptr;
  // accounting of the last read
  int last_mode = 0;                    // 0 none, 1 full, 2 page list
  const int32_t* last_pages = nullptr;
  int last_n_sel = 0;
  bool quest_ran = false;               // gkv_quest_select ran and no read has consumed its result yet
  bool last_read_scored = false;        // the last page-list read followed a gkv_quest_select (its boxes count as read)
  bool budget_flag = false;
};

}  // namespace

struct gkv_cache {
  gkv_config cfg;
  uint8_t* arena = nullptr;
  size_t arena_bytes = 0;
  int n_streams = 0, group = 0, head_groups = 1, n_hgroups = 0, max_blocks = 0, table_stride = 0, max_warps = 0, res_cap = 0, box_stride = 0;
  float scale = 0.f;
  SlotHeap heap;
  std::vector<LayerState> layers;
  int device = -1;                      // the device that owns the arena
  int desc_src = -1;                    // layer whose work lists were last built from scratch
  // shared device scratch
  uint32_t* status_d = nullptr;
  uint8_t* debug_d = nullptr;
  float* partial_d = nullptr;
  float* range_d = nullptr;
  float* mass_d = nullptr;
  int8_t* levels_d = nullptr;
  float* scores_d = nullptr;            // residual scores [n_streams][max_ctx] or page scores
  int32_t* kper_d = nullptr;
  int32_t* tickets_d = nullptr;         // per-head-group arrival counters of the decode kernel's final merge
  float2* mass_raw_d = nullptr;         // scratch of an observing decode call: [n_streams][max_blocks + 1][8]
  float2* res_raw_d = nullptr;          // [n_streams][res_cap][8]
  float* lse2_d = nullptr;              // [n_streams][8]
  EncodeJob* jobs_d = nullptr;
  size_t jobs_cap = 0;
  // Small job lists of decode-time demotions go through a ring of pinned slots with an event each,
  // so that consecutive layers' block closes do not wait for one another's copies.
  static constexpr int kDemoteSlots = 8;
  EncodeJob* demote_h = nullptr;        // pinned [kDemoteSlots][demote_cap]
  size_t demote_cap = 0;
  int demote_next = 0;
  cudaEvent_t ev_demote[kDemoteSlots] = {};
  // shared pinned staging (jobs | levels | k-per-stream), guarded by ev_stage
  uint8_t* stage_h = nullptr;
  size_t stage_bytes = 0;
  cudaEvent_t ev_stage = nullptr;
  int last_cuda = 0;
};

namespace {

inline bool is_mla(const gkv_config& c) { return c.v_aliases_k != 0; }
inline int geo_slot_bytes(const gkv_config& c, int level) { return is_mla(c) ? mla_slot_bytes(level) : slot_bytes(level); }
inline uint64_t nval_per_token(const gkv_config& c) { return is_mla(c) ? c.d_k : c.d_k + c.d_v; }
constexpr int kMlaTargetCtas = 148;          // one CTA per SM (212 KB of shared memory, all of tensor memory)

struct ArenaPlan {
  size_t status, debug, partial, range, mass, levels, scores, kper, tickets, jobs, mass_raw, res_raw, lse2, per_layer, heap_begin, total_meta;
  size_t l_table, l_warps, l_units, l_parts, l_resoff, l_rescount, l_residx, l_respool, l_boxes, l_ema, l_range, l_err, layer_bytes;
};

struct Derived {
  int n_streams, group, head_groups, n_hgroups, max_blocks, table_stride, max_warps, res_cap, box_stride, unit_stride;
};

int validate_config(const gkv_config* c) {
  if (!c) return GKV_ERR_INVALID_ARG;
  if (c->struct_size != sizeof(gkv_config) || c->abi_version != GKV_ABI_VERSION) return GKV_ERR_INVALID_ARG;
  if (c->n_layers <= 0 || c->batch <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0) return GKV_ERR_INVALID_ARG;
  if (c->n_q_heads % c->n_kv_heads != 0) return GKV_ERR_INVALID_ARG;
  if (c->max_ctx <= 0) return GKV_ERR_INVALID_ARG;
  if (c->block_tokens != kBlock || c->group != kGroup) return GKV_ERR_UNSUPPORTED;
  if (c->v_aliases_k) {
    // latent attention: one 576-wide stream per sequence, 16 heads, values = channels [0, 512)
    if (c->d_k != kMlaDk || c->d_v != kMlaDv || c->n_kv_heads != 1 || c->n_q_heads != kMlaHeads) return GKV_ERR_UNSUPPORTED;
    if (c->page_tokens != 0 || c->residual_fraction != 0.f || c->policy == GKV_POLICY_RD) return GKV_ERR_UNSUPPORTED;
    if (c->policy == GKV_POLICY_STAIRCASE && c->stair_tokens[3] != 0) return GKV_ERR_UNSUPPORTED;   // no 2-bit rung
  } else {
    if (c->d_k != kD || c->d_v != kD) return GKV_ERR_UNSUPPORTED;
    if (c->n_q_heads / c->n_kv_heads > kMaxHeadsPerKv) return GKV_ERR_UNSUPPORTED;
  }
  if (c->page_tokens != 0 && c->page_tokens != 16 && c->page_tokens != 32 && c->page_tokens != 64)
    return GKV_ERR_INVALID_ARG;
  if (c->policy < GKV_POLICY_STAIRCASE || c->policy > GKV_POLICY_EXTERNAL) return GKV_ERR_INVALID_ARG;
  if (c->residual_fraction < 0.f || c->residual_fraction > 1.f) return GKV_ERR_INVALID_ARG;
  if (c->n_sink_blocks < 0 || c->retire_after < 0) return GKV_ERR_INVALID_ARG;
  if (c->quest_reduce != GKV_REDUCE_MAX && c->quest_reduce != GKV_REDUCE_SUM) return GKV_ERR_INVALID_ARG;
  if (c->policy == GKV_POLICY_STAIRCASE)
    for (int i = 0; i < 4; ++i)
      if (c->stair_tokens[i] < -1 || (c->stair_tokens[i] > 0 && c->stair_tokens[i] % kBlock)) return GKV_ERR_INVALID_ARG;
  return GKV_OK;
}

Derived derive(const gkv_config& c) {
  Derived d;
  d.n_streams = c.batch * c.n_kv_heads;
  d.group = c.n_q_heads / c.n_kv_heads;
  // a warp of the decode kernel serves up to four query heads: a larger group is read as two head groups
  d.head_groups = is_mla(c) ? 1 : (d.group + kHeadsPerWarp - 1) / kHeadsPerWarp;
  d.n_hgroups = d.n_streams * d.head_groups;
  d.max_blocks = (c.max_ctx + kBlock - 1) / kBlock;
  d.table_stride = d.max_blocks + 2;
  d.max_warps = static_cast<int>(align_up(kTargetWarps + 2 * d.n_hgroups, kDecodeWarps));
  d.max_warps = std::max(d.max_warps, d.n_hgroups * sparse_ctas_per_stream(d.n_hgroups) * kDecodeWarps);
  d.res_cap = c.residual_fraction > 0.f
                  ? static_cast<int>(align_up(static_cast<size_t>(std::floor(static_cast<double>(c.residual_fraction) * c.max_ctx)) + 16, 16))
                  : 0;
  d.unit_stride = d.max_blocks + 1 + d.res_cap / 16 + 3 * (kTargetWarps / 2);      // small workloads list sub-block units
  d.box_stride = c.page_tokens > 0 ? static_cast<int>(align_up((c.max_ctx + c.page_tokens - 1) / c.page_tokens, 8)) : 0;
  return d;
}

ArenaPlan plan_arena(const gkv_config& c, const Derived& d) {
  ArenaPlan a;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  a.status = take(256);
  a.debug = take(kBlock * kMlaDk + 2 * 4096 + kBlock * kMlaDk * 2);
  a.partial = take(is_mla(c) ? static_cast<size_t>(kMlaTargetCtas + 2 * d.n_streams) * kMlaPartialFloats * sizeof(float)
                             : static_cast<size_t>(d.max_warps) * kPartialFloats * sizeof(float));
  a.range = take(static_cast<size_t>(d.n_streams) * d.max_blocks * sizeof(float));
  a.mass = take(static_cast<size_t>(d.n_streams) * d.max_blocks * sizeof(float));
  a.levels = take(static_cast<size_t>(d.n_streams) * d.max_blocks);
  const size_t score_elems = std::max<size_t>(c.residual_fraction > 0.f ? c.max_ctx : 0, d.box_stride);
  a.scores = take(static_cast<size_t>(d.n_streams) * score_elems * sizeof(float));
  a.kper = take(static_cast<size_t>(d.n_streams) * sizeof(int32_t));
  a.tickets = take(static_cast<size_t>(d.n_hgroups) * sizeof(int32_t));
  a.jobs = take(static_cast<size_t>(d.n_streams) * d.max_blocks * sizeof(EncodeJob));
  // block-mass observation (grouped-query layout only)
  const size_t mass_items = is_mla(c) ? 0 : static_cast<size_t>(d.n_streams) * (d.max_blocks + 1);
  a.mass_raw = take(mass_items * kMaxHeadsPerKv * sizeof(float2));
  a.res_raw = take(is_mla(c) ? 0 : static_cast<size_t>(d.n_streams) * d.res_cap * kMaxHeadsPerKv * sizeof(float2));
  a.lse2 = take(static_cast<size_t>(d.n_streams) * kMaxHeadsPerKv * sizeof(float));
  a.per_layer = off;
  size_t lo = 0;
  auto ltake = [&](size_t bytes) { size_t o = lo; lo = align_up(lo + bytes, 256); return o; };
  a.l_table = ltake(static_cast<size_t>(d.n_streams) * d.table_stride * sizeof(TableEntry));
  a.l_warps = ltake(static_cast<size_t>(d.max_warps) * sizeof(WarpDesc));
  a.l_units = ltake(static_cast<size_t>(d.n_streams) * d.unit_stride * sizeof(uint32_t));
  a.l_parts = ltake(static_cast<size_t>(d.n_hgroups) * sizeof(StreamParts));
  a.l_resoff = ltake(static_cast<size_t>(d.n_streams) * sizeof(uint32_t));
  a.l_rescount = ltake(static_cast<size_t>(d.n_streams) * sizeof(int32_t));
  a.l_residx = ltake(static_cast<size_t>(d.n_streams) * std::max(d.res_cap, 1) * sizeof(int32_t));
  a.l_respool = ltake(static_cast<size_t>(d.n_streams) * d.res_cap * 2 * kRowBytes);
  a.l_boxes = ltake(static_cast<size_t>(d.n_streams) * kD * 2 * d.box_stride * sizeof(uint16_t));
  a.l_ema = ltake(mass_items * sizeof(float));
  a.l_range = ltake(c.policy == GKV_POLICY_RD ? static_cast<size_t>(d.n_streams) * d.max_blocks * sizeof(float) : 0);
  a.l_err = ltake(is_mla(c) ? 0 : static_cast<size_t>(d.n_streams) * d.max_blocks * sizeof(float4));
  a.layer_bytes = lo;
  a.heap_begin = align_up(a.per_layer + static_cast<size_t>(c.n_layers) * a.layer_bytes, 256);
  a.total_meta = a.heap_begin;
  return a;
}

// Level per closed block (0 = oldest) from rung widths, newest first (Sec. 3.2: blocks leave the
// recent window and walk down the ladder; sinks stay exact, Fig. 1).
void staircase_levels(const gkv_config& c, int n_closed, int8_t* lv) {
  long long edge[4];
  long long acc = 0;
  bool unbounded = false;
  for (int i = 0; i < 4; ++i) {
    if (c.stair_tokens[i] < 0) unbounded = true;
    if (!unbounded) acc += c.stair_tokens[i] / kBlock;
    edge[i] = unbounded ? -1 : acc;
  }
  static const int8_t rung[4] = {16, 8, 4, 2};
  for (int i = 0; i < n_closed; ++i) {
    const long long age = n_closed - 1 - i;
    int8_t L = 1;
    for (int k = 0; k < 4; ++k) {
      if (edge[k] < 0 || age < edge[k]) {
        L = rung[k];
        break;
      }
    }
    if (i < c.n_sink_blocks) L = 16;
    lv[i] = L;
  }
}

// Worst-case slot bytes of one stream under the configured policy at max_ctx.
size_t worst_stream_bytes(const gkv_config& c, const Derived& d) {
  size_t bytes = 0;
  if (c.policy == GKV_POLICY_STAIRCASE) {
    // the population of each rung is bounded by its width (or by max_blocks when unbounded)
    std::vector<int8_t> lv(d.max_blocks);
    staircase_levels(c, d.max_blocks, lv.data());
    for (int i = 0; i < d.max_blocks; ++i) bytes += geo_slot_bytes(c, lv[i]);
    for (int L : kLevels) bytes += 2 * geo_slot_bytes(c, L);     // allocate-before-free slack + tail
  } else {
    bytes = static_cast<size_t>(d.max_blocks + 2) * geo_slot_bytes(c, 16);
  }
  return bytes;
}

int cuda_fail(gkv_cache* c, cudaError_t e) {
  if (c) c->last_cuda = static_cast<int>(e);
  return GKV_ERR_CUDA;
}
#define CK(c, expr)                                   \
  do {                                                \
    cudaError_t e__ = (expr);                         \
    if (e__ != cudaSuccess) return cuda_fail(c, e__); \
  } while (0)

// Upload from a pinned mirror; the caller must have waited for `ev` before modifying the mirror.
int upload(gkv_cache* c, void* dst, const void* src, size_t bytes, cudaStream_t st, cudaEvent_t ev) {
  if (bytes == 0) return GKV_OK;
  CK(c, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, st));
  CK(c, cudaEventRecord(ev, st));
  return GKV_OK;
}

// Copy the table entries of block `block` of every stream (one column of the [stream][block] table).
int upload_table_column(gkv_cache* c, LayerState& L, int block, cudaStream_t st) {
  const size_t pitch = static_cast<size_t>(c->table_stride) * sizeof(TableEntry);
  CK(c, cudaMemcpy2DAsync(L.table_d + block, pitch, L.table_h + block, pitch, sizeof(TableEntry), c->n_streams,
                          cudaMemcpyHostToDevice, st));
  CK(c, cudaEventRecord(L.ev, st));
  return GKV_OK;
}

// ---- RD allocator (Sec. 3.3) -------------------------------------------------------------------
// The paper's bit depth b* = ceil(log2(c|q| e_b / (2 eps_t) + 1)) with eps_t = tau / (N_b m_b)
// means "b bits suffice iff y_b = m_b e_b <= tau (2^b - 1)" once constants are folded into tau.
// Levels snap up to the ladder (b* <= 1 -> centroid); tau is the smallest breakpoint whose plan,
// after the projections (pinned exact, never above the previous level, never rising toward older
// blocks), fits the bit budget.
void rd_levels_for_tau(const std::vector<double>& y, double tau, const std::vector<char>& pinned,
                       const int8_t* prev, bool mono, std::vector<int8_t>& lv) {
  const int n = static_cast<int>(y.size());
  for (int b = 0; b < n; ++b) {
    int8_t L;
    if (y[b] <= tau) L = 1;
    else if (y[b] <= tau * 3.0) L = 2;
    else if (y[b] <= tau * 15.0) L = 4;
    else if (y[b] <= tau * 255.0) L = 8;
    else L = 16;
    if (pinned[b]) L = 16;
    if (prev && prev[b] < L) L = prev[b];
    lv[b] = L;
  }
  if (mono) {
    int nxt = -1;
    for (int b = n - 1; b >= 0; --b) {
      if (pinned[b]) continue;
      if (nxt >= 0 && nxt < lv[b]) lv[b] = static_cast<int8_t>(nxt);
      nxt = lv[b];
    }
  }
}

// prev: nullable current levels; with them no block's level rises (Sec. 3.2: demotion only).
bool rd_allocate(const gkv_config& c, const float* mass, const float* range, int n, int n_tail, const int8_t* prev, int8_t* out) {
  std::vector<double> y(n);
  std::vector<char> pinned(n, 0);
  const int recent = c.retire_after / kBlock;
  for (int b = 0; b < n; ++b) {
    y[b] = static_cast<double>(mass[b]) * static_cast<double>(range[b]);
    if (b < c.n_sink_blocks || (n - 1 - b) < recent) pinned[b] = 1;
  }
  const long long nval_tok = c.d_k + c.d_v;
  const long long T = static_cast<long long>(n) * kBlock + n_tail;
  const long long budget_bits = static_cast<long long>(std::floor(static_cast<double>(c.rd_budget_bpv) * static_cast<double>(T * nval_tok)));
  const long long tail_bits = static_cast<long long>(n_tail) * 16 * nval_tok;
  std::vector<double> cands;
  cands.reserve(4 * n + 1);
  cands.push_back(0.0);
  static const double ks[4] = {1.0, 3.0, 15.0, 255.0};
  for (int b = 0; b < n; ++b)
    for (double k : ks) cands.push_back(y[b] / k);
  std::sort(cands.begin(), cands.end());
  cands.erase(std::unique(cands.begin(), cands.end()), cands.end());
  std::vector<int8_t> lv(n);
  auto feasible = [&](double tau) {
    rd_levels_for_tau(y, tau, pinned, prev, c.monotone_in_age != 0, lv);
    long long bits = tail_bits;
    for (int b = 0; b < n; ++b) bits += static_cast<long long>(block_bits(lv[b], nval_tok));
    return bits <= budget_bits;
  };
  // bits(tau) never increases with tau, so the smallest feasible candidate is found by bisection
  size_t lo = 0, hi = cands.size();
  while (lo < hi) {
    const size_t mid = (lo + hi) / 2;
    if (feasible(cands[mid])) hi = mid;
    else lo = mid + 1;
  }
  bool budget_miss = false;
  if (lo == cands.size()) {
    budget_miss = true;
    lo = cands.size() - 1;
  }
  rd_levels_for_tau(y, cands[lo], pinned, prev, c.monotone_in_age != 0, lv);
  std::memcpy(out, lv.data(), n);
  return budget_miss;
}

// The streams' allocations are independent: a handful of host threads share them (each stream's
// plan depends only on its own masses and ranges, so the result does not depend on the thread count).
// Returns true when some stream missed its budget.
bool rd_allocate_streams(const gkv_config& c, const float* mass, const float* range, int n, int n_tail, int ns,
                         const int8_t* prev, size_t prev_stride, int8_t* out, size_t out_stride) {
  std::vector<char> miss(ns, 0);
  auto run = [&](int s) {
    miss[s] = rd_allocate(c, mass + static_cast<size_t>(s) * n, range + static_cast<size_t>(s) * n, n, n_tail,
                          prev ? prev + static_cast<size_t>(s) * prev_stride : nullptr, out + static_cast<size_t>(s) * out_stride);
  };
  const unsigned hw = std::thread::hardware_concurrency();
  const int n_thr = std::min({ns / 2, 8, static_cast<int>(hw ? hw : 1u)});
  if (n_thr < 2 || static_cast<size_t>(ns) * n < 2048) {
    for (int s = 0; s < ns; ++s) run(s);
  } else {
    std::vector<std::thread> pool;
    pool.reserve(n_thr - 1);
    for (int t = 1; t < n_thr; ++t)
      pool.emplace_back([&, t] {
        for (int s = t; s < ns; s += n_thr) run(s);
      });
    for (int s = 0; s < ns; s += n_thr) run(s);
    for (std::thread& th : pool) th.join();
  }
  return std::find(miss.begin(), miss.end(), 1) != miss.end();
}

// ---- decode work split ---------------------------------------------------------------------------
// Cost of one item for the work split: cycles a warp needs for it while the whole GPU runs the
// mixed workload, measured on B200 by timing every step of individual warps of the config-2 launch
// (in units where a 4-bit block is 1000): an exact block 1590, 8-bit 1070, 4-bit 1000, 2-bit 1015, a
// centroid block 47 (a run of 16 costs 745).  Bytes are the wrong weight: below 8 bits the kernel
// is bound by instruction issue and a block costs the same whatever its code width.
size_t item_cost(const gkv_cache* c, const LayerState& L, int stream, int item) {
  if (item < L.n_closed) {
    switch (L.level[static_cast<size_t>(stream) * c->max_blocks + item]) {
      case 16: return 1590;
      case 8: return 1070;
      case 4: return 1000;
      case 2: return 1015;
      default: return 47;
    }
  }
  if (item == L.n_closed) return 800;      // tail: mid-fill estimate (its size changes every step)
  return 550;                              // residual group of 16 exact rows
}

// Units of a stream (a block, a run of up to 16 neighbouring centroid blocks, the tail, a residual
// group) are dealt to the stream's warps longest-first onto the least loaded warp, so that every
// warp ends up with the same cost whatever the order of levels along the context; each warp then
// walks its units in a mixed order (see below).
void build_descs(gkv_cache* c, LayerState& L, bool allow_split) {
  const int ns = c->n_streams;
  // The lists depend only on the streams' levels and residual counts.  Layers usually close a block
  // in the same step and, under the staircase, with the same plan: a layer whose levels equal those
  // of the layer built last takes a copy of that layer's lists instead of building its own.
  const int self = static_cast<int>(&L - c->layers.data());
  if (c->desc_src >= 0 && c->desc_src != self) {
    const LayerState& S = c->layers[c->desc_src];
    bool same = !S.desc_dirty && S.desc_allow_split == allow_split && S.n_closed == L.n_closed &&
                std::memcmp(S.res_count_h, L.res_count_h, static_cast<size_t>(ns) * sizeof(int32_t)) == 0;
    for (int s = 0; same && s < ns; ++s)
      same = std::memcmp(S.level.data() + static_cast<size_t>(s) * c->max_blocks, L.level.data() + static_cast<size_t>(s) * c->max_blocks,
                         static_cast<size_t>(L.n_closed)) == 0;
    if (same) {
      std::memcpy(L.warps_h, S.warps_h, static_cast<size_t>(S.n_warps) * sizeof(WarpDesc));
      std::memcpy(L.units_h, S.units_h, static_cast<size_t>(S.n_units) * sizeof(uint32_t));
      std::memcpy(L.parts_h, S.parts_h, static_cast<size_t>(c->n_hgroups) * sizeof(StreamParts));
      L.n_warps = S.n_warps;
      L.n_units = S.n_units;
      L.desc_split = S.desc_split;
      L.desc_allow_split = allow_split;
      L.desc_dirty = false;
      return;
    }
  }
  c->desc_src = self;
  L.desc_allow_split = allow_split;
  struct Unit { uint32_t word; uint32_t cost; };
  // Pass 1: the units of every stream and their total cost.  Streams with the same levels and the
  // same number of residual rows (all streams under the staircase policy) have the same units:
  // stream s then refers to the first stream it equals (same_as[s]) and nothing is built twice.
  std::vector<int> same_as(ns);
  std::vector<std::vector<Unit>> units(ns);
  std::vector<size_t> cost(ns, 0);
  size_t total = 0;
  // A small workload leaves most warps of the GPU without work, and its launch then lasts as long
  // as its longest unit (an exact block: eight steps).  Such lists are cut finer: an exact block
  // into its four tiles and, when the workload is smaller still, a quantised block into its two
  // halves, a warp holding as little as one of them (more, finer units also mean more partial rows
  // to merge at the end, which is why this stops at some size).
  bool split = false, split_all = false;
  if (allow_split) {
    size_t rough = 0;
    for (int s = 0; s < ns; ++s) rough += static_cast<size_t>(L.n_closed + 1) * 1000 + static_cast<size_t>(L.res_count_h[s] / 16) * 550;
    split = rough < static_cast<size_t>(kTargetWarps) * kMinWarpCost / 2;          // exact blocks only
    split_all = rough < static_cast<size_t>(kTargetWarps) * kMinWarpCost / 8;      // quantised blocks too
  }
  L.desc_split = split;
  for (int s = 0; s < ns; ++s) {
    const int8_t* lv = L.level.data() + static_cast<size_t>(s) * c->max_blocks;
    same_as[s] = s;
    if (s > 0) {
      const int r = same_as[s - 1];
      if (L.res_count_h[s] == L.res_count_h[r] &&
          std::memcmp(lv, L.level.data() + static_cast<size_t>(r) * c->max_blocks, static_cast<size_t>(L.n_closed)) == 0)
        same_as[s] = r;
    }
    if (same_as[s] != s) {
      cost[s] = cost[same_as[s]];
      total += cost[s];
      continue;
    }
    const int groups = (L.res_count_h[s] + 15) / 16;
    const int n_items = L.n_closed + 1 + groups;
    std::vector<Unit>& u = units[s];
    u.reserve(n_items);
    for (int i = 0; i < n_items;) {
      int run = 1;
      if (i < L.n_closed && lv[i] != 16 && lv[i] != 8 && lv[i] != 4 && lv[i] != 2) {
        while (run < 16 && i + run < L.n_closed) {
          const int8_t l2 = lv[i + run];
          if (l2 == 16 || l2 == 8 || l2 == 4 || l2 == 2) break;
          ++run;
        }
      }
      size_t k = 0;
      for (int j = 0; j < run; ++j) k += item_cost(c, L, s, i + j);
      const uint32_t base = static_cast<uint32_t>(i) | (static_cast<uint32_t>(run) << 24);
      const int8_t lvl = (run == 1 && i < L.n_closed) ? lv[i] : int8_t{0};
      if (split && lvl == 16) {
        for (uint32_t t = 0; t < 4; ++t) u.push_back(Unit{base | ((1u << t) << 20), static_cast<uint32_t>(k / 4)});
      } else if (split_all && (lvl == 8 || lvl == 4 || lvl == 2)) {
        u.push_back(Unit{base | (3u << 20), static_cast<uint32_t>(k / 2)});
        u.push_back(Unit{base | (12u << 20), static_cast<uint32_t>(k - k / 2)});
      } else {
        u.push_back(Unit{base | (15u << 20), static_cast<uint32_t>(k)});
      }
      cost[s] += k;
      i += run;
    }
    total += cost[s];
  }
  // every head group of a stream (up to four query heads each) walks the stream's units with warps of its own
  const int hg = c->head_groups;
  total *= static_cast<size_t>(hg);
  const size_t target = std::max(split_all ? kMinWarpCost / 4 : kMinWarpCost, (total + kTargetWarps - 1) / kTargetWarps);
  // Pass 2: deal each distinct stream's units to its warps, then lay the warps out.
  int w = 0, pos = 0, row = 0;
  int dealt_for = -1, dealt_nw = 0;                 // the stream and warp count `lists` was dealt for
  std::vector<std::vector<uint32_t>> lists;         // per warp (in layout order): its units, ascending
  std::vector<std::pair<size_t, int>> heap;         // (load, warp): least loaded first, then lowest index
  for (int s = 0; s < ns; ++s) {
    const int src = same_as[s];
    const std::vector<Unit>& u0 = units[src];
    int nw = static_cast<int>((cost[s] + target / 2) / target);
    nw = std::max(1, std::min(nw, static_cast<int>(u0.size())));
    nw = std::min(nw, (c->max_warps - w) / hg - (ns - 1 - s));
    if (dealt_for != src || dealt_nw != nw) {
      std::vector<Unit> u(u0);
      std::stable_sort(u.begin(), u.end(), [](const Unit& a, const Unit& b) { return a.cost > b.cost; });
      std::vector<std::vector<uint32_t>> mine(nw);
      heap.clear();
      for (int k = 0; k < nw; ++k) heap.emplace_back(0, k);
      auto later = [](const std::pair<size_t, int>& a, const std::pair<size_t, int>& b) { return a > b; };
      std::make_heap(heap.begin(), heap.end(), later);
      for (const Unit& x : u) {                      // longest first onto the least loaded warp
        std::pop_heap(heap.begin(), heap.end(), later);
        std::pair<size_t, int>& best = heap.back();
        best.first += x.cost;
        mine[best.second].push_back(x.word);
        std::push_heap(heap.begin(), heap.end(), later);
      }
      // Longest-first dealing hands the costliest units (exact blocks, then 8-bit ones) to the first
      // warps, and a CTA is a window of consecutive warps: walk the warps with a golden-ratio stride
      // so that every window holds the same mixture of levels.  Warps of one SM share its issue
      // slots, and a CTA whose warps all run the issue-heavy levels would finish last.
      int stride = std::max(1, static_cast<int>(nw * 0.6180339887 + 0.5));
      while (std::gcd(stride, nw) != 1) ++stride;
      lists.assign(nw, {});
      for (int k = 0; k < nw; ++k) {
        std::vector<uint32_t>& m = mine[static_cast<size_t>((static_cast<long long>(k) * stride) % nw)];
        std::sort(m.begin(), m.end(), [](uint32_t a, uint32_t b) {       // by block, then by tile mask
          return (((a & kUnitItemMask) << 4) | ((a >> 20) & 15u)) < (((b & kUnitItemMask) << 4) | ((b >> 20) & 15u));
        });
        // Ascending token order runs from the oldest, narrowest blocks to the newest, widest ones, and
        // the warps of an SM would walk it in step: all of them unpacking 2- and 4-bit codes (bound
        // by instruction issue, memory idle), later all of them waiting for 8-bit and exact tiles
        // (issue slots idle).  Taking the units alternately from both ends makes every warp follow a
        // byte-heavy unit with an issue-heavy one, so its two-stage pipeline always has a long
        // compute to hide a long copy behind; starting every warp at a different place of its list
        // (below) also keeps both kinds of step in every SM at all times.  (Shifting whole CTAs
        // against one another instead - every SM uniform, the GPU mixed - gains nothing.)
        std::vector<uint32_t>& out = lists[k];
        out.clear();
        for (size_t lo = 0, hi = m.size(); lo < hi;) {
          out.push_back(m[lo++]);
          if (lo < hi) out.push_back(m[--hi]);
        }
        if (out.size() > 1) std::rotate(out.begin(), out.begin() + (static_cast<size_t>(k) * 5) % out.size(), out.end());
      }
      dealt_for = src;
      dealt_nw = nw;
    }
    // One partial row per (CTA, head group): the kernel merges the warps of a CTA that share a head
    // group.  The head groups of a stream get the same lists (stored once) and neighbouring warps, so
    // that the second reader of a block finds it in L2.
    const int pos0 = pos;
    for (int g = 0; g < hg; ++g) {
      const int hgi = s * hg + g;
      L.parts_h[hgi].begin = row;
      pos = pos0;
      for (int k = 0; k < nw; ++k) {
        const std::vector<uint32_t>& m = lists[k];
        WarpDesc& d = L.warps_h[w];
        d.stream = hgi;
        d.item_begin = pos;
        if (g == 0) std::memcpy(L.units_h + pos, m.data(), m.size() * sizeof(uint32_t));
        pos += static_cast<int>(m.size());
        d.item_end = pos;
        if (k > 0 && w % kDecodeWarps == 0) ++row;
        d.partial = row;
        ++w;
      }
      ++row;
      L.parts_h[hgi].end = row;
    }
  }
  const int padded = static_cast<int>(align_up(w, kDecodeWarps));
  for (int i = w; i < padded; ++i) L.warps_h[i] = WarpDesc{-1, 0, 0, 0};
  L.n_warps = padded;
  L.n_units = pos;
  L.desc_dirty = false;
}

void set_entry(gkv_cache* c, LayerState& L, int stream, int block, uint32_t off, int level) {
  TableEntry& e = L.table_h[static_cast<size_t>(stream) * c->table_stride + block];
  e.off256 = off;
  e.level = static_cast<uint32_t>(level);
}

int wait_event(gkv_cache* c, cudaEvent_t ev) {
  CK(c, cudaEventSynchronize(ev));
  return GKV_OK;
}

int bulk_ingest(gkv_cache* c, int layer, const uint16_t* k_new, const uint16_t* v_new, int n_new,
                const float* token_mass, const int8_t* level_plan, cudaStream_t st) {
  const gkv_config& cfg = c->cfg;
  LayerState& L = c->layers[layer];
  const int ns = c->n_streams, n_closed = n_new / kBlock, n_tail = n_new % kBlock;
  int warn = GKV_OK;
  int rc;
  if ((rc = wait_event(c, L.ev)) != GKV_OK) return rc;
  if ((rc = wait_event(c, c->ev_stage)) != GKV_OK) return rc;

  // 1. boxes / range / mass of every closed block
  const bool need_rd = cfg.policy == GKV_POLICY_RD;
  if ((cfg.page_tokens > 0 || need_rd) && n_closed > 0) {
    StatsParams sp{};
    sp.arena = c->arena;
    sp.k_in = k_new;
    sp.token_mass = token_mass;
    sp.n_tok = n_new;
    sp.n_kv_heads = cfg.n_kv_heads;
    sp.first_block = 0;
    sp.n_blocks = n_closed;
    sp.n_streams = ns;
    sp.page_tokens = cfg.page_tokens;
    sp.boxes = L.boxes_d;
    sp.box_stride = c->box_stride;
    sp.block_range = need_rd ? c->range_d : nullptr;
    sp.block_mass = need_rd ? c->mass_d : nullptr;
    CK(c, launch_stats(sp, st));
  }

  // 2. level plan
  std::fill(L.level.begin(), L.level.end(), 0);
  if (cfg.policy == GKV_POLICY_STAIRCASE) {
    std::vector<int8_t> lv(std::max(n_closed, 1));
    staircase_levels(cfg, n_closed, lv.data());
    for (int s = 0; s < ns; ++s) std::memcpy(&L.level[static_cast<size_t>(s) * c->max_blocks], lv.data(), n_closed);
  } else if (cfg.policy == GKV_POLICY_EXTERNAL) {
    for (int s = 0; s < ns; ++s)
      for (int b = 0; b < n_closed; ++b) {
        const int8_t v = level_plan[static_cast<size_t>(s) * n_closed + b];
        if (v != 16 && v != 8 && v != 4 && v != 2 && v != 1) return GKV_ERR_INVALID_ARG;
        L.level[static_cast<size_t>(s) * c->max_blocks + b] = v;
      }
  } else if (n_closed > 0) {
    std::vector<float> range(static_cast<size_t>(ns) * n_closed), mass(static_cast<size_t>(ns) * n_closed);
    CK(c, cudaMemcpyAsync(range.data(), c->range_d, range.size() * sizeof(float), cudaMemcpyDeviceToHost, st));
    CK(c, cudaMemcpyAsync(mass.data(), c->mass_d, mass.size() * sizeof(float), cudaMemcpyDeviceToHost, st));
    CK(c, cudaStreamSynchronize(st));
    // the prefill observer's block masses start the running mass of the decode phase (Sec. 3.1)
    CK(c, cudaMemcpy2DAsync(L.ema_d, static_cast<size_t>(c->max_blocks + 1) * sizeof(float), c->mass_d,
                            static_cast<size_t>(n_closed) * sizeof(float), static_cast<size_t>(n_closed) * sizeof(float), ns,
                            cudaMemcpyDeviceToDevice, st));
    CK(c, cudaMemcpy2DAsync(L.range_d, static_cast<size_t>(c->max_blocks) * sizeof(float), c->range_d,
                            static_cast<size_t>(n_closed) * sizeof(float), static_cast<size_t>(n_closed) * sizeof(float), ns,
                            cudaMemcpyDeviceToDevice, st));
    if (rd_allocate_streams(cfg, mass.data(), range.data(), n_closed, n_tail, ns, nullptr, 0, L.level.data(), c->max_blocks)) {
      L.budget_flag = true;
      warn = GKV_ERR_BUDGET;
    }
  }

  // 3. slots + table mirror.  The fast encoder takes its work from the table itself, so on its path
  // the sequences go up in groups: slots of a group, its table rows, its encode launch, and the
  // host allocates the next group's slots while the GPU encodes this one.
  const bool has_res = cfg.residual_fraction > 0.f && token_mass && n_closed > 0;
  const bool fast = n_closed > 0 && v_new &&
                    ((reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new)) & 15u) == 0;
  auto alloc_streams = [&](int s0, int s1) -> int {
    for (int s = s0; s < s1; ++s) {
      for (int b = 0; b <= n_closed; ++b) {
        const int lvl = b < n_closed ? L.level[static_cast<size_t>(s) * c->max_blocks + b] : 16;
        uint32_t off;
        if (!c->heap.alloc(lvl, &off)) return GKV_ERR_ARENA_TOO_SMALL;
        set_entry(c, L, s, b, off, lvl);
        L.table_h[static_cast<size_t>(s) * c->table_stride + b].resmask = 0;
      }
      L.res_count_h[s] = 0;
      L.res_idx[s].clear();
    }
    return GKV_OK;
  };
  // table rows of streams [s0, s1) to the device, then every closed block of theirs encoded once at its planned level
  auto encode_streams = [&](int s0, int s1) -> int {
    const size_t row = static_cast<size_t>(c->table_stride);
    int r2;
    if ((r2 = upload(c, L.table_d + s0 * row, L.table_h + s0 * row, (s1 - s0) * row * sizeof(TableEntry), st, L.ev)) != GKV_OK) return r2;
    EncodeParams ep{};
    ep.arena = c->arena;
    ep.jobs = nullptr;
    ep.n_jobs = (s1 - s0) * n_closed;
    ep.k_in = k_new;
    ep.v_in = v_new;
    ep.n_tok = n_new;
    ep.n_kv_heads = cfg.n_kv_heads;
    ep.status = c->status_d;
    ep.err = L.err_d;
    ep.err_stride = c->max_blocks;
    ep.table = L.table_d;
    ep.table_stride = c->table_stride;
    ep.n_blocks = n_closed;
    ep.first_seq = s0 / cfg.n_kv_heads;
    CK(c, launch_ingest(ep, st));
    return GKV_OK;
  };
  bool encoded = false;
  if (fast && !has_res) {
    const int per_seq = n_closed * cfg.n_kv_heads;
    const int seqs = std::max(1, (8192 + per_seq - 1) / per_seq);       // at least ~8192 blocks per launch
    for (int q0 = 0; q0 < cfg.batch; q0 += seqs) {
      const int s0 = q0 * cfg.n_kv_heads, s1 = std::min(cfg.batch, q0 + seqs) * cfg.n_kv_heads;
      if ((rc = alloc_streams(s0, s1)) != GKV_OK) return rc;
      if ((rc = encode_streams(s0, s1)) != GKV_OK) return rc;
    }
    encoded = true;
  } else if ((rc = alloc_streams(0, ns)) != GKV_OK) {
    return rc;
  }
  L.has_tail_slot = true;

  // 4. exact residual (Sec. 3.4): score, top fraction per stream, gather rows, mask the blocks
  uint8_t* stage = c->stage_h;
  size_t stage_off = 0;
  if (cfg.residual_fraction > 0.f && token_mass && n_closed > 0) {
    const int n_res_nom = static_cast<int>(std::floor(static_cast<double>(cfg.residual_fraction) * static_cast<double>(n_new)));
    int8_t* lv_stage = reinterpret_cast<int8_t*>(stage + stage_off);
    std::memcpy(lv_stage, L.level.data(), L.level.size());
    stage_off = align_up(stage_off + L.level.size(), 256);
    int32_t* k_stage = reinterpret_cast<int32_t*>(stage + stage_off);
    stage_off = align_up(stage_off + ns * sizeof(int32_t), 256);
    int max_k = 0;
    for (int s = 0; s < ns; ++s) {
      int eligible = 0;
      for (int b = 0; b < n_closed; ++b)
        if (b >= cfg.n_sink_blocks && L.level[static_cast<size_t>(s) * c->max_blocks + b] != 16) eligible += kBlock;
      k_stage[s] = std::min(std::min(n_res_nom, eligible), c->res_cap);
      max_k = std::max(max_k, k_stage[s]);
      L.res_count_h[s] = k_stage[s];
    }
    CK(c, cudaMemcpyAsync(c->levels_d, lv_stage, L.level.size(), cudaMemcpyHostToDevice, st));
    CK(c, cudaMemcpyAsync(c->kper_d, k_stage, ns * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    CK(c, launch_residual_scores(v_new, token_mass, c->levels_d, c->max_blocks, cfg.n_sink_blocks, ns,
                                 cfg.n_kv_heads, n_new, n_closed, c->scores_d, st));
    CK(c, launch_topk(c->scores_d, n_new, n_closed * kBlock, c->kper_d, 0, L.res_idx_d, c->res_cap, ns, st));
    if (max_k > 0) {
      std::vector<int32_t> idx(static_cast<size_t>(ns) * c->res_cap);
      CK(c, cudaMemcpyAsync(idx.data(), L.res_idx_d, idx.size() * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
      CK(c, cudaStreamSynchronize(st));
      for (int s = 0; s < ns; ++s) {
        L.res_idx[s].assign(idx.begin() + static_cast<size_t>(s) * c->res_cap,
                            idx.begin() + static_cast<size_t>(s) * c->res_cap + L.res_count_h[s]);
        for (int32_t tok : L.res_idx[s]) {
          if (tok < 0 || tok >= n_closed * kBlock) return GKV_ERR_BAD_STATE;
          L.table_h[static_cast<size_t>(s) * c->table_stride + tok / kBlock].resmask |= 1ull << (tok % kBlock);
        }
      }
    }
  }

  // 5. uploads, then encode every closed block once at its planned level (unless done above), copy the tail rows
  if (!encoded && !fast &&
      (rc = upload(c, L.table_d, L.table_h, static_cast<size_t>(ns) * c->table_stride * sizeof(TableEntry), st, L.ev)) != GKV_OK)
    return rc;
  if ((rc = upload(c, L.res_count_d, L.res_count_h, ns * sizeof(int32_t), st, L.ev)) != GKV_OK) return rc;
  if (L.res_count_d && cfg.residual_fraction > 0.f) {
    int max_k = 0;
    for (int s = 0; s < ns; ++s) max_k = std::max(max_k, L.res_count_h[s]);
    CK(c, launch_residual_gather(c->arena, k_new, v_new, n_new, cfg.n_kv_heads, L.res_idx_d, c->res_cap,
                                 L.res_count_d, L.res_off_d, max_k, ns, st));
  }
  const size_t n_jobs = static_cast<size_t>(ns) * n_closed;
  if (!encoded && fast) {
    if ((rc = encode_streams(0, ns)) != GKV_OK) return rc;
  } else if (!encoded && n_jobs > 0) {
    // inputs that the fast encoder does not take (unaligned rows): the general block encoder, one job per block
    EncodeJob* jobs = reinterpret_cast<EncodeJob*>(stage + stage_off);
    size_t j = 0;
    for (int s = 0; s < ns; ++s)
      for (int b = 0; b < n_closed; ++b) {
        EncodeJob& job = jobs[j++];
        job.src_off256 = 0;
        job.dst_off256 = L.table_h[static_cast<size_t>(s) * c->table_stride + b].off256;
        job.src_level = 0;
        job.dst_level = L.level[static_cast<size_t>(s) * c->max_blocks + b];
        job.stream = s;
        job.block = b;
        job.pad = 0;
      }
    CK(c, cudaMemcpyAsync(c->jobs_d, jobs, n_jobs * sizeof(EncodeJob), cudaMemcpyHostToDevice, st));
    EncodeParams ep{};
    ep.arena = c->arena;
    ep.jobs = c->jobs_d;
    ep.n_jobs = static_cast<int32_t>(n_jobs);
    ep.k_in = k_new;
    ep.v_in = v_new;
    ep.n_tok = n_new;
    ep.n_kv_heads = cfg.n_kv_heads;
    ep.status = c->status_d;
    ep.err = L.err_d;
    ep.err_stride = c->max_blocks;
    CK(c, launch_encode(ep, st));
  }
  CK(c, cudaEventRecord(c->ev_stage, st));
  CK(c, launch_append_rows(c->arena, L.table_d, c->table_stride, n_closed, ns, cfg.n_kv_heads, k_new, v_new, n_new,
                           n_closed * kBlock, n_tail, 0, st));
  L.n_closed = n_closed;
  L.n_tail = n_tail;
  L.desc_dirty = true;
  L.last_mode = 0;
  L.quest_ran = false;
  return warn;
}

// Requantise every block whose target level lies below its current one (monotone: levels only
// fall), each from its current representation, in one encode launch.  target: [n_closed] shared by
// all streams (stride 0) or [n_streams][stride].
int demote_to_targets(gkv_cache* c, LayerState& L, const int8_t* target, size_t stride, cudaStream_t st) {
  const gkv_config& cfg = c->cfg;
  const int ns = c->n_streams;
  int rc;
  std::vector<std::pair<int, int>> want_list;            // (stream, block) whose level falls
  for (int s = 0; s < ns; ++s) {
    const int8_t* tg = target + static_cast<size_t>(s) * stride;
    const int8_t* cur = L.level.data() + static_cast<size_t>(s) * c->max_blocks;
    for (int b = 0; b < L.n_closed; ++b)
      if (tg[b] < cur[b]) want_list.emplace_back(s, b);    // monotone: levels only fall
  }
  if (want_list.empty()) return GKV_OK;
  EncodeJob* jobs;
  cudaEvent_t ev_jobs;
  if (want_list.size() <= c->demote_cap) {
    const int slot = c->demote_next++ % gkv_cache::kDemoteSlots;
    jobs = c->demote_h + static_cast<size_t>(slot) * c->demote_cap;
    ev_jobs = c->ev_demote[slot];
  } else {
    jobs = reinterpret_cast<EncodeJob*>(c->stage_h);
    ev_jobs = c->ev_stage;
  }
  if ((rc = wait_event(c, ev_jobs)) != GKV_OK) return rc;
  if ((rc = wait_event(c, L.ev)) != GKV_OK) return rc;
  // Phase 1: a destination slot for every job.  If the arena cannot hold them all, everything taken
  // so far goes back and nothing else has changed: the host mirrors, the device table and the
  // levels still describe the cache as it was, and the call can be repeated with a larger arena.
  std::vector<uint32_t> dst(want_list.size());
  for (size_t i = 0; i < want_list.size(); ++i) {
    const int8_t want = target[static_cast<size_t>(want_list[i].first) * stride + want_list[i].second];
    if (!c->heap.alloc(want, &dst[i])) {
      for (size_t k = 0; k < i; ++k)
        c->heap.release(target[static_cast<size_t>(want_list[k].first) * stride + want_list[k].second], dst[k]);
      return GKV_ERR_ARENA_TOO_SMALL;
    }
  }
  // Phase 2: the job list and the mirrors.
  size_t n_jobs = 0;
  std::vector<std::pair<int, uint32_t>> to_free;
  to_free.reserve(want_list.size());
  for (size_t i = 0; i < want_list.size(); ++i) {
    const int s = want_list[i].first, b = want_list[i].second;
    const int8_t want = target[static_cast<size_t>(s) * stride + b];
    int8_t& cur = L.level[static_cast<size_t>(s) * c->max_blocks + b];
    TableEntry& e = L.table_h[static_cast<size_t>(s) * c->table_stride + b];
    const uint32_t off = dst[i];
    EncodeJob& job = jobs[n_jobs++];
    job.src_off256 = e.off256;
    job.dst_off256 = off;
    job.src_level = cur;
    job.dst_level = want;
    job.stream = s;
    job.block = b;
    job.pad = 0;
    to_free.emplace_back(cur, e.off256);
    e.off256 = off;
    e.level = static_cast<uint32_t>(want);
    cur = want;
  }
  CK(c, cudaMemcpyAsync(c->jobs_d, jobs, n_jobs * sizeof(EncodeJob), cudaMemcpyHostToDevice, st));
  CK(c, cudaEventRecord(ev_jobs, st));
  EncodeParams ep{};
  ep.arena = c->arena;
  ep.jobs = c->jobs_d;
  ep.n_jobs = static_cast<int32_t>(n_jobs);
  ep.n_kv_heads = cfg.n_kv_heads;
  ep.status = c->status_d;
  ep.err = L.err_d;
  ep.err_stride = c->max_blocks;
  ep.table = L.table_d;             // the kernel repoints the device table; the host mirror is already updated
  ep.table_stride = c->table_stride;
  CK(c, launch_encode(ep, st));
  for (auto& f : to_free) c->heap.release(f.first, f.second);
  L.desc_dirty = true;
  return GKV_OK;
}

int append_one(gkv_cache* c, int layer, const uint16_t* k_new, const uint16_t* v_new, cudaStream_t st) {
  const gkv_config& cfg = c->cfg;
  LayerState& L = c->layers[layer];
  const int ns = c->n_streams;
  int rc;
  if (!L.has_tail_slot) {
    // a new tail block starts: give every stream an exact slot for it
    if ((rc = wait_event(c, L.ev)) != GKV_OK) return rc;
    // all or nothing: when the arena cannot hold a slot for every stream, the slots taken so far go
    // back and the layer is as it was
    std::vector<uint32_t> slots(ns);
    for (int s = 0; s < ns; ++s) {
      if (!c->heap.alloc(16, &slots[s])) {
        for (int k = 0; k < s; ++k) c->heap.release(16, slots[k]);
        return GKV_ERR_ARENA_TOO_SMALL;
      }
    }
    for (int s = 0; s < ns; ++s) {
      set_entry(c, L, s, L.n_closed, slots[s], 16);
      L.table_h[static_cast<size_t>(s) * c->table_stride + L.n_closed].resmask = 0;
    }
    L.has_tail_slot = true;
    if ((rc = upload_table_column(c, L, L.n_closed, st)) != GKV_OK) return rc;
    // The work lists stay valid: they always hold the partial block as item n_closed (skipped by the
    // kernel while it is empty), so a new partial block changes only its table entry.
  }
  CK(c, launch_append_rows(c->arena, L.table_d, c->table_stride, L.n_closed, ns, cfg.n_kv_heads, k_new, v_new, 1, 0, 1,
                           L.n_tail, st));
  L.n_tail += 1;
  if (L.n_tail < kBlock) return GKV_OK;

  // the tail block closes (still level 16, in place): boxes from its unquantised keys, then the
  // staircase moves every block that crossed a rung boundary one or more rungs down
  const int closed_block = L.n_closed;
  {
    StatsParams sp{};
    sp.arena = c->arena;
    sp.k_in = nullptr;
    sp.table = L.table_d;
    sp.table_stride = c->table_stride;
    sp.n_tok = 0;
    sp.n_kv_heads = cfg.n_kv_heads;
    sp.first_block = closed_block;
    sp.n_blocks = 1;
    sp.n_streams = ns;
    sp.page_tokens = cfg.page_tokens;
    sp.boxes = L.boxes_d;
    sp.box_stride = c->box_stride;
    sp.err = L.err_d;                        // largest value-row norm of the closing block (certificate)
    sp.err_stride = c->max_blocks;
    if (cfg.policy == GKV_POLICY_RD) {       // range proxy of the closing block, kept for later re-allocation
      sp.block_range = L.range_d;
      sp.stat_stride = c->max_blocks;
      sp.stat_base = closed_block;
    }
    CK(c, launch_stats(sp, st));
  }
  for (int s = 0; s < ns; ++s) L.level[static_cast<size_t>(s) * c->max_blocks + closed_block] = 16;
  L.n_closed += 1;
  L.n_tail = 0;
  L.has_tail_slot = false;
  L.desc_dirty = true;
  if (cfg.policy != GKV_POLICY_STAIRCASE) return GKV_OK;

  std::vector<int8_t> target(L.n_closed);
  staircase_levels(cfg, L.n_closed, target.data());
  return demote_to_targets(c, L, target.data(), 0, st);
}

// ---- latent-attention (MLA) host paths -----------------------------------------------------------
// One stream per sequence; staircase or external plans only.  The block table, slot heap and
// staging are shared with the GQA path; the kernels are those of gkv_mla.cu.
size_t mla_item_cost(const gkv_cache* c, const LayerState& L, int stream, int item) {
  // Cost of a block for the split of a stream over the CTAs and their quads, in units where a 4-bit
  // block is 1000.  Exact, 8-bit and 4-bit blocks: measured on B200 as the time of a call over a cache that
  // holds one rung only (262,144 tokens), less the call's fixed part.  A centroid block is one row of a
  // 16-row unit: swept on the 1M-token staircase (a call over centroid blocks only is all fixed cost).
  if (item < L.n_closed) {
    switch (L.level[static_cast<size_t>(stream) * c->max_blocks + item]) {
      case 16: return 1100;
      case 8: return 1005;
      case 4: return 1000;
      default: return 24;
    }
  }
  return 900;                     // tail
}

void mla_build_descs(gkv_cache* c, LayerState& L) {
  const int ns = c->n_streams;
  std::vector<size_t> cost(ns, 0);
  size_t total = 0;
  const int n_items = L.n_closed + 1;
  for (int s = 0; s < ns; ++s) {
    for (int i = 0; i < n_items; ++i) cost[s] += mla_item_cost(c, L, s, i);
    total += cost[s];
  }
  const size_t target = std::max<size_t>(800, (total + kMlaTargetCtas - 1) / kMlaTargetCtas);
  std::vector<WarpDesc> cta(static_cast<size_t>(kMlaTargetCtas) + 2 * ns);
  int w = 0;
  for (int s = 0; s < ns; ++s) {
    int nw = static_cast<int>((cost[s] + target / 2) / target);
    nw = std::max(1, std::min(nw, n_items));
    nw = std::min(nw, kMlaTargetCtas + 2 * ns - w - (ns - 1 - s));
    L.parts_h[s].begin = w;
    size_t acc = 0;
    int item = 0;
    for (int k = 0; k < nw; ++k) {
      const size_t limit = cost[s] * (k + 1) / nw;
      const int begin = item;
      const int max_end = n_items - (nw - 1 - k);
      do {
        acc += mla_item_cost(c, L, s, item);
        ++item;
      } while (item < max_end && acc < limit);
      cta[w] = WarpDesc{s, begin, item, w};
      ++w;
    }
    cta[w - 1].item_end = n_items;
    L.parts_h[s].end = w;
  }
  // a CTA's range is cut once more, by cost, into the contiguous ranges of its quads (descriptor
  // kMlaQuads * cta + quad; all of them name the CTA's partial row)
  for (int i = 0; i < w; ++i) {
    size_t tot = 0;
    for (int it = cta[i].item_begin; it < cta[i].item_end; ++it) tot += mla_item_cost(c, L, cta[i].stream, it);
    size_t acc = 0;
    int item = cta[i].item_begin;
    for (int qd = 0; qd < kMlaQuads; ++qd) {
      const size_t limit = tot * (qd + 1) / kMlaQuads;
      const int begin = item;
      while (item < cta[i].item_end && (qd == kMlaQuads - 1 || acc + mla_item_cost(c, L, cta[i].stream, item) / 2 < limit)) {
        acc += mla_item_cost(c, L, cta[i].stream, item);
        ++item;
      }
      L.warps_h[kMlaQuads * i + qd] = WarpDesc{cta[i].stream, begin, item, cta[i].partial};
    }
  }
  L.n_warps = w;                  // here: number of CTAs
  L.desc_dirty = false;
}

int mla_bulk_ingest(gkv_cache* c, int layer, const uint16_t* k_new, int n_new, const int8_t* level_plan, cudaStream_t st) {
  const gkv_config& cfg = c->cfg;
  LayerState& L = c->layers[layer];
  const int ns = c->n_streams, n_closed = n_new / kBlock, n_tail = n_new % kBlock;
  int rc;
  if ((rc = wait_event(c, L.ev)) != GKV_OK) return rc;
  if ((rc = wait_event(c, c->ev_stage)) != GKV_OK) return rc;
  std::fill(L.level.begin(), L.level.end(), 0);
  if (cfg.policy == GKV_POLICY_STAIRCASE) {
    std::vector<int8_t> lv(std::max(n_closed, 1));
    staircase_levels(cfg, n_closed, lv.data());
    for (int s = 0; s < ns; ++s) std::memcpy(&L.level[static_cast<size_t>(s) * c->max_blocks], lv.data(), n_closed);
  } else {
    for (int s = 0; s < ns; ++s)
      for (int b = 0; b < n_closed; ++b) {
        const int8_t v = level_plan[static_cast<size_t>(s) * n_closed + b];
        if (v != 16 && v != 8 && v != 4 && v != 1) return v == 2 ? GKV_ERR_UNSUPPORTED : GKV_ERR_INVALID_ARG;
        L.level[static_cast<size_t>(s) * c->max_blocks + b] = v;
      }
  }
  for (int s = 0; s < ns; ++s) {
    for (int b = 0; b <= n_closed; ++b) {
      const int lvl = b < n_closed ? L.level[static_cast<size_t>(s) * c->max_blocks + b] : 16;
      uint32_t off;
      if (!c->heap.alloc(lvl, &off)) return GKV_ERR_ARENA_TOO_SMALL;
      set_entry(c, L, s, b, off, lvl);
      L.table_h[static_cast<size_t>(s) * c->table_stride + b].resmask = 0;
    }
    L.res_count_h[s] = 0;
  }
  L.has_tail_slot = true;
  if ((rc = upload(c, L.table_d, L.table_h, static_cast<size_t>(ns) * c->table_stride * sizeof(TableEntry), st, L.ev)) != GKV_OK) return rc;
  const size_t n_jobs = static_cast<size_t>(ns) * n_closed;
  if (n_jobs > 0) {
    EncodeJob* jobs = reinterpret_cast<EncodeJob*>(c->stage_h);
    size_t j = 0;
    for (int s = 0; s < ns; ++s)
      for (int b = 0; b < n_closed; ++b) {
        EncodeJob& job = jobs[j++];
        job.src_off256 = 0;
        job.dst_off256 = L.table_h[static_cast<size_t>(s) * c->table_stride + b].off256;
        job.src_level = 0;
        job.dst_level = L.level[static_cast<size_t>(s) * c->max_blocks + b];
        job.stream = s;
        job.block = b;
        job.pad = 0;
      }
    CK(c, cudaMemcpyAsync(c->jobs_d, jobs, n_jobs * sizeof(EncodeJob), cudaMemcpyHostToDevice, st));
    MlaEncodeParams ep{};
    ep.arena = c->arena;
    ep.jobs = c->jobs_d;
    ep.n_jobs = static_cast<int32_t>(n_jobs);
    ep.k_in = k_new;
    ep.n_tok = n_new;
    ep.status = c->status_d;
    // 16-byte aligned rows take the bulk encoder; the general block encoder stores the same bits
    if ((reinterpret_cast<uintptr_t>(k_new) & 15u) == 0) CK(c, launch_mla_ingest(ep, st));
    else CK(c, launch_mla_encode(ep, st));
  }
  CK(c, cudaEventRecord(c->ev_stage, st));
  CK(c, launch_mla_append_rows(c->arena, L.table_d, c->table_stride, n_closed, ns, k_new, n_new, n_closed * kBlock, n_tail, 0, st));
  L.n_closed = n_closed;
  L.n_tail = n_tail;
  L.desc_dirty = true;
  L.last_mode = 0;
  return GKV_OK;
}

int mla_append_one(gkv_cache* c, int layer, const uint16_t* k_new, cudaStream_t st) {
  const gkv_config& cfg = c->cfg;
  LayerState& L = c->layers[layer];
  const int ns = c->n_streams;
  int rc;
  const size_t table_bytes = static_cast<size_t>(ns) * c->table_stride * sizeof(TableEntry);
  if (!L.has_tail_slot) {
    if ((rc = wait_event(c, L.ev)) != GKV_OK) return rc;
    std::vector<uint32_t> slots(ns);                     // all or nothing, as in append_one
    for (int s = 0; s < ns; ++s) {
      if (!c->heap.alloc(16, &slots[s])) {
        for (int k = 0; k < s; ++k) c->heap.release(16, slots[k]);
        return GKV_ERR_ARENA_TOO_SMALL;
      }
    }
    for (int s = 0; s < ns; ++s) {
      set_entry(c, L, s, L.n_closed, slots[s], 16);
      L.table_h[static_cast<size_t>(s) * c->table_stride + L.n_closed].resmask = 0;
    }
    L.has_tail_slot = true;
    if ((rc = upload(c, L.table_d, L.table_h, table_bytes, st, L.ev)) != GKV_OK) return rc;
    L.desc_dirty = true;
  }
  CK(c, launch_mla_append_rows(c->arena, L.table_d, c->table_stride, L.n_closed, ns, k_new, 1, 0, 1, L.n_tail, st));
  L.n_tail += 1;
  if (L.n_tail < kBlock) return GKV_OK;
  const int closed_block = L.n_closed;
  for (int s = 0; s < ns; ++s) L.level[static_cast<size_t>(s) * c->max_blocks + closed_block] = 16;
  L.n_closed += 1;
  L.n_tail = 0;
  L.has_tail_slot = false;
  L.desc_dirty = true;
  if (cfg.policy != GKV_POLICY_STAIRCASE) return GKV_OK;
  std::vector<int8_t> target(L.n_closed);
  staircase_levels(cfg, L.n_closed, target.data());
  if ((rc = wait_event(c, c->ev_stage)) != GKV_OK) return rc;
  if ((rc = wait_event(c, L.ev)) != GKV_OK) return rc;
  EncodeJob* jobs = reinterpret_cast<EncodeJob*>(c->stage_h);
  size_t n_jobs = 0;
  // phase 1: a destination slot for every block that falls; on failure they all go back and the
  // mirrors, the levels and the device table are untouched
  std::vector<std::pair<int, int>> want_list;
  for (int s = 0; s < ns; ++s)
    for (int b = 0; b < L.n_closed; ++b)
      if (target[b] < L.level[static_cast<size_t>(s) * c->max_blocks + b]) want_list.emplace_back(s, b);
  std::vector<uint32_t> dst(want_list.size());
  for (size_t i = 0; i < want_list.size(); ++i) {
    if (!c->heap.alloc(target[want_list[i].second], &dst[i])) {
      for (size_t k = 0; k < i; ++k) c->heap.release(target[want_list[k].second], dst[k]);
      return GKV_ERR_ARENA_TOO_SMALL;
    }
  }
  // phase 2: jobs and mirrors
  std::vector<std::pair<int, uint32_t>> to_free;
  for (size_t i = 0; i < want_list.size(); ++i) {
    const int s = want_list[i].first, b = want_list[i].second;
    int8_t& cur = L.level[static_cast<size_t>(s) * c->max_blocks + b];
    TableEntry& e = L.table_h[static_cast<size_t>(s) * c->table_stride + b];
    EncodeJob& job = jobs[n_jobs++];
    job.src_off256 = e.off256;
    job.dst_off256 = dst[i];
    job.src_level = cur;
    job.dst_level = target[b];
    job.stream = s;
    job.block = b;
    job.pad = 0;
    to_free.emplace_back(cur, e.off256);
    e.off256 = dst[i];
    e.level = static_cast<uint32_t>(target[b]);
    cur = target[b];
  }
  if (n_jobs > 0) {
    CK(c, cudaMemcpyAsync(c->jobs_d, jobs, n_jobs * sizeof(EncodeJob), cudaMemcpyHostToDevice, st));
    CK(c, cudaEventRecord(c->ev_stage, st));
    MlaEncodeParams ep{};
    ep.arena = c->arena;
    ep.jobs = c->jobs_d;
    ep.n_jobs = static_cast<int32_t>(n_jobs);
    ep.status = c->status_d;
    CK(c, launch_mla_encode(ep, st));
    for (auto& f : to_free) c->heap.release(f.first, f.second);
    if ((rc = upload(c, L.table_d, L.table_h, table_bytes, st, L.ev)) != GKV_OK) return rc;
  }
  return GKV_OK;
}

int mla_decode(gkv_cache* c, LayerState& L, const void* q, float* out, float* lse, cudaStream_t st) {
  if (L.desc_dirty) {
    int rc = wait_event(c, L.ev_desc);
    if (rc != GKV_OK) return rc;
    mla_build_descs(c, L);
    if ((rc = upload(c, L.warps_d, L.warps_h, static_cast<size_t>(L.n_warps) * kMlaQuads * sizeof(WarpDesc), st, L.ev_desc)) != GKV_OK) return rc;
    if ((rc = upload(c, L.parts_d, L.parts_h, static_cast<size_t>(c->n_streams) * sizeof(StreamParts), st, L.ev_desc)) != GKV_OK) return rc;
  }
  MlaDecodeParams p{};
  p.arena = c->arena;
  p.table = L.table_d;
  p.ctas = L.warps_d;
  p.q = static_cast<const uint16_t*>(q);
  p.partial = c->partial_d;
  p.table_stride = c->table_stride;
  p.n_closed = L.n_closed;
  p.n_tail = L.n_tail;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  p.status = c->status_d;
  L.last_mode = 1;
  CK(c, launch_mla_decode(p, L.n_warps, L.parts_d, c->n_streams, out, lse, st));
  return GKV_OK;
}

uint64_t full_read_bits(const gkv_cache* c, const LayerState& L) {
  const uint64_t nval_tok = nval_per_token(c->cfg);
  uint64_t bits = 0;
  for (int s = 0; s < c->n_streams; ++s) {
    for (int b = 0; b < L.n_closed; ++b) bits += block_bits(L.level[static_cast<size_t>(s) * c->max_blocks + b], nval_tok);
    bits += static_cast<uint64_t>(L.n_tail) * 16 * nval_tok;
    bits += static_cast<uint64_t>(L.res_count_h[s]) * 16 * nval_tok;
  }
  return bits;
}

// ---- page selection without any allocation -----------------------------------------------------
// Scratch for gkv_quest_select_static: page scores of one call, [n_streams][score_stride] fp32.
// Every GPU that loads the library holds these 4 MiB until the process exits.
constexpr size_t kStaticScoreFloats = size_t(1) << 20;
static __device__ __align__(256) float g_static_scores[kStaticScoreFloats];
constexpr int kMaxDevices = 64;
static float* g_static_scores_ptr[kMaxDevices] = {};

// In host code the array's name is only a handle; the device address has to be asked for, once
// per device, with that device current.  The device is the one that owns the cache's arena (not
// whatever device the calling thread happens to have current), and the first look-up per device
// is serialised between host threads.
std::mutex g_static_scores_mutex;
int static_scores_address(gkv_cache* c, float** out) {
  const int dev = c->device;
  if (dev < 0 || dev >= kMaxDevices) return GKV_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_scores_mutex);
  if (!g_static_scores_ptr[dev]) {
    int cur = -1;
    CK(c, cudaGetDevice(&cur));
    if (cur != dev) CK(c, cudaSetDevice(dev));
    void* ptr = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scores);
    if (cur != dev) cudaSetDevice(cur);
    if (e != cudaSuccess) return cuda_fail(c, e);
    g_static_scores_ptr[dev] = static_cast<float*>(ptr);
  }
  *out = g_static_scores_ptr[dev];
  return GKV_OK;
}

}  // namespace

// ================================================================================================
extern "C" {

const char* gkv_strerror(int status) {
  switch (status) {
    case GKV_OK: return "ok";
    case GKV_ERR_INVALID_ARG: return "invalid argument";
    case GKV_ERR_ARENA_TOO_SMALL: return "arena too small";
    case GKV_ERR_CTX_FULL: return "context full";
    case GKV_ERR_BAD_STATE: return "bad state";
    case GKV_ERR_UNSUPPORTED: return "unsupported shape or combination";
    case GKV_ERR_RANGE: return "scale or zero saturated at fp16 range";
    case GKV_ERR_BUDGET: return "rate-distortion budget unreachable";
    case GKV_ERR_CUDA: return "CUDA runtime error";
    default: return "unknown status";
  }
}

int gkv_last_cuda_error(gkv_cache* c) { return c ? c->last_cuda : 0; }

int gkv_query_arena_bytes(const gkv_config* cfg, size_t* bytes) {
  int rc = validate_config(cfg);
  if (rc != GKV_OK) return rc;
  if (!bytes) return GKV_ERR_INVALID_ARG;
  const Derived d = derive(*cfg);
  const ArenaPlan a = plan_arena(*cfg, d);
  const size_t heap = static_cast<size_t>(cfg->n_layers) * d.n_streams * worst_stream_bytes(*cfg, d);
  *bytes = a.heap_begin + align_up(heap, 256) + 4096;
  return GKV_OK;
}

int gkv_create(const gkv_config* cfg, void* arena, size_t arena_bytes, gkv_cache** out) {
  int rc = validate_config(cfg);
  if (rc != GKV_OK) return rc;
  if (!arena || !out || (reinterpret_cast<uintptr_t>(arena) & 255)) return GKV_ERR_INVALID_ARG;
  const Derived d = derive(*cfg);
  const ArenaPlan a = plan_arena(*cfg, d);
  if (arena_bytes < a.heap_begin + geo_slot_bytes(*cfg, 16)) return GKV_ERR_ARENA_TOO_SMALL;
  if ((arena_bytes / 256) > 0xffffffffull) return GKV_ERR_UNSUPPORTED;
  gkv_cache* c = new (std::nothrow) gkv_cache();
  if (!c) return GKV_ERR_INVALID_ARG;
  c->cfg = *cfg;
  {
    cudaPointerAttributes attr{};
    if (cudaPointerGetAttributes(&attr, arena) == cudaSuccess && attr.type == cudaMemoryTypeDevice) c->device = attr.device;
    else cudaGetDevice(&c->device);
  }
  c->arena = static_cast<uint8_t*>(arena);
  c->arena_bytes = arena_bytes;
  c->n_streams = d.n_streams;
  c->group = d.group;
  c->head_groups = d.head_groups;
  c->n_hgroups = d.n_hgroups;
  c->max_blocks = d.max_blocks;
  c->table_stride = d.table_stride;
  c->max_warps = d.max_warps;
  c->res_cap = d.res_cap;
  c->box_stride = d.box_stride;
  c->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : static_cast<float>(1.0 / std::sqrt(static_cast<double>(cfg->d_k)));
  for (int i = 0; i < 5; ++i) c->heap.units[i] = static_cast<uint32_t>(geo_slot_bytes(*cfg, kLevels[i]) / 256);
  c->heap.begin = c->heap.bump = static_cast<uint32_t>(a.heap_begin / 256);
  c->heap.end = static_cast<uint32_t>(arena_bytes / 256);
  c->status_d = reinterpret_cast<uint32_t*>(c->arena + a.status);
  c->debug_d = c->arena + a.debug;
  c->partial_d = reinterpret_cast<float*>(c->arena + a.partial);
  c->range_d = reinterpret_cast<float*>(c->arena + a.range);
  c->mass_d = reinterpret_cast<float*>(c->arena + a.mass);
  c->levels_d = reinterpret_cast<int8_t*>(c->arena + a.levels);
  c->scores_d = reinterpret_cast<float*>(c->arena + a.scores);
  c->kper_d = reinterpret_cast<int32_t*>(c->arena + a.kper);
  c->tickets_d = reinterpret_cast<int32_t*>(c->arena + a.tickets);
  c->mass_raw_d = reinterpret_cast<float2*>(c->arena + a.mass_raw);
  c->res_raw_d = reinterpret_cast<float2*>(c->arena + a.res_raw);
  c->lse2_d = reinterpret_cast<float*>(c->arena + a.lse2);
  c->jobs_d = reinterpret_cast<EncodeJob*>(c->arena + a.jobs);
  c->jobs_cap = static_cast<size_t>(d.n_streams) * d.max_blocks;

  auto fail = [&](cudaError_t e) {
    c->last_cuda = static_cast<int>(e);
    gkv_destroy(c);
    return GKV_ERR_CUDA;
  };
  cudaError_t e = cudaMemset(c->arena, 0, a.heap_begin);
  if (e != cudaSuccess) return fail(e);
  c->stage_bytes = align_up(c->jobs_cap * sizeof(EncodeJob), 256) + align_up(static_cast<size_t>(d.n_streams) * d.max_blocks, 256) +
                   align_up(d.n_streams * sizeof(int32_t), 256) + 1024;
  if ((e = cudaHostAlloc(reinterpret_cast<void**>(&c->stage_h), c->stage_bytes, cudaHostAllocDefault)) != cudaSuccess) return fail(e);
  if ((e = cudaEventCreateWithFlags(&c->ev_stage, cudaEventDisableTiming)) != cudaSuccess) return fail(e);
  c->demote_cap = static_cast<size_t>(d.n_streams) * 8;
  if ((e = cudaHostAlloc(reinterpret_cast<void**>(&c->demote_h), gkv_cache::kDemoteSlots * c->demote_cap * sizeof(EncodeJob),
                         cudaHostAllocDefault)) != cudaSuccess) return fail(e);
  for (int i = 0; i < gkv_cache::kDemoteSlots; ++i)
    if ((e = cudaEventCreateWithFlags(&c->ev_demote[i], cudaEventDisableTiming)) != cudaSuccess) return fail(e);
  c->layers.resize(cfg->n_layers);
  for (int l = 0; l < cfg->n_layers; ++l) {
    LayerState& L = c->layers[l];
    uint8_t* lb = c->arena + a.per_layer + static_cast<size_t>(l) * a.layer_bytes;
    L.table_d = reinterpret_cast<TableEntry*>(lb + a.l_table);
    L.warps_d = reinterpret_cast<WarpDesc*>(lb + a.l_warps);
    L.units_d = reinterpret_cast<uint32_t*>(lb + a.l_units);
    L.parts_d = reinterpret_cast<StreamParts*>(lb + a.l_parts);
    L.res_off_d = reinterpret_cast<uint32_t*>(lb + a.l_resoff);
    L.res_count_d = reinterpret_cast<int32_t*>(lb + a.l_rescount);
    L.res_idx_d = reinterpret_cast<int32_t*>(lb + a.l_residx);
    L.boxes_d = reinterpret_cast<uint16_t*>(lb + a.l_boxes);
    L.ema_d = reinterpret_cast<float*>(lb + a.l_ema);
    L.range_d = reinterpret_cast<float*>(lb + a.l_range);
    L.err_d = reinterpret_cast<float4*>(lb + a.l_err);
    L.level.assign(static_cast<size_t>(d.n_streams) * d.max_blocks, 0);
    L.res_idx.resize(d.n_streams);
    const size_t tb = static_cast<size_t>(d.n_streams) * d.table_stride * sizeof(TableEntry);
    if ((e = cudaHostAlloc(reinterpret_cast<void**>(&L.table_h), tb, cudaHostAllocDefault)) != cudaSuccess) return fail(e);
    std::memset(L.table_h, 0, tb);
    if ((e = cudaHostAlloc(reinterpret_cast<void**>(&L.warps_h), d.max_warps * sizeof(WarpDesc), cudaHostAllocDefault)) != cudaSuccess) return fail(e);
    if ((e = cudaHostAlloc(reinterpret_cast<void**>(&L.units_h), static_cast<size_t>(d.n_streams) * d.unit_stride * sizeof(uint32_t),
                           cudaHostAllocDefault)) != cudaSuccess) return fail(e);
    if ((e = cudaHostAlloc(reinterpret_cast<void**>(&L.parts_h), d.n_hgroups * sizeof(StreamParts), cudaHostAllocDefault)) != cudaSuccess) return fail(e);
    if ((e = cudaHostAlloc(reinterpret_cast<void**>(&L.res_off_h), d.n_streams * sizeof(uint32_t), cudaHostAllocDefault)) != cudaSuccess) return fail(e);
    if ((e = cudaHostAlloc(reinterpret_cast<void**>(&L.res_count_h), d.n_streams * sizeof(int32_t), cudaHostAllocDefault)) != cudaSuccess) return fail(e);
    for (int s = 0; s < d.n_streams; ++s) {
      L.res_count_h[s] = 0;
      L.res_off_h[s] = static_cast<uint32_t>((a.per_layer + static_cast<size_t>(l) * a.layer_bytes + a.l_respool +
                                              static_cast<size_t>(s) * d.res_cap * 2 * kRowBytes) / 256);
    }
    if ((e = cudaEventCreateWithFlags(&L.ev, cudaEventDisableTiming)) != cudaSuccess) return fail(e);
    if ((e = cudaEventCreateWithFlags(&L.ev_desc, cudaEventDisableTiming)) != cudaSuccess) return fail(e);
    if ((e = cudaMemcpy(L.res_off_d, L.res_off_h, d.n_streams * sizeof(uint32_t), cudaMemcpyHostToDevice)) != cudaSuccess) return fail(e);
  }
  if ((e = cudaDeviceSynchronize()) != cudaSuccess) return fail(e);
  *out = c;
  return GKV_OK;
}

int gkv_debug_plan_levels(const gkv_config* cfg, int32_t n_closed, int32_t n_tail, const float* mass, const float* range,
                          int8_t* levels, int32_t* budget_miss) {
  int rc = validate_config(cfg);
  if (rc != GKV_OK) return rc;
  if (n_closed < 0 || n_tail < 0 || n_tail >= kBlock || (n_closed > 0 && !levels)) return GKV_ERR_INVALID_ARG;
  if (budget_miss) *budget_miss = 0;
  if (n_closed == 0) return GKV_OK;
  if (cfg->policy == GKV_POLICY_STAIRCASE) {
    staircase_levels(*cfg, n_closed, levels);
    return GKV_OK;
  }
  if (cfg->policy == GKV_POLICY_RD) {
    if (!mass || !range) return GKV_ERR_INVALID_ARG;
    const bool miss = rd_allocate(*cfg, mass, range, n_closed, n_tail, nullptr, levels);
    if (budget_miss) *budget_miss = miss ? 1 : 0;
    return GKV_OK;
  }
  return GKV_ERR_UNSUPPORTED;      // external plans are the caller's
}

int gkv_debug_replan_levels(const gkv_config* cfg, int32_t n_closed, int32_t n_tail, const float* mass, const float* range,
                            const int8_t* prev, int8_t* levels, int32_t* budget_miss) {
  int rc = validate_config(cfg);
  if (rc != GKV_OK) return rc;
  if (cfg->policy != GKV_POLICY_RD) return GKV_ERR_BAD_STATE;
  if (n_closed <= 0 || n_tail < 0 || n_tail >= kBlock || !mass || !range || !prev || !levels) return GKV_ERR_INVALID_ARG;
  const bool miss = rd_allocate(*cfg, mass, range, n_closed, n_tail, prev, levels);
  if (budget_miss) *budget_miss = miss ? 1 : 0;
  return GKV_OK;
}

namespace {
// Largest number of closed blocks whose breakpoints the device allocator sorts in shared memory.
constexpr int kRdPlanMaxBlocks = 4095;

// Level plan of every stream of a layer from its running masses and range proxies: on the device when
// the breakpoints fit (one small launch and n bytes per stream back instead of 8 n and the host's
// sort), else on the host.  target: [n_streams][n].  *missed: some stream cannot meet the budget.
int rd_plan_layer(gkv_cache* c, LayerState& L, int8_t* target, bool* missed, cudaStream_t st) {
  const gkv_config& cfg = c->cfg;
  const int n = L.n_closed, ns = c->n_streams;
  *missed = false;
  if (n <= kRdPlanMaxBlocks) {
    const long long nval_tok = cfg.d_k + cfg.d_v;
    const long long T = static_cast<long long>(n) * kBlock + L.n_tail;
    RdPlanParams p{};
    p.mass = L.ema_d;
    p.range = L.range_d;
    p.table = L.table_d;
    p.levels_out = c->levels_d;
    p.miss_flag = reinterpret_cast<uint32_t*>(c->mass_d);        // ingest scratch, idle here
    p.n = n;
    p.mass_stride = c->max_blocks + 1;
    p.range_stride = c->max_blocks;
    p.table_stride = c->table_stride;
    p.out_stride = c->max_blocks;
    rd_plan_smem_bytes(n, &p.m_pad);
    p.n_sink_blocks = cfg.n_sink_blocks;
    p.retire_after = cfg.retire_after;
    p.monotone = cfg.monotone_in_age != 0;
    p.use_prev = 1;
    p.nval_tok = static_cast<unsigned long long>(nval_tok);
    p.budget_bits = static_cast<unsigned long long>(std::floor(static_cast<double>(cfg.rd_budget_bpv) * static_cast<double>(T * nval_tok)));
    p.tail_bits = static_cast<unsigned long long>(L.n_tail) * 16ull * static_cast<unsigned long long>(nval_tok);
    uint32_t flag = 0;
    CK(c, cudaMemsetAsync(p.miss_flag, 0, sizeof(uint32_t), st));
    CK(c, launch_rd_plan(p, ns, st));
    CK(c, cudaMemcpy2DAsync(target, static_cast<size_t>(n), c->levels_d, static_cast<size_t>(c->max_blocks), static_cast<size_t>(n), ns,
                            cudaMemcpyDeviceToHost, st));
    CK(c, cudaMemcpyAsync(&flag, p.miss_flag, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
    CK(c, cudaStreamSynchronize(st));
    *missed = flag != 0;
    return GKV_OK;
  }
  std::vector<float> mass(static_cast<size_t>(ns) * n), range(static_cast<size_t>(ns) * n);
  CK(c, cudaMemcpy2DAsync(mass.data(), static_cast<size_t>(n) * sizeof(float), L.ema_d,
                          static_cast<size_t>(c->max_blocks + 1) * sizeof(float), static_cast<size_t>(n) * sizeof(float), ns,
                          cudaMemcpyDeviceToHost, st));
  CK(c, cudaMemcpy2DAsync(range.data(), static_cast<size_t>(n) * sizeof(float), L.range_d,
                          static_cast<size_t>(c->max_blocks) * sizeof(float), static_cast<size_t>(n) * sizeof(float), ns,
                          cudaMemcpyDeviceToHost, st));
  CK(c, cudaStreamSynchronize(st));
  *missed = rd_allocate_streams(cfg, mass.data(), range.data(), n, L.n_tail, ns, L.level.data(), c->max_blocks, target, n);
  return GKV_OK;
}
}  // namespace

int gkv_rd_reallocate(gkv_cache* c, int32_t layer, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return GKV_ERR_INVALID_ARG;
  const gkv_config& cfg = c->cfg;
  if (cfg.policy != GKV_POLICY_RD || is_mla(cfg)) return GKV_ERR_BAD_STATE;
  LayerState& L = c->layers[layer];
  const int n = L.n_closed, ns = c->n_streams;
  if (n == 0) return GKV_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  std::vector<int8_t> target(static_cast<size_t>(ns) * n);
  bool missed = false;
  int rc = rd_plan_layer(c, L, target.data(), &missed, st);
  if (rc != GKV_OK) return rc;
  int warn = GKV_OK;
  if (missed) {
    L.budget_flag = true;
    warn = GKV_ERR_BUDGET;
  }
  rc = demote_to_targets(c, L, target.data(), static_cast<size_t>(n), st);
  return rc != GKV_OK ? rc : warn;
}

int gkv_debug_device_plan(gkv_cache* c, int32_t layer, int8_t* levels_out, float* mass_out, float* range_out, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !levels_out) return GKV_ERR_INVALID_ARG;
  const gkv_config& cfg = c->cfg;
  if (cfg.policy != GKV_POLICY_RD || is_mla(cfg)) return GKV_ERR_BAD_STATE;
  LayerState& L = c->layers[layer];
  const int n = L.n_closed, ns = c->n_streams;
  if (n == 0) return GKV_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  bool missed = false;
  const int rc = rd_plan_layer(c, L, levels_out, &missed, st);
  if (rc != GKV_OK) return rc;
  if (mass_out)
    CK(c, cudaMemcpy2D(mass_out, static_cast<size_t>(n) * sizeof(float), L.ema_d, static_cast<size_t>(c->max_blocks + 1) * sizeof(float),
                       static_cast<size_t>(n) * sizeof(float), ns, cudaMemcpyDeviceToHost));
  if (range_out)
    CK(c, cudaMemcpy2D(range_out, static_cast<size_t>(n) * sizeof(float), L.range_d, static_cast<size_t>(c->max_blocks) * sizeof(float),
                       static_cast<size_t>(n) * sizeof(float), ns, cudaMemcpyDeviceToHost));
  return missed ? GKV_ERR_BUDGET : GKV_OK;
}

int gkv_destroy(gkv_cache* c) {
  if (!c) return GKV_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  for (LayerState& L : c->layers) {
    if (L.table_h) cudaFreeHost(L.table_h);
    if (L.warps_h) cudaFreeHost(L.warps_h);
    if (L.units_h) cudaFreeHost(L.units_h);
    if (L.parts_h) cudaFreeHost(L.parts_h);
    if (L.res_off_h) cudaFreeHost(L.res_off_h);
    if (L.res_count_h) cudaFreeHost(L.res_count_h);
    if (L.ev) cudaEventDestroy(L.ev);
    if (L.ev_desc) cudaEventDestroy(L.ev_desc);
  }
  if (c->stage_h) cudaFreeHost(c->stage_h);
  if (c->demote_h) cudaFreeHost(c->demote_h);
  for (cudaEvent_t ev : c->ev_demote)
    if (ev) cudaEventDestroy(ev);
  if (c->ev_stage) cudaEventDestroy(c->ev_stage);
  delete c;
  return GKV_OK;
}

int gkv_ctx_len(gkv_cache* c, int32_t layer, int32_t* ctx) {
  if (!c || !ctx || layer < 0 || layer >= c->cfg.n_layers) return GKV_ERR_INVALID_ARG;
  const LayerState& L = c->layers[layer];
  *ctx = L.n_closed * kBlock + L.n_tail;
  return GKV_OK;
}

namespace {
// The kernels read queries, new rows and index lists and write results with 4- to 16-byte accesses:
// a pointer off its natural boundary is refused here instead of faulting on the device.
inline bool misaligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }
}  // namespace

int gkv_append_demote(gkv_cache* c, int32_t layer, const void* k_new, const void* v_new, int32_t n_new,
                      const float* token_mass, const int8_t* level_plan, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !k_new || n_new <= 0) return GKV_ERR_INVALID_ARG;
  if (is_mla(c->cfg) ? (v_new != nullptr) : (v_new == nullptr)) return GKV_ERR_INVALID_ARG;
  if (misaligned(k_new, 4) || misaligned(v_new, 4) || misaligned(token_mass, 4)) return GKV_ERR_INVALID_ARG;
  LayerState& L = c->layers[layer];
  const int ctx = L.n_closed * kBlock + L.n_tail;
  if (static_cast<long long>(ctx) + n_new > c->cfg.max_ctx) return GKV_ERR_CTX_FULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (is_mla(c->cfg)) {
    if (n_new == 1) return mla_append_one(c, layer, static_cast<const uint16_t*>(k_new), st);
    if (ctx != 0) return GKV_ERR_BAD_STATE;
    if (c->cfg.policy == GKV_POLICY_EXTERNAL && !level_plan && n_new >= kBlock) return GKV_ERR_INVALID_ARG;
    return mla_bulk_ingest(c, layer, static_cast<const uint16_t*>(k_new), n_new, level_plan, st);
  }
  if (n_new == 1) return append_one(c, layer, static_cast<const uint16_t*>(k_new), static_cast<const uint16_t*>(v_new), st);
  if (ctx != 0) return GKV_ERR_BAD_STATE;
  if (c->cfg.policy == GKV_POLICY_RD && !token_mass) return GKV_ERR_INVALID_ARG;
  if (c->cfg.policy == GKV_POLICY_EXTERNAL && !level_plan && n_new >= kBlock) return GKV_ERR_INVALID_ARG;
  return bulk_ingest(c, layer, static_cast<const uint16_t*>(k_new), static_cast<const uint16_t*>(v_new), n_new,
                     token_mass, level_plan, st);
}

namespace {
int decode_impl(gkv_cache* c, int32_t layer, const void* q, const int32_t* page_idx, int32_t n_sel, float* out, float* lse,
                bool observe, float* block_mass, float* certificate, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !q || !out) return GKV_ERR_INVALID_ARG;
  if (!page_idx && n_sel != 0) return GKV_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(out, 16) || misaligned(lse, 4) || misaligned(page_idx, 4) || misaligned(block_mass, 4) ||
      misaligned(certificate, 4))
    return GKV_ERR_INVALID_ARG;
  LayerState& L = c->layers[layer];
  if (L.n_closed * kBlock + L.n_tail == 0) return GKV_ERR_BAD_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const gkv_config& cfg = c->cfg;
  if (is_mla(cfg)) {
    if (page_idx) return GKV_ERR_BAD_STATE;
    if (observe) return GKV_ERR_UNSUPPORTED;
    return mla_decode(c, L, q, out, lse, st);
  }
  DecodeParams p{};
  if (observe) {
    p.mass_raw = c->mass_raw_d;
    p.res_raw = c->res_raw_d;
    p.lse2 = c->lse2_d;
    p.mass_stride = c->max_blocks + 1;
    p.res_cap = c->res_cap;
  }
  p.arena = c->arena;
  p.table = L.table_d;
  p.q = static_cast<const uint16_t*>(q);
  p.partial = c->partial_d;
  p.res_off256 = L.res_off_d;
  p.res_count = L.res_count_d;
  p.table_stride = c->table_stride;
  p.n_closed = L.n_closed;
  p.n_tail = L.n_tail;
  p.n_kv_heads = cfg.n_kv_heads;
  p.group = c->group;
  p.head_groups = c->head_groups;
  p.scale_log2 = c->scale * 1.4426950408889634f;
  p.status = c->status_d;
  p.tickets = c->tickets_d;
  p.out = out;
  p.lse = lse;
  int n_ctas;
  if (page_idx) {
    if (cfg.page_tokens <= 0) return GKV_ERR_BAD_STATE;
    if (n_sel < 0 || n_sel > L.n_closed * (kBlock / cfg.page_tokens)) return GKV_ERR_INVALID_ARG;
    p.page_idx = page_idx;
    p.res_idx = L.res_idx_d;
    p.res_cap = c->res_cap;
    p.n_sel = n_sel;
    p.page_tokens = cfg.page_tokens;
    p.warps_per_stream = sparse_ctas_per_stream(c->n_hgroups) * kDecodeWarps;      // per head group
    p.n_warps = c->n_hgroups * p.warps_per_stream;
    p.warps = nullptr;
    p.parts = nullptr;
    n_ctas = (p.n_warps + kDecodeWarps - 1) / kDecodeWarps;
    L.last_mode = 2;
    L.last_pages = page_idx;
    L.last_n_sel = n_sel;
    L.last_read_scored = L.quest_ran;     // a later read with a list of the caller's own does not inherit it
    L.quest_ran = false;
  } else {
    if (L.desc_dirty || (observe && L.desc_split)) {      // an observing call needs whole-block units
      // the work lists have their own event: waiting for the table's would wait for copies that
      // the append of this very step has just queued, i.e. drain the stream
      int rc = wait_event(c, L.ev_desc);
      if (rc != GKV_OK) return rc;
      build_descs(c, L, !observe);
      if ((rc = upload(c, L.warps_d, L.warps_h, static_cast<size_t>(L.n_warps) * sizeof(WarpDesc), st, L.ev_desc)) != GKV_OK) return rc;
      if ((rc = upload(c, L.units_d, L.units_h, static_cast<size_t>(L.n_units) * sizeof(uint32_t), st, L.ev_desc)) != GKV_OK) return rc;
      if ((rc = upload(c, L.parts_d, L.parts_h, static_cast<size_t>(c->n_hgroups) * sizeof(StreamParts), st, L.ev_desc)) != GKV_OK) return rc;
    }
    p.warps = L.warps_d;
    p.units = L.units_d;
    p.n_warps = L.n_warps;
    p.parts = L.parts_d;
    n_ctas = L.n_warps / kDecodeWarps;
    L.last_mode = 1;
    L.quest_ran = false;
  }
  CK(c, launch_decode(p, n_ctas, st));
  if (observe) {
    MassFinishParams m{};
    m.mass_raw = c->mass_raw_d;
    m.res_raw = c->res_raw_d;
    m.lse2 = c->lse2_d;
    m.res_idx = L.res_idx_d;
    m.res_count = L.res_count_d;
    m.ema = L.ema_d;
    m.observed = block_mass;
    m.n_streams = c->n_streams;
    m.n_items = L.n_closed + (L.n_tail > 0 ? 1 : 0);
    m.mass_stride = c->max_blocks + 1;
    m.res_cap = c->res_cap;
    m.group = c->group;
    CK(c, launch_mass_finish(m, st));
    if (certificate) {
      CertificateParams cp{};
      cp.arena = c->arena;
      cp.table = L.table_d;
      cp.mass_raw = c->mass_raw_d;
      cp.res_raw = c->res_raw_d;
      cp.lse2 = c->lse2_d;
      cp.err = L.err_d;
      cp.res_count = L.res_count_d;
      cp.q = static_cast<const uint16_t*>(q);
      cp.out = certificate;
      cp.n_streams = c->n_streams;
      cp.group = c->group;
      cp.n_closed = L.n_closed;
      cp.n_tail = L.n_tail;
      cp.table_stride = c->table_stride;
      cp.mass_stride = c->max_blocks + 1;
      cp.res_cap = c->res_cap;
      cp.err_stride = c->max_blocks;
      cp.scale = c->scale;
      CK(c, launch_certificate(cp, st));
    }
  }
  return GKV_OK;
}
}  // namespace

int gkv_decode_attn(gkv_cache* c, int32_t layer, const void* q, const int32_t* page_idx, int32_t n_sel,
                    float* out, float* lse, void* stream) {
  return decode_impl(c, layer, q, page_idx, n_sel, out, lse, false, nullptr, nullptr, stream);
}

int gkv_decode_attn_observe(gkv_cache* c, int32_t layer, const void* q, float* out, float* lse, float* block_mass,
                            float* certificate, void* stream) {
  return decode_impl(c, layer, q, nullptr, 0, out, lse, true, block_mass, certificate, stream);
}

int gkv_debug_export_bounds(gkv_cache* c, int32_t layer, float* bounds_out) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !bounds_out) return GKV_ERR_INVALID_ARG;
  if (is_mla(c->cfg)) return GKV_ERR_UNSUPPORTED;
  LayerState& L = c->layers[layer];
  CK(c, cudaDeviceSynchronize());
  if (L.n_closed == 0) return GKV_OK;
  CK(c, cudaMemcpy2D(bounds_out, static_cast<size_t>(L.n_closed) * sizeof(float4), L.err_d,
                     static_cast<size_t>(c->max_blocks) * sizeof(float4), static_cast<size_t>(L.n_closed) * sizeof(float4),
                     c->n_streams, cudaMemcpyDeviceToHost));
  return GKV_OK;
}

int gkv_debug_export_mass(gkv_cache* c, int32_t layer, float* mass_out) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !mass_out) return GKV_ERR_INVALID_ARG;
  if (is_mla(c->cfg)) return GKV_ERR_UNSUPPORTED;
  LayerState& L = c->layers[layer];
  CK(c, cudaDeviceSynchronize());
  const int n_items = L.n_closed + (L.n_tail > 0 ? 1 : 0);
  if (n_items == 0) return GKV_OK;
  CK(c, cudaMemcpy2D(mass_out, static_cast<size_t>(n_items) * sizeof(float), L.ema_d,
                     static_cast<size_t>(c->max_blocks + 1) * sizeof(float), static_cast<size_t>(n_items) * sizeof(float),
                     c->n_streams, cudaMemcpyDeviceToHost));
  return GKV_OK;
}

int gkv_quest_select(gkv_cache* c, int32_t layer, const void* q, int32_t budget_tokens, int32_t* page_idx_out,
                     int32_t* n_sel_out, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !q || !page_idx_out || !n_sel_out || budget_tokens < 0)
    return GKV_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(page_idx_out, 4)) return GKV_ERR_INVALID_ARG;
  const gkv_config& cfg = c->cfg;
  if (cfg.page_tokens <= 0) return GKV_ERR_BAD_STATE;
  LayerState& L = c->layers[layer];
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n_pages = L.n_closed * (kBlock / cfg.page_tokens);
  const int k = std::min(budget_tokens / cfg.page_tokens, n_pages);
  *n_sel_out = k;
  L.quest_ran = true;
  if (k <= 0) return GKV_OK;
  CK(c, launch_quest_scores(L.boxes_d, c->box_stride, n_pages, static_cast<const uint16_t*>(q), c->n_streams,
                            cfg.n_kv_heads, c->group, cfg.quest_reduce, c->scores_d, c->box_stride, st));
  CK(c, launch_topk(c->scores_d, c->box_stride, n_pages, nullptr, k, page_idx_out, k, c->n_streams, st));
  return GKV_OK;
}

int gkv_debug_export_boxes(gkv_cache* c, int32_t layer, int32_t b, int32_t kv_head, uint16_t* lo, uint16_t* hi,
                           int32_t cap_pages, int32_t* n_pages) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !lo || !hi || !n_pages) return GKV_ERR_INVALID_ARG;
  const gkv_config& cfg = c->cfg;
  if (b < 0 || b >= cfg.batch || kv_head < 0 || kv_head >= cfg.n_kv_heads) return GKV_ERR_INVALID_ARG;
  if (cfg.page_tokens <= 0) return GKV_ERR_BAD_STATE;
  LayerState& L = c->layers[layer];
  const int np = L.n_closed * (kBlock / cfg.page_tokens);
  *n_pages = np;
  if (np > cap_pages) return GKV_ERR_INVALID_ARG;
  if (np == 0) return GKV_OK;
  CK(c, cudaDeviceSynchronize());
  // device layout [stream][channel][min | max][page] -> [page][channel]
  std::vector<uint16_t> raw(static_cast<size_t>(kD) * 2 * c->box_stride);
  const int stream = b * cfg.n_kv_heads + kv_head;
  CK(c, cudaMemcpy(raw.data(), L.boxes_d + static_cast<size_t>(stream) * kD * 2 * c->box_stride, raw.size() * sizeof(uint16_t),
                   cudaMemcpyDeviceToHost));
  for (int pg = 0; pg < np; ++pg)
    for (int ch = 0; ch < kD; ++ch) {
      lo[static_cast<size_t>(pg) * kD + ch] = raw[(static_cast<size_t>(ch) * 2) * c->box_stride + pg];
      hi[static_cast<size_t>(pg) * kD + ch] = raw[(static_cast<size_t>(ch) * 2 + 1) * c->box_stride + pg];
    }
  return GKV_OK;
}

int gkv_debug_export_scores(gkv_cache* c, int32_t layer, const void* q, float* scores, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !q || !scores || misaligned(q, 16)) return GKV_ERR_INVALID_ARG;
  const gkv_config& cfg = c->cfg;
  if (cfg.page_tokens <= 0) return GKV_ERR_BAD_STATE;
  LayerState& L = c->layers[layer];
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int np = L.n_closed * (kBlock / cfg.page_tokens);
  if (np == 0) return GKV_OK;
  CK(c, launch_quest_scores(L.boxes_d, c->box_stride, np, static_cast<const uint16_t*>(q), c->n_streams, cfg.n_kv_heads, c->group,
                            cfg.quest_reduce, c->scores_d, c->box_stride, st));
  CK(c, cudaStreamSynchronize(st));
  CK(c, cudaMemcpy2D(scores, static_cast<size_t>(np) * sizeof(float), c->scores_d, static_cast<size_t>(c->box_stride) * sizeof(float),
                     static_cast<size_t>(np) * sizeof(float), c->n_streams, cudaMemcpyDeviceToHost));
  return GKV_OK;
}

int gkv_quest_select_static(gkv_cache* c, int32_t layer, const void* q, int32_t budget_tokens,
                            int32_t* page_idx_out, int32_t* n_sel_out, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !q || !page_idx_out || !n_sel_out || budget_tokens < 0)
    return GKV_ERR_INVALID_ARG;
  if (misaligned(q, 16) || misaligned(page_idx_out, 4)) return GKV_ERR_INVALID_ARG;
  const gkv_config& cfg = c->cfg;
  if (cfg.page_tokens <= 0) return GKV_ERR_BAD_STATE;
  LayerState& L = c->layers[layer];
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n_pages = L.n_closed * (kBlock / cfg.page_tokens);
  // the scores of all streams must fit the fixed scratch: n_streams * stride floats
  const size_t stride = align_up(static_cast<size_t>(std::max(n_pages, 1)), 8);
  if (stride * static_cast<size_t>(c->n_streams) > kStaticScoreFloats) return GKV_ERR_UNSUPPORTED;
  float* scores = nullptr;
  int rc = static_scores_address(c, &scores);
  if (rc != GKV_OK) return rc;
  const int k = std::min(budget_tokens / cfg.page_tokens, n_pages);
  *n_sel_out = k;
  L.quest_ran = true;
  if (k <= 0) return GKV_OK;
  // every score in [0, n_pages) of every stream is rewritten by the scorer before the selection
  // reads it, so nothing left over from an earlier call is ever looked at
  CK(c, launch_quest_scores(L.boxes_d, c->box_stride, n_pages, static_cast<const uint16_t*>(q), c->n_streams,
                            cfg.n_kv_heads, c->group, cfg.quest_reduce, scores, static_cast<int>(stride), st));
  CK(c, launch_topk(scores, static_cast<int>(stride), n_pages, nullptr, k, page_idx_out, k, c->n_streams, st));
  return GKV_OK;
}

int gkv_bits_report(gkv_cache* c, int32_t layer, gkv_bits* out) {
  if (!c || !out || layer < -1 || layer >= c->cfg.n_layers) return GKV_ERR_INVALID_ARG;
  std::memset(out, 0, sizeof(*out));
  const gkv_config& cfg = c->cfg;
  const uint64_t nval_tok = nval_per_token(cfg);
  const int l0 = layer < 0 ? 0 : layer, l1 = layer < 0 ? cfg.n_layers : layer + 1;
  int warn = GKV_OK;
  for (int l = l0; l < l1; ++l) {
    LayerState& L = c->layers[l];
    const int ctx = L.n_closed * kBlock + L.n_tail;
    for (int s = 0; s < c->n_streams; ++s) {
      out->values += static_cast<uint64_t>(ctx) * nval_tok;
      for (int b = 0; b < L.n_closed; ++b) {
        const int lv = L.level[static_cast<size_t>(s) * c->max_blocks + b];
        out->blocks_by_level[level_index(lv)] += 1;
        if (lv == 16) out->exact_bits += 16ull * kBlock * nval_tok;
        else if (lv == 1) out->centroid_bits += 16ull * nval_tok;
        else {
          out->code_bits += static_cast<uint64_t>(lv) * kBlock * nval_tok;
          out->param_bits += (kBlock * nval_tok / kGroup) * 32ull;
        }
      }
      out->tail_bits += static_cast<uint64_t>(L.n_tail) * 16 * nval_tok;
      out->residual_bits += static_cast<uint64_t>(L.res_count_h[s]) * 16 * nval_tok;
      out->residual_index_bits += static_cast<uint64_t>(L.res_count_h[s]) * 32;
      if (cfg.page_tokens > 0) out->box_bits += static_cast<uint64_t>(L.n_closed) * (kBlock / cfg.page_tokens) * 2 * cfg.d_k * 16;
      out->meta_bits += static_cast<uint64_t>(L.n_closed + 1) * sizeof(TableEntry) * 8;
    }
    out->meta_bits += static_cast<uint64_t>(L.n_warps) * sizeof(WarpDesc) * 8 + static_cast<uint64_t>(L.n_units) * 32;
    if (L.last_mode == 1) out->last_read_bits += full_read_bits(c, L);
    if (L.last_mode == 2) {
      // fetch the page list that was used and count what it touched
      std::vector<int32_t> pages(static_cast<size_t>(c->n_streams) * std::max(L.last_n_sel, 1));
      if (L.last_n_sel > 0) {
        cudaError_t e = cudaMemcpy(pages.data(), L.last_pages, static_cast<size_t>(c->n_streams) * L.last_n_sel * sizeof(int32_t), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return cuda_fail(c, e);
      }
      const int page = cfg.page_tokens, ppb = kBlock / page;
      for (int s = 0; s < c->n_streams; ++s) {
        std::vector<char> group_seen(static_cast<size_t>(L.n_closed) * 2, 0), cent_seen(L.n_closed, 0);
        for (int i = 0; i < L.last_n_sel; ++i) {
          const int pg = pages[static_cast<size_t>(s) * L.last_n_sel + i];
          if (pg < 0 || pg >= L.n_closed * ppb) return GKV_ERR_BAD_STATE;
          const int blk = pg / ppb;
          const int lv = L.level[static_cast<size_t>(s) * c->max_blocks + blk];
          if (lv == 16) out->last_read_bits += static_cast<uint64_t>(page) * 16 * nval_tok;
          else if (lv == 1) cent_seen[blk] = 1;
          else {
            out->last_read_bits += static_cast<uint64_t>(page) * nval_tok * lv;
            out->last_read_bits += static_cast<uint64_t>(page) * (cfg.d_v / kGroup) * 32;
            for (int t0 = pg * page; t0 < (pg + 1) * page; t0 += kGroup) group_seen[t0 / kGroup] = 1;
          }
        }
        for (char g : group_seen) if (g) out->last_read_bits += static_cast<uint64_t>(cfg.d_k) * 32;
        for (char g : cent_seen) if (g) out->last_read_bits += 16ull * nval_tok;
        // exact residual rows are read where the page of their token is listed
        if (!L.res_idx.empty() && !L.res_idx[s].empty()) {
          const int32_t* lb = pages.data() + static_cast<size_t>(s) * L.last_n_sel;
          for (int32_t tok : L.res_idx[s])
            if (std::binary_search(lb, lb + L.last_n_sel, tok / page)) out->last_read_bits += 16ull * nval_tok;
        }
        out->last_read_bits += static_cast<uint64_t>(L.n_tail) * 16 * nval_tok;
      }
    }
    if (L.last_read_scored && L.last_mode == 2)
      out->last_read_bits += static_cast<uint64_t>(c->n_streams) * L.n_closed * (kBlock / cfg.page_tokens) * 2 * cfg.d_k * 16;
    if (L.budget_flag) warn = GKV_ERR_BUDGET;
  }
  out->resident_bits = out->code_bits + out->param_bits + out->exact_bits + out->centroid_bits + out->tail_bits +
                       out->residual_bits + out->residual_index_bits + out->box_bits;
  const double v = static_cast<double>(std::max<uint64_t>(out->values, 1));
  out->bpv_resident = static_cast<double>(out->resident_bits) / v;
  out->bpv_paper = static_cast<double>(out->resident_bits - out->residual_index_bits) / v;
  out->bpv_read = static_cast<double>(out->last_read_bits) / v;
  // device-detected conditions surface here (this call may synchronise)
  uint32_t status = 0;
  cudaError_t e = cudaMemcpy(&status, c->status_d, sizeof(status), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(c, e);
  if (status & kStatusInternal) return GKV_ERR_BAD_STATE;
  if (status & kStatusRange) warn = GKV_ERR_RANGE;
  return warn;
}

int gkv_debug_export_levels(gkv_cache* c, int32_t layer, int32_t b, int32_t kv_head, int8_t* levels, int32_t cap,
                            int32_t* n) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || b < 0 || b >= c->cfg.batch || kv_head < 0 ||
      kv_head >= c->cfg.n_kv_heads || !levels || !n)
    return GKV_ERR_INVALID_ARG;
  const LayerState& L = c->layers[layer];
  const int s = b * c->cfg.n_kv_heads + kv_head;
  *n = L.n_closed;
  for (int i = 0; i < std::min(cap, L.n_closed); ++i) levels[i] = L.level[static_cast<size_t>(s) * c->max_blocks + i];
  return GKV_OK;
}

int gkv_debug_export_residual(gkv_cache* c, int32_t layer, int32_t b, int32_t kv_head, int32_t* idx, int32_t cap,
                              int32_t* n) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || b < 0 || b >= c->cfg.batch || kv_head < 0 ||
      kv_head >= c->cfg.n_kv_heads || !idx || !n)
    return GKV_ERR_INVALID_ARG;
  const LayerState& L = c->layers[layer];
  const int s = b * c->cfg.n_kv_heads + kv_head;
  *n = static_cast<int32_t>(L.res_idx[s].size());
  for (int i = 0; i < std::min<int>(cap, *n); ++i) idx[i] = L.res_idx[s][i];
  return GKV_OK;
}

int gkv_debug_export_block(gkv_cache* c, int32_t layer, int32_t b, int32_t kv_head, int32_t block, int32_t which,
                           int32_t* level, uint8_t* codes, uint16_t* scale_fp16, uint16_t* zero_fp16,
                           uint16_t* rows_bf16, int32_t* n_rows) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || b < 0 || b >= c->cfg.batch || kv_head < 0 ||
      kv_head >= c->cfg.n_kv_heads || (which != GKV_TENSOR_K && which != GKV_TENSOR_V))
    return GKV_ERR_INVALID_ARG;
  LayerState& L = c->layers[layer];
  if (block < 0 || block > L.n_closed || (block == L.n_closed && !L.has_tail_slot)) return GKV_ERR_INVALID_ARG;
  const int s = b * c->cfg.n_kv_heads + kv_head;
  const TableEntry& e = L.table_h[static_cast<size_t>(s) * c->table_stride + block];
  const int lv = block == L.n_closed ? 16 : static_cast<int>(e.level);
  if (level) *level = lv;
  if (n_rows) *n_rows = block == L.n_closed ? L.n_tail : (lv == 1 ? 1 : kBlock);
  CK(c, cudaDeviceSynchronize());
  if (is_mla(c->cfg)) {
    if (which != GKV_TENSOR_K) return GKV_ERR_INVALID_ARG;     // values are channels [0, 512) of the key row
    uint8_t* m_codes = c->debug_d;
    uint16_t* m_scale = reinterpret_cast<uint16_t*>(c->debug_d + kBlock * kMlaDk);
    uint16_t* m_zero = reinterpret_cast<uint16_t*>(c->debug_d + kBlock * kMlaDk + 4096);
    uint16_t* m_rows = reinterpret_cast<uint16_t*>(c->debug_d + kBlock * kMlaDk + 8192);
    CK(c, launch_mla_export(c->arena, e.off256, lv, m_codes, m_scale, m_zero, m_rows, 0));
    CK(c, cudaDeviceSynchronize());
    if (lv == 16) {
      if (rows_bf16) CK(c, cudaMemcpy(rows_bf16, m_rows, kBlock * kMlaDk * 2, cudaMemcpyDeviceToHost));
    } else if (lv == 1) {
      if (rows_bf16) CK(c, cudaMemcpy(rows_bf16, m_rows, kMlaDk * 2, cudaMemcpyDeviceToHost));
    } else {
      if (codes) CK(c, cudaMemcpy(codes, m_codes, kBlock * kMlaDk, cudaMemcpyDeviceToHost));
      if (scale_fp16) CK(c, cudaMemcpy(scale_fp16, m_scale, 2 * kMlaDk * 2, cudaMemcpyDeviceToHost));
      if (zero_fp16) CK(c, cudaMemcpy(zero_fp16, m_zero, 2 * kMlaDk * 2, cudaMemcpyDeviceToHost));
    }
    return GKV_OK;
  }
  uint8_t* d_codes = c->debug_d;
  uint16_t* d_scale = reinterpret_cast<uint16_t*>(c->debug_d + kBlock * kD);
  uint16_t* d_zero = reinterpret_cast<uint16_t*>(c->debug_d + kBlock * kD + 1024);
  uint16_t* d_rows = reinterpret_cast<uint16_t*>(c->debug_d + kBlock * kD + 2048);
  CK(c, launch_export_block(c->arena, e.off256, lv, which, d_codes, d_scale, d_zero, d_rows, 0));
  CK(c, cudaDeviceSynchronize());
  if (lv == 16) {
    if (rows_bf16) CK(c, cudaMemcpy(rows_bf16, d_rows, kBlock * kD * 2, cudaMemcpyDeviceToHost));
  } else if (lv == 1) {
    if (rows_bf16) CK(c, cudaMemcpy(rows_bf16, d_rows, kD * 2, cudaMemcpyDeviceToHost));
  } else {
    const size_t np = which == GKV_TENSOR_K ? 2 * kD : kBlock * (kD / kGroup);
    if (codes) CK(c, cudaMemcpy(codes, d_codes, kBlock * kD, cudaMemcpyDeviceToHost));
    if (scale_fp16) CK(c, cudaMemcpy(scale_fp16, d_scale, np * 2, cudaMemcpyDeviceToHost));
    if (zero_fp16) CK(c, cudaMemcpy(zero_fp16, d_zero, np * 2, cudaMemcpyDeviceToHost));
  }
  return GKV_OK;
}

}  // extern "C"
