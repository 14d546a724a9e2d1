// Structures shared by the host library (gkv_api.cu) and the kernels, and the launch
// prototypes of every kernel file.  Nothing here is part of the public ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gkv_layout.cuh"

namespace gkv {

// One entry of a stream's block table (device + pinned host mirror).  Index i < n_closed is a
// closed block, index n_closed is the tail block (level 16, partially filled).
struct alignas(16) TableEntry {
  uint32_t off256;   // slot offset from the arena base in 256-byte units
  uint32_t level;    // 16, 8, 4, 2, 1
  uint64_t resmask;  // bit t set: token t of the block is served from the residual pool instead
};

// Work of one warp of the decode kernel: positions [item_begin, item_end) of the layer's unit
// list, all of one stream; `stream` is the index of the warp's head group (up to four query heads of
// one KV head): stream * head_groups + group number.  A unit is one item or a run of consecutive centroid blocks:
// `first item | run << 24`.  Items: [0, n_closed) closed blocks, n_closed = tail block,
// n_closed + 1 + j = residual group j (16 residual rows each).  (The MLA kernel uses the same
// struct per CTA with item_begin / item_end as a plain item range.)
struct alignas(16) WarpDesc {
  int32_t stream;      // -1 = idle warp
  int32_t item_begin;
  int32_t item_end;
  int32_t partial;     // row of the partial buffer this warp writes
};

// Unit word of the dense work lists: first item | tile mask << 20 | run length << 24.  The tile
// mask (four 16-token tiles; 15 = the whole block) lets a unit cover part of a block: any tiles of an
// exact block, one half (3 or 12) of a quantised one.
constexpr uint32_t kUnitItemMask = 0xfffffu;

struct alignas(8) StreamParts {
  int32_t begin, end;  // partial rows [begin, end) belong to this head group (GQA) / stream (MLA)
};

constexpr int kDecodeWarps = 16;            // warps per CTA of the decode kernel
constexpr int kStageBytes = 5120;           // per-warp pipeline stage
constexpr int kStages = 2;
constexpr int kDecodeCtasPerSm = 1;
constexpr int kMaxHeadsPerKv = 8;           // query heads per KV head
constexpr int kHeadsPerWarp = 4;            // a warp's head group: the n = 8 tensor-core dimension holds (hi, lo) column pairs
constexpr int kPartialFloats = kHeadsPerWarp * (kD + 2);    // per partial row: m, l, o[128] per head

struct DecodeParams {
  const uint8_t* arena;
  const TableEntry* table;      // [n_streams][table_stride]
  const WarpDesc* warps;        // [n_warps]
  const uint32_t* units;        // the layer's unit list (dense mode)
  const uint16_t* q;            // bf16 [batch][n_q_heads][128]
  float* partial;               // [n_partials][kPartialFloats]
  const uint32_t* res_off256;   // [n_streams] residual pool offset (rows of 512 B: K row | V row)
  const int32_t* res_count;     // [n_streams]
  int32_t table_stride;
  int32_t n_warps;
  int32_t n_closed, n_tail;
  int32_t n_kv_heads, group;    // group = query heads per KV head
  int32_t head_groups;          // head groups per KV head: ceil(group / kHeadsPerWarp)
  float scale_log2;             // softmax scale * log2(e)
  // sparse (page list) mode
  const int32_t* page_idx;      // [n_streams][n_sel] or nullptr
  int32_t n_sel, page_tokens, warps_per_stream;
  const int32_t* res_idx;       // sparse mode: [n_streams][res_cap] ascending token indices of the residual rows
  uint32_t* status;             // device status word (bit flags)
  // final merge: the CTA that completes a stream's last partial row normalises and writes it
  const StreamParts* parts;     // [head groups]; nullptr in sparse mode (rows of a head group = its CTAs)
  int32_t* tickets;             // [head groups] arrival counters, zero between launches
  float* out;                   // [batch][n_q_heads][128]
  float* lse;                   // nullable
  // Block attention mass (Sec. 3.1), dense mode, nullable: unnormalised (running max, sum of exp2)
  // pairs per (stream, item, head), items = blocks 0 .. n_closed (the last is the partial block), and
  // per (stream, residual row, head); lse2 = log2 of the softmax denominator per query head.
  float2* mass_raw;             // [n_streams][mass_stride][8]
  float2* res_raw;              // [n_streams][res_cap][8]
  float* lse2;                  // [batch][n_q_heads]
  int32_t mass_stride, res_cap;
};

// Attention error certificate of the observing decode launch that just ran (Sec. 3.6, Eq. 9).
struct CertificateParams {
  const uint8_t* arena;
  const TableEntry* table;
  const float2* mass_raw;
  const float2* res_raw;
  const float* lse2;
  const float4* err;            // [n_streams][err_stride]
  const int32_t* res_count;
  const uint16_t* q;            // bf16 [batch][n_q_heads][128]
  float* out;                   // [batch][n_q_heads]
  int32_t n_streams, group, n_closed, n_tail;
  int32_t table_stride, mass_stride, res_cap, err_stride;
  float scale;                  // softmax scale (natural-log domain)
};

// Turns the raw pairs of a decode launch into block masses a_b (mean over the KV head's query heads
// of the block's softmax weight, residual rows added to the block they sit in) and updates the running
// mass m_b <- 0.9 m_b + 0.1 a_b.
struct MassFinishParams {
  const float2* mass_raw;
  const float2* res_raw;
  const float* lse2;
  const int32_t* res_idx;       // [n_streams][res_cap] ascending token indices of the residual rows
  const int32_t* res_count;     // [n_streams]
  float* ema;                   // [n_streams][mass_stride]
  float* observed;              // nullable [n_streams][n_items]
  int32_t n_streams, n_items;   // items = n_closed + (n_tail > 0)
  int32_t mass_stride, res_cap, group;
};

// One block to encode: read 64 tokens from `src`, write level `dst_level` at dst.
struct alignas(16) EncodeJob {
  uint32_t src_off256;   // source slot (when src_level != 0)
  uint32_t dst_off256;
  int16_t src_level;     // 0 = bf16 input rows (bulk ingest); else level of the source slot
  int16_t dst_level;
  int32_t stream;        // for src_level == 0: which (b, kv head); token base = block * 64
  int32_t block;
  int32_t pad;
};

struct EncodeParams {
  uint8_t* arena;
  const EncodeJob* jobs;
  int32_t n_jobs;
  const uint16_t* k_in;   // bf16 [batch][n_tok][n_kv_heads][128] (src_level == 0)
  const uint16_t* v_in;
  int32_t n_tok, n_kv_heads;
  uint32_t* status;
  // Error bounds for the certificate (Sec. 3.6), nullable: per (stream, block) x = bound on
  // max_j |k_j - k^_j|, y = the same for values, z = max_j |v_j| of the original rows.
  float4* err;            // [n_streams][err_stride]
  int32_t err_stride;
  // Decode-time demotions: the kernel also points the block table at the new slot (nullable;
  // offset and level of entry [stream][block], the residual mask stays).
  TableEntry* table;
  int32_t table_stride;
  // Bulk ingest without a job list (jobs == nullptr): work item i is block (i / n_kv_heads) % n_blocks of
  // KV head i % n_kv_heads of sequence first_seq + i / (n_blocks * n_kv_heads); its slot and level are read
  // from the table (which is not written).
  int32_t n_blocks, first_seq;
};

// Statistics of freshly closed blocks: page boxes, key range proxy, block mass.
struct StatsParams {
  uint8_t* arena;
  const uint16_t* k_in;        // bf16 input rows, or nullptr to read the block's exact slot
  const float* token_mass;     // [n_streams][n_tok] or nullptr
  const TableEntry* table;
  int32_t table_stride;
  int32_t n_tok, n_kv_heads;
  int32_t first_block, n_blocks;     // blocks [first_block, first_block + n_blocks) of every stream
  int32_t n_streams;
  int32_t page_tokens;               // 0 = no boxes
  uint16_t* boxes;                   // [n_streams][128][2][box_stride] bf16
  int32_t box_stride;                // pages (padded)
  float* block_range;                // [n_streams][n_blocks] or nullptr
  float* block_mass;                 // [n_streams][n_blocks] or nullptr
  int32_t stat_stride, stat_base;    // range / mass land at [stream * stat_stride + stat_base + i]; stride 0 = n_blocks
  float4* err;                       // nullable; with k_in == nullptr: (0, 0, max_j |v_j|, 0) of the block's exact rows
  int32_t err_stride;
};

constexpr uint32_t kStatusRange = 1u;      // a scale or zero saturated
constexpr uint32_t kStatusInternal = 2u;   // an index check failed inside a kernel

cudaError_t launch_decode(const DecodeParams& p, int n_ctas, cudaStream_t st);
cudaError_t launch_mass_finish(const MassFinishParams& p, cudaStream_t st);
cudaError_t launch_certificate(const CertificateParams& p, cudaStream_t st);
cudaError_t launch_encode(const EncodeParams& p, cudaStream_t st);
cudaError_t launch_ingest(const EncodeParams& p, cudaStream_t st);   // every job reads the bf16 input rows; 16-byte aligned inputs
cudaError_t launch_stats(const StatsParams& p, cudaStream_t st);

// RD allocator on the device (Sec. 3.3; gkv_rdplan.cu): one level plan per stream from block masses
// and range proxies, identical to the host allocator's on the same numbers.
struct RdPlanParams {
  const float* mass;            // [n_streams][mass_stride] running block mass m_b
  const float* range;           // [n_streams][range_stride] range proxy e_b
  const TableEntry* table;      // [n_streams][table_stride]: the blocks' present levels
  int8_t* levels_out;           // [n_streams][out_stride]
  uint32_t* miss_flag;          // set to 1 when a stream cannot meet the budget (its plan is still written)
  int32_t n, mass_stride, range_stride, table_stride, out_stride;
  int32_t m_pad;                // power of two >= 4 n + 1 (rd_plan_smem_bytes)
  int32_t n_sink_blocks, retire_after, monotone, use_prev;
  unsigned long long nval_tok, budget_bits, tail_bits;
};
size_t rd_plan_smem_bytes(int n, int* m_pad_out);
cudaError_t launch_rd_plan(const RdPlanParams& p, int n_streams, cudaStream_t st);
cudaError_t launch_append_rows(uint8_t* arena, const TableEntry* table, int table_stride, int tail_index,
                               int n_streams, int n_kv_heads, const uint16_t* k_in, const uint16_t* v_in,
                               int n_tok, int first_tok, int n_rows, int dst_row0, cudaStream_t st);
cudaError_t launch_residual_scores(const uint16_t* v_in, const float* token_mass, const int8_t* levels,
                                   int levels_stride, int n_sink_blocks, int n_streams, int n_kv_heads, int n_tok,
                                   int n_closed, float* scores, cudaStream_t st);
cudaError_t launch_topk(const float* scores, int score_stride, int n, const int32_t* k_per_stream, int k_uniform,
                        int32_t* idx_out, int idx_stride, int n_streams, cudaStream_t st);
cudaError_t launch_residual_gather(uint8_t* arena, const uint16_t* k_in, const uint16_t* v_in, int n_tok,
                                   int n_kv_heads, const int32_t* idx, int idx_stride, const int32_t* count,
                                   const uint32_t* res_off256, int max_count, int n_streams, cudaStream_t st);
cudaError_t launch_quest_scores(const uint16_t* boxes, int box_stride, int n_pages, const uint16_t* q,
                                int n_streams, int n_kv_heads, int group, int reduce, float* scores,
                                int score_stride, cudaStream_t st);
cudaError_t launch_export_block(const uint8_t* arena, uint32_t off256, int level, int which, uint8_t* codes,
                                uint16_t* scale, uint16_t* zero, uint16_t* rows, cudaStream_t st);
size_t decode_smem_bytes();

}  // namespace gkv
