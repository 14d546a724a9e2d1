/*
 * gkv.h - C ABI of the graded KV-cache decode-attention library (Geodesia-KV hot path).
 *
 * One cache object holds, for every (layer, sequence, KV head) "stream", a sequence of
 * 64-token blocks, each on one rung of the precision ladder {16, 8, 4, 2, centroid}
 * (paper Sec. 3.2), an always-exact partial tail block, optional exact residual tokens
 * (Sec. 3.4) and optional exact per-page key min/max boxes (Sec. 3.5).  All compute runs
 * in CUDA kernels for sm_100a; there is no CPU fallback.
 *
 * Conventions
 *  - "device" pointers are CUDA device memory owned by the caller; "host" pointers are
 *    ordinary host memory.  The library never allocates device memory: everything it
 *    keeps on the device lives in the caller's arena.
 *  - `stream` is a cudaStream_t passed as void*.  All calls on one cache must be issued
 *    in order on one stream (or externally ordered).  Calls are asynchronous unless the
 *    function's comment says it synchronises.
 *  - Every function returns 0 (GKV_OK) or a negative gkv_status.  Arguments are validated
 *    on the host before anything is launched; nothing traps or asserts on the device.
 *  - bf16 / fp16 data are raw 16-bit patterns.  Values must be finite and, for blocks
 *    below level 16 and for queries, within +-65504 (fp16 range).
 *  - Alignment of device buffers: queries and attention outputs 16 bytes; new key / value
 *    rows 4 bytes (16 bytes lets a bulk ingest take the fast encoder; other rows are
 *    encoded by the general one, with the same bits); float and int32 arrays 4 bytes.
 *    A pointer off these boundaries is refused with GKV_ERR_INVALID_ARG.
 */
#ifndef GKV_H_
#define GKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GKV_ABI_VERSION 1u
#if defined(__GNUC__)
#define GKV_API __attribute__((visibility("default")))
#else
#define GKV_API
#endif

typedef enum gkv_status {
  GKV_OK = 0,
  GKV_ERR_INVALID_ARG = -1,     /* null pointer, bad shape, bad index */
  GKV_ERR_ARENA_TOO_SMALL = -2, /* arena cannot hold the metadata or a needed block slot */
  GKV_ERR_CTX_FULL = -3,        /* append would exceed max_ctx */
  GKV_ERR_BAD_STATE = -4,       /* e.g. page selection without page_tokens, ingest on a non-empty stream */
  GKV_ERR_UNSUPPORTED = -5,     /* shape or combination not compiled */
  GKV_ERR_RANGE = -6,           /* a scale/zero saturated at +-65504, or a value scale exceeds what the read path
                                   takes (4094); result stored, flag returned */
  GKV_ERR_BUDGET = -7,          /* RD budget unreachable even with every free block at centroid (plan applied) */
  GKV_ERR_CUDA = -8             /* CUDA runtime error; see gkv_last_cuda_error */
} gkv_status;

enum { GKV_POLICY_STAIRCASE = 0, GKV_POLICY_RD = 1, GKV_POLICY_EXTERNAL = 2 };
enum { GKV_REDUCE_MAX = 0, GKV_REDUCE_SUM = 1 };
enum { GKV_TENSOR_K = 0, GKV_TENSOR_V = 1 };

typedef struct gkv_cache gkv_cache; /* opaque; host object owned by the library */

/* Shape and policy of a cache.  Zero-initialise, then set struct_size / abi_version. */
typedef struct gkv_config {
  uint32_t struct_size;  /* sizeof(gkv_config) */
  uint32_t abi_version;  /* GKV_ABI_VERSION */
  int32_t n_layers, batch, n_q_heads, n_kv_heads; /* n_q_heads % n_kv_heads == 0 */
  int32_t d_k, d_v;      /* head dims: 128 / 128, or 576 / 512 with v_aliases_k */
  int32_t v_aliases_k;   /* 1: values are channels [0, d_v) of the key row (latent attention) */
  int32_t max_ctx;       /* capacity in tokens per sequence */
  int32_t block_tokens;  /* 64 (Sec. 3.2) */
  int32_t group;         /* 32: keys 32 tokens x 1 channel, values 1 token x 32 channels */
  int32_t page_tokens;   /* 0 = no page scorer; else 16, 32 or 64 (Sec. 3.5) */
  int32_t policy;        /* GKV_POLICY_* */
  int32_t stair_tokens[4]; /* STAIRCASE: widths in tokens of the 16/8/4/2 rungs, newest first;
                              -1 = unbounded; older blocks are centroid */
  int32_t n_sink_blocks; /* oldest blocks kept at 16 bits (Fig. 1) */
  int32_t retire_after;  /* RD: newest retire_after tokens' blocks stay at 16 bits (Sec. 3.2) */
  float rd_budget_bpv;   /* RD: bits/value incl. scales over all ingested tokens (Eq. 4) */
  float residual_fraction; /* exact residual tokens per stream = floor(fraction * ctx) (Sec. 3.4) */
  int32_t quest_reduce;  /* GKV_REDUCE_*: page score over the query heads of a KV head */
  int32_t monotone_in_age; /* RD: 1 = levels never rise toward older blocks */
  float softmax_scale;   /* 0 -> 1/sqrt(d_k) */
} gkv_config;

/* Exact integer accounting of resident and read bits (Sec. 3.5 Eq. 7-8, Sec. 4.4). */
typedef struct gkv_bits {
  uint64_t values;        /* K and V values addressed: ctx * (d_k + d_v) per stream, summed */
  uint64_t code_bits, param_bits, exact_bits, centroid_bits, tail_bits;
  uint64_t residual_bits, residual_index_bits, box_bits;
  uint64_t resident_bits; /* sum of the eight categories above */
  uint64_t meta_bits;     /* block table, residual masks, work descriptors (not in resident_bits) */
  uint64_t last_read_bits;/* graded bits touched by the last gkv_decode_attn, plus all boxes if a
                             gkv_quest_select preceded it on that layer */
  uint64_t blocks_by_level[5]; /* closed blocks at 16, 8, 4, 2, centroid */
  double bpv_resident, bpv_paper /* without residual index bits */, bpv_read;
} gkv_bits;

/* Bytes of device arena that are certainly enough for `cfg` (metadata + block slots).
 * A smaller arena is accepted by gkv_create as long as the metadata fits; appends then
 * fail with GKV_ERR_ARENA_TOO_SMALL when slots run out.  bytes: host out. */
GKV_API int gkv_query_arena_bytes(const gkv_config* cfg, size_t* bytes);

/* Create a cache inside `arena` (device, 256-byte aligned, arena_bytes long, owned by the
 * caller and kept alive until gkv_destroy).  The arena's metadata region is initialised on
 * the default ordering of `stream`-less cudaMemset, so the call synchronises.  out: host. */
GKV_API int gkv_create(const gkv_config* cfg, void* arena, size_t arena_bytes, gkv_cache** out);

/* Free the host object (synchronises the device first).  The arena is not touched. */
GKV_API int gkv_destroy(gkv_cache* c);

/* Append n_new tokens to every sequence of `layer`, then move full blocks down the ladder
 * (Sec. 3.2: monotone demotion, never upward, requantised from the block's current
 * representation).  The only mutating call.
 *   k_new  device bf16 [batch][n_new][n_kv_heads][d_k]
 *   v_new  device bf16 [batch][n_new][n_kv_heads][d_v]; NULL iff v_aliases_k
 *   n_new  1 = decode step; >1 only on an empty layer (bulk ingest: each full block is
 *          encoded once, directly at its planned level)
 *   token_mass  device fp32 [batch][n_kv_heads][n_new], prompt attention mass per token already
 *          aggregated over observed queries and the KV head's query heads (Sec. 3.1);
 *          required for GKV_POLICY_RD and for residual_fraction > 0 at bulk ingest, else NULL
 *   level_plan  HOST int8 [batch][n_kv_heads][n_new/64], values in {16,8,4,2,1};
 *          required for GKV_POLICY_EXTERNAL at bulk ingest, else NULL
 * Bulk ingest under GKV_POLICY_RD (and residual selection) synchronises the stream once, to
 * run the allocator (Sec. 3.3) on the host.  Decode-step appends never synchronise.
 * May return GKV_ERR_RANGE / GKV_ERR_BUDGET as warnings after completing the work. */
GKV_API int gkv_append_demote(gkv_cache* c, int32_t layer, const void* k_new, const void* v_new, int32_t n_new,
                      const float* token_mass, const int8_t* level_plan, void* stream);

/* Single-query attention of every query head over the graded cache of `layer`
 * (Sec. 3.7; Eq. 1 over the reconstructed keys/values; split-context partials are merged inside
 * the same launch, in a fixed order).
 *   q        device bf16 [batch][n_q_heads][d_k]
 *   page_idx device int32 [batch][n_kv_heads][n_sel] ascending closed-page indices, or NULL with
 *            n_sel = 0 for a full read.  With a list, only those pages and the partial tail block
 *            are read; every other token is hard-masked (Sec. 3.5), exact residual tokens of
 *            pages that are not listed included.  An entry outside [0, closed pages) is skipped
 *            by the kernel (nothing is read through it) and the next gkv_bits_report returns
 *            GKV_ERR_BAD_STATE.  The library keeps the pointer, not a copy: the list must stay
 *            allocated and unchanged until the next gkv_bits_report of this layer if that report
 *            is to count the bits the read touched (a later read of the layer replaces it)
 *   out      device fp32 [batch][n_q_heads][d_v]
 *   lse      device fp32 [batch][n_q_heads] natural-log sum of exp(logit), or NULL */
GKV_API int gkv_decode_attn(gkv_cache* c, int32_t layer, const void* q, const int32_t* page_idx, int32_t n_sel,
                    float* out, float* lse, void* stream);

/* gkv_decode_attn over the full context that, in the same pass over the cache, observes the
 * attention mass of every block (Sec. 3.1, Eq. 2 with this query as the observed one):
 *   a_b = mean over the KV head's query heads of the summed softmax weight of block b's tokens,
 * b = 0 .. n_closed - 1 and, when it holds tokens, the partial block as the last entry; tokens
 * served from the exact residual count for the block they sit in.  The cache's running mass is
 * then updated, m_b <- 0.9 m_b + 0.1 a_b; it starts from the prompt masses given at bulk ingest
 * under GKV_POLICY_RD and from 0 otherwise (also for blocks that appear during decode).
 *   q, out, lse  as for gkv_decode_attn
 *   block_mass   device fp32 [batch][n_kv_heads][n_items], n_items = blocks that hold tokens
 *                (ceil(ctx / 64)), or NULL: receives a_b of this call
 *   certificate  device fp32 [batch][n_q_heads], or NULL: the attention error certificate of this
 *                query (Sec. 3.6, Eq. 9), a bound on |o - o^|_2 between attention over the original
 *                rows and the output written to `out`:
 *                  sum_b a^_b delta_b + min(2, M+/M- - M-/M+) max_j |v_j|,  M+- = sum_b a^_b exp(+-eps_b),
 *                with a^_b the weight of block b's non-exact tokens for this head, eps_b = scale |q|
 *                kappa_b, and kappa_b / delta_b the bounds on max_j |k_j - k^_j|_2 / max_j |v_j - v^_j|_2
 *                that the library keeps per block: the distance itself when a block is encoded from
 *                its original rows, grown by the distance between old and new reconstruction at every
 *                later demotion (triangle inequality).  Exact tokens (exact blocks, the partial block,
 *                residual rows) enter with eps = delta = 0; max_j |v_j| is over the original rows.
 * Grouped-query layout only (GKV_ERR_UNSUPPORTED with v_aliases_k).  Costs one or two extra small
 * launches and 64 B of scratch writes per block and stream; the graded cache is read once. */
GKV_API int gkv_decode_attn_observe(gkv_cache* c, int32_t layer, const void* q, float* out, float* lse,
                                    float* block_mass, float* certificate, void* stream);

/* Per-block bounds behind the certificate (parity checks; synchronises the device).
 *   bounds_out  HOST fp32 [batch][n_kv_heads][n_closed][4]: kappa_b, delta_b, max_j |v_j|, 0 */
GKV_API int gkv_debug_export_bounds(gkv_cache* c, int32_t layer, float* bounds_out);

/* Decode-time re-allocation under GKV_POLICY_RD (Sec. 3.1-3.3): runs the allocator of Eq. 4 again
 * for every stream of `layer` on the running masses m_b (gkv_decode_attn_observe) and the range
 * proxies recorded when each block closed, at the budget rd_budget_bpv of the current context.
 * The temporal constraint of Sec. 3.2 holds: no level rises, sink blocks and the newest
 * retire_after tokens' blocks stay at 16 bits; blocks whose level falls are requantised from their
 * current representation.  The plan is made on the device (the threshold search of Eq. 4 over the
 * sorted breakpoints, one thread block per stream; up to 4095 closed blocks, beyond that on the host
 * from masses read back); the host reads the plan back - one byte per block - to do the slot
 * bookkeeping, so the call synchronises `stream` once.  Meant to be called when a block has closed
 * (every 64 tokens), not every step.
 * May return GKV_ERR_BUDGET / GKV_ERR_RANGE as warnings after completing the work. */
GKV_API int gkv_rd_reallocate(gkv_cache* c, int32_t layer, void* stream);

/* Parity only: the plan gkv_rd_reallocate would apply now, made the way it makes it (on the device),
 * without applying it, together with the numbers it was made from.  Synchronises `stream`.
 *   levels_out  HOST int8 [batch][n_kv_heads][n_closed]
 *   mass_out    HOST fp32 [batch][n_kv_heads][n_closed] running masses m_b, or NULL
 *   range_out   HOST fp32 [batch][n_kv_heads][n_closed] range proxies e_b, or NULL
 * Returns GKV_ERR_BUDGET (with the plan written) when a stream cannot meet the budget. */
GKV_API int gkv_debug_device_plan(gkv_cache* c, int32_t layer, int8_t* levels_out, float* mass_out, float* range_out,
                                  void* stream);

/* Host-only (no device work): the plan gkv_rd_reallocate decides for one stream.  mass / range
 * fp32 [n_closed]; prev int8 [n_closed] current levels; levels int8 [n_closed] out. */
GKV_API int gkv_debug_replan_levels(const gkv_config* cfg, int32_t n_closed, int32_t n_tail, const float* mass,
                                    const float* range, const int8_t* prev, int8_t* levels, int32_t* budget_miss);

/* Running block masses m_b of `layer` (parity checks; synchronises the device).
 *   mass_out  HOST fp32 [batch][n_kv_heads][ceil(ctx / 64)] */
GKV_API int gkv_debug_export_mass(gkv_cache* c, int32_t layer, float* mass_out);

/* Compressed-Quest page selection (Sec. 3.5): score every page of every closed block with the
 * box upper bound sum_d max(q_d * min_d, q_d * max_d), reduce over the KV head's query heads,
 * keep the k = min(budget_tokens / page_tokens, closed pages) best per (sequence, KV head).
 *   q            device bf16 [batch][n_q_heads][d_k]
 *   page_idx_out device int32 [batch][n_kv_heads][k], ascending
 *   n_sel_out    host int32, receives k */
GKV_API int gkv_quest_select(gkv_cache* c, int32_t layer, const void* q, int32_t budget_tokens,
                     int32_t* page_idx_out, int32_t* n_sel_out, void* stream);

/* Parity helpers of the page scorer (Sec. 3.5; both synchronise the device).
 * gkv_debug_export_boxes: the exact per-page per-channel key minima and maxima of one stream, as
 * recorded from the unquantised keys when each block closed.
 *   lo / hi   HOST bf16 bits [n_pages][d_k] each, n_pages = closed blocks * (64 / page_tokens);
 *             cap_pages is the room of the two arrays in pages, *n_pages receives the count
 * gkv_debug_export_scores: the page scores that gkv_quest_select ranks, for every stream of `layer`
 * and the query q (device bf16 [batch][n_q_heads][d_k]): per query head sum_d q_d * (q_d >= 0 ? max_d :
 * min_d) added in ascending d in fp32, reduced over the KV head's query heads (cfg.quest_reduce).
 *   scores    HOST fp32 [batch][n_kv_heads][n_pages]
 * Both return GKV_ERR_BAD_STATE without a page scorer (page_tokens == 0). */
GKV_API int gkv_debug_export_boxes(gkv_cache* c, int32_t layer, int32_t b, int32_t kv_head, uint16_t* lo, uint16_t* hi,
                                   int32_t cap_pages, int32_t* n_pages);
GKV_API int gkv_debug_export_scores(gkv_cache* c, int32_t layer, const void* q, float* scores, void* stream);

/* The same page selection as gkv_quest_select for callers that cannot have any device memory
 * allocated on their behalf while they run: a plug-in that was handed a fixed arena by a serving
 * engine whose pool is fully committed, a real-time loop that forbids allocation after start-up,
 * or code that runs where cudaMalloc is not allowed.  (The paper has no counterpart; this is a
 * packaging variant of the Sec. 3.5 selection.)  The page scores, which gkv_quest_select keeps in
 * the arena, go to a fixed 4 MiB array that is part of the library image, so the call performs no
 * cudaMalloc / cudaFree and uses no allocating library routine.
 *   - Limit: batch * n_kv_heads * round_up(closed pages, 8) <= 1,048,576 scores; larger caches get
 *     GKV_ERR_UNSUPPORTED (use gkv_quest_select).
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress);
 *     make that first call before any stream capture begins.
 *   - All calls on a device share the one array and it keeps the previous call's contents.  Each
 *     call overwrites every score it later reads, so stale contents are harmless, but two calls
 *     whose kernels overlap on the GPU (different streams, or different caches) race: issue them
 *     on one stream or order them yourself.
 * Arguments and results are exactly those of gkv_quest_select. */
GKV_API int gkv_quest_select_static(gkv_cache* c, int32_t layer, const void* q, int32_t budget_tokens,
                                    int32_t* page_idx_out, int32_t* n_sel_out, void* stream);

/* Resident / read bit accounting of `layer` (-1 = all layers).  Synchronises when the last
 * read used a page list (it is fetched to count the bits touched).  out: host. */
GKV_API int gkv_bits_report(gkv_cache* c, int32_t layer, gkv_bits* out);

/* Parity helpers (synchronise).  Logical contents of one closed block of one tensor:
 *   level       host int32: 16, 8, 4, 2 or 1
 *   codes       host uint8 [64][d] (levels 8/4/2)
 *   scale/zero  host fp16 bits; K: [2][d_k] (32-token halves), V: [64][d_v/32]
 *   rows_bf16   host bf16 bits; level 16: [64][d]; level 1: [d] centroid
 * Unused outputs may be NULL.  block == number of closed blocks addresses the tail (level 16,
 * n_rows receives its token count). */
GKV_API int gkv_debug_export_block(gkv_cache* c, int32_t layer, int32_t b, int32_t kv_head, int32_t block,
                           int32_t which, int32_t* level, uint8_t* codes, uint16_t* scale_fp16,
                           uint16_t* zero_fp16, uint16_t* rows_bf16, int32_t* n_rows);
/* Residual token indices of one stream, ascending.  idx: host int32 [cap]; n: host. */
GKV_API int gkv_debug_export_residual(gkv_cache* c, int32_t layer, int32_t b, int32_t kv_head, int32_t* idx,
                              int32_t cap, int32_t* n);
/* Levels of all closed blocks of one stream.  levels: host int8 [cap]; n: host. */
GKV_API int gkv_debug_export_levels(gkv_cache* c, int32_t layer, int32_t b, int32_t kv_head, int8_t* levels,
                            int32_t cap, int32_t* n);
/* The host-side level plan on its own, without a cache or a device (all pointers host): what
 * gkv_append_demote decides for one stream whose n_closed blocks are closed and whose tail holds
 * n_tail tokens.  Staircase policy (Sec. 3.2, Fig. 1): from cfg->stair_tokens / n_sink_blocks;
 * mass and range are ignored and may be NULL.  RD policy (Sec. 3.3, the monotone allocator):
 * mass / range are fp32 [n_closed] per-block attention mass and range proxy; *budget_miss is set
 * when even the cheapest plan exceeds rd_budget_bpv.  levels: int8 [n_closed], index 0 = oldest.
 * Used by the CPU tests to hold the host logic against the oracle. */
GKV_API int gkv_debug_plan_levels(const gkv_config* cfg, int32_t n_closed, int32_t n_tail, const float* mass,
                                  const float* range, int8_t* levels, int32_t* budget_miss);
/* Current context length (tokens) of a layer. */
GKV_API int gkv_ctx_len(gkv_cache* c, int32_t layer, int32_t* ctx);

GKV_API const char* gkv_strerror(int status);
GKV_API int gkv_last_cuda_error(gkv_cache* c); /* cudaError_t of the last GKV_ERR_CUDA */

#ifdef __cplusplus
}
#endif
#endif /* GKV_H_ */
