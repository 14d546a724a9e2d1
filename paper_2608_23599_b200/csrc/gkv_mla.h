// Parameter blocks and launchers of the latent-attention (MLA) kernels (gkv_mla.cu).
#pragma once
#include "gkv_internal.h"

namespace gkv {

constexpr int kMlaPartialFloats = kMlaHeads * (kMlaDv + 2);   // per CTA partial: m, l, o[512] per head
constexpr int kMlaQuads = 4;                                  // groups of four warps per CTA of the decode kernel, each with a block range of its own

struct MlaEncodeParams {
  uint8_t* arena;
  const EncodeJob* jobs;
  int32_t n_jobs;
  const uint16_t* k_in;     // bf16 [batch][n_tok][576] (src_level == 0)
  int32_t n_tok;
  uint32_t* status;
};

struct MlaDecodeParams {
  const uint8_t* arena;
  const TableEntry* table;  // [n_streams][table_stride]
  const WarpDesc* ctas;     // kMlaQuads descriptors per CTA: contiguous item ranges of one stream, one partial row
  const uint16_t* q;        // bf16 [batch][16][576]
  float* partial;           // [n_ctas][kMlaPartialFloats]
  int32_t table_stride, n_closed, n_tail;
  float scale_log2;
  uint32_t* status;
};

cudaError_t launch_mla_encode(const MlaEncodeParams& p, cudaStream_t st);
cudaError_t launch_mla_ingest(const MlaEncodeParams& p, cudaStream_t st);   // all jobs from the bf16 input, 16-byte aligned
cudaError_t launch_mla_append_rows(uint8_t* arena, const TableEntry* table, int table_stride, int tail_index, int n_streams,
                                   const uint16_t* k_in, int n_tok, int first_tok, int n_rows, int dst_row0, cudaStream_t st);
cudaError_t launch_mla_export(const uint8_t* arena, uint32_t off256, int level, uint8_t* codes, uint16_t* scale,
                              uint16_t* zero, uint16_t* rows, cudaStream_t st);
cudaError_t launch_mla_decode(const MlaDecodeParams& p, int n_ctas, const StreamParts* parts, int n_streams, float* out,
                              float* lse, cudaStream_t st);

}  // namespace gkv
