// Physical layout of graded blocks in the arena and the logical<->physical index maps.
//
// A block is 64 tokens of one (layer, sequence, KV head) stream (paper Sec. 3.2).  Head dim
// D = 128 in this build.  Slots are multiples of 512 bytes:
//
//   level 16 : [K rows 64 x 128 bf16][V rows 64 x 128 bf16]                    32768 B
//   level 1  : [K centroid 128 bf16][V centroid 128 bf16]                        512 B
//   level b in {8,4,2}: two halves (tokens 0-31, 32-63), each
//       Kp   512 B     key scale/zero per channel for this half (keys are grouped along time)
//       Kc   2 x CB    key codes of the half's two 16-token tiles, CB = 256*b bytes each
//       Vp   2 x 256 B value scale/zero per (token, 32-channel group) of each tile
//       Vc   2 x CB    value codes of the two tiles
//     slot = 2 * (1024 + 4*CB) = 18432 / 10240 / 6144 B
//
// Codes are stored in the order the attention kernel's tensor-core fragments consume them, so
// that a 16-byte load per lane feeds mma.m16n8k16 A operands without any shuffle:
//   tile (16 tokens), lane = 4*r + c4, mma index s in 0..7, A register a in 0..3, half hlf in 0..1
//   K role (A = K tile [16 tokens x 16 channels]):
//       token = 16*tile + r + 8*(a&1),  channel = 16*s + 8*(a>>1) + 2*c4 + hlf
//   V role (A = V^T tile [16 channels x 16 tokens]):
//       channel = 16*s + r + 8*(a&1),   token = 16*tile + 8*(a>>1) + 2*c4 + hlf
// A lane's 64 values of a tile form 32 pairs (s, a) (lo = hlf 0 in bits 0-15, hi = hlf 1 in bits
// 16-31 of a 32-bit word).  The bit position of a pair is chosen so that the kernel can turn a
// code into an fp16 number "bias + code" with one shift per word and one LOP3 per pair (the code
// is OR-ed into the mantissa of 2^E; a field at mantissa bit p with E = 10 - p has weight 1):
//   8-bit: word = 2 s + (a >> 1); pair at byte (a & 1) and byte 2 + (a & 1)      bias 1024
//   4-bit: word = s;              pair at bit 4 a                    bias 256 (a even) / 16 (a odd)
//   2-bit: word = s >> 1;         pair at bit 4 (s & 1) + 2 (a & 1) + 8 (a >> 1)
//                                 bias 256 / 64 (s even, a even / odd), 16 / 4 (s odd)
// so that within one MMA the bias depends only on the A-row half (a & 1) and can be removed after
// the MMA.  Value codes (V role) swap the fields of registers 1 and 2 (field f = (a >> 1) | ((a & 1) << 1)
// takes the place of a in the 4-bit and 2-bit positions): the kernel reads them as the bias-free
// numbers code * 2^(p - 24) (a code in the mantissa of an fp16 with a zero exponent field), whose
// weight then depends only on the token half a >> 1 and is evened out in the probabilities.
// Word w of a lane lives at byte ((w/4)*32 + lane)*16 + (w%4)*4
// of the tile's code region (chunk-major: 512 contiguous bytes per warp-wide 16-byte load).
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define GKV_HD __host__ __device__ __forceinline__
#else
#define GKV_HD inline
#endif

namespace gkv {

constexpr int kBlock = 64;     // tokens per block
constexpr int kGroup = 32;     // quantisation group
constexpr int kD = 128;        // head dim of this build
constexpr int kTile = 16;      // tokens per tensor-core tile
constexpr int kRowBytes = kD * 2;

// Item levels as stored in the block table.
constexpr int kLvlExact = 16, kLvlCentroid = 1;

GKV_HD int code_bytes_per_tile(int bits) { return 256 * bits; }
GKV_HD int half_bytes(int bits) { return 1024 + 4 * code_bytes_per_tile(bits); }
GKV_HD int slot_bytes(int level) {
  return level == 16 ? 2 * kBlock * kRowBytes : (level == 1 ? 2 * kRowBytes : 2 * half_bytes(level));
}
// Offsets inside one half of a quantised slot.
GKV_HD int off_kp() { return 0; }
GKV_HD int off_kc(int bits, int t) { return 512 + t * code_bytes_per_tile(bits); }
GKV_HD int off_vp(int bits, int t) { return 512 + 2 * code_bytes_per_tile(bits) + t * 256; }
GKV_HD int off_vc(int bits, int t) { return 1024 + (2 + t) * code_bytes_per_tile(bits); }

// Where code (lane, s, a, hlf) of a tile sits: byte offset of its 32-bit word inside the tile's
// code region, and the bit position inside the word.
// Largest value scale the read path takes: the kernel multiplies the probabilities by the scale and by the
// power of two that evens out the fields' weights (up to 2^4) in fp16.  A larger scale (a 32-channel
// value group spanning more than 1.0e6 / 6.1e4 / 1.2e4 at 8 / 4 / 2 bits) is reported like a saturated one.
GKV_HD float v_scale_limit(int bits) { (void)bits; return 4094.f; }
GKV_HD int code_field(bool is_v, int a) { return is_v ? ((a >> 1) | ((a & 1) << 1)) : a; }
GKV_HD void code_pos(int bits, bool is_v, int lane, int s, int a, int hlf, int* byte_off, int* bit) {
  int w, b;
  if (bits == 8) {
    w = 2 * s + (a >> 1);
    b = 8 * (a & 1);
  } else if (bits == 4) {
    w = s;
    b = 4 * code_field(is_v, a);
  } else {
    const int f = code_field(is_v, a);
    w = s >> 1;
    b = 4 * (s & 1) + 2 * (f & 1) + 8 * (f >> 1);
  }
  *byte_off = ((w >> 2) * 32 + lane) * 16 + (w & 3) * 4;
  *bit = b + 16 * hlf;
}

// K role: logical (token in block, channel) -> (tile, lane, s, a, hlf)
GKV_HD void k_coord(int tok, int ch, int* tile, int* lane, int* s, int* a, int* hlf) {
  *tile = tok >> 4;
  const int t16 = tok & 15, c16 = ch & 15;
  const int r = t16 & 7, c4 = (c16 & 7) >> 1;
  *lane = 4 * r + c4;
  *s = ch >> 4;
  *a = (t16 >> 3) | ((c16 >> 3) << 1);
  *hlf = c16 & 1;
}
// V role: logical (token in block, channel) -> (tile, lane, s, a, hlf)
GKV_HD void v_coord(int tok, int ch, int* tile, int* lane, int* s, int* a, int* hlf) {
  *tile = tok >> 4;
  const int t16 = tok & 15, c16 = ch & 15;
  const int r = c16 & 7, c4 = (t16 & 7) >> 1;
  *lane = 4 * r + c4;
  *s = ch >> 4;
  *a = (c16 >> 3) | ((t16 >> 3) << 1);
  *hlf = t16 & 1;
}
// Key params of a half: 32 bytes per (channel slab j of 32 channels, c4): a 16-byte record of zero points,
// then one of scales, each {s0: c0 c1, s1: c0 c1, s0: c2 c3, s1: c2 c3} for the slab's two MMA indices
// s0 = 2 j, s1 = 2 j + 1 and the lane's channel pairs c0 = 16 s + 2 c4, c1 = c0 + 1, c2 = c0 + 8,
// c3 = c2 + 1.  The zero-point record is the A operand of the one MMA per slab that forms sum q z for both
// MMA indices (rows r from s0, rows r + 8 from s1); the scale record feeds q' = q s of both.
// Returns the index (in fp16 units) of channel ch's scale inside the 512-byte array; its zero point
// sits 8 entries before.
GKV_HD int kp_index(int ch) {
  const int s = ch >> 4, c16 = ch & 15;
  const int c4 = (c16 & 7) >> 1;
  return ((s >> 1) * 4 + c4) * 16 + 8 + ((c16 >> 3) * 2 + (s & 1)) * 2 + (c16 & 1);
}
GKV_HD int kp_zero_index(int ch) { return kp_index(ch) - 8; }
// Value params of a tile (256 B): scales first, then zeros, both as fp16 pairs of the lane's
// token pairs tA = (2 c4, 2 c4 + 1) and tB = (8 + 2 c4, 9 + 2 c4):
//   scales [c4][group] = {s tA0, s tA1, s tB0, s tB1}   (one lane reads its 4 groups as 32 contiguous bytes)
//   zeros  [group][c4] = {z tA0, z tA1, z tB0, z tB1}   at byte 128 (lane r < 4 reads group r)
// Returns the fp16 index of the scale / of the zero of (token t16 of the tile, group grp).
GKV_HD int vp_scale_index(int t16, int grp) {
  const int c4 = (t16 & 7) >> 1;
  return (c4 * 4 + grp) * 4 + (t16 >> 3) * 2 + (t16 & 1);
}
GKV_HD int vp_zero_index(int t16, int grp) {
  const int c4 = (t16 & 7) >> 1;
  return 64 + (grp * 4 + c4) * 4 + (t16 >> 3) * 2 + (t16 & 1);
}

}  // namespace gkv

// ---- latent-attention (MLA) streams: one 576-wide row per token, values = channels [0, 512) ----
// The row is quantised once with the key rule (32 tokens x 1 channel per group).  A quantised slot
// is two halves of 32 tokens: [params 2304 B][codes 32 rows x 72 chunks]; a chunk is 8 neighbouring
// channels of one token (8 bytes at 8 bits, one 32-bit word at 4 bits).  The params are the 576 fp16
// scales, then the 576 fp16 zero points (a chunk's eight scales are one 16-byte piece, neighbouring
// chunks neighbouring pieces: a warp reads them without gaps).  Inside a chunk the codes are placed so
// that one "mask, or in an exponent" (4 bits) or one byte permute (8 bits) yields the fp16 pair
// of two neighbouring channels: 4-bit channel c sits at bit 4 (c >> 1) + 16 (c & 1); 8-bit channel c
// sits in word c >> 2 at byte ((c & 3) >> 1) + 2 (c & 1).
namespace gkv {
constexpr int kMlaDk = 576, kMlaDv = 512, kMlaHeads = 16, kMlaKSteps = kMlaDk / 16;   // 36
constexpr int kMlaChunks = kMlaDk / 8;                                                // 72
constexpr int kMlaRowBytes = kMlaDk * 2;                                              // 1152
GKV_HD int mla_kp_bytes() { return kMlaChunks * 32; }                                     // 2304 per half
GKV_HD int mla_code_row_bytes(int bits) { return kMlaChunks * bits; }                     // 576 / 288
GKV_HD int mla_half_bytes(int bits) { return mla_kp_bytes() + 32 * mla_code_row_bytes(bits); }
GKV_HD int mla_slot_bytes(int level) {
  return level == 16 ? kBlock * kMlaRowBytes : (level == 1 ? 1280 : 2 * mla_half_bytes(level));
}
// fp16 index of channel ch's scale inside a half's params; its zero point sits kMlaZeroOff entries later
GKV_HD int mla_kp_index(int ch) { return ch; }
constexpr int kMlaZeroOff = kMlaDk;   // fp16 entries from a channel's scale to its zero point
// position of the code of (token t32 of the half, channel ch): byte offset of its 32-bit word from
// the start of the half's code rows, and the bit inside that word
GKV_HD void mla_code_pos(int bits, int t32, int ch, int* byte_off, int* bit) {
  const int j = ch >> 3, c = ch & 7;
  if (bits == 8) {
    *byte_off = t32 * mla_code_row_bytes(8) + j * 8 + (c >> 2) * 4;
    *bit = 8 * (((c & 3) >> 1) + 2 * (c & 1));
  } else {
    *byte_off = t32 * mla_code_row_bytes(4) + j * 4;
    *bit = 4 * (c >> 1) + 16 * (c & 1);
  }
}
}  // namespace gkv
