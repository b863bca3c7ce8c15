// Packed cache layout in HBM (head_dim = 128).  Shared by the quantise, append, decode and
// export kernels of this library.
//
// A quantised tensor lives in one of two stores:
//
//   ROW store   (per-token groups along channels; InnerQ keys).  One row of 16*b bytes per
//               token, so one evicted token is one contiguous write.  Metadata: one 32-bit
//               word per (token, group) = fp16 scale (mask M in the sign bit) | fp16
//               zero-point << 16; in symmetric mode only the 16-bit scale is stored.
//   BLOCK store (per-channel groups along tokens; InnerQ values).  Chunks of 32 tokens x 128
//               channels, 512*b bytes each.  Metadata: one word per (group of G tokens,
//               channel), reused by the G tokens of the group.
//
// Both stores of a cache are interleaved in "chunk records" of 32 tokens (see struct Store), so
// that everything a decode step needs for 32 tokens is one contiguous, 16-byte aligned range.
//
// Inside a row / chunk the codes are permuted so that a 32-lane warp reads its tensor-core
// operand fragments with 64/128-bit loads and extracts them with one LOP3 per pair:
// lane L = 4*gid + tid4 owns the fragment entries that mma.m16n8k16 assigns to it, and a
// 32-bit word holds pairs (low half, high half) at equal field positions, so that
// `word & (mask << pos)` is a half2 of two codes scaled by 2^pos (as fp16 subnormals).
//
// b = 3 is stored as a 2-bit plane followed by a 1-bit plane (code = lo + 4*hi).
#pragma once
#include <cstddef>
#include <cstdint>

#ifdef __CUDACC__
#define IQ_HD __host__ __device__ __forceinline__
#else
#define IQ_HD inline
#endif

namespace iq {

constexpr int kD = 128;           // head_dim
constexpr int kChunk = 32;        // tokens per BLOCK-store chunk
constexpr int kTile = 128;        // capacity granularity in tokens

enum StoreKind : int { kRow = 0, kBlock = 1, kNone = 2 };

struct Store {
  int kind;            // StoreKind: how the tensor is grouped (kRow: groups of G channels inside a token, metadata
                       // per token; kBlock: per-channel groups of G tokens, metadata per group)
  int code_kind;       // how its codes are laid out: kRow = one packed row per token (the operand order of q.K^T),
                       // kBlock = 32-token chunks (the operand order of p.V).  Equal to `kind` under inner grouping;
                       // under outer grouping keys keep rows and values keep chunks, only the metadata changes sides.
  int bits, mode;
  int perm;            // order of the codes inside a packed row / chunk: 0 = pairs for the fp16 tensor-core fragments
                       // (word & mask is a half2; outer-grouped caches), 1 = bytes for the 8-bit integer fragments
                       // (inner-grouped caches; see row_pos_i8 / block_pos_i8 / row_pos_i8_3 / block_pos_i8_3)
  int ring_cap;        // slots of the recent ring: w_recent + 1 (ROW) or w_recent + G (BLOCK)
  int cap_q;           // capacity in quantised tokens (multiple of kTile)
  int n_groups;        // metadata entries per row (ROW: D/G) or per group (BLOCK: D)
  int meta_bytes;      // 4: fp16 scale | fp16 zero << 16;  2: fp16 scale only (symmetric mode stores no zero-points)
  size_t sink_off, ring_off;          // byte offsets of unit 0's fp16 windows
  size_t sink_stride, ring_stride;    // bytes per unit
  // Packed records.  The ROW store and the BLOCK store of a cache share one record area per unit:
  // for every group of G tokens, G/32 chunk records followed by the BLOCK store's metadata of the group;
  // a chunk record holds, for 32 consecutive tokens, the ROW store's packed rows, the ROW store's
  // metadata rows and the BLOCK store's packed chunk.  A decoding warp fetches a chunk record (plus the
  // group metadata behind the last chunk of a group) with ONE contiguous bulk copy.
  size_t rec_off, rec_unit_stride;    // byte offset of unit 0's record area, bytes per unit
  int group_stride, chunk_stride;     // bytes per group record / per chunk record
  int chunks_per_group;               // G / 32
  int chunk0;                         // offset of the first chunk record inside a group record (non-zero when the
                                      // per-group metadata comes first: outer grouping, where keys need it up front)
  int code_in_rec;                    // offset of this store's codes inside a chunk record
  int meta_in_rec;                    // ROW: offset of its metadata rows inside a chunk record;
                                      // BLOCK: offset of the group's metadata inside a group record
};

// Byte offset of chunk record ci inside its group record.
IQ_HD size_t chunk_in_group_off(const Store& S, int ci) {
  return S.chunk0 + (size_t)(ci % S.chunks_per_group) * S.chunk_stride;
}

struct Layout {
  int B, Hq, Hkv, U, r;
  int G, w_sink, w_recent, sym_variant, grouping, k_normalize;
  int max_tokens, max_splits;
  float sm_scale;
  size_t norm_off;     // float [U][D]
  size_t appended_off; // uint32 [U]: token count of the unit after the last append (or prefill) whose writes are
                       // complete; a decode of N tokens that reads N there may read the rings and the newest rows.
                       // Then uint32 [U]: tickets of the CTAs that share the append of one unit (zero between appends)
  size_t cache_bytes;
  // workspace
  size_t ws_partial_off;   // float [B*Hq][max_splits][kPartialStride]
  size_t ws_absmax_off;    // uint32 [U][D]
  size_t ws_ticket_off;    // uint32 [U]
  size_t workspace_bytes;
  // Paged record area (page_groups > 0): the group records of a cache live in pages of a pool that several caches
  // share, `page_groups` consecutive groups of every unit per page, and a table in the cache's own memory names the
  // page of each page slot.  Inside a page the layout is the contiguous one ([unit][group]) with rec_unit_stride =
  // page_groups * group_stride.  page_groups == 0: one contiguous record area per unit inside the cache buffer.
  int page_groups, max_pages;
  int page_chunk_mask;     // chunks per page - 1 (a page holds 2^k chunks of 32 tokens); contiguous: 0x3fffffff
  int page_chunk_shift;    // k
  size_t page_bytes;
  size_t page_table_off;   // uint32 [max_pages] in the cache buffer: pool page of page slot p
  unsigned char* pool;     // device address of page 0
  Store k, v;
};

// The record area of one unit, as the kernels address it: group record g starts at group_ptr(R, g).
struct Rec {
  unsigned char* base;       // contiguous: the unit's record area; paged: the unit's slice of pool page 0
  const uint32_t* table;     // paged: pool page of every page slot of the cache (device memory); null when contiguous
  size_t page_bytes;
  int page_groups;
  int group_stride;
};
IQ_HD Rec unit_rec(const Layout& L, const unsigned char* cache, int u) {
  Rec R;
  unsigned char* c = const_cast<unsigned char*>(cache);
  const bool paged = L.page_groups > 0;
  R.base = (paged ? L.pool : c + L.k.rec_off) + (size_t)u * L.k.rec_unit_stride;
  R.table = paged ? reinterpret_cast<const uint32_t*>(c + L.page_table_off) : nullptr;
  R.page_bytes = L.page_bytes;
  R.page_groups = L.page_groups;
  R.group_stride = L.k.group_stride;
  return R;
}
IQ_HD unsigned char* group_ptr(const Rec& R, int g) {
  if (!R.table) return R.base + (size_t)g * R.group_stride;
  const int slot = g / R.page_groups;
  return R.base + (size_t)R.table[slot] * R.page_bytes + (size_t)(g - slot * R.page_groups) * R.group_stride;
}
IQ_HD unsigned char* chunk_rec_ptr(const Rec& R, const Store& S, int ci) {
  return group_ptr(R, ci / S.chunks_per_group) + chunk_in_group_off(S, ci);
}
// Row-coded tensor: packed row of quantised token i.  kRow tensor: base of token i's metadata entries.
IQ_HD unsigned char* row_code_ptr(const Rec& R, const Store& S, int i) {
  return chunk_rec_ptr(R, S, i / kChunk) + S.code_in_rec + (size_t)(i % kChunk) * (16 * S.bits);
}
IQ_HD unsigned char* row_meta_ptr(const Rec& R, const Store& S, int i) {
  return chunk_rec_ptr(R, S, i / kChunk) + S.meta_in_rec + (size_t)(i % kChunk) * S.n_groups * S.meta_bytes;
}
// Chunk-coded tensor: packed chunk ci.  kBlock tensor: metadata of group j.
IQ_HD unsigned char* block_code_ptr(const Rec& R, const Store& S, int ci) { return chunk_rec_ptr(R, S, ci) + S.code_in_rec; }
IQ_HD unsigned char* block_meta_ptr(const Rec& R, const Store& S, int j) { return group_ptr(R, j) + S.meta_in_rec; }

constexpr int kPartialStride = kD + 4;   // acc[D], m, l, pad, pad

// Token bookkeeping: a function of N alone.
// Most caches one batched call (append / decode over independent caches of one configuration) takes.
constexpr int kMaxSeqs = 32;

struct Counts {
  int N, n_sink, n_qk, n_qv, n_k_recent, n_v_recent;
};

IQ_HD int n_quantised(int kind, int N, int w_sink, int w_recent, int G) {
  int mid = N - w_sink - w_recent;
  if (kind == kNone || mid <= 0) return 0;
  return kind == kRow ? mid : (mid / G) * G;
}

IQ_HD Counts counts_for(const Layout& L, int N) {
  Counts c;
  c.N = N;
  c.n_sink = N < L.w_sink ? N : L.w_sink;
  c.n_qk = n_quantised(L.k.kind, N, L.w_sink, L.w_recent, L.G);
  c.n_qv = n_quantised(L.v.kind, N, L.w_sink, L.w_recent, L.G);
  c.n_k_recent = N - c.n_sink - c.n_qk;
  c.n_v_recent = N - c.n_sink - c.n_qv;
  return c;
}

// ---------------------------------------------------------------- code positions
// ROW store: bit position of channel c inside a row of 16*b bytes.
//   k-step s = c / 16 (16 channels feed one mma k-step), col = c % 16,
//   tid4 = (col % 8) / 2 owns the column pair, hf = col % 2 selects the half-word,
//   odd = col / 8 selects the second pair of the k-step.
struct BitPos { int word; int bit; };      // 32-bit word index inside the row/chunk, bit inside the word

IQ_HD BitPos row_pos_plane(int c, int plane_bits) {
  int s = c >> 4, col = c & 15;
  int j = (col & 7) >> 1, hf = col & 1, odd = col >> 3;
  BitPos p;
  if (plane_bits == 2) {         // lane chunk = 2 words; word serves 4 k-steps, 2 fields each
    p.word = 2 * j + (s >> 2);
    p.bit = 16 * hf + 2 * (2 * (s & 3) + odd);
  } else if (plane_bits == 4) {  // lane chunk = 4 words; word serves 2 k-steps
    p.word = 4 * j + (s >> 1);
    p.bit = 16 * hf + 4 * (2 * (s & 1) + odd);
  } else {                       // 1-bit plane: lane chunk = 1 word; 8 k-steps x 2 fields
    p.word = j;
    p.bit = 16 * hf + (2 * s + odd);
  }
  return p;
}

// BLOCK store: position of (token tau in 0..31, channel c) inside a chunk.
//   PV mma: row = channel, k = token.  ks = tau / 16 is the k-step, kh = (tau / 8) % 2, tid4 = (tau % 8) / 2,
//   tp = tau % 2.  Channels are dealt to fragment rows so that the 16 channels a lane owns are two
//   contiguous runs of 8 (c = 64*h + 8*gid + 2*k + rh): the same ownership an unquantised fp16 value row
//   gives when a lane loads its 16-byte pieces gid and gid + 8, so fp16 window tokens and packed tokens
//   accumulate into the same registers.  m-tile m = 4*h + k, rh = upper row half.
IQ_HD BitPos block_pos_plane(int tau, int c, int plane_bits) {
  int ks = tau >> 4, kh = (tau >> 3) & 1, j = (tau & 7) >> 1, tp = tau & 1;
  int m = 4 * (c >> 6) + ((c >> 1) & 3), gid = (c >> 3) & 7, rh = c & 1;
  int lane = 4 * gid + j;
  BitPos p;
  if (plane_bits == 2) {         // 8 words per lane: word = m; fields (rh, ks, kh)
    p.word = (m >> 2) * 128 + lane * 4 + (m & 3);
    p.bit = 16 * tp + 2 * (4 * rh + 2 * ks + kh);
  } else if (plane_bits == 4) {  // 16 words per lane: word = (ks, m); fields (rh, kh)
    p.word = ks * 256 + (m >> 2) * 128 + lane * 4 + (m & 3);
    p.bit = 16 * tp + 4 * (2 * rh + kh);
  } else {                       // 1-bit plane, 4 words per lane: word = m / 2; fields (m % 2, rh, ks, kh)
    p.word = lane * 4 + (m >> 1);
    p.bit = 16 * tp + (((m & 1) * 2 + rh) * 4 + 2 * ks + kh);
  }
  return p;
}

// ---- 2-bit codes in byte order (Store::perm = 1): operands of the integer tensor-core instruction m16n8k32 -------
// A byte holds four codes at bit positions 0, 2, 4, 6; `word & (0x03030303 << 2p)` is four 8-bit operand values
// (the codes at position p times 4^p; the factor is taken out after the sum).
// ROW store: byte k (0..31) of the 32-byte row holds channels k, 32 + k, 64 + k, 96 + k at positions 0..3, so that
// position p is one k-step of 32 channels = the p-th run of 32 channels (a whole group at G = 32).  The fragment of
// lane (gid, j) is bytes 4j..4j+3 and 16+4j..16+4j+3 of rows gid and gid + 8: the two words are stored next to each
// other (physical word 2j + h holds bytes 16h + 4j ..), one 64-bit load per row.
// 4-bit codes: a byte holds two codes (masks 0x0F0F0F0F / 0xF0F0F0F0, the high one times 16); the 64-byte row is two
// halves of 32 bytes, half h2 holding channel runs 2 h2 (low nibbles) and 2 h2 + 1 (high nibbles); a lane's four words
// per row (bytes 4j.. and 16+4j.. of both halves) are adjacent: one 128-bit load.
IQ_HD BitPos row_pos_i8(int c, int bits = 2) {
  const int p = c >> 5, k = c & 31, lw = k >> 2;
  BitPos r;
  if (bits == 4) {
    r.word = 4 * (lw & 3) + 2 * (p >> 1) + (lw >> 2);
    r.bit = 8 * (k & 3) + 4 * (p & 1);
  } else {
    r.word = 2 * (lw & 3) + (lw >> 2);
    r.bit = 8 * (k & 3) + 2 * p;
  }
  return r;
}
// BLOCK store: one chunk = one k-step of 32 tokens for each of 8 m-tiles of 16 channels.  Token tau sits at
// k = 4 * (tau % 8) + tau / 8 (the four tokens whose scores one lane holds after the key MMAs are adjacent in k).
// Channel c = 64 W + 8 gid + 2 p + rh is fragment row gid (rh = 0) or gid + 8 (rh = 1) of m-tile 4 W + p, the same
// ownership as with perm = 0; the four m-tiles 4 W .. 4 W + 3 share their words, one per bit position.
// Lane 4 gid + j holds words [W][2 * (k / 16) + rh] with bytes k % 4, for k / 4 % 4 == j.
// 4-bit codes: the two m-tiles 2 W, 2 W + 1 share their words (low / high nibble), W = 0 .. 3: 16 words per lane.
IQ_HD BitPos block_pos_i8(int tau, int c, int bits = 2) {
  const int k = 4 * (tau & 7) + (tau >> 3);
  const int m = 4 * (c >> 6) + ((c >> 1) & 3), gid = (c >> 3) & 7, rh = c & 1;
  const int j = (k & 15) >> 2, half = k >> 4;
  const int W = bits == 4 ? m >> 1 : m >> 2, p = bits == 4 ? m & 1 : m & 3;
  BitPos r;
  r.word = W * 128 + (4 * gid + j) * 4 + 2 * half + rh;
  r.bit = 8 * (k & 3) + bits * p;
  return r;
}

// 3-bit codes in byte order: a 2-bit plane laid out exactly as the 2-bit codes above (row words 0..7, chunk words
// 0..255) followed by a 1-bit plane (row words 8..11, chunk words 256..383).  The split of a code between the planes
// alternates with the bit position p of its 2-bit field, so that one bit-select of the two planes yields 3-bit fields
// that no shift has to align:
//   p even: 2-bit plane = code & 3,  1-bit plane = code >> 2, put right ABOVE the field: bits 4(p/2) + {0,1,2},
//           i.e. the code times 16^(p/2);
//   p odd:  2-bit plane = code >> 1, 1-bit plane = code & 1,  put right BELOW the field: bits 4(p/2) + {1,2,3},
//           i.e. the code times 2 * 16^(p/2).
// The 1-bit plane word of a lane pairs with two 2-bit words (ROW: h = 0, 1, the two k halves of a row; BLOCK: W = 0,
// 1, the two sets of four m-tiles); its bits for the first one sit where they are used (p = 0,1,2,3 -> bit 2,1,6,5 of
// the byte), those for the second one next to them (bit 3,0,7,4: `>> 1` for even p, `<< 1` for odd p).
IQ_HD int hi_bit_i8(int p, int second) {
  const int b = ((p & 1) ? 1 : 2) + 4 * (p >> 1);
  return second ? b + ((p & 1) ? -1 : 1) : b;
}
// weight of the 3-bit field of bit position p after the bit-select: 1, 2, 16, 32
IQ_HD int field_weight_i8_3(int p) { return (1 + (p & 1)) << (4 * (p >> 1)); }
struct BitPos3 { BitPos lo, hi; int odd; };      // positions in the two planes; odd: the split of the code (see above)
IQ_HD BitPos3 row_pos_i8_3(int c) {
  const int p = c >> 5, k = c & 31, lw = k >> 2, j = lw & 3, h = lw >> 2;
  BitPos3 r;
  r.lo.word = 2 * j + h;
  r.lo.bit = 8 * (k & 3) + 2 * p;
  r.hi.word = 8 + j;
  r.hi.bit = 8 * (k & 3) + hi_bit_i8(p, h);
  r.odd = p & 1;
  return r;
}
IQ_HD BitPos3 block_pos_i8_3(int tau, int c) {
  const int k = 4 * (tau & 7) + (tau >> 3);
  const int m = 4 * (c >> 6) + ((c >> 1) & 3), gid = (c >> 3) & 7, rh = c & 1;
  const int j = (k & 15) >> 2, half = k >> 4, W = m >> 2, p = m & 3;
  BitPos3 r;
  r.lo.word = W * 128 + (4 * gid + j) * 4 + 2 * half + rh;
  r.lo.bit = 8 * (k & 3) + 2 * p;
  r.hi.word = 256 + (4 * gid + j) * 4 + 2 * half + rh;
  r.hi.bit = 8 * (k & 3) + hi_bit_i8(p, W);
  r.odd = p & 1;
  return r;
}
// the two plane values of a 3-bit code, and the code from them
IQ_HD uint32_t code3_lo(uint32_t code, int odd) { return odd ? (code >> 1) & 3u : code & 3u; }
IQ_HD uint32_t code3_hi(uint32_t code, int odd) { return odd ? code & 1u : (code >> 2) & 1u; }
IQ_HD uint32_t code3_join(uint32_t lo, uint32_t hi, int odd) { return odd ? (lo << 1) | hi : lo | (hi << 2); }

// BLOCK store metadata: the 128 per-channel entries of a group are ordered so that the 16 channels a
// lane owns in the PV fragments are contiguous (entry 2*m + rh of lane gid): 4 x 128-bit loads.
IQ_HD int block_meta_index(int c) { return ((c >> 3) & 7) * 16 + (c >> 6) * 8 + (c & 7); }
IQ_HD int block_meta_channel(int pos) { return ((pos >> 3) & 1) * 64 + (pos >> 4) * 8 + (pos & 7); }
// channel of fragment row (m-tile m, row half rh) of lane group gid
IQ_HD int block_row_channel(int m, int rh, int gid) { return 64 * (m >> 2) + 8 * gid + 2 * (m & 3) + rh; }

IQ_HD int row_bytes(int bits) { return 16 * bits; }
IQ_HD int chunk_bytes(int bits) { return 512 * bits; }
// word offset of the 1-bit plane of a 3-bit row / chunk
IQ_HD int row_hi_plane_word() { return 8; }
IQ_HD int chunk_hi_plane_word() { return 256; }

}  // namespace iq
