// Interface between the host side of the fused decode kernel (innerq_decode_mma.cu) and the translation
// units that compile its kernels, one per packed format (innerq_decode_mma_k*v*_m*.cu).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "innerq_layout.h"

namespace iq {

// Launch parameters shared by every format's kernels (filled by launch_decode_mma).
struct DecodeArgs {
  const unsigned char* cache;
  unsigned char* ws;
  const __half* q;
  __half* out;
  int grid_y;            // grid rows (blockIdx.y) that work on this cache: the launch's gridDim.y, or fewer for a
                         // short sequence of a batched launch (the rows beyond it return at once)
  int n_splits;          // CTAs per unit that stream packed chunks (blockIdx.y < n_splits <= grid_y)
  int n_tail_tiles;      // tiles of 16 tokens outside the packed-K/packed-V range: skew tiles first, then fp16 tiles;
                         // tile x belongs to CTA x % grid_y, warp (x / grid_y) % 8
  int n_skew_tiles;      // of those, tiles whose keys are packed rows (values still fp16)
  int tiles_q0, tiles_rem;   // n_tail_tiles / grid_y and n_tail_tiles % grid_y
  int k_ring_pos0, v_ring_pos0;   // ring slot of the oldest recent key token / oldest fp16 value token
  int units_per_split;   // range units (max(value group, iteration) of chunks) per CTA, before the tail discount
  int tail_cost_units;   // a warp streams this many range units less per tail tile it handles (load balance)
  int safe_chunks;       // chunks [0, safe_chunks) of every unit were complete before the previous decode of this cache
                         // was launched: no kernel that may still be running writes them, so they are streamed
                         // before this kernel waits for its predecessors (programmatic dependent launch)
  int head0;             // first query row (within the KV head's r * n_q) handled by this launch
  int n_q;               // consecutive query tokens per sequence (1: plain decode).  Row v = i * r + h of a KV head is
                         // head h of query token i; q / out are [B, n_q, Hq, D]; query i does not see the newest
                         // n_q - 1 - i tokens (all of them outside the chunks where keys AND values are packed)
  int ablation;          // timing experiments only (results are then wrong on purpose): bit 0 leaves out the key side's
                         // unpack + MMA work of the streaming loop (scores are taken as 0), bit 1 the value side's
  float* partials;       // split partials [rows][max_splits][kPartialStride]: row = global query head (n_q == 1) or
                         // unit * 4 + column of the launch (n_q > 1)
  // HOST side only (paged caches): the cache's page list, which the launcher copies into the kernel's parameter
  // space when it fits (PageIds), so that no copy of a CTA waits for a look-up in the table in device memory
  const uint32_t* pages_host;
  int n_pages_host;
};

// A paged cache's table (pool page of every page slot) as a kernel parameter.
constexpr int kParamPages = 512;
struct PageIds {
  uint32_t id[kParamPages];
};

// Batched launch over several caches of one configuration, each with its own length (continuous batching):
// block x = sequence * U + unit; every sequence has its own token counts and launch parameters.
struct SeqArgs {
  Counts cn;
  DecodeArgs a;
};
struct SeqTable {
  SeqArgs s[kMaxSeqs];
};

// Launchers by format: k<key bits>v<value bits>_m<bytes per key metadata entry><bytes per value metadata entry>, every
// combination of 2 / 3 / 4-bit keys and values with 2-byte (scale only: symmetric mode) or 4-byte (scale | zero-point)
// metadata.  cpi: chunks of 32 tokens per loop iteration (0 = automatic).  Return the number of launches, or < 0.
// The _batched form takes a table of sequences (n_seqs <= kMaxSeqs entries with cn and the N-dependent fields of a).
#define IQ_FOR_EACH_META(X, KB, VB) X(KB, VB, 2, 2) X(KB, VB, 2, 4) X(KB, VB, 4, 2) X(KB, VB, 4, 4)
#define IQ_FOR_EACH_MMA_FORMAT(X)                                                                        \
  IQ_FOR_EACH_META(X, 2, 2)                                                                              \
  IQ_FOR_EACH_META(X, 2, 3) IQ_FOR_EACH_META(X, 2, 4) IQ_FOR_EACH_META(X, 3, 2) IQ_FOR_EACH_META(X, 3, 3) \
  IQ_FOR_EACH_META(X, 3, 4) IQ_FOR_EACH_META(X, 4, 2) IQ_FOR_EACH_META(X, 4, 3) IQ_FOR_EACH_META(X, 4, 4)
#define IQ_DECLARE_MMA_FORMAT(KB, VB, KM, VM)                                                                      \
  int launch_decode_mma_k##KB##v##VB##_m##KM##VM(const Layout& L, const Counts& cn, const DecodeArgs& a,          \
                                                 int n_splits, int cpi, cudaStream_t st);                           \
  int launch_decode_mma_k##KB##v##VB##_m##KM##VM##_batched(const Layout& L, SeqTable& T, int n_seqs, int n_splits, \
                                                           int cpi, cudaStream_t st);
IQ_FOR_EACH_MMA_FORMAT(IQ_DECLARE_MMA_FORMAT)
#undef IQ_DECLARE_MMA_FORMAT
int launch_decode_mma_outer_k2v2_batched(const Layout& L, SeqTable& T, int n_seqs, int n_splits, int cpi, cudaStream_t st);
int launch_decode_mma_outer_k4v4_batched(const Layout& L, SeqTable& T, int n_seqs, int n_splits, int cpi, cudaStream_t st);

// Outer-grouped comparison cache (same argument list; cpi is ignored).
int launch_decode_mma_outer_k2v2(const Layout& L, const Counts& cn, const DecodeArgs& a, int n_splits, int cpi, cudaStream_t st);
int launch_decode_mma_outer_k4v4(const Layout& L, const Counts& cn, const DecodeArgs& a, int n_splits, int cpi, cudaStream_t st);

}  // namespace iq
