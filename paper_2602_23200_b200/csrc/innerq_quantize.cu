// Quantise-side kernels: per-channel key norm, group quantisation into the ROW / BLOCK stores
// (prefill and quantise-on-evict share the same device routines), window copies, canonical export.
#include "innerq_device.cuh"
#include "innerq_kernels.h"

namespace iq {

// ------------------------------------------------------------------ key norm
// absmax[u][c] = max_t |K[u][t][c]| as fp32 bit patterns (non-negative floats order like uints).
__global__ void __launch_bounds__(256) k_absmax_kernel(const __half* __restrict__ K, int N, int rows_per_block,
                                                       uint32_t* __restrict__ absmax) {
  const int u = blockIdx.y;
  const int t0 = blockIdx.x * rows_per_block;
  const int t1 = min(N, t0 + rows_per_block);
  const int cg = threadIdx.x & 15;      // 8 channels each
  const int rg = threadIdx.x >> 4;      // 16 rows in flight
  const uint4* base = reinterpret_cast<const uint4*>(K + (size_t)u * N * kD);
  __half2 m[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) m[i] = __float2half2_rn(0.f);
  for (int t = t0 + rg; t < t1; t += 16) {
    uint4 v = __ldg(base + (size_t)t * 16 + cg);
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) m[i] = __hmax2(m[i], __habs2(h[i]));
  }
  __shared__ float red[16][kD];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    red[rg][cg * 8 + 2 * i] = __low2float(m[i]);
    red[rg][cg * 8 + 2 * i + 1] = __high2float(m[i]);
  }
  __syncthreads();
  if (threadIdx.x < kD) {
    float v = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) v = fmaxf(v, red[i][threadIdx.x]);
    atomicMax(absmax + (size_t)u * kD + threadIdx.x, __float_as_uint(v));
  }
}

// norm = sqrt(absmax), 0 -> 1  (Section "Per-channel Normalization of K"); the absmax word is replaced by the
// reciprocal 1 / norm (correctly rounded) that the quantisers multiply keys with
__global__ void finalize_norm_kernel(uint32_t* __restrict__ absmax, float* __restrict__ norm, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) {
    float n_ = __fsqrt_rn(__uint_as_float(absmax[i]));
    n_ = n_ == 0.f ? 1.0f : n_;
    norm[i] = n_;
    absmax[i] = __float_as_uint(__fdiv_rn(1.0f, n_));
  }
}

__global__ void fill_u32_kernel(uint32_t* p, uint32_t v, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}
__global__ void fill_float_kernel(float* p, float v, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = v;
}

// ------------------------------------------------------------------ ROW store quantiser
// One warp quantises one token (quantised row i of the unit whose record area is `rec`): lane l holds channels
// 4l..4l+3; a group of G channels is G/4 adjacent lanes.  `stage` is this warp's packed row in shared memory.
// `inv_norm4`: reciprocal key norms of this lane's four channels (1.0f / norm, correctly rounded), or null.
// Codes go to the token's packed row, or (chunk-coded tensor) are OR-ed into the token's 32-token chunk in
// global memory, whose words other tokens share: that area must be zero before its first token arrives.
__device__ __forceinline__ void quantize_row_warp(const __half* __restrict__ src, const float* __restrict__ inv_norm4,
                                                  const Layout& L, const Store& S, uint32_t* stage,
                                                  const Rec& rec, int i_row) {
  const int lane = threadIdx.x & 31;
  const int gl = L.G >> 2;   // lanes per group
  float x[4];
  {
    uint2 raw = *reinterpret_cast<const uint2*>(src + 4 * lane);
    const __half2* h = reinterpret_cast<const __half2*>(&raw);
    float2 a = __half22float2(h[0]), b = __half22float2(h[1]);
    x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
  }
  if (inv_norm4) {
#pragma unroll
    for (int i = 0; i < 4; ++i) x[i] = __fmul_rn(x[i], inv_norm4[i]);
  }
  float mn = fminf(fminf(x[0], x[1]), fminf(x[2], x[3]));
  float mx = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
  float am = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
  for (int o = gl >> 1; o > 0; o >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
  }
  GroupParams p = group_params(mn, mx, am, S.bits, L.sym_variant);
  float ua[4], qs[4], ea = 0.f, es = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    ua[i] = asym_code(p, x[i]);
    qs[i] = sym_code(p, x[i]);
    ea += asym_err(p, x[i], ua[i]);
    es += sym_err(p, x[i], qs[i]);
  }
  for (int o = gl >> 1; o > 0; o >>= 1) {
    ea += __shfl_xor_sync(0xffffffffu, ea, o);
    es += __shfl_xor_sync(0xffffffffu, es, o);
  }
  const bool asym = choose_asym(S.mode, ea, es);
  if (S.code_kind == kRow) {
    const int words = row_bytes(S.bits) / 4;
    uint32_t* dst_row = reinterpret_cast<uint32_t*>(row_code_ptr(rec, S, i_row));
    if (lane < words) stage[lane] = 0u;
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t code = (uint32_t)(int)(asym ? ua[i] : qs[i] + p.half);
      row_put(stage, 4 * lane + i, S.bits, code, S.perm);
    }
    __syncwarp();
    if (lane < words) dst_row[lane] = stage[lane];
  } else {
    uint32_t* chunk = reinterpret_cast<uint32_t*>(block_code_ptr(rec, S, i_row / kChunk));
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t code = (uint32_t)(int)(asym ? ua[i] : qs[i] + p.half);
      chunk_put(chunk, i_row % kChunk, 4 * lane + i, S.bits, code, S.perm);
    }
  }
  if ((lane % gl) == 0) store_meta(row_meta_ptr(rec, S, i_row), lane / gl, S.meta_bytes, group_meta(p, asym));
  __syncwarp();
}

// ------------------------------------------------------------------ BLOCK store quantiser
// A 128-thread CTA quantises one group of G tokens x 128 channels; thread c owns channel c.
// tile: fp16 [G][D] staging; words: the group's packed chunks, or its packed rows (row-coded tensor), zeroed here.
__device__ void quantize_block_cta(const TokSrc& src, int t_first, const float* __restrict__ norm, const Layout& L,
                                   const Store& S, __half* tile, uint32_t* words, const Rec& rec, int group_j) {
  const int G = L.G, c = threadIdx.x;
  const int cw = chunk_bytes(S.bits) / 4, rw = row_bytes(S.bits) / 4;
  const bool rows = S.code_kind == kRow;
  const int n_words = (G / kChunk) * cw;                   // = G * rw
  for (int i = threadIdx.x; i < G * 16; i += 128) {        // 16 x 16-byte pieces per token row
    int t = i >> 4, piece = i & 15;
    reinterpret_cast<uint4*>(tile)[i] = *reinterpret_cast<const uint4*>(src.row(t_first + t) + piece * 8);
  }
  for (int i = threadIdx.x; i < n_words; i += 128) words[i] = 0u;
  __syncthreads();
  const float inv = norm ? __fdiv_rn(1.0f, norm[c]) : 1.0f;
  float mn = INFINITY, mx = -INFINITY, am = 0.f;
  for (int t = 0; t < G; ++t) {
    float x = __half2float(tile[t * kD + c]);
    if (norm) x = __fmul_rn(x, inv);
    mn = fminf(mn, x); mx = fmaxf(mx, x); am = fmaxf(am, fabsf(x));
  }
  GroupParams p = group_params(mn, mx, am, S.bits, L.sym_variant);
  float ea = 0.f, es = 0.f;
  if (S.mode == 2) {
    for (int t = 0; t < G; ++t) {
      float x = __half2float(tile[t * kD + c]);
      if (norm) x = __fmul_rn(x, inv);
      ea += asym_err(p, x, asym_code(p, x));
      es += sym_err(p, x, sym_code(p, x));
    }
  }
  const bool asym = choose_asym(S.mode, ea, es);
  for (int t = 0; t < G; ++t) {
    float x = __half2float(tile[t * kD + c]);
    if (norm) x = __fmul_rn(x, inv);
    uint32_t code = (uint32_t)(int)(asym ? asym_code(p, x) : sym_code(p, x) + p.half);
    if (rows) row_put(words + t * rw, c, S.bits, code, S.perm);
    else chunk_put(words + (t / kChunk) * cw, t % kChunk, c, S.bits, code, S.perm);
  }
  store_meta(block_meta_ptr(rec, S, group_j), block_meta_index(c), S.meta_bytes, group_meta(p, asym));
  __syncthreads();
  for (int i = threadIdx.x; i < n_words; i += 128) {
    if (rows) {
      const int t = i / rw;
      reinterpret_cast<uint32_t*>(row_code_ptr(rec, S, group_j * G + t))[i - t * rw] = words[i];
    } else {
      const int ch = i / cw;
      reinterpret_cast<uint32_t*>(block_code_ptr(rec, S, group_j * (G / kChunk) + ch))[i - ch * cw] = words[i];
    }
  }
  __syncthreads();
}

// Prefill with these generic routines (tensors whose code layout differs from their grouping: the outer-grouped
// comparison cache).  One warp per token / one CTA per group of G tokens.
__global__ void __launch_bounds__(128) quantize_rows_generic_kernel(Layout L, Store S, const __half* __restrict__ X, int N,
                                                                    int n_q, unsigned char* __restrict__ cache) {
  __shared__ uint32_t stage[4][16];
  const int u = blockIdx.y, warp = threadIdx.x >> 5;
  const Rec rec = unit_rec(L, cache, u);
  for (int i = blockIdx.x * 4 + warp; i < n_q; i += gridDim.x * 4)
    quantize_row_warp(X + ((size_t)u * N + L.w_sink + i) * kD, nullptr, L, S, stage[warp], rec, i);
}
__global__ void __launch_bounds__(128) quantize_blocks_generic_kernel(Layout L, Store S, const __half* __restrict__ X,
                                                                      int N, int n_q, unsigned char* __restrict__ cache) {
  __shared__ __align__(16) __half tile[128 * kD];
  __shared__ uint32_t words[4 * 512];
  const int u = blockIdx.y;
  const Rec rec = unit_rec(L, cache, u);
  TokSrc src{X + (size_t)u * N * kD, 0, 0};
  for (int j = blockIdx.x; j < n_q / L.G; j += gridDim.x)
    quantize_block_cta(src, L.w_sink + j * L.G, nullptr, L, S, tile, words, rec, j);
}

// Paged record area: zeroes the pool page of page slot blockIdx.y.
__global__ void zero_pages_kernel(Layout L, const unsigned char* __restrict__ cache) {
  const uint32_t page = reinterpret_cast<const uint32_t*>(cache + L.page_table_off)[blockIdx.y];
  uint4* dst = reinterpret_cast<uint4*>(L.pool + (size_t)page * L.page_bytes);
  const size_t n = L.page_bytes / 16;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = make_uint4(0u, 0u, 0u, 0u);
}

// ------------------------------------------------------------------ window copies (prefill)
// Copies tokens [t0, t1) of the input into the sink (t < w_sink) or the recent ring.
__global__ void copy_window_kernel(Layout L, Store S, const __half* __restrict__ X, int N, int t0, int t1,
                                   unsigned char* __restrict__ cache) {
  const int u = blockIdx.y;
  const int n = (t1 - t0) * 16;
  __half* sink = reinterpret_cast<__half*>(cache + S.sink_off + (size_t)u * S.sink_stride);
  __half* ring = reinterpret_cast<__half*>(cache + S.ring_off + (size_t)u * S.ring_stride);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    int t = t0 + (i >> 4), piece = i & 15;
    uint4 v = *reinterpret_cast<const uint4*>(X + ((size_t)u * N + t) * kD + piece * 8);
    __half* dst = t < L.w_sink ? sink + (size_t)t * kD : ring + (size_t)((t - L.w_sink) % S.ring_cap) * kD;
    *reinterpret_cast<uint4*>(dst + piece * 8) = v;
  }
}

// ------------------------------------------------------------------ append (quantise-on-evict)
// N is the token count after this append.  Which evictions happen is a function of N alone.
// One CTA of 128 threads per unit.  The per-step work (ring writes, eviction of one ROW-store token) is a chain of
// dependent memory accesses, so everything whose address is known up front is requested at once: the new key and
// value rows, the evicted token's row (in the ring since w_recent steps, or the new row itself if w_recent = 0)
// and the key norms.  Warp 0 quantises the ROW store's evicted token while the others write the rings; the BLOCK
// store's eviction (G tokens, every G steps) then runs on the whole CTA.

// ROW store: eviction of its oldest recent token, if this append causes one (warp 0 only).
__device__ __forceinline__ void append_evict_row(const Layout& L, const Store& R, const __half* __restrict__ x_new, int N,
                                                 int u, unsigned char* __restrict__ cache, bool use_norm, uint32_t* words) {
  const int t_new = N - 1;
  if (R.kind != kRow || t_new < L.w_sink || threadIdx.x >= 32) return;
  const int nq_before = n_quantised(kRow, N - 1, L.w_sink, L.w_recent, L.G);
  if (n_quantised(kRow, N, L.w_sink, L.w_recent, L.G) == nq_before) return;
  const __half* ring = reinterpret_cast<const __half*>(cache + R.ring_off + (size_t)u * R.ring_stride);
  const float* norm = reinterpret_cast<const float*>(cache + L.norm_off) + (size_t)u * kD;
  float inv4[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) inv4[e] = use_norm ? __fdiv_rn(1.0f, norm[4 * threadIdx.x + e]) : 1.0f;
  const Rec rec = unit_rec(L, cache, u);
  TokSrc src{ring, R.ring_cap, L.w_sink};
  // with an empty recent window the evicted token is the new one, which is not in the ring yet
  const __half* row = L.w_sink + nq_before == t_new ? x_new : src.row(L.w_sink + nq_before);
  quantize_row_warp(row, use_norm ? inv4 : nullptr, L, R, words, rec, nq_before);
}

// The new token goes to the sink or the ring of the store.
__device__ __forceinline__ void append_write(const Layout& L, const Store& R, __half x, int N, int u,
                                             unsigned char* __restrict__ cache) {
  const int t_new = N - 1;
  __half* sink = reinterpret_cast<__half*>(cache + R.sink_off + (size_t)u * R.sink_stride);
  __half* ring = reinterpret_cast<__half*>(cache + R.ring_off + (size_t)u * R.ring_stride);
  if (R.kind == kNone || t_new < L.w_sink) sink[(size_t)t_new * kD + threadIdx.x] = x;
  else ring[(size_t)((t_new - L.w_sink) % R.ring_cap) * kD + threadIdx.x] = x;
}

// BLOCK store: every G steps the oldest G tokens of its ring (the row written by this append may be among them).
__device__ __forceinline__ void append_evict_block(const Layout& L, const Store& R, int N, int u,
                                                   unsigned char* __restrict__ cache, bool use_norm, __half* tile,
                                                   uint32_t* words) {
  if (R.kind != kBlock || N - 1 < L.w_sink) return;
  const int nq_before = n_quantised(kBlock, N - 1, L.w_sink, L.w_recent, L.G);
  if (n_quantised(kBlock, N, L.w_sink, L.w_recent, L.G) == nq_before) return;
  __syncthreads();
  const float* norm = use_norm ? reinterpret_cast<const float*>(cache + L.norm_off) + (size_t)u * kD : nullptr;
  const __half* ring = reinterpret_cast<const __half*>(cache + R.ring_off + (size_t)u * R.ring_stride);
  TokSrc src{ring, R.ring_cap, L.w_sink};
  quantize_block_cta(src, L.w_sink + nq_before, norm, L, R, tile, words, unit_rec(L, cache, u),
                     nq_before / L.G);
}

// One appended token of one unit: ring write of the new key / value rows, eviction of the oldest key row and, when
// a group of G tokens has filled up, of the oldest G value rows (outer grouping: the other way round).
// Publish: everything this unit's append writes is written.  A decode of N tokens that reads N in the unit's counter
// (acquire) may read the rings and the newest packed rows without waiting for this kernel to end.  The packed rows
// will be read by bulk async copies (another memory proxy than these ordinary stores): every thread orders its
// stores ahead of that proxy first.  n_parts CTAs share the unit's append (one, or five on the step that packs a
// chunk-coded group): each takes a ticket after its writes, the last one publishes.
__device__ __forceinline__ void append_publish(const Layout& L, int N, int u, unsigned char* __restrict__ cache, int n_parts) {
  asm volatile("fence.proxy.async.global;" ::: "memory");
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t* counts = reinterpret_cast<uint32_t*>(cache + L.appended_off);
    __threadfence();
    if (n_parts > 1) {
      if (atomicAdd(counts + L.U + u, 1u) != (uint32_t)(n_parts - 1)) return;
      counts[L.U + u] = 0u;          // ready for the next append
      __threadfence();               // the other parts' writes (published before their tickets) precede the count
    }
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(counts + u), "r"((uint32_t)N) : "memory");
  }
}

// skip_v_block: the value store's group eviction of this step is done by other CTAs (quarters, see append_kernel)
__device__ __forceinline__ void append_unit(const Layout& L, const __half* __restrict__ xk, const __half* __restrict__ xv,
                                            int N, int u, unsigned char* __restrict__ cache, __half* tile, uint32_t* words,
                                            bool skip_v_block = false, int n_parts = 1) {
  const __half k_x = xk[threadIdx.x], v_x = xv[threadIdx.x];
  const bool k_norm = L.k_normalize != 0;
  append_evict_row(L, L.k, xk, N, u, cache, k_norm, words);
  append_evict_row(L, L.v, xv, N, u, cache, false, words);
  append_write(L, L.k, k_x, N, u, cache);
  append_write(L, L.v, v_x, N, u, cache);
  append_evict_block(L, L.k, N, u, cache, k_norm, tile, words);
  if (!skip_v_block) append_evict_block(L, L.v, N, u, cache, false, tile, words);
  append_publish(L, N, u, cache, n_parts);
}

// Quarter of a group eviction of a chunk-coded BLOCK store: 32 channels of the G oldest ring tokens (first token
// t_first; the row appended by this very step, token N - 1, is taken from the call's input x_new, which another CTA
// is writing to the ring at the same time).  128 threads: lane = channel of the quarter, warp = quarter of the tokens.
// The quarters write disjoint words of the packed chunks.  Pair order (perm = 0): quarter q = channels 32 q ..
// 32 q + 31; a word belongs to one lane group gid and one half W of the channels (see block_pos_plane).  Byte order
// (perm = 1): a word belongs to one lane group gid, and the 1-bit plane of 3-bit codes holds both halves W in one
// word, so quarter q is the channels of lane groups 2 q and 2 q + 1: 16 q .. 16 q + 15 and 64 + 16 q .. 64 + 16 q + 15.
__device__ __forceinline__ int quarter_channel(int q, int cl, int perm) {      // channel of lane cl of quarter q
  return perm == 1 ? 64 * (cl >> 4) + 16 * q + (cl & 15) : 32 * q + cl;
}
__device__ __forceinline__ int chunk_word_quarter(int i, int bits, int perm) {
  if (perm == 1) return (i & 127) >> 5;                    // word = set * 128 + lane * 4 + role, gid = lane / 4
  if (bits == 3 && i >= chunk_hi_plane_word()) {
    const int r = i - chunk_hi_plane_word();
    return 2 * ((r & 3) >> 1) + ((r >> 2) >> 4);          // word = lane * 4 + (m >> 1), m >> 1 = 2 W + ..; gid = lane / 4
  }
  const int r = i & 255;                                   // 4-bit codes in pair order: two k-step halves of 256 words
  return 2 * (r >> 7) + (((r & 127) >> 2) >> 4);           // W = r / 128, gid = ((r % 128) / 4) / 4 -> 2 W + gid / 4
}
__device__ void quantize_block_quarter(const TokSrc& src, const __half* __restrict__ x_new, int t_new, int t_first,
                                       const Layout& L, const Store& S, __half* tile, uint32_t* words, float* red,
                                       const Rec& rec, int group_j, int q) {
  const int G = L.G, cl = threadIdx.x & 31, part = threadIdx.x >> 5, c = quarter_channel(q, cl, S.perm);
  const int cw = chunk_bytes(S.bits) / 4, n_words = (G / kChunk) * cw, per = G >> 2;
  for (int i = threadIdx.x; i < G * 4; i += 128) {         // 4 x 16-byte pieces of the quarter per token row
    const int t = i >> 2, piece = i & 3;
    const __half* row = t_first + t == t_new ? x_new : src.row(t_first + t);
    reinterpret_cast<uint4*>(tile)[i] = *reinterpret_cast<const uint4*>(row + quarter_channel(q, piece * 8, S.perm));
  }
  for (int i = threadIdx.x; i < n_words; i += 128) words[i] = 0u;
  __syncthreads();
  float mn = INFINITY, mx = -INFINITY;
  for (int t = part * per; t < (part + 1) * per; ++t) {
    const float x = __half2float(tile[t * 32 + cl]);
    mn = fminf(mn, x); mx = fmaxf(mx, x);
  }
  red[(part * 32 + cl) * 2] = mn; red[(part * 32 + cl) * 2 + 1] = mx;
  __syncthreads();
  for (int pp = 0; pp < 4; ++pp) { mn = fminf(mn, red[(pp * 32 + cl) * 2]); mx = fmaxf(mx, red[(pp * 32 + cl) * 2 + 1]); }
  const GroupParams p = group_params(mn, mx, fmaxf(fabsf(mn), fabsf(mx)), S.bits, L.sym_variant);
  float ea = 0.f, es = 0.f;
  if (S.mode == 2) {
    for (int t = part * per; t < (part + 1) * per; ++t) {
      const float x = __half2float(tile[t * 32 + cl]);
      ea += asym_err(p, x, asym_code(p, x));
      es += sym_err(p, x, sym_code(p, x));
    }
    __syncthreads();                                       // the minima / maxima have been read
    red[(part * 32 + cl) * 2] = ea; red[(part * 32 + cl) * 2 + 1] = es;
    __syncthreads();
    ea = 0.f; es = 0.f;
    for (int pp = 0; pp < 4; ++pp) { ea += red[(pp * 32 + cl) * 2]; es += red[(pp * 32 + cl) * 2 + 1]; }
  }
  const bool asym = choose_asym(S.mode, ea, es);
  for (int t = part * per; t < (part + 1) * per; ++t) {
    const float x = __half2float(tile[t * 32 + cl]);
    const uint32_t code = (uint32_t)(int)(asym ? asym_code(p, x) : sym_code(p, x) + p.half);
    chunk_put(words + (t / kChunk) * cw, t % kChunk, c, S.bits, code, S.perm);
  }
  if (part == 0) store_meta(block_meta_ptr(rec, S, group_j), block_meta_index(c), S.meta_bytes, group_meta(p, asym));
  __syncthreads();
  for (int i = threadIdx.x; i < n_words; i += 128) {
    const int ch = i / cw, wi = i - ch * cw;
    if (chunk_word_quarter(wi, S.bits, S.perm) == q)
      reinterpret_cast<uint32_t*>(block_code_ptr(rec, S, group_j * (G / kChunk) + ch))[wi] = words[i];
  }
}

// Programmatic dependent launch: the decode that follows may start while this kernel runs (it streams what this
// kernel cannot write and waits for this kernel's completion before it touches the rest).  This kernel in turn
// waits for the kernels before it, either before its first global access or, with late_wait (the host knows that
// the last kernel on this cache was a fused decode, which lets its dependents start only after its last read of
// what an append writes: the fp16 rings and the packed rows / groups behind the range it streams), after its work:
// it then runs while that decode streams the packed cache.  The kernel still completes after that decode, so that
// whatever follows sees both finished: the CTA of unit 0 waits at its end; the others leave (and free their SM
// slots for the next decode's first CTAs) as soon as their unit's token count is published.
__global__ void __launch_bounds__(128) append_kernel(Layout L, const __half* __restrict__ k_new,
                                                     const __half* __restrict__ v_new, int N,
                                                     unsigned char* __restrict__ cache, int late_wait) {
  extern __shared__ __align__(16) unsigned char append_smem[];      // see append_smem_bytes
  __half* tile = reinterpret_cast<__half*>(append_smem);
  uint32_t* words = reinterpret_cast<uint32_t*>(append_smem + (size_t)L.G * kD * 2);
  const int u = blockIdx.x;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (!late_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
  // gridDim.y = 5 on the step that packs a group of G value tokens (inner grouping): row 0 does the per-token work,
  // rows 1 .. 4 a quarter of the group's channels each, so that this step costs about as much as any other
  const int n_parts = gridDim.y;
  if (blockIdx.y == 0) {
    append_unit(L, k_new + (size_t)u * kD, v_new + (size_t)u * kD, N, u, cache, tile, words, n_parts > 1, n_parts);
  } else {
    const Store& R = L.v;
    const int nq_before = n_quantised(kBlock, N - 1, L.w_sink, L.w_recent, L.G);
    const __half* ring = reinterpret_cast<const __half*>(cache + R.ring_off + (size_t)u * R.ring_stride);
    TokSrc src{ring, R.ring_cap, L.w_sink};
    quantize_block_quarter(src, v_new + (size_t)u * kD, N - 1, L.w_sink + nq_before, L, R, tile, words,
                           reinterpret_cast<float*>(words + (L.G / kChunk) * 512), unit_rec(L, cache, u), nq_before / L.G,
                           blockIdx.y - 1);
    append_publish(L, N, u, cache, n_parts);
  }
  // one CTA keeps the kernel alive until its predecessor has ended (the chain of completions); the others leave
  if (late_wait && u == 0 && blockIdx.y == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// The same for several caches of one configuration, each with its own token count: block x = sequence * U + unit,
// k_new / v_new are [n][U][D].
struct AppendSeq {
  unsigned char* cache;
  int N;           // token count after this append
  int late_wait;   // as for append_kernel
};
struct AppendTable {
  AppendSeq s[kMaxSeqs];
};
__global__ void __launch_bounds__(128) append_batched_kernel(const __grid_constant__ Layout L,
                                                             const __half* __restrict__ k_new,
                                                             const __half* __restrict__ v_new,
                                                             const __grid_constant__ AppendTable T) {
  extern __shared__ __align__(16) unsigned char append_smem[];
  __half* tile = reinterpret_cast<__half*>(append_smem);
  uint32_t* words = reinterpret_cast<uint32_t*>(append_smem + (size_t)L.G * kD * 2);
  const int seq = blockIdx.x / L.U, u = blockIdx.x - seq * L.U;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int late_wait = T.s[seq].late_wait;
  if (!late_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
  append_unit(L, k_new + (size_t)blockIdx.x * kD, v_new + (size_t)blockIdx.x * kD, T.s[seq].N, u, T.s[seq].cache, tile, words);
  if (late_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ------------------------------------------------------------------ canonical export
__global__ void export_store_kernel(Layout L, Store S, const unsigned char* __restrict__ cache, int n_q, int n_sink,
                                    int n_recent, uint8_t* __restrict__ code, uint16_t* __restrict__ scale,
                                    uint16_t* __restrict__ zero, uint16_t* __restrict__ sink_out,
                                    uint16_t* __restrict__ recent_out) {
  const int u = blockIdx.y;
  const int cap = L.max_tokens;
  const Rec rec = unit_rec(L, cache, u);
  const int stride = gridDim.x * blockDim.x, tid0 = blockIdx.x * blockDim.x + threadIdx.x;
  if (code && S.kind != kNone) {
    for (int i = tid0; i < n_q * kD; i += stride) {
      int t = i / kD, c = i % kD;
      uint32_t v = S.code_kind == kRow
                       ? row_code(reinterpret_cast<const uint32_t*>(row_code_ptr(rec, S, t)), c, S.bits, S.perm)
                       : chunk_code(reinterpret_cast<const uint32_t*>(block_code_ptr(rec, S, t / kChunk)), t % kChunk, c,
                                    S.bits, S.perm);
      code[((size_t)u * cap + t) * kD + c] = (uint8_t)v;
    }
  }
  if (S.kind != kNone) {
    const int n_meta_rows = S.kind == kRow ? n_q : n_q / L.G;
    const int rows_cap = S.kind == kRow ? cap : cap / L.G + 1;
    for (int i = tid0; i < n_meta_rows * S.n_groups; i += stride) {
      const int mr = i / S.n_groups, me = i % S.n_groups;
      uint32_t m = S.kind == kRow ? load_meta(row_meta_ptr(rec, S, mr), me, S.meta_bytes)
                                  : load_meta(block_meta_ptr(rec, S, mr), me, S.meta_bytes);
      const int ic = S.kind == kRow ? i : mr * kD + block_meta_channel(me);   // canonical position
      size_t o = (size_t)u * rows_cap * S.n_groups + ic;
      if (scale) scale[o] = (uint16_t)(m & 0xFFFFu);
      if (zero) zero[o] = (uint16_t)(m >> 16);
    }
  }
  const uint16_t* sink = reinterpret_cast<const uint16_t*>(cache + S.sink_off + (size_t)u * S.sink_stride);
  const uint16_t* ring = reinterpret_cast<const uint16_t*>(cache + S.ring_off + (size_t)u * S.ring_stride);
  const int sink_cap = S.kind == kNone ? L.max_tokens : L.w_sink;
  if (sink_out)
    for (int i = tid0; i < n_sink * kD; i += stride) sink_out[(size_t)u * sink_cap * kD + i] = sink[i];
  if (recent_out && S.kind != kNone) {
    const int t_first = n_sink + n_q;   // absolute token of the oldest recent entry
    for (int i = tid0; i < n_recent * kD; i += stride) {
      int t = t_first + i / kD, c = i % kD;
      recent_out[(size_t)u * (L.w_recent + L.G) * kD + i] = ring[(size_t)((t - L.w_sink) % S.ring_cap) * kD + c];
    }
  }
}

// ------------------------------------------------------------------ canonical import (the inverse of the export)
// Pass 0 clears the packed rows / chunks of the first n_q tokens (the codes are OR-ed in), pass 1 writes codes,
// metadata and the fp16 windows from the canonical arrays (same shapes as export_store_kernel's).
__global__ void import_store_kernel(Layout L, Store S, unsigned char* __restrict__ cache, int n_q, int n_sink, int n_recent,
                                    const uint8_t* __restrict__ code, const uint16_t* __restrict__ scale,
                                    const uint16_t* __restrict__ zero, const uint16_t* __restrict__ sink_in,
                                    const uint16_t* __restrict__ recent_in, int pass) {
  const int u = blockIdx.y;
  const int cap = L.max_tokens;
  const Rec rec = unit_rec(L, cache, u);
  const int stride = gridDim.x * blockDim.x, tid0 = blockIdx.x * blockDim.x + threadIdx.x;
  if (S.kind != kNone && pass == 0) {
    if (S.code_kind == kRow) {
      const int rw = row_bytes(S.bits) / 4;
      for (int i = tid0; i < n_q * rw; i += stride) reinterpret_cast<uint32_t*>(row_code_ptr(rec, S, i / rw))[i % rw] = 0u;
    } else {
      const int cw = chunk_bytes(S.bits) / 4, n_ch = (n_q + kChunk - 1) / kChunk;
      for (int i = tid0; i < n_ch * cw; i += stride) reinterpret_cast<uint32_t*>(block_code_ptr(rec, S, i / cw))[i % cw] = 0u;
    }
    return;
  }
  if (S.kind != kNone) {
    for (int i = tid0; i < n_q * kD; i += stride) {
      const int t = i / kD, c = i % kD;
      const uint32_t v = code[((size_t)u * cap + t) * kD + c];
      if (S.code_kind == kRow) row_put(reinterpret_cast<uint32_t*>(row_code_ptr(rec, S, t)), c, S.bits, v, S.perm);
      else chunk_put(reinterpret_cast<uint32_t*>(block_code_ptr(rec, S, t / kChunk)), t % kChunk, c, S.bits, v, S.perm);
    }
    const int n_meta_rows = S.kind == kRow ? n_q : n_q / L.G;
    const int rows_cap = S.kind == kRow ? cap : cap / L.G + 1;
    for (int i = tid0; i < n_meta_rows * S.n_groups; i += stride) {
      const int mr = i / S.n_groups, me = i % S.n_groups;
      const int ic = S.kind == kRow ? i : mr * kD + block_meta_channel(me);   // canonical position
      const size_t o = (size_t)u * rows_cap * S.n_groups + ic;
      const uint32_t m = (uint32_t)scale[o] | ((uint32_t)(zero ? zero[o] : 0) << 16);
      if (S.kind == kRow) store_meta(row_meta_ptr(rec, S, mr), me, S.meta_bytes, m);
      else store_meta(block_meta_ptr(rec, S, mr), me, S.meta_bytes, m);
    }
  }
  uint16_t* sink = reinterpret_cast<uint16_t*>(cache + S.sink_off + (size_t)u * S.sink_stride);
  uint16_t* ring = reinterpret_cast<uint16_t*>(cache + S.ring_off + (size_t)u * S.ring_stride);
  const int sink_cap = S.kind == kNone ? L.max_tokens : L.w_sink;
  for (int i = tid0; i < n_sink * kD; i += stride) sink[i] = sink_in[(size_t)u * sink_cap * kD + i];
  if (S.kind != kNone) {
    const int t_first = n_sink + n_q;   // absolute token of the oldest recent entry
    for (int i = tid0; i < n_recent * kD; i += stride) {
      const int t = t_first + i / kD, c = i % kD;
      ring[(size_t)((t - L.w_sink) % S.ring_cap) * kD + c] = recent_in[(size_t)u * (L.w_recent + L.G) * kD + i];
    }
  }
}

// ------------------------------------------------------------------ host launchers
static inline int grid_for(int n, int per_block, int cap) {
  int g = (n + per_block - 1) / per_block;
  return g < 1 ? 1 : (g > cap ? cap : g);
}

int launch_prefill(const Layout& L, unsigned char* cache, unsigned char* ws, const __half* K, const __half* V, int N,
                   cudaStream_t st) {
  int launches = 0;
  const Counts cn = counts_for(L, N);
  float* norm = reinterpret_cast<float*>(cache + L.norm_off);
  const bool use_norm = L.k_normalize != 0 && L.k.kind != kNone;
  if (use_norm && N > 0) {
    uint32_t* absmax = reinterpret_cast<uint32_t*>(ws + L.ws_absmax_off);
    if (cudaMemsetAsync(absmax, 0, (size_t)L.U * kD * 4, st) != cudaSuccess) return -1;
    const int rows_per_block = 512;
    dim3 g((N + rows_per_block - 1) / rows_per_block, L.U);
    k_absmax_kernel<<<g, 256, 0, st>>>(K, N, rows_per_block, absmax);
    finalize_norm_kernel<<<(L.U * kD + 255) / 256, 256, 0, st>>>(absmax, norm, L.U * kD);
    launches += 2;
  } else {
    fill_float_kernel<<<(L.U * kD + 255) / 256, 256, 0, st>>>(norm, 1.0f, L.U * kD);
    launches += 1;
  }
  if (L.k.kind != kNone && L.k.code_kind != L.k.kind) {
    // chunk words of the outer-grouped cache are filled token by token with OR: they start from zero
    if (L.page_groups == 0) {
      if (cudaMemsetAsync(cache + L.k.rec_off, 0, L.k.rec_unit_stride * L.U, st) != cudaSuccess) return -1;
    } else {      // the pages this prefill fills (the caller has assigned them)
      const int n_rec = cn.n_qk > cn.n_qv ? cn.n_qk : cn.n_qv;
      const int n_pages = ((n_rec + L.G - 1) / L.G + L.page_groups - 1) / L.page_groups;
      if (n_pages > 0) {
        zero_pages_kernel<<<dim3(64, n_pages), 256, 0, st>>>(L, cache);
        launches += 1;
      }
    }
  }
  const Store* stores[2] = {&L.k, &L.v};
  const __half* srcs[2] = {K, V};
  const int nq[2] = {cn.n_qk, cn.n_qv};
  for (int i = 0; i < 2; ++i) {
    const Store& S = *stores[i];
    if (N == 0) break;
    if (S.kind == kNone) {      // unquantised: the whole input goes to the "sink" array
      Layout Lf = L;
      Lf.w_sink = L.max_tokens;
      copy_window_kernel<<<dim3(grid_for(N * 16, 256, 1024), L.U), 256, 0, st>>>(Lf, S, srcs[i], N, 0, N, cache);
      launches += 1;
      continue;
    }
    const bool nrm = use_norm && i == 0;
    if (nq[i] > 0 && S.code_kind != S.kind) {      // outer-grouped comparison cache: generic routines, no key norm
      if (S.kind == kRow)
        quantize_rows_generic_kernel<<<dim3(grid_for(nq[i], 4 * 8, 4096), L.U), 128, 0, st>>>(L, S, srcs[i], N, nq[i], cache);
      else
        quantize_blocks_generic_kernel<<<dim3(grid_for(nq[i] / L.G, 1, 8192), L.U), 128, 0, st>>>(L, S, srcs[i], N, nq[i],
                                                                                               cache);
      launches += 1;
    } else if (nq[i] > 0) {
      const float* inv_norm = nrm ? reinterpret_cast<const float*>(ws + L.ws_absmax_off) : nullptr;
      if (launch_quantize_store_prefill(L, S, srcs[i], N, nq[i], cache, inv_norm, st) < 0) return -1;
      launches += 1;
    }
    // fp16 windows: sink, then everything after the quantised middle
    if (cn.n_sink > 0) {
      copy_window_kernel<<<dim3(1, L.U), 256, 0, st>>>(L, S, srcs[i], N, 0, cn.n_sink, cache);
      launches += 1;
    }
    const int t_rec = cn.n_sink + nq[i];
    if (N > t_rec) {
      copy_window_kernel<<<dim3(grid_for((N - t_rec) * 16, 256, 64), L.U), 256, 0, st>>>(L, S, srcs[i], N, t_rec, N, cache);
      launches += 1;
    }
  }
  // the counts the decode kernel compares with its own N (see append_unit)
  fill_u32_kernel<<<(L.U + 255) / 256, 256, 0, st>>>(reinterpret_cast<uint32_t*>(cache + L.appended_off), (uint32_t)N, L.U);
  launches += 1;
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// Shared memory of an append CTA: the fp16 staging tile of one group of G tokens and the group's packed words (a
// 32-token chunk is at most 512 words; a row-coded group G rows of at most 16 words).  Sized by G, not for the
// largest G: with G = 32 four of these CTAs fit beside a resident decode CTA, so the append of every unit of the
// benchmark shapes runs while the previous decode is still streaming.
static size_t append_smem_bytes(const Layout& L) {
  return (size_t)L.G * kD * 2 + (size_t)(L.G / kChunk) * 512 * 4 + 4 * 32 * 2 * 4;      // + the quarters' reduction words
}

int launch_append(const Layout& L, unsigned char* cache, const __half* k_new, const __half* v_new, int N_after,
                  cudaStream_t st, int late_wait) {
  cudaLaunchConfig_t cfg = {};
  // the step on which a chunk-coded group of G value tokens is packed gets four more CTAs per unit (see append_kernel)
  const bool v_group = L.v.kind == kBlock && L.v.code_kind == kBlock && N_after - 1 >= L.w_sink &&
                       n_quantised(kBlock, N_after, L.w_sink, L.w_recent, L.G) !=
                           n_quantised(kBlock, N_after - 1, L.w_sink, L.w_recent, L.G);
  cfg.gridDim = dim3(L.U, v_group ? 5 : 1); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = append_smem_bytes(L); cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, append_kernel, L, k_new, v_new, N_after, cache, late_wait) == cudaSuccess ? 1 : -1;
}

int launch_append_batched(const Layout& L, int n, unsigned char* const* caches, const int* Ns_after, const int* late_wait,
                          const __half* k_new, const __half* v_new, cudaStream_t st) {
  if (n < 1 || n > kMaxSeqs) return -1;
  AppendTable T;
  for (int i = 0; i < kMaxSeqs; ++i) {
    T.s[i].cache = caches[i < n ? i : 0];
    T.s[i].N = Ns_after[i < n ? i : 0];
    T.s[i].late_wait = late_wait[i < n ? i : 0];
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n * L.U); cfg.blockDim = dim3(128); cfg.dynamicSmemBytes = append_smem_bytes(L); cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, append_batched_kernel, L, k_new, v_new, T) == cudaSuccess ? 1 : -1;
}

int launch_export(const Layout& L, const unsigned char* cache, int N, const ExportPtrs& e, cudaStream_t st) {
  const Counts cn = counts_for(L, N);
  const bool fp16 = L.k.kind == kNone;
  export_store_kernel<<<dim3(64, L.U), 256, 0, st>>>(L, L.k, cache, cn.n_qk, fp16 ? N : cn.n_sink, cn.n_k_recent, e.k_code,
                                                    e.k_scale, e.k_zero, e.k_sink, e.k_recent);
  export_store_kernel<<<dim3(64, L.U), 256, 0, st>>>(L, L.v, cache, cn.n_qv, fp16 ? N : cn.n_sink, cn.n_v_recent, e.v_code,
                                                    e.v_scale, e.v_zero, e.v_sink, e.v_recent);
  if (e.norm)
    if (cudaMemcpyAsync(e.norm, cache + L.norm_off, (size_t)L.U * kD * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
      return -1;
  return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

int launch_import(const Layout& L, unsigned char* cache, int N, const ExportPtrs& e, cudaStream_t st) {
  const Counts cn = counts_for(L, N);
  const bool fp16 = L.k.kind == kNone;
  const Store* S[2] = {&L.k, &L.v};
  const int nq[2] = {cn.n_qk, cn.n_qv}, nrec[2] = {cn.n_k_recent, cn.n_v_recent};
  const uint8_t* code[2] = {e.k_code, e.v_code};
  const uint16_t* scale[2] = {e.k_scale, e.v_scale};
  const uint16_t* zero[2] = {e.k_zero, e.v_zero};
  const uint16_t* sink[2] = {e.k_sink, e.v_sink};
  const uint16_t* recent[2] = {e.k_recent, e.v_recent};
  int launches = 0;
  for (int pass = 0; pass < 2; ++pass)      // all packed words are cleared before any code is OR-ed in
    for (int i = 0; i < 2; ++i) {
      if (pass == 0 && (S[i]->kind == kNone || nq[i] == 0)) continue;
      import_store_kernel<<<dim3(64, L.U), 256, 0, st>>>(L, *S[i], cache, nq[i], fp16 ? N : cn.n_sink, nrec[i], code[i],
                                                        scale[i], zero[i], sink[i], recent[i], pass);
      ++launches;
    }
  if (cudaMemcpyAsync(cache + L.norm_off, e.norm, (size_t)L.U * kD * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return -1;
  fill_u32_kernel<<<(L.U + 255) / 256, 256, 0, st>>>(reinterpret_cast<uint32_t*>(cache + L.appended_off), (uint32_t)N, L.U);
  return cudaGetLastError() == cudaSuccess ? launches + 1 : -1;
}

}  // namespace iq
