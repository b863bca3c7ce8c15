// C ABI of libinnerq (see include/innerq.h): argument validation, layout computation, host-side
// token bookkeeping, kernel dispatch.  No device allocation, no synchronisation.
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/innerq.h"
#include "innerq_kernels.h"

using namespace iq;

struct innerq_cache {
  innerq_config_t cfg;
  Layout L;
  unsigned char* cache;
  unsigned char* ws;
  int N;
  int N_safe;      // token count when the last decode of this cache was launched (or at prefill): what was packed by then
                   // is complete and is not written again; a later decode may stream it before its predecessors finish
  int reads_settled;   // the last kernel enqueued for this cache was a fused decode: when its dependents may start, it
                       // has read everything that an append writes (the fp16 rings, the newest packed rows); an
                       // append can then run without waiting first
  int opt_splits, opt_variant;
  int launches[3];
  int pool_pages;                 // paged cache: pages in the pool (page ids are checked against it)
  std::vector<uint32_t> pages;    // paged cache: pool page of every assigned page slot (host copy of the device table)
};

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool valid_bits(int b) { return b == 2 || b == 3 || b == 4; }
bool valid_mode(int m) { return m >= 0 && m <= 2; }

int check_config(const innerq_config_t* c) {
  if (!c) return INNERQ_ERR_INVALID_ARG;
  if (c->batch <= 0 || c->n_q_heads <= 0 || c->n_kv_heads <= 0 || c->max_tokens <= 0 || c->w_sink < 0 ||
      c->w_recent < 0 || c->n_q_heads % c->n_kv_heads != 0 || !(c->sm_scale >= 0.f))
    return INNERQ_ERR_INVALID_ARG;
  if (c->grouping < 0 || c->grouping > 2 || c->sym_variant < 0 || c->sym_variant > 1) return INNERQ_ERR_INVALID_ARG;
  if (c->head_dim != kD) return INNERQ_ERR_UNSUPPORTED;
  if (c->grouping != INNERQ_GROUPING_FP16) {
    if (!valid_mode(c->k_mode) || !valid_mode(c->v_mode)) return INNERQ_ERR_INVALID_ARG;
    if (!valid_bits(c->k_bits) || !valid_bits(c->v_bits)) return INNERQ_ERR_UNSUPPORTED;
    if (c->group != 32 && c->group != 64 && c->group != 128) return INNERQ_ERR_UNSUPPORTED;
    if (c->grouping == INNERQ_GROUPING_OUTER && c->k_normalize) return INNERQ_ERR_INVALID_ARG;
  }
  if ((long long)c->batch * c->n_kv_heads > 65535) return INNERQ_ERR_UNSUPPORTED;
  return INNERQ_OK;
}

void place_store(Store& S, int kind, int bits, int mode, const innerq_config_t& c, int U, size_t& off) {
  std::memset(&S, 0, sizeof(S));
  S.kind = kind;
  S.bits = bits;
  S.mode = mode;
  S.code_kind = kind;
  if (kind == kNone) {
    S.sink_stride = (size_t)c.max_tokens * kD * 2;
    S.sink_off = off;
    off = align_up(off + S.sink_stride * U, 256);
    return;
  }
  const int G = c.group;
  int mid = c.max_tokens - c.w_sink - c.w_recent;
  if (mid < 1) mid = 1;
  // one chunk to spare: the decode kernel's copies take two chunks at a time and may read (never use) the one behind
  // the last packed token
  S.cap_q = (int)align_up((size_t)mid + kChunk, kTile);
  S.ring_cap = kind == kRow ? c.w_recent + 1 : c.w_recent + G;
  S.n_groups = kind == kRow ? kD / G : kD;
  S.meta_bytes = mode == INNERQ_MODE_SYM ? 2 : 4;
  S.sink_stride = (size_t)c.w_sink * kD * 2;
  S.ring_stride = (size_t)S.ring_cap * kD * 2;
  S.sink_off = off; off = align_up(off + S.sink_stride * U, 256);
  S.ring_off = off; off = align_up(off + S.ring_stride * U, 256);
}

// Geometry of the shared record area of a ROW store and a BLOCK store (see struct Store).
void place_records(Store& row, Store& blk, int G, int U, size_t& off, int page_groups) {
  const int row_codes = kChunk * row_bytes(row.bits);
  const int row_meta = kChunk * row.n_groups * row.meta_bytes;
  const int blk_codes = chunk_bytes(blk.bits);
  const int blk_meta = kD * blk.meta_bytes;
  const int chunk_stride = row_codes + row_meta + blk_codes;
  const int cpg = G / kChunk;
  const int group_stride = cpg * chunk_stride + blk_meta;
  const size_t unit = page_groups > 0 ? (size_t)page_groups * group_stride : align_up((size_t)(row.cap_q / G) * group_stride, 256);
  Store* both[2] = {&row, &blk};
  for (Store* S : both) {
    S->rec_off = off;
    S->rec_unit_stride = unit;
    S->group_stride = group_stride;
    S->chunk_stride = chunk_stride;
    S->chunks_per_group = cpg;
  }
  row.code_in_rec = 0;
  row.meta_in_rec = row_codes;
  blk.code_in_rec = row_codes + row_meta;
  blk.meta_in_rec = cpg * chunk_stride;
  if (page_groups == 0) off = align_up(off + unit * U, 256);
}

// Outer grouping: keys are grouped per channel along tokens (kBlock metadata) but keep one packed row per token,
// values are grouped per token along channels (kRow metadata) but keep 32-token chunks.  A chunk record holds the
// key rows, the values' metadata rows and the value chunk; the keys' per-group metadata comes FIRST in the group
// record, because scores need it from the group's first token on.
void place_records_outer(Store& k, Store& v, int G, int U, size_t& off, int page_groups) {
  k.code_kind = kRow;
  v.code_kind = kBlock;
  const int row_codes = kChunk * row_bytes(k.bits);
  const int row_meta = kChunk * v.n_groups * v.meta_bytes;
  const int blk_codes = chunk_bytes(v.bits);
  const int blk_meta = kD * k.meta_bytes;
  const int chunk_stride = row_codes + row_meta + blk_codes;
  const int cpg = G / kChunk;
  const int group_stride = blk_meta + cpg * chunk_stride;
  const size_t unit = page_groups > 0 ? (size_t)page_groups * group_stride : align_up((size_t)(v.cap_q / G) * group_stride, 256);
  Store* both[2] = {&k, &v};
  for (Store* S : both) {
    S->rec_off = off;
    S->rec_unit_stride = unit;
    S->group_stride = group_stride;
    S->chunk_stride = chunk_stride;
    S->chunks_per_group = cpg;
    S->chunk0 = blk_meta;
  }
  k.code_in_rec = 0;
  k.meta_in_rec = 0;
  v.meta_in_rec = row_codes;
  v.code_in_rec = row_codes + row_meta;
  if (page_groups == 0) off = align_up(off + unit * U, 256);
}

// page_tokens > 0: paged record area (see struct Layout); the pool pointer is set by the caller.
void make_layout(const innerq_config_t& c, Layout& L, int page_tokens = 0) {
  std::memset(&L, 0, sizeof(L));
  L.B = c.batch; L.Hq = c.n_q_heads; L.Hkv = c.n_kv_heads;
  L.U = c.batch * c.n_kv_heads;
  L.r = c.n_q_heads / c.n_kv_heads;
  L.G = c.grouping == INNERQ_GROUPING_FP16 ? 32 : c.group;
  L.w_sink = c.w_sink; L.w_recent = c.w_recent;
  L.sym_variant = c.sym_variant; L.grouping = c.grouping;
  L.k_normalize = (c.grouping == INNERQ_GROUPING_INNER && c.k_normalize) ? 1 : 0;
  L.max_tokens = c.max_tokens;
  L.sm_scale = c.sm_scale > 0.f ? c.sm_scale : 0.08838834764831845f;   // 1/sqrt(128)
  // partial slots per query head: token-range splits plus one per 32 tokens of the fp16 tail
  int ms = (4 * 148 + L.U - 1) / L.U;
  ms = ms < 1 ? 1 : (ms > 64 ? 64 : ms);
  L.max_splits = ms + (c.w_sink + c.w_recent + L.G + 31) / 32 + 1;
  size_t off = 0;
  L.norm_off = off; off = align_up(off + (size_t)L.U * kD * 4, 256);
  L.appended_off = off; off = align_up(off + (size_t)L.U * 8, 256);      // counts [U], then append part tickets [U]
  if (c.grouping == INNERQ_GROUPING_FP16) {
    place_store(L.k, kNone, 16, 0, c, L.U, off);
    place_store(L.v, kNone, 16, 0, c, L.U, off);
  } else if (c.grouping == INNERQ_GROUPING_INNER) {
    place_store(L.k, kRow, c.k_bits, c.k_mode, c, L.U, off);
    place_store(L.v, kBlock, c.v_bits, c.v_mode, c, L.U, off);
    // codes in byte order, for the decode kernel built on the 8-bit integer MMA
    L.k.perm = L.v.perm = 1;
    place_records(L.k, L.v, L.G, L.U, off, page_tokens / L.G);
  } else {   // outer grouping: asymmetric, K per channel along tokens, V per token along channels
    place_store(L.k, kBlock, c.k_bits, INNERQ_MODE_ASYM, c, L.U, off);
    place_store(L.v, kRow, c.v_bits, INNERQ_MODE_ASYM, c, L.U, off);
    place_records_outer(L.k, L.v, L.G, L.U, off, page_tokens / L.G);
  }
  L.page_chunk_mask = page_tokens > 0 ? page_tokens / kChunk - 1 : 0x3fffffff;
  if (page_tokens > 0) {
    for (int n = page_tokens / kChunk; n > 1; n >>= 1) L.page_chunk_shift += 1;
    L.page_groups = page_tokens / L.G;
    L.max_pages = (L.k.cap_q / L.G + L.page_groups - 1) / L.page_groups;
    L.page_bytes = align_up(L.k.rec_unit_stride * L.U, 256);
    L.page_table_off = off;
    off = align_up(off + (size_t)L.max_pages * 4, 256);
  }
  L.cache_bytes = off;
  size_t w = 0;
  L.ws_partial_off = w; w = align_up(w + (size_t)L.B * L.Hq * L.max_splits * kPartialStride * 4, 256);
  L.ws_absmax_off = w; w = align_up(w + (size_t)L.U * kD * 4, 256);
  L.ws_ticket_off = w; w = align_up(w + (size_t)(L.U + 8) * 4, 256);   // tickets [U], then the device error word
  L.workspace_bytes = w;
}

// Page slots that a cache of N tokens uses: every group record that holds a packed key row or value chunk.
int pages_for(const Layout& L, int N) {
  if (L.page_groups == 0) return 0;
  const Counts cn = counts_for(L, N);
  const int n_rec = cn.n_qk > cn.n_qv ? cn.n_qk : cn.n_qv;
  const int groups = (n_rec + L.G - 1) / L.G;
  return (groups + L.page_groups - 1) / L.page_groups;
}
bool has_pages_for(const innerq_cache* c, int N) { return (int)c->pages.size() >= pages_for(c->L, N); }

int create_cache(const innerq_config_t* cfg, int page_tokens, void* dev_cache, size_t cache_bytes, void* dev_workspace,
                 size_t workspace_bytes, void* dev_pool, int pool_pages, void* cuda_stream, innerq_cache_t** out) {
  int st = check_config(cfg);
  if (st != INNERQ_OK) return st;
  if (!dev_cache || !dev_workspace || !out) return INNERQ_ERR_INVALID_ARG;
  if (((uintptr_t)dev_cache & 255u) || ((uintptr_t)dev_workspace & 255u)) return INNERQ_ERR_INVALID_ARG;
  innerq_cache* c = new (std::nothrow) innerq_cache();
  if (!c) return INNERQ_ERR_INVALID_ARG;
  c->cfg = *cfg;
  make_layout(*cfg, c->L, page_tokens);
  c->L.pool = static_cast<unsigned char*>(dev_pool);
  c->pool_pages = pool_pages;
  if (cache_bytes < c->L.cache_bytes || workspace_bytes < c->L.workspace_bytes) {
    delete c;
    return INNERQ_ERR_BUFFER_TOO_SMALL;
  }
  c->cache = static_cast<unsigned char*>(dev_cache);
  c->ws = static_cast<unsigned char*>(dev_workspace);
  c->N = 0;
  c->N_safe = 0;
  c->reads_settled = 0;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(c->cache, 0, c->L.cache_bytes, s) != cudaSuccess ||
      cudaMemsetAsync(c->ws, 0, c->L.workspace_bytes, s) != cudaSuccess) {
    delete c;
    return INNERQ_ERR_CUDA;
  }
  // norm = 1 until a prefill computes it
  if (launch_prefill(c->L, c->cache, c->ws, nullptr, nullptr, 0, s) < 0) {
    delete c;
    return INNERQ_ERR_CUDA;
  }
  *out = c;
  return INNERQ_OK;
}

int check_page_tokens(const innerq_config_t* cfg, int page_tokens) {
  int st = check_config(cfg);
  if (st != INNERQ_OK) return st;
  if (page_tokens < kTile || (page_tokens & (page_tokens - 1)) != 0) return INNERQ_ERR_INVALID_ARG;
  if (cfg->grouping == INNERQ_GROUPING_FP16) return INNERQ_ERR_UNSUPPORTED;    // only packed records are paged
  return INNERQ_OK;
}

}  // namespace

extern "C" {

int innerq_cache_bytes(const innerq_config_t* cfg, size_t* cache_bytes, size_t* workspace_bytes) {
  int st = check_config(cfg);
  if (st != INNERQ_OK) return st;
  if (!cache_bytes || !workspace_bytes) return INNERQ_ERR_INVALID_ARG;
  Layout L;
  make_layout(*cfg, L);
  *cache_bytes = L.cache_bytes;
  *workspace_bytes = L.workspace_bytes;
  return INNERQ_OK;
}

int innerq_token_payload_bytes(const innerq_config_t* cfg, double* k_bytes, double* v_bytes) {
  int st = check_config(cfg);
  if (st != INNERQ_OK) return st;
  if (!k_bytes || !v_bytes) return INNERQ_ERR_INVALID_ARG;
  Layout L;
  make_layout(*cfg, L);
  const Store* S[2] = {&L.k, &L.v};
  double out[2];
  for (int i = 0; i < 2; ++i) {
    if (S[i]->kind == kNone) out[i] = kD * 2.0;
    else if (S[i]->kind == kRow) out[i] = row_bytes(S[i]->bits) + (double)S[i]->n_groups * S[i]->meta_bytes;
    else out[i] = chunk_bytes(S[i]->bits) / (double)kChunk + (double)kD * S[i]->meta_bytes / L.G;
  }
  *k_bytes = out[0];
  *v_bytes = out[1];
  return INNERQ_OK;
}

int innerq_cache_create(const innerq_config_t* cfg, void* dev_cache, size_t cache_bytes, void* dev_workspace,
                        size_t workspace_bytes, void* cuda_stream, innerq_cache_t** out) {
  return create_cache(cfg, 0, dev_cache, cache_bytes, dev_workspace, workspace_bytes, nullptr, 0, cuda_stream, out);
}

// ---- paged record area --------------------------------------------------------------------------------
int innerq_paged_cache_bytes(const innerq_config_t* cfg, int32_t page_tokens, size_t* cache_bytes, size_t* workspace_bytes,
                             size_t* page_bytes, int32_t* max_pages) {
  const int st = check_page_tokens(cfg, page_tokens);
  if (st != INNERQ_OK) return st;
  if (!cache_bytes || !workspace_bytes || !page_bytes || !max_pages) return INNERQ_ERR_INVALID_ARG;
  Layout L;
  make_layout(*cfg, L, page_tokens);
  *cache_bytes = L.cache_bytes;
  *workspace_bytes = L.workspace_bytes;
  *page_bytes = L.page_bytes;
  *max_pages = L.max_pages;
  return INNERQ_OK;
}

int innerq_cache_create_paged(const innerq_config_t* cfg, int32_t page_tokens, void* dev_cache, size_t cache_bytes,
                              void* dev_workspace, size_t workspace_bytes, void* dev_pool, int32_t pool_pages,
                              void* cuda_stream, innerq_cache_t** out) {
  const int st = check_page_tokens(cfg, page_tokens);
  if (st != INNERQ_OK) return st;
  if (!dev_pool || ((uintptr_t)dev_pool & 255u) || pool_pages < 1) return INNERQ_ERR_INVALID_ARG;
  return create_cache(cfg, page_tokens, dev_cache, cache_bytes, dev_workspace, workspace_bytes, dev_pool, pool_pages,
                      cuda_stream, out);
}

int innerq_cache_pages_for(const innerq_cache_t* c, int32_t n_tokens) {
  if (!c || n_tokens < 0) return INNERQ_ERR_INVALID_ARG;
  if (n_tokens > c->L.max_tokens) return INNERQ_ERR_CAPACITY;
  return pages_for(c->L, n_tokens);
}

int innerq_cache_pages_assigned(const innerq_cache_t* c) { return c ? (int)c->pages.size() : INNERQ_ERR_INVALID_ARG; }

int innerq_cache_assign_pages(innerq_cache_t* c, const int32_t* pages_host, int32_t n, void* cuda_stream) {
  if (!c || !pages_host || n < 1 || c->L.page_groups == 0) return INNERQ_ERR_INVALID_ARG;
  const size_t have = c->pages.size();
  if (have + (size_t)n > (size_t)c->L.max_pages) return INNERQ_ERR_CAPACITY;
  for (int i = 0; i < n; ++i) {
    if (pages_host[i] < 0 || pages_host[i] >= c->pool_pages) return INNERQ_ERR_INVALID_ARG;
    for (size_t j = 0; j < have; ++j)
      if (c->pages[j] == (uint32_t)pages_host[i]) return INNERQ_ERR_INVALID_ARG;
    for (int j = 0; j < i; ++j)
      if (pages_host[j] == pages_host[i]) return INNERQ_ERR_INVALID_ARG;
  }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (c->L.k.code_kind != c->L.k.kind) {
    // outer grouping fills chunk words token by token with OR: its pages start from zero
    for (int i = 0; i < n; ++i)
      if (cudaMemsetAsync(c->L.pool + (size_t)pages_host[i] * c->L.page_bytes, 0, c->L.page_bytes, s) != cudaSuccess)
        return INNERQ_ERR_CUDA;
  }
  c->pages.reserve(c->L.max_pages);        // the copy below reads the vector's storage: it must not move later
  for (int i = 0; i < n; ++i) c->pages.push_back((uint32_t)pages_host[i]);
  // a copy is ordered after every kernel before it in the stream and before every kernel after it, whatever their
  // launch attributes: no kernel ever sees a table entry half-way
  if (cudaMemcpyAsync(c->cache + c->L.page_table_off + have * 4, c->pages.data() + have, (size_t)n * 4,
                      cudaMemcpyHostToDevice, s) != cudaSuccess) {
    c->pages.resize(have);
    return INNERQ_ERR_CUDA;
  }
  return INNERQ_OK;
}

int innerq_cache_release_pages(innerq_cache_t* c, int32_t* pages_host, int32_t capacity) {
  if (!c || c->L.page_groups == 0 || capacity < 0 || (capacity > 0 && !pages_host)) return INNERQ_ERR_INVALID_ARG;
  const int n = (int)c->pages.size();
  if (capacity < n) return INNERQ_ERR_BUFFER_TOO_SMALL;
  for (int i = 0; i < n; ++i) pages_host[i] = (int32_t)c->pages[i];
  c->pages.clear();
  c->N = 0;
  c->N_safe = 0;
  c->reads_settled = 0;
  return n;
}

int innerq_cache_destroy(innerq_cache_t* cache) {
  if (!cache) return INNERQ_ERR_INVALID_ARG;
  delete cache;
  return INNERQ_OK;
}

int innerq_cache_n_tokens(const innerq_cache_t* cache) { return cache ? cache->N : INNERQ_ERR_INVALID_ARG; }

int innerq_quantize_prefill(innerq_cache_t* c, const void* k, const void* v, int32_t n_tokens, void* cuda_stream) {
  if (!c || n_tokens < 0 || (n_tokens > 0 && (!k || !v))) return INNERQ_ERR_INVALID_ARG;
  if (n_tokens > c->L.max_tokens || !has_pages_for(c, n_tokens)) return INNERQ_ERR_CAPACITY;
  int n = launch_prefill(c->L, c->cache, c->ws, static_cast<const __half*>(k), static_cast<const __half*>(v), n_tokens,
                         static_cast<cudaStream_t>(cuda_stream));
  if (n < 0) return INNERQ_ERR_CUDA;
  c->N = n_tokens;
  // Nothing of a fresh prefill counts as settled: the first decode after it waits for its predecessors before it
  // reads any packed chunk (the prefill kernels are ordinary launches, whose writes a dependent launch may rely on
  // only after that wait).  The decode that follows then streams ahead again.
  c->N_safe = 0;
  c->reads_settled = 0;
  c->launches[0] = n;
  return INNERQ_OK;
}

int innerq_append_token(innerq_cache_t* c, const void* k_new, const void* v_new, void* cuda_stream) {
  if (!c || !k_new || !v_new) return INNERQ_ERR_INVALID_ARG;
  if (c->N + 1 > c->L.max_tokens || !has_pages_for(c, c->N + 1)) return INNERQ_ERR_CAPACITY;
  int n = launch_append(c->L, c->cache, static_cast<const __half*>(k_new), static_cast<const __half*>(v_new), c->N + 1,
                        static_cast<cudaStream_t>(cuda_stream), c->reads_settled);
  if (n < 0) return INNERQ_ERR_CUDA;
  c->reads_settled = 0;
  c->N += 1;
  c->launches[1] = n;
  return INNERQ_OK;
}

int innerq_decode_attention(innerq_cache_t* c, const void* q, void* out, void* cuda_stream) {
  if (!c || !q || !out || c->N < 1) return INNERQ_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  int n = -2;
  bool fused = false;
  if (c->opt_variant != 1 && c->L.k.kind == kNone)
    n = launch_decode_fp16(c->L, c->cache, c->ws, c->N, static_cast<const __half*>(q), static_cast<__half*>(out),
                           c->opt_splits, s);
  else if (c->opt_variant != 1 && decode_mma_supported(c->L)) {
    n = launch_decode_mma(c->L, c->cache, c->ws, c->N, static_cast<const __half*>(q), static_cast<__half*>(out),
                          c->opt_splits, s, 1, nullptr, c->N_safe, c->pages.data(), (int)c->pages.size());
    fused = n >= 0;
  }
  if (n == -2) {
    if (c->opt_variant == 2) return INNERQ_ERR_UNSUPPORTED;
    n = launch_decode_simt(c->L, c->cache, c->ws, c->N, static_cast<const __half*>(q), static_cast<__half*>(out),
                           c->opt_splits, s);
  }
  if (n < 0) return INNERQ_ERR_CUDA;
  c->N_safe = c->N;
  c->reads_settled = fused ? 1 : 0;
  c->launches[2] = n;
  return INNERQ_OK;
}

// ---- several query tokens per sequence ----------------------------------------------------------------
int innerq_multi_query_scratch_bytes(const innerq_config_t* cfg, size_t* bytes) {
  if (!bytes) return INNERQ_ERR_INVALID_ARG;
  const int st = check_config(cfg);
  if (st != INNERQ_OK) return st;
  Layout L;
  make_layout(*cfg, L);
  *bytes = align_up((size_t)L.U * 4 * L.max_splits * kPartialStride * 4, 256);
  return INNERQ_OK;
}

int innerq_decode_attention_multi(innerq_cache_t* c, const void* q, void* out, int32_t n_q, void* dev_scratch,
                                  size_t scratch_bytes, void* cuda_stream) {
  if (!c || !q || !out || !dev_scratch || n_q < 1 || n_q > c->N) return INNERQ_ERR_INVALID_ARG;
  if ((uintptr_t)dev_scratch & 255u) return INNERQ_ERR_INVALID_ARG;
  if (scratch_bytes < align_up((size_t)c->L.U * 4 * c->L.max_splits * kPartialStride * 4, 256)) return INNERQ_ERR_BUFFER_TOO_SMALL;
  if ((c->opt_variant != 0 && c->opt_variant != 2) || c->L.k.kind == kNone || !decode_mma_supported(c->L))
    return INNERQ_ERR_UNSUPPORTED;
  // the hidden tokens (positions N - n_q + 1 .. N - 1) must be sink, skew-zone or recent tokens: those are
  // scored in tiles that can mask by position; the chunks where keys and values are both packed cannot
  const Counts cn = counts_for(c->L, c->N);
  const int n_packed = cn.n_qk < cn.n_qv ? cn.n_qk : cn.n_qv;
  if (n_packed > 0 && c->N - n_q + 1 < cn.n_sink + n_packed) return INNERQ_ERR_UNSUPPORTED;
  const int n = launch_decode_mma(c->L, c->cache, c->ws, c->N, static_cast<const __half*>(q), static_cast<__half*>(out),
                                  c->opt_splits, static_cast<cudaStream_t>(cuda_stream), n_q,
                                  static_cast<float*>(dev_scratch), c->N_safe, c->pages.data(), (int)c->pages.size());
  if (n == -2) return INNERQ_ERR_UNSUPPORTED;
  if (n < 0) return INNERQ_ERR_CUDA;
  c->N_safe = c->N;
  c->reads_settled = 1;
  c->launches[2] = n;
  return INNERQ_OK;
}

// ---- several caches per call (sequences of different lengths) -----------------------------------------
namespace {
constexpr int kMaxBatchedCaches = 4096;      // per call; a launch takes kMaxSeqs of them
// All caches of a batched call must have been created from the same configuration: the kernels take one layout.
bool same_layout(innerq_cache_t* const* caches, int n) {
  for (int i = 0; i < n; ++i) {
    if (!caches[i]) return false;
    if (i && std::memcmp(&caches[i]->L, &caches[0]->L, sizeof(Layout)) != 0) return false;
  }
  return true;
}
}  // namespace

int innerq_append_token_batched(innerq_cache_t* const* caches, int32_t n, const void* k_new, const void* v_new,
                                void* cuda_stream) {
  if (!caches || !k_new || !v_new || n < 1 || n > kMaxBatchedCaches || !same_layout(caches, n)) return INNERQ_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    for (int j = 0; j < i; ++j)
      if (caches[j] == caches[i]) return INNERQ_ERR_INVALID_ARG;      // one token per cache and call
    if (caches[i]->N + 1 > caches[i]->L.max_tokens || !has_pages_for(caches[i], caches[i]->N + 1)) return INNERQ_ERR_CAPACITY;
  }
  const Layout& L = caches[0]->L;
  const size_t row = (size_t)L.U * kD;                                 // fp16 elements per cache in k_new / v_new
  int launches = 0;
  for (int i0 = 0; i0 < n; i0 += kMaxSeqs) {                          // one launch per kMaxSeqs caches
    const int m = n - i0 < kMaxSeqs ? n - i0 : kMaxSeqs;
    unsigned char* ptr[kMaxSeqs];
    int Ns[kMaxSeqs], late[kMaxSeqs];
    for (int i = 0; i < m; ++i) {
      ptr[i] = caches[i0 + i]->cache;
      Ns[i] = caches[i0 + i]->N + 1;
      late[i] = caches[i0 + i]->reads_settled;
    }
    const int l = launch_append_batched(L, m, ptr, Ns, late, static_cast<const __half*>(k_new) + i0 * row,
                                        static_cast<const __half*>(v_new) + i0 * row, static_cast<cudaStream_t>(cuda_stream));
    if (l < 0) return INNERQ_ERR_CUDA;
    for (int i = 0; i < m; ++i) {
      caches[i0 + i]->N += 1;
      caches[i0 + i]->reads_settled = 0;
    }
    launches += l;
  }
  for (int i = 0; i < n; ++i) caches[i]->launches[1] = launches;
  return INNERQ_OK;
}

int innerq_decode_attention_batched(innerq_cache_t* const* caches, int32_t n, const void* q, void* out, void* cuda_stream) {
  if (!caches || !q || !out || n < 1 || n > kMaxBatchedCaches || !same_layout(caches, n)) return INNERQ_ERR_INVALID_ARG;
  const innerq_cache_t* c0 = caches[0];
  if ((c0->opt_variant != 0 && c0->opt_variant != 2) || c0->L.k.kind == kNone || !decode_mma_supported(c0->L))
    return INNERQ_ERR_UNSUPPORTED;
  for (int i = 0; i < n; ++i) {
    if (caches[i]->N < 1) return INNERQ_ERR_INVALID_ARG;
    for (int j = 0; j < i; ++j)
      if (caches[j]->ws == caches[i]->ws) return INNERQ_ERR_INVALID_ARG;      // partials and tickets are per cache
  }
  const Layout& L = c0->L;
  const size_t row = (size_t)L.B * L.Hq * kD;                          // fp16 elements per cache in q / out
  int launches = 0;
  for (int i0 = 0; i0 < n; i0 += kMaxSeqs) {
    const int m = n - i0 < kMaxSeqs ? n - i0 : kMaxSeqs;
    const unsigned char* ptr[kMaxSeqs];
    unsigned char* ws[kMaxSeqs];
    int Ns[kMaxSeqs], Ns_safe[kMaxSeqs];
    for (int i = 0; i < m; ++i) {
      ptr[i] = caches[i0 + i]->cache;
      ws[i] = caches[i0 + i]->ws;
      Ns[i] = caches[i0 + i]->N;
      Ns_safe[i] = caches[i0 + i]->N_safe;
    }
    const int l = launch_decode_mma_batched(L, m, ptr, ws, Ns, Ns_safe, static_cast<const __half*>(q) + i0 * row,
                                            static_cast<__half*>(out) + i0 * row, c0->opt_splits,
                                            static_cast<cudaStream_t>(cuda_stream));
    if (l == -2) return INNERQ_ERR_UNSUPPORTED;
    if (l < 0) return INNERQ_ERR_CUDA;
    for (int i = 0; i < m; ++i) {
      caches[i0 + i]->N_safe = caches[i0 + i]->N;
      caches[i0 + i]->reads_settled = 1;
    }
    launches += l;
  }
  for (int i = 0; i < n; ++i) caches[i]->launches[2] = launches;
  return INNERQ_OK;
}

// ---- one step from host buffers ----------------------------------------------------------------------
static size_t align256(size_t x) { return (x + 255) / 256 * 256; }

int innerq_step_staging_bytes(const innerq_config_t* cfg, size_t* bytes) {
  if (!cfg || !bytes || check_config(cfg) != INNERQ_OK) return INNERQ_ERR_INVALID_ARG;
  const size_t kv = align256((size_t)cfg->batch * cfg->n_kv_heads * cfg->head_dim * 2);
  const size_t qo = align256((size_t)cfg->batch * cfg->n_q_heads * cfg->head_dim * 2);
  *bytes = 2 * kv + 2 * qo;
  return INNERQ_OK;
}

int innerq_decode_step_host(innerq_cache_t* c, const void* k_new_host, const void* v_new_host, const void* q_host,
                            void* out_host, void* dev_staging, void* cuda_stream) {
  if (!c || !k_new_host || !v_new_host || !q_host || !out_host || !dev_staging) return INNERQ_ERR_INVALID_ARG;
  if (c->N + 1 > c->L.max_tokens || !has_pages_for(c, c->N + 1)) return INNERQ_ERR_CAPACITY;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  const size_t kv_bytes = (size_t)c->L.U * kD * 2, q_bytes = (size_t)c->L.B * c->L.Hq * kD * 2;
  unsigned char* d = static_cast<unsigned char*>(dev_staging);
  unsigned char* dk = d;
  unsigned char* dv = dk + align256(kv_bytes);
  unsigned char* dq = dv + align256(kv_bytes);
  unsigned char* dout = dq + align256(q_bytes);
  // Pinned (page-locked, mapped) host buffers are addressable by the GPU: the kernels then read the 10-30 KB of
  // inputs and write the result in place over the bus, and no copy is enqueued at all.  Anything else is staged.
  const void* src[3] = {k_new_host, v_new_host, q_host};
  void* mapped[4] = {nullptr, nullptr, nullptr, nullptr};
  bool zero_copy = true;
  for (int i = 0; i < 4 && zero_copy; ++i) {
    cudaPointerAttributes at;
    const void* p = i < 3 ? src[i] : out_host;
    if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); zero_copy = false; break; }
    if (at.type != cudaMemoryTypeHost || at.devicePointer == nullptr) zero_copy = false;
    else mapped[i] = at.devicePointer;
  }
  if (zero_copy) {
    int st = innerq_append_token(c, mapped[0], mapped[1], cuda_stream);
    if (st != INNERQ_OK) return st;
    return innerq_decode_attention(c, mapped[2], mapped[3], cuda_stream);
  }
  if (cudaMemcpyAsync(dk, k_new_host, kv_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(dv, v_new_host, kv_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(dq, q_host, q_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess)
    return INNERQ_ERR_CUDA;
  int st = innerq_append_token(c, dk, dv, cuda_stream);
  if (st != INNERQ_OK) return st;
  st = innerq_decode_attention(c, dq, dout, cuda_stream);
  if (st != INNERQ_OK) return st;
  if (cudaMemcpyAsync(out_host, dout, q_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return INNERQ_ERR_CUDA;
  return INNERQ_OK;
}

// ---- decode on library-owned scratch ---------------------------------------------------------------
// The split partials, merge tickets and error word of the decode kernel normally live in the workspace
// the caller handed to innerq_cache_create.  This variant keeps them in a fixed array inside the library
// image instead, so it needs no device memory from the caller beyond inputs and outputs.
constexpr size_t kStaticScratchBytes = 4u << 20;     // 4 MiB per GPU that loads the library, held until exit
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel can use:
// the device address has to be looked up, once per device, while that device is current.
int static_scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return INNERQ_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return INNERQ_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = static_cast<unsigned char*>(g_scratch_ptr[dev]);
  return INNERQ_OK;
}
}  // namespace

int innerq_decode_attention_static(innerq_cache_t* c, const void* q, void* out, void* cuda_stream) {
  if (!c || !q || !out || c->N < 1) return INNERQ_ERR_INVALID_ARG;
  if (c->L.workspace_bytes > kStaticScratchBytes) return INNERQ_ERR_BUFFER_TOO_SMALL;
  // the array that is used is the current device's: the cache has to live on that device
  {
    int dev = -1;
    cudaPointerAttributes at;
    if (cudaGetDevice(&dev) != cudaSuccess) return INNERQ_ERR_CUDA;
    if (cudaPointerGetAttributes(&at, c->cache) != cudaSuccess) { cudaGetLastError(); return INNERQ_ERR_INVALID_ARG; }
    if (at.type != cudaMemoryTypeDevice || at.device != dev) return INNERQ_ERR_INVALID_ARG;
  }
  unsigned char* scratch = nullptr;
  int st = static_scratch_for_current_device(&scratch);
  if (st != INNERQ_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  // the array keeps whatever the previous call (of any cache) left: tickets and the error word must start at zero
  if (cudaMemsetAsync(scratch + c->L.ws_ticket_off, 0, (size_t)(c->L.U + 8) * 4, s) != cudaSuccess) return INNERQ_ERR_CUDA;
  int n = -2;
  bool fused = false;
  if (c->opt_variant != 1 && c->L.k.kind == kNone)
    n = launch_decode_fp16(c->L, c->cache, scratch, c->N, static_cast<const __half*>(q), static_cast<__half*>(out),
                           c->opt_splits, s);
  else if (c->opt_variant != 1 && decode_mma_supported(c->L)) {
    n = launch_decode_mma(c->L, c->cache, scratch, c->N, static_cast<const __half*>(q), static_cast<__half*>(out),
                          c->opt_splits, s, 1, nullptr, c->N_safe, c->pages.data(), (int)c->pages.size());
    fused = n >= 0;
  }
  if (n == -2) {
    if (c->opt_variant == 2) return INNERQ_ERR_UNSUPPORTED;
    n = launch_decode_simt(c->L, c->cache, scratch, c->N, static_cast<const __half*>(q), static_cast<__half*>(out),
                           c->opt_splits, s);
  }
  if (n < 0) return INNERQ_ERR_CUDA;
  c->N_safe = c->N;
  c->reads_settled = fused ? 1 : 0;
  c->launches[2] = n;
  return INNERQ_OK;
}

int innerq_cache_export(innerq_cache_t* c, innerq_export_t* ex, void* cuda_stream) {
  if (!c || !ex) return INNERQ_ERR_INVALID_ARG;
  const Counts cn = counts_for(c->L, c->N);
  const bool fp16 = c->L.k.kind == kNone;
  ex->n_tokens = cn.N;
  ex->n_sink = fp16 ? cn.N : cn.n_sink;
  ex->n_qk = cn.n_qk;
  ex->n_qv = cn.n_qv;
  ex->n_k_recent = fp16 ? 0 : cn.n_k_recent;
  ex->n_v_recent = fp16 ? 0 : cn.n_v_recent;
  ExportPtrs p{ex->k_code, ex->v_code, ex->k_scale, ex->k_zero, ex->v_scale, ex->v_zero,
               ex->norm,   ex->k_sink, ex->v_sink,  ex->k_recent, ex->v_recent};
  if (launch_export(c->L, c->cache, c->N, p, static_cast<cudaStream_t>(cuda_stream)) < 0) return INNERQ_ERR_CUDA;
  return INNERQ_OK;
}

int innerq_cache_import(innerq_cache_t* c, const innerq_export_t* ex, int32_t n_tokens, void* cuda_stream) {
  if (!c || !ex || n_tokens < 0) return INNERQ_ERR_INVALID_ARG;
  if (n_tokens > c->L.max_tokens || !has_pages_for(c, n_tokens)) return INNERQ_ERR_CAPACITY;
  const bool fp16 = c->L.k.kind == kNone;
  if (!ex->norm || !ex->k_sink || !ex->v_sink) return INNERQ_ERR_INVALID_ARG;
  if (!fp16) {
    if (!ex->k_code || !ex->v_code || !ex->k_scale || !ex->v_scale || !ex->k_recent || !ex->v_recent) return INNERQ_ERR_INVALID_ARG;
    if ((c->L.k.meta_bytes == 4 && !ex->k_zero) || (c->L.v.meta_bytes == 4 && !ex->v_zero)) return INNERQ_ERR_INVALID_ARG;
  }
  ExportPtrs p{ex->k_code, ex->v_code, ex->k_scale, ex->k_zero, ex->v_scale, ex->v_zero,
               ex->norm,   ex->k_sink, ex->v_sink,  ex->k_recent, ex->v_recent};
  const int n = launch_import(c->L, c->cache, n_tokens, p, static_cast<cudaStream_t>(cuda_stream));
  if (n < 0) return INNERQ_ERR_CUDA;
  c->N = n_tokens;
  c->N_safe = 0;              // as after a prefill: the next decode waits for these kernels before it reads anything
  c->reads_settled = 0;
  c->launches[0] = n;
  return INNERQ_OK;
}

int innerq_set_decode_options(innerq_cache_t* c, int32_t n_splits, int32_t variant) {
  if (!c || n_splits < 0 || variant < 0 || variant > 7 || variant == 5) return INNERQ_ERR_INVALID_ARG;
  c->opt_splits = n_splits;
  // variants 3 and 4 force the fast kernel with one / two 32-token chunks per loop iteration (process-wide knob)
  if (variant == 3 || variant == 4) { decode_mma_set_chunks_per_iter(variant - 2); variant = 2; }
  else decode_mma_set_chunks_per_iter(0);
  // variants 6 and 7: the fast kernel without its key-side / value-side arithmetic (timing only, process-wide knob)
  if (variant == 6 || variant == 7) { decode_mma_set_ablation(variant - 5); variant = 2; }
  else decode_mma_set_ablation(0);
  c->opt_variant = variant;
  return INNERQ_OK;
}

int innerq_selftest_wait_expiry(innerq_cache_t* c, void* cuda_stream) {
  if (!c) return INNERQ_ERR_INVALID_ARG;
  return launch_wait_expiry_selftest(c->L, c->ws, static_cast<cudaStream_t>(cuda_stream)) < 0 ? INNERQ_ERR_CUDA : INNERQ_OK;
}

int innerq_read_device_error(innerq_cache_t* c, void* cuda_stream) {
  if (!c) return INNERQ_ERR_INVALID_ARG;
  unsigned int flag = 0;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(&flag, c->ws + c->L.ws_ticket_off + (size_t)c->L.U * 4, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return INNERQ_ERR_CUDA;
  // a call of innerq_decode_attention_static keeps its error word in the library's own array (same offset, this
  // cache's layout; every such call clears it first, so it tells about the last one on the current device)
  int dev = -1;
  if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices && c->L.workspace_bytes <= kStaticScratchBytes) {
    void* p = nullptr;
    {
      std::lock_guard<std::mutex> lock(g_scratch_mutex);
      p = g_scratch_ptr[dev];
    }
    if (p) {
      unsigned int flag2 = 0;
      if (cudaMemcpyAsync(&flag2, static_cast<unsigned char*>(p) + c->L.ws_ticket_off + (size_t)c->L.U * 4, 4,
                          cudaMemcpyDeviceToHost, s) != cudaSuccess ||
          cudaStreamSynchronize(s) != cudaSuccess)
        return INNERQ_ERR_CUDA;
      flag |= flag2;
    }
  }
  return (int)flag;
}

int innerq_last_launch_count(const innerq_cache_t* c, int32_t which) {
  if (!c || which < 0 || which > 2) return INNERQ_ERR_INVALID_ARG;
  return c->launches[which];
}

const char* innerq_status_string(int status) {
  switch (status) {
    case INNERQ_OK: return "ok";
    case INNERQ_ERR_INVALID_ARG: return "invalid argument";
    case INNERQ_ERR_UNSUPPORTED: return "unsupported configuration";
    case INNERQ_ERR_CAPACITY: return "token capacity exceeded";
    case INNERQ_ERR_BUFFER_TOO_SMALL: return "caller buffer too small";
    case INNERQ_ERR_CUDA: return "CUDA error";
    default: return "unknown status";
  }
}

}  // extern "C"
