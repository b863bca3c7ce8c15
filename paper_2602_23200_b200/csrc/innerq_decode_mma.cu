// Host side of the fused decode kernel over the packed InnerQ cache: picks the kernel family of the cache's
// packed format and fills the launch parameters.  The kernels are in innerq_decode_i8.cuh (inner-grouped caches,
// one translation unit per format: innerq_decode_mma_k*v*_m*.cu) and innerq_decode_mma.cuh (outer-grouped caches).
#include "innerq_decode_mma.h"
#include "innerq_kernels.h"

namespace iq {

namespace {

int g_chunks_per_iter = 0;    // tuning knob: 0 automatic, else 1 or 2 chunks of 32 tokens per loop iteration
int g_ablation = 0;           // timing experiments: see DecodeArgs::ablation

using FormatLauncher = int (*)(const Layout&, const Counts&, const DecodeArgs&, int, int, cudaStream_t);

// The formats with kernels: every combination of 2 / 3 / 4-bit keys and values with full or scale-only metadata
// (all instances of the integer-MMA kernel, innerq_decode_i8.cuh), and the outer-grouped comparison cache at 2 and 4
// bits (the fp16-operand kernel, innerq_decode_mma.cuh).
struct FormatEntry {
  int kb, vb, km, vm;
  FormatLauncher one;
  int (*batched)(const Layout&, SeqTable&, int, int, int, cudaStream_t);
};
#define IQ_FORMAT_ENTRY(KB, VB, KM, VM) \
  {KB, VB, KM, VM, &launch_decode_mma_k##KB##v##VB##_m##KM##VM, &launch_decode_mma_k##KB##v##VB##_m##KM##VM##_batched},
const FormatEntry kFormats[] = {IQ_FOR_EACH_MMA_FORMAT(IQ_FORMAT_ENTRY)};
#undef IQ_FORMAT_ENTRY

const FormatEntry* find_format(const Layout& L) {
  if (L.G != 32 && L.G != 64 && L.G != 128) return nullptr;
  if (L.grouping != 0 || L.k.kind != kRow || L.v.kind != kBlock) return nullptr;
  for (const FormatEntry& f : kFormats)
    if (f.kb == L.k.bits && f.vb == L.v.bits && f.km == L.k.meta_bytes && f.vm == L.v.meta_bytes) return &f;
  return nullptr;
}

bool is_outer(const Layout& L) {
  return L.grouping == 1 && (L.G == 32 || L.G == 64 || L.G == 128) && L.k.kind == kBlock && L.k.code_kind == kRow &&
         L.v.kind == kRow && L.v.code_kind == kBlock && L.k.meta_bytes == 4 && L.v.meta_bytes == 4 &&
         L.k.bits == L.v.bits && (L.k.bits == 2 || L.k.bits == 4);
}

FormatLauncher format_launcher(const Layout& L) {
  if (is_outer(L)) return L.k.bits == 2 ? &launch_decode_mma_outer_k2v2 : &launch_decode_mma_outer_k4v4;
  const FormatEntry* f = find_format(L);
  return f ? f->one : nullptr;
}

using BatchedLauncher = int (*)(const Layout&, SeqTable&, int, int, int, cudaStream_t);

BatchedLauncher batched_launcher(const Layout& L) {
  if (is_outer(L)) return L.k.bits == 2 ? &launch_decode_mma_outer_k2v2_batched : &launch_decode_mma_outer_k4v4_batched;
  const FormatEntry* f = find_format(L);
  return f ? f->batched : nullptr;
}

// The launch parameters of one cache that follow from its token count alone.
void fill_count_args(const Layout& L, const Counts& cn, DecodeArgs& a) {
  // tokens where only one tensor is packed (inner: keys, outer: values), then the tokens that are fp16 in both
  const bool outer = L.grouping == 1;
  a.n_skew_tiles = ((outer ? cn.n_qv - cn.n_qk : cn.n_qk - cn.n_qv) + 15) / 16;
  a.n_tail_tiles = a.n_skew_tiles + (cn.n_sink + (outer ? cn.n_v_recent : cn.n_k_recent) + 15) / 16;
  a.units_per_split = 0;
  a.tail_cost_units = 0;
  a.tiles_q0 = a.tiles_rem = 0;
  a.k_ring_pos0 = L.k.ring_cap ? cn.n_qk % L.k.ring_cap : 0;
  a.v_ring_pos0 = L.v.ring_cap ? cn.n_qv % L.v.ring_cap : 0;
  a.head0 = 0;
}

int default_splits(const Layout& L, int n_units_total) {
  int n_splits = (2 * 148) / n_units_total;      // two resident CTAs per SM, one wave
  if (n_splits < 1) n_splits = 1;
  if (n_splits > L.max_splits) n_splits = L.max_splits;
  if (n_splits > 128) n_splits = 128;            // slots of the merge tables in shared memory
  return n_splits;
}

}  // namespace

bool decode_mma_supported(const Layout& L) { return format_launcher(L) != nullptr; }

static int safe_chunks_for(const Layout& L, int N_safe, const Counts& cn_now);

// n caches of the same layout L with their own token counts: q and out are [n][B * Hq * D].
int launch_decode_mma_batched(const Layout& L, int n, const unsigned char* const* caches, unsigned char* const* wss,
                              const int* Ns, const int* Ns_safe, const __half* q, __half* out, int n_splits,
                              cudaStream_t st) {
  const BatchedLauncher launch = batched_launcher(L);
  if (!launch) return -2;
  if (n < 1 || n > kMaxSeqs) return -1;
  // rows (of U CTAs each) for all sequences together: one wave of two CTAs per SM, or n_splits per sequence on average
  int row_budget = n_splits > 0 ? n_splits * n : (2 * 148) / L.U;
  if (row_budget < n) row_budget = n;
  SeqTable T;
  for (int i = 0; i < n; ++i) {
    SeqArgs& e = T.s[i];
    e.cn = counts_for(L, Ns[i]);
    e.a.cache = caches[i]; e.a.ws = wss[i];
    e.a.q = q + (size_t)i * L.B * L.Hq * kD;
    e.a.out = out + (size_t)i * L.B * L.Hq * kD;
    e.a.n_splits = 0;
    fill_count_args(L, e.cn, e.a);
    e.a.safe_chunks = safe_chunks_for(L, Ns_safe[i], e.cn);
    e.a.n_q = 1;
    e.a.ablation = g_ablation;
    e.a.partials = reinterpret_cast<float*>(wss[i] + L.ws_partial_off);
    e.a.pages_host = nullptr;      // paged caches: a batched launch reads every cache's table from its buffer
    e.a.n_pages_host = 0;
  }
  for (int i = n; i < kMaxSeqs; ++i) T.s[i] = T.s[0];
  return launch(L, T, n, row_budget, g_chunks_per_iter, st);
}

void decode_mma_set_chunks_per_iter(int n) { g_chunks_per_iter = (n == 1 || n == 2) ? n : 0; }
void decode_mma_set_ablation(int mask) { g_ablation = mask & 3; }

// n_q > 1: q and out are [B, n_q, Hq, D], the partials of a launch's (up to) four rows per unit go to
// multi_partials [U * 4][max_splits][kPartialStride]
// N_safe: token count of the cache when its previous decode was launched (or it was prefilled): chunks packed by
// then are not written by any kernel that can still be running.
static int safe_chunks_for(const Layout& L, int N_safe, const Counts& cn_now) {
  const Counts old = counts_for(L, N_safe < 0 ? 0 : N_safe);
  const bool outer = L.grouping == 1;
  int s = (outer ? old.n_qk : old.n_qv) / kChunk;
  const int now = (outer ? cn_now.n_qk : cn_now.n_qv) / kChunk;
  return s < now ? s : now;
}

int launch_decode_mma(const Layout& L, const unsigned char* cache, unsigned char* ws, int N, const __half* q,
                      __half* out, int n_splits, cudaStream_t st, int n_q, float* multi_partials, int N_safe,
                      const uint32_t* pages_host, int n_pages_host) {
  const FormatLauncher launch = format_launcher(L);
  if (!launch) return -2;
  const Counts cn = counts_for(L, N);
  if (n_splits <= 0) n_splits = default_splits(L, L.U);
  if (n_splits > L.max_splits) n_splits = L.max_splits;
  if (n_splits > 128) n_splits = 128;            // slots of the merge tables in shared memory
  DecodeArgs a;
  a.cache = cache; a.ws = ws; a.q = q; a.out = out;
  a.n_splits = n_splits;
  fill_count_args(L, cn, a);
  a.safe_chunks = safe_chunks_for(L, N_safe, cn);
  a.n_q = n_q;
  a.ablation = g_ablation;
  a.partials = n_q > 1 ? multi_partials : reinterpret_cast<float*>(ws + L.ws_partial_off);
  a.pages_host = pages_host;
  a.n_pages_host = n_pages_host;
  if (n_q < 1 || (n_q > 1 && !multi_partials)) return -1;
  return launch(L, cn, a, n_splits, g_chunks_per_iter, st);
}

}  // namespace iq
