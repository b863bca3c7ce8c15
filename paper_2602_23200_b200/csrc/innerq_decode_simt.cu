// Generic decode attention: plain SIMT, fp32, per-element dequantisation through the packed-code
// accessors.  Serves every store kind (ROW / BLOCK / unquantised), bit width and group size; it is
// the fallback for shapes the fast kernel does not cover and an on-device cross-check for it.
// Split-K over token ranges with a separate merge kernel.
#include "innerq_device.cuh"
#include "innerq_kernels.h"

namespace iq {

constexpr int kSimtHeads = 8;    // query heads per pass (grid.z covers r > 8)
constexpr int kSimtTile = 32;

struct TensorView {              // one unit's view of a store
  const __half* sink;
  const __half* ring;
  Rec rec;
  Store S;
  int kind, bits, ring_cap, n_groups, meta_bytes;
  int n_sink, n_q, w_sink;
};

__device__ __forceinline__ TensorView make_view(const Layout& L, const Store& S, const unsigned char* cache, int u,
                                                int n_sink, int n_q) {
  TensorView v;
  v.sink = reinterpret_cast<const __half*>(cache + S.sink_off + (size_t)u * S.sink_stride);
  v.ring = reinterpret_cast<const __half*>(cache + S.ring_off + (size_t)u * S.ring_stride);
  v.rec = unit_rec(L, cache, u);
  v.S = S;
  v.meta_bytes = S.meta_bytes;
  v.kind = S.kind; v.bits = S.bits; v.ring_cap = S.ring_cap; v.n_groups = S.n_groups;
  v.n_sink = n_sink; v.n_q = n_q; v.w_sink = L.w_sink;
  return v;
}

// Value of element (token t, channel c); `quant` tells whether it came from the packed store
// (keys from the packed store are in the normalised domain).
__device__ __forceinline__ float element(const TensorView& v, int G, int t, int c, bool& quant) {
  quant = false;
  if (v.kind == kNone || t < v.n_sink) return __half2float(v.sink[(size_t)t * kD + c]);
  const int i = t - v.n_sink;
  if (i >= v.n_q) return __half2float(v.ring[(size_t)((t - v.w_sink) % v.ring_cap) * kD + c]);
  quant = true;
  float s, z;
  uint32_t code;
  if (v.kind == kRow) decode_meta(load_meta(row_meta_ptr(v.rec, v.S, i), c / G, v.meta_bytes), v.bits, s, z);
  else decode_meta(load_meta(block_meta_ptr(v.rec, v.S, i / G), block_meta_index(c), v.meta_bytes), v.bits, s, z);
  if (v.S.code_kind == kRow)
    code = row_code(reinterpret_cast<const uint32_t*>(row_code_ptr(v.rec, v.S, i)), c, v.bits, v.S.perm);
  else
    code = chunk_code(reinterpret_cast<const uint32_t*>(block_code_ptr(v.rec, v.S, i / kChunk)), i % kChunk, c, v.bits, v.S.perm);
  return fmaf(s, (float)code, z);
}

__global__ void __launch_bounds__(128) decode_simt_kernel(Layout L, Counts cn, const __half* __restrict__ q,
                                                          const unsigned char* __restrict__ cache,
                                                          float* __restrict__ partials, int n_splits, int split_len) {
  __shared__ float q_raw[kSimtHeads][kD], q_nrm[kSimtHeads][kD];
  __shared__ float sc[kSimtTile][kSimtHeads];
  __shared__ float m_run[kSimtHeads], l_run[kSimtHeads], corr[kSimtHeads];
  const int s = blockIdx.x, u = blockIdx.y, h0 = blockIdx.z * kSimtHeads;
  const int nh = min(kSimtHeads, L.r - h0);
  const int b = u / L.Hkv, hkv = u % L.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* norm = reinterpret_cast<const float*>(cache + L.norm_off) + (size_t)u * kD;
  const bool use_norm = L.k_normalize != 0 && L.k.kind == kRow;
  for (int h = 0; h < nh; ++h) {
    float v = __half2float(q[((size_t)b * L.Hq + hkv * L.r + h0 + h) * kD + tid]);
    q_raw[h][tid] = v;
    q_nrm[h][tid] = use_norm ? v * norm[tid] : v;
  }
  if (tid < kSimtHeads) { m_run[tid] = -INFINITY; l_run[tid] = 0.f; }
  __syncthreads();
  const TensorView kv = make_view(L, L.k, cache, u, L.k.kind == kNone ? cn.N : cn.n_sink, cn.n_qk);
  const TensorView vv = make_view(L, L.v, cache, u, L.v.kind == kNone ? cn.N : cn.n_sink, cn.n_qv);
  float acc[kSimtHeads];
#pragma unroll
  for (int h = 0; h < kSimtHeads; ++h) acc[h] = 0.f;
  const int t_begin = s * split_len, t_end = min(cn.N, t_begin + split_len);
  for (int t0 = t_begin; t0 < t_end; t0 += kSimtTile) {
    // scores: warp w takes tokens t0 + w, t0 + w + 4, ...; lane l takes channels 4l .. 4l+3
    for (int tt = warp; tt < kSimtTile; tt += 4) {
      const int t = t0 + tt;
      float d[kSimtHeads];
#pragma unroll
      for (int h = 0; h < kSimtHeads; ++h) d[h] = 0.f;
      if (t < t_end) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int c = 4 * lane + i;
          bool quant;
          const float kx = element(kv, L.G, t, c, quant);
#pragma unroll
          for (int h = 0; h < kSimtHeads; ++h)
            if (h < nh) d[h] = fmaf(kx, quant ? q_nrm[h][c] : q_raw[h][c], d[h]);
        }
      }
#pragma unroll
      for (int h = 0; h < kSimtHeads; ++h) {
        float v = d[h];
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) sc[tt][h] = t < t_end ? v * L.sm_scale : -INFINITY;
      }
    }
    __syncthreads();
    // online softmax: warp w takes heads w and w + 4; lane = token of the tile
    for (int h = warp; h < nh; h += 4) {
      const float sv = sc[lane][h];
      float mt = sv;
      for (int o = 16; o > 0; o >>= 1) mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, o));
      const float m_new = fmaxf(m_run[h], mt);
      const float p = __expf(sv - m_new);
      float ps = p;
      for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
      sc[lane][h] = p;
      if (lane == 0) {
        const float cr = __expf(m_run[h] - m_new);
        corr[h] = cr;
        l_run[h] = l_run[h] * cr + ps;
        m_run[h] = m_new;
      }
    }
    __syncthreads();
    // values: thread c owns channel c
    {
      float add[kSimtHeads];
#pragma unroll
      for (int h = 0; h < kSimtHeads; ++h) add[h] = 0.f;
      const int nt = min(kSimtTile, t_end - t0);
      for (int tt = 0; tt < nt; ++tt) {
        bool quant;
        const float vx = element(vv, L.G, t0 + tt, tid, quant);
#pragma unroll
        for (int h = 0; h < kSimtHeads; ++h)
          if (h < nh) add[h] = fmaf(sc[tt][h], vx, add[h]);
      }
#pragma unroll
      for (int h = 0; h < kSimtHeads; ++h)
        if (h < nh) acc[h] = fmaf(acc[h], corr[h], add[h]);
    }
    __syncthreads();
  }
  for (int h = 0; h < nh; ++h) {
    float* P = partials + (((size_t)b * L.Hq + hkv * L.r + h0 + h) * n_splits + s) * kPartialStride;
    P[tid] = acc[h];
    if (tid == 0) { P[kD] = m_run[h]; P[kD + 1] = l_run[h]; }
  }
}

// out[head] = sum_s acc_s * exp(m_s - m) / sum_s l_s * exp(m_s - m)
__global__ void __launch_bounds__(128) merge_partials_kernel(const float* __restrict__ partials, int n_splits,
                                                             __half* __restrict__ out) {
  const int head = blockIdx.x, c = threadIdx.x;
  const float* P = partials + (size_t)head * n_splits * kPartialStride;
  float m = -INFINITY;
  for (int s = 0; s < n_splits; ++s) m = fmaxf(m, P[s * kPartialStride + kD]);
  float num = 0.f, den = 0.f;
  for (int s = 0; s < n_splits; ++s) {
    const float ms = P[s * kPartialStride + kD];
    if (ms == -INFINITY) continue;
    const float w = __expf(ms - m);
    num = fmaf(P[s * kPartialStride + c], w, num);
    den = fmaf(P[s * kPartialStride + kD + 1], w, den);
  }
  out[(size_t)head * kD + c] = __float2half_rn(num / den);
}

int launch_decode_simt(const Layout& L, const unsigned char* cache, unsigned char* ws, int N, const __half* q,
                       __half* out, int n_splits, cudaStream_t st) {
  const Counts cn = counts_for(L, N);
  if (n_splits <= 0) {
    n_splits = (4 * 148 + L.U - 1) / L.U;
    const int max_by_len = (N + 4 * kSimtTile - 1) / (4 * kSimtTile);
    if (n_splits > max_by_len) n_splits = max_by_len;
  }
  if (n_splits > L.max_splits) n_splits = L.max_splits;
  if (n_splits < 1) n_splits = 1;
  int split_len = (N + n_splits - 1) / n_splits;
  split_len = (split_len + kSimtTile - 1) / kSimtTile * kSimtTile;
  float* partials = reinterpret_cast<float*>(ws + L.ws_partial_off);
  dim3 grid(n_splits, L.U, (L.r + kSimtHeads - 1) / kSimtHeads);
  decode_simt_kernel<<<grid, 128, 0, st>>>(L, cn, q, cache, partials, n_splits, split_len);
  merge_partials_kernel<<<L.B * L.Hq, 128, 0, st>>>(partials, n_splits, out);
  return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace iq
