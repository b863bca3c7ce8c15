// Decode attention over an UNQUANTISED fp16 cache (grouping = FP16): the comparison point of the same
// shape for the packed kernels.  Same structure as the packed kernel where it applies: split over token
// ranges, per-warp online soft-max, warp-level MMA with hi/lo split operands, cross-CTA merge by the last
// CTA to arrive.  It streams 16x the bytes per element of a 2-bit cache and is purely HBM-bound, so
// operands go straight from global memory to registers with coalesced 128-bit loads (no staging): per
// 16-token tile a warp reads 4 KB of keys and 4 KB of values.
//
// Fragment mapping.  Keys are the A operand of q.K^T (rows = tokens): lane (gid, tid4) loads, for token
// rows gid and gid+8, the 16-byte pieces tid4, tid4+4, tid4+8, tid4+12 of the 256-byte row; a piece holds
// the two channel pairs of two k-steps, and q is permuted to match (the permutation does not depend on
// the row).  Values are the A operand of V^T.p (rows = channels): lane (gid, tid4) loads, for token rows
// 2*tid4, 2*tid4+1, 2*tid4+8, 2*tid4+9, the pieces gid and gid+8, and byte-permutes two rows into
// (channel; token, token+1) pairs.
#include "innerq_device.cuh"
#include "innerq_kernels.h"

namespace iq {

namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kHeads = 4;
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t split_hi_lo(float x) {
  const __half hi = __float2half_rn(x);
  const __half lo = __float2half_rn(x - __half2float(hi));
  return (uint32_t)__half_as_ushort(hi) | ((uint32_t)__half_as_ushort(lo) << 16);
}
__device__ __forceinline__ float pow2i(int e) { return __int_as_float((e + 127) << 23); }

struct Fp16Args {
  const unsigned char* cache;
  unsigned char* ws;
  const __half* q;
  __half* out;
  int n_tokens, n_splits, tiles_per_split, head0;
};

__global__ void __launch_bounds__(kThreads, 2) decode_fp16_kernel(const Layout L, const Fp16Args a) {
  __shared__ float q_s[kHeads][kD];
  __shared__ int qe_s[kHeads];
  __shared__ float wres[kWarps][kHeads][kD + 2];
  __shared__ float mw[kHeads][128], lw[kHeads][128];
  __shared__ unsigned int s_ticket;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gid = lane >> 2, j = lane & 3;
  const int u = blockIdx.x, split = blockIdx.y;
  const int b = u / L.Hkv, hkv = u % L.Hkv;
  const int nh = min(kHeads, L.r - a.head0);
  const int head_base = b * L.Hq + hkv * L.r + a.head0;
  const int N = a.n_tokens;

  // ---- q'' = q * sm_scale * log2(e), per-head exponent for the fp16 hi/lo split
  for (int i = tid; i < kHeads * kD; i += kThreads) {
    const int h = i >> 7, c = i & (kD - 1);
    q_s[h][c] = h < nh ? __half2float(a.q[(size_t)(head_base + h) * kD + c]) * (L.sm_scale * kLog2e) : 0.f;
  }
  __syncthreads();
  if (warp < kHeads) {
    float am = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) am = fmaxf(am, fabsf(q_s[warp][e * 32 + lane]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, o));
    if (lane == 0) {
      int e = 0;
      if (am > 0.f && am < INFINITY) frexpf(am, &e);
      qe_s[warp] = e;
    }
  }
  __syncthreads();
  // B fragments of q'' for the 8 k-steps: column gid = (head gid/2, hi|lo); k rows follow the key permutation
  uint32_t Bq[8][2];
  {
    const int h = gid >> 1, part = gid & 1;
    const float bscale = pow2i(14 - qe_s[h]);
#pragma unroll
    for (int s = 0; s < 8; ++s) {
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int c0 = 8 * (j + 4 * (s >> 1)) + 4 * (s & 1) + 2 * rr;      // channels of (k-step s, column pair rr)
        const uint32_t v0 = split_hi_lo(q_s[h][c0] * bscale), v1 = split_hi_lo(q_s[h][c0 + 1] * bscale);
        Bq[s][rr] = part ? ((v0 >> 16) | (v1 & 0xFFFF0000u)) : ((v0 & 0xFFFFu) | (v1 << 16));
      }
    }
  }
  const float kfac = pow2i(-(14 - qe_s[j]));          // scores of head j: accumulator * kfac

  // ---- this warp's range of 16-token tiles
  const int n_tiles = (N + 15) / 16;
  const int t_lo = min(n_tiles, split * a.tiles_per_split), t_hi = min(n_tiles, t_lo + a.tiles_per_split);
  const int n_t = t_hi - t_lo;
  const int w_lo = t_lo + (n_t * warp) / kWarps, w_hi = t_lo + (n_t * (warp + 1)) / kWarps;
  const uint4* Kb = reinterpret_cast<const uint4*>(a.cache + L.k.sink_off + (size_t)u * L.k.sink_stride);
  const uint4* Vb = reinterpret_cast<const uint4*>(a.cache + L.v.sink_off + (size_t)u * L.v.sink_stride);

  float m_run = -INFINITY, l_part = 0.f;
  float out_acc[8][4];
#pragma unroll
  for (int m = 0; m < 8; ++m)
#pragma unroll
    for (int e = 0; e < 4; ++e) out_acc[m][e] = 0.f;

#pragma unroll 1
  for (int tile = w_lo; tile < w_hi; ++tile) {
    const int t0 = tile * 16;
    // ---- loads (rows beyond N are clamped to the last token and masked below)
    const int rA = min(t0 + gid, N - 1), rB = min(t0 + gid + 8, N - 1);
    uint4 ka[4], kb[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      ka[i] = __ldg(Kb + (size_t)rA * 16 + j + 4 * i);
      kb[i] = __ldg(Kb + (size_t)rB * 16 + j + 4 * i);
    }
    uint4 v[4][2];
    {
      const int tr[4] = {min(t0 + 2 * j, N - 1), min(t0 + 2 * j + 1, N - 1), min(t0 + 2 * j + 8, N - 1),
                         min(t0 + 2 * j + 9, N - 1)};
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        v[r][0] = __ldg(Vb + (size_t)tr[r] * 16 + gid);
        v[r][1] = __ldg(Vb + (size_t)tr[r] * 16 + gid + 8);
      }
    }
    // ---- scores
    float c4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      mma16816(c4, ka[i].x, kb[i].x, ka[i].y, kb[i].y, Bq[2 * i][0], Bq[2 * i][1]);
      mma16816(c4, ka[i].z, kb[i].z, ka[i].w, kb[i].w, Bq[2 * i + 1][0], Bq[2 * i + 1][1]);
    }
    float sA = (c4[0] + c4[1]) * kfac, sB = (c4[2] + c4[3]) * kfac;
    if (t0 + gid >= N) sA = -INFINITY;
    if (t0 + gid + 8 >= N) sB = -INFINITY;
    // ---- online softmax (log2 domain), head j
    float cmax = fmaxf(sA, sB);
    cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 4));
    cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 8));
    cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, 16));
    const float m_new = fmaxf(m_run, cmax);
    if (__any_sync(0xffffffffu, m_new > m_run)) {
      const float alpha = ex2_approx(m_run - m_new);
      l_part *= alpha;
#pragma unroll
      for (int m = 0; m < 8; ++m)
#pragma unroll
        for (int e = 0; e < 4; ++e) out_acc[m][e] *= alpha;
    }
    m_run = m_new;
    const float pA = ex2_approx(sA - m_new), pB = ex2_approx(sB - m_new);
    l_part += pA + pB;
    const uint32_t b0 = movmatrix_trans(split_hi_lo(pA * 1024.f)), b1 = movmatrix_trans(split_hi_lo(pB * 1024.f));
    // ---- values: m-tile k = channel pair (2k, 2k+1) of piece gid (k < 4) or gid + 8 (k >= 4)
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const uint32_t* T0 = reinterpret_cast<const uint32_t*>(&v[0][half]);
      const uint32_t* T1 = reinterpret_cast<const uint32_t*>(&v[1][half]);
      const uint32_t* T8 = reinterpret_cast<const uint32_t*>(&v[2][half]);
      const uint32_t* T9 = reinterpret_cast<const uint32_t*>(&v[3][half]);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t a0 = __byte_perm(T0[k], T1[k], 0x5410), a1 = __byte_perm(T0[k], T1[k], 0x7632);
        const uint32_t a2 = __byte_perm(T8[k], T9[k], 0x5410), a3 = __byte_perm(T8[k], T9[k], 0x7632);
        mma16816(out_acc[half * 4 + k], a0, a1, a2, a3, b0, b1);
      }
    }
  }

  // ---- warp result -> CTA partial (channel of out_acc[m][2*rh + e]: piece base + 2*(m%4) + rh)
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 4);
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 8);
  l_part += __shfl_xor_sync(0xffffffffu, l_part, 16);
  {
    float* mine = wres[warp][j];
    const bool any = w_hi > w_lo;
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      const int ch = (m < 4 ? 8 * gid : 64 + 8 * gid) + 2 * (m & 3);
      mine[ch] = any ? (out_acc[m][0] + out_acc[m][1]) * 0x1p-10f : 0.f;
      mine[ch + 1] = any ? (out_acc[m][2] + out_acc[m][3]) * 0x1p-10f : 0.f;
    }
    if (gid == 0) {
      mine[kD] = any ? m_run : -INFINITY;
      mine[kD + 1] = any ? l_part : 0.f;
    }
  }
  __syncthreads();
  float* partials = reinterpret_cast<float*>(a.ws + L.ws_partial_off);
  for (int i = tid; i < nh * kD; i += kThreads) {
    const int h = i >> 7, c = i & (kD - 1);
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, wres[w][h][kD]);
    float num = 0.f, den = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float wgt = wres[w][h][kD] == -INFINITY ? 0.f : exp2f(wres[w][h][kD] - M);
      num = fmaf(wres[w][h][c], wgt, num);
      den = fmaf(wres[w][h][kD + 1], wgt, den);
    }
    float* P = partials + ((size_t)(head_base + h) * L.max_splits + split) * kPartialStride;
    P[c] = num;
    if (c == 0) { P[kD] = M; P[kD + 1] = den; }
  }

  // ---- cross-CTA merge by the last CTA of the unit to arrive
  __syncthreads();                 // all partial writes of this CTA happen-before thread 0's ticket below
  if (tid == 0) {
    // release: publishes the whole CTA's partial (ordered before this thread by the barrier) with the ticket;
    // acquire: the CTA that draws the last ticket sees every other CTA's partial
    unsigned int t;
    asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;"
                 : "=r"(t) : "l"(reinterpret_cast<unsigned int*>(a.ws + L.ws_ticket_off) + u) : "memory");
    s_ticket = t;
  }
  __syncthreads();
  if (s_ticket != gridDim.y - 1) return;
  const int n_parts = gridDim.y;
  for (int i = tid; i < nh * n_parts; i += kThreads) {
    const int h = i / n_parts, s = i % n_parts;
    const float* P = partials + ((size_t)(head_base + h) * L.max_splits + s) * kPartialStride;
    mw[h][s] = __ldcg(P + kD);
    lw[h][s] = __ldcg(P + kD + 1);
  }
  __syncthreads();
  for (int i = tid; i < nh * kD; i += kThreads) {
    const int h = i >> 7, c = i & (kD - 1);
    const float* P = partials + (size_t)(head_base + h) * L.max_splits * kPartialStride + c;
    float M = -INFINITY;
    for (int s = 0; s < n_parts; ++s) M = fmaxf(M, mw[h][s]);
    float num = 0.f, den = 0.f;
    for (int s0 = 0; s0 < n_parts; s0 += 16) {
      float vv[16];
#pragma unroll
      for (int e = 0; e < 16; ++e) vv[e] = s0 + e < n_parts ? __ldcg(P + (size_t)(s0 + e) * kPartialStride) : 0.f;
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        if (s0 + e < n_parts) {
          const float ms = mw[h][s0 + e];
          const float wgt = ms == -INFINITY ? 0.f : exp2f(ms - M);
          num = fmaf(vv[e], wgt, num);
          den = fmaf(lw[h][s0 + e], wgt, den);
        }
      }
    }
    a.out[(size_t)(head_base + h) * kD + c] = __float2half_rn(num / den);
  }
  if (tid == 0) reinterpret_cast<unsigned int*>(a.ws + L.ws_ticket_off)[u] = 0u;
}

}  // namespace

int launch_decode_fp16(const Layout& L, const unsigned char* cache, unsigned char* ws, int N, const __half* q,
                       __half* out, int n_splits, cudaStream_t st) {
  if (L.k.kind != kNone || L.v.kind != kNone) return -2;
  const int n_tiles = (N + 15) / 16;
  if (n_splits <= 0) n_splits = (2 * 148) / L.U;
  if (n_splits < 1) n_splits = 1;
  const int by_work = (n_tiles + kWarps - 1) / kWarps;
  if (n_splits > by_work) n_splits = by_work;
  if (n_splits > L.max_splits) n_splits = L.max_splits;
  if (n_splits > 128) n_splits = 128;
  Fp16Args a;
  a.cache = cache; a.ws = ws; a.q = q; a.out = out;
  a.n_tokens = N;
  a.n_splits = n_splits;
  a.tiles_per_split = (n_tiles + n_splits - 1) / n_splits;
  int launches = 0;
  for (int h0 = 0; h0 < L.r; h0 += kHeads) {
    a.head0 = h0;
    decode_fp16_kernel<<<dim3(L.U, n_splits), kThreads, 0, st>>>(L, a);
    ++launches;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace iq
