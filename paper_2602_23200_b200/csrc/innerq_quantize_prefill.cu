// Prefill quantisers: the middle tokens of every unit into the ROW store (groups of G channels inside a token,
// Section "InnerQ" for keys) and the BLOCK store (per-channel groups of G tokens, values).
//
// Both are built around one work item: 32 values of one group held in the registers of one thread (a group of
// 64 or 128 values is 2 or 4 such threads, which exchange their minima / maxima and error sums).  The thread
// makes the passes the method needs over its registers: min / max, then (hybrid mode only) the L1 errors of both
// candidates, then the codes of the chosen mode.  All value arithmetic is the same sequence of single, correctly
// rounded fp32 operations as in group_params / asym_code / sym_code, so stored bits do not depend on the kernel:
// rounding to an integer is done by adding 1.5 * 2^23 (round-to-nearest-even at unit granularity, identical to
// rintf for |t| < 2^22; codes are bounded by a few times 2^b), which leaves the code in the low mantissa bits.
#include "innerq_device.cuh"
#include "innerq_kernels.h"

namespace iq {

namespace {

constexpr float kMagic = 12582912.0f;       // 1.5 * 2^23
constexpr int kSeg = 32;                    // values per thread

struct SegCoder {
  float z_a, inv_a, s_a, lo_a, hi_a;        // asymmetric: clamp bounds in the magic domain
  float inv_s, s_s, off_s, lo_s, hi_s;      // symmetric (offset-binary): magic + 2^(b-1), bounds
  __device__ __forceinline__ explicit SegCoder(const GroupParams& p) {
    z_a = p.z_a; inv_a = p.inv_a; s_a = p.s_a; lo_a = kMagic; hi_a = kMagic + p.L;
    inv_s = p.inv_s; s_s = p.s_s; off_s = kMagic + p.half; lo_s = off_s + p.q_lo; hi_s = off_s + p.q_hi;
  }
  // code plus magic (asymmetric) / plus magic + 2^(b-1) (symmetric): the low mantissa bits are the stored code.
  // CLAMP = false leaves out the clamp to the code range, for groups where no_clip() holds.
  template <bool CLAMP> __device__ __forceinline__ float asym(float x) const {
    const float t = __fadd_rn(__fmul_rn(__fsub_rn(x, z_a), inv_a), kMagic);
    return CLAMP ? fminf(fmaxf(t, lo_a), hi_a) : t;
  }
  template <bool CLAMP> __device__ __forceinline__ float sym(float x) const {
    const float t = __fadd_rn(__fmul_rn(x, inv_s), off_s);
    return CLAMP ? fminf(fmaxf(t, lo_s), hi_s) : t;
  }
  // Both coders are non-decreasing in x (each step is a correctly rounded monotone operation and the reciprocal
  // scales are >= 0), so if the group's minimum and maximum land inside the code range, every value does.
  __device__ __forceinline__ bool no_clip(float mn, float mx) const {
    return asym<false>(mn) >= lo_a && asym<false>(mx) <= hi_a && sym<false>(mn) >= lo_s && sym<false>(mx) <= hi_s;
  }
  // L1 reconstruction errors of one value (used only to pick the mode of a hybrid group)
  template <bool CLAMP> __device__ __forceinline__ float err_asym(float x) const {
    return fabsf(__fmaf_rn(-s_a, asym<CLAMP>(x) - kMagic, __fsub_rn(x, z_a)));
  }
  template <bool CLAMP> __device__ __forceinline__ float err_sym(float x) const {
    return fabsf(__fmaf_rn(-s_s, sym<CLAMP>(x) - off_s, x));
  }
};

// The coder of the chosen mode as one formula, clamp(((x - z) * inv) + off): symmetric is z = 0 (x - 0 is exact).
struct ChosenCoder {
  float z, inv, off, lo, hi;
  __device__ __forceinline__ ChosenCoder(const SegCoder& c, bool asym)
      : z(asym ? c.z_a : 0.f), inv(asym ? c.inv_a : c.inv_s), off(asym ? kMagic : c.off_s), lo(asym ? c.lo_a : c.lo_s),
        hi(asym ? c.hi_a : c.hi_s) {}
  // bits of (1.5 * 2^23 + code): 0x4B400000 + code
  template <bool CLAMP> __device__ __forceinline__ uint32_t code_bits(float x) const {
    const float t = __fadd_rn(__fmul_rn(__fsub_rn(x, z), inv), off);
    return __float_as_uint(CLAMP ? fminf(fmaxf(t, lo), hi) : t);
  }
};

__device__ __forceinline__ float min3(float a, float b, float c) {
  float r;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// min / max of 32 registers (three-input min / max: two values per instruction)
__device__ __forceinline__ void seg_minmax(const float (&x)[kSeg], float& mn, float& mx) {
  float a = fminf(x[0], x[1]), b = fmaxf(x[0], x[1]);
#pragma unroll
  for (int e = 2; e < kSeg; e += 2) { a = min3(a, x[e], x[e + 1]); b = max3(b, x[e], x[e + 1]); }
  mn = a; mx = b;
}

template <bool CLAMP>
__device__ __forceinline__ void seg_errors(const SegCoder& sc, const float (&x)[kSeg], float& ea, float& es) {
  float a0 = 0.f, a1 = 0.f, s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int e = 0; e < kSeg; e += 2) {
    a0 += sc.template err_asym<CLAMP>(x[e]); a1 += sc.template err_asym<CLAMP>(x[e + 1]);
    s0 += sc.template err_sym<CLAMP>(x[e]);  s1 += sc.template err_sym<CLAMP>(x[e + 1]);
  }
  ea = a0 + a1; es = s0 + s1;
}

constexpr uint32_t kMagicBits = 0x4B400000u;     // bit pattern of kMagic

// Packs the 32 codes of a ROW-store segment into its local words (positions of segment 0, see the kernel).
// Codes arrive as kMagicBits + code; with 2 or 4 bits the fields are filled by wrap-around adds of the shifted
// patterns, the shifted kMagicBits being taken off at the end (a compile-time constant per word).
template <int BITS, bool CLAMP>
__device__ __forceinline__ void pack_row_segment(const ChosenCoder& cc, const float (&x)[kSeg], uint32_t (&lw)[4],
                                                 uint32_t (&hw)[4]) {
  constexpr int PB = BITS == 3 ? 2 : BITS, WM = PB == 2 ? 2 : 4;
  uint32_t cw[4] = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int i = 0; i < 4; ++i) { lw[i] = 0u; hw[i] = 0u; }
#pragma unroll
  for (int e = 0; e < kSeg; ++e) {
    const uint32_t code = cc.template code_bits<CLAMP>(x[e]);
    const BitPos lo = row_pos_plane(e, PB);            // constants: segment 0's positions
    if constexpr (BITS == 3) {
      const BitPos hi = row_pos_plane(e, 1);
      lw[lo.word / WM] |= (code & 3u) << lo.bit;
      hw[hi.word] |= ((code >> 2) & 1u) << hi.bit;
    } else {
      lw[lo.word / WM] += code << lo.bit;
      cw[lo.word / WM] += kMagicBits << lo.bit;
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) lw[i] -= cw[i];
}

// Same for a BLOCK-store segment (32 tokens of one channel; positions of channel 0).
template <int BITS, bool CLAMP>
__device__ __forceinline__ void pack_block_segment(const ChosenCoder& cc, const float (&x)[kSeg],
                                                   uint32_t (&lw)[BITS == 4 ? 8 : 4], uint32_t (&hw)[4]) {
  constexpr int PB = BITS == 3 ? 2 : BITS, NW = PB == 4 ? 8 : 4;
  uint32_t cw[NW];
#pragma unroll
  for (int i = 0; i < NW; ++i) { lw[i] = 0u; cw[i] = 0u; }
#pragma unroll
  for (int i = 0; i < 4; ++i) hw[i] = 0u;
#pragma unroll
  for (int t = 0; t < kSeg; ++t) {
    const uint32_t code = cc.template code_bits<CLAMP>(x[t]);
    const BitPos lo = block_pos_plane(t, 0, PB);       // constants: channel 0's positions
    const int li = PB == 4 ? (lo.word >> 8) * 4 + ((lo.word >> 2) & 3) : (lo.word >> 2) & 3;   // (k-step,) tid4
    if constexpr (BITS == 3) {
      const BitPos hi = block_pos_plane(t, 0, 1);
      lw[li] |= (code & 3u) << lo.bit;
      hw[(hi.word >> 2) & 3] |= ((code >> 2) & 1u) << hi.bit;
    } else {
      lw[li] += code << lo.bit;
      cw[li] += kMagicBits << lo.bit;
    }
  }
#pragma unroll
  for (int i = 0; i < NW; ++i) lw[i] -= cw[i];
}

// Byte-order layout (Store::perm = 1, 2- or 4-bit codes).  ROW segment = 32 consecutive channels = one bit position of
// 32 bytes of the row: the codes go to position 0 of 8 words here (index 2 * j + h, see row_pos_i8), the caller
// places them in the row and shifts them to its position.
template <int BITS, bool CLAMP>
__device__ __forceinline__ void pack_row_segment_i8(const ChosenCoder& cc, const float (&x)[kSeg], uint32_t (&w8)[8]) {
  uint32_t cw[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { w8[i] = 0u; cw[i] = 0u; }
#pragma unroll
  for (int e = 0; e < kSeg; ++e) {
    const uint32_t code = cc.template code_bits<CLAMP>(x[e]);
    const BitPos p = row_pos_i8(e, BITS);               // constants: positions of channels 0..31 (bit position 0)
    const int li = BITS == 4 ? 2 * (p.word >> 2) + (p.word & 1) : p.word;
    w8[li] += code << p.bit;
    cw[li] += kMagicBits << p.bit;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) w8[i] -= cw[i];
}
// BLOCK segment = 32 tokens of one channel: bytes of the 8 words [j][half] of its fragment row (see block_pos_i8), at
// bit position 0 here.  Word index: 2 * j + half.
template <int BITS, bool CLAMP>
__device__ __forceinline__ void pack_block_segment_i8(const ChosenCoder& cc, const float (&x)[kSeg], uint32_t (&w8)[8]) {
  uint32_t cw[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) { w8[i] = 0u; cw[i] = 0u; }
#pragma unroll
  for (int t = 0; t < kSeg; ++t) {
    const uint32_t code = cc.template code_bits<CLAMP>(x[t]);
    const BitPos p = block_pos_i8(t, 0, BITS);          // constants: channel 0 (W = 0, gid = 0, position 0, rh = 0)
    const int li = 2 * ((p.word >> 2) & 3) + ((p.word >> 1) & 1);      // 2 * j + half
    w8[li] += code << p.bit;
    cw[li] += kMagicBits << p.bit;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) w8[i] -= cw[i];
}

// 3-bit codes in byte order (see row_pos_i8_3 / block_pos_i8_3): the 2-bit plane's words as above (bit position 0)
// and the 1-bit plane's bits at bit 0 of their bytes; `odd` (bit position of the segment is odd) picks the split of
// a code between the planes.  ROW: hw[h][j] = 1-bit plane word j, bits of row half h.
template <bool CLAMP>
__device__ __forceinline__ void pack_row_segment_i8_3(const ChosenCoder& cc, const float (&x)[kSeg], int odd,
                                                      uint32_t (&w8)[8], uint32_t (&hw)[2][4]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) { w8[i] = 0u; hw[i >> 2][i & 3] = 0u; }
  const int sh_lo = odd, sh_hi = odd ? 0 : 2;
#pragma unroll
  for (int e = 0; e < kSeg; ++e) {
    const uint32_t code = cc.template code_bits<CLAMP>(x[e]);      // kMagicBits + code: the low bits are the code
    const int lw = e >> 2, j = lw & 3, h = lw >> 2, sh = 8 * (e & 3);
    w8[2 * j + h] |= ((code >> sh_lo) & 3u) << sh;
    hw[h][j] |= ((code >> sh_hi) & 1u) << sh;
  }
}
// BLOCK: word index 2 * j + half in both planes.
template <bool CLAMP>
__device__ __forceinline__ void pack_block_segment_i8_3(const ChosenCoder& cc, const float (&x)[kSeg], int odd,
                                                        uint32_t (&w8)[8], uint32_t (&h8)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) { w8[i] = 0u; h8[i] = 0u; }
  const int sh_lo = odd, sh_hi = odd ? 0 : 2;
#pragma unroll
  for (int t = 0; t < kSeg; ++t) {
    const uint32_t code = cc.template code_bits<CLAMP>(x[t]);
    const int k = 4 * (t & 7) + (t >> 3), li = 2 * ((k & 15) >> 2) + (k >> 4), sh = 8 * (k & 3);
    w8[li] |= ((code >> sh_lo) & 3u) << sh;
    h8[li] |= ((code >> sh_hi) & 1u) << sh;
  }
}

__device__ __forceinline__ void unpack8(const uint4& v, float* x) {
  const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(h[i]);
    x[2 * i] = f.x; x[2 * i + 1] = f.y;
  }
}

// ------------------------------------------------------------------ ROW store
// A warp quantises 8 consecutive tokens per iteration: lane = 4 * (token in the batch) + segment, segment =
// channels 32*seg .. 32*seg+31.  The 8 packed rows and their metadata entries are contiguous in the chunk record.
// Positions of the segment's codes (see row_pos_plane): element e of segment 0 sits in local word j = tid4(e);
// for segment seg the word index and the bit offset move by a per-plane amount that depends on seg only.
template <int BITS, bool NORM, bool I8 = false>
__global__ void __launch_bounds__(128) quantize_rows_prefill_kernel(Layout L, Store S, const __half* __restrict__ X, int N,
                                                                    int n_q, unsigned char* __restrict__ cache,
                                                                    const float* __restrict__ inv_norm) {
  constexpr int RW = 4 * BITS;                // 32-bit words per packed row
  constexpr int PB = BITS == 3 ? 2 : BITS;    // bits of the primary plane
  __shared__ uint32_t stage_all[4][8 * RW];
  const int u = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int seg = lane & 3, tk = lane >> 2;
  const int gl = L.G >> 5;                    // lanes per group: 1, 2 or 4
  uint32_t* stage = stage_all[warp];
#pragma unroll
  for (int k = 0; k < RW / 4; ++k) stage[lane + 32 * k] = 0u;
  float inv[NORM ? kSeg : 1];
  if constexpr (NORM) {
    const float4* p = reinterpret_cast<const float4*>(inv_norm + (size_t)u * kD + kSeg * seg);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float4 v = __ldg(p + k);
      inv[4 * k] = v.x; inv[4 * k + 1] = v.y; inv[4 * k + 2] = v.z; inv[4 * k + 3] = v.w;
    }
  }
  // where this segment's local words go inside the row, and by how much its fields are shifted
  constexpr int WM = PB == 2 ? 2 : 4;        // row words between consecutive local words
  const int w_add = PB == 2 ? (seg >> 1) : seg;
  const int sh_lo = PB == 2 ? 8 * (seg & 1) : 0, sh_hi = 4 * seg;
  const Rec rec = unit_rec(L, cache, u);
  const __half* Xu = X + ((size_t)u * N + L.w_sink) * kD + kSeg * seg;
  const int n_batches = (n_q + 7) >> 3;
  const int stride = gridDim.x * 4;
  int bi = blockIdx.x * 4 + warp;
  uint4 raw[4];
  if (bi < n_batches) {
    const uint4* src = reinterpret_cast<const uint4*>(Xu + (size_t)min(bi * 8 + tk, n_q - 1) * kD);
#pragma unroll
    for (int k = 0; k < 4; ++k) raw[k] = __ldg(src + k);
  }
  for (; bi < n_batches; bi += stride) {
    const int i0 = bi * 8;
    float x[kSeg];
#pragma unroll
    for (int k = 0; k < 4; ++k) unpack8(raw[k], x + 8 * k);
    if (bi + stride < n_batches) {            // next batch's rows are requested before this one is worked on
      const uint4* src = reinterpret_cast<const uint4*>(Xu + (size_t)min((bi + stride) * 8 + tk, n_q - 1) * kD);
#pragma unroll
      for (int k = 0; k < 4; ++k) raw[k] = __ldg(src + k);
    }
    if constexpr (NORM) {
#pragma unroll
      for (int e = 0; e < kSeg; ++e) x[e] = __fmul_rn(x[e], inv[e]);
    }
    float mn, mx;
    seg_minmax(x, mn, mx);
    for (int o = 1; o < gl; o <<= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    const GroupParams p = group_params(mn, mx, fmaxf(fabsf(mn), fabsf(mx)), BITS, L.sym_variant);
    const SegCoder sc(p);
    const bool no_clip = sc.no_clip(mn, mx);        // the same for all lanes of a group
    bool asym = S.mode == 1;
    if (S.mode == 2) {
      float ea, es;
      if (no_clip) seg_errors<false>(sc, x, ea, es);
      else seg_errors<true>(sc, x, ea, es);
      for (int o = 1; o < gl; o <<= 1) {
        ea += __shfl_xor_sync(0xffffffffu, ea, o);
        es += __shfl_xor_sync(0xffffffffu, es, o);
      }
      asym = ea < es;
    }
    const ChosenCoder cc(sc, asym);
    uint32_t* row = stage + tk * RW;
    if constexpr (I8 && BITS == 3) {
      uint32_t w8[8], hw[2][4];
      if (no_clip) pack_row_segment_i8_3<false>(cc, x, seg & 1, w8, hw);
      else pack_row_segment_i8_3<true>(cc, x, seg & 1, w8, hw);
      __syncwarp();                                        // the stage is zero and no longer being read
      const int b0 = hi_bit_i8(seg, 0), b1 = hi_bit_i8(seg, 1);
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) atomicOr(&row[jj], w8[jj] << (2 * seg));
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) atomicOr(&row[8 + jj], (hw[0][jj] << b0) | (hw[1][jj] << b1));
    } else if constexpr (I8) {
      uint32_t w8[8];
      if (no_clip) pack_row_segment_i8<BITS, false>(cc, x, w8);
      else pack_row_segment_i8<BITS, true>(cc, x, w8);
      __syncwarp();                                        // the stage is zero and no longer being read
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) {
        if constexpr (BITS == 2) atomicOr(&row[jj], w8[jj] << (2 * seg));
        else atomicOr(&row[4 * (jj >> 1) + 2 * (seg >> 1) + (jj & 1)], w8[jj] << (4 * (seg & 1)));
      }
    } else {
      uint32_t lw[4], hw[4];
      if (no_clip) pack_row_segment<BITS, false>(cc, x, lw, hw);
      else pack_row_segment<BITS, true>(cc, x, lw, hw);
      __syncwarp();                                        // the stage is zero and no longer being read
#pragma unroll
      for (int jj = 0; jj < 4; ++jj) {
        atomicOr(&row[WM * jj + w_add], lw[jj] << sh_lo);
        if constexpr (BITS == 3) atomicOr(&row[row_hi_plane_word() + jj], hw[jj] << sh_hi);
      }
    }
    const int i = i0 + tk;
    if (i < n_q && (lane & (gl - 1)) == 0)
      store_meta(row_meta_ptr(rec, S, i0), (size_t)tk * S.n_groups + (seg >> (gl >> 1)), S.meta_bytes, group_meta(p, asym));
    __syncwarp();
    uint32_t* dst = reinterpret_cast<uint32_t*>(row_code_ptr(rec, S, i0));
#pragma unroll
    for (int k = 0; k < RW / 4; ++k) {
      const int idx = lane + 32 * k;
      if (i0 + idx / RW < n_q) dst[idx] = stage[idx];
      stage[idx] = 0u;
    }
  }
}

// ------------------------------------------------------------------ BLOCK store
// A CTA of 64 * (G / 32) threads quantises one group of G tokens x 128 channels per iteration: thread
// (channel pair cp, chunk k) owns tokens 32k .. 32k+31 of channels 2cp and 2cp+1, read straight from global memory
// (one 32-bit load per token: a warp reads 128 contiguous bytes of each token row).  The two channels of a pair
// are the two row halves of one MMA fragment row pair, so between them they fill whole words of the packed chunk
// and no staging or atomics are needed (3-bit: the 1-bit plane's words are shared with the neighbouring pair).
template <int BITS, bool NORM, bool I8 = false>
__global__ void __launch_bounds__(256) quantize_blocks_prefill_kernel(Layout L, Store S, const __half* __restrict__ X,
                                                                      int N, int n_q, unsigned char* __restrict__ cache,
                                                                      const float* __restrict__ inv_norm) {
  constexpr int PB = BITS == 3 ? 2 : BITS;
  constexpr int NW = PB == 4 ? 8 : 4;
  extern __shared__ __align__(16) unsigned char smem_q[];
  const int G = L.G, CH = G >> 5;
  float4* red = reinterpret_cast<float4*>(smem_q);                               // [CH][128]: mn, mx, ea, es
  const int u = blockIdx.y, tid = threadIdx.x, cp = tid & 63, k = tid >> 6, c0 = 2 * cp;
  float inv[2] = {1.0f, 1.0f};
  if constexpr (NORM) { inv[0] = inv_norm[(size_t)u * kD + c0]; inv[1] = inv_norm[(size_t)u * kD + c0 + 1]; }
  const Rec rec = unit_rec(L, cache, u);
  const __half* Xu = X + ((size_t)u * N + L.w_sink) * kD + c0;
  // positions (see block_pos_plane): fragment coordinates of the pair (row halves rh = 0, 1)
  const int m = 4 * (c0 >> 6) + ((c0 >> 1) & 3), gid = (c0 >> 3) & 7;
  const int base_lo = (m >> 2) * 128 + 16 * gid + (m & 3);                        // + 4 * tid4 (+ 256 * k-step for 4 bits)
  const int base_hi = chunk_hi_plane_word() + 16 * gid + (m >> 1);
  for (int j = blockIdx.x; j < n_q / G; j += gridDim.x) {
    uint32_t raw[kSeg];
    const __half* src = Xu + ((size_t)j * G + kSeg * k) * kD;
#pragma unroll
    for (int t = 0; t < kSeg; ++t) raw[t] = __ldg(reinterpret_cast<const uint32_t*>(src + (size_t)t * kD));
    uint32_t wlo[NW], whi[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int i = 0; i < NW; ++i) wlo[i] = 0u;
    [[maybe_unused]] uint32_t w16[2][8];      // byte order: words [rh][2 * j + half] of this channel pair, at its bit position
    [[maybe_unused]] uint32_t h16[I8 && BITS == 3 ? 2 : 1][8];      // ... of the 1-bit plane of 3-bit codes
    uint32_t meta2[2];
    if (CH > 1 || (I8 && BITS == 3)) __syncthreads();       // the previous group's exchange words are no longer read
#pragma unroll
    for (int rh = 0; rh < 2; ++rh) {
      float x[kSeg];
#pragma unroll
      for (int t = 0; t < kSeg; ++t) {
        const __half2 h2 = *reinterpret_cast<const __half2*>(&raw[t]);
        x[t] = rh ? __high2float(h2) : __low2float(h2);
        if constexpr (NORM) x[t] = __fmul_rn(x[t], inv[rh]);
      }
      float mn, mx;
      seg_minmax(x, mn, mx);
      if (CH > 1) {
        red[k * 128 + c0 + rh] = make_float4(mn, mx, 0.f, 0.f);
        __syncthreads();
        for (int kk = 0; kk < CH; ++kk) {
          const float4 o = red[kk * 128 + c0 + rh];
          mn = fminf(mn, o.x); mx = fmaxf(mx, o.y);
        }
      }
      const GroupParams p = group_params(mn, mx, fmaxf(fabsf(mn), fabsf(mx)), BITS, L.sym_variant);
      const SegCoder sc(p);
      const bool no_clip = sc.no_clip(mn, mx);
      bool asym = S.mode == 1;
      if (S.mode == 2) {
        float ea, es;
        if (no_clip) seg_errors<false>(sc, x, ea, es);
        else seg_errors<true>(sc, x, ea, es);
        if (CH > 1) {
          red[k * 128 + c0 + rh].z = ea;
          red[k * 128 + c0 + rh].w = es;
          __syncthreads();
          ea = 0.f; es = 0.f;
          for (int kk = 0; kk < CH; ++kk) {
            const float4 o = red[kk * 128 + c0 + rh];
            ea += o.z; es += o.w;
          }
        }
        asym = ea < es;
      }
      const ChosenCoder cc(sc, asym);
      if constexpr (I8 && BITS == 3) {
        if (no_clip) pack_block_segment_i8_3<false>(cc, x, cp & 1, w16[rh], h16[rh]);
        else pack_block_segment_i8_3<true>(cc, x, cp & 1, w16[rh], h16[rh]);
        const int sh_hi = hi_bit_i8(cp & 3, c0 >> 6);
#pragma unroll
        for (int i = 0; i < 8; ++i) { w16[rh][i] <<= 2 * (cp & 3); h16[rh][i] <<= sh_hi; }
      } else if constexpr (I8) {
        if (no_clip) pack_block_segment_i8<BITS, false>(cc, x, w16[rh]);
        else pack_block_segment_i8<BITS, true>(cc, x, w16[rh]);
#pragma unroll
        for (int i = 0; i < 8; ++i) w16[rh][i] <<= BITS * (BITS == 2 ? cp & 3 : cp & 1);      // this pair's bit position
      } else {
        uint32_t lw[NW], hw[4];
        if (no_clip) pack_block_segment<BITS, false>(cc, x, lw, hw);
        else pack_block_segment<BITS, true>(cc, x, lw, hw);
#pragma unroll
        for (int i = 0; i < NW; ++i) wlo[i] |= lw[i] << (8 * rh);
        if constexpr (BITS == 3) {
#pragma unroll
          for (int i = 0; i < 4; ++i) whi[i] |= hw[i] << (4 * (2 * (m & 1) + rh));
        }
      }
      meta2[rh] = group_meta(p, asym);
    }
    uint32_t* chunk = reinterpret_cast<uint32_t*>(block_code_ptr(rec, S, j * CH + k));
    if constexpr (I8 && BITS == 4) {
      // The two channel pairs cp = 2q, 2q + 1 (adjacent lanes) fill the two nibbles of the same 16 words: after one
      // exchange lane `pos` holds the complete words of j = 2 pos, 2 pos + 1 (16 contiguous bytes each).
      const int pos = cp & 1, W = m >> 1;
#pragma unroll
      for (int jj = 0; jj < 2; ++jj) {
        uint32_t f4[4];
#pragma unroll
        for (int rh = 0; rh < 2; ++rh)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const uint32_t keep = pos ? w16[rh][2 * (2 + jj) + half] : w16[rh][2 * jj + half];
            const uint32_t give = pos ? w16[rh][2 * jj + half] : w16[rh][2 * (2 + jj) + half];
            f4[2 * half + rh] = keep | __shfl_xor_sync(0xffffffffu, give, 1);
          }
        *reinterpret_cast<uint4*>(chunk + W * 128 + (4 * gid + 2 * pos + jj) * 4) = make_uint4(f4[0], f4[1], f4[2], f4[3]);
      }
    } else if constexpr (I8) {
      // The four channel pairs cp = 4q .. 4q+3 (adjacent lanes) fill the four bit positions of the same 16 words.
      // Reduce-scatter by OR: after two exchange steps lane `pos` holds the complete words of j = pos (two halves,
      // two row halves), which are 16 contiguous bytes of the chunk.
      const int pos = cp & 3;
      auto reduce_scatter = [&](const uint32_t (&w)[2][8]) {
        uint32_t h8[2][4];                    // step 1: keep j of my parity (j = 2 * i + (pos & 1)), index [rh][2 * i + half]
#pragma unroll
        for (int rh = 0; rh < 2; ++rh)
#pragma unroll
          for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              const uint32_t keep = (pos & 1) ? w[rh][2 * (2 * i + 1) + half] : w[rh][2 * (2 * i) + half];
              const uint32_t give = (pos & 1) ? w[rh][2 * (2 * i) + half] : w[rh][2 * (2 * i + 1) + half];
              h8[rh][2 * i + half] = keep | __shfl_xor_sync(0xffffffffu, give, 1);
            }
        uint32_t f4[4];                       // step 2: keep i = pos >> 1; index 2 * half + rh (the word order in the chunk)
#pragma unroll
        for (int rh = 0; rh < 2; ++rh)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const uint32_t keep = (pos & 2) ? h8[rh][2 + half] : h8[rh][half];
            const uint32_t give = (pos & 2) ? h8[rh][half] : h8[rh][2 + half];
            f4[2 * half + rh] = keep | __shfl_xor_sync(0xffffffffu, give, 2);
          }
        return make_uint4(f4[0], f4[1], f4[2], f4[3]);
      };
      const int W = c0 >> 6;
      *reinterpret_cast<uint4*>(chunk + W * 128 + (4 * gid + pos) * 4) = reduce_scatter(w16);
      if constexpr (BITS == 3) {
        // 1-bit plane: the words of lane group gid hold the bits of both halves W of the channels, which two warps
        // of this chunk's 64 threads computed: the second hands its words to the first through shared memory
        uint4* hx = reinterpret_cast<uint4*>(smem_q + (size_t)CH * 128 * 16) + k * 32 + (cp & 31);
        const uint4 mine = reduce_scatter(h16);
        if (W == 1) *hx = mine;
        __syncthreads();
        if (W == 0) {
          const uint4 o = *hx;
          *reinterpret_cast<uint4*>(chunk + 256 + (4 * gid + pos) * 4) =
              make_uint4(mine.x | o.x, mine.y | o.y, mine.z | o.z, mine.w | o.w);
        }
      }
    } else {
#pragma unroll
      for (int i = 0; i < NW; ++i) chunk[base_lo + 4 * (i & 3) + 256 * (i >> 2)] = wlo[i];
    }
    if constexpr (BITS == 3 && !I8) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t full = whi[i] | __shfl_xor_sync(0xffffffffu, whi[i], 1);   // the pair with the other m & 1
        if ((cp & 1) == 0) chunk[base_hi + 4 * i] = full;
      }
    }
    if (k == 0) {
      store_meta(block_meta_ptr(rec, S, j), block_meta_index(c0), S.meta_bytes, meta2[0]);
      store_meta(block_meta_ptr(rec, S, j), block_meta_index(c0 + 1), S.meta_bytes, meta2[1]);
    }
  }
}

}  // namespace

static inline int grid_cap(int n, int cap) { return n < 1 ? 1 : (n > cap ? cap : n); }

template <int BITS>
static int launch_store_bits(const Layout& L, const Store& S, const __half* X, int N, int n_q, unsigned char* cache,
                             const float* inv_norm, cudaStream_t st) {
  if (S.kind == kRow) {
    // a warp takes batches of 8 tokens; several batches per warp amortise its set-up (32 reciprocal norms)
    const int n_batches = (n_q + 7) / 8;
    const int per_unit = grid_cap((n_batches + 4 * 8 - 1) / (4 * 8), grid_cap(148 * 16 / L.U, 1 << 16));
    dim3 grid(per_unit, L.U);
    if (S.perm == 1) {
      if (inv_norm) quantize_rows_prefill_kernel<BITS, true, true><<<grid, 128, 0, st>>>(L, S, X, N, n_q, cache, inv_norm);
      else quantize_rows_prefill_kernel<BITS, false, true><<<grid, 128, 0, st>>>(L, S, X, N, n_q, cache, nullptr);
      return cudaGetLastError() == cudaSuccess ? 1 : -1;
    }
    if (inv_norm) quantize_rows_prefill_kernel<BITS, true><<<grid, 128, 0, st>>>(L, S, X, N, n_q, cache, inv_norm);
    else quantize_rows_prefill_kernel<BITS, false><<<grid, 128, 0, st>>>(L, S, X, N, n_q, cache, nullptr);
  } else {
    const int CH = L.G / kChunk;
    // reduction words of groups spanning several chunks; 3-bit codes in byte order: exchange of the 1-bit plane's words
    const int smem = CH * 128 * 16 + (BITS == 3 && S.perm == 1 ? CH * 32 * 16 : 0);
    auto kern = inv_norm ? quantize_blocks_prefill_kernel<BITS, true> : quantize_blocks_prefill_kernel<BITS, false>;
    if (S.perm == 1)
      kern = inv_norm ? quantize_blocks_prefill_kernel<BITS, true, true> : quantize_blocks_prefill_kernel<BITS, false, true>;
    const int n_groups = n_q / L.G;
    dim3 grid(grid_cap(n_groups, grid_cap(148 * 16 / L.U, 1 << 16)), L.U);
    kern<<<grid, 64 * CH, smem, st>>>(L, S, X, N, n_q, cache, inv_norm);
  }
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

// Quantises rows / groups [0, n_q) of every unit of store S from the prefill input X ([U][N][128] fp16; the token
// of row i is w_sink + i).  inv_norm: reciprocal key norms [U][128], or null for unnormalised values.
int launch_quantize_store_prefill(const Layout& L, const Store& S, const __half* X, int N, int n_q, unsigned char* cache,
                                  const float* inv_norm, cudaStream_t st) {
  if (S.bits == 2) return launch_store_bits<2>(L, S, X, N, n_q, cache, inv_norm, st);
  if (S.bits == 3) return launch_store_bits<3>(L, S, X, N, n_q, cache, inv_norm, st);
  if (S.bits == 4) return launch_store_bits<4>(L, S, X, N, n_q, cache, inv_norm, st);
  return -1;
}

}  // namespace iq
