// Device helpers shared by the kernels of this library: fp16 bit casts, packed-code access,
// the group quantiser.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "innerq_layout.h"

namespace iq {

__device__ __forceinline__ float h2f_bits(uint16_t b) { return __half2float(__ushort_as_half(b)); }
__device__ __forceinline__ uint16_t f2h_bits(float f) { return __half_as_ushort(__float2half_rn(f)); }

// ---- packed-code accessors (generic, slow; the fast kernels extract fragments directly) ----
__device__ __forceinline__ uint32_t row_code(const uint32_t* __restrict__ row, int c, int bits, int perm = 0) {
  if (perm == 1 && bits == 3) {
    const BitPos3 p = row_pos_i8_3(c);
    return code3_join((row[p.lo.word] >> p.lo.bit) & 3u, (row[p.hi.word] >> p.hi.bit) & 1u, p.odd);
  }
  if (perm == 1) {
    BitPos p = row_pos_i8(c, bits);
    return (row[p.word] >> p.bit) & ((1u << bits) - 1u);
  }
  if (bits == 3) {
    BitPos lo = row_pos_plane(c, 2), hi = row_pos_plane(c, 1);
    return ((row[lo.word] >> lo.bit) & 3u) | (((row[row_hi_plane_word() + hi.word] >> hi.bit) & 1u) << 2);
  }
  BitPos p = row_pos_plane(c, bits);
  return (row[p.word] >> p.bit) & ((1u << bits) - 1u);
}

__device__ __forceinline__ uint32_t chunk_code(const uint32_t* __restrict__ chunk, int tau, int c, int bits, int perm = 0) {
  if (perm == 1 && bits == 3) {
    const BitPos3 p = block_pos_i8_3(tau, c);
    return code3_join((chunk[p.lo.word] >> p.lo.bit) & 3u, (chunk[p.hi.word] >> p.hi.bit) & 1u, p.odd);
  }
  if (perm == 1) {
    BitPos p = block_pos_i8(tau, c, bits);
    return (chunk[p.word] >> p.bit) & ((1u << bits) - 1u);
  }
  if (bits == 3) {
    BitPos lo = block_pos_plane(tau, c, 2), hi = block_pos_plane(tau, c, 1);
    return ((chunk[lo.word] >> lo.bit) & 3u) | (((chunk[chunk_hi_plane_word() + hi.word] >> hi.bit) & 1u) << 2);
  }
  BitPos p = block_pos_plane(tau, c, bits);
  return (chunk[p.word] >> p.bit) & ((1u << bits) - 1u);
}

// OR a code into a zero-initialised packed row / chunk held in shared memory.
__device__ __forceinline__ void row_put(uint32_t* row, int c, int bits, uint32_t code, int perm = 0) {
  if (perm == 1 && bits == 3) {
    const BitPos3 p = row_pos_i8_3(c);
    atomicOr(&row[p.lo.word], code3_lo(code, p.odd) << p.lo.bit);
    atomicOr(&row[p.hi.word], code3_hi(code, p.odd) << p.hi.bit);
  } else if (perm == 1) {
    BitPos p = row_pos_i8(c, bits);
    atomicOr(&row[p.word], code << p.bit);
  } else if (bits == 3) {
    BitPos lo = row_pos_plane(c, 2), hi = row_pos_plane(c, 1);
    atomicOr(&row[lo.word], (code & 3u) << lo.bit);
    atomicOr(&row[row_hi_plane_word() + hi.word], (code >> 2) << hi.bit);
  } else {
    BitPos p = row_pos_plane(c, bits);
    atomicOr(&row[p.word], code << p.bit);
  }
}
__device__ __forceinline__ void chunk_put(uint32_t* chunk, int tau, int c, int bits, uint32_t code, int perm = 0) {
  if (perm == 1 && bits == 3) {
    const BitPos3 p = block_pos_i8_3(tau, c);
    atomicOr(&chunk[p.lo.word], code3_lo(code, p.odd) << p.lo.bit);
    atomicOr(&chunk[p.hi.word], code3_hi(code, p.odd) << p.hi.bit);
  } else if (perm == 1) {
    BitPos p = block_pos_i8(tau, c, bits);
    atomicOr(&chunk[p.word], code << p.bit);
  } else if (bits == 3) {
    BitPos lo = block_pos_plane(tau, c, 2), hi = block_pos_plane(tau, c, 1);
    atomicOr(&chunk[lo.word], (code & 3u) << lo.bit);
    atomicOr(&chunk[chunk_hi_plane_word() + hi.word], (code >> 2) << hi.bit);
  } else {
    BitPos p = block_pos_plane(tau, c, bits);
    atomicOr(&chunk[p.word], code << p.bit);
  }
}

// Decoder parameters of one group from its metadata word: x^ = s * u + z
// (z = Z when the mask bit is set, else -s * 2^(b-1): symmetric codes are offset-binary).
__device__ __forceinline__ void decode_meta(uint32_t meta, int bits, float& s, float& z) {
  uint16_t sb = (uint16_t)(meta & 0xFFFFu), zb = (uint16_t)(meta >> 16);
  s = h2f_bits(sb & 0x7FFFu);
  z = (sb & 0x8000u) ? h2f_bits(zb) : -s * (float)(1 << (bits - 1));
}

// Metadata entry i of a store (32-bit word, or a bare 16-bit scale in symmetric mode).
__device__ __forceinline__ uint32_t load_meta(const void* __restrict__ meta, size_t i, int meta_bytes) {
  return meta_bytes == 4 ? reinterpret_cast<const uint32_t*>(meta)[i]
                         : (uint32_t) reinterpret_cast<const uint16_t*>(meta)[i];
}
__device__ __forceinline__ void store_meta(void* __restrict__ meta, size_t i, int meta_bytes, uint32_t m) {
  if (meta_bytes == 4) reinterpret_cast<uint32_t*>(meta)[i] = m;
  else reinterpret_cast<uint16_t*>(meta)[i] = (uint16_t)m;
}

// ---- group quantiser ------------------------------------------------------------------
// Parameters of both candidates of one group, from its min / max / max-abs.  Every step is a
// single correctly rounded IEEE operation (no contraction, no approximate division), so the
// stored bits do not depend on the compiler or on how the statistics were reduced.
struct GroupParams {
  float s_a, z_a, inv_a;   // asymmetric: stored-precision scale, zero-point, 1/scale (0 if scale == 0)
  float s_s, inv_s;        // symmetric
  uint16_t sa_bits, z_bits, ss_bits;
  float L, q_lo, q_hi, half;
};

__device__ __forceinline__ GroupParams group_params(float mn, float mx, float am, int bits, int sym_variant) {
  GroupParams p;
  const int Li = (1 << bits) - 1, halfi = 1 << (bits - 1);
  p.L = (float)Li;
  p.half = (float)halfi;
  // asymmetric: Z = min, S = (max - min) / (2^b - 1), both rounded to fp16
  p.sa_bits = f2h_bits(__fdiv_rn(__fsub_rn(mx, mn), p.L));
  p.z_bits = f2h_bits(mn);
  p.s_a = h2f_bits(p.sa_bits);
  p.z_a = h2f_bits(p.z_bits);
  p.inv_a = p.s_a == 0.f ? 0.f : __fdiv_rn(1.0f, p.s_a);
  // symmetric: S = max|x| / den
  int den;
  if (sym_variant == 0) { den = halfi - 1; p.q_lo = -(float)den; p.q_hi = (float)den; }
  else { den = Li; p.q_lo = -(float)halfi; p.q_hi = (float)(halfi - 1); }
  p.ss_bits = f2h_bits(__fdiv_rn(am, (float)den));
  p.s_s = h2f_bits(p.ss_bits);
  p.inv_s = p.s_s == 0.f ? 0.f : __fdiv_rn(1.0f, p.s_s);
  return p;
}

__device__ __forceinline__ float asym_code(const GroupParams& p, float x) {
  float u = rintf(__fmul_rn(__fsub_rn(x, p.z_a), p.inv_a));
  u = fminf(fmaxf(u, 0.f), p.L);
  return p.s_a == 0.f ? 0.f : u;
}
__device__ __forceinline__ float sym_code(const GroupParams& p, float x) {   // signed
  float q = rintf(__fmul_rn(x, p.inv_s));
  q = fminf(fmaxf(q, p.q_lo), p.q_hi);
  return p.s_s == 0.f ? 0.f : q;
}
__device__ __forceinline__ float asym_err(const GroupParams& p, float x, float u) {
  return fabsf(__fsub_rn(x, __fmaf_rn(p.s_a, u, p.z_a)));
}
__device__ __forceinline__ float sym_err(const GroupParams& p, float x, float q) {
  return fabsf(__fsub_rn(x, __fmul_rn(p.s_s, q)));
}
// mask decision: mode 0 SYM, 1 ASYM, 2 HYBRID (lower L1 reconstruction error, tie -> symmetric)
__device__ __forceinline__ bool choose_asym(int mode, float e_a, float e_s) {
  return mode == 1 || (mode == 2 && e_a < e_s);
}
__device__ __forceinline__ uint32_t group_meta(const GroupParams& p, bool asym) {
  return asym ? ((uint32_t)(p.sa_bits | 0x8000u) | ((uint32_t)p.z_bits << 16)) : (uint32_t)p.ss_bits;
}

// Where a token's fp16 row lives: a contiguous [n][D] array (prefill input) or a ring buffer.
struct TokSrc {
  const __half* base;
  int ring_cap;     // 0: contiguous, indexed by absolute token; else slot = (t - w_sink) % ring_cap
  int w_sink;
  __device__ __forceinline__ const __half* row(int t) const {
    return ring_cap ? base + (size_t)((t - w_sink) % ring_cap) * kD : base + (size_t)t * kD;
  }
};

}  // namespace iq
