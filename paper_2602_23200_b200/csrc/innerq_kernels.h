// Host-callable launchers of the library's kernels (internal interface between the .cu files).
// Each returns the number of kernels it launched, or -1 on a CUDA error.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <atomic>

#include "innerq_layout.h"

namespace iq {

// More than 48 KB of dynamic shared memory is an opt-in per kernel AND per device: `done` (one per kernel, a bit per
// device ordinal) remembers where it has been set, so a process that drives several GPUs sets it on each of them.
template <typename Kernel>
inline bool opt_in_dynamic_smem(Kernel kernel, int bytes, std::atomic<unsigned long long>& done) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  const unsigned long long bit = 1ull << dev;
  if (done.load(std::memory_order_acquire) & bit) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
  done.fetch_or(bit, std::memory_order_release);
  return true;
}

struct ExportPtrs {
  uint8_t *k_code, *v_code;
  uint16_t *k_scale, *k_zero, *v_scale, *v_zero;
  float* norm;
  uint16_t *k_sink, *v_sink, *k_recent, *v_recent;
};

int launch_prefill(const Layout& L, unsigned char* cache, unsigned char* ws, const __half* K, const __half* V, int N,
                   cudaStream_t st);
// Prefill quantiser of one store: rows / groups [0, n_q) of every unit from X ([U][N][128] fp16).
// inv_norm: reciprocal key norms [U][128], or null.
int launch_quantize_store_prefill(const Layout& L, const Store& S, const __half* X, int N, int n_q, unsigned char* cache,
                                  const float* inv_norm, cudaStream_t st);
int launch_append(const Layout& L, unsigned char* cache, const __half* k_new, const __half* v_new, int N_after,
                  cudaStream_t st, int late_wait = 0);
int launch_export(const Layout& L, const unsigned char* cache, int N, const ExportPtrs& e, cudaStream_t st);
// The inverse: fills the cache (packed records, windows, norms, counts) for N tokens from canonical arrays.
int launch_import(const Layout& L, unsigned char* cache, int N, const ExportPtrs& e, cudaStream_t st);

// Generic SIMT decode (any store kinds, bits, group sizes): split kernel + merge kernel.
int launch_decode_simt(const Layout& L, const unsigned char* cache, unsigned char* ws, int N, const __half* q,
                       __half* out, int n_splits, cudaStream_t st);

// Warp-MMA decode for the INNER layout.  Returns -2 if the configuration is not supported.
// pages_host: a paged cache's page list on the host (optional: saves the kernel its look-ups in device memory).
int launch_decode_mma(const Layout& L, const unsigned char* cache, unsigned char* ws, int N, const __half* q,
                      __half* out, int n_splits, cudaStream_t st, int n_q = 1, float* multi_partials = nullptr,
                      int N_safe = 0, const uint32_t* pages_host = nullptr, int n_pages_host = 0);
int launch_decode_mma_batched(const Layout& L, int n, const unsigned char* const* caches, unsigned char* const* wss,
                              const int* Ns, const int* Ns_safe, const __half* q, __half* out, int n_splits,
                              cudaStream_t st);
int launch_append_batched(const Layout& L, int n, unsigned char* const* caches, const int* Ns_after, const int* late_wait,
                          const __half* k_new, const __half* v_new, cudaStream_t st);
bool decode_mma_supported(const Layout& L);

// Warp-MMA decode over an unquantised fp16 cache (grouping = FP16).  Returns -2 for other layouts.
int launch_decode_fp16(const Layout& L, const unsigned char* cache, unsigned char* ws, int N, const __half* q,
                       __half* out, int n_splits, cudaStream_t st);
// Test support: a one-warp kernel whose bounded wait runs out and sets the workspace's error word.
int launch_wait_expiry_selftest(const Layout& L, unsigned char* ws, cudaStream_t st);
void decode_mma_set_chunks_per_iter(int n);   // tuning: 32-token chunks per loop iteration (1 or 2)
void decode_mma_set_ablation(int mask);       // timing experiments: bit 0 / 1 = no key-side / value-side work in the loop


}  // namespace iq
