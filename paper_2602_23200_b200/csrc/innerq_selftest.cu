// Test support: the give-up path of the decode kernels' bounded wait, exercised without a copy that fails.
#include "innerq_decode_mma.cuh"

namespace iq {

namespace {

// One warp waits, with the decode kernels' own wait routine and a short limit, on a barrier on which nothing ever
// arrives, and records the expiry in the error word the way a decode warp does.  The kernel returns normally.
__global__ void wait_expiry_kernel(unsigned int* error_word) {
  __shared__ uint64_t bar;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  const bool arrived = mbar_wait(b, 0u, 256u);
  if (!arrived && threadIdx.x == 0) atomicExch(error_word, 1u);
}

}  // namespace

int launch_wait_expiry_selftest(const Layout& L, unsigned char* ws, cudaStream_t st) {
  wait_expiry_kernel<<<1, 32, 0, st>>>(reinterpret_cast<unsigned int*>(ws + L.ws_ticket_off) + L.U);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace iq
