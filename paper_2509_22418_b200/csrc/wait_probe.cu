// Self-test of the bounded-wait error path used by every tcgen05 kernel of this library: a
// one-CTA kernel waits on an mbarrier that nothing ever arrives at, with a small iteration
// limit; when the limit runs out it sets an error word and returns normally.  The CUDA context
// stays usable - nothing traps, faults or spins without bound.
#include "../../include/ppu.h"
#include "tc_common.cuh"

int ppu_fail(int code, const char* fmt, ...);

namespace {

__device__ int g_probe_flag;

__global__ void wait_probe_kernel(uint32_t limit) {
  __shared__ uint64_t bar;
  const uint32_t b = tc::smem_u32(&bar);
  if (threadIdx.x == 0) {
    tc::mbar_init(b, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    bool seen = false;
    for (uint32_t it = 0; it < limit && !seen; ++it) seen = tc::mbar_try(b, 0);
    if (!seen) atomicExch(&g_probe_flag, 1);     // the wait gave up: report, then leave normally
  }
}

}  // namespace

extern "C" int ppu_wait_probe(int limit, void* cuda_stream) {
  if (limit < 1 || limit > (1 << 16)) return ppu_fail(PPU_EINVAL, "limit must lie in [1, 65536]");
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int zero = 0, flag = 0;
  cudaError_t e = cudaMemcpyToSymbolAsync(g_probe_flag, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) {
    wait_probe_kernel<<<1, 32, 0, st>>>((uint32_t)limit);
    e = cudaMemcpyFromSymbolAsync(&flag, g_probe_flag, sizeof(int), 0, cudaMemcpyDeviceToHost, st);
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return ppu_fail(PPU_ECUDA, "wait probe failed: %s", cudaGetErrorString(e));
  if (flag) return ppu_fail(PPU_ETIMEOUT, "a bounded wait inside a kernel expired (probe: as intended)");
  return PPU_OK;
}
