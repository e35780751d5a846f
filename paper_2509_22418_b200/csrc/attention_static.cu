// Attention backward for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a region that is being
// stream-captured, under a framework whose allocator owns all device memory, or in a process
// that is handed fixed buffers and nothing else.  ppu_attention_bwd needs a per-row scratch
// vector (delta = rowsum(dU * U)); this variant keeps that vector in a fixed array that lives
// in the library image instead of asking the caller for it.
#include <mutex>
#include "../../include/ppu.h"
#include "common.cuh"

int ppu_fail(int code, const char* fmt, ...);

namespace {

// Every GPU that loads the library holds this array (4 MiB) until the process exits.
__device__ __align__(256) float g_static_delta[PPU_STATIC_SCRATCH_FLOATS];

constexpr int MAX_DEVICES = 64;
float* g_delta_ptr[MAX_DEVICES] = {};   // device address of g_static_delta, per device
std::mutex g_delta_lock;                // two threads may make the first call on a device at once

// In host code `g_static_delta` is only a handle; the address a kernel can use has to be asked
// for, once per device, with that device current.
int static_scratch(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return ppu_fail(PPU_ECUDA, "cudaGetDevice failed: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= MAX_DEVICES) return ppu_fail(PPU_ECUDA, "device index %d not supported", dev);
  std::lock_guard<std::mutex> lk(g_delta_lock);
  if (!g_delta_ptr[dev]) {
    float* p = nullptr;
    e = cudaGetSymbolAddress((void**)&p, g_static_delta);
    if (e != cudaSuccess || !p)
      return ppu_fail(PPU_ECUDA, "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
    g_delta_ptr[dev] = p;
  }
  *out = g_delta_ptr[dev];
  return PPU_OK;
}

}  // namespace

extern "C" int ppu_attention_bwd_static(const void* qkv, const void* U, const float* lse,
                                        const void* dU, void* dqkv, int batch, int seq, int n_head,
                                        int d_head, int backend, void* cuda_stream) {
  if (!qkv || !U || !lse || !dU || !dqkv) return ppu_fail(PPU_EINVAL, "null operand");
  if (batch < 1 || seq < 1 || n_head < 1) return ppu_fail(PPU_EINVAL, "non-positive size");
  const long long need = (long long)batch * n_head * seq;
  if (need > (long long)PPU_STATIC_SCRATCH_FLOATS)
    return ppu_fail(PPU_ESHAPE,
                    "batch*n_head*seq = %lld exceeds the built-in scratch of %lld rows; use "
                    "ppu_attention_bwd with caller scratch",
                    need, (long long)PPU_STATIC_SCRATCH_FLOATS);
  float* scratch = nullptr;
  int rc = static_scratch(&scratch);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // Every row the kernels read from the scratch is written first by the same call, so nothing
  // left over from an earlier call is ever used and no clearing is needed.
  if (backend < 0 || backend > 1) return ppu_fail(PPU_EINVAL, "unknown attention backend %d", backend);
  if (backend == 0) {
    if (!attn_tc_supported(seq, d_head))
      return ppu_fail(PPU_ESHAPE, "shape not covered by the tensor-core attention");
    rc = launch_attn_bwd_tc((const bf16*)qkv, (const bf16*)U, lse, (const bf16*)dU, (bf16*)dqkv, scratch,
                            batch, seq, n_head, d_head, nullptr, st);
  } else {
    rc = launch_attn_bwd_simt((const bf16*)qkv, (const bf16*)U, lse, (const bf16*)dU, (bf16*)dqkv,
                              scratch, batch, seq, n_head, d_head, st);
  }
  if (rc) return ppu_fail(PPU_ESHAPE, "attention backward launch failed (%d)", rc);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return ppu_fail(PPU_ECUDA, "launch failed: %s", cudaGetErrorString(e));
  return PPU_OK;
}
