// Development instrumentation of the tensor-core kernels: per-phase cycle counters and per-CTA time stamps.
// The default build never includes this file: tc_device.cuh pulls it in only under -DTRI_INV_PHASE_CLOCKS
// and otherwise defines the three macros as no-ops.  With it, the kernels add the cycles between PHASE
// marks of thread block 0 into words 8.. of the device status array (12 counters per warp) and record each
// block's start / end time and SM; two extra exports read them back.
#pragma once
#include "common.cuh"

namespace tri_inv {
namespace {
__device__ unsigned long long g_cta_times[4096 * 4];
__device__ __forceinline__ unsigned long long dev_gtime() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
__device__ __forceinline__ unsigned dev_smid() { unsigned r; asm volatile("mov.u32 %0, %%smid;" : "=r"(r)); return r; }
}  // namespace
}  // namespace tri_inv

#define CTA_MARK(k) do { if (threadIdx.x == 0 && blockIdx.x < 4096) g_cta_times[blockIdx.x * 4 + (k)] = (k) == 3 ? dev_smid() : dev_gtime(); } while (0)
#define PHASE_BEGIN() long long ph_t = clock64()
#define PHASE(k)                                                                  \
  do {                                                                            \
    long long now = clock64();                                                    \
    if (blockIdx.x == 0 && (threadIdx.x & 31) == 0) atomicAdd(p.status + 8 + 12 * (threadIdx.x >> 5) + (k), (int)(now - ph_t)); \
    ph_t = now;                                                                   \
  } while (0)

// Chunk scan: the clock of one chunk's steps (the 21st chunk of thread block 0), per warp, as a snapshot in the
// same status words; `warp`, `lane` and the chunk index `c` are the kernel's own variables at the mark.
#define TL(k) do { if (blockIdx.x == 0 && c == 20 && lane == 0) p.status[8 + 12 * warp + (k)] = (int)clock64(); } while (0)

#ifdef TRI_INV_DEV_DEFINE_EXPORTS
// One translation unit (the one that defines TRI_INV_DEV_DEFINE_EXPORTS) carries the read-back calls.
extern "C" int tri_inv_debug_cta_times(unsigned long long* out, int n) {
  return cudaMemcpyFromSymbol(out, tri_inv::g_cta_times, sizeof(unsigned long long) * n) == cudaSuccess ? 0 : 3;
}
extern "C" int tri_inv_debug_counters(int* out) {
  cudaError_t err;
  int* word = tri_inv::status_word_for_current_device(&err);
  if (!word) return 3;
  if (cudaMemcpy(out, word, 128 * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return 3;
  return cudaMemset(word, 0, 128 * sizeof(int)) == cudaSuccess ? 0 : 3;
}
#endif
