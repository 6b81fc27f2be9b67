// Latency probe for the building blocks of the kernels' hand-offs on sm_100a: one CTA, clock64 stamps.
// It measures, in SM cycles (median of 200 repetitions each):
//   * tcgen05.mma chains (bf16, K = 16 per instruction) from the first issue to the moment the issuing thread
//     sees the mbarrier that tcgen05.commit arrives on, for several shapes and chain lengths;
//   * the same completion as seen by a thread of another warp that was already waiting;
//   * tcgen05.ld (16 lanes x 64 columns) + tcgen05.wait::ld;
//   * 16 shared-memory stores followed by fence.proxy.async;
//   * stmatrix.x4 x 4 followed by fence.proxy.async;
//   * mbarrier.arrive by 128 threads until a polling thread of a fifth warp sees the phase complete;
//   * a chain of eight instructions split between two issuing threads of different warps.
// Stand-alone (not part of the library):
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -I include \
//        paper_2605_21325_b200/csrc/probes/latency_probe.cu -o latency_probe && ./latency_probe
// Every wait is bounded; operands are zeros (timing only).
#include "../tc_device.cuh"

#include <algorithm>
#include <cstdio>
#include <vector>

namespace tri_inv {
namespace {

constexpr int kReps = 200;
constexpr int kKinds = 14;

__global__ void __launch_bounds__(192) probe(int* out, int* status) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sA = smem_u32(smem), sB = sA + 32768;            // 128 rows x 2 boxes and 256 rows x 2 boxes of zeros
  const uint32_t bar_mma = smem_u32(smem + 98304), bar_cnt = bar_mma + 8, bar_mma2 = bar_mma + 24;
  uint32_t* slot = reinterpret_cast<uint32_t*>(smem + 98304 + 16);
  volatile long long* stamp = reinterpret_cast<volatile long long*>(smem + 98304 + 40);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int e = tid; e < 98304 / 16; e += blockDim.x) reinterpret_cast<uint4*>(smem)[e] = make_uint4(0, 0, 0, 0);
  if (tid == 0) { mbar_init(bar_mma, 1); mbar_init(bar_mma2, 1); mbar_init(bar_cnt, 128); fence_mbar_init(); }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *slot;
  uint32_t ph_mma = 0, ph_cnt = 0;
  bool ok = true;

  // kinds 0..5: MMA chains seen by the issuer; shapes (M, N, instructions)
  const int shapes[6][3] = {{128, 128, 1}, {128, 128, 8}, {128, 64, 4}, {64, 64, 8}, {64, 32, 8}, {128, 192, 8}};
  for (int kind = 0; kind < 6 && ok; ++kind) {
    const uint32_t idesc = umma_idesc(shapes[kind][0], shapes[kind][1], 0);
    for (int r = 0; r < kReps && ok; ++r) {
      __syncthreads();
      if (tid == 128) {   // the fifth warp issues, as the kernels' control warp does
        const long long t0 = clock64();
        for (int ks = 0; ks < shapes[kind][2]; ++ks)
          umma_bf16(tmem, umma_desc(sA + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                    umma_desc(sB + (ks >> 2) * 32768 + (ks & 3) * 32, 16, 1024), idesc, ks > 0);
        umma_commit(bar_mma);
        const long long t1 = clock64();
        ok = mbar_wait_bounded(bar_mma, ph_mma);
        const long long t2 = clock64();
        out[(kind * kReps + r) * 2 + 0] = (int)(t1 - t0);   // issue
        out[(kind * kReps + r) * 2 + 1] = (int)(t2 - t0);   // issue + execution + completion seen
        *stamp = t0;
      }
      // kind 6: the same completion (8 x 128x128) seen by a waiting thread of warp 0
      if (kind == 1 && tid == 0) {
        ok = mbar_wait_bounded(bar_mma, ph_mma);
        const long long t2 = clock64();
        __threadfence_block();
        out[(6 * kReps + r) * 2 + 1] = (int)(t2 - *stamp);   // approximate: the stamp is written after the wait of the issuer
      }
      ph_mma ^= 1;
      tc_fence_after();
    }
  }
  // kinds 12, 13: two threads of different warps issue half of a chain each (4 + 4 instructions, separate
  // accumulators), 128x128 and 64x64: from the common start to the moment each has seen its own commit
  for (int kind = 12; kind < 14 && ok; ++kind) {
    const int M = kind == 12 ? 128 : 64, N = kind == 12 ? 128 : 64;
    const uint32_t idesc = umma_idesc(M, N, 0);
    uint32_t ph2 = 0;
    for (int r = 0; r < kReps && ok; ++r) {
      __syncthreads();
      if (tid == 128 || tid == 160) {
        const int part = tid == 160;
        const uint32_t bar = part ? bar_mma2 : bar_mma;
        const long long t0 = clock64();
        for (int ks = 4 * part; ks < 4 * part + 4; ++ks)
          umma_bf16(tmem + 128 * part, umma_desc(sA + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024),
                    umma_desc(sB + (ks >> 2) * 32768 + (ks & 3) * 32, 16, 1024), idesc, ks > 4 * part);
        umma_commit(bar);
        const long long t1 = clock64();
        ok = mbar_wait_bounded(bar, part ? ph2 : ph_mma);
        const long long t2 = clock64();
        if (part == 1) { out[(kind * kReps + r) * 2 + 0] = (int)(t1 - t0); out[(kind * kReps + r) * 2 + 1] = (int)(t2 - t0); }
      }
      ph_mma ^= 1;
      ph2 ^= 1;
      tc_fence_after();
    }
  }
  // kind 7: tcgen05.ld 16 lanes x 64 columns + wait (warps 0..3)
  for (int r = 0; r < kReps; ++r) {
    __syncthreads();
    if (warp < 4) {
      float f[8][4];
      const long long t0 = clock64();
      tmem_ld_16x64(f, tmem + ((uint32_t)(32 * warp) << 16));
      tmem_wait_ld();
      const long long t1 = clock64();
      if (tid == 0) out[(7 * kReps + r) * 2 + 1] = (int)(t1 - t0) + (f[0][0] != 0.f);
    }
  }
  // kind 8: 16 x st.shared.b32 + fence.proxy.async; kind 9: 4 x stmatrix.x4 + fence.proxy.async
  for (int r = 0; r < kReps; ++r) {
    __syncthreads();
    if (warp < 4) {
      long long t0 = clock64();
      for (int i = 0; i < 16; ++i) *reinterpret_cast<volatile uint32_t*>(smem + 65536 + (tid * 16 + i) * 4) = (uint32_t)i;
      long long t1 = clock64();
      fence_proxy_async();
      long long t2 = clock64();
      if (tid == 0) { out[(8 * kReps + r) * 2 + 0] = (int)(t1 - t0); out[(8 * kReps + r) * 2 + 1] = (int)(t2 - t1); }
      __syncwarp();
      t0 = clock64();
      for (int i = 0; i < 4; ++i)
        asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(sA + 65536 + warp * 4096 + i * 512 + lane * 16),
                     "r"(0u), "r"(0u), "r"(0u), "r"(0u) : "memory");
      t1 = clock64();
      fence_proxy_async();
      t2 = clock64();
      if (tid == 0) { out[(9 * kReps + r) * 2 + 0] = (int)(t1 - t0); out[(9 * kReps + r) * 2 + 1] = (int)(t2 - t1); }
    }
  }
  // kind 10: 128 arrivals -> seen by the polling thread of warp 4
  for (int r = 0; r < kReps && ok; ++r) {
    __syncthreads();
    if (warp < 4) {
      if (tid == 0) *stamp = clock64();
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_cnt) : "memory");
    } else if (tid == 128) {
      ok = mbar_wait_bounded(bar_cnt, ph_cnt);
      const long long t1 = clock64();
      out[(10 * kReps + r) * 2 + 1] = (int)(t1 - *stamp);
    }
    ph_cnt ^= 1;
  }
  // kind 11: __syncthreads of 160 threads
  for (int r = 0; r < kReps; ++r) {
    const long long t0 = clock64();
    __syncthreads();
    const long long t1 = clock64();
    if (tid == 0) out[(11 * kReps + r) * 2 + 1] = (int)(t1 - t0);
  }
  if (!ok) atomicMax(status, 1);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
}

int median(std::vector<int> v) { std::sort(v.begin(), v.end()); return v[v.size() / 2]; }

int run_probe() {
  int *out, *status;
  const size_t n = (size_t)kKinds * kReps * 2;
  if (cudaMalloc(&out, n * sizeof(int)) != cudaSuccess || cudaMalloc(&status, sizeof(int)) != cudaSuccess) return 1;
  cudaMemset(out, 0, n * sizeof(int));
  cudaMemset(status, 0, sizeof(int));
  const int smem_bytes = 98304 + 64;
  cudaFuncSetAttribute(probe, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  probe<<<1, 192, smem_bytes>>>(out, status);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { printf("launch: %s\n", cudaGetErrorString(e)); return 1; }
  std::vector<int> h(n);
  int st = 0;
  cudaMemcpy(h.data(), out, n * sizeof(int), cudaMemcpyDeviceToHost);
  cudaMemcpy(&st, status, sizeof(int), cudaMemcpyDeviceToHost);
  const char* names[kKinds] = {"mma 128x128x16 x1", "mma 128x128x16 x8", "mma 128x64x16 x4", "mma 64x64x16 x8", "mma 64x32x16 x8",
                               "mma 128x192x16 x8", "  (x8 128x128 seen from another warp)", "tcgen05.ld 16x64 + wait",
                               "16 st.shared | fence.proxy.async", "4 stmatrix.x4 | fence.proxy.async",
                               "128 mbarrier arrivals -> seen by a poller", "__syncthreads (192 threads)",
                               "mma 128x128x16 4+4 from two warps", "mma 64x64x16 4+4 from two warps"};
  printf("timeout flag %d\n%-44s %8s %8s\n", st, "step (cycles, median of 200)", "first", "total");
  for (int k = 0; k < kKinds; ++k) {
    std::vector<int> a(kReps), b(kReps);
    for (int r = 0; r < kReps; ++r) { a[r] = h[(k * kReps + r) * 2]; b[r] = h[(k * kReps + r) * 2 + 1]; }
    printf("%-44s %8d %8d\n", names[k], median(a), median(b));
  }
  return 0;
}

}  // namespace
}  // namespace tri_inv

int main() { return tri_inv::run_probe(); }
