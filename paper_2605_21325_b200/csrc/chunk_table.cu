// Chunk table of a packed batch, built on the device.
//
// The sequence offsets (host memory) travel as kernel parameters, a few hundred sequences per
// launch, so no host-to-device copy, staging buffer or synchronisation is involved: the table is
// ready in stream order before the kernel that reads it.
#include "common.cuh"

namespace tri_inv {
namespace {

constexpr int kSeqsPerLaunch = 960;

struct SeqBatch {
  int32_t cu[kSeqsPerLaunch + 1];  // offsets of the sequences of this launch
  int32_t n_seqs;
  int32_t first_chunk;             // index of this batch's first table entry
  int32_t C;
};

__global__ void __launch_bounds__(256) chunk_table_kernel(ChunkEntry* tab, const __grid_constant__ SeqBatch b) {
  for (int s = blockIdx.x * blockDim.x + threadIdx.x; s < b.n_seqs; s += gridDim.x * blockDim.x) {
    int idx = b.first_chunk;
    for (int q = 0; q < s; ++q) idx += (b.cu[q + 1] - b.cu[q] + b.C - 1) / b.C;
    const int beg = b.cu[s], end = b.cu[s + 1];
    for (int t = beg; t < end; t += b.C) tab[idx++] = ChunkEntry{t, (end - t) < b.C ? (end - t) : b.C};
  }
}

}  // namespace

cudaError_t launch_chunk_table(ChunkEntry* dev_tab, const tri_inv_desc* d, cudaStream_t stream) {
  int first_chunk = 0;
  for (int s0 = 0; s0 < d->n_seqs; s0 += kSeqsPerLaunch) {
    SeqBatch b;
    b.n_seqs = d->n_seqs - s0 < kSeqsPerLaunch ? d->n_seqs - s0 : kSeqsPerLaunch;
    b.first_chunk = first_chunk;
    b.C = d->C;
    for (int q = 0; q <= b.n_seqs; ++q) b.cu[q] = d->cu_seqlens[s0 + q];
    for (int q = 0; q < b.n_seqs; ++q) first_chunk += (b.cu[q + 1] - b.cu[q] + d->C - 1) / d->C;
    chunk_table_kernel<<<(b.n_seqs + 255) / 256, 256, 0, stream>>>(dev_tab, b);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace tri_inv
