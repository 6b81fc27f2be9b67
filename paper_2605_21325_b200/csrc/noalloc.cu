// tri_inv_fused_packed_static: the packed-sequence fused call for callers that must not allocate.
//
// The ordinary packed path keeps its chunk table (first token and row count of every chunk) in
// device memory that it allocates and frees in stream order.  Some callers cannot do that:
// code running where cudaMalloc is forbidden or unsafe (inside a region that must not touch
// the allocator, under a memory budget fixed at start-up, or in a process whose allocator is
// owned by someone else).  This variant keeps the table in a fixed array that is part of the
// library image instead, so the call performs no device or pinned-host allocation at all.
#include <mutex>

#include "common.cuh"

namespace tri_inv {
namespace {

// The whole scratch of the packed path: one entry per chunk of tokens.  Every GPU that loads the
// library holds these 128 KiB until the process exits.  All calls share it.
__device__ __align__(256) ChunkEntry g_static_chunk_table[TRI_INV_STATIC_MAX_CHUNKS];

// In host code `g_static_chunk_table` names a host-side shadow of the symbol, not device memory:
// the device address is looked up once per device (with that device current) and cached.
ChunkEntry* static_table_for_current_device(cudaError_t* err) {
  static std::mutex mu;
  static ChunkEntry* cache[64] = {nullptr};
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= 64) { *err = cudaErrorInvalidDevice; return nullptr; }
  std::lock_guard<std::mutex> lock(mu);
  if (!cache[dev]) {
    void* ptr = nullptr;
    *err = cudaGetSymbolAddress(&ptr, g_static_chunk_table);
    if (*err != cudaSuccess) return nullptr;
    cache[dev] = static_cast<ChunkEntry*>(ptr);
  }
  return cache[dev];
}

}  // namespace
}  // namespace tri_inv

using namespace tri_inv;

extern "C" int tri_inv_fused_packed_static(const void* K, const void* V, const float* beta, const float* g,
                                           float* A, void* W, void* U,
                                           const tri_inv_desc* desc, int method, void* cuda_stream) {
  // Descriptor checks are those of every other entry point (this also walks cu_seqlens).
  int64_t n_matrices = 0;
  int rc = tri_inv_count_matrices(desc, &n_matrices);
  if (rc != TRI_INV_OK) return rc;
  if (!desc->cu_seqlens) return TRI_INV_ERR_INVALID_ARG;  // dense calls need no scratch: use tri_inv_fused
  if (desc->d_v < 8 || (desc->d_v & 7)) return TRI_INV_ERR_INVALID_ARG;
  if (!K || !V || !beta || !g || !W || !U) return TRI_INV_ERR_INVALID_ARG;
  const void* ptrs[] = {K, V, beta, g, A, W, U};
  for (const void* q : ptrs)
    if (reinterpret_cast<uintptr_t>(q) & 15u) return TRI_INV_ERR_INVALID_ARG;
  const int m = method & TRI_INV_METHOD_MASK;
  if (m != TRI_INV_BLOCK_RECURSIVE && m != TRI_INV_PRODUCT_SERIES) return TRI_INV_ERR_UNSUPPORTED;
  if (method & ~(TRI_INV_METHOD_MASK | TRI_INV_LEAF_SERIES | TRI_INV_FORCE_SIMT)) return TRI_INV_ERR_UNSUPPORTED;
  if ((method & TRI_INV_LEAF_SERIES) && m != TRI_INV_BLOCK_RECURSIVE) return TRI_INV_ERR_UNSUPPORTED;

  if (n_matrices > 0x7fffffffLL) return TRI_INV_ERR_INVALID_ARG;  // the kernels index work items in 32 bits
  const int64_t n_chunks = n_matrices / desc->H;
  if (n_chunks > TRI_INV_STATIC_MAX_CHUNKS) return TRI_INV_ERR_TOO_LARGE;
  if (n_chunks == 0) return TRI_INV_OK;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t err;
  ChunkEntry* dev_tab = static_table_for_current_device(&err);
  if (!dev_tab) return TRI_INV_ERR_CUDA;

  KParams p{};
  p.K = K; p.V = V; p.beta = beta; p.g = g; p.A = A; p.W = W; p.U = U;
  p.method = method;
  p.ops = kDoWY | (A ? kStoreA : 0) | kFixedStride;  // no counter pair: handing one out may create an event on first use
  p.H = desc->H; p.d_k = desc->d_k; p.d_v = desc->d_v; p.T = desc->T;
  p.kv_dtype = desc->kv_dtype;
  p.n_chunks = static_cast<int32_t>(n_chunks);
  p.chunks_per_seq = 0;
  p.chunk_tab = dev_tab;
  p.wait_limit_ns = 2000000000ull;
  p.n_tokens = desc->T;   // packed mode: T is the total
  p.status = status_word_for_current_device(&err);
  if (!p.status) return TRI_INV_ERR_CUDA;

  // Only the first n_chunks entries are read by the kernel, and all of them are rewritten here (by a small
  // kernel on the same stream), so nothing left by an earlier call needs clearing.
  if (launch_chunk_table(dev_tab, desc, stream) != cudaSuccess) return TRI_INV_ERR_CUDA;

  bool handled = false;
  err = cudaSuccess;
  if (!(method & TRI_INV_FORCE_SIMT)) err = launch_tc(p, desc->C, stream, &handled);
  if (err == cudaSuccess && !handled) err = launch_simt(p, desc->C, stream);
  if (err == cudaSuccess) count_launch();
  return err == cudaSuccess ? TRI_INV_OK : TRI_INV_ERR_CUDA;
}
