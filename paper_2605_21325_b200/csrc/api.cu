// extern "C" boundary: argument validation, chunk table for packed sequences, dispatch.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "common.cuh"

namespace tri_inv {
namespace {

__device__ int g_device_status[128] = {0};  // word 0: raised by kernels that give up on a bounded wait

std::atomic<long long> g_launches{0};

}  // namespace

int* status_word_for_current_device(cudaError_t* err) {
  // One address per device; looked up once per device under a lock.
  static std::mutex mu;
  static int* cache[64] = {nullptr};
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= 64) { *err = cudaErrorInvalidDevice; return nullptr; }
  std::lock_guard<std::mutex> lock(mu);
  if (!cache[dev]) {
    void* ptr = nullptr;
    *err = cudaGetSymbolAddress(&ptr, g_device_status);
    if (*err != cudaSuccess) return nullptr;
    cache[dev] = (int*)ptr;
  }
  return cache[dev];
}

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

namespace {

// Stream-ordered pool for the packed path's chunk tables.  It keeps what it has allocated (release
// threshold at the maximum), so steady-state calls reuse the same few kilobytes instead of going back
// to the driver; being private to the library it leaves the process's default pool untouched.
cudaMemPool_t table_pool_for_current_device() {
  static std::mutex mu;
  static cudaMemPool_t pools[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!pools[dev]) {
    cudaMemPoolProps props = {};
    props.allocType = cudaMemAllocationTypePinned;
    props.handleTypes = cudaMemHandleTypeNone;
    props.location.type = cudaMemLocationTypeDevice;
    props.location.id = dev;
    cudaMemPool_t pool = nullptr;
    if (cudaMemPoolCreate(&pool, &props) != cudaSuccess) return nullptr;
    unsigned long long keep = ~0ull;
    cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
    pools[dev] = pool;
  }
  return pools[dev];
}

// TRI_INV_LOG=1 in the environment: one line per kernel launch of the build / WY / fused calls on stderr (host side only).
bool log_enabled() {
  static const bool on = [] { const char* v = getenv("TRI_INV_LOG"); return v && *v && *v != '0'; }();
  return on;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_desc(const tri_inv_desc* d, bool need_dv) {
  if (!d) return TRI_INV_ERR_INVALID_ARG;
  if (d->B < 1 || d->T < 0 || d->H < 1) return TRI_INV_ERR_INVALID_ARG;
  if (d->d_k < 8 || (d->d_k & 7)) return TRI_INV_ERR_INVALID_ARG;
  if (need_dv && (d->d_v < 8 || (d->d_v & 7))) return TRI_INV_ERR_INVALID_ARG;
  if (d->C != 16 && d->C != 32 && d->C != 64 && d->C != 128) return TRI_INV_ERR_INVALID_ARG;
  if (d->kv_dtype != TRI_INV_F32 && d->kv_dtype != TRI_INV_BF16) return TRI_INV_ERR_INVALID_ARG;
  if ((long long)d->B * d->T > 0x7fffffffLL) return TRI_INV_ERR_INVALID_ARG;
  if (d->cu_seqlens) {
    if (d->B != 1 || d->n_seqs < 0) return TRI_INV_ERR_INVALID_ARG;
    if (d->cu_seqlens[0] != 0 || d->cu_seqlens[d->n_seqs] != d->T) return TRI_INV_ERR_INVALID_ARG;
    for (int s = 0; s < d->n_seqs; ++s)
      if (d->cu_seqlens[s + 1] < d->cu_seqlens[s]) return TRI_INV_ERR_INVALID_ARG;
  } else if (d->n_seqs != 0) {
    return TRI_INV_ERR_INVALID_ARG;
  }
  return TRI_INV_OK;
}

int check_method(int method, bool w_decay_ok = false, bool shift_ok = true) {
  int m = method & TRI_INV_METHOD_MASK;
  if (method & TRI_INV_GATE_SHIFTED) {
    if (!shift_ok) return TRI_INV_ERR_UNSUPPORTED;
    method &= ~TRI_INV_GATE_SHIFTED;
  }
  if (method & TRI_INV_W_DECAY) {
    if (!w_decay_ok) return TRI_INV_ERR_UNSUPPORTED;
    method &= ~TRI_INV_W_DECAY;
  }
  if (m != TRI_INV_BLOCK_RECURSIVE && m != TRI_INV_PRODUCT_SERIES && m != TRI_INV_NEWTON_SCHULZ) return TRI_INV_ERR_UNSUPPORTED;
  if (method & ~(TRI_INV_METHOD_MASK | TRI_INV_LEAF_SERIES | TRI_INV_REFINE | TRI_INV_NS_ITERS(15) | TRI_INV_FORCE_SIMT | TRI_INV_OPERANDS_F16)) return TRI_INV_ERR_UNSUPPORTED;
  if ((method & TRI_INV_OPERANDS_F16) && (m != TRI_INV_PRODUCT_SERIES || (method & TRI_INV_FORCE_SIMT))) return TRI_INV_ERR_UNSUPPORTED;
  if ((method & TRI_INV_LEAF_SERIES) && m != TRI_INV_BLOCK_RECURSIVE) return TRI_INV_ERR_UNSUPPORTED;
  if ((method & TRI_INV_REFINE) && m == TRI_INV_PRODUCT_SERIES) return TRI_INV_ERR_UNSUPPORTED;
  if ((method & TRI_INV_NS_ITERS(15)) && m != TRI_INV_NEWTON_SCHULZ) return TRI_INV_ERR_UNSUPPORTED;
  return TRI_INV_OK;
}

// Fills the parameter block, builds the ragged chunk table when needed, picks a kernel.
int run(KParams p, const tri_inv_desc* d, void* stream_v) {
  cudaStream_t stream = (cudaStream_t)stream_v;
  p.H = d->H; p.d_k = d->d_k; p.d_v = d->d_v; p.T = d->T;
  p.kv_dtype = d->kv_dtype;
  p.chunk_tab = nullptr;
  if (!p.wait_limit_ns) p.wait_limit_ns = 2000000000ull;
  p.n_tokens = d->cu_seqlens ? (long long)d->T : (long long)d->T * d->B;
  if (p.ops & kTestShrink) p.n_tokens -= d->C;
  cudaError_t err;
  p.status = status_word_for_current_device(&err);
  if (!p.status) return TRI_INV_ERR_CUDA;

  ChunkEntry* dev_tab = nullptr;
  if (d->cu_seqlens) {
    long long n = 0;
    for (int s = 0; s < d->n_seqs; ++s) n += ((long long)d->cu_seqlens[s + 1] - d->cu_seqlens[s] + d->C - 1) / d->C;
    if (n > 0x7fffffffLL) return TRI_INV_ERR_INVALID_ARG;
    p.n_chunks = (int)n;
    p.chunks_per_seq = 0;
    if (p.n_chunks == 0) return TRI_INV_OK;
    // The table is scratch owned by this call: allocated, filled (by a small kernel) and freed in stream order.
    cudaMemPool_t pool = table_pool_for_current_device();
    if (!pool || cudaMallocFromPoolAsync((void**)&dev_tab, (size_t)n * sizeof(ChunkEntry), pool, stream) != cudaSuccess) return TRI_INV_ERR_CUDA;
    if (launch_chunk_table(dev_tab, d, stream) != cudaSuccess) {
      cudaFreeAsync(dev_tab, stream);
      return TRI_INV_ERR_CUDA;
    }
    p.chunk_tab = dev_tab;
  } else {
    p.chunks_per_seq = (d->T + d->C - 1) / d->C;
    long long n = (long long)p.chunks_per_seq * d->B;
    if (n > 0x7fffffffLL) return TRI_INV_ERR_INVALID_ARG;
    p.n_chunks = (int)n;
    if (p.n_chunks == 0) return TRI_INV_OK;
  }

  if ((long long)p.n_chunks * d->H > 0x7fffffffLL) return TRI_INV_ERR_INVALID_ARG;  // kernels index work items in 32 bits
  if (log_enabled())
    fprintf(stderr, "[tri_inv] launch: B=%d T=%d H=%d d_k=%d d_v=%d C=%d dtype=%s %s, %d chunks x %d heads, method=0x%x ops=0x%x stream=%p\n",
            d->B, d->T, d->H, d->d_k, d->d_v, d->C, d->kv_dtype == TRI_INV_BF16 ? "bf16" : "f32", d->cu_seqlens ? "packed" : "dense",
            p.n_chunks, d->H, p.method, p.ops, stream_v);
  bool handled = false;
  err = cudaSuccess;
  // Newton-Schulz exists on the fp32 CUDA-core kernel only; so does refinement with the per-channel decay
  const bool simt_only = (p.method & TRI_INV_FORCE_SIMT) || (p.method & TRI_INV_METHOD_MASK) == TRI_INV_NEWTON_SCHULZ ||
                         ((p.ops & kKda) && (p.method & TRI_INV_REFINE));
  if (!simt_only) err = (p.ops & kKda) ? launch_kda_tc(p, d->C, stream, &handled) : launch_tc(p, d->C, stream, &handled);
  if (err == cudaSuccess && !handled && (p.method & TRI_INV_OPERANDS_F16)) {   // only the tensor-core kernel has fp16 operands
    if (dev_tab) cudaFreeAsync(dev_tab, stream);
    return TRI_INV_ERR_UNSUPPORTED;
  }
  if (err == cudaSuccess && !handled) err = launch_simt(p, d->C, stream);
  if (err == cudaSuccess) g_launches.fetch_add(1, std::memory_order_relaxed);
  if (dev_tab) cudaFreeAsync(dev_tab, stream);
  if (log_enabled()) fprintf(stderr, "[tri_inv]   -> %s kernel, %s\n", handled ? "tensor-core" : "CUDA-core", cudaGetErrorString(err));
  return err == cudaSuccess ? TRI_INV_OK : TRI_INV_ERR_CUDA;
}

}  // namespace
}  // namespace tri_inv

using namespace tri_inv;

extern "C" {

int tri_inv_build(const void* K, const float* beta, const float* g, float* A,
                  const tri_inv_desc* desc, int method, void* cuda_stream) {
  int rc = check_desc(desc, false);
  if (rc) return rc;
  if (!K || !beta || !g || !A) return TRI_INV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(beta) || !aligned16(g) || !aligned16(A)) return TRI_INV_ERR_INVALID_ARG;
  if ((rc = check_method(method))) return rc;
  KParams p{};
  p.K = K; p.beta = beta; p.g = g; p.A = A;
  p.method = method;
  p.ops = kStoreA;
  return run(p, desc, cuda_stream);
}

int tri_inv_wy(const float* A, const void* K, const void* V, const float* beta,
               void* W, void* U, const tri_inv_desc* desc, void* cuda_stream) {
  bool with_v = V || U;
  int rc = check_desc(desc, with_v);
  if (rc) return rc;
  if (!A || !K || !beta || !W) return TRI_INV_ERR_INVALID_ARG;
  if ((V == nullptr) != (U == nullptr)) return TRI_INV_ERR_INVALID_ARG;
  if (!aligned16(A) || !aligned16(K) || !aligned16(V) || !aligned16(beta) || !aligned16(W) || !aligned16(U))
    return TRI_INV_ERR_INVALID_ARG;
  KParams p{};
  p.A_in = A; p.K = K; p.V = V; p.beta = beta; p.W = W; p.U = U;
  p.method = TRI_INV_BLOCK_RECURSIVE;
  p.ops = kLoadA | kDoWY;
  return run(p, desc, cuda_stream);
}

int tri_inv_fused(const void* K, const void* V, const float* beta, const float* g,
                  float* A, void* W, void* U,
                  const tri_inv_desc* desc, int method, void* cuda_stream) {
  int rc = check_desc(desc, true);
  if (rc) return rc;
  if (!K || !V || !beta || !g || !W || !U) return TRI_INV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(beta) || !aligned16(g) || !aligned16(A) || !aligned16(W) || !aligned16(U))
    return TRI_INV_ERR_INVALID_ARG;
  if ((rc = check_method(method, true))) return rc;
  KParams p{};
  p.K = K; p.V = V; p.beta = beta; p.g = g; p.A = A; p.W = W; p.U = U;
  p.method = method & ~TRI_INV_W_DECAY;
  p.ops = kDoWY | (A ? kStoreA : 0) | ((method & TRI_INV_W_DECAY) ? kWDecay : 0);
  return run(p, desc, cuda_stream);
}

int tri_inv_fused_raw(const void* K_raw, const void* V, const float* beta_logit, const float* gate_logit,
                      float* A, void* W, void* U, float* beta_out, float* g_out,
                      const tri_inv_desc* desc, int method, void* cuda_stream) {
  int rc = check_desc(desc, true);
  if (rc) return rc;
  if (!K_raw || !V || !beta_logit || !gate_logit || !W || !U) return TRI_INV_ERR_INVALID_ARG;
  if (!aligned16(K_raw) || !aligned16(V) || !aligned16(beta_logit) || !aligned16(gate_logit) || !aligned16(A) ||
      !aligned16(W) || !aligned16(U) || !aligned16(beta_out) || !aligned16(g_out))
    return TRI_INV_ERR_INVALID_ARG;
  if ((rc = check_method(method, true))) return rc;
  KParams p{};
  p.K = K_raw; p.V = V; p.beta = beta_logit; p.g = gate_logit; p.A = A; p.W = W; p.U = U;
  p.beta_out = beta_out; p.g_out = g_out;
  p.method = method & ~TRI_INV_W_DECAY;
  p.ops = kDoWY | kRaw | (A ? kStoreA : 0) | ((method & TRI_INV_W_DECAY) ? kWDecay : 0);
  return run(p, desc, cuda_stream);
}

int tri_inv_build_kda(const void* K, const float* G, const float* beta, float* A,
                       const tri_inv_desc* desc, int method, void* cuda_stream) {
  int rc = check_desc(desc, false);
  if (rc) return rc;
  if (!K || !G || !beta || !A) return TRI_INV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(G) || !aligned16(beta) || !aligned16(A)) return TRI_INV_ERR_INVALID_ARG;
  if ((rc = check_method(method, false, false))) return rc;
  KParams p{};
  p.K = K; p.G = G; p.beta = beta; p.g = nullptr; p.A = A;
  p.method = method;
  p.ops = kStoreA | kKda;
  return run(p, desc, cuda_stream);
}

}  // extern "C"

namespace {
// Shared body of the two chunk-scan entry points: exactly one of g (scalar gate) and G (per-channel gate) is given.
int chunk_scan_any(const void* Q, const void* K, const void* W, const void* U, const float* g, const float* G, const float* S0,
                   void* O, float* S_out, float scale, const tri_inv_desc* desc, void* cuda_stream,
                   unsigned long long wait_limit_ns = 0, int test_stall = 0) {
  int rc = check_desc(desc, true);
  if (rc) return rc;
  if (!Q || !K || !W || !U || (!g && !G) || !O) return TRI_INV_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(W) || !aligned16(U) || !aligned16(g) || !aligned16(G) || !aligned16(O) ||
      !aligned16(S0) || !aligned16(S_out))
    return TRI_INV_ERR_INVALID_ARG;
  // the tensor-core kernel's shape; with a per-channel gate its operands are prepared first (one more launch)
  const bool tc = desc->kv_dtype == TRI_INV_BF16 && desc->d_k == 128 && desc->d_v == 128 && desc->C == 64;
  if (!tc && desc->d_k > 256) return TRI_INV_ERR_UNSUPPORTED;   // the CUDA-core kernel keeps a d_k x 32 slice of S in shared memory
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  ScanParams p{};
  p.U = U; p.g = g; p.G = G; p.S0 = S0; p.O = O; p.S_out = S_out; p.scale = scale;
  p.wait_limit_ns = wait_limit_ns; p.test_stall = test_stall;
  p.H = desc->H; p.T = desc->T;
  p.n_seqs = desc->cu_seqlens ? desc->n_seqs : desc->B;
  cudaError_t err;
  p.status = status_word_for_current_device(&err);
  if (!p.status) return TRI_INV_ERR_CUDA;
  const long long tokens = desc->cu_seqlens ? (long long)desc->T : (long long)desc->T * desc->B;
  if (p.n_seqs == 0 || (tokens == 0 && !S_out)) return TRI_INV_OK;
  int* dev_off = nullptr;
  if (desc->cu_seqlens) {
    cudaMemPool_t pool = table_pool_for_current_device();
    if (!pool || cudaMallocFromPoolAsync((void**)&dev_off, (size_t)(p.n_seqs + 1) * sizeof(int), pool, stream) != cudaSuccess) return TRI_INV_ERR_CUDA;
    if (launch_seq_offsets(dev_off, desc, stream) != cudaSuccess) {
      cudaFreeAsync(dev_off, stream);
      return TRI_INV_ERR_CUDA;
    }
    p.seq_off = dev_off;
  }
  void* work = nullptr;
  if (tc && G && tokens > 0) {
    // Per-channel gate on the tensor cores: Q+, K-, W- (bf16, the tensors' own shape) and the per-chunk vectors
    // exp(G_last), exp(G_ref), exp(G_last - G_ref), in stream-ordered scratch memory that is released behind the scan.
    int max_len = desc->T;
    if (desc->cu_seqlens) {
      max_len = 0;
      for (int q = 0; q < desc->n_seqs; ++q) max_len = std::max(max_len, desc->cu_seqlens[q + 1] - desc->cu_seqlens[q]);
    }
    const size_t tensor_bytes = ((size_t)tokens * desc->H * 128 * 2 + 255) & ~(size_t)255;
    const size_t slots = (size_t)(tokens / 64) + (size_t)p.n_seqs + 1;
    const size_t vec_bytes = (slots * desc->H * 128 * sizeof(float) + 255) & ~(size_t)255;
    cudaMemPool_t pool = table_pool_for_current_device();
    if (!pool || cudaMallocFromPoolAsync(&work, 3 * tensor_bytes + 3 * vec_bytes, pool, stream) != cudaSuccess) {
      if (dev_off) cudaFreeAsync(dev_off, stream);
      return TRI_INV_ERR_CUDA;
    }
    char* w = reinterpret_cast<char*>(work);
    void *Qp = w, *Km = w + tensor_bytes, *Wm = w + 2 * tensor_bytes;
    float* EL = reinterpret_cast<float*>(w + 3 * tensor_bytes);
    float* ER = reinterpret_cast<float*>(w + 3 * tensor_bytes + vec_bytes);
    float* EX = reinterpret_cast<float*>(w + 3 * tensor_bytes + 2 * vec_bytes);
    p.EL = EL; p.ER = ER; p.EX = EX;
    err = launch_kda_scan_prep(p, Q, K, W, Qp, Km, Wm, EL, ER, EX, (max_len + 63) / 64, stream);
    if (err == cudaSuccess) {
      g_launches.fetch_add(1, std::memory_order_relaxed);
      err = launch_chunk_scan(p, Qp, Km, Wm, tokens, stream, true);
    }
  } else {
    err = (tc && !G) ? launch_chunk_scan(p, Q, K, W, tokens > 0 ? tokens : 1, stream)
                     : launch_chunk_scan_simt(p, Q, K, W, desc->d_k, desc->d_v, desc->C, desc->kv_dtype, stream);
  }
  if (err == cudaSuccess) g_launches.fetch_add(1, std::memory_order_relaxed);
  if (work) cudaFreeAsync(work, stream);
  if (dev_off) cudaFreeAsync(dev_off, stream);
  return err == cudaSuccess ? TRI_INV_OK : TRI_INV_ERR_CUDA;
}
}  // namespace

extern "C" {

int tri_inv_chunk_scan(const void* Q, const void* K, const void* W, const void* U, const float* g, const float* S0,
                       void* O, float* S_out, float scale, const tri_inv_desc* desc, void* cuda_stream) {
  if (!g) return TRI_INV_ERR_INVALID_ARG;
  return chunk_scan_any(Q, K, W, U, g, nullptr, S0, O, S_out, scale, desc, cuda_stream);
}

int tri_inv_chunk_scan_kda(const void* Q, const void* K, const void* W, const void* U, const float* G, const float* S0,
                           void* O, float* S_out, float scale, const tri_inv_desc* desc, void* cuda_stream) {
  if (!G) return TRI_INV_ERR_INVALID_ARG;
  return chunk_scan_any(Q, K, W, U, nullptr, G, S0, O, S_out, scale, desc, cuda_stream);
}

int tri_inv_selftest_scan_wait_timeout(const void* Q, const void* K, const void* W, const void* U, const float* g, void* O,
                                       const tri_inv_desc* desc, uint64_t wait_limit_ns, void* cuda_stream) {
  int rc = check_desc(desc, true);
  if (rc) return rc;
  if (!g || wait_limit_ns == 0) return TRI_INV_ERR_INVALID_ARG;
  // only the tensor-core kernel has the stall hook
  if (desc->kv_dtype != TRI_INV_BF16 || desc->d_k != 128 || desc->d_v != 128 || desc->C != 64) return TRI_INV_ERR_UNSUPPORTED;
  rc = chunk_scan_any(Q, K, W, U, g, nullptr, nullptr, O, nullptr, 1.f, desc, cuda_stream, wait_limit_ns, 1);
  if (rc) return rc;
  return cudaStreamSynchronize((cudaStream_t)cuda_stream) == cudaSuccess ? TRI_INV_OK : TRI_INV_ERR_CUDA;
}

int tri_inv_fused_kda(const void* K, const void* V, const float* G, const float* beta,
                      float* A, void* W, void* U, const tri_inv_desc* desc, int method, void* cuda_stream) {
  int rc = check_desc(desc, true);
  if (rc) return rc;
  if (!K || !V || !G || !beta || !A || !W || !U) return TRI_INV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(G) || !aligned16(beta) || !aligned16(A) || !aligned16(W) || !aligned16(U))
    return TRI_INV_ERR_INVALID_ARG;
  if ((rc = check_method(method, false, false))) return rc;
  const bool tc = !(method & (TRI_INV_FORCE_SIMT | TRI_INV_REFINE)) && (method & TRI_INV_METHOD_MASK) == TRI_INV_BLOCK_RECURSIVE &&
                  desc->kv_dtype == TRI_INV_BF16 && desc->d_k == 128 && desc->d_v == 128 && (desc->C == 64 || desc->C == 128);
  if (tc && desc->C == 64) {
    // one kernel: build, inversion and both factors (W's columns scaled by exp(G_ref) on the way out)
    KParams p{};
    p.K = K; p.V = V; p.G = G; p.beta = beta; p.g = nullptr; p.A = A; p.W = W; p.U = U;
    p.method = method;
    p.ops = kStoreA | kDoWY | kKda;
    return run(p, desc, cuda_stream);
  }
  if (tc) {
    // C = 128, two launches on the stream: the per-channel build kernel, which also writes K' = K * exp(G) into
    // the W buffer while it has K and G in shared memory; then W = A diag(beta) K' and U = A diag(beta) V by the WY kernel,
    // which reads each K' tile whole into shared memory before it writes the same rows of W.
    KParams p{};
    p.K = K; p.G = G; p.beta = beta; p.g = nullptr; p.A = A; p.W = W;
    p.method = method;
    p.ops = kStoreA | kKda;
    if ((rc = run(p, desc, cuda_stream))) return rc;
    return tri_inv_wy(A, W, V, beta, W, U, desc, cuda_stream);
  }
  KParams p{};
  p.K = K; p.V = V; p.G = G; p.beta = beta; p.g = nullptr; p.A = A; p.W = W; p.U = U;
  p.method = method | TRI_INV_FORCE_SIMT;
  p.ops = kStoreA | kDoWY | kKda;
  return run(p, desc, cuda_stream);
}

int tri_inv_selftest_wait_timeout(const void* K, const void* V, const float* beta, const float* g,
                                  float* A, void* W, void* U, const tri_inv_desc* desc,
                                  uint64_t wait_limit_ns, int* counters_idle, void* cuda_stream) {
  int rc = check_desc(desc, true);
  if (rc) return rc;
  if (!K || !V || !beta || !g || !A || !W || !U || !counters_idle || wait_limit_ns == 0) return TRI_INV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(beta) || !aligned16(g) || !aligned16(A) || !aligned16(W) || !aligned16(U))
    return TRI_INV_ERR_INVALID_ARG;
  // only the tensor-core kernel has the stall hook
  if (desc->kv_dtype != TRI_INV_BF16 || desc->d_k != 128 || desc->d_v != 128 || (desc->C != 64 && desc->C != 128))
    return TRI_INV_ERR_UNSUPPORTED;
  KParams p{};
  p.K = K; p.V = V; p.beta = beta; p.g = g; p.A = A; p.W = W; p.U = U;
  p.method = TRI_INV_BLOCK_RECURSIVE;
  p.ops = kDoWY | kStoreA | kTestStall;
  p.wait_limit_ns = wait_limit_ns;
  rc = run(p, desc, cuda_stream);
  if (rc) return rc;
  if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return TRI_INV_ERR_CUDA;
  bool idle = false;
  if (work_counters_idle(&idle) != cudaSuccess) return TRI_INV_ERR_CUDA;
  *counters_idle = idle ? 1 : 0;
  return TRI_INV_OK;
}

int tri_inv_selftest_kda_wait_timeout(const void* K, const void* V, const float* G, const float* beta,
                                      float* A, void* W, void* U, const tri_inv_desc* desc,
                                      uint64_t wait_limit_ns, void* cuda_stream) {
  int rc = check_desc(desc, true);
  if (rc) return rc;
  if (!K || !G || !beta || !A || wait_limit_ns == 0) return TRI_INV_ERR_INVALID_ARG;
  const bool wy = V || W || U;
  if (wy && (!V || !W || !U)) return TRI_INV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(G) || !aligned16(beta) || !aligned16(A) || (wy && (!aligned16(V) || !aligned16(W) || !aligned16(U))))
    return TRI_INV_ERR_INVALID_ARG;
  // only the tensor-core kernels have the stall hook
  if (desc->kv_dtype != TRI_INV_BF16 || desc->d_k != 128 || desc->d_v != 128 || (desc->C != 64 && desc->C != 128))
    return TRI_INV_ERR_UNSUPPORTED;
  KParams p{};
  p.K = K; p.G = G; p.beta = beta; p.g = nullptr; p.A = A;
  p.method = TRI_INV_BLOCK_RECURSIVE;
  p.wait_limit_ns = wait_limit_ns;
  if (wy && desc->C == 64) {          // the one-kernel form
    p.V = V; p.W = W; p.U = U;
    p.ops = kStoreA | kDoWY | kKda | kTestStall;
    rc = run(p, desc, cuda_stream);
  } else {                            // the build kernel (C = 128 with W, U: its instance that also writes K exp(G), then the WY kernel)
    p.W = wy ? W : nullptr;
    p.ops = kStoreA | kKda | kTestStall;
    rc = run(p, desc, cuda_stream);
    if (!rc && wy) rc = tri_inv_wy(A, W, V, beta, W, U, desc, cuda_stream);
  }
  if (rc) return rc;
  return cudaStreamSynchronize((cudaStream_t)cuda_stream) == cudaSuccess ? TRI_INV_OK : TRI_INV_ERR_CUDA;
}

int tri_inv_selftest_bounds_check(const void* K, const void* V, const float* beta, const float* g,
                                  float* A, void* W, void* U, const tri_inv_desc* desc, void* cuda_stream) {
  int rc = check_desc(desc, true);
  if (rc) return rc;
  if (!K || !V || !beta || !g || !A || !W || !U) return TRI_INV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(beta) || !aligned16(g) || !aligned16(A) || !aligned16(W) || !aligned16(U))
    return TRI_INV_ERR_INVALID_ARG;
  KParams p{};
  p.K = K; p.V = V; p.beta = beta; p.g = g; p.A = A; p.W = W; p.U = U;
  p.method = TRI_INV_BLOCK_RECURSIVE;
  p.ops = kDoWY | kStoreA | kTestShrink;
  return run(p, desc, cuda_stream);
}

int tri_inv_count_matrices(const tri_inv_desc* desc, int64_t* out) {
  int rc = check_desc(desc, false);
  if (rc) return rc;
  if (!out) return TRI_INV_ERR_INVALID_ARG;
  long long n = 0;
  if (desc->cu_seqlens) {
    for (int s = 0; s < desc->n_seqs; ++s) {
      long long len = desc->cu_seqlens[s + 1] - desc->cu_seqlens[s];
      n += (len + desc->C - 1) / desc->C;
    }
  } else {
    n = (long long)desc->B * ((desc->T + desc->C - 1) / desc->C);
  }
  *out = n * desc->H;
  return TRI_INV_OK;
}

int tri_inv_last_device_status(int* out) {
  if (!out) return TRI_INV_ERR_INVALID_ARG;
  cudaError_t err;
  int* word = status_word_for_current_device(&err);
  if (!word) return TRI_INV_ERR_CUDA;
  int v = 0;
  if (cudaMemcpy(&v, word, sizeof v, cudaMemcpyDeviceToHost) != cudaSuccess) return TRI_INV_ERR_CUDA;
  if (v != 0) {
    int zero = 0;
    if (cudaMemcpy(word, &zero, sizeof zero, cudaMemcpyHostToDevice) != cudaSuccess) return TRI_INV_ERR_CUDA;
  }
  *out = v;
  return TRI_INV_OK;
}

#ifdef TRI_INV_DEBUG
// Bounds-checking build only: source line (in the kernels' files) of the first check that failed since the last call; 0 if none.
int tri_inv_debug_first_failed_check(int* line) {
  cudaError_t err;
  int* word = status_word_for_current_device(&err);
  if (!word || !line) return TRI_INV_ERR_CUDA;
  if (cudaMemcpy(line, word + 1, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return TRI_INV_ERR_CUDA;
  return cudaMemset(word + 1, 0, sizeof(int)) == cudaSuccess ? TRI_INV_OK : TRI_INV_ERR_CUDA;
}
#endif

int64_t tri_inv_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

const char* tri_inv_status_string(int status) {
  switch (status) {
    case TRI_INV_OK: return "ok";
    case TRI_INV_ERR_INVALID_ARG: return "invalid argument";
    case TRI_INV_ERR_UNSUPPORTED: return "unsupported request";
    case TRI_INV_ERR_CUDA: return "CUDA runtime error";
    case TRI_INV_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case TRI_INV_ERR_TOO_LARGE: return "more chunks than the static scratch table holds";
    case TRI_INV_ERR_DEBUG_CHECK: return "a bounds or phase check of the debug build failed";
    default: return "unknown status";
  }
}

}  // extern "C"
