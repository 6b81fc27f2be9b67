// tri_inv_fused_host: the fused call for callers whose tensors live in HOST memory.
//
// The batch is cut into slices of whole chunks; each slice goes host -> device, through tri_inv_fused, and
// device -> host on one of three internal streams, so the upload of a slice overlaps the kernel of the one
// before and the download of the one before that.  Device memory comes from the caller (a workspace of
// tri_inv_fused_host_workspace bytes); streams and events are created once per device and kept.
#include <mutex>

#include "common.cuh"

namespace tri_inv {
namespace {

constexpr int kStreams = 3, kMaxSlices = 16;

struct HostPipe {
  cudaStream_t streams[kStreams] = {};
  cudaEvent_t start = nullptr, done[kStreams] = {};
  bool ready = false;
};
std::mutex g_pipe_mu;
HostPipe g_pipes[64];

HostPipe* pipe_for_current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_pipe_mu);
  HostPipe& hp = g_pipes[dev];
  if (!hp.ready) {
    for (int i = 0; i < kStreams; ++i) {
      if (cudaStreamCreateWithFlags(&hp.streams[i], cudaStreamNonBlocking) != cudaSuccess) return nullptr;
      if (cudaEventCreateWithFlags(&hp.done[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    if (cudaEventCreateWithFlags(&hp.start, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    hp.ready = true;
  }
  return &hp;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

struct Sizes { size_t K, V, bg, A, W, U, total; };
Sizes sizes_of(const tri_inv_desc* d) {
  const size_t tokens = d->cu_seqlens ? (size_t)d->T : (size_t)d->T * d->B;
  const size_t elt = d->kv_dtype == TRI_INV_BF16 ? 2 : 4;
  Sizes s;
  s.K = align256(tokens * d->H * d->d_k * elt);
  s.V = align256(tokens * d->H * d->d_v * elt);
  s.bg = align256(tokens * d->H * 4);
  s.A = align256(tokens * d->H * d->C * 4);
  s.W = s.K;
  s.U = s.V;
  s.total = s.K + s.V + 2 * s.bg + s.A + s.W + s.U;
  return s;
}

}  // namespace
}  // namespace tri_inv

using namespace tri_inv;

extern "C" int tri_inv_fused_host_workspace(const tri_inv_desc* desc, size_t* bytes) {
  int64_t n = 0;
  int rc = tri_inv_count_matrices(desc, &n);   // validates the descriptor
  if (rc) return rc;
  if (!bytes || desc->d_v < 8 || (desc->d_v & 7)) return TRI_INV_ERR_INVALID_ARG;
  *bytes = sizes_of(desc).total;
  return TRI_INV_OK;
}

extern "C" int tri_inv_fused_host(const void* K, const void* V, const float* beta, const float* g,
                                  float* A, void* W, void* U, void* workspace, size_t workspace_bytes,
                                  const tri_inv_desc* desc, int method, void* cuda_stream) {
  size_t need = 0;
  int rc = tri_inv_fused_host_workspace(desc, &need);
  if (rc) return rc;
  if (!K || !V || !beta || !g || !W || !U || !workspace || workspace_bytes < need) return TRI_INV_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return TRI_INV_ERR_INVALID_ARG;
  HostPipe* hp = pipe_for_current_device();
  if (!hp) return TRI_INV_ERR_CUDA;
  const Sizes sz = sizes_of(desc);
  char* base = static_cast<char*>(workspace);
  char* dK = base;
  char* dV = dK + sz.K;
  char* db = dV + sz.V;
  char* dg = db + sz.bg;
  char* dA = dg + sz.bg;
  char* dW = dA + sz.A;
  char* dU = dW + sz.W;
  const size_t elt = desc->kv_dtype == TRI_INV_BF16 ? 2 : 4;
  const long long tokens = desc->cu_seqlens ? (long long)desc->T : (long long)desc->T * desc->B;
  // Slices: runs of whole chunks.  A dense batch whose sequences are whole chunks long is one run of chunks end to end
  // (chunks restart at sequence starts, which are chunk boundaries), so any cut at a chunk boundary is a dense batch of
  // one sequence.  Anything else (packed sequences, a ragged last chunk) goes as one slice.
  const bool sliceable = !desc->cu_seqlens && desc->T % desc->C == 0 && tokens >= 2LL * desc->C;
  long long n_chunks = sliceable ? tokens / desc->C : 1;
  int n_slices = sliceable ? (int)(n_chunks < kMaxSlices ? n_chunks : kMaxSlices) : 1;
  cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);
  if (cudaEventRecord(hp->start, user) != cudaSuccess) return TRI_INV_ERR_CUDA;
  for (int i = 0; i < kStreams; ++i)
    if (cudaStreamWaitEvent(hp->streams[i], hp->start, 0) != cudaSuccess) return TRI_INV_ERR_CUDA;
  const size_t row_k = (size_t)desc->H * desc->d_k * elt, row_v = (size_t)desc->H * desc->d_v * elt, row_s = (size_t)desc->H * 4,
               row_a = (size_t)desc->H * desc->C * 4;
  for (int s = 0; s < n_slices; ++s) {
    const long long t0 = sliceable ? (n_chunks * s / n_slices) * desc->C : 0;
    const long long t1 = sliceable ? (n_chunks * (s + 1) / n_slices) * desc->C : tokens;
    const size_t nt = (size_t)(t1 - t0);
    if (nt == 0) continue;
    cudaStream_t st = hp->streams[s % kStreams];
    bool ok = cudaMemcpyAsync(dK + t0 * row_k, (const char*)K + t0 * row_k, nt * row_k, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(dV + t0 * row_v, (const char*)V + t0 * row_v, nt * row_v, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(db + t0 * row_s, (const char*)beta + t0 * row_s, nt * row_s, cudaMemcpyHostToDevice, st) == cudaSuccess &&
              cudaMemcpyAsync(dg + t0 * row_s, (const char*)g + t0 * row_s, nt * row_s, cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (!ok) return TRI_INV_ERR_CUDA;
    tri_inv_desc sub = *desc;
    if (sliceable) { sub.B = 1; sub.T = (int32_t)nt; }
    rc = tri_inv_fused(dK + t0 * row_k, dV + t0 * row_v, (const float*)(db + t0 * row_s), (const float*)(dg + t0 * row_s),
                       A ? (float*)(dA + t0 * row_a) : nullptr, dW + t0 * row_k, dU + t0 * row_v, &sub, method, st);
    if (rc) return rc;
    ok = (!A || cudaMemcpyAsync((char*)A + t0 * row_a, dA + t0 * row_a, nt * row_a, cudaMemcpyDeviceToHost, st) == cudaSuccess) &&
         cudaMemcpyAsync((char*)W + t0 * row_k, dW + t0 * row_k, nt * row_k, cudaMemcpyDeviceToHost, st) == cudaSuccess &&
         cudaMemcpyAsync((char*)U + t0 * row_v, dU + t0 * row_v, nt * row_v, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (!ok) return TRI_INV_ERR_CUDA;
  }
  for (int i = 0; i < kStreams; ++i) {
    if (cudaEventRecord(hp->done[i], hp->streams[i]) != cudaSuccess) return TRI_INV_ERR_CUDA;
    if (cudaStreamWaitEvent(user, hp->done[i], 0) != cudaSuccess) return TRI_INV_ERR_CUDA;
  }
  return TRI_INV_OK;
}
