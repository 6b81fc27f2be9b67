// Host side of the tensor-core kernel: the work-counter table, the self-test read-back and the dispatch to the
// kernel's instantiations, which are compiled in the tc_inst_*.cu files (one group per file, so that they build
// in parallel).
#include <mutex>

#include "tc_device.cuh"

namespace tri_inv {
namespace {

// Work counters: a launch draws its later items from a {next item, finished CTAs} pair in a static device
// array, which the last CTA out returns to zero.  A pair must serve ONE launch at a time.  Kernels launched
// into the same stream run one after the other, so each stream gets a pair of its own (by the stream's unique
// id) and nothing has to be tracked: no event, no flag, no synchronisation.  There are kCounterSlots pairs per
// device; launches on further streams, and every launch made during stream capture (a captured launch is
// replayed later on whatever stream the graph is launched into), get no pair at all and walk their items with
// a fixed stride instead: same results, slightly less even load.
constexpr int kCounterSlots = 64;
__device__ int g_work_counters[kCounterSlots * 2];

struct CounterTable {
  int* base = nullptr;
  unsigned long long stream_id[kCounterSlots] = {};
  int used = 0;
};
std::mutex g_table_mu;
CounterTable g_tables[64];

// The pair of this stream, or nullptr for "no pair: use the fixed stride".
}  // namespace

int* work_counter_for(cudaStream_t stream) {
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return nullptr;
  unsigned long long id = 0;
  if (cudaStreamGetId(stream, &id) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_table_mu);
  CounterTable& t = g_tables[dev];
  if (!t.base) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_work_counters) != cudaSuccess) return nullptr;
    t.base = static_cast<int*>(ptr);
  }
  for (int s = 0; s < t.used; ++s)
    if (t.stream_id[s] == id) return t.base + 2 * s;
  if (t.used == kCounterSlots) return nullptr;
  t.stream_id[t.used] = id;
  return t.base + 2 * t.used++;
}

// Self-test support: true when every work-counter pair of the current device reads zero (call after a synchronise).
cudaError_t work_counters_idle(bool* idle) {
  int host[kCounterSlots * 2];
  cudaError_t e = cudaMemcpyFromSymbol(host, g_work_counters, sizeof host);
  if (e != cudaSuccess) return e;
  *idle = true;
  for (int v : host) if (v != 0) *idle = false;
  return cudaSuccess;
}

namespace {
cudaError_t launch_tc_c64(const KParams& p, cudaStream_t stream, bool series, bool raw) {
  return series ? launch_tc_c64_series(p, stream, raw) : launch_tc_c64_br(p, stream, raw);
}
cudaError_t launch_tc_c128(const KParams& p, cudaStream_t stream, bool series, bool raw) {
  return series ? launch_tc_c128_series(p, stream, raw) : launch_tc_c128_br(p, stream, raw);
}
}  // namespace

cudaError_t launch_tc(const KParams& p, int C, cudaStream_t stream, bool* handled) {
  *handled = false;
  if (p.kv_dtype != TRI_INV_BF16) return cudaSuccess;
  const bool series = (p.method & TRI_INV_METHOD_MASK) == TRI_INV_PRODUCT_SERIES;
  if ((p.method & TRI_INV_METHOD_MASK) == TRI_INV_NEWTON_SCHULZ) return cudaSuccess;   // CUDA-core kernel only
  if (C != 64 && C != 128) return cudaSuccess;
  const bool raw = (p.ops & (kRaw | kWDecay)) != 0;  // both need the variant that rewrites the K tile
  if (p.d_k == 64 && C == 64 && !series && !raw && !(p.method & (TRI_INV_REFINE | TRI_INV_OPERANDS_F16)) &&
      !((p.ops & kDoWY) && p.V && p.d_v != 64)) {
    // head dimension 64: block recursion (and series leaves) of the plain calls; everything else stays on the CUDA cores
    *handled = true;
    return launch_tc_c64_d64(p, stream);
  }
  if (p.d_k != 128 || ((p.ops & kDoWY) && p.V && p.d_v != 128)) return cudaSuccess;
  // the stride of the 2-D view (H * d * 2 bytes) is a multiple of 16 because d is a multiple of 8
  *handled = true;
  if ((p.method & TRI_INV_REFINE) && !(p.ops & kLoadA)) return launch_tc_refine(p, C, stream, raw);
  if ((p.method & TRI_INV_OPERANDS_F16) && series) return launch_tc_series_f16(p, C, stream, raw);
  if (C == 64) {
    if (!raw && !series && !(p.ops & (kDoWY | kLoadA))) return launch_tc_c64_build(p, stream);  // tri_inv_build
    return launch_tc_c64(p, stream, series, raw);
  }
  return launch_tc_c128(p, stream, series, raw);
}

}  // namespace tri_inv
