// Shared declarations of the CUDA side: kernel parameter block, chunk lookup, launchers.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tri_inv.h"

namespace tri_inv {

// What a launch does besides inverting.
enum : int {
  kStoreA = 1,  // write A to global memory
  kDoWY = 2,    // compute W (and U when V != nullptr)
  kLoadA = 4,   // skip build + inversion, read A from A_in (tri_inv_wy)
  kRaw = 8,     // K is un-normalised, beta and g are logits: normalise, sigmoid, log-sigmoid + chunk cumsum in the kernel
  kKda = 16,    // per-channel decay (KParams::G); with kDoWY, W = A diag(beta) (K * exp G)
  kFixedStride = 64,  // tensor-core kernel: take no work-counter pair (and create no event for one); items by a fixed stride
  kTestShrink = 256,  // self-test: the token bound the debug build checks against is understated by one chunk
  kTestStall = 128,   // self-test: CTA 0 leaves out the first Gram product so that its bounded wait runs out
  kWDecay = 32, // W = A diag(beta) diag(exp g) K: the decay-weighted factor the chunk-state recurrence consumes
};

// One entry per chunk of tokens in ragged mode.
struct ChunkEntry {
  int32_t tok0;  // first flat token of the chunk
  int32_t rows;  // real tokens in it (1..C)
};

struct KParams {
  const void* K;
  const void* V;
  const float* beta;
  const float* g;
  const float* A_in;
  const float* G;               // per-channel decay (kKda): cumulative log-decay [B,T,H,d_k] fp32
  float* A;
  void* W;
  void* U;
  float* beta_out;              // raw front end: sigmoid(beta logits), optional
  float* g_out;                 // raw front end: within-chunk cumulative log-decay, optional
  const ChunkEntry* chunk_tab;  // ragged mode, else nullptr
  int* status;                  // device status word (0 = ok); kernels only ever raise it
  int* work_counter;            // tensor-core kernel: {next dynamic item, finished CTAs}; both zero between launches
  int32_t H, d_k, d_v, T;
  int32_t chunks_per_seq;       // dense mode: ceil(T / C)
  int32_t n_chunks;             // token chunks (all sequences); matrices = n_chunks * H
  int32_t kv_dtype;
  int32_t method;               // TRI_INV_* method with flags
  int32_t ops;                  // kStoreA | kDoWY | kLoadA | ...
  unsigned long long wait_limit_ns;  // per bounded device-side wait (run() fills in the default of two seconds)
  int32_t a_box;                // build-only tensor-core kernel: 1 when the W tensor-map slot carries the 3-D map of A (whole-matrix store)
  long long n_tokens;           // flat tokens of the tensors (B * T, or T when packed): the bound the debug build checks rows against
};

// Bounds-checking build (-DTRI_INV_DEBUG, libtri_inv_debug.so): TRI_INV_CHECK(p, cond) raises TRI_INV_ERR_DEBUG_CHECK in
// the device status word when cond is false and evaluates to cond, so that the guarded access can be skipped; in the
// ordinary build it is the constant true and costs nothing.  Never a trap or a device assert.
#ifdef TRI_INV_DEBUG
#define TRI_INV_CHECK(p, cond) ((cond) ? true : (atomicMax((p).status, (int)TRI_INV_ERR_DEBUG_CHECK), atomicCAS((p).status + 1, 0, __LINE__), false))   // word 1: source line of the first failed check
#else
#define TRI_INV_CHECK(p, cond) (true)
#endif

// Flat work item -> (first token, real rows, head).  Consecutive items walk the heads of
// one chunk of tokens, so neighbouring CTAs touch neighbouring memory.  Items and tokens are
// below 2^31 (checked on the host), so 32-bit unsigned division is enough.
__device__ __forceinline__ void locate(const KParams& p, int C, int item, int& tok0, int& rows, int& h) {
  const unsigned c = (unsigned)item / (unsigned)p.H;
  h = (int)((unsigned)item - c * (unsigned)p.H);
  if (p.chunk_tab) {
    ChunkEntry e = TRI_INV_CHECK(p, c < (unsigned)p.n_chunks) ? p.chunk_tab[c] : ChunkEntry{0, 0};
    tok0 = e.tok0;
    rows = e.rows;
  } else {
    const unsigned b = c / (unsigned)p.chunks_per_seq;
    const int ci = (int)(c - b * (unsigned)p.chunks_per_seq);
    tok0 = (int)b * p.T + ci * C;
    const int left = p.T - ci * C;
    rows = left < C ? left : C;
  }
}

__device__ __forceinline__ float load_kv(const void* base, int dtype, size_t idx) {
  if (dtype == TRI_INV_F32) return ((const float*)base)[idx];
  return __bfloat162float(((const __nv_bfloat16*)base)[idx]);
}

// Launchers (defined next to their kernels).  Return a cudaError_t from the launch.
cudaError_t launch_simt(const KParams& p, int C, cudaStream_t stream);
// Tensor-core path: returns cudaErrorNotSupported when it has no kernel for the request.
cudaError_t launch_tc(const KParams& p, int C, cudaStream_t stream, bool* handled);
// Instantiations of the tensor-core kernel, one group per tc_inst_*.cu file; raw = the variant that rewrites the K tile.
cudaError_t launch_tc_c64_br(const KParams& p, cudaStream_t stream, bool raw);
cudaError_t launch_tc_c64_series(const KParams& p, cudaStream_t stream, bool raw);
cudaError_t launch_tc_c64_build(const KParams& p, cudaStream_t stream);
cudaError_t launch_tc_c64_d64(const KParams& p, cudaStream_t stream);   // head dimension 64
cudaError_t launch_tc_c128_br(const KParams& p, cudaStream_t stream, bool raw);
cudaError_t launch_tc_c128_series(const KParams& p, cudaStream_t stream, bool raw);
cudaError_t launch_tc_refine(const KParams& p, int C, cudaStream_t stream, bool raw);
cudaError_t launch_tc_series_f16(const KParams& p, int C, cudaStream_t stream, bool raw);
// The work-counter pair of a stream (tc_launch.cu), or nullptr: the kernel then walks its items with a fixed stride.
int* work_counter_for(cudaStream_t stream);
// Chunk scan (consumer of W and U): parameters other than the three TMA-staged tensors.
struct ScanParams {
  const void* U;        // [tokens,H,d_v]
  const float* g;       // [tokens,H]
  const float* G;       // [tokens,H,d_k] per-channel cumulative log-decay (KDA row) or null; CUDA-core kernel and preparation kernel
  const float* EL;      // per-channel form on the tensor cores: exp(G_last) per chunk slot [slots,H,d_k] ...
  const float* ER;      // ... exp(G_ref) ...
  const float* EX;      // ... and exp(G_last - G_ref), all written by the preparation kernel (slot of a chunk: first token / C + sequence index)
  const float* S0;      // [n_seqs,H,d_k,d_v] fp32 or null (zero state)
  void* O;              // [tokens,H,d_v], storage type of U
  float* S_out;         // [n_seqs,H,d_k,d_v] fp32 or null
  const int* seq_off;   // device copy of cu_seqlens (ragged) or null (dense: sequence s = tokens [s T, (s+1) T))
  int* status;
  int H, T, n_seqs;
  float scale;
  unsigned long long wait_limit_ns;   // limit of every device-side wait of the tensor-core scan; 0: two seconds
  int test_stall;                     // self-test: the first CTA leaves out the second product of its second chunk
};
cudaError_t launch_seq_offsets(int* dev_out, const tri_inv_desc* d, cudaStream_t stream);
cudaError_t launch_chunk_scan(const ScanParams& p, const void* Q, const void* K, const void* W, long long tokens,
                              cudaStream_t stream, bool kda = false);
// Per-channel form: the operands of the tensor-core scan from Q, K, W (bf16, [tokens,H,128]) and G, C = 64:
// Qp = Q exp(G - G_ref), Km = K exp(G_ref - G), Wm = W exp(-G_ref) and the per-chunk vectors EL = exp(G_last),
// ER = exp(G_ref), EX = exp(G_last - G_ref) ([slots,H,128] fp32), G_ref the middle row of each chunk, G_last its last.
cudaError_t launch_kda_scan_prep(const ScanParams& p, const void* Q, const void* K, const void* W, void* Qp, void* Km, void* Wm,
                                 float* EL, float* ER, float* EX, int max_chunks_per_seq, cudaStream_t stream);
// The same scan on the CUDA cores, for every other shape and storage type (fp32 arithmetic).
cudaError_t launch_chunk_scan_simt(const ScanParams& p, const void* Q, const void* K, const void* W, int d_k, int d_v, int C,
                                   int kv_dtype, cudaStream_t stream);
// Per-channel decay variant on the tensor cores (bf16 keys, d_k = 128, C = 64 or 128, block recursion).
cudaError_t launch_kda_tc(const KParams& p, int C, cudaStream_t stream, bool* handled);
cudaError_t launch_kda_tc_c128(const KParams& p, cudaStream_t stream);
// Per-channel decay, build + inversion + W and U in one kernel (bf16, d_k = d_v = 128, C = 64, block recursion).
cudaError_t launch_kda_fused_tc(const KParams& p, cudaStream_t stream);

// Fills dev_tab (one entry per chunk of tokens, in sequence order) from the host offsets in d->cu_seqlens
// with small kernels on the stream; no copy and no synchronisation.
cudaError_t launch_chunk_table(ChunkEntry* dev_tab, const tri_inv_desc* d, cudaStream_t stream);

// True when every work-counter pair of the tensor-core kernel on the current device is back at zero.
cudaError_t work_counters_idle(bool* idle);

// Adds one to the library's launch counter (tri_inv_launch_count).
void count_launch();

// Address of the device status word (0 = ok) of the current device; nullptr and *err on failure.
int* status_word_for_current_device(cudaError_t* err);

}  // namespace tri_inv
