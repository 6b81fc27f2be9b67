// Per-channel decay (the KDA row of Table 1) through the chunk scan: the operands of the tensor-core scan kernel.
// With G [tokens,H,128] the cumulative per-channel log-decay inside each chunk of 64 tokens, G_ref the chunk's middle
// row and G_last its last row, the chunk form
//     P_ij = sum_k Q_ik K_jk exp(G_ik - G_jk),   O = (Q exp G) S + P U~,   S <- diag(exp G_last) S + (K exp(G_last - G))^T U~
// becomes the scalar-gate kernel's three products on
//     Q+ = Q exp(G - G_ref),   K- = K exp(G_ref - G),   W- = W exp(-G_ref)
// (each factor within exp(+-|G over 32 tokens|)), with the state operand scaled per row by exp(G_ref),
//     [W- ; Q+] . [diag(exp G_ref) S | K-^T]  =  [W S | . ; (Q exp G) S | Q+ K-^T],
// and the state increment taken from K- as well: (K exp(G_last - G))^T U~ = diag(exp(G_last - G_ref)) K-^T U~.
// One pass over Q, K, W and G writes the three bf16 tensors and, per chunk, exp(G_last), exp(G_ref) and
// exp(G_last - G_ref); the exponent of each difference is taken once per element instead of once per (i, j, k).
#include "common.cuh"

namespace tri_inv {
namespace {

constexpr int C = 64, D = 128, NT = 256;
constexpr float kLog2e = 1.4426950408889634f;

struct PrepArgs {
  const __nv_bfloat16 *Q, *K, *W;
  const float* G;
  __nv_bfloat16 *Qp, *Km, *Wm;
  float *EL, *ER, *EX;
  const int* seq_off;
  int H, T, n_seqs;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&v);
}

// blockIdx.x: (sequence, head); blockIdx.y strides over the sequence's chunks.  16 threads per token row (8 features
// each: 16 bytes of bf16, 32 of fp32), 16 rows per pass, four passes per chunk.
__global__ void __launch_bounds__(NT) kda_scan_prep_kernel(PrepArgs a) {
  const int s = blockIdx.x / a.H, h = blockIdx.x % a.H;
  const int beg = a.seq_off ? a.seq_off[s] : s * a.T;
  const int end = a.seq_off ? a.seq_off[s + 1] : (s + 1) * a.T;
  const int n_chunks = (end - beg + C - 1) / C;
  const int tid = threadIdx.x, r0 = tid >> 4, f0 = 8 * (tid & 15);
  for (int c = blockIdx.y; c < n_chunks; c += gridDim.y) {
    const int tok0 = beg + c * C, rows = end - tok0 < C ? end - tok0 : C;
    const size_t ref_row = ((size_t)(tok0 + (rows >> 1)) * a.H + h) * D + f0, last_row = ((size_t)(tok0 + rows - 1) * a.H + h) * D + f0;
    float gref[8], glast[8];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const float4 x = *reinterpret_cast<const float4*>(a.G + ref_row + 4 * q), y = *reinterpret_cast<const float4*>(a.G + last_row + 4 * q);
      gref[4 * q] = x.x * kLog2e; gref[4 * q + 1] = x.y * kLog2e; gref[4 * q + 2] = x.z * kLog2e; gref[4 * q + 3] = x.w * kLog2e;
      glast[4 * q] = y.x * kLog2e; glast[4 * q + 1] = y.y * kLog2e; glast[4 * q + 2] = y.z * kLog2e; glast[4 * q + 3] = y.w * kLog2e;
    }
    if (r0 == 0) {
      const size_t slot = ((size_t)(tok0 / C + s) * a.H + h) * D + f0;
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        *reinterpret_cast<float4*>(a.EL + slot + 4 * q) = make_float4(ex2f(glast[4 * q]), ex2f(glast[4 * q + 1]), ex2f(glast[4 * q + 2]), ex2f(glast[4 * q + 3]));
        *reinterpret_cast<float4*>(a.ER + slot + 4 * q) = make_float4(ex2f(gref[4 * q]), ex2f(gref[4 * q + 1]), ex2f(gref[4 * q + 2]), ex2f(gref[4 * q + 3]));
        *reinterpret_cast<float4*>(a.EX + slot + 4 * q) = make_float4(ex2f(glast[4 * q] - gref[4 * q]), ex2f(glast[4 * q + 1] - gref[4 * q + 1]),
                                                                      ex2f(glast[4 * q + 2] - gref[4 * q + 2]), ex2f(glast[4 * q + 3] - gref[4 * q + 3]));
      }
    }
    float wneg[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) wneg[e] = ex2f(-gref[e]);
#pragma unroll
    for (int pass = 0; pass < 4; ++pass) {
      const int r = r0 + 16 * pass;
      if (r >= rows) break;
      const size_t idx = ((size_t)(tok0 + r) * a.H + h) * D + f0;
      const uint4 qv = *reinterpret_cast<const uint4*>(a.Q + idx), kv = *reinterpret_cast<const uint4*>(a.K + idx),
                  wv = *reinterpret_cast<const uint4*>(a.W + idx);
      float g[8];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const float4 x = *reinterpret_cast<const float4*>(a.G + idx + 4 * q);
        g[4 * q] = x.x * kLog2e; g[4 * q + 1] = x.y * kLog2e; g[4 * q + 2] = x.z * kLog2e; g[4 * q + 3] = x.w * kLog2e;
      }
      const uint32_t* qw = reinterpret_cast<const uint32_t*>(&qv);
      const uint32_t* kw = reinterpret_cast<const uint32_t*>(&kv);
      const uint32_t* ww = reinterpret_cast<const uint32_t*>(&wv);
      uint4 qo, mo, wo;
      uint32_t *qp = reinterpret_cast<uint32_t*>(&qo), *mp = reinterpret_cast<uint32_t*>(&mo), *wp = reinterpret_cast<uint32_t*>(&wo);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 qf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&qw[e]));
        const float2 kf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kw[e]));
        const float2 wf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&ww[e]));
        const float x0 = g[2 * e] - gref[2 * e], x1 = g[2 * e + 1] - gref[2 * e + 1];
        qp[e] = pack2(qf.x * ex2f(x0), qf.y * ex2f(x1));
        mp[e] = pack2(kf.x * ex2f(-x0), kf.y * ex2f(-x1));
        wp[e] = pack2(wf.x * wneg[2 * e], wf.y * wneg[2 * e + 1]);
      }
      *reinterpret_cast<uint4*>(a.Qp + idx) = qo;
      *reinterpret_cast<uint4*>(a.Km + idx) = mo;
      *reinterpret_cast<uint4*>(a.Wm + idx) = wo;
    }
  }
}

}  // namespace

cudaError_t launch_kda_scan_prep(const ScanParams& p, const void* Q, const void* K, const void* W, void* Qp, void* Km, void* Wm,
                                 float* EL, float* ER, float* EX, int max_chunks_per_seq, cudaStream_t stream) {
  PrepArgs a{reinterpret_cast<const __nv_bfloat16*>(Q), reinterpret_cast<const __nv_bfloat16*>(K), reinterpret_cast<const __nv_bfloat16*>(W), p.G,
             reinterpret_cast<__nv_bfloat16*>(Qp), reinterpret_cast<__nv_bfloat16*>(Km), reinterpret_cast<__nv_bfloat16*>(Wm), EL, ER, EX,
             p.seq_off, p.H, p.T, p.n_seqs};
  const long long gx = (long long)p.n_seqs * p.H;
  if (gx > 0x7fffffffLL) return cudaErrorInvalidValue;
  if (gx == 0 || max_chunks_per_seq <= 0) return cudaSuccess;
  // enough CTAs to fill the machine several times over, no more: each strides over its sequence's chunks
  long long gy = max_chunks_per_seq;
  const long long want = 4096 / (gx < 4096 ? gx : 4096);
  if (gy > want) gy = want > 0 ? want : 1;
  if (gy > 65535) gy = 65535;
  kda_scan_prep_kernel<<<dim3((unsigned)gx, (unsigned)gy), NT, 0, stream>>>(a);
  return cudaGetLastError();
}

}  // namespace tri_inv
