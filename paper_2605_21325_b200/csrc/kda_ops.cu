// Helper of the per-channel (KDA) fused call: K' = K * exp(G), element by element, in the storage type of K.
// W = A diag(beta) (K * Gamma) is then the ordinary WY product on K', which the tensor-core kernel takes as it is.
// HBM-bound streaming kernel: 16-byte loads of K, 32-byte loads of G, 16-byte stores (8 elements per thread and step).
#include "common.cuh"

namespace tri_inv {
namespace {

__global__ void __launch_bounds__(256) kda_scale_bf16_kernel(const uint4* __restrict__ K, const float4* __restrict__ G,
                                                             uint4* __restrict__ out, long long n8) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (long long)gridDim.x * blockDim.x) {
    uint4 k = K[i];
    const float4 g0 = G[2 * i], g1 = G[2 * i + 1];
    const float gs[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
    uint32_t* w = reinterpret_cast<uint32_t*>(&k);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float2 f = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&w[q]));
      __nv_bfloat162 r = __floats2bfloat162_rn(f.x * __expf(gs[2 * q]), f.y * __expf(gs[2 * q + 1]));
      w[q] = *reinterpret_cast<uint32_t*>(&r);
    }
    out[i] = k;
  }
}

__global__ void __launch_bounds__(256) kda_scale_f32_kernel(const float4* __restrict__ K, const float4* __restrict__ G,
                                                            float4* __restrict__ out, long long n4) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
    const float4 k = K[i], g = G[i];
    out[i] = make_float4(k.x * expf(g.x), k.y * expf(g.y), k.z * expf(g.z), k.w * expf(g.w));
  }
}

}  // namespace

// n = tokens * H * d_k elements (d_k is a multiple of 8, all bases 16-byte aligned: checked by the caller).
cudaError_t launch_kda_scale_keys(const void* K, const float* G, void* out, long long n, int kv_dtype, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  const long long vec = kv_dtype == TRI_INV_BF16 ? n / 8 : n / 4;
  long long blocks = (vec + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  if (kv_dtype == TRI_INV_BF16)
    kda_scale_bf16_kernel<<<(int)blocks, 256, 0, stream>>>((const uint4*)K, (const float4*)G, (uint4*)out, vec);
  else
    kda_scale_f32_kernel<<<(int)blocks, 256, 0, stream>>>((const float4*)K, (const float4*)G, (float4*)out, vec);
  return cudaGetLastError();
}

}  // namespace tri_inv
