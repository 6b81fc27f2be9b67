// Chunk scan on the CUDA cores: the same chunk form as scan_kernel.cu for every shape and storage type the
// tensor-core kernel does not take (fp32 tensors, d_k or d_v other than 128, C other than 64).  fp32 arithmetic.
//
// One CTA of 256 threads per (sequence, head, slice of 32 value columns).  Shared memory holds the slice of the
// state S [d_k][32], U~ [C][32], P [C][C+1] and the chunk's g; W, Q and K are read from global memory (one address
// per warp and step, or staged 32 features at a time for the C x C product).  Per chunk, with barriers in between:
//   1. U~[i][n] = U[i][n] - sum_k W[i][k] S[k][n]
//   2. P[i][j]  = (q_i . k_j) exp(g_i - g_j)  for j <= i, else 0
//   3. O[i][n]  = scale (exp(g_i) sum_k Q[i][k] S[k][n] + sum_{j<=i} P[i][j] U~[j][n])
//   4. S[k][n]  = exp(g_last) S[k][n] + sum_j K[j][k] exp(g_last - g_j) U~[j][n]
// With a per-channel gate (ScanParams::G, the KDA row of Table 1) every decay factor moves inside its sum over the key
// features: P[i][j] = sum_k Q[i][k] K[j][k] exp(G[i][k] - G[j][k]), the state term of O weights Q[i][k] by exp(G[i][k]), and row k
// of S decays by exp(G_last[k]) with K[j][k] weighted by exp(G_last[k] - G[j][k]).  The exponent is taken of each difference.
#include "common.cuh"

namespace tri_inv {
namespace {

constexpr int kThreads = 256, kNS = 32, kSlice = 32;

__device__ __forceinline__ void store_out(void* base, int dtype, size_t idx, float v) {
  if (dtype == TRI_INV_F32) ((float*)base)[idx] = v;
  else ((__nv_bfloat16*)base)[idx] = __float2bfloat16_rn(v);
}

struct SimtScanArgs {
  const void *Q, *K, *W;
  int d_k, d_v, C, kv_dtype;
};

__global__ void __launch_bounds__(kThreads) scan_simt_kernel(ScanParams p, SimtScanArgs a) {
  extern __shared__ float sm[];
  const int C = a.C, d_k = a.d_k, d_v = a.d_v, LDP = C + 1;
  float* S = sm;                       // [d_k][32]
  float* Ut = S + d_k * kNS;           // [C][32]
  float* P = Ut + C * kNS;             // [C][C+1]
  float* sg = P + C * LDP;             // [C]
  float* Qs = sg + C;                  // [C][33] feature slice of Q
  float* Ks = Qs + C * (kSlice + 1);   // [C][33] feature slice of K
  float* Gs = Ks + C * (kSlice + 1);   // [C][33] feature slice of G (per-channel gate only)
  const float* G = p.G;
  const int tid = threadIdx.x, n = tid & 31, wrow = tid >> 5;   // 8 rows of 32 columns per pass
  const int n_slices = (d_v + kNS - 1) / kNS;
  const int slice = blockIdx.x % n_slices, h = (blockIdx.x / n_slices) % p.H, s = blockIdx.x / (n_slices * p.H);
  const int beg = p.seq_off ? p.seq_off[s] : s * p.T;
  const int end = p.seq_off ? p.seq_off[s + 1] : (s + 1) * p.T;
  const int col = slice * kNS + n;
  const bool col_ok = col < d_v;
  const size_t state_base = ((size_t)s * p.H + h) * d_k * d_v;

  for (int k = wrow; k < d_k; k += 8) S[k * kNS + n] = (p.S0 && col_ok) ? p.S0[state_base + (size_t)k * d_v + col] : 0.f;
  __syncthreads();

  for (int tok0 = beg; tok0 < end; tok0 += C) {
    const int rows = end - tok0 < C ? end - tok0 : C;
    for (int i = tid; i < C; i += kThreads) sg[i] = G ? 0.f : p.g[(size_t)(tok0 + (i < rows ? i : rows - 1)) * p.H + h];
    // 1. U~
    for (int i = wrow; i < C; i += 8) {
      float acc = 0.f;
      if (i < rows) {
        const size_t row = ((size_t)(tok0 + i) * p.H + h);
        for (int k = 0; k < d_k; ++k) acc = fmaf(load_kv(a.W, a.kv_dtype, row * d_k + k), S[k * kNS + n], acc);
        acc = (col_ok ? load_kv(p.U, a.kv_dtype, row * d_v + col) : 0.f) - acc;
      }
      Ut[i * kNS + n] = acc;
    }
    // 2. P, 32 features at a time through shared memory
    for (int e = tid; e < C * LDP; e += kThreads) P[e] = 0.f;
    __syncthreads();
    for (int k0 = 0; k0 < d_k; k0 += kSlice) {
      for (int e = tid; e < C * kSlice; e += kThreads) {
        const int i = e / kSlice, kk = e - i * kSlice;
        float q = 0.f, k = 0.f, gv = 0.f;
        if (i < rows && k0 + kk < d_k) {
          const size_t idx = ((size_t)(tok0 + i) * p.H + h) * d_k + k0 + kk;
          q = load_kv(a.Q, a.kv_dtype, idx);
          k = load_kv(a.K, a.kv_dtype, idx);
          if (G) gv = G[idx];
        }
        Qs[i * (kSlice + 1) + kk] = q;
        Ks[i * (kSlice + 1) + kk] = k;
        if (G) Gs[i * (kSlice + 1) + kk] = gv;
      }
      __syncthreads();
      for (int e = tid; e < C * C; e += kThreads) {
        const int i = e / C, j = e - i * C;
        if (j <= i && i < rows) {
          float acc = P[i * LDP + j];
          if (G) {
            for (int kk = 0; kk < kSlice; ++kk)
              acc = fmaf(Qs[i * (kSlice + 1) + kk] * Ks[j * (kSlice + 1) + kk], expf(Gs[i * (kSlice + 1) + kk] - Gs[j * (kSlice + 1) + kk]), acc);
          } else {
            for (int kk = 0; kk < kSlice; ++kk) acc = fmaf(Qs[i * (kSlice + 1) + kk], Ks[j * (kSlice + 1) + kk], acc);
          }
          P[i * LDP + j] = acc;
        }
      }
      __syncthreads();
    }
    for (int e = tid; e < C * C; e += kThreads) {
      const int i = e / C, j = e - i * C;
      if (j <= i && i < rows) P[i * LDP + j] *= expf(sg[i] - sg[j]);
    }
    __syncthreads();
    // 3. O
    for (int i = wrow; i < rows; i += 8) {
      const size_t row = ((size_t)(tok0 + i) * p.H + h);
      float acc = 0.f;
      if (G) {
        for (int k = 0; k < d_k; ++k) acc = fmaf(load_kv(a.Q, a.kv_dtype, row * d_k + k) * expf(G[row * d_k + k]), S[k * kNS + n], acc);
      } else {
        for (int k = 0; k < d_k; ++k) acc = fmaf(load_kv(a.Q, a.kv_dtype, row * d_k + k), S[k * kNS + n], acc);
        acc *= expf(sg[i]);
      }
      for (int j = 0; j <= i; ++j) acc = fmaf(P[i * LDP + j], Ut[j * kNS + n], acc);
      if (col_ok) store_out(p.O, a.kv_dtype, row * d_v + col, p.scale * acc);
    }
    __syncthreads();   // every read of the old S is done
    // 4. S
    const float g_last = sg[rows - 1];
    for (int k = wrow; k < d_k; k += 8) {
      float acc;
      if (G) {
        const float gl = G[((size_t)(tok0 + rows - 1) * p.H + h) * d_k + k];
        acc = expf(gl) * S[k * kNS + n];
        for (int j = 0; j < rows; ++j) {
          const size_t idx = ((size_t)(tok0 + j) * p.H + h) * d_k + k;
          acc = fmaf(load_kv(a.K, a.kv_dtype, idx) * expf(gl - G[idx]), Ut[j * kNS + n], acc);
        }
      } else {
        acc = expf(g_last) * S[k * kNS + n];
        for (int j = 0; j < rows; ++j)
          acc = fmaf(load_kv(a.K, a.kv_dtype, ((size_t)(tok0 + j) * p.H + h) * d_k + k) * expf(g_last - sg[j]), Ut[j * kNS + n], acc);
      }
      S[k * kNS + n] = acc;
    }
    __syncthreads();
  }
  if (p.S_out && col_ok)
    for (int k = wrow; k < d_k; k += 8) p.S_out[state_base + (size_t)k * d_v + col] = S[k * kNS + n];
}

}  // namespace

cudaError_t launch_chunk_scan_simt(const ScanParams& p, const void* Q, const void* K, const void* W, int d_k, int d_v, int C,
                                   int kv_dtype, cudaStream_t stream) {
  SimtScanArgs a{Q, K, W, d_k, d_v, C, kv_dtype};
  const size_t bytes = sizeof(float) * ((size_t)d_k * kNS + (size_t)C * kNS + (size_t)C * (C + 1) + C + 3 * (size_t)C * (kSlice + 1));
  if (bytes > 220 * 1024) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(scan_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) return e;
  const long long grid = (long long)p.n_seqs * p.H * ((d_v + kNS - 1) / kNS);
  if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
  if (grid == 0) return cudaSuccess;
  scan_simt_kernel<<<(int)grid, kThreads, bytes, stream>>>(p, a);
  return cudaGetLastError();
}

}  // namespace tri_inv
