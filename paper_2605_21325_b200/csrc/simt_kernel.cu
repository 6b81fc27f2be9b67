// Plain fp32 CUDA-core kernel: every step of the path with FFMA on shared-memory matrices.
//
// It is the kernel for fp32 inputs (where single-pass tensor-core operands would not
// meet the 1e-5 bound) and for shapes the tensor-core kernel does not cover; the
// TRI_INV_FORCE_SIMT flag routes any request here.  One CTA per chunk matrix,
// 256 threads, all of N / X / a scratch matrix resident in shared memory.
//
// Steps (notation of the header): Gram S = K K^T in d-slices of 32, gate
// N_ij = beta_i S_ij exp(g_i - g_j) under the strict-lower mask, then either
//   * block recursion from 16x16 leaves (Sec. 3.3), leaves by forward substitution
//     (Sec. 3.1) or by the product series on the leaf (Alg. 2), or
//   * the product series on the whole chunk (Alg. 5),
// then A is stored and W = A diag(beta) K, U = A diag(beta) V are formed.
#include "common.cuh"

namespace tri_inv {
namespace {

constexpr int kThreads = 256;
constexpr int kSlice = 32;            // columns of K / V staged per pass
constexpr int kSliceLd = kSlice + 1;  // padded row length of the staging tile

template <int C>
struct SimtSmem {
  static constexpr int LD = C + 1;
  static constexpr size_t floats = 3 * (size_t)C * LD + (size_t)C * kSliceLd + 3 * C;
  static constexpr size_t bytes = floats * sizeof(float);
};

// dst = lower-triangular product restricted to diagonal blocks of size bs:
// dst_ij = sum_{k=j..i} a_ik b_kj for i >= j in the same block, else 0.
template <int C>
__device__ void tri_matmul_blocks(float* dst, const float* a, const float* b, int bs, int tid) {
  constexpr int LD = C + 1;
  for (int e = tid; e < C * bs; e += kThreads) {
    int i = e / bs, jj = e - i * bs;
    int base = (i / bs) * bs;
    int j = base + jj;
    float s = 0.f;
    if (j <= i)
      for (int k = j; k <= i; ++k) s = fmaf(a[i * LD + k], b[k * LD + j], s);
    dst[i * LD + j] = s;
  }
}

// Product series (Alg. 5) on every bs x bs diagonal block of N at once.
// y holds N on entry (only its diagonal blocks are read) and is destroyed; the result
// (diagonal blocks only, zero elsewhere inside them above the diagonal) ends in the
// returned buffer, one of {x, y, z}.
template <int C>
__device__ float* product_series_blocks(float* y, float* x, float* z, int bs, int tid) {
  constexpr int LD = C + 1;
  for (int e = tid; e < C * bs; e += kThreads) {  // X <- I - N on the diagonal blocks
    int i = e / bs, jj = e - i * bs;
    int j = (i / bs) * bs + jj;
    x[i * LD + j] = (i == j) ? 1.f : (j < i ? -y[i * LD + j] : 0.f);
  }
  __syncthreads();
  int rounds = 0;
  for (int m = bs; m > 2; m >>= 1) ++rounds;  // log2(bs) - 1
  for (int r = 0; r < rounds; ++r) {
    tri_matmul_blocks<C>(z, y, y, bs, tid);    // Y <- Y.Y   (into z)
    __syncthreads();
    for (int e = tid; e < C * bs; e += kThreads) {  // X <- X + X.Y   (into y's old buffer)
      int i = e / bs, jj = e - i * bs;
      int j = (i / bs) * bs + jj;
      float s = 0.f;
      if (j <= i) {
        s = x[i * LD + j];
        for (int k = j; k <= i; ++k) s = fmaf(x[i * LD + k], z[k * LD + j], s);
      }
      y[i * LD + j] = s;
    }
    __syncthreads();
    float* nx = y;  // rotate: new X = old Y buffer, new Y = z, free = old X
    y = z;
    z = x;
    x = nx;
  }
  return x;
}

// acc[m] = (a . b)_ij for the element e = tid + m * kThreads of a C x C lower-triangular product
// (a and b lower triangular, sum over k = j..i); elements above the diagonal give 0.
template <int C, int kAcc>
__device__ __forceinline__ void tri_matmul_regs(float (&acc)[kAcc], const float* a, const float* b, int tid) {
  constexpr int LD = C + 1;
#pragma unroll
  for (int m = 0; m < kAcc; ++m) {
    const int e = tid + m * kThreads;
    const int i = e / C, j = e - i * C;
    float s = 0.f;
    if (e < C * C && j <= i)
      for (int k = j; k <= i; ++k) s = fmaf(a[i * LD + k], b[k * LD + j], s);
    acc[m] = s;
  }
}

template <int C>
__global__ void __launch_bounds__(kThreads) simt_kernel(KParams p) {
  constexpr int LD = C + 1;
  extern __shared__ float smem[];
  float* Nm = smem;
  float* Xm = Nm + C * LD;
  float* Zm = Xm + C * LD;
  float* Ks = Zm + C * LD;  // [C][kSliceLd]
  float* sb = Ks + C * kSliceLd;
  float* sg = sb + C;
  float* sr = sg + C;  // raw front end: 1 / |k_i|
  const bool raw = (p.ops & kRaw) != 0;
  const bool kda = (p.ops & kKda) != 0;  // per-channel decay: each Gram term weighted by exp(G_ic - G_jc); W rows weighted by exp(G_j) per feature
  const int tid = threadIdx.x;
  const int total = p.n_chunks * p.H;
  constexpr int kAcc = (C * C + kThreads - 1) / kThreads;
  const int method = p.method & TRI_INV_METHOD_MASK;
  const int gshift = (p.method & TRI_INV_GATE_SHIFTED) ? 1 : 0;  // Comba row: row i decays from the token before it

  for (int item = blockIdx.x; item < total; item += gridDim.x) {
    int tok0, rows, h;
    locate(p, C, item, tok0, rows, h);
    // bounds-checking build: an item outside the tensors is reduced to no rows (nothing of it is then read or stored)
    if (!TRI_INV_CHECK(p, rows >= 1 && rows <= C && tok0 >= 0 && (long long)tok0 + rows <= p.n_tokens && h >= 0 && h < p.H)) { tok0 = 0; rows = 0; h = 0; }
    __syncthreads();  // previous item's readers are done with shared memory
    for (int i = tid; i < C; i += kThreads) {
      size_t bi = (size_t)(tok0 + i) * p.H + h;
      float b = (i < rows) ? p.beta[bi] : 0.f;
      float gg = (i < rows && p.g) ? p.g[bi] : 0.f;
      if (raw) {  // beta logits -> sigmoid; gate logits -> log sigmoid (summed over the chunk below)
        b = (i < rows) ? 1.f / (1.f + expf(-b)) : 0.f;
        gg = (i < rows) ? fminf(gg, 0.f) - log1pf(expf(-fabsf(gg))) : 0.f;
        if (p.beta_out && i < rows) p.beta_out[bi] = b;
      }
      sb[i] = b;
      sg[i] = gg;
      sr[i] = 1.f;
    }
    if (raw) {
      __syncthreads();
      if (tid == 0) {  // within-chunk cumulative log-decay, in token order
        float run = 0.f;
        for (int i = 0; i < C; ++i) { run += sg[i]; sg[i] = run; }
      }
      __syncthreads();
      if (p.g_out)
        for (int i = tid; i < rows; i += kThreads) p.g_out[(size_t)(tok0 + i) * p.H + h] = sg[i];
    }
    for (int e = tid; e < C * LD; e += kThreads) { Xm[e] = 0.f; Zm[e] = 0.f; Nm[e] = 0.f; }
    float* Xres = Xm;

    if (p.ops & kLoadA) {
      __syncthreads();
      for (int e = tid; e < C * C; e += kThreads) {
        int i = e / C, j = e - i * C;
        if (i < rows && j <= i) Xm[i * LD + j] = p.A_in[((size_t)(tok0 + i) * p.H + h) * C + j];
      }
      __syncthreads();
    } else {
      // ---- Gram matrix, strictly lower part, in slices of the key dimension
      float acc[kAcc];
#pragma unroll
      for (int m = 0; m < kAcc; ++m) acc[m] = 0.f;
      for (int ks = 0; ks < p.d_k; ks += kSlice) {
        __syncthreads();
        for (int e = tid; e < C * kSlice; e += kThreads) {
          int i = e / kSlice, kk = e - i * kSlice;
          float v = 0.f;
          if (i < rows && ks + kk < p.d_k) v = load_kv(p.K, p.kv_dtype, ((size_t)(tok0 + i) * p.H + h) * p.d_k + ks + kk);
          Ks[i * kSliceLd + kk] = v;
          if (kda) {  // the scratch matrix is free during the Gram phase: it holds the slice of G
            float gv = 0.f;
            if (i < rows && ks + kk < p.d_k) gv = p.G[((size_t)(tok0 + i) * p.H + h) * p.d_k + ks + kk];
            Zm[i * kSliceLd + kk] = gv;
          }
        }
        __syncthreads();
#pragma unroll
        for (int m = 0; m < kAcc; ++m) {
          int e = tid + m * kThreads;
          int i = e / C, j = e - i * C;
          if (e < C * C && (j < i || (raw && j == i))) {
            float s = acc[m];
            if (kda) {
              for (int kk = 0; kk < kSlice; ++kk)
                s = fmaf(Ks[i * kSliceLd + kk] * Ks[j * kSliceLd + kk], expf(Zm[i * kSliceLd + kk] - Zm[j * kSliceLd + kk]), s);
            } else {
#pragma unroll
              for (int kk = 0; kk < kSlice; ++kk) s = fmaf(Ks[i * kSliceLd + kk], Ks[j * kSliceLd + kk], s);
            }
            acc[m] = s;
          }
        }
      }
      if (kda) {
        __syncthreads();
        for (int e = tid; e < C * LD; e += kThreads) Zm[e] = 0.f;
      }
      if (raw) {  // 1 / |k_i| from the Gram diagonal; the Gram of the normalised keys is S_ij r_i r_j
#pragma unroll
        for (int m = 0; m < kAcc; ++m) {
          int e = tid + m * kThreads;
          int i = e / C, j = e - i * C;
          if (e < C * C && j == i) sr[i] = acc[m] > 0.f ? rsqrtf(acc[m]) : 0.f;
        }
        __syncthreads();
      }
      // ---- gate and mask: select, never multiply an overflowed exp by zero
#pragma unroll
      for (int m = 0; m < kAcc; ++m) {
        int e = tid + m * kThreads;
        int i = e / C, j = e - i * C;
        if (e < C * C && j < i && i < rows) Nm[i * LD + j] = sb[i] * (acc[m] * sr[i] * sr[j]) * expf(sg[i - gshift] - sg[j]);  // i > j >= 0, so i - 1 is in the chunk
      }
      __syncthreads();

      if (method == TRI_INV_PRODUCT_SERIES) {
        Xres = product_series_blocks<C>(Nm, Xm, Zm, C, tid);
      } else if (method == TRI_INV_NEWTON_SCHULZ) {
        // Alg. 3: M = I + N, X_0 = I / C, then m rounds of Y <- M.X, X <- 2X - X.Y.
        // All iterates are lower triangular, so the products run over k = j..i only.
        int iters = (p.method >> 12) & 0xf;
        if (iters == 0) { iters = 0; for (int m = C; m > 1; m >>= 1) iters += 2; }  // 2 log2(C)
        for (int e = tid; e < C * C; e += kThreads) {
          const int i = e / C, j = e - i * C;
          if (i == j) { Nm[i * LD + j] = 1.f; Xm[i * LD + j] = 1.f / C; }
        }
        __syncthreads();
        for (int it = 0; it < iters; ++it) {
          tri_matmul_blocks<C>(Zm, Nm, Xm, C, tid);   // Y <- M.X
          __syncthreads();
          float q[kAcc];
          tri_matmul_regs<C, kAcc>(q, Xm, Zm, tid);   // X.Y, held in registers until every read of X is done
          __syncthreads();
#pragma unroll
          for (int m = 0; m < kAcc; ++m) {
            const int e = tid + m * kThreads;
            const int i = e / C, j = e - i * C;
            if (e < C * C && j <= i) Xm[i * LD + j] = 2.f * Xm[i * LD + j] - q[m];
          }
          __syncthreads();
        }
        for (int e = tid; e < C; e += kThreads) Nm[e * LD + e] = 0.f;  // back to N for an optional refinement step
        __syncthreads();
      } else {
        constexpr int kLeaf = C < 16 ? C : 16;
        if (p.method & TRI_INV_LEAF_SERIES) {
          // Alg. 2: series on the leaves.  Work on a copy so N's off-diagonal blocks survive.
          // Ks ([C][33]) is free now and holds two compact [C][16] block-diagonal matrices.
          float* Yc = Ks;
          float* Y2 = Ks + C * kLeaf;
          for (int e = tid; e < C * kLeaf; e += kThreads) {
            int i = e / kLeaf, jj = e - i * kLeaf;
            int j = (i / kLeaf) * kLeaf + jj;
            float n = (j < i) ? Nm[i * LD + j] : 0.f;
            Yc[e] = n;
            Xm[i * LD + j] = (i == j) ? 1.f : -n;
          }
          __syncthreads();
          int rounds = 0;
          for (int m = kLeaf; m > 2; m >>= 1) ++rounds;
          for (int r = 0; r < rounds; ++r) {
            for (int e = tid; e < C * kLeaf; e += kThreads) {  // Y2 <- Yc.Yc
              int i = e / kLeaf, jj = e - i * kLeaf, ii = i % kLeaf, base = i - ii;
              float s = 0.f;
              for (int k = jj; k <= ii; ++k) s = fmaf(Yc[i * kLeaf + k], Yc[(base + k) * kLeaf + jj], s);
              Y2[e] = s;
            }
            __syncthreads();
            for (int e = tid; e < C * kLeaf; e += kThreads) {  // Z <- X + X.Y2 on the leaves
              int i = e / kLeaf, jj = e - i * kLeaf, ii = i % kLeaf, base = i - ii;
              float s = Xm[i * LD + base + jj];
              for (int k = jj; k <= ii; ++k) s = fmaf(Xm[i * LD + base + k], Y2[(base + k) * kLeaf + jj], s);
              Zm[i * LD + base + jj] = s;
            }
            __syncthreads();
            for (int e = tid; e < C * kLeaf; e += kThreads) {
              int i = e / kLeaf, jj = e - i * kLeaf, base = i - i % kLeaf;
              Xm[i * LD + base + jj] = Zm[i * LD + base + jj];
            }
            float* t = Yc; Yc = Y2; Y2 = t;
            __syncthreads();
          }
        } else {
          // forward substitution, one thread per column of its leaf (Sec. 3.1)
          if (tid < C) {
            int base = (tid / kLeaf) * kLeaf, j = tid % kLeaf;
            float x[kLeaf];
#pragma unroll
            for (int i = 0; i < kLeaf; ++i) {
              float s = 0.f;
#pragma unroll
              for (int k = 0; k < i; ++k)
                if (k >= j) s = fmaf(Nm[(base + i) * LD + base + k], x[k], s);
              x[i] = (i < j) ? 0.f : (i == j ? 1.f : -s);
            }
#pragma unroll
            for (int i = 0; i < kLeaf; ++i) Xm[(base + i) * LD + base + j] = x[i];
          }
          __syncthreads();
        }
        // merges: X21 = -(X22 . N21) . X11 for every adjacent pair of b x b blocks
        for (int b = kLeaf; b < C; b <<= 1) {
          int n_el = (C / (2 * b)) * b * b;
          for (int e = tid; e < n_el; e += kThreads) {  // T = X22 . N21 into Zm at the (2,1) block
            int pr = e / (b * b), rem = e - pr * b * b;
            int i = rem / b, j = rem - i * b;
            int r0 = pr * 2 * b + b, c0 = pr * 2 * b;
            float s = 0.f;
            for (int k = 0; k <= i; ++k) s = fmaf(Xm[(r0 + i) * LD + r0 + k], Nm[(r0 + k) * LD + c0 + j], s);
            Zm[(r0 + i) * LD + c0 + j] = s;
          }
          __syncthreads();
          for (int e = tid; e < n_el; e += kThreads) {  // X21 = -T . X11
            int pr = e / (b * b), rem = e - pr * b * b;
            int i = rem / b, j = rem - i * b;
            int r0 = pr * 2 * b + b, c0 = pr * 2 * b;
            float s = 0.f;
            for (int k = j; k < b; ++k) s = fmaf(Zm[(r0 + i) * LD + c0 + k], Xm[(c0 + k) * LD + c0 + j], s);
            Xm[(r0 + i) * LD + c0 + j] = -s;
          }
          __syncthreads();
        }
      }
    }

    // ---- optional refinement (Alg. 6): R <- I - X.M with M = I + N, then X <- X + R.X
    if ((p.method & TRI_INV_REFINE) && !(p.ops & kLoadA)) {
      float* Rm = (Xres == Zm) ? Xm : Zm;  // a buffer that is neither N nor the current result
      float q[kAcc];
      tri_matmul_regs<C, kAcc>(q, Xres, Nm, tid);  // X.N (N strictly lower; X.M = X + X.N)
#pragma unroll
      for (int m = 0; m < kAcc; ++m) {
        const int e = tid + m * kThreads;
        const int i = e / C, j = e - i * C;
        if (e < C * C) Rm[i * LD + j] = (j <= i) ? ((i == j ? 1.f : 0.f) - Xres[i * LD + j] - q[m]) : 0.f;
      }
      __syncthreads();
      tri_matmul_regs<C, kAcc>(q, Rm, Xres, tid);  // R.X
      __syncthreads();
#pragma unroll
      for (int m = 0; m < kAcc; ++m) {
        const int e = tid + m * kThreads;
        const int i = e / C, j = e - i * C;
        if (e < C * C && j <= i) Xres[i * LD + j] += q[m];
      }
      __syncthreads();
    }

    // ---- store A: computed strict-lower part, constant diagonal and upper triangle
    if ((p.ops & kStoreA) && p.A) {
      for (int e = tid; e < C * C; e += kThreads) {
        int i = e / C, j = e - i * C;
        if (i < rows && TRI_INV_CHECK(p, (long long)tok0 + i < p.n_tokens)) {
          float v = (j < i) ? Xres[i * LD + j] : (j == i ? 1.f : 0.f);
          p.A[((size_t)(tok0 + i) * p.H + h) * C + j] = v;
        }
      }
    }

    // ---- WY: W = A diag(beta) K, U = A diag(beta) V, 32 columns at a time
    if (p.ops & kDoWY) {
      for (int which = 0; which < 2; ++which) {
        const void* src = which ? p.V : p.K;
        void* dst = which ? p.U : p.W;
        int d = which ? p.d_v : p.d_k;
        if (!src || !dst) continue;
        for (int c0 = 0; c0 < d; c0 += kSlice) {
          __syncthreads();
          for (int e = tid; e < C * kSlice; e += kThreads) {
            int j = e / kSlice, cc = e - j * kSlice;
            float v = 0.f;
            if (j < rows && c0 + cc < d) {
              const size_t idx = ((size_t)(tok0 + j) * p.H + h) * d + c0 + cc;
              v = sb[j] * (which ? 1.f : sr[j] * ((p.ops & kWDecay) ? ((gshift && j == 0) ? 1.f : expf(sg[j - gshift])) : 1.f)) * load_kv(src, p.kv_dtype, idx);
              if (kda && !which) v *= expf(p.G[idx]);   // W = A diag(beta) (K * Gamma): the decay-weighted factor of the per-channel form
            }
            Ks[j * kSliceLd + cc] = v;
          }
          __syncthreads();
          int cc = tid % kSlice;
          for (int i = tid / kSlice; i < rows; i += kThreads / kSlice) {
            float s = Ks[i * kSliceLd + cc];  // diagonal term, A_ii = 1
            for (int j = 0; j < i; ++j) s = fmaf(Xres[i * LD + j], Ks[j * kSliceLd + cc], s);
            if (c0 + cc < d && TRI_INV_CHECK(p, (long long)tok0 + i < p.n_tokens)) {
              size_t o = ((size_t)(tok0 + i) * p.H + h) * d + c0 + cc;
              if (p.kv_dtype == TRI_INV_F32) ((float*)dst)[o] = s;
              else ((__nv_bfloat16*)dst)[o] = __float2bfloat16_rn(s);
            }
          }
        }
      }
    }
  }
}

template <int C>
cudaError_t launch_one(const KParams& p, cudaStream_t stream) {
  size_t bytes = SimtSmem<C>::bytes;
  cudaError_t e = cudaFuncSetAttribute(simt_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e != cudaSuccess) return e;
  long long total = (long long)p.n_chunks * p.H;
  if (total == 0) return cudaSuccess;
  int grid = (int)(total < 148LL * 64 ? total : 148LL * 64);
  simt_kernel<C><<<grid, kThreads, bytes, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_simt(const KParams& p, int C, cudaStream_t stream) {
  switch (C) {
    case 16: return launch_one<16>(p, stream);
    case 32: return launch_one<32>(p, stream);
    case 64: return launch_one<64>(p, stream);
    case 128: return launch_one<128>(p, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace tri_inv
