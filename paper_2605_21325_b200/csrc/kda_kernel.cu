// Per-channel decay variant (the KDA row of Table 1): phi = (K * Gamma)(K / Gamma)^T with Gamma = exp(G),
// G [B,T,H,d] the cumulative per-channel log-decay inside each chunk:
//     N_ij = beta_i * sum_c K_ic K_jc exp(G_ic - G_jc)   (i > j),      A = (I + N)^{-1}.
//
// Tensor-core kernel for bf16 keys, fp32 G, d = 128, C = 64 (build only).  Per item:
//   1. TMA stages the K tile (bf16) and the G tile (fp32, four boxes of 32 channels) in shared memory.
//   2. Two bf16 operands are formed in shared memory: K+ = K * exp(G - G_ref) (over K itself) and
//      K- = K * exp(G_ref - G), with G_ref the row in the middle of the chunk, so that each factor stays
//      within exp(+-|G_0 - G_mid|); their product carries exp(G_i - G_j) per channel.
//   3. S = K+ (K-)^T as tcgen05.mma (kind::f16, fp32 accumulator in tensor memory).
//   4. Gate (beta_i, strict-lower mask) and block recursion from 16x16 leaves exactly as in the scalar-gate
//      kernel; the fp32 matrix reuses the G tile's space.  A whole chunk's A leaves as one tiled bulk store
//      straight from that matrix (a 3-D map of A whose box is as wide as the padded rows in shared memory:
//      the padding columns fall outside the tensor and are dropped); a chunk cut short by its sequence's end
//      takes 16-byte stores.
// Every mbarrier wait is bounded; on expiry the kernel raises the status word, frees its tensor memory
// and returns.
#include "tc_device.cuh"

namespace tri_inv {
namespace {

constexpr int C = 64, D = 128, NW = 4, NT = 128, LD = C + 4;
constexpr int OFF_K = 0;                    // K tile, then K+            (16 KB: 2 boxes of 64 rows x 128 B)
constexpr int OFF_KM = 16384;               // K-                         (16 KB)
constexpr int OFF_G = 32768;                // G tile                     (32 KB: 4 boxes of 64 rows x 128 B)
constexpr int OFF_X = OFF_G;                // fp32 N / X matrix over G   (17,408 B)
constexpr int OFF_LEAF = OFF_X + C * LD * 4;  // series-leaf scratch, also inside the G tile's space
constexpr int LEAF_LD = 20;
constexpr int OFF_BETA = 65536;
constexpr int OFF_BAR = OFF_BETA + C * 4;   // bar_k, bar_mma, bar_g, TMEM slot
constexpr int SMEM_BYTES = OFF_BAR + 32;
constexpr int TMEM_COLS = 64;
constexpr int CTAS_PER_SM = 3;
static_assert(OFF_LEAF + NW * 16 * LEAF_LD * 4 <= OFF_BETA, "leaf scratch must fit behind the fp32 matrix");

__global__ void __launch_bounds__(NT, CTAS_PER_SM) kda_build_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                     const __grid_constant__ CUtensorMap tmG,
                                                                 const __grid_constant__ CUtensorMap tmA, KParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  float* sX = reinterpret_cast<float*>(smem + OFF_X);
  float* sBeta = reinterpret_cast<float*>(smem + OFF_BETA);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + 24);
  const uint32_t sK = smem_u32(smem + OFF_K), sKm = smem_u32(smem + OFF_KM), sG = smem_u32(smem + OFF_G);
  const uint32_t bar_k = smem_u32(smem + OFF_BAR), bar_mma = bar_k + 8, bar_g = bar_k + 16;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int rb = warp;                       // M = 64: rows 16q..16q+15 sit in TMEM lanes 32q..32q+15
  const int total = p.n_chunks * p.H;
  const bool misaligned = (sK & 1023u) != 0;

  auto issue_k = [&](int tok0, int h) {
    fence_proxy_async();
    mbar_expect_tx(bar_k, 16384u);
#pragma unroll
    for (int bx = 0; bx < 2; ++bx) tma_load_2d(sK + bx * 8192, &tmK, bar_k, h * D + 64 * bx, tok0);
  };
  auto issue_g = [&](int tok0, int h) {
    fence_proxy_async();
    mbar_expect_tx(bar_g, 32768u);
#pragma unroll
    for (int bx = 0; bx < 4; ++bx) tma_load_2d(sG + bx * 8192, &tmG, bar_g, h * D + 32 * bx, tok0);
  };
  auto fetch_beta = [&](int tok0, int rows, int h) -> float {
    return (tid < C && tid < rows) ? p.beta[(size_t)(tok0 + tid) * p.H + h] : 0.f;
  };

  float beta_next = 0.f;
  {
    int tok0 = 0, rows = 0, h = 0;
    const bool any = (int)blockIdx.x < total && !misaligned;
    if (any) locate(p, C, blockIdx.x, tok0, rows, h);
    if (tid == 64) { prefetch_tmap(&tmK); mbar_init(bar_k, 1); fence_mbar_init(); if (any) issue_k(tok0, h); }
    if (tid == 96) { prefetch_tmap(&tmG); mbar_init(bar_g, 1); fence_mbar_init(); if (any) issue_g(tok0, h); }
    if (tid == 0) { mbar_init(bar_mma, 1); fence_mbar_init(); }
    if (any) beta_next = fetch_beta(tok0, rows, h);
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_rows = tmem + ((32u * warp) << 16);
  uint32_t ph = 0, ph_mma = 0;   // K and G complete once per item: one parity for both
  // Give-up protocol as in the main kernel: a thread whose bounded wait runs out remembers it, skips its later waits and
  // finishes the item on whatever data is there; it raises the CTA's flag before the item's last barrier, behind which
  // every thread reads it, so the whole CTA leaves the loop at one place.
  __shared__ int s_gave_up;
  bool bad = false;
  auto wait = [&](uint32_t bar, uint32_t parity) {
    if (!bad) bad = !mbar_wait_bounded(bar, parity, p.wait_limit_ns);
  };
  if (tid == 0) s_gave_up = 0;   // read only behind later barriers
  bool k_pending = false;        // thread 64: a K tile has been requested that nobody has waited for yet

  for (int item = blockIdx.x; item < total && !misaligned; item += gridDim.x) {
    int tok0, rows, h;
    locate(p, C, item, tok0, rows, h);
    const int nx_item = item + gridDim.x;
    const bool has_next = nx_item < total;
    int nx_tok0 = 0, nx_rows = 0, nx_h = 0;
    if (has_next) locate(p, C, nx_item, nx_tok0, nx_rows, nx_h);
    if (tid < C) sBeta[tid] = beta_next;
    if (tid == 32 && has_next) {   // next tiles into L2 now
#pragma unroll
      for (int bx = 0; bx < 2; ++bx) tma_prefetch_l2_2d(&tmK, nx_h * D + 64 * bx, nx_tok0);
#pragma unroll
      for (int bx = 0; bx < 4; ++bx) tma_prefetch_l2_2d(&tmG, nx_h * D + 32 * bx, nx_tok0);
    }

    // ---- 2. K+ = K * 2^x over K, K- = K * 2^-x, x = (G - G_ref) log2(e); rows past the chunk's end are zero
    wait(bar_k, ph);
    wait(bar_g, ph);
    const int rref = rows >> 1;
    {
      // This thread's 8 channels are the same in every pass (NT is a multiple of 16): the reference row is read once.  The
      // passes are branch-free (rows past the chunk's end are read like the others and replaced by zeros), so that the
      // loads of one pass are in flight while the exponentials of the pass before are formed.
      const int cf = tid & 15;                            // 16-byte chunk of 8 features
      const int q0 = 2 * (cf & 3);                        // first of the two float4 of G for these 8 channels
      const uint32_t gbox = sG + (cf >> 2) * 8192;
      float gr[8];
#pragma unroll
      for (int hq = 0; hq < 2; ++hq)
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(gr[4 * hq]), "=f"(gr[4 * hq + 1]), "=f"(gr[4 * hq + 2]), "=f"(gr[4 * hq + 3])
                     : "r"(gbox + rref * 128 + (((q0 + hq) ^ (rref & 7)) << 4)));
#pragma unroll
      for (int q = 0; q < 8; ++q) gr[q] *= 1.4426950408889634f;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        // the loads of four passes first (shared-memory loads and stores keep their program order), then their arithmetic
        uint4 kv[4];
        float gv[4][8];
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const int r = (tid >> 4) + 8 * (4 * half + m);
          const uint32_t koff = (uint32_t)((cf >> 3) * 8192 + r * 128 + (((cf & 7) ^ (r & 7)) << 4));
          asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(kv[m].x), "=r"(kv[m].y), "=r"(kv[m].z), "=r"(kv[m].w) : "r"(sK + koff));
#pragma unroll
          for (int hq = 0; hq < 2; ++hq)
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(gv[m][4 * hq]), "=f"(gv[m][4 * hq + 1]), "=f"(gv[m][4 * hq + 2]), "=f"(gv[m][4 * hq + 3])
                         : "r"(gbox + r * 128 + (((q0 + hq) ^ (r & 7)) << 4)));
        }
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const int r = (tid >> 4) + 8 * (4 * half + m);
          const uint32_t koff = (uint32_t)((cf >> 3) * 8192 + r * 128 + (((cf & 7) ^ (r & 7)) << 4));
          uint4 kp, km;
          const uint32_t* kw = reinterpret_cast<const uint32_t*>(&kv[m]);
          uint32_t* pw = reinterpret_cast<uint32_t*>(&kp);
          uint32_t* mw = reinterpret_cast<uint32_t*>(&km);
          const bool live = r < rows;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float2 kf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kw[q]));
            const float x0 = fmaf(gv[m][2 * q], 1.4426950408889634f, -gr[2 * q]), x1 = fmaf(gv[m][2 * q + 1], 1.4426950408889634f, -gr[2 * q + 1]);
            const uint32_t vp = pack_bf16(kf.x * ex2_approx(x0), kf.y * ex2_approx(x1));
            const uint32_t vm = pack_bf16(kf.x * ex2_approx(-x0), kf.y * ex2_approx(-x1));
            pw[q] = live ? vp : 0u;
            mw[q] = live ? vm : 0u;
          }
          asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(sK + koff), "r"(kp.x), "r"(kp.y), "r"(kp.z), "r"(kp.w) : "memory");
          asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(sKm + koff), "r"(km.x), "r"(km.y), "r"(km.z), "r"(km.w) : "memory");
        }
      }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();

    // ---- 3. S = K+ (K-)^T
    // (self-test, kTestStall: thread block 0 leaves out the product of its first item, so that the wait below runs out)
    if (tid == 0 && !((p.ops & kTestStall) && item == 0)) {
      tc_fence_after();
      constexpr uint32_t idesc = umma_idesc(C, C, 0);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const uint32_t koff = (ks >> 2) * 8192 + (ks & 3) * 32;
        umma_bf16(tmem, umma_desc(sK + koff, 16, 1024), umma_desc(sKm + koff, 16, 1024), idesc, ks > 0);
      }
      umma_commit(bar_mma);
    }
    wait(bar_mma, ph_mma);
    ph_mma ^= 1;
    tc_fence_after();
    k_pending = false;
    if (tid == 64 && has_next && !bad) { issue_k(nx_tok0, nx_h); k_pending = true; }  // the operands' only reader has completed
    if (has_next) beta_next = fetch_beta(nx_tok0, nx_rows, nx_h);

    // ---- 4. gate (beta_i, strict-lower mask), N -> shared memory over the G tile (all of G has been consumed)
    {
      const int ra = 16 * rb + g, rbw = ra + 8;
      const float beta_a = sBeta[ra], beta_b = sBeta[rbw];
      float sacc[8][4];
      tmem_ld_16x64(sacc, tmem_rows);
      tmem_wait_ld();
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        const int c = 8 * nt + 2 * t;
        float2 va = make_float2(0.f, 0.f), vb = va;
        if (nt / 2 <= rb) {
          va.x = (c < ra) ? beta_a * sacc[nt][0] : 0.f;
          va.y = (c + 1 < ra) ? beta_a * sacc[nt][1] : 0.f;
          vb.x = (c < rbw) ? beta_b * sacc[nt][2] : 0.f;
          vb.y = (c + 1 < rbw) ? beta_b * sacc[nt][3] : 0.f;
        }
        *reinterpret_cast<float2*>(sX + ra * LD + c) = va;
        *reinterpret_cast<float2*>(sX + rbw * LD + c) = vb;
      }
    }
    __syncwarp();
    if (p.method & TRI_INV_LEAF_SERIES)
      leaf_series<LD, LEAF_LD>(sX + 16 * rb * LD + 16 * rb, reinterpret_cast<float*>(smem + OFF_LEAF) + warp * 16 * LEAF_LD, lane);
    else
      leaf_substitution<LD>(sX + 16 * rb * LD + 16 * rb, lane);
    __syncthreads();
    merge_level<C, 16>(sX, warp, lane);
    merge_level<C, 32>(sX, warp, lane);

    // ---- 5. store A (the matrix in shared memory is complete: zeros above the diagonal, ones on it)
    if (p.A && rows == C && p.a_box) {
      // a whole chunk: ONE tiled bulk store of 64 tokens x LD floats straight from the matrix (3-D map of A; the padding
      // columns fall outside the tensor and are dropped).  The thread that requests the next G tile issues it and waits
      // until the copy engine has read the matrix, whose space that tile lands in.
      fence_proxy_async();   // the merges' stores become visible to the copy engine
      __syncthreads();
      if (tid == 96) {
        tma_store_3d(&tmA, smem_u32(sX), 0, h, tok0);
        bulk_commit();
        bulk_wait_read();
      }
    } else if (p.A) {
      const size_t a_step = (size_t)(NT / (C / 4)) * p.H * C;
      float* a_dst = p.A + ((size_t)(tok0 + tid / (C / 4)) * p.H + h) * C + 4 * (tid % (C / 4));
#pragma unroll
      for (int m = 0; m < C / 8; ++m) {
        const int e = tid + m * NT;
        const int i = e / (C / 4), j = 4 * (e - i * (C / 4));
        const float4 v = *reinterpret_cast<const float4*>(sX + i * LD + j);
        if (i < rows) *reinterpret_cast<float4*>(a_dst + (size_t)m * a_step) = v;
      }
    }
    if (bad) s_gave_up = 1;
    tc_fence_before();
    __syncthreads();   // the fp32 matrix has been read by everyone: the next G tile may land in its space
    if (s_gave_up) break;   // uniform: every thread reads the flag behind the same barrier
    ph ^= 1;
    if (tid == 96 && has_next) issue_g(nx_tok0, nx_h);
  }
  if (bad || misaligned) atomicMax(p.status, TRI_INV_ERR_DEVICE_TIMEOUT);
  if (s_gave_up) {
    // what may still be in flight: the K tile requested for the next item (the G tile is requested after the exit test)
    if (tid == 64 && k_pending) mbar_wait_bounded(bar_k, ph ^ 1, p.wait_limit_ns);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
}

}  // namespace

// G is KParams::G (an fp32 [B,T,H,d_k] tensor).  Handles bf16 keys with d_k = 128 at C = 64 (here) and C = 128
// (kda_kernel_c128.cu) and the block recursion; anything else is left to the CUDA-core kernel.
cudaError_t launch_kda_tc(const KParams& p, int Cc, cudaStream_t stream, bool* handled) {
  *handled = false;
  if (p.kv_dtype != TRI_INV_BF16 || p.d_k != 128 || (Cc != 64 && Cc != 128)) return cudaSuccess;
  if ((p.method & TRI_INV_METHOD_MASK) != TRI_INV_BLOCK_RECURSIVE) return cudaSuccess;
  if (p.ops & kDoWY) {   // build + inversion + WY in one kernel: C = 64 only (tri_inv_fused_kda makes two launches at C = 128)
    if (Cc != 64 || p.d_v != 128 || !p.V || !p.W || !p.U) return cudaSuccess;
    *handled = true;
    return launch_kda_fused_tc(p, stream);
  }
  *handled = true;
  if (Cc == 128) return launch_kda_tc_c128(p, stream);
  if (p.W) return cudaErrorNotSupported;   // K exp(G) as a by-product is the C = 128 kernel's; nothing asks for it here
  static std::mutex mu;
  static int n_sm_of[64] = {0}, ctas_of[64] = {0};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int n_sm, ctas;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!n_sm_of[dev]) {
      if ((e = cudaFuncSetAttribute(kda_build_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)) != cudaSuccess) return e;
      if ((e = cudaFuncSetAttribute(kda_build_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared)) != cudaSuccess) return e;
      int sms = 0, smem_per_sm = 0;
      if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
      if ((e = cudaDeviceGetAttribute(&smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev)) != cudaSuccess) return e;
      int occ = smem_per_sm / (SMEM_BYTES + 1024);
      occ = occ < CTAS_PER_SM ? occ : CTAS_PER_SM;
      ctas_of[dev] = occ > 0 ? occ : 1;
      n_sm_of[dev] = sms > 0 ? sms : 1;
    }
    n_sm = n_sm_of[dev];
    ctas = ctas_of[dev];
  }
  long long tokens = p.chunk_tab ? (long long)p.T : (long long)p.T * (p.n_chunks / p.chunks_per_seq);
  CUtensorMap tmK, tmG, tmA;
  if (!make_tmap(&tmK, p.K, tokens, p.H, D, C, 2)) return cudaErrorUnknown;
  if (!make_tmap(&tmG, p.G, tokens, p.H, D, C, 4)) return cudaErrorUnknown;
  KParams q = p;
  q.a_box = (p.A && make_tmap_a(&tmA, p.A, tokens, p.H, C, LD)) ? 1 : 0;   // refused: A leaves through ordinary stores
  if (!q.a_box) tmA = tmK;
  long long total = (long long)p.n_chunks * p.H, cap = (long long)n_sm * ctas;
  int grid = (int)(total < cap ? total : cap);
  kda_build_kernel<<<grid, NT, SMEM_BYTES, stream>>>(tmK, tmG, tmA, q);
  return cudaGetLastError();
}

}  // namespace tri_inv
