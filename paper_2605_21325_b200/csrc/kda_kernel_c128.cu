// Per-channel decay variant (the KDA row of Table 1) at C = 128: the chunk of 128 tokens of kda_kernel.cu's
//     N_ij = beta_i * sum_c K_ic K_jc exp(G_ic - G_jc)   (i > j),      A = (I + N)^{-1},
// for bf16 keys, fp32 G, d = 128, on the tensor cores (build only; with KParams::W also K * exp(G) for the WY step).
//
// The exponent of each difference is never formed per pair: the keys are scaled once per row, K+ = K exp(G - G_ref) on
// the row side and K- = K exp(G_ref - G) on the column side, and the products of the two carry exp(G_i - G_j).  One
// reference row for 128 tokens would double the range each factor has to cover, so every half of the chunk has its
// own, the row in its middle (G_ref0, G_ref1): each factor then stays within exp(+-|G over 32 tokens|) as at C = 64.
// The three blocks of the lower triangle come from two products with M = 64:
//     rows 0..63  :  K+ (ref 0) . [K- (ref 0), tokens 0..63]^T                                   64 x 64
//     rows 64..127:  K+ (ref 1) . [K- (ref 1), tokens 0..63 ; K- (ref 1), tokens 64..127]^T      64 x 128
// (tokens 0..63 against reference 1 have G_ref1 - G_j <= 0, G being non-increasing along a chunk: no overflow).
// An M = 64 accumulator puts rows 16 q .. 16 q + 15 on tensor-memory lanes 32 q .. 32 q + 15, so warp w of eight reads
// the 16 rows it also inverts the diagonal block of.  Gate, 16 x 16 leaves, three merge levels and the store of A follow
// the scalar-gate kernels.  Two CTAs of eight warps per SM: G (64 KB per item in fp32) passes through two 16 KB slots,
// one box of 32 channels at a time, and the fp32 matrix lies over the K- operand and the slots once they are spent.
// Every mbarrier wait is bounded; on expiry the kernel raises the status word, frees its tensor memory and returns.
#include "tc_device.cuh"

namespace tri_inv {
namespace {

constexpr int C = 128, D = 128, NW = 8, NT = 256, LD = C + 4;
constexpr int K_BOX = C * 128;                 // one box of the K tile: 128 rows x 64 features (bf16)
constexpr int KM_ROWS = 192, KM_BOX = KM_ROWS * 128;   // K- operand: tokens 0..63 (ref 0), tokens 0..63 (ref 1), tokens 64..127 (ref 1)
constexpr int G_BOX = C * 128;                 // one box of the G tile: 128 rows x 32 channels (fp32)
constexpr int OFF_K = 0;                       // K tile, then K+                      (32 KB)
constexpr int OFF_KM = OFF_K + 2 * K_BOX;      // K-                                    (48 KB)
constexpr int OFF_G = OFF_KM + 2 * KM_BOX;     // two slots for boxes of G             (2 x 16 KB)
constexpr int OFF_X = OFF_KM;                  // the fp32 N / X matrix (67,584 B) over K- and the slots, once they are spent
constexpr int X_BYTES = C * LD * 4;
constexpr int OFF_LEAF = OFF_X + X_BYTES;      // series-leaf scratch: behind the matrix, in the second slot's space
constexpr int LEAF_LD = 20;
constexpr int OFF_BETA = OFF_G + 2 * G_BOX;
constexpr int OFF_BAR = OFF_BETA + C * 4;      // bar_k, bar_mma, bar_g0, bar_g1, TMEM slot
constexpr int SMEM_BYTES = OFF_BAR + 40;
constexpr int TMEM_COLS = 256;                 // columns 0..63: rows 0..63; columns 64..191: rows 64..127
static_assert(OFF_LEAF + NW * 16 * LEAF_LD * 4 <= OFF_BETA, "the fp32 matrix and the leaf scratch must fit over K- and the slots");
static_assert(OFF_G % 1024 == 0 && OFF_KM % 1024 == 0 && KM_BOX % 1024 == 0, "swizzled tiles start on 1 KiB");
static_assert(2 * (SMEM_BYTES + 1024 + 8) <= 228 * 1024, "two CTAs per SM");

template <bool KG>   // KG: also write K * exp(G) into p.W (the fused call)
__global__ void __launch_bounds__(NT, 2) kda_build_kernel_c128(const __grid_constant__ CUtensorMap tmK,
                                                               const __grid_constant__ CUtensorMap tmG,
                                                               const __grid_constant__ CUtensorMap tmA, KParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  float* sX = reinterpret_cast<float*>(smem + OFF_X);
  float* sBeta = reinterpret_cast<float*>(smem + OFF_BETA);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + 32);
  const uint32_t sK = smem_u32(smem + OFF_K), sKm = smem_u32(smem + OFF_KM), sG = smem_u32(smem + OFF_G);
  const uint32_t bar_k = smem_u32(smem + OFF_BAR), bar_mma = bar_k + 8, bar_g0 = bar_k + 16, bar_g1 = bar_k + 24;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int rb = warp;                         // this warp's 16 rows: half rb >> 2, tensor-memory quadrant rb & 3
  const int total = p.n_chunks * p.H;
  const bool misaligned = (sK & 1023u) != 0;

  auto issue_k = [&](int tok0, int h) {
    fence_proxy_async();
    mbar_expect_tx(bar_k, 2u * K_BOX);
#pragma unroll
    for (int bx = 0; bx < 2; ++bx) tma_load_2d(sK + bx * K_BOX, &tmK, bar_k, h * D + 64 * bx, tok0);
  };
  // box bx of G (channels 32 bx .. + 31) into slot bx & 1
  auto issue_g = [&](int tok0, int h, int bx) {
    const uint32_t bar = (bx & 1) ? bar_g1 : bar_g0;
    fence_proxy_async();
    mbar_expect_tx(bar, (uint32_t)G_BOX);
    tma_load_2d(sG + (bx & 1) * G_BOX, &tmG, bar, h * D + 32 * bx, tok0);
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
    if (tid == 96) {
      prefetch_tmap(&tmG); mbar_init(bar_g0, 1); mbar_init(bar_g1, 1); fence_mbar_init();
      if (any) { issue_g(tok0, h, 0); issue_g(tok0, h, 1); }
    }
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
  const uint32_t tmem_rows = tmem + ((32u * (warp & 3)) << 16);
  uint32_t ph = 0, ph_mma = 0;   // K completes once per item; each slot of G twice (parities 0, 1 within every item)
  // Give-up protocol as in the other kernels: a thread whose bounded wait runs out remembers it, skips its later waits
  // and finishes the item on whatever data is there; it raises the CTA's flag before the item's last barrier, behind
  // which every thread reads it, so the whole CTA leaves the loop at one place.
  int* const gave_up = reinterpret_cast<int*>(smem + OFF_BAR + 36);   // (in the dynamic block: a static one would cost 1 KiB)
  bool bad = false;
  auto wait = [&](uint32_t bar, uint32_t parity) {
    if (!bad) bad = !mbar_wait_bounded(bar, parity, p.wait_limit_ns);
  };
  if (tid == 0) *gave_up = 0;   // read only behind later barriers
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

    // ---- 2. K+ = K * 2^x over K, K- = K * 2^-x, x = (G - G_ref) log2(e), G_ref the middle row of the row's half of
    // the chunk; tokens 0..63 also against the second half's reference.  Rows past the chunk's end are zero.
    wait(bar_k, ph);
    const int rows0 = rows < 64 ? rows : 64, rows1 = rows - rows0;
    const int rref0 = rows0 >> 1, rref1 = 64 + (rows1 >> 1);   // (rref1 is used only where rows1 > 0)
    // G comes through two slots, a box of 32 channels at a time: boxes 0 and 1 were requested before the item, boxes
    // 2 and 3 follow into the slots that boxes 0 and 1 leave (behind a barrier: every thread has read the slot).
#pragma unroll 1
    for (int bx = 0; bx < 4; ++bx) {
    wait((bx & 1) ? bar_g1 : bar_g0, (uint32_t)(bx >> 1));
    {
      // Branch-free (rows past the chunk's end are read like the others and replaced by zeros) and loads first: the
      // thread's 8 channels are the same for its two rows (r and r + 64), so the two reference rows are read once per box.
      constexpr float kL2e = 1.4426950408889634f;
      const int cf = 4 * bx + (tid & 3);                  // 16-byte chunk of 8 features (four per box of G)
      const int q0 = 2 * (tid & 3);                       // first of the two float4 of G for these 8 channels
      const uint32_t gbox = sG + (bx & 1) * G_BOX;
      float gr0[8], gr1[8];
#pragma unroll
      for (int hq = 0; hq < 2; ++hq) {
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(gr0[4 * hq]), "=f"(gr0[4 * hq + 1]), "=f"(gr0[4 * hq + 2]), "=f"(gr0[4 * hq + 3])
                     : "r"(gbox + rref0 * 128 + (((q0 + hq) ^ (rref0 & 7)) << 4)));
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(gr1[4 * hq]), "=f"(gr1[4 * hq + 1]), "=f"(gr1[4 * hq + 2]), "=f"(gr1[4 * hq + 3])
                     : "r"(gbox + rref1 * 128 + (((q0 + hq) ^ (rref1 & 7)) << 4)));
      }
      uint4 kv[2];
      float gv[2][8];
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        const int r = (tid >> 2) + 64 * m;
        const uint32_t sw = (uint32_t)((((cf & 7) ^ (r & 7)) << 4));   // (rows r, r + 64 and r + 128 share r & 7)
        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(kv[m].x), "=r"(kv[m].y), "=r"(kv[m].z), "=r"(kv[m].w)
                     : "r"(sK + (uint32_t)((cf >> 3) * K_BOX + r * 128) + sw));
#pragma unroll
        for (int hq = 0; hq < 2; ++hq)
          asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(gv[m][4 * hq]), "=f"(gv[m][4 * hq + 1]), "=f"(gv[m][4 * hq + 2]), "=f"(gv[m][4 * hq + 3])
                       : "r"(gbox + r * 128 + (((q0 + hq) ^ (r & 7)) << 4)));
      }
#pragma unroll
      for (int q = 0; q < 8; ++q) { gr0[q] *= kL2e; gr1[q] *= kL2e; }
#pragma unroll
      for (int m = 0; m < 2; ++m) {
        const int r = (tid >> 2) + 64 * m;                // m is the row's half of the chunk
        const uint32_t sw = (uint32_t)((((cf & 7) ^ (r & 7)) << 4));
        const uint32_t koff = (uint32_t)((cf >> 3) * K_BOX + r * 128) + sw;
        const uint32_t moff = (uint32_t)((cf >> 3) * KM_BOX + (m ? r + 64 : r) * 128) + sw;   // K- against the row's own reference
        const bool live = r < rows;
        const bool cross = live && rows1 > 0;             // m = 0: a token of the first half that the second half's rows see
        uint4 kp, km, km1, kg;                            // kg = K * exp(G): the key operand of the WY step that follows (fused call)
        const uint32_t* kw = reinterpret_cast<const uint32_t*>(&kv[m]);
        uint32_t* pw = reinterpret_cast<uint32_t*>(&kp);
        uint32_t* mw = reinterpret_cast<uint32_t*>(&km);
        uint32_t* xw = reinterpret_cast<uint32_t*>(&km1);
        uint32_t* gw = reinterpret_cast<uint32_t*>(&kg);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float2 kf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kw[q]));
          const float ga = gv[m][2 * q] * kL2e, gb = gv[m][2 * q + 1] * kL2e;
          const float x0 = ga - (m ? gr1[2 * q] : gr0[2 * q]), x1 = gb - (m ? gr1[2 * q + 1] : gr0[2 * q + 1]);
          const uint32_t vp = pack_bf16(kf.x * ex2_approx(x0), kf.y * ex2_approx(x1));
          const uint32_t vm = pack_bf16(kf.x * ex2_approx(-x0), kf.y * ex2_approx(-x1));
          pw[q] = live ? vp : 0u;
          mw[q] = live ? vm : 0u;
          if (m == 0) {
            const uint32_t vx = pack_bf16(kf.x * ex2_approx(gr1[2 * q] - ga), kf.y * ex2_approx(gr1[2 * q + 1] - gb));
            xw[q] = cross ? vx : 0u;
          }
          if constexpr (KG) gw[q] = pack_bf16(kf.x * ex2_approx(ga), kf.y * ex2_approx(gb));
        }
        // 16 consecutive threads cover the 256 contiguous bytes of one token's keys of this head
        if constexpr (KG) {
          if (live) *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.W) + ((size_t)(tok0 + r) * p.H + h) * D + 8 * cf) = kg;
        }
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(sK + koff), "r"(kp.x), "r"(kp.y), "r"(kp.z), "r"(kp.w) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(sKm + moff), "r"(km.x), "r"(km.y), "r"(km.z), "r"(km.w) : "memory");
        if (m == 0) asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(sKm + moff + 64 * 128), "r"(km1.x), "r"(km1.y), "r"(km1.z), "r"(km1.w) : "memory");
      }
    }
    if (bx < 2) {
      __syncthreads();
      if (tid == 96 && !bad) issue_g(tok0, h, bx + 2);
    }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();

    // ---- 3. the two products (one thread): rows 0..63 against tokens 0..63, rows 64..127 against all tokens
    // (self-test, kTestStall: thread block 0 leaves out the products of its first item, so that the wait below runs out)
    if (tid == 0 && !((p.ops & kTestStall) && item == 0)) {
      tc_fence_after();
      constexpr uint32_t idesc0 = umma_idesc(64, 64, 0), idesc1 = umma_idesc(64, 128, 0);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const uint32_t ko = (ks >> 2) * K_BOX + (ks & 3) * 32, mo = (ks >> 2) * KM_BOX + (ks & 3) * 32;
        umma_bf16(tmem, umma_desc(sK + ko, 16, 1024), umma_desc(sKm + mo, 16, 1024), idesc0, ks > 0);
      }
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const uint32_t ko = (ks >> 2) * K_BOX + (ks & 3) * 32, mo = (ks >> 2) * KM_BOX + (ks & 3) * 32;
        umma_bf16(tmem + 64, umma_desc(sK + 64 * 128 + ko, 16, 1024), umma_desc(sKm + 64 * 128 + mo, 16, 1024), idesc1, ks > 0);
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
      const bool upper = rb >= 4;   // rows 64..127: 128 columns of products; rows 0..63: 64, the rest of the row is zero
#pragma unroll
      for (int cb = 0; cb < 2; ++cb) {
        float sacc[8][4];
        if (upper || cb == 0) {
          tmem_ld_16x64(sacc, tmem_rows + (upper ? 64 + 64 * cb : 0));
          tmem_wait_ld();
        }
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          const int c = 64 * cb + 8 * nt + 2 * t;
          float2 va = make_float2(0.f, 0.f), vb = va;
          if ((upper || cb == 0) && (8 * cb + nt) / 2 <= rb) {
            va.x = (c < ra) ? beta_a * sacc[nt][0] : 0.f;
            va.y = (c + 1 < ra) ? beta_a * sacc[nt][1] : 0.f;
            vb.x = (c < rbw) ? beta_b * sacc[nt][2] : 0.f;
            vb.y = (c + 1 < rbw) ? beta_b * sacc[nt][3] : 0.f;
          }
          *reinterpret_cast<float2*>(sX + ra * LD + c) = va;
          *reinterpret_cast<float2*>(sX + rbw * LD + c) = vb;
        }
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
    merge_level<C, 64>(sX, warp, lane);

    // ---- 5. store A (the matrix in shared memory is complete: zeros above the diagonal, ones on it)
    if (p.A && rows == C && p.a_box) {
      // a whole chunk: ONE tiled bulk store of 128 tokens x LD floats straight from the matrix (3-D map of A; the padding
      // columns fall outside the tensor and are dropped).  The thread that requests the next G boxes issues it and waits
      // until the copy engine has read the matrix, whose space those boxes land in.
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
#pragma unroll 4
      for (int m = 0; m < C * C / 4 / NT; ++m) {
        const int e = tid + m * NT;
        const int i = e / (C / 4), j = 4 * (e - i * (C / 4));
        const float4 v = *reinterpret_cast<const float4*>(sX + i * LD + j);
        if (i < rows) *reinterpret_cast<float4*>(a_dst + (size_t)m * a_step) = v;
      }
    }
    if (bad) *gave_up = 1;
    tc_fence_before();
    __syncthreads();   // the fp32 matrix has been read by everyone: the next G tile may land in its space
    if (*gave_up) break;   // uniform: every thread reads the flag behind the same barrier
    ph ^= 1;
    if (tid == 96 && has_next) { issue_g(nx_tok0, nx_h, 0); issue_g(nx_tok0, nx_h, 1); }
  }
  if (bad || misaligned) atomicMax(p.status, TRI_INV_ERR_DEVICE_TIMEOUT);
  if (*gave_up) {
    // what may still be in flight: the K tile requested for the next item (the G tile is requested after the exit test)
    if (tid == 64 && k_pending) mbar_wait_bounded(bar_k, ph ^ 1, p.wait_limit_ns);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
}

}  // namespace

// G is KParams::G (an fp32 [B,T,H,d_k] tensor): bf16 keys with d_k = 128 at C = 128, block recursion.
cudaError_t launch_kda_tc_c128(const KParams& p, cudaStream_t stream) {
  static std::mutex mu;
  static int n_sm_of[64] = {0};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int n_sm;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!n_sm_of[dev]) {
      if ((e = cudaFuncSetAttribute(kda_build_kernel_c128<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)) != cudaSuccess) return e;
      if ((e = cudaFuncSetAttribute(kda_build_kernel_c128<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)) != cudaSuccess) return e;
      if ((e = cudaFuncSetAttribute(kda_build_kernel_c128<false>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared)) != cudaSuccess) return e;
      if ((e = cudaFuncSetAttribute(kda_build_kernel_c128<true>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared)) != cudaSuccess) return e;
      int sms = 0;
      if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
      n_sm_of[dev] = sms > 0 ? sms : 1;
    }
    n_sm = n_sm_of[dev];
  }
  long long tokens = p.chunk_tab ? (long long)p.T : (long long)p.T * (p.n_chunks / p.chunks_per_seq);
  CUtensorMap tmK, tmG, tmA;
  if (!make_tmap(&tmK, p.K, tokens, p.H, D, C, 2)) return cudaErrorUnknown;
  if (!make_tmap(&tmG, p.G, tokens, p.H, D, C, 4)) return cudaErrorUnknown;
  KParams q = p;
  q.a_box = (p.A && make_tmap_a(&tmA, p.A, tokens, p.H, C, LD)) ? 1 : 0;   // refused: A leaves through ordinary stores
  if (!q.a_box) tmA = tmK;
  long long total = (long long)p.n_chunks * p.H;
  const long long cap = 2LL * n_sm;   // two CTAs per SM
  int grid = (int)(total < cap ? total : cap);
  if (grid == 0) return cudaSuccess;
  if (p.W) kda_build_kernel_c128<true><<<grid, NT, SMEM_BYTES, stream>>>(tmK, tmG, tmA, q);
  else kda_build_kernel_c128<false><<<grid, NT, SMEM_BYTES, stream>>>(tmK, tmG, tmA, q);
  return cudaGetLastError();
}

}  // namespace tri_inv
