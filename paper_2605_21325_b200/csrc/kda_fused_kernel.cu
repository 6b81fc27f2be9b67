// Per-channel decay (the KDA row of Table 1), build + inversion + WY factors in one kernel (bf16, d_k = d_v = 128, C = 64,
// block recursion):
//     N_ij = beta_i sum_c K_ic K_jc exp(G_ic - G_jc) (i > j),   A = (I + N)^{-1},
//     W = A diag(beta) (K * exp G),   U = A diag(beta) V.
// The front half is the build kernel's (K+ = K exp(G - G_ref), K- = K exp(G_ref - G), G_ref the chunk's middle row,
// S = K+ K-^T on tcgen05, gate, leaves, merges).  The WY half never forms K exp(G): with e_c = exp(G_ref,c)
//     A diag(beta) (K * exp G) = (A' K+) diag(e),      A' = A diag(beta) (bf16 operand),
// so the W product reads the K+ tile that is in shared memory already (every factor within exp(+-|G over 32 tokens|))
// and its columns are scaled by e on the way out.  U = A' V with the V tile fetched into K-'s space once the Gram
// product has read it.  Both products are tcgen05.mma (M = 64, N = 128) into the same 128 tensor-memory columns, W
// first; W and U leave as bf16 through stmatrix-staged tiles and tiled bulk stores.
//
// Shared memory (74.6 KB, three CTAs per SM): K -> K+ -> staging of W | K- -> V -> staging of half of U | G -> fp32 N / X
// | A' -> staging of the other half of U | beta, e, barriers.  The next item's G tile is requested as soon as the fp32
// matrix has been read (it lands behind the WY products), its K tile when the W stores have read their staging.
// Every mbarrier wait is bounded; on expiry the kernel raises the status word, waits (bounded) for what it has in
// flight, frees its tensor memory and returns.
#include "tc_device.cuh"

namespace tri_inv {
namespace {

constexpr int C = 64, D = 128, NW = 4, NT = 128, LD = C + 4;
constexpr int OFF_K = 0;                      // K tile, then K+, then the staging tiles of W       (16 KB)
constexpr int OFF_KM = 16384;                 // K-, then V, then staging of U's second half        (16 KB)
constexpr int OFF_G = 32768;                  // G tile (4 boxes of 64 rows x 128 B)                (32 KB)
constexpr int OFF_X = OFF_G;                  // fp32 N / X matrix over G                           (17,408 B)
constexpr int OFF_LEAF = OFF_X + C * LD * 4;  // series-leaf scratch, inside the G tile's space
constexpr int LEAF_LD = 20;
constexpr int OFF_AP = 65536;                 // A' = A diag(beta), bf16 K-major swizzled; then staging of U's first half (8 KB)
constexpr int OFF_BETA = OFF_AP + C * C * 2;
constexpr int OFF_ER = OFF_BETA + C * 4;      // exp(G_ref), one per channel
constexpr int OFF_BAR = OFF_ER + D * 4;       // bar_k, bar_mma, bar_g, TMEM slot, bar_v, bar_exit, give-up flag
constexpr int SMEM_BYTES = OFF_BAR + 64;
constexpr int TMEM_COLS = 128;
constexpr int CTAS_PER_SM = 3;
constexpr float kLog2e = 1.4426950408889634f;
static_assert(OFF_LEAF + NW * 16 * LEAF_LD * 4 <= OFF_AP, "leaf scratch must fit behind the fp32 matrix");
static_assert(CTAS_PER_SM * (SMEM_BYTES + 1024) <= 227 * 1024, "three CTAs per SM");

__global__ void __launch_bounds__(NT, CTAS_PER_SM) kda_fused_kernel(const __grid_constant__ CUtensorMap tmK,
                                                                     const __grid_constant__ CUtensorMap tmG,
                                                                     const __grid_constant__ CUtensorMap tmV,
                                                                     const __grid_constant__ CUtensorMap tmW,
                                                                     const __grid_constant__ CUtensorMap tmU,
                                                                     const __grid_constant__ CUtensorMap tmA, KParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  float* sX = reinterpret_cast<float*>(smem + OFF_X);
  float* sBeta = reinterpret_cast<float*>(smem + OFF_BETA);
  float* sER = reinterpret_cast<float*>(smem + OFF_ER);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + OFF_BAR + 24);
  volatile int* const s_gave_up = reinterpret_cast<volatile int*>(smem + OFF_BAR + 48);
  const uint32_t sK = smem_u32(smem + OFF_K), sKm = smem_u32(smem + OFF_KM), sG = smem_u32(smem + OFF_G);
  const uint32_t sAp = smem_u32(smem + OFF_AP);
  const uint32_t bar_k = smem_u32(smem + OFF_BAR), bar_mma = bar_k + 8, bar_g = bar_k + 16, bar_v = bar_k + 32, bar_exit = bar_k + 40;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int rb = warp;                       // M = 64: rows 16q..16q+15 sit in TMEM lanes 32q..32q+15
  const int total = p.n_chunks * p.H;
  const bool misaligned = (sK & 1023u) != 0;
  constexpr int kTidK = 64, kTidG = 96, kTidV = 32;
  int n_k = 0, n_g = 0, n_v = 0;             // copies requested so far by this thread (the give-up path waits for the last)

  auto issue_k = [&](int tok0, int h) {
    ++n_k;
    fence_proxy_async();
    mbar_expect_tx(bar_k, 16384u);
#pragma unroll
    for (int bx = 0; bx < 2; ++bx) tma_load_2d(sK + bx * 8192, &tmK, bar_k, h * D + 64 * bx, tok0);
  };
  auto issue_v = [&](int tok0, int h) {
    ++n_v;
    fence_proxy_async();
    mbar_expect_tx(bar_v, 16384u);
#pragma unroll
    for (int bx = 0; bx < 2; ++bx) tma_load_2d(sKm + bx * 8192, &tmV, bar_v, h * D + 64 * bx, tok0);
  };
  auto issue_g = [&](int tok0, int h) {
    ++n_g;
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
    if (tid == kTidK) { prefetch_tmap(&tmK); mbar_init(bar_k, 1); fence_mbar_init(); if (any) issue_k(tok0, h); }
    if (tid == kTidG) { prefetch_tmap(&tmG); mbar_init(bar_g, 1); fence_mbar_init(); if (any) issue_g(tok0, h); }
    if (tid == kTidV) { prefetch_tmap(&tmV); mbar_init(bar_v, 1); fence_mbar_init(); }
    if (tid == 0) { mbar_init(bar_mma, 1); mbar_init(bar_exit, 1); fence_mbar_init(); *s_gave_up = 0; }
    if (tid == 1) { prefetch_tmap(&tmW); prefetch_tmap(&tmU); }
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
  uint32_t ph = 0, ph_mma = 0;   // K, G and V complete once per item: one parity for the three
  // Give-up protocol as in the main kernel: a thread whose bounded wait runs out remembers it, skips its later waits and
  // finishes the item on whatever data is there; it raises the CTA's flag before the item's last barrier, behind which
  // every thread reads it, so the whole CTA leaves the loop at one place.
  bool bad = false;
  auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
    if (!bad) bad = !mbar_wait_bounded(bar, parity, p.wait_limit_ns);
    return !bad;
  };

  for (int item = blockIdx.x; item < total && !misaligned; item += gridDim.x) {
    int tok0, rows, h;
    locate(p, C, item, tok0, rows, h);
    PHASE_BEGIN();
    const int nx_item = item + gridDim.x;
    const bool has_next = nx_item < total;
    int nx_tok0 = 0, nx_rows = 0, nx_h = 0;
    if (has_next) locate(p, C, nx_item, nx_tok0, nx_rows, nx_h);
    if (tid < C) sBeta[tid] = beta_next;
    if (tid == 1 && has_next) {   // next tiles into L2 now
#pragma unroll
      for (int bx = 0; bx < 2; ++bx) {
        tma_prefetch_l2_2d(&tmK, nx_h * D + 64 * bx, nx_tok0);
        tma_prefetch_l2_2d(&tmV, nx_h * D + 64 * bx, nx_tok0);
      }
#pragma unroll
      for (int bx = 0; bx < 4; ++bx) tma_prefetch_l2_2d(&tmG, nx_h * D + 32 * bx, nx_tok0);
    }

    // ---- 2. K+ = K * 2^x over K, K- = K * 2^-x, x = (G - G_ref) log2(e); rows past the chunk's end are zero
    wait(bar_k, ph);
    wait(bar_g, ph);
    // The item before: its U stores must have read their staging tiles (K-'s and A''s space) before this item writes there;
    // that wait runs behind the copies' above.  The barrier is also where a CTA that gave up leaves, all threads at once.
    if (lane == 0) bulk_wait_read();
    if (bad) *s_gave_up = 1;
    tc_fence_before();
    __syncthreads();
    if (*s_gave_up) break;
    PHASE(0);
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
      for (int q = 0; q < 8; ++q) gr[q] *= kLog2e;
      if ((tid >> 4) == 0) {   // exp(G_ref) of the 128 channels, for W's columns
#pragma unroll
        for (int q = 0; q < 8; ++q) sER[8 * cf + q] = ex2_approx(gr[q]);
      }
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
            const float x0 = fmaf(gv[m][2 * q], kLog2e, -gr[2 * q]), x1 = fmaf(gv[m][2 * q + 1], kLog2e, -gr[2 * q + 1]);
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
    PHASE(1);

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
    if (tid == kTidV && !bad) issue_v(tok0, h);
    PHASE(2);   // K-'s only reader has completed: V comes into its space
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
    PHASE(3);
    if (p.method & TRI_INV_LEAF_SERIES)
      leaf_series<LD, LEAF_LD>(sX + 16 * rb * LD + 16 * rb, reinterpret_cast<float*>(smem + OFF_LEAF) + warp * 16 * LEAF_LD, lane);
    else
      leaf_substitution<LD>(sX + 16 * rb * LD + 16 * rb, lane);
    __syncthreads();
    PHASE(4);
    merge_level<C, 16>(sX, warp, lane);
    merge_level<C, 32>(sX, warp, lane);
    PHASE(5);

    // ---- 5. one pass over the finished matrix (zeros above the diagonal, ones on it): A to global memory, A' = A diag(beta)
    //         as the bf16 K-major swizzled operand of the two products
    // A whole chunk's A leaves as ONE tiled bulk store straight from the matrix (3-D map of A, box of 64 tokens x LD floats:
    // the padding columns fall outside the tensor and are dropped); the thread that requests the next G tile issues it and
    // waits, before that request, until the copy engine has read the matrix.
    const bool a_tma = p.A && rows == C && p.a_box;
    if (a_tma) {
      fence_proxy_async();   // the merges' stores become visible to the copy engine
      __syncthreads();
      if (tid == kTidG) {
        tma_store_3d(&tmA, smem_u32(sX), 0, h, tok0);
        bulk_commit();
      }
    }
    {
      const size_t a_step = (size_t)(NT / (C / 4)) * p.H * C;
      float* a_dst = (p.A && !a_tma) ? p.A + ((size_t)(tok0 + tid / (C / 4)) * p.H + h) * C + 4 * (tid % (C / 4)) : nullptr;
#pragma unroll
      for (int m = 0; m < C / 8; ++m) {
        const int e = tid + m * NT;
        const int i = e / (C / 4), j = 4 * (e - i * (C / 4));
        const float4 v = *reinterpret_cast<const float4*>(sX + i * LD + j);
        if (a_dst && i < rows && TRI_INV_CHECK(p, (long long)tok0 + i < p.n_tokens)) *reinterpret_cast<float4*>(a_dst + (size_t)m * a_step) = v;
        const float4 b = *reinterpret_cast<const float4*>(sBeta + j);
        const uint32_t lo = pack_bf16(v.x * b.x, v.y * b.y), hi = pack_bf16(v.z * b.z, v.w * b.w);
        const uint32_t off = (uint32_t)(i * 128 + ((((j >> 3) ^ (i & 7)) << 4) | ((j & 7) * 2)));
        asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(sAp + off), "r"(lo), "r"(hi) : "memory");
      }
    }
    if (rows < C) {
      // V's rows past the chunk's end belong to another sequence (or to nobody): beta is zero there, but 0 * NaN is not
      wait(bar_v, ph);
      for (int e = tid; e < (C - rows) * 16; e += NT) {
        const int r = rows + (e >> 4), cf = e & 15;
        asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};" ::"r"(sKm + (cf >> 3) * 8192 + r * 128 + ((cf & 7) << 4)), "r"(0u) : "memory");
      }
    }
    fence_proxy_async();   // generic-proxy writes of A' (and V's cleared rows) become visible to the tensor core's reads
    tc_fence_before();
    __syncthreads();       // the fp32 matrix has been read by everyone: the next G tile may land in its space
    if (tid == kTidG) {
      if (a_tma) bulk_wait_read();
      if (has_next && !bad) issue_g(nx_tok0, nx_h);
    }
    PHASE(6);

    // ---- 6. W = (A' K+) diag(exp G_ref), U = A' V: the tiles are the MN-major B operand, 16 tokens per k-step
    constexpr uint32_t idesc_wy = umma_idesc(C, D, 1);
    auto issue_wy = [&](uint32_t b_tile) {
#pragma unroll
      for (int ks = 0; ks < C / 16; ++ks)
        umma_bf16(tmem, umma_desc(sAp + ks * 32, 16, 1024), umma_desc(b_tile + ks * 2048, 8192, 1024), idesc_wy, ks > 0);
      umma_commit(bar_mma);
    };
    if (tid == 0 && !bad) { tc_fence_after(); issue_wy(sK); }
    wait(bar_mma, ph_mma);
    ph_mma ^= 1;
    tc_fence_after();
    PHASE(7);
    const int row0 = 16 * rb;
    const size_t row_stride = (size_t)p.H * D;
    __nv_bfloat16* w_row0 = reinterpret_cast<__nv_bfloat16*>(p.W) + ((size_t)(tok0 + row0) * p.H + h) * D;
    __nv_bfloat16* u_row0 = reinterpret_cast<__nv_bfloat16*>(p.U) + ((size_t)(tok0 + row0) * p.H + h) * D;
    float f0[8][4], f1[8][4];
    tmem_ld_16x64(f0, tmem_rows);
    tmem_ld_16x64(f1, tmem_rows + 64);
    tmem_wait_ld();
    tc_fence_before();
    __syncthreads();   // every warp holds its rows of W in registers: U may overwrite the columns, K+ has been read
    PHASE(8);
    if (tid == 0) {
      if (wait(bar_v, ph)) { tc_fence_after(); issue_wy(sKm); }
    }
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const float2 e0 = *reinterpret_cast<const float2*>(sER + 8 * nt + 2 * t), e1 = *reinterpret_cast<const float2*>(sER + 64 + 8 * nt + 2 * t);
      f0[nt][0] *= e0.x; f0[nt][1] *= e0.y; f0[nt][2] *= e0.x; f0[nt][3] *= e0.y;
      f1[nt][0] *= e1.x; f1[nt][1] *= e1.y; f1[nt][2] *= e1.x; f1[nt][3] *= e1.y;
    }
    // four staging tiles per warp and item, each used once: nothing to wait for before they are written
    store_frag_piece_bf16<3>(f0, sK + warp * 2048, lane, w_row0, row_stride, rows - row0, &tmW, h * D, tok0 + row0);
    store_frag_piece_bf16<3>(f1, sK + 8192 + warp * 2048, lane, w_row0 + 64, row_stride, rows - row0, &tmW, h * D + 64, tok0 + row0);
    PHASE(9);
    wait(bar_mma, ph_mma);
    ph_mma ^= 1;
    tc_fence_after();
    PHASE(10);
    tmem_ld_16x64(f0, tmem_rows);
    tmem_ld_16x64(f1, tmem_rows + 64);
    tmem_wait_ld();
    if (lane == 0) bulk_wait_read();   // this warp's W stores have read their staging tiles in the K tile's space
    tc_fence_before();
    __syncthreads();   // all products done, all accumulators read: tiles, A' and tensor memory are free
    if (tid == kTidK && has_next && !bad) issue_k(nx_tok0, nx_h);
    store_frag_piece_bf16<3>(f0, sAp + warp * 2048, lane, u_row0, row_stride, rows - row0, &tmU, h * D, tok0 + row0);
    store_frag_piece_bf16<3>(f1, sKm + warp * 2048, lane, u_row0 + 64, row_stride, rows - row0, &tmU, h * D + 64, tok0 + row0);
    ph ^= 1;
    PHASE(11);
  }
  if (lane == 0) bulk_wait_read();
  if (bad) *s_gave_up = 1;   // a wait of the last item ran out: nobody has looked at the flag since
  if (bad || misaligned) atomicMax(p.status, TRI_INV_ERR_DEVICE_TIMEOUT);
  __syncthreads();           // every thread has left the item loop
  if (*s_gave_up) {
    // what may still be in flight: the last copy each tile thread requested, and every product issued so far
    if (tid == kTidK && n_k) mbar_wait_bounded(bar_k, (n_k - 1) & 1, p.wait_limit_ns);
    if (tid == kTidG && n_g) mbar_wait_bounded(bar_g, (n_g - 1) & 1, p.wait_limit_ns);
    if (tid == kTidV && n_v) mbar_wait_bounded(bar_v, (n_v - 1) & 1, p.wait_limit_ns);
    if (tid == 0) {
      umma_commit(bar_exit);
      mbar_wait_bounded(bar_exit, 0, p.wait_limit_ns);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
}

}  // namespace

// One launch for tri_inv_fused_kda at C = 64 (bf16, d_k = d_v = 128, block recursion): p.K, p.V, p.G, p.beta in; p.A (optional),
// p.W, p.U out.
cudaError_t launch_kda_fused_tc(const KParams& p, cudaStream_t stream) {
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
      if ((e = cudaFuncSetAttribute(kda_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES)) != cudaSuccess) return e;
      if ((e = cudaFuncSetAttribute(kda_fused_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared)) != cudaSuccess) return e;
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
  const long long tokens = p.chunk_tab ? (long long)p.T : (long long)p.T * (p.n_chunks / p.chunks_per_seq);
  CUtensorMap tmK, tmG, tmV, tmW, tmU, tmA;
  if (!make_tmap(&tmK, p.K, tokens, p.H, D, C, 2)) return cudaErrorUnknown;
  if (!make_tmap(&tmG, p.G, tokens, p.H, D, C, 4)) return cudaErrorUnknown;
  if (!make_tmap(&tmV, p.V, tokens, p.H, D, C, 2)) return cudaErrorUnknown;
  if (!make_tmap(&tmW, p.W, tokens, p.H, D, 16, 2)) return cudaErrorUnknown;
  if (!make_tmap(&tmU, p.U, tokens, p.H, D, 16, 2)) return cudaErrorUnknown;
  KParams q = p;
  q.a_box = (p.A && make_tmap_a(&tmA, p.A, tokens, p.H, C, LD)) ? 1 : 0;   // refused: A leaves through ordinary stores
  if (!q.a_box) tmA = tmK;
  const long long total = (long long)p.n_chunks * p.H, cap = (long long)n_sm * ctas;
  const int grid = (int)(total < cap ? total : cap);
  kda_fused_kernel<<<grid, NT, SMEM_BYTES, stream>>>(tmK, tmG, tmV, tmW, tmU, tmA, q);
  return cudaGetLastError();
}

}  // namespace tri_inv
