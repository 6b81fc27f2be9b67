// Tensor-core kernel for bf16 keys/values, d = 128, C = 64 or 128 (sm_100a).
//
// One CTA works on one chunk matrix at a time (first two items fixed, later ones from a device
// counter), one warp per 16 rows, 4 CTAs per SM at C = 64.  Per item:
//   1. TMA (cp.async.bulk.tensor, 128-byte swizzle) stages the C x d tiles of K and V in shared
//      memory on separate mbarriers; the next item's tiles are prefetched into L2 an item ahead and
//      copied as soon as a buffer's last reader has finished; beta and g travel one item ahead in a register.
//   2. Gram S = K K^T: tcgen05.mma (kind::f16, bf16 operands straight from the TMA-written tile,
//      fp32 accumulator in tensor memory), issued by one thread, completion through an mbarrier.
//   3. Each warp reads its 16 rows of S from tensor memory (tcgen05.ld 16x256b: the m16n8 accumulator
//      fragment layout), applies gate + strict-lower mask, writes N to shared memory in fp32.
//   4. Block recursion (Sec. 3.3): 16x16 leaves by forward substitution, one lane per column (Sec. 3.1),
//      or by the product series on the leaf (Alg. 2); merges X21 = -(X22 N21) X11 for b = 16, 32, (64)
//      as TF32 m16n8k8 MMAs on fp32 data in shared memory.
//      Product-series variant (Alg. 5): Y.Y and X.Y as tcgen05.mma kind::tf32 on fp32 operands kept in
//      shared memory, accumulators in tensor memory, log2(C) round trips.
//   5. A' = A diag(beta) is written as a bf16 K-major swizzled operand over the fp32 matrix's space;
//      W = A' K and U = A' V are tcgen05.mma with the K / V tiles as the MN-major B operand; A goes to
//      global memory with 16-byte coalesced stores while the W product runs.
//   6. W and U come back from tensor memory, are packed to bf16, transposed through a per-warp swizzled
//      staging tile with stmatrix and leave as 16-byte stores covering 128 contiguous bytes per row.
// Every mbarrier wait is bounded; on expiry the kernel raises the status word, frees its tensor
// memory and returns.
#pragma once
#include <cuda.h>

#include <cstdlib>
#include <mutex>

#include "tc_device.cuh"

namespace tri_inv {
namespace {

// ------------------------------------------------------------------------------------------ layout
template <int C, int D, bool SER, bool BO = false, bool REF = false, bool H16 = false>
struct Cfg {
  // BO: build-only specialisation (tri_inv_build at C = 64): no V tile, no WY operand or staging, 64 TMEM
  // columns, so six CTAs fit on an SM instead of four.
  static_assert(!BO || (C == 64 && !SER), "the build-only variant exists for the C = 64 block recursion");
  static constexpr int NW = C / 16;             // warps, one per 16 rows
  static constexpr int NT = NW * 32;
  static constexpr int LD = C + 4;              // fp32 row length of the N/X matrix (LD % 16 == 4)
  static constexpr int NBOX = D / 64;           // TMA boxes per tile: 64 features (128 B) wide
  static constexpr int BOX_BYTES = C * 128;
  static constexpr int TILE_BYTES = NBOX * BOX_BYTES;
  // Block recursion at C = 128: the K / V tiles share the space of the fp32 N/X matrix (K is only needed
  // for the Gram product before N is written, and both tiles are fetched again, from L2, for the WY step),
  // which brings the CTA under half an SM's shared memory: two CTAs per SM instead of one.
  // REF (one step of iterative refinement after the recursion): N is kept, in fp32, where the K and V tiles are
  // (the Gram product is done with K by then), so both tiles are fetched again afterwards as in the series variant.
  static_assert(!REF || (!SER && !BO), "refinement follows the block recursion of the full kernel");
  // H16 (product series with fp16 operands): Y and X are half the size and one copy of Y serves as both operands, so
  // they fit in the space of the fp32 matrix and the series needs none of the tiles' space: the layout is the
  // block recursion's (tiles kept at C = 64, aliased with the matrix at C = 128), not the fp32 series'.
  static_assert(!H16 || SER, "fp16 operands are a variant of the product series");
  static constexpr bool ALIAS = (C == 128) && (!SER || H16) && !REF;
  static constexpr bool RELOAD = (SER && !H16) || ALIAS || REF;    // K (and V) are requested after the inversion
  static constexpr int OFF_K = 0;
  static constexpr int OFF_V = TILE_BYTES;
  static constexpr int X_BYTES = C * LD * 4;
  static constexpr int TILES_BYTES = (REF && X_BYTES > 2 * TILE_BYTES) ? (X_BYTES + 1023) / 1024 * 1024 : 2 * TILE_BYTES;  // REF: room for N
  static constexpr int OFF_X = ALIAS ? 0 : (BO ? TILE_BYTES : TILES_BYTES);
  // A' (bf16, C x C) and the per-warp 2 KiB output staging tiles: inside the N/X matrix's space once it has
  // been read (A' first, staging behind it), or, with ALIAS, in a region of their own where the staging
  // reuses A' after the WY products have completed.
  static constexpr int OFF_AP = ALIAS ? (X_BYTES + 1023) / 1024 * 1024 : OFF_X;
  static constexpr int OFF_STAGE = ALIAS ? OFF_AP : OFF_AP + C * C * 2;
  static_assert(ALIAS || C * C * 2 + NW * 2048 <= X_BYTES, "A' and staging must fit in the N/X matrix's space");
  static_assert(NW * 2048 <= C * C * 2, "staging must fit in A'");
  static constexpr int OFF_BETA = ALIAS ? OFF_AP + C * C * 2 : OFF_X + X_BYTES;
  static constexpr int OFF_G = OFF_BETA + C * 4;
  static constexpr int OFF_BAR = OFF_G + C * 4;
  static constexpr int LEAF_LD = 20;             // per-warp 16 x 16 fp32 scratch of the series leaf
  static constexpr int LEAF_BYTES = NW * 16 * LEAF_LD * 4;
  // 64 bytes of control words: three mbarriers, the TMEM base-address slot, the next-item slot, the exit
  // mbarrier and the three give-up flags; then the leaf scratch (inside A' with ALIAS)
  static constexpr int OFF_LEAF = ALIAS ? OFF_AP : (BO ? OFF_K : OFF_BAR + 64);  // BO: in the K tile, dead after the Gram product
  // raw front end: 1 / |k_i| per row, and the per-warp totals of the log-decay scan
  static constexpr int OFF_R = (ALIAS || BO) ? OFF_BAR + 64 : OFF_LEAF + LEAF_BYTES;
  static constexpr int END_PLAIN = OFF_R + C * 4 + 32;
  // product-series variant at C = 128: X needs a buffer of its own (at C = 64 it fits where the V tile was)
  static constexpr int OFF_XS = (END_PLAIN + 1023) / 1024 * 1024;
  static constexpr int BYTES = (SER && !H16 && C == 128) ? OFF_XS + C * C * 4 : END_PLAIN;
  static_assert(!H16 || 2 * C * C * 2 <= X_BYTES, "the two fp16 operands live in the fp32 matrix's space");
  static constexpr int SMEM = BYTES;
  static constexpr int CTAS_PER_SM = (C == 64) ? (BO ? 6 : 4) : (ALIAS ? 2 : 1);
  static constexpr int TMEM_COLS = (C == 64) ? (BO ? 64 : 128) : 256;
};

// Byte offset of the 16-byte chunk holding features [f, f+8) of row r inside a swizzled tile.
// VAR specialises two run-time switches away so that the common case carries less code (the instruction cache is shared
// by four CTAs in different phases): 0 = fused / build call with substitution leaves, 1 = with series leaves,
// 2 = tri_inv_wy (A read from memory), 3 = decided at run time.
template <int C, int D, bool SER, bool RAW, bool BO, bool REF, bool H16, int VAR>
__global__ void __launch_bounds__(Cfg<C, D, SER, BO, REF, H16>::NT, Cfg<C, D, SER, BO, REF, H16>::CTAS_PER_SM) tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmU,
                                                                             const __grid_constant__ CUtensorMap tmV, const __grid_constant__ KParams p) {
  using cfg = Cfg<C, D, SER, BO, REF, H16>;
  static_assert(D == 128 || (D == 64 && C == 64 && !SER && !RAW && !REF && !H16),
                "tiles are two 64-feature boxes wide; one box only for the plain block recursion at C = 64");
  constexpr int LD = cfg::LD;
  constexpr int TMEM_COLS = cfg::TMEM_COLS;
  extern __shared__ __align__(1024) uint8_t smem[];  // swizzled tiles need a 1024-byte aligned base
  float* sX = reinterpret_cast<float*>(smem + cfg::OFF_X);
  float* sN = reinterpret_cast<float*>(smem + cfg::OFF_K);          // REF only: N kept for the refinement step, where the tiles were
  float* sBeta = reinterpret_cast<float*>(smem + cfg::OFF_BETA);
  float* sG = reinterpret_cast<float*>(smem + cfg::OFF_G);
  float* sR = reinterpret_cast<float*>(smem + cfg::OFF_R);          // raw front end: 1 / |k_i|
  float* sScan = sR + C;                                            // raw front end: scan totals per warp
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + cfg::OFF_BAR + 24);
  volatile int* s_next_item = reinterpret_cast<volatile int*>(smem + cfg::OFF_BAR + 28);
  const uint32_t sK = smem_u32(smem + cfg::OFF_K);
  const uint32_t sV = smem_u32(smem + cfg::OFF_V);
  const uint32_t sAp = smem_u32(smem + cfg::OFF_AP);  // A' = A diag(beta), bf16 K-major swizzled operand
  const uint32_t bar_k = smem_u32(smem + cfg::OFF_BAR);  // K tile landed
  const uint32_t bar_mma = bar_k + 8;                    // a batch of MMAs completed
  const uint32_t bar_v = bar_k + 16;                     // V tile landed
  const uint32_t bar_exit = bar_k + 32;                  // give-up path only: every product issued so far has retired
  const uint32_t bar_mma_u = bar_k + 48;                 // C = 128: the U product, committed right behind W (a barrier of its own:
                                                         // two phases of one barrier must not complete before the first is seen)
  // Give-up protocol.  A thread whose bounded wait runs out remembers it ("bad"), skips its later waits, and
  // carries on with the item on whatever data is there (all indices come from the item number, never from
  // data).  It raises the CTA's flag in shared memory just before the barrier at the top of the next item;
  // behind that barrier every thread reads the flag and the whole CTA leaves the loop together, so no thread is
  // left at a barrier or using tensor memory while another frees it.
  volatile int* const s_gave_up = reinterpret_cast<volatile int*>(smem + cfg::OFF_BAR + 40);
  bool bad = false;
  uint32_t n_issue = 0;  // copies requested by this thread (the K thread: K tiles, the V thread: V tiles): the exit path waits for the last one
  auto wait = [&](uint32_t bar, uint32_t parity) -> bool {
    if (bad) return false;
#ifdef TRI_INV_DEBUG
    // mbarrier bookkeeping, checked by the thread that requests the copies: the phase it waits for must be the one its
    // most recent request completes
    if ((bar == bar_k && threadIdx.x == 64) || (bar == bar_v && threadIdx.x == 96))
      TRI_INV_CHECK(p, n_issue > 0 && ((n_issue - 1) & 1u) == parity);
#endif
    bad = !mbar_wait_bounded(bar, parity, p.wait_limit_ns);
    return !bad;
  };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  CTA_MARK(0);
  CTA_MARK(3);
  // Row block of this warp.  TMEM lanes are reachable only from the warp whose id % 4 matches
  // the 32-lane quadrant: M = 64 puts rows 16q..16q+15 in lanes 32q..32q+15, M = 128 puts row i in lane i.
  const int rb = (C == 64) ? warp : 2 * (warp & 3) + (warp >> 2);
  const uint32_t lane_base = (C == 64) ? 32u * warp : 16u * rb;
  const bool do_wy = !BO && (p.ops & kDoWY) != 0;
  const bool need_v = do_wy && p.V != nullptr;
  const bool load_a = VAR == 3 ? (p.ops & kLoadA) != 0 : VAR == 2;
  const bool leaf_series_on = VAR == 3 ? (p.method & TRI_INV_LEAF_SERIES) != 0 : VAR == 1;
  // RAW compiles in the code that rewrites the K tile in shared memory before the WY step and the per-row
  // factors of the gate.  Two run-time uses: the front end (sigmoid, log-sigmoid + chunk cumsum, key
  // normalisation: kRaw) and the decay-weighted W (rows of K times exp(g_i): kWDecay).
  constexpr bool raw = RAW;
  const bool front = RAW && (p.ops & kRaw) != 0;
  const bool wdecay = RAW && (p.ops & kWDecay) != 0;
  // Comba row of Table 1 (decay matrix A^{i-1/j}): row i of N, and row i of the decay-weighted W, take the cumulative
  // log-decay of the token before it (the first row of a chunk has nothing below the diagonal and weight 1)
  const int gshift = (p.method & TRI_INV_GATE_SHIFTED) ? 1 : 0;
  const int total = p.n_chunks * p.H;

  // Thread 0 requests the tiles of an item; K and V complete on separate barriers so that the Gram
  // product can start on K alone and each buffer is refilled as soon as its last reader is done.
  // The tiles of an item are requested by single threads of different warps, so that no warp carries
  // all of the control work: K by warp 2, V by warp 3, the L2 prefetch by warp 1, the MMAs by warp 0.
  // K and V complete on separate barriers: the Gram product starts on K alone, and each buffer is
  // refilled as soon as its last reader is done.
  constexpr int kTidL2 = 32, kTidK = 64, kTidV = 96;
  auto issue_k = [&](int tok0, int h) {
    if (bad) return;
    ++n_issue;
#ifdef TRI_INV_DEBUG
    if (!TRI_INV_CHECK(p, tok0 >= 0 && tok0 < p.n_tokens && h >= 0 && h < p.H)) return;
#endif
    fence_proxy_async();
    mbar_expect_tx(bar_k, (uint32_t)cfg::TILE_BYTES);
#pragma unroll
    for (int bx = 0; bx < cfg::NBOX; ++bx) tma_load_2d(sK + bx * cfg::BOX_BYTES, &tmK, bar_k, h * D + 64 * bx, tok0);
  };
  auto issue_v = [&](int tok0, int h) {
    if (bad) return;
    ++n_issue;
#ifdef TRI_INV_DEBUG
    if (!TRI_INV_CHECK(p, tok0 >= 0 && tok0 < p.n_tokens && h >= 0 && h < p.H)) return;
#endif
    fence_proxy_async();
    mbar_expect_tx(bar_v, (uint32_t)cfg::TILE_BYTES);
#pragma unroll
    for (int bx = 0; bx < cfg::NBOX; ++bx) tma_load_2d(sV + bx * cfg::BOX_BYTES, &tmV, bar_v, h * D + 64 * bx, tok0);
  };
  // beta (threads 0..C-1) and g (threads C..2C-1) of an item, fetched one item ahead into a register
  auto fetch_bg = [&](int tok0, int rows, int h) -> float {
    const int i = tid < C ? tid : tid - C;
    const float* src = tid < C ? p.beta : p.g;
    return (i < rows && src && TRI_INV_CHECK(p, (long long)tok0 + i < p.n_tokens)) ? src[(size_t)(tok0 + i) * p.H + h] : 0.f;
  };
  // Prologue.  The threads that own the K and V barriers initialise them and request the first
  // item's tiles at once, so that the copies run while tensor memory is being allocated.
  const bool misaligned = (sK & 1023u) != 0;  // never expected; the swizzle pattern would not match the copies
  float bg_next = 0.f;
  {
    int tok0 = 0, rows = 0, h = 0;
    const bool any = (int)blockIdx.x < total && !misaligned;
    if (any) locate(p, C, blockIdx.x, tok0, rows, h);
    // the give-up flag is zeroed here; nobody can raise it before the barrier that ends the prologue
    if (tid == kTidK) {
      *s_gave_up = 0;
      prefetch_tmap(&tmK);
      mbar_init(bar_k, 1);
      fence_mbar_init();
      if (any && !(cfg::ALIAS && load_a)) issue_k(tok0, h);  // with ALIAS, tri_inv_wy fills the matrix first and fetches K later
    }
    if (tid == kTidV) {
      if (need_v) prefetch_tmap(&tmV);
      mbar_init(bar_v, 1);
      fence_mbar_init();
      if (any && need_v && !cfg::RELOAD) issue_v(tok0, h);  // otherwise V is requested after the inversion
    }
    if (tid == 0) {
      mbar_init(bar_mma, 1);
      mbar_init(bar_mma_u, 1);
      mbar_init(bar_exit, 1);
      fence_mbar_init();
    }
    if (any) bg_next = fetch_bg(tok0, rows, h);
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_rows = tmem + (lane_base << 16);
  uint32_t ph_k = 0, ph_v = 0, ph_mma = 0, ph_u = 0;  // parities of the next completion to wait for on each barrier

  // Gram S = K K^T: D/16 MMAs of C x C x 16 into the first C columns of tensor memory (thread 0)
  auto issue_gram = [&]() {
    constexpr uint32_t idesc = umma_idesc(C, C, 0);
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      const uint64_t dk = umma_desc(sK + (ks >> 2) * cfg::BOX_BYTES + (ks & 3) * 32, 16, 1024);
      umma_bf16(tmem, dk, dk, idesc, ks > 0);
    }
    umma_commit(bar_mma);
  };
  bool gram_early = false;  // thread 0: the Gram product of the coming item was already issued at the end of the last one
  // Work distribution: the first two items of a CTA are fixed (blockIdx, blockIdx + grid), every
  // later one comes from a device counter, fetched one item ahead of its use so that prefetches
  // know their target.  SMs that run faster simply take more items.  A launch without a counter
  // pair (p.work_counter == nullptr) walks its items with the fixed stride gridDim.x.
  int item = blockIdx.x, nx_item = blockIdx.x + gridDim.x;
  while (item < total && !misaligned) {
    int tok0, rows, h;
    locate(p, C, item, tok0, rows, h);
    // bounds-checking build: an item outside the tensors is reduced to no rows (nothing of it is then stored)
    if (!TRI_INV_CHECK(p, rows >= 1 && rows <= C && tok0 >= 0 && (long long)tok0 + rows <= p.n_tokens && h >= 0 && h < p.H)) { tok0 = 0; rows = 0; h = 0; }
    PHASE_BEGIN();

    // ---- 1. beta, g were fetched during the previous item (sBeta and sG are adjacent: one store each)
    // g is kept multiplied by log2(e) so that the gate can use ex2 directly
    if (!raw || !front) {
      sBeta[tid] = bg_next * (tid < C ? 1.f : 1.4426950408889634f);
    } else {
      // raw front end: beta = sigmoid(logit); g = cumulative sum over the chunk of log sigmoid(gate logit)
      const int i = tid < C ? tid : tid - C;
      const size_t gi = (size_t)(tok0 + i) * p.H + h;
      if (tid < C) {
        const float b = (i < rows) ? 1.f / (1.f + __expf(-bg_next)) : 0.f;
        sBeta[i] = b;
        if (p.beta_out && i < rows) p.beta_out[gi] = b;
      }
      float a = 0.f;
      if (tid >= C && i < rows) a = fminf(bg_next, 0.f) - log1pf(__expf(-fabsf(bg_next)));
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const float y = __shfl_up_sync(0xffffffffu, a, off);
        if (lane >= off) a += y;
      }
      if (tid >= C && lane == 31) sScan[warp - cfg::NW / 2] = a;
      __syncthreads();
      if (tid >= C) {
        for (int w = 0; w < warp - cfg::NW / 2; ++w) a += sScan[w];
        sG[i] = a * 1.4426950408889634f;
        if (p.g_out && i < rows) p.g_out[gi] = a;
      }
    }
    const bool has_next = nx_item < total;
    int nx_tok0 = 0, nx_rows = 0, nx_h = 0;   // the next item of this CTA
    if (has_next) locate(p, C, nx_item, nx_tok0, nx_rows, nx_h);
    if (has_next) {
      // next item's beta / g element of this thread: into L2 now, into a register later
      const int i = tid < C ? tid : tid - C;
      const float* src = tid < C ? p.beta : p.g;
      if (i < nx_rows && src) asm volatile("prefetch.global.L2 [%0];" ::"l"(src + (size_t)(nx_tok0 + i) * p.H + nx_h));
    }
    if (tid == kTidL2 && has_next) {
      // pull the next tiles into L2 now; the copies into shared memory follow when the buffers are free
#pragma unroll
      for (int bx = 0; bx < cfg::NBOX; ++bx) {
        tma_prefetch_l2_2d(&tmK, nx_h * D + 64 * bx, nx_tok0);
        if (need_v) tma_prefetch_l2_2d(&tmV, nx_h * D + 64 * bx, nx_tok0);
      }
    }
    if (load_a) {
      // The staging tiles of the last item's W / U stores lie in the matrix's space, which every thread is about to
      // write: each warp's stores must have read their tile first (its lane 0 issued them), and everyone must know.
      if (lane == 0) bulk_wait_read();
      __syncthreads();
      // tri_inv_wy: the stored A comes in with 16-byte loads; only its strict lower triangle is used
      // (unit diagonal and zero upper triangle are written as constants)
      const size_t a_step = (size_t)(cfg::NT / (C / 4)) * p.H * C;
      const float* a_src = p.A_in + ((size_t)(tok0 + tid / (C / 4)) * p.H + h) * C + 4 * (tid % (C / 4));
#pragma unroll
      for (int m = 0; m < C / 8; ++m) {
        const int e = tid + m * cfg::NT;
        const int i = e / (C / 4), j = 4 * (e - i * (C / 4));
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < rows && j < i && TRI_INV_CHECK(p, (long long)tok0 + i < p.n_tokens)) v = *reinterpret_cast<const float4*>(a_src + (size_t)m * a_step);
        v.x = (j + 0 < i) ? v.x : (j + 0 == i ? 1.f : 0.f);
        v.y = (j + 1 < i) ? v.y : (j + 1 == i ? 1.f : 0.f);
        v.z = (j + 2 < i) ? v.z : (j + 2 == i ? 1.f : 0.f);
        v.w = (j + 3 < i) ? v.w : (j + 3 == i ? 1.f : 0.f);
        *reinterpret_cast<float4*>(sX + i * LD + j) = v;
      }
    }
    // rows past the sequence end hold a neighbour's tokens (or zero fill): they are cleared before any MMA
    auto clear_tail_rows = [&](bool k_tile, bool v_tile) {
      for (int e = tid; e < (C - rows) * 8 * cfg::NBOX * 2; e += cfg::NT) {
        int which = e / ((C - rows) * 8 * cfg::NBOX);
        if (which ? !v_tile : !k_tile) continue;
        int rem = e - which * (C - rows) * 8 * cfg::NBOX;
        int bx = rem / ((C - rows) * 8);
        int rem2 = rem - bx * (C - rows) * 8;
        int r = rows + rem2 / 8, c = rem2 & 7;
        uint8_t* base = smem + (which ? cfg::OFF_V : cfg::OFF_K) + bx * cfg::BOX_BYTES + r * 128 + c * 16;
        *reinterpret_cast<uint4*>(base) = make_uint4(0, 0, 0, 0);
      }
      fence_proxy_async();
    };
    // raw front end: the K tile in shared memory becomes the normalised keys (row i times 1 / |k_i|, bf16 in place)
    auto rescale_k_tile = [&]() {
      constexpr int PER = C * 8 * cfg::NBOX / cfg::NT;   // 16-byte pieces per thread
      static_assert(PER % 4 == 0 && PER * cfg::NT == C * 8 * cfg::NBOX, "four pieces at a time");
#pragma unroll
      for (int m0 = 0; m0 < PER; m0 += 4) {
        // four pieces' loads first: a load behind a store to the tile would wait for it
        uint4 v[4];
        float sc[4];
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const int e = tid + (m0 + m) * cfg::NT;
          const int bx = e / (C * 8), rem = e - bx * (C * 8), r = rem >> 3, c = rem & 7;
          v[m] = *reinterpret_cast<const uint4*>(smem + cfg::OFF_K + bx * cfg::BOX_BYTES + r * 128 + c * 16);
          sc[m] = wdecay ? sR[r] * ((gshift && r == 0) ? 1.f : ex2_approx(sG[r - gshift])) : sR[r];
        }
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const int e = tid + (m0 + m) * cfg::NT;
          const int bx = e / (C * 8), rem = e - bx * (C * 8), r = rem >> 3, c = rem & 7;
          uint32_t* w = reinterpret_cast<uint32_t*>(&v[m]);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const float2 f = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&w[q]));
            w[q] = pack_bf16(f.x * sc[m], f.y * sc[m]);
          }
          *reinterpret_cast<uint4*>(smem + cfg::OFF_K + bx * cfg::BOX_BYTES + r * 128 + c * 16) = v[m];
        }
      }
    };
    // after K (and V) were requested again for the WY step: padding rows cleared, keys normalised
    auto finish_reload = [&]() {
      if (rows < C || raw) {
        wait(bar_k, ph_k);
        if (need_v && rows < C) wait(bar_v, ph_v);
        if (rows < C) clear_tail_rows(true, need_v);
        if (raw) { rescale_k_tile(); fence_proxy_async(); }
        __syncthreads();
      }
    };
    if (rows < C) {
      const bool v_now = need_v && !cfg::RELOAD, k_now = !(cfg::ALIAS && load_a);
      if (k_now) wait(bar_k, ph_k);
      if (v_now) wait(bar_v, ph_v);
      clear_tail_rows(k_now, v_now);
    }
    if (lane == 0) bulk_wait_read();   // this warp's last W / U stores have read their staging tile, which lies in the matrix's space
    if (bad) *s_gave_up = 1;
    __syncthreads();
    // The one exit on a wait that gave up: every thread reads the flag behind this barrier (a thread can raise it
    // again only before the next item's barrier, which it reaches after everyone has read it here).
    if (*s_gave_up) break;
    // the item after next: the ticket is drawn now and used after the inversion, so that its round trip to
    // global memory does not hold this warp (and, at the next barrier, the CTA)
    int ticket = 0;
    if (tid == kTidL2 && has_next && p.work_counter) ticket = atomicAdd(p.work_counter, 1);
    PHASE(0);
    // build only: nothing later in the item hides this load, so it is issued now (the element is in L2 already)
    if (BO && has_next) bg_next = fetch_bg(nx_tok0, nx_rows, nx_h);

    if (!load_a) {
      // ---- 2. Gram S = K K^T on the tensor core: one thread issues D/16 MMAs of C x C x 16 into TMEM
      if (tid == 0 && !gram_early) {
        // self-test (kTestStall): CTA 0 leaves out the Gram product of its first item, so the wait below runs out
        const bool stall = (p.ops & kTestStall) && item == 0;
        if (wait(bar_k, ph_k) && !stall) {
          tc_fence_after();
          issue_gram();
        }
      }
      gram_early = false;
      wait(bar_mma, ph_mma);
      ph_mma ^= 1;
      tc_fence_after();
      if (!BO && tid == kTidK && !do_wy && !cfg::RELOAD && has_next) issue_k(nx_tok0, nx_h);  // K's last reader was the Gram product
      PHASE(1);
      // raw front end: the Gram diagonal is |k_i|^2; 1 / |k_i| of this warp's rows goes to shared memory for
      // every warp's gate (S_ij r_i r_j is the Gram entry of the normalised keys) and for the K tile's rescaling
      auto publish_inv_norms = [&](const float (&sacc)[C / 8][4]) {
#pragma unroll
        for (int jb = 0; jb < cfg::NW; ++jb) {
          if (jb == rb && t == (g >> 1)) {
            const float da = (g & 1) ? sacc[2 * jb][1] : sacc[2 * jb][0];
            const float db = (g & 1) ? sacc[2 * jb + 1][3] : sacc[2 * jb + 1][2];
            sR[16 * rb + g] = !front ? 1.f : (da > 0.f ? rsqrtf(da) : 0.f);
            sR[16 * rb + g + 8] = !front ? 1.f : (db > 0.f ? rsqrtf(db) : 0.f);
          }
        }
        __syncthreads();
      };

      if constexpr (SER && H16) {
        // ---- 3''. product series (Alg. 5) with fp16 operands (the paper's preferred half-precision format, Sec. 4.1).
        // Y (= N at first) and the operand copy of X are fp16 K-major swizzled tiles (64 columns per 128-byte row)
        // in the space of the fp32 matrix; one stored copy of Y is the A operand (K-major) of Y.Y and the B operand
        // (MN-major, which 16-bit types allow) of both products.  X itself lives in tensor memory in fp32: it is
        // put there once (I - N) and every round accumulates X.Y on top of it, so only its fp16 copy is rewritten.
        // Operands are written with stmatrix straight from the accumulator-fragment registers.
        constexpr int R = (C == 64) ? 5 : 6;  // log2(C) - 1 rounds
        const uint32_t sYh = smem_u32(smem + cfg::OFF_X), sXh = sYh + C * C * 2;
        const int ra = 16 * rb + g, rbw = ra + 8;
        // 16 rows x 16 columns (n-tiles nt, nt + 1) of this warp's rows -> fp16 -> one stmatrix into an operand tile
        auto put16 = [&](uint32_t tile, int nt, const float (&lo)[4], const float (&hi)[4]) {
          const int mi = lane >> 3, r = 16 * rb + (lane & 7) + 8 * (mi & 1);
          const int chunk = (nt & 7) + (mi >> 1);
          const uint32_t addr = tile + (nt >> 3) * cfg::BOX_BYTES + r * 128 + ((chunk ^ (r & 7)) << 4);
          stmatrix_x4(addr, pack_f16(lo[0], lo[1]), pack_f16(lo[2], lo[3]), pack_f16(hi[0], hi[1]), pack_f16(hi[2], hi[3]));
        };
        {
          const float beta_a = sBeta[ra], beta_b = sBeta[rbw], g_a = sG[ra - (gshift && ra > 0)], g_b = sG[rbw - gshift];
          float sacc[C / 8][4];
          if constexpr (C == 64) tmem_ld_16x64(sacc, tmem_rows); else tmem_ld_16x128(sacc, tmem_rows);
          tmem_wait_ld();
          float ba = beta_a, bb = beta_b;
          if (raw) {
            publish_inv_norms(sacc);
            ba *= sR[ra];
            bb *= sR[rbw];
          }
#pragma unroll
          for (int nt = 0; nt < C / 8; ++nt) {
            const int c = 8 * nt + 2 * t;
            float n4[4] = {0.f, 0.f, 0.f, 0.f};
            if (nt / 2 <= rb) {  // tiles on or below the diagonal of this row block
              const float2 gc = *reinterpret_cast<const float2*>(sG + c);
              const float2 rc = raw ? *reinterpret_cast<const float2*>(sR + c) : make_float2(1.f, 1.f);
              n4[0] = (c < ra) ? ba * rc.x * sacc[nt][0] * ex2_approx(g_a - gc.x) : 0.f;
              n4[1] = (c + 1 < ra) ? ba * rc.y * sacc[nt][1] * ex2_approx(g_a - gc.y) : 0.f;
              n4[2] = (c < rbw) ? bb * rc.x * sacc[nt][2] * ex2_approx(g_b - gc.x) : 0.f;
              n4[3] = (c + 1 < rbw) ? bb * rc.y * sacc[nt][3] * ex2_approx(g_b - gc.y) : 0.f;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) sacc[nt][e] = n4[e];     // N replaces S in the registers
          }
          // the Gram product has completed (the K tile, where the operands go at C = 128, has no reader left)
#pragma unroll
          for (int nt = 0; nt < C / 8; nt += 2) put16(sYh, nt, sacc[nt], sacc[nt + 1]);
#pragma unroll
          for (int nt = 0; nt < C / 8; ++nt) {
            const int c = 8 * nt + 2 * t;
            sacc[nt][0] = (c == ra ? 1.f : 0.f) - sacc[nt][0];
            sacc[nt][1] = (c + 1 == ra ? 1.f : 0.f) - sacc[nt][1];
            sacc[nt][2] = (c == rbw ? 1.f : 0.f) - sacc[nt][2];
            sacc[nt][3] = (c + 1 == rbw ? 1.f : 0.f) - sacc[nt][3];
          }
#pragma unroll
          for (int nt = 0; nt < C / 8; nt += 2) put16(sXh, nt, sacc[nt], sacc[nt + 1]);
          // X = I - N into tensor memory (columns C .. 2C - 1), where the rounds accumulate on it
#pragma unroll
          for (int b4 = 0; b4 < C / 8; b4 += 4) {
            const float q4[4][4] = {{sacc[b4][0], sacc[b4][1], sacc[b4][2], sacc[b4][3]},
                                    {sacc[b4 + 1][0], sacc[b4 + 1][1], sacc[b4 + 1][2], sacc[b4 + 1][3]},
                                    {sacc[b4 + 2][0], sacc[b4 + 2][1], sacc[b4 + 2][2], sacc[b4 + 2][3]},
                                    {sacc[b4 + 3][0], sacc[b4 + 3][1], sacc[b4 + 3][2], sacc[b4 + 3][3]}};
            tmem_st_16x32(q4, tmem_rows + C + 8 * b4);
          }
          tmem_wait_st();
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        constexpr uint32_t idesc_h = umma_idesc_f16(C, C, 1);
#pragma unroll 1
        for (int s = 0; s <= R; ++s) {
          if (tid == 0 && !bad) {
            tc_fence_after();
            // Y = N^p with p = 2^s is zero within p of the diagonal: steps of sixteen k whose operands are structurally
            // zero are not issued (Y.Y: k in [p, C-1-p]; X.Y: k in [p, C-1]).
            const int pw = 1 << s;
            auto da = [&](uint32_t tile, int ks) { return umma_desc(tile + (ks >> 2) * cfg::BOX_BYTES + (ks & 3) * 32, 16, 1024); };
            auto db = [&](int ks) { return umma_desc(sYh + ks * 2048, cfg::BOX_BYTES, 1024); };
            if (s < R) {
              const int k_lo = pw >> 4, k_hi = (C - 1 - pw) >> 4;
#pragma unroll
              for (int ks = 0; ks < C / 16; ++ks) {
                if (ks < k_lo || ks > k_hi) continue;
                umma_bf16(tmem, da(sYh, ks), db(ks), idesc_h, ks > k_lo);
              }
            }
            if (s >= 1) {
              const int k_lo = pw >> 4;
#pragma unroll
              for (int ks = 0; ks < C / 16; ++ks) {
                if (ks < k_lo) continue;
                umma_bf16(tmem + C, da(sXh, ks), db(ks), idesc_h, 1u);   // on top of X
              }
            }
            umma_commit(bar_mma);
          }
          wait(bar_mma, ph_mma);
          ph_mma ^= 1;
          tc_fence_after();
          if (s < R) {
            // new operands, 32 columns at a time: Y <- Y.Y (its readers, the MMAs, have completed), X's fp16 copy
#pragma unroll
            for (int b4 = 0; b4 < C / 8; b4 += 4) {
              float f[4][4];
              tmem_ld_16x32(f, tmem_rows + 8 * b4);
              tmem_wait_ld();
              put16(sYh, b4, f[0], f[1]);
              put16(sYh, b4 + 2, f[2], f[3]);
              if (s >= 1) {
                tmem_ld_16x32(f, tmem_rows + C + 8 * b4);
                tmem_wait_ld();
                put16(sXh, b4, f[0], f[1]);
                put16(sXh, b4 + 2, f[2], f[3]);
              }
            }
            fence_proxy_async();
            tc_fence_before();
            __syncthreads();
          }
        }
        // the result leaves tensor memory for the fp32 matrix used by the store and WY steps (over the operands, whose
        // readers have completed); the structure of a unit lower triangular matrix is written as constants
#pragma unroll
        for (int b4 = 0; b4 < C / 8; b4 += 4) {
          float f[4][4];
          tmem_ld_16x32(f, tmem_rows + C + 8 * b4);
          tmem_wait_ld();
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const int c = 8 * (b4 + q4) + 2 * t;
            float2 va, vb;
            va.x = (c < ra) ? f[q4][0] : (c == ra ? 1.f : 0.f);
            va.y = (c + 1 < ra) ? f[q4][1] : (c + 1 == ra ? 1.f : 0.f);
            vb.x = (c < rbw) ? f[q4][2] : (c == rbw ? 1.f : 0.f);
            vb.y = (c + 1 < rbw) ? f[q4][3] : (c + 1 == rbw ? 1.f : 0.f);
            *reinterpret_cast<float2*>(sX + ra * LD + c) = va;
            *reinterpret_cast<float2*>(sX + rbw * LD + c) = vb;
          }
        }
        tc_fence_before();
        __syncthreads();
      } else if constexpr (SER) {
        // ---- 3'. product series (Alg. 5) on the tensor core.  Y (= N at first) and X (= I - N at first)
        // are kept in shared memory as fp32 K-major swizzled operands (32 floats per 128-byte row, blocks of
        // 32 columns); one stored copy of Y serves as the A operand (K-major) and as the B operand
        // (MN-major).  Step s issues Y.Y (for s < R) and X.Y (for s >= 1) together: the squaring of round
        // s + 1 does not depend on the X update of round s (App. D.1), so they share one round trip.
        constexpr int R = (C == 64) ? 5 : 6;  // log2(C) - 1 rounds
        // Operand storage during the series: Y in the space of the fp32 result matrix (written last),
        // Y^T where the K tile was and X where the V tile was (C = 128: Y^T over both tiles, X in a buffer of
        // its own) -- the Gram product is done with K, and K and V are fetched (again) for the WY step afterwards.  TF32 operands must be K-major here:
        // Y is the A operand of Y.Y, X the A operand of X.Y, and Y^T (rows = columns of Y) the B operand.
        uint8_t* yb = smem + cfg::OFF_X;
        uint8_t* ytb = smem + cfg::OFF_K;
        uint8_t* xb = smem + (C == 64 ? cfg::OFF_V : cfg::OFF_XS);
        const uint32_t sYb = smem_u32(yb), sYtb = smem_u32(ytb), sXb = smem_u32(xb);
        auto canon = [](int r, int c) -> uint32_t {  // byte offset of element (r, c) in the swizzled fp32 operand layout
          return (uint32_t)((c >> 5) * (C * 128) + r * 128 + (((((c & 31) >> 2) ^ (r & 7)) << 4) | ((c & 3) * 4)));
        };
        const int ra = 16 * rb + g, rbw = ra + 8;
        const float beta_a = sBeta[ra], beta_b = sBeta[rbw], g_a = sG[ra - (gshift && ra > 0)], g_b = sG[rbw - gshift];
        float xr[C / 8][4];  // this warp's 16 rows of X, accumulator-fragment layout, kept across rounds
        // rows ra, rbw of Y (pairs of columns) and the same values into Y^T (column ra / rbw of rows c, c+1)
        auto put_y = [&](int c, float2 ya, float2 yw) {
          *reinterpret_cast<float2*>(yb + canon(ra, c)) = ya;
          *reinterpret_cast<float2*>(yb + canon(rbw, c)) = yw;
          *reinterpret_cast<float*>(ytb + canon(c, ra)) = ya.x;
          *reinterpret_cast<float*>(ytb + canon(c + 1, ra)) = ya.y;
          *reinterpret_cast<float*>(ytb + canon(c, rbw)) = yw.x;
          *reinterpret_cast<float*>(ytb + canon(c + 1, rbw)) = yw.y;
        };
        {
          float sacc[C / 8][4];
          if constexpr (C == 64) tmem_ld_16x64(sacc, tmem_rows); else tmem_ld_16x128(sacc, tmem_rows);
          tmem_wait_ld();
          float ba = beta_a, bb = beta_b;
          if (raw) {
            publish_inv_norms(sacc);
            ba *= sR[ra];
            bb *= sR[rbw];
          }
#pragma unroll
          for (int nt = 0; nt < C / 8; ++nt) {
            const int c = 8 * nt + 2 * t;
            float2 na = make_float2(0.f, 0.f), nb = na;
            if (nt / 2 <= rb) {  // tiles on or below the diagonal of this row block
              const float2 gc = *reinterpret_cast<const float2*>(sG + c);
              const float2 rc = raw ? *reinterpret_cast<const float2*>(sR + c) : make_float2(1.f, 1.f);
              na.x = (c < ra) ? ba * rc.x * sacc[nt][0] * ex2_approx(g_a - gc.x) : 0.f;
              na.y = (c + 1 < ra) ? ba * rc.y * sacc[nt][1] * ex2_approx(g_a - gc.y) : 0.f;
              nb.x = (c < rbw) ? bb * rc.x * sacc[nt][2] * ex2_approx(g_b - gc.x) : 0.f;
              nb.y = (c + 1 < rbw) ? bb * rc.y * sacc[nt][3] * ex2_approx(g_b - gc.y) : 0.f;
            }
            xr[nt][0] = (c == ra ? 1.f : 0.f) - na.x;
            xr[nt][1] = (c + 1 == ra ? 1.f : 0.f) - na.y;
            xr[nt][2] = (c == rbw ? 1.f : 0.f) - nb.x;
            xr[nt][3] = (c + 1 == rbw ? 1.f : 0.f) - nb.y;
            put_y(c, na, nb);
            *reinterpret_cast<float2*>(xb + canon(ra, c)) = make_float2(xr[nt][0], xr[nt][1]);
            *reinterpret_cast<float2*>(xb + canon(rbw, c)) = make_float2(xr[nt][2], xr[nt][3]);
          }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        constexpr uint32_t idesc_s = umma_idesc_tf32(C, C, 0);
#pragma unroll 1
        for (int s = 0; s <= R; ++s) {
          if (tid == 0) {
            tc_fence_after();
            // Y = N^p with p = 2^s is zero within p of the diagonal: Y[i][k] needs k <= i - p, Y[k][j] needs
            // k >= j + p.  Steps of eight k whose operands are structurally zero are not issued.
            const int pw = 1 << s;
            if (s < R) {   // Y.Y: k in [p, C-1-p]
              const int k_lo = pw >> 3, k_hi = (C - 1 - pw) >> 3;
#pragma unroll
              for (int ks = 0; ks < C / 8; ++ks) {
                if (ks < k_lo || ks > k_hi) continue;
                const uint32_t koff = (ks >> 2) * (C * 128) + (ks & 3) * 32;
                umma_tf32(tmem, umma_desc(sYb + koff, 16, 1024), umma_desc(sYtb + koff, 16, 1024), idesc_s, ks > k_lo);
              }
            }
            if (s >= 1) {  // X.Y: k in [p, C-1]
              const int k_lo = pw >> 3;
#pragma unroll
              for (int ks = 0; ks < C / 8; ++ks) {
                if (ks < k_lo) continue;
                const uint32_t koff = (ks >> 2) * (C * 128) + (ks & 3) * 32;
                umma_tf32(tmem + C, umma_desc(sXb + koff, 16, 1024), umma_desc(sYtb + koff, 16, 1024), idesc_s, ks > k_lo);
              }
            }
            umma_commit(bar_mma);
          }
          wait(bar_mma, ph_mma);
          ph_mma ^= 1;
          tc_fence_after();
          if (s < R) {  // Y <- Y.Y, written over the old Y and Y^T (their readers, the MMAs, have completed)
            float yn[C / 8][4];
            if constexpr (C == 64) tmem_ld_16x64(yn, tmem_rows); else tmem_ld_16x128(yn, tmem_rows);
            tmem_wait_ld();
#pragma unroll
            for (int nt = 0; nt < C / 8; ++nt)
              put_y(8 * nt + 2 * t, make_float2(yn[nt][0], yn[nt][1]), make_float2(yn[nt][2], yn[nt][3]));
          }
          if (s >= 1) {  // X <- X + X.Y
            float xn[C / 8][4];
            if constexpr (C == 64) tmem_ld_16x64(xn, tmem_rows + C); else tmem_ld_16x128(xn, tmem_rows + C);
            tmem_wait_ld();
#pragma unroll
            for (int nt = 0; nt < C / 8; ++nt) {
              const int c = 8 * nt + 2 * t;
#pragma unroll
              for (int e = 0; e < 4; ++e) xr[nt][e] += xn[nt][e];
              if (s < R) {
                *reinterpret_cast<float2*>(xb + canon(ra, c)) = make_float2(xr[nt][0], xr[nt][1]);
                *reinterpret_cast<float2*>(xb + canon(rbw, c)) = make_float2(xr[nt][2], xr[nt][3]);
              }
            }
          }
          if (s < R) {
            fence_proxy_async();
            tc_fence_before();
            __syncthreads();
          }
        }
        // the result goes to the fp32 matrix used by the store and WY steps; the structure of a unit lower
        // triangular matrix is written as constants
#pragma unroll
        for (int nt = 0; nt < C / 8; ++nt) {
          const int c = 8 * nt + 2 * t;
          float2 va, vb;
          va.x = (c < ra) ? xr[nt][0] : (c == ra ? 1.f : 0.f);
          va.y = (c + 1 < ra) ? xr[nt][1] : (c + 1 == ra ? 1.f : 0.f);
          vb.x = (c < rbw) ? xr[nt][2] : (c == rbw ? 1.f : 0.f);
          vb.y = (c + 1 < rbw) ? xr[nt][3] : (c + 1 == rbw ? 1.f : 0.f);
          *reinterpret_cast<float2*>(sX + ra * LD + c) = va;
          *reinterpret_cast<float2*>(sX + rbw * LD + c) = vb;
        }
        tc_fence_before();
        __syncthreads();
        if (do_wy) {
          // K and V come (back) into their tiles for the WY step
          if (tid == kTidK) issue_k(tok0, h);
          if (tid == kTidV && need_v) issue_v(tok0, h);
          ph_k ^= 1;
          finish_reload();
        }
      } else {
      // ---- 3. gate + mask on this warp's rows, N -> shared memory
      const int ra = 16 * rb + g, rbw = ra + 8;
      const float beta_a = sBeta[ra], beta_b = sBeta[rbw], g_a = sG[ra - (gshift && ra > 0)], g_b = sG[rbw - gshift];
      {
        float sacc[C / 8][4];   // this warp's 16 rows of S, all C columns, in one tensor-memory load
        if constexpr (C == 64) tmem_ld_16x64(sacc, tmem_rows); else tmem_ld_16x128(sacc, tmem_rows);
        tmem_wait_ld();
        float ba = beta_a, bb = beta_b;
        if (raw) {
          publish_inv_norms(sacc);
          ba *= sR[ra];
          bb *= sR[rbw];
        }
        // g of every column this lane meets, before the first store to the matrix (a load behind such a store would wait for it:
        // the compiler cannot tell the two apart)
        float2 gcs[C / 8];
#pragma unroll
        for (int q = 0; q < C / 8; ++q) gcs[q] = *reinterpret_cast<const float2*>(sG + 8 * q + 2 * t);
#pragma unroll
        for (int jb = 0; jb < cfg::NW; ++jb) {
          if (jb > rb) {
            // tiles above the diagonal: exact +0.0, so the stored A and the A' operand need no masking later
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
              const int c = 16 * jb + 8 * nt + 2 * t;
              *reinterpret_cast<float2*>(sX + ra * LD + c) = make_float2(0.f, 0.f);
              *reinterpret_cast<float2*>(sX + rbw * LD + c) = make_float2(0.f, 0.f);
              if constexpr (REF) {
                *reinterpret_cast<float2*>(sN + ra * LD + c) = make_float2(0.f, 0.f);
                *reinterpret_cast<float2*>(sN + rbw * LD + c) = make_float2(0.f, 0.f);
              }
            }
          } else {
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
              const int c = 16 * jb + 8 * nt + 2 * t;
              const float2 gc = gcs[2 * jb + nt];
              const float2 rc = raw ? *reinterpret_cast<const float2*>(sR + c) : make_float2(1.f, 1.f);
              const float (&a4)[4] = sacc[2 * jb + nt];
              float2 va, vb;
              va.x = ba * rc.x * a4[0] * ex2_approx(g_a - gc.x);
              va.y = ba * rc.y * a4[1] * ex2_approx(g_a - gc.y);
              vb.x = bb * rc.x * a4[2] * ex2_approx(g_b - gc.x);
              vb.y = bb * rc.y * a4[3] * ex2_approx(g_b - gc.y);
              if (jb == rb) {  // the diagonal tile: strict-lower mask by selection
                va.x = (c < ra) ? va.x : 0.f;
                va.y = (c + 1 < ra) ? va.y : 0.f;
                vb.x = (c < rbw) ? vb.x : 0.f;
                vb.y = (c + 1 < rbw) ? vb.y : 0.f;
              }
              *reinterpret_cast<float2*>(sX + ra * LD + c) = va;
              *reinterpret_cast<float2*>(sX + rbw * LD + c) = vb;
              if constexpr (REF) {   // the Gram product, the K tile's only reader so far, has completed
                *reinterpret_cast<float2*>(sN + ra * LD + c) = va;
                *reinterpret_cast<float2*>(sN + rbw * LD + c) = vb;
              }
            }
          }
        }
      }
      __syncwarp();
      PHASE(2);

      // ---- 4. leaf: invert this warp's 16x16 diagonal block
      if (leaf_series_on) {
        leaf_series<LD, cfg::LEAF_LD>(sX + 16 * rb * LD + 16 * rb,
                                      reinterpret_cast<float*>(smem + cfg::OFF_LEAF) + warp * 16 * cfg::LEAF_LD, lane);
      } else {
        leaf_substitution<LD>(sX + 16 * rb * LD + 16 * rb, lane);
      }
      __syncthreads();
      if (BO && tid == kTidK && has_next) issue_k(nx_tok0, nx_h);  // the leaf scratch inside the K tile is no longer needed
      PHASE(3);

      // ---- 5. merges
      merge_level<C, 16>(sX, warp, lane);
      PHASE(4);
      merge_level<C, 32>(sX, warp, lane);
      if constexpr (C == 128 && cfg::ALIAS) {
        // Top level at C = 128, X21 = -A22 . N21 . A11 with 64 x 64 blocks, as two tcgen05.mma (kind::tf32) products
        // instead of about 650 warp-level MMAs per matrix on the legacy pipe, which two resident CTAs share.
        // Operands (fp32 rounded to TF32, K-major, 128-byte swizzle, two blocks of 32 columns) live in the A' space,
        // idle until the inversion is done: first N21 and A11^T, then A22 and T^T; accumulators in tensor memory.
        auto canon64 = [](int r, int c) -> uint32_t {
          return (uint32_t)((c >> 5) * 8192 + r * 128 + (((((c & 31) >> 2) ^ (r & 7)) << 4) | ((c & 3) * 4)));
        };
        uint8_t* opa = smem + cfg::OFF_AP;
        uint8_t* opb = opa + 16384;
        constexpr uint32_t idesc_m = umma_idesc_tf32(64, 64, 0);
        auto copy_block = [&](uint8_t* dst, int r0, int c0) {   // 64 x 64 block of the matrix, row-major -> operand layout
          float4 v[4];   // loads first: a load behind a store to shared memory waits for it
#pragma unroll
          for (int m = 0; m < 4; ++m) {
            const int e = tid + m * cfg::NT, i = e >> 4, k4 = (e & 15) * 4;
            v[m] = *reinterpret_cast<const float4*>(sX + (r0 + i) * LD + c0 + k4);
          }
#pragma unroll
          for (int m = 0; m < 4; ++m) {
            const int e = tid + m * cfg::NT, i = e >> 4, k4 = (e & 15) * 4;
            uint4 w;
            w.x = to_tf32(v[m].x); w.y = to_tf32(v[m].y); w.z = to_tf32(v[m].z); w.w = to_tf32(v[m].w);
            *reinterpret_cast<uint4*>(dst + canon64(i, k4)) = w;
          }
        };
        auto issue_merge = [&](uint32_t d_col) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const uint32_t koff = (ks >> 2) * 8192 + (ks & 3) * 32;
            umma_tf32(tmem + d_col, umma_desc(sAp + koff, 16, 1024), umma_desc(sAp + 16384 + koff, 16, 1024), idesc_m, ks > 0);
          }
          umma_commit(bar_mma);
        };
        const int mq = warp & 3, mh = warp >> 2;           // tensor-memory quadrant (16 rows of an M = 64 result) and column half
        const uint32_t tm_m = tmem + ((uint32_t)(32 * mq) << 16) + 32 * mh;
        // product 1: T = N21 . A11  (A = N21 as stored; B = A11^T: element (n, k) = A11[k][n])
        {
          const int nn = lane & 7, kk = lane >> 3;         // an 8 (n) x 4 (k) patch per warp and step: conflict-free stores
          float av[16];
#pragma unroll
          for (int m = 0; m < 16; ++m) {
            const int patch = warp * 16 + m;
            av[m] = sX[(4 * (patch >> 3) + kk) * LD + 8 * (patch & 7) + nn];
          }
          copy_block(opa, 64, 0);   // (behind the loads above: its stores would hold them up)
#pragma unroll
          for (int m = 0; m < 16; ++m) {
            const int patch = warp * 16 + m, n = 8 * (patch & 7) + nn, k = 4 * (patch >> 3) + kk;
            *reinterpret_cast<uint32_t*>(opb + canon64(n, k)) = to_tf32(av[m]);
          }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) { tc_fence_after(); issue_merge(0); }
        wait(bar_mma, ph_mma);
        ph_mma ^= 1;
        tc_fence_after();
        // product 2: X21 = -(A22 . T)  (A = A22; B = T^T: element (n, k) = T[k][n], from this thread's fragments)
        {
          float tf[4][4];
          tmem_ld_16x32(tf, tm_m);
          copy_block(opa, 64, 64);   // while the tensor-memory load is in flight (product 1, the last reader of opa, has completed)
          tmem_wait_ld();
          const int ka = 16 * mq + g, kb = ka + 8;
#pragma unroll
          for (int nt = 0; nt < 4; ++nt) {
            const int n = 32 * mh + 8 * nt + 2 * t;
            *reinterpret_cast<uint32_t*>(opb + canon64(n, ka)) = to_tf32(tf[nt][0]);
            *reinterpret_cast<uint32_t*>(opb + canon64(n + 1, ka)) = to_tf32(tf[nt][1]);
            *reinterpret_cast<uint32_t*>(opb + canon64(n, kb)) = to_tf32(tf[nt][2]);
            *reinterpret_cast<uint32_t*>(opb + canon64(n + 1, kb)) = to_tf32(tf[nt][3]);
          }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) { tc_fence_after(); issue_merge(64); }
        wait(bar_mma, ph_mma);
        ph_mma ^= 1;
        tc_fence_after();
        {
          float xf[4][4];
          tmem_ld_16x32(xf, tm_m + 64);
          tmem_wait_ld();
          const int ia = 64 + 16 * mq + g, ib = ia + 8;
#pragma unroll
          for (int nt = 0; nt < 4; ++nt) {
            const int c = 32 * mh + 8 * nt + 2 * t;
            *reinterpret_cast<float2*>(sX + ia * LD + c) = make_float2(-xf[nt][0], -xf[nt][1]);
            *reinterpret_cast<float2*>(sX + ib * LD + c) = make_float2(-xf[nt][2], -xf[nt][3]);
          }
        }
        tc_fence_before();
        __syncthreads();
      } else if constexpr (C == 128) {
        merge_level<C, 64>(sX, warp, lane);
      }
      PHASE(5);
      if constexpr (REF) {
        // ---- 5b. one step of iterative refinement (Alg. 6): X <- X + (I - X (I + N)) X, then K and V come back
        refine_step<C>(sX, sN, warp, lane);
        if (do_wy) {
          if (tid == kTidK) issue_k(tok0, h);
          if (tid == kTidV && need_v) issue_v(tok0, h);
          ph_k ^= 1;
          finish_reload();
        }
      }
      }
    }

    // ---- 6. A leaves shared memory once: stored to global, and scaled by beta into the bf16 operand A'
    constexpr int NV = C / 8;  // float4 per thread
    // thread's first float4 of A: row tid / (C/4), columns 4 (tid % (C/4)); later ones are NT / (C/4) rows further down
    const size_t a_step = (size_t)(cfg::NT / (C / 4)) * p.H * C;
    float* a_dst = ((p.ops & kStoreA) && p.A)
                       ? p.A + ((size_t)(tok0 + tid / (C / 4)) * p.H + h) * C + 4 * (tid % (C / 4)) : nullptr;
    // bf16 pair stores of one float4 of A scaled by beta: K-major, 128-byte swizzle, 64 tokens per row block
    // (a thread's columns j are the same in every pass: NT is a multiple of C / 4)
    const float4 beta_j = *reinterpret_cast<const float4*>(sBeta + 4 * (tid % (C / 4)));
    auto put_ap = [&](int i, int j, const float4& v) {
      const float4 b = beta_j;
      const uint32_t lo = pack_bf16(v.x * b.x, v.y * b.y), hi = pack_bf16(v.z * b.z, v.w * b.w);
      const uint32_t off = (uint32_t)((j >> 6) * (C * 128) + i * 128 + (((((j & 63) >> 3) ^ (i & 7)) << 4) | ((j & 7) * 2)));
      if (TRI_INV_CHECK(p, off + 8 <= (uint32_t)(C * C * 2) && i < C && j + 4 <= C))
        asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(sAp + off), "r"(lo), "r"(hi) : "memory");
    };
    float4 xv[cfg::ALIAS ? 1 : NV];
    if constexpr (cfg::ALIAS) {
      // A' has a region of its own: one pass reads the matrix (8 rows per step), stores A and writes A'.  K and V come
      // back into the matrix's space box by box as the pass frees it: a 16 KB box covers 31 rows of the matrix, so
      // K's boxes are requested after rows 0..31 and 0..63, V's first after rows 0..95 and its second after the pass.
      static_assert(C != 128 || (cfg::NT == 256 && LD * 4 * 32 >= cfg::BOX_BYTES && LD * 4 * 31 <= cfg::BOX_BYTES),
                    "the box-by-box reload assumes 8 rows per step and 31 to 32 matrix rows per box");
      static_assert(NV % 4 == 0, "four passes at a time");
#pragma unroll
      for (int m0 = 0; m0 < NV; m0 += 4) {
        // four passes' loads first: the operand stores below keep their program order with every later shared-memory load
        float4 v4[4];
#pragma unroll
        for (int mm = 0; mm < 4; ++mm) {
          const int e = tid + (m0 + mm) * cfg::NT;
          const int i = e / (C / 4), j = 4 * (e - i * (C / 4));
          v4[mm] = *reinterpret_cast<const float4*>(sX + i * LD + j);
        }
#pragma unroll
        for (int mm = 0; mm < 4; ++mm) {
        const int m = m0 + mm;
        const int e = tid + m * cfg::NT;
        const int i = e / (C / 4), j = 4 * (e - i * (C / 4));
        const float4 v = v4[mm];
        if (a_dst && i < rows && TRI_INV_CHECK(p, (long long)tok0 + i < p.n_tokens && j + 4 <= C)) *reinterpret_cast<float4*>(a_dst + (size_t)m * a_step) = v;
        if (do_wy) put_ap(i, j, v);
        }
        const int m = m0 + 3;
        if (C == 128 && do_wy && (m == 3 || m == 7 || m == 11)) {
          fence_proxy_async();
          __syncthreads();   // rows 0 .. 8 m + 7 have been read by everyone
          if (m == 3 && tid == kTidK) {
            ++n_issue;
            mbar_expect_tx(bar_k, (uint32_t)cfg::TILE_BYTES);
            tma_load_2d(sK, &tmK, bar_k, h * D, tok0);
          }
          if (m == 7 && tid == kTidK) tma_load_2d(sK + cfg::BOX_BYTES, &tmK, bar_k, h * D + 64, tok0);
          if (m == 11 && tid == kTidV && need_v) {
            ++n_issue;
            mbar_expect_tx(bar_v, (uint32_t)cfg::TILE_BYTES);
            tma_load_2d(sV, &tmV, bar_v, h * D, tok0);
          }
        }
      }
    } else if constexpr (BO) {
      // Build only: A leaves straight from shared memory, one 256-byte bulk copy per row (no trip through
      // registers and the load/store pipe, which is what bounds this variant).  The matrix is complete in
      // shared memory: +0.0 above the diagonal, 1.0f on it.  Rows past the sequence end are not copied.
      fence_proxy_async();   // the merges' stores become visible to the copy engine
      __syncthreads();
      if ((p.ops & kStoreA) && p.A && rows == C && p.a_box) {
        // a whole chunk: ONE tiled bulk store of C tokens x LD floats (tmW is the 3-D map of A here; the LD - C padding
        // columns fall outside the tensor's innermost extent and are dropped) instead of C row copies
        if (tid == 0 && TRI_INV_CHECK(p, (long long)tok0 + C <= p.n_tokens)) {
          tma_store_3d(&tmW, smem_u32(sX), 0, h, tok0);
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      } else if ((p.ops & kStoreA) && p.A && tid < rows && TRI_INV_CHECK(p, (long long)tok0 + tid < p.n_tokens)) {
        float* dst = p.A + ((size_t)(tok0 + tid) * p.H + h) * C;
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_u32(sX + tid * LD)), "r"(C * 4) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    } else {
#pragma unroll
      for (int m = 0; m < NV; ++m) {
        const int e = tid + m * cfg::NT;
        const int i = e / (C / 4), j = 4 * (e - i * (C / 4));
        // the matrix in shared memory is complete: +0.0 above the diagonal, 1.0f on it
        const float4 v = *reinterpret_cast<const float4*>(sX + i * LD + j);
        xv[m] = v;
        // without a WY product there is nothing to overlap the stores with: issue them right away
        if (!do_wy && a_dst && i < rows && TRI_INV_CHECK(p, (long long)tok0 + i < p.n_tokens && j + 4 <= C)) *reinterpret_cast<float4*>(a_dst + (size_t)m * a_step) = v;
      }
    }
    // the item after next (read after this item's last barrier): by ticket, or by a fixed stride without a counter pair
    if (tid == kTidL2) *s_next_item = !has_next ? total : (p.work_counter ? 2 * (int)gridDim.x + ticket : nx_item + (int)gridDim.x);
    PHASE(6);

    if (do_wy) {
      if constexpr (cfg::ALIAS) {
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();  // the fp32 matrix has been read by everyone: the last box may land in its space
        if (C == 128) {
          if (tid == kTidV && need_v) tma_load_2d(sV + cfg::BOX_BYTES, &tmV, bar_v, h * D + 64, tok0);
        } else {
          if (tid == kTidK) issue_k(tok0, h);
          if (tid == kTidV && need_v) issue_v(tok0, h);
        }
        if (!load_a) ph_k ^= 1;  // second K copy of this item
        finish_reload();
      } else {
        tc_fence_before();
        __syncthreads();  // every read of the fp32 matrix (and of S in TMEM) is done: its space becomes A'
#pragma unroll
        for (int m = 0; m < NV; ++m) {
          const int e = tid + m * cfg::NT;
          const int i = e / (C / 4), j = 4 * (e - i * (C / 4));
          put_ap(i, j, xv[m]);
        }
        if (raw && !cfg::RELOAD) rescale_k_tile();  // the Gram product, K's only reader so far, has completed
        fence_proxy_async();  // generic-proxy writes of A' become visible to the tensor core's reads
        __syncthreads();
      }
      PHASE(7);
      if (has_next) bg_next = fetch_bg(nx_tok0, nx_rows, nx_h);  // consumed at the top of the next item

      // ---- 7. WY: [W | U] = A' . [K | V] with the staged tiles as the MN-major B operand
      // W and U are two products of D columns each: at C = 64 through the same columns (W leaves before U arrives), at C = 128
      // side by side, U behind a commit of its own so that W is stored while U runs (and V's last box may still be on its way)
      static_assert(D == 128 || (D == 64 && C == 64), "head dimensions: 128, or 64 at C = 64");
      constexpr uint32_t idesc_wy = umma_idesc(C, D, 1);
      auto issue_wy = [&](uint32_t b_tile, uint32_t d_col = 0, bool second = false) {
#pragma unroll
        for (int ks = 0; ks < C / 16; ++ks) {
          const uint64_t da = umma_desc(sAp + (ks >> 2) * (C * 128) + (ks & 3) * 32, 16, 1024);
          const uint64_t db = umma_desc(b_tile + ks * 2048, cfg::BOX_BYTES, 1024);
          umma_bf16(tmem + d_col, da, db, idesc_wy, ks > 0);
        }
        umma_commit(second ? bar_mma_u : bar_mma);
      };
      if (tid == 0) {
        if (wait(bar_k, ph_k)) { tc_fence_after(); issue_wy(sK); }
        if (C == 128 && need_v) {
          if (wait(bar_v, ph_v)) { tc_fence_after(); issue_wy(sV, D, true); }
        }
      }
      // A goes to global memory while the W product runs (its registers are free again before W returns)
      if (!cfg::ALIAS && a_dst) {
#pragma unroll
        for (int m = 0; m < NV; ++m) {
          const int i = (tid + m * cfg::NT) / (C / 4);
          if (i < rows && TRI_INV_CHECK(p, (long long)tok0 + i < p.n_tokens)) *reinterpret_cast<float4*>(a_dst + (size_t)m * a_step) = xv[m];
        }
      }
      wait(bar_mma, ph_mma);
      ph_mma ^= 1;
      tc_fence_after();
      PHASE(8);
      // this warp's 16 rows of W leave in two 64-column pieces
      const int row0 = 16 * rb;
      const size_t row_stride = (size_t)p.H * D;
      __nv_bfloat16* w_row0 = reinterpret_cast<__nv_bfloat16*>(p.W) + ((size_t)(tok0 + row0) * p.H + h) * D;
      __nv_bfloat16* u_row0 = reinterpret_cast<__nv_bfloat16*>(p.U) + ((size_t)(tok0 + row0) * p.H + h) * D;
      const uint32_t stage = smem_u32(smem + cfg::OFF_STAGE) + warp * 2048;
      if (C == 64 && need_v) {
        float f0[8][4], f1[8][4];
        tmem_ld_16x64(f0, tmem_rows);
        if constexpr (D == 128) tmem_ld_16x64(f1, tmem_rows + 64);
        tmem_wait_ld();
        tc_fence_before();
        __syncthreads();  // every warp holds its rows of W in registers: U may overwrite the columns
        if (tid == 0) {
          if (wait(bar_v, ph_v)) { tc_fence_after(); issue_wy(sV); }
        }
        if (tid == kTidK && has_next) issue_k(nx_tok0, nx_h);  // K's last reader (the W product) is done
        store_frag_piece_bf16(f0, stage, lane, w_row0, row_stride, rows - row0, &tmW, h * D + 0, tok0 + row0);
        if constexpr (D == 128) store_frag_piece_bf16(f1, stage, lane, w_row0 + 64, row_stride, rows - row0, &tmW, h * D + 64, tok0 + row0);
        PHASE(9);
        wait(bar_mma, ph_mma);
        ph_mma ^= 1;
        tc_fence_after();
        PHASE(10);
        tmem_ld_16x64(f0, tmem_rows);
        if constexpr (D == 128) tmem_ld_16x64(f1, tmem_rows + 64);
        tmem_wait_ld();
        tc_fence_before();
        __syncthreads();  // all MMAs done and all accumulators read: tiles, A' and tensor memory are free
        ph_k ^= 1;
        ph_v ^= 1;
        if (tid == kTidV && has_next && !cfg::RELOAD) issue_v(nx_tok0, nx_h);
        if (tid == 0 && has_next && nx_rows == C && !load_a && mbar_try_wait(bar_k, ph_k)) {
          // the next K tile has landed and tensor memory is free: start the next Gram product now
          tc_fence_after();
          issue_gram();
          gram_early = true;
        }
        store_frag_piece_bf16(f0, stage, lane, u_row0, row_stride, rows - row0, &tmU, h * D + 0, tok0 + row0);
        // second staging tile: the A' operand's space, whose last reader (the U product) has completed
        if constexpr (D == 128) store_frag_piece_bf16<1>(f1, sAp + warp * 2048, lane, u_row0 + 64, row_stride, rows - row0, &tmU, h * D + 64, tok0 + row0);
      } else {
        // C = 128 (W and U side by side in 256 columns, U behind its own commit) or W only
        // With ALIAS the staging tiles lie in the A' region, which the U product is still reading: W is then staged in the
        // K tile (its last reader, the W product, has completed), and the next K tile is requested once those stores
        // have read it.
        constexpr bool kSplit = cfg::ALIAS && C == 128;
        const bool split = kSplit && need_v;
        if (cfg::ALIAS && !split && tid == kTidK && has_next && !load_a) issue_k(nx_tok0, nx_h);  // all MMAs on the tiles are done
        // two staging tiles in turn where there is room for a second one (with ALIAS: the upper half of the A' region;
        // every product that reads A' has completed)
        const uint32_t stage2 = cfg::ALIAS ? stage + cfg::NW * 2048 : stage;
        constexpr int KEEP = cfg::ALIAS ? 1 : 0;
        const uint32_t stage_w = split ? sK + warp * 2048 : stage, stage_w2 = split ? sK + cfg::BOX_BYTES + warp * 2048 : stage2;
        store_piece_bf16<0>(tmem_rows, stage_w, lane, w_row0, row_stride, rows - row0, &tmW, h * D, tok0 + row0);
        if constexpr (D == 128) store_piece_bf16<KEEP>(tmem_rows + 64, stage_w2, lane, w_row0 + 64, row_stride, rows - row0, &tmW, h * D + 64, tok0 + row0);
        if (need_v && C == 128) {
          wait(bar_mma_u, ph_u);   // the U product
          ph_u ^= 1;
          tc_fence_after();
          if (split) {
            if (lane == 0) bulk_wait_read();   // this warp's W stores have read their tiles in the K tile's space
            tc_fence_before();
            __syncthreads();
            if (tid == kTidK && has_next && !load_a) issue_k(nx_tok0, nx_h);
          }
          store_piece_bf16<KEEP>(tmem_rows + 128, stage, lane, u_row0, row_stride, rows - row0, &tmU, h * D, tok0 + row0);
          store_piece_bf16<KEEP>(tmem_rows + 192, stage2, lane, u_row0 + 64, row_stride, rows - row0, &tmU, h * D + 64, tok0 + row0);
        }
        tc_fence_before();
        __syncthreads();
        ph_k ^= 1;
        ph_v ^= 1;
        if (!cfg::ALIAS && tid == kTidK && has_next) issue_k(nx_tok0, nx_h);
        if (tid == kTidV && has_next && need_v && !cfg::RELOAD) issue_v(nx_tok0, nx_h);
      }
    } else {
      // build only: the fp32 matrix has been read by everyone after this barrier
      if (!BO && has_next) bg_next = fetch_bg(nx_tok0, nx_rows, nx_h);
      if (BO && tid < C) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // the copies have read their rows
      tc_fence_before();
      __syncthreads();
      ph_k ^= 1;
      ph_v ^= 1;
      if (tid == kTidK && has_next && ((p.ops & kLoadA) || cfg::RELOAD)) issue_k(nx_tok0, nx_h);  // otherwise requested after the Gram product
      if (tid == 0 && has_next && nx_rows == C && !load_a && mbar_try_wait(bar_k, ph_k)) {
        // the next K tile has landed and tensor memory is free: start the next Gram product now
        tc_fence_after();
        issue_gram();
        gram_early = true;
      }
    }
    PHASE(11);
    item = nx_item;
    nx_item = *s_next_item;  // written early in this item, several barriers ago
  }
  CTA_MARK(2);
  if (tid == 0 && p.work_counter && atomicAdd(p.work_counter + 1, 1) == (int)gridDim.x - 1) {
    // last CTA out: leave both counters at zero for the next launch that uses this slot
    p.work_counter[0] = 0;
    p.work_counter[1] = 0;
    __threadfence();
  }
  if (lane == 0) bulk_wait_read();
  if (bad) *s_gave_up = 1;
  if (bad || misaligned) atomicMax(p.status, TRI_INV_ERR_DEVICE_TIMEOUT);
  __syncthreads();  // every thread has left the item loop
  if (*s_gave_up) {
    // A wait gave up.  Before shared and tensor memory go back to the SM, give what this CTA still has in flight a
    // (bounded) chance to finish: the last copy each tile thread requested, and every product issued so far.
    if (tid == kTidK && n_issue) mbar_wait_bounded(bar_k, (n_issue - 1) & 1, p.wait_limit_ns);
    if (tid == kTidV && n_issue) mbar_wait_bounded(bar_v, (n_issue - 1) & 1, p.wait_limit_ns);
    if (tid == 0) {
      umma_commit(bar_exit);
      mbar_wait_bounded(bar_exit, 0, p.wait_limit_ns);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
}

// ------------------------------------------------------------------------------------------ host side
template <int C, int D, bool SER, bool RAW, bool BO = false, bool REF = false, bool H16 = false, int VAR = 3>
cudaError_t launch_one(const KParams& p_in, cudaStream_t stream) {
  using cfg = Cfg<C, D, SER, BO, REF, H16>;
  KParams p = p_in;
  // Per-device set-up (function attributes are per device) and grid size, done once per device under a lock.
  static std::mutex mu;
  static int ctas_per_sm_of[64] = {0}, n_sm_of[64] = {0};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  int ctas_per_sm, n_sm;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!ctas_per_sm_of[dev]) {
      e = cudaFuncSetAttribute(tc_kernel<C, D, SER, RAW, BO, REF, H16, VAR>, cudaFuncAttributeMaxDynamicSharedMemorySize, cfg::SMEM);
      if (e != cudaSuccess) return e;
      e = cudaFuncSetAttribute(tc_kernel<C, D, SER, RAW, BO, REF, H16, VAR>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
      if (e != cudaSuccess) return e;
      int sms = 0, smem_per_sm = 0;
      if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
      if ((e = cudaDeviceGetAttribute(&smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev)) != cudaSuccess) return e;
      // Resident CTAs per SM: bounded by tensor memory (512 columns per SM, TMEM_COLS per CTA), by shared
      // memory and by registers (the launch bound).  The runtime's occupancy query does not model
      // tensor-memory allocation, so the bound is taken from the layout itself.
      int by_smem = smem_per_sm / (cfg::SMEM + 1024);  // 1 KiB per CTA is reserved by the system
      int by_tmem = 512 / cfg::TMEM_COLS;
      int occ = by_smem < by_tmem ? by_smem : by_tmem;
      occ = occ < cfg::CTAS_PER_SM ? occ : cfg::CTAS_PER_SM;
      n_sm_of[dev] = sms > 0 ? sms : 1;
      ctas_per_sm_of[dev] = occ > 0 ? occ : 1;
    }
    ctas_per_sm = ctas_per_sm_of[dev];
    n_sm = n_sm_of[dev];
  }
  long long tokens = p.chunk_tab ? (long long)p.T : (long long)p.T * (p.n_chunks / p.chunks_per_seq);
  CUtensorMap tmK, tmV;
  if (!make_tmap(&tmK, p.K, tokens, p.H, D, C)) return cudaErrorUnknown;
  if (p.V) { if (!make_tmap(&tmV, p.V, tokens, p.H, D, C)) return cudaErrorUnknown; }
  else tmV = tmK;
  // W and U leave in boxes of 64 columns x 16 tokens (one warp's piece)
  CUtensorMap tmW = tmK, tmU = tmK;
  if constexpr (BO) {
    // build only: the W slot carries the map of A for the whole-matrix store (if the driver refuses the map, rows go one by one)
    p.a_box = (p.A && (p.ops & kStoreA) && make_tmap_a(&tmW, p.A, tokens, p.H, C, C + 4)) ? 1 : 0;
    if (!p.a_box) tmW = tmK;
  }
  if (!BO && p.W && !make_tmap(&tmW, p.W, tokens, p.H, D, 16)) return cudaErrorUnknown;
  if (p.U && !make_tmap(&tmU, p.U, tokens, p.H, D, 16)) return cudaErrorUnknown;
  long long total = (long long)p.n_chunks * p.H;
  long long cap = (long long)n_sm * ctas_per_sm;
  int grid = (int)(total < cap ? total : cap);
#ifdef TRI_INV_PHASE_CLOCKS
  if (const char* gc = getenv("TRI_INV_GRID_CAP")) { int g2 = atoi(gc); if (g2 > 0 && g2 < grid) grid = g2; }
#endif
  p.work_counter = (p.ops & kFixedStride) ? nullptr : work_counter_for(stream);  // tc_launch.cu
  tc_kernel<C, D, SER, RAW, BO, REF, H16, VAR><<<grid, cfg::NT, cfg::SMEM, stream>>>(tmK, tmW, tmU, tmV, p);
  return cudaGetLastError();
}

}  // namespace
}  // namespace tri_inv
