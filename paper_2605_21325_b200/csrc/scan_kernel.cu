// Chunk scan: the consumer of W and U.  The chunk form of the layer's recurrence (the re-formulation that
// Sec. 1 refers to; (I+N)^{-1} enters through W and U), per sequence and head, chunk after chunk, with the
// state S [d_k x d_v] carried in registers:
//
//     U~ = U - W S                                   W = A diag(beta exp g) K (decay-weighted), U = A diag(beta) V
//     O  = scale * (diag(gamma) Q S + P U~)          gamma_i = exp(g_i),  P_ij = (q_i . k_j) gamma_i / gamma_j  (j <= i)
//     S <- gamma_last S + K^T diag(gamma_last / gamma) U~
//
// Columns of S (the d_v axis) never mix, so a CTA owns one (sequence, head, slice of DVS value columns) and walks
// the chunks in order.
//
// The tensor pipe spends a near-constant time per tcgen05.mma at these sizes, so the chunk is cut into as few,
// as large products as the data flow allows -- three per chunk, 16 instructions in all:
//   P1 [128 x (DVS+64)] = [W ; Q] . [S | K^T]     rows 0..63: W S (and W K^T, unused); rows 64..127: Q S | Q K^T
//   P3 [128 x DVS]      = K^T . U~'               U~' = decay-scaled U~ (bf16); the K tile is read MN-major
//   PU [128 x DVS]      = [any ; P] . U~          rows 64..127 = P U~, on the lanes that also hold Q S
// The dependent chain of a chunk is  P1 -> U~ -> P3 -> S.  Warp 8 holds the one thread that issues every product;
// warps 0..7 compute.  Warp w works on tensor-memory lanes 32 (w & 3) .. +31 and on half (w >> 2) of the value
// columns; lanes 0..63 carry W S, so warps of quadrants 0 and 1 form U~ ("chain warps"), those of quadrants 2
// and 3 form P and the output ("output warps"); all eight update their part of S.  Hand-offs are mbarriers:
// commits from the products, counted arrivals from the compute threads after their operand writes.
// TMA brings W, Q and K (K twice: once beside S^T as the B operand of P1, once as the A operand of P3, so that
// each copy is refilled as early as its own reader allows); U and g come through registers one chunk ahead.
// Every mbarrier wait is bounded; on expiry the CTA raises the status word, frees its tensor memory and returns.
#include "tc_device.cuh"

namespace tri_inv {
namespace {

constexpr int C = 64, D = 128, NT = 256;   // NT compute threads (8 warps) + one control warp
constexpr float kLog2e = 1.4426950408889634f;

template <int DVS>
struct ScanCfg {
  static constexpr int CW = DVS / 2;                     // value columns per compute warp
  static constexpr int NTW = CW / 8;                     // accumulator n-tiles per compute warp
  static constexpr int N1 = DVS + 64;                    // columns of P1
  // A operand of P1: [W ; Q], two boxes (64 features each) of 128 rows x 128 B
  static constexpr int OFF_A = 0, A_BOX = 16384;
  // B operand of P1: [S^T ; K], two boxes of (DVS + 64) rows x 128 B
  static constexpr int OFF_B = 32768, B_BOX = N1 * 128;
  static constexpr int OFF_KA = OFF_B + 2 * B_BOX;       // K tile for P3 (MN-major A); its second box doubles as the
  static constexpr int OFF_P = OFF_KA + 16384;           // unused upper half of PU's A operand, P being the lower half
  static constexpr int OFF_UT = OFF_P + 8192;            // U~  bf16 [64 tokens][DVS], boxes of 64 columns (MN-major B)
  static constexpr int U_BYTES = 8192 * (DVS > 64 ? DVS / 64 : 1);   // a narrower slice fills the first DVS columns of one box
  static constexpr int OFF_UD = OFF_UT + U_BYTES;        // U~' bf16, same layout
  static constexpr int OFF_G = OFF_UD + U_BYTES;         // g * log2(e): 2 x 64 floats; column factors: 2 x 64 floats
  static constexpr int OFF_BAR = OFF_G + 1024;           // 9 mbarriers, tensor-memory slot
  static constexpr int SMEM = OFF_BAR + 96;
  static constexpr int TM_P1 = 0, TM_DS = N1, TM_PU = N1 + DVS;
  static constexpr int TMEM_COLS = (N1 + 2 * DVS) <= 256 ? 256 : 512;
  // DVS = 64: 9 warps at the kernel's natural register count fill an SM once.  DVS = 32 halves the state and the
  // operand registers, and two CTAs (99 KiB of shared memory and 256 tensor-memory columns each) share an SM.
  static constexpr int CTAS_PER_SM = DVS <= 32 ? 2 : 1;
};

template <int NTL>
__device__ __forceinline__ void tmem_ld_frag(float (&r)[NTL][4], uint32_t taddr) {
  if constexpr (NTL == 8) tmem_ld_16x64(r, taddr);
  else if constexpr (NTL == 4) tmem_ld_16x32(r, taddr);
  else tmem_ld_16x16(r, taddr);
}
template <int NTL>
__device__ __forceinline__ void tmem_st_frag(const float (&r)[NTL][4], uint32_t taddr) {
  if constexpr (NTL == 2) { tmem_st_16x16(r, taddr); return; }
#pragma unroll
  for (int b = 0; b < NTL; b += 4) {
    const float q[4][4] = {{r[b][0], r[b][1], r[b][2], r[b][3]}, {r[b + 1][0], r[b + 1][1], r[b + 1][2], r[b + 1][3]},
                           {r[b + 2][0], r[b + 2][1], r[b + 2][2], r[b + 2][3]}, {r[b + 3][0], r[b + 3][1], r[b + 3][2], r[b + 3][3]}};
    tmem_st_16x32(q, taddr + 8 * b);
  }
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void stmatrix_x4_trans(uint32_t addr, uint32_t m0, uint32_t m1, uint32_t m2, uint32_t m3) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(m0), "r"(m1), "r"(m2), "r"(m3) : "memory");
}
// kind::f16 instruction descriptor, fp32 accumulate, bf16 operands; a_mn / b_mn: operand stored MN-major
__host__ __device__ constexpr uint32_t umma_idesc_ab(int M, int N, int a_mn, int b_mn) {
  return umma_idesc(M, N, b_mn) | ((uint32_t)a_mn << 15);
}

template <int DVS>
__global__ void __launch_bounds__(NT + 32, ScanCfg<DVS>::CTAS_PER_SM)
chunk_scan_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmQ,
                  const __grid_constant__ CUtensorMap tmK, ScanParams p) {
  using cfg = ScanCfg<DVS>;
  constexpr int NTW = cfg::NTW, CW = cfg::CW, NS = D / DVS;
  extern __shared__ __align__(1024) uint8_t smem[];
  float* sG = reinterpret_cast<float*>(smem + cfg::OFF_G);
  float* sCf = sG + 2 * C;   // 2^(g_ref(j) - g_j), g_ref(j) = g of the first token of j's block of eight
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + cfg::OFF_BAR + 80);
  const uint32_t sA = smem_u32(smem + cfg::OFF_A), sB = smem_u32(smem + cfg::OFF_B), sKa = smem_u32(smem + cfg::OFF_KA);
  const uint32_t sP = smem_u32(smem + cfg::OFF_P), sUt = smem_u32(smem + cfg::OFF_UT), sUd = smem_u32(smem + cfg::OFF_UD);
  // copies (TMA):            bar_a (W and Q), bar_kb (K beside S^T), bar_ka (K for P3)
  // products done (commit):  bar_t1 (P1), bar_s (P3), bar_pu (PU)
  // operands written:        bar_sr (S^T, all NT compute threads), bar_ut (U~ and U~', chain warps), bar_p (P, output warps)
  const uint32_t bar_a = smem_u32(smem + cfg::OFF_BAR), bar_kb = bar_a + 8, bar_ka = bar_a + 16, bar_t1 = bar_a + 24,
                 bar_s = bar_a + 32, bar_pu = bar_a + 40, bar_sr = bar_a + 48, bar_ut = bar_a + 56, bar_p = bar_a + 64;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool control = warp == 8;
  const int quad = warp & 3, half = (warp >> 2) & 1;
  const bool chain = quad < 2;                   // lanes 0..63 of P1 hold W S
  const int gq = lane >> 2, t = lane & 3;
  const int tok_w = 32 * (quad & 1);             // first token row of this warp in P1 and PU (either role)
  const int krow_w = 32 * quad;                  // first row of S of this warp
  const int cw0 = half * CW;                     // first value column of this warp inside the CTA's slice

  const int slice = blockIdx.x % NS, h = (blockIdx.x / NS) % p.H, s = blockIdx.x / (NS * p.H);
  const int beg = p.seq_off ? p.seq_off[s] : s * p.T;
  const int end = p.seq_off ? p.seq_off[s + 1] : (s + 1) * p.T;
  const int n_chunks = (end - beg + C - 1) / C;
  const int col0 = slice * DVS + cw0;            // this warp's first column in the value dimension

  // State in accumulator-fragment layout: lane group lg (rows krow_w + 16 lg + gq and + 8), n-tile nt
  // (columns cw0 + 8 nt + 2 t and + 1):  S[lg][nt][0..3] = (row, col), (row, col+1), (row+8, col), (row+8, col+1).
  float S[2][NTW][4];
  if (!control) {
#pragma unroll
    for (int lg = 0; lg < 2; ++lg)
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt) {
        const int k = krow_w + 16 * lg + gq, n = col0 + 8 * nt + 2 * t;
        float2 a = make_float2(0.f, 0.f), b = a;
        if (p.S0) {
          const float* s0 = p.S0 + ((size_t)s * p.H + h) * D * D;
          a = *reinterpret_cast<const float2*>(s0 + (size_t)k * D + n);
          b = *reinterpret_cast<const float2*>(s0 + (size_t)(k + 8) * D + n);
        }
        S[lg][nt][0] = a.x; S[lg][nt][1] = a.y; S[lg][nt][2] = b.x; S[lg][nt][3] = b.y;
      }
  }
  auto store_state = [&]() {
    if (!p.S_out || control) return;
    float* dst = p.S_out + ((size_t)s * p.H + h) * D * D;
#pragma unroll
    for (int lg = 0; lg < 2; ++lg)
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt) {
        const int k = krow_w + 16 * lg + gq, n = col0 + 8 * nt + 2 * t;
        *reinterpret_cast<float2*>(dst + (size_t)k * D + n) = make_float2(S[lg][nt][0], S[lg][nt][1]);
        *reinterpret_cast<float2*>(dst + (size_t)(k + 8) * D + n) = make_float2(S[lg][nt][2], S[lg][nt][3]);
      }
  };
  if (n_chunks == 0) { store_state(); return; }
  const bool misaligned = (sA & 1023u) != 0;     // never expected; the swizzle pattern would not match the copies

  // S^T as rows 0..DVS-1 of the K-major B operand of P1: row n = value column, 16-byte pieces of eight key features.
  // stmatrix.trans turns the fragments (rows = features, column pairs) into exactly those pieces.
  auto write_state_operand = [&]() {
    const int mi = lane >> 3, r = lane & 7;      // this lane addresses row r of matrix mi of each x4 store
#pragma unroll
    for (int lg = 0; lg < 2; ++lg)
#pragma unroll
      for (int nt = 0; nt < NTW; nt += 2) {
        // matrices: (features +0..7, tile nt), (features +8..15, tile nt), (+0..7, nt+1), (+8..15, nt+1)
        const int k0 = krow_w + 16 * lg + 8 * (mi & 1);          // first feature of this lane's matrix
        const int n = cw0 + 8 * (nt + (mi >> 1)) + r;            // row of the operand
        const uint32_t addr = sB + (k0 >> 6) * cfg::B_BOX + n * 128 + ((((k0 & 63) >> 3) ^ (n & 7)) << 4);
        stmatrix_x4_trans(addr, pack_bf16(S[lg][nt][0], S[lg][nt][1]), pack_bf16(S[lg][nt][2], S[lg][nt][3]),
                          pack_bf16(S[lg][nt + 1][0], S[lg][nt + 1][1]), pack_bf16(S[lg][nt + 1][2], S[lg][nt + 1][3]));
      }
  };
  auto issue_wq = [&](int tok0) {
    mbar_expect_tx(bar_a, 32768u);
    tma_load_2d(sA, &tmW, bar_a, h * D, tok0);
    tma_load_2d(sA + 8192, &tmQ, bar_a, h * D, tok0);
    tma_load_2d(sA + cfg::A_BOX, &tmW, bar_a, h * D + 64, tok0);
    tma_load_2d(sA + cfg::A_BOX + 8192, &tmQ, bar_a, h * D + 64, tok0);
  };
  auto issue_kb = [&](int tok0) {
    mbar_expect_tx(bar_kb, 16384u);
    tma_load_2d(sB + DVS * 128, &tmK, bar_kb, h * D, tok0);
    tma_load_2d(sB + cfg::B_BOX + DVS * 128, &tmK, bar_kb, h * D + 64, tok0);
  };
  auto issue_ka = [&](int tok0) {
    mbar_expect_tx(bar_ka, 16384u);
    tma_load_2d(sKa, &tmK, bar_ka, h * D, tok0);
    tma_load_2d(sKa + 8192, &tmK, bar_ka, h * D + 64, tok0);
  };
  // U of the chain warps in fragment layout: u[lg][nt][0] = row tok_w + 16 lg + gq, [1] = that row + 8 (bf16 pairs)
  const __nv_bfloat16* Ug = reinterpret_cast<const __nv_bfloat16*>(p.U);
  auto fetch_u = [&](uint32_t (&u)[2][NTW][2], int tok0, int rows) {
#pragma unroll
    for (int lg = 0; lg < 2; ++lg)
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt) {
        const int i = tok_w + 16 * lg + gq, cidx = col0 + 8 * nt + 2 * t;
        u[lg][nt][0] = i < rows ? *reinterpret_cast<const uint32_t*>(Ug + ((size_t)(tok0 + i) * p.H + h) * D + cidx) : 0u;
        u[lg][nt][1] = i + 8 < rows ? *reinterpret_cast<const uint32_t*>(Ug + ((size_t)(tok0 + i + 8) * p.H + h) * D + cidx) : 0u;
      }
  };
  // rows past the sequence end take the last real row's g, so that every exponent stays a difference of real values
  auto fetch_g = [&](int tok0, int rows) -> float {
    const int i = tid < rows ? tid : rows - 1;
    return tid < C ? p.g[(size_t)(tok0 + i) * p.H + h] : 0.f;   // raw: scaled where it is stored, not where it is loaded
  };
  // g * log2(e) of a chunk and its column factors: the decay 2^(g_i - g_j) of P is formed as
  // 2^(g_i - g_ref) * 2^(g_ref - g_j) with g_ref the first token of j's block of eight -- one exponential per
  // (row, block) instead of one per element; the second factor spans at most seven tokens of decay
  auto store_g = [&](int buf, float g_raw) {
    const float gl2 = g_raw * kLog2e;
    const float gref = __shfl_sync(0xffffffffu, gl2, lane & ~7);
    sG[buf * C + tid] = gl2;
    sCf[buf * C + tid] = ex2_approx(gref - gl2);
  };

  uint32_t xr[2][NTW][2];   // chain warps: the next chunk's U (bf16 pairs)
  float g_next = 0.f;
  {
    const int rows0 = end - beg < C ? end - beg : C;
    if (tid == NT) {
      prefetch_tmap(&tmW); prefetch_tmap(&tmQ); prefetch_tmap(&tmK);
      for (int b = 0; b < 6; ++b) mbar_init(bar_a + 8 * b, 1);
      mbar_init(bar_sr, NT);
      mbar_init(bar_ut, NT / 2);
      mbar_init(bar_p, NT / 2);
      fence_mbar_init();
      if (!misaligned) {
        issue_wq(beg);
        issue_kb(beg);
        issue_ka(beg);
      }
    }
    if (!control && chain) fetch_u(xr, beg, rows0);
    if (!control) g_next = fetch_g(beg, rows0);
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(cfg::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (!control) {
    write_state_operand();
    if (tid < C) store_g(0, g_next);
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();   // barriers initialised, tensor memory allocated, first operand of S and first g in place
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmem_w = tmem + ((uint32_t)(32 * quad) << 16);   // this warp's lanes, column 0
  bool failed = misaligned;

  if (control) {
    // ---------------------------------------------------------------- control thread: every tcgen05.mma of the CTA
    if (lane == 0 && !misaligned) {
      constexpr uint32_t idesc_p1 = umma_idesc_ab(128, cfg::N1, 0, 0);   // [W;Q] K-major, [S^T;K] K-major
      constexpr uint32_t idesc_p3 = umma_idesc_ab(128, DVS, 1, 1);       // K tile MN-major, U~' MN-major
      constexpr uint32_t idesc_pu = umma_idesc_ab(128, DVS, 0, 1);       // [any;P] K-major, U~ MN-major
      // descriptors differ from these bases only in the address field (bits 0..13, units of 16 bytes)
      const uint64_t dA = umma_desc(sA, 16, 1024), dB = umma_desc(sB, 16, 1024), dKa = umma_desc(sKa, 8192, 1024),
                     dUd = umma_desc(sUd, 8192, 1024), dUt = umma_desc(sUt, 8192, 1024),
                     dPa = umma_desc(sKa + 8192, 16, 1024);              // 128 rows: second K box, then P
      uint32_t ph = 0;
      for (int c = 0; c < n_chunks; ++c) {
        // the copies land long before the compute threads are done: check them first, S last
        if (!mbar_wait_bounded(bar_a, ph) || !mbar_wait_bounded(bar_kb, ph) || !mbar_wait_bounded(bar_sr, ph)) { failed = true; break; }
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          umma_bf16(tmem + cfg::TM_P1, dA + (((ks >> 2) * cfg::A_BOX + (ks & 3) * 32) >> 4),
                    dB + (((ks >> 2) * cfg::B_BOX + (ks & 3) * 32) >> 4), idesc_p1, ks > 0);
        umma_commit(bar_t1);
        if (!mbar_wait_bounded(bar_ka, ph) || !mbar_wait_bounded(bar_ut, ph)) { failed = true; break; }
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < C / 16; ++ks)   // 16 tokens (2048 bytes of either operand) per step
          umma_bf16(tmem + cfg::TM_DS, dKa + ((ks * 2048) >> 4), dUd + ((ks * 2048) >> 4), idesc_p3, ks > 0);
        umma_commit(bar_s);
        if (!mbar_wait_bounded(bar_p, ph)) { failed = true; break; }
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < C / 16; ++ks)
          umma_bf16(tmem + cfg::TM_PU, dPa + ((ks * 32) >> 4), dUt + ((ks * 2048) >> 4), idesc_pu, 1u);   // on top of gamma_i Q S
        umma_commit(bar_pu);
        ph ^= 1;
      }
    }
  } else {
    // ---------------------------------------------------------------- compute warps
    mbar_arrive(bar_sr);   // the first S^T operand (written before the CTA barrier above)
    uint32_t ph = 0;
    int o_tok0 = 0, o_rows = 0;
    // O = scale * (gamma_i QS + P U~) of the previous chunk (the PU accumulator starts from gamma_i QS): written
    // while the next chunk's first product runs
    auto write_output = [&](uint32_t parity) -> bool {
      if (!mbar_wait_bounded(bar_pu, parity)) return false;
      tc_fence_after();
      __nv_bfloat16* Og = reinterpret_cast<__nv_bfloat16*>(p.O);
#pragma unroll
      for (int lg = 0; lg < 2; ++lg) {
        float pu[NTW][4];
        tmem_ld_frag<NTW>(pu, tmem_w + ((uint32_t)(16 * lg) << 16) + cfg::TM_PU + cw0);
        tmem_wait_ld();
        const int i = tok_w + 16 * lg + gq;
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt) {
          const int cc = col0 + 8 * nt + 2 * t;
          if (i < o_rows)
            *reinterpret_cast<uint32_t*>(Og + ((size_t)(o_tok0 + i) * p.H + h) * D + cc) =
                pack_bf16(p.scale * pu[nt][0], p.scale * pu[nt][1]);
          if (i + 8 < o_rows)
            *reinterpret_cast<uint32_t*>(Og + ((size_t)(o_tok0 + i + 8) * p.H + h) * D + cc) =
                pack_bf16(p.scale * pu[nt][2], p.scale * pu[nt][3]);
        }
      }
      tc_fence_before();
      return true;
    };
    for (int c = 0; c < n_chunks && !misaligned; ++c) {
      const int tok0 = beg + c * C;
      const int rows = end - tok0 < C ? end - tok0 : C;
      const bool has_next = c + 1 < n_chunks;
      const int nx_tok0 = tok0 + C, nx_rows = end - nx_tok0 < C ? end - nx_tok0 : C;
      const float* gb = sG + (c & 1) * C;
      PHASE_BEGIN();
      if (has_next) g_next = fetch_g(nx_tok0, nx_rows);
      if (chain && has_next && t == 0) {
        // next chunk's U rows of this thread into L2 now; the loads into registers follow when this chunk's U is used up
#pragma unroll
        for (int rr = 0; rr < 4; ++rr) {
          const int i = tok_w + 8 * rr + gq;
          if (i < nx_rows) asm volatile("prefetch.global.L2 [%0];" ::"l"(Ug + ((size_t)(nx_tok0 + i) * p.H + h) * D + col0));
        }
      }
      if (!chain && c > 0) {
        if (!write_output(ph ^ 1)) { failed = true; break; }
        if (tid == 64) issue_ka(tok0);   // PU of the last chunk, the last reader of that buffer, has retired
      }
      PHASE(0);

      if (!mbar_wait_bounded(bar_t1, ph)) { failed = true; break; }
      tc_fence_after();
      PHASE(1);
      if (has_next && tid == 32) issue_wq(nx_tok0);    // P1, the only reader of W, Q and of the K beside S^T, has retired
      if (has_next && tid == 96) issue_kb(nx_tok0);
      // (this chunk's g was written by other threads during the last chunk: read only after the wait above,
      // which follows every compute thread's arrival on bar_sr)
      const float g_last = gb[rows - 1];
      if (chain) {
        // ---- U~ = U - W S  ->  bf16 operands U~ and (decay-scaled) U~', [token rows][value columns]
        const int mi = lane >> 3, r = lane & 7;
#pragma unroll
        for (int lg = 0; lg < 2; ++lg) {
          float t1[NTW][4];
          tmem_ld_frag<NTW>(t1, tmem_w + ((uint32_t)(16 * lg) << 16) + cfg::TM_P1 + cw0);
          tmem_wait_ld();
          const int i = tok_w + 16 * lg + gq;
          const float da = ex2_approx(g_last - gb[i]), db = ex2_approx(g_last - gb[i + 8]);
          const bool va = i < rows, vb = i + 8 < rows;
          // the x4 store: matrices (tokens +0..7, tile nt), (tokens +8..15, tile nt), (+0..7, nt+1), (+8..15, nt+1)
          const int tok = tok_w + 16 * lg + 8 * (mi & 1) + r;
#pragma unroll
          for (int nt = 0; nt < NTW; nt += 2) {
            float v[2][4];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const uint32_t wa = xr[lg][nt + q][0], wb = xr[lg][nt + q][1];   // bf16 pairs: low half = first column
              const float2 ua = make_float2(__uint_as_float(wa << 16), __uint_as_float(wa & 0xffff0000u));
              const float2 ub = make_float2(__uint_as_float(wb << 16), __uint_as_float(wb & 0xffff0000u));
              v[q][0] = va ? ua.x - t1[nt + q][0] : 0.f; v[q][1] = va ? ua.y - t1[nt + q][1] : 0.f;
              v[q][2] = vb ? ub.x - t1[nt + q][2] : 0.f; v[q][3] = vb ? ub.y - t1[nt + q][3] : 0.f;
            }
            const int n = cw0 + 8 * (nt + (mi >> 1));   // first column of this lane's matrix
            const uint32_t off = (n >> 6) * 8192 + tok * 128 + ((((n & 63) >> 3) ^ (tok & 7)) << 4);
            stmatrix_x4(sUt + off, pack_bf16(v[0][0], v[0][1]), pack_bf16(v[0][2], v[0][3]), pack_bf16(v[1][0], v[1][1]), pack_bf16(v[1][2], v[1][3]));
            stmatrix_x4(sUd + off, pack_bf16(v[0][0] * da, v[0][1] * da), pack_bf16(v[0][2] * db, v[0][3] * db),
                        pack_bf16(v[1][0] * da, v[1][1] * da), pack_bf16(v[1][2] * db, v[1][3] * db));
          }
        }
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(bar_ut);
        if (tid < C && has_next) store_g((c + 1) & 1, g_next);   // before new loads are issued: waiting for g must not wait for them
        if (has_next) fetch_u(xr, nx_tok0, nx_rows);   // consumed one chunk from now
      } else {
        // ---- P = (Q K^T) * decay, lower triangle with its diagonal; Q S kept for the output
        const float* cf = sCf + (c & 1) * C;
#pragma unroll
        for (int lg = 0; lg < 2; ++lg) {
          float qk[4][4];   // this warp's half of the columns (tokens j): four blocks of eight
          float qsf[NTW][4];
          const uint32_t trow = tmem_w + ((uint32_t)(16 * lg) << 16) + cfg::TM_P1;
          tmem_ld_16x32(qk, trow + DVS + 32 * half);
          tmem_ld_frag<NTW>(qsf, trow + cw0);
          tmem_wait_ld();
          const int ia = tok_w + 16 * lg + gq, ib = ia + 8;
          const float g_a = gb[ia], g_b = gb[ib];
          {
            // gamma_i Q S becomes the starting value of the PU accumulator (same lanes, same columns)
            const float ya = ex2_approx(g_a), yb = ex2_approx(g_b);
#pragma unroll
            for (int nt = 0; nt < NTW; ++nt) { qsf[nt][0] *= ya; qsf[nt][1] *= ya; qsf[nt][2] *= yb; qsf[nt][3] *= yb; }
            tmem_st_frag<NTW>(qsf, tmem_w + ((uint32_t)(16 * lg) << 16) + cfg::TM_PU + cw0);
          }
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const int nt = 4 * half + q4;
            const int j = 8 * nt + 2 * t;
            uint32_t wa = 0u, wb = 0u;
            if (8 * nt <= ib) {   // blocks right of both rows' diagonals are all zero
              const float gref = gb[8 * nt];
              const float2 cj = *reinterpret_cast<const float2*>(cf + j);
              // (row a may lie above this block altogether: its entries are masked, the exponent is not formed)
              const float ea = ex2_approx(8 * nt <= ia ? g_a - gref : 0.f), eb = ex2_approx(g_b - gref);
              const float p0 = j <= ia ? qk[q4][0] * ea * cj.x : 0.f, p1 = j + 1 <= ia ? qk[q4][1] * ea * cj.y : 0.f;
              const float p2 = j <= ib ? qk[q4][2] * eb * cj.x : 0.f, p3 = j + 1 <= ib ? qk[q4][3] * eb * cj.y : 0.f;
              wa = pack_bf16(p0, p1);
              wb = pack_bf16(p2, p3);
            }
            *reinterpret_cast<uint32_t*>(smem + cfg::OFF_P + ia * 128 + ((nt ^ (ia & 7)) << 4) + 4 * t) = wa;
            *reinterpret_cast<uint32_t*>(smem + cfg::OFF_P + ib * 128 + ((nt ^ (ib & 7)) << 4) + 4 * t) = wb;
          }
        }
        tmem_wait_st();
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(bar_p);
        o_tok0 = tok0; o_rows = rows;
      }
      PHASE(2);

      // ---- state update and the bf16 operand for the next chunk
      if (!mbar_wait_bounded(bar_s, ph)) { failed = true; break; }
      tc_fence_after();
      PHASE(3);
      {
        const float gl = ex2_approx(g_last);
#pragma unroll
        for (int lg = 0; lg < 2; ++lg) {
          float ds[NTW][4];
          tmem_ld_frag<NTW>(ds, tmem_w + ((uint32_t)(16 * lg) << 16) + cfg::TM_DS + cw0);
          tmem_wait_ld();
#pragma unroll
          for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) S[lg][nt][e] = fmaf(gl, S[lg][nt][e], ds[nt][e]);
        }
        if (has_next) {
          write_state_operand();   // its reader (P1 of this chunk) retired before bar_t1
          fence_proxy_async();
          tc_fence_before();
          mbar_arrive(bar_sr);
        }
      }
      PHASE(4);
      ph ^= 1;
    }
    if (!chain && !failed && !misaligned && !write_output(ph ^ 1)) failed = true;
  }
  if (failed) atomicMax(p.status, TRI_INV_ERR_DEVICE_TIMEOUT);
  else store_state();
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(cfg::TMEM_COLS) : "memory");
}

constexpr int kSeqsPerLaunch = 960;
struct OffsetBatch {
  int32_t cu[kSeqsPerLaunch + 1];
  int32_t n, first;
};
__global__ void __launch_bounds__(256) seq_offsets_kernel(int* out, const __grid_constant__ OffsetBatch b) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i <= b.n; i += gridDim.x * blockDim.x) out[b.first + i] = b.cu[i];
}

template <int DVS>
cudaError_t launch_scan_one(const ScanParams& p, const CUtensorMap& tmW, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                            cudaStream_t stream) {
  using cfg = ScanCfg<DVS>;
  static std::mutex mu;
  static bool ready[64] = {false};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!ready[dev]) {
      if ((e = cudaFuncSetAttribute(chunk_scan_kernel<DVS>, cudaFuncAttributeMaxDynamicSharedMemorySize, cfg::SMEM)) != cudaSuccess) return e;
      if ((e = cudaFuncSetAttribute(chunk_scan_kernel<DVS>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared)) != cudaSuccess) return e;
      ready[dev] = true;
    }
  }
  const long long grid = (long long)p.n_seqs * p.H * (D / DVS);
  if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
  chunk_scan_kernel<DVS><<<(int)grid, NT + 32, cfg::SMEM, stream>>>(tmW, tmQ, tmK, p);
  return cudaGetLastError();
}

}  // namespace

// The device copy of cu_seqlens (n_seqs + 1 ints), written from kernel parameters: no host-to-device copy.
cudaError_t launch_seq_offsets(int* dev_out, const tri_inv_desc* d, cudaStream_t stream) {
  for (int s0 = 0; s0 <= d->n_seqs; s0 += kSeqsPerLaunch) {
    OffsetBatch b;
    b.first = s0;
    b.n = d->n_seqs - s0 < kSeqsPerLaunch ? d->n_seqs - s0 : kSeqsPerLaunch;
    for (int q = 0; q <= b.n; ++q) b.cu[q] = d->cu_seqlens[s0 + q];
    seq_offsets_kernel<<<(b.n + 256) / 256, 256, 0, stream>>>(dev_out, b);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (s0 + kSeqsPerLaunch >= d->n_seqs) break;
  }
  return cudaSuccess;
}

// bf16 Q, K, W, U with d_k = d_v = 128 and C = 64: two CTAs per (sequence, head), 64 value columns each.  (One CTA
// per head with 128 columns was measured too: the same time per unit of work, at a register count that spills.)
// A launch whose (sequence, head) pairs would leave three quarters of the SMs idle takes four CTAs of 32 columns
// per pair instead, still at most one per SM: the per-chunk chain of a CTA is a little shorter (7 % on one sequence
// of 32 heads), and every output column is computed by the same operations in the same order either way.  With more
// pairs than that the narrow slices would share SMs and repeat the Q K^T part of the first product: measured slower.
cudaError_t launch_chunk_scan(const ScanParams& p, const void* Q, const void* K, const void* W, long long tokens,
                              cudaStream_t stream) {
  CUtensorMap tmW, tmQ, tmK;
  if (!make_tmap(&tmW, W, tokens, p.H, D, C, 2) || !make_tmap(&tmQ, Q, tokens, p.H, D, C, 2) || !make_tmap(&tmK, K, tokens, p.H, D, C, 2))
    return cudaErrorUnknown;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return cudaErrorUnknown;
  if ((long long)p.n_seqs * p.H * 4 <= sms) return launch_scan_one<32>(p, tmW, tmQ, tmK, stream);
  return launch_scan_one<64>(p, tmW, tmQ, tmK, stream);
}

}  // namespace tri_inv
