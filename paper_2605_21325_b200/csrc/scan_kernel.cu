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
// The dependent chain of a chunk is  P1 -> U~' -> P3 -> S.  Warp 8 holds the one thread that issues every product
// and every tile copy; warp 9 brings g; warps 0..7 compute.  Warp w works on tensor-memory lanes 32 (w & 3) .. +31
// and on half (w >> 2) of the value columns; lanes 0..63 carry W S, so warps of quadrants 0 and 1 form U~' and U~
// ("chain warps"), those of quadrants 2 and 3 form P and the output ("output warps"); all eight update their
// part of S.  Hand-offs are mbarriers: commits from the products, one arrival per warp after its operand writes
// (U~' first: the second product, on the chain, needs only that; U~, for the third, follows).
// TMA brings W, Q, K and U.  Both operands of P1 ([W ; Q] and [S^T ; K]) exist twice and are used by the chunks in
// turn: a chunk's copies are issued a whole chunk before its first product (a copy that misses L2 takes most of a
// chunk's time), and the K rows of the B tile stay in place to serve as the MN-major A operand of P3.  g is loaded
// by a warp of its own a chunk ahead, because a compute warp with a global load in flight would also wait for it at
// its next tensor-memory load.
// Every mbarrier wait is bounded; on expiry the CTA raises the status word, frees its tensor memory and returns.
#include "tc_device.cuh"

namespace tri_inv {
namespace {

constexpr int C = 64, D = 128, NT = 256;   // NT compute threads (8 warps) + the control warp + the gate warp
constexpr float kLog2e = 1.4426950408889634f;

// KDA: the per-channel form (one decay per key feature, the KDA row of Table 1).  Its decays are folded into the
// operands beforehand (kda_scan_prep_kernel, scan_kda_prep.cu): with G_ref the middle row of a chunk and G_last its last,
//     W- = W exp(-G_ref),  Q+ = Q exp(G - G_ref),  K- = K exp(G_ref - G),
// P1 = [W- ; Q+] . [(diag(exp G_ref) S) | K-^T] gives W S, (Q exp G) S and the decayed Q K^T at once; P3 = K-^T U~,
// scaled per row by exp(G_last - G_ref), is the state increment (K exp(G_last - G) = K- exp(G_last - G_ref): no second,
// decay-scaled copy of U~, and the K rows of the B tile serve as in the scalar form); S decays by exp(G_last) per row.
// The kernel then differs from the scalar-gate one only in where its operands come from and in a few scalings: the
// S^T operand is scaled per row by exp(G_ref) of the coming chunk, P needs no decay, the state update has two per-row
// factors.
template <int DVS, bool KDA = false>
struct ScanCfg {
  static constexpr int CW = DVS / 2;                     // value columns per compute warp
  static constexpr int NTW = CW / 8;                     // accumulator n-tiles per compute warp
  static constexpr int N1 = DVS + 64;                    // columns of P1
  // Both operands of P1 exist twice, used by the chunks in turn, so that a chunk's copies can start a whole chunk
  // before its first product (a copy that misses L2 takes most of a chunk's time).
  // A operand of P1: [W ; Q], two boxes (64 features each) of 128 rows x 128 B
  static constexpr int OFF_A = 0, A_BOX = 16384, A_TILE = 2 * A_BOX;
  // B operand of P1: [S^T ; K], two boxes of (DVS + 64) rows x 128 B
  static constexpr int OFF_B = 2 * A_TILE, B_BOX = N1 * 128, B_TILE = 2 * B_BOX;
  // (the K rows of the B tile are also the MN-major A operand of P3: the tile stays whole until the chunk after next)
  static constexpr int OFF_P = OFF_B + 2 * B_TILE;       // P, the lower half of PU's A operand; the unused upper half is whatever precedes it
  static constexpr int OFF_UT = OFF_P + 8192;            // U~  bf16 [64 tokens][DVS], boxes of 64 columns (MN-major B)
  static constexpr int U_BYTES = 8192 * (DVS > 64 ? DVS / 64 : 1);   // a narrower slice fills the first DVS columns of one box
  static constexpr int OFF_UD = OFF_UT + U_BYTES;        // U~' bf16, same layout
  static constexpr int OFF_U = OFF_UD + U_BYTES;         // U tiles of two chunks in turn: bf16 [64 tokens][64 columns], as copied
  static constexpr int OFF_G = OFF_U + 2 * 8192;         // g * log2(e): 2 x 64 floats; column factors: 2 x 64 floats
                                                         // per-channel form: exp(G_last), exp(G_ref), exp(G_last - G_ref), 128 floats each, of three chunks in turn
  static constexpr int OFF_BAR = OFF_G + (KDA ? 4608 : 1024);   // 12 mbarriers, tensor-memory slot
  static constexpr int SMEM = OFF_BAR + 128;
  static constexpr int TM_P1 = 0, TM_DS = N1, TM_PU = N1 + DVS;
  static constexpr int TMEM_COLS = (N1 + 2 * DVS) <= 256 ? 256 : 512;
  // 9 warps at the kernel's natural register count fill an SM once (the narrow slice is only launched when its
  // CTAs get an SM each).
  static constexpr int CTAS_PER_SM = 1;
};

template <int NTL>
__device__ __forceinline__ void tmem_ld_frag(float (&r)[NTL][4], uint32_t taddr) {
  if constexpr (NTL == 8) tmem_ld_16x64(r, taddr);
  else if constexpr (NTL == 4) tmem_ld_16x32(r, taddr);
  else tmem_ld_16x16(r, taddr);
}
template <int NTL>
__device__ __forceinline__ void tmem_st_frag(const float (&r)[NTL][4], uint32_t taddr) {
  if constexpr (NTL == 2) tmem_st_16x16(r, taddr);
#pragma unroll
  for (int b = 0; b + 4 <= NTL; b += 4) {
    const float q[4][4] = {{r[b][0], r[b][1], r[b][2], r[b][3]}, {r[b + 1][0], r[b + 1][1], r[b + 1][2], r[b + 1][3]},
                           {r[b + 2][0], r[b + 2][1], r[b + 2][2], r[b + 2][3]}, {r[b + 3][0], r[b + 3][1], r[b + 3][2], r[b + 3][3]}};
    tmem_st_16x32(q, taddr + 8 * b);
  }
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// One arrival for the whole warp: every lane has made its operand writes visible to the async proxy (the caller's
// fences) before the lanes meet; lane 0 then arrives for all of them.  Eight arrivals per hand-off instead of 256
// on one shared-memory word.
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane) {
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& m0, uint32_t& m1, uint32_t& m2, uint32_t& m3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(m0), "=r"(m1), "=r"(m2), "=r"(m3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void stmatrix_x4_trans(uint32_t addr, uint32_t m0, uint32_t m1, uint32_t m2, uint32_t m3) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(m0), "r"(m1), "r"(m2), "r"(m3) : "memory");
}
// kind::f16 instruction descriptor, fp32 accumulate, bf16 operands; a_mn / b_mn: operand stored MN-major
__host__ __device__ constexpr uint32_t umma_idesc_ab(int M, int N, int a_mn, int b_mn) {
  return umma_idesc(M, N, b_mn) | ((uint32_t)a_mn << 15);
}

template <int DVS, bool KDA>
__global__ void __launch_bounds__(NT + 64, ScanCfg<DVS, KDA>::CTAS_PER_SM)
chunk_scan_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmQ,
                  const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmU, ScanParams p) {
  using cfg = ScanCfg<DVS, KDA>;
  constexpr int NTW = cfg::NTW, CW = cfg::CW, NS = D / DVS;
  extern __shared__ __align__(1024) uint8_t smem[];
  float* sG = reinterpret_cast<float*>(smem + cfg::OFF_G);
  float* sCf = sG + 2 * C;   // 2^(g_ref(j) - g_j), g_ref(j) = g of the first token of j's block of eight
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + cfg::OFF_BAR + 80);
  const uint32_t sA = smem_u32(smem + cfg::OFF_A), sB = smem_u32(smem + cfg::OFF_B);
  const uint32_t sP = smem_u32(smem + cfg::OFF_P), sUt = smem_u32(smem + cfg::OFF_UT), sUd = smem_u32(smem + cfg::OFF_UD);
  const uint32_t sU = smem_u32(smem + cfg::OFF_U);
  float* sEl = sG;                 // per-channel form: exp(G_last) [3][128], exp(G_ref) [3][128], exp(G_last - G_ref) [3][128]
  float* sEr = sG + 3 * D;
  float* sEx = sG + 6 * D;
  // copies (TMA):            bar_a (W, Q, the K beside S^T and, per-channel form, K^), bar_u0 / bar_u1 (U, chunks in turn)
  // products done (commit):  bar_t1 (P1), bar_s (P3), bar_pu (PU)
  // operands written:        bar_sr (S^T by the compute warps, the next chunk's g by the gate warp), bar_ut (U~ and U~',
  //                          chain warps), bar_p (P, output warps); one arrival per warp
  const uint32_t bar_a = smem_u32(smem + cfg::OFF_BAR), bar_exit = bar_a + 8, bar_t1 = bar_a + 24,
                 bar_s = bar_a + 32, bar_pu = bar_a + 40, bar_sr = bar_a + 48, bar_ut = bar_a + 56, bar_p = bar_a + 64,
                 bar_u0 = bar_a + 72, bar_u1 = bar_a + 88, bar_ud = bar_a + 96;
  const unsigned long long lim = p.wait_limit_ns ? p.wait_limit_ns : kWaitLimitNs;   // every wait of the kernel gives up after this long
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool control = warp == 8;
  const bool gate_warp = warp == 9;              // brings g of the chunks to come into shared memory
  const bool compute = warp < 8;
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
  if (compute) {
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
    if (!p.S_out || !compute) return;
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
  // (per-channel form: row k of S times er[k], exp(G_ref) of the chunk that will read the operand)
  auto write_state_operand = [&](int buf, const float* er) {
    const int mi = lane >> 3, r = lane & 7;      // this lane addresses row r of matrix mi of each x4 store
#pragma unroll
    for (int lg = 0; lg < 2; ++lg) {
      float ea = 1.f, eb = 1.f;
      if constexpr (KDA) { ea = er[krow_w + 16 * lg + gq]; eb = er[krow_w + 16 * lg + gq + 8]; }
#pragma unroll
      for (int nt = 0; nt < NTW; nt += 2) {
        // matrices: (features +0..7, tile nt), (features +8..15, tile nt), (+0..7, nt+1), (+8..15, nt+1)
        const int k0 = krow_w + 16 * lg + 8 * (mi & 1);          // first feature of this lane's matrix
        const int n = cw0 + 8 * (nt + (mi >> 1)) + r;            // row of the operand
        const uint32_t addr = sB + buf * cfg::B_TILE + (k0 >> 6) * cfg::B_BOX + n * 128 + ((((k0 & 63) >> 3) ^ (n & 7)) << 4);
        stmatrix_x4_trans(addr, pack_bf16(ea * S[lg][nt][0], ea * S[lg][nt][1]), pack_bf16(eb * S[lg][nt][2], eb * S[lg][nt][3]),
                          pack_bf16(ea * S[lg][nt + 1][0], ea * S[lg][nt + 1][1]), pack_bf16(eb * S[lg][nt + 1][2], eb * S[lg][nt + 1][3]));
      }
    }
  };
  // W, Q and the K beside S^T of chunk c, into the tiles of c's parity
  auto issue_wq = [&](int c) {
    const uint32_t dst = sA + (c & 1) * cfg::A_TILE;
    const int tok0 = beg + c * C;
    mbar_expect_tx(bar_a, 32768u + 16384u);   // with the K copy below: one barrier, one wait
    tma_load_2d(dst, &tmW, bar_a, h * D, tok0);
    tma_load_2d(dst + 8192, &tmQ, bar_a, h * D, tok0);
    tma_load_2d(dst + cfg::A_BOX, &tmW, bar_a, h * D + 64, tok0);
    tma_load_2d(dst + cfg::A_BOX + 8192, &tmQ, bar_a, h * D + 64, tok0);
  };
  auto issue_kb = [&](int c) {
    const uint32_t dst = sB + (c & 1) * cfg::B_TILE + DVS * 128;
    const int tok0 = beg + c * C;
    tma_load_2d(dst, &tmK, bar_a, h * D, tok0);
    tma_load_2d(dst + cfg::B_BOX, &tmK, bar_a, h * D + 64, tok0);
  };
  // U of chunk c: the 64-column box that holds this CTA's slice, into the buffer of c's parity
  auto issue_u = [&](int c) {
    const uint32_t bar = (c & 1) ? bar_u1 : bar_u0;
    mbar_expect_tx(bar, 8192u);
    tma_load_2d(sU + (c & 1) * 8192, &tmU, bar, h * D + (slice * DVS) / 64 * 64, beg + c * C);
  };
  // g of a chunk, by the gate warp (lane l: tokens l and l + 32).  Rows past the sequence end take the last real
  // row's g, so that every exponent stays a difference of real values.
  auto fetch_g = [&](int c, float (&gr)[2]) {
    const int tok0 = beg + c * C, rows = end - tok0 < C ? end - tok0 : C;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int i = lane + 32 * q < rows ? lane + 32 * q : rows - 1;
      gr[q] = p.g[(size_t)(tok0 + i) * p.H + h];
    }
  };
  // g * log2(e) of a chunk and its column factors: the decay 2^(g_i - g_j) of P is formed as
  // 2^(g_i - g_ref) * 2^(g_ref - g_j) with g_ref the first token of j's block of eight -- one exponential per
  // (row, block) instead of one per element; the second factor spans at most seven tokens of decay
  auto store_g = [&](int buf, const float (&gr)[2]) {
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const float gl2 = gr[q] * kLog2e;
      const float gref = __shfl_sync(0xffffffffu, gl2, lane & ~7);
      sG[buf * C + lane + 32 * q] = gl2;
      sCf[buf * C + lane + 32 * q] = ex2_approx(gref - gl2);
    }
  };

  // per-channel form: exp(G_last) and exp(G_ref) of a chunk (128 floats each, written by the preparation kernel at the
  // chunk's slot), by the gate warp: lane l brings features 4 l .. 4 l + 3 of both; three chunks' worth are kept in turn
  auto fetch_e = [&](int c, float4 (&ev)[3]) {
    const size_t slot = (size_t)((beg + c * C) / C + s);
    ev[0] = *reinterpret_cast<const float4*>(p.EL + (slot * p.H + h) * D + 4 * lane);
    ev[1] = *reinterpret_cast<const float4*>(p.ER + (slot * p.H + h) * D + 4 * lane);
    ev[2] = *reinterpret_cast<const float4*>(p.EX + (slot * p.H + h) * D + 4 * lane);
  };
  auto store_e = [&](int c, const float4 (&ev)[3]) {
    *reinterpret_cast<float4*>(sEl + (c % 3) * D + 4 * lane) = ev[0];
    *reinterpret_cast<float4*>(sEr + (c % 3) * D + 4 * lane) = ev[1];
    *reinterpret_cast<float4*>(sEx + (c % 3) * D + 4 * lane) = ev[2];
  };
  float4 e_raw[3] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
  float g_raw[2] = {0.f, 0.f};   // gate warp: g of the chunk it stores next
  if (tid == NT) {
    prefetch_tmap(&tmW); prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmU);
    for (int b = 0; b < 6; ++b) mbar_init(bar_a + 8 * b, 1);
    mbar_init(bar_u0, 1);
    mbar_init(bar_u1, 1);
    mbar_init(bar_sr, NT / 32 + 1);   // one arrival per warp (lane 0, after the warp's lanes have fenced and met); the gate warp too
    mbar_init(bar_ud, NT / 64);
    mbar_init(bar_ut, NT / 64);
    mbar_init(bar_p, NT / 64);
    fence_mbar_init();
    if (!misaligned) {
      issue_wq(0);   // (announces the bytes of all three copies on their common barrier)
      issue_kb(0);
      issue_u(0);
    }
  }
  if (gate_warp) {
    if constexpr (KDA) {
      // the vectors of the first two chunks are in place before the loop starts, the third chunk's in registers
      fetch_e(0, e_raw);
      store_e(0, e_raw);
      if (n_chunks > 1) { fetch_e(1, e_raw); store_e(1, e_raw); }
      if (n_chunks > 2) fetch_e(2, e_raw);
    } else {
      fetch_g(0, g_raw);
      store_g(0, g_raw);
      if (n_chunks > 1) fetch_g(1, g_raw);
    }
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(cfg::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (compute && !KDA) write_state_operand(0, nullptr);
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();   // barriers initialised, tensor memory allocated, first operand of S and first g in place
  tc_fence_after();
  if constexpr (KDA) {
    // the first operand of S needs exp(G_ref) of the first chunk, which the gate warp has just stored
    if (compute) {
      write_state_operand(0, sEr);
      fence_proxy_async();
    }
  }
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
      const uint64_t dA = umma_desc(sA, 16, 1024), dB = umma_desc(sB, 16, 1024), dKa = umma_desc(sB + DVS * 128, cfg::B_BOX, 1024),   // the K rows of the B tile, MN-major
                     dUd = umma_desc(sUd, 8192, 1024), dUt = umma_desc(sUt, 8192, 1024),
                     dPa = umma_desc(sP - 8192, 16, 1024);               // 128 rows: 64 of whatever lies before P (results unused), then P
      uint32_t ph = 0;
      int pending = 0;   // chunk whose copies have been requested and not yet seen to land (-1: none)
      for (int c = 0; c < n_chunks; ++c) {
        // the copies land long before the compute threads are done: check them first, S last (one barrier for all of
        // a chunk's copies: every wait costs this thread some 90 cycles, and its phase has to be over anyway before
        // the copies of the next chunk are announced on it, below)
        TL(9);
        if (!mbar_wait_bounded(bar_a, ph, lim)) { failed = true; break; }
        pending = -1;
        TL(7);
        if (!mbar_wait_bounded(bar_sr, ph, lim)) { failed = true; break; }
        tc_fence_after();
        TL(0);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          umma_bf16(tmem + cfg::TM_P1, dA + (((c & 1) * cfg::A_TILE + (ks >> 2) * cfg::A_BOX + (ks & 3) * 32) >> 4),
                    dB + (((c & 1) * cfg::B_TILE + (ks >> 2) * cfg::B_BOX + (ks & 3) * 32) >> 4), idesc_p1, ks > 0);
        umma_commit(bar_t1);
        TL(1);
        // Copies for the next chunk, from this thread so that no compute warp spends issue slots on them.  They go
        // into the other tiles, whose last readers (P1 and P3 of the chunk before this one; for U the chain warps, a
        // chunk ago) were done before the arrivals on bar_sr seen above: nothing to wait for.
        if (c + 1 < n_chunks) {
          issue_wq(c + 1);
          issue_kb(c + 1);
          issue_u(c + 1);
          pending = c + 1;
        }
        TL(2);
        if (!mbar_wait_bounded(bar_ud, ph, lim)) { failed = true; break; }
        tc_fence_after();
        TL(3);
        // self-test (ScanParams::test_stall): the first CTA leaves out this product in its second chunk, so that the
        // waits for it, and then every other wait of the CTA, run out
        if (!(p.test_stall && blockIdx.x == 0 && c == 1)) {
#pragma unroll
          for (int ks = 0; ks < C / 16; ++ks)   // 16 tokens (2048 bytes of either operand) per step
            umma_bf16(tmem + cfg::TM_DS, dKa + (((c & 1) * cfg::B_TILE + ks * 2048) >> 4),
                      (KDA ? dUt : dUd) + ((ks * 2048) >> 4), idesc_p3, ks > 0);   // per-channel form: U~ itself, the decay is in K- and in the update
          umma_commit(bar_s);
        }
        TL(4);
        if (!mbar_wait_bounded(bar_ut, ph, lim) || !mbar_wait_bounded(bar_p, ph, lim)) { failed = true; break; }
        tc_fence_after();
        TL(5);
#pragma unroll
        for (int ks = 0; ks < C / 16; ++ks)
          umma_bf16(tmem + cfg::TM_PU, dPa + ((ks * 32) >> 4), dUt + ((ks * 2048) >> 4), idesc_pu, 1u);   // on top of gamma_i Q S
        umma_commit(bar_pu);
        TL(6);
        ph ^= 1;
      }
      if (failed) {
        // A wait has run out and this CTA is about to give up its shared and tensor memory: what it may still have in
        // flight is waited for first, again with a limit -- the copies requested for the coming chunk (U on its own
        // barrier) and every product issued so far (a commit on a spare barrier).
        if (pending >= 0) {
          mbar_wait_bounded(bar_a, (uint32_t)(pending & 1), lim);
          mbar_wait_bounded((pending & 1) ? bar_u1 : bar_u0, (uint32_t)((pending >> 1) & 1), lim);
        }
        umma_commit(bar_exit);
        mbar_wait_bounded(bar_exit, 0u, lim);
      }
    }
  } else if (gate_warp) {
    // ---------------------------------------------------------------- gate warp: g of chunk c + 1, during chunk c
    // Its arrival on bar_sr tells the control thread, and through the first product's commit every reader, that
    // the chunk's g is in place.  The global loads run a chunk ahead of their use, in a warp that waits for nothing
    // else: a compute warp with a global load in flight would also wait for it at its next tensor-memory load.
    warp_arrive(bar_sr, lane);   // g of the first chunk (written before the CTA barrier above)
    for (int c = 0; c + 1 < n_chunks && !misaligned; ++c) {
      // the buffer of c + 1 held g of c - 1: every compute warp has left that chunk once the arrivals that end it are in
      if (c > 0 && !mbar_wait_bounded(bar_sr, (uint32_t)(c & 1), lim)) { failed = true; break; }
      if constexpr (KDA) {
        // The vectors run one chunk further ahead than g: exp(G_ref) of chunk c + 1 is read at the end of chunk c (it
        // scales the S^T operand), so it has to be in place, and announced by an arrival, a chunk earlier.  Those of
        // c + 2 go where those of c - 1 were.
        if (c + 2 < n_chunks) store_e(c + 2, e_raw);
        warp_arrive(bar_sr, lane);
        if (c + 3 < n_chunks) fetch_e(c + 3, e_raw);
      } else {
        store_g((c + 1) & 1, g_raw);
        warp_arrive(bar_sr, lane);
        if (c + 2 < n_chunks) fetch_g(c + 2, g_raw);
      }
    }
  } else {
    // ---------------------------------------------------------------- compute warps
    warp_arrive(bar_sr, lane);   // the first S^T operand (written before the CTA barrier above)
    uint32_t ph = 0;
    int o_tok0 = 0, o_rows = 0;
    // O = scale * (gamma_i QS + P U~) of the previous chunk (the PU accumulator starts from gamma_i QS): written
    // while the next chunk's first product runs
    auto write_output = [&](uint32_t parity) -> bool {
      if (!mbar_wait_bounded(bar_pu, parity, lim)) return false;
      tc_fence_after();
      __nv_bfloat16* Og = reinterpret_cast<__nv_bfloat16*>(p.O);
      float pu[2][NTW][4];
      tmem_ld_frag<NTW>(pu[0], tmem_w + cfg::TM_PU + cw0);
      tmem_ld_frag<NTW>(pu[1], tmem_w + (16u << 16) + cfg::TM_PU + cw0);
      tmem_wait_ld();
#pragma unroll
      for (int lg = 0; lg < 2; ++lg) {
        const int i = tok_w + 16 * lg + gq;
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt) {
          const int cc = col0 + 8 * nt + 2 * t;
          if (i < o_rows)
            *reinterpret_cast<uint32_t*>(Og + ((size_t)(o_tok0 + i) * p.H + h) * D + cc) =
                pack_bf16(p.scale * pu[lg][nt][0], p.scale * pu[lg][nt][1]);
          if (i + 8 < o_rows)
            *reinterpret_cast<uint32_t*>(Og + ((size_t)(o_tok0 + i + 8) * p.H + h) * D + cc) =
                pack_bf16(p.scale * pu[lg][nt][2], p.scale * pu[lg][nt][3]);
        }
      }
      tc_fence_before();
      return true;
    };
    for (int c = 0; c < n_chunks && !misaligned; ++c) {
      const int tok0 = beg + c * C;
      const int rows = end - tok0 < C ? end - tok0 : C;
      const bool has_next = c + 1 < n_chunks;
      const float* gb = sG + (c & 1) * C;
      TL(0);
      if (!chain && c > 0) {
        if (!write_output(ph ^ 1)) { failed = true; break; }
      }
      TL(1);

      if (!mbar_wait_bounded(bar_t1, ph, lim)) { failed = true; break; }
      tc_fence_after();
      TL(2);
      // (this chunk's g was written by the gate warp during the last chunk: read only after the wait above,
      // which follows that warp's arrival on bar_sr)
      const float g_last = KDA ? 0.f : gb[rows - 1];
      if (chain) {
        // ---- U~ = U - W S  ->  bf16 operands [token rows][value columns]: first the decay-scaled U~' that the chain
        // waits for (its own arrival), then U~ itself for the third product
        const int mi = lane >> 3, r = lane & 7;
        if (!mbar_wait_bounded((c & 1) ? bar_u1 : bar_u0, (uint32_t)((c >> 1) & 1), lim)) { failed = true; break; }   // landed a chunk ago
        TL(3);
        const uint32_t sUc = sU + (c & 1) * 8192;
        const int u_shift = DVS < 64 ? ((slice * DVS) & 63) : 0;   // a narrow slice: which part of the copied 64-column box is ours
        float v[2][NTW][4];
        tmem_ld_frag<NTW>(v[0], tmem_w + cfg::TM_P1 + cw0);
        tmem_ld_frag<NTW>(v[1], tmem_w + (16u << 16) + cfg::TM_P1 + cw0);
        // while those are in flight: U out of its tile the way U~ goes into its own (the same four 8 x 8 matrices per
        // instruction: (tokens +0..7, tile nt), (tokens +8..15, tile nt), (+0..7, nt+1), (+8..15, nt+1)), and the decays
        uint32_t xu[2][NTW][2], off[2][NTW / 2];
        float da[2], db[2];
#pragma unroll
        for (int lg = 0; lg < 2; ++lg) {
          const int tok = tok_w + 16 * lg + 8 * (mi & 1) + r;
#pragma unroll
          for (int nt = 0; nt < NTW; nt += 2) {
            const int n = cw0 + 8 * (nt + (mi >> 1));   // first column of this lane's matrix
            off[lg][nt / 2] = (n >> 6) * 8192 + tok * 128 + ((((n & 63) >> 3) ^ (tok & 7)) << 4);
            ldmatrix_x4(sUc + tok * 128 + (((((n + u_shift) & 63) >> 3) ^ (tok & 7)) << 4), xu[lg][nt][0], xu[lg][nt][1], xu[lg][nt + 1][0], xu[lg][nt + 1][1]);
          }
          const int i = tok_w + 16 * lg + gq;
          if constexpr (!KDA) {
            da[lg] = ex2_approx(g_last - gb[i]);
            db[lg] = ex2_approx(g_last - gb[i + 8]);
          }
        }
        tmem_wait_ld();
        TL(4);
#pragma unroll
        for (int lg = 0; lg < 2; ++lg)
#pragma unroll
          for (int nt = 0; nt < NTW; ++nt) {
            const uint32_t wa = xu[lg][nt][0], wb = xu[lg][nt][1];   // bf16 pairs: low half = first column
            v[lg][nt][0] = __uint_as_float(wa << 16) - v[lg][nt][0];
            v[lg][nt][1] = __uint_as_float(wa & 0xffff0000u) - v[lg][nt][1];
            v[lg][nt][2] = __uint_as_float(wb << 16) - v[lg][nt][2];
            v[lg][nt][3] = __uint_as_float(wb & 0xffff0000u) - v[lg][nt][3];
          }
        if (rows < C) {   // rows past the sequence end count as zero
#pragma unroll
          for (int lg = 0; lg < 2; ++lg) {
            const int i = tok_w + 16 * lg + gq;
            const bool va = i < rows, vb = i + 8 < rows;
#pragma unroll
            for (int nt = 0; nt < NTW; ++nt) {
              v[lg][nt][0] = va ? v[lg][nt][0] : 0.f; v[lg][nt][1] = va ? v[lg][nt][1] : 0.f;
              v[lg][nt][2] = vb ? v[lg][nt][2] : 0.f; v[lg][nt][3] = vb ? v[lg][nt][3] : 0.f;
            }
          }
        }
        if constexpr (!KDA) {
#pragma unroll
          for (int lg = 0; lg < 2; ++lg)
#pragma unroll
            for (int nt = 0; nt < NTW; nt += 2)
              stmatrix_x4(sUd + off[lg][nt / 2], pack_bf16(v[lg][nt][0] * da[lg], v[lg][nt][1] * da[lg]), pack_bf16(v[lg][nt][2] * db[lg], v[lg][nt][3] * db[lg]),
                          pack_bf16(v[lg][nt + 1][0] * da[lg], v[lg][nt + 1][1] * da[lg]), pack_bf16(v[lg][nt + 1][2] * db[lg], v[lg][nt + 1][3] * db[lg]));
          fence_proxy_async();
          tc_fence_before();
          warp_arrive(bar_ud, lane);
        }
        TL(5);
#pragma unroll
        for (int lg = 0; lg < 2; ++lg)
#pragma unroll
          for (int nt = 0; nt < NTW; nt += 2)
            stmatrix_x4(sUt + off[lg][nt / 2], pack_bf16(v[lg][nt][0], v[lg][nt][1]), pack_bf16(v[lg][nt][2], v[lg][nt][3]),
                        pack_bf16(v[lg][nt + 1][0], v[lg][nt + 1][1]), pack_bf16(v[lg][nt + 1][2], v[lg][nt + 1][3]));
        fence_proxy_async();
        if constexpr (KDA) {   // U~ itself is the operand of both later products
          tc_fence_before();
          warp_arrive(bar_ud, lane);
        }
        warp_arrive(bar_ut, lane);
        TL(6);
      } else {
        // ---- P = (Q K^T) * decay, lower triangle with its diagonal; Q S kept for the output
        const float* cf = sCf + (c & 1) * C;
        float qk[2][4][4];   // this warp's half of the columns (tokens j): four blocks of eight
        float qsf[2][NTW][4];
#pragma unroll
        for (int lg = 0; lg < 2; ++lg) {
          const uint32_t trow = tmem_w + ((uint32_t)(16 * lg) << 16) + cfg::TM_P1;
          tmem_ld_16x32(qk[lg], trow + DVS + 32 * half);
          tmem_ld_frag<NTW>(qsf[lg], trow + cw0);
        }
        // what the blocks need from shared memory, while the loads above are in flight
        float gref[4];
        float2 cj[4];
        if constexpr (!KDA) {
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            gref[q4] = gb[8 * (4 * half + q4)];
            cj[q4] = *reinterpret_cast<const float2*>(cf + 8 * (4 * half + q4) + 2 * t);
          }
        }
        tmem_wait_ld();
        TL(3);
#pragma unroll
        for (int lg = 0; lg < 2; ++lg) {
          const int ia = tok_w + 16 * lg + gq, ib = ia + 8;
          const float g_a = KDA ? 0.f : gb[ia], g_b = KDA ? 0.f : gb[ib];
          {
            // gamma_i Q S becomes the starting value of the PU accumulator (same lanes, same columns); in the
            // per-channel form the decay is inside the product already
            if constexpr (!KDA) {
              const float ya = ex2_approx(g_a), yb = ex2_approx(g_b);
#pragma unroll
              for (int nt = 0; nt < NTW; ++nt) { qsf[lg][nt][0] *= ya; qsf[lg][nt][1] *= ya; qsf[lg][nt][2] *= yb; qsf[lg][nt][3] *= yb; }
            }
            tmem_st_frag<NTW>(qsf[lg], tmem_w + ((uint32_t)(16 * lg) << 16) + cfg::TM_PU + cw0);
          }
          // No branch around a block: entries right of a row's diagonal are masked by selection, and the exponent of
          // a row that lies above the whole block is not formed (its argument is replaced by zero), so the four
          // blocks are independent straight-line code that the scheduler can interleave.
          uint32_t wa[4], wb[4];
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const int nt = 4 * half + q4;
            const int j = 8 * nt + 2 * t;
            float p0, p1, p2, p3;
            if constexpr (KDA) {   // the product carries its decay: only the mask is left
              p0 = j <= ia ? qk[lg][q4][0] : 0.f; p1 = j + 1 <= ia ? qk[lg][q4][1] : 0.f;
              p2 = j <= ib ? qk[lg][q4][2] : 0.f; p3 = j + 1 <= ib ? qk[lg][q4][3] : 0.f;
            } else {
              const float ea = ex2_approx(8 * nt <= ia ? g_a - gref[q4] : 0.f), eb = ex2_approx(8 * nt <= ib ? g_b - gref[q4] : 0.f);
              p0 = j <= ia ? qk[lg][q4][0] * ea * cj[q4].x : 0.f; p1 = j + 1 <= ia ? qk[lg][q4][1] * ea * cj[q4].y : 0.f;
              p2 = j <= ib ? qk[lg][q4][2] * eb * cj[q4].x : 0.f; p3 = j + 1 <= ib ? qk[lg][q4][3] * eb * cj[q4].y : 0.f;
            }
            wa[q4] = pack_bf16(p0, p1);
            wb[q4] = pack_bf16(p2, p3);
          }
          // into the K-major operand (row i, 16-byte pieces of eight tokens j, swizzled): two x4 stores of the matrices
          // (rows +0..7, block), (rows +8..15, block), (rows +0..7, block + 1), (rows +8..15, block + 1)
          {
            const int mi = lane >> 3, row = tok_w + 16 * lg + 8 * (mi & 1) + (lane & 7);
#pragma unroll
            for (int q4 = 0; q4 < 4; q4 += 2) {
              const int blk = 4 * half + q4 + (mi >> 1);
              stmatrix_x4(sP + row * 128 + ((blk ^ (row & 7)) << 4), wa[q4], wb[q4], wa[q4 + 1], wb[q4 + 1]);
            }
          }
          if (lg == 0) TL(5);
        }
        tmem_wait_st();
        fence_proxy_async();
        tc_fence_before();
        warp_arrive(bar_p, lane);
        TL(6);
        o_tok0 = tok0; o_rows = rows;
      }

      // ---- state update and the bf16 operand for the next chunk
      if (!mbar_wait_bounded(bar_s, ph, lim)) { failed = true; break; }
      tc_fence_after();
      TL(7);
      {
        const float gl = ex2_approx(g_last);
        float el[2][2], ex[2][2];   // per-channel form: exp(G_last) and exp(G_last - G_ref) of this thread's four rows of S
        if constexpr (KDA) {
#pragma unroll
          for (int lg = 0; lg < 2; ++lg) {
            el[lg][0] = sEl[(c % 3) * D + krow_w + 16 * lg + gq];
            el[lg][1] = sEl[(c % 3) * D + krow_w + 16 * lg + gq + 8];
            ex[lg][0] = sEx[(c % 3) * D + krow_w + 16 * lg + gq];
            ex[lg][1] = sEx[(c % 3) * D + krow_w + 16 * lg + gq + 8];
          }
        }
        float ds[2][NTW][4];
        tmem_ld_frag<NTW>(ds[0], tmem_w + cfg::TM_DS + cw0);
        tmem_ld_frag<NTW>(ds[1], tmem_w + (16u << 16) + cfg::TM_DS + cw0);
        tmem_wait_ld();
#pragma unroll
        for (int lg = 0; lg < 2; ++lg)
#pragma unroll
          for (int nt = 0; nt < NTW; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e)
              S[lg][nt][e] = KDA ? fmaf(el[lg][e >> 1], S[lg][nt][e], ex[lg][e >> 1] * ds[lg][nt][e]) : fmaf(gl, S[lg][nt][e], ds[lg][nt][e]);
        TL(8);
        if (has_next) {
          write_state_operand((c + 1) & 1, sEr + ((c + 1) % 3) * D);   // that tile's last reader was P1 of the chunk before this one
          TL(9);
          fence_proxy_async();
          tc_fence_before();
          warp_arrive(bar_sr, lane);
        }
      }
      TL(10);
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

template <int DVS, bool KDA>
cudaError_t launch_scan_one(const ScanParams& p, const CUtensorMap& tmW, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                            const CUtensorMap& tmU, cudaStream_t stream) {
  using cfg = ScanCfg<DVS, KDA>;
  static std::mutex mu;
  static bool ready[64] = {false};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!ready[dev]) {
      if ((e = cudaFuncSetAttribute(chunk_scan_kernel<DVS, KDA>, cudaFuncAttributeMaxDynamicSharedMemorySize, cfg::SMEM)) != cudaSuccess) return e;
      if ((e = cudaFuncSetAttribute(chunk_scan_kernel<DVS, KDA>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared)) != cudaSuccess) return e;
      ready[dev] = true;
    }
  }
  const long long grid = (long long)p.n_seqs * p.H * (D / DVS);
  if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
  chunk_scan_kernel<DVS, KDA><<<(int)grid, NT + 64, cfg::SMEM, stream>>>(tmW, tmQ, tmK, tmU, p);
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
// kda selects the per-channel form: Q, K, W are then the prepared operands Q+, K-, W- (scan_kda_prep.cu), with p.EL,
// p.ER, p.EX the per-chunk vectors.
cudaError_t launch_chunk_scan(const ScanParams& p, const void* Q, const void* K, const void* W, long long tokens,
                              cudaStream_t stream, bool kda) {
  CUtensorMap tmW, tmQ, tmK, tmU;
  if (!make_tmap(&tmW, W, tokens, p.H, D, C, 2) || !make_tmap(&tmQ, Q, tokens, p.H, D, C, 2) || !make_tmap(&tmK, K, tokens, p.H, D, C, 2) ||
      !make_tmap(&tmU, p.U, tokens, p.H, D, C, 2))
    return cudaErrorUnknown;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return cudaErrorUnknown;
  const bool narrow = (long long)p.n_seqs * p.H * 4 <= sms;
  if (kda) return narrow ? launch_scan_one<32, true>(p, tmW, tmQ, tmK, tmU, stream) : launch_scan_one<64, true>(p, tmW, tmQ, tmK, tmU, stream);
  return narrow ? launch_scan_one<32, false>(p, tmW, tmQ, tmK, tmU, stream) : launch_scan_one<64, false>(p, tmW, tmQ, tmK, tmU, stream);
}

}  // namespace tri_inv
