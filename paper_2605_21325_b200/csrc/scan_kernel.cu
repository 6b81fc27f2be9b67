// Chunk scan: the consumer of W and U.  The chunk form of the layer's recurrence (the re-formulation that
// Sec. 1 refers to; (I+N)^{-1} enters through W and U), per sequence and head, chunk after chunk, with the
// state S [d_k x d_v] carried in registers:
//
//     U~ = U - W S                                   W = A diag(beta exp g) K (decay-weighted), U = A diag(beta) V
//     O  = scale * (diag(gamma) Q S + P U~)          gamma_i = exp(g_i),  P_ij = (q_i . k_j) gamma_i / gamma_j  (j <= i)
//     S <- gamma_last S + K^T diag(gamma_last / gamma) U~
//
// Columns of S (the d_v axis) never mix, so a CTA owns one (sequence, head, slice of DVS value columns) and walks
// the chunks in order; the slices of one head run side by side and share W, Q, K through L2.
//
// Per chunk, on the tensor cores (tcgen05.mma kind::f16, fp32 accumulators in tensor memory):
//   T1 = W S   and  QS = Q S   (B operand: S rounded to bf16, kept K-major in shared memory),
//   QK = Q K^T,   dS = K^T U~' (A operand: the K tile read MN-major; U~' = decay-scaled U~ in bf16),   PU = P U~.
// The dependent chain of a chunk is  T1 -> U~ -> dS -> S;  QS, QK, P and PU hang off it.
// TMA brings the W, Q and K tiles (one buffer each, refilled as soon as their last reader has retired);
// U and g come through registers one chunk ahead.
// Every mbarrier wait is bounded; on expiry the CTA raises the status word, frees its tensor memory and returns.
#include "tc_device.cuh"

namespace tri_inv {
namespace {

#ifdef TRI_INV_PHASE_CLOCKS
#define PHASE_BEGIN() long long ph_t = clock64()
#define PHASE(k)                                                                  \
  do {                                                                            \
    long long now = clock64();                                                    \
    if (blockIdx.x == 0 && (threadIdx.x & 31) == 0) atomicAdd(p.status + 8 + 12 * (threadIdx.x >> 5) + (k), (int)(now - ph_t)); \
    ph_t = now;                                                                   \
  } while (0)
#define SUBPHASE(k) do { long long now = clock64(); atomicAdd(p.status + 64 + (k), (int)(now - sub_t)); sub_t = now; } while (0)
#else
#define PHASE_BEGIN() do {} while (0)
#define PHASE(k) do {} while (0)
#define SUBPHASE(k) do {} while (0)
#endif

constexpr int C = 64, D = 128, NT = 128;
constexpr float kLog2e = 1.4426950408889634f;

template <int DVS>
struct ScanCfg {
  static constexpr int OFF_W = 0, OFF_Q = 16384, OFF_K = 32768;   // bf16 tiles: 2 boxes of 64 rows x 128 B
  static constexpr int OFF_S = 49152;                             // S^T bf16 [DVS rows][128 d_k]: 2 boxes of DVS rows x 128 B
  static constexpr int S_BOX = DVS * 128;
  static constexpr int OFF_UT = OFF_S + 2 * S_BOX;                // U~^T  bf16 [DVS rows][64 tokens]
  static constexpr int OFF_UD = OFF_UT + DVS * 128;               // U~'^T bf16 (rows scaled by gamma_last / gamma_i)
  static constexpr int OFF_P = OFF_UD + DVS * 128;                // P bf16 [64][64]
  static constexpr int OFF_G = OFF_P + 8192;                      // g * log2(e): two buffers of 64 floats, then two of column factors
  static constexpr int OFF_BAR = OFF_G + 1024;                     // 10 mbarriers, tensor-memory slot
  static constexpr int SMEM = OFF_BAR + 96;
  static constexpr int TM_QK = 0, TM_T1 = 64, TM_QS = 64 + DVS, TM_PU = 64 + 2 * DVS, TM_DS = 64 + 3 * DVS;
  static constexpr int TMEM_COLS = (64 + 4 * DVS) <= 256 ? 256 : 512;
  static constexpr int CTAS_PER_SM = TMEM_COLS == 256 ? 2 : 1;
  static constexpr int NTL = DVS / 8;                             // accumulator n-tiles per row block
};

// kind::f16 instruction descriptor with an MN-major A operand (bit 15): A is read as stored [k][m].
__host__ __device__ constexpr uint32_t umma_idesc_amn(int M, int N) { return umma_idesc(M, N, 0) | (1u << 15); }

__device__ __forceinline__ void tmem_ld_16x32(float (&r)[4][4], uint32_t taddr) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=f"(r[0][0]), "=f"(r[0][1]), "=f"(r[0][2]), "=f"(r[0][3]), "=f"(r[1][0]), "=f"(r[1][1]), "=f"(r[1][2]), "=f"(r[1][3]),
        "=f"(r[2][0]), "=f"(r[2][1]), "=f"(r[2][2]), "=f"(r[2][3]), "=f"(r[3][0]), "=f"(r[3][1]), "=f"(r[3][2]), "=f"(r[3][3])
      : "r"(taddr));
}
template <int NTL>
__device__ __forceinline__ void tmem_ld_frag(float (&r)[NTL][4], uint32_t taddr) {
  if constexpr (NTL == 8) tmem_ld_16x64(r, taddr);
  else tmem_ld_16x32(r, taddr);
}
// 32 lanes x 32 columns: thread = lane, 32 consecutive columns
__device__ __forceinline__ void tmem_ld_32x32(float* r, uint32_t taddr) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7]), "=f"(r[8]), "=f"(r[9]), "=f"(r[10]),
        "=f"(r[11]), "=f"(r[12]), "=f"(r[13]), "=f"(r[14]), "=f"(r[15]), "=f"(r[16]), "=f"(r[17]), "=f"(r[18]), "=f"(r[19]), "=f"(r[20]),
        "=f"(r[21]), "=f"(r[22]), "=f"(r[23]), "=f"(r[24]), "=f"(r[25]), "=f"(r[26]), "=f"(r[27]), "=f"(r[28]), "=f"(r[29]), "=f"(r[30]),
        "=f"(r[31])
      : "r"(taddr));
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

template <int DVS>
__global__ void __launch_bounds__(NT + 32, ScanCfg<DVS>::CTAS_PER_SM)
chunk_scan_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmQ,
                  const __grid_constant__ CUtensorMap tmK, ScanParams p) {
  using cfg = ScanCfg<DVS>;
  constexpr int NTL = cfg::NTL, NS = D / DVS;
  extern __shared__ __align__(1024) uint8_t smem[];
  float* sG = reinterpret_cast<float*>(smem + cfg::OFF_G);
  float* sCf = sG + 2 * C;   // 2^(g_ref(j) - g_j), g_ref(j) = g of the first token of j's block of eight
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + cfg::OFF_BAR + 88);
  const uint32_t sW = smem_u32(smem + cfg::OFF_W), sQ = smem_u32(smem + cfg::OFF_Q), sK = smem_u32(smem + cfg::OFF_K);
  const uint32_t sS = smem_u32(smem + cfg::OFF_S), sUt = smem_u32(smem + cfg::OFF_UT), sUd = smem_u32(smem + cfg::OFF_UD);
  const uint32_t sP = smem_u32(smem + cfg::OFF_P);
  // copies (TMA):            bar_w, bar_q, bar_k
  // products done (commit):  bar_t1 (W S), bar_o (Q S, Q K^T), bar_s (K^T U~'), bar_pu (P U~)
  // operands written (128 arrivals of the compute threads): bar_sr (S^T), bar_ut (U~^T, U~'^T), bar_p (P)
  const uint32_t bar_w = smem_u32(smem + cfg::OFF_BAR), bar_q = bar_w + 8, bar_k = bar_w + 16, bar_t1 = bar_w + 24,
                 bar_o = bar_w + 32, bar_s = bar_w + 40, bar_pu = bar_w + 48, bar_sr = bar_w + 56, bar_ut = bar_w + 64,
                 bar_p = bar_w + 72;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool control = warp == 4;               // warp 4: one thread issues every product; warps 0..3 compute
  const int gq = lane >> 2, t = lane & 3;
  const int ra = 16 * (warp & 3) + gq, rb = ra + 8;   // this thread's two rows of every M = 64 accumulator

  const int slice = blockIdx.x % NS, h = (blockIdx.x / NS) % p.H, s = blockIdx.x / (NS * p.H);
  const int beg = p.seq_off ? p.seq_off[s] : s * p.T;
  const int end = p.seq_off ? p.seq_off[s + 1] : (s + 1) * p.T;
  const int n_chunks = (end - beg + C - 1) / C;
  const int col0 = slice * DVS;                  // first value column of this CTA

  // state: compute thread tid owns row tid (a key feature) of S, DVS columns
  float S[DVS];
  if (!control) {
    const float* s0 = p.S0 ? p.S0 + (((size_t)s * p.H + h) * D + tid) * D + col0 : nullptr;
#pragma unroll
    for (int n = 0; n < DVS; n += 4) {
      float4 v = s0 ? *reinterpret_cast<const float4*>(s0 + n) : make_float4(0.f, 0.f, 0.f, 0.f);
      S[n] = v.x; S[n + 1] = v.y; S[n + 2] = v.z; S[n + 3] = v.w;
    }
  }
  auto store_state = [&]() {
    if (!p.S_out || control) return;
    float* dst = p.S_out + (((size_t)s * p.H + h) * D + tid) * D + col0;
#pragma unroll
    for (int n = 0; n < DVS; n += 4) *reinterpret_cast<float4*>(dst + n) = make_float4(S[n], S[n + 1], S[n + 2], S[n + 3]);
  };
  if (n_chunks == 0) { store_state(); return; }
  const bool misaligned = (sW & 1023u) != 0;     // never expected; the swizzle pattern would not match the copies

  // S^T as the K-major B operand: element (n, k) of a [DVS rows][128] bf16 tile, two boxes of 64 features
  auto write_state_operand = [&]() {
    uint8_t* base = smem + cfg::OFF_S + (tid >> 6) * cfg::S_BOX + (tid & 7) * 2;
    const int kc = (tid & 63) >> 3;
#pragma unroll
    for (int n = 0; n < DVS; ++n)
      *reinterpret_cast<__nv_bfloat16*>(base + n * 128 + ((kc ^ (n & 7)) << 4)) = __float2bfloat16_rn(S[n]);
  };
  auto issue_tile = [&](uint32_t dst, const CUtensorMap* tm, uint32_t bar, int tok0) {
    mbar_expect_tx(bar, 16384u);
    tma_load_2d(dst, tm, bar, h * D, tok0);
    tma_load_2d(dst + 8192, tm, bar, h * D + 64, tok0);
  };
  const __nv_bfloat16* Ug = reinterpret_cast<const __nv_bfloat16*>(p.U);
  auto fetch_u = [&](uint32_t (&u)[NTL][2], int tok0, int rows) {
#pragma unroll
    for (int nt = 0; nt < NTL; ++nt) {
      const int c = col0 + 8 * nt + 2 * t;
      u[nt][0] = ra < rows ? *reinterpret_cast<const uint32_t*>(Ug + ((size_t)(tok0 + ra) * p.H + h) * D + c) : 0u;
      u[nt][1] = rb < rows ? *reinterpret_cast<const uint32_t*>(Ug + ((size_t)(tok0 + rb) * p.H + h) * D + c) : 0u;
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
  uint32_t u_next[NTL][2];
  float g_next = 0.f;
  {
    const int rows0 = end - beg < C ? end - beg : C;
    if (tid == NT) {
      prefetch_tmap(&tmW); prefetch_tmap(&tmQ); prefetch_tmap(&tmK);
      for (int b = 0; b < 7; ++b) mbar_init(bar_w + 8 * b, 1);
      for (int b = 7; b < 10; ++b) mbar_init(bar_w + 8 * b, NT);
      fence_mbar_init();
      if (!misaligned) {
        issue_tile(sW, &tmW, bar_w, beg);
        issue_tile(sQ, &tmQ, bar_q, beg);
        issue_tile(sK, &tmK, bar_k, beg);
      }
    }
    if (!control) {
      fetch_u(u_next, beg, rows0);
      g_next = fetch_g(beg, rows0);
    }
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
  const uint32_t tmem_rows = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
  bool failed = misaligned;

  if (control) {
    // ---------------------------------------------------------------- control thread: every tcgen05.mma of the CTA
    if (lane == 0 && !misaligned) {
      constexpr uint32_t idesc_n = umma_idesc(C, DVS, 0), idesc_qk = umma_idesc(C, C, 0), idesc_ds = umma_idesc_amn(D, DVS);
      // descriptors differ from these bases only in the address field (bits 0..13, units of 16 bytes)
      const uint64_t dW = umma_desc(sW, 16, 1024), dQ = umma_desc(sQ, 16, 1024), dK = umma_desc(sK, 16, 1024),
                     dS = umma_desc(sS, 16, 1024), dKt = umma_desc(sK, 8192, 1024), dUd = umma_desc(sUd, 16, 1024),
                     dP = umma_desc(sP, 16, 1024), dUt = umma_desc(sUt, 16, 1024);
      auto mma_k128 = [&](uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t b_box, uint32_t idesc) {
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks)
          umma_bf16(d_tmem, a + (((ks >> 2) * 8192 + (ks & 3) * 32) >> 4), b + (((ks >> 2) * b_box + (ks & 3) * 32) >> 4), idesc, ks > 0);
      };
      uint32_t ph = 0;
      for (int c = 0; c < n_chunks; ++c) {
        // T1 = W S: the head of the chunk's dependent chain, issued first
        if (!mbar_wait_bounded(bar_sr, ph) || !mbar_wait_bounded(bar_w, ph)) { failed = true; break; }
        tc_fence_after();
        mma_k128(tmem + cfg::TM_T1, dW, dS, cfg::S_BOX, idesc_n);
        umma_commit(bar_t1);
        if (!mbar_wait_bounded(bar_q, ph) || !mbar_wait_bounded(bar_k, ph)) { failed = true; break; }
        tc_fence_after();
        mma_k128(tmem + cfg::TM_QK, dQ, dK, 8192, idesc_qk);
        mma_k128(tmem + cfg::TM_QS, dQ, dS, cfg::S_BOX, idesc_n);
        umma_commit(bar_o);
        // dS = K^T U~' as soon as the compute threads have written U~'
        if (!mbar_wait_bounded(bar_ut, ph)) { failed = true; break; }
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < C / 16; ++ks)   // K tile read MN-major: 16 tokens (2048 bytes) per step
          umma_bf16(tmem + cfg::TM_DS, dKt + ((ks * 2048) >> 4), dUd + ((ks * 32) >> 4), idesc_ds, ks > 0);
        umma_commit(bar_s);
        if (!mbar_wait_bounded(bar_p, ph)) { failed = true; break; }
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < C / 16; ++ks)
          umma_bf16(tmem + cfg::TM_PU, dP + ((ks * 32) >> 4), dUt + ((ks * 32) >> 4), idesc_n, ks > 0);
        umma_commit(bar_pu);
        ph ^= 1;
      }
    }
  } else {
    // ---------------------------------------------------------------- compute warps
    mbar_arrive(bar_sr);   // the first S^T operand (written before the CTA barrier above)
    uint32_t ph = 0;
    float qs[NTL][4];      // Q S of the chunk whose output is still to be written
    float o_sa = 0.f, o_sb = 0.f;
    int o_tok0 = 0, o_rows = 0;
    // O = scale * (gamma_i QS + PU) of the previous chunk: written while the next chunk's first product runs
    auto write_output = [&](uint32_t parity) -> bool {
      if (!mbar_wait_bounded(bar_pu, parity)) return false;
      tc_fence_after();
      float pu[NTL][4];
      tmem_ld_frag<NTL>(pu, tmem_rows + cfg::TM_PU);
      tmem_wait_ld();
      __nv_bfloat16* Og = reinterpret_cast<__nv_bfloat16*>(p.O);
#pragma unroll
      for (int nt = 0; nt < NTL; ++nt) {
        const int cc = col0 + 8 * nt + 2 * t;
        if (ra < o_rows)
          *reinterpret_cast<uint32_t*>(Og + ((size_t)(o_tok0 + ra) * p.H + h) * D + cc) =
              pack_bf16(fmaf(o_sa, qs[nt][0], p.scale * pu[nt][0]), fmaf(o_sa, qs[nt][1], p.scale * pu[nt][1]));
        if (rb < o_rows)
          *reinterpret_cast<uint32_t*>(Og + ((size_t)(o_tok0 + rb) * p.H + h) * D + cc) =
              pack_bf16(fmaf(o_sb, qs[nt][2], p.scale * pu[nt][2]), fmaf(o_sb, qs[nt][3], p.scale * pu[nt][3]));
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
      uint32_t u_cur[NTL][2];
#pragma unroll
      for (int nt = 0; nt < NTL; ++nt) { u_cur[nt][0] = u_next[nt][0]; u_cur[nt][1] = u_next[nt][1]; }
      if (has_next) {
        fetch_u(u_next, nx_tok0, nx_rows);
        g_next = fetch_g(nx_tok0, nx_rows);
      }
      if (c > 0 && !write_output(ph ^ 1)) { failed = true; break; }
      PHASE(0);

      // ---- U~ = U - W S  ->  bf16 operands U~^T and (decay-scaled) U~'^T
      if (!mbar_wait_bounded(bar_t1, ph)) { failed = true; break; }
      tc_fence_after();
      PHASE(1);
      // (this chunk's g was written by other threads during the last chunk: read only after the wait above,
      // which follows every compute thread's arrival on bar_sr)
      const float g_a = gb[ra], g_b = gb[rb], g_last = gb[rows - 1];
      if (tid == 32 && has_next) issue_tile(sW, &tmW, bar_w, nx_tok0);   // W's only reader has retired
      {
        float t1[NTL][4];
        tmem_ld_frag<NTL>(t1, tmem_rows + cfg::TM_T1);
        tmem_wait_ld();
        const float da = ex2_approx(g_last - g_a), db = ex2_approx(g_last - g_b);
        const int ca = ra >> 3, cb = rb >> 3;
#pragma unroll
        for (int nt = 0; nt < NTL; ++nt) {
          const float2 ua = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u_cur[nt][0]));
          const float2 ub = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u_cur[nt][1]));
          const float v0 = ra < rows ? ua.x - t1[nt][0] : 0.f, v1 = ra < rows ? ua.y - t1[nt][1] : 0.f;
          const float v2 = rb < rows ? ub.x - t1[nt][2] : 0.f, v3 = rb < rows ? ub.y - t1[nt][3] : 0.f;
          const int n0 = 8 * nt + 2 * t, n1 = n0 + 1;
          // element (n, token) of a [DVS rows][64 tokens] bf16 tile, 128-byte rows, 16-byte pieces swizzled by the row
          const uint32_t o0a = n0 * 128 + ((ca ^ (n0 & 7)) << 4) + (ra & 7) * 2, o1a = n1 * 128 + ((ca ^ (n1 & 7)) << 4) + (ra & 7) * 2;
          const uint32_t o0b = n0 * 128 + ((cb ^ (n0 & 7)) << 4) + (rb & 7) * 2, o1b = n1 * 128 + ((cb ^ (n1 & 7)) << 4) + (rb & 7) * 2;
          *reinterpret_cast<__nv_bfloat16*>(smem + cfg::OFF_UD + o0a) = __float2bfloat16_rn(v0 * da);
          *reinterpret_cast<__nv_bfloat16*>(smem + cfg::OFF_UD + o1a) = __float2bfloat16_rn(v1 * da);
          *reinterpret_cast<__nv_bfloat16*>(smem + cfg::OFF_UD + o0b) = __float2bfloat16_rn(v2 * db);
          *reinterpret_cast<__nv_bfloat16*>(smem + cfg::OFF_UD + o1b) = __float2bfloat16_rn(v3 * db);
          *reinterpret_cast<__nv_bfloat16*>(smem + cfg::OFF_UT + o0a) = __float2bfloat16_rn(v0);
          *reinterpret_cast<__nv_bfloat16*>(smem + cfg::OFF_UT + o1a) = __float2bfloat16_rn(v1);
          *reinterpret_cast<__nv_bfloat16*>(smem + cfg::OFF_UT + o0b) = __float2bfloat16_rn(v2);
          *reinterpret_cast<__nv_bfloat16*>(smem + cfg::OFF_UT + o1b) = __float2bfloat16_rn(v3);
        }
      }
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive(bar_ut);
      PHASE(2);

      // ---- P = (Q K^T) * decay, lower triangle with its diagonal (while K^T U~' runs); QS kept for the output
      if (!mbar_wait_bounded(bar_o, ph)) { failed = true; break; }
      tc_fence_after();
      PHASE(3);
      if (tid == 64 && has_next) issue_tile(sQ, &tmQ, bar_q, nx_tok0);   // Q's readers have retired
      {
        float qk[8][4];
        tmem_ld_16x64(qk, tmem_rows + cfg::TM_QK);
        tmem_ld_frag<NTL>(qs, tmem_rows + cfg::TM_QS);
        tmem_wait_ld();
        const float* cf = sCf + (c & 1) * C;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          const int j = 8 * nt + 2 * t;
          uint32_t wa = 0u, wb = 0u;
          if (8 * nt <= rb) {   // blocks right of both rows' diagonals are all zero
            const float gref = gb[8 * nt];
            const float2 cj = *reinterpret_cast<const float2*>(cf + j);
            const float ea = ex2_approx(fminf(g_a - gref, 0.f)), eb = ex2_approx(g_b - gref);
            const float p0 = j <= ra ? qk[nt][0] * ea * cj.x : 0.f, p1 = j + 1 <= ra ? qk[nt][1] * ea * cj.y : 0.f;
            const float p2 = j <= rb ? qk[nt][2] * eb * cj.x : 0.f, p3 = j + 1 <= rb ? qk[nt][3] * eb * cj.y : 0.f;
            wa = pack_bf16(p0, p1);
            wb = pack_bf16(p2, p3);
          }
          *reinterpret_cast<uint32_t*>(smem + cfg::OFF_P + ra * 128 + ((nt ^ (ra & 7)) << 4) + 4 * t) = wa;
          *reinterpret_cast<uint32_t*>(smem + cfg::OFF_P + rb * 128 + ((nt ^ (rb & 7)) << 4) + 4 * t) = wb;
        }
      }
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive(bar_p);
      o_sa = p.scale * ex2_approx(g_a); o_sb = p.scale * ex2_approx(g_b);
      o_tok0 = tok0; o_rows = rows;
      if (tid < C && has_next) store_g((c + 1) & 1, g_next);
      PHASE(4);

      // ---- state update (thread = row of S) and the bf16 operand for the next chunk
      if (!mbar_wait_bounded(bar_s, ph)) { failed = true; break; }
      tc_fence_after();
      PHASE(5);
      if (tid == 96 && has_next) issue_tile(sK, &tmK, bar_k, nx_tok0);   // K's readers (Q K^T, K^T U~') have retired
      {
        const float gl = ex2_approx(g_last);
#pragma unroll
        for (int n0 = 0; n0 < DVS; n0 += 32) {
          float ds[32];
          tmem_ld_32x32(ds, tmem_rows + cfg::TM_DS + n0);
          tmem_wait_ld();
#pragma unroll
          for (int n = 0; n < 32; ++n) S[n0 + n] = fmaf(gl, S[n0 + n], ds[n]);
        }
        if (has_next) {
          write_state_operand();   // its readers (W S, Q S of this chunk) retired before bar_s
          fence_proxy_async();
          tc_fence_before();
          mbar_arrive(bar_sr);
        }
      }
      PHASE(6);
      ph ^= 1;
    }
    if (!failed && !misaligned && !write_output(ph ^ 1)) failed = true;
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

// bf16 Q, K, W, U with d_k = d_v = 128 and C = 64.  32 value columns per CTA (two CTAs per SM) unless the batch
// alone fills the GPU twice over, in which case 64 columns per CTA halve the re-reads of W, Q and K through L2.
cudaError_t launch_chunk_scan(const ScanParams& p, const void* Q, const void* K, const void* W, long long tokens,
                              cudaStream_t stream) {
  CUtensorMap tmW, tmQ, tmK;
  if (!make_tmap(&tmW, W, tokens, p.H, D, C, 2) || !make_tmap(&tmQ, Q, tokens, p.H, D, C, 2) || !make_tmap(&tmK, K, tokens, p.H, D, C, 2))
    return cudaErrorUnknown;
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if ((long long)p.n_seqs * p.H * 2 >= 2LL * sms) return launch_scan_one<64>(p, tmW, tmQ, tmK, stream);
  return launch_scan_one<32>(p, tmW, tmQ, tmK, stream);
}

}  // namespace tri_inv
