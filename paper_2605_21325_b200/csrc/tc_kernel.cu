// Tensor-core kernel for bf16 keys/values (sm_100a).
//
// One CTA works on one chunk matrix at a time (grid-stride over all (chunk, head) items),
// one warp per 16 rows.  Per item:
//   1. TMA (cp.async.bulk.tensor, 128-byte swizzle) stages the C x d tiles of K and V in
//      shared memory; beta and g come in with plain loads.
//   2. Gram tiles S = K K^T on or below the diagonal: bf16 MMA (m16n8k16), fp32 accumulate.
//   3. Gate + strict-lower mask in registers, N written to shared memory in fp32.
//   4. 16x16 leaves inverted by forward substitution, one lane per column (Sec. 3.1).
//   5. Block-recursive merges X21 = -(X22 N21) X11 for b = 16, 32, (64) as TF32 MMAs
//      (m16n8k8, fp32 accumulate) on fp32 data kept in shared memory (Sec. 3.3).
//   6. A stored with 16-byte coalesced stores; upper triangle and diagonal are constants.
//   7. W = (A diag(beta)) K and U = (A diag(beta)) V: bf16 MMA with the K / V tiles still in
//      shared memory as the B operand; results leave as 16-byte stores straight from registers.
// Inputs of the inversion stay fp32 in shared memory; only the Gram product and the WY
// apply see bf16 operands (the Gram operands are the bf16 inputs themselves, so exact).
#include <cuda.h>

#include <mutex>

#include "common.cuh"

namespace tri_inv {
namespace {

// ------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls (each poll itself blocks for a
// hardware-defined time slice), so a lost copy cannot hang the GPU.
constexpr uint32_t kSpinLimit = 1u << 22;
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(tm), "r"(bar), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_tf32(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Optional per-phase cycle counters (development builds only: -DTRI_INV_PHASE_CLOCKS).
#ifdef TRI_INV_PHASE_CLOCKS
#define PHASE_BEGIN() long long ph_t = clock64()
#define PHASE(k)                                                                  \
  do {                                                                            \
    long long now = clock64();                                                    \
    if (blockIdx.x == 0 && (threadIdx.x & 31) == 0) atomicAdd(p.status + 8 + 8 * (threadIdx.x >> 5) + (k), (int)(now - ph_t)); \
    ph_t = now;                                                                   \
  } while (0)
#else
#define PHASE_BEGIN() do {} while (0)
#define PHASE(k) do {} while (0)
#endif

// ------------------------------------------------------------------------------------------ layout
template <int C, int D>
struct Cfg {
  static constexpr int NW = C / 16;             // warps, one per 16 rows
  static constexpr int NT = NW * 32;
  static constexpr int LD = C + 4;              // fp32 row length of the N/X matrix (LD % 16 == 4)
  static constexpr int NBOX = D / 64;           // TMA boxes per tile: 64 features (128 B) wide
  static constexpr int BOX_BYTES = C * 128;
  static constexpr int TILE_BYTES = NBOX * BOX_BYTES;
  static constexpr int OFF_K = 0;
  static constexpr int OFF_V = TILE_BYTES;
  static constexpr int OFF_X = 2 * TILE_BYTES;
  static constexpr int OFF_BETA = OFF_X + C * LD * 4;
  static constexpr int OFF_G = OFF_BETA + C * 4;
  static constexpr int OFF_BAR = OFF_G + C * 4;
  static constexpr int BYTES = OFF_BAR + 16;
  static constexpr int SMEM = BYTES + 1024;     // slack to align the base to 1024 B (swizzle atom)
};

// Byte offset of the 16-byte chunk holding features [f, f+8) of row r inside a swizzled tile.
template <int C>
__device__ __forceinline__ uint32_t tile_off(int r, int f) {
  int box = f >> 6, c = (f & 63) >> 3;
  return (uint32_t)(box * (C * 128) + r * 128 + ((c ^ (r & 7)) << 4));
}

// One merge level of the block recursion: for every adjacent pair of B x B diagonal blocks,
// X21 = -(X22 . N21) . X11.  Two warps share each 16-row slab of X21 and split its columns.
template <int C, int B>
__device__ __forceinline__ void merge_level(float* sX, int warp, int lane) {
  constexpr int LD = C + 4;
  constexpr int MT = B / 16;   // 16-row slabs per X21 block
  constexpr int NTT = B / 8;   // n-tiles (and k-steps) across a block
  constexpr int NTR = B / 16;  // n-tiles of the result this warp owns
  const int g = lane >> 2, t = lane & 3;
  const int mt = warp >> 1, nh = warp & 1;
  const int pair = mt / MT, ml = mt - pair * MT;
  const int c0 = pair * 2 * B, r0 = c0 + B, R0 = r0 + 16 * ml;

  float T[NTT][4];
#pragma unroll
  for (int i = 0; i < NTT; ++i) { T[i][0] = T[i][1] = T[i][2] = T[i][3] = 0.f; }
  // T = X22[slab] . N21 ; X22 is lower triangular: slab ml needs k < 16 (ml + 1)
#pragma unroll
  for (int q = 0; q < NTT; ++q) {
    if (q < 2 * (ml + 1)) {
      const float* ap = sX + (R0 + g) * LD + r0 + 8 * q + t;
      uint32_t a0 = to_tf32(ap[0]), a1 = to_tf32(ap[8 * LD]), a2 = to_tf32(ap[4]), a3 = to_tf32(ap[8 * LD + 4]);
      const float* bp = sX + (r0 + 8 * q + t) * LD + c0 + g;
#pragma unroll
      for (int nt = 0; nt < NTT; ++nt) {
        uint32_t b0 = to_tf32(bp[8 * nt]), b1 = to_tf32(bp[4 * LD + 8 * nt]);
        mma_tf32(T[nt], a0, a1, a2, a3, b0, b1);
      }
    }
  }
  // R = T . X11[:, my columns].  T's accumulator fragment is reused as the A operand with the
  // k index permuted (slot t <-> k = 2t, slot t+4 <-> k = 2t+1); B rows are read with the same map.
  float R[NTR][4];
#pragma unroll
  for (int j = 0; j < NTR; ++j) {
    R[j][0] = R[j][1] = R[j][2] = R[j][3] = 0.f;
    const int nt = nh * NTR + j;
#pragma unroll
    for (int q = 0; q < NTT; ++q) {
      if (q >= nt) {  // X11 lower triangular: rows k >= column
        const float* bp = sX + (c0 + 8 * q + 2 * t) * LD + c0 + 8 * nt + g;
        uint32_t b0 = to_tf32(bp[0]), b1 = to_tf32(bp[LD]);
        mma_tf32(R[j], to_tf32(T[q][0]), to_tf32(T[q][2]), to_tf32(T[q][1]), to_tf32(T[q][3]), b0, b1);
      }
    }
  }
  __syncthreads();  // every warp has finished reading N21 before anyone overwrites it
#pragma unroll
  for (int j = 0; j < NTR; ++j) {
    const int col = c0 + 8 * (nh * NTR + j) + 2 * t;
    *reinterpret_cast<float2*>(sX + (R0 + g) * LD + col) = make_float2(-R[j][0], -R[j][1]);
    *reinterpret_cast<float2*>(sX + (R0 + g + 8) * LD + col) = make_float2(-R[j][2], -R[j][3]);
  }
  __syncthreads();
}

// W (or U) = A' . tile for this warp's 16 rows; A' fragments are already scaled by beta and in bf16.
template <int C, int D>
__device__ __forceinline__ void wy_apply(const uint32_t (&af)[C / 16][4], uint32_t tile, int warp, int lane,
                                         __nv_bfloat16* out, long long tok0, int rows, int h, int H) {
  constexpr int NTN = D / 8;
  float acc[NTN][4];
#pragma unroll
  for (int i = 0; i < NTN; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }
  const int krow_l = (lane & 7) + 8 * ((lane >> 3) & 1);
  const int ncol_l = 8 * (lane >> 4);
#pragma unroll
  for (int ks = 0; ks < C / 16; ++ks) {
    if (ks <= warp) {
#pragma unroll
      for (int np = 0; np < NTN / 2; ++np) {
        uint32_t b[4];
        ldsm_x4_t(b, tile + tile_off<C>(16 * ks + krow_l, 16 * np + ncol_l));
        mma_bf16(acc[2 * np], af[ks], b[0], b[1]);
        mma_bf16(acc[2 * np + 1], af[ks], b[2], b[3]);
      }
    }
  }
  // Quad transpose so each lane owns 8 consecutive columns of one row, then 16-byte stores.
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int q = 0; q < NTN / 4; ++q) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t v[4], o[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = pack_bf16(acc[4 * q + j][2 * half], acc[4 * q + j][2 * half + 1]);
      // lane t keeps tile t's pair in slot t and fetches, from lane s, that lane's pair of tile t
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        int s = t ^ r;                       // partner lane within the quad
        uint32_t send = v[0];
        send = (s == 1) ? v[1] : send;
        send = (s == 2) ? v[2] : send;
        send = (s == 3) ? v[3] : send;       // my pair of the tile the partner owns
        uint32_t got = __shfl_xor_sync(0xffffffffu, send, r);
        // partner s holds columns 2s, 2s+1 of my tile: slot s of my output
        o[0] = (s == 0) ? got : o[0];
        o[1] = (s == 1) ? got : o[1];
        o[2] = (s == 2) ? got : o[2];
        o[3] = (s == 3) ? got : o[3];
      }
      int row = 16 * warp + g + 8 * half;
      if (row < rows) {
        __nv_bfloat16* dst = out + ((size_t)(tok0 + row) * H + h) * D + 8 * (4 * q + t);
        *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
  }
}

template <int C, int D>
__global__ void __launch_bounds__(Cfg<C, D>::NT, (C == 64 ? 4 : 1)) tc_kernel(const __grid_constant__ CUtensorMap tmK,
                                                         const __grid_constant__ CUtensorMap tmV, KParams p) {
  using cfg = Cfg<C, D>;
  constexpr int LD = cfg::LD;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* sX = reinterpret_cast<float*>(smem + cfg::OFF_X);
  float* sBeta = reinterpret_cast<float*>(smem + cfg::OFF_BETA);
  float* sG = reinterpret_cast<float*>(smem + cfg::OFF_G);
  const uint32_t sK = smem_u32(smem + cfg::OFF_K);
  const uint32_t sV = smem_u32(smem + cfg::OFF_V);
  const uint32_t bar = smem_u32(smem + cfg::OFF_BAR);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const bool do_wy = (p.ops & kDoWY) != 0;
  const bool need_v = do_wy && p.V != nullptr;
  const bool load_a = (p.ops & kLoadA) != 0;
  const long long total = (long long)p.n_chunks * p.H;

  if (tid == 0) {
    prefetch_tmap(&tmK);
    if (need_v) prefetch_tmap(&tmV);
    mbar_init(bar, 1);
    fence_mbar_init();
  }
  __syncthreads();
  uint32_t phase = 0;

  for (long long item = blockIdx.x; item < total; item += gridDim.x) {
    long long tok0;
    int rows, h;
    locate(p, C, item, tok0, rows, h);
    PHASE_BEGIN();

    // ---- 1. stage K, V (TMA) and beta, g
    if (tid == 0) {
      fence_proxy_async();  // earlier generic-proxy accesses to the tiles are ordered before the async writes
      mbar_expect_tx(bar, (uint32_t)(cfg::TILE_BYTES * (need_v ? 2 : 1)));
#pragma unroll
      for (int bx = 0; bx < cfg::NBOX; ++bx) {
        tma_load_2d(sK + bx * cfg::BOX_BYTES, &tmK, bar, h * D + 64 * bx, (int)tok0);
        if (need_v) tma_load_2d(sV + bx * cfg::BOX_BYTES, &tmV, bar, h * D + 64 * bx, (int)tok0);
      }
    }
    for (int i = tid; i < C; i += cfg::NT) {
      size_t bi = (size_t)(tok0 + i) * p.H + h;
      sBeta[i] = (i < rows) ? p.beta[bi] : 0.f;
      sG[i] = (i < rows && p.g) ? p.g[bi] : 0.f;
    }
    if (load_a) {
      for (int e = tid; e < C * C; e += cfg::NT) {
        int i = e / C, j = e - i * C;
        float v = (i == j) ? 1.f : 0.f;
        if (i < rows && j < i) v = p.A_in[((size_t)(tok0 + i) * p.H + h) * C + j];
        sX[i * LD + j] = v;
      }
    }
    bool arrived = mbar_wait_bounded(bar, phase);
    phase ^= 1;
    if (!arrived) {
      // Give the copy one more bounded chance to land before leaving, then report and stop.
      atomicMax(p.status, TRI_INV_ERR_DEVICE_TIMEOUT);
      mbar_wait_bounded(bar, phase ^ 1);
      return;
    }
    if (rows < C) {
      // rows past the sequence end hold a neighbour's tokens (or zero fill): clear them
      for (int e = tid; e < (C - rows) * 8 * cfg::NBOX * 2; e += cfg::NT) {
        int which = e / ((C - rows) * 8 * cfg::NBOX);
        int rem = e - which * (C - rows) * 8 * cfg::NBOX;
        int bx = rem / ((C - rows) * 8);
        int rem2 = rem - bx * (C - rows) * 8;
        int r = rows + rem2 / 8, c = rem2 & 7;
        uint8_t* base = smem + (which ? cfg::OFF_V : cfg::OFF_K) + bx * cfg::BOX_BYTES + r * 128 + c * 16;
        *reinterpret_cast<uint4*>(base) = make_uint4(0, 0, 0, 0);
      }
    }
    __syncthreads();
    PHASE(0);

    if (!load_a) {
      // ---- 2. Gram tiles of this warp's rows, 3. gate + mask, N -> shared memory
      uint32_t af[D / 16][4];
      {
        const int r = 16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1);
        const int fo = 8 * (lane >> 4);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) ldsm_x4(af[ks], sK + tile_off<C>(r, 16 * ks + fo));
      }
      const int ra = 16 * warp + g, rb = ra + 8;
      const float beta_a = sBeta[ra], beta_b = sBeta[rb], g_a = sG[ra], g_b = sG[rb];
#pragma unroll
      for (int jb = 0; jb < cfg::NW; ++jb) {
        if (jb <= warp) {
          float acc[2][4];
#pragma unroll
          for (int i = 0; i < 2; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }
          const int n = 16 * jb + (lane & 7) + 8 * (lane >> 4);
          const int fo = 8 * ((lane >> 3) & 1);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            uint32_t b[4];
            ldsm_x4(b, sK + tile_off<C>(n, 16 * ks + fo));
            mma_bf16(acc[0], af[ks], b[0], b[1]);
            mma_bf16(acc[1], af[ks], b[2], b[3]);
          }
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            const int c = 16 * jb + 8 * nt + 2 * t;
            const float gc0 = sG[c], gc1 = sG[c + 1];
            float2 va, vb;
            va.x = (c < ra) ? beta_a * acc[nt][0] * __expf(g_a - gc0) : 0.f;
            va.y = (c + 1 < ra) ? beta_a * acc[nt][1] * __expf(g_a - gc1) : 0.f;
            vb.x = (c < rb) ? beta_b * acc[nt][2] * __expf(g_b - gc0) : 0.f;
            vb.y = (c + 1 < rb) ? beta_b * acc[nt][3] * __expf(g_b - gc1) : 0.f;
            *reinterpret_cast<float2*>(sX + ra * LD + c) = va;
            *reinterpret_cast<float2*>(sX + rb * LD + c) = vb;
          }
        }
      }
      __syncwarp();
      PHASE(1);

      // ---- 4. leaf: invert this warp's 16x16 diagonal block, lane j owns column j
      {
        const int base = 16 * warp, j = lane & 15;
        const float* nb = sX + base * LD + base;
        float x[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float s = 0.f;
#pragma unroll
          for (int k4 = 0; k4 < (i + 3) / 4; ++k4) {
            float4 nv = *reinterpret_cast<const float4*>(nb + i * LD + 4 * k4);
            if (4 * k4 + 0 < i) s = fmaf(nv.x, x[4 * k4 + 0], s);
            if (4 * k4 + 1 < i) s = fmaf(nv.y, x[4 * k4 + 1], s);
            if (4 * k4 + 2 < i) s = fmaf(nv.z, x[4 * k4 + 2], s);
            if (4 * k4 + 3 < i) s = fmaf(nv.w, x[4 * k4 + 3], s);
          }
          x[i] = (i < j) ? 0.f : (i == j ? 1.f : -s);
        }
        __syncwarp();
        if (lane < 16) {
#pragma unroll
          for (int i = 0; i < 16; ++i) sX[(base + i) * LD + base + j] = x[i];
        }
      }
      __syncthreads();
      PHASE(2);

      // ---- 5. merges
      merge_level<C, 16>(sX, warp, lane);
      PHASE(3);
      merge_level<C, 32>(sX, warp, lane);
      if constexpr (C == 128) merge_level<C, 64>(sX, warp, lane);
      PHASE(4);
    }

    // ---- 6. store A
    if ((p.ops & kStoreA) && p.A) {
      for (int e = tid; e < C * (C / 4); e += cfg::NT) {
        const int i = e / (C / 4), c4 = e - i * (C / 4);
        if (i < rows) {
          float4 v = *reinterpret_cast<const float4*>(sX + i * LD + 4 * c4);
          const int j = 4 * c4;
          v.x = (j + 0 < i) ? v.x : (j + 0 == i ? 1.f : 0.f);
          v.y = (j + 1 < i) ? v.y : (j + 1 == i ? 1.f : 0.f);
          v.z = (j + 2 < i) ? v.z : (j + 2 == i ? 1.f : 0.f);
          v.w = (j + 3 < i) ? v.w : (j + 3 == i ? 1.f : 0.f);
          *reinterpret_cast<float4*>(p.A + ((size_t)(tok0 + i) * p.H + h) * C + j) = v;
        }
      }
    }

    PHASE(5);
    // ---- 7. WY apply
    if (do_wy) {
      uint32_t af[C / 16][4];
      const int ra = 16 * warp + g;
#pragma unroll
      for (int ks = 0; ks < C / 16; ++ks) {
        if (ks <= warp) {
          const int c = 16 * ks + 2 * t;
          const float2 b0 = *reinterpret_cast<const float2*>(sBeta + c);
          const float2 b1 = *reinterpret_cast<const float2*>(sBeta + c + 8);
          const float2 x00 = *reinterpret_cast<const float2*>(sX + ra * LD + c);
          const float2 x10 = *reinterpret_cast<const float2*>(sX + (ra + 8) * LD + c);
          const float2 x01 = *reinterpret_cast<const float2*>(sX + ra * LD + c + 8);
          const float2 x11 = *reinterpret_cast<const float2*>(sX + (ra + 8) * LD + c + 8);
          af[ks][0] = pack_bf16(x00.x * b0.x, x00.y * b0.y);
          af[ks][1] = pack_bf16(x10.x * b0.x, x10.y * b0.y);
          af[ks][2] = pack_bf16(x01.x * b1.x, x01.y * b1.y);
          af[ks][3] = pack_bf16(x11.x * b1.x, x11.y * b1.y);
        } else {
          af[ks][0] = af[ks][1] = af[ks][2] = af[ks][3] = 0u;
        }
      }
      wy_apply<C, D>(af, sK, warp, lane, reinterpret_cast<__nv_bfloat16*>(p.W), tok0, rows, h, p.H);
      if (need_v) wy_apply<C, D>(af, sV, warp, lane, reinterpret_cast<__nv_bfloat16*>(p.U), tok0, rows, h, p.H);
    }
    PHASE(6);
    __syncthreads();  // all warps are done with the tiles and sX before the next item's copies land
    PHASE(7);
  }
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)ptr;
  });
  return fn;
}

// 2-D view of a [tokens, H*d] bf16 tensor; one box = 64 features (128 B, swizzled) x C tokens.
bool make_tmap(CUtensorMap* tm, const void* base, long long tokens, int H, int d, int C) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)H * d, (cuuint64_t)tokens};
  cuuint64_t strides[1] = {(cuuint64_t)H * d * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)C};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int C, int D>
cudaError_t launch_one(const KParams& p, cudaStream_t stream) {
  using cfg = Cfg<C, D>;
  static int ctas_per_sm = 0, n_sm = 0;
  if (!ctas_per_sm) {
    cudaError_t e = cudaFuncSetAttribute(tc_kernel<C, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, cfg::SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(tc_kernel<C, D>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    int dev = 0, occ = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, tc_kernel<C, D>, cfg::NT, cfg::SMEM);
    if (e != cudaSuccess) return e;
    ctas_per_sm = occ > 0 ? occ : 1;
  }
  long long tokens = p.chunk_tab ? (long long)p.T : (long long)p.T * (p.n_chunks / p.chunks_per_seq);
  CUtensorMap tmK, tmV;
  if (!make_tmap(&tmK, p.K, tokens, p.H, D, C)) return cudaErrorUnknown;
  if (p.V) { if (!make_tmap(&tmV, p.V, tokens, p.H, D, C)) return cudaErrorUnknown; }
  else tmV = tmK;
  long long total = (long long)p.n_chunks * p.H;
  long long cap = (long long)n_sm * ctas_per_sm;
  int grid = (int)(total < cap ? total : cap);
  tc_kernel<C, D><<<grid, cfg::NT, cfg::SMEM, stream>>>(tmK, tmV, p);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_tc(const KParams& p, int C, cudaStream_t stream, bool* handled) {
  *handled = false;
  if (p.kv_dtype != TRI_INV_BF16) return cudaSuccess;
  if ((p.method & TRI_INV_METHOD_MASK) != TRI_INV_BLOCK_RECURSIVE || (p.method & TRI_INV_LEAF_SERIES)) return cudaSuccess;
  if (p.d_k != 128 || ((p.ops & kDoWY) && p.V && p.d_v != 128)) return cudaSuccess;
  // the stride of the 2-D view (H * d * 2 bytes) is a multiple of 16 because d is a multiple of 8
  *handled = true;
  if (C == 64) return launch_one<64, 128>(p, stream);
  if (C == 128) return launch_one<128, 128>(p, stream);
  *handled = false;
  return cudaSuccess;
}

}  // namespace tri_inv
