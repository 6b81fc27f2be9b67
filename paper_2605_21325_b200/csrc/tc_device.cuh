// Device-side building blocks shared by the tensor-core kernels: PTX wrappers (mbarrier, TMA, tcgen05,
// tensor-memory loads, warp MMAs), the series leaf, the merge level of the block recursion and the bf16
// epilogue pieces.  Everything here is __device__ __forceinline__ and lives in an unnamed namespace, so each
// translation unit gets its own copy.
#pragma once
#include <cuda.h>

#include <mutex>

#include "common.cuh"

#ifdef TRI_INV_PHASE_CLOCKS
#include "dev_phase_clocks.cuh"
#else
#define CTA_MARK(k) do {} while (0)
#define PHASE_BEGIN() do {} while (0)
#define PHASE(k) do {} while (0)
#define TL(k) do {} while (0)
#endif

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
// Bounded wait: gives up after limit_ns of wall time (the global timer is read every 64 polls, each poll
// itself blocks for a hardware-defined time slice) or after kSpinLimit polls, whichever comes first, so a
// lost copy or product cannot hang the GPU.  The default limit is two seconds.
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, unsigned long long limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  for (uint32_t i = 1; i < kSpinLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63u) == 0 && global_timer_ns() - t0 > limit_ns) return false;
  }
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
// Pulls a tile into L2 only (no shared memory needed): issued an item ahead so that the real
// copy, which has to wait for its buffer, finds the data on chip.
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap* tm, int x, int y) {
  asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(tm), "r"(x), "r"(y) : "memory");
}
// Tile from shared memory to global memory through the copy engine (bulk async-group completion).
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, uint32_t src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tm), "r"(src), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tm, uint32_t src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(tm), "r"(src), "r"(x), "r"(y), "r"(z) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// every bulk store this thread has committed has finished READING its shared-memory source
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// ... all but the KEEP most recent ones have (two staging tiles used in turn: KEEP = 1)
template <int KEEP>
__device__ __forceinline__ void bulk_wait_read_keep() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(KEEP) : "memory"); }
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

__device__ __forceinline__ void mma_tf32(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ float ex2_approx(float x) {  // 2^x, relative error about 2^-22
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {   // round-to-nearest-even, lo in the low half
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int C>
__device__ __forceinline__ uint32_t tile_off(int r, int f) {
  int box = f >> 6, c = (f & 63) >> 3;
  return (uint32_t)(box * (C * 128) + r * 128 + ((c ^ (r & 7)) << 4));
}

// 16x16 leaf by the product series (Alg. 5 on the leaf, the first phase of Alg. 2): X <- I - N, Y <- N,
// three rounds of Y <- Y.Y, X <- X + X.Y as TF32 m16n8k8 MMAs.  X lives in the leaf's place inside the
// fp32 matrix (row length LDX), Y in a per-warp scratch (row length LDY); both are re-read as operands.
template <int LDX, int LDY>
__device__ __forceinline__ void leaf_series(float* xblk, float* ys, int lane) {
  const int g = lane >> 2, t = lane & 3;
  float x[2][4], y[2][4];
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    const int c = 8 * nt + 2 * t;
    const float2 na = *reinterpret_cast<const float2*>(xblk + g * LDX + c);
    const float2 nb = *reinterpret_cast<const float2*>(xblk + (g + 8) * LDX + c);
    y[nt][0] = na.x; y[nt][1] = na.y; y[nt][2] = nb.x; y[nt][3] = nb.y;
    x[nt][0] = (c == g ? 1.f : 0.f) - na.x;
    x[nt][1] = (c + 1 == g ? 1.f : 0.f) - na.y;
    x[nt][2] = (c == g + 8 ? 1.f : 0.f) - nb.x;
    x[nt][3] = (c + 1 == g + 8 ? 1.f : 0.f) - nb.y;
  }
  __syncwarp();
  auto put = [&](float* dst, int ld, const float (&v)[2][4]) {
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int c = 8 * nt + 2 * t;
      *reinterpret_cast<float2*>(dst + g * ld + c) = make_float2(v[nt][0], v[nt][1]);
      *reinterpret_cast<float2*>(dst + (g + 8) * ld + c) = make_float2(v[nt][2], v[nt][3]);
    }
  };
  // acc += P . Q for 16x16 matrices in shared memory
  auto mm = [&](float (&acc)[2][4], const float* pm, int ldp, const float* qm, int ldq) {
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const float* ap = pm + g * ldp + 8 * q + t;
      const uint32_t a0 = to_tf32(ap[0]), a1 = to_tf32(ap[8 * ldp]), a2 = to_tf32(ap[4]), a3 = to_tf32(ap[8 * ldp + 4]);
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const float* bp = qm + (8 * q + t) * ldq + 8 * nt + g;
        mma_tf32(acc[nt], a0, a1, a2, a3, to_tf32(bp[0]), to_tf32(bp[4 * ldq]));
      }
    }
  };
  put(ys, LDY, y);
  put(xblk, LDX, x);
  __syncwarp();
#pragma unroll
  for (int r = 0; r < 3; ++r) {
    float y2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    mm(y2, ys, LDY, ys, LDY);   // Y <- Y.Y
    __syncwarp();               // every lane has read the old Y
    put(ys, LDY, y2);
    __syncwarp();
    mm(x, xblk, LDX, ys, LDY);  // X <- X + X.Y (the accumulator starts as X)
    __syncwarp();               // every lane has read the old X
    put(xblk, LDX, x);
    __syncwarp();
  }
  // exact structure of a unit lower triangular block: constants on and above the diagonal
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    const int c = 8 * nt + 2 * t;
    float2 va = *reinterpret_cast<float2*>(xblk + g * LDX + c), vb = *reinterpret_cast<float2*>(xblk + (g + 8) * LDX + c);
    va.x = (c < g) ? va.x : (c == g ? 1.f : 0.f);
    va.y = (c + 1 < g) ? va.y : (c + 1 == g ? 1.f : 0.f);
    vb.x = (c < g + 8) ? vb.x : (c == g + 8 ? 1.f : 0.f);
    vb.y = (c + 1 < g + 8) ? vb.y : (c + 1 == g + 8 ? 1.f : 0.f);
    *reinterpret_cast<float2*>(xblk + g * LDX + c) = va;
    *reinterpret_cast<float2*>(xblk + (g + 8) * LDX + c) = vb;
  }
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

// One step of iterative refinement (Alg. 6 / Sec. 3.6) for the matrix I + N on the warp-level tensor cores:
//     R = I - X (I + N) = (I - X) - X N,        X <- X + R X.
// sX holds X (fp32, unit lower triangular, complete), sN holds N (fp32, strictly lower triangular, zeros
// elsewhere); both C x C with row length C + 4.  On return sX holds the refined X; sN is overwritten (by R).
// The residual needs more than one TF32 pass (a single pass has the very error the step is to remove), so
// X N is formed from the TF32 splits X = Xh + Xl, N = Nh + Nl as Xh Nh + Xl Nh + Xh Nl with fp32 accumulation
// (the dropped Xl Nl is 2^-22 relative); R is then about as small as the inverse's error, and R X needs one
// pass only.  8-column tiles of the lower triangle are dealt out to the C / 16 warps by column (warp w takes
// columns w and C/8 - 1 - w), so the triangular work is shared about evenly; only the k-steps where both operands can be non-zero
// are issued (X and R lower triangular: k <= i; N strictly lower, X lower: k >= j).
template <int C>
__device__ __forceinline__ void refine_step(float* sX, float* sN, int warp, int lane) {
  constexpr int LD = C + 4, NT8 = C / 8;
  constexpr int CPW = 2;                   // tile columns per warp: column w and column NT8 - 1 - w (long and short k ranges paired)
  constexpr int MAXT = (C / 16) * CPW;     // tiles a warp can own: row blocks x its columns
  const int g = lane >> 2, t = lane & 3;
  float acc[MAXT][4];
  auto split = [](float x, uint32_t& hi, uint32_t& lo) {
    hi = to_tf32(x);
    lo = to_tf32(x - __uint_as_float(hi));
  };
  // ---- R tiles of this warp
#pragma unroll
  for (int rb = 0; rb < C / 16; ++rb) {
#pragma unroll
    for (int c = 0; c < CPW; ++c) {
      const int slot = rb * (CPW) + c;
      acc[slot][0] = acc[slot][1] = acc[slot][2] = acc[slot][3] = 0.f;
    }
#pragma unroll 1                               // (a run-time loop: unrolled, the step's code would not fit the instruction cache)
    for (int q = 0; q < 2 * rb + 2; ++q) {     // k-step of eight: columns 8q .. 8q+7 of X, rows of N
      bool any = false;
#pragma unroll
      for (int c = 0; c < CPW; ++c) any = any || ((c == 0 ? warp : NT8 - 1 - warp) <= q);
      if (!any) continue;                      // warp-uniform: none of this warp's columns reaches this k-step
      const float* ap = sX + (16 * rb + g) * LD + 8 * q + t;
      uint32_t ah[4], al[4];
      split(ap[0], ah[0], al[0]);
      split(ap[8 * LD], ah[1], al[1]);
      split(ap[4], ah[2], al[2]);
      split(ap[8 * LD + 4], ah[3], al[3]);
#pragma unroll
      for (int c = 0; c < CPW; ++c) {
        const int nt = (c == 0 ? warp : NT8 - 1 - warp);
        if (nt <= q && nt < 2 * rb + 2) {
          const float* bp = sN + (8 * q + t) * LD + 8 * nt + g;
          uint32_t bh0, bl0, bh1, bl1;
          split(bp[0], bh0, bl0);
          split(bp[4 * LD], bh1, bl1);
          float (&d)[4] = acc[rb * (CPW) + c];
          mma_tf32(d, ah[0], ah[1], ah[2], ah[3], bh0, bh1);
          mma_tf32(d, al[0], al[1], al[2], al[3], bh0, bh1);
          mma_tf32(d, ah[0], ah[1], ah[2], ah[3], bl0, bl1);
        }
      }
    }
  }
  __syncthreads();   // every warp has read all it needs of N: its space takes R
#pragma unroll
  for (int rb = 0; rb < C / 16; ++rb) {
#pragma unroll
    for (int c = 0; c < CPW; ++c) {
      const int nt = (c == 0 ? warp : NT8 - 1 - warp);
      if (nt < 2 * rb + 2) {
        const float (&d)[4] = acc[rb * (CPW) + c];
        const int ra = 16 * rb + g, col = 8 * nt + 2 * t;
        const float2 xa = *reinterpret_cast<const float2*>(sX + ra * LD + col);
        const float2 xb = *reinterpret_cast<const float2*>(sX + (ra + 8) * LD + col);
        // R = I - X - X N, rounded to TF32 once (it is only ever an MMA operand)
        float2 r0, r1;
        r0.x = __uint_as_float(to_tf32((col == ra ? 1.f : 0.f) - xa.x - d[0]));
        r0.y = __uint_as_float(to_tf32((col + 1 == ra ? 1.f : 0.f) - xa.y - d[1]));
        r1.x = __uint_as_float(to_tf32((col == ra + 8 ? 1.f : 0.f) - xb.x - d[2]));
        r1.y = __uint_as_float(to_tf32((col + 1 == ra + 8 ? 1.f : 0.f) - xb.y - d[3]));
        *reinterpret_cast<float2*>(sN + ra * LD + col) = r0;
        *reinterpret_cast<float2*>(sN + (ra + 8) * LD + col) = r1;
      }
    }
  }
  __syncthreads();
  // ---- X + R X on the same tiles (R from shared memory, already TF32; X rounded on the fly)
#pragma unroll
  for (int rb = 0; rb < C / 16; ++rb) {
#pragma unroll
    for (int c = 0; c < CPW; ++c) {
      const int nt = (c == 0 ? warp : NT8 - 1 - warp);
      const int ra = 16 * rb + g, col = 8 * nt + 2 * t;
      float (&d)[4] = acc[rb * (CPW) + c];
      if (nt < 2 * rb + 2) {
        const float2 xa = *reinterpret_cast<const float2*>(sX + ra * LD + col);
        const float2 xb = *reinterpret_cast<const float2*>(sX + (ra + 8) * LD + col);
        d[0] = xa.x; d[1] = xa.y; d[2] = xb.x; d[3] = xb.y;
      }
    }
#pragma unroll 1
    for (int q = 0; q < 2 * rb + 2; ++q) {
      bool any = false;
#pragma unroll
      for (int c = 0; c < CPW; ++c) any = any || ((c == 0 ? warp : NT8 - 1 - warp) <= q);
      if (!any) continue;
      const float* ap = sN + (16 * rb + g) * LD + 8 * q + t;
      const uint32_t a0 = __float_as_uint(ap[0]), a1 = __float_as_uint(ap[8 * LD]), a2 = __float_as_uint(ap[4]),
                     a3 = __float_as_uint(ap[8 * LD + 4]);
#pragma unroll
      for (int c = 0; c < CPW; ++c) {
        const int nt = (c == 0 ? warp : NT8 - 1 - warp);
        if (nt <= q && nt < 2 * rb + 2) {
          const float* bp = sX + (8 * q + t) * LD + 8 * nt + g;
          mma_tf32(acc[rb * (CPW) + c], a0, a1, a2, a3, to_tf32(bp[0]), to_tf32(bp[4 * LD]));
        }
      }
    }
  }
  __syncthreads();   // every warp has read the old X
#pragma unroll
  for (int rb = 0; rb < C / 16; ++rb) {
#pragma unroll
    for (int c = 0; c < CPW; ++c) {
      const int nt = (c == 0 ? warp : NT8 - 1 - warp);
      if (nt < 2 * rb + 2) {
        const float (&d)[4] = acc[rb * (CPW) + c];
        const int ra = 16 * rb + g, col = 8 * nt + 2 * t;
        float2 va, vb;   // the structure of a unit lower triangular matrix is written as constants
        va.x = (col < ra) ? d[0] : (col == ra ? 1.f : 0.f);
        va.y = (col + 1 < ra) ? d[1] : (col + 1 == ra ? 1.f : 0.f);
        vb.x = (col < ra + 8) ? d[2] : (col == ra + 8 ? 1.f : 0.f);
        vb.y = (col + 1 < ra + 8) ? d[3] : (col + 1 == ra + 8 ? 1.f : 0.f);
        *reinterpret_cast<float2*>(sX + ra * LD + col) = va;
        *reinterpret_cast<float2*>(sX + (ra + 8) * LD + col) = vb;
      }
    }
  }
  __syncthreads();
}

// 16x16 leaf by forward substitution (Sec. 3.1): lane j owns column j of the inverse; rows of N are read as
// broadcast float4; the block is overwritten by its inverse (zeros above the diagonal, ones on it).
template <int LD>
__device__ __forceinline__ void leaf_substitution(float* blk, int lane) {
  const int j = lane & 15;
  float x[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    float s = 0.f;
#pragma unroll
    for (int k4 = 0; k4 < (i + 3) / 4; ++k4) {
      float4 nv = *reinterpret_cast<const float4*>(blk + i * LD + 4 * k4);
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
    for (int i = 0; i < 16; ++i) blk[i * LD + j] = x[i];
  }
}

// ------------------------------------------------------------------------------------------ tcgen05 helpers
// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte offsets
// (all >> 4), descriptor version 1 at bit 46, 128-byte swizzle (code 2) at bits 61..63.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3fffu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor for kind::f16: fp32 accumulate, bf16 x bf16, A K-major,
// B K-major (b_mn = 0) or MN-major (b_mn = 1), shape M x N.
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same with fp16 x fp16 operands (format code 0 for both): only the instruction descriptor differs.
__host__ __device__ constexpr uint32_t umma_idesc_f16(int M, int N, int b_mn) {
  return (1u << 4) | ((uint32_t)b_mn << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// kind::tf32: fp32 data in shared memory read as TF32, fp32 accumulate, K = 8 per instruction.
__host__ __device__ constexpr uint32_t umma_idesc_tf32(int M, int N, int b_mn) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 16 lanes x 64 columns -> 8 n-tiles of accumulator fragments.
__device__ __forceinline__ void tmem_ld_16x64(float (&r)[8][4], uint32_t taddr) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=f"(r[0][0]), "=f"(r[0][1]), "=f"(r[0][2]), "=f"(r[0][3]), "=f"(r[1][0]), "=f"(r[1][1]), "=f"(r[1][2]), "=f"(r[1][3]),
        "=f"(r[2][0]), "=f"(r[2][1]), "=f"(r[2][2]), "=f"(r[2][3]), "=f"(r[3][0]), "=f"(r[3][1]), "=f"(r[3][2]), "=f"(r[3][3]),
        "=f"(r[4][0]), "=f"(r[4][1]), "=f"(r[4][2]), "=f"(r[4][3]), "=f"(r[5][0]), "=f"(r[5][1]), "=f"(r[5][2]), "=f"(r[5][3]),
        "=f"(r[6][0]), "=f"(r[6][1]), "=f"(r[6][2]), "=f"(r[6][3]), "=f"(r[7][0]), "=f"(r[7][1]), "=f"(r[7][2]), "=f"(r[7][3])
      : "r"(taddr));
}
// 16 lanes x 32 columns -> 4 n-tiles of accumulator fragments.
__device__ __forceinline__ void tmem_ld_16x32(float (&r)[4][4], uint32_t taddr) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=f"(r[0][0]), "=f"(r[0][1]), "=f"(r[0][2]), "=f"(r[0][3]), "=f"(r[1][0]), "=f"(r[1][1]), "=f"(r[1][2]), "=f"(r[1][3]),
        "=f"(r[2][0]), "=f"(r[2][1]), "=f"(r[2][2]), "=f"(r[2][3]), "=f"(r[3][0]), "=f"(r[3][1]), "=f"(r[3][2]), "=f"(r[3][3])
      : "r"(taddr));
}
// 16 lanes x 16 columns -> 2 n-tiles of accumulator fragments.
__device__ __forceinline__ void tmem_ld_16x16(float (&r)[2][4], uint32_t taddr) {
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(r[0][0]), "=f"(r[0][1]), "=f"(r[0][2]), "=f"(r[0][3]), "=f"(r[1][0]), "=f"(r[1][1]), "=f"(r[1][2]), "=f"(r[1][3])
               : "r"(taddr));
}
// 16 lanes x 128 columns -> 16 n-tiles of accumulator fragments.
__device__ __forceinline__ void tmem_ld_16x128(float (&r)[16][4], uint32_t taddr) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x16.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,"
      "%32,%33,%34,%35,%36,%37,%38,%39,%40,%41,%42,%43,%44,%45,%46,%47,%48,%49,%50,%51,%52,%53,%54,%55,%56,%57,%58,%59,%60,%61,%62,%63}, [%64];"
      : "=f"(r[0][0]), "=f"(r[0][1]), "=f"(r[0][2]), "=f"(r[0][3]), "=f"(r[1][0]), "=f"(r[1][1]), "=f"(r[1][2]), "=f"(r[1][3]),
        "=f"(r[2][0]), "=f"(r[2][1]), "=f"(r[2][2]), "=f"(r[2][3]), "=f"(r[3][0]), "=f"(r[3][1]), "=f"(r[3][2]), "=f"(r[3][3]),
        "=f"(r[4][0]), "=f"(r[4][1]), "=f"(r[4][2]), "=f"(r[4][3]), "=f"(r[5][0]), "=f"(r[5][1]), "=f"(r[5][2]), "=f"(r[5][3]),
        "=f"(r[6][0]), "=f"(r[6][1]), "=f"(r[6][2]), "=f"(r[6][3]), "=f"(r[7][0]), "=f"(r[7][1]), "=f"(r[7][2]), "=f"(r[7][3]),
        "=f"(r[8][0]), "=f"(r[8][1]), "=f"(r[8][2]), "=f"(r[8][3]), "=f"(r[9][0]), "=f"(r[9][1]), "=f"(r[9][2]), "=f"(r[9][3]),
        "=f"(r[10][0]), "=f"(r[10][1]), "=f"(r[10][2]), "=f"(r[10][3]), "=f"(r[11][0]), "=f"(r[11][1]), "=f"(r[11][2]), "=f"(r[11][3]),
        "=f"(r[12][0]), "=f"(r[12][1]), "=f"(r[12][2]), "=f"(r[12][3]), "=f"(r[13][0]), "=f"(r[13][1]), "=f"(r[13][2]), "=f"(r[13][3]),
        "=f"(r[14][0]), "=f"(r[14][1]), "=f"(r[14][2]), "=f"(r[14][3]), "=f"(r[15][0]), "=f"(r[15][1]), "=f"(r[15][2]), "=f"(r[15][3])
      : "r"(taddr));
}

// Accumulator fragments back into tensor memory (16 lanes x 32 columns), and the wait that makes them visible.
__device__ __forceinline__ void tmem_st_16x32(const float (&r)[4][4], uint32_t taddr) {
  asm volatile(
      "tcgen05.st.sync.aligned.16x256b.x4.b32 [%16], {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"
      ::"f"(r[0][0]), "f"(r[0][1]), "f"(r[0][2]), "f"(r[0][3]), "f"(r[1][0]), "f"(r[1][1]), "f"(r[1][2]), "f"(r[1][3]),
        "f"(r[2][0]), "f"(r[2][1]), "f"(r[2][2]), "f"(r[2][3]), "f"(r[3][0]), "f"(r[3][1]), "f"(r[3][2]), "f"(r[3][3]),
        "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_16x16(const float (&r)[2][4], uint32_t taddr) {
  asm volatile("tcgen05.st.sync.aligned.16x256b.x2.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
               ::"f"(r[0][0]), "f"(r[0][1]), "f"(r[0][2]), "f"(r[0][3]), "f"(r[1][0]), "f"(r[1][1]), "f"(r[1][2]), "f"(r[1][3]), "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void stmatrix_x4(uint32_t addr, uint32_t m0, uint32_t m1, uint32_t m2, uint32_t m3) {
  asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(m0), "r"(m1), "r"(m2), "r"(m3) : "memory");
}

// Epilogue of one 16-row x 64-column piece of W or U: accumulator fragments from tensor memory ->
// bf16 -> stmatrix into a per-warp, swizzled 2 KiB staging tile.  A piece with all 16 rows inside its sequence
// then leaves through the copy engine (one tiled bulk store: tm is a 2-D map of the output with boxes of 64
// columns x 16 rows in the same 128-byte swizzle, x / y the piece's first column and token), which costs
// the warp no load/store instructions; lane 0 owns the stores, and waits for the previous one to have read the
// staging tile before it is rewritten (with two tiles used in turn, KEEP = 1 lets the latest store go on).  The caller waits again (bulk_wait_read, lane 0) before the staging
// space is used for anything else.  A piece cut short by its sequence's end takes 16-byte loads and
// coalesced 16-byte global stores of its real rows only (8 lanes cover one 128-byte row segment).
template <int KEEP = 0>
__device__ __forceinline__ void store_frag_piece_bf16(const float (&f)[8][4], uint32_t stage, int lane, __nv_bfloat16* out_row0,
                                                      size_t row_stride, int rows_left, const CUtensorMap* tm, int x, int y) {
  const int mi = lane >> 3, r = (lane & 7) + 8 * (mi & 1);
  if (lane == 0) bulk_wait_read_keep<KEEP>();   // KEEP = 1: the store issued just before this one used the other staging tile
  __syncwarp();
#pragma unroll
  for (int nt = 0; nt < 8; nt += 2) {
    const uint32_t m0 = pack_bf16(f[nt][0], f[nt][1]), m1 = pack_bf16(f[nt][2], f[nt][3]);
    const uint32_t m2 = pack_bf16(f[nt + 1][0], f[nt + 1][1]), m3 = pack_bf16(f[nt + 1][2], f[nt + 1][3]);
    const int chunk = nt + (mi >> 1);
    const uint32_t addr = stage + r * 128 + ((chunk ^ (r & 7)) << 4);
    asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(m0), "r"(m1), "r"(m2), "r"(m3) : "memory");
  }
  if (rows_left >= 16) {
#ifdef TRI_INV_DEBUG
    if (x < 0 || y < 0 || (x & 7)) return;   // a tiled store must start on a 16-byte boundary and inside the tensor (the caller's item check covers y + 16)
#endif
    fence_proxy_async();   // this lane's staging writes become visible to the copy engine
    __syncwarp();
    if (lane == 0) {
      tma_store_2d(tm, stage, x, y);
      bulk_commit();
    }
    return;
  }
  __syncwarp();
#pragma unroll
  for (int m = 0; m < 4; ++m) {
    const int rr = 4 * m + (lane >> 3), c = lane & 7;
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(stage + rr * 128 + ((c ^ (rr & 7)) << 4)));
    if (rr < rows_left) *reinterpret_cast<uint4*>(out_row0 + rr * row_stride + 8 * c) = v;
  }
  __syncwarp();
}
template <int KEEP = 0>
__device__ __forceinline__ void store_piece_bf16(uint32_t taddr, uint32_t stage, int lane, __nv_bfloat16* out_row0,
                                                 size_t row_stride, int rows_left, const CUtensorMap* tm, int x, int y) {
  float f[8][4];
  tmem_ld_16x64(f, taddr);
  tmem_wait_ld();
  store_frag_piece_bf16<KEEP>(f, stage, lane, out_row0, row_stride, rows_left, tm, x, y);
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
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

// 2-D view of a [tokens, H*d] tensor of bf16 (elt = 2) or fp32 (elt = 4); one box = 128 bytes of features
// (64 bf16 or 32 fp32, swizzled) x C tokens.
// 3-D view of A [tokens, H, C] fp32 for the store of one whole chunk matrix straight from its padded rows in shared memory:
// one box = C tokens x one head x LD floats (LD >= C, the row length in shared memory, a multiple of 4), no swizzle.  The
// box is wider than the tensor's innermost extent; the columns past C fall outside the tensor and are not written.
inline bool make_tmap_a(CUtensorMap* tm, const float* base, long long tokens, int H, int C, int LD) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)C, (cuuint64_t)H, (cuuint64_t)tokens};
  cuuint64_t strides[2] = {(cuuint64_t)C * 4, (cuuint64_t)H * C * 4};
  cuuint32_t box[3] = {(cuuint32_t)LD, 1, (cuuint32_t)C};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

inline bool make_tmap(CUtensorMap* tm, const void* base, long long tokens, int H, int d, int C, int elt = 2) {   // C = tokens per box
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)H * d, (cuuint64_t)tokens};
  cuuint64_t strides[1] = {(cuuint64_t)H * d * elt};
  cuuint32_t box[2] = {(cuuint32_t)(128 / elt), (cuuint32_t)C};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, elt == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}


}  // namespace
}  // namespace tri_inv
