/*
 * fp64 CPU oracle for the chunkwise delta-rule triangular inversion.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * tests, the smoke check and the bench's cpu_baseline leg compare the CUDA
 * library against.  It shares no code with the CUDA path and the product
 * never calls it.
 *
 * What it computes, per (sequence, head, chunk) with r <= C real rows:
 *
 *   S_ij = k_i . k_j                                   (Gram entries, j < i)
 *   N_ij = beta_i * S_ij * exp(g_i - g_j)   for j < i  (Eq. 3 with the GDN row
 *          0 otherwise                                   of Table 1; the decay
 *                                                        matrix is exp(g_i-g_j))
 *   A    = (I + N)^{-1}   by forward substitution      (Sec. 3.1, column sweep
 *                                                        in its scalar form)
 *   W    = A diag(beta) K,   U = A diag(beta) V        (WY factors)
 *
 * Inputs arrive in their storage type (fp32, bf16 bit patterns, or double for
 * keys prepared in double by the raw front end) and are widened exactly to
 * double; every sum runs in double in index order.  There is no blocking,
 * tiling or reordering: each loop is the formula.
 *
 * Layouts (all contiguous, row-major):
 *   K [B,T,H,d_k], V [B,T,H,d_v], beta and g [B,T,H] (g is the within-chunk
 *   cumulative log-decay), A and N [B,T,H,C] (row = token, C columns of its
 *   chunk), W [B,T,H,d_k], U [B,T,H,d_v].
 * Dense mode: cu_seqlens == NULL, B sequences of T tokens.  Ragged mode:
 * B == 1, T == total tokens, sequence s covers [cu_seqlens[s], cu_seqlens[s+1]).
 * Chunks restart at every sequence start; a short last chunk is the leading
 * r x r block of an identity-padded C x C problem, and only its r rows are
 * written (columns >= r of those rows are 0).
 *
 * OpenMP runs independent chunks on separate threads; that is the only
 * parallelism.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1, ORACLE_F64 = 2 };

static double widen(const void* base, int dtype, size_t idx) {
  if (dtype == ORACLE_F32) return (double)((const float*)base)[idx];
  if (dtype == ORACLE_F64) return ((const double*)base)[idx];
  uint32_t bits = ((uint32_t)((const uint16_t*)base)[idx]) << 16; /* bf16 = top half of fp32 */
  float f;
  memcpy(&f, &bits, sizeof f);
  return (double)f;
}

typedef struct { int64_t tok0; int rows; } chunk_t;

/* List every chunk as (first token, real rows).  Returns count, or -1 on a bad cu_seqlens. */
static int64_t list_chunks(int B, int T, int C, const int32_t* cu, int n_seqs, chunk_t** out) {
  int64_t n = 0, cap = 0;
  int nseq = cu ? n_seqs : B;
  for (int pass = 0; pass < 2; ++pass) {
    n = 0;
    for (int s = 0; s < nseq; ++s) {
      int64_t beg = cu ? cu[s] : (int64_t)s * T;
      int64_t end = cu ? cu[s + 1] : (int64_t)(s + 1) * T;
      if (end < beg) return -1;
      for (int64_t t = beg; t < end; t += C) {
        if (pass) { (*out)[n].tok0 = t; (*out)[n].rows = (int)((end - t) < C ? (end - t) : C); }
        ++n;
      }
    }
    if (!pass) { cap = n; *out = (chunk_t*)malloc(sizeof(chunk_t) * (size_t)(cap ? cap : 1)); if (!*out) return -1; }
  }
  return n;
}

/*
 * A = (I+N)^{-1} for every chunk; N_out (nullable) receives N itself.
 * All pointers are HOST pointers.  Returns 0, or 1 on invalid arguments.
 */
int tri_inv_oracle_build_ex(const void* K, int kv_dtype, const float* beta, const float* g, const float* G, int gate_shift,
                            double* A, double* N_out,
                            int B, int T, int H, int d_k, int C,
                            const int32_t* cu_seqlens, int n_seqs, int n_threads);

int tri_inv_oracle_build(const void* K, int kv_dtype, const float* beta, const float* g,
                         double* A, double* N_out,
                         int B, int T, int H, int d_k, int C,
                         const int32_t* cu_seqlens, int n_seqs, int n_threads) {
  return tri_inv_oracle_build_ex(K, kv_dtype, beta, g, NULL, 0, A, N_out, B, T, H, d_k, C, cu_seqlens, n_seqs, n_threads);
}

/*
 * The same with the other decay matrices of Table 1:
 *   G != NULL (g ignored):  per-channel decay, the KDA row,   N_ij = beta_i sum_c K_ic K_jc exp(G_ic - G_jc);
 *                           G [B,T,H,d_k] fp32 is the cumulative per-channel log-decay inside each chunk;
 *   gate_shift != 0:        the Comba row's decay A^{i-1/j},  N_ij = beta_i (k_i . k_j) exp(g_{i-1} - g_j)
 *                           (row i takes the cumulative log-decay of the token before it; the first row of a chunk
 *                           has no entry below the diagonal, so no g_{-1} is ever needed).
 * The exponent is always taken of the difference.
 */
int tri_inv_oracle_build_ex(const void* K, int kv_dtype, const float* beta, const float* g, const float* G, int gate_shift,
                            double* A, double* N_out,
                            int B, int T, int H, int d_k, int C,
                            const int32_t* cu_seqlens, int n_seqs, int n_threads) {
  if (!K || !beta || (!g && !G) || !A || B < 1 || T < 0 || H < 1 || d_k < 1 || C < 1) return 1;
  if (G && gate_shift) return 1;
  if (cu_seqlens && (B != 1 || n_seqs < 0 || cu_seqlens[0] != 0 || cu_seqlens[n_seqs] != T)) return 1;
  chunk_t* ch = NULL;
  int64_t n_chunks = list_chunks(B, T, C, cu_seqlens, n_seqs, &ch);
  if (n_chunks < 0) { free(ch); return 1; }
#ifdef _OPENMP
  if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
  int64_t total = n_chunks * H;
#pragma omp parallel
  {
    double* N = (double*)malloc(sizeof(double) * (size_t)C * C);
    double* X = (double*)malloc(sizeof(double) * (size_t)C * C);
#pragma omp for schedule(static)
    for (int64_t w = 0; w < total; ++w) {
      int64_t c = w / H;
      int h = (int)(w % H);
      int64_t t0 = ch[c].tok0;
      int r = ch[c].rows;
      /* N: strictly lower, row-scaled by beta, decayed by exp(g_i - g_j) */
      for (int i = 0; i < C; ++i)
        for (int j = 0; j < C; ++j) N[i * C + j] = 0.0;
      for (int i = 0; i < r; ++i) {
        size_t bi = (size_t)(t0 + i) * H + h;
        for (int j = 0; j < i; ++j) {
          size_t bj = (size_t)(t0 + j) * H + h;
          double s = 0.0;
          if (G) {
            for (int k = 0; k < d_k; ++k)
              s += widen(K, kv_dtype, bi * d_k + k) * widen(K, kv_dtype, bj * d_k + k) *
                   exp((double)G[bi * d_k + k] - (double)G[bj * d_k + k]);
            N[i * C + j] = (double)beta[bi] * s;
          } else {
            for (int k = 0; k < d_k; ++k)
              s += widen(K, kv_dtype, bi * d_k + k) * widen(K, kv_dtype, bj * d_k + k);
            double g_row = gate_shift ? (double)g[bi - (size_t)H] : (double)g[bi];   /* i >= 1 here: the token before is in the chunk */
            N[i * C + j] = (double)beta[bi] * s * exp(g_row - (double)g[bj]);
          }
        }
      }
      /* forward substitution on (I+N) X = I, one column at a time */
      for (int i = 0; i < C; ++i)
        for (int j = 0; j < C; ++j) X[i * C + j] = 0.0;
      for (int j = 0; j < r; ++j) {
        X[j * C + j] = 1.0;
        for (int i = j + 1; i < r; ++i) {
          double s = 0.0;
          for (int k = j; k < i; ++k) s += N[i * C + k] * X[k * C + j];
          X[i * C + j] = -s;
        }
      }
      for (int i = 0; i < r; ++i) {
        size_t row = ((size_t)(t0 + i) * H + h) * C;
        for (int j = 0; j < C; ++j) {
          A[row + j] = X[i * C + j];
          if (N_out) N_out[row + j] = N[i * C + j];
        }
      }
    }
    free(N);
    free(X);
  }
  free(ch);
  return 0;
}

/*
 * W = A diag(beta) K and U = A diag(beta) V from a given A (double, layout
 * [B,T,H,C]).  V, U may both be NULL to skip U.  HOST pointers.
 */
int tri_inv_oracle_wy(const double* A, const void* K, const void* V, int kv_dtype, const float* beta,
                      double* W, double* U,
                      int B, int T, int H, int d_k, int d_v, int C,
                      const int32_t* cu_seqlens, int n_seqs, int n_threads) {
  if (!A || !K || !beta || !W || B < 1 || T < 0 || H < 1 || d_k < 1 || C < 1) return 1;
  if ((V == NULL) != (U == NULL)) return 1;
  if (V && d_v < 1) return 1;
  if (cu_seqlens && (B != 1 || n_seqs < 0 || cu_seqlens[0] != 0 || cu_seqlens[n_seqs] != T)) return 1;
  chunk_t* ch = NULL;
  int64_t n_chunks = list_chunks(B, T, C, cu_seqlens, n_seqs, &ch);
  if (n_chunks < 0) { free(ch); return 1; }
#ifdef _OPENMP
  if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
  int64_t total = n_chunks * H;
#pragma omp parallel for schedule(static)
  for (int64_t w = 0; w < total; ++w) {
    int64_t c = w / H;
    int h = (int)(w % H);
    int64_t t0 = ch[c].tok0;
    int r = ch[c].rows;
    for (int i = 0; i < r; ++i) {
      size_t ri = (size_t)(t0 + i) * H + h;
      for (int k = 0; k < d_k; ++k) {
        double s = 0.0;
        for (int j = 0; j <= i; ++j) {
          size_t rj = (size_t)(t0 + j) * H + h;
          s += A[ri * C + j] * (double)beta[rj] * widen(K, kv_dtype, rj * d_k + k);
        }
        W[ri * d_k + k] = s;
      }
      if (V) {
        for (int k = 0; k < d_v; ++k) {
          double s = 0.0;
          for (int j = 0; j <= i; ++j) {
            size_t rj = (size_t)(t0 + j) * H + h;
            s += A[ri * C + j] * (double)beta[rj] * widen(V, kv_dtype, rj * d_v + k);
          }
          U[ri * d_v + k] = s;
        }
      }
    }
  }
  free(ch);
  return 0;
}

/* Threads an OpenMP region would use for a given request (0 = runtime default). */
int tri_inv_oracle_threads(int n_threads) {
#ifdef _OPENMP
  if (n_threads > 0) return n_threads;
  return omp_get_max_threads();
#else
  (void)n_threads;
  return 1;
#endif
}

/*
 * The gated delta-rule layer as its token-by-token linear recurrence (Sec. 1's recurrent form with the
 * delta-rule update and the decay gate of the GDN row of Table 1; the chunkwise path with (I+N)^{-1},
 * W and U is a re-formulation of exactly this).  Per sequence and head, with the state S [d_k][d_v]
 * starting at S0 (zero when NULL), for every token t in order:
 *
 *     a_t   = g_t - g_{t-1}  (g_{t-1} = 0 at the first row of a chunk: g is the within-chunk cumulative sum)
 *     S    <- exp(a_t) * S                                   decay
 *     S    <- S + beta_t * k_t (v_t - S^T k_t)^T             delta-rule write
 *     o_t   = scale * S^T q_t                                read
 *
 * Q, K [B,T,H,d_k], V [B,T,H,d_v] in one storage type; beta, g [B,T,H] fp32; S0, S_out
 * [n_sequences,H,d_k,d_v] double (both nullable); O [B,T,H,d_v] double.  HOST pointers.
 * OpenMP over (sequence, head); every sum in double in index order.
 */
int tri_inv_oracle_recurrence_ex(const void* Q, const void* K, const void* V, int kv_dtype,
                                 const float* beta, const float* g, const float* G, int read_before_decay, const double* S0,
                                 double* O, double* S_out, double scale,
                                 int B, int T, int H, int d_k, int d_v, int C,
                                 const int32_t* cu_seqlens, int n_seqs, int n_threads);

int tri_inv_oracle_gdn_recurrence(const void* Q, const void* K, const void* V, int kv_dtype,
                                  const float* beta, const float* g, const double* S0,
                                  double* O, double* S_out, double scale,
                                  int B, int T, int H, int d_k, int d_v, int C,
                                  const int32_t* cu_seqlens, int n_seqs, int n_threads) {
  return tri_inv_oracle_recurrence_ex(Q, K, V, kv_dtype, beta, g, NULL, 0, S0, O, S_out, scale, B, T, H, d_k, d_v, C,
                                      cu_seqlens, n_seqs, n_threads);
}

/*
 * The same recurrence for the other two decay forms of Table 1.
 *   G != NULL (g ignored): one decay per key feature (KDA row): a_{t,c} = G_{t,c} - G_{t-1,c}, row c of S is
 *                          multiplied by exp(a_{t,c}); everything else as above.
 *   read_before_decay:     the write's correction reads the state BEFORE this token's decay (Comba row, whose decay
 *                          matrix therefore runs from j to i-1):
 *                              r = v_t - S^T k_t;   S <- exp(a_t) S;   S <- S + beta_t k_t r^T;   o_t = scale S^T q_t.
 */
int tri_inv_oracle_recurrence_ex(const void* Q, const void* K, const void* V, int kv_dtype,
                                 const float* beta, const float* g, const float* G, int read_before_decay, const double* S0,
                                 double* O, double* S_out, double scale,
                                 int B, int T, int H, int d_k, int d_v, int C,
                                 const int32_t* cu_seqlens, int n_seqs, int n_threads) {
  if (!Q || !K || !V || !beta || (!g && !G) || !O || B < 1 || T < 0 || H < 1 || d_k < 1 || d_v < 1 || C < 1) return 1;
  if (G && read_before_decay) return 1;
  if (cu_seqlens && (B != 1 || n_seqs < 0 || cu_seqlens[0] != 0 || cu_seqlens[n_seqs] != T)) return 1;
  int nseq = cu_seqlens ? n_seqs : B;
#ifdef _OPENMP
  if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
  int64_t total = (int64_t)nseq * H;
#pragma omp parallel
  {
    double* S = (double*)malloc(sizeof(double) * (size_t)d_k * d_v);
    double* r = (double*)malloc(sizeof(double) * (size_t)d_v);
#pragma omp for schedule(dynamic, 1)
    for (int64_t w = 0; w < total; ++w) {
      int s = (int)(w / H), h = (int)(w % H);
      int64_t beg = cu_seqlens ? cu_seqlens[s] : (int64_t)s * T;
      int64_t end = cu_seqlens ? cu_seqlens[s + 1] : (int64_t)(s + 1) * T;
      for (int i = 0; i < d_k * d_v; ++i) S[i] = S0 ? S0[((size_t)s * H + h) * d_k * d_v + i] : 0.0;
      for (int64_t t = beg; t < end; ++t) {
        size_t th = (size_t)t * H + h;
        int first_of_chunk = ((t - beg) % C) == 0;
        double b = (double)beta[th];
        if (read_before_decay) {   /* the correction term sees the state as the previous token left it */
          for (int j = 0; j < d_v; ++j) {
            double acc = 0.0;
            for (int i = 0; i < d_k; ++i) acc += widen(K, kv_dtype, th * d_k + i) * S[i * d_v + j];
            r[j] = widen(V, kv_dtype, th * d_v + j) - acc;
          }
        }
        if (G) {
          for (int i = 0; i < d_k; ++i) {
            double a = (double)G[th * d_k + i] - (first_of_chunk ? 0.0 : (double)G[(th - H) * d_k + i]);
            double alpha = exp(a);
            for (int j = 0; j < d_v; ++j) S[i * d_v + j] *= alpha;
          }
        } else {
          double a = (double)g[th] - (first_of_chunk ? 0.0 : (double)g[th - H]);
          double alpha = exp(a);
          for (int i = 0; i < d_k * d_v; ++i) S[i] *= alpha;
        }
        if (!read_before_decay) {
          for (int j = 0; j < d_v; ++j) {
            double acc = 0.0;
            for (int i = 0; i < d_k; ++i) acc += widen(K, kv_dtype, th * d_k + i) * S[i * d_v + j];
            r[j] = widen(V, kv_dtype, th * d_v + j) - acc;
          }
        }
        for (int i = 0; i < d_k; ++i) {
          double ki = b * widen(K, kv_dtype, th * d_k + i);
          for (int j = 0; j < d_v; ++j) S[i * d_v + j] += ki * r[j];
        }
        for (int j = 0; j < d_v; ++j) {
          double acc = 0.0;
          for (int i = 0; i < d_k; ++i) acc += widen(Q, kv_dtype, th * d_k + i) * S[i * d_v + j];
          O[th * d_v + j] = scale * acc;
        }
      }
      if (S_out) for (int i = 0; i < d_k * d_v; ++i) S_out[((size_t)s * H + h) * d_k * d_v + i] = S[i];
    }
    free(S);
    free(r);
  }
  return 0;
}
