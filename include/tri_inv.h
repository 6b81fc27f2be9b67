/*
 * tri_inv.h -- C ABI of the B200 (sm_100a) chunkwise delta-rule triangular inversion.
 *
 * For every chunk of C tokens of every (sequence, head) the library forms the
 * strictly lower triangular matrix
 *
 *     N_ij = beta_i * (k_i . k_j) * exp(g_i - g_j)   (i > j),   0 otherwise
 *
 * (Eq. 3 of the paper with the DeltaNet/GDN rows of Table 1: phi = diag(beta) K K^T
 * masked by the strictly-lower ones matrix and scaled by the decay matrix
 * exp(g_i - g_j); the matrix inverted is I + N), computes
 *
 *     A = (I + N)^{-1}
 *
 * by one of the direct schemes of Sec. 3 and optionally applies it:
 *
 *     W = A diag(beta) K,      U = A diag(beta) V          (WY factors).
 *
 * Everything here is plain C: pointers and sizes, no C++ or torch types.
 * All tensor pointers are DEVICE pointers unless stated otherwise; the caller
 * allocates and owns every buffer.  Calls are asynchronous on the given CUDA
 * stream (a cudaStream_t passed as void*; NULL = the legacy default stream)
 * and never synchronise the device.  No function throws, aborts or traps;
 * every function returns a TRI_INV_* status.  There is no CPU fallback: on a
 * machine without a usable GPU the compute calls return TRI_INV_ERR_CUDA.
 *
 * TRI_INV_LOG=1 in the environment makes the build / WY / fused calls print one line per kernel launch on stderr
 * (shape, method, which kernel took it); nothing else in the library writes to a stream.
 *
 * Shared state and its limits.  (1) One status word per device, shared by all streams and all
 * entry points: tri_inv_last_device_status() reports that SOME kernel since the last read gave up
 * on a wait, not which.  (2) The tensor-core kernels spread their work with a counter pair in
 * device memory that must serve one launch at a time.  Launches into one stream run one after the
 * other, so every stream gets a pair of its own; 64 pairs exist per device.  Launches on a 65th and
 * further streams, and every launch made while its stream is being captured into a CUDA graph, use a
 * fixed work distribution instead: same results, slightly less even load.  Neither case is an error.
 * (Programmatic dependent launch, which lets kernels of one stream overlap, must not be enabled on
 * this library's launches.)
 *
 * Tensor layouts (contiguous, row-major, flat token index t in [0, B*T)):
 *   K     [B, T, H, d_k]   kv_dtype (fp32, or bf16 as 16-bit patterns)
 *   V     [B, T, H, d_v]   kv_dtype
 *   beta  [B, T, H]        fp32
 *   g     [B, T, H]        fp32, cumulative log-decay within each chunk (only
 *                          differences inside a chunk are used)
 *   A     [B, T, H, C]     fp32; row = token, column j = j-th token of its chunk.
 *                          Upper triangle is +0.0 and the diagonal 1.0f, bit-exact.
 *   W     [B, T, H, d_k]   kv_dtype (round-to-nearest-even from fp32 accumulators)
 *   U     [B, T, H, d_v]   kv_dtype
 * Base pointers must be 16-byte aligned.
 *
 * Chunking: dense mode (cu_seqlens == NULL) has B sequences of T tokens; ragged
 * mode has B == 1, T == total tokens and sequence s = [cu_seqlens[s], cu_seqlens[s+1]).
 * Chunks restart at each sequence start.  A short last chunk with r < C tokens
 * is the leading r x r block of an identity-padded problem: only its r rows
 * are written, with columns >= r of A equal to +0.0.  Rows that belong to no
 * token are never read as data nor written.
 */
#ifndef TRI_INV_H_
#define TRI_INV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------- */
enum {
  TRI_INV_OK = 0,
  TRI_INV_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, bad size, bad cu_seqlens */
  TRI_INV_ERR_UNSUPPORTED = 2,   /* a valid request this build has no kernel for */
  TRI_INV_ERR_CUDA = 3,          /* a CUDA runtime call or the launch failed */
  TRI_INV_ERR_DEVICE_TIMEOUT = 4,/* a bounded device-side wait expired (see tri_inv_last_device_status) */
  TRI_INV_ERR_TOO_LARGE = 5,     /* more chunks than the fixed scratch of tri_inv_fused_packed_static holds */
  TRI_INV_ERR_DEBUG_CHECK = 6    /* device status word only, bounds-checking build only (-DTRI_INV_DEBUG): a kernel
                                    found an index outside its buffer or tile, or an mbarrier phase out of step;
                                    the access concerned was skipped, nothing trapped */
};

/* ---- storage type of K, V, W, U ------------------------------------------ */
enum { TRI_INV_F32 = 0, TRI_INV_BF16 = 1 };

/* ---- inversion scheme ("method" argument) -------------------------------- */
enum {
  /* 2x2 block recursion A = [[A11, 0], [-A22 N21 A11, A22]] from 16x16 leaves
   * (Sec. 3.3, Eq. for the block inverse written for a lower-triangular matrix;
   * the unrolled form is Alg. 4).  Leaves by forward substitution (Sec. 3.1). */
  TRI_INV_BLOCK_RECURSIVE = 0,
  /* Repeated squaring of the nilpotent series (Alg. 5 / Sec. 3.2):
   * X <- I - N, Y <- N, then log2(C) - 1 rounds of Y <- Y.Y, X <- X + X.Y,
   * i.e. prod_k (I + (-N)^(2^k)).  Exact in exact arithmetic, not stable. */
  TRI_INV_PRODUCT_SERIES = 1,
  /* Newton-Schulz iteration (Alg. 3 / Sec. 3.5): X_0 = I / C, X <- X (2I - (I + N) X).  Iterative: the
   * result converges to the inverse; TRI_INV_NS_ITERS(m) sets the count (default 2 log2(C), the count
   * the paper reports as converged at C = 64).  Runs on the fp32 CUDA-core kernel. */
  TRI_INV_NEWTON_SCHULZ = 2,
  TRI_INV_METHOD_MASK = 0xff,
  /* flag, block-recursive only: invert the 16x16 leaves with the product series
   * instead of substitution -- the mixed recursion of Alg. 2 (r = 0). */
  TRI_INV_LEAF_SERIES = 0x100,
  /* flag: one step of iterative refinement after the inversion (Alg. 6 / Sec. 3.6):
   * R <- I - A (I + N), A <- A + R A.  Block recursion and Newton-Schulz only.  After the block recursion on the
   * tensor-core kernel the residual is formed from TF32 hi/lo splits of both factors (three products, fp32
   * accumulation) and the correction R A in one TF32 product; Newton-Schulz and fp32 inputs use the CUDA cores. */
  TRI_INV_REFINE = 0x200,
  /* flag, product series on the tensor-core kernel only (bf16 keys, d = 128, C = 64 or 128): the series' matrix
   * products take fp16 operands instead of TF32 ones -- the half-precision format Sec. 4.1 prefers to bf16; same
   * 11-bit significand as TF32, fp32 accumulation, but a range of 6e-8 .. 65504: powers of N that leave it overflow,
   * which the unstable series (Sec. 3.2) can produce on badly conditioned chunks.  Half the operand bytes and one
   * stored copy of Y for both operand roles: the fast form of the series.  Elsewhere TRI_INV_ERR_UNSUPPORTED. */
  TRI_INV_OPERANDS_F16 = 0x400,
  /* flag, tri_inv_build / tri_inv_fused / tri_inv_fused_raw: the decay matrix of Table 1's Comba row, A^{i-1/j}:
   *     N_ij = beta_i (k_i . k_j) exp(g_{i-1} - g_j)      (i > j)
   * -- row i decays from token j up to the token BEFORE i, which is what the recurrence
   * S_t = (alpha_t I - beta_t k_t k_t^T) S_{t-1} + beta_t k_t v_t^T gives (its correction term reads the state before
   * this token's decay).  With TRI_INV_W_DECAY, row i of W is weighted by exp(g_{i-1}) (1 for the first row of a
   * chunk); tri_inv_chunk_scan then consumes W and U unchanged.  Other entry points: TRI_INV_ERR_UNSUPPORTED. */
  TRI_INV_GATE_SHIFTED = 0x800,
  /* Newton-Schulz iteration count, 1..15, in bits 12..15 (0 = default) */
#define TRI_INV_NS_ITERS(m) (((m) & 0xf) << 12)
  /* flag: run the plain fp32 CUDA-core kernel even where a tensor-core kernel
   * exists (same results up to rounding; for cross-checks and odd shapes).  Tensor-core kernels exist for bf16
   * storage with d_k = d_v = 128 at C = 64 and 128 (every scheme but Newton-Schulz) and with d_k = d_v = 64 at
   * C = 64 (block recursion, with or without TRI_INV_LEAF_SERIES, no other flag). */
  TRI_INV_FORCE_SIMT = 0x10000,
  /* flag, tri_inv_fused / tri_inv_fused_raw only: W = A diag(beta) diag(exp g) K, the decay-weighted factor
   * that the chunk form of the layer's recurrence subtracts from U (tri_inv_chunk_scan consumes it).  U is
   * unchanged.  Other entry points answer TRI_INV_ERR_UNSUPPORTED. */
  TRI_INV_W_DECAY = 0x20000
};

/* ---- problem descriptor --------------------------------------------------- */
typedef struct tri_inv_desc {
  int32_t B;        /* sequences in dense mode; must be 1 in ragged mode */
  int32_t T;        /* tokens per sequence (dense) or total tokens (ragged) */
  int32_t H;        /* heads */
  int32_t d_k;      /* key dimension   (multiple of 8) */
  int32_t d_v;      /* value dimension (multiple of 8); ignored by tri_inv_build */
  int32_t C;        /* chunk size: 16, 32, 64 or 128 */
  int32_t kv_dtype; /* TRI_INV_F32 or TRI_INV_BF16 */
  int32_t n_seqs;   /* ragged mode: number of sequences; else 0 */
  const int32_t* cu_seqlens; /* HOST pointer to n_seqs+1 non-decreasing offsets with
                                cu_seqlens[0] == 0 and cu_seqlens[n_seqs] == T, or NULL.
                                Read during the call only. */
} tri_inv_desc;

/*
 * A = (I + N)^{-1} for every chunk: the matrix of Eq. 3 with the phi of Table 1's DeltaNet / GDN rows,
 * inverted by one of the direct schemes of Sec. 3 (`method`).
 *   K, beta, g : inputs (device).   A : output (device), rows of real tokens only.
 * Errors: INVALID_ARG for null/misaligned pointers or an inconsistent descriptor,
 * UNSUPPORTED for an unknown method, CUDA if the launch fails.
 */
int tri_inv_build(const void* K, const float* beta, const float* g, float* A,
                  const tri_inv_desc* desc, int method, void* cuda_stream);

/*
 * W = A diag(beta) K and U = A diag(beta) V from a given A
 * (the WY/UT transform that the inverse exists for, Sec. 1).  A is read as stored by tri_inv_build;
 * only its strict lower triangle is used (the diagonal is taken as 1, the upper
 * triangle as 0).  V and U may both be NULL to compute W only.
 */
int tri_inv_wy(const float* A, const void* K, const void* V, const float* beta,
               void* W, void* U, const tri_inv_desc* desc, void* cuda_stream);

/*
 * Fused build + invert + WY in one kernel: K and V tiles are read once.
 * A may be NULL when only W and U are wanted.
 */
int tri_inv_fused(const void* K, const void* V, const float* beta, const float* g,
                  float* A, void* W, void* U,
                  const tri_inv_desc* desc, int method, void* cuda_stream);

/*
 * Per-channel decay (the KDA row of Table 1: phi = (K * Gamma)(K / Gamma)^T, Gamma = exp(G)):
 *     N_ij = beta_i * sum_c K_ic K_jc exp(G_ic - G_jc)   (i > j),      A = (I + N)^{-1}
 * G [B,T,H,d_k] fp32 is the cumulative per-channel log-decay inside each chunk (only differences inside a
 * chunk are used).  Same layouts, chunking modes, methods and error codes as tri_inv_build.  On the tensor
 * cores (bf16 keys, d_k = 128, C = 64 or 128, block recursion) the two factors are formed around a reference
 * row -- the chunk's middle row at C = 64, the middle row of each half at C = 128 -- so |G_i - G_ref| log2(e)
 * must stay inside the fp32 exponent range (about 88 in natural-log units), and at C = 128 G must not increase
 * from the first half of a chunk to the middle of the second (a cumulative log-decay never does);
 * other shapes take the exponent of each difference directly.
 */
int tri_inv_build_kda(const void* K, const float* G, const float* beta, float* A,
                      const tri_inv_desc* desc, int method, void* cuda_stream);

/*
 * tri_inv_fused for tensors in HOST memory (no step of the paper's method: the end-to-end form of the fused call).
 *   K, V, beta, g        HOST inputs, layouts as above; pinned (page-locked) memory makes the copies asynchronous
 *   A (nullable), W, U   HOST outputs
 *   workspace            DEVICE memory, 256-byte aligned, at least tri_inv_fused_host_workspace(desc) bytes, the caller's
 * The batch is cut into up to 16 slices of whole chunks (a dense batch whose T is a multiple of C; anything else goes as
 * one slice); each slice is copied in, run through tri_inv_fused and copied out on one of three streams the library keeps
 * per device, so uploads, kernels and downloads overlap.  The work is ordered after what is already in cuda_stream, and
 * cuda_stream is made to wait for all of it: synchronising cuda_stream (or an event recorded on it) after the call
 * covers the outputs.  The call itself returns after enqueueing when the host buffers are pinned.  One call at a time per
 * device: calls from several host threads must be serialised by the caller (they share the three streams).  Results are
 * those of tri_inv_fused.  Errors as for tri_inv_fused; INVALID_ARG also for a workspace that is too small or misaligned.
 */
int tri_inv_fused_host_workspace(const tri_inv_desc* desc, size_t* bytes);
int tri_inv_fused_host(const void* K, const void* V, const float* beta, const float* g,
                       float* A, void* W, void* U, void* workspace, size_t workspace_bytes,
                       const tri_inv_desc* desc, int method, void* cuda_stream);

/*
 * Per-channel decay through the WY step (KDA row of Table 1, with the decay-weighted factor the layer's chunk form needs):
 *     A = (I + N)^{-1},  N as for tri_inv_build_kda;     W = A diag(beta) (K * Gamma),  Gamma = exp(G);     U = A diag(beta) V
 * (the recurrence S_t = (I - beta_t k_t k_t^T) diag(alpha_t) S_{t-1} + beta_t k_t v_t^T re-bracketed per chunk gives
 * (I + N) U~ = diag(beta) V - diag(beta) (K * Gamma) S, i.e. U~ = U - W S; tri_inv_chunk_scan_kda consumes W and U).
 *   K, V, W, U [B,T,H,d] kv_dtype;  G [B,T,H,d_k] fp32;  beta [B,T,H] fp32;  A [B,T,H,C] fp32 -- all required (at C = 128
 *   A is also the hand-over between two launches).  W may not alias K; G as for tri_inv_build_kda (and exp(G_ref) must be
 *   representable: G is a cumulative log-decay, at most 0).
 * bf16 with d_k = d_v = 128 and the block recursion runs on the tensor cores: at C = 64 as ONE kernel (build, inversion and
 * both factors; W is formed as (A diag(beta) (K * exp(G - G_ref))) diag(exp G_ref), G_ref the chunk's middle row, so no
 * factor leaves exp(+-|G over 32 tokens|)), at C = 128 as two launches on the stream (tri_inv_build_kda's kernel, which
 * also writes K * Gamma into the W buffer while it holds K and G on chip; then tri_inv_wy's kernel on that buffer, in
 * place); everything else is one launch of the CUDA-core kernel.  TRI_INV_GATE_SHIFTED and TRI_INV_W_DECAY do not apply
 * (W is always the decay-weighted one).
 */
int tri_inv_fused_kda(const void* K, const void* V, const float* G, const float* beta,
                      float* A, void* W, void* U, const tri_inv_desc* desc, int method, void* cuda_stream);

/*
 * The chunk scan with one decay per key feature (KDA row): as tri_inv_chunk_scan with g replaced by G [B,T,H,d_k] fp32,
 *     U~ = U - W S,     P_ij = sum_c Q_ic K_jc exp(G_ic - G_jc)  (j <= i),
 *     O  = scale * ((Q * Gamma) S + P U~),     S <- diag(Gamma_last) S + (K * exp(G_last - G))^T U~,
 * W and U from tri_inv_fused_kda.  bf16 with d_k = d_v = 128 and C = 64 runs on the tensor cores, in two launches on the
 * stream: a pass that folds the decays into the operands around each chunk's middle row G_ref and last row G_last
 * (Q exp(G - G_ref), K exp(G_ref - G), W exp(-G_ref), and per chunk the vectors exp(G_last), exp(G_ref),
 * exp(G_last - G_ref): |G_i - G_ref| must stay inside the fp32 exponent range, about 88 in natural-log units, and G must
 * not increase along a chunk), then the scan kernel of
 * tri_inv_chunk_scan on them.  The pass writes into stream-ordered scratch memory of three times the size of K (from a
 * memory pool that the library keeps per device: handed back to the pool behind the scan and reused by later calls, so
 * it stays reserved for the life of the process); TRI_INV_ERR_CUDA if it cannot be had.  Every other shape and fp32
 * storage run on the CUDA cores in fp32 (d_k <= 256), where the exponent is taken of each difference and G is not
 * restricted.
 */
int tri_inv_chunk_scan_kda(const void* Q, const void* K, const void* W, const void* U, const float* G, const float* S0,
                           void* O, float* S_out, float scale, const tri_inv_desc* desc, void* cuda_stream);

/*
 * Chunk scan: the consumer of W and U -- the chunk form of the layer's recurrence (the re-formulation Sec. 1
 * refers to, in which (I+N)^{-1} appears through W and U).  Per sequence and head, chunk after chunk, with the
 * state S [d_k x d_v] entering the chunk (S0, or zero) and gamma_i = exp(g_i):
 *     U~ = U - W S
 *     O  = scale * (diag(gamma) Q S + ((Q K^T) * D) U~),     D_ij = gamma_i / gamma_j for j <= i, else 0
 *     S <- gamma_last S + (diag(gamma_last / gamma) K)^T U~
 * W must be the decay-weighted factor (TRI_INV_W_DECAY of the fused calls), U the plain one.  With exact W and U
 * this equals the token-by-token recurrence  S <- exp(a_t) S;  S <- S + beta_t k_t (v_t - S^T k_t)^T;
 * o_t = scale S^T q_t.
 *   Q, K, W [B,T,H,d_k], U [B,T,H,d_v]: device, desc->kv_dtype, 16-byte aligned;  g [B,T,H] fp32 device;
 *   S0, S_out [n_sequences,H,d_k,d_v] fp32 device, each may be NULL (zero initial state / final state not wanted);
 *   O [B,T,H,d_v] device, desc->kv_dtype: rows of real tokens are written.
 * Dense and ragged chunking as in tri_inv_build (desc->cu_seqlens on the HOST).  bf16 with d_k = d_v = 128 and
 * C = 64 runs on the tensor cores; every other shape and fp32 storage run on the CUDA cores in fp32 (d_k <= 256,
 * else TRI_INV_ERR_UNSUPPORTED).  g is used as given (it need not decrease); the tensor-core path forms exp(g_i - g_j)
 * as a product of two factors around the first token of j's block of eight, so g may vary by at most about 88
 * inside eight consecutive tokens of a chunk.  Launch is asynchronous on
 * cuda_stream; nothing is allocated except, in ragged mode, n_sequences + 1 ints from the library's
 * stream-ordered pool.  A device-side wait that expires raises TRI_INV_ERR_DEVICE_TIMEOUT in the status word.
 */
int tri_inv_chunk_scan(const void* Q, const void* K, const void* W, const void* U, const float* g, const float* S0,
                       void* O, float* S_out, float scale, const tri_inv_desc* desc, void* cuda_stream);

/*
 * Fused call with the layer's front end folded in: the kernel takes what the projections produce and
 * does the three producers that otherwise run as separate passes over memory before the inversion
 * (the gating recipe of a Gated-DeltaNet layer; in the paper these are among the kernels its fused
 * layer kernel absorbs, Sec. 5.2):
 *     beta_t = sigmoid(beta_logit_t)
 *     g_t    = sum over s <= t of the same chunk of log sigmoid(gate_logit_s)
 *     k^_t   = K_raw_t / ||K_raw_t||_2            (a zero key stays zero)
 * and then N, A, W = A diag(beta) K^ and U = A diag(beta) V exactly as tri_inv_fused does with K^, beta, g.
 * The norms come from the diagonal of the Gram product, so normalising costs no extra pass.
 *   K_raw, V            [B,T,H,d] kv_dtype;   beta_logit, gate_logit  [B,T,H] fp32
 *   beta_out, g_out     optional [B,T,H] fp32 outputs (beta and the cumulative log-decay, for the
 *                       layer's later steps); NULL to skip
 * A may be NULL.  All methods and both chunking modes of tri_inv_fused apply.
 */
int tri_inv_fused_raw(const void* K_raw, const void* V, const float* beta_logit, const float* gate_logit,
                      float* A, void* W, void* U, float* beta_out, float* g_out,
                      const tri_inv_desc* desc, int method, void* cuda_stream);

/*
 * Packed-sequence fused call that allocates nothing.  (The paper has no counterpart: this is a
 * deployment variant of tri_inv_fused, not a step of the method.)
 *
 * tri_inv_fused in packed mode (cu_seqlens != NULL) keeps a small table of chunk positions in device
 * memory that it allocates and frees on the stream.  Callers that may not allocate -- code that runs
 * where cudaMalloc is forbidden or would stall, a process with a memory budget fixed at start-up, a
 * host whose allocator belongs to another component -- can use this entry point instead: the table
 * lives in a fixed device array inside the library (128 KiB, held by every GPU that loads the library
 * until the process exits).  No cudaMalloc, cudaFree or other allocating call is made; inputs and
 * outputs are the caller's, exactly as for tri_inv_fused, and results are identical.
 *
 *   - Packed mode only: desc->cu_seqlens must be non-NULL (dense calls never allocate; use tri_inv_fused).
 *   - At most TRI_INV_STATIC_MAX_CHUNKS chunks of tokens (sum over sequences of ceil(len / C));
 *     more returns TRI_INV_ERR_TOO_LARGE and does nothing.
 *   - The first call on each device looks up the array's device address (with that device current);
 *     make that first call outside of any stream capture.
 *   - All calls share the one array.  Two calls whose kernels can overlap on the GPU (different
 *     streams, or the same stream from different host threads without ordering) race on it: order
 *     them.  Calls on one stream are safe.
 */
#define TRI_INV_STATIC_MAX_CHUNKS 16384
int tri_inv_fused_packed_static(const void* K, const void* V, const float* beta, const float* g,
                                float* A, void* W, void* U,
                                const tri_inv_desc* desc, int method, void* cuda_stream);

/*
 * Self-test of the give-up path of the device-side waits (no step of the paper's method).  Runs tri_inv_fused
 * (block recursion; bf16, d_k = d_v = 128, C = 64 or 128 only) with every wait limited to wait_limit_ns
 * nanoseconds instead of two seconds, and with the first thread block leaving out the Gram product of its first
 * chunk matrix, so that its wait for that product runs out.  Nothing faults, traps or spins without a limit: the
 * block raises the status word, finishes that one matrix on undefined data (its rows of A, W, U are then
 * undefined), waits -- again bounded -- for what it still has in flight, frees its tensor memory and returns
 * without taking further work (with more matrices than resident thread blocks, its second matrix stays
 * unwritten too); the other blocks do the rest of the batch as usual.  The call synchronises the stream and sets *counters_idle to 1 if
 * the kernel left every work-distribution counter of the device at zero.  Afterwards
 * tri_inv_last_device_status() reads TRI_INV_ERR_DEVICE_TIMEOUT (once), and the library is usable as before.
 */
int tri_inv_selftest_wait_timeout(const void* K, const void* V, const float* beta, const float* g,
                                  float* A, void* W, void* U, const tri_inv_desc* desc,
                                  uint64_t wait_limit_ns, int* counters_idle, void* cuda_stream);

/*
 * The same for the tensor-core chunk scan (bf16, d_k = d_v = 128, C = 64; no step of the paper's method): tri_inv_chunk_scan
 * (zero initial state, scale 1, final state not returned) with every device-side wait limited to wait_limit_ns nanoseconds
 * and with the first thread block -- sequence 0, head 0, the first slice of value columns -- leaving out the state-update
 * product of its second chunk.  The block's waits run out one after the other (each warp gives up at its next wait and
 * leaves its loop), it raises the status word, frees its tensor memory and returns; what it had written of O stays (its
 * first chunk), the rest of its columns of sequence 0, head 0 is undefined.  All other blocks finish as usual.  The limit
 * should leave a tile copy time to land (tens of microseconds are plenty).  The call synchronises the stream; afterwards
 * tri_inv_last_device_status() reads TRI_INV_ERR_DEVICE_TIMEOUT (once), and the library is usable as before.
 */
int tri_inv_selftest_scan_wait_timeout(const void* Q, const void* K, const void* W, const void* U, const float* g, void* O,
                                       const tri_inv_desc* desc, uint64_t wait_limit_ns, void* cuda_stream);

/*
 * The same for the per-channel kernels (bf16, d_k = d_v = 128, C = 64 or 128, block recursion; no step of the paper's
 * method): tri_inv_fused_kda -- or, with V, W and U all NULL, tri_inv_build_kda -- with every device-side wait limited to
 * wait_limit_ns nanoseconds and with the first thread block leaving out the Gram product of its first chunk matrix (chunk
 * 0, head 0).  That block's waits run out, it raises the status word, finishes the one matrix on undefined data (its rows
 * of A, W, U are then undefined), waits -- bounded -- for the copies it still has in flight, frees its tensor memory and
 * returns without taking further work: these kernels hand out work with a fixed stride, so with more matrices than
 * resident thread blocks (three per SM at C = 64, two at C = 128) the block's later matrices stay unwritten as well.  All
 * other blocks finish as usual.  The call synchronises the stream; afterwards tri_inv_last_device_status() reads
 * TRI_INV_ERR_DEVICE_TIMEOUT (once), and the library is usable as before.
 */
int tri_inv_selftest_kda_wait_timeout(const void* K, const void* V, const float* G, const float* beta,
                                      float* A, void* W, void* U, const tri_inv_desc* desc,
                                      uint64_t wait_limit_ns, void* cuda_stream);

/*
 * Self-test of the bounds-checking build (no step of the paper's method).  tri_inv_fused (block recursion) with the token
 * bound that the debug build's checks use understated by one chunk: the buffers are as large as the descriptor says, so
 * no access is out of range either way.  In the bounds-checking build (libtri_inv_debug.so) the work items of the last
 * chunk of tokens fail their range check, are reduced to no rows (their rows of A, W, U stay unwritten) and the status
 * word reads TRI_INV_ERR_DEBUG_CHECK; in the ordinary build the call is tri_inv_fused.
 */
int tri_inv_selftest_bounds_check(const void* K, const void* V, const float* beta, const float* g,
                                  float* A, void* W, void* U, const tri_inv_desc* desc, void* cuda_stream);

/*
 * Number of chunk matrices (chunks x heads) the descriptor describes.
 * Host-only arithmetic; no device work.
 */
int tri_inv_count_matrices(const tri_inv_desc* desc, int64_t* out);

/*
 * After the caller has synchronised the stream: reads and clears the device
 * status word of the current device.  *out is TRI_INV_OK, or
 * TRI_INV_ERR_DEVICE_TIMEOUT if a kernel gave up on a bounded wait (the
 * kernel then returned early and its outputs are incomplete).  This call
 * copies 4 bytes from the device and so synchronises with it.
 */
int tri_inv_last_device_status(int* out);

/* Kernel launches issued by this library in this process so far (host counter). */
int64_t tri_inv_launch_count(void);

/* Static string for a status code. */
const char* tri_inv_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* TRI_INV_H_ */
