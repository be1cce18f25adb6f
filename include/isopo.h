/*
 * isopo.h - C ABI of the B200 (sm_100a) implementation of the ISOPO per-linear-layer path.
 *
 * ISOPO ("Isometric Policy Optimization") transforms, layer by layer inside one backward pass,
 * the advantages of the B sequences of a ragged microbatch before they are contracted with the
 * per-sequence log-probability gradients of the layer's weight.  For one linear layer with packed
 * input activations X [T, d_in] and output gradients dY [T, d_out] (the backward pass is run on
 * sum(log_prob) WITHOUT advantages; Algorithm 1 and Algorithm 2 of the paper) the path is
 *
 *     G_i  = sum_{t in sequence i} dY[t,:]^T X[t,:]          [d_out, d_in]   (Alg. 1/2, reduce loop)
 *     K_ij = <G_i, G_j>                                       [B, B]          (Alg. 2, NTK; Sec. 3 K = J J^T)
 *     c    = transform(K, A)                                  [B]             (Sec. 2.1, 2.3, Fig. 3, Sec. 3)
 *     dW   = sum_i c_i G_i = (c_seq(t) * dY)^T X              [d_out, d_in]   (Alg. 1/2, accumulate)
 *
 * Conventions shared by every entry point
 *   - "dev" pointers are CUDA device pointers of the current device, "host" pointers are ordinary
 *     host memory.  The caller owns every buffer; the library never allocates or frees device memory.
 *   - X and dY are row-major, contiguous, 16-byte aligned; row t is token t of the packed microbatch;
 *     sequence i owns rows seq_offsets[i] .. seq_offsets[i+1]-1, with seq_offsets[0] = 0,
 *     seq_offsets[B] = T and every length >= 1.
 *   - All work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and the call returns without synchronising.  The three calls of one layer must be issued in
 *     order on the same stream with the same workspace.
 *   - The return value reports what the host can detect (bad arguments, unsupported shapes, a
 *     workspace that is too small, a CUDA launch error).  Conditions found on the device are
 *     written to `*info` (dev, int32), which the caller zeroes beforehand and reads after
 *     synchronising the stream: 0 = ok; 1..B = the leading minor of that order of K + lambda*I is
 *     not positive definite (interacting transform); ISOPO_INFO_TIMEOUT | id = a bounded wait inside
 *     kernel `id` ran out.  The library only ever overwrites a zero `*info`.  When `*info` != 0 the
 *     outputs are unspecified (but every access stayed in bounds).
 *   - There is no CPU fallback; one GPU per call (the current device).
 *   - Process-wide state, all of it host side: the measurement hooks' event list (isopo_profile_*), the
 *     deterministic-mode switch (isopo_set_deterministic), per-device caches of launch limits, and the
 *     device address of isopo_layer_gram_static's scratch.  Host threads: isopo_status_string,
 *     isopo_kernel_name, isopo_choose_path, the *_workspace_bytes queries and isopo_last_cuda_error
 *     (thread-local) may be called from any thread at any time.  The entry points that enqueue work may
 *     be called from several host threads at once as long as profiling is disabled, no thread changes
 *     the deterministic-mode switch meanwhile, and each thread uses its own workspace, outputs and
 *     `info`; the per-device caches are filled with identical values by whichever thread comes first.
 *     isopo_profile_enable / isopo_profile_collect, isopo_set_deterministic and
 *     isopo_layer_gram_static (it pauses profiling and shares one scratch array) must not run
 *     concurrently with any other call of the library.
 *   - Under a profiler every entry point that enqueues work shows as an NVTX range of its own name.
 */
#ifndef ISOPO_H_
#define ISOPO_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ISOPO_API __attribute__((visibility("default")))
#else
#define ISOPO_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ISOPO_OK = 0,
  ISOPO_ERR_INVALID_ARG = 1,  /* null pointer, bad size, bad offsets, misaligned buffer */
  ISOPO_ERR_UNSUPPORTED = 2,  /* valid request that the library has no kernel for */
  ISOPO_ERR_WORKSPACE = 3,    /* ws_bytes smaller than isopo_workspace_bytes(...) */
  ISOPO_ERR_CUDA = 4          /* a CUDA runtime/driver call failed; see isopo_last_cuda_error() */
} isopo_status;

typedef enum {
  ISOPO_F32 = 0,   /* X, dY float32; SIMT FFMA kernels, K accumulated in float64 */
  ISOPO_BF16 = 1   /* X, dY bfloat16; tcgen05 tensor-core kernels, float32 accumulation */
} isopo_dtype;

typedef enum {
  ISOPO_PATH_AUTO = 0,        /* cost model picks one of the two below (isopo_choose_path) */
  ISOPO_PATH_GRAM = 1,        /* K from token Grams, never forms G_i */
  ISOPO_PATH_MATERIALISE = 2  /* forms every G_i in the workspace, K from them, dW from them */
} isopo_path;

typedef enum {
  ISOPO_VAR_REINFORCE = 0,      /* c_i = A_i */
  ISOPO_VAR_NORMALISED = 1,     /* c_i = A_i / sqrt(F_i^2 + lambda)           Sec. 2.1 display; Fig. 3 p = -1 */
  ISOPO_VAR_DIRECTION = 2,      /* c_i = A_i / (F_i^2 / K_ii + lambda)        Sec. 2.3 display; Fig. 3 r = -2 */
  ISOPO_VAR_EUCLID = 3,         /* c_i = A_i / sqrt(K_ii + lambda)            Fig. 3 q = -1 */
  ISOPO_VAR_GENERAL = 4,        /* Fig. 3 with free p, q, r and three absolute regularisers */
  ISOPO_VAR_INTERACTING = 5,    /* (K + lambda I) c = A                       Sec. 3 display; Alg. 2 */
  ISOPO_VAR_NORMALISED_RAW = 6  /* as NORMALISED with F_i^2 = (1/B) sum_j K_ij^2 (Eq. F-norm-basic as printed) */
} isopo_variant;

#define ISOPO_INFO_TIMEOUT 0x40000000
#define ISOPO_INFO_NO_CONVERGENCE 0x20000000 /* isopo_transform_spectral: sweeps ran out; low bits = sweeps done */
#define ISOPO_INFO_SATURATED 0x04000000 /* split e4m3 store: an element of some s_i G_i exceeded the format's range (448) and was clamped */
#define ISOPO_INFO_BOUNDS 0x08000000 /* debug build only (isopo_debug_build): kernel `id` computed an index outside its buffer; the access was skipped */
#define ISOPO_INFO_STALE_WORKSPACE 0x10000000 /* isopo_weight_grad(MATERIALISE): the workspace holds another layer's or microbatch's gradients */

/* Human-readable name of a status code (static storage, never NULL). */
ISOPO_API const char* isopo_status_string(isopo_status s);

/* Text of the last CUDA error seen by this thread inside the library (static storage). */
ISOPO_API const char* isopo_last_cuda_error(void);

/*
 * Path that ISOPO_PATH_AUTO resolves to for these sizes.  The Gram route costs
 * (d_in + d_out) * sum_i-over-token-pairs ~ (d_in + d_out) T^2 flops; the materialised route adds
 * B^2 d_in d_out flops and three passes over B d_in d_out stored gradients to the plain dW GEMM
 * (whose 2 T d_in d_out flops it re-uses).  Gram wins only for short sequences.
 */
ISOPO_API isopo_path isopo_choose_path(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B);

/*
 * Bytes of device workspace the three calls of one layer need for `path` (AUTO allowed).
 * The workspace holds the device copy of the offsets, the token -> sequence map and, on the
 * materialised path, all B per-sequence gradients (bf16 for ISOPO_BF16, float32 for ISOPO_F32)
 * in a piece-blocked order private to the library; on the bf16 Gram path, the per-token-scaled
 * copy of the narrower of X and dY that isopo_weight_grad feeds to its GEMM
 * (2 * T * min(d_in, d_out) bytes).  It must be 1024-byte aligned (cudaMalloc promises 256 bytes only: allocate
 * 1024 bytes more and round the pointer up).  Returns 0 for invalid sizes.
 */
ISOPO_API size_t isopo_workspace_bytes(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, isopo_path path);

/*
 * isopo_layer_gram: K_ij = <G_i, G_j>  (Alg. 2 "make neural tangent kernel"; K = J J^T of Sec. 3).
 *
 * GRAM path: uses that each token gradient is the rank-one matrix dY_t x_t^T (Eq. one, Eq. two), so
 *   K_ij = sum_{t in i, s in j} (dY_t . dY_s)(x_t . x_s): tiles of X X^T and dY dY^T are formed in
 *   tensor memory, multiplied elementwise and segment-summed; no T x T matrix reaches memory.
 * MATERIALISE path: forms G_i = dY_i^T X_i (Alg. 2 reduce loop) for every i into the workspace, then
 *   K = G_flat G_flat^T.
 *
 *   X, dY            dev, [T, d_in] and [T, d_out] of `dtype`, row-major
 *   seq_offsets_host host, int64 [B+1]; copied before the call returns
 *   K                dev, float32 [B, B] row-major, overwritten; exactly symmetric on return
 *   ws, ws_bytes     dev workspace, see isopo_workspace_bytes
 *   info             dev int32, see above
 * ISOPO_BF16 requires d_in and d_out to be multiples of 8; the bf16 MATERIALISE path requires B <= 256.
 */
ISOPO_API isopo_status isopo_layer_gram(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in, int d_out,
                              const int64_t* seq_offsets_host, int B, isopo_path path, float* K, void* ws,
                              size_t ws_bytes, int32_t* info, void* cuda_stream);

/*
 * isopo_layer_gram_shared_x: isopo_layer_gram on the Gram route for up to three projections that
 * read the SAME input X (q/k/v, gate/up of a transformer block): K^(h) = layer NTK of projection h
 * (Eq. one / Eq. two per layer).  The token Gram X X^T is formed once per pair of token tiles and
 * multiplied with each projection's dY^(h) dY^(h)^T, so the X contraction and the loads of X are paid
 * once instead of n_proj times.  bfloat16 only; results as n_proj calls of isopo_layer_gram with
 * ISOPO_PATH_GRAM (float atomics: not bit-identical).
 *
 *   X        dev, bf16 [T, d_in]
 *   n_proj   1 .. 3
 *   dY       HOST array of n_proj device pointers, dY[h] bf16 [T, d_out[h]]
 *   d_out    HOST array of n_proj widths (multiples of 8)
 *   K        HOST array of n_proj device pointers, each float32 [B, B], overwritten
 *   ws       dev, isopo_workspace_bytes(dtype, T, d_in, max_h d_out[h], B, ISOPO_PATH_GRAM) bytes, 1024-byte aligned
 * Follow it with isopo_weight_grad(X, dY[h], ..., ISOPO_PATH_GRAM, ...) per projection (each with a
 * workspace of its own size; the call refreshes what it needs).
 */
ISOPO_API isopo_status isopo_layer_gram_shared_x(const void* X, int n_proj, const void* const* dY, const int* d_out,
                                                 isopo_dtype dtype, int64_t T, int d_in,
                                                 const int64_t* seq_offsets_host, int B, float* const* K, void* ws,
                                                 size_t ws_bytes, int32_t* info, void* cuda_stream);

/*
 * isopo_layer_gram_shared_x_stored: isopo_layer_gram on the MATERIALISE route for up to three
 * projections that read the same input X (Alg. 2 reduce loop and NTK, per layer).  All projections'
 * G_i = dY_i^(h)T X_i are formed by ONE launch of the per-sequence gradient GEMM: their tile rows are
 * stacked into one grid, so X is staged once for all of them and narrow projections (the k/v shapes)
 * no longer leave the machine half empty; K^(h) = G^(h) G^(h)T follows per projection.  bfloat16 only,
 * B <= 256; results bit-identical to n_proj calls of isopo_layer_gram with ISOPO_PATH_MATERIALISE except for
 * the order of the float atomic additions into K.
 *
 *   dY, d_out, K   HOST arrays of n_proj entries as for isopo_layer_gram_shared_x
 *   ws, ws_bytes   HOST arrays: ws[h] is projection h's own workspace of at least
 *                  isopo_workspace_bytes(dtype, T, d_in, d_out[h], B, ISOPO_PATH_MATERIALISE) bytes (1024-byte
 *                  aligned, all distinct); it receives that projection's stored gradients and tag
 * Follow it with isopo_weight_grad(X, dY[h], ..., ISOPO_PATH_MATERIALISE, ..., ws[h], ...) per projection.
 */
ISOPO_API isopo_status isopo_layer_gram_shared_x_stored(const void* X, int n_proj, const void* const* dY, const int* d_out,
                                                        isopo_dtype dtype, int64_t T, int d_in,
                                                        const int64_t* seq_offsets_host, int B, float* const* K,
                                                        void* const* ws, const size_t* ws_bytes, int32_t* info,
                                                        void* cuda_stream);

/*
 * isopo_transform_advantages: advantages A -> coefficients c (dW = sum_i c_i G_i).
 *
 * With F_i^2 = sum_j K_ij^2 / sum_j K_jj (the Fisher norm of Eq. F-norm-basic evaluated with the B
 * sequence gradients as samples and normalised by their summed squared norms as in
 * Eq. formal-F-norm) the variants are those listed at isopo_variant.  ISOPO_VAR_GENERAL computes
 *   c_i = A_i * reg2(F_i; g[3])^g[0] * reg2(sqrt(K_ii); g[4])^g[1] * reg2(F_i / sqrt(K_ii); g[5])^g[2],
 *   reg2(v; reg) = sqrt(v^2 + reg + 1e-8)                                         (Fig. 3),
 * with g = opt_pqr_regs = {p, q, r, reg_F, reg_G, reg_rel} (host, 6 floats; required for GENERAL,
 * ignored otherwise; `lambda` is ignored for GENERAL).  ISOPO_VAR_INTERACTING factors K + lambda*I
 * by Cholesky in shared memory (float32) and refines the solution with float64 residuals; it
 * requires B <= 256 (isopo_transform_advantages_large takes up to 1024) and reports a non-positive pivot k
 * (1-based) as *info = k.
 *
 *   K       dev, float32 [B, B] row-major (as written by isopo_layer_gram)
 *   A       dev, float32 [B]
 *   lambda  absolute regulariser, >= 0 (the caller multiplies by its running mean if it wants a relative one)
 *   coeffs  dev, float32 [B], overwritten
 */
ISOPO_API isopo_status isopo_transform_advantages(const float* K, const float* A, int B, isopo_variant variant, float lambda,
                                        const float* opt_pqr_regs, float* coeffs, int32_t* info, void* cuda_stream);

/*
 * isopo_transform_advantages_large: the interacting variant, (K + lambda I) c = A (Sec. 3 display; Alg. 2), for
 * up to ISOPO_MAX_LARGE_SEQS sequences.  Same blocked Cholesky and float64-residual refinement as
 * isopo_transform_advantages, with the block triangle of the factor kept in `workspace` (2.1 MB at 1024
 * sequences: it stays in the L2) instead of shared memory; one CTA, milliseconds rather than 0.1 ms.  K of more than
 * 256 sequences comes from the GRAM path of isopo_layer_gram; the simple variants take any B in
 * isopo_transform_advantages.  A non-positive pivot k (1-based) is reported as *info = k, coeffs are then zero.
 *
 *   K          dev, float32 [B, B] row-major, symmetric; 1 <= B <= ISOPO_MAX_LARGE_SEQS
 *   A, coeffs  dev, float32 [B]
 *   lambda     absolute regulariser, >= 0
 *   workspace  dev, 16-byte aligned, at least isopo_transform_large_workspace_bytes(B) bytes (0 for a B out of
 *              range); scratch, contents undefined afterwards; must not be shared by calls that overlap
 * Errors: ISOPO_ERR_INVALID_ARG, ISOPO_ERR_UNSUPPORTED (B too large), ISOPO_ERR_WORKSPACE (too small).
 */
#define ISOPO_MAX_LARGE_SEQS 1024
ISOPO_API size_t isopo_transform_large_workspace_bytes(int B);
ISOPO_API isopo_status isopo_transform_advantages_large(const float* K, const float* A, int B, float lambda, float* coeffs,
                                                        void* workspace, size_t workspace_bytes, int32_t* info,
                                                        void* cuda_stream);

/*
 * Relative regularisation (Alg. 1: "use e.g. EMA of trailing minibatch means for the regularization";
 * generalised re-scaling figure: reg(val) = val + regularization * expectation(val); Sec. 4:
 * "regularization factor 1.0 * E[mean(D)] ... EMA over minibatches with 0.9 decay").
 *
 * isopo_reg_ema_update folds one microbatch's K into running means kept on the device, so that the
 * whole layer (gram -> update -> transform -> weight_grad) runs without the host reading anything:
 *     state[0] = E[F_i^2]   state[1] = E[K_ii] = E[mean(D)], the mean eigenvalue of K
 *     state[2] = E[F_i^2 / K_ii]   state[3] = number of updates so far
 * with F_i^2 = sum_j K_ij^2 / sum_j K_jj.  The caller zeroes the four floats once; the first update
 * stores the microbatch means, later ones blend  s <- decay * s + (1 - decay) * mean,  0 <= decay < 1.
 *
 * isopo_transform_advantages_rel is isopo_transform_advantages with the regulariser given as a
 * factor of the matching running mean, read on the device (the state as updated so far, i.e.
 * including the current microbatch if the update was issued first):
 *     NORMALISED(_RAW): lambda = factor * E[F^2]      DIRECTION: lambda = factor * E[F^2 / K_ii]
 *     EUCLID, INTERACTING: lambda = factor * E[K_ii]
 *     GENERAL: opt_pqr_factors = {p, q, r, factor_F, factor_G, factor_rel} (host), `factor` ignored.
 *
 *   state   dev, float32 [4]
 */
ISOPO_API isopo_status isopo_reg_ema_update(const float* K, int B, float decay, float* state, void* cuda_stream);
ISOPO_API isopo_status isopo_transform_advantages_rel(const float* K, const float* A, int B, isopo_variant variant,
                                                      float factor, const float* opt_pqr_factors, const float* state,
                                                      float* coeffs, int32_t* info, void* cuda_stream);

/*
 * isopo_transform_advantages_batched: the transform for several layers of one microbatch in ONE
 * launch (layer l on its own CTA, so the layers' solves run side by side instead of one after the
 * other).  The interacting solve of Alg. 2 is a single-CTA, latency-bound computation; a caller that keeps
 * the K of several projections (e.g. the seven of a transformer block) before asking for their
 * coefficients pays for one solve instead of n_layers.  All layers share A, B and the variant.
 *
 *   n_layers  1 .. ISOPO_MAX_BATCH
 *   K         HOST array of n_layers device pointers, each float32 [B, B] as for isopo_transform_advantages
 *   lambda    HOST array of n_layers regularisers (>= 0): absolute if states == NULL, else factors of
 *             the running means as in isopo_transform_advantages_rel (GENERAL: ignored either way,
 *             opt_pqr_regs holds the three absolute regularisers or factors for all layers)
 *   states    NULL, or HOST array of n_layers device pointers to float32 [4] running-mean states
 *   coeffs    HOST array of n_layers device pointers, each float32 [B], overwritten
 * The host arrays are read before the call returns.  A non-positive pivot k of layer l is reported
 * as *info = k + (l << 16) (the first one found wins).  Results are those of n_layers single calls.
 */
ISOPO_API isopo_status isopo_transform_advantages_batched(int n_layers, const float* const* K, const float* A, int B,
                                                          isopo_variant variant, const float* lambda,
                                                          const float* opt_pqr_regs, const float* const* states,
                                                          float* const* coeffs, int32_t* info, void* cuda_stream);

/*
 * isopo_transform_spectral: the interacting transform in the spectral form Alg. 2 prints,
 *     K = U D U^T,   c = U ((1 / (D + lambda)) * (U^T A)),
 * with the spectrum D as a second output (the quantity whose running mean regularises the
 * interacting experiment of Sec. 4).  Eigen-directions with D_k <= rel_cutoff * max(D) are left out
 * of the sum: rel_cutoff = 0 and a positive definite K give the coefficients of
 * ISOPO_VAR_INTERACTING; lambda = 0 with a cut-off gives the pseudo-inverse on the kept range, which
 * the Cholesky route cannot (it stops at a non-positive pivot).
 *
 * K is diagonalised by one-sided Jacobi rotations in float32 with float64 inner products, a cluster
 * of eight CTAs per K: milliseconds at B = 256, against ~0.1 ms for isopo_transform_advantages.  It is the
 * diagnostic variant; its float32 eigenbasis limits the coefficients to a relative error of about
 * 1e-7 * cond(K + lambda I) (kept range), the eigenvalues to ~1e-6 of the largest.
 *
 *   K            dev, float32 [B, B] row-major, symmetric (as written by isopo_layer_gram); B <= 256
 *   A            dev, float32 [B]
 *   lambda       >= 0;   rel_cutoff in [0, 1)
 *   coeffs       dev, float32 [B], overwritten
 *   eigenvalues  dev, float32 [B], from the largest down; may be NULL
 *   ws           dev, isopo_spectral_workspace_bytes() bytes, 16-byte aligned; contents destroyed
 * If the rotations have not died out after 30 sweeps, *info = ISOPO_INFO_NO_CONVERGENCE | sweeps
 * and the outputs are those of the last sweep.
 */
ISOPO_API size_t isopo_spectral_workspace_bytes(void);
ISOPO_API isopo_status isopo_transform_spectral(const float* K, const float* A, int B, float lambda, float rel_cutoff,
                                                float* coeffs, float* eigenvalues, void* ws, size_t ws_bytes,
                                                int32_t* info, void* cuda_stream);

/*
 * isopo_transform_spectral_batched: isopo_transform_spectral for several layers of one microbatch in
 * one launch, one cluster per layer side by side (the decomposition is latency-bound, so n_layers
 * of them take about the time of one).  Shared: A, B, rel_cutoff.
 *
 *   K, coeffs    HOST arrays of n_layers device pointers (1 <= n_layers <= ISOPO_MAX_BATCH)
 *   lambda       HOST array of n_layers regularisers
 *   eigenvalues  NULL, or HOST array of n_layers device pointers (entries may be NULL)
 *   ws           dev, n_layers * isopo_spectral_workspace_bytes() bytes, 16-byte aligned
 * A layer l that does not converge reports *info = ISOPO_INFO_NO_CONVERGENCE | (l << 16) | sweeps.
 */
ISOPO_API isopo_status isopo_transform_spectral_batched(int n_layers, const float* const* K, const float* A, int B,
                                                        const float* lambda, float rel_cutoff, float* const* coeffs,
                                                        float* const* eigenvalues, void* ws, size_t ws_bytes,
                                                        int32_t* info, void* cuda_stream);

/*
 * isopo_weight_grad: dW = beta * dW + sum_i coeffs[i] * G_i   (Alg. 1 "grad += advantages * rescaled
 * gradient" and "mod.grad += grad"; Alg. 2 "stack(seq_grads) @ advantages_preconditioned").
 *
 * `path` must be the value given to isopo_layer_gram for this layer (AUTO resolves identically).
 * MATERIALISE: streams the G_i left in the workspace by isopo_layer_gram.  The workspace carries a
 * tag (dtype, T, d_in, d_out, B, a hash of the offsets) written by that call; if this call's
 * arguments do not match it, dW is left untouched and *info = ISOPO_INFO_STALE_WORKSPACE.
 * GRAM: one GEMM over all tokens, dW = (coeffs[seq(t)] * dY)^T X.  bf16, layers whose wider side is
 * at most 2048 (and sequences of about 100 tokens or more): every run of tokens of one sequence is
 * accumulated on its own in tensor memory and multiplied by its coefficient when the accumulator
 * is drained, so no operand is rounded a second time.  Wider bf16 layers: the per-token scale is
 * applied to the narrower operand (rounded to nearest even in bf16) in one pass before a plain
 * GEMM, or, for layers with few rows, to the rows as they land in shared memory.
 *
 *   coeffs  dev, float32 [B]
 *   dW      dev, float32 [d_out, d_in] row-major (the layout of `grad_out.T @ act_in`)
 *   beta    0 (overwrite) or 1 (accumulate into the existing gradient)
 * Other arguments as for isopo_layer_gram; seq_offsets_host must hold the same offsets.
 */
ISOPO_API isopo_status isopo_weight_grad(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in, int d_out,
                               const float* coeffs, const int64_t* seq_offsets_host, int B, isopo_path path,
                               float* dW, float beta, void* ws, size_t ws_bytes, int32_t* info, void* cuda_stream);

/*
 * isopo_sampled_coefficients: the non-interacting update as Algorithm 1 prints it, with the Fisher
 * norm of every sequence gradient estimated from sampled token positions (Sec. 2.2, "Estimating the
 * Fisher metric" and "Efficient implementation") instead of from K.
 *
 * With a0 = X[sample_rows], g0 = dY[sample_rows] (Algorithm 1's `overlap_samples`; the caller draws
 * them, e.g. the first n of a random permutation of the T token rows):
 *     F_i^2 = sum_j (g0_j . G_i a0_j)^2 / sum_j (||g0_j|| ||a0_j||)^2        (Eq. one over Eq. two)
 *     coeffs[i] = A_i / sqrt(F_i^2 + lambda)                                  (`rescaling`)
 * G_i is never formed: g0_j . G_i a0_j = sum_{t in i} (g0_j . dY_t)(a0_j . x_t), so tiles of
 * a0 X^T and g0 dY^T are formed in tensor memory, multiplied elementwise and summed per sequence,
 * at about n_samples (d_in + d_out) / (d_in d_out) of the cost of the weight-gradient GEMM.
 * Follow it with isopo_weight_grad(..., ISOPO_PATH_GRAM, ...) for dW = sum_i coeffs[i] G_i; a
 * workspace of isopo_sampled_workspace_bytes() bytes serves that call too.
 *
 *   sample_rows_host  host, int64 [n_samples], each in [0, T); read before the call returns
 *   n_samples         1 .. ISOPO_MAX_SAMPLES
 *   A                 dev, float32 [B]
 *   lambda            absolute regulariser, >= 0
 *   coeffs            dev, float32 [B], overwritten
 *   F2                dev, float32 [B] or NULL: the estimates F_i^2 themselves
 *   ws, ws_bytes      dev workspace of isopo_sampled_workspace_bytes(...) bytes, 1024-byte aligned
 * Other arguments and conventions as for isopo_layer_gram.
 */
#define ISOPO_MAX_SAMPLES 4096
#define ISOPO_MAX_BATCH 32
ISOPO_API size_t isopo_sampled_workspace_bytes(isopo_dtype dtype, int64_t T, int d_in, int d_out, int B, int n_samples);
ISOPO_API isopo_status isopo_sampled_coefficients(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in,
                                                  int d_out, const int64_t* seq_offsets_host, int B,
                                                  const int64_t* sample_rows_host, int n_samples, const float* A,
                                                  float lambda, float* coeffs, float* F2, void* ws, size_t ws_bytes,
                                                  int32_t* info, void* cuda_stream);

/*
 * isopo_layer_gram_static: isopo_layer_gram on the GRAM route without a caller workspace and
 * without any allocation (the paper has no counterpart; this exists for the way the library gets
 * embedded).
 *
 * Who needs it: callers that may not allocate device memory where the layer hook runs - a hook
 * inside a framework whose caching allocator owns the device and rejects raw cudaMalloc, code that
 * runs while that allocator is locked, or an embedder that gave the whole device to another pool.
 * The scratch the route needs (device copy of the offsets, token -> sequence map, float64
 * accumulators of the float32 route) lives in a fixed array inside the library's device image:
 * about 0.8 MB that every GPU which loads the library keeps reserved until the process exits.
 *
 * Limits: T <= ISOPO_STATIC_MAX_TOKENS and B <= ISOPO_STATIC_MAX_SEQS; larger problems return
 * ISOPO_ERR_UNSUPPORTED (isopo_last_cuda_error() then says why) and must use isopo_layer_gram.
 * The call makes no cudaMalloc / cudaFree and calls no allocating routine; event timing
 * (isopo_profile_enable) is suspended for its duration.
 *
 * The first call on each device looks up the array's device address (one cudaGetSymbolAddress with
 * that device current); make that first call outside any stream capture.  All calls on a device
 * share the one array: calls whose kernels could overlap on the GPU (different streams, no
 * ordering between them) race on it and must be serialised by the caller.  On the host the call is
 * not thread-safe against any other call of the library either (it pauses the process-wide event
 * timing for its duration and fills the address cache unlocked).  The array keeps what
 * the previous call left; every part that is read is rewritten or cleared first.
 *
 * Arguments and the result are those of isopo_layer_gram with path = ISOPO_PATH_GRAM; K agrees
 * with it up to the order of the float atomic additions.
 */
#define ISOPO_STATIC_MAX_TOKENS 65536
#define ISOPO_STATIC_MAX_SEQS 256
ISOPO_API isopo_status isopo_layer_gram_static(const void* X, const void* dY, isopo_dtype dtype, int64_t T, int d_in,
                                               int d_out, const int64_t* seq_offsets_host, int B, float* K,
                                               int32_t* info, void* cuda_stream);

/*
 * Deterministic mode (the paper has no counterpart; a diagnostic that tells a race from rounding).
 * Normally K of the bf16 MATERIALISE route is summed over the CTAs with float atomics, so two runs
 * differ in the last bits.  With the mode on, every CTA stores its partial K in the workspace and a
 * second kernel adds the partials in a fixed order: K, the coefficients and dW of that route are
 * then bit-identical from run to run.  The switch is process-wide and changes
 * isopo_workspace_bytes(..., MATERIALISE) (160 * B * B * 4 more bytes for bf16): set it before
 * sizing workspaces.  The GRAM route and the GEMM-route weight gradient keep their float atomics.
 *
 * isopo_debug_build() is 1 when the library was compiled with -DISOPO_DEBUG (libisopo_debug.so): every
 * data-dependent index of the kernels is then range-checked before use, a violation skips the access
 * and sets *info = ISOPO_INFO_BOUNDS | kernel id.
 */
/*
 * Store format of the bf16 MATERIALISE route (the paper has no counterpart: an 8-bit storage of G for the K
 * pass).  ISOPO_STORE_BF16 (default): every G_i is kept as bf16.  ISOPO_STORE_E4M3_SPLIT: every element is kept as
 * two e4m3 bytes, hi = round(s_i g) and lo = round(16 (s_i g - hi)), in two planes (the same 2 bytes per element; s_i
 * a power of two per sequence, estimated from a sample of the sequence's token rows).  The K pass then reads only the
 * hi plane - half the bytes, kind::f8f6f4 tensor-core instructions, about 0.6 x the time - and takes the diagonal of K
 * from float32 sums of squares that the gradient GEMM forms from its accumulators (more exact than the bf16
 * store's); the weight gradient reads both planes (8 significant bits, as bf16).  What it costs: the off-diagonal
 * entries of K carry rounding noise of about 0.05 / sqrt(d_in d_out) of sqrt(K_ii K_jj), thirty times that of the
 * bf16 store, which the interacting solve amplifies by cond(K + lambda I): meant for layers of a million weights and
 * more and well-conditioned K; elements beyond 448 / s_i are clamped and reported (*info = ISOPO_INFO_SATURATED |
 * kernel id: inputs with outlier channels hundreds of times the typical size need the bf16 store).  Process-wide; set it before isopo_layer_gram and
 * leave it unchanged until the layer's isopo_weight_grad (the workspace tag records the format, a mismatch is
 * reported as ISOPO_INFO_STALE_WORKSPACE).  Layers that take the 1-CTA gradient kernel (an odd number, below 7, of
 * 128-row tiles), ISOPO_F32 and deterministic mode keep the bf16 / float32 store.
 */
typedef enum { ISOPO_STORE_BF16 = 0, ISOPO_STORE_E4M3_SPLIT = 1 } isopo_store_format;
ISOPO_API isopo_status isopo_set_store_format(isopo_store_format format);
ISOPO_API isopo_store_format isopo_get_store_format(void);

ISOPO_API void isopo_set_deterministic(int on);
ISOPO_API int isopo_get_deterministic(void);
ISOPO_API int isopo_debug_build(void);

/*
 * isopo_selftest_bounded_wait (the paper has no counterpart): runs the library's bounded mbarrier wait
 * on a barrier that nothing ever arrives on, in a kernel that owns no TMA copy and no tensor memory,
 * so that the give-up path of the tensor-core kernels can be exercised without hanging or faulting
 * anything.  After synchronising the stream: *info == (ISOPO_INFO_TIMEOUT | kernel id of
 * "k_wait_probe"), *roles_at_teardown == 3 (the role that timed out, the role that saw its abort
 * flag, and the role without waits all reached the common teardown), and the context is as usable as
 * before.
 *
 *   limit_clocks       1 .. 2^28 SM clock ticks the first role waits before it gives up (1e5 = ~50 us)
 *   info               dev int32, zeroed by the caller
 *   roles_at_teardown  dev int32, overwritten
 */
ISOPO_API isopo_status isopo_selftest_bounded_wait(int64_t limit_clocks, int32_t* info, int32_t* roles_at_teardown,
                                                   void* cuda_stream);

/*
 * Measurement hooks (the paper has no counterpart).  While enabled, every kernel the library
 * launches is bracketed by CUDA events on its stream.  isopo_profile_collect synchronises those
 * events, adds the elapsed milliseconds and launch counts per kernel into the caller's arrays
 * (host, ISOPO_NUM_KERNELS entries each, overwritten) and forgets them.  Launch counts are kept
 * even while event timing is disabled.  Not thread-safe; meant for benchmarks.
 */
#define ISOPO_NUM_KERNELS 17
ISOPO_API void isopo_profile_enable(int on);
ISOPO_API isopo_status isopo_profile_collect(double* ms_by_kernel, int64_t* launches_by_kernel);
ISOPO_API const char* isopo_kernel_name(int kernel_id);

#ifdef __cplusplus
}
#endif
#endif /* ISOPO_H_ */
