/*
 * pkv.h — C ABI of the PatchKV patch-construction library (libpkv.so, CUDA, sm_100a).
 *
 * What the library computes (per transformer block; paper Sec. 2.2-2.3, Algorithm 1):
 * reference tokens are run through the block twice, once attending to the full KV cache
 * (teacher) and once to a compressed cache (student); the target t = W(h-h') + (z-z')
 * (Eq. 5) and the student's MLP features h' give the sufficient statistics
 * S_H = H'^T H', S_T = T^T H' (Eq. 9); the patch of the MLP down projection is
 * dW = S_T (S_H + lambda I)^{-1} (Eq. 8) with lambda = lambda0 ||S_H||_F^2 / tr(S_H)
 * (Eq. 7); the patch is merged as W <- W + dW (Algorithm 1, Merge).
 *
 * Conventions
 *   - "device" pointers are CUDA device memory owned by the caller (any allocator); the
 *     library never frees or keeps them after the call returns.  "host" pointers are plain
 *     host memory.  Inputs are read-only.  Outputs must not alias inputs.
 *   - All matrices are dense row-major.  Weight matrices are [out][in] (the paper writes the
 *     down projection as W in R^{d x d_ff}); the patch dW has the layout of W, [d][F].
 *   - Weights and caches have the element type pkv_dims.dtype (bf16 or fp32).  Residual-stream
 *     states (xF, xC, next states) and dW are always fp32.
 *   - Every function returns PKV_OK (0) or a negative pkv_error; nothing throws, aborts or
 *     traps on the device.  After an error the contents of the outputs are unspecified.
 *   - Work is ordered after whatever is already queued on the CUDA stream given at pkv_create and is
 *     complete when a call returns: pkv_build_patch and the other building calls end with one stream
 *     synchronisation to read the device status word, so the return code is truthful.  Inside a call
 *     the tensor-core engine also uses streams of its own (the teacher half of a block, the targets and
 *     S_T run beside the ridge solve; the solve itself spans four streams), all forked from and joined
 *     back into the context's stream before the call returns; none of this may be issued while the
 *     caller's stream is being captured.
 *   - A context is not thread-safe; use one per host thread / stream.
 */
#ifndef PKV_H_
#define PKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum pkv_error {
    PKV_OK = 0,
    PKV_ERR_INVALID_ARG = -1,  /* null/misaligned pointer, lambda <= 0 or non-finite, N = 0, bad chunk offsets */
    PKV_ERR_UNSUPPORTED = -2,  /* hd not in {64,128}, Hq % Hkv != 0, F > 32768, sizes the kernels do not cover */
    PKV_ERR_BAD_INDEX = -3,    /* kept-index set not strictly ascending within [0, L); first offender in stats */
    PKV_ERR_NOT_PD = -4,       /* Cholesky pivot <= 0 or non-finite; column in stats.err_info */
    PKV_ERR_DEGENERATE = -5,   /* tr(S_H) = 0 under the adaptive ridge scale (Eq. 7) */
    PKV_ERR_NONFINITE = -6,    /* NaN/Inf met in the statistics, or a cached key outside fp16's range (hd = 128) */
    PKV_ERR_TIMEOUT = -7,      /* a bounded device-side wait (TMA / tensor-core pipeline) expired */
    PKV_ERR_CUDA = -8,         /* a CUDA runtime call failed; see pkv_last_cuda_error */
    PKV_ERR_NOMEM = -9         /* workspace allocation failed or caller-provided workspace too small */
} pkv_error;

enum { PKV_BF16 = 0, PKV_FP32 = 1 };

/* How the ridge coefficient handed to pkv_build_patch is read. */
enum {
    PKV_LAMBDA_PAPER = 0,      /* lambda = lambda0 * ||S_H||_F^2 / tr(S_H)   (Eq. 7; default) */
    PKV_LAMBDA_ABSOLUTE = 1,   /* lambda = lambda0                            (Eq. 6 as written) */
    PKV_LAMBDA_TRACE_MEAN = 2  /* lambda = lambda0 * tr(S_H) / F              (ridge-scale ablation) */
};

/* Which linear system the ridge patch is solved through.  Both give the same dW (Woodbury identity):
 *   primal: dW = S_T (S_H + lambda I)^{-1}, an F x F system on the sufficient statistics (Eq. 8-9);
 *   dual:   dW = T^T (H' H'^T + lambda I)^{-1} H', an N x N system on the reference tokens of the call.
 * The dual is cheaper when N < F but needs all reference tokens in one call (no running sums). */
enum {
    PKV_SOLVER_PRIMAL = 0,     /* default: the paper's form */
    PKV_SOLVER_DUAL = 1        /* tensor-core engine only, requires N <= F */
};

enum {
    PKV_ENGINE_AUTO = 0,       /* tcgen05/TMA tensor-core kernels for bf16, SIMT fp32 kernels for fp32 */
    PKV_ENGINE_SIMT = 1        /* force the SIMT fp32 kernels (on-device cross-check of the tensor path) */
};

/* Geometry of one block and the capacity the context is sized for. */
typedef struct pkv_dims {
    int32_t d;            /* hidden size */
    int32_t Hq, Hkv, hd;  /* query heads, key/value heads (Hq % Hkv == 0), head dim (64 or 128) */
    int32_t F;            /* MLP intermediate width (<= 32768; the models the paper names have 14336 and 18944) */
    int32_t L;            /* rows of the full cache per KV head */
    int32_t N_max;        /* most reference tokens one call may bring */
    int32_t b_max;        /* most kept rows per KV head in a compressed cache */
    int32_t dtype;        /* PKV_BF16 | PKV_FP32: element type of weights and caches */
    float rope_theta;     /* rotary base; 0 disables the rotation */
    float eps;            /* RMSNorm epsilon */
} pkv_dims;

typedef struct pkv_opts {
    int32_t engine;          /* PKV_ENGINE_* */
    int32_t kv_split;        /* cache rows per attention split; 0 = choose from L and the SM count */
    void* workspace;         /* optional caller-provided device workspace (256-byte aligned) ... */
    size_t workspace_bytes;  /* ... of at least pkv_workspace_bytes(); NULL/0: the context allocates */
    int32_t solver;          /* PKV_SOLVER_* (used by pkv_build_patch / pkv_build_stack) */
    int32_t reserve_sms;     /* pkv_build_stack: SMs the teacher stream leaves free for the student stream and
                                the ridge solve; 0 = default (12), negative = none (teacher on every SM) */
} pkv_opts;

/* Block weights, all device, element type dims.dtype except the fp32 norm gains.
 * Layout [out][in]: Wq[Hq*hd][d] Wk[Hkv*hd][d] Wv[Hkv*hd][d] Wo[d][Hq*hd]
 *                   Wgate[F][d] Wup[F][d] Wdown[d][F].  Pointers 16-byte aligned. */
typedef struct pkv_block_weights {
    const float* g_attn;  /* [d] */
    const void* Wq;
    const void* Wk;
    const void* Wv;
    const void* Wo;
    const float* g_mlp;   /* [d] */
    const void* Wgate;
    const void* Wup;
    const void* Wdown;    /* the matrix the patch is built for (unpatched base weights) */
} pkv_block_weights;

/* Full cache of the block: K, V [Hkv][L][hd], device, keys already rotated. */
typedef struct pkv_kv {
    const void* K;
    const void* V;
} pkv_kv;

/* Compressed cache, one of three forms (Sec. 2.1: eviction or approximation compressors; appendix: quantised caches).
 *  (a) kept-index set:  idx != NULL.  Head h keeps rows idx[head_off[h] .. head_off[h+1])
 *      of the full cache, strictly ascending, each in [0, L).  Heads may keep different counts.
 *  (b) explicit cache:  idx == NULL, qbits == 0, Kc/Vc != NULL, packed [head_off[Hkv]][hd] (element type
 *      dims.dtype) with head h's rows at head_off[h]...; optional per-key logit bias (fp32, same packing) or NULL.
 *  (c) quantised explicit cache:  idx == NULL, qbits = 8 or 4.  Kc/Vc hold integer codes, same row packing:
 *      qbits 8: int8 [rows][hd]; qbits 4: bytes [rows][hd/2], element 2j in the low nibble of byte j, element
 *      2j+1 in the high nibble, 4-bit two's complement.  k_scale/v_scale: fp32 [rows][hd/qgroup], one scale per
 *      qgroup consecutive elements of a row (qgroup a multiple of 8 that divides hd).  An element decodes to
 *      scale * code computed in fp32 and rounded to dims.dtype; the student attends to the decoded cache, which
 *      the library materialises in its workspace during the index/compaction stage.  bias as in (b).
 * head_off is a HOST array of Hkv+1 ints starting at 0; idx/Kc/Vc/bias/scales are device. */
typedef struct pkv_kv_compressed {
    const int32_t* head_off;
    const int32_t* idx;
    const void* Kc;
    const void* Vc;
    const float* bias;
    const float* k_scale;    /* form (c) only */
    const float* v_scale;
    int32_t qbits;           /* 0 (forms a, b), 8 or 4 */
    int32_t qgroup;
} pkv_kv_compressed;

/* Reference tokens entering the block (Algorithm 1: states x^F, x^C of every chunk).
 * xF, xC: device fp32 [N][d] (may alias each other at the first block).  chunk_off: HOST
 * array of n_chunks+1 strictly increasing offsets, chunk_off[0]=0, chunk_off[n_chunks]=N.
 * A token attends to the whole cache and causally inside its own chunk; token i of a chunk
 * starting at s has position pos0 + (i - s) in both streams. */
typedef struct pkv_ref {
    const float* xF;
    const float* xC;
    int32_t N;
    int32_t n_chunks;
    const int32_t* chunk_off;
    int32_t pos0;
} pkv_ref;

/* Optional outputs: states entering the next block, device fp32 [N][d].
 * xF_next = z + W h (teacher, never patched); xC_next = z' + (W + dW) h' (patched student). */
typedef struct pkv_ref_next {
    float* xF_next;
    float* xC_next;
} pkv_ref_next;

/* Scalars of one build (host). */
typedef struct pkv_stats {
    double lambda_eff;   /* ridge coefficient actually added to the diagonal */
    double trace;        /* tr(S_H) */
    double fro2;         /* ||S_H||_F^2 */
    double target_fro2;  /* ||T||_F^2 */
    double resid_fro2;   /* ||T - H' dW^T||_F^2 (only when next states were requested) */
    double dW_fro2;      /* ||dW||_F^2 */
    double min_pivot;    /* smallest Cholesky pivot (squared diagonal of the factor) */
    int32_t err_info[2]; /* BAD_INDEX: (head, position); NOT_PD: (column, 0); TIMEOUT: (site, 0) */
    float stage_ms[12];  /* per-stage device time when timing is enabled with pkv_set_timing */
    /* Conditioning of the ridge matrix G = S_H + lambda I (ridge-scale ablation: a small coefficient makes the solve
     * ill conditioned).  lambda_max(G) lies between the weighted eigenvalue mean ||S_H||_F^2 / tr(S_H) + lambda and
     * ||S_H||_F + lambda; lambda_min(G) between lambda and the smallest pivot.  Hence
     *   cond_lower_bound = (fro2 / trace + lambda_eff) / min_pivot  <=  cond(G)  <=
     *   cond_upper_bound = (sqrt(fro2) + lambda_eff) / lambda_eff.
     * cond_warning = 1 when the lower bound exceeds 1e4: the fp32-equivalent factorisation (relative rounding
     * 2^-24, amplified by cond(G)) may then miss the 5e-3 tolerance the build is checked to; the patch is still
     * returned.  All three are 0 when the solve did not run. */
    double cond_lower_bound;
    double cond_upper_bound;
    int32_t cond_warning;
    int32_t reserved;
} pkv_stats;

typedef struct pkv_ctx pkv_ctx;

/* Device bytes a context of these dims needs (Algorithm 1 keeps only one chunk's activations
 * and the running statistics; here: one call's activations, S_H, S_T, the factor). */
size_t pkv_workspace_bytes(const pkv_dims* dims, const pkv_opts* opts);

/* Create a context on the current device.  cuda_stream is a cudaStream_t (NULL = default). */
int pkv_create(pkv_ctx** out, const pkv_dims* dims, const pkv_opts* opts, void* cuda_stream);
void pkv_destroy(pkv_ctx* ctx);

/* One block of Algorithm 1 (Eq. 4-9): teacher forward with `full`, student forward with `cb`,
 * targets, statistics, ridge solve.  dW: device fp32 [d][F] out.  next, stats: optional (NULL). */
int pkv_build_patch(pkv_ctx* ctx, const pkv_block_weights* w, const pkv_kv* full,
                    const pkv_kv_compressed* cb, const pkv_ref* ref, float lambda, int lambda_mode,
                    float* dW, const pkv_ref_next* next, pkv_stats* stats);

/* Streamed reference sets (Sec. 2.3, chunked query encoding; Eq. 9).  The reference set of a context may be far
 * larger than one call's N_max: it is fed in parts, each a whole number of chunks, and only the running sums
 * S_H, S_T stay in the context between the calls, so that the workspace does not grow with the reference set.
 *   pkv_stream_begin     clears the sums and fixes the ridge coefficient and its reading;
 *   pkv_stream_add       teacher and student forward of ref->N <= N_max tokens (same arguments as
 *                        pkv_build_patch), targets, S_H += H'^T H', S_T += T^T H'; xF_next (optional, device fp32
 *                        [N][d]) receives the teacher's states of these tokens entering the next block;
 *   pkv_stream_finish    lambda from the sums (Eq. 7), dW = S_T (S_H + lambda I)^{-1} (Eq. 8); stats->target_fro2 is
 *                        the sum over the parts, resid_fro2 is not available;
 *   pkv_stream_propagate Algorithm 1's student propagation for one part: the student block re-run with the
 *                        patched W + dW against the compressed cache, xC_next = z' + (W + dW) h' (device fp32 [N][d];
 *                        tensor-core engine only).
 * Any number of parts gives the statistics of one call on all tokens up to rounding order (chunks are independent).
 * A failed pkv_stream_add closes the stream (begin again).  Not available with PKV_SOLVER_DUAL. */
int pkv_stream_begin(pkv_ctx* ctx, float lambda, int lambda_mode);
int pkv_stream_add(pkv_ctx* ctx, const pkv_block_weights* w, const pkv_kv* full, const pkv_kv_compressed* cb,
                   const pkv_ref* ref, float* xF_next);
int pkv_stream_finish(pkv_ctx* ctx, float* dW, pkv_stats* stats);
int pkv_stream_propagate(pkv_ctx* ctx, const pkv_block_weights* w, const pkv_kv* full, const pkv_kv_compressed* cb,
                         const pkv_ref* ref, const float* dW, float* xC_next);

/* Algorithm 1, Merge: W[i] <- W[i] + dW[i] for the d*F entries, the sum taken in fp32 and
 * rounded once to W's type (w_dtype = PKV_BF16 | PKV_FP32).  Asynchronous on cuda_stream. */
int pkv_merge(void* W, int w_dtype, const float* dW, int64_t count, void* cuda_stream);

/* Algorithm 1, outer loop: blocks first_layer..n_layers-1 in sequence, each solved with the
 * blocks below it already patched in the student (greedy construction, Sec. 2.2).  Arrays are
 * HOST arrays of n_layers entries.  x0F/x0C enter block first_layer; states are carried in
 * fp32 inside the context.  dW[l]: device fp32 [d][F].  stats: NULL or n_layers entries.
 * final: optional states leaving the last block.
 * Scheduling: the teacher of Algorithm 1 never sees a patch, so with the tensor-core engine, two or
 * more blocks, at most 128 layers and stage timing off, the teacher half of up to two later blocks
 * runs on a second stream owned by the context, beside the student half and the solve of the
 * current block; results are the same as block-by-block calls up to rounding order.  That stream is
 * confined to all SMs but a small reserve (pkv_opts.reserve_sms) so that its long-running attention
 * CTAs never starve the student's kernels and the solve.  That stream is
 * ordered after the work already queued on the context's stream and is drained before the call
 * returns; the call returns after one synchronisation.  In this mode stage_ms stays zero.  With
 * stage timing on, with the SIMT engine or for a single block the blocks run strictly in sequence.
 * Errors: the status of the first failing block is returned; stats[l].err_info locates it. */
int pkv_build_stack(pkv_ctx* ctx, int n_layers, int first_layer, const pkv_block_weights* w,
                    const pkv_kv* full, const pkv_kv_compressed* cb, const pkv_ref* ref0,
                    float lambda, int lambda_mode, float* const* dW, const pkv_ref_next* final,
                    pkv_stats* stats);

/* Algorithm 1 for several ridge coefficients on the same context and reference set (the ridge-scale ablation
 * sweeps lambda0).  The teacher stream of Algorithm 1 sees neither a patch nor lambda, so it is run once: its
 * per-block outputs (attention output, residual term, MLP features, next state: N (Hq hd + 2 d + F) floats per
 * block) are kept in `teacher_cache`, a caller-owned device buffer of at least pkv_teacher_cache_bytes(), and the
 * student half, the statistics and the solve of every block are then run once per coefficient.
 * dW: HOST array of n_lambda * n_layers device pointers, entry [j * n_layers + l] = patch of block l for
 * lambdas[j]; stats: NULL or n_lambda * n_layers entries in the same order.  Both streams start from ref0->xF
 * / ref0->xC.  Tensor-core engine only.  Errors as pkv_build_stack; PKV_ERR_NOMEM if the cache is too small. */
size_t pkv_teacher_cache_bytes(const pkv_dims* dims, int n_layers, int N);
int pkv_build_stack_sweep(pkv_ctx* ctx, int n_layers, const pkv_block_weights* w, const pkv_kv* full,
                          const pkv_kv_compressed* cb, const pkv_ref* ref0, int n_lambda, const float* lambdas,
                          int lambda_mode, float* const* dW, void* teacher_cache, size_t cache_bytes,
                          pkv_stats* stats);

/* ---- single stages, exported for unit parity tests and per-kernel measurement ---- */

/* Index check + compaction of a kept-index set (bit-exact): Kc[i] = K[h][idx[i]], same for V.
 * Kc, Vc: device [head_off[Hkv]][hd] out.  Returns PKV_ERR_BAD_INDEX without touching memory
 * outside the arrays when the set is invalid; bad_head/bad_pos (host, optional) get the first
 * offender. */
int pkv_gather_kept(pkv_ctx* ctx, const pkv_kv* full, const int32_t* head_off_host,
                    const int32_t* idx, void* Kc, void* Vc, int32_t* bad_head, int32_t* bad_pos);

/* Decode of a quantised compact cache alone (form (c) of pkv_kv_compressed; bit-exact unit check of the student's
 * load path): Kc, Vc device [head_off[Hkv]][hd] of dims.dtype out. */
int pkv_dequant_cache(pkv_ctx* ctx, const pkv_kv_compressed* cb, void* Kc, void* Vc);

/* Dual-cache attention alone (Sec. 2.2, teacher and student forward passes over the reference
 * tokens).  q: device fp32 [2][N][Hq*hd] rotated queries of the teacher (0) and student (1)
 * stream; k_new, v_new: device fp32 [2][N][Hkv*hd] the reference tokens' own keys/values (all 16-byte aligned).
 * Outputs device fp32 [N][Hq*hd], 16-byte aligned: aF, aC and dA = aF - aC (formed before any rounding). */
int pkv_attention(pkv_ctx* ctx, const float* q, const float* k_new, const float* v_new,
                  const pkv_kv* full, const pkv_kv_compressed* cb, int32_t N, int32_t n_chunks,
                  const int32_t* chunk_off, float* aF, float* aC, float* dA);

/* Sufficient statistics alone (Eq. 9): S_H (+)= X^T X, S_T (+)= R^T X for X [n][F], R [n][d]
 * device fp32; S_H [F][F], S_T [d][F] device fp32; accumulate != 0 adds to the running sums. */
int pkv_gram(pkv_ctx* ctx, const float* X, const float* R, int32_t n, float* S_H, float* S_T,
             int accumulate);

/* The statistics of pkv_gram for callers that cannot allocate device memory (no counterpart in the
 * paper: an addition of this library).  Hosts that own all device memory through their own pool, or
 * that sit in a latency-critical loop where cudaMalloc (a device-wide synchronisation) is not
 * acceptable, cannot create a pkv_ctx, because a context allocates its workspace.  This call needs no
 * context: the scratch its kernels use (bf16 operand copies, the status word) lives in a fixed device
 * array inside the library image, about 4.2 MB, which every GPU that loads the library holds until
 * the process exits.  It calls no cudaMalloc/cudaFree and no allocating library routine.
 *   X [n][F], R [n][d], S_H [F][F], S_T [d][F]: device fp32, 16-byte aligned; meaning as in pkv_gram.
 *   Limits: n <= PKV_NOALLOC_MAX_N, F <= PKV_NOALLOC_MAX_F, d <= PKV_NOALLOC_MAX_D, F % 8 == d % 8 == 0;
 *   anything larger returns PKV_ERR_UNSUPPORTED (as does a device without tcgen05 tensor cores).
 *   The first call on a device resolves the array's address and sets kernel attributes: make that
 *   call before any stream capture begins.  All calls share the one array, which keeps the previous
 *   call's contents (the call clears what must start at zero): calls whose kernels may overlap on the
 *   GPU, e.g. from two streams or two host threads, race and must be serialised by the caller.
 *   The call ends with one synchronisation of cuda_stream to read its status word. */
#define PKV_NOALLOC_MAX_N 512
#define PKV_NOALLOC_MAX_F 1024
#define PKV_NOALLOC_MAX_D 1024
int pkv_gram_noalloc(const float* X, const float* R, int32_t n, int32_t F, int32_t d, float* S_H, float* S_T,
                     int accumulate, void* cuda_stream);

/* Rank-r patch (appendix, low-rank weight patches): with M = dW S_H dW^T (d x d) and U_r its r leading
 * eigenvectors, the patch is stored as U_r [d][r] and B_r = U_r^T dW [r][F] ((d + F) r numbers), dW_r = U_r B_r.
 * dW [d][F] and S_H [F][F] (full symmetric matrix): device fp32, read only.  U, Br: device fp32 out; dW_r: optional
 * device fp32 [d][F] out (the expanded rank-r patch) or NULL; ritz_values: optional device fp32 [r + 8] out, the
 * leading approximate eigenvalues of M in descending order (the gap after the r-th says how well U_r is determined;
 * eigenvector signs are arbitrary).  M is formed on the tensor cores (fp32-equivalent products), the eigenvectors by
 * `iterations` sweeps (0 = 24) of subspace iteration with Rayleigh-Ritz on r + 8 vectors in fp64.  scratch: caller-
 * owned device memory of pkv_low_rank_scratch_bytes().  Tensor-core engine; r <= 40 and r + 8 <= d.  Synchronises. */
size_t pkv_low_rank_scratch_bytes(const pkv_dims* dims, int r);
int pkv_low_rank(pkv_ctx* ctx, const float* dW, const float* S_H, int32_t r, int32_t iterations, void* scratch,
                 size_t scratch_bytes, float* U, float* Br, float* dW_r, float* ritz_values);

/* Ridge solve alone (Eq. 7-8): dW = S_T (S_H + lambda I)^{-1}.  S_H, S_T are read, not
 * modified. */
int pkv_ridge_solve(pkv_ctx* ctx, const float* S_H, const float* S_T, float lambda, int lambda_mode,
                    float* dW, pkv_stats* stats);

/* Ridge solve with iterative refinement (Eq. 6 read with lambda as written, and the small coefficients of the
 * ridge-scale ablation: S_H + lambda I is then ill conditioned, and the rounding of the factorisation and of the
 * explicit inverse factor reaches dW amplified by its condition number).  After the solve of pkv_ridge_solve,
 * `steps` times: R = S_T - dW (S_H + lambda I) as an fp32-equivalent product against the caller's S_H, then
 * dW += R (S_H + lambda I)^{-1} through the factor already computed.  Each step costs one d x F x F product in six
 * passes and the two triangular products of Eq. 8 again; what it cannot remove is the rounding of the fp32 residual
 * itself (about 2^-24 cond(G)), so one step is normally all that helps.  steps = 0 is pkv_ridge_solve; at most 8.
 * S_H must be the full symmetric matrix.  stats->resid_fro2 = ||S_T - dW (S_H + lambda I)||_F^2 of the iterate
 * BEFORE the last correction (0 for steps = 0); dW_fro2 is the final iterate's.  Tensor-core engine only
 * (PKV_ERR_UNSUPPORTED otherwise); pointers 16-byte aligned. */
int pkv_ridge_solve_refined(pkv_ctx* ctx, const float* S_H, const float* S_T, float lambda, int lambda_mode,
                            int32_t steps, float* dW, pkv_stats* stats);

/* The same refinement after every ridge solve the context runs from now on (pkv_build_patch, pkv_build_stack and
 * its sweep, pkv_stream_finish, pkv_ridge_solve): steps = 0 (default) switches it off.  A build keeps a full
 * symmetric copy of S_H beside the matrix it factors in place; the student's next state is formed with the
 * refined patch.  Tensor-core engine with the primal solver only (PKV_ERR_UNSUPPORTED otherwise). */
int pkv_set_refinement(pkv_ctx* ctx, int steps);

/* The product the ridge solve is built from (Eq. 8 needs fp32 accuracy; the tensor cores take bf16): C [M][N]
 * (+)= alpha * A B^T with A [M][K], B [N][K], C device fp32 row-major, 16-byte aligned.  Each operand is split
 * into bf16 parts (hi, mid, lo) and multiplied in `passes` passes accumulating in fp32: 6 = fp32-equivalent
 * (triples), 3 = pairs (about 16 mantissa bits).  accumulate != 0 adds to C.  accumulators = 1, 2 or 4 tensor-
 * memory accumulators per tile: the tensor core truncates when it adds to an accumulator, so the large hi x hi
 * pass is kept apart from the cross terms (2) and split in three (4), the parts being added with round to
 * nearest; the solve uses 4 in its factorisation.  Exported for unit parity tests; tensor-core engine only;
 * M*K and N*K (K rounded up to 8) must not exceed d*F of the context. */
int pkv_fp32_product(pkv_ctx* ctx, const float* A, const float* B, int32_t M, int32_t N, int32_t K, float alpha,
                     float* C, int accumulate, int passes, int accumulators);

/* Failure-detection self-test: launches one CTA whose pipeline wait is on a barrier that nothing ever
 * completes, with a short limit (about a millisecond).  The wait must give up, raise the device status
 * word and let the CTA exit; the call then returns PKV_ERR_TIMEOUT (err site in *site if not NULL) and
 * the context stays usable.  Nothing faults, traps or spins without a limit. */
int pkv_selftest_bounded_wait(pkv_ctx* ctx, int32_t* site);

/* Per-stage CUDA-event timing into pkv_stats.stage_ms.  0: off.  1: every stage; a block then runs teacher and student
 * stacked on one stream and a stack block by block, so that every stage has an interval of its own.  2: only the ridge
 * solve's interval (stage_ms[7]) on the caller's stream, without changing the schedule. */
int pkv_set_timing(pkv_ctx* ctx, int on);

/* pkv_build_stack scheduling: 0 = default (teacher run ahead where it applies), 1 = strictly block by block on
 * the context's stream (what stage timing also forces); for measuring one against the other. */
int pkv_set_stack_schedule(pkv_ctx* ctx, int schedule);

/* Measures the device's fp32 fused-multiply-add rate (TFLOP/s, two flops per FMA) with a register-resident FMA
 * kernel timed by CUDA events on the context's stream: the denominator for the ridge solve's roofline, which
 * stands for fp32 arithmetic.  Uses the context's workspace as scratch; synchronises the stream. */
int pkv_measure_fma_peak(pkv_ctx* ctx, double* tflops);

/* Number of kernels the context launched since creation (for launch accounting). */
int64_t pkv_launch_count(const pkv_ctx* ctx);

/* SMs the teacher stream of pkv_build_stack may occupy: the device's SM count minus the reserve when the
 * driver granted the partition, the full count otherwise. */
int pkv_teacher_sm_count(const pkv_ctx* ctx);

const char* pkv_strerror(int code);
const char* pkv_last_cuda_error(const pkv_ctx* ctx);
const char* pkv_stage_name(int stage);

#ifdef __cplusplus
}
#endif
#endif /* PKV_H_ */
