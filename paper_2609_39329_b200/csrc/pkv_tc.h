// Tensor-core engine (tcgen05 + TMEM + TMA, sm_100a): interface used by pkv_api.cu.
#pragma once

#include <cuda.h>

#include "pkv_internal.h"

namespace pkv {

constexpr int kGemmMaxPass = 6;

// A bf16 matrix as the TMA engine sees it (whole allocation: rows x cols, row stride ld).
struct TcMat {
    const __nv_bfloat16* p;
    long long ld, rows, cols;
};

// C = alpha * sum_p A_p B_p^T (+ addend) (+ C): bf16 operands, fp32 accumulate.  Operand tiles are
// addressed by (row0, col0) offsets into whole matrices, with per-batch increments (blockIdx.z);
// rows/columns past a matrix edge read as zero.  Results go to fp32 C and/or to up to three bf16
// arrays holding successive roundings of the value (hi, mid, lo).
struct TcGemm {
    TcMat A[kGemmMaxPass], B[kGemmMaxPass];
    int npass;
    // Grouped B: the product's columns are the concatenation of ngrp (2 or 3) matrices Bgrp[k] [grp_n[k]][K]
    // (separately stored weights applied to the same activations: Wq | Wk | Wv, Wgate | Wup), every pass taking
    // the group's matrix as its B operand (B[] is then ignored); each grp_n[k] must be a multiple of the tile width
    TcMat Bgrp[3];
    int ngrp, grp_n[3];
    int a_row0, a_col0, a_zrow, a_zcol;
    int b_row0, b_col0, b_zrow, b_zcol;
    int M, N, K, batch;
    float* C;
    float* const* C_ind;   // optional: device location holding the fp32 output base (C then only gives the alignment)
    long long ldc;
    const float* addend;
    long long ldadd;
    int c_row0, c_col0, c_zrow, c_zcol, c_rows, c_cols;   // stores are clipped to [0,c_rows) x [0,c_cols)
    __nv_bfloat16* out[3];
    long long ldo;
    int nout;
    int out_col_off;   // the bf16 parts are stored at column (absolute column - out_col_off)
    float alpha;
    bool accumulate, lower_only;
    int k_tri;      // 0: dense; 1: B lower triangular (skip k tiles past the row); 2: B upper triangular
    int a_tri;      // the same for the A operand (1: A[m][k] = 0 for k > m; 2: A[m][k] = 0 for k < m)
    bool skip_tile00;     // leave the first tile (rows and columns [0,128) of the product) alone
    bool out_col0_only;   // write the bf16 parts only for the first 128-column block of the product
    unsigned long long* stamps;   // optional device array of 16 global-timer marks (phases of the first CTA, epilogue chunks)
    bool f16;       // the operands are fp16 (same 16-bit containers; both operands of a pass must share the type)
    // optional: device words holding the bit pattern of max|x| of the fp32 arrays the A / B operands were made from
    // by scaled_f16_from_max (pkv_ptx.cuh); the product is divided by the two power-of-two scales
    const unsigned* amax_a;
    const unsigned* amax_b;
    int nacc;       // 0/1: one fp32 accumulator; 2 or 4: the hi x hi pass of a split product is accumulated apart
                    // from the cross passes (and in several parts), which removes most of the tensor core's
                    // truncation bias from sums of same-signed terms; pass 0 must be the hi x hi pass
};
struct MapCache;
MapCache* tc_map_cache_create();
void tc_map_cache_destroy(MapCache* c);
int gemm_tc(const Lc& lc, const TcGemm& g, DevStatus* status);
bool tc_encode_available();
void tc_selftest_wait(const Lc& lc, DevStatus* status);
int tc_make_map_2d(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows);
int tc_make_map_3d(CUtensorMap* m, const void* ptr, uint64_t d2, uint64_t rows, uint64_t cols, uint64_t ld1,
                   uint64_t ld2, uint32_t box_rows);

struct Pair;
// Workspace of the tensor-core ridge solve: bf16 triples (hi, mid, lo) of the factor L, its inverse X,
// the inverse's transpose, the current panel, the doubling temporaries; pairs of S_T and S_T X^T.
constexpr int kSolveEvents = 9;
constexpr int kSolveGraphs = 4;
// One captured solve: replayed when the operands, the shape and the precision plan are the same.
struct SolveGraph {
    const float *G, *S_T;
    int n, ld, d;
    bool well, triple, aligned, wait;
    const void *pair_hi, *pair_lo;
    cudaGraphExec_t exec;
    cudaGraphExec_t exec2;     // final products, where the solve waits for S_T between two graphs (else null)
    int64_t launches;
    unsigned long long used;
};
struct TcSolveBuffers {
    __nv_bfloat16* L3[3];
    __nv_bfloat16* X3[3];
    __nv_bfloat16* XT3[3];
    __nv_bfloat16* P3[3];
    __nv_bfloat16* TT3[3];
    __nv_bfloat16* S2[3];
    __nv_bfloat16* Z2[3];
    int nmax;              // largest system the arrays are sized for
    cudaStream_t aux;      // high-priority helper stream of the factorisation's critical chain
    cudaStream_t bulk;     // helper stream: panels and the first two block columns of every trailing update
    cudaStream_t bulk2;    // helper stream: the rest of every trailing update
    cudaStream_t aux2;     // helper stream: the doubling levels of the inverse beside the factorisation
    cudaEvent_t ev[kSolveEvents];
    cudaEvent_t st_ready;  // recorded by a caller that produces S_T on another stream beside the factorisation
    CUtensorMap chainP[3], chainX[3];   // tensor maps of the chain kernel's operands, valid for (chain_n, chain_ld)
    int chain_n, chain_ld;
    long long* stamps;     // phase marks of the chain kernel (profiling aid)
    float** slot;          // device location of the result's address, read by a captured solve's final products
    DevStatus* gstatus;    // status word of a captured solve (copied from / to the caller's)
    cudaStream_t origin;   // stream the solve is captured on
    SolveGraph graphs[kSolveGraphs];
    int n_graphs, graph_off;
    unsigned long long graph_clock;
};
void tc_solve_destroy(TcSolveBuffers* t);
size_t tc_solve_carve(TcSolveBuffers* t, char* base, size_t off, int nmax, int dmax);
int tc_solve_init(TcSolveBuffers* t);
// dW [d][n] = S_T (S + lambda I)^{-1}, lambda = status->lam; S [n][n] (lower part read) is destroyed.
// ld: row stride of S, S_T, dW (multiple of 8).  zero_fill: ld differs from the previous call's.
int tc_ridge_solve_impl(const Lc& lc, TcSolveBuffers* t, const float* G, const float* S_T, int n, int ld, int d,
                        float* dW, bool well_conditioned, bool zero_fill, DevStatus* status, const Pair* dW_pair,
                        __nv_bfloat16* const* S_T_triple,    // optional: dW's bf16 pair out; S_T already split
                        bool wait_S_T = false);              // S_T is complete only once t->st_ready has fired

// dW [d][n] += (R X^T) X with the inverse factor X of the system solved last on t (one correction of iterative
// refinement); R [d][n] fp32, row stride ld.
int tc_solve_apply_add(const Lc& lc, TcSolveBuffers* t, const float* R, int n, int ld, int d, float* dW,
                       bool well_conditioned, DevStatus* status);

int tc_fp32_product(const Lc& lc, TcSolveBuffers* t, size_t cap_elems, const float* A, const float* B, int M, int N,
                    int K, float alpha, float* C, bool accumulate, int passes, int nacc, DevStatus* status,
                    bool b_in_factor_buffer = false);


// bf16 hi/lo pairs of fp32 activations: v ~= hi + lo with hi = bf16(v), lo = bf16(v - hi).
struct Pair {
    __nv_bfloat16* hi;
    __nv_bfloat16* lo;
};

struct TcBuffers {
    int ldT;            // leading dimension of the token-contiguous (transposed) operands
    Pair u;             // [2N][d]   norm outputs (attention norm, then MLP norm)
    Pair a;             // [2N][Dq]  [aF; dA]
    Pair hF, hC, dh;    // [N][F]
    Pair XT;            // [F][ldT]  student features, token-contiguous
    Pair RT;            // [d][ldT]  targets, token-contiguous
    unsigned* stat;     // [0], [1]: bit patterns of max|H'|, max|T| of the current statistics (fp16 single-pass form)
    int stats_f16;      // the operands in XT.hi / RT.hi are scaled fp16 copies (else bf16 pairs)
    __nv_bfloat16* XT3; // third bf16 parts of XT / RT (statistics in six passes when the ridge coefficient is small)
    __nv_bfloat16* RT3;
    Pair dW;            // [d][F]
    float* qkv;         // [2N][Dq+2Dkv]
    float* o;           // [2N][d]
    float* gu;          // [2N][2F]
    float* dAbuf;       // unused placeholder
    Pair q;             // [2][Hq][N][hd]   rotated, pre-scaled queries for the attention kernel
    __nv_bfloat16* kn;  // [2][Hkv][N][hd]  reference tokens' keys
    __nv_bfloat16* vn;  // [2][Hkv][N][hd]  reference tokens' values
    void* K16;          // fp16 copy of the full cache's keys [Hkv][L][hd] (hd = 128 attention, fp16 key operands)
    void* Kc16;         // fp16 copy of the compact cache's keys [Hkv * b_max][hd]
    float* part_m;      // attention split partials [splits][Hkv][N*g]
    float* part_l;
    float* part_O;      // [splits][Hkv][N*g][hd]
    TcSolveBuffers solve;
    __nv_bfloat16* S3[3];   // bf16 triple of the build's own S_T (aliases solve.S2), written by the Gram epilogue
    int S3_ready;
    const float* own_S_T;
    // Side stream: S_T needs the targets, the factorisation of S_H + lambda I does not.  The target product (S6),
    // the cross statistics S_T and the teacher's next state are issued on `side` (lowest priority) and run in the
    // SMs the latency-bound factorisation leaves idle; the solve waits for solve.st_ready before its first use of
    // S_T.  S_T_async: such work is in flight for the next solve; next_async: the teacher's next state as well.
    cudaStream_t side;
    cudaEvent_t evSide, evSideDone;
    int S_T_async, next_async;
    // Single-block build with the whole teacher half beside the solve (tc_forward_overlapped): the student half runs
    // first, on `fast` (high priority), the teacher half on `side`; evq orders the two (see there).
    cudaStream_t fast;
    cudaEvent_t evq[6];
    cudaEvent_t tr[6];  // PKV_BUILD_TRACE=1: timed marks (start, S_H, teacher attention, S_T, solve, end), else null
    // dual (N x N) solver: its own work arrays and the fp32 staging of G_d, T^T and Y
    int dual_enabled, dual_ld_prev;
    TcSolveBuffers dual;
    float* Gd;          // [N][ldn]
    float* RTf;         // [d][ldn]
    float* Yd;          // [d][ldn]
    Pair Yp;            // [d][ldn]
};

struct TcForwardArgs {
    const pkv_block_weights* w;
    const pkv_kv* full;
    const void* Kc; const void* Vc; const float* bias;
    const float* xF; const float* xC;
    int N, pos0, max_b, total_kept, kv_split;
    const int32_t* head_off; const int32_t* tok_cs; float* rope_tab;
    float *zF, *zC, *dz, *hF, *hC, *R, *S_H, *S_T, *aF, *aC, *dA;
    float* xF_next;     // optional: teacher state entering the next block
    const float* dx;    // student half: xF - xC entering this block (state difference carried between blocks)
    float *part_m, *part_l, *part_O;
    int dual;           // 1: only the token-contiguous copy of the student features is prepared in S7
    int accumulate_stats;   // 1: S_H, S_T are added to (streamed reference sets, Eq. 9) instead of overwritten
    int precise_stats;  // 1: statistics from bf16 triples in six passes (small ridge coefficient), else pairs in three
    DevStatus* status;
    cudaEvent_t* ev;    // stage marks (index = stage) or nullptr
    cudaEvent_t* evT;   // 6 marks around the teacher half's stages (S1-2, S3, S4, S5, S9 share) or nullptr
};

// Rank-r patch (appendix): U [d][r], Br [r][F] = U^T dW, optional dWr [d][F] = U Br, optional evals [r + 8].
size_t tc_lowrank_scratch_bytes(int d, int F, int r);
int tc_lowrank(const Lc& lc, TcBuffers* t, const pkv_dims* D, const float* dW, const float* S_H, int r, int iters,
               void* scratch, float* U, float* Br, float* dWr, float* evals_out, DevStatus* status);

void tc_attn_plan(const pkv_dims* d, int N, int max_b, int mode, int* tps, int* nsplitF, int* nsplitC, int* zoffC);
int tc_attn_partial_slots(const pkv_dims* d);
// q/k_new/v_new of `a` are fp32; rope_tab != nullptr rotates q and k on the way in.
int attention_tc(const Lc& lc, TcBuffers* t, const pkv_dims* d, const AttnArgs& a, const float* rope_tab,
                 DevStatus* status);
int tc_supported(const pkv_dims* d, int cc_major, int cc_minor);
size_t tc_carve(TcBuffers* t, char* base, size_t off, const pkv_dims* d, int dual);
// S7'+S8 of the dual form: G_d = X X^T, lambda, Y = T^T (G_d + lambda I)^{-1}, dW = Y X.
int tc_dual_solve(const Lc& lc, TcBuffers* t, const pkv_dims* d, int N, const float* R, float lam0, int mode,
                  float* dW, DevStatus* status);
int tc_init(TcBuffers* t, const pkv_dims* d);
void tc_destroy(TcBuffers* t);
int tc_forward(const Lc& lc, TcBuffers* t, const pkv_dims* d, const TcForwardArgs& a);
// Same results as tc_forward up to rounding, scheduled for one block with nothing else to overlap: student half and
// S_H first, so that the factorisation can start; teacher half, targets and S_T on the side stream beside it.
// Returns false (nothing issued) where that schedule does not apply (stage marks, dual form, accumulation, switched
// off by PKV_SIDE_STREAM=0 or PKV_BUILD_OVERLAP=0).
bool tc_forward_overlapped_applies(const TcBuffers* t, const TcForwardArgs& a);
int tc_forward_overlapped(const Lc& lc, TcBuffers* t, const pkv_dims* d, const TcForwardArgs& a,
                          cudaStream_t teacher_stream);   // stream of the teacher half (nullptr: the side stream)
int tc_teacher_forward(const Lc& lc, TcBuffers* t, const pkv_dims* d, const TcForwardArgs& a, float* xF_next);
int tc_student_forward(const Lc& lc, TcBuffers* t, const pkv_dims* d, const TcForwardArgs& a);
int tc_attention(const Lc& lc, TcBuffers* t, const pkv_dims* d, const AttnArgs& a, DevStatus* status);
void tc_gram(const Lc& lc, TcBuffers* t, const pkv_dims* d, const float* X, const float* R, int n, float* S_H,
             float* S_T, bool accumulate, DevStatus* status, bool precise = false);
// The precision rule shared by the statistics and the solve.  Under the adaptive scale of Eq. 7,
// cond(S_H + lambda I) is about (sigma_max / (||S_H||_F^2 / tr S_H)) / lambda0, a few tens when lambda0 >= 0.05:
// bf16 pairs (about 16 bits) are enough.  A smaller lambda0, or the absolute / trace-mean coefficients (no such
// bound), take triples everywhere.
inline bool tc_well_conditioned(float lam0, int mode) { return mode == PKV_LAMBDA_PAPER && lam0 >= 0.05f; }
int tc_gram_with_buffers(const Lc& lc, Pair XT, Pair RT, int ldT, const float* X, const float* R, int n, int F, int dm,
                         float* S_H, float* S_T, bool accumulate, DevStatus* status);
// S [F][F] is destroyed; S_T is only read.
void tc_ridge_solve(const Lc& lc, TcBuffers* t, float* S, const float* S_T, int F, int d, float* dW, float lam0,
                    int mode, DevStatus* status);
void tc_next_states(const Lc& lc, TcBuffers* t, const pkv_dims* d, int N, const void* Wdown, const float* dW,
                    const float* zF, const float* R, float* xF_next, float* D, DevStatus* status);
// xF_next = zF + hF Wdown^T on the side stream (only while S_T_async is set: returns false otherwise, nothing issued);
// tc_side_join makes lc.st wait for it.
bool tc_teacher_next_async(const Lc& lc, TcBuffers* t, const pkv_dims* d, int N, const void* Wdown, const float* zF,
                           float* xF_next, DevStatus* status);
void tc_side_join(const Lc& lc, TcBuffers* t);
// after a failed issue: waits (host) for whatever the internal streams still hold
void tc_side_quiesce(TcBuffers* t);
// PKV_BUILD_TRACE=1: mark i on a stream; tc_build_trace_print after the call's synchronisation
void tc_build_trace_mark(TcBuffers* t, int i, cudaStream_t st);
void tc_build_trace_print(TcBuffers* t);
// Student block re-run with the patched down projection (Algorithm 1, student propagation):
// xC_next = z' + (W + dW) h' for the tokens in a.xC against the compact cache.  zero_nd: scratch [N][d].
int tc_student_propagate(const Lc& lc, TcBuffers* t, const pkv_dims* d, const TcForwardArgs& a, const float* dW,
                         float* zero_nd, float* xC_next);
void tc_split_pair(const Lc& lc, const float* src, long long rows, long long cols, Pair out);

}  // namespace pkv
