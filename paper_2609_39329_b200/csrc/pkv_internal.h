// Internal declarations shared by the translation units of libpkv.so.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pkv.h"

namespace pkv {

// Device-resident status and scalar results of one call (zeroed at the start of a call).
struct DevStatus {
    int code;                         // first pkv_error raised on the device (0 = none)
    int info0, info1;                 // see pkv_stats.err_info
    int pad;
    unsigned long long bad_index;     // smallest flat position of an invalid kept index (+1), 0 = none
    unsigned long long bad_column;    // smallest non-positive Cholesky pivot column (+1), 0 = none
    double tr, fro2, t_fro2, res_fro2, dw_fro2;
    float lam;
    float min_pivot;
};

// Kernel attributes (the opt-in to more than 48 KB of dynamic shared memory) belong to the function as
// loaded on ONE device: a launcher keeps one flag per device ordinal and sets the attribute the first
// time it runs with that device current.  Two host threads racing on a flag both set the attribute, which
// is harmless.
constexpr int kMaxDeviceOrdinals = 64;
struct PerDeviceOnce {
    bool done[kMaxDeviceOrdinals] = {};
    // true when the caller still has to do its once-per-device work; dev gets the current ordinal
    bool needed(int* dev) {
        int d = 0;
        if (cudaGetDevice(&d) != cudaSuccess || d < 0 || d >= kMaxDeviceOrdinals) { *dev = -1; return true; }
        *dev = d;
        return !done[d];
    }
    void mark(int dev) { if (dev >= 0) done[dev] = true; }
};

// Every launcher takes the stream and a launch counter.
struct Lc {
    cudaStream_t st;
    int64_t* launches;
    void* map_cache = nullptr;            // tensor-map cache of the tensor-core engine (optional)
    bool pdl = false;                     // launch with programmatic stream serialisation (dependent launch)
    void count(int n = 1) const { if (launches) *launches += n; }
};

// ---- SM partitions (pkv_api.cu): a green context owning a subset of the SMs, and streams inside it ----
bool green_partition_create(int want_sms, void** gctx_out, int* got_sms);
bool green_partition_stream(void* gctx, int priority, cudaStream_t* stream);
void green_partition_destroy(void* gctx);

// ---- pkv_simt.cu -----------------------------------------------------------------------
void gather_kept(const Lc& lc, int elem_bytes, const void* K, const void* V, const int32_t* idx,
                 const int32_t* head_off_dev, int Hkv, int L, int hd, int total, void* Kc, void* Vc,
                 DevStatus* status);
// out [rows][hd] (element type of the cache) = scale * code for a quantised compact cache (bits 8 or 4).
void dequant_cache(const Lc& lc, int elem_bytes, const void* codes, const float* scales, int bits, int group, int hd,
                   int rows, void* out);
// out[r] = x[r] * gain / rms(x[r]) for the rows of x0 (N rows) followed by the rows of x1.
void rmsnorm_f32(const Lc& lc, const float* x0, const float* x1, int N, int d, const float* gain, float eps,
                 float* out);
// C[M][N] = alpha * A[M][K] * B[N][K]^T (+ addend) (+ C if accumulate); B is fp32 or bf16.
// lower_only: tiles strictly above the diagonal are skipped (symmetric updates).
void gemm_tn_simt(const Lc& lc, const float* A, int64_t lda, const void* B, int64_t ldb, bool b_bf16, float* C,
                  int64_t ldc, int M, int N, int K, float alpha, const float* addend, int64_t ldadd,
                  bool accumulate, bool lower_only = false);
// cos/sin table [N][hd/2] of pos = pos0 + (i - chunk_start[i]) (double-precision angles).
void rope_table(const Lc& lc, const int32_t* tok_cs, int N, int hd, int pos0, float theta, float* cs_table);
// rotate `heads` heads of width hd in rows [0, rows) of buf (row stride ld, column offset col0);
// token of row r is r % N.
void rope_apply(const Lc& lc, float* buf, int64_t ld, int col0, int heads, int hd, int rows, int N,
                const float* cs_table);

struct AttnArgs {
    const float* q; int64_t ldq;          // [2*N][..] rotated queries, row = stream*N + token
    const float* k_new; const float* v_new; int64_t ldkv;   // [2*N][..] reference tokens' keys/values
    const void* K; const void* V;         // full cache [Hkv][L][hd]
    const void* Kc; const void* Vc;       // compact cache [total][hd]
    const float* bias;                    // optional logit bias for the compact cache
    const int32_t* head_off;              // device [Hkv+1]
    const int32_t* tok_cs;                // device [N] chunk start of each token
    int N, Hq, Hkv, hd, L, elem_bytes;
    int kv_split, nsplitF, nsplitC;
    int zoffC;                            // slot of the student's first split in the partial buffers (teacher: 0)
    int total_kept, max_b;                // rows of the compact cache (all heads), largest head
    int mode;                             // 0: both streams; 1: teacher only (aF); 2: student only (aC, dA from a given aF)
    float* part_m; float* part_l; float* part_O;   // [nsplit][Hkv][N*g] and [..][hd]
    float* aF; float* aC; float* dA;      // [N][Hq*hd]
    __nv_bfloat16* pair_hi; __nv_bfloat16* pair_lo;   // optional: bf16 hi/lo parts of [aF; dA] as [2N][Hq*hd]
    // Student before teacher (a build whose teacher half runs beside the solve).  With mode 2 the combine writes aC
    // and its pair into rows [N,2N) and no difference; with mode 1 it reads that aC, writes aF and dA = aF - aC and
    // puts the pair of dA (not of aF) into rows [0,N).
    int student_first;
    void* combine_wait;                   // host side only: a cudaEvent_t the combine's stream waits for first
};
void attention_simt(const Lc& lc, const AttnArgs& a);
void attention_combine(const Lc& lc, const AttnArgs& a);

// zF = xF + o[0:N]; dz = (xF - xC) + o[N:2N]; zC = zF - dz.   o is [2N][d].
void oproj_epilogue(const Lc& lc, const float* xF, const float* xC, const float* o, int N, int d, float* zF,
                    float* zC, float* dz);
// gu [2N][2F] (gate | up): hF, hC = silu(gate)*up of the two streams, dh = hF - hC.
void swiglu(const Lc& lc, const float* gu, int N, int F, float* hF, float* hC, float* dh);
void transpose_f32(const Lc& lc, const float* in, int rows, int cols, float* out);
// status->tr, fro2 from S [F][F]; optional sum of squares of an arbitrary buffer into *dst.
// ld = 0: contiguous.  lower: only entries on or below the diagonal are read (S symmetric).
void trace_fro2(const Lc& lc, const float* S, int F, DevStatus* status, int ld = 0, bool lower = false);
void sumsq(const Lc& lc, const float* a, int64_t n, double* dst);
// lambda from the statistics (mode) into status->lam (and min_pivot reset).
void ridge_lambda(const Lc& lc, int F, float lam0, int mode, DevStatus* status);
// lambda from the statistics (mode), G = S_H + lambda I written to G.
void make_ridge_matrix(const Lc& lc, const float* S_H, int F, float lam0, int mode, float* G, DevStatus* status);
// out = a - b (n elements); out may alias a.
void sub_f32(const Lc& lc, const float* a, const float* b, int64_t n, float* out);
// P <- S_T - status->lam * dW - P (n elements), P = dW S_H on entry; status->dw_fro2 (and res_fro2) are reset.
void refine_residual(const Lc& lc, const float* S_T, const float* dW, float* P, int64_t n, DevStatus* status, bool clear_res);
// G [F][F] full symmetric from the lower triangle of S [F][F]; G may be S (the upper part is then filled in place).
void symmetric_from_lower(const Lc& lc, const float* S, float* G, int F);
void merge_weights(const Lc& lc, void* W, int w_dtype, const float* dW, int64_t count);
int fma_peak_tflops(cudaStream_t st, float* scratch, size_t scratch_floats, int sm_count, double* tflops);

// ---- pkv_solve.cu ----------------------------------------------------------------------
struct SolveWs {
    float* G;       // [F][F] ridge matrix, destroyed by the factorisation
    float* Lm;      // [F][F] lower Cholesky factor (upper part zero)
    float* LT;      // [F][F] its transpose
    float* inv;     // [nblk][nb][nb] inverses of the diagonal blocks
    float* invT;    // [nblk][nb][nb] their transposes
    float* Y;       // [d][F] right-hand side, overwritten while solving
};
constexpr int kSolveNb = 64;
// dW [d][F] = S_T G^{-1}; ws.G holds G on entry, ws.Y holds a copy of S_T on entry.
void ridge_solve_simt(const Lc& lc, const SolveWs& ws, int F, int d, float* dW, DevStatus* status);

}  // namespace pkv
