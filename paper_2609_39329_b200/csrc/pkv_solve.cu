// Ridge solve in fp32 (Eq. 8): blocked Cholesky factorisation G = L L^T and the two triangular
// solves dW = S_T L^{-T} L^{-1}, written as GEMM-rich block steps: the diagonal blocks are
// factored and inverted inside one CTA's shared memory, panels and trailing updates are GEMMs.
#include <math.h>

#include "pkv_internal.h"

namespace pkv {

__device__ __forceinline__ void raise_s(DevStatus* s, int code) { atomicCAS(&s->code, 0, code); }

// One CTA factors the nb x nb diagonal block at (k0, k0) of G, stores it into Lm (upper part of
// the block zeroed) and writes the inverse of the factor (and its transpose) for the panel and
// solve steps.  A pivot that is not positive and finite is reported and replaced by 1, so that
// the rest of the call stays finite and ends with PKV_ERR_NOT_PD.
__global__ void __launch_bounds__(256) k_potrf_diag(const float* __restrict__ G, float* __restrict__ Lm, int F,
                                                    int k0, float* __restrict__ inv, float* __restrict__ invT,
                                                    DevStatus* status) {
    constexpr int NB = kSolveNb;
    __shared__ float A[NB][NB + 1];
    __shared__ float X[NB][NB + 1];
    const int tid = threadIdx.x;
    const int nbk = min(NB, F - k0);
    for (int i = tid; i < NB * NB; i += 256) {
        int r = i / NB, c = i % NB;
        float v = (r == c) ? 1.f : 0.f;
        if (r < nbk && c <= r) v = G[(size_t)(k0 + r) * F + k0 + c];
        A[r][c] = v;
        X[r][c] = 0.f;
    }
    __syncthreads();
    float minpiv = INFINITY;
    for (int j = 0; j < NB; ++j) {
        float piv = A[j][j];
        __syncthreads();
        if (!(piv > 0.f) || !isfinite(piv)) {
            if (tid == 0 && j < nbk) {
                raise_s(status, PKV_ERR_NOT_PD);
                unsigned long long key = (unsigned long long)(k0 + j) + 1ull;
                unsigned long long old = status->bad_column;
                while (old == 0ull || key < old) {
                    unsigned long long prev = atomicCAS(&status->bad_column, old, key);
                    if (prev == old) break;
                    old = prev;
                }
            }
            piv = 1.f;
        }
        if (j < nbk) minpiv = fminf(minpiv, piv);
        float dj = sqrtf(piv);
        float rdj = 1.f / dj;
        if (tid == 0) A[j][j] = dj;
        for (int i = j + 1 + tid; i < NB; i += 256) A[i][j] *= rdj;
        __syncthreads();
        // rank-1 update of the trailing lower triangle
        int rem = NB - 1 - j;
        for (int e = tid; e < rem * rem; e += 256) {
            int r = j + 1 + e / rem, c = j + 1 + e % rem;
            if (c <= r) A[r][c] -= A[r][j] * A[c][j];
        }
        __syncthreads();
    }
    if (tid == 0) status->min_pivot = fminf(status->min_pivot, minpiv);
    // inverse of the lower-triangular factor, one column per thread
    if (tid < NB) {
        int c = tid;
        for (int i = c; i < NB; ++i) {
            float s = (i == c) ? 1.f : 0.f;
            for (int k = c; k < i; ++k) s -= A[i][k] * X[k][c];
            X[i][c] = s / A[i][i];
        }
    }
    __syncthreads();
    for (int i = tid; i < NB * NB; i += 256) {
        int r = i / NB, c = i % NB;
        if (r < nbk && c < nbk) Lm[(size_t)(k0 + r) * F + k0 + c] = (c <= r) ? A[r][c] : 0.f;
        inv[i] = X[r][c];
        invT[i] = X[c][r];
    }
}

void ridge_solve_simt(const Lc& lc, const SolveWs& ws, int F, int d, float* dW, DevStatus* status) {
    constexpr int NB = kSolveNb;
    const int nblk = (F + NB - 1) / NB;
    // ---- factorisation, right-looking ----
    cudaMemsetAsync(ws.Lm, 0, (size_t)F * F * sizeof(float), lc.st);
    for (int b = 0; b < nblk; ++b) {
        int k0 = b * NB, k1 = min(F, k0 + NB), nbk = k1 - k0;
        float* inv = ws.inv + (size_t)b * NB * NB;
        float* invT = ws.invT + (size_t)b * NB * NB;
        k_potrf_diag<<<1, 256, 0, lc.st>>>(ws.G, ws.Lm, F, k0, inv, invT, status);
        lc.count();
        int rem = F - k1;
        if (rem > 0) {
            // panel: L21 = G21 L11^{-T}
            gemm_tn_simt(lc, ws.G + (size_t)k1 * F + k0, F, inv, NB, false, ws.Lm + (size_t)k1 * F + k0, F, rem, nbk,
                         nbk, 1.f, nullptr, 0, false);
            // trailing update of the lower triangle: G22 -= L21 L21^T
            gemm_tn_simt(lc, ws.Lm + (size_t)k1 * F + k0, F, ws.Lm + (size_t)k1 * F + k0, F, false,
                         ws.G + (size_t)k1 * F + k1, F, rem, rem, nbk, -1.f, nullptr, 0, true, true);
        }
    }
    transpose_f32(lc, ws.Lm, F, F, ws.LT);
    // ---- Z L^T = S_T, block columns ascending; P = ws.Y (holds S_T), Z goes to dW ----
    float* P = ws.Y;
    float* Z = dW;
    for (int b = 0; b < nblk; ++b) {
        int k0 = b * NB, k1 = min(F, k0 + NB), nbk = k1 - k0;
        const float* inv = ws.inv + (size_t)b * NB * NB;
        gemm_tn_simt(lc, P + k0, F, inv, NB, false, Z + k0, F, d, nbk, nbk, 1.f, nullptr, 0, false);
        int rem = F - k1;
        if (rem > 0)
            gemm_tn_simt(lc, Z + k0, F, ws.Lm + (size_t)k1 * F + k0, F, false, P + k1, F, d, rem, nbk, -1.f, nullptr, 0,
                         true);
    }
    // ---- dW L = Z, block columns descending; result written to P ----
    for (int b = nblk - 1; b >= 0; --b) {
        int k0 = b * NB, k1 = min(F, k0 + NB), nbk = k1 - k0;
        const float* invT = ws.invT + (size_t)b * NB * NB;
        gemm_tn_simt(lc, Z + k0, F, invT, NB, false, P + k0, F, d, nbk, nbk, 1.f, nullptr, 0, false);
        if (k0 > 0)
            gemm_tn_simt(lc, P + k0, F, ws.LT + k0, F, false, Z, F, d, k0, nbk, -1.f, nullptr, 0, true);
    }
    cudaMemcpyAsync(dW, P, (size_t)d * F * sizeof(float), cudaMemcpyDeviceToDevice, lc.st);
}

}  // namespace pkv
