// Rank-r patch (appendix, low-rank weight patches): with M = dW S_H dW^T (d x d, symmetric positive
// semi-definite) and U_r its r leading eigenvectors, the stored patch is the pair (U_r, B_r = U_r^T dW),
// dW_r = U_r B_r: (d + F) r numbers instead of d F.
//
//   1. M on the tensor cores: Y = dW S_H and M = Y dW^T as split-bf16 products (fp32-equivalent);
//   2. the r leading eigenvectors of M by subspace iteration with Rayleigh-Ritz on a block of p = r + 8
//      vectors, in fp64 on the CUDA cores (d^2 p multiply-adds per sweep: small next to step 1): Z = M Q,
//      orthonormalise (Gram-Schmidt twice), T = Q^T M Q, eigenvectors of the p x p matrix T by cyclic Jacobi
//      rotations in one CTA, Q <- Q V ordered by eigenvalue;
//   3. B_r = U_r^T dW and (optionally) dW_r = U_r B_r.
// This is not on the per-block hot path (one call per block after the patch is built).
#include <math.h>

#include "pkv_tc.h"

namespace pkv {

constexpr int kLrMaxP = 48;         // block width limit: r + 8 <= 48 (two p x p fp64 matrices in static shared memory)

// Q [d][p] fp64 column block, deterministic start: a fixed pseudo-random pattern (any start not orthogonal to the
// leading eigenvectors will do)
__global__ void k_lr_init(double* Q, int d, int p) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)d * p) return;
    unsigned long long x = (unsigned long long)i * 0x9E3779B97F4A7C15ull + 0xD1B54A32D192ED03ull;
    x ^= x >> 29; x *= 0xBF58476D1CE4E5B9ull; x ^= x >> 32;
    Q[i] = ((double)(x & 0xFFFFFF) / 16777216.0) - 0.5;
}

// Z [d][p] = M [d][d] (fp32, symmetric) * Q [d][p] (fp64); one CTA per 8 rows, thread (row, column group)
__global__ void __launch_bounds__(256) k_lr_mult(const float* __restrict__ M, const double* __restrict__ Q,
                                                  double* __restrict__ Z, int d, int p) {
    __shared__ double qs[32][kLrMaxP];
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    double acc[2] = {0.0, 0.0};             // columns lane, lane + 32
    for (int k0 = 0; k0 < d; k0 += 32) {
        __syncthreads();
        for (int i = threadIdx.x; i < 32 * p; i += 256) {
            const int kk = i / p, c = i % p;
            qs[kk][c] = (k0 + kk < d) ? Q[(size_t)(k0 + kk) * p + c] : 0.0;
        }
        __syncthreads();
        if (row < d) {
            const int kmax = min(32, d - k0);
            for (int kk = 0; kk < kmax; ++kk) {
                const double m = (double)M[(size_t)row * d + k0 + kk];
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int c = lane + 32 * j;
                    if (c < p) acc[j] = fma(m, qs[kk][c], acc[j]);
                }
            }
        }
    }
    if (row < d) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int c = lane + 32 * j;
            if (c < p) Z[(size_t)row * p + c] = acc[j];
        }
    }
}

__device__ __forceinline__ double lr_block_sum(double v, double* red) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    __syncthreads();
    if (l == 0) red[w] = v;
    __syncthreads();
    double t = (threadIdx.x < (blockDim.x >> 5)) ? red[threadIdx.x] : 0.0;
    if (w == 0) {
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (l == 0) red[0] = t;
    }
    __syncthreads();
    return red[0];
}

// Orthonormalises the p columns of Z [d][p] in place (modified Gram-Schmidt, every projection done twice); one CTA.
__global__ void __launch_bounds__(1024) k_lr_orth(double* Z, int d, int p) {
    __shared__ double red[32];
    for (int c = 0; c < p; ++c) {
        for (int pass = 0; pass < 2; ++pass) {
            for (int j = 0; j < c; ++j) {
                double dot = 0.0;
                for (int i = threadIdx.x; i < d; i += blockDim.x) dot += Z[(size_t)i * p + j] * Z[(size_t)i * p + c];
                dot = lr_block_sum(dot, red);
                for (int i = threadIdx.x; i < d; i += blockDim.x) Z[(size_t)i * p + c] -= dot * Z[(size_t)i * p + j];
                __syncthreads();
            }
        }
        double nn = 0.0;
        for (int i = threadIdx.x; i < d; i += blockDim.x) nn += Z[(size_t)i * p + c] * Z[(size_t)i * p + c];
        nn = lr_block_sum(nn, red);
        const double inv = nn > 0.0 ? rsqrt(nn) : 0.0;
        for (int i = threadIdx.x; i < d; i += blockDim.x) Z[(size_t)i * p + c] *= inv;
        __syncthreads();
    }
}

// T [p][p] = Q^T Z (Q, Z [d][p]); one CTA per (a, b) pair block
__global__ void __launch_bounds__(256) k_lr_gram(const double* __restrict__ Q, const double* __restrict__ Z, double* T,
                                                  int d, int p) {
    __shared__ double red[32];
    const int a = blockIdx.x, b = blockIdx.y;
    double s = 0.0;
    for (int i = threadIdx.x; i < d; i += blockDim.x) s += Q[(size_t)i * p + a] * Z[(size_t)i * p + b];
    s = lr_block_sum(s, red);
    if (threadIdx.x == 0) T[a * p + b] = s;
}

// Eigen-decomposition of the symmetric p x p matrix T by cyclic Jacobi rotations (one CTA, the rotations of a
// sweep in sequence, each applied by the threads in parallel); V's columns ordered by descending eigenvalue.
__global__ void __launch_bounds__(128) k_lr_jacobi(const double* __restrict__ Tin, double* Vout, double* evals, int p) {
    __shared__ double T[kLrMaxP][kLrMaxP + 1];
    __shared__ double V[kLrMaxP][kLrMaxP + 1];
    __shared__ int order[kLrMaxP];
    const int tid = threadIdx.x;
    for (int i = tid; i < p * p; i += blockDim.x) {
        const int a = i / p, b = i % p;
        T[a][b] = 0.5 * (Tin[a * p + b] + Tin[b * p + a]);
        V[a][b] = (a == b) ? 1.0 : 0.0;
    }
    __syncthreads();
    for (int sweep = 0; sweep < 12; ++sweep) {
        for (int a = 0; a < p - 1; ++a) {
            for (int b = a + 1; b < p; ++b) {
                const double apq = T[a][b];
                double c = 1.0, s = 0.0;
                if (fabs(apq) > 1e-300) {
                    const double theta = (T[b][b] - T[a][a]) / (2.0 * apq);
                    const double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
                    c = 1.0 / sqrt(t * t + 1.0);
                    s = t * c;
                }
                __syncthreads();
                // columns a, b of T and V
                for (int k = tid; k < p; k += blockDim.x) {
                    const double ta = T[k][a], tb = T[k][b];
                    T[k][a] = c * ta - s * tb;
                    T[k][b] = s * ta + c * tb;
                    const double va = V[k][a], vb = V[k][b];
                    V[k][a] = c * va - s * vb;
                    V[k][b] = s * va + c * vb;
                }
                __syncthreads();
                // rows a, b of T
                for (int k = tid; k < p; k += blockDim.x) {
                    const double ta = T[a][k], tb = T[b][k];
                    T[a][k] = c * ta - s * tb;
                    T[b][k] = s * ta + c * tb;
                }
                __syncthreads();
            }
        }
    }
    if (tid == 0) {
        for (int i = 0; i < p; ++i) order[i] = i;
        for (int i = 1; i < p; ++i) {                    // insertion sort, descending
            const int o = order[i];
            int j = i - 1;
            while (j >= 0 && T[order[j]][order[j]] < T[o][o]) { order[j + 1] = order[j]; --j; }
            order[j + 1] = o;
        }
    }
    __syncthreads();
    for (int i = tid; i < p * p; i += blockDim.x) {
        const int a = i / p, b = i % p;
        Vout[a * p + b] = V[a][order[b]];
    }
    for (int i = tid; i < p; i += blockDim.x) evals[i] = T[order[i]][order[i]];
}

// Qout [d][p] = Q [d][p] V [p][p]
__global__ void __launch_bounds__(256) k_lr_rotate(const double* __restrict__ Q, const double* __restrict__ V,
                                                    double* __restrict__ Qout, int d, int p) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)d * p) return;
    const size_t row = i / p;
    const int c = (int)(i % p);
    double s = 0.0;
    for (int k = 0; k < p; ++k) s += Q[row * p + k] * V[k * p + c];
    Qout[i] = s;
}

// U [d][r] fp32 = first r columns of Q
__global__ void k_lr_take(const double* __restrict__ Q, int d, int p, int r, float* __restrict__ U) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)d * r) return;
    U[i] = (float)Q[(i / r) * p + (i % r)];
}

// Br [r][F] = U^T dW   (U [d][r], dW [d][F]); thread per (j, f), fp64 accumulation
__global__ void __launch_bounds__(256) k_lr_project(const float* __restrict__ U, const float* __restrict__ dW, int d,
                                                     int F, int r, float* __restrict__ Br) {
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    const int j = blockIdx.y;
    if (f >= F) return;
    double s = 0.0;
    for (int i = 0; i < d; ++i) s += (double)U[(size_t)i * r + j] * (double)dW[(size_t)i * F + f];
    Br[(size_t)j * F + f] = (float)s;
}

// dWr [d][F] = U Br
__global__ void __launch_bounds__(256) k_lr_expand(const float* __restrict__ U, const float* __restrict__ Br, int d,
                                                    int F, int r, float* __restrict__ dWr) {
    const int f = blockIdx.x * blockDim.x + threadIdx.x;
    const int i = blockIdx.y;
    if (f >= F) return;
    float s = 0.f;
    for (int j = 0; j < r; ++j) s = fmaf(U[(size_t)i * r + j], Br[(size_t)j * F + f], s);
    dWr[(size_t)i * F + f] = s;
}

// scratch: M [d][d] fp32, Y [d][F] fp32, Q, Z, Q2 [d][p] fp64, T, V [p][p] fp64, ev [p] fp64
size_t tc_lowrank_scratch_bytes(int d, int F, int r) {
    const size_t p = (size_t)r + 8;
    return ((size_t)d * d + (size_t)d * F) * sizeof(float) + (3 * (size_t)d * p + 2 * p * p + p) * sizeof(double) + 1024;
}

int tc_lowrank(const Lc& lc, TcBuffers* t, const pkv_dims* D, const float* dW, const float* S_H, int r, int iters,
               void* scratch, float* U, float* Br, float* dWr, float* evals_out, DevStatus* status) {
    const int d = D->d, F = D->F;
    const int p = r + 8;
    if (r <= 0 || p > kLrMaxP || p > d) return PKV_ERR_UNSUPPORTED;
    char* base = (char*)scratch;
    float* M = (float*)base; base += (size_t)d * d * sizeof(float);
    float* Y = (float*)base; base += (size_t)d * F * sizeof(float);
    base = (char*)(((uintptr_t)base + 255) & ~(uintptr_t)255);
    double* Q = (double*)base; base += (size_t)d * p * sizeof(double);
    double* Z = (double*)base; base += (size_t)d * p * sizeof(double);
    double* Q2 = (double*)base; base += (size_t)d * p * sizeof(double);
    double* T = (double*)base; base += (size_t)p * p * sizeof(double);
    double* V = (double*)base; base += (size_t)p * p * sizeof(double);
    double* ev = (double*)base;
    // 1. M = (dW S_H) dW^T through the solver's fp32-equivalent product (operand buffers of the solve as scratch)
    t->S3_ready = 0;
    int rc = tc_fp32_product(lc, &t->solve, (size_t)d * F, dW, S_H, d, F, F, 1.f, Y, false, 6, 2, status, true);
    if (rc != PKV_OK) return rc;
    rc = tc_fp32_product(lc, &t->solve, (size_t)d * F, Y, dW, d, d, F, 1.f, M, false, 6, 2, status);
    if (rc != PKV_OK) return rc;
    // 2. subspace iteration with Rayleigh-Ritz
    const unsigned nb = (unsigned)(((size_t)d * p + 255) / 256);
    k_lr_init<<<nb, 256, 0, lc.st>>>(Q, d, p);
    k_lr_orth<<<1, 1024, 0, lc.st>>>(Q, d, p);
    lc.count(2);
    for (int it = 0; it < iters; ++it) {
        k_lr_mult<<<(d + 7) / 8, 256, 0, lc.st>>>(M, Q, Z, d, p);
        k_lr_orth<<<1, 1024, 0, lc.st>>>(Z, d, p);
        // Rayleigh-Ritz in the orthonormal basis Z: T = Z^T (M Z)
        k_lr_mult<<<(d + 7) / 8, 256, 0, lc.st>>>(M, Z, Q2, d, p);
        k_lr_gram<<<dim3(p, p), 256, 0, lc.st>>>(Z, Q2, T, d, p);
        k_lr_jacobi<<<1, 128, 0, lc.st>>>(T, V, ev, p);
        k_lr_rotate<<<nb, 256, 0, lc.st>>>(Z, V, Q, d, p);
        lc.count(6);
    }
    // 3. outputs
    k_lr_take<<<(unsigned)(((size_t)d * r + 255) / 256), 256, 0, lc.st>>>(Q, d, p, r, U);
    k_lr_project<<<dim3((F + 255) / 256, r), 256, 0, lc.st>>>(U, dW, d, F, r, Br);
    lc.count(2);
    if (dWr) {
        k_lr_expand<<<dim3((F + 255) / 256, d), 256, 0, lc.st>>>(U, Br, d, F, r, dWr);
        lc.count();
    }
    if (evals_out) {
        // leading r + 8 Ritz values as fp32 (diagnostics: the gap after the r-th tells how well U_r is determined)
        k_lr_take<<<1, 256, 0, lc.st>>>(ev, 1, p, p, evals_out);
        lc.count();
    }
    return PKV_OK;
}

}  // namespace pkv
