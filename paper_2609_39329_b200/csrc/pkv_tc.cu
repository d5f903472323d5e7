// Tensor-core engine: stage sequence of one block for bf16 weights and caches.
//
// Precision plan.  Weights and caches are bf16 as given.  Every fp32 activation that feeds a
// tensor-core product is carried as a bf16 pair (hi, lo) and multiplied in two passes against
// the same bf16 weight tile (three passes when both factors are fp32), all accumulating in
// fp32 tensor memory; differences (dA, dz, dh) are formed in fp32 before any rounding so that
// the target T = W dh + dz of Eq. 5 does not inherit the rounding of two nearly equal streams.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <cuda_fp16.h>

#include "pkv_tc.h"
#include "pkv_ptx.cuh"

namespace pkv {

// ---------------------------------------------------------------------------------------------
// element-wise kernels producing bf16 pairs
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void split2(float v, __nv_bfloat16& hi, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(v);
    lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// The element-wise kernels below are bound by HBM: every thread moves four consecutive elements (16-byte loads of
// fp32, 8-byte stores of bf16 parts).  Row lengths (d, F) are multiples of 8 and every buffer is 16-byte aligned.
__device__ __forceinline__ uint32_t pack_bf16x2(__nv_bfloat16 a, __nv_bfloat16 b) {
    return (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
}
// hi/lo parts of four consecutive values at element index i (a multiple of 4)
__device__ __forceinline__ void store_pair4(__nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo, size_t i, float4 v) {
    __nv_bfloat16 h0, h1, h2, h3, l0, l1, l2, l3;
    split2(v.x, h0, l0); split2(v.y, h1, l1); split2(v.z, h2, l2); split2(v.w, h3, l3);
    *reinterpret_cast<uint2*>(hi + i) = make_uint2(pack_bf16x2(h0, h1), pack_bf16x2(h2, h3));
    *reinterpret_cast<uint2*>(lo + i) = make_uint2(pack_bf16x2(l0, l1), pack_bf16x2(l2, l3));
}
__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void st4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ float4 sub4(float4 a, float4 b) { return make_float4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w); }
__device__ __forceinline__ float4 add4(float4 a, float4 b) { return make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); }

// rows [row0, row0 + gridDim.x) of the stacked input (rows [0,N) from x0, rows [N,2N) from x1)
__global__ void __launch_bounds__(256) k_rmsnorm_split(const float* __restrict__ x0, const float* __restrict__ x1,
                                                       int N, int d, const float* __restrict__ gain, float eps,
                                                       __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                                       int row0) {
    __shared__ float red[32];
    int r = blockIdx.x + row0;
    const float* x = (r < N) ? x0 + (size_t)r * d : x1 + (size_t)(r - N) * d;
    const int d4 = d >> 2;
    float ss = 0.f;
    for (int c = threadIdx.x; c < d4; c += blockDim.x) {
        const float4 v = ld4(x + 4 * c);
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float t = (threadIdx.x < 8) ? red[threadIdx.x] : 0.f;
    if (threadIdx.x < 32) {
        for (int o = 4; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (threadIdx.x == 0) red[0] = t;
    }
    __syncthreads();
    float inv = 1.0f / sqrtf(red[0] / (float)d + eps);
    for (int c = threadIdx.x; c < d4; c += blockDim.x) {
        const float4 v = ld4(x + 4 * c), g = ld4(gain + 4 * c);
        store_pair4(hi, lo, (size_t)r * d + 4 * c, make_float4(v.x * g.x * inv, v.y * g.y * inv, v.z * g.z * inv, v.w * g.w * inv));
    }
}

__device__ __forceinline__ float silu_f(float t) { return t / (1.0f + expf(-t)); }
// silu(gate) * up for four consecutive features of the row a [2F] (gate | up)
__device__ __forceinline__ float4 swiglu4(const float* __restrict__ a, size_t c, int F) {
    const float4 g = ld4(a + c), u = ld4(a + F + c);
    return make_float4(silu_f(g.x) * u.x, silu_f(g.y) * u.y, silu_f(g.z) * u.z, silu_f(g.w) * u.w);
}

// gu [2N][2F] (gate | up) -> hF, hC (fp32 + pairs), dh = hF - hC (pair); one thread per four features
__global__ void __launch_bounds__(256) k_swiglu_split(const float* __restrict__ gu, int N, int F,
                                                      float* __restrict__ hF32, float* __restrict__ hC32, Pair hF,
                                                      Pair hC, Pair dh) {
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= (size_t)N * F) return;
    const size_t r = i / F, c = i % F;
    const float4 f = swiglu4(gu + r * 2 * F, c, F);
    const float4 s = swiglu4(gu + (r + N) * 2 * F, c, F);
    st4(hF32 + i, f);
    st4(hC32 + i, s);
    store_pair4(hF.hi, hF.lo, i, f);
    store_pair4(hC.hi, hC.lo, i, s);
    store_pair4(dh.hi, dh.lo, i, sub4(f, s));
}

// teacher half: hF (fp32 + pair) from gu rows [0,N)
__global__ void __launch_bounds__(256) k_swiglu_teacher(const float* __restrict__ gu, int N, int F,
                                                        float* __restrict__ hF32, Pair hF) {
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= (size_t)N * F) return;
    const size_t r = i / F, c = i % F;
    const float4 f = swiglu4(gu + r * 2 * F, c, F);
    st4(hF32 + i, f);
    store_pair4(hF.hi, hF.lo, i, f);
}
// student half: hC (fp32 + pair) from gu rows [N,2N), dh = hF - hC (pair) with the teacher's hF
__global__ void __launch_bounds__(256) k_swiglu_student(const float* __restrict__ gu, int N, int F,
                                                        const float* __restrict__ hF32, float* __restrict__ hC32,
                                                        Pair hC, Pair dh) {
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= (size_t)N * F) return;
    const size_t r = i / F, c = i % F;
    const float4 s = swiglu4(gu + (r + N) * 2 * F, c, F);
    st4(hC32 + i, s);
    store_pair4(hC.hi, hC.lo, i, s);
    store_pair4(dh.hi, dh.lo, i, sub4(ld4(hF32 + i), s));
}
// teacher half of the o-projection epilogue: zF = xF + o[0:N]   (n elements, four per thread)
__global__ void k_oproj_teacher(const float* __restrict__ xF, const float* __restrict__ o, size_t n,
                                float* __restrict__ zF) {
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i < n) st4(zF + i, add4(ld4(xF + i), ld4(o + i)));
}
// student half: dz = dx + o[N:2N] (dx = xF - xC entering the block, o[N:2N] the projection of dA); zC = zF - dz
__global__ void k_oproj_student(const float* __restrict__ dx, const float* __restrict__ o,
                                const float* __restrict__ zF, size_t n, float* __restrict__ zC,
                                float* __restrict__ dz) {
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= n) return;
    const float4 dd = add4(ld4(dx + i), ld4(o + n + i));
    st4(dz + i, dd);
    st4(zC + i, sub4(ld4(zF + i), dd));
}

// teacher half after the student's: dz = (xF - xC) + o[0:N] (the projection of dA), zF = zC + dz; dx, if given, is
// the incoming state difference carried between the blocks of a stack
__global__ void k_oproj_teacher_diff(const float* __restrict__ xF, const float* __restrict__ xC,
                                     const float* __restrict__ dx, const float* __restrict__ o,
                                     const float* __restrict__ zC, size_t n, float* __restrict__ zF,
                                     float* __restrict__ dz) {
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= n) return;
    const float4 dd = add4(dx ? ld4(dx + i) : sub4(ld4(xF + i), ld4(xC + i)), ld4(o + i));
    st4(dz + i, dd);
    st4(zF + i, add4(ld4(zC + i), dd));
}
// teacher half after the student's: hF (fp32 + pair) from gu rows [0,N), dh = hF - hC (pair) with the student's hC
__global__ void __launch_bounds__(256) k_swiglu_teacher_diff(const float* __restrict__ gu, int N, int F,
                                                             const float* __restrict__ hC32, float* __restrict__ hF32,
                                                             Pair hF, Pair dh) {
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= (size_t)N * F) return;
    const size_t r = i / F, c = i % F;
    const float4 f = swiglu4(gu + r * 2 * F, c, F);
    st4(hF32 + i, f);
    store_pair4(hF.hi, hF.lo, i, f);
    store_pair4(dh.hi, dh.lo, i, sub4(f, ld4(hC32 + i)));
}

// in [rows][cols] fp32 -> out pair [cols][ldo] (token-contiguous operands of the statistics).  A block transposes a
// tile of 64 rows x 32 columns; on the way out a thread stores two consecutive tokens of one feature (4 bytes).
// ldo is even, and rows beyond the matrix are left alone (their bytes are never read: the contraction stops at n).
__global__ void k_transpose_split(const float* __restrict__ in, int rows, int cols, int ldo, Pair out,
                                  __nv_bfloat16* __restrict__ out3) {
    __shared__ float t[64][33];
    int c0 = blockIdx.x * 32, r0 = blockIdx.y * 64;
    for (int j = threadIdx.y; j < 64; j += 8) {
        int r = r0 + j, c = c0 + threadIdx.x;
        t[j][threadIdx.x] = (r < rows && c < cols) ? in[(size_t)r * cols + c] : 0.f;
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        int c = c0 + j, r = r0 + 2 * threadIdx.x;
        if (r < rows && c < cols) {
            const float v0 = t[2 * threadIdx.x][j], v1 = t[2 * threadIdx.x + 1][j];
            __nv_bfloat16 h0, l0, h1, l1;
            split2(v0, h0, l0);
            split2(v1, h1, l1);
            const size_t o = (size_t)c * ldo + r;
            if (r + 1 < rows) {
                *reinterpret_cast<uint32_t*>(out.hi + o) = pack_bf16x2(h0, h1);
                *reinterpret_cast<uint32_t*>(out.lo + o) = pack_bf16x2(l0, l1);
                if (out3)
                    *reinterpret_cast<uint32_t*>(out3 + o) =
                        pack_bf16x2(__float2bfloat16_rn((v0 - __bfloat162float(h0)) - __bfloat162float(l0)),
                                    __float2bfloat16_rn((v1 - __bfloat162float(h1)) - __bfloat162float(l1)));
            } else {
                out.hi[o] = h0;
                out.lo[o] = l0;
                if (out3) out3[o] = __float2bfloat16_rn((v0 - __bfloat162float(h0)) - __bfloat162float(l0));
            }
        }
    }
}

// out3 != nullptr: also the third bf16 part (triples, 24 mantissa bits)
// max |x| of an fp32 array as a bit pattern (non-negative floats order like their bits); *out zeroed before
__global__ void __launch_bounds__(256) k_absmax(const float4* __restrict__ x, size_t n4, unsigned* __restrict__ out) {
    unsigned m = 0u;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        const float4 v = x[i];
        m = max(max(m, __float_as_uint(fabsf(v.x))), max(__float_as_uint(fabsf(v.y)), max(__float_as_uint(fabsf(v.z)), __float_as_uint(fabsf(v.w)))));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m) atomicMax(out, m);
}
// in [rows][cols] fp32 -> out [cols][ldo] fp16 of in * 2^e, e from the array's maximum (f16_scale_from_max); tiles and
// stores as in k_transpose_split
__global__ void k_transpose_f16(const float* __restrict__ in, int rows, int cols, int ldo, __half* __restrict__ out,
                                const unsigned* __restrict__ amax) {
    __shared__ float t[64][33];
    const float sc = ptx::f16_scale_from_max(*amax);
    int c0 = blockIdx.x * 32, r0 = blockIdx.y * 64;
    for (int j = threadIdx.y; j < 64; j += 8) {
        int r = r0 + j, c = c0 + threadIdx.x;
        t[j][threadIdx.x] = (r < rows && c < cols) ? in[(size_t)r * cols + c] : 0.f;
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        int c = c0 + j, r = r0 + 2 * threadIdx.x;
        if (r < rows && c < cols) {
            const size_t o = (size_t)c * ldo + r;
            if (r + 1 < rows) *reinterpret_cast<__half2*>(out + o) = __floats2half2_rn(t[2 * threadIdx.x][j] * sc, t[2 * threadIdx.x + 1][j] * sc);
            else out[o] = __float2half_rn(t[2 * threadIdx.x][j] * sc);
        }
    }
}

static bool stats_f16_on() {
    static const bool v = [] { const char* e = getenv("PKV_STATS_F16"); return !e || atoi(e) != 0; }();
    return v;
}

// Token-contiguous operand of the build's own statistics from X [rows][cols] (which = 0: student features, 1: targets).
// Well-conditioned plan: one scaled fp16 copy (eleven bits: the statistics then take one pass instead of three; the
// rounding reaches dW as about 3.5e-4 relative, against 1e-5 for pairs, under a tolerance of 5e-3).  Else bf16 pairs,
// with third parts when `precise`.
static void stats_operand(const Lc& lc, TcBuffers* t, const float* X, int rows, int cols, int which, bool precise) {
    Pair out = which ? t->RT : t->XT;
    if (which ? t->stats_f16 != 0 : (!precise && stats_f16_on())) {      // cols is a multiple of 8 (tc_supported)
        cudaMemsetAsync(t->stat + which, 0, sizeof(unsigned), lc.st);
        const size_t n4 = (size_t)rows * cols / 4;
        const size_t nb = (n4 + 255) / 256;
        k_absmax<<<(unsigned)(nb < 1184 ? nb : 1184), 256, 0, lc.st>>>(reinterpret_cast<const float4*>(X), n4, t->stat + which);
        lc.count();
        dim3 grid((cols + 31) / 32, (rows + 63) / 64), block(32, 8);
        k_transpose_f16<<<grid, block, 0, lc.st>>>(X, rows, cols, t->ldT, reinterpret_cast<__half*>(out.hi), t->stat + which);
        lc.count();
        if (which == 0) t->stats_f16 = 1;
        return;
    }
    if (which == 0) t->stats_f16 = 0;
    dim3 grid((cols + 31) / 32, (rows + 63) / 64), block(32, 8);
    k_transpose_split<<<grid, block, 0, lc.st>>>(X, rows, cols, t->ldT, out, precise ? (which ? t->RT3 : t->XT3) : nullptr);
    lc.count();
}

static void transpose_split(const Lc& lc, const float* in, int rows, int cols, int ldo, Pair out,
                            __nv_bfloat16* out3 = nullptr) {
    dim3 grid((cols + 31) / 32, (rows + 63) / 64), block(32, 8);
    k_transpose_split<<<grid, block, 0, lc.st>>>(in, rows, cols, ldo, out, out3);
    lc.count();
}

// ---------------------------------------------------------------------------------------------
// helpers
// ---------------------------------------------------------------------------------------------
static TcGemm plain_gemm(int M, int Nn, int K, float* C, long long ldc, float alpha, const float* addend,
                         long long ldadd, bool accumulate) {
    TcGemm g{};
    g.M = M; g.N = Nn; g.K = K; g.batch = 1;
    g.C = C; g.ldc = ldc; g.alpha = alpha; g.addend = addend; g.ldadd = ldadd; g.accumulate = accumulate;
    g.c_rows = M; g.c_cols = Nn;
    return g;
}

// C = alpha * (A_hi + A_lo) W^T (+ addend): fp32 activation pair against a bf16 weight [Nn][K].
static int gemm_act_weight(const Lc& lc, Pair A, long long lda, const void* W, long long ldw, float* C,
                           long long ldc, int M, int Nn, int K, float alpha, const float* addend, long long ldadd,
                           DevStatus* st) {
    TcGemm g = plain_gemm(M, Nn, K, C, ldc, alpha, addend, ldadd, false);
    g.A[0] = TcMat{A.hi, lda, M, K};
    g.A[1] = TcMat{A.lo, lda, M, K};
    g.B[0] = g.B[1] = TcMat{(const __nv_bfloat16*)W, ldw, Nn, K};
    g.npass = 2;
    return gemm_tc(lc, g, st);
}

// The same for two or three weight matrices applied to the same activations, their outputs side by side in C
// (q | k | v, gate | up): one launch when every width is a multiple of 256, else one per matrix.
static int gemm_act_weights(const Lc& lc, Pair A, long long lda, const void* const* W, const int* widths, int nw,
                            long long ldw, float* C, long long ldc, int M, int K, DevStatus* st) {
    bool grouped = nw > 1 && nw <= 3;
    int total = 0;
    for (int k = 0; k < nw; ++k) { grouped = grouped && widths[k] % 256 == 0; total += widths[k]; }
    if (!grouped) {
        int off = 0;
        for (int k = 0; k < nw; ++k) {
            const int rc = gemm_act_weight(lc, A, lda, W[k], ldw, C + off, ldc, M, widths[k], K, 1.f, nullptr, 0, st);
            if (rc != PKV_OK) return rc;
            off += widths[k];
        }
        return PKV_OK;
    }
    TcGemm g = plain_gemm(M, total, K, C, ldc, 1.f, nullptr, 0, false);
    g.A[0] = TcMat{A.hi, lda, M, K};
    g.A[1] = TcMat{A.lo, lda, M, K};
    g.B[0] = g.B[1] = TcMat{(const __nv_bfloat16*)W[0], ldw, widths[0], K};
    g.npass = 2;
    g.ngrp = nw;
    for (int k = 0; k < nw; ++k) {
        g.Bgrp[k] = TcMat{(const __nv_bfloat16*)W[k], ldw, widths[k], K};
        g.grp_n[k] = widths[k];
    }
    return gemm_tc(lc, g, st);
}

// C = alpha * (A_hi + A_lo)(B_hi + B_lo)^T without the lo*lo term (+ addend) (+ C).
static int gemm_pair_pair(const Lc& lc, Pair A, long long lda, Pair B, long long ldb, float* C, long long ldc, int M,
                          int Nn, int K, float alpha, const float* addend, long long ldadd, bool accumulate,
                          DevStatus* st) {
    TcGemm g = plain_gemm(M, Nn, K, C, ldc, alpha, addend, ldadd, accumulate);
    g.A[0] = TcMat{A.hi, lda, M, K}; g.B[0] = TcMat{B.hi, ldb, Nn, K};
    g.A[1] = TcMat{A.hi, lda, M, K}; g.B[1] = TcMat{B.lo, ldb, Nn, K};
    g.A[2] = TcMat{A.lo, lda, M, K}; g.B[2] = TcMat{B.hi, ldb, Nn, K};
    g.npass = 3;
    return gemm_tc(lc, g, st);
}

int tc_supported(const pkv_dims* d, int cc_major, int cc_minor) {
    (void)cc_minor;
    if (cc_major != 10) return PKV_ERR_UNSUPPORTED;                      // tcgen05 / TMEM: sm_100 only
    if (d->dtype != PKV_BF16) return PKV_ERR_UNSUPPORTED;
    if (d->d % 8 || d->F % 8) return PKV_ERR_UNSUPPORTED;                // 16-byte TMA row strides
    if (!tc_encode_available()) return PKV_ERR_UNSUPPORTED;
    return PKV_OK;
}

struct Carver2 {
    char* base;
    size_t off;
    template <typename T>
    T* take(size_t n) {
        off = (off + 255) & ~(size_t)255;
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
    Pair pair(size_t n) {
        Pair p;
        p.hi = take<__nv_bfloat16>(n);
        p.lo = take<__nv_bfloat16>(n);
        return p;
    }
};

size_t tc_carve(TcBuffers* t, char* base, size_t off, const pkv_dims* d, int dual) {
    Carver2 c{base, off};
    const size_t N = d->N_max, dm = d->d, F = d->F, Dq = (size_t)d->Hq * d->hd, Dkv = (size_t)d->Hkv * d->hd;
    t->ldT = (int)((N + 7) / 8 * 8);
    t->u = c.pair(2 * N * dm);
    t->a = c.pair(2 * N * Dq);
    t->hF = c.pair(N * F);
    t->hC = c.pair(N * F);
    t->dh = c.pair(N * F);
    t->XT = c.pair(F * (size_t)t->ldT);
    t->RT = c.pair(dm * (size_t)t->ldT);
    t->stat = c.take<unsigned>(64);
    t->stats_f16 = 0;
    t->XT3 = c.take<__nv_bfloat16>(F * (size_t)t->ldT);
    t->RT3 = c.take<__nv_bfloat16>(dm * (size_t)t->ldT);
    t->dW = c.pair(dm * F);
    t->qkv = c.take<float>(2 * N * (Dq + 2 * Dkv));
    t->o = c.take<float>(2 * N * dm);
    t->gu = c.take<float>(2 * N * 2 * F);
    t->dAbuf = nullptr;
    t->q = c.pair(2 * N * Dq);
    t->kn = c.take<__nv_bfloat16>(2 * N * Dkv);
    t->vn = c.take<__nv_bfloat16>(2 * N * Dkv);
    t->K16 = t->Kc16 = nullptr;
    if (d->hd == 128) {
        t->K16 = c.take<__nv_bfloat16>((size_t)d->Hkv * d->L * d->hd + 8);
        t->Kc16 = c.take<__nv_bfloat16>((size_t)d->Hkv * d->b_max * d->hd + 128 * d->hd);
    }
    const size_t rows = N * (d->Hq / d->Hkv);
    const size_t nsp = (size_t)tc_attn_partial_slots(d);
    t->part_m = c.take<float>(nsp * d->Hkv * rows);
    t->part_l = c.take<float>(nsp * d->Hkv * rows);
    t->part_O = c.take<float>(nsp * d->Hkv * rows * d->hd);
    c.off = tc_solve_carve(&t->solve, base, c.off, d->F, d->d);
    for (int i = 0; i < 3; ++i) t->S3[i] = t->solve.S2[i];     // the solver's S_T operand buffers
    t->S3_ready = 0;
    t->own_S_T = nullptr;
    t->dual_enabled = dual;
    t->dual_ld_prev = 0;
    if (dual) {
        const size_t ldn = (size_t)t->ldT;
        t->Gd = c.take<float>(N * ldn);
        t->RTf = c.take<float>(dm * ldn);
        t->Yd = c.take<float>(dm * ldn);
        t->Yp = c.pair(dm * ldn);
        c.off = tc_solve_carve(&t->dual, base, c.off, (int)ldn, d->d);
    }
    return c.off;
}

int tc_init(TcBuffers* t, const pkv_dims*) {
    int rc = tc_solve_init(&t->solve);
    if (rc == PKV_OK && t->dual_enabled) rc = tc_solve_init(&t->dual);
    if (rc != PKV_OK) return rc;
    int least = 0, greatest = 0;
    cudaDeviceGetStreamPriorityRange(&least, &greatest);
    if (cudaStreamCreateWithPriority(&t->side, cudaStreamNonBlocking, least) != cudaSuccess ||
        cudaEventCreateWithFlags(&t->evSide, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&t->evSideDone, cudaEventDisableTiming) != cudaSuccess)
        return PKV_ERR_CUDA;
    t->S_T_async = t->next_async = 0;
    if (cudaStreamCreateWithPriority(&t->fast, cudaStreamNonBlocking, greatest) != cudaSuccess) return PKV_ERR_CUDA;
    for (cudaEvent_t& e : t->evq)
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return PKV_ERR_CUDA;
    return PKV_OK;
}
void tc_destroy(TcBuffers* t) {
    if (t->side) {
        cudaStreamSynchronize(t->side);
        cudaStreamDestroy(t->side);
        t->side = nullptr;
    }
    if (t->fast) {
        cudaStreamSynchronize(t->fast);
        cudaStreamDestroy(t->fast);
        t->fast = nullptr;
    }
    for (cudaEvent_t& e : t->evq)
        if (e) { cudaEventDestroy(e); e = nullptr; }
    for (cudaEvent_t& e : t->tr)
        if (e) { cudaEventDestroy(e); e = nullptr; }
    if (t->evSide) { cudaEventDestroy(t->evSide); t->evSide = nullptr; }
    if (t->evSideDone) { cudaEventDestroy(t->evSideDone); t->evSideDone = nullptr; }
    tc_solve_destroy(&t->solve);
    if (t->dual_enabled) tc_solve_destroy(&t->dual);
}

// in [rows][cols] fp32 -> out [cols][ldo] fp32
__global__ void k_transpose_ld(const float* __restrict__ in, int rows, int cols, int ldo, float* __restrict__ out) {
    __shared__ float t[32][33];
    int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (int j = threadIdx.y; j < 32; j += 8) {
        int r = r0 + j, c = c0 + threadIdx.x;
        if (r < rows && c < cols) t[j][threadIdx.x] = in[(size_t)r * cols + c];
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        int c = c0 + j, r = r0 + threadIdx.x;
        if (r < rows && c < cols) out[(size_t)c * ldo + r] = t[threadIdx.x][j];
    }
}

int tc_dual_solve(const Lc& lc, TcBuffers* t, const pkv_dims* D, int N, const float* R, float lam0, int mode,
                  float* dW, DevStatus* status) {
    const int F = D->F, d = D->d;
    const int ldn = (N + 7) / 8 * 8;
    int rc;
    // G_d = X X^T from the student features (bf16 pair, row-major: the contraction runs over F)
    if ((rc = gemm_pair_pair(lc, t->hC, F, t->hC, F, t->Gd, ldn, N, N, F, 1.f, nullptr, 0, false, status))) return rc;
    {
        dim3 grid((d + 31) / 32, (N + 31) / 32), block(32, 8);
        k_transpose_ld<<<grid, block, 0, lc.st>>>(R, N, d, ldn, t->RTf);
        lc.count();
    }
    // tr(X X^T) = tr(X^T X) and ||X X^T||_F = ||X^T X||_F: the ridge scale of Eq. 7 is the same number
    trace_fro2(lc, t->Gd, N, status, ldn);
    ridge_lambda(lc, F, lam0, mode, status);
    const bool well = tc_well_conditioned(lam0, mode);
    const bool zero_fill = (ldn != t->dual_ld_prev);
    t->dual_ld_prev = ldn;
    if ((rc = tc_ridge_solve_impl(lc, &t->dual, t->Gd, t->RTf, N, ldn, d, t->Yd, well, zero_fill, status, &t->Yp, nullptr)))
        return rc;
    // dW = Y X, contraction over the tokens: both operands token-contiguous
    TcGemm g = plain_gemm(d, F, N, dW, F, 1.f, nullptr, 0, false);
    g.A[0] = TcMat{t->Yp.hi, ldn, d, N}; g.B[0] = TcMat{t->XT.hi, t->ldT, F, N};
    g.A[1] = TcMat{t->Yp.hi, ldn, d, N}; g.B[1] = TcMat{t->XT.lo, t->ldT, F, N};
    g.A[2] = TcMat{t->Yp.lo, ldn, d, N}; g.B[2] = TcMat{t->XT.hi, t->ldT, F, N};
    g.npass = 3;
    g.out[0] = t->dW.hi; g.out[1] = t->dW.lo; g.ldo = F; g.nout = 2;     // operand of the next-state product
    return gemm_tc(lc, g, status);
}

static void mark(const TcForwardArgs& a, const Lc& lc, int stage) {
    if (a.ev) cudaEventRecord(a.ev[stage], lc.st);
}

// fp32 x fp32 statistics product from token-contiguous triples: all six passes (fp32-equivalent)
static void six_pass_stats(TcGemm& g, Pair A, const __nv_bfloat16* A3, long long arows, Pair B, const __nv_bfloat16* B3,
                           long long brows, long long ld, long long n) {
    const __nv_bfloat16* a[3] = {A.hi, A.lo, A3};
    const __nv_bfloat16* b[3] = {B.hi, B.lo, B3};
    const int ia[6] = {0, 0, 1, 0, 2, 1}, ib[6] = {0, 1, 0, 2, 0, 1};
    for (int i = 0; i < 6; ++i) {
        g.A[i] = TcMat{a[ia[i]], ld, arows, n};
        g.B[i] = TcMat{b[ib[i]], ld, brows, n};
    }
    g.npass = 6;
    g.nacc = 4;
}

// The build's own statistics (Eq. 9).  S_H is symmetric and its consumers (ridge scale, factorisation) read the
// lower triangle only, so only tiles on or below the diagonal are computed; S_T is also left as the bf16 triple the
// solver's first product reads.  precise: a small ridge coefficient amplifies the rounding of the statistics:
// triples, six passes.  The operands are the token-contiguous copies t->XT, t->RT.
static int gram_self_own(const Lc& lc, TcBuffers* t, int F, int n, float* S_H, bool precise, DevStatus* status) {
    TcGemm h = plain_gemm(F, F, n, S_H, F, 1.f, nullptr, 0, false);
    if (precise) {
        six_pass_stats(h, t->XT, t->XT3, F, t->XT, t->XT3, F, t->ldT, n);
    } else if (t->stats_f16) {
        h.A[0] = TcMat{t->XT.hi, t->ldT, F, n}; h.B[0] = TcMat{t->XT.hi, t->ldT, F, n};
        h.npass = 1;
        h.f16 = true;
        h.amax_a = t->stat; h.amax_b = t->stat;
    } else {
        h.A[0] = TcMat{t->XT.hi, t->ldT, F, n}; h.B[0] = TcMat{t->XT.hi, t->ldT, F, n};
        h.A[1] = TcMat{t->XT.hi, t->ldT, F, n}; h.B[1] = TcMat{t->XT.lo, t->ldT, F, n};
        h.A[2] = TcMat{t->XT.lo, t->ldT, F, n}; h.B[2] = TcMat{t->XT.hi, t->ldT, F, n};
        h.npass = 3;
    }
    h.lower_only = true;
    return gemm_tc(lc, h, status);
}
static int gram_cross_own(const Lc& lc, TcBuffers* t, int F, int dm, int n, float* S_T, bool precise, DevStatus* status) {
    TcGemm g = plain_gemm(dm, F, n, S_T, F, 1.f, nullptr, 0, false);
    if (precise) {
        six_pass_stats(g, t->RT, t->RT3, dm, t->XT, t->XT3, F, t->ldT, n);
    } else if (t->stats_f16) {
        g.A[0] = TcMat{t->RT.hi, t->ldT, dm, n}; g.B[0] = TcMat{t->XT.hi, t->ldT, F, n};
        g.npass = 1;
        g.f16 = true;
        g.amax_a = t->stat + 1; g.amax_b = t->stat;
    } else {
        g.A[0] = TcMat{t->RT.hi, t->ldT, dm, n}; g.B[0] = TcMat{t->XT.hi, t->ldT, F, n};
        g.A[1] = TcMat{t->RT.hi, t->ldT, dm, n}; g.B[1] = TcMat{t->XT.lo, t->ldT, F, n};
        g.A[2] = TcMat{t->RT.lo, t->ldT, dm, n}; g.B[2] = TcMat{t->XT.hi, t->ldT, F, n};
        g.npass = 3;
    }
    // the solver's first product reads two parts of S_T on the well-conditioned plan, three otherwise
    g.out[0] = t->S3[0]; g.out[1] = t->S3[1]; g.out[2] = t->S3[2]; g.ldo = F; g.nout = precise ? 3 : 2;
    const int rc = gemm_tc(lc, g, status);
    if (rc == PKV_OK) t->S3_ready = 1;
    return rc;
}

void tc_gram(const Lc& lc, TcBuffers* t, const pkv_dims* d, const float* X, const float* R, int n, float* S_H,
             float* S_T, bool accumulate, DevStatus* status, bool precise) {
    const int F = d->F, dm = d->d;
    t->S3_ready = 0;
    if (!accumulate && S_T == t->own_S_T) {
        stats_operand(lc, t, X, n, F, 0, precise);
        stats_operand(lc, t, R, n, dm, 1, precise);
        gram_self_own(lc, t, F, n, S_H, precise, status);
        gram_cross_own(lc, t, F, dm, n, S_T, precise, status);
        return;
    }
    t->stats_f16 = 0;
    transpose_split(lc, X, n, F, t->ldT, t->XT, precise ? t->XT3 : nullptr);
    transpose_split(lc, R, n, dm, t->ldT, t->RT, precise ? t->RT3 : nullptr);
    // S_H is symmetric: the tiles on and below the diagonal are computed (and, for a running sum, added to), the
    // upper part is then copied from the lower one, so that the caller still gets the full matrix
    TcGemm h = plain_gemm(F, F, n, S_H, F, 1.f, nullptr, 0, accumulate);
    TcGemm g = plain_gemm(dm, F, n, S_T, F, 1.f, nullptr, 0, accumulate);
    if (precise) {
        six_pass_stats(h, t->XT, t->XT3, F, t->XT, t->XT3, F, t->ldT, n);
        six_pass_stats(g, t->RT, t->RT3, dm, t->XT, t->XT3, F, t->ldT, n);
    } else {
        const Pair hp[2] = {t->XT, t->RT};
        TcGemm* gs[2] = {&h, &g};
        const int rows[2] = {F, dm};
        for (int i = 0; i < 2; ++i) {
            gs[i]->A[0] = TcMat{hp[i].hi, t->ldT, rows[i], n}; gs[i]->B[0] = TcMat{t->XT.hi, t->ldT, F, n};
            gs[i]->A[1] = TcMat{hp[i].hi, t->ldT, rows[i], n}; gs[i]->B[1] = TcMat{t->XT.lo, t->ldT, F, n};
            gs[i]->A[2] = TcMat{hp[i].lo, t->ldT, rows[i], n}; gs[i]->B[2] = TcMat{t->XT.hi, t->ldT, F, n};
            gs[i]->npass = 3;
        }
    }
    h.lower_only = true;
    gemm_tc(lc, h, status);
    symmetric_from_lower(lc, S_H, S_H, F);
    gemm_tc(lc, g, status);
}

static bool side_stream_on() {
    static const bool v = [] { const char* e = getenv("PKV_SIDE_STREAM"); return !e || atoi(e) != 0; }();
    return v;
}

// S6 (targets, Eq. 5) and S7 (statistics, Eq. 9) at the end of a forward.  Only S_H is needed to start the
// factorisation, so where the build's own solve follows (not the dual form, not a streamed accumulation, no stage
// marks) the caller's stream makes the student features' token-contiguous copy and S_H, and everything that involves
// the targets - T = dh Wdown^T + dz, its norm, its copy, S_T - goes to the side stream: the solve picks it up at its
// last two products.
static int targets_and_stats(const Lc& lc, TcBuffers* t, const pkv_dims* D, const TcForwardArgs& a, bool accumulate) {
    const int N = a.N, d = D->d, F = D->F;
    DevStatus* st = a.status;
    const bool precise = a.precise_stats != 0;
    int rc;
    t->own_S_T = a.S_T;
    if (!side_stream_on() || !t->side || a.ev || a.dual || accumulate) {
        if ((rc = gemm_act_weight(lc, t->dh, F, a.w->Wdown, F, a.R, d, N, d, F, 1.f, a.dz, d, st))) return rc;
        sumsq(lc, a.R, (int64_t)N * d, &st->t_fro2);
        mark(a, lc, 6);
        if (a.dual) transpose_split(lc, a.hC, N, F, t->ldT, t->XT);
        else tc_gram(lc, t, D, a.hC, a.R, N, a.S_H, a.S_T, accumulate, st, precise);
        mark(a, lc, 7);
        return PKV_OK;
    }
    t->S3_ready = 0;
    stats_operand(lc, t, a.hC, N, F, 0, precise);
    cudaEventRecord(t->evSide, lc.st);
    cudaStreamWaitEvent(t->side, t->evSide, 0);
    const Lc ls{t->side, lc.launches, lc.map_cache};
    rc = gemm_act_weight(ls, t->dh, F, a.w->Wdown, F, a.R, d, N, d, F, 1.f, a.dz, d, st);
    if (rc == PKV_OK) {
        sumsq(ls, a.R, (int64_t)N * d, &st->t_fro2);
        stats_operand(ls, t, a.R, N, d, 1, precise);
        rc = gram_cross_own(ls, t, F, d, N, a.S_T, precise, st);
    }
    // recorded in every case, so that the solve's wait ends
    cudaEventRecord(t->solve.st_ready, t->side);
    t->S_T_async = 1;
    t->next_async = 0;
    if (rc != PKV_OK) return rc;
    return gram_self_own(lc, t, F, N, a.S_H, precise, st);
}

bool tc_teacher_next_async(const Lc& lc, TcBuffers* t, const pkv_dims* D, int N, const void* Wdown, const float* zF,
                           float* xF_next, DevStatus* status) {
    if (!t->S_T_async) return false;
    const Lc ls{t->side, lc.launches, lc.map_cache};
    cudaStreamWaitEvent(t->side, t->solve.st_ready, 0);      // the teacher half may have run on another stream
    gemm_act_weight(ls, t->hF, D->F, Wdown, D->F, xF_next, D->d, N, D->d, D->F, 1.f, zF, D->d, status);
    cudaEventRecord(t->evSideDone, t->side);
    t->next_async = 1;
    return true;
}

static bool build_trace_on() {
    static const bool v = getenv("PKV_BUILD_TRACE") != nullptr;
    return v;
}
void tc_build_trace_mark(TcBuffers* t, int i, cudaStream_t st) {
    if (!build_trace_on()) return;
    if (!t->tr[0])
        for (cudaEvent_t& e : t->tr) cudaEventCreate(&e);
    cudaEventRecord(t->tr[i], st);
}
void tc_build_trace_print(TcBuffers* t) {
    if (!build_trace_on() || !t->tr[0]) return;
    float ms[6] = {};
    for (int i = 1; i < 6; ++i)
        if (cudaEventElapsedTime(&ms[i], t->tr[0], t->tr[i]) != cudaSuccess) { cudaGetLastError(); ms[i] = -1.f; }
    fprintf(stderr, "build timeline (ms from the start): S_H %.3f | teacher attention %.3f | S_T %.3f | solve %.3f | end %.3f\n",
            ms[1], ms[2], ms[3], ms[4], ms[5]);
}

void tc_side_quiesce(TcBuffers* t) {
    if (t->fast) cudaStreamSynchronize(t->fast);
    if (t->side) cudaStreamSynchronize(t->side);
    t->S_T_async = t->next_async = 0;
}

void tc_side_join(const Lc& lc, TcBuffers* t) {
    if (t->next_async) cudaStreamWaitEvent(lc.st, t->evSideDone, 0);
    t->next_async = 0;
}

// The statistics of Eq. 9 with caller-supplied operand buffers (used by the entry point that owns a
// fixed device array instead of a context workspace).
int tc_gram_with_buffers(const Lc& lc, Pair XT, Pair RT, int ldT, const float* X, const float* R, int n, int F, int dm,
                         float* S_H, float* S_T, bool accumulate, DevStatus* status) {
    transpose_split(lc, X, n, F, ldT, XT);
    transpose_split(lc, R, n, dm, ldT, RT);
    int rc = gemm_pair_pair(lc, XT, ldT, XT, ldT, S_H, F, F, F, n, 1.f, nullptr, 0, accumulate, status);
    if (rc != PKV_OK) return rc;
    return gemm_pair_pair(lc, RT, ldT, XT, ldT, S_T, F, dm, F, n, 1.f, nullptr, 0, accumulate, status);
}

int tc_attention(const Lc& lc, TcBuffers* t, const pkv_dims* d, const AttnArgs& a, DevStatus* status) {
    return attention_tc(lc, t, d, a, nullptr, status);
}

void tc_ridge_solve(const Lc& lc, TcBuffers* t, float* S, const float* S_T, int F, int d, float* dW, float lam0,
                    int mode, DevStatus* status) {
    const bool well = tc_well_conditioned(lam0, mode);
    tc_ridge_solve_impl(lc, &t->solve, S, S_T, F, F, d, dW, well, false, status, &t->dW, t->S3_ready ? t->S3 : nullptr,
                        t->S_T_async != 0);
    t->S3_ready = 0;
    t->S_T_async = 0;
}

static void fill_attn(AttnArgs& at, TcBuffers* t, const pkv_dims* D, const TcForwardArgs& a, int mode) {
    const int N = a.N, hd = D->hd, Dq = D->Hq * hd, Dkv = D->Hkv * hd, QKV = Dq + 2 * Dkv;
    at.q = t->qkv; at.ldq = QKV; at.k_new = t->qkv + Dq; at.v_new = t->qkv + Dq + Dkv; at.ldkv = QKV;
    at.K = a.full->K; at.V = a.full->V; at.Kc = a.Kc; at.Vc = a.Vc; at.bias = a.bias;
    at.head_off = a.head_off; at.tok_cs = a.tok_cs;
    at.N = N; at.Hq = D->Hq; at.Hkv = D->Hkv; at.hd = hd; at.L = D->L; at.elem_bytes = 2;
    at.total_kept = a.total_kept; at.max_b = a.max_b;
    at.aF = a.aF; at.aC = a.aC; at.dA = a.dA;
    at.pair_hi = t->a.hi; at.pair_lo = t->a.lo;
    at.mode = mode;
}

// Teacher half of one block (Algorithm 1, teacher forward): it reads only xF, the block weights and the full
// cache, never a patch, and touches only the teacher halves of the stacked scratch buffers (rows [0,N),
// stream 0 of the attention operands, the teacher's split partials), so that it may run beside the student
// half / the solve of an earlier block.  Outputs: aF, zF, hF (fp32; hF also as a bf16 pair) and, if asked,
// xF_next = zF + hF W^T.  The RoPE table must already be there.
int tc_teacher_forward(const Lc& lc, TcBuffers* t, const pkv_dims* D, const TcForwardArgs& a, float* xF_next) {
    const int N = a.N, d = D->d, F = D->F, hd = D->hd;
    const int Dq = D->Hq * hd, Dkv = D->Hkv * hd, QKV = Dq + 2 * Dkv;
    const pkv_block_weights* w = a.w;
    DevStatus* st = a.status;
    int rc;
    auto markT = [&](int i) { if (a.evT) cudaEventRecord(a.evT[i], lc.st); };
    markT(0);
    k_rmsnorm_split<<<N, 256, 0, lc.st>>>(a.xF, a.xF, N, d, w->g_attn, D->eps, t->u.hi, t->u.lo, 0);
    lc.count();
    {
        const void* const Ws[3] = {w->Wq, w->Wk, w->Wv};
        const int widths[3] = {Dq, Dkv, Dkv};
        if ((rc = gemm_act_weights(lc, t->u, d, Ws, widths, 3, d, t->qkv, QKV, N, d, st))) return rc;
    }
    markT(1);
    AttnArgs at{};
    fill_attn(at, t, D, a, 1);
    if ((rc = attention_tc(lc, t, D, at, a.rope_tab, st))) return rc;
    markT(2);
    // o-projection of aF, residual
    if ((rc = gemm_act_weight(lc, t->a, Dq, w->Wo, Dq, t->o, d, N, d, Dq, 1.f, nullptr, 0, st))) return rc;
    {
        size_t n = (size_t)N * d;
        k_oproj_teacher<<<(unsigned)((n / 4 + 255) / 256), 256, 0, lc.st>>>(a.xF, t->o, n, a.zF);
        lc.count();
    }
    markT(3);
    k_rmsnorm_split<<<N, 256, 0, lc.st>>>(a.zF, a.zF, N, d, w->g_mlp, D->eps, t->u.hi, t->u.lo, 0);
    lc.count();
    {
        const void* const Ws[2] = {w->Wgate, w->Wup};
        const int widths[2] = {F, F};
        if ((rc = gemm_act_weights(lc, t->u, d, Ws, widths, 2, d, t->gu, 2 * F, N, d, st))) return rc;
    }
    {
        size_t n = (size_t)N * F;
        k_swiglu_teacher<<<(unsigned)((n / 4 + 255) / 256), 256, 0, lc.st>>>(t->gu, N, F, a.hF, t->hF);
        lc.count();
    }
    markT(4);
    if (xF_next) rc = gemm_act_weight(lc, t->hF, F, w->Wdown, F, xF_next, d, N, d, F, 1.f, a.zF, d, st);
    markT(5);
    return rc;
}

// Student half (Algorithm 1, student forward + targets + statistics), rows [N,2N) of the stacked buffers.
// Reads the teacher's aF, zF, hF.  Differences (dA, dz, dh) are formed in fp32 before any rounding.
int tc_student_forward(const Lc& lc, TcBuffers* t, const pkv_dims* D, const TcForwardArgs& a) {
    const int N = a.N, d = D->d, F = D->F, hd = D->hd;
    const int Dq = D->Hq * hd, Dkv = D->Hkv * hd, QKV = Dq + 2 * Dkv;
    const pkv_block_weights* w = a.w;
    DevStatus* st = a.status;
    int rc;
    const size_t uo = (size_t)N * d;                   // offsets of the student rows
    Pair uS{t->u.hi + uo, t->u.lo + uo};
    k_rmsnorm_split<<<N, 256, 0, lc.st>>>(a.xC, a.xC, N, d, w->g_attn, D->eps, t->u.hi, t->u.lo, N);
    lc.count();
    float* qkvS = t->qkv + (size_t)N * QKV;
    {
        const void* const Ws[3] = {w->Wq, w->Wk, w->Wv};
        const int widths[3] = {Dq, Dkv, Dkv};
        if ((rc = gemm_act_weights(lc, uS, d, Ws, widths, 3, d, qkvS, QKV, N, d, st))) return rc;
    }
    mark(a, lc, 2);
    AttnArgs at{};
    fill_attn(at, t, D, a, 2);
    if ((rc = attention_tc(lc, t, D, at, a.rope_tab, st))) return rc;
    mark(a, lc, 3);
    // o-projection of dA: dz, zC
    Pair aS{t->a.hi + (size_t)N * Dq, t->a.lo + (size_t)N * Dq};
    if ((rc = gemm_act_weight(lc, aS, Dq, w->Wo, Dq, t->o + uo, d, N, d, Dq, 1.f, nullptr, 0, st))) return rc;
    {
        size_t n = (size_t)N * d;
        k_oproj_student<<<(unsigned)((n / 4 + 255) / 256), 256, 0, lc.st>>>(a.dx, t->o, a.zF, n, a.zC, a.dz);
        lc.count();
    }
    mark(a, lc, 4);
    k_rmsnorm_split<<<N, 256, 0, lc.st>>>(a.zC, a.zC, N, d, w->g_mlp, D->eps, t->u.hi, t->u.lo, N);
    lc.count();
    float* guS = t->gu + (size_t)N * 2 * F;
    {
        const void* const Ws[2] = {w->Wgate, w->Wup};
        const int widths[2] = {F, F};
        if ((rc = gemm_act_weights(lc, uS, d, Ws, widths, 2, d, guS, 2 * F, N, d, st))) return rc;
    }
    {
        size_t n = (size_t)N * F;
        k_swiglu_student<<<(unsigned)((n / 4 + 255) / 256), 256, 0, lc.st>>>(t->gu, N, F, a.hF, a.hC, t->hC, t->dh);
        lc.count();
    }
    mark(a, lc, 5);
    // S6: T = dh Wdown^T + dz (Eq. 5); S7 (Eq. 9); the dual solver only needs the token-contiguous copy of the
    // student features
    return targets_and_stats(lc, t, D, a, false);
}

int tc_student_propagate(const Lc& lc, TcBuffers* t, const pkv_dims* D, const TcForwardArgs& a, const float* dW,
                         float* zero_nd, float* xC_next) {
    const int N = a.N, d = D->d, F = D->F, hd = D->hd;
    const int Dq = D->Hq * hd, Dkv = D->Hkv * hd, QKV = Dq + 2 * Dkv;
    const pkv_block_weights* w = a.w;
    DevStatus* st = a.status;
    int rc;
    const size_t uo = (size_t)N * d;
    Pair uS{t->u.hi + uo, t->u.lo + uo};
    // with a zero "teacher" attention output and a zero incoming state difference the student half of the
    // forward computes dA = -a', dz = -a' Wo^T and z' = x' - dz, i.e. the plain student block
    cudaMemsetAsync(a.aF, 0, (size_t)N * Dq * sizeof(float), lc.st);
    cudaMemsetAsync(zero_nd, 0, (size_t)N * d * sizeof(float), lc.st);
    k_rmsnorm_split<<<N, 256, 0, lc.st>>>(a.xC, a.xC, N, d, w->g_attn, D->eps, t->u.hi, t->u.lo, N);
    lc.count();
    float* qkvS = t->qkv + (size_t)N * QKV;
    {
        const void* const Ws[3] = {w->Wq, w->Wk, w->Wv};
        const int widths[3] = {Dq, Dkv, Dkv};
        if ((rc = gemm_act_weights(lc, uS, d, Ws, widths, 3, d, qkvS, QKV, N, d, st))) return rc;
    }
    AttnArgs at{};
    fill_attn(at, t, D, a, 2);
    if ((rc = attention_tc(lc, t, D, at, a.rope_tab, st))) return rc;
    Pair aS{t->a.hi + (size_t)N * Dq, t->a.lo + (size_t)N * Dq};
    if ((rc = gemm_act_weight(lc, aS, Dq, w->Wo, Dq, t->o + uo, d, N, d, Dq, 1.f, nullptr, 0, st))) return rc;
    {
        size_t n = (size_t)N * d;
        k_oproj_student<<<(unsigned)((n / 4 + 255) / 256), 256, 0, lc.st>>>(zero_nd, t->o, a.xC, n, a.zC, a.dz);
        lc.count();
    }
    k_rmsnorm_split<<<N, 256, 0, lc.st>>>(a.zC, a.zC, N, d, w->g_mlp, D->eps, t->u.hi, t->u.lo, N);
    lc.count();
    float* guS = t->gu + (size_t)N * 2 * F;
    {
        const void* const Ws[2] = {w->Wgate, w->Wup};
        const int widths[2] = {F, F};
        if ((rc = gemm_act_weights(lc, uS, d, Ws, widths, 2, d, guS, 2 * F, N, d, st))) return rc;
    }
    {
        size_t n = (size_t)N * F;
        k_swiglu_student<<<(unsigned)((n / 4 + 255) / 256), 256, 0, lc.st>>>(t->gu, N, F, a.hF, a.hC, t->hC, t->dh);
        lc.count();
    }
    // xC_next = z' + h' W^T + h' dW^T
    if ((rc = gemm_act_weight(lc, t->hC, F, w->Wdown, F, xC_next, d, N, d, F, 1.f, a.zC, d, st))) return rc;
    tc_split_pair(lc, dW, d, F, t->dW);
    return gemm_pair_pair(lc, t->hC, F, t->dW, F, xC_next, d, N, d, F, 1.f, nullptr, 0, true, st);
}

// One block on one stream with teacher and student fused: every product runs once on the stacked rows
// (rows [0,N) teacher, [N,2N) student) and the attention is one launch.  Fastest when nothing can overlap.
int tc_forward(const Lc& lc, TcBuffers* t, const pkv_dims* D, const TcForwardArgs& a) {
    const int N = a.N, d = D->d, F = D->F, hd = D->hd;
    const int Dq = D->Hq * hd, Dkv = D->Hkv * hd, QKV = Dq + 2 * Dkv;
    const pkv_block_weights* w = a.w;
    DevStatus* st = a.status;
    int rc;
    // S1-S2: both streams stacked, rows [0,N) teacher, [N,2N) student
    k_rmsnorm_split<<<2 * N, 256, 0, lc.st>>>(a.xF, a.xC, N, d, w->g_attn, D->eps, t->u.hi, t->u.lo, 0);
    lc.count();
    {
        const void* const Ws[3] = {w->Wq, w->Wk, w->Wv};
        const int widths[3] = {Dq, Dkv, Dkv};
        if ((rc = gemm_act_weights(lc, t->u, d, Ws, widths, 3, d, t->qkv, QKV, 2 * N, d, st))) return rc;
    }
    rope_table(lc, a.tok_cs, N, hd, a.pos0, D->rope_theta, a.rope_tab);
    mark(a, lc, 2);
    // S3
    AttnArgs at{};
    at.q = t->qkv; at.ldq = QKV; at.k_new = t->qkv + Dq; at.v_new = t->qkv + Dq + Dkv; at.ldkv = QKV;
    at.K = a.full->K; at.V = a.full->V; at.Kc = a.Kc; at.Vc = a.Vc; at.bias = a.bias;
    at.head_off = a.head_off; at.tok_cs = a.tok_cs;
    at.N = N; at.Hq = D->Hq; at.Hkv = D->Hkv; at.hd = hd; at.L = D->L; at.elem_bytes = 2;
    at.total_kept = a.total_kept; at.max_b = a.max_b;
    at.aF = a.aF; at.aC = a.aC; at.dA = a.dA;
    at.pair_hi = t->a.hi; at.pair_lo = t->a.lo;
    // the S2 outputs are not rotated yet: the operand-preparation kernel applies RoPE
    if ((rc = attention_tc(lc, t, D, at, a.rope_tab, st))) return rc;
    mark(a, lc, 3);
    // S4: [aF; dA] Wo^T, then zF, dz, zC
    if ((rc = gemm_act_weight(lc, t->a, Dq, w->Wo, Dq, t->o, d, 2 * N, d, Dq, 1.f, nullptr, 0, st))) return rc;
    oproj_epilogue(lc, a.xF, a.xC, t->o, N, d, a.zF, a.zC, a.dz);
    mark(a, lc, 4);
    // S5
    k_rmsnorm_split<<<2 * N, 256, 0, lc.st>>>(a.zF, a.zC, N, d, w->g_mlp, D->eps, t->u.hi, t->u.lo, 0);
    lc.count();
    {
        const void* const Ws[2] = {w->Wgate, w->Wup};
        const int widths[2] = {F, F};
        if ((rc = gemm_act_weights(lc, t->u, d, Ws, widths, 2, d, t->gu, 2 * F, 2 * N, d, st))) return rc;
    }
    {
        size_t n = (size_t)N * F;
        k_swiglu_split<<<(unsigned)((n / 4 + 255) / 256), 256, 0, lc.st>>>(t->gu, N, F, a.hF, a.hC, t->hF, t->hC, t->dh);
        lc.count();
    }
    mark(a, lc, 5);
    // S6: T = dh Wdown^T + dz (Eq. 5); S7 (Eq. 9)
    return targets_and_stats(lc, t, D, a, a.accumulate_stats != 0);
}

static bool build_overlap_on() {
    static const bool v = [] { const char* e = getenv("PKV_BUILD_OVERLAP"); return !e || atoi(e) != 0; }();
    return v;
}

bool tc_forward_overlapped_applies(const TcBuffers* t, const TcForwardArgs& a) {
    return side_stream_on() && build_overlap_on() && t->side && t->fast && !a.ev && !a.dual && !a.accumulate_stats;
}

// One block, student first.  The ridge solve needs S_H = H'^T H' (student only) for its long, latency-bound
// factorisation and S_T only for its last two products, and the teacher half of Algorithm 1 is about two thirds of the
// forward's work.  So: the student half and S_H run first on a high-priority stream and the caller's stream goes on to
// the solve; the teacher half, the differences, the targets (Eq. 5) and S_T (Eq. 9) run on the low-priority side stream
// in the SMs the factorisation leaves idle.  The differences are still formed in fp32 before any rounding: the
// attention combine of the teacher subtracts the student's aC, dz = (xF - xC) + dA Wo^T, the teacher's residual state
// is zF = zC + dz (so that zF - zC is dz exactly), dh = hF - hC from the two fp32 activations.
// Events: evq[0] set-up done (caller's stream -> student); evq[1] aC, evq[2] zC, evq[3] hC (student -> teacher);
// evSide token-contiguous student features; evq[4] S_H (student -> caller's stream and -> the teacher's start);
// solve.st_ready S_T.  teacher_stream is normally a stream of an SM partition, so that the teacher's long-running
// CTAs cannot occupy every SM while the factorisation's short dependent kernels wait for a slot.
int tc_forward_overlapped(const Lc& lc, TcBuffers* t, const pkv_dims* D, const TcForwardArgs& a,
                          cudaStream_t teacher_stream) {
    const int N = a.N, d = D->d, F = D->F, hd = D->hd;
    const int Dq = D->Hq * hd, Dkv = D->Hkv * hd, QKV = Dq + 2 * Dkv;
    const pkv_block_weights* w = a.w;
    DevStatus* st = a.status;
    const bool precise = a.precise_stats != 0;
    int rc;
    tc_build_trace_mark(t, 0, lc.st);
    rope_table(lc, a.tok_cs, N, hd, a.pos0, D->rope_theta, a.rope_tab);
    cudaEventRecord(t->evq[0], lc.st);
    cudaStreamWaitEvent(t->fast, t->evq[0], 0);
    cudaStream_t ts = teacher_stream ? teacher_stream : t->side;
    const Lc lf{t->fast, lc.launches, lc.map_cache}, ls{ts, lc.launches, lc.map_cache};
    const void* const Wqkv[3] = {w->Wq, w->Wk, w->Wv};
    const int wqkv[3] = {Dq, Dkv, Dkv};
    const void* const Wgu[2] = {w->Wgate, w->Wup};
    const int wgu[2] = {F, F};
    t->own_S_T = a.S_T;
    t->S3_ready = 0;

    // ---- student half (rows [N,2N) of the stacked buffers) and S_H ----
    {
        const size_t uo = (size_t)N * d;
        Pair uS{t->u.hi + uo, t->u.lo + uo};
        k_rmsnorm_split<<<N, 256, 0, lf.st>>>(a.xC, a.xC, N, d, w->g_attn, D->eps, t->u.hi, t->u.lo, N);
        lf.count();
        if ((rc = gemm_act_weights(lf, uS, d, Wqkv, wqkv, 3, d, t->qkv + (size_t)N * QKV, QKV, N, d, st))) return rc;
        AttnArgs at{};
        fill_attn(at, t, D, a, 2);
        at.student_first = 1;
        if ((rc = attention_tc(lf, t, D, at, a.rope_tab, st))) return rc;
        cudaEventRecord(t->evq[1], lf.st);
        Pair aS{t->a.hi + (size_t)N * Dq, t->a.lo + (size_t)N * Dq};
        if ((rc = gemm_act_weight(lf, aS, Dq, w->Wo, Dq, t->o + uo, d, N, d, Dq, 1.f, nullptr, 0, st))) return rc;
        k_oproj_teacher<<<(unsigned)((uo / 4 + 255) / 256), 256, 0, lf.st>>>(a.xC, t->o + uo, uo, a.zC);      // zC = xC + aC Wo^T
        lf.count();
        cudaEventRecord(t->evq[2], lf.st);
        k_rmsnorm_split<<<N, 256, 0, lf.st>>>(a.zC, a.zC, N, d, w->g_mlp, D->eps, t->u.hi, t->u.lo, N);
        lf.count();
        float* guS = t->gu + (size_t)N * 2 * F;
        if ((rc = gemm_act_weights(lf, uS, d, Wgu, wgu, 2, d, guS, 2 * F, N, d, st))) return rc;
        const size_t n = (size_t)N * F;
        k_swiglu_teacher<<<(unsigned)((n / 4 + 255) / 256), 256, 0, lf.st>>>(guS, N, F, a.hC, t->hC);
        lf.count();
        cudaEventRecord(t->evq[3], lf.st);
        stats_operand(lf, t, a.hC, N, F, 0, precise);
        cudaEventRecord(t->evSide, lf.st);
        if ((rc = gram_self_own(lf, t, F, N, a.S_H, precise, st))) return rc;
        tc_build_trace_mark(t, 1, lf.st);
        cudaEventRecord(t->evq[4], lf.st);
        cudaStreamWaitEvent(lc.st, t->evq[4], 0);
    }

    // ---- teacher half (rows [0,N)), differences, targets and S_T on the side stream ----
    {
        // not before S_H is done: whatever share of the SMs the teacher takes earlier delays the start of the solve
        cudaStreamWaitEvent(ls.st, t->evq[4], 0);
        k_rmsnorm_split<<<N, 256, 0, ls.st>>>(a.xF, a.xF, N, d, w->g_attn, D->eps, t->u.hi, t->u.lo, 0);
        ls.count();
        rc = gemm_act_weights(ls, t->u, d, Wqkv, wqkv, 3, d, t->qkv, QKV, N, d, st);
        if (rc == PKV_OK) {
            AttnArgs at{};
            fill_attn(at, t, D, a, 1);
            at.student_first = 1;
            at.combine_wait = t->evq[1];
            rc = attention_tc(ls, t, D, at, a.rope_tab, st);
            tc_build_trace_mark(t, 2, ls.st);
        }
        if (rc == PKV_OK) rc = gemm_act_weight(ls, t->a, Dq, w->Wo, Dq, t->o, d, N, d, Dq, 1.f, nullptr, 0, st);
        if (rc == PKV_OK) {
            const size_t n = (size_t)N * d;
            cudaStreamWaitEvent(ls.st, t->evq[2], 0);
            k_oproj_teacher_diff<<<(unsigned)((n / 4 + 255) / 256), 256, 0, ls.st>>>(a.xF, a.xC, a.dx, t->o, a.zC, n, a.zF, a.dz);
            ls.count();
            k_rmsnorm_split<<<N, 256, 0, ls.st>>>(a.zF, a.zF, N, d, w->g_mlp, D->eps, t->u.hi, t->u.lo, 0);
            ls.count();
            rc = gemm_act_weights(ls, t->u, d, Wgu, wgu, 2, d, t->gu, 2 * F, N, d, st);
        }
        if (rc == PKV_OK) {
            const size_t n = (size_t)N * F;
            cudaStreamWaitEvent(ls.st, t->evq[3], 0);
            k_swiglu_teacher_diff<<<(unsigned)((n / 4 + 255) / 256), 256, 0, ls.st>>>(t->gu, N, F, a.hC, a.hF, t->hF, t->dh);
            ls.count();
            // S6 (Eq. 5), S_T (Eq. 9)
            rc = gemm_act_weight(ls, t->dh, F, w->Wdown, F, a.R, d, N, d, F, 1.f, a.dz, d, st);
        }
        if (rc == PKV_OK) {
            sumsq(ls, a.R, (int64_t)N * d, &st->t_fro2);
            stats_operand(ls, t, a.R, N, d, 1, precise);
            cudaStreamWaitEvent(ls.st, t->evSide, 0);
            rc = gram_cross_own(ls, t, F, d, N, a.S_T, precise, st);
        }
        tc_build_trace_mark(t, 3, ls.st);
        // recorded in every case, so that the solve's wait ends
        cudaEventRecord(t->solve.st_ready, ls.st);
        t->S_T_async = 1;
        t->next_async = 0;
    }
    return rc;
}

void tc_next_states(const Lc& lc, TcBuffers* t, const pkv_dims* D, int N, const void* Wdown, const float* dW,
                    const float* zF, const float* R, float* xF_next, float* Dm, DevStatus* status) {
    const int d = D->d, F = D->F;
    // xF_next = zF + hF Wdown^T (skipped when the teacher half already produced it)
    if (xF_next) gemm_act_weight(lc, t->hF, F, Wdown, F, xF_next, d, N, d, F, 1.f, zF, d, status);
    // D = T - hC dW^T
    (void)dW;      // its bf16 pair was written by the solver's last product
    if (Dm) gemm_pair_pair(lc, t->hC, F, t->dW, F, Dm, d, N, d, F, -1.f, R, d, false, status);
}

}  // namespace pkv
