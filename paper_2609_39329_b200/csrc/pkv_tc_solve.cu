// Ridge solve dW = S_T (S_H + lambda I)^{-1} (Eq. 8) with the dense work on the tensor cores.
//
// fp32 quantities are carried as bf16 triples (hi, mid, lo: 24 mantissa bits) and multiplied in
// six passes (hh, hm, mh, hl, lh, mm) into fp32 tensor-memory accumulators, which reproduces an
// fp32 product to ~2^-24; the two large triangular products at the end use pairs (three passes).
//
//   1. blocked right-looking Cholesky G = L L^T, block 128: the diagonal block is factored and
//      inverted by one CTA in shared memory (k_potrf128), the panel is a GEMM with the block
//      inverse, the trailing update a GEMM on the lower triangle;
//   2. X = L^{-1} by recursive doubling from the 128-block inverses:
//      [A 0; C B]^{-1} = [A^{-1} 0; -B^{-1} C A^{-1}  B^{-1}], every level two batched GEMMs;
//   3. dW = (S_T X^T) X, two GEMMs that skip the zero tiles of the triangular factor.
#include <math.h>

#include "pkv_ptx.cuh"
#include "pkv_tc.h"

namespace pkv {

using ptx::pdl_launch_dependents;
using ptx::pdl_wait;

constexpr int PB = 128;     // Cholesky block
constexpr int SB = 16;      // sub-block inside the diagonal kernel
constexpr int LDS = PB + 1;

__device__ __forceinline__ void split3(float v, __nv_bfloat16& h, __nv_bfloat16& m, __nv_bfloat16& l) {
    h = __float2bfloat16_rn(v);
    float r1 = v - __bfloat162float(h);
    m = __float2bfloat16_rn(r1);
    l = __float2bfloat16_rn(r1 - __bfloat162float(m));
}

struct Trip {
    __nv_bfloat16* a[3];
};

// Factor the diagonal block at (k0, k0) of G = S + lambda I (lower part of S read, lambda from the
// status word added on the diagonal), invert the factor, write the
// inverse (X3) and its transpose (XT3) as bf16 triples.  A pivot that is not positive and finite is
// reported (smallest column wins) and replaced by 1 so that the call ends finite with
// PKV_ERR_NOT_PD.
//
// The block is processed in 16-column sub-steps: the 16 x 16 diagonal piece is factored by one warp
// entirely in registers (lane i holds row i, columns are exchanged with shuffles), the rows below
// it by forward substitution (one row per thread), then the trailing lower triangle is updated.
constexpr int kPotrfThreads = 1024;

// ---- warp-level TF32 tiles (mma.sync m16n8k8) in split form: each fp32 operand is the sum of three
// TF32 parts (11 + 11 + 11 significant bits) and six products (hh, hm, mh, hl, lh, mm) are accumulated in
// fp32, which reproduces the fp32 product to ~2^-24 while the shared-memory traffic is that of one
// fragment load per operand element.
__device__ __forceinline__ uint32_t to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ void split_tf32(float x, uint32_t& h, uint32_t& m, uint32_t& l) {
    h = to_tf32(x);
    const float r1 = x - __uint_as_float(h);
    m = to_tf32(r1);
    l = to_tf32(r1 - __uint_as_float(m));
}
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
// One 16 x 8 output tile: c += sum over k in [kb, ke) (multiples of 8) of A(i, k) B(k, n).
// fa(i, k) / fb(k, n) read the operands (shared memory).  Fragment ownership of lane (g = lane/4, t = lane%4):
// A: (g, t) (g+8, t) (g, t+4) (g+8, t+4);  B: (t, g) (t+4, g);  C: (g, 2t) (g, 2t+1) (g+8, 2t) (g+8, 2t+1).
// kSix: all six products (fp32-equivalent); otherwise the three leading ones (~2^-21), enough when the
// ridge keeps the system well conditioned.
template <bool kSix, typename FA, typename FB>
__device__ __forceinline__ void warp_tile_tf32(float (&c)[4], int kb, int ke, int lane, FA fa, FB fb) {
    const int g = lane >> 2, t = lane & 3;
    // independent accumulators: consecutive mma.sync do not wait on one another
    float c1[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f};
    for (int k0 = kb; k0 < ke; k0 += 8) {
        uint32_t ah[4], am[4], al[4], bh[2], bm[2], bl[2];
        split_tf32(fa(g, k0 + t), ah[0], am[0], al[0]);
        split_tf32(fa(g + 8, k0 + t), ah[1], am[1], al[1]);
        split_tf32(fa(g, k0 + t + 4), ah[2], am[2], al[2]);
        split_tf32(fa(g + 8, k0 + t + 4), ah[3], am[3], al[3]);
        split_tf32(fb(k0 + t, g), bh[0], bm[0], bl[0]);
        split_tf32(fb(k0 + t + 4, g), bh[1], bm[1], bl[1]);
        if (kSix) {
            mma_tf32(c2, al, bh);
            mma_tf32(c1, ah, bl);
            mma_tf32(c2, am, bm);
        }
        mma_tf32(c1, am, bh);
        mma_tf32(c2, ah, bm);
        mma_tf32(c, ah, bh);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) c[i] += c1[i] + c2[i];
}
template <typename FA, typename FB>
__device__ __forceinline__ void warp_tile_tf32x6(float (&c)[4], int kb, int ke, int lane, bool six, FA fa, FB fb) {
    if (six) warp_tile_tf32<true>(c, kb, ke, lane, fa, fb);
    else warp_tile_tf32<false>(c, kb, ke, lane, fa, fb);
}
constexpr int kPotrfTElems = 64 * 65;       // largest doubling temporary (one 64 x 64 block, padded)
constexpr int kPotrfSmemBytes = (2 * PB * LDS + PB + kPotrfTElems) * (int)sizeof(float);

__device__ __forceinline__ uint32_t pack_bf16(__nv_bfloat16 a, __nv_bfloat16 b) {
    return (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
}

__global__ void __launch_bounds__(kPotrfThreads) k_potrf128(const float* __restrict__ G, int n, int ld, int k0, Trip X3,
                                                            Trip XT3, int six_i, DevStatus* status) {
    const bool six = six_i != 0;
    extern __shared__ float smf[];
    float(*A)[LDS] = reinterpret_cast<float(*)[LDS]>(smf);
    float(*X)[LDS] = reinterpret_cast<float(*)[LDS]>(smf + PB * LDS);
    float* rd = smf + 2 * PB * LDS;              // [128] reciprocals of the factor's diagonal
    float* T = rd + PB;                          // doubling temporary
    pdl_launch_dependents();
    pdl_wait();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    {   // one thread reads the status word: the whole CTA takes the same branch
        __shared__ int s_skip;
        if (tid == 0) s_skip = status->code;
        __syncthreads();
        if (s_skip != 0) return;
    }
    const int nbk = min(PB, n - k0);
    const float lam = status->lam;
    // ---- load the lower part (identity outside the block's extent), lambda on the diagonal ----
    if (nbk == PB && (ld & 3) == 0) {
        constexpr int kLd = 4096 / kPotrfThreads;
        float4 v[kLd];
#pragma unroll
        for (int u = 0; u < kLd; ++u) {
            const int i = tid + u * kPotrfThreads;           // 4096 float4 of the block
            const int r = i >> 5, c4 = (i & 31) * 4;
            v[u] = (c4 <= r) ? *reinterpret_cast<const float4*>(G + (size_t)(k0 + r) * ld + k0 + c4)
                             : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kLd; ++u) {
            const int i = tid + u * kPotrfThreads;
            const int r = i >> 5, c4 = (i & 31) * 4;
            const float e[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int c = c4 + t;
                A[r][c] = (c < r) ? e[t] : ((c == r) ? e[t] + lam : 0.f);
                X[r][c] = 0.f;
            }
        }
    } else {
        for (int i = tid; i < PB * PB; i += kPotrfThreads) {
            const int r = i >> 7, c = i & 127;
            float v = (r == c) ? 1.f : 0.f;
            if (r < nbk && c <= r) {
                v = G[(size_t)(k0 + r) * ld + k0 + c];
                if (r == c) v += lam;                     // G = S_H + lambda I is never materialised
            }
            A[r][c] = v;
            X[r][c] = 0.f;
        }
    }
    __syncthreads();
    float minpiv = INFINITY;
    int bad_col = -1;
    // 16 x 16 diagonal piece at c0, factored by warp 0 entirely in registers
    auto diag16 = [&](int c0) {
        const int li = lane & 15;            // lanes 16..31 mirror lanes 0..15 so every shuffle source is live
        float a[SB];
#pragma unroll
        for (int k = 0; k < SB; ++k) a[k] = A[c0 + li][c0 + k];
#pragma unroll
        for (int j = 0; j < SB; ++j) {
            float piv = __shfl_sync(0xffffffffu, a[j], j);
            const bool okp = (piv > 0.f) && (piv < INFINITY);
            if (!okp && bad_col < 0 && c0 + j < nbk) bad_col = c0 + j;
            piv = okp ? piv : 1.f;
            if (c0 + j < nbk) minpiv = fminf(minpiv, piv);
            float rdj = rsqrtf(piv);
            rdj = rdj * fmaf(-0.5f * piv * rdj, rdj, 1.5f);    // one Newton step: full fp32 accuracy
            const float lij = a[j] * rdj;                       // row li of column j (the pivot row gets sqrt(piv))
            a[j] = lij;
            if (lane == j) rd[c0 + j] = rdj;
#pragma unroll
            for (int k = j + 1; k < SB; ++k) {
                const float lkj = __shfl_sync(0xffffffffu, lij, k);
                a[k] = fmaf(-lij, lkj, a[k]);                  // rows above the diagonal hold unused values
            }
        }
        if (lane < SB) {
#pragma unroll
            for (int k = 0; k < SB; ++k)
                if (k <= lane) A[c0 + lane][c0 + k] = a[k];
        }
    };
    // one 16 x 8 tile of the trailing update for the 16 columns at c0
    auto trail_tile = [&](int c0, int i0, int n0) {
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        warp_tile_tf32x6(c, 0, SB, lane, six,
                         [&](int i, int k) { return A[i0 + i][c0 + k]; },
                         [&](int k, int n) { return A[n0 + n][c0 + k]; });
        const int g = lane >> 2, t = lane & 3;
        A[i0 + g][n0 + 2 * t] -= c[0];
        A[i0 + g][n0 + 2 * t + 1] -= c[1];
        A[i0 + g + 8][n0 + 2 * t] -= c[2];
        A[i0 + g + 8][n0 + 2 * t + 1] -= c[3];
    };
    if (warp == 0) diag16(0);
    __syncthreads();
    for (int c0 = 0; c0 < PB; c0 += SB) {
        const int base = c0 + SB;
        if (tid < PB - base) {     // rows below: x L_ss^T = a by forward substitution, one row per thread
            const int r = base + tid;
            float a[SB];
#pragma unroll
            for (int c = 0; c < SB; ++c) a[c] = A[r][c0 + c];
#pragma unroll
            for (int c = 0; c < SB; ++c) {
                float x = a[c];
#pragma unroll
                for (int k = 0; k < c; ++k) x = fmaf(-a[k], A[c0 + c][c0 + k], x);
                a[c] = x * rd[c0 + c];
            }
#pragma unroll
            for (int c = 0; c < SB; ++c) A[r][c0 + c] = a[c];
        }
        __syncthreads();
        if (base < PB) {
            // trailing update of the lower triangle inside the block (16 x 8 warp tiles, K = the 16 new
            // columns).  Warp 0 takes the next diagonal piece first and factors it right away, beside the
            // other warps' tiles: the serial pivot chain is off the critical path.
            if (warp == 0) {
                trail_tile(c0, base, base);
                trail_tile(c0, base, base + 8);
                __syncwarp();
                diag16(base);
            } else {
                const int rem = PB - base;
                const int tm = (rem >> 4) - 1, tn = rem >> 3;          // row tiles below the first one
                for (int tile = warp - 1; tile < tm * tn; tile += kPotrfThreads / 32 - 1) {
                    const int i0 = base + 16 + (tile / tn) * 16, n0 = base + (tile % tn) * 8;
                    if (n0 > i0 + 15) continue;                     // entirely above the diagonal
                    trail_tile(c0, i0, n0);
                }
            }
        }
        __syncthreads();
    }
    if (tid == 0) {
        status->min_pivot = fminf(status->min_pivot, minpiv);
        if (bad_col >= 0) {
            atomicCAS(&status->code, 0, PKV_ERR_NOT_PD);
            unsigned long long key = (unsigned long long)(k0 + bad_col) + 1ull;
            unsigned long long old = status->bad_column;
            while (old == 0ull || key < old) {
                unsigned long long prev = atomicCAS(&status->bad_column, old, key);
                if (prev == old) break;
                old = prev;
            }
        }
    }
    // ---- inverse of the factor ----
    if (tid < PB) {      // 16 x 16 diagonal sub-blocks, one column per thread
        const int o = (tid >> 4) * SB, c = tid & 15;
        float x[SB];
#pragma unroll
        for (int i = 0; i < SB; ++i) {
            float s = (i == c) ? 1.f : 0.f;
#pragma unroll
            for (int k = 0; k < i; ++k) s = fmaf(-A[o + i][o + k], x[k], s);
            x[i] = (i < c) ? 0.f : s * rd[o + i];
        }
#pragma unroll
        for (int i = 0; i < SB; ++i) X[o + i][o + c] = x[i];
    }
    __syncthreads();
    // recursive doubling inside the block: [Xa 0; C Xb] -> bottom-left = -Xb (C Xa); every level is two
    // dense products over all pairs, done as 16 x 8 warp tiles
    for (int s = SB; s < PB; s *= 2) {
        const int lt = s + 1;
        const int tn = s >> 3, tpp = (s >> 4) * tn, ntile = (PB / (2 * s)) * tpp;
        for (int tile = warp; tile < ntile; tile += kPotrfThreads / 32) {      // T_p = C_p Xa_p
            const int p = tile / tpp, i0 = ((tile % tpp) / tn) * 16, n0 = ((tile % tpp) % tn) * 8;
            const int o = 2 * p * s;
            float c[4] = {0.f, 0.f, 0.f, 0.f};
            warp_tile_tf32x6(c, n0, s, lane, six,                  // Xa is lower triangular: rows k >= column n
                             [&](int i, int k) { return A[o + s + i0 + i][o + k]; },
                             [&](int k, int n) { return X[o + k][o + n0 + n]; });
            const int g = lane >> 2, t = lane & 3;
            float* tp = T + (p * s + i0 + g) * lt + n0 + 2 * t;
            tp[0] = c[0]; tp[1] = c[1];
            tp[8 * lt] = c[2]; tp[8 * lt + 1] = c[3];
        }
        __syncthreads();
        for (int tile = warp; tile < ntile; tile += kPotrfThreads / 32) {      // X_p(bottom-left) = -Xb_p T_p
            const int p = tile / tpp, i0 = ((tile % tpp) / tn) * 16, n0 = ((tile % tpp) % tn) * 8;
            const int o = 2 * p * s;
            float c[4] = {0.f, 0.f, 0.f, 0.f};
            warp_tile_tf32x6(c, 0, i0 + 16, lane, six,             // Xb is lower triangular: columns k <= row
                             [&](int i, int k) { return X[o + s + i0 + i][o + s + k]; },
                             [&](int k, int n) { return T[(p * s + k) * lt + n0 + n]; });
            const int g = lane >> 2, t = lane & 3;
            X[o + s + i0 + g][o + n0 + 2 * t] = -c[0];
            X[o + s + i0 + g][o + n0 + 2 * t + 1] = -c[1];
            X[o + s + i0 + g + 8][o + n0 + 2 * t] = -c[2];
            X[o + s + i0 + g + 8][o + n0 + 2 * t + 1] = -c[3];
        }
        __syncthreads();
    }
    // ---- write the inverse and its transpose as bf16 triples, two columns per thread ----
    for (int i = tid; i < PB * PB / 2; i += kPotrfThreads) {
        const int r = i >> 6, c = (i & 63) * 2;
        if (r < nbk && c < nbk) {
            const size_t o = (size_t)(k0 + r) * ld + k0 + c;
            __nv_bfloat16 h0, m0, l0, h1, m1, l1;
            split3((c <= r) ? X[r][c] : 0.f, h0, m0, l0);
            split3((c + 1 <= r) ? X[r][c + 1] : 0.f, h1, m1, l1);
            if (c + 1 < nbk) {
                *reinterpret_cast<uint32_t*>(X3.a[0] + o) = pack_bf16(h0, h1);
                *reinterpret_cast<uint32_t*>(X3.a[1] + o) = pack_bf16(m0, m1);
                *reinterpret_cast<uint32_t*>(X3.a[2] + o) = pack_bf16(l0, l1);
            } else {
                X3.a[0][o] = h0; X3.a[1][o] = m0; X3.a[2][o] = l0;
            }
            split3((r <= c) ? X[c][r] : 0.f, h0, m0, l0);
            split3((r <= c + 1) ? X[c + 1][r] : 0.f, h1, m1, l1);
            if (c + 1 < nbk) {
                *reinterpret_cast<uint32_t*>(XT3.a[0] + o) = pack_bf16(h0, h1);
                *reinterpret_cast<uint32_t*>(XT3.a[1] + o) = pack_bf16(m0, m1);
                *reinterpret_cast<uint32_t*>(XT3.a[2] + o) = pack_bf16(l0, l1);
            } else {
                XT3.a[0][o] = h0; XT3.a[1][o] = m0; XT3.a[2][o] = l0;
            }
        }
    }
}

// src [rows][cols] fp32 (row stride lds) -> bf16 triple, row stride ldo
__global__ void __launch_bounds__(256) k_split3(const float* __restrict__ src, long long lds, int rows, int cols,
                                                Trip out, long long ldo, int nout) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)rows * cols) return;
    const int r = (int)(i / cols), c = (int)(i % cols);
    __nv_bfloat16 h, m, l;
    split3(src[(size_t)r * lds + c], h, m, l);
    const size_t o = (size_t)r * ldo + c;
    out.a[0][o] = h;
    out.a[1][o] = m;
    if (nout > 2) out.a[2][o] = l;
}

static void launch_split3(const Lc& lc, const float* src, long long lds, int rows, int cols, Trip out, long long ldo,
                          int nout) {
    size_t n = (size_t)rows * cols;
    if (!n) return;
    k_split3<<<(unsigned)((n + 255) / 256), 256, 0, lc.st>>>(src, lds, rows, cols, out, ldo, nout);
    lc.count();
}

// XT3[2sz + c][s + 2sz + r] = X3[s + 2sz + r][2sz + c]   (r < s clipped to the n x n matrix, c < s); row stride ld
__global__ void k_transpose_blocks(Trip X3, Trip XT3, int n, int ld, int s) {
    __shared__ __nv_bfloat16 t[3][32][33];
    const int z = blockIdx.z;
    const int r0 = s + 2 * s * z + blockIdx.y * 32, c0 = 2 * s * z + blockIdx.x * 32;
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int r = r0 + j, c = c0 + threadIdx.x;
        if (r < n) {
#pragma unroll
            for (int a = 0; a < 3; ++a) t[a][j][threadIdx.x] = X3.a[a][(size_t)r * ld + c];
        }
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int c = c0 + j, r = r0 + threadIdx.x;
        if (r < n) {
#pragma unroll
            for (int a = 0; a < 3; ++a) XT3.a[a][(size_t)c * ld + r] = t[a][threadIdx.x][j];
        }
    }
}

static void six_pass(TcGemm& g, const Trip& A, long long lda, long long arows, long long acols, const Trip& B,
                     long long ldb, long long brows, long long bcols) {
    // (hi,hi) (hi,mid) (mid,hi) (hi,lo) (lo,hi) (mid,mid)
    const int ia[6] = {0, 0, 1, 0, 2, 1}, ib[6] = {0, 1, 0, 2, 0, 1};
    for (int i = 0; i < 6; ++i) {
        g.A[i] = TcMat{A.a[ia[i]], lda, arows, acols};
        g.B[i] = TcMat{B.a[ib[i]], ldb, brows, bcols};
    }
    g.npass = 6;
    g.nacc = 4;      // fp32-equivalent products: hi x hi accumulated apart, in three parts
}

static void three_pass(TcGemm& g, const Trip& A, long long lda, long long arows, long long acols, const Trip& B,
                       long long ldb, long long brows, long long bcols) {
    const int ia[3] = {0, 0, 1}, ib[3] = {0, 1, 0};
    for (int i = 0; i < 3; ++i) {
        g.A[i] = TcMat{A.a[ia[i]], lda, arows, acols};
        g.B[i] = TcMat{B.a[ib[i]], ldb, brows, bcols};
    }
    g.npass = 3;
    g.nacc = 2;
}

// C [M][N] (+)= alpha * A B^T for fp32 A [M][K], B [N][K]: both are split into bf16 parts in the solver's S_T / Z
// operand buffers (so M*K8 and N*K8 must fit in d*F elements, K8 = K rounded up to 8) and multiplied in `passes`
// tensor-core passes (6: triples, fp32-equivalent; 3: pairs).  The building block of the factorisation,
// exported for unit tests.
int tc_fp32_product(const Lc& lc, TcSolveBuffers* t, size_t cap_elems, const float* A, const float* B, int M, int N,
                    int K, float alpha, float* C, bool accumulate, int passes, int nacc, DevStatus* status) {
    const long long K8 = (K + 7) / 8 * 8;
    if ((size_t)M * K8 > cap_elems || (size_t)N * K8 > cap_elems) return PKV_ERR_UNSUPPORTED;
    if (passes != 3 && passes != 6) return PKV_ERR_INVALID_ARG;
    Trip A3{{t->S2[0], t->S2[1], t->S2[2]}}, B3{{t->Z2[0], t->Z2[1], t->Z2[2]}};
    if (K8 != K) {
        for (int i = 0; i < 3; ++i) {
            cudaMemsetAsync(A3.a[i], 0, (size_t)M * K8 * 2, lc.st);
            cudaMemsetAsync(B3.a[i], 0, (size_t)N * K8 * 2, lc.st);
        }
    }
    launch_split3(lc, A, K, M, K, A3, K8, 3);
    launch_split3(lc, B, K, N, K, B3, K8, 3);
    TcGemm g{};
    if (passes == 6) six_pass(g, A3, K8, M, K, B3, K8, N, K);
    else three_pass(g, A3, K8, M, K, B3, K8, N, K);
    g.M = M; g.N = N; g.K = K; g.batch = 1; g.alpha = alpha;
    g.C = C; g.ldc = N; g.c_rows = M; g.c_cols = N; g.accumulate = accumulate;
    g.nacc = nacc;
    return gemm_tc(lc, g, status);
}

// largest pairs * s * s over the doubling levels (elements of the TT workspace)
static size_t tt_elems(int F) {
    size_t best = (size_t)PB * PB;
    for (long long s = PB; s < F; s *= 2) {
        long long P = 0;
        while ((2 * P + 1) * s < F) ++P;
        if ((size_t)(P * s * s) > best) best = (size_t)(P * s * s);
    }
    return best;
}

size_t tc_solve_carve(TcSolveBuffers* t, char* base, size_t off, int nmax, int dmax) {
    const size_t F = (size_t)nmax, dm = (size_t)dmax;
    t->nmax = nmax;
    auto take = [&](size_t bytes) {
        off = (off + 255) & ~(size_t)255;
        char* p = base ? base + off : nullptr;
        off += bytes;
        return p;
    };
    for (int i = 0; i < 3; ++i) {
        t->L3[i] = (__nv_bfloat16*)take(F * F * 2);
        t->X3[i] = (__nv_bfloat16*)take(F * F * 2);
        t->XT3[i] = (__nv_bfloat16*)take(F * F * 2);
        t->P3[i] = (__nv_bfloat16*)take(F * PB * 2);
        t->TT3[i] = (__nv_bfloat16*)take(tt_elems((int)F) * 2);
    }
    for (int i = 0; i < 3; ++i) {
        t->S2[i] = (__nv_bfloat16*)take(dm * F * 2);
        t->Z2[i] = (__nv_bfloat16*)take(dm * F * 2);
    }
    return off;
}

int tc_solve_init(TcSolveBuffers* t) {
    // regions of the triangular factors that no kernel writes must read as zero
    const size_t F = (size_t)t->nmax;
    for (int i = 0; i < 3; ++i) {
        if (cudaMemset(t->X3[i], 0, F * F * 2) != cudaSuccess) return PKV_ERR_CUDA;
        if (cudaMemset(t->XT3[i], 0, F * F * 2) != cudaSuccess) return PKV_ERR_CUDA;
        if (cudaMemset(t->L3[i], 0, F * F * 2) != cudaSuccess) return PKV_ERR_CUDA;
        if (cudaMemset(t->P3[i], 0, F * PB * 2) != cudaSuccess) return PKV_ERR_CUDA;
        if (cudaMemset(t->TT3[i], 0, tt_elems((int)F) * 2) != cudaSuccess) return PKV_ERR_CUDA;
    }
    int least = 0, greatest = 0;
    cudaDeviceGetStreamPriorityRange(&least, &greatest);
    // the factorisation's critical chain (diagonal block, panel, next-column update) runs at the highest
    // priority so that its small kernels are not queued behind the bulk trailing update's CTAs
    if (cudaStreamCreateWithPriority(&t->aux, cudaStreamNonBlocking, greatest) != cudaSuccess) return PKV_ERR_CUDA;
    for (int i = 0; i < 3; ++i)
        if (cudaEventCreateWithFlags(&t->ev[i], cudaEventDisableTiming) != cudaSuccess) return PKV_ERR_CUDA;
    static PerDeviceOnce once;
    int dev;
    if (once.needed(&dev)) {
        if (cudaFuncSetAttribute(k_potrf128, cudaFuncAttributeMaxDynamicSharedMemorySize, kPotrfSmemBytes) != cudaSuccess)
            return PKV_ERR_CUDA;
        once.mark(dev);
    }
    return PKV_OK;
}

void tc_solve_destroy(TcSolveBuffers* t) {
    if (t->aux) {
        cudaStreamSynchronize(t->aux);
        cudaStreamDestroy(t->aux);
        t->aux = nullptr;
    }
    for (int i = 0; i < 3; ++i)
        if (t->ev[i]) {
            cudaEventDestroy(t->ev[i]);
            t->ev[i] = nullptr;
        }
}

static void launch_potrf(cudaStream_t st, int smem, const float* G, int n, int ld, int k0, Trip X3, Trip XT3, int six,
                         DevStatus* status) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(kPotrfThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, k_potrf128, G, n, ld, k0, X3, XT3, six, status);
}

int tc_ridge_solve_impl(const Lc& lc, TcSolveBuffers* t, const float* G, const float* S_T, int n, int ld, int d,
                        float* dW, bool well_conditioned, bool zero_fill, DevStatus* status, const Pair* dW_pair,
                        __nv_bfloat16* const* S_T_triple) {
    const int F = n;      // dimension of the system; ld is the row stride of G, S_T, dW and of every n x n work array
    const int nblk = (F + PB - 1) / PB;
    const int smem = kPotrfSmemBytes;
    Trip L3{{t->L3[0], t->L3[1], t->L3[2]}}, X3{{t->X3[0], t->X3[1], t->X3[2]}}, XT3{{t->XT3[0], t->XT3[1], t->XT3[2]}};
    Trip P3{{t->P3[0], t->P3[1], t->P3[2]}}, TT3{{t->TT3[0], t->TT3[1], t->TT3[2]}};
    int rc;
    if (zero_fill) {
        // the row stride changed since the last call: parts of X / X^T that no kernel writes must read as zero
        for (int i = 0; i < 3; ++i) {
            cudaMemsetAsync(t->X3[i], 0, (size_t)n * ld * 2, lc.st);
            cudaMemsetAsync(t->XT3[i], 0, (size_t)n * ld * 2, lc.st);
        }
    }
    // ---- 1. factorisation with look-ahead ----
    // Per block column b:  panel N_b (L21 = G21 L11^{-T});  T1_b = update of the next block column only
    // (its epilogue also leaves the bf16 triple of the updated column in P3, the next panel's operand);
    // T2_b = update of everything to the right, on the helper stream, beside the next diagonal block.
    // sA: critical chain on the high-priority helper stream; sB: bulk updates on the caller's stream
    cudaStream_t sA = t->aux, sB = lc.st;
    Lc lcA{sA, lc.launches, lc.map_cache, true};
    Lc lcB{sB, lc.launches, lc.map_cache};
    cudaEventRecord(t->ev[2], sB);
    cudaStreamWaitEvent(sA, t->ev[2], 0);
    launch_potrf(sA, smem, G, n, ld, 0, X3, XT3, well_conditioned ? 0 : 1, status);
    lc.count();
    if (F > PB) launch_split3(lcA, G + (size_t)PB * ld, ld, F - PB, PB, Trip{{P3.a[0] + (size_t)PB * PB, P3.a[1] + (size_t)PB * PB, P3.a[2] + (size_t)PB * PB}}, PB, 3);
    bool t2_pending = false;
    rc = PKV_OK;
    for (int b = 0; b < nblk && rc == PKV_OK; ++b) {
        const int k0 = b * PB, k1 = min(F, k0 + PB), rem = F - k1;
        if (rem <= 0) break;
        {   // N_b: panel, kept as a bf16 triple in L3
            TcGemm g{};
            six_pass(g, P3, PB, F, PB, X3, ld, F, F);
            g.a_row0 = k1;
            g.b_row0 = k0; g.b_col0 = k0;
            g.M = rem; g.N = PB; g.K = PB; g.batch = 1; g.alpha = 1.f;
            g.c_row0 = k1; g.c_col0 = k0; g.c_rows = F; g.c_cols = F;
            g.out[0] = L3.a[0]; g.out[1] = L3.a[1]; g.out[2] = L3.a[2]; g.ldo = ld; g.nout = 3;
            if ((rc = gemm_tc(lcA, g, status))) break;
        }
        cudaEventRecord(t->ev[0], sA);
        cudaStreamWaitEvent(sB, t->ev[0], 0);
        if (t2_pending) cudaStreamWaitEvent(sA, t->ev[1], 0);      // T2_{b-1} also updated this column
        {   // T1_b: next block column of G22 -= L21 L21^T, and its bf16 triple for the next panel
            TcGemm g{};
            six_pass(g, L3, ld, F, F, L3, ld, F, F);
            g.a_row0 = k1; g.a_col0 = k0; g.b_row0 = k1; g.b_col0 = k0;
            g.M = rem; g.N = min(PB, rem); g.K = PB; g.batch = 1; g.alpha = -1.f;
            g.C = const_cast<float*>(G); g.ldc = ld; g.accumulate = true;
            g.c_row0 = k1; g.c_col0 = k1; g.c_rows = F; g.c_cols = F;
            g.out[0] = P3.a[0]; g.out[1] = P3.a[1]; g.out[2] = P3.a[2]; g.ldo = PB; g.nout = 3; g.out_col_off = k1;
            if ((rc = gemm_tc(lcA, g, status))) break;
        }
        const int rem2 = rem - PB;
        if (rem2 > 0) {   // T2_b on the helper stream
            TcGemm g{};
            six_pass(g, L3, ld, F, F, L3, ld, F, F);
            g.a_row0 = k1 + PB; g.a_col0 = k0; g.b_row0 = k1 + PB; g.b_col0 = k0;
            g.M = rem2; g.N = rem2; g.K = PB; g.batch = 1; g.alpha = -1.f;
            g.C = const_cast<float*>(G); g.ldc = ld; g.accumulate = true; g.lower_only = true;
            g.c_row0 = k1 + PB; g.c_col0 = k1 + PB; g.c_rows = F; g.c_cols = F;
            if ((rc = gemm_tc(lcB, g, status))) break;
            cudaEventRecord(t->ev[1], sB);
            t2_pending = true;
        } else {
            t2_pending = false;
        }
        launch_potrf(sA, smem, G, n, ld, k1, X3, XT3, well_conditioned ? 0 : 1, status);
        lc.count();
    }
    // join: the caller's stream continues after the chain's last kernel
    cudaEventRecord(t->ev[0], sA);
    cudaStreamWaitEvent(sB, t->ev[0], 0);
    if (rc != PKV_OK) return rc;
    // ---- 2. X = L^{-1} by recursive doubling ----
    for (int s = PB; s < F; s *= 2) {
        int P = 0;
        while ((2 * P + 1) * s < F) ++P;
        if (P == 0) break;
        {   // TT_p = A_p^{-T} C_p^T   (A^{-1} the finished top-left inverse, C the block of L below it)
            TcGemm g{};
            six_pass(g, XT3, ld, F, F, L3, ld, F, F);
            g.a_zrow = 2 * s; g.a_zcol = 2 * s;
            g.b_row0 = s; g.b_zrow = 2 * s; g.b_zcol = 2 * s;
            g.M = s; g.N = s; g.K = s; g.batch = P; g.alpha = 1.f;
            g.c_zrow = s; g.c_rows = P * s; g.c_cols = s;
            g.out[0] = TT3.a[0]; g.out[1] = TT3.a[1]; g.out[2] = TT3.a[2]; g.ldo = s; g.nout = 3;
            if ((rc = gemm_tc(lc, g, status))) return rc;
        }
        {   // X_p(bottom-left) = -B_p^{-1} TT_p^T
            TcGemm g{};
            six_pass(g, X3, ld, F, F, TT3, s, (long long)P * s, s);
            g.a_row0 = s; g.a_col0 = s; g.a_zrow = 2 * s; g.a_zcol = 2 * s;
            g.b_zrow = s;
            g.M = s; g.N = s; g.K = s; g.batch = P; g.alpha = -1.f;
            g.c_row0 = s; g.c_zrow = 2 * s; g.c_zcol = 2 * s; g.c_rows = F; g.c_cols = F;
            g.out[0] = X3.a[0]; g.out[1] = X3.a[1]; g.out[2] = X3.a[2]; g.ldo = ld; g.nout = 3;
            if ((rc = gemm_tc(lc, g, status))) return rc;
        }
        dim3 grid(s / 32, s / 32, P), block(32, 8);
        k_transpose_blocks<<<grid, block, 0, lc.st>>>(X3, XT3, n, ld, s);
        lc.count();
    }
    // ---- 3. dW = (S_T X^T) X ----
    // The rounding of these two products is amplified by cond(L): pairs (2^-16, three passes) when
    // the ridge keeps G well conditioned, triples (2^-24, six passes) otherwise.
    const int nsp = well_conditioned ? 2 : 3;
    Trip S2{{t->S2[0], t->S2[1], t->S2[2]}}, Z2{{t->Z2[0], t->Z2[1], t->Z2[2]}};
    if (!S_T_triple) launch_split3(lc, S_T, ld, d, F, S2, ld, nsp);      // else: S2 already holds the triple
    {
        TcGemm g{};
        if (nsp == 2) three_pass(g, S2, ld, d, F, X3, ld, F, F);
        else six_pass(g, S2, ld, d, F, X3, ld, F, F);
        g.M = d; g.N = F; g.K = F; g.batch = 1; g.alpha = 1.f; g.k_tri = 1;
        g.nacc = 2;      // long contraction, no cancellation: two accumulators keep two CTAs per SM
        g.c_rows = d; g.c_cols = F;
        g.out[0] = Z2.a[0]; g.out[1] = Z2.a[1]; g.out[2] = Z2.a[2]; g.ldo = ld; g.nout = nsp;
        if ((rc = gemm_tc(lc, g, status))) return rc;
    }
    {
        TcGemm g{};
        if (nsp == 2) three_pass(g, Z2, ld, d, F, XT3, ld, F, F);
        else six_pass(g, Z2, ld, d, F, XT3, ld, F, F);
        g.M = d; g.N = F; g.K = F; g.batch = 1; g.alpha = 1.f; g.k_tri = 2;
        g.nacc = 2;
        g.C = dW; g.ldc = ld; g.c_rows = d; g.c_cols = F;
        if (dW_pair) { g.out[0] = dW_pair->hi; g.out[1] = dW_pair->lo; g.ldo = ld; g.nout = 2; }
        if ((rc = gemm_tc(lc, g, status))) return rc;
    }
    return PKV_OK;
}

}  // namespace pkv
