// Ridge solve dW = S_T (S_H + lambda I)^{-1} (Eq. 8) with the dense work on the tensor cores.
//
// fp32 quantities are carried as bf16 triples (hi, mid, lo: 24 mantissa bits) and multiplied in
// six passes (hh, hm, mh, hl, lh, mm) into fp32 tensor-memory accumulators, which reproduces an
// fp32 product to ~2^-24; the two large triangular products at the end use pairs (three passes).
//
//   1. blocked right-looking Cholesky G = L L^T, block 128: one CTA per block column (k_chain128)
//      applies the previous column's update to the diagonal block, factors it and inverts the factor
//      in shared memory; the panel (a GEMM with the block inverse) and the trailing update (two GEMMs on
//      the lower triangle: the two block columns that the next steps wait for, and the rest) of every
//      column run beside that chain on two further streams;
//   2. X = L^{-1} by recursive doubling from the 128-block inverses:
//      [A 0; C B]^{-1} = [A^{-1} 0; -B^{-1} C A^{-1}  B^{-1}], two GEMMs per pair of blocks, issued on a
//      fourth stream as soon as a pair's columns are factored (only the pairs that contain the last column
//      remain after the factorisation);
//   3. dW = (S_T X^T) X, two GEMMs that skip the zero tiles of the triangular factor.
// The launches of one solve (about 260 on four streams) are captured into a CUDA graph per operand set and
// replayed, see tc_ridge_solve_impl.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>

#include "pkv_ptx.cuh"
#include <time.h>
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
constexpr int kPotrfThreads = 512;       // 16 warps: up to 128 registers per thread keep the pivot chain free of spills

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

__device__ __forceinline__ uint32_t pack_bf16(__nv_bfloat16 a, __nv_bfloat16 b) {
    return (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
}

// ---------------------------------------------------------------------------------------------
// One step of the factorisation's critical chain, one CTA:
//   L_{k,k-1} = G~_{k,k-1} inv(L_{k-1,k-1})^T                      (tensor cores, bf16 triples from global)
//   A         = G~_{kk} + lambda I - L_{k,k-1} L_{k,k-1}^T        (tensor cores; G~ updated by columns < k-1)
//   A = L_kk L_kk^T, inv(L_kk)                                     (shared memory, warp shuffles, TF32 warp tiles)
// Everything else of block column k-1 (the rest of the panel, the trailing update) runs beside this kernel
// in ordinary GEMM launches; only this kernel sits between consecutive diagonal blocks.
//
// Shared memory (dynamic, 1 KB aligned), reused by phase:
//   R1  96 KB  operand triple of G~_{k,k-1} (TMA, 128B swizzle)  ->  triple of L_{k,k-1}  ->  X (inverse, fp32) + T
//   R2  96 KB  triple of inv(L_{k-1,k-1}) (TMA)                 ->  A (fp32) + reciprocal diagonal
// Tensor memory: four 128-column accumulators (hi x hi pass in three parts, cross passes apart; see the
// note on truncating accumulation in pkv_tc_gemm.cu).
// ---------------------------------------------------------------------------------------------
struct alignas(64) ChainParams {
    CUtensorMap mP[3];        // panel operand parts  [n][128]  (rows of G~ column k-1)
    CUtensorMap mX[3];        // parts of the block-diagonal inverse [n][ld]
    const float* G;
    int n, ld, k0;
    Trip X3, XT3;
    int six;
    DevStatus* status;
    long long* stamps;        // optional [blocks][kChainStamps] clock64 marks of thread 0 (phase profile), or null
};

constexpr int kChainStamps = 18;     // 16 clock64 marks + the global timer (ns) at the kernel's start and end
constexpr int kChainR = 3 * 128 * 128 * 2;                 // 96 KB: one operand triple
constexpr int kChainBar = 2 * kChainR;
constexpr int kChainSmemBytes = kChainBar + 64 + 1024;
static_assert(PB * LDS * 4 + kPotrfTElems * 4 <= kChainR, "X and T must fit in R1");
static_assert(PB * LDS * 4 + PB * 4 <= kChainR, "A and rd must fit in R2");

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

__global__ void __launch_bounds__(kPotrfThreads) k_chain128(const __grid_constant__ ChainParams p) {
    using namespace ptx;
    const float* __restrict__ G = p.G;
    const int n = p.n, ld = p.ld, k0 = p.k0;
    const Trip X3 = p.X3, XT3 = p.XT3;
    DevStatus* status = p.status;
    const bool six = p.six != 0;
    extern __shared__ uint8_t chain_smem_raw[];
    const uint32_t raw = smem_u32(chain_smem_raw);
    const uint32_t sbase = (raw + 1023u) & ~1023u;
    uint8_t* sm = chain_smem_raw + (sbase - raw);
    float(*A)[LDS] = reinterpret_cast<float(*)[LDS]>(sm + kChainR);                 // R2
    float* rd = reinterpret_cast<float*>(sm + kChainR + PB * LDS * 4);              // [128] reciprocals of the factor's diagonal
    float(*X)[LDS] = reinterpret_cast<float(*)[LDS]>(sm);                           // R1
    float* T = reinterpret_cast<float*>(sm + PB * LDS * 4);                         // doubling temporary
    const uint32_t bar_tma = sbase + kChainBar, bar_mma = sbase + kChainBar + 8;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + kChainBar + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* skip_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool with_update = k0 > 0;
    long long* stamps = p.stamps ? p.stamps + (size_t)(k0 / PB) * kChainStamps : nullptr;
    auto stamp = [&](int i) { if (stamps && tid == 0) stamps[i] = clock64(); };
    auto wall = [&](int i) {
        if (stamps && tid == 0) {
            unsigned long long ns;
            asm volatile("mov.u64 %0, %globaltimer;" : "=l"(ns));
            stamps[i] = (long long)ns;
        }
    };
    stamp(0);
    wall(16);

    pdl_launch_dependents();
    if (tid == 0) {
        mbar_init(bar_tma, 1);
        mbar_init(bar_mma, 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1 && with_update) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = with_update ? *tmem_slot : 0u;
    pdl_wait();
    if (tid == 0) *skip_flag = status->code;      // one thread reads the status word: the whole CTA takes the same branch
    __syncthreads();
    const bool skip = *skip_flag != 0;
    stamp(1);
    const int nbk = min(PB, n - k0);
    const float lam = status->lam;
    bool ok = !skip;

    if (ok && with_update) {
        // ---- operands by TMA: parts of G~_{k,k-1} (rows k0.., the panel operand array) and of inv(L_{k-1,k-1})
        if (tid == 0) {
            mbar_expect_tx(bar_tma, 2 * kChainR);
#pragma unroll
            for (int i = 0; i < 3; ++i)
#pragma unroll
                for (int sb = 0; sb < 2; ++sb) {
                    tma_load_2d(sbase + i * 32768 + sb * 16384, &p.mP[i], bar_tma, sb * 64, k0);
                    tma_load_2d(sbase + kChainR + i * 32768 + sb * 16384, &p.mX[i], bar_tma, k0 - PB + sb * 64, k0 - PB);
                }
        }
        const int npass = six ? 6 : 3;
        const int ia[6] = {0, 0, 1, 0, 2, 1}, ib[6] = {0, 1, 0, 2, 0, 1};
        constexpr uint32_t idesc = idesc_bf16(128, 128);
        // product `which`: 0: R1 x R2^T (panel block), 1: R1 x R1^T (its Gram)
        auto issue = [&](int which) {
            uint32_t used = 0u, hh = 0u;
            for (int ps = 0; ps < npass; ++ps) {
                const uint32_t pa = sbase + ia[ps] * 32768;
                const uint32_t pb = (which == 0 ? sbase + kChainR : sbase) + ib[ps] * 32768;
                const bool big = ps == 0;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t off = (uint32_t)(kk >> 2) * 16384u;
                    const uint32_t acc = big ? 1u + (hh++ % 3u) : 0u;
                    mma_bf16_ss(tbase + acc * 128u, smem_desc_sw128(pa + off) + (uint64_t)((kk & 3) * 2),
                                smem_desc_sw128(pb + off) + (uint64_t)((kk & 3) * 2), idesc, (used >> acc) & 1u);
                    used |= 1u << acc;
                }
            }
            mma_commit(bar_mma);
        };
        if (warp == 1 && lane == 0) {
            if (mbar_wait(bar_tma, 0, abort_flag, status, 40)) {
                tc_fence_after();
                issue(0);
            }
        }
        // ---- L_{k,k-1}: accumulators -> fp32 -> bf16 triple in R1 (the operand triple there is dead once the
        //      MMAs have completed).  Warps 0..15: lane quarter = warp & 3, 32 columns each.
        const int q = warp & 3, cb = warp >> 2;
        const int row = q * 32 + lane;
        ok = mbar_wait(bar_mma, 0, abort_flag, status, 41);
        tc_fence_after();
        stamp(2);
        if (ok && warp < 16) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int c0 = cb * 32 + half * 16;
                uint32_t r[16], r2[16];
                const uint32_t ta = tbase + ((uint32_t)(q * 32) << 16) + (uint32_t)c0;
                tmem_ld16(ta, r);
                tmem_ld_wait();
#pragma unroll
                for (int a = 1; a < 4; ++a) {
                    tmem_ld16(ta + (uint32_t)(a * 128), r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
                }
                // 16 columns = two 16-byte chunks per part; chunk index inside the 64-column sub-tile is XOR-swizzled
                const int sb = c0 >> 6, ch0 = (c0 & 63) >> 3;
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    uint32_t hv[4], mv[4], lv[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        __nv_bfloat16 h0, m0, l0, h1, m1, l1;
                        const float v0 = (row < nbk) ? __uint_as_float(r[ch * 8 + 2 * e]) : 0.f;
                        const float v1 = (row < nbk) ? __uint_as_float(r[ch * 8 + 2 * e + 1]) : 0.f;
                        split3(v0, h0, m0, l0);
                        split3(v1, h1, m1, l1);
                        hv[e] = pack_bf16(h0, h1); mv[e] = pack_bf16(m0, m1); lv[e] = pack_bf16(l0, l1);
                    }
                    uint8_t* dst = sm + sb * 16384 + row * 128 + (((ch0 + ch) ^ (row & 7)) << 4);
                    *reinterpret_cast<uint4*>(dst) = make_uint4(hv[0], hv[1], hv[2], hv[3]);
                    *reinterpret_cast<uint4*>(dst + 32768) = make_uint4(mv[0], mv[1], mv[2], mv[3]);
                    *reinterpret_cast<uint4*>(dst + 65536) = make_uint4(lv[0], lv[1], lv[2], lv[3]);
                }
            }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        ok = *abort_flag == 0;
        if (ok && warp == 1 && lane == 0) issue(1);
        ok = ok && mbar_wait(bar_mma, 1, abort_flag, status, 42);
        tc_fence_after();
        stamp(3);
        // ---- A = G~_kk + lambda I - L L^T (lower part; identity outside the block's extent) into R2
        if (ok && warp < 16) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int c0 = cb * 32 + half * 16;
                float g[16];
                const bool inrow = row < nbk;
                if (nbk == PB && c0 <= row && (ld & 3) == 0) {   // 16-byte loads; entries right of the diagonal are not used
                    const float4* gp = reinterpret_cast<const float4*>(G + (size_t)(k0 + row) * ld + k0 + c0);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float4 v = (c0 + 4 * j <= row) ? gp[j] : make_float4(0.f, 0.f, 0.f, 0.f);
                        g[4 * j] = v.x; g[4 * j + 1] = v.y; g[4 * j + 2] = v.z; g[4 * j + 3] = v.w;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int c = c0 + j;
                        g[j] = (inrow && c <= row) ? G[(size_t)(k0 + row) * ld + k0 + c] : 0.f;
                    }
                }
                uint32_t r[16], r2[16];
                const uint32_t ta = tbase + ((uint32_t)(q * 32) << 16) + (uint32_t)c0;
                tmem_ld16(ta, r);
                tmem_ld_wait();
#pragma unroll
                for (int a = 1; a < 4; ++a) {
                    tmem_ld16(ta + (uint32_t)(a * 128), r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int c = c0 + j;
                    float v = (row == c) ? 1.f : 0.f;
                    if (inrow && c <= row) v = (g[j] - __uint_as_float(r[j])) + ((c == row) ? lam : 0.f);
                    A[row][c] = v;
                }
            }
        }
        // clear X (R1: the triple of L is dead, its MMAs have completed)
        if (ok)
            for (int i = tid; i < PB * PB; i += kPotrfThreads) X[i >> 7][i & 127] = 0.f;
        __syncthreads();
    } else if (ok) {
        // ---- first block: the lower part from global memory (identity outside the block's extent), lambda on the diagonal
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
        __syncthreads();
    }
    stamp(4);
    if (ok) {
    float minpiv = INFINITY;
    int bad_col = -1;
    // 16 x 16 diagonal piece at c0 in registers of warp 0: lane i (and its mirror i + 16, so that every shuffle
    // source is live) holds row i, already loaded into a[].  Four pivots per round: the 4 x 4 leading block
    // (ten values, shuffled from lanes j..j+3) is factored redundantly by every lane, so that the dependent
    // shuffle -> rsqrt -> shuffle round trip is paid four times per piece instead of sixteen.
    auto diag16 = [&](int c0, float (&a)[SB]) {
#pragma unroll
        for (int j = 0; j < SB; j += 4) {
            float p[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int cc = 0; cc <= r; ++cc) p[r][cc] = __shfl_sync(0xffffffffu, a[j + cc], j + r);
            float l[4][4], rr[4];
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                float q = p[cc][cc];
#pragma unroll
                for (int k = 0; k < cc; ++k) q = fmaf(-l[cc][k], l[cc][k], q);
                const bool okp = (q > 0.f) && (q < INFINITY);
                if (!okp && bad_col < 0 && c0 + j + cc < nbk) bad_col = c0 + j + cc;
                q = okp ? q : 1.f;
                if (c0 + j + cc < nbk) minpiv = fminf(minpiv, q);
                float rq = rsqrtf(q);
                rq = rq * fmaf(-0.5f * q * rq, rq, 1.5f);      // one Newton step: full fp32 accuracy
                rr[cc] = rq;
#pragma unroll
                for (int r = cc + 1; r < 4; ++r) {
                    float v = p[r][cc];
#pragma unroll
                    for (int k = 0; k < cc; ++k) v = fmaf(-l[r][k], l[cc][k], v);
                    l[r][cc] = v * rq;
                }
            }
            // this lane's row: columns j..j+3 of L (rows j..j+2 hold unused values right of their diagonal)
            float x[4];
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                float v = a[j + cc];
#pragma unroll
                for (int k = 0; k < cc; ++k) v = fmaf(-x[k], l[cc][k], v);
                x[cc] = v * rr[cc];
                a[j + cc] = x[cc];
            }
            if (lane == j) {
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) rd[c0 + j + cc] = rr[cc];
            }
#pragma unroll
            for (int k = j + 4; k < SB; ++k) {
                float v = a[k];
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) v = fmaf(-x[cc], __shfl_sync(0xffffffffu, x[cc], k), v);
                a[k] = v;                                       // rows above the diagonal hold unused values
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
    long long d_fs = 0, d_up = 0, d_dg = 0, d_sy = 0, tq = clock64();
    auto lap = [&](long long& acc) { if (stamps) { const long long now = clock64(); acc += now - tq; tq = now; } };
    if (warp == 0) {
        float a[SB];
#pragma unroll
        for (int k = 0; k < SB; ++k) a[k] = A[lane & 15][k];
        diag16(0, a);
    }
    __syncthreads();
    lap(d_dg);
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
        lap(d_fs);
        if (base < PB) {
            // Trailing update of the lower triangle inside the block (K = the 16 new columns).  Warp 0 owns the
            // next diagonal piece: it applies the update to that 16 x 16 block in fp32 registers (each half-warp
            // sums eight of the sixteen columns) and factors it right away, beside the other warps' tiles: the
            // serial pivot chain never waits for them.
            if (warp == 0) {
                const int li = lane & 15, kh = (lane >> 4) * 8;
                float own[8], acc[SB];
#pragma unroll
                for (int k = 0; k < 8; ++k) own[k] = A[base + li][c0 + kh + k];
#pragma unroll
                for (int m = 0; m < SB; ++m) {
                    float sacc = 0.f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) sacc = fmaf(own[k], A[base + m][c0 + kh + k], sacc);
                    acc[m] = sacc;
                }
                float a[SB];
#pragma unroll
                for (int m = 0; m < SB; ++m) {
                    acc[m] += __shfl_xor_sync(0xffffffffu, acc[m], 16);
                    a[m] = A[base + li][base + m] - acc[m];
                }
                lap(d_up);
                diag16(base, a);
                lap(d_dg);
            } else if ((warp & 3) != 0) {
                // warps 4, 8, ... share warp 0's scheduler: they stay out of the way of the pivot chain
                const int rem = PB - base;
                const int tm = (rem >> 4) - 1, tn = rem >> 3;          // row tiles below the first one
                constexpr int kWork = (kPotrfThreads / 32) - (kPotrfThreads / 128);   // warps with (warp & 3) != 0
                const int wi = warp - 1 - (warp >> 2);                  // index among the working warps
                for (int tile = wi; tile < tm * tn; tile += kWork) {
                    const int i0 = base + 16 + (tile / tn) * 16, n0 = base + (tile % tn) * 8;
                    if (n0 > i0 + 15) continue;                     // entirely above the diagonal
                    trail_tile(c0, i0, n0);
                }
            }
        }
        __syncthreads();
        lap(d_sy);
    }
    if (stamps && tid == 0) { stamps[8] = d_fs; stamps[9] = d_up; stamps[10] = d_dg; stamps[11] = d_sy; }
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
    stamp(5);
    // ---- inverse of the factor (plain fp32 FMAs: exact roundings, no operand splitting) ----
    if (tid < PB) {      // 16 x 16 diagonal sub-blocks, one column per thread
        const int o = (tid >> 4) * SB, c = tid & 15;
        float x[SB];
#pragma unroll
        for (int i = 0; i < SB; ++i) {
            float sacc = (i == c) ? 1.f : 0.f;
#pragma unroll
            for (int k = 0; k < i; ++k) sacc = fmaf(-A[o + i][o + k], x[k], sacc);
            x[i] = (i < c) ? 0.f : sacc * rd[o + i];
        }
#pragma unroll
        for (int i = 0; i < SB; ++i) X[o + i][o + c] = x[i];
    }
    __syncthreads();
    if (stamps && tid == 0) stamps[12] = clock64();
    // recursive doubling inside the block: [Xa 0; C Xb]^-1 has bottom-left -Xb (C Xa).  Every level is two
    // products over all pairs; each thread owns a 4 x 4 patch of the output.
    for (int sz = SB; sz < PB; sz *= 2) {
        const int lt = sz + 1;
        const int q4 = sz >> 2;                       // patches per side of one pair's block
        const int npatch = (PB / (2 * sz)) * q4 * q4;
        if (tid < npatch) {                           // T_p = C_p Xa_p ; Xa lower triangular: k >= n
            const int pp = tid / (q4 * q4), rest = tid % (q4 * q4);
            const int i0 = (rest % q4) * 4, n0 = (rest / q4) * 4, o = 2 * pp * sz;
            float acc[4][4] = {};
            for (int k4 = n0; k4 < sz; k4 += 4) {      // n0 and sz are multiples of 4: four steps with all loads up front
                float av[4][4], bv[4][4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
#pragma unroll
                    for (int r = 0; r < 4; ++r) av[u][r] = A[o + sz + i0 + r][o + k4 + u];
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) bv[u][cc] = X[o + k4 + u][o + n0 + cc];
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int r = 0; r < 4; ++r)
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) acc[r][cc] = fmaf(av[u][r], bv[u][cc], acc[r][cc]);
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) T[(pp * sz + i0 + r) * lt + n0 + cc] = acc[r][cc];
        }
        __syncthreads();
        if (tid < npatch) {                           // X_p(bottom-left) = -Xb_p T_p ; Xb lower triangular: k <= i
            const int pp = tid / (q4 * q4), rest = tid % (q4 * q4);
            const int i0 = (rest % q4) * 4, n0 = (rest / q4) * 4, o = 2 * pp * sz;
            float acc[4][4] = {};
            for (int k4 = 0; k4 < i0 + 4; k4 += 4) {
                float av[4][4], bv[4][4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
#pragma unroll
                    for (int r = 0; r < 4; ++r) av[u][r] = X[o + sz + i0 + r][o + sz + k4 + u];
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) bv[u][cc] = T[(pp * sz + k4 + u) * lt + n0 + cc];
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int r = 0; r < 4; ++r)
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) acc[r][cc] = fmaf(av[u][r], bv[u][cc], acc[r][cc]);
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) X[o + sz + i0 + r][o + n0 + cc] = -acc[r][cc];
        }
        __syncthreads();
        if (stamps && tid == 0) stamps[12 + (sz == 16 ? 1 : (sz == 32 ? 2 : 3))] = clock64();
    }
    stamp(6);
    // ---- write the inverse as bf16 triples, eight columns (16 bytes per part) per thread; chunks right of the
    //      diagonal stay zero (cleared once, never written).  The transposed copy is made off the chain.
    if (nbk == PB && (ld & 7) == 0) {
        for (int i = tid; i < PB * PB / 8; i += kPotrfThreads) {
            const int r = i >> 4, c8 = (i & 15) * 8;
            if (c8 > r) continue;
            const size_t o = (size_t)(k0 + r) * ld + k0 + c8;
            uint32_t hv[4], mv[4], lv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int c = c8 + 2 * e;
                const float v0 = (c <= r) ? X[r][c] : 0.f, v1 = (c + 1 <= r) ? X[r][c + 1] : 0.f;
                __nv_bfloat16 h0, m0, l0, h1, m1, l1;
                split3(v0, h0, m0, l0);
                split3(v1, h1, m1, l1);
                hv[e] = pack_bf16(h0, h1); mv[e] = pack_bf16(m0, m1); lv[e] = pack_bf16(l0, l1);
            }
            *reinterpret_cast<uint4*>(X3.a[0] + o) = make_uint4(hv[0], hv[1], hv[2], hv[3]);
            *reinterpret_cast<uint4*>(X3.a[1] + o) = make_uint4(mv[0], mv[1], mv[2], mv[3]);
            *reinterpret_cast<uint4*>(X3.a[2] + o) = make_uint4(lv[0], lv[1], lv[2], lv[3]);
        }
    } else {
        for (int i = tid; i < PB * PB; i += kPotrfThreads) {
            const int r = i >> 7, c = i & 127;
            if (r < nbk && c <= r) {
                const size_t o = (size_t)(k0 + r) * ld + k0 + c;
                __nv_bfloat16 h, m, l;
                split3(X[r][c], h, m, l);
                X3.a[0][o] = h; X3.a[1][o] = m; X3.a[2][o] = l;
            }
        }
    }
    }      // ok
    stamp(7);
    wall(17);
    // teardown: after an abort give copies in flight time to land before the CTA's smem is released
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1 && with_update) {
        tc_fence_after();
        tmem_dealloc(tbase, 512);
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

// Diagonal blocks: XT3[k0 + c][k0 + r] = X3[k0 + r][k0 + c] for the 128-blocks on the diagonal (clipped to n x n).
__global__ void k_transpose_diag(Trip X3, Trip XT3, int n, int ld, int blk0) {
    __shared__ __nv_bfloat16 t[3][32][33];
    const int k0 = (blk0 + blockIdx.z) * PB;
    const int r0 = k0 + blockIdx.y * 32, c0 = k0 + blockIdx.x * 32;
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int r = r0 + j, c = c0 + threadIdx.x;
        if (r < n && c < n) {
#pragma unroll
            for (int a = 0; a < 3; ++a) t[a][j][threadIdx.x] = X3.a[a][(size_t)r * ld + c];
        }
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int c = c0 + j, r = r0 + threadIdx.x;
        if (r < n && c < n) {
#pragma unroll
            for (int a = 0; a < 3; ++a) XT3.a[a][(size_t)c * ld + r] = t[a][threadIdx.x][j];
        }
    }
}

// XT3[2sz + c][s + 2sz + r] = X3[s + 2sz + r][2sz + c]   (r < s clipped to the n x n matrix, c < s); row stride ld
__global__ void k_transpose_blocks(Trip X3, Trip XT3, int n, int ld, int s, int pair0) {
    __shared__ __nv_bfloat16 t[3][32][33];
    const int z = pair0 + blockIdx.z;
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

void tc_split_pair(const Lc& lc, const float* src, long long rows, long long cols, Pair out) {
    launch_split3(lc, src, cols, (int)rows, (int)cols, Trip{{out.hi, out.lo, nullptr}}, cols, 2);
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
                    int K, float alpha, float* C, bool accumulate, int passes, int nacc, DevStatus* status,
                    bool b_in_factor_buffer) {
    const long long K8 = (K + 7) / 8 * 8;
    // B's parts go to the S_T X^T operand buffer, or (a square operand as large as the system) to the factor's
    // buffer, which is cleared again afterwards: parts of it that no kernel of the solve writes must read as zero
    const size_t capB = b_in_factor_buffer ? (size_t)t->nmax * t->nmax : cap_elems;
    if ((size_t)M * K8 > cap_elems || (size_t)N * K8 > capB) return PKV_ERR_UNSUPPORTED;
    if (passes != 3 && passes != 6) return PKV_ERR_INVALID_ARG;
    Trip A3{{t->S2[0], t->S2[1], t->S2[2]}}, B3{{t->Z2[0], t->Z2[1], t->Z2[2]}};
    if (b_in_factor_buffer) B3 = Trip{{t->L3[0], t->L3[1], t->L3[2]}};
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
    // PKV_GEMM_TRACE=1: phase times of the product's first CTA, and the launch-to-launch time around it
    static const bool gtrace = getenv("PKV_GEMM_TRACE") != nullptr;
    static unsigned long long* dstamps = nullptr;
    if (gtrace) {
        if (!dstamps) cudaMalloc(&dstamps, 3 * 16 * sizeof(unsigned long long));
        cudaMemsetAsync(dstamps, 0, 3 * 16 * sizeof(unsigned long long), lc.st);
        for (int rep = 0; rep < 2; ++rep) { g.stamps = dstamps + 16 * rep; gemm_tc(lc, g, status); }
        g.stamps = dstamps + 32;
    }
    const int rc = gemm_tc(lc, g, status);
    if (gtrace) {
        unsigned long long h[48];
        cudaStreamSynchronize(lc.st);
        cudaMemcpy(h, dstamps, sizeof(h), cudaMemcpyDeviceToHost);
        for (int rep = 0; rep < 3; ++rep) {
            const unsigned long long* s = h + 16 * rep;
            fprintf(stderr, "gemm %dx%dx%d passes %d acc %d, launch %d: entry +0 | dependencies met %.2f | status read %.2f | first k-tile "
                            "landed %.2f | last MMA issued %.2f | accumulator ready %.2f | epilogue done %.2f | exit %.2f us",
                    M, N, K, passes, nacc, rep, (s[1] - s[0]) * 1e-3, (s[2] - s[0]) * 1e-3, (s[3] - s[0]) * 1e-3, (s[4] - s[0]) * 1e-3,
                    (s[5] - s[0]) * 1e-3, (s[6] - s[0]) * 1e-3, (s[7] - s[0]) * 1e-3);
            if (rep > 0) fprintf(stderr, " ; entry %.2f us after the previous launch's exit", ((double)s[0] - (double)h[16 * (rep - 1) + 7]) * 1e-3);
            fprintf(stderr, " ; chunks (loaded/summed):");
            for (int c = 0; c < 8; ++c) fprintf(stderr, " %.2f", (s[8 + c] - s[0]) * 1e-3);
            fprintf(stderr, "\n");
        }
    }
    if (b_in_factor_buffer)
        for (int i = 0; i < 3; ++i) cudaMemsetAsync(t->L3[i], 0, (size_t)t->nmax * t->nmax * 2, lc.st);
    return rc;
}

// elements of the doubling's temporary TT
static size_t tt_elems(int F) {
    size_t sum = (size_t)PB * PB;       // one s x s region per doubling level s = 128, 256, ... below F
    for (long long s = PB; s < F; s *= 2) sum += (size_t)(s * s);
    return sum;
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
    t->stamps = (long long*)take(((F + PB - 1) / PB) * kChainStamps * sizeof(long long));
    t->slot = (float**)take(256);
    t->gstatus = (DevStatus*)take(256);
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
    // ... the panels and trailing updates (needed two chain steps later) below it, and the doubling levels of the
    // inverse (needed only at the end) below those, filling the SMs the others leave idle
    const int mid = (least + greatest) / 2;
    if (cudaStreamCreateWithPriority(&t->bulk, cudaStreamNonBlocking, greatest < least ? greatest + 1 : greatest) != cudaSuccess)
        return PKV_ERR_CUDA;
    if (cudaStreamCreateWithPriority(&t->bulk2, cudaStreamNonBlocking, mid) != cudaSuccess) return PKV_ERR_CUDA;
    if (cudaStreamCreateWithPriority(&t->aux2, cudaStreamNonBlocking, least) != cudaSuccess) return PKV_ERR_CUDA;
    if (cudaStreamCreateWithFlags(&t->origin, cudaStreamNonBlocking) != cudaSuccess) return PKV_ERR_CUDA;
    if (cudaEventCreateWithFlags(&t->st_ready, cudaEventDisableTiming) != cudaSuccess) return PKV_ERR_CUDA;
    t->n_graphs = 0;
    t->graph_off = 0;
    t->graph_clock = 0;
    for (int i = 0; i < kSolveEvents; ++i)
        if (cudaEventCreateWithFlags(&t->ev[i], cudaEventDisableTiming) != cudaSuccess) return PKV_ERR_CUDA;
    t->chain_n = t->chain_ld = 0;
    static PerDeviceOnce once;
    int dev;
    if (once.needed(&dev)) {
        if (cudaFuncSetAttribute(k_chain128, cudaFuncAttributeMaxDynamicSharedMemorySize, kChainSmemBytes) != cudaSuccess)
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
    for (int i = 0; i < t->n_graphs; ++i) {
        cudaGraphExecDestroy(t->graphs[i].exec);
        if (t->graphs[i].exec2) cudaGraphExecDestroy(t->graphs[i].exec2);
    }
    t->n_graphs = 0;
    for (cudaStream_t* st : {&t->origin, &t->bulk, &t->bulk2, &t->aux2})
        if (*st) {
            cudaStreamSynchronize(*st);
            cudaStreamDestroy(*st);
            *st = nullptr;
        }
    for (int i = 0; i < kSolveEvents; ++i)
        if (t->ev[i]) {
            cudaEventDestroy(t->ev[i]);
            t->ev[i] = nullptr;
        }
    if (t->st_ready) {
        cudaEventDestroy(t->st_ready);
        t->st_ready = nullptr;
    }
}

static int launch_chain(cudaStream_t st, const ChainParams& cp) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(kPotrfThreads);
    cfg.dynamicSmemBytes = kChainSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_chain128, cp) == cudaSuccess ? PKV_OK : PKV_ERR_CUDA;
}

// PKV_SOLVE_TRACE=1: launch-by-launch issue with the chain kernel's phase profile and the stream timeline;
// PKV_SOLVE_TRACE=graph: the replayed graph, with only the chain kernels' start and end times
static bool solve_trace_graph() {
    static const bool v = [] { const char* e = getenv("PKV_SOLVE_TRACE"); return e && e[0] == 'g'; }();
    return v;
}
static bool solve_trace() {
    static const bool v = getenv("PKV_SOLVE_TRACE") != nullptr && !solve_trace_graph();
    return v;
}

// The whole solve, issued from lc.st.  dW is the result's address, or, with dW_ind set, only has its alignment,
// the address being read on the device from *dW_ind (the form a captured graph replays with another destination).
static int solve_body(const Lc& lc, TcSolveBuffers* t, const float* G, const float* S_T, int n, int ld, int d,
                      float* dW, float* const* dW_ind, bool well_conditioned, bool zero_fill,
                      DevStatus* status, const Pair* dW_pair, __nv_bfloat16* const* S_T_triple, bool wait_S_T,
                      int phase = 0,        // 0: the whole solve; 1: factorisation and inverse only; 2: final products only
                      bool add_to_dW = false) {      // the last product adds to dW instead of overwriting it
    const int F = n;      // dimension of the system; ld is the row stride of G, S_T, dW and of every n x n work array
    const int nblk = (F + PB - 1) / PB;
    Trip L3{{t->L3[0], t->L3[1], t->L3[2]}}, X3{{t->X3[0], t->X3[1], t->X3[2]}}, XT3{{t->XT3[0], t->XT3[1], t->XT3[2]}};
    Trip P3{{t->P3[0], t->P3[1], t->P3[2]}}, TT3{{t->TT3[0], t->TT3[1], t->TT3[2]}};
    int rc;
    if (zero_fill && phase != 2) {
        // the row stride changed since the last call: parts of X / X^T that no kernel writes must read as zero
        for (int i = 0; i < 3; ++i) {
            cudaMemsetAsync(t->X3[i], 0, (size_t)n * ld * 2, lc.st);
            cudaMemsetAsync(t->XT3[i], 0, (size_t)n * ld * 2, lc.st);
        }
    }
    // ---- 1. factorisation ----
    // Critical chain (high-priority helper stream sA): one k_chain128 per block column, which applies column
    // k-1's update to the diagonal block itself, factors it and inverts the factor.  Beside it, on the caller's
    // stream sB, the bulk of every column: P_k = the panel L_{r,k} = G~_{r,k} inv(L_kk)^T for all rows below
    // (kept as a bf16 triple), U_k = the trailing update by column k of everything except the next diagonal
    // block (which the chain kernel does not read back from memory); U_k's first block column also leaves
    // the bf16 triple of the updated column k+1, the operand of P_{k+1} and of the next chain kernel.
    //   chain(k)  needs chain(k-1) and U_{k-2};   P_k needs chain(k) and U_{k-1};   U_k needs P_k.
    // priorities: chain (sA) > panel + first columns of the update (sB) > rest of the update (sE) > the inverse's doubling (sC)
    cudaStream_t sA = t->aux, sB = t->bulk, sE = t->bulk2;
    Lc lcB{sB, lc.launches, lc.map_cache}, lcE{sE, lc.launches, lc.map_cache};
    if (t->chain_n != n || t->chain_ld != ld) {
        for (int i = 0; i < 3; ++i) {
            if ((rc = tc_make_map_2d(&t->chainP[i], P3.a[i], F, PB, PB, 128))) return rc;
            if ((rc = tc_make_map_2d(&t->chainX[i], X3.a[i], F, F, ld, 128))) return rc;
        }
        t->chain_n = n;
        t->chain_ld = ld;
    }
    ChainParams cp;
    for (int i = 0; i < 3; ++i) { cp.mP[i] = t->chainP[i]; cp.mX[i] = t->chainX[i]; }
    cp.G = G; cp.n = n; cp.ld = ld; cp.X3 = X3; cp.XT3 = XT3; cp.six = well_conditioned ? 0 : 1; cp.status = status;
    // phase profile of the chain kernel (environment variable PKV_SOLVE_TRACE=1): clock64 marks, printed to stderr
    const bool trace = solve_trace();
    cp.stamps = (trace || solve_trace_graph()) ? t->stamps : nullptr;
    cudaEvent_t evFork = t->ev[0], evF = t->ev[1];
    cudaEvent_t evU[2] = {t->ev[2], t->ev[3]};
    cudaEvent_t evP = t->ev[4], evC = t->ev[5];
    cudaEvent_t evUb[3] = {t->ev[6], t->ev[7], t->ev[8]};
    // Third stream sC: X = L^{-1} by recursive doubling, [A 0; C B]^{-1} = [A^{-1} 0; -B^{-1} C A^{-1}  B^{-1}],
    // pair by pair as soon as a pair's columns are factored, beside the factorisation (whose panel products and
    // chain kernels leave most SMs idle); only the levels that need the last columns remain for the end.
    cudaStream_t sC = t->aux2;
    Lc lcC{sC, lc.launches, lc.map_cache};
    auto pass_plan = [&](TcGemm& g, const Trip& A, long long lda, long long ar, long long ac, const Trip& B, long long ldb,
                         long long br, long long bc) {
        if (well_conditioned) three_pass(g, A, lda, ar, ac, B, ldb, br, bc);
        else six_pass(g, A, lda, ar, ac, B, ldb, br, bc);
    };
    // Pair p of level s: rows/columns [o, o + 2s) clipped to F, o = 2 s p.  Its first product needs only the top
    // half (inverse A^{-1} and the block C of L below it) and is issued as soon as that half is factored; the
    // second one waits for the bottom-right inverse.  Every level has its own TT region (a pair's first product
    // precedes its second, and the next pair of the level starts after that).
    auto tt_level = [&](int s) {
        size_t off = 0;
        for (long long q = PB; q < s; q *= 2) off += (size_t)(q * q);
        return Trip{{TT3.a[0] + off, TT3.a[1] + off, TT3.a[2] + off}};
    };
    auto pair_first = [&](int s, int p) -> int {      // TT [s][bot] = A^{-T} C^T   (A^{-T} upper triangular: k >= row)
        const int o = 2 * s * p, bot = min(s, F - (o + s));
        const Trip TT = tt_level(s);
        TcGemm g{};
        pass_plan(g, XT3, ld, F, F, L3, ld, F, F);
        g.a_row0 = o; g.a_col0 = o; g.a_tri = 2;
        g.b_row0 = o + s; g.b_col0 = o;
        g.M = s; g.N = bot; g.K = s; g.batch = 1; g.alpha = 1.f;
        g.c_rows = s; g.c_cols = s;
        g.out[0] = TT.a[0]; g.out[1] = TT.a[1]; g.out[2] = TT.a[2]; g.ldo = s; g.nout = 3;
        return gemm_tc(lcC, g, status);
    };
    auto pair_second = [&](int s, int p) -> int {     // X(bottom-left) [bot][s] = -B^{-1} TT^T   (B^{-1} lower triangular: k <= row)
        const int o = 2 * s * p, bot = min(s, F - (o + s));
        const Trip TT = tt_level(s);
        TcGemm g{};
        pass_plan(g, X3, ld, F, F, TT, s, s, s);
        g.a_row0 = o + s; g.a_col0 = o + s; g.a_tri = 1;
        g.M = bot; g.N = s; g.K = bot; g.batch = 1; g.alpha = -1.f;
        g.c_row0 = o + s; g.c_col0 = o; g.c_rows = F; g.c_cols = F;
        g.out[0] = X3.a[0]; g.out[1] = X3.a[1]; g.out[2] = X3.a[2]; g.ldo = ld; g.nout = 3;
        const int r = gemm_tc(lcC, g, status);
        if (r) return r;
        dim3 grid(s / 32, s / 32, 1), block(32, 8);
        k_transpose_blocks<<<grid, block, 0, sC>>>(X3, XT3, n, ld, s, p);
        lc.count();
        return PKV_OK;
    };
    const int nsp = well_conditioned ? 2 : 3;
    Trip S2{{t->S2[0], t->S2[1], t->S2[2]}}, Z2{{t->Z2[0], t->Z2[1], t->Z2[2]}};
    static cudaEvent_t tev[5];      // trace mode only: stream timeline of the call
    if (trace && !tev[0]) for (auto& e : tev) cudaEventCreate(&e);
    timespec ts0{};
    if (phase != 2) {
    if (trace) { cudaEventRecord(tev[0], lc.st); clock_gettime(CLOCK_MONOTONIC, &ts0); }
    cudaEventRecord(evFork, lc.st);
    cudaStreamWaitEvent(sA, evFork, 0);
    cudaStreamWaitEvent(sB, evFork, 0);
    cudaStreamWaitEvent(sE, evFork, 0);
    cudaStreamWaitEvent(sC, evFork, 0);
    if (F > PB) {
        launch_split3(lcB, G + (size_t)PB * ld, ld, F - PB, PB,
                      Trip{{P3.a[0] + (size_t)PB * PB, P3.a[1] + (size_t)PB * PB, P3.a[2] + (size_t)PB * PB}}, PB, 3);
        cudaEventRecord(evU[1], sB);
    }
    rc = PKV_OK;
    for (int b = 0; b < nblk && rc == PKV_OK; ++b) {
        const int k0 = b * PB, k1 = min(F, k0 + PB), rem = F - k1;
        if (b > 0) cudaStreamWaitEvent(sA, evU[b & 1], 0);       // U^a_{b-2}, or the split of the first column for b = 1
        if (b > 2) cudaStreamWaitEvent(sA, evUb[(b - 3) % 3], 0); // U^b_{b-3}: the last bulk part that touches block column b
        cp.k0 = k0;
        if ((rc = launch_chain(sA, cp))) break;
        lc.count();
        cudaEventRecord(evF, sA);
        {   // sC: transposed copy of this block's inverse, then every pair that block b completes, lowest level first
            cudaStreamWaitEvent(sC, evF, 0);
            if (b > 0) cudaStreamWaitEvent(sC, evP, 0);          // P_{b-1}: the last panel such a pair reads
            dim3 grid(PB / 32, PB / 32, 1), block(32, 8);
            k_transpose_diag<<<grid, block, 0, sC>>>(X3, XT3, n, ld, b);
            lc.count();
            // first products of the pairs whose top half ended with block b - 1 (its panel P_{b-1} is the block C)
            for (long long s = PB; s < F && rc == PKV_OK; s *= 2) {
                const int per = (int)(2 * s / PB), p = b / per;
                if (b % per != per / 2 || (2LL * p + 1) * s >= F) continue;
                rc = pair_first((int)s, p);
            }
            // second products of the pairs that block b completes, lowest level first
            for (long long s = PB; s < F && rc == PKV_OK; s *= 2) {
                const int per = (int)(2 * s / PB), p = b / per;
                if ((2LL * p + 1) * s >= F) continue;            // no bottom half: nothing to do at this level
                if (b + 1 != min(nblk, (p + 1) * per)) continue; // the pair's last block is not b
                rc = pair_second((int)s, p);
            }
            if (rc != PKV_OK) break;
        }
        if (rem <= 0) break;
        cudaStreamWaitEvent(sB, evF, 0);
        {   // P_b: panel, kept as a bf16 triple in L3
            TcGemm g{};
            pass_plan(g, P3, PB, F, PB, X3, ld, F, F);
            g.a_row0 = k1;
            g.b_row0 = k0; g.b_col0 = k0;
            g.M = rem; g.N = PB; g.K = PB; g.batch = 1; g.alpha = 1.f;
            g.c_row0 = k1; g.c_col0 = k0; g.c_rows = F; g.c_cols = F;
            g.out[0] = L3.a[0]; g.out[1] = L3.a[1]; g.out[2] = L3.a[2]; g.ldo = ld; g.nout = 3;
            if ((rc = gemm_tc(lcB, g, status))) break;
        }
        cudaEventRecord(evP, sB);
        // U_b: G22 -= L21 L21^T on the lower triangle, in two launches.  U^a_b, the first two block columns (on sB):
        // column b+1 gets its last update here and leaves the bf16 triple of the next panel operand, column b+2
        // holds the next-but-one diagonal block; the first diagonal tile is left to the chain kernel.  U^b_b, all
        // further columns (on sE), has two chain steps to finish.  Updates of one tile by U^a and U^b of different
        // steps may overlap in time: both add through the memory system's reductions; the one launch that reads a
        // column back (U^a's first column) waits for the bulk parts that touched it.
        if (rem > PB) {
            if (b > 1) cudaStreamWaitEvent(sB, evUb[(b - 2) % 3], 0);
            TcGemm g{};
            pass_plan(g, L3, ld, F, F, L3, ld, F, F);
            g.a_row0 = k1; g.a_col0 = k0; g.b_row0 = k1; g.b_col0 = k0;
            g.M = rem; g.N = min(rem, 2 * PB); g.K = PB; g.batch = 1; g.alpha = -1.f;
            g.C = const_cast<float*>(G); g.ldc = ld; g.accumulate = true; g.lower_only = true; g.skip_tile00 = true;
            g.c_row0 = k1; g.c_col0 = k1; g.c_rows = F; g.c_cols = F;
            g.out[0] = P3.a[0]; g.out[1] = P3.a[1]; g.out[2] = P3.a[2]; g.ldo = PB; g.nout = 3; g.out_col_off = k1;
            g.out_col0_only = true;
            if ((rc = gemm_tc(lcB, g, status))) break;
        }
        if (rem > 2 * PB) {
            const int o = k1 + 2 * PB;
            cudaStreamWaitEvent(sE, evP, 0);
            TcGemm g{};
            pass_plan(g, L3, ld, F, F, L3, ld, F, F);
            g.a_row0 = o; g.a_col0 = k0; g.b_row0 = o; g.b_col0 = k0;
            g.M = F - o; g.N = F - o; g.K = PB; g.batch = 1; g.alpha = -1.f;
            g.C = const_cast<float*>(G); g.ldc = ld; g.accumulate = true; g.lower_only = true;
            g.c_row0 = o; g.c_col0 = o; g.c_rows = F; g.c_cols = F;
            if ((rc = gemm_tc(lcE, g, status))) break;
        }
        cudaEventRecord(evUb[b % 3], sE);
        cudaEventRecord(evU[b & 1], sB);
    }
    if (trace) {
        timespec ts; clock_gettime(CLOCK_MONOTONIC, &ts);
        fprintf(stderr, "host: factorisation loop issued in %.3f ms\n", (ts.tv_sec - ts0.tv_sec) * 1e3 + (ts.tv_nsec - ts0.tv_nsec) * 1e-6);
    }
    // join: the caller's stream continues after the chain's last kernel and the last doubling level
    cudaEventRecord(evF, sA);
    cudaEventRecord(evP, sB);
    cudaEventRecord(evC, sC);
    if (trace) { cudaEventRecord(tev[1], sA); cudaEventRecord(tev[2], sC); }
    cudaEventRecord(evUb[0], sE);
    for (cudaEvent_t e : {evF, evP, evC, evUb[0]}) cudaStreamWaitEvent(lc.st, e, 0);
    if (rc != PKV_OK) return rc;
    if (trace && nblk <= 64) {
        static long long host_stamps[64 * kChainStamps];
        cudaStreamSynchronize(lc.st);
        cudaMemcpy(host_stamps, t->stamps, (size_t)nblk * kChainStamps * sizeof(long long), cudaMemcpyDeviceToHost);
        double acc[kChainStamps] = {0};
        for (int b = 1; b < nblk; ++b)
            for (int i = 1; i < 8; ++i) acc[i] += (double)(host_stamps[b * kChainStamps + i] - host_stamps[b * kChainStamps + i - 1]);
        fprintf(stderr, "chain kernel phases, mean cycles over blocks 1..%d: setup+wait %.0f | tma+mma1 %.0f | L->smem+mma2 %.0f | "
                        "A write %.0f | factor %.0f | inverse %.0f | output %.0f ; start-to-start %.0f ns\n", nblk - 1,
                acc[1] / (nblk - 1), acc[2] / (nblk - 1), acc[3] / (nblk - 1), acc[4] / (nblk - 1), acc[5] / (nblk - 1),
                acc[6] / (nblk - 1), acc[7] / (nblk - 1),
                nblk > 2 ? (double)(host_stamps[(nblk - 1) * kChainStamps + 16] - host_stamps[kChainStamps + 16]) / (nblk - 2) : 0.0);
        fprintf(stderr, "   start-to-start / busy per block (us, global timer):");
        for (int b = 1; b < nblk; ++b)
            fprintf(stderr, " %.1f/%.1f", (host_stamps[b * kChainStamps + 16] - host_stamps[(b - 1) * kChainStamps + 16]) * 1e-3,
                    (host_stamps[b * kChainStamps + 17] - host_stamps[b * kChainStamps + 16]) * 1e-3);
        fprintf(stderr, "\n");
        const long long* h1 = host_stamps + kChainStamps;
        fprintf(stderr, "   block 1, factor phase (cycles): forward substitution+sync %lld | warp 0 update %lld | diagonal pieces %lld | "
                        "wait for the other warps %lld ; inverse: 16x16 pieces %lld | level 16 %lld | 32 %lld | 64 %lld\n",
                h1[8], h1[9], h1[10], h1[11], h1[12] - h1[5], h1[13] - h1[12], h1[14] - h1[13], h1[15] - h1[14]);

    }
    }
    if (phase == 1) return PKV_OK;
    // (2. X = L^{-1} was built beside the factorisation, see sC above.)  cond(L) = sqrt(cond(G)): with a
    // well-conditioned ridge matrix (a few tens) the rounding of those products (pairs: 2^-16) reaches dW
    // unamplified and three passes are enough.  The same holds for the factorisation: lambda is then of the order
    // of the diagonal of S_H and the trailing updates do not cancel; with a small lambda0 they do, and everything
    // takes triples in six passes with separated accumulators.
    // ---- 3. dW = (S_T X^T) X ----
    // The rounding of these two products is amplified by cond(L): pairs (2^-16, three passes) when
    // the ridge keeps G well conditioned, triples (2^-24, six passes) otherwise.
    // S_T produced on another stream beside the factorisation: its event was recorded (by the host) before this
    // solve was issued.  (A captured solve is split in two graphs at this point and waits between them.)
    if (wait_S_T && cudaStreamWaitEvent(lc.st, t->st_ready, 0) != cudaSuccess) return PKV_ERR_CUDA;
    if (!S_T_triple) launch_split3(lc, S_T, ld, d, F, S2, ld, nsp);      // else: S2 already holds the triple
    {
        TcGemm g{};
        if (nsp == 2) three_pass(g, S2, ld, d, F, X3, ld, F, F);
        else six_pass(g, S2, ld, d, F, X3, ld, F, F);
        g.M = d; g.N = F; g.K = F; g.batch = 1; g.alpha = 1.f; g.k_tri = 1;
        g.nacc = well_conditioned ? 1 : 2;      // long contraction, no cancellation; one accumulator keeps two CTAs per SM
        g.c_rows = d; g.c_cols = F;
        g.out[0] = Z2.a[0]; g.out[1] = Z2.a[1]; g.out[2] = Z2.a[2]; g.ldo = ld; g.nout = nsp;
        if ((rc = gemm_tc(lc, g, status))) return rc;
    }
    if (trace) cudaEventRecord(tev[3], lc.st);
    {
        TcGemm g{};
        if (nsp == 2) three_pass(g, Z2, ld, d, F, XT3, ld, F, F);
        else six_pass(g, Z2, ld, d, F, XT3, ld, F, F);
        g.M = d; g.N = F; g.K = F; g.batch = 1; g.alpha = 1.f; g.k_tri = 2;
        g.nacc = well_conditioned ? 1 : 2;
        g.C = dW; g.C_ind = dW_ind; g.ldc = ld; g.c_rows = d; g.c_cols = F; g.accumulate = add_to_dW;
        if (dW_pair) { g.out[0] = dW_pair->hi; g.out[1] = dW_pair->lo; g.ldo = ld; g.nout = 2; }
        if ((rc = gemm_tc(lc, g, status))) return rc;
    }
    if (trace) {
        cudaEventRecord(tev[4], lc.st);
        cudaEventSynchronize(tev[4]);
        float a, b, c2, e;
        cudaEventElapsedTime(&a, tev[0], tev[1]);
        cudaEventElapsedTime(&b, tev[0], tev[2]);
        cudaEventElapsedTime(&c2, tev[0], tev[3]);
        cudaEventElapsedTime(&e, tev[0], tev[4]);
        fprintf(stderr, "solve timeline (ms from the start): last chain kernel %.3f | last doubling level %.3f | S_T X^T %.3f | dW %.3f\n",
                a, b, c2, e);
    }
    return PKV_OK;
}

// One correction of iterative refinement: dW += (R X^T) X with the inverse factor X = L^{-1} that the last solve of
// this system left in the solver's buffers (Eq. 8 applied to a residual R [d][n] instead of S_T).
int tc_solve_apply_add(const Lc& lc, TcSolveBuffers* t, const float* R, int n, int ld, int d, float* dW,
                       bool well_conditioned, DevStatus* status) {
    return solve_body(lc, t, nullptr, R, n, ld, d, dW, nullptr, well_conditioned, false, status, nullptr, nullptr, false, 2,
                      true);
}

__global__ void k_solve_begin(float** slot, float* dW, DevStatus* gstatus, const DevStatus* status) {
    if (threadIdx.x == 0) {
        *slot = dW;
        *gstatus = *status;
    }
}
__global__ void k_solve_end(DevStatus* status, const DevStatus* gstatus) {
    if (threadIdx.x == 0) {
        DevStatus s = *gstatus;
        // what another stream put into the caller's word while the solve ran (the targets' norm, a raised code):
        // the solve itself never touches t_fro2
        s.t_fro2 = status->t_fro2;
        if (s.code == 0 && status->code != 0) {
            s.code = status->code;
            s.info0 = status->info0;
            s.info1 = status->info1;
        }
        *status = s;
    }
}

// The solve is some hundreds of small dependent launches on four streams: issued one by one they cost the host
// more than a millisecond and the device several microseconds of stream bookkeeping each.  The body is therefore
// captured once per (operands, shape, precision plan) into a CUDA graph on an internal stream and replayed;
// what changes from call to call goes through device memory: the result's address (a pointer slot the final
// products read) and the status word (copied in before, out after).  PKV_SOLVE_GRAPH=0 in the environment, the
// phase trace, a changed row stride or any failure to capture select the launch-by-launch path.
int tc_ridge_solve_impl(const Lc& lc, TcSolveBuffers* t, const float* G, const float* S_T, int n, int ld, int d,
                        float* dW, bool well_conditioned, bool zero_fill, DevStatus* status, const Pair* dW_pair,
                        __nv_bfloat16* const* S_T_triple, bool wait_S_T) {
    static const bool graphs_on = [] { const char* e = getenv("PKV_SOLVE_GRAPH"); return !e || atoi(e) != 0; }();
    if (!graphs_on || t->graph_off || solve_trace() || zero_fill)
        return solve_body(lc, t, G, S_T, n, ld, d, dW, nullptr, well_conditioned, zero_fill, status, dW_pair, S_T_triple, wait_S_T);
    const bool aligned = ((uintptr_t)dW & 15) == 0;
    SolveGraph* e = nullptr;
    for (int i = 0; i < t->n_graphs; ++i) {
        SolveGraph& c = t->graphs[i];
        if (c.G == G && c.S_T == S_T && c.n == n && c.ld == ld && c.d == d && c.well == well_conditioned &&
            c.triple == (S_T_triple != nullptr) && c.aligned == aligned && c.wait == wait_S_T && c.pair_hi == (dW_pair ? dW_pair->hi : nullptr) &&
            c.pair_lo == (dW_pair ? dW_pair->lo : nullptr))
            e = &c;
    }
    k_solve_begin<<<1, 32, 0, lc.st>>>(t->slot, dW, t->gstatus, status);
    lc.count();
    if (!e) {
        const int64_t before = lc.launches ? *lc.launches : 0;
        const Lc lco{t->origin, lc.launches, lc.map_cache};
        // S_T arriving from another stream: two graphs, split where the final products begin, and an ordinary wait
        // for the producer's event between them
        const int n_parts = wait_S_T ? 2 : 1;
        cudaGraphExec_t exec[2] = {nullptr, nullptr};
        int rc = PKV_OK;
        bool captured = true;
        for (int part = 0; part < n_parts && captured && rc == PKV_OK; ++part) {
            if (cudaStreamBeginCapture(t->origin, cudaStreamCaptureModeRelaxed) != cudaSuccess) {
                captured = false;
                break;
            }
            rc = solve_body(lco, t, G, S_T, n, ld, d, dW, t->slot, well_conditioned, false, t->gstatus, dW_pair, S_T_triple,
                            false, wait_S_T ? part + 1 : 0);
            cudaGraph_t gr = nullptr;
            const cudaError_t ce = cudaStreamEndCapture(t->origin, &gr);
            if (rc == PKV_OK && (ce != cudaSuccess || !gr || cudaGraphInstantiate(&exec[part], gr, 0) != cudaSuccess)) {
                exec[part] = nullptr;
                captured = false;
            }
            if (gr) cudaGraphDestroy(gr);
        }
        if (rc != PKV_OK || !captured) {
            for (cudaGraphExec_t x : exec) if (x) cudaGraphExecDestroy(x);
            cudaGetLastError();
            if (rc != PKV_OK) return rc;
            // capture is not available here: stay on the launch-by-launch path from now on
            t->graph_off = 1;
            if (lc.launches) *lc.launches = before;
            return solve_body(lc, t, G, S_T, n, ld, d, dW, nullptr, well_conditioned, zero_fill, status, dW_pair, S_T_triple, wait_S_T);
        }
        int slot = t->n_graphs;
        if (slot == kSolveGraphs) {      // evict the least recently used
            slot = 0;
            for (int i = 1; i < kSolveGraphs; ++i) if (t->graphs[i].used < t->graphs[slot].used) slot = i;
            cudaGraphExecDestroy(t->graphs[slot].exec);
            if (t->graphs[slot].exec2) cudaGraphExecDestroy(t->graphs[slot].exec2);
        } else {
            ++t->n_graphs;
        }
        e = &t->graphs[slot];
        *e = SolveGraph{G, S_T, n, ld, d, well_conditioned, S_T_triple != nullptr, aligned, wait_S_T, dW_pair ? dW_pair->hi : nullptr,
                        dW_pair ? dW_pair->lo : nullptr, exec[0], exec[1], (lc.launches ? *lc.launches : 0) - before, 0};
    } else {
        lc.count((int)e->launches);
    }
    e->used = ++t->graph_clock;
    if (cudaGraphLaunch(e->exec, lc.st) != cudaSuccess) return PKV_ERR_CUDA;
    if (e->exec2) {
        if (cudaStreamWaitEvent(lc.st, t->st_ready, 0) != cudaSuccess || cudaGraphLaunch(e->exec2, lc.st) != cudaSuccess)
            return PKV_ERR_CUDA;
    }
    k_solve_end<<<1, 32, 0, lc.st>>>(status, t->gstatus);
    lc.count();
    if (solve_trace_graph()) {
        const int nblk = (n + PB - 1) / PB;
        static long long hs[64 * kChainStamps];
        if (nblk <= 64) {
            cudaStreamSynchronize(lc.st);
            cudaMemcpy(hs, t->stamps, (size_t)nblk * kChainStamps * sizeof(long long), cudaMemcpyDeviceToHost);
            fprintf(stderr, "chain kernels of the replayed solve, start-to-start / busy per block (us, global timer):");
            for (int b = 1; b < nblk; ++b)
                fprintf(stderr, " %.1f/%.1f", (hs[b * kChainStamps + 16] - hs[(b - 1) * kChainStamps + 16]) * 1e-3,
                        (hs[b * kChainStamps + 17] - hs[b * kChainStamps + 16]) * 1e-3);
            fprintf(stderr, " ; first start to last end %.1f us\n",
                    (hs[(nblk - 1) * kChainStamps + 17] - hs[16]) * 1e-3);
        }
    }
    return PKV_OK;
}

}  // namespace pkv
