// Tensor-core GEMM for sm_100a:  C[M][N] = alpha * sum_p A_p[M][K] B_p[N][K]^T (+ addend) (+ C).
//
// bf16 operands, fp32 accumulation in tensor memory.  One CTA computes a 128 x BN tile:
//   warp 0   TMA producer: 128x64 / BNx64 bf16 tiles into a ring of 128B-swizzled smem stages
//   warp 1   allocates TMEM, one elected thread issues tcgen05.mma (4 x K=16 per stage) and
//            commits each stage back to the producer
//   warps 2-5 epilogue: tcgen05.ld the accumulator (each warp its own 32-lane quarter), scale,
//            add, store fp32
// Several (A_p, B_p) pairs accumulate into the same tile ("passes"): an fp32 activation split
// into bf16 hi + lo parts is multiplied as two passes against the same bf16 weight, an fp32 x
// fp32 product as three or six passes.  Ragged M, N, K are handled by TMA zero fill and
// predicated stores.
#include <cuda.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "pkv_ptx.cuh"
#include "pkv_tc.h"

namespace pkv {

using namespace ptx;

struct alignas(64) GemmTcParams {
    CUtensorMap mapA[3];      // distinct A operands (e.g. hi, mid, lo parts)
    CUtensorMap mapB[3];      // distinct B operands
    int nA, nB, npass;
    int ngrp, grp_end[3];     // grouped B (see TcGemm): mapB[k] serves output columns [grp_end[k-1], grp_end[k])
    int pa[kGemmMaxPass], pb[kGemmMaxPass];   // pass i multiplies A operand pa[i] with B operand pb[i]
    int stages;
    int M, N, K;
    int a_row0, a_col0, a_zrow, a_zcol;
    int b_row0, b_col0, b_zrow, b_zcol;
    int c_row0, c_col0, c_zrow, c_zcol, c_rows, c_cols;
    float* C;
    float* const* C_ind;      // if set, the fp32 output base is read from this device location instead of C
    long long ldc;
    float alpha;
    const unsigned* amax_a;   // optional power-of-two operand scales to divide out, see TcGemm
    const unsigned* amax_b;
    int f16;                  // fp16 operands
    const float* addend;
    long long ldadd;
    __nv_bfloat16* out[3];
    long long ldo;
    int nout, out_col_off;
    int accumulate, lower_only, k_tri, a_tri, vec_ok;
    int nacc;                 // TMEM accumulators per tile (1, 2 or 4), see TcGemm::nacc
    int skip_tile00;          // the tile at (blockIdx.x, blockIdx.y) = (0, 0) is left alone
    int out_col0_only;        // bf16 parts are written by the tiles of the first block column only
    int out_vec;              // the bf16 parts can be stored 16 bytes at a time (alignment of pointers, stride, offsets)
    DevStatus* status;
    unsigned long long* stamps;   // optional: global-timer marks of the first CTA's phases (profiling aid)
};

constexpr int kGemmMaxStages = 6;

__device__ __forceinline__ uint32_t pack2_bf16(__nv_bfloat16 a, __nv_bfloat16 b) {
    return (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
}
constexpr int kGemmBarBytes = (2 * kGemmMaxStages + 1) * 8 + 16;

// 32 consecutive values of one output row as up to three bf16 parts (successive roundings), 16-byte stores
__device__ __forceinline__ void store_parts_row(const GemmTcParams& p, const float (&v)[32], size_t o) {
#pragma unroll
    for (int c8 = 0; c8 < 4; ++c8) {
        uint32_t h[4], m[4], l[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float x0 = v[c8 * 8 + 2 * e], x1 = v[c8 * 8 + 2 * e + 1];
            const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
            const float r0 = x0 - __bfloat162float(h0), r1 = x1 - __bfloat162float(h1);
            const __nv_bfloat16 m0 = __float2bfloat16_rn(r0), m1 = __float2bfloat16_rn(r1);
            h[e] = pack2_bf16(h0, h1);
            m[e] = pack2_bf16(m0, m1);
            l[e] = pack2_bf16(__float2bfloat16_rn(r0 - __bfloat162float(m0)), __float2bfloat16_rn(r1 - __bfloat162float(m1)));
        }
        *reinterpret_cast<uint4*>(p.out[0] + o + c8 * 8) = make_uint4(h[0], h[1], h[2], h[3]);
        if (p.nout > 1) *reinterpret_cast<uint4*>(p.out[1] + o + c8 * 8) = make_uint4(m[0], m[1], m[2], m[3]);
        if (p.nout > 2) *reinterpret_cast<uint4*>(p.out[2] + o + c8 * 8) = make_uint4(l[0], l[1], l[2], l[3]);
    }
}

__device__ __forceinline__ void gemm_stamp(const GemmTcParams& p, int i) {
    if (p.stamps && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) {
        unsigned long long ns;
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(ns));
        p.stamps[i] = ns;
    }
}

// One k-tile stage holds every distinct operand tile once: nA x [128][64] and nB x [BN][64] bf16,
// and all passes are issued from it (the shared operand of a split product is not re-read).
// (A variant whose epilogue warps prefetched the fp32 C tile of a read-modify-write product during the main loop
// needed 240 registers per thread, one CTA per SM; without it two or three CTAs share an SM and hide the
// read's latency better: the solve went from 2.51 to 2.45 ms at F = 4096 and from 3.66 to 3.55 ms at F = 5120.)
//
// Accumulators.  The tensor core adds each MMA's result to the fp32 accumulator with truncation, not
// round-to-nearest: a sum of same-signed terms (the diagonal of a Gram or of L L^T) comes out low by about
// 2^-25 of the running sum per MMA.  When a small difference C - A B^T is wanted (trailing updates of a
// rank-deficient ridge matrix) that bias is what limits the result.  With nacc > 1 the large hi x hi pass goes
// round-robin to accumulators 1..nacc-1, each of which so sees only a few adds at a fraction of the full
// magnitude, every other pass to accumulator 0 where its truncation is relative to the small cross terms;
// the epilogue adds the accumulators in registers with round-to-nearest.
template <int BN>
__global__ void __launch_bounds__(192) k_gemm_tc(const __grid_constant__ GemmTcParams p) {
    // Tiles are handed out in grid order; where a triangular operand makes the contraction grow with the tile's
    // column (k_tri 1) or row (a_tri 1), the order is reversed so that the long tiles start first
    const int bx = (p.k_tri == 1) ? (int)(gridDim.x - 1 - blockIdx.x) : (int)blockIdx.x;
    const int by = (p.a_tri == 1) ? (int)(gridDim.y - 1 - blockIdx.y) : (int)blockIdx.y;
    const int m0 = by * 128, n0 = bx * BN, z = blockIdx.z;
    if (p.lower_only && n0 > m0 + 127) return;
    if (p.skip_tile00 && blockIdx.x == 0 && blockIdx.y == 0) return;
    pdl_launch_dependents();
    if (threadIdx.x == 0) gemm_stamp(p, 0);
    // absolute coordinates of this tile's output; tiles entirely outside the stored region do nothing
    const int crow0 = p.c_row0 + z * p.c_zrow + m0, ccol0 = p.c_col0 + z * p.c_zcol + n0;
    if (crow0 >= p.c_rows || ccol0 >= p.c_cols) return;

    constexpr int kA = 128 * 64 * 2, kB = BN * 64 * 2;
    const int stage_bytes = p.nA * kA + p.nB * kB;
    const int STAGES = p.stages;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw);
    const uint32_t bars = base + STAGES * stage_bytes;        // full[STAGES], empty[STAGES], tmem_full
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + STAGES * stage_bytes + (2 * STAGES + 1) * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* staging = reinterpret_cast<float*>(sm);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // contraction range in 64-wide tiles; a triangular B operand lets whole tiles be skipped:
    //   k_tri = 1: B[n][k] = 0 for k > n (lower triangular)   -> tiles beyond the tile's last row are zero
    //   k_tri = 2: B[n][k] = 0 for k < n (upper triangular)   -> tiles before the tile's first row are zero
    int kt_begin = 0, kt_end = (p.K + 63) / 64;
    if (p.k_tri == 1) kt_end = min(kt_end, (n0 + BN + 63) / 64);
    if (p.k_tri == 2) kt_begin = min(kt_end, n0 / 64);
    //   a_tri: the same for a triangular A operand (1: A[m][k] = 0 for k > m; 2: A[m][k] = 0 for k < m)
    if (p.a_tri == 1) kt_end = min(kt_end, (m0 + 128 + 63) / 64);
    if (p.a_tri == 2) kt_begin = max(kt_begin, min(kt_end, m0 / 64));
    const int ktiles = kt_end - kt_begin;

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(bars + 8 * i, 1);
            mbar_init(bars + 8 * (STAGES + i), 1);
        }
        mbar_init(bars + 8 * (2 * STAGES), 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    const int nacc = p.nacc;
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), (uint32_t)(BN * nacc));
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_slot;
    // everything above is independent of earlier kernels; from here on their results are read
    pdl_wait();
    // an earlier stage already failed: the call reports it.  The status word may change while the CTA starts
    // (another CTA's error), so one thread reads it and the whole CTA takes the same branch.
    volatile int* skip_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);
    if (threadIdx.x == 0) { gemm_stamp(p, 1); *skip_flag = p.status->code; }
    __syncthreads();
    const bool skip = *skip_flag != 0;
    if (threadIdx.x == 0) gemm_stamp(p, 2);

    if (skip) {
        // nothing to do: fall through to the teardown
    } else if (warp == 0) {
        if (lane == 0) {
            const int ar = p.a_row0 + z * p.a_zrow + m0, ac = p.a_col0 + z * p.a_zcol;
            int br = p.b_row0 + z * p.b_zrow + n0;
            const int bc = p.b_col0 + z * p.b_zcol;
            int gsel = 0;      // grouped B: the matrix this tile's columns belong to, rows counted from its start
            if (p.ngrp > 1) {
                while (gsel + 1 < p.ngrp && n0 >= p.grp_end[gsel]) ++gsel;
                if (gsel > 0) br -= p.grp_end[gsel - 1];
            }
            for (int it = 0; it < ktiles; ++it) {
                const int s = it % STAGES;
                if (!mbar_wait(bars + 8 * (STAGES + s), ((it / STAGES) & 1) ^ 1, abort_flag, p.status, 1)) break;
                const int kt = kt_begin + it;
                const uint32_t full = bars + 8 * s;
                const uint32_t sa = base + s * stage_bytes;
                mbar_expect_tx(full, stage_bytes);
                for (int i = 0; i < p.nA; ++i) tma_load_2d(sa + i * kA, &p.mapA[i], full, ac + kt * 64, ar);
                for (int i = 0; i < p.nB; ++i) tma_load_2d(sa + p.nA * kA + i * kB, &p.mapB[p.ngrp > 1 ? gsel : i], full, bc + kt * 64, br);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = p.f16 ? idesc_f16(128, BN) : idesc_bf16(128, BN);
            bool ok = true;
            uint32_t used = 0u;          // accumulators that already hold a partial sum
            uint32_t hh = 0u;            // running index of the hi x hi MMAs
            for (int it = 0; it < ktiles; ++it) {
                const int s = it % STAGES;
                if (!mbar_wait(bars + 8 * s, (it / STAGES) & 1, abort_flag, p.status, 2)) { ok = false; break; }
                tc_fence_after();
                if (it == 0) gemm_stamp(p, 3);
                const uint32_t sa = base + s * stage_bytes;
                for (int ps = 0; ps < p.npass; ++ps) {
                    const uint64_t da = smem_desc_sw128(sa + p.pa[ps] * kA);
                    const uint64_t db = smem_desc_sw128(sa + p.nA * kA + p.pb[ps] * kB);
                    const bool big = nacc > 1 && p.pa[ps] == 0 && p.pb[ps] == 0;      // hi x hi
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint32_t acc = big ? 1u + (hh++ % (uint32_t)(nacc - 1)) : 0u;
                        mma_bf16_ss(tbase + acc * (uint32_t)BN, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc,
                                    (used >> acc) & 1u);
                        used |= 1u << acc;
                    }
                }
                mma_commit(bars + 8 * (STAGES + s));
            }
            if (ok) mma_commit(bars + 8 * (2 * STAGES));
            gemm_stamp(p, 4);
        }
    } else {
        // epilogue: TMEM -> registers -> per-warp smem tile -> row-contiguous global accesses
        const int q = warp & 3;
        const int rl0 = m0 + q * 32;                 // first row of this warp inside the batch element
        const int rowa0 = crow0 + q * 32;            // ... and its absolute output row
        const int nrows = max(0, min(32, min(p.M - rl0, p.c_rows - rowa0)));
        const bool vec_ok = p.vec_ok != 0;
        float* const Cp = p.C_ind ? *p.C_ind : p.C;
        bool ok = true;
        if (ktiles > 0) {
            ok = mbar_wait(bars + 8 * (2 * STAGES), 0, abort_flag, p.status, 3);
            tc_fence_after();
        }
        if (warp == 2 && lane == 0) gemm_stamp(p, 5);
        if (ok) {
            float alpha = p.alpha;
            if (p.amax_a) alpha *= f16_inv_scale_from_max(*p.amax_a);
            if (p.amax_b) alpha *= f16_inv_scale_from_max(*p.amax_b);
            float* stg = staging + q * (32 * 33);
            // not unrolled: a CTA runs each chunk's code once, and a short-K tile's time is mostly instruction fetch
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                if (ktiles > 0) {
                    tmem_ld32(tbase + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
                    tmem_ld_wait();
                    if (warp == 2 && lane == 0 && c0 < 128) gemm_stamp(p, 8 + (c0 >> 5) * 2);
                    // further accumulators: added in registers with round to nearest (the launcher only asks for
                    // them when every one of them receives at least one MMA)
                    for (int a = 1; a < nacc; ++a) {
                        uint32_t r2[32];
                        tmem_ld32(tbase + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * BN + c0), r2);
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
                if (warp == 2 && lane == 0 && c0 < 128) gemm_stamp(p, 9 + (c0 >> 5) * 2);
                const int col = ccol0 + c0;                    // absolute output column of r[0]
                const int ncol = min(min(32, p.N - (n0 + c0)), p.c_cols - col);
                if (ncol <= 0) break;
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = alpha * __uint_as_float(r[j]);
                if (Cp && lane < nrows) {
                    // fp32 output: every lane owns one row; 128 contiguous bytes, loads batched ahead of stores
                    const size_t row = (size_t)(rowa0 + lane);
                    float* crow = Cp + row * p.ldc + col;
                    const float* arow = p.addend ? p.addend + row * p.ldadd + col : nullptr;
                    if (vec_ok && ncol == 32) {
                        if (arow) {
                            float4 a4[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) a4[j] = *reinterpret_cast<const float4*>(arow + 4 * j);
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                v[4 * j] += a4[j].x; v[4 * j + 1] += a4[j].y; v[4 * j + 2] += a4[j].z; v[4 * j + 3] += a4[j].w;
                            }
                        }
                        // C += v.  Where this tile does not also have to write bf16 parts of the sum, the addition is
                        // left to the memory system (a vector reduction: same single rounding of C + v, no load, and so
                        // no DRAM round trip per chunk inside the epilogue); every element has one writer per launch.
                        const bool parts_here = p.nout > 0 && (!p.out_col0_only || blockIdx.x == 0);
                        if (p.accumulate && !parts_here) {
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(crow + 4 * j), "f"(v[4 * j]),
                                             "f"(v[4 * j + 1]), "f"(v[4 * j + 2]), "f"(v[4 * j + 3])
                                             : "memory");
                        } else {
                            if (p.accumulate) {
                                float4 c4[8];
#pragma unroll
                                for (int j = 0; j < 8; ++j) c4[j] = *reinterpret_cast<const float4*>(crow + 4 * j);
#pragma unroll
                                for (int j = 0; j < 8; ++j) {
                                    v[4 * j] += c4[j].x; v[4 * j + 1] += c4[j].y; v[4 * j + 2] += c4[j].z; v[4 * j + 3] += c4[j].w;
                                }
                            }
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                *reinterpret_cast<float4*>(crow + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (j < ncol) {
                                if (arow) v[j] += arow[j];
                                if (p.accumulate) v[j] += crow[j];
                                crow[j] = v[j];
                            }
                        }
                    }
                }
                if (p.nout > 0 && (!p.out_col0_only || blockIdx.x == 0) && p.out_vec && ncol == 32) {
                    // bf16 parts straight from the registers: the lane owns 32 consecutive columns of its row,
                    // four 16-byte stores per part
                    if (lane < nrows) store_parts_row(p, v, (size_t)(rowa0 + lane) * p.ldo + (col - p.out_col_off));
                } else if (p.nout > 0 && (!p.out_col0_only || blockIdx.x == 0)) {
                    // bf16 parts: through the warp's smem tile so that a warp writes 64 contiguous bytes per row
#pragma unroll
                    for (int j = 0; j < 32; ++j) stg[lane * 33 + j] = v[j];
                    __syncwarp();
                    if (lane < ncol) {
                        for (int rr = 0; rr < nrows; ++rr) {
                            const float x = stg[rr * 33 + lane];
                            const size_t o = (size_t)(rowa0 + rr) * p.ldo + (col - p.out_col_off) + lane;
                            __nv_bfloat16 h = __float2bfloat16_rn(x);
                            p.out[0][o] = h;
                            if (p.nout > 1) {
                                const float r1 = x - __bfloat162float(h);
                                __nv_bfloat16 m = __float2bfloat16_rn(r1);
                                p.out[1][o] = m;
                                if (p.nout > 2) p.out[2][o] = __float2bfloat16_rn(r1 - __bfloat162float(m));
                            }
                        }
                    }
                    __syncwarp();
                }
            }
        }
    }
    // teardown: after an abort give copies in flight time to land before the CTA's smem is released
    if (warp == 2 && lane == 0) gemm_stamp(p, 6);
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tbase, (uint32_t)(BN * nacc));
    }
    if (threadIdx.x == 0) gemm_stamp(p, 7);
}


// ---------------------------------------------------------------------------------------------
// CTA-pair variant (cta_group::2): a cluster of two CTAs computes one 256 x 256 tile.  Each CTA loads its own 128
// rows of every A part and its own 128-row half of every B part (every load lands in the issuing CTA only), the leader's
// single MMA thread issues M = 256, N = 256 instructions that read both CTAs' shared memory, and each CTA's epilogue
// warps store the 128 rows its tensor memory holds.  Against 128 x 256 tiles of single CTAs this halves the B bytes
// an SM pulls from L2 per flop (a two-pass stage is 48 KB instead of 64 KB), which is what bounds the long products.
// Taken for plain dense products whose M and N are multiples of 256 (the launcher decides); everything else stays
// on k_gemm_tc.  Barriers per CTA: full[s] (used in the leader only: it counts the bytes of BOTH CTAs' loads of stage
// s - the peer's loads name the leader's barrier -, so one wait tells the MMA thread that the whole stage is
// there), empty[s] and the accumulator barrier (both arrived on by the leader's commits, in both CTAs).
// ---------------------------------------------------------------------------------------------
constexpr int kPairBarBytes = (3 * kGemmMaxStages + 1) * 8 + 32;

__global__ void __launch_bounds__(192) k_gemm_tc_pair(const __grid_constant__ GemmTcParams p) {
    constexpr int BN = 256;
    const uint32_t rank = cluster_ctarank();          // 0: leader, 1: peer
    const int ntn = (int)(gridDim.x >> 1);
    const int tn = (p.k_tri == 1) ? ntn - 1 - (int)(blockIdx.x >> 1) : (int)(blockIdx.x >> 1);
    const int m0 = (int)blockIdx.y * 256 + (int)rank * 128, n0 = tn * BN, z = blockIdx.z;
    // symmetric products: tiles entirely above the diagonal are not computed (both CTAs of the pair leave together,
    // before anything is shared between them)
    if (p.lower_only && tn > (int)blockIdx.y) return;
    const int crow0 = p.c_row0 + z * p.c_zrow + m0, ccol0 = p.c_col0 + z * p.c_zcol + n0;

    constexpr int kT = 128 * 64 * 2;                  // every operand tile of a CTA: 128 rows x 64 bf16
    const int stage_bytes = (p.nA + p.nB) * kT;
    const int STAGES = p.stages;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw);
    const uint32_t bars = base + STAGES * stage_bytes;        // full[S], empty[S], (unused [S]), accumulator
    const uint32_t bar_full = bars, bar_empty = bars + 8 * STAGES, bar_acc = bars + 24 * STAGES;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + STAGES * stage_bytes + (3 * STAGES + 1) * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* skip_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int kt_begin = 0, kt_end = (p.K + 63) / 64;
    if (p.k_tri == 1) kt_end = min(kt_end, (n0 + BN + 63) / 64);
    if (p.k_tri == 2) kt_begin = min(kt_end, n0 / 64);
    const int ktiles = kt_end - kt_begin;

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, 1);
        }
        mbar_init(bar_acc, 1);
        *abort_flag = 0;
        fence_barrier_init();
        // an earlier stage already failed: the leader reads the status word once and both CTAs take its branch
        // (the peer reads the leader's copy after the cluster barrier below)
        *skip_flag = p.status->code;
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), (uint32_t)BN);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tbase = *tmem_slot;
    const bool skip = ld_shared_cluster_u32(mapa_shared(smem_u32(const_cast<int*>(skip_flag)), 0)) != 0u;

    if (skip) {
        // nothing to do: fall through to the teardown
    } else if (warp == 0) {
        if (lane == 0) {
            const int ar = p.a_row0 + z * p.a_zrow + m0, ac = p.a_col0 + z * p.a_zcol;
            int br = p.b_row0 + z * p.b_zrow + n0;
            const int bc = p.b_col0 + z * p.b_zcol;
            int gsel = 0;
            if (p.ngrp > 1) {
                while (gsel + 1 < p.ngrp && n0 >= p.grp_end[gsel]) ++gsel;
                if (gsel > 0) br -= p.grp_end[gsel - 1];
            }
            br += (int)rank * 128;                    // this CTA's half of the B tile
            const uint32_t leader_full = mapa_shared(bar_full, 0);
            for (int it = 0; it < ktiles; ++it) {
                const int s = it % STAGES;
                if (!mbar_wait_cluster(bar_empty + 8 * s, ((it / STAGES) & 1) ^ 1, abort_flag, p.status, 11)) break;
                const int kt = kt_begin + it;
                const uint32_t full = leader_full + 8 * s;
                const uint32_t sa = base + s * stage_bytes;
                // the leader announces both CTAs' bytes (the peer's may be counted before this: the phase cannot
                // complete before the leader's arrival)
                if (rank == 0) mbar_expect_tx(bar_full + 8 * s, 2 * stage_bytes);
                for (int i = 0; i < p.nA; ++i) tma_load_2d_pair(sa + i * kT, &p.mapA[i], full, ac + kt * 64, ar);
                for (int i = 0; i < p.nB; ++i)
                    tma_load_2d_pair(sa + (p.nA + i) * kT, &p.mapB[p.ngrp > 1 ? gsel : i], full, bc + kt * 64, br);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = p.f16 ? idesc_f16(256, BN) : idesc_bf16(256, BN);
            const uint32_t peer_empty = mapa_shared(bar_empty, 1), peer_acc = mapa_shared(bar_acc, 1);
            bool ok = true;
            uint32_t used = 0u;
            for (int it = 0; it < ktiles; ++it) {
                const int s = it % STAGES;
                if (!mbar_wait_cluster(bar_full + 8 * s, (it / STAGES) & 1, abort_flag, p.status, 13)) { ok = false; break; }
                tc_fence_after();
                const uint32_t sa = base + s * stage_bytes;
                for (int ps = 0; ps < p.npass; ++ps) {
                    const uint64_t da = smem_desc_sw128(sa + p.pa[ps] * kT);
                    const uint64_t db = smem_desc_sw128(sa + (p.nA + p.pb[ps]) * kT);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        mma_f16_ss_pair(tbase, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, used);
                        used = 1u;
                    }
                }
                // the stage is free again in both CTAs once these MMAs have read it
                mma_commit_pair(bar_empty + 8 * s);
                mma_commit_pair(peer_empty + 8 * s);
            }
            if (ok) {
                mma_commit_pair(bar_acc);
                mma_commit_pair(peer_acc);
            }
        }
    } else {
        const int q = warp & 3;
        const int rl0 = m0 + q * 32;
        const int rowa0 = crow0 + q * 32;
        const int nrows = max(0, min(32, min(p.M - rl0, p.c_rows - rowa0)));
        float* const Cp = p.C_ind ? *p.C_ind : p.C;
        bool ok = true;
        if (ktiles > 0) {
            ok = mbar_wait_cluster(bar_acc, 0, abort_flag, p.status, 15);
            tc_fence_after();
        }
        if (ok) {
            float alpha = p.alpha;
            if (p.amax_a) alpha *= f16_inv_scale_from_max(*p.amax_a);
            if (p.amax_b) alpha *= f16_inv_scale_from_max(*p.amax_b);
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                if (ktiles > 0) {
                    tmem_ld32(tbase + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = 0u;
                }
                const int col = ccol0 + c0;
                if (min(p.N - (n0 + c0), p.c_cols - col) < 32) break;      // (the launcher only sends whole tiles)
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = alpha * __uint_as_float(r[j]);
                const size_t row = (size_t)(rowa0 + min(lane, max(nrows - 1, 0)));
                if (Cp && lane < nrows) {
                    float* crow = Cp + row * p.ldc + col;
                    if (p.addend) {
                        const float* arow = p.addend + row * p.ldadd + col;
                        float4 a4[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) a4[j] = *reinterpret_cast<const float4*>(arow + 4 * j);
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            v[4 * j] += a4[j].x; v[4 * j + 1] += a4[j].y; v[4 * j + 2] += a4[j].z; v[4 * j + 3] += a4[j].w;
                        }
                    }
                    if (p.accumulate && p.nout == 0) {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(crow + 4 * j), "f"(v[4 * j]),
                                         "f"(v[4 * j + 1]), "f"(v[4 * j + 2]), "f"(v[4 * j + 3])
                                         : "memory");
                    } else {
                        if (p.accumulate) {
                            float4 c4[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) c4[j] = *reinterpret_cast<const float4*>(crow + 4 * j);
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                v[4 * j] += c4[j].x; v[4 * j + 1] += c4[j].y; v[4 * j + 2] += c4[j].z; v[4 * j + 3] += c4[j].w;
                            }
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            *reinterpret_cast<float4*>(crow + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    }
                }
                if (p.nout > 0 && lane < nrows) store_parts_row(p, v, row * p.ldo + (col - p.out_col_off));
                __syncwarp();
            }
        }
    }
    // teardown: neither CTA may leave (its shared memory is read by the leader's MMAs, its barriers are arrived on
    // from the other CTA) before both are done; after an abort give copies in flight time to land first
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tbase, (uint32_t)BN);
    }
}

// Self-test of the bounded wait: the barrier below is initialised and never arrived on.
__global__ void k_selftest_wait(DevStatus* status) {
    __shared__ uint64_t bar_mem;
    __shared__ int abort_flag;
    const uint32_t bar = smem_u32(&bar_mem);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait(bar, 0, &abort_flag, status, 99, 2000000LL);   // ~1 ms
    __syncthreads();
}

void tc_selftest_wait(const Lc& lc, DevStatus* status) {
    k_selftest_wait<<<1, 32, 0, lc.st>>>(status);
    lc.count();
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

bool tc_encode_available() { return encode_fn() != nullptr; }

// bf16 matrix [rows][cols], row stride ld elements, tiles of box_rows x 64, 128-byte swizzle.
int tc_make_map_2d(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return PKV_ERR_UNSUPPORTED;
    if (((uintptr_t)ptr & 15) || (ld * 2) % 16 != 0 || rows == 0 || cols == 0) return PKV_ERR_INVALID_ARG;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t es[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PKV_OK : PKV_ERR_CUDA;
}

// bf16 tensor [d2][rows][cols] (strides ld1, ld2 elements), tiles of 1 x box_rows x 64.
int tc_make_map_3d(CUtensorMap* m, const void* ptr, uint64_t d2, uint64_t rows, uint64_t cols, uint64_t ld1,
                   uint64_t ld2, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return PKV_ERR_UNSUPPORTED;
    if (((uintptr_t)ptr & 15) || (ld1 * 2) % 16 != 0 || (ld2 * 2) % 16 != 0 || rows == 0 || cols == 0 || d2 == 0)
        return PKV_ERR_INVALID_ARG;
    cuuint64_t dims[3] = {cols, rows, d2};
    cuuint64_t strides[2] = {ld1 * 2, ld2 * 2};
    cuuint32_t box[3] = {64, box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PKV_OK : PKV_ERR_CUDA;
}

// Tensor maps of operands that keep their address and shape (workspace buffers, weights of the
// current block) are encoded once and reused.
struct MapCacheEntry {
    const void* ptr;
    uint64_t rows, cols, ld;
    uint32_t box;
    int valid;
    CUtensorMap map;
};
struct MapCache {
    static constexpr int kSize = 512;
    MapCacheEntry e[kSize];
};

MapCache* tc_map_cache_create() {
    MapCache* c = new (std::nothrow) MapCache();
    if (c) memset(c, 0, sizeof(*c));
    return c;
}
void tc_map_cache_destroy(MapCache* c) { delete c; }

static int cached_map(MapCache* cache, CUtensorMap* out, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld,
                      uint32_t box) {
    if (!cache) return tc_make_map_2d(out, ptr, rows, cols, ld, box);
    uint64_t h = (uint64_t)(uintptr_t)ptr * 0x9E3779B97F4A7C15ull ^ (rows * 0xC2B2AE3D27D4EB4Full) ^ (cols << 17) ^
                 (ld << 33) ^ box;
    h ^= h >> 29;
    for (int probe = 0; probe < 4; ++probe) {
        MapCacheEntry& e = cache->e[(h + probe) % MapCache::kSize];
        if (e.valid && e.ptr == ptr && e.rows == rows && e.cols == cols && e.ld == ld && e.box == box) {
            *out = e.map;
            return PKV_OK;
        }
    }
    int rc = tc_make_map_2d(out, ptr, rows, cols, ld, box);
    if (rc != PKV_OK) return rc;
    int slot = -1;
    for (int probe = 0; probe < 4; ++probe)
        if (!cache->e[(h + probe) % MapCache::kSize].valid) { slot = (int)((h + probe) % MapCache::kSize); break; }
    if (slot < 0) slot = (int)(h % MapCache::kSize);
    MapCacheEntry& e = cache->e[slot];
    e.ptr = ptr; e.rows = rows; e.cols = cols; e.ld = ld; e.box = box; e.map = *out; e.valid = 1;
    return PKV_OK;
}

template <int BN>
static int launch_gemm(const Lc& lc, GemmTcParams& p, int batch) {
    static PerDeviceOnce once;
    constexpr int kMaxSmem = 227 * 1024;
    int dev;
    if (once.needed(&dev)) {
        if (cudaFuncSetAttribute(k_gemm_tc<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess)
            return PKV_ERR_CUDA;
        once.mark(dev);
    }
    const int stage_bytes = p.nA * 128 * 128 + p.nB * BN * 128;
    const int fixed = kGemmBarBytes + 1024;
    const int ktiles = (p.K + 63) / 64;
    // Two CTAs per SM let one tile's epilogue overlap the other's main loop: taken when the contraction
    // is short (epilogue-bound) or when two stages still fit in half an SM's shared memory.
    const int half = 112 * 1024 - fixed;
    const long long ctas = (long long)((p.N + BN - 1) / BN) * ((p.M + 127) / 128) * batch;
    int stages;
    const bool one_per_sm = BN * p.nacc > 256;      // two CTAs of this kernel would not fit in the 512 TMEM columns
    if (ctas <= 148 || one_per_sm) stages = (kMaxSmem - fixed) / stage_bytes;      // occupancy is moot: deepest pipeline
    else if (ktiles <= 8 || 2 * stage_bytes <= half) stages = half / stage_bytes;
    else stages = (kMaxSmem - fixed) / stage_bytes;
    if (stages < 1) stages = 1;
    if (stages > kGemmMaxStages) stages = kGemmMaxStages;
    if (stages > ktiles) stages = ktiles > 0 ? ktiles : 1;
    p.stages = stages;
    int smem = stages * stage_bytes + fixed;
    if (one_per_sm && smem < 120 * 1024) smem = 120 * 1024;      // keeps a second CTA (and its TMEM request) off the SM
    dim3 grid((p.N + BN - 1) / BN, (p.M + 127) / 128, batch);
    if (lc.pdl) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = grid;
        cfg.blockDim = dim3(192);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = lc.st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, k_gemm_tc<BN>, p) != cudaSuccess) return PKV_ERR_CUDA;
    } else {
        k_gemm_tc<BN><<<grid, 192, smem, lc.st>>>(p);
    }
    lc.count();
    return PKV_OK;
}

// PKV_GEMM_PAIR=0 keeps every product on single CTAs; so does a cluster launch that the driver refused once (a
// device or an SM partition that cannot co-schedule two CTAs of this size).
static bool g_pair_refused = false;
static bool pair_enabled() {
    static const bool v = [] { const char* e = getenv("PKV_GEMM_PAIR"); return !e || atoi(e) != 0; }();
    return v && !g_pair_refused;
}

// Fewest 256 x 256 tiles for which a product goes to CTA pairs (PKV_GEMM_PAIR_MIN overrides).  Measured on the
// config-2 block, whose 512-row halves give 32 - 48 tiles per projection: 2.71 ms with 24, 2.72 - 2.73 with 60.
static int pair_min_tiles() {
    static const int v = [] { const char* e = getenv("PKV_GEMM_PAIR_MIN"); return e ? atoi(e) : 24; }();
    return v;
}

static int launch_gemm_pair(const Lc& lc, GemmTcParams& p, int batch) {
    static PerDeviceOnce once;
    constexpr int kMaxSmem = 227 * 1024;
    int dev;
    if (once.needed(&dev)) {
        if (cudaFuncSetAttribute(k_gemm_tc_pair, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem) != cudaSuccess)
            return PKV_ERR_CUDA;
        once.mark(dev);
    }
    const int stage_bytes = (p.nA + p.nB) * 128 * 128;
    const int fixed = kPairBarBytes + 1024;
    const int ktiles = (p.K + 63) / 64;
    int stages = (kMaxSmem - fixed) / stage_bytes;
    if (stages > kGemmMaxStages) stages = kGemmMaxStages;
    if (stages > ktiles) stages = ktiles > 0 ? ktiles : 1;
    if (stages < 1) return PKV_ERR_UNSUPPORTED;
    p.stages = stages;
    const int smem = stages * stage_bytes + fixed;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (p.N / 256), p.M / 256, batch);
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = lc.st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, k_gemm_tc_pair, p) != cudaSuccess) return PKV_ERR_CUDA;
    lc.count();
    return PKV_OK;
}

// (A persistent variant - one CTA per SM walking over the tiles with a second accumulator buffer so that one tile's
// epilogue overlaps the next tile's MMAs - was built and measured: statistics at d = F = 5120 1.12 vs 1.20 ms, a
// whole config-2 block 4.54 vs 4.39 ms.  The split-bf16 products are bound by operand traffic from L2 and, at few
// reference tokens, by the number of tiles, not by the epilogue; the simpler kernel stayed.)
int gemm_tc(const Lc& lc, const TcGemm& g, DevStatus* status) {
    if (g.M <= 0 || g.N <= 0 || g.batch <= 0) return PKV_OK;
    if (g.K < 0 || g.npass <= 0 || g.npass > kGemmMaxPass || (!g.C && g.nout == 0)) return PKV_ERR_INVALID_ARG;
    GemmTcParams p;
    // 128 x 256 tiles move a third fewer operand bytes per flop than 128 x 128: taken whenever they still fill most
    // of the SMs once (measured, three-pass products: 4096 x 2048 x 2048 607 vs 449 TFLOP/s executed, 4096 x 1024 x
    // 1024 358 vs 278; the earlier rule asked for two full waves)
    const long long tiles256 = (long long)((g.N + 255) / 256) * ((g.M + 127) / 128) * g.batch;
    // CTA pairs on 256 x 256 tiles for plain dense products of whole tiles (see k_gemm_tc_pair; its epilogue has the
    // 16-byte paths only); a lower-triangle-only product counts the tiles on and below the diagonal
    const bool c_vec = g.C && ((uintptr_t)g.C & 15) == 0 && g.ldc % 4 == 0 && g.c_col0 % 4 == 0 && g.c_zcol % 4 == 0 &&
                       (!g.addend || (((uintptr_t)g.addend & 15) == 0 && g.ldadd % 4 == 0));
    bool o_vec = g.nout > 0 && g.ldo % 8 == 0 && (g.c_col0 - g.out_col_off) % 8 == 0 && g.c_zcol % 8 == 0;
    for (int i = 0; i < g.nout; ++i) o_vec = o_vec && (((uintptr_t)g.out[i]) & 15) == 0;
    const long long tm = g.M / 256, tnn = g.N / 256;
    const long long pair_tiles = (g.lower_only ? (tm == tnn ? tm * (tm + 1) / 2 : 0) : tm * tnn) * g.batch;
    const bool pair = pair_enabled() && !lc.pdl && g.M % 256 == 0 && g.N % 256 == 0 && g.N >= 512 && g.a_tri == 0 && g.nacc <= 1 &&
                      !g.stamps && !g.skip_tile00 && !g.out_col0_only && (!g.lower_only || g.k_tri == 0) &&
                      g.c_rows >= g.c_row0 + (g.batch - 1) * g.c_zrow + g.M && g.c_cols >= g.c_col0 + (g.batch - 1) * g.c_zcol + g.N &&
                      pair_tiles >= pair_min_tiles() && (c_vec || !g.C) && (g.nout == 0 || o_vec);
    const bool wide = g.N >= 512 && tiles256 >= 120 && !g.lower_only && g.nacc < 4;
    const int BN = pair ? 256 : ((g.skip_tile00 || g.out_col0_only) ? 128 : ((g.N <= 64) ? 64 : (wide ? 256 : 128)));
    const int boxB = pair ? 128 : BN;
    MapCache* cache = (MapCache*)lc.map_cache;
    // distinct operands
    const __nv_bfloat16* da[3];
    const __nv_bfloat16* db[3];
    p.nA = p.nB = 0;
    for (int i = 0; i < g.npass; ++i) {
        int ia = -1, ib = -1;
        for (int k = 0; k < p.nA; ++k) if (da[k] == g.A[i].p) ia = k;
        for (int k = 0; k < p.nB; ++k) if (db[k] == g.B[i].p) ib = k;
        if (ia < 0) {
            if (p.nA == 3) return PKV_ERR_INVALID_ARG;
            int rc = cached_map(cache, &p.mapA[p.nA], g.A[i].p, g.A[i].rows, g.A[i].cols, g.A[i].ld, 128);
            if (rc != PKV_OK) return rc;
            da[p.nA] = g.A[i].p;
            ia = p.nA++;
        }
        if (ib < 0) {
            if (p.nB == 3) return PKV_ERR_INVALID_ARG;
            int rc = cached_map(cache, &p.mapB[p.nB], g.B[i].p, g.B[i].rows, g.B[i].cols, g.B[i].ld, boxB);
            if (rc != PKV_OK) return rc;
            db[p.nB] = g.B[i].p;
            ib = p.nB++;
        }
        p.pa[i] = ia;
        p.pb[i] = ib;
    }
    p.ngrp = 0;
    if (g.ngrp > 1) {
        // grouped B: one operand slot in shared memory, one tensor map per group
        if (g.ngrp > 3 || p.nB != 1) return PKV_ERR_INVALID_ARG;
        int end = 0;
        for (int k = 0; k < g.ngrp; ++k) {
            if (g.grp_n[k] <= 0 || g.grp_n[k] % BN != 0) return PKV_ERR_INVALID_ARG;
            int rc = cached_map(cache, &p.mapB[k], g.Bgrp[k].p, g.Bgrp[k].rows, g.Bgrp[k].cols, g.Bgrp[k].ld, boxB);
            if (rc != PKV_OK) return rc;
            end += g.grp_n[k];
            p.grp_end[k] = end;
        }
        if (end != g.N) return PKV_ERR_INVALID_ARG;
        p.ngrp = g.ngrp;
    }
    p.npass = g.npass; p.M = g.M; p.N = g.N; p.K = g.K;
    p.a_row0 = g.a_row0; p.a_col0 = g.a_col0; p.a_zrow = g.a_zrow; p.a_zcol = g.a_zcol;
    p.b_row0 = g.b_row0; p.b_col0 = g.b_col0; p.b_zrow = g.b_zrow; p.b_zcol = g.b_zcol;
    p.c_row0 = g.c_row0; p.c_col0 = g.c_col0; p.c_zrow = g.c_zrow; p.c_zcol = g.c_zcol;
    p.c_rows = g.c_rows; p.c_cols = g.c_cols;
    p.C = g.C; p.C_ind = g.C_ind; p.ldc = g.ldc; p.alpha = g.alpha; p.addend = g.addend; p.ldadd = g.ldadd;
    p.amax_a = g.amax_a; p.amax_b = g.amax_b; p.f16 = g.f16 ? 1 : 0;
    for (int i = 0; i < 3; ++i) p.out[i] = g.out[i];
    p.ldo = g.ldo; p.nout = g.nout; p.out_col_off = g.out_col_off;
    p.accumulate = g.accumulate ? 1 : 0;
    p.lower_only = g.lower_only ? 1 : 0;
    p.k_tri = g.k_tri;
    p.a_tri = g.a_tri;
    p.skip_tile00 = g.skip_tile00 ? 1 : 0;
    p.out_col0_only = g.out_col0_only ? 1 : 0;
    // several accumulators only for products with one hi x hi pass and cross passes, and only if they fit
    p.nacc = 1;
    if (g.nacc > 1 && g.npass >= 2 && p.pa[0] == 0 && p.pb[0] == 0) {
        int hh_passes = 0;
        for (int i = 0; i < g.npass; ++i) hh_passes += (p.pa[i] == 0 && p.pb[i] == 0) ? 1 : 0;
        if (hh_passes == 1) p.nacc = (g.nacc >= 4 && BN * 4 <= 512) ? 4 : (BN * 2 <= 512 ? 2 : 1);
    }
    p.vec_ok = (g.C && ((uintptr_t)g.C & 15) == 0 && g.ldc % 4 == 0 && g.c_col0 % 4 == 0 && g.c_zcol % 4 == 0 &&
                (!g.addend || (((uintptr_t)g.addend & 15) == 0 && g.ldadd % 4 == 0))) ? 1 : 0;
    p.status = status;
    p.stamps = g.stamps;
    p.out_vec = 0;
    if (g.nout > 0) {
        bool ok = g.ldo % 8 == 0 && (g.c_col0 - g.out_col_off) % 8 == 0 && g.c_zcol % 8 == 0;
        for (int i = 0; i < g.nout; ++i) ok = ok && (((uintptr_t)g.out[i]) & 15) == 0;
        // every row offset (c_row0 + z c_zrow + ...) * ldo is then a multiple of 8 elements as well
        p.out_vec = ok ? 1 : 0;
    }
    if (pair) {
        const int rc = launch_gemm_pair(lc, p, g.batch);
        if (rc != PKV_ERR_CUDA) return rc;
        cudaGetLastError();                 // the launch was refused: nothing ran; from now on single CTAs
        g_pair_refused = true;
        return gemm_tc(lc, g, status);
    }
    if (BN == 64) return launch_gemm<64>(lc, p, g.batch);
    if (BN == 256) return launch_gemm<256>(lc, p, g.batch);
    return launch_gemm<128>(lc, p, g.batch);
}

}  // namespace pkv
