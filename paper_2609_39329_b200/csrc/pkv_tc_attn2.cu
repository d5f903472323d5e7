// Dual-cache attention, second-generation kernel for head dim 128 (sm_100a).
//
// One CTA owns TWO tiles of 128 query rows (same KV head, same stream, same key split), so every
// K/V tile fetched by TMA feeds 256 query rows, and two softmax warpgroups take turns against one
// MMA-issuing thread: while warpgroup 0 turns S0 into P0, the tensor core computes S1, and so on.
//
//   warp 0      TMA producer: both Q tiles (bf16 hi + lo) once; K tiles through one stage, V tiles
//               through two
//   warp 1      tcgen05.mma issuer.  S_g = Q_g,hi K^T + Q_g,lo K^T into TMEM; O_g += P_g V with P_g
//               read from TMEM (it overwrites S_g in place as packed bf16) and V as an MN-major
//               shared-memory operand straight from the cache layout
//   warps 2-5   softmax warpgroup of tile 0, warps 6-9 of tile 1: one thread per query row, the
//               whole S row in registers (single pass), exp2 with the row's reference maximum,
//               P -> TMEM.  O stays in TMEM across key tiles; it is rescaled (TMEM load, multiply,
//               store) only when some row of the warp saw a new maximum, which is rare after the
//               first tiles.  The reference is the exact running maximum (kRescaleThreshold = 0).
// TMEM: S0 S1 O0 O1, 128 columns each.  Every wait is bounded (see pkv_ptx.cuh).
#include <cuda.h>
#include <math.h>

#include "pkv_ptx.cuh"
#include "pkv_tc.h"
#include "pkv_tc_attn2_params.h"

namespace pkv {

using namespace ptx;

namespace a2 {
constexpr int HD = 128;
constexpr float kRescaleThreshold = 0.f;     // log2 units. 0 keeps the exact running maximum: the dominant key then has
                                             // p = 1, exact in bf16; a stale reference (e.g. 8) triples the output error
constexpr int kTile = 128 * HD * 2;            // 32 KB: one 128-row operand tile (two 64-column sub-tiles)
constexpr int kQ = 0;                          // Q0hi Q0lo Q1hi Q1lo
constexpr int kK = 4 * kTile;                  // one stage
constexpr int kV = 5 * kTile;                  // two stages
constexpr int kBar = 7 * kTile;
constexpr int kNumBar = 12;
constexpr int kTotal = kBar + kNumBar * 8 + 16 + 1024;
enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 2, B_VFULL = 3, B_VEMPTY = 5, B_SFULL = 7, B_PFULL = 9, B_ODONE = 11 };
}  // namespace a2

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint64_t desc_mn_sw128(uint32_t smem_addr, uint32_t lbo) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// D[tmem] (+)= A[tmem] * B[smem]: A holds bf16 pairs, one 32-bit column per two K elements.
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() {
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Fewer issue slots per score (the softmax warps are bound by instruction issue, not by any one pipe): the
// subtraction of the reference maximum as one packed instruction per pair, the running maximum three inputs at a
// time, the row sum straight from the packed bf16 pair (fp32 + bf16 -> fp32).
__device__ __forceinline__ uint64_t pack_f32x2(float a, float b) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void sub_f32x2(uint32_t a0, uint32_t a1, uint64_t mm, float& r0, float& r1) {
    asm("{ .reg .b64 t; mov.b64 t, {%2, %3}; sub.f32x2 t, t, %4; mov.b64 {%0, %1}, t; }"
        : "=f"(r0), "=f"(r1) : "r"(a0), "r"(a1), "l"(mm));
}
__device__ __forceinline__ float max3f(float a, uint32_t b, uint32_t c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(__uint_as_float(b)), "f"(__uint_as_float(c)));
    return r;
}
__device__ __forceinline__ void add_bf16x2(float& l0, float& l1, uint32_t pk) {
    asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %2; add.rn.f32.bf16 %0, lo, %0; add.rn.f32.bf16 %1, hi, %1; }"
        : "+f"(l0), "+f"(l1) : "r"(pk));
}

__global__ void __launch_bounds__(320, 1) k_attn_tc2(const __grid_constant__ Attn2Params p) {
    using namespace a2;
    {   // an earlier stage already failed: the call reports it.  One thread reads the status word so that the
        // whole CTA takes the same branch even if the word changes while the CTA starts.
        __shared__ int s_skip;
        if (threadIdx.x == 0) s_skip = p.status->code;
        __syncthreads();
        if (s_skip != 0) return;
    }
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw);
    const uint32_t bars = base + kBar;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + kBar + kNumBar * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kh = blockIdx.y;
    const int z = blockIdx.z + p.z0;
    const int stream = (z >= p.nsplitF) ? 1 : 0;
    const int split = stream ? z - p.nsplitF : z;
    const int r0 = blockIdx.x * 256;

    int Lc, crow0;
    if (stream == 0) {
        Lc = p.L;
        crow0 = 0;
    } else {
        crow0 = p.head_off[kh];
        Lc = p.head_off[kh + 1] - crow0;
    }
    const int nC = (Lc + 127) >> 7;
    const int tok_max = min(p.N - 1, (r0 + 255) / p.g);
    const int nN = (tok_max >> 7) + 1;                 // later reference tiles are invisible to these rows
    const int t_begin = split * p.tps;
    const int t_end = min(nC + nN, t_begin + p.tps);
    const int ntiles = max(0, t_end - t_begin);

    if (threadIdx.x == 0) {
        mbar_init(bar(B_QFULL), 1);
        mbar_init(bar(B_KFULL), 1);
        mbar_init(bar(B_KEMPTY), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B_VFULL + i), 1);
            mbar_init(bar(B_VEMPTY + i), 1);
            mbar_init(bar(B_SFULL + i), 1);
            mbar_init(bar(B_PFULL + i), 128);
        }
        mbar_init(bar(B_ODONE), 1);
        mbar_init(bar(B_ODONE + 1), 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_slot;

    if (warp == 0) {
        if (lane == 0 && ntiles > 0) {
            const int zq = stream * p.Hkv + kh;
            mbar_expect_tx(bar(B_QFULL), (p.q_f16 ? 2 : 4) * kTile);
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
                for (int sb = 0; sb < 2; ++sb) {
                    tma_load_3d(base + kQ + (2 * t) * kTile + sb * 16384, &p.mQhi, bar(B_QFULL), sb * 64, r0 + t * 128, zq);
                    if (!p.q_f16)
                        tma_load_3d(base + kQ + (2 * t + 1) * kTile + sb * 16384, &p.mQlo, bar(B_QFULL), sb * 64, r0 + t * 128, zq);
                }
            for (int j = 0; j < ntiles; ++j) {
                const int t = t_begin + j;
                if (!mbar_wait(bar(B_KEMPTY), (j & 1) ^ 1, abort_flag, p.status, 10)) break;
                mbar_expect_tx(bar(B_KFULL), kTile);
#pragma unroll
                for (int sb = 0; sb < 2; ++sb) {
                    const uint32_t kd = base + kK + sb * 16384;
                    if (t >= nC) tma_load_3d(kd, &p.mKn, bar(B_KFULL), sb * 64, (t - nC) * 128, zq);
                    else if (stream == 0) tma_load_3d(kd, &p.mK, bar(B_KFULL), sb * 64, t * 128, kh);
                    else tma_load_2d(kd, &p.mKc, bar(B_KFULL), sb * 64, crow0 + t * 128);
                }
                const int st = j & 1;
                if (!mbar_wait(bar(B_VEMPTY + st), ((j >> 1) & 1) ^ 1, abort_flag, p.status, 11)) break;
                mbar_expect_tx(bar(B_VFULL + st), kTile);
#pragma unroll
                for (int sb = 0; sb < 2; ++sb) {
                    const uint32_t vd = base + kV + st * kTile + sb * 16384;
                    if (t >= nC) tma_load_3d(vd, &p.mVn, bar(B_VFULL + st), sb * 64, (t - nC) * 128, zq);
                    else if (stream == 0) tma_load_3d(vd, &p.mV, bar(B_VFULL + st), sb * 64, t * 128, kh);
                    else tma_load_2d(vd, &p.mVc, bar(B_VFULL + st), sb * 64, crow0 + t * 128);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && ntiles > 0) {
            // fp16 mode: queries AND keys are fp16 (both operand format fields 0); the two operands of one MMA must
            // have the same 16-bit type
            const uint32_t idesc_qk = p.q_f16 ? (idesc_bf16(128, 128) & ~((7u << 7) | (7u << 10))) : idesc_bf16(128, 128);
            const int q_passes = p.q_f16 ? 1 : 2;
            constexpr uint32_t idesc_pv = idesc_bf16(128, HD) | (1u << 16);      // B operand MN-major
            auto issue_qk = [&](int gq) {
                const uint32_t kd = base + kK;
                for (int ps = 0; ps < q_passes; ++ps) {
                    const uint32_t qd = base + kQ + (2 * gq + ps) * kTile;
#pragma unroll
                    for (int ks = 0; ks < HD / 16; ++ks) {
                        const uint32_t off = (uint32_t)(ks >> 2) * 16384u + (uint32_t)(ks & 3) * 32u;
                        mma_bf16_ss(tbase + gq * 128u, smem_desc_sw128(qd + off), smem_desc_sw128(kd + off), idesc_qk,
                                    (ps | ks) != 0);
                    }
                }
                mma_commit(bar(B_SFULL + gq));
            };
            auto issue_pv = [&](int gq, int j) {
                const uint32_t vd = base + kV + (j & 1) * kTile;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)      // 16 keys per step: 8 packed columns of P, 16 rows of V
                    mma_bf16_ts(tbase + 256u + gq * 128u, tbase + gq * 128u + (uint32_t)ks * 8u,
                                desc_mn_sw128(vd + (uint32_t)ks * 2048u, 16384u), idesc_pv, (j | ks) != 0);
                mma_commit(bar(B_ODONE + gq));
            };
            bool ok = mbar_wait(bar(B_QFULL), 0, abort_flag, p.status, 20) &&
                      mbar_wait(bar(B_KFULL), 0, abort_flag, p.status, 21);
            if (ok) {
                tc_fence_after();
                issue_qk(0);
                issue_qk(1);
                mma_commit(bar(B_KEMPTY));
            }
            for (int j = 0; ok && j < ntiles; ++j) {
                const bool more = (j + 1 < ntiles);
                ok = mbar_wait(bar(B_VFULL + (j & 1)), (j >> 1) & 1, abort_flag, p.status, 22) &&
                     mbar_wait(bar(B_PFULL), j & 1, abort_flag, p.status, 23);
                if (!ok) break;
                tc_fence_after();
                issue_pv(0, j);
                if (more) {
                    ok = mbar_wait(bar(B_KFULL), (j + 1) & 1, abort_flag, p.status, 24);
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(0);
                }
                ok = mbar_wait(bar(B_PFULL + 1), j & 1, abort_flag, p.status, 25);
                if (!ok) break;
                tc_fence_after();
                issue_pv(1, j);
                mma_commit(bar(B_VEMPTY + (j & 1)));
                if (more) {
                    issue_qk(1);
                    mma_commit(bar(B_KEMPTY));
                }
            }
        }
    } else {
        const int gq = (warp - 2) >> 2;                 // query tile / warpgroup
        const int q = warp & 3;                         // TMEM lane quarter this warp may access
        const int row_in = q * 32 + lane;
        const int r = r0 + gq * 128 + row_in;
        const bool valid = r < p.rows;
        const int tok = valid ? r / p.g : 0;
        const int cs = valid ? p.tok_cs[tok] : 0;
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        const uint32_t tS = tbase + gq * 128u + lane_off;
        const uint32_t tO = tbase + 256u + gq * 128u + lane_off;
        float m_ref = -INFINITY, l = 0.f;
        bool ok = true;

        for (int j = 0; ok && j < ntiles; ++j) {
            const int t = t_begin + j;
            int lo = 0, hi = 128;
            const float* bias = nullptr;
            if (t < nC) {
                hi = min(128, Lc - t * 128);
                if (stream == 1 && p.bias) bias = p.bias + crow0 + t * 128;
            } else {
                const int jt = (t - nC) * 128;
                lo = max(0, cs - jt);
                hi = min(128, tok - jt + 1);
            }
            const bool need_mask = (lo > 0) || (hi < 128) || (bias != nullptr);
            ok = mbar_wait(bar(B_SFULL + gq), j & 1, abort_flag, p.status, 31);
            if (!ok) break;
            tc_fence_after();
            uint32_t s[128];
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) tmem_ld32(tS + (uint32_t)c0, *reinterpret_cast<uint32_t(*)[32]>(&s[c0]));
            tmem_ld_wait();
            if (need_mask) {
#pragma unroll
                for (int c = 0; c < 128; ++c) {
                    float v = __uint_as_float(s[c]);
                    if (bias && c < hi) v = fmaf(bias[c], 1.4426950408889634f, v);
                    s[c] = __float_as_uint((c >= lo && c < hi) ? v : -INFINITY);
                }
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
            for (int c = 0; c < 128; c += 8) {
                mx0 = max3f(mx0, s[c], s[c + 1]);
                mx1 = max3f(mx1, s[c + 2], s[c + 3]);
                mx2 = max3f(mx2, s[c + 4], s[c + 5]);
                mx3 = max3f(mx3, s[c + 6], s[c + 7]);
            }
            const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
            // reference maximum: the exact running maximum (moved whenever the tile's maximum exceeds it)
            float alpha = 1.f;
            const bool move = mx > m_ref + kRescaleThreshold;         // also true for the first finite maximum (m_ref = -inf)
            if (move) {
                alpha = ex2f(m_ref - mx);                // m_ref = -inf -> 0
                m_ref = mx;
            }
            const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
            float l0 = 0.f, l1 = 0.f;
            // P as packed bf16 pairs, written over the first half of s[] (entry c/2 is dead by then)
            const uint64_t mm = pack_f32x2(m_use, m_use);
#pragma unroll
            for (int c = 0; c < 128; c += 2) {
                float x0, x1;
                sub_f32x2(s[c], s[c + 1], mm, x0, x1);
                const float p0 = ex2f(x0), p1 = ex2f(x1);
                __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
                const uint32_t pk = *reinterpret_cast<uint32_t*>(&b);
                // the row sum uses the ROUNDED probabilities, the ones the P V product sees, so that the
                // rounding of a dominant key cancels between numerator and denominator
                add_bf16x2(l0, l1, pk);
                s[c >> 1] = pk;
            }
            l = l * alpha + (l0 + l1);
            // P overwrites S: the previous P V product must have finished reading it; O is then stable too
            const bool rescale = __any_sync(0xffffffffu, move) && (j > 0);
            if (j > 0) {
                ok = mbar_wait(bar(B_ODONE + gq), (j - 1) & 1, abort_flag, p.status, 32);
                if (!ok) break;
                tc_fence_after();
            }
            if (rescale) {
#pragma unroll 1
                for (int c0 = 0; c0 < HD; c0 += 32) {
                    uint32_t o[32];
                    tmem_ld32(tO + (uint32_t)c0, o);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    tmem_st32(tO + (uint32_t)c0, o);
                }
            }
            tmem_st32(tS, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
            tmem_st32(tS + 32u, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
            tmem_st_wait();
            tc_fence_before();
            mbar_arrive(bar(B_PFULL + gq));
        }
        if (ok && ntiles > 0) ok = mbar_wait(bar(B_ODONE + gq), (ntiles - 1) & 1, abort_flag, p.status, 33);
        if (ok) {
            tc_fence_after();
            const size_t pr = ((size_t)(stream ? p.zoffC + split : split) * p.Hkv + kh) * p.rows + r;
            if (valid) {
                p.part_m[pr] = (m_ref == -INFINITY) ? -INFINITY : m_ref * 0.6931471805599453f;   // natural-log units
                p.part_l[pr] = l;
            }
#pragma unroll 1
            for (int c0 = 0; c0 < HD; c0 += 32) {
                uint32_t o[32];
                if (ntiles > 0) {
                    tmem_ld32(tO + (uint32_t)c0, o);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = 0u;
                }
                if (valid) {
                    float4* po = reinterpret_cast<float4*>(p.part_O + pr * HD + c0);
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        po[i] = make_float4(__uint_as_float(o[4 * i]), __uint_as_float(o[4 * i + 1]),
                                            __uint_as_float(o[4 * i + 2]), __uint_as_float(o[4 * i + 3]));
                }
            }
        }
    }
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tbase, 512);
    }
}

int launch_attn2(const Lc& lc, const Attn2Params& p, int qpairs, int zcount) {
    static PerDeviceOnce once;
    int dev;
    if (once.needed(&dev)) {
        if (cudaFuncSetAttribute(k_attn_tc2, cudaFuncAttributeMaxDynamicSharedMemorySize, a2::kTotal) != cudaSuccess)
            return PKV_ERR_CUDA;
        once.mark(dev);
    }
    dim3 grid(qpairs, p.Hkv, zcount);
    k_attn_tc2<<<grid, 320, a2::kTotal, lc.st>>>(p);
    lc.count();
    return PKV_OK;
}

}  // namespace pkv
