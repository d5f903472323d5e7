// Dual-cache attention on the 5th-gen tensor cores (sm_100a).
//
// A CTA owns one tile of 128 query rows of one KV head of one stream (teacher: full cache,
// student: compact cache) and one split of that stream's key sequence.  Query row r stands for
// (token r / g, head kh*g + r % g), so one K/V tile serves the whole GQA group.  The key
// sequence is the cache, in tiles of 128 rows, followed by the reference tokens' own keys, in
// tiles of 128, visible causally inside the token's chunk.
//
//   warp 0    TMA producer: Q (bf16 hi + lo parts) once, then K and V tiles through 2-stage rings
//   warp 1    one thread issues tcgen05.mma: S = Q_hi K^T + Q_lo K^T into a double-buffered TMEM
//             accumulator, then O_tile = P V (V read as an MN-major operand straight from the
//             cache layout) into a third accumulator
//   warps 2-5 softmax: each thread owns one query row (one TMEM lane): row max, exp2, P -> bf16
//             into 128B-swizzled smem for the PV product, running (m, l) in fp32, O kept in
//             registers as alpha * O + O_tile
// Partial (m, l, O) per split go to global memory; the combine kernel merges the splits of both
// streams and forms dA = aF - aC in fp32.
#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>
#include <math.h>

#include "pkv_ptx.cuh"
#include <mutex>
#include <vector>

#include "pkv_tc.h"
#include "pkv_tc_attn2_params.h"

namespace pkv {

using namespace ptx;

// ---------------------------------------------------------------------------------------------
// operand preparation: RoPE (optional), query pre-scaling, bf16 hi/lo split, head-major layouts
// ---------------------------------------------------------------------------------------------
// q  -> hi/lo [2][Hkv][N*g][hd] (row = token*g + head-in-group), scaled by log2(e)/sqrt(hd)
// k,v-> bf16  [2][Hkv][N][hd]
// One thread per four consecutive rotation pairs (c .. c+3 and their partners at + hd/2): 16-byte loads, 8-byte
// stores.  All row strides are multiples of 4 floats and every base pointer is 16-byte aligned.
__device__ __forceinline__ uint2 pack4_f16(float a, float b, float c, float d) {
    const __half2 x = __floats2half2_rn(a, b), y = __floats2half2_rn(c, d);
    return make_uint2(*reinterpret_cast<const uint32_t*>(&x), *reinterpret_cast<const uint32_t*>(&y));
}
__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c, float d) {
    const __nv_bfloat162 x = __floats2bfloat162_rn(a, b), y = __floats2bfloat162_rn(c, d);
    return make_uint2(*reinterpret_cast<const uint32_t*>(&x), *reinterpret_cast<const uint32_t*>(&y));
}
__global__ void __launch_bounds__(256) k_attn_prep(const float* __restrict__ q, long long ldq,
                                                   const float* __restrict__ k, const float* __restrict__ v,
                                                   long long ldkv, const float* __restrict__ rope_tab, int N, int Hq,
                                                   int Hkv, int hd, int s_begin, int s_count, int q_f16,
                                                   __nv_bfloat16* __restrict__ qhi,
                                                   __nv_bfloat16* __restrict__ qlo, __nv_bfloat16* __restrict__ kn,
                                                   __nv_bfloat16* __restrict__ vn) {
    const int half = hd / 2, quads = half / 4;
    const int heads = Hq + 2 * Hkv;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t total = (size_t)s_count * N * heads * quads;
    if (i >= total) return;
    int c = (int)(i % quads) * 4;
    int h = (int)((i / quads) % heads);
    int row = (int)(i / ((size_t)quads * heads)) + s_begin * N;
    int s = row / N, tok = row % N;
    float co[4] = {1.f, 1.f, 1.f, 1.f}, si[4] = {0.f, 0.f, 0.f, 0.f};
    if (rope_tab) {      // (cos, sin) interleaved per pair
        const float4 t0 = *reinterpret_cast<const float4*>(rope_tab + 2 * ((size_t)tok * half + c));
        const float4 t1 = *reinterpret_cast<const float4*>(rope_tab + 2 * ((size_t)tok * half + c) + 4);
        co[0] = t0.x; si[0] = t0.y; co[1] = t0.z; si[1] = t0.w;
        co[2] = t1.x; si[2] = t1.y; co[3] = t1.z; si[3] = t1.w;
    }
    if (h < Hq) {
        const int g = Hq / Hkv;
        const float* p = q + (size_t)row * ldq + (size_t)h * hd + c;
        const float4 l4 = *reinterpret_cast<const float4*>(p), h4 = *reinterpret_cast<const float4*>(p + half);
        const float lo[4] = {l4.x, l4.y, l4.z, l4.w}, hi[4] = {h4.x, h4.y, h4.z, h4.w};
        const float sc = 1.4426950408889634f * rsqrtf((float)hd);
        float a[4], b[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            a[e] = (lo[e] * co[e] - hi[e] * si[e]) * sc;
            b[e] = (hi[e] * co[e] + lo[e] * si[e]) * sc;
        }
        int kh = h / g, hg = h % g;
        size_t o = (((size_t)s * Hkv + kh) * ((size_t)N * g) + (size_t)tok * g + hg) * hd + c;
        if (q_f16) {
            // one fp16 part (11 significant bits): the attention kernel multiplies it with the fp16 keys in one pass
            *reinterpret_cast<uint2*>(qhi + o) = pack4_f16(a[0], a[1], a[2], a[3]);
            *reinterpret_cast<uint2*>(qhi + o + half) = pack4_f16(b[0], b[1], b[2], b[3]);
        } else {
            float ar[4], br[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                ar[e] = a[e] - __bfloat162float(__float2bfloat16_rn(a[e]));
                br[e] = b[e] - __bfloat162float(__float2bfloat16_rn(b[e]));
            }
            *reinterpret_cast<uint2*>(qhi + o) = pack4_bf16(a[0], a[1], a[2], a[3]);
            *reinterpret_cast<uint2*>(qhi + o + half) = pack4_bf16(b[0], b[1], b[2], b[3]);
            *reinterpret_cast<uint2*>(qlo + o) = pack4_bf16(ar[0], ar[1], ar[2], ar[3]);
            *reinterpret_cast<uint2*>(qlo + o + half) = pack4_bf16(br[0], br[1], br[2], br[3]);
        }
    } else if (h < Hq + Hkv) {
        int kh = h - Hq;
        const float* p = k + (size_t)row * ldkv + (size_t)kh * hd + c;
        const float4 l4 = *reinterpret_cast<const float4*>(p), h4 = *reinterpret_cast<const float4*>(p + half);
        const float lo[4] = {l4.x, l4.y, l4.z, l4.w}, hi[4] = {h4.x, h4.y, h4.z, h4.w};
        float a[4], b[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            a[e] = lo[e] * co[e] - hi[e] * si[e];
            b[e] = hi[e] * co[e] + lo[e] * si[e];
        }
        size_t o = (((size_t)s * Hkv + kh) * N + tok) * hd + c;
        if (q_f16) {
            *reinterpret_cast<uint2*>(kn + o) = pack4_f16(a[0], a[1], a[2], a[3]);
            *reinterpret_cast<uint2*>(kn + o + half) = pack4_f16(b[0], b[1], b[2], b[3]);
        } else {
            *reinterpret_cast<uint2*>(kn + o) = pack4_bf16(a[0], a[1], a[2], a[3]);
            *reinterpret_cast<uint2*>(kn + o + half) = pack4_bf16(b[0], b[1], b[2], b[3]);
        }
    } else {
        int kh = h - Hq - Hkv;
        const float* p = v + (size_t)row * ldkv + (size_t)kh * hd + c;
        const float4 l4 = *reinterpret_cast<const float4*>(p), h4 = *reinterpret_cast<const float4*>(p + half);
        size_t o = (((size_t)s * Hkv + kh) * N + tok) * hd + c;
        *reinterpret_cast<uint2*>(vn + o) = pack4_bf16(l4.x, l4.y, l4.z, l4.w);
        *reinterpret_cast<uint2*>(vn + o + half) = pack4_bf16(h4.x, h4.y, h4.z, h4.w);
    }
}

// bf16 -> fp16, eight elements per thread.  Exact for every bf16 value of magnitude in [2^-14, 65504] (8 significant
// bits fit in fp16's 11); smaller magnitudes round to fp16 subnormals (absolute error below 3e-8).
// A bf16 value is exact in fp16 when its magnitude is inside fp16's range (keys of a cache are; below 6e-8 they
// flush towards zero, which no logit notices).  A key beyond 65504 or not finite would turn into an infinity:
// the call reports PKV_ERR_NONFINITE instead (such a cache needs the bf16-pair path, PKV_ATTN_Q=pair).
__global__ void __launch_bounds__(256) k_bf16_to_f16(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t n8,
                                                     DevStatus* status) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n8) return;
    const uint4 v = src[i];
    const uint32_t in[4] = {v.x, v.y, v.z, v.w};
    uint32_t out[4];
    bool bad = false;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const float lo = __uint_as_float(in[e] << 16), hi = __uint_as_float(in[e] & 0xffff0000u);
        bad = bad || !(fabsf(lo) <= 65504.f) || !(fabsf(hi) <= 65504.f);
        const __half2 h = __floats2half2_rn(lo, hi);
        out[e] = *reinterpret_cast<const uint32_t*>(&h);
    }
    dst[i] = make_uint4(out[0], out[1], out[2], out[3]);
    if (bad) atomicCAS(&status->code, 0, PKV_ERR_NONFINITE);
}

static void to_f16(const Lc& lc, const void* src, void* dst, size_t elems, DevStatus* status) {
    const size_t n8 = elems / 8;
    if (!n8) return;
    k_bf16_to_f16<<<(unsigned)((n8 + 255) / 256), 256, 0, lc.st>>>((const uint4*)src, (uint4*)dst, n8, status);
    lc.count();
}

// ---------------------------------------------------------------------------------------------
// the attention kernel
// ---------------------------------------------------------------------------------------------
struct alignas(64) AttnTcParams {
    CUtensorMap mQhi, mQlo;   // {hd, N*g, 2*Hkv}
    CUtensorMap mK, mV;       // {hd, L, Hkv}
    CUtensorMap mKc, mVc;     // {hd, total kept rows}
    CUtensorMap mKn, mVn;     // {hd, N, 2*Hkv}
    const int32_t* head_off;
    const int32_t* tok_cs;
    const float* bias;
    int N, g, Hkv, L, rows;
    int tps, nsplitF, nsplitC;
    int z0, zoffC;
    float* part_m;
    float* part_l;
    float* part_O;
    DevStatus* status;
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// MN-major operand (V tile: rows = keys, 64 head-dim columns per 128-byte row, 128B swizzle):
// 64-column blocks `lbo` bytes apart, 8-key groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t smem_addr, uint32_t lbo) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

template <int HD>
struct AttnSmem {
    static constexpr int kSub = HD / 64;              // 64-column sub-tiles per row
    static constexpr int kTile = 128 * HD * 2;        // one 128-row operand tile, bytes
    static constexpr int kQhi = 0;
    static constexpr int kQlo = kTile;
    static constexpr int kK = 2 * kTile;              // 2 stages
    static constexpr int kV = 4 * kTile;              // 2 stages
    static constexpr int kP = 6 * kTile;              // [2][128][64] bf16 = 32 KB
    static constexpr int kBar = kP + 32768;
    static constexpr int kNumBar = 16;
    static constexpr int kTotal = kBar + kNumBar * 8 + 16 + 1024;
};

enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 3, B_VFULL = 5, B_VEMPTY = 7, B_SFULL = 9, B_SEMPTY = 11, B_PFULL = 13,
       B_OFULL = 14, B_OEMPTY = 15 };

template <int HD>
__global__ void __launch_bounds__(192, 1) k_attn_tc(const __grid_constant__ AttnTcParams p) {
    using S = AttnSmem<HD>;
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
    const uint32_t bars = base + S::kBar;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + S::kBar + S::kNumBar * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kh = blockIdx.y;
    const int z = blockIdx.z + p.z0;
    const int stream = (z >= p.nsplitF) ? 1 : 0;
    const int split = stream ? z - p.nsplitF : z;
    const int r0 = blockIdx.x * 128;

    // key tiles of this CTA: cache tiles [0, nC) then reference-token tiles [nC, nC + nN)
    int Lc, crow0;
    if (stream == 0) {
        Lc = p.L;
        crow0 = 0;
    } else {
        crow0 = p.head_off[kh];
        Lc = p.head_off[kh + 1] - crow0;
    }
    const int nC = (Lc + 127) >> 7;
    const int tok_max = min(p.N - 1, (r0 + 127) / p.g);
    const int nN = (tok_max >> 7) + 1;                 // later reference tiles are invisible to this row tile
    const int t_begin = split * p.tps;
    const int t_end = min(nC + nN, t_begin + p.tps);
    const int ntiles = max(0, t_end - t_begin);

    if (threadIdx.x == 0) {
        mbar_init(bar(B_QFULL), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B_KFULL + i), 1);
            mbar_init(bar(B_KEMPTY + i), 1);
            mbar_init(bar(B_VFULL + i), 1);
            mbar_init(bar(B_VEMPTY + i), 1);
            mbar_init(bar(B_SFULL + i), 1);
            mbar_init(bar(B_SEMPTY + i), 128);
        }
        mbar_init(bar(B_PFULL), 128);
        mbar_init(bar(B_OFULL), 1);
        mbar_init(bar(B_OEMPTY), 128);
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
    const uint32_t tS[2] = {tbase, tbase + 128u};
    const uint32_t tO = tbase + 256u;

    if (warp == 0) {
        if (lane == 0 && ntiles > 0) {
            const int zq = stream * p.Hkv + kh;
            mbar_expect_tx(bar(B_QFULL), 2 * S::kTile);
#pragma unroll
            for (int sb = 0; sb < S::kSub; ++sb) {
                tma_load_3d(base + S::kQhi + sb * 16384, &p.mQhi, bar(B_QFULL), sb * 64, r0, zq);
                tma_load_3d(base + S::kQlo + sb * 16384, &p.mQlo, bar(B_QFULL), sb * 64, r0, zq);
            }
            for (int j = 0; j < ntiles; ++j) {
                const int t = t_begin + j;
                const int st = j & 1;
                const uint32_t ph = ((j >> 1) & 1) ^ 1;
                if (!mbar_wait(bar(B_KEMPTY + st), ph, abort_flag, p.status, 10)) break;
                mbar_expect_tx(bar(B_KFULL + st), S::kTile);
                const uint32_t kd = base + S::kK + st * S::kTile;
#pragma unroll
                for (int sb = 0; sb < S::kSub; ++sb) {
                    if (t >= nC) tma_load_3d(kd + sb * 16384, &p.mKn, bar(B_KFULL + st), sb * 64, (t - nC) * 128, zq);
                    else if (stream == 0) tma_load_3d(kd + sb * 16384, &p.mK, bar(B_KFULL + st), sb * 64, t * 128, kh);
                    else tma_load_2d(kd + sb * 16384, &p.mKc, bar(B_KFULL + st), sb * 64, crow0 + t * 128);
                }
                if (!mbar_wait(bar(B_VEMPTY + st), ph, abort_flag, p.status, 11)) break;
                mbar_expect_tx(bar(B_VFULL + st), S::kTile);
                const uint32_t vd = base + S::kV + st * S::kTile;
#pragma unroll
                for (int sb = 0; sb < S::kSub; ++sb) {
                    if (t >= nC) tma_load_3d(vd + sb * 16384, &p.mVn, bar(B_VFULL + st), sb * 64, (t - nC) * 128, zq);
                    else if (stream == 0) tma_load_3d(vd + sb * 16384, &p.mV, bar(B_VFULL + st), sb * 64, t * 128, kh);
                    else tma_load_2d(vd + sb * 16384, &p.mVc, bar(B_VFULL + st), sb * 64, crow0 + t * 128);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && ntiles > 0) {
            constexpr uint32_t idesc_qk = idesc_bf16(128, 128);
            constexpr uint32_t idesc_pv = idesc_bf16(128, HD) | (1u << 16);      // B operand MN-major
            auto issue_qk = [&](int j) {
                const int st = j & 1;
                const uint32_t kd = base + S::kK + st * S::kTile;
#pragma unroll
                for (int ps = 0; ps < 2; ++ps) {
                    const uint32_t qd = base + (ps ? S::kQlo : S::kQhi);
#pragma unroll
                    for (int ks = 0; ks < HD / 16; ++ks) {
                        const uint32_t off = (uint32_t)(ks >> 2) * 16384u + (uint32_t)(ks & 3) * 32u;
                        mma_bf16_ss(tS[st], smem_desc_sw128(qd + off), smem_desc_sw128(kd + off), idesc_qk,
                                    (ps | ks) != 0);
                    }
                }
                mma_commit(bar(B_SFULL + st));
                mma_commit(bar(B_KEMPTY + st));
            };
            bool ok = mbar_wait(bar(B_QFULL), 0, abort_flag, p.status, 20) &&
                      mbar_wait(bar(B_KFULL), 0, abort_flag, p.status, 21);
            if (ok) {
                tc_fence_after();
                issue_qk(0);
            }
            for (int j = 0; ok && j < ntiles; ++j) {
                if (j + 1 < ntiles) {
                    const int n = j + 1, st = n & 1;
                    ok = mbar_wait(bar(B_KFULL + st), (n >> 1) & 1, abort_flag, p.status, 22) &&
                         mbar_wait(bar(B_SEMPTY + st), ((n >> 1) & 1) ^ 1, abort_flag, p.status, 23);
                    if (!ok) break;
                    tc_fence_after();
                    issue_qk(n);
                }
                const int st = j & 1;
                ok = mbar_wait(bar(B_VFULL + st), (j >> 1) & 1, abort_flag, p.status, 24) &&
                     mbar_wait(bar(B_PFULL), j & 1, abort_flag, p.status, 25) &&
                     mbar_wait(bar(B_OEMPTY), (j & 1) ^ 1, abort_flag, p.status, 26);
                if (!ok) break;
                tc_fence_after();
                const uint32_t vd = base + S::kV + st * S::kTile;
                const uint32_t pd = base + S::kP;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {      // 16 keys per step
                    const uint64_t da = smem_desc_sw128(pd + (uint32_t)(ks >> 2) * 16384u + (uint32_t)(ks & 3) * 32u);
                    const uint64_t db = smem_desc_mn_sw128(vd + (uint32_t)ks * 2048u, 16384u);
                    mma_bf16_ss(tO, da, db, idesc_pv, ks != 0);
                }
                mma_commit(bar(B_OFULL));
                mma_commit(bar(B_VEMPTY + st));
            }
        }
    } else {
        const int q = warp & 3;
        const int row_in = q * 32 + lane;
        const int r = r0 + row_in;
        const bool valid = r < p.rows;
        const int tok = valid ? r / p.g : 0;
        const int cs = valid ? p.tok_cs[tok] : 0;
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        float m = -INFINITY, l = 0.f, alpha_pend = 1.f;
        float O[HD];
#pragma unroll
        for (int i = 0; i < HD; ++i) O[i] = 0.f;
        bool ok = true;

        auto accumulate_o = [&](int j) {
            ok = mbar_wait(bar(B_OFULL), j & 1, abort_flag, p.status, 30);
            if (!ok) return;
            tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < HD; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tO + lane_off + (uint32_t)c0, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) O[c0 + i] = fmaf(alpha_pend, O[c0 + i], __uint_as_float(v[i]));
            }
            tc_fence_before();
            mbar_arrive(bar(B_OEMPTY));
        };

        for (int j = 0; ok && j < ntiles; ++j) {
            const int t = t_begin + j;
            const int st = j & 1;
            // visible key columns [lo, hi) of this tile for this row
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
            ok = mbar_wait(bar(B_SFULL + st), (j >> 1) & 1, abort_flag, p.status, 31);
            if (!ok) break;
            tc_fence_after();
            // pass 1: row maximum
            float mx = -INFINITY;
#pragma unroll 1
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tS[st] + lane_off + (uint32_t)c0, v);
                tmem_ld_wait();
                if (need_mask) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int c = c0 + i;
                        float s = __uint_as_float(v[i]);
                        if (bias && c < hi) s = fmaf(bias[c], 1.4426950408889634f, s);
                        mx = fmaxf(mx, (c >= lo && c < hi) ? s : -INFINITY);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(v[i]));
                }
            }
            const float m_new = fmaxf(m, mx);
            const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
            const float alpha = ex2(m - m_safe);              // m = -inf -> 0
            // fold in the previous tile's P V product (it also frees the P buffer)
            if (j > 0) accumulate_o(j - 1);
            if (!ok) break;
            // pass 2: P = 2^(S - m) as bf16 into swizzled smem, row sum
            float ls = 0.f;
            uint8_t* prow = sm + S::kP + row_in * 128;
#pragma unroll 1
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tS[st] + lane_off + (uint32_t)c0, v);
                tmem_ld_wait();
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    float s0 = __uint_as_float(v[i]), s1 = __uint_as_float(v[i + 1]);
                    if (need_mask) {
                        const int c = c0 + i;
                        if (bias && c < hi) s0 = fmaf(bias[c], 1.4426950408889634f, s0);
                        if (bias && c + 1 < hi) s1 = fmaf(bias[c + 1], 1.4426950408889634f, s1);
                        if (!(c >= lo && c < hi)) s0 = -INFINITY;
                        if (!(c + 1 >= lo && c + 1 < hi)) s1 = -INFINITY;
                    }
                    const float p0 = ex2(s0 - m_safe), p1 = ex2(s1 - m_safe);
                    ls += p0 + p1;
                    __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
                    pk[i >> 1] = *reinterpret_cast<uint32_t*>(&b);
                }
                // 32 columns = 4 chunks of 16 bytes; chunk index inside the 64-column sub-tile is
                // XOR-swizzled with the row (128B swizzle), sub-tiles are 16 KB apart
                uint8_t* psub = prow + (c0 >> 6) * 16384;
                const int ch0 = (c0 & 63) >> 3;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint4 val = make_uint4(pk[ch * 4], pk[ch * 4 + 1], pk[ch * 4 + 2], pk[ch * 4 + 3]);
                    *reinterpret_cast<uint4*>(psub + (((ch0 + ch) ^ (row_in & 7)) << 4)) = val;
                }
            }
            l = l * alpha + ls;
            m = m_new;
            alpha_pend = alpha;
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(bar(B_PFULL));
            mbar_arrive(bar(B_SEMPTY + st));
        }
        if (ok && ntiles > 0) accumulate_o(ntiles - 1);
        if (valid && ok) {
            const size_t pr = ((size_t)(stream ? p.zoffC + split : split) * p.Hkv + kh) * p.rows + r;
            p.part_m[pr] = (m == -INFINITY) ? -INFINITY : m * 0.6931471805599453f;   // back to natural-log units
            p.part_l[pr] = l;
            float4* po = reinterpret_cast<float4*>(p.part_O + pr * HD);
#pragma unroll
            for (int i = 0; i < HD / 4; ++i) po[i] = make_float4(O[4 * i], O[4 * i + 1], O[4 * i + 2], O[4 * i + 3]);
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

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
// Split planning.  Every CTA takes one (query tile pair, KV head, split) and `tps` key tiles; CTAs are handed to
// the SMs in grid order (all units of the teacher's first split, then its second, ..., then the student's).
// With one CTA per SM (hd = 128: the kernel owns all of tensor memory) the time is that of the last SM to
// finish, and a split count that leaves a nearly empty last round (3.03 rounds of 148) wastes a quarter of the
// machine: the planner therefore replays that hand-out for every candidate split count, each CTA costing its key
// tiles plus a fixed part (prologue, partial results written and merged later), and keeps the cheapest.  The
// choice depends on the context's dimensions only (N_max, b_max), so that buffers sized once fit every call.
constexpr long long kAttnWaves = 3;         // hd = 64: CTAs of the teacher stream ~ kAttnWaves x the SM count
constexpr int kAttnCtaOverheadTiles = 4;    // fixed cost of a CTA in units of one key tile's work
constexpr int kAttnTeacherReserve = 12;     // SMs the stack driver's teacher stream leaves free by default

static long long attn_makespan(int slots, long long base, long long tF, long long tC, long long t) {
    // min-heap of the slots' free times; CTAs in grid order
    std::vector<long long> heap((size_t)slots, 0);
    auto push_cta = [&](long long cost) {
        // replace the smallest element (heap[0]) by heap[0] + cost and restore the heap
        long long v = heap[0] + cost;
        size_t i = 0, n = heap.size();
        for (;;) {
            size_t l = 2 * i + 1, r = l + 1, m = i;
            long long mv = v;
            if (l < n && heap[l] < mv) { m = l; mv = heap[l]; }
            if (r < n && heap[r] < mv) { m = r; mv = heap[r]; }
            if (m == i) break;
            heap[i] = heap[m];
            i = m;
        }
        heap[i] = v;
    };
    for (long long done = 0; done < tF; done += t)
        for (long long u = 0; u < base; ++u) push_cta(kAttnCtaOverheadTiles + (tF - done < t ? tF - done : t));
    for (long long done = 0; done < tC; done += t)
        for (long long u = 0; u < base; ++u) push_cta(kAttnCtaOverheadTiles + (tC - done < t ? tC - done : t));
    long long worst = 0;
    for (long long v : heap) worst = v > worst ? v : worst;
    return worst;
}

// tps for one launch mode (0: both streams, 1: teacher only, 2: student only); remembered per (dimensions, mode)
static long long attn_tps(const pkv_dims* d, int mode) {
    const int g = d->Hq / d->Hkv;
    const int rows_per_cta = (d->hd == 128) ? 256 : 128;     // the hd = 128 kernel owns two query tiles
    const long long qtiles = ((long long)d->N_max * g + rows_per_cta - 1) / rows_per_cta;
    const long long base = qtiles * d->Hkv;
    const long long tilesF = (d->L + 127) / 128 + (d->N_max + 127) / 128;
    if (d->hd != 128) {
        long long want = (kAttnWaves * 148 + base - 1) / base;
        if (want < 1) want = 1;
        if (want > 64) want = 64;
        const long long t = (tilesF + want - 1) / want;
        return t < 4 ? 4 : t;
    }
    struct Seen { pkv_dims d; long long t; };
    static std::mutex mu;
    static Seen seen[3] = {};
    std::lock_guard<std::mutex> lock(mu);
    Seen& e = seen[mode];
    if (e.t > 0 && e.d.L == d->L && e.d.N_max == d->N_max && e.d.b_max == d->b_max && e.d.Hq == d->Hq && e.d.Hkv == d->Hkv &&
        e.d.hd == d->hd)
        return e.t;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        sms <= 0) {
        cudaGetLastError();
        sms = 148;
    }
    // the teacher alone runs on its stream's SM partition (all SMs but the default reserve of the stack driver)
    const int slots = (mode == 1 && sms > kAttnTeacherReserve) ? sms - kAttnTeacherReserve : sms;
    const long long tF = (mode == 2) ? 0 : tilesF;
    const long long tC = (mode == 1) ? 0 : (d->b_max + 127) / 128 + (d->N_max + 127) / 128;
    const long long longest = tF > tC ? tF : tC;
    long long best = -1, best_t = longest;
    for (long long sp = 1; sp <= 64; ++sp) {
        long long cand = (longest + sp - 1) / sp;
        if (cand < 4) cand = 4;
        if (base * ((tF + cand - 1) / cand + (tC + cand - 1) / cand) > 262144) break;   // keep the replay cheap
        const long long cost = attn_makespan(slots, base, tF, tC, cand);
        if (best < 0 || cost < best) { best = cost; best_t = cand; }
        if (cand == 4) break;
    }
    e.d = *d;
    e.t = best_t;
    if (getenv("PKV_ATTN_TRACE"))
        fprintf(stderr, "attention plan, mode %d on %d SMs: %lld units, %lld + %lld key tiles -> %lld tiles per split, modelled time %lld tile units\n",
                mode, slots, base, tF, tC, best_t, best);
    return best_t;
}

static void attn_counts(const pkv_dims* d, int N, int max_b, long long t, int* nF, int* nC) {
    const long long tF = (d->L + 127) / 128 + (N + 127) / 128;
    const long long tC = (max_b + 127) / 128 + (N + 127) / 128;
    *nF = (int)((tF + t - 1) / t);
    *nC = (int)((tC + t - 1) / t);
    if (*nC < 1) *nC = 1;
}

// Partials of the teacher's splits sit at [0, nsplitF), those of the student's at [zoffC, zoffC + nsplitC): zoffC is
// the largest teacher split count of any mode at the context's N_max, so that a teacher-only launch of one block
// and a student-only launch of another (stack driver) never share a slot.
void tc_attn_plan(const pkv_dims* d, int N, int max_b, int mode, int* tps, int* nsplitF, int* nsplitC, int* zoffC) {
    const long long t = attn_tps(d, mode);
    *tps = (int)t;
    attn_counts(d, N, max_b, t, nsplitF, nsplitC);
    int z = 0;
    for (int m = 0; m < 2; ++m) {
        int nF, nC;
        attn_counts(d, d->N_max, d->b_max, attn_tps(d, m), &nF, &nC);
        if (nF > z) z = nF;
    }
    *zoffC = z;
}

// Split slots the partial buffers must hold.
int tc_attn_partial_slots(const pkv_dims* d) {
    int z = 0, c = 0;
    for (int m = 0; m < 3; ++m) {
        int nF, nC;
        attn_counts(d, d->N_max, d->b_max, attn_tps(d, m), &nF, &nC);
        if (m != 2 && nF > z) z = nF;
        if (m != 1 && nC > c) c = nC;
    }
    return z + c;
}

template <int HD>
static int launch_attn(const Lc& lc, const AttnTcParams& p, int qtiles, int zcount) {
    using S = AttnSmem<HD>;
    static PerDeviceOnce once;
    int dev;
    if (once.needed(&dev)) {
        if (cudaFuncSetAttribute(k_attn_tc<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kTotal) != cudaSuccess)
            return PKV_ERR_CUDA;
        once.mark(dev);
    }
    dim3 grid(qtiles, p.Hkv, zcount);
    k_attn_tc<HD><<<grid, 192, S::kTotal, lc.st>>>(p);
    lc.count();
    return PKV_OK;
}

// Query operand of the hd = 128 kernel: one fp16 part (default) or a bf16 hi + lo pair (PKV_ATTN_Q=pair)
static bool attn_q_f16() {
    static const bool v = [] { const char* e = getenv("PKV_ATTN_Q"); return !(e && e[0] == 'p'); }();
    return v;
}

// hd = 128: the two-tile kernel of pkv_tc_attn2.cu (operands already prepared in t->q, t->kn, t->vn)
int launch_attn2(const Lc& lc, const Attn2Params& p, int qpairs, int zcount);
static int attention_tc2(const Lc& lc, TcBuffers* t, const pkv_dims* d, const AttnArgs& a, DevStatus* status) {
    const int N = a.N, hd = d->hd, Hkv = d->Hkv, g = d->Hq / d->Hkv;
    const int rows = N * g;
    Attn2Params p;
    int rc;
    if ((rc = tc_make_map_3d(&p.mQhi, t->q.hi, 2 * Hkv, rows, hd, hd, (uint64_t)rows * hd, 128))) return rc;
    if ((rc = tc_make_map_3d(&p.mQlo, t->q.lo, 2 * Hkv, rows, hd, hd, (uint64_t)rows * hd, 128))) return rc;
    if ((rc = tc_make_map_3d(&p.mKn, t->kn, 2 * Hkv, N, hd, hd, (uint64_t)N * hd, 128))) return rc;
    if ((rc = tc_make_map_3d(&p.mVn, t->vn, 2 * Hkv, N, hd, hd, (uint64_t)N * hd, 128))) return rc;
    // fp16 mode: the key operands are fp16 copies of the (bf16) caches, made here; values stay bf16
    const bool f16 = attn_q_f16();
    const void* Kfull = a.K;
    const void* Kcomp = a.Kc;
    if (f16) {
        if (d->L > 0 && a.mode != 2) {
            to_f16(lc, a.K, t->K16, (size_t)Hkv * d->L * hd, status);
            Kfull = t->K16;
        } else {
            Kfull = t->K16;
        }
        if (a.total_kept > 0 && a.mode != 1) to_f16(lc, a.Kc, t->Kc16, (size_t)a.total_kept * hd, status);
        Kcomp = t->Kc16;
    }
    if (d->L > 0) {
        if ((rc = tc_make_map_3d(&p.mK, Kfull, Hkv, d->L, hd, hd, (uint64_t)d->L * hd, 128))) return rc;
        if ((rc = tc_make_map_3d(&p.mV, a.V, Hkv, d->L, hd, hd, (uint64_t)d->L * hd, 128))) return rc;
    } else {
        p.mK = p.mKn;
        p.mV = p.mVn;
    }
    if (a.total_kept > 0) {
        if ((rc = tc_make_map_2d(&p.mKc, Kcomp, a.total_kept, hd, hd, 128))) return rc;
        if ((rc = tc_make_map_2d(&p.mVc, a.Vc, a.total_kept, hd, hd, 128))) return rc;
    } else {
        p.mKc = p.mKn;      // never read: no compact-cache tiles exist
        p.mVc = p.mVn;
    }
    p.head_off = a.head_off; p.tok_cs = a.tok_cs; p.bias = a.bias;
    p.N = N; p.g = g; p.Hkv = Hkv; p.L = d->L; p.rows = rows;
    tc_attn_plan(d, N, a.max_b, a.mode, &p.tps, &p.nsplitF, &p.nsplitC, &p.zoffC);
    p.part_m = t->part_m; p.part_l = t->part_l; p.part_O = t->part_O;
    p.status = status;
    p.z0 = (a.mode == 2) ? p.nsplitF : 0;
    p.q_f16 = f16 ? 1 : 0;
    rc = launch_attn2(lc, p, (rows + 255) / 256,
                      a.mode == 0 ? p.nsplitF + p.nsplitC : (a.mode == 1 ? p.nsplitF : p.nsplitC));
    if (rc != PKV_OK) return rc;
    AttnArgs c = a;
    c.nsplitF = p.nsplitF; c.nsplitC = p.nsplitC; c.zoffC = p.zoffC;
    c.part_m = t->part_m; c.part_l = t->part_l; c.part_O = t->part_O;
    attention_combine(lc, c);
    return PKV_OK;
}

int attention_tc(const Lc& lc, TcBuffers* t, const pkv_dims* d, const AttnArgs& a, const float* rope_tab,
                 DevStatus* status) {
    const int N = a.N, hd = d->hd, Hkv = d->Hkv, g = d->Hq / d->Hkv;
    const int rows = N * g;
    const int s_begin = (a.mode == 2) ? 1 : 0, s_count = (a.mode == 0) ? 2 : 1;
    {
        size_t total = (size_t)s_count * N * (d->Hq + 2 * Hkv) * (hd / 8);      // four rotation pairs per thread
        k_attn_prep<<<(unsigned)((total + 255) / 256), 256, 0, lc.st>>>(a.q, a.ldq, a.k_new, a.v_new, a.ldkv, rope_tab, N,
                                                                        d->Hq, Hkv, hd, s_begin, s_count,
                                                                        (hd == 128 && attn_q_f16()) ? 1 : 0, t->q.hi, t->q.lo,
                                                                        t->kn, t->vn);
        lc.count();
    }
    if (hd == 128) return attention_tc2(lc, t, d, a, status);
    AttnTcParams p;
    int rc;
    if ((rc = tc_make_map_3d(&p.mQhi, t->q.hi, 2 * Hkv, rows, hd, hd, (uint64_t)rows * hd, 128))) return rc;
    if ((rc = tc_make_map_3d(&p.mQlo, t->q.lo, 2 * Hkv, rows, hd, hd, (uint64_t)rows * hd, 128))) return rc;
    if ((rc = tc_make_map_3d(&p.mKn, t->kn, 2 * Hkv, N, hd, hd, (uint64_t)N * hd, 128))) return rc;
    if ((rc = tc_make_map_3d(&p.mVn, t->vn, 2 * Hkv, N, hd, hd, (uint64_t)N * hd, 128))) return rc;
    if (d->L > 0) {
        if ((rc = tc_make_map_3d(&p.mK, a.K, Hkv, d->L, hd, hd, (uint64_t)d->L * hd, 128))) return rc;
        if ((rc = tc_make_map_3d(&p.mV, a.V, Hkv, d->L, hd, hd, (uint64_t)d->L * hd, 128))) return rc;
    } else {
        p.mK = p.mKn;
        p.mV = p.mVn;
    }
    const int total_kept = a.total_kept;
    if (total_kept > 0) {
        if ((rc = tc_make_map_2d(&p.mKc, a.Kc, total_kept, hd, hd, 128))) return rc;
        if ((rc = tc_make_map_2d(&p.mVc, a.Vc, total_kept, hd, hd, 128))) return rc;
    } else {
        p.mKc = p.mKn;      // never read: no compact-cache tiles exist
        p.mVc = p.mVn;
    }
    p.head_off = a.head_off; p.tok_cs = a.tok_cs; p.bias = a.bias;
    p.N = N; p.g = g; p.Hkv = Hkv; p.L = d->L; p.rows = rows;
    tc_attn_plan(d, N, a.max_b, a.mode, &p.tps, &p.nsplitF, &p.nsplitC, &p.zoffC);
    p.part_m = t->part_m; p.part_l = t->part_l; p.part_O = t->part_O;
    p.status = status;
    const int qtiles = (rows + 127) / 128;
    p.z0 = (a.mode == 2) ? p.nsplitF : 0;
    const int zcount = a.mode == 0 ? p.nsplitF + p.nsplitC : (a.mode == 1 ? p.nsplitF : p.nsplitC);
    rc = launch_attn<64>(lc, p, qtiles, zcount);      // hd = 128 left above for the two-tile kernel
    if (rc != PKV_OK) return rc;
    AttnArgs c = a;
    c.nsplitF = p.nsplitF; c.nsplitC = p.nsplitC; c.zoffC = p.zoffC;
    c.part_m = t->part_m; c.part_l = t->part_l; c.part_O = t->part_O;
    attention_combine(lc, c);
    return PKV_OK;
}

}  // namespace pkv
