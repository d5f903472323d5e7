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

#include "pkv_ptx.cuh"
#include "pkv_tc.h"

namespace pkv {

using namespace ptx;

struct alignas(64) GemmTcParams {
    CUtensorMap mapA[kGemmMaxPass];
    CUtensorMap mapB[kGemmMaxPass];
    int npass, M, N, K;
    float* C;
    long long ldc;
    float alpha;
    const float* addend;
    long long ldadd;
    int accumulate, lower_only, vec_ok;
    DevStatus* status;
};

template <int BN, int STAGES>
struct GemmSmem {
    static constexpr int kA = 128 * 64 * 2;
    static constexpr int kB = BN * 64 * 2;
    static constexpr int kStage = kA + kB;
    static constexpr int kBars = 2 * STAGES + 1;
    static constexpr int kTotal = STAGES * kStage + kBars * 8 + 16 + 1024;   // + alignment slack
};

template <int BN, int STAGES>
__global__ void __launch_bounds__(192) k_gemm_tc(const __grid_constant__ GemmTcParams p) {
    using S = GemmSmem<BN, STAGES>;
    const int m0 = blockIdx.y * 128, n0 = blockIdx.x * BN;
    if (p.lower_only && n0 > m0 + 127) return;
    if (p.status->code != 0) return;      // an earlier stage already failed: the call reports it

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - raw);
    const uint32_t bars = base + STAGES * S::kStage;          // full[STAGES], empty[STAGES], tmem_full
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + STAGES * S::kStage + S::kBars * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ktiles = (p.K + 63) / 64;
    const int total = p.npass * ktiles;

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(bars + 8 * i, 1);
            mbar_init(bars + 8 * (STAGES + i), 1);
        }
        mbar_init(bars + 8 * (2 * STAGES), 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            for (int ps = 0; ps < p.npass; ++ps) {
                prefetch_tmap(&p.mapA[ps]);
                prefetch_tmap(&p.mapB[ps]);
            }
            for (int it = 0; it < total; ++it) {
                const int s = it % STAGES;
                if (!mbar_wait(bars + 8 * (STAGES + s), ((it / STAGES) & 1) ^ 1, abort_flag, p.status, 1)) break;
                const int ps = it / ktiles, kt = it - ps * ktiles;
                const uint32_t full = bars + 8 * s;
                mbar_expect_tx(full, S::kStage);
                tma_load_2d(base + s * S::kStage, &p.mapA[ps], full, kt * 64, m0);
                tma_load_2d(base + s * S::kStage + S::kA, &p.mapB[ps], full, kt * 64, n0);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(128, BN);
            bool ok = true;
            for (int it = 0; it < total; ++it) {
                const int s = it % STAGES;
                if (!mbar_wait(bars + 8 * s, (it / STAGES) & 1, abort_flag, p.status, 2)) { ok = false; break; }
                tc_fence_after();
                const uint64_t da = smem_desc_sw128(base + s * S::kStage);
                const uint64_t db = smem_desc_sw128(base + s * S::kStage + S::kA);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    mma_bf16_ss(tbase, da + (uint64_t)(kk * 2), db + (uint64_t)(kk * 2), idesc, (it | kk) != 0);
                mma_commit(bars + 8 * (STAGES + s));
            }
            if (ok) mma_commit(bars + 8 * (2 * STAGES));
        }
    } else {
        const int q = warp & 3;
        const bool ok = mbar_wait(bars + 8 * (2 * STAGES), 0, abort_flag, p.status, 3);
        tc_fence_after();
        if (ok) {
            const int row = m0 + q * 32 + lane;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tbase + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
                tmem_ld_wait();
                if (row < p.M && n0 + c0 < p.N) {
                    float* crow = p.C + (size_t)row * p.ldc + n0 + c0;
                    const float* arow = p.addend ? p.addend + (size_t)row * p.ldadd + n0 + c0 : nullptr;
                    if (p.vec_ok && n0 + c0 + 32 <= p.N) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            float4 v = make_float4(p.alpha * __uint_as_float(r[j]), p.alpha * __uint_as_float(r[j + 1]),
                                                   p.alpha * __uint_as_float(r[j + 2]), p.alpha * __uint_as_float(r[j + 3]));
                            if (arow) {
                                float4 a = *reinterpret_cast<const float4*>(arow + j);
                                v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
                            }
                            if (p.accumulate) {
                                float4 c = *reinterpret_cast<const float4*>(crow + j);
                                v.x += c.x; v.y += c.y; v.z += c.z; v.w += c.w;
                            }
                            *reinterpret_cast<float4*>(crow + j) = v;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (n0 + c0 + j < p.N) {
                                float v = p.alpha * __uint_as_float(r[j]);
                                if (arow) v += arow[j];
                                if (p.accumulate) v += crow[j];
                                crow[j] = v;
                            }
                        }
                    }
                }
            }
        }
    }
    // teardown: after an abort give copies in flight time to land before the CTA's smem is released
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tbase, BN);
    }
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

template <int BN, int STAGES>
static int launch_gemm(const Lc& lc, const GemmTcParams& p) {
    using S = GemmSmem<BN, STAGES>;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(k_gemm_tc<BN, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kTotal) !=
            cudaSuccess)
            return PKV_ERR_CUDA;
        attr_set = true;
    }
    dim3 grid((p.N + BN - 1) / BN, (p.M + 127) / 128);
    k_gemm_tc<BN, STAGES><<<grid, 192, S::kTotal, lc.st>>>(p);
    lc.count();
    return PKV_OK;
}

int gemm_tc(const Lc& lc, const TcGemm& g, DevStatus* status) {
    if (g.M <= 0 || g.N <= 0) return PKV_OK;
    if (g.K <= 0 || g.npass <= 0 || g.npass > kGemmMaxPass) return PKV_ERR_INVALID_ARG;
    GemmTcParams p;
    const int BN = (g.N <= 64) ? 64 : 128;
    for (int i = 0; i < g.npass; ++i) {
        int rc = tc_make_map_2d(&p.mapA[i], g.A[i], g.M, g.K, g.lda[i], 128);
        if (rc != PKV_OK) return rc;
        rc = tc_make_map_2d(&p.mapB[i], g.B[i], g.N, g.K, g.ldb[i], BN);
        if (rc != PKV_OK) return rc;
    }
    p.npass = g.npass; p.M = g.M; p.N = g.N; p.K = g.K;
    p.C = g.C; p.ldc = g.ldc; p.alpha = g.alpha; p.addend = g.addend; p.ldadd = g.ldadd;
    p.accumulate = g.accumulate ? 1 : 0;
    p.lower_only = g.lower_only ? 1 : 0;
    p.vec_ok = (((uintptr_t)g.C & 15) == 0 && g.ldc % 4 == 0 &&
                (!g.addend || (((uintptr_t)g.addend & 15) == 0 && g.ldadd % 4 == 0))) ? 1 : 0;
    p.status = status;
    if (BN == 64) return launch_gemm<64, 4>(lc, p);
    return launch_gemm<128, 3>(lc, p);
}

}  // namespace pkv
