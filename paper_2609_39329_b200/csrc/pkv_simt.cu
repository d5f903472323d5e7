// SIMT fp32 kernels: index check + compaction, norms, rotary embedding, a tiled fp32 GEMM, a
// tiled flash-style attention with split-K partials, the split-K combine (which also forms
// dA = aF - aC before any rounding), element-wise epilogues, reductions and the merge.
//
// These kernels are the whole path for fp32 weights/caches and an on-device cross-check of the
// tensor-core kernels for bf16 (PKV_ENGINE_SIMT).  Nothing here traps: invalid inputs set a
// status word and the offending access is skipped.
#include <math.h>

#include "pkv_internal.h"

namespace pkv {

__device__ __forceinline__ float ld_as_float(const float* p) { return *p; }
__device__ __forceinline__ float ld_as_float(const __nv_bfloat16* p) { return __bfloat162float(*p); }

__device__ __forceinline__ void raise(DevStatus* s, int code) { atomicCAS(&s->code, 0, code); }

// ------------------------------------------------------------------------------------------
// index check + compaction (bit-exact)
// ------------------------------------------------------------------------------------------
// One warp per kept row.  Row i of head h is valid iff 0 <= idx[i] < L and it exceeds its
// predecessor inside the head.  Invalid rows are reported (smallest flat position wins) and not
// copied.  Copies move 16-byte chunks, so K/V rows must be 16-byte multiples (hd*elem >= 16).
__global__ void __launch_bounds__(256) k_gather_kept(const uint4* __restrict__ K, const uint4* __restrict__ V,
                                                     const int32_t* __restrict__ idx,
                                                     const int32_t* __restrict__ head_off, int Hkv, int L,
                                                     int row_chunks, int total, uint4* __restrict__ Kc,
                                                     uint4* __restrict__ Vc, DevStatus* status) {
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (warp >= total) return;
    int h = 0;
    while (h + 1 < Hkv && head_off[h + 1] <= warp) ++h;
    int v = idx[warp];
    bool ok = v >= 0 && v < L;
    if (ok && warp > head_off[h]) ok = v > idx[warp - 1];
    if (!ok) {
        if (lane == 0) {
            raise(status, PKV_ERR_BAD_INDEX);
            unsigned long long key = (unsigned long long)warp + 1ull;
            unsigned long long old = status->bad_index;
            while (old == 0ull || key < old) {
                unsigned long long prev = atomicCAS(&status->bad_index, old, key);
                if (prev == old) break;
                old = prev;
            }
        }
        return;
    }
    const uint4* ks = K + ((size_t)h * L + v) * row_chunks;
    const uint4* vs = V + ((size_t)h * L + v) * row_chunks;
    uint4* kd = Kc + (size_t)warp * row_chunks;
    uint4* vd = Vc + (size_t)warp * row_chunks;
    for (int c = lane; c < row_chunks; c += 32) {
        kd[c] = ks[c];
        vd[c] = vs[c];
    }
}

void gather_kept(const Lc& lc, int elem_bytes, const void* K, const void* V, const int32_t* idx,
                 const int32_t* head_off_dev, int Hkv, int L, int hd, int total, void* Kc, void* Vc,
                 DevStatus* status) {
    if (total <= 0) return;
    int row_chunks = hd * elem_bytes / 16;
    int warps_per_block = 8;
    int blocks = (total + warps_per_block - 1) / warps_per_block;
    k_gather_kept<<<blocks, 256, 0, lc.st>>>((const uint4*)K, (const uint4*)V, idx, head_off_dev, Hkv, L,
                                             row_chunks, total, (uint4*)Kc, (uint4*)Vc, status);
    lc.count();
}

// Quantised compact cache (appendix, quantised caches): codes are signed integers, 8 bits (one byte per element)
// or 4 bits (two per byte, even element in the low nibble, two's complement), with one fp32 scale per
// `group` consecutive elements of a row; an element decodes to scale * code, rounded to the cache's element
// type.  One thread decodes eight elements (a 16-byte bf16 store or two 16-byte fp32 stores).
template <typename T>
__global__ void __launch_bounds__(256) k_dequant_rows(const uint8_t* __restrict__ codes, const float* __restrict__ scales,
                                                      int bits, int group, int hd, size_t rows, T* __restrict__ out) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;      // chunk of eight elements
    const int chunks = hd / 8;
    if (i >= rows * (size_t)chunks) return;
    const size_t r = i / chunks;
    const int c0 = (int)(i % chunks) * 8;
    const float* sc = scales + r * (size_t)(hd / group);
    float v[8];
    if (bits == 8) {
        const int8_t* q = reinterpret_cast<const int8_t*>(codes) + r * (size_t)hd + c0;
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = sc[(c0 + e) / group] * (float)q[e];
    } else {
        const uint8_t* q = codes + r * (size_t)(hd / 2) + c0 / 2;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint8_t byte = q[e >> 1];
            int nib = (e & 1) ? (byte >> 4) : (byte & 15);
            nib = (nib ^ 8) - 8;                                 // sign-extend the 4-bit two's complement code
            v[e] = sc[(c0 + e) / group] * (float)nib;
        }
    }
    T* o = out + r * (size_t)hd + c0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        if constexpr (sizeof(T) == 2) o[e] = __float2bfloat16_rn(v[e]);
        else o[e] = v[e];
    }
}

void dequant_cache(const Lc& lc, int elem_bytes, const void* codes, const float* scales, int bits, int group, int hd,
                   int rows, void* out) {
    if (rows <= 0) return;
    const size_t n = (size_t)rows * (hd / 8);
    const unsigned blocks = (unsigned)((n + 255) / 256);
    if (elem_bytes == 2)
        k_dequant_rows<__nv_bfloat16><<<blocks, 256, 0, lc.st>>>((const uint8_t*)codes, scales, bits, group, hd, (size_t)rows,
                                                                  (__nv_bfloat16*)out);
    else
        k_dequant_rows<float><<<blocks, 256, 0, lc.st>>>((const uint8_t*)codes, scales, bits, group, hd, (size_t)rows, (float*)out);
    lc.count();
}

// ------------------------------------------------------------------------------------------
// RMSNorm
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float block_sum(float v, float* red) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    __syncthreads();
    if (l == 0) red[w] = v;
    __syncthreads();
    float t = (threadIdx.x < (blockDim.x >> 5)) ? red[threadIdx.x] : 0.f;
    if (w == 0) {
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (l == 0) red[0] = t;
    }
    __syncthreads();
    return red[0];
}

__global__ void __launch_bounds__(256) k_rmsnorm_f32(const float* __restrict__ x0, const float* __restrict__ x1,
                                                     int N, int d, const float* __restrict__ gain, float eps,
                                                     float* __restrict__ out) {
    __shared__ float red[32];
    int r = blockIdx.x;
    const float* x = (r < N) ? x0 + (size_t)r * d : x1 + (size_t)(r - N) * d;
    float ss = 0.f;
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
        float v = x[c];
        ss += v * v;
    }
    float tot = block_sum(ss, red);
    float inv = 1.0f / sqrtf(tot / (float)d + eps);
    for (int c = threadIdx.x; c < d; c += blockDim.x) out[(size_t)r * d + c] = x[c] * gain[c] * inv;
}

void rmsnorm_f32(const Lc& lc, const float* x0, const float* x1, int N, int d, const float* gain, float eps,
                 float* out) {
    k_rmsnorm_f32<<<2 * N, 256, 0, lc.st>>>(x0, x1, N, d, gain, eps, out);
    lc.count();
}

// ------------------------------------------------------------------------------------------
// tiled fp32 GEMM, C = alpha * A B^T (+ addend) (+ C)
// ------------------------------------------------------------------------------------------
template <typename TB>
__global__ void __launch_bounds__(256) k_gemm_tn(const float* __restrict__ A, int64_t lda,
                                                 const TB* __restrict__ B, int64_t ldb, float* C, int64_t ldc,
                                                 int M, int N, int K, float alpha, const float* addend,
                                                 int64_t ldadd, int accumulate, int lower_only) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    int bm = blockIdx.y * BM, bn = blockIdx.x * BN;
    if (lower_only && bn > bm + BM - 1) return;
    int tid = threadIdx.x;
    int tx = tid & 15, ty = tid >> 4;
    int lr = tid >> 2, lk = (tid & 3) * 4;     // loader: row 0..63, k offset 0,4,8,12
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < K; k0 += BK) {
        float av[4] = {0.f, 0.f, 0.f, 0.f}, bv[4] = {0.f, 0.f, 0.f, 0.f};
        int ar = bm + lr, br = bn + lr;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int kk = k0 + lk + i;
            if (ar < M && kk < K) av[i] = A[(size_t)ar * lda + kk];
            if (br < N && kk < K) bv[i] = ld_as_float(B + (size_t)br * ldb + kk);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            As[lk + i][lr] = av[i];
            Bs[lk + i][lr] = bv[i];
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int r = bm + ty * 4 + i;
        if (r >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int c = bn + tx * 4 + j;
            if (c >= N) continue;
            float v = alpha * acc[i][j];
            if (addend) v += addend[(size_t)r * ldadd + c];
            if (accumulate) v += C[(size_t)r * ldc + c];
            C[(size_t)r * ldc + c] = v;
        }
    }
}

void gemm_tn_simt(const Lc& lc, const float* A, int64_t lda, const void* B, int64_t ldb, bool b_bf16, float* C,
                  int64_t ldc, int M, int N, int K, float alpha, const float* addend, int64_t ldadd,
                  bool accumulate, bool lower_only) {
    if (M <= 0 || N <= 0) return;
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    if (b_bf16)
        k_gemm_tn<__nv_bfloat16><<<grid, 256, 0, lc.st>>>(A, lda, (const __nv_bfloat16*)B, ldb, C, ldc, M, N, K,
                                                          alpha, addend, ldadd, accumulate, lower_only);
    else
        k_gemm_tn<float><<<grid, 256, 0, lc.st>>>(A, lda, (const float*)B, ldb, C, ldc, M, N, K, alpha, addend,
                                                  ldadd, accumulate, lower_only);
    lc.count();
}

// ------------------------------------------------------------------------------------------
// rotary embedding: half-split pairs (c, c + hd/2), angle pos * theta^(-2c/hd)
// ------------------------------------------------------------------------------------------
// The angle is formed in double precision: at positions near 2e5 an fp32 product pos*freq
// would already be off by ~1e-2 rad.
__global__ void k_rope_table(const int32_t* __restrict__ tok_cs, int N, int hd, int pos0, double theta,
                             float* __restrict__ tab) {
    int half = hd / 2;
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N * half) return;
    int tok = i / half, c = i % half;
    double pos = (double)pos0 + (double)(tok - tok_cs[tok]);
    double ang = (theta > 0.0) ? pos * pow(theta, -2.0 * (double)c / (double)hd) : 0.0;
    double s, co;
    sincos(ang, &s, &co);
    tab[2 * (size_t)i] = (float)co;
    tab[2 * (size_t)i + 1] = (float)s;
}

void rope_table(const Lc& lc, const int32_t* tok_cs, int N, int hd, int pos0, float theta, float* cs_table) {
    int n = N * (hd / 2);
    k_rope_table<<<(n + 255) / 256, 256, 0, lc.st>>>(tok_cs, N, hd, pos0, (double)theta, cs_table);
    lc.count();
}

__global__ void k_rope_apply(float* __restrict__ buf, int64_t ld, int col0, int heads, int hd, int rows, int N,
                             const float* __restrict__ tab) {
    int half = hd / 2;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t total = (size_t)rows * heads * half;
    if (i >= total) return;
    int c = (int)(i % half);
    int h = (int)((i / half) % heads);
    int r = (int)(i / ((size_t)half * heads));
    int tok = r % N;
    float co = tab[2 * ((size_t)tok * half + c)], s = tab[2 * ((size_t)tok * half + c) + 1];
    float* p = buf + (size_t)r * ld + col0 + h * hd + c;
    float lo = p[0], hi = p[half];
    p[0] = lo * co - hi * s;
    p[half] = hi * co + lo * s;
}

void rope_apply(const Lc& lc, float* buf, int64_t ld, int col0, int heads, int hd, int rows, int N,
                const float* cs_table) {
    size_t total = (size_t)rows * heads * (hd / 2);
    k_rope_apply<<<(unsigned)((total + 255) / 256), 256, 0, lc.st>>>(buf, ld, col0, heads, hd, rows, N, cs_table);
    lc.count();
}

// ------------------------------------------------------------------------------------------
// attention, SIMT fp32: tile of 32 query rows x 32 keys, online softmax, split-K partials
// ------------------------------------------------------------------------------------------
// Query row r of KV head kh stands for (token r / g, head kh*g + r % g) so that one key/value
// tile serves the whole GQA group.  The key sequence of a stream is its cache rows followed by
// the N reference tokens; reference key j is visible to token t iff chunk_start(t) <= j <= t.
template <typename TC, int HD>
__global__ void __launch_bounds__(128) k_attn_simt(AttnArgs a) {
    constexpr int BM = 32, BN = 32;
    extern __shared__ float sm[];
    float* Qs = sm;                          // [BM][HD+1]
    float* Ks = Qs + BM * (HD + 1);          // [BN][HD+1]
    float* Vs = Ks + BN * (HD + 1);          // [BN][HD]
    float* Ss = Vs + BN * HD;                // [BM][BN+1]
    int* row_tok = (int*)(Ss + BM * (BN + 1));   // [BM]
    int* row_cs = row_tok + BM;                  // [BM]

    const int tid = threadIdx.x;
    const int kh = blockIdx.y;
    const int z = blockIdx.z;
    const int stream = (z >= a.nsplitF) ? 1 : 0;
    const int split = stream ? z - a.nsplitF : z;
    const int g = a.Hq / a.Hkv;
    const int rows = a.N * g;
    const int r0 = blockIdx.x * BM;

    const TC* Kbase;
    const TC* Vbase;
    const float* bias = nullptr;
    int Lc_rows;
    if (stream == 0) {
        Kbase = (const TC*)a.K + (size_t)kh * a.L * HD;
        Vbase = (const TC*)a.V + (size_t)kh * a.L * HD;
        Lc_rows = a.L;
    } else {
        int off = a.head_off[kh];
        Kbase = (const TC*)a.Kc + (size_t)off * HD;
        Vbase = (const TC*)a.Vc + (size_t)off * HD;
        Lc_rows = a.head_off[kh + 1] - off;
        if (a.bias) bias = a.bias + off;
    }
    const int Lt = Lc_rows + a.N;
    const int k_begin = split * a.kv_split;
    const int k_end = min(Lt, k_begin + a.kv_split);
    const float scale = rsqrtf((float)HD);

    if (tid < BM) {
        int r = r0 + tid;
        int tok = (r < rows) ? r / g : 0;
        row_tok[tid] = (r < rows) ? tok : -1;
        row_cs[tid] = (r < rows) ? a.tok_cs[tok] : 0;
    }
    for (int i = tid; i < BM * HD; i += 128) {
        int rr = i / HD, c = i % HD;
        int r = r0 + rr;
        float v = 0.f;
        if (r < rows) {
            int tok = r / g, hg = r % g;
            v = a.q[((size_t)stream * a.N + tok) * a.ldq + (size_t)(kh * g + hg) * HD + c] * scale;
        }
        Qs[rr * (HD + 1) + c] = v;
    }

    const int row = tid >> 2, sub = tid & 3;
    float m = -INFINITY, l = 0.f;
    float O[HD / 4];
#pragma unroll
    for (int i = 0; i < HD / 4; ++i) O[i] = 0.f;

    for (int kt = k_begin; kt < k_end; kt += BN) {
        __syncthreads();
        for (int i = tid; i < BN * HD; i += 128) {
            int key = i / HD, c = i % HD;
            int kk = kt + key;
            float kv = 0.f, vv = 0.f;
            if (kk < k_end) {
                if (kk < Lc_rows) {
                    kv = ld_as_float(Kbase + (size_t)kk * HD + c);
                    vv = ld_as_float(Vbase + (size_t)kk * HD + c);
                } else {
                    size_t rr = ((size_t)stream * a.N + (kk - Lc_rows)) * a.ldkv + (size_t)kh * HD + c;
                    kv = a.k_new[rr];
                    vv = a.v_new[rr];
                }
            }
            Ks[key * (HD + 1) + c] = kv;
            Vs[key * HD + c] = vv;
        }
        __syncthreads();
        {   // scores: 2 rows x 4 keys per thread
            int ty = tid >> 3, tx = tid & 7;
            float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
            const float* q0 = Qs + (ty * 2) * (HD + 1);
            const float* q1 = q0 + (HD + 1);
            const float* kp = Ks + (tx * 4) * (HD + 1);
#pragma unroll 8
            for (int c = 0; c < HD; ++c) {
                float a0 = q0[c], a1 = q1[c];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float kvv = kp[j * (HD + 1) + c];
                    s[0][j] = fmaf(a0, kvv, s[0][j]);
                    s[1][j] = fmaf(a1, kvv, s[1][j]);
                }
            }
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                int rr = ty * 2 + i;
                int tok = row_tok[rr], cs = row_cs[rr];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    int kk = kt + tx * 4 + j;
                    float v = s[i][j];
                    bool vis = (kk < k_end) && (tok >= 0);
                    if (vis) {
                        if (kk < Lc_rows) {
                            if (bias) v += bias[kk];
                        } else {
                            int jn = kk - Lc_rows;
                            vis = (jn >= cs) && (jn <= tok);
                        }
                    }
                    Ss[rr * (BN + 1) + tx * 4 + j] = vis ? v : -INFINITY;
                }
            }
        }
        __syncthreads();
        {   // online softmax for `row`, 8 keys per thread, 4 threads per row (same warp)
            float* sr = Ss + row * (BN + 1) + sub * 8;
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 8; ++j) mx = fmaxf(mx, sr[j]);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            float m_new = fmaxf(m, mx);
            float alpha = 1.f, ps = 0.f;
            if (m_new == -INFINITY) {
#pragma unroll
                for (int j = 0; j < 8; ++j) sr[j] = 0.f;
            } else {
                alpha = expf(m - m_new);          // m = -inf -> 0
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float p = expf(sr[j] - m_new);
                    sr[j] = p;
                    ps += p;
                }
            }
            ps += __shfl_xor_sync(0xffffffffu, ps, 1);
            ps += __shfl_xor_sync(0xffffffffu, ps, 2);
            l = l * alpha + ps;
            m = m_new;
            __syncwarp();
#pragma unroll
            for (int i = 0; i < HD / 4; ++i) O[i] *= alpha;
            const float* pr = Ss + row * (BN + 1);
            for (int k = 0; k < BN; ++k) {
                float p = pr[k];
                const float* vr = Vs + k * HD + sub;
#pragma unroll
                for (int i = 0; i < HD / 4; ++i) O[i] = fmaf(p, vr[i * 4], O[i]);
            }
        }
    }
    int r = r0 + row;
    if (r < rows) {
        size_t pr = ((size_t)z * a.Hkv + kh) * rows + r;
        if (sub == 0) {
            a.part_m[pr] = m;
            a.part_l[pr] = l;
        }
        float* po = a.part_O + pr * HD;
#pragma unroll
        for (int i = 0; i < HD / 4; ++i) po[i * 4 + sub] = O[i];
    }
}

template <typename TC, int HD>
static void launch_attn_simt(const Lc& lc, const AttnArgs& a) {
    int g = a.Hq / a.Hkv;
    int rows = a.N * g;
    dim3 grid((rows + 31) / 32, a.Hkv, a.nsplitF + a.nsplitC);
    size_t smem = (size_t)(32 * (HD + 1) * 2 + 32 * HD + 32 * 33) * sizeof(float) + 64 * sizeof(int);
    cudaFuncSetAttribute(k_attn_simt<TC, HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    k_attn_simt<TC, HD><<<grid, 128, smem, lc.st>>>(a);
    lc.count();
}

void attention_simt(const Lc& lc, const AttnArgs& a) {
    if (a.elem_bytes == 2) {
        if (a.hd == 128) launch_attn_simt<__nv_bfloat16, 128>(lc, a);
        else launch_attn_simt<__nv_bfloat16, 64>(lc, a);
    } else {
        if (a.hd == 128) launch_attn_simt<float, 128>(lc, a);
        else launch_attn_simt<float, 64>(lc, a);
    }
}

// Split-K combine and residual epilogue: one warp per (kv head, query row); merges the
// (m, l, O) partials of each stream and writes aF, aC and dA = aF - aC in fp32.  A lane owns PER = hd / 32
// consecutive columns and moves them as one vector (16 bytes of fp32 at hd = 128, 8 bytes of bf16 parts).
template <int PER>
struct VecF;
template <>
struct VecF<4> {
    static __device__ __forceinline__ void ld(const float* p, float (&v)[4]) {
        const float4 t = *reinterpret_cast<const float4*>(p);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    static __device__ __forceinline__ void st(float* p, const float (&v)[4]) {
        *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
    static __device__ __forceinline__ void st_pair(__nv_bfloat16* hi, __nv_bfloat16* lo, const float (&v)[4]) {
        unsigned short h[4], l[4];
        for (int c = 0; c < 4; ++c) {
            const __nv_bfloat16 hh = __float2bfloat16_rn(v[c]);
            h[c] = __bfloat16_as_ushort(hh);
            l[c] = __bfloat16_as_ushort(__float2bfloat16_rn(v[c] - __bfloat162float(hh)));
        }
        *reinterpret_cast<uint2*>(hi) = make_uint2(h[0] | ((unsigned)h[1] << 16), h[2] | ((unsigned)h[3] << 16));
        *reinterpret_cast<uint2*>(lo) = make_uint2(l[0] | ((unsigned)l[1] << 16), l[2] | ((unsigned)l[3] << 16));
    }
};
template <>
struct VecF<2> {
    static __device__ __forceinline__ void ld(const float* p, float (&v)[2]) {
        const float2 t = *reinterpret_cast<const float2*>(p);
        v[0] = t.x; v[1] = t.y;
    }
    static __device__ __forceinline__ void st(float* p, const float (&v)[2]) {
        *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]);
    }
    static __device__ __forceinline__ void st_pair(__nv_bfloat16* hi, __nv_bfloat16* lo, const float (&v)[2]) {
        unsigned short h[2], l[2];
        for (int c = 0; c < 2; ++c) {
            const __nv_bfloat16 hh = __float2bfloat16_rn(v[c]);
            h[c] = __bfloat16_as_ushort(hh);
            l[c] = __bfloat16_as_ushort(__float2bfloat16_rn(v[c] - __bfloat162float(hh)));
        }
        *reinterpret_cast<unsigned*>(hi) = h[0] | ((unsigned)h[1] << 16);
        *reinterpret_cast<unsigned*>(lo) = l[0] | ((unsigned)l[1] << 16);
    }
};

template <int PER>
__global__ void __launch_bounds__(256) k_attn_combine(AttnArgs a) {
    using V = VecF<PER>;
    int g = a.Hq / a.Hkv;
    int rows = a.N * g;
    int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (w >= a.Hkv * rows) return;
    int kh = w / rows, r = w % rows;
    int tok = r / g, hg = r % g;
    constexpr int hd = PER * 32;
    float res[2][PER];
    const size_t o = (size_t)tok * a.Hq * hd + (size_t)(kh * g + hg) * hd + lane * PER;
    const size_t o2 = o + (size_t)a.N * a.Hq * hd;      // the same entry of rows [N,2N) of the stacked pair
    if (a.mode == 2 && !a.student_first) V::ld(a.aF + o, res[0]);      // the teacher's output was produced earlier
    for (int s = (a.mode == 2 ? 1 : 0); s < (a.mode == 1 ? 1 : 2); ++s) {
        int z0 = s ? a.zoffC : 0;
        int ns = s ? a.nsplitC : a.nsplitF;
        float M = -INFINITY;
        for (int i = 0; i < ns; ++i) M = fmaxf(M, a.part_m[((size_t)(z0 + i) * a.Hkv + kh) * rows + r]);
        float den = 0.f, num[PER];
#pragma unroll
        for (int c = 0; c < PER; ++c) num[c] = 0.f;
        for (int i = 0; i < ns; ++i) {
            size_t pr = ((size_t)(z0 + i) * a.Hkv + kh) * rows + r;
            float mi = a.part_m[pr];
            if (mi == -INFINITY) continue;
            float wgt = expf(mi - M);
            den += wgt * a.part_l[pr];
            float po[PER];
            V::ld(a.part_O + pr * hd + lane * PER, po);
#pragma unroll
            for (int c = 0; c < PER; ++c) num[c] += wgt * po[c];
        }
        float inv = (den > 0.f) ? 1.f / den : 0.f;
#pragma unroll
        for (int c = 0; c < PER; ++c) res[s][c] = num[c] * inv;
    }
    if (a.student_first) {
        if (a.mode == 2) {          // student alone: aC and its pair in rows [N,2N)
            V::st(a.aC + o, res[1]);
            if (a.pair_hi) V::st_pair(a.pair_hi + o2, a.pair_lo + o2, res[1]);
        } else {                    // teacher after the student: aF, dA = aF - aC, pair of dA in rows [0,N)
            float ac[PER], dd[PER];
            V::ld(a.aC + o, ac);
#pragma unroll
            for (int c = 0; c < PER; ++c) dd[c] = res[0][c] - ac[c];
            V::st(a.aF + o, res[0]);
            V::st(a.dA + o, dd);
            if (a.pair_hi) V::st_pair(a.pair_hi + o, a.pair_lo + o, dd);
        }
        return;
    }
    if (a.mode != 2) {
        V::st(a.aF + o, res[0]);
        // operands of the o-projection: rows [0,N) aF, rows [N,2N) dA
        if (a.pair_hi) V::st_pair(a.pair_hi + o, a.pair_lo + o, res[0]);
    }
    if (a.mode != 1) {
        float dd[PER];
#pragma unroll
        for (int c = 0; c < PER; ++c) dd[c] = res[0][c] - res[1][c];
        V::st(a.aC + o, res[1]);
        V::st(a.dA + o, dd);
        if (a.pair_hi) V::st_pair(a.pair_hi + o2, a.pair_lo + o2, dd);
    }
}

void attention_combine(const Lc& lc, const AttnArgs& a) {
    int g = a.Hq / a.Hkv;
    long long warps = (long long)a.Hkv * a.N * g;
    if (a.combine_wait) cudaStreamWaitEvent(lc.st, (cudaEvent_t)a.combine_wait, 0);
    if (a.hd == 128) k_attn_combine<4><<<(unsigned)((warps + 7) / 8), 256, 0, lc.st>>>(a);
    else k_attn_combine<2><<<(unsigned)((warps + 7) / 8), 256, 0, lc.st>>>(a);
    lc.count();
}

// ------------------------------------------------------------------------------------------
// element-wise epilogues
// ------------------------------------------------------------------------------------------
__global__ void k_oproj_epilogue(const float* __restrict__ xF, const float* __restrict__ xC,
                                 const float* __restrict__ o, size_t n, float* __restrict__ zF,
                                 float* __restrict__ zC, float* __restrict__ dz) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float f = xF[i], c = xC[i];
    float zf = f + o[i];
    float d = (f - c) + o[n + i];
    zF[i] = zf;
    dz[i] = d;
    zC[i] = zf - d;
}

void oproj_epilogue(const Lc& lc, const float* xF, const float* xC, const float* o, int N, int d, float* zF,
                    float* zC, float* dz) {
    size_t n = (size_t)N * d;
    k_oproj_epilogue<<<(unsigned)((n + 255) / 256), 256, 0, lc.st>>>(xF, xC, o, n, zF, zC, dz);
    lc.count();
}

__device__ __forceinline__ float silu_f(float t) { return t / (1.0f + expf(-t)); }

__global__ void k_swiglu(const float* __restrict__ gu, int N, int F, float* __restrict__ hF,
                         float* __restrict__ hC, float* __restrict__ dh) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t n = (size_t)N * F;
    if (i >= n) return;
    size_t r = i / F, c = i % F;
    const float* a = gu + r * 2 * F;
    const float* b = gu + (r + N) * 2 * F;
    float f = silu_f(a[c]) * a[F + c];
    float s = silu_f(b[c]) * b[F + c];
    hF[i] = f;
    hC[i] = s;
    dh[i] = f - s;
}

void swiglu(const Lc& lc, const float* gu, int N, int F, float* hF, float* hC, float* dh) {
    size_t n = (size_t)N * F;
    k_swiglu<<<(unsigned)((n + 255) / 256), 256, 0, lc.st>>>(gu, N, F, hF, hC, dh);
    lc.count();
}

__global__ void k_transpose(const float* __restrict__ in, int rows, int cols, float* __restrict__ out) {
    __shared__ float t[32][33];
    int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (int j = threadIdx.y; j < 32; j += 8) {
        int r = r0 + j, c = c0 + threadIdx.x;
        if (r < rows && c < cols) t[j][threadIdx.x] = in[(size_t)r * cols + c];
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        int c = c0 + j, r = r0 + threadIdx.x;
        if (r < rows && c < cols) out[(size_t)c * rows + r] = t[threadIdx.x][j];
    }
}

void transpose_f32(const Lc& lc, const float* in, int rows, int cols, float* out) {
    dim3 grid((cols + 31) / 32, (rows + 31) / 32), block(32, 8);
    k_transpose<<<grid, block, 0, lc.st>>>(in, rows, cols, out);
    lc.count();
}

// ------------------------------------------------------------------------------------------
// reductions and the ridge matrix
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum_d(double v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum of a double over the block: warp shuffles, then one value per warp through shared memory.  Returns the
// total in thread 0 (other threads: unspecified).
__device__ __forceinline__ double block_sum_d(double v) {
    __shared__ double part[32];
    v = warp_sum_d(v);
    const int w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    if ((threadIdx.x & 31) == 0) part[w] = v;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x < 32) {
        t = (threadIdx.x < nw) ? part[threadIdx.x] : 0.0;
        t = warp_sum_d(t);
    }
    __syncthreads();
    return t;
}

// tr(S) and ||S||_F^2: one row per block iteration, float4 loads, fp32 partial sums per thread
// (a few hundred terms each), double precision across threads; one atomic per block.
__global__ void __launch_bounds__(256) k_trace_fro2(const float* __restrict__ S, int F, int ld, int lower,
                                                    DevStatus* status) {
    float fro[4] = {0.f, 0.f, 0.f, 0.f};
    double tr = 0.0;
    const bool vec = (ld % 4 == 0) && (((uintptr_t)S & 15) == 0);
    for (int r = blockIdx.x; r < F; r += gridDim.x) {
        const float* row = S + (size_t)r * ld;
        // symmetric matrix of which only the lower triangle is valid: entries left of the diagonal count twice
        const int ncol = lower ? r : F;
        const float w = lower ? 2.f : 1.f;
        const int n4 = vec ? (ncol & ~3) : 0;
        for (int c = threadIdx.x * 4; c < n4; c += 1024) {
            float4 v = *reinterpret_cast<const float4*>(row + c);
            fro[0] = fmaf(w * v.x, v.x, fro[0]); fro[1] = fmaf(w * v.y, v.y, fro[1]);
            fro[2] = fmaf(w * v.z, v.z, fro[2]); fro[3] = fmaf(w * v.w, v.w, fro[3]);
        }
        for (int c = n4 + threadIdx.x; c < ncol; c += 256) fro[0] = fmaf(w * row[c], row[c], fro[0]);
        if (threadIdx.x == 0) {
            if (lower) fro[1] = fmaf(row[r], row[r], fro[1]);
            tr += (double)row[r];
        }
    }
    const float f = (fro[0] + fro[1]) + (fro[2] + fro[3]);
    const int bad = __syncthreads_or(!isfinite(f));
    const double fd = block_sum_d((double)f);
    if (threadIdx.x == 0) {
        atomicAdd(&status->fro2, fd);
        if (tr != 0.0) atomicAdd(&status->tr, tr);
        if (bad) raise(status, PKV_ERR_NONFINITE);
    }
}

void trace_fro2(const Lc& lc, const float* S, int F, DevStatus* status, int ld, bool lower) {
    k_trace_fro2<<<min(F, 1184), 256, 0, lc.st>>>(S, F, ld > 0 ? ld : F, lower ? 1 : 0, status);
    lc.count();
}

// Sum of squares: four independent 16-byte loads in flight per thread, one atomic per block.
__global__ void __launch_bounds__(256) k_sumsq(const float* __restrict__ a, size_t n, double* dst) {
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const size_t n4 = (((uintptr_t)a & 15) == 0) ? n / 4 : 0;
    const float4* a4 = reinterpret_cast<const float4*>(a);
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n4; i += 4 * stride) {
        const float4 v0 = a4[i], v1 = a4[i + stride], v2 = a4[i + 2 * stride], v3 = a4[i + 3 * stride];
        acc[0] = fmaf(v0.x, v0.x, acc[0]); acc[1] = fmaf(v0.y, v0.y, acc[1]); acc[2] = fmaf(v0.z, v0.z, acc[2]); acc[3] = fmaf(v0.w, v0.w, acc[3]);
        acc[0] = fmaf(v1.x, v1.x, acc[0]); acc[1] = fmaf(v1.y, v1.y, acc[1]); acc[2] = fmaf(v1.z, v1.z, acc[2]); acc[3] = fmaf(v1.w, v1.w, acc[3]);
        acc[0] = fmaf(v2.x, v2.x, acc[0]); acc[1] = fmaf(v2.y, v2.y, acc[1]); acc[2] = fmaf(v2.z, v2.z, acc[2]); acc[3] = fmaf(v2.w, v2.w, acc[3]);
        acc[0] = fmaf(v3.x, v3.x, acc[0]); acc[1] = fmaf(v3.y, v3.y, acc[1]); acc[2] = fmaf(v3.z, v3.z, acc[2]); acc[3] = fmaf(v3.w, v3.w, acc[3]);
    }
    for (; i < n4; i += stride) {
        const float4 v = a4[i];
        acc[0] = fmaf(v.x, v.x, acc[0]); acc[1] = fmaf(v.y, v.y, acc[1]);
        acc[2] = fmaf(v.z, v.z, acc[2]); acc[3] = fmaf(v.w, v.w, acc[3]);
    }
    for (size_t k = n4 * 4 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; k < n; k += stride)
        acc[0] = fmaf(a[k], a[k], acc[0]);
    const double s = block_sum_d((double)((acc[0] + acc[1]) + (acc[2] + acc[3])));
    if (threadIdx.x == 0) atomicAdd(dst, s);
}

void sumsq(const Lc& lc, const float* a, int64_t n, double* dst) {
    if (n <= 0) return;
    int blocks = (int)((n / 4 + 255) / 256);
    if (blocks > 1184) blocks = 1184;
    if (blocks < 1) blocks = 1;
    k_sumsq<<<blocks, 256, 0, lc.st>>>(a, (size_t)n, dst);
    lc.count();
}

// lambda from the statistics (Eq. 7 or a variant), then G = S_H + lambda I.
__global__ void k_lambda(int F, float lam0, int mode, DevStatus* status) {
    double tr = status->tr, fro2 = status->fro2;
    double lam;
    if (mode == PKV_LAMBDA_ABSOLUTE) {
        lam = lam0;
    } else {
        if (!(tr > 0.0)) {
            raise(status, PKV_ERR_DEGENERATE);
            lam = 1.0;      // keeps the factorisation finite; the call reports the error
        } else if (mode == PKV_LAMBDA_TRACE_MEAN) {
            lam = (double)lam0 * tr / (double)F;
        } else {
            lam = (double)lam0 * fro2 / tr;
        }
    }
    status->lam = (float)lam;
    status->min_pivot = INFINITY;
}

__global__ void k_ridge_matrix(const float* __restrict__ S, int F, float* __restrict__ G,
                               const DevStatus* __restrict__ status) {
    size_t n = (size_t)F * F;
    float lam = status->lam;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        float v = S[i];
        if (i / F == i % F) v += lam;
        G[i] = v;
    }
}

void ridge_lambda(const Lc& lc, int F, float lam0, int mode, DevStatus* status) {
    k_lambda<<<1, 1, 0, lc.st>>>(F, lam0, mode, status);
    lc.count();
}

void make_ridge_matrix(const Lc& lc, const float* S_H, int F, float lam0, int mode, float* G, DevStatus* status) {
    ridge_lambda(lc, F, lam0, mode, status);
    k_ridge_matrix<<<592, 256, 0, lc.st>>>(S_H, F, G, status);
    lc.count();
}

__global__ void k_sub(const float* __restrict__ a, const float* __restrict__ b, size_t n, float* __restrict__ out) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = a[i] - b[i];
}

void sub_f32(const Lc& lc, const float* a, const float* b, int64_t n, float* out) {
    if (n <= 0) return;
    k_sub<<<(unsigned)((n + 255) / 256), 256, 0, lc.st>>>(a, b, (size_t)n, out);
    lc.count();
}

// Residual of the ridge system for iterative refinement: R = S_T - lambda dW - P with P = dW S_H given (in place:
// R overwrites P); lambda is the coefficient the solve used (status->lam).  The norm of dW is reported anew after the
// correction and is cleared here, the residual's norm too where the caller reports it.
__global__ void k_refine_residual(const float* __restrict__ S_T, const float* __restrict__ dW, float* __restrict__ P, size_t n,
                                  DevStatus* status) {
    const float lam = status->lam;
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) P[i] = (S_T[i] - P[i]) - lam * dW[i];
}
__global__ void k_clear_refine_norms(DevStatus* status, int clear_res) {
    if (clear_res) status->res_fro2 = 0.0;
    status->dw_fro2 = 0.0;
}

void refine_residual(const Lc& lc, const float* S_T, const float* dW, float* P, int64_t n, DevStatus* status, bool clear_res) {
    if (n <= 0) return;
    k_clear_refine_norms<<<1, 1, 0, lc.st>>>(status, clear_res ? 1 : 0);
    k_refine_residual<<<(unsigned)((n + 255) / 256), 256, 0, lc.st>>>(S_T, dW, P, (size_t)n, status);
    lc.count(2);
}

// G (full symmetric) from the lower triangle of S: G[i][j] = S[max(i,j)][min(i,j)].  G may be S itself (no entry
// above the diagonal is read).
__global__ void k_symmetric_from_lower(const float* S, float* G, int F) {
    __shared__ float t[32][33];
    const int bi = blockIdx.y, bj = blockIdx.x;
    if (bj > bi) return;
    const int r0 = bi * 32, c0 = bj * 32;
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int r = r0 + j, c = c0 + threadIdx.x;
        float v = 0.f;
        if (r < F && c < F) {
            v = c <= r ? S[(size_t)r * F + c] : S[(size_t)c * F + r];      // diagonal tiles: mirror inside the tile
            G[(size_t)r * F + c] = v;
        }
        t[j][threadIdx.x] = v;
    }
    if (bj == bi) return;
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += 8) {
        const int r = c0 + j, c = r0 + threadIdx.x;      // the mirrored tile
        if (r < F && c < F) G[(size_t)r * F + c] = t[threadIdx.x][j];
    }
}

void symmetric_from_lower(const Lc& lc, const float* S, float* G, int F) {
    dim3 grid((F + 31) / 32, (F + 31) / 32), block(32, 8);
    k_symmetric_from_lower<<<grid, block, 0, lc.st>>>(S, G, F);
    lc.count();
}

// ------------------------------------------------------------------------------------------
// merge: W <- W + dW, sum in fp32, one rounding to W's type
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_merge_bf16(__nv_bfloat16* __restrict__ W, const float* __restrict__ dW,
                                                    size_t n) {
    size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 8;
    if (i + 8 <= n) {
        uint4 wv = *reinterpret_cast<const uint4*>(W + i);
        float4 d0 = *reinterpret_cast<const float4*>(dW + i);
        float4 d1 = *reinterpret_cast<const float4*>(dW + i + 4);
        __nv_bfloat162* wp = reinterpret_cast<__nv_bfloat162*>(&wv);
        float2 f;
        f = __bfloat1622float2(wp[0]); wp[0] = __floats2bfloat162_rn(f.x + d0.x, f.y + d0.y);
        f = __bfloat1622float2(wp[1]); wp[1] = __floats2bfloat162_rn(f.x + d0.z, f.y + d0.w);
        f = __bfloat1622float2(wp[2]); wp[2] = __floats2bfloat162_rn(f.x + d1.x, f.y + d1.y);
        f = __bfloat1622float2(wp[3]); wp[3] = __floats2bfloat162_rn(f.x + d1.z, f.y + d1.w);
        *reinterpret_cast<uint4*>(W + i) = wv;
    } else {
        for (size_t j = i; j < n; ++j) W[j] = __float2bfloat16_rn(__bfloat162float(W[j]) + dW[j]);
    }
}

__global__ void __launch_bounds__(256) k_merge_f32(float* __restrict__ W, const float* __restrict__ dW, size_t n) {
    size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i + 4 <= n) {
        float4 w = *reinterpret_cast<const float4*>(W + i);
        float4 d = *reinterpret_cast<const float4*>(dW + i);
        w.x += d.x; w.y += d.y; w.z += d.z; w.w += d.w;
        *reinterpret_cast<float4*>(W + i) = w;
    } else {
        for (size_t j = i; j < n; ++j) W[j] += dW[j];
    }
}

void merge_weights(const Lc& lc, void* W, int w_dtype, const float* dW, int64_t count) {
    if (count <= 0) return;
    size_t n = (size_t)count;
    if (w_dtype == PKV_BF16) {
        size_t thr = (n + 7) / 8;
        k_merge_bf16<<<(unsigned)((thr + 255) / 256), 256, 0, lc.st>>>((__nv_bfloat16*)W, dW, n);
    } else {
        size_t thr = (n + 3) / 4;
        k_merge_f32<<<(unsigned)((thr + 255) / 256), 256, 0, lc.st>>>((float*)W, dW, n);
    }
    lc.count();
}

// fp32 FMA throughput probe: every thread runs `iters` rounds of 16 independent fused multiply-adds (enough
// independent chains to cover the pipeline latency); the result is stored so that nothing is optimised away.
__global__ void __launch_bounds__(256) k_fma_probe(float* __restrict__ out, int iters, float a, float b) {
    float v[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = (float)(threadIdx.x + i) * 1e-3f;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = fmaf(v[i], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) s += v[i];
    out[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = s;
}

// Measures the device's sustained fp32 FMA rate (TFLOP/s, 2 flops per FMA) with CUDA events on `st`.
int fma_peak_tflops(cudaStream_t st, float* scratch, size_t scratch_floats, int sm_count, double* tflops) {
    const int blocks = sm_count * 8, threads = 256, iters = 4096;
    if ((size_t)blocks * threads > scratch_floats) return PKV_ERR_NOMEM;
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return PKV_ERR_CUDA;
    double best = 0.0;
    for (int rep = 0; rep < 5; ++rep) {       // first repetitions warm up; the best of the rest is reported
        cudaEventRecord(e0, st);
        k_fma_probe<<<blocks, threads, 0, st>>>(scratch, iters, 0.999f, 1e-4f);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess) { cudaEventDestroy(e0); cudaEventDestroy(e1); return PKV_ERR_CUDA; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double fl = 2.0 * 16.0 * iters * (double)blocks * threads;
        if (rep >= 2 && ms > 0.f) best = fmax(best, fl / (ms * 1e-3) / 1e12);
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    *tflops = best;
    return cudaGetLastError() == cudaSuccess ? PKV_OK : PKV_ERR_CUDA;
}

}  // namespace pkv
