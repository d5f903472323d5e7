// C ABI of libpkv.so: context, workspace carving, argument validation and the per-block stage
// sequence of Algorithm 1 (teacher/student forward, targets, statistics, ridge solve, next
// states).  All arithmetic happens in the kernels of the other translation units.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include <cuda.h>

#include "pkv_internal.h"
#include "pkv_tc.h"

using namespace pkv;

// ---------------------------------------------------------------------------------------------
// SM partition for the teacher stream of the stack driver.
//
// The teacher's attention CTAs each hold a whole SM (all of its shared memory and tensor memory) for
// hundreds of microseconds, and there are several waves of them: while they run, the student's kernels
// and the latency-bound chain of the ridge solve find no free SM, whatever their stream priority, and
// the two streams end up running one after the other.  The teacher stream is therefore created inside a
// green context that owns all SMs but a reserve; the student's kernels and the solve (ordinary streams,
// all SMs) then always find the reserve free of long-running CTAs.  Driver entry points are looked up at
// run time; if anything is missing the teacher stream is an ordinary stream (correct, less overlap).
// ---------------------------------------------------------------------------------------------
namespace {
struct GreenApi {
    CUresult (*DeviceGet)(CUdevice*, int);
    CUresult (*DeviceGetDevResource)(CUdevice, CUdevResource*, CUdevResourceType);
    CUresult (*SplitByCount)(CUdevResource*, unsigned int*, const CUdevResource*, CUdevResource*, unsigned int,
                             unsigned int);
    CUresult (*GenerateDesc)(CUdevResourceDesc*, CUdevResource*, unsigned int);
    CUresult (*GreenCtxCreate)(CUgreenCtx*, CUdevResourceDesc, CUdevice, unsigned int);
    CUresult (*GreenCtxStreamCreate)(CUstream*, CUgreenCtx, unsigned int, int);
    CUresult (*GreenCtxDestroy)(CUgreenCtx);
    bool ok;
};

template <typename Fn>
bool entry(const char* name, Fn* out) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
        cudaGetLastError();
        return false;
    }
    *out = reinterpret_cast<Fn>(p);
    return true;
}

const GreenApi& green_api() {
    static GreenApi api = [] {
        GreenApi a{};
        a.ok = entry("cuDeviceGet", &a.DeviceGet) && entry("cuDeviceGetDevResource", &a.DeviceGetDevResource) &&
               entry("cuDevSmResourceSplitByCount", &a.SplitByCount) && entry("cuDevResourceGenerateDesc", &a.GenerateDesc) &&
               entry("cuGreenCtxCreate", &a.GreenCtxCreate) && entry("cuGreenCtxStreamCreate", &a.GreenCtxStreamCreate) &&
               entry("cuGreenCtxDestroy", &a.GreenCtxDestroy);
        return a;
    }();
    return api;
}

}  // namespace

namespace pkv {
// A green context that owns at least `want_sms` SMs of the current device and leaves the rest alone.
// Returns false (nothing created) when the partition cannot be made.
bool green_partition_create(int want_sms, void** gctx_out, int* got_sms) {
    const GreenApi& a = green_api();
    if (!a.ok || want_sms <= 0) return false;
    // PKV_SM_PARTITIONS=0: ordinary streams everywhere (a profiler that cannot prepare kernels launched into a green
    // context can still list every launch; the schedules stay the same, only the SM split is gone)
    static const bool off = [] { const char* e = getenv("PKV_SM_PARTITIONS"); return e && atoi(e) == 0; }();
    if (off) return false;
    int ord = 0;
    if (cudaGetDevice(&ord) != cudaSuccess) return false;
    CUdevice dev;
    if (a.DeviceGet(&dev, ord) != CUDA_SUCCESS) return false;
    CUdevResource all, part, rest;
    if (a.DeviceGetDevResource(dev, &all, CU_DEV_RESOURCE_TYPE_SM) != CUDA_SUCCESS) return false;
    if ((int)all.sm.smCount <= want_sms) return false;
    unsigned int groups = 1;
    if (a.SplitByCount(&part, &groups, &all, &rest, 0, (unsigned int)want_sms) != CUDA_SUCCESS || groups != 1) return false;
    if (part.sm.smCount >= all.sm.smCount) return false;      // rounding left no reserve
    CUdevResourceDesc desc;
    if (a.GenerateDesc(&desc, &part, 1) != CUDA_SUCCESS) return false;
    CUgreenCtx g;
    if (a.GreenCtxCreate(&g, desc, dev, CU_GREEN_CTX_DEFAULT_STREAM) != CUDA_SUCCESS) return false;
    *gctx_out = (void*)g;
    *got_sms = (int)part.sm.smCount;
    return true;
}

// A stream of that partition: its kernels run on the partition's SMs only.
bool green_partition_stream(void* gctx, int priority, cudaStream_t* stream) {
    CUstream st;
    if (!gctx || green_api().GreenCtxStreamCreate(&st, (CUgreenCtx)gctx, CU_STREAM_NON_BLOCKING, priority) != CUDA_SUCCESS)
        return false;
    *stream = (cudaStream_t)st;
    return true;
}

void green_partition_destroy(void* gctx) {
    if (gctx) green_api().GreenCtxDestroy((CUgreenCtx)gctx);
}
}  // namespace pkv

namespace {
bool make_partition_stream(int want_sms, cudaStream_t* stream, void** gctx_out, int* got_sms) {
    void* g = nullptr;
    if (!green_partition_create(want_sms, &g, got_sms)) return false;
    if (!green_partition_stream(g, 0, stream)) {
        green_partition_destroy(g);
        return false;
    }
    *gctx_out = g;
    return true;
}
}  // namespace

enum Stage { ST_INDEX = 0, ST_QKV, ST_ATTN, ST_OPROJ, ST_MLP, ST_TARGET, ST_GRAM, ST_SOLVE, ST_NEXT, ST_COUNT };
static const char* kStageNames[ST_COUNT] = {"S0 index check + compaction", "S1-S2 norm + QKV + RoPE",
                                            "S3 dual-cache attention",     "S4 o-proj + residual",
                                            "S5 norm + gate/up + SiLU",    "S6 targets",
                                            "S7 Gram + cross statistics",  "S8 ridge solve",
                                            "S9 next states"};

constexpr int kMaxStackLayers = 128;
constexpr int kRing = 3;                    // teacher blocks in flight ahead of the student (ring slots of aF, zF, hF)
constexpr int kRingX = kRing + 2;           // ring of the teacher's next states: read again after the student's solve
constexpr int kDefaultReserveSms = 12;      // SMs the teacher stream leaves to the student and the solve (stack driver)
// Single-block build with a light teacher half (see build_teacher_stream): SMs its partition leaves to the solve.
// Measured at d = F = 4096, N = 512, L = 32768: 3.24 ms per block without the overlap, 3.07 / 2.94 / 2.92 / 2.91 / 3.35
// with 32 / 56 / 76 / 90 / 104 SMs left to the solve.
constexpr int kBuildReserveSms = 80;

struct Carver {
    char* base;
    size_t off;
    template <typename T>
    T* take(size_t n) {
        off = (off + 255) & ~(size_t)255;
        T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

struct Buffers {
    DevStatus* status;
    int32_t* head_off;
    int32_t* tok_cs;
    float* rope_tab;
    void* Kc;
    void* Vc;
    float* u;       // [2N][d]
    float* qkv;     // [2N][Dq+2Dkv]
    float* part_m;
    float* part_l;
    float* part_O;
    float* a2;      // [2N][Dq]: aF rows then dA rows
    float* aC;      // [N][Dq]
    float* o;       // [2N][d]
    float* zF;
    float* zC;
    float* dz;
    float* gu;      // [2N][2F]
    float* hF;
    float* hC;
    float* dh;
    float* R;       // [N][d]
    float* XT;      // [F][N]
    float* RT;      // [d][N]
    float* S_H;
    float* S_T;
    SolveWs solve;
    float* D;       // [N][d]
    float* xs[4];   // stack states, ping-pong: xF a/b, xC a/b
    // overlapped stack driver (tensor-core engine): teacher outputs of two blocks in flight, the state
    // difference xF - xC (ping-pong), per-layer status words and kept-set offsets
    float* ringA[kRing];   // aF [N][Dq]
    float* ringZ[kRing];   // zF [N][d]
    float* ringH[kRing];   // hF [N][F]
    float* ringX[kRingX];  // xF_next [N][d]
    float* dxbuf[2];   // [N][d]
    DevStatus* lstatus;    // [kMaxStackLayers]
    int32_t* lhead_off;    // [kMaxStackLayers][Hkv+1]
    pkv::TcBuffers tc;
};

struct pkv_ctx {
    pkv_dims dims;
    pkv_opts opts;
    cudaStream_t st;
    int engine;
    int dual;
    int elem_bytes;
    int kv_split, cap_splitF, cap_splitC;
    int sm_count;
    char* ws;
    bool own_ws;
    size_t ws_bytes;
    Buffers b;
    int32_t* host_stage;     // pinned: head_off + tok_cs
    DevStatus* host_status;  // pinned
    int32_t* host_lhead;     // pinned: per-layer kept-set offsets of a stack call
    DevStatus* host_lstatus; // pinned: per-layer status words of a stack call
    cudaStream_t tstream;    // teacher stream of the overlapped stack driver
    void* tgreen;            // green context that owns the teacher stream's SM partition (or null)
    int teacher_sms;         // SMs the teacher stream may use (sm_count when not partitioned)
    cudaStream_t bstream;    // single-block build: stream of a smaller partition for a light teacher half (or null)
    void* bgreen;
    int build_teacher_sms;
    cudaEvent_t evTea[kRing], evStu[kRing], evSetup;
    int64_t launches;
    int stream_open, stream_mode, stream_tokens;   // streamed reference set in progress (pkv_stream_*)
    float stream_lambda;
    double stream_tfro2;
    int refine_steps;        // corrections of iterative refinement after every ridge solve of a build (pkv_set_refinement)
    int force_sequential;    // pkv_build_stack: 1 = block by block on one stream even where the overlapped driver applies
    int teacher_timed;
    void* map_cache;
    int timing;
    cudaEvent_t ev[ST_COUNT + 1];
    cudaEvent_t evT[6];      // marks of the teacher half (tensor-core engine)
    char cuda_err[256];
};

static int choose_engine(const pkv_dims* d, const pkv_opts* o) {
    if (o && o->engine == PKV_ENGINE_SIMT) return PKV_ENGINE_SIMT;
    return (d->dtype == PKV_BF16) ? PKV_ENGINE_AUTO : PKV_ENGINE_SIMT;
}

static void split_plan(const pkv_dims* d, const pkv_opts* o, int sm_count, int* kv_split, int* capF, int* capC) {
    int g = d->Hq / d->Hkv;
    long long rows = (long long)d->N_max * g;
    long long qtiles = (rows + 31) / 32;
    long long Lt = (long long)d->L + d->N_max;
    int ks = o ? o->kv_split : 0;
    if (ks <= 0) {
        long long want = (4LL * sm_count + qtiles * d->Hkv - 1) / (qtiles * d->Hkv);
        if (want < 1) want = 1;
        if (want > 64) want = 64;
        long long per = (Lt + want - 1) / want;
        per = ((per + 63) / 64) * 64;
        if (per < 256) per = 256;
        ks = (int)per;
    }
    ks = ((ks + 31) / 32) * 32;
    *kv_split = ks;
    *capF = (int)((Lt + ks - 1) / ks);
    long long Ls = (long long)d->b_max + d->N_max;
    *capC = (int)((Ls + ks - 1) / ks);
    if (*capC < 1) *capC = 1;
}

static size_t carve(Buffers* b, char* base, const pkv_dims* d, int engine, int elem_bytes, int capF, int capC,
                    int dual) {
    Carver c{base, 0};
    const size_t N = d->N_max, dm = d->d, F = d->F, Dq = (size_t)d->Hq * d->hd, Dkv = (size_t)d->Hkv * d->hd;
    const size_t g = d->Hq / d->Hkv, rows = N * g;
    const size_t tot_kept = (size_t)d->Hkv * d->b_max;
    b->status = c.take<DevStatus>(1);
    b->head_off = c.take<int32_t>(d->Hkv + 1);
    b->tok_cs = c.take<int32_t>(N);
    b->rope_tab = c.take<float>(N * d->hd);
    b->Kc = c.take<char>(tot_kept * d->hd * elem_bytes + 256);
    b->Vc = c.take<char>(tot_kept * d->hd * elem_bytes + 256);
    b->u = c.take<float>(2 * N * dm);
    b->qkv = c.take<float>(2 * N * (Dq + 2 * Dkv));
    size_t nsp = (size_t)capF + capC;
    b->part_m = c.take<float>(nsp * d->Hkv * rows);
    b->part_l = c.take<float>(nsp * d->Hkv * rows);
    b->part_O = c.take<float>(nsp * d->Hkv * rows * d->hd);
    b->a2 = c.take<float>(2 * N * Dq);
    b->aC = c.take<float>(N * Dq);
    b->o = c.take<float>(2 * N * dm);
    b->zF = c.take<float>(N * dm);
    b->zC = c.take<float>(N * dm);
    b->dz = c.take<float>(N * dm);
    b->gu = c.take<float>(2 * N * 2 * F);
    b->hF = c.take<float>(N * F);
    b->hC = c.take<float>(N * F);
    b->dh = c.take<float>(N * F);
    b->R = c.take<float>(N * dm);
    b->XT = c.take<float>(F * N);
    b->RT = c.take<float>(dm * N);
    b->S_H = c.take<float>(F * F);
    b->S_T = c.take<float>(dm * F);
    size_t nblk = (F + kSolveNb - 1) / kSolveNb;
    b->solve.G = c.take<float>(F * F);
    b->solve.Lm = c.take<float>(F * F);
    b->solve.LT = c.take<float>(F * F);
    b->solve.inv = c.take<float>(nblk * kSolveNb * kSolveNb);
    b->solve.invT = c.take<float>(nblk * kSolveNb * kSolveNb);
    b->solve.Y = c.take<float>(dm * F);
    b->D = c.take<float>(N * dm);
    for (int i = 0; i < 4; ++i) b->xs[i] = c.take<float>(N * dm);
    if (engine != PKV_ENGINE_SIMT) {
        for (int i = 0; i < kRing; ++i) {
            b->ringA[i] = c.take<float>(N * Dq);
            b->ringZ[i] = c.take<float>(N * dm);
            b->ringH[i] = c.take<float>(N * F);
        }
        for (int i = 0; i < kRingX; ++i) b->ringX[i] = c.take<float>(N * dm);
        for (int i = 0; i < 2; ++i) b->dxbuf[i] = c.take<float>(N * dm);
        b->lstatus = c.take<DevStatus>(kMaxStackLayers);
        b->lhead_off = c.take<int32_t>((size_t)kMaxStackLayers * (d->Hkv + 1));
        c.off = pkv::tc_carve(&b->tc, base, c.off, d, dual);
    }
    return (c.off + 255) & ~(size_t)255;
}

static int dims_ok(const pkv_dims* d) {
    if (!d) return PKV_ERR_INVALID_ARG;
    if (d->d <= 0 || d->Hq <= 0 || d->Hkv <= 0 || d->F <= 0 || d->L < 0 || d->N_max <= 0 || d->b_max < 0)
        return PKV_ERR_INVALID_ARG;
    if (d->dtype != PKV_BF16 && d->dtype != PKV_FP32) return PKV_ERR_INVALID_ARG;
    if (!(d->eps >= 0.f) || !(d->rope_theta >= 0.f)) return PKV_ERR_INVALID_ARG;
    if (d->hd != 64 && d->hd != 128) return PKV_ERR_UNSUPPORTED;
    if (d->Hq % d->Hkv != 0) return PKV_ERR_UNSUPPORTED;
    if (d->F > 32768) return PKV_ERR_UNSUPPORTED;
    if ((long long)d->L + d->N_max > (1LL << 30)) return PKV_ERR_UNSUPPORTED;
    return PKV_OK;
}

extern "C" size_t pkv_workspace_bytes(const pkv_dims* dims, const pkv_opts* opts) {
    if (dims_ok(dims) != PKV_OK) return 0;
    int ks, cf, cc;
    split_plan(dims, opts, 148, &ks, &cf, &cc);
    Buffers b;
    int engine = choose_engine(dims, opts);
    return carve(&b, nullptr, dims, engine, dims->dtype == PKV_BF16 ? 2 : 4, cf, cc,
                 (opts && opts->solver == PKV_SOLVER_DUAL && engine != PKV_ENGINE_SIMT) ? 1 : 0);
}

extern "C" int pkv_create(pkv_ctx** out, const pkv_dims* dims, const pkv_opts* opts, void* cuda_stream) {
    if (!out) return PKV_ERR_INVALID_ARG;
    *out = nullptr;
    int rc = dims_ok(dims);
    if (rc != PKV_OK) return rc;
    pkv_ctx* c = new (std::nothrow) pkv_ctx();
    if (!c) return PKV_ERR_NOMEM;
    memset(c, 0, sizeof(*c));
    c->dims = *dims;
    if (opts) c->opts = *opts;
    c->st = (cudaStream_t)cuda_stream;
    c->engine = choose_engine(dims, opts);
    c->elem_bytes = dims->dtype == PKV_BF16 ? 2 : 4;
    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        delete c;
        return PKV_ERR_CUDA;
    }
    c->sm_count = prop.multiProcessorCount;
    if (c->engine != PKV_ENGINE_SIMT) {
        rc = pkv::tc_supported(dims, prop.major, prop.minor);
        if (rc != PKV_OK) {
            delete c;
            return rc;
        }
    }
    // the split plan uses 148 SMs so that pkv_workspace_bytes (no device needed) agrees with it
    split_plan(dims, opts, 148, &c->kv_split, &c->cap_splitF, &c->cap_splitC);
    c->dual = (opts && opts->solver == PKV_SOLVER_DUAL) ? 1 : 0;
    if (c->dual && (c->engine == PKV_ENGINE_SIMT || dims->N_max > dims->F)) {
        delete c;
        return PKV_ERR_UNSUPPORTED;
    }
    size_t need = carve(&c->b, nullptr, dims, c->engine, c->elem_bytes, c->cap_splitF, c->cap_splitC, c->dual);
    c->ws_bytes = need;
    if (opts && opts->workspace) {
        if (opts->workspace_bytes < need || ((uintptr_t)opts->workspace & 255)) {
            delete c;
            return PKV_ERR_NOMEM;
        }
        c->ws = (char*)opts->workspace;
        c->own_ws = false;
    } else {
        if (cudaMalloc((void**)&c->ws, need) != cudaSuccess) {
            cudaGetLastError();
            delete c;
            return PKV_ERR_NOMEM;
        }
        c->own_ws = true;
    }
    carve(&c->b, c->ws, dims, c->engine, c->elem_bytes, c->cap_splitF, c->cap_splitC, c->dual);
    size_t stage_ints = (size_t)dims->Hkv + 1 + dims->N_max;
    if (cudaMallocHost((void**)&c->host_stage, stage_ints * sizeof(int32_t)) != cudaSuccess ||
        cudaMallocHost((void**)&c->host_status, sizeof(DevStatus)) != cudaSuccess) {
        cudaGetLastError();
        pkv_destroy(c);
        return PKV_ERR_NOMEM;
    }
    if (c->engine != PKV_ENGINE_SIMT) {
        if (cudaMallocHost((void**)&c->host_lhead, (size_t)kMaxStackLayers * (dims->Hkv + 1) * sizeof(int32_t)) != cudaSuccess ||
            cudaMallocHost((void**)&c->host_lstatus, (size_t)kMaxStackLayers * sizeof(DevStatus)) != cudaSuccess) {
            cudaGetLastError();
            pkv_destroy(c);
            return PKV_ERR_NOMEM;
        }
        // teacher stream: on all SMs but a reserve (see the note at the top of this file), else ordinary
        c->teacher_sms = c->sm_count;
        const int reserve = (opts && opts->reserve_sms != 0) ? opts->reserve_sms : kDefaultReserveSms;
        if (reserve > 0 && reserve < c->sm_count)
            make_partition_stream(c->sm_count - reserve, &c->tstream, &c->tgreen, &c->teacher_sms);
        if (!c->tstream && cudaStreamCreateWithFlags(&c->tstream, cudaStreamNonBlocking) != cudaSuccess) {
            cudaGetLastError();
            pkv_destroy(c);
            return PKV_ERR_NOMEM;
        }
        {
            int keep = kBuildReserveSms;
            if (const char* e = getenv("PKV_BUILD_RESERVE_SMS")) keep = atoi(e);
            c->build_teacher_sms = 0;
            if (keep > 0 && keep + 8 <= c->sm_count)
                make_partition_stream(c->sm_count - keep, &c->bstream, &c->bgreen, &c->build_teacher_sms);
        }
        for (int i = 0; i < kRing; ++i) {
            cudaEventCreateWithFlags(&c->evTea[i], cudaEventDisableTiming);
            cudaEventCreateWithFlags(&c->evStu[i], cudaEventDisableTiming);
        }
        cudaEventCreateWithFlags(&c->evSetup, cudaEventDisableTiming);
    }
    for (int i = 0; i <= ST_COUNT; ++i) cudaEventCreate(&c->ev[i]);
    for (int i = 0; i < 6; ++i) cudaEventCreate(&c->evT[i]);
    if (c->engine != PKV_ENGINE_SIMT) {
        c->map_cache = pkv::tc_map_cache_create();
        rc = pkv::tc_init(&c->b.tc, dims);
        if (rc != PKV_OK) {
            pkv_destroy(c);
            return rc;
        }
    }
    *out = c;
    return PKV_OK;
}

extern "C" void pkv_destroy(pkv_ctx* c) {
    if (!c) return;
    cudaStreamSynchronize(c->st);
    if (c->own_ws && c->ws) cudaFree(c->ws);
    if (c->host_stage) cudaFreeHost(c->host_stage);
    if (c->host_status) cudaFreeHost(c->host_status);
    if (c->host_lhead) cudaFreeHost(c->host_lhead);
    if (c->host_lstatus) cudaFreeHost(c->host_lstatus);
    if (c->engine != PKV_ENGINE_SIMT && c->b.tc.side) cudaStreamSynchronize(c->b.tc.side);
    if (c->tstream) { cudaStreamSynchronize(c->tstream); cudaStreamDestroy(c->tstream); }
    green_partition_destroy(c->tgreen);
    if (c->bstream) { cudaStreamSynchronize(c->bstream); cudaStreamDestroy(c->bstream); }
    green_partition_destroy(c->bgreen);
    for (int i = 0; i < kRing; ++i) {
        if (c->evTea[i]) cudaEventDestroy(c->evTea[i]);
        if (c->evStu[i]) cudaEventDestroy(c->evStu[i]);
    }
    if (c->evSetup) cudaEventDestroy(c->evSetup);
    if (c->map_cache) pkv::tc_map_cache_destroy((pkv::MapCache*)c->map_cache);
    if (c->engine != PKV_ENGINE_SIMT) pkv::tc_destroy(&c->b.tc);
    for (int i = 0; i <= ST_COUNT; ++i)
        if (c->ev[i]) cudaEventDestroy(c->ev[i]);
    for (int i = 0; i < 6; ++i)
        if (c->evT[i]) cudaEventDestroy(c->evT[i]);
    delete c;
}

extern "C" int pkv_selftest_bounded_wait(pkv_ctx* c, int32_t* site) {
    if (!c) return PKV_ERR_INVALID_ARG;
    if (c->engine == PKV_ENGINE_SIMT) return PKV_ERR_UNSUPPORTED;      // the SIMT engine has no waits
    Lc lc{c->st, &c->launches, c->map_cache};
    cudaMemsetAsync(c->b.status, 0, sizeof(DevStatus), c->st);
    pkv::tc_selftest_wait(lc, c->b.status);
    cudaError_t e = cudaMemcpyAsync(c->host_status, c->b.status, sizeof(DevStatus), cudaMemcpyDeviceToHost, c->st);
    if (e != cudaSuccess || cudaStreamSynchronize(c->st) != cudaSuccess) return PKV_ERR_CUDA;
    if (site) *site = c->host_status->info0;
    return c->host_status->code;
}

extern "C" int pkv_set_timing(pkv_ctx* c, int on) {
    if (!c) return PKV_ERR_INVALID_ARG;
    c->timing = (on == 2) ? 2 : (on ? 1 : 0);
    return PKV_OK;
}

extern "C" int64_t pkv_launch_count(const pkv_ctx* c) { return c ? c->launches : 0; }
extern "C" int pkv_teacher_sm_count(const pkv_ctx* c) { return c ? c->teacher_sms : 0; }

extern "C" int pkv_set_stack_schedule(pkv_ctx* c, int schedule) {
    if (!c || (schedule != 0 && schedule != 1)) return PKV_ERR_INVALID_ARG;
    c->force_sequential = schedule;
    return PKV_OK;
}

extern "C" int pkv_set_refinement(pkv_ctx* c, int steps) {
    if (!c || steps < 0 || steps > 8) return PKV_ERR_INVALID_ARG;
    if (steps > 0 && (c->engine == PKV_ENGINE_SIMT || c->dual)) return PKV_ERR_UNSUPPORTED;
    c->refine_steps = steps;
    return PKV_OK;
}

extern "C" int pkv_measure_fma_peak(pkv_ctx* c, double* tflops) {
    if (!c || !tflops) return PKV_ERR_INVALID_ARG;
    cudaStreamSynchronize(c->st);
    // scratch: the activation buffer u (2 N d floats) is always large enough for one store per thread
    return fma_peak_tflops(c->st, c->b.gu, (size_t)2 * c->dims.N_max * 2 * c->dims.F, c->sm_count, tflops);
}

extern "C" const char* pkv_strerror(int code) {
    switch (code) {
        case PKV_OK: return "ok";
        case PKV_ERR_INVALID_ARG: return "invalid argument";
        case PKV_ERR_UNSUPPORTED: return "unsupported shape or device";
        case PKV_ERR_BAD_INDEX: return "kept-index set is not strictly ascending within [0, L)";
        case PKV_ERR_NOT_PD: return "ridge matrix is not positive definite in fp32";
        case PKV_ERR_DEGENERATE: return "tr(S_H) = 0: adaptive ridge scale undefined";
        case PKV_ERR_NONFINITE: return "non-finite value in the statistics";
        case PKV_ERR_TIMEOUT: return "bounded device-side wait expired";
        case PKV_ERR_CUDA: return "CUDA runtime error";
        case PKV_ERR_NOMEM: return "workspace allocation failed or too small";
        default: return "unknown error";
    }
}

extern "C" const char* pkv_last_cuda_error(const pkv_ctx* c) { return c ? c->cuda_err : ""; }
extern "C" const char* pkv_stage_name(int s) { return (s >= 0 && s < ST_COUNT) ? kStageNames[s] : ""; }

// ---------------------------------------------------------------------------------------------

static int cuda_fail(pkv_ctx* c, cudaError_t e, const char* where) {
    snprintf(c->cuda_err, sizeof(c->cuda_err), "%s: %s", where, cudaGetErrorString(e));
    return PKV_ERR_CUDA;
}

static void mark(pkv_ctx* c, int i) {
    if (c->timing == 1 || (c->timing == 2 && (i == ST_SOLVE || i == ST_NEXT))) cudaEventRecord(c->ev[i], c->st);
}

static int check_compressed(const pkv_ctx* c, const pkv_kv_compressed* cb, int* total, int* max_b) {
    if (!cb || !cb->head_off) return PKV_ERR_INVALID_ARG;
    const int Hkv = c->dims.Hkv;
    if (cb->head_off[0] != 0) return PKV_ERR_INVALID_ARG;
    int mb = 0;
    for (int h = 0; h < Hkv; ++h) {
        int bh = cb->head_off[h + 1] - cb->head_off[h];
        if (bh < 0 || bh > c->dims.b_max) return PKV_ERR_INVALID_ARG;
        if (bh > mb) mb = bh;
    }
    *total = cb->head_off[Hkv];
    *max_b = mb;
    if (*total > 0) {
        if (cb->qbits != 0) {
            if (cb->idx) return PKV_ERR_INVALID_ARG;          // a quantised cache is an explicit cache
            if (cb->qbits != 8 && cb->qbits != 4) return PKV_ERR_UNSUPPORTED;
            if (cb->qgroup <= 0 || c->dims.hd % cb->qgroup != 0 || cb->qgroup % 8 != 0) return PKV_ERR_UNSUPPORTED;
            if (!cb->Kc || !cb->Vc || !cb->k_scale || !cb->v_scale) return PKV_ERR_INVALID_ARG;
            if (((uintptr_t)cb->k_scale & 3) || ((uintptr_t)cb->v_scale & 3)) return PKV_ERR_INVALID_ARG;
        } else if (cb->idx) {
            if ((uintptr_t)cb->idx & 3) return PKV_ERR_INVALID_ARG;
        } else {
            if (!cb->Kc || !cb->Vc) return PKV_ERR_INVALID_ARG;
            if (((uintptr_t)cb->Kc & 15) || ((uintptr_t)cb->Vc & 15)) return PKV_ERR_INVALID_ARG;
        }
    }
    return PKV_OK;
}

static int check_chunks(const pkv_ctx* c, int N, int n_chunks, const int32_t* chunk_off) {
    if (N <= 0 || N > c->dims.N_max || n_chunks <= 0 || !chunk_off) return PKV_ERR_INVALID_ARG;
    if (chunk_off[0] != 0 || chunk_off[n_chunks] != N) return PKV_ERR_INVALID_ARG;
    for (int i = 0; i < n_chunks; ++i)
        if (chunk_off[i + 1] <= chunk_off[i]) return PKV_ERR_INVALID_ARG;
    return PKV_OK;
}

// uploads head_off and the per-token chunk starts
static void upload_meta(pkv_ctx* c, const int32_t* head_off, int N, int n_chunks, const int32_t* chunk_off) {
    const int Hkv = c->dims.Hkv;
    int32_t* hs = c->host_stage;
    for (int h = 0; h <= Hkv; ++h) hs[h] = head_off ? head_off[h] : 0;
    int32_t* cs = hs + Hkv + 1;
    for (int ch = 0; ch < n_chunks; ++ch)
        for (int i = chunk_off[ch]; i < chunk_off[ch + 1]; ++i) cs[i] = chunk_off[ch];
    cudaMemcpyAsync(c->b.head_off, hs, (Hkv + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, c->st);
    if (N > 0) cudaMemcpyAsync(c->b.tok_cs, cs, (size_t)N * sizeof(int32_t), cudaMemcpyHostToDevice, c->st);
}

static void begin_call(pkv_ctx* c) {
    cudaMemsetAsync(c->b.status, 0, sizeof(DevStatus), c->st);
}

// bounds on cond(S_H + lambda I) from what the solve leaves in the status word (see pkv_stats)
static void fill_cond(const DevStatus& s, pkv_stats* stats) {
    stats->cond_lower_bound = stats->cond_upper_bound = 0.0;
    stats->cond_warning = stats->reserved = 0;
    if (!(s.lam > 0.f) || !(s.min_pivot > 0.f) || !(s.tr > 0.0)) return;
    stats->cond_lower_bound = (s.fro2 / s.tr + (double)s.lam) / (double)s.min_pivot;
    stats->cond_upper_bound = (sqrt(s.fro2) + (double)s.lam) / (double)s.lam;
    stats->cond_warning = stats->cond_lower_bound > 1e4 ? 1 : 0;
}

// reads the status word; fills stats; returns the call's code
static int end_call(pkv_ctx* c, pkv_stats* stats, const int32_t* head_off) {
    cudaError_t e = cudaMemcpyAsync(c->host_status, c->b.status, sizeof(DevStatus), cudaMemcpyDeviceToHost, c->st);
    if (e != cudaSuccess) return cuda_fail(c, e, "status copy");
    e = cudaStreamSynchronize(c->st);
    if (e != cudaSuccess) return cuda_fail(c, e, "stream synchronize");
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(c, e, "kernel launch");
    const DevStatus& s = *c->host_status;
    if (stats) {
        stats->lambda_eff = s.lam;
        stats->trace = s.tr;
        stats->fro2 = s.fro2;
        stats->target_fro2 = s.t_fro2;
        stats->resid_fro2 = s.res_fro2;
        stats->dW_fro2 = s.dw_fro2;
        stats->min_pivot = s.min_pivot;
        fill_cond(s, stats);
        stats->err_info[0] = stats->err_info[1] = 0;
        if (s.code == PKV_ERR_BAD_INDEX && s.bad_index && head_off) {
            int pos = (int)(s.bad_index - 1), h = 0;
            while (h + 1 < c->dims.Hkv && head_off[h + 1] <= pos) ++h;
            stats->err_info[0] = h;
            stats->err_info[1] = pos - head_off[h];
        } else if (s.code == PKV_ERR_NOT_PD && s.bad_column) {
            stats->err_info[0] = (int)(s.bad_column - 1);
        } else if (s.code == PKV_ERR_TIMEOUT) {
            stats->err_info[0] = s.info0;
            stats->err_info[1] = s.info1;
        }
        for (int i = 0; i < 12; ++i) stats->stage_ms[i] = 0.f;
        if (c->timing == 2) {      // the solve's interval on the caller's stream, default schedule
            cudaEventElapsedTime(&stats->stage_ms[ST_SOLVE], c->ev[ST_SOLVE], c->ev[ST_NEXT]);
        } else if (c->timing) {
            for (int i = 0; i < ST_COUNT; ++i) cudaEventElapsedTime(&stats->stage_ms[i], c->ev[i], c->ev[i + 1]);
            if (c->teacher_timed) {
                // the teacher half ran first, inside the interval the student's marks call "S1-S2":
                // move its stages to where they belong
                const int stage_of[5] = {ST_QKV, ST_ATTN, ST_OPROJ, ST_MLP, ST_NEXT};
                float total = 0.f;
                for (int i = 0; i < 5; ++i) {
                    float ms = 0.f;
                    cudaEventElapsedTime(&ms, c->evT[i], c->evT[i + 1]);
                    total += ms;
                    if (stage_of[i] != ST_QKV) stats->stage_ms[stage_of[i]] += ms;
                }
                float qkv = 0.f;
                cudaEventElapsedTime(&qkv, c->evT[0], c->evT[1]);
                stats->stage_ms[ST_QKV] -= (total - qkv);
                c->teacher_timed = 0;
            }
        }
    }
    return s.code;
}

static AttnArgs attn_args(pkv_ctx* c, const float* q, int64_t ldq, const float* k_new, const float* v_new,
                          int64_t ldkv, const pkv_kv* full, const void* Kc, const void* Vc, const float* bias,
                          int N, int max_b, int total) {
    AttnArgs a;
    memset(&a, 0, sizeof(a));
    a.total_kept = total; a.max_b = max_b;
    a.q = q; a.ldq = ldq; a.k_new = k_new; a.v_new = v_new; a.ldkv = ldkv;
    a.K = full->K; a.V = full->V; a.Kc = Kc; a.Vc = Vc; a.bias = bias;
    a.head_off = c->b.head_off; a.tok_cs = c->b.tok_cs;
    a.N = N; a.Hq = c->dims.Hq; a.Hkv = c->dims.Hkv; a.hd = c->dims.hd; a.L = c->dims.L;
    a.elem_bytes = c->elem_bytes;
    a.kv_split = c->kv_split;
    a.nsplitF = (c->dims.L + N + c->kv_split - 1) / c->kv_split;
    a.nsplitC = (max_b + N + c->kv_split - 1) / c->kv_split;
    if (a.nsplitC < 1) a.nsplitC = 1;
    a.zoffC = a.nsplitF;
    a.part_m = c->b.part_m; a.part_l = c->b.part_l; a.part_O = c->b.part_O;
    return a;
}

// Single-block build, teacher half beside the solve: which stream it runs on.  The solve's factorisation is a chain of
// about 45 us per 128 columns that leaves most SMs idle but stalls when its trailing updates are starved.  A teacher
// half that fits into that idle time gets the small partition (it must not crowd the updates out); a heavier one is
// the bottleneck itself and gets the stack driver's partition (all SMs but a small reserve).
static cudaStream_t build_teacher_stream(const pkv_ctx* c, int N) {
    const pkv_dims& D = c->dims;
    const double Dq = (double)D.Hq * D.hd, Dkv = (double)D.Hkv * D.hd, d = D.d, F = D.F;
    const double attn = 4.0 * N * Dq * ((double)D.L + N);
    const double gemm = 2.0 * N * (d * (Dq + 2 * Dkv) + Dq * d + 2 * d * F + 2 * F * d) * 2.0;     // two passes each
    const double teacher_ms = (attn / 0.9e15 + gemm / 1.0e15) * 1e3;
    const double chain_ms = (F / 128.0) * 0.045;
    if (c->bstream && teacher_ms < 0.6 * chain_ms) return c->bstream;
    return c->tstream;
}

// S0: returns the compact cache pointers to use
static void stage_compact(pkv_ctx* c, const Lc& lc, const pkv_kv* full, const pkv_kv_compressed* cb, int total,
                          const void** Kc, const void** Vc, const int32_t* head_off_dev = nullptr,
                          DevStatus* status = nullptr) {
    if (cb->idx && total > 0) {
        gather_kept(lc, c->elem_bytes, full->K, full->V, cb->idx, head_off_dev ? head_off_dev : c->b.head_off,
                    c->dims.Hkv, c->dims.L, c->dims.hd, total, c->b.Kc, c->b.Vc, status ? status : c->b.status);
        *Kc = c->b.Kc;
        *Vc = c->b.Vc;
    } else if (cb->qbits != 0 && total > 0) {
        // quantised explicit cache: decoded into the context's compact-cache buffers, the load path of the student
        dequant_cache(lc, c->elem_bytes, cb->Kc, cb->k_scale, cb->qbits, cb->qgroup, c->dims.hd, total, c->b.Kc);
        dequant_cache(lc, c->elem_bytes, cb->Vc, cb->v_scale, cb->qbits, cb->qgroup, c->dims.hd, total, c->b.Vc);
        *Kc = c->b.Kc;
        *Vc = c->b.Vc;
    } else {
        *Kc = cb->Kc ? cb->Kc : c->b.Kc;
        *Vc = cb->Vc ? cb->Vc : c->b.Vc;
    }
}

// Statistics from X [n][F], R [n][d] (Eq. 9), SIMT path.
static void gram_simt(pkv_ctx* c, const Lc& lc, const float* X, const float* R, int n, float* S_H, float* S_T,
                      bool accumulate) {
    const int F = c->dims.F, d = c->dims.d;
    transpose_f32(lc, X, n, F, c->b.XT);
    transpose_f32(lc, R, n, d, c->b.RT);
    gemm_tn_simt(lc, c->b.XT, n, c->b.XT, n, false, S_H, F, F, F, n, 1.f, nullptr, 0, accumulate);
    gemm_tn_simt(lc, c->b.RT, n, c->b.XT, n, false, S_T, F, d, F, n, 1.f, nullptr, 0, accumulate);
}

// S8.  `S_H_scratch` says that S_H may be overwritten (it is the context's own statistics buffer).
// Iterative refinement of dW = S_T (S_H + lambda I)^{-1} after a tensor-core solve: `steps` times the residual
// R = S_T - dW (S_full + lambda I) as an fp32-equivalent product, then dW += (R X^T) X with the inverse factor the
// solve left behind.  S_full: the full symmetric S_H, untouched by the factorisation.
static int refine_solution(pkv_ctx* c, const Lc& lc, const float* S_full, const float* S_T, float lam0, int mode,
                           float* dW, DevStatus* st, int steps, bool report_residual) {
    const int F = c->dims.F, d = c->dims.d;
    Buffers& b = c->b;
    const bool well = pkv::tc_well_conditioned(lam0, mode);
    float* P = b.solve.Y;      // [d][F]: dW S_H, then the residual
    for (int s = 0; s < steps; ++s) {
        int rc = pkv::tc_fp32_product(lc, &b.tc.solve, (size_t)d * F, dW, S_full, d, F, F, 1.f, P, false, 6, 4, st, true);
        if (rc != PKV_OK) return rc;
        refine_residual(lc, S_T, dW, P, (int64_t)d * F, st, report_residual);
        if (report_residual) sumsq(lc, P, (int64_t)d * F, &st->res_fro2);
        if ((rc = pkv::tc_solve_apply_add(lc, &b.tc.solve, P, F, F, d, dW, well, st)) != PKV_OK) return rc;
        sumsq(lc, dW, (int64_t)d * F, &st->dw_fro2);
    }
    // the next-state product of a build reads dW as a bf16 pair, which the solve's last product wrote
    if (steps > 0) pkv::tc_split_pair(lc, dW, d, F, b.tc.dW);
    return PKV_OK;
}

// refine < 0: the context's setting (pkv_set_refinement); the standalone refined solve passes its own count and
// reports the residual's norm.
static int solve_stage(pkv_ctx* c, const Lc& lc, float* S_H, const float* S_T, float lam0, int mode, float* dW,
                       bool S_H_scratch, DevStatus* status = nullptr, int refine = -1) {
    const int F = c->dims.F, d = c->dims.d;
    Buffers& b = c->b;                 // the context's own buffers: the solver keeps state in b.tc
    DevStatus* st = status ? status : b.status;
    const int steps = refine >= 0 ? refine : c->refine_steps;
    // the tensor-core build leaves only the lower triangle of its own S_H
    trace_fro2(lc, S_H, F, st, 0, S_H_scratch && c->engine != PKV_ENGINE_SIMT);
    if (c->engine == PKV_ENGINE_SIMT) {
        make_ridge_matrix(lc, S_H, F, lam0, mode, b.solve.G, st);
        cudaMemcpyAsync(b.solve.Y, S_T, (size_t)d * F * sizeof(float), cudaMemcpyDeviceToDevice, c->st);
        ridge_solve_simt(lc, b.solve, F, d, dW, st);
    } else {
        ridge_lambda(lc, F, lam0, mode, st);
        float* S = S_H;
        const float* S_full = S_H;     // what a refinement step multiplies by: never the factored copy
        if (!S_H_scratch) {
            cudaMemcpyAsync(b.solve.G, S_H, (size_t)F * F * sizeof(float), cudaMemcpyDeviceToDevice, lc.st);
            S = b.solve.G;
            b.tc.S3_ready = 0;         // the caller's S_T, not the one a build's statistics left split in place
        } else if (steps > 0) {
            symmetric_from_lower(lc, S_H, b.solve.G, F);     // S_H itself is factored in place
            S_full = b.solve.G;
        }
        pkv::tc_ridge_solve(lc, &b.tc, S, S_T, F, d, dW, lam0, mode, st);
        if (steps > 0) {
            sumsq(lc, dW, (int64_t)d * F, &st->dw_fro2);     // (cleared again by the first step; keeps the code path uniform)
            return refine_solution(c, lc, S_full, S_T, lam0, mode, dW, st, steps, refine >= 0);
        }
    }
    sumsq(lc, dW, (int64_t)d * F, &st->dw_fro2);
    return PKV_OK;
}

// stats_only: the streamed form (Sec. 2.3, Eq. 9): teacher and student forward of these tokens, then the running
// sums S_H, S_T of the context are ADDED to, and the call returns before the solve; xF_next_only optionally receives
// the teacher's next states of these tokens.
static int build_patch_impl(pkv_ctx* c, const pkv_block_weights* w, const pkv_kv* full,
                            const pkv_kv_compressed* cb, const pkv_ref* ref, float lambda, int mode, float* dW,
                            const pkv_ref_next* next, pkv_stats* stats, bool stats_only = false,
                            float* xF_next_only = nullptr) {
    if (!c || !w || !full || !cb || !ref || (!dW && !stats_only)) return PKV_ERR_INVALID_ARG;
    if (!w->g_attn || !w->Wq || !w->Wk || !w->Wv || !w->Wo || !w->g_mlp || !w->Wgate || !w->Wup || !w->Wdown)
        return PKV_ERR_INVALID_ARG;
    if (c->dims.L > 0 && (!full->K || !full->V)) return PKV_ERR_INVALID_ARG;
    if (!ref->xF || !ref->xC) return PKV_ERR_INVALID_ARG;
    if (!(lambda > 0.f) || !isfinite(lambda)) return PKV_ERR_INVALID_ARG;
    if (mode != PKV_LAMBDA_PAPER && mode != PKV_LAMBDA_ABSOLUTE && mode != PKV_LAMBDA_TRACE_MEAN)
        return PKV_ERR_INVALID_ARG;
    const void* ptrs[] = {w->Wq, w->Wk, w->Wv, w->Wo, w->Wgate, w->Wup, w->Wdown, full->K, full->V,
                          ref->xF, ref->xC, dW, w->g_attn, w->g_mlp, xF_next_only};
    for (const void* p : ptrs)
        if ((uintptr_t)p & 15) return PKV_ERR_INVALID_ARG;
    if (next && (!next->xF_next || !next->xC_next)) return PKV_ERR_INVALID_ARG;
    int rc = check_chunks(c, ref->N, ref->n_chunks, ref->chunk_off);
    if (rc != PKV_OK) return rc;
    int total = 0, max_b = 0;
    rc = check_compressed(c, cb, &total, &max_b);
    if (rc != PKV_OK) return rc;

    const pkv_dims& D = c->dims;
    const int N = ref->N, d = D.d, F = D.F, hd = D.hd;
    const int Dq = D.Hq * hd, Dkv = D.Hkv * hd, QKV = Dq + 2 * Dkv;
    const bool bf = D.dtype == PKV_BF16;
    Buffers& b = c->b;
    Lc lc{c->st, &c->launches, c->map_cache};

    begin_call(c);
    upload_meta(c, cb->head_off, N, ref->n_chunks, ref->chunk_off);
    mark(c, ST_INDEX);
    const void *Kc, *Vc;
    stage_compact(c, lc, full, cb, total, &Kc, &Vc);
    mark(c, ST_QKV);

    if (c->engine == PKV_ENGINE_SIMT) {
        // S1-S2: both streams stacked, rows [0,N) teacher, [N,2N) student
        rmsnorm_f32(lc, ref->xF, ref->xC, N, d, w->g_attn, D.eps, b.u);
        gemm_tn_simt(lc, b.u, d, w->Wq, d, bf, b.qkv, QKV, 2 * N, Dq, d, 1.f, nullptr, 0, false);
        gemm_tn_simt(lc, b.u, d, w->Wk, d, bf, b.qkv + Dq, QKV, 2 * N, Dkv, d, 1.f, nullptr, 0, false);
        gemm_tn_simt(lc, b.u, d, w->Wv, d, bf, b.qkv + Dq + Dkv, QKV, 2 * N, Dkv, d, 1.f, nullptr, 0, false);
        rope_table(lc, b.tok_cs, N, hd, ref->pos0, D.rope_theta, b.rope_tab);
        rope_apply(lc, b.qkv, QKV, 0, D.Hq + D.Hkv, hd, 2 * N, N, b.rope_tab);
        mark(c, ST_ATTN);
        // S3
        AttnArgs a = attn_args(c, b.qkv, QKV, b.qkv + Dq, b.qkv + Dq + Dkv, QKV, full, Kc, Vc,
                               cb->idx ? nullptr : cb->bias, N, max_b, total);
        a.aF = b.a2; a.aC = b.aC; a.dA = b.a2 + (size_t)N * Dq;
        attention_simt(lc, a);
        attention_combine(lc, a);
        mark(c, ST_OPROJ);
        // S4: [aF; dA] Wo^T, then zF, dz, zC
        gemm_tn_simt(lc, b.a2, Dq, w->Wo, Dq, bf, b.o, d, 2 * N, d, Dq, 1.f, nullptr, 0, false);
        oproj_epilogue(lc, ref->xF, ref->xC, b.o, N, d, b.zF, b.zC, b.dz);
        mark(c, ST_MLP);
        // S5
        rmsnorm_f32(lc, b.zF, b.zC, N, d, w->g_mlp, D.eps, b.u);
        gemm_tn_simt(lc, b.u, d, w->Wgate, d, bf, b.gu, 2 * F, 2 * N, F, d, 1.f, nullptr, 0, false);
        gemm_tn_simt(lc, b.u, d, w->Wup, d, bf, b.gu + F, 2 * F, 2 * N, F, d, 1.f, nullptr, 0, false);
        swiglu(lc, b.gu, N, F, b.hF, b.hC, b.dh);
        mark(c, ST_TARGET);
        // S6: R = dh Wdown^T + dz   (Eq. 5)
        gemm_tn_simt(lc, b.dh, F, w->Wdown, F, bf, b.R, d, N, d, F, 1.f, b.dz, d, false);
        sumsq(lc, b.R, (int64_t)N * d, &b.status->t_fro2);
        mark(c, ST_GRAM);
        // S7 (Eq. 9)
        gram_simt(c, lc, b.hC, b.R, N, b.S_H, b.S_T, stats_only);
        mark(c, ST_SOLVE);
    } else {
        pkv::TcForwardArgs fa{};
        fa.w = w; fa.full = full; fa.Kc = Kc; fa.Vc = Vc; fa.bias = cb->idx ? nullptr : cb->bias;
        fa.xF = ref->xF; fa.xC = ref->xC; fa.N = N; fa.pos0 = ref->pos0; fa.max_b = max_b; fa.total_kept = total;
        fa.head_off = b.head_off; fa.tok_cs = b.tok_cs; fa.rope_tab = b.rope_tab;
        fa.zF = b.zF; fa.zC = b.zC; fa.dz = b.dz; fa.hF = b.hF; fa.hC = b.hC; fa.R = b.R;
        fa.S_H = b.S_H; fa.S_T = b.S_T; fa.status = b.status;
        fa.aF = b.a2; fa.aC = b.aC; fa.dA = b.a2 + (size_t)N * Dq;
        fa.xF_next = next ? next->xF_next : nullptr;
        fa.kv_split = c->kv_split;
        fa.dual = c->dual;
        fa.precise_stats = pkv::tc_well_conditioned(lambda, mode) ? 0 : 1;
        fa.accumulate_stats = stats_only ? 1 : 0;
        fa.part_m = b.part_m; fa.part_l = b.part_l; fa.part_O = b.part_O;
        fa.ev = (c->timing == 1) ? c->ev : nullptr;
        fa.evT = nullptr;
        c->teacher_timed = 0;
        if (pkv::tc_forward_overlapped_applies(&b.tc, fa)) rc = pkv::tc_forward_overlapped(lc, &b.tc, &c->dims, fa, build_teacher_stream(c, N));
        else rc = pkv::tc_forward(lc, &b.tc, &c->dims, fa);
        if (rc != PKV_OK) {      // issue failed half-way: let every internal stream run dry before reporting
            pkv::tc_side_quiesce(&b.tc);
            if (c->tstream) cudaStreamSynchronize(c->tstream);
            if (c->bstream) cudaStreamSynchronize(c->bstream);
            return rc;
        }
    }
    if (stats_only) {
        // teacher's next states of these tokens, if asked: xF_next = zF + hF W^T
        if (xF_next_only) {
            if (c->engine == PKV_ENGINE_SIMT)
                gemm_tn_simt(lc, b.hF, F, w->Wdown, F, bf, xF_next_only, d, N, d, F, 1.f, b.zF, d, false);
            else
                pkv::tc_next_states(lc, &b.tc, &c->dims, N, w->Wdown, nullptr, b.zF, b.R, xF_next_only, nullptr, b.status);
        }
        mark(c, ST_NEXT);
        mark(c, ST_COUNT);
        return end_call(c, stats, cb->head_off);
    }
    // S8 (Eq. 7-8)
    bool next_async = false;
    if (c->dual) {
        rc = pkv::tc_dual_solve(lc, &b.tc, &c->dims, N, b.R, lambda, mode, dW, b.status);
        if (rc != PKV_OK) return rc;
        sumsq(lc, dW, (int64_t)d * F, &b.status->dw_fro2);
    } else {
        // the teacher's next state does not depend on the patch: beside the solve where the side stream is in use
        if (c->timing == 2) mark(c, ST_SOLVE);
        if (next && c->engine != PKV_ENGINE_SIMT)
            next_async = pkv::tc_teacher_next_async(lc, &b.tc, &c->dims, N, w->Wdown, b.zF, next->xF_next, b.status);
        solve_stage(c, lc, b.S_H, b.S_T, lambda, mode, dW, true);
        if (c->engine != PKV_ENGINE_SIMT) pkv::tc_build_trace_mark(&b.tc, 4, c->st);
    }
    mark(c, ST_NEXT);
    // S9: xF_next = zF + hF W^T;  D = R - hC dW^T;  xC_next = xF_next - D
    if (next) {
        if (c->engine == PKV_ENGINE_SIMT) {
            gemm_tn_simt(lc, b.hF, F, w->Wdown, F, bf, next->xF_next, d, N, d, F, 1.f, b.zF, d, false);
            gemm_tn_simt(lc, b.hC, F, dW, F, false, b.D, d, N, d, F, -1.f, b.R, d, false);
        } else {
            pkv::tc_next_states(lc, &b.tc, &c->dims, N, w->Wdown, dW, b.zF, b.R, next_async ? nullptr : next->xF_next,
                                b.D, b.status);
            pkv::tc_side_join(lc, &b.tc);
        }
        sumsq(lc, b.D, (int64_t)N * d, &b.status->res_fro2);
        sub_f32(lc, next->xF_next, b.D, (int64_t)N * d, next->xC_next);
    }
    mark(c, ST_COUNT);
    if (c->engine != PKV_ENGINE_SIMT && !c->dual) pkv::tc_build_trace_mark(&b.tc, 5, c->st);
    rc = end_call(c, stats, cb->head_off);
    if (c->engine != PKV_ENGINE_SIMT && !c->dual) pkv::tc_build_trace_print(&b.tc);
    return rc;
}

extern "C" int pkv_build_patch(pkv_ctx* ctx, const pkv_block_weights* w, const pkv_kv* full,
                               const pkv_kv_compressed* cb, const pkv_ref* ref, float lambda, int lambda_mode,
                               float* dW, const pkv_ref_next* next, pkv_stats* stats) {
    return build_patch_impl(ctx, w, full, cb, ref, lambda, lambda_mode, dW, next, stats);
}

// ---- streamed reference sets (Sec. 2.3: chunked query encoding with running sufficient statistics) ----

extern "C" int pkv_stream_begin(pkv_ctx* c, float lambda, int lambda_mode) {
    if (!c) return PKV_ERR_INVALID_ARG;
    if (!(lambda > 0.f) || !isfinite(lambda)) return PKV_ERR_INVALID_ARG;
    if (lambda_mode != PKV_LAMBDA_PAPER && lambda_mode != PKV_LAMBDA_ABSOLUTE && lambda_mode != PKV_LAMBDA_TRACE_MEAN)
        return PKV_ERR_INVALID_ARG;
    if (c->dual) return PKV_ERR_UNSUPPORTED;          // the dual form needs every reference token in one call
    const size_t F = c->dims.F, d = c->dims.d;
    if (cudaMemsetAsync(c->b.S_H, 0, F * F * sizeof(float), c->st) != cudaSuccess ||
        cudaMemsetAsync(c->b.S_T, 0, d * F * sizeof(float), c->st) != cudaSuccess)
        return PKV_ERR_CUDA;
    c->stream_lambda = lambda;
    c->stream_mode = lambda_mode;
    c->stream_tokens = 0;
    c->stream_tfro2 = 0.0;
    c->stream_open = 1;
    return PKV_OK;
}

extern "C" int pkv_stream_add(pkv_ctx* c, const pkv_block_weights* w, const pkv_kv* full, const pkv_kv_compressed* cb,
                              const pkv_ref* ref, float* xF_next) {
    if (!c || !c->stream_open) return PKV_ERR_INVALID_ARG;
    pkv_stats st;
    int rc = build_patch_impl(c, w, full, cb, ref, c->stream_lambda, c->stream_mode, nullptr, nullptr, &st, true, xF_next);
    if (rc != PKV_OK) {
        c->stream_open = 0;                          // the running sums may be partly updated: start over
        return rc;
    }
    c->stream_tokens += ref->N;
    c->stream_tfro2 += st.target_fro2;
    return PKV_OK;
}

extern "C" int pkv_stream_finish(pkv_ctx* c, float* dW, pkv_stats* stats) {
    if (!c || !dW || !c->stream_open || ((uintptr_t)dW & 15)) return PKV_ERR_INVALID_ARG;
    if (c->stream_tokens <= 0) return PKV_ERR_INVALID_ARG;
    c->stream_open = 0;
    Lc lc{c->st, &c->launches, c->map_cache};
    begin_call(c);
    if (c->engine != PKV_ENGINE_SIMT) c->b.tc.S3_ready = 0;
    solve_stage(c, lc, c->b.S_H, c->b.S_T, c->stream_lambda, c->stream_mode, dW, true);
    int rc = end_call(c, stats, nullptr);
    if (stats) stats->target_fro2 = c->stream_tfro2;
    return rc;
}

extern "C" int pkv_stream_propagate(pkv_ctx* c, const pkv_block_weights* w, const pkv_kv* full,
                                    const pkv_kv_compressed* cb, const pkv_ref* ref, const float* dW, float* xC_next) {
    if (!c || !w || !full || !cb || !ref || !dW || !xC_next || !ref->xC) return PKV_ERR_INVALID_ARG;
    if (c->engine == PKV_ENGINE_SIMT) return PKV_ERR_UNSUPPORTED;
    if (((uintptr_t)dW & 15) || ((uintptr_t)xC_next & 15) || ((uintptr_t)ref->xC & 15)) return PKV_ERR_INVALID_ARG;
    int rc = check_chunks(c, ref->N, ref->n_chunks, ref->chunk_off);
    if (rc != PKV_OK) return rc;
    int total = 0, max_b = 0;
    rc = check_compressed(c, cb, &total, &max_b);
    if (rc != PKV_OK) return rc;
    const pkv_dims& D = c->dims;
    const int N = ref->N;
    Buffers& b = c->b;
    Lc lc{c->st, &c->launches, c->map_cache};
    begin_call(c);
    upload_meta(c, cb->head_off, N, ref->n_chunks, ref->chunk_off);
    const void *Kc, *Vc;
    stage_compact(c, lc, full, cb, total, &Kc, &Vc);
    rope_table(lc, b.tok_cs, N, D.hd, ref->pos0, D.rope_theta, b.rope_tab);
    pkv::TcForwardArgs fa{};
    fa.w = w; fa.full = full; fa.Kc = Kc; fa.Vc = Vc; fa.bias = cb->idx ? nullptr : cb->bias;
    fa.xC = ref->xC; fa.N = N; fa.pos0 = ref->pos0; fa.max_b = max_b; fa.total_kept = total;
    fa.head_off = b.head_off; fa.tok_cs = b.tok_cs; fa.rope_tab = b.rope_tab;
    fa.aF = b.a2; fa.aC = b.aC; fa.dA = b.a2 + (size_t)N * D.Hq * D.hd;
    fa.zC = b.zC; fa.dz = b.dz; fa.hF = b.hF; fa.hC = b.hC;
    fa.status = b.status;
    rc = pkv::tc_student_propagate(lc, &b.tc, &c->dims, fa, dW, b.D, xC_next);
    if (rc != PKV_OK) return rc;
    return end_call(c, nullptr, cb->head_off);
}

extern "C" int pkv_merge(void* W, int w_dtype, const float* dW, int64_t count, void* cuda_stream) {
    if (!W || !dW || count < 0) return PKV_ERR_INVALID_ARG;
    if (w_dtype != PKV_BF16 && w_dtype != PKV_FP32) return PKV_ERR_INVALID_ARG;
    if (((uintptr_t)W & 15) || ((uintptr_t)dW & 15)) return PKV_ERR_INVALID_ARG;
    Lc lc{(cudaStream_t)cuda_stream, nullptr};
    merge_weights(lc, W, w_dtype, dW, count);
    return cudaGetLastError() == cudaSuccess ? PKV_OK : PKV_ERR_CUDA;
}

static void fill_stats(pkv_ctx* c, const DevStatus& s, pkv_stats* stats, const int32_t* head_off) {
    memset(stats, 0, sizeof(*stats));
    stats->lambda_eff = s.lam;
    stats->trace = s.tr;
    stats->fro2 = s.fro2;
    stats->target_fro2 = s.t_fro2;
    stats->resid_fro2 = s.res_fro2;
    stats->dW_fro2 = s.dw_fro2;
    stats->min_pivot = s.min_pivot;
    fill_cond(s, stats);
    if (s.code == PKV_ERR_BAD_INDEX && s.bad_index && head_off) {
        int pos = (int)(s.bad_index - 1), h = 0;
        while (h + 1 < c->dims.Hkv && head_off[h + 1] <= pos) ++h;
        stats->err_info[0] = h;
        stats->err_info[1] = pos - head_off[h];
    } else if (s.code == PKV_ERR_NOT_PD && s.bad_column) {
        stats->err_info[0] = (int)(s.bad_column - 1);
    } else if (s.code == PKV_ERR_TIMEOUT) {
        stats->err_info[0] = s.info0;
        stats->err_info[1] = s.info1;
    }
}

// Stack driver with the teacher run ahead (tensor-core engine).  The teacher stream of Algorithm 1 never sees
// a patch, so the teacher half of blocks l+1 .. l+kRing runs on its own CUDA stream beside the student half and
// the latency-bound ridge solve of block l.  Teacher outputs aF, zF, hF live in a ring of kRing slots which the
// student releases as soon as its forward has read them (before its solve); the teacher's next states sit in a
// longer ring because the student reads them once more after the solve (stream order makes kRing + 2 slots
// enough: the teacher of block l + kRing + 2 starts after the student forward of block l + 2).  The student
// carries the state difference xF - xC itself.
//
// Teacher cache (ridge-coefficient sweeps): with `cache` set, the teacher outputs of every block go to their own
// slot of that buffer instead of the rings (no slot is reused, so the teacher is never throttled), and a later
// call with run_teacher = false replays the student half, the statistics and the solve of every block against
// the cached teacher: the teacher of Algorithm 1 does not depend on the ridge coefficient.
static size_t teacher_cache_floats_per_layer(const pkv_dims& D, int N) {
    return (size_t)N * ((size_t)D.Hq * D.hd + 2 * (size_t)D.d + D.F);
}

static int build_stack_overlapped(pkv_ctx* c, int n_layers, int first, const pkv_block_weights* w, const pkv_kv* full,
                                  const pkv_kv_compressed* cb, const pkv_ref* ref0, float lambda, int mode,
                                  float* const* dW, const pkv_ref_next* final, pkv_stats* stats,
                                  float* cache = nullptr, bool run_teacher = true) {
    const pkv_dims& D = c->dims;
    const int N = ref0->N, d = D.d, F = D.F, Hkv = D.Hkv;
    const int Dq = D.Hq * D.hd;
    Buffers& b = c->b;
    int rc = check_chunks(c, N, ref0->n_chunks, ref0->chunk_off);
    if (rc != PKV_OK) return rc;
    if (!(lambda > 0.f) || !isfinite(lambda)) return PKV_ERR_INVALID_ARG;
    if (!ref0->xF || !ref0->xC || (final && (!final->xF_next || !final->xC_next))) return PKV_ERR_INVALID_ARG;
    std::vector<int> totals(n_layers, 0), maxbs(n_layers, 0);
    for (int l = first; l < n_layers; ++l) {
        if ((rc = check_compressed(c, &cb[l], &totals[l], &maxbs[l])) != PKV_OK) return rc;
        if (!dW[l] || !w[l].Wq || !w[l].Wk || !w[l].Wv || !w[l].Wo || !w[l].Wgate || !w[l].Wup || !w[l].Wdown ||
            !w[l].g_attn || !w[l].g_mlp || (D.L > 0 && (!full[l].K || !full[l].V)))
            return PKV_ERR_INVALID_ARG;
        for (int h = 0; h <= Hkv; ++h) c->host_lhead[(size_t)l * (Hkv + 1) + h] = cb[l].head_off[h];
    }
    cudaStream_t S = c->st, T = c->tstream;
    Lc lcS{S, &c->launches, c->map_cache}, lcT{T, &c->launches, c->map_cache};
    // set-up on the student stream: status words, kept-set offsets, chunk starts, RoPE table, dx0 = xF0 - xC0
    cudaMemsetAsync(b.lstatus, 0, (size_t)n_layers * sizeof(DevStatus), S);
    cudaMemcpyAsync(b.lhead_off + (size_t)first * (Hkv + 1), c->host_lhead + (size_t)first * (Hkv + 1),
                    (size_t)(n_layers - first) * (Hkv + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, S);
    upload_meta(c, cb[first].head_off, N, ref0->n_chunks, ref0->chunk_off);
    rope_table(lcS, b.tok_cs, N, D.hd, ref0->pos0, D.rope_theta, b.rope_tab);
    sub_f32(lcS, ref0->xF, ref0->xC, (int64_t)N * d, b.dxbuf[0]);
    cudaEventRecord(c->evSetup, S);
    cudaStreamWaitEvent(T, c->evSetup, 0);

    // optional timeline (environment variable PKV_STACK_TRACE=1): five timed events per block, printed to stderr
    const bool trace = getenv("PKV_STACK_TRACE") != nullptr;
    std::vector<cudaEvent_t> tev;
    if (trace) {
        tev.resize((size_t)n_layers * 5);
        for (auto& e : tev) cudaEventCreate(&e);
    }
    auto tmark = [&](int l, int i, cudaStream_t st) { if (trace) cudaEventRecord(tev[(size_t)l * 5 + i], st); };

    const float* xF_in = ref0->xF;
    const float* xC_in = ref0->xC;
    for (int l = first; l < n_layers; ++l) {
        const int k = l - first, slot = k % kRing, pp = k & 1;
        const bool last = (l == n_layers - 1);
        DevStatus* st = b.lstatus + l;
        const int32_t* hoff = b.lhead_off + (size_t)l * (Hkv + 1);
        pkv::TcForwardArgs fa{};
        fa.w = &w[l]; fa.full = &full[l];
        fa.N = N; fa.pos0 = ref0->pos0; fa.max_b = maxbs[l]; fa.total_kept = totals[l];
        fa.head_off = hoff; fa.tok_cs = b.tok_cs; fa.rope_tab = b.rope_tab;
        float* cX = nullptr;
        if (cache) {
            float* base_l = cache + (size_t)l * teacher_cache_floats_per_layer(D, N);
            fa.aF = base_l; fa.zF = base_l + (size_t)N * Dq; fa.hF = fa.zF + (size_t)N * d;
            cX = fa.hF + (size_t)N * F;
        } else {
            fa.aF = b.ringA[slot]; fa.zF = b.ringZ[slot]; fa.hF = b.ringH[slot];
        }
        fa.aC = b.aC; fa.dA = b.a2 + (size_t)N * Dq;
        fa.zC = b.zC; fa.dz = b.dz; fa.hC = b.hC; fa.R = b.R; fa.S_H = b.S_H; fa.S_T = b.S_T;
        fa.status = st; fa.dual = c->dual; fa.kv_split = c->kv_split;
        fa.precise_stats = pkv::tc_well_conditioned(lambda, mode) ? 0 : 1;
        // ---- teacher half of block l on the teacher stream ----
        if (k >= kRing && !cache) cudaStreamWaitEvent(T, c->evStu[slot], 0);    // slot free: student forward of block l-kRing is done
        fa.xF = xF_in; fa.xC = xF_in;
        float* xFn = cache ? cX : ((last && final) ? final->xF_next : b.ringX[k % kRingX]);
        tmark(l, 0, T);
        if (run_teacher) {
            rc = pkv::tc_teacher_forward(lcT, &b.tc, &c->dims, fa, xFn);
            if (rc != PKV_OK) break;
            cudaEventRecord(c->evTea[slot], T);
        }
        tmark(l, 1, T);
        // ---- student half, statistics, solve, next student state on the caller's stream ----
        const void *Kc, *Vc;
        stage_compact(c, lcS, &full[l], &cb[l], totals[l], &Kc, &Vc, hoff, st);
        fa.Kc = Kc; fa.Vc = Vc; fa.bias = cb[l].idx ? nullptr : cb[l].bias;
        fa.xC = xC_in; fa.dx = b.dxbuf[pp];
        if (run_teacher) cudaStreamWaitEvent(S, c->evTea[slot], 0);
        tmark(l, 2, S);
        rc = pkv::tc_student_forward(lcS, &b.tc, &c->dims, fa);
        if (rc != PKV_OK) break;
        cudaEventRecord(c->evStu[slot], S);                           // aF, zF, hF of this slot are no longer needed
        tmark(l, 3, S);
        if (c->dual) {
            rc = pkv::tc_dual_solve(lcS, &b.tc, &c->dims, N, b.R, lambda, mode, dW[l], st);
            if (rc != PKV_OK) break;
            sumsq(lcS, dW[l], (int64_t)d * F, &st->dw_fro2);
        } else {
            solve_stage(c, lcS, b.S_H, b.S_T, lambda, mode, dW[l], true, st);
        }
        float* Dn = b.dxbuf[1 - pp];                                  // xF_next - xC_next = T - hC dW^T
        pkv::tc_next_states(lcS, &b.tc, &c->dims, N, w[l].Wdown, dW[l], nullptr, b.R, nullptr, Dn, st);
        sumsq(lcS, Dn, (int64_t)N * d, &st->res_fro2);
        float* xCn = (last && final) ? final->xC_next : b.xs[2 + (1 - pp)];
        sub_f32(lcS, xFn, Dn, (int64_t)N * d, xCn);
        if (cache && last && final)
            cudaMemcpyAsync(final->xF_next, xFn, (size_t)N * d * sizeof(float), cudaMemcpyDeviceToDevice, S);
        tmark(l, 4, S);
        xF_in = xFn;
        xC_in = xCn;
    }
    // the last student waited for the last teacher; one copy of all status words, one synchronisation
    cudaMemcpyAsync(c->host_lstatus, b.lstatus, (size_t)n_layers * sizeof(DevStatus), cudaMemcpyDeviceToHost, S);
    cudaError_t e = cudaStreamSynchronize(S);
    cudaError_t e2 = cudaStreamSynchronize(T);
    if (trace) {
        if (e == cudaSuccess && e2 == cudaSuccess && rc == PKV_OK) {
            fprintf(stderr, "block: teacher start..end | student start, forward end, solve+next end (ms since the first teacher)\n");
            for (int l = first; l < n_layers; ++l) {
                float t[5];
                for (int i = 0; i < 5; ++i) cudaEventElapsedTime(&t[i], tev[(size_t)first * 5], tev[(size_t)l * 5 + i]);
                fprintf(stderr, "%3d: %8.3f .. %8.3f | %8.3f %8.3f %8.3f\n", l, t[0], t[1], t[2], t[3], t[4]);
            }
        }
        for (auto& ev : tev) cudaEventDestroy(ev);
    }
    if (e != cudaSuccess) return cuda_fail(c, e, "stream synchronize");
    if (e2 != cudaSuccess) return cuda_fail(c, e2, "teacher stream synchronize");
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(c, e, "kernel launch");
    if (rc != PKV_OK) return rc;
    int code = PKV_OK;
    for (int l = first; l < n_layers; ++l) {
        if (stats) fill_stats(c, c->host_lstatus[l], &stats[l], cb[l].head_off);
        if (code == PKV_OK && c->host_lstatus[l].code != 0) code = c->host_lstatus[l].code;
    }
    return code;
}

extern "C" int pkv_build_stack(pkv_ctx* c, int n_layers, int first_layer, const pkv_block_weights* w,
                               const pkv_kv* full, const pkv_kv_compressed* cb, const pkv_ref* ref0, float lambda,
                               int lambda_mode, float* const* dW, const pkv_ref_next* final, pkv_stats* stats) {
    if (!c || !w || !full || !cb || !ref0 || !dW || n_layers <= 0 || first_layer < 0 || first_layer >= n_layers)
        return PKV_ERR_INVALID_ARG;
    if (c->engine != PKV_ENGINE_SIMT && c->timing != 1 && !c->force_sequential && n_layers - first_layer >= 2 &&
        n_layers <= kMaxStackLayers)
        return build_stack_overlapped(c, n_layers, first_layer, w, full, cb, ref0, lambda, lambda_mode, dW, final, stats);
    pkv_ref ref = *ref0;
    for (int l = first_layer; l < n_layers; ++l) {
        int pp = (l - first_layer) & 1;
        pkv_ref_next nx;
        bool last = (l == n_layers - 1);
        if (last && final) {
            nx = *final;
        } else {
            nx.xF_next = c->b.xs[pp];
            nx.xC_next = c->b.xs[2 + pp];
        }
        const pkv_ref_next* pnx = (last && !final) ? nullptr : &nx;
        int rc = build_patch_impl(c, &w[l], &full[l], &cb[l], &ref, lambda, lambda_mode, dW[l], pnx,
                                  stats ? &stats[l] : nullptr);
        if (rc != PKV_OK) return rc;
        ref.xF = nx.xF_next;
        ref.xC = nx.xC_next;
    }
    return PKV_OK;
}

extern "C" size_t pkv_teacher_cache_bytes(const pkv_dims* dims, int n_layers, int N) {
    if (dims_ok(dims) != PKV_OK || n_layers <= 0 || N <= 0) return 0;
    return (size_t)n_layers * teacher_cache_floats_per_layer(*dims, N) * sizeof(float);
}

extern "C" int pkv_build_stack_sweep(pkv_ctx* c, int n_layers, const pkv_block_weights* w, const pkv_kv* full,
                                     const pkv_kv_compressed* cb, const pkv_ref* ref0, int n_lambda,
                                     const float* lambdas, int lambda_mode, float* const* dW, void* teacher_cache,
                                     size_t cache_bytes, pkv_stats* stats) {
    if (!c || !w || !full || !cb || !ref0 || !dW || !lambdas || !teacher_cache || n_layers <= 0 || n_lambda <= 0)
        return PKV_ERR_INVALID_ARG;
    if (c->engine == PKV_ENGINE_SIMT || n_layers > kMaxStackLayers) return PKV_ERR_UNSUPPORTED;
    if (ref0->N <= 0 || ref0->N > c->dims.N_max) return PKV_ERR_INVALID_ARG;
    if (((uintptr_t)teacher_cache & 15) || cache_bytes < pkv_teacher_cache_bytes(&c->dims, n_layers, ref0->N))
        return PKV_ERR_NOMEM;
    for (int j = 0; j < n_lambda; ++j) {
        // the first coefficient runs the teacher (ahead of its students, filling the cache); the others replay
        int rc = build_stack_overlapped(c, n_layers, 0, w, full, cb, ref0, lambdas[j], lambda_mode,
                                        dW + (size_t)j * n_layers, nullptr, stats ? stats + (size_t)j * n_layers : nullptr,
                                        (float*)teacher_cache, j == 0);
        if (rc != PKV_OK) return rc;
    }
    return PKV_OK;
}

// ---- single stages ------------------------------------------------------------------------------

extern "C" int pkv_gather_kept(pkv_ctx* c, const pkv_kv* full, const int32_t* head_off_host, const int32_t* idx,
                               void* Kc, void* Vc, int32_t* bad_head, int32_t* bad_pos) {
    if (!c || !full || !head_off_host) return PKV_ERR_INVALID_ARG;
    pkv_kv_compressed cb{head_off_host, idx, nullptr, nullptr, nullptr};
    int total = 0, max_b = 0;
    int rc = check_compressed(c, &cb, &total, &max_b);
    if (rc != PKV_OK) return rc;
    if (total > 0 && (!idx || !Kc || !Vc || !full->K || !full->V)) return PKV_ERR_INVALID_ARG;
    if (((uintptr_t)Kc & 15) || ((uintptr_t)Vc & 15)) return PKV_ERR_INVALID_ARG;
    Lc lc{c->st, &c->launches, c->map_cache};
    begin_call(c);
    int32_t one[2] = {0, 0};
    upload_meta(c, head_off_host, 0, 0, one);
    gather_kept(lc, c->elem_bytes, full->K, full->V, idx, c->b.head_off, c->dims.Hkv, c->dims.L, c->dims.hd, total,
                Kc, Vc, c->b.status);
    pkv_stats st;
    rc = end_call(c, &st, head_off_host);
    if (bad_head) *bad_head = st.err_info[0];
    if (bad_pos) *bad_pos = st.err_info[1];
    return rc;
}

extern "C" int pkv_dequant_cache(pkv_ctx* c, const pkv_kv_compressed* cb, void* Kc, void* Vc) {
    if (!c || !cb || !Kc || !Vc) return PKV_ERR_INVALID_ARG;
    int total = 0, max_b = 0;
    int rc = check_compressed(c, cb, &total, &max_b);
    if (rc != PKV_OK) return rc;
    if (cb->qbits == 0) return PKV_ERR_INVALID_ARG;
    if (((uintptr_t)Kc & 15) || ((uintptr_t)Vc & 15)) return PKV_ERR_INVALID_ARG;
    Lc lc{c->st, &c->launches, c->map_cache};
    begin_call(c);
    dequant_cache(lc, c->elem_bytes, cb->Kc, cb->k_scale, cb->qbits, cb->qgroup, c->dims.hd, total, Kc);
    dequant_cache(lc, c->elem_bytes, cb->Vc, cb->v_scale, cb->qbits, cb->qgroup, c->dims.hd, total, Vc);
    return end_call(c, nullptr, nullptr);
}

extern "C" int pkv_attention(pkv_ctx* c, const float* q, const float* k_new, const float* v_new,
                             const pkv_kv* full, const pkv_kv_compressed* cb, int32_t N, int32_t n_chunks,
                             const int32_t* chunk_off, float* aF, float* aC, float* dA) {
    if (!c || !q || !k_new || !v_new || !full || !cb || !aF || !aC || !dA) return PKV_ERR_INVALID_ARG;
    const void* vec_ptrs[] = {q, k_new, v_new, aF, aC, dA};      // 16-byte loads and stores
    for (const void* vp : vec_ptrs)
        if ((uintptr_t)vp & 15) return PKV_ERR_INVALID_ARG;
    int rc = check_chunks(c, N, n_chunks, chunk_off);
    if (rc != PKV_OK) return rc;
    int total = 0, max_b = 0;
    rc = check_compressed(c, cb, &total, &max_b);
    if (rc != PKV_OK) return rc;
    const int Dq = c->dims.Hq * c->dims.hd, Dkv = c->dims.Hkv * c->dims.hd;
    Lc lc{c->st, &c->launches, c->map_cache};
    begin_call(c);
    upload_meta(c, cb->head_off, N, n_chunks, chunk_off);
    const void *Kc, *Vc;
    stage_compact(c, lc, full, cb, total, &Kc, &Vc);
    AttnArgs a = attn_args(c, q, Dq, k_new, v_new, Dkv, full, Kc, Vc, cb->idx ? nullptr : cb->bias, N, max_b, total);
    a.aF = aF; a.aC = aC; a.dA = dA;
    if (c->engine == PKV_ENGINE_SIMT) {
        attention_simt(lc, a);
        attention_combine(lc, a);
    } else {
        rc = pkv::tc_attention(lc, &c->b.tc, &c->dims, a, c->b.status);
        if (rc != PKV_OK) return rc;
    }
    return end_call(c, nullptr, cb->head_off);
}

extern "C" int pkv_gram(pkv_ctx* c, const float* X, const float* R, int32_t n, float* S_H, float* S_T,
                        int accumulate) {
    if (!c || !X || !R || !S_H || !S_T || n <= 0 || n > c->dims.N_max) return PKV_ERR_INVALID_ARG;
    Lc lc{c->st, &c->launches, c->map_cache};
    begin_call(c);
    if (c->engine == PKV_ENGINE_SIMT)
        gram_simt(c, lc, X, R, n, S_H, S_T, accumulate != 0);
    else
        pkv::tc_gram(lc, &c->b.tc, &c->dims, X, R, n, S_H, S_T, accumulate != 0, c->b.status);
    return end_call(c, nullptr, nullptr);
}

extern "C" int pkv_ridge_solve_refined(pkv_ctx* c, const float* S_H, const float* S_T, float lambda, int lambda_mode,
                                       int32_t steps, float* dW, pkv_stats* stats) {
    if (!c || !S_H || !S_T || !dW || steps < 0 || steps > 8) return PKV_ERR_INVALID_ARG;
    if (!(lambda > 0.f) || !isfinite(lambda)) return PKV_ERR_INVALID_ARG;
    if (lambda_mode != PKV_LAMBDA_PAPER && lambda_mode != PKV_LAMBDA_ABSOLUTE && lambda_mode != PKV_LAMBDA_TRACE_MEAN)
        return PKV_ERR_INVALID_ARG;
    if (((uintptr_t)S_H & 15) || ((uintptr_t)S_T & 15) || ((uintptr_t)dW & 15)) return PKV_ERR_INVALID_ARG;
    if (c->engine == PKV_ENGINE_SIMT) return PKV_ERR_UNSUPPORTED;
    Lc lc{c->st, &c->launches, c->map_cache};
    begin_call(c);
    const int rc = solve_stage(c, lc, const_cast<float*>(S_H), S_T, lambda, lambda_mode, dW, false, nullptr, steps);
    if (rc != PKV_OK) return rc;
    return end_call(c, stats, nullptr);
}

extern "C" int pkv_fp32_product(pkv_ctx* c, const float* A, const float* B, int32_t M, int32_t N, int32_t K, float alpha,
                                float* C, int accumulate, int passes, int accumulators) {
    if (!c || !A || !B || !C || M <= 0 || N <= 0 || K <= 0) return PKV_ERR_INVALID_ARG;
    if (c->engine == PKV_ENGINE_SIMT) return PKV_ERR_UNSUPPORTED;
    if (((uintptr_t)A & 15) || ((uintptr_t)B & 15) || ((uintptr_t)C & 15)) return PKV_ERR_INVALID_ARG;
    Lc lc{c->st, &c->launches, c->map_cache};
    begin_call(c);
    c->b.tc.S3_ready = 0;              // the operand buffers of the solver are used as scratch
    int rc = pkv::tc_fp32_product(lc, &c->b.tc.solve, (size_t)c->dims.d * c->dims.F, A, B, M, N, K, alpha, C,
                                  accumulate != 0, passes, accumulators, c->b.status);
    if (rc != PKV_OK) return rc;
    return end_call(c, nullptr, nullptr);
}

extern "C" size_t pkv_low_rank_scratch_bytes(const pkv_dims* dims, int r) {
    if (dims_ok(dims) != PKV_OK || r <= 0) return 0;
    return pkv::tc_lowrank_scratch_bytes(dims->d, dims->F, r);
}

extern "C" int pkv_low_rank(pkv_ctx* c, const float* dW, const float* S_H, int32_t r, int32_t iterations, void* scratch,
                            size_t scratch_bytes, float* U, float* Br, float* dW_r, float* ritz_values) {
    if (!c || !dW || !S_H || !scratch || !U || !Br || r <= 0) return PKV_ERR_INVALID_ARG;
    if (c->engine == PKV_ENGINE_SIMT) return PKV_ERR_UNSUPPORTED;
    const void* ptrs[] = {dW, S_H, scratch, U, Br, dW_r, ritz_values};
    for (const void* q : ptrs)
        if ((uintptr_t)q & 15) return PKV_ERR_INVALID_ARG;
    if (scratch_bytes < pkv::tc_lowrank_scratch_bytes(c->dims.d, c->dims.F, r)) return PKV_ERR_NOMEM;
    Lc lc{c->st, &c->launches, c->map_cache};
    begin_call(c);
    int rc = pkv::tc_lowrank(lc, &c->b.tc, &c->dims, dW, S_H, r, iterations > 0 ? iterations : 24, scratch, U, Br, dW_r,
                             ritz_values, c->b.status);
    if (rc != PKV_OK) return rc;
    return end_call(c, nullptr, nullptr);
}

extern "C" int pkv_ridge_solve(pkv_ctx* c, const float* S_H, const float* S_T, float lambda, int lambda_mode,
                               float* dW, pkv_stats* stats) {
    if (!c || !S_H || !S_T || !dW) return PKV_ERR_INVALID_ARG;
    if (!(lambda > 0.f) || !isfinite(lambda)) return PKV_ERR_INVALID_ARG;
    if (lambda_mode != PKV_LAMBDA_PAPER && lambda_mode != PKV_LAMBDA_ABSOLUTE && lambda_mode != PKV_LAMBDA_TRACE_MEAN)
        return PKV_ERR_INVALID_ARG;
    Lc lc{c->st, &c->launches, c->map_cache};
    begin_call(c);
    solve_stage(c, lc, const_cast<float*>(S_H), S_T, lambda, lambda_mode, dW, false);
    return end_call(c, stats, nullptr);
}
