// Tensor-core engine (tcgen05 + TMEM + TMA, sm_100a): interface used by pkv_api.cu.
#pragma once

#include "pkv_internal.h"

namespace pkv {

struct TcBuffers {
    int ready;
};

struct TcForwardArgs {
    const pkv_block_weights* w;
    const pkv_kv* full;
    const void* Kc; const void* Vc; const float* bias;
    const float* xF; const float* xC;
    int N, pos0, max_b, kv_split;
    const int32_t* head_off; const int32_t* tok_cs; float* rope_tab;
    float *zF, *zC, *dz, *hF, *hC, *R, *S_H, *S_T, *aF, *aC;
    float *part_m, *part_l, *part_O;
    DevStatus* status;
    cudaEvent_t* ev;    // stage marks (index = stage) or nullptr
};

int tc_supported(const pkv_dims* d, int cc_major, int cc_minor);
size_t tc_carve(TcBuffers* t, char* base, size_t off, const pkv_dims* d);
int tc_init(TcBuffers* t, const pkv_dims* d);
int tc_forward(const Lc& lc, TcBuffers* t, const pkv_dims* d, const TcForwardArgs& a);
int tc_attention(const Lc& lc, TcBuffers* t, const pkv_dims* d, const AttnArgs& a, DevStatus* status);
void tc_gram(const Lc& lc, TcBuffers* t, const pkv_dims* d, const float* X, const float* R, int n, float* S_H,
             float* S_T, bool accumulate, DevStatus* status);
void tc_ridge_solve(const Lc& lc, TcBuffers* t, const SolveWs& ws, int F, int d, float* dW, DevStatus* status);
void tc_next_states(const Lc& lc, TcBuffers* t, const pkv_dims* d, int N, const void* Wdown, const float* dW,
                    const float* zF, const float* R, float* xF_next, float* D);

}  // namespace pkv
