// Kernel parameters of the two-tile attention kernel (shared by its launcher and its caller).
#pragma once

#include <cuda.h>

#include "pkv_internal.h"

namespace pkv {

struct alignas(64) Attn2Params {
    CUtensorMap mQhi, mQlo;   // {hd, N*g, 2*Hkv}
    CUtensorMap mK, mV;       // {hd, L, Hkv}
    CUtensorMap mKc, mVc;     // {hd, total kept rows}
    CUtensorMap mKn, mVn;     // {hd, N, 2*Hkv}
    const int32_t* head_off;
    const int32_t* tok_cs;
    const float* bias;
    int N, g, Hkv, L, rows;
    int tps, nsplitF, nsplitC;
    int q_f16;                // queries are one fp16 part and every key operand is fp16 (one QK^T pass) instead of
                              // a bf16 hi + lo query pair against bf16 keys (two passes)
    int z0;                   // first split index of this launch (teacher splits come first, then the student's)
    int zoffC;                // slot of the student's first split in the partial buffers
    float* part_m;
    float* part_l;
    float* part_O;
    DevStatus* status;
};

}  // namespace pkv
