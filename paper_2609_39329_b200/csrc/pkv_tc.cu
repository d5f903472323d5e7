// Tensor-core engine: not built yet in this file's first form; creation of a bf16 context
// with PKV_ENGINE_AUTO reports PKV_ERR_UNSUPPORTED (there is no silent fallback).
#include "pkv_tc.h"

namespace pkv {

int tc_supported(const pkv_dims*, int, int) { return PKV_ERR_UNSUPPORTED; }
size_t tc_carve(TcBuffers*, char*, size_t off, const pkv_dims*) { return off; }
int tc_init(TcBuffers*, const pkv_dims*) { return PKV_ERR_UNSUPPORTED; }
int tc_forward(const Lc&, TcBuffers*, const pkv_dims*, const TcForwardArgs&) { return PKV_ERR_UNSUPPORTED; }
int tc_attention(const Lc&, TcBuffers*, const pkv_dims*, const AttnArgs&, DevStatus*) { return PKV_ERR_UNSUPPORTED; }
void tc_gram(const Lc&, TcBuffers*, const pkv_dims*, const float*, const float*, int, float*, float*, bool,
             DevStatus*) {}
void tc_ridge_solve(const Lc&, TcBuffers*, const SolveWs&, int, int, float*, DevStatus*) {}
void tc_next_states(const Lc&, TcBuffers*, const pkv_dims*, int, const void*, const float*, const float*,
                    const float*, float*, float*) {}

}  // namespace pkv
