// TF32 tensor-core GEMM for the GraphSage linear layers (placeholder until the tcgen05 kernel lands).
#include "mg_internal.cuh"

int mg_gemm_tf32(mg_ctx* ctx, const float*, const float*, const float*, float*, int64_t, int, int, bool) {
    return mg_fail(ctx, MG_ERR_STATE, "TF32 tensor-core GEMM not built");
}
