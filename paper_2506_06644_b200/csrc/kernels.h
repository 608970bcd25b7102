// Internal launch interfaces shared between the entry points (host side).
#pragma once

#include "common.cuh"

namespace spark {

// Spark FFN with the optional fusions the decoder layer uses.
struct FfnArgs {
    const float* x;          // [B][d]
    const float* norm_w;     // nullable: x is replaced by RMSNorm(x; norm_w) on the fly
    float rms_eps;
    const void* K1t;
    const void* K2t;
    const void* Vt;
    int wdtype;
    int64_t B, d, d_ff, r, k;
    int flags;
    const float* y_init;     // nullable: y = y_init + FFN(x) (y_init must not alias y)
    float* y;
    float* theta;
    int32_t* count;
    int32_t* idx;
};
int ffn_launch(spark_ctx* ctx, const FfnArgs& a, cudaStream_t stream);

// Dense GEMV with optional fused RMSNorm on the input.
struct GemvArgs {
    const float* x;          // [B][n_in]
    const float* norm_w;     // nullable
    float rms_eps;
    const void* Wt;          // [n_out][n_in]
    int wdtype;
    int64_t B, n_in, n_out;
    const float* y_add;      // nullable, may alias y
    float* y;
};
int gemv_launch(spark_ctx* ctx, const GemvArgs& a, cudaStream_t stream);

}  // namespace spark
