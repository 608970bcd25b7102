// Kernel parameters of the Spark FFN kernels (internal).
#pragma once

#include "common.cuh"

namespace spark {

constexpr int kFfnMaxTB = 16;     // tokens per pass over the weights

struct FfnParams {
    const float* x;
    const float* norm_w;
    float eps;
    const void* K1t;
    const void* K2t;
    const void* Vt;
    const float* K1s;             // nullable: per-neuron scales of the three matrices (FP8 storage), [d_ff] each
    const float* K2s;
    const float* Vs;
    int B, d, d_ff, r, rpc, xw;
    int ncopy;                    // B == 1 kernel: per-warp copies of y in shared memory
    int dense, erf_form, identity;
    int xres;                     // tensor-core kernel: both halves of the split input stay in shared memory
    int vrows, vstage_off;        // few-token kernel: rows of V per round and the byte offset of their staging area
    int overlap;                  // launched with the programmatic attribute: weights first, then dep_wait()
    int extra_arrivals;           // test hook (one-token kernel): arrivals waited for beyond the grid's blocks
    PrefetchSpec pf;              // one-token kernel: weights of the kernel after this one, asked into L2 during the exchange
    int check_finite;             // SPARK_CHECK_FINITE: non-finite score sums are reported in the device status
    double z;
    double inv_n, inv_nm1;        // 1 / d_ff and 1 / (d_ff - 1)
    const float* y_init;
    float* y;
    float* theta;
    int32_t* count;
    int32_t* idx;
    WsHeader* hdr;
    PhaseTrace trace;
};


// Tensor-core path for bf16 weights and 2..64 tokens (ffn_mma.cu); SPARK_ERR_WORKSPACE = shape not
// served, use the plain-ALU kernel.
int ffn_mma_launch(spark_ctx* ctx, FfnParams& p, cudaStream_t stream);

// Chunks of up to 64 tokens on tcgen05 tensor cores, every weight row read (ffn_tc.cu); SPARK_ERR_WORKSPACE =
// shape or workspace not served.
int ffn_tc_launch(spark_ctx* ctx, FfnParams& p, cudaStream_t stream);
size_t ffn_tc_workspace_bytes(int64_t d, int64_t d_ff);

// 2..4 tokens without tensor cores (ffn_few.cu); SPARK_ERR_WORKSPACE = shape not served.
int ffn_few_launch(spark_ctx* ctx, FfnParams& p, int wdtype, cudaStream_t stream);

// B == 1 fast path (ffn_b1.cu).
int ffn1_launch(spark_ctx* ctx, FfnParams& p, int wdtype, cudaStream_t stream);

}  // namespace spark
