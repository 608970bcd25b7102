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
    const float* K1s;        // per-neuron scales [d_ff] of K1t, K2t, Vt: required for SPARK_FP8_E4M3, nullptr otherwise
    const float* K2s;
    const float* Vs;
    int64_t B, d, d_ff, r, k;
    int flags;
    const float* y_init;     // nullable: y = y_init + FFN(x) (y_init must not alias y)
    float* y;
    float* theta;
    int32_t* count;
    int32_t* idx;
    PrefetchSpec pf = PrefetchSpec{nullptr, 0};      // weights of the kernel after this one, asked into L2 (one token)
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
    const float* x_div;      // nullable: x[b][i] is divided by x_div[b][i / x_div_group] (0 where that is 0)
    int64_t x_div_group;
    void* zero_ptr;          // nullable: this many bytes (multiple of 16) are cleared by the kernel as a side job
    size_t zero_bytes;
    const void* pf_ptr;      // nullable: weights of the kernel after this one, asked into L2 (one token)
    unsigned long long pf_bytes;
};
int gemv_launch(spark_ctx* ctx, const GemvArgs& a, cudaStream_t stream);
// The same product for 5..16 tokens and bf16 weights as a TMA-fed tcgen05 GEMM (gemm_tc.cu); SPARK_ERR_WORKSPACE = shape or
// workspace not served (n_in % 64, n_out % 128, room for the split input behind the attention's cells).
int gemm_tc_launch(spark_ctx* ctx, const GemvArgs& a, cudaStream_t stream);

// Spark attention; zs (nullable) holds Q(1 - k_attn / L_b) per sequence when an earlier kernel of the
// same stream has already computed it.  With lsum != nullptr the kernel leaves o unnormalised (the
// weighted value sums), writes the sums of weights to lsum[B][n_q] and leaves its score-sum cells
// for the caller's next kernel to clear (the first B * n_q * kAttnWays cells of the scratch area).  With k1s !=
// nullptr the predictor slice k1c is FP8 E4M3 and k1s[B][n_kv][cap] holds one scale per cached row (bf16 k2c / vc).
int attn_launch(spark_ctx* ctx, const float* q, const void* k1c, const void* k2c, const void* vc, int kvdtype, int64_t B,
                int64_t n_q, int64_t n_kv, int64_t hd, int64_t r, int64_t cap, const int32_t* ctx_len, const double* zs,
                int64_t window, int64_t k_attn, int flags, float* o, float* lsum, float* theta, int32_t* count, int32_t* idx,
                int64_t idx_cap, const float* k1s, cudaStream_t st, PrefetchSpec pf = PrefetchSpec{nullptr, 0},
                const float* k2s = nullptr, const float* vs = nullptr);      // k2s / vs: row scales of an FP8 k2c / vc

// Spark attention for a chunk of a prompt (T consecutive tokens of one sequence over one cache, bf16): predictor scores of
// the whole chunk as one tcgen05 GEMM per KV head (attn_chunk.cu).  o is written normalised; lsum (nullable) receives 1 per
// head (0 for an empty selection).  SPARK_ERR_WORKSPACE = shape or workspace not served.
int attn_chunk_launch(spark_ctx* ctx, const float* q, const void* k1c, const void* k2c, const void* vc, int64_t T, int64_t n_q,
                      int64_t n_kv, int64_t hd, int64_t r, int64_t cap, const int32_t* ctx_len, const double* zs, int64_t window,
                      int64_t k_attn, float* o, float* lsum, float* theta, int32_t* count, cudaStream_t stream);

// One token through n_layers decoder layers in one launch of the fused persistent kernel (layer1.cu); the layers' configurations
// are equal but for the attention window.  SPARK_ERR_WORKSPACE = shape, flags or sizes not served.
int layer1_launch(spark_ctx* ctx, const spark_layer_weights* w, const spark_layer_cfg* cfg, const spark_kv_cache* cache, int n_layers,
                  const int32_t* ctx_len, float* h, float* scratch, cudaStream_t stream);

}  // namespace spark
