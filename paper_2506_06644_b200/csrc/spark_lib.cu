// Context management, status handling and host-side helpers of the Spark decode library.
#include <cmath>
#include <cstdlib>
#include <limits>
#include <new>

#include "ffn_params.h"

using namespace spark;

extern "C" {

const char* spark_status_string(int status) {
    switch (status) {
        case SPARK_OK: return "ok";
        case SPARK_ERR_INVALID_ARG: return "invalid argument";
        case SPARK_ERR_UNSUPPORTED: return "unsupported layout, dtype or size";
        case SPARK_ERR_WORKSPACE: return "workspace too small";
        case SPARK_ERR_CUDA: return "CUDA runtime or launch failure";
        case SPARK_ERR_TIMEOUT: return "device: bounded inter-block wait ran out";
        case SPARK_ERR_OVERFLOW: return "device: index list truncated at its capacity";
        case SPARK_ERR_NONFINITE: return "device: non-finite score statistics (SPARK_CHECK_FINITE)";
        default: return "unknown status";
    }
}

// Q(1 - p) of Eq. 11 for the threshold, as the root of 0.5 * erfc(z / sqrt 2) = p.
// Start from the classical rational approximation for the normal tail (Abramowitz & Stegun
// 26.2.23, |error| < 4.5e-4) and polish with Newton steps on the tail function, whose derivative
// is minus the normal density.  The upper-tail form keeps small p free of cancellation.
double spark_normal_upper_quantile(double p) {
    if (!(p > 0.0 && p < 1.0)) return std::numeric_limits<double>::quiet_NaN();
    if (p > 0.5) return -spark_normal_upper_quantile(1.0 - p);
    const double t = std::sqrt(-2.0 * std::log(p));
    double z = t - (2.515517 + t * (0.802853 + t * 0.010328)) /
                       (1.0 + t * (1.432788 + t * (0.189269 + t * 0.001308)));
    const double inv_sqrt2 = 0.70710678118654752440;
    const double inv_sqrt2pi = 0.39894228040143267794;
    for (int it = 0; it < 60; ++it) {
        const double tail = 0.5 * std::erfc(z * inv_sqrt2);
        const double dens = inv_sqrt2pi * std::exp(-0.5 * z * z);
        const double step = (tail - p) / dens;
        z += step;
        if (std::fabs(step) <= 1e-16 * std::fmax(1.0, std::fabs(z))) break;
    }
    return z;
}

size_t spark_workspace_bytes(int64_t max_batch, int64_t max_dff, int64_t max_cap, int64_t n_q,
                             int64_t hd, int64_t max_d) {
    if (max_batch < 1) max_batch = 1;
    if (max_dff < 0) max_dff = 0;
    if (max_cap < 0) max_cap = 0;
    if (n_q < 1) n_q = 1;
    if (hd < 8) hd = 8;
    if (max_d < 0) max_d = 0;
    const size_t grid_bound = 1024;   // more thread blocks than any device has SMs x residency
    // attention: score-sum cells, per-piece partial outputs, and room for the predictor scores of
    // blocks whose share does not fit in shared memory.
    const size_t pieces = grid_bound + static_cast<size_t>(max_batch) * n_q;
    const size_t need = kAttnCellBytes +
                        round_up(pieces * 8 * (static_cast<size_t>(hd) + 8) * 4, 256) +
                        round_up((static_cast<size_t>(max_batch) * n_q * max_cap + grid_bound * 8) * 4, 256);
    // FFN over chunks of five and more tokens: split inputs, scores and activations of the tensor-core path,
    // placed behind the attention's cells (the two never run at the same time on one context)
    size_t need_ffn = 0;
    if (max_batch >= 5 && max_dff > 0 && max_d > 0) need_ffn = kAttnCellBytes + ffn_tc_workspace_bytes(max_d, max_dff);
    // attention over a chunk of a prompt (16 and more tokens sharing one cache): split queries and the score matrix of the
    // tensor-core path, at most n_q KV heads x 128 columns x (max_cap + 32) scores
    size_t need_chunk = 0;
    if (max_batch >= 16)
        need_chunk = kAttnCellBytes + 4096 + 4 * round_up(static_cast<size_t>(n_q) * 128 * 128 * 2, 1024) +      // both query parts
                     round_up(static_cast<size_t>(n_q) * 128 * (static_cast<size_t>(max_cap) + 32) * 4, 1024) +
                     round_up(static_cast<size_t>(n_q) * (128 * 16 + 64 * 4), 1024) + 1024;                    // column facts of the dense stage
    size_t most = need > need_ffn ? need : need_ffn;
    if (need_chunk > most) most = need_chunk;
    return sizeof(WsHeader) + most + 256;
}

int spark_create(spark_ctx** out, int device, void* workspace, size_t workspace_bytes) {
    if (out == nullptr || workspace == nullptr) return SPARK_ERR_INVALID_ARG;
    *out = nullptr;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return SPARK_ERR_UNSUPPORTED;
    if (workspace_bytes < sizeof(WsHeader) + 256) return SPARK_ERR_WORKSPACE;
    if (cudaSetDevice(device) != cudaSuccess) return SPARK_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SPARK_ERR_CUDA;
    // the whole workspace starts zeroed: header words, score-sum cells and per-segment counters are
    // idle at zero, and the kernels leave them so
    // (the memset runs on the legacy default stream and may still be in flight when it returns; kernels the caller
    // then launches on a non-blocking stream are not ordered behind it, hence the synchronisation)
    if (cudaMemset(workspace, 0, workspace_bytes) != cudaSuccess) return SPARK_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return SPARK_ERR_CUDA;
    spark_ctx* c = new (std::nothrow) spark_ctx;
    if (c == nullptr) return SPARK_ERR_INVALID_ARG;
    c->device = device;
    c->num_sms = prop.multiProcessorCount;
    c->max_smem_optin = static_cast<int>(prop.sharedMemPerBlockOptin);
    c->ws = static_cast<char*>(workspace);
    c->ws_bytes = workspace_bytes;
    c->hdr = reinterpret_cast<WsHeader*>(workspace);
    c->scratch = c->ws + sizeof(WsHeader);
    c->scratch_bytes = workspace_bytes - sizeof(WsHeader);
    c->trace = nullptr;
    c->trace_cap = 0;
    c->overlap = 0;
    c->wait_kcycles = 0;
    c->fused = 0;
    c->chunk_dense = 1;
    c->len_hint = 0;
    c->l2_prefetch = 0;
    c->next_wqkv = nullptr;
    c->debug_extra_arrivals = 0;
    *out = c;
    return SPARK_OK;
}

int spark_destroy(spark_ctx* ctx) {
    delete ctx;
    return SPARK_OK;
}

int spark_set_phase_trace(spark_ctx* ctx, uint64_t* trace, int64_t capacity) {
    if (ctx == nullptr || (trace != nullptr && capacity < 16)) return SPARK_ERR_INVALID_ARG;
    ctx->trace = reinterpret_cast<unsigned long long*>(trace);
    ctx->trace_cap = trace != nullptr ? capacity : 0;
    return SPARK_OK;
}

int spark_set_launch_overlap(spark_ctx* ctx, int on) {
    if (ctx == nullptr) return SPARK_ERR_INVALID_ARG;
    ctx->overlap = on ? 1 : 0;
    return SPARK_OK;
}

int spark_grid_size(const spark_ctx* ctx) { return ctx ? ctx->num_sms : 0; }

int spark_set_l2_prefetch(spark_ctx* ctx, int on) {
    if (ctx == nullptr) return SPARK_ERR_INVALID_ARG;
    ctx->l2_prefetch = on ? 1 : 0;
    return SPARK_OK;
}

int spark_set_chunk_dense(spark_ctx* ctx, int mode) {
    if (ctx == nullptr || mode < 0 || mode > 2) return SPARK_ERR_INVALID_ARG;
    ctx->chunk_dense = mode;
    return SPARK_OK;
}

int spark_set_fused_layer(spark_ctx* ctx, int on) {
    if (ctx == nullptr) return SPARK_ERR_INVALID_ARG;
    ctx->fused = on ? 1 : 0;
    return SPARK_OK;
}

int spark_set_wait_limit(spark_ctx* ctx, void* stream, int64_t cycles) {
    if (ctx == nullptr || cycles < 0) return SPARK_ERR_INVALID_ARG;
    if (!on_device(ctx)) return SPARK_ERR_INVALID_ARG;
    int64_t k = (cycles + 1023) >> 10;
    if (k > 0xffffffffll) k = 0xffffffffll;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return SPARK_ERR_CUDA;      // no kernel of this context reads the word meanwhile
    ctx->wait_kcycles = static_cast<unsigned>(k);
    if (cudaMemcpy(&ctx->hdr->wait_kcycles, &ctx->wait_kcycles, sizeof(unsigned), cudaMemcpyHostToDevice) != cudaSuccess)
        return SPARK_ERR_CUDA;
    return cudaDeviceSynchronize() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

int spark_debug_expect_arrivals(spark_ctx* ctx, int extra) {
    if (ctx == nullptr || extra < 0) return SPARK_ERR_INVALID_ARG;
    ctx->debug_extra_arrivals = extra;
    return SPARK_OK;
}

int spark_device_status(spark_ctx* ctx, void* stream, int* host_out) {
    if (ctx == nullptr || host_out == nullptr) return SPARK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return SPARK_ERR_CUDA;
    int status = 0;
    if (cudaMemcpy(&status, &ctx->hdr->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
        return SPARK_ERR_CUDA;
    *host_out = status;
    if (status != SPARK_OK) {
        // a failed phase may have left arrivals or partial sums behind: back to the idle (zero) state
        if (cudaMemset(ctx->ws, 0, ctx->ws_bytes) != cudaSuccess) return SPARK_ERR_CUDA;
        if (ctx->wait_kcycles != 0u &&
            cudaMemcpy(&ctx->hdr->wait_kcycles, &ctx->wait_kcycles, sizeof(unsigned), cudaMemcpyHostToDevice) != cudaSuccess)
            return SPARK_ERR_CUDA;
        if (cudaDeviceSynchronize() != cudaSuccess) return SPARK_ERR_CUDA;      // the reset is complete before the next launch, on any stream
    }
    return SPARK_OK;
}

}  // extern "C"
