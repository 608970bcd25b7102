// Dense glue of a decoder layer (Section 4): GEMV with optional fused RMSNorm / residual, rotary
// position encoding on each half of q and k with the cache append, and spark_layer_decode, which
// chains them around Spark attention and Spark FFN.  The projections stay dense: the method does
// not change them (Table "FLOPs per token").
#include <cmath>

#include <new>

#include "kernels.h"
#include "mma_rows.cuh"
#include "rowdot.cuh"

using namespace spark;

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / kWarp;

struct GemvParams {
    const float* x;
    const float* norm_w;
    float eps;
    const void* Wt;
    int B, n_in, n_out;
    const float* y_add;
    float* y;
    const float* x_div;
    int x_div_group;
    uint4* zero_ptr;
    int zero_n16;
    int overlap;             // launched with the programmatic attribute: weights first, then dep_wait()
    PrefetchSpec pf;         // weights of the kernel after this one: asked into L2 once this kernel's own loads are in flight
};

// Input staging shared by the GEMV kernels: x (optionally divided per group, optionally RMS-normalised)
// into shared memory as [TB][n_in]; also the kernel's clear-region side job.  Ends with a block sync.
// One token: the input is requested into registers BEFORE the weight loads are issued (requests are
// served in issue order, so this is what puts x in shared memory by the time the first rows land).
struct EarlyX {
    float4 v0, v1;           // the thread's two float4 of x
    float4 w0, w1;           // the norm weights at the same places
    float d0, d1;            // the divisors of their groups
    bool on;
};
__device__ __forceinline__ EarlyX early_x_request(const GemvParams& p, bool after_dependency) {
    EarlyX e;
    e.v0 = make_float4(0.f, 0.f, 0.f, 0.f);
    e.v1 = e.v0;
    e.w0 = make_float4(1.f, 1.f, 1.f, 1.f);
    e.w1 = e.w0;
    e.d0 = e.d1 = 1.f;
    const int n4 = p.n_in / 4, tid = threadIdx.x;
    e.on = p.B == 1 && n4 <= 2 * kThreads;
    if (e.on && (!p.overlap || after_dependency)) {
        const bool h0 = tid < n4, h1 = tid + kThreads < n4;
        if (h0) e.v0 = reinterpret_cast<const float4*>(p.x)[tid];
        if (h1) e.v1 = reinterpret_cast<const float4*>(p.x)[tid + kThreads];
        if (p.x_div != nullptr) {
            if (h0) e.d0 = p.x_div[(tid * 4) / p.x_div_group];
            if (h1) e.d1 = p.x_div[((tid + kThreads) * 4) / p.x_div_group];
        }
        if (p.norm_w != nullptr) {
            if (h0) e.w0 = reinterpret_cast<const float4*>(p.norm_w)[tid];
            if (h1) e.w1 = reinterpret_cast<const float4*>(p.norm_w)[tid + kThreads];
        }
    }
    return e;
}

template <int TB>
__device__ __forceinline__ void stage_input(const GemvParams& p, float* xs, float* rstd, const EarlyX& ex) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_in = p.n_in;
    const int w4 = n_in / 4;
    if (ex.on) {
        // one token, everything already in registers: divide, normalise, store -- one block-wide sum
        for (int i = blockIdx.x * kThreads + tid; i < p.zero_n16; i += gridDim.x * kThreads)
            p.zero_ptr[i] = make_uint4(0u, 0u, 0u, 0u);
        float4 v0 = ex.v0, v1 = ex.v1;
        if (p.x_div != nullptr) {
            const float i0 = ex.d0 > 0.f ? 1.f / ex.d0 : 0.f, i1 = ex.d1 > 0.f ? 1.f / ex.d1 : 0.f;
            v0.x *= i0; v0.y *= i0; v0.z *= i0; v0.w *= i0;
            v1.x *= i1; v1.y *= i1; v1.z *= i1; v1.w *= i1;
        }
        if (p.norm_w != nullptr) {
            float ss = v0.x * v0.x + v0.y * v0.y + v0.z * v0.z + v0.w * v0.w + v1.x * v1.x + v1.y * v1.y + v1.z * v1.z + v1.w * v1.w;
            ss = warp_sum(ss);
            if (lane == 0) rstd[warp] = ss;
            __syncthreads();
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) tot += rstd[w];
            const float sc = rsqrtf(tot / static_cast<float>(n_in) + p.eps);
            v0.x *= sc * ex.w0.x; v0.y *= sc * ex.w0.y; v0.z *= sc * ex.w0.z; v0.w *= sc * ex.w0.w;
            v1.x *= sc * ex.w1.x; v1.y *= sc * ex.w1.y; v1.z *= sc * ex.w1.z; v1.w *= sc * ex.w1.w;
        }
        if (tid < w4) reinterpret_cast<float4*>(xs)[tid] = v0;
        if (tid + kThreads < w4) reinterpret_cast<float4*>(xs)[tid + kThreads] = v1;
        for (int i = w4 + tid; i < TB * w4; i += kThreads) reinterpret_cast<float4*>(xs)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        __syncthreads();
        return;
    }
    for (int i = tid; i < TB * w4; i += kThreads) {
        const int t = i / w4, c = i - t * w4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (t < p.B) {
            v = reinterpret_cast<const float4*>(p.x + static_cast<int64_t>(t) * n_in)[c];
            if (p.x_div != nullptr) {
                const float dv = p.x_div[static_cast<int64_t>(t) * (n_in / p.x_div_group) + (c * 4) / p.x_div_group];
                const float inv = dv > 0.f ? 1.f / dv : 0.f;
                v.x *= inv; v.y *= inv; v.z *= inv; v.w *= inv;
            }
        }
        reinterpret_cast<float4*>(xs + static_cast<size_t>(t) * n_in)[c] = v;
    }
    for (int i = blockIdx.x * kThreads + tid; i < p.zero_n16; i += gridDim.x * kThreads)
        p.zero_ptr[i] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    if (p.norm_w != nullptr) {
        for (int t = warp; t < TB; t += kWarps) {
            float ss = 0.f;
            for (int i = lane; i < n_in; i += 32) {
                const float v = xs[static_cast<size_t>(t) * n_in + i];
                ss = fmaf(v, v, ss);
            }
            ss = warp_sum(ss);
            if (lane == 0) rstd[t] = rsqrtf(ss / static_cast<float>(n_in) + p.eps);
        }
        __syncthreads();
        for (int i = tid; i < TB * n_in; i += kThreads) {
            const int t = i / n_in, c = i - t * n_in;
            xs[i] *= rstd[t] * p.norm_w[c];
        }
        __syncthreads();
    }
}

// y[b][o] = Wt[o][:] . xhat[b][:] (+ y_add[b][o]);  xhat = x or RMSNorm(x; norm_w).
template <typename WT, int TB, int RW>
__global__ void __launch_bounds__(kThreads, 1) gemv_kernel(const GemvParams p) {
    extern __shared__ __align__(16) float xs[];       // [TB][n_in]
    __shared__ float rstd[16];
    const int n_in = p.n_in;
    const int row0 = static_cast<int>(static_cast<int64_t>(blockIdx.x) * p.n_out / gridDim.x);
    const int row1 = static_cast<int>(static_cast<int64_t>(blockIdx.x + 1) * p.n_out / gridDim.x);
    EarlyX ex = early_x_request(p, false);
    auto dependency = [&]() {                                     // runs once the first slice of weight loads is in flight
        if (threadIdx.x == kThreads - 1) prefetch_l2_share(p.pf, blockIdx.x, gridDim.x);
        if (p.overlap) {
            dep_wait();
            dep_trigger();
            ex = early_x_request(p, true);
        }
    };
    auto fill_x = [&]() { stage_input<TB>(p, xs, rstd, ex); };   // runs once the first batch is in flight
    rows_dot<WT, TB, RW>(static_cast<const WT*>(p.Wt), n_in, row0, row1 - row0, n_in / 8, xs, n_in, dependency, fill_x,
                         [&](int j, int t, float v) {
                             if (t < p.B) {
                                 const int64_t o = static_cast<int64_t>(t) * p.n_out + row0 + j;
                                 p.y[o] = p.y_add != nullptr ? v + p.y_add[o] : v;
                             }
                         });
}

// The same product for 5..16 tokens on the tensor cores: with that many tokens the plain-ALU kernel is bound by
// the shared-memory reads of the inputs (every 16 bytes of weights meet 16 x 32 bytes of activations).  The
// inputs (divided, normalised) are staged once as a two-term bf16 split; the block's rows go through mma_rows.
template <int TB>
__global__ void __launch_bounds__(kThreads, 1) gemv_mma_kernel(const GemvParams p) {
    using namespace spark::mma;
    constexpr int NT = TB / 8;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int n_in = p.n_in, xsd = Plan::pad(n_in), tb_stride = TB * xsd;
    __nv_bfloat16* xs2 = reinterpret_cast<__nv_bfloat16*>(smem_raw);                 // [2][TB][xsd]
    float4* part = reinterpret_cast<float4*>(xs2 + 2 * tb_stride);                   // [kWarps][NT][32]
    __shared__ float rstd[16];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row0 = static_cast<int>(static_cast<int64_t>(blockIdx.x) * p.n_out / gridDim.x);
    const int row1 = static_cast<int>(static_cast<int64_t>(blockIdx.x + 1) * p.n_out / gridDim.x);
    dep_wait();
    dep_trigger();
    for (int i = blockIdx.x * kThreads + tid; i < p.zero_n16; i += gridDim.x * kThreads) p.zero_ptr[i] = make_uint4(0u, 0u, 0u, 0u);
    const int w4 = n_in / 4;
    auto divisor = [&](int t, int c4) -> float {
        if (p.x_div == nullptr) return 1.f;
        const float dv = p.x_div[static_cast<int64_t>(t) * (n_in / p.x_div_group) + (c4 * 4) / p.x_div_group];
        return dv > 0.f ? 1.f / dv : 0.f;
    };
    if (p.norm_w != nullptr) {                        // a warp per token: sum of squares of the (divided) input
        for (int t = warp; t < TB; t += kWarps) {
            float ss = 0.f;
            if (t < p.B) {
                const float4* xr = reinterpret_cast<const float4*>(p.x + static_cast<int64_t>(t) * n_in);
                for (int i = lane; i < w4; i += 32) {
                    const float4 v = xr[i];
                    const float iv = divisor(t, i);
                    ss += (v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w) * iv * iv;
                }
                ss = warp_sum(ss);
            }
            if (lane == 0) rstd[t] = rsqrtf(ss / static_cast<float>(n_in) + p.eps);
        }
        __syncthreads();
    }
    constexpr int SB = 8;                             // loads a thread keeps in flight
    for (int i0 = tid; i0 < TB * w4; i0 += kThreads * SB) {
        float4 v[SB];
        float sc[SB];
        int tt[SB], cc[SB];
#pragma unroll
        for (int j = 0; j < SB; ++j) {
            const int i = i0 + j * kThreads;
            tt[j] = i / w4;
            cc[j] = i - tt[j] * w4;
            v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            sc[j] = 1.f;
            if (i < TB * w4 && tt[j] < p.B) {
                v[j] = reinterpret_cast<const float4*>(p.x + static_cast<int64_t>(tt[j]) * n_in)[cc[j]];
                sc[j] = divisor(tt[j], cc[j]);
            }
        }
#pragma unroll
        for (int j = 0; j < SB; ++j) {
            const int i = i0 + j * kThreads;
            if (i >= TB * w4) break;
            float4 w = make_float4(1.f, 1.f, 1.f, 1.f);
            float s = sc[j];
            if (p.norm_w != nullptr) {
                w = __ldg(reinterpret_cast<const float4*>(p.norm_w) + cc[j]);
                s *= tt[j] < p.B ? rstd[tt[j]] : 0.f;
            }
            const float f[4] = {v[j].x * s * w.x, v[j].y * s * w.y, v[j].z * s * w.z, v[j].w * s * w.w};
            const unsigned h01 = pack_bf16x2(f[0], f[1]), h23 = pack_bf16x2(f[2], f[3]);
            const unsigned m01 = pack_bf16x2(f[0] - __uint_as_float(h01 << 16), f[1] - __uint_as_float(h01 & 0xffff0000u));
            const unsigned m23 = pack_bf16x2(f[2] - __uint_as_float(h23 << 16), f[3] - __uint_as_float(h23 & 0xffff0000u));
            __nv_bfloat16* dst = xs2 + static_cast<size_t>(tt[j]) * xsd + 4 * cc[j];
            *reinterpret_cast<uint2*>(dst) = make_uint2(h01, h23);
            *reinterpret_cast<uint2*>(dst + tb_stride) = make_uint2(m01, m23);
        }
    }
    __syncthreads();
    const __nv_bfloat16* Wt = static_cast<const __nv_bfloat16*>(p.Wt);
    mma_rows<NT, 8>([&](int i) { return Wt + static_cast<int64_t>(row0 + i) * n_in; }, row1 - row0, n_in / 32, xs2, xsd, tb_stride, part,
                    [&](int i, int tok, float v) {
                        if (tok < p.B) {
                            const int64_t o = static_cast<int64_t>(tok) * p.n_out + row0 + i;
                            p.y[o] = p.y_add != nullptr ? v + p.y_add[o] : v;
                        }
                    });
}

template <int TB>
int gemv_mma_launch(spark_ctx* ctx, GemvParams& p, int grid, cudaStream_t stream) {
    static bool configured[64] = {};
    const size_t smem = static_cast<size_t>(2) * TB * spark::mma::Plan::pad(p.n_in) * 2 + static_cast<size_t>(kWarps) * (TB / 8) * 32 * 16;
    if (smem > static_cast<size_t>(ctx->max_smem_optin - 1024)) return SPARK_ERR_WORKSPACE;
    auto kern = gemv_mma_kernel<TB>;
    if (ctx->device >= 0 && ctx->device < 64 && !configured[ctx->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin - 1024) != cudaSuccess)
            return SPARK_ERR_CUDA;
        configured[ctx->device] = true;
    }
    p.overlap = ctx->overlap;
    void* args[] = {&p};
    return launch_kernel(ctx, reinterpret_cast<const void*>(kern), static_cast<unsigned>(grid), kThreads, smem, stream, false, args) == cudaSuccess
               ? SPARK_OK : SPARK_ERR_CUDA;
}

template <typename WT, int TB, int RW>
int gemv_launch_one(spark_ctx* ctx, GemvParams& p, size_t smem, int grid, cudaStream_t stream) {
    static bool configured[64] = {};
    auto kern = gemv_kernel<WT, TB, RW>;
    if (ctx->device >= 0 && ctx->device < 64 && !configured[ctx->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin - 1024) != cudaSuccess)
            return SPARK_ERR_CUDA;
        configured[ctx->device] = true;
    }
    p.overlap = ctx->overlap;
    void* args[] = {&p};
    return launch_kernel(ctx, reinterpret_cast<const void*>(kern), static_cast<unsigned>(grid), kThreads, smem, stream, false, args) == cudaSuccess
               ? SPARK_OK : SPARK_ERR_CUDA;
}

template <typename WT, int TB>
int gemv_dispatch_rw(spark_ctx* ctx, GemvParams& p, int rw, size_t smem, int grid, cudaStream_t stream) {
    if (rw == 1) return gemv_launch_one<WT, TB, 1>(ctx, p, smem, grid, stream);
    if (rw == 2) return gemv_launch_one<WT, TB, 2>(ctx, p, smem, grid, stream);
    return gemv_launch_one<WT, TB, 4>(ctx, p, smem, grid, stream);
}

template <typename WT>
int gemv_dispatch(spark_ctx* ctx, GemvParams& p, int tb, int rw, size_t smem, int grid, cudaStream_t stream) {
    if (tb == 1) return gemv_dispatch_rw<WT, 1>(ctx, p, rw, smem, grid, stream);
    if (tb == 4) return gemv_dispatch_rw<WT, 4>(ctx, p, rw, smem, grid, stream);
    return gemv_dispatch_rw<WT, 16>(ctx, p, rw, smem, grid, stream);
}

// ---------------------------------------------------------------------------------------------
// Rotary position encoding on each half of q and k, 1/sqrt(hd) on q, cache append (Section 4:
// the encoding is applied to q[:r], q[r:], and to the columns of K1 and of K2).
// Part of m dims: pairs (i, i + m/2), pair i turned by pos * base^(-2i/m).
// ---------------------------------------------------------------------------------------------
struct RopeParams {
    const float* qkv;        // [B][(n_q + 2 n_kv) hd]
    float* q_out;            // [B][n_q][hd]
    __nv_bfloat16* k1c;
    __nv_bfloat16* k2c;
    __nv_bfloat16* vc;
    const int32_t* ctx_len;
    int B, n_q, n_kv, hd, r;
    int shared;              // 1: one cache [n_kv][cap][.] for all B tokens (consecutive tokens of one sequence)
    int64_t cap;
    float base, q_scale;
    double* zs;              // [B] out: Q(1 - k_attn / L_b) for the attention kernel that follows
    int window, k_attn;
    float* k1f32;            // nullable: the rotated predictor part of the new keys goes here in fp32 (element i of KV head g of
                             // token b at b * k1f32_sb + g * k1f32_sg + i) instead of into k1c: an FP8 slice is quantised by its own kernel
    int64_t k1f32_sb, k1f32_sg;
    double inv_freq[2][64];  // base^(-2i/m) for the pairs of the first part (m = r) and of the second (m = hd - r)
};

__global__ void rope_append_kernel(const RopeParams p) {
    dep_wait();        // the projections come from the kernel ahead
    dep_trigger();
    if (blockIdx.x == 0 && threadIdx.x < p.B) {         // the threshold quantile of each sequence's window
        int n = p.ctx_len[threadIdx.x];
        n = n < 1 ? 1 : (n > p.cap ? static_cast<int>(p.cap) : n);
        const int L = (p.window > 0 && p.window < n) ? p.window : n;
        p.zs[threadIdx.x] = p.k_attn >= L ? 0.0 : -normcdfinv(static_cast<double>(p.k_attn) / static_cast<double>(L));
    }
    const int heads = p.n_q + 2 * p.n_kv;
    const int half_hd = p.hd / 2;
    const int64_t total = static_cast<int64_t>(p.B) * heads * half_hd;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int pr = static_cast<int>(i % half_hd);
        const int h = static_cast<int>((i / half_hd) % heads);
        const int b = static_cast<int>(i / (static_cast<int64_t>(half_hd) * heads));
        int n = p.ctx_len[b];
        n = n < 1 ? 1 : (n > p.cap ? static_cast<int>(p.cap) : n);
        const int pos = n - 1;
        const float* src = p.qkv + (static_cast<int64_t>(b) * heads + h) * p.hd;
        if (h >= p.n_q + p.n_kv) {                       // value head: plain copy of two elements
            const int g = h - p.n_q - p.n_kv;
            __nv_bfloat16* dst = p.vc + ((static_cast<int64_t>(p.shared ? 0 : b) * p.n_kv + g) * p.cap + pos) * p.hd;
            dst[2 * pr] = __float2bfloat16_rn(src[2 * pr]);
            dst[2 * pr + 1] = __float2bfloat16_rn(src[2 * pr + 1]);
            continue;
        }
        // pair index inside its part: the first r/2 pairs belong to [0, r), the rest to [r, hd)
        const int hr = p.r / 2;
        int part0, m, pi;
        if (pr < hr) { part0 = 0; m = p.r; pi = pr; }
        else { part0 = p.r; m = p.hd - p.r; pi = pr - hr; }
        const int ia = part0 + pi, ib = part0 + pi + m / 2;
        // angle = pos * base^(-2i/m): the product and its reduction to one turn in fp64 (positions reach
        // tens of thousands of radians), sine and cosine of the reduced angle in fp32
        const double turns = static_cast<double>(pos) * p.inv_freq[part0 ? 1 : 0][pi] * 0.15915494309189533577;
        const float ang = static_cast<float>((turns - floor(turns)) * 6.28318530717958647692);
        float sn, cs;
        sincosf(ang, &sn, &cs);
        const float a = src[ia], bb = src[ib];
        const float ra = a * cs - bb * sn, rb = a * sn + bb * cs;
        if (h < p.n_q) {
            float* dst = p.q_out + (static_cast<int64_t>(b) * p.n_q + h) * p.hd;
            dst[ia] = ra * p.q_scale;
            dst[ib] = rb * p.q_scale;
        } else {
            const int g = h - p.n_q;
            const int64_t rowi = (static_cast<int64_t>(p.shared ? 0 : b) * p.n_kv + g) * p.cap + pos;
            if (part0 == 0 && p.k1f32 != nullptr) {
                float* dst = p.k1f32 + static_cast<int64_t>(b) * p.k1f32_sb + static_cast<int64_t>(g) * p.k1f32_sg;
                dst[pi] = ra;
                dst[pi + m / 2] = rb;
            } else if (part0 == 0) {
                __nv_bfloat16* dst = p.k1c + rowi * p.r;
                dst[pi] = __float2bfloat16_rn(ra);
                dst[pi + m / 2] = __float2bfloat16_rn(rb);
            } else {
                __nv_bfloat16* dst = p.k2c + rowi * (p.hd - p.r);
                dst[pi] = __float2bfloat16_rn(ra);
                dst[pi + m / 2] = __float2bfloat16_rn(rb);
            }
        }
    }
}

// The appended row of an FP8 predictor slice: a warp per (token, KV head) takes the fp32 row the projection left, its largest
// magnitude gives the row's scale s = max|k| / 448 (1 for an all-zero row), the row is stored as e4m3(k / s) (the storage rule of
// spark_attn_decode_fp8k; format and per-row scales are this library's choice, the paper's closing section only names quantisation).
struct K1QuantParams {
    const float* k1f32;
    int64_t sb, sg;
    unsigned char* k1c;      // [B or 1][n_kv][cap][r] E4M3 codes
    float* k1s;              // [B or 1][n_kv][cap]
    const int32_t* ctx_len;
    int B, n_kv, r, shared;
    int64_t cap;
};
__global__ void k1_quant_kernel(const K1QuantParams p) {
    dep_wait();
    dep_trigger();
    const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (w >= p.B * p.n_kv) return;
    const int b = w / p.n_kv, g = w - b * p.n_kv;
    int n = p.ctx_len[b];
    n = n < 1 ? 1 : (n > p.cap ? static_cast<int>(p.cap) : n);
    const float* src = p.k1f32 + static_cast<int64_t>(b) * p.sb + static_cast<int64_t>(g) * p.sg;
    float v[4], amax = 0.f;                       // r <= 128: four values per lane
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int i = lane * 4 + e;
        v[e] = i < p.r ? src[i] : 0.f;
        amax = fmaxf(amax, fabsf(v[e]));
    }
    amax = warp_max(amax);
    const float scale = amax > 0.f ? amax / 448.0f : 1.0f;
    const int64_t rowi = (static_cast<int64_t>(p.shared ? 0 : b) * p.n_kv + g) * p.cap + (n - 1);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int i = lane * 4 + e;
        if (i < p.r) p.k1c[rowi * p.r + i] = static_cast<unsigned char>(__nv_cvt_float_to_fp8(v[e] / scale, __NV_SATFINITE, __NV_E4M3));
    }
    if (lane == 0) p.k1s[rowi] = scale;
}

// QKV projection with the rotary encoding and the cache append in its epilogue: a warp computes the
// two output rows of a rotary pair together (rows i and i + m/2 of a head's part), so the pair can be
// turned and written to q / the caches straight from registers; value rows go to the cache as they
// are.  Saves the [q|k|v] round trip through memory and one kernel per layer.
struct QkvRopeParams {
    GemvParams g;
    RopeParams r;
};

template <int TB>
__global__ void __launch_bounds__(kThreads, 1) qkv_rope_kernel(const QkvRopeParams p) {
    extern __shared__ __align__(16) float xs[];       // [TB][n_in]
    __shared__ float rstd[16];
    const GemvParams& g = p.g;
    const RopeParams& rp = p.r;
    const int tid = threadIdx.x;
    const int hd = rp.hd, hp = hd / 2, hr = rp.r / 2;
    const int P = g.n_out / 2;                        // output pairs
    const int p0 = static_cast<int>(static_cast<int64_t>(blockIdx.x) * P / gridDim.x);
    const int p1 = static_cast<int>(static_cast<int64_t>(blockIdx.x + 1) * P / gridDim.x);
    auto rowmap = [&](int j) -> int {
        const int pp = p0 + (j >> 1), which = j & 1;
        const int head = pp / hp, q = pp - head * hp;
        if (head >= rp.n_q + rp.n_kv) return head * hd + 2 * q + which;
        if (q < hr) return head * hd + q + which * hr;
        return head * hd + rp.r + (q - hr) + which * ((hd - rp.r) / 2);
    };
    EarlyX ex = early_x_request(g, false);
    auto dependency = [&]() {
        if (tid == kThreads - 1) prefetch_l2_share(g.pf, blockIdx.x, gridDim.x);
        if (g.overlap) {
            dep_wait();
            dep_trigger();
            ex = early_x_request(g, true);
        }
    };
    auto fill_x = [&]() {
        if (blockIdx.x == gridDim.x - 1 && tid >= kThreads - 32 && tid - (kThreads - 32) < rp.B) {
            // the threshold quantile of each sequence's window, for the attention kernel that follows
            const int b = tid - (kThreads - 32);
            int n = rp.ctx_len[b];
            n = n < 1 ? 1 : (n > rp.cap ? static_cast<int>(rp.cap) : n);
            const int L = (rp.window > 0 && rp.window < n) ? rp.window : n;
            rp.zs[b] = rp.k_attn >= L ? 0.0 : -normcdfinv(static_cast<double>(rp.k_attn) / static_cast<double>(L));
        }
        stage_input<TB>(g, xs, rstd, ex);
    };
    rows_dot_mapped<__nv_bfloat16, TB, 2>(
        static_cast<const __nv_bfloat16*>(g.Wt), g.n_in, 2 * (p1 - p0), g.n_in / 8, xs, g.n_in, rowmap, dependency, fill_x,
        [&](int rg, int t, const float (&v)[2]) {
            if (t >= rp.B) return;
            const int pp = p0 + rg;
            const int head = pp / hp, q = pp - head * hp;
            int n = rp.ctx_len[t];
            n = n < 1 ? 1 : (n > rp.cap ? static_cast<int>(rp.cap) : n);
            const int pos = n - 1;
            if (head >= rp.n_q + rp.n_kv) {
                const int gk = head - rp.n_q - rp.n_kv;
                __nv_bfloat16* dst = rp.vc + ((static_cast<int64_t>(rp.shared ? 0 : t) * rp.n_kv + gk) * rp.cap + pos) * hd;
                dst[2 * q] = __float2bfloat16_rn(v[0]);
                dst[2 * q + 1] = __float2bfloat16_rn(v[1]);
                return;
            }
            const bool second = q >= hr;
            const int pi = second ? q - hr : q;
            const int m = second ? hd - rp.r : rp.r;
            const double turns = static_cast<double>(pos) * rp.inv_freq[second ? 1 : 0][pi] * 0.15915494309189533577;
            const float ang = static_cast<float>((turns - floor(turns)) * 6.28318530717958647692);
            float sn, cs;
            sincosf(ang, &sn, &cs);
            const float ra = v[0] * cs - v[1] * sn, rb = v[0] * sn + v[1] * cs;
            if (head < rp.n_q) {
                float* dst = rp.q_out + (static_cast<int64_t>(t) * rp.n_q + head) * hd + (second ? rp.r : 0);
                dst[pi] = ra * rp.q_scale;
                dst[pi + m / 2] = rb * rp.q_scale;
            } else {
                const int gk = head - rp.n_q;
                const int64_t rowi = (static_cast<int64_t>(rp.shared ? 0 : t) * rp.n_kv + gk) * rp.cap + pos;
                if (!second && rp.k1f32 != nullptr) {
                    float* dst = rp.k1f32 + static_cast<int64_t>(t) * rp.k1f32_sb + static_cast<int64_t>(gk) * rp.k1f32_sg;
                    dst[pi] = ra;
                    dst[pi + m / 2] = rb;
                } else {
                    __nv_bfloat16* dst = second ? rp.k2c + rowi * (hd - rp.r) : rp.k1c + rowi * rp.r;
                    dst[pi] = __float2bfloat16_rn(ra);
                    dst[pi + m / 2] = __float2bfloat16_rn(rb);
                }
            }
        });
}

template <int TB>
int qkv_rope_launch_one(spark_ctx* ctx, const QkvRopeParams& p, size_t smem, int grid, cudaStream_t stream) {
    static bool configured[64] = {};
    auto kern = qkv_rope_kernel<TB>;
    if (ctx->device >= 0 && ctx->device < 64 && !configured[ctx->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin - 1024) != cudaSuccess)
            return SPARK_ERR_CUDA;
        configured[ctx->device] = true;
    }
    QkvRopeParams q = p;
    q.g.overlap = ctx->overlap;
    void* args[] = {&q};
    return launch_kernel(ctx, reinterpret_cast<const void*>(kern), static_cast<unsigned>(grid), kThreads, smem, stream, false, args) == cudaSuccess
               ? SPARK_OK : SPARK_ERR_CUDA;
}

}  // namespace

namespace spark {

int gemv_launch(spark_ctx* ctx, const GemvArgs& a, cudaStream_t stream) {
    if (ctx == nullptr || a.x == nullptr || a.Wt == nullptr || a.y == nullptr) return SPARK_ERR_INVALID_ARG;
    if (a.B < 1 || a.B > 64 || a.n_in < 8 || a.n_out < 1) return SPARK_ERR_INVALID_ARG;
    if (a.wdtype != SPARK_F32 && a.wdtype != SPARK_BF16) return SPARK_ERR_UNSUPPORTED;
    if ((a.n_in & 7) != 0 || !aligned16(a.x) || !aligned16(a.Wt) || !aligned16(a.norm_w)) return SPARK_ERR_UNSUPPORTED;
    if (a.x_div != nullptr && (a.x_div_group < 4 || (a.x_div_group & 3) != 0 || a.n_in % a.x_div_group != 0)) return SPARK_ERR_UNSUPPORTED;
    if (a.zero_ptr != nullptr && (!aligned16(a.zero_ptr) || (a.zero_bytes & 15) != 0)) return SPARK_ERR_UNSUPPORTED;
    if (a.n_out > (1LL << 30) || a.n_in > (1 << 20)) return SPARK_ERR_UNSUPPORTED;
    if (!on_device(ctx)) return SPARK_ERR_INVALID_ARG;
    const size_t limit = static_cast<size_t>(ctx->max_smem_optin - 1024);
    if (static_cast<size_t>(a.n_in) * 4 > limit) return SPARK_ERR_UNSUPPORTED;
    if (a.B >= 5 && a.wdtype == SPARK_BF16) {      // five and more tokens: a real GEMM, on the tcgen05 tensor cores when the shape allows
        const int rc = gemm_tc_launch(ctx, a, stream);
        if (rc != SPARK_ERR_WORKSPACE) return rc;
    }
    // Tokens are processed in sub-batches whose inputs fit in shared memory together.
    int64_t done = 0;
    while (done < a.B) {
        int64_t nb = a.B - done;
        int tb = nb == 1 ? 1 : (nb <= 4 ? 4 : 16);
        while (static_cast<size_t>(tb) * a.n_in * 4 > limit) tb = tb == 16 ? 4 : 1;
        if (nb > tb) nb = tb;
        const int grid = a.n_out < ctx->num_sms ? static_cast<int>(a.n_out) : ctx->num_sms;
        const int64_t rows_per_block = (a.n_out + grid - 1) / grid;
        // rows a warp takes at once: as few as keeps all 16 warps of a block busy
        const int rw = rows_per_block <= kWarps ? 1 : (rows_per_block <= 2 * kWarps ? 2 : 4);
        GemvParams p;
        p.x = a.x + done * a.n_in; p.norm_w = a.norm_w; p.eps = a.rms_eps; p.Wt = a.Wt;
        p.B = static_cast<int>(nb); p.n_in = static_cast<int>(a.n_in); p.n_out = static_cast<int>(a.n_out);
        p.y_add = a.y_add ? a.y_add + done * a.n_out : nullptr;
        p.y = a.y + done * a.n_out;
        p.x_div = a.x_div ? a.x_div + done * (a.n_in / a.x_div_group) : nullptr;
        p.x_div_group = static_cast<int>(a.x_div ? a.x_div_group : 1);
        p.zero_ptr = done == 0 ? static_cast<uint4*>(a.zero_ptr) : nullptr;
        p.zero_n16 = done == 0 ? static_cast<int>(a.zero_bytes / 16) : 0;
        p.pf = PrefetchSpec{done == 0 ? a.pf_ptr : nullptr, a.pf_bytes};
        if (nb >= 5 && a.wdtype == SPARK_BF16 && (a.n_in & 31) == 0 && a.n_out >= 16) {      // tensor cores
            const int rc = nb <= 8 ? gemv_mma_launch<8>(ctx, p, grid, stream) : gemv_mma_launch<16>(ctx, p, grid, stream);
            if (rc == SPARK_OK) {
                done += nb;
                continue;
            }
            if (rc != SPARK_ERR_WORKSPACE) return rc;
        }
        const size_t smem = static_cast<size_t>(tb) * a.n_in * 4;
        const int st = a.wdtype == SPARK_BF16 ? gemv_dispatch<__nv_bfloat16>(ctx, p, tb, rw, smem, grid, stream)
                                              : gemv_dispatch<float>(ctx, p, tb, rw, smem, grid, stream);
        if (st != SPARK_OK) return st;
        done += nb;
    }
    return SPARK_OK;
}

}  // namespace spark

extern "C" int spark_dense_gemv(spark_ctx* ctx, const float* x, int64_t B, const void* Wt, int wdtype, int64_t n_in,
                                int64_t n_out, const float* y_add, float* y, void* stream) {
    GemvArgs a;
    a.x = x; a.norm_w = nullptr; a.rms_eps = 0.f; a.Wt = Wt; a.wdtype = wdtype;
    a.B = B; a.n_in = n_in; a.n_out = n_out; a.y_add = y_add; a.y = y;
    a.x_div = nullptr; a.x_div_group = 1; a.zero_ptr = nullptr; a.zero_bytes = 0;
    a.pf_ptr = nullptr; a.pf_bytes = 0;
    return gemv_launch(ctx, a, static_cast<cudaStream_t>(stream));
}

extern "C" int spark_layer_decode(spark_ctx* ctx, const spark_layer_weights* w, const spark_layer_cfg* cfg,
                                  const spark_kv_cache* cache, const int32_t* ctx_len, float* h, int64_t B,
                                  float* scratch, void* stream) {
    if (ctx == nullptr || w == nullptr || cfg == nullptr || cache == nullptr || ctx_len == nullptr || h == nullptr ||
        scratch == nullptr)
        return SPARK_ERR_INVALID_ARG;
    if (B < 1 || B > 64) return SPARK_ERR_INVALID_ARG;
    if (((cfg->n_q + 2 * cfg->n_kv) * cfg->hd + 2 * cfg->n_q * cfg->hd + cfg->d) % 2 != 0) return SPARK_ERR_UNSUPPORTED;
    if (w->norm1 == nullptr || w->norm2 == nullptr || w->Wqkv == nullptr || w->Wo == nullptr || w->K1t == nullptr ||
        w->K2t == nullptr || w->Vt == nullptr || cache->k1c == nullptr || cache->k2c == nullptr || cache->vc == nullptr)
        return SPARK_ERR_INVALID_ARG;
    if (cfg->hd < 16 || (cfg->hd & 1) || (cfg->r_attn & 1) || ((cfg->hd - cfg->r_attn) & 1) || cfg->n_q < 1 ||
        cfg->n_kv < 1 || cfg->d < 16)
        return SPARK_ERR_INVALID_ARG;
    if (!aligned16(scratch) || !aligned16(h)) return SPARK_ERR_UNSUPPORTED;
    const bool ffn_f8 = (cfg->flags & SPARK_FFN_FP8) != 0, k1_f8 = (cfg->flags & SPARK_K1C_FP8) != 0;
    if (ffn_f8 && (w->K1s == nullptr || w->K2s == nullptr || w->Vs == nullptr)) return SPARK_ERR_INVALID_ARG;
    if (k1_f8 && cache->k1s == nullptr) return SPARK_ERR_INVALID_ARG;
    if (ffn_f8 && B > 4) return SPARK_ERR_UNSUPPORTED;          // the chunk kernels take bf16 weights
    if (k1_f8 && (cfg->flags & SPARK_SHARED_CACHE) && B >= 16) return SPARK_ERR_UNSUPPORTED;      // the chunk attention takes a bf16 slice
    if (!on_device(ctx)) return SPARK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (B == 1 && ctx->fused) {           // one token: the whole layer as one persistent kernel when it serves the shape
        const int rc1 = layer1_launch(ctx, w, cfg, cache, 1, ctx_len, h, scratch, st);
        if (rc1 != SPARK_ERR_WORKSPACE) return rc1;
    }
    const int64_t nqkv = (cfg->n_q + 2 * cfg->n_kv) * cfg->hd, nqo = cfg->n_q * cfg->hd;
    const bool pf_on = ctx->l2_prefetch && B <= 4;      // the latency-bound case
    float* qkv = scratch;                 // [B][nqkv]
    float* qr = qkv + B * nqkv;           // [B][n_q][hd]  position-encoded, scaled queries
    float* ao = qr + B * nqo;             // [B][n_q][hd]  attention output
    float* h2 = ao + B * nqo;             // [B][d]        h + Wo . attention
    double* zs = reinterpret_cast<double*>(h2 + B * cfg->d);   // [B] threshold quantiles (8-byte aligned: see below)
    float* lsum = reinterpret_cast<float*>(zs + B);            // [B][n_q] sums of attention weights

    // 1 + 2. a = RMSNorm(h; norm1); [q|k|v] = Wqkv a; rotary encoding per half, query scale, cache
    //        append -- one kernel when the batch's inputs fit in shared memory together, else two.
    RopeParams rp;
    rp.qkv = qkv; rp.q_out = qr;
    rp.k1c = static_cast<__nv_bfloat16*>(cache->k1c); rp.k2c = static_cast<__nv_bfloat16*>(cache->k2c);
    rp.vc = static_cast<__nv_bfloat16*>(cache->vc);
    rp.ctx_len = ctx_len; rp.B = static_cast<int>(B); rp.n_q = static_cast<int>(cfg->n_q); rp.n_kv = static_cast<int>(cfg->n_kv);
    rp.hd = static_cast<int>(cfg->hd); rp.r = static_cast<int>(cfg->r_attn); rp.cap = cfg->cap;
    rp.shared = (cfg->flags & SPARK_SHARED_CACHE) ? 1 : 0;
    rp.base = cfg->rope_base; rp.q_scale = 1.0f / std::sqrt(static_cast<float>(cfg->hd));
    if (cfg->r_attn > 128 || cfg->hd - cfg->r_attn > 128) return SPARK_ERR_UNSUPPORTED;
    for (int part = 0; part < 2; ++part) {
        const int64_t m = part == 0 ? cfg->r_attn : cfg->hd - cfg->r_attn;
        for (int64_t i = 0; i < m / 2; ++i)
            rp.inv_freq[part][i] = std::pow(static_cast<double>(cfg->rope_base), -2.0 * static_cast<double>(i) / static_cast<double>(m));
    }
    rp.zs = zs; rp.window = static_cast<int>(cfg->window > 0x7fffffff ? 0x7fffffff : cfg->window);
    rp.k1f32 = nullptr; rp.k1f32_sb = 0; rp.k1f32_sg = 0;
    rp.k_attn = static_cast<int>(cfg->k_attn > 0x7fffffff ? 0x7fffffff : cfg->k_attn);
    int rc;
    const int tbq = B == 1 ? 1 : (B <= 4 ? 4 : 16);
    const size_t smem_q = static_cast<size_t>(tbq) * cfg->d * 4;
    // up to four tokens: projection, rotary encoding and cache append in one kernel; more: the tensor-core GEMV,
    // then a small kernel for the rotary encoding and the append
    if (B <= 4 && (cfg->d & 7) == 0 && smem_q <= static_cast<size_t>(ctx->max_smem_optin - 1024) && nqkv / 2 >= 1 &&
        aligned16(w->Wqkv) && aligned16(w->norm1)) {
        if (k1_f8) { rp.k1f32 = qkv; rp.k1f32_sb = cfg->n_kv * cfg->r_attn; rp.k1f32_sg = cfg->r_attn; }      // the projection buffer is free here
        QkvRopeParams qp;
        qp.g.x = h; qp.g.norm_w = w->norm1; qp.g.eps = cfg->rms_eps; qp.g.Wt = w->Wqkv;
        qp.g.B = static_cast<int>(B); qp.g.n_in = static_cast<int>(cfg->d); qp.g.n_out = static_cast<int>(nqkv);
        qp.g.y_add = nullptr; qp.g.y = nullptr; qp.g.x_div = nullptr; qp.g.x_div_group = 1;
        qp.g.zero_ptr = nullptr; qp.g.zero_n16 = 0;
        qp.g.pf = PrefetchSpec{pf_on ? w->Wo : nullptr, static_cast<unsigned long long>(cfg->d) * nqo * 2ull};
        qp.r = rp;
        const int64_t pairs = nqkv / 2;
        const int gridq = pairs < ctx->num_sms ? static_cast<int>(pairs) : ctx->num_sms;
        rc = tbq == 1 ? qkv_rope_launch_one<1>(ctx, qp, smem_q, gridq, st)
                      : (tbq == 4 ? qkv_rope_launch_one<4>(ctx, qp, smem_q, gridq, st)
                                  : qkv_rope_launch_one<16>(ctx, qp, smem_q, gridq, st));
        if (rc != SPARK_OK) return rc;
    } else {
        GemvArgs g1;
        g1.x = h; g1.norm_w = w->norm1; g1.rms_eps = cfg->rms_eps; g1.Wt = w->Wqkv; g1.wdtype = SPARK_BF16;
        g1.B = B; g1.n_in = cfg->d; g1.n_out = nqkv; g1.y_add = nullptr; g1.y = qkv;
        g1.x_div = nullptr; g1.x_div_group = 1; g1.zero_ptr = nullptr; g1.zero_bytes = 0;
        g1.pf_ptr = nullptr; g1.pf_bytes = 0;
        rc = gemv_launch(ctx, g1, st);
        if (rc != SPARK_OK) return rc;
        if (k1_f8) { rp.k1f32 = qkv + cfg->n_q * cfg->hd; rp.k1f32_sb = nqkv; rp.k1f32_sg = cfg->hd; }      // rotated in place
        const int64_t total = B * (cfg->n_q + 2 * cfg->n_kv) * (cfg->hd / 2);
        const int blocks = static_cast<int>((total + 255) / 256);
        void* rargs[] = {&rp};
        if (launch_kernel(ctx, reinterpret_cast<const void*>(rope_append_kernel), static_cast<unsigned>(blocks), 256, 0, st, false, rargs) != cudaSuccess)
            return SPARK_ERR_CUDA;
    }

    // 2b. an FP8 predictor slice: the appended rows are quantised (one warp per token and KV head)
    if (k1_f8) {
        K1QuantParams kq;
        kq.k1f32 = rp.k1f32; kq.sb = rp.k1f32_sb; kq.sg = rp.k1f32_sg;
        kq.k1c = static_cast<unsigned char*>(cache->k1c); kq.k1s = cache->k1s; kq.ctx_len = ctx_len;
        kq.B = static_cast<int>(B); kq.n_kv = static_cast<int>(cfg->n_kv); kq.r = static_cast<int>(cfg->r_attn);
        kq.shared = rp.shared; kq.cap = cfg->cap;
        const unsigned warps = static_cast<unsigned>(B * cfg->n_kv);
        void* kargs[] = {&kq};
        if (launch_kernel(ctx, reinterpret_cast<const void*>(k1_quant_kernel), (warps + 7) / 8, 256, 0, st, false, kargs) != cudaSuccess)
            return SPARK_ERR_CUDA;
    }

    // 3. Spark attention over the cache (the new token included)
    rc = attn_launch(ctx, qr, cache->k1c, cache->k2c, cache->vc, SPARK_BF16, B, cfg->n_q, cfg->n_kv, cfg->hd, cfg->r_attn,
                     cfg->cap, ctx_len, zs, cfg->window, cfg->k_attn, cfg->flags & (SPARK_DENSE_LOADS | SPARK_SHARED_CACHE | SPARK_CHECK_FINITE), ao, lsum, nullptr, nullptr,
                     nullptr, 0, k1_f8 ? cache->k1s : nullptr, st,
                     PrefetchSpec{pf_on ? w->K1t : nullptr, static_cast<unsigned long long>(cfg->d_ff) * cfg->r_ff * (ffn_f8 ? 1ull : 2ull)});
    if (rc != SPARK_OK) return rc;

    // 4. h2 = h + Wo . (attention sums / sums of weights); the projection kernel also clears the
    //    attention kernel's score-sum cells for the next call
    GemvArgs g2;
    g2.x = ao; g2.norm_w = nullptr; g2.rms_eps = 0.f; g2.Wt = w->Wo; g2.wdtype = SPARK_BF16;
    g2.B = B; g2.n_in = nqo; g2.n_out = cfg->d; g2.y_add = h; g2.y = h2;
    g2.x_div = lsum; g2.x_div_group = cfg->hd;
    g2.zero_ptr = ctx->scratch; g2.zero_bytes = static_cast<size_t>(B * cfg->n_q) * kAttnWays * sizeof(SumCell);
    g2.pf_ptr = nullptr; g2.pf_bytes = 0;
    rc = gemv_launch(ctx, g2, st);
    if (rc != SPARK_OK) return rc;

    // 5. h = h2 + SparkFFN(RMSNorm(h2; norm2))
    FfnArgs f;
    f.x = h2; f.norm_w = w->norm2; f.rms_eps = cfg->rms_eps;
    f.K1t = w->K1t; f.K2t = w->K2t; f.Vt = w->Vt; f.wdtype = ffn_f8 ? SPARK_FP8_E4M3 : SPARK_BF16;
    f.K1s = ffn_f8 ? w->K1s : nullptr; f.K2s = ffn_f8 ? w->K2s : nullptr; f.Vs = ffn_f8 ? w->Vs : nullptr;
    f.B = B; f.d = cfg->d; f.d_ff = cfg->d_ff; f.r = cfg->r_ff; f.k = cfg->k_ff; f.flags = cfg->flags & (SPARK_GELU_ERF | SPARK_DENSE_LOADS | SPARK_CHECK_FINITE);
    f.y_init = h2; f.y = h; f.theta = nullptr; f.count = nullptr; f.idx = nullptr;
    f.pf = PrefetchSpec{pf_on ? ctx->next_wqkv : nullptr, static_cast<unsigned long long>(nqkv) * cfg->d * 2ull};
    return ffn_launch(ctx, f, st);
}

// A stack of layers for the same tokens: one launch of the fused kernel per 64 layers when it serves the call (one token,
// equal configurations but for the window), otherwise one spark_layer_decode per layer.
extern "C" int spark_stack_decode(spark_ctx* ctx, const spark_layer_weights* w, const spark_layer_cfg* cfg, const spark_kv_cache* cache,
                                  int64_t n_layers, const int32_t* ctx_len, float* h, int64_t B, float* scratch, void* stream) {
    if (ctx == nullptr || w == nullptr || cfg == nullptr || cache == nullptr || ctx_len == nullptr || h == nullptr || scratch == nullptr)
        return SPARK_ERR_INVALID_ARG;
    if (n_layers < 1 || B < 1 || B > 64) return SPARK_ERR_INVALID_ARG;
    if (!aligned16(scratch) || !aligned16(h)) return SPARK_ERR_UNSUPPORTED;
    if (!on_device(ctx)) return SPARK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int64_t done = 0;
    while (done < n_layers) {
        const int64_t n = n_layers - done < 64 ? n_layers - done : 64;
        int rc = SPARK_ERR_WORKSPACE;
        if (B == 1 && ctx->fused) rc = layer1_launch(ctx, w + done, cfg + done, cache + done, static_cast<int>(n), ctx_len, h, scratch, st);
        if (rc == SPARK_ERR_WORKSPACE) {
            for (int64_t l = 0; l < n; ++l) {
                // the FFN kernel of layer l asks L2 for the QKV matrix of layer l + 1 while its blocks exchange their sums
                ctx->next_wqkv = done + l + 1 < n_layers ? w[done + l + 1].Wqkv : nullptr;
                rc = spark_layer_decode(ctx, w + done + l, cfg + done + l, cache + done + l, ctx_len, h, B, scratch, stream);
                ctx->next_wqkv = nullptr;
                if (rc != SPARK_OK) return rc;
            }
        } else if (rc != SPARK_OK) {
            return rc;
        }
        done += n;
    }
    return SPARK_OK;
}

// ---------------------------------------------------------------------------------------------
// spark_prefill: a prompt through a stack of layers chunk by chunk (Section 4.3 measures prefill in chunks of 64 tokens).
// ---------------------------------------------------------------------------------------------
namespace {
__global__ void chunk_lengths_kernel(int32_t* len, int n, int first) {      // len[b] = first + b: token b of the chunk sees first + b tokens
    dep_wait();
    dep_trigger();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) len[i] = first + i;
}
}  // namespace

extern "C" int spark_prefill(spark_ctx* ctx, const spark_layer_weights* w, const spark_layer_cfg* cfg, const spark_kv_cache* cache,
                             int64_t n_layers, float* h, int64_t n_tokens, int64_t start, int64_t chunk, int32_t* len_buf, float* scratch,
                             void* stream) {
    if (ctx == nullptr || w == nullptr || cfg == nullptr || cache == nullptr || h == nullptr || len_buf == nullptr || scratch == nullptr)
        return SPARK_ERR_INVALID_ARG;
    if (n_layers < 1 || n_tokens < 1 || start < 0 || chunk < 1 || chunk > 64) return SPARK_ERR_INVALID_ARG;
    for (int64_t l = 0; l < n_layers; ++l) {
        if (!(cfg[l].flags & SPARK_SHARED_CACHE)) return SPARK_ERR_INVALID_ARG;      // the chunk's tokens share one cache
        if (start + n_tokens > cfg[l].cap || cfg[l].d != cfg[0].d) return SPARK_ERR_INVALID_ARG;
    }
    if (!on_device(ctx)) return SPARK_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int64_t c0 = 0; c0 < n_tokens; c0 += chunk) {
        const int64_t T = n_tokens - c0 < chunk ? n_tokens - c0 : chunk;
        int n = static_cast<int>(T), first = static_cast<int>(start + c0 + 1);
        void* args[] = {&len_buf, &n, &first};
        if (launch_kernel(ctx, reinterpret_cast<const void*>(chunk_lengths_kernel), 1u, 64u, 0, st, false, args) != cudaSuccess) return SPARK_ERR_CUDA;
        ctx->len_hint = start + c0 + T;          // the lengths are known here on the host: the chunk attention picks its second stage by them
        for (int64_t l = 0; l < n_layers; ++l) {
            const int rc = spark_layer_decode(ctx, w + l, cfg + l, cache + l, len_buf, h + c0 * cfg[0].d, T, scratch, stream);
            if (rc != SPARK_OK) {
                ctx->len_hint = 0;
                return rc;
            }
        }
    }
    ctx->len_hint = 0;
    return SPARK_OK;
}

// Several chunks in flight: chunk c runs on stream c % n with its own context (workspaces must not be shared between kernels
// that run at the same time); layer l of chunk c waits for layer l of chunk c - 1, which has filled that layer's cache up to
// the rows chunk c reads -- a wavefront over (chunk, layer).  The kernels of a chunk layer are latency-bound (a dozen launches
// of 5-10 us, each with an idle boundary): the other streams' kernels fill those gaps.
extern "C" int spark_prefill_pipelined(spark_ctx* const* ctxs, float* const* scratches, void* const* streams, int64_t n_inflight,
                                       const spark_layer_weights* w, const spark_layer_cfg* cfg, const spark_kv_cache* cache,
                                       int64_t n_layers, float* h, int64_t n_tokens, int64_t start, int64_t chunk, int32_t* len_buf) {
    constexpr int kMaxInflight = 8;
    if (ctxs == nullptr || scratches == nullptr || streams == nullptr || n_inflight < 2 || n_inflight > kMaxInflight || w == nullptr ||
        cfg == nullptr || cache == nullptr || h == nullptr || len_buf == nullptr)
        return SPARK_ERR_INVALID_ARG;
    const int n = static_cast<int>(n_inflight);
    for (int i = 0; i < n; ++i) {
        if (ctxs[i] == nullptr || scratches[i] == nullptr) return SPARK_ERR_INVALID_ARG;
        for (int j = 0; j < i; ++j)
            if (ctxs[i] == ctxs[j] || scratches[i] == scratches[j] || streams[i] == streams[j]) return SPARK_ERR_INVALID_ARG;
        if (ctxs[i]->device != ctxs[0]->device) return SPARK_ERR_INVALID_ARG;
    }
    if (n_layers < 1 || n_layers > 4096 || n_tokens < 1 || start < 0 || chunk < 1 || chunk > 64) return SPARK_ERR_INVALID_ARG;
    for (int64_t l = 0; l < n_layers; ++l) {
        if (!(cfg[l].flags & SPARK_SHARED_CACHE)) return SPARK_ERR_INVALID_ARG;
        if (start + n_tokens > cfg[l].cap || cfg[l].d != cfg[0].d) return SPARK_ERR_INVALID_ARG;
    }
    if (!on_device(ctxs[0])) return SPARK_ERR_INVALID_ARG;
    cudaStream_t st[kMaxInflight];
    for (int i = 0; i < n; ++i) st[i] = static_cast<cudaStream_t>(streams[i]);
    // done[s][l]: layer l of the newest chunk on stream s has finished; fork and join around the call
    const size_t n_ev = static_cast<size_t>(n) * static_cast<size_t>(n_layers) + 1 + static_cast<size_t>(n);
    cudaEvent_t* ev = new (std::nothrow) cudaEvent_t[n_ev];
    if (ev == nullptr) return SPARK_ERR_CUDA;
    size_t made = 0;
    int rc = SPARK_OK;
    for (; made < n_ev; ++made)
        if (cudaEventCreateWithFlags(&ev[made], cudaEventDisableTiming) != cudaSuccess) { rc = SPARK_ERR_CUDA; break; }
    auto done = [&](int s, int64_t l) -> cudaEvent_t& { return ev[1 + n + static_cast<size_t>(s) * n_layers + l]; };
    if (rc == SPARK_OK) {
        // what is queued on the caller's stream (the embeddings) comes before the other streams' first kernels
        if (cudaEventRecord(ev[0], st[0]) != cudaSuccess) rc = SPARK_ERR_CUDA;
        for (int i = 1; i < n && rc == SPARK_OK; ++i)
            if (cudaStreamWaitEvent(st[i], ev[0], 0) != cudaSuccess) rc = SPARK_ERR_CUDA;
    }
    int64_t c = 0;
    for (int64_t c0 = 0; c0 < n_tokens && rc == SPARK_OK; c0 += chunk, ++c) {
        const int s = static_cast<int>(c % n), prev = static_cast<int>((c + n - 1) % n);
        const int64_t T = n_tokens - c0 < chunk ? n_tokens - c0 : chunk;
        int32_t* lens = len_buf + s * chunk;
        int nt = static_cast<int>(T), first = static_cast<int>(start + c0 + 1);
        void* args[] = {&lens, &nt, &first};
        if (launch_kernel(ctxs[s], reinterpret_cast<const void*>(chunk_lengths_kernel), 1u, 64u, 0, st[s], false, args) != cudaSuccess) {
            rc = SPARK_ERR_CUDA;
            break;
        }
        ctxs[s]->len_hint = start + c0 + T;
        for (int64_t l = 0; l < n_layers && rc == SPARK_OK; ++l) {
            if (c > 0 && cudaStreamWaitEvent(st[s], done(prev, l), 0) != cudaSuccess) { rc = SPARK_ERR_CUDA; break; }
            rc = spark_layer_decode(ctxs[s], w + l, cfg + l, cache + l, lens, h + c0 * cfg[0].d, T, scratches[s], st[s]);
            if (rc == SPARK_OK && cudaEventRecord(done(s, l), st[s]) != cudaSuccess) rc = SPARK_ERR_CUDA;
        }
        ctxs[s]->len_hint = 0;
    }
    if (rc == SPARK_OK) {          // the caller's stream continues after all of them
        for (int i = 1; i < n && rc == SPARK_OK; ++i)
            if (cudaEventRecord(ev[i], st[i]) != cudaSuccess || cudaStreamWaitEvent(st[0], ev[i], 0) != cudaSuccess) rc = SPARK_ERR_CUDA;
    }
    for (size_t i = 0; i < made; ++i) cudaEventDestroy(ev[i]);      // released once the work that uses them has completed
    delete[] ev;
    return rc;
}
