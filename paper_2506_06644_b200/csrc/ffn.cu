// spark_ffn_decode: Spark FFN (Section 2.1, Eq. 2) for one to a few tokens, one persistent
// cooperative kernel, one thread block per SM.
//
//   phase A  every block streams its contiguous share of K1t once (coalesced 16-byte loads, fp32
//            accumulate) and forms the predictor scores s = K1^T x[:r] of its neurons;
//   stats    per-block (count, mean, M2) per token -> workspace; ONE grid-wide barrier (the
//            threshold of Eq. 11 needs every score); each block merges all partials itself;
//   phase C  theta, active masks and the union of the tokens' active sets over the block's own
//            neurons (ballot + prefix-sum compaction in shared memory);
//   phase D  only the union rows of K2t and Vt are read: a warp per row for t_i = K2[:,i].x[r:],
//            u_i = GELU(s_i - theta) t_i, then a thread per 8 output columns accumulates
//            sum_i u_i V[:,i] in registers and adds it to y with vector reductions.
// Individual masks gate the arithmetic, the union gates the loads (Appendix B).
#include <atomic>
#include <mutex>

#include "ffn_params.h"
#include "kernels.h"
#include "rowdot.cuh"

using namespace spark;

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / kWarp;
constexpr int kRows = 4;          // rows a warp works on at once in phase A

template <typename WT, int TB>
__global__ void __launch_bounds__(kThreads, 1) ffn_kernel(const FfnParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* xs = reinterpret_cast<float*>(smem_raw);                 // [TB][xw]
    float* s_loc = xs + static_cast<size_t>(TB) * p.xw;             // [TB][rpc]
    float* u_loc = s_loc + static_cast<size_t>(TB) * p.rpc;         // [TB][rpc]
    int* ulist = reinterpret_cast<int*>(u_loc + static_cast<size_t>(TB) * p.rpc);   // [rpc]
    unsigned* amask = reinterpret_cast<unsigned*>(ulist + p.rpc);   // [rpc]
    __shared__ float rstd[kFfnMaxTB];
    __shared__ float theta_s[kFfnMaxTB];
    __shared__ int wcnt[kWarps];
    __shared__ unsigned tok_any;
    __shared__ unsigned s_epoch;
    __shared__ int s_fail;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int grid = gridDim.x, cta = blockIdx.x;
    const int row0 = static_cast<int>(static_cast<int64_t>(cta) * p.d_ff / grid);
    const int row1 = static_cast<int>(static_cast<int64_t>(cta + 1) * p.d_ff / grid);
    const int nloc = row1 - row0;
    const int d = p.d, r = p.r, d2 = d - r, rpc = p.rpc, xw = p.xw;
    const WT* K1t = static_cast<const WT*>(p.K1t);
    const WT* K2t = static_cast<const WT*>(p.K2t);
    const WT* Vt = static_cast<const WT*>(p.Vt);
    dep_wait();        // these kernels read the batch's inputs first: nothing to do ahead of the dependency
    dep_trigger();
    if (tid == 0) {
        s_epoch = ld_acquire_u32(&p.hdr->epoch);      // consumed after phase A
        s_fail = 0;
    }
    if (cta == 0) {
        // clear the cells the launch after next will use (last used two launches ago)
        const unsigned e = ld_acquire_u32(&p.hdr->epoch);
        SumCell* c = &p.hdr->ffn_cells[(e + 2u) & 3u][0][0][0];
        for (int i = tid; i < 4 * 16 * kCellWays; i += kThreads) { c[i].s1 = 0.0; c[i].s2 = 0.0; c[i].count = 0u; }
    }
    p.trace.mark(0);

    for (int g0 = 0, grp = 0; g0 < p.B; g0 += TB, ++grp) {
        const int tbv = min(TB, p.B - g0);
        const float* xg = p.x + static_cast<int64_t>(g0) * d;
        float* yg = p.y + static_cast<int64_t>(g0) * d;

        auto stage = [&](int col0, int width) {     // xs[t][0:width] = x[t][col0:col0+width] (normalised)
            const int w4 = width / 4;
            for (int i = tid; i < TB * w4; i += kThreads) {
                const int t = i / w4, c = i - t * w4;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (t < tbv) {
                    v = reinterpret_cast<const float4*>(xg + static_cast<int64_t>(t) * d + col0)[c];
                    if (p.norm_w != nullptr) {
                        const float4 w = reinterpret_cast<const float4*>(p.norm_w + col0)[c];
                        const float sc = rstd[t];
                        v.x *= sc * w.x; v.y *= sc * w.y; v.z *= sc * w.z; v.w *= sc * w.w;
                    }
                }
                reinterpret_cast<float4*>(xs + static_cast<size_t>(t) * xw)[c] = v;
            }
        };
        // Runs once, after the first K1t loads are in flight: optional RMSNorm scale, y
        // initialisation, x[:r] into shared memory.
        auto prologue = [&]() {
            if (p.norm_w != nullptr) {
                for (int t = warp; t < TB; t += kWarps) {
                    float ss = 0.f;
                    if (t < tbv) {
                        const float4* xr = reinterpret_cast<const float4*>(xg + static_cast<int64_t>(t) * d);
                        for (int i = lane; i < d / 4; i += 32) {
                            const float4 v = xr[i];
                            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
                        }
                        ss = warp_sum(ss);
                    }
                    if (lane == 0) rstd[t] = rsqrtf(ss / static_cast<float>(d) + p.eps);
                }
                __syncthreads();
            }
            stage(0, r);
            {
                const int64_t total4 = static_cast<int64_t>(tbv) * d / 4;
                const float4* yi = p.y_init ? reinterpret_cast<const float4*>(p.y_init + static_cast<int64_t>(g0) * d) : nullptr;
                float4* yo = reinterpret_cast<float4*>(yg);
                for (int64_t i = static_cast<int64_t>(cta) * kThreads + tid; i < total4; i += static_cast<int64_t>(grid) * kThreads)
                    yo[i] = yi ? yi[i] : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            if (cta == 0 && p.count != nullptr && tid < tbv) p.count[g0 + tid] = 0;
            if (tid == 0) tok_any = 0u;
            __syncthreads();
            p.trace.mark(1);
        };

        // ---- phase A: predictor scores of this block's neurons ----------------------------------
        rows_dot<WT, TB, kRows>(K1t, r, row0, nloc, r / 8, xs, xw, [] {}, prologue, [&](int j, int t, float v) {
            s_loc[static_cast<size_t>(t) * rpc + j] = v;
        });
        __syncthreads();
        p.trace.mark(2);

        // ---- sums of the scores and of their squares (fp64), one warp per token, added to the token's
        //      grid-wide cell; the arrival follows them with release semantics --------------------------
        SumCell* cells = &p.hdr->ffn_cells[s_epoch & 3u][grp & 3][0][0];   // [token][way]
        for (int t = warp; t < tbv; t += kWarps) {
            const float* sr = s_loc + static_cast<size_t>(t) * rpc;
            double s1 = 0.0, s2 = 0.0;
            for (int j = lane; j < nloc; j += 32) {
                const double v = static_cast<double>(sr[j]);
                s1 += v;
                s2 = fma(v, v, s2);
            }
            s1 = warp_sum_f64(s1);
            s2 = warp_sum_f64(s2);
            if (lane == 0) cells_add(cells + t * kCellWays, cta, s1, s2);
        }
        p.trace.mark(3);
        __syncthreads();
        stage(r, d2);                                   // x[r:] replaces x[:r] while the cells fill
        // theta per token (Eq. 11, Bessel-corrected) once every block has added its sums
        for (int t = warp; t < tbv; t += kWarps) {
            double sa, sb;
            const bool ok = cells_wait(cells + t * kCellWays, static_cast<unsigned>(grid), sa, sb, p.hdr);
            if (lane == 0) {
                float th = -INFINITY;
                if (!ok) s_fail = 1;
                if (!p.identity) {
                    const double mean = sa * p.inv_n;
                    const float var = static_cast<float>((sb - sa * mean) * p.inv_nm1);
                    th = static_cast<float>(mean) + sqrtf(fmaxf(var, 0.f)) * static_cast<float>(p.z);
                }
                theta_s[t] = th;
                if (cta == 0 && p.theta != nullptr) p.theta[g0 + t] = th;
            }
        }
        __syncthreads();
        if (s_fail) return;
        p.trace.mark(4);

        p.trace.mark(5);
        // ---- phase C: masks and the ordered union list of this block's neurons --------------------
        int nU = 0;
        for (int j0 = 0; j0 < nloc; j0 += kThreads) {
            const int j = j0 + tid;
            unsigned m = 0u;
            if (j < nloc) {
#pragma unroll
                for (int t = 0; t < TB; ++t)
                    if (t < tbv && s_loc[static_cast<size_t>(t) * rpc + j] > theta_s[t]) m |= 1u << t;
                amask[j] = m;
            }
            const bool in = j < nloc && (m != 0u || p.dense);
            const unsigned bal = __ballot_sync(kFull, in);
            if (lane == 0) wcnt[warp] = __popc(bal);
            if (m != 0u) atomicOr(&tok_any, m);
            __syncthreads();
            int before = 0, all = 0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                if (w < warp) before += wcnt[w];
                all += wcnt[w];
            }
            if (in) ulist[nU + before + __popc(bal & ((1u << lane) - 1u))] = j;
            nU += all;
            __syncthreads();
        }

        // ---- optional outputs: per-token count and index list --------------------------------------
        if (p.count != nullptr) {
            for (int t = warp; t < tbv; t += kWarps) {
                int c = 0;
                for (int j = lane; j < nloc; j += 32) c += (amask[j] >> t) & 1u;
                c = warp_sum_int(c);
                int base = 0;
                if (lane == 0 && c > 0) base = atomicAdd(&p.count[g0 + t], c);
                base = __shfl_sync(kFull, base, 0);
                if (p.idx != nullptr && c > 0) {
                    int32_t* out = p.idx + static_cast<int64_t>(g0 + t) * p.d_ff;
                    for (int j0 = 0; j0 < nloc; j0 += 32) {
                        const int j = j0 + lane;
                        const bool a = j < nloc && ((amask[j] >> t) & 1u);
                        const unsigned bal = __ballot_sync(kFull, a);
                        if (a) out[base + __popc(bal & ((1u << lane) - 1u))] = row0 + j;
                        base += __popc(bal);
                    }
                }
            }
        }

        p.trace.mark(6);
        // ---- phase D: only the union rows of K2t and Vt are read -------------------------------------
        constexpr int RB = 8;                            // union rows a thread holds in flight
        const int ncd = d / 8;
        // The first batch of V rows is requested before the K2 dot products so that both gathers
        // share one trip to HBM; a thread owns 8 output columns.
        constexpr bool PRE = TB <= 4;                    // larger token groups need the registers
        Row8<WT> vpre[PRE ? RB : 1];
#pragma unroll
        for (int j = 0; j < (PRE ? RB : 1); ++j) {
            if (PRE && j < nU && tid < ncd) vpre[j].load_pinned(Vt + static_cast<int64_t>(row0 + ulist[j]) * d, tid);
            else vpre[j].zero();
        }
        p.trace.mark(9);
        // ---- D1: t_i = K2[:,i] . x[r:] for union rows (a warp takes one or two rows at a time),
        //          u = GELU(s - theta) * t
        {
            constexpr int KU = sizeof(WT) == 4 ? 4 : 8;  // chunks per lane per batch
            const int nc2 = d2 / 8;
            const unsigned all_tok = (1u << tbv) - 1u;
            constexpr int RR = TB >= 8 ? 1 : 2;          // rows a warp takes at a time
            for (int ui0 = warp * RR; ui0 < nU; ui0 += kWarps * RR) {
                int jj[RR];
                unsigned mask[RR], cm[RR];
                const WT* krow[RR];
#pragma unroll
                for (int rr = 0; rr < RR; ++rr) {
                    const bool ok = ui0 + rr < nU;
                    jj[rr] = ulist[ok ? ui0 + rr : ui0];
                    mask[rr] = ok ? amask[jj[rr]] : 0u;
                    cm[rr] = ok ? (p.dense ? all_tok : mask[rr]) : 0u;
                    krow[rr] = K2t + static_cast<int64_t>(row0 + jj[rr]) * d2;
                }
                float acc[RR][TB];
#pragma unroll
                for (int rr = 0; rr < RR; ++rr)
#pragma unroll
                    for (int t = 0; t < TB; ++t) acc[rr][t] = 0.f;
                for (int c0 = 0; c0 < nc2; c0 += 32 * KU) {
                    Row8<WT> w[RR][KU];
#pragma unroll
                    for (int rr = 0; rr < RR; ++rr)
#pragma unroll
                        for (int u = 0; u < KU; ++u) {
                            const int c = c0 + u * 32 + lane;
                            if (c < nc2 && cm[rr] != 0u) w[rr][u].load(krow[rr], c);
                            else w[rr][u].zero();
                        }
                    p.trace.mark(10);
#pragma unroll
                    for (int u = 0; u < KU; ++u) {
                        const int c = c0 + u * 32 + lane;
                        const int cs = c < nc2 ? c : 0;
#pragma unroll
                        for (int rr = 0; rr < RR; ++rr) {
                            float wf[8];
                            w[rr][u].unpack(wf);
#pragma unroll
                            for (int t = 0; t < TB; ++t) {
                                if ((cm[rr] >> t) & 1u) {
                                    const float4* xr = reinterpret_cast<const float4*>(xs + static_cast<size_t>(t) * xw) + 2 * cs;
                                    acc[rr][t] = dot8(wf, xr[0], xr[1], acc[rr][t]);
                                }
                            }
                        }
                    }
                }
                p.trace.mark(11);
#pragma unroll
                for (int rr = 0; rr < RR; ++rr) {
                    if (ui0 + rr >= nU) break;
#pragma unroll
                    for (int t = 0; t < TB; ++t) {
                        float u = 0.f;
                        if ((cm[rr] >> t) & 1u) {
                            const float tv = warp_sum(acc[rr][t]);
                            if ((mask[rr] >> t) & 1u) {
                                const float a = s_loc[static_cast<size_t>(t) * rpc + jj[rr]] - (p.identity ? 0.f : theta_s[t]);
                                u = (p.erf_form ? gelu_erf(a) : gelu_tanh(a)) * tv;
                            }
                        }
                        if (lane == 0) u_loc[static_cast<size_t>(t) * rpc + ui0 + rr] = u;
                    }
                }
            }
        }
        p.trace.mark(12);
        __syncthreads();
        p.trace.mark(7);

        // ---- D2: y += sum_i u_i V[:,i]; per-thread register accumulators, vector reductions to y -----
        {
            constexpr int TP = TB < 8 ? TB : 8;          // tokens accumulated in registers at once
            const unsigned anyt = tok_any;
            for (int cb = 0; cb * kThreads < ncd; ++cb) {
                const int cc = cb * kThreads + tid;
#pragma unroll 1
                for (int tp = 0; tp < TB; tp += TP) {
                    if (tp >= tbv) break;
                    if (!p.dense && ((anyt >> tp) & ((1u << TP) - 1u)) == 0u) continue;
                    float acc[TP][8];
#pragma unroll
                    for (int t = 0; t < TP; ++t)
#pragma unroll
                        for (int e = 0; e < 8; ++e) acc[t][e] = 0.f;
                    for (int ub = 0; ub < nU; ub += RB) {
                        Row8<WT> w[RB];
                        if (PRE && cb == 0 && tp == 0 && ub == 0) {
#pragma unroll
                            for (int j = 0; j < RB; ++j) w[j] = vpre[PRE ? j : 0];
                        } else {
#pragma unroll
                            for (int j = 0; j < RB; ++j) {
                                if (ub + j < nU && cc < ncd) w[j].load(Vt + static_cast<int64_t>(row0 + ulist[ub + j]) * d, cc);
                                else w[j].zero();
                            }
                        }
#pragma unroll
                        for (int j = 0; j < RB; ++j) {
                            if (ub + j < nU) {
                                float wf[8];
                                w[j].unpack(wf);
#pragma unroll
                                for (int t = 0; t < TP; ++t) {
                                    const float u = u_loc[static_cast<size_t>(tp + t) * rpc + ub + j];
                                    if (u != 0.f || p.dense) {
#pragma unroll
                                        for (int e = 0; e < 8; ++e) acc[t][e] = fmaf(u, wf[e], acc[t][e]);
                                    }
                                }
                            }
                        }
                    }
                    if (cc < ncd) {
#pragma unroll
                        for (int t = 0; t < TP; ++t) {
                            if (tp + t < tbv && ((anyt >> (tp + t)) & 1u)) {
                                float* dst = yg + static_cast<int64_t>(tp + t) * d + cc * 8;
                                red_add_v4(dst, acc[t][0], acc[t][1], acc[t][2], acc[t][3]);
                                red_add_v4(dst + 4, acc[t][4], acc[t][5], acc[t][6], acc[t][7]);
                            }
                        }
                    }
                }
            }
        }
        p.trace.mark(8);
        __syncthreads();      // shared buffers are reused by the next token group
    }
    if (cta == 0 && tid == 0) p.hdr->epoch = s_epoch + 1u;   // every block has read the epoch by now
}

template <typename WT, int TB>
int launch_one(spark_ctx* ctx, FfnParams& p, size_t smem, cudaStream_t stream) {
    static bool configured[64] = {};
    auto kern = ffn_kernel<WT, TB>;
    if (ctx->device >= 0 && ctx->device < 64 && !configured[ctx->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin - 1024) != cudaSuccess)
            return SPARK_ERR_CUDA;
        configured[ctx->device] = true;
    }
    p.overlap = ctx->overlap;
    void* args[] = {&p};
    return launch_kernel(ctx, reinterpret_cast<const void*>(kern), static_cast<unsigned>(ctx->num_sms), kThreads, smem, stream, true, args) == cudaSuccess
               ? SPARK_OK : SPARK_ERR_CUDA;
}

template <typename WT>
int launch_tb(spark_ctx* ctx, FfnParams& p, int tb, size_t smem, cudaStream_t stream) {
    switch (tb) {
        case 1: return launch_one<WT, 1>(ctx, p, smem, stream);
        case 4: return launch_one<WT, 4>(ctx, p, smem, stream);
        case 8: return launch_one<WT, 8>(ctx, p, smem, stream);
        default: return launch_one<WT, 16>(ctx, p, smem, stream);
    }
}

}  // namespace

namespace spark {

// From this many tokens on the chunk path on the tcgen05 tensor cores (reads every weight row) is at least as
// fast as the union-gather kernels, measured at the Gemma-2 shapes with independent and with correlated tokens.
constexpr int kTcMinTokens = 5;

int ffn_launch(spark_ctx* ctx, const FfnArgs& a, cudaStream_t stream) {
    if (ctx == nullptr || a.x == nullptr || a.K1t == nullptr || a.K2t == nullptr || a.Vt == nullptr || a.y == nullptr)
        return SPARK_ERR_INVALID_ARG;
    if (a.B < 1 || a.B > 64 || a.d < 16 || a.d_ff < 2 || a.r <= 0 || a.r >= a.d || a.k <= 0) return SPARK_ERR_INVALID_ARG;
    if (a.idx != nullptr && a.count == nullptr) return SPARK_ERR_INVALID_ARG;
    if (a.y_init == a.y && a.y_init != nullptr) return SPARK_ERR_INVALID_ARG;
    if (a.wdtype != SPARK_F32 && a.wdtype != SPARK_BF16 && a.wdtype != SPARK_FP8_E4M3) return SPARK_ERR_UNSUPPORTED;
    if (a.wdtype == SPARK_FP8_E4M3 && (a.K1s == nullptr || a.K2s == nullptr || a.Vs == nullptr)) return SPARK_ERR_INVALID_ARG;
    if (a.wdtype == SPARK_FP8_E4M3 && (a.B > 4 || a.d > 4096)) return SPARK_ERR_UNSUPPORTED;      // one to four tokens
    if ((a.r & 7) != 0 || (a.d & 7) != 0) return SPARK_ERR_UNSUPPORTED;
    if (!aligned16(a.x) || !aligned16(a.K1t) || !aligned16(a.K2t) || !aligned16(a.Vt) || !aligned16(a.y) ||
        !aligned16(a.y_init) || !aligned16(a.norm_w))
        return SPARK_ERR_UNSUPPORTED;
    if (a.d > (1 << 20) || a.d_ff > (1 << 24)) return SPARK_ERR_UNSUPPORTED;
    if (!on_device(ctx)) return SPARK_ERR_INVALID_ARG;

    const int grid = ctx->num_sms;
    const int tb = a.B == 1 ? 1 : (a.B <= 4 ? 4 : (a.B <= 8 ? 8 : 16));
    FfnParams p;
    p.x = a.x; p.norm_w = a.norm_w; p.eps = a.rms_eps;
    p.K1t = a.K1t; p.K2t = a.K2t; p.Vt = a.Vt;
    p.K1s = a.wdtype == SPARK_FP8_E4M3 ? a.K1s : nullptr;
    p.K2s = a.wdtype == SPARK_FP8_E4M3 ? a.K2s : nullptr;
    p.Vs = a.wdtype == SPARK_FP8_E4M3 ? a.Vs : nullptr;
    p.B = static_cast<int>(a.B); p.d = static_cast<int>(a.d); p.d_ff = static_cast<int>(a.d_ff); p.r = static_cast<int>(a.r);
    p.rpc = static_cast<int>((a.d_ff + grid - 1) / grid);
    p.xw = static_cast<int>(a.r > a.d - a.r ? a.r : a.d - a.r);
    p.dense = (a.flags & SPARK_DENSE_LOADS) ? 1 : 0;
    p.erf_form = (a.flags & SPARK_GELU_ERF) ? 1 : 0;
    p.identity = a.k >= a.d_ff ? 1 : 0;
    p.z = p.identity ? 0.0 : spark_normal_upper_quantile(static_cast<double>(a.k) / static_cast<double>(a.d_ff));
    p.y_init = a.y_init; p.y = a.y; p.theta = a.theta; p.count = a.count; p.idx = a.idx;
    p.ncopy = 0;
    p.inv_n = 1.0 / static_cast<double>(a.d_ff);
    p.inv_nm1 = 1.0 / static_cast<double>(a.d_ff - 1);
    p.hdr = ctx->hdr;
    p.trace = PhaseTrace{ctx->trace, ctx->trace_cap};
    p.extra_arrivals = ctx->debug_extra_arrivals;
    p.pf = a.pf;
    p.check_finite = (a.flags & SPARK_CHECK_FINITE) ? 1 : 0;
    const size_t smem = (static_cast<size_t>(tb) * p.xw + static_cast<size_t>(2) * tb * p.rpc) * sizeof(float) +
                        static_cast<size_t>(p.rpc) * 8;
    if (smem > static_cast<size_t>(ctx->max_smem_optin - 1024)) return SPARK_ERR_UNSUPPORTED;
    if (a.wdtype == SPARK_FP8_E4M3) {
        if (grid > 512) return SPARK_ERR_UNSUPPORTED;
        if (a.B == 1) return ffn1_launch(ctx, p, a.wdtype, stream);
        const int rc = ffn_few_launch(ctx, p, a.wdtype, stream);
        return rc == SPARK_ERR_WORKSPACE ? SPARK_ERR_UNSUPPORTED : rc;
    }
    if (a.B == 1 && grid <= 512 && a.d <= 4096) return ffn1_launch(ctx, p, a.wdtype, stream);
    if (a.B >= 2 && a.B <= 4 && grid <= 512) {
        const int rc = ffn_few_launch(ctx, p, a.wdtype, stream);
        if (rc != SPARK_ERR_WORKSPACE) return rc;
    }
    if (a.B >= kTcMinTokens && a.B <= 64 && a.wdtype == SPARK_BF16) {      // reads every row: SPARK_DENSE_LOADS changes nothing here
        const int rc = ffn_tc_launch(ctx, p, stream);
        if (rc != SPARK_ERR_WORKSPACE) return rc;
    }
    if (a.B >= 2 && a.wdtype == SPARK_BF16) {
        const int rc = ffn_mma_launch(ctx, p, stream);
        if (rc != SPARK_ERR_WORKSPACE) return rc;
    }
    if (a.wdtype == SPARK_BF16) return launch_tb<__nv_bfloat16>(ctx, p, tb, smem, stream);
    return launch_tb<float>(ctx, p, tb, smem, stream);
}

}  // namespace spark

extern "C" int spark_ffn_decode(spark_ctx* ctx, const float* x, int64_t B, const void* K1t, const void* K2t,
                                const void* Vt, int wdtype, int64_t d, int64_t d_ff, int64_t r, int64_t k,
                                int flags, float* y, float* theta, int32_t* count, int32_t* idx, void* stream) {
    FfnArgs a;
    a.x = x; a.norm_w = nullptr; a.rms_eps = 0.f;
    a.K1t = K1t; a.K2t = K2t; a.Vt = Vt; a.wdtype = wdtype;
    a.K1s = nullptr; a.K2s = nullptr; a.Vs = nullptr;
    a.B = B; a.d = d; a.d_ff = d_ff; a.r = r; a.k = k; a.flags = flags;
    a.y_init = nullptr; a.y = y; a.theta = theta; a.count = count; a.idx = idx;
    return ffn_launch(ctx, a, static_cast<cudaStream_t>(stream));
}

// FP8 storage of the three matrices with one fp32 scale per neuron (the paper's closing section expects
// quantisation to compound with activation sparsity: it halves the bytes of what is still read).
extern "C" int spark_ffn_decode_fp8(spark_ctx* ctx, const float* x, int64_t B, const void* K1t, const float* K1s,
                                    const void* K2t, const float* K2s, const void* Vt, const float* Vs, int64_t d,
                                    int64_t d_ff, int64_t r, int64_t k, int flags, float* y, float* theta, int32_t* count,
                                    int32_t* idx, void* stream) {
    FfnArgs a;
    a.x = x; a.norm_w = nullptr; a.rms_eps = 0.f;
    a.K1t = K1t; a.K2t = K2t; a.Vt = Vt; a.wdtype = SPARK_FP8_E4M3;
    a.K1s = K1s; a.K2s = K2s; a.Vs = Vs;
    a.B = B; a.d = d; a.d_ff = d_ff; a.r = r; a.k = k; a.flags = flags;
    a.y_init = nullptr; a.y = y; a.theta = theta; a.count = count; a.idx = idx;
    return ffn_launch(ctx, a, static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------
// spark_ffn_decode_noalloc: the same FFN for callers that cannot allocate device memory.
// ---------------------------------------------------------------------------------------------
namespace {

// The inter-block state the FFN kernels need (status word, launch epoch, score-sum cells) lives in
// this file-scope array instead of a caller-provided workspace.  It is zero when the module is
// loaded, which is the idle state (so the first call has nothing to clear); every device that loads
// the library carries its own copy (about 140 KB) until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_state[sizeof(WsHeader)];

struct NoallocDevice {
    std::atomic<bool> ready{false};
    WsHeader* state = nullptr;      // device address of g_noalloc_state on this device
    int num_sms = 0, max_smem_optin = 0;
};
NoallocDevice g_noalloc[64];
std::mutex g_noalloc_mutex;         // first calls from several host threads: one of them does the set-up

// Once per device, with that device current: in host code the array's name is only a stand-in for
// the symbol, so its device address has to be asked for.  Allocates nothing.
int noalloc_device(NoallocDevice** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SPARK_ERR_CUDA;
    if (dev < 0 || dev >= 64) return SPARK_ERR_UNSUPPORTED;
    NoallocDevice& nd = g_noalloc[dev];
    if (!nd.ready.load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (!nd.ready.load(std::memory_order_relaxed)) {
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_noalloc_state) != cudaSuccess || ptr == nullptr) return SPARK_ERR_CUDA;
            if (cudaDeviceGetAttribute(&nd.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return SPARK_ERR_CUDA;
            if (cudaDeviceGetAttribute(&nd.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess)
                return SPARK_ERR_CUDA;
            nd.state = static_cast<WsHeader*>(ptr);
            nd.ready.store(true, std::memory_order_release);
        }
    }
    *out = &nd;
    return SPARK_OK;
}

}  // namespace

extern "C" int spark_ffn_decode_noalloc(const float* x, int64_t B, const void* K1t, const void* K2t, const void* Vt,
                                        int wdtype, int64_t d, int64_t d_ff, int64_t r, int64_t k, int flags,
                                        float* y, float* theta, void* stream) {
    if (B > SPARK_NOALLOC_MAX_TOKENS) return SPARK_ERR_UNSUPPORTED;   // beyond what the static state serves
    NoallocDevice* nd = nullptr;
    const int rc = noalloc_device(&nd);
    if (rc != SPARK_OK) return rc;
    int dev = -1;
    cudaGetDevice(&dev);
    spark_ctx local;
    local.device = dev;
    local.num_sms = nd->num_sms;
    local.max_smem_optin = nd->max_smem_optin;
    local.ws = reinterpret_cast<char*>(nd->state);
    local.ws_bytes = sizeof(WsHeader);
    local.hdr = nd->state;
    local.scratch = nullptr;
    local.scratch_bytes = 0;
    local.trace = nullptr;
    local.trace_cap = 0;
    local.overlap = 0;
    local.wait_kcycles = 0;
    local.fused = 0;
    local.chunk_dense = 0;
    local.len_hint = 0;
    local.l2_prefetch = 0;
    local.next_wqkv = nullptr;
    local.debug_extra_arrivals = 0;
    FfnArgs a;
    a.x = x; a.norm_w = nullptr; a.rms_eps = 0.f;
    a.K1t = K1t; a.K2t = K2t; a.Vt = Vt; a.wdtype = wdtype;
    a.K1s = nullptr; a.K2s = nullptr; a.Vs = nullptr;
    a.B = B; a.d = d; a.d_ff = d_ff; a.r = r; a.k = k; a.flags = flags;
    a.y_init = nullptr; a.y = y; a.theta = theta; a.count = nullptr; a.idx = nullptr;
    return ffn_launch(&local, a, static_cast<cudaStream_t>(stream));
}

// The device status of the no-allocation entry point: what spark_device_status is for a context.
extern "C" int spark_noalloc_status(void* stream, int* host_out) {
    if (host_out == nullptr) return SPARK_ERR_INVALID_ARG;
    NoallocDevice* nd = nullptr;
    const int rc = noalloc_device(&nd);
    if (rc != SPARK_OK) return rc;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return SPARK_ERR_CUDA;
    int status = 0;
    if (cudaMemcpy(&status, &nd->state->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return SPARK_ERR_CUDA;
    *host_out = status;
    if (status != SPARK_OK) {
        // a wait that ran out left arrivals and partial sums behind: back to the idle (zero) state
        if (cudaMemset(nd->state, 0, sizeof(WsHeader)) != cudaSuccess) return SPARK_ERR_CUDA;
        if (cudaDeviceSynchronize() != cudaSuccess) return SPARK_ERR_CUDA;
    }
    return SPARK_OK;
}
