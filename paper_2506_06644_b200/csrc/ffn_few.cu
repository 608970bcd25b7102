// Spark FFN (Section 2.1, Eq. 2) for TWO TO FOUR tokens: the one-token kernel's structure (no staging of
// split activations, no tensor cores, one exchange of score sums) with the gather turned around so that
// it needs no per-warp copies of the output:
//   A   each block streams its share of K1t once (registers) and forms the scores of every token;
//   S   per-token score sums into the cell sets of a token group, ONE arrival per block, theta per token;
//   C   the block's union list (neurons active for any token, Appendix B) with a token mask per entry;
//   D   up to 32 entries per round: every thread copies "its" 16-byte column chunk of each entry's Vt row into
//       shared memory (cp.async: no registers, all rows in flight at once) while a warp per two entries
//       requests their K2t rows, forms t = K2[:,i] . x[r:] and u = GELU(s - theta) t per token and leaves u
//       in shared memory; the threads then add u V[:,i] into register accumulators: a thread owns eight
//       columns of y for all tokens;
//   R   every thread adds its eight columns to global memory with vector reductions.
// y is initialised by the first few blocks at kernel start; the released arrival of S orders that
// before any block's reductions into y.
#include <type_traits>

#include "ffn_params.h"
#include "kernels.h"
#include "rowdot.cuh"

using namespace spark;

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / kWarp;
constexpr int kRows = 4;
constexpr int kKB = 5;            // K2t chunks per lane per batch (a batch spans 1280 columns)
constexpr int kXV = 5;            // float4 of the tokens' inputs a thread holds (NT * d / 4 <= kXV * 512)

template <typename WT, int NT>
__global__ void __launch_bounds__(kThreads, 1) ffn_few_kernel(const FfnParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* xs = reinterpret_cast<float*>(smem_raw);                          // [NT][d]   the (normalised) inputs
    float* s_loc = xs + static_cast<size_t>(NT) * p.d;                       // [NT][rpc] scores of this block's neurons
    float* uval = s_loc + static_cast<size_t>(NT) * p.rpc;                   // [NT][32]  u of the entries in flight
    int* ulist = reinterpret_cast<int*>(uval + NT * 32);                     // [rpc]     union list (local neuron index)
    unsigned* umask = reinterpret_cast<unsigned*>(ulist + p.rpc);            // [rpc]     tokens that entry is active for
    unsigned char* vstage = smem_raw + p.vstage_off;                         // [vrows][d] the round's rows of V (16-byte aligned)
    __shared__ float red_s[kWarps][NT];
    __shared__ float theta_s[NT];
    __shared__ unsigned s_epoch;
    __shared__ int s_nu, s_fail;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int grid = gridDim.x, cta = blockIdx.x;
    const int row0 = static_cast<int>(static_cast<int64_t>(cta) * p.d_ff / grid);
    const int row1 = static_cast<int>(static_cast<int64_t>(cta + 1) * p.d_ff / grid);
    const int nloc = row1 - row0;
    const int d = p.d, r = p.r, d2 = d - r, rpc = p.rpc, B = p.B;
    const WT* K1t = static_cast<const WT*>(p.K1t);
    const WT* K2t = static_cast<const WT*>(p.K2t);
    const WT* Vt = static_cast<const WT*>(p.Vt);
    const int d4 = d / 4, tot4 = NT * d4;
    constexpr bool kScaled = sizeof(WT) == 1;      // FP8 storage: one fp32 scale per neuron and matrix
    constexpr unsigned kChunkB = 8 * sizeof(WT);   // bytes of a thread's eight columns of a row of V

    // Everything another kernel may have written is read in after_dependency(): with launch overlap after the
    // first batch of K1t loads has been issued, otherwise before them (requests are served in issue order).
    float4 xv[kXV];
    auto after_dependency = [&]() {
        dep_wait();
        dep_trigger();
#pragma unroll
        for (int k = 0; k < kXV; ++k) {
            const int i = tid + k * kThreads;
            xv[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i < tot4) {
                const int t = i / d4, c = i - t * d4;
                if (t < B) xv[k] = reinterpret_cast<const float4*>(p.x + static_cast<int64_t>(t) * d)[c];
            }
        }
        if (tid == 0) {
            s_epoch = ld_acquire_u32(&p.hdr->epoch);            // consumed after phase A
            s_nu = 0;
            s_fail = 0;
        }
        if (cta == 0) {
            // clear the cells the launch after next will use (last used two launches ago)
            const unsigned e = ld_acquire_u32(&p.hdr->epoch);
            SumCell* c = &p.hdr->ffn_cells[(e + 2u) & 3u][0][0][0];
            for (int i = tid; i < 4 * 16 * kCellWays; i += kThreads) { c[i].s1 = 0.0; c[i].s2 = 0.0; c[i].count = 0u; }
        }
        p.trace.mark(0);
    };
    if (!p.overlap) after_dependency();
    // Runs once the first K1t loads are in flight: y initialisation, optional RMSNorm, x to shared memory.
    auto prologue = [&]() {
        {
            const int64_t total4 = static_cast<int64_t>(B) * d4;
            const float4* yi = p.y_init ? reinterpret_cast<const float4*>(p.y_init) : nullptr;
            float4* yo = reinterpret_cast<float4*>(p.y);
            for (int64_t i = static_cast<int64_t>(cta) * kThreads + tid; i < total4; i += static_cast<int64_t>(grid) * kThreads)
                yo[i] = yi ? yi[i] : make_float4(0.f, 0.f, 0.f, 0.f);
            if (cta == 0 && p.count != nullptr && tid < B) p.count[tid] = 0;
        }
        float sc[NT];
#pragma unroll
        for (int t = 0; t < NT; ++t) sc[t] = 1.f;
        if (p.norm_w != nullptr) {
            float ss[NT];
#pragma unroll
            for (int t = 0; t < NT; ++t) ss[t] = 0.f;
#pragma unroll
            for (int k = 0; k < kXV; ++k) {
                const int t = (tid + k * kThreads) / d4;
                const float q = xv[k].x * xv[k].x + xv[k].y * xv[k].y + xv[k].z * xv[k].z + xv[k].w * xv[k].w;
#pragma unroll
                for (int u = 0; u < NT; ++u) ss[u] += t == u ? q : 0.f;
            }
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                const float v = warp_sum(ss[t]);
                if (lane == 0) red_s[warp][t] = v;
            }
            __syncthreads();
#pragma unroll
            for (int t = 0; t < NT; ++t) {
                float tot = 0.f;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) tot += red_s[w][t];
                sc[t] = rsqrtf(tot / static_cast<float>(d) + p.eps);
            }
        }
#pragma unroll
        for (int k = 0; k < kXV; ++k) {
            const int i = tid + k * kThreads;
            if (i < tot4) {
                const int t = i / d4;
                float s = 1.f;
#pragma unroll
                for (int u = 0; u < NT; ++u) s = t == u ? sc[u] : s;
                // the norm weights are read here, not with the inputs: registers are short while the first batch
                // of K1t rows is held, and this read hides behind their latency
                const float4 nw = p.norm_w != nullptr ? __ldg(reinterpret_cast<const float4*>(p.norm_w) + (i - t * d4))
                                                      : make_float4(1.f, 1.f, 1.f, 1.f);
                reinterpret_cast<float4*>(xs)[i] = make_float4(xv[k].x * s * nw.x, xv[k].y * s * nw.y, xv[k].z * s * nw.z, xv[k].w * s * nw.w);
            }
        }
        __syncthreads();
        p.trace.mark(1);
    };

    // ---- A: predictor scores s = K1^T x[:r] of this block's neurons, every token -----------------------
    rows_dot<WT, NT, kRows>(K1t, r, row0, nloc, r / 8, xs, d, [&]() { if (p.overlap) after_dependency(); }, prologue,
                            [&](int j, int t, float v) { s_loc[static_cast<size_t>(t) * rpc + j] = kScaled ? v * __ldg(p.K1s + row0 + j) : v; });
    __syncthreads();
    p.trace.mark(2);

    // ---- S: per-token sums into the group's cell sets, one arrival per block, theta per token ------------
    SumCell* cells = &p.hdr->ffn_cells[s_epoch & 3u][0][0][0];               // [token][way]
    if (warp < B) {
        const float* sr = s_loc + static_cast<size_t>(warp) * rpc;
        double s1 = 0.0, s2 = 0.0;
        for (int j = lane; j < nloc; j += 32) {
            const double v = static_cast<double>(sr[j]);
            s1 += v;
            s2 = fma(v, v, s2);
        }
        s1 = warp_sum_f64(s1);
        s2 = warp_sum_f64(s2);
        if (lane == 0) cells_add_sums_w<kCellWays>(cells + warp * kCellWays, cta, s1, s2);
    }
    __syncthreads();
    if (tid == 0) cells_arrive_w<kCellWays>(cells, cta);       // after every token's sums; also orders y's initialisation
    p.trace.mark(3);
    if (warp == 0) {
        const bool ok = cells_wait_arrivals_w<kCellWays>(cells, static_cast<unsigned>(grid), p.hdr);
        if (lane == 0 && !ok) s_fail = 1;
    }
    __syncthreads();
    if (s_fail) return;
    if (warp < B) {
        double sa, sb;
        cells_read_w<kCellWays>(cells + warp * kCellWays, sa, sb);
        if (lane == 0) {
            float th = -INFINITY;
            if (!p.identity) {
                const double mean = sa * p.inv_n;
                const float var = static_cast<float>((sb - sa * mean) * p.inv_nm1);
                th = static_cast<float>(mean) + sqrtf(fmaxf(var, 0.f)) * static_cast<float>(p.z);
            }
            theta_s[warp] = th;
            if (cta == 0 && p.theta != nullptr) p.theta[warp] = th;
        }
    } else if (warp < NT && lane == 0) {
        theta_s[warp] = INFINITY;                   // token slots beyond B select nothing
    }
    __syncthreads();
    p.trace.mark(4);
    if (cta == 0 && tid == 0) p.hdr->epoch = s_epoch + 1u;     // every block has read the epoch by now

    // ---- C: the block's union list -------------------------------------------------------------------
    for (int j = tid; j < nloc; j += kThreads) {
        unsigned m = 0u;
#pragma unroll
        for (int t = 0; t < NT; ++t)
            if (s_loc[static_cast<size_t>(t) * rpc + j] > theta_s[t]) m |= 1u << t;
        if (m != 0u || p.dense) {
            const int pos = atomicAdd(&s_nu, 1);
            ulist[pos] = j;
            umask[pos] = m;
        }
    }
    __syncthreads();
    const int nU = s_nu;
    if (p.count != nullptr && warp < B) {           // optional outputs: per-token count and index list (any order)
        int c = 0;
        for (int e = lane; e < nU; e += 32) c += (umask[e] >> warp) & 1u;
        c = warp_sum_int(c);
        int base = 0;
        if (lane == 0 && c > 0) base = atomicAdd(&p.count[warp], c);
        base = __shfl_sync(kFull, base, 0);
        if (p.idx != nullptr && c > 0) {
            int32_t* out = p.idx + static_cast<int64_t>(warp) * p.d_ff;
            for (int e0 = 0; e0 < nU; e0 += 32) {
                const int e = e0 + lane;
                const bool a = e < nU && ((umask[e] >> warp) & 1u);
                const unsigned bal = __ballot_sync(kFull, a);
                if (a) out[base + __popc(bal & ((1u << lane) - 1u))] = row0 + ulist[e];
                base += __popc(bal);
            }
        }
    }
    p.trace.mark(5);

    // ---- D: up to kE union entries per round ------------------------------------------------------------
    const int nc2 = d2 / 8, ncd = d / 8;
    const bool vcol = tid < ncd;                    // this thread owns columns [8 tid, 8 tid + 8) of y
    const int E = p.vrows;                          // entries per round: 16 or 32 (rows of V the staging area holds)
    float acc[NT][8];
#pragma unroll
    for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[t][e] = 0.f;
    const unsigned vs0 = static_cast<unsigned>(__cvta_generic_to_shared(vstage));
#pragma unroll 1
    for (int e0 = 0; e0 < nU; e0 += E) {
        const int ne = min(E, nU - e0);
        // the rows of V go to shared memory without passing through registers: every thread copies "its" 16-byte
        // column chunk of every row of the round, all in flight at once
        if (vcol) {
            for (int q = 0; q < ne; ++q) {
                const WT* src = Vt + static_cast<int64_t>(row0 + ulist[e0 + q]) * d + 8 * tid;
                if constexpr (kScaled)
                    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(vs0 + kChunkB * static_cast<unsigned>(q * ncd + tid)), "l"(src) : "memory");
                else
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(vs0 + kChunkB * static_cast<unsigned>(q * ncd + tid)), "l"(src) : "memory");
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        // a warp takes entries w and w + 16: their K2t rows are requested together
        bool mine[2];
        int jm[2];
        const WT* krow[2];
        Row8<WT> kw[2][kKB];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mine[h] = warp + 16 * h < ne;
            jm[h] = mine[h] ? ulist[e0 + warp + 16 * h] : 0;
            krow[h] = K2t + static_cast<int64_t>(row0 + jm[h]) * d2;
#pragma unroll
            for (int u = 0; u < kKB; ++u) {
                const int c = u * 32 + lane;
                if (mine[h] && c < nc2) kw[h][u].load(krow[h], c); else kw[h][u].zero();
            }
        }
        float tv[2][NT];
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int t = 0; t < NT; ++t) tv[h][t] = 0.f;
#pragma unroll 1
        for (int c0 = 0;;) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int u = 0; u < kKB; ++u) {
                    const int c = c0 + u * 32 + lane;
                    const int cs = c < nc2 ? c : 0;
                    float wf[8];
                    kw[h][u].unpack(wf);
#pragma unroll
                    for (int t = 0; t < NT; ++t) {
                        const float4* xr = reinterpret_cast<const float4*>(xs + static_cast<size_t>(t) * d + r) + 2 * cs;
                        tv[h][t] = dot8(wf, xr[0], xr[1], tv[h][t]);
                    }
                }
            }
            c0 += kKB * 32;
            if (c0 >= nc2) break;
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int u = 0; u < kKB; ++u) {       // rows longer than one batch: further batches
                    const int c = c0 + u * 32 + lane;
                    if (mine[h] && c < nc2) kw[h][u].load(krow[h], c); else kw[h][u].zero();
                }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
#pragma unroll
            for (int t = 0; t < NT; ++t) tv[h][t] = warp_sum(tv[h][t]);
            if (lane < NT) {
                float u = 0.f;
                if (mine[h] && ((umask[e0 + warp + 16 * h] >> lane) & 1u)) {
                    float tl = tv[h][0];
#pragma unroll
                    for (int t = 1; t < NT; ++t) tl = lane == t ? tv[h][t] : tl;
                    const float a = s_loc[static_cast<size_t>(lane) * rpc + jm[h]] - (p.identity ? 0.f : theta_s[lane]);
                    u = (p.erf_form ? gelu_erf(a) : gelu_tanh(a)) * tl;
                    if constexpr (kScaled) u *= __ldg(p.K2s + row0 + jm[h]) * __ldg(p.Vs + row0 + jm[h]);
                }
                uval[lane * 32 + warp + 16 * h] = u;
            }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        if (vcol) {
            for (int q = 0; q < ne; ++q) {
                Row8<WT> v8;
                v8.raw = reinterpret_cast<const decltype(v8.raw)*>(vstage)[q * ncd + tid];
                float wf[8];
                v8.unpack(wf);
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                    const float u = uval[t * 32 + q];
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[t][e] = fmaf(u, wf[e], acc[t][e]);
                }
            }
        }
        __syncthreads();        // the staging area and uval are rewritten by the next round
    }
    p.trace.mark(7);

    // ---- R: every thread's eight columns, every token ---------------------------------------------------
    if (vcol && nU > 0) {
#pragma unroll
        for (int t = 0; t < NT; ++t) {
            if (t < B) {
                float* yt = p.y + static_cast<int64_t>(t) * d + 8 * tid;
                red_add_v4(yt, acc[t][0], acc[t][1], acc[t][2], acc[t][3]);
                red_add_v4(yt + 4, acc[t][4], acc[t][5], acc[t][6], acc[t][7]);
            }
        }
    }
    p.trace.mark(8);
}

}  // namespace

namespace spark {

// Serves 2..4 tokens, bf16 weights, with d <= 4096 (a thread owns one 16-byte column chunk of V) and inputs that fit the
// registers of the prologue; anything else: SPARK_ERR_WORKSPACE (the caller takes the tensor-core kernel).
int ffn_few_launch(spark_ctx* ctx, FfnParams& p, int wdtype, cudaStream_t stream) {
    static bool configured[4][64] = {};
    const int nt = p.B <= 2 ? 2 : 4;
    const bool f8 = wdtype == SPARK_FP8_E4M3;
    if (p.B < 2 || p.B > 4 || p.d / 8 > kThreads || nt * (p.d / 4) > kXV * kThreads) return SPARK_ERR_WORKSPACE;
    if (wdtype != SPARK_BF16 && wdtype != SPARK_FP8_E4M3) return SPARK_ERR_WORKSPACE;        // fp32 weights double the registers per chunk: not served
    size_t fixed = (static_cast<size_t>(nt) * p.d + static_cast<size_t>(nt) * p.rpc + nt * 32 + 2 * static_cast<size_t>(p.rpc)) * 4;
    fixed = (fixed + 15) & ~static_cast<size_t>(15);
    const size_t limit = static_cast<size_t>(ctx->max_smem_optin - 2048);
    const size_t rowb = static_cast<size_t>(p.d) * (f8 ? 1 : 2);
    if (fixed + 16 * rowb > limit) return SPARK_ERR_WORKSPACE;
    p.vrows = fixed + 32 * rowb <= limit ? 32 : 16;
    p.vstage_off = static_cast<int>(fixed);
    const size_t smem = fixed + static_cast<size_t>(p.vrows) * rowb;
    const void* kern = f8 ? (nt == 2 ? reinterpret_cast<const void*>(ffn_few_kernel<__nv_fp8_e4m3, 2>)
                                     : reinterpret_cast<const void*>(ffn_few_kernel<__nv_fp8_e4m3, 4>))
                          : (nt == 2 ? reinterpret_cast<const void*>(ffn_few_kernel<__nv_bfloat16, 2>)
                                     : reinterpret_cast<const void*>(ffn_few_kernel<__nv_bfloat16, 4>));
    const int ki = (nt == 2 ? 0 : 1) + (f8 ? 2 : 0);
    if (ctx->device >= 0 && ctx->device < 64 && !configured[ki][ctx->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin - 1024) != cudaSuccess)
            return SPARK_ERR_CUDA;
        configured[ki][ctx->device] = true;
    }
    p.overlap = ctx->overlap;
    void* args[] = {&p};
    return launch_kernel(ctx, kern, static_cast<unsigned>(ctx->num_sms), kThreads, smem, stream, true, args) == cudaSuccess
               ? SPARK_OK : SPARK_ERR_CUDA;
}

}  // namespace spark
