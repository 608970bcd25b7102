// Spark FFN (Section 2.1, Eq. 2) for ONE token: the latency-critical decode case.
//
// One cooperative kernel, one 512-thread block per SM, no fence and no atomic counter on the
// critical path:
//   A  each block streams its share of K1t (all 16-byte loads of a warp's four rows in flight at
//      once); x[:r] reaches shared memory while those loads fly; scores stay in shared memory;
//   S  warp 0 adds the block's sum of scores and sum of squares (fp64) into one of 16 32-byte cells
//      and then, with release semantics, its arrival; half a warp per block polls the 16 cells
//      (one 32-byte load each) and forms theta (Eq. 11) as soon as every block has arrived;
//   C  threads push the block's active neurons (s > theta) onto a shared-memory list;
//   D  a warp per active neuron requests its K2t row and its Vt row together (one trip to HBM),
//      forms t = K2[:,i] . x[r:], u = GELU(s - theta) t, and adds u V[:,i] into a shared-memory y;
//   R  the block adds its y to global memory with 16-byte vector reductions.
// y is initialised by the first few blocks at kernel start; the released arrival above orders
// that before any block's reductions into y.
#include "ffn_params.h"
#include "kernels.h"
#include "rowdot.cuh"

using namespace spark;

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / kWarp;
constexpr int kRows = 4;
constexpr int kKB = 8;            // K2t chunks per lane per batch (a batch spans 2048 columns)
constexpr int kVB = 9;            // Vt chunks per lane per batch (a batch spans 2304 columns)

template <typename WT>
__global__ void __launch_bounds__(kThreads, 1) ffn1_kernel(const FfnParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* xs = reinterpret_cast<float*>(smem_raw);             // [d]    the (normalised) input
    float* ys = xs + p.d;                                       // [ncopy][d] per-warp shares of y
    float* s_loc = ys + static_cast<size_t>(p.ncopy) * p.d;                                    // [rpc]  scores of this block's neurons
    int* lst_j = reinterpret_cast<int*>(s_loc + p.rpc);         // [rpc]  active neurons (local index)
    float* lst_a = reinterpret_cast<float*>(lst_j + p.rpc);     // [rpc]  s - theta (or -inf: read, not used)
    float* ksc = lst_a + p.rpc;                                 // [rpc]  scales of this block's K1t rows (1 without)
    __shared__ double red_a[kWarps];
    __shared__ float s_theta;
    __shared__ unsigned s_epoch;
    __shared__ int s_nact, s_fail;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int grid = gridDim.x, cta = blockIdx.x;
    const int row0 = static_cast<int>(static_cast<int64_t>(cta) * p.d_ff / grid);
    const int row1 = static_cast<int>(static_cast<int64_t>(cta + 1) * p.d_ff / grid);
    const int nloc = row1 - row0;
    const int d = p.d, r = p.r, d2 = d - r;
    const WT* K1t = static_cast<const WT*>(p.K1t);
    const WT* K2t = static_cast<const WT*>(p.K2t);
    const WT* Vt = static_cast<const WT*>(p.Vt);
    const int d4 = d / 4;
    const int n_init = (d4 + kThreads - 1) / kThreads;          // blocks that initialise y
    constexpr bool kScaled = sizeof(WT) == 1;                   // FP8 storage: one scale per neuron and matrix
    if constexpr (kScaled)
        for (int j = tid; j < nloc; j += kThreads) ksc[j] = __ldg(p.K1s + row0 + j);   // weights: never written
    // Everything that another kernel may have written is read in after_dependency(): with launch overlap
    // that is after the first batch of K1t loads has been issued (they fly while the kernel before
    // this one in the stream drains); otherwise before them, so that the token's input is in shared memory
    // when the first rows arrive (requests are served in issue order).
    const bool has0 = tid < d4, has1 = tid + kThreads < d4;
    float4 xv0 = make_float4(0.f, 0.f, 0.f, 0.f), xv1 = xv0, nw0 = make_float4(1.f, 1.f, 1.f, 1.f), nw1 = nw0;
    auto after_dependency = [&]() {
        dep_wait();
        dep_trigger();
        if (has0) xv0 = reinterpret_cast<const float4*>(p.x)[tid];
        if (has1) xv1 = reinterpret_cast<const float4*>(p.x)[tid + kThreads];
        if (p.norm_w != nullptr) {
            if (has0) nw0 = reinterpret_cast<const float4*>(p.norm_w)[tid];
            if (has1) nw1 = reinterpret_cast<const float4*>(p.norm_w)[tid + kThreads];
        }
        if (tid == 0) {
            s_epoch = ld_acquire_u32(&p.hdr->epoch);            // consumed after phase A
            s_nact = 0;
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
        if (cta < n_init) {
            const int i = cta * kThreads + tid;
            if (i < d4)
                reinterpret_cast<float4*>(p.y)[i] =
                    p.y_init ? reinterpret_cast<const float4*>(p.y_init)[i] : make_float4(0.f, 0.f, 0.f, 0.f);
            if (cta == 0 && tid == 0 && p.count != nullptr) p.count[0] = 0;
        }
        float sc = 1.f;
        if (p.norm_w != nullptr) {
            float ss = xv0.x * xv0.x + xv0.y * xv0.y + xv0.z * xv0.z + xv0.w * xv0.w +
                       xv1.x * xv1.x + xv1.y * xv1.y + xv1.z * xv1.z + xv1.w * xv1.w;
            ss = warp_sum(ss);
            if (lane == 0) red_a[warp] = static_cast<double>(ss);
            __syncthreads();
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) tot += static_cast<float>(red_a[w]);
            sc = rsqrtf(tot / static_cast<float>(d) + p.eps);
        }
        if (has0) reinterpret_cast<float4*>(xs)[tid] =
            make_float4(xv0.x * sc * nw0.x, xv0.y * sc * nw0.y, xv0.z * sc * nw0.z, xv0.w * sc * nw0.w);
        if (has1) reinterpret_cast<float4*>(xs)[tid + kThreads] =
            make_float4(xv1.x * sc * nw1.x, xv1.y * sc * nw1.y, xv1.z * sc * nw1.z, xv1.w * sc * nw1.w);
        __syncthreads();
        p.trace.mark(1);
    };

    // ---- A: predictor scores s = K1^T x[:r] of this block's neurons ---------------------------------
    rows_dot<WT, 1, kRows>(K1t, r, row0, nloc, r / 8, xs, 0, [&]() { if (p.overlap) after_dependency(); }, prologue,
                           [&](int j, int, float v) { s_loc[j] = kScaled ? v * ksc[j] : v; });
    __syncthreads();
    p.trace.mark(2);

    // While warp 0 exchanges the sums, the other warps ask L2 for the rows this block will most likely gather: the
    // neurons above the threshold estimated from the block's own scores alone.  The gather then finds most of its
    // rows in L2 instead of waiting for DRAM after the exchange (a lower estimate, which catches more of them, measured
    // slower: the extra requests delay the exchange).
    if (tid == kThreads - 1) prefetch_l2_share(p.pf, cta, grid);      // the next kernel's weights: HBM idles during the exchange
    if (warp > 0 && !p.identity && !p.dense && nloc >= 8) {
        float a1 = 0.f, a2 = 0.f;
        for (int j = lane; j < nloc; j += 32) {
            const float v = s_loc[j];
            a1 += v;
            a2 = fmaf(v, v, a2);
        }
        a1 = warp_sum(a1);
        a2 = warp_sum(a2);
        const float mean = a1 / nloc, var = fmaxf((a2 - a1 * mean) / (nloc - 1), 0.f);
        const float guess = mean + sqrtf(var) * static_cast<float>(p.z);
        int seen = 0;
        for (int j0 = 0; j0 < nloc; j0 += 32) {
            const int j = j0 + lane;
            const unsigned bal = __ballot_sync(kFull, j < nloc && s_loc[j] > guess);
            for (unsigned m = bal; m != 0u; m &= m - 1u) {
                if (seen++ % (kWarps - 1) != warp - 1) continue;
                const int jj = j0 + __ffs(m) - 1;
                const char* krow = reinterpret_cast<const char*>(K2t + static_cast<int64_t>(row0 + jj) * d2);
                const char* vrow = reinterpret_cast<const char*>(Vt + static_cast<int64_t>(row0 + jj) * d);
                for (int o = lane * 128; o < d2 * static_cast<int>(sizeof(WT)); o += 32 * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(krow + o));
                for (int o = lane * 128; o < d * static_cast<int>(sizeof(WT)); o += 32 * 128) asm volatile("prefetch.global.L2 [%0];" ::"l"(vrow + o));
            }
        }
    }
    // ---- S: add this block's sums to the grid-wide cell, wait for everybody's, theta ------------------
    if (warp == 0) {
        SumCell* ways = &p.hdr->ffn_cells[s_epoch & 3u][0][0][0];
        double s1 = 0.0, s2 = 0.0;
        for (int j = lane; j < nloc; j += 32) {
            const double v = static_cast<double>(s_loc[j]);
            s1 += v;
            s2 = fma(v, v, s2);
        }
        s1 = warp_sum_f64(s1);
        s2 = warp_sum_f64(s2);
        if (lane == 0) cells_add(ways, cta, s1, s2);    // also orders y's initialisation before the arrival
        p.trace.mark(3);
        double sa, sb;
        const bool ok = cells_wait(ways, static_cast<unsigned>(grid + p.extra_arrivals), sa, sb, p.hdr);
        if (lane == 0) {
            float th = -INFINITY;
            if (!ok) s_fail = 1;
            if (ok && p.check_finite && !(isfinite(sa) && isfinite(sb))) atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_NONFINITE);
            if (!p.identity) {
                const double mean = sa * p.inv_n;
                const float var = static_cast<float>((sb - sa * mean) * p.inv_nm1);
                th = static_cast<float>(mean) + sqrtf(fmaxf(var, 0.f)) * static_cast<float>(p.z);
            }
            s_theta = th;
        }
    }
    __syncthreads();
    if (s_fail) return;
    const float theta = s_theta;
    p.trace.mark(4);
    if (cta == 0 && tid == 0) {
        if (p.theta != nullptr) p.theta[0] = theta;
        p.hdr->epoch = s_epoch + 1u;                // every block has read the epoch by now
    }
    p.trace.mark(5);

    // ---- C: this block's active neurons ------------------------------------------------------------
    for (int j = tid; j < nloc; j += kThreads) {
        const float s = s_loc[j];
        const bool act = s > theta;
        if (act || p.dense) {
            const int pos = atomicAdd(&s_nact, 1);
            lst_j[pos] = j;
            lst_a[pos] = act ? (p.identity ? s : s - theta) : -INFINITY;
        }
    }
    __syncthreads();
    const int nact = s_nact;
    if (p.count != nullptr && tid == 0) {           // optional outputs: count and the index list
        int mine = 0;
        for (int e = 0; e < nact; ++e) mine += lst_a[e] != -INFINITY;
        if (mine > 0) {
            int pos = atomicAdd(&p.count[0], mine);
            if (p.idx != nullptr)
                for (int e = 0; e < nact; ++e)
                    if (lst_a[e] != -INFINITY) p.idx[pos++] = row0 + lst_j[e];
        }
    }
    p.trace.mark(6);

    // ---- D: a warp per active neuron: K2t row and Vt row requested together --------------------------
    const int nc2 = d2 / 8, ncd = d / 8;
    // Warp w < ncopy owns copy w of y in shared memory: its first neuron stores, the others add.
    const int ncopy = p.ncopy;
    float* ymine = ys + static_cast<size_t>(warp) * d;
    bool first = true;
#pragma unroll 1
    for (int e = warp; e < nact && warp < ncopy; e += ncopy) {
        const int j = lst_j[e];
        const float aj = lst_a[e];
        const WT* krow = K2t + static_cast<int64_t>(row0 + j) * d2;
        const WT* vrow = Vt + static_cast<int64_t>(row0 + j) * d;
        float rsc = 1.f;
        if constexpr (kScaled) rsc = __ldg(p.K2s + row0 + j) * __ldg(p.Vs + row0 + j);
        Row8<WT> kw[kKB], vw[kVB];
#pragma unroll
        for (int u = 0; u < kKB; ++u) {
            const int c = u * 32 + lane;
            if (c < nc2) kw[u].load(krow, c); else kw[u].zero();
        }
#pragma unroll
        for (int u = 0; u < kVB; ++u) {
            const int c = u * 32 + lane;
            if (c < ncd) vw[u].load(vrow, c); else vw[u].zero();
        }
        float t = 0.f;
#pragma unroll 1
        for (int c0 = 0;;) {
#pragma unroll
            for (int u = 0; u < kKB; ++u) {
                const int c = c0 + u * 32 + lane;
                const int cs = c < nc2 ? c : 0;
                float wf[8];
                kw[u].unpack(wf);
                const float4* xr = reinterpret_cast<const float4*>(xs + r) + 2 * cs;
                t = dot8(wf, xr[0], xr[1], t);
            }
            c0 += kKB * 32;
            if (c0 >= nc2) break;
#pragma unroll
            for (int u = 0; u < kKB; ++u) {         // rows longer than 2048 columns: further batches
                const int c = c0 + u * 32 + lane;
                if (c < nc2) kw[u].load(krow, c); else kw[u].zero();
            }
        }
        t = warp_sum(t);
        float uval = aj == -INFINITY ? 0.f : (p.erf_form ? gelu_erf(aj) : gelu_tanh(aj)) * t;
        if constexpr (kScaled) uval *= rsc;
#pragma unroll 1
        for (int c0 = 0;;) {
#pragma unroll
            for (int u = 0; u < kVB; ++u) {
                const int c = c0 + u * 32 + lane;
                if (c < ncd) {
                    float wf[8];
                    vw[u].unpack(wf);
                    float4* dst = reinterpret_cast<float4*>(ymine + c * 8);
                    float4 y0 = make_float4(0.f, 0.f, 0.f, 0.f), y1 = y0;
                    if (!first) { y0 = dst[0]; y1 = dst[1]; }
                    y0.x = fmaf(uval, wf[0], y0.x); y0.y = fmaf(uval, wf[1], y0.y);
                    y0.z = fmaf(uval, wf[2], y0.z); y0.w = fmaf(uval, wf[3], y0.w);
                    y1.x = fmaf(uval, wf[4], y1.x); y1.y = fmaf(uval, wf[5], y1.y);
                    y1.z = fmaf(uval, wf[6], y1.z); y1.w = fmaf(uval, wf[7], y1.w);
                    dst[0] = y0; dst[1] = y1;
                }
            }
            c0 += kVB * 32;
            if (c0 >= ncd) break;
#pragma unroll
            for (int u = 0; u < kVB; ++u) {
                const int c = c0 + u * 32 + lane;
                if (c < ncd) vw[u].load(vrow, c); else vw[u].zero();
            }
        }
        first = false;
    }
    __syncthreads();
    p.trace.mark(7);

    // ---- R: sum the warps' copies and add them to global memory -------------------------------------
    const int nused = nact < ncopy ? nact : ncopy;
    if (nused > 0) {
#pragma unroll 1
        for (int i = tid; i < d4; i += kThreads) {
            float4 v = reinterpret_cast<const float4*>(ys)[i];
            for (int w = 1; w < nused; ++w) {
                const float4 o = reinterpret_cast<const float4*>(ys + static_cast<size_t>(w) * d)[i];
                v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
            }
            red_add_v4(p.y + 4 * i, v.x, v.y, v.z, v.w);
        }
    }
    p.trace.mark(8);
}

}  // namespace

namespace spark {

int ffn1_launch(spark_ctx* ctx, FfnParams& p, int wdtype, cudaStream_t stream) {
    static bool configured[3][64] = {};
    if (p.d / 4 > 2 * kThreads) return SPARK_ERR_UNSUPPORTED;    // the input is held in two float4 per thread
    const size_t fixed = (static_cast<size_t>(p.d) + 4 * static_cast<size_t>(p.rpc)) * 4 + 16;
    const size_t limit = static_cast<size_t>(ctx->max_smem_optin - 2048);
    if (fixed + static_cast<size_t>(p.d) * 4 > limit) return SPARK_ERR_UNSUPPORTED;
    size_t ncopy = (limit - fixed) / (static_cast<size_t>(p.d) * 4);
    if (ncopy > 16) ncopy = 16;
    p.ncopy = static_cast<int>(ncopy);
    const size_t smem = fixed + ncopy * p.d * 4;
    if ((p.d / 4 + kThreads - 1) / kThreads > ctx->num_sms) return SPARK_ERR_UNSUPPORTED;
    const void* kern = wdtype == SPARK_BF16 ? reinterpret_cast<const void*>(ffn1_kernel<__nv_bfloat16>)
                     : (wdtype == SPARK_FP8_E4M3 ? reinterpret_cast<const void*>(ffn1_kernel<__nv_fp8_e4m3>)
                                                 : reinterpret_cast<const void*>(ffn1_kernel<float>));
    const int wi = wdtype == SPARK_BF16 ? 1 : (wdtype == SPARK_FP8_E4M3 ? 2 : 0);
    if (ctx->device >= 0 && ctx->device < 64 && !configured[wi][ctx->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin - 1024) != cudaSuccess)
            return SPARK_ERR_CUDA;
        configured[wi][ctx->device] = true;
    }
    p.overlap = ctx->overlap;
    void* args[] = {&p};
    return launch_kernel(ctx, kern, static_cast<unsigned>(ctx->num_sms), kThreads, smem, stream, true, args) == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

}  // namespace spark
