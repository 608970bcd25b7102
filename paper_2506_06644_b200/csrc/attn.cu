// spark_attn_decode: Spark attention (Section 2.2, Eq. 7) for one new token per sequence, one
// persistent cooperative kernel, one thread block per SM.
//
// The (sequence, KV head, token) space of all windows is laid out flat and cut into equal
// contiguous ranges, one per block, so that the predictor slice of the cache is streamed evenly
// whatever the mix of context lengths.  A range may cross (sequence, KV head) "segments"; the
// intersection of a block's range with one segment is a "piece".
//
//   pass 1  per piece: s_t = k1c[t] . q[:r] for the query heads of the KV group (half a warp per
//           token row, coalesced 16-byte loads), scores to the workspace, per-piece moments;
//   barrier ONE grid-wide barrier (Eq. 11 needs every score of a window);
//   pass 2  per piece and query head: theta from the merged moments, ordered compaction of the
//           selected tokens into shared memory, then only those rows of k2c / vc are read:
//           gate = softplus(k2c[t] . q[r:]), online softmax over the survivors, value reduction;
//           piece partials (max, sum, acc) go to the workspace and the block that finishes a
//           segment last merges its pieces and writes o.
#include "kernels.h"

using namespace spark;

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / kWarp;
constexpr int kHalves = 2 * kWarps;   // half-warps
constexpr int kCH = 2048;             // tokens per selection list
constexpr int kZc = 4;                // pieces per block whose quantile is cached between the passes
constexpr int kPartPad = 8;           // floats in front of a partial accumulator: [0] max, [1] sum

struct AttnParams {
    const float* q;
    const void* k1c;
    const void* k2c;
    const void* vc;
    int B, n_q, n_kv, hd, r;
    int64_t cap;
    const int32_t* ctx_len;
    int window, k_attn, dense;
    float* o;
    float* theta;
    int32_t* count;
    int32_t* idx;
    int64_t idx_cap;
    float* scores;     // [B][n_q][cap]
    float4* pstats;    // [pieces][GQ]
    float* part;       // [pieces][GQ][hd + kPartPad]
    WsHeader* hdr;
    PhaseTrace trace;
};

__device__ __forceinline__ float dot8r(const float (&w)[8], const float (&q)[8]) {
    float a = w[0] * q[0];
#pragma unroll
    for (int e = 1; e < 8; ++e) a = fmaf(w[e], q[e], a);
    return a;
}
__device__ __forceinline__ float half_sum(float v) {   // sum over the 16 lanes of a half-warp
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

// Rank of this thread's flag among the block's flags in thread order, and their total.
__device__ __forceinline__ int block_rank(bool flag, int* wcnt, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned bal = __ballot_sync(kFull, flag);
    if (lane == 0) wcnt[warp] = __popc(bal);
    __syncthreads();
    int before = 0, all = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        if (w < warp) before += wcnt[w];
        all += wcnt[w];
    }
    __syncthreads();
    total = all;
    return before + __popc(bal & ((1u << lane) - 1u));
}

template <typename KT, int GQ>
__global__ void __launch_bounds__(kThreads, 1) attn_kernel(const AttnParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int NS = p.B * p.n_kv;
    const int hd = p.hd, r = p.r, d2 = hd - r;
    int* segoff = reinterpret_cast<int*>(smem_raw);                       // [NS + 1], padded
    float* qs = reinterpret_cast<float*>(segoff + ((NS + 1 + 3) & ~3));   // [GQ][hd]
    int* sel_t = reinterpret_cast<int*>(qs + GQ * hd);                    // [kCH]
    float* sel_a = reinterpret_cast<float*>(sel_t + kCH);                 // [kCH]
    float* wpart = sel_a + kCH;                                           // [kWarps][hd + kPartPad]
    __shared__ float s_mom[kHalves][GQ][3];
    __shared__ float theta_s[GQ];
    __shared__ double zcache[kZc];
    __shared__ double s_z;
    __shared__ int wcnt[kWarps];
    __shared__ int s_base, s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int half = lane >> 4, hl = lane & 15, hw = warp * 2 + half;
    const int G = gridDim.x, cta = blockIdx.x;
    const int nc1 = r / 8, nc2 = d2 / 8, ncv = hd / 8;
    const int pstride = hd + kPartPad;
    const KT* k1c = static_cast<const KT*>(p.k1c);
    const KT* k2c = static_cast<const KT*>(p.k2c);
    const KT* vc = static_cast<const KT*>(p.vc);

    auto seq_len = [&](int b) -> int {            // valid tokens of sequence b, clamped into [1, cap]
        int n = p.ctx_len[b];
        n = n < 1 ? 1 : n;
        return n > p.cap ? static_cast<int>(p.cap) : n;
    };
    auto win_len = [&](int n) -> int { return (p.window > 0 && p.window < n) ? p.window : n; };

    // ---- flat layout: prefix sums of the window lengths over the segments -------------------------
    if (warp == 0) {
        int run = 0;
        for (int s0 = 0; s0 < NS; s0 += 32) {
            const int s = s0 + lane;
            int incl = s < NS ? win_len(seq_len(s / p.n_kv)) : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(kFull, incl, o);
                if (lane >= o) incl += t;
            }
            if (s < NS) segoff[s + 1] = run + incl;
            run += __shfl_sync(kFull, incl, 31);
        }
        if (lane == 0) segoff[0] = 0;
    }
    __syncthreads();
    const int64_t T = segoff[NS];
    const int Gp = T < G ? static_cast<int>(T) : G;        // blocks that own a non-empty range
    const bool has = cta < Gp;
    const int64_t f0 = has ? T * cta / Gp : 0, f1 = has ? T * (cta + 1) / Gp : 0;
    int seg0 = 0;
    {
        int lo = 0, hi = NS - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (segoff[mid] <= f0) lo = mid; else hi = mid - 1;
        }
        seg0 = lo;
    }
    auto cta_of = [&](int64_t f) -> int { return static_cast<int>(((f + 1) * Gp - 1) / T); };

    GridBarrier bar{p.hdr, static_cast<unsigned>(G), 0u, 0u};
    bar.begin();
    p.trace.mark(0);

    // =============================== pass 1: predictor scores =====================================
    {
        int64_t f = f0;
        for (int seg = seg0, ord = 0; f < f1; ++seg, ++ord) {
            const int sb = segoff[seg], se = segoff[seg + 1], L = se - sb;
            const int tb = static_cast<int>(f - sb);
            const int te = static_cast<int>((f1 < se ? f1 : se) - sb);
            const int b = seg / p.n_kv, g = seg - b * p.n_kv;
            const int lo = seq_len(b) - L;
            for (int i = tid; i < GQ * hd; i += kThreads) qs[i] = p.q[(static_cast<int64_t>(b) * p.n_q + g * GQ) * hd + i];
            if (tb == 0 && p.count != nullptr && tid < GQ) p.count[b * p.n_q + g * GQ + tid] = 0;
            if (tid == kThreads - 1 && ord < kZc)
                zcache[ord] = p.k_attn >= L ? 0.0 : -normcdfinv(static_cast<double>(p.k_attn) / static_cast<double>(L));
            __syncthreads();
            float qreg[GQ][8];
#pragma unroll
            for (int hq = 0; hq < GQ; ++hq)
#pragma unroll
                for (int e = 0; e < 8; ++e) qreg[hq][e] = hl < nc1 ? qs[hq * hd + hl * 8 + e] : 0.f;
            float wn = 0.f, wmean[GQ], wm2[GQ];
#pragma unroll
            for (int hq = 0; hq < GQ; ++hq) { wmean[hq] = 0.f; wm2[hq] = 0.f; }
            const KT* kbase = k1c + (static_cast<int64_t>(seg) * p.cap + lo) * r;
            float* sbase = p.scores + (static_cast<int64_t>(b) * p.n_q + g * GQ) * p.cap + lo;
            for (int ib = tb + warp * 2; ib < te; ib += kHalves * 4) {   // warp-uniform trip count
                const int i0 = ib + half;
                Row8<KT> w[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + u * kHalves;
                    if (i < te && hl < nc1) w[u].load(kbase + static_cast<int64_t>(i) * r, hl);
                    else w[u].zero();
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + u * kHalves;
                    float wf[8];
                    w[u].unpack(wf);
                    float sc[GQ];
#pragma unroll
                    for (int hq = 0; hq < GQ; ++hq) sc[hq] = half_sum(dot8r(wf, qreg[hq]));
                    if (hl == 0 && i < te) {
                        wn += 1.f;
                        const float inv = 1.f / wn;
#pragma unroll
                        for (int hq = 0; hq < GQ; ++hq) {
                            sbase[static_cast<int64_t>(hq) * p.cap + i] = sc[hq];
                            const float dl = sc[hq] - wmean[hq];
                            wmean[hq] += dl * inv;
                            wm2[hq] = fmaf(dl, sc[hq] - wmean[hq], wm2[hq]);
                        }
                    }
                }
            }
            if (hl == 0) {
#pragma unroll
                for (int hq = 0; hq < GQ; ++hq) {
                    s_mom[hw][hq][0] = wn; s_mom[hw][hq][1] = wmean[hq]; s_mom[hw][hq][2] = wm2[hq];
                }
            }
            __syncthreads();
            if (warp < GQ) {
                Moments m{static_cast<double>(s_mom[lane][warp][0]), static_cast<double>(s_mom[lane][warp][1]),
                          static_cast<double>(s_mom[lane][warp][2])};
                m = warp_merge(m);
                if (lane == 0)
                    p.pstats[static_cast<size_t>(cta + seg) * GQ + warp] =
                        make_float4(static_cast<float>(m.n), static_cast<float>(m.mean), static_cast<float>(m.m2), 0.f);
            }
            __syncthreads();
            f = sb + te;
        }
    }
    p.trace.mark(1);
    bar.arrive();
    if (!bar.wait()) return;
    p.trace.mark(2);

    // =============================== pass 2: select, gather, reduce ================================
    {
        int64_t f = f0;
        for (int seg = seg0, ord = 0; f < f1; ++seg, ++ord) {
            const int sb = segoff[seg], se = segoff[seg + 1], L = se - sb;
            const int tb = static_cast<int>(f - sb);
            const int te = static_cast<int>((f1 < se ? f1 : se) - sb);
            const int b = seg / p.n_kv, g = seg - b * p.n_kv;
            const int lo = seq_len(b) - L;
            const bool ident = p.k_attn >= L;
            const int c_lo = cta_of(sb), c_hi = cta_of(static_cast<int64_t>(se) - 1);
            const size_t pid = static_cast<size_t>(cta + seg);
            for (int i = tid; i < GQ * hd; i += kThreads) qs[i] = p.q[(static_cast<int64_t>(b) * p.n_q + g * GQ) * hd + i];
            if (ord >= kZc && tid == 0)
                s_z = ident ? 0.0 : -normcdfinv(static_cast<double>(p.k_attn) / static_cast<double>(L));
            __syncthreads();
            if (warp < GQ) {
                Moments m{0.0, 0.0, 0.0};
                for (int c = c_lo + lane; c <= c_hi; c += 32) {
                    const float4 v = ld_cg_f4(&p.pstats[static_cast<size_t>(c + seg) * GQ + warp]);
                    m = merge(m, Moments{static_cast<double>(v.x), static_cast<double>(v.y), static_cast<double>(v.z)});
                }
                m = warp_merge(m);
                const double z = ord < kZc ? zcache[ord] : s_z;
                const float th = ident ? -INFINITY : theta_from(m, z);
                if (lane == 0) {
                    theta_s[warp] = th;
                    if (tb == 0 && p.theta != nullptr) p.theta[b * p.n_q + g * GQ + warp] = th;
                }
            }
            __syncthreads();
            const KT* k2base = k2c + static_cast<int64_t>(seg) * p.cap * d2;
            const KT* vbase = vc + static_cast<int64_t>(seg) * p.cap * hd;

#pragma unroll 1
            for (int hq = 0; hq < GQ; ++hq) {
                const float th = theta_s[hq];
                const int bh = b * p.n_q + g * GQ + hq;
                float q2[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) q2[e] = hl < nc2 ? qs[hq * hd + r + hl * 8 + e] : 0.f;
                float m_w = -INFINITY, l_w = 0.f, acc[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = 0.f;
                const float* srow = p.scores + static_cast<int64_t>(bh) * p.cap + lo;

                for (int c0 = tb; c0 < te; c0 += kCH) {
                    const int c1 = te < c0 + kCH ? te : c0 + kCH;
                    int nlist = 0;
                    for (int j0 = c0; j0 < c1; j0 += kThreads) {
                        const int i = j0 + tid;
                        const bool valid = i < c1;
                        const float s = valid ? __ldcg(srow + i) : 0.f;
                        const bool sel = valid && (ident || s > th);
                        const bool in = valid && (sel || p.dense);
                        int tot;
                        const int rank = block_rank(in, wcnt, tot);
                        if (in) {
                            sel_t[nlist + rank] = lo + i;
                            sel_a[nlist + rank] = sel ? (ident ? s : s - th) : -INFINITY;
                        }
                        nlist += tot;
                        if (p.count != nullptr) {
                            int nt;
                            const int rk = p.dense ? block_rank(sel, wcnt, nt) : rank;
                            if (!p.dense) nt = tot;
                            if (nt > 0) {
                                if (tid == 0) s_base = atomicAdd(&p.count[bh], nt);
                                __syncthreads();
                                const int64_t pos = static_cast<int64_t>(s_base) + rk;
                                if (sel && p.idx != nullptr) {
                                    if (pos < p.idx_cap) p.idx[static_cast<int64_t>(bh) * p.idx_cap + pos] = lo + i;
                                    else atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_OVERFLOW);
                                }
                                __syncthreads();
                            }
                        }
                    }
                    __syncthreads();
                    const int npairs = (nlist + 1) >> 1;
                    for (int pi = warp; pi < npairs; pi += kWarps) {
                        const int e0 = 2 * pi, e1 = e0 + 1;
                        const bool v1 = e1 < nlist;
                        const int t0 = sel_t[e0], t1 = v1 ? sel_t[e1] : t0;
                        const float a0 = sel_a[e0], a1 = v1 ? sel_a[e1] : -INFINITY;
                        const int tm = half ? t1 : t0;
                        Row8<KT> kw, v0w, v1w;
                        if ((half == 0 || v1) && hl < nc2) kw.load(k2base + static_cast<int64_t>(tm) * d2, hl);
                        else kw.zero();
                        if (lane < ncv) v0w.load(vbase + static_cast<int64_t>(t0) * hd, lane);
                        else v0w.zero();
                        if (lane < ncv && v1) v1w.load(vbase + static_cast<int64_t>(t1) * hd, lane);
                        else v1w.zero();
                        float wf[8];
                        kw.unpack(wf);
                        const float gate = softplus(half_sum(dot8r(wf, q2)));
                        const float g0 = __shfl_sync(kFull, gate, 0), g1 = __shfl_sync(kFull, gate, 16);
                        const float mn = fmaxf(m_w, fmaxf(a0, a1));
                        if (mn != -INFINITY) {
                            const float sc = m_w == -INFINITY ? 0.f : expf(m_w - mn);
                            const float p0 = a0 == -INFINITY ? 0.f : expf(a0 - mn);
                            const float p1 = a1 == -INFINITY ? 0.f : expf(a1 - mn);
                            l_w = l_w * sc + p0 + p1;
                            const float w0 = p0 * g0, w1 = p1 * g1;
                            float f0v[8], f1v[8];
                            v0w.unpack(f0v);
                            v1w.unpack(f1v);
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[e] = fmaf(w1, f1v[e], fmaf(w0, f0v[e], acc[e] * sc));
                            m_w = mn;
                        } else if (p.dense) {
                            // nothing selected so far: the rows were still read; keep the loads alive
                            float f0v[8], f1v[8];
                            v0w.unpack(f0v);
                            v1w.unpack(f1v);
#pragma unroll
                            for (int e = 0; e < 8; ++e) acc[e] = fmaf(0.f * g0, f0v[e], fmaf(0.f * g1, f1v[e], acc[e]));
                        }
                    }
                    __syncthreads();
                }
                // ---- combine the warps' online-softmax states into the piece partial ---------------
                float* wp = wpart + warp * pstride;
                if (lane == 0) { wp[0] = m_w; wp[1] = l_w; }
                if (lane < ncv) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) wp[kPartPad + lane * 8 + e] = acc[e];
                }
                __syncthreads();
                float M = -INFINITY;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) M = fmaxf(M, wpart[w * pstride]);
                float* dst = p.part + (pid * GQ + hq) * pstride;
                for (int dd = tid; dd < hd; dd += kThreads) {
                    float sum = 0.f;
#pragma unroll
                    for (int w = 0; w < kWarps; ++w) {
                        const float mw = wpart[w * pstride];
                        if (mw != -INFINITY) sum = fmaf(expf(mw - M), wpart[w * pstride + kPartPad + dd], sum);
                    }
                    dst[kPartPad + dd] = sum;
                }
                if (tid == 0) {
                    float l = 0.f;
                    for (int w = 0; w < kWarps; ++w) {
                        const float mw = wpart[w * pstride];
                        if (mw != -INFINITY) l = fmaf(expf(mw - M), wpart[w * pstride + 1], l);
                    }
                    dst[0] = M;
                    dst[1] = l;
                }
                __syncthreads();
            }

            // ---- the block that completes a segment last merges its pieces and writes o -------------
            __threadfence();
            __syncthreads();
            if (tid == 0) {
                const unsigned prev = atom_add_acqrel_u32(&p.hdr->seg_done[seg], 1u);
                const int last = prev == static_cast<unsigned>(c_hi - c_lo);
                if (last) p.hdr->seg_done[seg] = 0u;
                s_last = last;
            }
            __syncthreads();
            if (s_last && warp < GQ) {
                const int hq = warp;
                float M = -INFINITY;
                for (int c = c_lo + lane; c <= c_hi; c += 32)
                    M = fmaxf(M, __ldcg(p.part + (static_cast<size_t>(c + seg) * GQ + hq) * pstride));
                M = warp_max(M);
                float Lsum = 0.f, out[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) out[e] = 0.f;
                for (int c = c_lo; c <= c_hi; ++c) {
                    const float* src = p.part + (static_cast<size_t>(c + seg) * GQ + hq) * pstride;
                    const float mp = __ldcg(src);
                    if (mp == -INFINITY) continue;
                    const float w = expf(mp - M);
                    Lsum = fmaf(w, __ldcg(src + 1), Lsum);
                    if (lane < ncv) {
                        const float4 a = __ldcg(reinterpret_cast<const float4*>(src + kPartPad + lane * 8));
                        const float4 c4 = __ldcg(reinterpret_cast<const float4*>(src + kPartPad + lane * 8 + 4));
                        out[0] = fmaf(w, a.x, out[0]); out[1] = fmaf(w, a.y, out[1]);
                        out[2] = fmaf(w, a.z, out[2]); out[3] = fmaf(w, a.w, out[3]);
                        out[4] = fmaf(w, c4.x, out[4]); out[5] = fmaf(w, c4.y, out[5]);
                        out[6] = fmaf(w, c4.z, out[6]); out[7] = fmaf(w, c4.w, out[7]);
                    }
                }
                const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
                if (lane < ncv) {
                    float* od = p.o + (static_cast<int64_t>(b) * p.n_q + g * GQ + hq) * hd + lane * 8;
                    reinterpret_cast<float4*>(od)[0] = make_float4(out[0] * inv, out[1] * inv, out[2] * inv, out[3] * inv);
                    reinterpret_cast<float4*>(od)[1] = make_float4(out[4] * inv, out[5] * inv, out[6] * inv, out[7] * inv);
                }
            }
            __syncthreads();
            f = sb + te;
        }
    }
    p.trace.mark(3);
}

template <typename KT, int GQ>
int launch_one(spark_ctx* ctx, AttnParams& p, size_t smem, cudaStream_t stream) {
    static bool configured[64] = {};
    auto kern = attn_kernel<KT, GQ>;
    if (ctx->device >= 0 && ctx->device < 64 && !configured[ctx->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin - 8192) != cudaSuccess)
            return SPARK_ERR_CUDA;
        configured[ctx->device] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(ctx->num_sms));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p) == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

template <typename KT>
int launch_gq(spark_ctx* ctx, AttnParams& p, int gq, size_t smem, cudaStream_t stream) {
    switch (gq) {
        case 1: return launch_one<KT, 1>(ctx, p, smem, stream);
        case 2: return launch_one<KT, 2>(ctx, p, smem, stream);
        case 4: return launch_one<KT, 4>(ctx, p, smem, stream);
        case 8: return launch_one<KT, 8>(ctx, p, smem, stream);
        default: return SPARK_ERR_UNSUPPORTED;
    }
}

}  // namespace

extern "C" int spark_attn_decode(spark_ctx* ctx, const float* q, const void* k1c, const void* k2c, const void* vc,
                                 int kvdtype, int64_t B, int64_t n_q, int64_t n_kv, int64_t hd, int64_t r,
                                 int64_t cap, const int32_t* ctx_len, int64_t window, int64_t k_attn, int flags,
                                 float* o, float* theta, int32_t* count, int32_t* idx, int64_t idx_cap,
                                 void* stream) {
    if (ctx == nullptr || q == nullptr || k1c == nullptr || k2c == nullptr || vc == nullptr || ctx_len == nullptr ||
        o == nullptr)
        return SPARK_ERR_INVALID_ARG;
    if (B < 1 || n_q < 1 || n_kv < 1 || n_q % n_kv != 0 || hd < 16 || r <= 0 || r >= hd || cap < 1 || window < 0 ||
        k_attn <= 0)
        return SPARK_ERR_INVALID_ARG;
    if (idx != nullptr && (count == nullptr || idx_cap < 1)) return SPARK_ERR_INVALID_ARG;
    if (kvdtype != SPARK_F32 && kvdtype != SPARK_BF16) return SPARK_ERR_UNSUPPORTED;
    const int64_t gq = n_q / n_kv;
    if (hd > 256 || (r & 7) != 0 || ((hd - r) & 7) != 0 || r > 128 || hd - r > 128) return SPARK_ERR_UNSUPPORTED;
    if (gq != 1 && gq != 2 && gq != 4 && gq != 8) return SPARK_ERR_UNSUPPORTED;
    if (B * n_kv > kMaxSegments || B * n_kv * cap >= (1LL << 31) || B * n_q * cap >= (1LL << 40)) return SPARK_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k1c) || !aligned16(k2c) || !aligned16(vc) || !aligned16(o)) return SPARK_ERR_UNSUPPORTED;
    if (!on_device(ctx)) return SPARK_ERR_INVALID_ARG;

    const int grid = ctx->num_sms;
    const size_t pieces = static_cast<size_t>(grid) + static_cast<size_t>(B * n_kv);
    const size_t scores_b = round_up(static_cast<size_t>(B * n_q * cap) * 4, 256);
    const size_t pstats_b = round_up(pieces * gq * sizeof(float4), 256);
    const size_t part_b = round_up(pieces * gq * (hd + kPartPad) * 4, 256);
    if (scores_b + pstats_b + part_b > ctx->scratch_bytes) return SPARK_ERR_WORKSPACE;

    AttnParams p;
    p.q = q; p.k1c = k1c; p.k2c = k2c; p.vc = vc;
    p.B = static_cast<int>(B); p.n_q = static_cast<int>(n_q); p.n_kv = static_cast<int>(n_kv);
    p.hd = static_cast<int>(hd); p.r = static_cast<int>(r); p.cap = cap; p.ctx_len = ctx_len;
    p.window = static_cast<int>(window > 0x7fffffff ? 0x7fffffff : window);
    p.k_attn = static_cast<int>(k_attn > 0x7fffffff ? 0x7fffffff : k_attn);
    p.dense = (flags & SPARK_DENSE_LOADS) ? 1 : 0;
    p.o = o; p.theta = theta; p.count = count; p.idx = idx; p.idx_cap = idx_cap;
    p.scores = reinterpret_cast<float*>(ctx->scratch);
    p.pstats = reinterpret_cast<float4*>(ctx->scratch + scores_b);
    p.part = reinterpret_cast<float*>(ctx->scratch + scores_b + pstats_b);
    p.hdr = ctx->hdr;
    p.trace = PhaseTrace{ctx->trace, ctx->trace_cap};

    const size_t ns_pad = (static_cast<size_t>(B * n_kv) + 1 + 3) & ~static_cast<size_t>(3);
    const size_t smem = ns_pad * 4 + static_cast<size_t>(gq * hd) * 4 + static_cast<size_t>(kCH) * 8 +
                        static_cast<size_t>(kWarps) * (hd + kPartPad) * 4;
    if (smem > static_cast<size_t>(ctx->max_smem_optin - 8192)) return SPARK_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (kvdtype == SPARK_BF16) return launch_gq<__nv_bfloat16>(ctx, p, static_cast<int>(gq), smem, st);
    return launch_gq<float>(ctx, p, static_cast<int>(gq), smem, st);
}
