// spark_attn_decode: Spark attention (Section 2.2, Eq. 7) for one new token per sequence, one
// persistent cooperative kernel, one thread block per SM.
//
// The (sequence, KV head, token) space of all windows is laid out flat and cut into equal
// contiguous ranges, one per block, so that the predictor slice of the cache is streamed evenly
// whatever the mix of context lengths.  A range may cross (sequence, KV head) "segments"; the
// intersection of a block's range with one segment is a "piece"; inside a piece every warp owns a
// contiguous run of tokens through both passes.
//
//   pass 1  s_t = k1c[t] . q[:r] for the query heads of the KV group.  Half a warp reads one token
//           row (coalesced 16-byte loads, eight rows in flight per lane); the sixteen partial sums
//           of eight tokens are reduced with a butterfly that leaves one token per lane pair
//           (one shuffle per token and head instead of four).  Scores stay in shared memory; the
//           piece's sum and sum of squares (fp64) go to the (sequence, head) cells, followed by the
//           released arrival.
//   wait    a warp per head polls that head's cells until every piece of the segment has arrived
//           and forms theta (Eq. 11); no grid-wide barrier: only the blocks that share a segment
//           wait for one another.
//   pass 2  every warp selects among its own tokens (ballot), and only for those reads the k2c and
//           vc rows: gate = softplus(k2c[t] . q[r:]), weights exp(s_t - max score) (the cells carry
//           the head's largest score, so every piece uses the same reference), value reduction;
//           the block adds its sum of weights and its weighted values to the head's accumulators
//           with vector reductions; the block that completes a segment last divides.  Inside
//           spark_layer_decode the division is left to the output projection that follows.
#include "kernels.h"

using namespace spark;

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / kWarp;
constexpr int kZc = 4;                // pieces per block whose quantile is cached between the passes
constexpr int kPartPad = 8;           // floats in front of a partial accumulator: [0] max, [1] sum

// FP8 predictor slice on the tensor cores (r = 128, one or two query heads per KV head): a warp takes 16 cached
// rows as the M dimension of mma.m16n8k32 e4m3 tiles -- the stored bytes are the A operand as they are, nothing
// is unpacked -- and the query as four e4m3 terms per head in the eight columns (term i of head h in column
// 4 h + i, scaled by qsc[4 h + i]; each term carries four significant bits, 16 in all).  q8 row stride 160 bytes:
// the 8-byte fragment reads of a half warp fall on distinct banks.
constexpr int kQ8Stride = 160;
// bf16 predictor slice on the tensor cores, for blocks with a long share of the slice (the scalar pass is half issue-bound
// there): 16 cached rows are the M dimension of mma.m16n8k16 bf16 tiles, the query enters as three bf16 terms per head
// (exact to fp32) in columns 4 h .. 4 h + 2.  q16 row stride 320 bytes: the 16-byte fragment reads of a quarter warp fall on
// distinct banks.
constexpr int kQ16Stride = 320;
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_e4m3_16832(float (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned char to_e4m3(float x) { return static_cast<unsigned char>(__nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E4M3)); }
__device__ __forceinline__ float from_e4m3(unsigned char b) { return __half2float(__half(__nv_cvt_fp8_to_halfraw(b, __NV_E4M3))); }

constexpr int kMaxAlignedSegs = 256;   // segment-aligned cut of the token space: at most this many segments ...
constexpr int kMinAlignedSegs = 8;     // ... and at least this many (below, the set-up costs more than it saves)

struct AttnParams {
    const float* q;
    const void* k1c;
    const void* k2c;
    const void* vc;
    int B, n_q, n_kv, hd, r;
    int64_t cap;
    const int32_t* ctx_len;
    const float* k1s;  // nullable: k1c is FP8 E4M3 and k1s[B][n_kv][cap] holds one scale per cached row
    const float* k2s;  // with KT = FP8 E4M3 (k2c and vc quantised too): their row scales, [B][n_kv][cap] each
    const float* vs;
    const double* zs;  // nullable: Q(1 - k_attn / L_b) per sequence, precomputed by an earlier kernel
    int window, k_attn, dense;
    int seg_mask;      // cache segment of (sequence b, KV head g) = (b n_kv + g) & seg_mask: all ones, or n_kv - 1 when the B
                       // queries belong to one sequence and read one cache [n_kv][cap][.] (a chunk of a prompt; n_kv a power of two)
    float* o;
    float* theta;
    int32_t* count;
    int32_t* idx;
    int64_t idx_cap;
    float* scores;     // fallback when a block's scores do not fit in shared memory: [grid][GQ][ntok]
    int ntok;          // capacity (tokens) of a block's score buffer
    int sc_smem;       // 1: scores live in shared memory
    int al_ok;         // host: the even share of a block is short enough for the segment-aligned cut to pay
    int sel_list;      // 1: pass 2 first compacts a piece's survivors into a shared-memory list per head
    SumCell* cells;    // [B * n_q][kAttnWays], zero between launches (the block that merges a segment clears its cells)
    float* lsum;       // [B][n_q] sum of softmax weights per head (o accumulates the weighted values)
    int defer;         // 1: leave o unnormalised and the cells for the next kernel to clear
    PrefetchSpec pf;   // weights of the kernel after this one, asked into L2 once the first predictor rows are in flight
    int check_finite;  // SPARK_CHECK_FINITE: non-finite score sums are reported in the device status
    int long_share;    // 1: a block owns 800 or more tokens of the slice
    int mma_pass;      // 1: bf16 predictor pass on the tensor cores (long shares; r = 128, at most two heads per KV head)
    int pre_stable;    // 1: the kernel directly before this one writes neither ctx_len nor cache rows other than each
                       //    sequence's newest, so lengths and older rows may be read before dep_wait()
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

// MODE 0: flat cut of the token space; 1: segment-aligned cut (the host asks for it when the batch has enough segments);
// 2: flat cut, all queries read one shared cache (a chunk of a prompt).
// K1T: storage of the predictor slice k1c (KT, or FP8 E4M3 with one fp32 scale per cached row in p.k1s).
template <typename KT, typename K1T, int GQ, int MODE, bool M16 = false>
__global__ void __launch_bounds__(kThreads, 1) attn_kernel(const AttnParams p) {
    constexpr bool AL = MODE == 1;      // segment-aligned cut
    constexpr bool SH = MODE == 2;      // one cache shared by all queries (flat cut)
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int NS = p.B * p.n_kv;
    const int hd = p.hd, r = p.r, d2 = hd - r;
    int* segoff = reinterpret_cast<int*>(smem_raw);                       // [NS + 1], padded
    float* qs = reinterpret_cast<float*>(segoff + ((NS + 1 + 3) & ~3));   // [GQ][hd]
    float* wpart = qs + GQ * hd;                                          // [kWarps][hd + kPartPad]
    float* sc_s = wpart + kWarps * (hd + kPartPad);                       // [GQ][ntok] when sc_smem
    int* sel_tok = reinterpret_cast<int*>(sc_s + GQ * p.ntok);            // [GQ][ntok] when sel_list: surviving tokens
    float* sel_a = reinterpret_cast<float*>(sel_tok + GQ * p.ntok);       // [GQ][ntok]              their s - s_max
    __shared__ int sel_n[GQ];
    __shared__ double red[kWarps][GQ][2];
    __shared__ float redm[kWarps][GQ];
    __shared__ float theta_s[GQ], smax_s[GQ];
    __shared__ double zcache[kZc];
    __shared__ double s_z;
    __shared__ int s_last, s_fail, s_aligned;
    __shared__ __align__(16) unsigned char q8[sizeof(K1T) == 1 ? 8 * kQ8Stride : (M16 ? 8 * kQ16Stride : 16)];   // tensor-core pass 1: query terms
    __shared__ float qsc[8];                                                             //   and their scales, per column
    __shared__ int segblk[AL ? kMaxAlignedSegs + 1 : 1];   // first block of every segment (aligned cut)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int half = lane >> 4, hl = lane & 15;
    const int G = gridDim.x, cta = blockIdx.x;
    const int nc1 = r / 8, nc2 = d2 / 8, ncv = hd / 8;
    const int pstride = hd + kPartPad;
    const bool mma8 = sizeof(K1T) == 1 && GQ <= 2 && r == 128;          // FP8 tensor-core pass 1
    constexpr bool mma16 = M16;                                         // bf16 tensor-core pass 1 (the host checks r = 128)
    const int mg = lane >> 2, mt = lane & 3;                            // fragment row group and column pair
    const K1T* k1c = static_cast<const K1T*>(p.k1c);
    const KT* k2c = static_cast<const KT*>(p.k2c);
    const KT* vc = static_cast<const KT*>(p.vc);
    float* sc = p.sc_smem ? sc_s : p.scores + static_cast<size_t>(cta) * GQ * p.ntok;
    const int ntok = p.ntok;

    auto seq_len = [&](int b) -> int {            // valid tokens of sequence b, clamped into [1, cap]
        int n = p.ctx_len[b];
        n = n < 1 ? 1 : n;
        return n > p.cap ? static_cast<int>(p.cap) : n;
    };
    auto win_len = [&](int n) -> int { return (p.window > 0 && p.window < n) ? p.window : n; };
    // cache rows of segment (sequence b, KV head g): sequence b's own cache, or the one cache all queries share
    auto cseg = [&](int seg) -> int64_t { return static_cast<int64_t>(SH ? (seg & p.seg_mask) : seg); };

    if (!p.pre_stable) {   // lengths, queries and cache rows may all come from the kernel before this one
        dep_wait();
        dep_trigger();
    }
    // ---- flat layout: prefix sums of the window lengths over the segments -------------------------
    if (tid == 32) s_fail = 0;
    if constexpr (sizeof(K1T) == 1)
        for (int i = tid; i < 8 * kQ8Stride / 4; i += kThreads) reinterpret_cast<unsigned*>(q8)[i] = 0u;
    if constexpr (M16)
        for (int i = tid; i < 8 * kQ16Stride / 4; i += kThreads) reinterpret_cast<unsigned*>(q8)[i] = 0u;
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
        // Two ways to cut the flat token space.  With a batch (many segments, yet no more than blocks) every
        // segment gets a whole number of blocks in proportion to its length, so that no block works on two
        // segments one after the other: such a block arrives late at both thresholds, holds up every block of
        // both segments and finishes last.  Otherwise: equal flat ranges, which may span segments.  The
        // aligned cut is taken only if every block's share fits the score buffer (sized by the host from the
        // capacity, not from the lengths).
        bool ok = AL && NS >= kMinAlignedSegs && NS <= G && NS <= kMaxAlignedSegs;
        if (AL && ok) {
            __syncwarp();
            const int64_t Tw = run;
            int carry = -(1 << 29);
            for (int s0 = 0; s0 < NS; s0 += 32) {
                const int s = s0 + lane;
                // first block: proportional, at least one block per segment before it, room for those after it
                int key = s < NS ? static_cast<int>(static_cast<int64_t>(G) * segoff[s] / Tw) - s : -(1 << 29);
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(kFull, key, o);
                    if (lane >= o) key = max(key, t);
                }
                key = max(key, carry);
                carry = __shfl_sync(kFull, key, 31);
                if (s < NS) segblk[s] = min(key + s, G - NS + s);
            }
            if (lane == 0) segblk[NS] = G;
            __syncwarp();
            bool fits = true;
            for (int s = lane; s < NS; s += 32) {
                const int nb = segblk[s + 1] - segblk[s], L = segoff[s + 1] - segoff[s];
                fits = fits && (L + nb - 1) / nb <= p.ntok;
            }
            ok = __all_sync(kFull, fits);
        }
        if (AL && lane == 0) s_aligned = ok ? 1 : 0;
    }
    __syncthreads();
    SumCell* cells = p.cells;
    const int64_t T = segoff[NS];
    const bool aligned = AL && s_aligned != 0;
    const int Gp = T < G ? static_cast<int>(T) : G;        // flat cut: blocks that own a non-empty range
    int64_t f0 = 0, f1 = 0;
    int seg0 = 0;
    if (aligned) {
        int lo = 0, hi = NS - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (segblk[mid] <= cta) lo = mid; else hi = mid - 1;
        }
        seg0 = lo;
        const int64_t i = cta - segblk[lo], nb = segblk[lo + 1] - segblk[lo], L = segoff[lo + 1] - segoff[lo];
        f0 = segoff[lo] + L * i / nb;
        f1 = segoff[lo] + L * (i + 1) / nb;
    } else {
        if (cta < Gp) { f0 = T * cta / Gp; f1 = T * (cta + 1) / Gp; }
        int lo = 0, hi = NS - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (segoff[mid] <= f0) lo = mid; else hi = mid - 1;
        }
        seg0 = lo;
    }
    const bool has = f1 > f0;
    // pieces (non-empty block ranges) of a segment: the arrivals its threshold waits for
    auto pieces_of = [&](int seg) -> int {
        if (aligned) {
            const int nb = segblk[seg + 1] - segblk[seg], L = segoff[seg + 1] - segoff[seg];
            return nb < L ? nb : L;
        }
        const int64_t a = segoff[seg], b = static_cast<int64_t>(segoff[seg + 1]) - 1;
        return static_cast<int>(((b + 1) * Gp - 1) / T) - static_cast<int>(((a + 1) * Gp - 1) / T) + 1;
    };
    // tokens of a piece that warp w owns: [w0, w1), runs of a multiple of 16 tokens
    auto warp_range = [&](int tb, int te, int& w0, int& w1) {
        const int n = te - tb;
        const int cw = (((n + kWarps - 1) / kWarps) + 15) & ~15;
        w0 = tb + warp * cw;
        w1 = w0 + cw;
        if (w0 > te) w0 = te;
        if (w1 > te) w1 = te;
    };

    // The first batch of predictor rows is requested before anything else is waited for: before the
    // query is staged and, when the lengths are known to be stable, before the kernel ahead of this one
    // has finished (its newest cache row is held back until it has).
    Row8<K1T> wpre[8];
    [[maybe_unused]] uint4 wq[sizeof(K1T) == 1 ? 4 : 1];      // FP8 tensor-core pass: the first tile's rows, 16-byte pieces
    bool have_pre = false;
    {
        int held = -1;
        const K1T* held_row = nullptr;
        if (has) {
            const int sb = segoff[seg0], se = segoff[seg0 + 1], L = se - sb;
            const int tb = static_cast<int>(f0 - sb);
            const int te = static_cast<int>((f1 < se ? f1 : se) - sb);
            const int lo = seq_len(seg0 / p.n_kv) - L;
            const K1T* kbase = k1c + (cseg(seg0) * p.cap + lo) * r;
            int w0, w1;
            warp_range(tb, te, w0, w1);
            if (w0 < w1 && mma8) {          // rows w0 + mg and w0 + mg + 8, their 16-byte pieces mt and mt + 4
#pragma unroll
                for (int hrow = 0; hrow < 2; ++hrow) {
                    const int t = w0 + mg + 8 * hrow;
#pragma unroll
                    for (int j = 0; j < 2; ++j)
                        wq[2 * hrow + j] = t < w1 ? ld_stream16(reinterpret_cast<const uint4*>(kbase + static_cast<int64_t>(t) * r) + mt + 4 * j)
                                                  : make_uint4(0u, 0u, 0u, 0u);
                }
                have_pre = true;
            } else if (w0 < w1 && !mma16) {
                const int tok0 = w0 + half * 8;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int t = tok0 + j;
                    const bool newest = p.pre_stable && t == L - 1;
                    if (t < w1 && hl < nc1 && !newest) wpre[j].load(kbase + static_cast<int64_t>(t) * r, hl);
                    else wpre[j].zero();
                    if (newest && t < w1 && hl < nc1) { held = j; held_row = kbase + static_cast<int64_t>(t) * r; }
                }
                have_pre = true;
            }
        }
        if (tid == kThreads - 1) prefetch_l2_share(p.pf, cta, G);
        if (p.pre_stable) {
            dep_wait();
            dep_trigger();
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (j == held) wpre[j].load(held_row, hl);
        }
    }
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
            const int off = static_cast<int>(f - f0) - tb;           // score slot of token t: off + t
            for (int i = tid; i < GQ * hd; i += kThreads) qs[i] = p.q[(static_cast<int64_t>(b) * p.n_q + g * GQ) * hd + i];
            if (tb == 0 && p.count != nullptr && tid < GQ) p.count[b * p.n_q + g * GQ + tid] = 0;
            if (tb == 0) {      // the segment's first piece clears the heads' accumulators before it arrives
                float* ob = p.o + (static_cast<int64_t>(b) * p.n_q + g * GQ) * hd;
                for (int i = tid; i < GQ * hd; i += kThreads) ob[i] = 0.f;
                if (tid < GQ) p.lsum[b * p.n_q + g * GQ + tid] = 0.f;
            }
            if (tid == kThreads - 1 && ord < kZc)
                zcache[ord] = p.k_attn >= L ? 0.0
                              : (p.zs != nullptr ? p.zs[b] : -normcdfinv(static_cast<double>(p.k_attn) / static_cast<double>(L)));
            __syncthreads();
            if constexpr (sizeof(K1T) == 1) {
                if (mma8) {
                    // The query as four e4m3 terms per head: term i holds what the terms before it left, at a scale 16
                    // times finer (an e4m3 value carries four significant bits).  A warp per head, four values per lane.
                    if (warp < GQ) {
                        float v[4], amax = 0.f;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            v[e] = qs[warp * hd + lane * 4 + e];
                            amax = fmaxf(amax, fabsf(v[e]));
                        }
                        amax = warp_max(amax);
                        float scale = amax > 0.f ? amax * (1.f / 448.f) : 1.f;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float inv = 1.f / scale;
                            unsigned packed = 0u;
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const unsigned char code = to_e4m3(v[e] * inv);
                                v[e] -= scale * from_e4m3(code);
                                packed |= static_cast<unsigned>(code) << (8 * e);
                            }
                            *reinterpret_cast<unsigned*>(q8 + (4 * warp + i) * kQ8Stride + lane * 4) = packed;
                            if (lane == 0) qsc[4 * warp + i] = scale;
                            scale *= 0.0625f;
                        }
                    }
                    __syncthreads();
                }
            }
            // Heads in groups of at most four: with eight heads per KV head the query fragments and the partial products of all
            // of them at once do not fit the register file (the group's fragments are then re-read from shared memory per step).
            constexpr int HG = GQ > 4 ? 4 : GQ;
            if constexpr (M16) {
                {
                    // The query as three bf16 terms per head (hi + mid + lo = the fp32 value to its last bit but one): a warp per
                    // head, four values per lane, term i of head h in row 4 h + i of q16.
                    if (warp < GQ) {
#pragma unroll
                        for (int i = 0; i < 3; ++i) {
                            unsigned packed[2];
#pragma unroll
                            for (int e2 = 0; e2 < 2; ++e2) {
                                float a = qs[warp * hd + lane * 4 + 2 * e2], b = qs[warp * hd + lane * 4 + 2 * e2 + 1];
                                for (int k = 0; k < i; ++k) {          // what the earlier terms left
                                    a -= __bfloat162float(__float2bfloat16_rn(a));
                                    b -= __bfloat162float(__float2bfloat16_rn(b));
                                }
                                const __nv_bfloat162 hb = __floats2bfloat162_rn(a, b);
                                packed[e2] = *reinterpret_cast<const unsigned*>(&hb);
                            }
                            *reinterpret_cast<uint2*>(q8 + (4 * warp + i) * kQ16Stride + lane * 8) = make_uint2(packed[0], packed[1]);
                        }
                    }
                    __syncthreads();
                }
            }
            float qreg[HG][8];
            if constexpr (GQ <= 4) {
#pragma unroll
                for (int hq = 0; hq < GQ; ++hq)
#pragma unroll
                    for (int e = 0; e < 8; ++e) qreg[hq][e] = hl < nc1 ? qs[hq * hd + hl * 8 + e] : 0.f;
            }
            double s1[GQ], s2[GQ];
            float mx[GQ];
#pragma unroll
            for (int hq = 0; hq < GQ; ++hq) { s1[hq] = 0.0; s2[hq] = 0.0; mx[hq] = -INFINITY; }
            const K1T* kbase = k1c + (cseg(seg) * p.cap + lo) * r;
            int w0, w1;
            warp_range(tb, te, w0, w1);
            const int jidx = ((hl >> 3) & 1) * 4 + ((hl >> 2) & 1) * 2 + ((hl >> 1) & 1);
            if (mma8) {
                const int myh = mt >> 1;                                  // the head whose terms this lane's two columns hold
                const bool owner = (mt & 1) == 0 && myh < GQ;              // ... and the lane that ends up with its scores
                const float c0 = qsc[2 * mt], c1 = qsc[2 * mt + 1];
                double t1 = 0.0, t2 = 0.0;
                float tm = -INFINITY;
#pragma unroll 1
                for (int base = w0; base < w1; base += 32) {               // two 16-row tiles per trip: eight 16-byte loads in flight per lane
                    // A lane takes the 16-byte pieces mt and mt + 4 of rows mg and mg + 8: the k-slots of an MMA may be any
                    // permutation of the columns as long as both operands use it, so a piece feeds two MMAs (its two halves).
                    uint4 w[2][4];
                    float rs[2][2];
#pragma unroll
                    for (int nb = 0; nb < 2; ++nb)
#pragma unroll
                        for (int hrow = 0; hrow < 2; ++hrow) {
                            const int t = base + 16 * nb + mg + 8 * hrow;
                            rs[nb][hrow] = (owner && t < w1) ? p.k1s[cseg(seg) * p.cap + lo + t] : 0.f;
#pragma unroll
                            for (int j = 0; j < 2; ++j) {
                                if (nb == 0 && have_pre && ord == 0 && base == w0) w[0][2 * hrow + j] = wq[2 * hrow + j];
                                else w[nb][2 * hrow + j] = t < w1 ? ld_stream16(reinterpret_cast<const uint4*>(kbase + static_cast<int64_t>(t) * r) + mt + 4 * j)
                                                                  : make_uint4(0u, 0u, 0u, 0u);
                            }
                        }
#pragma unroll
                    for (int nb = 0; nb < 2; ++nb) {
                        float dd[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const uint4 qb = *reinterpret_cast<const uint4*>(q8 + mg * kQ8Stride + 16 * (mt + 4 * j));
                            const uint4 a_lo = w[nb][j], a_hi = w[nb][2 + j];
                            mma_e4m3_16832(dd, a_lo.x, a_hi.x, a_lo.y, a_hi.y, qb.x, qb.y);
                            mma_e4m3_16832(dd, a_lo.z, a_hi.z, a_lo.w, a_hi.w, qb.z, qb.w);
                        }
                        float sa = c0 * dd[0] + c1 * dd[1], sb2 = c0 * dd[2] + c1 * dd[3];
                        sa += __shfl_xor_sync(kFull, sa, 1);
                        sb2 += __shfl_xor_sync(kFull, sb2, 1);
                        if (owner) {
                            const int ta = base + 16 * nb + mg, tb2 = ta + 8;
                            if (ta < w1) {
                                const float v32 = sa * rs[nb][0];
                                sc[static_cast<size_t>(myh) * ntok + off + ta] = v32;
                                const double v = static_cast<double>(v32);
                                t1 += v; t2 = fma(v, v, t2); tm = fmaxf(tm, v32);
                            }
                            if (tb2 < w1) {
                                const float v32 = sb2 * rs[nb][1];
                                sc[static_cast<size_t>(myh) * ntok + off + tb2] = v32;
                                const double v = static_cast<double>(v32);
                                t1 += v; t2 = fma(v, v, t2); tm = fmaxf(tm, v32);
                            }
                        }
                    }
                }
                // sums over the eight row groups (lane bits 2..4); lanes with mg == 0 hold a head's totals
#pragma unroll
                for (int o = 4; o < 32; o <<= 1) {
                    t1 += __shfl_xor_sync(kFull, t1, o);
                    t2 += __shfl_xor_sync(kFull, t2, o);
                    tm = fmaxf(tm, __shfl_xor_sync(kFull, tm, o));
                }
                if (owner && mg == 0) { red[warp][myh][0] = t1; red[warp][myh][1] = t2; redm[warp][myh] = tm; }
            } else if constexpr (M16) {
                {
                    const int myh = mt >> 1;                                  // the head whose terms this lane's two columns hold
                    const bool owner = (mt & 1) == 0 && myh < GQ;              // ... and the lane that ends up with its scores
                    double t1 = 0.0, t2 = 0.0;
                    float tm = -INFINITY;
#pragma unroll 1
                    for (int base = w0; base < w1; base += 16) {               // a 16-row tile per trip: eight 16-byte loads in flight per lane
                        // A lane takes the 16-byte pieces mt, mt + 4, mt + 8, mt + 12 of rows mg and mg + 8: the k-slots of an MMA
                        // may be any permutation of the columns as long as both operands use it, so a piece feeds two MMAs.
                        uint4 w[2][4];
#pragma unroll
                        for (int hrow = 0; hrow < 2; ++hrow) {
                            const int t = base + mg + 8 * hrow;
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                w[hrow][j] = t < w1 ? ld_stream16(reinterpret_cast<const uint4*>(kbase + static_cast<int64_t>(t) * r) + mt + 4 * j)
                                                    : make_uint4(0u, 0u, 0u, 0u);
                        }
                        float dd[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint4 qb = *reinterpret_cast<const uint4*>(q8 + mg * kQ16Stride + 16 * (mt + 4 * j));
                            mma_bf16_16816(dd, w[0][j].x, w[1][j].x, w[0][j].y, w[1][j].y, qb.x, qb.y);
                            mma_bf16_16816(dd, w[0][j].z, w[1][j].z, w[0][j].w, w[1][j].w, qb.z, qb.w);
                        }
                        float sa = dd[0] + dd[1], sb2 = dd[2] + dd[3];       // the head's four columns sit in this lane and its neighbour
                        sa += __shfl_xor_sync(kFull, sa, 1);
                        sb2 += __shfl_xor_sync(kFull, sb2, 1);
                        if (owner) {
                            const int ta = base + mg, tb2 = ta + 8;
                            if (ta < w1) {
                                sc[static_cast<size_t>(myh) * ntok + off + ta] = sa;
                                const double v = static_cast<double>(sa);
                                t1 += v; t2 = fma(v, v, t2); tm = fmaxf(tm, sa);
                            }
                            if (tb2 < w1) {
                                sc[static_cast<size_t>(myh) * ntok + off + tb2] = sb2;
                                const double v = static_cast<double>(sb2);
                                t1 += v; t2 = fma(v, v, t2); tm = fmaxf(tm, sb2);
                            }
                        }
                    }
                    // sums over the eight row groups (lane bits 2..4); lanes with mg == 0 hold a head's totals
#pragma unroll
                    for (int o = 4; o < 32; o <<= 1) {
                        t1 += __shfl_xor_sync(kFull, t1, o);
                        t2 += __shfl_xor_sync(kFull, t2, o);
                        tm = fmaxf(tm, __shfl_xor_sync(kFull, tm, o));
                    }
                    if (owner && mg == 0) { red[warp][myh][0] = t1; red[warp][myh][1] = t2; redm[warp][myh] = tm; }
                }
            } else {
#pragma unroll 1
            for (int base = w0; base < w1; base += 16) {
                const int tok0 = base + half * 8;
                Row8<K1T> w[8];
                // the scale of the row whose score this lane ends up with (FP8 predictor slice), requested with the rows
                [[maybe_unused]] float ksc = 1.f;
                if constexpr (sizeof(K1T) == 1) {
                    const int tsc = tok0 + jidx;
                    if ((hl & 1) == 0 && tsc < w1) ksc = p.k1s[cseg(seg) * p.cap + lo + tsc];
                }
                if (have_pre && ord == 0 && base == w0) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) w[j] = wpre[j];
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        if (tok0 + j < w1 && hl < nc1) w[j].load(kbase + static_cast<int64_t>(tok0 + j) * r, hl);
                        else w[j].zero();
                    }
                }
                const bool b8 = hl & 8, b4 = hl & 4, b2 = hl & 2;
                const int t = tok0 + jidx;
#pragma unroll
                for (int h0 = 0; h0 < GQ; h0 += HG) {
                    if constexpr (GQ > 4) {
#pragma unroll
                        for (int hq = 0; hq < HG; ++hq)
#pragma unroll
                            for (int e = 0; e < 8; ++e) qreg[hq][e] = hl < nc1 ? qs[(h0 + hq) * hd + hl * 8 + e] : 0.f;
                    }
                    float pj[8][HG];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float wf[8];
                        w[j].unpack(wf);
#pragma unroll
                        for (int hq = 0; hq < HG; ++hq) pj[j][hq] = dot8r(wf, qreg[hq]);
                    }
                    // butterfly over the 16 lanes of the half-warp: 8 tokens -> 4 -> 2 -> 1 per lane
                    float a4[4][HG], a2[2][HG], a1[HG];
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj)
#pragma unroll
                        for (int hq = 0; hq < HG; ++hq) {
                            const float keep = b8 ? pj[jj + 4][hq] : pj[jj][hq];
                            const float send = b8 ? pj[jj][hq] : pj[jj + 4][hq];
                            a4[jj][hq] = keep + __shfl_xor_sync(kFull, send, 8);
                        }
#pragma unroll
                    for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                        for (int hq = 0; hq < HG; ++hq) {
                            const float keep = b4 ? a4[jj + 2][hq] : a4[jj][hq];
                            const float send = b4 ? a4[jj][hq] : a4[jj + 2][hq];
                            a2[jj][hq] = keep + __shfl_xor_sync(kFull, send, 4);
                        }
#pragma unroll
                    for (int hq = 0; hq < HG; ++hq) {
                        const float keep = b2 ? a2[1][hq] : a2[0][hq];
                        const float send = b2 ? a2[0][hq] : a2[1][hq];
                        a1[hq] = keep + __shfl_xor_sync(kFull, send, 2);
                        a1[hq] += __shfl_xor_sync(kFull, a1[hq], 1);
                        if constexpr (sizeof(K1T) == 1) a1[hq] *= ksc;
                    }
                    if ((hl & 1) == 0 && t < w1) {
#pragma unroll
                        for (int hq = 0; hq < HG; ++hq) {
                            sc[static_cast<size_t>(h0 + hq) * ntok + off + t] = a1[hq];
                            const double v = static_cast<double>(a1[hq]);
                            s1[h0 + hq] += v;
                            s2[h0 + hq] = fma(v, v, s2[h0 + hq]);
                            mx[h0 + hq] = fmaxf(mx[h0 + hq], a1[hq]);
                        }
                    }
                }
            }
#pragma unroll
            for (int hq = 0; hq < GQ; ++hq) {
                const double a = warp_sum_f64(s1[hq]), c = warp_sum_f64(s2[hq]);
                const float m = warp_max(mx[hq]);
                if (lane == 0) { red[warp][hq][0] = a; red[warp][hq][1] = c; redm[warp][hq] = m; }
            }
            }
            __syncthreads();
            if (warp < GQ) {
                double a = lane < kWarps ? red[lane][warp][0] : 0.0, c = lane < kWarps ? red[lane][warp][1] : 0.0;
                float m = lane < kWarps ? redm[lane][warp] : -INFINITY;
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) {
                    a += __shfl_xor_sync(kFull, a, o);
                    c += __shfl_xor_sync(kFull, c, o);
                    m = fmaxf(m, __shfl_xor_sync(kFull, m, o));
                }
                if (lane == 0)
                    cells_add_max_w<kAttnWays>(cells + static_cast<size_t>(b * p.n_q + g * GQ + warp) * kAttnWays, cta, a, c, m);
            }
            __syncthreads();
            f = sb + te;
        }
    }
    p.trace.mark(1);

    // =============================== pass 2: select, gather, reduce ================================
    {
        int64_t f = f0;
        for (int seg = seg0, ord = 0; f < f1; ++seg, ++ord) {
            const int sb = segoff[seg], se = segoff[seg + 1], L = se - sb;
            const int tb = static_cast<int>(f - sb);
            const int te = static_cast<int>((f1 < se ? f1 : se) - sb);
            const int b = seg / p.n_kv, g = seg - b * p.n_kv;
            const int lo = seq_len(b) - L;
            const int off = static_cast<int>(f - f0) - tb;
            const bool ident = p.k_attn >= L;
            const int npieces = pieces_of(seg);
            for (int i = tid; i < GQ * hd; i += kThreads) qs[i] = p.q[(static_cast<int64_t>(b) * p.n_q + g * GQ) * hd + i];
            if (tid < GQ) sel_n[tid] = 0;
            if (ord >= kZc && tid == 0)
                s_z = ident ? 0.0 : (p.zs != nullptr ? p.zs[b] : -normcdfinv(static_cast<double>(p.k_attn) / static_cast<double>(L)));
            __syncthreads();
            if (warp < GQ) {        // theta of this head once every piece of the segment has arrived
                double sa, sq;
                float smax;
                const bool ok = cells_wait_max_w<kAttnWays>(cells + static_cast<size_t>(b * p.n_q + g * GQ + warp) * kAttnWays,
                                                            static_cast<unsigned>(npieces), sa, sq, smax, p.hdr);
                if (lane == 0) {
                    if (!ok) s_fail = 1;
                    if (ok && p.check_finite && !(isfinite(sa) && isfinite(sq))) atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_NONFINITE);
                    float th = -INFINITY;
                    if (!ident) {
                        const double z = ord < kZc ? zcache[ord] : s_z;
                        const double n = static_cast<double>(L), mean = sa / n;
                        double var = (sq - sa * mean) / (n - 1.0);
                        var = var > 0.0 ? var : 0.0;
                        th = static_cast<float>(mean + sqrt(var) * z);
                    }
                    theta_s[warp] = th;
                    smax_s[warp] = smax;
                    if (tb == 0 && p.theta != nullptr) p.theta[b * p.n_q + g * GQ + warp] = th;
                }
            }
            __syncthreads();
            if (s_fail) return;
            if (ord == 0) p.trace.mark(2);
            const KT* k2base = k2c + cseg(seg) * p.cap * d2;
            const KT* vbase = vc + cseg(seg) * p.cap * hd;
            // In this pass warp w serves query head w % GQ; the kWarps / GQ warps of a head split the
            // piece's tokens into contiguous runs (multiples of 32 tokens).
            constexpr int NSUB = kWarps / GQ;
            const int hq = warp % GQ, wsub = warp / GQ;
            int w0, w1;
            {
                const int n = te - tb;
                const int cw = (((n + NSUB - 1) / NSUB) + 31) & ~31;
                w0 = tb + wsub * cw;
                w1 = w0 + cw;
                if (w0 > te) w0 = te;
                if (w1 > te) w1 = te;
            }
            const float th = theta_s[hq], smax = smax_s[hq];
            const int bh = b * p.n_q + g * GQ + hq;
            float q2[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) q2[e] = hl < nc2 ? qs[hq * hd + r + hl * 8 + e] : 0.f;
            float l_w = 0.f, acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
            const float* srow = sc + static_cast<size_t>(hq) * ntok + off;
            // the k2c and vc rows of up to four surviving tokens (tk: token inside the window), requested together
            auto gather4 = [&](const int (&tk)[4], const bool (&v)[4], const float (&av)[4]) {
                Row8<KT> kw[2], vw[4];
                [[maybe_unused]] float ksc[2] = {1.f, 1.f}, vsc[4] = {1.f, 1.f, 1.f, 1.f};      // row scales of an FP8 cache
#pragma unroll
                for (int i = 0; i < 2; ++i) {      // half h reads the k2c rows of entries h and h + 2
                    const bool vv = half ? v[1 + 2 * i] : v[2 * i];
                    const int tt = half ? tk[1 + 2 * i] : tk[2 * i];
                    if (vv && hl < nc2) kw[i].load(k2base + static_cast<int64_t>(lo + tt) * d2, hl);
                    else kw[i].zero();
                    if constexpr (sizeof(KT) == 1) ksc[i] = vv ? __ldg(p.k2s + cseg(seg) * p.cap + lo + tt) : 1.f;
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (v[i] && lane < ncv) vw[i].load(vbase + static_cast<int64_t>(lo + tk[i]) * hd, lane);
                    else vw[i].zero();
                    if constexpr (sizeof(KT) == 1) vsc[i] = v[i] ? __ldg(p.vs + cseg(seg) * p.cap + lo + tk[i]) : 1.f;
                }
                float gt[4];
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    float wf[8];
                    kw[i].unpack(wf);
                    const float gate = softplus(sizeof(KT) == 1 ? ksc[i] * half_sum(dot8r(wf, q2)) : half_sum(dot8r(wf, q2)));
                    gt[2 * i] = __shfl_sync(kFull, gate, 0);
                    gt[2 * i + 1] = __shfl_sync(kFull, gate, 16);
                }
                float wt[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float pe = av[i] == -INFINITY ? 0.f : expf(av[i]);
                    l_w += pe;
                    wt[i] = pe * gt[i];         // unselected rows of the dense comparator get weight 0 * gate
                    if constexpr (sizeof(KT) == 1) wt[i] *= vsc[i];
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float fv[8];
                    vw[i].unpack(fv);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e] = fmaf(wt[i], fv[e], acc[e]);
                }
            };
            int* ltok = sel_tok + static_cast<size_t>(hq) * ntok;
            float* la = sel_a + static_cast<size_t>(hq) * ntok;
            bool listed = false;
            if constexpr (M16 || sizeof(K1T) == 1) {
            if (p.sel_list && (M16 || p.long_share)) {
                listed = true;
                // Two sweeps over the warp's scores, four 32-token steps per trip with their loads issued together (a step per
                // trip left every warp waiting on its own chain of load, compare and vote: 0.3 us per step).  The first sweep
                // counts what the warp will list; a single shared-memory atomic reserves that many entries of the head's list.
                int mine = 0;
#pragma unroll 1
                for (int base = w0; base < w1; base += 128) {
                    float sv[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int t = base + 32 * u + lane;
                        sv[u] = t < w1 ? srow[t] : -INFINITY;
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const bool valid = base + 32 * u + lane < w1;
                        mine += __popc(__ballot_sync(kFull, valid && (p.dense || ident || sv[u] > th)));
                    }
                }
                int lpos = 0;
                if (lane == 0 && mine > 0) lpos = atomicAdd(&sel_n[hq], mine);
                lpos = __shfl_sync(kFull, lpos, 0);
#pragma unroll 1
                for (int base = w0; base < w1; base += 128) {
                    float sv[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int t = base + 32 * u + lane;
                        sv[u] = t < w1 ? srow[t] : 0.f;
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int t = base + 32 * u + lane;
                        const bool valid = t < w1;
                        const float s = sv[u];
                        const bool sel = valid && (ident || s > th);
                        const float a = sel ? s - smax : -INFINITY;        // softmax is shift-invariant: the head's largest score is the reference
                        const unsigned bsel = __ballot_sync(kFull, sel);
                        const unsigned bal = p.dense ? __ballot_sync(kFull, valid) : bsel;
                        if (p.count != nullptr && bsel != 0u) {
                            int cbase = 0;
                            if (lane == 0) cbase = atomicAdd(&p.count[bh], __popc(bsel));
                            cbase = __shfl_sync(kFull, cbase, 0);
                            if (sel && p.idx != nullptr) {
                                const int64_t pos = static_cast<int64_t>(cbase) + __popc(bsel & ((1u << lane) - 1u));
                                if (pos < p.idx_cap) p.idx[static_cast<int64_t>(bh) * p.idx_cap + pos] = lo + t;
                                else atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_OVERFLOW);
                            }
                        }
                        // The survivors of the whole piece go to one list per head, from which the head's warps then take four
                        // entries each: a warp that found many does not make the block wait for a second round of loads while
                        // others found none.
                        if ((bal >> lane) & 1u) {
                            const int pos = lpos + __popc(bal & ((1u << lane) - 1u));
                            ltok[pos] = t;
                            la[pos] = a;
                        }
                        lpos += __popc(bal);
                    }
                }
            }
            }
            if (!listed) {
#pragma unroll 1
            for (int base = w0; base < w1; base += 32) {
                const int t = base + lane;
                const bool valid = t < w1;
                const float s = valid ? srow[t] : 0.f;
                const bool sel = valid && (ident || s > th);
                const float a = sel ? s - smax : -INFINITY;        // softmax is shift-invariant: the head's largest score is the reference
                const unsigned bsel = __ballot_sync(kFull, sel);
                unsigned bal = p.dense ? __ballot_sync(kFull, valid) : bsel;
                if (p.count != nullptr && bsel != 0u) {
                    int cbase = 0;
                    if (lane == 0) cbase = atomicAdd(&p.count[bh], __popc(bsel));
                    cbase = __shfl_sync(kFull, cbase, 0);
                    if (sel && p.idx != nullptr) {
                        const int64_t pos = static_cast<int64_t>(cbase) + __popc(bsel & ((1u << lane) - 1u));
                        if (pos < p.idx_cap) p.idx[static_cast<int64_t>(bh) * p.idx_cap + pos] = lo + t;
                        else atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_OVERFLOW);
                    }
                }
                if (p.sel_list) {
                    // The survivors of the whole piece go to one list per head, from which the head's warps
                    // then take four entries each: a warp that found many does not make the block wait for a
                    // second round of loads while others found none.
                    if (bal != 0u) {
                        int pos0 = 0;
                        if (lane == 0) pos0 = atomicAdd(&sel_n[hq], __popc(bal));
                        pos0 = __shfl_sync(kFull, pos0, 0);
                        if ((bal >> lane) & 1u) {
                            const int pos = pos0 + __popc(bal & ((1u << lane) - 1u));
                            ltok[pos] = t;
                            la[pos] = a;
                        }
                    }
                    continue;
                }
                while (bal != 0u) {          // four listed tokens per trip: their rows are requested together
                    int tk[4];
                    bool v[4];
                    float av[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        v[i] = bal != 0u;
                        const int l = v[i] ? __ffs(bal) - 1 : 0;
                        if (v[i]) bal &= bal - 1u;
                        const float x = __shfl_sync(kFull, a, l);
                        av[i] = v[i] ? x : -INFINITY;
                        tk[i] = base + l;
                    }
                    gather4(tk, v, av);
                }
            }
            }
            if (p.sel_list) {
                __syncthreads();
                const int n = sel_n[hq];
#pragma unroll 1
                for (int e0 = wsub * 4; e0 < n; e0 += NSUB * 4) {
                    int tk[4];
                    bool v[4];
                    float av[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        v[i] = e0 + i < n;
                        tk[i] = v[i] ? ltok[e0 + i] : 0;
                        av[i] = v[i] ? la[e0 + i] : -INFINITY;
                    }
                    gather4(tk, v, av);
                }
            }
            // ---- add the block's sum of weights and weighted values to the heads' accumulators ----------
            {
                float* wp = wpart + warp * pstride;
                if (lane == 0) wp[1] = l_w;
                if (lane < ncv) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) wp[kPartPad + lane * 8 + e] = acc[e];
                }
                __syncthreads();
                for (int i = tid; i < GQ * (hd / 4); i += kThreads) {
                    const int h = i / (hd / 4), d4 = i - h * (hd / 4);
                    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
                    float l = 0.f;
#pragma unroll
                    for (int u = 0; u < NSUB; ++u) {
                        const float* e = wpart + (u * GQ + h) * pstride;
                        const float4 x = *reinterpret_cast<const float4*>(e + kPartPad + d4 * 4);
                        sum.x += x.x; sum.y += x.y; sum.z += x.z; sum.w += x.w;
                        l += e[1];
                    }
                    if (l > 0.f || p.dense) {
                        const int64_t hb = static_cast<int64_t>(b) * p.n_q + g * GQ + h;
                        red_add_v4(p.o + hb * hd + d4 * 4, sum.x, sum.y, sum.z, sum.w);
                        if (d4 == 0) atomicAdd(&p.lsum[hb], l);
                    }
                }
                __syncthreads();
            }
            // ---- the block that completes a segment last divides by the sum of weights -----------------
            if (!p.defer) {
                if (tid == 0) {
                    __threadfence();
                    const unsigned prev = atom_add_acqrel_u32(&p.hdr->seg_done[seg], 1u);
                    const int last = prev == static_cast<unsigned>(npieces - 1);
                    if (last) p.hdr->seg_done[seg] = 0u;
                    s_last = last;
                }
                __syncthreads();
                if (s_last) {
                    for (int i = tid; i < GQ * hd; i += kThreads) {
                        const int h = i / hd;
                        const int64_t hb = static_cast<int64_t>(b) * p.n_q + g * GQ + h;
                        const float l = __ldcg(&p.lsum[hb]);
                        float* od = p.o + hb * hd + (i - h * hd);
                        const float v = __ldcg(od);
                        *od = l > 0.f ? v / l : 0.f;
                    }
                }
            } else if (tid == 0) {
                s_last = 0;
            }
            __syncthreads();
            // every piece of the segment has read the cells by now: leave them zero for the next launch
            if (s_last && tid < GQ * kAttnWays) {
                SumCell* c = cells + static_cast<size_t>(b * p.n_q + g * GQ) * kAttnWays + tid;
                c->s1 = 0.0; c->s2 = 0.0; c->count = 0u; c->pad[0] = 0u;
            }
            __syncthreads();
            f = sb + te;
        }
    }
    p.trace.mark(3);
}

template <typename KT, typename K1T, int GQ, int MODE, bool M16 = false>
int launch_al(spark_ctx* ctx, AttnParams& p, size_t smem, cudaStream_t stream) {
    static bool configured[64] = {};
    auto kern = attn_kernel<KT, K1T, GQ, MODE, M16>;
    if (ctx->device >= 0 && ctx->device < 64 && !configured[ctx->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin - 8192) != cudaSuccess)
            return SPARK_ERR_CUDA;
        configured[ctx->device] = true;
    }
    void* args[] = {&p};
    return launch_kernel(ctx, reinterpret_cast<const void*>(kern), static_cast<unsigned>(ctx->num_sms), kThreads, smem, stream, true, args) == cudaSuccess
               ? SPARK_OK : SPARK_ERR_CUDA;
}

template <typename KT, typename K1T, int GQ>
int launch_one(spark_ctx* ctx, AttnParams& p, size_t smem, cudaStream_t stream) {
    // The aligned cut removes the blocks that work on two segments in turn (about one pass-2 round, 5-6 us) but
    // gives the segments 1/(blocks per segment) uneven shares of the streaming pass: worth it while a block's
    // share of that pass is short.
    const int ns = p.B * p.n_kv;
    const bool aligned = p.al_ok && ns >= kMinAlignedSegs && ns <= ctx->num_sms && ns <= kMaxAlignedSegs;
    if constexpr (sizeof(KT) == 2 && sizeof(K1T) == 2 && GQ <= 2) {      // long shares: the predictor pass on the tensor cores
        if (p.mma_pass && p.r == 128) {
            if (p.seg_mask != -1) return launch_al<KT, K1T, GQ, 2, true>(ctx, p, smem, stream);
            if (aligned) return launch_al<KT, K1T, GQ, 1, true>(ctx, p, smem, stream);
            return launch_al<KT, K1T, GQ, 0, true>(ctx, p, smem, stream);
        }
    }
    if (p.seg_mask != -1) return launch_al<KT, K1T, GQ, 2>(ctx, p, smem, stream);
    if (aligned) return launch_al<KT, K1T, GQ, 1>(ctx, p, smem, stream);
    return launch_al<KT, K1T, GQ, 0>(ctx, p, smem, stream);
}

template <typename KT, typename K1T>
int launch_gq(spark_ctx* ctx, AttnParams& p, int gq, size_t smem, cudaStream_t stream) {
    switch (gq) {
        case 1: return launch_one<KT, K1T, 1>(ctx, p, smem, stream);
        case 2: return launch_one<KT, K1T, 2>(ctx, p, smem, stream);
        case 4: return launch_one<KT, K1T, 4>(ctx, p, smem, stream);
        case 8: return launch_one<KT, K1T, 8>(ctx, p, smem, stream);
        default: return SPARK_ERR_UNSUPPORTED;
    }
}

}  // namespace

namespace spark {

int attn_launch(spark_ctx* ctx, const float* q, const void* k1c, const void* k2c, const void* vc, int kvdtype, int64_t B,
                int64_t n_q, int64_t n_kv, int64_t hd, int64_t r, int64_t cap, const int32_t* ctx_len, const double* zs,
                int64_t window, int64_t k_attn, int flags, float* o, float* lsum, float* theta, int32_t* count, int32_t* idx,
                int64_t idx_cap, const float* k1s, cudaStream_t st, PrefetchSpec pf, const float* k2s, const float* vs) {
    if (ctx == nullptr || q == nullptr || k1c == nullptr || k2c == nullptr || vc == nullptr || ctx_len == nullptr ||
        o == nullptr)
        return SPARK_ERR_INVALID_ARG;
    if (B < 1 || n_q < 1 || n_kv < 1 || n_q % n_kv != 0 || hd < 16 || r <= 0 || r >= hd || cap < 1 || window < 0 ||
        k_attn <= 0)
        return SPARK_ERR_INVALID_ARG;
    if (idx != nullptr && (count == nullptr || idx_cap < 1)) return SPARK_ERR_INVALID_ARG;
    if (kvdtype != SPARK_F32 && kvdtype != SPARK_BF16) return SPARK_ERR_UNSUPPORTED;
    if (k1s != nullptr && kvdtype != SPARK_BF16) return SPARK_ERR_UNSUPPORTED;      // FP8 predictor slice: beside bf16 k2c / vc
    const int64_t gq = n_q / n_kv;
    if (hd > 256 || (r & 7) != 0 || ((hd - r) & 7) != 0 || r > 128 || hd - r > 128) return SPARK_ERR_UNSUPPORTED;
    if (gq != 1 && gq != 2 && gq != 4 && gq != 8) return SPARK_ERR_UNSUPPORTED;
    if (B * n_kv > kMaxSegments || B * n_kv * cap >= (1LL << 31) || B * n_q * cap >= (1LL << 40)) return SPARK_ERR_UNSUPPORTED;
    if (!aligned16(q) || !aligned16(k1c) || !aligned16(k2c) || !aligned16(vc) || !aligned16(o)) return SPARK_ERR_UNSUPPORTED;
    if (!on_device(ctx)) return SPARK_ERR_INVALID_ARG;

    if ((flags & SPARK_SHARED_CACHE) && !(flags & SPARK_DENSE_LOADS) && B >= 16 && kvdtype == SPARK_BF16 && k1s == nullptr && idx == nullptr) {
        // a chunk of a prompt: the predictor scores of all its queries as one GEMM per KV head (measured: pays from
        // about 16 tokens on; shorter chunks stream the slice per query out of L2 as fast)
        const int rc = attn_chunk_launch(ctx, q, k1c, k2c, vc, B, n_q, n_kv, hd, r, cap, ctx_len, zs, window, k_attn, o, lsum, theta, count, st);
        if (rc != SPARK_ERR_WORKSPACE) return rc;
    }
    const int grid = ctx->num_sms;
    const int64_t span = (window > 0 && window < cap) ? window : cap;          // longest window of a sequence
    int64_t ntok = (B * n_kv * span + grid - 1) / grid + 1;                  // tokens one block may own (equal flat ranges)
    // The cells keep a fixed place and size in the workspace whatever the call's shape: they must be
    // zero between launches, so nothing else may ever be written there.
    const size_t cells_b = kAttnCellBytes;
    if (static_cast<size_t>(B * n_q) * kAttnWays * sizeof(SumCell) > cells_b) return SPARK_ERR_UNSUPPORTED;
    const size_t part_b = round_up(static_cast<size_t>(B * n_q) * 4, 256);     // sums of weights (standalone calls)
    const size_t ns_pad = (static_cast<size_t>(B * n_kv) + 1 + 3) & ~static_cast<size_t>(3);
    const size_t smem_fixed = ns_pad * 4 + static_cast<size_t>(gq * hd) * 4 + static_cast<size_t>(kWarps) * (hd + kPartPad) * 4;
    const size_t smem_limit = static_cast<size_t>(ctx->max_smem_optin - 8192);
    if (smem_fixed > smem_limit) return SPARK_ERR_UNSUPPORTED;
    // room for the segment-aligned cut, whose shares are uneven, when everything still fits shared memory
    const bool al_ok = B * n_kv >= kMinAlignedSegs && ntok <= 6144;    // measured: pays at 3500 tokens a block, a tie at 7000
    if (al_ok) {
        const int64_t flat = ntok;
        for (int num : {12, 9, 8, 7}) {      // 2, 1.5, 1.33, 1.17 times the even share
            const int64_t cand = flat * num / 6 + 16;
            if (smem_fixed + 3 * static_cast<size_t>(gq) * cand * 4 <= smem_limit) {
                ntok = cand;
                break;
            }
        }
    }
    const size_t sc_bytes = static_cast<size_t>(gq) * ntok * 4;
    const bool sc_smem = smem_fixed + sc_bytes <= smem_limit;
    const size_t scores_b = sc_smem ? 0 : round_up(static_cast<size_t>(grid) * sc_bytes, 256);
    if (cells_b + part_b + scores_b > ctx->scratch_bytes) return SPARK_ERR_WORKSPACE;

    AttnParams p;
    p.q = q; p.k1c = k1c; p.k2c = k2c; p.vc = vc;
    p.B = static_cast<int>(B); p.n_q = static_cast<int>(n_q); p.n_kv = static_cast<int>(n_kv);
    p.hd = static_cast<int>(hd); p.r = static_cast<int>(r); p.cap = cap; p.ctx_len = ctx_len; p.zs = zs;
    p.window = static_cast<int>(window > 0x7fffffff ? 0x7fffffff : window);
    p.k_attn = static_cast<int>(k_attn > 0x7fffffff ? 0x7fffffff : k_attn);
    p.dense = (flags & SPARK_DENSE_LOADS) ? 1 : 0;
    p.check_finite = (flags & SPARK_CHECK_FINITE) ? 1 : 0;
    p.pf = pf;
    const bool shared = (flags & SPARK_SHARED_CACHE) != 0;
    if (shared && (n_kv & (n_kv - 1)) != 0) return SPARK_ERR_UNSUPPORTED;
    p.seg_mask = shared ? static_cast<int>(n_kv - 1) : -1;
    p.o = o; p.theta = theta; p.count = count; p.idx = idx; p.idx_cap = idx_cap;
    p.cells = reinterpret_cast<SumCell*>(ctx->scratch);
    p.lsum = lsum != nullptr ? lsum : reinterpret_cast<float*>(ctx->scratch + cells_b);
    p.defer = lsum != nullptr ? 1 : 0;
    // a chunk's rows are all fresh from the kernel ahead; the FP8 tensor-core pass requests its first tile without holding
    // the newest row back, so it waits for the kernel ahead first
    p.pre_stable = p.defer && !shared && k1s == nullptr;
    // measured: the tensor-core pass wins from about 450 tokens a block on (16384 tokens, one sequence: 16.3 -> 15.5 us; eight
    // sequences x 32768: 77.2 -> 71.9) but gives up the rows requested before the kernel ahead has finished, which a layer
    // call of one 9B-shaped sequence (443 tokens a block) still wants: from 800 tokens a block
    p.long_share = ntok >= 800 ? 1 : 0;
    p.mma_pass = (kvdtype == SPARK_BF16 && k1s == nullptr && p.long_share) ? 1 : 0;
    p.scores = reinterpret_cast<float*>(ctx->scratch + cells_b + part_b);
    p.ntok = static_cast<int>(ntok);
    p.sc_smem = sc_smem ? 1 : 0;
    p.al_ok = al_ok ? 1 : 0;
    const bool sel_list = sc_smem && smem_fixed + 3 * sc_bytes <= smem_limit;
    p.sel_list = sel_list ? 1 : 0;
    p.hdr = ctx->hdr;
    p.trace = PhaseTrace{ctx->trace, ctx->trace_cap};
    const size_t smem = smem_fixed + (sel_list ? 3 * sc_bytes : (sc_smem ? sc_bytes : 0));
    p.k1s = k1s; p.k2s = k2s; p.vs = vs;
    if (k2s != nullptr) {          // the whole cache in FP8: predictor slice, gate slice and values
        if (k1s == nullptr || vs == nullptr) return SPARK_ERR_INVALID_ARG;
        return launch_gq<__nv_fp8_e4m3, __nv_fp8_e4m3>(ctx, p, static_cast<int>(gq), smem, st);
    }
    if (k1s != nullptr) return launch_gq<__nv_bfloat16, __nv_fp8_e4m3>(ctx, p, static_cast<int>(gq), smem, st);
    if (kvdtype == SPARK_BF16) return launch_gq<__nv_bfloat16, __nv_bfloat16>(ctx, p, static_cast<int>(gq), smem, st);
    return launch_gq<float, float>(ctx, p, static_cast<int>(gq), smem, st);
}

}  // namespace spark

extern "C" int spark_attn_decode(spark_ctx* ctx, const float* q, const void* k1c, const void* k2c, const void* vc,
                                 int kvdtype, int64_t B, int64_t n_q, int64_t n_kv, int64_t hd, int64_t r,
                                 int64_t cap, const int32_t* ctx_len, int64_t window, int64_t k_attn, int flags,
                                 float* o, float* theta, int32_t* count, int32_t* idx, int64_t idx_cap,
                                 void* stream) {
    return attn_launch(ctx, q, k1c, k2c, vc, kvdtype, B, n_q, n_kv, hd, r, cap, ctx_len, nullptr, window, k_attn, flags, o,
                       nullptr, theta, count, idx, idx_cap, nullptr, static_cast<cudaStream_t>(stream));
}

// The predictor slice of the cache in FP8 E4M3 with one fp32 scale per cached row; k2c and vc stay bf16.
extern "C" int spark_attn_decode_fp8k(spark_ctx* ctx, const float* q, const void* k1c, const float* k1s, const void* k2c,
                                      const void* vc, int64_t B, int64_t n_q, int64_t n_kv, int64_t hd, int64_t r, int64_t cap,
                                      const int32_t* ctx_len, int64_t window, int64_t k_attn, int flags, float* o, float* theta,
                                      int32_t* count, int32_t* idx, int64_t idx_cap, void* stream) {
    if (k1s == nullptr) return SPARK_ERR_INVALID_ARG;
    return attn_launch(ctx, q, k1c, k2c, vc, SPARK_BF16, B, n_q, n_kv, hd, r, cap, ctx_len, nullptr, window, k_attn, flags, o,
                       nullptr, theta, count, idx, idx_cap, k1s, static_cast<cudaStream_t>(stream));
}

// The whole cache in FP8 E4M3 with one fp32 scale per cached row and tensor (k1s, k2s, vs).
extern "C" int spark_attn_decode_fp8kv(spark_ctx* ctx, const float* q, const void* k1c, const float* k1s, const void* k2c, const float* k2s,
                                       const void* vc, const float* vs, int64_t B, int64_t n_q, int64_t n_kv, int64_t hd, int64_t r, int64_t cap,
                                       const int32_t* ctx_len, int64_t window, int64_t k_attn, int flags, float* o, float* theta, int32_t* count,
                                       int32_t* idx, int64_t idx_cap, void* stream) {
    if (k1s == nullptr || k2s == nullptr || vs == nullptr) return SPARK_ERR_INVALID_ARG;
    if (flags & SPARK_SHARED_CACHE) return SPARK_ERR_UNSUPPORTED;
    return attn_launch(ctx, q, k1c, k2c, vc, SPARK_BF16, B, n_q, n_kv, hd, r, cap, ctx_len, nullptr, window, k_attn, flags, o,
                       nullptr, theta, count, idx, idx_cap, k1s, static_cast<cudaStream_t>(stream), PrefetchSpec{nullptr, 0}, k2s, vs);
}
