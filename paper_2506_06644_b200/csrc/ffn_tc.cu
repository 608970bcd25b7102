// Spark FFN (Section 2.1, Eq. 2) for a chunk of 5..64 tokens with bf16 weights, on the fifth-generation
// tensor cores.  With this many tokens the union of the tokens' active sets (Appendix B) covers most
// neurons, every weight row is read anyway, and the three products are real GEMMs with the tokens as
// the N dimension.  Four kernels, ordered by the stream (no block waits on another block):
//   prep    RMSNorm scale (optional), x -> two bf16 terms (x = hi + lo), y = y_init, sums cleared
//   scores  S^T = K1t . X[:, :r]^T and T^T = K2t . X[:, r:]^T: TMA-fed tcgen05.mma, M = 128 neurons,
//           N = tokens, accumulators in tensor memory; two blocks per 128 neurons split the K range;
//           per-token score sums for Eq. 11 leave with the epilogue
//   act     theta per token (Eq. 10/11), U = [S > theta] . GELU(S - theta) . T as two bf16 terms,
//           counts and index lists
//   out     Y^T += Vt^T . U: M = 128 model columns (Vt enters MN-major, as it is stored), N = tokens,
//           K = neurons split over blocks, fp32 vector reductions into y
// The fp32 activations enter every product as an error-compensated two-term bf16 split (one MMA per
// term): the scores decide index sets, so a bare bf16 rounding (2^-9) is not enough, and the two
// terms carry 16 mantissa bits.  The weight streams are requested before the kernel waits for the
// one ahead of it, so they overlap its tail.
#include "ffn_params.h"
#include "kernels.h"
#include "tc_common.cuh"

using namespace spark;
using namespace spark::tc;

namespace {

constexpr int kTok = 64;              // token rows of the padded operands
constexpr int kSumWays = 16;
constexpr int kMaxTParts = 2;         // blocks that share the K range of the K2 product of one row tile

// ---- layout of the chunk path's part of the workspace ----------------------------------------------
struct TcRegion {
    double* sums;                 // [kSumWays][kTok][2]
    __nv_bfloat16* xhi;           // [kTok][d]
    __nv_bfloat16* xlo;
    float* S;                     // [kTok][d_ff] scores, token-major
    float* T;                     // [kMaxTParts][kTok][d_ff] K2 products, one per K part
    __nv_bfloat16* uhi;           // [kTok][d_ff]
    __nv_bfloat16* ulo;
};
inline size_t tc_region_bytes(int64_t d, int64_t d_ff) {
    return round_up(sizeof(double) * kSumWays * kTok * 2, 1024) + 2 * round_up(static_cast<size_t>(kTok) * d * 2, 1024) +
           (1 + kMaxTParts) * round_up(static_cast<size_t>(kTok) * d_ff * 4, 1024) + 2 * round_up(static_cast<size_t>(kTok) * d_ff * 2, 1024);
}
inline TcRegion tc_region(char* base, int64_t d, int64_t d_ff) {
    TcRegion g;
    char* p = base;
    g.sums = reinterpret_cast<double*>(p); p += round_up(sizeof(double) * kSumWays * kTok * 2, 1024);
    g.xhi = reinterpret_cast<__nv_bfloat16*>(p); p += round_up(static_cast<size_t>(kTok) * d * 2, 1024);
    g.xlo = reinterpret_cast<__nv_bfloat16*>(p); p += round_up(static_cast<size_t>(kTok) * d * 2, 1024);
    g.S = reinterpret_cast<float*>(p); p += round_up(static_cast<size_t>(kTok) * d_ff * 4, 1024);
    g.T = reinterpret_cast<float*>(p); p += kMaxTParts * round_up(static_cast<size_t>(kTok) * d_ff * 4, 1024);
    g.uhi = reinterpret_cast<__nv_bfloat16*>(p); p += round_up(static_cast<size_t>(kTok) * d_ff * 2, 1024);
    g.ulo = reinterpret_cast<__nv_bfloat16*>(p);
    return g;
}

struct TcParams {
    FfnParams f;
    TcRegion g;
    int ntok;            // MMA N: B rounded up to a multiple of 16
    int cs;              // K chunks of the predictor (r / 64)
    int call;            // K chunks of both products (d / 64)
    int chalf;           // chunks of the first block of a pair (it holds all of the predictor's)
    int tfirst;          // first partial K2 product that exists (0, or 1 when the first block has none)
    int ksplit;          // out kernel: blocks per column block
};

// ---- prep: four blocks per (padded) token row, a quarter of the row each -----------------------------------
constexpr int kPrepSplit = 4;
__global__ void __launch_bounds__(256) ffn_tc_prep_kernel(const TcParams p) {
    __shared__ float red[8];
    const int n = blockIdx.x / kPrepSplit, qr = blockIdx.x % kPrepSplit, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d = p.f.d, q4 = d / 4 / kPrepSplit;          // float4 per quarter row (d is a multiple of 256)
    dep_wait();
    dep_trigger();
    if (blockIdx.x == 0) {
        for (int i = tid; i < kSumWays * kTok * 2; i += 256) p.g.sums[i] = 0.0;
        if (p.f.count != nullptr && tid < p.f.B) p.f.count[tid] = 0;
    }
    if (n >= p.ntok) return;       // rows the operand boxes never touch
    uint2* hi = reinterpret_cast<uint2*>(p.g.xhi + static_cast<int64_t>(n) * d) + qr * q4;
    uint2* lo = reinterpret_cast<uint2*>(p.g.xlo + static_cast<int64_t>(n) * d) + qr * q4;
    if (n >= p.f.B) {              // padding rows of the operands
        for (int i = tid; i < q4; i += 256) {
            hi[i] = make_uint2(0u, 0u);
            lo[i] = make_uint2(0u, 0u);
        }
        return;
    }
    const float4* xr = reinterpret_cast<const float4*>(p.f.x + static_cast<int64_t>(n) * d);
    float sc = 1.f;
    if (p.f.norm_w != nullptr) {   // every quarter sums the whole row (9 KB out of L2)
        float ss = 0.f;
        for (int i = tid; i < d / 4; i += 256) {
            const float4 v = xr[i];
            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        ss = warp_sum(ss);
        if (lane == 0) red[warp] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot += red[w];
        sc = rsqrtf(tot / static_cast<float>(d) + p.f.eps);
    }
    for (int i = tid; i < q4; i += 256) {
        float4 v = xr[qr * q4 + i];
        if (p.f.norm_w != nullptr) {
            const float4 w = reinterpret_cast<const float4*>(p.f.norm_w)[qr * q4 + i];
            v = make_float4(v.x * sc * w.x, v.y * sc * w.y, v.z * sc * w.z, v.w * sc * w.w);
        }
        const unsigned h01 = pack2_bf16(v.x, v.y), h23 = pack2_bf16(v.z, v.w);
        const unsigned l01 = pack2_bf16(v.x - __uint_as_float(h01 << 16), v.y - __uint_as_float(h01 & 0xffff0000u));
        const unsigned l23 = pack2_bf16(v.z - __uint_as_float(h23 << 16), v.w - __uint_as_float(h23 & 0xffff0000u));
        hi[i] = make_uint2(h01, h23);
        lo[i] = make_uint2(l01, l23);
    }
}

// ---- scores: S^T and T^T tiles of 128 neurons; the two blocks of a tile split the K range ----------------
// The first block of a pair takes the predictor's chunks (its scores are complete, so their sums can
// leave with the epilogue) and the first chunks of the K2 product, the second block the rest; the
// activation kernel adds the partial products.  Both terms of X sit in one operand tile (hi rows, then
// lo rows), so one MMA of N = 2 ntok serves both and the weight tile is read from shared memory once;
// the epilogue adds the two halves of the accumulator.  (Shared-memory bandwidth -- TMA writes plus
// operand reads -- is what bounds the main loop, not HBM.)
constexpr int kScoreRows = 128;
constexpr int kScoreStages = 6;
constexpr int kScoreWBytes = kScoreRows * kChunk * 2;                           // 16 KB of weights per stage
constexpr int kScoreStageBytes = kScoreWBytes + 2 * kTok * kChunk * 2;          // + x hi, x lo (8 KB each at 64 tokens)
constexpr uint32_t kScoreCols = 256;                                            // S: columns 0..127 (hi | lo), T: 128..255

__global__ void __launch_bounds__(kTcThreads, 1)
ffn_tc_scores_kernel(const TcParams p, const __grid_constant__ CUtensorMap map_k1, const __grid_constant__ CUtensorMap map_k2,
                     const __grid_constant__ CUtensorMap map_xhi, const __grid_constant__ CUtensorMap map_xlo) {
    extern __shared__ unsigned char tc_raw[];
    __shared__ TcShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x >> 1, part = blockIdx.x & 1;
    // chunk range over the combined index (predictor chunks first, then the K2 product's)
    const int c0 = part == 0 ? 0 : p.chalf, c1 = part == 0 ? p.chalf : p.call, nch = c1 - c0;
    const int row0 = tile * kScoreRows;
    const uint32_t xbytes = static_cast<uint32_t>(p.ntok) * kChunk * 2;         // one term of one chunk of X
    const uint32_t base = tc_setup<kScoreStages>(sh, tc_raw, kScoreCols);
    const uint32_t tmem = sh.tmem;
    volatile int* abort_flag = &sh.abort_flag;
    dep_trigger();          // the kernel behind (act) holds next to nothing while it waits for this one

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&map_k1);
            tma_prefetch_desc(&map_k2);
            tma_prefetch_desc(&map_xhi);
            tma_prefetch_desc(&map_xlo);
            auto load_w = [&](int i) {
                const int c = c0 + i, s = i % kScoreStages;
                const uint32_t bar = smem_addr(&sh.full[s]), dst = base + s * kScoreStageBytes;
                mbar_expect_tx(bar, kScoreWBytes + 2 * xbytes);
                if (c < p.cs) tma_load_2d(dst, &map_k1, bar, c * kChunk, row0);
                else tma_load_2d(dst, &map_k2, bar, (c - p.cs) * kChunk, row0);
            };
            auto load_x = [&](int i) {
                const int c = c0 + i, s = i % kScoreStages;
                const uint32_t bar = smem_addr(&sh.full[s]), dst = base + s * kScoreStageBytes + kScoreWBytes;
                tma_load_2d(dst, &map_xhi, bar, c * kChunk, 0);
                tma_load_2d(dst + xbytes, &map_xlo, bar, c * kChunk, 0);        // lo rows right behind the hi rows
            };
            const int pre = min(nch, kScoreStages);
            for (int i = 0; i < pre; ++i) load_w(i);      // the weights do not depend on the kernel ahead
            dep_wait();
            for (int i = 0; i < pre; ++i) load_x(i);
            int issued = pre;
            for (int i = pre; i < nch; ++i) {
                if (!mbar_wait(smem_addr(&sh.empty[i % kScoreStages]), ((i / kScoreStages) & 1) ^ 1, abort_flag)) break;
                load_w(i);
                load_x(i);
                issued = i + 1;
            }
            if (*abort_flag != 0) tc_drain<kScoreStages>(sh, issued);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(128, 2 * p.ntok, false);
            bool ok = true;
            for (int i = 0; i < nch && ok; ++i) {
                const int s = i % kScoreStages, c = c0 + i;
                ok = mbar_wait(smem_addr(&sh.full[s]), (i / kScoreStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a0 = base + s * kScoreStageBytes, b0 = a0 + kScoreWBytes;
                const uint32_t dcol = tmem + (c < p.cs ? 0u : 128u);
                const bool fresh = i == 0 || c == p.cs;             // first chunk of this accumulator in this block
#pragma unroll
                for (int j = 0; j < kChunk / 16; ++j)
                    umma_bf16(dcol, smem_desc(a0 + 32 * j, 0u, 1024u), smem_desc(b0 + 32 * j, 0u, 1024u), idesc, (fresh && j == 0) ? 0u : 1u);
                umma_commit(smem_addr(&sh.empty[s]));
            }
            if (ok) umma_commit(smem_addr(&sh.accum));
        }
    } else {
        const int q = warp & 3;                                    // tensor-memory lanes 32 q .. 32 q + 31
        const int B = p.f.B, row = row0 + q * 32 + lane;
        const int64_t dff = p.f.d_ff;
        dep_wait();
        {   // y = y_init (or 0) while the weights stream: the output kernel adds into it
            const int64_t total4 = static_cast<int64_t>(B) * p.f.d / 4;
            const float4* yi = reinterpret_cast<const float4*>(p.f.y_init);
            float4* yo = reinterpret_cast<float4*>(p.f.y);
            for (int64_t i = static_cast<int64_t>(blockIdx.x) * 128 + (tid - 64); i < total4; i += static_cast<int64_t>(gridDim.x) * 128)
                yo[i] = yi != nullptr ? yi[i] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        const bool ok = __all_sync(kFull, mbar_wait(smem_addr(&sh.accum), 0u, abort_flag));   // warp-uniform: tcgen05.ld is warp-wide
        const bool has_s = c0 < p.cs, has_t = c1 > p.cs;
        if (ok) {
            tc_fence_after();
            const uint32_t taddr = tmem + (static_cast<uint32_t>(q * 32) << 16);
            float v[32], w[32];
            if (has_s) {
                // the stages are idle now: a 32 x 33 transposition window per warp for the per-token sums
                float* win = reinterpret_cast<float*>(tc_raw + (base - smem_addr(tc_raw))) + (warp - 2) * (32 * 33);
                for (int hb = 0; hb * 32 < B; ++hb) {
                    tmem_ld32(taddr + hb * 32, v);
                    tmem_ld32(taddr + p.ntok + hb * 32, w);
#pragma unroll
                    for (int n = 0; n < 32; ++n) {
                        const float sv = v[n] + w[n];
                        if (hb * 32 + n < B) p.g.S[(hb * 32 + n) * dff + row] = sv;
                        win[n * 33 + lane] = sv;
                    }
                    __syncwarp();
                    double s1 = 0.0, s2 = 0.0;
#pragma unroll 8
                    for (int i = 0; i < 32; ++i) {
                        const double x = static_cast<double>(win[lane * 33 + i]);
                        s1 += x;
                        s2 = fma(x, x, s2);
                    }
                    sh.colsum[q][hb * 32 + lane][0] = s1;
                    sh.colsum[q][hb * 32 + lane][1] = s2;
                    __syncwarp();
                }
            }
            if (has_t) {
                float* T = p.g.T + static_cast<int64_t>(part) * kTok * dff;
                for (int hb = 0; hb * 32 < B; ++hb) {
                    tmem_ld32(taddr + 128 + hb * 32, v);
                    tmem_ld32(taddr + 128 + p.ntok + hb * 32, w);
#pragma unroll
                    for (int n = 0; n < 32; ++n)
                        if (hb * 32 + n < B) T[(hb * 32 + n) * dff + row] = v[n] + w[n];
                }
            }
        }
        if (has_s) {
            asm volatile("bar.sync 1, 128;" ::: "memory");               // the four epilogue warps
            const int n = tid - 64;
            if (ok && n < B) {
                double s1 = 0.0, s2 = 0.0;
#pragma unroll
                for (int w4 = 0; w4 < 4; ++w4) {
                    s1 += sh.colsum[w4][n][0];
                    s2 += sh.colsum[w4][n][1];
                }
                double* cell = p.g.sums + (static_cast<size_t>(tile % kSumWays) * kTok + n) * 2;
                red_add_f64(cell, s1);
                red_add_f64(cell + 1, s2);
            }
        }
    }
    tc_finish(sh, kScoreCols, p.f.hdr);
}

// ---- act: theta, masks, U = [S > theta] . GELU(S - theta) . T in two bf16 terms -----------------------------
constexpr int kActThreads = 256;
constexpr int kActSpan = kActThreads * 8;        // neurons per block, eight per thread

__global__ void __launch_bounds__(kActThreads) ffn_tc_act_kernel(const TcParams p, int blocks_per_token) {
    __shared__ float theta_s;
    __shared__ int wsum[kActThreads / 32];
    __shared__ int base_s;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = blockIdx.x / blocks_per_token, bx = blockIdx.x - n * blocks_per_token;
    const int64_t dff = p.f.d_ff;
    dep_trigger();          // the kernel behind (out) starts on its weight stream while this one runs
    dep_wait();
    // the block's scores and products are requested before theta is known
    const int j0 = bx * kActSpan + tid * 8;
    const int64_t off = static_cast<int64_t>(n) * dff + j0;
    float s[8], t[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] = t[i] = 0.f;
    if (j0 < dff) {
        *reinterpret_cast<float4*>(s) = __ldcg(reinterpret_cast<const float4*>(p.g.S + off));
        *reinterpret_cast<float4*>(s + 4) = __ldcg(reinterpret_cast<const float4*>(p.g.S + off) + 1);
        for (int tp = p.tfirst; tp < kMaxTParts; ++tp) {
            const float4* src = reinterpret_cast<const float4*>(p.g.T + static_cast<int64_t>(tp) * kTok * dff + off);
            const float4 a = __ldcg(src), b = __ldcg(src + 1);
            t[0] += a.x; t[1] += a.y; t[2] += a.z; t[3] += a.w;
            t[4] += b.x; t[5] += b.y; t[6] += b.z; t[7] += b.w;
        }
    }
    if (warp == 0) {
        double s1 = 0.0, s2 = 0.0;
        if (lane < kSumWays) {
            const double* cell = p.g.sums + (static_cast<size_t>(lane) * kTok + n) * 2;
            s1 = cell[0];
            s2 = cell[1];
        }
        s1 = warp_sum_f64(s1);
        s2 = warp_sum_f64(s2);
        if (lane == 0) {
            float th = -INFINITY;
            if (!p.f.identity) {
                const double mean = s1 * p.f.inv_n;
                const float var = static_cast<float>((s2 - s1 * mean) * p.f.inv_nm1);
                th = static_cast<float>(mean) + sqrtf(fmaxf(var, 0.f)) * static_cast<float>(p.f.z);
            }
            theta_s = th;
            if (bx == 0 && p.f.theta != nullptr) p.f.theta[n] = th;
        }
    }
    __syncthreads();
    const float th = theta_s, shift = p.f.identity ? 0.f : th;
    unsigned mask = 0u;
    if (j0 < dff) {
        float u[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const bool on = s[i] > th;
            const float a = s[i] - shift;
            u[i] = on ? (p.f.erf_form ? gelu_erf(a) : gelu_tanh(a)) * t[i] : 0.f;
            mask |= on ? 1u << i : 0u;
        }
        unsigned h[4], l[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            h[i] = pack2_bf16(u[2 * i], u[2 * i + 1]);
            l[i] = pack2_bf16(u[2 * i] - __uint_as_float(h[i] << 16), u[2 * i + 1] - __uint_as_float(h[i] & 0xffff0000u));
        }
        *reinterpret_cast<uint4*>(p.g.uhi + off) = make_uint4(h[0], h[1], h[2], h[3]);
        *reinterpret_cast<uint4*>(p.g.ulo + off) = make_uint4(l[0], l[1], l[2], l[3]);
    }
    if (p.f.count != nullptr) {
        // the block's share of the token's list is contiguous and ascending; blocks take their places in
        // the order in which they get here
        const int c = __popc(mask);
        int incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) wsum[warp] = incl;
        __syncthreads();
        int before = 0, total = 0;
#pragma unroll
        for (int w = 0; w < kActThreads / 32; ++w) {
            if (w < warp) before += wsum[w];
            total += wsum[w];
        }
        if (tid == 0) base_s = total > 0 ? atomicAdd(&p.f.count[n], total) : 0;
        __syncthreads();
        if (p.f.idx != nullptr && c > 0) {
            int32_t* out = p.f.idx + static_cast<int64_t>(n) * dff + base_s + before + incl - c;
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if ((mask >> i) & 1u) *out++ = j0 + i;
        }
    }
}

// ---- out: Y^T[256 columns of the block] += Vt[neurons of the block]^T . U ------------------------------------
constexpr int kOutStages = 4;
constexpr int kOutVBytes = 4 * kChunk * 128;                                  // four boxes of 64 neurons x 64 columns
constexpr int kOutStageBytes = kOutVBytes + 2 * kTok * kChunk * 2;            // + u hi, u lo
constexpr uint32_t kOutCols = 256;                                            // two accumulators of 128 model columns x (hi | lo) tokens

__global__ void __launch_bounds__(kTcThreads, 1)
ffn_tc_out_kernel(const TcParams p, const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_uhi,
                  const __grid_constant__ CUtensorMap map_ulo) {
    extern __shared__ unsigned char tc_raw[];
    __shared__ TcShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nb = blockIdx.x / p.ksplit, ks = blockIdx.x - nb * p.ksplit;
    const int cn = p.f.d_ff / kChunk;
    const int c0 = static_cast<int>(static_cast<int64_t>(ks) * cn / p.ksplit), c1 = static_cast<int>(static_cast<int64_t>(ks + 1) * cn / p.ksplit);
    const int nch = c1 - c0, col0 = nb * 256;
    const uint32_t base = tc_setup<kOutStages>(sh, tc_raw, kOutCols);
    const uint32_t tmem = sh.tmem;
    volatile int* abort_flag = &sh.abort_flag;
    dep_trigger();

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&map_v);
            tma_prefetch_desc(&map_uhi);
            tma_prefetch_desc(&map_ulo);
            auto load_v = [&](int i) {
                const int s = i % kOutStages;
                const uint32_t bar = smem_addr(&sh.full[s]);
                mbar_expect_tx(bar, kOutVBytes + 2 * static_cast<uint32_t>(p.ntok) * kChunk * 2);
#pragma unroll
                for (int b = 0; b < 4; ++b) tma_load_2d(base + s * kOutStageBytes + b * (kChunk * 128), &map_v, bar, col0 + 64 * b, (c0 + i) * kChunk);
            };
            auto load_u = [&](int i) {
                const int s = i % kOutStages;
                const uint32_t bar = smem_addr(&sh.full[s]), dst = base + s * kOutStageBytes + kOutVBytes;
                tma_load_2d(dst, &map_uhi, bar, (c0 + i) * kChunk, 0);
                tma_load_2d(dst + static_cast<uint32_t>(p.ntok) * kChunk * 2, &map_ulo, bar, (c0 + i) * kChunk, 0);   // lo rows behind the hi rows
            };
            const int pre = min(nch, kOutStages);
            for (int i = 0; i < pre; ++i) load_v(i);      // the rows of V do not depend on the kernels ahead
            dep_wait();
            for (int i = 0; i < pre; ++i) load_u(i);
            int issued = pre;
            for (int i = pre; i < nch; ++i) {
                if (!mbar_wait(smem_addr(&sh.empty[i % kOutStages]), ((i / kOutStages) & 1) ^ 1, abort_flag)) break;
                load_v(i);
                load_u(i);
                issued = i + 1;
            }
            if (*abort_flag != 0) tc_drain<kOutStages>(sh, issued);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(128, 2 * p.ntok, true);
            bool ok = true;
            for (int i = 0; i < nch && ok; ++i) {
                const int s = i % kOutStages;
                ok = mbar_wait(smem_addr(&sh.full[s]), (i / kOutStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t v0 = base + s * kOutStageBytes, b0 = v0 + kOutVBytes;
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
                    for (int j = 0; j < kChunk / 16; ++j) {
                        // A: 16 neurons (K) x 128 columns (M) of V, MN-major: 8-neuron groups 1024 bytes apart, the
                        // second 64 columns in the next box (8192 bytes on)
                        const uint64_t ad = smem_desc(v0 + mt * (2 * kChunk * 128) + j * 2048, kChunk * 128, 1024u);
                        umma_bf16(tmem + mt * 128, ad, smem_desc(b0 + 32 * j, 0u, 1024u), idesc, (i == 0 && j == 0) ? 0u : 1u);
                    }
                }
                umma_commit(smem_addr(&sh.empty[s]));
            }
            if (ok) umma_commit(smem_addr(&sh.accum));
        }
    } else {
        const int q = warp & 3, B = p.f.B;
        const int64_t d = p.f.d;
        dep_wait();
        if (nch > 0 && __all_sync(kFull, mbar_wait(smem_addr(&sh.accum), 0u, abort_flag))) {
            tc_fence_after();
            const uint32_t taddr = tmem + (static_cast<uint32_t>(q * 32) << 16);
            float v[32], w[32];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                float* ycol = p.f.y + col0 + mt * 128 + q * 32 + lane;
                for (int hb = 0; hb * 32 < B; ++hb) {
                    tmem_ld32(taddr + mt * 128 + hb * 32, v);
                    tmem_ld32(taddr + mt * 128 + p.ntok + hb * 32, w);
#pragma unroll
                    for (int n = 0; n < 32; ++n)
                        if (hb * 32 + n < B) atomicAdd(ycol + (hb * 32 + n) * d, v[n] + w[n]);
                }
            }
        }
    }
    tc_finish(sh, kOutCols, p.f.hdr);
}

}  // namespace

namespace spark {

size_t ffn_tc_workspace_bytes(int64_t d, int64_t d_ff) { return tc_region_bytes(d, d_ff); }

// SPARK_ERR_WORKSPACE = shape or workspace not served by this path (the caller falls back).
int ffn_tc_launch(spark_ctx* ctx, FfnParams& f, cudaStream_t stream) {
    const int d = f.d, r = f.r, d_ff = f.d_ff, B = f.B;
    if (B < 1 || B > kTok || d % 256 != 0 || r % kChunk != 0 || r <= 0 || r >= d || d_ff % 128 != 0 || f.K1s != nullptr) return SPARK_ERR_WORKSPACE;
    // The first block of a pair takes all of the predictor's chunks (its sums must be complete) and, where that
    // leaves it short, some of the K2 product's.  Epilogues in units of a chunk's time (measured): scores
    // and sums about eight, a partial K2 product about four.
    const int call = d / kChunk, cs = r / kChunk;
    if (cs >= call) return SPARK_ERR_WORKSPACE;
    int chalf = cs, best = 1 << 30;
    for (int c = cs; c < call; ++c) {
        const int first = c + 8 + (c > cs ? 4 : 0), second = call - c + 4, worst = first > second ? first : second;
        if (worst < best) {
            best = worst;
            chalf = c;
        }
    }
    if (ctx->scratch == nullptr || ctx->scratch_bytes < kAttnCellBytes + tc_region_bytes(d, d_ff)) return SPARK_ERR_WORKSPACE;
    const size_t smem_scores = static_cast<size_t>(kScoreStages) * kScoreStageBytes + 1024;
    const size_t smem_out = static_cast<size_t>(kOutStages) * kOutStageBytes + 1024;
    if (smem_scores + sizeof(TcShared) + 64 > static_cast<size_t>(ctx->max_smem_optin) ||
        smem_out + sizeof(TcShared) + 64 > static_cast<size_t>(ctx->max_smem_optin))
        return SPARK_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(f.K1t) | reinterpret_cast<uintptr_t>(f.K2t) | reinterpret_cast<uintptr_t>(f.Vt)) & 15u) return SPARK_ERR_WORKSPACE;

    TcParams p;
    p.f = f;
    p.g = tc_region(ctx->scratch + kAttnCellBytes, d, d_ff);       // behind the attention's persistent cells
    p.ntok = (B + 15) & ~15;
    p.cs = cs;
    p.call = call;
    p.chalf = chalf;
    p.tfirst = chalf > cs ? 0 : 1;
    const int nbk = d / 256;
    p.ksplit = ctx->num_sms / nbk > 0 ? ctx->num_sms / nbk : 1;
    if (p.ksplit > d_ff / kChunk) p.ksplit = d_ff / kChunk;

    CUtensorMap m_k1, m_k2, m_xhi, m_xlo, m_v, m_uhi, m_ulo;
    if (!make_map(&m_k1, f.K1t, d_ff, r, r, 128, true) || !make_map(&m_k2, f.K2t, d_ff, d - r, d - r, 128, true) ||
        !make_map(&m_xhi, p.g.xhi, kTok, d, d, p.ntok, false) || !make_map(&m_xlo, p.g.xlo, kTok, d, d, p.ntok, false) ||
        !make_map(&m_v, f.Vt, d_ff, d, d, kChunk, true) || !make_map(&m_uhi, p.g.uhi, kTok, d_ff, d_ff, p.ntok, false) ||
        !make_map(&m_ulo, p.g.ulo, kTok, d_ff, d_ff, p.ntok, false))
        return SPARK_ERR_WORKSPACE;

    if (cudaFuncSetAttribute(ffn_tc_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_scores)) != cudaSuccess ||
        cudaFuncSetAttribute(ffn_tc_out_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_out)) != cudaSuccess)
        return SPARK_ERR_CUDA;
    {
        void* args[] = {&p};
        if (launch_kernel(ctx, reinterpret_cast<const void*>(ffn_tc_prep_kernel), kTok * kPrepSplit, 256, 0, stream, false, args) != cudaSuccess) return SPARK_ERR_CUDA;
    }
    {
        void* args[] = {&p, &m_k1, &m_k2, &m_xhi, &m_xlo};
        if (launch_kernel(ctx, reinterpret_cast<const void*>(ffn_tc_scores_kernel), static_cast<unsigned>(2 * (d_ff / kScoreRows)), kTcThreads, smem_scores, stream, false, args) != cudaSuccess)
            return SPARK_ERR_CUDA;
    }
    {
        int bpt = (d_ff + kActSpan - 1) / kActSpan;
        void* args[] = {&p, &bpt};
        if (launch_kernel(ctx, reinterpret_cast<const void*>(ffn_tc_act_kernel), static_cast<unsigned>(bpt * B), kActThreads, 0, stream, false, args) != cudaSuccess)
            return SPARK_ERR_CUDA;
    }
    {
        void* args[] = {&p, &m_v, &m_uhi, &m_ulo};
        if (launch_kernel(ctx, reinterpret_cast<const void*>(ffn_tc_out_kernel), static_cast<unsigned>(nbk * p.ksplit), kTcThreads, smem_out, stream, false, args) != cudaSuccess)
            return SPARK_ERR_CUDA;
    }
    return SPARK_OK;
}

}  // namespace spark
