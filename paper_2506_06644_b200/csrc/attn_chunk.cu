// Spark attention (Section 2.2, Eq. 7) for a chunk of a prompt: T consecutive tokens of one sequence, all
// reading one cache, token t seeing rows [lo_t, n_t).  Here the predictor scores of all of the chunk's queries
// against a cached row are one row of a GEMM -- S[j][(t, head)] = k1c[j] . q1[t, head] -- so every cached row of
// the predictor slice is read once for the whole chunk instead of once per query, and the product runs on the
// fifth-generation tensor cores.  Three kernels, ordered by the stream (no block waits on another block):
//   prep    q[:, :, :r] -> two bf16 terms (hi + lo) as operand rows per KV head; Q(1 - k/L_t), row ranges
//   scores  per KV head: S = k1c . Q1^T, M = 128 cached rows per tile, N = 2 x (tokens x heads per KV head), K = r;
//           TMA-fed tcgen05.mma into double-buffered tensor-memory accumulators; eight epilogue warps add the two
//           halves of the accumulator and write S column-major
//   select  one block per (token, query head): sums of its column over the rows it may see -> theta (Eq. 10/11),
//           survivors, softmax over the survivors, softplus gate from the k2c rows, weighted sum of the vc rows
//           (only the survivors' rows are read)
// or, in place of select when a KV head serves many (token, head) pairs and the rows are few thousand (see "dense second
// stage" below): stats (theta, maximum, sum of exponentials per column) and dense (every row read once per block; gate and
// weighted value sum as two more tensor-core products under the selection mask).
// Same pipeline skeleton and bounded waits as the other tensor-core kernels (tc_common.cuh).
#include <cstddef>

#include "kernels.h"
#include "tc_common.cuh"

using namespace spark;
using namespace spark::tc;

namespace {

constexpr int kColMax = 128;          // (token, head-in-group) columns per KV head
constexpr int kSelThreads = 256;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kColRows = 8192;        // visible rows of a column the select kernel keeps in shared memory

struct ChunkParams {
    const float* q;            // [T][n_q][hd]
    const __nv_bfloat16* k2c;  // [n_kv][cap][hd - r]
    const __nv_bfloat16* vc;   // [n_kv][cap][hd]
    const int32_t* ctx_len;    // [T]
    const double* zs_in;       // nullable: Q(1 - k_attn / L_t) per token from an earlier kernel
    int T, n_q, n_kv, gq, hd, r, window, k_attn;
    int ncol, ncolp;           // T * gq, rounded up to a multiple of 16
    int64_t cap;
    float* o;                  // [T][n_q][hd], normalised
    float* lsum;               // nullable: [T][n_q] = 1 (0 for an empty selection): the caller divides by it
    float* theta;              // nullable [T][n_q]
    int32_t* count;            // nullable [T][n_q]
    // workspace
    double* zt;                // [T]
    int* range;                // [T][2] = lo_t, n_t
    __nv_bfloat16* qhi;        // [n_kv][kColMax][r]
    __nv_bfloat16* qlo;
    float* S;                  // [n_kv][kColMax][scap]
    int64_t scap;              // column stride of S: cap + 32, so that the columns' lines do not all fall on the same slices
    // dense second stage (masked weights x value rows on the tensor cores) only
    __nv_bfloat16* q2hi;       // [n_kv][kColMax][hd - r]: the gate's query part as two bf16 terms
    __nv_bfloat16* q2lo;
    float4* colinfo;           // [n_kv][kColMax] = theta, maximum of the survivors' scores, lo, n (the last two as int bits)
    float* zsum;               // [T][n_q] sum of exp(s - max) over the survivors
    int dense;
    WsHeader* hdr;
};

__device__ __forceinline__ void token_range(const ChunkParams& p, int t, int& lo, int& n) {
    n = p.ctx_len[t];
    n = n < 1 ? 1 : (n > p.cap ? static_cast<int>(p.cap) : n);
    lo = (p.window > 0 && p.window < n) ? n - p.window : 0;
}

// ---- prep: one block per (KV head, column) ---------------------------------------------------------------------
__global__ void __launch_bounds__(128) attn_chunk_prep_kernel(const ChunkParams p) {
    const int g = blockIdx.x / kColMax, col = blockIdx.x % kColMax, tid = threadIdx.x;
    dep_wait();
    dep_trigger();
    if (blockIdx.x == 0) {
        for (int t = tid; t < p.T; t += 128) {
            int lo, n;
            token_range(p, t, lo, n);
            p.range[2 * t] = lo;
            p.range[2 * t + 1] = n;
            const int L = n - lo;
            p.zt[t] = p.zs_in != nullptr ? p.zs_in[t]
                                         : (p.k_attn >= L ? 0.0 : -normcdfinv(static_cast<double>(p.k_attn) / static_cast<double>(L)));
        }
    }
    if (col >= (p.dense ? ((p.ncol + 63) & ~63) : p.ncolp)) return;                 // rows the operand boxes never touch
    __nv_bfloat16* hi = p.qhi + (static_cast<int64_t>(g) * kColMax + col) * p.r;
    __nv_bfloat16* lo = p.qlo + (static_cast<int64_t>(g) * kColMax + col) * p.r;
    const int t = col / p.gq, hq = col - t * p.gq;
    for (int i = tid; i < p.r; i += 128) {
        float v = 0.f;
        if (col < p.ncol) v = p.q[(static_cast<int64_t>(t) * p.n_q + g * p.gq + hq) * p.hd + i];
        const __nv_bfloat16 h = __float2bfloat16_rn(v);
        hi[i] = h;
        lo[i] = __float2bfloat16_rn(v - __bfloat162float(h));
    }
    if (p.dense) {
        const int d2 = p.hd - p.r;
        __nv_bfloat16* h2 = p.q2hi + (static_cast<int64_t>(g) * kColMax + col) * d2;
        __nv_bfloat16* l2 = p.q2lo + (static_cast<int64_t>(g) * kColMax + col) * d2;
        for (int i = tid; i < d2; i += 128) {
            float v = 0.f;
            if (col < p.ncol) v = p.q[(static_cast<int64_t>(t) * p.n_q + g * p.gq + hq) * p.hd + p.r + i];
            const __nv_bfloat16 h = __float2bfloat16_rn(v);
            h2[i] = h;
            l2[i] = __float2bfloat16_rn(v - __bfloat162float(h));
        }
    }
}

// ---- scores: S = k1c . Q1^T per KV head, 128 cached rows per tile ------------------------------------------------------
constexpr int kChunkStages = 2;
constexpr int kChunkABytes = 2 * 128 * kChunk * 2;           // up to two K chunks of 128 rows x 128 bytes
constexpr int kChunkBBytes = 2 * 2 * kColMax * kChunk * 2;   // per K chunk: hi rows, lo rows of the query operand
constexpr int kChunkStageBytes = kChunkABytes + kChunkBBytes;
constexpr uint32_t kChunkCols = 512;                         // two accumulators of 128 rows x (hi | lo) columns

struct ChunkShared {
    unsigned long long full[kChunkStages], empty[kChunkStages];
    unsigned long long acc_full[2], acc_empty[2];
    uint32_t tmem;
    int abort_flag;
    int n_max;
};
constexpr int kChunkThreads = 64 + 8 * 32;      // warp 0: TMA, warp 1: MMA + tensor memory, warps 2..9: epilogue

__global__ void __launch_bounds__(kChunkThreads, 1)
attn_chunk_scores_kernel(const ChunkParams p, const __grid_constant__ CUtensorMap map_k1, const __grid_constant__ CUtensorMap map_qhi,
                         const __grid_constant__ CUtensorMap map_qlo) {
    extern __shared__ unsigned char tc_raw[];
    __shared__ ChunkShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nkc = p.r / kChunk;
    if (tid == 0) {
        for (int s = 0; s < kChunkStages; ++s) {
            mbar_init(smem_addr(&sh.full[s]), 1u);
            mbar_init(smem_addr(&sh.empty[s]), 1u);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_addr(&sh.acc_full[b]), 1u);
            mbar_init(smem_addr(&sh.acc_empty[b]), 1u);
        }
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_addr(&sh.tmem), kChunkCols);
    dep_wait();                  // everything this kernel reads comes from the kernels ahead (cache rows, queries, ranges)
    dep_trigger();
    if (tid == 0) {
        int m = 1;
        for (int t = 0; t < p.T; ++t) m = max(m, p.range[2 * t + 1]);
        sh.n_max = m;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t base = (smem_addr(tc_raw) + 1023u) & ~1023u;
    const uint32_t tmem = sh.tmem;
    volatile int* abort_flag = &sh.abort_flag;
    const int n_max = sh.n_max;
    const int tiles_h = (n_max + 127) / 128, total = p.n_kv * tiles_h;
    const int t0 = static_cast<int>(static_cast<int64_t>(blockIdx.x) * total / gridDim.x);
    const int t1 = static_cast<int>(static_cast<int64_t>(blockIdx.x + 1) * total / gridDim.x);
    const uint32_t qbytes = static_cast<uint32_t>(p.ncolp) * kChunk * 2;          // one term of one K chunk of the queries
    const uint32_t stage_tx = static_cast<uint32_t>(nkc) * (128 * kChunk * 2 + 2 * qbytes);

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&map_k1);
            tma_prefetch_desc(&map_qhi);
            tma_prefetch_desc(&map_qlo);
            int issued = 0;
            for (int tile = t0; tile < t1; ++tile) {
                const int i = tile - t0, s = i % kChunkStages;
                if (i >= kChunkStages && !mbar_wait(smem_addr(&sh.empty[s]), ((i / kChunkStages) & 1) ^ 1, abort_flag)) break;
                const int g = tile / tiles_h, rb = tile - g * tiles_h;
                const uint32_t bar = smem_addr(&sh.full[s]), dst = base + s * kChunkStageBytes;
                mbar_expect_tx(bar, stage_tx);
                for (int kc = 0; kc < nkc; ++kc) {
                    tma_load_2d(dst + kc * (128 * kChunk * 2), &map_k1, bar, kc * kChunk, static_cast<int>(g * p.cap + rb * 128));
                    const uint32_t qd = dst + kChunkABytes + kc * (2 * kColMax * kChunk * 2);
                    tma_load_2d(qd, &map_qhi, bar, kc * kChunk, g * kColMax);
                    tma_load_2d(qd + qbytes, &map_qlo, bar, kc * kChunk, g * kColMax);    // lo rows right behind the hi rows
                }
                issued = i + 1;
            }
            if (*abort_flag != 0) {
                for (int i = max(0, issued - kChunkStages); i < issued; ++i) {
                    const long long c0 = clock64();
                    while (!mbar_try(smem_addr(&sh.full[i % kChunkStages]), (i / kChunkStages) & 1))
                        if (clock64() - c0 > kTcSpinLimit) break;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(128, 2 * p.ncolp, false);
            for (int tile = t0; tile < t1; ++tile) {
                const int i = tile - t0, s = i % kChunkStages, b = i & 1;
                if (i >= 2 && !mbar_wait(smem_addr(&sh.acc_empty[b]), ((i >> 1) & 1) ^ 1, abort_flag)) break;
                if (!mbar_wait(smem_addr(&sh.full[s]), (i / kChunkStages) & 1, abort_flag)) break;
                tc_fence_after();
                const uint32_t a0 = base + s * kChunkStageBytes, q0 = a0 + kChunkABytes;
                for (int kc = 0; kc < nkc; ++kc)
#pragma unroll
                    for (int j = 0; j < kChunk / 16; ++j)
                        umma_bf16(tmem + b * 256, smem_desc(a0 + kc * (128 * kChunk * 2) + 32 * j, 0u, 1024u),
                                  smem_desc(q0 + kc * (2 * kColMax * kChunk * 2) + 32 * j, 0u, 1024u), idesc, (kc == 0 && j == 0) ? 0u : 1u);
                umma_commit(smem_addr(&sh.empty[s]));
                umma_commit(smem_addr(&sh.acc_full[b]));
            }
        }
    } else {
        // eight warps: two per tensor-memory lane quadrant, each taking half of the columns
        const int q = warp & 3, half = (warp - 2) >> 2;
        bool ok = true;
        for (int tile = t0; tile < t1 && ok; ++tile) {
            const int i = tile - t0, b = i & 1;
            const int g = tile / tiles_h, rb = tile - g * tiles_h;
            ok = __all_sync(kFull, mbar_wait(smem_addr(&sh.acc_full[b]), (i >> 1) & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const int j = rb * 128 + q * 32 + lane;
            const uint32_t tacc = tmem + b * 256 + (static_cast<uint32_t>(q * 32) << 16);
            float* scol = p.S + static_cast<int64_t>(g) * kColMax * p.scap + j;
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
                const int cb = 2 * half + cc;
                if (cb * 32 < p.ncol) {
                    float v[32], w[32];
                    tmem_ld32(tacc + cb * 32, v);
                    tmem_ld32(tacc + p.ncolp + cb * 32, w);
                    if (j < n_max) {
#pragma unroll
                        for (int c = 0; c < 32; ++c)
                            if (cb * 32 + c < p.ncol) scol[static_cast<int64_t>(cb * 32 + c) * p.scap] = v[c] + w[c];
                    }
                }
            }
            tc_fence_before();
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (tid == 64) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&sh.acc_empty[b])) : "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_free(tmem, kChunkCols);
    }
    if (tid == 0 && sh.abort_flag != 0) atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_TIMEOUT);
}

// ---- select: one block per (token, query head) ---------------------------------------------------------------------------
// The column's visible scores are read once into shared memory: every warp compacts the survivors of its slice into a
// list (index, score) and tracks their maximum; after the block-wide maximum is known each warp walks its list
// four survivors at a time (four blocks per SM -- all 512 (token, head) pairs of a 64-token chunk resident at once --
// matter more than loads in flight: the gather is bound by what L2 delivers): the k2c rows give the softplus gates, the vc rows are accumulated with weight
// exp(s - max) . gate, eight columns of the output per lane.  The sum of exp(s - max) normalises the result.
// REGS: see the kernel below (the list capacity and the column buffer differ between its two variants)
template <bool REGS>
struct SelShared {
    static constexpr int kListCap = REGS ? 512 : 192;      // survivors a warp lists before it gathers them
    int idx[kSelWarps][kListCap];
    float sc[kSelWarps][kListCap];
    float q2[128];
    float red[kSelWarps];
    float acc[kSelWarps][256];
    float esum[kSelWarps];
    int cnt[kSelWarps];
    double part[kSelWarps][2];
    float theta;
    __align__(16) float col[REGS ? 4 : kColRows + 4];
};

// REGS: a slice of up to 1024 rows per warp stays in registers (three blocks per SM; the faster block when all blocks
// are resident anyway); otherwise the column is staged in shared memory (64 registers, four blocks per SM).
template <bool REGS>
__global__ void __launch_bounds__(kSelThreads, REGS ? 3 : 4) attn_chunk_select_kernel(const ChunkParams p) {
    extern __shared__ __align__(16) unsigned char sel_raw[];
    SelShared<REGS>& sh = *reinterpret_cast<SelShared<REGS>*>(sel_raw);
    constexpr int kListCap = SelShared<REGS>::kListCap;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t = blockIdx.x / p.n_q, h = blockIdx.x - t * p.n_q;
    const int g = h / p.gq, col = t * p.gq + (h - g * p.gq);
    const int d2 = p.hd - p.r;
    dep_wait();
    dep_trigger();
    const int lo = p.range[2 * t], n = p.range[2 * t + 1], L = n - lo;
    if (tid < d2) sh.q2[tid] = p.q[(static_cast<int64_t>(t) * p.n_q + h) * p.hd + p.r + tid];
    const float* scol = p.S + (static_cast<int64_t>(g) * kColMax + col) * p.scap;
    // slices of the visible range, one per warp; with the column in shared memory they start on 16-byte boundaries
    // of the column (lo4 <= lo)
    const int lo4 = REGS ? lo : (lo & ~3);
    const int per = REGS ? (L + kSelWarps - 1) / kSelWarps : ((((n - lo4) + kSelWarps - 1) / kSelWarps + 3) & ~3);
    const int w0 = max(lo, lo4 + warp * per), w1 = min(n, lo4 + (warp + 1) * per);
    constexpr int kKeep = REGS ? 32 : 1;
    const bool kept = REGS ? per <= 32 * kKeep : n - lo4 <= kColRows;
    [[maybe_unused]] float keep[kKeep];
    if constexpr (REGS) {
        if (kept) {      // up to 1024 rows of the slice in registers, all loads in flight at once
#pragma unroll
            for (int u = 0; u < kKeep; ++u) {
                const int j = w0 + 32 * u + lane;
                keep[u] = j < w1 ? __ldcg(scol + j) : -INFINITY;
            }
        }
    } else if (kept) {
        // asynchronous 16-byte copies straight into shared memory: the whole slice is in flight at once and no
        // registers are held (rows past n inside the last 16 bytes are copied too and never looked at)
        const int c0 = lo4 + warp * per, c1 = min((n + 3) & ~3, c0 + per);
        const unsigned dst0 = static_cast<unsigned>(__cvta_generic_to_shared(sh.col));
        for (int j = c0 + 4 * lane; j < c1; j += 128)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst0 + 4u * static_cast<unsigned>(j - lo4)), "l"(scol + j) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
    }
    if (p.k_attn < L) {
        // sums of the column over the rows this query may see, around the column's first value (keeps the fp32
        // partial sums accurate when |mean| >> std); combined in fp64
        const float c0 = __ldcg(scol + lo);
        float f1 = 0.f, f2 = 0.f;
        if (kept) {
            if constexpr (REGS) {
#pragma unroll
                for (int u = 0; u < kKeep; ++u) {
                    const float d = w0 + 32 * u + lane < w1 ? keep[u] - c0 : 0.f;
                    f1 += d;
                    f2 = fmaf(d, d, f2);
                }
            } else {
                for (int j = w0 + lane; j < w1; j += 32) {
                    const float d = sh.col[j - lo4] - c0;
                    f1 += d;
                    f2 = fmaf(d, d, f2);
                }
            }
        } else {
            for (int j0 = w0; j0 < w1; j0 += 32 * 16) {
                float sv[16];
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    const int j = j0 + 32 * u + lane;
                    sv[u] = j < w1 ? __ldcg(scol + j) - c0 : 0.f;
                }
#pragma unroll
                for (int u = 0; u < 16; ++u) {
                    f1 += sv[u];
                    f2 = fmaf(sv[u], sv[u], f2);
                }
            }
        }
        const double s1 = warp_sum_f64(static_cast<double>(f1)), s2 = warp_sum_f64(static_cast<double>(f2));
        if (lane == 0) {
            sh.part[warp][0] = s1;
            sh.part[warp][1] = s2;
        }
    }
    __syncthreads();
    if (tid == 0) {
        float th = -INFINITY;
        if (p.k_attn < L) {
            double s1 = 0.0, s2 = 0.0;
#pragma unroll
            for (int w = 0; w < kSelWarps; ++w) {
                s1 += sh.part[w][0];
                s2 += sh.part[w][1];
            }
            const double dm = s1 / static_cast<double>(L);                 // mean - c0
            const double var = (s2 - s1 * dm) / static_cast<double>(L - 1);
            th = static_cast<float>(static_cast<double>(__ldcg(scol + lo)) + dm + sqrt(var > 0.0 ? var : 0.0) * p.zt[t]);
        }
        sh.theta = th;
        if (p.theta != nullptr) p.theta[blockIdx.x] = th;
    }
    __syncthreads();
    const float th = sh.theta;
    const __nv_bfloat16* k2 = p.k2c + static_cast<int64_t>(g) * p.cap * d2;
    const __nv_bfloat16* vv = p.vc + static_cast<int64_t>(g) * p.cap * p.hd;
    const int nc2 = d2 / 8, ncv = p.hd / 8;          // 16-byte pieces of a k2c row and of a vc row
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    float run_max = -INFINITY, esum = 0.f;           // of this warp so far: weights are exp(s - run_max)
    int total = 0;
    // The warp's list is drained (its survivors gathered) when the slice is done, or earlier when it is about to overflow.
    auto drain = [&](int cnt, float mx) {
        mx = warp_max(mx);
        __syncwarp();
        if (cnt == 0) return;
        total += cnt;
        if (mx > run_max) {              // rescale what has been accumulated to the new reference
            const float f = run_max == -INFINITY ? 0.f : __expf(run_max - mx);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] *= f;
            esum *= f;
            run_max = mx;
        }
        for (int i0 = 0; i0 < cnt; i0 += 4) {
            uint4 kr[2], vr[4];
            // k2c rows: half a warp per survivor, two loads for four survivors; vc rows: a warp per survivor
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int i = i0 + 2 * u + (lane >> 4);
                kr[u] = (i < cnt && (lane & 15) < nc2) ? ld_stream16(reinterpret_cast<const uint4*>(k2 + static_cast<int64_t>(sh.idx[warp][i]) * d2) + (lane & 15))
                                                       : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u;
                vr[u] = (i < cnt && lane < ncv) ? ld_stream16(reinterpret_cast<const uint4*>(vv + static_cast<int64_t>(sh.idx[warp][i]) * p.hd) + lane)
                                                : make_uint4(0u, 0u, 0u, 0u);
            }
            float gate[4];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const unsigned wds[4] = {kr[u].x, kr[u].y, kr[u].z, kr[u].w};
                const float* qq = sh.q2 + 8 * (lane & 15);
                float d = 0.f;
                if ((lane & 15) < nc2) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        d = fmaf(__uint_as_float(wds[e] << 16), qq[2 * e], d);
                        d = fmaf(__uint_as_float(wds[e] & 0xffff0000u), qq[2 * e + 1], d);
                    }
                }
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) d += __shfl_xor_sync(kFull, d, o);       // within each half-warp
                gate[2 * u] = __shfl_sync(kFull, d, 0);
                gate[2 * u + 1] = __shfl_sync(kFull, d, 16);
            }
            // lane u < 4 evaluates survivor u's exponential and gate once; the others receive them
            float e_l = 0.f, w_l = 0.f;
            if (lane < 4 && i0 + lane < cnt) {
                const float gl = lane == 0 ? gate[0] : (lane == 1 ? gate[1] : (lane == 2 ? gate[2] : gate[3]));
                e_l = __expf(sh.sc[warp][i0 + lane] - run_max);
                w_l = e_l * softplus(gl);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u;
                const float e = __shfl_sync(kFull, e_l, u), wgt = __shfl_sync(kFull, w_l, u);
                if (i < cnt) {
                    esum += e;
                    const unsigned wds[4] = {vr[u].x, vr[u].y, vr[u].z, vr[u].w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        acc[2 * k] = fmaf(wgt, __uint_as_float(wds[k] << 16), acc[2 * k]);
                        acc[2 * k + 1] = fmaf(wgt, __uint_as_float(wds[k] & 0xffff0000u), acc[2 * k + 1]);
                    }
                }
            }
        }
        __syncwarp();
    };
    {
        int cnt = 0;
        float mx = -INFINITY;
        auto take = [&](int j, float sv, bool in_range) {      // one 32-row step: the survivors join the list
            const bool on = in_range && sv > th;
            const unsigned bal = __ballot_sync(kFull, on);
            if (cnt + 32 > kListCap) {
                drain(cnt, mx);
                cnt = 0;
                mx = -INFINITY;
            }
            if (on) {
                const int at = cnt + __popc(bal & ((1u << lane) - 1u));
                sh.idx[warp][at] = j;
                sh.sc[warp][at] = sv;
                mx = fmaxf(mx, sv);
            }
            cnt += __popc(bal);
        };
        bool listed = false;
        if (kept) {
            // the order of the list does not matter: every lane counts its own survivors, a scan of the counts gives it
            // a place, and it writes them there -- no ballot per 32 rows
            int mine = 0;
            if constexpr (REGS) {
#pragma unroll
                for (int u = 0; u < kKeep; ++u) mine += (keep[u] > th) ? 1 : 0;          // rows past the slice hold -inf
            } else {
                for (int j = w0 + lane; j < w1; j += 32) mine += (sh.col[j - lo4] > th) ? 1 : 0;
            }
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(kFull, incl, o);
                if (lane >= o) incl += v;
            }
            const int all = __shfl_sync(kFull, incl, 31);
            if (all <= kListCap) {
                int at = incl - mine;
                if constexpr (REGS) {
#pragma unroll
                    for (int u = 0; u < kKeep; ++u) {
                        if (keep[u] > th) {
                            sh.idx[warp][at] = w0 + 32 * u + lane;
                            sh.sc[warp][at] = keep[u];
                            mx = fmaxf(mx, keep[u]);
                            ++at;
                        }
                    }
                } else {
                    for (int j = w0 + lane; j < w1; j += 32) {
                        const float v = sh.col[j - lo4];
                        if (v > th) {
                            sh.idx[warp][at] = j;
                            sh.sc[warp][at] = v;
                            mx = fmaxf(mx, v);
                            ++at;
                        }
                    }
                }
                cnt = all;
                listed = true;
            }
        }
        if (listed) {
            // done
        } else if (kept) {
            if constexpr (REGS) {
#pragma unroll
                for (int u = 0; u < kKeep; ++u) {
                    const int j = w0 + 32 * u + lane;
                    if (w0 + 32 * u < w1) take(j, keep[u], j < w1);
                }
            } else {
                for (int j0 = w0; j0 < w1; j0 += 32) {
                    const int j = j0 + lane;
                    take(j, j < w1 ? sh.col[j - lo4] : -INFINITY, j < w1);
                }
            }
        } else {
            for (int j0 = w0; j0 < w1; j0 += 32 * 8) {          // eight loads per lane in flight
                float sv[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int j = j0 + 32 * u + lane;
                    sv[u] = j < w1 ? __ldcg(scol + j) : -INFINITY;
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int j = j0 + 32 * u + lane;
                    if (j0 + 32 * u < w1) take(j, sv[u], j < w1);
                }
            }
        }
        drain(cnt, mx);
    }
    // merge the warps: common reference = the block's maximum
    if (lane == 0) {
        sh.red[warp] = run_max;
        sh.cnt[warp] = total;
    }
    __syncthreads();
    float bmax = -INFINITY;
    int btotal = 0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) {
        bmax = fmaxf(bmax, sh.red[w]);
        btotal += sh.cnt[w];
    }
    const float f = (run_max == -INFINITY) ? 0.f : __expf(run_max - bmax);
    if (lane < ncv) {
#pragma unroll
        for (int e = 0; e < 8; ++e) sh.acc[warp][8 * lane + e] = acc[e] * f;
    }
    if (lane == 0) sh.esum[warp] = esum * f;
    __syncthreads();
    float es = 0.f;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) es += sh.esum[w];
    float* orow = p.o + static_cast<int64_t>(blockIdx.x) * p.hd;
    for (int c = tid; c < p.hd; c += kSelThreads) {
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < kSelWarps; ++w) v += sh.acc[w][c];
        orow[c] = btotal > 0 ? v / es : 0.f;
    }
    if (tid == 0) {
        if (p.lsum != nullptr) p.lsum[blockIdx.x] = btotal > 0 ? 1.f : 0.f;
        if (p.count != nullptr) p.count[blockIdx.x] = btotal;
    }
}


// ---- dense second stage ------------------------------------------------------------------------------------------------------
// With many queries per KV head the union of their selections is most of the cache, and the per-query gather above reads
// every selected k2c / vc row once per query out of L2.  The dense form reads every cached row once per block instead and
// leaves the selection to a mask:  o[c] = sum_j w[c][j] v[j] / Z[c],  w[c][j] = [s1 > theta_c] exp(s1 - m_c) softplus(q2_c . k2_j),
// both products on the tensor cores.  Three kernels:
//   stats  one block per (token, query head): theta (Eq. 10/11) from the column of predictor scores, the maximum m of the
//          survivors' scores, Z = sum of exp(s1 - m) over them, their number; clears the column's output row
//   dense  one block per (KV head, 64 columns, share of the cached rows), per tile of 128 rows:
//            S2 = k2c . Q2^T                      (tcgen05, M = 128 rows, N = 64 columns, K = hd - r; Q2 as two bf16 terms)
//            W  = mask . exp(S1 - m) . softplus(S2)   (eight epilogue warps: tensor memory -> registers -> two bf16 terms in
//                                                  shared memory, written in the swizzled K-major layout the MMA reads)
//            O^T += V^T . W                       (tcgen05, M = 128 of the hd value columns, N = 64, K = 128 rows; V^T is the vc
//                                                  tile as it lands, read MN-major)
//          the accumulated O^T leaves as warp-wide reductions into o (a warp's 32 lanes are 32 consecutive floats of a row)
//   norm   (only without lsum) o /= Z
// Cached rows at or beyond the last token of the chunk may hold anything: their weights are zero by selection, and their vc
// rows are cleared in shared memory before the product (0 x NaN would poison the sum).
constexpr int kDN = 64;                          // columns per dense block
constexpr int kDSlotBytes = 32768;               // a k2c tile (<= 2 K chunks x 128 rows x 128 B) or 128 value columns of a vc tile
constexpr int kDSlots = 4;
constexpr int kDQBytes = 2 * 2 * kDN * 128;      // Q2: (hi, lo) x K chunks x 64 rows x 128 B
constexpr int kDWBytes = 2 * 2 * kDN * 128;      // W:  (hi, lo) x 2 chunks of 64 cached rows x 64 rows x 128 B; two such buffers
constexpr uint32_t kDCols = 256;                 // tensor memory: two S2 accumulators of 64 columns, two O^T tiles of 64
constexpr int kDEpiWarps = 16;
constexpr int kDThreads = 64 + kDEpiWarps * 32;  // warp 0: TMA, warp 1: MMA + tensor memory, warps 2..17: weights / output

struct DenseShared {
    unsigned long long full[kDSlots], empty[kDSlots];
    unsigned long long q_full, d1_full[2], d1_empty[2], w_full[2], w_empty[2], d2_full;
    uint32_t tmem;
    int abort_flag;
    int lo_min, n_max, n_all, lo_max, n_min;
    float4 info[kDN];
    float* orow[kDN];            // output row of each of the block's columns (nullptr: no such column)
};

__global__ void __launch_bounds__(256, 4) attn_chunk_stats_kernel(const ChunkParams p) {
    __shared__ double part[8][2];
    __shared__ float redf[8];
    __shared__ int redi[8];
    __shared__ float s_th, s_mx;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t = blockIdx.x / p.n_q, h = blockIdx.x - t * p.n_q;
    const int g = h / p.gq, col = t * p.gq + (h - g * p.gq);
    dep_wait();
    dep_trigger();
    const int lo = p.range[2 * t], n = p.range[2 * t + 1], L = n - lo;
    const float* scol = p.S + (static_cast<int64_t>(g) * kColMax + col) * p.scap;
    if (tid < p.hd) p.o[static_cast<int64_t>(blockIdx.x) * p.hd + tid] = 0.f;       // the dense kernel adds into it
    // The column's visible part stays in registers between the three sweeps: eight 16-byte loads per thread starting at the
    // 16-byte boundary at or below lo (rows outside [lo, n) read as -inf); longer columns are swept from L2 three times.
    constexpr int kKeep4 = 8;
    const int lo4 = lo & ~3;
    const bool kept = n - lo4 <= kKeep4 * 4 * 256;
    float keep[kKeep4][4];
    if (kept) {
#pragma unroll
        for (int u = 0; u < kKeep4; ++u) {
            const int j = lo4 + 4 * (256 * u + tid);
            float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
            if (j < n) v = __ldcg(reinterpret_cast<const float4*>(scol + j));      // the column is padded beyond the capacity
            keep[u][0] = (j >= lo && j < n) ? v.x : -INFINITY;
            keep[u][1] = (j + 1 >= lo && j + 1 < n) ? v.y : -INFINITY;
            keep[u][2] = (j + 2 >= lo && j + 2 < n) ? v.z : -INFINITY;
            keep[u][3] = (j + 3 >= lo && j + 3 < n) ? v.w : -INFINITY;
        }
    }
    float th = -INFINITY;
    if (p.k_attn < L) {
        // sums around the column's first value (keeps the fp32 partial sums accurate when |mean| >> std); fp64 above
        const float c0 = __ldcg(scol + lo);
        float f1 = 0.f, f2 = 0.f;
        if (kept) {
#pragma unroll
            for (int u = 0; u < kKeep4; ++u)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float d = keep[u][e] == -INFINITY ? 0.f : keep[u][e] - c0;
                    f1 += d;
                    f2 = fmaf(d, d, f2);
                }
        } else {
            for (int j = lo + tid; j < n; j += 256) {
                const float d = __ldcg(scol + j) - c0;
                f1 += d;
                f2 = fmaf(d, d, f2);
            }
        }
        const double s1 = warp_sum_f64(static_cast<double>(f1)), s2 = warp_sum_f64(static_cast<double>(f2));
        if (lane == 0) {
            part[warp][0] = s1;
            part[warp][1] = s2;
        }
        __syncthreads();
        if (tid == 0) {
            double a = 0.0, b = 0.0;
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                a += part[w][0];
                b += part[w][1];
            }
            const double dm = a / static_cast<double>(L);                  // mean - c0
            const double var = (b - a * dm) / static_cast<double>(L - 1);
            s_th = static_cast<float>(static_cast<double>(c0) + dm + sqrt(var > 0.0 ? var : 0.0) * p.zt[t]);
        }
        __syncthreads();
        th = s_th;
    }
    // the survivors: their number and their maximum, then the sum of their exponentials
    float mx = -INFINITY;
    int cnt = 0;
    if (kept) {
#pragma unroll
        for (int u = 0; u < kKeep4; ++u)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool on = keep[u][e] > th;
                mx = fmaxf(mx, on ? keep[u][e] : -INFINITY);
                cnt += on ? 1 : 0;
            }
    } else {
        for (int j = lo + tid; j < n; j += 256) {
            const float v = __ldcg(scol + j);
            if (v > th) {
                mx = fmaxf(mx, v);
                ++cnt;
            }
        }
    }
    mx = warp_max(mx);
    cnt = __reduce_add_sync(kFull, cnt);
    if (lane == 0) {
        redf[warp] = mx;
        redi[warp] = cnt;
    }
    __syncthreads();
    if (tid == 0) {
        float m = -INFINITY;
#pragma unroll
        for (int w = 0; w < 8; ++w) m = fmaxf(m, redf[w]);
        s_mx = m;
    }
    int total = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) total += redi[w];
    __syncthreads();
    mx = s_mx;
    float es = 0.f;
    if (kept) {
#pragma unroll
        for (int u = 0; u < kKeep4; ++u)
#pragma unroll
            for (int e = 0; e < 4; ++e) es += keep[u][e] > th ? __expf(keep[u][e] - mx) : 0.f;
    } else {
        for (int j = lo + tid; j < n; j += 256) {
            const float v = __ldcg(scol + j);
            if (v > th) es += __expf(v - mx);
        }
    }
    es = warp_sum(es);
    if (lane == 0) redf[warp] = es;
    __syncthreads();
    if (tid == 0) {
        float z = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) z += redf[w];
        p.colinfo[g * kColMax + col] = make_float4(th, mx, __int_as_float(lo), __int_as_float(n));
        p.zsum[blockIdx.x] = total > 0 ? z : 0.f;
        if (p.lsum != nullptr) p.lsum[blockIdx.x] = total > 0 ? z : 0.f;
        if (p.theta != nullptr) p.theta[blockIdx.x] = th;
        if (p.count != nullptr) p.count[blockIdx.x] = total;
    }
}

__global__ void __launch_bounds__(256) attn_chunk_norm_kernel(const ChunkParams p) {
    dep_wait();
    dep_trigger();
    const float z = p.zsum[blockIdx.x];
    if (threadIdx.x < p.hd) {
        float* o = p.o + static_cast<int64_t>(blockIdx.x) * p.hd + threadIdx.x;
        *o = z > 0.f ? *o / z : 0.f;
    }
}

__global__ void __launch_bounds__(kDThreads, 1)
attn_chunk_dense_kernel(const ChunkParams p, const __grid_constant__ CUtensorMap map_k2, const __grid_constant__ CUtensorMap map_v,
                        const __grid_constant__ CUtensorMap map_q2hi, const __grid_constant__ CUtensorMap map_q2lo, int nsplit) {
    extern __shared__ unsigned char tc_raw[];
    __shared__ DenseShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int d2 = p.hd - p.r, nk2 = d2 / kChunk, nvh = p.hd / 128;
    const int ncg = (p.ncol + kDN - 1) / kDN;
    const int grp = blockIdx.x / nsplit, part = blockIdx.x - grp * nsplit;
    const int g = grp / ncg, cg = grp - g * ncg;
    const int col0 = cg * kDN;                                  // first column of this block within the KV head
    if (tid == 0) {
        for (int s = 0; s < kDSlots; ++s) {
            mbar_init(smem_addr(&sh.full[s]), 1u);
            mbar_init(smem_addr(&sh.empty[s]), 1u);
        }
        mbar_init(smem_addr(&sh.q_full), 1u);
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_addr(&sh.d1_full[b]), 1u);
            mbar_init(smem_addr(&sh.d1_empty[b]), 1u);
            mbar_init(smem_addr(&sh.w_full[b]), 1u);
            mbar_init(smem_addr(&sh.w_empty[b]), 1u);
        }
        mbar_init(smem_addr(&sh.d2_full), 1u);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_addr(&sh.tmem), kDCols);
    dep_wait();                  // everything read here comes from the kernels ahead
    dep_trigger();
    if (tid < kDN) {
        const int col = col0 + tid;
        sh.info[tid] = col < p.ncol ? p.colinfo[g * kColMax + col] : make_float4(INFINITY, 0.f, __int_as_float(0), __int_as_float(0));
        const int t = col / p.gq, h = g * p.gq + (col - t * p.gq);
        sh.orow[tid] = col < p.ncol ? p.o + (static_cast<int64_t>(t) * p.n_q + h) * p.hd : nullptr;
    }
    if (tid == 0) {
        // rows any of this block's columns may see, and the end of what the chunk has written
        int lo_min = 0x7fffffff, n_max = 0, n_all = 0, lo_max = 0, n_min = 0x7fffffff;
        for (int t = 0; t < p.T; ++t) n_all = max(n_all, p.range[2 * t + 1]);
        const int c_end = min(p.ncol, col0 + kDN);
        for (int t = col0 / p.gq; t <= (c_end - 1) / p.gq; ++t) {
            lo_min = min(lo_min, p.range[2 * t]);
            n_max = max(n_max, p.range[2 * t + 1]);
            lo_max = max(lo_max, p.range[2 * t]);
            n_min = min(n_min, p.range[2 * t + 1]);
        }
        sh.lo_max = lo_max;
        sh.n_min = n_min;
        sh.lo_min = lo_min;
        sh.n_max = n_max;
        sh.n_all = n_all;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t base = (smem_addr(tc_raw) + 1023u) & ~1023u;
    const uint32_t qbase = base + kDSlots * kDSlotBytes, wbase = qbase + kDQBytes;
    unsigned char* wgen = tc_raw + (base - smem_addr(tc_raw)) + kDSlots * kDSlotBytes + kDQBytes;      // W, generic address
    unsigned char* ring_gen = tc_raw + (base - smem_addr(tc_raw));
    const uint32_t tmem = sh.tmem;
    volatile int* abort_flag = &sh.abort_flag;
    const int tile_lo = sh.lo_min / 128, tile_hi = (sh.n_max + 127) / 128, nt_all = max(0, tile_hi - tile_lo);
    const int ta = tile_lo + static_cast<int>(static_cast<int64_t>(part) * nt_all / nsplit);
    const int tb = tile_lo + static_cast<int>(static_cast<int64_t>(part + 1) * nt_all / nsplit);
    const int n = tb - ta;                                      // this block's tiles
    // ring items in the order both ends walk them: K(0), then per tile i: K(i + 1) if there is one, V(i, 0..nvh-1)
    if (warp == 0) {
        if (lane == 0 && n > 0) {
            tma_prefetch_desc(&map_k2);
            tma_prefetch_desc(&map_v);
            tma_prefetch_desc(&map_q2hi);
            tma_prefetch_desc(&map_q2lo);
            {
                const uint32_t bar = smem_addr(&sh.q_full);
                mbar_expect_tx(bar, static_cast<uint32_t>(2 * nk2) * kDN * 128);
                for (int kc = 0; kc < nk2; ++kc) {
                    tma_load_2d(qbase + kc * (kDN * 128), &map_q2hi, bar, kc * kChunk, g * kColMax + col0);
                    tma_load_2d(qbase + (nk2 + kc) * (kDN * 128), &map_q2lo, bar, kc * kChunk, g * kColMax + col0);
                }
            }
            int it = 0;
            bool ok = true;
            auto slot_for = [&](int item) -> bool {             // waits until the ring slot of `item` is free
                if (item >= kDSlots && !mbar_wait(smem_addr(&sh.empty[item % kDSlots]), ((item / kDSlots) & 1) ^ 1, abort_flag)) return false;
                return true;
            };
            auto load_k = [&](int i) {
                if (!(ok = ok && slot_for(it))) return;
                const uint32_t bar = smem_addr(&sh.full[it % kDSlots]), dst = base + (it % kDSlots) * kDSlotBytes;
                mbar_expect_tx(bar, static_cast<uint32_t>(nk2) * 128 * 128);
                for (int kc = 0; kc < nk2; ++kc)
                    tma_load_2d(dst + kc * (128 * 128), &map_k2, bar, kc * kChunk, static_cast<int>(g * p.cap + (ta + i) * 128));
                ++it;
            };
            auto load_v = [&](int i, int hh) {
                if (!(ok = ok && slot_for(it))) return;
                const uint32_t bar = smem_addr(&sh.full[it % kDSlots]), dst = base + (it % kDSlots) * kDSlotBytes;
                mbar_expect_tx(bar, 2u * 128 * 128);
                for (int b = 0; b < 2; ++b)
                    tma_load_2d(dst + b * (128 * 128), &map_v, bar, hh * 128 + b * kChunk, static_cast<int>(g * p.cap + (ta + i) * 128));
                ++it;
            };
            load_k(0);
            for (int i = 0; i < n && ok; ++i) {
                if (i + 1 < n) load_k(i + 1);
                for (int hh = 0; hh < nvh; ++hh) load_v(i, hh);
            }
            if (*abort_flag != 0) {            // let the copies in flight land before the block goes
                for (int i = max(0, it - kDSlots); i < it; ++i) {
                    const long long c0 = clock64();
                    while (!mbar_try(smem_addr(&sh.full[i % kDSlots]), (i / kDSlots) & 1))
                        if (clock64() - c0 > kTcSpinLimit) break;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && n > 0) {
            const uint32_t idesc1 = instr_desc(128, kDN, false), idesc2 = instr_desc(128, kDN, true);
            int it = 0;
            bool ok = mbar_wait(smem_addr(&sh.q_full), 0u, abort_flag);
            auto gemm1 = [&](int i) {          // S2 of tile i into accumulator i & 1
                const int b = i & 1;
                if (i >= 2) ok = ok && mbar_wait(smem_addr(&sh.d1_empty[b]), ((i >> 1) & 1) ^ 1, abort_flag);
                ok = ok && mbar_wait(smem_addr(&sh.full[it % kDSlots]), (it / kDSlots) & 1, abort_flag);
                if (!ok) return;
                tc_fence_after();
                const uint32_t a0 = base + (it % kDSlots) * kDSlotBytes;
                for (int tt = 0; tt < 2; ++tt)
                    for (int kc = 0; kc < nk2; ++kc)
#pragma unroll
                        for (int j = 0; j < kChunk / 16; ++j)
                            umma_bf16(tmem + b * kDN, smem_desc(a0 + kc * (128 * 128) + 32 * j, 0u, 1024u),
                                      smem_desc(qbase + (tt * nk2 + kc) * (kDN * 128) + 32 * j, 0u, 1024u), idesc1,
                                      (tt == 0 && kc == 0 && j == 0) ? 0u : 1u);
                umma_commit(smem_addr(&sh.empty[it % kDSlots]));
                umma_commit(smem_addr(&sh.d1_full[b]));
                ++it;
            };
            gemm1(0);
            for (int i = 0; i < n && ok; ++i) {
                if (i + 1 < n) gemm1(i + 1);
                ok = ok && mbar_wait(smem_addr(&sh.w_full[i & 1]), static_cast<uint32_t>((i >> 1) & 1), abort_flag);
                for (int hh = 0; hh < nvh && ok; ++hh) {
                    ok = mbar_wait(smem_addr(&sh.full[it % kDSlots]), (it / kDSlots) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t v0 = base + (it % kDSlots) * kDSlotBytes;
                    for (int tt = 0; tt < 2; ++tt)
#pragma unroll
                        for (int j = 0; j < 8; ++j)          // 16 cached rows per step: V^T MN-major (8-row groups 1024 B apart, next 64 columns 16 KB on)
                            umma_bf16(tmem + 2 * kDN + hh * kDN, smem_desc(v0 + j * 2048, 128 * 128, 1024u),
                                      smem_desc(wbase + (i & 1) * kDWBytes + (tt * 2 + (j >> 2)) * (kDN * 128) + 32 * (j & 3), 0u, 1024u), idesc2,
                                      (i == 0 && tt == 0 && j == 0) ? 0u : 1u);
                    umma_commit(smem_addr(&sh.empty[it % kDSlots]));
                    ++it;
                }
                if (ok) umma_commit(smem_addr(&sh.w_empty[i & 1]));
            }
            if (ok) umma_commit(smem_addr(&sh.d2_full));
        }
    } else if (n > 0) {
        // sixteen warps: four per tensor-memory lane quadrant, each with sixteen of the 64 columns
        const int q = warp & 3, part4 = (warp - 2) >> 2, cbase = 16 * part4;
        const int n_all = sh.n_all;
        bool ok = true;
        const int row = q * 32 + lane;                              // this thread's row of every tile
        const int etid = tid - 64;                                  // 0..511 among the sixteen warps
        // predictor scores of the thread's row for its 16 columns, requested one tile ahead
        float s1n[16];
        auto request_s1 = [&](int i) {
            const int tok = (ta + i) * 128 + row;
            const float* srow = p.S + (static_cast<int64_t>(g) * kColMax + col0 + cbase) * p.scap + tok;
#pragma unroll
            for (int c = 0; c < 16; ++c)
                s1n[c] = (tok < n_all && col0 + cbase + c < p.ncol) ? __ldcg(srow + static_cast<int64_t>(c) * p.scap) : -INFINITY;
        };
        request_s1(0);
        for (int i = 0; i < n && ok; ++i) {
            const int b = i & 1;
            const int tok = (ta + i) * 128 + row;
            float s1[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) s1[c] = s1n[c];
            if (i >= 2) ok = __all_sync(kFull, mbar_wait(smem_addr(&sh.w_empty[b]), static_cast<uint32_t>(((i >> 1) & 1) ^ 1), abort_flag));
            if (!ok) break;
            // W starts as zeros (64 bytes per thread); only the rows that pass are written below
            {
                uint4* wz = reinterpret_cast<uint4*>(wgen + b * kDWBytes) + etid * 4;
#pragma unroll
                for (int u = 0; u < 4; ++u) wz[u] = make_uint4(0u, 0u, 0u, 0u);
            }
            ok = __all_sync(kFull, mbar_wait(smem_addr(&sh.d1_full[b]), (i >> 1) & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            float s2[16];
            tmem_ld16(tmem + b * kDN + cbase + (static_cast<uint32_t>(q * 32) << 16), s2);
            asm volatile("bar.sync 1, %0;" ::"n"(kDEpiWarps * 32) : "memory");      // the zeros are in place
            // W[column][row] as two bf16 terms, K-major with the 128-byte swizzle: row `c` of a 64-row chunk holds 64 cached
            // rows; its 16-byte unit u sits at u ^ (c % 8)
            unsigned char* wchunk = wgen + b * kDWBytes + (row >> 6) * (kDN * 128);
            const int unit = (row & 63) >> 3, within = (row & 7) * 2;
            // a tile that every column of the block sees whole needs no range test per element
            const bool inner = (ta + i) * 128 >= sh.lo_max && (ta + i) * 128 + 128 <= sh.n_min;
            // no branch per element: the sixteen columns' arithmetic interleaves (a branch per column left every warp waiting
            // on its own chain of dependent instructions: 2.4 us per tile instead of 1)
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                const float4 ci = sh.info[cbase + c];
                const bool on = s1[c] > ci.x && (inner || (tok >= __float_as_int(ci.z) && tok < __float_as_int(ci.w)));
                // softplus(a) = max(a, 0) + log(1 + e), e = exp(-|a|): the hardware logarithm of 1 + e loses e below 1e-4
                const float e = __expf(-fabsf(s2[c]));
                const float l1p = e < 1e-4f ? e * (1.f - 0.5f * e) : __logf(1.f + e);
                const float w = __expf(fminf(s1[c] - ci.y, 0.f)) * (fmaxf(s2[c], 0.f) + l1p);
                const __nv_bfloat16 hi = __float2bfloat16_rn(w);
                const __nv_bfloat16 lo = __float2bfloat16_rn(w - __bfloat162float(hi));
                const int cr = cbase + c;
                const int off = (cr >> 3) * 1024 + (cr & 7) * 128 + ((unit ^ (cr & 7)) << 4) + within;
                if (on) {                   // three rows in a hundred
                    *reinterpret_cast<__nv_bfloat16*>(wchunk + off) = hi;
                    *reinterpret_cast<__nv_bfloat16*>(wchunk + 2 * (kDN * 128) + off) = lo;
                }
            }
            // value rows nobody has written yet: cleared once they have landed
            if ((ta + i) * 128 + 128 > n_all && tok >= n_all) {
                // items before V(i, 0): K(0), and for every earlier tile its K(next) and its nvh value pieces, then K(i + 1)
                for (int hh = part4; hh < nvh; hh += 4) {
                    const int item = 1 + i * (1 + nvh) + (i + 1 < n ? 1 : 0) + hh;
                    if (mbar_wait(smem_addr(&sh.full[item % kDSlots]), (item / kDSlots) & 1, abort_flag)) {
                        unsigned char* vs = ring_gen + (item % kDSlots) * kDSlotBytes + row * 128;
#pragma unroll
                        for (int bx = 0; bx < 2; ++bx)
#pragma unroll
                            for (int u = 0; u < 8; ++u) *reinterpret_cast<uint4*>(vs + bx * (128 * 128) + 16 * u) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
            }
            if (i + 1 < n) request_s1(i + 1);          // in flight across the hand-over below and the next tile's waits
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // generic writes -> the tensor core's reads
            tc_fence_before();
            asm volatile("bar.sync 1, %0;" ::"n"(kDEpiWarps * 32) : "memory");
            if (tid == 64) {
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&sh.w_full[b])) : "memory");
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(&sh.d1_empty[b])) : "memory");
            }
        }
        // the accumulated O^T: lane = value column; a warp takes sixteen (token, head) columns of one or two value tiles
        if (ok && __all_sync(kFull, mbar_wait(smem_addr(&sh.d2_full), 0u, abort_flag))) {
            tc_fence_after();
            for (int hh = 0; hh < nvh; ++hh) {
                float v[16];
                tmem_ld16(tmem + 2 * kDN + hh * kDN + cbase + (static_cast<uint32_t>(q * 32) << 16), v);
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    float* orow = sh.orow[cbase + c];
                    if (orow != nullptr) atomicAdd(orow + hh * 128 + q * 32 + lane, v[c]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_free(tmem, kDCols);
    }
    if (tid == 0 && sh.abort_flag != 0) atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_TIMEOUT);
}

}  // namespace

namespace spark {

// SPARK_ERR_WORKSPACE = shape or workspace not served by this path (the caller falls back to the per-query kernel).
int attn_chunk_launch(spark_ctx* ctx, const float* q, const void* k1c, const void* k2c, const void* vc, int64_t T, int64_t n_q,
                      int64_t n_kv, int64_t hd, int64_t r, int64_t cap, const int32_t* ctx_len, const double* zs, int64_t window,
                      int64_t k_attn, float* o, float* lsum, float* theta, int32_t* count, cudaStream_t stream) {
    const int64_t gq = n_q / n_kv, d2 = hd - r;
    if (T < 1 || T > 64 || T * gq > kColMax || (gq != 1 && gq != 2 && gq != 4 && gq != 8)) return SPARK_ERR_WORKSPACE;
    if ((r != 64 && r != 128) || d2 < 8 || d2 > 128 || (d2 & 7) != 0 || hd > 256 || (hd & 7) != 0) return SPARK_ERR_WORKSPACE;
    if ((cap & 3) != 0) return SPARK_ERR_WORKSPACE;          // 16-byte copies out of the score columns
    if (n_kv * cap >= (1LL << 31) || ((reinterpret_cast<uintptr_t>(k1c) | reinterpret_cast<uintptr_t>(k2c) | reinterpret_cast<uintptr_t>(vc)) & 15u) != 0)
        return SPARK_ERR_WORKSPACE;
    const size_t small_b = round_up(static_cast<size_t>(T) * (sizeof(double) + 2 * sizeof(int)), 1024);
    const size_t q_b = round_up(static_cast<size_t>(n_kv) * kColMax * r * 2, 1024);
    const size_t s_b = round_up(static_cast<size_t>(n_kv) * kColMax * (cap + 32) * 4, 1024);
    if (ctx->scratch == nullptr || ctx->scratch_bytes < kAttnCellBytes + small_b + 2 * q_b + s_b) return SPARK_ERR_WORKSPACE;
    // the dense second stage: enough columns per KV head that reading every row once beats gathering per query
    const size_t q2_b = round_up(static_cast<size_t>(n_kv) * kColMax * d2 * 2, 1024);
    const size_t info_b = round_up(static_cast<size_t>(n_kv) * kColMax * sizeof(float4) + static_cast<size_t>(T) * n_q * 4, 1024);
    const size_t smem_dense = static_cast<size_t>(kDSlots) * kDSlotBytes + kDQBytes + 2 * kDWBytes + 1024;
    // measured at the 2B head shape with 64-token chunks: ahead of the gather up to about 4096 visible rows (31 against 36 us
    // at 2048), level at 6000, behind beyond (its work grows with the rows, the gather's with k_attn); the caller's hint of
    // the current length decides, else the capacity
    int64_t rows_hint = ctx->len_hint > 0 ? ctx->len_hint : cap;
    if (window > 0 && window + T < rows_hint) rows_hint = window + T;          // a local layer sees no more than its window
    const bool dense = (ctx->chunk_dense == 2 || (ctx->chunk_dense == 1 && rows_hint <= 4160)) && T * gq >= 32 && (d2 == 64 || d2 == 128) && (hd == 128 || hd == 256) &&
                       ctx->scratch_bytes >= kAttnCellBytes + small_b + 2 * q_b + s_b + 2 * q2_b + info_b &&
                       smem_dense + sizeof(DenseShared) + 64 <= static_cast<size_t>(ctx->max_smem_optin);
    const size_t smem_scores = static_cast<size_t>(kChunkStages) * kChunkStageBytes + 1024;
    if (smem_scores + sizeof(ChunkShared) + 64 > static_cast<size_t>(ctx->max_smem_optin)) return SPARK_ERR_WORKSPACE;

    ChunkParams p;
    p.q = q; p.k2c = static_cast<const __nv_bfloat16*>(k2c); p.vc = static_cast<const __nv_bfloat16*>(vc);
    p.ctx_len = ctx_len; p.zs_in = zs;
    p.T = static_cast<int>(T); p.n_q = static_cast<int>(n_q); p.n_kv = static_cast<int>(n_kv); p.gq = static_cast<int>(gq);
    p.hd = static_cast<int>(hd); p.r = static_cast<int>(r);
    p.window = static_cast<int>(window > 0x7fffffff ? 0x7fffffff : window);
    p.k_attn = static_cast<int>(k_attn > 0x7fffffff ? 0x7fffffff : k_attn);
    p.ncol = static_cast<int>(T * gq);
    p.ncolp = (p.ncol + 15) & ~15;
    p.cap = cap;
    p.scap = cap + 32;
    p.o = o; p.lsum = lsum; p.theta = theta; p.count = count;
    char* w = ctx->scratch + kAttnCellBytes;
    p.zt = reinterpret_cast<double*>(w);
    p.range = reinterpret_cast<int*>(w + static_cast<size_t>(T) * sizeof(double)); w += small_b;
    p.qhi = reinterpret_cast<__nv_bfloat16*>(w); w += q_b;
    p.qlo = reinterpret_cast<__nv_bfloat16*>(w); w += q_b;
    p.S = reinterpret_cast<float*>(w); w += s_b;
    p.dense = dense ? 1 : 0;
    p.q2hi = reinterpret_cast<__nv_bfloat16*>(w); w += q2_b;
    p.q2lo = reinterpret_cast<__nv_bfloat16*>(w); w += q2_b;
    p.colinfo = reinterpret_cast<float4*>(w);
    p.zsum = reinterpret_cast<float*>(w + static_cast<size_t>(n_kv) * kColMax * sizeof(float4));
    p.hdr = ctx->hdr;

    CUtensorMap m_k1, m_qhi, m_qlo;
    if (!make_map(&m_k1, k1c, n_kv * cap, r, r, 128, true) || !make_map(&m_qhi, p.qhi, n_kv * kColMax, r, r, p.ncolp, false) ||
        !make_map(&m_qlo, p.qlo, n_kv * kColMax, r, r, p.ncolp, false))
        return SPARK_ERR_WORKSPACE;
    if (cudaFuncSetAttribute(attn_chunk_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_scores)) != cudaSuccess ||
        cudaFuncSetAttribute(attn_chunk_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sizeof(SelShared<true>))) != cudaSuccess ||
        cudaFuncSetAttribute(attn_chunk_select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(sizeof(SelShared<false>))) != cudaSuccess)
        return SPARK_ERR_CUDA;
    {
        void* args[] = {&p};
        if (launch_kernel(ctx, reinterpret_cast<const void*>(attn_chunk_prep_kernel), static_cast<unsigned>(n_kv * kColMax), 128, 0, stream, false, args) != cudaSuccess)
            return SPARK_ERR_CUDA;
    }
    {
        void* args[] = {&p, &m_k1, &m_qhi, &m_qlo};
        if (launch_kernel(ctx, reinterpret_cast<const void*>(attn_chunk_scores_kernel), static_cast<unsigned>(ctx->num_sms), kChunkThreads, smem_scores, stream, false, args) != cudaSuccess)
            return SPARK_ERR_CUDA;
    }
    if (dense) {
        CUtensorMap m_k2, m_v, m_q2hi, m_q2lo;
        if (!make_map(&m_k2, k2c, n_kv * cap, d2, d2, 128, true) || !make_map(&m_v, vc, n_kv * cap, hd, hd, 128, true) ||
            !make_map(&m_q2hi, p.q2hi, n_kv * kColMax, d2, d2, kDN, false) || !make_map(&m_q2lo, p.q2lo, n_kv * kColMax, d2, d2, kDN, false))
            return SPARK_ERR_WORKSPACE;
        if (cudaFuncSetAttribute(attn_chunk_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem_dense)) != cudaSuccess)
            return SPARK_ERR_CUDA;
        {
            void* args[] = {&p};
            if (launch_kernel(ctx, reinterpret_cast<const void*>(attn_chunk_stats_kernel), static_cast<unsigned>(T * n_q), 256, 0, stream, false, args) != cudaSuccess)
                return SPARK_ERR_CUDA;
        }
        const int groups = static_cast<int>(n_kv) * ((p.ncol + kDN - 1) / kDN);
        int nsplit = ctx->num_sms / groups;
        if (nsplit < 1) nsplit = 1;
        {
            void* args[] = {&p, &m_k2, &m_v, &m_q2hi, &m_q2lo, &nsplit};
            if (launch_kernel(ctx, reinterpret_cast<const void*>(attn_chunk_dense_kernel), static_cast<unsigned>(groups * nsplit), kDThreads, smem_dense, stream, false, args) != cudaSuccess)
                return SPARK_ERR_CUDA;
        }
        if (lsum == nullptr) {
            void* args[] = {&p};
            if (launch_kernel(ctx, reinterpret_cast<const void*>(attn_chunk_norm_kernel), static_cast<unsigned>(T * n_q), 256, 0, stream, false, args) != cudaSuccess)
                return SPARK_ERR_CUDA;
        }
        return SPARK_OK;
    }
    {
        void* args[] = {&p};
        // all blocks resident at three per SM: the register variant; more blocks than that: four per SM
        const bool regs = T * n_q <= 3 * static_cast<int64_t>(ctx->num_sms);
        const size_t sel_smem = regs ? sizeof(SelShared<true>) : sizeof(SelShared<false>);
        const void* sel = regs ? reinterpret_cast<const void*>(attn_chunk_select_kernel<true>) : reinterpret_cast<const void*>(attn_chunk_select_kernel<false>);
        if (launch_kernel(ctx, sel, static_cast<unsigned>(T * n_q), kSelThreads, sel_smem, stream, false, args) != cudaSuccess)
            return SPARK_ERR_CUDA;
    }
    return SPARK_OK;
}

}  // namespace spark
