// Dense projection for 5..64 tokens with bf16 weights on the fifth-generation tensor cores:
// y[b][:] = Wt . f(x[b][:]) (+ y_add[b][:]), f = optional division per group, optional RMSNorm -- the
// decoder layer's QKV and output projections for a batch or a chunk of a prompt.  Two kernels:
//   prep   f(x) -> two bf16 terms (x = hi + lo, 16 mantissa bits) in the workspace, padded to a multiple of 16 tokens;
//          y = y_add (or 0); the caller's clear-region side job
//   gemm   M = 128 output rows per tile, N = 2 x tokens (hi rows, lo rows of the token operand), K split over
//          the blocks of a tile so that every SM has one block; TMA-fed tcgen05.mma, accumulator in tensor
//          memory, epilogue adds the two halves and reduces into y (fp32 reductions)
// The weights do not depend on the kernel ahead: their first stages are requested before
// griddepcontrol.wait.  Same pipeline skeleton and bounded waits as the FFN chunk kernels (tc_common.cuh).
#include "kernels.h"
#include "tc_common.cuh"

using namespace spark;
using namespace spark::tc;

namespace {

constexpr int kGemmMaxTok = 64;
constexpr int kGemmRows = 128;
constexpr int kGemmWBytes = kGemmRows * kChunk * 2;            // 16 KB of weights per stage
constexpr int kGemmPrepSplit = 4;
// TOK = token rows of the operand tile a stage has room for (16: 8 stages of 20 KB; 64: 6 stages of 32 KB)
template <int TOK> struct GemmCfg {
    static constexpr int kStages = TOK <= 16 ? 8 : 6;
    static constexpr int kStageBytes = kGemmWBytes + 2 * TOK * kChunk * 2;
    static constexpr uint32_t kCols = TOK <= 16 ? 32 : 128;    // tensor-memory columns: hi | lo
};

struct GemmParams {
    const float* x;
    const float* norm_w;
    float eps;
    int B, n_in, n_out;
    const float* y_add;
    float* y;
    const float* x_div;
    int x_div_group;
    uint4* zero_ptr;
    int zero_n16;
    int ntok;                // B rounded up to a multiple of 16: rows of the operand boxes, half of the MMA's N
    __nv_bfloat16* xhi;      // [ntok][n_in]
    __nv_bfloat16* xlo;
    int ksplit, nchunks;
    WsHeader* hdr;
};

// Four blocks per (padded) token row, a quarter of the row each.
__global__ void __launch_bounds__(256) gemm_tc_prep_kernel(const GemmParams p) {
    __shared__ float red[8];
    const int n = blockIdx.x / kGemmPrepSplit, qr = blockIdx.x % kGemmPrepSplit, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_in = p.n_in, w4 = n_in / 4;
    const int q0 = static_cast<int>(static_cast<int64_t>(qr) * w4 / kGemmPrepSplit), q1 = static_cast<int>(static_cast<int64_t>(qr + 1) * w4 / kGemmPrepSplit);
    dep_wait();
    dep_trigger();
    for (int i = blockIdx.x * 256 + tid; i < p.zero_n16; i += gridDim.x * 256) p.zero_ptr[i] = make_uint4(0u, 0u, 0u, 0u);
    if (p.y_add != p.y) {            // y = y_add, or 0; when they alias y already holds the addend
        const int64_t total4 = static_cast<int64_t>(p.B) * p.n_out / 4;
        const float4* ya = reinterpret_cast<const float4*>(p.y_add);
        float4* yo = reinterpret_cast<float4*>(p.y);
        for (int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + tid; i < total4; i += static_cast<int64_t>(gridDim.x) * 256)
            yo[i] = ya != nullptr ? ya[i] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    uint2* hi = reinterpret_cast<uint2*>(p.xhi + static_cast<int64_t>(n) * n_in);
    uint2* lo = reinterpret_cast<uint2*>(p.xlo + static_cast<int64_t>(n) * n_in);
    if (n >= p.B) {                  // padding rows of the operand
        for (int i = q0 + tid; i < q1; i += 256) {
            hi[i] = make_uint2(0u, 0u);
            lo[i] = make_uint2(0u, 0u);
        }
        return;
    }
    const float4* xr = reinterpret_cast<const float4*>(p.x + static_cast<int64_t>(n) * n_in);
    auto divided = [&](int c4) -> float4 {
        float4 v = xr[c4];
        if (p.x_div != nullptr) {
            const float dv = p.x_div[static_cast<int64_t>(n) * (n_in / p.x_div_group) + (c4 * 4) / p.x_div_group];
            const float inv = dv > 0.f ? 1.f / dv : 0.f;
            v = make_float4(v.x * inv, v.y * inv, v.z * inv, v.w * inv);
        }
        return v;
    };
    float sc = 1.f;
    if (p.norm_w != nullptr) {       // every quarter sums the whole (divided) row
        float ss = 0.f;
        for (int i = tid; i < w4; i += 256) {
            const float4 v = divided(i);
            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        ss = warp_sum(ss);
        if (lane == 0) red[warp] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot += red[w];
        sc = rsqrtf(tot / static_cast<float>(n_in) + p.eps);
    }
    for (int i = q0 + tid; i < q1; i += 256) {
        float4 v = divided(i);
        if (p.norm_w != nullptr) {
            const float4 w = reinterpret_cast<const float4*>(p.norm_w)[i];
            v = make_float4(v.x * sc * w.x, v.y * sc * w.y, v.z * sc * w.z, v.w * sc * w.w);
        }
        const unsigned h01 = pack2_bf16(v.x, v.y), h23 = pack2_bf16(v.z, v.w);
        const unsigned l01 = pack2_bf16(v.x - __uint_as_float(h01 << 16), v.y - __uint_as_float(h01 & 0xffff0000u));
        const unsigned l23 = pack2_bf16(v.z - __uint_as_float(h23 << 16), v.w - __uint_as_float(h23 & 0xffff0000u));
        hi[i] = make_uint2(h01, h23);
        lo[i] = make_uint2(l01, l23);
    }
}

template <int TOK>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tc_kernel(const GemmParams p, const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_xhi,
               const __grid_constant__ CUtensorMap map_xlo) {
    extern __shared__ unsigned char tc_raw[];
    __shared__ TcShared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile = blockIdx.x / p.ksplit, ks = blockIdx.x - tile * p.ksplit;
    const int c0 = static_cast<int>(static_cast<int64_t>(ks) * p.nchunks / p.ksplit), c1 = static_cast<int>(static_cast<int64_t>(ks + 1) * p.nchunks / p.ksplit);
    const int nch = c1 - c0, row0 = tile * kGemmRows;
    constexpr int kGemmStages = GemmCfg<TOK>::kStages, kGemmStageBytes = GemmCfg<TOK>::kStageBytes;
    constexpr uint32_t kGemmCols = GemmCfg<TOK>::kCols;
    const uint32_t xbytes = static_cast<uint32_t>(p.ntok) * kChunk * 2;         // one term of one chunk of X
    const uint32_t base = tc_setup<kGemmStages>(sh, tc_raw, kGemmCols);
    const uint32_t tmem = sh.tmem;
    volatile int* abort_flag = &sh.abort_flag;
    dep_trigger();

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&map_w);
            tma_prefetch_desc(&map_xhi);
            tma_prefetch_desc(&map_xlo);
            auto load_w = [&](int i) {
                const int s = i % kGemmStages;
                const uint32_t bar = smem_addr(&sh.full[s]);
                mbar_expect_tx(bar, kGemmWBytes + 2 * xbytes);
                tma_load_2d(base + s * kGemmStageBytes, &map_w, bar, (c0 + i) * kChunk, row0);
            };
            auto load_x = [&](int i) {
                const int s = i % kGemmStages;
                const uint32_t bar = smem_addr(&sh.full[s]), dst = base + s * kGemmStageBytes + kGemmWBytes;
                tma_load_2d(dst, &map_xhi, bar, (c0 + i) * kChunk, 0);
                tma_load_2d(dst + xbytes, &map_xlo, bar, (c0 + i) * kChunk, 0);          // lo rows right behind the hi rows
            };
            const int pre = min(nch, kGemmStages);
            for (int i = 0; i < pre; ++i) load_w(i);      // the weights do not depend on the kernel ahead
            dep_wait();
            for (int i = 0; i < pre; ++i) load_x(i);
            int issued = pre;
            for (int i = pre; i < nch; ++i) {
                if (!mbar_wait(smem_addr(&sh.empty[i % kGemmStages]), ((i / kGemmStages) & 1) ^ 1, abort_flag)) break;
                load_w(i);
                load_x(i);
                issued = i + 1;
            }
            if (*abort_flag != 0) tc_drain<kGemmStages>(sh, issued);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(128, 2 * p.ntok, false);
            bool ok = true;
            for (int i = 0; i < nch && ok; ++i) {
                const int s = i % kGemmStages;
                ok = mbar_wait(smem_addr(&sh.full[s]), (i / kGemmStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a0 = base + s * kGemmStageBytes, b0 = a0 + kGemmWBytes;
#pragma unroll
                for (int j = 0; j < kChunk / 16; ++j)
                    umma_bf16(tmem, smem_desc(a0 + 32 * j, 0u, 1024u), smem_desc(b0 + 32 * j, 0u, 1024u), idesc, (i == 0 && j == 0) ? 0u : 1u);
                umma_commit(smem_addr(&sh.empty[s]));
            }
            if (ok) umma_commit(smem_addr(&sh.accum));
        }
    } else {
        const int q = warp & 3;                                    // tensor-memory lanes 32 q .. 32 q + 31
        dep_wait();
        if (nch > 0 && __all_sync(kFull, mbar_wait(smem_addr(&sh.accum), 0u, abort_flag))) {
            tc_fence_after();
            const uint32_t taddr = tmem + (static_cast<uint32_t>(q * 32) << 16);
            float* ycol = p.y + row0 + q * 32 + lane;
            float v[32];
            if (TOK <= 16) {
                tmem_ld32(taddr, v);                                              // columns 0..15 hi, 16..31 lo
#pragma unroll
                for (int n = 0; n < 16; ++n)
                    if (n < p.B) atomicAdd(ycol + static_cast<int64_t>(n) * p.n_out, v[n] + v[16 + n]);
            } else {
                float w[32];
                for (int hb = 0; hb * 32 < p.B; ++hb) {
                    tmem_ld32(taddr + hb * 32, v);
                    tmem_ld32(taddr + p.ntok + hb * 32, w);
#pragma unroll
                    for (int n = 0; n < 32; ++n)
                        if (hb * 32 + n < p.B) atomicAdd(ycol + static_cast<int64_t>(hb * 32 + n) * p.n_out, v[n] + w[n]);
                }
            }
        }
    }
    tc_finish(sh, kGemmCols, p.hdr);
}

}  // namespace

namespace spark {

// SPARK_ERR_WORKSPACE = shape or workspace not served by this path (the caller falls back).
int gemm_tc_launch(spark_ctx* ctx, const GemvArgs& a, cudaStream_t stream) {
    if (a.wdtype != SPARK_BF16 || a.B < 5 || a.B > kGemmMaxTok || a.n_in % kChunk != 0 || a.n_out % kGemmRows != 0) return SPARK_ERR_WORKSPACE;
    const int ntok = static_cast<int>((a.B + 15) & ~15);
    if ((reinterpret_cast<uintptr_t>(a.Wt) & 15u) != 0 || (reinterpret_cast<uintptr_t>(a.y) & 15u) != 0 ||
        (a.y_add != nullptr && (reinterpret_cast<uintptr_t>(a.y_add) & 15u) != 0))
        return SPARK_ERR_WORKSPACE;
    // the split input sits behind the attention's cells, where the FFN chunk path keeps its own (neither outlives its call)
    const size_t xb = round_up(static_cast<size_t>(ntok) * a.n_in * 2, 1024);
    if (ctx->scratch == nullptr || ctx->scratch_bytes < kAttnCellBytes + 2 * xb) return SPARK_ERR_WORKSPACE;
    const size_t smem = (ntok <= 16 ? static_cast<size_t>(GemmCfg<16>::kStages) * GemmCfg<16>::kStageBytes
                                    : static_cast<size_t>(GemmCfg<64>::kStages) * GemmCfg<64>::kStageBytes) + 1024;
    if (smem + sizeof(TcShared) + 64 > static_cast<size_t>(ctx->max_smem_optin)) return SPARK_ERR_WORKSPACE;

    GemmParams p;
    p.x = a.x; p.norm_w = a.norm_w; p.eps = a.rms_eps;
    p.B = static_cast<int>(a.B); p.n_in = static_cast<int>(a.n_in); p.n_out = static_cast<int>(a.n_out);
    p.y_add = a.y_add; p.y = a.y;
    p.x_div = a.x_div; p.x_div_group = static_cast<int>(a.x_div ? a.x_div_group : 1);
    p.zero_ptr = static_cast<uint4*>(a.zero_ptr); p.zero_n16 = static_cast<int>(a.zero_bytes / 16);
    p.ntok = ntok;
    p.xhi = reinterpret_cast<__nv_bfloat16*>(ctx->scratch + kAttnCellBytes);
    p.xlo = reinterpret_cast<__nv_bfloat16*>(ctx->scratch + kAttnCellBytes + xb);
    const int tiles = static_cast<int>(a.n_out / kGemmRows);
    p.nchunks = static_cast<int>(a.n_in / kChunk);
    p.ksplit = ctx->num_sms / tiles > 0 ? ctx->num_sms / tiles : 1;
    if (p.ksplit > p.nchunks) p.ksplit = p.nchunks;
    p.hdr = ctx->hdr;

    CUtensorMap m_w, m_xhi, m_xlo;
    if (!make_map(&m_w, a.Wt, a.n_out, a.n_in, a.n_in, kGemmRows, true) || !make_map(&m_xhi, p.xhi, ntok, a.n_in, a.n_in, ntok, false) ||
        !make_map(&m_xlo, p.xlo, ntok, a.n_in, a.n_in, ntok, false))
        return SPARK_ERR_WORKSPACE;
    const void* kern = ntok <= 16 ? reinterpret_cast<const void*>(gemm_tc_kernel<16>) : reinterpret_cast<const void*>(gemm_tc_kernel<64>);
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) return SPARK_ERR_CUDA;
    {
        void* args[] = {&p};
        if (launch_kernel(ctx, reinterpret_cast<const void*>(gemm_tc_prep_kernel), static_cast<unsigned>(ntok * kGemmPrepSplit), 256, 0, stream, false, args) != cudaSuccess)
            return SPARK_ERR_CUDA;
    }
    {
        void* args[] = {&p, &m_w, &m_xhi, &m_xlo};
        if (launch_kernel(ctx, kern, static_cast<unsigned>(tiles * p.ksplit), kTcThreads, smem, stream, false, args) != cudaSuccess)
            return SPARK_ERR_CUDA;
    }
    return SPARK_OK;
}

}  // namespace spark
