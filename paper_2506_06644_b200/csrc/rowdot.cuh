// Streaming "rows times a few vectors" kernel body shared by the Spark FFN predictor and the
// dense GEMV: out[j][t] = W[row0 + j][:] . xs[t][:] for the nloc rows a block owns.
#pragma once

#include "common.cuh"

namespace spark {

// W: row-major weights with `ld` elements per row; xs: [TB][xw] fp32 in shared memory holding the
// first nck*8 elements of every token's input.  A warp works on RW rows at once; every 16-byte
// load of a batch (CU chunks x RW rows per lane) is issued before the first use so that a block
// keeps its whole share of the matrix in flight.  With TB >= 16 the two half-warps take eight
// tokens each.  emit(j, t, value) is called by exactly one lane per (row, token).
// before_use() is called exactly once by every thread of the block, after the first batch of
// weight loads has been issued and before anything is read from xs: the caller fills xs there
// (and synchronises the block), so that the input's latency hides behind the weights'.
// after_first() is called exactly once by every thread as well, just before: a kernel that may
// start under the tail of the kernel before it waits for that kernel there and requests its input.
// (Waiting earlier, after the first quarter of the batch, so that the input queues behind fewer
// weight requests, measured slower: the rest of the batch then cannot fly during the wait.)
// Must be called by all threads of a 512-thread block.  rows_dot_mapped takes the row of the weight
// matrix for each of the block's nloc logical rows from rowmap(j) and hands the RW values of a
// warp's row group to emit_group(group, token, values) together.
template <typename WT, int TB, int RW, typename RowMap, typename Pre, typename Hook, typename EmitGroup>
__device__ __forceinline__ void rows_dot_mapped(const WT* __restrict__ W, int64_t ld, int nloc, int nck, const float* xs,
                                                int xw, RowMap rowmap, Pre after_first, Hook before_use, EmitGroup emit_group) {
    constexpr int kWarpsPerBlock = 16;
    constexpr int TS = TB >= 16 ? 2 : 1;     // lane groups that split the tokens
    constexpr int TPL = TB / TS;             // tokens per lane group
    constexpr int GL = 32 / TS;              // lanes per group
    // chunks per lane held in flight per batch (upper bound); the batches of a row are made equal
    constexpr int CU = (TB == 1 ? (RW >= 4 ? 4 : (RW == 2 ? 10 : 8)) : (TB <= 4 && RW == 4 && sizeof(WT) == 2 ? 4 : 2)) / (sizeof(WT) == 4 ? 2 : 1);
    const int per_lane = (nck + GL - 1) / GL;
    const int nbatch = (per_lane + CU - 1) / CU;
    const int cu = nbatch > 0 ? (per_lane + nbatch - 1) / nbatch : 1;      // <= CU
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int lg = lane / GL, gl = lane % GL;
    bool hooked = false;
    int rg = warp;
#pragma unroll 1
    do {
        const bool has = rg * RW < nloc;
        float acc[RW][TPL];
#pragma unroll
        for (int i = 0; i < RW; ++i)
#pragma unroll
            for (int t = 0; t < TPL; ++t) acc[i][t] = 0.f;
        const WT* rowp[RW];
#pragma unroll
        for (int i = 0; i < RW; ++i) {
            const int j = rg * RW + i;
            rowp[i] = W + static_cast<int64_t>(rowmap(j < nloc ? j : (nloc > 0 ? nloc - 1 : 0))) * ld;
        }
#pragma unroll 1
        for (int c0 = 0; c0 < nck; c0 += GL * cu) {
            Row8<WT> w[CU][RW];
#pragma unroll
            for (int u = 0; u < CU; ++u) {
                const int c = c0 + u * GL + gl;
#pragma unroll
                for (int i = 0; i < RW; ++i) {
                    if (has && u < cu && c < nck) w[u][i].load_pinned(rowp[i], c);
                    else w[u][i].zero();
                }
                if (u == CU - 1 && !hooked) after_first();
            }
            if (!hooked) {
                before_use();
                hooked = true;
            }
            if (!has) break;
#pragma unroll
            for (int u = 0; u < CU; ++u) {
                const int c = c0 + u * GL + gl;
                const int cs = (u < cu && c < nck) ? c : 0;          // zero weights meet a valid x address
                float wf[RW][8];
#pragma unroll
                for (int i = 0; i < RW; ++i) w[u][i].unpack(wf[i]);
#pragma unroll
                for (int t = 0; t < TPL; ++t) {
                    const float4* xr = reinterpret_cast<const float4*>(xs + static_cast<size_t>(lg * TPL + t) * xw) + 2 * cs;
                    const float4 xa = xr[0], xb = xr[1];
#pragma unroll
                    for (int i = 0; i < RW; ++i) acc[i][t] = dot8(wf[i], xa, xb, acc[i][t]);
                }
            }
        }
        if (has) {
#pragma unroll
            for (int t = 0; t < TPL; ++t) {
                float v[RW];
#pragma unroll
                for (int i = 0; i < RW; ++i) {
                    v[i] = acc[i][t];
#pragma unroll
                    for (int o = GL / 2; o > 0; o >>= 1) v[i] += __shfl_xor_sync(kFull, v[i], o);
                }
                if (gl == 0) emit_group(rg, lg * TPL + t, v);
            }
        }
        rg += kWarpsPerBlock;
    } while (rg * RW < nloc);
}

// The common case: the block owns the contiguous rows [row0, row0 + nloc); emit(j, t, value) is
// called by exactly one lane per (row, token).
template <typename WT, int TB, int RW, typename Pre, typename Hook, typename Emit>
__device__ __forceinline__ void rows_dot(const WT* __restrict__ W, int64_t ld, int row0, int nloc, int nck,
                                         const float* xs, int xw, Pre after_first, Hook before_use, Emit emit) {
    rows_dot_mapped<WT, TB, RW>(
        W, ld, nloc, nck, xs, xw, [&](int j) { return row0 + j; }, after_first, before_use,
        [&](int rg, int t, const float (&v)[RW]) {
#pragma unroll
            for (int i = 0; i < RW; ++i)
                if (rg * RW + i < nloc) emit(rg * RW + i, t, v[i]);
        });
}

}  // namespace spark
