// Tensor-core building blocks shared by the batched kernels (Spark FFN for 5..64 tokens, dense GEMV for
// 5..16 tokens): mma.sync m16n8k16 bf16 with fp32 accumulation; activations as an error-compensated two-term
// bf16 split in shared memory; weight fragments straight from global memory.
#pragma once

#include "common.cuh"

namespace spark {
namespace mma {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / kWarp;

__device__ __forceinline__ void mma_bf16(float (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3,
                                         unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi) {      // {bf16(lo) in bits 0-15, bf16(hi) in bits 16-31}
    unsigned r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ unsigned short bf16_bits(float f) { return __bfloat16_as_ushort(__float2bfloat16_rn(f)); }
__device__ __forceinline__ float bf16_val(unsigned short b) { return __uint_as_float(static_cast<unsigned>(b) << 16); }

// Shared-memory plan of the kernel (element counts), computed the same way on host and device.
struct Plan {
    int xs;        // row stride (bf16 elements) of the split activations: = 32 mod 64 keeps 16-byte fragment reads conflict-free
    int us;        // row stride (bf16 elements) of the split u values: = 8 mod 64
    __host__ __device__ Plan(int xw, int rpc) {
        xs = pad(xw);
        us = ((rpc + 15 + 63) / 64) * 64 + 8;
    }
    __host__ __device__ static int pad(int w) { return ((w + 63) / 64) * 64 + 32; }
    // bf16 elements of the activation region (two split parts).  Resident: x[:r] and x[r:] side by side, staged
    // once; otherwise one area that x[r:] takes over from x[:r] between the phases.
    __host__ __device__ static size_t region(bool resident, int tb, int r, int d2) {
        return resident ? static_cast<size_t>(2) * tb * (pad(r) + pad(d2)) : static_cast<size_t>(2) * tb * pad(r > d2 ? r : d2);
    }
};

// S[tile rows][tokens] = W[rows] . X^T for the block's row tiles.  rowptr(i) gives the weight row of
// the block's i-th row (i < nrows) -- rows beyond nrows contribute zeros.  The split activations
// xs3[part][token][xs] (two parts) cover K = 32 * nch columns.  emit(i, token, value) is called once per
// (row, token) by some thread.  Called by the whole block; ends with a block sync.
template <int NT, int CB, typename RowPtr, typename Emit>
__device__ __forceinline__ void mma_rows(RowPtr rowptr, int nrows, int nch, const __nv_bfloat16* xs3, int xs, int tb_stride,
                                         float4* part, Emit emit) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int MT = (nrows + 15) >> 4;
    for (int mt0 = 0; mt0 < MT; mt0 += kWarps) {
        const int mtn = min(kWarps, MT - mt0);                 // tiles in this group
        int tp = 1;
        while (tp < mtn) tp <<= 1;
        const int ks = kWarps / tp;                            // warps that split K for one tile
        const int tile = warp / ks, kp = warp - tile * ks;
        const bool active = tile < mtn;
        const int r_lo = (mt0 + tile) * 16 + g, r_hi = r_lo + 8;
        const __nv_bfloat16* p_lo = (active && r_lo < nrows) ? rowptr(r_lo) : nullptr;
        const __nv_bfloat16* p_hi = (active && r_hi < nrows) ? rowptr(r_hi) : nullptr;
        float acc[NT][4];
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[n][e] = 0.f;
        // CB chunks per batch: 2 * CB loads of 16 bytes in flight per lane
#pragma unroll 1
        for (int c0 = kp; c0 < nch; c0 += ks * CB) {
            uint4 alo[CB], ahi[CB];
#pragma unroll
            for (int u = 0; u < CB; ++u) {
                const int c = c0 + u * ks;
                alo[u] = (p_lo != nullptr && c < nch) ? ld_stream16(reinterpret_cast<const uint4*>(p_lo) + 4 * c + t) : make_uint4(0u, 0u, 0u, 0u);
                ahi[u] = (p_hi != nullptr && c < nch) ? ld_stream16(reinterpret_cast<const uint4*>(p_hi) + 4 * c + t) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < CB; ++u) {
                const int c = c0 + u * ks;
                if (c < nch && active) {
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
#pragma unroll
                        for (int sp = 0; sp < 2; ++sp) {
                            const uint4 b = *reinterpret_cast<const uint4*>(xs3 + static_cast<size_t>(sp) * tb_stride +
                                                                            static_cast<size_t>(n * 8 + g) * xs + 32 * c + 8 * t);
                            mma_bf16(acc[n], alo[u].x, ahi[u].x, alo[u].y, ahi[u].y, b.x, b.y);
                            mma_bf16(acc[n], alo[u].z, ahi[u].z, alo[u].w, ahi[u].w, b.z, b.w);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int n = 0; n < NT; ++n) part[(warp * NT + n) * 32 + lane] = make_float4(acc[n][0], acc[n][1], acc[n][2], acc[n][3]);
        __syncthreads();
        // sum the K-splits: value index = (tile, n, lane, e)
        for (int i = tid; i < mtn * NT * 128; i += kThreads) {
            const int e = i & 3, ln = (i >> 2) & 31, n = (i >> 7) % NT, tl = i / (128 * NT);
            float v = 0.f;
            for (int k = 0; k < ks; ++k) v += reinterpret_cast<const float*>(&part[((tl * ks + k) * NT + n) * 32 + ln])[e];
            const int row = (mt0 + tl) * 16 + (ln >> 2) + ((e & 2) ? 8 : 0);
            const int tok = n * 8 + (ln & 3) * 2 + (e & 1);
            if (row < nrows) emit(row, tok, v);
        }
        __syncthreads();
    }
}


}  // namespace mma
}  // namespace spark
