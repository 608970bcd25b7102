// Spark FFN (Section 2.1, Eq. 2) for 2..16 tokens per pass with bf16 weights: the three products
// become small GEMMs (neurons x tokens), so they run on the tensor cores while the kernel stays
// HBM-bound.  One cooperative kernel, one 512-thread block per SM, same phases as the one-token
// kernel:
//   A   S = K1t[rows of the block] . X[:, :r]^T         16-row tiles x 8-token tiles, K = r
//   S   score sums into the grid-wide cells, theta per token (Eq. 11)
//   C   per-token masks and the union list of the block's neurons (Appendix B: the union gates the
//       loads, each token's own mask gates what enters its output)
//   D1  T = K2t[union rows] . X[:, r:]^T, U = mask * GELU(S - theta) * T
//   D2  Y^T += U . Vt[union rows]                          tokens x 64-column blocks, K = union rows
// Tensor-core use: mma.sync m16n8k16 bf16 with fp32 accumulation.  The fp32 activations enter as an
// error-compensated two-term bf16 split (x = hi + lo, 16 mantissa bits, one MMA per term): the scores
// decide index sets, and a bare bf16 rounding of x (2^-9 relative) would move them far outside the
// band in which the sets may differ, whereas the two-term split moves them by about 1e-5 of their
// spread, a tenth of that band; u enters D2 the same way.  Both halves of the split input, x[:r] and
// x[r:], are staged once at the start when they fit side by side.  Weight fragments are loaded
// straight from global memory with 16-byte loads: the k-slots of an MMA may be any permutation of
// the columns as long as both operands use the same one, so a lane's 8 consecutive bf16 of a row feed
// two MMAs without any shuffle.  (The contraction is far too small for tcgen05 tiles: M = 16 rows,
// N = 8 tokens; the kernel's time is the HBM stream.)
#include "ffn_params.h"
#include "kernels.h"
#include "mma_rows.cuh"

using namespace spark;
using namespace spark::mma;

namespace {

template <int TB>
__global__ void __launch_bounds__(kThreads, 1) ffn_mma_kernel(const FfnParams p) {
    constexpr int NT = TB / 8;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const Plan plan(p.xw, p.rpc);
    const int xs = plan.xs, us = plan.us, rpc = p.rpc;
    const bool xres = p.xres != 0;
    const int xs1 = xres ? Plan::pad(p.r) : xs, xs2 = xres ? Plan::pad(p.d - p.r) : xs;   // row strides of x[:r] and x[r:]
    const int tb_stride = TB * xs1, tb_stride2 = TB * xs2;                           // one split part of each
    const size_t region = Plan::region(xres, TB, p.r, p.d - p.r);
    __nv_bfloat16* xs3 = reinterpret_cast<__nv_bfloat16*>(smem_raw);                 // [2][TB][xs1]: x[:r]
    __nv_bfloat16* xr2 = xres ? xs3 + 2 * tb_stride : xs3;                           // [2][TB][xs2]: x[r:]
    __nv_bfloat16* u2 = xs3 + region;                                                // [2][16][us]
    float4* part = reinterpret_cast<float4*>(u2 + 2 * 16 * us);                      // [kWarps][NT][32]
    float* s_loc = reinterpret_cast<float*>(part + kWarps * NT * 32);                // [TB][rpc]
    int* ulist = reinterpret_cast<int*>(s_loc + static_cast<size_t>(TB) * rpc);      // [rpc]
    unsigned* amask = reinterpret_cast<unsigned*>(ulist + rpc);                      // [rpc]
    __shared__ float rstd[16];
    __shared__ float theta_s[16];
    __shared__ int wcnt[kWarps];
    __shared__ unsigned tok_any;
    __shared__ unsigned s_epoch;
    __shared__ int s_fail;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int grid = gridDim.x, cta = blockIdx.x;
    const int row0 = static_cast<int>(static_cast<int64_t>(cta) * p.d_ff / grid);
    const int row1 = static_cast<int>(static_cast<int64_t>(cta + 1) * p.d_ff / grid);
    const int nloc = row1 - row0;
    const int d = p.d, r = p.r, d2 = d - r;
    const __nv_bfloat16* K1t = static_cast<const __nv_bfloat16*>(p.K1t);
    const __nv_bfloat16* K2t = static_cast<const __nv_bfloat16*>(p.K2t);
    const __nv_bfloat16* Vt = static_cast<const __nv_bfloat16*>(p.Vt);
    dep_wait();        // these kernels read the batch's inputs first: nothing to do ahead of the dependency
    dep_trigger();
    if (tid == 0) {
        s_epoch = ld_acquire_u32(&p.hdr->epoch);
        s_fail = 0;
    }
    if (cta == 0) {      // clear the cells the launch after next will use (last used two launches ago)
        const unsigned e = ld_acquire_u32(&p.hdr->epoch);
        SumCell* c = &p.hdr->ffn_cells[(e + 2u) & 3u][0][0][0];
        for (int i = tid; i < 4 * 16 * kCellWays; i += kThreads) { c[i].s1 = 0.0; c[i].s2 = 0.0; c[i].count = 0u; }
    }
    p.trace.mark(0);

    for (int g0 = 0, grp = 0; g0 < p.B; g0 += TB, ++grp) {
        const int tbv = min(TB, p.B - g0);
        const float* xg = p.x + static_cast<int64_t>(g0) * d;
        float* yg = p.y + static_cast<int64_t>(g0) * d;

        // ---- prologue: RMSNorm scale, y initialisation, x[:r] split into shared memory ---------------
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
        // split x[t][col0:col0+width] (normalised) into two bf16 parts (hi + lo carry 16 mantissa bits: scores move by
        // about 1e-5 of their spread, a tenth of the band inside which the index sets may differ)
        auto stage = [&](int col0, int width, __nv_bfloat16* dst0, int stride) {
            const int w4 = width / 4;
            const int part_stride = TB * stride;
            constexpr int SB = 8;                    // loads a thread keeps in flight
            for (int i0 = tid; i0 < TB * w4; i0 += kThreads * SB) {
                float4 v[SB], w[SB];
                int tt[SB], cc[SB];
#pragma unroll
                for (int j = 0; j < SB; ++j) {
                    const int i = i0 + j * kThreads;
                    tt[j] = i / w4;
                    cc[j] = i - tt[j] * w4;
                    v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                    w[j] = make_float4(1.f, 1.f, 1.f, 1.f);
                    if (i < TB * w4 && tt[j] < tbv) {
                        v[j] = reinterpret_cast<const float4*>(xg + static_cast<int64_t>(tt[j]) * d + col0)[cc[j]];
                        if (p.norm_w != nullptr) w[j] = reinterpret_cast<const float4*>(p.norm_w + col0)[cc[j]];
                    }
                }
#pragma unroll
                for (int j = 0; j < SB; ++j) {
                    const int i = i0 + j * kThreads;
                    if (i >= TB * w4) break;
                    const float sc = (p.norm_w != nullptr && tt[j] < tbv) ? rstd[tt[j]] : 1.f;
                    const float f[4] = {v[j].x * sc * w[j].x, v[j].y * sc * w[j].y, v[j].z * sc * w[j].z, v[j].w * sc * w[j].w};
                    // two values per conversion: hi = bf16x2(f), lo = bf16x2(f - hi); a bf16 widens by a 16-bit shift
                    const unsigned h01 = pack_bf16x2(f[0], f[1]), h23 = pack_bf16x2(f[2], f[3]);
                    const unsigned m01 = pack_bf16x2(f[0] - __uint_as_float(h01 << 16), f[1] - __uint_as_float(h01 & 0xffff0000u));
                    const unsigned m23 = pack_bf16x2(f[2] - __uint_as_float(h23 << 16), f[3] - __uint_as_float(h23 & 0xffff0000u));
                    __nv_bfloat16* dst = dst0 + static_cast<size_t>(tt[j]) * stride + 4 * cc[j];
                    *reinterpret_cast<uint2*>(dst) = make_uint2(h01, h23);
                    *reinterpret_cast<uint2*>(dst + part_stride) = make_uint2(m01, m23);
                }
            }
        };
        stage(0, r, xs3, xs1);
        if (xres) stage(r, d2, xr2, xs2);
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

        // ---- phase A: predictor scores of this block's neurons (zero-padded K when r % 32 != 0) ------
        mma_rows<NT, 8>([&](int i) { return K1t + static_cast<int64_t>(row0 + i) * r; }, nloc, r / 32, xs3, xs1, tb_stride, part,
                     [&](int i, int tok, float v) { s_loc[static_cast<size_t>(tok) * rpc + i] = v; });
        p.trace.mark(2);

        // ---- score sums into the token's cells, arrival released after them ------------------------------
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
            if (lane == 0) cells_add_sums_w<kCellWays>(cells + t * kCellWays, cta, s1, s2);
        }
        p.trace.mark(3);
        __syncthreads();
        if (tid == 0) cells_arrive_w<kCellWays>(cells, cta);      // one arrival for the group, after every token's sums
        if (!xres) stage(r, d2, xr2, xs2);              // x[r:] replaces x[:r] while the cells fill
        for (int i = tid; i < 2 * 16 * us / 2; i += kThreads) reinterpret_cast<unsigned*>(u2)[i] = 0u;
        if (warp == 0) {
            const bool ok = cells_wait_arrivals_w<kCellWays>(cells, static_cast<unsigned>(grid), p.hdr);
            if (lane == 0 && !ok) s_fail = 1;
        }
        __syncthreads();
        if (s_fail) return;
        for (int t = warp; t < tbv; t += kWarps) {
            double sa, sb;
            cells_read_w<kCellWays>(cells + t * kCellWays, sa, sb);
            if (lane == 0) {
                float th = -INFINITY;
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

        // ---- phase C: masks and the ordered union list of this block's neurons --------------------------
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
        p.trace.mark(5);

        // ---- D1: T = K2t[union rows] . X[:, r:]^T; U = mask * GELU(S - theta) * T, split in two bf16 parts
        mma_rows<NT, 10>([&](int i) { return K2t + static_cast<int64_t>(row0 + ulist[i]) * d2; }, nU, d2 / 32, xr2, xs2, tb_stride2, part,
                     [&](int i, int tok, float tv) {
                         const int j = ulist[i];
                         float u = 0.f;
                         if ((amask[j] >> tok) & 1u) {
                             const float a = s_loc[static_cast<size_t>(tok) * rpc + j] - (p.identity ? 0.f : theta_s[tok]);
                             u = (p.erf_form ? gelu_erf(a) : gelu_tanh(a)) * tv;
                         }
                         const unsigned short h = bf16_bits(u);
                         u2[static_cast<size_t>(tok) * us + i] = __ushort_as_bfloat16(h);
                         u2[static_cast<size_t>(16 + tok) * us + i] = __float2bfloat16_rn(u - bf16_val(h));
                     });
        p.trace.mark(6);

        // ---- D2: Y^T += U . Vt[union rows].  The union rows are staged stripe by stripe into the shared
        //      memory the activation splits no longer need (cp.async: every thread's requests are in flight
        //      at once, no registers held), B fragments come out of it with ldmatrix.trans, a warp owns
        //      64-column blocks, K = union rows in steps of 16.
        {
            const int g = lane >> 2, t = lane & 3;
            const unsigned anyt = tok_any;
            const int nUp = (nU + 15) & ~15, nks = nUp >> 4;
            unsigned char* vs = smem_raw;                                  // reuses xs3
            const int sv_bytes = static_cast<int>(region) * 2;
            // two staging buffers: the next stripe's rows are requested while the current one is multiplied
            int WC = nUp > 0 ? (((sv_bytes / 2 / nUp) - 16) / 2) & ~63 : 0;
            if (WC > ((d + 63) & ~63)) WC = (d + 63) & ~63;
            const int RS = WC * 2 + 16;                                    // row stride: 16 mod 128 bytes
            const unsigned vs_base = static_cast<unsigned>(__cvta_generic_to_shared(vs));
            if (nU > 0 && WC >= 64) {
                auto request = [&](int col0, int buf) {
                    const int wc = min(WC, d - col0), nch8 = wc >> 3;
                    unsigned char* vb = vs + static_cast<size_t>(buf) * nUp * RS;
                    const unsigned va = vs_base + buf * nUp * RS;
                    for (int row = warp; row < nUp; row += kWarps) {       // a warp per row, lanes over 16-byte pieces
                        if (row < nU) {
                            const __nv_bfloat16* src = Vt + static_cast<int64_t>(row0 + ulist[row]) * d + col0;
                            for (int ch = lane; ch < nch8; ch += 32)
                                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(va + row * RS + ch * 16), "l"(src + ch * 8) : "memory");
                        } else {
                            for (int ch = lane; ch < nch8; ch += 32)
                                *reinterpret_cast<uint4*>(vb + row * RS + ch * 16) = make_uint4(0u, 0u, 0u, 0u);
                        }
                    }
                    asm volatile("cp.async.commit_group;" ::: "memory");
                };
                request(0, 0);
                int buf = 0;
                for (int col0 = 0; col0 < d; col0 += WC, buf ^= 1) {
                    const int wc = min(WC, d - col0);
                    if (col0 + WC < d) {
                        request(col0 + WC, buf ^ 1);
                        asm volatile("cp.async.wait_group 1;" ::: "memory");
                    } else {
                        asm volatile("cp.async.wait_group 0;" ::: "memory");
                    }
                    __syncthreads();
                    const unsigned vs_addr = vs_base + buf * nUp * RS;
                    const int nblk = (wc + 63) >> 6;
                    for (int cb = warp; cb < nblk; cb += kWarps) {
                        float acc[8][4];
#pragma unroll
                        for (int i = 0; i < 8; ++i)
#pragma unroll
                            for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
#pragma unroll 1
                        for (int ks = 0; ks < nks; ++ks) {
                            const int kb = ks * 16;
                            unsigned a[2][4];
#pragma unroll
                            for (int sp = 0; sp < 2; ++sp) {
                                const __nv_bfloat16* ub = u2 + static_cast<size_t>(sp * 16) * us + kb + 2 * t;
                                a[sp][0] = *reinterpret_cast<const unsigned*>(ub + static_cast<size_t>(g) * us);
                                a[sp][1] = TB > 8 ? *reinterpret_cast<const unsigned*>(ub + static_cast<size_t>(g + 8) * us) : 0u;
                                a[sp][2] = *reinterpret_cast<const unsigned*>(ub + static_cast<size_t>(g) * us + 8);
                                a[sp][3] = TB > 8 ? *reinterpret_cast<const unsigned*>(ub + static_cast<size_t>(g + 8) * us + 8) : 0u;
                            }
                            // lane l addresses row (l & 7) of matrix l >> 3: matrices 0,1 = rows kb.., kb+8.. of
                            // column tile 2q; matrices 2,3 = the same rows of column tile 2q + 1
                            const int mrow = kb + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int mcol = cb * 64 + (2 * q + (lane >> 4)) * 8;
                                unsigned b0, b1, b2, b3;
                                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                                             : "=r"(b0), "=r"(b1), "=r"(b2), "=r"(b3)
                                             : "r"(vs_addr + mrow * RS + mcol * 2));
#pragma unroll
                                for (int sp = 0; sp < 2; ++sp) {
                                    mma_bf16(acc[2 * q], a[sp][0], a[sp][1], a[sp][2], a[sp][3], b0, b1);
                                    mma_bf16(acc[2 * q + 1], a[sp][0], a[sp][1], a[sp][2], a[sp][3], b2, b3);
                                }
                            }
                        }
                        // lane holds tokens g and g + 8, columns cb*64 + 8 i + 2 t, + 1 of tile i
#pragma unroll
                        for (int hrow = 0; hrow < 2; ++hrow) {
                            const int tok = g + 8 * hrow;
                            if (tok < tbv && ((anyt >> tok) & 1u)) {
                                float* dst = yg + static_cast<int64_t>(tok) * d + col0 + cb * 64 + 2 * t;
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    if (cb * 64 + 8 * i + 2 * t < wc)
                                        asm volatile("red.global.add.v2.f32 [%0], {%1,%2};" ::"l"(dst + 8 * i), "f"(acc[i][2 * hrow]),
                                                     "f"(acc[i][2 * hrow + 1])
                                                     : "memory");
                                }
                            }
                        }
                    }
                    __syncthreads();      // this buffer is requested into again two stripes later
                }
            } else if (nU > 0) {
            const int g = lane >> 2, t = lane & 3;
            const int ncb = d / 64;                          // full 64-column blocks (d % 64 handled below)
            const unsigned anyt = tok_any;
            const int nks = (nU + 15) >> 4;
            for (int cb = warp; cb * 64 < d; cb += kWarps) {
                const bool full = cb < ncb;
                float acc[8][4];
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
                constexpr int KB = 4;                        // k-steps per batch: 16 loads of 16 bytes in flight per lane
#pragma unroll 1
                for (int k0 = 0; k0 < nks; k0 += KB) {
                    uint4 rv[KB][4];
#pragma unroll
                    for (int kk = 0; kk < KB; ++kk) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int ui = (k0 + kk) * 16 + 2 * t + (q & 1) + (q >> 1) * 8;
                            const int col = cb * 64 + 8 * g;
                            rv[kk][q] = (ui < nU && (full || col + 8 <= d))
                                            ? ld_stream16(reinterpret_cast<const uint4*>(Vt + static_cast<int64_t>(row0 + ulist[ui]) * d + col))
                                            : make_uint4(0u, 0u, 0u, 0u);
                        }
                    }
#pragma unroll
                    for (int kk = 0; kk < KB; ++kk) {
                        if (k0 + kk < nks) {
                            const int kb = (k0 + kk) * 16;
                            unsigned a[2][4];
#pragma unroll
                            for (int sp = 0; sp < 2; ++sp) {
                                const __nv_bfloat16* ub = u2 + static_cast<size_t>(sp * 16) * us + kb + 2 * t;
                                a[sp][0] = *reinterpret_cast<const unsigned*>(ub + static_cast<size_t>(g) * us);
                                a[sp][1] = TB > 8 ? *reinterpret_cast<const unsigned*>(ub + static_cast<size_t>(g + 8) * us) : 0u;
                                a[sp][2] = *reinterpret_cast<const unsigned*>(ub + static_cast<size_t>(g) * us + 8);
                                a[sp][3] = TB > 8 ? *reinterpret_cast<const unsigned*>(ub + static_cast<size_t>(g + 8) * us + 8) : 0u;
                            }
                            const unsigned wa[4] = {rv[kk][0].x, rv[kk][0].y, rv[kk][0].z, rv[kk][0].w};
                            const unsigned wb[4] = {rv[kk][1].x, rv[kk][1].y, rv[kk][1].z, rv[kk][1].w};
                            const unsigned wc[4] = {rv[kk][2].x, rv[kk][2].y, rv[kk][2].z, rv[kk][2].w};
                            const unsigned wd[4] = {rv[kk][3].x, rv[kk][3].y, rv[kk][3].z, rv[kk][3].w};
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const unsigned sel = (i & 1) ? 0x7632u : 0x5410u;
                                const unsigned b0 = __byte_perm(wa[i >> 1], wb[i >> 1], sel);
                                const unsigned b1 = __byte_perm(wc[i >> 1], wd[i >> 1], sel);
#pragma unroll
                                for (int sp = 0; sp < 2; ++sp) mma_bf16(acc[i], a[sp][0], a[sp][1], a[sp][2], a[sp][3], b0, b1);
                            }
                        }
                    }
                }
                // lane holds, for tokens g and g + 8, columns cb*64 + 16 t + [0, 8) (element 0 of tile i) and + 8 + [0, 8) (element 1)
                const int colb = cb * 64 + 16 * t;
#pragma unroll
                for (int hrow = 0; hrow < 2; ++hrow) {
                    const int tok = g + 8 * hrow;
                    if (tok < tbv && ((anyt >> tok) & 1u)) {
                        float* dst = yg + static_cast<int64_t>(tok) * d + colb;
                        const int e0 = 2 * hrow;
                        if (colb + 8 <= d) {
                            red_add_v4(dst, acc[0][e0], acc[1][e0], acc[2][e0], acc[3][e0]);
                            red_add_v4(dst + 4, acc[4][e0], acc[5][e0], acc[6][e0], acc[7][e0]);
                        }
                        if (colb + 16 <= d) {
                            red_add_v4(dst + 8, acc[0][e0 + 1], acc[1][e0 + 1], acc[2][e0 + 1], acc[3][e0 + 1]);
                            red_add_v4(dst + 12, acc[4][e0 + 1], acc[5][e0 + 1], acc[6][e0 + 1], acc[7][e0 + 1]);
                        }
                    }
                }
            }
            }
        }
        p.trace.mark(7);
        __syncthreads();      // shared buffers are reused by the next token group
    }
    if (cta == 0 && tid == 0) p.hdr->epoch = s_epoch + 1u;   // every block has read the epoch by now
}

template <int TB>
int launch_mma(spark_ctx* ctx, FfnParams& p, cudaStream_t stream) {
    static bool configured[64] = {};
    const Plan plan(p.xw, p.rpc);
    const size_t rest = static_cast<size_t>(2) * 16 * plan.us * 2 + static_cast<size_t>(kWarps) * (TB / 8) * 32 * 16 +
                        static_cast<size_t>(TB) * p.rpc * 4 + static_cast<size_t>(p.rpc) * 8 + 64;
    const size_t limit = static_cast<size_t>(ctx->max_smem_optin - 1024);
    p.xres = Plan::region(true, TB, p.r, p.d - p.r) * 2 + rest <= limit ? 1 : 0;
    const size_t smem = Plan::region(p.xres != 0, TB, p.r, p.d - p.r) * 2 + rest;
    if (smem > limit) return SPARK_ERR_WORKSPACE;   // caller falls back
    auto kern = ffn_mma_kernel<TB>;
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

}  // namespace

namespace spark {

// bf16 weights, 2..64 tokens.  Returns SPARK_ERR_WORKSPACE when the shape does not fit this kernel's
// shared-memory plan or its layout rules (the caller then uses the plain-ALU kernel).
int ffn_mma_launch(spark_ctx* ctx, FfnParams& p, cudaStream_t stream) {
    if ((p.r & 31) != 0 || ((p.d - p.r) & 31) != 0 || (p.d & 15) != 0) return SPARK_ERR_WORKSPACE;
    if (p.B <= 8) return launch_mma<8>(ctx, p, stream);
    return launch_mma<16>(ctx, p, stream);
}

}  // namespace spark
