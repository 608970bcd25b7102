// spark_stat_topk: standalone statistical top-k over many rows (Section 3, Eq. 9-11).
//
// Two kernels.  Rows of 16K..64K values: one persistent block per SM holds a whole row on chip
// (stat_topk_row_kernel below).  All other lengths: one thread-block cluster per row; each block
// of the cluster streams its contiguous part of the row from HBM exactly once into shared memory,
// and every later sweep (squared deviations around the exact mean, counting, ordered compaction /
// dense output) reads shared memory.  Partial sums travel between the blocks of a cluster through
// distributed shared memory.  Rows too long to be held on chip fall back to re-reading global
// memory in the later sweeps.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;
using namespace spark;

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / kWarp;

struct TopkParams {
    const float* x;
    int64_t rows, n, ld, k;
    int64_t chunk;        // elements per block (multiple of 4)
    int fill;
    int identity;         // k >= n: keep everything unshifted
    double z;             // Q(1 - k/n)
    float* theta;
    int32_t* count;
    int32_t* idx;
    float* val;
    int64_t idx_cap;
    float* y_dense;
    const float* theta_in;   // nullable: thresholds given by the caller (sharded rows: theta of the whole row); no statistics
    double* moments_out;     // nullable: [rows][3] = (n, mean, sum of squared deviations) of each row; nothing else is produced
    WsHeader* hdr;
};

__device__ __forceinline__ double block_sum_f64(double v, double* red /*[kWarps]*/) {
    v = warp_sum_f64(v);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    __syncthreads();
    if (l == 0) red[w] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) t += red[i];
    return t;
}

template <bool RESIDENT>
__global__ void __launch_bounds__(kThreads) stat_topk_kernel(const TopkParams p) {
    extern __shared__ __align__(16) float srow[];           // RESIDENT: this block's part of the row
    __shared__ double red[kWarps];
    __shared__ double part_sum, part_m2;                    // read by the other blocks of the cluster
    __shared__ int part_cnt;
    __shared__ int warp_tot[kWarps];

    cg::cluster_group cluster = cg::this_cluster();
    const unsigned cl = cluster.num_blocks();
    const unsigned rank = cluster.block_rank();
    const int64_t row = blockIdx.x / cl;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const float* xrow = p.x + row * p.ld;
    const int64_t begin = static_cast<int64_t>(rank) * p.chunk;
    int64_t len = p.n - begin;
    if (len > p.chunk) len = p.chunk;
    if (len < 0) len = 0;
    const int nvec = static_cast<int>((len + 3) >> 2);      // the last vector may be partly valid
    const float4* gsrc = reinterpret_cast<const float4*>(xrow + begin);
    float4* ssrc = reinterpret_cast<float4*>(srow);

    auto valid_in = [&](int v) -> int {                     // valid elements in vector v
        const int64_t rem = len - (static_cast<int64_t>(v) << 2);
        return rem >= 4 ? 4 : static_cast<int>(rem);
    };
    auto fetch = [&](int v) -> float4 {
        if (RESIDENT) return ssrc[v];
        uint4 u = ld_stream16(gsrc + v);
        return make_float4(__uint_as_float(u.x), __uint_as_float(u.y), __uint_as_float(u.z), __uint_as_float(u.w));
    };

    float theta = -INFINITY;
    if (!p.identity && p.theta_in == nullptr) {
        // ---- sweep 1: the only HBM read of the row; sum -> mean --------------------------------
        float s0 = 0.f, s1 = 0.f;
        constexpr int LB = 8;                 // 16-byte loads a thread keeps in flight
        for (int v0 = tid; v0 < nvec; v0 += kThreads * LB) {
            uint4 u[LB];
#pragma unroll
            for (int j = 0; j < LB; ++j) {
                const int v = v0 + j * kThreads;
                if (v < nvec) u[j] = ld_stream16(gsrc + v);
                else u[j] = make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int j = 0; j < LB; ++j) {
                const int v = v0 + j * kThreads;
                if (v < nvec) {
                    float4 f = make_float4(__uint_as_float(u[j].x), __uint_as_float(u[j].y), __uint_as_float(u[j].z), __uint_as_float(u[j].w));
                    const int nv = valid_in(v);
                    if (nv < 4) {
                        if (nv < 2) f.y = 0.f;
                        if (nv < 3) f.z = 0.f;
                        f.w = 0.f;
                    }
                    if (RESIDENT) ssrc[v] = f;
                    s0 += f.x + f.y;
                    s1 += f.z + f.w;
                }
            }
        }
        double bs = block_sum_f64(static_cast<double>(s0) + static_cast<double>(s1), red);
        if (tid == 0) part_sum = bs;
        cluster.sync();
        double tot = 0.0;
        for (unsigned c = 0; c < cl; ++c) tot += *cluster.map_shared_rank(&part_sum, c);
        const double mean = tot / static_cast<double>(p.n);
        const float meanf = static_cast<float>(mean);
        // ---- sweep 2: squared deviations around the mean (two-pass form of the text below Eq. 11)
        float q0 = 0.f, q1 = 0.f, e0 = 0.f;
        for (int v = tid; v < nvec; v += kThreads) {
            const float4 f = fetch(v);
            const int nv = valid_in(v);
            const float a = f.x - meanf, b = f.y - meanf, c = f.z - meanf, dd = f.w - meanf;
            q0 += a * a; e0 += a;
            if (nv > 1) { q1 += b * b; e0 += b; }
            if (nv > 2) { q0 += c * c; e0 += c; }
            if (nv > 3) { q1 += dd * dd; e0 += dd; }
        }
        // m2 around the fp32-rounded mean, corrected to the exact mean: sum (x-m)^2 = sum (x-mf)^2 - n (m-mf)^2,
        // with the first-order term carried by e0 = sum (x - mf).
        const double bq = block_sum_f64(static_cast<double>(q0) + static_cast<double>(q1), red);
        const double be = block_sum_f64(static_cast<double>(e0), red);
        if (tid == 0) {
            const double dm = mean - static_cast<double>(meanf);
            part_m2 = bq - 2.0 * dm * be + static_cast<double>(len) * dm * dm;
        }
        cluster.sync();
        double m2 = 0.0;
        for (unsigned c = 0; c < cl; ++c) m2 += *cluster.map_shared_rank(&part_m2, c);
        if (m2 < 0.0) m2 = 0.0;
        Moments m{static_cast<double>(p.n), mean, m2};
        if (p.moments_out != nullptr) {      // a shard's moments for the caller to merge (Appendix: global statistical top-k)
            if (rank == 0 && tid == 0) {
                p.moments_out[row * 3 + 0] = m.n;
                p.moments_out[row * 3 + 1] = m.mean;
                p.moments_out[row * 3 + 2] = m.m2;
            }
            cluster.sync();   // no block may leave while a peer can still read its shared memory
            return;
        }
        theta = theta_from(m, p.z);
    } else if (RESIDENT) {
        for (int v = tid; v < nvec; v += kThreads) {
            uint4 u = ld_stream16(gsrc + v);
            ssrc[v] = make_float4(__uint_as_float(u.x), __uint_as_float(u.y), __uint_as_float(u.z), __uint_as_float(u.w));
        }
        __syncthreads();
    }
    if (p.theta_in != nullptr) theta = p.theta_in[row];
    // a given threshold of -inf is spark_stat_merge's "k >= n_total": everything survives, unshifted
    const float shift = (p.identity || theta == -INFINITY) ? 0.f : theta;
    const bool want_lists = (p.idx != nullptr) || (p.val != nullptr);

    // ---- sweep 3: count the active entries; each warp owns a contiguous run of vectors ----------
    const int vpw = (nvec + kWarps - 1) / kWarps;
    const int vbeg = min(nvec, warp * vpw), vend = min(nvec, vbeg + vpw);
    int cnt = 0;
    for (int v = vbeg + lane; v < vend; v += 32) {
        const float4 f = fetch(v);
        const int nv = valid_in(v);
        cnt += (f.x > theta) + (nv > 1 && f.y > theta) + (nv > 2 && f.z > theta) + (nv > 3 && f.w > theta);
    }
    cnt = warp_sum_int(cnt);
    if (lane == 0) warp_tot[warp] = cnt;
    __syncthreads();
    int block_cnt = 0, warp_base = 0;
#pragma unroll
    for (int i = 0; i < kWarps; ++i) {
        if (i < warp) warp_base += warp_tot[i];
        block_cnt += warp_tot[i];
    }
    if (tid == 0) part_cnt = block_cnt;
    cluster.sync();
    int64_t cluster_base = 0, total = 0;
    for (unsigned c = 0; c < cl; ++c) {
        const int pc = *cluster.map_shared_rank(&part_cnt, c);
        if (c < rank) cluster_base += pc;
        total += pc;
    }
    if (rank == 0 && tid == 0) {
        if (p.theta) p.theta[row] = theta;
        if (p.count) p.count[row] = static_cast<int32_t>(total);
        if (want_lists && total > p.idx_cap) atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_OVERFLOW);
    }

    // ---- sweep 4: ordered compaction and / or the dense output ----------------------------------
    if (want_lists || p.y_dense != nullptr) {
        const float fillv = p.fill == SPARK_FILL_NEGINF ? -INFINITY : 0.f;
        int64_t off = cluster_base + warp_base;
        int32_t* idx_row = p.idx ? p.idx + row * p.idx_cap : nullptr;
        float* val_row = p.val ? p.val + row * p.idx_cap : nullptr;
        float* yrow = p.y_dense ? p.y_dense + row * p.ld + begin : nullptr;
        for (int v0 = vbeg; v0 < vend; v0 += 32) {
            const int v = v0 + lane;
            float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
            int nv = 0;
            if (v < vend) { f = fetch(v); nv = valid_in(v); }
            const bool a0 = nv > 0 && f.x > theta, a1 = nv > 1 && f.y > theta;
            const bool a2 = nv > 2 && f.z > theta, a3 = nv > 3 && f.w > theta;
            if (yrow != nullptr && nv > 0) {
                float4 o;
                o.x = a0 ? f.x - shift : fillv; o.y = a1 ? f.y - shift : fillv;
                o.z = a2 ? f.z - shift : fillv; o.w = a3 ? f.w - shift : fillv;
                if (nv == 4) {
                    reinterpret_cast<float4*>(yrow)[v] = o;
                } else {
                    float* t = yrow + (static_cast<int64_t>(v) << 2);
                    t[0] = o.x;
                    if (nv > 1) t[1] = o.y;
                    if (nv > 2) t[2] = o.z;
                }
            }
            if (want_lists) {
                const int c = a0 + a1 + a2 + a3;
                int incl = c;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(kFull, incl, o);
                    if (lane >= o) incl += t;
                }
                int64_t pos = off + incl - c;
                const int64_t e = begin + (static_cast<int64_t>(v) << 2);
                const float fv[4] = {f.x, f.y, f.z, f.w};
                const bool av[4] = {a0, a1, a2, a3};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (av[j]) {
                        if (pos < p.idx_cap) {
                            if (idx_row) idx_row[pos] = static_cast<int32_t>(e + j);
                            if (val_row) val_row[pos] = fv[j] - shift;
                        }
                        ++pos;
                    }
                }
                off += __shfl_sync(kFull, incl, 31);
            }
        }
    }
    cluster.sync();   // no block may leave while a peer can still read its shared memory
}

// ---------------------------------------------------------------------------------------------
// Rows of 16K..64K values: a persistent 512-thread block per SM keeps one whole row on chip -- the
// leading part (up to 184 KB) in shared memory, brought in by bulk asynchronous copies that signal
// one mbarrier per 32 KB piece, and the last (up to) 4608 float4 in registers, nine per thread.  The
// register part is double-buffered: the next row's is requested as soon as the current row's last
// piece has landed, so HBM stays busy while the block reduces, counts and writes its lists; the
// next row's bulk copies start when the last sweep over shared memory is done.  Each row is read
// from HBM exactly once.  The sums are those of (x - c) and (x - c)^2 around c = the row's first
// value (shifting keeps the fp32 partial sums accurate when |mean| >> std); they are combined in fp64.
//
// Selection: every thread owns a run of 23 consecutive float4 in shared memory (an odd run length
// keeps the 16-byte reads of a quarter warp on distinct banks); the register part is owned warp by
// warp, lane-strided, as it was loaded.  The counting sweep leaves one bit per value; scans of the counts
// give each run its rank; a warp's share of the lists is contiguous and goes through a 256-entry
// staging window of its own in shared memory, so that it leaves the SM as coalesced stores.
// ---------------------------------------------------------------------------------------------
constexpr int kRowThreads = 512;
constexpr int kRowWarps = kRowThreads / 32;
constexpr int kRowRegVec = 9;                                    // float4 per thread kept in registers
constexpr int kRowRunVec = 23;                                   // float4 per thread in shared memory
constexpr int kRowSmemVec = kRowRunVec * kRowThreads;            // 11776 float4 = 184 KB
constexpr int kRowPieceVec = 2048;                               // float4 per bulk copy (32 KB)
constexpr int kRowPieces = (kRowSmemVec + kRowPieceVec - 1) / kRowPieceVec;   // 12 (the last one is half)
constexpr int kRowMaxVec = kRowSmemVec + kRowRegVec * kRowThreads;   // 16384 float4 = 65536 values
constexpr int kRowWin = 256;                                     // entries of a warp's staging window
constexpr int kRowSmemBytes = kRowSmemVec * 16 + kRowWarps * kRowWin * 8;
constexpr long long kRowSpinLimit = 400000000ll;                 // bound of a wait for one 32 KB copy

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > kRowSpinLimit) return false;
    return true;
}

struct RowGeom {
    int n, nvec, ns, npiece;
};

// Thread 0: start the bulk copies of one row's shared-memory part.
__device__ __forceinline__ void row_issue_bulk(const float* xrow, float* srow, unsigned long long* mbar, const RowGeom& g) {
    for (int c = 0; c < g.npiece; ++c) {
        const int vec = min(kRowPieceVec, g.ns - c * kRowPieceVec);
        const uint32_t bytes = static_cast<uint32_t>(vec) * 16u, bar = smem_u32(mbar + c);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(srow + c * kRowPieceVec * 4)), "l"(xrow + static_cast<int64_t>(c) * kRowPieceVec * 4), "r"(bytes), "r"(bar)
                     : "memory");
    }
}
// All threads: request one row's register part (warp w, lane l: vectors ns + w*288 + i*32 + l).
__device__ __forceinline__ void row_load_regs(const float* xrow, const RowGeom& g, uint4 (&r)[kRowRegVec]) {
    const int v0 = g.ns + static_cast<int>(threadIdx.x >> 5) * (kRowRegVec * 32) + static_cast<int>(threadIdx.x & 31);
    const uint4* gsrc = reinterpret_cast<const uint4*>(xrow);
#pragma unroll
    for (int i = 0; i < kRowRegVec; ++i) r[i] = v0 + i * 32 < g.nvec ? ld_stream16_pinned(gsrc + v0 + i * 32) : make_uint4(0u, 0u, 0u, 0u);
}

struct RowShared {
    unsigned long long mbar[kRowPieces];
    double red1[kRowWarps], red2[kRowWarps];
    int scan[kRowWarps];
    float theta;
    int abort;
};

// One row: cur holds its register part, nxt receives the next row's.  Returns false after a timeout.
__device__ __forceinline__ bool row_body(const TopkParams& p, const RowGeom& g, float* srow, RowShared& sh, int64_t row, int64_t next_row,
                                         uint32_t parity, uint4 (&cur)[kRowRegVec], uint4 (&nxt)[kRowRegVec], float c, float& c_next) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float4* ssrc = reinterpret_cast<const float4*>(srow);
    const int rv0 = g.ns + warp * (kRowRegVec * 32) + lane;           // register vectors: rv0 + 32 * i
    const int sv0 = tid * kRowRunVec;                                 // first shared-memory vector of its run
    const int last_nv = g.n - ((g.nvec - 1) << 2);                    // valid values of the last vector (1..4)
    auto f4 = [](const uint4& u) { return make_float4(__uint_as_float(u.x), __uint_as_float(u.y), __uint_as_float(u.z), __uint_as_float(u.w)); };

    float a1 = 0.f, a2 = 0.f;
    auto accumulate = [&](const float4& f) {
        const float d0 = f.x - c, d1 = f.y - c, d2 = f.z - c, d3 = f.w - c;
        a1 += (d0 + d1) + (d2 + d3);
        a2 = fmaf(d0, d0, fmaf(d1, d1, fmaf(d2, d2, fmaf(d3, d3, a2))));
    };
    bool ok = true;
    if (!p.identity) {
#pragma unroll
        for (int i = 0; i < kRowRegVec; ++i) {
            const int v = rv0 + i * 32;
            if (v < g.nvec) {
                float4 f = f4(cur[i]);
                if (v == g.nvec - 1) {                                 // a ragged tail counts as c (adds nothing)
                    if (last_nv < 2) f.y = c;
                    if (last_nv < 3) f.z = c;
                    if (last_nv < 4) f.w = c;
                }
                accumulate(f);
            }
        }
    }
    // the shared-memory part, piece by piece as the copies land
    for (int pc = 0; pc < g.npiece; ++pc) {
        ok = mbar_wait(smem_u32(sh.mbar + pc), parity) && ok;
        if (!p.identity) {
#pragma unroll
            for (int h = 0; h < kRowPieceVec / kRowThreads; ++h) {
                const int v = pc * kRowPieceVec + h * kRowThreads + tid;
                if (v < g.ns) accumulate(ssrc[v]);
            }
        }
    }
    // HBM would idle from here to the end of the row: fetch the next row's register part meanwhile
    if (next_row < p.rows) {
        const float* xn = p.x + next_row * p.ld;
        c_next = p.identity ? 0.f : __ldg(xn);
        row_load_regs(xn, g, nxt);
    }

    float theta = -INFINITY;
    {
        const double w1 = warp_sum_f64(static_cast<double>(a1)), w2 = warp_sum_f64(static_cast<double>(a2));
        if (lane == 0) { sh.red1[warp] = w1; sh.red2[warp] = w2; }
        if (!ok) sh.abort = 1;
        __syncthreads();
        if (warp == 0) {
            double t1 = lane < kRowWarps ? sh.red1[lane] : 0.0, t2 = lane < kRowWarps ? sh.red2[lane] : 0.0;
            t1 = warp_sum_f64(t1);
            t2 = warp_sum_f64(t2);
            if (lane == 0) {
                const double nn = static_cast<double>(g.n);
                const double mean = static_cast<double>(c) + t1 / nn;
                double m2 = t2 - t1 * t1 / nn;
                if (m2 < 0.0) m2 = 0.0;
                sh.theta = p.identity ? -INFINITY : theta_from(Moments{nn, mean, m2}, p.z);
            }
        }
        __syncthreads();
        theta = sh.theta;
        if (sh.abort) return false;
    }
    const float shift = p.identity ? 0.f : theta;

    // ---- count: one bit per value of the thread's two runs ------------------------------------------
    unsigned ms[3] = {0u, 0u, 0u};                                    // 92 bits: shared-memory run
    unsigned long long mr = 0ull;                                     // 36 bits: register run
#pragma unroll
    for (int i = 0; i < kRowRunVec; ++i) {
        if (sv0 + i < g.ns) {
            const float4 f = ssrc[sv0 + i];
            const unsigned nib = (f.x > theta ? 1u : 0u) | (f.y > theta ? 2u : 0u) | (f.z > theta ? 4u : 0u) | (f.w > theta ? 8u : 0u);
            ms[(4 * i) >> 5] |= nib << ((4 * i) & 31);
        }
    }
#pragma unroll
    for (int i = 0; i < kRowRegVec; ++i) {
        const int v = rv0 + i * 32;
        if (v < g.nvec) {
            const float4 f = f4(cur[i]);
            unsigned nib = (f.x > theta ? 1u : 0u) | (f.y > theta ? 2u : 0u) | (f.z > theta ? 4u : 0u) | (f.w > theta ? 8u : 0u);
            if (v == g.nvec - 1) nib &= (1u << last_nv) - 1u;
            mr |= static_cast<unsigned long long>(nib) << (4 * i);
        }
    }
    const int cs = __popc(ms[0]) + __popc(ms[1]) + __popc(ms[2]), cr = __popcll(mr);
    // block-wide exclusive scan of (cs, cr), packed 16 + 16 bits (the totals stay below 2^16)
    const int packed = cs | (cr << 16);
    int inc = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) sh.scan[warp] = inc;
    __syncthreads();
    int base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kRowWarps; ++w) {
        const int a = sh.scan[w];
        if (w < warp) base += a;
        tot += a;
    }
    const int excl = base + inc - packed;
    const int tot_s = tot & 0xffff, total = tot_s + (tot >> 16);
    const bool want_lists = (p.idx != nullptr) || (p.val != nullptr);
    if (tid == 0) {
        if (p.theta) p.theta[row] = theta;
        if (p.count) p.count[row] = total;
        if (want_lists && total > p.idx_cap) atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_OVERFLOW);
    }

    // ---- ordered lists: each warp stages its (contiguous) share in a 256-entry window of its own -------
    if (want_lists) {
        int* wi = reinterpret_cast<int*>(srow + kRowSmemVec * 4) + warp * (2 * kRowWin);
        float* wv = reinterpret_cast<float*>(wi + kRowWin);
        int32_t* idx_row = p.idx ? p.idx + row * p.idx_cap : nullptr;
        float* val_row = p.val ? p.val + row * p.idx_cap : nullptr;
        const int wpacked = sh.scan[warp];
        auto flush = [&](int first, int cnt) {                         // window -> lists, lanes over consecutive entries
            __syncwarp();
            for (int t = lane; t < cnt; t += 32) {
                const int at = first + t;
                if (at < p.idx_cap) {
                    if (idx_row) idx_row[at] = wi[t];
                    if (val_row) val_row[at] = wv[t];
                }
            }
            __syncwarp();
        };
        // shared-memory runs: ranks of this warp start at wbase; a thread's values follow one another
        {
            const int wbase = base & 0xffff, wtot = wpacked & 0xffff;
            int rel = (excl & 0xffff) - wbase;
            unsigned long long lo = static_cast<unsigned long long>(ms[0]) | (static_cast<unsigned long long>(ms[1]) << 32);
            unsigned hi = ms[2];
            const int es = sv0 << 2;
#pragma unroll 1
            for (int w0 = 0; w0 < wtot; w0 += kRowWin) {
                while ((lo != 0ull || hi != 0u) && rel < w0 + kRowWin) {
                    const bool in_lo = lo != 0ull;
                    const int bit = in_lo ? __ffsll(static_cast<long long>(lo)) - 1 : 63 + __ffs(hi);
                    lo &= lo - (in_lo ? 1ull : 0ull);                  // lo == 0 stays 0
                    hi &= hi - (in_lo ? 0u : 1u);
                    wi[rel - w0] = es + bit;
                    wv[rel - w0] = srow[es + bit] - shift;
                    ++rel;
                }
                flush(wbase + w0, min(kRowWin, wtot - w0));
            }
        }
        // register part: a warp owns 288 consecutive vectors, vector i of lane l being number 32 i + l of
        // them.  Rank inside the warp = totals of the earlier i + the lower lanes' counts in this i + the
        // lower neighbours in the vector.  The per-i counts (<= 4 per lane, <= 128 per warp) are scanned
        // across the lanes four to a word.
        const int wtot_r = wpacked >> 16;
        if (wtot_r != 0) {
            const int wbase = tot_s + (base >> 16);
            unsigned exq[3], offs[5];                                  // lane prefixes (8 bits per i), starts of each i (16 bits)
            {
                unsigned q[3] = {0u, 0u, 0u};
#pragma unroll
                for (int i = 0; i < kRowRegVec; ++i) q[i >> 2] |= static_cast<unsigned>(__popc(static_cast<unsigned>(mr >> (4 * i)) & 15u)) << (8 * (i & 3));
                unsigned inc_q[3] = {q[0], q[1], q[2]};
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
                    for (int w = 0; w < 3; ++w) {
                        const unsigned t = __shfl_up_sync(kFull, inc_q[w], o);
                        if (lane >= o) inc_q[w] += t;
                    }
                }
                unsigned off = 0u;
#pragma unroll
                for (int w = 0; w < 5; ++w) offs[w] = 0u;
#pragma unroll
                for (int i = 0; i < kRowRegVec; ++i) {
                    offs[i >> 1] |= off << (16 * (i & 1));
                    off += (__shfl_sync(kFull, inc_q[i >> 2], 31) >> (8 * (i & 3))) & 0xffu;
                }
#pragma unroll
                for (int w = 0; w < 3; ++w) exq[w] = inc_q[w] - q[w];
            }
#pragma unroll 1
            for (int w0 = 0; w0 < wtot_r; w0 += kRowWin) {
                for (unsigned long long m = mr; m != 0ull; m &= m - 1ull) {
                    const int bit = __ffsll(static_cast<long long>(m)) - 1, i = bit >> 2, j = bit & 3;
                    const unsigned ew = i < 4 ? exq[0] : (i < 8 ? exq[1] : exq[2]);
                    const unsigned ow = i < 2 ? offs[0] : (i < 4 ? offs[1] : (i < 6 ? offs[2] : (i < 8 ? offs[3] : offs[4])));
                    const unsigned nib = static_cast<unsigned>(mr >> (4 * i)) & 15u;
                    const int rel = static_cast<int>((ow >> (16 * (i & 1))) & 0xffffu) + static_cast<int>((ew >> (8 * (i & 3))) & 0xffu) +
                                    __popc(nib & ((1u << j) - 1u)) - w0;
                    if (rel >= 0 && rel < kRowWin) {
                        uint4 u = cur[0];                                 // registers cannot be indexed: select
#pragma unroll
                        for (int t = 1; t < kRowRegVec; ++t)
                            if (i == t) u = cur[t];
                        const unsigned bits = j == 0 ? u.x : (j == 1 ? u.y : (j == 2 ? u.z : u.w));
                        wi[rel] = ((rv0 + 32 * i) << 2) + j;
                        wv[rel] = __uint_as_float(bits) - shift;
                    }
                }
                flush(wbase + w0, min(kRowWin, wtot_r - w0));
            }
        }
    }
    // ---- dense output -----------------------------------------------------------------------------
    if (p.y_dense != nullptr) {
        const float fillv = p.fill == SPARK_FILL_NEGINF ? -INFINITY : 0.f;
        float* yrow = p.y_dense + row * p.ld;
        auto emit4 = [&](const float4& f, int v, int nv) {
            float4 o;
            o.x = f.x > theta ? f.x - shift : fillv; o.y = f.y > theta ? f.y - shift : fillv;
            o.z = f.z > theta ? f.z - shift : fillv; o.w = f.w > theta ? f.w - shift : fillv;
            if (nv == 4) {
                __stcs(reinterpret_cast<float4*>(yrow) + v, o);
            } else {
                float* t = yrow + (v << 2);
                t[0] = o.x;
                if (nv > 1) t[1] = o.y;
                if (nv > 2) t[2] = o.z;
            }
        };
        for (int v = tid; v < g.ns; v += kRowThreads) emit4(ssrc[v], v, 4);
#pragma unroll
        for (int i = 0; i < kRowRegVec; ++i) {
            const int v = rv0 + i * 32;
            if (v < g.nvec) emit4(f4(cur[i]), v, v == g.nvec - 1 ? last_nv : 4);
        }
    }
    // shared memory is free again: start the next row's copies
    __syncthreads();
    if (tid == 0 && next_row < p.rows) row_issue_bulk(p.x + next_row * p.ld, srow, sh.mbar, g);
    return true;
}

__global__ void __launch_bounds__(kRowThreads, 1) stat_topk_row_kernel(const TopkParams p) {
    extern __shared__ __align__(16) float srow[];
    __shared__ RowShared sh;
    const int tid = threadIdx.x;
    RowGeom g;
    g.n = static_cast<int>(p.n);
    g.nvec = (g.n + 3) >> 2;
    const int nr = min(g.nvec, kRowRegVec * kRowThreads);
    g.ns = g.nvec - nr;
    g.npiece = (g.ns + kRowPieceVec - 1) / kRowPieceVec;

    int64_t row = blockIdx.x;
    if (row >= p.rows) return;
    if (tid == 0) {
        for (int c = 0; c < kRowPieces; ++c)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(sh.mbar + c)) : "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        sh.abort = 0;
        row_issue_bulk(p.x + row * p.ld, srow, sh.mbar, g);
    }
    uint4 ra[kRowRegVec], rb[kRowRegVec];
    float ca = p.identity ? 0.f : __ldg(p.x + row * p.ld), cb = 0.f;
    row_load_regs(p.x + row * p.ld, g, ra);
    __syncthreads();                                                  // barrier objects visible to every thread
    const int64_t step = gridDim.x;
    bool ok = true;
    uint32_t parity = 0;
#pragma unroll 1
    for (;;) {
        ok = row_body(p, g, srow, sh, row, row + step, parity, ra, rb, ca, cb);
        row += step;
        if (!ok || row >= p.rows) break;
        parity ^= 1u;
        ok = row_body(p, g, srow, sh, row, row + step, parity, rb, ra, cb, ca);
        row += step;
        if (!ok || row >= p.rows) break;
        parity ^= 1u;
    }
    if (!ok) {
        // a copy did not land in time: report it, then give copies still in flight one more bounded wait
        if (tid == 0) {
            atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_TIMEOUT);
            for (int c = 0; c < g.npiece; ++c) {
                const long long t0 = clock64();
                while (!mbar_try_wait(smem_u32(sh.mbar + c), parity))
                    if (clock64() - t0 > kRowSpinLimit) break;
            }
        }
    }
}

bool g_attr_done[64] = {};   // per device: opt-in shared memory configured

}  // namespace

// theta_in / moments_out: the two halves of the sharded form (see spark_stat_moments, spark_stat_select).
static int topk_launch(spark_ctx* ctx, const float* x, int64_t rows, int64_t n, int64_t ld, int64_t k, int fill, float* theta, int32_t* count,
                int32_t* idx, float* val, int64_t idx_cap, float* y_dense, const float* theta_in, double* moments_out, void* stream) {
    if (ctx == nullptr || x == nullptr) return SPARK_ERR_INVALID_ARG;
    if (rows < 0 || n < 1 || ld < n || k <= 0) return SPARK_ERR_INVALID_ARG;
    if (fill != SPARK_FILL_ZERO && fill != SPARK_FILL_NEGINF) return SPARK_ERR_INVALID_ARG;
    if ((idx != nullptr || val != nullptr) && idx_cap < 1) return SPARK_ERR_INVALID_ARG;
    if (k < n && n < 2) return SPARK_ERR_INVALID_ARG;
    if (!aligned16(x) || (ld & 3) != 0) return SPARK_ERR_UNSUPPORTED;
    if (y_dense != nullptr && !aligned16(y_dense)) return SPARK_ERR_UNSUPPORTED;
    if (rows * 8 > 0x7fffffffLL || n > (1LL << 40)) return SPARK_ERR_UNSUPPORTED;
    if (rows == 0) return SPARK_OK;

    // Cluster size: the smallest of 1/2/4/8 that brings one block's part down to 64 KB (three
    // blocks per SM); longer rows take 8 blocks with up to 200 KB each, longer still are re-read.
    const int64_t target = 16384, hard = 51200;
    int cl = 1;
    while (cl < 8 && (n + cl - 1) / cl > target) cl *= 2;
    int64_t chunk = ((n + cl - 1) / cl + 3) / 4 * 4;
    const bool resident = chunk <= hard;

    TopkParams p;
    p.x = x; p.rows = rows; p.n = n; p.ld = ld; p.k = k; p.chunk = chunk; p.fill = fill;
    p.identity = k >= n ? 1 : 0;
    p.z = p.identity ? 0.0 : spark_normal_upper_quantile(static_cast<double>(k) / static_cast<double>(n));
    p.theta = theta; p.count = count; p.idx = idx; p.val = val; p.idx_cap = idx_cap; p.y_dense = y_dense;
    p.theta_in = theta_in; p.moments_out = moments_out;
    p.hdr = ctx->hdr;

    if (ctx->device >= 0 && ctx->device < 64 && !g_attr_done[ctx->device]) {
        if (cudaFuncSetAttribute(stat_topk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(hard * 4)) != cudaSuccess)
            return SPARK_ERR_CUDA;
        g_attr_done[ctx->device] = true;
    }

    if (n > 16384 && (n + 3) / 4 <= kRowMaxVec && theta_in == nullptr && moments_out == nullptr) {      // the whole row fits one block: no cluster needed
        static bool row_attr_done[64] = {};
        if (ctx->device >= 0 && ctx->device < 64 && !row_attr_done[ctx->device]) {
            if (cudaFuncSetAttribute(stat_topk_row_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRowSmemBytes) != cudaSuccess)
                return SPARK_ERR_CUDA;
            row_attr_done[ctx->device] = true;
        }
        const size_t smem = kRowSmemBytes;
        const int64_t grid = rows < ctx->num_sms ? rows : ctx->num_sms;
        stat_topk_row_kernel<<<static_cast<unsigned>(grid), kRowThreads, smem, static_cast<cudaStream_t>(stream)>>>(p);
        return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
    }

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(rows * cl));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = resident ? static_cast<size_t>(chunk) * 4 : 0;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cl;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = resident ? cudaLaunchKernelEx(&cfg, stat_topk_kernel<true>, p)
                             : cudaLaunchKernelEx(&cfg, stat_topk_kernel<false>, p);
    return e == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}

extern "C" int spark_stat_topk(spark_ctx* ctx, const float* x, int64_t rows, int64_t n, int64_t ld,
                               int64_t k, int fill, float* theta, int32_t* count, int32_t* idx,
                               float* val, int64_t idx_cap, float* y_dense, void* stream) {
    return topk_launch(ctx, x, rows, n, ld, k, fill, theta, count, idx, val, idx_cap, y_dense, nullptr, nullptr, stream);
}

extern "C" int spark_stat_moments(spark_ctx* ctx, const float* x, int64_t rows, int64_t n, int64_t ld, double* moments, void* stream) {
    if (moments == nullptr || n < 1) return SPARK_ERR_INVALID_ARG;
    // k = 1 < n keeps the statistics branch; for n == 1 the row is its own mean
    if (n == 1) return SPARK_ERR_UNSUPPORTED;
    return topk_launch(ctx, x, rows, n, ld, 1, SPARK_FILL_ZERO, nullptr, nullptr, nullptr, nullptr, 0, nullptr, nullptr, moments, stream);
}

extern "C" int spark_stat_select(spark_ctx* ctx, const float* x, int64_t rows, int64_t n, int64_t ld, const float* theta_in, int fill,
                                 int32_t* count, int32_t* idx, float* val, int64_t idx_cap, float* y_dense, void* stream) {
    if (theta_in == nullptr) return SPARK_ERR_INVALID_ARG;
    // k = 1 < n: not the identity case, so survivors are shifted by the given threshold
    if (n < 2) return SPARK_ERR_UNSUPPORTED;
    return topk_launch(ctx, x, rows, n, ld, 1, fill, nullptr, count, idx, val, idx_cap, y_dense, theta_in, nullptr, stream);
}

namespace {

// One thread per row: merge the m shards' moments (pairwise update of count, mean and sum of squared deviations) and
// form theta = mean + std * Q(1 - k/n) of the whole row (Eq. 10/11 on the merged moments).
__global__ void stat_merge_kernel(const double* parts, int64_t m, int64_t rows, double z, int identity, float* theta, double* merged) {
    const int64_t row = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (row >= rows) return;
    Moments acc{0.0, 0.0, 0.0};
    for (int64_t s = 0; s < m; ++s) {
        const double* q = parts + (s * rows + row) * 3;
        acc = merge(acc, Moments{q[0], q[1], q[2]});
    }
    if (merged != nullptr) {
        merged[row * 3 + 0] = acc.n;
        merged[row * 3 + 1] = acc.mean;
        merged[row * 3 + 2] = acc.m2;
    }
    theta[row] = identity ? -INFINITY : theta_from(acc, z);
}

}  // namespace

extern "C" int spark_stat_merge(spark_ctx* ctx, const double* parts, int64_t m, int64_t rows, int64_t k, int64_t n_total, float* theta,
                                double* merged, void* stream) {
    if (ctx == nullptr || parts == nullptr || theta == nullptr || m < 1 || rows < 0 || k <= 0 || n_total < 1) return SPARK_ERR_INVALID_ARG;
    if (k < n_total && n_total < 2) return SPARK_ERR_INVALID_ARG;
    if (rows == 0) return SPARK_OK;
    const int identity = k >= n_total ? 1 : 0;
    const double z = identity ? 0.0 : spark_normal_upper_quantile(static_cast<double>(k) / static_cast<double>(n_total));
    stat_merge_kernel<<<static_cast<unsigned>((rows + 127) / 128), 128, 0, static_cast<cudaStream_t>(stream)>>>(parts, m, rows, z, identity, theta, merged);
    return cudaGetLastError() == cudaSuccess ? SPARK_OK : SPARK_ERR_CUDA;
}
