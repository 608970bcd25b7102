// spark_stat_topk: standalone statistical top-k over many rows (Section 3, Eq. 9-11).
//
// One thread-block cluster per row.  Each block of the cluster streams its contiguous part of the
// row from HBM exactly once into shared memory, and every later sweep (squared deviations around
// the exact mean, counting, ordered compaction / dense output) reads shared memory.  Partial sums
// travel between the blocks of a cluster through distributed shared memory.  Rows too long to be
// held on chip fall back to re-reading global memory in the later sweeps.
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
    if (!p.identity) {
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
        theta = theta_from(m, p.z);
    } else if (RESIDENT) {
        for (int v = tid; v < nvec; v += kThreads) {
            uint4 u = ld_stream16(gsrc + v);
            ssrc[v] = make_float4(__uint_as_float(u.x), __uint_as_float(u.y), __uint_as_float(u.z), __uint_as_float(u.w));
        }
        __syncthreads();
    }
    const float shift = p.identity ? 0.f : theta;
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

bool g_attr_done[64] = {};   // per device: opt-in shared memory configured

}  // namespace

extern "C" int spark_stat_topk(spark_ctx* ctx, const float* x, int64_t rows, int64_t n, int64_t ld,
                               int64_t k, int fill, float* theta, int32_t* count, int32_t* idx,
                               float* val, int64_t idx_cap, float* y_dense, void* stream) {
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
    p.hdr = ctx->hdr;

    if (ctx->device >= 0 && ctx->device < 64 && !g_attr_done[ctx->device]) {
        if (cudaFuncSetAttribute(stat_topk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(hard * 4)) != cudaSuccess)
            return SPARK_ERR_CUDA;
        g_attr_done[ctx->device] = true;
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
