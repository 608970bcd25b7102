// Shared device/host helpers of the Spark decode library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <stdint.h>

#include "../../include/spark.h"

namespace spark {

constexpr int kWarp = 32;
constexpr unsigned kFull = 0xffffffffu;

// ---------------------------------------------------------------------------
// Context (host object) and workspace header (device)
// ---------------------------------------------------------------------------
// One 32-byte sector that every block adds into and polls: the sum of its scores, the sum of their
// squares, and the number of blocks that have added both (added last, with release semantics, so a
// reader that sees the full count sees the full sums).  Reading the sector is one 32-byte load.
struct __align__(32) SumCell {
    double s1, s2;
    unsigned count;
    unsigned pad[3];
};

// Blocks spread their additions over this many cells per quantity (block b uses way b % 16): a
// single cell would serialise 3 x #blocks atomics on one address, which costs microseconds.
constexpr int kCellWays = 16;

constexpr int kMaxSegments = 2048;
// Attention keeps kAttnWays cells per (sequence, query head) in a fixed region at the start of the
// workspace scratch (room for 16384 heads).
constexpr int kAttnWays = 4;
constexpr size_t kAttnCellBytes = static_cast<size_t>(16384) * kAttnWays * 32;   // (sequence, KV head) pairs one attention call may cover

struct WsHeader {            // lives at the start of the caller's workspace; zero when idle
    int status;              // device status word (SPARK_OK or a SPARK_ERR_* device code)
    unsigned wait_kcycles;   // bound of the inter-block waits in units of 1024 SM cycles; 0 = kSpinLimitCycles (spark_set_wait_limit)
    unsigned reserved;
    unsigned epoch;          // launches of the FFN kernels so far (selects their accumulator ring slot)
    unsigned pad[60];
    unsigned seg_done[kMaxSegments];   // attention: finished pieces per segment (self-resetting)
    SumCell ffn_cells[4][4][16][kCellWays];   // FFN: [epoch & 3][token group][token][way] score sums
    // fused one-token layer kernel: grid-wide barriers as arrival counters that only ever grow (one 32-byte sector per way);
    // barrier number j since the workspace was last reset is complete when the ways add up to j x blocks (modulo 2^32)
    unsigned l1_gen;         // barriers completed by the launches so far
    unsigned l1_pad[63];      // keeps the header a multiple of 256 bytes
    struct { unsigned count; unsigned pad[7]; } l1_ways[kCellWays];
};
static_assert(sizeof(WsHeader) == 256 + 4 * kMaxSegments + 32 * 256 * kCellWays + 256 + 32 * kCellWays && sizeof(WsHeader) % 256 == 0, "header layout");

}  // namespace spark

struct spark_ctx {
    int device;
    int num_sms;
    int max_smem_optin;
    char* ws;                // device workspace base (header first)
    size_t ws_bytes;
    spark::WsHeader* hdr;    // == ws
    char* scratch;           // ws + sizeof(WsHeader)
    size_t scratch_bytes;
    unsigned long long* trace;   // optional phase trace (device), see spark_set_phase_trace
    long long trace_cap;
    int overlap;             // launch with programmatic stream serialization, see spark_set_launch_overlap
    unsigned wait_kcycles;   // host copy of the header's wait bound (restored after a workspace reset)
    const void* next_wqkv;   // set by spark_stack_decode around a layer call: the QKV matrix of the layer after it (or nullptr)
    int l2_prefetch;         // one-token layer calls ask L2 for the next kernel's weights (spark_set_l2_prefetch)
    int fused;               // one token: take the fused layer kernel when it serves the shape (spark_set_fused_layer)
    int chunk_dense;         // prompt chunks: second stage of the attention as masked dense products: 0 never, 1 where it measured faster, 2 wherever it serves the shape (spark_set_chunk_dense)
    int64_t len_hint;        // rows of the cache in use after the current call, when the caller knows them on the host (spark_prefill); 0 = unknown
    int debug_extra_arrivals;   // test hook: the one-token kernels wait for this many arrivals more than blocks exist
};

namespace spark {

// ---------------------------------------------------------------------------
// Programmatic dependent launch.  A kernel launched with the stream-serialization attribute may
// start while the kernel before it in the stream still runs; dep_wait() returns once that kernel
// has completed and its writes are visible.  Only immutable data (weights) may be touched before
// it.  dep_trigger() lets the kernel after this one be scheduled as blocks of this one leave; it
// is called right after dep_wait(), so that a dependent never starts before the grid two places
// back has completed.  Both are no-ops in a kernel launched the ordinary way.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Host: one launch.  `cooperative` asks for the co-residency guarantee; with ctx->overlap the
// launch carries the programmatic attribute instead (the two cannot be combined), and co-residency
// rests on the grid being one block per SM on a GPU that runs nothing else (a block that waits in
// vain gives up after its spin limit and reports SPARK_ERR_TIMEOUT).
inline cudaError_t launch_kernel(const spark_ctx* ctx, const void* kern, unsigned grid, unsigned block, size_t smem,
                                 cudaStream_t stream, bool cooperative, void** args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    cfg.attrs = attr;
    cfg.numAttrs = 0;
    if (ctx->overlap) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.numAttrs = 1;
    } else if (cooperative) {
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        cfg.numAttrs = 1;
    }
    return cudaLaunchKernelExC(&cfg, kern, args);
}

// ---------------------------------------------------------------------------
// L2 prefetch of data a LATER kernel of the stream will read (weights: never written).  At one token the steps are
// latency-bound and HBM idles most of the time; asking L2 for the next kernel's weights meanwhile turns that kernel's
// streaming phase from an HBM stream into an L2 stream.  One bulk-prefetch instruction covers up to 32 KB, so a block's
// share (tens of KB) costs one thread a handful of instructions -- unlike a per-line prefetch it does not compete for issue
// slots or load/store queue entries with the loads on the critical path.
// ---------------------------------------------------------------------------
struct PrefetchSpec {
    const void* ptr;         // nullptr: nothing to prefetch
    unsigned long long bytes;
};
// Called by ONE thread of every block: the block's 1/nparts of the range, in 16-byte aligned pieces.
__device__ __forceinline__ void prefetch_l2_share(const PrefetchSpec& sp, int part, int nparts) {
    if (sp.ptr == nullptr) return;
    const unsigned long long per = ((sp.bytes / nparts) + 127ull) & ~127ull;
    unsigned long long off = per * part;
    if (off >= sp.bytes) return;
    unsigned long long n = sp.bytes - off < per ? sp.bytes - off : per;
    n &= ~15ull;
    const char* q = static_cast<const char*>(sp.ptr) + off;
    while (n > 0) {
        const unsigned piece = n > 32768ull ? 32768u : static_cast<unsigned>(n);
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(q), "r"(piece) : "memory");
        q += piece;
        n -= piece;
    }
}

// ---------------------------------------------------------------------------
// Loads
// ---------------------------------------------------------------------------
// Streaming 16-byte read-only load that does not allocate in L1 (weights and cache rows are
// touched once per call).
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Same, but pinned in program order (used to issue loads ahead of a block-wide sync).
__device__ __forceinline__ uint4 ld_stream16_pinned(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// 8 consecutive weights starting at element index `chunk*8` of a row, widened to fp32.
template <typename WT>
struct Row8;

template <>
struct Row8<__nv_bfloat16> {
    uint4 raw;
    __device__ __forceinline__ void load(const __nv_bfloat16* row, int64_t chunk) {
        raw = ld_stream16(reinterpret_cast<const uint4*>(row) + chunk);
    }
    __device__ __forceinline__ void load_pinned(const __nv_bfloat16* row, int64_t chunk) {
        raw = ld_stream16_pinned(reinterpret_cast<const uint4*>(row) + chunk);
    }
    __device__ __forceinline__ void zero() { raw = make_uint4(0u, 0u, 0u, 0u); }
    __device__ __forceinline__ void unpack(float (&f)[8]) const {
        // bf16 -> fp32 is a 16-bit shift; element 0 sits in the low half of each word
        f[0] = __uint_as_float(raw.x << 16); f[1] = __uint_as_float(raw.x & 0xffff0000u);
        f[2] = __uint_as_float(raw.y << 16); f[3] = __uint_as_float(raw.y & 0xffff0000u);
        f[4] = __uint_as_float(raw.z << 16); f[5] = __uint_as_float(raw.z & 0xffff0000u);
        f[6] = __uint_as_float(raw.w << 16); f[7] = __uint_as_float(raw.w & 0xffff0000u);
    }
};

// FP8 E4M3 storage (per-row scales are applied by the caller): eight values = eight bytes.
template <>
struct Row8<__nv_fp8_e4m3> {
    uint2 raw;
    __device__ __forceinline__ void load(const __nv_fp8_e4m3* row, int64_t chunk) {
        asm("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(raw.x), "=r"(raw.y) : "l"(reinterpret_cast<const uint2*>(row) + chunk));
    }
    __device__ __forceinline__ void load_pinned(const __nv_fp8_e4m3* row, int64_t chunk) {
        asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(raw.x), "=r"(raw.y) : "l"(reinterpret_cast<const uint2*>(row) + chunk));
    }
    __device__ __forceinline__ void zero() { raw = make_uint2(0u, 0u); }
    __device__ __forceinline__ void unpack(float (&f)[8]) const {
        // two e4m3 -> two f16 in one conversion, then f16 -> f32; element 0 sits in the lowest byte
        const unsigned w[2] = {raw.x, raw.y};
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            unsigned h01, h23;
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h01) : "h"(static_cast<unsigned short>(w[i] & 0xffffu)));
            asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h23) : "h"(static_cast<unsigned short>(w[i] >> 16)));
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&h01));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&h23));
            f[4 * i] = a.x; f[4 * i + 1] = a.y; f[4 * i + 2] = b.x; f[4 * i + 3] = b.y;
        }
    }
};

template <>
struct Row8<float> {
    uint4 lo, hi;
    __device__ __forceinline__ void load(const float* row, int64_t chunk) {
        lo = ld_stream16(reinterpret_cast<const uint4*>(row) + 2 * chunk);
        hi = ld_stream16(reinterpret_cast<const uint4*>(row) + 2 * chunk + 1);
    }
    __device__ __forceinline__ void load_pinned(const float* row, int64_t chunk) {
        lo = ld_stream16_pinned(reinterpret_cast<const uint4*>(row) + 2 * chunk);
        hi = ld_stream16_pinned(reinterpret_cast<const uint4*>(row) + 2 * chunk + 1);
    }
    __device__ __forceinline__ void zero() { lo = make_uint4(0u, 0u, 0u, 0u); hi = lo; }
    __device__ __forceinline__ void unpack(float (&f)[8]) const {
        f[0] = __uint_as_float(lo.x); f[1] = __uint_as_float(lo.y);
        f[2] = __uint_as_float(lo.z); f[3] = __uint_as_float(lo.w);
        f[4] = __uint_as_float(hi.x); f[5] = __uint_as_float(hi.y);
        f[6] = __uint_as_float(hi.z); f[7] = __uint_as_float(hi.w);
    }
};

__device__ __forceinline__ float dot8(const float (&w)[8], const float4& a, const float4& b, float acc) {
    acc = fmaf(w[0], a.x, acc); acc = fmaf(w[1], a.y, acc);
    acc = fmaf(w[2], a.z, acc); acc = fmaf(w[3], a.w, acc);
    acc = fmaf(w[4], b.x, acc); acc = fmaf(w[5], b.y, acc);
    acc = fmaf(w[6], b.z, acc); acc = fmaf(w[7], b.w, acc);
    return acc;
}

// ---------------------------------------------------------------------------
// Warp reductions
// ---------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
    return v;
}
__device__ __forceinline__ int warp_sum_int(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

// ---------------------------------------------------------------------------
// Moments (count, mean, sum of squared deviations) and their pairwise merge
// ---------------------------------------------------------------------------
struct Moments {
    double n, mean, m2;
};
__device__ __forceinline__ Moments merge(const Moments& a, const Moments& b) {
    if (b.n == 0.0) return a;
    if (a.n == 0.0) return b;
    Moments o;
    o.n = a.n + b.n;
    const double delta = b.mean - a.mean;
    const double fb = b.n / o.n;
    o.mean = a.mean + delta * fb;
    o.m2 = a.m2 + b.m2 + delta * delta * a.n * fb;
    return o;
}
__device__ __forceinline__ Moments warp_merge(Moments m) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Moments other;
        other.n = __shfl_xor_sync(kFull, m.n, o);
        other.mean = __shfl_xor_sync(kFull, m.mean, o);
        other.m2 = __shfl_xor_sync(kFull, m.m2, o);
        m = merge(m, other);
    }
    return m;
}
// theta = mean + std * z with the Bessel-corrected std (Eq. 11).
__device__ __forceinline__ float theta_from(const Moments& m, double z) {
    const double var = m.n > 1.0 ? m.m2 / (m.n - 1.0) : 0.0;
    return static_cast<float>(m.mean + sqrt(var) * z);
}

// ---------------------------------------------------------------------------
// Activations
// ---------------------------------------------------------------------------
__device__ __forceinline__ float gelu_tanh(float a) {
    const float c = 0.7978845608028654f;   // sqrt(2/pi)
    return 0.5f * a * (1.0f + tanhf(c * (a + 0.044715f * a * a * a)));
}
__device__ __forceinline__ float gelu_erf(float a) {
    return 0.5f * a * (1.0f + erff(a * 0.7071067811865476f));
}
__device__ __forceinline__ float softplus(float a) {
    return fmaxf(a, 0.0f) + log1pf(expf(-fabsf(a)));
}

// ---------------------------------------------------------------------------
// Inter-block barrier with a bounded wait
// ---------------------------------------------------------------------------
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned atom_add_acqrel_u32(unsigned* p, unsigned v) {
    unsigned old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ void st_release_u32(unsigned* p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Optional phase trace: thread 0 of a block stores its SM's cycle counter at a phase boundary
// (phases 0..14); phase 0 also stores the GPU-wide nanosecond timer in entry 15, which lets a
// reader line the blocks up.  The cycle counter is cheap to read; the global timer is not.
struct PhaseTrace {
    unsigned long long* buf;
    long long cap;
    __device__ __forceinline__ void mark(int phase) const {
        if (buf != nullptr && threadIdx.x == 0) {
            const long long i = static_cast<long long>(blockIdx.x) * 16 + phase;
            if (i + 15 < cap) {
                buf[i] = static_cast<unsigned long long>(clock64());
                if (phase == 0) buf[i + 15] = global_ns();
            }
        }
    }
};

// Bound of every spin-wait, in SM cycles (about two seconds at 2 GHz), unless the workspace header carries another.
constexpr long long kSpinLimitCycles = 4000000000ll;
__device__ __forceinline__ long long spin_limit(const WsHeader* hdr) {
    const unsigned k = __ldg(&hdr->wait_kcycles);      // constant while kernels run: written by the host only
    return k != 0u ? static_cast<long long>(k) << 10 : kSpinLimitCycles;
}

// Sum-cell helpers.
__device__ __forceinline__ void red_add_f64(double* p, double v) {
    asm volatile("red.relaxed.gpu.global.add.f64 [%0], %1;" ::"l"(p), "d"(v) : "memory");
}
__device__ __forceinline__ void red_release_add_u32(unsigned* p, unsigned v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Order-preserving map between fp32 and u32 (for atomic max on floats); 0 decodes below every float.
__device__ __forceinline__ unsigned f32_to_ordered(float f) {
    const unsigned u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float ordered_to_f32(unsigned u) {
    if (u == 0u) return -INFINITY;
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}
// One 32-byte read of a cell (sm_100 has 256-bit global loads): {s1, s2, count, pad[0]}.
__device__ __forceinline__ void ld_cell_x(const SumCell* c, double& s1, double& s2, unsigned& count, unsigned& extra) {
    unsigned long long a, b, d;
    [[maybe_unused]] unsigned long long e;   // padding half of the sector: loaded with the rest, not used
    asm volatile("ld.acquire.gpu.global.v4.u64 {%0,%1,%2,%3}, [%4];"
                 : "=l"(a), "=l"(b), "=l"(d), "=l"(e)
                 : "l"(c)
                 : "memory");
    s1 = __longlong_as_double(static_cast<long long>(a));
    s2 = __longlong_as_double(static_cast<long long>(b));
    count = static_cast<unsigned>(d & 0xffffffffull);
    extra = static_cast<unsigned>(d >> 32);
    (void)e;
}
__device__ __forceinline__ void ld_cell(const SumCell* c, double& s1, double& s2, unsigned& count) {
    unsigned extra;
    ld_cell_x(c, s1, s2, count, extra);
}
// Add this block's two sums to its way of a cell group, then its arrival (release: ordered after
// the sums and after everything the block wrote before).  One thread calls this.
template <int WAYS>
__device__ __forceinline__ void cells_add_w(SumCell* ways, int block, double s1, double s2) {
    SumCell* c = ways + (block % WAYS);
    red_add_f64(&c->s1, s1);
    red_add_f64(&c->s2, s2);
    red_release_add_u32(&c->count, 1u);
}
// Lanes 0..WAYS-1 of one warp poll the ways (one 32-byte acquire load each) until all `nblocks`
// blocks have arrived, then every lane of the warp gets the totals.  Called by a full warp.
// Returns false after about two seconds (SPARK_ERR_TIMEOUT recorded).
template <int WAYS>
__device__ __forceinline__ bool cells_wait_w(const SumCell* ways, unsigned nblocks, double& s1, double& s2, WsHeader* hdr) {
    static_assert(WAYS == 1 || WAYS == 2 || WAYS == 4 || WAYS == 8 || WAYS == 16, "ways");
    const int lane = threadIdx.x & 31;
    const long long t0 = clock64(), limit = spin_limit(hdr);
    for (;;) {
        double a = 0.0, b = 0.0;
        unsigned cnt = 0u;
        if (lane < WAYS) ld_cell(ways + lane, a, b, cnt);
        unsigned tot = cnt;
#pragma unroll
        for (int o = WAYS / 2; o > 0; o >>= 1) tot += __shfl_xor_sync(kFull, tot, o);
        tot = __shfl_sync(kFull, tot, 0);
        if (tot == nblocks) {
#pragma unroll
            for (int o = WAYS / 2; o > 0; o >>= 1) {
                a += __shfl_xor_sync(kFull, a, o);
                b += __shfl_xor_sync(kFull, b, o);
            }
            s1 = __shfl_sync(kFull, a, 0);
            s2 = __shfl_sync(kFull, b, 0);
            return true;
        }
        if (clock64() - t0 > limit) {
            if (lane == 0) atomicCAS(&hdr->status, SPARK_OK, SPARK_ERR_TIMEOUT);
            return false;
        }
    }
}
// Group protocol for several cell sets that fill together (the tokens of a batch): every block adds its
// sums to each set without an arrival (cells_add_sums_w, any thread), then -- after a block-wide sync --
// ONE thread releases one arrival on the first set (cells_arrive_w); a single warp waits for the arrivals
// (cells_wait_arrivals_w) and, after another block-wide sync, the sets are read once each (cells_read_w).
// Polling one set instead of all of them keeps the poll traffic independent of the batch size.
template <int WAYS>
__device__ __forceinline__ void cells_add_sums_w(SumCell* ways, int block, double s1, double s2) {
    SumCell* c = ways + (block % WAYS);
    red_add_f64(&c->s1, s1);
    red_add_f64(&c->s2, s2);
}
template <int WAYS>
__device__ __forceinline__ void cells_arrive_w(SumCell* ways, int block) {
    red_release_add_u32(&ways[block % WAYS].count, 1u);
}
template <int WAYS>
__device__ __forceinline__ bool cells_wait_arrivals_w(const SumCell* ways, unsigned nblocks, WsHeader* hdr) {
    double a, b;
    return cells_wait_w<WAYS>(ways, nblocks, a, b, hdr);
}
template <int WAYS>
__device__ __forceinline__ void cells_read_w(const SumCell* ways, double& s1, double& s2) {
    const int lane = threadIdx.x & 31;
    double a = 0.0, b = 0.0;
    unsigned cnt = 0u;
    if (lane < WAYS) ld_cell(ways + lane, a, b, cnt);
#pragma unroll
    for (int o = WAYS / 2; o > 0; o >>= 1) {
        a += __shfl_xor_sync(kFull, a, o);
        b += __shfl_xor_sync(kFull, b, o);
    }
    s1 = __shfl_sync(kFull, a, 0);
    s2 = __shfl_sync(kFull, b, 0);
}
// The same with a running maximum kept in the cell's spare word (attention needs the largest score).
template <int WAYS>
__device__ __forceinline__ void cells_add_max_w(SumCell* ways, int block, double s1, double s2, float mx) {
    SumCell* c = ways + (block % WAYS);
    red_add_f64(&c->s1, s1);
    red_add_f64(&c->s2, s2);
    asm volatile("red.relaxed.gpu.global.max.u32 [%0], %1;" ::"l"(&c->pad[0]), "r"(f32_to_ordered(mx)) : "memory");
    red_release_add_u32(&c->count, 1u);
}
template <int WAYS>
__device__ __forceinline__ bool cells_wait_max_w(const SumCell* ways, unsigned nblocks, double& s1, double& s2, float& mx,
                                                 WsHeader* hdr) {
    const int lane = threadIdx.x & 31;
    const long long t0 = clock64(), limit = spin_limit(hdr);
    for (;;) {
        double a = 0.0, b = 0.0;
        unsigned cnt = 0u, ex = 0u;
        if (lane < WAYS) ld_cell_x(ways + lane, a, b, cnt, ex);
        unsigned tot = cnt;
#pragma unroll
        for (int o = WAYS / 2; o > 0; o >>= 1) tot += __shfl_xor_sync(kFull, tot, o);
        tot = __shfl_sync(kFull, tot, 0);
        if (tot == nblocks) {
#pragma unroll
            for (int o = WAYS / 2; o > 0; o >>= 1) {
                a += __shfl_xor_sync(kFull, a, o);
                b += __shfl_xor_sync(kFull, b, o);
                const unsigned e2 = __shfl_xor_sync(kFull, ex, o);
                ex = e2 > ex ? e2 : ex;
            }
            s1 = __shfl_sync(kFull, a, 0);
            s2 = __shfl_sync(kFull, b, 0);
            mx = ordered_to_f32(__shfl_sync(kFull, ex, 0));
            return true;
        }
        if (clock64() - t0 > limit) {
            if (lane == 0) atomicCAS(&hdr->status, SPARK_OK, SPARK_ERR_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ void cells_add(SumCell* ways, int block, double s1, double s2) {
    cells_add_w<kCellWays>(ways, block, s1, s2);
}
__device__ __forceinline__ bool cells_wait(const SumCell* ways, unsigned nblocks, double& s1, double& s2, WsHeader* hdr) {
    return cells_wait_w<kCellWays>(ways, nblocks, s1, s2, hdr);
}

// Vector reduction into global memory: y[0..3] += v (16-byte aligned address).
__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}
// Read that bypasses L1 (data written by other SMs earlier in the same kernel).
__device__ __forceinline__ float4 ld_cg_f4(const float4* p) { return __ldcg(p); }

// ---------------------------------------------------------------------------
// Host helpers
// ---------------------------------------------------------------------------
inline bool on_device(const spark_ctx* ctx) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == ctx->device;
}
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

}  // namespace spark
