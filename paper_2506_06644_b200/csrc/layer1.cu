// One decoder layer (Section 4) for ONE token as ONE persistent kernel: Spark attention (Section 2.2, Eq. 7) and Spark FFN
// (Section 2.1, Eq. 2) with their statistical top-k (Section 3, Eq. 9-11) and the dense projections around them.
//
// Why one kernel.  At one token a layer touches about 60 MB (2B shape) -- nine microseconds of HBM time -- but its steps are
// chained by six grid-wide dependencies (query, score sums of the attention, attention output, hidden state, score sums of
// the FFN, hidden state again), and 85 % of the bytes (Wqkv, Wo, K1t, the predictor slice of the cache) do not depend on the
// activations at all.  Here one block per SM stays resident for the whole layer (or a whole stack of layers):
//   * a PRODUCER warp streams the block's share of those activation-independent bytes, in the order the phases consume them,
//     into a ring of shared-memory slots with bulk copies (cp.async.bulk + mbarrier transaction counts).  It never waits for
//     a phase boundary, only for a free slot, so HBM keeps streaming while the consumers sit in a grid-wide wait; the
//     ring (about 130 KB per SM, 19 MB per GPU) is the look-ahead;
//   * sixteen CONSUMER warps take slots round-robin, compute from shared memory with the input vector held in registers, and
//     meet at grid-wide barriers (arrival counters that only grow, spread over 16 sectors) and at the score-sum cells;
//   * the activation-DEPENDENT rows (K2t / Vt rows of the active neurons, k2c / vc rows of the selected tokens) are fetched
//     after the threshold is known, all of a block's rows at once as bulk copies into a gather area of their own, so a
//     gather is one round trip whatever the count.
// Phases of a layer (G = grid barrier, X = exchange of score sums):
//   P1 a = RMSNorm(h), [q|k|v] = Wqkv a, rotary encoding, cache append            G1
//   P2 predictor scores of the block's tokens (one KV head per block)              X2
//   P3 theta per query head, selection, gather, partial softmax x gate x value     G3
//   P4 h += Wo (o / sum of weights)                                                G4
//   P5 x = RMSNorm(h), predictor scores of the block's neurons                     X5
//   P6 theta, active neurons, gather, h += V u                                     G6
#include <cmath>
#include <cstdlib>

#include "kernels.h"

using namespace spark;

namespace {

constexpr int kCons = 512;                 // consumer threads (16 warps)
constexpr int kConsWarps = kCons / 32;
constexpr int kThreadsL1 = kCons + 32;     // + the producer warp
constexpr int kMaxLayers = 64;
constexpr int kEmptyCount = kConsWarps;    // arrivals that free a slot: every consumer warp passes through every slot

struct L1Layer {
    const float* norm1;
    const float* norm2;
    const __nv_bfloat16* Wqkv;
    const __nv_bfloat16* Wo;
    const __nv_bfloat16* K1t;
    const __nv_bfloat16* K2t;
    const __nv_bfloat16* Vt;
    __nv_bfloat16* k1c;
    __nv_bfloat16* k2c;
    __nv_bfloat16* vc;
    int window;
    int pad;
};

struct L1Params {
    float* h;                // [d] in/out
    float* qbuf;             // [n_q][hd] rotated, scaled query
    float* obuf;             // [n_q][hd] weighted value sums (blocks add into it)
    float* lsum;             // [n_q] sums of softmax weights
    const int32_t* ctx_len;  // [1]
    int n_layers;
    int d, d_ff, r_ff, n_q, n_kv, hd, r_attn, k_attn, gq;
    int64_t cap;
    float eps, q_scale;
    int erf_form, extra_arrivals;
    double z_ff;             // Q(1 - k_ff / d_ff); identity_ff: k_ff >= d_ff
    int identity_ff;
    double inv_n, inv_nm1;
    // shared-memory plan (bytes from the dynamic base; every offset a multiple of 128)
    int slot_bytes, n_slots;
    int off_ring, off_gather, off_act, off_sc, off_misc;
    int gather_bytes;        // size of the gather area
    int ntok_cap;            // score slots per query head
    int rpc;                 // neurons per block (upper bound)
    int tps;                 // tokens of the predictor slice per slot (a multiple of 16)
    int max_inflight;        // slots the producer keeps in flight at most (pacing)
    int off_xsp, xstride, qstride;   // the input as three bf16 terms: offset, bytes between the terms' rows (x; queries)
    SumCell* attn_cells;     // [n_q][kAttnWays]
    WsHeader* hdr;
    PhaseTrace trace;
    double inv_freq[2][64];
    L1Layer layer[kMaxLayers];
};

// ---- PTX helpers -----------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t saddr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mb_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mb_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mb_arrive_n(uint32_t bar, uint32_t n) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
}
__device__ __forceinline__ bool mb_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait on an mbarrier; `fail` is the block's abort flag (set by whoever gives up first, ends everybody's waits).
__device__ __forceinline__ bool mb_wait(uint32_t bar, uint32_t parity, volatile int* fail, long long limit) {
    if (mb_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mb_try(bar, parity)) {
        if (*fail != 0) return false;
        if (clock64() - t0 > limit) {
            *fail = 1;
            return false;
        }
    }
    return true;
}
// global -> shared bulk copy (both addresses 16-byte aligned, bytes a multiple of 16), completion on an mbarrier
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void cons_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kCons) : "memory"); }
// Barrier of the consumer threads that also ORs a flag over them: every thread gets the same answer, so a decision to leave
// a phase (a wait that ran out somewhere in the block) is taken by all of them or by none.
__device__ __forceinline__ bool cons_any(bool v) {
    uint32_t r;
    asm volatile("{\n .reg .pred p, q;\n setp.ne.u32 q, %1, 0;\n bar.red.or.pred p, 1, %2, q;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(r) : "r"(static_cast<uint32_t>(v)), "n"(kCons) : "memory");
    return r != 0u;
}
__device__ __forceinline__ void red_release_add(unsigned* p, unsigned v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void unpack8(const uint4& raw, float (&f)[8]) {
    f[0] = __uint_as_float(raw.x << 16); f[1] = __uint_as_float(raw.x & 0xffff0000u);
    f[2] = __uint_as_float(raw.y << 16); f[3] = __uint_as_float(raw.y & 0xffff0000u);
    f[4] = __uint_as_float(raw.z << 16); f[5] = __uint_as_float(raw.z & 0xffff0000u);
    f[6] = __uint_as_float(raw.w << 16); f[7] = __uint_as_float(raw.w & 0xffff0000u);
}

// Where a block stands in the streamed sequence: consumer and producer count the same tasks in the same order.
struct BlockPlan {
    int p0, npair;           // P1: output pairs [p0, p0 + npair) of the QKV projection (2 npair logical rows)
    int o0, norow;           // P4: rows of Wo
    int f0, nfrow;           // P5: neurons
    int g, nb, bi;           // P2: KV head of this block, blocks of that head, index among them
};
__device__ __forceinline__ BlockPlan make_plan(const L1Params& p, int cta, int G) {
    BlockPlan b;
    const int P = (p.n_q + 2 * p.n_kv) * p.hd / 2;
    b.p0 = static_cast<int>(static_cast<int64_t>(cta) * P / G);
    b.npair = static_cast<int>(static_cast<int64_t>(cta + 1) * P / G) - b.p0;
    b.o0 = static_cast<int>(static_cast<int64_t>(cta) * p.d / G);
    b.norow = static_cast<int>(static_cast<int64_t>(cta + 1) * p.d / G) - b.o0;
    b.f0 = static_cast<int>(static_cast<int64_t>(cta) * p.d_ff / G);
    b.nfrow = static_cast<int>(static_cast<int64_t>(cta + 1) * p.d_ff / G) - b.f0;
    int g = static_cast<int>((static_cast<int64_t>(cta + 1) * p.n_kv - 1) / G);      // largest g with g G / n_kv <= cta
    while (g + 1 < p.n_kv && static_cast<int>(static_cast<int64_t>(g + 1) * G / p.n_kv) <= cta) ++g;
    while (g > 0 && static_cast<int>(static_cast<int64_t>(g) * G / p.n_kv) > cta) --g;
    const int b0 = static_cast<int>(static_cast<int64_t>(g) * G / p.n_kv), b1 = static_cast<int>(static_cast<int64_t>(g + 1) * G / p.n_kv);
    b.g = g; b.nb = b1 - b0; b.bi = cta - b0;
    return b;
}
// window of the sequence: tokens [lo, lo + L) of the cache, the newest at lo + L - 1
__device__ __forceinline__ void window_of(const L1Params& p, int n_raw, int window, int& lo, int& L) {
    int n = n_raw < 1 ? 1 : n_raw;
    n = n > p.cap ? static_cast<int>(p.cap) : n;
    L = (window > 0 && window < n) ? window : n;
    lo = n - L;
}
// the block's tokens [t0, t1) in window coordinates, and how many of them are streamed (all but the newest token of the window)
__device__ __forceinline__ void token_range(const BlockPlan& b, int L, int& t0, int& t1, int& nstream) {
    t0 = static_cast<int>(static_cast<int64_t>(L) * b.bi / b.nb);
    t1 = static_cast<int>(static_cast<int64_t>(L) * (b.bi + 1) / b.nb);
    nstream = (t1 == L ? t1 - 1 : t1) - t0;
    if (nstream < 0) nstream = 0;
}
// weight row of logical row j of P1 (the two rows of a rotary pair are neighbours: j even / odd)
__device__ __forceinline__ int qkv_row(const L1Params& p, int pp, int which) {
    const int hp = p.hd / 2, hr = p.r_attn / 2;
    const int head = pp / hp, q = pp - head * hp;
    if (head >= p.n_q + p.n_kv) return head * p.hd + 2 * q + which;
    if (q < hr) return head * p.hd + q + which * hr;
    return head * p.hd + p.r_attn + (q - hr) + which * ((p.hd - p.r_attn) / 2);
}
__device__ __forceinline__ int cdiv(int a, int b) { return (a + b - 1) / b; }

// Optional per-task cycle stamps of blocks 0..3 (build with -DSPARK_L1_DEBUG), stored behind the phase marks of the trace
// buffer: [kind 0 issued, 1 seen full, 2 freed][block][task < 512].  Compiled out otherwise.
__device__ __forceinline__ void dbg_stamp(const PhaseTrace& tr, int kind, long long task) {
#ifdef SPARK_L1_DEBUG
    if (tr.buf != nullptr && blockIdx.x < 4 && task < 512) {
        const long long i = 148 * 16 + (static_cast<long long>(kind) * 4 + blockIdx.x) * 512 + task;
        if (i < tr.cap) tr.buf[i] = static_cast<unsigned long long>(clock64());
    }
#endif
}

// Optional fine-grained marks (same debug build): block b < 4 stores its cycle counter in entry k < 64 behind the task stamps.
__device__ __forceinline__ void dbg_mark(const PhaseTrace& tr, int k) {
#ifdef SPARK_L1_DEBUG
    if (tr.buf != nullptr && blockIdx.x < 4 && threadIdx.x == 0 && k < 64) {
        const long long i = 148 * 16 + 3 * 4 * 512 + blockIdx.x * 64 + k;
        if (i < tr.cap) tr.buf[i] = static_cast<unsigned long long>(clock64());
    }
#endif
}

// ---- the producer: one lane streams the block's activation-independent bytes through the ring ----------------------------
struct Ring {
    uint32_t base;           // shared-memory address of slot 0
    uint32_t full0, empty0;  // addresses of the first full / empty mbarrier (8 bytes apart per slot)
    volatile unsigned* fillseq;   // per slot: 1 + the number of the use the producer is filling (or has filled) it for
    int slot_bytes, n_slots;
};
struct RingPos {             // position in the task sequence: slot and the parity of its use
    int slot;
    uint32_t use;
    __device__ __forceinline__ void next(int n_slots) {
        if (++slot == n_slots) { slot = 0; ++use; }
    }
    __device__ __forceinline__ void skip(int n, int n_slots) {      // n is a few ring lengths at most: no division
        slot += n;
        while (slot >= n_slots) { slot -= n_slots; ++use; }
    }
    __device__ __forceinline__ RingPos plus(int n, int n_slots) const {      // n < n_slots: no division
        RingPos q{slot + n, use};
        if (q.slot >= n_slots) { q.slot -= n_slots; ++q.use; }
        return q;
    }
};
// Consumer side: wait until use `q.use` of slot `q.slot` has landed.  A parity wait alone is ambiguous when the waiting warp is
// not the one that consumed the slot's previous use (the barrier may still be a whole phase behind), so the producer first
// publishes which use it is filling; the parity wait follows.
__device__ __forceinline__ bool wait_full(const Ring& rg, const RingPos& q, volatile int* fail, long long limit) {
    if (rg.fillseq[q.slot] != q.use + 1u) {
        const long long t0 = clock64();
        while (rg.fillseq[q.slot] != q.use + 1u) {
            if (*fail != 0) return false;
            if (clock64() - t0 > limit) {
                *fail = 1;
                return false;
            }
        }
    }
    return mb_wait(rg.full0 + 8u * q.slot, q.use & 1u, fail, limit);
}
// Producer side: wait until the slot is free for use `q.use`, then publish that use.
__device__ __forceinline__ bool claim_slot(const Ring& rg, const RingPos& q, volatile int* fail, long long limit) {
    if (!mb_wait(rg.empty0 + 8u * q.slot, (q.use & 1u) ^ 1u, fail, limit)) return false;
    rg.fillseq[q.slot] = q.use + 1u;
    return true;
}

// Slots.  A streamed matrix phase puts `rps` whole rows into a slot (a power of two up to 16), `rstride` bytes apart: 64 bytes
// more than a row's length, so that the 16-byte fragment loads of the tensor-core tiles (rows g and g + 1 in one wavefront)
// fall on distinct banks.  Every row is one bulk copy (a copy costs the copy engine about the same whatever its size, so
// rows are not cut further).  Sixteen consecutive rows are a row group: the M dimension of the MMA tiles.  The tokens of the
// attention's predictor slice arrive as they are stored, a multiple of 16 of them per slot.
struct RowPhase {
    int rps, rstride;        // rows per slot, bytes between rows
};
__device__ __forceinline__ RowPhase row_phase_of(int K, int slot_bytes) {
    RowPhase rp;
    rp.rstride = K * 2 + 64;
    rp.rps = 1;
    while (rp.rps < 16 && 2 * rp.rps * rp.rstride <= slot_bytes) rp.rps *= 2;
    return rp;
}

// Pacing.  The SM's path to memory serves requests in order: a small load that an activation depends on (the hidden state after
// a grid barrier, a barrier's own atomic) issued behind a full ring of bulk copies comes back only when those have drained,
// microseconds later.  The producer therefore keeps at most `max_inflight` slots in flight (issued, not yet landed): enough to
// cover bandwidth x latency, no more; the rest of the ring holds what has already landed.
struct Pace {
    RingPos land;            // oldest slot not yet known to have landed
    long long landed;        // slots known to have landed
    int max_inflight;
};
// Called by one lane before `n` more slots are issued (issued = slots issued so far): waits until n more fit.
__device__ __forceinline__ bool pace_wait(const Ring& rg, Pace& pc, long long issued, int n, volatile int* fail, long long limit) {
    while (issued + n - pc.landed > pc.max_inflight && pc.landed < issued) {
        if (!mb_wait(rg.full0 + 8u * pc.land.slot, pc.land.use & 1u, fail, limit)) return false;
        pc.land.next(rg.n_slots);
        ++pc.landed;
    }
    return true;
}

// A task of the attention's predictor slice: m consecutive slots (not across the ring's end) holding n tokens (a multiple of 16
// unless they are the last).  Producer and consumers derive the same tasks from the same ring position.
constexpr int kP2Slots = 8;
__device__ __forceinline__ void p2_task(const Ring& rg, const RingPos& pos, int remaining, uint32_t tok_b, int& m, int& n) {
    int mm = rg.n_slots - pos.slot;
    if (mm > kP2Slots) mm = kP2Slots;
    int cap_tok = static_cast<int>(static_cast<uint32_t>(mm) * rg.slot_bytes / tok_b) & ~15;
    if (cap_tok < 16) {      // the ring's last slot alone holds fewer than 16 tokens only if a slot does (the host rules that out)
        cap_tok = 16;
    }
    n = remaining < cap_tok ? remaining : cap_tok;
    m = static_cast<int>((static_cast<uint32_t>(n) * tok_b + rg.slot_bytes - 1) / rg.slot_bytes);
}

// One matrix phase of the producer (all 32 lanes): rows `rowmap(j)` of W (ld elements per row, K of them used).  A lane per row;
// the lane of a slot's first row waits until the slot is free and announces the bytes.
template <typename RowMap>
__device__ __forceinline__ bool produce_rows(const Ring& rg, RingPos& pos, long long& issued, Pace& pc, const __nv_bfloat16* W, int64_t ld, int K, int nrows,
                                             RowMap rowmap, volatile int* fail, long long limit, const PhaseTrace& tr) {
    const int lane = threadIdx.x & 31;
    const RowPhase rp = row_phase_of(K, rg.slot_bytes);
    int spi = 32;                                              // slots per trip, a lane each
    if (spi > rg.n_slots - 1) spi = rg.n_slots - 1;
    if (spi > pc.max_inflight) spi = pc.max_inflight;
    const int nslot = cdiv(nrows, rp.rps);
    bool all_ok = true;
    for (int s0 = 0; s0 < nslot && all_ok; s0 += spi) {
        const int done = min(spi, nslot - s0);
        bool ok = true;
        if (lane == 0) ok = pace_wait(rg, pc, issued, done, fail, limit);
        if (__any_sync(kFull, !ok)) return false;
        // A lane claims its slot and issues that slot's copies at once: a lane whose slot is not free yet (its previous use is
        // still being consumed) must not hold back the copies of the lanes before it -- the consumers may be waiting for those.
        if (lane < done) {
            const int sl = s0 + lane;
            const RingPos my = pos.plus(lane, rg.n_slots);
            const uint32_t bar = rg.full0 + 8u * my.slot;
            ok = claim_slot(rg, my, fail, limit);
            if (ok) {
                const int n = min(rp.rps, nrows - sl * rp.rps);
                mb_expect_tx(bar, static_cast<uint32_t>(n) * K * 2u);
                for (int j = 0; j < n; ++j)
                    bulk_g2s(rg.base + static_cast<uint32_t>(my.slot) * rg.slot_bytes + j * rp.rstride,
                             W + static_cast<int64_t>(rowmap(sl * rp.rps + j)) * ld, static_cast<uint32_t>(K) * 2u, bar);
            }
            dbg_stamp(tr, 0, issued + lane);
        }
        all_ok = !__any_sync(kFull, !ok);
        pos.skip(done, rg.n_slots);
        issued += done;
    }
    return all_ok;
}

__device__ __noinline__ void l1_producer(const L1Params& p, const BlockPlan& bp, const Ring& rg, volatile int* fail, long long limit) {
    const int lane = threadIdx.x & 31;
    RingPos pos{0, 0u};
    long long issued = 0;
    Pace pc{RingPos{0, 0u}, 0, p.max_inflight};
    bool waited = false, ok = true;
    const uint32_t tok_b = static_cast<uint32_t>(p.r_attn) * 2u;
    for (int l = 0; l < p.n_layers && ok; ++l) {
        const L1Layer& ly = p.layer[l];
        // P1: rows of Wqkv in the order of the block's rotary pairs
        ok = produce_rows(rg, pos, issued, pc, ly.Wqkv, p.d, p.d, 2 * bp.npair,
                           [&](int j) { return qkv_row(p, bp.p0 + (j >> 1), j & 1); }, fail, limit, p.trace);
        if (!ok) break;
        if (!waited) {       // the sequence length may come from the kernel ahead in the stream
            dep_wait();
            waited = true;
        }
        // P2: the predictor slice of the block's tokens (all but the newest of the window, which P1 is writing), as stored
        int lo, L, t0, t1, ns;
        window_of(p, *reinterpret_cast<const volatile int*>(p.ctx_len), ly.window, lo, L);
        token_range(bp, L, t0, t1, ns);
        const __nv_bfloat16* kb = ly.k1c + (static_cast<int64_t>(bp.g) * p.cap + lo + t0) * p.r_attn;
        for (int i = 0; i < ns && ok;) {
            // a task: as many consecutive slots as hold the next tokens (up to kP2Slots, not across the ring's end), one copy
            int m, n;
            p2_task(rg, pos, ns - i, tok_b, m, n);
            bool mine_ok = true;
            if (lane == 0) mine_ok = pace_wait(rg, pc, issued, m, fail, limit);
            if (__any_sync(kFull, !mine_ok)) { ok = false; break; }
            if (lane < m) {
                const RingPos my = pos.plus(lane, rg.n_slots);
                mine_ok = claim_slot(rg, my, fail, limit);
                if (mine_ok && lane > 0) mb_arrive_n(rg.full0 + 8u * my.slot, 1u);       // the copy completes on the first slot's barrier
            }
            ok = !__any_sync(kFull, !mine_ok);
            if (ok && lane == 0) {
                const uint32_t bar = rg.full0 + 8u * pos.slot;
                mb_expect_tx(bar, n * tok_b);
                bulk_g2s(rg.base + static_cast<uint32_t>(pos.slot) * rg.slot_bytes, kb + static_cast<int64_t>(i) * p.r_attn, n * tok_b, bar);
                dbg_stamp(p.trace, 0, issued);
            }
            pos.skip(m, rg.n_slots);
            issued += m;
            i += n;
        }
        if (!ok) break;
        // P4: rows of Wo;  P5: rows of K1t
        ok = produce_rows(rg, pos, issued, pc, ly.Wo, p.n_q * p.hd, p.n_q * p.hd, bp.norow, [&](int j) { return bp.o0 + j; }, fail, limit, p.trace);
        if (!ok) break;
        ok = produce_rows(rg, pos, issued, pc, ly.K1t, p.r_ff, p.r_ff, bp.nfrow, [&](int j) { return bp.f0 + j; }, fail, limit, p.trace);
    }
    if (!waited) dep_wait();
    // Nothing may still be landing in shared memory when the block leaves: wait (bounded, whatever the abort flag says) for
    // the last copies issued into each slot.  In a run without a failure the consumers have waited for all of them already.
    if (lane == 0) {
        const int back = issued < rg.n_slots ? static_cast<int>(issued) : rg.n_slots;
        for (int k = 0; k < back; ++k) {
            if (--pos.slot < 0) { pos.slot = rg.n_slots - 1; --pos.use; }
            const long long t0 = clock64();
            while (!mb_try(rg.full0 + 8u * pos.slot, pos.use & 1u)) {
                if (clock64() - t0 > 20000000ll) break;
            }
        }
    }
}

// ---- consumer pieces ----------------------------------------------------------------------------------------------------
struct ConsCtx {
    Ring rg;
    volatile int* fail;
    long long limit;
    int tid, lane, warp;
    PhaseTrace tr;
    int mk;                  // debug: base index of the fine-grained marks of the current step
};

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ unsigned bf16_bits(float x) { return static_cast<unsigned>(__bfloat16_as_ushort(__float2bfloat16_rn(x))); }

// The input vector as three bf16 terms (hi + mid + lo = x to fp32 accuracy: 24 significant bits), one row per term,
// `stride` bytes apart (64 bytes more than a multiple of 128: the fragment loads of the three rows fall on distinct banks).
// The tensor-core tiles multiply the bf16 weights by each term (products exact in fp32) and the three columns are added.
__device__ __forceinline__ void stage_split3(const ConsCtx& c, const float* xs, int K, unsigned char* xsp, int stride) {
    for (int i = c.tid; i < K / 2; i += kCons) {
        const float2 v = reinterpret_cast<const float2*>(xs)[i];
        unsigned w[3];
        float a = v.x, b = v.y;
#pragma unroll
        for (int t = 0; t < 3; ++t) {
            const unsigned ha = bf16_bits(a), hb = bf16_bits(b);
            w[t] = ha | (hb << 16);
            a -= __uint_as_float(ha << 16);
            b -= __uint_as_float(hb << 16);
        }
#pragma unroll
        for (int t = 0; t < 3; ++t) *reinterpret_cast<unsigned*>(xsp + static_cast<size_t>(t) * stride + 4 * i) = w[t];
    }
}

// Column parts a row group's work is split into: as many as give every warp a task (a power of two, at most the number of
// 32-column blocks).
__device__ __forceinline__ int group_parts(int nrows, int K) {
    const int ngroups = cdiv(nrows, 16);
    int m = 1;
    while (2 * m * ngroups <= kConsWarps && 2 * m <= K / 32) m *= 2;
    return m;
}

// A streamed matrix phase on the tensor cores.  A task is (row group of 16 rows = the M dimension, column part); task tau goes to
// warp tau % 16, which waits for the group's slots, multiplies its columns and frees the slots with its share of the sixteen
// arrivals.  A lane takes 16-byte pieces of rows g = lane / 4 and g + 8: the k-slots of an MMA may be any permutation of the
// columns as long as both operands use it, so a piece feeds two m16n8k16 MMAs; the B operand holds the three terms of the
// input in columns 0..2.  out[row * 16 + part] receives the partial dot products.  `pos`: ring position of the phase's first
// slot on entry, of the next phase's first slot on return.
__device__ __forceinline__ bool group_phase(const ConsCtx& c, RingPos& pos, int nrows, int K, const unsigned char* xsp, int xstride, float* out) {
    dbg_mark(c.tr, c.mk + 14);
    const RowPhase rp = row_phase_of(K, c.rg.slot_bytes);
    const int lrps = 31 - __clz(rp.rps), spg = 16 >> lrps;
    const int g = c.lane >> 2, t = c.lane & 3;
    const int nb = K / 32, ngroups = cdiv(nrows, 16), m = group_parts(nrows, K), lm = 31 - __clz(m);
    const unsigned char* ring = reinterpret_cast<const unsigned char*>(__cvta_shared_to_generic(c.rg.base));
    const unsigned char* bp = xsp + static_cast<size_t>(g) * xstride + t * 16;
    bool ok = true;
    for (int tau = c.warp; tau < (ngroups << lm) && ok; tau += kConsWarps) {
        const int gi = tau >> lm, part = tau & (m - 1);
        const int r0 = gi * 16, nr = min(16, nrows - r0), nsl = (nr + rp.rps - 1) >> lrps;
        RingPos base = pos;
        base.skip(gi * spg, c.rg.n_slots);
        const RingPos my = base.plus(c.lane < nsl ? c.lane : 0, c.rg.n_slots);
        bool mine_ok = true;
        if (tau == 0) dbg_mark(c.tr, c.mk + 11);
        if (c.lane < nsl) mine_ok = wait_full(c.rg, my, c.fail, c.limit);
        ok = !__any_sync(kFull, !mine_ok);
        if (c.lane == 0) dbg_stamp(c.tr, 1, static_cast<long long>(my.use) * c.rg.n_slots + my.slot);
        dbg_mark(c.tr, c.mk + 9);
        if (ok) {
            const int kb0 = part * nb >> lm, kb1 = (part + 1) * nb >> lm;
            int s_lo = base.slot + (g >> lrps), s_hi = base.slot + ((g + 8) >> lrps);
            s_lo -= s_lo >= c.rg.n_slots ? c.rg.n_slots : 0;
            s_hi -= s_hi >= c.rg.n_slots ? c.rg.n_slots : 0;
            const unsigned char* ra = ring + static_cast<size_t>(s_lo) * c.rg.slot_bytes + (g & (rp.rps - 1)) * rp.rstride + t * 16;
            const unsigned char* rb = ring + static_cast<size_t>(s_hi) * c.rg.slot_bytes + ((g + 8) & (rp.rps - 1)) * rp.rstride + t * 16;
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
            for (int kb = kb0; kb < kb1; ++kb) {
                const uint4 a_lo = *reinterpret_cast<const uint4*>(ra + kb * 64);
                const uint4 a_hi = *reinterpret_cast<const uint4*>(rb + kb * 64);
                uint4 b = make_uint4(0u, 0u, 0u, 0u);
                if (g < 3) b = *reinterpret_cast<const uint4*>(bp + kb * 64);
                mma_bf16_16816(acc, a_lo.x, a_hi.x, a_lo.y, a_hi.y, b.x, b.y);
                mma_bf16_16816(acc, a_lo.z, a_hi.z, a_lo.w, a_hi.w, b.z, b.w);
            }
            if (tau == 0) dbg_mark(c.tr, c.mk + 12);
            __syncwarp();
            if (c.lane < nsl) mb_arrive_n(c.rg.empty0 + 8u * my.slot, static_cast<uint32_t>(kConsWarps >> lm));
            if (tau == 0) dbg_mark(c.tr, c.mk + 13);
            if (c.lane == 0) dbg_stamp(c.tr, 2, static_cast<long long>(my.use) * c.rg.n_slots + my.slot);
            // columns 0, 1 (lane t = 0) and 2 (lane t = 1) of the accumulator tile are the three terms
            const float lo = acc[0] + acc[1] + __shfl_down_sync(kFull, acc[0], 1);
            const float hi = acc[2] + acc[3] + __shfl_down_sync(kFull, acc[2], 1);
            if (t == 0) {
                if (g < nr) out[(r0 + g) * kConsWarps + part] = lo;
                if (g + 8 < nr) out[(r0 + g + 8) * kConsWarps + part] = hi;
            }
        }
    }
    dbg_mark(c.tr, c.mk + 10);
    pos.skip((nrows + rp.rps - 1) >> lrps, c.rg.n_slots);
    return ok;
}

// Grid-wide barrier number `target_gen` (counted since the workspace was reset): one thread adds the block's arrival to its way,
// sixteen lanes poll the ways until they add up to target_gen x blocks.  Called by all consumer threads.
__device__ __forceinline__ bool grid_barrier(const ConsCtx& c, WsHeader* hdr, unsigned target_gen, int G, int cta) {
    dbg_mark(c.tr, c.mk);
    cons_sync();             // everything this block wrote before is ordered before the arrival (bar.sync + release)
    dbg_mark(c.tr, c.mk + 1);
    bool ok = true;
    if (c.warp == 0) {
        if (c.lane == 0) {
            __threadfence();
            dbg_mark(c.tr, c.mk + 2);
            red_release_add(&hdr->l1_ways[cta % kCellWays].count, 1u);
            dbg_mark(c.tr, c.mk + 3);
        }
        const unsigned target = target_gen * static_cast<unsigned>(G);
        const long long t0 = clock64();
        for (;;) {
            unsigned v = c.lane < kCellWays ? ld_acquire_u32(&hdr->l1_ways[c.lane].count) : 0u;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
            if (static_cast<int>(v - target) >= 0) break;
            if (*c.fail != 0 || clock64() - t0 > c.limit) {
                if (c.lane == 0) {
                    atomicCAS(&hdr->status, SPARK_OK, SPARK_ERR_TIMEOUT);
                    *c.fail = 1;
                }
                ok = false;
                break;
            }
        }
    }
    dbg_mark(c.tr, c.mk + 4);
    const bool bad = cons_any(!ok || *c.fail != 0);
    dbg_mark(c.tr, c.mk + 5);
    return !bad;
}

// Block-wide sum over the consumer threads (scratch: 16 floats of shared memory).
__device__ __forceinline__ float cons_sum(const ConsCtx& c, float v, float* scratch) {
    v = warp_sum(v);
    cons_sync();
    if (c.lane == 0) scratch[c.warp] = v;
    cons_sync();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kConsWarps; ++w) t += scratch[w];
    return t;
}

// x = RMSNorm(h; w) into shared memory as fp32 and as three bf16 terms (all consumer threads; h read past L1: other blocks
// wrote it; the norm weights are requested together with h: one trip to memory, not two).
__device__ __forceinline__ void stage_rmsnorm(const ConsCtx& c, const L1Params& p, const float* norm_w, float* xs, float* scratch,
                                              unsigned char* xsp, int xstride) {
    const int d4 = p.d / 4;
    const bool h0 = c.tid < d4, h1 = c.tid + kCons < d4;          // d <= 4096: at most two float4 per thread
    float4 v0 = make_float4(0.f, 0.f, 0.f, 0.f), v1 = v0, w0 = v0, w1 = v0;
    if (h0) { v0 = __ldcg(reinterpret_cast<const float4*>(p.h) + c.tid); w0 = __ldg(reinterpret_cast<const float4*>(norm_w) + c.tid); }
    if (h1) { v1 = __ldcg(reinterpret_cast<const float4*>(p.h) + c.tid + kCons); w1 = __ldg(reinterpret_cast<const float4*>(norm_w) + c.tid + kCons); }
    const float ss = v0.x * v0.x + v0.y * v0.y + v0.z * v0.z + v0.w * v0.w + v1.x * v1.x + v1.y * v1.y + v1.z * v1.z + v1.w * v1.w;
    dbg_mark(c.tr, c.mk + 6);
    const float tot = cons_sum(c, ss, scratch);
    dbg_mark(c.tr, c.mk + 7);
    const float sc = rsqrtf(tot / static_cast<float>(p.d) + p.eps);
    if (h0) reinterpret_cast<float4*>(xs)[c.tid] = make_float4(v0.x * sc * w0.x, v0.y * sc * w0.y, v0.z * sc * w0.z, v0.w * sc * w0.w);
    if (h1) reinterpret_cast<float4*>(xs)[c.tid + kCons] = make_float4(v1.x * sc * w1.x, v1.y * sc * w1.y, v1.z * sc * w1.z, v1.w * sc * w1.w);
    cons_sync();
    stage_split3(c, xs, p.d, xsp, xstride);
    cons_sync();
    dbg_mark(c.tr, c.mk + 8);
}

__device__ __noinline__ double upper_quantile(int k, int L) {
    return k >= L ? 0.0 : -normcdfinv(static_cast<double>(k) / static_cast<double>(L));
}
__device__ __noinline__ void sincos_turns(double turns, float& sn, float& cs) {
    // angle reduced to one turn in fp64 (positions reach tens of thousands of radians), sine and cosine in fp32
    const float ang = static_cast<float>((turns - floor(turns)) * 6.28318530717958647692);
    sincosf(ang, &sn, &cs);
}

// ---- the kernel ---------------------------------------------------------------------------------------------------------
struct L1Shared {            // static shared memory
    unsigned long long bars[2 * 64 + 1];      // full[64], empty[64], gather
    unsigned fillseq[64];
    double red_d[kConsWarps][4][2];
    float red_m[kConsWarps][4];
    float scratch[kConsWarps];
    float theta_s[4], smax_s[4], l_s[4];
    int sel_n[4];
    double z_attn[kMaxLayers];                // Q(1 - k_attn / L) of every layer's window
    float theta_ff;
    int nact;
    int fail;
    unsigned epoch0, gen0;
    int flist_j[256];
    float flist_a[256];
    float uval[256];
    float s_loc[256];
    float outp[2048];
};

template <int GQ>
__global__ void __launch_bounds__(kThreadsL1, 1) layer1_kernel(const __grid_constant__ L1Params p) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ L1Shared sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int G = gridDim.x, cta = blockIdx.x;
    const BlockPlan bp = make_plan(p, cta, G);
    Ring rg;
    rg.base = saddr(smem + p.off_ring);
    rg.full0 = saddr(&sh.bars[0]);
    rg.empty0 = saddr(&sh.bars[64]);
    rg.fillseq = sh.fillseq;
    rg.slot_bytes = p.slot_bytes;
    rg.n_slots = p.n_slots;
    const uint32_t gbar = saddr(&sh.bars[128]);
    if (tid == 0) {
        for (int i = 0; i < p.n_slots; ++i) {
            mb_init(rg.full0 + 8u * i, 1u);
            mb_init(rg.empty0 + 8u * i, kEmptyCount);
        }
        mb_init(gbar, 1u);
        for (int i = 0; i < 64; ++i) sh.fillseq[i] = 0u;
        sh.fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    volatile int* fail = &sh.fail;
    if (warp == kConsWarps) {                  // ---------------- producer warp ----------------
        l1_producer(p, bp, rg, fail, spin_limit(p.hdr));
        return;
    }
    // ---------------- consumers ----------------
    dep_wait();
    dep_trigger();
    ConsCtx c;
    c.rg = rg; c.fail = fail; c.limit = spin_limit(p.hdr); c.tid = tid; c.lane = lane; c.warp = warp; c.tr = p.trace;
    if (tid == 0) {
        sh.epoch0 = ld_acquire_u32(&p.hdr->epoch);
        sh.gen0 = ld_acquire_u32(&p.hdr->l1_gen);
    }
    float* xs = reinterpret_cast<float*>(smem + p.off_act);
    unsigned char* xsp = smem + p.off_xsp;                                     // three bf16 terms of the staged input (or of the queries)
    float* sc = reinterpret_cast<float*>(smem + p.off_sc);                     // [GQ][ntok_cap] predictor scores
    int* sel_tok = reinterpret_cast<int*>(sc + GQ * p.ntok_cap);               // [GQ][ntok_cap] selected tokens (block-local index)
    float* sel_a = reinterpret_cast<float*>(sel_tok + GQ * p.ntok_cap);        // [GQ][ntok_cap] s - s_max, then weight x gate
    unsigned char* gat = smem + p.off_gather;
    const uint32_t gat_s = saddr(gat);
    const int hd = p.hd, r = p.r_attn, d2 = hd - r, nqo = p.n_q * hd;
    const int half = lane >> 4, hl = lane & 15;
    RingPos pos{0, 0u};
    uint32_t gpar = 0u;                        // parity of the gather barrier's next completion
    unsigned nbar = 0u;                        // grid barriers passed in this launch
    cons_sync();
    const unsigned epoch0 = sh.epoch0, gen0 = sh.gen0;
    const int n_raw = *reinterpret_cast<const volatile int*>(p.ctx_len);
    const int n_clamped = n_raw < 1 ? 1 : (n_raw > p.cap ? static_cast<int>(p.cap) : n_raw);
    const int tpos = n_clamped - 1;            // position of the token being decoded
    if (tid < p.n_layers) {                    // the threshold quantile of every layer's window, once per launch
        int lo_, L_;
        window_of(p, n_raw, p.layer[tid].window, lo_, L_);
        sh.z_attn[tid] = upper_quantile(p.k_attn, L_);
    }
    p.trace.mark(0);

    for (int l = 0; l < p.n_layers; ++l) {
        const L1Layer& ly = p.layer[l];
        int lo, L, t0, t1, ns;
        window_of(p, n_raw, ly.window, lo, L);
        token_range(bp, L, t0, t1, ns);
        const int ntok = t1 - t0;
        const bool ident = p.k_attn >= L;

        // =========================== P1: QKV projection, rotary encoding, cache append ===========================
        c.mk = 0;
        stage_rmsnorm(c, p, ly.norm1, xs, sh.scratch, xsp, p.xstride);
        for (int i = cta * kCons + tid; i < nqo; i += G * kCons) p.obuf[i] = 0.f;
        if (cta == 0 && tid < p.n_q) p.lsum[tid] = 0.f;
        if (!group_phase(c, pos, 2 * bp.npair, p.d, xsp, p.xstride, sh.outp)) *fail = 1;
        if (cons_any(*fail != 0)) break;
        for (int pr = tid; pr < bp.npair; pr += kCons) {
            float v0 = 0.f, v1 = 0.f;
            const int nkc = kConsWarps, np = group_parts(2 * bp.npair, p.d);
            for (int s = 0; s < np; ++s) { v0 += sh.outp[(2 * pr) * nkc + s]; v1 += sh.outp[(2 * pr + 1) * nkc + s]; }
            const int pp = bp.p0 + pr, hp = hd / 2, hr = r / 2;
            const int head = pp / hp, q = pp - head * hp;
            if (head >= p.n_q + p.n_kv) {                               // value rows: stored as they are
                const int gk = head - p.n_q - p.n_kv;
                __nv_bfloat16* dst = ly.vc + (static_cast<int64_t>(gk) * p.cap + tpos) * hd;
                dst[2 * q] = __float2bfloat16_rn(v0);
                dst[2 * q + 1] = __float2bfloat16_rn(v1);
                continue;
            }
            const bool second = q >= hr;
            const int pi = second ? q - hr : q, m = second ? d2 : r;
            // angle = pos * base^(-2i/m): product and reduction to one turn in fp64, sine and cosine in fp32
            const double turns = static_cast<double>(tpos) * p.inv_freq[second ? 1 : 0][pi] * 0.15915494309189533577;
            float sn, cs;
            sincos_turns(turns, sn, cs);
            const float ra = v0 * cs - v1 * sn, rb = v0 * sn + v1 * cs;
            if (head < p.n_q) {
                float* dst = p.qbuf + static_cast<int64_t>(head) * hd + (second ? r : 0);
                dst[pi] = ra * p.q_scale;
                dst[pi + m / 2] = rb * p.q_scale;
            } else {
                const int64_t rowi = static_cast<int64_t>(head - p.n_q) * p.cap + tpos;
                __nv_bfloat16* dst = second ? ly.k2c + rowi * d2 : ly.k1c + rowi * r;
                dst[pi] = __float2bfloat16_rn(ra);
                dst[pi + m / 2] = __float2bfloat16_rn(rb);
            }
        }
        p.trace.mark(1);
        if (!grid_barrier(c, p.hdr, gen0 + (++nbar), G, cta)) break;
        p.trace.mark(2);

        // =========================== P2: predictor scores of the block's tokens ===================================
        // the query heads of this block's KV head (written by other blocks: read past L1), as fp32 and as three bf16 terms
        float* qs = xs;                                                  // [GQ][hd]
        for (int i = tid; i < GQ * hd / 4; i += kCons)
            reinterpret_cast<float4*>(qs)[i] = __ldcg(reinterpret_cast<const float4*>(p.qbuf + static_cast<int64_t>(bp.g) * GQ * hd) + i);
        if (tid < GQ) { sh.sel_n[tid] = 0; sh.l_s[tid] = 0.f; }
        cons_sync();
        for (int i = tid; i < GQ * (r / 2); i += kCons) {                // rows 3 h + term of the split: q[h][:r]
            const int h = i / (r / 2), j = i - h * (r / 2);
            const float2 v = reinterpret_cast<const float2*>(qs + h * hd)[j];
            float a = v.x, b = v.y;
#pragma unroll
            for (int t = 0; t < 3; ++t) {
                const unsigned ha = bf16_bits(a), hb = bf16_bits(b);
                *reinterpret_cast<unsigned*>(xsp + static_cast<size_t>(3 * h + t) * p.qstride + 4 * j) = ha | (hb << 16);
                a -= __uint_as_float(ha << 16);
                b -= __uint_as_float(hb << 16);
            }
        }
        cons_sync();
        {
            double s1[GQ], s2[GQ];
            float mx[GQ];
#pragma unroll
            for (int h = 0; h < GQ; ++h) { s1[h] = 0.0; s2[h] = 0.0; mx[h] = -INFINITY; }
            auto keep = [&](int h, int tl, float v) {                    // one lane per (token, head)
                sc[h * p.ntok_cap + tl] = v;
                const double dv = static_cast<double>(v);
                s1[h] += dv;
                s2[h] = fma(dv, dv, s2[h]);
                mx[h] = fmaxf(mx[h], v);
            };
            // Sixteen tokens are the M dimension of an MMA tile, the columns hold the three terms of up to two query heads
            // (columns 3 h' + term); lane pieces as in group_phase.  Token rows lie r_attn values apart, as stored.
            const int mg = lane >> 2, mt = lane & 3, nk32 = r / 32;
            constexpr int NP = (GQ + 1) / 2;                             // passes of two heads
            int tile_no = 0;                                             // tiles of 16 tokens go to the warps round-robin
            const uint32_t tok_b = static_cast<uint32_t>(r) * 2u;
            for (int i = 0; i < ns;) {
                int m, n;
                p2_task(rg, pos, ns - i, tok_b, m, n);                   // the producer's task: m slots, n tokens, one copy
                const RingPos my = pos.plus(lane < m ? lane : 0, rg.n_slots);
                bool mine_ok = true;
                if (lane < m) mine_ok = wait_full(rg, my, fail, c.limit);
                if (__any_sync(kFull, !mine_ok)) break;
                if (lane == 0) dbg_stamp(c.tr, 1, static_cast<long long>(pos.use) * rg.n_slots + pos.slot);
                const unsigned char* sp = smem + p.off_ring + static_cast<size_t>(pos.slot) * rg.slot_bytes;
                for (int tb = 0; tb < n; tb += 16, ++tile_no) {
                    if ((tile_no & (kConsWarps - 1)) != warp) continue;
                    float acc[NP][4];
#pragma unroll
                    for (int hp = 0; hp < NP; ++hp) { acc[hp][0] = acc[hp][1] = acc[hp][2] = acc[hp][3] = 0.f; }
                    for (int kb = 0; kb < nk32; ++kb) {
                        const uint4 a_lo = *reinterpret_cast<const uint4*>(sp + static_cast<size_t>(tb + mg) * r * 2 + kb * 64 + mt * 16);
                        const uint4 a_hi = *reinterpret_cast<const uint4*>(sp + static_cast<size_t>(tb + mg + 8) * r * 2 + kb * 64 + mt * 16);
#pragma unroll
                        for (int hp = 0; hp < NP; ++hp) {
                            uint4 bq = make_uint4(0u, 0u, 0u, 0u);
                            if (mg < 3 * (GQ - 2 * hp >= 2 ? 2 : 1))
                                bq = *reinterpret_cast<const uint4*>(xsp + static_cast<size_t>(6 * hp + mg) * p.qstride + kb * 64 + mt * 16);
                            mma_bf16_16816(acc[hp], a_lo.x, a_hi.x, a_lo.y, a_hi.y, bq.x, bq.y);
                            mma_bf16_16816(acc[hp], a_lo.z, a_hi.z, a_lo.w, a_hi.w, bq.z, bq.w);
                        }
                    }
#pragma unroll
                    for (int hp = 0; hp < NP; ++hp) {
                        // head 2 hp: columns 0..2 (lane t = 0: both, t = 1: first); head 2 hp + 1: columns 3..5 (t = 1: second, t = 2: both)
                        float pa0 = mt == 0 ? acc[hp][0] + acc[hp][1] : (mt == 1 ? acc[hp][0] : 0.f);
                        float pa1 = mt == 0 ? acc[hp][2] + acc[hp][3] : (mt == 1 ? acc[hp][2] : 0.f);
                        float pb0 = mt == 1 ? acc[hp][1] : (mt == 2 ? acc[hp][0] + acc[hp][1] : 0.f);
                        float pb1 = mt == 1 ? acc[hp][3] : (mt == 2 ? acc[hp][2] + acc[hp][3] : 0.f);
#pragma unroll
                        for (int o = 1; o <= 2; o <<= 1) {
                            pa0 += __shfl_xor_sync(kFull, pa0, o);
                            pa1 += __shfl_xor_sync(kFull, pa1, o);
                            pb0 += __shfl_xor_sync(kFull, pb0, o);
                            pb1 += __shfl_xor_sync(kFull, pb1, o);
                        }
                        const int tl0 = i + tb + mg;
                        if (mt == 0) {
                            if (tb + mg < n) keep(2 * hp, tl0, pa0);
                            if (tb + mg + 8 < n) keep(2 * hp, tl0 + 8, pa1);
                        }
                        if (mt == 1 && 2 * hp + 1 < GQ) {
                            if (tb + mg < n) keep(2 * hp + 1 < GQ ? 2 * hp + 1 : 0, tl0, pb0);
                            if (tb + mg + 8 < n) keep(2 * hp + 1 < GQ ? 2 * hp + 1 : 0, tl0 + 8, pb1);
                        }
                    }
                }
                __syncwarp();
                if (lane < m) mb_arrive_n(rg.empty0 + 8u * my.slot, 1u);      // every warp passes through every task
                if (lane == 0) dbg_stamp(c.tr, 2, static_cast<long long>(pos.use) * rg.n_slots + pos.slot);
                pos.skip(m, rg.n_slots);
                i += n;
            }
            // the newest token of the window (the row P1 has just written) comes straight from memory: plain fp32 arithmetic
            if (warp == kConsWarps - 1 && t1 == L && ntok > 0) {
                const __nv_bfloat16* row = ly.k1c + (static_cast<int64_t>(bp.g) * p.cap + lo + L - 1) * r;
                float wf[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                if (lane < r / 8) unpack8(__ldcg(reinterpret_cast<const uint4*>(row) + lane), wf);
#pragma unroll
                for (int h = 0; h < GQ; ++h) {
                    float a = 0.f;
                    if (lane < r / 8) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) a = fmaf(wf[e], qs[h * hd + lane * 8 + e], a);
                    }
                    a = warp_sum(a);
                    if (lane == 0) keep(h, ntok - 1, a);
                }
            }
#pragma unroll
            for (int h = 0; h < GQ; ++h) {
                const double a = warp_sum_f64(s1[h]), b2 = warp_sum_f64(s2[h]);
                const float m = warp_max(mx[h]);
                if (lane == 0) { sh.red_d[warp][h][0] = a; sh.red_d[warp][h][1] = b2; sh.red_m[warp][h] = m; }
            }
        }
        if (cons_any(*fail != 0)) break;
        p.trace.mark(3);
        // ---- X2: the block's sums to the cells of its heads; theta per head once every block of the KV head has arrived
        if (warp < GQ) {
            double a = lane < kConsWarps ? sh.red_d[lane][warp][0] : 0.0, b = lane < kConsWarps ? sh.red_d[lane][warp][1] : 0.0;
            float m = lane < kConsWarps ? sh.red_m[lane][warp] : -INFINITY;
            a = warp_sum_f64(a);
            b = warp_sum_f64(b);
            m = warp_max(m);
            SumCell* ways = p.attn_cells + static_cast<size_t>(bp.g * GQ + warp) * kAttnWays;
            if (lane == 0) cells_add_max_w<kAttnWays>(ways, bp.bi, a, b, m);
            double sa, sq;
            float smax;
            const bool ok = cells_wait_max_w<kAttnWays>(ways, static_cast<unsigned>(bp.nb), sa, sq, smax, p.hdr);
            if (lane == 0) {
                if (!ok) *fail = 1;
                float th = -INFINITY;
                if (!ident) {
                    const double n = static_cast<double>(L), mean = sa / n;
                    double var = (sq - sa * mean) / (n - 1.0);
                    var = var > 0.0 ? var : 0.0;
                    th = static_cast<float>(mean + sqrt(var) * sh.z_attn[l]);
                }
                sh.theta_s[warp] = th;
                sh.smax_s[warp] = smax;
            }
        }
        if (cons_any(*fail != 0)) break;
        p.trace.mark(4);

        // =========================== P3: selection, gather, softmax x gate x value ================================
        for (int i = tid; i < GQ * ntok; i += kCons) {
            const int h = i / ntok, t = i - h * ntok;
            const float s = sc[h * p.ntok_cap + t];
            if (ident || s > sh.theta_s[h]) {
                const int e = atomicAdd(&sh.sel_n[h], 1);
                sel_tok[h * p.ntok_cap + e] = t;
                sel_a[h * p.ntok_cap + e] = s - sh.smax_s[h];           // softmax is shift-invariant: the head's largest score is the reference
            }
        }
        cons_sync();
        {
            int nsel[GQ], total = 0;
#pragma unroll
            for (int h = 0; h < GQ; ++h) { nsel[h] = sh.sel_n[h]; total += nsel[h]; }
            const int tokb = (d2 + hd) * 2, cap_e = p.gather_bytes / tokb;
            const int64_t krow0 = (static_cast<int64_t>(bp.g) * p.cap + lo + t0) * d2, vrow0 = (static_cast<int64_t>(bp.g) * p.cap + lo + t0) * hd;
            // entry e of the concatenated lists -> (head, index in that head's list)
            auto entry = [&](int e, int& h, int& k) {
                h = 0;
                k = e;
#pragma unroll
                for (int hh = 0; hh < GQ - 1; ++hh)
                    if (h == hh && k >= nsel[hh]) { k -= nsel[hh]; h = hh + 1; }
            };
            constexpr int NV = 2;                                        // output columns per thread (GQ hd <= 1024)
            float oacc[NV] = {0.f, 0.f};
            const int nc2 = d2 / 8;
            for (int e0 = 0; e0 < total; e0 += cap_e) {
                const int ne = min(cap_e, total - e0);
                if (warp == 0) {
                    fence_proxy_async();                                 // rows written by P1's ordinary stores, read by the copy engine
                    if (lane == 0) mb_expect_tx(gbar, static_cast<uint32_t>(ne) * tokb);
                    for (int e = lane; e < ne; e += 32) {
                        int h, k;
                        entry(e0 + e, h, k);
                        const int t = sel_tok[h * p.ntok_cap + k];
                        bulk_g2s(gat_s + e * tokb, ly.k2c + krow0 + static_cast<int64_t>(t) * d2, d2 * 2, gbar);
                        bulk_g2s(gat_s + e * tokb + d2 * 2, ly.vc + vrow0 + static_cast<int64_t>(t) * hd, hd * 2, gbar);
                    }
                }
                mb_wait(gbar, gpar, fail, c.limit);                      // a wait that runs out raises the flag checked below
                gpar ^= 1u;
                if (e0 == 0) p.trace.mark(5);
                // gate and weight of every entry: half a warp per entry
                for (int eb = warp * 2; eb < ne; eb += 2 * kConsWarps) {      // both halves of a warp make the same trips
                    const int e = eb + half;
                    const bool valid = e < ne;
                    int h = 0, k = 0;
                    if (valid) entry(e0 + e, h, k);
                    float a = 0.f;
                    if (valid && hl < nc2) {
                        float wf[8];
                        unpack8(reinterpret_cast<const uint4*>(gat + static_cast<size_t>(e) * tokb)[hl], wf);
                        const float* q2 = qs + h * hd + r + hl * 8;
#pragma unroll
                        for (int x = 0; x < 8; ++x) a = fmaf(wf[x], q2[x], a);
                    }
#pragma unroll
                    for (int o = 8; o > 0; o >>= 1) a += __shfl_xor_sync(kFull, a, o, 16);
                    if (valid && hl == 0) {
                        const float pe = expf(sel_a[h * p.ntok_cap + k]);
                        atomicAdd(&sh.l_s[h], pe);
                        sel_a[h * p.ntok_cap + k] = pe * softplus(a);
                    }
                }
                if (cons_any(*fail != 0)) break;
                // value reduction: a thread per output column of a head, over that head's entries of this round
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    const int i = tid + v * kCons;
                    if (i < GQ * hd) {
                        const int h = i / hd, col = i - h * hd;
                        int first = 0;
#pragma unroll
                        for (int hh = 0; hh < GQ; ++hh)
                            if (hh < h) first += nsel[hh];
                        const int a0 = max(first, e0), a1 = min(first + nsel[h], e0 + ne);
                        float acc = oacc[v];
                        for (int e = a0; e < a1; ++e) {
                            const __nv_bfloat16* vrow = reinterpret_cast<const __nv_bfloat16*>(gat + static_cast<size_t>(e - e0) * tokb + d2 * 2);
                            acc = fmaf(sel_a[h * p.ntok_cap + (e - first)], __bfloat162float(vrow[col]), acc);
                        }
                        oacc[v] = acc;
                    }
                }
                cons_sync();                                             // the gather area is free again
            }
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int i = tid + v * kCons;
                if (i < GQ * hd && total > 0) atomicAdd(p.obuf + static_cast<int64_t>(bp.g) * GQ * hd + i, oacc[v]);
            }
            if (tid < GQ && sh.sel_n[tid] > 0) atomicAdd(p.lsum + bp.g * GQ + tid, sh.l_s[tid]);
        }
        c.mk = 48;
        p.trace.mark(6);
        if (!grid_barrier(c, p.hdr, gen0 + (++nbar), G, cta)) break;
        p.trace.mark(7);

        // =========================== P4: h += Wo . (o / sum of weights) ===========================================
        for (int i = tid; i < nqo / 4; i += kCons) {
            float4 v = __ldcg(reinterpret_cast<const float4*>(p.obuf) + i);
            const float ls = __ldcg(p.lsum + (4 * i) / hd);
            const float inv = ls > 0.f ? 1.f / ls : 0.f;                 // an empty selection attends to nothing
            v.x *= inv; v.y *= inv; v.z *= inv; v.w *= inv;
            reinterpret_cast<float4*>(xs)[i] = v;
        }
        if (cta == 0 && tid < p.n_q * kAttnWays) {                       // every block has read the attention's cells: idle state again
            SumCell* cc = p.attn_cells + tid;
            cc->s1 = 0.0; cc->s2 = 0.0; cc->count = 0u; cc->pad[0] = 0u;
        }
        c.mk = 16;
        dbg_mark(c.tr, 16 + 6);
        float hrow = 0.f;                                                // the block's rows of h, requested before the tiles are consumed
        if (tid < bp.norow) hrow = __ldcg(p.h + bp.o0 + tid);
        cons_sync();
        stage_split3(c, xs, nqo, xsp, p.xstride);
        cons_sync();
        if (!group_phase(c, pos, bp.norow, nqo, xsp, p.xstride, sh.outp)) *fail = 1;
        if (cons_any(*fail != 0)) break;
        if (tid < bp.norow) {                                            // at most 256 rows per block
            const int nkc = kConsWarps, np = group_parts(bp.norow, nqo);
            float v = 0.f;
            for (int s = 0; s < np; ++s) v += sh.outp[tid * nkc + s];
            p.h[bp.o0 + tid] = hrow + v;
        }
        p.trace.mark(8);
        if (!grid_barrier(c, p.hdr, gen0 + (++nbar), G, cta)) break;
        p.trace.mark(9);

        // =========================== P5: x = RMSNorm(h), predictor scores of the block's neurons ==================
        const unsigned epoch = epoch0 + static_cast<unsigned>(l);
        SumCell* fways = &p.hdr->ffn_cells[epoch & 3u][0][0][0];
        if (cta == 0) {      // clear the cells the layer after next will use (last used two layers ago)
            SumCell* cc = &p.hdr->ffn_cells[(epoch + 2u) & 3u][0][0][0];
            for (int i = tid; i < 4 * 16 * kCellWays; i += kCons) { cc[i].s1 = 0.0; cc[i].s2 = 0.0; cc[i].count = 0u; }
        }
        c.mk = 32;
        stage_rmsnorm(c, p, ly.norm2, xs, sh.scratch, xsp, p.xstride);
        if (!group_phase(c, pos, bp.nfrow, p.r_ff, xsp, p.xstride, sh.outp)) *fail = 1;
        if (cons_any(*fail != 0)) break;
        float* s_loc = sh.s_loc;                                         // the block's scores (at most 256 neurons)
        if (tid < bp.nfrow) {
            const int nkc = kConsWarps, np = group_parts(bp.nfrow, p.r_ff);
            float v = 0.f;
            for (int s = 0; s < np; ++s) v += sh.outp[tid * nkc + s];
            s_loc[tid] = v;
        }
        if (tid == 0) sh.nact = 0;
        cons_sync();
        p.trace.mark(10);
        // ---- X5: score sums to the cells, theta (Eq. 10/11) once every block has arrived
        if (warp == 0) {
            double s1 = 0.0, s2 = 0.0;
            for (int j = lane; j < bp.nfrow; j += 32) {
                const double v = static_cast<double>(s_loc[j]);
                s1 += v;
                s2 = fma(v, v, s2);
            }
            s1 = warp_sum_f64(s1);
            s2 = warp_sum_f64(s2);
            if (lane == 0) cells_add(fways, cta, s1, s2);
            double sa, sb;
            const bool ok = cells_wait(fways, static_cast<unsigned>(G + p.extra_arrivals), sa, sb, p.hdr);
            if (lane == 0) {
                if (!ok) *fail = 1;
                float th = -INFINITY;
                if (!p.identity_ff) {
                    const double mean = sa * p.inv_n;
                    const float var = static_cast<float>((sb - sa * mean) * p.inv_nm1);
                    th = static_cast<float>(mean) + sqrtf(fmaxf(var, 0.f)) * static_cast<float>(p.z_ff);
                }
                sh.theta_ff = th;
            }
        }
        if (cons_any(*fail != 0)) break;
        p.trace.mark(11);

        // =========================== P6: active neurons, gather, h += V u ==========================================
        {
            const float theta = sh.theta_ff;
            if (tid < bp.nfrow) {
                const float s = s_loc[tid];
                if (s > theta) {
                    const int e = atomicAdd(&sh.nact, 1);
                    sh.flist_j[e] = tid;
                    sh.flist_a[e] = p.identity_ff ? s : s - theta;       // GELU sees the shifted survivor (Eq. 10)
                }
            }
            cons_sync();
            const int nact = sh.nact;
            const int dff2 = p.d - p.r_ff, rowb = (dff2 + p.d) * 2, cap_e = p.gather_bytes / rowb;
            const int ncd = p.d / 8, nck = dff2 / 8;
            float yacc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) yacc[e] = 0.f;
            for (int e0 = 0; e0 < nact; e0 += cap_e) {
                const int ne = min(cap_e, nact - e0);
                if (warp == 0) {
                    if (lane == 0) mb_expect_tx(gbar, static_cast<uint32_t>(ne) * rowb);
                    for (int e = lane; e < ne; e += 32) {
                        const int64_t row = bp.f0 + sh.flist_j[e0 + e];
                        bulk_g2s(gat_s + e * rowb, ly.K2t + row * dff2, dff2 * 2, gbar);
                        bulk_g2s(gat_s + e * rowb + dff2 * 2, ly.Vt + row * p.d, p.d * 2, gbar);
                    }
                }
                mb_wait(gbar, gpar, fail, c.limit);
                gpar ^= 1u;
                if (e0 == 0) p.trace.mark(12);
                // t = K2[:, i] . x[r:], u = GELU(s - theta) t: a warp per active neuron
                for (int e = warp; e < ne; e += kConsWarps) {
                    const uint4* krow = reinterpret_cast<const uint4*>(gat + static_cast<size_t>(e) * rowb);
                    float t = 0.f;
                    for (int ch = lane; ch < nck; ch += 32) {
                        float wf[8];
                        unpack8(krow[ch], wf);
                        const float4 xa = reinterpret_cast<const float4*>(xs + p.r_ff)[2 * ch], xb = reinterpret_cast<const float4*>(xs + p.r_ff)[2 * ch + 1];
                        t = dot8(wf, xa, xb, t);
                    }
                    t = warp_sum(t);
                    if (lane == 0) {
                        const float a = sh.flist_a[e0 + e];
                        sh.uval[e] = (p.erf_form ? gelu_erf(a) : gelu_tanh(a)) * t;
                    }
                }
                if (cons_any(*fail != 0)) break;
                // y: a thread per 8 columns, over this round's rows of V
                if (tid < ncd) {
                    for (int e = 0; e < ne; ++e) {
                        float wf[8];
                        unpack8(reinterpret_cast<const uint4*>(gat + static_cast<size_t>(e) * rowb + dff2 * 2)[tid], wf);
                        const float u = sh.uval[e];
#pragma unroll
                        for (int x = 0; x < 8; ++x) yacc[x] = fmaf(u, wf[x], yacc[x]);
                    }
                }
                cons_sync();                                             // the gather area and uval are free again
            }
            if (nact > 0 && tid < ncd) {
                red_add_v4(p.h + tid * 8, yacc[0], yacc[1], yacc[2], yacc[3]);
                red_add_v4(p.h + tid * 8 + 4, yacc[4], yacc[5], yacc[6], yacc[7]);
            }
        }
        p.trace.mark(13);
        if (!grid_barrier(c, p.hdr, gen0 + (++nbar), G, cta)) break;
        p.trace.mark(14);
    }
    // the launch's last barrier has passed (or the launch has failed): publish where the counters stand
    if (cta == 0 && tid == 0 && *fail == 0) {
        p.hdr->epoch = epoch0 + static_cast<unsigned>(p.n_layers);
        p.hdr->l1_gen = gen0 + nbar;
    }
    if (tid == 0 && *fail != 0) atomicCAS(&p.hdr->status, SPARK_OK, SPARK_ERR_TIMEOUT);
}

template <int GQ>
int launch_gq(spark_ctx* ctx, L1Params& p, size_t dyn_smem, cudaStream_t stream) {
    static bool configured[64] = {};
    auto kern = layer1_kernel<GQ>;
    if (ctx->device >= 0 && ctx->device < 64 && !configured[ctx->device]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(ctx->max_smem_optin - sizeof(L1Shared) - 512)) != cudaSuccess)
            return SPARK_ERR_CUDA;
        configured[ctx->device] = true;
    }
    void* args[] = {&p};
    return launch_kernel(ctx, reinterpret_cast<const void*>(kern), static_cast<unsigned>(ctx->num_sms), kThreadsL1, dyn_smem, stream, true, args) == cudaSuccess
               ? SPARK_OK : SPARK_ERR_CUDA;
}

}  // namespace

namespace spark {

// One token through n_layers layers (equal configurations but for the attention window) in one launch of the fused kernel.
// SPARK_ERR_WORKSPACE = shape, flags or sizes not served: the caller takes the kernel-per-step path.
int layer1_launch(spark_ctx* ctx, const spark_layer_weights* w, const spark_layer_cfg* cfg, const spark_kv_cache* cache, int n_layers,
                  const int32_t* ctx_len, float* h, float* scratch, cudaStream_t stream) {
    const spark_layer_cfg& c0 = cfg[0];
    if (n_layers < 1 || n_layers > kMaxLayers) return SPARK_ERR_WORKSPACE;
    if ((c0.flags & ~SPARK_GELU_ERF) != 0) return SPARK_ERR_WORKSPACE;
    const int64_t d = c0.d, hd = c0.hd, r = c0.r_attn, d2 = hd - r, nqo = c0.n_q * hd, G = ctx->num_sms;
    if (c0.n_kv < 1 || c0.n_q % c0.n_kv != 0) return SPARK_ERR_WORKSPACE;
    const int64_t gq = c0.n_q / c0.n_kv;
    if (gq != 1 && gq != 2 && gq != 4) return SPARK_ERR_WORKSPACE;
    if ((d & 7) || (c0.r_ff & 7) || ((d - c0.r_ff) & 7) || (hd & 7) || (r & 7) || (d2 & 7) || r > 128 || d2 > 128 || r < 8 || d2 < 8 ||
        c0.r_ff <= 0 || c0.r_ff >= d || hd > 256)
        return SPARK_ERR_WORKSPACE;
    if (d > 4096 || gq * hd > 2 * kCons || c0.n_q * kAttnWays > kCons || G < c0.n_kv || G > 1024) return SPARK_ERR_WORKSPACE;
    if ((c0.d_ff + G - 1) / G > 256 || c0.d_ff < 2 || c0.k_ff <= 0 || c0.k_attn <= 0 || c0.cap < 1 || c0.cap >= (1LL << 31) / 256)
        return SPARK_ERR_WORKSPACE;
    if (ctx->scratch_bytes < static_cast<size_t>(c0.n_q) * kAttnWays * sizeof(SumCell)) return SPARK_ERR_WORKSPACE;
    L1Params p;
    int64_t span = 0;
    for (int l = 0; l < n_layers; ++l) {
        const spark_layer_cfg& c = cfg[l];
        if (c.d != d || c.d_ff != c0.d_ff || c.r_ff != c0.r_ff || c.k_ff != c0.k_ff || c.n_q != c0.n_q || c.n_kv != c0.n_kv || c.hd != hd ||
            c.r_attn != r || c.k_attn != c0.k_attn || c.cap != c0.cap || c.rms_eps != c0.rms_eps || c.rope_base != c0.rope_base ||
            c.flags != c0.flags || c.window < 0)
            return SPARK_ERR_WORKSPACE;
        const void* ptrs[] = {w[l].norm1, w[l].norm2, w[l].Wqkv, w[l].Wo, w[l].K1t, w[l].K2t, w[l].Vt, cache[l].k1c, cache[l].k2c, cache[l].vc};
        for (const void* q : ptrs)
            if (q == nullptr || !aligned16(q)) return SPARK_ERR_WORKSPACE;
        L1Layer& ly = p.layer[l];
        ly.norm1 = w[l].norm1; ly.norm2 = w[l].norm2;
        ly.Wqkv = static_cast<const __nv_bfloat16*>(w[l].Wqkv); ly.Wo = static_cast<const __nv_bfloat16*>(w[l].Wo);
        ly.K1t = static_cast<const __nv_bfloat16*>(w[l].K1t); ly.K2t = static_cast<const __nv_bfloat16*>(w[l].K2t);
        ly.Vt = static_cast<const __nv_bfloat16*>(w[l].Vt);
        ly.k1c = static_cast<__nv_bfloat16*>(cache[l].k1c); ly.k2c = static_cast<__nv_bfloat16*>(cache[l].k2c);
        ly.vc = static_cast<__nv_bfloat16*>(cache[l].vc);
        ly.window = static_cast<int>(c.window > 0x7fffffff ? 0x7fffffff : c.window);
        ly.pad = 0;
        const int64_t sp = (c.window > 0 && c.window < c.cap) ? c.window : c.cap;
        span = sp > span ? sp : span;
    }
    // the tensor-core tiles take 32 columns at a time
    if ((d & 31) || (nqo & 31) || (c0.r_ff & 31) || (r & 31)) return SPARK_ERR_WORKSPACE;
    // a slot holds the longest row (plus its padding), and at least sixteen tokens of the predictor slice
    const int64_t slot = static_cast<int64_t>(round_up(static_cast<size_t>(std::max<int64_t>(std::max<int64_t>(std::max<int64_t>(d, nqo), c0.r_ff) * 2 + 64, 16 * r * 2)), 128));
    p.slot_bytes = static_cast<int>(slot);
    p.tps = static_cast<int>(slot / (r * 2)) & ~15;
    const int64_t P = (c0.n_q + 2 * c0.n_kv) * hd / 2;
    if (2 * (P / G + 1) > 128 || d / G + 1 > 128 || c0.d_ff / G + 1 > 128) return SPARK_ERR_WORKSPACE;      // 16 partial sums per row in outp
    if (d / G + 1 > kCons) return SPARK_ERR_WORKSPACE;
    p.xstride = static_cast<int>(round_up(static_cast<size_t>(std::max<int64_t>(d, nqo)) * 2, 128) + 64);
    p.qstride = static_cast<int>(round_up(static_cast<size_t>(r) * 2, 128) + 64);
    const size_t xsp_b = round_up(std::max<size_t>(3 * static_cast<size_t>(p.xstride), 3 * static_cast<size_t>(gq) * p.qstride), 128);
    const int64_t nb_min = G / c0.n_kv;
    p.ntok_cap = static_cast<int>((span + nb_min - 1) / nb_min + 2);
    const size_t act_b = round_up(static_cast<size_t>(std::max<int64_t>(std::max<int64_t>(d, nqo), gq * hd)) * 4, 128);
    const size_t sc_b = round_up(static_cast<size_t>(gq) * p.ntok_cap * 12, 128);
    const size_t limit = static_cast<size_t>(ctx->max_smem_optin) - sizeof(L1Shared) - 1024;
    const size_t rowb = static_cast<size_t>(2 * d - c0.r_ff) * 2, tokb = static_cast<size_t>(d2 + hd) * 2;
    size_t gather_b = 0;
    int n_slots = 0;
    // a row group (16 rows) must be resident at once: the ring needs the slots of the longest-rowed phase's group, and a few more
    auto slots_per_group = [&](int64_t K) {
        int64_t rps = 1;
        while (rps < 16 && 2 * rps * (K * 2 + 64) <= slot) rps *= 2;
        return static_cast<int>(16 / rps);
    };
    const int need_slots = std::max(10, std::max(std::max(slots_per_group(d), slots_per_group(nqo)), slots_per_group(c0.r_ff)) + 2);
    for (int ge : {8, 6, 4, 2}) {        // active neurons fetched per round: as many as leaves the ring what it needs
        gather_b = round_up(std::max(ge * rowb, 16 * tokb), 128);
        n_slots = 0;
        if (act_b + sc_b + xsp_b + gather_b >= limit) continue;
        n_slots = static_cast<int>((limit - act_b - sc_b - xsp_b - gather_b) / slot);
        if (n_slots >= need_slots) break;
    }
    if (n_slots < need_slots) return SPARK_ERR_WORKSPACE;
    if (n_slots > 64) n_slots = 64;
    p.n_slots = n_slots;
    {
        // slots in flight at most; measured: any limit below the ring's size only slows the stream down (2 slots: 71 us per
        // layer, 8: 51, 20: 50.7 at the 2B shape), so the default is the whole ring; SPARK_L1_INFLIGHT overrides it for experiments
        int q = n_slots - 1;
        if (const char* e = std::getenv("SPARK_L1_INFLIGHT")) q = std::atoi(e);
        if (q < 2) q = 2;
        if (q > n_slots - 1) q = n_slots - 1;
        p.max_inflight = q;
    }
    p.off_ring = 0;
    p.off_gather = static_cast<int>(static_cast<size_t>(n_slots) * slot);
    p.off_act = p.off_gather + static_cast<int>(gather_b);
    p.off_sc = p.off_act + static_cast<int>(act_b);
    p.off_xsp = p.off_sc + static_cast<int>(sc_b);
    p.off_misc = p.off_xsp + static_cast<int>(xsp_b);
    p.gather_bytes = static_cast<int>(gather_b);
    const size_t dyn = static_cast<size_t>(p.off_misc);
    p.h = h; p.qbuf = scratch; p.obuf = scratch + nqo; p.lsum = scratch + 2 * nqo; p.ctx_len = ctx_len;
    p.n_layers = n_layers;
    p.d = static_cast<int>(d); p.d_ff = static_cast<int>(c0.d_ff); p.r_ff = static_cast<int>(c0.r_ff);
    p.n_q = static_cast<int>(c0.n_q); p.n_kv = static_cast<int>(c0.n_kv); p.hd = static_cast<int>(hd); p.r_attn = static_cast<int>(r);
    p.k_attn = static_cast<int>(c0.k_attn > 0x7fffffff ? 0x7fffffff : c0.k_attn); p.gq = static_cast<int>(gq);
    p.cap = c0.cap; p.eps = c0.rms_eps; p.q_scale = 1.0f / std::sqrt(static_cast<float>(hd));
    p.erf_form = (c0.flags & SPARK_GELU_ERF) ? 1 : 0;
    p.extra_arrivals = ctx->debug_extra_arrivals;
    p.identity_ff = c0.k_ff >= c0.d_ff ? 1 : 0;
    p.z_ff = p.identity_ff ? 0.0 : spark_normal_upper_quantile(static_cast<double>(c0.k_ff) / static_cast<double>(c0.d_ff));
    p.inv_n = 1.0 / static_cast<double>(c0.d_ff); p.inv_nm1 = 1.0 / static_cast<double>(c0.d_ff - 1);
    p.rpc = static_cast<int>((c0.d_ff + G - 1) / G);
    p.attn_cells = reinterpret_cast<SumCell*>(ctx->scratch);
    p.hdr = ctx->hdr;
    p.trace = PhaseTrace{ctx->trace, ctx->trace_cap};
    for (int part = 0; part < 2; ++part) {
        const int64_t m = part == 0 ? r : d2;
        for (int64_t i = 0; i < 64; ++i)
            p.inv_freq[part][i] = i < m / 2 ? std::pow(static_cast<double>(c0.rope_base), -2.0 * static_cast<double>(i) / static_cast<double>(m)) : 0.0;
    }
    if (gq == 1) return launch_gq<1>(ctx, p, dyn, stream);
    if (gq == 2) return launch_gq<2>(ctx, p, dyn, stream);
    return launch_gq<4>(ctx, p, dyn, stream);
}

}  // namespace spark
