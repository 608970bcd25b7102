/*
 * spark.h -- C ABI of the B200 (sm_100a) Spark Transformer decode library.
 *
 * The library implements the per-token, activation-sparse decode step of the
 * Spark Transformer: statistical top-k (Section 3, Eq. 9-11), Spark FFN
 * (Section 2.1, Eq. 2) and Spark attention (Section 2.2, Eq. 7), plus the dense
 * glue a decoder layer needs around them (Section 4, "Implementation details").
 *
 * Conventions that hold for every entry point
 * -------------------------------------------
 * - All tensor arguments are DEVICE pointers on the context's device unless a
 *   comment says "host".  The caller owns every buffer, including the
 *   workspace handed to spark_create; the library never allocates or frees
 *   device memory and keeps no pointer beyond a call except that workspace.
 * - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   Calls only enqueue work; outputs are valid once the stream has been
 *   synchronised.  Calls that share one context must be issued on one stream
 *   (they share the workspace); use one context per concurrent stream.
 * - Return value: 0 (SPARK_OK) or one of the SPARK_ERR_* codes below.  Argument
 *   errors are detected on the host before anything is enqueued.  Conditions
 *   only the device can see (a bounded wait that ran out, ...) are recorded in a
 *   device status word read by spark_device_status.  Nothing aborts or traps.
 * - Activations (x, q, y, o, h, theta) are fp32.  Weights and KV caches are
 *   fp32 (SPARK_F32) or bf16 (SPARK_BF16), accumulated in fp32.  Every row of a
 *   weight / cache tensor must start on a 16-byte boundary: base pointers
 *   16-byte aligned and row lengths a multiple of 8 elements (bf16) or 4 (fp32),
 *   otherwise SPARK_ERR_UNSUPPORTED.
 * - FFN weights are stored neuron-major, i.e. as the transposes of the paper's
 *   matrices: K1t[d_ff][r] = K1^T, K2t[d_ff][d-r] = K2^T, Vt[d_ff][d] = V^T,
 *   row-major, so that one neuron's weights are one contiguous run ("we store
 *   the matrix in row format", Appendix B).
 * - KV caches are token-major with each key split into its predictor slice and
 *   the rest (Section 2.2: K1 = first r rows of K, K2 = the others):
 *   k1c[B][n_kv][cap][r], k2c[B][n_kv][cap][hd-r], vc[B][n_kv][cap][hd].
 * - Degenerate k (the paper leaves them open): k >= n keeps every entry
 *   unshifted (theta reported as -inf); k <= 0 is SPARK_ERR_INVALID_ARG.
 *   Selection is the strict comparison x_i > theta; the number selected is
 *   whatever exceeds theta (about k, not capped at k).
 */
#ifndef SPARK_H_
#define SPARK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------- */
enum {
    SPARK_OK = 0,
    SPARK_ERR_INVALID_ARG = 1, /* null pointer, k <= 0, r outside (0, d), n_q % n_kv != 0, ...      */
    SPARK_ERR_UNSUPPORTED = 2, /* misaligned pointer / row length, unknown dtype, size over a limit */
    SPARK_ERR_WORKSPACE = 3,   /* the context's workspace is too small for this call                */
    SPARK_ERR_CUDA = 4,        /* a CUDA runtime call or a launch failed                            */
    SPARK_ERR_TIMEOUT = 5,     /* device: a bounded wait between thread blocks ran out              */
    SPARK_ERR_OVERFLOW = 6,    /* device: an index list did not fit its capacity (truncated)        */
    SPARK_ERR_NONFINITE = 7    /* device: the score statistics of a call made with SPARK_CHECK_FINITE
                                  were not finite (a NaN or infinity in its inputs or weights)     */
};

/* ---- dtypes and flags ----------------------------------------------------- */
enum { SPARK_F32 = 0, SPARK_BF16 = 1, SPARK_FP8_E4M3 = 2 /* spark_ffn_decode_fp8 only */ };

enum {
    SPARK_FILL_ZERO = 0,   /* Eq. 10: entries not above theta become 0                       */
    SPARK_FILL_NEGINF = 1  /* the Top_k^(-inf) variant of Section 3 used by Spark attention   */
};

enum {
    SPARK_GELU_TANH = 0,     /* tanh form of GELU (the one Gemma uses); the default            */
    SPARK_GELU_ERF = 1,      /* exact form x * Phi(x)                                          */
    SPARK_DENSE_LOADS = 2,   /* comparator: same result, but every row of K2/V (or of the cache)
                                is read and multiplied by its (possibly zero) activation       */
    SPARK_SHARED_CACHE = 4,  /* attention and layer: the B tokens are consecutive tokens of ONE
                                sequence (a chunk of its prompt) and share one cache
                                [n_kv][cap][.]; token b is the sequence's token number ctx_len[b]
                                (1-based) and sees rows [0, ctx_len[b]), so with ctx_len[b] =
                                L0 + b + 1 the chunk is causal; caches lose their [B] dimension  */
    SPARK_FFN_FP8 = 16,      /* layer: K1t, K2t, Vt are FP8 E4M3 with the per-neuron scales K1s, K2s, Vs of
                                spark_layer_weights (as in spark_ffn_decode_fp8; one to four tokens)    */
    SPARK_K1C_FP8 = 32,      /* layer: the predictor slice of the cache is FP8 E4M3 with one fp32 scale per
                                cached row in spark_kv_cache.k1s (as in spark_attn_decode_fp8k); the
                                appended row is stored as e4m3(k / s) with s = max|k| / 448              */
    SPARK_CHECK_FINITE = 8   /* debugging aid: a threshold whose score sums are not finite (a NaN or an
                                infinity reached the predictor) records SPARK_ERR_NONFINITE in the
                                device status.  Honoured by the one-token FFN kernel and by the
                                per-query attention kernel, also inside spark_layer_decode; the
                                other kernels ignore it.  The paper leaves non-finite inputs
                                undefined; outputs are then undefined here too                     */
};

typedef struct spark_ctx spark_ctx;

/* ---- context -------------------------------------------------------------- */

/* Bytes of workspace a context needs so that every call with batch <= max_batch,
 * d_ff <= max_dff, cache capacity <= max_cap, n_q query heads of head_dim hd and model
 * width <= max_d fits.  Pure host arithmetic. */
size_t spark_workspace_bytes(int64_t max_batch, int64_t max_dff, int64_t max_cap, int64_t n_q,
                             int64_t hd, int64_t max_d);

/* Create a context on `device` around a caller-owned device workspace (256-byte aligned).
 * Zeroes the workspace (its idle state is all zero) and waits for the device, so that the first
 * call may go to any stream; queries the SM count.
 * *out is a host object released by spark_destroy (which leaves the workspace alone). */
int spark_create(spark_ctx** out, int device, void* workspace, size_t workspace_bytes);
int spark_destroy(spark_ctx* ctx);

/* Synchronise `stream`, copy the device status word to *host_out (host pointer), clear it, and
 * if it was not SPARK_OK also reset the workspace to its idle (zero) state (synchronously: the
 * context is usable again when the call returns).  Returns SPARK_OK when the read itself worked
 * (the device status is in *host_out). */
int spark_device_status(spark_ctx* ctx, void* stream, int* host_out);

/* Static string for a status code (host pointer, never freed). */
const char* spark_status_string(int status);

/* Number of thread blocks the context launches for its cooperative kernels (= SM count). */
int spark_grid_size(const spark_ctx* ctx);

/* Phase tracing (profiling aid; the paper has no counterpart).  With a non-NULL device buffer of
 * `capacity` uint64 values, the cooperative kernels (FFN, attention) make thread 0 of block b
 * store its SM's cycle counter at each phase boundary into trace[b * 16 + phase] (phase < 15) and
 * the GPU-wide nanosecond timer at phase 0 into trace[b * 16 + 15].  `capacity` must cover
 * 16 entries per block.  NULL switches tracing off (the default). */
int spark_set_phase_trace(spark_ctx* ctx, uint64_t* trace, int64_t capacity);

/* Launch overlap (scheduling aid; the paper has no counterpart).  With on != 0 every kernel of
 * this context is launched with the programmatic stream-serialization attribute: it may start
 * while the kernel before it in the stream still runs, requests its first weights, and only then
 * waits for that kernel to complete.  The caller promises that (1) the work placed in the stream
 * directly before a call does not write the WEIGHT buffers of that call (everything else is read
 * after the wait), and (2) the GPU runs no other kernels meanwhile: the inter-block exchanges rely
 * on all blocks being resident, which the cooperative launch used otherwise (on == 0, the default)
 * guarantees and this mode only obtains from an otherwise idle GPU; a block that waits in vain
 * gives up after its limit and the device status becomes SPARK_ERR_TIMEOUT.  Host-only setting. */
int spark_set_launch_overlap(spark_ctx* ctx, int on);

/* Bound of the waits between thread blocks (failure detection; the paper has no counterpart).  The
 * kernels that exchange score sums between blocks (FFN, attention, the fused one-token layer) poll
 * until every block has arrived; a block that has waited `cycles` SM cycles gives up, records
 * SPARK_ERR_TIMEOUT in the device status and returns, the kernel ends by itself and the outputs of
 * that call are incomplete.  spark_device_status then reports the code and resets the workspace,
 * after which the context is usable again.  cycles == 0 restores the default (about two seconds).
 * Synchronises `stream` and the device: call it between steps, not during a stream capture.  The
 * tensor-core chunk kernels and the top-k row kernel keep their own fixed bounds. */
int spark_set_wait_limit(spark_ctx* ctx, void* stream, int64_t cycles);

/* Test hook for that path (host-only setting; 0 = off, the default): the one-token FFN kernel waits
 * for `extra` more arrivals than its grid has blocks, so its wait runs out exactly as it would if a
 * block never became resident.  Nothing faults: the kernel returns after the wait limit. */
int spark_debug_expect_arrivals(spark_ctx* ctx, int extra);

/* Gaussian upper quantile used for the threshold: z with P(N(0,1) > z) = p, i.e. Q(1 - p) of
 * Eq. 11.  Host function (no device work); exported so that it can be checked on its own.
 * Returns NaN for p outside (0, 1). */
double spark_normal_upper_quantile(double p);

/* ---- statistical top-k (Section 3, Eq. 9-11) -------------------------------
 * For each of `rows` rows x[row*ld .. row*ld + n): theta = mean + std * Q(1 - k/n) with the
 * Bessel-corrected std, active set A = { i : x_i > theta }, values x_i - theta.
 *   theta  [rows]               fp32, nullable
 *   count  [rows]               int32, nullable: |A| (the full count even when idx_cap is smaller)
 *   idx    [rows][idx_cap]      int32, nullable: A in ascending order, first min(|A|, idx_cap)
 *   val    [rows][idx_cap]      fp32,  nullable: x_i - theta for those entries
 *   y_dense[rows][ld]           fp32,  nullable: the dense result of Eq. 10 (fill = 0) or of the
 *                               -inf variant (fill = SPARK_FILL_NEGINF)
 * If |A| > idx_cap the lists are truncated and SPARK_ERR_OVERFLOW is recorded in the device
 * status.  x needs 16-byte aligned rows (x aligned, ld % 4 == 0).  n >= 2 unless k >= n. */
int spark_stat_topk(spark_ctx* ctx, const float* x, int64_t rows, int64_t n, int64_t ld, int64_t k,
                    int fill, float* theta, int32_t* count, int32_t* idx, float* val,
                    int64_t idx_cap, float* y_dense, void* stream);

/* ---- statistical top-k of a row sharded over several devices (Appendix, "global statistical top-k") ----
 * Each device holds a contiguous part of every row.  The global form needs one small exchange: every
 * device takes the moments of its part (spark_stat_moments), the parts' moments are gathered (the
 * caller's collective; 24 bytes per row and device), merged into theta of the whole row
 * (spark_stat_merge; the same on every device), and each device selects from its part with that
 * threshold (spark_stat_select).  The result equals spark_stat_topk on the concatenated row.  The local
 * form of the same appendix needs no exchange: spark_stat_topk on the part with k / m.
 *
 * spark_stat_moments: moments[row] = (n, mean, sum of squared deviations from the mean) of
 *   x[row*ld .. row*ld + n) as three doubles, [rows][3].  n >= 2.
 * spark_stat_merge: parts [m][rows][3] (device memory, part after part as gathered); theta[rows] =
 *   mean + std * Q(1 - k / n_total) of the merged moments, Bessel-corrected (Eq. 11), -inf for
 *   k >= n_total; merged [rows][3] nullable.  The parts' counts must add up to n_total.
 * spark_stat_select: like spark_stat_topk with the thresholds given (theta_in [rows], device): count,
 *   idx (indices within the part), val, y_dense as there; survivors are shifted by theta_in, except that
 *   theta_in = -inf (what spark_stat_merge gives for k >= n_total) keeps every entry unshifted. */
int spark_stat_moments(spark_ctx* ctx, const float* x, int64_t rows, int64_t n, int64_t ld, double* moments,
                       void* stream);
int spark_stat_merge(spark_ctx* ctx, const double* parts, int64_t m, int64_t rows, int64_t k, int64_t n_total,
                     float* theta, double* merged, void* stream);
int spark_stat_select(spark_ctx* ctx, const float* x, int64_t rows, int64_t n, int64_t ld, const float* theta_in,
                      int fill, int32_t* count, int32_t* idx, float* val, int64_t idx_cap, float* y_dense,
                      void* stream);

/* ---- Spark FFN (Section 2.1, Eq. 2) ------------------------------------------
 * y_b = V . ( GELU(StatTop_k(K1^T x_b[:r])) * (K2^T x_b[r:]) ) for each of the B tokens, every
 * token with its own threshold and active set; weight rows are loaded once per call for the
 * union of the tokens' active sets (Appendix B).  Chunks of 5 to 64 tokens with bf16 weights, where
 * that union covers most rows, read every row instead and run the three products as GEMMs on the
 * tensor cores (same results; SPARK_DENSE_LOADS changes nothing there); this needs d % 256 == 0,
 * r % 64 == 0, d_ff % 128 == 0 and a workspace sized by spark_workspace_bytes for max_batch >= 5,
 * max_dff >= d_ff and max_d >= d -- any other call with 5..64 tokens takes the union-gather kernels.
 *   x [B][d] fp32;  K1t[d_ff][r], K2t[d_ff][d-r], Vt[d_ff][d] of dtype wdtype
 *   flags: SPARK_GELU_TANH or SPARK_GELU_ERF, optionally | SPARK_DENSE_LOADS
 *   y     [B][d]     fp32 (overwritten)
 *   theta [B]        fp32,  nullable
 *   count [B]        int32, nullable
 *   idx   [B][d_ff]  int32, nullable (needs count): active neurons of token b in unspecified order;
 *                    entries past count[b] are not written
 * Limits: 1 <= B <= 64, 0 < r < d, r % 8 == 0, d % 8 == 0, d_ff >= 2. */
int spark_ffn_decode(spark_ctx* ctx, const float* x, int64_t B, const void* K1t, const void* K2t,
                     const void* Vt, int wdtype, int64_t d, int64_t d_ff, int64_t r, int64_t k,
                     int flags, float* y, float* theta, int32_t* count, int32_t* idx, void* stream);

/* The same FFN with the three matrices stored as FP8 E4M3 (1-4-3 bits, bias 7, largest finite 448) and one
 * fp32 scale per neuron: row i of K1t / K2t / Vt stands for K1s[i] / K2s[i] / Vs[i] times its stored values
 * (quantised weights are named in the paper's closing section as the natural companion of activation sparsity;
 * the format and the per-neuron scales are this library's choice).  K1t [d_ff][r], K2t [d_ff][d-r], Vt [d_ff][d]
 * uint8 device buffers, 16-byte aligned, r and d multiples of 8; K1s, K2s, Vs [d_ff] fp32.  One to four tokens
 * (B <= 4, d <= 4096): SPARK_ERR_UNSUPPORTED otherwise.  Everything else as spark_ffn_decode. */
int spark_ffn_decode_fp8(spark_ctx* ctx, const float* x, int64_t B, const void* K1t, const float* K1s, const void* K2t,
                         const float* K2s, const void* Vt, const float* Vs, int64_t d, int64_t d_ff, int64_t r, int64_t k,
                         int flags, float* y, float* theta, int32_t* count, int32_t* idx, void* stream);

/* ---- Spark FFN without any allocation (the paper has no counterpart) ----------------------
 * Some callers may not call cudaMalloc at all: code that runs where device memory has been
 * handed out in full up front (an inference server's arena, a plugin inside another runtime), or
 * that must not touch the allocator because a stream capture or a latency-critical section is
 * under way elsewhere in the process.  They cannot give spark_create a workspace.  This entry point
 * computes what spark_ffn_decode computes, within the library's stated tolerances (for 5 to 16
 * tokens it takes the union-gather kernels, where spark_ffn_decode with a workspace may take the
 * tensor-core chunk kernels), with the small amount of inter-block state the kernels need (a status
 * word, a launch counter, the cells the blocks add their score sums into) kept in a fixed array
 * inside the library's device image: about 140 KB on every GPU that loads the library, held until
 * the process exits.  Inputs and outputs are still the caller's.
 *   - Limit: B <= SPARK_NOALLOC_MAX_TOKENS; a larger B returns SPARK_ERR_UNSUPPORTED.  All other
 *     limits and argument checks are those of spark_ffn_decode.  count / idx are not offered.
 *   - The device is the current one.  The first call on a device looks up the array's device
 *     address (the array is zero, its idle state, from the moment the library is loaded; nothing
 *     is cleared and nothing is enqueued besides the kernel, so the first call may go to any
 *     stream); make that first call before any stream capture begins.  No call allocates or frees
 *     device memory.
 *   - All calls on a device share the array, and it keeps what the last call left (the kernels
 *     themselves clear the cells a later call will use).  Two calls whose kernels overlap on the
 *     GPU -- different streams, or one process-wide array used from two threads -- race on it:
 *     issue them on one stream, or otherwise order them.  spark_ffn_decode with its own context
 *     has no such restriction across contexts.
 *   - spark_noalloc_status plays the part of spark_device_status: it synchronises `stream`, copies
 *     the array's status word to *host_out (host pointer) and, if that is not SPARK_OK (a bounded
 *     wait ran out: y of that call is incomplete), puts the array back into its idle state so that
 *     later calls work again.  It allocates nothing either. */
#define SPARK_NOALLOC_MAX_TOKENS 16
int spark_ffn_decode_noalloc(const float* x, int64_t B, const void* K1t, const void* K2t, const void* Vt,
                             int wdtype, int64_t d, int64_t d_ff, int64_t r, int64_t k, int flags,
                             float* y, float* theta, void* stream);
int spark_noalloc_status(void* stream, int* host_out);

/* ---- Spark attention (Section 2.2, Eq. 7) ------------------------------------
 * For sequence b and query head h (KV head g = h / (n_q / n_kv)), over the tokens t of the window
 * [max(0, n_b - window), n_b), n_b = ctx_len[b] (window == 0: all n_b tokens):
 *   s_t = k1c[b][g][t] . q[b][h][:r];  A = StatTop_{k_attn}^{(-inf)}(s);
 *   o[b][h] = sum_{t in A} softmax_A(s)_t * softplus(k2c[b][g][t] . q[b][h][r:]) * vc[b][g][t]
 * q is used as given (apply the position encoding and any 1/sqrt(hd) scale before the call).
 * A window of at most k_attn tokens is attended to densely; an empty A gives o = 0.
 *   q [B][n_q][hd] fp32;  ctx_len [B] int32 DEVICE array, 1 <= ctx_len[b] <= cap
 *   flags: 0 or SPARK_DENSE_LOADS
 *   o     [B][n_q][hd]       fp32 (overwritten)
 *   theta [B][n_q]           fp32,  nullable
 *   count [B][n_q]           int32, nullable
 *   idx   [B][n_q][idx_cap]  int32, nullable (needs count): selected token positions, unspecified order,
 *                            truncated at idx_cap (SPARK_ERR_OVERFLOW recorded)
 * ctx_len values outside [1, cap] are clamped into it.
 * Limits: hd <= 256, r and hd - r multiples of 8 and at most 128, n_q / n_kv in {1, 2, 4, 8},
 * B * n_kv <= 2048. */
int spark_attn_decode(spark_ctx* ctx, const float* q, const void* k1c, const void* k2c,
                      const void* vc, int kvdtype, int64_t B, int64_t n_q, int64_t n_kv, int64_t hd,
                      int64_t r, int64_t cap, const int32_t* ctx_len, int64_t window, int64_t k_attn,
                      int flags, float* o, float* theta, int32_t* count, int32_t* idx,
                      int64_t idx_cap, void* stream);

/* The same attention with the predictor slice of the cache stored as FP8 E4M3: k1c [B][n_kv][cap][r] uint8 and
 * k1s [B][n_kv][cap] fp32, cached row t of a head standing for k1s[t] times its stored values; k2c and vc stay
 * bf16.  The predictor slice is all that a long context streams, so this halves the bytes read there (the paper's
 * closing section names quantisation as the companion of activation sparsity; format and per-row scales are this
 * library's choice).  Everything else as spark_attn_decode. */
int spark_attn_decode_fp8k(spark_ctx* ctx, const float* q, const void* k1c, const float* k1s, const void* k2c,
                           const void* vc, int64_t B, int64_t n_q, int64_t n_kv, int64_t hd, int64_t r, int64_t cap,
                           const int32_t* ctx_len, int64_t window, int64_t k_attn, int flags, float* o, float* theta,
                           int32_t* count, int32_t* idx, int64_t idx_cap, void* stream);

/* The same with the WHOLE cache in FP8 E4M3: k1c, k2c, vc uint8 with the row scales k1s, k2s, vs [B][n_kv][cap] fp32 each (a cached
 * row of a tensor stands for its scale times its stored values): the rows gathered for the selected tokens are halved as well.
 * Not with SPARK_SHARED_CACHE.  Everything else as spark_attn_decode. */
int spark_attn_decode_fp8kv(spark_ctx* ctx, const float* q, const void* k1c, const float* k1s, const void* k2c, const float* k2s,
                            const void* vc, const float* vs, int64_t B, int64_t n_q, int64_t n_kv, int64_t hd, int64_t r, int64_t cap,
                            const int32_t* ctx_len, int64_t window, int64_t k_attn, int flags, float* o, float* theta,
                            int32_t* count, int32_t* idx, int64_t idx_cap, void* stream);

/* ---- dense GEMV (the projections the method leaves dense: Table "FLOPs per token") ----
 * y[b][n_out] = Wt[n_out][n_in] . x[b][n_in] (+ y_add[b][n_out] if y_add != NULL).
 * Wt of dtype wdtype, output-major; n_in % 8 == 0; 1 <= B <= 64.  y_add may equal y. */
int spark_dense_gemv(spark_ctx* ctx, const float* x, int64_t B, const void* Wt, int wdtype,
                     int64_t n_in, int64_t n_out, const float* y_add, float* y, void* stream);

/* ---- one decoder layer (Section 4) ---------------------------------------------
 * Pre-norm block around the two operators, for one new token per sequence:
 *   a = RMSNorm(h; norm1);  [q|k|v] = Wqkv a;  rotary position encoding applied separately to
 *   q[:r], q[r:], k[:r], k[r:] at position ctx_len[b]-1;  q *= 1/sqrt(hd);
 *   k, v written to row ctx_len[b]-1 of the caches;  h += Wo . SparkAttention;  h += SparkFFN(RMSNorm(h; norm2)).
 * With SPARK_SHARED_CACHE in cfg->flags the B tokens are consecutive tokens of one sequence (a chunk of
 * its prompt): the caches are [n_kv][cap][.], token b is appended at row ctx_len[b]-1 and attends to rows
 * [0, ctx_len[b]); ctx_len[b] = L0 + b + 1 gives what decoding the chunk token by token gives (n_kv a
 * power of two).  1 <= B <= 64 either way.
 * All pointers inside the structs are device pointers; the structs themselves are host objects. */
typedef struct spark_layer_weights {
    const float* norm1;   /* [d]                          */
    const float* norm2;   /* [d]                          */
    const void* Wqkv;     /* [(n_q + 2 n_kv) hd][d] bf16  */
    const void* Wo;       /* [d][n_q hd]            bf16  */
    const void* K1t;      /* [d_ff][r_ff]           bf16  */
    const void* K2t;      /* [d_ff][d - r_ff]       bf16  */
    const void* Vt;       /* [d_ff][d]              bf16  */
    const float* K1s;     /* [d_ff] per-neuron scales of K1t, K2t, Vt: only with SPARK_FFN_FP8 (the three    */
    const float* K2s;     /*        matrices are then uint8 E4M3 codes), NULL otherwise                   */
    const float* Vs;
} spark_layer_weights;

typedef struct spark_layer_cfg {
    int64_t d, d_ff, r_ff, k_ff;
    int64_t n_q, n_kv, hd, r_attn, k_attn;
    int64_t window;       /* 0 = global attention, else the local window length          */
    int64_t cap;          /* cache capacity in tokens                                     */
    float rms_eps;        /* e.g. 1e-6                                                    */
    float rope_base;      /* e.g. 10000                                                   */
    int flags;            /* SPARK_GELU_* | SPARK_DENSE_LOADS (applies to FFN and attention) */
} spark_layer_cfg;

typedef struct spark_kv_cache {
    void* k1c;            /* [B][n_kv][cap][r_attn]      bf16, row ctx_len[b]-1 is written */
    void* k2c;            /* [B][n_kv][cap][hd-r_attn]   bf16                              */
    void* vc;             /* [B][n_kv][cap][hd]          bf16                              */
    float* k1s;           /* [B][n_kv][cap] row scales of k1c: only with SPARK_K1C_FP8 (k1c is then uint8
                             E4M3 codes; entry ctx_len[b]-1 is written), NULL otherwise             */
} spark_kv_cache;

/* scratch: B * ((n_q + 2 n_kv) hd + 2 n_q hd + d + 2 + n_q) fp32 values, 16-byte aligned, caller-owned, contents
 * undefined after the call.  h [B][d] fp32 is updated in place.  1 <= B <= 64.
 * Four kernels are enqueued for B <= 4: QKV projection with position encoding and cache
 * append, attention, output projection, FFN.  For B >= 5 the position encoding and the append follow the projection as a
 * kernel of their own, and where the shapes allow (see spark_ffn_decode; projections: inputs % 64 == 0, outputs % 128 == 0)
 * the projections and the FFN run as tensor-core GEMMs of two and four kernels each, and the attention of a chunk
 * (SPARK_SHARED_CACHE, B >= 16) as three: up to thirteen kernels per call. */
int spark_layer_decode(spark_ctx* ctx, const spark_layer_weights* w, const spark_layer_cfg* cfg,
                       const spark_kv_cache* cache, const int32_t* ctx_len, float* h, int64_t B,
                       float* scratch, void* stream);

/* The same for a stack of n_layers layers applied one after the other to the same tokens (Section 4: the decoder is a stack
 * of such layers; local and global attention layers alternate, so the layers' configurations may differ in `window`):
 * w, cfg and cache are HOST arrays of n_layers structs, h and scratch as for one layer.  With one token and equal
 * configurations but for the window, the fused kernel takes up to 64 layers per launch, so that its weight stream runs on
 * across the layer boundaries; every other call is the loop over spark_layer_decode. */
int spark_stack_decode(spark_ctx* ctx, const spark_layer_weights* w, const spark_layer_cfg* cfg,
                       const spark_kv_cache* cache, int64_t n_layers, const int32_t* ctx_len, float* h, int64_t B,
                       float* scratch, void* stream);

/* A prompt through a stack of layers, chunk by chunk (Section 4.3 reports prefill in chunks of 64 tokens; here 1 <= chunk <= 64):
 * h [n_tokens][d] fp32 holds the prompt's embeddings and is replaced in place by the stack's outputs; the tokens are appended to
 * every layer's cache at rows start .. start + n_tokens - 1 (start = tokens already cached), every token attending causally to
 * the rows before it and to itself, later chunks seeing earlier ones through the caches -- what decoding the prompt token by token
 * gives.  w, cfg, cache: HOST arrays of n_layers structs; every cfg must carry SPARK_SHARED_CACHE (caches [n_kv][cap][.]) and
 * cap >= start + n_tokens.  len_buf: caller-owned DEVICE buffer of `chunk` int32 (the library writes each chunk's lengths there);
 * scratch as for spark_layer_decode with B = chunk.  The call only enqueues: one tiny kernel plus n_layers layer calls per chunk. */
int spark_prefill(spark_ctx* ctx, const spark_layer_weights* w, const spark_layer_cfg* cfg, const spark_kv_cache* cache,
                  int64_t n_layers, float* h, int64_t n_tokens, int64_t start, int64_t chunk, int32_t* len_buf, float* scratch,
                  void* stream);

/* The same with several chunks in flight (scheduling only; the paper has no counterpart): chunk c runs on stream c % n_inflight
 * with context c % n_inflight, and layer l of a chunk starts once layer l of the chunk before it has finished, which is all it
 * needs (the caches of layer l up to its own rows).  The kernels of a chunk layer are short and latency-bound, so the other
 * chunks fill the gaps each one leaves.  ctxs, scratches, streams: HOST arrays of n_inflight (2 to 8) distinct contexts on one
 * device (kernels that run at the same time must not share a workspace), scratch areas like spark_prefill's, and streams;
 * len_buf: n_inflight * chunk int32.  The call forks from streams[0] and joins back into it: work queued there before the call
 * is seen by all, work queued after it sees all of the prefill.  Creates and destroys n_inflight * (n_layers + 1) + 1 events
 * (no device memory).  Results equal spark_prefill's up to the order of floating-point reductions. */
int spark_prefill_pipelined(spark_ctx* const* ctxs, float* const* scratches, void* const* streams, int64_t n_inflight,
                            const spark_layer_weights* w, const spark_layer_cfg* cfg, const spark_kv_cache* cache,
                            int64_t n_layers, float* h, int64_t n_tokens, int64_t start, int64_t chunk, int32_t* len_buf);

/* Scheduling option (the paper has no counterpart; default off): in layer calls of one to four tokens every kernel asks L2,
 * with a few bulk-prefetch instructions per block, for the weights the NEXT kernel will stream (QKV kernel: Wo; attention:
 * K1t; FFN, inside spark_stack_decode: the next layer's Wqkv).  Measured on B200 it LOSES (2B layer 30.8 -> 32.0 us, 9B
 * 57.8 -> 61-63 us): the prefetch traffic delays the few loads the step's critical path waits for by more than the L2-resident
 * stream saves.  Kept as a switch so that the comparison can be repeated.  Host-only setting. */
int spark_set_l2_prefetch(spark_ctx* ctx, int on);

/* Scheduling option (the paper has no counterpart): on != 0 makes one-token layer calls take the fused persistent kernel
 * where it serves the shape; the default (0) is the kernel-per-step path, which measures faster on B200 (the fused kernel's
 * critical path is bound by serial bookkeeping and grid-wide barriers).  Host-only setting. */
int spark_set_fused_layer(spark_ctx* ctx, int on);

/* Prompt chunks (SPARK_SHARED_CACHE with 16 to 64 tokens; Section 4.3 evaluates prompts in chunks): how the attention forms its
 * output once the predictor scores of the chunk are known.  Either every (token, head) gathers the k2c / vc rows of its own
 * selection, or -- when a KV head serves 32 or more (token, head) pairs of the chunk and the head sizes fit (hd 128 or 256,
 * hd - r_attn 64 or 128) -- every cached row is read once per block and the selection of Eq. 7 becomes a mask on dense weights,
 * both products on the tensor cores.  Same results up to rounding order.  mode 0: always the gather; 1 (default): the dense
 * form where it measured faster on B200 (up to about 4096 visible rows: the window of a local layer, else the length
 * spark_prefill knows, else the cache capacity); 2: the dense form wherever it serves the shape.  Host-only setting;
 * SPARK_ERR_INVALID_ARG for another mode. */
int spark_set_chunk_dense(spark_ctx* ctx, int mode);

#ifdef __cplusplus
}
#endif
#endif /* SPARK_H_ */
