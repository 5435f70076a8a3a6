/*
 * exfold.h - C ABI of the B200 (sm_100a) folded Mixture-of-Experts layer (ExFold).
 *
 * One MoE layer with N routed SwiGLU experts (+ an optional always-on shared expert):
 *     E_e(x) = W_down^(e) ( silu(W_gate^(e) x) * (W_up^(e) x) )                 (Eq. 1)
 *     S_K(x) = Top-K router logits, a_e = softmax restricted to S_K              (Eq. 2)
 *     MoE(x) = sum_{e in S_K} a_e E_e(x)  (+ shared expert, weight 1)            (Eq. 3)
 * Folding executes only a retained subset of the routed experts and moves the gate
 * weight of every excluded expert s onto its minimum-loss retained expert t, scaled by
 * the calibrated pairwise scalar S[s][t] (Eq. 4, 12). Two modes:
 *     prefill: per token, keep the K' routes with the largest a_e h_e   (Eq. 10, 13)
 *     decode : per batch, keep a pool of at most M experts ranked by
 *              sum_i a_{i,e} h_e, remap every other route in place       (Eq. 11, 14)
 *
 * Conventions for every call
 *   - All tensors are dense, row-major. Weights are stored like nn.Linear (out x in):
 *     W_gate, W_up [N+n_shared][I][d], W_down [N+n_shared][d][I]; the shared expert, if
 *     any, is expert index N. x, W_*, y have the layer dtype; router logits and all
 *     tables are fp32; indices are int32.
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the
 *     caller. The library allocates no device memory: all scratch lives in the caller's
 *     workspace `ws` (exfold_workspace_bytes; 256-byte aligned). Calls that share a
 *     workspace must be ordered on one stream.
 *   - What the library keeps between calls, and nothing else: (a) per host thread and device,
 *     created on first use and freed by exfold_thread_release: one extra CUDA stream (highest priority) with
 *     three events (large prefill calls run two kernel chains side by side on it) and two copy streams
 *     with ten events (chunked host-buffer prefill). Calls issued by one host thread on
 *     different caller streams share them, so the parts that use them run one after the other;
 *     results do not depend on it. (b) per process: the launch counter, the optional
 *     per-kernel timing events (exfold_profile_*, off by default, not thread-safe) and the
 *     built-in scratch array of exfold_moe_decode_noalloc. No environment variable is read.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL = the
 *     default stream) and return without synchronising, except exfold_device_status.
 *   - Return value: EXFOLD_OK (0), a negative error (nothing was launched), or a positive
 *     warning. Arguments are validated on the host before anything is launched.
 *   - Every wait inside a kernel is bounded; a kernel that gives up records
 *     EXFOLD_ERR_DEVICE_TIMEOUT in the workspace's status word and returns.
 *   - bf16 layers need d and I to be multiples of 64; N <= 256, K <= 32.
 */
#ifndef EXFOLD_H_
#define EXFOLD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { EXFOLD_F32 = 0, EXFOLD_BF16 = 1 } exfold_dtype;

enum {
    EXFOLD_OK = 0,
    EXFOLD_ERR_INVALID_ARG = -1,
    EXFOLD_ERR_UNSUPPORTED = -2,
    EXFOLD_ERR_WORKSPACE_TOO_SMALL = -3,
    EXFOLD_ERR_CUDA = -4,
    EXFOLD_ERR_DEVICE_TIMEOUT = -5,
    EXFOLD_ERR_EXCEEDS_STATIC_SCRATCH = -6,
    EXFOLD_WARN_UNOBSERVED_EXPERT = 1
};

/* Shape of the layer (Eq. 1-3). */
typedef struct {
    int32_t n_experts; /* N routed experts, 2..256 */
    int32_t n_shared;  /* 0 or 1 shared expert, stored as expert N */
    int32_t hidden;    /* d */
    int32_t inter;     /* I */
    int32_t top_k;     /* K of the original router, 1..32, <= N */
    int32_t dtype;     /* exfold_dtype of x, W_*, y */
} exfold_layer;

/*
 * Calibration tables of one layer (device, caller-owned, fp32).
 *   S [N][N]  scalar projector, row = source expert, column = target expert (Eq. 8)
 *   L [N][N]  projection loss (Eq. 9)
 *   h [N]     output-norm estimate of each expert; lnh[e] = (float)log((double)h[e])
 *   n_obs [N][N] number of calibration tokens seen per pair (written by calibrate; may be NULL)
 */
typedef struct {
    float *S;
    float *L;
    float *h;
    float *lnh;
    int32_t *n_obs;
} exfold_tables;

/* Options of exfold_calibrate ("Calibration protocol": lambda = 1e-3, clip [-4,4]). */
typedef struct {
    float lambda;  /* ridge term of Eq. 8 */
    float clip_lo; /* scalars are clipped to [clip_lo, clip_hi] before the loss is taken */
    float clip_hi;
    float eps;     /* added to the denominator of the normalised loss (appendix form of Eq. 9) */
    int32_t mode;  /* 0: pairs observed when both experts are in a token's Top-K; 1: every expert sees every token */
} exfold_calib_opts;

/* Optional routing metadata written by exfold_moe_prefill (device pointers; any may be NULL). */
typedef struct {
    int32_t *ids;      /* [T][K']   retained experts, descending a_e h_e            */
    float *w;          /* [T][K']   folded weights (Eq. 13)                         */
    int32_t *omit_src; /* [T][K-K'] omitted experts, descending a_e h_e             */
    int32_t *omit_tgt; /* [T][K-K'] their minimum-loss targets (Eq. 12)             */
    int32_t *perm;     /* [T*K']    route indices i*K'+j sorted by (expert, i, j)   */
    int32_t *offsets;  /* [N+1]     first sorted position of each expert            */
} exfold_prefill_meta;

/* Optional routing metadata written by exfold_moe_decode (device pointers; any may be NULL). */
typedef struct {
    int32_t *pool_ids;   /* [M]  pool experts, descending score, -1 padded (Eq. 11)        */
    int32_t *pool_size;  /* [1]  min(M, size of the batch's expert union)                  */
    uint32_t *pool_mask; /* [ceil(N/32)] bit e set when expert e is in the pool            */
    int32_t *ids;        /* [B][K] remapped expert of every routed slot (Eq. 14)           */
    float *w;            /* [B][K] remapped weight of every routed slot                    */
    int32_t *target;     /* [N]  target[s]: s itself if in the pool, else its min-loss pool expert */
    float *scale;        /* [N]  1 or S[s][target[s]]                                      */
} exfold_decode_meta;

/*
 * Bytes of workspace needed by any call on `layer` with up to max_tokens tokens
 * (T, B or calibration tokens) and up to routes_per_token executed routes per token
 * (K' for prefill, K for decode and calibration). Returns 0 for an invalid layer.
 */
size_t exfold_workspace_bytes(const exfold_layer *layer, int64_t max_tokens, int32_t routes_per_token);

/*
 * Offline calibration of the pairwise scalar projector (Eq. 6-9 and the appendix's
 * shared-scalar and normalised-loss forms). Runs the routed experts on m calibration
 * tokens x_cal [m][d] with logits_cal [m][N], accumulates per ordered pair (s,t) the
 * sums of w<v,u>, w|v|^2, w|u|^2 with w = |u| (u = E_s(x), v = E_t(x)) in double, and
 * writes S, L, h, lnh (and n_obs if non-NULL) into `out`. S_ee = 1, L_ee = 0; a pair
 * never observed gets S = 0, L = 1e30; an expert never observed gets the mean h of the
 * others and the call returns EXFOLD_WARN_UNOBSERVED_EXPERT after synchronising the
 * stream (this call is off the serving path and does synchronise).
 * Expert outputs: fp32 layers use the fp32 SIMT expert kernel; bf16 layers run the same grouped
 * tensor-core GEMMs as prefill (the SwiGLU activation is rounded to bf16 between the two GEMMs, the
 * outputs stay fp32), so the tables of a bf16 layer carry that rounding (~1e-3 relative per token).
 * Workspace: exfold_workspace_bytes(layer, m, K) for mode 0, (layer, m, N) for mode 1 (every expert
 * runs on every token; m*N <= 2^30). bf16 layers need x_cal and the weights 16-byte aligned.
 */
int exfold_calibrate(const exfold_layer *layer, const void *x_cal, const float *logits_cal, int64_t m,
                     const void *w_gate, const void *w_up, const void *w_down,
                     const exfold_calib_opts *opts, exfold_tables *out, void *ws, size_t ws_bytes,
                     void *cuda_stream);

/*
 * Calibration of several layers of one model in one call ("Calibration protocol": every MoE layer gets its own
 * tables from the same calibration prompts). All jobs share the layer description (shape, dtype) and the options;
 * each job names its own calibration inputs, expert weights and output tables (device pointers, as for
 * exfold_calibrate). The jobs are enqueued back to back on the stream and the call synchronises once, at the end;
 * tables are bit-identical to those of one exfold_calibrate call per job. `unobserved` (host, [n_jobs], may be NULL)
 * receives each job's number of never-observed experts; the call returns EXFOLD_WARN_UNOBSERVED_EXPERT if any is
 * positive. Workspace: exfold_workspace_bytes for the largest job (see exfold_calibrate). n_jobs <= EXFOLD_MAX_CALIB_JOBS.
 */
#define EXFOLD_MAX_CALIB_JOBS 256
typedef struct {
    const void *x_cal;        /* [m][d] */
    const float *logits_cal;  /* [m][N] (mode 0) or NULL (mode 1) */
    int64_t m;
    const void *w_gate, *w_up, *w_down;
    exfold_tables *out;
} exfold_calib_job;
int exfold_calibrate_layers(const exfold_layer *layer, const exfold_calib_job *jobs, int32_t n_jobs,
                            const exfold_calib_opts *opts, int32_t *unobserved, void *ws, size_t ws_bytes,
                            void *cuda_stream);

/*
 * Prefill: token-level Top-K folding (Eq. 10, 12, 13, then Eq. 1 and 4 over the retained
 * routes only). x [T][d], logits [T][N] -> y [T][d]. k_pre = K' in [1, K]; k_pre = K is the
 * unfolded layer. Each token executes exactly K' routed experts (+ the shared expert).
 * Ranking uses key = logit + lnh[e] (one fp32 add; same order as a_e h_e).
 * bf16 layers: the two grouped GEMMs of a call of >= 24 row tiles (128 sorted rows each) run the experts' row tiles
 * two at a time on pairs of CTAs and, beside them, the experts' odd last tiles on the one-CTA-per-tile kernel;
 * smaller calls use the latter alone. The results are bit-identical either way. The odd-tile kernels run on a
 * second stream (highest priority) that the library creates once per host thread; with a shared expert, the gate/up
 * projection of its whole row-tile pairs also runs there, beside the kernel that gathers the routed rows (its inputs
 * are x and the weights only). That work is ordered after the caller's earlier work and before its later work by
 * events on the caller's stream (also under stream capture). exfold_fold_opts.gemm_path overrides the choice of
 * kernels (tests and measurements).
 */
int exfold_moe_prefill(const exfold_layer *layer, const void *x, const float *logits, int64_t T,
                       const void *w_gate, const void *w_up, const void *w_down,
                       const exfold_tables *tables, int32_t k_pre, void *y,
                       const exfold_prefill_meta *meta, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Prefill with the safeguards the paper applies on other model families (cross-model results and
 * the DeepSeek-V4 appendix). opts == NULL, or all fields at their "off" values, is exfold_moe_prefill.
 *   loss_threshold    directed pairs with calibrated loss above it are excluded from target
 *                     assignment (the paper uses 0.99); an omitted route with no admissible target is
 *                     dropped and reported with omit_tgt = -1. Off: +infinity.
 *   rescale           != 0: after folding, a token's retained weights are scaled so that they sum
 *                     to the original sum of its K routed weights (skipped when the folded sum is
 *                     not positive).
 *   confidence_split  != 0: with c = clip(1 - L[s][t], 0, 1) for the minimum-loss target t, the part
 *                     w_s c S[s][t] is folded onto t and w_s (1 - c) is spread over the retained
 *                     routes in proportion to their original router weights.
 *   gemm_path         0: the library chooses the tensor-core kernels (above); 1: one-CTA kernel only;
 *                     2: CTA pairs wherever a group has a pair of row tiles. Same results bit for bit.
 */
typedef struct {
    float loss_threshold;
    int32_t rescale;
    int32_t confidence_split;
    int32_t gemm_path;
} exfold_fold_opts;

int exfold_moe_prefill_ex(const exfold_layer *layer, const void *x, const float *logits, int64_t T,
                          const void *w_gate, const void *w_up, const void *w_down,
                          const exfold_tables *tables, int32_t k_pre, const exfold_fold_opts *opts, void *y,
                          const exfold_prefill_meta *meta, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Decode: batch-level expert-pool folding (Eq. 11, 12, 14, then Eq. 1 and 4 over the pool
 * only). x [B][d], logits [B][N] -> y [B][d], B <= 256. pool_m = M in [1, N]; the pool is
 * the whole expert union of the batch when that has at most M experts, so pool_m = N is the
 * unfolded layer. Scores are sums of the double-precision routed weights (exact in 2^-53 fixed
 * point, so independent of any order). Only the pool's (and the shared expert's) weights are
 * read, each byte once. bf16 layers: four kernels chained by programmatic dependent launch
 * (per-token Top-K; gate/up projection with the batch-level routing in its prologue, x read in
 * place; grouped down projection over one row per distinct (token, pool expert); per-token sum
 * of those rows in slot order). No atomics are used: the same inputs give the same bits.
 */
int exfold_moe_decode(const exfold_layer *layer, const void *x, const float *logits, int64_t B,
                      const void *w_gate, const void *w_up, const void *w_down,
                      const exfold_tables *tables, int32_t pool_m, void *y,
                      const exfold_decode_meta *meta, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Static decode pool (appendix, "static implementation"): the pool is formed once from the
 * calibration-time norms, pool = TopK_e(h_e, M) over all routed experts (ties -> lower id), and
 * one target and one scalar are cached for every possible source expert, which removes the
 * per-step batch reduction of Eq. 11. exfold_static_pool_build fills the caller's device arrays;
 * exfold_moe_decode_static then runs a decode step whose routing is the per-route remap of the
 * appendix listing (out_id = target[id], out_w = w * scale[id], [B][K] layout kept) followed by
 * the expert FFN over the pool experts that received rows. Metadata, workspace, stream and
 * error conventions are those of exfold_moe_decode; pool experts without a route this step are
 * not read.
 */
typedef struct {
    int32_t *pool_ids; /* [pool_m] pool experts, descending h           */
    int32_t *target;   /* [N]  s itself if in the pool, else its minimum-loss pool expert */
    float *scale;      /* [N]  1 or S[s][target[s]]                     */
    int32_t pool_m;    /* M in [1, N]                                   */
} exfold_static_pool;

int exfold_static_pool_build(const exfold_layer *layer, const exfold_tables *tables, int32_t pool_m,
                             exfold_static_pool *out, void *cuda_stream);
int exfold_moe_decode_static(const exfold_layer *layer, const void *x, const float *logits, int64_t B,
                             const void *w_gate, const void *w_up, const void *w_down,
                             const exfold_static_pool *pool, void *y, const exfold_decode_meta *meta,
                             void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Router scores that Eq. 2 ranks: logits[i][e] = <w_router[e], x[i]> for T tokens, fp32 out.
 * x [T][d] and w_router [N][d] are in the layer dtype (device), logits [T][N] fp32 (device, 16-byte aligned).
 * bf16 layers with more than 128 tokens run on the tensor cores (bf16 products, fp32 accumulation, order
 * unspecified); fp32 layers and batches of at most 128 tokens on a dot-product kernel (fp32 accumulation in a
 * fixed order). The result is the `logits` argument of the prefill / decode calls; a Top-K
 * decision on scores closer than the accumulation error (~1e-6 relative) is not reproducible bit for bit
 * against another summation order. Workspace: exfold_workspace_bytes(layer, T, 1). Enqueues on the stream
 * and returns without synchronising. The shared expert and the tables play no part.
 */
int exfold_router_logits(const exfold_layer *layer, const void *x, const void *w_router, int64_t T, float *logits,
                         void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * A whole layer from hidden states: the router scores of Eq. 2 (r = W_r x) followed by the folded layer, for
 * callers that hold the router matrix rather than logits (a stack of layers, each reading the previous
 * layer's output, captured in one CUDA graph). w_router [N][d] in the layer dtype; `logits` [T][N] fp32 is a
 * caller-owned device buffer that receives the scores (16-byte aligned; the layer needs them as scratch and
 * the caller may want them). Everything else as in exfold_moe_prefill / exfold_moe_decode, including the
 * workspace size. The scores are those of exfold_router_logits, bit for bit: decode batches (and prefill calls of
 * at most 128 tokens) take the fixed-order dot-product kernel, which joins the decode call's chain of programmatic
 * dependent launches; longer prefill calls compute the scores with a separate tensor-core launch (a Top-K taken
 * inside a tensor-core epilogue could not be reproduced bit for bit by another summation order, so the two
 * steps stay separate kernels there).
 */
int exfold_moe_prefill_layer(const exfold_layer *layer, const void *x, const void *w_router, int64_t T,
                             const void *w_gate, const void *w_up, const void *w_down,
                             const exfold_tables *tables, int32_t k_pre, float *logits, void *y,
                             const exfold_prefill_meta *meta, void *ws, size_t ws_bytes, void *cuda_stream);
int exfold_moe_decode_layer(const exfold_layer *layer, const void *x, const void *w_router, int64_t B,
                            const void *w_gate, const void *w_up, const void *w_down,
                            const exfold_tables *tables, int32_t pool_m, float *logits, void *y,
                            const exfold_decode_meta *meta, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The same two calls for activations that live in HOST memory (pinned for real overlap):
 * x_host, logits_host and y_host are host pointers; the call stages them through the
 * workspace with asynchronous copies on the stream (x and logits in before the layer, y out
 * after it). Weights, tables, metadata and workspace stay device pointers. The workspace
 * must be exfold_workspace_bytes(...) + exfold_host_staging_bytes(...) large.
 * A prefill call of 4096 tokens or more that asks for no metadata is run as up to four chunks of whole
 * 128-row tiles: the next chunk is copied in and the previous one copied out on two helper streams
 * (created once per host thread and device), while the caller's stream computes; the call still completes in
 * the caller's stream order and the result is the same bit for bit (tokens do not interact).
 */
size_t exfold_host_staging_bytes(const exfold_layer *layer, int64_t max_tokens);
int exfold_moe_prefill_host(const exfold_layer *layer, const void *x_host, const float *logits_host,
                            int64_t T, const void *w_gate, const void *w_up, const void *w_down,
                            const exfold_tables *tables, int32_t k_pre, void *y_host,
                            const exfold_prefill_meta *meta, void *ws, size_t ws_bytes, void *cuda_stream);
int exfold_moe_decode_host(const exfold_layer *layer, const void *x_host, const float *logits_host,
                           int64_t B, const void *w_gate, const void *w_up, const void *w_down,
                           const exfold_tables *tables, int32_t pool_m, void *y_host,
                           const exfold_decode_meta *meta, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Decode for callers that cannot allocate device memory. (The paper has no counterpart: this is
 * a packaging variant of exfold_moe_decode, same arguments minus the workspace, same results.)
 *
 * Who needs it: a host that must not call cudaMalloc while it runs - an engine whose memory pool
 * is fixed at start-up, a plugin living in a process whose allocator it does not own, a caller
 * that has already entered a phase where allocations are refused. Such a caller has nowhere to
 * get the workspace from, so here the scratch is a fixed array of EXFOLD_STATIC_SCRATCH_BYTES
 * inside the library image. Every GPU that loads the library holds those bytes until the process
 * ends. The caller still passes inputs, outputs and optional metadata buffers as device pointers.
 *
 * Limits and rules:
 *   - the call needs exfold_workspace_bytes(layer, B, layer->top_k) bytes of scratch; if that
 *     exceeds EXFOLD_STATIC_SCRATCH_BYTES it returns EXFOLD_ERR_EXCEEDS_STATIC_SCRATCH and launches
 *     nothing (e.g. Qwen3- and Mixtral-shaped layers fit up to B = 64, the GLM-4.5-Air-shaped
 *     one up to B = 32);
 *   - it calls no cudaMalloc, cudaFree or any allocating library routine;
 *   - the first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture;
 *   - all calls on a device share the one array, which keeps what the previous call left in it;
 *     the call itself clears what must start at zero, but two calls that overlap on the GPU
 *     (different streams, no ordering between them) race on it: keep them on one stream or order
 *     them with events;
 *   - the status record of these calls sits at the start of that array: read it with
 *     exfold_device_status_noalloc (same meaning and behaviour as exfold_device_status: it
 *     synchronises the stream, reports a bounded wait that ran out, and clears the record). Without
 *     that check a timed-out call goes unnoticed, because the next call clears the record first.
 * exfold_static_scratch_address writes the array's device address on the current device to
 * *address (host pointer), for diagnostics and memory checkers; the array is never to be freed.
 */
#define EXFOLD_STATIC_SCRATCH_BYTES (8u << 20)
int exfold_moe_decode_noalloc(const exfold_layer *layer, const void *x, const float *logits, int64_t B,
                              const void *w_gate, const void *w_up, const void *w_down,
                              const exfold_tables *tables, int32_t pool_m, void *y,
                              const exfold_decode_meta *meta, void *cuda_stream);
int exfold_device_status_noalloc(void *cuda_stream);
int exfold_static_scratch_address(void **address);

/*
 * Synchronises the stream and decodes the status word the kernels keep at the start of the
 * workspace: EXFOLD_OK, EXFOLD_ERR_DEVICE_TIMEOUT (a bounded wait ran out), or
 * EXFOLD_ERR_CUDA. Clears the word. The only synchronising call on the serving path.
 */
int exfold_device_status(void *ws, void *cuda_stream);

/*
 * Destroys the CUDA streams and events the library created for the calling host thread on the current
 * device (see the conventions above); they are created again by the next call that needs them. The
 * caller makes sure none of its calls is still running on them (synchronise first).
 */
int exfold_thread_release(void);

/* Human-readable name of a status code (static storage). */
const char *exfold_status_string(int status);

/* Number of kernels of this library launched by this process so far (for launch accounting). */
int64_t exfold_launch_count(void);

/*
 * Per-kernel timing for benchmarks (host-side state; not thread-safe; off by default).
 * exfold_profile_enable(1) creates one CUDA event pair per kernel slot; while enabled, every
 * launch of the serving calls is bracketed by event records on the call's stream.
 * exfold_profile_read synchronises on the recorded events of the LAST call and writes, for
 * each slot < n_slots, the elapsed milliseconds (or -1 if that kernel did not run in the last
 * call). Slots: 0 prefill route/fold, 1 prefill scan, 2 prefill scatter+gather, 3 grouped GEMM-1
 * (gate/up + SwiGLU), 4 grouped GEMM-2 (down + scatter-combine), 5 fp32->bf16 conversion,
 * 6 decode pool/remap, 7 decode row gather, 8 decode GEMM-1 (gate/up stream), 9 decode GEMM-2 (down stream),
 * 10 SIMT expert FFN, 11 SIMT combine, 12 / 13 the CTA-pair pass of GEMM-1 / GEMM-2 alone (slots 3 and 4 cover a
 * whole GEMM: the pair pass, when it runs, and the one-CTA pass), 14 decode expert FFN of bf16 layers (one kernel:
 * pool / remap prologue + gate, up and down weight stream; slot 6 is then the per-token Top-K kernel and slots
 * 7-9 stay empty). Returns EXFOLD_OK or EXFOLD_ERR_CUDA.
 */
#define EXFOLD_PROFILE_SLOTS 15
int exfold_profile_enable(int enable);
int exfold_profile_read(float *ms, int32_t n_slots);

#ifdef __cplusplus
}
#endif
#endif /* EXFOLD_H_ */
