// Shared declarations of the folded-MoE CUDA library (sm_100a only).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/exfold.h"

namespace exfold {

// The first 256 bytes of every workspace hold the device status record.
struct DeviceStatus {
    int code;    // 0 or EXFOLD_ERR_DEVICE_TIMEOUT
    int where;   // which wait gave up (kernel-specific tag)
    int detail;  // block index
    int pad[61];
};
static_assert(sizeof(DeviceStatus) == 256, "status record is 256 bytes");

constexpr int kMaxExperts = 256;  // routed experts
constexpr int kMaxTopK = 32;
constexpr int kMaxGroups = kMaxExperts + 1;  // + shared expert
constexpr int kTileM = 128;                  // token rows per prefill GEMM tile
#ifndef EXFOLD_BK
#define EXFOLD_BK 64
#endif
// K elements per pipeline stage of the tensor-core GEMMs: 64 (128-byte rows, 128-byte swizzle) or 32 (64-byte rows,
// 64-byte swizzle: half the bytes per stage, so twice as many stages fit in shared memory)
constexpr int kGemmBK = EXFOLD_BK;
constexpr int kMaxDecodeBatch = 256;
constexpr int kMaxCtas = 160;                // persistent grids never exceed this (148 SMs on B200)

__device__ __forceinline__ void report_timeout(DeviceStatus* st, int where) {
    if (atomicCAS(&st->code, 0, EXFOLD_ERR_DEVICE_TIMEOUT) == 0) {
        st->where = where;
        st->detail = (int)blockIdx.x;
    }
}

// host-side launch accounting
void count_launch(int n = 1);
// Synchronises the stream, decodes and clears the device status record at `rec`
int read_status_record(void* rec, cudaStream_t s);

// Programmatic dependent launch: every kernel of the library is launched with the "programmatic stream
// serialization" attribute, lets its successor be scheduled early (grid_dep_launch) and waits for its
// predecessor's results (grid_dep_wait) before it touches global memory. This removes the several
// microseconds of launch latency between dependent kernels of one call. Both are no-ops when the
// kernel was launched without the attribute.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Programmatic launch is requested per call chain: it pays for the short, latency-bound decode chain and
// measured slower for prefill (early-resident successors compete with the running kernel).
void set_pdl(bool on);
bool pdl_enabled();

// Order-preserving map float -> uint32 (larger float <=> larger key), so warp arg-max / arg-min can use
// the hardware integer reductions (redux.sync) instead of shuffle trees.
// -0.0 and +0.0 compare equal as floats, so they get one key (a tie, which the lower expert id then wins).
__device__ __forceinline__ uint32_t float_order_key(float f) {
    uint32_t b = __float_as_uint(f);
    if (b == 0x80000000u) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float float_from_order_key(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
// Warp-wide (value desc, id asc) arg-max. Lanes without a candidate pass has = false. Returns the
// winning id to every lane and its key through *key_out. At least one lane must have a candidate.
__device__ __forceinline__ int warp_argmax(bool has, uint32_t key, int id, uint32_t* key_out) {
    const uint32_t m = __reduce_max_sync(0xffffffffu, has ? key : 0u);
    const int best = __reduce_min_sync(0xffffffffu, (has && key == m) ? id : 0x7fffffff);
    *key_out = m;
    return best;
}
// Warp-wide (value asc, id asc) arg-min over lanes with has = true.
__device__ __forceinline__ int warp_argmin(bool has, uint32_t key, int id) {
    const uint32_t m = __reduce_min_sync(0xffffffffu, has ? key : 0xffffffffu);
    return __reduce_min_sync(0xffffffffu, (has && key == m) ? id : 0x7fffffff);
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
    count_launch();
    return e;
}

// Same, with the grid split into thread-block clusters of `cluster` CTAs (distributed shared memory)
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, unsigned cluster,
                               cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 2 : 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
    count_launch();
    return e;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---------------------------------------------------------------- routing (prefill)
struct PrefillRouteParams {
    const float* logits;  // [T][N]
    const float* S;       // [N][N]
    const float* L;       // [N][N]
    const float* lnh;     // [N]
    int64_t T;
    int N, K, Kp;
    float loss_thr;     // pairs with loss above it are not admissible targets (+inf: off)
    int rescale;        // keep the original routed-weight sum after folding
    int confidence;     // confidence-aware split of the folded weight
    int32_t* ids;       // [T][Kp]
    float* w;           // [T][Kp]
    int32_t* omit_src;  // [T][K-Kp] or null
    int32_t* omit_tgt;  // [T][K-Kp] or null
    int32_t* block_hist;  // [nblk][N]
    int32_t* sb_hist;     // [ceil(nblk / kRouteSuperBlock)][N] retained routes per (super-block, expert); the
                          //   launcher clears it, the blocks add to it
    DeviceStatus* status; // cleared by block 0 (first kernel of a call); may be null
};
constexpr int kRouteTokensPerBlock = 32;
constexpr int kRouteThreads = 512;
constexpr int kRouteSuperBlock = 64;  // blocks per super-block of the two-level histogram

struct PrefillScatterParams {
    int64_t T;
    int N, n_shared, Kp, d_bytes;  // d_bytes: bytes of one x row (0: no gather)
    int nblk;                   // blocks of the route kernel (= blocks of this kernel)
    const int32_t* ids;         // [T][Kp]
    const float* w;             // [T][Kp]
    const int32_t* block_hist;  // [nblk][N] retained routes per (block, expert)
    const int32_t* sb_hist;     // [ceil(nblk / kRouteSuperBlock)][N] the same per super-block
    int32_t* offsets;           // [G+1] out: first sorted row of each group
    int32_t* work_start;        // [G+1] out: prefix of 128-row tiles per group
    const void* x;      // [T][d]
    void* xs;           // [R][d] gathered rows (may be null)
    int32_t* perm;      // [R]
    int32_t* row_tok;   // [R + T*n_shared]
    float* row_w;       // [R + T*n_shared]
    int32_t* row_exp;   // [R + T*n_shared]
    int32_t* inv_pos;   // [R] sorted row of each route (inverse of perm); may be null
};

cudaError_t launch_prefill_route(const PrefillRouteParams& p, cudaStream_t s);
cudaError_t launch_prefill_scatter(const PrefillScatterParams& p, cudaStream_t s);

// ---------------------------------------------------------------- routing (decode)
struct DecodeRouteParams {
    const float* logits;  // [B][N]
    const float* S;
    const float* L;
    const float* h;
    int B, N, K, M, n_shared;
    // static pool (all null for the dynamic pool of Eq. 11): precomputed pool, targets and scalars
    const int32_t* st_pool;    // [M]
    const int32_t* st_target;  // [N]
    const float* st_scale;     // [N]
    // metadata (workspace copies)
    int32_t* pool_ids;    // [N] (-1 padded)
    int32_t* pool_size;   // [1]
    uint32_t* pool_mask;  // [8]
    int32_t* ids;         // [B][K]
    float* w;             // [B][K]
    int32_t* target;      // [N]
    float* scale;         // [N]
    // execution lists: rows sorted by pool rank (then shared expert), duplicates merged
    int32_t* row_tok;     // [B*K + B]
    float* row_w;         // [B*K + B]
    int32_t* grp_expert;  // [N+1] expert id of each group (pool order; shared last)
    int32_t* grp_off;     // [N+2] first row of each group
    int32_t* grp_tiles;   // [N+2] prefix of 128-row tiles per group (work list of the grouped GEMMs)
    int32_t* n_groups;    // [2]: number of groups, total rows
    DeviceStatus* status; // cleared here (first kernel of a decode call)
};
cudaError_t launch_decode_route(const DecodeRouteParams& p, cudaStream_t s);

// Token-parallel half of decode routing for bf16 layers (one CTA per token): optional router scores, Top-K,
// softmax weights in double; clears the status record
struct DecodeTopkParams {
    const float* logits;            // [B][N] (w_router == null)
    const __nv_bfloat16* x;         // [B][d]  (w_router != null)
    const __nv_bfloat16* w_router;  // [N][d] or null
    float* logits_out;              // [B][N] (w_router != null)
    int B, N, K, d;
    int32_t* ids;   // [B][K] routed experts in router order
    double* w64;    // [B][K] their softmax weights
    DeviceStatus* status;
};
cudaError_t launch_decode_topk(const DecodeTopkParams& p, cudaStream_t s);

// Decode, bf16 layers: the gate/up half of the expert FFN over the pool. The kernel finishes the routing in its
// prologue (every CTA: pool of Eq. 11 from the routed weights, minimum-loss targets of Eq. 12, remap of Eq. 14,
// rows per group), streams the pool's gate and up weights once against x read in place, and leaves H (compact rows)
// and the execution lists for the grouped down projection (ffn_decode.cu)
struct DecodeFfnParams {
    CUtensorMap tm_x;     // x [B][d], box a_rows x 64
    CUtensorMap tm_wg;    // W_gate as [(E*I)][d], box 128 x 64
    CUtensorMap tm_wu;    // W_up
    CUtensorMap tm_wg64;  // the same with 64-row boxes (half-width items)
    CUtensorMap tm_wu64;
    CUtensorMap tm_wg96;  // and with 96-row boxes (a single round of 96-wide items)
    CUtensorMap tm_wu96;
    const int32_t* ids;   // [B][K] from the top-k kernel
    const double* w64;    // [B][K]
    const float* S;       // tables (dynamic pool)
    const float* L;
    const float* h;
    const int32_t* st_pool;    // static pool (all null for the dynamic pool)
    const int32_t* st_target;
    const float* st_scale;
    int B, N, K, M, n_shared, d, I, a_rows;
    int stages, scratch_off;  // shared-memory plan made by the launcher
    // metadata written by CTA 0 (workspace copies)
    int32_t* pool_ids;    // [N] (-1 padded)
    int32_t* pool_size;   // [1]
    uint32_t* pool_mask;  // [8]
    int32_t* out_ids;     // [B][K] remapped
    float* out_w;         // [B][K]
    int32_t* target;      // [N]
    float* scale;         // [N]
    // execution lists: one row per distinct (token, pool expert), grouped by pool rank (shared expert last)
    __nv_bfloat16* H;     // [rows][I]
    int32_t* row_tok;     // [rows]
    float* row_w;         // [rows] merged weight of the row
    int32_t* slot_row;    // [B][K] row of each routed slot, -1 for a slot merged into an earlier one
    int32_t* grp_expert;  // [G]
    int32_t* grp_off;     // [G+1]
    int32_t* grp_tiles;   // [G+1] prefix of 128-row tiles per group
    int32_t* n_groups;    // [3]: groups, rows, first row of the shared expert's group
    DeviceStatus* status;
};
cudaError_t launch_decode_ffn(const DecodeFfnParams& p, int sms, cudaStream_t s);
size_t decode_ffn_smem_plan(int B, int K, int N, int* stages, int* scratch_off, int* a_rows);
cudaError_t launch_static_pool(int N, int M, const float* S, const float* L, const float* h, int32_t* pool_ids,
                               int32_t* target, float* scale, cudaStream_t s);

// ---------------------------------------------------------------- SIMT expert FFN (fp32 accumulate)
struct SimtFfnParams {
    const void* x;  // [T][d]
    const void* wg;
    const void* wu;
    const void* wd;
    int dtype, d, I;
    int64_t T;           // tokens
    int Kr;              // routes per token; row r < T*Kr is route (r / Kr, r % Kr)
    int n_shared, N;     // rows T*Kr + i run the shared expert (index N) on token i
    const int32_t* ids;  // [T][Kr] expert of each route
    float* out;          // [T*Kr + T*n_shared][d] unweighted expert outputs
};
cudaError_t launch_simt_ffn(const SimtFfnParams& p, cudaStream_t s);
// y[i] = sum_j w[i][j] out[i*Kr+j] (+ out[T*Kr+i] for the shared expert); y in the layer dtype
cudaError_t launch_combine_routes(const float* out, const float* w, int64_t T, int Kr, int d, int n_shared,
                                  void* y, int dtype, cudaStream_t s);
cudaError_t launch_router_simt(const void* x, const void* wr, int dtype, int64_t T, int N, int d, float* out,
                               cudaStream_t s);
// y[i] = sum_j O[inv_pos[i*Kr+j]] (entries < 0 skipped) (+ O[shared0 + i] for the shared expert), fp32 sum in slot
// order, bf16 out. shared0 = T*Kr, or *shared0_dev when that is given (decode: known only on the device). A row may
// be stored as `parts` partial rows (decode's K split), part k at row k * part_rows + row: summed in that order.
cudaError_t launch_combine_rows(const __nv_bfloat16* O, const int32_t* inv_pos, int64_t T, int Kr, int d,
                                int n_shared, const int32_t* shared0_dev, int parts, int64_t part_rows,
                                __nv_bfloat16* y, cudaStream_t s);
constexpr int kMaxDecodeKsplit = 2;

// ---------------------------------------------------------------- calibration
struct CalibStatsParams {
    const float* out;    // expert outputs, one row of d floats per (token, slot)
    // row of (token i, slot a): inv_pos[i*Ke + a] if inv_pos is set, else i*tok_stride + a*slot_stride
    const int32_t* inv_pos;
    int64_t tok_stride, slot_stride;
    const int32_t* ids;  // [m][Ke]
    int64_t m;
    int Ke, d, N;
    double* A;  // [N][N]
    double* Bv;
    double* C;
    int32_t* cnt;  // [N][N]
    double* H;     // [N]
    int32_t* hc;   // [N]
};
cudaError_t launch_calib_stats(const CalibStatsParams& p, cudaStream_t s);
// Common-input mode with identity slots (slot a = expert a, inv_pos unused): same sums via per-token Gram
// products held in registers; nrm is scratch for m*Ke doubles
cudaError_t launch_calib_stats_common(const CalibStatsParams& p, double* nrm, int sms, cudaStream_t s);
cudaError_t launch_calib_finalize(const CalibStatsParams& p, const exfold_calib_opts& o, float* S, float* L,
                                  float* h, float* lnh, int32_t* n_obs, int32_t* unobserved, cudaStream_t s);
cudaError_t launch_iota_ids(int32_t* ids, int64_t m, int N, cudaStream_t s);
// Common-input calibration on the grouped GEMMs: every expert e owns rows [e*m, (e+1)*m) = all tokens in order
cudaError_t launch_calib_common_rows(int32_t* offsets, int32_t* work_start, int64_t m, int N, cudaStream_t s);

// ---------------------------------------------------------------- tcgen05 grouped GEMMs (bf16)
// SM pairs, of n_clusters, that the CTA-pair passes keep when the odd-tile passes run beside them on the other
// 2 * (n_clusters - P) SMs. Every kernel of a call (both passes of both GEMMs) evaluates this on the device from the
// same group offsets, so they agree, and the split is the same for GEMM-1 and GEMM-2: `pairs` whole pairs of row tiles
// and `odd` odd tiles, each times the column tiles (nt) and k-blocks per item (nkb) of the two GEMMs. Side by side,
// a pair item takes a cluster ~0.73 of the time an odd item takes one SM (measured on the Mixtral shape: 25.9 against
// 35.7 us per 64-k-block item; the one-CTA kernel is the hungrier of the two for L2 bandwidth and slows down more
// beside the other). The choice minimises the longer of the two chains (GEMM-1 pass, then GEMM-2 pass), each pass
// counted in rounds of items. The odd-tile pass cannot get more than the odd_ctas CTAs it was launched with.
struct SideBySide {
    int nt1, nkb1, nt2, nkb2;  // column tiles and k-blocks per work item of GEMM-1 and GEMM-2
    int n_sm_pairs;            // SM pairs the pair passes are launched over
    int odd_ctas;              // CTAs the odd-tile passes are launched with (even); 0: the passes do not run side by side
    int shared_pairs1;         // whole row-tile pairs of the shared expert that GEMM-1's pair pass does not run (they
                               // ran beside the routing kernels, GroupedGemmParams::shared_split), else 0
};
__host__ __device__ inline int pair_pass_clusters(int pairs, int odd, const SideBySide& sb) {
    const int n = sb.n_sm_pairs;
    if (odd <= 0) return n;
    const int p_min = n - sb.odd_ctas / 2 > 0 ? n - sb.odd_ctas / 2 : 0;
    if (pairs <= 0) return p_min;
    int best = p_min > 1 ? p_min : 1;
    float best_t = 3.0e38f;
    for (int P = best; P < n; ++P) {
        const int Q = 2 * (n - P);
        const int pairs1 = pairs - sb.shared_pairs1;
        const float tp = 0.73f * (float)(((pairs1 * sb.nt1 + P - 1) / P) * sb.nkb1 + ((pairs * sb.nt2 + P - 1) / P) * sb.nkb2);
        const float to = (float)(((odd * sb.nt1 + Q - 1) / Q) * sb.nkb1 + ((odd * sb.nt2 + Q - 1) / Q) * sb.nkb2);
        const float t = tp > to ? tp : to;
        if (t < best_t) {
            best_t = t;
            best = P;
        }
    }
    return best;
}
struct GroupedGemmParams {
    CUtensorMap tm_a;    // GEMM-1: gathered rows Xs [R][d]; GEMM-2: H [Rtot][I]
    CUtensorMap tm_a2;   // GEMM-1: x [T][d] for the shared expert's rows
    CUtensorMap tm_b0;   // GEMM-1: W_gate as [(E*I)][d]; GEMM-2: W_down as [(E*d)][I]
    CUtensorMap tm_b1;   // GEMM-1: W_up; GEMM-2 on CTA pairs: W_down with 128-row boxes (each CTA stages half a tile)
    const int32_t* offsets;     // [G+1]
    const int32_t* work_start;  // [G+1] prefix of row tiles
    int G;                      // groups (N + n_shared)
    int n_routed;               // N
    int R;                      // routed rows (shared rows start here)
    int d, I;
    int n_ntiles;               // column tiles
    int ksplit;                 // GEMM-2, decode: K parts per tile; part k of a row goes to plane k of the row buffer
    int a_rows;                 // decode: rows of the A (token) box, a multiple of 32 <= 128; prefill: 128
    const int32_t* grp_expert;  // [G] expert whose weights group g uses (null: g itself)
    const int32_t* n_groups_dev;  // device-side group count (null: G)
    // epilogues
    __nv_bfloat16* H;           // GEMM-1 out [Rtot][I]
    const int32_t* row_tok;     // GEMM-2
    const float* row_w;         // GEMM-2
    __nv_bfloat16* y;           // GEMM-2 bf16 target: row = token (store_rows == 0) or the sorted row itself
    int store_rows;             // 1: y is the per-route buffer O[row][d] that the combine kernel sums
    float* o32;                 // GEMM-2, calibration: unweighted fp32 outputs O32[row][d] (null: the epilogues above)
    int x_rows;                 // GEMM-1: rows of x; a group that reads x directly starts at row (row0 - R) % x_rows
    int shared_split;           // CTA-pair GEMM-1. 1: this launch runs only the whole row-tile pairs of the shared expert
                                //    (rows [R, R + x_rows) of expert n_routed, read from x: nothing the routing kernels
                                //    write is touched, so it runs beside them); 2: those pairs ran that way, skip them
    int odd_only;               // 1: only each group's last row tile, and only if its tile count is odd (the rest ran on CTA pairs)
    SideBySide sbs;             // odd_ctas > 0: the CTA-pair pass and the odd-tile pass run at the same time (two
                                //    streams); each keeps its share of the SM pairs (pair_pass_clusters) and the CTAs
                                //    beyond it leave at once
    DeviceStatus* status;
};
cudaError_t launch_grouped_gemm1(const GroupedGemmParams& p, int grid, cudaStream_t s);
cudaError_t launch_grouped_gemm2(const GroupedGemmParams& p, int grid, cudaStream_t s);
// Prefill on CTA pairs: every group's row tiles two at a time (a last odd tile is left to the kernels above with
// odd_only = 1). GEMM-2 needs tm_b1 = W_down with 128-row boxes. No grp_expert, no K split, o32 = null.
cudaError_t launch_grouped_gemm1_pair(const GroupedGemmParams& p, int grid, cudaStream_t s);
cudaError_t launch_grouped_gemm2_pair(const GroupedGemmParams& p, int grid, cudaStream_t s);
// The odd-tile pass beside them (p.odd_only = 1; prefill instantiation), launched two CTAs at a time so that the two
// grids share the GPU by whole SM pairs
cudaError_t launch_grouped_gemm1_odd(const GroupedGemmParams& p, int grid, cudaStream_t s);
cudaError_t launch_grouped_gemm2_odd(const GroupedGemmParams& p, int grid, cudaStream_t s);

}  // namespace exfold
