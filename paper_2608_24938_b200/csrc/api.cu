// C ABI of the folded-MoE library: argument validation, workspace planning, TMA tensor maps
// and the launch sequences of the three calls. No device memory is allocated here.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstdlib>
#include <cmath>
#include <cstring>

#include "common.cuh"
#include "ptx.cuh"


namespace exfold {

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
static thread_local bool t_pdl = false;
static thread_local bool t_keep_status = false;  // set while a host-buffer call runs its second and later chunks
void set_pdl(bool on) { t_pdl = on; }
bool pdl_enabled() { return t_pdl; }

namespace {

// ------------------------------------------------------------------ optional per-kernel event timing
struct Profiler {
    bool on = false;
    cudaEvent_t beg[EXFOLD_PROFILE_SLOTS];
    cudaEvent_t end[EXFOLD_PROFILE_SLOTS];
    bool used[EXFOLD_PROFILE_SLOTS];
} g_prof;

struct ProfScope {  // records an event pair around one launch when profiling is enabled
    int slot;
    cudaStream_t s;
    ProfScope(int slot_, cudaStream_t s_) : slot(slot_), s(s_) {
        if (g_prof.on) cudaEventRecord(g_prof.beg[slot], s);
    }
    ~ProfScope() {
        if (g_prof.on) {
            cudaEventRecord(g_prof.end[slot], s);
            g_prof.used[slot] = true;
        }
    }
};
void prof_reset() {
    for (int i = 0; i < EXFOLD_PROFILE_SLOTS; ++i) g_prof.used[i] = false;
}

// ------------------------------------------------------------------ workspace plan
struct Plan {
    size_t status, ids, w, omit_src, omit_tgt, block_hist, sb_hist, offsets, work_start, totals, perm, row_tok, row_w,
        row_exp, pool_ids, pool_size, pool_mask, target, scale, grp_expert, grp_off, n_groups, zeros, calib, big,
        xs, H, out, grp_tiles, obuf, inv_pos, calib_nrm, calib_warn, w64, total;
};

bool valid_layer(const exfold_layer* l) {
    if (!l) return false;
    if (l->n_experts < 2 || l->n_experts > kMaxExperts) return false;
    if (l->n_shared < 0 || l->n_shared > 1) return false;
    if (l->top_k < 1 || l->top_k > kMaxTopK || l->top_k > l->n_experts) return false;
    if (l->hidden < 1 || l->inter < 1) return false;
    if (l->dtype != EXFOLD_F32 && l->dtype != EXFOLD_BF16) return false;
    if (l->dtype == EXFOLD_BF16 && (l->hidden % 64 != 0 || l->inter % 64 != 0)) return false;
    if (l->dtype == EXFOLD_F32 && (l->hidden % 4 != 0)) return false;
    return true;
}

Plan make_plan(const exfold_layer& l, int64_t Tm, int Kr) {
    Plan p{};
    const int N = l.n_experts, G = N + l.n_shared;
    const size_t Rm = (size_t)Tm * Kr, Rtot = Rm + (size_t)Tm * l.n_shared;
    const size_t nblk = (size_t)(Tm + kRouteTokensPerBlock - 1) / kRouteTokensPerBlock;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t at = off;
        off = align_up(off + bytes, 256);
        return at;
    };
    p.status = take(sizeof(DeviceStatus));
    // calibration: unobserved-expert count of each job of a call (ahead of everything whose size depends on the
    // token count, so that jobs of different lengths share the slots)
    p.calib_warn = take((size_t)EXFOLD_MAX_CALIB_JOBS * 4);
    p.ids = take(Rm * 4);
    p.w = take(Rm * 4);
    p.omit_src = take((size_t)Tm * l.top_k * 4);
    p.omit_tgt = take((size_t)Tm * l.top_k * 4);
    p.block_hist = take(nblk * N * 4);
    p.sb_hist = take((nblk + kRouteSuperBlock - 1) / kRouteSuperBlock * N * 4);
    p.offsets = take((G + 2) * 4);
    p.work_start = take((G + 2) * 4);
    p.totals = take(16);
    p.perm = take(Rm * 4);
    p.inv_pos = take(Rm * 4);
    p.row_tok = take(Rtot * 4);
    p.row_w = take(Rtot * 4);
    p.row_exp = take(Rtot * 4);
    p.w64 = take((size_t)std::min<int64_t>(Tm, kMaxDecodeBatch) * l.top_k * 8);  // decode: routed weights in double
    p.pool_ids = take((size_t)N * 4);
    p.pool_size = take(16);
    p.pool_mask = take(32);
    p.target = take((size_t)N * 4);
    p.scale = take((size_t)N * 4);
    p.grp_expert = take((G + 2) * 4);
    p.grp_off = take((G + 2) * 4);
    p.grp_tiles = take((G + 2) * 4);
    p.n_groups = take(16);
    p.zeros = take((size_t)N * 4);
    p.calib = take((size_t)N * N * (3 * 8 + 4) + (size_t)N * (8 + 4) + 256);
    p.calib_nrm = take(Rm * 8);  // calibration, common-input mode: squared output norms per (token, expert)
    // large buffers: the bf16 pipeline (sorted rows, H, fp32 accumulator) and the SIMT path's
    // per-route outputs are never live at the same time and share one region
    p.big = off;
    size_t a = 0;
    if (l.dtype == EXFOLD_BF16) {
        // xs and obuf are adjacent: calibration reuses the two together (>= Rtot*d*4 bytes) for the
        // fp32 per-row expert outputs once GEMM-1 has consumed the gathered rows
        p.xs = p.big;
        a = align_up(Rtot * (size_t)l.hidden * 2, 1024);
        p.obuf = p.big + a;  // per-row bf16 outputs O [Rtot][d] (decode: one plane per K part)
        a += align_up(std::max((size_t)Tm * l.hidden * 4, Rtot * (size_t)l.hidden * 2), 1024);
        p.H = p.big + a;
        a += align_up(Rtot * (size_t)l.inter * 2, 1024);
    }
    p.out = p.big;
    size_t b = align_up(Rtot * (size_t)l.hidden * 4, 1024);
    p.total = p.big + (a > b ? a : b);
    return p;
}

template <typename T>
T* at(void* ws, size_t off) {
    return reinterpret_cast<T*>(reinterpret_cast<char*>(ws) + off);
}

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

constexpr int kMaxHostChunks = 4;  // host-buffer prefill: chunks of >= 2048 tokens in flight

// bf16 matrix [rows][cols] row-major; box = box_rows x kGemmBK columns, swizzle as wide as a box row
bool make_tmap(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)kGemmBK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, kGemmBK == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Host-side CUDA objects the library keeps per (host thread, device), created on first use and kept until
// exfold_thread_release() or the end of the process:
//   side stream + fork / join / mid events: the odd-tile passes of a prefill call run beside the CTA-pair passes;
//   in / out streams + events: the chunked host-buffer prefill copies the next chunk in and the previous one out
//   while the caller's stream computes.
// Nothing else survives a call. Two caller streams used from one host thread share these objects, so the parts of
// their calls that run on them are ordered one after the other (results are unaffected).
constexpr int kMaxDevices = 64;
struct ThreadDeviceState {
    cudaStream_t side = nullptr, in = nullptr, out = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr, mid = nullptr;
    cudaEvent_t start = nullptr, done = nullptr, copied[kMaxHostChunks] = {}, computed[kMaxHostChunks] = {};
    bool side_ok = false, host_ok = false;
    int sms = 0;
    void release() {
        auto ev = [](cudaEvent_t& e) { if (e) cudaEventDestroy(e); e = nullptr; };
        auto st = [](cudaStream_t& s) { if (s) cudaStreamDestroy(s); s = nullptr; };
        ev(fork); ev(join); ev(mid); ev(start); ev(done);
        for (int c = 0; c < kMaxHostChunks; ++c) { ev(copied[c]); ev(computed[c]); }
        st(side); st(in); st(out);
        side_ok = host_ok = false;
    }
};
thread_local ThreadDeviceState t_state[kMaxDevices];

ThreadDeviceState* thread_state() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    return &t_state[dev];
}
bool new_event(cudaEvent_t* e) { return cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; }
// second stream (and fork / join events) for the odd-tile passes of a prefill call
ThreadDeviceState* side_stream() {
    ThreadDeviceState* h = thread_state();
    if (h && !h->side_ok) {
        // highest priority: what runs here beside a bandwidth-bound kernel of the caller's stream (the shared
        // expert's GEMM-1 beside the scatter kernel) gets its SMs first and the other kernel fills the rest
        int lo = 0, hi = 0;
        if (cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess) hi = 0;
        h->side_ok = cudaStreamCreateWithPriority(&h->side, cudaStreamNonBlocking, hi) == cudaSuccess &&
                     new_event(&h->fork) && new_event(&h->join) && new_event(&h->mid);
    }
    return h && h->side_ok ? h : nullptr;
}
// copy-in / copy-out streams and events of the chunked host-buffer prefill
ThreadDeviceState* host_helpers() {
    ThreadDeviceState* h = thread_state();
    if (h && !h->host_ok) {
        bool ok = cudaStreamCreateWithFlags(&h->in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&h->out, cudaStreamNonBlocking) == cudaSuccess && new_event(&h->start) &&
                  new_event(&h->done);
        for (int c = 0; ok && c < kMaxHostChunks; ++c) ok = new_event(&h->copied[c]) && new_event(&h->computed[c]);
        h->host_ok = ok;
    }
    return h && h->host_ok ? h : nullptr;
}
// Once the side stream has been forked off the caller's stream it is joined again on every way out of the call
// (also the error returns): later work on the caller's stream, or the end of a stream capture, must not overtake it.
struct SideJoin {
    ThreadDeviceState* side;
    cudaStream_t s;
    bool armed = true;
    cudaError_t join() {
        armed = false;
        cudaError_t e = cudaEventRecord(side->join, side->side);
        return e != cudaSuccess ? e : cudaStreamWaitEvent(s, side->join, 0);
    }
    ~SideJoin() {
        if (armed) join();
    }
};

int sm_count() {  // of the current device
    ThreadDeviceState* h = thread_state();
    int n = h ? h->sms : 0;
    if (n <= 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        if (h) h->sms = n;
    }
    return n;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

#define EXFOLD_CUDA(call)                                 \
    do {                                                  \
        cudaError_t e__ = (call);                         \
        if (e__ != cudaSuccess) return EXFOLD_ERR_CUDA;   \
    } while (0)

int copy_meta(void* dst, const void* src, size_t bytes, cudaStream_t s) {
    if (dst == nullptr || bytes == 0) return EXFOLD_OK;
    EXFOLD_CUDA(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, s));
    return EXFOLD_OK;
}

int check_common(const exfold_layer* layer, const void* x, const float* logits, int64_t T, const void* wg,
                 const void* wu, const void* wd, const exfold_tables* t, void* y, void* ws) {
    if (!valid_layer(layer)) return EXFOLD_ERR_INVALID_ARG;
    if (!x || !logits || !wg || !wu || !wd || !y || !ws) return EXFOLD_ERR_INVALID_ARG;
    if (!t || !t->S || !t->L || !t->h || !t->lnh) return EXFOLD_ERR_INVALID_ARG;
    if (T < 1 || T > (int64_t)1 << 24) return EXFOLD_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y) || !aligned16(wg) || !aligned16(wu) || !aligned16(wd) ||
        (reinterpret_cast<uintptr_t>(ws) & 255) != 0)
        return EXFOLD_ERR_INVALID_ARG;
    return EXFOLD_OK;
}

}  // namespace

// Synchronises the stream, decodes and clears the status record at `rec` (device memory)
int read_status_record(void* rec, cudaStream_t s) {
    if (cudaStreamSynchronize(s) != cudaSuccess) return EXFOLD_ERR_CUDA;
    int code = 0;
    if (cudaMemcpy(&code, rec, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return EXFOLD_ERR_CUDA;
    if (cudaMemset(rec, 0, sizeof(DeviceStatus)) != cudaSuccess) return EXFOLD_ERR_CUDA;
    if (code == 0) return EXFOLD_OK;
    return code == EXFOLD_ERR_DEVICE_TIMEOUT ? EXFOLD_ERR_DEVICE_TIMEOUT : EXFOLD_ERR_CUDA;
}
}  // namespace exfold

using namespace exfold;

extern "C" {

size_t exfold_workspace_bytes(const exfold_layer* layer, int64_t max_tokens, int32_t routes_per_token) {
    if (!valid_layer(layer) || max_tokens < 1 || routes_per_token < 1 || routes_per_token > kMaxExperts) return 0;
    return make_plan(*layer, max_tokens, routes_per_token).total;
}

size_t exfold_host_staging_bytes(const exfold_layer* layer, int64_t max_tokens) {
    if (!valid_layer(layer) || max_tokens < 1) return 0;
    const size_t el = layer->dtype == EXFOLD_BF16 ? 2 : 4;
    return 2 * align_up((size_t)max_tokens * layer->hidden * el, 256) +
           align_up((size_t)max_tokens * layer->n_experts * 4, 256);
}

int64_t exfold_launch_count(void) { return g_launches.load(); }

int exfold_profile_enable(int enable) {
    if (enable && !g_prof.on) {
        for (int i = 0; i < EXFOLD_PROFILE_SLOTS; ++i) {
            if (cudaEventCreate(&g_prof.beg[i]) != cudaSuccess) return EXFOLD_ERR_CUDA;
            if (cudaEventCreate(&g_prof.end[i]) != cudaSuccess) return EXFOLD_ERR_CUDA;
        }
        prof_reset();
        g_prof.on = true;
    } else if (!enable && g_prof.on) {
        g_prof.on = false;
        for (int i = 0; i < EXFOLD_PROFILE_SLOTS; ++i) {
            cudaEventDestroy(g_prof.beg[i]);
            cudaEventDestroy(g_prof.end[i]);
        }
    }
    return EXFOLD_OK;
}

int exfold_profile_read(float* ms, int32_t n_slots) {
    if (!ms || n_slots < 0) return EXFOLD_ERR_INVALID_ARG;
    for (int i = 0; i < n_slots; ++i) {
        ms[i] = -1.0f;
        if (!g_prof.on || i >= EXFOLD_PROFILE_SLOTS || !g_prof.used[i]) continue;
        if (cudaEventSynchronize(g_prof.end[i]) != cudaSuccess) return EXFOLD_ERR_CUDA;
        if (cudaEventElapsedTime(&ms[i], g_prof.beg[i], g_prof.end[i]) != cudaSuccess) return EXFOLD_ERR_CUDA;
    }
    return EXFOLD_OK;
}

const char* exfold_status_string(int status) {
    switch (status) {
        case EXFOLD_OK: return "ok";
        case EXFOLD_ERR_INVALID_ARG: return "invalid argument";
        case EXFOLD_ERR_UNSUPPORTED: return "unsupported configuration";
        case EXFOLD_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case EXFOLD_ERR_CUDA: return "CUDA error";
        case EXFOLD_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
        case EXFOLD_ERR_EXCEEDS_STATIC_SCRATCH:
            return "layer and batch need more scratch than the built-in EXFOLD_STATIC_SCRATCH_BYTES array holds";
        case EXFOLD_WARN_UNOBSERVED_EXPERT: return "warning: an expert was never observed during calibration";
        default: return "unknown status";
    }
}

int exfold_device_status(void* ws, void* cuda_stream) {
    if (!ws) return EXFOLD_ERR_INVALID_ARG;
    return read_status_record(ws, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int exfold_thread_release(void) {
    ThreadDeviceState* h = thread_state();
    if (!h) return EXFOLD_ERR_CUDA;
    h->release();
    return EXFOLD_OK;
}

int exfold_moe_prefill(const exfold_layer* layer, const void* x, const float* logits, int64_t T, const void* w_gate,
                       const void* w_up, const void* w_down, const exfold_tables* tables, int32_t k_pre, void* y,
                       const exfold_prefill_meta* meta, void* ws, size_t ws_bytes, void* cuda_stream) {
    return exfold_moe_prefill_ex(layer, x, logits, T, w_gate, w_up, w_down, tables, k_pre, nullptr, y, meta, ws,
                                 ws_bytes, cuda_stream);
}

int exfold_moe_prefill_ex(const exfold_layer* layer, const void* x, const float* logits, int64_t T,
                          const void* w_gate, const void* w_up, const void* w_down, const exfold_tables* tables,
                          int32_t k_pre, const exfold_fold_opts* opts, void* y, const exfold_prefill_meta* meta,
                          void* ws, size_t ws_bytes, void* cuda_stream) {
    int rc = check_common(layer, x, logits, T, w_gate, w_up, w_down, tables, y, ws);
    if (rc != EXFOLD_OK) return rc;
    const exfold_layer& l = *layer;
    if (k_pre < 1 || k_pre > l.top_k) return EXFOLD_ERR_INVALID_ARG;
    const int N = l.n_experts, K = l.top_k, Kp = k_pre, d = l.hidden, I = l.inter, G = N + l.n_shared;
    const int64_t R = T * Kp, Rtot = R + T * l.n_shared;
    if (Rtot > (int64_t)1 << 30) return EXFOLD_ERR_UNSUPPORTED;
    const Plan pl = make_plan(l, T, Kp);
    if (ws_bytes < pl.total) return EXFOLD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    const bool bf16 = l.dtype == EXFOLD_BF16;
    const bool direct = bf16 && Kp == 1 && l.n_shared == 0;  // every token is written exactly once

    CUtensorMap tm_xs, tm_x, tm_wg, tm_wu, tm_h, tm_wd, tm_wd_half;
    // A call with enough work (>= 24 row tiles of 128 sorted rows) runs every group's row tiles two at a time on CTA
    // pairs (gemm_pair.cu: a third less operand traffic per SM, a deeper ring, the tensor pipe busy > 95 % of the
    // main loop) and only a group's odd last tile on the one-CTA kernel, the two passes side by side (below).
    // Measured against the one-CTA kernel alone: Mixtral shape 4096 / 8192 / 16384 / 32768 tokens -3 / -9 / -14 /
    // -16 %, GLM shape -8 %, Qwen3 shape (half of the experts own a single tile) -1 %.
    const int64_t tiles_est = Rtot / kTileM + G / 2;
    const int mode = opts == nullptr || opts->gemm_path < 0 || opts->gemm_path > 2 ? 0 : opts->gemm_path;
    const bool pairs = bf16 && kGemmBK == 64 && (mode == 2 ? Rtot >= 2 * kTileM : mode == 0 && tiles_est >= 24);
    const int sms = sm_count() & ~1;
    if (bf16) {
        const uint64_t E = (uint64_t)G;
        bool ok = make_tmap(&tm_xs, at<char>(ws, pl.xs), (uint64_t)R, d, 128) && make_tmap(&tm_x, x, (uint64_t)T, d, 128) &&
                  make_tmap(&tm_wg, w_gate, E * I, d, 128) && make_tmap(&tm_wu, w_up, E * I, d, 128) &&
                  make_tmap(&tm_h, at<char>(ws, pl.H), (uint64_t)Rtot, I, 128) &&
                  make_tmap(&tm_wd, w_down, E * d, I, 256) && make_tmap(&tm_wd_half, w_down, E * d, I, 128);
        if (!ok) return EXFOLD_ERR_CUDA;
    }

    prof_reset();

    PrefillRouteParams rp{};
    rp.logits = logits; rp.S = tables->S; rp.L = tables->L; rp.lnh = tables->lnh;
    rp.T = T; rp.N = N; rp.K = K; rp.Kp = Kp;
    rp.loss_thr = opts ? opts->loss_threshold : INFINITY;
    rp.rescale = opts ? opts->rescale : 0;
    rp.confidence = opts ? opts->confidence_split : 0;
    rp.ids = at<int32_t>(ws, pl.ids); rp.w = at<float>(ws, pl.w);
    rp.omit_src = at<int32_t>(ws, pl.omit_src); rp.omit_tgt = at<int32_t>(ws, pl.omit_tgt);
    rp.block_hist = at<int32_t>(ws, pl.block_hist);
    rp.sb_hist = at<int32_t>(ws, pl.sb_hist);
    // the first kernel of the call clears the status record (not for the later chunks of a chunked host call)
    rp.status = t_keep_status ? nullptr : at<DeviceStatus>(ws, pl.status);
    { ProfScope ps(0, s); EXFOLD_CUDA(launch_prefill_route(rp, s)); }

    // The shared expert's gate/up projection needs nothing the routing kernels produce (its rows are x itself, its
    // rows of H lie behind the routed ones): its whole row-tile pairs run on the second stream beside the scatter
    // kernel, which moves bytes while the tensor pipes would idle. (After the routing kernel, which clears the status
    // record every kernel's waits look at.) The CTA-pair GEMM-1 that follows the scatter kernel skips those pairs.
    // Not with per-kernel timing on: the timed kernels are then the plain sequence, GEMM-1 with all its pairs.
    const int shared_pairs = pairs && l.n_shared && !g_prof.on ? (int)(((T + kTileM - 1) / kTileM) / 2) : 0;
    ThreadDeviceState* early_side = nullptr;
    if (shared_pairs > 0) {
        early_side = side_stream();
        if (!early_side) return EXFOLD_ERR_CUDA;
        GroupedGemmParams gs{};
        gs.tm_a = tm_xs; gs.tm_a2 = tm_x; gs.tm_b0 = tm_wg; gs.tm_b1 = tm_wu; gs.x_rows = (int)T;
        gs.G = G; gs.n_routed = N; gs.R = (int)R; gs.d = d; gs.I = I; gs.n_ntiles = (I + 127) / 128; gs.ksplit = 1;
        gs.a_rows = kTileM; gs.H = at<__nv_bfloat16>(ws, pl.H); gs.status = at<DeviceStatus>(ws, pl.status);
        gs.shared_split = 1;
        gs.sbs = SideBySide{(I + 127) / 128, d / kGemmBK, (d + 255) / 256, I / kGemmBK, sms / 2, 0, 0};
        EXFOLD_CUDA(cudaEventRecord(early_side->fork, s));
        EXFOLD_CUDA(cudaStreamWaitEvent(early_side->side, early_side->fork, 0));
        EXFOLD_CUDA(launch_grouped_gemm1_pair(gs, sms, early_side->side));
        EXFOLD_CUDA(cudaEventRecord(early_side->mid, early_side->side));
    }
    SideJoin early_join{early_side, s};  // joins the second stream on the error returns before the passes below take over
    early_join.armed = early_side != nullptr;

    PrefillScatterParams cp{};
    cp.T = T; cp.N = N; cp.n_shared = l.n_shared; cp.Kp = Kp; cp.d_bytes = bf16 ? d * 2 : 0;
    cp.nblk = (int)((T + kRouteTokensPerBlock - 1) / kRouteTokensPerBlock);
    cp.ids = rp.ids; cp.w = rp.w; cp.block_hist = rp.block_hist; cp.sb_hist = rp.sb_hist;
    cp.offsets = at<int32_t>(ws, pl.offsets); cp.work_start = at<int32_t>(ws, pl.work_start);
    cp.x = x; cp.xs = bf16 ? at<char>(ws, pl.xs) : nullptr;
    cp.perm = at<int32_t>(ws, pl.perm); cp.row_tok = at<int32_t>(ws, pl.row_tok);
    cp.row_w = at<float>(ws, pl.row_w); cp.row_exp = at<int32_t>(ws, pl.row_exp);
    cp.inv_pos = at<int32_t>(ws, pl.inv_pos);
    { ProfScope ps(2, s); EXFOLD_CUDA(launch_prefill_scatter(cp, s)); }

    if (bf16) {
        GroupedGemmParams g{};
        g.tm_a = tm_xs; g.tm_a2 = tm_x; g.tm_b0 = tm_wg; g.tm_b1 = tm_wu; g.x_rows = (int)T; g.o32 = nullptr;
        g.offsets = cp.offsets; g.work_start = cp.work_start; g.G = G; g.n_routed = N; g.R = (int)R;
        g.d = d; g.I = I; g.n_ntiles = (I + 127) / 128; g.ksplit = 1; g.a_rows = kTileM;
        g.grp_expert = nullptr; g.n_groups_dev = nullptr;
        g.H = at<__nv_bfloat16>(ws, pl.H); g.row_tok = cp.row_tok; g.row_w = cp.row_w;
        g.y = nullptr; g.status = at<DeviceStatus>(ws, pl.status);
        const int64_t max_tiles = Rtot / kTileM + G;
        const int nt1 = (I + 127) / 128, nt2 = (d + 255) / 256;
        GroupedGemmParams g2 = g;  // GEMM-2: H x W_down -> y (or the per-route buffer O)
        g2.tm_a = tm_h; g2.tm_b0 = tm_wd; g2.tm_b1 = tm_wd_half; g2.n_ntiles = nt2;
        // K' = 1 without a shared expert: every token is written once, straight into y. Otherwise each
        // route's weighted output goes to O (bf16, sorted rows) and the combine kernel sums per token.
        g2.y = direct ? reinterpret_cast<__nv_bfloat16*>(y) : at<__nv_bfloat16>(ws, pl.obuf);
        g2.store_rows = direct ? 0 : 1;
        if (!pairs) {
            { ProfScope ps(3, s); EXFOLD_CUDA(launch_grouped_gemm1(g, (int)std::min<int64_t>(sm_count(), max_tiles * nt1), s)); }
            { ProfScope ps(4, s); EXFOLD_CUDA(launch_grouped_gemm2(g2, (int)std::min<int64_t>(sm_count(), max_tiles * nt2), s)); }
        } else {
            // Both passes are launched over all SMs, the pair pass on the caller's stream and the odd-tile pass on a
            // second one; on the device each keeps its share of the SM pairs (pair_pass_clusters of the actual tile
            // counts) and its other CTAs leave at once, so the two grids settle side by side whatever the routing.
            // Rows of whole tile pairs and rows of odd last tiles never meet before the combine step, so each pass
            // of GEMM-2 follows the same pass of GEMM-1 on its own stream: caller's stream: GEMM-1 pairs -> GEMM-2
            // pairs; side stream: GEMM-1 odd tiles -> GEMM-2 odd tiles; joined before the combine kernel (or the
            // end of the call). With per-kernel timing on, the streams also join between the two GEMMs.
            ThreadDeviceState* sidep = side_stream();
            if (!sidep) return EXFOLD_ERR_CUDA;
            ThreadDeviceState& side = *sidep;
            GroupedGemmParams go1 = g, go2 = g2;
            go1.odd_only = go2.odd_only = 1;
            // The odd-tile pass is launched with about twice the CTAs its expected share of the work needs (its share
            // is decided on the device, where the tile counts are known): CTAs without work leave at once, but every
            // one of them has to pass through one of the pass's few SMs first.
            const double odd_est = std::max<double>(1.0, G / 2.0), pair_est = std::max<double>(1.0, (tiles_est - G / 2.0) / 2.0);
            const double q_est = sms * odd_est / (odd_est + 2 * 0.73 * pair_est);
            const int odd_grid = std::min(sms, 2 * (int)std::ceil(q_est) + 8) & ~1;
            const SideBySide sbs{nt1, d / kGemmBK, nt2, I / kGemmBK, sms / 2, odd_grid, shared_pairs};
            g.sbs = g2.sbs = go1.sbs = go2.sbs = sbs;
            if (shared_pairs > 0) {  // the shared expert's pairs of GEMM-1 are done (or running) on the second stream
                g.shared_split = 2;
                EXFOLD_CUDA(cudaStreamWaitEvent(s, side.mid, 0));
            }
            EXFOLD_CUDA(cudaEventRecord(side.fork, s));
            EXFOLD_CUDA(cudaStreamWaitEvent(side.side, side.fork, 0));
            SideJoin joiner{sidep, s};
            early_join.armed = false;
            {
                ProfScope ps(3, s);
                { ProfScope pp(12, s); EXFOLD_CUDA(launch_grouped_gemm1_pair(g, sms, s)); }
                EXFOLD_CUDA(launch_grouped_gemm1_odd(go1, odd_grid, side.side));
                if (g_prof.on) {
                    EXFOLD_CUDA(cudaEventRecord(side.mid, side.side));
                    EXFOLD_CUDA(cudaStreamWaitEvent(s, side.mid, 0));
                }
            }
            {
                ProfScope ps(4, s);
                { ProfScope pp(13, s); EXFOLD_CUDA(launch_grouped_gemm2_pair(g2, sms, s)); }
                EXFOLD_CUDA(launch_grouped_gemm2_odd(go2, odd_grid, side.side));
                EXFOLD_CUDA(joiner.join());
            }
        }
        if (!direct) {
            ProfScope ps(5, s);
            EXFOLD_CUDA(launch_combine_rows(at<__nv_bfloat16>(ws, pl.obuf), cp.inv_pos, T, Kp, d, l.n_shared, nullptr, 1, 0,
                                            reinterpret_cast<__nv_bfloat16*>(y), s));
        }
    } else {
        SimtFfnParams fp{};
        fp.x = x; fp.wg = w_gate; fp.wu = w_up; fp.wd = w_down; fp.dtype = l.dtype; fp.d = d; fp.I = I;
        fp.T = T; fp.Kr = Kp; fp.n_shared = l.n_shared; fp.N = N; fp.ids = rp.ids; fp.out = at<float>(ws, pl.out);
        { ProfScope ps(10, s); EXFOLD_CUDA(launch_simt_ffn(fp, s)); }
        { ProfScope ps(11, s); EXFOLD_CUDA(launch_combine_routes(fp.out, rp.w, T, Kp, d, l.n_shared, y, l.dtype, s)); }
    }
    if (meta) {
        if ((rc = copy_meta(meta->ids, rp.ids, (size_t)R * 4, s))) return rc;
        if ((rc = copy_meta(meta->w, rp.w, (size_t)R * 4, s))) return rc;
        if ((rc = copy_meta(meta->omit_src, rp.omit_src, (size_t)T * (K - Kp) * 4, s))) return rc;
        if ((rc = copy_meta(meta->omit_tgt, rp.omit_tgt, (size_t)T * (K - Kp) * 4, s))) return rc;
        if ((rc = copy_meta(meta->perm, cp.perm, (size_t)R * 4, s))) return rc;
        if ((rc = copy_meta(meta->offsets, cp.offsets, (size_t)(N + 1) * 4, s))) return rc;
    }
    return EXFOLD_OK;
}

static int router_enqueue(const exfold_layer* layer, const void* x, const void* w_router, int64_t T, float* logits,
                          void* ws, size_t ws_bytes, cudaStream_t s, bool clear_status);

// Dynamic (tables != null) or static (spool != null) decode step.
// w_router != null: the router scores are computed first (into `logits`, which is then an output).
static int decode_impl(const exfold_layer* layer, const void* x, const float* logits, int64_t B, const void* w_gate,
                       const void* w_up, const void* w_down, const exfold_tables* tables,
                       const exfold_static_pool* spool, int32_t pool_m, void* y, const exfold_decode_meta* meta,
                       void* ws, size_t ws_bytes, void* cuda_stream, const void* w_router = nullptr) {
    exfold_tables dummy{};  // the static path needs no tables: satisfy the common pointer checks
    if (spool != nullptr) {
        if (!spool->pool_ids || !spool->target || !spool->scale) return EXFOLD_ERR_INVALID_ARG;
        dummy.S = dummy.L = dummy.h = dummy.lnh = spool->scale;
        tables = &dummy;
        pool_m = spool->pool_m;
    }
    int rc = check_common(layer, x, logits, B, w_gate, w_up, w_down, tables, y, ws);
    if (rc != EXFOLD_OK) return rc;
    const exfold_layer& l = *layer;
    if (pool_m < 1 || pool_m > l.n_experts) return EXFOLD_ERR_INVALID_ARG;
    if (B > kMaxDecodeBatch || B * l.top_k > 4096) return EXFOLD_ERR_UNSUPPORTED;
    const int N = l.n_experts, K = l.top_k, d = l.hidden, I = l.inter, G = N + l.n_shared;
    const Plan pl = make_plan(l, B, K);
    if (ws_bytes < pl.total) return EXFOLD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    const bool bf16 = l.dtype == EXFOLD_BF16;
    const int max_rows = (int)(B * K + B * l.n_shared);
    // a group has at most B rows: the token box of the GEMMs needs only that many (multiple of 32, <= 128)
    const int a_rows = (int)std::min<int64_t>(kTileM, (B + 31) / 32 * 32);

    CUtensorMap tm_wg, tm_wu, tm_h, tm_wd;
    if (bf16) {
        const uint64_t E = (uint64_t)G;
        bool ok = make_tmap(&tm_wg, w_gate, E * I, d, 128) && make_tmap(&tm_wu, w_up, E * I, d, 128) &&
                  make_tmap(&tm_h, at<char>(ws, pl.H), (uint64_t)max_rows, I, a_rows) &&
                  make_tmap(&tm_wd, w_down, E * d, I, 256);
        if (!ok) return EXFOLD_ERR_CUDA;
    }
    prof_reset();
    struct PdlScope {
        PdlScope() { set_pdl(true); }
        ~PdlScope() { set_pdl(false); }
    } pdl_scope;

    DecodeRouteParams rp{};
    rp.logits = logits; rp.S = tables->S; rp.L = tables->L; rp.h = tables->h;
    rp.B = (int)B; rp.N = N; rp.K = K; rp.M = pool_m; rp.n_shared = l.n_shared;
    if (spool != nullptr) {
        rp.st_pool = spool->pool_ids; rp.st_target = spool->target; rp.st_scale = spool->scale;
    }
    rp.pool_ids = at<int32_t>(ws, pl.pool_ids); rp.pool_size = at<int32_t>(ws, pl.pool_size);
    rp.pool_mask = at<uint32_t>(ws, pl.pool_mask); rp.ids = at<int32_t>(ws, pl.ids); rp.w = at<float>(ws, pl.w);
    rp.target = at<int32_t>(ws, pl.target); rp.scale = at<float>(ws, pl.scale);
    rp.row_tok = at<int32_t>(ws, pl.row_tok); rp.row_w = at<float>(ws, pl.row_w);
    rp.grp_expert = at<int32_t>(ws, pl.grp_expert); rp.grp_off = at<int32_t>(ws, pl.grp_off);
    rp.grp_tiles = at<int32_t>(ws, pl.grp_tiles); rp.n_groups = at<int32_t>(ws, pl.n_groups);
    rp.status = at<DeviceStatus>(ws, pl.status);
    if (bf16) {
        // Token-parallel Top-K (with the router scores when w_router is given) -> gate/up kernel that finishes the
        // routing in its prologue and streams the pool's gate and up weights against x in place -> grouped down
        // projection over the compact rows -> per-token sum of the rows.
        int stages = 0, scratch_off = 0, ar = 0;
        decode_ffn_smem_plan((int)B, K, N, &stages, &scratch_off, &ar);
        if (stages < 2) return EXFOLD_ERR_UNSUPPORTED;
        CUtensorMap tm_x, tm_wg64, tm_wu64, tm_wg96, tm_wu96;
        const uint64_t E = (uint64_t)G;
        if (!make_tmap(&tm_x, x, (uint64_t)B, d, ar) || !make_tmap(&tm_wg64, w_gate, E * I, d, 64) ||
            !make_tmap(&tm_wu64, w_up, E * I, d, 64) || !make_tmap(&tm_wg96, w_gate, E * I, d, 96) ||
            !make_tmap(&tm_wu96, w_up, E * I, d, 96))
            return EXFOLD_ERR_CUDA;
        DecodeTopkParams tp{};
        tp.logits = logits; tp.x = reinterpret_cast<const __nv_bfloat16*>(x);
        tp.w_router = reinterpret_cast<const __nv_bfloat16*>(w_router); tp.logits_out = const_cast<float*>(logits);
        tp.B = (int)B; tp.N = N; tp.K = K; tp.d = d;
        tp.ids = rp.ids; tp.w64 = at<double>(ws, pl.w64); tp.status = rp.status;
        { ProfScope ps(6, s); EXFOLD_CUDA(launch_decode_topk(tp, s)); }
        DecodeFfnParams fp{};
        fp.tm_x = tm_x; fp.tm_wg = tm_wg; fp.tm_wu = tm_wu; fp.tm_wg64 = tm_wg64; fp.tm_wu64 = tm_wu64; fp.tm_wg96 = tm_wg96; fp.tm_wu96 = tm_wu96;
        fp.ids = rp.ids; fp.w64 = tp.w64; fp.S = tables->S; fp.L = tables->L; fp.h = tables->h;
        fp.st_pool = rp.st_pool; fp.st_target = rp.st_target; fp.st_scale = rp.st_scale;
        fp.B = (int)B; fp.N = N; fp.K = K; fp.M = pool_m; fp.n_shared = l.n_shared; fp.d = d; fp.I = I; fp.a_rows = ar;
        fp.stages = stages; fp.scratch_off = scratch_off;
        fp.pool_ids = rp.pool_ids; fp.pool_size = rp.pool_size; fp.pool_mask = rp.pool_mask;
        // the remapped slots go to a second array: the Top-K ids are read by every CTA while CTA 0 writes
        fp.out_ids = at<int32_t>(ws, pl.perm); fp.out_w = rp.w; fp.target = rp.target; fp.scale = rp.scale;
        fp.H = at<__nv_bfloat16>(ws, pl.H); fp.row_tok = rp.row_tok; fp.row_w = rp.row_w;
        fp.slot_row = at<int32_t>(ws, pl.inv_pos);
        fp.grp_expert = rp.grp_expert; fp.grp_off = rp.grp_off; fp.grp_tiles = rp.grp_tiles; fp.n_groups = rp.n_groups;
        fp.status = rp.status;
        { ProfScope ps(14, s); EXFOLD_CUDA(launch_decode_ffn(fp, sm_count(), s)); }
        // Down projection on the grouped GEMM-2 kernel over the compact rows (the whole intermediate dimension is
        // its K, so no partial outputs meet in memory); each row's weighted output is stored once, in bf16, and a
        // token's rows are then summed in slot order: no atomics, so a decode step is reproducible bit for bit.
        const int max_groups = std::min(pool_m, N) + l.n_shared;
        const int tiles_per_group = (int)((B + kTileM - 1) / kTileM);
        const int sms = std::min(sm_count(), kMaxCtas);
        GroupedGemmParams g{};
        g.tm_a = tm_h; g.tm_a2 = tm_h; g.tm_b0 = tm_wd; g.tm_b1 = tm_wd; g.x_rows = 1; g.o32 = nullptr;
        g.offsets = rp.grp_off; g.work_start = rp.grp_tiles; g.G = max_groups; g.n_routed = 0x7fffffff;
        g.R = max_rows; g.d = d; g.I = I; g.n_ntiles = (d + 255) / 256; g.ksplit = 1; g.a_rows = a_rows;
        g.grp_expert = rp.grp_expert; g.n_groups_dev = rp.n_groups;
        g.H = fp.H; g.row_tok = rp.row_tok; g.row_w = rp.row_w;
        g.y = at<__nv_bfloat16>(ws, pl.obuf); g.store_rows = 1; g.status = rp.status;
        // Fewer (expert, column tile) items than half the SMs (few experts, large I): K is split in two so that
        // enough SMs stream W_down; each part's rows go to a plane of their own (the two planes are the row buffer
        // and the unused gathered-rows region before it) and are summed, in order, by the kernel after.
        const int nkb2 = I / 64;
        const int64_t base_items = (int64_t)max_groups * tiles_per_group * g.n_ntiles;
        g.ksplit = (2 * base_items < sms && nkb2 >= 8) ? kMaxDecodeKsplit : 1;
        g.y = g.ksplit > 1 ? at<__nv_bfloat16>(ws, pl.obuf) - (size_t)max_rows * d : at<__nv_bfloat16>(ws, pl.obuf);
        { ProfScope ps(9, s); EXFOLD_CUDA(launch_grouped_gemm2(g, (int)std::min<int64_t>(sms, base_items * g.ksplit), s)); }
        { ProfScope ps(5, s); EXFOLD_CUDA(launch_combine_rows(g.y, fp.slot_row, B, K, d, l.n_shared, rp.n_groups + 2, g.ksplit,
                                                       max_rows, reinterpret_cast<__nv_bfloat16*>(y), s)); }
        rp.ids = fp.out_ids;  // for the metadata copies below
    } else {
    if (w_router != nullptr) {
        rc = router_enqueue(layer, x, w_router, B, const_cast<float*>(logits), ws, ws_bytes, s, false);
        if (rc != EXFOLD_OK) return rc;
    }
    { ProfScope ps(6, s); EXFOLD_CUDA(launch_decode_route(rp, s)); }

    {
        SimtFfnParams fp{};
        fp.x = x; fp.wg = w_gate; fp.wu = w_up; fp.wd = w_down; fp.dtype = l.dtype; fp.d = d; fp.I = I;
        fp.T = B; fp.Kr = K; fp.n_shared = l.n_shared; fp.N = N; fp.ids = rp.ids; fp.out = at<float>(ws, pl.out);
        { ProfScope ps(10, s); EXFOLD_CUDA(launch_simt_ffn(fp, s)); }
        { ProfScope ps(11, s); EXFOLD_CUDA(launch_combine_routes(fp.out, rp.w, B, K, d, l.n_shared, y, l.dtype, s)); }
    }
    }
    if (meta) {
        if ((rc = copy_meta(meta->pool_ids, rp.pool_ids, (size_t)pool_m * 4, s))) return rc;
        if ((rc = copy_meta(meta->pool_size, rp.pool_size, 4, s))) return rc;
        if ((rc = copy_meta(meta->pool_mask, rp.pool_mask, (size_t)((N + 31) / 32) * 4, s))) return rc;
        if ((rc = copy_meta(meta->ids, rp.ids, (size_t)B * K * 4, s))) return rc;
        if ((rc = copy_meta(meta->w, rp.w, (size_t)B * K * 4, s))) return rc;
        if ((rc = copy_meta(meta->target, rp.target, (size_t)N * 4, s))) return rc;
        if ((rc = copy_meta(meta->scale, rp.scale, (size_t)N * 4, s))) return rc;
    }
    return EXFOLD_OK;
}

int exfold_moe_decode(const exfold_layer* layer, const void* x, const float* logits, int64_t B, const void* w_gate,
                      const void* w_up, const void* w_down, const exfold_tables* tables, int32_t pool_m, void* y,
                      const exfold_decode_meta* meta, void* ws, size_t ws_bytes, void* cuda_stream) {
    return decode_impl(layer, x, logits, B, w_gate, w_up, w_down, tables, nullptr, pool_m, y, meta, ws, ws_bytes,
                       cuda_stream);
}

int exfold_moe_decode_static(const exfold_layer* layer, const void* x, const float* logits, int64_t B,
                             const void* w_gate, const void* w_up, const void* w_down, const exfold_static_pool* pool,
                             void* y, const exfold_decode_meta* meta, void* ws, size_t ws_bytes, void* cuda_stream) {
    if (pool == nullptr) return EXFOLD_ERR_INVALID_ARG;
    return decode_impl(layer, x, logits, B, w_gate, w_up, w_down, nullptr, pool, pool->pool_m, y, meta, ws, ws_bytes,
                       cuda_stream);
}

int exfold_static_pool_build(const exfold_layer* layer, const exfold_tables* tables, int32_t pool_m,
                             exfold_static_pool* out, void* cuda_stream) {
    if (!valid_layer(layer) || !tables || !tables->S || !tables->L || !tables->h || !out) return EXFOLD_ERR_INVALID_ARG;
    if (!out->pool_ids || !out->target || !out->scale) return EXFOLD_ERR_INVALID_ARG;
    if (pool_m < 1 || pool_m > layer->n_experts) return EXFOLD_ERR_INVALID_ARG;
    out->pool_m = pool_m;
    EXFOLD_CUDA(launch_static_pool(layer->n_experts, pool_m, tables->S, tables->L, tables->h, out->pool_ids,
                                   out->target, out->scale, reinterpret_cast<cudaStream_t>(cuda_stream)));
    return EXFOLD_OK;
}

// Enqueues one calibration on the stream (no synchronisation); the number of unobserved experts lands in
// warn_slot (device memory) when the stream gets there.
static int calibrate_enqueue(const exfold_layer* layer, const void* x_cal, const float* logits_cal, int64_t m,
                             const void* w_gate, const void* w_up, const void* w_down, const exfold_calib_opts* opts,
                             exfold_tables* out, void* ws, size_t ws_bytes, void* cuda_stream, int job) {
    if (!valid_layer(layer) || !x_cal || !w_gate || !w_up || !w_down || !opts || !out || !ws)
        return EXFOLD_ERR_INVALID_ARG;
    if (!out->S || !out->L || !out->h || !out->lnh) return EXFOLD_ERR_INVALID_ARG;
    if (m < 1 || m > (int64_t)1 << 22) return EXFOLD_ERR_INVALID_ARG;
    if (opts->mode != 0 && opts->mode != 1) return EXFOLD_ERR_INVALID_ARG;
    if (opts->mode == 0 && !logits_cal) return EXFOLD_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ws) & 255) != 0) return EXFOLD_ERR_INVALID_ARG;
    const exfold_layer& l = *layer;
    const int N = l.n_experts, K = l.top_k, d = l.hidden, I = l.inter;
    const int Ke = opts->mode == 1 ? N : K;
    exfold_layer lc = l;
    lc.n_shared = 0;  // the shared expert is never folded, so it is not calibrated
    const Plan pl = make_plan(lc, m, Ke);
    if (ws_bytes < pl.total) return EXFOLD_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);

    EXFOLD_CUDA(cudaMemsetAsync(at<char>(ws, pl.status), 0, sizeof(DeviceStatus), s));
    int32_t* ids = at<int32_t>(ws, pl.ids);
    if (opts->mode == 0) {
        // Top-K in router order: the prefill route kernel with K' = K and a zero ln(h) table
        EXFOLD_CUDA(cudaMemsetAsync(at<char>(ws, pl.zeros), 0, (size_t)N * 4, s));
        PrefillRouteParams rp{};
        rp.logits = logits_cal; rp.S = out->S; rp.L = out->L; rp.lnh = at<float>(ws, pl.zeros);
        rp.T = m; rp.N = N; rp.K = K; rp.Kp = K; rp.ids = ids; rp.w = at<float>(ws, pl.w);
        rp.loss_thr = INFINITY;
        rp.omit_src = nullptr; rp.omit_tgt = nullptr; rp.block_hist = at<int32_t>(ws, pl.block_hist);
        rp.sb_hist = at<int32_t>(ws, pl.sb_hist);
        rp.status = nullptr;
        EXFOLD_CUDA(launch_prefill_route(rp, s));
    } else {
        EXFOLD_CUDA(launch_iota_ids(ids, m, N, s));
    }
    const bool tensor_path = l.dtype == EXFOLD_BF16;
    if (tensor_path && (!aligned16(x_cal) || !aligned16(w_gate) || !aligned16(w_up) || !aligned16(w_down)))
        return EXFOLD_ERR_INVALID_ARG;
    const int64_t Rc = m * Ke;
    if (tensor_path && Rc > (int64_t)1 << 30) return EXFOLD_ERR_UNSUPPORTED;
    CalibStatsParams cs{};
    if (tensor_path) {
        // Expert outputs on the tensor cores: rows sorted by expert -> GEMM-1 (SwiGLU, H in bf16) -> GEMM-2
        // with the raw fp32 accumulators stored per sorted row. Mode 0 sorts the routed rows like prefill;
        // in mode 1 every expert's rows are the tokens themselves, read from x_cal without a copy.
        CUtensorMap tm_xs, tm_x, tm_wg, tm_wu, tm_h, tm_wd;
        const uint64_t E = (uint64_t)N;
        bool ok = make_tmap(&tm_xs, at<char>(ws, pl.xs), (uint64_t)Rc, d, 128) &&
                  make_tmap(&tm_x, x_cal, (uint64_t)m, d, 128) && make_tmap(&tm_wg, w_gate, E * I, d, 128) &&
                  make_tmap(&tm_wu, w_up, E * I, d, 128) && make_tmap(&tm_h, at<char>(ws, pl.H), (uint64_t)Rc, I, 128) &&
                  make_tmap(&tm_wd, w_down, E * d, I, 256);
        if (!ok) return EXFOLD_ERR_CUDA;
        int32_t* offsets = at<int32_t>(ws, pl.offsets);
        int32_t* work_start = at<int32_t>(ws, pl.work_start);
        if (opts->mode == 0) {
            PrefillScatterParams cp{};
            cp.T = m; cp.N = N; cp.n_shared = 0; cp.Kp = K; cp.d_bytes = d * 2;
            cp.nblk = (int)((m + kRouteTokensPerBlock - 1) / kRouteTokensPerBlock);
            cp.ids = ids; cp.w = at<float>(ws, pl.w); cp.block_hist = at<int32_t>(ws, pl.block_hist);
            cp.sb_hist = at<int32_t>(ws, pl.sb_hist);
            cp.offsets = offsets; cp.work_start = work_start;
            cp.x = x_cal; cp.xs = at<char>(ws, pl.xs);
            cp.perm = at<int32_t>(ws, pl.perm); cp.row_tok = at<int32_t>(ws, pl.row_tok);
            cp.row_w = at<float>(ws, pl.row_w); cp.row_exp = at<int32_t>(ws, pl.row_exp);
            cp.inv_pos = at<int32_t>(ws, pl.inv_pos);
            EXFOLD_CUDA(launch_prefill_scatter(cp, s));
            cs.inv_pos = cp.inv_pos;
        } else {
            EXFOLD_CUDA(launch_calib_common_rows(offsets, work_start, m, N, s));
            cs.inv_pos = nullptr; cs.tok_stride = 1; cs.slot_stride = m;
        }
        GroupedGemmParams g{};
        g.tm_a = tm_xs; g.tm_a2 = tm_x; g.tm_b0 = tm_wg; g.tm_b1 = tm_wu;
        g.offsets = offsets; g.work_start = work_start; g.G = N;
        g.n_routed = opts->mode == 0 ? N : 0;  // mode 1: every group reads x_cal directly
        g.R = 0; g.x_rows = (int)m;
        g.d = d; g.I = I; g.n_ntiles = (I + 127) / 128; g.ksplit = 1; g.a_rows = kTileM;
        g.H = at<__nv_bfloat16>(ws, pl.H); g.row_tok = at<int32_t>(ws, pl.row_tok); g.row_w = at<float>(ws, pl.row_w);
        g.status = at<DeviceStatus>(ws, pl.status);
        const int64_t max_tiles = Rc / kTileM + N;
        EXFOLD_CUDA(launch_grouped_gemm1(g, (int)std::min<int64_t>(sm_count(), max_tiles * g.n_ntiles), s));
        g.tm_a = tm_h; g.tm_b0 = tm_wd; g.n_ntiles = (d + 255) / 256;
        g.o32 = at<float>(ws, pl.xs);  // spans the xs and obuf regions (GEMM-1 is done with xs)
        EXFOLD_CUDA(launch_grouped_gemm2(g, (int)std::min<int64_t>(sm_count(), max_tiles * g.n_ntiles), s));
        cs.out = g.o32;
    } else {
        SimtFfnParams fp{};
        fp.x = x_cal; fp.wg = w_gate; fp.wu = w_up; fp.wd = w_down; fp.dtype = l.dtype; fp.d = d; fp.I = I;
        fp.T = m; fp.Kr = Ke; fp.n_shared = 0; fp.N = N; fp.ids = ids; fp.out = at<float>(ws, pl.out);
        EXFOLD_CUDA(launch_simt_ffn(fp, s));
        cs.out = fp.out; cs.inv_pos = nullptr; cs.tok_stride = Ke; cs.slot_stride = 1;
    }

    char* cb = at<char>(ws, pl.calib);
    const size_t NN = (size_t)N * N;
    EXFOLD_CUDA(cudaMemsetAsync(cb, 0, NN * (3 * 8 + 4) + (size_t)N * (8 + 4) + 256, s));
    cs.ids = ids; cs.m = m; cs.Ke = Ke; cs.d = d; cs.N = N;
    cs.A = reinterpret_cast<double*>(cb); cs.Bv = cs.A + NN; cs.C = cs.Bv + NN;
    cs.H = cs.C + NN;
    cs.cnt = reinterpret_cast<int32_t*>(cs.H + N);
    cs.hc = cs.cnt + NN;
    int32_t* unobs = cs.hc + N;
    if (opts->mode == 1 && Ke >= 32)  // many experts per token: Gram-product form of the same sums
        EXFOLD_CUDA(launch_calib_stats_common(cs, at<double>(ws, pl.calib_nrm), sm_count(), s));
    else
        EXFOLD_CUDA(launch_calib_stats(cs, s));
    EXFOLD_CUDA(launch_calib_finalize(cs, *opts, out->S, out->L, out->h, out->lnh, out->n_obs, unobs, s));
    EXFOLD_CUDA(cudaMemcpyAsync(at<int32_t>(ws, pl.calib_warn) + job, unobs, 4, cudaMemcpyDeviceToDevice, s));
    return EXFOLD_OK;
}

// The jobs' unobserved-expert counts, after the stream has drained
static int calibrate_collect(const exfold_layer* layer, int64_t m_max, int Ke, int n_jobs, int32_t* warn, void* ws,
                             cudaStream_t s) {
    exfold_layer lc = *layer;
    lc.n_shared = 0;
    const Plan pl = make_plan(lc, m_max, Ke);
    int32_t un[EXFOLD_MAX_CALIB_JOBS];
    EXFOLD_CUDA(cudaMemcpyAsync(un, at<int32_t>(ws, pl.calib_warn), (size_t)n_jobs * 4, cudaMemcpyDeviceToHost, s));
    EXFOLD_CUDA(cudaStreamSynchronize(s));
    int any = 0;
    for (int j = 0; j < n_jobs; ++j) {
        if (warn) warn[j] = un[j];
        any |= un[j] > 0;
    }
    return any ? EXFOLD_WARN_UNOBSERVED_EXPERT : EXFOLD_OK;
}

int exfold_calibrate(const exfold_layer* layer, const void* x_cal, const float* logits_cal, int64_t m,
                     const void* w_gate, const void* w_up, const void* w_down, const exfold_calib_opts* opts,
                     exfold_tables* out, void* ws, size_t ws_bytes, void* cuda_stream) {
    int rc = calibrate_enqueue(layer, x_cal, logits_cal, m, w_gate, w_up, w_down, opts, out, ws, ws_bytes, cuda_stream, 0);
    if (rc != EXFOLD_OK) return rc;
    return calibrate_collect(layer, m, opts->mode == 1 ? layer->n_experts : layer->top_k, 1, nullptr, ws,
                             reinterpret_cast<cudaStream_t>(cuda_stream));
}

int exfold_calibrate_layers(const exfold_layer* layer, const exfold_calib_job* jobs, int32_t n_jobs,
                            const exfold_calib_opts* opts, int32_t* unobserved, void* ws, size_t ws_bytes,
                            void* cuda_stream) {
    if (!valid_layer(layer) || !jobs || !opts || n_jobs < 1 || n_jobs > EXFOLD_MAX_CALIB_JOBS) return EXFOLD_ERR_INVALID_ARG;
    if (opts->mode != 0 && opts->mode != 1) return EXFOLD_ERR_INVALID_ARG;
    int64_t m_max = 0;
    for (int j = 0; j < n_jobs; ++j) {
        if (!jobs[j].out || jobs[j].m < 1) return EXFOLD_ERR_INVALID_ARG;
        m_max = std::max<int64_t>(m_max, jobs[j].m);
    }
    // Every job uses the plan of the largest one, so that the jobs' warning slots sit at one place; the jobs run
    // one after the other on the stream and share the rest of the workspace.
    const int Ke = opts->mode == 1 ? layer->n_experts : layer->top_k;
    if (ws_bytes < exfold_workspace_bytes(layer, m_max, Ke)) return EXFOLD_ERR_WORKSPACE_TOO_SMALL;
    for (int j = 0; j < n_jobs; ++j) {
        const exfold_calib_job& b = jobs[j];
        int rc = calibrate_enqueue(layer, b.x_cal, b.logits_cal, b.m, b.w_gate, b.w_up, b.w_down, opts, b.out, ws,
                                   ws_bytes, cuda_stream, j);
        if (rc != EXFOLD_OK) return rc;
    }
    return calibrate_collect(layer, m_max, Ke, n_jobs, unobserved, ws, reinterpret_cast<cudaStream_t>(cuda_stream));
}

// Router scores on the stream; `clear_status`: the call stands alone (clears the status record itself)
static int router_enqueue(const exfold_layer* layer, const void* x, const void* w_router, int64_t T, float* logits,
                          void* ws, size_t ws_bytes, cudaStream_t s, bool clear_status) {
    if (!valid_layer(layer) || !x || !w_router || !logits || !ws || T < 1) return EXFOLD_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(ws) & 255) != 0 || (reinterpret_cast<uintptr_t>(logits) & 15) != 0)
        return EXFOLD_ERR_INVALID_ARG;
    const exfold_layer& l = *layer;
    const int N = l.n_experts, d = l.hidden;
    if (T > (int64_t)1 << 30) return EXFOLD_ERR_UNSUPPORTED;
    exfold_layer lc = l;
    lc.n_shared = 0;
    const Plan pl = make_plan(lc, T, 1);
    if (ws_bytes < pl.total) return EXFOLD_ERR_WORKSPACE_TOO_SMALL;
    if (clear_status) EXFOLD_CUDA(cudaMemsetAsync(at<char>(ws, pl.status), 0, sizeof(DeviceStatus), s));
    // fp32 layers, and bf16 batches of at most one row tile (decode): dot products in a fixed order. One 128-row
    // tile on the tensor cores would walk the whole K loop on a single SM (10-19 us of latency).
    if (l.dtype == EXFOLD_F32 || (T <= kTileM && aligned16(x) && aligned16(w_router))) {
        EXFOLD_CUDA(launch_router_simt(x, w_router, l.dtype, T, N, d, logits, s));
        return EXFOLD_OK;
    }
    // bf16: one group of T rows through GEMM-2's instantiation of the grouped kernel (K = d, N output columns in
    // one 256-column tile, raw fp32 row epilogue); W_r rows past N are zero-filled by the tensor map
    if (!aligned16(x) || !aligned16(w_router)) return EXFOLD_ERR_INVALID_ARG;
    CUtensorMap tm_x, tm_wr;
    if (!make_tmap(&tm_x, x, (uint64_t)T, d, 128) || !make_tmap(&tm_wr, w_router, (uint64_t)N, d, 256))
        return EXFOLD_ERR_CUDA;
    GroupedGemmParams g{};
    g.tm_a = tm_x; g.tm_a2 = tm_x; g.tm_b0 = tm_wr; g.tm_b1 = tm_wr;
    g.offsets = nullptr; g.work_start = nullptr; g.G = 1;  // one group of R = T rows
    g.n_routed = 1; g.R = (int)T; g.x_rows = (int)T;
    g.d = N;   // output width
    g.I = d;   // contraction length
    g.n_ntiles = 1; g.ksplit = 1; g.a_rows = kTileM;
    g.row_tok = at<int32_t>(ws, pl.row_tok); g.row_w = at<float>(ws, pl.row_w);  // read, not used, by this epilogue
    g.o32 = logits; g.status = at<DeviceStatus>(ws, pl.status);
    const int64_t tiles = (T + kTileM - 1) / kTileM;
    EXFOLD_CUDA(launch_grouped_gemm2(g, (int)std::min<int64_t>(sm_count(), tiles), s));
    return EXFOLD_OK;
}

int exfold_router_logits(const exfold_layer* layer, const void* x, const void* w_router, int64_t T, float* logits,
                         void* ws, size_t ws_bytes, void* cuda_stream) {
    return router_enqueue(layer, x, w_router, T, logits, ws, ws_bytes, reinterpret_cast<cudaStream_t>(cuda_stream),
                          true);
}

int exfold_moe_prefill_layer(const exfold_layer* layer, const void* x, const void* w_router, int64_t T,
                             const void* w_gate, const void* w_up, const void* w_down, const exfold_tables* tables,
                             int32_t k_pre, float* logits, void* y, const exfold_prefill_meta* meta, void* ws,
                             size_t ws_bytes, void* cuda_stream) {
    if (!valid_layer(layer) || k_pre < 1 || k_pre > layer->top_k) return EXFOLD_ERR_INVALID_ARG;
    if (ws_bytes < exfold_workspace_bytes(layer, T < 1 ? 1 : T, k_pre)) return EXFOLD_ERR_WORKSPACE_TOO_SMALL;
    int rc = router_enqueue(layer, x, w_router, T, logits, ws, ws_bytes, reinterpret_cast<cudaStream_t>(cuda_stream),
                            true);
    if (rc != EXFOLD_OK) return rc;
    // the routing kernel would clear the status record again: an error of the router GEMM must stay visible
    t_keep_status = true;
    rc = exfold_moe_prefill(layer, x, logits, T, w_gate, w_up, w_down, tables, k_pre, y, meta, ws, ws_bytes, cuda_stream);
    t_keep_status = false;
    return rc;
}

int exfold_moe_decode_layer(const exfold_layer* layer, const void* x, const void* w_router, int64_t B,
                            const void* w_gate, const void* w_up, const void* w_down, const exfold_tables* tables,
                            int32_t pool_m, float* logits, void* y, const exfold_decode_meta* meta, void* ws,
                            size_t ws_bytes, void* cuda_stream) {
    if (!valid_layer(layer) || !w_router || !logits) return EXFOLD_ERR_INVALID_ARG;
    if (B < 1 || B > kMaxDecodeBatch) return B < 1 ? EXFOLD_ERR_INVALID_ARG : EXFOLD_ERR_UNSUPPORTED;
    if (ws_bytes < exfold_workspace_bytes(layer, B, layer->top_k)) return EXFOLD_ERR_WORKSPACE_TOO_SMALL;
    if ((reinterpret_cast<uintptr_t>(logits) & 15) != 0 || !aligned16(w_router)) return EXFOLD_ERR_INVALID_ARG;
    return decode_impl(layer, x, logits, B, w_gate, w_up, w_down, tables, nullptr, pool_m, y, meta, ws, ws_bytes,
                       cuda_stream, w_router);
}

int exfold_moe_prefill_host(const exfold_layer* layer, const void* x_host, const float* logits_host, int64_t T,
                            const void* w_gate, const void* w_up, const void* w_down, const exfold_tables* tables,
                            int32_t k_pre, void* y_host, const exfold_prefill_meta* meta, void* ws, size_t ws_bytes,
                            void* cuda_stream) {
    if (!valid_layer(layer) || !x_host || !logits_host || !y_host || !ws || T < 1) return EXFOLD_ERR_INVALID_ARG;
    if (k_pre < 1 || k_pre > layer->top_k) return EXFOLD_ERR_INVALID_ARG;
    const size_t main_bytes = exfold_workspace_bytes(layer, T, k_pre);
    const size_t el = layer->dtype == EXFOLD_BF16 ? 2 : 4;
    const size_t xb = (size_t)T * layer->hidden * el, lb = (size_t)T * layer->n_experts * 4;
    if (ws_bytes < main_bytes + exfold_host_staging_bytes(layer, T)) return EXFOLD_ERR_WORKSPACE_TOO_SMALL;
    char* stage = reinterpret_cast<char*>(ws) + main_bytes;
    char* xd = stage;
    char* yd = xd + align_up(xb, 256);
    char* ld = yd + align_up(xb, 256);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    // Tokens are independent, so a long prompt goes through in chunks: chunk c+1 is copied in and chunk c-1 copied
    // out (two helper streams, both PCIe directions) while chunk c is computed on the caller's stream. Routing
    // metadata describes the whole call (one permutation over all routes), so a call that asks for it is not split.
    const int64_t chunk_tokens = 2048;
    int chunks = meta != nullptr ? 1 : (int)std::min<int64_t>(kMaxHostChunks, T / chunk_tokens);
    // a chunk of at least 12 row tiles still runs its whole tile pairs on the CTA-pair kernel
    const int64_t chunk_rows = chunks > 1 ? (T / chunks) * (k_pre + layer->n_shared) : 0;
    exfold_fold_opts chunk_opts{INFINITY, 0, 0, chunk_rows >= 12 * kTileM ? 2 : 0};
    if (chunks <= 1) {
        EXFOLD_CUDA(cudaMemcpyAsync(xd, x_host, xb, cudaMemcpyHostToDevice, s));
        EXFOLD_CUDA(cudaMemcpyAsync(ld, logits_host, lb, cudaMemcpyHostToDevice, s));
        int rc = exfold_moe_prefill(layer, xd, reinterpret_cast<const float*>(ld), T, w_gate, w_up, w_down, tables,
                                    k_pre, yd, meta, ws, main_bytes, cuda_stream);
        if (rc != EXFOLD_OK) return rc;
        EXFOLD_CUDA(cudaMemcpyAsync(y_host, yd, xb, cudaMemcpyDeviceToHost, s));
        return EXFOLD_OK;
    }
    ThreadDeviceState* hp = host_helpers();  // created once per host thread and device
    if (!hp) return EXFOLD_ERR_CUDA;
    ThreadDeviceState& h = *hp;
    // the staging buffers may still be in use by earlier work on the caller's stream
    EXFOLD_CUDA(cudaEventRecord(h.start, s));
    EXFOLD_CUDA(cudaStreamWaitEvent(h.in, h.start, 0));
    EXFOLD_CUDA(cudaStreamWaitEvent(h.out, h.start, 0));
    const size_t row_x = (size_t)layer->hidden * el, row_l = (size_t)layer->n_experts * 4;
    const int64_t per = (T / chunks + 127) / 128 * 128;  // whole row tiles per chunk
    for (int c = 0; c < chunks; ++c) {
        const int64_t t0 = c * per, n = std::min<int64_t>(per, T - t0);
        if (n <= 0) break;
        EXFOLD_CUDA(cudaMemcpyAsync(xd + t0 * row_x, reinterpret_cast<const char*>(x_host) + t0 * row_x, n * row_x,
                                    cudaMemcpyHostToDevice, h.in));
        EXFOLD_CUDA(cudaMemcpyAsync(ld + t0 * row_l, reinterpret_cast<const char*>(logits_host) + t0 * row_l,
                                    n * row_l, cudaMemcpyHostToDevice, h.in));
        EXFOLD_CUDA(cudaEventRecord(h.copied[c], h.in));
    }
    for (int c = 0; c < chunks; ++c) {
        const int64_t t0 = c * per, n = std::min<int64_t>(per, T - t0);
        if (n <= 0) break;
        EXFOLD_CUDA(cudaStreamWaitEvent(s, h.copied[c], 0));
        t_keep_status = c > 0;  // an error recorded by an earlier chunk stays visible
        int rc = exfold_moe_prefill_ex(layer, xd + t0 * row_x, reinterpret_cast<const float*>(ld + t0 * row_l), n, w_gate,
                                       w_up, w_down, tables, k_pre, &chunk_opts, yd + t0 * row_x, nullptr, ws, main_bytes,
                                       cuda_stream);
        t_keep_status = false;
        if (rc != EXFOLD_OK) return rc;
        EXFOLD_CUDA(cudaEventRecord(h.computed[c], s));
        EXFOLD_CUDA(cudaStreamWaitEvent(h.out, h.computed[c], 0));
        EXFOLD_CUDA(cudaMemcpyAsync(reinterpret_cast<char*>(y_host) + t0 * row_x, yd + t0 * row_x, n * row_x,
                                    cudaMemcpyDeviceToHost, h.out));
    }
    EXFOLD_CUDA(cudaEventRecord(h.done, h.out));
    EXFOLD_CUDA(cudaStreamWaitEvent(s, h.done, 0));  // the call is complete, in the caller's stream order, when y_host is
    return EXFOLD_OK;
}

int exfold_moe_decode_host(const exfold_layer* layer, const void* x_host, const float* logits_host, int64_t B,
                           const void* w_gate, const void* w_up, const void* w_down, const exfold_tables* tables,
                           int32_t pool_m, void* y_host, const exfold_decode_meta* meta, void* ws, size_t ws_bytes,
                           void* cuda_stream) {
    if (!valid_layer(layer) || !x_host || !logits_host || !y_host || !ws || B < 1) return EXFOLD_ERR_INVALID_ARG;
    const size_t main_bytes = exfold_workspace_bytes(layer, B, layer->top_k);
    const size_t el = layer->dtype == EXFOLD_BF16 ? 2 : 4;
    const size_t xb = (size_t)B * layer->hidden * el, lb = (size_t)B * layer->n_experts * 4;
    if (ws_bytes < main_bytes + exfold_host_staging_bytes(layer, B)) return EXFOLD_ERR_WORKSPACE_TOO_SMALL;
    char* stage = reinterpret_cast<char*>(ws) + main_bytes;
    char* xd = stage;
    char* yd = xd + align_up(xb, 256);
    char* ld = yd + align_up(xb, 256);
    cudaStream_t s = reinterpret_cast<cudaStream_t>(cuda_stream);
    EXFOLD_CUDA(cudaMemcpyAsync(xd, x_host, xb, cudaMemcpyHostToDevice, s));
    EXFOLD_CUDA(cudaMemcpyAsync(ld, logits_host, lb, cudaMemcpyHostToDevice, s));
    int rc = exfold_moe_decode(layer, xd, reinterpret_cast<const float*>(ld), B, w_gate, w_up, w_down, tables, pool_m,
                               yd, meta, ws, main_bytes, cuda_stream);
    if (rc != EXFOLD_OK) return rc;
    EXFOLD_CUDA(cudaMemcpyAsync(y_host, yd, xb, cudaMemcpyDeviceToHost, s));
    return EXFOLD_OK;
}

}  // extern "C"
