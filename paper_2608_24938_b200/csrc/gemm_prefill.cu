// Prefill expert FFN as two grouped GEMMs on the 5th-generation tensor cores (Eq. 1, 3, 4).
//
//   GEMM-1  H[r, :] = silu(X_r W_gate^T) * (X_r W_up^T)     rows r sorted by expert
//   GEMM-2  y[tok(r), :] += w~(r) * (H[r, :] W_down^T)       weighted scatter-combine
//
// One persistent CTA per SM, 6 warps: warp 0 issues TMA loads (operands land in shared memory
// with the 128-byte swizzle), warp 1 issues tcgen05.mma (one thread) into TMEM, warps 2-5 drain
// the accumulators with tcgen05.ld and run the fused epilogue. Shared-memory stages and the two
// TMEM accumulator stages are handed around with mbarriers, so the epilogue of one tile
// overlaps the main loop of the next.
//
// Tile = 128 sorted rows x 256 accumulator columns (GEMM-1: 128 gate + 128 up columns of the
// same output features; GEMM-2: 256 output features). Work items are ordered expert-major,
// then column tile, then row tile, so the CTAs running at the same time share one weight tile
// through L2 and stream each expert's weights from HBM once. Rows past the end of an expert's
// group are computed and masked, never padded in memory.
#include <algorithm>

#include "common.cuh"
#include "ptx.cuh"

namespace exfold {

namespace {

constexpr int kBK = kGemmBK;                  // K elements per stage: one swizzle row (128 or 64 bytes)
#ifndef EXFOLD_STAGES
#define EXFOLD_STAGES (EXFOLD_BK == 64 ? 4 : 9)
#endif
constexpr int kStages = EXFOLD_STAGES;
constexpr int kMaxStages = kBK == 64 ? 6 : 12;  // decode loads a shorter A box per stage and fits more stages
constexpr int kATileBytes = kTileM * kBK * 2;  // 16 KB
constexpr int kBTileBytes = 256 * kBK * 2;     // 32 KB
constexpr int kStageBytes = kATileBytes + kBTileBytes;
constexpr int kGemmSmem = kStages * kStageBytes + 1024;
#ifndef EXFOLD_PRODUCERS
#define EXFOLD_PRODUCERS (EXFOLD_BK == 64 ? 2 : 3)
#endif
// One thread's loop {wait for the stage, expect_tx, 2-3 TMA issues} takes ~600-700 cycles: longer than the 512
// cycles the tensor pipe needs for a k-block. The k-blocks are therefore dealt round-robin over kProducers
// one-thread producers in warps of their own (warp 0 and the warps after the epilogue warps).
constexpr int kProducers = EXFOLD_PRODUCERS;
constexpr int kGemmThreads = 192 + 32 * (kProducers - 1);
constexpr int kTmemCols = 512;

struct WorkItem {
    int g, row0, rows, n_idx, kpart, m_idx;
};

// Work index -> (group, row tile, column tile, K part). Order: group, column tile, row tile, K part
// (fastest), so CTAs running together share weight tiles through L2.
__device__ __forceinline__ WorkItem decode_work(int w_all, int G, int nt, int ks, const int* s_off, const int* s_ws,
                                                int odd_only = 0) {
    const int w = ks == 1 ? w_all : w_all / ks;
    int lo = 0, hi = G;  // find g with s_ws[g]*nt <= w < s_ws[g+1]*nt
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (s_ws[mid] * nt <= w) lo = mid;
        else hi = mid;
    }
    // skip empty groups that share the same start
    while (lo + 1 < G && s_ws[lo + 1] * nt <= w) ++lo;
    WorkItem it;
    it.g = lo;
    it.kpart = w_all - w * ks;
    const int tiles = s_ws[lo + 1] - s_ws[lo];
    const int local = w - s_ws[lo] * nt;
    const int m_idx = local % tiles;
    it.m_idx = m_idx;
    it.n_idx = local / tiles;
    // odd_only: the group's one item is its LAST row tile (the tiles before it ran two at a time on CTA pairs)
    const int first = odd_only ? (s_off[lo + 1] - s_off[lo] - 1) / kTileM : 0;
    it.row0 = s_off[lo] + (first + m_idx) * kTileM;
    const int left = s_off[lo + 1] - it.row0;
    it.rows = left < kTileM ? left : kTileM;
    return it;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}

// MODE 0: gate/up + SwiGLU -> H; MODE 1: down + weighted scatter -> y.
// DEC (decode) adds what only the expert-pool path needs: a group -> expert map, a group count that is
// known only on the device, and split-K for GEMM-2. The prefill instantiations compile all of it away.
template <int MODE, bool DEC>
__global__ void __launch_bounds__(kGemmThreads, 1) grouped_gemm_kernel(const __grid_constant__ GroupedGemmParams p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t tfull_bar[2];
    __shared__ __align__(8) uint64_t tempty_bar[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int s_off[kMaxGroups + 1];
    __shared__ int s_ws[kMaxGroups + 1];
    __shared__ int s_exp[kMaxGroups + 1];
    __shared__ int s_n_pairs;  // odd-tile pass: whole pairs of row tiles over all groups (the other pass's work)

    unsigned char* tiles =
        reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // ---- prologue that does not depend on earlier kernels: overlaps their tail under programmatic launch
    if (threadIdx.x == 0) {
        ptx::prefetch_tmap(&p.tm_a);
        ptx::prefetch_tmap(&p.tm_b0);
        if (MODE == 0) {
            ptx::prefetch_tmap(&p.tm_a2);
            ptx::prefetch_tmap(&p.tm_b1);
        }
        for (int s = 0; s < kMaxStages; ++s) {
            ptx::mbar_init(&full_bar[s], 1);
            ptx::mbar_init(&empty_bar[s], 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&tfull_bar[s], 1);
            ptx::mbar_init(&tempty_bar[s], 4);
        }
        abort_s = 0;
        ptx::fence_mbar_init();
    }
    // The odd-tile pass beside the CTA-pair pass is launched over all SMs and most of its CTAs have nothing to do:
    // they must leave quickly (they queue for the few SMs of this pass), so tensor memory is allocated only once a
    // CTA knows that it has work.
    const bool late_alloc = !DEC && p.odd_only && p.sbs.odd_ctas > 0;
    if (warp == 1 && !late_alloc) {
        ptx::tmem_alloc(&tmem_base_s, kTmemCols);
        ptx::tmem_relinquish();
    }
    grid_dep_wait();  // everything below reads what the routing kernels (or GEMM-1) wrote
    int G = p.G;
    // DEC: the number of groups (pool size) is known only on the device; the tables are read up to the host's upper
    // bound in the same round trip (rows past the device's count are never used)
    const int gd = DEC ? *p.n_groups_dev : G;
    for (int i = threadIdx.x; i <= G; i += kGemmThreads) {
        // offsets == null: one group of p.R rows (a plain GEMM, e.g. the router scores)
        s_off[i] = p.offsets != nullptr ? p.offsets[i] : i * p.R;
        s_ws[i] = p.offsets != nullptr ? p.work_start[i] : i * ((p.R + kTileM - 1) / kTileM);
        if (DEC) s_exp[i] = i < G ? p.grp_expert[i] : i;  // group -> expert whose weights it uses
    }
    if (DEC) G = gd < G ? gd : G;
    ptx::tc_fence_before();
    __syncthreads();
    if (!DEC && p.odd_only) {
        // work table of the odd-tile pass: one row tile for every group whose tile count is odd
        if (warp == 0) {
            int carry = 0, pairs = 0;
            for (int g0 = 0; g0 < G; g0 += 32) {
                const int g = g0 + lane;
                int odd = 0;
                if (g < G) {
                    const int tiles = (s_off[g + 1] - s_off[g] + kTileM - 1) / kTileM;
                    odd = tiles & 1;
                    pairs += tiles >> 1;
                }
                int incl = odd;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += v;
                }
                if (g < G) s_ws[g] = carry + incl - odd;
                carry += __shfl_sync(0xffffffffu, incl, 31);
            }
            pairs = __reduce_add_sync(0xffffffffu, pairs);
            if (lane == 0) {
                s_ws[G] = carry;
                s_n_pairs = pairs;
            }
        }
        __syncthreads();
    }
    ptx::tc_fence_after();
    const int nt = p.n_ntiles;
    const int ks = (DEC && MODE == 1) ? p.ksplit : 1;  // K parts per tile (each part's rows go to a plane of their own)
    const int total = s_ws[G] * nt * ks;
    // Effective grid: with `rounds` items per CTA, ceil(total / rounds) CTAs finish together; the rest
    // stay idle instead of leaving a few CTAs one item behind (448 items on 148 SMs: 112 x 4, not
    // 144 x 3 + 4 x 4). A hundred SMs are enough to saturate HBM when the kernel is memory-bound.
    // The odd-tile pass beside the CTA-pair pass keeps only the SMs that pass leaves it (the same function of the same
    // offsets on both sides); the CTAs beyond them leave at once.
    int grid_ctas = (int)gridDim.x;
    if (late_alloc) grid_ctas = 2 * (p.sbs.n_sm_pairs - pair_pass_clusters(s_n_pairs, s_ws[G], p.sbs));
    const int rounds = grid_ctas > 0 ? (total + grid_ctas - 1) / grid_ctas : 0;
    const int eff_grid = rounds > 0 ? (total + rounds - 1) / rounds : 0;
    const int w_begin = (int)blockIdx.x < eff_grid ? (int)blockIdx.x : total;  // idle CTAs see no work
    const int w_stride = eff_grid > 0 ? eff_grid : 1;
    if (late_alloc) {
        if ((int)blockIdx.x >= eff_grid) return;  // the whole CTA: nothing allocated, nothing in flight
        if (warp == 1) {
            ptx::tmem_alloc(&tmem_base_s, kTmemCols);
            ptx::tmem_relinquish();
        }
        ptx::tc_fence_before();
        __syncthreads();
        ptx::tc_fence_after();
    }
    const uint32_t tmem_base = tmem_base_s;
    const int nkb = (MODE == 0 ? p.d : p.I) / kBK;
    const int kb_per = (nkb + ks - 1) / ks;
    // Stage geometry. Prefill: 16 KB A + 32 KB B, 4 stages (compile-time). Decode: the A box has only
    // a_rows rows (the rest of the 128-row MMA operand is whatever follows in shared memory: those
    // accumulator rows are masked), so a stage is smaller and more stages of weights are in flight.
    const int a_bytes = DEC ? p.a_rows * kBK * 2 : kATileBytes;
    const int stage_bytes = DEC ? a_bytes + kBTileBytes : kStageBytes;
    const int stages = DEC ? min(kMaxStages, (kStages * kStageBytes - (kATileBytes - a_bytes)) / stage_bytes) : kStages;
    volatile int* abort_flag = &abort_s;

    if (warp == 0 || warp >= 6) {
        // ------------------------------------------------ TMA producers (k-block c belongs to producer c % kProducers)
        if (lane == 0) {
            const int me = warp == 0 ? 0 : warp - 5;
            int stage = 0, phase = 0, turn = 0;
            bool ok = true;
            for (int w = w_begin; w < total && ok; w += w_stride) {
                const WorkItem it = decode_work(w, G, nt, ks, s_off, s_ws, DEC ? 0 : p.odd_only);
                const int kb0 = it.kpart * kb_per, kb1 = min(nkb, kb0 + kb_per);
                // per-tile constants stay in registers: the k-loop below is the latency-critical path
                const int expert = DEC ? s_exp[it.g] : it.g;
                const bool from_x = !DEC && MODE == 0 && expert >= p.n_routed;  // prefill's shared expert reads x directly
                const CUtensorMap* tma_a = from_x ? &p.tm_a2 : &p.tm_a;
                const int arow = from_x ? (it.row0 - p.R) % p.x_rows : it.row0;
                const int brow = MODE == 0 ? expert * p.I + it.n_idx * 128 : expert * p.d + it.n_idx * 256;
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (turn == me) {
                        const bool got = ptx::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, p.status, 1);
                        if (!got) {
                            ok = false;
                            break;
                        }
                        unsigned char* a_dst = tiles + stage * stage_bytes;
                        unsigned char* b_dst = a_dst + a_bytes;
                        ptx::mbar_expect_tx(&full_bar[stage], stage_bytes);
                        ptx::tma_load_2d(a_dst, tma_a, &full_bar[stage], kb * kBK, arow);
                        ptx::tma_load_2d(b_dst, &p.tm_b0, &full_bar[stage], kb * kBK, brow);
                        if (MODE == 0) ptx::tma_load_2d(b_dst + 128 * kBK * 2, &p.tm_b1, &full_bar[stage], kb * kBK, brow);
                    }
                    if (++turn == kProducers) turn = 0;
                    if (++stage == stages) {
                        stage = 0;
                        phase ^= 1;
                    }
                }
            }
            if (me == 0) {
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::make_idesc_bf16(128, 256);
            int stage = 0, phase = 0, iter = 0;
            // This one thread's instruction stream paces the tensor pipe (a k-block is 4 MMAs = 512 pipe cycles),
            // so the loop carries as little as possible: the descriptors' low words advance by a constant per stage
            // (the high word never changes), and the readiness of the NEXT stage is polled before this stage's MMAs
            // are issued, so that the poll's round trip overlaps them.
            const uint32_t lo0 = (ptx::smem_u32(tiles) & 0x3FFFFu) >> 4;
            const uint32_t lo_step = (uint32_t)stage_bytes >> 4, lo_b = (uint32_t)a_bytes >> 4;
            const uint32_t desc_hi32 = (uint32_t)(ptx::make_kmajor_sw128_desc(0) >> 32);
            uint32_t a_lo = lo0;
            bool ok = true;
            bool ready = false;
            for (int w = w_begin; w < total && ok; w += w_stride, ++iter) {
                const int as = iter & 1, aphase = (iter >> 1) & 1;
                const bool got = ptx::mbar_wait(&tempty_bar[as], aphase ^ 1, abort_flag, p.status, 2);
                if (!got) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + as * 256;
                const int kpart = ks == 1 ? 0 : w % ks;
                const int kb0 = kpart * kb_per, kb1 = min(nkb, kb0 + kb_per);
                if constexpr (!DEC && kStages == 4) {
                    // Prefill: the k-loop is written out once per ring stage (switch into the stage the ring stands
                    // at), so a k-block costs this thread the MMA sequence, one compare and one branch.
                    int kb = kb0;
#define EXFOLD_KBLOCK(S)                                                                                            \
    {                                                                                                                \
        constexpr int NS = (S) + 1 == kStages ? 0 : (S) + 1;                                                         \
        const uint32_t nphase = NS == 0 ? phase ^ 1 : phase;                                                         \
        if (!ready && !ptx::mbar_wait(&full_bar[S], phase, abort_flag, p.status, 3)) {                               \
            ok = false;                                                                                              \
            break;                                                                                                   \
        }                                                                                                            \
        constexpr uint32_t step = (uint32_t)kStageBytes >> 4, off_b = (uint32_t)kATileBytes >> 4;                    \
        ready = ptx::umma_kblock_bf16(d_tmem, lo0 + (S) * step, lo0 + (S) * step + off_b, desc_hi32, idesc,         \
                                      kb > kb0 ? 1u : 0u, &empty_bar[S], &full_bar[NS], nphase);                     \
        if (NS == 0) phase ^= 1;                                                                                     \
        if (++kb == kb1) {                                                                                           \
            stage = NS;                                                                                              \
            break;                                                                                                   \
        }                                                                                                            \
    }
                    while (ok && kb < kb1) {
                        switch (stage) {
                            case 0: EXFOLD_KBLOCK(0)
                            case 1: EXFOLD_KBLOCK(1)
                            case 2: EXFOLD_KBLOCK(2)
                            default: EXFOLD_KBLOCK(3)
                        }
                        if (kb < kb1) stage = 0;  // fell through the last stage: the ring wraps
                    }
#undef EXFOLD_KBLOCK
                } else {
                    for (int kb = kb0; kb < kb1; ++kb) {
                        if (!ready) {
                            if (!ptx::mbar_wait(&full_bar[stage], phase, abort_flag, p.status, 3)) {
                                ok = false;
                                break;
                            }
                        }
                        const int ns = stage + 1 == stages ? 0 : stage + 1;
                        const int nphase = ns == 0 ? phase ^ 1 : phase;
                        ready = ptx::umma_kblock_bf16(d_tmem, a_lo, a_lo + lo_b, desc_hi32, idesc, kb > kb0 ? 1u : 0u,
                                                      &empty_bar[stage], &full_bar[ns], nphase);
                        a_lo = ns == 0 ? lo0 : a_lo + lo_step;
                        stage = ns;
                        phase = nphase;
                    }
                }
                if (ok) ptx::umma_commit(&tfull_bar[as]);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue warps (TMEM lane quadrant = warp % 4)
        const int q = warp & 3;
        int iter = 0;
        for (int w = w_begin; w < total; w += w_stride, ++iter) {
            const int as = iter & 1, aphase = (iter >> 1) & 1;
            const WorkItem it = decode_work(w, G, nt, ks, s_off, s_ws, DEC ? 0 : p.odd_only);
            const int row = q * 32 + lane;
            const bool valid = row < it.rows && it.kpart * kb_per < nkb;  // a K part without k-blocks adds nothing
            const int64_t grow = (int64_t)it.row0 + row;
            int tok = 0;  // GEMM-2: the row's token and weight, asked for before the wait for the accumulator
            float wv = 0.f;
            if (MODE == 1 && valid) {
                tok = p.row_tok[grow];
                wv = p.row_w[grow];
            }
            // lane 0 waits; the warp takes one decision, so the warp-wide TMEM loads below stay convergent
            int ok = 1;
            if (lane == 0) {
                const bool got = ptx::mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status, 4);
                ok = got ? 1 : 0;
            }
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            ptx::tc_fence_after();
            const uint32_t taddr = tmem_base + as * 256 + ((uint32_t)(q * 32) << 16);
            if (MODE == 0) {
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t gv[32], uv[32];
                    ptx::tmem_ld32(taddr + c * 32, gv);
                    ptx::tmem_ld32(taddr + 128 + c * 32, uv);
                    ptx::tmem_ld_wait();
                    const int col0 = it.n_idx * 128 + c * 32;
                    if (valid && col0 < p.I) {
                        uint32_t pk[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            float g0 = __uint_as_float(gv[2 * j]), g1 = __uint_as_float(gv[2 * j + 1]);
                            float u0 = __uint_as_float(uv[2 * j]), u1 = __uint_as_float(uv[2 * j + 1]);
                            float h0 = __fdividef(g0, 1.0f + __expf(-g0)) * u0;
                            float h1 = __fdividef(g1, 1.0f + __expf(-g1)) * u1;
                            pk[j] = pack_bf16(h0, h1);
                        }
                        uint4* dst = reinterpret_cast<uint4*>(p.H + grow * p.I + col0);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            dst[j] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                    }
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < 8; ++c) {
                    uint32_t v[32];
                    ptx::tmem_ld32(taddr + c * 32, v);
                    ptx::tmem_ld_wait();
                    const int col0 = it.n_idx * 256 + c * 32;
                    if (valid && col0 < p.d) {
                        if (!DEC && p.o32 != nullptr) {  // raw fp32 rows (calibration outputs, router scores)
                            float* dstf = p.o32 + grow * p.d + col0;
                            if (col0 + 32 <= p.d && (p.d & 3) == 0) {
                                float4* dst = reinterpret_cast<float4*>(dstf);
#pragma unroll
                                for (int j = 0; j < 8; ++j)
                                    dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                         __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                            } else {  // ragged or unaligned row end
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (col0 + j < p.d) dstf[j] = __uint_as_float(v[j]);
                            }
                        } else {
                            uint32_t pk[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                pk[j] = pack_bf16(wv * __uint_as_float(v[2 * j]), wv * __uint_as_float(v[2 * j + 1]));
                            // decode with a K split: part k of a row goes to plane k of the row buffer (p.R rows each)
                            const int64_t drow = (p.store_rows ? grow : (int64_t)tok) + (DEC ? (int64_t)it.kpart * p.R : 0);
                            uint4* dst = reinterpret_cast<uint4*>(p.y + drow * p.d + col0);
#pragma unroll
                            for (int j = 0; j < 4; ++j)
                                dst[j] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                        }
                    }
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&tempty_bar[as]);
        }
    }

    // ------------------------------------------------ teardown
    // Only now may the next kernel's CTAs be scheduled: released earlier they would sit on the SMs
    // waiting for this grid and compete for issue slots with the few warps that drive the pipeline.
    // One thread fires it, after the epilogue loop (a single call marks the whole CTA as triggered).
    if (threadIdx.x == 64) {
        grid_dep_launch();
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (abort_s) __nanosleep(100000);  // let any copy still in flight land before shared memory is released
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

// whole_tpcs: launch as clusters of two CTAs. The CTAs do not use the cluster; the launch then occupies SMs two at a
// time, like the CTA-pair kernel it runs beside, and the two grids cannot leave each other half-filled SM pairs.
template <int MODE, bool DEC>
static cudaError_t launch_gemm_t(const GroupedGemmParams& p, int grid, cudaStream_t s, bool whole_tpcs = false) {
    cudaError_t err = cudaFuncSetAttribute(grouped_gemm_kernel<MODE, DEC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kGemmSmem);
    if (err != cudaSuccess) return err;
    if (whole_tpcs)
        return launch_pdl_cluster(grouped_gemm_kernel<MODE, DEC>, std::max(2, grid & ~1), kGemmThreads, kGemmSmem, 2, s, p);
    return launch_pdl(grouped_gemm_kernel<MODE, DEC>, grid, kGemmThreads, kGemmSmem, s, p);
}

cudaError_t launch_grouped_gemm1(const GroupedGemmParams& p, int grid, cudaStream_t s) {
    return launch_gemm_t<0, false>(p, grid, s);  // decode has its own gate/up kernel (ffn_decode.cu)
}
cudaError_t launch_grouped_gemm2(const GroupedGemmParams& p, int grid, cudaStream_t s) {
    return p.grp_expert != nullptr ? launch_gemm_t<1, true>(p, grid, s) : launch_gemm_t<1, false>(p, grid, s);
}
cudaError_t launch_grouped_gemm1_odd(const GroupedGemmParams& p, int grid, cudaStream_t s) {
    return launch_gemm_t<0, false>(p, grid, s, true);
}
cudaError_t launch_grouped_gemm2_odd(const GroupedGemmParams& p, int grid, cudaStream_t s) {
    return launch_gemm_t<1, false>(p, grid, s, true);
}

}  // namespace exfold
