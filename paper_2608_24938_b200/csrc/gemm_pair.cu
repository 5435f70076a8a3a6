// Prefill expert GEMMs on CTA pairs (Eq. 1, 3, 4): 256 token rows x 256 accumulator columns per pair of CTAs.
//
// The one-CTA kernel in gemm_prefill.cu needs 48 KB of operands per k-block (four M128 N256 K16 MMAs = 512 tensor-pipe
// cycles). An SM takes in about 70 bytes per cycle from L2 when all SMs load at once, and a refilled stage arrives
// ~2700 cycles after the MMAs that used it were issued, so with 4 x 48 KB of shared memory the pipe waits for
// operands about a quarter of the time (measured: 680 cycles per k-block). With tcgen05.mma.cta_group::2 a cluster of two CTAs works on two consecutive
// 128-row tiles of one expert against one 256-column weight tile: each CTA stages its own 128 token rows and HALF
// of the weight tile (GEMM-1: CTA 0 the gate rows, CTA 1 the up rows; GEMM-2: 128 output features each), the
// hardware feeds both tensor cores from both halves, and each CTA's tensor memory receives the 128 x 256
// accumulator of its own rows. Per CTA and k-block that is 32 KB instead of 48, and the ring holds 6 stages
// (measured: 514-534 cycles per k-block, the next stage complete at 93-97 % of the polls).
//
// Only whole pairs of row tiles run here; a group's odd last tile is left to the one-CTA kernel (odd_only = 1).
//
// Roles per CTA: warps 0 and 6 TMA producers (k-blocks dealt alternately; own A rows, own half of B; the bytes of
// both CTAs are counted on the leader's barrier), warp 1 MMA issuer (leader CTA only), warps 2-5 epilogue (own
// rows). The leader's commits arrive on both CTAs' stage-release and accumulator-ready barriers; both CTAs'
// epilogue warps arrive on the leader's accumulator-free barrier. Every wait is bounded.
#include "common.cuh"
#include "ptx.cuh"

namespace exfold {

namespace {

constexpr int kPBK = 64;
constexpr int kPStages = 6;
constexpr int kPATileBytes = kTileM * kPBK * 2;  // 16 KB: this CTA's token rows
constexpr int kPBHalfBytes = 128 * kPBK * 2;     // 16 KB: this CTA's half of the weight tile
constexpr int kPStageBytes = kPATileBytes + kPBHalfBytes;
constexpr int kPSmem = kPStages * kPStageBytes + 1024;
constexpr int kPProducers = 2;
constexpr int kPThreads = 192 + 32 * (kPProducers - 1);
constexpr int kPTmemCols = 512;
static_assert(kGemmBK == 64, "the pair kernel stages 64 K elements (one 128-byte swizzle row) per k-block");

struct PairItem {
    int g, row0, rows1, n_idx;  // rows1: valid rows of the second tile (the first is always full)
};

// Work index -> (group, column tile, pair of row tiles); order: group, then see below
__device__ __forceinline__ PairItem decode_pair(int w, int G, int nt, const int* s_off, const int* s_wp) {
    int lo = 0, hi = G;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (s_wp[mid] * nt <= w) lo = mid;
        else hi = mid;
    }
    while (lo + 1 < G && s_wp[lo + 1] * nt <= w) ++lo;  // skip groups without pairs that share the same start
    PairItem it;
    it.g = lo;
    const int pairs = s_wp[lo + 1] - s_wp[lo];
    const int local = w - s_wp[lo] * nt;
    // Within a group the faster index is the one with fewer values: clusters that run together then share the
    // larger operand through L2 (few pairs: they share a weight tile and each re-reads its rows per column tile;
    // more pairs than column tiles, e.g. a shared expert that sees every token: they share rows and re-read weights)
    const bool rows_outer = pairs > nt;
    const int j = rows_outer ? local / nt : local % pairs;
    it.n_idx = rows_outer ? local - j * nt : local / pairs;
    it.row0 = s_off[lo] + j * 2 * kTileM;
    const int left1 = s_off[lo + 1] - it.row0 - kTileM;
    it.rows1 = left1 < kTileM ? left1 : kTileM;
    return it;
}

__device__ __forceinline__ uint32_t pack2_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}

// MODE 0: gate/up + SwiGLU -> H; MODE 1: down projection -> weighted bf16 rows (into y or the per-route buffer).
template <int MODE>
__global__ void __launch_bounds__(kPThreads, 1) grouped_gemm_pair_kernel(const __grid_constant__ GroupedGemmParams p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kPStages];   // used in the leader
    __shared__ __align__(8) uint64_t empty_bar[kPStages];  // one per CTA, released by the leader's commits
    __shared__ __align__(8) uint64_t tfull_bar[2];         // one per CTA
    __shared__ __align__(8) uint64_t tempty_bar[2];        // used in the leader: 8 epilogue warps of the pair
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int s_off[kMaxGroups + 1];
    __shared__ int s_wp[kMaxGroups + 1];
    __shared__ int s_n_odd;  // groups with an odd number of row tiles

    unsigned char* tiles =
        reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)ptx::cluster_ctarank();  // 0 = leader
    const int pair_id = (int)blockIdx.x >> 1, n_launched = (int)gridDim.x >> 1;
    // GEMM-1: the leader stages W_gate rows, its peer W_up rows; GEMM-2: both halves come from W_down (tm_b1: 128-row box)
    const CUtensorMap* tma_b = MODE == 0 ? (rank == 0 ? &p.tm_b0 : &p.tm_b1) : &p.tm_b1;
    if (threadIdx.x == 0) {
        ptx::prefetch_tmap(&p.tm_a);
        ptx::prefetch_tmap(tma_b);
        if (MODE == 0) ptx::prefetch_tmap(&p.tm_a2);
        for (int s = 0; s < kPStages; ++s) {
            ptx::mbar_init(&full_bar[s], 1);
            ptx::mbar_init(&empty_bar[s], 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&tfull_bar[s], 1);
            ptx::mbar_init(&tempty_bar[s], 8);
        }
        abort_s = 0;
        ptx::fence_mbar_init();
    }
    // Beside the odd-tile pass this kernel is launched over all SMs and the clusters beyond its share must leave
    // quickly (the other pass waits for their SMs): tensor memory is then allocated only once a cluster knows that
    // it has work.
    if (warp == 1 && p.sbs.odd_ctas == 0) {
        ptx::tmem_alloc_pair(&tmem_base_s, kPTmemCols);
        ptx::tmem_relinquish_pair();
    }
    grid_dep_wait();  // everything below reads what the routing kernels (or GEMM-1) wrote
    // shared_split == 1: one group, the shared expert's rows; the offsets table is not read (the kernel that writes it
    // may still be running)
    const bool shared_only = MODE == 0 && p.shared_split == 1;
    const int G = shared_only ? 1 : p.G;
    for (int i = threadIdx.x; i <= G; i += kPThreads) s_off[i] = shared_only ? p.R + i * p.x_rows : p.offsets[i];
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) {  // prefix of whole row-tile pairs per group, 32 groups per step
        int carry = 0, odd = 0;
        for (int g0 = 0; g0 < G; g0 += 32) {
            const int g = g0 + lane;
            int pairs = 0;
            if (g < G) {
                const int tiles = (s_off[g + 1] - s_off[g] + kTileM - 1) / kTileM;
                pairs = (MODE == 0 && p.shared_split == 2 && g == p.n_routed) ? 0 : tiles >> 1;
                odd += tiles & 1;
            }
            int incl = pairs;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            if (g < G) s_wp[g] = carry + incl - pairs;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        odd = __reduce_add_sync(0xffffffffu, odd);
        if (lane == 0) {
            s_wp[G] = carry;
            s_n_odd = odd;
        }
    }
    __syncthreads();
    const int nt = p.n_ntiles;
    const int total = s_wp[G] * nt;
    // beside the odd-tile pass this pass keeps only its share of the SM pairs; the other clusters leave at once
    // (both CTAs of a cluster take the same decision: nothing allocated, no cluster barrier entered)
    const bool side = p.sbs.odd_ctas > 0;
    // (the split is taken on ALL pairs, in every kernel of the two passes alike; it discounts the skipped ones itself)
    const int skipped = MODE == 0 && p.shared_split == 2 ? p.sbs.shared_pairs1 : 0;
    const int n_pairs = side ? pair_pass_clusters(s_wp[G] + skipped, s_n_odd, p.sbs) : n_launched;
    const int rounds = n_pairs > 0 ? (total + n_pairs - 1) / n_pairs : 0;
    const int eff = rounds > 0 ? (total + rounds - 1) / rounds : 0;  // pairs that take work and finish together
    const int w_begin = pair_id < eff ? pair_id : total;
    const int w_stride = eff > 0 ? eff : 1;
    if (side) {
        if (pair_id >= eff) return;
        if (warp == 1) {
            ptx::tmem_alloc_pair(&tmem_base_s, kPTmemCols);
            ptx::tmem_relinquish_pair();
        }
        ptx::tc_fence_before();
        __syncthreads();
    }
    ptx::cluster_sync_all();  // both CTAs' barriers are initialised and their tensor memory allocated
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    const int nkb = (MODE == 0 ? p.d : p.I) / kPBK;
    volatile int* abort_flag = &abort_s;

    if (warp == 0 || warp == 6) {
        // ------------------------------------------------ TMA producers (both CTAs; k-block c belongs to producer c % 2)
        if (lane == 0) {
            const int me = warp == 0 ? 0 : 1;
            int stage = 0, phase = 0, turn = 0;
            bool ok = true;
            for (int w = w_begin; w < total && ok; w += w_stride) {
                const PairItem it = decode_pair(w, G, nt, s_off, s_wp);
                const int expert = shared_only ? p.n_routed : it.g;
                const bool from_x = MODE == 0 && expert >= p.n_routed;  // rows read from x itself, no gathered copy
                const CUtensorMap* tma_a = from_x ? &p.tm_a2 : &p.tm_a;
                const int arow = (from_x ? (it.row0 - p.R) % p.x_rows : it.row0) + rank * kTileM;
                const int brow = MODE == 0 ? expert * p.I + it.n_idx * 128 : expert * p.d + it.n_idx * 256 + rank * 128;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (turn == me) {
                        if (!ptx::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, p.status, 1)) {
                            ok = false;
                            break;
                        }
                        unsigned char* a_dst = tiles + stage * kPStageBytes;
                        if (rank == 0) ptx::mbar_expect_tx(&full_bar[stage], 2 * kPStageBytes);  // both CTAs' bytes
                        ptx::tma_load_2d_pair(a_dst, tma_a, &full_bar[stage], kb * kPBK, arow);
                        ptx::tma_load_2d_pair(a_dst + kPATileBytes, tma_b, &full_bar[stage], kb * kPBK, brow);
                    }
                    turn ^= 1;
                    if (++stage == kPStages) {
                        stage = 0;
                        phase ^= 1;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = ptx::make_idesc_bf16(256, 256);
            const uint32_t lo0 = (ptx::smem_u32(tiles) & 0x3FFFFu) >> 4;
            constexpr uint32_t lo_step = (uint32_t)kPStageBytes >> 4, lo_b = (uint32_t)kPATileBytes >> 4;
            const uint32_t desc_hi32 = (uint32_t)(ptx::make_kmajor_sw128_desc(0) >> 32);
            int stage = 0, phase = 0, iter = 0;
            bool ok = true, ready = false;
            static_assert(kPStages == 6, "the k-loop below is written out for six ring stages");
            for (int w = w_begin; w < total && ok; w += w_stride, ++iter) {
                const int as = iter & 1, aphase = (iter >> 1) & 1;
                if (!ptx::mbar_wait(&tempty_bar[as], aphase ^ 1, abort_flag, p.status, 2)) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + as * 256;
                // The k-loop is written out once per ring stage (switch into the stage the ring stands at): this
                // thread's instruction stream paces the tensor pipe, and with the stage a compile-time constant a
                // k-block costs it the MMA sequence, one compare and one branch.
                int kb = 0;
#define EXFOLD_PAIR_KBLOCK(S)                                                                                      \
    {                                                                                                               \
        constexpr int NS = (S) + 1 == kPStages ? 0 : (S) + 1;                                                       \
        const uint32_t nphase = NS == 0 ? phase ^ 1 : phase;                                                        \
        if (!ready && !ptx::mbar_wait(&full_bar[S], phase, abort_flag, p.status, 3)) {                              \
            ok = false;                                                                                             \
            break;                                                                                                  \
        }                                                                                                           \
        ready = ptx::umma_kblock_bf16_pair(d_tmem, lo0 + (S) * lo_step, lo0 + (S) * lo_step + lo_b, desc_hi32,    \
                                           idesc, kb > 0 ? 1u : 0u, &empty_bar[S], &full_bar[NS], nphase);          \
        if (NS == 0) phase ^= 1;                                                                                    \
        if (++kb == nkb) {                                                                                          \
            stage = NS;                                                                                             \
            break;                                                                                                  \
        }                                                                                                           \
    }
                while (ok && kb < nkb) {
                    switch (stage) {
                        case 0: EXFOLD_PAIR_KBLOCK(0)
                        case 1: EXFOLD_PAIR_KBLOCK(1)
                        case 2: EXFOLD_PAIR_KBLOCK(2)
                        case 3: EXFOLD_PAIR_KBLOCK(3)
                        case 4: EXFOLD_PAIR_KBLOCK(4)
                        default: EXFOLD_PAIR_KBLOCK(5)
                    }
                    if (kb < nkb) stage = 0;  // fell through the last stage: the ring wraps
                }
#undef EXFOLD_PAIR_KBLOCK
                if (ok) ptx::umma_commit_pair(&tfull_bar[as], 3);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue warps (own rows; TMEM lane quadrant = warp % 4)
        const int q = warp & 3;
        int iter = 0;
        for (int w = w_begin; w < total; w += w_stride, ++iter) {
            const int as = iter & 1, aphase = (iter >> 1) & 1;
            const PairItem it = decode_pair(w, G, nt, s_off, s_wp);
            const int rows = rank ? it.rows1 : kTileM;
            const int row = q * 32 + lane;
            const bool valid = row < rows;
            const int64_t grow = (int64_t)it.row0 + rank * kTileM + row;
            int tok = 0;  // GEMM-2: the row's token and weight, asked for before the wait for the accumulator
            float wv = 0.f;
            if (MODE == 1 && valid) {
                tok = p.row_tok[grow];
                wv = p.row_w[grow];
            }
            int ok = 1;
            if (lane == 0) ok = ptx::mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status, 4) ? 1 : 0;
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
                            pk[j] = pack2_bf16(h0, h1);
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
                        uint32_t pk[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            pk[j] = pack2_bf16(wv * __uint_as_float(v[2 * j]), wv * __uint_as_float(v[2 * j + 1]));
                        const int64_t drow = p.store_rows ? grow : (int64_t)tok;
                        uint4* dst = reinterpret_cast<uint4*>(p.y + drow * p.d + col0);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            dst[j] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                    }
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive_leader(&tempty_bar[as]);
        }
    }

    // ------------------------------------------------ teardown
    if (threadIdx.x == 64) grid_dep_launch();  // after the epilogue loop, as in the one-CTA kernel
    ptx::tc_fence_before();
    __syncthreads();
    if (abort_s) __nanosleep(100000);  // let any copy still in flight land before shared memory is released
    ptx::cluster_sync_all();           // the peer is done with this CTA's shared and tensor memory
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc_pair(tmem_base, kPTmemCols);
    }
}

template <int MODE>
cudaError_t launch_pair_t(const GroupedGemmParams& p, int grid, cudaStream_t s) {
    cudaError_t err = cudaFuncSetAttribute(grouped_gemm_pair_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           kPSmem);
    if (err != cudaSuccess) return err;
    grid &= ~1;  // whole pairs
    if (grid < 2) grid = 2;
    return launch_pdl_cluster(grouped_gemm_pair_kernel<MODE>, grid, kPThreads, kPSmem, 2, s, p);
}

}  // namespace

cudaError_t launch_grouped_gemm1_pair(const GroupedGemmParams& p, int grid, cudaStream_t s) {
    return launch_pair_t<0>(p, grid, s);
}
cudaError_t launch_grouped_gemm2_pair(const GroupedGemmParams& p, int grid, cudaStream_t s) {
    return launch_pair_t<1>(p, grid, s);
}

}  // namespace exfold
