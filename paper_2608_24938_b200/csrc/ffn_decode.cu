// Decode: gate/up half of the expert FFN over the expert pool (Eq. 1 with the pool of Eq. 11 / 14), with the
// batch-level half of the routing in the kernel's prologue.
//
// Decode cost is the bytes of the distinct experts that are loaded ("Phase-specific budgets"), so every SM should
// stream weights from the first microsecond on and nothing else should cross HBM. One persistent CTA per SM. A
// work item is (pool expert, tile of <= 128 tokens, slice of s = 128 or 64 intermediate features):
//
//   acc[tokens, gate s | up s] = x[tokens, :] * [W_gate[slice, :]; W_up[slice, :]]^T        K = d
//   H[row(token, expert), slice] = silu(gate) * up   -> bf16, only for the tokens the expert serves
//
// Tokens are the 128-row M operand, read from x IN PLACE (all B tokens of the tile: no gathered copy; a token the
// expert does not serve costs nothing extra and is simply not stored), weights the N = 256 operand, which is the
// orientation in which a tcgen05.mma consumes weight bytes fastest (its cost follows M, not N). The two halves of
// tensor memory alternate between items, so the SwiGLU epilogue of one item overlaps the MMAs of the next.
// H is compact: one row per distinct (token, pool expert) pair, grouped by pool rank, tokens ascending. The down
// projection then runs on the grouped GEMM-2 kernel with the whole intermediate dimension as K, which keeps the
// cross-CTA reduction out of memory: measured, a version that also did the down projection per slice spent more
// time on the fp32 reductions of its partial outputs (about 1.9 TB/s of reduction traffic is all L2 takes) than
// on the weights.
//
// The batch-level half of the routing runs in this kernel's prologue, redundantly in every CTA, from the per-token
// Top-K the previous kernel left: routed weights summed per expert in 2^-53 fixed point (exact, order-independent),
// pool by counting ranks on (score desc, id asc), minimum-loss target and scalar per source, remap of every slot,
// rows per group. With the dynamic pool and at most 128 tokens the work list is known once the pool is: the
// producer and MMA warps start streaming then, and the epilogue warps finish the routing beside them. The CTAs
// that own a group's first slice write its execution lists (row -> token, merged weight, slot -> row); CTA 0 writes
// the routing metadata and the group table.
//
// Item sizes: full slices of 128 features; the last partial round of full items is cut into halves (s = 64) when
// that lets more SMs share it, and a trailing 64-wide slice of I is a half by itself.
#include <algorithm>
#include <climits>

#include "common.cuh"
#include "ptx.cuh"

namespace exfold {

namespace {

constexpr int kFThreads = 224;   // warp 0 and 6: TMA producers, warp 1: MMA issuer, warps 2-5: epilogue
constexpr int kFBK = 64;         // K elements per ring stage (one 128-byte swizzle row)
constexpr int kFBBytes = 256 * kFBK * 2;   // weight part of a stage: 128 gate rows + 128 up rows
constexpr int kFMaxStages = 8;
constexpr int kFTmemCols = 512;
constexpr int kFMaxPairs = 2 * kMaxGroups;      // (group, token tile) pairs: B <= 256 is at most two tiles
constexpr int kFSmemLimit = 227 * 1024 - 2048;  // dynamic shared memory the kernel may ask for
static_assert(kGemmBK == 64, "the decode FFN kernel stages 64 K elements per k-block");
static_assert(kMaxDecodeBatch <= 256, "two token tiles per group at most");

struct Scratch {  // per-batch routing state, one copy per CTA
    long long key[kMaxExperts];        // order-preserving integer image of score_e (LLONG_MIN: not in the union)
    unsigned acc32[3 * kMaxExperts];   // sum_i w_{i,e} in 2^-53 units, as three 21-bit limbs
    int in_union[kMaxExperts];
    int rank_of[kMaxExperts];  // pool rank or -1
    int pool[kMaxExperts];     // pool experts by rank
    int target[kMaxExperts];
    float scale[kMaxExperts];
    float h[kMaxExperts];      // norm table (dynamic pool), staged before the dependency wait
    int cnt[kFMaxPairs];       // rows of (group, token tile): distinct tokens of the tile that the group serves
    int goff[kFMaxPairs + 2];  // exclusive prefix of cnt: first compact row of (group, token tile)
    int pairs[kFMaxPairs];     // the pairs that have rows, in order: group * 2 + token tile
    int P, n_pairs;
};
constexpr int kFScratchFixed = (int)((sizeof(Scratch) + 15) / 16 * 16);

struct Item {
    int expert, g, mt, j0, s;
};

struct Sched {  // the same in every role of a CTA
    int n_pairs, nfull, has_half, f_keep, split, total;
    int n96;       // > 0: every item is a 96-wide slice, n96 per pair (see make_sched)
    int identity;  // pair p is (group p, token tile 0): no list needed
    int ctas;      // CTAs that take work: item w belongs to CTA w % ctas
};

// Two ways to deal F full items (plus a few natural halves) over the grid, both static:
//   (a) all CTAs, the last partial round of r full items cut into 2r halves when every half finds its own SM;
//   (b) only eff = ceil(F / rounds) CTAs, each exactly `rounds` items, so that all of them finish together.
// In units of the time one SM needs for a full item alone, a phase of n SMs working at once takes z * max(1, n / c)
// for items of size z: about c = 110 SMs of this kernel saturate HBM (measured: it streams ~55 GB/s per SM, ~6 TB/s together).
// (b) wins when the remainder would leave a few SMs working alone (448 items: 112 x 4 rather than 148 x 3 + 8 halves).
__device__ __forceinline__ Sched make_sched(int n_pairs, int I, int grid, int identity) {
    Sched sc;
    sc.identity = identity;
    sc.n_pairs = n_pairs;
    sc.nfull = I / 128;
    sc.has_half = (I % 128) != 0 ? 1 : 0;
    const int F = n_pairs * sc.nfull, H = n_pairs * sc.has_half;
    const float c = 110.0f;
    const int q = F / grid, r = F % grid;
    const bool can_split = r > 0 && 2 * r + H <= grid;
    // Less than one round of full items, too many to halve: 96-wide slices when they divide I and still fit one round.
    // What an SM streams is bounded by the bytes its ring keeps in flight over the loaded HBM latency (~60 GB/s), so a
    // single round goes faster on more SMs with smaller items (16 experts x 768: 128 items of 0.75 MB, not 96 of 1 MB).
    sc.n96 = 0;
    if (q == 0 && r > 0 && !can_split && H == 0 && I % 96 == 0 && n_pairs * (I / 96) <= grid && I / 96 > sc.nfull) {
        sc.n96 = I / 96;
        sc.split = 0;
        sc.ctas = grid;
        sc.f_keep = 0;
        sc.total = n_pairs * sc.n96;
        return sc;
    }
    float ta = (float)q * fmaxf(1.0f, (float)grid / c);
    if (can_split) ta += 0.5f * fmaxf(1.0f, (float)(2 * r) / c);
    else if (r > 0) ta += fmaxf(1.0f, (float)r / c);
    const int rounds = (F + grid - 1) / grid;
    const int eff = rounds > 0 ? (F + rounds - 1) / rounds : grid;
    const float tb = (float)rounds * fmaxf(1.0f, (float)eff / c);
    if (F > 0 && tb < ta) {
        sc.split = 0;
        sc.ctas = eff;
    } else {
        sc.split = can_split ? r : 0;
        sc.ctas = grid;
    }
    sc.f_keep = F - sc.split;
    sc.total = sc.f_keep + 2 * sc.split + H;
    return sc;
}

__device__ __forceinline__ Item decode_item(int w, const Sched& sc, const Scratch& s, int N) {
    Item it;
    int pair;
    if (sc.n96 > 0) {
        pair = w / sc.n96;
        it.j0 = (w - pair * sc.n96) * 96;
        it.s = 96;
    } else if (w < sc.f_keep) {
        pair = w / sc.nfull;
        it.j0 = (w - pair * sc.nfull) * 128;
        it.s = 128;
    } else if (w < sc.f_keep + 2 * sc.split) {
        const int u = w - sc.f_keep, f = sc.f_keep + (u >> 1);
        pair = f / sc.nfull;
        it.j0 = (f - pair * sc.nfull) * 128 + (u & 1) * 64;
        it.s = 64;
    } else {
        pair = w - sc.f_keep - 2 * sc.split;
        it.j0 = sc.nfull * 128;
        it.s = 64;
    }
    const int code = sc.identity ? pair * 2 : s.pairs[pair];
    it.g = code >> 1;
    it.mt = code & 1;
    it.expert = it.g < s.P ? s.pool[it.g] : N;  // group P is the shared expert
    return it;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(kFThreads, 1) decode_ffn_kernel(const __grid_constant__ DecodeFfnParams p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kFMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kFMaxStages];
    __shared__ __align__(8) uint64_t tfull_bar[2];
    __shared__ __align__(8) uint64_t tempty_bar[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    unsigned char* tiles =
        reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int stages = p.stages;
    const int a_bytes = p.a_rows * kFBK * 2;
    const int stage_bytes = a_bytes + kFBBytes;
    Scratch& sc = *reinterpret_cast<Scratch*>(tiles + p.scratch_off);
    int* ids2 = reinterpret_cast<int*>(tiles + p.scratch_off + kFScratchFixed);
    float* w2 = reinterpret_cast<float*>(ids2 + p.B * p.K);

    // ---- set-up that does not depend on the previous kernel: overlaps its tail under programmatic launch
    if (threadIdx.x == 0) {
        ptx::prefetch_tmap(&p.tm_x);
        ptx::prefetch_tmap(&p.tm_wg);
        ptx::prefetch_tmap(&p.tm_wu);
        ptx::prefetch_tmap(&p.tm_wg96);
        ptx::prefetch_tmap(&p.tm_wu96);
        for (int s = 0; s < kFMaxStages; ++s) {
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
    if (warp == 1) {
        ptx::tmem_alloc(&tmem_base_s, kFTmemCols);
        ptx::tmem_relinquish();
    }
    const int B = p.B, N = p.N, K = p.K, BK = B * K;
    const bool is_static = p.st_pool != nullptr;
    const int nmt = (B + 127) >> 7;
    // With the dynamic pool and one token tile every pool expert has a row (it is in the union), so the work list
    // is known as soon as the pool is: the producer and MMA warps leave for their roles then, and the epilogue
    // warps finish the routing (targets, remap, row lists, metadata) while the first weights stream in.
    const bool early = !is_static && nmt == 1;
    for (int e = threadIdx.x; e < N; e += kFThreads) {
        sc.acc32[3 * e] = sc.acc32[3 * e + 1] = sc.acc32[3 * e + 2] = 0u;
        sc.in_union[e] = 0;
        sc.rank_of[e] = -1;
    }
    for (int i = threadIdx.x; i < kFMaxPairs; i += kFThreads) sc.cnt[i] = 0;
    if (!is_static) {  // the norm table into shared memory, the loss and scalar tables into L2, while the previous kernel runs
        for (int e = threadIdx.x; e < N; e += kFThreads) sc.h[e] = __ldg(p.h + e);
        const size_t n_el = (size_t)N * N, lines = (n_el * 4 + 127) / 128;
        for (size_t i = (size_t)blockIdx.x * kFThreads + threadIdx.x; i < lines; i += (size_t)gridDim.x * kFThreads) {
            const size_t el = i * 32 < n_el ? i * 32 : n_el - 1;
            ptx::prefetch_l2(p.L + el);
            ptx::prefetch_l2(p.S + el);
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    grid_dep_wait();  // the per-token Top-K of the previous kernel; the previous call's readers of the workspace

    // ---- routing, batch level (Eq. 11, 12, 14), the same in every CTA
    // (a thread's loads first, eight slots at a time: independent L2 round trips instead of one per slot)
    for (int s0 = threadIdx.x; s0 < BK; s0 += kFThreads * 8) {
        int id[8];
        double wv[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int s = s0 + u * kFThreads;
            id[u] = s < BK ? p.ids[s] : -1;
            wv[u] = s < BK && !is_static ? p.w64[s] : 0.0;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int s = s0 + u * kFThreads;
            if (id[u] < 0) continue;
            ids2[s] = id[u];
            if (!is_static) {
                // The routed weight in 2^-53 fixed point, added as three 21-bit limbs with 32-bit integer atomics (at
                // most 256 addends per expert, so no limb overflows): exact, and independent of the order of arrival.
                const unsigned long long fx = (unsigned long long)(wv[u] * 9007199254740992.0);
                atomicAdd(&sc.acc32[3 * id[u]], (unsigned)(fx & 0x1FFFFFull));
                atomicAdd(&sc.acc32[3 * id[u] + 1], (unsigned)((fx >> 21) & 0x1FFFFFull));
                atomicAdd(&sc.acc32[3 * id[u] + 2], (unsigned)(fx >> 42));
                sc.in_union[id[u]] = 1;
            }
        }
    }
    __syncthreads();
    if (is_static) {
        for (int e = threadIdx.x; e < N; e += kFThreads) {
            sc.target[e] = p.st_target[e];
            sc.scale[e] = p.st_scale[e];
        }
        for (int j = threadIdx.x; j < p.M; j += kFThreads) {
            const int e = p.st_pool[j];
            sc.pool[j] = e;
            sc.rank_of[e] = j;
        }
        if (threadIdx.x == 0) sc.P = p.M;
        __syncthreads();
    } else {
        // Eq. 11: score_e = h_e * sum_i w_{i,e} in double; ranked through an order-preserving integer key
        for (int e = threadIdx.x; e < N; e += kFThreads) {
            long long key = LLONG_MIN;  // not in the union: never counted, never ranked
            if (sc.in_union[e]) {
                const unsigned long long acc = (unsigned long long)sc.acc32[3 * e] +
                                               ((unsigned long long)sc.acc32[3 * e + 1] << 21) +
                                               ((unsigned long long)sc.acc32[3 * e + 2] << 42);
                const double score = (double)acc * (1.0 / 9007199254740992.0) * (double)sc.h[e] + 0.0;
                key = __double_as_longlong(score);
                if (key < 0) key ^= 0x7FFFFFFFFFFFFFFFll;  // negative doubles: larger magnitude = smaller
            }
            sc.key[e] = key;
        }
        __syncthreads();
        // pool = best min(M, |U|) experts of the union by (score desc, id asc): rank by counting, a thread per expert
        // (integer compares on the keys; every lane of a warp reads the same other key: one broadcast load each)
        for (int e = threadIdx.x; e < N; e += kFThreads) {
            const long long ke = sc.key[e];
            if (ke == LLONG_MIN) continue;
            int better = 0;
#pragma unroll 4
            for (int o = 0; o < N; ++o) {
                const long long ko = sc.key[o];
                better += (ko > ke || (ko == ke && o < e)) ? 1 : 0;
            }
            if (better < p.M) {
                sc.rank_of[e] = better;
                sc.pool[better] = e;
            }
        }
        if (warp == 0) {
            int usz = 0;
            for (int o = lane; o < N; o += 32) usz += sc.in_union[o] ? 1 : 0;
            usz = __reduce_add_sync(0xffffffffu, usz);
            if (lane == 0) sc.P = usz < p.M ? usz : p.M;
        }
        __syncthreads();
    }
    const bool mine = !early || (warp >= 2 && warp <= 5);  // threads that run the rest of the routing
    const int tid = early ? (int)threadIdx.x - 64 : (int)threadIdx.x, nth = early ? 128 : kFThreads;
    auto sync_group = [&]() {
        if (early) asm volatile("bar.sync 1, 128;" ::: "memory");
        else __syncthreads();
    };
    if (mine) {
        const int P = sc.P, G = P + (p.n_shared ? 1 : 0);
        if (!is_static) {
            // Eq. 12: a source in the pool keeps itself; any other takes its minimum-loss pool expert (ties -> lower
            // id). Only sources that occur in the batch matter for the execution; CTA 0 fills the whole table.
            for (int s = tid; s < N; s += nth) {
                if (blockIdx.x != 0 && !sc.in_union[s]) continue;
                int bt = s;
                float scl = 1.0f;
                if (sc.rank_of[s] < 0) {
                    const float* row = p.L + (size_t)s * N;
                    float bl = INFINITY;
                    bt = 0x7fffffff;
                    for (int j0 = 0; j0 < P; j0 += 8) {  // eight independent loads in flight
                        float l[8];
                        int tt[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            tt[u] = j0 + u < P ? sc.pool[j0 + u] : -1;
                            l[u] = tt[u] >= 0 ? __ldg(row + tt[u]) : INFINITY;
                        }
#pragma unroll
                        for (int u = 0; u < 8; ++u)
                            if (tt[u] >= 0 && (bt == 0x7fffffff || l[u] < bl || (l[u] == bl && tt[u] < bt))) {
                                bl = l[u];
                                bt = tt[u];
                            }
                    }
                    scl = __ldg(p.S + (size_t)s * N + bt);
                }
                sc.target[s] = bt;
                sc.scale[s] = scl;
            }
            sync_group();
        }
        // Eq. 14: every slot in place; [B][K] layout kept
        for (int s = tid; s < BK; s += nth) {
            const int e = ids2[s];
            const int t = sc.target[e];
            const float wv = (float)(p.w64[s] * (double)sc.scale[e]);
            ids2[s] = t;
            w2[s] = wv;
            if (blockIdx.x == 0) {
                p.out_ids[s] = t;
                p.out_w[s] = wv;
            }
        }
        if (blockIdx.x == 0) {
            for (int e = tid; e < N; e += nth) {
                p.target[e] = sc.target[e];
                p.scale[e] = sc.scale[e];
                p.pool_ids[e] = e < P ? sc.pool[e] : -1;
            }
            if (tid < 8) {
                uint32_t m = 0;
                for (int b = 0; b < 32; ++b) {
                    const int e = tid * 32 + b;
                    if (e < N && sc.rank_of[e] >= 0) m |= 1u << b;
                }
                p.pool_mask[tid] = m;
            }
            if (tid == 0) *p.pool_size = P;
        }
        sync_group();
        // rows per (group, token tile): a token counts once per distinct target among its slots
        for (int i = tid; i < B; i += nth) {
            for (int k = 0; k < K; ++k) {
                const int t = ids2[i * K + k];
                bool first = true;
                for (int k2 = 0; k2 < k; ++k2) first = first && ids2[i * K + k2] != t;
                if (first) atomicAdd(&sc.cnt[sc.rank_of[t] * 2 + (i >> 7)], 1);
            }
        }
        if (p.n_shared && tid < 2) sc.cnt[P * 2 + tid] = tid == 0 ? min(B, 128) : max(B - 128, 0);
        sync_group();
        // exclusive prefix over (group, tile) = first compact row of each; the pairs that have rows
        if (tid < 32) {
            int carry = 0, n = 0;
            for (int c0 = 0; c0 < 2 * G; c0 += 32) {
                const int c = c0 + tid;
                const int v = c < 2 * G ? sc.cnt[c] : 0;
                int incl = v;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int u = __shfl_up_sync(0xffffffffu, incl, o);
                    if (tid >= o) incl += u;
                }
                if (c < 2 * G) sc.goff[c] = carry + incl - v;
                carry += __shfl_sync(0xffffffffu, incl, 31);
                const unsigned m = __ballot_sync(0xffffffffu, v > 0);
                if (v > 0) sc.pairs[n + __popc(m & ((1u << tid) - 1u))] = c;
                n += __popc(m);
            }
            if (tid == 0) {
                sc.goff[2 * G] = carry;
                sc.n_pairs = n;
            }
        }
        sync_group();
        if (blockIdx.x == 0) {  // group table of the down-projection kernel
            for (int g = tid; g <= G; g += nth) {
                p.grp_off[g] = sc.goff[2 * g];
                if (g < G) p.grp_expert[g] = g < P ? sc.pool[g] : N;
            }
            if (tid == 0) {
                int tiles = 0;
                for (int g = 0; g < G; ++g) {
                    p.grp_tiles[g] = tiles;
                    tiles += (sc.goff[2 * g + 2] - sc.goff[2 * g] + kTileM - 1) / kTileM;
                }
                p.grp_tiles[G] = tiles;
                p.n_groups[0] = G;
                p.n_groups[1] = sc.goff[2 * G];
                p.n_groups[2] = sc.goff[2 * P];  // first row of the shared expert's group
            }
        }
    }
    if (!early) __syncthreads();
    ptx::tc_fence_after();

    const Sched sched = make_sched(early ? sc.P + (p.n_shared ? 1 : 0) : sc.n_pairs, p.I, (int)gridDim.x, early ? 1 : 0);
    const int total = sched.total;
    const int w_begin = (int)blockIdx.x < sched.ctas ? (int)blockIdx.x : total, w_stride = sched.ctas;
    const uint32_t tmem_base = tmem_base_s;
    const int nkb = p.d / kFBK;
    volatile int* abort_flag = &abort_s;

    if (warp == 0 || warp == 6) {
        // ------------------------------------------------ TMA producers (k-block c belongs to producer c % 2)
        if (lane == 0) {
            const int me = warp == 0 ? 0 : 1;
            int stage = 0, phase = 0, turn = 0;
            bool ok = true;
            for (int w = w_begin; w < total && ok; w += w_stride) {
                const Item it = decode_item(w, sched, sc, N);
                const int xrow = it.mt * 128;
                const int wrow = it.expert * p.I + it.j0;
                const uint32_t tx = (uint32_t)(a_bytes + 2 * it.s * kFBK * 2);
                for (int kb = 0; kb < nkb; ++kb) {
                    if (turn == me) {
                        if (!ptx::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, p.status, 1)) {
                            ok = false;
                            break;
                        }
                        unsigned char* a_dst = tiles + stage * stage_bytes;
                        unsigned char* b_dst = a_dst + a_bytes;
                        ptx::mbar_expect_tx(&full_bar[stage], tx);
                        ptx::tma_load_2d(a_dst, &p.tm_x, &full_bar[stage], kb * kFBK, xrow);
                        if (it.s == 128) {
                            ptx::tma_load_2d(b_dst, &p.tm_wg, &full_bar[stage], kb * kFBK, wrow);
                            ptx::tma_load_2d(b_dst + 128 * kFBK * 2, &p.tm_wu, &full_bar[stage], kb * kFBK, wrow);
                        } else if (it.s == 96) {
                            ptx::tma_load_2d(b_dst, &p.tm_wg96, &full_bar[stage], kb * kFBK, wrow);
                            ptx::tma_load_2d(b_dst + 96 * kFBK * 2, &p.tm_wu96, &full_bar[stage], kb * kFBK, wrow);
                        } else {
                            ptx::tma_load_2d(b_dst, &p.tm_wg64, &full_bar[stage], kb * kFBK, wrow);
                            ptx::tma_load_2d(b_dst + 64 * kFBK * 2, &p.tm_wu64, &full_bar[stage], kb * kFBK, wrow);
                        }
                    }
                    turn ^= 1;
                    if (++stage == stages) {
                        stage = 0;
                        phase ^= 1;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t lo0 = (ptx::smem_u32(tiles) & 0x3FFFFu) >> 4;
            const uint32_t lo_step = (uint32_t)stage_bytes >> 4, lo_b = (uint32_t)a_bytes >> 4;
            const uint32_t desc_hi32 = (uint32_t)(ptx::make_kmajor_sw128_desc(0) >> 32);
            constexpr uint32_t idesc256 = ptx::make_idesc_bf16(128, 256), idesc128 = ptx::make_idesc_bf16(128, 128),
                               idesc192 = ptx::make_idesc_bf16(128, 192);
            int stage = 0, phase = 0, item = 0;
            uint32_t a_lo = lo0;
            bool ok = true, ready = false;
            for (int w = w_begin; w < total && ok; w += w_stride, ++item) {
                const Item it = decode_item(w, sched, sc, N);
                const int as = item & 1, aphase = (item >> 1) & 1;
                if (!ptx::mbar_wait(&tempty_bar[as], aphase ^ 1, abort_flag, p.status, 2)) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + as * 256;
                const uint32_t idesc = it.s == 128 ? idesc256 : (it.s == 96 ? idesc192 : idesc128);
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ready && !ptx::mbar_wait(&full_bar[stage], phase, abort_flag, p.status, 3)) {
                        ok = false;
                        break;
                    }
                    const int ns = stage + 1 == stages ? 0 : stage + 1;
                    const int nphase = ns == 0 ? phase ^ 1 : phase;
                    ready = ptx::umma_kblock_bf16(d_tmem, a_lo, a_lo + lo_b, desc_hi32, idesc, kb > 0 ? 1u : 0u,
                                                  &empty_bar[stage], &full_bar[ns], nphase);
                    a_lo = ns == 0 ? lo0 : a_lo + lo_step;
                    stage = ns;
                    phase = nphase;
                }
                if (ok) ptx::umma_commit(&tfull_bar[as]);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue warps (TMEM lane quadrant = warp % 4)
        const int q = warp & 3;
        const int row = q * 32 + lane;
        int item = 0;
        for (int w = w_begin; w < total; w += w_stride, ++item) {
            const Item it = decode_item(w, sched, sc, N);
            const int as = item & 1, aphase = (item >> 1) & 1;
            // Which tokens of the tile does this expert serve? Every warp looks at all four quadrants, so that
            // it knows how many rows come before its own without talking to the other warps.
            const bool shared_grp = it.g >= sc.P;
            unsigned m[4];
#pragma unroll
            for (int qq = 0; qq < 4; ++qq) {
                const int tq = it.mt * 128 + qq * 32 + lane;
                bool v = false;
                if (tq < B) {
                    v = shared_grp;
                    for (int k = 0; k < K && !v; ++k) v = ids2[tq * K + k] == it.expert;
                }
                m[qq] = __ballot_sync(0xffffffffu, v);
            }
            int before = 0;
#pragma unroll
            for (int qq = 0; qq < 4; ++qq)
                if (qq < q) before += __popc(m[qq]);
            const bool valid = (m[q] >> lane) & 1u;
            const int tok = it.mt * 128 + row;
            const int64_t rowpos = sc.goff[it.g * 2 + it.mt] + before + __popc(m[q] & ((1u << lane) - 1u));
            if (it.j0 == 0 && valid) {
                // this CTA owns the group's first slice: it writes the group's rows of the execution lists
                float cw = 1.0f;
                if (!shared_grp) {
                    bool has = false;
                    for (int k = 0; k < K; ++k)
                        if (ids2[tok * K + k] == it.expert) {  // duplicates merged, weights summed in slot order
                            cw = has ? __fadd_rn(cw, w2[tok * K + k]) : w2[tok * K + k];
                            p.slot_row[tok * K + k] = has ? -1 : (int32_t)rowpos;
                            has = true;
                        }
                }
                p.row_tok[rowpos] = tok;
                p.row_w[rowpos] = cw;
            }
            int ok = 1;
            if (lane == 0) ok = ptx::mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status, 4) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            ptx::tc_fence_after();
            if (m[q] != 0u) {  // warp-uniform: some row of this quadrant is stored
                const uint32_t taddr = tmem_base + as * 256 + ((uint32_t)(q * 32) << 16);
                const int nch = it.s / 32;
#pragma unroll 1
                for (int c = 0; c < nch; ++c) {
                    uint32_t gv[32], uv[32];
                    ptx::tmem_ld32(taddr + c * 32, gv);
                    ptx::tmem_ld32(taddr + it.s + c * 32, uv);
                    ptx::tmem_ld_wait();
                    if (valid) {
                        uint32_t pk[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float g0 = __uint_as_float(gv[2 * j]), g1 = __uint_as_float(gv[2 * j + 1]);
                            const float u0 = __uint_as_float(uv[2 * j]), u1 = __uint_as_float(uv[2 * j + 1]);
                            const float h0 = __fdividef(g0, 1.0f + __expf(-g0)) * u0;
                            const float h1 = __fdividef(g1, 1.0f + __expf(-g1)) * u1;
                            pk[j] = pack_bf16x2(h0, h1);
                        }
                        uint4* dst = reinterpret_cast<uint4*>(p.H + rowpos * p.I + it.j0 + c * 32);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            dst[j] = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
                    }
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&tempty_bar[as]);
        }
    }

    // ------------------------------------------------ teardown
    if (threadIdx.x == 64) grid_dep_launch();  // after the epilogue loop: the successor's CTAs would only compete
    ptx::tc_fence_before();
    __syncthreads();
    if (abort_s) __nanosleep(100000);  // let any copy still in flight land before shared memory is released
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kFTmemCols);
    }
}

}  // namespace

// Shared-memory plan: [ring: stages x (token box + 32 KB of weights)][routing state][ids', w']
size_t decode_ffn_smem_plan(int B, int K, int N, int* stages, int* scratch_off, int* a_rows) {
    (void)N;
    const int ar = std::min(kTileM, (B + 31) / 32 * 32);
    const int stage_bytes = ar * kFBK * 2 + kFBBytes;
    const size_t scratch = (kFScratchFixed + (size_t)B * K * 8 + 15) / 16 * 16;
    const long avail = (long)kFSmemLimit - 1024 - (long)scratch;
    int st = (int)(avail / stage_bytes);
    if (st > kFMaxStages) st = kFMaxStages;
    *stages = st;
    *a_rows = ar;
    *scratch_off = st * stage_bytes;
    return 1024 + (size_t)st * stage_bytes + scratch;
}

cudaError_t launch_decode_ffn(const DecodeFfnParams& p, int sms, cudaStream_t s) {
    int stages, scratch_off, a_rows;
    const size_t smem = decode_ffn_smem_plan(p.B, p.K, p.N, &stages, &scratch_off, &a_rows);
    if (stages < 2 || stages != p.stages || scratch_off != p.scratch_off) return cudaErrorInvalidValue;
    cudaError_t err = cudaFuncSetAttribute(decode_ffn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    return launch_pdl(decode_ffn_kernel, std::min(sms, kMaxCtas), kFThreads, smem, s, p);
}

}  // namespace exfold
