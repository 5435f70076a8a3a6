// Decode routing: batch-level expert pool (Eq. 11), minimum-loss targets (Eq. 12) and the
// in-place remap of every routed slot (Eq. 14). B*K <= 4096 slots live in the shared memory of one
// CTA. The kernel runs as one cluster of 8 CTAs, each holding a full copy of that state: the per-token
// Top-K (instruction-issue bound on a single SM), the target search (each CTA keeps its slice of the
// loss / scalar table rows in shared memory) and the row lists are dealt over the CTAs and their results
// broadcast into every copy through distributed shared memory; the cheap steps in between are replicated.
// Also builds the execution lists for the weight-streaming FFN: rows sorted by pool rank, duplicate
// (token, expert) slots merged so that each pool expert runs once per token (Method, "Unified Expert
// Folding", the remark after Eq. 4).
#include "common.cuh"
#include "ptx.cuh"

#include <cooperative_groups.h>

namespace exfold {

namespace {

namespace cg = cooperative_groups;

constexpr int kDecThreads = 1024;
constexpr int kDecMaxSlots = 4096;
constexpr int kDecCluster = 8;  // CTAs that share the Top-K phase

struct DecSmem {
    double w64[kDecMaxSlots];
    int ids[kDecMaxSlots];
    float wrm[kDecMaxSlots];  // remapped weights
    double score[kMaxExperts];
    unsigned long long acc[kMaxExperts];  // sum_i w_{i,e} in fixed point (2^-53 units): exact, order-independent
    int in_union[kMaxExperts];
    int rank_of[kMaxExperts];   // pool rank or -1
    int pool[kMaxExperts];      // pool ids by rank
    int target[kMaxExperts];
    float scale[kMaxExperts];
    float hh[kMaxExperts];      // norm table h
    int gcnt[kMaxExperts + 2];
    int goff[kMaxExperts + 2];
    int P;
};
constexpr size_t kDecSmemBytes = (sizeof(DecSmem) + 15) / 16 * 16;  // the table rows follow

__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(ptx::smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}

template <int NPL>
__global__ void __launch_bounds__(kDecThreads) decode_route_kernel(DecodeRouteParams p) {
    extern __shared__ __align__(16) unsigned char smraw[];
    DecSmem& sm = *reinterpret_cast<DecSmem*>(smraw);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int kWarps = kDecThreads / 32;
    const int B = p.B, N = p.N, K = p.K, M = p.M;
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank(), nct = (int)cluster.num_blocks();
    // Every CTA keeps a full copy of the small per-batch state; results are broadcast into all copies.
    DecSmem* peer[kDecCluster];
#pragma unroll
    for (int r = 0; r < kDecCluster; ++r) peer[r] = r < nct ? cluster.map_shared_rank(&sm, r) : &sm;
    const bool is_static = p.st_pool != nullptr;
    // this CTA's slice of source experts and its rows of the loss / scalar tables (shared memory)
    const int rows_per = (N + nct - 1) / nct;
    const int s_lo = min(N, rank * rows_per), s_hi = min(N, s_lo + rows_per);
    float* tL = reinterpret_cast<float*>(smraw + kDecSmemBytes);
    float* tS = tL + (size_t)rows_per * N;
    grid_dep_launch();
    grid_dep_wait();
    if (p.status != nullptr && rank == 0 && threadIdx.x < 4) reinterpret_cast<int*>(p.status)[threadIdx.x] = 0;
    for (int e = threadIdx.x; e < N; e += kDecThreads) {
        sm.acc[e] = 0ull;
        sm.in_union[e] = 0;
        sm.rank_of[e] = -1;  // pool ranks arrive from other CTAs later
    }
    // Every copy must be cleared before any CTA adds to it: arrive now, wait just before the first remote
    // write, so the barrier's latency hides behind the logits load and the Top-K rounds.
    cluster.barrier_arrive();
    bool cleared = false;
    // ---- Eq. 2 per token (warp per token, tokens dealt round-robin over the cluster's CTAs), weights in
    // double; the first token's logits are requested before the table rows so that they arrive first.
    const int i_first = rank + nct * warp, i_step = nct * kWarps;
    float vn[NPL];
#pragma unroll
    for (int q = 0; q < NPL; ++q) {
        const int e = lane + 32 * q;
        vn[q] = (i_first < B && e < N) ? p.logits[(size_t)i_first * N + e] : -INFINITY;
    }
    if (!is_static) {
        // Rows [s_lo, s_hi) of L and S and the norm table, needed once the sums are in: asynchronous copies
        // into shared memory that stay in flight during the Top-K (waited for before the next cluster barrier).
        const int n_el = (s_hi - s_lo) * N;
        const float* gL = p.L + (size_t)s_lo * N;
        const float* gS = p.S + (size_t)s_lo * N;
        for (int idx = threadIdx.x; idx < n_el; idx += kDecThreads) {
            cp_async4(tL + idx, gL + idx);
            cp_async4(tS + idx, gS + idx);
        }
        for (int e = threadIdx.x; e < N; e += kDecThreads) cp_async4(&sm.hh[e], p.h + e);
    }
    for (int i = i_first; i < B; i += i_step) {
        uint32_t key_q[NPL];
        uint32_t used = 0;
#pragma unroll
        for (int q = 0; q < NPL; ++q) {
            key_q[q] = float_order_key(vn[q]);
            if (lane + 32 * q >= N) used |= 1u << q;
        }
#pragma unroll
        for (int q = 0; q < NPL; ++q) {
            const int e = lane + 32 * q;
            vn[q] = (i + i_step < B && e < N) ? p.logits[(size_t)(i + i_step) * N + e] : -INFINITY;
        }
        int my_id = -1;
        float my_r = 0.f;
        for (int k = 0; k < K; ++k) {
            uint32_t bk = 0;
            int be = 0x7fffffff;
#pragma unroll
            for (int q = 0; q < NPL; ++q) {
                const bool free_q = !((used >> q) & 1u);
                if (free_q && (be == 0x7fffffff || key_q[q] > bk)) {
                    bk = key_q[q];
                    be = lane + 32 * q;
                }
            }
            uint32_t mk;
            be = warp_argmax(be != 0x7fffffff, bk, be, &mk);
            if ((be & 31) == lane) used |= 1u << (be >> 5);
            if (lane == k) {
                my_id = be;
                my_r = float_from_order_key(mk);
            }
        }
        const float rmax = __shfl_sync(0xffffffffu, my_r, 0);
        double ex = lane < K ? exp((double)my_r - (double)rmax) : 0.0;
        double sum = 0.0;
        for (int k = 0; k < K; ++k) sum += __shfl_sync(0xffffffffu, ex, k);  // slot order, like the definition
        if (!cleared) {  // warp-uniform
            cluster.barrier_wait();
            cleared = true;
        }
        if (lane < K) {
            const double wv = ex / sum;
            // fixed-point (2^-53) integer atomics: the sum does not depend on the order of arrival
            const unsigned long long fx = (unsigned long long)(wv * 9007199254740992.0);
#pragma unroll
            for (int r = 0; r < kDecCluster; ++r)
                if (r < nct) {
                    peer[r]->ids[i * K + lane] = my_id;
                    peer[r]->w64[i * K + lane] = wv;
                    atomicAdd(&peer[r]->acc[my_id], fx);
                    peer[r]->in_union[my_id] = 1;
                }
        }
    }
    if (!cleared) cluster.barrier_wait();  // warps without a token
    asm volatile("cp.async.wait_all;" ::: "memory");
    cluster.sync();  // all routes and sums have landed in every copy; this CTA's table rows are in place

    const int nslots = B * K;
    if (is_static) {
        // static pool: precomputed pool, targets and scalars; no batch reduction
        for (int e = threadIdx.x; e < N; e += kDecThreads) {
            sm.rank_of[e] = -1;
            sm.target[e] = p.st_target[e];
            sm.scale[e] = p.st_scale[e];
        }
        __syncthreads();
        for (int j = threadIdx.x; j < M; j += kDecThreads) {
            const int e = p.st_pool[j];
            sm.pool[j] = e;
            sm.rank_of[e] = j;
        }
        if (threadIdx.x == 0) sm.P = M;
    }
    // ---- Eq. 11: score_e = h_e * sum_i w_{i,e} (every CTA computes the same pool from the same sums)
    if (!is_static)
        for (int e = threadIdx.x; e < N; e += kDecThreads)
            sm.score[e] = (double)sm.acc[e] * (1.0 / 9007199254740992.0) * (double)sm.hh[e];
    __syncthreads();
    // pool = best min(M, |U|) experts of the union by (score desc, id asc): rank by counting. Experts are
    // dealt round-robin over the CTAs, one warp per expert; ranks are broadcast to every copy.
    if (!is_static) {
        int usz = 0;
        for (int o = lane; o < N; o += 32) usz += sm.in_union[o] ? 1 : 0;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) usz += __shfl_xor_sync(0xffffffffu, usz, off);
        if (threadIdx.x == 0) sm.P = usz < M ? usz : M;
        for (int e = rank + nct * warp; e < N; e += nct * kWarps) {
            if (!sm.in_union[e]) continue;  // warp-uniform
            const double se = sm.score[e];
            int better = 0;
            for (int o = lane; o < N; o += 32)
                if (sm.in_union[o] && (sm.score[o] > se || (sm.score[o] == se && o < e))) better++;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) better += __shfl_xor_sync(0xffffffffu, better, off);
            if (better < M && lane < nct) {
                DecSmem* dst = cluster.map_shared_rank(&sm, lane);
                dst->rank_of[e] = better;
                dst->pool[better] = e;
            }
        }
        cluster.sync();  // the pool is in every copy
    } else {
        __syncthreads();
    }
    const int P = sm.P;
    // ---- Eq. 12 for the source experts of this CTA's slice (one warp per source, table rows in shared
    // memory): itself if in the pool, else its min-loss pool expert; the result goes to every copy.
    if (!is_static) {
        for (int s = s_lo + warp; s < s_hi; s += kWarps) {
            int bt = s;
            float sc = 1.0f;
            if (sm.rank_of[s] < 0) {  // warp-uniform
                const float* row = tL + (size_t)(s - s_lo) * N;
                float bl = INFINITY;
                int bj = 0x7fffffff;
                for (int j = lane; j < P; j += 32) {
                    const int t = sm.pool[j];
                    const float l = row[t];
                    if (bj == 0x7fffffff || l < bl || (l == bl && t < bj)) {
                        bl = l;
                        bj = t;
                    }
                }
                bt = warp_argmin(bj != 0x7fffffff, float_order_key(bl), bj);
                sc = tS[(size_t)(s - s_lo) * N + bt];
            }
            if (lane < nct) {
                DecSmem* dst = cluster.map_shared_rank(&sm, lane);
                dst->target[s] = bt;
                dst->scale[s] = sc;
            }
        }
        cluster.sync();  // targets of all slices are in every copy
    }
    // ---- Eq. 14: remap every slot in place (each CTA on its own copy); [B][K] layout kept
    for (int s = threadIdx.x; s < nslots; s += kDecThreads) {
        int e = sm.ids[s];
        int t = sm.target[e];
        float wv = (float)(sm.w64[s] * (double)sm.scale[e]);
        sm.ids[s] = t;
        sm.wrm[s] = wv;
        if (rank == 0) {
            p.ids[s] = t;
            p.w[s] = wv;
        }
    }
    if (rank == 0) {
        for (int e = threadIdx.x; e < N; e += kDecThreads) {
            p.target[e] = sm.target[e];
            p.scale[e] = sm.scale[e];
            p.pool_ids[e] = e < P ? sm.pool[e] : -1;
        }
        if (threadIdx.x < 8) {
            uint32_t m = 0;
            for (int b = 0; b < 32; ++b) {
                int e = threadIdx.x * 32 + b;
                if (e < N && sm.rank_of[e] >= 0) m |= 1u << b;
            }
            p.pool_mask[threadIdx.x] = m;
        }
        if (threadIdx.x == 0) *p.pool_size = P;
    }
    __syncthreads();
    // ---- execution lists: one row per distinct (token, pool expert), grouped by pool rank. Groups are
    // dealt round-robin over the cluster's CTAs; pass 0 counts and broadcasts, pass 1 writes the rows.
    for (int pass = 0; pass < 2; ++pass) {
        for (int g = rank + nct * warp; g < P; g += nct * kWarps) {
            const int t = sm.pool[g];
            int run = pass ? sm.goff[g] : 0;
            for (int i0 = 0; i0 < B; i0 += 32) {
                int i = i0 + lane;
                bool has = false;
                float ws = 0.f;
                if (i < B)
                    for (int k = 0; k < K; ++k)
                        if (sm.ids[i * K + k] == t) {
                            ws = has ? __fadd_rn(ws, sm.wrm[i * K + k]) : sm.wrm[i * K + k];
                            has = true;
                        }
                unsigned m = __ballot_sync(0xffffffffu, has);
                if (pass && has) {
                    int q = run + __popc(m & ((1u << lane) - 1u));
                    p.row_tok[q] = i;
                    p.row_w[q] = ws;
                }
                run += __popc(m);
            }
            if (!pass && lane < nct) cluster.map_shared_rank(&sm, lane)->gcnt[g] = run;
        }
        if (!pass) {
            cluster.sync();  // all group sizes are in every copy
            if (warp == 0) {  // exclusive prefix over the groups, 32 at a time
                int carry = 0;
                for (int g0 = 0; g0 < P; g0 += 32) {
                    const int g = g0 + lane;
                    const int c = g < P ? sm.gcnt[g] : 0;
                    int incl = c;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const int v = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= o) incl += v;
                    }
                    if (g < P) sm.goff[g] = carry + incl - c;
                    carry += __shfl_sync(0xffffffffu, incl, 31);
                }
                if (lane == 0) {
                    sm.goff[P] = carry;
                    if (p.n_shared) sm.goff[P + 1] = carry + B;
                }
            }
            __syncthreads();
        }
    }
    if (rank != 0) return;
    const int G = P + (p.n_shared ? 1 : 0);
    for (int g = threadIdx.x; g <= G; g += kDecThreads) {
        p.grp_off[g] = sm.goff[g];
        if (g < G) p.grp_expert[g] = g < P ? sm.pool[g] : N;
    }
    if (threadIdx.x == 0) {  // prefix of 128-row tiles per group
        int tiles = 0;
        for (int g = 0; g < G; ++g) {
            p.grp_tiles[g] = tiles;
            tiles += (sm.goff[g + 1] - sm.goff[g] + kTileM - 1) / kTileM;
        }
        p.grp_tiles[G] = tiles;
    }
    if (p.n_shared)
        for (int i = threadIdx.x; i < B; i += kDecThreads) {
            p.row_tok[sm.goff[P] + i] = i;
            p.row_w[sm.goff[P] + i] = 1.0f;
        }
    if (threadIdx.x == 0) {
        p.n_groups[0] = G;
        p.n_groups[1] = sm.goff[G];  // total rows
    }
}


// ---------------------------------------------------------------- token-parallel first half of decode routing
// Per token: (optionally) the router scores of Eq. 2 as fixed-order dot products - the same lane partition, the
// same fused multiply-adds and the same shuffle tree as router_simt_kernel, so the scores are those of
// exfold_router_logits bit for bit -, then the token's Top-K and its softmax weights in double (slot order).
// Without the router: one CTA per token. With it: a cluster of 8 CTAs per token, each taking an eighth of the
// experts (one CTA alone would walk the whole router matrix with a handful of loads in flight); the scores meet
// in the shared memory of the cluster's first CTA, which then ranks them. CTA 0 also clears the status record.
// The batch-level half (pool, targets, remap) runs in the prologue of the gate/up kernel (ffn_decode.cu).
constexpr int kTopkCluster = 8;

template <int NPL, bool ROUTER>
__global__ void __launch_bounds__(256) decode_topk_kernel(DecodeTopkParams p) {
    __shared__ float s_lg[kMaxExperts];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int N = p.N, K = p.K, d = p.d;
    const int i = ROUTER ? (int)blockIdx.x / kTopkCluster : (int)blockIdx.x;
    grid_dep_launch();
    grid_dep_wait();  // x may be the previous layer's output; the workspace may still be read by the previous call
    if (blockIdx.x == 0 && threadIdx.x < 4) reinterpret_cast<int*>(p.status)[threadIdx.x] = 0;
    if (ROUTER) {
        cg::cluster_group cluster = cg::this_cluster();
        const int rank = (int)cluster.block_rank();
        float* lead = cluster.map_shared_rank(s_lg, 0);
        const int per = (N + kTopkCluster - 1) / kTopkCluster;
        const int e_lo = rank * per, e_hi = min(N, e_lo + per);
        const __nv_bfloat16* xi = p.x + (size_t)i * d;
        for (int e = e_lo + warp; e < e_hi; e += 8) {
            const __nv_bfloat16* we = p.w_router + (size_t)e * d;
            float acc = 0.f;
            for (int c = lane * 8; c < d; c += 256) {
                const uint4 a = *reinterpret_cast<const uint4*>(we + c), b = *reinterpret_cast<const uint4*>(xi + c);
                const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
                const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float2 fa = __bfloat1622float2(pa[j]), fb = __bfloat1622float2(pb[j]);
                    acc = fmaf(fa.x, fb.x, acc);
                    acc = fmaf(fa.y, fb.y, acc);
                }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (lane == 0) {
                lead[e] = acc;
                p.logits_out[(size_t)i * N + e] = acc;
            }
        }
        cluster.sync();  // every score of the token is in the first CTA's shared memory
        if (rank != 0) return;
    }
    if (warp != 0) return;
    float v[NPL];
#pragma unroll
    for (int q = 0; q < NPL; ++q) {
        const int e = lane + 32 * q;
        v[q] = e < N ? (ROUTER ? s_lg[e] : p.logits[(size_t)i * N + e]) : -INFINITY;
    }
    uint32_t key_q[NPL];
    uint32_t used = 0;
#pragma unroll
    for (int q = 0; q < NPL; ++q) {
        key_q[q] = float_order_key(v[q]);
        if (lane + 32 * q >= N) used |= 1u << q;
    }
    int my_id = -1;
    float my_r = 0.f;
    for (int k = 0; k < K; ++k) {
        uint32_t bk = 0;
        int be = 0x7fffffff;
#pragma unroll
        for (int q = 0; q < NPL; ++q) {
            const bool free_q = !((used >> q) & 1u);
            if (free_q && (be == 0x7fffffff || key_q[q] > bk)) {
                bk = key_q[q];
                be = lane + 32 * q;
            }
        }
        uint32_t mk;
        be = warp_argmax(be != 0x7fffffff, bk, be, &mk);
        if ((be & 31) == lane) used |= 1u << (be >> 5);
        if (lane == k) {
            my_id = be;
            my_r = float_from_order_key(mk);
        }
    }
    const float rmax = __shfl_sync(0xffffffffu, my_r, 0);
    const double ex = lane < K ? exp((double)my_r - (double)rmax) : 0.0;
    double sum = 0.0;
    for (int k = 0; k < K; ++k) sum += __shfl_sync(0xffffffffu, ex, k);  // slot order, like the definition
    if (lane < K) {
        p.ids[(size_t)i * K + lane] = my_id;
        p.w64[(size_t)i * K + lane] = ex / sum;
    }
}

// Static pool: pool = TopK_e(h_e, M) (ties -> lower id, descending h), then Eq. 12 for every source.
__global__ void __launch_bounds__(256) static_pool_kernel(int N, int M, const float* __restrict__ S,
                                                          const float* __restrict__ L, const float* __restrict__ h,
                                                          int32_t* pool_ids, int32_t* target, float* scale) {
    __shared__ int pool[kMaxExperts];
    __shared__ int rank_of[kMaxExperts];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    grid_dep_launch();
    grid_dep_wait();
    for (int e = threadIdx.x; e < N; e += blockDim.x) {
        const float he = h[e];
        int better = 0;
        for (int o = 0; o < N; ++o) {
            const float ho = h[o];
            if (ho > he || (ho == he && o < e)) better++;
        }
        rank_of[e] = better < M ? better : -1;
        if (better < M) {
            pool[better] = e;
            pool_ids[better] = e;
        }
    }
    __syncthreads();
    for (int s = warp; s < N; s += nwarps) {
        if (rank_of[s] >= 0) {
            if (lane == 0) {
                target[s] = s;
                scale[s] = 1.0f;
            }
            continue;
        }
        float bl = INFINITY;
        int bt = 0x7fffffff;
        for (int j = lane; j < M; j += 32) {
            const int t = pool[j];
            const float l = L[(size_t)s * N + t];
            if (bt == 0x7fffffff || l < bl || (l == bl && t < bt)) {
                bl = l;
                bt = t;
            }
        }
        bt = warp_argmin(bt != 0x7fffffff, float_order_key(bl), bt);
        if (lane == 0) {
            target[s] = bt;
            scale[s] = S[(size_t)s * N + bt];
        }
    }
}

}  // namespace

cudaError_t launch_decode_route(const DecodeRouteParams& p, cudaStream_t s) {
    const int npl = (p.N + 31) / 32;
    // state + this CTA's rows of the two tables
    const size_t smem = kDecSmemBytes + 2 * (size_t)((p.N + kDecCluster - 1) / kDecCluster) * p.N * sizeof(float);
    cudaError_t err = cudaSuccess;
#define EXFOLD_DEC_LAUNCH(NPL)                                                                              \
    err = cudaFuncSetAttribute(decode_route_kernel<NPL>, cudaFuncAttributeMaxDynamicSharedMemorySize,       \
                               (int)smem);                                                                  \
    if (err != cudaSuccess) return err;                                                                     \
    err = launch_pdl_cluster(decode_route_kernel<NPL>, kDecCluster, kDecThreads, smem, kDecCluster, s, p);
    switch (npl) {
        case 1: EXFOLD_DEC_LAUNCH(1) break;
        case 2: EXFOLD_DEC_LAUNCH(2) break;
        case 3: case 4: EXFOLD_DEC_LAUNCH(4) break;
        default: EXFOLD_DEC_LAUNCH(8) break;
    }
#undef EXFOLD_DEC_LAUNCH
    return err;
}

cudaError_t launch_decode_topk(const DecodeTopkParams& p, cudaStream_t s) {
    const int npl = (p.N + 31) / 32;
    if (p.w_router != nullptr) {
        const unsigned grid = (unsigned)p.B * kTopkCluster;
        switch (npl) {
            case 1: return launch_pdl_cluster(decode_topk_kernel<1, true>, grid, 256, 0, kTopkCluster, s, p);
            case 2: return launch_pdl_cluster(decode_topk_kernel<2, true>, grid, 256, 0, kTopkCluster, s, p);
            case 3: case 4: return launch_pdl_cluster(decode_topk_kernel<4, true>, grid, 256, 0, kTopkCluster, s, p);
            default: return launch_pdl_cluster(decode_topk_kernel<8, true>, grid, 256, 0, kTopkCluster, s, p);
        }
    }
    switch (npl) {
        case 1: return launch_pdl(decode_topk_kernel<1, false>, p.B, 256, 0, s, p);
        case 2: return launch_pdl(decode_topk_kernel<2, false>, p.B, 256, 0, s, p);
        case 3: case 4: return launch_pdl(decode_topk_kernel<4, false>, p.B, 256, 0, s, p);
        default: return launch_pdl(decode_topk_kernel<8, false>, p.B, 256, 0, s, p);
    }
}

cudaError_t launch_static_pool(int N, int M, const float* S, const float* L, const float* h, int32_t* pool_ids,
                               int32_t* target, float* scale, cudaStream_t s) {
    return launch_pdl(static_pool_kernel, 1, 256, 0, s, N, M, S, L, h, pool_ids, target, scale);
}

}  // namespace exfold
