// Prefill routing: Top-K gate (Eq. 2), retained-set selection (Eq. 10), minimum-loss
// assignment (Eq. 12), weight folding (Eq. 13) and the expert-sorted permutation.
//
//   route kernel   one warp per token; lane l holds logits l, l+32, ...; after the Top-K
//                  rounds lane k (k < K) owns route k. Writes ids/w/omitted pairs and a
//                  per-block histogram of retained experts.
//   sort kernel    one CTA: prefix over blocks per expert, prefix over experts -> offsets,
//                  row-tile prefix for the GEMM work list.
//   scatter kernel same token->block map as the route kernel; ranks routes inside the block in
//                  (token, slot) order, so the permutation is the stable sort by expert and is
//                  bit-reproducible; also gathers the token rows into sorted order.
#include "common.cuh"

namespace exfold {

namespace {

template <int NPL>  // logits per lane = ceil(N / 32)
__global__ void __launch_bounds__(kRouteThreads) prefill_route_kernel(PrefillRouteParams p) {
    __shared__ int hist[kMaxExperts];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    constexpr int kWarps = kRouteThreads / 32;
    grid_dep_launch();
    for (int e = threadIdx.x; e < p.N; e += blockDim.x) hist[e] = 0;
    __syncthreads();
    grid_dep_wait();
    if (p.status != nullptr && blockIdx.x == 0 && threadIdx.x < 4) reinterpret_cast<int*>(p.status)[threadIdx.x] = 0;

    const int N = p.N, K = p.K, Kp = p.Kp, Ko = p.K - p.Kp;
    const int64_t tok0 = (int64_t)blockIdx.x * kRouteTokensPerBlock;
    for (int tl = warp; tl < kRouteTokensPerBlock; tl += kWarps) {
        const int64_t i = tok0 + tl;
        if (i >= p.T) break;
        const float* r = p.logits + i * N;
        float v[NPL];
        uint32_t used = 0;
#pragma unroll
        for (int q = 0; q < NPL; ++q) {
            int e = lane + 32 * q;
            v[q] = e < N ? r[e] : -INFINITY;
            if (e >= N) used |= 1u << q;
        }
        // ---- Eq. 2: K rounds of warp arg-max; ties -> lower expert id
        int my_id = -1;
        float my_r = 0.f;
        for (int k = 0; k < K; ++k) {
            float bv = -INFINITY;
            int be = 0x7fffffff;
#pragma unroll
            for (int q = 0; q < NPL; ++q) {
                bool free_q = !((used >> q) & 1u);
                if (free_q && (be == 0x7fffffff || v[q] > bv)) {
                    bv = v[q];
                    be = lane + 32 * q;
                }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                float ov = __shfl_xor_sync(0xffffffffu, bv, off);
                int oe = __shfl_xor_sync(0xffffffffu, be, off);
                if (oe != 0x7fffffff && (be == 0x7fffffff || ov > bv || (ov == bv && oe < be))) {
                    bv = ov;
                    be = oe;
                }
            }
            if ((be & 31) == lane) used |= 1u << (be >> 5);
            if (lane == k) {
                my_id = be;
                my_r = bv;
            }
        }
        const bool has = lane < K;
        // softmax restricted to the Top-K set (slot 0 holds the largest logit)
        const float rmax = __shfl_sync(0xffffffffu, my_r, 0);
        float ex = has ? expf(my_r - rmax) : 0.f;
        float sum = ex;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        const float w = ex / sum;
        // ---- Eq. 10 on log scale: key = logit + ln h (one fp32 add); rank by (key desc, id asc)
        const float key = has ? __fadd_rn(my_r, p.lnh[my_id]) : -INFINITY;
        int rank = 0;
        for (int j = 0; j < K; ++j) {
            float kj = __shfl_sync(0xffffffffu, key, j);
            int ij = __shfl_sync(0xffffffffu, my_id, j);
            if (has && j != lane && (kj > key || (kj == key && ij < my_id))) rank++;
        }
        if (!has) rank = 0x7fff;
        const bool kept = has && rank < Kp;
        const bool omitted = has && rank >= Kp;
        // ---- Eq. 12: each omitted route picks the retained expert with the smallest loss
        float bl = INFINITY;
        int bt = 0x7fffffff;
        for (int j = 0; j < K; ++j) {
            int ij = __shfl_sync(0xffffffffu, my_id, j);
            int rj = __shfl_sync(0xffffffffu, rank, j);
            if (omitted && rj < Kp) {
                float l = __ldg(p.L + (size_t)my_id * N + ij);
                if (bt == 0x7fffffff || l < bl || (l == bl && ij < bt)) {
                    bl = l;
                    bt = ij;
                }
            }
        }
        const float contrib = omitted ? __fmul_rn(w, __ldg(p.S + (size_t)my_id * N + bt)) : 0.f;
        // ---- Eq. 13: add the omitted routes' scaled weights to their targets, in rank order
        float wt = w;
        for (int rr = Kp; rr < K; ++rr) {
            unsigned m = __ballot_sync(0xffffffffu, rank == rr);
            int src = __ffs(m) - 1;
            float c = __shfl_sync(0xffffffffu, contrib, src);
            int t = __shfl_sync(0xffffffffu, bt, src);
            if (kept && my_id == t) wt = __fadd_rn(wt, c);
        }
        if (kept) {
            p.ids[i * Kp + rank] = my_id;
            p.w[i * Kp + rank] = wt;
            atomicAdd(&hist[my_id], 1);
        } else if (omitted) {
            if (p.omit_src) p.omit_src[i * Ko + (rank - Kp)] = my_id;
            if (p.omit_tgt) p.omit_tgt[i * Ko + (rank - Kp)] = bt;
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < N; e += blockDim.x) p.block_hist[(size_t)blockIdx.x * N + e] = hist[e];
}

// One CTA. block_hist[b][e] (counts) -> exclusive prefix over blocks; offsets, work_start, totals.
__global__ void __launch_bounds__(1024) prefill_sort_kernel(PrefillSortParams p) {
    __shared__ int tot[kMaxGroups + 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int N = p.N;
    grid_dep_launch();
    grid_dep_wait();
    for (int e = warp; e < N; e += nwarps) {
        int run = 0;
        for (int b0 = 0; b0 < p.nblk; b0 += 32) {
            int b = b0 + lane;
            int c = b < p.nblk ? p.block_hist[(size_t)b * N + e] : 0;
            int inc = c;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                int o = __shfl_up_sync(0xffffffffu, inc, off);
                if (lane >= off) inc += o;
            }
            if (b < p.nblk) p.block_hist[(size_t)b * N + e] = run + inc - c;
            run += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) tot[e] = run;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int G = N + p.n_shared;
        int off = 0, tiles = 0;
        for (int g = 0; g < G; ++g) {
            int rows = g < N ? tot[g] : (int)p.T;
            p.offsets[g] = off;
            p.work_start[g] = tiles;
            off += rows;
            tiles += (rows + kTileM - 1) / kTileM;
        }
        p.offsets[G] = off;
        p.work_start[G] = tiles;
        p.totals[0] = tiles;
        p.totals[1] = off;
    }
}

__global__ void __launch_bounds__(kRouteThreads) prefill_scatter_kernel(PrefillScatterParams p) {
    __shared__ int cnt[kMaxExperts];
    __shared__ int pos[kRouteTokensPerBlock * kMaxTopK];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int N = p.N, Kp = p.Kp;
    const int64_t tok0 = (int64_t)blockIdx.x * kRouteTokensPerBlock;
    const int ntok = (int)min((int64_t)kRouteTokensPerBlock, p.T - tok0);
    const int n = ntok * Kp;
    const int64_t r0 = tok0 * Kp;
    grid_dep_launch();
    grid_dep_wait();
    if (p.y32 != nullptr) {  // clear this block's rows of the fp32 accumulator
        float4* z = reinterpret_cast<float4*>(p.y32 + (size_t)tok0 * p.d);
        const int n4 = ntok * p.d / 4;
        for (int c = threadIdx.x; c < n4; c += blockDim.x) z[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (int e = threadIdx.x; e < N; e += blockDim.x)
        cnt[e] = p.offsets[e] + p.block_hist[(size_t)blockIdx.x * N + e];
    __syncthreads();
    if (warp == 0) {
        // routes of this block in (token, slot) order, 32 at a time
        for (int c0 = 0; c0 < n; c0 += 32) {
            int r = c0 + lane;
            int e = r < n ? p.ids[r0 + r] : -1 - lane;
            unsigned m = __match_any_sync(0xffffffffu, e);
            int before = __popc(m & ((1u << lane) - 1u));
            int base = r < n ? cnt[e] : 0;
            __syncwarp();
            if (r < n) {
                pos[r] = base + before;
                if (before == __popc(m) - 1) cnt[e] = base + __popc(m);  // last lane of the group updates
            }
            __syncwarp();
        }
    }
    __syncthreads();
    for (int r = threadIdx.x; r < n; r += blockDim.x) {
        int q = pos[r];
        int64_t route = r0 + r;
        p.perm[q] = (int32_t)route;
        p.row_tok[q] = (int32_t)(route / Kp);
        p.row_w[q] = p.w[route];
        p.row_exp[q] = p.ids[route];
    }
    if (p.n_shared) {  // shared-expert rows follow the routed rows, identity order, weight 1
        const int64_t R = p.T * Kp;
        for (int t = threadIdx.x; t < ntok; t += blockDim.x) {
            p.row_tok[R + tok0 + t] = (int32_t)(tok0 + t);
            p.row_w[R + tok0 + t] = 1.0f;
            p.row_exp[R + tok0 + t] = N;
        }
    }
    if (p.xs != nullptr && p.d_bytes > 0) {
        // gather: sorted row pos[r] <- token row; one warp per route, 16-byte chunks
        const int chunks = p.d_bytes >> 4;
        const int nwarps = blockDim.x >> 5;
        for (int r = warp; r < n; r += nwarps) {
            const uint4* src = reinterpret_cast<const uint4*>(
                reinterpret_cast<const char*>(p.x) + (size_t)((r0 + r) / Kp) * p.d_bytes);
            uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<char*>(p.xs) + (size_t)pos[r] * p.d_bytes);
            for (int c = lane; c < chunks; c += 32) dst[c] = __ldg(src + c);
        }
    }
}

}  // namespace

cudaError_t launch_prefill_route(const PrefillRouteParams& p, cudaStream_t s) {
    const int nblk = (int)((p.T + kRouteTokensPerBlock - 1) / kRouteTokensPerBlock);
    const int npl = (p.N + 31) / 32;
    switch (npl) {
        case 1: return launch_pdl(prefill_route_kernel<1>, nblk, kRouteThreads, 0, s, p);
        case 2: return launch_pdl(prefill_route_kernel<2>, nblk, kRouteThreads, 0, s, p);
        case 3: case 4: return launch_pdl(prefill_route_kernel<4>, nblk, kRouteThreads, 0, s, p);
        default: return launch_pdl(prefill_route_kernel<8>, nblk, kRouteThreads, 0, s, p);
    }
}

cudaError_t launch_prefill_sort(const PrefillSortParams& p, cudaStream_t s) {
    return launch_pdl(prefill_sort_kernel, 1, 1024, 0, s, p);
}

cudaError_t launch_prefill_scatter(const PrefillScatterParams& p, cudaStream_t s) {
    const int nblk = (int)((p.T + kRouteTokensPerBlock - 1) / kRouteTokensPerBlock);
    return launch_pdl(prefill_scatter_kernel, nblk, kRouteThreads, 0, s, p);
}

}  // namespace exfold
