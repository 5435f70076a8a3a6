// Prefill routing: Top-K gate (Eq. 2), retained-set selection (Eq. 10), minimum-loss
// assignment (Eq. 12), weight folding (Eq. 13) and the expert-sorted permutation.
//
//   route kernel   one warp per token; lane l holds logits l, l+32, ...; after the Top-K
//                  rounds lane k (k < K) owns route k. Writes ids/w/omitted pairs and a
//                  per-block histogram of retained experts.
//   scatter kernel same token->block map as the route kernel. Each block first derives its own
//                  bases: the route kernel left one histogram row per block and, added up with
//                  integer atomics (order-independent), one per super-block of 64 blocks; a block
//                  sums the super-block rows (all of them: group sizes; those before its own:
//                  earlier routes) and the at most 63 block rows before it inside its super-block,
//                  then takes a prefix over experts (block 0 also publishes offsets and the
//                  row-tile prefix for the GEMM work list). It then ranks its routes in (token,
//                  slot) order, so the permutation is the stable sort by expert and is
//                  bit-reproducible; it also gathers the token rows into sorted order.
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
    // the next token's logits are fetched while the current token is processed
    float vn[NPL];
    {
        const int64_t i0 = tok0 + warp;
#pragma unroll
        for (int q = 0; q < NPL; ++q) {
            const int e = lane + 32 * q;
            vn[q] = (i0 < p.T && warp < kRouteTokensPerBlock && e < N) ? p.logits[i0 * N + e] : -INFINITY;
        }
    }
    for (int tl = warp; tl < kRouteTokensPerBlock; tl += kWarps) {
        const int64_t i = tok0 + tl;
        if (i >= p.T) break;
        uint32_t key_q[NPL];
        uint32_t used = 0;
#pragma unroll
        for (int q = 0; q < NPL; ++q) {
            key_q[q] = float_order_key(vn[q]);
            if (lane + 32 * q >= N) used |= 1u << q;
        }
        {
            const int64_t in = i + kWarps;
            const bool more = tl + kWarps < kRouteTokensPerBlock && in < p.T;
#pragma unroll
            for (int q = 0; q < NPL; ++q) {
                const int e = lane + 32 * q;
                vn[q] = (more && e < N) ? p.logits[in * N + e] : -INFINITY;
            }
        }
        // ---- Eq. 2: K rounds of warp arg-max (hardware reductions); ties -> lower expert id
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
        // ---- Eq. 12 + 13, omitted routes in rank order, four at a time. For an omitted source s every
        // retained lane t loads L[s][t] and S[s][t] itself (independent loads, all in flight together);
        // a warp arg-min over (loss, id) picks the target, which then adds w_s * S[s][t] to its weight.
        float wt = w;
        int my_tgt = -1;  // for omitted lanes: the chosen target (-1: dropped, no admissible target)
        float kept_sum = 0.f;  // sum of the retained routes' original weights (confidence split only)
        if (p.confidence) {
            kept_sum = kept ? w : 0.f;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) kept_sum += __shfl_xor_sync(0xffffffffu, kept_sum, off);
        }
        for (int rr0 = Kp; rr0 < K; rr0 += 4) {
            int src_lane[4], src_id[4];
            float lv[4], sv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int rr = rr0 + u;
                const unsigned m = __ballot_sync(0xffffffffu, rank == rr);
                src_lane[u] = m ? __ffs(m) - 1 : 0;
                src_id[u] = __shfl_sync(0xffffffffu, my_id, src_lane[u]);
                const bool act = kept && rr < K;
                lv[u] = act ? __ldg(p.L + (size_t)src_id[u] * N + my_id) : INFINITY;
                sv[u] = act ? __ldg(p.S + (size_t)src_id[u] * N + my_id) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (rr0 + u >= K) break;  // warp-uniform
                const bool adm = kept && !(lv[u] > p.loss_thr);  // loss-threshold safeguard
                const int bt = warp_argmin(adm, float_order_key(lv[u]), my_id);
                const float ws = __shfl_sync(0xffffffffu, w, src_lane[u]);
                if (bt != 0x7fffffff) {  // warp-uniform: a target exists
                    const bool is_t = kept && my_id == bt;
                    float c = 1.0f;
                    if (p.confidence) {
                        const unsigned tm = __ballot_sync(0xffffffffu, is_t);
                        const float lt = __shfl_sync(0xffffffffu, lv[u], __ffs(tm) - 1);
                        c = fminf(fmaxf(1.0f - lt, 0.0f), 1.0f);
                        if (kept) wt = __fadd_rn(wt, ws * (1.0f - c) * (w / kept_sum));
                    }
                    if (is_t) wt = __fadd_rn(wt, __fmul_rn(ws * c, sv[u]));
                }
                if (lane == src_lane[u]) my_tgt = bt == 0x7fffffff ? -1 : bt;
            }
        }
        if (p.rescale) {  // keep the original routed-weight sum
            float fs = kept ? wt : 0.f, as = has ? w : 0.f;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                fs += __shfl_xor_sync(0xffffffffu, fs, off);
                as += __shfl_xor_sync(0xffffffffu, as, off);
            }
            if (fs > 0.f) wt *= as / fs;
        }
        const int bt = my_tgt;
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
    for (int e = threadIdx.x; e < N; e += blockDim.x) {
        const int h = hist[e];
        p.block_hist[(size_t)blockIdx.x * N + e] = h;
        if (h != 0 && p.sb_hist != nullptr) atomicAdd(&p.sb_hist[(size_t)(blockIdx.x / kRouteSuperBlock) * N + e], h);
    }
}

__global__ void __launch_bounds__(kRouteThreads) prefill_scatter_kernel(PrefillScatterParams p) {
    __shared__ int cnt[kMaxExperts];
    __shared__ int pos[kRouteTokensPerBlock * kMaxTopK];
    __shared__ int pre[kMaxExperts];  // routes of expert e in earlier blocks
    __shared__ int tot[kMaxExperts];  // routes of expert e in all blocks
    __shared__ int warp_tot[kMaxExperts / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int N = p.N, Kp = p.Kp;
    const int64_t tok0 = (int64_t)blockIdx.x * kRouteTokensPerBlock;
    const int ntok = (int)min((int64_t)kRouteTokensPerBlock, p.T - tok0);
    const int n = ntok * Kp;
    const int64_t r0 = tok0 * Kp;
    for (int e = threadIdx.x; e < N; e += blockDim.x) pre[e] = tot[e] = 0;
    __syncthreads();
    grid_dep_launch();
    grid_dep_wait();
    // Bases of this block: first sorted position of expert e = (rows of experts < e) + (rows of e in
    // earlier blocks). Super-block rows first (nsb of them), then the block rows before this one inside
    // its super-block: nsb + 63 rows of N counters at most, whatever the token count.
    {
        const int sb = (int)blockIdx.x / kRouteSuperBlock, nsb = (p.nblk + kRouteSuperBlock - 1) / kRouteSuperBlock;
        const int b0 = sb * kRouteSuperBlock, n_inner = (int)blockIdx.x - b0;
        const int n_rows = nsb + n_inner;
        for (int idx = threadIdx.x; idx < n_rows * N; idx += blockDim.x) {
            const int row = idx / N, e = idx - row * N;
            if (row < nsb) {
                const int v = p.sb_hist[(size_t)row * N + e];
                if (v != 0) {
                    atomicAdd(&tot[e], v);
                    if (row < sb) atomicAdd(&pre[e], v);
                }
            } else {
                const int v = p.block_hist[(size_t)(b0 + row - nsb) * N + e];
                if (v != 0) atomicAdd(&pre[e], v);
            }
        }
    }
    __syncthreads();
    // exclusive prefix of tot over the experts: warp w scans experts [32w, 32w + 32)
    if (warp * 32 < N) {
        const int e = warp * 32 + lane;
        const int v = e < N ? tot[e] : 0;
        int incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int u = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += u;
        }
        if (e < N) cnt[e] = incl - v;
        if (lane == 31) warp_tot[warp] = incl;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < N; e += blockDim.x) {
        int off = 0;
        for (int w = 0; w < (e >> 5); ++w) off += warp_tot[w];
        cnt[e] += off + pre[e];
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {  // group offsets and the row-tile prefix for the GEMM work list
        const int G = N + p.n_shared;
        int off = 0, tiles = 0;
        for (int g = 0; g < G; ++g) {
            const int rows = g < N ? tot[g] : (int)p.T;
            p.offsets[g] = off;
            p.work_start[g] = tiles;
            off += rows;
            tiles += (rows + kTileM - 1) / kTileM;
        }
        p.offsets[G] = off;
        p.work_start[G] = tiles;
    }
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
        if (p.inv_pos != nullptr) p.inv_pos[route] = q;
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
    if (p.sb_hist != nullptr) {  // the super-block histograms are added up with atomics: they start at zero
        const size_t nsb = (size_t)(nblk + kRouteSuperBlock - 1) / kRouteSuperBlock;
        cudaError_t e = cudaMemsetAsync(p.sb_hist, 0, nsb * p.N * sizeof(int32_t), s);
        if (e != cudaSuccess) return e;
    }
    switch (npl) {
        case 1: return launch_pdl(prefill_route_kernel<1>, nblk, kRouteThreads, 0, s, p);
        case 2: return launch_pdl(prefill_route_kernel<2>, nblk, kRouteThreads, 0, s, p);
        case 3: case 4: return launch_pdl(prefill_route_kernel<4>, nblk, kRouteThreads, 0, s, p);
        default: return launch_pdl(prefill_route_kernel<8>, nblk, kRouteThreads, 0, s, p);
    }
}

cudaError_t launch_prefill_scatter(const PrefillScatterParams& p, cudaStream_t s) {
    const int nblk = (int)((p.T + kRouteTokensPerBlock - 1) / kRouteTokensPerBlock);
    return launch_pdl(prefill_scatter_kernel, nblk, kRouteThreads, 0, s, p);
}

}  // namespace exfold
