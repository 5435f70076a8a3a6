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
#include "common.cuh"
#include "ptx.cuh"

namespace exfold {

namespace {

constexpr int kBK = 64;                       // K elements per stage: 128 bytes = one swizzle row
constexpr int kStages = 4;
constexpr int kATileBytes = kTileM * kBK * 2;  // 16 KB
constexpr int kBTileBytes = 256 * kBK * 2;     // 32 KB
constexpr int kStageBytes = kATileBytes + kBTileBytes;
constexpr int kGemmSmem = kStages * kStageBytes + 1024;
constexpr int kGemmThreads = 192;
constexpr int kTmemCols = 512;

struct WorkItem {
    int g, row0, rows, n_idx;
};

__device__ __forceinline__ WorkItem decode_work(int w, int G, int nt, const int* s_off, const int* s_ws) {
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
    const int tiles = s_ws[lo + 1] - s_ws[lo];
    const int local = w - s_ws[lo] * nt;
    const int m_idx = local % tiles;
    it.n_idx = local / tiles;
    it.row0 = s_off[lo] + m_idx * kTileM;
    const int left = s_off[lo + 1] - it.row0;
    it.rows = left < kTileM ? left : kTileM;
    return it;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int MODE>  // 0: gate/up + SwiGLU -> H; 1: down + weighted scatter -> y
__global__ void __launch_bounds__(kGemmThreads, 1) grouped_gemm_kernel(const __grid_constant__ GroupedGemmParams p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kStages];
    __shared__ __align__(8) uint64_t empty_bar[kStages];
    __shared__ __align__(8) uint64_t tfull_bar[2];
    __shared__ __align__(8) uint64_t tempty_bar[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int s_off[kMaxGroups + 1];
    __shared__ int s_ws[kMaxGroups + 1];

    unsigned char* tiles =
        reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.G;

    for (int i = threadIdx.x; i <= G; i += kGemmThreads) {
        s_off[i] = p.offsets[i];
        s_ws[i] = p.work_start[i];
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(&full_bar[s], 1);
            ptx::mbar_init(&empty_bar[s], 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(&tfull_bar[s], 1);
            ptx::mbar_init(&tempty_bar[s], 4);
        }
        abort_s = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&p.tm_a);
        ptx::prefetch_tmap(&p.tm_b0);
        if (MODE == 0) {
            ptx::prefetch_tmap(&p.tm_a2);
            ptx::prefetch_tmap(&p.tm_b1);
        }
    }
    if (warp == 1) {
        ptx::tmem_alloc(&tmem_base_s, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    const int nt = p.n_ntiles;
    const int total = s_ws[G] * nt;
    const int nkb = (MODE == 0 ? p.d : p.I) / kBK;
    volatile int* abort_flag = &abort_s;

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            int stage = 0, phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
                const WorkItem it = decode_work(w, G, nt, s_off, s_ws);
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ptx::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, p.status, 1)) {
                        ok = false;
                        break;
                    }
                    unsigned char* a_dst = tiles + stage * kStageBytes;
                    unsigned char* b_dst = a_dst + kATileBytes;
                    ptx::mbar_expect_tx(&full_bar[stage], kStageBytes);
                    if (MODE == 0) {
                        if (it.g < p.n_routed) ptx::tma_load_2d(a_dst, &p.tm_a, &full_bar[stage], kb * kBK, it.row0);
                        else ptx::tma_load_2d(a_dst, &p.tm_a2, &full_bar[stage], kb * kBK, it.row0 - p.R);
                        const int brow = it.g * p.I + it.n_idx * 128;
                        ptx::tma_load_2d(b_dst, &p.tm_b0, &full_bar[stage], kb * kBK, brow);
                        ptx::tma_load_2d(b_dst + 128 * 128, &p.tm_b1, &full_bar[stage], kb * kBK, brow);
                    } else {
                        ptx::tma_load_2d(a_dst, &p.tm_a, &full_bar[stage], kb * kBK, it.row0);
                        ptx::tma_load_2d(b_dst, &p.tm_b0, &full_bar[stage], kb * kBK, it.g * p.d + it.n_idx * 256);
                    }
                    if (++stage == kStages) {
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
            constexpr uint32_t idesc = ptx::make_idesc_bf16(128, 256);
            int stage = 0, phase = 0, iter = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < total && ok; w += gridDim.x, ++iter) {
                const int as = iter & 1, aphase = (iter >> 1) & 1;
                if (!ptx::mbar_wait(&tempty_bar[as], aphase ^ 1, abort_flag, p.status, 2)) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + as * 256;
                for (int kb = 0; kb < nkb; ++kb) {
                    if (!ptx::mbar_wait(&full_bar[stage], phase, abort_flag, p.status, 3)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t a_addr = ptx::smem_u32(tiles + stage * kStageBytes);
                    const uint64_t adesc = ptx::make_kmajor_sw128_desc(a_addr);
                    const uint64_t bdesc = ptx::make_kmajor_sw128_desc(a_addr + kATileBytes);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k)
                        ptx::umma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0);
                    ptx::umma_commit(&empty_bar[stage]);
                    if (++stage == kStages) {
                        stage = 0;
                        phase ^= 1;
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
        for (int w = blockIdx.x; w < total; w += gridDim.x, ++iter) {
            const int as = iter & 1, aphase = (iter >> 1) & 1;
            const WorkItem it = decode_work(w, G, nt, s_off, s_ws);
            if (!ptx::mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status, 4)) break;
            ptx::tc_fence_after();
            const int row = q * 32 + lane;
            const bool valid = row < it.rows;
            const int64_t grow = (int64_t)it.row0 + row;
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
                int tok = 0;
                float wv = 0.f;
                if (valid) {
                    tok = p.row_tok[grow];
                    wv = p.row_w[grow];
                }
#pragma unroll 1
                for (int c = 0; c < 8; ++c) {
                    uint32_t v[32];
                    ptx::tmem_ld32(taddr + c * 32, v);
                    ptx::tmem_ld_wait();
                    const int col0 = it.n_idx * 256 + c * 32;
                    if (valid && col0 < p.d) {
                        if (p.y32 != nullptr) {
                            float* dst = p.y32 + (int64_t)tok * p.d + col0;
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                ptx::red_add_v4(dst + 4 * j, wv * __uint_as_float(v[4 * j]),
                                                wv * __uint_as_float(v[4 * j + 1]), wv * __uint_as_float(v[4 * j + 2]),
                                                wv * __uint_as_float(v[4 * j + 3]));
                        } else {
                            uint32_t pk[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                pk[j] = pack_bf16(wv * __uint_as_float(v[2 * j]), wv * __uint_as_float(v[2 * j + 1]));
                            uint4* dst = reinterpret_cast<uint4*>(p.y + (int64_t)tok * p.d + col0);
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
    ptx::tc_fence_before();
    __syncthreads();
    if (abort_s) __nanosleep(100000);  // let any copy still in flight land before shared memory is released
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

static cudaError_t launch_gemm(const GroupedGemmParams& p, int grid, cudaStream_t s, int mode) {
    cudaError_t err;
    if (mode == 0) {
        err = cudaFuncSetAttribute(grouped_gemm_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
        if (err != cudaSuccess) return err;
        grouped_gemm_kernel<0><<<grid, kGemmThreads, kGemmSmem, s>>>(p);
    } else {
        err = cudaFuncSetAttribute(grouped_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
        if (err != cudaSuccess) return err;
        grouped_gemm_kernel<1><<<grid, kGemmThreads, kGemmSmem, s>>>(p);
    }
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_grouped_gemm1(const GroupedGemmParams& p, int grid, cudaStream_t s) {
    return launch_gemm(p, grid, s, 0);
}
cudaError_t launch_grouped_gemm2(const GroupedGemmParams& p, int grid, cudaStream_t s) {
    return launch_gemm(p, grid, s, 1);
}

}  // namespace exfold
