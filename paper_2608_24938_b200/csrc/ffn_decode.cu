// Decode expert FFN over the expert pool only (Eq. 1 and Eq. 4 after the Eq. 14 remap): a
// weight-streaming pair of kernels bound by HBM bandwidth on the pool's weight bytes.
//
// The few tokens of a decode batch are the N dimension of the MMA ("swap-AB"): a 128-row slab
// of expert weights is the M operand, streamed once from HBM by TMA in 16 KB tiles; the
// (gathered) activations of the expert's tokens are the tiny second operand, re-read from L2.
//
//   gate/up kernel  work item = (pool expert, 128 intermediate features): full reduction over d,
//                   SwiGLU in the epilogue, H[row, feature] written as bf16.
//   down kernel     work item = (pool expert, 128 output features, K split): partial reduction
//                   over a slice of I, rows scaled by the remapped weight and added to the fp32
//                   accumulator y32[token] with coalesced reductions.
//
// Persistent CTAs, same warp roles and mbarrier hand-off as the prefill GEMMs.
#include "common.cuh"
#include "ptx.cuh"

namespace exfold {

namespace {

constexpr int kBK = 64;
constexpr int kWTileBytes = 128 * kBK * 2;  // 16 KB weight tile
constexpr int kMaxStages = 8;
constexpr int kDecThreads = 192;
constexpr int kTmemCols = 512;
constexpr int kSmemBudget = 200 * 1024;

template <int MODE>  // 0: gate/up, 1: down
__global__ void __launch_bounds__(kDecThreads, 1) decode_ffn_kernel(const __grid_constant__ DecodeFfnParams p) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ __align__(8) uint64_t tfull_bar[2];
    __shared__ __align__(8) uint64_t tempty_bar[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ int s_off[kMaxGroups + 1];
    __shared__ int s_exp[kMaxGroups + 1];

    unsigned char* tiles =
        reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NB = p.NB;
    const int act_bytes = NB * kBK * 2;
    const int n_w = MODE == 0 ? 2 : 1;  // weight tiles per stage
    const int stage_bytes = n_w * kWTileBytes + ((act_bytes + 1023) & ~1023);
    int stages = kSmemBudget / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    const int acc_stages = NB <= 128 ? 2 : 1;
    int G = *p.n_groups;
    if (G > p.max_groups) G = p.max_groups;

    for (int i = threadIdx.x; i <= G; i += kDecThreads) {
        s_off[i] = p.grp_off[i];
        s_exp[i] = i < G ? p.grp_expert[i] : 0;
    }
    if (threadIdx.x == 0) {
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
        ptx::prefetch_tmap(&p.tm_w0);
        ptx::prefetch_tmap(&p.tm_act);
        if (MODE == 0) ptx::prefetch_tmap(&p.tm_w1);
    }
    if (warp == 1) {
        ptx::tmem_alloc(&tmem_base_s, kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    volatile int* abort_flag = &abort_s;

    // work decomposition
    const int out_dim = MODE == 0 ? p.I : p.d;   // features produced (M of the MMA)
    const int red_dim = MODE == 0 ? p.d : p.I;   // reduction length
    const int n_slices = (out_dim + 127) / 128;
    const int ks = MODE == 0 ? 1 : p.ksplit;
    const int nkb_all = red_dim / kBK;
    const int kb_per = (nkb_all + ks - 1) / ks;
    const int per_group = n_slices * ks;
    const int total = G * per_group;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0, phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < total && ok; w += gridDim.x) {
                const int g = w / per_group, rem = w % per_group;
                const int slice = rem / ks, kpart = rem % ks;
                const int e = s_exp[g];
                const int kb0 = kpart * kb_per;
                const int kb1 = min(nkb_all, kb0 + kb_per);
                const int wrow = e * out_dim + slice * 128;
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!ptx::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, p.status, 11)) {
                        ok = false;
                        break;
                    }
                    unsigned char* dst = tiles + stage * stage_bytes;
                    ptx::mbar_expect_tx(&full_bar[stage], n_w * kWTileBytes + act_bytes);
                    ptx::tma_load_2d(dst, &p.tm_w0, &full_bar[stage], kb * kBK, wrow);
                    if (MODE == 0) ptx::tma_load_2d(dst + kWTileBytes, &p.tm_w1, &full_bar[stage], kb * kBK, wrow);
                    ptx::tma_load_2d(dst + n_w * kWTileBytes, &p.tm_act, &full_bar[stage], kb * kBK, s_off[g]);
                    if (++stage == stages) {
                        stage = 0;
                        phase ^= 1;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = ptx::make_idesc_bf16(128, NB);
            int stage = 0, phase = 0, iter = 0;
            bool ok = true;
            for (int w = blockIdx.x; w < total && ok; w += gridDim.x, ++iter) {
                const int rem = w % per_group;
                const int kpart = rem % ks;
                const int kb0 = kpart * kb_per;
                const int kb1 = min(nkb_all, kb0 + kb_per);
                const int as = acc_stages == 2 ? (iter & 1) : 0;
                const int aphase = acc_stages == 2 ? ((iter >> 1) & 1) : (iter & 1);
                if (!ptx::mbar_wait(&tempty_bar[as], aphase ^ 1, abort_flag, p.status, 12)) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + as * 256;
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!ptx::mbar_wait(&full_bar[stage], phase, abort_flag, p.status, 13)) {
                        ok = false;
                        break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t base = ptx::smem_u32(tiles + stage * stage_bytes);
                    const uint64_t w0desc = ptx::make_kmajor_sw128_desc(base);
                    const uint64_t actdesc = ptx::make_kmajor_sw128_desc(base + n_w * kWTileBytes);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
                        const uint32_t acc = (kb > kb0 || k > 0) ? 1u : 0u;
                        ptx::umma_bf16(d_tmem, w0desc + 2 * k, actdesc + 2 * k, idesc, acc);
                        if (MODE == 0) {
                            const uint64_t w1desc = ptx::make_kmajor_sw128_desc(base + kWTileBytes);
                            ptx::umma_bf16(d_tmem + NB, w1desc + 2 * k, actdesc + 2 * k, idesc, acc);
                        }
                    }
                    ptx::umma_commit(&empty_bar[stage]);
                    if (++stage == stages) {
                        stage = 0;
                        phase ^= 1;
                    }
                }
                if (ok) ptx::umma_commit(&tfull_bar[as]);
            }
        }
        __syncwarp();
    } else {
        const int q = warp & 3;
        int iter = 0;
        for (int w = blockIdx.x; w < total; w += gridDim.x, ++iter) {
            const int g = w / per_group, rem = w % per_group;
            const int slice = rem / ks;
            const int as = acc_stages == 2 ? (iter & 1) : 0;
            const int aphase = acc_stages == 2 ? ((iter >> 1) & 1) : (iter & 1);
            const int kpart = rem % ks;
            const bool empty_k = kpart * kb_per >= nkb_all;  // a K split with no work: nothing was accumulated
            if (!ptx::mbar_wait(&tfull_bar[as], aphase, abort_flag, p.status, 14)) break;
            ptx::tc_fence_after();
            const int row0 = s_off[g];
            const int n_e = s_off[g + 1] - row0;
            const int feat = slice * 128 + q * 32 + lane;
            const bool valid = feat < out_dim && !empty_k;
            const uint32_t taddr = tmem_base + as * 256 + ((uint32_t)(q * 32) << 16);
            for (int c0 = 0; c0 < NB && c0 < n_e; c0 += 16) {
                if (MODE == 0) {
                    uint32_t gv[16], uv[16];
                    ptx::tmem_ld16(taddr + c0, gv);
                    ptx::tmem_ld16(taddr + NB + c0, uv);
                    ptx::tmem_ld_wait();
                    if (valid) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            if (c0 + j < n_e) {
                                float g0 = __uint_as_float(gv[j]), u0 = __uint_as_float(uv[j]);
                                float h0 = __fdividef(g0, 1.0f + __expf(-g0)) * u0;
                                p.H[(size_t)(row0 + c0 + j) * p.I + feat] = __float2bfloat16_rn(h0);
                            }
                        }
                    }
                } else {
                    uint32_t v[16];
                    ptx::tmem_ld16(taddr + c0, v);
                    ptx::tmem_ld_wait();
                    if (valid) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            if (c0 + j < n_e) {
                                const int tok = p.row_tok[row0 + c0 + j];
                                const float wv = p.row_w[row0 + c0 + j];
                                ptx::red_add_f32(p.y32 + (size_t)tok * p.d + feat, wv * __uint_as_float(v[j]));
                            }
                        }
                    }
                }
            }
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&tempty_bar[as]);
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (abort_s) __nanosleep(100000);
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

static int decode_smem_bytes() { return kSmemBudget + 1024; }

cudaError_t launch_decode_gateup(const DecodeFfnParams& p, int grid, cudaStream_t s) {
    cudaError_t err = cudaFuncSetAttribute(decode_ffn_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           decode_smem_bytes());
    if (err != cudaSuccess) return err;
    decode_ffn_kernel<0><<<grid, kDecThreads, decode_smem_bytes(), s>>>(p);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_decode_down(const DecodeFfnParams& p, int grid, cudaStream_t s) {
    cudaError_t err = cudaFuncSetAttribute(decode_ffn_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           decode_smem_bytes());
    if (err != cudaSuccess) return err;
    decode_ffn_kernel<1><<<grid, kDecThreads, decode_smem_bytes(), s>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace exfold
