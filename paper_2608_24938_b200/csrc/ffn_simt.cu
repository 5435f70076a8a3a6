// SIMT (CUDA-core) expert FFN with fp32 accumulation, one CTA per route (Eq. 1).
// Serves the fp32 layers end to end (tensor cores would round fp32 inputs), the
// calibration pass (which needs each routed expert's unweighted output) and small
// on-device cross-checks of the bf16 tensor-core path. Also the final combine /
// conversion kernels (Eq. 3 / Eq. 4 weighted sums).
#include "common.cuh"

namespace exfold {

namespace {

__device__ __forceinline__ float ldf(const float* p, size_t i) { return __ldg(p + i); }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p, size_t i) {
    return __bfloat162float(p[i]);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

template <typename T>
__global__ void __launch_bounds__(256) simt_ffn_kernel(SimtFfnParams p) {
    extern __shared__ float sm[];
    float* xs = sm;          // [d]
    float* act = sm + p.d;   // [I]
    const int64_t row = blockIdx.x;
    grid_dep_launch();
    grid_dep_wait();
    const int64_t n_routed = p.T * p.Kr;
    int64_t tok;
    int e;
    if (row < n_routed) {
        tok = row / p.Kr;
        e = p.ids[row];
    } else {
        tok = row - n_routed;
        e = p.N;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const T* x = reinterpret_cast<const T*>(p.x) + (size_t)tok * p.d;
    for (int c = threadIdx.x; c < p.d; c += blockDim.x) xs[c] = ldf(x, c);
    __syncthreads();
    const T* wg = reinterpret_cast<const T*>(p.wg) + (size_t)e * p.I * p.d;
    const T* wu = reinterpret_cast<const T*>(p.wu) + (size_t)e * p.I * p.d;
    const T* wd = reinterpret_cast<const T*>(p.wd) + (size_t)e * p.d * p.I;
    for (int j = warp; j < p.I; j += nwarps) {
        float g = 0.f, u = 0.f;
        const size_t base = (size_t)j * p.d;
        for (int c = lane; c < p.d; c += 32) {
            float xv = xs[c];
            g = fmaf(ldf(wg, base + c), xv, g);
            u = fmaf(ldf(wu, base + c), xv, u);
        }
        g = warp_sum(g);
        u = warp_sum(u);
        if (lane == 0) act[j] = (g / (1.0f + expf(-g))) * u;
    }
    __syncthreads();
    float* out = p.out + (size_t)row * p.d;
    for (int r = warp; r < p.d; r += nwarps) {
        float o = 0.f;
        const size_t base = (size_t)r * p.I;
        for (int j = lane; j < p.I; j += 32) o = fmaf(ldf(wd, base + j), act[j], o);
        o = warp_sum(o);
        if (lane == 0) out[r] = o;
    }
}

// y[i][c] = sum_j w[i][j] out[i*Kr+j][c] (+ out[T*Kr + i][c] for the shared expert), slot order
template <typename T>
__global__ void combine_routes_kernel(const float* __restrict__ out, const float* __restrict__ w, int64_t Tn,
                                      int Kr, int d, int n_shared, T* __restrict__ y) {
    const int64_t i = blockIdx.x;
    grid_dep_launch();
    grid_dep_wait();
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
        float acc = 0.f;
        for (int j = 0; j < Kr; ++j) acc = fmaf(w[i * Kr + j], out[(size_t)(i * Kr + j) * d + c], acc);
        if (n_shared) acc += out[(size_t)(Tn * Kr + i) * d + c];
        if constexpr (sizeof(T) == 2) y[(size_t)i * d + c] = __float2bfloat16_rn(acc);
        else y[(size_t)i * d + c] = acc;
    }
}

// Eq. 4's weighted sum for the tensor-core path: GEMM-2 stored w~ * E(x) per route in bf16, sorted by
// expert; a token's routes are found through the inverse permutation and summed in fp32, slot order
// (a decode step with a K split: the `parts` planes of a row, in order, inside that).
// BATCHED: the row indices first, then up to eight row loads in flight together - for the few blocks of a decode
// step, where the chain index -> row -> next index is all there is (10 -> 3 us for 64 tokens); with thousands of
// tokens the plain loop is faster (more blocks per SM hide the chain; measured 50 vs 65 us on 8192 tokens).
template <bool BATCHED>
__global__ void __launch_bounds__(256) combine_rows_kernel(const __nv_bfloat16* __restrict__ O,
                                                           const int32_t* __restrict__ inv_pos, int64_t Tn, int Kr, int d,
                                                           int n_shared, const int32_t* __restrict__ shared0_dev,
                                                           int parts, int64_t part_rows, __nv_bfloat16* __restrict__ y) {
    const int64_t i = blockIdx.x;
    grid_dep_launch();
    grid_dep_wait();
    const int64_t shared0 = shared0_dev != nullptr ? (int64_t)*shared0_dev : Tn * Kr;
    const int n_src = Kr + (n_shared ? 1 : 0);
    for (int c = threadIdx.x * 8; c < d; c += blockDim.x * 8) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        auto add = [&](const uint4& v) {
            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 f = __bfloat1622float2(h2[q]);
                acc[2 * q] += f.x;
                acc[2 * q + 1] += f.y;
            }
        };
        if (BATCHED) {
            for (int j0 = 0; j0 < n_src; j0 += 8) {
                int64_t row[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int j = j0 + u;
                    row[u] = j < Kr ? (int64_t)inv_pos[i * Kr + j] : (j < n_src ? shared0 + i : -1);
                }
                for (int part = 0; part < parts; ++part) {
                    uint4 v[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (row[u] >= 0) v[u] = *reinterpret_cast<const uint4*>(O + (part * part_rows + row[u]) * d + c);
#pragma unroll
                    for (int u = 0; u < 8; ++u)  // slot order; a row < 0 is a slot merged into an earlier one
                        if (row[u] >= 0) add(v[u]);
                }
            }
        } else {  // prefill: every slot has a row of its own and there is one plane
            for (int j = 0; j <= Kr; ++j) {
                if (j == Kr && !n_shared) break;
                const int64_t row = j < Kr ? (int64_t)inv_pos[i * Kr + j] : shared0 + i;
                add(*reinterpret_cast<const uint4*>(O + row * d + c));
            }
        }
        uint4 o;
        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
        for (int u = 0; u < 4; ++u) o2[u] = __floats2bfloat162_rn(acc[2 * u], acc[2 * u + 1]);
        *reinterpret_cast<uint4*>(y + i * d + c) = o;
    }
}

// r[i][e] = <W_r[e], x_i>, fp32 accumulation in a fixed order, one warp per (token, expert): fp32 layers, and
// bf16 batches too small to fill the tensor-core kernel (a single 128-row tile would walk K on one SM)
template <typename T>
__global__ void __launch_bounds__(256) router_simt_kernel(const T* __restrict__ x, const T* __restrict__ wr, int64_t Tn,
                                                          int N, int d, float* __restrict__ out) {
    const int64_t w = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    grid_dep_launch();
    grid_dep_wait();  // x may be the output of the previous layer's last kernel
    if (w >= Tn * N) return;
    const int64_t i = w / N;
    const int e = (int)(w % N);
    const T* xi = x + i * d;
    const T* we = wr + (size_t)e * d;
    float acc = 0.f;
    if constexpr (sizeof(T) == 2) {  // bf16: 8 elements (16 bytes) per lane and step; d is a multiple of 64
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
    } else {
        for (int c = lane; c < d; c += 32) acc = fmaf((float)we[c], (float)xi[c], acc);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) out[w] = acc;
}

}  // namespace

cudaError_t launch_router_simt(const void* x, const void* wr, int dtype, int64_t T, int N, int d, float* out,
                               cudaStream_t s) {
    const int64_t warps = T * N;
    if (warps == 0) return cudaSuccess;
    const unsigned grid = (unsigned)((warps + 7) / 8);
    if (dtype == EXFOLD_BF16)
        return launch_pdl(router_simt_kernel<__nv_bfloat16>, grid, 256, 0, s, reinterpret_cast<const __nv_bfloat16*>(x),
                          reinterpret_cast<const __nv_bfloat16*>(wr), T, N, d, out);
    return launch_pdl(router_simt_kernel<float>, grid, 256, 0, s, reinterpret_cast<const float*>(x),
                      reinterpret_cast<const float*>(wr), T, N, d, out);
}

cudaError_t launch_simt_ffn(const SimtFfnParams& p, cudaStream_t s) {
    const int64_t rows = p.T * p.Kr + p.T * p.n_shared;
    if (rows == 0) return cudaSuccess;
    const size_t smem = (size_t)(p.d + p.I) * sizeof(float);
    cudaError_t err;
    if (p.dtype == EXFOLD_BF16) {
        err = cudaFuncSetAttribute(simt_ffn_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)smem);
        if (err != cudaSuccess) return err;
        return launch_pdl(simt_ffn_kernel<__nv_bfloat16>, (unsigned)rows, 256, smem, s, p);
    } else {
        err = cudaFuncSetAttribute(simt_ffn_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return err;
        return launch_pdl(simt_ffn_kernel<float>, (unsigned)rows, 256, smem, s, p);
    }
}

cudaError_t launch_combine_routes(const float* out, const float* w, int64_t T, int Kr, int d, int n_shared,
                                  void* y, int dtype, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    if (dtype == EXFOLD_BF16)
        return launch_pdl(combine_routes_kernel<__nv_bfloat16>, (unsigned)T, 256, 0, s, out, w, T, Kr, d, n_shared,
                          reinterpret_cast<__nv_bfloat16*>(y));
    return launch_pdl(combine_routes_kernel<float>, (unsigned)T, 256, 0, s, out, w, T, Kr, d, n_shared,
                      reinterpret_cast<float*>(y));
}

cudaError_t launch_combine_rows(const __nv_bfloat16* O, const int32_t* inv_pos, int64_t T, int Kr, int d,
                                int n_shared, const int32_t* shared0_dev, int parts, int64_t part_rows,
                                __nv_bfloat16* y, cudaStream_t s) {
    if (T == 0) return cudaSuccess;
    if (T <= 1024 || parts > 1 || shared0_dev != nullptr)  // decode (merged slots are marked -1, K planes)
        return launch_pdl(combine_rows_kernel<true>, (unsigned)T, 256, 0, s, O, inv_pos, T, Kr, d, n_shared, shared0_dev,
                          parts, part_rows, y);
    return launch_pdl(combine_rows_kernel<false>, (unsigned)T, 256, 0, s, O, inv_pos, T, Kr, d, n_shared, shared0_dev, parts,
                      part_rows, y);
}

}  // namespace exfold
