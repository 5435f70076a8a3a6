// Offline calibration of the pairwise scalar projector (Eq. 6-9): per ordered pair (s,t) of
// experts observed on the same calibration token, with u = E_s(x), v = E_t(x) and token
// weight w = |u|, accumulate A = sum w<v,u>, B = sum w|v|^2, C = sum w|u|^2 in double;
// then S = clip(A / (B + lambda)), L = max(0, C - 2 S A + S^2 B) / (C + eps).
#include "common.cuh"

namespace exfold {

namespace {

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// one CTA per calibration token; warps take the ordered pairs of that token's experts
__global__ void __launch_bounds__(256) calib_stats_kernel(CalibStatsParams p) {
    const int64_t i = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int Ke = p.Ke, d = p.d, N = p.N;
    const float* base = p.out + (size_t)i * Ke * d;
    const int32_t* ids = p.ids + i * Ke;
    for (int q = warp; q < Ke * Ke; q += nwarps) {
        const int a = q / Ke, b = q % Ke;
        const float* u = base + (size_t)a * d;  // source output
        const float* v = base + (size_t)b * d;  // target output
        double uu = 0.0, vu = 0.0, vv = 0.0;
        for (int c = lane; c < d; c += 32) {
            double uc = (double)u[c], vc = (double)v[c];
            uu += uc * uc;
            vu += vc * uc;
            vv += vc * vc;
        }
        uu = warp_sum_d(uu);
        vu = warp_sum_d(vu);
        vv = warp_sum_d(vv);
        if (lane == 0) {
            const double wi = sqrt(uu);
            const int s = ids[a], t = ids[b];
            if (a == b) {
                atomicAdd(&p.H[s], wi);
                atomicAdd(&p.hc[s], 1);
            } else {
                const size_t pq = (size_t)s * N + t;
                atomicAdd(&p.A[pq], wi * vu);
                atomicAdd(&p.Bv[pq], wi * vv);
                atomicAdd(&p.C[pq], wi * uu);
                atomicAdd(&p.cnt[pq], 1);
            }
        }
    }
}

__global__ void calib_finalize_kernel(CalibStatsParams p, exfold_calib_opts o, float* S, float* L, float* h,
                                      float* lnh, int32_t* n_obs, int32_t* unobserved) {
    const int N = p.N;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < N * N) {
        const int s = idx / N, t = idx % N;
        float sv, lv;
        if (s == t) {
            sv = 1.0f;
            lv = 0.0f;
        } else if (p.cnt[idx] == 0) {
            sv = 0.0f;
            lv = 1e30f;
        } else {
            double a = p.A[idx], b = p.Bv[idx], c = p.C[idx];
            double sc = a / (b + (double)o.lambda);
            if (sc < (double)o.clip_lo) sc = (double)o.clip_lo;
            if (sc > (double)o.clip_hi) sc = (double)o.clip_hi;
            double num = c - 2.0 * sc * a + sc * sc * b;
            if (num < 0.0) num = 0.0;
            sv = (float)sc;
            lv = (float)(num / (c + (double)o.eps));
        }
        S[idx] = sv;
        L[idx] = lv;
        if (n_obs) n_obs[idx] = p.cnt[idx];
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        double hsum = 0.0;
        int hn = 0, un = 0;
        for (int e = 0; e < N; ++e)
            if (p.hc[e] > 0) {
                hsum += p.H[e] / (double)p.hc[e];
                hn++;
            }
        for (int e = 0; e < N; ++e) {
            double he;
            if (p.hc[e] > 0) he = p.H[e] / (double)p.hc[e];
            else {
                he = hn ? hsum / hn : 1.0;
                un++;
            }
            float hf = (float)he;
            h[e] = hf;
            lnh[e] = (float)log((double)hf);
        }
        *unobserved = un;
    }
}

// ids[i][e] = e: every expert sees every token (common-input calibration)
__global__ void iota_ids_kernel(int32_t* ids, int64_t m, int N) {
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < m * N) ids[i] = (int32_t)(i % N);
}

}  // namespace

cudaError_t launch_calib_stats(const CalibStatsParams& p, cudaStream_t s) {
    if (p.m == 0) return cudaSuccess;
    calib_stats_kernel<<<(unsigned)p.m, 256, 0, s>>>(p);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_calib_finalize(const CalibStatsParams& p, const exfold_calib_opts& o, float* S, float* L,
                                  float* h, float* lnh, int32_t* n_obs, int32_t* unobserved, cudaStream_t s) {
    const int n = p.N * p.N;
    calib_finalize_kernel<<<(n + 255) / 256, 256, 0, s>>>(p, o, S, L, h, lnh, n_obs, unobserved);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_iota_ids(int32_t* ids, int64_t m, int N, cudaStream_t s) {
    const int64_t n = m * N;
    if (n == 0) return cudaSuccess;
    iota_ids_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(ids, m, N);
    count_launch();
    return cudaGetLastError();
}

}  // namespace exfold
