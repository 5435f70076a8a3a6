// Offline calibration of the pairwise scalar projector (Eq. 6-9): per ordered pair (s,t) of
// experts observed on the same calibration token, with u = E_s(x), v = E_t(x) and token
// weight w = |u|, accumulate A = sum w<v,u>, B = sum w|v|^2, C = sum w|u|^2 in double;
// then S = clip(A / (B + lambda)), L = max(0, C - 2 S A + S^2 B) / (C + eps).
#include "common.cuh"

#include <algorithm>

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
    const int32_t* ids = p.ids + i * Ke;
    const int32_t* inv = p.inv_pos ? p.inv_pos + i * Ke : nullptr;
    for (int q = warp; q < Ke * Ke; q += nwarps) {
        const int a = q / Ke, b = q % Ke;
        const int64_t ra = inv ? (int64_t)inv[a] : i * p.tok_stride + a * p.slot_stride;
        const int64_t rb = inv ? (int64_t)inv[b] : i * p.tok_stride + b * p.slot_stride;
        const float* u = p.out + ra * d;  // source output
        const float* v = p.out + rb * d;  // target output
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

// ---- common-input mode (slot a = expert a for every token), many experts: the pair sums as Gram products.
// A[s][t] = sum_i w_is <o_is, o_it>,  B[s][t] = sum_i w_is |o_it|^2,  C[s][t] = sum_i w_is^3,  w_is = |o_is|.
// Only A needs the off-diagonal inner products; B and C follow from the per-token squared norms.

// nrm[i][a] = |o_ia|^2 in double; one warp per (token, expert)
__global__ void __launch_bounds__(256) calib_norms_kernel(CalibStatsParams p, double* __restrict__ nrm) {
    const int64_t w = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (w >= p.m * p.Ke) return;
    const int64_t i = w / p.Ke;
    const int a = (int)(w % p.Ke);
    const float* u = p.out + (i * p.tok_stride + a * p.slot_stride) * p.d;
    double uu = 0.0;
    for (int c = lane; c < p.d; c += 32) {
        const double uc = (double)u[c];
        uu += uc * uc;
    }
    uu = warp_sum_d(uu);
    if (lane == 0) nrm[w] = uu;
}

// Each CTA walks its share of the tokens and keeps a 128 x 128 block of A in registers (4 x 4 per thread,
// 32 x 32 threads); 16-column chunks of the token's outputs are staged in shared memory, the source side
// already scaled by its weight w_is (in double, so nothing is rounded before the double accumulation).
__global__ void __launch_bounds__(1024, 1) calib_gram_kernel(CalibStatsParams p, const double* __restrict__ nrm) {
    __shared__ double sa[128][17];
    __shared__ float sb[128][17];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int lx = threadIdx.x & 15, ly = threadIdx.x >> 4;  // loader coordinates: 16 columns x 64 rows
    const int Ke = p.Ke, d = p.d, N = p.N;
    for (int ab = 0; ab < Ke; ab += 128)
        for (int bb = 0; bb < Ke; bb += 128) {
            double acc[4][4];
#pragma unroll
            for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) acc[ii][jj] = 0.0;
            for (int64_t i = blockIdx.x; i < p.m; i += gridDim.x) {
                for (int c0 = 0; c0 < d; c0 += 16) {
                    __syncthreads();
                    const bool cin = c0 + lx < d;
                    for (int r = ly; r < 128; r += 64) {
                        const int a = ab + r, b = bb + r;
                        double av = 0.0;
                        float bv = 0.f;
                        if (cin && a < Ke)
                            av = sqrt(nrm[i * Ke + a]) *
                                 (double)p.out[(i * p.tok_stride + a * p.slot_stride) * d + c0 + lx];
                        if (cin && b < Ke) bv = p.out[(i * p.tok_stride + b * p.slot_stride) * d + c0 + lx];
                        sa[r][lx] = av;
                        sb[r][lx] = bv;
                    }
                    __syncthreads();
#pragma unroll 4
                    for (int c = 0; c < 16; ++c) {
                        double a4[4], b4[4];
#pragma unroll
                        for (int ii = 0; ii < 4; ++ii) a4[ii] = sa[ty + 32 * ii][c];
#pragma unroll
                        for (int jj = 0; jj < 4; ++jj) b4[jj] = (double)sb[tx + 32 * jj][c];
#pragma unroll
                        for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj) acc[ii][jj] += a4[ii] * b4[jj];
                    }
                }
            }
#pragma unroll
            for (int ii = 0; ii < 4; ++ii)
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int a = ab + ty + 32 * ii, b = bb + tx + 32 * jj;
                    if (a < Ke && b < Ke && a != b) atomicAdd(&p.A[(size_t)a * N + b], acc[ii][jj]);
                }
        }
}

// B, C, the pair counts and the per-expert norm sums from the squared norms; one thread per ordered pair
__global__ void __launch_bounds__(256) calib_common_finish_kernel(CalibStatsParams p, const double* __restrict__ nrm) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int Ke = p.Ke, N = p.N;
    if (idx >= Ke * Ke) return;
    const int s = idx / Ke, t = idx % Ke;
    double bsum = 0.0, csum = 0.0, hsum = 0.0;
    for (int64_t i = 0; i < p.m; ++i) {
        const double ns = nrm[i * Ke + s], nt = nrm[i * Ke + t];
        const double w = sqrt(ns);
        bsum += w * nt;
        csum += w * ns;
        hsum += w;
    }
    if (s == t) {
        p.H[s] = hsum;
        p.hc[s] = (int32_t)p.m;
    } else {
        const size_t pq = (size_t)s * N + t;
        p.Bv[pq] = bsum;
        p.C[pq] = csum;
        p.cnt[pq] = (int32_t)p.m;
    }
}

// common-input mode on the grouped GEMMs: group e = all m tokens in order
__global__ void calib_common_rows_kernel(int32_t* offsets, int32_t* work_start, int64_t m, int N) {
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g <= N) {
        offsets[g] = (int32_t)(g * m);
        work_start[g] = (int32_t)(g * ((m + kTileM - 1) / kTileM));
    }
}

}  // namespace

cudaError_t launch_calib_common_rows(int32_t* offsets, int32_t* work_start, int64_t m, int N, cudaStream_t s) {
    calib_common_rows_kernel<<<(N + 1 + 255) / 256, 256, 0, s>>>(offsets, work_start, m, N);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_calib_stats_common(const CalibStatsParams& p, double* nrm, int sms, cudaStream_t s) {
    if (p.m == 0) return cudaSuccess;
    const int64_t warps = p.m * p.Ke;
    calib_norms_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, s>>>(p, nrm);
    count_launch();
    calib_gram_kernel<<<(unsigned)std::min<int64_t>(p.m, sms), 1024, 0, s>>>(p, nrm);
    count_launch();
    calib_common_finish_kernel<<<(p.Ke * p.Ke + 255) / 256, 256, 0, s>>>(p, nrm);
    count_launch();
    return cudaGetLastError();
}

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
