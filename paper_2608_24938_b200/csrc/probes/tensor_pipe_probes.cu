// Rate probes for the design of the grouped GEMMs (development tool, not part of the library):
//   mma   back-to-back tcgen05.mma (M128 x N x K16, bf16) of one thread on resident shared-memory operands, by N and by
//         the number of k-blocks (4 MMAs + commit) in flight, alone and beside bulk copies into other shared memory
//   pair  the same for tcgen05.mma.cta_group::2 (M256 x N256 x K16 over a cluster of two CTAs)
//   copy  cycles per iteration of a one-thread producer loop {try_wait, expect_tx, n bulk copies}, by n, chunk size and
//         number of issuing threads (each in a warp of its own)
// Every wait is bounded. Build and run: python -m paper_2608_24938_b200.rate_probes
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <cuda_bf16.h>
#include "../ptx.cuh"

using namespace exfold;

struct ProbeOut {
    unsigned long long cycles, ns, err, copy_bytes, copy_cycles;
};

__device__ __forceinline__ bool spin_wait(uint64_t* bar, uint32_t parity, int limit = 1 << 20) {
    int spins = 0;
    while (!ptx::mbar_try_wait(bar, parity))
        if (++spins > limit) return false;
    return true;
}
__device__ __forceinline__ void fill_random(__nv_bfloat16* a, int n, int tid, int nthreads) {
    for (int i = tid; i < n; i += nthreads) {
        uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x * 977u;
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        a[i] = __float2bfloat16(((int)(h & 0xffff) - 32768) * (1.0f / 32768.0f));
    }
}
__device__ __forceinline__ void bulk_copy(uint32_t dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(ptx::smem_u32(bar)) : "memory");
}

// ---------------------------------------------------------------- mma: one CTA per SM, thread 0 issues
// Operands: 2 stages of [128 x 64 A | 256 x 64 B] (48 KB each) read by the MMAs; with `copies`, thread 64 streams
// 48 KB bulk copies from an L2-resident window into two more stages, pausing `delay` cycles after each.
// (the loop of the issuing thread must stay short: a runtime modulo in it already costs more than the MMAs take)
template <int N, int IN_FLIGHT>
__global__ void __launch_bounds__(128, 1) mma_probe(int iters, int copies, int delay, const uint8_t* src, ProbeOut* out) {
    constexpr int in_flight = IN_FLIGHT;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bars[8], cbars[2];
    __shared__ uint32_t tmem_base;
    __shared__ volatile int done;
    const int tid = threadIdx.x, warp = tid >> 5;
    fill_random((__nv_bfloat16*)base, 2 * (128 + 256) * 64, tid, blockDim.x);
    if (tid == 0) {
        for (int i = 0; i < 8; ++i) ptx::mbar_init(&bars[i], 1);
        ptx::mbar_init(&cbars[0], 1);
        ptx::mbar_init(&cbars[1], 1);
        ptx::fence_mbar_init();
        done = 0;
    }
    if (warp == 0) {
        ptx::tmem_alloc(&tmem_base, 512);
        ptx::tmem_relinquish();
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tb = tmem_base;
    if (tid == 0) {
        const uint32_t a0 = ptx::smem_u32(base);
        constexpr uint32_t idesc = ptx::make_idesc_bf16(128, N);
        unsigned long long t0 = clock64(), g0 = ptx::globaltimer_ns();
        int bad = 0;
        for (int it = 0; it < iters && !bad; ++it) {
            const int slot = it % in_flight;
            if (it >= in_flight && !spin_wait(&bars[slot], ((it / in_flight) - 1) & 1)) { bad = 1; break; }
            const uint64_t ad = ptx::make_kmajor_sw128_desc(a0 + (it & 1) * 49152);
            const uint64_t bd = ptx::make_kmajor_sw128_desc(a0 + 16384 + (it & 1) * 49152);
#pragma unroll
            for (int k = 0; k < 4; ++k) ptx::umma_bf16(tb, ad + 2 * k, bd + 2 * k, idesc, 1u);
            ptx::umma_commit(&bars[slot]);
        }
        for (int s = 0; s < in_flight && !bad; ++s) {
            if (iters <= s) continue;
            const int n = (iters - s + in_flight - 1) / in_flight;
            if (!spin_wait(&bars[s], (n - 1) & 1, 1 << 22)) bad = 1;
        }
        out[blockIdx.x].cycles = clock64() - t0;
        out[blockIdx.x].ns = ptx::globaltimer_ns() - g0;
        out[blockIdx.x].err = bad;
        done = 1;
    } else if (copies && tid == 64) {
        const uint8_t* win = src + (size_t)blockIdx.x * (256u << 10);
        unsigned long long bytes = 0, c0 = clock64();
        int n = 0, bad = 0;
        while (!done && n < (1 << 22) && !bad) {
            const int j = n & 1;
            if (n >= 2 && !spin_wait(&cbars[j], ((n >> 1) - 1) & 1)) { bad = 1; break; }
            ptx::mbar_expect_tx(&cbars[j], 49152);
            const uint32_t dst = ptx::smem_u32(base + (2 + j) * 49152);
#pragma unroll
            for (int c = 0; c < 3; ++c) bulk_copy(dst + c * 16384, win + ((size_t)((n * 3 + c) & 15) << 14), 16384, &cbars[j]);
            bytes += 49152;
            ++n;
            if (delay > 0) {
                const long long t = clock64();
                while (clock64() - t < delay) {}
            }
        }
        for (int j = 0; j < 2 && !bad; ++j) {  // the copies still in flight
            const int cnt = (n - j + 1) / 2;
            if (cnt > 0 && !spin_wait(&cbars[j], (cnt - 1) & 1, 1 << 22)) bad = 1;
        }
        out[blockIdx.x].copy_bytes = bytes;
        out[blockIdx.x].copy_cycles = clock64() - c0;
        if (bad) out[blockIdx.x].err = 2;
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    if (warp == 0) ptx::tmem_dealloc(tb, 512);
}

template <int N, int IN_FLIGHT>
static void run_mma(const char* name, int grid, int iters, int copies, int delay, const uint8_t* src, ProbeOut* d,
                    ProbeOut* h) {
    const int smem = 4 * 49152 + 1024;
    cudaFuncSetAttribute(mma_probe<N, IN_FLIGHT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaMemset(d, 0, sizeof(ProbeOut) * 148);
    for (int rep = 0; rep < 2; ++rep) {
        mma_probe<N, IN_FLIGHT><<<grid, 128, smem>>>(iters, copies, delay, src, d);
        cudaError_t e = cudaDeviceSynchronize();
        if (e != cudaSuccess) { printf("%s: CUDA error %s\n", name, cudaGetErrorString(e)); exit(1); }
    }
    cudaMemcpy(h, d, sizeof(ProbeOut) * 148, cudaMemcpyDeviceToHost);
    double cyc = 0, ns = 0, cb = 0, cc = 0; int bad = 0;
    for (int i = 0; i < grid; ++i) { cyc += h[i].cycles; ns += h[i].ns; bad += (int)h[i].err; cb += h[i].copy_bytes; cc += h[i].copy_cycles; }
    cyc /= grid; ns /= grid;
    const double kb = cyc / iters, ghz = cyc / ns;
    printf("%-44s SMs %3d: %6.1f cycles/k-block (%5.1f per MMA), %.3f GHz, %6.1f ns/k-block, %7.1f TFLOP/s", name, grid, kb,
           kb / 4, ghz, kb / ghz, grid * (2.0 * 128 * N * 64) * iters / ns * 1e-3);
    if (copies) printf(", copies %.1f KB per k-block", cc > 0 ? cb / cc * kb / 1024 : 0.0);
    printf("%s\n", bad ? "  WAIT LIMIT HIT" : "");
}

// ---------------------------------------------------------------- pair: clusters of two CTAs, the leader's thread 0 issues
// FUSED 1 / 2: the library's one-sequence k-block (4 MMAs with a poll before the last, commit) instead of separate
// instructions; 1 keeps this loop's own wait for the k-block issued four earlier (two barrier polls per k-block)
template <int FUSED>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128, 1) pair_probe(int iters, ProbeOut* out) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bars[5];
    __shared__ uint32_t tmem_base;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int rank = (int)ptx::cluster_ctarank();
    fill_random((__nv_bfloat16*)base, 4 * 256 * 64, tid, blockDim.x);  // 4 stages of [128 x 64 A | 128 x 64 half of B]
    if (tid == 0) {
        for (int i = 0; i < 5; ++i) ptx::mbar_init(&bars[i], 1);
        ptx::fence_mbar_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc_pair(&tmem_base, 512);
        ptx::tmem_relinquish_pair();
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync_all();
    ptx::tc_fence_after();
    const uint32_t tb = tmem_base;
    if (tid == 0 && rank == 0) {
        const uint32_t a0 = (ptx::smem_u32(base) & 0x3FFFFu) >> 4;
        const uint64_t hi = ptx::make_kmajor_sw128_desc(0) & 0xFFFFFFFF00000000ull;
        constexpr uint32_t idesc = ptx::make_idesc_bf16(256, 256);
        unsigned long long t0 = clock64(), g0 = ptx::globaltimer_ns();
        int bad = 0;
        for (int it = 0; it < iters && !bad; ++it) {
            const int slot = it & 3;
            // FUSED 2: the library sequence's own poll is the only barrier instruction of the loop, as in the kernel
            if (FUSED != 2 && it >= 4 && !spin_wait(&bars[slot], ((it >> 2) - 1) & 1)) { bad = 1; break; }
            const uint32_t a_lo = a0 + (uint32_t)(it & 3) * (32768u >> 4);
            if (FUSED) {  // polls bars[4] (never arrived on: parity 1 reads as complete); the commit goes to both CTAs
                ptx::umma_kblock_bf16_pair(tb, a_lo, a_lo + (16384u >> 4), (uint32_t)(hi >> 32), idesc, 1u, &bars[slot],
                                           &bars[4], 1u);
            } else {
                const uint64_t ad = hi | a_lo, bd = hi | (a_lo + (16384u >> 4));
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    asm volatile("tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, 1;" ::"r"(tb), "l"(ad + 2 * k),
                                 "l"(bd + 2 * k), "r"(idesc) : "memory");
                ptx::umma_commit_pair(&bars[slot], 1);  // the leader's barrier only
            }
        }
        for (int s = 0; s < 4 && !bad; ++s) {
            if (iters <= s) continue;
            if (!spin_wait(&bars[s], (((iters - s + 3) / 4) - 1) & 1, 1 << 22)) bad = 1;
        }
        out[blockIdx.x >> 1].cycles = clock64() - t0;
        out[blockIdx.x >> 1].ns = ptx::globaltimer_ns() - g0;
        out[blockIdx.x >> 1].err = bad;
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::cluster_sync_all();
    ptx::tc_fence_after();
    if (warp == 0) ptx::tmem_dealloc_pair(tb, 512);
}

// ---------------------------------------------------------------- copy: producer-loop cost
template <int NC>
__global__ void __launch_bounds__(128, 1) copy_probe(int iters, int chunk, int nthr, const uint8_t* src, ProbeOut* out) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bars[4][4];
    if (threadIdx.x == 0) {
        for (int i = 0; i < 16; ++i) ptx::mbar_init(&bars[0][0] + i, 1);
        ptx::fence_mbar_init();
    }
    __syncthreads();
    const int me = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0 && me < nthr) {  // each issuing thread: 4 buffers of NC * chunk bytes in its own 48 KB
        uint8_t* mybase = base + (size_t)me * 49152;
        const uint8_t* win = src + ((size_t)blockIdx.x * 4 + me) * (256 << 10);
        unsigned long long c0 = clock64(), bytes = 0;
        int bad = 0;
        for (int n = 0; n < iters && !bad; ++n) {
            const int j = n & 3;
            if (n >= 4 && !spin_wait(&bars[me][j], ((n >> 2) - 1) & 1)) { bad = 1; break; }
            ptx::mbar_expect_tx(&bars[me][j], NC * chunk);
#pragma unroll
            for (int c = 0; c < NC; ++c)
                bulk_copy(ptx::smem_u32(mybase + (size_t)(j * NC + c) * chunk), win + (size_t)((n * NC + c) & 15) * 16384, chunk,
                          &bars[me][j]);
            bytes += NC * chunk;
        }
        for (int j = 0; j < 4 && !bad; ++j) {
            if (iters <= j) continue;
            if (!spin_wait(&bars[me][j], (((iters - j + 3) / 4) - 1) & 1, 1 << 22)) bad = 1;
        }
        ProbeOut& o = out[blockIdx.x * 4 + me];
        o.cycles = clock64() - c0; o.copy_bytes = bytes; o.err = bad;
    }
    __syncthreads();
}
template <int NC>
static void run_copy(int grid, int chunk, int nthr, const uint8_t* src, ProbeOut* d, ProbeOut* h) {
    const int smem = 200 * 1024, iters = 8000;
    cudaFuncSetAttribute(copy_probe<NC>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaMemset(d, 0, sizeof(ProbeOut) * 148 * 4);
    for (int rep = 0; rep < 2; ++rep) {
        copy_probe<NC><<<grid, 128, smem>>>(iters, chunk, nthr, src, d);
        cudaError_t e = cudaDeviceSynchronize();
        if (e != cudaSuccess) { printf("CUDA error %s\n", cudaGetErrorString(e)); exit(1); }
    }
    cudaMemcpy(h, d, sizeof(ProbeOut) * 148 * 4, cudaMemcpyDeviceToHost);
    double cyc = 0, by = 0; int bad = 0, cnt = 0;
    for (int i = 0; i < grid * 4; ++i) if (h[i].cycles) { cyc += h[i].cycles; by += h[i].copy_bytes; bad += (int)h[i].err; ++cnt; }
    cyc /= cnt;
    printf("SMs %3d, issuing threads %d, %d x %5d B per iteration: %6.1f cycles per iteration, %6.1f B/cycle/SM%s\n", grid, nthr,
           NC, chunk, cyc / iters, by / grid / cyc, bad ? "  WAIT LIMIT HIT" : "");
}

int main(int argc, char** argv) {
    const char* what = argc > 1 ? argv[1] : "all";
    const bool all = !strcmp(what, "all");
    ProbeOut *d, *h = (ProbeOut*)malloc(sizeof(ProbeOut) * 148 * 4);
    cudaMalloc(&d, sizeof(ProbeOut) * 148 * 4);
    uint8_t* src;
    cudaMalloc(&src, (size_t)148 << 20);   // L2-resident windows: 256 KB per CTA (mma), 256 KB per issuing thread (copy)
    cudaMemset(src, 1, (size_t)148 << 20);
    if (all || !strcmp(what, "mma")) {
        printf("== tcgen05.mma cta_group::1, M128 x N x K16, operands resident in shared memory; a k-block = 4 MMAs + commit\n");
        for (int grid : {1, 148}) {
            run_mma<256, 8>("N=256, 8 k-blocks in flight", grid, 20000, 0, 0, src, d, h);
            run_mma<128, 8>("N=128, 8 k-blocks in flight", grid, 20000, 0, 0, src, d, h);
            run_mma<64, 8>("N=64,  8 k-blocks in flight", grid, 20000, 0, 0, src, d, h);
        }
        run_mma<256, 1>("N=256, 1 k-block in flight", 1, 20000, 0, 0, src, d, h);
        run_mma<256, 2>("N=256, 2 k-blocks in flight", 1, 20000, 0, 0, src, d, h);
        run_mma<256, 4>("N=256, 4 k-blocks in flight", 1, 20000, 0, 0, src, d, h);
    }
    if (all || !strcmp(what, "pair")) {
        printf("== tcgen05.mma cta_group::2, M256 x N256 x K16 over a cluster of two CTAs, operands resident, 4 k-blocks in flight\n");
        const int smem = 4 * 32768 + 1024 + 64 * 1024;
        cudaFuncSetAttribute(pair_probe<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        cudaFuncSetAttribute(pair_probe<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        cudaFuncSetAttribute(pair_probe<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        for (int fused : {0, 1, 2})
        for (int grid : {2, 148}) {
            for (int rep = 0; rep < 2; ++rep) {
                if (fused == 2) pair_probe<2><<<grid, 128, smem>>>(20000, d);
                else if (fused == 1) pair_probe<1><<<grid, 128, smem>>>(20000, d);
                else pair_probe<0><<<grid, 128, smem>>>(20000, d);
                cudaError_t e = cudaDeviceSynchronize();
                if (e != cudaSuccess) { printf("CUDA error %s\n", cudaGetErrorString(e)); return 1; }
            }
            cudaMemcpy(h, d, sizeof(ProbeOut) * 74, cudaMemcpyDeviceToHost);
            double cyc = 0, ns = 0; int bad = 0;
            for (int i = 0; i < grid / 2; ++i) { cyc += h[i].cycles; ns += h[i].ns; bad += (int)h[i].err; }
            const double kb = cyc / (grid / 2) / 20000, ghz = cyc / ns;
            printf("%s SMs %3d: %6.1f cycles/k-block (%5.1f per M256 MMA), %.3f GHz, %6.1f ns/k-block%s\n",
                   fused == 2 ? "library k-block sequence, one poll per k-block, " : fused == 1 ? "library k-block sequence, two polls per k-block," : "separate instructions, one poll per k-block,    ", grid, kb, kb / 4, ghz, kb / ghz,
                   bad ? "  WAIT LIMIT HIT" : "");
        }
    }
    if (all || !strcmp(what, "mma")) {
        printf("== the same (N=256, all SMs, ~12 ms) beside 48 KB bulk copies from L2, paced by a delay after each\n");
        run_mma<256, 8>("no copies", 148, 40000, 0, 0, src, d, h);
        for (int delay : {1200, 700, 400, 200, 0}) {
            char nm[64]; snprintf(nm, 64, "copies, delay %d cycles", delay);
            run_mma<256, 8>(nm, 148, 40000, 1, delay, src, d, h);
        }
    }
    if (all || !strcmp(what, "copy")) {
        printf("== one-thread producer loop {try_wait, expect_tx, n bulk copies}, 4 buffers per thread, source in L2\n");
        for (int grid : {1, 148})
            for (int nthr : {1, 2, 4}) {
                run_copy<1>(grid, 4096, nthr, src, d, h);
                run_copy<3>(grid, 4096, nthr, src, d, h);
                run_copy<1>(grid, 12288, nthr, src, d, h);
            }
    }
    return 0;
}
