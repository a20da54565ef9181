// Micro-benchmark: rate of TMA 1-D bulk copies L2 -> shared memory per SM against chunk size, ring depth and the
// number of issuing threads (one per warp, each with its own ring).  No division in the issue loops.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* b, int n) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(n)); }
__device__ __forceinline__ void mbar_expect(uint32_t b, uint32_t bytes) { asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b), "r"(bytes) : "memory"); }
__device__ __forceinline__ bool mbar_try(uint32_t b, uint32_t ph) {
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }" : "=r"(ok) : "r"(b), "r"(ph) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t b, uint32_t ph) {
    for (int i = 0; i < 20000000; ++i) if (mbar_try(b, ph)) return true;
    return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

constexpr int MAX_ISSUERS = 8, MAX_STAGES = 16;

__global__ void __launch_bounds__(256, 1) tma_rate_kernel(const uint8_t* __restrict__ data, size_t region, int chunk, int stages,
                                                          int issuers, int iters, unsigned long long* out_ns, int* err, int lanes_mode) {
    extern __shared__ __align__(1024) uint8_t smem[];
    __shared__ uint64_t bars[MAX_ISSUERS * MAX_STAGES];
    const uint8_t* base = data + static_cast<size_t>(blockIdx.x) * region;
    if (threadIdx.x == 0) {
        for (int i = 0; i < MAX_ISSUERS * MAX_STAGES; ++i) mbar_init(&bars[i], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    unsigned long long t0 = 0, t1 = 0;
    if (threadIdx.x == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int me = lanes_mode ? lane : warp;
    if ((lanes_mode ? warp == 0 : lane == 0) && me < issuers) {
        const uint32_t buf0 = smem_u32(smem) + me * stages * chunk;
        const uint32_t bar0 = smem_u32(&bars[me * MAX_STAGES]);
        const uint8_t* src0 = base + static_cast<size_t>(me) * (region / issuers);
        const uint8_t* src_end = src0 + region / issuers;
        const uint8_t* src = src0;
        // prologue: fill the ring
        for (int s = 0; s < stages; ++s) {
            mbar_expect(bar0 + s * 8, chunk);
            bulk_load(buf0 + s * chunk, src, chunk, bar0 + s * 8);
            src += chunk; if (src + chunk > src_end) src = src0;
        }
        int s = 0; uint32_t ph = 0;
        for (int i = 0; i < iters; ++i) {
            if (!mbar_wait(bar0 + s * 8, ph)) { *err = 1; break; }
            if (i + stages < iters + stages) {   // always refill (the tail is waited for below)
                mbar_expect(bar0 + s * 8, chunk);
                bulk_load(buf0 + s * chunk, src, chunk, bar0 + s * 8);
                src += chunk; if (src + chunk > src_end) src = src0;
            }
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
        // drain the ring
        for (int k = 0; k < stages; ++k) {
            if (!mbar_wait(bar0 + s * 8, ph)) { *err = 1; break; }
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        out_ns[blockIdx.x] = t1 - t0;
    }
}

int main() {
    const size_t region = 192 * 1024;
    int sms = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
    uint8_t* data; unsigned long long* ns; int* err;
    cudaMalloc(&data, region * sms);
    cudaMemset(data, 1, region * sms);
    cudaMalloc(&ns, sizeof(unsigned long long) * sms);
    cudaMalloc(&err, sizeof(int));
    cudaMemset(err, 0, sizeof(int));
    const int smem_bytes = 200 * 1024;
    cudaFuncSetAttribute(tma_rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    unsigned long long* h = (unsigned long long*)malloc(sizeof(unsigned long long) * sms);
    const int chunks[] = {4096, 8192, 16384};
    const int cfgs[][2] = {{1, 6}, {2, 6}, {3, 4}, {4, 3}};   // issuers, stages
    for (int lanes_mode = 0; lanes_mode < 2; ++lanes_mode)
    for (int grid : {148}) {
        for (auto& cfg : cfgs) {
            for (int chunk : chunks) {
                const int issuers = cfg[0], stages = cfg[1];
                if (issuers * stages * chunk > 192 * 1024) continue;
                if (region / issuers < (size_t)chunk) continue;
                const int iters = 32 * 1024 * 1024 / chunk / issuers;
                for (int rep = 0; rep < 2; ++rep) {
                    tma_rate_kernel<<<grid, 256, smem_bytes>>>(data, region, chunk, stages, issuers, iters, ns, err, lanes_mode);
                    cudaError_t e = cudaDeviceSynchronize();
                    if (e != cudaSuccess) { printf("cuda error %s\n", cudaGetErrorString(e)); return 1; }
                }
                cudaMemcpy(h, ns, sizeof(unsigned long long) * grid, cudaMemcpyDeviceToHost);
                unsigned long long mx = 0;
                for (int i = 0; i < grid; ++i) mx = h[i] > mx ? h[i] : mx;
                const double bytes = static_cast<double>(iters + stages) * chunk * issuers;
                printf("%s grid %3d issuers %d stages %2d chunk %5d: %6.1f GB/s per SM (%.0f ns per copy and issuer)\n", lanes_mode ? "lanes" : "warps", grid, issuers, stages,
                       chunk, bytes / mx, (double)mx / (iters + stages));
            }
        }
    }
    int herr = 0;
    cudaMemcpy(&herr, err, sizeof(int), cudaMemcpyDeviceToHost);
    printf("err %d\n", herr);
    return 0;
}
