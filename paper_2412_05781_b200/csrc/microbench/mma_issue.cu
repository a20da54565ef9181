// Micro-benchmark: what one thread pays per tcgen05.mma (kind::f16, M = 128, K = 16) against N, with the operands
// resident in shared memory (no loads): issue loop time and time to completion.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include "../ptx.cuh"
using namespace sdw;

__global__ void __launch_bounds__(128, 1) mma_issue_kernel(int n_tile, int ksteps, int mode, long long* out) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t bars[8];
    __shared__ uint32_t tmem_slot;
    for (int i = threadIdx.x; i < 4 * 49152 / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem)[i] = 0;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 8; ++i) mbar_init(&bars[i], 1);
        fence_barrier_init();
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 1) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_slot;
    if (warp == 1 && lane == 0) {
        const uint32_t idesc = make_idesc_f16_f32(128, n_tile, true, false);
        const uint32_t smem_base = smem_u32(smem);
        const uint64_t adesc0 = make_smem_desc_sw128(smem_base, 8192, 1024);
        const uint64_t bdesc0 = make_smem_desc_sw128(smem_base + 16384, 16, 1024);
        const uint64_t stage_step = 49152 >> 4;
        uint64_t adesc = adesc0, bdesc = bdesc0;
        int stage = 0;
        const uint32_t bar0 = smem_u32(&bars[0]);
        uint32_t bar = bar0;
        const long long t0 = clock64();
        for (int k = 0; k < ksteps; ++k) {
            if (mode & 1) tc_fence_after_sync();
            umma_f16(tmem_base, adesc, bdesc, idesc, static_cast<uint32_t>(k));
            umma_f16_acc(tmem_base, adesc + 128, bdesc + 2, idesc);
            umma_f16_acc(tmem_base, adesc + 256, bdesc + 4, idesc);
            umma_f16_acc(tmem_base, adesc + 384, bdesc + 6, idesc);
            if (mode & 2) umma_commit_a32(bar);
            adesc += stage_step; bdesc += stage_step; bar += 8;
            if (++stage == 4) { stage = 0; adesc = adesc0; bdesc = bdesc0; bar = bar0; }
        }
        const long long t1 = clock64();
        umma_commit(&bars[7]);
        uint32_t ok = 0;
        for (int i = 0; i < 100000000 && !ok; ++i) ok = mbar_try_wait(&bars[7], 0u);
        const long long t2 = clock64();
        if (blockIdx.x == 0) { out[0] = t1 - t0; out[1] = t2 - t0; out[2] = ok; }
    }
    __syncthreads();
    if (warp == 1) { tc_fence_after_sync(); tmem_dealloc(tmem_base, 512); }
}

int main() {
    long long* out;
    cudaMalloc(&out, 64);
    const int smem_bytes = 4 * 49152 + 2048;
    cudaFuncSetAttribute(mma_issue_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    const int ksteps = 2000;
    for (int grid : {148})
        for (int mode : {0, 3})
            for (int n : {16, 64, 128, 144, 192, 256}) {
                long long h[3];
                for (int rep = 0; rep < 2; ++rep) {
                    mma_issue_kernel<<<grid, 128, smem_bytes>>>(n, ksteps, mode, out);
                    cudaError_t e = cudaDeviceSynchronize();
                    if (e != cudaSuccess) { printf("cuda error %s\n", cudaGetErrorString(e)); return 1; }
                }
                cudaMemcpy(h, out, 24, cudaMemcpyDeviceToHost);
                printf("grid %3d mode %d (fence %d, commit per k-step %d) N %3d: issue %.0f cycles per k-step (4 MMAs), to completion %.0f (tensor time %d) ok %lld\n",
                       grid, mode, mode & 1, (mode >> 1) & 1, n, (double)h[0] / ksteps, (double)h[1] / ksteps, 2 * n, h[2]);
            }
    return 0;
}
