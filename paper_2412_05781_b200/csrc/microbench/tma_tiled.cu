// Micro-benchmark: rate of TILED TMA loads (cp.async.bulk.tensor.2d, 128-byte swizzle) L2 -> shared memory per SM
// against the box shape and the number of issuing warps.
#include <cuda.h>
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
__device__ __forceinline__ void tma_2d(uint32_t dst, const CUtensorMap* m, uint32_t bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(x), "r"(y) : "memory");
}

constexpr int MAX_ISSUERS = 8, MAX_STAGES = 16;

// tensor: fp16 [rows_total][cols]; CTA b owns rows [b * rows_per_cta, ...); an issuer walks boxes of box_rows rows
__global__ void __launch_bounds__(256, 1) tiled_kernel(const __grid_constant__ CUtensorMap tm, int rows_per_cta, int cols, int box_cols,
                                                       int box_rows, int stages, int issuers, int iters,
                                                       unsigned long long* out_ns, int* err) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ uint64_t bars[MAX_ISSUERS * MAX_STAGES];
    if (threadIdx.x == 0) {
        for (int i = 0; i < MAX_ISSUERS * MAX_STAGES; ++i) mbar_init(&bars[i], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    unsigned long long t0 = 0, t1 = 0;
    if (threadIdx.x == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int box_bytes = box_cols * box_rows * 2;
    if (lane == 0 && warp < issuers) {
        const uint32_t buf0 = smem_u32(smem) + warp * stages * box_bytes;
        const uint32_t bar0 = smem_u32(&bars[warp * MAX_STAGES]);
        const int row_begin = blockIdx.x * rows_per_cta + warp * (rows_per_cta / issuers);
        const int row_end = row_begin + rows_per_cta / issuers;
        int x = 0, y = row_begin;
        auto next = [&]() { x += box_cols; if (x >= cols) { x = 0; y += box_rows; if (y + box_rows > row_end) y = row_begin; } };
        for (int s = 0; s < stages; ++s) {
            mbar_expect(bar0 + s * 8, box_bytes);
            tma_2d(buf0 + s * box_bytes, &tm, bar0 + s * 8, x, y);
            next();
        }
        int s = 0; uint32_t ph = 0;
        for (int i = 0; i < iters; ++i) {
            if (!mbar_wait(bar0 + s * 8, ph)) { *err = 1; break; }
            mbar_expect(bar0 + s * 8, box_bytes);
            tma_2d(buf0 + s * box_bytes, &tm, bar0 + s * 8, x, y);
            next();
            if (++s == stages) { s = 0; ph ^= 1u; }
        }
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

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int main() {
    int sms = 0;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
    void* fnp = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fnp, cudaEnableDefault, &q) != cudaSuccess || !fnp) { printf("no encode fn\n"); return 1; }
    EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(fnp);
    const int cols = 512;                 // fp16 elements per row: 1 KB rows
    const int rows_per_cta = 192;         // 192 KB per CTA, 28 MB in all: L2 resident
    const size_t rows_total = static_cast<size_t>(rows_per_cta) * sms;
    uint8_t* data; unsigned long long* ns; int* err;
    cudaMalloc(&data, rows_total * cols * 2);
    cudaMemset(data, 1, rows_total * cols * 2);
    cudaMalloc(&ns, sizeof(unsigned long long) * sms);
    cudaMalloc(&err, sizeof(int));
    cudaMemset(err, 0, sizeof(int));
    const int smem_bytes = 200 * 1024;
    cudaFuncSetAttribute(tiled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
    unsigned long long* h = (unsigned long long*)malloc(sizeof(unsigned long long) * sms);
    struct Cfg { int box_cols, box_rows, swz; };
    const Cfg boxes[] = {{64, 64, 1}, {64, 128, 1}, {64, 256, 1}, {64, 32, 1}, {256, 16, 0}, {256, 32, 0}, {128, 64, 0}};
    const int icfg[][2] = {{1, 6}, {2, 4}, {3, 3}, {4, 3}};
    for (auto& b : boxes) {
        CUtensorMap tm;
        cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows_total)};
        cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
        cuuint32_t box[2] = {static_cast<cuuint32_t>(b.box_cols), static_cast<cuuint32_t>(b.box_rows)};
        cuuint32_t es[2] = {1, 1};
        CUresult r = encode(&tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, data, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            b.swz ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { printf("encode failed %d\n", (int)r); continue; }
        for (auto& ic : icfg) {
            const int issuers = ic[0], stages = ic[1];
            const int box_bytes = b.box_cols * b.box_rows * 2;
            if (issuers * stages * box_bytes > 190 * 1024) continue;
            if (rows_per_cta / issuers < b.box_rows) continue;
            const int iters = 32 * 1024 * 1024 / box_bytes / issuers;
            for (int rep = 0; rep < 2; ++rep) {
                tiled_kernel<<<sms, 256, smem_bytes>>>(tm, rows_per_cta, cols, b.box_cols, b.box_rows, stages, issuers, iters, ns, err);
                cudaError_t e = cudaDeviceSynchronize();
                if (e != cudaSuccess) { printf("cuda error %s\n", cudaGetErrorString(e)); return 1; }
            }
            cudaMemcpy(h, ns, sizeof(unsigned long long) * sms, cudaMemcpyDeviceToHost);
            unsigned long long mx = 0;
            for (int i = 0; i < sms; ++i) mx = h[i] > mx ? h[i] : mx;
            const double bytes = static_cast<double>(iters + stages) * box_bytes * issuers;
            printf("box %3d x %3d (%5d B, %s) issuers %d stages %d: %6.1f GB/s per SM (%.0f ns per box and issuer)\n", b.box_cols,
                   b.box_rows, box_bytes, b.swz ? "sw128" : "plain", issuers, stages, bytes / mx, (double)mx / (iters + stages));
        }
    }
    int herr = 0;
    cudaMemcpy(&herr, err, sizeof(int), cudaMemcpyDeviceToHost);
    printf("err %d\n", herr);
    return 0;
}
