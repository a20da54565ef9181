// Postprocess Y = A^T M A of F(4x4,3x3) (step (iii) of Section "Techniques") + bias (+ residual, activation) with the
// 36 transform positions of a block of tiles staged in shared memory by TMA.
//
// A CTA owns 256 consecutive tiles (two per thread) and walks `steps` consecutive output channels.  Per channel
// one thread issues one 3-D TMA load {256 tiles, 1 channel, 36 positions} of M (18 KB), up to OUT_TMA_STAGES
// channels ahead of the arithmetic; a thread reads its 36 packed pairs from shared memory, releases the stage after
// the first half of the transform and stores four rows of eight pixels.  The tile decode (image, tile row, tile
// column) is done once per thread instead of once per channel.  Same arithmetic and bits as
// output_transform_vec_kernel<4, 2>, which loads the 36 values of a thread straight from global memory and whose
// warps wait on those loads (long scoreboard 7.9 per issued instruction on a 151 MB layer).
#pragma once
#include <cuda_fp16.h>

#include "ptx.cuh"
#include "transforms.cuh"

namespace sdw {

constexpr int OUT_TMA_STAGES = 4;
constexpr int OUT_TMA_THREADS = 128;
constexpr int OUT_TMA_TILES = 256;                                // tiles per CTA
constexpr int OUT_TMA_STAGE_BYTES = 36 * OUT_TMA_TILES * 2;       // 18432
constexpr uint64_t OUT_TMA_WAIT_LIMIT_NS = 2000000000ull;

// tmM: fp16 [36][K][Pstride], box {256 tiles, 1 channel, 36 positions}, no swizzle (tiles and channels outside the
// tensor read as zeros)
template <bool EP, typename YT = __half>
__global__ void __launch_bounds__(OUT_TMA_THREADS, 3)
output_transform_f4_tma_kernel(const __grid_constant__ CUtensorMap tmM, const YT* __restrict__ bias,
                               YT* __restrict__ y, TileGeom geo, int K, long long p_begin, int steps_per_cta,
                               WtCheck chk, Epilogue ep, int* __restrict__ status_word) {
    constexpr int A = 6, M = 4;
    extern __shared__ uint8_t out_tma_smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(out_tma_smem_raw) + 127) & ~uintptr_t(127));
    __shared__ uint64_t full_bar[OUT_TMA_STAGES];
    __shared__ int abort_flag;
    const int tid = threadIdx.x;
    pdl_launch_dependents();
    const bool wt_ok = wt_check(chk);   // before the wait: see output_transform_kernel
    if (tid == 0) {
        for (int s = 0; s < OUT_TMA_STAGES; ++s) mbar_init(&full_bar[s], 1);
        abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmM);
    }
    __syncthreads();
    pdl_wait();
    if (!wt_ok) return;

    const int pl0 = blockIdx.x * OUT_TMA_TILES;            // first tile of the block inside the pass
    const int k_first = blockIdx.y * steps_per_cta;
    int steps = K - k_first;
    steps = steps < steps_per_cta ? steps : steps_per_cta;
    if (tid == 0) {
        const int pre = steps < OUT_TMA_STAGES ? steps : OUT_TMA_STAGES;
        for (int s = 0; s < pre; ++s) {
            mbar_arrive_expect_tx(&full_bar[s], OUT_TMA_STAGE_BYTES);
            tma_load_3d(smem + s * OUT_TMA_STAGE_BYTES, &tmM, &full_bar[s], pl0, k_first + s, 0);
        }
    }
    // this thread's two tiles: the same for every channel
    const long long p = p_begin + pl0 + 2 * tid;
    const bool tile_ok = p < geo.P;          // P is even (W % 8 == 0): tile p + 1 exists with tile p
    int tw = 0, th = 0;
    long long n = 0;
    if (tile_ok) decode_tile(geo, p, n, th, tw);
    const long long hw = static_cast<long long>(geo.H) * geo.W;
    [[maybe_unused]] float ys = 1.f;
    if constexpr (sizeof(YT) == 4) ys = scalbnf(1.f, range_exponent(ep.amax));   // after the wait above: the word is final
    const int i0 = M * th, j0 = M * tw;
    const long long pix = static_cast<long long>(i0) * geo.W + j0;    // first output pixel inside a channel image

    for (int it = 0; it < steps; ++it) {
        const int s = it % OUT_TMA_STAGES;
        const uint32_t parity = static_cast<uint32_t>(it / OUT_TMA_STAGES) & 1u;
        const bool ok = mbar_wait_bounded(&full_bar[s], parity, &abort_flag, OUT_TMA_WAIT_LIMIT_NS);
        float2 tt[M][A];   // A^T m, one column nu at a time; every float2 holds (tile 0, tile 1)
        if (ok) {
            const uint32_t* src = reinterpret_cast<const uint32_t*>(smem + s * OUT_TMA_STAGE_BYTES) + tid;
#pragma unroll
            for (int c = 0; c < A; ++c) {
                float2 col[A], o[M];
#pragma unroll
                for (int r = 0; r < A; ++r) {
                    const uint32_t w = src[(r * A + c) * (OUT_TMA_TILES / 2)];
                    col[r] = __half22float2(*reinterpret_cast<const __half2*>(&w));
                }
                at4_packed(col, o);
#pragma unroll
                for (int i = 0; i < M; ++i) tt[i][c] = o[i];
            }
        }
        if (!__syncthreads_and(ok)) {
            if (tid == 0 && abort_flag == 0) {
                atomicCAS(status_word, 0, 6 | (11 << 8));   // 6 = timeout, where = 11: the staging of M
                abort_flag = 1;
            }
            break;
        }
        if (tid == 0 && it + OUT_TMA_STAGES < steps) {
            mbar_arrive_expect_tx(&full_bar[s], OUT_TMA_STAGE_BYTES);
            tma_load_3d(smem + s * OUT_TMA_STAGE_BYTES, &tmM, &full_bar[s], pl0, k_first + it + OUT_TMA_STAGES, 0);
        }
        if (!tile_ok) continue;
        const int k = k_first + it;
        const float b = load_bias(bias, k);
        YT* img = y + (n * K + k) * hw + pix;
        uint4 res[M];
        if constexpr (EP && sizeof(YT) == 2) {
#pragma unroll
            for (int i = 0; i < M; ++i) {
                res[i] = make_uint4(0u, 0u, 0u, 0u);
                if (ep.residual && i0 + i < geo.H)
                    res[i] = __ldg(reinterpret_cast<const uint4*>(static_cast<const __half*>(ep.residual) + (img - y) +
                                                                   static_cast<long long>(i) * geo.W));
            }
        }
        [[maybe_unused]] float4 resf[M][2];   // fp32 residual rows, loaded ahead of the second half of the transform
        if constexpr (EP && sizeof(YT) == 4) {
#pragma unroll
            for (int i = 0; i < M; ++i) {
                resf[i][0] = resf[i][1] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (ep.residual && i0 + i < geo.H) {
                    const float4* rp = reinterpret_cast<const float4*>(static_cast<const float*>(ep.residual) + (img - y) +
                                                                       static_cast<long long>(i) * geo.W);
                    resf[i][0] = __ldg(rp);
                    resf[i][1] = __ldg(rp + 1);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < M; ++i) {
            float2 o[M];
            at4_packed(tt[i], o);
            if (i0 + i >= geo.H) continue;
            if constexpr (sizeof(YT) == 4) {
#pragma unroll
                for (int j = 0; j < M; ++j) { o[j].x *= ys; o[j].y *= ys; }
            }
            float v[8] = {o[0].x + b, o[1].x + b, o[2].x + b, o[3].x + b, o[0].y + b, o[1].y + b, o[2].y + b, o[3].y + b};
            if constexpr (EP && sizeof(YT) == 4)
                store_row8_f32_res(reinterpret_cast<float*>(img) + static_cast<long long>(i) * geo.W, v, resf[i], ep);
            else
                store_row8<EP>(img + static_cast<long long>(i) * geo.W, v, res[i], ep, y);
        }
    }
    if (abort_flag != 0) {
        // loads that may still be in flight get a bounded time to land before the shared memory is released
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
}

}  // namespace sdw
