// Step (ii) of Section "Techniques": the "element-wise multiplication" of the transformed
// filter and activation.  With C input channels it is, for each of the a*a transform
// positions, the dense contraction  M[pos][k][p] = sum_c U[pos][k][c] * V[pos][c][p],
// i.e. a batched GEMM.  It runs on the tcgen05 tensor cores: operands are brought into
// shared memory by TMA (128-byte swizzle), accumulated in fp32 in tensor memory, and the
// result is rounded once to fp16 and written back by a TMA store.
//
// One persistent CTA per SM walks the list of (pos, k-tile, p-tile) output tiles.
//   warp 0   : TMA producer        (one lane)
//   warp 1   : TMEM owner + MMA issuer (one lane)
//   warps 2-5: epilogue, one TMEM lane quarter each; TMEM accumulators are double-buffered so
//              the epilogue of tile i overlaps the MMAs of tile i+1.
#pragma once
#include <cuda_fp16.h>

#include "ptx.cuh"

namespace sdw {

constexpr int GEMM_BLOCK_M = 128;  // output channels per tile (TMEM lanes)
constexpr int GEMM_BLOCK_K = 64;   // input channels per pipeline stage (one 128-byte swizzle row of U)
constexpr int GEMM_THREADS = 192;
constexpr uint64_t GEMM_WAIT_LIMIT_NS = 2000000000ull;  // a wait longer than 2 s is reported, not spun on

template <int BLOCK_N, int STAGES>
struct GemmSmem {
    static constexpr int A_BYTES = GEMM_BLOCK_M * GEMM_BLOCK_K * 2;
    static constexpr int B_BOX_BYTES = 64 * GEMM_BLOCK_K * 2;  // one [64 p] x [64 c] box
    static constexpr int B_BYTES = (BLOCK_N / 64) * B_BOX_BYTES;
    static constexpr int C_BOX_BYTES = GEMM_BLOCK_M * 64 * 2;  // one [64 p] x [128 k] box
    static constexpr int C_BYTES = (BLOCK_N / 64) * C_BOX_BYTES;
    static constexpr int OFF_A = 0;
    static constexpr int OFF_B = OFF_A + STAGES * A_BYTES;
    static constexpr int OFF_C = OFF_B + STAGES * B_BYTES;
    static constexpr int OFF_BAR = OFF_C + C_BYTES;
    static constexpr int NUM_BARS = 2 * STAGES + 4;
    static constexpr int OFF_MISC = OFF_BAR + NUM_BARS * 8;
    static constexpr int TOTAL = OFF_MISC + 16;
    static constexpr int DYN_BYTES = TOTAL + 1024;  // slack to align the base to 1024 bytes
};

// tmU: fp16 [pos][Kp][Cp]      box {64 c, 128 k, 1}, 128B swizzle  (A operand, K-major)
// tmV: fp16 [pos][C][Pstride]  box {64 p,  64 c, 1}, 128B swizzle  (B operand, MN-major; rows c >= C read as 0)
// tmM: fp16 [pos][Kp][Pstride] box {64 p, 128 k, 1}, 128B swizzle  (result)
template <int BLOCK_N, int STAGES>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
wino_gemm_kernel(const __grid_constant__ CUtensorMap tmU, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmM, int num_k_tiles, int num_p_tiles, int num_pos,
                 int num_c_blocks, int* __restrict__ status_word) {
    using L = GemmSmem<BLOCK_N, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + L::OFF_BAR);
    uint64_t* empty_bar = full_bar + STAGES;
    uint64_t* acc_full_bar = empty_bar + STAGES;
    uint64_t* acc_empty_bar = acc_full_bar + 2;
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(smem + L::OFF_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::OFF_MISC + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int num_tiles = num_k_tiles * num_p_tiles * num_pos;
    constexpr uint32_t TMEM_COLS = 2 * BLOCK_N;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full_bar[b], 1);
            mbar_init(&acc_empty_bar[b], 4);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmU);
        prefetch_tmap(&tmV);
        prefetch_tmap(&tmM);
    }
    if (warp == 1) {
        tmem_alloc(tmem_base_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                const int pt = tile % num_p_tiles;
                const int kt = (tile / num_p_tiles) % num_k_tiles;
                const int pos = tile / (num_p_tiles * num_k_tiles);
                for (int cb = 0; cb < num_c_blocks; ++cb) {
                    ok = mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&full_bar[stage], L::A_BYTES + L::B_BYTES);
                    tma_load_3d(smem + L::OFF_A + stage * L::A_BYTES, &tmU, &full_bar[stage], cb * GEMM_BLOCK_K,
                                kt * GEMM_BLOCK_M, pos);
#pragma unroll
                    for (int j = 0; j < BLOCK_N / 64; ++j)
                        tma_load_3d(smem + L::OFF_B + stage * L::B_BYTES + j * L::B_BOX_BYTES, &tmV, &full_bar[stage],
                                    pt * BLOCK_N + j * 64, cb * GEMM_BLOCK_K, pos);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) { *abort_flag = 1; atomicExch(status_word, 6); }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_f16_f32(GEMM_BLOCK_M, BLOCK_N, false, true);
            int stage = 0;
            uint32_t phase = 0;
            int buf = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
                ok = mbar_wait_bounded(&acc_empty_bar[buf], acc_phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * BLOCK_N);
                for (int cb = 0; cb < num_c_blocks; ++cb) {
                    ok = mbar_wait_bounded(&full_bar[stage], phase, abort_flag, GEMM_WAIT_LIMIT_NS);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(smem + L::OFF_A + stage * L::A_BYTES);
                    const uint32_t b_addr = smem_u32(smem + L::OFF_B + stage * L::B_BYTES);
#pragma unroll
                    for (int s = 0; s < GEMM_BLOCK_K / 16; ++s) {
                        // A (K-major): 16 channels = 32 bytes further along the swizzled 128-byte row.
                        // B (MN-major): 16 channels = 16 rows of 128 bytes; 64-wide p blocks are B_BOX_BYTES apart.
                        const uint64_t adesc = make_smem_desc_sw128(a_addr + s * 32, 16, 1024);
                        const uint64_t bdesc = make_smem_desc_sw128(b_addr + s * 2048, L::B_BOX_BYTES, 1024);
                        umma_f16(d_tmem, adesc, bdesc, idesc, (cb > 0 || s > 0) ? 1u : 0u);
                    }
                    umma_commit(&empty_bar[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit(&acc_full_bar[buf]);
                buf ^= 1;
                if (buf == 0) acc_phase ^= 1u;
            }
            if (!ok) { *abort_flag = 1; atomicExch(status_word, 6); }
        }
    } else {
        // ------------------------------ epilogue ------------------------------
        const int quarter = warp & 3;               // TMEM lanes this warp may read: 32*quarter ..
        const int row = quarter * 32 + lane;        // output channel within the tile
        const int epi_tid = threadIdx.x - 64;
        uint8_t* stage_c = smem + L::OFF_C;
        int buf = 0;
        uint32_t acc_phase = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
            const int pt = tile % num_p_tiles;
            const int kt = (tile / num_p_tiles) % num_k_tiles;
            const int pos = tile / (num_p_tiles * num_k_tiles);
            bool ok = mbar_wait_bounded(&acc_full_bar[buf], acc_phase, abort_flag, GEMM_WAIT_LIMIT_NS);
            if (!ok) { *abort_flag = 1; atomicExch(status_word, 6); }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (*abort_flag != 0) break;
            tc_fence_after_sync();
#pragma unroll 1
            for (int chunk = 0; chunk < BLOCK_N / 32; ++chunk) {
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                  static_cast<uint32_t>(buf * BLOCK_N + chunk * 32), r);
                tmem_ld_wait();
                uint8_t* box = stage_c + (chunk >> 1) * L::C_BOX_BYTES + row * 128;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 v;
                    __half2 h;
                    h = __floats2half2_rn(__uint_as_float(r[8 * i + 0]), __uint_as_float(r[8 * i + 1]));
                    v.x = *reinterpret_cast<uint32_t*>(&h);
                    h = __floats2half2_rn(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3]));
                    v.y = *reinterpret_cast<uint32_t*>(&h);
                    h = __floats2half2_rn(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5]));
                    v.z = *reinterpret_cast<uint32_t*>(&h);
                    h = __floats2half2_rn(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7]));
                    v.w = *reinterpret_cast<uint32_t*>(&h);
                    const int c16 = ((chunk & 1) * 4 + i) ^ (row & 7);  // 128-byte swizzle of the 16-byte chunk
                    *reinterpret_cast<uint4*>(box + c16 * 16) = v;
                }
            }
            // accumulator drained: hand the TMEM buffer back to the MMA warp
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty_bar[buf]);
            fence_proxy_async_smem();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (epi_tid == 0) {
#pragma unroll
                for (int j = 0; j < BLOCK_N / 64; ++j)
                    tma_store_3d(&tmM, stage_c + j * L::C_BOX_BYTES, pt * BLOCK_N + j * 64, kt * GEMM_BLOCK_M, pos);
                tma_store_commit();
                tma_store_wait_read();
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            buf ^= 1;
            if (buf == 0) acc_phase ^= 1u;
        }
        if (epi_tid == 0) tma_store_wait_all();
    }

    __syncwarp();
    __syncthreads();
    if (*abort_flag != 0) {
        // give copies and MMAs that may still be in flight a bounded time to land before TMEM and
        // shared memory are released
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace sdw
