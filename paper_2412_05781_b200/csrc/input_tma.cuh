// Activation transform V = B^T d B of F(4x4,3x3) (step (i) of Section "Techniques") with the overlapping input
// tiles staged in shared memory by TMA.
//
// A CTA owns a block of TRb x TCb tiles of CPB channel images (TRb * TCb * CPB <= 256 tiles, two per thread) and
// walks `steps` consecutive groups of CPB channels.  Per step one thread issues one 3-D TMA load (two, side by
// side, where the image is wide enough for block rows of 64 tiles) of the pixel window of the block, rows 4 th0 - 1 .. 4 (th0 + TRb) and columns 4 tw0 - 8 .. 4 (tw0 + TCb) + 7 (the column
// origin is rounded down to a 16-byte boundary, as TMA requires; the rows and columns outside the image are the
// zero padding of the convolution and come back as zeros from the TMA unit, so the kernel has no border code at
// all).  Loads run up to IN_TMA_STAGES steps ahead of the arithmetic, which is what the register-only kernel
// (input_transform_f4_kernel: load, wait, compute, store per thread) lacks: on large layers it sat at 42 % of
// the DRAM bandwidth with its warps waiting on their loads.  A thread reads the six rows of its two tiles from
// shared memory (one 16-byte and two 4-byte reads per row), releases the stage and applies B^T . B in packed
// two-wide fp32 exactly like the register-only kernel, so both produce the same bits.
//
// A launch covers a pass of whole tile rows (the passes of a large layer are cut at multiples of the tiles per
// row).  Needs W % 8 == 0 and a 16-byte aligned x; other cases keep the register-only kernels.
#pragma once
#include <cuda_fp16.h>

#include "ptx.cuh"
#include "transforms.cuh"

namespace sdw {

constexpr int IN_TMA_STAGES = 4;
constexpr int IN_TMA_THREADS = 128;
constexpr uint64_t IN_TMA_WAIT_LIMIT_NS = 2000000000ull;

struct InTmaParams {
    int C, TH, TW;
    int tcb_half;        // threads per tile row of a box = TCb / 2
    int nb;              // boxes side by side per block (1 or 2): a block row is nb * TCb tiles
    int box_bytes;       // bw * bh * cpb * 2, rounded up to 128
    int trb;             // tile rows per block
    int cpb;             // channel images per step
    int bw, bh;          // box of the TMA load in pixels: 4 TCb + 16 columns, 4 TRb + 2 rows
    int sb_c, sb_r;      // blocks per image along the columns / rows
    int steps;           // steps (groups of cpb channels) per CTA
    int stage_bytes;     // nb * box_bytes
    long long Pstride;   // tiles per row of V (a multiple of 128)
    long long p_begin;   // first tile of this pass (a multiple of TW)
    long long g_begin, g_end;   // this pass covers the tile rows g = n * TH + th in [g_begin, g_end)
    long long tail_begin, tail_end;   // tiles (relative to p_begin) past the last one of the pass: stored as zeros
    int tail_block;      // the block (blockIdx.x) that stores them
};

// tmX: fp16 [N * C][H][W], box {bw, bh, cpb}, no swizzle, zero fill outside
__global__ void __launch_bounds__(IN_TMA_THREADS, 5)
input_transform_f4_tma_kernel(const __grid_constant__ CUtensorMap tmX, __half* __restrict__ V, const InTmaParams prm,
                              int* __restrict__ status_word) {
    constexpr int A = 6;
    extern __shared__ uint8_t in_tma_smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(in_tma_smem_raw) + 127) & ~uintptr_t(127));
    __shared__ uint64_t full_bar[IN_TMA_STAGES];
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    // block -> (image n, block row, block column); blockIdx.y -> first channel
    const int sb = prm.sb_c * prm.sb_r;
    const int n = blockIdx.x / sb;
    const int br = (blockIdx.x - n * sb) / prm.sb_c;
    const int bc = blockIdx.x - n * sb - br * prm.sb_c;
    const int tcb = prm.tcb_half * 2;
    const int th0 = br * prm.trb, tw0 = bc * tcb * prm.nb;
    // a block none of whose tile rows belong to this pass has nothing to do (a layer done in several passes)
    {
        const long long g_lo = static_cast<long long>(n) * prm.TH + th0;
        const long long g_hi = static_cast<long long>(n) * prm.TH + (th0 + prm.trb < prm.TH ? th0 + prm.trb : prm.TH);
        if (g_hi <= prm.g_begin || g_lo >= prm.g_end) return;
    }
    const int c_first = blockIdx.y * prm.steps * prm.cpb;
    int steps = (prm.C - c_first + prm.cpb - 1) / prm.cpb;
    steps = steps < prm.steps ? steps : prm.steps;

    if (tid == 0) {
        for (int s = 0; s < IN_TMA_STAGES; ++s) mbar_init(&full_bar[s], 1);
        abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmX);
    }
    __syncthreads();
    // thread -> (channel within the step, tile row within the block, pair of tiles within the row)
    const int row_threads = prm.tcb_half * prm.nb;
    const int rest = tid / row_threads;
    const int jf = tid - rest * row_threads;          // pair of tiles within the block row
    const int sub = jf >= prm.tcb_half ? 1 : 0;       // which box
    const int j = jf - sub * prm.tcb_half;
    const int r = rest % prm.trb;
    const int cl = rest / prm.trb;
    const int th = th0 + r, tw = tw0 + 2 * jf;
    const long long g = static_cast<long long>(n) * prm.TH + th;   // tile row over all images
    // W % 8 == 0: TW is even, so tile tw + 1 exists whenever tile tw does
    const bool tile_ok = cl < prm.cpb && th < prm.TH && tw < prm.TW && g >= prm.g_begin && g < prm.g_end;
    const long long plane = static_cast<long long>(prm.C) * prm.Pstride;
    const long long p = g * prm.TW + tw - prm.p_begin;   // tile index inside the pass
    // first of the six window rows of this thread inside a stage; the 16-byte segment starts at column 8 j + 8
    const uint32_t win = sub * prm.box_bytes + (static_cast<uint32_t>(cl * prm.bh + 4 * r) * prm.bw + 8 * j + 8) * 2u;
    const uint32_t row_pitch = static_cast<uint32_t>(prm.bw) * 2u;

    // the index arithmetic above runs while the preceding kernel drains
    pdl_wait();                 // x may be the output of the preceding kernel: wait first, release the GEMM second
    pdl_launch_dependents();

    const int x0 = 4 * tw0 - 8, y0 = 4 * th0 - 1;
    const uint32_t tx_bytes = static_cast<uint32_t>(prm.bw) * prm.bh * prm.cpb * 2u * prm.nb;
    if (tid == 0) {
        const int pre = steps < IN_TMA_STAGES ? steps : IN_TMA_STAGES;
        for (int s = 0; s < pre; ++s) {
            mbar_arrive_expect_tx(&full_bar[s], tx_bytes);
            for (int bx = 0; bx < prm.nb; ++bx)
                tma_load_3d(smem + s * prm.stage_bytes + bx * prm.box_bytes, &tmX, &full_bar[s], x0 + bx * 4 * tcb, y0,
                            n * prm.C + c_first + s * prm.cpb);
        }
    }

    for (int it = 0; it < steps; ++it) {
        const int s = it % IN_TMA_STAGES;
        const uint32_t parity = static_cast<uint32_t>(it / IN_TMA_STAGES) & 1u;
        bool ok = mbar_wait_bounded(&full_bar[s], parity, &abort_flag, IN_TMA_WAIT_LIMIT_NS);
        // first half of the transform (along the columns of every window row) straight from shared memory, so
        // that the stage can be released before the second half and the stores
        float2 e2[A][A];   // e2[r][nu]: rows transformed along the columns, (tile 0, tile 1)
        if (ok && cl < prm.cpb) {   // threads past the last channel image of a step have no window in the stage
            const uint8_t* src = smem + s * prm.stage_bytes + win;
#pragma unroll
            for (int rr = 0; rr < A; ++rr) {
                const uint8_t* q = src + rr * row_pitch;
                const uint4 v = *reinterpret_cast<const uint4*>(q);
                const uint32_t lw = *reinterpret_cast<const uint32_t*>(q - 4);    // columns 8 j + 6, 8 j + 7
                const uint32_t rw = *reinterpret_cast<const uint32_t*>(q + 16);   // columns 8 j + 16, 8 j + 17
                // pixels: L = lw.hi, px0..px7 = v.x.lo .. v.w.hi, R = rw.lo; tile 0 uses L..px4, tile 1 px3..R
                uint32_t h[A];
                h[0] = __byte_perm(lw, v.y, 0x7632);    // (L,   px3)
                h[1] = __byte_perm(v.x, v.z, 0x5410);   // (px0, px4)
                h[2] = __byte_perm(v.x, v.z, 0x7632);   // (px1, px5)
                h[3] = __byte_perm(v.y, v.w, 0x5410);   // (px2, px6)
                h[4] = __byte_perm(v.y, v.w, 0x7632);   // (px3, px7)
                h[5] = __byte_perm(v.z, rw, 0x5410);    // (px4, R)
                float2 d[A];
#pragma unroll
                for (int s2 = 0; s2 < A; ++s2) d[s2] = __half22float2(*reinterpret_cast<const __half2*>(&h[s2]));
                bt4_packed(d, e2[rr]);
            }
        }
        // every thread has read the stage (or nobody uses it): it can be refilled
        if (!__syncthreads_and(ok)) {
            if (tid == 0 && abort_flag == 0) {
                atomicCAS(status_word, 0, 6 | (10 << 8));   // 6 = timeout, where = 10: the input staging
                abort_flag = 1;
            }
            break;
        }
        if (tid == 0 && it + IN_TMA_STAGES < steps) {
            mbar_arrive_expect_tx(&full_bar[s], tx_bytes);
            for (int bx = 0; bx < prm.nb; ++bx)
                tma_load_3d(smem + s * prm.stage_bytes + bx * prm.box_bytes, &tmX, &full_bar[s], x0 + bx * 4 * tcb, y0,
                            n * prm.C + c_first + (it + IN_TMA_STAGES) * prm.cpb);
        }
        const int c = c_first + it * prm.cpb + cl;
        if (!tile_ok || c >= prm.C) continue;
        __half* vp = V + static_cast<long long>(c) * prm.Pstride + p;
#pragma unroll
        for (int nu = 0; nu < A; ++nu) {
            float2 col[A], o[A];
#pragma unroll
            for (int rr = 0; rr < A; ++rr) col[rr] = e2[rr][nu];
            bt4_packed(col, o);
#pragma unroll
            for (int xi = 0; xi < A; ++xi)
                *reinterpret_cast<uint32_t*>(vp + (xi * A + nu) * plane) = pack2(o[xi].x, o[xi].y);
        }
    }

    // the tiles between the last one of the pass and the end of its last block of 128 are zero, as the
    // register-only kernels leave them
    if (static_cast<int>(blockIdx.x) == prm.tail_block) {
        const int tail2 = static_cast<int>((prm.tail_end - prm.tail_begin) / 2);   // both are even
        const int chans = steps * prm.cpb < prm.C - c_first ? steps * prm.cpb : prm.C - c_first;
        for (int i = tid; i < chans * tail2 * A * A; i += IN_TMA_THREADS) {
            const int t2 = i % tail2;
            const int rest2 = i / tail2;
            const int pos = rest2 % (A * A), c = c_first + rest2 / (A * A);
            *reinterpret_cast<uint32_t*>(V + pos * plane + static_cast<long long>(c) * prm.Pstride + prm.tail_begin +
                                         2 * t2) = 0u;
        }
    }
    if (abort_flag != 0) {
        // loads that may still be in flight get a bounded time to land before the shared memory is released
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
    }
}

}  // namespace sdw
