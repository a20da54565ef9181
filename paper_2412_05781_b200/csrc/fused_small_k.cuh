// All three steps of F(2x2,3x3) in ONE kernel for layers with at most 8 output channels per
// CTA (the 320 -> 4 and 128 -> 3 output convolutions of the UNet and the VAE decoder).
//
// With so few output channels the unfused path is dominated by writing V (alpha^2 = 16 values per
// tile and input channel) to the workspace and reading it back.  Here a CTA owns 128 tiles:
//   warps 8-23 : input transform.  A warp owns one of the 16 input channels of a stage, a lane owns 4
//                consecutive tiles of a tile row (one aligned 16-byte load per input row plus two halo
//                values); V = B^T d B is rounded to fp16 and written straight into shared memory in the
//                layout the tensor core reads (M-major A operand, 128-byte swizzle) -- V never exists in
//                global memory.  The loads of the next stage are issued before the arithmetic of this one.
//   warps 0-3  : one thread each issues, per stage of 16 channels, the tcgen05.mma of 4 of the 16 transform
//                positions (128 tiles x 16 channels x 16 output channels each) into 16 x 16 TMEM columns;
//                warp 0 also fetches the transformed filters U (blocks of [8 k][64 c], all 16 positions
//                at once, by TMA).
//   warps 4-7  : epilogue.  A thread owns one tile: it reads the 16 position accumulators of 4 output
//                channels at a time from TMEM, applies A^T M A, adds the bias and stores 2x2 pixels.
// All 16 accumulators of a tile live in TMEM (16 x 16 columns, double-buffered), which is what limits this
// design to few output channels per CTA: a layer with more of them would repeat the input transform once
// per chunk (grid.y), and three 64 KB stages of V leave room for the filters of only 8.
#pragma once
#include <cuda_fp16.h>

#include "ptx.cuh"
#include "transforms.cuh"
#include "wino_gemm.cuh"

namespace sdw {

constexpr int FK_N = 16;                       // UMMA N (the smallest for M = 128)
constexpr int FK_KMAX = 8;                     // output channels per CTA: only 8 of the 16 rows of the B operand are
                                               // loaded; accumulator columns 8-15 hold garbage that nobody reads
constexpr int FK_CSTEP = 16;                   // input channels per stage (one UMMA K step)
constexpr int FK_MMA_WARPS = 4;                // warps 0-3: one issuing thread each, 4 transform positions each
constexpr int FK_EPI_WARP0 = 4;                // warps 4-7
constexpr int FK_TR_WARP0 = 8;                 // warps 8-23
constexpr int FK_TR_WARPS = 16;
constexpr int FK_THREADS = (FK_TR_WARP0 + FK_TR_WARPS) * 32;   // 768
constexpr int FK_POS_BYTES = 2 * 16 * 128;     // per position: two boxes of [16 c][64 p] fp16
constexpr int FK_V_STAGE_BYTES = 16 * FK_POS_BYTES;            // 64 KB
constexpr int FK_V_STAGES = 3;
constexpr int FK_U_POS_BYTES = FK_KMAX * 128;  // per position: [8 k][64 c] fp16, one swizzle atom
constexpr int FK_U_BUF_BYTES = 16 * FK_U_POS_BYTES;            // 16 KB per block of 64 input channels
constexpr int FK_U_BUFS = 2;
constexpr int FK_ACC_COLS = 16 * FK_N;         // 256 TMEM columns per accumulator set
constexpr int FK_DYN_SMEM = FK_V_STAGES * FK_V_STAGE_BYTES + FK_U_BUFS * FK_U_BUF_BYTES + 1024 + 256;

struct FusedKParams {
    const uint32_t* wt_header;   // header of the transformed filter (see wt_header_ok)
    TileGeom geo;
    int C, K;
    int num_stages;     // ceil(C / 16)
    int num_cblocks;    // ceil(C / 64)
    int num_p_tiles;    // ceil(P / 128)
};

// raw input of one unit (4 tiles of one channel): four rows of 8 pixels plus the halo pixel on each side
struct FkRaw {
    uint4 row[4];
    uint32_t left[4], right[4];   // the aligned 32-bit words before / after the segment: the pixel left of it is
                                  // the high half of left[], the pixel right of it the low half of right[]
};

// where the 4 tiles of a lane sit in the image (decoded once per 128-tile block)
struct FkUnitGeo {
    long long base;     // element offset of (n, c = 0, row 2*th - 1, column 2*tw)
    int rows_ok;        // bit r set: input row 2*th - 1 + r is inside the image
    bool left_ok, right_ok, valid;
};

__device__ __forceinline__ FkUnitGeo fk_decode(const TileGeom& geo, int C, long long p) {
    FkUnitGeo g;
    g.valid = p < geo.P;
    const long long pp = g.valid ? p : 0;
    int tw, th;
    long long n;
    decode_tile(geo, pp, n, th, tw);
    const int i0 = 2 * th - 1, j0 = 2 * tw;
    g.base = n * C * static_cast<long long>(geo.H) * geo.W + static_cast<long long>(i0) * geo.W + j0;
    g.rows_ok = 0;
#pragma unroll
    for (int r = 0; r < 4; ++r)
        if (i0 + r >= 0 && i0 + r < geo.H) g.rows_ok |= 1 << r;
    g.left_ok = j0 > 0;
    g.right_ok = j0 + 8 < geo.W;
    return g;
}

// fp32 x (the fp32 interface): the pixels are rounded to fp16 as they are loaded, into the same packed words the
// fp16 loads deliver; what follows is the packed fp16 arithmetic of fk_transform either way.
template <typename XT>
__device__ __forceinline__ void fk_load(const XT* __restrict__ x, const TileGeom& geo, const FkUnitGeo& g, int c,
                                        bool c_ok, FkRaw& raw) {
    const long long plane = static_cast<long long>(geo.H) * geo.W;
    const XT* p0 = x + g.base + c * plane;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const bool ok = c_ok && g.valid && ((g.rows_ok >> r) & 1);
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        uint32_t lo = 0u, hi = 0u;
        if (ok) {
            const long long off = static_cast<long long>(r) * geo.W;
            if constexpr (sizeof(XT) == 4) {
                const float4 a = __ldg(reinterpret_cast<const float4*>(p0 + off));
                const float4 b = __ldg(reinterpret_cast<const float4*>(p0 + off) + 1);
                v = make_uint4(pack2(a.x, a.y), pack2(a.z, a.w), pack2(b.x, b.y), pack2(b.z, b.w));
                if (g.left_ok) lo = pack2(0.f, __ldg(p0 + off - 1));     // the pixel left of the segment in the high half
                if (g.right_ok) hi = pack2(__ldg(p0 + off + 8), 0.f);    // the pixel right of it in the low half
            } else {
            v = __ldg(reinterpret_cast<const uint4*>(p0 + off));
            if (g.left_ok) lo = __ldg(reinterpret_cast<const uint32_t*>(p0 + off - 2));
            if (g.right_ok) hi = __ldg(reinterpret_cast<const uint32_t*>(p0 + off + 8));
            }
        }
        raw.row[r] = v;
        raw.left[r] = lo;
        raw.right[r] = hi;
    }
}

// V = B^T d B for the 4 tiles of a unit, written as packed fp16 to the 16 position planes of the stage.
// F(2x2,3x3)'s B^T only adds and subtracts, so the transform runs in packed fp16 arithmetic on tile PAIRS
// (the two halves of a register are tiles 2h and 2h+1, which is also the layout of the operand in
// shared memory): 32 byte-permutes, 64 half2 additions and 16 8-byte stores per unit, against three times
// as many instructions in fp32.  Cost: V carries two fp16 roundings instead of one; the accumulators of
// this kernel are never rounded to fp16 (no M in memory), so the end-to-end error stays at the level of
// the unfused path (parity tests).
__device__ __forceinline__ void fk_transform_store(const FkRaw& raw, uint8_t* stage_base, uint32_t voff) {
    uint32_t v[2][16];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        __half2 e[4][4];   // e[r][nu] for the tile pair: rows transformed along the columns
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const uint32_t p0 = raw.row[r].x, p1 = raw.row[r].y, p2 = raw.row[r].z, p3 = raw.row[r].w;
            uint32_t d0, d1, d2, d3;   // d_s = (pixel 2*t + s of tile t = 2h, of tile t = 2h + 1)
            if (h == 0) {
                d0 = __byte_perm(raw.left[r], p0, 0x7632);                          // (left halo, px 1)
                d1 = __byte_perm(p0, p1, 0x5410);                                   // (px 0, px 2)
                d2 = __byte_perm(p0, p1, 0x7632);                                   // (px 1, px 3)
                d3 = __byte_perm(p1, p2, 0x5410);                                   // (px 2, px 4)
            } else {
                d0 = __byte_perm(p1, p2, 0x7632);                                   // (px 3, px 5)
                d1 = __byte_perm(p2, p3, 0x5410);                                   // (px 4, px 6)
                d2 = __byte_perm(p2, p3, 0x7632);                                   // (px 5, px 7)
                d3 = __byte_perm(p3, raw.right[r], 0x5410);                         // (px 6, right halo)
            }
            const __half2 a0 = *reinterpret_cast<const __half2*>(&d0), a1 = *reinterpret_cast<const __half2*>(&d1),
                          a2 = *reinterpret_cast<const __half2*>(&d2), a3 = *reinterpret_cast<const __half2*>(&d3);
            e[r][0] = __hsub2(a0, a2);
            e[r][1] = __hadd2(a1, a2);
            e[r][2] = __hsub2(a2, a1);
            e[r][3] = __hsub2(a1, a3);
        }
#pragma unroll
        for (int nu = 0; nu < 4; ++nu) {
            const __half2 v0 = __hsub2(e[0][nu], e[2][nu]);
            const __half2 v1 = __hadd2(e[1][nu], e[2][nu]);
            const __half2 v2 = __hsub2(e[2][nu], e[1][nu]);
            const __half2 v3 = __hsub2(e[1][nu], e[3][nu]);
            v[h][0 * 4 + nu] = *reinterpret_cast<const uint32_t*>(&v0);
            v[h][1 * 4 + nu] = *reinterpret_cast<const uint32_t*>(&v1);
            v[h][2 * 4 + nu] = *reinterpret_cast<const uint32_t*>(&v2);
            v[h][3 * 4 + nu] = *reinterpret_cast<const uint32_t*>(&v3);
        }
    }
#pragma unroll
    for (int pos = 0; pos < 16; ++pos)
        *reinterpret_cast<uint2*>(stage_base + pos * FK_POS_BYTES + voff) = make_uint2(v[0][pos], v[1][pos]);
}

// Grid: x = persistent workers over the 128-tile blocks, y = chunks of 16 output channels.
template <typename T = __half>   // element type of x, bias and y
__global__ void __launch_bounds__(FK_THREADS, 1)
fused_small_k_kernel(const __grid_constant__ CUtensorMap tmU, const T* __restrict__ x,
                     const T* __restrict__ bias, T* __restrict__ y, FusedKParams prm, int* status_word) {
    // The header may have been written by the kernel right before this one: wait for it before anything else.
    // (Uniform early return: no barrier or TMEM has been set up yet.)
    pdl_wait();
    if (!wt_header_ok(prm.wt_header, prm.K, prm.C, 2, status_word)) return;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    // The filter buffers come first: the MMA reads 16 rows of B where only 8 are loaded, i.e. up to 1 KB past
    // the last position of a buffer, which must still be shared memory of this CTA (it is the first V stage).
    uint8_t* u_smem = smem;                                             // FK_U_BUFS x 16 KB
    uint8_t* v_smem = smem + FK_U_BUFS * FK_U_BUF_BYTES;                // FK_V_STAGES x 64 KB
    uint64_t* bars = reinterpret_cast<uint64_t*>(v_smem + FK_V_STAGES * FK_V_STAGE_BYTES);
    uint64_t* v_full = bars;                 // [3] 16 arrivals (one per transform warp)
    uint64_t* v_empty = bars + 3;            // [3] tcgen05.commit
    uint64_t* u_full = bars + 6;             // [2] TMA bytes
    uint64_t* u_empty = bars + 8;            // [2] tcgen05.commit
    uint64_t* acc_full = bars + 10;          // [2] tcgen05.commit
    uint64_t* acc_empty = bars + 12;         // [2] 4 arrivals (one per epilogue warp)
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(bars + 14);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 15);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int worker = blockIdx.x, num_workers = gridDim.x;
    const int k0 = blockIdx.y * FK_KMAX;
    const int nstages = prm.num_stages;
    const bool u_resident = prm.num_cblocks <= FK_U_BUFS;   // the whole filter chunk stays in shared memory

    if (threadIdx.x == 0) {
        for (int i = 0; i < FK_V_STAGES; ++i) {
            mbar_init(&v_full[i], FK_TR_WARPS);
            mbar_init(&v_empty[i], FK_MMA_WARPS);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&u_full[i], 1);
            mbar_init(&u_empty[i], FK_MMA_WARPS);
            mbar_init(&acc_full[i], FK_MMA_WARPS);
            mbar_init(&acc_empty[i], 4);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmU);
    }
    if (warp == FK_EPI_WARP0) { tmem_alloc(tmem_base_slot, 2 * FK_ACC_COLS); tmem_relinquish(); }
    pdl_launch_dependents();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;

    if (warp < FK_MMA_WARPS) {
        // ------------------- MMA issue (one thread per warp) and filter loads (warp 0) -------------------
        // A single thread needs about 67 cycles per tcgen05.mma of this size (measured: the time is the same
        // with 4, 8 or 16 of them per stage and adds to everything else), so the 16 positions of a stage are
        // issued by four threads, four positions each; their accumulators are disjoint TMEM columns, so the
        // order between the threads does not matter.  Every barrier they signal counts four arrivals.
        if (lane == 0) {
            pdl_wait();   // U may have been written by the kernel before this one
            const int pos0 = warp * 4;
            const bool loader = warp == 0;
            const uint32_t idesc = make_idesc_f16_f32(128, FK_N, true, false);
            const uint32_t v_base = smem_u32(v_smem) + pos0 * FK_POS_BYTES;
            const uint32_t u_base = smem_u32(u_smem);
            uint32_t u_issued = 0;        // filter blocks requested so far (running count over all tiles; loader only)
            uint32_t u_used = 0;          // filter blocks consumed so far
            uint32_t vs = 0, v_phase = 0;   // V stage to consume next and the parity of its full barrier
            int buf = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            const int my_tiles = worker < prm.num_p_tiles ? (prm.num_p_tiles - worker + num_workers - 1) / num_workers : 0;
            const uint32_t total_blocks = u_resident ? static_cast<uint32_t>(prm.num_cblocks)
                                                     : static_cast<uint32_t>(my_tiles) * prm.num_cblocks;
            // Request the next filter block if a buffer is free.  The buffer was released by the commits of
            // all four issuers a moment ago: unless the block is needed right now (`must`), an unfinished
            // release only postpones the request to the next stage instead of stalling the MMA issue.
            auto request_u = [&](bool must) -> bool {
                if (u_issued >= total_blocks || u_issued - u_used >= FK_U_BUFS) return true;
                const int cb = static_cast<int>(u_issued % prm.num_cblocks);
                const uint32_t ub = u_resident ? static_cast<uint32_t>(cb) : (u_issued & 1u);
                if (!u_resident && u_issued >= FK_U_BUFS) {
                    const uint32_t ph = ((u_issued >> 1) - 1u) & 1u;
                    if (!mbar_try_wait(&u_empty[ub], ph)) {
                        if (!must) return true;
                        if (!mbar_wait_bounded(&u_empty[ub], ph, abort_flag, GEMM_WAIT_LIMIT_NS)) return false;
                    }
                }
                const uint32_t bar = smem_u32(&u_full[ub]);
                mbar_arrive_expect_tx_a32(bar, FK_U_BUF_BYTES);
                tma_load_5d_k_a32(u_base + ub * FK_U_BUF_BYTES, &tmU, bar, (k0 & 8), cb, k0 >> 4, 0);
                ++u_issued;
                return true;
            };
            if (loader) {
                for (int i = 0; i < FK_U_BUFS && ok; ++i) ok = request_u(true);
                if (!ok) report_timeout(status_word, 5, 0);
            }
            for (int tile = worker; tile < prm.num_p_tiles && ok; tile += num_workers) {
                ok = mbar_wait_bounded(&acc_empty[buf], acc_phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 2, 0); break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * FK_ACC_COLS + pos0 * FK_N);
                for (int s = 0; s < nstages; ++s) {
                    const int cb = s >> 2, ks = s & 3;
                    if (loader) {
                        ok = request_u(ks == 0 && u_issued == u_used);
                        if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 5, 0); break; }
                    }
                    uint32_t ub;
                    if (u_resident) {
                        ub = static_cast<uint32_t>(cb);
                        if (ks == 0 && tile == worker) {
                            ok = mbar_wait_bounded(&u_full[ub], 0u, abort_flag, GEMM_WAIT_LIMIT_NS);
                            if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 6, 0); break; }
                        }
                    } else {
                        ub = u_used & 1u;
                        if (ks == 0) {
                            ok = mbar_wait_bounded(&u_full[ub], (u_used >> 1) & 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                            if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 6, 0); break; }
                        }
                    }
                    ok = mbar_wait_bounded(&v_full[vs], v_phase, abort_flag, GEMM_WAIT_LIMIT_NS);
                    if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 3, 0); break; }
                    tc_fence_after_sync();
                    uint64_t adesc = make_smem_desc_sw128(v_base + vs * FK_V_STAGE_BYTES, 2048, 1024);
                    // only rows 0-7 of B are loaded: rows 8-15 are read from the next position's block
                    uint64_t bdesc = make_smem_desc_sw128(u_base + ub * FK_U_BUF_BYTES + pos0 * FK_U_POS_BYTES + ks * 32,
                                                          16, 1024);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        umma_f16(d_tmem + j * FK_N, adesc, bdesc, idesc, s > 0 ? 1u : 0u);
                        adesc += FK_POS_BYTES >> 4;
                        bdesc += FK_U_POS_BYTES >> 4;
                    }
                    umma_commit(&v_empty[vs]);
                    if (++vs == FK_V_STAGES) { vs = 0; v_phase ^= 1u; }
                    if (!u_resident && (ks == 3 || s == nstages - 1)) {
                        umma_commit(&u_empty[ub]);
                        ++u_used;
                    }
                }
                if (!ok) break;
                umma_commit(&acc_full[buf]);
                buf ^= 1;
                if (buf == 0) acc_phase ^= 1u;
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp < FK_TR_WARP0) {
        // ------------------------------ epilogue (warps 4-7) ------------------------------
        using Wm = Wino<2>;
        const int quarter = warp & 3;          // TMEM lanes this warp may read: 32*quarter .. +31
        pdl_wait();
        int buf = 0;
        uint32_t acc_phase = 0;
        const int kcount = (prm.K - k0) < FK_KMAX ? (prm.K - k0) : FK_KMAX;
        for (int tile = worker; tile < prm.num_p_tiles; tile += num_workers) {
            bool ok = mbar_wait_bounded(&acc_full[buf], acc_phase, abort_flag, GEMM_WAIT_LIMIT_NS);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (lane == 0) {
                    if (*abort_flag == 0) report_timeout(status_word, 4, 0);
                    *abort_flag = 1;
                }
                break;
            }
            tc_fence_after_sync();
            const long long p = static_cast<long long>(tile) * 128 + quarter * 32 + lane;
            const bool valid = p < prm.geo.P;
            const long long pp = valid ? p : 0;
            int tw, th;
            long long n;
            decode_tile(prm.geo, pp, n, th, tw);
            const long long plane = static_cast<long long>(prm.geo.H) * prm.geo.W;
            T* out0 = y + (n * prm.K + k0) * plane + static_cast<long long>(2 * th) * prm.geo.W + 2 * tw;
            const bool row1_ok = 2 * th + 1 < prm.geo.H;
            const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                    static_cast<uint32_t>(buf * FK_ACC_COLS);
            for (int kc = 0; kc < kcount; kc += 4) {
                // m[pos][kk]: the 16 position accumulators of output channels kc .. kc+3
                uint32_t m[16][4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint32_t r[16];
                    const uint32_t a = t_addr + static_cast<uint32_t>(kc + q * 4 * FK_N);
                    tmem_ld_4x_32x4_sync(a, a + FK_N, a + 2 * FK_N, a + 3 * FK_N, r);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) m[q * 4 + j][kk] = r[j * 4 + kk];
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    if (kc + kk >= kcount) break;
                    // Y = A^T M A with M[xi][nu] = m[xi*4+nu]
                    float t[2][4];
#pragma unroll
                    for (int nu = 0; nu < 4; ++nu) {
                        float col[4], o[2];
#pragma unroll
                        for (int xi = 0; xi < 4; ++xi) col[xi] = __uint_as_float(m[xi * 4 + nu][kk]);
                        mat_apply<2, 4>(typename Wm::At{}, col, o);
                        t[0][nu] = o[0];
                        t[1][nu] = o[1];
                    }
                    const float b = load_bias(bias, k0 + kc + kk);
                    float o0[2], o1[2];
                    mat_apply<2, 4>(typename Wm::At{}, t[0], o0);
                    mat_apply<2, 4>(typename Wm::At{}, t[1], o1);
                    if (valid) {
                        T* q = out0 + (kc + kk) * plane;
                        if constexpr (sizeof(T) == 4) {
                            *reinterpret_cast<float2*>(q) = make_float2(o0[0] + b, o0[1] + b);
                            if (row1_ok) *reinterpret_cast<float2*>(q + prm.geo.W) = make_float2(o1[0] + b, o1[1] + b);
                        } else {
                            *reinterpret_cast<uint32_t*>(q) = pack2(o0[0] + b, o0[1] + b);
                            if (row1_ok) *reinterpret_cast<uint32_t*>(q + prm.geo.W) = pack2(o1[0] + b, o1[1] + b);
                        }
                    }
                }
            }
            // accumulators drained: hand the TMEM buffer back to the MMA thread
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
            buf ^= 1;
            if (buf == 0) acc_phase ^= 1u;
        }
    } else {
        // ------------------------------ input transform (warps 8-23) ------------------------------
        const int wi = warp - FK_TR_WARP0;     // channel of the stage owned by this warp
        // byte offset of this lane's 4 tiles inside a position plane: box, channel row, swizzled 16-byte chunk
        const uint32_t voff = static_cast<uint32_t>((lane >> 4) * 2048 + wi * 128 +
                                                    ((((lane & 15) >> 1) ^ (wi & 7)) << 4) + (lane & 1) * 8);
        pdl_wait();   // x may have been written by the kernel before this one
        uint32_t vs = 0, v_phase = 0;   // V stage to fill next and the parity of its full barrier
        int tile = worker;
        int s = 0;
        bool ok = true;
        // geometry of the unit whose loads are issued next (the unit being processed no longer needs it)
        FkUnitGeo g = fk_decode(prm.geo, prm.C, static_cast<long long>(tile) * 128 + 4 * lane);
        FkRaw cur;
        if (tile < prm.num_p_tiles) fk_load(x, prm.geo, g, wi, wi < prm.C, cur);

        while (tile < prm.num_p_tiles) {
            // issue the loads of the next unit before working on this one
            int tile_n = tile, s_n = s + 1;
            if (s_n == nstages) {
                s_n = 0;
                tile_n = tile + num_workers;
                if (tile_n < prm.num_p_tiles) g = fk_decode(prm.geo, prm.C, static_cast<long long>(tile_n) * 128 + 4 * lane);
            }
            FkRaw nxt;
            if (tile_n < prm.num_p_tiles) {
                const int c = s_n * FK_CSTEP + wi;
                fk_load(x, prm.geo, g, c, c < prm.C, nxt);
            }
            ok = mbar_wait_bounded(&v_empty[vs], v_phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) {
                if (lane == 0) {
                    if (*abort_flag == 0) report_timeout(status_word, 1, 0);
                    *abort_flag = 1;
                }
                break;
            }
            fk_transform_store(cur, v_smem + vs * FK_V_STAGE_BYTES, voff);
            fence_proxy_async_smem();   // the tensor core reads these generic-proxy writes through the async proxy
            __syncwarp();
            if (lane == 0) mbar_arrive(&v_full[vs]);
            if (++vs == FK_V_STAGES) { vs = 0; v_phase ^= 1u; }
            tile = tile_n;
            s = s_n;
            cur = nxt;
        }
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
    if (warp == FK_EPI_WARP0) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 2 * FK_ACC_COLS);
    }
}

}  // namespace sdw
