// Step (ii) of Section "Techniques": the "element-wise multiplication" of the transformed
// filter and activation.  With C input channels it is, for each of the a*a transform
// positions, the dense contraction  M[pos][k][p] = sum_c U[pos][k][c] * V[pos][c][p],
// i.e. a batched GEMM.  It runs on the tcgen05 tensor cores: operands are brought into
// shared memory by TMA (128-byte swizzle), accumulated in fp32 in tensor memory, and the
// result is rounded once to fp16 and written back by TMA stores.
//
// Orientation: the 128 TMEM lanes hold 128 consecutive tiles p (operand A = V, M-major), the
// TMEM columns hold n_tile output channels k (operand B = U, K-major), n_tile any multiple of
// 16 up to 256, so that channel counts such as 320 = 2 x 160 waste nothing.
//
// The instantiations share the code.  CTAS == 1: one persistent CTA per SM, 128 p x n_tile k per
// tile.  CTAS == 2: persistent CTA pairs (a 2-CTA cluster) drive one 256-row MMA (cta_group::2);
// each CTA loads its own 128 p rows of V but only half of the n_tile rows of U, which cuts the
// bytes fetched from L2 per MMA cycle -- the measured limit of the single-CTA shape.  The leader
// (even rank) issues the MMAs; completion is signalled to the barriers of both CTAs.
//
// Filter-resident mode (single CTAs, layers whose filter block n_tile x C fits beside the ring): a layer with few
// channels and many tiles re-reads the same n_tile x C filter block for every tile p, and at C = K = 256 those
// re-reads are two thirds of the bytes that cross from L2 to the SMs, which is what bounds the kernel there.  The CTAs
// then work in groups: a group takes whole (pos, k-tile) pairs, its CTAs share out the tiles p of a pair, load the
// pair's filter block once into a resident buffer and stream only V through the ring.
//
// Two blocks of tiles per CTA tile (DUAL, single CTAs): a stage holds V of 256 tiles and one filter box, every k-step
// issues one MMA per block of 128 tiles into the two accumulator buffers, which the epilogue then drains one after
// the other.  The filter box is fetched once per 256 instead of once per 128 tiles (like a CTA pair, but on one SM
// and with programmatic dependent launch), and a layer of 2 j blocks of tiles makes half as many CTA tiles, which
// turns two waves into one where the tiles number about twice the SMs.  The accumulators are no longer
// double-buffered across tiles, so this pays where a CTA has one or two tiles or many stages per tile.
//
// One persistent CTA (pair) per SM (pair) walks the list of (pos, k-tile, p-tile) output tiles.
//   warp 0   : TMA producer        (one lane)
//   warp 1   : TMEM owner + MMA issuer (one lane)
//   warps 2-9: epilogue in two groups of four warps (one TMEM lane quarter per warp); group g drains
//              channels [g * epi_rows, (g + 1) * epi_rows) of the tile; TMEM accumulators are double-buffered so
//              the epilogue of tile i overlaps the MMAs of tile i+1.  A thread owns one tile p and
//              reads its channels from TMEM; the fp16 results are transposed through a shared-memory
//              staging buffer [k][128 p] and leave with one TMA store per epi_rows channels, so M is
//              written in full 256-byte rows.
#pragma once
#include <cuda_fp16.h>

#include "ptx.cuh"
#include "transforms.cuh"

namespace sdw {

// first device-side failure wins: low byte = status code (6 = timeout), next byte = which wait gave up
__device__ __forceinline__ void report_timeout(int* status_word, int where, uint32_t rank) {
    atomicCAS(status_word, 0, 6 | ((where | (static_cast<int>(rank) << 4)) << 8));
}

constexpr int GEMM_BLOCK_P = 128;  // tiles per output tile (TMEM lanes, UMMA M)
constexpr int GEMM_BLOCK_C = 64;   // input channels per pipeline stage (one 128-byte swizzle row of U)
constexpr int GEMM_MAX_N = 256;    // output channels per output tile (UMMA N), multiple of 16
constexpr int GEMM_THREADS = 320;  // warp 0 producer, warp 1 MMA, warps 2-9 epilogue (two groups of four)
constexpr int GEMM_LAUNCH_THREADS = GEMM_THREADS + 32;   // ... and warp 10: the second producer (filters) of the streaming kernel
constexpr int PIPE_TRANSFORM_THREADS = 320;                            // pipelined mode: warps 10-19 run the transforms, each on its own
constexpr int PIPE_THREADS = GEMM_THREADS + PIPE_TRANSFORM_THREADS;
constexpr int GEMM_MAX_STAGES = 8;
constexpr uint64_t GEMM_WAIT_LIMIT_NS = 2000000000ull;  // a wait longer than 2 s is reported, not spun on

struct GemmSmemLayout {
    static constexpr int A_BYTES = GEMM_BLOCK_P * GEMM_BLOCK_C * 2;          // two [64 p][64 c] boxes
    static constexpr int A_BOX_BYTES = 64 * GEMM_BLOCK_C * 2;
    static constexpr int EPI_ROW_BYTES = GEMM_BLOCK_P * 2;                   // one staged row: 128 p fp16
    static constexpr int BAR_BYTES = (4 * GEMM_MAX_STAGES + 6) * 8 + 16 + 16;   // barriers, two words, four item slots
    // `rows` = rows of U this CTA loads per stage: n_tile (single CTA) or n_tile / 2 (CTA pair)
    __host__ __device__ static constexpr int b_bytes(int rows) { return rows * GEMM_BLOCK_C * 2; }
    __host__ __device__ static constexpr int stage_bytes(int rows) {
        return (A_BYTES + b_bytes(rows) + 1023) / 1024 * 1024;
    }
    // 8-bit filters: a stage also holds the raw bytes of its filter box (64 per row) next to their fp16 expansion
    __host__ __device__ static constexpr int raw_bytes(int rows) { return rows * GEMM_BLOCK_C; }
    __host__ __device__ static constexpr int stage_bytes_u8(int rows) {
        return (A_BYTES + b_bytes(rows) + raw_bytes(rows) + 1023) / 1024 * 1024;
    }
    // epilogue staging: `bufs` buffers of [epi_rows k][128 p] fp16
    __host__ __device__ static constexpr int epi_bytes(int epi_rows, int bufs) {
        return bufs * epi_rows * EPI_ROW_BYTES;
    }
    // dynamic shared memory for `stages` stages, including slack to align the base to 1024 bytes; `resident` =
    // bytes of filter blocks kept in shared memory across tiles (0 when the filters travel with the stages)
    __host__ __device__ static constexpr int dyn_bytes(int rows, int stages, int epi_rows, int bufs, int resident = 0) {
        return stages * stage_bytes(rows) + resident + epi_bytes(epi_rows, bufs) + BAR_BYTES + 1024;
    }
};

struct GemmParams {
    const uint32_t* wt_header;   // header of the transformed filter (see wt_header_ok)
    int K, tile;                 // what the header must say (C is below)
    int num_k_tiles;   // ceil(K / n_tile)
    int num_p_tiles;   // tiles of 128 p (single CTA) or 256 p (CTA pair) in this pass
    int num_pos;       // a*a
    int num_c_blocks;  // ceil(C / 64)
    int C;             // input channels (for the k-steps of the last block)
    int n_tile;        // UMMA N
    int stages;
    int epi_rows;      // channels staged per TMA store and epilogue group: n_tile or n_tile / 2, multiple of 16
    int epi_bufs;      // staging buffers = epilogue groups with work (1 or 2)
    int epi_chunks;    // TMA stores per group and tile: a group drains epi_rows * epi_chunks channels
    int epi_dbuf;      // 1: a group alternates between two staging buffers of epi_rows channels, so that it rounds and
                       // stages one piece while the TMA store still reads the other (epi_bufs then counts both)
    int epi_stm;       // 1: staging through stmatrix into two swizzled boxes of 64 tiles (tmM has that box); 0: 2-byte
                       // stores into one plain box of 128 tiles (launches of one tile per CTA, whose tail it shortens)
    int resident;      // 1: the filter blocks of a (position, k-tile) stay in shared memory while the CTA walks the
                       // tiles p of that pair (stages then hold V only)
    int group;         // filter-resident mode: CTAs that share out the tiles of one (position, k-tile) pair
    int epi_alias;     // 1: no CTA has more than one tile, so the epilogue stages its rows in the (by then idle) first
                       // pipeline stages instead of a buffer of its own, which leaves room for one more stage
    int dual;          // 1: the kernel instantiation with two blocks of 128 tiles per CTA tile (host side only)
    long long p_stride;  // tiles per pass (row pitch of V and M)
    const float* scales; // 8-bit filters: S[pos][kpad], the factor of every (position, output channel) row
    int kpad;            // Kb * 16
    int raw_slots;       // 8-bit filters: slots of the raw ring (at most GEMM_MAX_STAGES)
    FastDiv fd_p, fd_k, fd_keys;   // divisions by num_p_tiles, num_k_tiles, num_k_tiles * num_pos (the roles are single
                                   // threads: a hardware-less integer division is a few hundred cycles of their time)
};

// Pipelined mode (template flag PIPE): the three steps of a layer run inside ONE persistent launch.  V and M are rings
// of `ring` blocks of 128 tiles that stay in L2; ten extra warps per CTA pull transform items -- the activation
// transform of (block of tiles, group of input channels) and, `lead` blocks behind it, the output transform of (block,
// group of output channels) -- from an atomic queue, while the GEMM roles walk the (block, position, k-tile) tiles in
// block order.  Counters in global memory carry the dependencies:
//   v_ready[b]  activation-transform items of block b completed       (the producer waits for it_items before it loads V)
//   m_done[b]   epilogue groups that have stored their part of M of b (an output item waits for m_target; so does the
//               activation transform of block b + ring, which overwrites the V slot of b)
//   o_done[b]   output-transform items of block b completed           (the epilogue of block b + ring waits for ot_items
//               before it overwrites the M slot)
// Every item depends only on items earlier in queue order, and every role works through its list in order, so the
// earliest unfinished item can always run: the scheme cannot deadlock as long as all CTAs are resident (the launch is
// cooperative).  Every wait is bounded all the same and gives up through the status word and the abort word.
struct PipeParams {
    unsigned int* v_ready;
    unsigned int* m_done;
    unsigned int* o_done;
    unsigned int* q_head;      // next transform item
    int* abort_word;           // set by the first wait that gives up: every other wait then returns
    int num_pblocks;           // blocks of 128 tiles in the layer
    int ring;                  // ring slots (blocks of 128 tiles) of V and of M
    int lead;                  // the output items of block j - lead are queued behind the activation items of block j
    int it_items, ot_items;    // items per block: ceil(C / cg), ceil(K / kg)
    int cg, kg;                // channels per item
    unsigned int m_target;     // (position, k-tile) pairs x epilogue groups that store
    const __half* x;
    __half* V;                 // ring [pos][C][ring * 128]
    const __half* Mws;         // ring [pos][K][ring * 128]
    const __half* bias;
    __half* y;
    TileGeom geo;
    FastDiv fd64;              // division by 64 (pairs of tiles per block)
    int defer;                 // 1: a tile's stores are announced one tile later (needs ring > distance between a CTA's tiles)
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Spins until *ctr >= target.  Bounded: gives up after limit_ns, or as soon as the abort word is set.
__device__ __noinline__ bool wait_counter(const unsigned int* ctr, unsigned int target, const int* abort_word,
                                          uint64_t limit_ns) {
    unsigned int polls = 0;
    uint64_t t0 = 0;
    for (;;) {
        unsigned int v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
        if (v >= target) return true;
        if ((++polls & 63u) == 0u) {
            if (*reinterpret_cast<const volatile int*>(abort_word) != 0) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) return false;
        }
        __nanosleep(40);
    }
}
// Publishes the stores made before it (by this thread, and by the threads it has synchronised with) and counts up.
__device__ __forceinline__ void signal_counter(unsigned int* ctr) {
    __threadfence();
    atomicAdd(ctr, 1u);
}
// The same as one release operation (for a thread whose own earlier writes have already completed).
__device__ __forceinline__ void signal_counter_release(unsigned int* ctr) {
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ctr) : "memory");
}

// tmV: fp16 [pos][C][Pstride]   box {64 p, 64 c, 1},      128B swizzle  (A operand; rows c >= C read as 0)
// tmU: fp16 [pos][Cb][Kb][16][64] box {64 c, 16 k, 1, n_tile/16, 1}, 128B swizzle (B operand: n_tile rows of 128
//      bytes in k order; blocks past Kb read as 0)
// tmM: fp16 [pos][K][Pstride]   box {64 p, epi_rows k, 1}, 128B swizzle (result; rows k >= K are clipped), or, with
//      epi_stm == 0 (one tile per CTA, 8-bit filters): box {128 p, epi_rows k, 1}, no swizzle
// RES: the filter-resident mode, DUAL: two blocks of 128 tiles per CTA tile; separate instantiations, so that the
// plain streaming kernel pays nothing for them.
// U8: 8-bit filters (see filter_quantize_kernel).  The producer brings the bytes of a filter box into the stage's raw
// area; the eight epilogue warps, idle during a mainloop, expand them to fp16 in the swizzled operand layout (an
// integer of at most 127 is exact in fp16) and complete the stage's barrier; the scale of every (position, output
// channel) row multiplies the accumulator in the epilogue.  Half the filter bytes cross HBM and L2; the contraction is
// still kind::f16.  Meant for the weight-streaming layers (one tile per CTA): with several tiles per CTA the epilogue
// of one tile no longer overlaps the mainloop of the next.
// STM: the epilogue stages M through stmatrix into two swizzled boxes of 64 tiles (launches whose CTAs have several
// tiles); without it, through 2-byte stores into one plain box of 128 tiles (one tile per CTA, 8-bit filters).  A
// template flag like the others: with both forms in one kernel either was 1-3 % slower.
template <int CTAS, bool RES = false, bool DUAL = false, bool PIPE = false, bool U8 = false, bool STM = true>
__global__ void __launch_bounds__(PIPE ? PIPE_THREADS : GEMM_LAUNCH_THREADS, 1)
wino_gemm_kernel(const __grid_constant__ CUtensorMap tmU, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmM, const GemmParams prm, int* __restrict__ status_word,
                 const PipeParams pp) {
    using L = GemmSmemLayout;
    static_assert(!PIPE || (CTAS == 1 && !DUAL), "the pipelined mode runs single CTAs, one block of tiles per CTA tile");
    static_assert(!U8 || (CTAS == 1 && !RES && !DUAL && !PIPE), "8-bit filters: single CTAs, streaming mode");
    static_assert(!(U8 && STM), "8-bit filters use the plain staging (their scales are fetched per column)");
    // The activation transform before this kernel has waited for everything before it, so the filter header is
    // final: its load is issued first and looked at after the set-up below (uniform over the CTA).
    const uint4 wt_hdr = *reinterpret_cast<const uint4*>(prm.wt_header);
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int b_rows = prm.n_tile / CTAS;            // rows of U this CTA loads per stage
    static_assert(!RES || CTAS == 1, "filter-resident mode is for single CTAs");
    static_assert(!DUAL || (CTAS == 1 && !RES), "two blocks of tiles per CTA: single CTAs, streaming mode");
    constexpr bool resident = RES;
    // Two producers (single CTAs, streaming): a thread that issues TMA loads spends about 100 ns per load on its own
    // instruction latencies, so the boxes of V (warp 0) and the filter boxes (warp 10) go out from two warps.
    constexpr bool SPLIT = CTAS == 1 && !RES && !PIPE && !U8;
    constexpr int PT = DUAL ? 2 : 1;                 // blocks of 128 tiles p per CTA tile (one accumulator each)
    constexpr int a_bytes = PT * L::A_BYTES;         // V part of a stage
    const int stage_bytes = resident ? L::A_BYTES : (PT - 1) * L::A_BYTES + L::stage_bytes(b_rows);
    const int ures_cb_bytes = L::b_bytes(prm.n_tile);                       // one 64-channel block of the resident filters
    // 8-bit filters: the same area holds a ring of raw filter boxes (64 bytes per row), deeper than the operand ring
    [[maybe_unused]] const int raw_slot_bytes = L::raw_bytes(b_rows);
    const int ures_bytes = resident ? prm.num_c_blocks * ures_cb_bytes : (U8 ? prm.raw_slots * raw_slot_bytes : 0);
    const int stages = prm.stages;
    const uint32_t cta_rank = CTAS == 2 ? cluster_ctarank() : 0u;
    const bool leader = cta_rank == 0;
    const int worker = blockIdx.x / CTAS;            // index of this CTA (pair) among the persistent workers
    const int num_workers = gridDim.x / CTAS;
    uint8_t* ures_base = smem + stages * stage_bytes;
    uint8_t* epi_base = prm.epi_alias ? smem : ures_base + ures_bytes;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(ures_base + ures_bytes +
                                                     (prm.epi_alias ? 0 : L::epi_bytes(prm.epi_rows, prm.epi_bufs)));
    uint64_t* empty_bar = full_bar + GEMM_MAX_STAGES;
    uint64_t* acc_full_bar = empty_bar + GEMM_MAX_STAGES;
    uint64_t* acc_empty_bar = acc_full_bar + 2;
    uint64_t* ures_full_bar = acc_empty_bar + 2;     // the resident filter block has arrived
    uint64_t* ures_empty_bar = ures_full_bar + 1;    // the MMAs that read it have completed
    uint64_t* raw_full_bar = ures_empty_bar + 1;     // 8-bit filters: the bytes of a raw slot have arrived
    uint64_t* raw_empty_bar = raw_full_bar + GEMM_MAX_STAGES;   // ... and have been expanded by all eight warps
    uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(raw_empty_bar + GEMM_MAX_STAGES);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_slot + 1);
    [[maybe_unused]] volatile unsigned int* item_slots = reinterpret_cast<volatile unsigned int*>(tmem_base_slot + 2);   // 4 words

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int num_tiles = prm.num_k_tiles * prm.num_p_tiles * prm.num_pos;
    constexpr uint32_t TMEM_COLS = 2 * GEMM_MAX_N;
    // The tiles of this worker, numbered i = 0 .. my_count - 1.  Streaming mode: every num_workers-th tile of the
    // list.  Filter-resident mode: the workers form groups of `group` CTAs; a group takes every num_groups-th
    // (position, k-tile) pair and its CTAs share out the tiles p of the pair round-robin, so that a CTA stays with
    // one filter block for many tiles while the CTAs of a group read neighbouring pieces of V at the same time.
    const int grp_size = resident ? prm.group : 1;
    const int num_groups = num_workers / grp_size;
    const int grp_id = worker / grp_size, grp_lane = worker - grp_id * grp_size;
    int run_len = 0;      // tiles per (position, k-tile) pair for this CTA
    int my_count;
    if constexpr (resident) {
        const int num_keys = prm.num_k_tiles * prm.num_pos;
        run_len = grp_lane < prm.num_p_tiles ? (prm.num_p_tiles - grp_lane + grp_size - 1) / grp_size : 0;
        my_count = grp_id < num_groups ? run_len * ((num_keys - grp_id + num_groups - 1) / num_groups) : 0;
        if (grp_id >= num_keys) my_count = 0;
    } else {
        my_count = worker < num_tiles ? (num_tiles - worker + num_workers - 1) / num_workers : 0;
    }
    auto tile_of = [&](int i) -> int {
        if constexpr (!resident) {
            return worker + i * num_workers;
        } else {
            const int r = i / run_len;
            return (grp_id + r * num_groups) * prm.num_p_tiles + grp_lane + (i - r * run_len) * grp_size;
        }
    };

    // tile -> (block of tiles pt, k-tile kt, position pos).  The plain list has the tiles p fastest (all CTAs at one
    // position: its filters are small and V streams); the pipelined streaming list has them slowest, so that the
    // CTAs move through the blocks of tiles together, behind the transform that produces them.
    auto decode = [&](int tile, int& pt, int& kt, int& pos) {
        if constexpr (PIPE && !RES) {
            const int keys = prm.num_k_tiles * prm.num_pos;
            pt = static_cast<int>(fast_div(static_cast<uint32_t>(tile), prm.fd_keys));
            const int key = tile - pt * keys;
            pos = static_cast<int>(fast_div(static_cast<uint32_t>(key), prm.fd_k));
            kt = key - pos * prm.num_k_tiles;
        } else {
            const int q = static_cast<int>(fast_div(static_cast<uint32_t>(tile), prm.fd_p));
            pt = tile - q * prm.num_p_tiles;
            pos = static_cast<int>(fast_div(static_cast<uint32_t>(q), prm.fd_k));
            kt = q - pos * prm.num_k_tiles;
        }
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full_bar[s], U8 ? 9 : (SPLIT ? 2 : 1));   // 8-bit filters: the producer and the eight converting warps
            mbar_init(&empty_bar[s], 1);
        }
        for (int s = 0; s < GEMM_MAX_STAGES; ++s) {
            mbar_init(&raw_full_bar[s], 1);
            mbar_init(&raw_empty_bar[s], 8);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full_bar[b], 1);
            mbar_init(&acc_empty_bar[b], 8 * CTAS);   // one arrival per epilogue warp of every CTA
        }
        mbar_init(ures_full_bar, 1);
        mbar_init(ures_empty_bar, 1);
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tmU);
        prefetch_tmap(&tmV);
        prefetch_tmap(&tmM);
    }
    if (warp == 1) {
        if constexpr (CTAS == 2) { tmem_alloc_pair(tmem_base_slot, TMEM_COLS); tmem_relinquish_pair(); }
        else { tmem_alloc(tmem_base_slot, TMEM_COLS); tmem_relinquish(); }
    }
    pdl_launch_dependents();
    tc_fence_before_sync();
    __syncthreads();
    if constexpr (CTAS == 2) cluster_sync_all();   // the peer's barriers are initialised before anyone signals them
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;

    const bool wt_ok = wt_hdr.x == WT_MAGIC && wt_hdr.y == static_cast<uint32_t>(prm.K) &&
                       wt_hdr.z == static_cast<uint32_t>(prm.C) && wt_hdr.w == static_cast<uint32_t>(prm.tile);
    if (!wt_ok) {
        // a filter buffer made for another layer: nothing is read from it, nothing is computed
        if (threadIdx.x == 0) atomicCAS(status_word, 0, 1 | (9 << 8));   // 1 = SDWINO_ERR_INVALID_ARG
    } else if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (resident && lane == 0) {
            // filter-resident mode: the filter block of a (position, k-tile) is loaded once, V streams through the ring
            const uint32_t smem_base = smem_u32(smem);
            const uint32_t ures_a = smem_u32(ures_base);
            const uint32_t ures_full_a = smem_u32(ures_full_bar);
            const uint32_t full0 = smem_u32(&full_bar[0]);
            auto load_filters = [&](int pos, int kt) {
                mbar_arrive_expect_tx_a32(ures_full_a, static_cast<uint32_t>(ures_bytes));
                for (int cb = 0; cb < prm.num_c_blocks; ++cb)
                    tma_load_5d_a32(ures_a + cb * ures_cb_bytes, &tmU, ures_full_a, cb, (kt * prm.n_tile) >> 4, pos);
            };
            int cur_key = -1;
            uint32_t reloads = 0;
            if (my_count > 0) {
                // the filters do not depend on the preceding kernel: the first block goes out before the wait
                int pt, kt, pos;
                decode(tile_of(0), pt, kt, pos);
                load_filters(pos, kt);
                cur_key = pos * prm.num_k_tiles + kt;
            }
            pdl_wait();   // V is written by the preceding kernel
            int stage = 0;
            uint32_t phase = 0;
            uint32_t sa = smem_base, fb = full0;
            bool ok = true;
            [[maybe_unused]] int seen_pt = -1;            // pipelined mode: the block whose counter was read ahead
            [[maybe_unused]] unsigned int seen = 0;
            for (int i = 0; i < my_count && ok; ++i) {
                int pt, kt, pos;
                decode(tile_of(i), pt, kt, pos);
                if (pos * prm.num_k_tiles + kt != cur_key) {
                    // the MMAs of the previous run of tiles have finished reading the resident block
                    ok = mbar_wait_bounded(ures_empty_bar, reloads & 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                    if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 5, cta_rank); break; }
                    ++reloads;
                    load_filters(pos, kt);
                    cur_key = pos * prm.num_k_tiles + kt;
                }
                int p0 = pt * GEMM_BLOCK_P;
                if constexpr (PIPE) {
                    // V of this block of tiles is written by the transform warps of this launch.  The counter was read
                    // one tile ahead (the read is a round trip to L2 on this one thread's critical path).
                    if (seen_pt != pt || seen < static_cast<unsigned int>(pp.it_items)) {
                        ok = wait_counter(&pp.v_ready[pt], static_cast<unsigned int>(pp.it_items), pp.abort_word, GEMM_WAIT_LIMIT_NS);
                        if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 12, cta_rank); break; }
                    }
                    fence_proxy_async_all();
                    p0 = (pt % pp.ring) * GEMM_BLOCK_P;
                    if (i + 1 < my_count) {
                        int kt1, pos1;
                        decode(tile_of(i + 1), seen_pt, kt1, pos1);
                        seen = ld_acquire_u32(&pp.v_ready[seen_pt]);
                    }
                }
                for (int c0 = 0; c0 < prm.C; c0 += GEMM_BLOCK_C) {
                    ok = mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                    if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 1, cta_rank); break; }
                    mbar_arrive_expect_tx_a32(fb, L::A_BYTES);
                    tma_load_3d_a32(sa, &tmV, fb, p0, c0, pos);
                    tma_load_3d_a32(sa + L::A_BOX_BYTES, &tmV, fb, p0 + 64, c0, pos);
                    sa += stage_bytes;
                    fb += 8;
                    if (++stage == stages) { stage = 0; phase ^= 1u; sa = smem_base; fb = full0; }
                }
            }
            if (!ok) *abort_flag = 1;
        } else if (U8 && lane == 0) {
            // 8-bit filters.  Two streams from one thread: the raw filter boxes, which come from HBM and depend on
            // nothing, run `lead` steps ahead of the boxes of V through a ring of their own; a step's operand stage is
            // completed by V (this thread) and by the warps that expand the raw box into it.
            const int R = prm.raw_slots, lead = R - 1;
            const int spt = prm.num_c_blocks;                  // steps per tile
            const int total = my_count * spt;
            const uint32_t smem_base = smem_u32(smem);
            const uint32_t raw_base = smem_u32(ures_base);
            const uint64_t u_policy = l2_policy_evict_first();
            bool ok = true;
            // running state of the two streams (no division in this single-thread loop)
            int r_slot = 0, r_cb = 0, r_tile = 0, r_kb = 0, r_pos = 0;
            uint32_t r_par = 1;                                // parity to wait for on raw_empty: passes in the first round
            int v_stage = 0, v_cb = 0, v_tile = 0, v_p0 = 0, v_pos = 0;
            uint32_t v_par = 1;
            if (total > 0) {
                int pt, kt;
                decode(tile_of(0), pt, kt, r_pos);
                r_kb = (kt * prm.n_tile) >> 4;
                v_p0 = pt * GEMM_BLOCK_P;
                v_pos = r_pos;
            }
            for (int j = 0; j < total + lead && ok; ++j) {
                if (j < total) {
                    ok = mbar_wait_bounded(&raw_empty_bar[r_slot], r_par, abort_flag, GEMM_WAIT_LIMIT_NS);
                    if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 8, cta_rank); break; }
                    const uint32_t rb = smem_u32(&raw_full_bar[r_slot]);
                    mbar_arrive_expect_tx_a32(rb, static_cast<uint32_t>(raw_slot_bytes));
                    tma_load_5d_hint_a32(raw_base + r_slot * raw_slot_bytes, &tmU, rb, r_cb, r_kb, r_pos, u_policy);
                    if (++r_slot == R) { r_slot = 0; r_par ^= 1u; }
                    if (++r_cb == spt) {
                        r_cb = 0;
                        if (++r_tile < my_count) {
                            int pt, kt;
                            decode(tile_of(r_tile), pt, kt, r_pos);
                            r_kb = (kt * prm.n_tile) >> 4;
                        }
                    }
                }
                if (j >= lead) {
                    if (j == lead) pdl_wait();                 // V is written by the preceding kernel
                    ok = mbar_wait_bounded(&empty_bar[v_stage], v_par, abort_flag, GEMM_WAIT_LIMIT_NS);
                    if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 1, cta_rank); break; }
                    const uint32_t fb = smem_u32(&full_bar[v_stage]);
                    const uint32_t sa = smem_base + v_stage * stage_bytes;
                    mbar_arrive_expect_tx_a32(fb, static_cast<uint32_t>(a_bytes));
                    tma_load_3d_a32(sa, &tmV, fb, v_p0, v_cb * GEMM_BLOCK_C, v_pos);
                    tma_load_3d_a32(sa + L::A_BOX_BYTES, &tmV, fb, v_p0 + 64, v_cb * GEMM_BLOCK_C, v_pos);
                    if (++v_stage == stages) { v_stage = 0; v_par ^= 1u; }
                    if (++v_cb == spt) {
                        v_cb = 0;
                        if (++v_tile < my_count) {
                            int pt, kt;
                            decode(tile_of(v_tile), pt, kt, v_pos);
                            v_p0 = pt * GEMM_BLOCK_P;
                        }
                    }
                }
            }
            if (total == 0) pdl_wait();
            if (!ok) *abort_flag = 1;
        } else if (!resident && lane == 0) {
            // the full barrier of a pair lives in the leader and counts the bytes of both CTAs
            const uint32_t tx_bytes = CTAS * (a_bytes + L::b_bytes(b_rows));
            // single-thread loop: shared-memory and barrier addresses are running 32-bit values
            const uint32_t smem_base = smem_u32(smem);
            const uint32_t full0_local = smem_u32(&full_bar[0]);
            const uint32_t full0 = CTAS == 2 ? map_to_cta(full0_local, 0) : full0_local;
            uint32_t sa = smem_base, fb = full0, fb_local = full0_local;
            // The filters do not depend on the preceding kernel (the activation transform), and everything before
            // that kernel has completed by the time this one runs: every activation transform waits for its
            // predecessors first and releases its dependents second, whatever came before it (a filter transform
            // releases its own dependents at once).  So the filter loads of the first ring-full of stages go out
            // before the wait, and the weight stream from HBM starts while the activation transform is still running.
            // (pipelined mode: the filters are read again for every block of tiles and must stay in L2)
            const uint64_t u_policy = PIPE ? l2_policy_evict_last() : l2_policy_evict_first();
            int pre = 0;
            if constexpr (SPLIT) {
                // the filters are the other producer's: this one brings the boxes of V
                pdl_wait();   // V is written by the preceding kernel
                int stage = 0;
                uint32_t phase = 0;
                bool ok = true;
                for (int i = 0; i < my_count && ok; ++i) {
                    int pt, kt, pos;
                    decode(tile_of(i), pt, kt, pos);
                    const int p0 = pt * PT * GEMM_BLOCK_P;
                    for (int c0 = 0; c0 < prm.C; c0 += GEMM_BLOCK_C) {
                        ok = mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                        if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 1, cta_rank); break; }
                        mbar_arrive_expect_tx_a32(fb, static_cast<uint32_t>(a_bytes));
#pragma unroll
                        for (int sub = 0; sub < PT; ++sub) {
                            tma_load_3d_a32(sa + sub * L::A_BYTES, &tmV, fb, p0 + sub * GEMM_BLOCK_P, c0, pos);
                            tma_load_3d_a32(sa + sub * L::A_BYTES + L::A_BOX_BYTES, &tmV, fb, p0 + sub * GEMM_BLOCK_P + 64, c0, pos);
                        }
                        sa += stage_bytes;
                        fb += 8;
                        if (++stage == stages) { stage = 0; phase ^= 1u; sa = smem_base; fb = full0; }
                    }
                }
                if (!ok) *abort_flag = 1;
            } else {
            if constexpr (CTAS == 1) {
                uint32_t sa_u = smem_base + a_bytes, fb_u = full0;
                for (int i = 0; i < my_count && pre < stages; ++i) {
                    int pt, kt, pos;
                    decode(tile_of(i), pt, kt, pos);
                    const int k0 = kt * prm.n_tile;
                    for (int c0 = 0; c0 < prm.C && pre < stages; c0 += GEMM_BLOCK_C) {
                        mbar_arrive_expect_tx_a32(fb_u, tx_bytes);
                        tma_load_5d_hint_a32(sa_u, &tmU, fb_u, c0 >> 6, k0 >> 4, pos, u_policy);
                        sa_u += stage_bytes;
                        fb_u += 8;
                        ++pre;
                    }
                }
            }
            pdl_wait();   // V is written by the preceding kernel
            int stage = 0;
            int issued = 0;
            uint32_t phase = 0;
            bool ok = true;
            [[maybe_unused]] int seen_pt = -1;            // pipelined mode: the block whose counter was read ahead
            [[maybe_unused]] unsigned int seen = 0;
            for (int i = 0; i < my_count && ok; ++i) {
                int pt, kt, pos;
                decode(tile_of(i), pt, kt, pos);
                int p0 = (pt * CTAS * PT + static_cast<int>(cta_rank)) * GEMM_BLOCK_P;
                if constexpr (PIPE) {
                    // V of this block of tiles is written by the transform warps of this launch (counter read one
                    // tile ahead, as in the filter-resident producer)
                    if (seen_pt != pt || seen < static_cast<unsigned int>(pp.it_items)) {
                        ok = wait_counter(&pp.v_ready[pt], static_cast<unsigned int>(pp.it_items), pp.abort_word, GEMM_WAIT_LIMIT_NS);
                        if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 12, cta_rank); break; }
                    }
                    fence_proxy_async_all();
                    p0 = (pt % pp.ring) * GEMM_BLOCK_P;
                    if (i + 1 < my_count) {
                        int kt1, pos1;
                        decode(tile_of(i + 1), seen_pt, kt1, pos1);
                        seen = ld_acquire_u32(&pp.v_ready[seen_pt]);
                    }
                }
                const int k0 = kt * prm.n_tile + static_cast<int>(cta_rank) * b_rows;
                for (int c0 = 0; c0 < prm.C; c0 += GEMM_BLOCK_C) {
                    if (issued < pre) {
                        // the barrier is armed and the filter box is on its way: add the boxes of V
#pragma unroll
                        for (int sub = 0; sub < PT; ++sub) {
                            tma_load_3d_a32(sa + sub * L::A_BYTES, &tmV, fb, p0 + sub * GEMM_BLOCK_P, c0, pos);
                            tma_load_3d_a32(sa + sub * L::A_BYTES + L::A_BOX_BYTES, &tmV, fb, p0 + sub * GEMM_BLOCK_P + 64, c0, pos);
                        }
                        ++issued;
                        sa += stage_bytes;
                        fb += 8;
                        fb_local += 8;
                        if (++stage == stages) { stage = 0; phase ^= 1u; sa = smem_base; fb = full0; fb_local = full0_local; }
                        continue;
                    }
                    ok = mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                    if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 1, cta_rank); break; }
                    if constexpr (CTAS == 2) {
                        if (leader) mbar_arrive_expect_tx_a32(fb_local, tx_bytes);
                        tma_load_3d_pair(sa, &tmV, fb, p0, c0, pos);
                        tma_load_3d_pair(sa + L::A_BOX_BYTES, &tmV, fb, p0 + 64, c0, pos);
                        tma_load_5d_pair(sa + L::A_BYTES, &tmU, fb, c0 >> 6, k0 >> 4, pos);
                    } else {
                        mbar_arrive_expect_tx_a32(fb, tx_bytes);
#pragma unroll
                        for (int sub = 0; sub < PT; ++sub) {
                            tma_load_3d_a32(sa + sub * L::A_BYTES, &tmV, fb, p0 + sub * GEMM_BLOCK_P, c0, pos);
                            tma_load_3d_a32(sa + sub * L::A_BYTES + L::A_BOX_BYTES, &tmV, fb, p0 + sub * GEMM_BLOCK_P + 64, c0, pos);
                        }
                        tma_load_5d_hint_a32(sa + a_bytes, &tmU, fb, c0 >> 6, k0 >> 4, pos, u_policy);
                    }
                    sa += stage_bytes;
                    fb += 8;
                    fb_local += 8;
                    if (++stage == stages) { stage = 0; phase ^= 1u; sa = smem_base; fb = full0; fb_local = full0_local; }
                }
            }
            if (!ok) *abort_flag = 1;
            }   // !SPLIT
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0 && leader) {
            const uint32_t idesc = make_idesc_f16_f32(GEMM_BLOCK_P * CTAS, prm.n_tile, true, false);
            // This loop is executed by ONE thread, so every instruction in it costs its full latency: the
            // descriptors of stage 0 are built once and then only advanced by additions (the 14-bit
            // address field cannot overflow inside 227 KB of shared memory).
            //   A (M-major): 16 channels = 16 rows of 128 bytes = +2048 bytes; the two 64-wide p blocks are
            //   A_BOX_BYTES apart.  B (K-major): 16 channels = +32 bytes along the swizzled 128-byte row.
            const uint32_t smem_base = smem_u32(smem);
            const uint64_t adesc0 = make_smem_desc_sw128(smem_base, L::A_BOX_BYTES, 1024);
            const uint64_t bdesc0 = make_smem_desc_sw128(smem_base + a_bytes, 16, 1024);
            const uint64_t stage_step = static_cast<uint64_t>(stage_bytes >> 4);
            const uint64_t ures_desc0 = make_smem_desc_sw128(smem_u32(ures_base), 16, 1024);
            const uint64_t ures_step = static_cast<uint64_t>(ures_cb_bytes >> 4);
            int cur_key = -1;          // filter-resident mode: the (position, k-tile) whose filters are in shared memory
            uint32_t loads_seen = 0;
            uint64_t adesc = adesc0, bdesc = bdesc0;
            const uint32_t full0_a = smem_u32(&full_bar[0]), empty0_a = smem_u32(&empty_bar[0]);
            uint32_t full_a = full0_a, empty_a = empty0_a;
            const int last_ksteps = ((prm.C - (prm.num_c_blocks - 1) * GEMM_BLOCK_C) + 15) / 16;  // 1..4
            const int full_blocks = last_ksteps == 4 ? prm.num_c_blocks : prm.num_c_blocks - 1;
            int stage = 0;
            uint32_t phase = 0;
            int buf = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int i = 0; i < my_count && ok; ++i) {
                const int tile = tile_of(i);
                int key = 0;
                if (resident) {
                    key = static_cast<int>(fast_div(static_cast<uint32_t>(tile), prm.fd_p));      // pos * num_k_tiles + kt
                    if (key != cur_key) {
                        ok = mbar_wait_bounded(ures_full_bar, loads_seen & 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                        if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 6, cta_rank); break; }
                        ++loads_seen;
                        cur_key = key;
                    }
                }
                ok = mbar_wait_bounded(&acc_empty_bar[buf], acc_phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                if constexpr (DUAL) {   // this tile fills both accumulator buffers
                    if (ok) ok = mbar_wait_bounded(&acc_empty_bar[1], acc_phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                }
                if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 2, cta_rank); break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(buf * GEMM_MAX_N);
                [[maybe_unused]] const uint32_t d_tmem1 = tmem_base + static_cast<uint32_t>(GEMM_MAX_N);
                [[maybe_unused]] constexpr uint64_t a_sub = static_cast<uint64_t>(L::A_BYTES >> 4);   // second block of tiles
                for (int cb = 0; cb < prm.num_c_blocks; ++cb) {
                    if (!mbar_try_wait_a32(full_a, phase)) {
                        ok = mbar_wait_slow(&full_bar[stage], phase, abort_flag, GEMM_WAIT_LIMIT_NS);
                        if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 3, cta_rank); break; }
                    }
                    tc_fence_after_sync();
                    const uint64_t bd = resident ? ures_desc0 + static_cast<uint64_t>(cb) * ures_step : bdesc;
                    if (cb < full_blocks) {
                        if constexpr (CTAS == 2) {
                            umma_f16_pair(d_tmem, adesc, bdesc, idesc, static_cast<uint32_t>(cb));
                            umma_f16_pair_acc(d_tmem, adesc + 128, bdesc + 2, idesc);
                            umma_f16_pair_acc(d_tmem, adesc + 256, bdesc + 4, idesc);
                            umma_f16_pair_acc(d_tmem, adesc + 384, bdesc + 6, idesc);
                        } else {
                            umma_f16(d_tmem, adesc, bd, idesc, static_cast<uint32_t>(cb));
                            umma_f16_acc(d_tmem, adesc + 128, bd + 2, idesc);
                            umma_f16_acc(d_tmem, adesc + 256, bd + 4, idesc);
                            umma_f16_acc(d_tmem, adesc + 384, bd + 6, idesc);
                            if constexpr (DUAL) {
                                umma_f16(d_tmem1, adesc + a_sub, bd, idesc, static_cast<uint32_t>(cb));
                                umma_f16_acc(d_tmem1, adesc + a_sub + 128, bd + 2, idesc);
                                umma_f16_acc(d_tmem1, adesc + a_sub + 256, bd + 4, idesc);
                                umma_f16_acc(d_tmem1, adesc + a_sub + 384, bd + 6, idesc);
                            }
                        }
                    } else {
                        for (int s = 0; s < last_ksteps; ++s) {
                            if constexpr (CTAS == 2)
                                umma_f16_pair(d_tmem, adesc + 128 * s, bdesc + 2 * s, idesc, (cb > 0 || s > 0) ? 1u : 0u);
                            else
                                umma_f16(d_tmem, adesc + 128 * s, bd + 2 * s, idesc, (cb > 0 || s > 0) ? 1u : 0u);
                            if constexpr (DUAL)
                                umma_f16(d_tmem1, adesc + a_sub + 128 * s, bd + 2 * s, idesc, (cb > 0 || s > 0) ? 1u : 0u);
                        }
                    }
                    if constexpr (CTAS == 2) umma_commit_pair_a32(empty_a);
                    else umma_commit_a32(empty_a);
                    adesc += stage_step;
                    bdesc += stage_step;
                    full_a += 8;
                    empty_a += 8;
                    if (++stage == stages) {
                        stage = 0; phase ^= 1u; adesc = adesc0; bdesc = bdesc0; full_a = full0_a; empty_a = empty0_a;
                    }
                }
                if (!ok) break;
                if constexpr (CTAS == 2) umma_commit_pair(&acc_full_bar[buf]);
                else umma_commit(&acc_full_bar[buf]);
                if constexpr (DUAL) umma_commit(&acc_full_bar[1]);
                // the last tile of a run: once its MMAs have completed the resident filters may be replaced
                if (resident && i + 1 < my_count &&
                    static_cast<int>(fast_div(static_cast<uint32_t>(tile_of(i + 1)), prm.fd_p)) != key)
                    umma_commit(ures_empty_bar);
                if constexpr (DUAL) {
                    acc_phase ^= 1u;          // both buffers were used: buf stays 0
                } else {
                    buf ^= 1;
                    if (buf == 0) acc_phase ^= 1u;
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp < GEMM_THREADS / 32) {
        // ------------------------------ epilogue ------------------------------
        const int quarter = warp & 3;          // TMEM lanes this warp may read: 32*quarter .. +31
        pdl_wait();   // nothing is written to global memory before the predecessor has completed
        const int group = (warp - 2) >> 2;           // 0: warps 2-5, 1: warps 6-9
        const int group_tid = threadIdx.x - 64 - group * 128;
        int buf = 0;
        uint32_t acc_phase = 0;
        // the accumulator-empty barrier of a pair lives in the leader
        const uint32_t acc_empty_addr0 = CTAS == 2 ? map_to_cta(smem_u32(&acc_empty_bar[0]), 0) : 0u;
        // one iteration per accumulator: a tile of two blocks of 128 tiles p (DUAL) fills both buffers, which are
        // drained in turn exactly as two consecutive tiles would be
        int stg_seq = 0;                       // pieces staged so far by this group (selects the staging buffer)
        [[maybe_unused]] int pend_pt = -1;     // pipelined mode, group_tid 0: block whose stores are to be announced
        [[maybe_unused]] int cv_stage = 0;     // 8-bit filters: the stage these warps expand next
        [[maybe_unused]] uint32_t cv_phase = 0;
        [[maybe_unused]] int cv_raw = 0;       // ... and the raw slot they read next
        [[maybe_unused]] uint32_t cv_raw_par = 0;
        for (int i2 = 0; i2 < my_count * PT; ++i2) {
            int pt, kt, pos;
            decode(tile_of(i2 / PT), pt, kt, pos);
            pt = pt * PT + (i2 % PT);
            if constexpr (U8) {
                // Expand the filter bytes of every stage of this tile: thread -> (row, 16 channels) of the box; the
                // 16 bytes become two 16-byte pieces of the row's 128 bytes, placed where the 128-byte swizzle puts
                // them (piece j of row r at position j ^ (r & 7)).  q + 128 is a byte; 0x6400 | byte is the fp16
                // number 1024 + byte, and subtracting 1152 leaves q exactly.
                const int ct = static_cast<int>(threadIdx.x) - 64;       // 0 .. 255
                const __half2 bias1152 = __half2half2(__ushort_as_half(static_cast<unsigned short>(0x6480)));
                for (int cb = 0; cb < prm.num_c_blocks; ++cb) {
                    // the operand stage is free once the MMAs that read its previous contents have completed, and the
                    // raw box of this step has arrived (one lane polls, the warp follows)
                    bool cv_ok = true;
                    if (lane == 0) {
                        cv_ok = mbar_wait_bounded(&empty_bar[cv_stage], cv_phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS) &&
                                mbar_wait_bounded(&raw_full_bar[cv_raw], cv_raw_par, abort_flag, GEMM_WAIT_LIMIT_NS);
                    }
                    cv_ok = __all_sync(0xffffffffu, cv_ok);
                    if (!cv_ok) {
                        // This warp stops converting but does NOT leave: with the abort flag set the accumulator wait
                        // below fails for every warp, and each group then leaves through its named barrier together.
                        if (lane == 0) {
                            if (*abort_flag == 0) report_timeout(status_word, 15, cta_rank);
                            *abort_flag = 1;
                        }
                        break;
                    }
                    const uint8_t* raw = ures_base + cv_raw * raw_slot_bytes;
                    uint8_t* bop = smem + cv_stage * stage_bytes + a_bytes;
                    for (int idx = ct; idx < b_rows * 4; idx += 256) {
                        const int row = idx >> 2, q = idx & 3;
                        const uint4 v = *reinterpret_cast<const uint4*>(raw + row * GEMM_BLOCK_C + q * 16);
                        const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
                        uint32_t h[8];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint32_t lo = __byte_perm(wds[i], 0x64646464u, 0x4140);   // (0x6400 | b0, 0x6400 | b1)
                            uint32_t hi = __byte_perm(wds[i], 0x64646464u, 0x4342);   // (0x6400 | b2, 0x6400 | b3)
                            const __half2 l2 = __hsub2(*reinterpret_cast<const __half2*>(&lo), bias1152);
                            const __half2 h2 = __hsub2(*reinterpret_cast<const __half2*>(&hi), bias1152);
                            h[2 * i] = *reinterpret_cast<const uint32_t*>(&l2);
                            h[2 * i + 1] = *reinterpret_cast<const uint32_t*>(&h2);
                        }
                        uint8_t* rowp = bop + row * 128;
                        *reinterpret_cast<uint4*>(rowp + (((2 * q) ^ (row & 7)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
                        *reinterpret_cast<uint4*>(rowp + (((2 * q + 1) ^ (row & 7)) << 4)) = make_uint4(h[4], h[5], h[6], h[7]);
                    }
                    fence_proxy_async_smem();      // the MMA reads the operand through the async proxy
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(&full_bar[cv_stage]);
                        mbar_arrive(&raw_empty_bar[cv_raw]);
                    }
                    if (++cv_stage == stages) { cv_stage = 0; cv_phase ^= 1u; }
                    if (++cv_raw == prm.raw_slots) { cv_raw = 0; cv_raw_par ^= 1u; }
                }
            }
            // the staging buffer about to be overwritten must have been read by the TMA store that used it last
            if (group_tid == 0) { if (prm.epi_dbuf) tma_store_wait_read_pending<1>(); else tma_store_wait_read_pending<0>(); }
            [[maybe_unused]] unsigned int seen_o = 0;
            if constexpr (PIPE) {
                if (group_tid == 0 && pt >= pp.ring) seen_o = ld_acquire_u32(&pp.o_done[pt - pp.ring]);   // used before the store
            }
            bool ok = mbar_wait_bounded(&acc_full_bar[buf], acc_phase, abort_flag, GEMM_WAIT_LIMIT_NS);
            // The four warps of a group give up together or not at all (a warp that left on its own would leave the
            // other three at the group's named barrier for good); the same barrier orders the reuse of the buffer.
            ok = named_barrier_and(1 + group, 128, ok);
            if (!ok) {
                if (group_tid == 0) {
                    if (*abort_flag == 0) report_timeout(status_word, 4, cta_rank);
                    *abort_flag = 1;
                }
                break;
            }
            tc_fence_after_sync();
            const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                    static_cast<uint32_t>(buf * GEMM_MAX_N);
            const int p0 = ((PIPE ? pt % pp.ring : pt * CTAS) + static_cast<int>(cta_rank)) * GEMM_BLOCK_P + quarter * 32;
            const int k0 = kt * prm.n_tile;
            const bool p_ok = p0 < prm.p_stride;   // the second CTA of the last pair may hang over the pass
            // lane = tile p, registers = output channels: staging row k receives 32 consecutive p from
            // each warp (64 contiguous bytes, no bank conflict).  Group g owns staging buffer g.
            // a group drains its channels in epi_chunks pieces of epi_rows, one TMA store each
            const int chunks = prm.epi_chunks;
            for (int ch = 0; ch < chunks; ++ch) {
            const int row0 = (group * chunks + ch) * prm.epi_rows;
            if (row0 < prm.n_tile) {
                uint8_t* stg = epi_base + (prm.epi_dbuf ? group * 2 + (stg_seq & 1) : group) * prm.epi_rows * L::EPI_ROW_BYTES;
                ++stg_seq;
                if (ch > 0) {   // (the first piece of a tile is ordered by the barrier after the accumulator wait)
                    if (group_tid == 0) { if (prm.epi_dbuf) tma_store_wait_read_pending<1>(); else tma_store_wait_read_pending<0>(); }
                    if (group == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
                    else asm volatile("bar.sync 2, 128;" ::: "memory");
                }
                if constexpr (STM) {
                    // The staging buffer of a group is two boxes [epi_rows k][64 p] with the 128-byte swizzle of the
                    // TMA store.  A warp reads its 32 lanes as two halves of 16 in the fragment layout of stmatrix
                    // (thread t: lanes t / 4 and t / 4 + 8, columns 2 (t % 4), + 1 of every 8), rounds pairs of
                    // columns with one packed conversion and stores four transposed 8 x 8 blocks per instruction:
                    // matrix j of an instruction = tiles p 8 (j & 1) .. + 7, channels 8 (j >> 1) .. + 7 of a 16 x 16
                    // piece, and thread 8 j + i supplies the 16-byte row of channel i of that matrix.  The swizzle
                    // puts the eight rows of a matrix into eight different bank groups.
                    const uint32_t stg_a = smem_u32(stg);
                    const uint32_t sub_bytes = static_cast<uint32_t>(prm.epi_rows) * 128u;
                    const int mj = lane >> 3, mi = lane & 7;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int p_local = quarter * 32 + 16 * h + (mj & 1) * 8;
                        const uint32_t sub = stg_a + static_cast<uint32_t>(p_local >> 6) * sub_bytes;
                        const uint32_t pc = static_cast<uint32_t>((p_local & 63) >> 3);
                        const uint32_t t_h = t_addr + (static_cast<uint32_t>(16 * h) << 16) + static_cast<uint32_t>(row0);
                        auto store16 = [&](int c, const uint32_t* r) {
                            const uint32_t krow = static_cast<uint32_t>(c + (mj >> 1) * 8 + mi);
                            const __half2 a = __floats2half2_rn(__uint_as_float(r[0]), __uint_as_float(r[1]));
                            const __half2 b = __floats2half2_rn(__uint_as_float(r[2]), __uint_as_float(r[3]));
                            const __half2 c2 = __floats2half2_rn(__uint_as_float(r[4]), __uint_as_float(r[5]));
                            const __half2 d = __floats2half2_rn(__uint_as_float(r[6]), __uint_as_float(r[7]));
                            stmatrix_x4_trans(sub + krow * 128u + ((pc ^ (krow & 7u)) << 4),
                                              *reinterpret_cast<const uint32_t*>(&a), *reinterpret_cast<const uint32_t*>(&b),
                                              *reinterpret_cast<const uint32_t*>(&c2), *reinterpret_cast<const uint32_t*>(&d));
                        };
                        int col = 0;
                        for (; col + 64 <= prm.epi_rows; col += 64) {
                            uint32_t r[32];
                            tmem_ld_16x256_sync<8>(t_h + col, r);
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj) store16(col + 16 * jj, r + 8 * jj);
                        }
                        if (col + 32 <= prm.epi_rows) {
                            uint32_t r[16];
                            tmem_ld_16x256_sync<4>(t_h + col, r);
                            store16(col, r);
                            store16(col + 16, r + 8);
                            col += 32;
                        }
                        if (col + 16 <= prm.epi_rows) {
                            uint32_t r[8];
                            tmem_ld_16x256_sync<2>(t_h + col, r);
                            store16(col, r);
                        }
                    }
                } else {
                __half* dst = reinterpret_cast<__half*>(stg) + quarter * 32 + lane;
                // 8-bit filters: the factor of every output channel of this position (rows past K read padding)
                [[maybe_unused]] const float* sc = U8 ? prm.scales + static_cast<long long>(pos) * prm.kpad + k0 + row0 : nullptr;
                // (the scales of 16 or 32 columns are fetched as 16-byte vectors ahead of the accumulator load: one
                // scalar load per column cost 6 us on a 25 us GEMM; kpad is a multiple of 16, so a vector is in or out)
                auto load_scales = [&](int col, int n4, float4 (&s4)[8]) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        s4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (i < n4 && k0 + row0 + col + 4 * i < prm.kpad) s4[i] = __ldg(reinterpret_cast<const float4*>(sc + col) + i);
                    }
                };
                int col = 0;
                for (; col + 32 <= prm.epi_rows; col += 32) {
                    [[maybe_unused]] float4 s4[8];
                    if constexpr (U8) load_scales(col, 8, s4);
                    uint32_t r[32];
                    tmem_ld_32x32_sync(t_addr + row0 + col, r);
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        float v = __uint_as_float(r[i]);
                        if constexpr (U8) v *= reinterpret_cast<const float*>(s4)[i];
                        dst[(col + i) * GEMM_BLOCK_P] = __float2half_rn(v);
                    }
                }
                if (col < prm.epi_rows) {
                    [[maybe_unused]] float4 s4[8];
                    if constexpr (U8) load_scales(col, 4, s4);
                    uint32_t r[16];
                    tmem_ld_32x16_sync(t_addr + row0 + col, r);
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        float v = __uint_as_float(r[i]);
                        if constexpr (U8) v *= reinterpret_cast<const float*>(s4)[i];
                        dst[(col + i) * GEMM_BLOCK_P] = __float2half_rn(v);
                    }
                }
                }   // U8: plain staging
                fence_proxy_async_smem();
                if (group == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
                else asm volatile("bar.sync 2, 128;" ::: "memory");
                if (group_tid == 0) {
                    bool slot_free = true;
                    if constexpr (PIPE) {
                        // the slot of M still holds block pt - ring until its output transform has read it (the
                        // counter was read at the start of the tile)
                        if (ch == 0 && pt >= pp.ring) {
                            if (seen_o < static_cast<unsigned int>(pp.ot_items))
                                slot_free = wait_counter(&pp.o_done[pt - pp.ring], static_cast<unsigned int>(pp.ot_items),
                                                         pp.abort_word, GEMM_WAIT_LIMIT_NS);
                            if (!slot_free) {
                                if (*abort_flag == 0) report_timeout(status_word, 13, cta_rank);
                                *abort_flag = 1;
                            }
                            fence_proxy_async_all();
                        }
                    }
                    if (p_ok && (slot_free || *abort_flag == 0)) {
                        if constexpr (!STM) {
                            tma_store_3d_hint(&tmM, stg, p0 - quarter * 32, k0 + row0, pos, l2_policy_evict_last());
                        } else {
                            const uint64_t pol = l2_policy_evict_last();
                            tma_store_3d_hint(&tmM, stg, p0 - quarter * 32, k0 + row0, pos, pol);
                            tma_store_3d_hint(&tmM, stg + prm.epi_rows * 128, p0 - quarter * 32 + 64, k0 + row0, pos, pol);
                        }
                    }
                    tma_store_commit();
                    if constexpr (PIPE) {
                        if (ch == chunks - 1) {
                            if (pp.defer) {
                                // Announce the tile BEFORE this one: its stores were issued a whole tile ago, so
                                // waiting for all but the newest `chunks` groups returns at once.  (The host sets
                                // `defer` only when the ring is longer than the distance between two tiles of a CTA:
                                // otherwise the transform that feeds the next tile could be waiting for this very
                                // announcement.)
                                if (pend_pt >= 0) {
                                    if (chunks == 1) tma_store_wait_pending<1>();
                                    else if (chunks == 2) tma_store_wait_pending<2>();
                                    else tma_store_wait_pending<4>();
                                    fence_proxy_async_all();
                                    signal_counter_release(&pp.m_done[pend_pt]);
                                }
                            } else {
                                tma_store_wait_all();
                                fence_proxy_async_all();
                                signal_counter_release(&pp.m_done[pt]);
                            }
                            pend_pt = pt;
                        }
                    }
                }
            }
            }   // chunks
            // accumulator drained: hand the TMEM buffer back to the MMA warp
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if constexpr (CTAS == 2) mbar_arrive_cluster(acc_empty_addr0 + static_cast<uint32_t>(buf) * 8u);
                else mbar_arrive(&acc_empty_bar[buf]);
            }
            buf ^= 1;
            if (buf == 0) acc_phase ^= 1u;
        }
        if (group_tid == 0) {
            tma_store_wait_all();
            if constexpr (PIPE) {
                if (pp.defer && pend_pt >= 0 && *abort_flag == 0) {
                    fence_proxy_async_all();
                    signal_counter_release(&pp.m_done[pend_pt]);
                }
            }
        }
    } else if constexpr (SPLIT) {
        // ------------------------------ second producer: the filter boxes ------------------------------
        // The filters depend on nothing before this launch (see the comment in the first producer), so this thread
        // never waits for the preceding kernel: the first ring-full of boxes goes out at once, the rest as stages
        // are released.
        if (lane == 0) {
            const uint32_t smem_base = smem_u32(smem);
            const uint32_t full0 = smem_u32(&full_bar[0]);
            const uint32_t u_bytes = static_cast<uint32_t>(L::b_bytes(b_rows));
            const uint64_t u_policy = l2_policy_evict_first();
            uint32_t sa = smem_base + a_bytes, fb = full0;
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int i = 0; i < my_count && ok; ++i) {
                int pt, kt, pos;
                decode(tile_of(i), pt, kt, pos);
                const int k0 = kt * prm.n_tile;
                for (int c0 = 0; c0 < prm.C; c0 += GEMM_BLOCK_C) {
                    ok = mbar_wait_bounded(&empty_bar[stage], phase ^ 1u, abort_flag, GEMM_WAIT_LIMIT_NS);
                    if (!ok) { if (*abort_flag == 0) report_timeout(status_word, 11, cta_rank); break; }
                    mbar_arrive_expect_tx_a32(fb, u_bytes);
                    tma_load_5d_hint_a32(sa, &tmU, fb, c0 >> 6, k0 >> 4, pos, u_policy);
                    sa += stage_bytes;
                    fb += 8;
                    if (++stage == stages) { stage = 0; phase ^= 1u; sa = smem_base + a_bytes; fb = full0; }
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if constexpr (PIPE) {
        // ------------------------------ transforms (pipelined mode) ------------------------------
        // The transform warps work as one team through the queue of transform items: one thread takes the next item
        // and waits for what it depends on, then every thread handles one pair of tiles of one channel per round.
        // (Warps that pull items independently of one another were built too: with ten times as many waiting
        // parties polling the same few counters in L2 the whole launch ran 1.5-3x slower.)  Queue order, for
        // j = 0, 1, ...: the activation-transform items of block j, then the output-transform items of block j - lead.
        const int tt = static_cast<int>(threadIdx.x) - GEMM_THREADS;       // 0 .. 319: (channel lane, pair of tiles)
        const unsigned int NB = static_cast<unsigned int>(pp.num_pblocks);
        const unsigned int D = static_cast<unsigned int>(pp.lead) < NB ? static_cast<unsigned int>(pp.lead) : NB;
        const unsigned int n_it = static_cast<unsigned int>(pp.it_items), n_ot = static_cast<unsigned int>(pp.ot_items);
        const unsigned int head = D * n_it, per = n_it + n_ot, body = (NB - D) * per, total = NB * per;
        const long long ring_p = static_cast<long long>(pp.ring) * GEMM_BLOCK_P;
        const Epilogue no_ep{nullptr, 0, nullptr};
        unsigned int iter = 0;
        int pend_kind = -1, pend_pb = 0;      // thread 0: the item just finished, announced after the team barrier
        for (;;) {
            __threadfence();                                   // this thread's stores of the previous item
            named_barrier_sync(3, PIPE_TRANSFORM_THREADS);     // everyone has finished the previous item
            if (tt == 0) {
                if (pend_kind == 0) atomicAdd(&pp.v_ready[pend_pb], 1u);
                else if (pend_kind == 1) atomicAdd(&pp.o_done[pend_pb], 1u);
                const unsigned int idx = atomicAdd(pp.q_head, 1u);
                int kind = -1;
                unsigned int pb = 0, sub = 0;
                if (idx < head) {
                    kind = 0; pb = idx / n_it; sub = idx - pb * n_it;
                } else if (idx - head < body) {
                    const unsigned int r0 = idx - head, jj = r0 / per, r = r0 - jj * per;
                    if (r < n_it) { kind = 0; pb = D + jj; sub = r; }
                    else { kind = 1; pb = jj; sub = r - n_it; }
                } else if (idx < total) {
                    const unsigned int r0 = idx - head - body, jj = r0 / n_ot;
                    kind = 1; pb = NB - D + jj; sub = r0 - jj * n_ot;
                }
                bool ok = true;
                // an activation item overwrites the V slot of block pb - ring: its GEMM tiles must have completed
                if (kind == 0 && pb >= static_cast<unsigned int>(pp.ring))
                    ok = wait_counter(&pp.m_done[pb - pp.ring], pp.m_target, pp.abort_word, GEMM_WAIT_LIMIT_NS);
                // an output item reads M of block pb: all (position, k-tile) tiles of the block must have been stored
                if (kind == 1) ok = wait_counter(&pp.m_done[pb], pp.m_target, pp.abort_word, GEMM_WAIT_LIMIT_NS);
                if (!ok) {
                    if (*reinterpret_cast<volatile int*>(pp.abort_word) == 0) report_timeout(status_word, 14, 0);
                    *reinterpret_cast<volatile int*>(pp.abort_word) = 1;
                    kind = -1;
                }
                pend_kind = kind;
                pend_pb = static_cast<int>(pb);
                item_slots[(iter & 1u) * 2u] = static_cast<unsigned int>(kind + 1) | (sub << 2);
                item_slots[(iter & 1u) * 2u + 1u] = pb;
            }
            named_barrier_sync(4, PIPE_TRANSFORM_THREADS);
            const unsigned int w0 = item_slots[(iter & 1u) * 2u], pb = item_slots[(iter & 1u) * 2u + 1u];
            ++iter;
            const int kind = static_cast<int>(w0 & 3u) - 1;
            const int sub = static_cast<int>(w0 >> 2);
            if (kind < 0) break;
            const long long slot_off = static_cast<long long>(pb % static_cast<unsigned int>(pp.ring)) * GEMM_BLOCK_P;
            const long long p_begin = static_cast<long long>(pb) * GEMM_BLOCK_P;
            const uint32_t pair = static_cast<uint32_t>(tt & 63);        // which two tiles of the block
            if (kind == 0) {
                const int c_end = (sub + 1) * pp.cg < prm.C ? (sub + 1) * pp.cg : prm.C;
                for (int c = sub * pp.cg + (tt >> 6); c < c_end; c += PIPE_TRANSFORM_THREADS / 64)
                    input_unit_f4<1, __half, false, true>(pp.x, pp.V + slot_off, pp.geo, prm.C, p_begin, pp.fd64, ring_p,
                                                          static_cast<uint32_t>(c) * 64u + pair);
            } else {
                const int k_end = (sub + 1) * pp.kg < prm.K ? (sub + 1) * pp.kg : prm.K;
                for (int k = sub * pp.kg + (tt >> 6); k < k_end; k += PIPE_TRANSFORM_THREADS / 64)
                    output_unit_vec<4, 2, false, __half, true>(pp.Mws + slot_off, pp.bias, pp.y, pp.geo, prm.K, p_begin,
                                                               pp.fd64, ring_p, static_cast<uint32_t>(k) * 64u + pair, no_ep);
            }
        }
    }

    __syncwarp();
    __syncthreads();
    if (*abort_flag != 0) {
        if constexpr (PIPE) {
            if (threadIdx.x == 0) *reinterpret_cast<volatile int*>(pp.abort_word) = 1;   // the other CTAs stop waiting
        }
        // give copies and MMAs that may still be in flight a bounded time to land before TMEM and
        // shared memory are released
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if constexpr (CTAS == 2) cluster_sync_all();   // no CTA leaves while its peer may still signal it
    if (warp == 1) {
        tc_fence_after_sync();
        if constexpr (CTAS == 2) tmem_dealloc_pair(tmem_base, TMEM_COLS);
        else tmem_dealloc(tmem_base, TMEM_COLS);
    }
}


// Exercises the bounded wait and the status word without disturbing anything: one thread waits on a barrier
// that nothing ever signals, gives up after `limit_ns`, records the timeout (where = 7) and returns.
__global__ void wait_timeout_selftest_kernel(int* status_word, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&bar, 1);
        fence_barrier_init();
        if (!mbar_wait_bounded(&bar, 0u, &abort_flag, limit_ns)) report_timeout(status_word, 7, 0);
    }
}

}  // namespace sdw
