// Host side of the sdwino C ABI: argument checks, workspace planning, tensor-map
// construction and kernel launches.  See include/sdwino.h for the contract.
#include "../../include/sdwino.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <stdio.h>
#include <stdlib.h>

#include <algorithm>
#include <atomic>
#include <utility>
#include <mutex>
#include <vector>

#include "transforms.cuh"
#include "wino_gemm.cuh"
#include "fused_small_k.cuh"
#include "input_tma.cuh"
#include "output_tma.cuh"

namespace {

using namespace sdw;

__device__ int g_status_word = 0;

std::atomic<unsigned long long> g_launches{0};
std::mutex g_mutex;
// Test / tuning overrides of the GEMM launch shape (0 = choose automatically).  Compute calls may run on several
// host threads at once: the overrides are atomics, and a call reads each of them once.
std::atomic<int> g_force_ctas{0};
std::atomic<int> g_input_staging{1};  // 0 never, 1 where it is faster, 2 wherever possible (sdwino_set_input_staging)
std::atomic<bool> g_disable_fused{false};  // forcing a GEMM shape also forces the GEMM path for few-channel layers
std::atomic<int> g_force_n_tile{0};
// Pipelined single-launch path (see wino_gemm.cuh): 0 never, 1 where it is faster, 2 wherever it is possible (tests);
// ring / lead in blocks of 128 tiles, 0 = chosen by the library.
std::atomic<int> g_pipe_mode{1};
std::atomic<int> g_pipe_ring{0};
std::atomic<int> g_pipe_lead{0};
void* g_workspace = nullptr;
size_t g_workspace_bytes = 0;

// Optional per-kernel timing: when enabled every launch is bracketed by CUDA events on its stream.
// Mode 1 brackets every kernel, mode 2 every convolution call as a whole (KIND_LAYER: one record per call, so that
// the kernels of a call keep their programmatic overlap and the records of a step add up to the step).
enum KernelKind { KIND_FILTER = 0, KIND_INPUT = 1, KIND_GEMM = 2, KIND_OUTPUT = 3, KIND_FUSED = 4, KIND_LAYER = 5, KIND_COUNT = 6 };
struct ProfRecord { int kind; cudaEvent_t beg, end; };
std::atomic<int> g_profile{0};
std::vector<ProfRecord> g_prof_records;   // guarded by g_mutex, like the event pool
std::vector<cudaEvent_t> g_event_pool;

cudaEvent_t prof_event() {
    cudaEvent_t e = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!g_event_pool.empty()) { e = g_event_pool.back(); g_event_pool.pop_back(); return e; }
    }
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    return e;
}
// While the stream is being captured into a CUDA graph the records must be external event nodes,
// otherwise their elapsed time cannot be queried after a replay.
void prof_record(cudaEvent_t e, cudaStream_t st) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusActive)
        cudaEventRecordWithFlags(e, st, cudaEventRecordExternal);
    else
        cudaEventRecord(e, st);
}
struct ProfScope {
    cudaStream_t st; int kind; cudaEvent_t beg = nullptr;
    ProfScope(int k, cudaStream_t s) : st(s), kind(k) {
        if (g_profile.load(std::memory_order_relaxed) == (k == KIND_LAYER ? 2 : 1)) {
            beg = prof_event();
            if (beg) prof_record(beg, st);
        }
    }
    ~ProfScope() {
        if (beg) {
            cudaEvent_t end = prof_event();
            if (end) prof_record(end, st);
            std::lock_guard<std::mutex> lock(g_mutex);
            if (end) g_prof_records.push_back({kind, beg, end});
            else g_event_pool.push_back(beg);
        }
    }
};

constexpr int MAX_DYN_SMEM = 232448;  // 227 KB opt-in limit per CTA on sm_100
// Budget for V and M of one pass over the tile list.  Passes that keep both inside the 126 MB L2 (64 MB) were
// the first design; with the filter stream marked evict-first, one long pass that streams V and M through HBM
// beats many short L2-resident ones, whose kernels are mostly ramp and tail (512->512 at 256x256, F4: 236 us
// with 64 MB passes, 216 us with 128 MB, 202 us in a single pass).  The cap only bounds the memory asked for.
constexpr size_t PASS_BUDGET = 4096ull << 20;
constexpr size_t WS_ALIGN = 1024;
constexpr int STATIC_MAX_DEVICES_HOST = 64;

// SDWINO_ERR_CUDA, with the place and the runtime's last error on stderr when SDWINO_LOG is set
int err_cuda(int line) {
    if (getenv("SDWINO_LOG"))
        fprintf(stderr, "sdwino: SDWINO_ERR_CUDA at sdwino.cu:%d (last CUDA error: %s)\n", line,
                cudaGetErrorString(cudaPeekAtLastError()));
    return SDWINO_ERR_CUDA;
}
inline int round_up(int v, int m) { return (v + m - 1) / m * m; }
inline long long round_up_ll(long long v, long long m) { return (v + m - 1) / m * m; }

struct Plan {
    int a2;            // transform positions
    int Kb, Cb;        // blocks of 16 output channels / 64 input channels of the filter tensor
    int TH, TW;
    long long P;       // tiles in the whole batch
    long long P128;    // P rounded up to the GEMM tile
    size_t per_tile;   // workspace bytes per tile column (V + M)
    int Ho, Wo;        // output image (equal to H, W except for the strided direct convolution)
};

// tile 2 / 4: Winograd; tile 1 with stride >= 1: the direct convolution (a tile is one output pixel)
bool make_plan(int N, int C, int H, int W, int K, int tile, Plan* pl, int stride = 0) {
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0) return false;
    if (tile == 1 && stride == 0) stride = 1;      // tile 1 through the ordinary entries: the direct convolution, stride 1
    if (stride > 0 ? (tile != 1 || stride > 2) : (tile != 2 && tile != 4)) return false;
    const int a = tile + 2;
    pl->a2 = a * a;
    pl->Kb = (K + 15) / 16;
    pl->Cb = (C + 63) / 64;
    pl->Ho = stride > 0 ? (H - 1) / stride + 1 : H;
    pl->Wo = stride > 0 ? (W - 1) / stride + 1 : W;
    pl->TH = stride > 0 ? pl->Ho : (H + tile - 1) / tile;
    pl->TW = stride > 0 ? pl->Wo : (W + tile - 1) / tile;
    pl->P = static_cast<long long>(N) * pl->TH * pl->TW;
    if (pl->P >= (1ll << 31) - GEMM_BLOCK_P) return false;   // tile indices are 32-bit on the device
    pl->P128 = round_up_ll(pl->P, GEMM_BLOCK_P);
    pl->per_tile = static_cast<size_t>(pl->a2) * (static_cast<size_t>(C) + K) * sizeof(__half);
    // element counts must stay far inside int64
    const long double big = 9.0e18L;
    if (static_cast<long double>(N) * C * H * W > big || static_cast<long double>(N) * K * H * W > big) return false;
    if (pl->P128 > (1ll << 40)) return false;
    return true;
}

// Tiles per pass for a workspace of `bytes` (0 = not even one GEMM tile fits).
long long tiles_per_pass(const Plan& pl, size_t bytes) {
    long long fit = static_cast<long long>(bytes / pl.per_tile) / GEMM_BLOCK_P * GEMM_BLOCK_P;
    long long want = static_cast<long long>(PASS_BUDGET / pl.per_tile) / GEMM_BLOCK_P * GEMM_BLOCK_P;
    if (want < 4 * GEMM_BLOCK_P) want = 4 * GEMM_BLOCK_P;
    long long pc = fit < want ? fit : want;
    if (pc > pl.P128) pc = pl.P128;
    return pc;
}

// ---- driver entry point for tensor maps (no link-time dependency on libcuda) ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// cuTensorMapEncodeTiled (fp16, no interleave, 256-byte L2 promotion, no NaN fill).  It is a driver call and wants a
// current context: a host thread that has made no runtime call needing one yet -- a fresh worker thread whose first
// convolution finds everything else cached -- has none and gets CUDA_ERROR_INVALID_CONTEXT.  Then, and only then
// (a thread that is capturing a stream has a context, and cudaFree is not allowed inside a capture), the runtime
// is asked to bind the device's primary context to the thread and the call is repeated.
CUresult encode_tiled(CUtensorMap* m, cuuint32_t rank, const void* base, const cuuint64_t* dims, const cuuint64_t* strides,
                      const cuuint32_t* box, const cuuint32_t* estr, CUtensorMapSwizzle swizzle,
                      CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_FLOAT16) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return CUDA_ERROR_NOT_INITIALIZED;
    CUresult r = fn(m, dtype, rank, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r == CUDA_ERROR_INVALID_CONTEXT) {
        cudaFree(nullptr);
        r = fn(m, dtype, rank, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    return r;
}

// fp16 tensor [d2][d1][d0] (d0 contiguous, row pitch `pitch0` elements, plane pitch `pitch1`
// elements) with a {b0, b1, 1} box, with the 128-byte swizzle or none.  Encoding costs about a
// microsecond of host time, so the last few maps are kept (a map depends only on these arguments).
struct MapKey {
    const void* base; uint64_t d0, d1, d2, pitch0, pitch1; uint32_t b0, b1; bool sw;
    bool operator==(const MapKey& o) const {
        return base == o.base && d0 == o.d0 && d1 == o.d1 && d2 == o.d2 && pitch0 == o.pitch0 && pitch1 == o.pitch1 &&
               b0 == o.b0 && b1 == o.b1 && sw == o.sw;
    }
};
struct MapSlot { MapKey key; CUtensorMap map; bool used = false; };
constexpr int MAP_CACHE_SLOTS = 256;
MapSlot g_map_cache[MAP_CACHE_SLOTS];
std::mutex g_map_mutex;

bool encode_map_uncached(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t pitch0,
                         uint64_t pitch1, uint32_t b0, uint32_t b1, bool swizzle128);

bool encode_map(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t pitch0,
                uint64_t pitch1, uint32_t b0, uint32_t b1, bool swizzle128) {
    const MapKey key{base, d0, d1, d2, pitch0, pitch1, b0, b1, swizzle128};
    uint64_t h = reinterpret_cast<uintptr_t>(base) >> 8;
    h = h * 1000003u ^ d0 * 31u ^ d1 * 131u ^ pitch0 * 7u ^ (static_cast<uint64_t>(b1) << 20) ^ (b0 << 3) ^ swizzle128;
    MapSlot& slot = g_map_cache[h % MAP_CACHE_SLOTS];
    std::lock_guard<std::mutex> lock(g_map_mutex);
    if (slot.used && slot.key == key) { *m = slot.map; return true; }
    if (!encode_map_uncached(m, base, d0, d1, d2, pitch0, pitch1, b0, b1, swizzle128)) return false;
    slot.key = key;
    slot.map = *m;
    slot.used = true;
    return true;
}

bool encode_map_uncached(CUtensorMap* m, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t pitch0,
                         uint64_t pitch1, uint32_t b0, uint32_t b1, bool swizzle128) {
    cuuint64_t dims[3] = {d0, d1, d2};
    cuuint64_t strides[2] = {pitch0 * sizeof(__half), pitch1 * sizeof(__half)};
    cuuint32_t box[3] = {b0, b1, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = encode_tiled(m, 3, base, dims, strides, box, estr,
                                    swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE);
    if (r != CUDA_SUCCESS && getenv("SDWINO_LOG"))
        fprintf(stderr, "sdwino: cuTensorMapEncodeTiled failed (%d): base %p dims %llu %llu %llu pitch %llu %llu box %u %u sw %d\n",
                static_cast<int>(r), base, (unsigned long long)d0, (unsigned long long)d1, (unsigned long long)d2,
                (unsigned long long)pitch0, (unsigned long long)pitch1, b0, b1, swizzle128 ? 1 : 0);
    return r == CUDA_SUCCESS;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// The blocked filter tensor U[pos][Cb][Kb][16][64] as a 5-D map (dimension order {c, k, c-block, k-block, pos}) whose box is `kblocks` blocks of 16 rows
// of `posbox` consecutive transform positions (`krows` < 16: only the first rows of a block).
bool encode_filter_map(CUtensorMap* m, const void* base, uint64_t Cb, uint64_t Kb, uint64_t npos, uint32_t kblocks,
                       uint32_t posbox = 1, uint32_t krows = 16) {
    const MapKey key{base, Cb, Kb, npos, ~0ull, ~0ull, kblocks | (posbox << 16) | (krows << 24), 5, true};
    const uint64_t h = (reinterpret_cast<uintptr_t>(base) >> 8) * 1000003u ^ Cb * 31u ^ Kb * 131u ^ (kblocks << 7) ^
                       (posbox << 13) ^ (krows << 20) ^ 5u;
    MapSlot& slot = g_map_cache[h % MAP_CACHE_SLOTS];
    std::lock_guard<std::mutex> lock(g_map_mutex);
    if (slot.used && slot.key == key) { *m = slot.map; return true; }
    cuuint64_t dims[5] = {64, 16, Cb, Kb, npos};
    cuuint64_t strides[4] = {128, 2048 * Kb, 2048, Kb * Cb * 2048};   // memory order [pos][Cb][Kb][16][64]
    cuuint32_t box[5] = {64, krows, 1, kblocks, posbox};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    if (encode_tiled(m, 5, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_128B) != CUDA_SUCCESS) {
        if (getenv("SDWINO_LOG"))
            fprintf(stderr, "sdwino: cuTensorMapEncodeTiled failed for the filters: base %p Cb %llu Kb %llu positions %llu box %u %u %u\n",
                    base, (unsigned long long)Cb, (unsigned long long)Kb, (unsigned long long)npos, krows, kblocks, posbox);
        return false;
    }
    slot.key = key;
    slot.map = *m;
    slot.used = true;
    return true;
}

// The 8-bit blocked filter tensor (one byte per element, same blocking): box of `kblocks` blocks of 16 rows of 64 bytes,
// not swizzled (the bytes are expanded to fp16 by the kernel, which places them in the swizzled operand layout itself).
bool encode_filter_map_q8(CUtensorMap* m, const void* base, uint64_t Cb, uint64_t Kb, uint64_t npos, uint32_t kblocks) {
    const MapKey key{base, Cb, Kb, npos, ~2ull, ~2ull, kblocks, 8, false};
    const uint64_t h = (reinterpret_cast<uintptr_t>(base) >> 8) * 1000003u ^ Cb * 31u ^ Kb * 131u ^ (kblocks << 7) ^ 8u;
    MapSlot& slot = g_map_cache[h % MAP_CACHE_SLOTS];
    std::lock_guard<std::mutex> lock(g_map_mutex);
    if (slot.used && slot.key == key) { *m = slot.map; return true; }
    cuuint64_t dims[5] = {64, 16, Cb, Kb, npos};
    cuuint64_t strides[4] = {64, 1024 * Kb, 1024, Kb * Cb * 1024};   // memory order [pos][Cb][Kb][16][64], bytes
    cuuint32_t box[5] = {64, 16, 1, kblocks, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    if (encode_tiled(m, 5, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_DATA_TYPE_UINT8) !=
        CUDA_SUCCESS)
        return false;
    slot.key = key;
    slot.map = *m;
    slot.used = true;
    return true;
}

// Per-device facts, looked up once per device (a process may drive several GPUs: everything that belongs to a
// device -- the SM count, the address of the status word, the shared-memory limit of a kernel -- is kept per device).
int current_device() {
    int dev = -1;
    return (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < STATIC_MAX_DEVICES_HOST) ? dev : -1;
}

int sm_count() {
    static std::atomic<int> n[STATIC_MAX_DEVICES_HOST];
    const int dev = current_device();
    if (dev < 0) return 0;
    int v = n[dev].load(std::memory_order_relaxed);
    if (v == 0) {
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) v = 0;
        n[dev].store(v, std::memory_order_relaxed);
    }
    return v;
}

// Device address of the status word on the current device.
int* status_word_ptr() {
    static std::atomic<int*> ptr[STATIC_MAX_DEVICES_HOST];
    const int dev = current_device();
    if (dev < 0) return nullptr;
    int* v = ptr[dev].load(std::memory_order_relaxed);
    if (!v) {
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&v), g_status_word) != cudaSuccess) v = nullptr;
        ptr[dev].store(v, std::memory_order_relaxed);
    }
    return v;
}

// Raises the dynamic shared-memory limit of a kernel, once per kernel and device.
bool ensure_dyn_smem(const void* kernel, int bytes) {
    static std::mutex mutex;
    static std::vector<std::pair<const void*, int>> done;
    const int dev = current_device();
    if (dev < 0) return false;
    std::lock_guard<std::mutex> lock(mutex);
    for (const auto& e : done)
        if (e.first == kernel && e.second == dev) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    done.emplace_back(kernel, dev);
    return true;
}
// 8-bit filter buffer: header, the bytes, the scales (each part padded to 1 KiB)
inline size_t q8_bytes_part(int a2, int Kb, int Cb) {
    return (static_cast<size_t>(a2) * Kb * Cb * 1024 + WS_ALIGN - 1) / WS_ALIGN * WS_ALIGN;
}
inline size_t q8_scale_part(int a2, int Kb) {
    return (static_cast<size_t>(a2) * Kb * 16 * sizeof(float) + WS_ALIGN - 1) / WS_ALIGN * WS_ALIGN;
}
inline const uint32_t* wt_header_of(const void* wT) { return static_cast<const uint32_t*>(wT); }
inline const void* wt_filters_of(const void* wT) { return static_cast<const uint8_t*>(wT) + WT_HEADER_BYTES; }

// x as a 3-D tensor [N * C][H][W] with a box of bw x bh pixels of cpb channel images (no swizzle, zeros outside).
bool encode_image_map(CUtensorMap* m, const void* base, uint64_t W, uint64_t H, uint64_t NC, uint32_t bw, uint32_t bh,
                      uint32_t cpb) {
    const MapKey key{base, W, H, NC, ~1ull, cpb, bw, bh, false};
    const uint64_t h = (reinterpret_cast<uintptr_t>(base) >> 8) * 1000003u ^ W * 31u ^ H * 131u ^ NC * 7u ^ (bw << 9) ^
                       (bh << 17) ^ (cpb << 25) ^ 3u;
    MapSlot& slot = g_map_cache[h % MAP_CACHE_SLOTS];
    std::lock_guard<std::mutex> lock(g_map_mutex);
    if (slot.used && slot.key == key) { *m = slot.map; return true; }
    cuuint64_t dims[3] = {W, H, NC};
    cuuint64_t strides[2] = {W * sizeof(__half), H * W * sizeof(__half)};
    cuuint32_t box[3] = {bw, bh, cpb};
    cuuint32_t estr[3] = {1, 1, 1};
    if (encode_tiled(m, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_SWIZZLE_NONE) != CUDA_SUCCESS) return false;
    slot.key = key;
    slot.map = *m;
    slot.used = true;
    return true;
}

// Kernels are launched with programmatic stream serialization (see pdl_wait in ptx.cuh); cluster_x: 0 for
// the transform kernels, 1 or 2 CTAs per cluster for the GEMM.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster_x,
                       Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    // Cluster launches do not get the attribute: CTA-pair GEMMs launched with it stalled the stream
    // intermittently (two-pass convolutions with few output channels), single-CTA launches never did.
    if (cluster_x <= 1) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (cluster_x > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster_x;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
    if (e != cudaSuccess && getenv("SDWINO_LOG"))
        fprintf(stderr, "sdwino: kernel launch failed: %s (grid %u x %u, block %u, %zu bytes of dynamic shared memory)\n",
                cudaGetErrorString(e), grid.x, grid.y, block.x, smem);
    return e;
}

// A cooperative launch (all CTAs resident at once: the pipelined kernel's CTAs wait on one another), ordered after
// everything before it in the stream.
template <typename... KArgs, typename... Args>
cudaError_t launch_coop(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
    if (e != cudaSuccess && getenv("SDWINO_LOG"))
        fprintf(stderr, "sdwino: cooperative launch failed: %s (grid %u, block %u, %zu bytes of dynamic shared memory)\n",
                cudaGetErrorString(e), grid.x, block.x, smem);
    return e;
}

// A grid of x by `rows` blocks: grid.y holds at most 65535 rows, the rest continue along grid.z (the kernels
// number their rows blockIdx.z * gridDim.y + blockIdx.y and skip those past the end).
inline dim3 grid_rows(unsigned x, long long rows) {
    if (rows <= 65535) return dim3(x, static_cast<unsigned>(rows), 1);
    return dim3(x, 65535, static_cast<unsigned>((rows + 65534) / 65535));
}

template <int M, typename WT>
int launch_filter(const WT* w, void* wT, int K, int C, int Kb, int Cb, cudaStream_t st) {
    const dim3 grid = grid_rows((Cb * 32 + 127) / 128, static_cast<long long>(Kb) * 16);   // a thread transforms two neighbouring input channels
    ProfScope prof(KIND_FILTER, st);
    uint32_t* header = static_cast<uint32_t*>(wT);
    __half* U = reinterpret_cast<__half*>(static_cast<uint8_t*>(wT) + WT_HEADER_BYTES);
    const cudaError_t e = launch_pdl(filter_transform_kernel<M, WT>, grid, dim3(128), 0, st, 0, w, header, U, K, C, Kb, Cb);
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}

template <int M, typename XT>
int launch_input(const XT* x, __half* V, const TileGeom& geo, int C, long long p_begin, int p_count,
                 long long Pstride, cudaStream_t st, const float* amax = nullptr) {
    ProfScope prof(KIND_INPUT, st);
    constexpr int TPT = 8 / M;
    cudaError_t e;
    const long long units = static_cast<long long>(p_count / TPT) * C;   // one thread each
    if constexpr (M == 1) {
        const dim3 grid = grid_rows((p_count + 127) / 128, C);
        e = launch_pdl(input_transform_kernel<M, XT>, grid, dim3(128), 0, st, 0, x, V, geo, C, p_begin, p_count, Pstride, amax);
    } else if (geo.W % 8 == 0 && aligned(x, 16) && units < (1ll << 31) - 128) {
        if constexpr (M == 4) {
            constexpr int CH = 1;   // channels per thread
            const long long threads = static_cast<long long>(p_count / TPT) * ((C + CH - 1) / CH);
            dim3 grid(static_cast<unsigned>((threads + 127) / 128));
            e = launch_pdl(input_transform_f4_kernel<CH, XT>, grid, dim3(128), 0, st, 0, x, V, geo, C, p_begin,
                           make_fastdiv(static_cast<uint32_t>(p_count / TPT)), Pstride, amax);
        } else {
            dim3 grid(static_cast<unsigned>((units + 127) / 128));
            e = launch_pdl(input_transform_vec_kernel<M, TPT, XT>, grid, dim3(128), 0, st, 0, x, V, geo, C, p_begin,
                           make_fastdiv(static_cast<uint32_t>(p_count / TPT)), Pstride, amax);
        }
    } else {
        const dim3 grid = grid_rows((p_count + 127) / 128, C);
        e = launch_pdl(input_transform_kernel<M, XT>, grid, dim3(128), 0, st, 0, x, V, geo, C, p_begin, p_count, Pstride, amax);
    }
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}


// The TMA-staged F(4x4) activation transform covers a layer done in one pass whose rows TMA can address.
bool input_tma_possible(const TileGeom& geo, int N, int C, const void* x) {
    return geo.W % 8 == 0 && aligned(x, 16) && static_cast<long long>(N) * C < (1ll << 31) && geo.TH < (1 << 20) &&
           static_cast<long long>(N) * geo.TH < (1ll << 31);
}

bool use_input_tma(const TileGeom& geo, int N, int C, const void* x, long long p_begin, long long p_count) {
    // a pass of whole tile rows (the last one may end with the layer)
    const bool possible = input_tma_possible(geo, N, C, x) && p_begin % geo.TW == 0 &&
                          (p_count % geo.TW == 0 || p_begin + p_count >= geo.P);
    if (!possible || g_input_staging == 0) return false;
    // Faster where a block row is a whole number of 32-byte sectors of V (W % 64 == 0: 15.8 against 17.0 us on
    // 960->320 at 64x64, 45.6 against 60.5 us on 512->512 at 256x256).  Image widths of 32 (8 tiles per row,
    // four channel images per step) come out even, widths of 24, 48 and 96 up to 2x slower: their rows of 6, 12
    // and 24 tiles leave runs of V that start and end inside sectors, where the register-only kernel, whose
    // threads follow the tile index, always stores whole 128-byte lines.
    return g_input_staging == 2 || geo.TW % 16 == 0;
}

int launch_input_tma(const __half* x, __half* V, const TileGeom& geo, int N, int C, long long p_begin, long long p_count,
                     long long Pstride, cudaStream_t st) {
    ProfScope prof(KIND_INPUT, st);
    const int sms = sm_count();
    int* status = status_word_ptr();
    if (sms <= 0 || !status) return err_cuda(__LINE__);
    InTmaParams q;
    q.C = C; q.TH = geo.TH; q.TW = geo.TW; q.Pstride = Pstride;
    q.p_begin = p_begin;
    const long long p_end = std::min(p_begin + p_count, geo.P);   // one past the last tile of the pass
    q.g_begin = p_begin / geo.TW;
    q.g_end = p_end / geo.TW;                                      // P = N * TH * TW: whole rows
    q.tail_begin = p_end - p_begin;
    q.tail_end = p_count;                                          // a multiple of 128
    // A block of up to 256 tiles (128 threads).  Blocks span the full width of the image when it has at most 60
    // tiles per row, otherwise at least 32 tiles: the tiles of a block row (of the whole block, at full width) are
    // then consecutive in V, and a warp stores runs of at least 64 bytes (narrower blocks measured 2-3x slower:
    // 8-byte pieces per store).  Among those, the shape that leaves the fewest threads without a tile -- over the
    // tiles that hang over the right and bottom edges and the threads that no channel image fills --, and among
    // equals the one that fetches the smallest halo.
    int best_half = 1, best_trb = 1;
    double best_score = -1e30;
    const int half_full = geo.TW / 2;   // W % 8 == 0: TW is even
    // two boxes side by side where a block row can then be 64 tiles = one 128-byte line of V per warp store
    // (256->256 at 1024x1024: 365 -> 340 us)
    q.nb = geo.TW % 64 == 0 ? 2 : 1;
    for (int half = (half_full <= 30 ? half_full : 16); half <= (half_full <= 30 ? half_full : 30); ++half) {
        const int sbc = (geo.TW + 2 * half * q.nb - 1) / (2 * half * q.nb);
        for (int trb = 1; trb <= 32 && half * q.nb * trb <= 128; ++trb) {
            const int sbr = (geo.TH + trb - 1) / trb;
            const int cpb = std::min(16, 128 / (half * q.nb * trb));
            double used = static_cast<double>(geo.TW) * geo.TH / (static_cast<double>(sbc) * 2 * half * q.nb * sbr * trb) *
                          (half * q.nb * trb * cpb / 128.0);
            const int run = half_full <= 30 ? std::min(trb, geo.TH) * geo.TW : 2 * half;   // consecutive tiles in V
            if (run < 32) used *= run / 32.0;
            const double halo = (8.0 * half + 16) * (4.0 * trb + 2) / (32.0 * half * trb);
            const double score = used - 0.02 * halo;
            if (score > best_score) { best_score = score; best_half = half; best_trb = trb; }
        }
    }
    const int tcb = 2 * best_half;
    q.tcb_half = best_half;
    q.trb = best_trb;
    q.cpb = std::min(16, 128 / (best_half * q.nb * best_trb));
    q.bw = 4 * tcb + 16;
    q.bh = 4 * q.trb + 2;
    q.sb_c = (geo.TW + tcb * q.nb - 1) / (tcb * q.nb);
    q.sb_r = (geo.TH + q.trb - 1) / q.trb;
    q.box_bytes = (q.bw * q.bh * q.cpb * 2 + 127) / 128 * 128;
    q.stage_bytes = q.nb * q.box_bytes;
    {
        const long long g_last = q.g_end - 1;
        q.tail_block = static_cast<int>((g_last / geo.TH) * q.sb_c * q.sb_r + ((g_last % geo.TH) / q.trb) * q.sb_c);
    }
    const long long blocks = static_cast<long long>(N) * q.sb_c * q.sb_r;
    const long long csteps = (C + q.cpb - 1) / q.cpb;
    // Steps per CTA (at most 16): five CTAs are resident per SM and an SM needs about four of them to keep its
    // issue slots busy; the time follows the SM with the most CTA-steps (one more step per CTA for the fill).
    long long steps = 1;
    double best_cost = 1e300;
    for (long long cand = 1; cand <= 16 && cand <= csteps; ++cand) {
        const long long ctas = blocks * ((csteps + cand - 1) / cand);
        const long long per_sm = (ctas + sms - 1) / sms;
        const double cost = per_sm <= 5 ? per_sm * (cand + 1.0) * std::max(1.0, 4.0 / per_sm)
                                        : static_cast<double>((ctas + 5ll * sms - 1) / (5ll * sms)) * 5.0 * (cand + 1.0);
        if (cost <= best_cost) { best_cost = cost; steps = cand; }
    }
    q.steps = static_cast<int>(steps);
    const long long grid_y = (csteps + steps - 1) / steps;
    if (blocks >= (1ll << 31) || grid_y > 65535) return SDWINO_ERR_UNSUPPORTED;
    CUtensorMap tmX;
    if (!encode_image_map(&tmX, x, geo.W, geo.H, static_cast<uint64_t>(N) * C, q.bw, q.bh, q.cpb)) return err_cuda(__LINE__);
    const size_t smem = static_cast<size_t>(IN_TMA_STAGES) * q.stage_bytes + 128;
    if (smem > IN_TMA_STAGES * 32 * 1024 + 128 ||
        !ensure_dyn_smem(reinterpret_cast<const void*>(input_transform_f4_tma_kernel), IN_TMA_STAGES * 32 * 1024 + 128))
        return err_cuda(__LINE__);
    dim3 grid(static_cast<unsigned>(blocks), static_cast<unsigned>(grid_y));
    const cudaError_t e = launch_pdl(input_transform_f4_tma_kernel, grid, dim3(IN_TMA_THREADS), smem, st, 0, tmX, V, q,
                                     status);
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}

// The TMA-staged F(4x4) output transform: see output_tma.cuh.
bool use_output_tma(const TileGeom& geo, int K, const void* y, const Epilogue& ep, int p_count) {
    const bool possible = geo.W % 8 == 0 && aligned(y, 16) && aligned(ep.residual, 16) && K <= 65535 * 16;
    if (!possible || g_input_staging == 0) return false;
    // 7-13 % faster on layers of thousands of tiles (256->256 at 512x512: 73.5 -> 65.9 us), even at 512, a few
    // percent slower on the 128-tile passes of the 32x32 layers
    return g_input_staging == 2 || p_count >= 512;
}

template <typename YT>
int launch_output_tma(const __half* Mws, const YT* bias, YT* y, const TileGeom& geo, int K, long long p_begin,
                      int p_count, long long Pstride, const WtCheck& chk, const Epilogue& ep, cudaStream_t st) {
    ProfScope prof(KIND_OUTPUT, st);
    const int sms = sm_count();
    int* status = status_word_ptr();
    if (sms <= 0 || !status) return err_cuda(__LINE__);
    CUtensorMap tmM;
    if (!encode_image_map(&tmM, Mws, static_cast<uint64_t>(Pstride), static_cast<uint64_t>(K), 36, OUT_TMA_TILES, 1, 36))
        return err_cuda(__LINE__);
    const long long blocks = (p_count + OUT_TMA_TILES - 1) / OUT_TMA_TILES;
    // channels per CTA (at most 16): three CTAs are resident per SM; the time follows the SM with the most
    // CTA-steps (one more step per CTA for the fill)
    long long steps = 1;
    double best_cost = 1e300;
    for (long long cand = 1; cand <= 16 && cand <= K; ++cand) {
        const long long ctas = blocks * ((K + cand - 1) / cand);
        const long long per_sm = (ctas + sms - 1) / sms;
        const double cost = per_sm <= 3 ? per_sm * (cand + 1.0) * std::max(1.0, 3.0 / per_sm)
                                        : static_cast<double>((ctas + 3ll * sms - 1) / (3ll * sms)) * 3.0 * (cand + 1.0);
        if (cost <= best_cost) { best_cost = cost; steps = cand; }
    }
    if ((K + steps - 1) / steps > 65535) steps = (K + 65534) / 65535;   // grid limit; K <= 65535 * 16 was checked
    const size_t smem = static_cast<size_t>(OUT_TMA_STAGES) * OUT_TMA_STAGE_BYTES + 128;
    if (blocks >= (1ll << 31) ||
        !ensure_dyn_smem(reinterpret_cast<const void*>(output_transform_f4_tma_kernel<false, YT>), static_cast<int>(smem)))
        return err_cuda(__LINE__);
    if (!ensure_dyn_smem(reinterpret_cast<const void*>(output_transform_f4_tma_kernel<true, YT>), static_cast<int>(smem)))
        return err_cuda(__LINE__);
    dim3 grid(static_cast<unsigned>(blocks), static_cast<unsigned>((K + steps - 1) / steps));
    cudaError_t e;
    if (ep.residual == nullptr && ep.act == 0) {
        e = launch_pdl(output_transform_f4_tma_kernel<false, YT>, grid, dim3(OUT_TMA_THREADS), smem, st, 0, tmM, bias, y, geo, K,
                       p_begin, static_cast<int>(steps), chk, ep, status);
    } else {
        e = launch_pdl(output_transform_f4_tma_kernel<true, YT>, grid, dim3(OUT_TMA_THREADS), smem, st, 0, tmM, bias, y, geo, K,
                       p_begin, static_cast<int>(steps), chk, ep, status);
    }
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}

template <int M, typename YT>
int launch_output(const __half* Mws, const YT* bias, YT* y, const TileGeom& geo, int K,
                  long long p_begin, int p_count, long long Pstride, const WtCheck& chk, const Epilogue& ep,
                  cudaStream_t st) {
    ProfScope prof(KIND_OUTPUT, st);
    constexpr int TPT = 8 / M;
    cudaError_t e;
    const long long units = static_cast<long long>(p_count / TPT) * K;   // one thread each
    if constexpr (M == 1) {
        const dim3 grid = grid_rows((p_count + 127) / 128, K);
        e = launch_pdl(output_transform_kernel<M, YT>, grid, dim3(128), 0, st, 0, Mws, bias, y, geo, K, p_begin, p_count,
                       Pstride, chk, ep);
    } else if (geo.W % 8 == 0 && aligned(y, 16) && aligned(ep.residual, 16) && units < (1ll << 31) - 128) {
        dim3 grid(static_cast<unsigned>((units + 127) / 128));
        if (ep.residual == nullptr && ep.act == 0) {
            e = launch_pdl(output_transform_vec_kernel<M, TPT, false, YT>, grid, dim3(128), 0, st, 0, Mws, bias, y, geo, K,
                           p_begin, make_fastdiv(static_cast<uint32_t>(p_count / TPT)), Pstride, chk, ep);
        } else {
            e = launch_pdl(output_transform_vec_kernel<M, TPT, true, YT>, grid, dim3(128), 0, st, 0, Mws, bias, y, geo, K,
                           p_begin, make_fastdiv(static_cast<uint32_t>(p_count / TPT)), Pstride, chk, ep);
        }
    } else {
        const dim3 grid = grid_rows((p_count + 127) / 128, K);
        e = launch_pdl(output_transform_kernel<M, YT>, grid, dim3(128), 0, st, 0, Mws, bias, y, geo, K, p_begin, p_count,
                       Pstride, chk, ep);
    }
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}

// Layers with at most 8 (tile 2) or 4 (tile 4) input channels run as one fused kernel without a workspace.
bool use_fused_small_c(int C, int tile) { return tile == 2 ? C <= 8 : (tile == 4 && C <= 4); }

template <int M, int CP>
int launch_fused_small_c(const __half* x, const void* wT, const __half* bias, __half* y, const TileGeom& geo, int C,
                         int K, int Kb, int Cb, cudaStream_t st) {
    int* status = status_word_ptr();
    if (!status) return err_cuda(__LINE__);
    const dim3 grid = grid_rows(static_cast<unsigned>((geo.P + 127) / 128), (K + FUSED_KC - 1) / FUSED_KC);
    ProfScope prof(KIND_FUSED, st);
    const cudaError_t e = launch_pdl(fused_small_c_kernel<M, CP>, grid, dim3(128), 0, st, 0, x, wt_header_of(wT),
                                     static_cast<const __half*>(wt_filters_of(wT)), bias, y, geo, C, K, Kb, Cb, status);
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}

// Layers with at most 8 output channels run F(2x2,3x3) as one fused tensor-core kernel (no workspace traffic):
// see fused_small_k.cuh.  It needs the vector loads of the input transform (W % 8 == 0, aligned x) and
// 4-byte output stores.
// A CTA takes 128 tiles and all input channels, so the kernel only pays off when there are enough blocks
// of tiles to occupy the SMs (measured: 64 blocks 32 us against 48 us unfused; 16 blocks 32 us against 15 us).
constexpr long long FK_MIN_P_TILES = 48;
std::atomic<long long> g_fk_min_p_tiles{FK_MIN_P_TILES};
bool use_fused_small_k(int K, int W, int tile, long long p_tiles, const void* x, const void* y) {
    return tile == 2 && K <= FK_KMAX && p_tiles >= g_fk_min_p_tiles && (W % 8) == 0 && aligned(x, 16) && aligned(y, 4);
}

template <typename T>
int launch_fused_small_k(const T* x, const void* wT, const T* bias, T* y, const Plan& pl, int C, int H,
                         int W, int K, cudaStream_t st) {
    const int sms = sm_count();
    if (sms <= 0) return err_cuda(__LINE__);
    int* status = status_word_ptr();
    if (!status || !ensure_dyn_smem(reinterpret_cast<const void*>(fused_small_k_kernel<T>), FK_DYN_SMEM)) return err_cuda(__LINE__);
    CUtensorMap tmU;
    if (!encode_filter_map(&tmU, wt_filters_of(wT), pl.Cb, pl.Kb, pl.a2, 1, 16, FK_KMAX)) return err_cuda(__LINE__);
    FusedKParams prm;
    prm.wt_header = wt_header_of(wT);
    prm.geo = make_geom(H, W, pl.TH, pl.TW, pl.P);
    prm.C = C;
    prm.K = K;
    prm.num_stages = (C + FK_CSTEP - 1) / FK_CSTEP;
    prm.num_cblocks = static_cast<int>(pl.Cb);
    prm.num_p_tiles = static_cast<int>(pl.P128 / 128);
    const int grid_x = prm.num_p_tiles < sms ? prm.num_p_tiles : sms;
    ProfScope prof(KIND_FUSED, st);
    const cudaError_t e = launch_pdl(fused_small_k_kernel<T>, dim3(grid_x, (K + FK_KMAX - 1) / FK_KMAX), dim3(FK_THREADS),
                                     static_cast<size_t>(FK_DYN_SMEM), st, 1, tmU, x, bias, y, prm, status);
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}

// F(2x2,3x3) layers with at most 8 input channels: one warp-MMA kernel (see fused_small_c_mma_kernel).
template <typename T>
int launch_fused_small_c_mma(const T* x, const void* wT, const T* bias, T* y, const TileGeom& geo, int C,
                             int K, int Kb, cudaStream_t st) {
    const int sms = sm_count();
    int* status = status_word_ptr();
    if (sms <= 0 || !status) return err_cuda(__LINE__);
    const long long groups = (geo.P + 7) / 8;
    const long long blocks_x = (groups + 3) / 4;
    // The kernel is a latency chain per warp (load, transform, then per block of output channels MMAs, output
    // transform, store): it runs best with 12-14 warps per SM.  Fewer output-channel blocks per CTA shorten the
    // chain but repeat the input transform and the filter staging; more than 3.5 CTAs per SM measured slower
    // again (4->320 at 64x64, batch 2: 10.2 / 9.0 / 7.6 / 8.9 / 11.7 us with 1 / 2 / 3 / 4 / 7 blocks per CTA).
    int kb_per_block = Kb;
    for (int cand = 1; cand <= Kb; ++cand) {
        if (blocks_x * ((Kb + cand - 1) / cand) * 2 <= static_cast<long long>(sms) * 7) { kb_per_block = cand; break; }
    }
    dim3 grid(static_cast<unsigned>(blocks_x), static_cast<unsigned>((Kb + kb_per_block - 1) / kb_per_block));
    ProfScope prof(KIND_FUSED, st);
    const cudaError_t e = launch_pdl(fused_small_c_mma_kernel<T>, grid, dim3(128), 0, st, 0, x, wt_header_of(wT),
                                     static_cast<const __half*>(wt_filters_of(wT)), bias, y, geo, C, K, Kb, kb_per_block,
                                     status);
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}

// Shape of the GEMM launch: CTA pairs or single CTAs, and the output channels per tile (UMMA N, a
// multiple of 16 up to 256).  The candidate with the smallest modelled time wins: a tile costs its
// pipeline stages, each limited by the tensor pipe (2 n cycles per stage) or by the bytes the CTA must
// fetch from L2 per stage (about 40 bytes per cycle per SM were measured), plus an epilogue that is
// hidden unless the tile is short; tiles run in waves over the SMs.
//
// A CTA pair fetches half of the filter rows per CTA.  Measured over the layers of all workloads it is 4-10 % faster
// for the layer where the mainloop dominates (C >= 512, several waves of 256-channel tiles), and slower where
// tiles are short (its epilogue hand-off crosses two CTAs), where an odd number of 128-tile blocks leaves half a
// pair idle, and for short launches (it runs without programmatic dependent launch, see launch_gemm_shape).  The
// constants below reproduce that: 35 bytes per cycle per CTA of a pair (on the scale where a single CTA gets 40),
// epilogue x 1.35 and a fixed charge for the lost overlap.
struct GemmShape { int ctas; int n_tile; int dual; };   // dual: two blocks of 128 tiles per CTA tile (single CTAs)
GemmShape choose_gemm_shape(int K, int C, long long p_tiles128, int a2, int sms, int force_ctas) {
    const long long cblocks = (C + GEMM_BLOCK_C - 1) / GEMM_BLOCK_C;
    GemmShape best{1, 16, 0};
    double best_cost = 1e300;
    // a pair needs two blocks of 128 tiles; with fewer than 8 stages per tile it measured 4-35 % slower
    const int max_ctas = p_tiles128 >= 2 && (cblocks >= 8 || force_ctas == 2) ? 2 : 1;
    for (int ctas = 1; ctas <= max_ctas; ++ctas) {
        if (force_ctas != 0 && ctas != (force_ctas < max_ctas ? force_ctas : max_ctas)) continue;
        const long long p_tiles = (p_tiles128 + ctas - 1) / ctas;
        const long long workers = sms / ctas;
        const int step = 16 * ctas;   // each CTA of a pair loads whole 16-row blocks
        for (int n = step; n <= GEMM_MAX_N; n += step) {
            const long long ktiles = (K + n - 1) / n;
            if (n > step && (ktiles == (K + n - step - 1) / (n - step))) continue;  // a smaller n needs as many tiles
            const long long tiles = ktiles * p_tiles * a2;
            const long long waves = (tiles + workers - 1) / workers;
            // with one or two tiles per pair the fixed cost of a pair is not paid back (measured 9-12 % slower)
            if (ctas == 2 && force_ctas != 2 && waves < 3) continue;
            const double mma = 2.0 * n;
            const double load = ctas == 1 ? (GemmSmemLayout::A_BYTES + 128.0 * n) / 40.0
                                          : (GemmSmemLayout::A_BYTES + 64.0 * n) / 35.0;
            const double main = cblocks * (mma > load ? mma : load);
            const double epi = (300.0 + 14.0 * n) * (ctas == 2 ? 1.35 : 1.0);
            const double per_tile = (main > epi ? main : epi) + (ctas == 2 ? 400.0 : 200.0);
            const double fixed = ctas == 2 ? 7000.0 : 0.0;
            const double cost = waves * per_tile + epi + fixed;
            if (cost < best_cost) { best_cost = cost; best = GemmShape{ctas, n, 0}; }
        }
    }
    // Single CTAs with two blocks of 128 tiles per CTA tile (see wino_gemm.cuh): the filter box is fetched once per
    // 256 tiles and there are half as many CTA tiles, but the accumulators are not double-buffered across tiles, so
    // the epilogues of a tile are added to its mainloop.  n_tile up to 192 leaves room for three stages.
    // Taken for layers of 2 to 15 blocks of tiles (larger ones have the filter-resident mode and CTA pairs).
    if (force_ctas == 0 && p_tiles128 >= 2 && p_tiles128 < 16) {
        const long long p_tiles = (p_tiles128 + 1) / 2;
        for (int n = 16; n <= 192; n += 16) {
            const long long ktiles = (K + n - 1) / n;
            if (n > 16 && (ktiles == (K + n - 17) / (n - 16))) continue;
            const long long tiles = ktiles * p_tiles * a2;
            const long long waves = (tiles + sms - 1) / sms;
            const double mma = 4.0 * n;
            const double load = (2.0 * GemmSmemLayout::A_BYTES + 128.0 * n) / 40.0;
            const double main = cblocks * (mma > load ? mma : load);
            const double epi = 300.0 + 14.0 * n;
            const double cost = 1.08 * waves * (main + 2.0 * epi + 200.0);   // measured gains are 5-10 %, not the modelled 20
            if (cost < best_cost) { best_cost = cost; best = GemmShape{1, n, 1}; }
        }
    }
    return best;
}

template <int CTAS, bool RES, bool DUAL = false, bool U8 = false, bool STM = true>
int launch_gemm_shape(const CUtensorMap& tmU, const CUtensorMap& tmV, const CUtensorMap& tmM, const GemmParams& prm,
                      int sms, int* status, cudaStream_t st) {
    using L = GemmSmemLayout;
    if (!ensure_dyn_smem(reinterpret_cast<const void*>(wino_gemm_kernel<CTAS, RES, DUAL, false, U8, STM>), MAX_DYN_SMEM)) return err_cuda(__LINE__);
    const long long tiles = static_cast<long long>(prm.num_k_tiles) * prm.num_p_tiles * prm.num_pos;
    const long long workers = sms / CTAS;
    const int grid = static_cast<int>(tiles < workers ? tiles : workers) * CTAS;
    ProfScope prof(KIND_GEMM, st);
    const cudaError_t e =
        launch_pdl(wino_gemm_kernel<CTAS, RES, DUAL, false, U8, STM>, dim3(grid), dim3(GEMM_LAUNCH_THREADS),
                   static_cast<size_t>(L::dyn_bytes(RES ? 0 : prm.n_tile / CTAS, prm.stages, prm.epi_rows,
                                                    prm.epi_alias ? 0 : prm.epi_bufs,
                                                    RES ? prm.num_c_blocks * L::b_bytes(prm.n_tile)
                                                        : (DUAL ? prm.stages * L::A_BYTES
                                                                : (U8 ? prm.raw_slots * L::raw_bytes(prm.n_tile) : 0)))),
                   st, CTAS, tmU, tmV, tmM, prm, status, PipeParams{});
    if (e != cudaSuccess && getenv("SDWINO_LOG"))
        fprintf(stderr, "sdwino: GEMM launch failed: %s (grid %d, stages %d, n_tile %d, resident %d)\n", cudaGetErrorString(e),
                grid, prm.stages, prm.n_tile, prm.resident);
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}

int launch_gemm(const CUtensorMap& tmU, const CUtensorMap& tmV, const CUtensorMap& tmM, const GemmParams& prm,
                int ctas, cudaStream_t st, bool q8 = false) {
    const int sms = sm_count();
    if (sms <= 0) return err_cuda(__LINE__);
    int* status = status_word_ptr();
    if (!status) return err_cuda(__LINE__);
    if (q8) return launch_gemm_shape<1, false, false, true, false>(tmU, tmV, tmM, prm, sms, status, st);
    if (ctas == 2) return launch_gemm_shape<2, false>(tmU, tmV, tmM, prm, sms, status, st);
    if (prm.resident) return launch_gemm_shape<1, true>(tmU, tmV, tmM, prm, sms, status, st);
    if (!prm.epi_stm) {   // one tile per CTA: single CTAs in streaming mode
        if (prm.dual) return launch_gemm_shape<1, false, true, false, false>(tmU, tmV, tmM, prm, sms, status, st);
        return launch_gemm_shape<1, false, false, false, false>(tmU, tmV, tmM, prm, sms, status, st);
    }
    if (prm.dual) return launch_gemm_shape<1, false, true>(tmU, tmV, tmM, prm, sms, status, st);
    return launch_gemm_shape<1, false>(tmU, tmV, tmM, prm, sms, status, st);
}


// ---- the pipelined single-launch path for F(4x4) layers with many tiles and filters that stay in L2 ----
// Workspace: V ring [36][C][ring * 128], M ring [36][K][ring * 128], then the counters.
struct PipePlan {
    int n_tile, resident, group, stages, epi_rows, epi_bufs, epi_chunks;
    int ring, lead, nb;
    size_t v_bytes, m_bytes, ctr_bytes;
};
constexpr int PIPE_CG = 20, PIPE_KG = 20;   // channels per transform item: four rounds of the team's five channel lanes

bool plan_pipeline(const Plan& pl, int C, int K, int sms, int mode, PipePlan* pp) {
    using L = GemmSmemLayout;
    const int nb = static_cast<int>(pl.P128 / GEMM_BLOCK_P);
    const int cblocks = (C + GEMM_BLOCK_C - 1) / GEMM_BLOCK_C;
    const size_t u_bytes = static_cast<size_t>(pl.a2) * pl.Kb * pl.Cb * 2048;
    if (pl.a2 != 36 || nb < 1) return false;
    // the filters are read again for every block of tiles: they must stay in L2 beside the rings
    if (u_bytes > (40u << 20)) return false;
    // Measured on every long layer of the SD VAE / SDXL sweeps the pipelined launch moves a third of the DRAM bytes of
    // the three kernels but takes 17-60 % longer (512->512 at 256x256: 204 against 170 us; 256->256 at 512x512: 408
    // against 257 us): its ten transform warps per SM cannot hide their memory latency the way the transform kernels do
    // with 12-20 resident warps and TMA staging, and the GEMM roles lose time to the per-tile dependency checks.  The
    // library therefore never takes it by itself; mode 2 is for callers who trade time for DRAM traffic, and for tests.
    if (mode == 1) return false;
    const int smem_budget = MAX_DYN_SMEM - 1024;
    // Filter-resident shape first: one (position, k-tile) pair per group of CTAs for the whole launch, so the filter
    // block is loaded once per CTA; the largest n_tile whose block fits beside three or more stages of V.
    pp->resident = 0;
    for (int n = GEMM_MAX_N; n >= 16; n -= 16) {
        const int ktiles = (K + n - 1) / n;
        if (n > 16 && ktiles == (K + n - 17) / (n - 16)) continue;     // a smaller n needs as many tiles
        const int keys = ktiles * pl.a2;
        if (keys > sms) break;
        const bool split = (n / 2) % 16 == 0;
        const int grp = split ? n / 2 : n;
        const int rows = (grp > 64 && grp % 64 == 0) ? 64 : grp;
        const int bufs = split ? 2 : 1;
        const int ures = cblocks * L::b_bytes(n);
        const int stages = (smem_budget - L::dyn_bytes(0, 0, rows, bufs, ures)) / L::A_BYTES;
        if (stages < 3) continue;
        pp->resident = 1;
        pp->n_tile = n;
        pp->group = sms / keys;
        pp->stages = stages > GEMM_MAX_STAGES ? GEMM_MAX_STAGES : stages;
        pp->epi_rows = rows;
        pp->epi_bufs = bufs;
        pp->epi_chunks = grp / rows;
        break;
    }
    if (!pp->resident) {
        const GemmShape shape = choose_gemm_shape(K, C, nb >= 16 ? nb : 16, pl.a2, sms, 1);
        pp->n_tile = shape.n_tile;
        pp->group = 1;
        const bool split = (pp->n_tile / 2) % 16 == 0;
        pp->epi_rows = split ? pp->n_tile / 2 : pp->n_tile;
        pp->epi_bufs = split ? 2 : 1;
        pp->epi_chunks = 1;
        pp->stages = (smem_budget - L::dyn_bytes(pp->n_tile, 0, pp->epi_rows, pp->epi_bufs)) / L::stage_bytes(pp->n_tile);
        if (pp->stages > GEMM_MAX_STAGES) pp->stages = GEMM_MAX_STAGES;
        if (pp->stages < 2) return false;
    }
    const int keys = ((K + pp->n_tile - 1) / pp->n_tile) * pl.a2;
    const int inflight = (sms + keys - 1) / keys;          // blocks of tiles the GEMM roles work on at a time
    int lead = g_pipe_lead.load(), ring = g_pipe_ring.load();
    if (lead <= 0) lead = inflight + 2;
    if (ring <= 0) ring = lead + inflight + 3;
    if (ring > nb) ring = nb;
    if (ring < 1) ring = 1;
    pp->lead = lead;
    pp->ring = ring;
    pp->nb = nb;
    auto up = [](size_t v) { return (v + WS_ALIGN - 1) / WS_ALIGN * WS_ALIGN; };
    pp->v_bytes = up(static_cast<size_t>(pl.a2) * C * ring * GEMM_BLOCK_P * sizeof(__half));
    pp->m_bytes = up(static_cast<size_t>(pl.a2) * K * ring * GEMM_BLOCK_P * sizeof(__half));
    pp->ctr_bytes = up((3 * static_cast<size_t>(nb) + 8) * sizeof(unsigned int));
    return true;
}

int launch_pipeline(const __half* x, const void* wT, const __half* bias, __half* y, const Plan& pl, const TileGeom& geo,
                    int C, int K, const PipePlan& pq, void* ws, cudaStream_t st) {
    using L = GemmSmemLayout;
    const int sms = sm_count();
    int* status = status_word_ptr();
    if (sms <= 0 || !status) return err_cuda(__LINE__);
    uint8_t* base = static_cast<uint8_t*>(ws);
    __half* V = reinterpret_cast<__half*>(base);
    __half* Mws = reinterpret_cast<__half*>(base + pq.v_bytes);
    unsigned int* ctr = reinterpret_cast<unsigned int*>(base + pq.v_bytes + pq.m_bytes);
    const long long ring_p = static_cast<long long>(pq.ring) * GEMM_BLOCK_P;

    GemmParams prm;
    prm.wt_header = wt_header_of(wT);
    prm.K = K;
    prm.tile = 4;
    prm.n_tile = pq.n_tile;
    prm.num_k_tiles = (K + pq.n_tile - 1) / pq.n_tile;
    prm.num_p_tiles = pq.nb;
    prm.fd_p = make_fastdiv(static_cast<uint32_t>(prm.num_p_tiles));
    prm.fd_k = make_fastdiv(static_cast<uint32_t>(prm.num_k_tiles));
    prm.fd_keys = make_fastdiv(static_cast<uint32_t>(prm.num_k_tiles * pl.a2));
    prm.num_pos = pl.a2;
    prm.num_c_blocks = (C + GEMM_BLOCK_C - 1) / GEMM_BLOCK_C;
    prm.C = C;
    prm.stages = pq.stages;
    prm.epi_rows = pq.epi_rows;
    prm.epi_bufs = pq.epi_bufs;
    prm.epi_chunks = pq.epi_chunks;
    prm.resident = pq.resident;
    prm.group = pq.group;
    prm.epi_alias = 0;
    prm.dual = 0;
    prm.p_stride = ring_p;
    prm.scales = nullptr;
    prm.kpad = pl.Kb * 16;
    prm.raw_slots = 0;
    prm.epi_stm = 1;
    prm.epi_dbuf = 0;

    PipeParams pp;
    pp.v_ready = ctr;
    pp.m_done = ctr + pq.nb;
    pp.o_done = ctr + 2 * static_cast<size_t>(pq.nb);
    pp.q_head = ctr + 3 * static_cast<size_t>(pq.nb);
    pp.abort_word = reinterpret_cast<int*>(ctr + 3 * static_cast<size_t>(pq.nb) + 1);
    pp.num_pblocks = pq.nb;
    pp.ring = pq.ring;
    pp.lead = pq.lead;
    pp.cg = PIPE_CG;
    pp.kg = PIPE_KG;
    pp.it_items = (C + PIPE_CG - 1) / PIPE_CG;
    pp.ot_items = (K + PIPE_KG - 1) / PIPE_KG;
    pp.m_target = static_cast<unsigned int>(prm.num_k_tiles * pl.a2 * pq.epi_bufs);
    pp.x = x;
    pp.V = V;
    pp.Mws = Mws;
    pp.bias = bias;
    pp.y = y;
    pp.geo = geo;
    pp.fd64 = make_fastdiv(64);
    {
        // blocks of tiles between two consecutive tiles of one CTA
        const int keys = prm.num_k_tiles * pl.a2;
        const int dist = pq.resident ? pq.group : (sms + keys - 1) / keys + 1;
        pp.defer = pq.ring > dist + 1 ? 1 : 0;
    }

    CUtensorMap tmU, tmV, tmM;
    if (!encode_filter_map(&tmU, wt_filters_of(wT), pl.Cb, pl.Kb, pl.a2, pq.n_tile / 16) ||
        !encode_map(&tmV, V, ring_p, C, pl.a2, ring_p, static_cast<uint64_t>(C) * ring_p, 64, GEMM_BLOCK_C, true) ||
        !encode_map(&tmM, Mws, ring_p, K, pl.a2, ring_p, static_cast<uint64_t>(K) * ring_p, 64, prm.epi_rows, true))
        return err_cuda(__LINE__);
    if (cudaMemsetAsync(ctr, 0, (3 * static_cast<size_t>(pq.nb) + 8) * sizeof(unsigned int), st) != cudaSuccess)
        return err_cuda(__LINE__);
    const size_t smem = static_cast<size_t>(
        L::dyn_bytes(pq.resident ? 0 : pq.n_tile, pq.stages, pq.epi_rows, pq.epi_bufs,
                     pq.resident ? prm.num_c_blocks * L::b_bytes(pq.n_tile) : 0));
    ProfScope prof(KIND_FUSED, st);
    cudaError_t e;
    if (pq.resident) {
        if (!ensure_dyn_smem(reinterpret_cast<const void*>(wino_gemm_kernel<1, true, false, true>), MAX_DYN_SMEM)) return err_cuda(__LINE__);
        e = launch_coop(wino_gemm_kernel<1, true, false, true>, dim3(sms), dim3(PIPE_THREADS), smem, st, tmU, tmV, tmM, prm,
                        status, pp);
    } else {
        if (!ensure_dyn_smem(reinterpret_cast<const void*>(wino_gemm_kernel<1, false, false, true>), MAX_DYN_SMEM)) return err_cuda(__LINE__);
        e = launch_coop(wino_gemm_kernel<1, false, false, true>, dim3(sms), dim3(PIPE_THREADS), smem, st, tmU, tmV, tmM, prm,
                        status, pp);
    }
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}


int conv_impl(const void* x, const void* wT, const void* bias, void* y, int N, int C, int H, int W, int K, int tile,
              void* ws, size_t ws_bytes, cudaStream_t st, const Epilogue& ep_in = Epilogue{nullptr, 0, nullptr},
              bool io32 = false, bool range_safe = false, bool q8 = false, int stride = 0) {
    // io32: x, bias and y are fp32 (the filters come from the fp32 filter transform); stride > 0: the direct
    // convolution (tile 1, fp16 interface), whose tiles are single output pixels
    if (tile == 1 && stride == 0) stride = 1;
    if (stride > 0 ? (tile != 1 || stride > 2 || io32 || q8) : (tile != 2 && tile != 4)) {
        return (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0 || !x || !wT || !y) ? SDWINO_ERR_INVALID_ARG
                                                                                     : SDWINO_ERR_UNSUPPORTED;
    }
    Plan pl;
    if (!x || !wT || !y || !make_plan(N, C, H, W, K, tile, &pl, stride)) return SDWINO_ERR_INVALID_ARG;
    // the overrides are read once per call
    const int force_ctas = g_force_ctas.load(), force_n_tile = g_force_n_tile.load();
    const bool disable_fused = g_disable_fused.load();
    const size_t elem = io32 ? 4 : 2;
    if (!aligned(x, elem) || !aligned(y, elem) || (bias && !aligned(bias, elem)) || !aligned(wT, WS_ALIGN))
        return SDWINO_ERR_MISALIGNED;
    if (!ws || ws_bytes == 0) return SDWINO_ERR_WORKSPACE;
    if (!aligned(ws, WS_ALIGN)) return SDWINO_ERR_MISALIGNED;
    long long pc = tiles_per_pass(pl, ws_bytes);
    if (pc < GEMM_BLOCK_P) return SDWINO_ERR_WORKSPACE;
    ProfScope layer_prof(KIND_LAYER, st);   // profile mode 2: one record for the whole call
    if (tile == 4 && pc < pl.P128) {
        // several passes: cut them at whole tile rows where that keeps the TMA-staged activation transform usable
        const TileGeom g0 = make_geom(H, W, pl.TH, pl.TW, pl.P);
        long long a = pl.TW, b = GEMM_BLOCK_P;
        while (b != 0) { const long long t = a % b; a = b; b = t; }
        const long long lcm = static_cast<long long>(pl.TW) / a * GEMM_BLOCK_P;
        if (pc >= lcm && !io32 && use_input_tma(g0, N, C, x, 0, lcm)) pc = pc / lcm * lcm;
    }
    Epilogue ep = ep_in;
    if (range_safe) {
        // fp32 interface, range-safe call: max|x| goes into a word at the end of the workspace, which the transforms
        // read (see range_exponent); the single-kernel paths are not taken
        if (!io32 || ws_bytes < 2 * WS_ALIGN) return io32 ? SDWINO_ERR_WORKSPACE : SDWINO_ERR_INVALID_ARG;
        ws_bytes -= WS_ALIGN;
        unsigned int* word = reinterpret_cast<unsigned int*>(static_cast<uint8_t*>(ws) + ws_bytes);
        pc = tiles_per_pass(pl, ws_bytes);
        if (pc < GEMM_BLOCK_P) return SDWINO_ERR_WORKSPACE;
        const long long n = static_cast<long long>(N) * C * H * W;
        const int sms = sm_count();
        if (sms <= 0) return err_cuda(__LINE__);
        if (cudaMemsetAsync(word, 0, sizeof(unsigned int), st) != cudaSuccess) return err_cuda(__LINE__);
        const long long want = (n / 4 + 255) / 256;
        const unsigned blocks = static_cast<unsigned>(std::min<long long>(std::max<long long>(want, 1), 8ll * sms));
        if (launch_pdl(absmax_kernel, dim3(blocks), dim3(256), 0, st, 0, static_cast<const float*>(x), n, word) != cudaSuccess)
            return err_cuda(__LINE__);
        g_launches.fetch_add(1);
        ep.amax = reinterpret_cast<const float*>(word);
    }
    // the single-kernel paths end at the bias
    // (8-bit filters: only the GEMM can read them, so neither the single-kernel paths nor the pipelined launch)
    const bool no_ep = ep.residual == nullptr && ep.act == 0 && ep.amax == nullptr && !q8;
    const bool plain = no_ep && !io32;
    if (no_ep && use_fused_small_k(K, W, tile, pl.P128 / 128, x, y) && !use_fused_small_c(C, tile) &&
        (!io32 || aligned(y, 8)) && !disable_fused) {
        if (io32)
            return launch_fused_small_k(static_cast<const float*>(x), wT, static_cast<const float*>(bias),
                                        static_cast<float*>(y), pl, C, H, W, K, st);
        return launch_fused_small_k(static_cast<const __half*>(x), wT, static_cast<const __half*>(bias),
                                    static_cast<__half*>(y), pl, C, H, W, K, st);
    }
    if (no_ep && io32 && tile == 2 && use_fused_small_c(C, tile) && !disable_fused) {
        // the F(2x2) kernel for few input channels also serves the fp32 interface (F(4x4): the three kernels)
        const TileGeom geo = make_geom(H, W, pl.TH, pl.TW, pl.P);
        return launch_fused_small_c_mma(static_cast<const float*>(x), wT, static_cast<const float*>(bias),
                                        static_cast<float*>(y), geo, C, K, pl.Kb, st);
    }
    if (plain && use_fused_small_c(C, tile) && !disable_fused) {
        const TileGeom geo = make_geom(H, W, pl.TH, pl.TW, pl.P);
        const __half* xh = static_cast<const __half*>(x);
        const __half* bh = static_cast<const __half*>(bias);
        __half* yh = static_cast<__half*>(y);
        if (tile == 4) return launch_fused_small_c<4, 4>(xh, wT, bh, yh, geo, C, K, pl.Kb, pl.Cb, st);
        return launch_fused_small_c_mma(xh, wT, bh, yh, geo, C, K, pl.Kb, st);
    }

    // Long F(4x4) layers with small filters: one pipelined launch in which V and M are rings that stay in L2.
    {
        const int pipe_mode = g_pipe_mode.load();
        PipePlan pq;
        if (pipe_mode != 0 && plain && tile == 4 && force_ctas == 0 && force_n_tile == 0 && !use_fused_small_c(C, tile) &&
            W % 8 == 0 && aligned(x, 16) && aligned(y, 16) && plan_pipeline(pl, C, K, sm_count(), pipe_mode, &pq) &&
            pq.v_bytes + pq.m_bytes + pq.ctr_bytes <= ws_bytes) {
            const TileGeom geo = make_geom(H, W, pl.TH, pl.TW, pl.P);
            return launch_pipeline(static_cast<const __half*>(x), wT, static_cast<const __half*>(bias), static_cast<__half*>(y),
                                   pl, geo, C, K, pq, ws, st);
        }
    }

    // workspace: V[a2][C][pc] then M[a2][K][pc]; pc is a multiple of 128 elements, so every row starts
    // on a 256-byte boundary.
    __half* V = static_cast<__half*>(ws);
    size_t v_bytes = static_cast<size_t>(pl.a2) * C * pc * sizeof(__half);
    v_bytes = (v_bytes + WS_ALIGN - 1) / WS_ALIGN * WS_ALIGN;
    __half* Mws = reinterpret_cast<__half*>(static_cast<uint8_t*>(ws) + v_bytes);
    const size_t m_bytes = static_cast<size_t>(pl.a2) * K * pc * sizeof(__half);
    if (v_bytes + m_bytes > ws_bytes) return SDWINO_ERR_WORKSPACE;

    const int sms = sm_count();
    if (sms <= 0) return err_cuda(__LINE__);
    GemmParams prm;
    prm.wt_header = wt_header_of(wT);
    prm.K = K;
    prm.tile = q8 ? (tile | static_cast<int>(WT_Q8_FLAG)) : tile;
    prm.scales = q8 ? reinterpret_cast<const float*>(static_cast<const uint8_t*>(wT) + WT_HEADER_BYTES +
                                                      q8_bytes_part(pl.a2, pl.Kb, pl.Cb))
                    : nullptr;
    prm.kpad = pl.Kb * 16;
    GemmShape shape = choose_gemm_shape(K, C, pc / GEMM_BLOCK_P, pl.a2, sms, q8 ? 1 : force_ctas);
    if (q8) shape.dual = 0;
    if (force_n_tile >= 16 && force_n_tile <= GEMM_MAX_N && force_n_tile % 16 == 0) shape.n_tile = force_n_tile;
    if (shape.ctas == 2) shape.n_tile = round_up(shape.n_tile, 32);  // each CTA of a pair loads whole 16-row blocks
    prm.n_tile = shape.n_tile;
    prm.num_k_tiles = (K + prm.n_tile - 1) / prm.n_tile;
    prm.num_pos = pl.a2;
    prm.fd_k = make_fastdiv(static_cast<uint32_t>(prm.num_k_tiles));
    prm.fd_keys = make_fastdiv(static_cast<uint32_t>(prm.num_k_tiles * pl.a2));
    prm.num_c_blocks = (C + GEMM_BLOCK_C - 1) / GEMM_BLOCK_C;
    prm.C = C;
    const int b_rows = prm.n_tile / shape.ctas;
    if (force_n_tile != 0) shape.dual = 0;
    prm.dual = shape.dual;
    // epilogue staging: two groups of epilogue warps each take half a tile when that is a multiple of 16 channels
    const bool split = (prm.n_tile / 2) % 16 == 0;
    prm.epi_rows = split ? prm.n_tile / 2 : prm.n_tile;
    prm.epi_bufs = split ? 2 : 1;
    prm.epi_chunks = 1;
    prm.resident = 0;
    prm.group = 1;
    {
        // Single CTAs, one pass, at most one tile per CTA: the epilogue borrows the first pipeline stages, and the
        // ring gets the 16-64 KB of the staging buffer (SD v2.1 sweep at batch 1, whose 144-tile layers run two
        // blocks per CTA tile on three stages otherwise: 0.440 -> 0.425 ms; SD v1.5 sweep 0.3379 -> 0.3367 ms).
        // A forced GEMM shape (test hook) keeps the separate buffer, so the tests that compare forced with automatic
        // shapes bit for bit compare both placements.
        const long long p_blocks = shape.dual ? 2 : 1;
        const long long tiles = ((pc / GEMM_BLOCK_P + p_blocks - 1) / p_blocks) * prm.num_k_tiles * pl.a2;
        prm.epi_alias = (shape.ctas == 1 && pc >= pl.P128 && tiles <= sms && force_ctas == 0 && force_n_tile == 0) ? 1 : 0;
    }
    prm.stages = (MAX_DYN_SMEM - GemmSmemLayout::dyn_bytes(b_rows, 0, prm.epi_rows, prm.epi_alias ? 0 : prm.epi_bufs)) /
                 (GemmSmemLayout::stage_bytes(b_rows) + (shape.dual ? GemmSmemLayout::A_BYTES : 0));
    if (prm.stages > GEMM_MAX_STAGES) prm.stages = GEMM_MAX_STAGES;
    prm.raw_slots = 0;
    if (q8) {
        // 8-bit filters: give up one operand stage (down to three at least) for a ring of raw filter boxes, which is
        // what keeps the weight stream from HBM deep: a raw slot is a third of an operand stage or less
        const int room = MAX_DYN_SMEM - GemmSmemLayout::dyn_bytes(b_rows, 0, prm.epi_rows, prm.epi_alias ? 0 : prm.epi_bufs);
        const int raw = GemmSmemLayout::raw_bytes(b_rows), stage = GemmSmemLayout::stage_bytes(b_rows);
        int best_s = 0, best_r = 0;
        for (int sgs = 2; sgs <= GEMM_MAX_STAGES; ++sgs) {
            int r = (room - sgs * stage) / raw;
            if (r > GEMM_MAX_STAGES) r = GEMM_MAX_STAGES;
            if (r < sgs + 1) continue;                       // the raw ring leads the operand ring
            if (sgs <= 3 || r >= 6) { best_s = sgs; best_r = r; }
        }
        if (best_s == 0) return SDWINO_ERR_UNSUPPORTED;
        prm.stages = best_s;
        prm.raw_slots = best_r;
    }
    {
        // Filter-resident mode (see wino_gemm.cuh): single CTAs, many tiles per CTA and long runs of tiles per
        // (position, k-tile), the filter block two thirds of a stage (n_tile 224-256), and room for it beside a ring
        // of at least four V stages once the epilogue stages 64 channels at a time.  Measured: 256->256 at 512x512
        // GEMM 146 -> 120 us, at 1024x1024 570 -> 472 us; with n_tile 128-160 (filters half of a stage or less, the
        // layer close to the HBM roof already) the pause at every change of filter block costs more than the
        // re-reads: 128->128 at 512x512 57 -> 74 us.
        const long long workers = sms / shape.ctas;
        const long long p_tiles = (pc / GEMM_BLOCK_P + shape.ctas - 1) / shape.ctas;     // tiles of 128 (256) tiles p
        const long long keys = ((K + prm.n_tile - 1) / prm.n_tile) * static_cast<long long>(pl.a2);
        const int ures = prm.num_c_blocks * GemmSmemLayout::b_bytes(b_rows);
        const int grp = prm.epi_rows;
        const int rows = (grp > 64 && grp % 64 == 0) ? 64 : grp;   // (32 at a time for a fifth stage measured 2-10 % slower)
        const int stages = (MAX_DYN_SMEM - GemmSmemLayout::dyn_bytes(0, 0, rows, prm.epi_bufs, ures)) / GemmSmemLayout::A_BYTES;
        // (CTA pairs gain nothing from it: with their half of a 512-channel block resident only four 16 KB stages
        // of V remain, too few bytes in flight: 512->512 at 256x256 99 against 94 us)
        if (!q8 && shape.ctas == 1 && !shape.dual && force_ctas == 0 && force_n_tile == 0 && p_tiles >= 16 && keys * p_tiles >= 4 * workers &&
            prm.n_tile >= 224 && stages >= 4) {
            prm.resident = 1;
            // CTAs per (position, k-tile) pair.  A group walks `rounds` pairs, each CTA `run` tiles per pair,
            // and every change of pair costs about a tile and a half (the MMAs that read the old filter block drain,
            // the new block arrives): the group size with the smallest rounds * (run + 1.5) wins, larger groups on
            // ties (their CTAs read neighbouring pieces of V at the same time); runs of at least 8 tiles.
            auto cost = [&](int g) {
                const long long ng = workers / g;
                const long long rounds = (keys + ng - 1) / ng;
                const long long run = (p_tiles + g - 1) / g;
                return static_cast<double>(rounds) * (static_cast<double>(run) + 1.5);
            };
            const int g_max = static_cast<int>(std::min<long long>(workers, p_tiles / 8));
            int best_g = 1;
            for (int g = 2; g <= g_max; ++g)
                if (cost(g) <= cost(best_g) + 1e-9) best_g = g;
            prm.group = best_g;
            prm.epi_chunks = grp / rows;
            prm.epi_rows = rows;
            prm.stages = stages > GEMM_MAX_STAGES ? GEMM_MAX_STAGES : stages;
        }
    }

    if (!prm.resident && !prm.epi_alias && !q8 && force_ctas == 0 && force_n_tile == 0) {
        // The ring is short of stages against its round trip (a stage's loads take 2-3.5 thousand cycles to arrive
        // under load, its MMAs 300-500): an epilogue group that stages its channels 64 or 32 at a time instead of all
        // at once leaves room for one more stage in most shapes.  Measured: CTA pairs at n_tile 256 go from five to
        // six stages, 1280->1280 at 64x64 (batch 2) 63.8 -> 58.3 us, 512->512 at 512x512 363 -> 345 us; 16 at a time
        // costs more in the epilogue than the stage returns (320->320 at 128x128: 28 -> 35 us).
        const int stage = GemmSmemLayout::stage_bytes(b_rows) + (shape.dual ? GemmSmemLayout::A_BYTES : 0);
        auto stages_for = [&](int rows) {
            const int st = (MAX_DYN_SMEM - GemmSmemLayout::dyn_bytes(b_rows, 0, rows, prm.epi_bufs)) / stage;
            return st > GEMM_MAX_STAGES ? GEMM_MAX_STAGES : st;
        };
        const int grp = prm.epi_rows;
        int best_rows = grp, best_stages = stages_for(grp);
        for (int rows = 64; rows >= 32; rows >>= 1) {
            if (rows >= grp || grp % rows != 0) continue;
            if (stages_for(rows) > best_stages) { best_stages = stages_for(rows); best_rows = rows; }
        }
        prm.epi_chunks = grp / best_rows;
        prm.epi_rows = best_rows;
        prm.stages = best_stages;
    }
    // Epilogue staging: stmatrix into swizzled boxes where a CTA has several tiles (throughput: 3-8 % on those GEMMs),
    // plain 2-byte stores into one box where it has one (its two TMA stores of 128-byte rows drain later at the tail
    // of the launch: 0.5-1.5 us per layer of the SD v1.5 sweep).
    prm.epi_dbuf = 0;
    if (!q8 && prm.epi_chunks >= 2 && prm.epi_rows == 64) {
        // Two buffers of 32 channels in the place of one of 64: a group then stages one piece while the TMA store still
        // reads the other, instead of waiting 1.3-1.8 thousand cycles for it between the pieces (-1.5 to -2 % on the
        // GEMMs with several tiles per CTA).
        prm.epi_dbuf = 1;
        prm.epi_rows = 32;
        prm.epi_chunks *= 2;
        prm.epi_bufs *= 2;
    }
    prm.epi_stm = (!q8 && !prm.epi_alias) ? 1 : 0;   // (an aliased staging buffer implies single CTAs in streaming mode)
    prm.p_stride = pc;
    CUtensorMap tmU, tmV, tmM;
    if (!(q8 ? encode_filter_map_q8(&tmU, wt_filters_of(wT), pl.Cb, pl.Kb, pl.a2, b_rows / 16)
             : encode_filter_map(&tmU, wt_filters_of(wT), pl.Cb, pl.Kb, pl.a2, b_rows / 16)) ||
        !encode_map(&tmV, V, pc, C, pl.a2, pc, static_cast<uint64_t>(C) * pc, 64, GEMM_BLOCK_C, true) ||
        !encode_map(&tmM, Mws, pc, K, pl.a2, pc, static_cast<uint64_t>(K) * pc, prm.epi_stm ? 64 : GEMM_BLOCK_P, prm.epi_rows,
                    prm.epi_stm != 0))
        return err_cuda(__LINE__);

    const TileGeom geo = make_geom(H, W, pl.TH, pl.TW, pl.P, stride > 0 ? stride : 1);
    const TileGeom geo_out = make_geom(pl.Ho, pl.Wo, pl.TH, pl.TW, pl.P);    // differs from geo for the strided convolution
    const __half* xh = static_cast<const __half*>(x);
    const __half* bh = static_cast<const __half*>(bias);
    __half* yh = static_cast<__half*>(y);
    const WtCheck chk{wt_header_of(wT), K, C, prm.tile, status_word_ptr()};
    if (!chk.status_word) return err_cuda(__LINE__);
    for (long long p0 = 0; p0 < pl.P; p0 += pc) {
        long long remaining = pl.P128 - p0;
        const int count = static_cast<int>(remaining < pc ? remaining : pc);  // multiple of 128
        int rc;
        if (io32) {
            const float* xf = static_cast<const float*>(x);
            rc = tile == 2 ? launch_input<2>(xf, V, geo, C, p0, count, pc, st, ep.amax)
                           : launch_input<4>(xf, V, geo, C, p0, count, pc, st, ep.amax);
        } else if (tile == 1) rc = launch_input<1>(xh, V, geo, C, p0, count, pc, st);
        else if (tile == 2) rc = launch_input<2>(xh, V, geo, C, p0, count, pc, st);
        else {
            rc = use_input_tma(geo, N, C, x, p0, count) ? launch_input_tma(xh, V, geo, N, C, p0, count, pc, st)
                                                        : SDWINO_ERR_UNSUPPORTED;
            if (rc == SDWINO_ERR_UNSUPPORTED) rc = launch_input<4>(xh, V, geo, C, p0, count, pc, st);   // grid limits
        }
        if (rc != SDWINO_OK) return rc;
        const int p_blocks = shape.ctas * (shape.dual ? 2 : 1);      // blocks of 128 tiles per CTA tile / pair tile
        prm.num_p_tiles = (count / GEMM_BLOCK_P + p_blocks - 1) / p_blocks;
        prm.fd_p = make_fastdiv(static_cast<uint32_t>(prm.num_p_tiles));
        rc = launch_gemm(tmU, tmV, tmM, prm, shape.ctas, st, q8);
        if (rc != SDWINO_OK) return rc;
        if (io32) {
            const float* bf = static_cast<const float*>(bias);
            float* yf = static_cast<float*>(y);
            if (tile == 2) rc = launch_output<2>(Mws, bf, yf, geo, K, p0, count, pc, chk, ep, st);
            else if (use_output_tma(geo, K, y, ep, count)) rc = launch_output_tma(Mws, bf, yf, geo, K, p0, count, pc, chk, ep, st);
            else rc = launch_output<4>(Mws, bf, yf, geo, K, p0, count, pc, chk, ep, st);
        } else if (tile == 1) rc = launch_output<1>(Mws, bh, yh, geo_out, K, p0, count, pc, chk, ep, st);
        else if (tile == 2) rc = launch_output<2>(Mws, bh, yh, geo, K, p0, count, pc, chk, ep, st);
        else if (use_output_tma(geo, K, y, ep, count)) rc = launch_output_tma(Mws, bh, yh, geo, K, p0, count, pc, chk, ep, st);
        else rc = launch_output<4>(Mws, bh, yh, geo, K, p0, count, pc, chk, ep, st);
        if (rc != SDWINO_OK) return rc;
    }
    return SDWINO_OK;
}

}  // namespace

extern "C" {

int sdwino_version(void) { return 100; }

int sdwino_set_gemm_shape(int ctas, int n_tile) {
    if (ctas < 0 || ctas > 2 || n_tile < 0 || n_tile > GEMM_MAX_N || n_tile % 16 != 0) return SDWINO_ERR_INVALID_ARG;
    g_force_ctas = ctas;
    g_force_n_tile = n_tile;
    g_disable_fused = (ctas != 0 || n_tile != 0);
    return SDWINO_OK;
}

int sdwino_set_input_staging(int mode) {
    if (mode < 0 || mode > 2) return SDWINO_ERR_INVALID_ARG;
    g_input_staging = mode;
    return SDWINO_OK;
}

int sdwino_set_pipeline(int mode, int ring, int lead) {
    if (mode < 0 || mode > 2 || ring < 0 || lead < 0) return SDWINO_ERR_INVALID_ARG;
    g_pipe_mode.store(mode);
    g_pipe_ring.store(ring);
    g_pipe_lead.store(lead);
    return SDWINO_OK;
}

int sdwino_choose_tile(int N, int C, int H, int W, int K) {
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0) return 0;
    // Layers with few input channels have a single-kernel F(2x2) path.  Otherwise F(4x4) moves 2.25 instead of 4 transform
    // values per pixel through the workspace and the tensor cores but streams 36 instead of 16 values per
    // weight: it wins once the tiles outnumber the weights per channel pair.  Measured on 97 layer shapes:
    // F4 is 15-40 % faster above twice the threshold below, within +-7 % around it, up to 2x slower far below.
    const long long P2 = static_cast<long long>(N) * ((H + 1) / 2) * ((W + 1) / 2);
    if (C <= 8) return 2;
    // few output channels: the single-kernel F(2x2) path needs many blocks of tiles to fill the SMs; below about
    // a hundred of them the three-kernel F(4x4) path is 5-20 % faster (320->4 at 64x64: 12.2 against 14.7 us)
    if (K <= 8) return P2 >= 12288 ? 2 : 4;
    const long long act = 2 * P2 * (static_cast<long long>(C) + K), wgt = static_cast<long long>(K) * C;
    if (act >= wgt) return 4;
    // between 0.65 and 1 of the threshold F4 is still 7-10 % faster once there are 256 tiles or more (2560->1280 at
    // 24x24, batch 2: 53 against 59 us), and 4-35 % slower with fewer (640->1280 at 24x24, batch 1)
    return (20 * act >= 13 * wgt && P2 >= 256) ? 4 : 2;
}

int sdwino_choose_algorithm(int N, int C, int H, int W, int K) {
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0) return 0;
    // Layers whose whole batch is at most one block of 128 output pixels (the 8x8 layers of the UNet at batch 2):
    // F(2x2) would fill a quarter of its block of 128 tiles and stream 16 values per weight, the direct form fills
    // its block and streams 9.  Measured: 1280->1280 at 8x8, batch 2: 22.5 against 26.6 us, 2560->1280: 32.8 against
    // 36.9 us; from two blocks of pixels on (12x12, 16x16) the direct form re-reads the filters per block and loses.
    if (C > 8 && K > 8 && static_cast<long long>(N) * H * W <= GEMM_BLOCK_P) return 1;
    return sdwino_choose_tile(N, C, H, W, K);
}

int sdwino_set_fused_min_tiles(long long p_tiles) {
    if (p_tiles < 0) return SDWINO_ERR_INVALID_ARG;
    g_fk_min_p_tiles = p_tiles == 0 ? FK_MIN_P_TILES : p_tiles;
    return SDWINO_OK;
}

const char* sdwino_status_string(int status) {
    switch (status) {
        case SDWINO_OK: return "ok";
        case SDWINO_ERR_INVALID_ARG: return "invalid argument";
        case SDWINO_ERR_UNSUPPORTED: return "unsupported tile size";
        case SDWINO_ERR_MISALIGNED: return "misaligned pointer";
        case SDWINO_ERR_WORKSPACE: return "workspace missing or too small";
        case SDWINO_ERR_CUDA: return "CUDA error";
        case SDWINO_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

size_t sdwino_filter_bytes(int K, int C, int tile) {
    if (K <= 0 || C <= 0 || (tile != 1 && tile != 2 && tile != 4)) return 0;
    const size_t a = tile + 2;
    const size_t bytes = a * a * static_cast<size_t>((K + 15) / 16) * ((C + 63) / 64) * 1024 * sizeof(__half);
    return WT_HEADER_BYTES + (bytes + WS_ALIGN - 1) / WS_ALIGN * WS_ALIGN;   // header + U
}

int sdwino_filter_transform(const void* w, void* wT, int K, int C, int tile, void* stream) {
    if (!w || !wT || K <= 0 || C <= 0) return SDWINO_ERR_INVALID_ARG;
    if (tile != 1 && tile != 2 && tile != 4) return SDWINO_ERR_UNSUPPORTED;
    if (!aligned(w, 2) || !aligned(wT, WS_ALIGN)) return SDWINO_ERR_MISALIGNED;
    if (static_cast<long double>(K) * C > 4.0e15L) return SDWINO_ERR_INVALID_ARG;
    const int Kb = (K + 15) / 16, Cb = (C + 63) / 64;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (tile == 1) return launch_filter<1>(static_cast<const __half*>(w), wT, K, C, Kb, Cb, st);
    if (tile == 2) return launch_filter<2>(static_cast<const __half*>(w), wT, K, C, Kb, Cb, st);
    return launch_filter<4>(static_cast<const __half*>(w), wT, K, C, Kb, Cb, st);
}

size_t sdwino_filter_q8_bytes(int K, int C, int tile) {
    if (K <= 0 || C <= 0 || (tile != 2 && tile != 4)) return 0;
    const int a2 = (tile + 2) * (tile + 2), Kb = (K + 15) / 16, Cb = (C + 63) / 64;
    return WT_HEADER_BYTES + q8_bytes_part(a2, Kb, Cb) + q8_scale_part(a2, Kb);
}

int sdwino_filter_quantize(const void* wT, void* wTq, int K, int C, int tile, void* stream) {
    if (!wT || !wTq || K <= 0 || C <= 0) return SDWINO_ERR_INVALID_ARG;
    if (tile != 2 && tile != 4) return SDWINO_ERR_UNSUPPORTED;
    if (!aligned(wT, WS_ALIGN) || !aligned(wTq, WS_ALIGN)) return SDWINO_ERR_MISALIGNED;
    if (static_cast<long double>(K) * C > 4.0e15L) return SDWINO_ERR_INVALID_ARG;
    const int a2 = (tile + 2) * (tile + 2), Kb = (K + 15) / 16, Cb = (C + 63) / 64;
    if (static_cast<long long>(a2) * Kb >= (1ll << 31)) return SDWINO_ERR_INVALID_ARG;
    int* status = status_word_ptr();
    if (!status) return err_cuda(__LINE__);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t* out = static_cast<uint8_t*>(wTq);
    ProfScope prof(KIND_FILTER, st);
    const cudaError_t e = launch_pdl(filter_quantize_kernel, dim3(static_cast<unsigned>(a2 * Kb)), dim3(128), 0, st, 0,
                                     wt_header_of(wT), static_cast<const __half*>(wt_filters_of(wT)),
                                     reinterpret_cast<uint32_t*>(out), out + WT_HEADER_BYTES,
                                     reinterpret_cast<float*>(out + WT_HEADER_BYTES + q8_bytes_part(a2, Kb, Cb)), K, C, tile,
                                     Kb, Cb, status);
    g_launches.fetch_add(1);
    return e == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}

int sdwino_conv3x3_q8(const void* x, const void* wTq, const void* bias, void* y, int N, int C, int H, int W, int K,
                      int tile, void* workspace, size_t workspace_bytes, void* stream) {
    return conv_impl(x, wTq, bias, y, N, C, H, W, K, tile, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                     Epilogue{nullptr, 0, nullptr}, false, false, true);
}

size_t sdwino_workspace_bytes_direct(int N, int C, int H, int W, int K, int stride) {
    Plan pl;
    if (stride < 1 || !make_plan(N, C, H, W, K, 1, &pl, stride)) return 0;
    const long long pc = tiles_per_pass(pl, static_cast<size_t>(-1) / 2);
    return static_cast<size_t>(pc) * pl.per_tile + WS_ALIGN;
}

int sdwino_conv3x3_direct(const void* x, const void* wT, const void* bias, void* y, int N, int C, int H, int W, int K,
                          int stride, void* workspace, size_t workspace_bytes, void* stream) {
    if (stride < 1) return SDWINO_ERR_INVALID_ARG;
    return conv_impl(x, wT, bias, y, N, C, H, W, K, 1, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                     Epilogue{nullptr, 0, nullptr}, false, false, false, stride);
}

int sdwino_filter_transform_f32(const float* w, void* wT, int K, int C, int tile, void* stream) {
    if (!w || !wT || K <= 0 || C <= 0) return SDWINO_ERR_INVALID_ARG;
    if (tile != 2 && tile != 4) return SDWINO_ERR_UNSUPPORTED;
    if (!aligned(w, 4) || !aligned(wT, WS_ALIGN)) return SDWINO_ERR_MISALIGNED;
    if (static_cast<long double>(K) * C > 4.0e15L) return SDWINO_ERR_INVALID_ARG;
    const int Kb = (K + 15) / 16, Cb = (C + 63) / 64;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (tile == 2) return launch_filter<2>(w, wT, K, C, Kb, Cb, st);
    return launch_filter<4>(w, wT, K, C, Kb, Cb, st);
}

size_t sdwino_workspace_bytes(int N, int C, int H, int W, int K, int tile) {
    Plan pl;
    if (!make_plan(N, C, H, W, K, tile, &pl)) return 0;
    const long long pc = tiles_per_pass(pl, static_cast<size_t>(-1) / 2);
    return static_cast<size_t>(pc) * pl.per_tile + WS_ALIGN;
}

size_t sdwino_workspace_min_bytes(int N, int C, int H, int W, int K, int tile) {
    Plan pl;
    if (!make_plan(N, C, H, W, K, tile, &pl)) return 0;
    return static_cast<size_t>(GEMM_BLOCK_P) * pl.per_tile + WS_ALIGN;
}

int sdwino_set_workspace(void* workspace, size_t bytes) {
    if ((workspace == nullptr) != (bytes == 0)) return SDWINO_ERR_INVALID_ARG;
    if (workspace && !aligned(workspace, WS_ALIGN)) return SDWINO_ERR_MISALIGNED;
    std::lock_guard<std::mutex> lock(g_mutex);
    g_workspace = workspace;
    g_workspace_bytes = bytes;
    return SDWINO_OK;
}

int sdwino_conv3x3_ws(const void* x, const void* wT, const void* bias, void* y, int N, int C, int H, int W, int K,
                      int tile, void* workspace, size_t workspace_bytes, void* stream) {
    return conv_impl(x, wT, bias, y, N, C, H, W, K, tile, workspace, workspace_bytes,
                     static_cast<cudaStream_t>(stream));
}

int sdwino_conv3x3_ex(const void* x, const void* wT, const void* bias, const void* residual, void* y, int N, int C,
                      int H, int W, int K, int tile, int activation, void* workspace, size_t workspace_bytes,
                      void* stream) {
    if (activation != SDWINO_ACT_NONE && activation != SDWINO_ACT_SILU) return SDWINO_ERR_UNSUPPORTED;
    if (residual && !aligned(residual, 2)) return SDWINO_ERR_MISALIGNED;
    return conv_impl(x, wT, bias, y, N, C, H, W, K, tile, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                     Epilogue{residual, activation, nullptr});
}

int sdwino_conv3x3_f32(const float* x, const void* wT, const float* bias, float* y, int N, int C, int H, int W, int K,
                       int tile, void* workspace, size_t workspace_bytes, void* stream) {
    return conv_impl(x, wT, bias, y, N, C, H, W, K, tile, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                     Epilogue{nullptr, 0, nullptr}, true);
}

int sdwino_conv3x3_f32_scaled(const float* x, const void* wT, const float* bias, float* y, int N, int C, int H, int W,
                              int K, int tile, void* workspace, size_t workspace_bytes, void* stream) {
    return conv_impl(x, wT, bias, y, N, C, H, W, K, tile, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                     Epilogue{nullptr, 0, nullptr}, true, true);
}

int sdwino_conv3x3_f32_ex(const float* x, const void* wT, const float* bias, const float* residual, float* y, int N,
                          int C, int H, int W, int K, int tile, int activation, void* workspace, size_t workspace_bytes,
                          void* stream) {
    if (activation != SDWINO_ACT_NONE && activation != SDWINO_ACT_SILU) return SDWINO_ERR_UNSUPPORTED;
    if (residual && !aligned(residual, 4)) return SDWINO_ERR_MISALIGNED;
    return conv_impl(x, wT, bias, y, N, C, H, W, K, tile, workspace, workspace_bytes, static_cast<cudaStream_t>(stream),
                     Epilogue{residual, activation, nullptr}, true);
}

int sdwino_conv3x3(const void* x, const void* wT, const void* bias, void* y, int N, int C, int H, int W, int K,
                   int tile, void* stream) {
    void* ws;
    size_t bytes;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        ws = g_workspace;
        bytes = g_workspace_bytes;
    }
    return conv_impl(x, wT, bias, y, N, C, H, W, K, tile, ws, bytes, static_cast<cudaStream_t>(stream));
}

namespace {
size_t host_staging_bytes(int N, int C, int H, int W, int K, int tile, size_t elem) {
    Plan pl;
    if (!make_plan(N, C, H, W, K, tile, &pl)) return 0;
    auto up = [](size_t v) { return (v + WS_ALIGN - 1) / WS_ALIGN * WS_ALIGN; };
    const size_t xb = up(static_cast<size_t>(N) * C * H * W * elem);
    const size_t yb = up(static_cast<size_t>(N) * K * H * W * elem);
    const size_t bb = up(static_cast<size_t>(K) * elem);
    return 2 * (xb + bb + yb);   // two slots: uploads, kernels and downloads of consecutive calls overlap
}
}  // namespace

size_t sdwino_host_staging_bytes(int N, int C, int H, int W, int K, int tile) {
    return host_staging_bytes(N, C, H, W, K, tile, sizeof(__half));
}
size_t sdwino_host_staging_bytes_f32(int N, int C, int H, int W, int K, int tile) {
    return host_staging_bytes(N, C, H, W, K, tile, sizeof(float));
}

namespace {
// Per-device state of the asynchronous host path: one copy stream per direction and a ring of the most recent
// calls (what memory each used, with which sizes and staging slot, and its three events).  A new call is ordered
// only after earlier calls that touch the same memory, so the copies of layers with workspaces of their own run
// ahead of the kernels as far as the copy streams allow.  Created on first use.
constexpr int HOST_RING = 32;
struct HostCall {
    bool used = false;
    const uint8_t* begin = nullptr;   // workspace of the call
    const uint8_t* end = nullptr;
    size_t sizes[3] = {0, 0, 0};      // bytes of x, bias, y
    int slot = 0;                     // half of the staging area
    cudaEvent_t uploaded = nullptr;   // on s_in: x (and bias) are on the device
    cudaEvent_t computed = nullptr;   // on the caller's stream: the kernels have read x and written y
    cudaEvent_t downloaded = nullptr; // on s_out: y has reached host memory
};
struct HostPipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    HostCall ring[HOST_RING];
    unsigned long long calls = 0;
};
HostPipe g_host_pipe[STATIC_MAX_DEVICES_HOST];

HostPipe* host_pipe() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= STATIC_MAX_DEVICES_HOST) return nullptr;
    HostPipe& hp = g_host_pipe[dev];
    if (!hp.ready) {
        if (cudaStreamCreateWithFlags(&hp.s_in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaStreamCreateWithFlags(&hp.s_out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        for (int i = 0; i < HOST_RING; ++i) {
            if (cudaEventCreateWithFlags(&hp.ring[i].uploaded, cudaEventDisableTiming) != cudaSuccess) return nullptr;
            if (cudaEventCreateWithFlags(&hp.ring[i].computed, cudaEventDisableTiming) != cudaSuccess) return nullptr;
            if (cudaEventCreateWithFlags(&hp.ring[i].downloaded, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        }
        hp.ready = true;
    }
    return &hp;
}
}  // namespace

namespace {
int host_async_impl(const void* x_host, const void* wT, const void* bias_host, void* y_host, int N, int C,
                    int H, int W, int K, int tile, void* workspace, size_t workspace_bytes, void* stream, bool io32) {
    if (!x_host || !y_host || !wT) return SDWINO_ERR_INVALID_ARG;
    if (tile != 2 && tile != 4 && !(tile == 1 && !io32)) return SDWINO_ERR_UNSUPPORTED;
    const size_t elem = io32 ? sizeof(float) : sizeof(__half);
    const size_t staging = host_staging_bytes(N, C, H, W, K, tile, elem);
    if (staging == 0) return SDWINO_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes <= staging) return SDWINO_ERR_WORKSPACE;
    if (!aligned(workspace, WS_ALIGN)) return SDWINO_ERR_MISALIGNED;
    HostPipe* hp = host_pipe();
    if (!hp) return err_cuda(__LINE__);
    auto up = [](size_t v) { return (v + WS_ALIGN - 1) / WS_ALIGN * WS_ALIGN; };
    const size_t xbytes = static_cast<size_t>(N) * C * H * W * elem;
    const size_t ybytes = static_cast<size_t>(N) * K * H * W * elem;
    const size_t bbytes = static_cast<size_t>(K) * elem;
    uint8_t* base = static_cast<uint8_t*>(workspace);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // Earlier calls, newest first.  One with the same workspace and sizes owns one half (slot) of the staging area:
    // this call takes the other half and waits only for the newest call that had its own half (its kernels before
    // the upload, its download before the kernels).  One that overlaps this workspace with other sizes laid its
    // copies and its scratch out differently: everything of it, download included, comes first.
    int slot = -1;
    bool waited_same_slot = false;
    const unsigned long long first = hp->calls > HOST_RING ? hp->calls - HOST_RING : 0;
    for (unsigned long long c = hp->calls; c-- > first;) {
        const HostCall& e = hp->ring[c % HOST_RING];
        if (!e.used || !(base < e.end && e.begin < base + workspace_bytes)) continue;
        const bool same = e.begin == base && e.end == base + workspace_bytes && e.sizes[0] == xbytes &&
                          e.sizes[1] == bbytes && e.sizes[2] == ybytes;
        if (same) {
            if (slot < 0) slot = 1 - e.slot;          // the newest one decides
            if (e.slot == slot && !waited_same_slot) {
                // (a wait for an event that has completed would still cost the copy stream a semaphore)
                if (cudaEventQuery(e.downloaded) != cudaSuccess &&
                    (cudaStreamWaitEvent(hp->s_in, e.computed, 0) != cudaSuccess ||
                     cudaStreamWaitEvent(st, e.downloaded, 0) != cudaSuccess))
                    return err_cuda(__LINE__);
                waited_same_slot = true;
            }
        } else {
            if (cudaStreamWaitEvent(hp->s_in, e.computed, 0) != cudaSuccess ||
                cudaStreamWaitEvent(hp->s_in, e.downloaded, 0) != cudaSuccess ||
                cudaStreamWaitEvent(st, e.downloaded, 0) != cudaSuccess)
                return err_cuda(__LINE__);
        }
    }
    if (slot < 0) slot = 0;
    // the ring entry this call takes over belongs to a call of HOST_RING calls ago: it is forgotten only once it
    // has completed
    HostCall& me = hp->ring[hp->calls % HOST_RING];
    if (me.used && cudaEventQuery(me.downloaded) != cudaSuccess &&   // its download is its last operation
        (cudaStreamWaitEvent(hp->s_in, me.downloaded, 0) != cudaSuccess ||
         cudaStreamWaitEvent(st, me.downloaded, 0) != cudaSuccess))
        return err_cuda(__LINE__);
    me.used = false;

    uint8_t* xd = base + slot * up(xbytes);
    uint8_t* bd = base + 2 * up(xbytes) + slot * up(bbytes);
    uint8_t* yd = base + 2 * (up(xbytes) + up(bbytes)) + slot * up(ybytes);
    uint8_t* ws = base + staging;
    // upload on the first copy stream
    if (cudaMemcpyAsync(xd, x_host, xbytes, cudaMemcpyHostToDevice, hp->s_in) != cudaSuccess) return err_cuda(__LINE__);
    if (bias_host && cudaMemcpyAsync(bd, bias_host, bbytes, cudaMemcpyHostToDevice, hp->s_in) != cudaSuccess)
        return err_cuda(__LINE__);
    if (cudaEventRecord(me.uploaded, hp->s_in) != cudaSuccess) return err_cuda(__LINE__);
    // kernels on the caller's stream
    if (cudaStreamWaitEvent(st, me.uploaded, 0) != cudaSuccess) return err_cuda(__LINE__);
    const int rc = conv_impl(xd, wT, bias_host ? bd : nullptr, yd, N, C, H, W, K, tile, ws, workspace_bytes - staging, st,
                             Epilogue{nullptr, 0, nullptr}, io32);
    if (rc != SDWINO_OK) return rc;
    if (cudaEventRecord(me.computed, st) != cudaSuccess) return err_cuda(__LINE__);
    // download on the second copy stream
    if (cudaStreamWaitEvent(hp->s_out, me.computed, 0) != cudaSuccess) return err_cuda(__LINE__);
    if (cudaMemcpyAsync(y_host, yd, ybytes, cudaMemcpyDeviceToHost, hp->s_out) != cudaSuccess) return err_cuda(__LINE__);
    if (cudaEventRecord(me.downloaded, hp->s_out) != cudaSuccess) return err_cuda(__LINE__);
    me.used = true;
    me.begin = base;
    me.end = base + workspace_bytes;
    me.sizes[0] = xbytes;
    me.sizes[1] = bbytes;
    me.sizes[2] = ybytes;
    me.slot = slot;
    ++hp->calls;
    return SDWINO_OK;
}
}  // namespace

int sdwino_conv3x3_host_async(const void* x_host, const void* wT, const void* bias_host, void* y_host, int N, int C,
                              int H, int W, int K, int tile, void* workspace, size_t workspace_bytes, void* stream) {
    return host_async_impl(x_host, wT, bias_host, y_host, N, C, H, W, K, tile, workspace, workspace_bytes, stream, false);
}

int sdwino_conv3x3_host_f32_async(const float* x_host, const void* wT, const float* bias_host, float* y_host, int N, int C,
                                  int H, int W, int K, int tile, void* workspace, size_t workspace_bytes, void* stream) {
    return host_async_impl(x_host, wT, bias_host, y_host, N, C, H, W, K, tile, workspace, workspace_bytes, stream, true);
}

int sdwino_host_join(void* stream) {
    HostPipe* hp = host_pipe();
    if (!hp) return err_cuda(__LINE__);
    if (hp->calls == 0) return SDWINO_OK;
    // the download stream works in order: the newest download is the last one to finish
    const HostCall& last = hp->ring[(hp->calls - 1) % HOST_RING];
    if (last.used && cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), last.downloaded, 0) != cudaSuccess)
        return err_cuda(__LINE__);
    return SDWINO_OK;
}

int sdwino_conv3x3_host(const void* x_host, const void* wT, const void* bias_host, void* y_host, int N, int C, int H,
                        int W, int K, int tile, void* workspace, size_t workspace_bytes, void* stream) {
    const int rc = sdwino_conv3x3_host_async(x_host, wT, bias_host, y_host, N, C, H, W, K, tile, workspace,
                                             workspace_bytes, stream);
    if (rc != SDWINO_OK) return rc;
    if (sdwino_host_join(stream) != SDWINO_OK) return err_cuda(__LINE__);
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return err_cuda(__LINE__);
    return SDWINO_OK;
}

int sdwino_conv3x3_host_f32(const float* x_host, const void* wT, const float* bias_host, float* y_host, int N, int C,
                            int H, int W, int K, int tile, void* workspace, size_t workspace_bytes, void* stream) {
    const int rc = sdwino_conv3x3_host_f32_async(x_host, wT, bias_host, y_host, N, C, H, W, K, tile, workspace,
                                                 workspace_bytes, stream);
    if (rc != SDWINO_OK) return rc;
    if (sdwino_host_join(stream) != SDWINO_OK) return err_cuda(__LINE__);
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return err_cuda(__LINE__);
    return SDWINO_OK;
}

int sdwino_last_device_status(void* stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return err_cuda(__LINE__);
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_status_word, sizeof(int)) != cudaSuccess) return err_cuda(__LINE__);
    if (v != 0) {
        int zero = 0;
        if (cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int)) != cudaSuccess) return err_cuda(__LINE__);
        if (getenv("SDWINO_LOG")) fprintf(stderr, "sdwino: device status word 0x%x\n", v);
    }
    return v & 0xFF;
}

unsigned long long sdwino_launch_count(void) { return g_launches.load(); }

int sdwino_selftest_wait_timeout(unsigned long long limit_ns, void* stream) {
    if (limit_ns == 0 || limit_ns > 10000000ull) return SDWINO_ERR_INVALID_ARG;   // at most 10 ms
    int* status = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&status), g_status_word) != cudaSuccess) return err_cuda(__LINE__);
    wait_timeout_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status, limit_ns);
    g_launches.fetch_add(1);
    return cudaGetLastError() == cudaSuccess ? SDWINO_OK : err_cuda(__LINE__);
}

}  // extern "C"

namespace {
// Scratch for sdwino_conv3x3_static: lives in the library's device image, so no allocation call is ever
// made for it.  In host code this name is only a stand-in for the device object (it is not a device
// address); the address kernels can use comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_static_scratch[SDWINO_STATIC_SCRATCH_BYTES];
constexpr int STATIC_MAX_DEVICES = 64;
void* g_static_scratch_ptr[STATIC_MAX_DEVICES] = {};
std::mutex g_static_mutex;
}  // namespace

extern "C" {

int sdwino_conv3x3_static(const void* x, const void* wT, const void* bias, void* y, int N, int C, int H, int W,
                          int K, int tile, void* stream) {
    if (tile != 1 && tile != 2 && tile != 4) {
        return (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0 || !x || !wT || !y) ? SDWINO_ERR_INVALID_ARG
                                                                                     : SDWINO_ERR_UNSUPPORTED;
    }
    Plan pl;
    if (!x || !wT || !y || !make_plan(N, C, H, W, K, tile, &pl)) return SDWINO_ERR_INVALID_ARG;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return err_cuda(__LINE__);
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return SDWINO_ERR_UNSUPPORTED;
    void* base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_scratch_ptr[dev]) {
            // set-up, once per device, with that device current
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return err_cuda(__LINE__);
            g_static_scratch_ptr[dev] = p;
        }
        base = g_static_scratch_ptr[dev];
    }
    // the convolution wants its scratch on a 1024-byte boundary; the array is only promised 256
    const uintptr_t raw = reinterpret_cast<uintptr_t>(base);
    const uintptr_t up = (raw + WS_ALIGN - 1) / WS_ALIGN * WS_ALIGN;
    const size_t usable = SDWINO_STATIC_SCRATCH_BYTES - static_cast<size_t>(up - raw);
    // sizes beyond the maximum: even one pass of 128 tiles would not fit
    if (static_cast<size_t>(GEMM_BLOCK_P) * pl.per_tile + WS_ALIGN > usable) return SDWINO_ERR_WORKSPACE;
    return conv_impl(x, wT, bias, y, N, C, H, W, K, tile, reinterpret_cast<void*>(up), usable,
                     static_cast<cudaStream_t>(stream));
}

}  // extern "C"

namespace {
// Issues the L2 prefetches of the first `bytes_per_pos` bytes of every transform position of a filter tensor, the
// positions advancing together (the GEMM's CTAs work on all positions at once, each through the channel blocks in
// order).  Nothing waits for the prefetches: the kernel ends as soon as they are queued.
constexpr uint32_t PREFETCH_CHUNK = 4096;
__global__ void __launch_bounds__(128) filter_prefetch_kernel(const uint8_t* __restrict__ base, size_t pos_stride,
                                                             size_t bytes_per_pos, int num_pos) {
    const size_t chunks_per_pos = (bytes_per_pos + PREFETCH_CHUNK - 1) / PREFETCH_CHUNK;
    const size_t total = chunks_per_pos * static_cast<size_t>(num_pos);
    for (size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < total;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const size_t j = i / num_pos;
        const size_t pos = i - j * num_pos;
        const size_t off = j * PREFETCH_CHUNK;
        const size_t left = bytes_per_pos - off;
        bulk_prefetch_l2(base + pos * pos_stride + off, static_cast<uint32_t>(left < PREFETCH_CHUNK ? left : PREFETCH_CHUNK));
    }
}

// The side stream and the events of sdwino_conv3x3_sequence, one set per device, made on first use.
struct SequenceResources {
    cudaStream_t side = nullptr;
    std::vector<cudaEvent_t> events;
};
SequenceResources g_seq[STATIC_MAX_DEVICES_HOST];
std::mutex g_seq_mutex;

bool layer_ok(const sdwino_layer& l) {
    return l.x && l.wT && l.y && l.N > 0 && l.C > 0 && l.H > 0 && l.W > 0 && l.K > 0;
}
}  // namespace

extern "C" {

size_t sdwino_workspace_bytes_sequence(const sdwino_layer* layers, int n) {
    if (!layers || n <= 0) return 0;
    size_t need = 0;
    for (int i = 0; i < n; ++i) {
        const sdwino_layer& l = layers[i];
        const size_t b = sdwino_workspace_bytes(l.N, l.C, l.H, l.W, l.K, l.tile);
        if (b == 0) return 0;
        need = std::max(need, b);
    }
    return need;
}

int sdwino_conv3x3_sequence(const sdwino_layer* layers, int n, void* workspace, size_t workspace_bytes,
                            size_t prefetch_bytes, void* stream) {
    if (!layers || n <= 0) return SDWINO_ERR_INVALID_ARG;
    // everything is checked before the first launch: a sequence runs whole or not at all
    for (int i = 0; i < n; ++i) {
        const sdwino_layer& l = layers[i];
        if (!layer_ok(l)) return SDWINO_ERR_INVALID_ARG;
        if (l.tile != 1 && l.tile != 2 && l.tile != 4) return SDWINO_ERR_UNSUPPORTED;
        Plan pl;
        if (!make_plan(l.N, l.C, l.H, l.W, l.K, l.tile, &pl)) return SDWINO_ERR_INVALID_ARG;
        if (!aligned(l.x, 2) || !aligned(l.y, 2) || (l.bias && !aligned(l.bias, 2)) || !aligned(l.wT, WS_ALIGN))
            return SDWINO_ERR_MISALIGNED;
        if (!workspace || tiles_per_pass(pl, workspace_bytes) < GEMM_BLOCK_P) return SDWINO_ERR_WORKSPACE;
    }
    if (!aligned(workspace, WS_ALIGN)) return SDWINO_ERR_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool prefetch = prefetch_bytes >= PREFETCH_CHUNK && n > 1;
    SequenceResources* res = nullptr;
    std::unique_lock<std::mutex> lock(g_seq_mutex, std::defer_lock);
    if (prefetch) {
        // one sequence at a time enqueues through the side stream (the calls only enqueue; the work itself overlaps)
        lock.lock();
        const int dev = current_device();
        if (dev < 0 || dev >= STATIC_MAX_DEVICES_HOST) return err_cuda(__LINE__);
        res = &g_seq[dev];
        if (!res->side) {
            int lo = 0, hi = 0;
            if (cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess) return err_cuda(__LINE__);
            if (cudaStreamCreateWithPriority(&res->side, cudaStreamNonBlocking, lo) != cudaSuccess) return err_cuda(__LINE__);
        }
        while (static_cast<int>(res->events.size()) < n + 1) {
            cudaEvent_t e;
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return err_cuda(__LINE__);
            res->events.push_back(e);
        }
    }
    bool forked = false;
    for (int i = 0; i < n; ++i) {
        if (prefetch && i + 1 < n) {
            // While layer i computes, the first bytes of every position of layer i + 1's filters travel to L2:
            // filters never depend on activations.  The side stream waits for what precedes layer i in `stream`.
            const sdwino_layer& nx = layers[i + 1];
            const size_t a2 = static_cast<size_t>(nx.tile + 2) * (nx.tile + 2);
            const size_t per_pos = static_cast<size_t>((nx.K + 15) / 16) * ((nx.C + 63) / 64) * 1024 * sizeof(__half);
            size_t want = std::min(per_pos, prefetch_bytes / a2) / PREFETCH_CHUNK * PREFETCH_CHUNK;
            if (want * a2 >= (1u << 20)) {     // small filters are not worth a launch
                if (cudaEventRecord(res->events[i], st) != cudaSuccess) return err_cuda(__LINE__);
                if (cudaStreamWaitEvent(res->side, res->events[i], 0) != cudaSuccess) return err_cuda(__LINE__);
                const size_t chunks = want / PREFETCH_CHUNK * a2;
                const unsigned blocks = static_cast<unsigned>(std::min<size_t>((chunks + 127) / 128, 64));
                filter_prefetch_kernel<<<blocks, 128, 0, res->side>>>(static_cast<const uint8_t*>(wt_filters_of(nx.wT)), per_pos,
                                                                      want, static_cast<int>(a2));
                if (cudaGetLastError() != cudaSuccess) return err_cuda(__LINE__);
                g_launches.fetch_add(1);
                forked = true;
            }
        }
        const sdwino_layer& l = layers[i];
        const int rc = conv_impl(l.x, l.wT, l.bias, l.y, l.N, l.C, l.H, l.W, l.K, l.tile, workspace, workspace_bytes, st);
        if (rc != SDWINO_OK) {
            if (forked) {   // rejoin before reporting, so that a stream capture stays valid
                if (cudaEventRecord(res->events[n], res->side) == cudaSuccess) cudaStreamWaitEvent(st, res->events[n], 0);
            }
            return rc;
        }
    }
    if (forked) {
        // the side stream joins `stream` again (a no-op in time: the prefetch kernels ended long ago)
        if (cudaEventRecord(res->events[n], res->side) != cudaSuccess) return err_cuda(__LINE__);
        if (cudaStreamWaitEvent(st, res->events[n], 0) != cudaSuccess) return err_cuda(__LINE__);
    }
    return SDWINO_OK;
}

int sdwino_profile_enable(int mode) {
    if (mode < 0 || mode > 2) return SDWINO_ERR_INVALID_ARG;
    g_profile.store(mode);
    return SDWINO_OK;
}

int sdwino_profile_records(int* kinds, float* ms, int capacity, int keep) {
    std::lock_guard<std::mutex> lock(g_mutex);
    int n = 0;
    for (const ProfRecord& r : g_prof_records) {
        float t = 0.f;
        if (cudaEventSynchronize(r.end) != cudaSuccess || cudaEventElapsedTime(&t, r.beg, r.end) != cudaSuccess) t = -1.f;
        if (n < capacity) {
            if (kinds) kinds[n] = r.kind;
            if (ms) ms[n] = t;
        }
        ++n;
        if (!keep) {
            g_event_pool.push_back(r.beg);
            g_event_pool.push_back(r.end);
        }
    }
    if (!keep) g_prof_records.clear();
    return n;
}

int sdwino_profile_collect(double* ms_by_kind, unsigned long long* launches_by_kind) {
    std::lock_guard<std::mutex> lock(g_mutex);
    int rc = SDWINO_OK;
    for (int k = 0; k < KIND_COUNT; ++k) {
        if (ms_by_kind) ms_by_kind[k] = 0.0;
        if (launches_by_kind) launches_by_kind[k] = 0;
    }
    for (const ProfRecord& r : g_prof_records) {
        float ms = 0.f;
        if (cudaEventSynchronize(r.end) != cudaSuccess || cudaEventElapsedTime(&ms, r.beg, r.end) != cudaSuccess) {
            rc = SDWINO_ERR_CUDA;
        } else {
            if (ms_by_kind) ms_by_kind[r.kind] += ms;
            if (launches_by_kind) launches_by_kind[r.kind] += 1;
        }
        g_event_pool.push_back(r.beg);
        g_event_pool.push_back(r.end);
    }
    g_prof_records.clear();
    return rc;
}

}  // extern "C"
