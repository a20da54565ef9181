// Steps (i) and (iii) of Section "Techniques": filter preprocess U = G g G^T, activation
// preprocess V = B^T d B on overlapping (m+2)x(m+2) windows, and postprocess
// Y = A^T M A followed by bias add, rounding to fp16 and a store masked at the image edge.
// These kernels are bandwidth-bound: one thread per (channel, tile), consecutive threads on
// consecutive tiles so that every global access of a warp is contiguous.
//
// The paper prints no matrices; these are the Toom-Cook matrices of the construction it cites.
// F(2x2,3x3) uses the points {0, 1, -1, inf}; F(4x4,3x3) uses {0, 3/4, -3/4, 3/2, -3/2, inf},
// whose B^T and A^T entries are dyadic and whose fp16 error is about a third of that of the
// integer points {0, +-1, +-2, inf}.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

#include "ptx.cuh"

namespace sdw {

template <int M> struct Wino;

// F(1x1,3x3): the degenerate member of the family, i.e. the direct convolution.  A tile is one output pixel, the
// nine transform positions are the nine filter taps, all three matrices are trivial (identity, identity, a row of
// ones): the same three steps then compute y = sum over taps of (per-tap GEMM over the channels), which is the
// convolution evaluated as nine shifted matrix products.  It also takes a stride (the input window of output pixel
// t starts at stride * t - 1), which Winograd's overlapping tiles cannot.
template <> struct Wino<1> {
    static constexpr int A = 3;
    struct Bt {
        __host__ __device__ constexpr float operator()(int i, int j) const { return i == j ? 1.f : 0.f; }
    };
    struct G {
        __host__ __device__ constexpr float operator()(int i, int j) const { return i == j ? 1.f : 0.f; }
    };
    struct At {
        __host__ __device__ constexpr float operator()(int, int) const { return 1.f; }
    };
};

template <> struct Wino<2> {
    static constexpr int A = 4;
    struct Bt {
        __host__ __device__ constexpr float operator()(int i, int j) const {
            constexpr float m[4][4] = {{1, 0, -1, 0}, {0, 1, 1, 0}, {0, -1, 1, 0}, {0, 1, 0, -1}};
            return m[i][j];
        }
    };
    struct G {
        __host__ __device__ constexpr float operator()(int i, int j) const {
            constexpr float m[4][3] = {{1, 0, 0}, {0.5f, 0.5f, 0.5f}, {0.5f, -0.5f, 0.5f}, {0, 0, 1}};
            return m[i][j];
        }
    };
    struct At {
        __host__ __device__ constexpr float operator()(int i, int j) const {
            constexpr float m[2][4] = {{1, 1, 1, 0}, {0, 1, -1, -1}};
            return m[i][j];
        }
    };
};

template <> struct Wino<4> {
    static constexpr int A = 6;
    struct Bt {
        __host__ __device__ constexpr float operator()(int i, int j) const {
            constexpr float m[6][6] = {{1.265625f, 0, -2.8125f, 0, 1, 0},    {0, -1.6875f, -2.25f, 0.75f, 1, 0},
                                       {0, 1.6875f, -2.25f, -0.75f, 1, 0},   {0, -0.84375f, -0.5625f, 1.5f, 1, 0},
                                       {0, 0.84375f, -0.5625f, -1.5f, 1, 0}, {0, 1.265625f, 0, -2.8125f, 0, 1}};
            return m[i][j];
        }
    };
    struct G {
        __host__ __device__ constexpr float operator()(int i, int j) const {
            constexpr float m[6][3] = {{64.f / 81.f, 0, 0},
                                       {-128.f / 243.f, -32.f / 81.f, -8.f / 27.f},
                                       {-128.f / 243.f, 32.f / 81.f, -8.f / 27.f},
                                       {32.f / 243.f, 16.f / 81.f, 8.f / 27.f},
                                       {32.f / 243.f, -16.f / 81.f, 8.f / 27.f},
                                       {0, 0, 1}};
            return m[i][j];
        }
    };
    struct At {
        __host__ __device__ constexpr float operator()(int i, int j) const {
            constexpr float m[4][6] = {{1, 1, 1, 1, 1, 0},
                                       {0, 0.75f, -0.75f, 1.5f, -1.5f, 0},
                                       {0, 0.5625f, 0.5625f, 2.25f, 2.25f, 0},
                                       {0, 0.421875f, -0.421875f, 3.375f, -3.375f, 1}};
            return m[i][j];
        }
    };
};

// Optional bias (NULL = 0).  A plain load under the null check: a read-only-path load (__ldg) may be
// hoisted above the check by the compiler, and then faults on the null pointer.
__device__ __forceinline__ float load_bias(const __half* bias, int k) {
    float b = 0.f;
    if (bias != nullptr) b = __half2float(bias[k]);
    return b;
}
__device__ __forceinline__ float load_bias(const float* bias, int k) {
    float b = 0.f;
    if (bias != nullptr) b = bias[k];
    return b;
}

// The fp32 interface (x, w, bias, y in fp32): the kernels below take the element type of the tensors they read
// from or write to the caller as a template argument.  Everything between the transforms is the same: U, V and M
// are fp16 (the 11-bit significand of the TF32 tensor-core format), accumulation is fp32.
__device__ __forceinline__ float to_f32(__half v) { return __half2float(v); }
__device__ __forceinline__ float to_f32(float v) { return v; }

// Range-safe fp32 calls: x is multiplied by 2^-e on its way into V and the result by 2^e on its way out of M, with e
// chosen from max|x| so that the scaled activations peak near 64: V and M are fp16 and would overflow (or lose their
// small values) otherwise.  Powers of two: the scaling itself rounds nothing.
__device__ __forceinline__ int range_exponent(const float* amax) {
    if (amax == nullptr) return 0;
    const float a = *amax;
    if (!(a > 0.f) || a > 3.0e38f) return 0;
    return ilogbf(a) - 6;
}
// max|x| over a tensor, as the bits of a non-negative float (which order like unsigned integers); *out starts at 0.
__global__ void __launch_bounds__(256)
absmax_kernel(const float* __restrict__ x, long long n, unsigned int* __restrict__ out) {
    pdl_wait();
    pdl_launch_dependents();
    float m = 0.f;
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if ((reinterpret_cast<uintptr_t>(x) & 15) == 0) {
        const long long n4 = n >> 2;
        for (long long j = i; j < n4; j += stride) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(x) + j);
            m = fmaxf(fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
        }
        for (long long j = (n4 << 2) + i; j < n; j += stride) m = fmaxf(m, fabsf(__ldg(x + j)));
    } else {
        for (long long j = i; j < n; j += stride) m = fmaxf(m, fabsf(__ldg(x + j)));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m > 0.f) atomicMax(out, __float_as_uint(m));
}

// out[i] = sum_j coef[i][j] * in[j] with compile-time coefficients: zero terms vanish and
// unit terms become adds once the loops are unrolled.
template <int R, int Cn, typename MatT>
__device__ __forceinline__ void mat_apply(MatT coef, const float (&in)[Cn], float (&out)[R]) {
#pragma unroll
    for (int i = 0; i < R; ++i) {
        float acc = 0.f;
        bool first = true;
#pragma unroll
        for (int j = 0; j < Cn; ++j) {
            const float cf = coef(i, j);
            if (cf != 0.f) {
                if (first) { acc = cf * in[j]; first = false; }
                else acc = fmaf(cf, in[j], acc);
            }
        }
        out[i] = acc;
    }
}

// ---------------------------------------------------------------------------------------
// Header of a transformed filter: the first 1024 bytes of wT, written by the filter transform.  Every kernel
// that reads U first compares it with the layer it was launched for: a buffer that was transformed for another
// tile size or other channel counts (it may be SMALLER than the one expected) is never read: the kernel records
// SDWINO_ERR_INVALID_ARG in the device status word and returns.
// ---------------------------------------------------------------------------------------
constexpr uint32_t WT_MAGIC = 0x55574453u;   // "SDWU"
constexpr int WT_HEADER_BYTES = 1024;
__device__ __forceinline__ bool wt_header_ok(const uint32_t* __restrict__ header, int K, int C, int tile,
                                             int* status_word) {
    const uint4 h = *reinterpret_cast<const uint4*>(header);   // plain load: written by an earlier kernel
    const bool ok = h.x == WT_MAGIC && h.y == static_cast<uint32_t>(K) && h.z == static_cast<uint32_t>(C) &&
                    h.w == static_cast<uint32_t>(tile);
    if (!ok && threadIdx.x == 0) atomicCAS(status_word, 0, 1 | (9 << 8));   // 1 = SDWINO_ERR_INVALID_ARG
    return ok;
}
// The same check as one kernel argument (the output transform reads no filters, but leaves y alone when the GEMM
// before it refused to run).
struct WtCheck {
    const uint32_t* header;
    int K, C, tile;
    int* status_word;
};
__device__ __forceinline__ bool wt_check(const WtCheck& c) {
    return wt_header_ok(c.header, c.K, c.C, c.tile, c.status_word);
}

// ---------------------------------------------------------------------------------------
// Filter preprocess.  U is stored in blocks of 16 output channels x 64 input channels,
//   U[a*a][Cb][Kb][16][64]   (Kb = ceil(K/16), Cb = ceil(C/64), zeros in the padding),
// with the blocks of consecutive output channels next to each other, so that the [n_tile k][64 c]
// operand box of one GEMM pipeline stage is ONE contiguous piece of n_tile/16 x 2 KB of DRAM instead of
// n_tile separate 128-byte rows (the weights are the one operand that is streamed from HBM).  One thread per (k, pair of c) of the padded plane.
// Writes all a*a positions.
// ---------------------------------------------------------------------------------------
template <int M, typename WT = __half>
__global__ void __launch_bounds__(128)
filter_transform_kernel(const WT* __restrict__ w, uint32_t* __restrict__ header, __half* __restrict__ U, int K,
                        int C, int Kb, int Cb) {
    using Wm = Wino<M>;
    constexpr int A = Wm::A;
    pdl_launch_dependents();
    pdl_wait();
    // two neighbouring input channels per thread: 4-byte stores (four per thread measured slower again)
    const int c = (blockIdx.x * blockDim.x + threadIdx.x) * 2;
    // one row of blocks per output channel; more than 65535 rows continue along grid.z
    const int k = static_cast<int>(blockIdx.z * gridDim.y + blockIdx.y);
    if (k >= Kb * 16) return;
    if (blockIdx.x == 0 && k == 0 && threadIdx.x == 0)
        *reinterpret_cast<uint4*>(header) = make_uint4(WT_MAGIC, static_cast<uint32_t>(K), static_cast<uint32_t>(C),
                                                       static_cast<uint32_t>(M));
    if (c >= Cb * 64) return;
    float u[2][A][A];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        float g[3][3];
        const bool live = (c + h < C) && (k < K);
#pragma unroll
        for (int r = 0; r < 3; ++r)
#pragma unroll
            for (int s = 0; s < 3; ++s)
                g[r][s] = live ? to_f32(w[(static_cast<size_t>(k) * C + c + h) * 9 + r * 3 + s]) : 0.f;
        // t = G g  (A x 3), u = t G^T (A x A)
        float t[A][3];
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            float col[3] = {g[0][s], g[1][s], g[2][s]};
            float o[A];
            mat_apply<A, 3>(typename Wm::G{}, col, o);
#pragma unroll
            for (int i = 0; i < A; ++i) t[i][s] = o[i];
        }
#pragma unroll
        for (int i = 0; i < A; ++i) mat_apply<A, 3>(typename Wm::G{}, t[i], u[h][i]);
    }
    const size_t plane = static_cast<size_t>(Kb) * Cb * 1024;   // one position: Kb x Cb blocks of 16 x 64
    __half* dst = U + ((static_cast<size_t>(c >> 6) * Kb + (k >> 4)) * 16 + (k & 15)) * 64 + (c & 63);
#pragma unroll
    for (int i = 0; i < A; ++i)
#pragma unroll
        for (int j = 0; j < A; ++j)
            *reinterpret_cast<__half2*>(dst + (i * A + j) * plane) = __floats2half2_rn(u[0][i][j], u[1][i][j]);
}

// ---------------------------------------------------------------------------------------
// 8-bit transformed filter (the quantised operators of Section "Evaluation", "Operator Support").  Input: the fp16
// blocked filter U[a*a][Cb][Kb][16][64] made by filter_transform_kernel.  Output, same blocking: one byte q + 128 per
// element with q = round(U / s) in [-127, 127] (fp32 quotient, ties to even) and s = max|U| / 127 taken over the row
// U[pos][k][:] (one transform position, one output channel, all input channels); the scales follow as
// S[a*a][Kb * 16] fp32.  The header keeps magic, K and C and marks the format in its tile word.
// One block of 128 threads per (position, block of 16 output channels): 8 threads per row.
// ---------------------------------------------------------------------------------------
constexpr uint32_t WT_Q8_FLAG = 0x100u;   // or-ed into the header's tile word
__global__ void __launch_bounds__(128)
filter_quantize_kernel(const uint32_t* __restrict__ header16, const __half* __restrict__ U, uint32_t* __restrict__ header8,
                       uint8_t* __restrict__ Uq, float* __restrict__ S, int K, int C, int tile, int Kb, int Cb,
                       int* __restrict__ status_word) {
    pdl_launch_dependents();
    pdl_wait();
    if (!wt_header_ok(header16, K, C, tile, status_word)) return;
    const int pos = blockIdx.x / Kb, kb = blockIdx.x - pos * Kb;
    const int row = threadIdx.x >> 3, sub = threadIdx.x & 7;
    if (blockIdx.x == 0 && threadIdx.x == 0)
        *reinterpret_cast<uint4*>(header8) = make_uint4(WT_MAGIC, static_cast<uint32_t>(K), static_cast<uint32_t>(C),
                                                        static_cast<uint32_t>(tile) | WT_Q8_FLAG);
    const size_t blk0 = (static_cast<size_t>(pos) * Cb * Kb + kb) * 1024 + row * 64 + sub * 8;   // cb = 0
    const size_t cb_step = static_cast<size_t>(Kb) * 1024;
    float amax = 0.f;
    for (int cb = 0; cb < Cb; ++cb) {
        const uint4 v = *reinterpret_cast<const uint4*>(U + blk0 + cb * cb_step);
        const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&wds[i]));
            amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
        }
    }
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
    amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 4));
    const float sc = amax > 0.f ? __fdiv_rn(amax, 127.f) : 1.f;
    if (sub == 0) S[static_cast<size_t>(pos) * Kb * 16 + kb * 16 + row] = sc;
    for (int cb = 0; cb < Cb; ++cb) {
        const uint4 v = *reinterpret_cast<const uint4*>(U + blk0 + cb * cb_step);
        const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
        uint32_t out[2] = {0u, 0u};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&wds[i]));
            const int q0 = static_cast<int>(fminf(fmaxf(rintf(__fdiv_rn(f.x, sc)), -127.f), 127.f)) + 128;
            const int q1 = static_cast<int>(fminf(fmaxf(rintf(__fdiv_rn(f.y, sc)), -127.f), 127.f)) + 128;
            out[i >> 1] |= (static_cast<uint32_t>(q0) | (static_cast<uint32_t>(q1) << 8)) << ((i & 1) * 16);
        }
        *reinterpret_cast<uint2*>(Uq + blk0 + cb * cb_step) = make_uint2(out[0], out[1]);
    }
}

// ---------------------------------------------------------------------------------------
// Tile index arithmetic shared by both activation-side kernels.  Tile p (global index over
// the whole batch) belongs to image n = p / (TH*TW), tile row th and tile column tw; its
// input window starts at pixel (m*th - 1, m*tw - 1) and its outputs at (m*th, m*tw).
// ---------------------------------------------------------------------------------------
// Division by a launch-invariant 32-bit divisor as multiply-high and shift (a 64-bit or even 32-bit integer
// division costs on the order of a hundred instructions per thread; the index decode of a transform thread
// needs three).  For 0 <= n < 2^31 and d >= 2: with L = ceil(log2 d) and mul = ceil(2^(31+L) / d) < 2^32,
// floor(n / d) = (n * mul) >> (31 + L), because mul * d = 2^(31+L) + e with 0 <= e < d <= 2^L makes the
// excess n * e / (d * 2^(31+L)) smaller than 1 / d.
struct FastDiv {
    uint32_t d, mul, shr;
};
inline FastDiv make_fastdiv(uint32_t d) {
    FastDiv f{d, 0u, 0u};
    if (d > 1) {
        uint32_t L = 0;
        while ((1ull << L) < d) ++L;
        f.mul = static_cast<uint32_t>(((1ull << (31 + L)) + d - 1) / d);
        f.shr = L - 1;
    }
    return f;
}
__device__ __forceinline__ uint32_t fast_div(uint32_t n, const FastDiv& f) {
    return f.d == 1 ? n : (__umulhi(n, f.mul) >> f.shr);
}

struct TileGeom {
    int H, W, TH, TW;
    long long P;  // N*TH*TW, below 2^31
    FastDiv tw_div, th_div;
    int stride;   // direct convolution (tile 1) only: distance of the input windows of neighbouring output pixels
};
inline TileGeom make_geom(int H, int W, int TH, int TW, long long P, int stride = 1) {
    return TileGeom{H, W, TH, TW, P, make_fastdiv(static_cast<uint32_t>(TW)), make_fastdiv(static_cast<uint32_t>(TH)), stride};
}
// tile p -> image n, tile row th, tile column tw
__device__ __forceinline__ void decode_tile(const TileGeom& geo, long long p, long long& n, int& th, int& tw) {
    const uint32_t pu = static_cast<uint32_t>(p);
    const uint32_t row = fast_div(pu, geo.tw_div);
    const uint32_t img = fast_div(row, geo.th_div);
    tw = static_cast<int>(pu - row * static_cast<uint32_t>(geo.TW));
    th = static_cast<int>(row - img * static_cast<uint32_t>(geo.TH));
    n = img;
}

// Activation preprocess.  V layout: [a*a][C][Pstride] with the chunk-local tile index
// (p - p_begin) contiguous.  Threads past the last tile write zeros so that the GEMM reads
// defined data.
template <int M, typename XT = __half>
__global__ void __launch_bounds__(128)
input_transform_kernel(const XT* __restrict__ x, __half* __restrict__ V, TileGeom geo, int C, long long p_begin,
                       int p_count, long long Pstride, const float* __restrict__ amax) {
    using Wm = Wino<M>;
    constexpr int A = Wm::A;
    // Wait first, release the GEMM second: once the GEMM runs, everything before this kernel has completed,
    // which is what lets it fetch its filters (written at the latest by the kernel before this one) early.
    pdl_wait();
    pdl_launch_dependents();
    const int pl = blockIdx.x * blockDim.x + threadIdx.x;  // chunk-local tile
    const int c = static_cast<int>(blockIdx.z * gridDim.y + blockIdx.y);   // grid.z continues grid.y past 65535
    if (pl >= p_count || c >= C) return;
    const long long p = p_begin + pl;
    float d[A][A];
    [[maybe_unused]] float xs = 1.f;
    if constexpr (sizeof(XT) == 4) xs = scalbnf(1.f, -range_exponent(amax));
    if (p < geo.P) {
        int tw, th;
        long long n;
        decode_tile(geo, p, n, th, tw);
        const XT* img = x + (n * C + c) * static_cast<long long>(geo.H) * geo.W;
        const int step = M == 1 ? geo.stride : M;          // distance of neighbouring windows
        const int i0 = step * th - 1, j0 = step * tw - 1;
#pragma unroll
        for (int r = 0; r < A; ++r) {
            const int i = i0 + r;
            const bool rin = (i >= 0) && (i < geo.H);
#pragma unroll
            for (int s = 0; s < A; ++s) {
                const int j = j0 + s;
                d[r][s] = (rin && j >= 0 && j < geo.W) ? to_f32(__ldg(img + static_cast<long long>(i) * geo.W + j))
                                                        : 0.f;
                if constexpr (sizeof(XT) == 4) d[r][s] *= xs;
            }
        }
    } else {
#pragma unroll
        for (int r = 0; r < A; ++r)
#pragma unroll
            for (int s = 0; s < A; ++s) d[r][s] = 0.f;
    }
    // t = B^T d (column by column), v = t B (row by row)
    float t[A][A];
#pragma unroll
    for (int s = 0; s < A; ++s) {
        float col[A], o[A];
#pragma unroll
        for (int r = 0; r < A; ++r) col[r] = d[r][s];
        mat_apply<A, A>(typename Wm::Bt{}, col, o);
#pragma unroll
        for (int r = 0; r < A; ++r) t[r][s] = o[r];
    }
    const long long plane = static_cast<long long>(C) * Pstride;
    __half* dst = V + static_cast<long long>(c) * Pstride + pl;
#pragma unroll
    for (int r = 0; r < A; ++r) {
        float o[A];
        mat_apply<A, A>(typename Wm::Bt{}, t[r], o);
#pragma unroll
        for (int s = 0; s < A; ++s) dst[(r * A + s) * plane] = __float2half_rn(o[s]);
    }
}

// What follows the postprocess in the same kernel: y = act(A^T M A + bias + residual).  The paper's operator ends at
// the convolution; the residual sum and the SiLU of the ResNet blocks around it are memory-bound element-wise
// passes over y that cost nothing extra here.  residual: fp16 [N][K][H][W] or null (may be y itself);
// act: 0 none, 1 SiLU z / (1 + exp(-z)).
struct Epilogue {
    const void* residual;   // element type of y
    int act;
    const float* amax;      // fp32 interface, range-safe calls: device word holding max|x| (null: no scaling)
};
__device__ __forceinline__ float epilogue_act(float v, int act) {
    return act == 1 ? __fdividef(v, 1.f + __expf(-v)) : v;   // fast division: 2 ulp, far below the fp16 rounding that follows
}

// Postprocess + bias + cast + masked store.  Mws layout: [a*a][K][Pstride]; y is NCHW.
template <int M, typename YT = __half>
__global__ void __launch_bounds__(128)
output_transform_kernel(const __half* __restrict__ Mws, const YT* __restrict__ bias, YT* __restrict__ y,
                        TileGeom geo, int K, long long p_begin, int p_count, long long Pstride, WtCheck chk,
                        Epilogue ep) {
    using Wm = Wino<M>;
    constexpr int A = Wm::A;
    pdl_launch_dependents();
    // the header is older than the activation transform two kernels back, which waited for everything before
    // it: reading it before this kernel's own wait takes the load off the critical path
    const bool wt_ok = wt_check(chk);
    pdl_wait();
    if (!wt_ok) return;
    const int pl = blockIdx.x * blockDim.x + threadIdx.x;
    const int k = static_cast<int>(blockIdx.z * gridDim.y + blockIdx.y);   // grid.z continues grid.y past 65535
    if (pl >= p_count || k >= K) return;
    const long long p = p_begin + pl;
    if (p >= geo.P) return;
    const long long plane = static_cast<long long>(K) * Pstride;
    const __half* src = Mws + static_cast<long long>(k) * Pstride + pl;
    float mm[A][A];
#pragma unroll
    for (int r = 0; r < A; ++r)
#pragma unroll
        for (int s = 0; s < A; ++s) mm[r][s] = __half2float(__ldg(src + (r * A + s) * plane));
    // t = A^T mm (M x A), Y = t A (M x M)
    float t[M][A];
#pragma unroll
    for (int s = 0; s < A; ++s) {
        float col[A], o[M];
#pragma unroll
        for (int r = 0; r < A; ++r) col[r] = mm[r][s];
        mat_apply<M, A>(typename Wm::At{}, col, o);
#pragma unroll
        for (int i = 0; i < M; ++i) t[i][s] = o[i];
    }
    int tw, th;
    long long n;
    decode_tile(geo, p, n, th, tw);
    const float b = load_bias(bias, k);
    [[maybe_unused]] float ys = 1.f;
    if constexpr (sizeof(YT) == 4) ys = scalbnf(1.f, range_exponent(ep.amax));
    YT* img = y + (n * K + k) * static_cast<long long>(geo.H) * geo.W;
    const int i0 = M * th, j0 = M * tw;
    const bool vec_ok = ((geo.W & 1) == 0) && ((reinterpret_cast<uintptr_t>(y) & 3) == 0);
#pragma unroll
    for (int i = 0; i < M; ++i) {
        float o[M];
        mat_apply<M, A>(typename Wm::At{}, t[i], o);
        const int oi = i0 + i;
        if (oi >= geo.H) continue;
        if constexpr (sizeof(YT) == 4) {   // fp32 output: no residual, no activation, no rounding
            float* rowf = reinterpret_cast<float*>(img) + static_cast<long long>(oi) * geo.W + j0;
            const float* resf = ep.residual ? static_cast<const float*>(ep.residual) + (rowf - reinterpret_cast<float*>(y))
                                            : nullptr;
#pragma unroll
            for (int j = 0; j < M; ++j)
                if (j0 + j < geo.W) {
                    float v = fmaf(o[j], ys, b);
                    if (resf) v += resf[j];
                    rowf[j] = epilogue_act(v, ep.act);
                }
            continue;
        } else {
        __half* rowp = img + static_cast<long long>(oi) * geo.W + j0;
        const __half* resp = ep.residual ? static_cast<const __half*>(ep.residual) + (rowp - y) : nullptr;
        if constexpr (M == 1) {   // one output pixel per tile
            float v0 = o[0] + b;
            if (resp) v0 += __half2float(resp[0]);
            rowp[0] = __float2half_rn(epilogue_act(v0, ep.act));
        } else {
#pragma unroll
        for (int j = 0; j < M; j += 2) {
            float v0 = o[j] + b, v1 = o[j + 1] + b;
            if (resp) {
                if (j0 + j < geo.W) v0 += __half2float(resp[j]);
                if (j0 + j + 1 < geo.W) v1 += __half2float(resp[j + 1]);
            }
            const __half h0 = __float2half_rn(epilogue_act(v0, ep.act)), h1 = __float2half_rn(epilogue_act(v1, ep.act));
            if (vec_ok && (j0 + j + 1 < geo.W)) {
                *reinterpret_cast<__half2*>(rowp + j) = __halves2half2(h0, h1);
            } else {
                if (j0 + j < geo.W) rowp[j] = h0;
                if (j0 + j + 1 < geo.W) rowp[j + 1] = h1;
            }
        }
        }   // M > 1
        }   // fp16 output
    }
}


// ---------------------------------------------------------------------------------------
// Vector variants for image widths that are multiples of 8 (every SD layer of 16 pixels or more):
// a thread owns TPT consecutive tiles of one tile row (m * TPT = 8 pixels), so each input or
// output row segment is one aligned 16-byte access, the halo pixels left and right of it are two
// scalar loads, and each transform position is stored / loaded as TPT packed fp16 values.
// Arithmetic is fp32 as in the scalar kernels (the row and column passes run in the other order).
// Requirements (checked by the host): W % 8 == 0, x / y 16-byte aligned, m * TPT == 8.
// ---------------------------------------------------------------------------------------
template <int N> struct PackedHalf;
template <> struct PackedHalf<2> { using type = uint32_t; };
template <> struct PackedHalf<4> { using type = uint2; };

__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void unpack2(uint32_t v, float& a, float& b) {
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&v));
    a = f.x;
    b = f.y;
}

// ---------------------------------------------------------------------------------------
// F(4x4,3x3) in packed fp32 (sm_100 has two-wide fp32 FMA/ADD/MUL): the two halves of a float2 are the
// two tiles a thread owns.  The rows of B^T and A^T for the points {0, +-3/4, +-3/2, inf} come in +- pairs,
// so each pair shares its even and its odd part: 14 packed operations for B^T d (6 -> 6) and 12 for
// A^T m (6 -> 4), against 22 and 18 scalar ones per tile when the matrix is applied row by row.  The vector
// transform kernels of F4 are bound by instruction issue, not by memory (ncu: 69 % issue-active).
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float2 f2s(float a) { return make_float2(a, a); }

__device__ __forceinline__ void bt4_packed(const float2 (&d)[6], float2 (&o)[6]) {
    const float2 e1 = __ffma2_rn(f2s(-2.25f), d[2], d[4]);
    const float2 o1 = __ffma2_rn(f2s(0.75f), d[3], __fmul2_rn(f2s(-1.6875f), d[1]));
    const float2 e2 = __ffma2_rn(f2s(-0.5625f), d[2], d[4]);
    const float2 o2 = __ffma2_rn(f2s(1.5f), d[3], __fmul2_rn(f2s(-0.84375f), d[1]));
    o[0] = __ffma2_rn(f2s(1.265625f), d[0], __ffma2_rn(f2s(-2.8125f), d[2], d[4]));
    o[1] = __fadd2_rn(e1, o1);
    o[2] = __ffma2_rn(f2s(-1.f), o1, e1);
    o[3] = __fadd2_rn(e2, o2);
    o[4] = __ffma2_rn(f2s(-1.f), o2, e2);
    o[5] = __ffma2_rn(f2s(1.265625f), d[1], __ffma2_rn(f2s(-2.8125f), d[3], d[5]));
}

__device__ __forceinline__ void at4_packed(const float2 (&m)[6], float2 (&o)[4]) {
    const float2 s1 = __fadd2_rn(m[1], m[2]);
    const float2 d1 = __ffma2_rn(f2s(-1.f), m[2], m[1]);
    const float2 s2 = __fadd2_rn(m[3], m[4]);
    const float2 d2 = __ffma2_rn(f2s(-1.f), m[4], m[3]);
    o[0] = __fadd2_rn(__fadd2_rn(m[0], s1), s2);
    o[1] = __ffma2_rn(f2s(1.5f), d2, __fmul2_rn(f2s(0.75f), d1));
    o[2] = __ffma2_rn(f2s(2.25f), s2, __fmul2_rn(f2s(0.5625f), s1));
    o[3] = __ffma2_rn(f2s(3.375f), d2, __ffma2_rn(f2s(0.421875f), d1, m[5]));
}

// One unit of the vector activation transform: channel c = idx / groups, TPT tiles of one tile row.  The flat
// index over (channel, group of TPT tiles) keeps blocks full when a pass has few tiles.  Called by the kernel
// below with one unit per thread.
template <int M, int TPT, typename XT = __half>
__device__ __forceinline__ void input_unit_vec(const XT* __restrict__ x, __half* __restrict__ V, const TileGeom& geo,
                                               int C, long long p_begin, const FastDiv& gdiv, long long Pstride,
                                               uint32_t idx, const float* __restrict__ amax = nullptr) {
    using Wm = Wino<M>;
    constexpr int A = Wm::A;
    static_assert(M * TPT == 8, "one 16-byte row segment per thread");
    const int c = static_cast<int>(fast_div(idx, gdiv));           // gdiv.d = p_count / TPT groups per channel
    if (c >= C) return;
    const int pl = static_cast<int>(idx - static_cast<uint32_t>(c) * gdiv.d) * TPT;  // first chunk-local tile of this thread
    const long long p = p_begin + pl;
    static_assert(M == 2, "F(4x4) has its own vector kernel (input_transform_f4_kernel)");
    {
    float e[A][TPT][A];  // rows transformed along the columns: e[r][t][nu] = sum_s Bt[nu][s] d[r][s]
    int tw = 0, th = 0;
    long long n = 0;
    if (p < geo.P) decode_tile(geo, p, n, th, tw);
    // The index arithmetic above needs nothing from memory and runs while the preceding kernel drains.  Wait
    // first, release the GEMM second: once the GEMM runs, everything before this kernel has completed, which is
    // what lets it fetch its filters (written at the latest by the kernel before this one) early.
    pdl_wait();
    pdl_launch_dependents();
    [[maybe_unused]] float xs = 1.f;
    if constexpr (sizeof(XT) == 4) xs = scalbnf(1.f, -range_exponent(amax));
    if (p < geo.P) {
        const XT* img = x + (n * C + c) * static_cast<long long>(geo.H) * geo.W;
        const int i0 = M * th - 1, j0 = M * tw;
#pragma unroll
        for (int r = 0; r < A; ++r) {
            const int i = i0 + r;
            float row[10];
            if (i >= 0 && i < geo.H) {
                const XT* rp = img + static_cast<long long>(i) * geo.W + j0;
                if constexpr (sizeof(XT) == 4) {   // fp32 input: the eight pixels are two 16-byte loads
                    const float4 a = __ldg(reinterpret_cast<const float4*>(rp));
                    const float4 b = __ldg(reinterpret_cast<const float4*>(rp) + 1);
                    row[1] = a.x * xs; row[2] = a.y * xs; row[3] = a.z * xs; row[4] = a.w * xs;
                    row[5] = b.x * xs; row[6] = b.y * xs; row[7] = b.z * xs; row[8] = b.w * xs;
                } else {
                    const uint4 v = __ldg(reinterpret_cast<const uint4*>(rp));
                    unpack2(v.x, row[1], row[2]);
                    unpack2(v.y, row[3], row[4]);
                    unpack2(v.z, row[5], row[6]);
                    unpack2(v.w, row[7], row[8]);
                }
                row[0] = j0 > 0 ? to_f32(__ldg(rp - 1)) : 0.f;
                row[9] = j0 + 8 < geo.W ? to_f32(__ldg(rp + 8)) : 0.f;
                if constexpr (sizeof(XT) == 4) { row[0] *= xs; row[9] *= xs; }
            } else {
#pragma unroll
                for (int s = 0; s < 10; ++s) row[s] = 0.f;
            }
#pragma unroll
            for (int t = 0; t < TPT; ++t) {
                float d[A], o[A];
#pragma unroll
                for (int s = 0; s < A; ++s) d[s] = row[M * t + s];
                mat_apply<A, A>(typename Wm::Bt{}, d, o);
#pragma unroll
                for (int s = 0; s < A; ++s) e[r][t][s] = o[s];
            }
        }
    } else {
#pragma unroll
        for (int r = 0; r < A; ++r)
#pragma unroll
            for (int t = 0; t < TPT; ++t)
#pragma unroll
                for (int s = 0; s < A; ++s) e[r][t][s] = 0.f;
    }
    const long long plane = static_cast<long long>(C) * Pstride;
    __half* dst = V + static_cast<long long>(c) * Pstride + pl;
#pragma unroll
    for (int nu = 0; nu < A; ++nu) {
        float v[A][TPT];  // v[xi][t]
#pragma unroll
        for (int t = 0; t < TPT; ++t) {
            float col[A], o[A];
#pragma unroll
            for (int r = 0; r < A; ++r) col[r] = e[r][t][nu];
            mat_apply<A, A>(typename Wm::Bt{}, col, o);
#pragma unroll
            for (int xi = 0; xi < A; ++xi) v[xi][t] = o[xi];
        }
#pragma unroll
        for (int xi = 0; xi < A; ++xi) {
            __half* q = dst + (xi * A + nu) * plane;
            if constexpr (TPT == 4) {
                uint2 w;
                w.x = pack2(v[xi][0], v[xi][1]);
                w.y = pack2(v[xi][2], v[xi][3]);
                *reinterpret_cast<uint2*>(q) = w;
            } else {
                *reinterpret_cast<uint32_t*>(q) = pack2(v[xi][0], v[xi][1]);
            }
        }
    }
    }   // M != 4
}

template <int M, int TPT, typename XT = __half>
__global__ void __launch_bounds__(128)
input_transform_vec_kernel(const XT* __restrict__ x, __half* __restrict__ V, TileGeom geo, int C,
                           long long p_begin, FastDiv gdiv, long long Pstride, const float* __restrict__ amax) {
    input_unit_vec<M, TPT, XT>(x, V, geo, C, p_begin, gdiv, Pstride, blockIdx.x * blockDim.x + threadIdx.x, amax);   // < 2^31
}

// F(4x4,3x3) activation transform, vector path: a thread owns 2 tiles (8 pixels of a tile row) and CH consecutive
// channels.  Loads go into zero-initialised registers under precomputed border masks (no selects), and the
// (tile 0, tile 1) operand pairs of the packed arithmetic are cut straight out of the loaded halves with byte
// permutes.  The kernel is bound by instruction issue, so this is where its time goes: 3-10 % per layer over
// the generic vector kernel.  CH = 1 is what runs: with 2 or 4 channels per thread the per-thread set-up is
// amortised, but the serial load -> compute chain per channel and the lower thread count cost more (measured).
// EARLY (fp16 input): all six row segments of a channel are loaded before the first one is used, so that a thread
// pays one memory latency per channel instead of six: for callers that run few warps per SM.
template <int CH, typename XT = __half, bool PDL = true, bool EARLY = false>
__device__ __forceinline__ void input_unit_f4(const XT* __restrict__ x, __half* __restrict__ V, const TileGeom& geo,
                                              int C, long long p_begin, const FastDiv& gdiv, long long Pstride,
                                              uint32_t idx, const float* __restrict__ amax = nullptr) {
    constexpr int A = 6;
    const int cg = static_cast<int>(fast_div(idx, gdiv));          // gdiv.d = groups of 2 tiles in this pass
    const int c0 = cg * CH;
    if (c0 >= C) return;
    const int pl = static_cast<int>(idx - static_cast<uint32_t>(cg) * gdiv.d) * 2;
    const long long p = p_begin + pl;
    const long long hw = static_cast<long long>(geo.H) * geo.W;
    const bool valid = p < geo.P;
    int rowmask = 0;
    bool left_ok = false, right_ok = false;
    const XT* xp = x;
    if (valid) {
        int tw, th;
        long long n;
        decode_tile(geo, p, n, th, tw);
        const int i0 = 4 * th - 1, j0 = 4 * tw;
#pragma unroll
        for (int r = 0; r < A; ++r)
            if (i0 + r >= 0 && i0 + r < geo.H) rowmask |= 1 << r;
        left_ok = j0 > 0;
        right_ok = j0 + 8 < geo.W;
        xp = x + (n * C + c0) * hw + static_cast<long long>(i0) * geo.W + j0;
    }
    const long long plane = static_cast<long long>(C) * Pstride;
    __half* vp = V + static_cast<long long>(c0) * Pstride + pl;
    const int cend = (C - c0) < CH ? (C - c0) : CH;
    // The index arithmetic above needs nothing from memory and runs while the preceding kernel drains.  Wait
    // first, release the GEMM second: once the GEMM runs, everything before this kernel has completed, which is
    // what lets it fetch its filters (written at the latest by the kernel before this one) early.
    if constexpr (PDL) {   // (a caller inside a larger kernel orders its own reads)
        pdl_wait();
        pdl_launch_dependents();
    }
    [[maybe_unused]] float xs = 1.f;
    if constexpr (sizeof(XT) == 4) xs = scalbnf(1.f, -range_exponent(amax));
    for (int cc = 0; cc < cend; ++cc) {
        float2 e2[A][A];   // e2[r][nu]: rows transformed along the columns, (tile 0, tile 1)
        [[maybe_unused]] uint4 raw_v[A];
        [[maybe_unused]] uint32_t raw_l[A], raw_r[A];
        if constexpr (EARLY && sizeof(XT) == 2) {
#pragma unroll
            for (int r = 0; r < A; ++r) {
                raw_v[r] = make_uint4(0u, 0u, 0u, 0u);
                raw_l[r] = raw_r[r] = 0u;
                if ((rowmask >> r) & 1) {
                    const __half* rp = reinterpret_cast<const __half*>(xp) + r * geo.W;
                    raw_v[r] = __ldg(reinterpret_cast<const uint4*>(rp));
                    if (left_ok) raw_l[r] = __ldg(reinterpret_cast<const uint32_t*>(rp - 2));
                    if (right_ok) raw_r[r] = __ldg(reinterpret_cast<const uint32_t*>(rp + 8));
                }
            }
        }
#pragma unroll
        for (int r = 0; r < A; ++r) {
            float2 d[A];
            if constexpr (sizeof(XT) == 4) {
                // fp32 input: pixels px0..px7 = a.x .. b.w, L and R the neighbours; pairs are (tile 0, tile 1)
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
                float L = 0.f, R = 0.f;
                if ((rowmask >> r) & 1) {
                    const XT* rp = xp + r * geo.W;
                    a = __ldg(reinterpret_cast<const float4*>(rp));
                    b = __ldg(reinterpret_cast<const float4*>(rp) + 1);
                    if (left_ok) L = to_f32(__ldg(rp - 1));
                    if (right_ok) R = to_f32(__ldg(rp + 8));
                }
                d[0] = make_float2(L * xs, a.w * xs);
                d[1] = make_float2(a.x * xs, b.x * xs);
                d[2] = make_float2(a.y * xs, b.y * xs);
                d[3] = make_float2(a.z * xs, b.z * xs);
                d[4] = make_float2(a.w * xs, b.w * xs);
                d[5] = make_float2(b.x * xs, R * xs);
            } else {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            uint32_t lw = 0u, rw = 0u;   // aligned words before / after the segment
            if constexpr (EARLY) {
                v = raw_v[r]; lw = raw_l[r]; rw = raw_r[r];
            } else if ((rowmask >> r) & 1) {
                const __half* rp = xp + r * geo.W;
                v = __ldg(reinterpret_cast<const uint4*>(rp));
                if (left_ok) lw = __ldg(reinterpret_cast<const uint32_t*>(rp - 2));
                if (right_ok) rw = __ldg(reinterpret_cast<const uint32_t*>(rp + 8));
            }
            // pixels: L = lw.hi, px0..px7 = v.x.lo, v.x.hi, ..., v.w.hi, R = rw.lo; tile 0 uses L..px4, tile 1 px3..R
            uint32_t h[A];
            h[0] = __byte_perm(lw, v.y, 0x7632);    // (L,   px3)
            h[1] = __byte_perm(v.x, v.z, 0x5410);   // (px0, px4)
            h[2] = __byte_perm(v.x, v.z, 0x7632);   // (px1, px5)
            h[3] = __byte_perm(v.y, v.w, 0x5410);   // (px2, px6)
            h[4] = __byte_perm(v.y, v.w, 0x7632);   // (px3, px7)
            h[5] = __byte_perm(v.z, rw, 0x5410);    // (px4, R)
#pragma unroll
            for (int s2 = 0; s2 < A; ++s2) d[s2] = __half22float2(*reinterpret_cast<const __half2*>(&h[s2]));
            }   // fp16 input
            bt4_packed(d, e2[r]);
        }
#pragma unroll
        for (int nu = 0; nu < A; ++nu) {
            float2 col[A], o[A];
#pragma unroll
            for (int r = 0; r < A; ++r) col[r] = e2[r][nu];
            bt4_packed(col, o);
#pragma unroll
            for (int xi = 0; xi < A; ++xi)
                *reinterpret_cast<uint32_t*>(vp + (xi * A + nu) * plane) = pack2(o[xi].x, o[xi].y);
        }
        xp += hw;
        vp += Pstride;
    }
}

template <int CH, typename XT = __half>
__global__ void __launch_bounds__(128, 5)
input_transform_f4_kernel(const XT* __restrict__ x, __half* __restrict__ V, TileGeom geo, int C, long long p_begin,
                          FastDiv gdiv, long long Pstride, const float* __restrict__ amax) {
    input_unit_f4<CH, XT>(x, V, geo, C, p_begin, gdiv, Pstride, blockIdx.x * blockDim.x + threadIdx.x, amax);   // < 2^31
}

// Eight output pixels of one row (bias already added): residual (its eight values loaded by the caller, ahead of
// the arithmetic), activation, one rounding, one 16-byte store.
template <bool EP>
__device__ __forceinline__ void store_row8(__half* rowp, float (&v)[8], const uint4& r, const Epilogue& ep,
                                           const __half* = nullptr) {
    if constexpr (EP) {
    if (ep.residual) {
        float a, b2;
        unpack2(r.x, a, b2); v[0] += a; v[1] += b2;
        unpack2(r.y, a, b2); v[2] += a; v[3] += b2;
        unpack2(r.z, a, b2); v[4] += a; v[5] += b2;
        unpack2(r.w, a, b2); v[6] += a; v[7] += b2;
    }
    if (ep.act != 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = epilogue_act(v[i], ep.act);
    }
    }   // EP
    uint4 w;
    w.x = pack2(v[0], v[1]);
    w.y = pack2(v[2], v[3]);
    w.z = pack2(v[4], v[5]);
    w.w = pack2(v[6], v[7]);
    *reinterpret_cast<uint4*>(rowp) = w;
}

// fp32 output: eight pixels are two 16-byte stores, not rounded; the residual row (same offset from ybase as rowp)
// is loaded here
template <bool EP>
__device__ __forceinline__ void store_row8(float* rowp, float (&v)[8], const uint4&, const Epilogue& ep,
                                           const float* ybase = nullptr) {
    if constexpr (EP) {
        if (ep.residual) {
            const float4* rp = reinterpret_cast<const float4*>(static_cast<const float*>(ep.residual) + (rowp - ybase));
            const float4 a = __ldg(rp), b = __ldg(rp + 1);
            v[0] += a.x; v[1] += a.y; v[2] += a.z; v[3] += a.w;
            v[4] += b.x; v[5] += b.y; v[6] += b.z; v[7] += b.w;
        }
        if (ep.act != 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = epilogue_act(v[i], ep.act);
        }
    }
    reinterpret_cast<float4*>(rowp)[0] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4*>(rowp)[1] = make_float4(v[4], v[5], v[6], v[7]);
}

// The same with the residual row already in registers (loaded ahead of the arithmetic by the caller).
__device__ __forceinline__ void store_row8_f32_res(float* rowp, float (&v)[8], const float4 (&rf)[2], const Epilogue& ep) {
    v[0] += rf[0].x; v[1] += rf[0].y; v[2] += rf[0].z; v[3] += rf[0].w;
    v[4] += rf[1].x; v[5] += rf[1].y; v[6] += rf[1].z; v[7] += rf[1].w;
    if (ep.act != 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = epilogue_act(v[i], ep.act);
    }
    reinterpret_cast<float4*>(rowp)[0] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4*>(rowp)[1] = make_float4(v[4], v[5], v[6], v[7]);
}

// LIVE: M is being written by other SMs during this launch (the pipelined kernel): its loads then bypass L1, which
// is not coherent across SMs and may still hold an earlier occupant of a ring slot.
template <int M, int TPT, bool EP, typename YT = __half, bool LIVE = false>
__device__ __forceinline__ void output_unit_vec(const __half* __restrict__ Mws, const YT* __restrict__ bias,
                                                YT* __restrict__ y, const TileGeom& geo, int K, long long p_begin,
                                                const FastDiv& gdiv, long long Pstride, uint32_t idx, const Epilogue& ep) {
    using Wm = Wino<M>;
    constexpr int A = Wm::A;
    static_assert(M * TPT == 8, "one 16-byte row segment per thread");
    const int k = static_cast<int>(fast_div(idx, gdiv));           // gdiv.d = p_count / TPT groups per channel
    if (k >= K) return;
    const int pl = static_cast<int>(idx - static_cast<uint32_t>(k) * gdiv.d) * TPT;
    const long long p = p_begin + pl;
    if (p >= geo.P) return;
    const long long plane = static_cast<long long>(K) * Pstride;
    const __half* src = Mws + static_cast<long long>(k) * Pstride + pl;
    if constexpr (M == 4) {
        // packed path: every float2 holds (tile 0, tile 1)
        float2 tt[M][A];   // A^T m, one column nu at a time
#pragma unroll
        for (int s = 0; s < A; ++s) {
            float2 col[A], o[M];
#pragma unroll
            for (int r = 0; r < A; ++r) {
                const uint32_t* wp = reinterpret_cast<const uint32_t*>(src + (r * A + s) * plane);
                const uint32_t w = LIVE ? __ldcg(wp) : __ldg(wp);
                col[r] = __half22float2(*reinterpret_cast<const __half2*>(&w));
            }
            at4_packed(col, o);
#pragma unroll
            for (int i = 0; i < M; ++i) tt[i][s] = o[i];
        }
        int tw, th;
        long long n;
        decode_tile(geo, p, n, th, tw);
        const float b = load_bias(bias, k);
        [[maybe_unused]] float ys = 1.f;
        if constexpr (sizeof(YT) == 4) ys = scalbnf(1.f, range_exponent(ep.amax));
        YT* img = y + (n * K + k) * static_cast<long long>(geo.H) * geo.W;
        const int i0 = M * th, j0 = M * tw;
        uint4 res[M];
        if constexpr (EP && sizeof(YT) == 2) {
#pragma unroll
            for (int i = 0; i < M; ++i) {
                res[i] = make_uint4(0u, 0u, 0u, 0u);
                if (ep.residual && i0 + i < geo.H)
                    res[i] = __ldg(reinterpret_cast<const uint4*>(static_cast<const __half*>(ep.residual) + (img - y) +
                                                                   static_cast<long long>(i0 + i) * geo.W + j0));
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
            YT* rowp = img + static_cast<long long>(i0 + i) * geo.W + j0;
            store_row8<EP>(rowp, v, res[i], ep, y);
        }
    } else {
    float mm[A][A][TPT];
#pragma unroll
    for (int r = 0; r < A; ++r)
#pragma unroll
        for (int s = 0; s < A; ++s) {
            const __half* q = src + (r * A + s) * plane;
            if constexpr (TPT == 4) {
                const uint2 w = __ldg(reinterpret_cast<const uint2*>(q));
                unpack2(w.x, mm[r][s][0], mm[r][s][1]);
                unpack2(w.y, mm[r][s][2], mm[r][s][3]);
            } else {
                const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(q));
                unpack2(w, mm[r][s][0], mm[r][s][1]);
            }
        }
    int tw, th;
    long long n;
    decode_tile(geo, p, n, th, tw);
    const float b = load_bias(bias, k);
    [[maybe_unused]] float ys = 1.f;
    if constexpr (sizeof(YT) == 4) ys = scalbnf(1.f, range_exponent(ep.amax));
    YT* img = y + (n * K + k) * static_cast<long long>(geo.H) * geo.W;
    const int i0 = M * th, j0 = M * tw;
    uint4 res[M];
    if constexpr (EP && sizeof(YT) == 2) {
#pragma unroll
        for (int i = 0; i < M; ++i) {
            res[i] = make_uint4(0u, 0u, 0u, 0u);
            if (ep.residual && i0 + i < geo.H)
                res[i] = __ldg(reinterpret_cast<const uint4*>(static_cast<const __half*>(ep.residual) + (img - y) +
                                                               static_cast<long long>(i0 + i) * geo.W + j0));
        }
    }
    float out[M][8];  // M output rows of 8 pixels
#pragma unroll
    for (int t = 0; t < TPT; ++t) {
        float tt[M][A];  // A^T mm (M x A)
#pragma unroll
        for (int s = 0; s < A; ++s) {
            float col[A], o[M];
#pragma unroll
            for (int r = 0; r < A; ++r) col[r] = mm[r][s][t];
            mat_apply<M, A>(typename Wm::At{}, col, o);
#pragma unroll
            for (int i = 0; i < M; ++i) tt[i][s] = o[i];
        }
#pragma unroll
        for (int i = 0; i < M; ++i) {
            float o[M];
            mat_apply<M, A>(typename Wm::At{}, tt[i], o);
#pragma unroll
            for (int j = 0; j < M; ++j) out[i][M * t + j] = sizeof(YT) == 4 ? fmaf(o[j], ys, b) : o[j] + b;
        }
    }
#pragma unroll
    for (int i = 0; i < M; ++i) {
        if (i0 + i >= geo.H) continue;
        store_row8<EP>(img + static_cast<long long>(i0 + i) * geo.W + j0, out[i], res[i], ep, y);
    }
    }   // M != 4
}

// EP = false: the plain convolution (the epilogue argument is ignored and costs no register)
template <int M, int TPT, bool EP, typename YT = __half>
__global__ void __launch_bounds__(128)
output_transform_vec_kernel(const __half* __restrict__ Mws, const YT* __restrict__ bias, YT* __restrict__ y,
                            TileGeom geo, int K, long long p_begin, FastDiv gdiv, long long Pstride, WtCheck chk,
                            Epilogue ep) {
    pdl_launch_dependents();
    const bool wt_ok = wt_check(chk);   // before the wait: see output_transform_kernel
    pdl_wait();
    if (!wt_ok) return;
    output_unit_vec<M, TPT, EP, YT>(Mws, bias, y, geo, K, p_begin, gdiv, Pstride, blockIdx.x * blockDim.x + threadIdx.x, ep);
}


// ---------------------------------------------------------------------------------------
// All three steps in one kernel for layers with very few input channels (the 4 -> 320 / 4 -> 512
// input convolutions of the UNet and the VAE decoder).  With C <= 8 the contraction over channels is
// too short for the tensor cores and V, M would only be round trips through L2: a thread owns one
// tile, keeps V[c][a*a] in registers (fp32, not rounded), and for every output channel of the
// block's chunk forms M = sum_c U (.) V from the filter chunk staged in shared memory, applies
// A^T M A, adds the bias and stores.  Consecutive threads own consecutive tiles, so stores coalesce.
// CP = channel count padded to 4 or 8; KC output channels per block.
// ---------------------------------------------------------------------------------------
constexpr int FUSED_KC = 8;

template <int M, int CP>
__global__ void __launch_bounds__(128)
fused_small_c_kernel(const __half* __restrict__ x, const uint32_t* __restrict__ wt_header,
                     const __half* __restrict__ U, const __half* __restrict__ bias, __half* __restrict__ y, TileGeom geo,
                     int C, int K, int Kb, int Cb, int* status_word) {
    using Wm = Wino<M>;
    constexpr int A = Wm::A;
    constexpr int A2 = A * A;
    __shared__ __align__(16) float Us[FUSED_KC][CP][A2];
    pdl_launch_dependents();
    pdl_wait();
    if (!wt_header_ok(wt_header, K, C, M, status_word)) return;
    const int k0 = static_cast<int>(blockIdx.z * gridDim.y + blockIdx.y) * FUSED_KC;   // grid.z continues grid.y
    if (k0 >= K) return;
    // stage the filter chunk: U[pos][Cb][Kb][16][64], this layer has Cb == 1
    const size_t plane = static_cast<size_t>(Kb) * Cb * 1024;
    for (int i = threadIdx.x; i < FUSED_KC * CP * A2; i += blockDim.x) {
        const int pos = i % A2;
        const int c = (i / A2) % CP;
        const int kk = i / (A2 * CP);
        const int k = k0 + kk;
        float v = 0.f;
        if (k < K && c < C)
            v = __half2float(U[pos * plane + (static_cast<size_t>(k >> 4) * Cb * 16 + (k & 15)) * 64 + c]);
        Us[kk][c][pos] = v;
    }
    __syncthreads();
    const long long p = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (p >= geo.P) return;
    int tw, th;
    long long n;
    decode_tile(geo, p, n, th, tw);
    float v[CP][A2];
#pragma unroll
    for (int c = 0; c < CP; ++c) {
        float d[A][A];
        const __half* img = x + (n * C + (c < C ? c : 0)) * static_cast<long long>(geo.H) * geo.W;
        const int i0 = M * th - 1, j0 = M * tw - 1;
#pragma unroll
        for (int r = 0; r < A; ++r) {
            const int i = i0 + r;
            const bool rin = (c < C) && (i >= 0) && (i < geo.H);
#pragma unroll
            for (int s2 = 0; s2 < A; ++s2) {
                const int j = j0 + s2;
                d[r][s2] = (rin && j >= 0 && j < geo.W)
                               ? __half2float(__ldg(img + static_cast<long long>(i) * geo.W + j)) : 0.f;
            }
        }
        float t[A][A];
#pragma unroll
        for (int s2 = 0; s2 < A; ++s2) {
            float col[A], o[A];
#pragma unroll
            for (int r = 0; r < A; ++r) col[r] = d[r][s2];
            mat_apply<A, A>(typename Wm::Bt{}, col, o);
#pragma unroll
            for (int r = 0; r < A; ++r) t[r][s2] = o[r];
        }
#pragma unroll
        for (int r = 0; r < A; ++r) {
            float o[A];
            mat_apply<A, A>(typename Wm::Bt{}, t[r], o);
#pragma unroll
            for (int s2 = 0; s2 < A; ++s2) v[c][r * A + s2] = o[s2];
        }
    }
    const int oi0 = M * th, oj0 = M * tw;
    const bool vec_ok = ((geo.W & 1) == 0) && ((reinterpret_cast<uintptr_t>(y) & 3) == 0);
    const int kend = (K - k0) < FUSED_KC ? (K - k0) : FUSED_KC;
    for (int kk = 0; kk < kend; ++kk) {
        float mm[A][A];
#pragma unroll
        for (int e = 0; e < A2; ++e) {
            float acc = 0.f;
#pragma unroll
            for (int c = 0; c < CP; ++c) acc = fmaf(Us[kk][c][e], v[c][e], acc);
            mm[e / A][e % A] = acc;
        }
        float tt[M][A];
#pragma unroll
        for (int s2 = 0; s2 < A; ++s2) {
            float col[A], o[M];
#pragma unroll
            for (int r = 0; r < A; ++r) col[r] = mm[r][s2];
            mat_apply<M, A>(typename Wm::At{}, col, o);
#pragma unroll
            for (int i = 0; i < M; ++i) tt[i][s2] = o[i];
        }
        const int k = k0 + kk;
        const float b = load_bias(bias, k);
        __half* img = y + (n * K + k) * static_cast<long long>(geo.H) * geo.W;
#pragma unroll
        for (int i = 0; i < M; ++i) {
            float o[M];
            mat_apply<M, A>(typename Wm::At{}, tt[i], o);
            if (oi0 + i >= geo.H) continue;
            __half* rowp = img + static_cast<long long>(oi0 + i) * geo.W + oj0;
#pragma unroll
            for (int j = 0; j < M; j += 2) {
                const __half h0 = __float2half_rn(o[j] + b), h1 = __float2half_rn(o[j + 1] + b);
                if (vec_ok && (oj0 + j + 1 < geo.W)) {
                    *reinterpret_cast<__half2*>(rowp + j) = __halves2half2(h0, h1);
                } else {
                    if (oj0 + j < geo.W) rowp[j] = h0;
                    if (oj0 + j + 1 < geo.W) rowp[j + 1] = h1;
                }
            }
        }
    }
}


// ---------------------------------------------------------------------------------------
// The same for F(2x2,3x3) on the warp-level tensor-core path: with C <= 8 the contraction per position
// is exactly one m16n8k8 MMA (16 output channels x 8 tiles x 8 input channels), and its fragment layout
// needs no data exchange at all.  A warp owns 16 output channels and groups of 8 consecutive tiles:
//   * lane (g = lane / 4, t = lane % 4) transforms tile g of the group for channels 2t and 2t+1 and packs
//     the pair as fp16 -- for every position that IS its B fragment (rows 2t, 2t+1 of column g);
//   * its A fragment per position is two 32-bit loads of the transformed filter (rows g and g+8, channels
//     2t, 2t+1 of the 16 x 64 block; channels past C and rows past K are stored as zeros);
//   * after the 16 MMAs it holds all 16 positions of output channels g, g+8 for tiles 2t, 2t+1, so the
//     output transform, bias and store stay in the lane.
// About 2 instructions per output value against 90 for the scalar kernel above (which stays for F(4x4):
// 36 positions x 4 accumulators would not fit the registers).  tcgen05 is not used here: its smallest tile
// (64 x 8 x 16 per instruction, operands staged in shared memory) does not pay for a contraction of 4.
// ---------------------------------------------------------------------------------------
// 16-byte asynchronous copy global -> shared memory (no register staging) and the wait for all copies of the thread
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst))),
                 "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

constexpr int FC_KB_CHUNK = 4;   // blocks of 16 output channels staged in shared memory at a time (16 KB)

__device__ __forceinline__ void mma_m16n8k8_f16f32(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5}, {%6}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(b0));
}

// Grid: x = groups of 8 tiles, four per block (one per warp); y = chunks of `kb_per_block` blocks of 16 output
// channels.  A warp transforms its 8 tiles once and then walks the chunk's output-channel blocks.
template <typename T = __half>   // element type of x, bias and y
__global__ void __launch_bounds__(128)
fused_small_c_mma_kernel(const T* __restrict__ x, const uint32_t* __restrict__ wt_header,
                         const __half* __restrict__ U, const T* __restrict__ bias, T* __restrict__ y,
                         TileGeom geo, int C, int K, int Kb, int kb_per_block, int* status_word) {
    using Wm = Wino<2>;
    pdl_launch_dependents();
    pdl_wait();
    if (!wt_header_ok(wt_header, K, C, 2, status_word)) return;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const long long hw = static_cast<long long>(geo.H) * geo.W;
    const long long num_groups = (geo.P + 7) / 8;
    const long long grp = static_cast<long long>(blockIdx.x) * 4 + warp;
    const bool active = grp < num_groups;   // warp-uniform; idle warps still help to stage the filters
    // The used part of a filter block (16 rows x 8 channels = 16 bytes of every 128-byte row) is staged in shared
    // memory once per block of four warps: fragment loads straight from global memory touch eight 128-byte
    // lines per instruction and kept the L1 at 77 % of its peak, which bounded the kernel.
    __shared__ uint4 sU[FC_KB_CHUNK][16][16];   // [block of 16 output channels][position][row]: channels 0..7
    const int kb_begin = blockIdx.y * kb_per_block;
    const int kb_end = min(Kb, kb_begin + kb_per_block);
    const size_t plane = static_cast<size_t>(Kb) * 1024;   // one position of U, in elements
    auto stage_filters = [&](int kb0, int chunk) {
        for (int i = threadIdx.x; i < chunk * 256; i += 128) {
            const int row = i & 15, pos = (i >> 4) & 15, kbi = i >> 8;
            cp_async_16(&sU[kbi][pos][row], U + pos * plane + (static_cast<size_t>(kb0 + kbi) * 16 + row) * 64);
        }
    };
    stage_filters(kb_begin, min(FC_KB_CHUNK, kb_end - kb_begin));   // in flight during the input transform

    // ---- input transform: lane (g, t) transforms tile g of the group for channel t (and t + 4 if C > 4) ----
    uint32_t bfrag[16];
    if (active) {
        const long long p = grp * 8 + g;
        int tw = 0, th = 0;
        long long n = 0;
        const bool p_ok = p < geo.P;
        if (p_ok) decode_tile(geo, p, n, th, tw);
        const int i0 = 2 * th - 1, j0 = 2 * tw - 1;
        uint32_t packed[2][16];   // per channel quad: (V[c even], V[c odd]) of tile g, valid in the even-channel lanes
#pragma unroll
        for (int quad = 0; quad < 2; ++quad) {
            const int c = 4 * quad + t;
            float d[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int s2 = 0; s2 < 4; ++s2) d[r][s2] = 0.f;
            if (p_ok && c < C) {       // the second quad is skipped by every lane when C <= 4
                const T* img = x + (n * C + c) * hw;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const int i = i0 + r;
                    if (i < 0 || i >= geo.H) continue;
                    const T* rowp = img + static_cast<long long>(i) * geo.W;
#pragma unroll
                    for (int s2 = 0; s2 < 4; ++s2) {
                        const int j = j0 + s2;
                        if (j >= 0 && j < geo.W) d[r][s2] = to_f32(rowp[j]);
                    }
                }
            }
            float e[4][4];
#pragma unroll
            for (int r = 0; r < 4; ++r) mat_apply<4, 4>(typename Wm::Bt{}, d[r], e[r]);   // along the columns
#pragma unroll
            for (int nu = 0; nu < 4; ++nu) {
                float col[4], o[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) col[r] = e[r][nu];
                mat_apply<4, 4>(typename Wm::Bt{}, col, o);
#pragma unroll
                for (int xi = 0; xi < 4; ++xi) {
                    const float mine = o[xi];
                    const float other = __shfl_xor_sync(0xffffffffu, mine, 1);   // channel c ^ 1 of the same tile
                    packed[quad][xi * 4 + nu] = pack2(mine, other);            // meaningful where c is even
                }
            }
            if (C <= 4) break;   // uniform
        }
        // B fragment of lane (g, t): channels 2t, 2t+1 of tile g = the packed pair of lane (g, (2t) & 3), quad t >> 1
        const int src = (g << 2) | ((2 * t) & 3);
#pragma unroll
        for (int pos = 0; pos < 16; ++pos) {
            const uint32_t r0 = __shfl_sync(0xffffffffu, packed[0][pos], src);
            uint32_t r1 = 0u;
            if (C > 4) r1 = __shfl_sync(0xffffffffu, packed[1][pos], src);      // uniform branch
            bfrag[pos] = t < 2 ? r0 : r1;
        }
    }

    // ---- this lane's output tiles: tiles 2t and 2t+1 of the group ----
    long long out_off[2];       // element offset of (n, k = 0, 2*th, 2*tw); -1 = tile past the end
    bool row1_ok[2], col1_ok[2];
#pragma unroll
    for (int jt = 0; jt < 2; ++jt) {
        const long long p = grp * 8 + 2 * t + jt;
        out_off[jt] = -1;
        row1_ok[jt] = col1_ok[jt] = false;
        if (p < geo.P) {
            int tw, th;
            long long n;
            decode_tile(geo, p, n, th, tw);
            out_off[jt] = n * K * hw + static_cast<long long>(2 * th) * geo.W + 2 * tw;
            row1_ok[jt] = 2 * th + 1 < geo.H;
            col1_ok[jt] = 2 * tw + 1 < geo.W;
        }
    }
    // two pixels (vec_ok) or four (pair_ok) per store: the base of y must be aligned to that many elements
    const bool vec_ok = ((geo.W & 1) == 0) && ((reinterpret_cast<uintptr_t>(y) & (2 * sizeof(T) - 1)) == 0);
    // W % 4 == 0 makes TW even, so tiles 2t and 2t+1 of a group always share a tile row
    const bool pair_ok = ((geo.W & 3) == 0) && ((reinterpret_cast<uintptr_t>(y) & (4 * sizeof(T) - 1)) == 0) && out_off[1] >= 0;

    for (int kb0 = kb_begin; kb0 < kb_end; kb0 += FC_KB_CHUNK) {
    const int chunk = min(FC_KB_CHUNK, kb_end - kb0);
    if (kb0 != kb_begin) {
        __syncthreads();   // the previous chunk has been read
        stage_filters(kb0, chunk);
    }
    cp_async_wait_all();
    __syncthreads();
    if (!active) continue;
    for (int kb = kb0; kb < kb0 + chunk; ++kb) {
        // A fragments: U[pos][kb][0][row][c], rows g and g+8, channels 2t, 2t+1 (zeros past K and C)
        float acc[16][4];   // acc[pos] = {M[g][2t], M[g][2t+1], M[g+8][2t], M[g+8][2t+1]}
#pragma unroll
        for (int pos = 0; pos < 16; ++pos) {
            acc[pos][0] = acc[pos][1] = acc[pos][2] = acc[pos][3] = 0.f;
            const uint32_t a0 = reinterpret_cast<const uint32_t*>(&sU[kb - kb0][pos][g])[t];
            const uint32_t a1 = reinterpret_cast<const uint32_t*>(&sU[kb - kb0][pos][g + 8])[t];
            mma_m16n8k8_f16f32(acc[pos], a0, a1, bfrag[pos]);
        }
#pragma unroll
        for (int hk = 0; hk < 2; ++hk) {
            const int k = kb * 16 + g + 8 * hk;
            if (k >= K) continue;
            const float b = load_bias(bias, k);
            uint32_t row0[2], row1[2];   // packed output pixels of the two tiles: first and second output row
            float o0[2][2], o1[2][2];
#pragma unroll
            for (int jt = 0; jt < 2; ++jt) {
                float tt[2][4];
#pragma unroll
                for (int nu = 0; nu < 4; ++nu) {
                    float col[4], o[2];
#pragma unroll
                    for (int xi = 0; xi < 4; ++xi) col[xi] = acc[xi * 4 + nu][2 * hk + jt];
                    mat_apply<2, 4>(typename Wm::At{}, col, o);
                    tt[0][nu] = o[0];
                    tt[1][nu] = o[1];
                }
                mat_apply<2, 4>(typename Wm::At{}, tt[0], o0[jt]);
                mat_apply<2, 4>(typename Wm::At{}, tt[1], o1[jt]);
                row0[jt] = pack2(o0[jt][0] + b, o0[jt][1] + b);
                row1[jt] = pack2(o1[jt][0] + b, o1[jt][1] + b);
            }
            if constexpr (sizeof(T) == 4) {
                // fp32 output: the same three cases with unrounded values (16-, 8- and 4-byte stores)
                if (pair_ok) {
                    float* q = reinterpret_cast<float*>(y) + out_off[0] + k * hw;
                    *reinterpret_cast<float4*>(q) = make_float4(o0[0][0] + b, o0[0][1] + b, o0[1][0] + b, o0[1][1] + b);
                    if (row1_ok[0])
                        *reinterpret_cast<float4*>(q + geo.W) = make_float4(o1[0][0] + b, o1[0][1] + b, o1[1][0] + b, o1[1][1] + b);
                    continue;
                }
#pragma unroll
                for (int jt = 0; jt < 2; ++jt) {
                    if (out_off[jt] < 0) continue;
                    float* q = reinterpret_cast<float*>(y) + out_off[jt] + k * hw;
                    if (vec_ok) {
                        *reinterpret_cast<float2*>(q) = make_float2(o0[jt][0] + b, o0[jt][1] + b);
                        if (row1_ok[jt]) *reinterpret_cast<float2*>(q + geo.W) = make_float2(o1[jt][0] + b, o1[jt][1] + b);
                    } else {
                        q[0] = o0[jt][0] + b;
                        if (col1_ok[jt]) q[1] = o0[jt][1] + b;
                        if (row1_ok[jt]) {
                            q[geo.W] = o1[jt][0] + b;
                            if (col1_ok[jt]) q[geo.W + 1] = o1[jt][1] + b;
                        }
                    }
                }
            } else {
            if (pair_ok) {
                // the lane's two tiles are neighbours in one tile row: 4 pixels = one 8-byte store per output row,
                // and the four lanes of an output channel complete a 32-byte sector
                __half* q = y + out_off[0] + k * hw;
                *reinterpret_cast<uint2*>(q) = make_uint2(row0[0], row0[1]);
                if (row1_ok[0]) *reinterpret_cast<uint2*>(q + geo.W) = make_uint2(row1[0], row1[1]);
                continue;
            }
#pragma unroll
            for (int jt = 0; jt < 2; ++jt) {
                if (out_off[jt] < 0) continue;
                __half* q = y + out_off[jt] + k * hw;
                if (vec_ok) {           // W even: both columns exist and q is 4-byte aligned
                    *reinterpret_cast<uint32_t*>(q) = row0[jt];
                    if (row1_ok[jt]) *reinterpret_cast<uint32_t*>(q + geo.W) = row1[jt];
                } else {
                    q[0] = __float2half_rn(o0[jt][0] + b);
                    if (col1_ok[jt]) q[1] = __float2half_rn(o0[jt][1] + b);
                    if (row1_ok[jt]) {
                        q[geo.W] = __float2half_rn(o1[jt][0] + b);
                        if (col1_ok[jt]) q[geo.W + 1] = __float2half_rn(o1[jt][1] + b);
                    }
                }
            }
            }   // fp16 output
        }
    }
    }   // chunks of output-channel blocks
}

}  // namespace sdw
