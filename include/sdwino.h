/*
 * sdwino -- stride-1, pad-1, 3x3 2-D convolution by the Winograd algorithm on one
 * NVIDIA B200 (sm_100a).  C ABI; every pointer is a DEVICE pointer unless stated;
 * `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *
 * The operation is the one the paper accelerates: the 3x3 `ggml_conv_2d` of Stable
 * Diffusion's UNet and VAE (Abstract; Section "Techniques"), split, as that section
 * lists, into (i) a preprocess of the filter and of the activation, (ii) an
 * element-wise multiplication of the preprocessed tensors and (iii) a postprocess of
 * the intermediate result.  Tensor layouts are those of the header of Table 1
 * (Filter = [KW,KH,IC,OC], Activation = [IW,IH,IC,N], fastest dimension first), i.e.
 * contiguous w[K][C][3][3] and x[N][C][H][W].
 *
 * Semantics: cross-correlation (no filter flip), zero padding 1, stride 1, dilation 1,
 * groups 1; fp16 storage, fp32 arithmetic and accumulation, one round-to-nearest-even
 * to fp16 per stored value.  `tile` is the output tile edge m of F(m x m, 3 x 3):
 * 2 or 4.  All calls are asynchronous on `stream`: SDWINO_OK means "enqueued".
 * The library never allocates device memory except where a function says so, keeps no
 * reference to caller buffers after a call except the registered workspace, and has no
 * CPU fallback: without a CUDA device every compute call returns SDWINO_ERR_CUDA.
 * Every call works on the calling thread's current CUDA device (cudaSetDevice); what the library keeps per
 * device (SM count, status word, kernel attributes, copy streams of the host path, the built-in scratch of
 * sdwino_conv3x3_static) is set up on first use there, for up to 64 devices per process.  The workspace
 * registered with sdwino_set_workspace and the test hooks are per process.
 * Threads: the filter transforms and the convolution calls that take their workspace as an argument may be
 * called from several host threads at once, each on its own stream and workspace (the library's shared state
 * -- the cache of tensor maps, the per-device facts, the launch counter -- is locked or atomic); functions that
 * say "not thread-safe" below must not run beside them.
 */
#ifndef SDWINO_H
#define SDWINO_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SDWINO_OK = 0,
    SDWINO_ERR_INVALID_ARG = 1, /* NULL required pointer, dimension <= 0, size overflow       */
    SDWINO_ERR_UNSUPPORTED = 2, /* tile not in {2,4}                                          */
    SDWINO_ERR_MISALIGNED = 3,  /* x, w, bias or y not 2-byte aligned; wT / workspace not 1024-byte aligned */
    SDWINO_ERR_WORKSPACE = 4,   /* no workspace registered / passed, or it is too small       */
    SDWINO_ERR_CUDA = 5,        /* a CUDA runtime or driver call failed (see cudaGetLastError) */
    SDWINO_ERR_TIMEOUT = 6      /* a bounded device-side wait gave up (sdwino_last_device_status) */
} sdwino_status;

/* Library version: major*10000 + minor*100 + patch. */
int sdwino_version(void);

/* Static, human-readable name of a status code. */
const char *sdwino_status_string(int status);

/*
 * Filter preprocess, step (i) of Section "Techniques": U[k][c] = G w[k][c] G^T.
 *
 * sdwino_filter_bytes: bytes the caller must allocate for wT (0 on bad arguments).
 * sdwino_filter_transform: w is fp16 [K][C][3][3]; wT receives a 1024-byte header (magic, K, C, tile: the
 *   kernels of sdwino_conv3x3 compare it with their arguments before they read the filters, and a
 *   mismatch is reported as SDWINO_ERR_INVALID_ARG by sdwino_last_device_status) followed by fp16 U laid out as
 *   [a*a][Cb][Kb][16][64] with a = tile+2, Kb = ceil(K/16), Cb = ceil(C/64): blocks of 16 output
 *   channels x 64 input channels (2 KB contiguous each; the blocks of consecutive output channels are
 *   adjacent), position index xi*a+nu, zero in the padding.  wT must be 1024-byte aligned (a cudaMalloc
 *   base is).  wT depends on `tile`; pass the same tile to sdwino_conv3x3.  Done once
 *   per weight; the caller owns both buffers.
 */
size_t sdwino_filter_bytes(int K, int C, int tile);
int sdwino_filter_transform(const void *w, void *wT, int K, int C, int tile, void *stream);

/*
 * Scratch for the transformed activation V and the per-position products M (steps (i)
 * and (ii)).  sdwino_workspace_bytes returns the size that lets the call run in one pass
 * over the tile list, capped at 4 GiB (0 on bad arguments); any workspace of at least
 * sdwino_workspace_min_bytes is accepted and only changes how many passes are made (fewer,
 * longer passes are faster).  The workspace is caller-owned,
 * must be 1024-byte aligned, is overwritten by every call, and may be shared by calls
 * that are ordered on one stream; calls on different streams need different workspaces.
 * sdwino_set_workspace registers the scratch that sdwino_conv3x3 uses (NULL, 0 clears).
 */
size_t sdwino_workspace_bytes(int N, int C, int H, int W, int K, int tile);
size_t sdwino_workspace_min_bytes(int N, int C, int H, int W, int K, int tile);
int sdwino_set_workspace(void *workspace, size_t bytes);

/*
 * The convolution, steps (i) activation preprocess V = B^T d B on overlapping
 * (tile+2)^2 windows, (ii) M = sum_c U (.) V per transform position (a batched GEMM on
 * the tensor cores) and (iii) postprocess Y = A^T M A, plus bias, cast and store.
 *
 *   x    fp16 [N][C][H][W]   (read only)         bias fp16 [K] or NULL (= 0)
 *   wT   from sdwino_filter_transform(K, C, tile)
 *   y    fp16 [N][K][H][W]   (written; must not overlap x or the workspace)
 *
 * H and W need not be multiples of tile: windows are zero-extended past every edge and
 * outputs outside the image are not stored.  sdwino_conv3x3 uses the registered
 * workspace; sdwino_conv3x3_ws takes it explicitly.
 */
int sdwino_conv3x3(const void *x, const void *wT, const void *bias, void *y,
                   int N, int C, int H, int W, int K, int tile, void *stream);
int sdwino_conv3x3_ws(const void *x, const void *wT, const void *bias, void *y,
                      int N, int C, int H, int W, int K, int tile,
                      void *workspace, size_t workspace_bytes, void *stream);

/*
 * The convolution with what follows it in the ResNet blocks of the UNet and the VAE fused into its last step:
 *     y = act(conv3x3(x) + bias + residual)
 * (the paper's operator ends at the convolution; the residual sum and the activation are element-wise passes
 * over y that the output transform absorbs at the cost of reading `residual` once).  residual: fp16
 * [N][K][H][W] device pointer or NULL; it may be y itself (every element is read before it is written, by the
 * same thread), any other overlap with y is not allowed.  activation: SDWINO_ACT_NONE or SDWINO_ACT_SILU
 * (z / (1 + exp(-z)), evaluated in fp32 before the single rounding to fp16); anything else returns
 * SDWINO_ERR_UNSUPPORTED.  Everything else as sdwino_conv3x3_ws.  With residual == NULL and SDWINO_ACT_NONE the
 * call is sdwino_conv3x3_ws; otherwise layers with very few channels take the general three-kernel path.
 */
#define SDWINO_ACT_NONE 0
#define SDWINO_ACT_SILU 1
int sdwino_conv3x3_ex(const void *x, const void *wT, const void *bias, const void *residual, void *y,
                      int N, int C, int H, int W, int K, int tile, int activation,
                      void *workspace, size_t workspace_bytes, void *stream);

/*
 * The fp32 interface: the same path for models kept in fp32 (the paper reports its largest end-to-end gains
 * for them, Tables 2 and 3 "Type F32").  w, x, bias and y are fp32 device tensors with the layouts of the fp16
 * calls; the transformed filters U, the transformed activations V and the products M stay fp16 -- the 11-bit
 * significand of the TF32 tensor-core format at half its bytes, on a path bound by those bytes -- with fp32
 * accumulation, an fp32 output transform and bias sum, and no rounding of y.  Same tolerance as the fp16 calls,
 * max|y - ref| <= 1e-2 max|ref| against the fp64 direct convolution of the fp32 inputs, and the same value
 * range (|x| <= 1e3 for tile 2, 1e2 for tile 4: V is fp16).
 *
 * sdwino_filter_transform_f32 writes the same wT as sdwino_filter_transform (size sdwino_filter_bytes; U is
 * computed in fp32 from the fp32 weights and rounded once), so the buffer serves either convolution call.
 * sdwino_conv3x3_f32 takes its workspace explicitly (sdwino_workspace_bytes, as for the fp16 calls).  The
 * single-kernel paths of tile 2 for layers with at most 8 input or output channels serve it too (the one for
 * few output channels rounds the pixels of x to fp16 as it loads them); with tile 4 such layers take the general
 * three kernels.  Pointers must be 4-byte aligned
 * (SDWINO_ERR_MISALIGNED); 16-byte aligned x and y with W % 8 == 0 take the vector kernels.  Arguments, errors
 * and asynchrony otherwise as sdwino_filter_transform / sdwino_conv3x3_ws.
 */
int sdwino_filter_transform_f32(const float *w, void *wT, int K, int C, int tile, void *stream);
int sdwino_conv3x3_f32(const float *x, const void *wT, const float *bias, float *y,
                       int N, int C, int H, int W, int K, int tile,
                       void *workspace, size_t workspace_bytes, void *stream);
/* The fp32 convolution for activations of any fp32 magnitude (the "Type F32" rows of the paper's Tables 2 and 3 run
 * fp32 models, whose activations are not bound to the fp16 range).  V and M are fp16 inside the library; this entry
 * first finds max|x| (one extra pass over x), multiplies x by the power of two that brings that maximum near 64 on its
 * way into V and multiplies the result by the inverse on its way out of M, so that neither overflows nor loses its
 * small values; powers of two round nothing.  Same arguments as sdwino_conv3x3_f32; the last 1 KiB of the workspace
 * holds the maximum (a workspace of sdwino_workspace_bytes still gives one pass).  The relative accuracy is that of
 * sdwino_conv3x3_f32 on inputs of moderate size: 1e-2 * max|ref| as long as max|y| / max|x| stays below about 500
 * (M must still fit fp16 after the scaling).  Layers with few channels take the three-kernel path here. */
int sdwino_conv3x3_f32_scaled(const float *x, const void *wT, const float *bias, float *y,
                              int N, int C, int H, int W, int K, int tile,
                              void *workspace, size_t workspace_bytes, void *stream);
/* y = act(conv3x3(x) + bias + residual) with fp32 tensors: sdwino_conv3x3_ex for the fp32 interface (residual fp32
 * [N][K][H][W] or NULL, may be y itself; activation SDWINO_ACT_NONE or SDWINO_ACT_SILU; nothing is rounded). */
int sdwino_conv3x3_f32_ex(const float *x, const void *wT, const float *bias, const float *residual, float *y,
                          int N, int C, int H, int W, int K, int tile, int activation,
                          void *workspace, size_t workspace_bytes, void *stream);

/*
 * 8-bit transformed filters (Section "Evaluation", "Operator Support": the quantised operators).  The filter stream
 * bounds the layers with few tiles and many channels; storing it in 8 bits halves it.  Reading of the paper, which
 * names no format: every row U[position][k][:] of the fp16 transformed filter becomes integers q = round(U / s) in
 * [-127, 127] with s = max|U| / 127 over the row (both formed in fp32, ties to even); the contraction runs on the
 * integers (exact in fp16, kind::f16 MMA, fp32 accumulation) and s multiplies the accumulator of the row.
 *   sdwino_filter_q8_bytes      size of the 8-bit buffer (0 for invalid arguments); 1024-byte aligned like wT.
 *   sdwino_filter_quantize      wT (made by sdwino_filter_transform[_f32] for the same K, C, tile) -> wTq; wT may
 *                               be freed afterwards.  A wT made for other K / C / tile is reported through
 *                               sdwino_last_device_status and nothing is written.
 *   sdwino_conv3x3_q8           sdwino_conv3x3_ws with an 8-bit filter: fp16 x, bias, y; same workspace.  Handing it
 *                               an fp16 wT, or an 8-bit buffer to the other entries, is caught by the header check
 *                               (SDWINO_ERR_INVALID_ARG from sdwino_last_device_status, y untouched).
 * Accuracy: the quantisation is part of the operator (the oracle applies the same rule); against the unquantised
 * convolution it costs about 1 % rms with tile 2 and 3-4 % with tile 4, whose transform amplifies filter noise.
 */
size_t sdwino_filter_q8_bytes(int K, int C, int tile);
int sdwino_filter_quantize(const void *wT, void *wTq, int K, int C, int tile, void *stream);
int sdwino_conv3x3_q8(const void *x, const void *wTq, const void *bias, void *y,
                      int N, int C, int H, int W, int K, int tile,
                      void *workspace, size_t workspace_bytes, void *stream);

/*
 * The direct convolution, stride 1 or 2 (Abstract / Section "Techniques": the operator the paper replaces is
 * ggml_conv_2d as a whole; the UNet's downsampling convolutions are 3x3, pad 1, stride 2, which Winograd's
 * overlapping tiles cannot express).  It is the degenerate member of the family, F(1x1,3x3): a tile is one output
 * pixel, the nine transform positions are the nine filter taps, and the same three steps run: the activation step
 * gathers the nine shifted copies of x (V[tap][c][pixel]), the tcgen05 GEMM contracts the channels per tap, the output
 * step adds the nine partial sums and the bias.  It streams 9 instead of 16 (tile 2) filter values per weight, at
 * 2.25 times the tensor work per output pixel.
 *   filters: sdwino_filter_bytes / sdwino_filter_transform with tile = 1 (the weights reordered tap by tap).
 *   y: fp16 [N][K][Ho][Wo] with Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1; stride 1 or 2
 *   (SDWINO_ERR_UNSUPPORTED above 2, SDWINO_ERR_INVALID_ARG below 1).  Workspace: sdwino_workspace_bytes_direct for
 *   one pass; smaller workspaces take several passes as in sdwino_conv3x3_ws.  Other arguments and errors as
 *   sdwino_conv3x3_ws.
 */
size_t sdwino_workspace_bytes_direct(int N, int C, int H, int W, int K, int stride);
int sdwino_conv3x3_direct(const void *x, const void *wT, const void *bias, void *y,
                          int N, int C, int H, int W, int K, int stride,
                          void *workspace, size_t workspace_bytes, void *stream);

/*
 * Several layers in one call, optionally with each layer's filters travelling to L2 while the layer before it
 * computes (Section "Techniques", second paragraph: a core that finishes its block is handed the next one at once;
 * here the memory system can be handed the next layer's filters, the one operand of a layer that depends on nothing
 * before it).
 * Layers run in order on `stream`, each exactly as sdwino_conv3x3_ws would run it (same kernels, same bits), so layer
 * i + 1 may read what layer i wrote.  With prefetch_bytes > 0, a small kernel on a stream of the library's own (lowest
 * priority, ordered after everything that precedes layer i in `stream`) queues L2 prefetches for up to prefetch_bytes
 * of layer i + 1's transformed filters, the same share of every transform position; it only issues the requests and
 * ends, nothing waits for the data, and the side stream is joined back into `stream` before the call returns, so the
 * call can be captured into a CUDA graph.  prefetch_bytes = 0 (the recommended value): no side stream, no extra
 * launches.  Measured on the UNet sweeps the prefetch does not pay: the GEMM already sends its first ring of filter
 * boxes out before it waits for the activation transform, its filter stream runs at the HBM rate once started, and
 * the early requests take bandwidth from the running layer (a sweep is 1-25 % slower with 8-128 MB prefetched per
 * layer), so the knob is there for other parts and other layer mixes, not as a default.
 *   layers[i]: device pointers x, wT (sdwino_filter_transform for K, C, tile), bias (or NULL), y, all fp16, and the
 *   sizes of the layer; tile 1, 2 or 4 (sdwino_choose_algorithm).  The array itself is host memory and is only read
 *   during the call.  workspace: device, 1024-byte aligned, shared by the layers one after the other;
 *   sdwino_workspace_bytes_sequence gives the size at which every layer runs in one pass (0 for an invalid list).
 * Errors: every layer is validated before the first launch (SDWINO_ERR_INVALID_ARG / _UNSUPPORTED / _MISALIGNED /
 * _WORKSPACE as for sdwino_conv3x3_ws), so a sequence is either enqueued whole or not at all, except for
 * SDWINO_ERR_CUDA from a launch.  Calls with prefetch_bytes > 0 from several threads are serialised while they
 * enqueue (they share the side stream).
 */
typedef struct sdwino_layer {
    const void *x;       /* device fp16 [N][C][H][W] */
    const void *wT;      /* device, transformed filters of this layer */
    const void *bias;    /* device fp16 [K], or NULL */
    void *y;             /* device fp16 [N][K][H][W] */
    int N, C, H, W, K;
    int tile;            /* 1, 2 or 4 */
} sdwino_layer;
size_t sdwino_workspace_bytes_sequence(const sdwino_layer *layers, int n);
int sdwino_conv3x3_sequence(const sdwino_layer *layers, int n, void *workspace, size_t workspace_bytes,
                            size_t prefetch_bytes, void *stream);

/*
 * The convolution for callers that must not allocate device memory.  (The paper has no
 * counterpart; this entry point exists for the embedding of the library.)  Some callers cannot
 * call cudaMalloc or any allocator at all: code that runs inside a CUDA-graph capture or another
 * region where allocation is forbidden, plug-ins whose host hands them fixed buffers and bans
 * further allocation, and processes whose memory budget is fixed at start-up.  They still pass x,
 * wT, bias and y exactly as to sdwino_conv3x3, but the scratch for V and M is a file-scope device
 * array of SDWINO_STATIC_SCRATCH_BYTES inside the library image, so every GPU that loads the library
 * holds that much memory until the process exits, and no allocation call is made on this path.
 *
 *   - Limit: a layer is accepted when one pass of 128 tiles fits, i.e. when
 *     128 * (tile+2)^2 * (C + K) * 2 bytes + 2 KiB <= SDWINO_STATIC_SCRATCH_BYTES (tile 2:
 *     C + K <= 8191; tile 4: C + K <= 3640); larger layers return SDWINO_ERR_WORKSPACE.  Large images
 *     simply take more passes.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls share the one array and it keeps the contents of the last call.  Nothing in it has to
 *     start at zero: every pass overwrites all elements it later reads.  Calls that may overlap on the
 *     GPU (different streams, or graphs replayed concurrently) race on the array; order them.
 */
#define SDWINO_STATIC_SCRATCH_BYTES (32u << 20)
int sdwino_conv3x3_static(const void *x, const void *wT, const void *bias, void *y,
                          int N, int C, int H, int W, int K, int tile, void *stream);

/*
 * The same convolution for callers whose tensors live in HOST memory (pageable or pinned):
 * x_host, bias_host and y_host are host pointers, wT stays a device pointer.  On `stream`
 * the call copies x (and bias) to the device, runs the three steps, copies y back and then
 * synchronises the stream, so y_host is complete on return.  It allocates nothing: the
 * device-side copies of x, bias and y are carved from the front of `workspace`, which must
 * therefore hold sdwino_host_staging_bytes(...) in addition to a scratch accepted by
 * sdwino_conv3x3_ws (at least sdwino_workspace_min_bytes).  Used for end-to-end timing.
 *
 * sdwino_conv3x3_host_async is the same without the final synchronisation: it returns once the work is
 * enqueued.  Uploads and downloads run on two copy streams owned by the library and alternate between two
 * slots of the staging area, so the upload of the next call and the download of the previous one overlap the
 * kernels of this one (PCIe is full duplex); the kernels stay on `stream`, in call order.  y_host of every
 * earlier call is complete once sdwino_host_join(stream) has been called (it makes `stream` wait for the
 * outstanding downloads) and `stream` has then been synchronised; x_host and bias_host must not change until
 * then.  While such calls are in flight the staging part of the workspace belongs to them: do not hand the
 * same workspace to other entry points before the join.  Calls with the same sizes may share a workspace and
 * still overlap (they alternate between the two slots); a call whose sizes differ from those of an in-flight
 * call on overlapping memory is ordered after that call's kernels and download, so give every layer of a
 * network its own workspace if their copies are to overlap.  The first call on a device creates the two streams
 * and 96 events (make it outside any stream capture); not thread-safe.
 */
size_t sdwino_host_staging_bytes(int N, int C, int H, int W, int K, int tile);
int sdwino_conv3x3_host(const void *x_host, const void *wT, const void *bias_host, void *y_host,
                        int N, int C, int H, int W, int K, int tile,
                        void *workspace, size_t workspace_bytes, void *stream);
int sdwino_conv3x3_host_async(const void *x_host, const void *wT, const void *bias_host, void *y_host,
                              int N, int C, int H, int W, int K, int tile,
                              void *workspace, size_t workspace_bytes, void *stream);
int sdwino_host_join(void *stream);
/* The host-buffer entries for the fp32 interface (the model type of the "Type F32" rows of the paper's Tables 2
 * and 3): x_host, bias_host and y_host are fp32 host arrays, wT comes from either filter transform; the staging
 * part of the workspace is sdwino_host_staging_bytes_f32(...).  Everything else as above; the two families may be
 * mixed on one stream and are joined by the same sdwino_host_join. */
size_t sdwino_host_staging_bytes_f32(int N, int C, int H, int W, int K, int tile);
int sdwino_conv3x3_host_f32(const float *x_host, const void *wT, const float *bias_host, float *y_host,
                            int N, int C, int H, int W, int K, int tile,
                            void *workspace, size_t workspace_bytes, void *stream);
int sdwino_conv3x3_host_f32_async(const float *x_host, const void *wT, const float *bias_host, float *y_host,
                                  int N, int C, int H, int W, int K, int tile,
                                  void *workspace, size_t workspace_bytes, void *stream);

/*
 * Device-side waits (on TMA / tensor-core completion barriers) are bounded; a wait that
 * gives up records SDWINO_ERR_TIMEOUT in a device status word and the kernel returns
 * normally.  This call synchronises `stream`, returns that word (SDWINO_OK if nothing
 * was recorded) and clears it.
 */
int sdwino_last_device_status(void *stream);

/*
 * Self-test of that mechanism: launches one thread that waits on a barrier nothing signals, with the
 * given limit (1 ns .. 10 ms, else SDWINO_ERR_INVALID_ARG).  The kernel returns normally after about
 * the limit (the timer is sampled every few thousand polls, so up to ~1 ms later) and
 * sdwino_last_device_status then reports SDWINO_ERR_TIMEOUT once.  Nothing else is touched: the
 * context stays usable and later calls are unaffected.
 */
int sdwino_selftest_wait_timeout(unsigned long long limit_ns, void *stream);

/* Kernel launches made by this library in the calling process so far (all entry points). */
unsigned long long sdwino_launch_count(void);

/*
 * Tuning and test hook for the batched GEMM of step (ii).  By default the library picks, per
 * call, between single-CTA tiles (128 tiles x n output channels; also with two blocks of 128 tiles per
 * CTA tile, or with the filter block of a position resident in shared memory) and CTA-pair tiles (256 tiles x
 * n output channels, tcgen05 cta_group::2; n is then rounded up to a multiple of 32) and the n that
 * fits the layer.  Forcing either field selects the plain kernel of that shape.  ctas in {1, 2} and/or
 * n_tile (a multiple of 16 in [16, 256]) force that choice for later calls of this process; 0
 * restores the automatic choice for that field.  Results do not depend on the choice beyond
 * the fp32 summation order inside the tensor core.  Returns SDWINO_ERR_INVALID_ARG otherwise.
 */
int sdwino_set_gemm_shape(int ctas, int n_tile);

/*
 * Test hook for the transforms of steps (i) and (iii) with tile = 4.  With W % 8 == 0 and 16-byte aligned x / y
 * they can stage their operands in shared memory by TMA, several channels ahead of the arithmetic (the
 * overlapping input tiles of a block; the 36 transform positions of a block of tiles), instead of loading them
 * into registers; both forms produce the same bits.  mode 1 (the default) stages where that measured faster
 * (activation transform: W % 64 == 0; output transform: passes of 512 tiles or more), mode 2 wherever it is
 * possible, mode 0 never.  Returns SDWINO_ERR_INVALID_ARG for any other value.  Not thread-safe against
 * concurrent compute calls.
 */
int sdwino_set_input_staging(int mode);

/*
 * Which of the two supported algorithms is expected to be faster for a layer: returns 2 for F(2x2,3x3),
 * 4 for F(4x4,3x3), 0 for non-positive sizes.  The paper leaves the tile size open; both satisfy the
 * accuracy bound (F4 with about 4x the error of F2).  Rule, with tiles = N * ceil(H/2) * ceil(W/2):
 * at most 8 input channels -> 2 (single-kernel path); at most 8 output channels -> 2 from 12288 tiles
 * (single-kernel path), 4 below; otherwise 4 when 2 * tiles * (C + K) >= K * C, i.e. when the
 * activation-side traffic outweighs the weights, and also from 0.65 of that threshold when there are at least
 * 256 tiles.
 * Pure host arithmetic: no device is touched.  The caller passes the result as `tile` to
 * sdwino_filter_transform and sdwino_conv3x3.
 */
int sdwino_choose_tile(int N, int C, int H, int W, int K);
/* The same choice with the direct form (tile 1, stride 1: see sdwino_conv3x3_direct) among the candidates: returns 1,
 * 2 or 4 (0 for invalid sizes).  The fp16 entries that take a workspace, a registered workspace, the built-in scratch
 * or host buffers accept tile 1 and then run the direct convolution with stride 1; the fp32 and 8-bit entries do not
 * (SDWINO_ERR_UNSUPPORTED). */
int sdwino_choose_algorithm(int N, int C, int H, int W, int K);

/*
 * Tuning and test knob.  F(2x2,3x3) layers with at most 8 output channels (the 320 -> 4 and 128 -> 3
 * output convolutions) run as ONE kernel that keeps V and M on chip (input transform into shared memory,
 * tcgen05 MMAs into TMEM, output transform from TMEM) when the batch has at least `p_tiles` blocks of 128
 * tiles (default 48: below that too few SMs get work and the three-kernel path is faster), W % 8 == 0,
 * x is 16-byte and y 4-byte aligned.  p_tiles = 0 restores the default; 1 sends every eligible layer
 * through the kernel (used by the tests).  Forcing a GEMM shape with sdwino_set_gemm_shape disables it.
 * Returns SDWINO_ERR_INVALID_ARG for a negative value.  Not thread-safe against concurrent compute calls.
 */
int sdwino_set_fused_min_tiles(long long p_tiles);

/*
 * Tuning / test hook for the pipelined single-launch path of F(4x4,3x3) (Section "Techniques": the B200 counterpart
 * of keeping the transformed data in the nearest memory and of handing work out dynamically).  Layers with
 * thousands of tiles and filters of at most a few tens of MB run all three steps in ONE persistent, cooperative
 * launch: V and M live in rings of a few blocks of 128 tiles that stay in L2, transform warps pull (block, channel
 * group) items from an atomic queue while the GEMM warps of the same CTAs multiply the blocks behind them.
 * mode 2: wherever the layer shape allows it (fp16 interface, tile 4, W % 8 == 0, 16-byte aligned x and y, more
 * than 4 input channels, plain convolution, transformed filters of at most 40 MB); mode 0: never; mode 1 (default):
 * where it is faster, which on the measured layers is nowhere (it moves a third of the DRAM bytes but takes 17-60 %
 * longer than the three kernels), so today mode 1 behaves like mode 0.
 * ring / lead: ring slots and the lag of the output transform behind the activation transform, in blocks of 128
 * tiles; 0 = chosen by the library.  Returns SDWINO_ERR_INVALID_ARG for other values.  Results are the bits of the
 * three-kernel path.  Safe against concurrent compute calls (a call reads the setting once).
 */
int sdwino_set_pipeline(int mode, int ring, int lead);

/*
 * Timing for benchmarks.  mode 1: every kernel launch of the library is bracketed by two CUDA
 * events recorded on the launch's stream (this adds a little idle time between kernels, so
 * whole-call timings should be taken with profiling disabled).  mode 2: every convolution call
 * as a whole is bracketed instead (one record of kind 5 per call; the kernels inside a call keep
 * their overlap, so the records of a step add up to the step).  mode 0: off; other values return
 * SDWINO_ERR_INVALID_ARG.
 * sdwino_profile_collect waits for the recorded events, adds the elapsed milliseconds and
 * the launch counts per kind into the two caller arrays of 6 entries (0 filter
 * transform, 1 activation transform, 2 batched GEMM, 3 output transform, 4 the single-kernel
 * paths for layers with few input or few output channels, 5 whole calls; either may be NULL)
 * and forgets the records.  Host arrays.  The mode switch and the record list are safe against
 * concurrent compute calls; the records of concurrent calls interleave.
 */
int sdwino_profile_enable(int mode);
int sdwino_profile_collect(double *ms_by_kind, unsigned long long *launches_by_kind);
/* The same records one by one, in launch order: fills kinds[i] and ms[i] (host arrays of `capacity`
 * entries, either may be NULL; ms < 0 marks an event error) for the first `capacity` launches since
 * the last collect and returns how many there were.  keep == 0 forgets the records; keep != 0
 * leaves them in place, which is how launches captured into a CUDA graph while profiling was
 * enabled are read again after every replay of that graph (the events are then graph nodes). */
int sdwino_profile_records(int *kinds, float *ms, int capacity, int keep);

#ifdef __cplusplus
}
#endif
#endif /* SDWINO_H */
