"""fp64 CPU oracle for the 3x3 stride-1 pad-1 convolution and its Winograd form.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this module;
only the tests, the smoke check and the benchmark's CPU-baseline leg do.  It
shares no code, table or constant with the CUDA library.

Ground truth is the plain definition of the operator the paper accelerates
(``ggml_conv_2d`` with a 3x3 filter; Abstract, Section "Techniques", layouts from
the header of Table 1): cross-correlation, zero padding 1, stride 1.  The
Winograd functions follow the three steps the paper lists in Section
"Techniques" (preprocess filter and activation, element-wise multiply,
postprocess) with the Toom-Cook matrices of the construction the paper cites
(Lavin & Gray); the paper prints no matrices, so they are derived here from
the interpolation points in exact rational arithmetic.

Pins (tests/test_oracle_*.py): exact rational identity of the matrices, the
four-multiply closed form of F(2,3), hand-worked 4x4 values, delta/all-ones
special cases, brute force on tiny inputs, agreement of the two routes to
1e-10 and with torch / scipy library routines; for the fused epilogue, known
values and identities of SiLU and torch's routine.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from fractions import Fraction

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "conv_oracle.c")
_LIB = os.path.join(_HERE, "libconv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile conv_oracle.c into a shared object next to it (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int)
        i = ctypes.c_int
        lib.oracle_direct.argtypes = [dp, dp, dp, dp, i, i, i, i, i]
        lib.oracle_direct_channels.argtypes = [dp, dp, dp, dp, i, i, i, i, i, ip, i]
        lib.oracle_direct_strided.argtypes = [dp, dp, dp, dp, i, i, i, i, i, i]
        lib.oracle_filter_transform.argtypes = [dp, dp, dp, i, i, i]
        lib.oracle_input_tile_transform.argtypes = [dp, dp, dp, i, i, i, i, i, i, i, i]
        lib.oracle_winograd.argtypes = [dp, dp, dp, dp, i, i, i, i, i, i, dp, dp, dp]
        lib.oracle_winograd_with_filter.argtypes = [dp, dp, dp, dp, i, i, i, i, i, i, dp, dp]
        lib.oracle_threads.restype = i
        _lib = lib
    return _lib


def threads() -> int:
    """Threads the OpenMP loops of the C oracle use on this host."""
    return int(_load().oracle_threads())


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if a is not None else None


# --------------------------------------------------------------------------
# What the library can fuse after the convolution: y = act(conv + bias + residual)
# --------------------------------------------------------------------------

def silu(z):
    """SiLU (swish) z * sigmoid(z) = z / (1 + exp(-z)), the activation of the ResNet blocks of Stable Diffusion's
    UNet and VAE (not part of the paper's operator).  fp64; for very negative z, exp overflows to inf and the
    quotient is -0, the limit."""
    z = np.asarray(z, dtype=np.float64)
    with np.errstate(over="ignore"):
        return z / (1.0 + np.exp(-z))


def epilogue(conv, residual=None, activation=None):
    """act(conv + residual) in fp64; ``conv`` already holds the bias.  activation: None or "silu"."""
    y = np.asarray(conv, dtype=np.float64)
    if residual is not None:
        y = y + np.asarray(residual, dtype=np.float64)
    if activation == "silu":
        y = silu(y)
    elif activation is not None:
        raise ValueError(activation)
    return y


# --------------------------------------------------------------------------
# Direct convolution (the definition)
# --------------------------------------------------------------------------

def direct_conv3x3(x, w, bias=None, channels=None):
    """y[n,k,i,j] = b[k] + sum_{c,u,v} xhat[n,c,i+u-1,j+v-1] * w[k,c,u,v] in fp64.

    ``channels``: optional list of output channels; the result then has shape
    [N, len(channels), H, W] (used to check very large layers on a subset).
    """
    x, w = _f64(x), _f64(w)
    N, C, H, W = x.shape
    K = w.shape[0]
    assert w.shape == (K, C, 3, 3)
    b = _f64(bias) if bias is not None else None
    if channels is None:
        y = np.empty((N, K, H, W), dtype=np.float64)
        rc = _load().oracle_direct(_ptr(x), _ptr(w), _ptr(b), _ptr(y), N, C, H, W, K)
    else:
        ks = np.ascontiguousarray(np.asarray(channels, dtype=np.int32))
        assert ks.ndim == 1 and ks.min() >= 0 and ks.max() < K
        y = np.empty((N, len(ks), H, W), dtype=np.float64)
        rc = _load().oracle_direct_channels(
            _ptr(x), _ptr(w), _ptr(b), _ptr(y), N, C, H, W, K,
            ks.ctypes.data_as(ctypes.POINTER(ctypes.c_int)), len(ks))
    if rc != 0:
        raise RuntimeError(f"oracle_direct failed ({rc})")
    return y


def direct_conv3x3_strided(x, w, bias=None, stride: int = 2):
    """The 3x3 convolution with zero padding 1 sampled with a stride (the downsampling convolutions of the UNet):
    y[n,k,i,j] = b[k] + sum_{c,u,v} xhat[n,c,s*i+u-1,s*j+v-1] * w[k,c,u,v], shape [N, K, (H-1)//s+1, (W-1)//s+1]."""
    x, w = _f64(x), _f64(w)
    N, C, H, W = x.shape
    K = w.shape[0]
    assert w.shape == (K, C, 3, 3) and stride >= 1
    b = _f64(bias) if bias is not None else None
    y = np.empty((N, K, (H - 1) // stride + 1, (W - 1) // stride + 1), dtype=np.float64)
    rc = _load().oracle_direct_strided(_ptr(x), _ptr(w), _ptr(b), _ptr(y), N, C, H, W, K, stride)
    if rc != 0:
        raise RuntimeError(f"oracle_direct_strided failed ({rc})")
    return y


def brute_conv3x3(x, w, bias=None):
    """The nine-term sum written out literally per output element, with explicit
    bounds checks, in pure Python floats.  Only for tiny inputs; written apart
    from the C loops so the two can disagree."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    N, C, H, W = x.shape
    K = w.shape[0]
    y = np.zeros((N, K, H, W), dtype=np.float64)
    for n in range(N):
        for k in range(K):
            for i in range(H):
                for j in range(W):
                    s = 0.0 if bias is None else float(bias[k])
                    for c in range(C):
                        for u in (0, 1, 2):
                            for v in (0, 1, 2):
                                ii, jj = i + u - 1, j + v - 1
                                if 0 <= ii < H and 0 <= jj < W:
                                    s += float(x[n, c, ii, jj]) * float(w[k, c, u, v])
                    y[n, k, i, j] = s
    return y


# --------------------------------------------------------------------------
# Winograd matrices (exact rationals)
# --------------------------------------------------------------------------

# The matrices of the standard F(2x2,3x3) construction, points {0, 1, -1, inf}.
_F2 = dict(
    Bt=[[1, 0, -1, 0], [0, 1, 1, 0], [0, -1, 1, 0], [0, 1, 0, -1]],
    G=[[1, 0, 0], [Fraction(1, 2), Fraction(1, 2), Fraction(1, 2)],
       [Fraction(1, 2), Fraction(-1, 2), Fraction(1, 2)], [0, 0, 1]],
    At=[[1, 1, 1, 0], [0, 1, -1, -1]],
)

DEFAULT_POINTS = {
    2: (Fraction(0), Fraction(1), Fraction(-1)),
    4: (Fraction(0), Fraction(1), Fraction(-1), Fraction(2), Fraction(-2)),
}


def _solve_exact(A, b):
    """Solve the (possibly overdetermined, consistent) system A z = b in Fractions."""
    rows, cols = len(A), len(A[0])
    M = [[Fraction(v) for v in A[r]] + [Fraction(b[r])] for r in range(rows)]
    piv_row = 0
    piv_cols = []
    for c in range(cols):
        p = next((r for r in range(piv_row, rows) if M[r][c] != 0), None)
        if p is None:
            raise ValueError("singular system")
        M[piv_row], M[p] = M[p], M[piv_row]
        pv = M[piv_row][c]
        M[piv_row] = [v / pv for v in M[piv_row]]
        for r in range(rows):
            if r != piv_row and M[r][c] != 0:
                f = M[r][c]
                M[r] = [vr - f * vp for vr, vp in zip(M[r], M[piv_row])]
        piv_cols.append(c)
        piv_row += 1
    for r in range(piv_row, rows):
        if M[r][cols] != 0:
            raise ValueError("inconsistent system")
    return [M[i][cols] for i in range(cols)]


def winograd_matrices(m: int, points=None):
    """Exact (Fraction) matrices Bt [a x a], G [a x 3], At [m x a] of F(m x m, 3 x 3)
    built from a-1 finite interpolation points plus the point at infinity.

    G[x] = [1, p, p^2] / prod_{j != x}(p_x - p_j), G[inf] = [0, 0, 1];
    At[i][x] = p_x^i, At[i][inf] = 1 if i == m-1 else 0;
    Bt is the unique solution of  sum_x At[i][x] G[x][u] Bt[x][s] = [s == i+u].
    With ``points=None`` and m == 2 the textbook F(2x2,3x3) matrices are returned.
    """
    a = m + 2
    if points is None and m == 2:
        conv = lambda M: [[Fraction(v) for v in row] for row in M]
        return conv(_F2["Bt"]), conv(_F2["G"]), conv(_F2["At"])
    pts = [Fraction(p) for p in (points if points is not None else DEFAULT_POINTS[m])]
    if len(pts) != a - 1 or len(set(pts)) != len(pts):
        raise ValueError("need a-1 distinct finite points")
    G = []
    for xi, p in enumerate(pts):
        den = Fraction(1)
        for j, q in enumerate(pts):
            if j != xi:
                den *= (p - q)
        G.append([1 / den, p / den, p * p / den])
    G.append([Fraction(0), Fraction(0), Fraction(1)])
    At = [[(p ** i if i > 0 else Fraction(1)) for p in pts] + [Fraction(1 if i == m - 1 else 0)]
          for i in range(m)]
    Bt = [[Fraction(0)] * a for _ in range(a)]
    for s in range(a):
        A_rows, rhs = [], []
        for i in range(m):
            for u in range(3):
                A_rows.append([At[i][xi] * G[xi][u] for xi in range(a)])
                rhs.append(1 if s == i + u else 0)
        col = _solve_exact(A_rows, rhs)
        for xi in range(a):
            Bt[xi][s] = col[xi]
    return Bt, G, At


def _mats_f64(m, points):
    Bt, G, At = winograd_matrices(m, points)
    tof = lambda M: np.ascontiguousarray(np.array([[float(v) for v in r] for r in M], dtype=np.float64))
    return tof(Bt), tof(G), tof(At)


# --------------------------------------------------------------------------
# Winograd evaluation (three steps)
# --------------------------------------------------------------------------

def filter_transform(w, m: int = 2, points=None):
    """U[k,c] = G w[k,c] G^T, shape [K, C, a, a], fp64 (filter preprocess)."""
    w = _f64(w)
    K, C = w.shape[:2]
    a = m + 2
    _, G, _ = _mats_f64(m, points)
    U = np.empty((K, C, a, a), dtype=np.float64)
    rc = _load().oracle_filter_transform(_ptr(w), _ptr(G), _ptr(U), K, C, a)
    if rc != 0:
        raise RuntimeError(f"oracle_filter_transform failed ({rc})")
    return U


def input_tile_transform(x, n: int, th: int, tw: int, m: int = 2, points=None):
    """V[c] = B^T d[c] B for the tile (n, th, tw): shape [C, a, a] (activation preprocess)."""
    x = _f64(x)
    N, C, H, W = x.shape
    a = m + 2
    Bt, _, _ = _mats_f64(m, points)
    V = np.empty((C, a, a), dtype=np.float64)
    rc = _load().oracle_input_tile_transform(_ptr(x), _ptr(Bt), _ptr(V), C, H, W, n, th, tw, m, a)
    if rc != 0:
        raise RuntimeError(f"oracle_input_tile_transform failed ({rc})")
    return V


def winograd_conv3x3(x, w, bias=None, m: int = 2, points=None):
    """The convolution by F(m x m, 3 x 3): transforms, per-position products summed
    over channels, inverse transform, bias; fp64 throughout."""
    x, w = _f64(x), _f64(w)
    N, C, H, W = x.shape
    K = w.shape[0]
    assert w.shape == (K, C, 3, 3)
    b = _f64(bias) if bias is not None else None
    Bt, G, At = _mats_f64(m, points)
    y = np.full((N, K, H, W), np.nan, dtype=np.float64)
    rc = _load().oracle_winograd(_ptr(x), _ptr(w), _ptr(b), _ptr(y), N, C, H, W, K, m,
                                 _ptr(G), _ptr(Bt), _ptr(At))
    if rc != 0:
        raise RuntimeError(f"oracle_winograd failed ({rc})")
    return y


# --------------------------------------------------------------------------
# 8-bit transformed filters (the quantised operators of Section "Evaluation", "Operator Support")
# --------------------------------------------------------------------------
# Reading (the paper names no format; its host framework quantises weights to 8-bit integers with a scale per
# group): the transformed filter U is first rounded to fp16, as the fp16 path stores it; then every row
# U[pos][k][:] (one transform position, one output channel, all input channels) gets the scale s = max|U| / 127
# and every element becomes the integer q = round(U / s) in [-127, 127] (ties to even).  The contraction runs on
# the integers; s multiplies the sum over the channels.  The scale and the quotient are formed in fp32, the
# precision in which the library takes this decision (both are correctly rounded IEEE operations, so that numpy's
# float32 gives the same integers).

def quantize_filter_int8(U):
    """U: transformed filter [K, C, a, a] (fp64).  Returns (q, s): q[K, C, a, a] integers in [-127, 127] (as fp64)
    and the scales s[K, a, a] (fp32 values as fp64), so that the filter used is q * s."""
    U16 = np.asarray(U, dtype=np.float64).astype(np.float16).astype(np.float32)   # the fp16 path's filter
    amax = np.abs(U16).max(axis=1)                                                # [K, a, a]: over the input channels
    s = np.where(amax > 0, amax / np.float32(127.0), np.float32(1.0)).astype(np.float32)
    q = np.clip(np.rint(U16 / s[:, None, :, :]), -127.0, 127.0)                   # fp32 quotient, ties to even
    return q.astype(np.float64), s.astype(np.float64)


def winograd_conv3x3_q8(x, w, bias=None, m: int = 2, points=None):
    """The Winograd convolution with the 8-bit transformed filter defined above; everything else fp64."""
    x, w = _f64(x), _f64(w)
    N, C, H, W = x.shape
    K = w.shape[0]
    b = _f64(bias) if bias is not None else None
    Bt, G, At = _mats_f64(m, points)
    q, s = quantize_filter_int8(filter_transform(w, m, points))
    U = np.ascontiguousarray(q * s[:, None, :, :])
    y = np.full((N, K, H, W), np.nan, dtype=np.float64)
    rc = _load().oracle_winograd_with_filter(_ptr(x), _ptr(U), _ptr(b), _ptr(y), N, C, H, W, K, m, _ptr(Bt), _ptr(At))
    if rc != 0:
        raise RuntimeError(f"oracle_winograd_with_filter failed ({rc})")
    return y
