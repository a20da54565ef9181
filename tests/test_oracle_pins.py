"""Pins for the fp64 oracle: facts fixed by the mathematics, by hand arithmetic, by brute
force and by library routines -- none of them produced by the oracle itself or by the
CUDA path."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

LAVIN_F4_BT = [[4, 0, -5, 0, 1, 0], [0, -4, -4, 1, 1, 0], [0, 4, -4, -1, 1, 0],
               [0, -2, -1, 2, 1, 0], [0, 2, -1, -2, 1, 0], [0, 4, 0, -5, 0, 1]]
POINT_SETS_F4 = [
    None,
    (0, 1, -1, 2, Fraction(-1, 2)),
    (0, Fraction(1, 2), Fraction(-1, 2), Fraction(3, 2), Fraction(-3, 2)),
    (0, Fraction(7, 10), Fraction(-7, 10), Fraction(7, 5), Fraction(-7, 5)),
    (0, Fraction(3, 4), Fraction(-3, 4), Fraction(3, 2), Fraction(-3, 2)),   # the set the CUDA kernels use
]


def _identity_holds(m, points):
    Bt, G, At = oracle.winograd_matrices(m, points)
    a = m + 2
    for i in range(m):
        for u in range(3):
            for s in range(a):
                tot = sum(At[i][x] * G[x][u] * Bt[x][s] for x in range(a))
                if tot != (1 if s == i + u else 0):
                    return False
    return True


@pytest.mark.parametrize("m,points", [(2, None), (2, (0, 1, -1)), (2, (0, 2, Fraction(-1, 3)))]
                         + [(4, p) for p in POINT_SETS_F4])
def test_matrices_exact_identity(m, points):
    # sum_x At[i][x] G[x][u] Bt[x][s] == [s == i+u] in exact rationals: this alone implies the
    # 1-D (and by separability 2-D) algorithm equals correlation.
    assert _identity_holds(m, points)


def test_generated_f4_matches_textbook_matrix_up_to_row_scaling():
    # With points {0, +-1, +-2, inf} the generated B^T must be the well-known integer matrix up to
    # one scale per row (the inverse scale sits in G).
    Bt, G, At = oracle.winograd_matrices(4, None)
    for row, ref in zip(Bt, LAVIN_F4_BT):
        nz = [(r, q) for r, q in zip(row, ref) if q != 0]
        ratio = nz[0][0] / nz[0][1]
        assert ratio != 0
        assert all(r == ratio * q for r, q in zip(row, ref))


def test_f23_four_multiply_closed_form():
    # 1-D F(2,3): m1=(d0-d2)g0, m2=(d1+d2)(g0+g1+g2)/2, m3=(d2-d1)(g0-g1+g2)/2, m4=(d1-d3)g2;
    # y0=m1+m2+m3, y1=m2-m3-m4.  The matrices must reproduce exactly these four products.
    Bt, G, At = oracle.winograd_matrices(2)
    d = [Fraction(3), Fraction(-7), Fraction(5), Fraction(11)]
    g = [Fraction(2), Fraction(-3), Fraction(1, 3)]
    V = [sum(Bt[x][s] * d[s] for s in range(4)) for x in range(4)]
    U = [sum(G[x][u] * g[u] for u in range(3)) for x in range(4)]
    prods = [U[x] * V[x] for x in range(4)]
    m1 = (d[0] - d[2]) * g[0]
    m2 = (d[1] + d[2]) * (g[0] + g[1] + g[2]) / 2
    m3 = (d[2] - d[1]) * (g[0] - g[1] + g[2]) / 2
    m4 = (d[1] - d[3]) * g[2]
    assert prods == [m1, m2, m3, m4]
    y = [sum(At[i][x] * prods[x] for x in range(4)) for i in range(2)]
    assert y == [m1 + m2 + m3, m2 - m3 - m4]
    assert y == [d[0] * g[0] + d[1] * g[1] + d[2] * g[2], d[1] * g[0] + d[2] * g[1] + d[3] * g[2]]


# Hand-worked example: x = 1..16 row-major (4x4), w = 1..9 row-major, bias 0.5.
# y[0][0] = 1*5 + 2*6 + 5*8 + 6*9 + 0.5 = 111.5 (taps that fall on the padding vanish);
# y[1][1] = sum_{u,v} x[u][v]*w[u][v] over the top-left 3x3 block
#         = 1*1+2*2+3*3 + 5*4+6*5+7*6 + 9*7+10*8+11*9 + 0.5 = 348.5;
# y[3][3] = 11*1+12*2 + 15*4+16*5 + 0.5 = 175.5.
HAND_Y = np.array([[111.5, 178.5, 217.5, 145.5], [231.5, 348.5, 393.5, 252.5],
                   [363.5, 528.5, 573.5, 360.5], [197.5, 274.5, 295.5, 175.5]])


def _load_golden(name):
    """Sections of a text fixture under tests/golden/ as float64 matrices ('#' lines are the citation)."""
    import os
    out, cur = {}, None
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("["):
                cur = line.strip("[]")
                out[cur] = []
            else:
                out[cur].append([float(v) for v in line.split()])
    return {k: np.array(v) for k, v in out.items()}


def test_golden_fixture_matches_the_inline_hand_values():
    g = _load_golden("hand_worked_4x4.txt")
    assert np.array_equal(g["y"], HAND_Y)
    x, w, b = _hand_inputs()
    assert np.array_equal(oracle.direct_conv3x3(x, w, b)[0, 0], g["y"])
    assert np.array_equal(oracle.filter_transform(w, 2)[0, 0], g["U"])
    assert np.array_equal(oracle.input_tile_transform(x, 0, 0, 0, 2)[0], g["V_tile00"])


def _hand_inputs():
    x = np.arange(1, 17, dtype=np.float64).reshape(1, 1, 4, 4)
    w = np.arange(1, 10, dtype=np.float64).reshape(1, 1, 3, 3)
    return x, w, np.array([0.5])


def test_hand_worked_values_direct_and_winograd():
    x, w, b = _hand_inputs()
    assert np.array_equal(oracle.direct_conv3x3(x, w, b)[0, 0], HAND_Y)
    assert np.array_equal(oracle.brute_conv3x3(x, w, b)[0, 0], HAND_Y)
    np.testing.assert_allclose(oracle.winograd_conv3x3(x, w, b, m=2)[0, 0], HAND_Y, rtol=0, atol=1e-12)
    for pts in POINT_SETS_F4:
        np.testing.assert_allclose(oracle.winograd_conv3x3(x, w, b, m=4, points=pts)[0, 0], HAND_Y,
                                   rtol=0, atol=1e-10)


def test_hand_worked_intermediates_f2():
    # U = G w G^T and the first tile's V = B^T d B, multiplied out by hand:
    # G w = [[1,2,3],[6,7.5,9],[2,2.5,3],[7,8,9]]; (G w) G^T row 0 = [1, 3, 1, 3].
    x, w, b = _hand_inputs()
    U = oracle.filter_transform(w, 2)[0, 0]
    assert np.array_equal(U, np.array([[1, 3, 1, 3], [6, 11.25, 3.75, 9], [2, 3.75, 1.25, 3], [7, 12, 4, 9]]))
    # tile (0,0): d rows [0 0 0 0],[0 1 2 3],[0 5 6 7],[0 9 10 11];
    # B^T d = [[0,-5,-6,-7],[0,6,8,10],[0,4,4,4],[0,-8,-8,-8]]; times B gives V below.
    V = oracle.input_tile_transform(x, 0, 0, 0, 2)[0]
    assert np.array_equal(V, np.array([[6, -11, -1, 2], [-8, 14, 2, -4], [-4, 8, 0, 0], [8, -16, 0, 0]]))


@pytest.mark.parametrize("u,v", [(0, 0), (0, 2), (1, 1), (2, 1), (2, 2)])
def test_shifted_delta_filter_is_a_shift(u, v):
    # w[u][v] = 1 alone  =>  y[i][j] = xhat[i+u-1][j+v-1]: pins "no flip" and the zero padding.
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 3, 5, 7))
    w = np.zeros((3, 3, 3, 3))
    for c in range(3):
        w[c, c, u, v] = 1.0
    xp = np.pad(x, ((0, 0), (0, 0), (1, 1), (1, 1)))
    want = xp[:, :, u:u + 5, v:v + 7]
    assert np.array_equal(oracle.direct_conv3x3(x, w), want)
    np.testing.assert_allclose(oracle.winograd_conv3x3(x, w, m=2), want, atol=1e-13)
    np.testing.assert_allclose(oracle.winograd_conv3x3(x, w, m=4), want, atol=1e-11)


def test_delta_example_from_hand():
    # (u,v) = (0,2) on the 4x4 ramp: y[i][j] = xhat[i-1][j+1]; row 0 and column 3 are zero, y[1][0] = 2.
    x, _, _ = _hand_inputs()
    w = np.zeros((1, 1, 3, 3)); w[0, 0, 0, 2] = 1
    y = oracle.direct_conv3x3(x, w)[0, 0]
    assert np.all(y[0] == 0) and np.all(y[:, 3] == 0) and y[1, 0] == 2 and y[3, 2] == 12


@pytest.mark.parametrize("H,W,want", [
    (4, 4, [[4, 6, 6, 4], [6, 9, 9, 6], [6, 9, 9, 6], [4, 6, 6, 4]]),
    (3, 5, [[4, 6, 6, 6, 4], [6, 9, 9, 9, 6], [4, 6, 6, 6, 4]]),
    (1, 1, [[1]]),
    (1, 3, [[2, 3, 2]]),
])
def test_all_ones_counts_inbounds_taps(H, W, want):
    x = np.ones((1, 1, H, W)); w = np.ones((1, 1, 3, 3))
    assert np.array_equal(oracle.direct_conv3x3(x, w)[0, 0], np.array(want, dtype=float))
    np.testing.assert_allclose(oracle.winograd_conv3x3(x, w, m=2)[0, 0], want, atol=1e-13)
    np.testing.assert_allclose(oracle.winograd_conv3x3(x, w, m=4)[0, 0], want, atol=1e-11)


def test_channel_sum_and_bias():
    # all-ones over C channels multiplies the tap count by C; bias is added once per output.
    x = np.ones((1, 5, 4, 4)); w = np.ones((2, 5, 3, 3)); b = np.array([0.25, -3.0])
    y = oracle.direct_conv3x3(x, w, b)
    assert y[0, 0, 1, 1] == 45.25 and y[0, 1, 0, 0] == 17.0


@pytest.mark.parametrize("shape", [(1, 1, 4, 4, 1), (2, 3, 5, 4, 2), (1, 2, 1, 1, 3), (1, 4, 3, 7, 1),
                                   (1, 7, 2, 9, 3)])
def test_brute_force_tiny(shape):
    N, C, H, W, K = shape
    rng = np.random.default_rng(sum(shape))
    x = rng.standard_normal((N, C, H, W)); w = rng.standard_normal((K, C, 3, 3)); b = rng.standard_normal(K)
    want = oracle.brute_conv3x3(x, w, b)
    np.testing.assert_allclose(oracle.direct_conv3x3(x, w, b), want, rtol=0, atol=1e-13 * np.abs(want).max())
    np.testing.assert_allclose(oracle.winograd_conv3x3(x, w, b, m=2), want, rtol=0,
                               atol=1e-12 * np.abs(want).max())


SHAPES_X = [(1, 1, 4, 4, 1), (2, 3, 7, 5, 4), (1, 33, 9, 12, 7), (3, 4, 1, 1, 3), (1, 7, 3, 2, 33),
            (1, 5, 17, 31, 2), (2, 16, 8, 8, 16), (1, 3, 6, 10, 1), (1, 2, 13, 1, 2)]


@pytest.mark.parametrize("shape", SHAPES_X)
@pytest.mark.parametrize("m,points", [(2, None)] + [(4, p) for p in POINT_SETS_F4])
def test_winograd_equals_direct(shape, m, points):
    N, C, H, W, K = shape
    rng = np.random.default_rng(7 + sum(shape))
    x = rng.standard_normal((N, C, H, W)); w = rng.standard_normal((K, C, 3, 3)); b = rng.standard_normal(K)
    d = oracle.direct_conv3x3(x, w, b)
    y = oracle.winograd_conv3x3(x, w, b, m=m, points=points)
    assert not np.isnan(y).any()          # every in-range output was written
    assert np.abs(y - d).max() <= 1e-10 * np.abs(d).max()


@pytest.mark.parametrize("shape", SHAPES_X)
def test_direct_matches_library_routines(shape):
    N, C, H, W, K = shape
    rng = np.random.default_rng(11 + sum(shape))
    x = rng.standard_normal((N, C, H, W)); w = rng.standard_normal((K, C, 3, 3)); b = rng.standard_normal(K)
    d = oracle.direct_conv3x3(x, w, b)
    t = torch.nn.functional.conv2d(torch.from_numpy(x), torch.from_numpy(w), torch.from_numpy(b), padding=1)
    assert np.abs(d - t.numpy()).max() <= 1e-12 * np.abs(d).max()
    from scipy.signal import correlate2d
    for n in range(N):
        for k in range(min(K, 2)):
            s = sum(correlate2d(x[n, c], w[k, c], mode="same", boundary="fill") for c in range(C)) + b[k]
            assert np.abs(d[n, k] - s).max() <= 1e-12 * np.abs(d).max()


def test_direct_channel_subset_matches_full():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 6, 9, 7)); w = rng.standard_normal((8, 6, 3, 3)); b = rng.standard_normal(8)
    full = oracle.direct_conv3x3(x, w, b)
    sub = oracle.direct_conv3x3(x, w, b, channels=[5, 0, 7])
    assert np.array_equal(sub, full[:, [5, 0, 7]])


def test_linearity_and_impulse_translation():
    rng = np.random.default_rng(3)
    x1 = rng.standard_normal((1, 2, 6, 6)); x2 = rng.standard_normal((1, 2, 6, 6))
    w = rng.standard_normal((2, 2, 3, 3))
    y = oracle.direct_conv3x3(2 * x1 - 3 * x2, w)
    np.testing.assert_allclose(y, 2 * oracle.direct_conv3x3(x1, w) - 3 * oracle.direct_conv3x3(x2, w), atol=1e-12)
    # an interior impulse at (r,s) stamps the flipped filter around it: y[r+1-u][s+1-v] = w[u][v]
    x = np.zeros((1, 1, 7, 7)); x[0, 0, 3, 2] = 1
    w1 = rng.standard_normal((1, 1, 3, 3))
    y = oracle.direct_conv3x3(x, w1)[0, 0]
    for u in range(3):
        for v in range(3):
            assert y[3 + 1 - u, 2 + 1 - v] == w1[0, 0, u, v]
    assert np.count_nonzero(y) == 9


def test_fp16_inputs_widen_exactly():
    x = torch.randn(1, 3, 5, 5).half(); w = torch.randn(2, 3, 3, 3).half()
    y16 = oracle.direct_conv3x3(x.numpy(), w.numpy())
    y64 = oracle.direct_conv3x3(x.double().numpy(), w.double().numpy())
    assert np.array_equal(y16, y64)


# ---- the epilogue the library can fuse after the convolution -------------------------------------------------

def test_silu_known_values_identities_and_library_routine():
    # sigmoid(0) = 1/2, sigmoid(ln 3) = 3/4, sigmoid(-ln 3) = 1/4: exact rationals
    assert oracle.silu(0.0) == 0.0
    assert abs(oracle.silu(np.log(3.0)) - 0.75 * np.log(3.0)) < 1e-15
    assert abs(oracle.silu(-np.log(3.0)) + 0.25 * np.log(3.0)) < 1e-15
    z = np.linspace(-30, 30, 2001)
    # silu(z) - silu(-z) = z (sigmoid(z) + sigmoid(-z) = 1); limits z and 0
    assert np.abs(oracle.silu(z) - oracle.silu(-z) - z).max() < 1e-13
    assert abs(oracle.silu(40.0) - 40.0) < 1e-14 and abs(oracle.silu(-40.0)) < 1e-15
    assert oracle.silu(-1e4) == 0.0                       # exp overflows: the limit, not NaN
    # minimum of z*sigmoid(z): -0.27846454276107379 at z = -1.2784645427610738
    assert abs(oracle.silu(z).min() + 0.27846454276107379) < 1e-4
    import torch
    t = torch.nn.functional.silu(torch.from_numpy(z)).numpy()
    assert np.abs(oracle.silu(z) - t).max() < 1e-14


def test_epilogue_adds_the_residual_before_the_activation():
    rng = np.random.default_rng(5)
    conv = rng.standard_normal((2, 3, 4, 5))
    res = rng.standard_normal((2, 3, 4, 5))
    assert np.array_equal(oracle.epilogue(conv), conv)
    assert np.array_equal(oracle.epilogue(conv, res) - res, (conv + res) - res)
    assert np.array_equal(oracle.epilogue(conv, -conv, "silu"), np.zeros_like(conv))       # silu(0) = 0
    y = oracle.epilogue(conv, res, "silu")
    zz = conv + res
    assert np.abs(y * (1.0 + np.exp(-zz)) - zz).max() < 1e-14                              # y (1 + e^-z) = z
    with pytest.raises(ValueError):
        oracle.epilogue(conv, None, "relu")


# ---------------------------------------------------------------------------------------------------------------
# 8-bit transformed filters (integers with one scale per transform position and output channel)
# ---------------------------------------------------------------------------------------------------------------
def test_int8_filter_quantisation_hand_values_ties_and_bounds():
    # one output channel, five input channels, at every position the row (1, -0.5, 0.25, 63.5/127, 0): the scale is
    # 1/127, so the quotients are 127, -63.5 (a tie: to the even -64), 31.75 (32), 63.5 (a tie: to the even 64), 0
    a = 4
    row = np.array([1.0, -0.5, 0.25, 0.5, 0.0])
    U = np.broadcast_to(row[None, :, None, None], (1, 5, a, a)).copy()
    q, s = oracle.quantize_filter_int8(U)
    assert np.array_equal(q[0, :, 0, 0], [127, -64, 32, 64, 0]) and np.array_equal(q[0, :, 3, 2], [127, -64, 32, 64, 0])
    assert np.all(s == np.float64(np.float32(1.0) / np.float32(127.0)))
    # a zero row keeps scale 1 and zeros; the sign of a row flips the integers
    z, sz = oracle.quantize_filter_int8(np.zeros((2, 3, a, a)))
    assert not z.any() and np.all(sz == 1.0)
    qn, sn = oracle.quantize_filter_int8(-U)
    assert np.array_equal(qn, -q) and np.array_equal(sn, s)
    rng = np.random.default_rng(5)
    w = (rng.standard_normal((7, 50, 3, 3)) / np.sqrt(450)).astype(np.float16).astype(np.float64)
    for m, pts in [(2, None), (4, (0, 0.75, -0.75, 1.5, -1.5))]:
        U = oracle.filter_transform(w, m, pts)
        U16 = U.astype(np.float16).astype(np.float64)
        q, s = oracle.quantize_filter_int8(U)
        assert np.array_equal(q, np.rint(q)) and np.abs(q).max() == 127
        assert np.all(np.abs(q).max(axis=1) == 127)                               # the largest element of every row
        assert np.all(np.abs(q * s[:, None] - U16) <= 0.50002 * s[:, None])         # nearest integer (the quotient is an fp32 value)
        # torch's float32 division and rounding (a library routine) give the same integers
        t16 = torch.from_numpy(U16).float()
        ts = torch.from_numpy(s).float()
        assert np.array_equal(torch.round(t16 / ts[:, None]).double().numpy(), q)


def test_int8_filter_convolution_is_close_to_the_exact_one_but_not_equal():
    rng = np.random.default_rng(3)
    w = (rng.standard_normal((6, 40, 3, 3)) / np.sqrt(360)).astype(np.float16).astype(np.float64)
    x = rng.standard_normal((1, 40, 9, 10))
    exact = oracle.direct_conv3x3(x, w)
    for m, pts, hi in [(2, None, 2.5e-2), (4, (0, 0.75, -0.75, 1.5, -1.5), 8e-2)]:
        yq = oracle.winograd_conv3x3_q8(x, w, None, m, pts)
        rel = np.abs(yq - exact).max() / np.abs(exact).max()
        assert 1e-4 < rel < hi, (m, rel)
    # with a filter whose transformed rows are integers times a common power of two the quantisation is exact:
    # w = delta at the centre tap gives U = G e G^T, entries in {0, 1/4, 1/2, 1} for F(2x2)
    wd = np.zeros((2, 3, 3, 3))
    wd[0, 0, 1, 1] = 1.0
    wd[1, 2, 1, 1] = -2.0
    xs = rng.standard_normal((1, 3, 6, 8))
    yq = oracle.winograd_conv3x3_q8(xs, wd, None, 2, None)
    # scale = 1/127 is not a power of two, so "exact" means: to the rounding of 127 * (1/127) in fp32
    assert np.abs(yq - oracle.direct_conv3x3(xs, wd)).max() <= 1e-6 * np.abs(xs).max() * 2


# ---------------------------------------------------------------------------------------------------------------
# strided direct convolution (the downsampling convolutions)
# ---------------------------------------------------------------------------------------------------------------
def test_strided_direct_conv_is_the_subsampled_stride_1_result_and_matches_torch():
    rng = np.random.default_rng(12)
    for (N, C, K, H, W) in [(1, 1, 1, 4, 4), (2, 3, 4, 7, 10), (1, 5, 2, 8, 5), (1, 2, 3, 1, 6)]:
        x = rng.standard_normal((N, C, H, W))
        w = rng.standard_normal((K, C, 3, 3))
        b = rng.standard_normal(K)
        y1 = oracle.direct_conv3x3(x, w, b)                      # pinned above by hand values, brute force, torch, scipy
        assert np.array_equal(oracle.direct_conv3x3_strided(x, w, b, 1), y1)
        for s in (2, 3):
            ys = oracle.direct_conv3x3_strided(x, w, b, s)
            assert ys.shape == (N, K, (H - 1) // s + 1, (W - 1) // s + 1)
            assert np.array_equal(ys, y1[:, :, ::s, ::s])         # output (i, j) of stride s is output (s i, s j) of stride 1
            ref = torch.nn.functional.conv2d(torch.from_numpy(x), torch.from_numpy(w), torch.from_numpy(b), stride=s, padding=1)
            assert np.abs(ys - ref.numpy()).max() <= 1e-12


def test_strided_direct_conv_hand_worked_values():
    # 1 x 1 x 4 x 4 input 1..16, all-ones filter, stride 2: output (i, j) sums the window centred at (2i, 2j):
    # (0,0): rows 0-1, cols 0-1 -> 1+2+5+6 = 14; (0,1): rows 0-1, cols 1-3 -> 2+3+4+6+7+8 = 30;
    # (1,0): rows 1-3, cols 0-1 -> 5+6+9+10+13+14 = 57; (1,1): rows 1-3, cols 1-3 -> 6+7+8+10+11+12+14+15+16 = 99
    x = np.arange(1, 17, dtype=np.float64).reshape(1, 1, 4, 4)
    w = np.ones((1, 1, 3, 3))
    y = oracle.direct_conv3x3_strided(x, w, None, 2)
    assert y.reshape(-1).tolist() == [14.0, 30.0, 57.0, 99.0]
