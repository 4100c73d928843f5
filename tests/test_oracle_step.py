"""Pins for the oracle's iteration (Algorithm 1) against what the paper and the
mathematics fix.  CPU only."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle as orc
from paper_1907_07346_b200 import inputs as I

GOLD = os.path.join(os.path.dirname(__file__), "golden")

GRAPHS = {"ring4": I.ring(4), "ring8": I.ring(8), "torus3x4": I.torus(3, 4),
          "exp16": I.exponential(16)}
COMPS = [(I.COMP_SIGN1_L1, 1), (I.COMP_UNIFORM_STOCH_MAXABS, 2),
         (I.COMP_UNIFORM_STOCH_MAXABS, 4), (I.COMP_UNIFORM_STOCH_MAXABS, 8),
         (I.COMP_IDENTITY, 32), (I.COMP_UNIFORM_NEAREST_L2, 2), (I.COMP_UNIFORM_NEAREST_L2, 4)]


def make_problem(graph, N, seed, pad=0):
    rng = np.random.default_rng(seed)
    n = graph.n
    ld = N + pad
    a = np.zeros((n, ld), np.float32)
    c = np.zeros((n, ld), np.float32)
    a[:, :N] = rng.uniform(0.5, 2.0, size=(n, N))
    c[:, :N] = rng.standard_normal((n, N))
    x = np.zeros((n, ld), np.float32)
    d = np.zeros((n, ld), np.float32)
    x[:, :N] = 0.3 * rng.standard_normal((n, N))
    d[:, :N] = 0.05 * rng.standard_normal((n, N))
    return x, d, a, c


# ------------------------------------------------------------ the graphs
@pytest.mark.parametrize("g", [I.ring(3), I.ring(8), I.ring(16), I.torus(4, 8),
                               I.exponential(64), I.exponential(16)])
def test_W_symmetric_doubly_stochastic(g):
    """Assumption 1 (symmetric doubly stochastic W); every node is its own
    neighbour (Algorithm 1, receive step)."""
    W = g.dense()
    assert np.allclose(W, W.T, atol=0)
    assert np.allclose(W.sum(0), 1, atol=1e-6) and np.allclose(W.sum(1), 1, atol=1e-6)
    assert np.all(np.diag(W) > 0)
    for i in range(g.n):
        cols = g.col_idx[g.row_ptr[i]:g.row_ptr[i + 1]]
        assert np.all(np.diff(cols) > 0)


def test_graph_degrees_and_ring_spectrum():
    assert np.all(np.diff(I.ring(16).row_ptr) == 3)
    assert np.all(np.diff(I.torus(4, 8).row_ptr) == 5)
    assert np.all(np.diff(I.exponential(64).row_ptr) == 12)     # +32 and -32 coincide
    n = 8
    ev = np.sort(np.linalg.eigvalsh(I.ring(n).dense()))
    closed = np.sort((1 + 2 * np.cos(2 * np.pi * np.arange(n) / n)) / 3)
    assert np.allclose(ev, closed, atol=1e-6)


# -------------------------------------------------- the hand-worked case
def test_hand_case_ring4_sign():
    rows = {}
    for ln in open(os.path.join(GOLD, "hand_case_ring4_N8_sign.txt")):
        if ln.strip() and not ln.startswith("#"):
            t = ln.split()
            rows[(t[0], int(t[1]))] = t[2:]
    fr = lambda name, i: np.array([float(Fraction(v)) for v in rows[(name, i)]])
    g = I.ring(4)
    N = 8
    c = np.stack([fr("c", i) for i in range(4)]).astype(np.float32)
    a = np.ones((4, N), np.float32)
    x = np.zeros((4, N), np.float32)
    d = np.zeros((4, N), np.float32)
    codes, scales, v, Cv = orc.step(g, I.COMP_SIGN1_L1, 1, 0, x, d, a, c, N, 0.0, I.NOISE_NONE,
                                    0.5, 0.5, 1, 0, want_vC=True)
    for i in range(4):
        assert scales[i, 0] == fr("scale", i)[0]
        assert np.array_equal(Cv[i], fr("C", i))
        assert np.array_equal(d[i], fr("delta", i))
        assert np.allclose(x[i], fr("x", i), atol=1e-7, rtol=0)
        assert int(codes[i, 0]) == int(rows[("bits", i)][0], 16)


# ----------------------------------------- identities valid for any input
@pytest.mark.parametrize("gname", list(GRAPHS))
@pytest.mark.parametrize("comp", COMPS)
@pytest.mark.parametrize("chunk", [0, 32, 96])
def test_compression_identity_and_mean_preservation(gname, comp, chunk):
    """(a) C[v] + delta_new = v = x - gamma g + delta_old (Algorithm 1,
    compression step).  (b) The node average moves by the local steps only:
    mean_i x'_i = mean_i (x_i - gamma g_i), since 1^T (W - I) = 0 (proof of
    the key lemma, update of the averaged iterate)."""
    g = GRAPHS[gname]
    kind, bits = comp
    N = 200
    x, d, a, c = make_problem(g, N, 11, pad=8)
    x0, d0 = x.copy(), d.copy()
    sigma, gamma, eta, seed, t = 0.1, 0.05, 0.5, 42, 3
    codes, scales, v, Cv = orc.step(g, kind, bits, chunk, x, d, a, c, N, sigma, I.NOISE_GAUSS,
                                    gamma, eta, seed, t, want_vC=True)
    # independent float64 evaluation of v with the oracle's own noise
    z = np.stack([orc.noise_row(I.NOISE_GAUSS, seed, i, t, 0, N) for i in range(g.n)]).astype(np.float64)
    G = a[:, :N].astype(np.float64) * (x0[:, :N].astype(np.float64) - c[:, :N]) + sigma * z
    H = x0[:, :N].astype(np.float64) - gamma * G
    V = H + d0[:, :N]
    assert np.allclose(v, V, atol=2e-6, rtol=0)
    # (a)
    assert np.abs(Cv.astype(np.float64) + d[:, :N] - v).max() <= 2.4e-7 * max(1.0, np.abs(v).max())
    if kind == I.COMP_IDENTITY:
        assert np.all(d[:, :N] == 0)
    # (b)
    assert np.allclose(x[:, :N].astype(np.float64).mean(0), H.mean(0), atol=3e-6, rtol=0)
    # padding columns untouched
    assert np.all(x[:, N:] == x0[:, N:]) and np.all(d[:, N:] == d0[:, N:])


@pytest.mark.parametrize("gname", ["ring8", "torus3x4", "exp16"])
@pytest.mark.parametrize("comp", COMPS)
def test_dense_matrix_forms(gname, comp):
    """Section 3, matrix form: X' = X - gamma G + eta C (W - I), and the
    equivalent (X - gamma G) W_eff + (Delta_old - Delta_new)(W_eff - I) with
    W_eff = (1 - eta) I + eta W.  Nodes are rows here, so W acts from the left
    (W is symmetric)."""
    g = GRAPHS[gname]
    kind, bits = comp
    N = 64
    x, d, a, c = make_problem(g, N, 5)
    x0, d0 = x.astype(np.float64), d.astype(np.float64)
    sigma, gamma, eta, seed, t = 0.1, 0.02, 0.4, 7, 0
    codes, scales, v, Cv = orc.step(g, kind, bits, 32, x, d, a, c, N, sigma, I.NOISE_GAUSS,
                                    gamma, eta, seed, t, want_vC=True)
    W = g.dense()
    z = np.stack([orc.noise_row(I.NOISE_GAUSS, seed, i, t, 0, N) for i in range(g.n)]).astype(np.float64)
    G = a.astype(np.float64) * (x0 - c) + sigma * z
    form1 = x0 - gamma * G + eta * (W - np.eye(g.n)) @ Cv.astype(np.float64)
    assert np.allclose(x, form1, atol=2e-6, rtol=0)
    Weff = (1 - eta) * np.eye(g.n) + eta * W
    form2 = Weff @ (x0 - gamma * G) + (Weff - np.eye(g.n)) @ (d0 - d.astype(np.float64))
    assert np.allclose(x, form2, atol=3e-6, rtol=0)


def test_identity_compressor_is_dpsgd_closed_form():
    """With C the identity and X_0 = 0, X_t = -gamma sum_s G_s W_eff^(t-s)
    (Section 3.2, D-PSGD closed form)."""
    g = I.ring(8)
    N, T = 16, 6
    gamma, eta = 0.05, 0.5
    _, _, a, c = make_problem(g, N, 3)
    x = np.zeros((g.n, N), np.float32)
    d = np.zeros((g.n, N), np.float32)
    W = g.dense()
    Weff = (1 - eta) * np.eye(g.n) + eta * W
    Gs = []
    for t in range(T):
        Gs.append(a.astype(np.float64) * (x.astype(np.float64) - c))
        orc.step(g, I.COMP_IDENTITY, 32, 0, x, d, a, c, N, 0.0, I.NOISE_NONE, gamma, eta, 1, t)
        closed = np.zeros((g.n, N))
        for s in range(t + 1):
            closed -= gamma * np.linalg.matrix_power(Weff, t + 1 - s) @ Gs[s]
        assert np.allclose(x, closed, atol=1e-5, rtol=0)
        assert np.all(d == 0)


@pytest.mark.parametrize("comp", [(I.COMP_SIGN1_L1, 1), (I.COMP_IDENTITY, 32)])
def test_homogeneous_nodes_reduce_to_gradient_descent(comp):
    """Equal objectives on all nodes and a deterministic compressor give equal
    C_j, so the mixing term vanishes (rows of W - I sum to 0) and every node
    runs plain gradient descent: x_t = c (1 - (1 - gamma a)^t)."""
    g = I.torus(3, 3)
    N, T, gamma = 40, 25, 0.1
    rng = np.random.default_rng(2)
    a1 = rng.uniform(0.5, 2.0, N).astype(np.float32)
    c1 = rng.standard_normal(N).astype(np.float32)
    a = np.tile(a1, (g.n, 1))
    c = np.tile(c1, (g.n, 1))
    x = np.zeros((g.n, N), np.float32)
    d = np.zeros((g.n, N), np.float32)
    for t in range(T):
        orc.step(g, comp[0], comp[1], 0, x, d, a, c, N, 0.0, I.NOISE_NONE, gamma, 0.5, 1, t)
        closed = c1.astype(np.float64) * (1 - (1 - gamma * a1.astype(np.float64)) ** (t + 1))
        assert np.allclose(x, closed[None, :], atol=2e-5, rtol=0)
    assert np.isfinite(d).all()


@pytest.mark.parametrize("comp", [(I.COMP_SIGN1_L1, 1, 16), (I.COMP_UNIFORM_STOCH_MAXABS, 4, 32),
                                  (I.COMP_UNIFORM_STOCH_MAXABS, 2, 32)])
def test_average_follows_gradient_descent_and_reaches_optimum(comp):
    """The averaged iterate obeys xbar' = xbar - gamma gbar for any compressor
    (key lemma); on the quadratic (Eq. 1) it approaches the closed-form
    optimum x* = sum_i a_i c_i / sum_i a_i."""
    kind, bits, chunk = comp
    g = I.ring(8)
    N, T, gamma, eta = 64, 400, 0.05, 0.3
    _, _, a, c = make_problem(g, N, 9)
    x = np.zeros((g.n, N), np.float32)
    d = np.zeros((g.n, N), np.float32)
    xstar = (a.astype(np.float64) * c).sum(0) / a.astype(np.float64).sum(0)
    xbar = np.zeros(N)
    dist0 = np.linalg.norm(xstar)
    for t in range(T):
        gbar = (a.astype(np.float64) * (x.astype(np.float64) - c)).mean(0)
        xbar = x.astype(np.float64).mean(0) - gamma * gbar
        orc.step(g, kind, bits, chunk, x, d, a, c, N, 0.0, I.NOISE_NONE, gamma, eta, 3, t)
        assert np.allclose(x.astype(np.float64).mean(0), xbar, atol=5e-6, rtol=0)
    dist = np.linalg.norm(x.astype(np.float64).mean(0) - xstar)
    # A constant step leaves the O(gamma) bias of decentralized SGD with
    # heterogeneous nodes, whatever the compressor; see the next test for the
    # exact limit point.
    assert dist < 0.12 * dist0, (dist, dist0)
    assert np.abs(x - x.mean(0, keepdims=True)).max() < 2.0
    assert np.isfinite(d).all() and np.abs(d).max() < 10.0


def test_limit_point_is_decentralized_fixed_point():
    """Noise-free, identity compressor: the iteration X' = W_eff (X - gamma G(X))
    is linear on the quadratic, so its limit solves, per coordinate,
    (I - W_eff D) x = gamma W_eff (a * c) with D = diag(1 - gamma a).  The
    4-bit error-compensated run settles around the same point, and the limit's
    node average tends to the optimum x* of Eq. 1 as gamma shrinks."""
    g = I.ring(8)
    N, T, eta = 24, 1500, 0.5
    _, _, a, c = make_problem(g, N, 13)
    a64, c64 = a.astype(np.float64), c.astype(np.float64)
    xstar = (a64 * c64).sum(0) / a64.sum(0)
    Weff = (1 - eta) * np.eye(g.n) + eta * g.dense()
    gaps = []
    for gamma in (0.1, 0.025):
        fixed = np.zeros((g.n, N))
        for k in range(N):
            D = np.diag(1 - gamma * a64[:, k])
            fixed[:, k] = np.linalg.solve(np.eye(g.n) - Weff @ D, gamma * Weff @ (a64[:, k] * c64[:, k]))
        gaps.append(np.abs(fixed.mean(0) - xstar).max())
        if gamma == 0.1:
            x = np.zeros((g.n, N), np.float32)
            d = np.zeros((g.n, N), np.float32)
            for t in range(T):
                orc.step(g, I.COMP_IDENTITY, 32, 0, x, d, a, c, N, 0.0, I.NOISE_NONE, gamma, eta, 1, t)
            assert np.allclose(x, fixed, atol=2e-5, rtol=0)
            x = np.zeros((g.n, N), np.float32)
            d = np.zeros((g.n, N), np.float32)
            for t in range(T):
                orc.step(g, I.COMP_UNIFORM_STOCH_MAXABS, 4, 0, x, d, a, c, N, 0.0, I.NOISE_NONE,
                         gamma, eta, 1, t)
            assert np.abs(x - fixed).max() < 0.25
            assert np.abs(x.mean(0) - fixed.mean(0)).max() < 0.05
    assert gaps[1] < 0.5 * gaps[0]


def test_codes_and_scales_layout():
    """codes row = chunks packed back to back; scales one per (node, chunk),
    the tail chunk scaled by its true length."""
    g = I.ring(4)
    N, chunk = 200, 64          # chunks of 64, 64, 64, 8
    x, d, a, c = make_problem(g, N, 21)
    codes, scales, v, Cv = orc.step(g, I.COMP_SIGN1_L1, 1, chunk, x, d, a, c, N, 0.0,
                                    I.NOISE_NONE, 0.05, 0.5, 1, 0, want_vC=True)
    assert codes.shape == (4, 7) and scales.shape == (4, 4)
    for i in range(4):
        for m in range(4):
            seg = v[i, m * chunk:(m + 1) * chunk].astype(np.float64)
            assert scales[i, m] == np.float32(np.abs(seg).sum() / seg.shape[0])
        bits = np.unpackbits(codes[i].view(np.uint8), bitorder="little")[:N]
        assert np.array_equal(bits, (v[i] >= 0).astype(np.uint8))
        assert np.all(np.unpackbits(codes[i].view(np.uint8), bitorder="little")[N:] == 0)


def test_student_t_noise_enters_gradient():
    g = I.ring(4)
    N = 64
    x, d, a, c = make_problem(g, N, 8)
    x0, d0 = x.copy(), d.copy()
    codes, scales, v, Cv = orc.step(g, I.COMP_IDENTITY, 32, 0, x, d, a, c, N, 0.1,
                                    I.NOISE_STUDENT_T3, 0.05, 0.5, 5, 2, want_vC=True)
    z = np.stack([orc.noise_row(I.NOISE_STUDENT_T3, 5, i, 2, 0, N) for i in range(4)]).astype(np.float64)
    G = a.astype(np.float64) * (x0.astype(np.float64) - c) + 0.1 * z
    assert np.allclose(v, x0 - 0.05 * G + d0, atol=2e-6, rtol=0)


@pytest.mark.parametrize("comp", [(I.COMP_SIGN1_L1, 1), (I.COMP_UNIFORM_STOCH_MAXABS, 4)])
def test_column_window_equals_slice_of_whole_problem(comp):
    """Chunks are independent columns: running the iteration on the columns
    [k_first, k_first + n_cols) alone (random streams indexed by the global
    column) reproduces that slice of the whole-problem result bit for bit."""
    g = I.ring(8)
    chunk, N = 64, 64 * 7 + 10
    x, d, a, c = make_problem(g, N, 17)
    xw, dw = x.copy(), d.copy()
    codes, scales, _, _ = orc.step(g, comp[0], comp[1], chunk, x, d, a, c, N, 0.1, I.NOISE_GAUSS,
                                   0.05, 0.5, 4, 6)
    for k_first, n_cols in ((0, 128), (128, 192), (384, N - 384)):
        sl = slice(k_first, k_first + n_cols)
        xs, dsl = np.ascontiguousarray(xw[:, sl]), np.ascontiguousarray(dw[:, sl])
        cw, sw, _, _ = orc.step(g, comp[0], comp[1], chunk, xs, dsl,
                                np.ascontiguousarray(a[:, sl]), np.ascontiguousarray(c[:, sl]),
                                n_cols, 0.1, I.NOISE_GAUSS, 0.05, 0.5, 4, 6, k_first=k_first)
        assert np.array_equal(xs, x[:, sl]) and np.array_equal(dsl, d[:, sl])
        assert np.array_equal(sw, scales[:, k_first // chunk:k_first // chunk + sw.shape[1]])
        w0 = k_first * comp[1] // 32
        assert np.array_equal(cw, codes[:, w0:w0 + cw.shape[1]])


@pytest.mark.parametrize("comp", [(I.COMP_SIGN1_L1, 1, 32), (I.COMP_UNIFORM_STOCH_MAXABS, 4, 64),
                                  (I.COMP_IDENTITY, 32, 0)])
def test_given_gradient_reproduces_synthetic_step(comp):
    """Algorithm 1 takes any stochastic gradient.  Feeding the iteration the
    gradient of the synthetic objective, evaluated outside (a (x - c) + sigma z
    in binary32, the product-sum with one rounding), must reproduce the
    synthetic step bit for bit; and the identities hold for an arbitrary g."""
    kind, bits, chunk = comp
    g = I.torus(3, 4)
    N = 150
    x, d, a, c = make_problem(g, N, 23, pad=2)
    x2, d2 = x.copy(), d.copy()
    sigma, gamma, eta, seed, t = 0.1, 0.05, 0.5, 9, 4
    z = np.zeros_like(x)
    for i in range(g.n):
        z[i, :N] = orc.noise_row(I.NOISE_GAUSS, seed, i, t, 0, N)
    dd = (x - c).astype(np.float32)
    nz = (np.float32(sigma) * z).astype(np.float32)
    grad = (a.astype(np.float64) * dd.astype(np.float64) + nz.astype(np.float64)).astype(np.float32)
    ref = orc.step(g, kind, bits, chunk, x, d, a, c, N, sigma, I.NOISE_GAUSS, gamma, eta, seed, t)
    got = orc.step(g, kind, bits, chunk, x2, d2, a, c, N, 0.0, I.NOISE_NONE, gamma, eta, seed, t,
                   g_given=grad)
    assert np.array_equal(x, x2) and np.array_equal(d, d2)
    assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])
    # arbitrary gradient: compression identity and mean preservation
    rng = np.random.default_rng(3)
    x3, d3, _, _ = make_problem(g, N, 24)
    x0, d0 = x3.copy(), d3.copy()
    grad = rng.standard_normal(x3.shape).astype(np.float32)
    _, _, v, Cv = orc.step(g, kind, bits, chunk, x3, d3, x3 * 0, x3 * 0, N, 0.0, I.NOISE_NONE, gamma, eta,
                           seed, t, want_vC=True, g_given=grad)
    H = x0.astype(np.float64) - gamma * grad
    assert np.allclose(v, H + d0, atol=2e-6, rtol=0)
    assert np.abs(Cv.astype(np.float64) + d3 - v).max() <= 2.4e-7 * max(1.0, np.abs(v).max())
    assert np.allclose(x3.astype(np.float64).mean(0), H.mean(0), atol=3e-6, rtol=0)


@pytest.mark.parametrize("bits", [2, 4])
def test_one_norm_per_tensor(bits):
    """Section 5, "Compression": b bits per element and ONE Euclidean norm per
    tensor, to which the receiver rescales what it decodes.  With chunk = 0
    the whole row of a node is the tensor: the scalar sent is ||v_i||_2
    (recomputed here in binary64 from v), the decoded C_i has that norm, the
    codes are the nearest of the 2^b levels spanning [-max|v_i|, max|v_i|], and
    C_i is a positive multiple of the decoded levels."""
    g = I.ring(8)
    N = 1000
    x, d, a, c = make_problem(g, N, 5)
    codes, scales, v, Cv = orc.step(g, I.COMP_UNIFORM_NEAREST_L2, bits, 0, x, d, a, c, N, 0.1,
                                    I.NOISE_GAUSS, 0.05, 0.5, 9, 2, want_vC=True)
    assert scales.shape == (8, 1)
    L = (1 << bits) - 1
    for i in range(8):
        v64 = v[i].astype(np.float64)
        assert abs(scales[i, 0] - np.sqrt((v64 ** 2).sum())) <= 1e-6 * scales[i, 0]
        assert abs(np.sqrt((Cv[i].astype(np.float64) ** 2).sum()) - scales[i, 0]) <= 2e-6 * scales[i, 0]
        q = np.zeros(N, np.int64)
        for k in range(N):
            q[k] = (int(codes[i, (k * bits) // 32]) >> ((k * bits) % 32)) & L
        gmax = np.abs(v64).max()
        levels = (2.0 * q - L) / L
        # nearest level: no other level is closer to v / max|v| (up to the rounding of the quotient)
        grid = (2.0 * np.arange(L + 1) - L) / L
        best = np.abs(v64[:, None] / gmax - grid[None, :]).min(axis=1)
        assert np.all(np.abs(v64 / gmax - levels) <= best + 1e-6)
        ratio = Cv[i].astype(np.float64) / levels
        assert np.all(ratio > 0) and np.ptp(ratio) <= 1e-6 * ratio.mean()
