"""Pins of the oracle's centralized error-compensated SGD step (Section 1:
g' = C[g + delta]; delta = (g + delta) - g'; x = x - gamma g') against things
other than itself: a restatement of the three updates on top of the separately
pinned compressor, the uncompressed closed form, the telescoping identity of
error feedback, and the optimum of the averaged quadratic."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_1907_07346_b200 import inputs as I
from test_oracle_step import make_problem

COMPS = [(I.COMP_SIGN1_L1, 1), (I.COMP_UNIFORM_STOCH_MAXABS, 2), (I.COMP_UNIFORM_STOCH_MAXABS, 4),
         (I.COMP_UNIFORM_NEAREST_L2, 4)]


def gradient(x, a, c, sigma, noise, seed, step, N):
    """binary32 gradient of the synthetic objective, from the noise-stream helper."""
    g = np.zeros_like(x)
    for i in range(x.shape[0]):
        z = orc.noise_row(noise, seed, i, step, 0, N) if noise != I.NOISE_NONE else np.zeros(N, np.float32)
        d = (x[i, :N] - c[i, :N]).astype(np.float32)
        nz = (np.float32(sigma) * z).astype(np.float32)
        g[i, :N] = (a[i, :N].astype(np.float64) * d.astype(np.float64) + nz.astype(np.float64)).astype(np.float32)
    return g


@pytest.mark.parametrize("comp", COMPS)
@pytest.mark.parametrize("chunk", [0, 64])
def test_single_worker_is_the_three_displayed_updates(comp, chunk):
    """n = 1 (W = [1]): the scheme exactly as the paper displays it, rebuilt from
    numpy and the compressor primitive."""
    kind, bits = comp
    if kind == I.COMP_UNIFORM_NEAREST_L2 and chunk == 0:
        chunk = 96
    g1 = I.complete(1)
    N = 200
    x, d, a, c = make_problem(g1, N, 5)
    rng = np.random.default_rng(0)
    gamma, seed = 0.07, 31
    for t in range(4):
        g = rng.standard_normal((1, N)).astype(np.float32)
        v = (g + d).astype(np.float32)                            # g + delta
        ch = chunk if chunk else N
        Cv = np.zeros(N, np.float32)
        for k0 in range(0, N, ch):
            m = min(ch, N - k0)
            r = orc.rnd24_row(seed, 0, t, k0, m) if kind == I.COMP_UNIFORM_STOCH_MAXABS else None
            _, _, Cv[k0:k0 + m] = orc.compress_chunk(kind, bits, v[0, k0:k0 + m], r)
        d_ref = (v[0] - Cv).astype(np.float32)                    # remaining error
        x_ref = x[0].astype(np.float64) - gamma_f32(gamma) * Cv.astype(np.float64)   # server update
        orc.ecsgd_step(g1, kind, bits, chunk, x, d, a, c, N, 0.0, I.NOISE_NONE, gamma, seed, t, g_given=g)
        assert np.array_equal(d[0], d_ref)
        assert np.allclose(x[0], x_ref, rtol=0, atol=1e-6)


def gamma_f32(gamma):
    return float(np.float32(gamma))


def test_without_compression_it_is_minibatch_sgd_on_the_average_gradient():
    g8 = I.complete(8)
    N = 333
    x, d, a, c = make_problem(g8, N, 9, pad=3)
    x[:] = x[0]                                                   # one model, n copies
    d[:] = 0
    gamma, sigma, seed = 0.05, 0.2, 77
    for t in range(5):
        g = gradient(x, a, c, sigma, I.NOISE_GAUSS, seed, t, N)
        x_ref = x[0, :N].astype(np.float64) - gamma_f32(gamma) * g[:, :N].astype(np.float64).mean(axis=0)
        orc.ecsgd_step(g8, I.COMP_IDENTITY, 32, 0, x, d, a, c, N, sigma, I.NOISE_GAUSS, gamma, seed, t)
        assert np.all(d == 0)                                     # nothing is lost, nothing to compensate
        assert np.all(x[:, :N] == x[0, :N])                       # the copies stay one model
        assert np.allclose(x[0, :N], x_ref, rtol=0, atol=2e-6)
        assert np.all(x[:, N:] == 0)


@pytest.mark.parametrize("comp", COMPS)
def test_error_feedback_telescopes(comp):
    """Summing delta' = g + delta - C over T steps: sum_t C_t = sum_t g_t + delta_0 - delta_T,
    hence x_T = x_0 - gamma mean_i (sum_t g_it + delta_i0 - delta_iT)."""
    kind, bits = comp
    gr = I.complete(4)
    N, chunk, T = 256, 64, 25
    x, d, a, c = make_problem(gr, N, 13)
    x[:] = x[0]
    x0, d0 = x.astype(np.float64), d.astype(np.float64)
    rng = np.random.default_rng(3)
    gsum = np.zeros((4, N))
    gamma = 0.03
    for t in range(T):
        g = rng.standard_normal((4, N)).astype(np.float32)
        gsum += g
        orc.ecsgd_step(gr, kind, bits, chunk, x, d, a, c, N, 0.0, I.NOISE_NONE, gamma, 5, t, g_given=g)
    x_ref = x0[0] - gamma_f32(gamma) * (gsum + d0 - d.astype(np.float64)).mean(axis=0)
    assert np.all(x == x[0])
    assert np.allclose(x[0], x_ref, rtol=0, atol=2e-5)
    # and the compressor was really lossy
    assert np.abs(d).max() > 1e-3


def test_first_step_sends_the_compressed_gradient_plus_error():
    gr = I.complete(3)
    N, chunk = 130, 64
    x, d, a, c = make_problem(gr, N, 21)
    g = gradient(x, a, c, 0.1, I.NOISE_STUDENT_T3, 8, 2, N)
    v = (g + d).astype(np.float32)
    codes, scales = orc.ecsgd_step(gr, I.COMP_SIGN1_L1, 1, chunk, x, d, a, c, N, 0.1, I.NOISE_STUDENT_T3, 0.1, 8, 2)
    for i in range(3):
        q_all = np.zeros(N, np.uint32)
        for mi, k0 in enumerate(range(0, N, chunk)):
            m = min(chunk, N - k0)
            s, q, _ = orc.compress_chunk(I.COMP_SIGN1_L1, 1, v[i, k0:k0 + m])
            assert scales[i, mi] == np.float32(s)
            q_all[k0:k0 + m] = q
        assert np.array_equal(codes[i], orc.pack_codes(1, q_all))


@pytest.mark.parametrize("comp", [(I.COMP_SIGN1_L1, 1), (I.COMP_UNIFORM_STOCH_MAXABS, 2)])
def test_reaches_the_optimum_of_the_average_objective(comp):
    kind, bits = comp
    gr = I.complete(8)
    N = 128
    x, d, a, c = make_problem(gr, N, 4)
    x[:] = 0
    d[:] = 0
    xstar = (a.astype(np.float64) * c).sum(axis=0) / a.astype(np.float64).sum(axis=0)
    e0 = np.abs(x[0] - xstar).max()
    tail = []
    for t in range(600):
        orc.ecsgd_step(gr, kind, bits, 64, x, d, a, c, N, 0.0, I.NOISE_NONE, 0.05, 1, t)
        if t >= 500:
            tail.append(x[0].astype(np.float64))
    # the iterate jitters by O(gamma * scale) around x*, its time average sits on it
    assert np.abs(np.mean(tail, axis=0) - xstar).max() < 0.02 * e0
    assert np.abs(x[0] - xstar).max() < 0.2 * e0


def test_differs_from_the_decentralized_step():
    """Guards against routing one algorithm through the other."""
    gr = I.complete(4)
    N = 64
    x, d, a, c = make_problem(gr, N, 2)
    x2, d2 = x.copy(), d.copy()
    orc.ecsgd_step(gr, I.COMP_SIGN1_L1, 1, 0, x, d, a, c, N, 0.1, I.NOISE_GAUSS, 0.05, 3, 0)
    orc.step(gr, I.COMP_SIGN1_L1, 1, 0, x2, d2, a, c, N, 0.1, I.NOISE_GAUSS, 0.05, 1.0, 3, 0)
    assert np.abs(x - x2).max() > 1e-3 and np.abs(d - d2).max() > 1e-3
