"""GPU parity of centralized error-compensated SGD (Section 1: g' = C[g + delta];
delta = (g + delta) - g'; x = x - gamma g') through the C ABI against the CPU
oracle: packed codes bit-exact, x, delta and scales within
max |gpu - ref| / max |ref| <= 1e-5 per node row and step, 1e-4 after 20
free-running steps."""
import numpy as np
import pytest

from paper_1907_07346_b200 import inputs as I
from test_gpu_parity import TOL_RUN, TOL_STEP, make_state, row_rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from oracle import oracle as orc
    from paper_1907_07346_b200 import binding as B
    from paper_1907_07346_b200 import build as libbuild
    libbuild.build()
    assert torch.cuda.is_available()
    B.lib()
    return torch, orc, B


def run_ecsgd(env, graph, N, kind, bits, chunk, noise, steps=1, seed=5, sigma=0.1, gamma=0.05,
              tol=TOL_STEP, given=False, zero_start=False, equal_rows=False, path=0):
    torch, orc, B = env
    ld = I.round_up(N, 4) + 8
    x, d, a, c = make_state(graph, N, ld, seed, zero_start=zero_start)
    if equal_rows:
        x[:, :N] = x[0, :N]
    ds = B.DeepSqueeze(graph, N, ld, kind, bits, chunk)
    ds.ds_set_path(path)          # 0: the fused kernel where the shape allows; 2: always two kernels
    dev = [torch.from_numpy(t.copy()).cuda() for t in (x, d, a, c)]
    rng = np.random.default_rng(seed + 1)
    for t in range(steps):
        if given:
            g = np.zeros((graph.n, ld), np.float32)
            g[:, :N] = rng.standard_normal((graph.n, N)).astype(np.float32)
            g[:, N:] = 11.0
            codes_ref, scales_ref = orc.ecsgd_step(graph, kind, bits, chunk, x, d, a, c, N, 0.0, I.NOISE_NONE,
                                                   gamma, 77 + seed, t, g_given=g)
            ds.ds_ecsgd_step_g(dev[0], dev[1], torch.from_numpy(g).cuda(), gamma, 77 + seed, t)
        else:
            codes_ref, scales_ref = orc.ecsgd_step(graph, kind, bits, chunk, x, d, a, c, N, sigma, noise,
                                                   gamma, 77 + seed, t)
            ds.ds_ecsgd_step(dev[0], dev[1], dev[2], dev[3], sigma, noise, gamma, 77 + seed, t)
        ds.ds_sync()
        gx, gd = dev[0].cpu().numpy(), dev[1].cpu().numpy()
        codes, scales = ds.codes_to_host()
        assert np.array_equal(codes, codes_ref), f"codes differ at step {t}"
        if kind != I.COMP_IDENTITY:
            assert row_rel_err(scales, scales_ref) <= tol
        ex, ed = row_rel_err(gx[:, :N], x[:, :N]), row_rel_err(gd[:, :N], d[:, :N])
        assert ex <= tol and ed <= tol, (t, ex, ed)
        assert np.array_equal(gx[:, N:], x[:, N:]) and np.array_equal(gd[:, N:], d[:, N:])
    ds.close()
    return dev[0].cpu().numpy()


COMPS = [(I.COMP_SIGN1_L1, 1, 128), (I.COMP_SIGN1_L1, 1, 0), (I.COMP_UNIFORM_STOCH_MAXABS, 2, 256),
         (I.COMP_UNIFORM_STOCH_MAXABS, 4, 512), (I.COMP_UNIFORM_STOCH_MAXABS, 4, 0),
         (I.COMP_UNIFORM_STOCH_MAXABS, 8, 64), (I.COMP_UNIFORM_NEAREST_L2, 4, 96), (I.COMP_IDENTITY, 32, 0),
         # the paper's codec at its own granularity (one norm per tensor) and on chunks several warps share
         (I.COMP_UNIFORM_NEAREST_L2, 4, 0), (I.COMP_UNIFORM_NEAREST_L2, 2, 1024)]


@pytest.mark.parametrize("path", [0, 2])
@pytest.mark.parametrize("comp", COMPS)
@pytest.mark.parametrize("noise", [I.NOISE_NONE, I.NOISE_GAUSS])
def test_parameter_server_steps(env, comp, noise, path):
    """Complete graph with W = 1/n (the parameter server); several tiles and a ragged tail."""
    kind, bits, chunk = comp
    run_ecsgd(env, I.complete(5), 512 * 5 + 40 + 3, kind, bits, chunk, noise, steps=3, path=path)


@pytest.mark.parametrize("path", [0, 2])
@pytest.mark.parametrize("comp", [(I.COMP_SIGN1_L1, 1, 1024), (I.COMP_UNIFORM_STOCH_MAXABS, 4, 512)])
def test_given_gradient(env, comp, path):
    kind, bits, chunk = comp
    run_ecsgd(env, I.complete(4), 4096 + 17, kind, bits, chunk, I.NOISE_NONE, steps=2, given=True, path=path)


def test_single_worker(env):
    """n = 1: the scheme exactly as the paper displays it."""
    run_ecsgd(env, I.complete(1), 3000, I.COMP_UNIFORM_STOCH_MAXABS, 2, 128, I.NOISE_GAUSS, steps=3)


@pytest.mark.parametrize("path", [0, 2])
def test_other_graphs_and_student_noise(env, path):
    run_ecsgd(env, I.ring(7), 2048 + 40, I.COMP_UNIFORM_STOCH_MAXABS, 2, 256, I.NOISE_STUDENT_T3, steps=2, path=path)
    run_ecsgd(env, I.torus(3, 4), 1500, I.COMP_SIGN1_L1, 1, 512, I.NOISE_GAUSS, steps=2, path=path)
    run_ecsgd(env, I.ring(16), 512 * 400 + 40, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, I.NOISE_GAUSS, steps=2, path=path)


def test_twenty_free_running_steps_and_equal_rows(env):
    """Free-running from x = delta = 0; with the complete graph every worker's
    copy of the model stays the same row."""
    for path in (0, 2):
        gx = run_ecsgd(env, I.complete(8), 65536 // 8 + 24, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, I.NOISE_GAUSS,
                       steps=20, tol=TOL_RUN, zero_start=True, path=path)
        assert np.array_equal(gx, np.broadcast_to(gx[0], gx.shape))


def test_deepsqueeze_step_unchanged_after_ecsgd(env):
    """The two iterations share one context: an EC-SGD step in between leaves
    the DeepSqueeze step's results as they are."""
    torch, orc, B = env
    g = I.ring(4)
    N, ld = 2048 + 40, 2096
    x, d, a, c = make_state(g, N, ld, 9)
    ds = B.DeepSqueeze(g, N, ld, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512)
    dev = [torch.from_numpy(t.copy()).cuda() for t in (x, d, a, c)]
    scratch = [t.clone() for t in dev[:2]]
    ds.ds_ecsgd_step(scratch[0], scratch[1], dev[2], dev[3], 0.1, I.NOISE_GAUSS, 0.05, 1, 0)
    codes_ref, _, _, _ = orc.step(g, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, x, d, a, c, N, 0.1, I.NOISE_GAUSS,
                                  0.05, 0.5, 1, 0)
    ds.ds_step(dev[0], dev[1], dev[2], dev[3], 0.1, I.NOISE_GAUSS, 0.05, 0.5, 1, 0)
    ds.ds_sync()
    codes, _ = ds.codes_to_host()
    assert np.array_equal(codes, codes_ref)
    assert row_rel_err(dev[0].cpu().numpy()[:, :N], x[:, :N]) <= TOL_STEP
    assert row_rel_err(dev[1].cpu().numpy()[:, :N], d[:, :N]) <= TOL_STEP
    ds.close()
