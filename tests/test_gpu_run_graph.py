"""GPU tests of ds_run: T iterations of Algorithm 1 with a learning-rate
schedule (Section 5), replayed as one CUDA graph, against the CPU oracle and
against T single-step calls."""
import numpy as np
import pytest

from paper_1907_07346_b200 import inputs as I
from test_gpu_parity import env, make_state, row_rel_err, TOL_RUN  # noqa: F401  (env is a fixture)

pytestmark = pytest.mark.gpu

CASES = {
    "per_node_sign_ring4": (I.ring(4), 65_536, I.COMP_SIGN1_L1, 1, 0, I.NOISE_GAUSS),
    "per_node_4bit_ring4": (I.ring(4), 3000, I.COMP_UNIFORM_STOCH_MAXABS, 4, 0, I.NOISE_GAUSS),
    "chunk512_4bit_ring16": (I.ring(16), 512 * 5 + 40, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, I.NOISE_GAUSS),
    "chunk1024_sign_torus": (I.torus(4, 8), 1024 * 3 + 130, I.COMP_SIGN1_L1, 1, 1024, I.NOISE_STUDENT_T3),
    "chunk256_norm2_exp16": (I.exponential(16), 256 * 9 + 8, I.COMP_UNIFORM_NEAREST_L2, 2, 256, I.NOISE_NONE),
    # one norm per tensor: five launches per iteration in the graph
    "per_tensor_norm4_ring8": (I.ring(8), 512 * 7 + 9, I.COMP_UNIFORM_NEAREST_L2, 4, 0, I.NOISE_GAUSS),
}


def schedule(T, t0):
    """Step-decayed learning rate and a slowly varying consensus step."""
    gam = [np.float32(0.05 * 0.1 ** ((t0 + t) // 7)) for t in range(T)]
    eta = [np.float32(0.5 - 0.01 * ((t0 + t) % 5)) for t in range(T)]
    return gam, eta


@pytest.mark.parametrize("path", [0, 2])
@pytest.mark.parametrize("name", sorted(CASES))
def test_run_matches_oracle_and_single_steps(env, name, path):
    torch, orc, B = env
    graph, N, kind, bits, chunk, noise = CASES[name]
    ld = I.round_up(N, 4) + 8
    x, d, a, c = make_state(graph, N, ld, seed=11)
    sigma, seed = 0.1, 4242
    ds = B.DeepSqueeze(graph, N, ld, kind, bits, chunk)
    ds.ds_set_path(path)
    run = [torch.from_numpy(t.copy()).cuda() for t in (x, d, a, c)]
    one = [torch.from_numpy(t.copy()).cuda() for t in (x, d, a, c)]
    t0 = 5
    # three calls: instantiate (T=12), same T again (arguments updated in place), other T (new graph)
    for T in (12, 12, 3):
        gam, eta = schedule(T, t0)
        for t in range(T):
            codes_ref, scales_ref, _, _ = orc.step(graph, kind, bits, chunk, x, d, a, c, N, sigma, noise,
                                                   float(gam[t]), float(eta[t]), seed, t0 + t)
            ds.ds_step(one[0], one[1], one[2], one[3], sigma, noise, float(gam[t]), float(eta[t]), seed, t0 + t)
        ds.ds_sync()
        ds.ds_run(run[0], run[1], run[2], run[3], sigma, noise, gam, eta, seed, t0)
        ds.ds_sync()
        gx, gd = run[0].cpu().numpy(), run[1].cpu().numpy()
        # the graph replays the very same launches
        assert np.array_equal(gx, one[0].cpu().numpy()) and np.array_equal(gd, one[1].cpu().numpy())
        codes, scales = ds.codes_to_host()
        assert row_rel_err(gx[:, :N], x[:, :N]) <= TOL_RUN and row_rel_err(gd[:, :N], d[:, :N]) <= TOL_RUN
        assert np.array_equal(gx[:, N:], x[:, N:]) and np.array_equal(gd[:, N:], d[:, N:])
        # codes of the last iteration: a free run may flip a rounding decision, so only count
        assert (codes != codes_ref).mean() < 1e-3
        t0 += T
    ds.close()


def test_run_on_a_side_stream_and_argument_errors(env):
    torch, orc, B = env
    graph, N = I.ring(4), 2048
    ld = N
    x, d, a, c = make_state(graph, N, ld, seed=2)
    ds = B.DeepSqueeze(graph, N, ld, I.COMP_UNIFORM_STOCH_MAXABS, 2, 512)
    dev = [torch.from_numpy(t.copy()).cuda() for t in (x, d, a, c)]
    for T, step0 in ((0, 0), (B.DS_RUN_MAX_STEPS + 1, 0), (2, (1 << 56) - 1), (1, 1 << 56)):
        with pytest.raises(B.DsError) as err:
            ds.ds_run(dev[0], dev[1], dev[2], dev[3], 0.1, I.NOISE_GAUSS, [0.01] * T, [0.5] * T, 1, step0)
        assert err.value.status == B.DS_ERR_ARG
    assert np.array_equal(dev[0].cpu().numpy(), x)          # nothing ran
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    T = 6
    gam, eta = schedule(T, 0)
    ds.ds_run(dev[0], dev[1], dev[2], dev[3], 0.1, I.NOISE_GAUSS, gam, eta, 1, 0, stream=side)
    ds.ds_sync(side)
    for t in range(T):
        orc.step(graph, I.COMP_UNIFORM_STOCH_MAXABS, 2, 512, x, d, a, c, N, 0.1, I.NOISE_GAUSS,
                 float(gam[t]), float(eta[t]), 1, t)
    assert row_rel_err(dev[0].cpu().numpy(), x) <= TOL_RUN and row_rel_err(dev[1].cpu().numpy(), d) <= TOL_RUN
    ds.close()
