"""GPU tests of ds_run_resident: T iterations of Algorithm 1 in one launch with
the state on chip (registers and shared memory) between iterations, against T
single-step calls (bit for bit) and against the CPU oracle."""
import numpy as np
import pytest

from paper_1907_07346_b200 import inputs as I
from test_gpu_parity import env, make_state, row_rel_err, TOL_RUN  # noqa: F401  (env is a fixture)
from test_gpu_run_graph import schedule

pytestmark = pytest.mark.gpu

CASES = {
    "per_node_sign_ring4_64k": (I.ring(4), 65_536, I.COMP_SIGN1_L1, 1, 0, I.NOISE_GAUSS),
    "per_node_4bit_ring4_ragged": (I.ring(4), 3000, I.COMP_UNIFORM_STOCH_MAXABS, 4, 0, I.NOISE_GAUSS),
    "per_node_2bit_torus12": (I.torus(3, 4), 512 * 9 + 7, I.COMP_UNIFORM_STOCH_MAXABS, 2, 0, I.NOISE_STUDENT_T3),
    "chunk512_4bit_ring16": (I.ring(16), 512 * 5 + 40, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, I.NOISE_GAUSS),
    "chunk512_sign_exp8": (I.exponential(8), 512 * 300 + 1, I.COMP_SIGN1_L1, 1, 512, I.NOISE_NONE),
    "single_node": (I.complete(1), 1000, I.COMP_UNIFORM_STOCH_MAXABS, 2, 0, I.NOISE_GAUSS),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_resident_matches_single_steps_and_oracle(env, name):
    torch, orc, B = env
    graph, N, kind, bits, chunk, noise = CASES[name]
    ld = I.round_up(N, 4) + 8
    x, d, a, c = make_state(graph, N, ld, seed=21)
    sigma, seed = 0.1, 777
    ds = B.DeepSqueeze(graph, N, ld, kind, bits, chunk)
    res = [torch.from_numpy(t.copy()).cuda() for t in (x, d, a, c)]
    one = [torch.from_numpy(t.copy()).cuda() for t in (x, d, a, c)]
    t0 = (1 << 32) - 3          # the step counter crosses 2^32 inside the run
    oracle_steps = 0
    for T in (9, 1, 14):
        gam, eta = schedule(T, t0)
        for t in range(T):
            if N <= 70_000:
                orc.step(graph, kind, bits, chunk, x, d, a, c, N, sigma, noise, float(gam[t]), float(eta[t]),
                         seed, t0 + t)
                oracle_steps += 1
            ds.ds_step(one[0], one[1], one[2], one[3], sigma, noise, float(gam[t]), float(eta[t]), seed, t0 + t)
        ds.ds_sync()
        codes_one, scales_one = ds.codes_to_host()
        ds.ds_run_resident(res[0], res[1], res[2], res[3], sigma, noise, gam, eta, seed, t0)
        ds.ds_sync()
        gx, gd = res[0].cpu().numpy(), res[1].cpu().numpy()
        assert np.array_equal(gx, one[0].cpu().numpy()) and np.array_equal(gd, one[1].cpu().numpy())
        codes, scales = ds.codes_to_host()
        assert np.array_equal(codes, codes_one) and np.array_equal(scales, scales_one)
        if oracle_steps:
            assert row_rel_err(gx[:, :N], x[:, :N]) <= TOL_RUN and row_rel_err(gd[:, :N], d[:, :N]) <= TOL_RUN
            assert np.array_equal(gx[:, N:], x[:, N:]) and np.array_equal(gd[:, N:], d[:, N:])
        t0 += T
    ds.close()


def test_resident_rejects_what_it_cannot_hold(env):
    torch, orc, B = env
    dummy = torch.zeros((32, 1024), dtype=torch.float32, device="cuda")

    def status_of(graph, N, kind, bits, chunk, T=2, step0=0, noise=I.NOISE_GAUSS):
        ds = B.DeepSqueeze(graph, N, N, kind, bits, chunk)
        t = dummy[:graph.n, :N].contiguous()
        try:
            ds.ds_run_resident(t, t.clone(), t.clone(), t.clone(), 0.1, noise, [0.01] * T, [0.5] * T, 1, step0)
            ds.ds_sync()
            return B.DS_OK
        except B.DsError as err:
            return err.status
        finally:
            ds.close()

    assert status_of(I.ring(4), 1024, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512) == B.DS_OK
    assert status_of(I.ring(4), 1024, I.COMP_UNIFORM_STOCH_MAXABS, 4, 256) == B.DS_ERR_UNSUPPORTED     # chunk
    assert status_of(I.ring(4), 1024, I.COMP_UNIFORM_STOCH_MAXABS, 8, 512) == B.DS_ERR_UNSUPPORTED     # bits
    assert status_of(I.torus(4, 8), 1024, I.COMP_SIGN1_L1, 1, 512) == B.DS_ERR_UNSUPPORTED             # 32 nodes
    assert status_of(I.ring(4), 1024, I.COMP_SIGN1_L1, 1, 512, noise=I.NOISE_STUDENT_T3_IID) == B.DS_ERR_UNSUPPORTED
    assert status_of(I.ring(4), 1024, I.COMP_SIGN1_L1, 1, 512, T=0) == B.DS_ERR_ARG
    assert status_of(I.ring(4), 1024, I.COMP_SIGN1_L1, 1, 512, T=B.DS_RESIDENT_MAX_STEPS + 1) == B.DS_ERR_ARG
    assert status_of(I.ring(4), 1024, I.COMP_SIGN1_L1, 1, 512, T=2, step0=(1 << 56) - 1) == B.DS_ERR_ARG


def test_resident_per_node_scale_too_large_for_one_wave(env):
    """One scale per node needs every tile's block resident at once."""
    torch, orc, B = env
    g = I.ring(16)
    N = 512 * 1000
    ds = B.DeepSqueeze(g, N, N, I.COMP_SIGN1_L1, 1, 0)
    t = torch.zeros((16, N), dtype=torch.float32, device="cuda")
    with pytest.raises(B.DsError) as err:
        ds.ds_run_resident(t, t.clone(), t.clone(), t.clone(), 0.1, I.NOISE_GAUSS, [0.01], [0.5], 1, 0)
    assert err.value.status == B.DS_ERR_UNSUPPORTED
    ds.close()
