"""The allocation-free entry point ds_node_scales_noalloc against the regular
per-node-scale path (ds_step with chunk = 0, scales read back via ds_codes).

Collected last on purpose: if it fails, a run that stops at the first failure
has already run every other test.  The entry point keeps its scratch in a
fixed array inside the library, shared by all calls, so the test calls it
twice in a row on different inputs: stale contents of the first call must not
leak into the second."""
import numpy as np
import pytest

from paper_1907_07346_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL = 1e-5      # the tolerance of the parity tests; the two paths run the same kernels


def _reference_scales(torch, B, g, N, ld, kind, bits, arrays, sigma, noise, gamma, seed, step):
    """Scales of the regular path: one ds_step with a per-node scale on copies."""
    ds = B.DeepSqueeze(g, N, ld, kind, bits, 0)
    dev = [t.clone() for t in arrays]
    ds.ds_step(dev[0], dev[1], dev[2], dev[3], sigma, noise, gamma, 0.5, seed, step)
    ds.ds_sync()
    _, scales = ds.codes_to_host()
    ds.close()
    return scales[:, 0]


@pytest.mark.parametrize("kind,bits", [(I.COMP_SIGN1_L1, 1), (I.COMP_UNIFORM_STOCH_MAXABS, 4)])
def test_noalloc_scales_match_regular_path_twice(kind, bits):
    import torch
    from paper_1907_07346_b200 import binding as B
    from paper_1907_07346_b200 import build as libbuild
    libbuild.build()
    g = I.ring(8)
    sigma, noise, gamma = 0.1, I.NOISE_GAUSS, 0.05
    out = torch.full((g.n,), -1.0, dtype=torch.float32, device="cuda")
    # two calls in a row: a larger problem first, then a smaller one with other data
    for call, (N, seed) in enumerate([(512 * 9 + 37, 11), (512 * 2 + 5, 12)]):
        ld = I.round_up(N, 4)
        rng = np.random.default_rng(100 + call)
        host = [np.zeros((g.n, ld), np.float32) for _ in range(4)]
        host[0][:, :N] = 0.3 * rng.standard_normal((g.n, N))
        host[1][:, :N] = 0.05 * rng.standard_normal((g.n, N))
        host[2][:, :N] = rng.uniform(0.5, 2.0, (g.n, N))
        host[3][:, :N] = rng.standard_normal((g.n, N))
        arrays = [torch.from_numpy(h).cuda() for h in host]
        want = _reference_scales(torch, B, g, N, ld, kind, bits, arrays, sigma, noise, gamma, seed, call)
        before = [t.clone() for t in arrays]
        out.fill_(-1.0)
        st = B.ds_node_scales_noalloc(out, arrays[0], arrays[1], arrays[2], arrays[3], sigma, noise,
                                      gamma, N, kind, seed, call)
        assert st == B.DS_OK, B.ds_strerror(st)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert np.all(got > 0)
        assert np.abs(got - want).max() <= TOL * np.abs(want).max(), (got, want)
        for t, b in zip(arrays, before):          # inputs are only read
            assert torch.equal(t, b)


def test_noalloc_rejects_sizes_beyond_the_fixed_scratch():
    import torch
    from paper_1907_07346_b200 import binding as B
    n, N = 64, 512 * 1025            # 64 * 1025 partials > 65536
    x = torch.zeros((n, 4), dtype=torch.float32, device="cuda")   # never touched: the size check comes first
    out = torch.zeros((n,), dtype=torch.float32, device="cuda")
    gp = B.ds_grad_params(x.data_ptr(), x.data_ptr(), 0.0, 0)
    import ctypes as C
    st = B.lib().ds_node_scales_noalloc(out.data_ptr(), x.data_ptr(), x.data_ptr(), C.byref(gp), 0.1,
                                        n, N, N, I.COMP_SIGN1_L1, 1, 0, None)
    assert st == B.DS_ERR_WORKSPACE
    assert "workspace" in B.ds_strerror(st)
