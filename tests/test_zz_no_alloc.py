"""The allocation-free entry point ds_node_scales_noalloc against the regular
per-node-scale path (ds_step with chunk = 0, scales read back via ds_codes)
and against the CPU oracle's per-node scales (independent code).

Collected last on purpose: if it fails, a run that stops at the first failure
has already run every other test.  The entry point keeps its scratch in a
fixed array inside the library, shared by all calls, so the test calls it
twice in a row on different inputs: stale contents of the first call must not
leak into the second."""
import numpy as np
import pytest

from paper_1907_07346_b200 import inputs as I

pytestmark = pytest.mark.gpu

TOL = 1e-5      # the tolerance of the parity tests (l1 scales; max-abs scales are compared bit for bit)


def _reference_scales(torch, B, g, N, ld, kind, bits, arrays, sigma, noise, gamma, seed, step):
    """Scales of the regular path: one ds_step with a per-node scale on copies."""
    ds = B.DeepSqueeze(g, N, ld, kind, bits, 0)
    dev = [t.clone() for t in arrays]
    ds.ds_step(dev[0], dev[1], dev[2], dev[3], sigma, noise, gamma, 0.5, seed, step)
    ds.ds_sync()
    _, scales = ds.codes_to_host()
    ds.close()
    return scales[:, 0]


def _oracle_scales(g, N, kind, bits, host, sigma, noise, gamma, seed, step):
    """Per-node scales of the CPU oracle: one step with chunk = 0 on copies."""
    from oracle import oracle as orc
    cp = [h.copy() for h in host]
    _, scales, _, _ = orc.step(g, kind, bits, 0, cp[0], cp[1], cp[2], cp[3], N, sigma, noise, gamma, 0.5,
                               seed, step)
    return scales[:, 0]


def _assert_scales(kind, got, want, what):
    if kind == I.COMP_UNIFORM_STOCH_MAXABS:          # an exact maximum: no tolerance
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (what, got, want)
    else:                                            # a binary64 sum rounded once to binary32
        assert np.abs(got - want).max() <= TOL * np.abs(want).max(), (what, got, want)


# (graph, noise, pitch beyond N rounded up to 4, sizes of the two calls)
CASES = [(I.ring(8), I.NOISE_GAUSS, 0, [(512 * 9 + 37, 11), (512 * 2 + 5, 12)]),
         # more than one batch of nodes per grid row, a padded pitch, the other noise kinds
         (I.ring(12), I.NOISE_STUDENT_T3, 8, [(512 * 3 + 100, 21), (512 * 7 + 1, 22)]),
         (I.ring(3), I.NOISE_NONE, 4, [(515, 31), (40, 32)])]


@pytest.mark.parametrize("kind,bits", [(I.COMP_SIGN1_L1, 1), (I.COMP_UNIFORM_STOCH_MAXABS, 4)])
@pytest.mark.parametrize("case", CASES, ids=["ring8-gauss", "ring12-t3-padded", "ring3-nonoise"])
def test_noalloc_scales_match_regular_path_and_oracle_twice(kind, bits, case):
    import torch
    from paper_1907_07346_b200 import binding as B
    from paper_1907_07346_b200 import build as libbuild
    libbuild.build()
    g, noise, pad, calls = case
    sigma, gamma = 0.1, 0.05
    out = torch.full((g.n,), -1.0, dtype=torch.float32, device="cuda")
    # two calls in a row on different sizes and data: nothing of the first may leak into the second
    for call, (N, seed) in enumerate(calls):
        ld = I.round_up(N, 4) + pad
        rng = np.random.default_rng(100 + call)
        host = [np.full((g.n, ld), 2.5, np.float32) for _ in range(4)]        # padding columns: never used
        host[0][:, :N] = 0.3 * rng.standard_normal((g.n, N))
        host[1][:, :N] = 0.05 * rng.standard_normal((g.n, N))
        host[2][:, :N] = rng.uniform(0.5, 2.0, (g.n, N))
        host[3][:, :N] = rng.standard_normal((g.n, N))
        arrays = [torch.from_numpy(h).cuda() for h in host]
        want = _reference_scales(torch, B, g, N, ld, kind, bits, arrays, sigma, noise, gamma, seed, call)
        oracle = _oracle_scales(g, N, kind, bits, host, sigma, noise, gamma, seed, call)
        before = [t.clone() for t in arrays]
        out.fill_(-1.0)
        st = B.ds_node_scales_noalloc(out, arrays[0], arrays[1], arrays[2], arrays[3], sigma, noise,
                                      gamma, N, kind, seed, call)
        assert st == B.DS_OK, B.ds_strerror(st)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        assert np.all(got > 0)
        _assert_scales(kind, got, want, "against ds_step with chunk = 0")
        _assert_scales(kind, got, oracle, "against the CPU oracle")
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
