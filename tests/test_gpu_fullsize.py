"""Parity at the workloads' full sizes, in the launch configuration the
benchmark times (default path, default tuning).

A whole-problem run of the CPU oracle at these sizes takes minutes, but chunks
are independent columns: the oracle run on a window of columns (random streams
indexed by the global column, pinned by
test_oracle_step.py::test_column_window_equals_slice_of_whole_problem)
reproduces that slice of the whole-problem result.  The test runs two
free-running GPU steps on the full problem and checks windows at the start, in
the middle and at the ragged end of the rows: codes bit-exact, x / delta /
scales within 1e-5."""
import numpy as np
import pytest

from paper_1907_07346_b200 import inputs as I

pytestmark = pytest.mark.gpu
TOL = 1e-5


def _rel(got, ref):
    num = np.abs(got.astype(np.float64) - ref.astype(np.float64)).max(axis=1)
    den = np.maximum(np.abs(ref.astype(np.float64)).max(axis=1), 1e-30)
    return float((num / den).max())


@pytest.mark.parametrize("name,N", [("cfg3", None), ("cfg2", None), ("cfg5", None), ("cfg4", None)])
def test_full_size_windows(name, N):
    import torch
    from oracle import oracle as orc
    from paper_1907_07346_b200 import binding as B
    from paper_1907_07346_b200 import build as libbuild
    libbuild.build()
    w = I.WORKLOADS[name]
    if N is not None:
        w = w.with_size(N)
    N = w.N
    g = w.build_graph()
    ld = I.row_pitch(N)
    rng = np.random.default_rng(w.seed)
    host = []
    for kind in ("x", "d", "a", "c"):
        arr = np.zeros((w.n, ld), np.float32)
        for i in range(w.n):
            if kind == "a":
                arr[i, :N] = rng.random(N, dtype=np.float32) * np.float32(1.5) + np.float32(0.5)
            else:
                arr[i, :N] = rng.standard_normal(N, dtype=np.float32) * np.float32(
                    {"x": 0.3, "d": 0.05, "c": 1.0}[kind])
        host.append(arr)
    ds = B.DeepSqueeze(g, N, ld, w.comp_kind, w.bits, w.chunk)
    dev = [torch.from_numpy(t).cuda() for t in host]
    steps = 2
    chunk = w.chunk
    M = (N + chunk - 1) // chunk
    bits = 1 if w.comp_kind == I.COMP_SIGN1_L1 else w.bits
    windows = [(0, 4 * chunk), ((M // 2) * chunk, 3 * chunk), ((M - 3) * chunk, N - (M - 3) * chunk)]
    # oracle state per window, advanced alongside the GPU
    wstate = []
    for k0, cols in windows:
        sl = slice(k0, k0 + cols)
        wstate.append([np.ascontiguousarray(h[:, sl]) for h in host])
    for t in range(steps):
        ds.ds_step(dev[0], dev[1], dev[2], dev[3], w.sigma, w.noise_kind, w.gamma, w.eta, w.seed, t)
        ds.ds_sync()
        codes, scales = ds.codes_to_host()
        gx, gd = dev[0].cpu().numpy(), dev[1].cpu().numpy()
        assert np.isfinite(gx).all() and np.isfinite(gd).all()
        assert np.all(gx[:, N:] == 0) and np.all(gd[:, N:] == 0)          # padding untouched
        for (k0, cols), st in zip(windows, wstate):
            cw, sw, _, _ = orc.step(g, w.comp_kind, w.bits, chunk, st[0], st[1], st[2], st[3], cols,
                                    w.sigma, w.noise_kind, w.gamma, w.eta, w.seed, t, k_first=k0)
            w0 = k0 * bits // 32
            assert np.array_equal(codes[:, w0:w0 + cw.shape[1]], cw), (name, t, k0)
            m0 = k0 // chunk
            assert _rel(scales[:, m0:m0 + sw.shape[1]], sw) <= TOL
            assert _rel(gx[:, k0:k0 + cols], st[0]) <= TOL, (name, t, k0)
            assert _rel(gd[:, k0:k0 + cols], st[1]) <= TOL, (name, t, k0)
    ds.close()


def test_host_buffer_entry_point_pipelined():
    """ds_step_host on arrays large enough (>= 64 MiB each) to take the slab
    pipeline (copies in, compute and copies out overlapped on internal streams):
    same result as the oracle, padding columns never written back."""
    import torch
    from oracle import oracle as orc
    from paper_1907_07346_b200 import binding as B
    g = I.ring(8)
    N = 512 * 4200 + 40
    ld = I.row_pitch(N) + 32
    rng = np.random.default_rng(5)
    host = []
    for scale in (0.3, 0.05, None, 1.0):
        arr = np.full((g.n, ld), 3.0, np.float32)
        if scale is None:
            arr[:, :N] = rng.random((g.n, N), dtype=np.float32) * np.float32(1.5) + np.float32(0.5)
        else:
            arr[:, :N] = rng.standard_normal((g.n, N), dtype=np.float32) * np.float32(scale)
        host.append(arr)
    assert host[0].nbytes >= 64 << 20
    ds = B.DeepSqueeze(g, N, ld, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512)
    pinned = [torch.from_numpy(h.copy()).pin_memory() for h in host]
    dev = [torch.empty((g.n, ld), dtype=torch.float32, device="cuda") for _ in range(4)]
    side = torch.cuda.Stream()
    for t in range(2):
        ds.ds_step_host(pinned[0], pinned[1], pinned[2], pinned[3], 0.1, I.NOISE_GAUSS, 0.01, 0.5, 9, t,
                        *dev, stream=side)
    ds.ds_sync(side)
    for t in range(2):
        codes_ref, scales_ref, _, _ = orc.step(g, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, host[0], host[1],
                                               host[2], host[3], N, 0.1, I.NOISE_GAUSS, 0.01, 0.5, 9, t)
    codes, scales = ds.codes_to_host()
    assert np.array_equal(codes, codes_ref)
    assert _rel(pinned[0].numpy()[:, :N], host[0][:, :N]) <= TOL
    assert _rel(pinned[1].numpy()[:, :N], host[1][:, :N]) <= TOL
    assert np.all(pinned[0].numpy()[:, N:] == 3.0) and np.all(pinned[1].numpy()[:, N:] == 3.0)
    ds.close()
