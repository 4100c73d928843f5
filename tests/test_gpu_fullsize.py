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


def _device_outputs(torch, ds):
    """Views (no copy) of the packed codes and scales the last step left in the workspace."""
    cptr, cpitch, sptr, spitch = ds.ds_codes()
    base = ds.workspace.data_ptr()
    codes = ds.workspace[cptr - base: cptr - base + ds.n * cpitch * 4].view(torch.int32).view(ds.n, cpitch)
    scales = ds.workspace[sptr - base: sptr - base + ds.n * spitch * 4].view(torch.int32).view(ds.n, spitch)
    return codes, scales


@pytest.mark.parametrize("name", ["cfg3", "cfg2", "cfg5", "cfg4", "cfg3_l2"])
def test_full_size_windows_and_paths(name):
    """Two free-running steps at the workload's full size on the default path (the kernel the
    benchmark times).  (1) 64 seeded random chunk columns plus windows at the start, in the
    middle and at the ragged end of the rows against the oracle: codes bit-exact, floats
    bit-exact for max-abs scales, within 1e-5 for l1 scales.  (2) The WHOLE arrays -- x, delta,
    packed codes, scales -- against the two-kernel path run from the same state, compared
    bit for bit on the device: the two paths share the canonical operation order, the scale
    of a chunk is summed in the same lane order, so any difference is a defect of one of them."""
    import torch
    from oracle import oracle as orc
    from paper_1907_07346_b200 import binding as B
    from paper_1907_07346_b200 import build as libbuild
    from test_gpu_parity import assert_state_matches
    libbuild.build()
    w = I.WORKLOADS[name]
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
    steps = 2
    chunk = w.chunk
    M = (N + chunk - 1) // chunk
    bits = 1 if w.comp_kind == I.COMP_SIGN1_L1 else w.bits
    windows = [(0, 4 * chunk), ((M // 2) * chunk, 3 * chunk), ((M - 3) * chunk, N - (M - 3) * chunk)]
    pick = np.random.default_rng(w.seed + 7).choice(M - 1, size=64, replace=False)
    windows += [(int(m) * chunk, chunk) for m in sorted(pick)]
    # oracle state per window, advanced alongside the GPU
    wstate = []
    for k0, cols in windows:
        sl = slice(k0, k0 + cols)
        wstate.append([np.ascontiguousarray(h[:, sl]) for h in host])

    results = {}
    for path in (B.DS_PATH_AUTO, B.DS_PATH_SPLIT):
        ds = B.DeepSqueeze(g, N, ld, w.comp_kind, w.bits, w.chunk)
        ds.ds_set_path(path)
        if path == B.DS_PATH_AUTO:
            assert ds.ds_get_info().path == B.DS_PATH_FUSED and ds.ds_get_info().grid_blocks == 148
        dev = [torch.from_numpy(t).cuda() for t in host]
        clean = [None] * len(windows)
        for t in range(steps):
            ds.ds_step(dev[0], dev[1], dev[2], dev[3], w.sigma, w.noise_kind, w.gamma, w.eta, w.seed, t)
            ds.ds_sync()
            if path != B.DS_PATH_AUTO:
                continue
            assert bool(torch.isfinite(dev[0]).all()) and bool(torch.isfinite(dev[1]).all())
            assert bool((dev[0][:, N:] == 0).all()) and bool((dev[1][:, N:] == 0).all())     # padding untouched
            codes_d, scales_d = _device_outputs(torch, ds)
            for wi, ((k0, cols), st) in enumerate(zip(windows, wstate)):
                cw, sw, _, _ = orc.step(g, w.comp_kind, w.bits, chunk, st[0], st[1], st[2], st[3], cols,
                                        w.sigma, w.noise_kind, w.gamma, w.eta, w.seed, t, k_first=k0)
                w0 = k0 * bits // 32
                got_codes = codes_d[:, w0:w0 + cw.shape[1]].cpu().numpy().view(np.uint32)
                assert np.array_equal(got_codes, cw), (name, t, k0)
                m0 = k0 // chunk
                got_scales = scales_d[:, m0:m0 + sw.shape[1]].cpu().numpy().view(np.float32)
                gx = dev[0][:, k0:k0 + cols].cpu().numpy()
                gd = dev[1][:, k0:k0 + cols].cpu().numpy()
                clean[wi] = assert_state_matches(w.comp_kind, cols, chunk, (gx, gd, got_scales),
                                                 (st[0], st[1], sw), TOL, f"{name} step {t} column {k0}", clean[wi])
        codes_d, scales_d = _device_outputs(torch, ds)
        words = (N * bits + 31) // 32
        results[path] = (dev[0], dev[1], codes_d[:, :words].clone(), scales_d[:, :M].clone())
        del dev
        ds.close()
    for u, v, what in zip(results[B.DS_PATH_AUTO], results[B.DS_PATH_SPLIT], ("x", "delta", "codes", "scales")):
        if u.dtype == torch.float32:
            u, v = u.view(torch.int32), v.view(torch.int32)
        assert torch.equal(u, v), f"{name}: {what} of the fused and the two-kernel path differ"


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


@pytest.mark.parametrize("path", [0, 2], ids=["default-path", "two-kernels"])
def test_longest_rows(path):
    """Maximum size: N just below the 2^31 limit of the interface (two nodes, 4-bit codes, chunks of
    512: 4,194,304 tiles per row, a ragged last one; 8.6 GB per array row, offsets beyond 2^32
    bytes).  The state is drawn on the device; windows at the start, around the 2^30-th and 2^31-th
    byte and element boundaries and at the very end of the rows are copied to the host and
    compared with the oracle run on those columns (random streams indexed by the global column):
    codes and floats bit for bit (max-abs scales), over two free-running steps."""
    import torch
    from oracle import oracle as orc
    from paper_1907_07346_b200 import binding as B
    from test_gpu_parity import assert_state_matches
    g = I.complete(2)
    chunk, bits, kind = 512, 4, I.COMP_UNIFORM_STOCH_MAXABS
    N = (1 << 31) - 48                      # the interface takes N < 2^31; ld a multiple of 4
    ld = N
    M = (N + chunk - 1) // chunk
    gen = torch.Generator(device="cuda")
    gen.manual_seed(12345)
    dev = []
    for scale in (0.3, 0.05, None, 1.0):
        t = torch.empty((g.n, ld), dtype=torch.float32, device="cuda")
        for i in range(g.n):
            if scale is None:
                t[i].uniform_(0.5, 2.0, generator=gen)
            else:
                t[i].normal_(0.0, scale, generator=gen)
        dev.append(t)
    ds = B.DeepSqueeze(g, N, ld, kind, bits, chunk)
    ds.ds_set_path(path)
    if path == 0:
        assert ds.ds_get_info().path == B.DS_PATH_FUSED and ds.ds_get_info().grid_blocks == 148
    first_tiles = [0, (1 << 30) // 4 // chunk - 1, (1 << 30) // chunk - 1, (1 << 31) // 4 // chunk - 1, M // 2, M - 3]
    windows = [(m * chunk, min(3 * chunk, N - m * chunk)) for m in first_tiles]
    wstate = [[np.ascontiguousarray(t[:, k0:k0 + cols].cpu().numpy()) for t in dev] for k0, cols in windows]
    sigma, gamma, eta, seed = 0.1, 0.01, 0.5, 4711
    for step in range(2):
        ds.ds_step(dev[0], dev[1], dev[2], dev[3], sigma, I.NOISE_GAUSS, gamma, eta, seed, step)
        ds.ds_sync()
        codes_d, scales_d = _device_outputs(torch, ds)
        for (k0, cols), st in zip(windows, wstate):
            cw, sw, _, _ = orc.step(g, kind, bits, chunk, st[0], st[1], st[2], st[3], cols, sigma, I.NOISE_GAUSS,
                                    gamma, eta, seed, step, k_first=k0)
            w0 = k0 * bits // 32
            assert np.array_equal(codes_d[:, w0:w0 + cw.shape[1]].cpu().numpy().view(np.uint32), cw), (step, k0)
            m0 = k0 // chunk
            got_scales = scales_d[:, m0:m0 + sw.shape[1]].cpu().numpy().view(np.float32)
            gx, gd = dev[0][:, k0:k0 + cols].cpu().numpy(), dev[1][:, k0:k0 + cols].cpu().numpy()
            assert_state_matches(kind, cols, chunk, (gx, gd, got_scales), (st[0], st[1], sw), TOL, f"step {step} column {k0}")
    assert bool(torch.isfinite(dev[0]).all()) and bool(torch.isfinite(dev[1]).all())
    ds.close()
