"""The checked build of the library (-DDS_DEBUG): every kernel validates the
index arithmetic behind its accesses before it touches a part of a row, and a
refused part is reported by ds_sync as DS_ERR_BOUNDS instead of being touched.

The binding loads one library per process, so the checked build runs in child
processes (DEEPSQUEEZE_LIB points at it): (1) its self-test -- a part in the
row after the last one -- must be refused and reported, and the context must
keep working; (2) the guard-band cases of every kernel family and a set of
parity cases run on it: same results as the oracle, and no ds_sync reports a
refused index."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SELFTEST = r"""
import numpy as np, torch
from paper_1907_07346_b200 import binding as B, inputs as I
from oracle import oracle as orc
g = I.ring(8)
N, ld = 512 * 3 + 5, 512 * 3 + 8
ds = B.DeepSqueeze(g, N, ld, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512)
assert ds.ds_selftest_bounds() == B.DS_OK
try:
    ds.ds_sync()
    raise SystemExit("the refused index was not reported")
except B.DsError as err:
    assert err.status == B.DS_ERR_BOUNDS, err
ds.ds_sync()                                    # reported once
rng = np.random.default_rng(1)
x = (0.3 * rng.standard_normal((8, ld))).astype(np.float32); d = np.zeros_like(x)
a = rng.uniform(0.5, 2.0, (8, ld)).astype(np.float32); c = rng.standard_normal((8, ld)).astype(np.float32)
dev = [torch.from_numpy(t.copy()).cuda() for t in (x, d, a, c)]
codes_ref, _, _, _ = orc.step(g, I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, x, d, a, c, N, 0.1, I.NOISE_GAUSS, 0.05, 0.5, 3, 0)
ds.ds_step(dev[0], dev[1], dev[2], dev[3], 0.1, I.NOISE_GAUSS, 0.05, 0.5, 3, 0)
ds.ds_sync()
codes, _ = ds.codes_to_host()
assert np.array_equal(codes, codes_ref)
assert np.array_equal(dev[0].cpu().numpy()[:, :N], x[:, :N])
print("checked build: self-test ok")
"""


@pytest.fixture(scope="module")
def debug_lib():
    from paper_1907_07346_b200 import build as libbuild
    return libbuild.build(debug=True)


def _child_env(debug_lib):
    env = dict(os.environ)
    env["DEEPSQUEEZE_LIB"] = debug_lib
    env["PYTHONPATH"] = ROOT + os.pathsep + env.get("PYTHONPATH", "")
    return env


def test_normal_build_has_no_index_checks():
    import torch  # noqa: F401
    from paper_1907_07346_b200 import binding as B, inputs as I
    ds = B.DeepSqueeze(I.ring(4), 1000, 1000, I.COMP_SIGN1_L1, 1, 0)
    assert ds.ds_selftest_bounds() == B.DS_ERR_UNSUPPORTED
    ds.ds_sync()
    ds.close()


def test_checked_build_reports_a_refused_index(debug_lib):
    res = subprocess.run([sys.executable, "-c", SELFTEST], cwd=ROOT, env=_child_env(debug_lib),
                         capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "self-test ok" in res.stdout


def test_every_kernel_family_passes_its_own_index_checks(debug_lib):
    """All guard-band cases and the persistent-loop and graph parity cases on the checked
    build: results as on the normal build (they are compared with the oracle), and every
    ds_sync() in them would raise on a refused index."""
    cmd = [sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
           "tests/test_gpu_guard_bands.py", "tests/test_gpu_persistent_loop.py", "tests/test_gpu_pair.py",
           "tests/test_gpu_resident.py", "tests/test_zz_no_alloc.py",
           "tests/test_gpu_parity.py", "-k",
           "guard or walks or pair or torus32 or resident or noalloc or single_step_graphs or per_node or "
           "one_norm or long_chunks or many_nodes or unusual"]
    res = subprocess.run(cmd, cwd=ROOT, env=_child_env(debug_lib), capture_output=True, text=True, timeout=3000)
    assert res.returncode == 0, (res.stdout + res.stderr)[-4000:]
