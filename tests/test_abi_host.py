"""Host-side tests of the C ABI: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching CUDA.  CPU only."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_1907_07346_b200 import binding as B
from paper_1907_07346_b200 import build as libbuild
from paper_1907_07346_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE_WS = 0x10000000          # aligned, never dereferenced by the host checks
BIG = 1 << 40


@pytest.fixture(scope="module", autouse=True)
def _built():
    libbuild.build()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "deepsqueeze.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ds_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_functions()
    assert set(names) == set(B.EXPORTS)
    raw = C.CDLL(B.LIB_PATH)
    for name in names:
        assert hasattr(raw, name), name


def test_strerror():
    assert B.ds_strerror(B.DS_OK) == "ok"
    seen = {B.ds_strerror(s) for s in range(0, 12)}
    assert len(seen) == 12


def test_workspace_size():
    g = I.ring(16)
    nnz = int(g.row_ptr[-1])
    N = 25_557_032
    size = B.ds_workspace_size(16, N, B.DS_COMP_UNIFORM_STOCH_MAXABS, 4, 512, nnz)
    words = (N * 4 + 31) // 32
    scales = (N + 511) // 512
    assert size >= 16 * words * 4 + 16 * scales * 4
    assert size < 16 * words * 4 + 16 * scales * 4 + 64 * 1024
    assert B.ds_workspace_size(16, N, B.DS_COMP_UNIFORM_STOCH_MAXABS, 3, 512, nnz) == 0
    assert B.ds_workspace_size(16, N, B.DS_COMP_UNIFORM_STOCH_MAXABS, 4, 100, nnz) == 0
    assert B.ds_workspace_size(0, N, B.DS_COMP_SIGN1_L1, 1, 512, nnz) == 0
    # the packed codes are b/32 of the float32 volume (Section 5: 4 bits save 7/8)
    assert words * 32 == N * 4


def _init(g, w=None, n=None, N=1000, ld=1024, kind=B.DS_COMP_SIGN1_L1, bits=1, chunk=64,
          ws=FAKE_WS, ws_bytes=BIG, row_ptr=None, col_idx=None):
    st, ctx = B.ds_init_raw(g.row_ptr if row_ptr is None else row_ptr,
                            g.col_idx if col_idx is None else col_idx,
                            g.w if w is None else w, g.n if n is None else n, N, ld,
                            kind, bits, chunk, ws, ws_bytes, graph_n=g.n)
    assert (st == B.DS_OK) == bool(ctx.value)
    return st


def _expect_ok_or_no_device(st):
    import torch
    if torch.cuda.is_available():
        assert st == B.DS_ERR_CUDA or st == B.DS_OK      # FAKE_WS is not device memory
    else:
        assert st == B.DS_ERR_CUDA


def test_init_argument_errors():
    g = I.ring(8)
    assert _init(g, N=0) == B.DS_ERR_ARG
    assert _init(g, N=1 << 31) == B.DS_ERR_ARG
    assert _init(g, n=7) == B.DS_ERR_ARG
    assert _init(g, N=1000, ld=996) == B.DS_ERR_ARG
    assert _init(g, N=1000, ld=1002) == B.DS_ERR_ALIGN
    assert _init(g, ws=FAKE_WS + 16) == B.DS_ERR_ALIGN
    assert _init(g, ws=0) == B.DS_ERR_NULL
    assert _init(g, kind=7) == B.DS_ERR_ARG
    assert _init(g, chunk=48) == B.DS_ERR_ARG
    assert _init(g, chunk=-32) == B.DS_ERR_ARG
    assert _init(g, kind=B.DS_COMP_UNIFORM_STOCH_MAXABS, bits=3) == B.DS_ERR_UNSUPPORTED
    assert _init(g, kind=B.DS_COMP_SIGN1_L1, bits=2) == B.DS_ERR_UNSUPPORTED
    assert _init(g, chunk=32768) == B.DS_ERR_UNSUPPORTED
    assert _init(g, kind=B.DS_COMP_UNIFORM_NEAREST_L2, bits=8, chunk=512) == B.DS_ERR_UNSUPPORTED
    assert _init(g, kind=B.DS_COMP_UNIFORM_NEAREST_L2, bits=1, chunk=0) == B.DS_ERR_UNSUPPORTED
    assert _init(g, ws_bytes=1024) == B.DS_ERR_WORKSPACE
    st, ctx = B.ds_init_raw(None, g.col_idx, g.w, 8, 1000, 1024, 1, 1, 64, FAKE_WS, BIG)
    assert st == B.DS_ERR_NULL


def test_init_graph_errors():
    g = I.ring(8)
    rp = g.row_ptr.copy(); rp[0] = 1
    assert _init(g, row_ptr=rp) == B.DS_ERR_GRAPH
    rp = g.row_ptr.copy(); rp[3] = rp[2] - 1
    assert _init(g, row_ptr=rp) == B.DS_ERR_GRAPH
    ci = g.col_idx.copy(); ci[4] = 99
    assert _init(g, col_idx=ci) == B.DS_ERR_GRAPH
    ci = g.col_idx.copy(); ci[3], ci[4] = ci[4], ci[3]          # unsorted row
    assert _init(g, col_idx=ci) == B.DS_ERR_GRAPH
    ci = g.col_idx.copy(); ci[4] = ci[3]                          # duplicate
    assert _init(g, col_idx=ci) == B.DS_ERR_GRAPH


def test_init_self_loop_required():
    # a ring without the diagonal: rows {i-1, i+1}
    n = 6
    cols, rp = [], [0]
    for i in range(n):
        cols += sorted({(i - 1) % n, (i + 1) % n})
        rp.append(len(cols))
    g = I.Graph(n, np.asarray(rp, np.int32), np.asarray(cols, np.int32),
                np.full(len(cols), 0.5, np.float32))
    assert _init(g) == B.DS_ERR_NO_SELF_LOOP


def test_init_W_errors():
    g = I.ring(8)
    w = g.w.copy(); w[0] += 1e-3
    assert _init(g, w=w) in (B.DS_ERR_W_NOT_SYMMETRIC, B.DS_ERR_W_NOT_STOCHASTIC)
    w = g.w.copy(); w[1] = -w[1]
    assert _init(g, w=w) == B.DS_ERR_W_NOT_STOCHASTIC
    # symmetric but rows do not sum to one
    assert _init(g, w=g.w * np.float32(0.9)) == B.DS_ERR_W_NOT_STOCHASTIC
    # row sums fine, symmetry broken: move weight between the two off-diagonals of every row
    w = g.w.copy().reshape(8, 3)
    w[:, 0] += 0.05
    w[:, 2] -= 0.05
    # rows of the ring are sorted by column, so positions 0 and 2 are not always (i-1, i+1);
    # the perturbation is asymmetric either way
    assert _init(g, w=w.reshape(-1)) == B.DS_ERR_W_NOT_SYMMETRIC
    # pattern asymmetry: edge 0->2 without 2->0
    cols, rp, vals = [], [0], []
    for i in range(4):
        members = sorted({(i - 1) % 4, i, (i + 1) % 4} | ({2} if i == 0 else set()))
        cols += members
        vals += [1.0 / len(members)] * len(members)
        rp.append(len(cols))
    g2 = I.Graph(4, np.asarray(rp, np.int32), np.asarray(cols, np.int32), np.asarray(vals, np.float32))
    assert _init(g2) == B.DS_ERR_W_NOT_SYMMETRIC


def test_valid_init_reaches_cuda():
    """Everything valid: the only thing left to fail on a machine without a GPU
    is the first CUDA call.  (With a GPU the fake workspace pointer fails too.)"""
    for g in (I.ring(16), I.torus(4, 8), I.exponential(64)):
        _expect_ok_or_no_device(_init(g, N=4096, ld=4096, chunk=512))
    # the norm-matched codec takes long chunks and one norm per node
    for chunk in (1024, 0):
        _expect_ok_or_no_device(_init(I.ring(8), N=4096, ld=4096, kind=B.DS_COMP_UNIFORM_NEAREST_L2, bits=4,
                                      chunk=chunk))


def test_null_handles():
    L = B.lib()
    assert L.ds_step(None, None, None, None, None, 0, 0, None) == B.DS_ERR_NULL
    assert L.ds_step_g(None, None, None, None, None, 0, 0, None) == B.DS_ERR_NULL
    assert L.ds_run(None, None, None, None, None, None, 1, 0, 0, None) == B.DS_ERR_NULL
    assert L.ds_set_path(None, 0) == B.DS_ERR_NULL
    assert L.ds_get_info(None, None) == B.DS_ERR_NULL
    assert L.ds_codes(None, None, None, None, None) == B.DS_ERR_NULL
    assert L.ds_noise(None, 1, 1, 1, 0, 0, 0, 0, None) == B.DS_ERR_NULL
    assert L.ds_sync(None, None) == B.DS_ERR_NULL
    assert L.ds_selftest_timeout(None, None) == B.DS_ERR_NULL
    assert L.ds_selftest_math(None, None) == B.DS_ERR_NULL
    L.ds_destroy(None)
