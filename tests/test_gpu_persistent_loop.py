"""Parity of the persistent kernels where their LOOP runs: every thread block
walks at least four column tiles, so staging slots are refilled, the noise of
a second tile is drawn ahead, both C[v] buffers and both phases of the per-node
ready barriers recur, and the last tile is ragged.

Each case is the launch shape of one benchmark workload (node count, graph,
compressor, chunk, noise, hyper-parameters) at N = chunk * (148 * 4 + 3) + 40
-- a B200 has 148 SMs, one block each -- run for 20 free-running iterations of
Algorithm 1 from x_0 = delta_0 = 0 against the whole-problem oracle: packed
codes bit-exact, floats as assert_state_matches() states (bit-exact for
max-abs scales)."""
import numpy as np
import pytest

from paper_1907_07346_b200 import inputs as I
from test_gpu_parity import env, run_case, make_state, assert_state_matches, TOL_RUN  # noqa: F401

pytestmark = pytest.mark.gpu

SMS = 148


def loop_size(chunk):
    return chunk * (SMS * 4 + 3) + 40


def geometry(env, w, N):
    torch, orc, B = env
    ds = B.DeepSqueeze(w.build_graph(), N, I.round_up(N, 4), w.comp_kind, w.bits, w.chunk)
    info = ds.ds_get_info()
    ds.close()
    return info


# workload, threads per block, node batches a block sweeps per column
SHAPES = [("cfg3", 512, 1),       # ds_fused_tma_kernel: 16 warps, one node each
          ("cfg4", 512, 1),       # ds_fused_tma_pair_kernel: 16 warps, two nodes each
          ("cfg2", 512, 4),       # ds_wide_tma_kernel: 8 nodes x chunk 4096, two nodes (8 warps each) at a time
          ("cfg5", 512, 8),       # ds_wide_tma_kernel: 64 nodes x chunk 1024, eight nodes (2 warps each) at a time
          ("cfg3_l2", 512, 1)]    # ds_fused_tma_kernel, norm-matched codec


@pytest.mark.parametrize("name,threads,batches", SHAPES)
def test_twenty_steps_every_block_walks_four_tiles(env, name, threads, batches):
    torch, orc, B = env
    w = I.WORKLOADS[name]
    N = loop_size(w.chunk)
    info = geometry(env, w, N)
    # the benchmark's launch configuration: persistent grid of one block per SM, TMA-staged
    assert info.path == B.DS_PATH_FUSED and info.grid_blocks == SMS
    assert info.block_threads == threads and info.node_batches == batches
    assert (N + w.chunk - 1) // w.chunk >= 4 * SMS
    run_case(env, w.build_graph(), N, w.comp_kind, w.bits, w.chunk, w.noise_kind, B.DS_PATH_FUSED,
             steps=20, seed=8, sigma=w.sigma, gamma=w.gamma, eta=w.eta, zero_start=True, tol=TOL_RUN,
             a_dist=w.a_dist)


@pytest.mark.parametrize("name", ["cfg3", "cfg2", "cfg5", "cfg4"])
def test_given_gradient_twenty_steps_every_block_walks_four_tiles(env, name):
    """ds_step_g on the same shapes (three staged arrays instead of four)."""
    torch, orc, B = env
    w = I.WORKLOADS[name]
    N = loop_size(w.chunk)
    g = w.build_graph()
    ld = I.round_up(N, 4)
    x, d, _, _ = make_state(g, N, ld, 17, zero_start=True)
    ds = B.DeepSqueeze(g, N, ld, w.comp_kind, w.bits, w.chunk)
    assert ds.ds_get_info().path == B.DS_PATH_FUSED and ds.ds_get_info().grid_blocks == SMS
    dx, dd = torch.from_numpy(x.copy()).cuda(), torch.from_numpy(d.copy()).cuda()
    zeros = np.zeros_like(x)
    rng = np.random.default_rng(23)
    clean = None
    for t in range(20):
        grad = np.zeros_like(x)
        grad[:, :N] = rng.standard_normal((g.n, N), dtype=np.float32)
        grad[:, N:] = 9.0
        codes_ref, scales_ref, _, _ = orc.step(g, w.comp_kind, w.bits, w.chunk, x, d, zeros, zeros, N, 0.0,
                                               I.NOISE_NONE, w.gamma, w.eta, w.seed, t, g_given=grad)
        ds.ds_step_g(dx, dd, torch.from_numpy(grad).cuda(), w.gamma, w.eta, w.seed, t)
        ds.ds_sync()
        codes, scales = ds.codes_to_host()
        assert np.array_equal(codes, codes_ref), f"codes differ at step {t}"
        gx, gd = dx.cpu().numpy(), dd.cpu().numpy()
        clean = assert_state_matches(w.comp_kind, N, w.chunk, (gx, gd, scales), (x, d, scales_ref), TOL_RUN,
                                     f"at step {t}", clean)
        assert np.array_equal(gx[:, N:], x[:, N:]) and np.array_equal(gd[:, N:], d[:, N:])
    ds.close()
