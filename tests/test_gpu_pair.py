"""GPU parity of the fused kernel that gives every warp two nodes (17..32
nodes, chunks of 256 elements) against the CPU oracle: packed codes bit-exact,
x, delta and scales within 1e-5 per node row and step."""
import numpy as np
import pytest

from paper_1907_07346_b200 import inputs as I
from test_gpu_parity import env, run_case, TOL_RUN  # noqa: F401  (env is a fixture)

pytestmark = pytest.mark.gpu

COMPS = [(I.COMP_SIGN1_L1, 1), (I.COMP_UNIFORM_STOCH_MAXABS, 1), (I.COMP_UNIFORM_STOCH_MAXABS, 2),
         (I.COMP_UNIFORM_STOCH_MAXABS, 4), (I.COMP_UNIFORM_STOCH_MAXABS, 8)]


def geometry(env, graph, N, kind, bits, chunk):
    torch, orc, B = env
    ds = B.DeepSqueeze(graph, N, I.round_up(N, 4), kind, bits, chunk)
    info = ds.ds_get_info()
    ds.close()
    return info


@pytest.mark.parametrize("comp", COMPS)
@pytest.mark.parametrize("noise", [I.NOISE_NONE, I.NOISE_GAUSS, I.NOISE_STUDENT_T3])
def test_torus32_chunk256(env, comp, noise):
    kind, bits = comp
    g = I.torus(4, 8)
    N = 256 * 9 + 40 + 3                      # nine full tiles and a ragged one
    info = geometry(env, g, N, kind, bits, 256)
    assert info.block_threads == 512 and info.elems_per_lane == 8      # 16 warps, two nodes each
    run_case(env, g, N, kind, bits, 256, noise, 1, steps=3, gamma=0.005, eta=0.4)


@pytest.mark.parametrize("graph", [I.ring(18), I.exponential(20), I.complete(26)], ids=lambda g: g.name)
def test_other_even_node_counts(env, graph):
    run_case(env, graph, 256 * 5 + 100, I.COMP_UNIFORM_STOCH_MAXABS, 2, 256, I.NOISE_GAUSS, 1, steps=2)
    run_case(env, graph, 256 * 5 + 100, I.COMP_SIGN1_L1, 1, 256, I.NOISE_STUDENT_T3, 1, steps=2)


def test_many_tiles_per_block_and_twenty_steps(env):
    """More tiles than blocks (every block walks several tiles, both buffers of
    C[v] in use), free-running for 20 steps."""
    g = I.torus(4, 8)
    run_case(env, g, 256 * 700 + 8, I.COMP_UNIFORM_STOCH_MAXABS, 2, 256, I.NOISE_STUDENT_T3, 1, steps=2)
    run_case(env, g, 256 * 40, I.COMP_UNIFORM_STOCH_MAXABS, 4, 256, I.NOISE_GAUSS, 1, steps=20,
             zero_start=True, tol=TOL_RUN)


def test_odd_node_count_keeps_the_one_node_per_warp_kernel(env):
    torch, orc, B = env
    g = I.ring(31)
    info = geometry(env, g, 256 * 4, I.COMP_UNIFORM_STOCH_MAXABS, 2, 256)
    assert info.block_threads == 31 * 32
    run_case(env, g, 256 * 4 + 7, I.COMP_UNIFORM_STOCH_MAXABS, 2, 256, I.NOISE_GAUSS, 1, steps=2)
