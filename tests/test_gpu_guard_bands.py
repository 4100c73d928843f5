"""Bounds evidence for every kernel family: each of x, delta, a, c (or the
caller's gradient) lives inside a larger device tensor with 256 bytes of a
fixed pattern directly before and after it, the workspace likewise, and after
every step all pattern bytes must be unchanged; so must the padding columns of
every row and the pad words at the end of every row of packed codes and
scales.  A store that runs past an array or a row shows up here even where
the parity comparison would not look.  Sizes have awkward tails
(N = chunk * k + 1, + 3, an odd number of float4 groups, a row pitch that is
not a multiple of 32)."""
import numpy as np
import pytest

from paper_1907_07346_b200 import inputs as I
from test_gpu_parity import env  # noqa: F401  (fixture)

pytestmark = pytest.mark.gpu

BAND = 64            # floats: 256 bytes
PATTERN = -1234.5


class Guarded:
    """An [n][ld] float32 device array between two pattern bands inside one allocation."""

    def __init__(self, torch, host):
        n, ld = host.shape
        self.big = torch.full((2 * BAND + n * ld,), PATTERN, dtype=torch.float32, device="cuda")
        self.t = self.big[BAND:BAND + n * ld].view(n, ld)
        self.t.copy_(torch.from_numpy(host))
        assert self.t.data_ptr() % 16 == 0 and self.t.is_contiguous()

    def intact(self):
        return bool((self.big[:BAND] == PATTERN).all()) and bool((self.big[-BAND:] == PATTERN).all())


def pad_words_untouched(torch, ds):
    """Words of a codes / scales row beyond the valid ones keep their initial zero."""
    cptr, cpitch, sptr, spitch = ds.ds_codes()
    base = ds.workspace.data_ptr()
    codes = ds.workspace[cptr - base: cptr - base + ds.n * cpitch * 4].view(torch.int32).view(ds.n, cpitch)
    words = (ds.N * ds.code_bits + 31) // 32
    ok = bool((codes[:, words:] == 0).all())
    if ds.kind != I.COMP_IDENTITY:
        ch = ds.chunk if ds.chunk > 0 else ds.N
        M = (ds.N + ch - 1) // ch
        scales = ds.workspace[sptr - base: sptr - base + ds.n * spitch * 4].view(torch.int32).view(ds.n, spitch)
        ok = ok and bool((scales[:, M:] == 0).all())
    return ok


def host_state(n, N, ld, seed):
    rng = np.random.default_rng(seed)
    out = []
    for scale, pad in ((0.3, 7.0), (0.05, -7.0), (None, 3.0), (1.0, 5.0)):
        arr = np.full((n, ld), pad, np.float32)
        if scale is None:
            arr[:, :N] = rng.uniform(0.5, 2.0, (n, N))
        else:
            arr[:, :N] = scale * rng.standard_normal((n, N))
        out.append(arr)
    return out


# name: (graph, compressor kind, bits, chunk, noise, path, entry point)
FAMILIES = {
    "fused_tma_4bit": (I.ring(16), I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, I.NOISE_GAUSS, 1, "step"),
    "fused_tma_sign_two_warps_per_chunk": (I.ring(8), I.COMP_SIGN1_L1, 1, 1024, I.NOISE_GAUSS, 1, "step"),
    "fused_tma_identity": (I.ring(8), I.COMP_IDENTITY, 32, 512, I.NOISE_GAUSS, 1, "step"),
    "fused_tma_norm_matched": (I.ring(8), I.COMP_UNIFORM_NEAREST_L2, 4, 512, I.NOISE_GAUSS, 1, "step"),
    "fused_tma_per_node_scale": (I.ring(4), I.COMP_SIGN1_L1, 1, 0, I.NOISE_GAUSS, 1, "step"),
    "fused_tma_given_gradient": (I.ring(16), I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, I.NOISE_NONE, 1, "step_g"),
    "fused_tma_ecsgd": (I.complete(8), I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, I.NOISE_GAUSS, 0, "ecsgd"),
    "pair_2bit_t3": (I.torus(4, 8), I.COMP_UNIFORM_STOCH_MAXABS, 2, 256, I.NOISE_STUDENT_T3, 1, "step"),
    "fused_tma_32_warps_independent_t3": (I.torus(4, 8), I.COMP_UNIFORM_STOCH_MAXABS, 2, 256, I.NOISE_STUDENT_T3_IID, 1, "step"),
    "wide_tma_sign_chunk4096": (I.ring(8), I.COMP_SIGN1_L1, 1, 4096, I.NOISE_GAUSS, 1, "step"),
    "wide_tma_sign_64_nodes": (I.exponential(64), I.COMP_SIGN1_L1, 1, 1024, I.NOISE_GAUSS, 1, "step"),
    "wide_tma_4bit_40_nodes": (I.ring(40), I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, I.NOISE_GAUSS, 1, "step"),
    "column_fused_direct_loads": (I.ring(16), I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, I.NOISE_GAUSS, 3, "step"),
    "wide_fused_direct_loads": (I.exponential(64), I.COMP_SIGN1_L1, 1, 1024, I.NOISE_GAUSS, 3, "step"),
    "two_kernels_8bit": (I.ring(8), I.COMP_UNIFORM_STOCH_MAXABS, 8, 96, I.NOISE_GAUSS, 2, "step"),
    "two_kernels_sign_per_node": (I.ring(4), I.COMP_SIGN1_L1, 1, 0, I.NOISE_STUDENT_T3, 2, "step"),
    "two_kernels_ecsgd": (I.complete(8), I.COMP_SIGN1_L1, 1, 256, I.NOISE_GAUSS, 2, "ecsgd"),
    "resident_chunk512": (I.ring(16), I.COMP_UNIFORM_STOCH_MAXABS, 4, 512, I.NOISE_GAUSS, 0, "resident"),
    "resident_per_node": (I.ring(4), I.COMP_SIGN1_L1, 1, 0, I.NOISE_GAUSS, 0, "resident"),
    "graph_of_steps": (I.ring(8), I.COMP_UNIFORM_STOCH_MAXABS, 2, 256, I.NOISE_GAUSS, 0, "graph"),
}


def tails(chunk):
    c = chunk if chunk > 0 else 512
    # (N, extra pitch): one element into a new chunk; three; an odd count of float4 groups with a
    # pitch that is not a multiple of 32; an exact multiple of the chunk
    return [(c * 3 + 1, 0), (c * 2 + 3, 4), (c * 4 + 4 * 7 + 2, 12), (c * 3, 0)]


@pytest.mark.parametrize("name", sorted(FAMILIES))
def test_pattern_bands_survive_every_step(env, name):
    torch, orc, B = env
    graph, kind, bits, chunk, noise, path, entry = FAMILIES[name]
    for N, extra in tails(chunk):
        ld = I.round_up(N, 4) + extra
        host = host_state(graph.n, N, ld, 1)
        arrs = [Guarded(torch, h) for h in host]
        x, d, a, c = (g.t for g in arrs)
        ds = B.DeepSqueeze(graph, N, ld, kind, bits, chunk, guard_bytes=256)
        ds.ds_set_path(path)
        if path == B.DS_PATH_FUSED:
            assert ds.ds_get_info().path == B.DS_PATH_FUSED, name      # the TMA-staged kernels
        for t in range(3):
            if entry == "step":
                ds.ds_step(x, d, a, c, 0.1, noise, 0.05, 0.5, 5, t)
            elif entry == "step_g":
                ds.ds_step_g(x, d, a, 0.05, 0.5, 5, t)
            elif entry == "ecsgd":
                ds.ds_ecsgd_step(x, d, a, c, 0.1, noise, 0.05, 5, t)
            elif entry == "resident":
                ds.ds_run_resident(x, d, a, c, 0.1, noise, [0.05, 0.04], [0.5, 0.4], 5, 2 * t)
            else:
                ds.ds_run(x, d, a, c, 0.1, noise, [0.05, 0.04, 0.03], [0.5, 0.4, 0.3], 5, 3 * t)
            ds.ds_sync()
            where = (name, N, ld, t)
            assert all(g.intact() for g in arrs), where
            assert ds.workspace_guards_intact(), where
            assert pad_words_untouched(torch, ds), where
            # padding columns of every row: read, never changed; a and c entirely unchanged
            assert bool((x[:, N:] == 7.0).all()) and bool((d[:, N:] == -7.0).all()), where
            assert torch.equal(a, torch.from_numpy(host[2]).cuda()), where
            assert torch.equal(c, torch.from_numpy(host[3]).cuda()), where
            assert bool(torch.isfinite(x[:, :N]).all()) and bool(torch.isfinite(d[:, :N]).all()), where
        ds.close()
