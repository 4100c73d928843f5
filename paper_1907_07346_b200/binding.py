"""Python binding of the DeepSqueeze C ABI (include/deepsqueeze.h).

Argument marshalling only: every step of the path runs in the CUDA kernels of
libdeepsqueeze.so.  torch is used for device memory and streams.  There is no
CPU fallback: if the library cannot be loaded, importing callers get an error.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# DEEPSQUEEZE_LIB: load another build of the library (e.g. a checked or experimental one)
LIB_PATH = os.environ.get("DEEPSQUEEZE_LIB") or os.path.join(_HERE, "libdeepsqueeze.so")

DS_OK = 0
(DS_ERR_NULL, DS_ERR_ARG, DS_ERR_GRAPH, DS_ERR_W_NOT_SYMMETRIC, DS_ERR_W_NOT_STOCHASTIC,
 DS_ERR_NO_SELF_LOOP, DS_ERR_ALIGN, DS_ERR_WORKSPACE, DS_ERR_UNSUPPORTED, DS_ERR_CUDA,
 DS_ERR_TIMEOUT, DS_ERR_BOUNDS) = range(1, 13)

DS_COMP_IDENTITY, DS_COMP_SIGN1_L1, DS_COMP_UNIFORM_STOCH_MAXABS, DS_COMP_UNIFORM_NEAREST_L2 = 0, 1, 2, 3
DS_NOISE_NONE, DS_NOISE_GAUSS, DS_NOISE_STUDENT_T3, DS_NOISE_STUDENT_T3_IID = 0, 1, 2, 3
DS_PATH_AUTO, DS_PATH_FUSED, DS_PATH_SPLIT, DS_PATH_FUSED_LDG = 0, 1, 2, 3
DS_RUN_MAX_STEPS = 4096
DS_RESIDENT_MAX_STEPS = 1024

EXPORTS = ["ds_workspace_size", "ds_init", "ds_step", "ds_step_g", "ds_ecsgd_step", "ds_ecsgd_step_g", "ds_run", "ds_run_resident", "ds_step_host", "ds_codes", "ds_set_path",
           "ds_tune", "ds_get_info", "ds_sync", "ds_selftest_timeout", "ds_selftest_bounds", "ds_selftest_math", "ds_noise", "ds_node_scales_noalloc",
           "ds_destroy", "ds_strerror"]


class ds_graph(C.Structure):
    _fields_ = [("n", C.c_int32), ("row_ptr", C.POINTER(C.c_int32)), ("col_idx", C.POINTER(C.c_int32))]


class ds_compressor(C.Structure):
    _fields_ = [("kind", C.c_int32), ("bits", C.c_int32), ("chunk", C.c_int64)]


class ds_grad_params(C.Structure):
    _fields_ = [("a", C.c_void_p), ("c", C.c_void_p), ("sigma", C.c_float), ("noise", C.c_int32)]


class ds_hparams(C.Structure):
    _fields_ = [("gamma", C.c_float), ("eta", C.c_float)]


class ds_info(C.Structure):
    _fields_ = [("path", C.c_int32), ("launches_per_step", C.c_int32), ("elems_per_lane", C.c_int32),
                ("warps_per_chunk", C.c_int32), ("block_threads", C.c_int32), ("grid_blocks", C.c_int32),
                ("chunks_per_row", C.c_int64), ("code_words_per_row", C.c_int64),
                ("node_batches", C.c_int32)]


_lib = None


def lib():
    """Load libdeepsqueeze.so (built in-tree by paper_1907_07346_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_1907_07346_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.ds_workspace_size.argtypes = [C.c_int32, C.c_int64, C.POINTER(ds_compressor), C.c_int32]
        L.ds_workspace_size.restype = C.c_size_t
        L.ds_init.argtypes = [C.POINTER(C.c_void_p), C.POINTER(ds_graph), C.POINTER(C.c_float), C.c_int32,
                              C.c_int64, C.c_int64, C.POINTER(ds_compressor), C.c_void_p, C.c_size_t]
        L.ds_init.restype = C.c_int
        L.ds_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(ds_grad_params),
                              C.POINTER(ds_hparams), C.c_uint64, C.c_uint64, C.c_void_p]
        L.ds_step.restype = C.c_int
        L.ds_step_g.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(ds_hparams),
                                C.c_uint64, C.c_uint64, C.c_void_p]
        L.ds_step_g.restype = C.c_int
        L.ds_ecsgd_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(ds_grad_params), C.c_float,
                                    C.c_uint64, C.c_uint64, C.c_void_p]
        L.ds_ecsgd_step.restype = C.c_int
        L.ds_ecsgd_step_g.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                      C.c_uint64, C.c_uint64, C.c_void_p]
        L.ds_ecsgd_step_g.restype = C.c_int
        L.ds_run.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(ds_grad_params), C.POINTER(C.c_float),
                             C.POINTER(C.c_float), C.c_int32, C.c_uint64, C.c_uint64, C.c_void_p]
        L.ds_run.restype = C.c_int
        L.ds_run_resident.argtypes = L.ds_run.argtypes
        L.ds_run_resident.restype = C.c_int
        L.ds_step_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float,
                                   C.c_int32, C.POINTER(ds_hparams), C.c_uint64, C.c_uint64,
                                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ds_step_host.restype = C.c_int
        L.ds_codes.argtypes = [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_int64),
                               C.POINTER(C.c_void_p), C.POINTER(C.c_int64)]
        L.ds_codes.restype = C.c_int
        L.ds_set_path.argtypes = [C.c_void_p, C.c_int32]
        L.ds_set_path.restype = C.c_int
        L.ds_tune.argtypes = [C.c_void_p, C.c_int32]
        L.ds_tune.restype = C.c_int
        L.ds_get_info.argtypes = [C.c_void_p, C.POINTER(ds_info)]
        L.ds_get_info.restype = C.c_int
        L.ds_sync.argtypes = [C.c_void_p, C.c_void_p]
        L.ds_sync.restype = C.c_int
        L.ds_selftest_timeout.argtypes = [C.c_void_p, C.c_void_p]
        L.ds_selftest_timeout.restype = C.c_int
        L.ds_selftest_bounds.argtypes = [C.c_void_p, C.c_void_p]
        L.ds_selftest_bounds.restype = C.c_int
        L.ds_selftest_math.argtypes = [C.c_void_p, C.c_void_p]
        L.ds_selftest_math.restype = C.c_int
        L.ds_noise.argtypes = [C.c_void_p, C.c_int32, C.c_int64, C.c_int64, C.c_int32, C.c_int32,
                               C.c_uint64, C.c_uint64, C.c_void_p]
        L.ds_noise.restype = C.c_int
        L.ds_node_scales_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(ds_grad_params),
                                             C.c_float, C.c_int32, C.c_int64, C.c_int64, C.c_int32,
                                             C.c_uint64, C.c_uint64, C.c_void_p]
        L.ds_node_scales_noalloc.restype = C.c_int
        L.ds_destroy.argtypes = [C.c_void_p]
        L.ds_destroy.restype = None
        L.ds_strerror.argtypes = [C.c_int]
        L.ds_strerror.restype = C.c_char_p
        _lib = L
    return _lib


class DsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {ds_strerror(status)} (status {status})")


def ds_strerror(status: int) -> str:
    return lib().ds_strerror(status).decode()


def _check(status: int, where: str):
    if status != DS_OK:
        raise DsError(status, where)


def ds_workspace_size(n: int, N: int, kind: int, bits: int, chunk: int, nnz: int) -> int:
    comp = ds_compressor(kind, bits, chunk)
    return int(lib().ds_workspace_size(n, N, C.byref(comp), nnz))


def ds_init_raw(row_ptr, col_idx, w, n: int, N: int, ld: int, kind: int, bits: int, chunk: int,
                workspace_ptr: int, workspace_bytes: int, graph_n: int | None = None):
    """ds_init with host numpy arrays and a raw device pointer; returns (status, ctx)."""
    rp = None if row_ptr is None else np.ascontiguousarray(row_ptr, dtype=np.int32)
    ci = None if col_idx is None else np.ascontiguousarray(col_idx, dtype=np.int32)
    wv = None if w is None else np.ascontiguousarray(w, dtype=np.float32)
    g = ds_graph(n if graph_n is None else graph_n,
                 None if rp is None else rp.ctypes.data_as(C.POINTER(C.c_int32)),
                 None if ci is None else ci.ctypes.data_as(C.POINTER(C.c_int32)))
    comp = ds_compressor(kind, bits, chunk)
    ctx = C.c_void_p(0)
    st = lib().ds_init(C.byref(ctx), C.byref(g),
                       None if wv is None else wv.ctypes.data_as(C.POINTER(C.c_float)),
                       n, N, ld, C.byref(comp), C.c_void_p(workspace_ptr), workspace_bytes)
    return st, ctx


class DeepSqueeze:
    """A context plus the workspace tensor that backs it (torch owns the memory)."""

    def __init__(self, graph, N: int, ld: int, kind: int, bits: int, chunk: int, device="cuda:0",
                 guard_bytes: int = 0):
        """guard_bytes > 0 (a multiple of 256) puts that many bytes of a fixed pattern directly
        before and after the workspace; workspace_guards_intact() tells whether any of them
        changed -- a bounds check for kernels that write into the workspace."""
        import torch
        self.torch = torch
        self.n, self.N, self.ld = graph.n, int(N), int(ld)
        self.kind, self.bits, self.chunk = kind, bits, chunk
        self.device = torch.device(device)
        nnz = int(graph.row_ptr[-1])
        size = ds_workspace_size(self.n, self.N, kind, bits, chunk, nnz)
        if size == 0:
            raise DsError(DS_ERR_UNSUPPORTED, "ds_workspace_size")
        assert guard_bytes >= 0 and guard_bytes % 256 == 0
        self.guard_bytes, self.ws_bytes = guard_bytes, size
        with torch.cuda.device(self.device):
            self.workspace = torch.full((size + 256 + 2 * guard_bytes,), 0xA5, dtype=torch.uint8, device=self.device)
            ptr = (self.workspace.data_ptr() + 255) // 256 * 256 + guard_bytes
            self.ws_ptr = ptr
            st, ctx = ds_init_raw(graph.row_ptr, graph.col_idx, graph.w, self.n, self.N, self.ld,
                                  kind, bits, chunk, ptr, size)
        _check(st, "ds_init")
        self.ctx = ctx
        self.code_bits = 32 if kind == DS_COMP_IDENTITY else (1 if kind == DS_COMP_SIGN1_L1 else bits)

    def workspace_guards_intact(self) -> bool:
        """True if the pattern bytes before and after the workspace are all unchanged."""
        off = self.ws_ptr - self.workspace.data_ptr()
        front = self.workspace[off - self.guard_bytes: off]
        back = self.workspace[off + self.ws_bytes: off + self.ws_bytes + self.guard_bytes]
        return bool((front == 0xA5).all()) and bool((back == 0xA5).all())

    def ds_set_path(self, path: int):
        _check(lib().ds_set_path(self.ctx, path), "ds_set_path")

    def ds_tune(self, elems_per_lane: int):
        _check(lib().ds_tune(self.ctx, elems_per_lane), "ds_tune")

    def ds_get_info(self) -> ds_info:
        info = ds_info()
        _check(lib().ds_get_info(self.ctx, C.byref(info)), "ds_get_info")
        return info

    def ds_step(self, x, delta, a, c, sigma: float, noise: int, gamma: float, eta: float,
                seed: int, step: int, stream=None):
        """One iteration in place on the device tensors x, delta ([n][ld] float32)."""
        torch = self.torch
        for t in (x, delta, a, c):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (self.n, self.ld)
        gp = ds_grad_params(a.data_ptr(), c.data_ptr(), sigma, noise)
        hp = ds_hparams(gamma, eta)
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        _check(lib().ds_step(self.ctx, x.data_ptr(), delta.data_ptr(), C.byref(gp), C.byref(hp),
                             seed, step, C.c_void_p(s.cuda_stream)), "ds_step")

    def ds_run(self, x, delta, a, c, sigma: float, noise: int, gammas, etas, seed: int, step0: int, stream=None):
        """len(gammas) consecutive iterations from step0, replayed as one CUDA graph;
        iteration step0 + t uses gammas[t], etas[t]."""
        torch = self.torch
        for t in (x, delta, a, c):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (self.n, self.ld)
        T = len(gammas)
        assert len(etas) == T
        gp = ds_grad_params(a.data_ptr(), c.data_ptr(), sigma, noise)
        ga = (C.c_float * max(T, 1))(*[float(v) for v in gammas])
        ea = (C.c_float * max(T, 1))(*[float(v) for v in etas])
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        _check(lib().ds_run(self.ctx, x.data_ptr(), delta.data_ptr(), C.byref(gp), ga, ea, T,
                            seed, step0, C.c_void_p(s.cuda_stream)), "ds_run")

    def ds_run_resident(self, x, delta, a, c, sigma: float, noise: int, gammas, etas, seed: int, step0: int,
                        stream=None):
        """len(gammas) consecutive iterations from step0 in one launch of the resident
        kernel (small shapes only; raises DsError(DS_ERR_UNSUPPORTED) otherwise)."""
        torch = self.torch
        for t in (x, delta, a, c):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (self.n, self.ld)
        T = len(gammas)
        assert len(etas) == T
        gp = ds_grad_params(a.data_ptr(), c.data_ptr(), sigma, noise)
        ga = (C.c_float * max(T, 1))(*[float(v) for v in gammas])
        ea = (C.c_float * max(T, 1))(*[float(v) for v in etas])
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        _check(lib().ds_run_resident(self.ctx, x.data_ptr(), delta.data_ptr(), C.byref(gp), ga, ea, T,
                                     seed, step0, C.c_void_p(s.cuda_stream)), "ds_run_resident")

    def ds_step_g(self, x, delta, g, gamma: float, eta: float, seed: int, step: int, stream=None):
        """One iteration with the gradient supplied as a device tensor g[n][ld]."""
        torch = self.torch
        for t in (x, delta, g):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (self.n, self.ld)
        hp = ds_hparams(gamma, eta)
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        _check(lib().ds_step_g(self.ctx, x.data_ptr(), delta.data_ptr(), g.data_ptr(), C.byref(hp),
                               seed, step, C.c_void_p(s.cuda_stream)), "ds_step_g")

    def ds_ecsgd_step(self, x, delta, a, c, sigma: float, noise: int, gamma: float, seed: int, step: int,
                      stream=None):
        """One iteration of centralized error-compensated SGD in place on x, delta."""
        torch = self.torch
        for t in (x, delta, a, c):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (self.n, self.ld)
        gp = ds_grad_params(a.data_ptr(), c.data_ptr(), sigma, noise)
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        _check(lib().ds_ecsgd_step(self.ctx, x.data_ptr(), delta.data_ptr(), C.byref(gp), gamma,
                                   seed, step, C.c_void_p(s.cuda_stream)), "ds_ecsgd_step")

    def ds_ecsgd_step_g(self, x, delta, g, gamma: float, seed: int, step: int, stream=None):
        """The same iteration with the gradient supplied as a device tensor g[n][ld]."""
        torch = self.torch
        for t in (x, delta, g):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (self.n, self.ld)
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        _check(lib().ds_ecsgd_step_g(self.ctx, x.data_ptr(), delta.data_ptr(), g.data_ptr(), gamma,
                                     seed, step, C.c_void_p(s.cuda_stream)), "ds_ecsgd_step_g")

    def ds_step_host(self, x_h, delta_h, a_h, c_h, sigma, noise, gamma, eta, seed, step,
                     dev_x, dev_delta, dev_a, dev_c, stream=None):
        """Same iteration for host (ideally pinned) tensors; enqueues the copies
        in and out on the stream.  The caller synchronises before reading."""
        torch = self.torch
        hp = ds_hparams(gamma, eta)
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        _check(lib().ds_step_host(self.ctx, x_h.data_ptr(), delta_h.data_ptr(), a_h.data_ptr(),
                                  c_h.data_ptr(), sigma, noise, C.byref(hp), seed, step,
                                  dev_x.data_ptr(), dev_delta.data_ptr(), dev_a.data_ptr(),
                                  dev_c.data_ptr(), C.c_void_p(s.cuda_stream)), "ds_step_host")

    def ds_sync(self, stream=None):
        """Synchronise the stream and raise if a kernel gave up on a bounded wait."""
        s = self.torch.cuda.current_stream(self.device) if stream is None else stream
        _check(lib().ds_sync(self.ctx, C.c_void_p(s.cuda_stream)), "ds_sync")

    def ds_selftest_timeout(self, stream=None):
        s = self.torch.cuda.current_stream(self.device) if stream is None else stream
        _check(lib().ds_selftest_timeout(self.ctx, C.c_void_p(s.cuda_stream)), "ds_selftest_timeout")

    def ds_selftest_bounds(self, stream=None) -> int:
        """Returns the ds_status (DS_ERR_UNSUPPORTED unless the library is the checked build)."""
        s = self.torch.cuda.current_stream(self.device) if stream is None else stream
        return int(lib().ds_selftest_bounds(self.ctx, C.c_void_p(s.cuda_stream)))

    def ds_codes(self):
        """(codes_ptr, code_pitch_words, scales_ptr, scales_pitch) of the last step."""
        codes, scales = C.c_void_p(0), C.c_void_p(0)
        cp, sp = C.c_int64(0), C.c_int64(0)
        _check(lib().ds_codes(self.ctx, C.byref(codes), C.byref(cp), C.byref(scales), C.byref(sp)), "ds_codes")
        return codes.value, cp.value, scales.value, sp.value

    def codes_to_host(self):
        """Copy the last step's packed codes [n][words] and scales [n][M] to numpy."""
        torch = self.torch
        cptr, cpitch, sptr, spitch = self.ds_codes()
        base = self.ws_ptr
        ws = self.workspace[base - self.workspace.data_ptr():]
        words = (self.N * self.code_bits + 31) // 32
        codes = ws[cptr - base: cptr - base + self.n * cpitch * 4].view(torch.int32).view(self.n, cpitch)
        codes = codes[:, :words].cpu().numpy().view(np.uint32)
        if self.kind == DS_COMP_IDENTITY:
            return codes, np.zeros((self.n, 0), np.float32)
        ch = self.chunk if self.chunk > 0 else self.N
        M = (self.N + ch - 1) // ch
        scales = ws[sptr - base: sptr - base + self.n * spitch * 4].view(torch.float32).view(self.n, spitch)
        return codes, scales[:, :M].cpu().numpy()

    def close(self):
        if getattr(self, "ctx", None) is not None and self.ctx.value:
            lib().ds_destroy(self.ctx)
            self.ctx = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def ds_noise(out, n: int, N: int, which: int, noise: int, seed: int, step: int, stream=None):
    """Fill the device tensor out[n][ld] with one of the random streams."""
    import torch
    s = torch.cuda.current_stream(out.device) if stream is None else stream
    _check(lib().ds_noise(out.data_ptr(), n, N, out.shape[1], which, noise, seed, step,
                          C.c_void_p(s.cuda_stream)), "ds_noise")


def ds_node_scales_noalloc(scales_out, x, delta, a, c, sigma: float, noise: int, gamma: float,
                           N: int, comp_kind: int, seed: int, step: int, stream=None) -> int:
    """Per-node scales into the device tensor scales_out[n] without any device
    allocation (see include/deepsqueeze.h).  Returns the ds_status."""
    import torch
    n, ld = x.shape
    gp = ds_grad_params(a.data_ptr(), c.data_ptr(), sigma, noise)
    s = torch.cuda.current_stream(x.device) if stream is None else stream
    return int(lib().ds_node_scales_noalloc(scales_out.data_ptr(), x.data_ptr(), delta.data_ptr(),
                                            C.byref(gp), gamma, n, N, ld, comp_kind, seed, step,
                                            C.c_void_p(s.cuda_stream)))


def ds_selftest_math(stream=None):
    """Run the arithmetic self-test; returns (differing logarithms, differing square
    roots of -2 ln u, differing square roots of the Student-t radii)."""
    import torch
    counts = torch.zeros(3, dtype=torch.int64, device="cuda")
    s = torch.cuda.current_stream() if stream is None else stream
    _check(lib().ds_selftest_math(counts.data_ptr(), C.c_void_p(s.cuda_stream)), "ds_selftest_math")
    torch.cuda.synchronize()
    return tuple(int(v) for v in counts.cpu())
