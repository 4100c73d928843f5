"""Seeded synthetic inputs: node graphs, mixing matrices and objective data.

This module only GENERATES inputs (graphs in CSR form, the weight values of W,
the diagonal quadratic's a and c, the workload table).  It holds none of the
method's arithmetic, so both the CUDA library's callers and the CPU checker
may use it.

The workloads stand in for the paper's CIFAR-10 / ResNet-20 runs (Section 5,
"Experimental Setup"): each node owns a diagonal quadratic
f_i(x) = 1/2 sum_k a_ik (x_k - c_ik)^2 whose stochastic gradient is
a_ik (x_k - c_ik) + sigma * noise, with vector lengths of ResNet-18 / ResNet-50
size and the graphs the decentralized setting uses (Section 3: a symmetric
doubly stochastic W over a connected graph, every node its own neighbour).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

COMP_IDENTITY = 0
COMP_SIGN1_L1 = 1
COMP_UNIFORM_STOCH_MAXABS = 2
COMP_UNIFORM_NEAREST_L2 = 3

NOISE_NONE = 0
NOISE_GAUSS = 1
NOISE_STUDENT_T3 = 2
NOISE_STUDENT_T3_IID = 3


@dataclass
class Graph:
    """CSR adjacency (columns ascending, self loop included) plus W values."""
    n: int
    row_ptr: np.ndarray   # int32 [n+1]
    col_idx: np.ndarray   # int32 [nnz]
    w: np.ndarray         # float32 [nnz], W_ij in CSR order
    name: str = ""

    def dense(self) -> np.ndarray:
        W = np.zeros((self.n, self.n), dtype=np.float64)
        for i in range(self.n):
            for e in range(self.row_ptr[i], self.row_ptr[i + 1]):
                W[i, self.col_idx[e]] = float(self.w[e])
        return W


def _from_neighbour_sets(nbrs: list[set[int]], name: str) -> Graph:
    n = len(nbrs)
    row_ptr = np.zeros(n + 1, dtype=np.int32)
    cols: list[int] = []
    vals: list[float] = []
    for i, s in enumerate(nbrs):
        members = sorted(s | {i})
        weight = 1.0 / len(members)
        cols.extend(members)
        vals.extend([weight] * len(members))
        row_ptr[i + 1] = len(cols)
    return Graph(n, row_ptr, np.asarray(cols, dtype=np.int32),
                 np.asarray(vals, dtype=np.float32), name)


def ring(n: int) -> Graph:
    """Ring: node i is linked to i-1 and i+1 (mod n); uniform weights."""
    if n < 3:
        raise ValueError("a ring needs n >= 3")
    return _from_neighbour_sets([{(i - 1) % n, (i + 1) % n} for i in range(n)],
                                f"ring{n}")


def complete(n: int) -> Graph:
    """Complete graph with W_ij = 1/n: every node averages all nodes (the
    parameter server of centralized training)."""
    if n < 1:
        raise ValueError("n >= 1")
    return _from_neighbour_sets([set(range(n)) - {i} for i in range(n)], f"complete{n}")


def torus(rows: int, cols: int) -> Graph:
    """2-D torus rows x cols: four neighbours (up, down, left, right, wrapped)."""
    if rows < 3 or cols < 3:
        raise ValueError("a torus needs both sides >= 3")
    nbrs = []
    for r in range(rows):
        for c in range(cols):
            nbrs.append({((r - 1) % rows) * cols + c, ((r + 1) % rows) * cols + c,
                         r * cols + (c - 1) % cols, r * cols + (c + 1) % cols})
    return _from_neighbour_sets(nbrs, f"torus{rows}x{cols}")


def exponential(n: int) -> Graph:
    """Exponential graph: i is linked to i +- 2^k (mod n) for 2^k < n.

    Offsets that coincide modulo n (for n = 64, +32 and -32) give one neighbour;
    all nodes have the same degree, so uniform weights over self and neighbours
    keep W symmetric and doubly stochastic.
    """
    nbrs = []
    for i in range(n):
        s = set()
        k = 1
        while k < n:
            s.add((i + k) % n)
            s.add((i - k) % n)
            k *= 2
        s.discard(i)
        nbrs.append(s)
    return _from_neighbour_sets(nbrs, f"exp{n}")


@dataclass
class Workload:
    """One synthetic configuration (all sizes in elements)."""
    name: str
    n: int
    graph: str                 # "ring" | "torus4x8" | "exp"
    N: int
    comp_kind: int
    bits: int
    chunk: int                 # 0 = one scale per node
    noise_kind: int
    sigma: float
    gamma: float
    eta: float
    steps: int
    a_dist: str                # "uniform" U[0.5,2] | "loguniform" 10^U[-1,1]
    seed: int
    extra: dict = field(default_factory=dict)

    def build_graph(self) -> Graph:
        if self.graph == "ring":
            return ring(self.n)
        if self.graph.startswith("torus"):
            r, c = self.graph[5:].split("x")
            return torus(int(r), int(c))
        if self.graph == "exp":
            return exponential(self.n)
        raise ValueError(self.graph)

    def with_size(self, N: int) -> "Workload":
        """Same configuration on a shorter (or longer) parameter vector."""
        w = Workload(**{**self.__dict__})
        w.N = int(N)
        return w

    def describe(self) -> str:
        comp = {COMP_IDENTITY: "identity", COMP_SIGN1_L1: "1-bit sign l1-scale",
                COMP_UNIFORM_STOCH_MAXABS: f"{self.bits}-bit uniform stochastic max-abs",
                COMP_UNIFORM_NEAREST_L2: f"{self.bits}-bit nearest-level norm-matched"}[self.comp_kind]
        chunk = f"chunk {self.chunk}" if self.chunk else "per-node scale"
        noise = {NOISE_NONE: "none", NOISE_GAUSS: "gauss", NOISE_STUDENT_T3: "student-t3(spherical pairs)",
                 NOISE_STUDENT_T3_IID: "student-t3(independent coordinates)"}[self.noise_kind]
        return (f"{self.name}: n={self.n} {self.graph} N={self.N} {comp} {chunk} "
                f"noise={noise} sigma={self.sigma} gamma={self.gamma} eta={self.eta}")


_BASE_SEED = 190707346

WORKLOADS = {
    "cfg1": Workload("cfg1", 4, "ring", 65_536, COMP_SIGN1_L1, 1, 0, NOISE_GAUSS,
                     0.1, 0.05, 0.5, 20, "uniform", _BASE_SEED + 1),
    "cfg2": Workload("cfg2", 8, "ring", 11_173_962, COMP_SIGN1_L1, 1, 4096, NOISE_GAUSS,
                     0.1, 0.01, 0.3, 100, "loguniform", _BASE_SEED + 2),
    "cfg3": Workload("cfg3", 16, "ring", 25_557_032, COMP_UNIFORM_STOCH_MAXABS, 4, 512,
                     NOISE_GAUSS, 0.1, 0.01, 0.5, 50, "uniform", _BASE_SEED + 3),
    "cfg4": Workload("cfg4", 32, "torus4x8", 25_557_032, COMP_UNIFORM_STOCH_MAXABS, 2, 256,
                     NOISE_STUDENT_T3, 0.1, 0.005, 0.4, 50, "uniform", _BASE_SEED + 4),
    # cfg3's shape with the paper's own codec (Section 5: 4 bits + Euclidean norm, nearest level)
    "cfg3_l2": Workload("cfg3_l2", 16, "ring", 25_557_032, COMP_UNIFORM_NEAREST_L2, 4, 512,
                        NOISE_GAUSS, 0.1, 0.01, 0.5, 50, "uniform", _BASE_SEED + 6),
    "cfg5": Workload("cfg5", 64, "exp", 4_194_304, COMP_SIGN1_L1, 1, 1024, NOISE_GAUSS,
                     0.1, 0.01, 0.5, 200, "uniform", _BASE_SEED + 5),
}


def round_up(v: int, m: int) -> int:
    return (v + m - 1) // m * m


def row_pitch(N: int) -> int:
    """Row pitch in elements used by the harness: N rounded up to 32."""
    return round_up(N, 32)


def objective(workload: Workload, ld: int | None = None):
    """Seeded a, c as float32 arrays [n][ld]; padding columns are zero.

    a ~ U[0.5, 2] or 10^U[-1, 1]; c ~ N(0, 1).  Rows are generated one at a
    time so that the full-size workloads need no float64 temporaries of the
    whole matrix.
    """
    n, N = workload.n, workload.N
    ld = row_pitch(N) if ld is None else ld
    a = np.zeros((n, ld), dtype=np.float32)
    c = np.zeros((n, ld), dtype=np.float32)
    for i in range(n):
        rng = np.random.Generator(np.random.Philox(key=workload.seed + 1000 * (i + 1)))
        u = rng.random(N, dtype=np.float32)
        if workload.a_dist == "uniform":
            a[i, :N] = np.float32(0.5) + np.float32(1.5) * u
        elif workload.a_dist == "loguniform":
            a[i, :N] = np.power(np.float32(10.0), np.float32(2.0) * u - np.float32(1.0),
                                dtype=np.float32)
        else:
            raise ValueError(workload.a_dist)
        c[i, :N] = rng.standard_normal(N, dtype=np.float32)
    return a, c


def code_words(N: int, code_bits: int) -> int:
    """32-bit words per node for N packed codes of code_bits bits."""
    return (N * code_bits + 31) // 32
