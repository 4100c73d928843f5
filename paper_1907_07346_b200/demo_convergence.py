"""Convergence on the synthetic quadratic for different compressors.

    python -m paper_1907_07346_b200.demo_convergence [--nodes 8] [--params 65536] [--steps 300]

Runs DeepSqueeze (Algorithm 1) on one GPU for a ring of workers with the same
objective, noise and step sizes and a different compressor each time, and prints
for each the distance of the node average to the optimum of Eq. 1 and the
consensus distance ||X (I - A_n)||_F (the quantity the paper's key lemma
bounds).  The uncompressed row is D-PSGD (Section 3.2), the baseline of the
paper's Figure 1; the paper reports that 4 bits track it closely and 2 bits
converge somewhat slower.
"""
from __future__ import annotations

import argparse

import numpy as np


def run(args):
    import torch
    from . import binding as B
    from . import inputs as I

    g = I.ring(args.nodes)
    N = args.params
    ld = I.row_pitch(N)
    w = I.Workload("demo", args.nodes, "ring", N, 0, 0, 0, I.NOISE_GAUSS, args.sigma, args.gamma, args.eta,
                   args.steps, "uniform", 20190707)
    a_h, c_h = I.objective(w, ld)
    xstar = (a_h[:, :N].astype(np.float64) * c_h[:, :N]).sum(0) / a_h[:, :N].astype(np.float64).sum(0)
    a, c = torch.from_numpy(a_h).cuda(), torch.from_numpy(c_h).cuda()
    rows = [("none (D-PSGD)", I.COMP_IDENTITY, 32, 0), ("8-bit stochastic", I.COMP_UNIFORM_STOCH_MAXABS, 8, 512),
            ("4-bit stochastic", I.COMP_UNIFORM_STOCH_MAXABS, 4, 512), ("2-bit stochastic", I.COMP_UNIFORM_STOCH_MAXABS, 2, 512),
            ("4-bit nearest + norm", I.COMP_UNIFORM_NEAREST_L2, 4, 512), ("2-bit nearest + norm", I.COMP_UNIFORM_NEAREST_L2, 2, 512),
            # the paper's own setting (Section 5): b bits per element and ONE norm per tensor
            ("4-bit + norm per tensor", I.COMP_UNIFORM_NEAREST_L2, 4, 0), ("2-bit + norm per tensor", I.COMP_UNIFORM_NEAREST_L2, 2, 0),
            ("1-bit sign", I.COMP_SIGN1_L1, 1, 512)]
    out = []
    for name, kind, bits, chunk in rows:
        ds = B.DeepSqueeze(g, N, ld, kind, bits, chunk)
        x = torch.zeros((args.nodes, ld), dtype=torch.float32, device="cuda")
        d = torch.zeros_like(x)
        for t in range(args.steps):
            ds.ds_step(x, d, a, c, args.sigma, I.NOISE_GAUSS, args.gamma, args.eta, 7, t)
        ds.ds_sync()
        xs = x[:, :N].double().cpu().numpy()
        xbar = xs.mean(0)
        out.append((name, bits, float(np.linalg.norm(xbar - xstar) / np.linalg.norm(xstar)),
                    float(np.linalg.norm(xs - xbar[None, :])), float(d[:, :N].double().norm().cpu())))
        ds.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--nodes", type=int, default=8)
    ap.add_argument("--params", type=int, default=65536)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--gamma", type=float, default=0.05)
    ap.add_argument("--eta", type=float, default=0.4)
    ap.add_argument("--sigma", type=float, default=0.1)
    args = ap.parse_args()
    print(f"ring of {args.nodes}, {args.params} parameters, {args.steps} steps, gamma={args.gamma}, eta={args.eta}")
    print(f"{'compressor':24s} {'bits':>4s} {'|xbar-x*|/|x*|':>15s} {'consensus':>11s} {'|delta|':>10s}")
    for name, bits, dist, cons, dn in run(args):
        print(f"{name:24s} {bits:4d} {dist:15.5f} {cons:11.4f} {dn:10.4f}")


if __name__ == "__main__":
    main()
