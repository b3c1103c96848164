"""Mask-flip statistics of the AdamS step under general N:M and a sweep of the L1 coefficient.

    python -m paper_2509_25996_b200.flip_sweep --workload llama2_7b --nm 4:8 1:4 --l1 0 1e-4 1e-3 1e-2 --steps 3

For every (N:M, lambda) the state is drawn afresh (same seed), then `steps` consecutive iterations run with a
fresh seeded gradient each; every iteration reselects the mask and counts ||M_t - M_{t-1}||_0 (App. C).  The
first iteration only establishes M_1 (there is no earlier mask), so flips are reported from the second on,
as a count and as the flip rate r_t = flips / parameters.  All arithmetic runs in the CUDA library; this
module allocates, draws gradients, launches and prints.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as B
from . import workloads
from .runner import DeviceModelState, Hyper


def run(workload: str, nm, l1_values, steps: int, seed: int = 0, device="cuda:0", first_step: int = 1000):
    wl = workloads.workload(workload)
    dev = torch.device(device)
    rows = []
    for N, M in nm:
        enc = 0 if (N, M) == (2, 4) else B.CAST_F_META_BITMASK
        for lam in l1_values:
            state = DeviceModelState(wl.shapes, N, M, seed=seed, device=dev, scale_mode="ones")
            hyper = Hyper(l1_coeff=lam, step=first_step, total_steps=wl.total_steps)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            flips, times = [], []
            for k in range(steps):
                if k > 0:                                    # fresh gradient for every later iteration
                    for i, mat in enumerate(state.mats):
                        mat.g.copy_(workloads.gen_gradient(mat.rows, mat.cols, seed, i, hyper.step, device=dev))
                state.flips.zero_()
                ev[0].record()
                state.step(hyper, B.CAST_F_RESELECT | B.CAST_F_COUNT_FLIPS | enc)
                ev[1].record()
                torch.cuda.synchronize(dev)
                times.append(ev[0].elapsed_time(ev[1]))
                flips.append(int(state.flips.item()))
                hyper.step += 1
            n = state.n_params
            state.close()
            del state
            torch.cuda.empty_cache()
            ms = min(times[1:]) if steps > 1 else times[0]
            rows.append(dict(workload=wl.name, nm=f"{N}:{M}", l1_coeff=lam, params=n, ms_per_step=ms,
                             gbs=n * 28.25 / ms / 1e6, flips_per_step=flips[1:], flip_rate=[f / n for f in flips[1:]]))
    return rows


def main():
    p = argparse.ArgumentParser()
    p.add_argument("--workload", default="llama2_7b")
    p.add_argument("--nm", nargs="+", default=["4:8", "1:4"])
    p.add_argument("--l1", nargs="+", type=float, default=[0.0, 1e-4, 1e-3, 1e-2])
    p.add_argument("--steps", type=int, default=3)
    p.add_argument("--seed", type=int, default=0)
    p.add_argument("--json", action="store_true")
    a = p.parse_args()
    nm = [tuple(int(x) for x in s.split(":")) for s in a.nm]
    rows = run(a.workload, nm, a.l1, a.steps, a.seed)
    if a.json:
        print(json.dumps(rows))
        return
    print(f"{'workload':12s} {'N:M':>5s} {'lambda':>8s} {'ms/step':>9s} {'GB/s':>7s}  flips per step (r_t)")
    for r in rows:
        fl = ", ".join(f"{f} ({q:.3e})" for f, q in zip(r["flips_per_step"], r["flip_rate"]))
        print(f"{r['workload']:12s} {r['nm']:>5s} {r['l1_coeff']:8.0e} {r['ms_per_step']:9.3f} {r['gbs']:7.0f}  {fl}")


if __name__ == "__main__":
    main()
