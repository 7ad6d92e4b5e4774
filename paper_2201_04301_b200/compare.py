"""G-CADA against its two special cases on one synthetic workload.

    python -m paper_2201_04301_b200.compare [--config linreg784] [--iters 2000] [--every 100]

The three schemes of the paper's comparison (Section VI) are one method with
different settings, all run by the same CUDA library:

  G-CADA            M workers in groups of M_G, threshold constant c
  CADA              groups of one worker (M_G = 1): every worker has its own shard
  distributed Adam  groups of one worker and c = 0: every worker uploads every iteration

For each scheme one JSON line per sampling point is printed: iteration,
simulated wall-clock (Section II-B), training loss over the first rows of the
training set (gcada_eval_loss), communication load (Eqs. 5, 19) and
computation load (Eqs. 6, 22), i.e. the three curves of the paper's figure on
synthetic data.  Only argument marshalling happens here.
"""
import argparse
import json

from . import binding
from .workloads import make_workload


def schemes(w, c_cada):
    return {
        "g-cada": dict(M_G=w["M_G"], c=w["c"]),
        "cada": dict(M_G=1, c=c_cada),
        "adam": dict(M_G=1, c=0.0),
    }


def run_scheme(w, M_G, c, iters, every, eval_rows, stream=None):
    """One run; returns a list of dicts (k, wall, loss, uploads, comm, comp)."""
    ws = dict(w)
    ws.update(M_G=M_G, c=c)
    g = binding.from_workload(ws, stream=stream)
    out = []
    k = 0
    while True:
        up, comm, comp = g.get_comm_count()
        out.append(dict(k=k, wall=g.get_wallclock()[0], loss=g.eval_loss(0, eval_rows), uploads=up, comm=comm,
                        comp=comp))
        if k >= iters:
            break
        n = min(every, iters - k)
        g.step(n)
        k += n
    g.close()
    return out


def main():
    import torch
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="linreg784")
    ap.add_argument("--iters", type=int, default=2000)
    ap.add_argument("--every", type=int, default=100)
    ap.add_argument("--eval-rows", type=int, default=10000)
    ap.add_argument("--c-cada", type=float, default=2.0, help="threshold constant of the CADA run (the paper's 2)")
    args = ap.parse_args()
    w = make_workload(args.config, device="cuda")
    stream = torch.cuda.Stream()
    for name, kw in schemes(w, args.c_cada).items():
        for rec in run_scheme(w, kw["M_G"], kw["c"], args.iters, args.every, min(args.eval_rows, w["X"].shape[0]),
                              stream):
            print(json.dumps(dict(scheme=name, **rec)), flush=True)


if __name__ == "__main__":
    main()
