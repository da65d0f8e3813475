"""Runs lbp_backward on one synthetic layer a few times: a small, fixed workload
for profilers (ncu) and quick timing.

  python -m paper_2309_15275_b200.profile_case --config 3 --layer 2 --rank 8 --iters 3
"""
from __future__ import annotations

import argparse
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def main() -> int:
    import torch
    import paper_2309_15275_b200 as lbp
    import synth

    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--layer", type=int, default=2)
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--rank", type=int, default=8)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--fullrank", action="store_true")
    args = ap.parse_args()

    dev = torch.device("cuda:0")
    case = synth.config_cases(args.config)[args.layer]
    x, gy, w = (t.to(dev) for t in synth.make_layer_inputs(case, batch=args.batch))
    k = case.k
    bases = lbp.lbp_select_bases(k, lbp.SEL_PREFIX, args.rank)
    r = k * k if args.fullrank else args.rank
    ws = lbp.alloc_workspace(x, gy, k, r)
    gx = torch.empty_like(x)
    gw = torch.empty((case.Cout, case.Cin), dtype=torch.float32, device=dev)
    beg, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for it in range(args.iters + 1):
        if it == 1:
            beg.record()
        if args.fullrank:
            lbp.lbp_backward_fullrank(x, gy, w, k, g_x=gx, g_W=gw, ws=ws)
        else:
            lbp.lbp_backward(x, gy, w, k, bases, g_x=gx, g_W=gw, ws=ws)
    end.record()
    st = lbp.lbp_poll_status(ws)
    print(f"{case.name} B={x.shape[0]} r={r}: {beg.elapsed_time(end) / max(args.iters, 1) * 1e3:.1f} us/call, "
          f"status {st}")
    return 0 if st == 0 else 1


if __name__ == "__main__":
    sys.exit(main())
