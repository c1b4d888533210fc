"""Runs one convolution layer a few times through the C ABI (for profiler captures and quick checks).

    python -m paper_2011_05630_b200.layer_cli N H W CIN COUT K [--as-chain] [--reps 3] [--stride 1]
"""
from __future__ import annotations

import argparse

import numpy as np


def main():
    ap = argparse.ArgumentParser()
    for name in ("n", "h", "w", "cin", "cout", "k"):
        ap.add_argument(name, type=int)
    ap.add_argument("--as-chain", action="store_true", help="use the fused-chain kernel for the single layer")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    a = ap.parse_args()
    from . import binding as B
    from .runtime import Session
    layer = dict(op="conv", act="relu", cin=a.cin, cout=a.cout, kh=a.k, kw=a.k, stride=a.stride, pad=a.k // 2, groups=1,
                 src=-1, res_src=-2, pool=0)
    rng = np.random.default_rng(0)
    params = [((rng.standard_normal((a.cout, a.k, a.k, a.cin)) * (a.k * a.k * a.cin) ** -0.5).astype(np.float16),
               (rng.standard_normal(a.cout) * 0.1).astype(np.float32))]
    x = rng.uniform(-1, 1, (a.n, a.h, a.w, a.cin)).astype(np.float16)
    sess = Session([layer], params, a.n, a.h, a.w, a.cin)
    xd = sess.upload(x)
    B.net_set_option(sess.net, B.OPT_CUDA_GRAPH, 0)
    B.net_set_option(sess.net, B.OPT_SINGLE_AS_CHAIN, 1 if a.as_chain else 0)
    sess.set_plan([0], [B.device_sm_count()])
    for _ in range(a.reps):
        sess.run(xd)
    print("ran", sess.kernels(), "x", a.reps)


if __name__ == "__main__":
    main()
