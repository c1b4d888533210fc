"""Re-characterisation of the device for the auto-tuner (the paper's Sec. II-B / IV-A procedure, on the GPU at hand).

The paper fits Eq. 5 - the core count of a layer as a function of its channel size and operation count - to
micro-benchmarks of synthesised single layers on its accelerator.  This module repeats that on the device in use:
it times single convolution layers of the characterisation sweep (channels x image size x kernel size x batch)
on every SM count of the reduced set through the C ABI (`dlf_net_time_span`, one layer = one candidate group),
takes for every layer the smallest SM count whose time is within `slack` of the best, and fits

    S = kappa_c * log2(C_out) + kappa_o * log2(ops) + kappa0          (least squares)

which is Eq. 5's proportionality with its two weights and the affine map to an SM count fitted together
(alpha = kappa_c / kappa, beta = kappa_o / kappa for any common scale kappa).  It also times the smaller layers on ONE
SM and reads off Algorithm 1's OpCount_critical as the paper defines it (Sec. IV-C): the operation count from which a
single core's throughput stays within a given fraction of its best.  Only argument marshalling and the fits happen here;
every timed step runs inside libdlfusion.so.

    python -m paper_2011_05630_b200.characterise [--quick]
"""
from __future__ import annotations

import argparse
import json
import math

import numpy as np


def sweep_layers(quick):
    chans = (16, 64, 256) if quick else (16, 32, 64, 128, 256, 512)
    sizes = (7, 28, 112) if quick else (7, 14, 28, 56, 112)
    batches = (1, 16) if quick else (1, 8, 16)
    for k in (1, 3):
        for c in chans:
            for hw in sizes:
                for n in batches:
                    if 2.0 * n * hw * hw * k * k * c * c > 4e11:   # keep one timing well under a millisecond
                        continue
                    yield n, hw, c, k


def time_layer(n, hw, c, k, sm_choices, warmup=1, iters=3):
    import torch
    from . import binding as B
    from .runtime import Session
    layer = dict(op="conv", act="relu", cin=c, cout=c, kh=k, kw=k, stride=1, pad=k // 2, groups=1, src=-1, res_src=-2, pool=0)
    rng = np.random.default_rng(1)
    params = [((rng.standard_normal((c, k, k, c)) * (k * k * c) ** -0.5).astype(np.float16),
               (rng.standard_normal(c) * 0.1).astype(np.float32))]
    x = rng.uniform(-1, 1, (n, hw, hw, c)).astype(np.float16)
    sess = Session([layer], params, n, hw, hw, c)
    xd = sess.upload(x)
    stream = torch.cuda.current_stream().cuda_stream
    times = [B.net_time_span(sess.net, 0, 0, s, xd.data_ptr(), stream, warmup, iters, prepare=False) for s in sm_choices]
    ops = B.net_layer_info(sess.net, 0)[1]
    sess.close()
    return ops, times


def fit(rows, slack=0.05):
    """rows: (c_out, ops, sm_choices, times).  Returns (kappa_c, kappa_o, kappa0, rms error in SMs)."""
    a, y = [], []
    for c, ops, choices, times in rows:
        best = min(times)
        s_star = min(s for s, t in zip(choices, times) if t <= best * (1.0 + slack))
        a.append([math.log2(c), math.log2(ops), 1.0])
        y.append(float(s_star))
    a, y = np.asarray(a), np.asarray(y)
    coef, *_ = np.linalg.lstsq(a, y, rcond=None)
    rms = float(np.sqrt(np.mean((a @ coef - y) ** 2)))
    return float(coef[0]), float(coef[1]), float(coef[2]), rms


def critical_ops(single, frac=0.8):
    """single: (ops, seconds on one SM) per layer.  The smallest operation count from which every layer reaches `frac` of
    the best single-SM throughput seen (Sec. IV-C: where single-core efficiency saturates)."""
    rows = sorted(single)
    thr = [o / t for o, t in rows]
    best = max(thr)
    crit = rows[-1][0]
    for (o, _), r in zip(reversed(rows), reversed(thr)):
        if r < frac * best:
            break
        crit = o
    return float(crit), float(best)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true", help="a third of the sweep")
    ap.add_argument("--slack", type=float, default=0.05, help="a smaller SM count counts as best within this fraction")
    args = ap.parse_args()
    from . import binding as B, plans
    choices = plans.sm_fractions(B.device_sm_count())
    rows, single = [], []
    for n, hw, c, k in sweep_layers(args.quick):
        ops, times = time_layer(n, hw, c, k, choices)
        rows.append((c, ops, choices, times))
        best = min(times)
        one = None
        if ops <= 2e10:   # one SM: up to ~150 times longer than on the whole chip
            one = time_layer(n, hw, c, k, [1])[1][0]
            single.append((ops, one * 1e-3))
        print("n %2d  %3dx%-3d c %3d k%d  ops %.3g  best %.1f us at S=%d%s" % (
            n, hw, hw, c, k, ops, best * 1e3, choices[times.index(best)],
            "" if one is None else "  one SM %.1f us (%.2f TFLOP/s)" % (one * 1e3, ops / (one * 1e-3) / 1e12)), flush=True)
    kc, ko, k0, rms = fit(rows, args.slack)
    crit, best_thr = critical_ops(single)
    print(json.dumps({"layers": len(rows), "sm_choices": choices, "kappa_c": kc, "kappa_o": ko, "kappa0": k0,
                      "alpha_over_beta": kc / ko if ko else None, "rms_error_sms": rms,
                      "paper_alpha_over_beta": 0.316 / 0.659, "op_critical_per_sm": crit,
                      "best_single_sm_tflops": best_thr / 1e12, "paper_op_critical": "10^1.25 G operations per core (MLU100)"}))


if __name__ == "__main__":
    main()
