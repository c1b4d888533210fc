"""Command line for one layer: builds a single convolution / depthwise / max-pool layer, or one fused inverted-residual
block, with the seeded synthetic tensors of the workloads, runs it a few times through the C ABI and prints which kernel
ran (handy under a profiler, or to try a shape before putting it into a network).

    python -m paper_2011_05630_b200.layer_cli N H W CIN COUT K [--as-chain] [--reps 3] [--stride 1]
                                              [--op conv|dwconv|maxpool] [--mbconv HID]
                                              [--then K:C,K:C,...] [--residual] [--group-kernel 0|1|2]

--then appends dense stride-1 convolutions (kernel:channels) and runs all of them as ONE group; --residual adds the
group's input to its last layer; --group-kernel picks the hand-over (1 shared memory, 2 L2, 0 the library's choice).
--op dwconv runs a depthwise KxK layer (COUT = CIN), --op maxpool a KxK max-pool; --mbconv HID runs the fused
inverted-residual block CIN -> HID (1x1) -> depthwise 3x3 (--stride) -> COUT (1x1) as one group.
"""
from __future__ import annotations

import argparse


def main():
    ap = argparse.ArgumentParser()
    for name in ("n", "h", "w", "cin", "cout", "k"):
        ap.add_argument(name, type=int)
    ap.add_argument("--as-chain", action="store_true", help="use the fused-chain kernel for the single layer")
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--op", default="conv", choices=["conv", "dwconv", "maxpool"])
    ap.add_argument("--mbconv", type=int, default=0, help="hidden width of a fused inverted-residual block")
    ap.add_argument("--then", default="", help="more dense convolutions K:C,K:C,... fused with the first into one group")
    ap.add_argument("--residual", action="store_true", help="add the group's input to its last layer (channels must match)")
    ap.add_argument("--group-kernel", type=int, default=0, choices=[0, 1, 2])
    a = ap.parse_args()
    from . import binding as B
    from .runtime import Session
    def mk(op, cin, cout, k, stride, src, act="relu", res=-2):
        return dict(op=op, act=act, cin=cin, cout=cout, kh=k, kw=k, stride=stride, pad=k // 2, groups=cin if op == "dwconv" else 1,
                    src=src, res_src=res, pool=0)
    if a.mbconv:
        res = -1 if (a.stride == 1 and a.cin == a.cout) else -2
        layers = [mk("conv", a.cin, a.mbconv, 1, 1, -1, "relu6"), mk("dwconv", a.mbconv, a.mbconv, 3, a.stride, 0, "relu6"),
                  mk("conv", a.mbconv, a.cout, 1, 1, 1, "none", res)]
    else:
        layers = [mk(a.op, a.cin, a.cin if a.op != "conv" else a.cout, a.k, a.stride, -1, "none" if a.op == "maxpool" else "relu")]
    for spec in [t for t in a.then.split(",") if t]:
        k, c = (int(v) for v in spec.split(":"))
        layers.append(mk("conv", layers[-1]["cout"], c, k, 1, len(layers) - 1))
    if a.residual:
        layers[-1]["res_src"] = -1
    from . import synth
    params = synth.layer_params("layer_cli", layers)
    x = synth.network_input("layer_cli", a.n, a.h, a.w, a.cin)
    sess = Session(layers, params, a.n, a.h, a.w, a.cin)
    xd = sess.upload(x)
    B.net_set_option(sess.net, B.OPT_CUDA_GRAPH, 0)
    B.net_set_option(sess.net, B.OPT_SINGLE_AS_CHAIN, 1 if a.as_chain else 0)
    B.net_set_option(sess.net, B.OPT_GROUP_KERNEL, a.group_kernel)
    sess.set_plan([len(layers) - 1], [B.device_sm_count()])
    for _ in range(a.reps):
        sess.run(xd)
    print("ran", sess.kernels(), "x", a.reps)


if __name__ == "__main__":
    main()
