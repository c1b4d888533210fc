"""GPU parity on the synthesized-layer sweep (chains of identical convolutions, the paper's
characterisation workload, Sec. II-B / III-B / IV): a seeded sample of the 1440 chain shapes plus
the layers the paper names, every contiguous fusion plan for chains of length <= 4 (unfused, all
fused, blocks of 2 and 4 beyond that), under both ways of fusing dense convolutions - hand-over in
shared memory where the fused kernel can hold the group, hand-over through L2 elsewhere.  No plan may
be refused.  The CPU checker runs in full where a chain is small and evaluates sampled output pixels
from their dependency cones (corners, edge midpoints, neighbours of tile boundaries) where it is not."""
import collections

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import executor as orc
from paper_2011_05630_b200 import binding as B, networks as nw, synth
from paper_2011_05630_b200.runtime import Session
from tests import gpu_util as G

DEPTHS, KS = (1, 2, 3, 4, 5, 6, 7, 8), (1, 3)
CS, HWS, NS = (16, 32, 64, 128, 256, 512), (7, 14, 28, 56, 112), (1, 8, 16)
FULL_FLOPS, CONE_BUDGET = 3e9, 4e9   # what the CPU checker may spend on one shape


def chain_flops(shape):
    d, k, c, hw, n = shape
    return 2.0 * d * n * hw * hw * k * k * c * c


def cone_flops(shape):
    """Work of the checker for ONE output pixel evaluated from its dependency cone."""
    d, k, c, hw, n = shape
    side = min(hw, 2 * d * (k // 2) + 1)
    return 2.0 * d * side * side * k * k * c * c


def sample_shapes(count, seed=7):
    """Seeded draw from the 1440 chain shapes (8 depths x 2 kernels x 6 widths x 5 sizes x 3 batches), keeping those the
    checker can afford in full or at three pixels at least."""
    rng = np.random.default_rng(seed)
    seen, out = set(), []
    while len(out) < count:
        s = (int(rng.choice(DEPTHS)), int(rng.choice(KS)), int(rng.choice(CS)), int(rng.choice(HWS)), int(rng.choice(NS)))
        if s not in seen and (chain_flops(s) <= FULL_FLOPS or 3 * cone_flops(s) <= CONE_BUDGET):
            seen.add(s)
            out.append(s)
    return out


# the layers the paper characterises fusion on: Fig. "Motivation"(b) {64,64,56x56}, {256,256,56x56}, {512,512,28x28};
# Fig. "Fusion"(b) {512,512,28x28} / {512,512,14x14}; Sec. IV-A's equal-operation triple; all 3x3, depth 4 and 8
NAMED = [(d, 3, c, hw, 1) for d in (4, 8) for c, hw in ((64, 56), (256, 56), (512, 28), (512, 14), (32, 224), (64, 112), (128, 56))]
SHAPES = sample_shapes(100) + NAMED + [(16, 3, 64, 56, 1)]   # ... and one chain of 16 (Fig. "Motivation"(b))


def cone_pixels(shape):
    d, k, c, hw, n = shape
    budget = int(max(3, min(32, CONE_BUDGET // cone_flops(shape))))
    pix = [(0, 0, 0), (n - 1, hw - 1, hw - 1), (n // 2, hw // 2, hw // 2), (0, 0, hw - 1), (n - 1, hw - 1, 0), (0, hw // 2, 0),
           (0, 0, hw // 2), (n - 1, hw // 2, hw - 1)]
    for t in (7, 8, 15, 16, 31, 32, 63, 64):   # neighbours of typical tile boundaries
        if t < hw:
            pix.append((n // 2, t, t))
            pix.append((0, t, hw - 1 - t))
    rng = np.random.default_rng(3)
    while len(pix) < budget:
        pix.append((int(rng.integers(n)), int(rng.integers(hw)), int(rng.integers(hw))))
    out = []
    for p in pix:
        if p not in out:
            out.append(p)
    return out[:budget]


def plans_of(depth):
    if depth <= 4:
        return list(G.all_contiguous_plans(depth))
    out = [list(range(depth)), list(range(1, depth, 2)) + ([depth - 1] if depth % 2 else []),
           list(range(3, depth, 4)) + ([depth - 1] if depth % 4 else [])]
    out.append([depth - 1] if depth <= 8 else list(range(7, depth, 8)) + ([depth - 1] if depth % 8 else []))
    return [sorted(set(p)) for p in out]


COVERAGE = collections.Counter()


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "L%d_k%d_c%d_hw%d_n%d" % s)
def test_sweep_chain_all_plans(shape):
    depth, k, c, hw, n = shape
    layers = nw.conv_chain(depth, c, k)
    tag = "sweep-%d-%d-%d-%d-%d" % shape
    params = synth.layer_params(tag, layers)
    x = synth.network_input(tag, n, hw, hw, c)
    sess = Session(layers, params, n, hw, hw, c)
    xd = sess.upload(x)
    sms = B.device_sm_count()
    full = chain_flops(shape) <= FULL_FLOPS
    if full:
        ref = orc.run_network(layers, params, x)
    else:
        pix = cone_pixels(shape)
        cone = orc.cone_outputs(layers, params, x, pix)
    fused_ran = collections.Counter()
    for option in (1, 2):   # hand-over in shared memory wherever the fused kernel holds the group / through L2
        B.net_set_option(sess.net, B.OPT_GROUP_KERNEL, option)
        for ends in plans_of(depth) + ([[depth - 1]] if option == 2 and 8 < depth <= 16 else []):   # (16 layers: one L2 group)
            if option == 2 and len(ends) == depth:
                continue   # the unfused plan does not depend on the option
            firsts = [0] + [e + 1 for e in ends[:-1]]
            assert all(B.net_group_is_legal(sess.net, a, e, sms) for a, e in zip(firsts, ends)), (shape, option, ends)
            what = "sweep %s option %d plan %s" % (shape, option, ends)
            if full:
                G.check_plan(sess, xd, ref, ends, [sms] * len(ends), what)
            else:
                sess.set_plan(ends, [sms] * len(ends))
                out = sess.run(xd).cpu().numpy()
                G.compare(np.stack([out[p[0], p[1], p[2], :] for p in pix]), cone, what + " (cone)")
            for kern, a, e in zip(sess.kernels(), firsts, ends):
                if e > a:
                    fused_ran[kern] += 1
    if depth > 1:   # every fused plan ran, through one of the two fused kernels - and on narrow chains through both
        assert sum(fused_ran.values()) >= 2 * (len(plans_of(depth)) - 1), (shape, fused_ran)
        assert fused_ran["conv_seq"] > 0
        COVERAGE["shapes with fused plans"] += 1
        COVERAGE["fused groups through chain_tc"] += fused_ran["chain_tc"]
        COVERAGE["fused groups through conv_seq"] += fused_ran["conv_seq"]
        if fused_ran["chain_tc"]:
            COVERAGE["shapes fused in shared memory"] += 1
    sess.close()


def test_sweep_coverage_report():
    """Runs after the sweep: most shapes must have been fused in shared memory too, wide layers included."""
    print("sweep coverage:", dict(COVERAGE))
    if COVERAGE["shapes with fused plans"]:
        assert COVERAGE["shapes fused in shared memory"] >= 0.8 * COVERAGE["shapes with fused plans"], dict(COVERAGE)
