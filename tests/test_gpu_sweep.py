"""GPU parity on the synthesized-layer sweep (chains of identical convolutions, the paper's
characterisation workload): a seeded sample of the 1440 chain shapes, every contiguous fusion
plan for chains of length <= 4, full CPU checker where a chain is small and the cone evaluation
(sampled output pixels, including the corners, edge midpoints and tile-boundary neighbours)
where it is not."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import executor as orc
from paper_2011_05630_b200 import binding as B, networks as nw, synth
from paper_2011_05630_b200.runtime import Session
from tests import gpu_util as G

DEPTHS, KS = (1, 2, 3, 4, 8), (1, 3)
CS, HWS, NS = (16, 32, 64, 128, 256, 512), (7, 14, 28, 56, 112), (1, 8, 16)


def sample_shapes(count, seed=7):
    """Seeded draw from the 1440 chain shapes, keeping those the checker can afford."""
    rng = np.random.default_rng(seed)
    seen, out = set(), []
    while len(out) < count:
        s = (int(rng.choice(DEPTHS)), int(rng.choice(KS)), int(rng.choice(CS)), int(rng.choice(HWS)), int(rng.choice(NS)))
        if s not in seen and (chain_flops(s) <= 12e9 or cone_flops(s) <= 2e9):
            seen.add(s)
            out.append(s)
    return out


def chain_flops(shape):
    d, k, c, hw, n = shape
    return 2.0 * d * n * hw * hw * k * k * c * c


def cone_flops(shape):
    """Work of the checker for ONE output pixel evaluated from its dependency cone."""
    d, k, c, hw, n = shape
    side = min(hw, 2 * d * (k // 2) + 1)
    return 2.0 * d * side * side * k * k * c * c


SHAPES = sample_shapes(14) + [(8, 3, 64, 56, 8), (4, 3, 512, 28, 16), (8, 1, 128, 112, 16), (2, 3, 16, 112, 16)]


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
    full = chain_flops(shape) <= 12e9
    if full:
        ref = orc.run_network(layers, params, x)
    else:  # cone evaluation of sampled output pixels of the last layer
        rng = np.random.default_rng(3)
        pix = {(0, 0, 0), (n - 1, hw - 1, hw - 1), (0, 0, hw - 1), (n - 1, hw - 1, 0), (0, hw // 2, 0), (0, 0, hw // 2),
               (n - 1, hw // 2, hw - 1), (n // 2, hw - 1, hw // 2)}
        for t in (7, 8, 15, 16, 31, 32, 63, 64):   # neighbours of typical tile boundaries
            if t < hw:
                pix.add((n // 2, t, t))
                pix.add((0, t, hw - 1 - t if hw - 1 - t >= 0 else 0))
        want = int(min(40, max(len(pix), 30e9 // cone_flops(shape))))
        while len(pix) < want:
            pix.add((int(rng.integers(n)), int(rng.integers(hw)), int(rng.integers(hw))))
        pix = sorted(pix)
        cone = orc.cone_outputs(layers, params, x, pix)
    if depth <= 4:
        plans = list(G.all_contiguous_plans(depth))
    else:  # unfused, all fused, blocks of 2 and of 4 (the block-size sweep of Sec. III-B)
        plans = [list(range(depth)), [depth - 1], list(range(1, depth, 2)), list(range(3, depth, 4))]
    ran = 0
    for ends in plans:
        firsts = [0] + [e + 1 for e in ends[:-1]]
        if not all(B.net_group_is_legal(sess.net, a, e, sms) for a, e in zip(firsts, ends)):
            with pytest.raises(B.DlfError):
                B.net_set_plan(sess.net, ends, [sms] * len(ends))
            continue
        ran += 1
        if full:
            G.check_plan(sess, xd, ref, ends, [sms] * len(ends), "sweep %s plan %s" % (shape, ends))
        else:
            sess.set_plan(ends, [sms] * len(ends))
            out = sess.run(xd).cpu().numpy()
            got = np.stack([out[p[0], p[1], p[2], :] for p in pix])
            G.compare(got, cone, "sweep %s plan %s (cone)" % (shape, ends))
    assert ran >= 1
    sess.close()
