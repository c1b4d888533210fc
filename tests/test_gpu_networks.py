"""GPU parity at the full workload sizes: VGG-16 b8, ResNet-50 b1/b32, MobileNetV2 b1/b64.

The device runs the whole batch in the launch configuration the benchmark times; the CPU
checker, whose images are independent (pinned bit-exactly on the CPU), runs a sample of the
batch (first and last image) through every layer, and every group boundary of those images is
compared element by element."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import executor as orc
from paper_2011_05630_b200 import binding as B, networks as nw, plans, synth
from paper_2011_05630_b200.runtime import Session
from tests import gpu_util as G

NETS = [("vgg16", nw.vgg16, 8), ("resnet50", nw.resnet50, 1), ("resnet50", nw.resnet50, 32),
        ("mobilenet_v2", nw.mobilenet_v2, 1), ("mobilenet_v2", nw.mobilenet_v2, 64)]


@pytest.mark.parametrize("name,builder,batch", NETS, ids=["%s_b%d" % (n, b) for n, _, b in NETS])
def test_network_every_boundary(name, builder, batch):
    layers = builder()
    params = synth.layer_params(name, layers)
    x = synth.network_input(name, batch, 224, 224, 3)
    sample = sorted({0, batch - 1})
    ref = orc.run_network(layers, params, np.ascontiguousarray(x[sample]))
    for r in ref:
        assert np.isfinite(r.astype(np.float32)).all()
    sess = Session(layers, params, batch, 224, 224, 3)
    xd = sess.upload(x)
    sms = B.device_sm_count()
    todo = [("unfused", None, None)]
    ends, smc = plans.tuned_plan(sess.net, len(layers))
    todo.append(("tuned", ends, smc))
    if name == "mobilenet_v2":   # every inverted-residual block as one group, the wide ones the tuner leaves apart too
        ends, i = [], 0
        while i < len(layers):
            span = 1
            if layers[i]["op"] == "dwconv" or (i + 1 < len(layers) and layers[i + 1]["op"] == "dwconv"):
                span = 2 if layers[i]["op"] == "dwconv" else 3
                if B.net_group_is_legal(sess.net, i, i + span - 1, sms) != 1:
                    span = 1
            ends.append(i + span - 1)
            i += span
        assert sum(1 for a, e in zip([0] + [e + 1 for e in ends[:-1]], ends) if e > a) == 17
        todo.append(("block-fused", ends, [sms] * len(ends)))
    for what, e, s in todo:
        ends_now, _ = sess.set_plan(e, s)
        out = sess.run(xd).cpu().numpy()
        for le in ends_now:
            got = out if le == len(layers) - 1 else sess.boundary(le)
            G.compare(got[sample], ref[le], "%s b%d %s layer %d" % (name, batch, what, le))
        assert G.rel_l2(out[sample], ref[-1]) <= G.TOL
    sess.close()
