"""GPU parity at the full workload sizes: VGG-16 b8, ResNet-50 b1/b32, MobileNetV2 b1/b64, and the paper's other Table 2
networks (VGG-19, ResNet-18, AlexNet).

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
        ("mobilenet_v2", nw.mobilenet_v2, 1), ("mobilenet_v2", nw.mobilenet_v2, 64),
        ("vgg19", nw.vgg19, 8), ("resnet18", nw.resnet18, 32), ("alexnet", nw.alexnet, 32)]


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
    if name == "resnet50":   # the four projection branches run as one product with the expansion layers they are added to
        assert len(ends) == len(layers) - 4
        for e in ends:
            if layers[e]["res_src"] == e - 1:
                assert e - 1 not in ends
    if name == "mobilenet_v2":   # inverted-residual blocks run fused where the estimate says the fused kernel pays
        assert len(ends) < len(layers) - 12
    if name in ("resnet50", "resnet18"):   # one group per residual block (its layers handed over through L2), stem and tail apart
        ends = [0, 1]
        for i in range(2, len(layers) - 2):
            if layers[i]["res_src"] != -2:
                ends.append(i)
        ends += [len(layers) - 2, len(layers) - 1]
        assert len(ends) == (16 if name == "resnet50" else 8) + 4
        todo.append(("block-fused", ends, [sms] * len(ends)))
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
