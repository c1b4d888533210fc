"""GPU parity: the CUDA path through the C ABI against the CPU checker, element by element, on
the same seeded inputs, at every group boundary, under several fusion plans and SM counts."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import executor as orc
from paper_2011_05630_b200 import binding as B, networks as nw, synth
from paper_2011_05630_b200.runtime import Session
from tests import gpu_util as G
from tests.test_oracle_layers import _tiny_resnet_like


def _mk(layers, tag, n, h, w, c):
    params = synth.layer_params(tag, layers)
    x = synth.network_input(tag, n, h, w, c)
    ref = orc.run_network(layers, params, x)
    sess = Session(layers, params, n, h, w, c)
    return sess, sess.upload(x), ref


def _conv(cin, cout, k, stride=1, pad=None, act="relu", pool=0, groups=1, op="conv", src=-1, res_src=-2):
    return dict(op=op, act=act, cin=cin, cout=cout, kh=k, kw=k, stride=stride, pad=k // 2 if pad is None else pad,
                groups=groups, src=src, res_src=res_src, pool=pool)


SMS = None


def sms():
    global SMS
    if SMS is None:
        SMS = B.device_sm_count()
    return SMS


# ---- config 1: the two-layer fusion group -------------------------------------------------------------
@pytest.mark.parametrize("s", [1, 4, 0])
def test_two_layer_group_unfused_and_fused(s):
    s = s or sms()
    sess, xd, ref = _mk(nw.two_layer_group(), "cfg1", 1, 32, 32, 16)
    G.check_plan(sess, xd, ref, [0, 1], [s, s], "cfg1 unfused")
    assert sess.kernels() == ["conv_tc", "conv_tc"]     # single layers run through the single-layer kernel
    G.check_plan(sess, xd, ref, [1], [s], "cfg1 fused")
    assert sess.kernels() == ["chain_tc"]
    # plan invariance on the device itself: fused and unfused agree to rounding flips
    fused = sess.boundary(1).copy()
    sess.set_plan([0, 1], [s, s])
    sess.run(xd)
    assert G.rel_l2(fused, sess.boundary(1)) < 2e-3


# ---- single layers: every kernel variant ------------------------------------------------------------------
SINGLE = [
    # (n, h, w, layer)
    (1, 32, 32, _conv(16, 16, 3)),
    (2, 19, 23, _conv(64, 64, 3)),                 # ragged tiles
    (1, 56, 56, _conv(64, 128, 1, act="none")),
    (3, 14, 14, _conv(128, 320, 3, act="relu6")),  # two channel tiles, K = 9 x 2 chunks
    (2, 28, 28, _conv(24, 144, 1, act="relu6")),   # channels not multiples of 16 / 64
    (2, 29, 31, _conv(32, 64, 3, stride=2)),       # strided window
    (2, 28, 28, _conv(256, 512, 1, stride=2, pad=0, act="none")),
    (2, 24, 24, _conv(64, 64, 3, pool=2)),         # fused 2x2 max-pool
    (9, 7, 7, _conv(512, 512, 3)),                 # several images per tile
    (2, 33, 35, _conv(3, 32, 3, stride=2, act="relu6")),   # C = 3 stem (direct kernel)
    (1, 45, 43, _conv(3, 64, 7, stride=2, pad=3)),
    (2, 37, 29, _conv(3, 64, 3)),                          # stride 1: patch rows start on odd halves
    (3, 30, 31, _conv(4, 16, 5, stride=2, pad=2, act="none")),
    (5, 6, 6, _conv(3, 24, 3, stride=2)),                  # several images per tile
    (2, 20, 20, _conv(3, 64, 3, pool=2)),
    (2, 21, 22, _conv(96, 96, 3, stride=1, act="relu6", groups=96, op="dwconv")),
    (2, 21, 22, _conv(144, 144, 3, stride=2, act="relu6", groups=144, op="dwconv")),
    (2, 23, 21, _conv(64, 64, 3, stride=2, pad=1, act="none", op="maxpool")),
]


@pytest.mark.parametrize("case", SINGLE, ids=lambda c: "%dx%dx%d_%s_%d_%d_k%d_s%d" % (c[0], c[1], c[2], c[3]["op"], c[3]["cin"], c[3]["cout"], c[3]["kh"], c[3]["stride"]))
def test_single_layer(case):
    n, h, w, layer = case
    sess, xd, ref = _mk([layer], "single", n, h, w, layer["cin"])
    for s in (sms(), 3):
        G.check_plan(sess, xd, ref, [0], [s], "single S=%d" % s)
    if layer["op"] == "conv" and layer["stride"] == 1 and layer["cin"] % 8 == 0:
        # the same layer through the fused-chain kernel (input tile read once)
        B.net_set_option(sess.net, B.OPT_SINGLE_AS_CHAIN, 1)
        for s in (sms(), 3):
            G.check_plan(sess, xd, ref, [0], [s], "single-as-chain S=%d" % s)
        assert sess.kernels() == ["chain_tc"]


ROW_MODE = [
    # 3x3 stride-1 layers through the row mode of the single-layer kernel (forced), then with it switched off
    (3, 9, 13, _conv(64, 128, 3)),                    # two tiles per image, the second one a single row
    (5, 7, 7, _conv(128, 64, 3, act="none")),        # two whole images per tile, ragged batch
    (1, 5, 126, _conv(64, 128, 3, act="relu6")),     # widest image: pitch 128, one row per tile
    (1, 6, 127, _conv(64, 128, 3)),                   # one pixel wider: no row mode, one window load per tap
    (2, 28, 28, _conv(192, 320, 3)),                  # three chunks, two channel tiles (the second one narrower)
]


@pytest.mark.parametrize("case", ROW_MODE, ids=lambda c: "%dx%dx%d_%d_%d" % (c[0], c[1], c[2], c[3]["cin"], c[3]["cout"]))
def test_single_3x3_layer_row_mode_on_and_off(case):
    n, h, w, layer = case
    sess, xd, ref = _mk([layer], "rowmode", n, h, w, layer["cin"])
    try:
        for mode in (2, 0):
            B.net_set_option(sess.net, B.OPT_CONV_ROW_MODE, mode)
            for s in (sms(), 5):
                G.check_plan(sess, xd, ref, [0], [s], "row mode %d S=%d" % (mode, s))
            assert sess.kernels() == ["conv_tc"]
    finally:
        B.net_set_option(sess.net, B.OPT_CONV_ROW_MODE, 1)


def test_row_mode_with_residual():
    layers = [_conv(64, 128, 1, act="none"), _conv(128, 128, 3, src=0, res_src=0)]
    sess, xd, ref = _mk(layers, "rowres", 3, 14, 14, 64)
    try:
        B.net_set_option(sess.net, B.OPT_CONV_ROW_MODE, 2)
        G.check_plan(sess, xd, ref, [0, 1], [sms(), sms()], "row mode residual")
    finally:
        B.net_set_option(sess.net, B.OPT_CONV_ROW_MODE, 1)


SPLIT_K = [
    # few tiles and a long K: the tile's K range is shared out over several work items (fp32 partial tiles, last one adds)
    (1, 7, 7, _conv(512, 512, 3)),                            # row mode, one pixel tile
    (1, 14, 14, _conv(1024, 256, 1, act="none")),             # image-shaped tiles, two per image
    (1, 14, 14, _conv(256, 264, 3, stride=2, act="relu6")),   # strided taps, a narrow second channel tile
    (2, 7, 7, _conv(2048, 512, 1)),
    (3, 1, 1, _conv(4096, 520, 1)),                           # 1x1 image: the pixel-list tiling
]


@pytest.mark.parametrize("case", SPLIT_K, ids=lambda c: "%dx%dx%d_%d_%d_k%d" % (c[0], c[1], c[2], c[3]["cin"], c[3]["cout"], c[3]["kh"]))
def test_single_layer_split_k(case):
    n, h, w, layer = case
    sess, xd, ref = _mk([layer], "splitk", n, h, w, layer["cin"])
    for s in (sms(), sms(), 40, 7, sms()):   # repeated: the arrival counters must be back at zero after every launch
        G.check_plan(sess, xd, ref, [0], [s], "split-K S=%d" % s)
    assert sess.kernels() == ["conv_tc"]


def test_fc_split_k_at_small_batch():
    fc = lambda cin, cout, act, src: dict(op="fc", act=act, cin=cin, cout=cout, kh=1, kw=1, stride=1, pad=0, groups=1, src=src, res_src=-2, pool=0)
    layers = [fc(4 * 4 * 256, 520, "relu", -1), fc(520, 24, "none", 0)]
    sess, xd, ref = _mk(layers, "fcsplit", 9, 4, 4, 256)   # more than 8 rows: the tensor-core kernel takes the first layer
    for _ in range(3):
        G.check_plan(sess, xd, ref, [0, 1], [sms(), sms()], "fc split-K")
    assert sess.kernels()[0] == "conv_tc"


def test_single_layer_with_residual_through_both_conv_kernels():
    layers = [_conv(64, 64, 1, act="none"), _conv(64, 64, 3, src=0, res_src=-1)]
    sess, xd, ref = _mk(layers, "res", 2, 17, 18, 64)
    G.check_plan(sess, xd, ref, [0, 1], [sms(), sms()], "residual tc")
    B.net_set_option(sess.net, B.OPT_NO_TENSOR_CORE, 1)
    G.check_plan(sess, xd, ref, [0, 1], [sms(), sms()], "residual direct")
    assert sess.kernels() == ["conv_direct", "conv_direct"]


def test_fc_and_avgpool():
    layers = [_conv(32, 64, 3), dict(_conv(64, 64, 1, op="gavgpool", act="none"), src=0),
              dict(op="fc", act="relu", cin=64, cout=40, kh=1, kw=1, stride=1, pad=0, groups=1, src=1, res_src=-2, pool=0),
              dict(op="fc", act="none", cin=40, cout=13, kh=1, kw=1, stride=1, pad=0, groups=1, src=2, res_src=-2, pool=0)]
    sess, xd, ref = _mk(layers, "fc", 11, 9, 9, 32)
    G.check_plan(sess, xd, ref, [0, 1, 2, 3], [sms()] * 4, "fc")


def test_tiny_network_with_every_layer_type():
    layers = _tiny_resnet_like()
    layers = [dict(l) for l in layers]   # widened below to channel counts the vector kernels accept
    scale = {3: 3, 4: 8, 8: 16, 16: 32, 5: 8}
    for l in layers:
        l["cin"], l["cout"] = scale[l["cin"]], scale[l["cout"]]
        if l["op"] == "dwconv":
            l["groups"] = l["cin"]
    layers[-1]["cin"] = 32
    sess, xd, ref = _mk(layers, "tinynet", 2, 37, 35, 3)
    G.check_plan(sess, xd, ref, list(range(len(layers))), [sms()] * len(layers), "tiny net")


# ---- fused chains: every contiguous plan, ragged tiles, 1x1 / 3x3 mixes --------------------------------
CHAINS = [
    # (n, h, w, c, kernel sizes)
    (1, 32, 32, 16, (3, 3)),
    (2, 19, 23, 64, (3, 3, 3)),
    (2, 14, 14, 64, (3, 1, 3)),
    (1, 56, 56, 32, (1, 1, 1, 1)),
    (3, 7, 7, (256, 64, 256), (1, 1)),
    (1, 28, 28, 64, (3, 3, 3, 3)),
    (2, 28, 28, (64, 64, 512), (3, 1)),       # bottleneck tail: more than 256 output channels
    (4, 14, 14, (128, 320, 64), (1, 1)),      # a wide intermediate map (5 planes, two channel chunks)
    (2, 14, 14, (32, 160, 32), (1, 3)),       # 3x3 layer reading a 3-plane intermediate
]


@pytest.mark.parametrize("case", CHAINS, ids=lambda c: "%dx%dx%dx%s_%s" % (c[0], c[1], c[2], c[3], "".join(map(str, c[4]))))
def test_chain_every_contiguous_plan(case):
    n, h, w, c, ks = case
    cs = c if isinstance(c, tuple) else (c,) * (len(ks) + 1)
    layers = [_conv(cs[i], cs[i + 1], k, src=i - 1) for i, k in enumerate(ks)]
    sess, xd, ref = _mk(layers, "chain", n, h, w, cs[0])
    ran_fused = 0
    for ends in G.all_contiguous_plans(len(ks)):
        for s in (sms(), 5):
            firsts = [0] + [e + 1 for e in ends[:-1]]
            if all(B.net_group_is_legal(sess.net, a, e, s) for a, e in zip(firsts, ends)):
                G.check_plan(sess, xd, ref, ends, [s] * len(ends), "chain %s S=%d" % (ends, s))
                ran_fused += len(ends) < len(ks)
            else:   # a group the kernel cannot hold is refused, never re-partitioned
                with pytest.raises(B.DlfError) as e:
                    B.net_set_plan(sess.net, ends, [s] * len(ends))
                assert e.value.status == B.E_PLAN
    assert ran_fused > 0


def test_chain_with_pool_and_residual_and_channel_change():
    layers = [_conv(32, 64, 1), _conv(64, 64, 3, src=0), _conv(64, 32, 1, src=1, res_src=-1, act="relu"),
              _conv(32, 48, 3, src=2, pool=2)]
    sess, xd, ref = _mk(layers, "chain2", 2, 18, 22, 32)
    G.check_plan(sess, xd, ref, [0, 1, 2, 3], [sms()] * 4, "unfused")
    G.check_plan(sess, xd, ref, [2, 3], [sms(), 7], "bottleneck-like + pooled tail")
    assert sess.kernels() == ["chain_tc", "conv_tc"]
    B.net_set_option(sess.net, B.OPT_SINGLE_AS_CHAIN, 1)   # the pooled single layer through the fused-group kernel
    G.check_plan(sess, xd, ref, [2, 3], [sms(), 7], "bottleneck-like + pooled tail, single layer as a group")
    assert sess.kernels() == ["chain_tc", "chain_tc"]
    B.net_set_option(sess.net, B.OPT_SINGLE_AS_CHAIN, 0)
    # a fused group that ends in a pooled layer, odd image size (the last row / column is dropped)
    layers = [_conv(32, 64, 3), _conv(64, 48, 3, src=0, pool=2), _conv(48, 48, 1, src=1)]
    sess, xd, ref = _mk(layers, "chain3", 2, 19, 21, 32)
    for s in (sms(), 7):
        G.check_plan(sess, xd, ref, [1, 2], [s, s], "pooled tail S=%d" % s)
        assert sess.kernels() == ["chain_tc", "conv_tc"]


def test_illegal_plans_are_rejected():
    layers = [_conv(32, 32, 3), _conv(32, 32, 3, stride=2, pad=1, act="none", op="maxpool", src=0), _conv(32, 32, 3, src=1)]
    sess, xd, ref = _mk(layers, "illegal", 1, 16, 16, 32)
    # a pool inside a group; ends not increasing; the last layer not covered; SM counts out of range
    for ends, sm in (([2], [4]), ([0, 2, 1], [1, 1, 1]), ([0, 1], [1, 1]), ([0, 1, 2], [0, 1, 1]), ([0, 1, 2], [1, 1, 10 ** 6]), ([1, 2], [4, 4])):
        with pytest.raises(B.DlfError) as e:
            B.net_set_plan(sess.net, ends, sm)
        assert e.value.status == B.E_PLAN
    G.check_plan(sess, xd, ref, [0, 1, 2], [2, 2, 2], "legal")
    # a stride-2 layer inside a group is no chain for the shared-memory kernel, but runs handed over through L2
    layers = [_conv(32, 32, 3), _conv(32, 32, 3, stride=2, src=0), _conv(32, 32, 3, src=1)]
    sess, xd, ref = _mk(layers, "strided-group", 1, 16, 16, 32)
    G.check_plan(sess, xd, ref, [2], [4], "stride 2 inside a group")
    assert sess.kernels() == ["conv_seq"]


# ---- fused inverted-residual blocks --------------------------------------------------------------------
def _mbconv(cin, t, cout, stride, first):
    """Layers of one inverted-residual block whose input is layer `first - 1` (or the network input)."""
    hid = cin * t
    L = []
    if t != 1:
        L.append(_conv(cin, hid, 1, act="relu6", src=first - 1))
    L.append(_conv(hid, hid, 3, stride=stride, act="relu6", groups=hid, op="dwconv", src=first + len(L) - 1))
    L.append(_conv(hid, cout, 1, act="none", src=first + len(L) - 1,
                   res_src=(first - 1) if (stride == 1 and cin == cout) else -2))
    return L


MBCONV = [
    # (n, h, w, cin, t, cout, stride)
    (2, 16, 16, 16, 6, 24, 2),      # hidden 96 = 64 + 32
    (2, 19, 21, 24, 6, 24, 1),      # hidden 144, residual, ragged tiles
    (3, 14, 14, 64, 6, 64, 1),      # six hidden chunks, residual
    (2, 15, 13, 32, 1, 16, 1),      # no expansion layer
    (2, 7, 7, 160, 6, 320, 1),      # three input planes, projection issued as two halves
    (1, 28, 28, 32, 6, 64, 2),
]


@pytest.mark.parametrize("case", MBCONV, ids=lambda c: "%dx%dx%d_c%d_t%d_o%d_s%d" % c)
def test_fused_inverted_residual_block(case):
    n, h, w, cin, t, cout, stride = case
    layers = _mbconv(cin, t, cout, stride, 0)
    for l in layers:
        l["src"] = max(l["src"], -1)
    sess, xd, ref = _mk(layers, "mbconv", n, h, w, cin)
    last = len(layers) - 1
    G.check_plan(sess, xd, ref, list(range(last + 1)), [sms()] * (last + 1), "block unfused")
    for s in (sms(), 5):
        G.check_plan(sess, xd, ref, [last], [s], "block fused S=%d" % s)
        assert sess.kernels() == ["mbconv_tc"]


def test_two_fused_blocks_in_a_row_and_partial_groups_are_refused():
    layers = [_conv(8, 24, 1, src=-1)] + _mbconv(24, 6, 24, 1, 1) + _mbconv(24, 6, 32, 2, 4)
    sess, xd, ref = _mk(layers, "mbconv2", 2, 18, 22, 8)
    G.check_plan(sess, xd, ref, [0, 3, 6], [sms()] * 3, "two fused blocks")
    assert sess.kernels() == ["conv_tc", "mbconv_tc", "mbconv_tc"]
    # depthwise + projection alone is the pattern without an expansion layer (here with a residual)
    G.check_plan(sess, xd, ref, [0, 1, 3, 6], [sms()] * 4, "expansion alone, then depthwise + projection")
    assert sess.kernels() == ["conv_tc", "conv_tc", "mbconv_tc", "mbconv_tc"]
    for ends in ([0, 2, 3, 6], [3, 6]):   # expansion + depthwise alone, or a 1x1 glued in front
        with pytest.raises(B.DlfError) as e:
            B.net_set_plan(sess.net, ends, [sms()] * len(ends))
        assert e.value.status == B.E_PLAN


# ---- groups handed over through L2: one persistent kernel, a device-wide barrier between the layers -------------------
def _bottleneck_with_projection():
    """A down-sampling bottleneck (stride on the 3x3, 1x1/2 projection of the block input added before the ReLU),
    a second block whose skip is the first block's output, then a pooled 3x3 layer."""
    return [_conv(32, 16, 1, src=-1), _conv(16, 16, 3, stride=2, src=0), _conv(32, 64, 1, stride=2, pad=0, act="none", src=-1),
            _conv(16, 64, 1, src=1, res_src=2), _conv(64, 16, 1, src=3), _conv(16, 16, 3, src=4),
            _conv(16, 64, 1, src=5, res_src=3), _conv(64, 72, 3, src=6, pool=2)]


def test_l2_groups_every_contiguous_plan():
    layers = _bottleneck_with_projection()
    n = len(layers)
    sess, xd, ref = _mk(layers, "l2group", 3, 18, 22, 32)
    B.net_set_option(sess.net, B.OPT_GROUP_KERNEL, 2)
    G.check_plan(sess, xd, ref, list(range(n)), [sms()] * n, "unfused")
    ran = 0
    for mask in range(1 << (n - 1)):
        if mask % 5 not in (0, 3) and mask != (1 << (n - 1)) - 1:   # a sample of the 128 plans, plus all-in-one
            continue
        ends = [i for i in range(n - 1) if mask >> i & 1] + [n - 1]
        for s in (sms(), 5):
            G.check_plan(sess, xd, ref, ends, [s] * len(ends), "L2 groups %s S=%d" % (ends, s))
            ran += 1
    assert ran > 20
    sess.set_plan([n - 1], [sms()])
    assert sess.kernels() == ["conv_seq"]
    for _ in range(3):   # the barrier counters are back at zero after every launch
        G.check_plan(sess, xd, ref, [2, n - 1], [7, sms()], "L2 groups, repeated")


def test_group_kernel_option_chooses_the_hand_over():
    layers = [_conv(128, 128, 1, src=-1), _conv(128, 128, 3, src=0), _conv(128, 128, 1, src=1, res_src=-1)]
    sess, xd, ref = _mk(layers, "handover", 2, 14, 14, 128)
    for opt, kernel in ((0, "conv_seq"), (1, "chain_tc"), (2, "conv_seq")):
        B.net_set_option(sess.net, B.OPT_GROUP_KERNEL, opt)
        G.check_plan(sess, xd, ref, [2], [sms()], "option %d" % opt)
        assert sess.kernels() == [kernel]


# ---- projection branch + expansion layer as one product (K runs over both inputs) ------------------------------------
@pytest.mark.parametrize("case", [(64, 64, 256, 1, 2, 19, 23), (128, 64, 128, 2, 3, 18, 22), (192, 128, 320, 2, 1, 7, 7),
                                  (64, 128, 72, 1, 5, 9, 5)])
def test_projection_and_expansion_as_one_group(case):
    cin, mid, cout, stride, n, h, w = case
    layers = [_conv(cin, mid, 1, src=-1), _conv(mid, mid, 3, stride=stride, src=0),
              _conv(cin, cout, 1, stride=stride, pad=0, act="none", src=-1), _conv(mid, cout, 1, src=1, res_src=2),
              _conv(cout, 64, 1, src=3)]
    sess, xd, ref = _mk(layers, "projadd%d" % cin, n, h, w, cin)
    G.check_plan(sess, xd, ref, [0, 1, 2, 3, 4], [sms()] * 5, "unfused")
    for s in (sms(), 7, 1):
        G.check_plan(sess, xd, ref, [0, 1, 3, 4], [sms(), sms(), s, sms()], "projection + expansion S=%d" % s)
        assert sess.kernels()[2] == "conv_tc"
    assert B.net_group_is_legal(sess.net, 2, 3, sms())
    assert B.net_tuner_may_fuse(sess.net, 2, 3, False, sms())
