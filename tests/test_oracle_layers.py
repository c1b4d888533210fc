"""Pins for the CPU checker's layers: brute force on tiny inputs, closed forms, special
cases that reduce to library routines (numpy matmul, torch CPU conv2d / pooling), and
invariants.  Chosen so that a dropped term, a wrong sign or index, or a transposed operand
fails at least one of them (asymmetric shapes everywhere: H != W, kh != kw, cin != cout)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import executor as orc
from tests import refs


def rnd(seed, shape, scale=1.0):
    return (np.random.default_rng(seed).uniform(-1, 1, shape) * scale).astype(np.float16)


CASES = [
    # n, h, w, cin, cout, kh, kw, stride, pad, groups
    (1, 5, 6, 3, 4, 3, 3, 1, 1, 1),
    (2, 6, 5, 4, 2, 3, 2, 1, 0, 1),
    (1, 7, 6, 4, 6, 3, 3, 2, 1, 2),
    (2, 6, 6, 4, 4, 3, 3, 2, 1, 4),   # depthwise
    (1, 6, 4, 2, 3, 1, 1, 1, 0, 1),
    (1, 6, 7, 2, 3, 1, 1, 2, 0, 1),
    (1, 9, 8, 3, 2, 7, 7, 2, 3, 1),
    (1, 4, 4, 2, 2, 3, 3, 1, 2, 1),   # pad larger than needed
    (1, 5, 5, 6, 4, 2, 3, 3, 1, 2),
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("act", ["none", "relu", "relu6"])
def test_conv_against_brute_force(case, act):
    n, h, w, cin, cout, kh, kw, stride, pad, groups = case
    x = rnd(1, (n, h, w, cin), 2.0)
    wt = rnd(2, (cout, kh, kw, cin // groups))
    b = np.random.default_rng(3).normal(0, 1.0, cout).astype(np.float32)
    got = orc.conv2d(x, wt, b, stride, pad, groups, None, act)
    ref = refs.conv_brute(x, wt, b, stride, pad, groups, None, act)
    assert got.shape == ref.shape
    refs.assert_matches_exact_math(got, ref)


def test_conv_residual_and_pool_against_brute_force():
    x = rnd(4, (2, 6, 8, 3), 2.0)
    wt = rnd(5, (5, 3, 3, 3))
    b = np.random.default_rng(6).normal(0, 0.5, 5).astype(np.float32)
    res = rnd(7, (2, 6, 8, 5), 3.0)
    got = orc.conv2d(x, wt, b, 1, 1, 1, res, "relu", pool=2)
    ref = refs.pool2(refs.conv_brute(x, wt, b, 1, 1, 1, res, "relu"))
    assert got.shape == (2, 3, 4, 5)
    refs.assert_matches_exact_math(got, ref)
    # the residual really is added before the activation, with a plus sign
    plain = orc.conv2d(x, wt, b, 1, 1, 1, None, "none").astype(np.float64)
    with_res = orc.conv2d(x, wt, b, 1, 1, 1, res, "none").astype(np.float64)
    assert np.abs(with_res - (plain + res.astype(np.float64))).max() < 8e-3


def test_pool_of_rounded_equals_rounded_of_pool():
    x = rnd(8, (1, 6, 6, 4), 2.0)
    wt = rnd(9, (4, 3, 3, 4))
    b = np.zeros(4, np.float32)
    full = orc.conv2d(x, wt, b, 1, 1, 1, None, "relu", pool=0)
    pooled = orc.conv2d(x, wt, b, 1, 1, 1, None, "relu", pool=2)
    assert np.array_equal(refs.pool2(full), pooled)


def test_one_by_one_conv_is_a_matrix_product():
    x = rnd(10, (2, 5, 7, 24))
    wt = rnd(11, (40, 1, 1, 24))
    b = np.random.default_rng(12).normal(0, 0.1, 40).astype(np.float32)
    got = orc.conv2d(x, wt, b, 1, 0, 1)
    ref = x.reshape(-1, 24).astype(np.float64) @ wt.reshape(40, 24).astype(np.float64).T + b
    refs.assert_matches_exact_math(got.reshape(-1, 40), ref)


def test_fc_is_a_matrix_product_in_nhwc_flatten_order():
    x = rnd(13, (3, 2, 3, 5))
    wt = rnd(14, (7, 30))
    b = np.random.default_rng(15).normal(0, 0.1, 7).astype(np.float32)
    got = orc.fc(x, wt, b, "relu")
    ref = np.maximum(x.reshape(3, 30).astype(np.float64) @ wt.astype(np.float64).T + b, 0)
    assert got.shape == (3, 1, 1, 7)
    refs.assert_matches_exact_math(got.reshape(3, 7), ref)


def test_delta_kernel_reproduces_input_bit_exactly():
    x = rnd(16, (2, 6, 5, 8), 4.0)
    wt = np.zeros((8, 3, 3, 8), np.float16)
    for c in range(8):
        wt[c, 1, 1, c] = 1.0
    got = orc.conv2d(x, wt, np.zeros(8, np.float32), 1, 1, 1)
    assert np.array_equal(got.view(np.uint16), x.view(np.uint16))
    # off-centre delta = shift by one pixel with zero fill (pins the tap -> offset sign)
    wt = np.zeros((8, 3, 3, 8), np.float16)
    for c in range(8):
        wt[c, 0, 2, c] = 1.0          # tap (r=0, s=2): reads x[h-1, w+1]
    got = orc.conv2d(x, wt, np.zeros(8, np.float32), 1, 1, 1)
    want = np.zeros_like(x)
    want[:, 1:, :-1, :] = x[:, :-1, 1:, :]
    assert np.array_equal(got, want)


def test_zero_weights_give_activated_bias():
    x = rnd(17, (1, 4, 4, 3))
    b = np.array([-1.0, 0.5, 7.0, 3.0003], np.float32)
    got = orc.conv2d(x, np.zeros((4, 3, 3, 3), np.float16), b, 1, 1, 1, None, "relu6")
    want = np.array([0.0, 0.5, 6.0, 3.0003], np.float32).astype(np.float16)
    assert np.array_equal(got, np.broadcast_to(want, got.shape))


def test_constant_kernel_on_constant_image_counts_in_range_taps():
    x = np.full((1, 5, 6, 2), 0.5, np.float16)
    wt = np.full((1, 3, 3, 2), 0.25, np.float16)
    got = orc.conv2d(x, wt, np.zeros(1, np.float32), 1, 1, 1).astype(np.float64)[0, :, :, 0]
    taps = np.full((5, 6), 9.0)
    taps[0, :] = taps[-1, :] = 6.0
    taps[:, 0] = taps[:, -1] = 6.0
    taps[0, 0] = taps[0, -1] = taps[-1, 0] = taps[-1, -1] = 4.0
    assert np.array_equal(got, taps * 2 * 0.5 * 0.25)


def test_depthwise_equals_per_channel_filter():
    x = rnd(18, (1, 6, 7, 5))
    wt = rnd(19, (5, 3, 3, 1))
    got = orc.conv2d(x, wt, np.zeros(5, np.float32), 2, 1, 5)
    for c in range(5):
        one = orc.conv2d(np.ascontiguousarray(x[..., c:c + 1]), np.ascontiguousarray(wt[c:c + 1]),
                         np.zeros(1, np.float32), 2, 1, 1)
        assert np.array_equal(got[..., c:c + 1], one)


@pytest.mark.parametrize("stride,pad,groups,k", [(1, 1, 1, 3), (2, 1, 1, 3), (2, 3, 1, 7), (1, 0, 1, 1),
                                                 (2, 1, 8, 3), (1, 1, 8, 3)])
def test_conv_against_torch_cpu(stride, pad, groups, k):
    x = rnd(20, (2, 13, 11, 8))
    wt = rnd(21, (16, k, k, 8 // groups), 0.3)
    b = np.random.default_rng(22).normal(0, 0.1, 16).astype(np.float32)
    got = orc.conv2d(x, wt, b, stride, pad, groups, None, "relu")
    tx = torch.from_numpy(x.astype(np.float32)).permute(0, 3, 1, 2)
    tw = torch.from_numpy(wt.astype(np.float32)).permute(0, 3, 1, 2)
    ref = F.relu(F.conv2d(tx, tw, torch.from_numpy(b), stride=stride, padding=pad, groups=groups))
    ref = ref.permute(0, 2, 3, 1).numpy()
    assert got.shape == ref.shape
    assert refs.ulp_diff(got, ref.astype(np.float16)).max() <= 1
    assert (got == ref.astype(np.float16)).mean() > 0.97


def test_maxpool_and_avgpool_against_torch_and_numpy():
    x = rnd(23, (2, 9, 8, 6))
    tx = torch.from_numpy(x.astype(np.float32)).permute(0, 3, 1, 2)
    got = orc.maxpool(x, 3, 2, 1)
    ref = F.max_pool2d(tx, 3, 2, 1).permute(0, 2, 3, 1).numpy().astype(np.float16)
    assert np.array_equal(got, ref)
    got2 = orc.maxpool(x, 2, 2, 0)
    assert np.array_equal(got2, refs.pool2(x))
    # negative inputs at the border: padding must not win the max
    neg = -np.abs(x) - np.float16(1.0)
    assert orc.maxpool(neg, 3, 2, 1).max() < 0
    avg = orc.gavgpool(x)
    refs.assert_matches_exact_math(avg.reshape(2, 6), x.astype(np.float64).mean(axis=(1, 2)), 0.9)


def test_batch_independence_bit_exact():
    x = rnd(24, (4, 6, 6, 4))
    wt = rnd(25, (6, 3, 3, 4))
    b = np.random.default_rng(26).normal(0, 0.1, 6).astype(np.float32)
    full = orc.conv2d(x, wt, b, 1, 1, 1, None, "relu")
    for i in range(4):
        assert np.array_equal(full[i:i + 1], orc.conv2d(np.ascontiguousarray(x[i:i + 1]), wt, b, 1, 1, 1, None, "relu"))


def test_translation_equivariance_in_the_interior():
    x = rnd(27, (1, 10, 10, 3))
    wt = rnd(28, (4, 3, 3, 3))
    b = np.zeros(4, np.float32)
    y = orc.conv2d(x, wt, b, 1, 1, 1)
    xs = np.zeros_like(x)
    xs[:, 2:, 1:, :] = x[:, :-2, :-1, :]
    ys = orc.conv2d(xs, wt, b, 1, 1, 1)
    assert np.array_equal(ys[:, 4:-1, 3:-1, :], y[:, 2:-3, 2:-2, :])


def test_thread_count_does_not_change_bits():
    x = rnd(29, (3, 9, 9, 8))
    wt = rnd(30, (8, 3, 3, 8))
    b = np.zeros(8, np.float32)
    a = orc.conv2d(x, wt, b, 1, 1, 1, None, "relu", 0, nthreads=1)
    c = orc.conv2d(x, wt, b, 1, 1, 1, None, "relu", 0, nthreads=4)
    assert np.array_equal(a, c)


def _tiny_resnet_like():
    mk = lambda **k: dict(dict(op="conv", act="relu", kh=1, kw=1, stride=1, pad=0, groups=1,
                               res_src=-2, pool=0), **k)
    return [
        mk(cin=3, cout=8, kh=3, kw=3, stride=2, pad=1, src=-1),
        mk(op="maxpool", act="none", cin=8, cout=8, kh=3, kw=3, stride=2, pad=1, src=0),
        mk(cin=8, cout=4, src=1),
        mk(cin=4, cout=4, kh=3, kw=3, pad=1, stride=2, src=2),
        mk(cin=8, cout=16, act="none", stride=2, src=1),
        mk(cin=4, cout=16, src=3, res_src=4),
        mk(op="dwconv", act="relu6", cin=16, cout=16, kh=3, kw=3, pad=1, groups=16, src=5),
        mk(cin=16, cout=16, act="none", src=6, res_src=5),
        mk(op="gavgpool", act="none", cin=16, cout=16, src=7),
        mk(op="fc", act="none", cin=16, cout=5, src=8),
    ]


def test_network_plumbing_against_torch_composite():
    from paper_2011_05630_b200 import synth
    layers = _tiny_resnet_like()
    params = synth.layer_params("tiny", layers)
    x = synth.network_input("tiny", 2, 17, 15, 3)
    outs = orc.run_network(layers, params, x)
    # the same graph in torch fp32 with a rounding to fp16 after every layer
    t = {-1: torch.from_numpy(x.astype(np.float32)).permute(0, 3, 1, 2)}
    act = {"none": lambda v: v, "relu": F.relu, "relu6": F.relu6}
    for i, l in enumerate(layers):
        s = t[l["src"]]
        if l["op"] in ("conv", "dwconv"):
            w, b = params[i]
            v = F.conv2d(s, torch.from_numpy(w.astype(np.float32)).permute(0, 3, 1, 2),
                         torch.from_numpy(b), stride=l["stride"], padding=l["pad"], groups=l["groups"])
            if l["res_src"] != -2:
                v = v + t[l["res_src"]]
            v = act[l["act"]](v)
        elif l["op"] == "maxpool":
            v = F.max_pool2d(s, l["kh"], l["stride"], l["pad"])
        elif l["op"] == "gavgpool":
            v = s.mean(dim=(2, 3), keepdim=True)
        else:
            w, b = params[i]
            flat = s.permute(0, 2, 3, 1).reshape(s.shape[0], -1)
            v = (flat @ torch.from_numpy(w.astype(np.float32)).T + torch.from_numpy(b))[:, :, None, None]
        t[i] = v.half().float()
        got = outs[i].astype(np.float32)
        ref = t[i].permute(0, 2, 3, 1).numpy()
        assert got.shape == ref.shape, (i, got.shape, ref.shape)
        assert np.abs(got - ref).max() <= 2e-2 * (1 + np.abs(ref).max()), i
        assert np.isfinite(got).all()
        # feed torch the checker's own tensor so rounding flips do not pile up
        t[i] = torch.from_numpy(got).permute(0, 3, 1, 2)
    assert outs[-1].shape == (2, 1, 1, 5)
    lean = orc.run_network(layers, params, x, keep=False)
    assert np.array_equal(lean[-1], outs[-1])


def test_cone_equals_full_run():
    from paper_2011_05630_b200 import networks, synth
    layers = networks.conv_chain(3, 8, 3)
    layers[1] = dict(layers[1], kh=1, kw=1, pad=0)
    params = synth.layer_params("cone", layers)
    x = synth.network_input("cone", 2, 12, 11, 8)
    full = orc.run_network(layers, params, x)[-1]
    pix = [(0, 0, 0), (0, 11, 10), (1, 0, 10), (1, 11, 0), (0, 5, 5), (1, 1, 9), (0, 6, 0)]
    got = orc.cone_outputs(layers, params, x, pix)
    for j, (n, h, w) in enumerate(pix):
        assert np.array_equal(got[j], full[n, h, w, :])


def test_bad_sizes_are_rejected():
    x = rnd(31, (1, 2, 2, 4))
    with pytest.raises(ValueError):
        orc.conv2d(x, rnd(32, (4, 5, 5, 4)), np.zeros(4, np.float32), 1, 0, 1)
