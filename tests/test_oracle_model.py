"""Pins for the restated formulas (Eq. 1-5) and structural checks of Algorithm 1."""
import math
import os

import pytest

from oracle import model
from paper_2011_05630_b200 import networks as nw

GI = 2 ** 30


def paper(golden_dir):
    vals = {}
    for line in open(os.path.join(golden_dir, "paper_values.txt")):
        line = line.split("#")[0].strip()
        if line:
            k, v = [s.strip() for s in line.split("=")]
            vals[k] = v
    return vals


def conv(cin, cout, k, stride=1, pad=None, groups=1):
    return dict(op="conv", act="relu", cin=cin, cout=cout, kh=k, kw=k, stride=stride,
                pad=k // 2 if pad is None else pad, groups=groups, src=None, res_src=-2, pool=0)


def chain(layers):
    for i, l in enumerate(layers):
        if l["src"] is None:
            l["src"] = i - 1
    return layers


def vgg19():
    L, cin = [], 3
    for width, reps in ((64, 2), (128, 2), (256, 4), (512, 4), (512, 4)):
        for r in range(reps):
            L.append(dict(conv(cin, width, 3), pool=2 if r == reps - 1 else 0))
            cin = width
    return chain(L)


def resnet18():
    L = [conv(3, 64, 7, 2, 3), dict(conv(64, 64, 3, 2, 1), op="maxpool")]
    cin, block_in = 64, 1
    for stage, width in enumerate((64, 128, 256, 512)):
        for b in range(2):
            s = 2 if (b == 0 and stage > 0) else 1
            L.append(dict(conv(cin, width, 3, s), src=block_in))
            if s == 2:
                L.append(dict(conv(cin, width, 1, s, 0), src=block_in))
            L.append(dict(conv(width, width, 3), src=len(L) - (2 if s == 2 else 1)))
            block_in, cin = len(L) - 1, width
    return chain(L)


def alexnet_single_tower():
    L = [conv(3, 64, 11, 4, 2), dict(conv(64, 64, 3, 2, 0), op="maxpool"),
         conv(64, 192, 5, 1, 2), dict(conv(192, 192, 3, 2, 0), op="maxpool"),
         conv(192, 384, 3), conv(384, 256, 3), conv(256, 256, 3)]
    return chain(L)


@pytest.mark.parametrize("name,layers,key", [
    ("resnet18", resnet18(), "resnet18"), ("resnet50", nw.resnet50(), "resnet50"),
    ("vgg19", vgg19(), "vgg19"), ("alexnet", alexnet_single_tower(), "alexnet"),
    ("mobilenet", nw.mobilenet_v2(), "mobilenet")])
def test_table2_operation_counts(golden_dir, name, layers, key):
    p = paper(golden_dir)
    ops = model.layer_ops(layers, 1, 224, 224, 3, literal=True)
    convs = [o for o, l in zip(ops, layers) if l["op"] in ("conv", "dwconv")]
    assert len(convs) == int(p["table2.%s.convs" % key])
    total = sum(convs) / GI
    assert abs(total - float(p["table2.%s.total" % key])) <= 0.006, total
    assert abs(total / len(convs) - float(p["table2.%s.avg" % key])) <= 0.0051, total / len(convs)


def test_workload_recipes_are_the_table2_networks():
    """The library's own builders (run on the GPU and timed) have the convolution layers of the builders above."""
    key = lambda l: (l["op"], l["cin"], l["cout"], l["kh"], l["stride"], l["pad"])
    for mine, theirs in ((vgg19(), nw.vgg19()), (resnet18(), nw.resnet18()), (alexnet_single_tower(), nw.alexnet())):
        convs = lambda layers: [key(l) for l in layers if l["op"] == "conv"]
        assert convs(mine) == convs(theirs)
    assert [l["src"] for l in resnet18()] == [l["src"] for l in nw.resnet18()[:len(resnet18())]]   # the skip wiring too
    for layers, hw in ((nw.vgg19(), 224), (nw.resnet18(), 224), (nw.alexnet(), 224)):
        shapes = model.infer_shapes(layers, 1, hw, hw, 3)
        assert shapes[-1] == (1, 1, 1, 1000)


def test_equal_op_count_triple_of_sec4a():
    a = model.eq1_conv_ops(224, 224, 3, 3, 32, 32)
    assert a == model.eq1_conv_ops(112, 112, 3, 3, 64, 64) == model.eq1_conv_ops(56, 56, 3, 3, 128, 128)


def test_sec4b_quoted_counts_are_macs(golden_dir):
    p = paper(golden_dir)
    assert round(model.eq1_conv_ops(28, 28, 3, 3, 512, 512) / 2 / GI, 2) == float(p["sec4b.conv1"])
    assert round(model.eq1_conv_ops(14, 14, 3, 3, 512, 512) / 2 / GI, 2) == float(p["sec4b.conv2"])


def test_work_count_scales_with_batch_and_groups():
    L = nw.mobilenet_v2()
    lit = model.layer_ops(L, 1, 224, 224, 3, literal=True)
    work = model.layer_ops(L, 4, 224, 224, 3, literal=False)
    for l, a, b in zip(L, lit, work):
        if l["op"] in ("conv", "dwconv"):
            assert b == a * 4 // l["groups"]
    assert abs(sum(model.layer_ops(L, 1, 224, 224, 3)[:-1]) / 1e9 - 0.60) < 0.01  # true grouped count
    fc = model.layer_ops(nw.vgg16(), 8, 224, 224, 3)[-3]
    assert fc == 2 * 8 * 25088 * 4096


def test_eq3_intensity():
    assert model.eq3_intensity(100, [10, 30, 10]) == 2.0


def test_eq4_matches_printed_value_and_closed_form(golden_dir):
    v = model.eq4_space(50)
    assert "%.2e" % v == "8.17e+75" and float(paper(golden_dir)["eq4.n50"]) == 8.17e75
    for n in (2, 3, 7, 50):
        assert model.eq4_space(n) == 32 * (33 ** (n - 1) - 1)


@pytest.mark.parametrize("n,q", [(1, 3), (2, 2), (3, 3), (4, 2), (5, 2)])
def test_plan_enumeration_count(n, q):
    plans = list(model.enumerate_plans(n, list(range(1, q + 1))))
    assert len(plans) == q * (q + 1) ** (n - 1)
    assert len(plans) - q == (model.eq4_space(n, q) if n > 1 else 0)
    assert len({(tuple(e), tuple(m)) for e, m in plans}) == len(plans)
    for ends, mps in plans:
        assert ends[-1] == n - 1 and ends == sorted(set(ends)) and len(mps) == len(ends)


P = dict(alpha=0.316, beta=0.659, kappa=1.0, kappa0=0.0, s_max=32, op_critical=10 ** 1.25 * 1e9)


def test_eq5_score_weights(golden_dir):
    p = paper(golden_dir)
    assert P["alpha"] == float(p["eq5.alpha"]) and P["beta"] == float(p["eq5.beta"])
    assert model.eq5_score(64, 2 ** 30, 0.316, 0.659) == pytest.approx(0.316 * 6 + 0.659 * 30)
    # more operations or more channels never lower the core count
    assert model.layer_mp(64, 2 ** 31, P) >= model.layer_mp(64, 2 ** 30, P)
    assert model.layer_mp(128, 2 ** 30, P) >= model.layer_mp(64, 2 ** 30, P)
    assert 1 <= model.layer_mp(1, 1, P) <= model.layer_mp(4096, 2 ** 50, P) <= 32


def _features(layers, n=1, hw=224):
    ops = model.layer_ops(layers, n, hw, hw, layers[0]["cin"])
    kinds = [l["op"] in ("conv", "dwconv", "fc") for l in layers]
    ch = [l["cout"] for l in layers]
    return kinds, ch, ops


@pytest.mark.parametrize("layers", [nw.vgg16(), nw.resnet50(), nw.mobilenet_v2(), nw.conv_chain(8, 64, 3)])
def test_algorithm1_structure(layers):
    kinds, ch, ops = _features(layers)
    n = len(layers)
    last = None
    for crit in (1.0, 1e6, 1e8, 1e9, 1e10, 1e12, 1e30):
        part, mps = model.algorithm1(kinds, ch, ops, dict(P, op_critical=crit))
        assert part[-1] == n - 1 and part == sorted(set(part)) and len(mps) == len(part)
        assert all(1 <= m <= 32 and (m & (m - 1)) == 0 for m in mps)
        if last is not None:
            assert len(part) <= last
        last = len(part)
    part, _ = model.algorithm1(kinds, ch, ops, dict(P, op_critical=1e-9))
    # threshold -> 0: every parametrised layer closes its own block; layers without weights
    # that follow join the next block (or the tail)
    param_idx = [i for i, k in enumerate(kinds) if k]
    assert part[:len(param_idx) - 1] == param_idx[:-1] or part == sorted(set(param_idx[:-1] + [n - 1]))
    part, mps = model.algorithm1(kinds, ch, ops, dict(P, op_critical=1e300))
    assert part == [n - 1] and len(mps) == 1


def test_algorithm1_identical_layers_give_equal_blocks():
    layers = nw.conv_chain(8, 64, 3)
    kinds = [True] * 8
    ops = [model.eq1_conv_ops(56, 56, 3, 3, 64, 64)] * 8
    mp1 = model.layer_mp(64, ops[0], P)
    part, mps = model.algorithm1(kinds, [64] * 8, ops, dict(P, op_critical=2 * ops[0] / mp1))
    assert part == [1, 3, 5, 7]
    assert mps == [2 ** int(math.floor(math.log2(mp1)))] * 4


def test_algorithm1_forced_boundaries_and_block_mp():
    kinds = [True, False, True, True, False, True]
    ch = [64] * 6
    ops = [2 ** 20, 0, 2 ** 20, 2 ** 30, 0, 2 ** 20]
    part, mps = model.algorithm1(kinds, ch, ops, dict(P, op_critical=1e300),
                                 must_close_after=lambda start, i: i in (1, 4))
    assert part == [1, 4, 5]
    mp_a, mp_b = model.layer_mp(64, 2 ** 20, P), model.layer_mp(64, 2 ** 30, P)
    assert mps[0] == 2 ** int(math.log2(mp_a))
    assert mps[1] == 2 ** int(math.floor(math.log2((mp_a + mp_b) / 2)))
    # a leading run of weight-less layers that is forced closed becomes its own block
    part, mps = model.algorithm1([False, True], [1, 64], [0, 2 ** 20], dict(P, op_critical=1e300),
                                 must_close_after=lambda start, i: i == 0)
    assert part == [0, 1] and mps[0] == 32


def test_exhaustive_search_on_a_hand_worked_table():
    # three layers, core counts {1, 2}; times worked out by hand:
    #   [0][1][2] -> 3 + 2.5 + 3.5 = 9;  [0,1][2] -> 4 + 3.5 = 7.5;  [0][1,2] -> 3 + 5.5 = 8.5
    table = {(0, 0, 1): 5, (0, 0, 2): 3, (1, 1, 1): 4, (1, 1, 2): 2.5, (2, 2, 1): 6, (2, 2, 2): 3.5,
             (0, 1, 1): 6, (0, 1, 2): 4, (1, 2, 1): 7, (1, 2, 2): 5.5}
    best = model.best_plan_exhaustive(3, [1, 2], lambda a, e, m: table.get((a, e, m)))
    assert best == (7.5, [1, 2], [2, 2])
    best = model.best_plan_exhaustive(3, [1, 2], lambda a, e, m: table.get((a, e, m)), max_len=1)
    assert best == (9.0, [0, 1, 2], [2, 2, 2])


# ---- hand-worked pins of the readings added to Eq. 5 and Algorithm 1 -----------------------------------
# alpha = beta = kappa = 1, kappa0 = 0 makes the per-layer count log2(C) + log2(ops): integers for powers of two.
UNIT = dict(alpha=1.0, beta=1.0, kappa=1.0, kappa0=0.0, s_max=32, op_critical=4.0)


def test_eq5_score_against_a_literal_number():
    # 0.316 * log2(64) + 0.659 * log2(2^30) = 1.896 + 19.77
    assert model.eq5_score(64, 2 ** 30, 0.316, 0.659) == pytest.approx(21.666, abs=1e-9)
    assert model.eq5_score(2, 4, 3.0, 0.5) == pytest.approx(4.0)   # 3 * 1 + 0.5 * 2


def test_layer_mp_rounding_and_clamps_by_hand():
    assert model.layer_mp(4, 8, UNIT) == 5                          # 2 + 3
    half = dict(UNIT, kappa=0.5)
    assert model.layer_mp(4, 8, half) == 3                          # 2.5 rounds away from zero
    assert model.layer_mp(4, 2, half) == 2                          # 1.5 -> 2
    assert model.layer_mp(2, 4, dict(UNIT, kappa=0.5, kappa0=-1.0)) == 1    # 0.5 -> 1
    assert model.layer_mp(1, 1, UNIT) == 1                          # score 0: lower clamp
    assert model.layer_mp(4, 8, dict(UNIT, kappa0=-9.0)) == 1       # negative: lower clamp
    assert model.layer_mp(2 ** 20, 2 ** 20, UNIT) == 32             # 40: upper clamp
    assert model.layer_mp(2 ** 20, 2 ** 20, dict(UNIT, s_max=148)) == 40


def test_algorithm1_deferred_close_by_hand():
    # per-layer counts 8, 4, 4, 6, 4; critical operation count 4 per core.
    kinds, ch, ops = [True] * 5, [4] * 5, [2 ** 6, 2 ** 2, 2 ** 2, 2 ** 4, 2 ** 2]
    # Plain pass: layer 0 alone has 64 / 8 = 8 >= 4 and closes; then 4/4, 8/4, 24/(14/3) = 5.1 closes at 3 with
    # floor(log2(4.67)) -> 4 cores; the tail closes at 4.
    assert model.algorithm1(kinds, ch, ops, UNIT) == ([0, 3, 4], [8, 4, 4])
    # The first block may not close before it holds layers 0..2 (a fusable pattern still growing): it closes at
    # layer 2 with average (8 + 4 + 4) / 3 = 5.33 -> 4 cores; then 16 / 6 < 4 keeps layer 3 open and
    # (16 + 4) / ((6 + 4) / 2) = 4 closes at layer 4 with average 5 -> 4 cores.
    part, mps = model.algorithm1(kinds, ch, ops, UNIT, may_close=lambda start, i: not (start == 0 and i < 2))
    assert (part, mps) == ([2, 4], [4, 4])
    # a forced end overrides the deferral
    part, mps = model.algorithm1(kinds, ch, ops, UNIT, must_close_after=lambda start, i: i == 1,
                                 may_close=lambda start, i: not (start == 0 and i < 2))
    assert part[0] == 1 and mps[0] == 4                              # average (8 + 4) / 2 = 6 -> 4


def test_algorithm1_top_step_on_a_chip_that_is_not_a_power_of_two():
    # alpha = 1, beta = 0: the per-layer count is log2(C), clamped to 148 cores
    p = dict(alpha=1.0, beta=0.0, kappa=1.0, kappa0=0.0, s_max=148, op_critical=1e300)
    full, almost = 2.0 ** 200, 2.0 ** 147
    assert model.layer_mp(full, 1, p) == 148 and model.layer_mp(almost, 1, p) == 147
    part, mps = model.algorithm1([True] * 10, [full] * 10, [1] * 10, p)
    assert (part, mps) == ([9], [148])                               # average 148: the whole chip
    part, mps = model.algorithm1([True] * 10, [full] * 9 + [almost], [1] * 10, p)
    assert (part, mps) == ([9], [128])                               # average 147.9: 2^floor(log2) = 128
