"""Host-side logic of the library, without a GPU: the shared object loads and exports every
symbol the header declares, layer lists are type-checked, operation counts and the auto-tuner
(Eq. 5 + Algorithm 1) agree with the restated formulas in oracle/model.py."""
import os
import re

import pytest

from oracle import model
from paper_2011_05630_b200 import binding as B, networks as nw

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "dlfusion.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(dlf_[a-z0-9_]+)\s*\(", hdr))
    assert len(names) >= 24
    lib = B.lib()
    for n in sorted(names):
        assert hasattr(lib, n), n
    assert B.strerror(B.E_PLAN) == "invalid fusion plan" and B.strerror(0) == "ok"


NETS = [("vgg16", nw.vgg16(), 8), ("resnet50", nw.resnet50(), 32), ("mobilenet_v2", nw.mobilenet_v2(), 64),
        ("two_layer", nw.two_layer_group(), 1)]


@pytest.mark.parametrize("name,layers,batch", NETS, ids=[n for n, _, _ in NETS])
def test_shapes_and_operation_counts_match_the_formulas(name, layers, batch):
    hw, c = (32, 16) if name == "two_layer" else (224, 3)
    net = B.net_create(layers, batch, hw, hw, c)
    shapes = model.infer_shapes(layers, batch, hw, hw, c)
    lit = model.layer_ops(layers, batch, hw, hw, c, literal=True)
    work = model.layer_ops(layers, batch, hw, hw, c, literal=False)
    for i in range(len(layers)):
        ops, fl, sh = B.net_layer_info(net, i)
        assert sh == shapes[i], (i, sh, shapes[i])
        assert ops == lit[i] and fl == work[i], (i, ops, lit[i], fl, work[i])
    assert B.net_workspace_bytes(net) > sum(2 * s[0] * s[1] * s[2] * s[3] for s in shapes)
    B.net_destroy(net)


def _conv(cin, cout, k=3, **kw):
    d = dict(op="conv", act="relu", cin=cin, cout=cout, kh=k, kw=k, stride=1, pad=k // 2, groups=1, src=-1, res_src=-2, pool=0)
    d.update(kw)
    return d


@pytest.mark.parametrize("layers,status", [
    ([_conv(8, 8), _conv(16, 8, src=0)], B.E_SHAPE),            # channel mismatch
    ([_conv(8, 8, src=0)], B.E_SHAPE),                            # reads itself
    ([_conv(8, 8, kh=9, kw=9, pad=0)], B.E_SHAPE),                # kernel larger than the image
    ([_conv(8, 8), _conv(8, 16, src=0, res_src=-1)], B.E_SHAPE),  # residual of another shape
    ([_conv(8, 8, groups=3)], B.E_SHAPE),
    ([_conv(8, 8, stride=0)], B.E_INVALID_ARG),
    ([_conv(8, 8, pool=3)], B.E_INVALID_ARG),
    ([dict(_conv(8, 8), op="fc", cin=7)], B.E_SHAPE),
    ([_conv(8, 12, groups=4)], B.E_UNSUPPORTED),                  # grouped conv without a kernel
    ([dict(_conv(12, 12, groups=12), op="dwconv")], B.E_UNSUPPORTED),
])
def test_bad_layer_lists_are_rejected(layers, status):
    with pytest.raises(B.DlfError) as e:
        B.net_create(layers, 1, 6, 6, layers[0]["cin"])
    assert e.value.status == status


def test_bad_arguments_and_call_order():
    import ctypes as C
    L = B.lib()
    assert L.dlf_net_create(None, 1, 1, 4, 4, 8, C.byref(C.c_void_p())) == B.E_INVALID_ARG
    arr = B.layer_descs([_conv(8, 8)])
    assert L.dlf_net_create(arr, 0, 1, 4, 4, 8, C.byref(C.c_void_p())) == B.E_INVALID_ARG
    assert L.dlf_net_create(arr, 1, 0, 4, 4, 8, C.byref(C.c_void_p())) == B.E_INVALID_ARG
    net = B.net_create([_conv(8, 8)], 1, 4, 4, 8)
    assert L.dlf_net_run(net, 256, 512, None) == B.E_WORKSPACE          # nothing bound yet
    assert L.dlf_net_bind_workspace(net, 256, 16) == B.E_WORKSPACE      # too small
    assert L.dlf_net_bind_workspace(net, 300, 1 << 30) == B.E_WORKSPACE  # misaligned
    assert L.dlf_net_set_weights(net, 0, None, None) == B.E_INVALID_ARG
    assert L.dlf_net_set_weights(net, 5, 256, 256) == B.E_INVALID_ARG
    assert L.dlf_net_set_weights(net, 0, 264, 256) == B.E_INVALID_ARG    # not 16-byte aligned
    assert L.dlf_net_layer_info(net, 3, None, None, None) == B.E_INVALID_ARG
    assert L.dlf_net_set_option(net, 99, 1) == B.E_INVALID_ARG
    assert L.dlf_net_boundary_tensor(net, 0, C.byref(C.c_void_p()), None) == B.E_WORKSPACE
    assert L.dlf_conv_chain_run_static(arr, 0, 1, 4, 4, 256, None, None, 256, 1, None) == B.E_INVALID_ARG
    B.net_destroy(net)


@pytest.mark.parametrize("layer,status", [
    (dict(cout=0), B.E_SHAPE), (dict(cin=0), B.E_SHAPE), (dict(cout=-8), B.E_SHAPE), (dict(act=7), B.E_INVALID_ARG),
    (dict(act=-1), B.E_INVALID_ARG), (dict(cout=12), B.E_UNSUPPORTED), (dict(pool=2), B.E_UNSUPPORTED),
    (dict(groups=2), B.E_UNSUPPORTED), (dict(src=0), B.E_SHAPE)])
def test_allocation_free_entry_rejects_bad_layers_before_any_launch(layer, status):
    # every refusal below is decided on the host from the descriptors alone: no device call is made (the pointers
    # are dummies), so the cases run without a GPU
    import ctypes as C
    d = _conv(8, 8)
    d["act"] = B.ACTS[d["act"]]
    d.update(layer)
    arr = (B.LayerDesc * 1)(B.LayerDesc(B.OPS["conv"], d["act"], d["cin"], d["cout"], d["kh"], d["kw"], d["stride"], d["pad"],
                                        d["groups"], d["src"], d["res_src"], d["pool"]))
    ptrs = (C.c_void_p * 1)(256)
    assert B.lib().dlf_conv_chain_run_static(arr, 1, 1, 6, 6, 256, ptrs, ptrs, 256, 1, None) == status


# ---- the auto-tuner against the restated Algorithm 1 ----------------------------------------------------
# Which spans one kernel can run, and which of them are worth proposing, is the library's own rule (four fused kernels
# and their cost estimates - nothing the paper defines): the test takes it from dlf_net_tuner_may_fuse as an INPUT and
# checks the pass itself - running sums, threshold, deferred close, forced ends, block core count - against oracle/model.py.
P = dict(alpha=0.316, beta=0.659, kappa=12.0, kappa0=-60.0, s_max=148)


@pytest.mark.parametrize("name,layers,batch", NETS + [("chain8", nw.conv_chain(8, 64, 3), 16),
                                                     ("chain_1x1", nw.conv_chain(6, 128, 1), 8)],
                         ids=[n for n, _, _ in NETS] + ["chain8", "chain_1x1"])
@pytest.mark.parametrize("crit", [1.0, 1e7, 2e8, 3e9, 1e11, 1e30])
def test_autotune_equals_restated_algorithm1(name, layers, batch, crit):
    hw, c = {"two_layer": (32, 16), "chain8": (56, 64), "chain_1x1": (28, 128)}.get(name, (224, 3))
    net = B.net_create(layers, batch, hw, hw, c)
    ops = model.layer_ops(layers, batch, hw, hw, c)
    kinds = [l["op"] in ("conv", "dwconv", "fc") for l in layers]
    ch = [l["cout"] for l in layers]
    n = len(layers)

    def can_extend(start, i):   # layers start..i+1 are, or can still become, one fused group
        return B.net_tuner_may_fuse(net, start, i + 1, True, 148)

    def may_close(start, i):    # layers start..i already are a group one kernel runs
        return i == start or B.net_tuner_may_fuse(net, start, i, False, 148)

    want = model.algorithm1(kinds, ch, ops, dict(P, op_critical=crit),
                            must_close_after=lambda start, i: i == n - 1 or not can_extend(start, i), may_close=may_close)
    got = B.net_autotune(net, n, P["alpha"], P["beta"], P["kappa"], P["kappa0"], crit, s_max=148, legalise=0)
    assert got == (want[0], want[1]), (got, want)
    if name == "mobilenet_v2" and crit == 1e30:   # the blocks whose fused kernel is estimated to pay become one group each
        firsts = [0] + [e + 1 for e in got[0][:-1]]
        assert sum(1 for a, e in zip(firsts, got[0]) if e - a + 1 >= 2) >= 6
    if name == "two_layer" and crit == 1e30:      # the two narrow 3x3 layers: the fused kernel is estimated to pay
        assert got[0] == [1]
    if name == "resnet50" and crit == 1e30:       # a projection branch and the expansion layer it is added to: one product
        pairs = [i for i, l in enumerate(layers) if l["res_src"] == i - 1 and l["op"] == "conv"]
        assert len(pairs) == 4
        for i in pairs:
            assert B.net_tuner_may_fuse(net, i - 1, i, False, 148) and i - 1 not in got[0] and i in got[0]
            assert not B.net_tuner_may_fuse(net, i - 2, i - 1, False, 148)   # (the 3x3 layer does not feed the projection)
        assert len(got[0]) == n - 4
    B.net_destroy(net)


# ---- the search's dynamic programme against exhaustive enumeration --------------------------------------------------
def test_bruteforce_table_on_the_hand_worked_example():
    # the table of tests/test_oracle_model.py: three layers, core counts {1, 2}
    table = {(0, 0, 1): 5, (0, 0, 2): 3, (1, 1, 1): 4, (1, 1, 2): 2.5, (2, 2, 1): 6, (2, 2, 2): 3.5,
             (0, 1, 1): 6, (0, 1, 2): 4, (1, 2, 1): 7, (1, 2, 2): 5.5}
    ms = [[[table.get((a, a + l, m), -1.0) for m in (1, 2)] for l in range(3)] for a in range(3)]
    assert B.bruteforce_table(3, 3, [1, 2], ms) == ([1, 2], [2, 2], 7.5)     # [0,1][2] -> 4 + 3.5
    assert B.bruteforce_table(3, 1, [1, 2], [[r[0]] for r in ms]) == ([0, 1, 2], [2, 2, 2], 9.0)


@pytest.mark.parametrize("seed", range(12))
def test_bruteforce_table_equals_exhaustive_search(seed):
    import random
    rnd = random.Random(seed)
    n, q, max_len = rnd.randint(1, 6), rnd.randint(1, 3), rnd.randint(1, 4)
    choices = sorted(rnd.sample(range(1, 149), q))
    ms = [[[(-1.0 if (l > 0 and rnd.random() < 0.3) or a + l >= n else round(rnd.uniform(0.5, 9.0), 3)) for _ in choices]
           for l in range(max_len)] for a in range(n)]

    def group_time(a, e, m):
        if e - a >= max_len:
            return None
        v = ms[a][e - a][choices.index(m)]
        return None if v < 0 else v

    want = model.best_plan_exhaustive(n, choices, group_time, max_len=max_len)
    ends, smc, best = B.bruteforce_table(n, max_len, choices, ms)
    assert best == pytest.approx(want[0], rel=1e-5)
    total = sum(group_time(a, e, m) for a, e, m in zip([0] + [x + 1 for x in ends[:-1]], ends, smc))   # the plan returned costs what is claimed
    assert total == pytest.approx(best, rel=1e-5)


def test_bruteforce_table_without_a_partition():
    import ctypes as C
    assert B.lib().dlf_bruteforce_table(2, 2, 1, (C.c_int32 * 1)(4), (C.c_float * 4)(1.0, -1.0, -1.0, -1.0), C.byref(C.c_int()),
                                        (C.c_int32 * 2)(), (C.c_int32 * 2)(), None) == B.E_PLAN
