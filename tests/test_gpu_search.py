"""GPU tests of the reduced brute-force search (Sec. V, "Oracle Case"), of the timing calls it is built from, of the
host-buffer entry point, of the ablation plans (Table 3) and of the bounded device-side waits."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import executor as orc
from paper_2011_05630_b200 import binding as B, networks as nw, plans, synth
from paper_2011_05630_b200.runtime import Session
from tests import gpu_util as G
from tests.test_gpu_parity import _conv, _bottleneck_with_projection


def _mk(layers, tag, n, h, w, c):
    params = synth.layer_params(tag, layers)
    x = synth.network_input(tag, n, h, w, c)
    ref = orc.run_network(layers, params, x)
    sess = Session(layers, params, n, h, w, c)
    return sess, sess.upload(x), x, ref


NETS = [("chain64", [_conv(64, 64, 3, src=-1), _conv(64, 64, 1, src=0), _conv(64, 64, 3, src=1), _conv(64, 64, 1, src=2)], 2, 28, 28, 64),
        ("bottlenecks", _bottleneck_with_projection(), 2, 18, 22, 32)]


@pytest.mark.parametrize("name,layers,n,h,w,c", NETS, ids=[t[0] for t in NETS])
def test_bruteforce_returns_a_legal_plan_that_is_not_slower_than_single_layers(name, layers, n, h, w, c):
    sess, xd, _, ref = _mk(layers, "bf-" + name, n, h, w, c)
    nl = len(layers)
    sms = B.device_sm_count()
    choices = plans.sm_fractions(sms)
    stream = torch.cuda.current_stream().cuda_stream
    pairs = sorted(set(list(range(1, nl, 2)) + [nl - 1]))             # some plan is in force: groups of two layers
    sess.set_plan(pairs, [sms] * len(pairs))
    before = B.net_get_plan(sess.net, nl)
    ends, smc, best_ms = B.net_bruteforce(sess.net, nl, choices, 4, xd.data_ptr(), stream, warmup=1, iters=3)
    assert B.net_get_plan(sess.net, nl) == before                      # the search installs nothing
    assert ends[-1] == nl - 1 and ends == sorted(set(ends)) and len(smc) == len(ends)
    firsts = [0] + [e + 1 for e in ends[:-1]]
    for a, e, s in zip(firsts, ends, smc):
        assert s in choices and e - a + 1 <= 4
        assert B.net_group_is_legal(sess.net, a, e, s)
    # the plan in force before the search still runs and is still right (its graph was not left stale)
    sess.run(xd)
    G.compare(sess.boundary(nl - 1), ref[nl - 1], "plan kept across the search")
    # the found plan computes the right thing, and its time is at most that of the best single-layer groups
    G.check_plan(sess, xd, ref, ends, smc, "brute-force plan " + name)
    singles = [min(B.net_time_span(sess.net, i, i, s, xd.data_ptr(), stream, 1, 3, prepare=(i == 0 and s == choices[0])) for s in choices)
               for i in range(nl)]
    assert best_ms <= 1.05 * sum(singles) + 0.002, (best_ms, singles)
    sess.close()


def test_time_span_and_per_group_times_add_up():
    layers = [_conv(128, 128, 3, src=i - 1) for i in range(4)]
    sess, xd, _, ref = _mk(layers, "timing", 8, 56, 56, 128)
    sms = B.device_sm_count()
    stream = torch.cuda.current_stream().cuda_stream
    sess.set_plan(None, None)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=sess.device)
    med, mn, per = B.net_time(sess.net, xd.data_ptr(), sess.out.data_ptr(), 4, stream, 3, 20, flush.data_ptr(), flush.numel())
    assert 0 < mn <= med and len(per) == 4 and all(p > 0 for p in per)
    # the instrumented pass records an event after every group, which keeps a kernel's set-up from overlapping its
    # predecessor's tail: a few microseconds per group on top of the plain run
    assert 0.85 * med <= sum(per) <= 1.15 * med + 0.007 * len(per), (per, med)
    G.compare(sess.boundary(3), ref[3], "output after the timed runs")
    one = B.net_time_span(sess.net, 1, 1, sms, xd.data_ptr(), stream, 2, 5, prepare=True)
    assert 0 < one <= 1.5 * max(per)                                   # warm L2, back to back: not slower than in the net
    with pytest.raises(B.DlfError) as e:                               # a span that is no group, an SM count out of range
        B.net_time_span(sess.net, 0, 1, sms + 1, xd.data_ptr(), stream, 1, 1, prepare=False)
    assert e.value.status == B.E_PLAN
    sess.close()


def test_run_host_matches_the_checker():
    layers = _bottleneck_with_projection()
    sess, xd, x, ref = _mk(layers, "runhost", 3, 18, 22, 32)
    nl = len(layers)
    sess.set_plan([2, 5, nl - 1], [B.device_sm_count()] * 3)
    xin = torch.from_numpy(x.view(np.int16)).pin_memory()
    out = torch.empty(ref[-1].shape, dtype=torch.int16).pin_memory()
    for _ in range(2):
        out.fill_(0)
        B.net_run_host(sess.net, xin.data_ptr(), out.data_ptr(), torch.cuda.current_stream().cuda_stream)
        G.compare(out.numpy().view(np.float16), ref[-1], "host-buffer run")
    sess.close()


def test_ablation_plans_have_the_shapes_of_table3():
    layers = nw.mobilenet_v2()
    params = synth.layer_params("abl", layers)
    sess = Session(layers, params, 1, 64, 64, 3)
    nl, sms = len(layers), B.device_sm_count()
    rows = plans.ablation_plans(sess.net, nl, sms)
    assert [r[0][0] for r in rows] == list("123456")
    by = {r[0][0]: r for r in rows}
    assert by["1"][1] == list(range(nl)) and by["1"][2] == [1] * nl                 # no fusion, one SM
    assert by["2"][1] == list(range(nl)) and by["2"][2] is None                     # no fusion, one SM count to be searched
    n_param = sum(1 for l in layers if l["op"] in ("conv", "dwconv", "fc"))
    assert n_param <= len(by["3"][1]) <= nl                                         # one block per parametrised layer (a pool may stand alone)
    assert all(1 <= s <= sms for s in by["3"][2])
    assert by["4"][2] == [sms] * len(by["4"][1]) and len(by["4"][1]) < len(by["3"][1])   # everything fused that can be
    assert by["5"][1] == by["6"][1] and by["5"][2] == [sms] * len(by["5"][1])       # Algorithm 1's blocks, all SMs / own SMs
    assert set(by["6"][1]) >= set(by["4"][1]) or len(by["6"][1]) >= len(by["4"][1]) # strategy 4's blocks are unions of 6's
    for name, ends, smc in rows:
        if smc is not None:
            sess.set_plan(ends, smc)                                                # every strategy is a legal plan
    sess.close()


def test_a_device_wait_that_never_ends_gives_up_and_reports():
    layers = nw.two_layer_group()
    sess, xd, _, ref = _mk(layers, "stall", 1, 32, 32, 16)
    stream = torch.cuda.current_stream().cuda_stream
    G.check_plan(sess, xd, ref, [1], [4], "before")
    B.net_debug_stall(sess.net, 1000, stream)          # a barrier nothing arrives at, limit 1 ms
    with pytest.raises(B.DlfError) as e:
        B.net_sync(sess.net, stream)
    assert e.value.status == B.E_TIMEOUT
    B.net_sync(sess.net, stream)                       # reported once, then clear
    G.check_plan(sess, xd, ref, [1], [4], "after")     # the context is intact, the next run is right
    G.check_plan(sess, xd, ref, [0, 1], [B.device_sm_count()] * 2, "after, unfused")
    sess.close()
