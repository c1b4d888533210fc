"""The allocation-free entry point against the regular one.

dlf_conv_chain_run_static serves callers that cannot allocate device memory (a process whose
GPU memory is already spoken for, a fixed budget, a loop that cannot afford cudaMalloc's
device-wide synchronisation): its scratch is a fixed array inside the library.  The test calls
it twice in a row through the C ABI - the second call finds the first call's leftovers in the
shared array - and checks both results against dlf_net_run on the same tensors, within the
tolerance of the other GPU tests.  It also checks that a chain whose intermediate map exceeds
the fixed scratch is refused.  Collected last on purpose."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle import executor as orc
from paper_2011_05630_b200 import binding as B, synth
from paper_2011_05630_b200.runtime import Session
from tests import gpu_util as G


def _conv(cin, cout, k, src, stride=1, act="relu"):
    return dict(op="conv", act=act, cin=cin, cout=cout, kh=k, kw=k, stride=stride, pad=k // 2, groups=1, src=src,
                res_src=-2, pool=0)


def test_static_scratch_entry_matches_workspace_entry_twice():
    layers = [_conv(32, 64, 3, -1), _conv(64, 64, 3, 0, stride=2), _conv(64, 128, 1, 1, act="none")]
    n, h, w = 3, 37, 41
    params = synth.layer_params("noalloc", layers)
    sms = B.device_sm_count()
    sess = Session(layers, params, n, h, w, 32)
    sess.set_plan(None, None)
    w_ptrs = [sess._keep[2 * i].data_ptr() for i in range(3)]
    b_ptrs = [sess._keep[2 * i + 1].data_ptr() for i in range(3)]
    y = torch.empty(sess.out_shape, dtype=torch.float16, device=sess.device)
    for call, tag in enumerate(("noalloc-x0", "noalloc-x1")):
        x = synth.network_input(tag, n, h, w, 32)
        xd = sess.upload(x)
        want = sess.run(xd).cpu().numpy()
        G.compare(want, orc.run_network(layers, params, x)[-1], "workspace entry against the CPU checker, call %d" % call)
        y.fill_(float("nan"))
        B.conv_chain_run_static(layers, n, h, w, xd.data_ptr(), w_ptrs, b_ptrs, y.data_ptr(), sms,
                                torch.cuda.current_stream().cuda_stream)
        G.compare(y.cpu().numpy(), want, "static scratch, call %d" % call)
        G.compare(y.cpu().numpy(), orc.run_network(layers, params, x)[-1], "static scratch against the CPU checker, call %d" % call)
    sess.close()


def test_static_scratch_entry_rejects_maps_beyond_its_array():
    layers = [_conv(16, 64, 3, -1), _conv(64, 16, 3, 0)]
    n, h, w = 8, 96, 96          # 8*96*96*64*2 bytes = 9.4 MB > half of the 16 MiB array
    assert n * h * w * 64 * 2 > B.STATIC_SCRATCH_BYTES // 2
    params = synth.layer_params("noalloc-big", layers)
    dev = torch.device("cuda:0")
    keep = [torch.from_numpy(a.view(np.int16) if a.dtype == np.float16 else a).to(dev) for p in params for a in p]
    x = torch.zeros((n, h, w, 16), dtype=torch.float16, device=dev)
    y = torch.zeros((n, h, w, 16), dtype=torch.float16, device=dev)
    with pytest.raises(B.DlfError) as e:
        B.conv_chain_run_static(layers, n, h, w, x.data_ptr(), [keep[0].data_ptr(), keep[2].data_ptr()],
                                [keep[1].data_ptr(), keep[3].data_ptr()], y.data_ptr(), 8, None)
    assert e.value.status == B.E_WORKSPACE
