"""Layer-by-layer CPU execution of a layer list (TEST INFRASTRUCTURE ONLY).

Runs every layer in full, one after another, through the C routines of
dlf_oracle.c; there are no fusion plans here because every plan must reproduce this
result (Sec. I, "mathematically equivalent" fusion; Sec. III-B, on-chip reuse of a fused
layer's output).  Shape rule: H_out = floor((H + 2 pad - k) / stride) + 1, the output
size that Eq. 1's H_Out/W_Out refer to.

`cone_outputs` evaluates single output pixels of a chain of convolutions from their
dependency cone only (a cropped window clipped to the image), for shapes too large to
run in full: no value of this checker depends on how other pixels are evaluated, so the
result is the same bits as the full run (Sec. IV-B: the halo of a tile is recomputed,
not approximated).
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

_ACT = {"none": 0, "relu": 1, "relu6": 2}
_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.ensure_built())
        u16p, f32p = C.POINTER(C.c_uint16), C.POINTER(C.c_float)
        L.orc_conv2d.argtypes = [u16p, C.c_int, C.c_int, C.c_int, C.c_int, u16p, f32p, C.c_int,
                                 C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, u16p, C.c_int,
                                 C.c_int, u16p, C.c_int]
        L.orc_fc.argtypes = [u16p, C.c_int, C.c_int, u16p, f32p, C.c_int, C.c_int, u16p, C.c_int]
        L.orc_maxpool.argtypes = [u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                  C.c_int, u16p]
        L.orc_gavgpool.argtypes = [u16p, C.c_int, C.c_int, C.c_int, C.c_int, u16p]
        L.orc_h2f_array.argtypes = [u16p, f32p, C.c_int64]
        L.orc_f2h_array.argtypes = [f32p, u16p, C.c_int64]
        L.orc_threads.restype = C.c_int
        _lib = L
    return _lib


def _u16(a):
    return a.ctypes.data_as(C.POINTER(C.c_uint16))


def _f32(a):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def _h(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float16, a.dtype
    return a


def threads() -> int:
    return int(lib().orc_threads())


def half_to_float(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float32)
    lib().orc_h2f_array(_u16(bits), _f32(out), bits.size)
    return out


def float_to_half(vals: np.ndarray) -> np.ndarray:
    vals = np.ascontiguousarray(vals, dtype=np.float32)
    out = np.empty(vals.shape, dtype=np.uint16)
    lib().orc_f2h_array(_f32(vals), _u16(out), vals.size)
    return out


def out_hw(h, w, l):
    if l["op"] in ("conv", "dwconv", "maxpool"):
        ho = (h + 2 * l["pad"] - l["kh"]) // l["stride"] + 1
        wo = (w + 2 * l["pad"] - l["kw"]) // l["stride"] + 1
        if l.get("pool", 0) == 2:
            ho, wo = ho // 2, wo // 2
        return ho, wo
    return 1, 1


def conv2d(x, w, bias, stride=1, pad=0, groups=1, res=None, act="none", pool=0, nthreads=0):
    x, w = _h(x), _h(w)
    bias = np.ascontiguousarray(bias, dtype=np.float32)
    n, h, wd, cin = x.shape
    cout, kh, kw, cg = w.shape
    assert cg * groups == cin, (w.shape, cin, groups)
    ho = (h + 2 * pad - kh) // stride + 1
    wo = (wd + 2 * pad - kw) // stride + 1
    if res is not None:
        res = _h(res)
        assert res.shape == (n, ho, wo, cout), (res.shape, (n, ho, wo, cout))
    y = np.empty((n, ho // 2, wo // 2, cout) if pool else (n, ho, wo, cout), dtype=np.float16)
    rc = lib().orc_conv2d(_u16(x), n, h, wd, cin, _u16(w), _f32(bias), cout, kh, kw, stride, pad,
                          groups, _u16(res) if res is not None else None, _ACT[act], pool,
                          _u16(y), nthreads)
    if rc:
        raise ValueError("orc_conv2d rejected the sizes")
    return y


def fc(x, w, bias, act="none", nthreads=0):
    x, w = _h(x), _h(w)
    bias = np.ascontiguousarray(bias, dtype=np.float32)
    n = x.shape[0]
    x2 = x.reshape(n, -1)
    m, k = w.shape
    assert x2.shape[1] == k
    y = np.empty((n, m), dtype=np.float16)
    if lib().orc_fc(_u16(x2), n, k, _u16(w), _f32(bias), m, _ACT[act], _u16(y), nthreads):
        raise ValueError("orc_fc rejected the sizes")
    return y.reshape(n, 1, 1, m)


def maxpool(x, k, stride, pad):
    x = _h(x)
    n, h, w, c = x.shape
    ho, wo = (h + 2 * pad - k) // stride + 1, (w + 2 * pad - k) // stride + 1
    y = np.empty((n, ho, wo, c), dtype=np.float16)
    if lib().orc_maxpool(_u16(x), n, h, w, c, k, stride, pad, _u16(y)):
        raise ValueError("orc_maxpool rejected the sizes")
    return y


def gavgpool(x):
    x = _h(x)
    n, h, w, c = x.shape
    y = np.empty((n, 1, 1, c), dtype=np.float16)
    if lib().orc_gavgpool(_u16(x), n, h, w, c, _u16(y)):
        raise ValueError("orc_gavgpool rejected the sizes")
    return y


def run_layer(l, x, params, res=None, nthreads=0):
    if l["op"] in ("conv", "dwconv"):
        w, b = params
        return conv2d(x, w, b, l["stride"], l["pad"], l["groups"], res, l["act"], l.get("pool", 0),
                      nthreads)
    if l["op"] == "fc":
        w, b = params
        return fc(x, w, b, l["act"], nthreads)
    if l["op"] == "maxpool":
        return maxpool(x, l["kh"], l["stride"], l["pad"])
    if l["op"] == "gavgpool":
        return gavgpool(x)
    raise ValueError(l["op"])


def run_network(layers, params, x, keep=True, nthreads=0):
    """Every layer's fp16 output (list, index = layer); with keep=False only tensors still
    needed by a later `src`/`res_src` are retained and the rest are None."""
    outs = []
    last_use = {}
    for i, l in enumerate(layers):
        for s in (l["src"], l.get("res_src", -2)):
            if s >= 0:
                last_use[s] = i
    for i, l in enumerate(layers):
        src = x if l["src"] < 0 else outs[l["src"]]
        r = l.get("res_src", -2)
        res = None if r == -2 else (x if r == -1 else outs[r])
        outs.append(run_layer(l, src, params[i], res, nthreads))
        if not keep:
            for s, u in last_use.items():
                if u == i and s != len(layers) - 1:
                    outs[s] = None
    return outs


def cone_outputs(layers, params, x, pixels):
    """Final-layer values at `pixels` [(n, h, w), ...] of a chain of stride-1, size-keeping
    convolutions (each layer reads the previous one; no residual, no pooling), computed from
    each pixel's dependency cone.  Returns fp16 [len(pixels), cout]."""
    reach = 0
    for l in layers:
        assert l["op"] == "conv" and l["stride"] == 1 and l["kh"] == l["kw"] == 2 * l["pad"] + 1
        assert l.get("pool", 0) == 0 and l.get("res_src", -2) == -2
        reach += l["pad"]
    _, h, w, _ = x.shape
    out = np.empty((len(pixels), layers[-1]["cout"]), dtype=np.float16)
    for j, (n, py, px) in enumerate(pixels):
        y0, y1 = max(0, py - reach), min(h, py + reach + 1)
        x0, x1 = max(0, px - reach), min(w, px + reach + 1)
        t = np.ascontiguousarray(x[n:n + 1, y0:y1, x0:x1, :])
        for l, p in zip(layers, params):
            t = run_layer(l, t, p, None, 0)
        out[j] = t[0, py - y0, px - x0, :]
    return out
