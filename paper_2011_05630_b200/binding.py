"""ctypes binding of libdlfusion.so: the same names as include/dlfusion.h, argument
marshalling only.  Device pointers are plain integers (e.g. torch.Tensor.data_ptr()).
Loading fails loudly when the library has not been built; there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdlfusion.so")

OK, E_INVALID_ARG, E_SHAPE, E_PLAN, E_WORKSPACE, E_UNSUPPORTED, E_CUDA, E_TIMEOUT, E_STATE = (
    0, -1, -2, -3, -4, -5, -6, -7, -8)
OPS = {"conv": 0, "dwconv": 1, "fc": 2, "maxpool": 3, "gavgpool": 4}
ACTS = {"none": 0, "relu": 1, "relu6": 2}
OPT_NO_TENSOR_CORE, OPT_SINGLE_AS_CHAIN, OPT_CUDA_GRAPH, OPT_PDL, OPT_CONV_ROW_MODE, OPT_GROUP_KERNEL = 1, 3, 4, 5, 6, 7


class LayerDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("op", "act", "cin", "cout", "kh", "kw", "stride", "pad",
                                         "groups", "src", "res_src", "pool")]


class TunerParams(C.Structure):
    _fields_ = [("alpha", C.c_double), ("beta", C.c_double), ("kappa", C.c_double),
                ("kappa0", C.c_double), ("op_critical", C.c_double), ("s_max", C.c_int32),
                ("legalise", C.c_int32)]


class SearchParams(C.Structure):
    _fields_ = [("n_sm_choices", C.c_int32), ("sm_choices", C.c_int32 * 16),
                ("max_group_len", C.c_int32), ("warmup", C.c_int32), ("iters", C.c_int32)]


class DlfError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__("%s: %s (status %d, cuda error %d)" % (what, strerror(status), status, last_cuda_error()))


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libdlfusion.so is not built: run `python -m paper_2011_05630_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i32p, i64p, fp = C.c_void_p, C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.POINTER(C.c_float)
        ip = C.POINTER(C.c_int)
        sig = {
            "dlf_strerror": (C.c_char_p, [C.c_int]),
            "dlf_last_cuda_error": (C.c_int, []),
            "dlf_device_sm_count": (C.c_int, []),
            "dlf_net_create": (C.c_int, [C.POINTER(LayerDesc), C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(vp)]),
            "dlf_net_destroy": (None, [vp]),
            "dlf_net_layer_info": (C.c_int, [vp, C.c_int, i64p, i64p, i64p]),
            "dlf_net_set_weights": (C.c_int, [vp, C.c_int, vp, vp]),
            "dlf_net_workspace_bytes": (C.c_int, [vp, C.POINTER(C.c_size_t)]),
            "dlf_net_bind_workspace": (C.c_int, [vp, vp, C.c_size_t]),
            "dlf_net_set_plan": (C.c_int, [vp, C.c_int, i32p, i32p]),
            "dlf_net_plan_unfused": (C.c_int, [vp]),
            "dlf_net_get_plan": (C.c_int, [vp, ip, i32p, i32p]),
            "dlf_net_group_is_legal": (C.c_int, [vp, C.c_int, C.c_int, C.c_int]),
            "dlf_net_tuner_may_fuse": (C.c_int, [vp, C.c_int, C.c_int, C.c_int, C.c_int]),
            "dlf_net_autotune": (C.c_int, [vp, C.POINTER(TunerParams), ip, i32p, i32p]),
            "dlf_net_bruteforce": (C.c_int, [vp, C.POINTER(SearchParams), vp, vp, ip, i32p, i32p, fp]),
            "dlf_bruteforce_table": (C.c_int, [C.c_int, C.c_int, C.c_int, i32p, fp, ip, i32p, i32p, fp]),
            "dlf_net_time_span": (C.c_int, [vp, C.c_int, C.c_int, C.c_int, vp, vp, C.c_int, C.c_int, C.c_int, fp]),
            "dlf_net_run": (C.c_int, [vp, vp, vp, vp]),
            "dlf_net_run_host": (C.c_int, [vp, vp, vp, vp]),
            "dlf_net_sync": (C.c_int, [vp, vp]),
            "dlf_net_debug_stall": (C.c_int, [vp, C.c_int, vp]),
            "dlf_net_time": (C.c_int, [vp, vp, vp, vp, C.c_int, C.c_int, vp, C.c_size_t, fp, fp, fp]),
            "dlf_net_boundary_tensor": (C.c_int, [vp, C.c_int, C.POINTER(vp), i64p]),
            "dlf_net_group_model": (C.c_int, [vp, C.c_int, i64p, i64p, C.POINTER(C.c_double), ip]),
            "dlf_net_group_kernel": (C.c_char_p, [vp, C.c_int]),
            "dlf_net_set_option": (C.c_int, [vp, C.c_int, C.c_int]),
            "dlf_conv_chain_run_static": (C.c_int, [C.POINTER(LayerDesc), C.c_int, C.c_int, C.c_int, C.c_int, vp,
                                                    C.POINTER(vp), C.POINTER(vp), vp, C.c_int, vp]),
        }
        for name, (res, args) in sig.items():
            f = getattr(L, name)
            f.restype, f.argtypes = res, args
        _lib = L
    return _lib


def _check(status, what):
    if status != OK:
        raise DlfError(status, what)


def strerror(status):
    return lib().dlf_strerror(status).decode()


def last_cuda_error():
    return lib().dlf_last_cuda_error()


def device_sm_count():
    n = lib().dlf_device_sm_count()
    if n < 0:
        raise DlfError(n, "dlf_device_sm_count")
    return n


def layer_descs(layers):
    arr = (LayerDesc * len(layers))()
    for i, l in enumerate(layers):
        arr[i] = LayerDesc(OPS[l["op"]], ACTS[l["act"]], l["cin"], l["cout"], l["kh"], l["kw"], l["stride"],
                           l["pad"], l["groups"], l["src"], l.get("res_src", -2), l.get("pool", 0))
    return arr


def net_create(layers, n, h, w, c):
    """layers: list of layer dicts (see networks.py) or a ctypes LayerDesc array."""
    arr = layers if isinstance(layers, C.Array) else layer_descs(layers)
    out = C.c_void_p()
    _check(lib().dlf_net_create(arr, len(arr), n, h, w, c, C.byref(out)), "dlf_net_create")
    return out


def net_destroy(net):
    lib().dlf_net_destroy(net)


def net_layer_info(net, i):
    ops, fl, sh = C.c_int64(), C.c_int64(), (C.c_int64 * 4)()
    _check(lib().dlf_net_layer_info(net, i, C.byref(ops), C.byref(fl), sh), "dlf_net_layer_info")
    return ops.value, fl.value, tuple(sh)


def net_set_weights(net, i, w_ptr, bias_ptr):
    _check(lib().dlf_net_set_weights(net, i, w_ptr, bias_ptr), "dlf_net_set_weights")


def net_workspace_bytes(net):
    b = C.c_size_t()
    _check(lib().dlf_net_workspace_bytes(net, C.byref(b)), "dlf_net_workspace_bytes")
    return b.value


def net_bind_workspace(net, ptr, nbytes):
    _check(lib().dlf_net_bind_workspace(net, ptr, nbytes), "dlf_net_bind_workspace")


def _i32(vals):
    return (C.c_int32 * len(vals))(*vals)


def net_set_plan(net, group_end, sm_count):
    _check(lib().dlf_net_set_plan(net, len(group_end), _i32(group_end), _i32(sm_count)), "dlf_net_set_plan")


def net_plan_unfused(net):
    _check(lib().dlf_net_plan_unfused(net), "dlf_net_plan_unfused")


def net_get_plan(net, n_layers):
    n = C.c_int()
    e, s = (C.c_int32 * n_layers)(), (C.c_int32 * n_layers)()
    _check(lib().dlf_net_get_plan(net, C.byref(n), e, s), "dlf_net_get_plan")
    return list(e[:n.value]), list(s[:n.value])


def net_group_is_legal(net, first, last, sm_count):
    r = lib().dlf_net_group_is_legal(net, first, last, sm_count)
    if r < 0:
        raise DlfError(r, "dlf_net_group_is_legal")
    return bool(r)


def net_tuner_may_fuse(net, first, last, prefix, s_max):
    r = lib().dlf_net_tuner_may_fuse(net, first, last, 1 if prefix else 0, s_max)
    if r < 0:
        raise DlfError(r, "dlf_net_tuner_may_fuse")
    return bool(r)


def net_autotune(net, n_layers, alpha, beta, kappa, kappa0, op_critical, s_max=0, legalise=0):
    p = TunerParams(alpha, beta, kappa, kappa0, op_critical, s_max, legalise)
    n = C.c_int()
    e, s = (C.c_int32 * n_layers)(), (C.c_int32 * n_layers)()
    _check(lib().dlf_net_autotune(net, C.byref(p), C.byref(n), e, s), "dlf_net_autotune")
    return list(e[:n.value]), list(s[:n.value])


def net_bruteforce(net, n_layers, sm_choices, max_group_len, in_ptr, stream=None, warmup=2, iters=5):
    sp = SearchParams()
    sp.n_sm_choices = len(sm_choices)
    for i, v in enumerate(sm_choices):
        sp.sm_choices[i] = v
    sp.max_group_len, sp.warmup, sp.iters = max_group_len, warmup, iters
    n, ms = C.c_int(), C.c_float()
    e, s = (C.c_int32 * n_layers)(), (C.c_int32 * n_layers)()
    _check(lib().dlf_net_bruteforce(net, C.byref(sp), in_ptr, stream, C.byref(n), e, s, C.byref(ms)), "dlf_net_bruteforce")
    return list(e[:n.value]), list(s[:n.value]), ms.value


def bruteforce_table(n_layers, max_group_len, sm_choices, ms):
    """ms[a][len - 1][c]: time of span a..a+len-1 on sm_choices[c] SMs, negative = cannot run."""
    flat = [float(ms[a][l][c]) for a in range(n_layers) for l in range(max_group_len) for c in range(len(sm_choices))]
    n, best = C.c_int(), C.c_float()
    e, s = (C.c_int32 * n_layers)(), (C.c_int32 * n_layers)()
    _check(lib().dlf_bruteforce_table(n_layers, max_group_len, len(sm_choices), _i32(sm_choices), (C.c_float * len(flat))(*flat),
                                      C.byref(n), e, s, C.byref(best)), "dlf_bruteforce_table")
    return list(e[:n.value]), list(s[:n.value]), best.value


def net_time_span(net, first, last, sm_count, in_ptr, stream=None, warmup=2, iters=5, prepare=True):
    ms = C.c_float()
    _check(lib().dlf_net_time_span(net, first, last, sm_count, in_ptr, stream, warmup, iters, 1 if prepare else 0,
                                   C.byref(ms)), "dlf_net_time_span")
    return ms.value


def net_run(net, in_ptr, out_ptr, stream=None):
    _check(lib().dlf_net_run(net, in_ptr, out_ptr, stream), "dlf_net_run")


def net_run_host(net, in_host_ptr, out_host_ptr, stream=None):
    _check(lib().dlf_net_run_host(net, in_host_ptr, out_host_ptr, stream), "dlf_net_run_host")


def net_sync(net, stream=None):
    _check(lib().dlf_net_sync(net, stream), "dlf_net_sync")


def net_debug_stall(net, limit_us, stream=None):
    _check(lib().dlf_net_debug_stall(net, limit_us, stream), "dlf_net_debug_stall")


def net_time(net, in_ptr, out_ptr, n_groups, stream=None, warmup=3, iters=10, flush_ptr=None, flush_bytes=0,
             per_group=True):
    med, mn = C.c_float(), C.c_float()
    pg = (C.c_float * max(n_groups, 1))() if per_group else None
    _check(lib().dlf_net_time(net, in_ptr, out_ptr, stream, warmup, iters, flush_ptr, flush_bytes, C.byref(med),
                              C.byref(mn), pg), "dlf_net_time")
    return med.value, mn.value, (list(pg[:n_groups]) if per_group else None)


def net_boundary_tensor(net, layer):
    p, sh = C.c_void_p(), (C.c_int64 * 4)()
    _check(lib().dlf_net_boundary_tensor(net, layer, C.byref(p), sh), "dlf_net_boundary_tensor")
    return p.value, tuple(sh)


def net_group_model(net, g):
    fl, by, red, la = C.c_int64(), C.c_int64(), C.c_double(), C.c_int()
    _check(lib().dlf_net_group_model(net, g, C.byref(fl), C.byref(by), C.byref(red), C.byref(la)), "dlf_net_group_model")
    return fl.value, by.value, red.value, la.value


def net_group_kernel(net, g):
    return lib().dlf_net_group_kernel(net, g).decode()


def net_set_option(net, option, value):
    _check(lib().dlf_net_set_option(net, option, value), "dlf_net_set_option")


STATIC_SCRATCH_BYTES = 16 << 20


def conv_chain_run_static(layers, n, h, w, x_ptr, w_ptrs, bias_ptrs, y_ptr, sm_count, stream=None):
    """Chain of dense convolutions with the library's built-in scratch array (no workspace, no
    allocation); waits for the stream.  Pointers are device addresses."""
    arr = layers if isinstance(layers, C.Array) else layer_descs(layers)
    wp = (C.c_void_p * len(arr))(*w_ptrs)
    bp = (C.c_void_p * len(arr))(*bias_ptrs)
    _check(lib().dlf_conv_chain_run_static(arr, len(arr), n, h, w, x_ptr, wp, bp, y_ptr, sm_count, stream),
           "dlf_conv_chain_run_static")
