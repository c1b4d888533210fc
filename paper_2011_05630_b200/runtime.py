"""Plumbing around the C ABI: device memory through PyTorch, nothing else.

`Session` uploads a layer list's parameters, allocates the workspace the library asks
for, and hands raw device pointers to the binding.  Every step of the computation runs
inside libdlfusion.so.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


def _to_dev(a: np.ndarray, device) -> torch.Tensor:
    if a.dtype == np.float16:
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.float16)
    return torch.from_numpy(a).to(device)


class Session:
    def __init__(self, layers, params, n, h, w, c, device="cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: there is no CPU path")
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.layers, self.shape = layers, (n, h, w, c)
        self.net = B.net_create(layers, n, h, w, c)
        self._keep = []
        for i, p in enumerate(params):
            if p is None:
                continue
            wt, bt = _to_dev(np.ascontiguousarray(p[0]), self.device), _to_dev(np.ascontiguousarray(p[1]), self.device)
            self._keep += [wt, bt]
            B.net_set_weights(self.net, i, wt.data_ptr(), bt.data_ptr())
        nbytes = B.net_workspace_bytes(self.net)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        ptr = (self.workspace.data_ptr() + 255) // 256 * 256
        B.net_bind_workspace(self.net, ptr, nbytes)
        self.out_shape = B.net_layer_info(self.net, len(layers) - 1)[2]
        self.out = torch.empty(self.out_shape, dtype=torch.float16, device=self.device)
        self.n_groups = 0

    def close(self):
        if self.net is not None:
            B.net_destroy(self.net)
            self.net = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_plan(self, group_end=None, sm_count=None):
        if group_end is None:
            B.net_plan_unfused(self.net)
        else:
            B.net_set_plan(self.net, group_end, sm_count)
        ends, sms = B.net_get_plan(self.net, len(self.layers))
        self.n_groups = len(ends)
        return ends, sms

    def upload(self, x: np.ndarray) -> torch.Tensor:
        assert x.dtype == np.float16 and tuple(x.shape) == self.shape
        return _to_dev(np.ascontiguousarray(x), self.device)

    def run(self, x_dev: torch.Tensor) -> torch.Tensor:
        stream = torch.cuda.current_stream().cuda_stream
        B.net_run(self.net, x_dev.data_ptr(), self.out.data_ptr(), stream)
        B.net_sync(self.net, stream)
        return self.out

    def boundary(self, layer: int) -> np.ndarray:
        """Host copy of a group-ending layer's output (fp16 NHWC)."""
        ptr, shape = B.net_boundary_tensor(self.net, layer)
        n = int(np.prod(shape))
        t = torch.empty(n, dtype=torch.float16, device=self.device)
        # device-to-device copy from the raw pointer through a zero-copy view
        src = _wrap(ptr, n, self.device)
        t.copy_(src)
        return t.cpu().numpy().reshape(shape)

    def kernels(self):
        return [B.net_group_kernel(self.net, g) for g in range(self.n_groups)]


class _Holder:
    def __init__(self, ptr, nbytes):
        self.__cuda_array_interface__ = {"shape": (nbytes // 2,), "typestr": "<f2", "data": (ptr, False), "version": 2}


def _wrap(ptr: int, n_half: int, device) -> torch.Tensor:
    return torch.as_tensor(_Holder(ptr, n_half * 2), device=device)
