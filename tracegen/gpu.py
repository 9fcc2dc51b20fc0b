"""CUDA sampler: fills a device buffer with the same bytes ``tracegen.cpu.generate`` returns.

Used for traces too large to build with numpy (2^28 .. 2^30 records).  Input generation only.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csrc", "tracegen.cu")
_LIB = os.path.join(_HERE, "libtracegen.so")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
                               "-shared", "-Xcompiler", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


class _Params(C.Structure):
    _fields_ = [("base", C.c_uint64), ("kind", C.c_uint32), ("n_apps", C.c_uint32), ("n_ops", C.c_uint32),
                ("n_shapes", C.c_uint32), ("n_phases", C.c_uint32), ("phase_cum", C.c_uint32 * 8),
                ("n_ranks", C.c_uint64), ("cum", C.c_void_p), ("perm_a", C.c_void_p), ("perm_b", C.c_void_p),
                ("kl_a", C.c_uint64), ("kl_b", C.c_uint64), ("hot_thresh", C.c_uint32), ("hot_phase", C.c_uint32),
                ("hot_op", C.c_uint32), ("hot_shape", C.c_uint32), ("dur_kind", C.c_uint32), ("dur_lo", C.c_uint32),
                ("dur_range", C.c_uint32), ("qtable", C.c_void_p)]


class GpuSampler:
    """Holds the device copies of a TraceSpec's tables; ``fill`` writes records into a tensor."""

    def __init__(self, spec, device="cuda:0"):
        import torch
        self._torch = torch
        self.spec = spec
        self.device = torch.device(device)
        self._lib = C.CDLL(build())
        self._lib.tracegen_generate.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
        self._keep = []

        def dev(a, dtype):
            if a is None:
                return None
            t = torch.from_numpy(np.ascontiguousarray(a).view(dtype)).to(self.device)
            self._keep.append(t)
            return t.data_ptr()

        p = _Params()
        p.base = spec.base
        p.kind, p.n_apps, p.n_ops, p.n_shapes, p.n_phases = spec.kind, spec.n_apps, spec.n_ops, spec.n_shapes, spec.n_phases
        for i in range(8):
            p.phase_cum[i] = int(spec.phase_cum[i])
        p.n_ranks = spec.n_ranks
        p.cum = dev(spec.cum, np.int64)
        p.perm_a = dev(spec.perm_a, np.int32)
        p.perm_b = dev(spec.perm_b, np.int32)
        p.kl_a, p.kl_b = spec.kl_a, spec.kl_b
        p.hot_thresh, p.hot_phase, p.hot_op, p.hot_shape = spec.hot_thresh, spec.hot_phase, spec.hot_op, spec.hot_shape
        p.dur_kind, p.dur_lo, p.dur_range = spec.dur_kind, spec.dur_lo, spec.dur_range
        p.qtable = dev(spec.qtable, np.int32)
        self._p = p

    def fill(self, out, start: int = 0, count: int | None = None):
        """``out``: uint8 CUDA tensor with room for ``count`` 16-byte records."""
        torch = self._torch
        if count is None:
            count = out.numel() // 16
        assert out.is_cuda and out.dtype == torch.uint8 and out.numel() >= count * 16
        stream = torch.cuda.current_stream(self.device).cuda_stream
        with torch.cuda.device(self.device):
            rc = self._lib.tracegen_generate(C.byref(self._p), start, count, out.data_ptr(), stream)
        if rc != 0:
            raise RuntimeError(f"tracegen_generate failed ({rc})")
        return out
