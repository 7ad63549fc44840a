"""ctypes binding of libpsmc_workload.so: the CUDA twins of `gen.logits_block` and `gen.kv_block`.

Input generation only; used by the GPU tests, the smoke check and the benchmark to fill device
buffers with the same seeded synthetic data the numpy generators produce.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from .. import build as _build
from . import gen

_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(_build.LIB_WORKLOAD):
            raise ImportError("libpsmc_workload.so is missing: run `python -m paper_2602_10273_b200.build`")
        L = C.CDLL(_build.LIB_WORKLOAD)
        L.psmc_wl_logits.restype = C.c_int
        L.psmc_wl_logits.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int64, C.c_uint64, C.c_int, C.c_int,
                                     C.c_int, C.c_void_p, C.c_double, C.c_void_p, C.c_void_p]
        L.psmc_wl_kv.restype = C.c_int
        L.psmc_wl_kv.argtypes = [C.c_void_p, C.c_int, C.c_uint64, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                 C.c_int, C.c_int, C.c_void_p]
        _lib = L
    return _lib


def _dt(t: torch.Tensor) -> int:
    return {torch.float32: 0, torch.bfloat16: 1}[t.dtype]


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def fill_logits(dst: torch.Tensor, seed: int, t: int, N: int, prev: torch.Tensor, scale: float, bias: torch.Tensor,
                g0: int = 0) -> None:
    """dst [R, V] on the GPU <- logits of step t; row r belongs to group g0 + r // N; prev int32 [R]; bias f64 [V]."""
    R, V = dst.shape
    assert dst.is_cuda and dst.stride(1) == 1 and prev.dtype == torch.int32 and prev.is_cuda and prev.numel() == R
    assert bias.dtype == torch.float64 and bias.is_cuda and bias.numel() == V
    rc = lib().psmc_wl_logits(dst.data_ptr(), _dt(dst), R, V, dst.stride(0), seed, t, g0, N, prev.data_ptr(),
                              float(scale), bias.data_ptr(), _stream())
    if rc:
        raise RuntimeError("psmc_wl_logits: CUDA error %d" % rc)


def fill_kv(dst: torch.Tensor, seed: int, layer: int, which: int, row0: int = 0) -> None:
    """dst contiguous [R, H, max_len, D] on the GPU <- hashed N(0,1) of rows row0.. of (layer, K/V)."""
    assert dst.is_cuda and dst.is_contiguous() and dst.dim() == 4
    R, H, L, D = dst.shape
    rc = lib().psmc_wl_kv(dst.data_ptr(), _dt(dst), seed, layer, which, row0, R, H, L, D, _stream())
    if rc:
        raise RuntimeError("psmc_wl_kv: CUDA error %d" % rc)


class DeviceWorkload:
    """Device-resident synthetic LM for one named configuration (or a cut-down copy of it)."""

    def __init__(self, cfg: gen.Workload, seed: int, G: int = None, device="cuda"):
        self.cfg, self.seed = cfg, seed
        self.G = cfg.G if G is None else G
        self.N, self.V, self.R = cfg.N, cfg.V, self.G * cfg.N
        self.device = torch.device(device)
        self.tdtype = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
        self.bias_host = gen.vocab_bias(seed, cfg.V, cfg.slope)
        self.bias = torch.from_numpy(self.bias_host).to(self.device)
        self.prompt_len = gen.prompt_lengths(seed, self.G, cfg.prompt_lo, cfg.prompt_hi)
        last = gen.prompt_last_token(seed, self.G, self.prompt_len, cfg.V)
        self.first_prev = torch.from_numpy(np.repeat(last, cfg.N).astype(np.int32)).to(self.device)

    def new_logits(self) -> torch.Tensor:
        return torch.empty((self.R, self.V), dtype=self.tdtype, device=self.device)

    def fill(self, dst: torch.Tensor, t: int, prev: torch.Tensor) -> None:
        fill_logits(dst, self.seed, t, self.N, prev, self.cfg.scale, self.bias)

    def new_kv(self):
        """Allocate and fill every layer's K and V: lists of [R, H, max_len, D] tensors."""
        c = self.cfg
        ks, vs = [], []
        for l in range(c.n_layers):
            for which, out in ((0, ks), (1, vs)):
                t = torch.empty((self.R, c.n_kv_heads, c.max_len, c.head_dim), dtype=self.tdtype, device=self.device)
                fill_kv(t, self.seed, l, which)
                out.append(t)
        return ks, vs
