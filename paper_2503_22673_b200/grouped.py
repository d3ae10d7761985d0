"""Projections that consume the same X (q/k/v, gate/up) as ONE grouped call of the C library.

For groups g = 1..G with weights W_g [d_g, d_in] and adapters A_g [r, d_in], B_g [d_g, r]

    Y_g = X W_g^T + s (X A_g^T) B_g^T        dX = sum_g (dY_g W_g + s (dY_g B_g) A_g)

`lora_linear_fwd_grouped` / `lora_linear_bwd_grouped` take the groups' tensors stacked (W, A, B along rows, Y and dY along
columns) and run one forward GEMM, one dX GEMM and two skinny launches for the whole group.  This module only creates the
plan, checks shapes, passes pointers and hands out per-group views; it does no arithmetic.
"""
from __future__ import annotations

import ctypes
from typing import List, Sequence, Tuple

import torch

from . import binding
from .binding import _check, _ptr, _stream_ptr, _want


class LoraGroupShape(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int64), ("d_in", ctypes.c_int64), ("r", ctypes.c_int64), ("n_groups", ctypes.c_int32),
                ("d_out", ctypes.c_int64 * 4)]


class GroupedLoraPlan:
    """Plan for G = 2..4 projections sharing X (T > 128, r in {16, 32, 48, 64}, every d_g a multiple of 256)."""

    def __init__(self, T: int, d_in: int, d_outs: Sequence[int], r: int, device: int = 0):
        if not torch.cuda.is_available():
            raise binding.LoraError(binding.LORA_ERR_NO_DEVICE, "GroupedLoraPlan")
        self._lib = binding.load()
        self.d_outs = [int(d) for d in d_outs]
        self.G, self.r, self.T, self.d_in = len(self.d_outs), int(r), int(T), int(d_in)
        self.offsets = [0]
        for d in self.d_outs:
            self.offsets.append(self.offsets[-1] + d)
        self.D = self.offsets[-1]
        self.device = torch.device("cuda", device)
        shape = LoraGroupShape(self.T, self.d_in, self.r, self.G, (ctypes.c_int64 * 4)(*(self.d_outs + [0] * (4 - self.G))))
        self._h = ctypes.c_void_p(0)
        _check(self._lib.lora_plan_create_grouped(ctypes.byref(shape), device, ctypes.byref(self._h)), "lora_plan_create_grouped")
        fwd, bwd = ctypes.c_size_t(0), ctypes.c_size_t(0)
        _check(self._lib.lora_plan_workspace_bytes(self._h, ctypes.byref(fwd), ctypes.byref(bwd)), "lora_plan_workspace_bytes")
        self._ws = torch.empty(max(int(bwd.value), 256), dtype=torch.uint8, device=self.device)
        _check(self._lib.lora_plan_set_workspace(self._h, _ptr(self._ws), self._ws.numel()), "lora_plan_set_workspace")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.lora_plan_destroy(self._h)
            self._h = ctypes.c_void_p(0)
            self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def device_status(self, stream=None) -> Tuple[int, str]:
        code = ctypes.c_int(0)
        buf = ctypes.create_string_buffer(256)
        _check(self._lib.lora_last_device_status(self._h, _stream_ptr(stream), ctypes.byref(code), buf, 256),
               "lora_last_device_status")
        return int(code.value), buf.value.decode()

    # -- operand layout (copies for set-up; the stacked tensors can serve as the adapters' own storage) ---------------
    def pack(self, Ws, As, Bs) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """(W_cat [sum d_g, d_in], A_cat [G r, d_in], B_cat [sum d_g, r])."""
        return (torch.cat(list(Ws), dim=0).contiguous(), torch.cat(list(As), dim=0).contiguous(),
                torch.cat(list(Bs), dim=0).contiguous())

    def views(self, A_cat: torch.Tensor, B_cat: torch.Tensor):
        """Per-projection views (no copies) of stacked adapters or of their gradients."""
        As = [A_cat[g * self.r:(g + 1) * self.r] for g in range(self.G)]
        Bs = [B_cat[self.offsets[g]:self.offsets[g + 1]] for g in range(self.G)]
        return As, Bs

    def split_outputs(self, Y_cat: torch.Tensor) -> List[torch.Tensor]:
        return [Y_cat[:, self.offsets[g]:self.offsets[g + 1]] for g in range(self.G)]

    def _want_inputs(self, X, W_cat, A_cat, B_cat):
        bf = torch.bfloat16
        _want(X, "X", (self.T, self.d_in), bf, self.device)
        _want(W_cat, "W_cat", (self.D, self.d_in), bf, self.device)
        _want(A_cat, "A_cat", (self.G * self.r, self.d_in), bf, self.device)
        _want(B_cat, "B_cat", (self.D, self.r), bf, self.device)

    # -- the two calls ---------------------------------------------------------------------------
    def fwd(self, X, W_cat, A_cat, B_cat, scale: float, Y_cat=None, stream=None) -> torch.Tensor:
        """Y_cat [T, sum d_g]; ``split_outputs`` gives the per-projection column blocks."""
        self._want_inputs(X, W_cat, A_cat, B_cat)
        if Y_cat is None:
            Y_cat = torch.empty((self.T, self.D), dtype=torch.bfloat16, device=self.device)
        _want(Y_cat, "Y_cat", (self.T, self.D), torch.bfloat16, self.device)
        _check(self._lib.lora_linear_fwd_grouped(self._h, _ptr(X), _ptr(W_cat), _ptr(A_cat), _ptr(B_cat), float(scale),
                                                 _ptr(Y_cat), _stream_ptr(stream)), "lora_linear_fwd_grouped")
        return Y_cat

    def bwd(self, dY_cat, X, W_cat, A_cat, B_cat, scale: float, dX=None, dA_cat=None, dB_cat=None, stream=None):
        """(dX, [dA_g], [dB_g]); dA_g / dB_g are views into dA_cat [G r, d_in] / dB_cat [sum d_g, r]."""
        self._want_inputs(X, W_cat, A_cat, B_cat)
        _want(dY_cat, "dY_cat", (self.T, self.D), torch.bfloat16, self.device)
        if dX is None:
            dX = torch.empty((self.T, self.d_in), dtype=torch.bfloat16, device=self.device)
        if dA_cat is None:
            dA_cat = torch.empty((self.G * self.r, self.d_in), dtype=torch.float32, device=self.device)
        if dB_cat is None:
            dB_cat = torch.empty((self.D, self.r), dtype=torch.float32, device=self.device)
        _want(dX, "dX", (self.T, self.d_in), torch.bfloat16, self.device)
        _want(dA_cat, "dA_cat", (self.G * self.r, self.d_in), torch.float32, self.device)
        _want(dB_cat, "dB_cat", (self.D, self.r), torch.float32, self.device)
        _check(self._lib.lora_linear_bwd_grouped(self._h, _ptr(dY_cat), _ptr(X), _ptr(W_cat), _ptr(A_cat), _ptr(B_cat),
                                                 float(scale), _ptr(dX), _ptr(dA_cat), _ptr(dB_cat), _stream_ptr(stream)),
               "lora_linear_bwd_grouped")
        dAs, dBs = self.views(dA_cat, dB_cat)
        return dX, dAs, dBs
