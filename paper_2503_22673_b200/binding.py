"""ctypes binding of liblora_linear.so: argument marshalling only.

Every step of the layer runs in the CUDA kernels behind the C ABI (include/lora_linear.h); torch is
used for device memory and streams.  There is no fallback: if the library cannot be built or loaded,
or no sm_100 device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

from . import build as _build

LORA_OK = 0
LORA_ERR_INVALID_ARG = -1
LORA_ERR_UNSUPPORTED_SHAPE = -2
LORA_ERR_MISALIGNED = -3
LORA_ERR_WORKSPACE = -4
LORA_ERR_CUDA = -5
LORA_ERR_DEVICE_TIMEOUT = -6
LORA_ERR_NO_DEVICE = -7

EXPORTS = [
    "lora_select_config", "lora_workspace_bytes", "lora_plan_create", "lora_plan_destroy",
    "lora_plan_workspace_bytes", "lora_plan_set_workspace", "lora_plan_set_grad_accumulation", "lora_plan_get_config", "lora_plan_describe",
    "lora_linear_fwd", "lora_linear_bwd", "lora_linear_bwd_saved_p", "lora_linear_bwd_q", "lora_linear_bwd_dx", "lora_linear_bwd_da", "lora_linear_bwd_db",
    "lora_dense_dw", "lora_nf4_quantize", "lora_nf4_dequantize", "lora_linear_fwd_nf4", "lora_linear_bwd_nf4", "lora_step_host_staging_bytes", "lora_linear_step_host",
    "lora_last_device_status", "lora_strerror", "lora_launch_count",
    "lora_grad_contract_noalloc", "lora_grad_contract_noalloc_max_scratch", "lora_grad_contract_noalloc_status",
    "lora_plan_set_wait_limit", "lora_debug_starved_wait", "lora_linear_bwd_sides", "lora_linear_bwd_grads",
    "lora_plan_last_gemm_clock", "lora_plan_create_grouped", "lora_linear_fwd_grouped", "lora_linear_bwd_grouped",
    "lora_plan_nf4_scratch_bytes", "lora_plan_set_nf4_scratch_bytes",
]


class LoraShape(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int64), ("d_in", ctypes.c_int64), ("d_out", ctypes.c_int64), ("r", ctypes.c_int64)]


class LoraKernelConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "block_m", "fwd_block_n", "dx_block_n", "block_k", "stages", "group_m", "split_k", "r_pad", "fwd_ctas",
        "dx_ctas", "tail_delay", "grad_feat_chunk", "grad_stages", "da_feat_chunks", "da_token_chunks",
        "db_feat_chunks", "db_token_chunks", "db_feat_chunk", "cta_group", "dx_stages", "prefetch_dist", "db_stages", "q_feat_chunk", "q_feat_chunks", "q_token_chunks", "q_stages", "dx_split_k", "fwd_ext", "bwd_merged", "pair_feat_chunk", "pair_feat_chunks", "pair_token_chunks", "da_with_p", "dan_feat_chunk", "dan_feat_chunks", "dan_token_chunks", "dbq_feat_chunk", "dbq_feat_chunks", "dbq_token_chunks",
        "dw_block_n", "dw_split_k", "dw_ctas")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class LoraError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None


def load(rebuild: bool = False) -> ctypes.CDLL:
    """Load (building first if sources are newer) the CUDA library.  Raises if that is impossible."""
    global _lib
    if _lib is not None and not rebuild:
        return _lib
    path = _build.build(force=rebuild)
    lib = ctypes.CDLL(path)
    vp, i64 = ctypes.c_void_p, ctypes.c_int64
    sz_p = ctypes.POINTER(ctypes.c_size_t)
    lib.lora_select_config.argtypes = [ctypes.POINTER(LoraShape), ctypes.c_int, ctypes.POINTER(LoraKernelConfig)]
    lib.lora_workspace_bytes.argtypes = [ctypes.POINTER(LoraShape), ctypes.c_int, sz_p]
    lib.lora_plan_create.argtypes = [ctypes.POINTER(LoraShape), ctypes.c_int, ctypes.POINTER(vp)]
    lib.lora_plan_destroy.argtypes = [vp]
    lib.lora_plan_workspace_bytes.argtypes = [vp, sz_p, sz_p]
    lib.lora_plan_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    lib.lora_plan_set_grad_accumulation.argtypes = [vp, ctypes.c_int]
    lib.lora_plan_get_config.argtypes = [vp, ctypes.POINTER(LoraKernelConfig)]
    lib.lora_plan_describe.argtypes = [vp, ctypes.c_char_p, ctypes.c_size_t]
    lib.lora_linear_fwd.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, vp, vp]
    lib.lora_linear_bwd.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp]
    lib.lora_linear_bwd_saved_p.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp]
    lib.lora_linear_bwd_q.argtypes = [vp, vp, vp, ctypes.c_float, vp]
    lib.lora_linear_bwd_dx.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, vp, vp]
    lib.lora_linear_bwd_sides.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, vp]
    lib.lora_linear_bwd_grads.argtypes = [vp, vp, vp, vp, ctypes.c_float, vp, vp, vp]
    lib.lora_linear_bwd_da.argtypes = [vp, vp, vp, ctypes.c_float, vp, vp]
    lib.lora_linear_bwd_db.argtypes = [vp, vp, ctypes.c_float, vp, vp]
    lib.lora_dense_dw.argtypes = [vp, vp, vp, vp, vp]
    lib.lora_nf4_quantize.argtypes = [vp, i64, i64, vp, vp, vp]
    lib.lora_nf4_dequantize.argtypes = [vp, vp, i64, i64, vp, vp]
    lib.lora_linear_fwd_nf4.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp]
    lib.lora_linear_bwd_nf4.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp]
    lib.lora_step_host_staging_bytes.argtypes = [ctypes.POINTER(LoraShape), sz_p]
    lib.lora_linear_step_host.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp, vp,
                                          ctypes.c_size_t, vp]
    lib.lora_last_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int), ctypes.c_char_p, ctypes.c_size_t]
    lib.lora_strerror.argtypes = [ctypes.c_int]
    lib.lora_strerror.restype = ctypes.c_char_p
    lib.lora_launch_count.argtypes = []
    lib.lora_launch_count.restype = i64
    lib.lora_grad_contract_noalloc.argtypes = [vp, vp, i64, i64, i64, i64, vp, vp]
    lib.lora_grad_contract_noalloc_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int)]
    lib.lora_plan_create_grouped.argtypes = [vp, ctypes.c_int, ctypes.POINTER(vp)]
    lib.lora_linear_fwd_grouped.argtypes = [vp, vp, vp, vp, vp, ctypes.c_float, vp, vp]
    lib.lora_linear_bwd_grouped.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, vp, vp, vp]
    lib.lora_plan_set_wait_limit.argtypes = [vp, i64]
    lib.lora_plan_last_gemm_clock.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    lib.lora_debug_starved_wait.argtypes = [vp, vp, i64, i64, vp, vp]
    lib.lora_plan_nf4_scratch_bytes.argtypes = [vp, sz_p, sz_p]
    lib.lora_plan_set_nf4_scratch_bytes.argtypes = [vp, ctypes.c_size_t]
    lib.lora_grad_contract_noalloc_max_scratch.argtypes = []
    lib.lora_grad_contract_noalloc_max_scratch.restype = i64
    for name in EXPORTS:
        if name not in ("lora_strerror", "lora_launch_count", "lora_grad_contract_noalloc_max_scratch"):
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().lora_strerror(int(code)).decode()


def launch_count() -> int:
    return int(load().lora_launch_count())


def _check(code: int, where: str) -> None:
    if code != LORA_OK:
        raise LoraError(code, where)


def select_config(T: int, d_in: int, d_out: int, r: int, num_sms: int = 148) -> dict:
    """Run the host-side tile selector (needs no GPU)."""
    cfg = LoraKernelConfig()
    shape = LoraShape(T, d_in, d_out, r)
    _check(load().lora_select_config(ctypes.byref(shape), num_sms, ctypes.byref(cfg)), "lora_select_config")
    return cfg.as_dict()


def workspace_bytes(T: int, d_in: int, d_out: int, r: int, num_sms: int = 148) -> int:
    out = ctypes.c_size_t(0)
    shape = LoraShape(T, d_in, d_out, r)
    _check(load().lora_workspace_bytes(ctypes.byref(shape), num_sms, ctypes.byref(out)), "lora_workspace_bytes")
    return int(out.value)


def _ptr(t: Optional[torch.Tensor]) -> ctypes.c_void_p:
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> ctypes.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _want(t: torch.Tensor, name: str, shape: Tuple[int, ...], dtype: torch.dtype, device: torch.device) -> None:
    if tuple(t.shape) != tuple(shape) or t.dtype != dtype or not t.is_contiguous() or t.device != device:
        raise ValueError(f"{name}: want contiguous {dtype} {tuple(shape)} on {device}, got {t.dtype} "
                         f"{tuple(t.shape)} contiguous={t.is_contiguous()} on {t.device}")


class LoraLinearPlan:
    """A plan for one (T, d_in, d_out, r) shape on one device; owns its backward workspace tensor."""

    def __init__(self, T: int, d_in: int, d_out: int, r: int, device: int = 0):
        if not torch.cuda.is_available():
            raise LoraError(LORA_ERR_NO_DEVICE, "LoraLinearPlan")
        self._lib = load()
        self.T, self.d_in, self.d_out, self.r = int(T), int(d_in), int(d_out), int(r)
        self.device = torch.device("cuda", device)
        self._shape = LoraShape(self.T, self.d_in, self.d_out, self.r)
        self._h = ctypes.c_void_p(0)
        _check(self._lib.lora_plan_create(ctypes.byref(self._shape), device, ctypes.byref(self._h)), "lora_plan_create")
        bwd, fwd = ctypes.c_size_t(0), ctypes.c_size_t(0)
        _check(self._lib.lora_plan_workspace_bytes(self._h, ctypes.byref(fwd), ctypes.byref(bwd)),
               "lora_plan_workspace_bytes")
        self.workspace_bytes = int(bwd.value)
        self.fwd_workspace_bytes = int(fwd.value)
        self._ws = None

    # -- lifetime ------------------------------------------------------------------------------
    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.lora_plan_destroy(self._h)
            self._h = ctypes.c_void_p(0)
            self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- introspection -------------------------------------------------------------------------
    def config(self) -> dict:
        cfg = LoraKernelConfig()
        _check(self._lib.lora_plan_get_config(self._h, ctypes.byref(cfg)), "lora_plan_get_config")
        return cfg.as_dict()

    def describe(self) -> str:
        buf = ctypes.create_string_buffer(1024)
        _check(self._lib.lora_plan_describe(self._h, buf, 1024), "lora_plan_describe")
        return buf.value.decode()

    def device_status(self, stream: Optional[torch.cuda.Stream] = None) -> Tuple[int, str]:
        code = ctypes.c_int(0)
        buf = ctypes.create_string_buffer(256)
        _check(self._lib.lora_last_device_status(self._h, _stream_ptr(stream), ctypes.byref(code), buf, 256),
               "lora_last_device_status")
        return int(code.value), buf.value.decode()

    # -- workspace -----------------------------------------------------------------------------
    def ensure_workspace(self) -> None:
        if self._ws is None:
            self._ws = torch.empty(max(self.workspace_bytes, 256), dtype=torch.uint8, device=self.device)
            _check(self._lib.lora_plan_set_workspace(self._h, _ptr(self._ws), self._ws.numel()),
                   "lora_plan_set_workspace")

    def set_workspace(self, ws: Optional[torch.Tensor]) -> None:
        self._ws = ws
        n = 0 if ws is None else ws.numel() * ws.element_size()
        _check(self._lib.lora_plan_set_workspace(self._h, _ptr(ws), n), "lora_plan_set_workspace")

    def last_gemm_clock(self, stream=None) -> Tuple[float, float]:
        """(SM MHz, microseconds) of this plan's last CTA-pair GEMM launch, measured inside the kernel."""
        mhz, us = ctypes.c_double(0.0), ctypes.c_double(0.0)
        _check(self._lib.lora_plan_last_gemm_clock(self._h, _stream_ptr(stream), ctypes.byref(mhz), ctypes.byref(us)),
               "lora_plan_last_gemm_clock")
        return float(mhz.value), float(us.value)

    def set_wait_limit(self, cycles: int) -> None:
        """Limit of every device-side wait of this plan's later launches, in SM clock ticks (0: the default, ~2 s)."""
        _check(self._lib.lora_plan_set_wait_limit(self._h, int(cycles)), "lora_plan_set_wait_limit")

    def debug_starved_wait(self, S: torch.Tensor, out: torch.Tensor, stream=None) -> None:
        """Test hook: one CTA of the adapter-gradient kernel whose second factor never arrives (its wait runs out)."""
        T, C = S.shape
        _check(self._lib.lora_debug_starved_wait(self._h, _ptr(S), T, C, _ptr(out), _stream_ptr(stream)),
               "lora_debug_starved_wait")

    def set_grad_accumulation(self, enable: bool) -> None:
        """Backward calls add dA / dB to the given buffers instead of overwriting them (micro-batch accumulation)."""
        _check(self._lib.lora_plan_set_grad_accumulation(self._h, 1 if enable else 0), "lora_plan_set_grad_accumulation")

    # -- the two calls -------------------------------------------------------------------------
    def fwd(self, X, W, A, B, scale: float, Y: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """Y = X W^T + scale (X A^T) B^T."""
        bf = torch.bfloat16
        _want(X, "X", (self.T, self.d_in), bf, self.device)
        _want(W, "W", (self.d_out, self.d_in), bf, self.device)
        _want(A, "A", (self.r, self.d_in), bf, self.device)
        _want(B, "B", (self.d_out, self.r), bf, self.device)
        if Y is None:
            Y = torch.empty((self.T, self.d_out), dtype=bf, device=self.device)
        _want(Y, "Y", (self.T, self.d_out), bf, self.device)
        if self.fwd_workspace_bytes:
            self.ensure_workspace()
        _check(self._lib.lora_linear_fwd(self._h, _ptr(X), _ptr(W), _ptr(A), _ptr(B), float(scale), _ptr(Y),
                                         _stream_ptr(stream)), "lora_linear_fwd")
        return Y

    def bwd(self, dY, X, W, A, B, scale: float, dX=None, dA=None, dB=None, stream=None, saved_p: bool = False):
        """(dX, dA, dB) = (dY W + scale (dY B) A,  scale (dY B)^T X,  scale dY^T (X A^T)).

        ``saved_p=True`` reuses X A^T from the preceding ``fwd`` on this plan (same X, A, scale; the workspace must
        have been registered before that forward: call ``ensure_workspace()`` first)."""
        bf = torch.bfloat16
        _want(dY, "dY", (self.T, self.d_out), bf, self.device)
        _want(X, "X", (self.T, self.d_in), bf, self.device)
        _want(W, "W", (self.d_out, self.d_in), bf, self.device)
        _want(A, "A", (self.r, self.d_in), bf, self.device)
        _want(B, "B", (self.d_out, self.r), bf, self.device)
        if dX is None:
            dX = torch.empty((self.T, self.d_in), dtype=bf, device=self.device)
        if dA is None:
            dA = torch.empty((self.r, self.d_in), dtype=torch.float32, device=self.device)
        if dB is None:
            dB = torch.empty((self.d_out, self.r), dtype=torch.float32, device=self.device)
        _want(dX, "dX", (self.T, self.d_in), bf, self.device)
        _want(dA, "dA", (self.r, self.d_in), torch.float32, self.device)
        _want(dB, "dB", (self.d_out, self.r), torch.float32, self.device)
        self.ensure_workspace()
        fn = self._lib.lora_linear_bwd_saved_p if saved_p else self._lib.lora_linear_bwd
        _check(fn(self._h, _ptr(dY), _ptr(X), _ptr(W), _ptr(A), _ptr(B), float(scale),
                  _ptr(dX), _ptr(dA), _ptr(dB), _stream_ptr(stream)), "lora_linear_bwd")
        return dX, dA, dB

    # -- NF4 frozen weight (Q+LoRA) ---------------------------------------------------------------
    def nf4_scratch_bytes(self) -> Tuple[int, int]:
        """(smallest scratch buffer the banded Q+LoRA form accepts, size of the whole bf16 weight), in bytes."""
        lo, full = ctypes.c_size_t(0), ctypes.c_size_t(0)
        _check(self._lib.lora_plan_nf4_scratch_bytes(self._h, ctypes.byref(lo), ctypes.byref(full)), "lora_plan_nf4_scratch_bytes")
        return int(lo.value), int(full.value)

    def _scratch_ptr(self, w_scratch):
        """Pointer of the scratch buffer; its size is announced to the plan (a buffer smaller than the weight selects the
        banded form: any contiguous bf16 tensor of at least nf4_scratch_bytes()[0] bytes)."""
        if w_scratch is None:
            return ctypes.c_void_p(0)
        if w_scratch.dtype != torch.bfloat16 or w_scratch.device != self.device or not w_scratch.is_contiguous():
            raise ValueError("w_scratch: want a contiguous bf16 tensor on the plan's device")
        _check(self._lib.lora_plan_set_nf4_scratch_bytes(self._h, w_scratch.numel() * 2), "lora_plan_set_nf4_scratch_bytes")
        return _ptr(w_scratch)

    def fwd_nf4(self, X, W_codes, W_absmax, A, B, scale: float, Y: Optional[torch.Tensor] = None, w_scratch=None, stream=None):
        """Y = X w_hat^T + scale (X A^T) B^T with w_hat = the NF4 weight (codes [d_out, d_in/2] uint8, absmax [d_in/64, d_out] fp32).

        ``w_scratch`` ([d_out, d_in] bf16, reusable across layers): expand the weight once and run the bf16 kernels (fast
        form); a smaller bf16 buffer (see ``nf4_scratch_bytes``): the same band by band; None: expand inside the GEMM
        kernels (no extra memory, slower for large batches)."""
        bf = torch.bfloat16
        _want(X, "X", (self.T, self.d_in), bf, self.device)
        _want(W_codes, "W_codes", (self.d_out, self.d_in // 2), torch.uint8, self.device)
        _want(W_absmax, "W_absmax", (self.d_in // 64, self.d_out), torch.float32, self.device)
        _want(A, "A", (self.r, self.d_in), bf, self.device)
        _want(B, "B", (self.d_out, self.r), bf, self.device)
        if Y is None:
            Y = torch.empty((self.T, self.d_out), dtype=bf, device=self.device)
        _want(Y, "Y", (self.T, self.d_out), bf, self.device)
        self.ensure_workspace()
        _check(self._lib.lora_linear_fwd_nf4(self._h, _ptr(X), _ptr(W_codes), _ptr(W_absmax), _ptr(A), _ptr(B), float(scale),
                                             _ptr(Y), self._scratch_ptr(w_scratch), _stream_ptr(stream)), "lora_linear_fwd_nf4")
        return Y

    def bwd_nf4(self, dY, X, W_codes, W_absmax, A, B, scale: float, dX=None, dA=None, dB=None, w_scratch=None, stream=None):
        """(dX, dA, dB) of the layer with the NF4 weight."""
        bf = torch.bfloat16
        _want(dY, "dY", (self.T, self.d_out), bf, self.device)
        _want(X, "X", (self.T, self.d_in), bf, self.device)
        _want(W_codes, "W_codes", (self.d_out, self.d_in // 2), torch.uint8, self.device)
        _want(W_absmax, "W_absmax", (self.d_in // 64, self.d_out), torch.float32, self.device)
        _want(A, "A", (self.r, self.d_in), bf, self.device)
        _want(B, "B", (self.d_out, self.r), bf, self.device)
        if dX is None:
            dX = torch.empty((self.T, self.d_in), dtype=bf, device=self.device)
        if dA is None:
            dA = torch.empty((self.r, self.d_in), dtype=torch.float32, device=self.device)
        if dB is None:
            dB = torch.empty((self.d_out, self.r), dtype=torch.float32, device=self.device)
        _want(dX, "dX", (self.T, self.d_in), bf, self.device)
        _want(dA, "dA", (self.r, self.d_in), torch.float32, self.device)
        _want(dB, "dB", (self.d_out, self.r), torch.float32, self.device)
        self.ensure_workspace()
        _check(self._lib.lora_linear_bwd_nf4(self._h, _ptr(dY), _ptr(X), _ptr(W_codes), _ptr(W_absmax), _ptr(A), _ptr(B),
                                             float(scale), _ptr(dX), _ptr(dA), _ptr(dB), self._scratch_ptr(w_scratch),
                                             _stream_ptr(stream)),
               "lora_linear_bwd_nf4")
        return dX, dA, dB

    def dense_dw(self, dY, X, dW: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """dW = dY^T X, the weight gradient of full fine-tuning ([d_out, d_in] bf16)."""
        bf = torch.bfloat16
        _want(dY, "dY", (self.T, self.d_out), bf, self.device)
        _want(X, "X", (self.T, self.d_in), bf, self.device)
        if dW is None:
            dW = torch.empty((self.d_out, self.d_in), dtype=bf, device=self.device)
        _want(dW, "dW", (self.d_out, self.d_in), bf, self.device)
        if self.config()["dw_split_k"] > 1:
            self.ensure_workspace()
        _check(self._lib.lora_dense_dw(self._h, _ptr(dY), _ptr(X), _ptr(dW), _stream_ptr(stream)), "lora_dense_dw")
        return dW

    def bwd_q(self, dY, B, scale: float, stream=None) -> None:
        """Stage scale (dY B)^T in the workspace; the next ``bwd_dx`` then launches the dX GEMM alone."""
        self.ensure_workspace()
        _check(self._lib.lora_linear_bwd_q(self._h, _ptr(dY), _ptr(B), float(scale), _stream_ptr(stream)), "lora_linear_bwd_q")

    def bwd_dx(self, dY, W, A, B, scale: float, dX, stream=None):
        """dX = dY W + scale (dY B) A alone (first stage of the backward pass)."""
        self.ensure_workspace()
        _check(self._lib.lora_linear_bwd_dx(self._h, _ptr(dY), _ptr(W), _ptr(A), _ptr(B), float(scale), _ptr(dX),
                                            _stream_ptr(stream)), "lora_linear_bwd_dx")
        return dX

    def bwd_stage_names(self) -> Tuple[str, ...]:
        """The launches ``bwd`` issues on this plan, in order (see ``bwd_stages``)."""
        return ("sides", "dx_gemm", "grads") if self.config()["bwd_merged"] else ("q_prepass", "dx_gemm", "dA", "dB")

    def bwd_stages(self, dY, X, W, A, B, scale: float, dX, dA, dB, stream=None, events=None):
        """The same kernels as ``bwd``, issued through the stage entry points.  Merged form: dY B and X A^T in one launch,
        the dX GEMM, dA and dB in one launch; split form: dY B pre-pass, dX GEMM, dA stage, dB.  ``events`` (one
        torch.cuda.Event more than there are stages, optional) are recorded on the stream before the first stage and
        after every stage, so that events k and k + 1 bracket exactly stage k of ``bwd_stage_names()``."""
        self.ensure_workspace()
        sp = _stream_ptr(stream)
        st = stream if stream is not None else torch.cuda.current_stream()
        lib, h, s = self._lib, self._h, float(scale)

        def mark(k):
            if events is not None:
                events[k].record(st)

        mark(0)
        if self.config()["bwd_merged"]:
            _check(lib.lora_linear_bwd_sides(h, _ptr(dY), _ptr(X), _ptr(A), _ptr(B), s, sp), "lora_linear_bwd_sides")
            mark(1)
            _check(lib.lora_linear_bwd_dx(h, _ptr(dY), _ptr(W), _ptr(A), _ptr(B), s, _ptr(dX), sp), "lora_linear_bwd_dx")
            mark(2)
            _check(lib.lora_linear_bwd_grads(h, _ptr(dY), _ptr(X), _ptr(A), s, _ptr(dA), _ptr(dB), sp), "lora_linear_bwd_grads")
            mark(3)
        else:
            _check(lib.lora_linear_bwd_q(h, _ptr(dY), _ptr(B), s, sp), "lora_linear_bwd_q")
            mark(1)
            _check(lib.lora_linear_bwd_dx(h, _ptr(dY), _ptr(W), _ptr(A), _ptr(B), s, _ptr(dX), sp), "lora_linear_bwd_dx")
            mark(2)
            _check(lib.lora_linear_bwd_da(h, _ptr(X), _ptr(A), s, _ptr(dA), sp), "lora_linear_bwd_da")
            mark(3)
            _check(lib.lora_linear_bwd_db(h, _ptr(dY), s, _ptr(dB), sp), "lora_linear_bwd_db")
            mark(4)
        return dX, dA, dB

    # -- host-buffer step (end-to-end measurement and host callers) ------------------------------
    def step_host_staging_bytes(self) -> int:
        out = ctypes.c_size_t(0)
        _check(self._lib.lora_step_host_staging_bytes(ctypes.byref(self._shape), ctypes.byref(out)),
               "lora_step_host_staging_bytes")
        return int(out.value)

    def step_host(self, hX, W, hA, hB, hdY, scale: float, hY, hdX, hdA, hdB, staging: torch.Tensor, stream=None):
        """fwd + bwd with host tensors for everything except the frozen W (device)."""
        self.ensure_workspace()
        for t in (hX, hA, hB, hdY, hY, hdX, hdA, hdB):
            if t.device.type != "cpu" or not t.is_contiguous():
                raise ValueError("step_host wants contiguous CPU tensors")
        _check(self._lib.lora_linear_step_host(
            self._h, _ptr(hX), _ptr(W), _ptr(hA), _ptr(hB), _ptr(hdY), float(scale), _ptr(hY), _ptr(hdX), _ptr(hdA),
            _ptr(hdB), _ptr(staging), staging.numel() * staging.element_size(), _stream_ptr(stream)),
            "lora_linear_step_host")


def lora_linear_fwd(plan: LoraLinearPlan, X, W, A, B, scale, Y=None, stream=None):
    return plan.fwd(X, W, A, B, scale, Y, stream)


def lora_linear_bwd(plan: LoraLinearPlan, dY, X, W, A, B, scale, dX=None, dA=None, dB=None, stream=None):
    return plan.bwd(dY, X, W, A, B, scale, dX, dA, dB, stream)


def grad_contract_noalloc(S: torch.Tensor, Rt: torch.Tensor, out: torch.Tensor, stream=None) -> torch.Tensor:
    """out[c, j] = sum_t S[t, c] * Rt[j, t] through the entry point that allocates nothing.

    For callers that may not allocate device memory at call time (fixed memory pools, latency-critical
    loops): the kernel's scratch is a static device array inside the library, so the caller passes only
    the inputs S [T, C] bf16, Rt [r, ld] bf16 (ld >= T) and the output out [C, r] fp32.  Calls share that
    array, so do not let two of them overlap on the GPU.
    """
    T, C = S.shape
    r, ld = Rt.shape
    if S.dtype != torch.bfloat16 or Rt.dtype != torch.bfloat16 or out.dtype != torch.float32:
        raise ValueError("grad_contract_noalloc: S, Rt bf16 and out fp32 expected")
    if not (S.is_contiguous() and Rt.is_contiguous() and out.is_contiguous()) or tuple(out.shape) != (C, r):
        raise ValueError("grad_contract_noalloc: contiguous S [T,C], Rt [r,ld], out [C,r] expected")
    _check(load().lora_grad_contract_noalloc(_ptr(S), _ptr(Rt), T, C, r, ld, _ptr(out), _stream_ptr(stream)),
           "lora_grad_contract_noalloc")
    return out


def grad_contract_noalloc_status(stream=None) -> int:
    """LORA_OK, or LORA_ERR_DEVICE_TIMEOUT when a bounded wait of an allocation-free call ran out (synchronises the stream)."""
    code = ctypes.c_int(0)
    _check(load().lora_grad_contract_noalloc_status(_stream_ptr(stream), ctypes.byref(code)), "lora_grad_contract_noalloc_status")
    return int(code.value)


def nf4_quantize(W: torch.Tensor, stream=None):
    """(codes [d_out, d_in/2] uint8, absmax [d_in/64, d_out] fp32) of a bf16 device weight, in this library's NF4 layout."""
    if W.dtype != torch.bfloat16 or not W.is_contiguous() or W.dim() != 2 or not W.is_cuda:
        raise ValueError("nf4_quantize: contiguous bf16 CUDA matrix expected")
    d_out, d_in = W.shape
    codes = torch.empty((d_out, d_in // 2), dtype=torch.uint8, device=W.device)
    absmax = torch.empty((d_in // 64, d_out), dtype=torch.float32, device=W.device)
    _check(load().lora_nf4_quantize(_ptr(W), d_out, d_in, _ptr(codes), _ptr(absmax), _stream_ptr(stream)), "lora_nf4_quantize")
    return codes, absmax


def nf4_dequantize(codes: torch.Tensor, absmax: torch.Tensor, W: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """bf16 weight [d_out, d_in] from NF4 codes and block scales: every element bf16(level * absmax)."""
    d_out, half = codes.shape
    d_in = half * 2
    if codes.dtype != torch.uint8 or absmax.dtype != torch.float32 or tuple(absmax.shape) != (d_in // 64, d_out):
        raise ValueError("nf4_dequantize: codes [d_out, d_in/2] uint8 and absmax [d_in/64, d_out] fp32 expected")
    if W is None:
        W = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=codes.device)
    _check(load().lora_nf4_dequantize(_ptr(codes), _ptr(absmax), d_out, d_in, _ptr(W), _stream_ptr(stream)), "lora_nf4_dequantize")
    return W
