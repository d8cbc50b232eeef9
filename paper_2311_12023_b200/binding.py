"""Thin Python binding of the C ABI declared in ``include/lqlora.h``.

Argument marshalling only: every step of the path runs in the CUDA library.  torch is
used for device memory and streams.  There is no fallback: if ``liblqlora.so`` is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblqlora.so")

EXPORTS = [
    "lqlora_storage_bits_per_param", "lqlora_packed_sizes", "lqlora_nf_codebook", "lqlora_encode",
    "lqlora_unpack", "lqlora_dequant", "lqlora_linear_workspace_bytes", "lqlora_linear_fwd",
    "lqlora_linear_bwd_input", "lqlora_workspace_status", "lqlora_linear_path", "lqlora_launch_count",
    "lqlora_status_string", "lqlora_encode_host", "lqlora_linear_fwd_host", "lqlora_linear_bwd_input_host",
    "lqlora_static_scratch_bytes", "lqlora_linear_fwd_static", "lqlora_static_scratch_status",
    "lqlora_encode_search_clearance",
    "lqlora_lora_grads_workspace_bytes", "lqlora_lora_grads",
    "lqlora_lq_workspace_bytes", "lqlora_lq_decompose", "lqlora_to_bf16", "lqlora_assign_configs",
    "lqlora_unpack_scales", "lqlora_linear_qfactors_workspace_bytes", "lqlora_linear_fwd_qfactors",
    "lqlora_linear_bwd_input_qfactors", "lqlora_selftest_bounded_wait",
]

STATIC_SCRATCH_BYTES = 8 << 20   # size of the scratch array compiled into the library (lqlora_static_scratch_bytes)


class LqloraError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class CConfig(ctypes.Structure):
    _fields_ = [("b0", ctypes.c_int), ("B0", ctypes.c_int), ("b1", ctypes.c_int), ("B1", ctypes.c_int),
                ("b2", ctypes.c_int)]


class CQMatrix(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scale_codes", ctypes.c_void_p), ("scale2", ctypes.c_void_p),
                ("N", ctypes.c_int64), ("K", ctypes.c_int64), ("cfg", CConfig)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the compiled library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2311_12023_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, ci, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
        L.lqlora_storage_bits_per_param.argtypes = [ctypes.POINTER(CConfig)]
        L.lqlora_storage_bits_per_param.restype = ctypes.c_double
        L.lqlora_packed_sizes.argtypes = [i64, i64, ctypes.POINTER(CConfig)] + [ctypes.POINTER(sz)] * 4
        L.lqlora_nf_codebook.argtypes = [ci, vp]
        L.lqlora_encode.argtypes = [vp, ctypes.POINTER(CQMatrix), vp, sz, vp]
        L.lqlora_unpack.argtypes = [ctypes.POINTER(CQMatrix), vp, vp]
        L.lqlora_dequant.argtypes = [ctypes.POINTER(CQMatrix), vp, vp, vp]
        L.lqlora_linear_workspace_bytes.argtypes = [i64, i64, ctypes.POINTER(CConfig), ci, i64, ctypes.POINTER(sz)]
        L.lqlora_linear_fwd.argtypes = [ctypes.POINTER(CQMatrix), vp, vp, ci, vp, i64, vp, vp, sz, vp]
        L.lqlora_linear_bwd_input.argtypes = [ctypes.POINTER(CQMatrix), vp, vp, ci, vp, i64, vp, vp, sz, vp]
        L.lqlora_lora_grads_workspace_bytes.argtypes = [i64, i64, ci, i64, ctypes.POINTER(sz)]
        L.lqlora_lora_grads.argtypes = [vp, vp, ci, i64, i64, vp, vp, i64, vp, vp, vp, sz, vp]
        L.lqlora_linear_intermediate_offset.argtypes = [i64, i64, ctypes.POINTER(CConfig), ci, i64, ci, ctypes.POINTER(sz)]
        L.lqlora_lora_grads_from.argtypes = [vp, vp, ci, i64, i64, vp, vp, i64, vp, vp, vp, sz, vp]
        L.lqlora_encode_host.argtypes = [vp, vp, ctypes.POINTER(CQMatrix), vp, sz, vp]
        L.lqlora_linear_fwd_host.argtypes = [ctypes.POINTER(CQMatrix), vp, vp, ci, vp, i64, vp, vp, vp, vp, sz, vp]
        L.lqlora_linear_bwd_input_host.argtypes = [ctypes.POINTER(CQMatrix), vp, vp, ci, vp, i64, vp, vp, vp, vp, sz, vp]
        L.lqlora_workspace_status.argtypes = [vp, vp]
        L.lqlora_static_scratch_bytes.restype = sz
        L.lqlora_encode_search_clearance.argtypes = [ci]
        L.lqlora_encode_search_clearance.restype = ctypes.c_double
        L.lqlora_linear_fwd_static.argtypes = [ctypes.POINTER(CQMatrix), vp, vp, ci, vp, i64, vp, vp]
        L.lqlora_static_scratch_status.argtypes = [vp]
        L.lqlora_selftest_bounded_wait.argtypes = [vp, i64, vp]
        L.lqlora_unpack_scales.argtypes = [ctypes.POINTER(CQMatrix), vp, vp, vp]
        L.lqlora_linear_qfactors_workspace_bytes.argtypes = [i64, i64, ctypes.POINTER(CConfig), ci, i64, ctypes.POINTER(sz)]
        L.lqlora_linear_fwd_qfactors.argtypes = [ctypes.POINTER(CQMatrix)] * 3 + [vp, i64, vp, vp, sz, vp]
        L.lqlora_linear_bwd_input_qfactors.argtypes = [ctypes.POINTER(CQMatrix)] * 3 + [vp, i64, vp, vp, sz, vp]
        L.lqlora_lq_workspace_bytes.argtypes = [i64, i64, ctypes.POINTER(CConfig), ci, ci, ctypes.POINTER(sz)]
        L.lqlora_lq_decompose.argtypes = [vp, vp, ctypes.POINTER(CQMatrix), vp, vp, ci, ci, vp, ci, ci, vp, ctypes.POINTER(ci), vp, sz, vp]
        L.lqlora_to_bf16.argtypes = [vp, vp, i64, vp]
        L.lqlora_assign_configs.argtypes = [vp, vp, ci, ci, ctypes.c_double, vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
        L.lqlora_linear_path.argtypes = [i64, i64, ctypes.POINTER(CConfig), ci, i64, ci, ctypes.POINTER(ci)]
        L.lqlora_launch_count.restype = i64
        L.lqlora_status_string.argtypes = [ci]
        L.lqlora_status_string.restype = ctypes.c_char_p
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().lqlora_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise LqloraError(status, where)


def _cfg(cfg) -> CConfig:
    """cfg: anything with b0, B0, b1, B1, b2 attributes (e.g. inputs.QuantConfig)."""
    return CConfig(int(cfg.b0), int(cfg.B0), int(cfg.b1), int(cfg.B1), int(cfg.b2))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


# ----------------------------------------------------------------------------- host-only calls
def storage_bits_per_param(cfg) -> float:
    c = _cfg(cfg)
    return float(lib().lqlora_storage_bits_per_param(ctypes.byref(c)))


def packed_sizes(N: int, K: int, cfg) -> Tuple[int, int, int, int]:
    """(code_bytes, scale_bytes, scale2_bytes, encode_workspace_bytes)."""
    c = _cfg(cfg)
    out = [ctypes.c_size_t(0) for _ in range(4)]
    _check(lib().lqlora_packed_sizes(N, K, ctypes.byref(c), *[ctypes.byref(o) for o in out]), "lqlora_packed_sizes")
    return tuple(int(o.value) for o in out)


def nf_codebook(b0: int) -> np.ndarray:
    out = np.zeros(1 << b0, dtype=np.float32)
    _check(lib().lqlora_nf_codebook(b0, out.ctypes.data_as(ctypes.c_void_p)), "lqlora_nf_codebook")
    return out


def linear_workspace_bytes(N: int, K: int, cfg, r: int, M: int) -> int:
    c = _cfg(cfg)
    out = ctypes.c_size_t(0)
    _check(lib().lqlora_linear_workspace_bytes(N, K, ctypes.byref(c), r, M, ctypes.byref(out)),
           "lqlora_linear_workspace_bytes")
    return int(out.value)


PATH_PLAIN, PATH_STREAM, PATH_TC_ONE, PATH_TC_PAIR = 0, 1, 2, 3


def linear_route(N: int, K: int, cfg, r: int, M: int, backward: bool) -> Tuple[int, int]:
    """lqlora_linear_path: (kernel id, CTAs sharing one output tile's contraction) of the dispatch for M rows."""
    c = _cfg(cfg)
    splits = ctypes.c_int(0)
    kernel = int(lib().lqlora_linear_path(N, K, ctypes.byref(c), r, M, int(backward), ctypes.byref(splits)))
    if kernel < 0:
        raise LqloraError(kernel, "lqlora_linear_path")
    return kernel, int(splits.value)


def linear_path(N: int, K: int, cfg, r: int, M: int, backward: bool) -> int:
    return linear_route(N, K, cfg, r, M, backward)[0]


def launch_count() -> int:
    return int(lib().lqlora_launch_count())


# ----------------------------------------------------------------------------- device calls
@dataclass
class QMatrix:
    """Device arrays of one quantized matrix (owned here, as torch tensors)."""
    codes: torch.Tensor        # uint8 buffer holding the packed code words
    scale_codes: torch.Tensor  # uint8: one code per byte (b1 = 8) or the packed bit stream (b1 < 8)
    scale2: torch.Tensor       # float32 [ngrp] (b2 = fp32) or a byte buffer holding fp16 / bf16 numbers
    N: int
    K: int
    cfg: object

    def cstruct(self) -> CQMatrix:
        return CQMatrix(self.codes.data_ptr(), self.scale_codes.data_ptr(), self.scale2.data_ptr(),
                        self.N, self.K, _cfg(self.cfg))

    @property
    def packed_bytes(self) -> int:
        return self.codes.numel() + self.scale_codes.numel() + self.scale2.numel() * self.scale2.element_size()


def alloc_qmatrix(N: int, K: int, cfg, device="cuda") -> QMatrix:
    cb, sb, s2b, _ = packed_sizes(N, K, cfg)
    if int(cfg.b2) == 32:
        s2 = torch.empty(s2b // 4, dtype=torch.float32, device=device)
    else:
        s2 = torch.zeros((s2b + 15) // 16 * 16, dtype=torch.uint8, device=device)
    return QMatrix(torch.empty(cb, dtype=torch.uint8, device=device),
                   torch.zeros((sb + 15) // 16 * 16, dtype=torch.uint8, device=device) if int(cfg.b1) != 8 else
                   torch.empty(sb, dtype=torch.uint8, device=device), s2, N, K, cfg)


def encode(W: torch.Tensor, cfg, out: Optional[QMatrix] = None, workspace: Optional[torch.Tensor] = None) -> QMatrix:
    """lqlora_encode: W fp32 [N, K] on the device -> packed codes, scale codes, second-level scales."""
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous() and W.dim() == 2
    N, K = W.shape
    q = out if out is not None else alloc_qmatrix(N, K, cfg, W.device)
    ws_bytes = packed_sizes(N, K, cfg)[3]
    if workspace is None:
        workspace = torch.empty(max(ws_bytes, 16), dtype=torch.uint8, device=W.device)
    cs = q.cstruct()
    _check(lib().lqlora_encode(W.data_ptr(), ctypes.byref(cs), workspace.data_ptr(), workspace.numel(), _stream()),
           "lqlora_encode")
    return q


def unpack(q: QMatrix) -> torch.Tensor:
    out = torch.empty((q.N, q.K), dtype=torch.uint8, device=q.codes.device)
    cs = q.cstruct()
    _check(lib().lqlora_unpack(ctypes.byref(cs), out.data_ptr(), _stream()), "lqlora_unpack")
    return out


def dequant(q: QMatrix, want32: bool = True, want16: bool = True):
    dev = q.codes.device
    d32 = torch.empty((q.N, q.K), dtype=torch.float32, device=dev) if want32 else None
    d16 = torch.empty((q.N, q.K), dtype=torch.bfloat16, device=dev) if want16 else None
    cs = q.cstruct()
    _check(lib().lqlora_dequant(ctypes.byref(cs), _ptr(d32), _ptr(d16), _stream()), "lqlora_dequant")
    return d32, d16


def unpack_scales(q: QMatrix):
    """lqlora_unpack_scales: (scale codes uint8 [nblk], second-level scales fp32 [ngrp]) in plain form."""
    nblk = q.N * q.K // q.cfg.B0
    ngrp = (nblk + q.cfg.B1 - 1) // q.cfg.B1
    sc = torch.empty(nblk, dtype=torch.uint8, device=q.codes.device)
    v = torch.empty(ngrp, dtype=torch.float32, device=q.codes.device)
    cs = q.cstruct()
    _check(lib().lqlora_unpack_scales(ctypes.byref(cs), sc.data_ptr(), v.data_ptr(), _stream()), "lqlora_unpack_scales")
    return sc, v


def linear_qfactors(q: QMatrix, qL1: QMatrix, qL2: QMatrix, A: torch.Tensor, backward: bool = False) -> torch.Tensor:
    """lqlora_linear_fwd_qfactors / lqlora_linear_bwd_input_qfactors: the layer with quantized (NF-8) factors."""
    assert A.is_cuda and A.dtype == torch.bfloat16 and A.is_contiguous() and A.dim() == 2
    M, r = A.shape[0], qL1.K
    c = _cfg(q.cfg)
    need = ctypes.c_size_t(0)
    _check(lib().lqlora_linear_qfactors_workspace_bytes(q.N, q.K, ctypes.byref(c), r, M, ctypes.byref(need)), "qfactors workspace")
    ws = torch.empty(int(need.value), dtype=torch.uint8, device=A.device)
    out = torch.empty((M, q.K if backward else q.N), dtype=torch.bfloat16, device=A.device)
    fn = lib().lqlora_linear_bwd_input_qfactors if backward else lib().lqlora_linear_fwd_qfactors
    a, b, cc = q.cstruct(), qL1.cstruct(), qL2.cstruct()
    _check(fn(ctypes.byref(a), ctypes.byref(b), ctypes.byref(cc), A.data_ptr(), M, out.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "lqlora_linear_qfactors")
    return out


def alloc_workspace(q: QMatrix, r: int, M: int) -> torch.Tensor:
    return torch.empty(linear_workspace_bytes(q.N, q.K, q.cfg, r, M), dtype=torch.uint8, device=q.codes.device)


def _linear(fn, name, q, L1, L2, A, out_cols, out, workspace):
    assert A.is_cuda and A.dtype == torch.bfloat16 and A.is_contiguous() and A.dim() == 2
    M = A.shape[0]
    r = 0 if L1 is None else L1.shape[1]
    if r:
        assert L1.dtype == torch.bfloat16 and L2.dtype == torch.bfloat16 and L1.is_contiguous() and L2.is_contiguous()
        assert tuple(L1.shape) == (q.N, r) and tuple(L2.shape) == (r, q.K)
    if out is None:
        out = torch.empty((M, out_cols), dtype=torch.bfloat16, device=A.device)
    if workspace is None:
        workspace = alloc_workspace(q, r, M)
    cs = q.cstruct()
    _check(fn(ctypes.byref(cs), _ptr(L1), _ptr(L2), r, A.data_ptr(), M, out.data_ptr(), workspace.data_ptr(),
              workspace.numel(), _stream()), name)
    return out


def linear_fwd(q: QMatrix, L1, L2, X: torch.Tensor, out=None, workspace=None) -> torch.Tensor:
    """lqlora_linear_fwd: Y = X deq(Q)^T + (X L2^T) L1^T, bf16 [M, N]."""
    assert X.shape[1] == q.K
    return _linear(lib().lqlora_linear_fwd, "lqlora_linear_fwd", q, L1, L2, X, q.N, out, workspace)


def linear_fwd_static(q: QMatrix, L1, L2, X: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """lqlora_linear_fwd_static: the forward pass with the library's built-in scratch array.

    For callers that must not allocate device memory while they run (a server with a fixed memory
    pool, code inside another framework's hook): pass ``out`` and this wrapper allocates nothing
    either.  Same result as ``linear_fwd``; problems that need more than ``STATIC_SCRATCH_BYTES`` of
    scratch raise ``LqloraError`` (workspace too small).  Calls share one array, so they must not
    overlap on the GPU.
    """
    assert X.is_cuda and X.dtype == torch.bfloat16 and X.is_contiguous() and X.dim() == 2 and X.shape[1] == q.K
    M = X.shape[0]
    r = 0 if L1 is None else L1.shape[1]
    if r:
        assert L1.dtype == torch.bfloat16 and L2.dtype == torch.bfloat16 and L1.is_contiguous() and L2.is_contiguous()
        assert tuple(L1.shape) == (q.N, r) and tuple(L2.shape) == (r, q.K)
    if out is None:
        out = torch.empty((M, q.N), dtype=torch.bfloat16, device=X.device)
    cs = q.cstruct()
    _check(lib().lqlora_linear_fwd_static(ctypes.byref(cs), _ptr(L1), _ptr(L2), r, X.data_ptr(), M, out.data_ptr(),
                                          _stream()), "lqlora_linear_fwd_static")
    return out


def linear_bwd_input(q: QMatrix, L1, L2, dY: torch.Tensor, out=None, workspace=None) -> torch.Tensor:
    """lqlora_linear_bwd_input: dX = dY deq(Q) + (dY L1) L2, bf16 [M, K]."""
    assert dY.shape[1] == q.N
    return _linear(lib().lqlora_linear_bwd_input, "lqlora_linear_bwd_input", q, L1, L2, dY, q.K, out, workspace)


def lora_grads_workspace_bytes(N: int, K: int, r: int, M: int) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().lqlora_lora_grads_workspace_bytes(N, K, r, M, ctypes.byref(n)), "lqlora_lora_grads_workspace_bytes")
    return int(n.value)


def lora_grads(L1: torch.Tensor, L2: torch.Tensor, X: torch.Tensor, dY: torch.Tensor, out=None, workspace=None):
    """lqlora_lora_grads: (dL1 [N, r], dL2 [r, K]) in fp32 from bf16 L1 [N, r], L2 [r, K], X [M, K], dY [M, N]."""
    N, r = L1.shape
    K = L2.shape[1]
    M = X.shape[0]
    assert L2.shape[0] == r and X.shape[1] == K and tuple(dY.shape) == (M, N)
    for t in (L1, L2, X, dY):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
    if out is None:
        out = (torch.empty(N, r, dtype=torch.float32, device=X.device), torch.empty(r, K, dtype=torch.float32, device=X.device))
    if workspace is None:
        workspace = torch.empty(lora_grads_workspace_bytes(N, K, r, M), dtype=torch.uint8, device=X.device)
    _check(lib().lqlora_lora_grads(L1.data_ptr(), L2.data_ptr(), r, N, K, X.data_ptr(), dY.data_ptr(), M, out[0].data_ptr(),
                                   out[1].data_ptr(), workspace.data_ptr(), workspace.numel(), _stream()), "lqlora_lora_grads")
    return out


def linear_intermediate(workspace: torch.Tensor, N: int, K: int, cfg, r: int, M: int, backward: bool) -> torch.Tensor:
    """View of the bf16 [M, r] intermediate (X L2^T or dY L1) that the last linear call left in `workspace`
    (lqlora_linear_intermediate_offset)."""
    off = ctypes.c_size_t(0)
    c = _cfg(cfg)
    _check(lib().lqlora_linear_intermediate_offset(N, K, ctypes.byref(c), r, M, 1 if backward else 0, ctypes.byref(off)),
           "lqlora_linear_intermediate_offset")
    return workspace[off.value:off.value + M * r * 2].view(torch.bfloat16).view(M, r)


def lora_grads_from(T: torch.Tensor, Tp: torch.Tensor, N: int, K: int, X: torch.Tensor, dY: torch.Tensor, out=None, workspace=None):
    """lqlora_lora_grads_from: (dL1 [N, r], dL2 [r, K]) in fp32 from the intermediates T = bf16(X L2^T), T' = bf16(dY L1)."""
    M, r = T.shape
    assert tuple(Tp.shape) == (M, r) and tuple(X.shape) == (M, K) and tuple(dY.shape) == (M, N)
    for t in (T, Tp, X, dY):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
    if out is None:
        out = (torch.empty(N, r, dtype=torch.float32, device=X.device), torch.empty(r, K, dtype=torch.float32, device=X.device))
    if workspace is None:
        workspace = torch.empty(256, dtype=torch.uint8, device=X.device)
    _check(lib().lqlora_lora_grads_from(T.data_ptr(), Tp.data_ptr(), r, N, K, X.data_ptr(), dY.data_ptr(), M, out[0].data_ptr(),
                                        out[1].data_ptr(), workspace.data_ptr(), workspace.numel(), _stream()), "lqlora_lora_grads_from")
    return out


def encode_host(W_host: torch.Tensor, W_stage: torch.Tensor, q: QMatrix, workspace: torch.Tensor) -> None:
    """lqlora_encode_host: W_host is (pinned) host fp32 [N, K]; q and the scratch are on the device."""
    assert not W_host.is_cuda and W_host.dtype == torch.float32 and W_stage.is_cuda
    cs = q.cstruct()
    _check(lib().lqlora_encode_host(W_host.data_ptr(), W_stage.data_ptr(), ctypes.byref(cs), workspace.data_ptr(),
                                    workspace.numel(), _stream()), "lqlora_encode_host")


def _linear_host(fn, name, q, L1, L2, A_host, out_host, A_stage, out_stage, workspace):
    assert not A_host.is_cuda and not out_host.is_cuda and A_stage.is_cuda and out_stage.is_cuda
    M = A_host.shape[0]
    r = 0 if L1 is None else L1.shape[1]
    cs = q.cstruct()
    _check(fn(ctypes.byref(cs), _ptr(L1), _ptr(L2), r, A_host.data_ptr(), M, out_host.data_ptr(), A_stage.data_ptr(),
              out_stage.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream()), name)


def linear_fwd_host(q, L1, L2, X_host, Y_host, X_stage, Y_stage, workspace) -> None:
    _linear_host(lib().lqlora_linear_fwd_host, "lqlora_linear_fwd_host", q, L1, L2, X_host, Y_host, X_stage, Y_stage, workspace)


def linear_bwd_input_host(q, L1, L2, dY_host, dX_host, dY_stage, dX_stage, workspace) -> None:
    _linear_host(lib().lqlora_linear_bwd_input_host, "lqlora_linear_bwd_input_host", q, L1, L2, dY_host, dX_host,
                 dY_stage, dX_stage, workspace)


def lq_decompose(W: torch.Tensor, cfg, r: int, omega: torch.Tensor, F: Optional[torch.Tensor] = None, max_steps: int = 20,
                 power_iters: int = 4):
    """lqlora_lq_decompose: W fp32 [N, K] -> (QMatrix, L1 fp32 [N, r], L2 fp32 [r, K], errors of the steps that ran)."""
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous() and W.dim() == 2
    N, K = W.shape
    assert omega.is_cuda and omega.dtype == torch.float32 and omega.is_contiguous() and omega.shape[0] == K and omega.shape[1] >= r
    p = omega.shape[1] - r
    q = alloc_qmatrix(N, K, cfg, W.device)
    L1 = torch.empty((N, r), dtype=torch.float32, device=W.device)
    L2 = torch.empty((r, K), dtype=torch.float32, device=W.device)
    c = _cfg(cfg)
    need = ctypes.c_size_t(0)
    _check(lib().lqlora_lq_workspace_bytes(N, K, ctypes.byref(c), r, p, ctypes.byref(need)), "lqlora_lq_workspace_bytes")
    ws = torch.empty(int(need.value), dtype=torch.uint8, device=W.device)
    errs = np.zeros(max_steps, dtype=np.float64)
    steps = ctypes.c_int(0)
    cs = q.cstruct()
    _check(lib().lqlora_lq_decompose(W.data_ptr(), _ptr(F), ctypes.byref(cs), L1.data_ptr(), L2.data_ptr(), r, max_steps,
                                     omega.data_ptr(), p, power_iters, errs.ctypes.data, ctypes.byref(steps), ws.data_ptr(),
                                     ws.numel(), _stream()), "lqlora_lq_decompose")
    return q, L1, L2, errs[:steps.value].copy()


def to_bf16(x: torch.Tensor) -> torch.Tensor:
    """lqlora_to_bf16."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    y = torch.empty(x.shape, dtype=torch.bfloat16, device=x.device)
    _check(lib().lqlora_to_bf16(x.data_ptr(), y.data_ptr(), x.numel(), _stream()), "lqlora_to_bf16")
    return y


def assign_configs(errors: np.ndarray, storage: np.ndarray, budget: float):
    """lqlora_assign_configs: errors, storage [n_matrices, n_configs] -> (assignment, total error, total storage) or None."""
    E = np.ascontiguousarray(errors, dtype=np.float64)
    S = np.ascontiguousarray(storage, dtype=np.float64)
    assert E.shape == S.shape and E.ndim == 2
    out = np.zeros(E.shape[0], dtype=np.int32)
    te, ts = ctypes.c_double(0), ctypes.c_double(0)
    rc = lib().lqlora_assign_configs(E.ctypes.data, S.ctypes.data, E.shape[0], E.shape[1], float(budget), out.ctypes.data,
                                     ctypes.byref(te), ctypes.byref(ts))
    if rc == -8:
        return None
    _check(rc, "lqlora_assign_configs")
    return [int(a) for a in out], float(te.value), float(ts.value)


def selftest_bounded_wait(workspace: torch.Tensor, budget_cycles: int) -> None:
    """lqlora_selftest_bounded_wait: a wait that nothing satisfies, abandoned after budget_cycles."""
    _check(lib().lqlora_selftest_bounded_wait(workspace.data_ptr(), int(budget_cycles), _stream()), "lqlora_selftest_bounded_wait")


def static_scratch_status() -> int:
    """lqlora_static_scratch_status: status word of the built-in scratch array after the calls on the current stream."""
    return int(lib().lqlora_static_scratch_status(_stream()))


def workspace_status(workspace: torch.Tensor) -> int:
    return int(lib().lqlora_workspace_status(workspace.data_ptr(), _stream()))


# ----------------------------------------------------------------------------- helpers for tests / bench
def bf16_from_bits(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bit patterns (host) -> bf16 tensor on the device, bit for bit."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device)
    return t.view(torch.bfloat16)


def bits_from_bf16(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
