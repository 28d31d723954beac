"""ctypes binding of ``libl4q.so`` (C ABI declared in ``include/l4q.h``).

Argument marshalling only: every function here checks dtypes/shapes, takes
``data_ptr()`` of torch CUDA tensors and calls the C entry point of the same
name.  No layer arithmetic happens in Python and there is no fallback: if the
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from .synth import LayerConfig

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libl4q.so")

L4Q_OK = 0
L4Q_BF16, L4Q_F32 = 0, 1
L4Q_OP_FWD, L4Q_OP_BWD, L4Q_OP_PACK = 0, 1, 2
L4Q_FLAG_SIGNED_GRID = 1
L4Q_MAX_RANK = 128

EXPORTED_SYMBOLS = (
    "l4q_workspace_bytes", "l4q_linear_fwd", "l4q_linear_bwd", "l4q_pack_int",
    "l4q_check", "l4q_launch_count", "l4q_status_string",
    "l4q_profile_enable", "l4q_profile_read", "l4q_kernel_name",
    "l4q_linear_fwd_static", "l4q_init_params", "l4q_quant_error", "l4q_linear_infer", "l4q_adamw_step",
    "l4q_lora_workspace_bytes", "l4q_lora_linear_fwd", "l4q_lora_linear_bwd", "l4q_selftest_timeout",
    "l4q_selftest_tile_copy", "l4q_adamw_step_multi",
)
L4Q_LORA_PLAIN, L4Q_LORA_QAT = 1, 2
LORA_KINDS = {"lora": L4Q_LORA_PLAIN, "qat_lora": L4Q_LORA_QAT}
INIT_METHODS = {"lsq+": 0, "symm": 1, "asymm": 2, "l4q": 3}

L4Q_STATIC_SCRATCH_BYTES = 32 * 1024 * 1024

KERNEL_IDS = {"dequant": 0, "pack": 1, "gemm_fwd": 2, "gemm_dgrad": 3, "gemm_wgrad": 4, "val_gemm": 5,
              "val_wgrad": 6, "init": 7, "error": 8, "infer": 9, "adamw": 10, "lora_side": 11, "tile_copy": 12}


class L4QDesc(ctypes.Structure):
    """Mirror of ``struct l4q_desc``."""

    _fields_ = [
        ("tokens", ctypes.c_int64), ("d_in", ctypes.c_int64), ("d_out", ctypes.c_int64),
        ("rank", ctypes.c_int32), ("alpha", ctypes.c_float),
        ("bits", ctypes.c_int32), ("group_size", ctypes.c_int32),
        ("io_dtype", ctypes.c_int32), ("flags", ctypes.c_uint32), ("grad_scale", ctypes.c_float),
    ]


class L4QAdamwTensor(ctypes.Structure):
    """Mirror of ``l4q_adamw_tensor``."""

    _fields_ = [("param", ctypes.c_void_p), ("grad", ctypes.c_void_p), ("m", ctypes.c_void_p), ("v", ctypes.c_void_p),
                ("n", ctypes.c_size_t)]


class L4QError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (l4q_status {status})")


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Load ``libl4q.so`` (once). Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} not found: build it with `python -m paper_2402_04902_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, fp, sz = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t
        dp = ctypes.POINTER(L4QDesc)
        L.l4q_workspace_bytes.restype = sz
        L.l4q_workspace_bytes.argtypes = [dp, ctypes.c_int]
        L.l4q_linear_fwd.restype = ctypes.c_int
        L.l4q_linear_fwd.argtypes = [dp, vp, vp, fp, fp, fp, fp, vp, vp, sz, vp]
        L.l4q_linear_fwd_static.restype = ctypes.c_int
        L.l4q_linear_fwd_static.argtypes = [dp, vp, vp, fp, fp, fp, fp, vp, vp]
        L.l4q_linear_bwd.restype = ctypes.c_int
        L.l4q_linear_bwd.argtypes = [dp, vp, vp, vp, fp, fp, fp, fp, vp, fp, fp, fp, fp, vp, sz, vp]
        L.l4q_lora_workspace_bytes.restype = sz
        L.l4q_lora_workspace_bytes.argtypes = [dp, ctypes.c_int, ctypes.c_int]
        L.l4q_lora_linear_fwd.restype = ctypes.c_int
        L.l4q_lora_linear_fwd.argtypes = [dp, ctypes.c_int, vp, vp, fp, fp, fp, fp, vp, vp, sz, vp]
        L.l4q_lora_linear_bwd.restype = ctypes.c_int
        L.l4q_lora_linear_bwd.argtypes = [dp, ctypes.c_int, vp, vp, vp, fp, fp, fp, fp, vp, fp, fp, fp, fp, vp, sz, vp]
        L.l4q_pack_int.restype = ctypes.c_int
        L.l4q_pack_int.argtypes = [dp, vp, fp, fp, fp, fp, vp, vp, vp, vp, sz, vp]
        L.l4q_linear_infer.restype = ctypes.c_int
        L.l4q_linear_infer.argtypes = [dp, vp, vp, vp, vp, vp, vp]
        L.l4q_adamw_step.restype = ctypes.c_int
        L.l4q_adamw_step.argtypes = [fp, fp, fp, fp, sz, ctypes.c_int64, ctypes.c_float, ctypes.c_float,
                                     ctypes.c_float, ctypes.c_float, ctypes.c_float, vp]
        L.l4q_init_params.restype = ctypes.c_int
        L.l4q_init_params.argtypes = [dp, vp, ctypes.c_int, fp, fp, vp]
        L.l4q_quant_error.restype = ctypes.c_int
        L.l4q_quant_error.argtypes = [dp, vp, fp, fp, fp, fp, vp, vp]
        L.l4q_adamw_step_multi.restype = ctypes.c_int
        L.l4q_adamw_step_multi.argtypes = [ctypes.POINTER(L4QAdamwTensor), ctypes.c_int, ctypes.c_int64, ctypes.c_float,
                                           ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_float, vp]
        L.l4q_selftest_timeout.restype = ctypes.c_int
        L.l4q_selftest_timeout.argtypes = [vp]
        L.l4q_selftest_tile_copy.restype = ctypes.c_int
        L.l4q_selftest_tile_copy.argtypes = [vp, vp, ctypes.c_int64, ctypes.c_int64, vp]
        L.l4q_check.restype = ctypes.c_int
        L.l4q_check.argtypes = [vp]
        L.l4q_launch_count.restype = ctypes.c_uint64
        L.l4q_launch_count.argtypes = []
        L.l4q_status_string.restype = ctypes.c_char_p
        L.l4q_status_string.argtypes = [ctypes.c_int]
        L.l4q_profile_enable.restype = ctypes.c_int
        L.l4q_profile_enable.argtypes = [ctypes.c_int]
        L.l4q_profile_read.restype = ctypes.c_int
        L.l4q_profile_read.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_double)]
        L.l4q_kernel_name.restype = ctypes.c_char_p
        L.l4q_kernel_name.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().l4q_status_string(int(status)).decode()


def make_desc(cfg: LayerConfig, grad_scale: float = 1.0, tokens: Optional[int] = None) -> L4QDesc:
    return L4QDesc(tokens=int(tokens if tokens is not None else cfg.tokens), d_in=cfg.d_in, d_out=cfg.d_out,
                   rank=cfg.rank, alpha=float(cfg.alpha), bits=cfg.bits, group_size=cfg.group_size,
                   io_dtype=L4Q_BF16 if cfg.io_dtype == "bf16" else L4Q_F32,
                   flags=L4Q_FLAG_SIGNED_GRID if cfg.signed_grid else 0, grad_scale=float(grad_scale))


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("L4Q tensors must be contiguous CUDA tensors")
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream if stream is not None else torch.cuda.current_stream()).cuda_stream


def _raise(status: int, where: str) -> None:
    if status != L4Q_OK:
        raise L4QError(status, where)


def l4q_workspace_bytes(desc: L4QDesc, op: int) -> int:
    return int(lib().l4q_workspace_bytes(ctypes.byref(desc), int(op)))


def alloc_workspace(desc: L4QDesc, op: int, device="cuda") -> torch.Tensor:
    """Device scratch for one op (torch is used for device memory only)."""
    n = max(l4q_workspace_bytes(desc, op), 256)
    return torch.empty(n, dtype=torch.uint8, device=device)


def l4q_linear_fwd(desc: L4QDesc, X, W0, A, B, s, b, Y, workspace, stream=None) -> None:
    st = lib().l4q_linear_fwd(ctypes.byref(desc), _ptr(X), _ptr(W0), _ptr(A), _ptr(B), _ptr(s), _ptr(b), _ptr(Y),
                              _ptr(workspace), workspace.numel() if workspace is not None else 0, _stream(stream))
    _raise(st, "l4q_linear_fwd")


def l4q_linear_fwd_static(desc: L4QDesc, X, W0, A, B, s, b, Y, stream=None) -> None:
    """Forward without a workspace: for callers that may not allocate device memory
    (the scratch is a fixed 32 MiB array inside the library; see include/l4q.h for
    the size limit and the sharing rules)."""
    st = lib().l4q_linear_fwd_static(ctypes.byref(desc), _ptr(X), _ptr(W0), _ptr(A), _ptr(B), _ptr(s), _ptr(b),
                                     _ptr(Y), _stream(stream))
    _raise(st, "l4q_linear_fwd_static")


def l4q_linear_bwd(desc: L4QDesc, X, dY, W0, A, B, s, b, dX, dA, dB, ds, db, workspace, stream=None) -> None:
    st = lib().l4q_linear_bwd(ctypes.byref(desc), _ptr(X), _ptr(dY), _ptr(W0), _ptr(A), _ptr(B), _ptr(s), _ptr(b),
                              _ptr(dX), _ptr(dA), _ptr(dB), _ptr(ds), _ptr(db),
                              _ptr(workspace), workspace.numel() if workspace is not None else 0, _stream(stream))
    _raise(st, "l4q_linear_bwd")


def l4q_lora_workspace_bytes(desc: L4QDesc, kind: int, op: int) -> int:
    return int(lib().l4q_lora_workspace_bytes(ctypes.byref(desc), int(kind), int(op)))


def alloc_lora_workspace(desc: L4QDesc, kind: int, op: int, device="cuda") -> torch.Tensor:
    n = max(l4q_lora_workspace_bytes(desc, kind, op), 256)
    return torch.empty(n, dtype=torch.uint8, device=device)


def l4q_lora_linear_fwd(desc: L4QDesc, kind: int, X, W0, A, B, s, b, Y, workspace, stream=None) -> None:
    """Forward of the LoRA (Eq. 1) or QAT-LoRA (Sec. 3.1) layer; kind = L4Q_LORA_PLAIN / L4Q_LORA_QAT."""
    st = lib().l4q_lora_linear_fwd(ctypes.byref(desc), int(kind), _ptr(X), _ptr(W0), _ptr(A), _ptr(B), _ptr(s),
                                   _ptr(b), _ptr(Y), _ptr(workspace),
                                   workspace.numel() if workspace is not None else 0, _stream(stream))
    _raise(st, "l4q_lora_linear_fwd")


def l4q_lora_linear_bwd(desc: L4QDesc, kind: int, X, dY, W0, A, B, s, b, dX, dA, dB, ds, db, workspace,
                        stream=None) -> None:
    """Backward of the LoRA (Eq. 2) or QAT-LoRA layer; ds, db only for L4Q_LORA_QAT."""
    st = lib().l4q_lora_linear_bwd(ctypes.byref(desc), int(kind), _ptr(X), _ptr(dY), _ptr(W0), _ptr(A), _ptr(B),
                                   _ptr(s), _ptr(b), _ptr(dX), _ptr(dA), _ptr(dB), _ptr(ds), _ptr(db),
                                   _ptr(workspace), workspace.numel() if workspace is not None else 0,
                                   _stream(stream))
    _raise(st, "l4q_lora_linear_bwd")


def l4q_pack_int(desc: L4QDesc, W0, A, B, s, b, codes, s_fp16, b_fp16, workspace=None, stream=None) -> None:
    st = lib().l4q_pack_int(ctypes.byref(desc), _ptr(W0), _ptr(A), _ptr(B), _ptr(s), _ptr(b), _ptr(codes),
                            _ptr(s_fp16), _ptr(b_fp16), _ptr(workspace),
                            workspace.numel() if workspace is not None else 0, _stream(stream))
    _raise(st, "l4q_pack_int")


def l4q_linear_infer(desc: L4QDesc, X, codes, s_fp16, b_fp16, Y, stream=None) -> None:
    """Y = X W_q^T from the packed export of l4q_pack_int (few-token inference, App. F)."""
    st = lib().l4q_linear_infer(ctypes.byref(desc), _ptr(X), _ptr(codes), _ptr(s_fp16), _ptr(b_fp16), _ptr(Y),
                                _stream(stream))
    _raise(st, "l4q_linear_infer")


def l4q_adamw_step(param, grad, m, v, step: int, lr: float, beta1: float = 0.9, beta2: float = 0.999,
                   eps: float = 1e-8, weight_decay: float = 0.01, stream=None) -> None:
    """In-place AdamW update of one fp32 parameter tensor (App. D); step counts from 1."""
    for t in (param, grad, m, v):
        if t.dtype != torch.float32 or t.numel() != param.numel():
            raise ValueError("AdamW tensors must be float32 and of one size")
    st = lib().l4q_adamw_step(_ptr(param), _ptr(grad), _ptr(m), _ptr(v), param.numel(), int(step), float(lr),
                              float(beta1), float(beta2), float(eps), float(weight_decay), _stream(stream))
    _raise(st, "l4q_adamw_step")


def l4q_adamw_step_multi(tensors, step: int, lr: float, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                         weight_decay: float = 0.01, stream=None) -> None:
    """In-place AdamW update (App. D) of up to 8 fp32 tensors in one launch; `tensors`: (param, grad, m, v) tuples."""
    table = (L4QAdamwTensor * len(tensors))()
    for k, (param, grad, m, v) in enumerate(tensors):
        for t in (param, grad, m, v):
            if t.dtype != torch.float32 or t.numel() != param.numel():
                raise ValueError("AdamW tensors must be float32 and of one size per entry")
        table[k] = L4QAdamwTensor(_ptr(param), _ptr(grad), _ptr(m), _ptr(v), param.numel())
    st = lib().l4q_adamw_step_multi(table, len(tensors), int(step), float(lr), float(beta1), float(beta2), float(eps),
                                    float(weight_decay), _stream(stream))
    _raise(st, "l4q_adamw_step_multi")


def l4q_init_params(desc: L4QDesc, W, method: str, s, b, stream=None) -> None:
    """s, b of every group from the weight W (App. B); method in INIT_METHODS."""
    st = lib().l4q_init_params(ctypes.byref(desc), _ptr(W), INIT_METHODS[method], _ptr(s), _ptr(b), _stream(stream))
    _raise(st, "l4q_init_params")


def l4q_quant_error(desc: L4QDesc, W0, A, B, s, b, errors, stream=None) -> None:
    """errors: CUDA tensor of two float64, receives (E_quant, E_clip) of Table 4."""
    if errors.dtype != torch.float64 or errors.numel() < 2:
        raise ValueError("errors must be a float64 CUDA tensor with two elements")
    st = lib().l4q_quant_error(ctypes.byref(desc), _ptr(W0), _ptr(A), _ptr(B), _ptr(s), _ptr(b), _ptr(errors),
                               _stream(stream))
    _raise(st, "l4q_quant_error")


def l4q_selftest_timeout(stream=None) -> None:
    """Make one bounded device-side wait expire (about a millisecond); the next l4q_check raises L4Q_ERR_TIMEOUT."""
    _raise(lib().l4q_selftest_timeout(_stream(stream)), "l4q_selftest_timeout")


def l4q_selftest_tile_copy(src, dst=None, stream=None) -> None:
    """Move the bf16 matrix `src` through shared memory in 128 x 128 tiles by TMA (and store it to `dst` if given):
    the memory-system floor of the weight-tile kernels on that size.  Timed by the library's per-launch events."""
    if src.dtype != torch.bfloat16 or src.dim() != 2 or (dst is not None and (dst.dtype != src.dtype or dst.shape != src.shape)):
        raise ValueError("src (and dst) must be 2-D bf16 CUDA tensors of the same shape")
    _raise(lib().l4q_selftest_tile_copy(_ptr(src), _ptr(dst), src.shape[0], src.shape[1], _stream(stream)),
           "l4q_selftest_tile_copy")


def l4q_check(stream=None) -> None:
    """Synchronise the stream and raise if a kernel recorded an error."""
    _raise(lib().l4q_check(_stream(stream)), "l4q_check")


def l4q_launch_count() -> int:
    return int(lib().l4q_launch_count())


def l4q_profile_enable(enable: bool) -> None:
    _raise(lib().l4q_profile_enable(1 if enable else 0), "l4q_profile_enable")


def l4q_profile_read() -> dict:
    """{kernel name: (timed launches, total device ms)} since profiling was enabled."""
    out = {}
    for name, kid in KERNEL_IDS.items():
        n, ms = ctypes.c_uint64(0), ctypes.c_double(0.0)
        _raise(lib().l4q_profile_read(kid, ctypes.byref(n), ctypes.byref(ms)), "l4q_profile_read")
        out[name] = (int(n.value), float(ms.value))
    return out


def l4q_kernel_name(kernel: int) -> str:
    return lib().l4q_kernel_name(int(kernel)).decode()


# ---------------------------------------------------------------------------
# Convenience: move one synthetic layer (numpy, from synth.make_layer_inputs)
# to the device in the dtypes the library expects.  Data movement only.
# ---------------------------------------------------------------------------

def to_device(cfg: LayerConfig, arrays: dict, device="cuda") -> dict:
    io = torch.bfloat16 if cfg.io_dtype == "bf16" else torch.float32
    out = {}
    for k, v in arrays.items():
        t = torch.from_numpy(v)
        if k in ("X", "dY", "W0"):
            t = t.to(io)           # exact: the values are representable in the io dtype
        out[k] = t.to(device).contiguous()
    return out


def alloc_outputs(cfg: LayerConfig, device="cuda", tokens: Optional[int] = None) -> dict:
    io = torch.bfloat16 if cfg.io_dtype == "bf16" else torch.float32
    M = tokens if tokens is not None else cfg.tokens
    G = cfg.d_in // cfg.group_size
    f32 = torch.float32
    return {
        "Y": torch.empty(M, cfg.d_out, dtype=io, device=device),
        "dX": torch.empty(M, cfg.d_in, dtype=io, device=device),
        "dA": torch.empty(cfg.rank, cfg.d_in, dtype=f32, device=device),
        "dB": torch.empty(cfg.d_out, cfg.rank, dtype=f32, device=device),
        "ds": torch.empty(cfg.d_out, G, dtype=f32, device=device),
        "db": torch.empty(cfg.d_out, G, dtype=f32, device=device),
    }


def alloc_pack_outputs(cfg: LayerConfig, device="cuda") -> dict:
    G = cfg.d_in // cfg.group_size
    return {
        "codes": torch.empty(cfg.d_out, cfg.d_in * cfg.bits // 32, dtype=torch.int32, device=device),
        "s16": torch.empty(cfg.d_out, G, dtype=torch.float16, device=device),
        "b16": torch.empty(cfg.d_out, G, dtype=torch.float16, device=device),
    }
