"""ctypes binding of libmonarch_attn.so: argument marshalling only.

Every step of the method runs inside the library's CUDA kernels.  torch is used for device
memory and streams.  If the shared library has not been built the binding raises; there is no
CPU fallback.
"""
from __future__ import annotations

import ctypes
import math
import os
import re

import torch

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libmonarch_attn.so")
INCLUDE_DIR = os.path.join(os.path.dirname(_PKG_DIR), "include")
HEADER_PATH = os.path.join(INCLUDE_DIR, "monarch_attn.h")

MA_F32, MA_F16, MA_BF16 = 0, 1, 2
MA_PATH_AUTO, MA_PATH_GENERIC, MA_PATH_TENSOR, MA_PATH_TENSOR_TMEM, MA_PATH_TENSOR_BASIC = 0, 1, 2, 3, 4
MA_PATH_FUSED_F32 = 5
MA_PATH_FUSED_JSPLIT = 6
MA_PATH_FUSED_SMALL = 7
MA_PATH_TILE_MMA = 8
MA_OK = 0

_TORCH_TO_CODE = {torch.float32: MA_F32, torch.float16: MA_F16, torch.bfloat16: MA_BF16}
_NAME_TO_TORCH = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}

_lib = None


class MonarchAttnError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"monarch_attn: {what} (status {code})")
        self.code = code


def declared_symbols(header_path: str | None = None):
    """Names of the functions the headers under include/ declare (or one header's)."""
    paths = [header_path] if header_path else sorted(
        os.path.join(INCLUDE_DIR, f) for f in os.listdir(INCLUDE_DIR) if f.endswith(".h"))
    names = set()
    for p in paths:
        text = re.sub(r"/\*.*?\*/", "", open(p).read(), flags=re.S)
        names.update(re.findall(r"\b(monarch_attn_\w+)\s*\(", text))
    return sorted(names)


def load_library(path: str = LIB_PATH):
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path):
        raise MonarchAttnError(-1, f"{path} is missing: build it with __graft_entry__.build()")
    lib = ctypes.CDLL(path)
    vp, i, sz, f = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t, ctypes.c_float
    lib.monarch_attn_fwd.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, vp]
    lib.monarch_attn_fwd.restype = i
    lib.monarch_attn_workspace_bytes.argtypes = [i, i, i, i, i, i, i, i]
    lib.monarch_attn_workspace_bytes.restype = sz
    lib.monarch_attn_fwd_ex.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, vp, sz, vp]
    lib.monarch_attn_fwd_ex.restype = i
    lib.monarch_attn_fwd_objective.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, vp, vp, sz, vp]
    lib.monarch_attn_fwd_objective.restype = i
    lib.monarch_attn_fwd_bshd.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, vp, sz, vp]
    lib.monarch_attn_fwd_bshd.restype = i
    lib.monarch_attn_fwd_padded.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, f, i, vp, sz, vp]
    lib.monarch_attn_fwd_padded.restype = i
    lib.monarch_attn_fwd_varlen.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, f, vp, vp, sz, vp]
    lib.monarch_attn_fwd_varlen.restype = i
    lib.monarch_attn_fwd_host.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, vp]
    lib.monarch_attn_fwd_host.restype = i
    lib.monarch_attn_fwd_noalloc.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, vp]
    lib.monarch_attn_fwd_noalloc.restype = i
    lib.monarch_attn_device_status.argtypes = [vp, vp]
    lib.monarch_attn_device_status.restype = i
    lib.monarch_attn_last_launch_count.argtypes = []
    lib.monarch_attn_last_launch_count.restype = i
    lib.monarch_attn_debug_knob.argtypes = [i, ctypes.c_longlong]
    lib.monarch_attn_debug_knob.restype = i
    lib.monarch_attn_set_trace_buffer.argtypes = [vp, sz]
    lib.monarch_attn_set_trace_buffer.restype = i
    lib.monarch_attn_status_string.argtypes = [i]
    lib.monarch_attn_status_string.restype = ctypes.c_char_p
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().monarch_attn_status_string(int(code)).decode()


def _check(code: int):
    if code != MA_OK:
        raise MonarchAttnError(code, status_string(code))


def _stream_ptr(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _shape_of(Q, K, V):
    if Q.dim() != 4:
        raise ValueError("Q, K, V must be (batch, heads, N, d)")
    if not (Q.shape == K.shape == V.shape and Q.dtype == K.dtype == V.dtype):
        raise ValueError("Q, K, V must share shape and dtype")
    if Q.dtype not in _TORCH_TO_CODE:
        raise ValueError(f"unsupported dtype {Q.dtype}")
    for t in (Q, K, V):
        if not t.is_contiguous():
            raise ValueError("Q, K, V must be contiguous")
    return tuple(int(x) for x in Q.shape)


class _on_device_of:
    """Runs the body with the tensor's device current; free when it already is."""
    __slots__ = ("idx", "prev")

    def __init__(self, t):
        self.idx = t.device.index if t.is_cuda else None
        self.prev = None

    def __enter__(self):
        if self.idx is not None and self.idx != torch.cuda.current_device():
            self.prev = torch.cuda.current_device()
            torch.cuda.set_device(self.idx)

    def __exit__(self, *exc):
        if self.prev is not None:
            torch.cuda.set_device(self.prev)
        return False


def _out_like(Y, Q, what="Y"):
    """A caller-supplied output must match the input exactly: the kernels write Q.numel() elements
    of Q's dtype through its pointer, on Q's device."""
    if Y is None:
        return torch.empty_like(Q)
    if not isinstance(Y, torch.Tensor) or Y.shape != Q.shape or Y.dtype != Q.dtype:
        raise ValueError(f"{what} must have the shape and dtype of Q")
    if not Y.is_contiguous():
        raise ValueError(f"{what} must be contiguous")
    if Y.device != Q.device:
        raise ValueError(f"{what} must be on the same device as Q")
    return Y


def _workspace_for(lib, workspace, Q, batch, heads, N, d, b, T, code, paths):
    """A caller-supplied workspace is checked; otherwise the largest any of `paths` needs."""
    if workspace is not None:
        if workspace.device != Q.device or workspace.dtype != torch.uint8 or not workspace.is_contiguous():
            raise ValueError("workspace must be a contiguous uint8 tensor on Q's device")
        return workspace
    need = max(int(lib.monarch_attn_workspace_bytes(batch, heads, N, d, b, T, code, p)) for p in paths)
    return torch.zeros(max(need, 256), dtype=torch.uint8, device=Q.device)


_ANY_PATH = (MA_PATH_TENSOR, MA_PATH_GENERIC, MA_PATH_TILE_MMA, MA_PATH_FUSED_SMALL, MA_PATH_FUSED_F32)


def monarch_attn_workspace_bytes(batch, heads, N, d, b, T, dtype, path=MA_PATH_AUTO) -> int:
    code = _TORCH_TO_CODE[dtype] if isinstance(dtype, torch.dtype) else int(dtype)
    return int(load_library().monarch_attn_workspace_bytes(batch, heads, N, d, b, T, code, path))


def monarch_attn_fwd(Q, K, V, b, T, Y=None, stream=None):
    """Y = MonarchAttention(Q, K, V) with block size b, T steps, scale 1/sqrt(d).
    Q, K, V: CUDA tensors (batch, heads, N, d)."""
    lib = load_library()
    if not Q.is_cuda:
        raise MonarchAttnError(-2, "monarch_attn_fwd needs CUDA tensors; there is no CPU path")
    batch, heads, N, d = _shape_of(Q, K, V)
    Y = _out_like(Y, Q)
    with _on_device_of(Q):
        _check(lib.monarch_attn_fwd(Q.data_ptr(), K.data_ptr(), V.data_ptr(), Y.data_ptr(),
                                    batch, heads, N, d, b, T, _TORCH_TO_CODE[Q.dtype],
                                    _stream_ptr(stream)))
    return Y


def monarch_attn_fwd_ex(Q, K, V, b, T, softmax_scale=None, path=MA_PATH_AUTO, workspace=None,
                        Y=None, stream=None):
    """As monarch_attn_fwd with explicit scale, path and (optionally) caller-owned workspace
    (a uint8 CUDA tensor).  Returns Y."""
    lib = load_library()
    if not Q.is_cuda:
        raise MonarchAttnError(-2, "monarch_attn_fwd_ex needs CUDA tensors; there is no CPU path")
    batch, heads, N, d = _shape_of(Q, K, V)
    code = _TORCH_TO_CODE[Q.dtype]
    if softmax_scale is None:
        softmax_scale = 1.0 / math.sqrt(d)
    Y = _out_like(Y, Q)
    workspace = _workspace_for(lib, workspace, Q, batch, heads, N, d, b, T, code, (path,))
    with _on_device_of(Q):
        _check(lib.monarch_attn_fwd_ex(Q.data_ptr(), K.data_ptr(), V.data_ptr(), Y.data_ptr(),
                                       batch, heads, N, d, b, T, code, float(softmax_scale), int(path),
                                       workspace.data_ptr(), workspace.numel(), _stream_ptr(stream)))
    return Y


def monarch_attn_fwd_objective(Q, K, V, b, T, softmax_scale=None, path=MA_PATH_AUTO, workspace=None,
                               Y=None, stream=None):
    """Forward pass plus the objective value: returns (Y, row_lse) with row_lse a float32 CUDA
    tensor [batch, heads, N]; row_lse.sum(-1) is f(M^(T)) of Eq. 6 per head."""
    lib = load_library()
    if not Q.is_cuda:
        raise MonarchAttnError(-2, "monarch_attn_fwd_objective needs CUDA tensors; there is no CPU path")
    batch, heads, N, d = _shape_of(Q, K, V)
    code = _TORCH_TO_CODE[Q.dtype]
    if softmax_scale is None:
        softmax_scale = 1.0 / math.sqrt(d)
    Y = _out_like(Y, Q)
    lse = torch.empty((batch, heads, N), dtype=torch.float32, device=Q.device)
    workspace = _workspace_for(lib, workspace, Q, batch, heads, N, d, b, T, code, _ANY_PATH)
    with _on_device_of(Q):
        _check(lib.monarch_attn_fwd_objective(Q.data_ptr(), K.data_ptr(), V.data_ptr(), Y.data_ptr(),
                                              batch, heads, N, d, b, T, code, float(softmax_scale),
                                              int(path), lse.data_ptr(), workspace.data_ptr(),
                                              workspace.numel(), _stream_ptr(stream)))
    return Y, lse


def monarch_attn_fwd_bshd(Q, K, V, b, T, softmax_scale=None, path=MA_PATH_AUTO, workspace=None,
                          Y=None, stream=None):
    """Forward pass on contiguous CUDA tensors [batch, N, heads, d] (no transpose to
    [batch, heads, N, d] needed).  path: MA_PATH_AUTO, MA_PATH_TENSOR, MA_PATH_FUSED_SMALL or MA_PATH_GENERIC."""
    lib = load_library()
    if not Q.is_cuda:
        raise MonarchAttnError(-2, "monarch_attn_fwd_bshd needs CUDA tensors; there is no CPU path")
    if not (Q.shape == K.shape == V.shape and Q.dim() == 4):
        raise ValueError("Q, K, V must share the shape [batch, N, heads, d]")
    if not (Q.is_contiguous() and K.is_contiguous() and V.is_contiguous()):
        raise ValueError("Q, K, V must be contiguous")
    batch, N, heads, d = Q.shape
    code = _TORCH_TO_CODE[Q.dtype]
    if softmax_scale is None:
        softmax_scale = 1.0 / math.sqrt(d)
    Y = _out_like(Y, Q)
    workspace = _workspace_for(lib, workspace, Q, batch, heads, N, d, b, T, code, _ANY_PATH)
    with _on_device_of(Q):
        _check(lib.monarch_attn_fwd_bshd(Q.data_ptr(), K.data_ptr(), V.data_ptr(), Y.data_ptr(),
                                         batch, N, heads, d, b, T, code, float(softmax_scale), int(path),
                                         workspace.data_ptr(), workspace.numel(), _stream_ptr(stream)))
    return Y


def monarch_attn_fwd_padded(Q, K, V, b, T, n_valid, softmax_scale=None, workspace=None, Y=None,
                            stream=None):
    """Forward pass on post-padded CUDA tensors [batch, heads, N, d] with N a multiple of b and
    n_valid real rows (N - b < n_valid <= N): keys beyond n_valid are masked out (App. C.3).
    Returns Y (rows n_valid.. carry no meaning)."""
    lib = load_library()
    if not Q.is_cuda:
        raise MonarchAttnError(-2, "monarch_attn_fwd_padded needs CUDA tensors; there is no CPU path")
    batch, heads, N, d = _shape_of(Q, K, V)
    code = _TORCH_TO_CODE[Q.dtype]
    if softmax_scale is None:
        softmax_scale = 1.0 / math.sqrt(d)
    Y = _out_like(Y, Q)
    workspace = _workspace_for(lib, workspace, Q, batch, heads, N, d, b, T, code, _ANY_PATH)
    with _on_device_of(Q):
        _check(lib.monarch_attn_fwd_padded(Q.data_ptr(), K.data_ptr(), V.data_ptr(), Y.data_ptr(),
                                           batch, heads, N, d, b, T, code, float(softmax_scale),
                                           int(n_valid), workspace.data_ptr(), workspace.numel(),
                                           _stream_ptr(stream)))
    return Y


def monarch_attn_fwd_varlen(Q, K, V, b, T, seq_len, softmax_scale=None, workspace=None, Y=None,
                            stream=None):
    """Forward pass on a batch of sequences of different lengths padded to N rows (App. C.3).
    seq_len: int32 CUDA tensor [batch] with the number of real rows of each batch entry.  Rows
    below seq_len[e] of Y are the result; rows from ceil(seq_len[e] / b) * b on are zero."""
    lib = load_library()
    if not Q.is_cuda:
        raise MonarchAttnError(-2, "monarch_attn_fwd_varlen needs CUDA tensors; there is no CPU path")
    batch, heads, N, d = _shape_of(Q, K, V)
    if not (isinstance(seq_len, torch.Tensor) and seq_len.dtype == torch.int32 and seq_len.is_contiguous()
            and seq_len.device == Q.device and tuple(seq_len.shape) == (batch,)):
        raise ValueError("seq_len must be a contiguous int32 tensor of shape [batch] on Q's device")
    code = _TORCH_TO_CODE[Q.dtype]
    if softmax_scale is None:
        softmax_scale = 1.0 / math.sqrt(d)
    Y = _out_like(Y, Q)
    workspace = _workspace_for(lib, workspace, Q, batch, heads, N, d, b, T, code,
                               (MA_PATH_GENERIC, MA_PATH_FUSED_SMALL, MA_PATH_TILE_MMA))
    with _on_device_of(Q):
        _check(lib.monarch_attn_fwd_varlen(Q.data_ptr(), K.data_ptr(), V.data_ptr(), Y.data_ptr(),
                                           batch, heads, N, d, b, T, code, float(softmax_scale),
                                           seq_len.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                           _stream_ptr(stream)))
    return Y


def monarch_attn_fwd_host(Qh, Kh, Vh, Yh, b, T, stream=None):
    """End-to-end call on HOST tensors (pinned for asynchronous copies): H2D, kernels, D2H on
    `stream`; returns Yh without synchronising."""
    lib = load_library()
    batch, heads, N, d = _shape_of(Qh, Kh, Vh)
    if Qh.is_cuda or Kh.is_cuda or Vh.is_cuda or Yh.is_cuda:
        raise ValueError("monarch_attn_fwd_host takes host tensors")
    _out_like(Yh, Qh, "Yh")
    _check(lib.monarch_attn_fwd_host(Qh.data_ptr(), Kh.data_ptr(), Vh.data_ptr(), Yh.data_ptr(),
                                     batch, heads, N, d, b, T, _TORCH_TO_CODE[Qh.dtype],
                                     _stream_ptr(stream)))
    return Yh


NOALLOC_SCRATCH_BYTES = 8 << 20


def monarch_attn_fwd_noalloc(Q, K, V, b, T, Y, stream=None):
    """Forward pass for callers that may not allocate device memory: the library's built-in
    scratch array holds the states, and the caller supplies the output tensor Y as well (so this
    wrapper allocates nothing either).  Small problems only (see the header for the limit);
    calls that overlap on the GPU race on the shared scratch."""
    lib = load_library()
    if not (Q.is_cuda and Y is not None and Y.is_cuda):
        raise MonarchAttnError(-2, "monarch_attn_fwd_noalloc needs CUDA tensors; there is no CPU path")
    batch, heads, N, d = _shape_of(Q, K, V)
    if Y is None:
        raise ValueError("monarch_attn_fwd_noalloc allocates nothing: pass the output tensor Y")
    _out_like(Y, Q)
    with _on_device_of(Q):
        _check(lib.monarch_attn_fwd_noalloc(Q.data_ptr(), K.data_ptr(), V.data_ptr(), Y.data_ptr(),
                                            batch, heads, N, d, b, T, _TORCH_TO_CODE[Q.dtype],
                                            _stream_ptr(stream)))
    return Y


def monarch_attn_device_status(workspace=None, stream=None) -> int:
    lib = load_library()
    ptr = None if workspace is None else workspace.data_ptr()
    return int(lib.monarch_attn_device_status(ptr, _stream_ptr(stream)))


def monarch_attn_last_launch_count() -> int:
    return int(load_library().monarch_attn_last_launch_count())


def monarch_attn_set_trace_buffer(buf=None):
    """buf: int64 CUDA tensor with >= 4*64*8 elements, or None to switch tracing off."""
    lib = load_library()
    if buf is None:
        _check(lib.monarch_attn_set_trace_buffer(None, 0))
    else:
        _check(lib.monarch_attn_set_trace_buffer(buf.data_ptr(), buf.numel() * buf.element_size()))


def monarch_attn_debug_knob(knob: int, value: int):
    _check(load_library().monarch_attn_debug_knob(int(knob), int(value)))


def torch_dtype(name: str) -> torch.dtype:
    return _NAME_TO_TORCH[name]


def to_device(x_f32_numpy, dtype_name: str, device="cuda"):
    """float32 numpy array whose values are representable in `dtype_name` -> torch tensor."""
    return torch.from_numpy(x_f32_numpy).to(device=device, dtype=_NAME_TO_TORCH[dtype_name]).contiguous()
