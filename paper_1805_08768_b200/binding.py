"""Thin ctypes binding over the C ABI declared in include/sbc.h.

Argument marshalling only: torch supplies device memory and the current CUDA
stream, every step of the method runs in the library's kernels.  The library
is loaded on first use; if it is missing or cannot be loaded the call raises
-- there is no other path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsbc_b200.so")

SBC_OK, SBC_EINVAL, SBC_ECAPACITY, SBC_ENONFINITE, SBC_ECORRUPT, SBC_ETIMEOUT, SBC_ECUDA = 0, -1, -2, -3, -4, -5, -6
STATUS_NONFINITE, STATUS_CORRUPT, STATUS_RANGE, STATUS_INTERNAL, STATUS_TIMEOUT = 1, 2, 4, 8, 16
_ERR = {SBC_EINVAL: "SBC_EINVAL", SBC_ECAPACITY: "SBC_ECAPACITY", SBC_ENONFINITE: "SBC_ENONFINITE",
        SBC_ECORRUPT: "SBC_ECORRUPT", SBC_ETIMEOUT: "SBC_ETIMEOUT", SBC_ECUDA: "SBC_ECUDA"}

EXPORTS = [
    "sbc_kept_count", "sbc_golomb_b", "sbc_mean_position_bits", "sbc_stream_bytes",
    "sbc_workspace_bytes", "sbc_encode", "sbc_encode_ex", "sbc_encode_launches", "sbc_decode_launches",
    "sbc_encode_diag_get", "sbc_encode_host", "sbc_stream_info_get", "sbc_decode_accumulate",
    "sbc_decode_accumulate_host", "sbc_encode_static", "sbc_workspace_bytes_batch", "sbc_encode_batch",
    "sbc_decode_workspace_bytes_batch", "sbc_decode_accumulate_batch", "sbc_decode_apply", "sbc_stream_bytes_values", "sbc_encode_values", "sbc_stream_bytes_sampled",
    "sbc_workspace_bytes_sampled", "sbc_encode_sampled", "sbc_decode_accumulate_sized", "sbc_decode_apply_sized",
    "sbc_debug_barrier_timeout",
]
SIDE_VALUES = 2
STATIC_WORKSPACE_BYTES = 8 << 20
MARK_BEGIN, MARK_BOUNDS, MARK_COLLECT, MARK_EXACT, MARK_SELECT, MARK_END, MARK_COUNT = range(7)
MARK_NAMES = ["bounds", "collect", "exact", "select", "golomb"]  # interval i = mark i -> mark i+1


class SbcError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where} failed: {_ERR.get(code, code)}")
        self.code = code


class StreamInfo(C.Structure):
    _fields_ = [
        ("magic", C.c_uint32), ("version", C.c_uint32),
        ("numel", C.c_uint64), ("k", C.c_uint64), ("nbits", C.c_uint64), ("payload_offset", C.c_uint64),
        ("b", C.c_uint32), ("side", C.c_uint32), ("mu", C.c_float),
        ("chunk_codewords", C.c_uint32), ("n_chunks", C.c_uint32), ("status", C.c_uint32),
        ("total_bytes", C.c_uint64),
    ]


class EncodeDiag(C.Structure):
    _fields_ = [
        ("status", C.c_uint32), ("exact_route", C.c_uint32), ("candidates", C.c_uint32 * 2),
        ("capacity", C.c_uint32), ("bound_lo", C.c_float), ("bound_hi", C.c_float),
        ("mu_pos", C.c_double), ("mu_neg", C.c_double), ("certain", C.c_uint32 * 2), ("regathered", C.c_uint32),
    ]


class TensorDesc(C.Structure):
    _fields_ = [("update", C.c_void_p), ("residual", C.c_void_p), ("numel", C.c_int64), ("p", C.c_double),
                ("out_stream", C.c_void_p), ("out_capacity", C.c_size_t), ("out_mu", C.c_void_p)]


class DecodeDesc(C.Structure):
    _fields_ = [("streams", C.POINTER(C.c_void_p)), ("out_dense", C.c_void_p), ("numel", C.c_int64),
                ("stream_bytes", C.POINTER(C.c_size_t))]


_lib = None


def lib() -> C.CDLL:
    """The loaded CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_1805_08768_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.sbc_kept_count.restype = C.c_int64
        L.sbc_kept_count.argtypes = [C.c_int64, C.c_double]
        L.sbc_golomb_b.restype = C.c_int
        L.sbc_golomb_b.argtypes = [C.c_double]
        L.sbc_mean_position_bits.restype = C.c_double
        L.sbc_mean_position_bits.argtypes = [C.c_double, C.c_int]
        L.sbc_stream_bytes.restype = C.c_size_t
        L.sbc_stream_bytes.argtypes = [C.c_int64, C.c_double]
        L.sbc_workspace_bytes.restype = C.c_size_t
        L.sbc_workspace_bytes.argtypes = [C.c_int64, C.c_double]
        L.sbc_encode.restype = C.c_int
        L.sbc_encode.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_double, C.c_void_p, C.c_size_t,
                                 C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.sbc_encode_ex.restype = C.c_int
        L.sbc_encode_ex.argtypes = L.sbc_encode.argtypes + [C.POINTER(C.c_void_p)]
        L.sbc_encode_launches.restype = C.c_int
        L.sbc_encode_launches.argtypes = []
        L.sbc_decode_launches.restype = C.c_int
        L.sbc_decode_launches.argtypes = [C.c_int]
        L.sbc_encode_diag_get.restype = C.c_int
        L.sbc_encode_diag_get.argtypes = [C.c_void_p, C.POINTER(EncodeDiag), C.c_void_p]
        L.sbc_encode_host.restype = C.c_int
        L.sbc_encode_host.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_double, C.c_void_p,
                                      C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t), C.POINTER(C.c_float),
                                      C.c_void_p, C.c_size_t, C.c_void_p]
        L.sbc_decode_accumulate_host.restype = C.c_int
        L.sbc_decode_accumulate_host.argtypes = [C.POINTER(C.c_void_p), C.POINTER(C.c_size_t), C.c_int,
                                                 C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t,
                                                 C.POINTER(C.c_uint32), C.c_void_p]
        L.sbc_encode_static.restype = C.c_int
        L.sbc_encode_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_double, C.c_void_p, C.c_size_t,
                                        C.c_void_p, C.c_void_p]
        L.sbc_workspace_bytes_batch.restype = C.c_size_t
        L.sbc_workspace_bytes_batch.argtypes = [C.c_int, C.POINTER(TensorDesc)]
        L.sbc_encode_batch.restype = C.c_int
        L.sbc_encode_batch.argtypes = [C.c_int, C.POINTER(TensorDesc), C.c_void_p, C.c_size_t, C.c_void_p]
        L.sbc_decode_workspace_bytes_batch.restype = C.c_size_t
        L.sbc_decode_workspace_bytes_batch.argtypes = [C.c_int]
        L.sbc_decode_accumulate_batch.restype = C.c_int
        L.sbc_decode_accumulate_batch.argtypes = [C.c_int, C.c_int, C.POINTER(DecodeDesc), C.c_void_p, C.c_void_p,
                                                  C.c_size_t, C.c_void_p]
        L.sbc_decode_apply.restype = C.c_int
        L.sbc_decode_apply.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_float, C.c_void_p, C.c_void_p, C.c_int64,
                                       C.c_void_p, C.c_void_p]
        L.sbc_stream_bytes_values.restype = C.c_size_t
        L.sbc_stream_bytes_values.argtypes = [C.c_int64, C.c_double]
        L.sbc_encode_values.restype = C.c_int
        L.sbc_encode_values.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_double, C.c_void_p, C.c_size_t,
                                        C.c_void_p, C.c_size_t, C.c_void_p]
        L.sbc_stream_bytes_sampled.restype = C.c_size_t
        L.sbc_stream_bytes_sampled.argtypes = [C.c_int64, C.c_double]
        L.sbc_workspace_bytes_sampled.restype = C.c_size_t
        L.sbc_workspace_bytes_sampled.argtypes = [C.c_int64, C.c_double, C.c_int64]
        L.sbc_encode_sampled.restype = C.c_int
        L.sbc_encode_sampled.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_double, C.c_void_p, C.c_int64,
                                         C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.sbc_stream_info_get.restype = C.c_int
        L.sbc_stream_info_get.argtypes = [C.c_void_p, C.POINTER(StreamInfo), C.c_void_p]
        L.sbc_decode_accumulate.restype = C.c_int
        L.sbc_decode_accumulate.argtypes = [C.POINTER(C.c_void_p), C.c_int, C.c_void_p, C.c_int64,
                                            C.c_void_p, C.c_void_p]
        L.sbc_decode_accumulate_sized.restype = C.c_int
        L.sbc_decode_accumulate_sized.argtypes = [C.POINTER(C.c_void_p), C.POINTER(C.c_size_t), C.c_int, C.c_void_p,
                                                  C.c_int64, C.c_void_p, C.c_void_p]
        L.sbc_decode_apply_sized.restype = C.c_int
        L.sbc_decode_apply_sized.argtypes = [C.POINTER(C.c_void_p), C.POINTER(C.c_size_t), C.c_int, C.c_float,
                                             C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != SBC_OK:
        raise SbcError(code, where)


def _cuda_stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dev_f32(t: torch.Tensor, name: str) -> None:
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous float32 CUDA tensor")


# ---- host-side pure functions --------------------------------------------------

def sbc_kept_count(numel: int, p: float) -> int:
    return int(lib().sbc_kept_count(numel, p))


def sbc_golomb_b(p: float) -> int:
    return int(lib().sbc_golomb_b(p))


def sbc_mean_position_bits(p: float, b: int) -> float:
    return float(lib().sbc_mean_position_bits(p, b))


def sbc_stream_bytes(numel: int, p: float) -> int:
    return int(lib().sbc_stream_bytes(numel, p))


def sbc_workspace_bytes(numel: int, p: float) -> int:
    return int(lib().sbc_workspace_bytes(numel, p))


# ---- device entry points ---------------------------------------------------------

def sbc_encode(update: torch.Tensor, residual: torch.Tensor, p: float,
               out_stream: Optional[torch.Tensor] = None, out_mu: Optional[torch.Tensor] = None,
               workspace: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Enqueue one client step; ``residual`` is updated in place.

    Returns (out_stream uint8 tensor of capacity bytes, out_mu float32[1]),
    both on the device and valid once the CUDA stream has run the work."""
    _dev_f32(update, "update")
    _dev_f32(residual, "residual")
    n = update.numel()
    if residual.numel() != n:
        raise ValueError("update and residual differ in size")
    dev = update.device
    if out_stream is None:
        out_stream = torch.empty(sbc_stream_bytes(n, p), dtype=torch.uint8, device=dev)
    if out_mu is None:
        out_mu = torch.empty(1, dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = torch.empty(sbc_workspace_bytes(n, p), dtype=torch.uint8, device=dev)
    code = lib().sbc_encode(update.data_ptr(), residual.data_ptr(), n, float(p),
                            out_stream.data_ptr(), out_stream.numel(), out_mu.data_ptr(),
                            workspace.data_ptr(), workspace.numel(), _cuda_stream(stream))
    _check(code, "sbc_encode")
    return out_stream, out_mu


def _tensor_descs(updates, residuals, ps, out_streams, out_mus):
    """One sbc_tensor_desc per tensor of a batch (the only place they are marshalled)."""
    n = len(updates)
    descs = (TensorDesc * n)()
    for t in range(n):
        _dev_f32(updates[t], "update")
        _dev_f32(residuals[t], "residual")
        d = descs[t]
        d.update, d.residual, d.numel, d.p = updates[t].data_ptr(), residuals[t].data_ptr(), updates[t].numel(), float(ps[t])
        d.out_stream, d.out_capacity, d.out_mu = out_streams[t].data_ptr(), out_streams[t].numel(), out_mus[t].data_ptr()
    return descs


def _decode_descs(streams_per_tensor, out_denses, sizes_per_tensor=None):
    """One sbc_decode_desc per tensor; returns (descs, n_clients, objects the descs point into)."""
    n = len(out_denses)
    n_clients = len(streams_per_tensor[0])
    descs = (DecodeDesc * n)()
    keep = []
    for t in range(n):
        if len(streams_per_tensor[t]) != n_clients:
            raise ValueError("every tensor needs the same number of client streams")
        _dev_f32(out_denses[t], "out_dense")
        ptrs = (C.c_void_p * n_clients)(*[s.data_ptr() for s in streams_per_tensor[t]])
        keep.append(ptrs)
        descs[t].streams = ptrs
        descs[t].out_dense = out_denses[t].data_ptr()
        descs[t].numel = out_denses[t].numel()
        if sizes_per_tensor is not None:
            lens = (C.c_size_t * n_clients)(*[int(x) for x in sizes_per_tensor[t]])
            keep.append(lens)
            descs[t].stream_bytes = lens
    return descs, n_clients, keep


def sbc_workspace_bytes_batch(numels: Sequence[int], ps: Sequence[float]) -> int:
    n = len(numels)
    descs = (TensorDesc * n)()
    for t in range(n):
        descs[t].numel = int(numels[t])
        descs[t].p = float(ps[t])
    return int(lib().sbc_workspace_bytes_batch(n, descs))


class EncodeBatch:
    """The marshalled descriptors of a batch, built once and reused every round (same tensors)."""

    def __init__(self, updates, residuals, ps, out_streams, out_mus, workspace):
        self.n = len(updates)
        self.descs = _tensor_descs(updates, residuals, ps, out_streams, out_mus)
        self.keep = (list(updates), list(residuals), list(out_streams), list(out_mus), workspace)
        self.ws_ptr, self.ws_bytes = workspace.data_ptr(), workspace.numel()

    def run(self, stream=None) -> None:
        _check(lib().sbc_encode_batch(self.n, self.descs, self.ws_ptr, self.ws_bytes, _cuda_stream(stream)),
               "sbc_encode_batch")


def sbc_encode_batch(updates: Sequence[torch.Tensor], residuals: Sequence[torch.Tensor], ps: Sequence[float],
                     out_streams: Sequence[torch.Tensor], out_mus: Sequence[torch.Tensor],
                     workspace: torch.Tensor, stream=None) -> None:
    """sbc_encode of every tensor of a round with one launch sequence for the whole batch."""
    EncodeBatch(updates, residuals, ps, out_streams, out_mus, workspace).run(stream)


class DecodeBatch:
    """The marshalled descriptors of a batched decode, built once and reused.  ``sizes_per_tensor``
    (readable bytes behind every stream) makes the decoder check each header against them."""

    def __init__(self, streams_per_tensor, out_denses, workspace, status=None, sizes_per_tensor=None):
        self.n = len(out_denses)
        self.descs, self.n_clients, keep = _decode_descs(streams_per_tensor, out_denses, sizes_per_tensor)
        self.keep = [streams_per_tensor, out_denses, workspace, status, keep]
        self.status_ptr = status.data_ptr() if status is not None else None
        self.ws_ptr, self.ws_bytes = workspace.data_ptr(), workspace.numel()

    def run(self, stream=None) -> None:
        _check(lib().sbc_decode_accumulate_batch(self.n, self.n_clients, self.descs, self.status_ptr,
                                                 self.ws_ptr, self.ws_bytes, _cuda_stream(stream)),
               "sbc_decode_accumulate_batch")


def sbc_decode_workspace_bytes_batch(n_tensors: int) -> int:
    return int(lib().sbc_decode_workspace_bytes_batch(n_tensors))


def sbc_decode_accumulate_batch(streams_per_tensor: Sequence[Sequence[torch.Tensor]],
                                out_denses: Sequence[torch.Tensor], workspace: torch.Tensor,
                                status: Optional[torch.Tensor] = None, stream=None, sizes_per_tensor=None) -> None:
    """out_denses[t][j] += mu for every client stream of every tensor t; one launch for the batch."""
    DecodeBatch(streams_per_tensor, out_denses, workspace, status, sizes_per_tensor).run(stream)


def sbc_encode_static(update: torch.Tensor, residual: torch.Tensor, p: float, out_stream: torch.Tensor,
                      out_mu: torch.Tensor, stream=None) -> None:
    """sbc_encode for callers that may not allocate: the scratch is a fixed array inside the
    library (one per GPU, shared by all calls -- do not overlap calls).  The caller passes every
    input and output; problems whose scratch exceeds STATIC_WORKSPACE_BYTES raise SBC_ECAPACITY."""
    _dev_f32(update, "update")
    _dev_f32(residual, "residual")
    code = lib().sbc_encode_static(update.data_ptr(), residual.data_ptr(), update.numel(), float(p),
                                   out_stream.data_ptr(), out_stream.numel(), out_mu.data_ptr(),
                                   _cuda_stream(stream))
    _check(code, "sbc_encode_static")


def sbc_encode_ex(update: torch.Tensor, residual: torch.Tensor, p: float, out_stream: torch.Tensor,
                  out_mu: torch.Tensor, workspace: torch.Tensor, marks: Sequence[torch.cuda.Event],
                  stream=None) -> None:
    """sbc_encode that also records the caller's CUDA events at the stage boundaries."""
    _dev_f32(update, "update")
    _dev_f32(residual, "residual")
    if len(marks) != MARK_COUNT:
        raise ValueError(f"need {MARK_COUNT} events")
    handles = (C.c_void_p * MARK_COUNT)(*[m.cuda_event for m in marks])
    code = lib().sbc_encode_ex(update.data_ptr(), residual.data_ptr(), update.numel(), float(p),
                               out_stream.data_ptr(), out_stream.numel(), out_mu.data_ptr(),
                               workspace.data_ptr(), workspace.numel(), _cuda_stream(stream), handles)
    _check(code, "sbc_encode_ex")


def sbc_encode_launches() -> int:
    return int(lib().sbc_encode_launches())


def sbc_decode_launches(n_clients: int) -> int:
    return int(lib().sbc_decode_launches(n_clients))


def sbc_debug_barrier_timeout(scratch: torch.Tensor, stream=None) -> None:
    """Enqueue the kernel whose barrier cannot be passed; scratch[1] then holds STATUS_TIMEOUT."""
    if not (scratch.is_cuda and scratch.dtype == torch.int32 and scratch.numel() >= 2):
        raise TypeError("scratch must be an int32 CUDA tensor of at least two elements")
    L = lib()
    L.sbc_debug_barrier_timeout.restype = C.c_int
    L.sbc_debug_barrier_timeout.argtypes = [C.c_void_p, C.c_void_p]
    _check(L.sbc_debug_barrier_timeout(scratch.data_ptr(), _cuda_stream(stream)), "sbc_debug_barrier_timeout")


def sbc_encode_diag_get(workspace: torch.Tensor, stream=None) -> EncodeDiag:
    d = EncodeDiag()
    _check(lib().sbc_encode_diag_get(workspace.data_ptr(), C.byref(d), _cuda_stream(stream)),
           "sbc_encode_diag_get")
    return d


def sbc_encode_host(update_host: torch.Tensor, update_dev: torch.Tensor, residual_dev: torch.Tensor,
                    p: float, out_stream_host: torch.Tensor, stream_dev: torch.Tensor,
                    workspace: torch.Tensor, stream=None) -> Tuple[int, float]:
    """Host-buffer encode; synchronises.  Returns (container bytes written, mu)."""
    nbytes, mu = C.c_size_t(), C.c_float()
    code = lib().sbc_encode_host(update_host.data_ptr(), update_dev.data_ptr(), residual_dev.data_ptr(),
                                 update_host.numel(), float(p), out_stream_host.data_ptr(),
                                 stream_dev.data_ptr(), min(stream_dev.numel(), out_stream_host.numel()),
                                 C.byref(nbytes), C.byref(mu), workspace.data_ptr(), workspace.numel(),
                                 _cuda_stream(stream))
    _check(code, "sbc_encode_host")
    return int(nbytes.value), float(mu.value)


def sbc_decode_accumulate_host(streams_host: Sequence[torch.Tensor], sizes: Sequence[int],
                               out_dense_host: torch.Tensor, dense_dev: torch.Tensor,
                               staging_dev: torch.Tensor, stream=None) -> int:
    """Host-buffer decode-and-sum into a zeroed tensor; synchronises.  Returns the status word."""
    nc = len(streams_host)
    ptrs = (C.c_void_p * max(nc, 1))(*[s.data_ptr() for s in streams_host])
    lens = (C.c_size_t * max(nc, 1))(*[int(x) for x in sizes])
    status = C.c_uint32()
    code = lib().sbc_decode_accumulate_host(ptrs, lens, nc, out_dense_host.data_ptr(), dense_dev.data_ptr(),
                                            dense_dev.numel(), staging_dev.data_ptr(), staging_dev.numel(),
                                            C.byref(status), _cuda_stream(stream))
    _check(code, "sbc_decode_accumulate_host")
    return int(status.value)


def sbc_stream_info_get(out_stream: torch.Tensor, stream=None, check: bool = True) -> StreamInfo:
    """Synchronise and read the container header.  With ``check`` a bad status raises."""
    info = StreamInfo()
    code = lib().sbc_stream_info_get(out_stream.data_ptr(), C.byref(info), _cuda_stream(stream))
    if check:
        _check(code, "sbc_stream_info_get")
    return info


def sbc_decode_accumulate(streams: Sequence[torch.Tensor], out_dense: torch.Tensor,
                          status: Optional[torch.Tensor] = None, stream=None,
                          sizes: Optional[Sequence[int]] = None) -> None:
    """Enqueue out_dense[j] += mu_c for every position j of every client stream c.  With ``sizes``
    (readable bytes behind every stream) the _sized entry point checks each header against them."""
    sbc_decode_apply(streams, 1.0, out_dense, None, status, stream, sizes, _plain=True)


def sbc_decode_apply(streams: Sequence[torch.Tensor], scale: float, weights: torch.Tensor,
                     momentum: Optional[torch.Tensor] = None, status: Optional[torch.Tensor] = None,
                     stream=None, sizes: Optional[Sequence[int]] = None, _plain: bool = False) -> None:
    """Enqueue weights[j] += scale * mu_c at every decoded position; momentum[j] = 0 there."""
    _dev_f32(weights, "weights")
    if momentum is not None:
        _dev_f32(momentum, "momentum")
    nc = len(streams)
    ptrs = (C.c_void_p * max(nc, 1))(*[s.data_ptr() for s in streams])
    st = status.data_ptr() if status is not None else None
    L = lib()
    if sizes is not None:
        if len(sizes) != nc:
            raise ValueError("one size per stream")
        lens = (C.c_size_t * max(nc, 1))(*[int(x) for x in sizes])
        if _plain:
            code = L.sbc_decode_accumulate_sized(ptrs, lens, nc, weights.data_ptr(), weights.numel(), st,
                                                 _cuda_stream(stream))
        else:
            code = L.sbc_decode_apply_sized(ptrs, lens, nc, float(scale), weights.data_ptr(),
                                            momentum.data_ptr() if momentum is not None else None,
                                            weights.numel(), st, _cuda_stream(stream))
    elif _plain:
        code = L.sbc_decode_accumulate(ptrs, nc, weights.data_ptr(), weights.numel(), st, _cuda_stream(stream))
    else:
        code = L.sbc_decode_apply(ptrs, nc, float(scale), weights.data_ptr(),
                                  momentum.data_ptr() if momentum is not None else None, weights.numel(), st,
                                  _cuda_stream(stream))
    _check(code, "sbc_decode_accumulate" if _plain else "sbc_decode_apply")


def sbc_stream_bytes_values(numel: int, p: float) -> int:
    return int(lib().sbc_stream_bytes_values(numel, p))


def sbc_encode_values(update: torch.Tensor, residual: torch.Tensor, p: float,
                      out_stream: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                      stream=None) -> torch.Tensor:
    """Gradient Dropping client step (top-p by magnitude, values sent); residual updated in place."""
    _dev_f32(update, "update")
    _dev_f32(residual, "residual")
    n = update.numel()
    if out_stream is None:
        out_stream = torch.empty(sbc_stream_bytes_values(n, p), dtype=torch.uint8, device=update.device)
    if workspace is None:
        workspace = torch.empty(sbc_workspace_bytes(n, p), dtype=torch.uint8, device=update.device)
    code = lib().sbc_encode_values(update.data_ptr(), residual.data_ptr(), n, float(p), out_stream.data_ptr(),
                                   out_stream.numel(), workspace.data_ptr(), workspace.numel(),
                                   _cuda_stream(stream))
    _check(code, "sbc_encode_values")
    return out_stream


def sbc_stream_bytes_sampled(numel: int, p: float) -> int:
    return int(lib().sbc_stream_bytes_sampled(numel, p))


def sbc_workspace_bytes_sampled(numel: int, p: float, sample_count: int) -> int:
    return int(lib().sbc_workspace_bytes_sampled(numel, p, sample_count))


def sbc_encode_sampled(update: torch.Tensor, residual: torch.Tensor, p: float, sample_idx: torch.Tensor,
                       out_stream: Optional[torch.Tensor] = None, out_mu: Optional[torch.Tensor] = None,
                       workspace: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """sbc_encode with the two thresholds taken from the caller's subsample (int32 CUDA positions)."""
    _dev_f32(update, "update")
    _dev_f32(residual, "residual")
    if not (sample_idx.is_cuda and sample_idx.dtype == torch.int32 and sample_idx.is_contiguous()):
        raise TypeError("sample_idx must be a contiguous int32 CUDA tensor")
    n, m = update.numel(), sample_idx.numel()
    dev = update.device
    if out_stream is None:
        out_stream = torch.empty(sbc_stream_bytes_sampled(n, p), dtype=torch.uint8, device=dev)
    if out_mu is None:
        out_mu = torch.empty(1, dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = torch.empty(sbc_workspace_bytes_sampled(n, p, m), dtype=torch.uint8, device=dev)
    code = lib().sbc_encode_sampled(update.data_ptr(), residual.data_ptr(), n, float(p), sample_idx.data_ptr(), m,
                                    out_stream.data_ptr(), out_stream.numel(), out_mu.data_ptr(),
                                    workspace.data_ptr(), workspace.numel(), _cuda_stream(stream))
    _check(code, "sbc_encode_sampled")
    return out_stream, out_mu
