"""ctypes/numpy wrapper around the C oracle (``sbc_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Argument marshalling and nothing else: every step
of the method runs in the C file, which follows the paper's Algorithms 1-4.
"""
import ctypes as C
from dataclasses import dataclass

import numpy as np

from . import build as _build

__all__ = [
    "kept_count", "golomb_b", "mean_position_bits", "accumulate", "topk",
    "exact_sum", "compress", "payload_bits_bound", "golomb_encode",
    "golomb_decode", "container_bytes", "stream_bytes", "encode",
    "decode_accumulate", "parse_header", "StreamHeader", "side_and_mu", "container", "decode_apply", "topk_abs", "stream_bytes_values", "encode_values", "encode_sampled",
    "HEADER_BYTES", "chunk_codewords", "CHUNK_ENTRY_BYTES", "MAGIC",
]

HEADER_BYTES = 64
CHUNK_ENTRY_BYTES = 16
MAGIC = 0x31434253

_lib = C.CDLL(_build.build())

_f32p = np.ctypeslib.ndpointer(dtype=np.float32, flags="C_CONTIGUOUS")
_i64p = np.ctypeslib.ndpointer(dtype=np.int64, flags="C_CONTIGUOUS")
_u8p = np.ctypeslib.ndpointer(dtype=np.uint8, flags="C_CONTIGUOUS")


def _sig(name, restype, *argtypes):
    fn = getattr(_lib, name)
    fn.restype = restype
    fn.argtypes = list(argtypes)
    return fn


_kept_count = _sig("sbc_oracle_kept_count", C.c_int64, C.c_int64, C.c_double)
_chunk_cw = _sig("sbc_oracle_chunk_codewords", C.c_uint32, C.c_int64)
_golomb_b = _sig("sbc_oracle_golomb_b", C.c_int, C.c_double)
_mean_bits = _sig("sbc_oracle_mean_position_bits", C.c_double, C.c_double, C.c_int)
_accumulate = _sig("sbc_oracle_accumulate", C.c_int, _f32p, _f32p, C.c_int64)
_topk = _sig("sbc_oracle_topk", C.c_int, _f32p, C.c_int64, C.c_int64, C.c_int, _i64p)
_exact_sum = _sig("sbc_oracle_exact_sum", C.c_double, _f32p, _i64p, C.c_int64)
_compress = _sig("sbc_oracle_compress", C.c_int, _f32p, C.c_int64, C.c_int64, _i64p,
                 C.POINTER(C.c_int), C.POINTER(C.c_float), C.POINTER(C.c_double),
                 C.POINTER(C.c_double))
_bits_bound = _sig("sbc_oracle_payload_bits_bound", C.c_uint64, C.c_int64, C.c_int64, C.c_int)
_g_encode = _sig("sbc_oracle_golomb_encode", C.c_uint64, _i64p, C.c_int64, C.c_int, _u8p, C.c_size_t)
_g_decode = _sig("sbc_oracle_golomb_decode", C.c_int64, _u8p, C.c_uint64, C.c_int, C.c_float,
                 _f32p, C.c_int64)
_container_bytes = _sig("sbc_oracle_container_bytes", C.c_size_t, C.c_int64, C.c_uint64)
_stream_bytes = _sig("sbc_oracle_stream_bytes", C.c_size_t, C.c_int64, C.c_double)
_encode = _sig("sbc_oracle_encode", C.c_int, _f32p, _f32p, C.c_int64, C.c_double, _u8p,
               C.c_size_t, C.POINTER(C.c_size_t), C.POINTER(C.c_float))
_side_mu = _sig("sbc_oracle_side_and_mu", None, C.c_double, C.c_double, C.c_int64, C.POINTER(C.c_int),
                C.POINTER(C.c_float), C.POINTER(C.c_double), C.POINTER(C.c_double))
_container = _sig("sbc_oracle_container", C.c_int, _i64p, C.c_int64, C.c_int64, C.c_int, C.c_int,
                  C.c_float, _u8p, C.c_size_t, C.POINTER(C.c_size_t))
_decode_acc = _sig("sbc_oracle_decode_accumulate", C.c_int, C.POINTER(C.c_void_p), C.c_int,
                   _f32p, C.c_int64)


def chunk_codewords(k: int) -> int:
    """Codewords per chunk-table entry of a message with k positions."""
    return int(_chunk_cw(int(k)))


def kept_count(n: int, p: float) -> int:
    return int(_kept_count(n, p))


def golomb_b(p: float) -> int:
    return int(_golomb_b(p))


def mean_position_bits(p: float, b: int) -> float:
    return float(_mean_bits(p, b))


def accumulate(update: np.ndarray, residual: np.ndarray) -> int:
    """residual <- fl32(residual + update) in place; returns 0 or -1 (non-finite)."""
    assert update.shape == residual.shape
    return int(_accumulate(update, residual, update.size))


def topk(a: np.ndarray, k: int, negate: bool = False) -> np.ndarray:
    out = np.empty(k, dtype=np.int64)
    rc = _topk(a, a.size, k, int(negate), out)
    if rc != 0:
        raise ValueError(f"sbc_oracle_topk failed: {rc}")
    return out


def exact_sum(a: np.ndarray, idx: np.ndarray) -> float:
    idx = np.ascontiguousarray(idx, dtype=np.int64)
    return float(_exact_sum(a, idx, idx.size))


def compress(a: np.ndarray, k: int):
    """Algorithm 2 + residual write-back on an accumulated tensor (in place).

    Returns (kept_sorted, side, mu32, mu_pos, mu_neg)."""
    kept = np.empty(k, dtype=np.int64)
    side, mu = C.c_int(), C.c_float()
    mp, mn = C.c_double(), C.c_double()
    rc = _compress(a, a.size, k, kept, C.byref(side), C.byref(mu), C.byref(mp), C.byref(mn))
    if rc != 0:
        raise ValueError(f"sbc_oracle_compress failed: {rc}")
    return kept, side.value, np.float32(mu.value), mp.value, mn.value


def payload_bits_bound(n: int, k: int, b: int) -> int:
    return int(_bits_bound(n, k, b))


def golomb_encode(sorted_idx, b: int, cap_bytes: int = None):
    """Algorithm 3.  Returns (payload bytes as np.uint8 array, nbits)."""
    idx = np.ascontiguousarray(sorted_idx, dtype=np.int64)
    if cap_bytes is None:
        last = int(idx[-1]) if idx.size else 0
        cap_bytes = (idx.size * (1 + b) + (last >> b) + 7) // 8 + 1
    buf = np.zeros(max(cap_bytes, 1), dtype=np.uint8)
    nbits = int(_g_encode(idx, idx.size, b, buf, cap_bytes))
    if nbits == 2**64 - 1:
        raise ValueError("payload capacity too small")
    return buf[: (nbits + 7) // 8].copy(), nbits


def golomb_decode(payload: np.ndarray, nbits: int, b: int, mu, dense: np.ndarray) -> int:
    """Algorithm 4: dense[j] += mu at each decoded position; returns the count."""
    payload = np.ascontiguousarray(payload, dtype=np.uint8)
    if payload.size == 0:
        payload = np.zeros(1, dtype=np.uint8)
    return int(_g_decode(payload, nbits, b, float(mu), dense, dense.size))


def container_bytes(k: int, nbits: int) -> int:
    return int(_container_bytes(k, nbits))


def stream_bytes(n: int, p: float) -> int:
    return int(_stream_bytes(n, p))


def encode(update: np.ndarray, residual: np.ndarray, p: float, cap: int = None):
    """One client step (Algorithm 1 client lines + Algorithms 2, 3).

    ``residual`` is updated in place.  Returns (stream bytes, mu32)."""
    n = update.size
    if cap is None:
        cap = stream_bytes(n, p)
    out = np.zeros(cap, dtype=np.uint8)
    out_len, mu = C.c_size_t(), C.c_float()
    rc = _encode(update, residual, n, p, out, cap, C.byref(out_len), C.byref(mu))
    if rc != 0:
        raise ValueError(f"sbc_oracle_encode failed: {rc}")
    return out[: out_len.value].copy(), np.float32(mu.value)


def side_and_mu(sum_top: float, sum_bottom: float, k: int):
    """Algorithm 2's decision from the two exact sums.  Returns (side, mu32, mu_pos, mu_neg)."""
    side, mu = C.c_int(), C.c_float()
    mp, mn = C.c_double(), C.c_double()
    _side_mu(sum_top, sum_bottom, k, C.byref(side), C.byref(mu), C.byref(mp), C.byref(mn))
    return side.value, np.float32(mu.value), mp.value, mn.value


def container(sorted_idx, n: int, p: float, side: int, mu) -> np.ndarray:
    """Header + chunk table + Algorithm 3 payload for an ascending position list."""
    idx = np.ascontiguousarray(sorted_idx, dtype=np.int64)
    cap = stream_bytes(n, p)
    out = np.zeros(cap, dtype=np.uint8)
    out_len = C.c_size_t()
    rc = _container(idx, idx.size, n, golomb_b(p), int(side), float(mu), out, cap, C.byref(out_len))
    if rc != 0:
        raise ValueError(f"sbc_oracle_container failed: {rc}")
    return out[: out_len.value].copy()


def decode_accumulate(streams, out_dense: np.ndarray) -> None:
    """Server sum: out_dense += decode(stream_c) for every client, in order."""
    arrs = [np.ascontiguousarray(s, dtype=np.uint8) for s in streams]
    ptrs = (C.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    rc = _decode_acc(ptrs, len(arrs), out_dense, out_dense.size)
    if rc != 0:
        raise ValueError(f"sbc_oracle_decode_accumulate failed: {rc}")


_decode_apply = _sig("sbc_oracle_decode_apply", C.c_int, C.POINTER(C.c_void_p), C.c_int, C.c_float,
                     _f32p, C.c_void_p, C.c_int64)


def decode_apply(streams, scale: float, weights: np.ndarray, momentum: np.ndarray = None) -> None:
    """weights += scale * sum of the decoded streams; momentum zeroed at transmitted positions."""
    arrs = [np.ascontiguousarray(s, dtype=np.uint8) for s in streams]
    ptrs = (C.c_void_p * max(len(arrs), 1))(*[a.ctypes.data for a in arrs])
    mom = momentum.ctypes.data if momentum is not None else None
    rc = _decode_apply(ptrs, len(arrs), float(scale), weights, mom, weights.size)
    if rc != 0:
        raise ValueError(f"sbc_oracle_decode_apply failed: {rc}")


_topk_abs = _sig("sbc_oracle_topk_abs", C.c_int, _f32p, C.c_int64, C.c_int64, _i64p)
_stream_bytes_values = _sig("sbc_oracle_stream_bytes_values", C.c_size_t, C.c_int64, C.c_double)
_encode_values = _sig("sbc_oracle_encode_values", C.c_int, _f32p, _f32p, C.c_int64, C.c_double, _u8p,
                      C.c_size_t, C.POINTER(C.c_size_t))


def topk_abs(a: np.ndarray, k: int) -> np.ndarray:
    out = np.empty(k, dtype=np.int64)
    if _topk_abs(a, a.size, k, out) != 0:
        raise ValueError("sbc_oracle_topk_abs failed")
    return out


def stream_bytes_values(n: int, p: float) -> int:
    return int(_stream_bytes_values(n, p))


def encode_values(update: np.ndarray, residual: np.ndarray, p: float) -> np.ndarray:
    """Gradient Dropping client step: ``residual`` updated in place; returns the stream bytes."""
    n = update.size
    cap = stream_bytes_values(n, p)
    out = np.zeros(cap, dtype=np.uint8)
    out_len = C.c_size_t()
    rc = _encode_values(update, residual, n, p, out, cap, C.byref(out_len))
    if rc != 0:
        raise ValueError(f"sbc_oracle_encode_values failed: {rc}")
    return out[: out_len.value].copy()


_u32p = np.ctypeslib.ndpointer(dtype=np.uint32, flags="C_CONTIGUOUS")
_encode_sampled = _sig("sbc_oracle_encode_sampled", C.c_int, _f32p, _f32p, C.c_int64, C.c_double, _u32p,
                       C.c_int64, _u8p, C.c_size_t, C.POINTER(C.c_size_t), C.POINTER(C.c_float))


def encode_sampled(update: np.ndarray, residual: np.ndarray, p: float, sample_idx: np.ndarray):
    """Client step with thresholds taken from the given subsample.  Returns (stream bytes, mu32)."""
    n = update.size
    k, b = kept_count(n, p), golomb_b(p)
    limit = min(n, 2 * k + 1024)
    cap = container_bytes(limit, limit * (1 + b) + 2 * (n >> b))
    out = np.zeros(cap, dtype=np.uint8)
    out_len, mu = C.c_size_t(), C.c_float()
    idx = np.ascontiguousarray(sample_idx, dtype=np.uint32)
    rc = _encode_sampled(update, residual, n, p, idx, idx.size, out, cap, C.byref(out_len), C.byref(mu))
    if rc != 0:
        raise ValueError(f"sbc_oracle_encode_sampled failed: {rc}")
    return out[: out_len.value].copy(), np.float32(mu.value)


@dataclass
class StreamHeader:
    magic: int
    version: int
    numel: int
    k: int
    nbits: int
    payload_offset: int
    b: int
    side: int
    mu: np.float32
    chunk_codewords: int
    n_chunks: int
    status: int


def parse_header(stream: np.ndarray) -> StreamHeader:
    """Unpack the 64-byte little-endian container header (layout only)."""
    h = np.ascontiguousarray(stream[:HEADER_BYTES], dtype=np.uint8)
    u32 = h.view("<u4")
    u64 = h.view("<u8")
    return StreamHeader(
        magic=int(u32[0]), version=int(u32[1]), numel=int(u64[1]), k=int(u64[2]),
        nbits=int(u64[3]), payload_offset=int(u64[4]), b=int(u32[10]), side=int(u32[11]),
        mu=h[48:52].view("<f4")[0], chunk_codewords=int(u32[13]), n_chunks=int(u32[14]),
        status=int(u32[15]),
    )
