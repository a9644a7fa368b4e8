"""Counter-based seeded matrix generator.

Every element is a pure function of (seed, matrix_id, logical linear index), so
a matrix has the same logical contents whatever its leading dimension, and the
CPU oracle and the CUDA path are always handed the very same host arrays.

The generator is SplitMix64 (Steele, Lea, Flood 2014: add the golden-ratio
increment, then the 3-step xor-shift-multiply finaliser) used in counter mode.
No GEMM arithmetic lives here.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

DTYPE_F32 = 0
DTYPE_F16 = 1
DTYPE_BF16 = 2
DTYPE_NAMES = {DTYPE_F32: "f32", DTYPE_F16: "f16", DTYPE_BF16: "bf16"}

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22

# canaries written into the padding rows (ld > rows); a kernel that reads or
# multiplies them poisons its result, one that writes them is caught by the tests
CANARY_F32 = np.uint32(0x7FC0DEAD)   # quiet NaN with a payload
CANARY_16 = np.uint16(0x7FFF)        # NaN in both fp16 and bf16


def _gen_threads() -> int:
    try:
        return max(1, min(32, len(os.sched_getaffinity(0))))
    except AttributeError:
        return max(1, min(32, os.cpu_count() or 1))


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _stream_key(seed: int, matrix_id: int) -> np.uint64:
    s = np.array([seed & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
    t = np.array([(matrix_id + 1) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
    return _mix(_mix(s + _GOLDEN) ^ (t * _GOLDEN))[0]


def raw_u64(seed: int, matrix_id: int, start: int, count: int) -> np.ndarray:
    """`count` 64-bit words for counters start .. start+count-1 of one stream."""
    key = _stream_key(seed, matrix_id)
    ctr = np.arange(start, start + count, dtype=np.uint64)
    return _mix(key + (ctr + np.uint64(1)) * _GOLDEN)


def _uniform_pm1(bits: np.ndarray) -> np.ndarray:
    # top 24 bits -> u * 2^-23 - 1 in [-1, 1): every value is an fp32 number
    u = (bits >> np.uint64(40)).astype(np.float64)
    return u * (2.0 ** -23) - 1.0


def _unit_open(bits: np.ndarray) -> np.ndarray:
    # 53-bit uniform in (0, 1]
    return ((bits >> np.uint64(11)).astype(np.float64) + 1.0) * (2.0 ** -53)


def _values(kind: str, seed: int, matrix_id: int, start: int, count: int,
            rows: int, scale: float) -> np.ndarray:
    """fp64 values of logical elements start..start+count-1 (column-major order)."""
    if kind == "uniform":
        return _uniform_pm1(raw_u64(seed, matrix_id, start, count))
    if kind in ("normal", "absnormal"):
        w = raw_u64(seed, matrix_id, 2 * start, 2 * count)
        u1 = _unit_open(w[0::2])
        u2 = _unit_open(w[1::2])
        z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        if kind == "absnormal":
            z = np.abs(z)
        return z * scale
    if kind == "int":
        r = raw_u64(seed, matrix_id, start, count) >> np.uint64(33)
        return (r % np.uint64(9)).astype(np.float64) - 4.0
    if kind == "ones":
        return np.ones(count, dtype=np.float64)
    if kind == "index":
        return np.arange(start, start + count, dtype=np.float64)
    if kind == "identity":
        idx = np.arange(start, start + count, dtype=np.int64)
        return ((idx % rows) == (idx // rows)).astype(np.float64)
    if kind == "zeros":
        return np.zeros(count, dtype=np.float64)
    raise ValueError(f"unknown value kind {kind!r}")


def encode_f16(x: np.ndarray) -> np.ndarray:
    """Round fp64/fp32 values to IEEE binary16 (nearest-even); returns uint16 bit patterns."""
    return np.asarray(x).astype(np.float16).view(np.uint16)


def encode_bf16(x: np.ndarray) -> np.ndarray:
    """Round values to bfloat16 (nearest-even) from their fp32 image; uint16 bit patterns.

    fp64 inputs are first rounded to fp32; every value the generators produce is
    either exactly an fp32 number or a continuous sample, for which the double
    rounding changes nothing that matters to the tests (both sides see the
    already-encoded bits).
    """
    f = np.ascontiguousarray(np.asarray(x, dtype=np.float32))
    b = f.view(np.uint32)
    nan = np.isnan(f)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = ((b + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)
    r[nan] = np.uint16(0x7FC0)
    return r


def decode_16(bits: np.ndarray, dtype: int) -> np.ndarray:
    """Exact fp64 image of fp16/bf16 bit patterns (test convenience; the oracle has its own decoder)."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if dtype == DTYPE_F16:
        return bits.view(np.float16).astype(np.float64)
    if dtype == DTYPE_BF16:
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    raise ValueError("decode_16 wants a 16-bit dtype")


@dataclass
class Matrix:
    """A column-major stored matrix: element (i, j) is buf[i + j*ld]."""
    buf: np.ndarray      # 1-D, float32 (f32) or uint16 bit patterns (f16/bf16), length ld*cols
    rows: int
    cols: int
    ld: int
    dtype: int

    def window(self) -> np.ndarray:
        """rows x cols view of the stored elements (no padding rows)."""
        return self.buf.reshape(self.cols, self.ld).T[: self.rows, :]

    def padding(self) -> np.ndarray:
        return self.buf.reshape(self.cols, self.ld).T[self.rows:, :]

    def as_f64(self) -> np.ndarray:
        w = self.window()
        if self.dtype == DTYPE_F32:
            return w.astype(np.float64)
        return decode_16(np.ascontiguousarray(w), self.dtype)

    def max_abs(self) -> float:
        return float(np.max(np.abs(self.as_f64()))) if self.rows * self.cols else 0.0

    def copy(self) -> "Matrix":
        return Matrix(self.buf.copy(), self.rows, self.cols, self.ld, self.dtype)

    def padding_intact(self) -> bool:
        p = self.padding()
        if p.size == 0:
            return True
        if self.dtype == DTYPE_F32:
            return bool(np.all(np.ascontiguousarray(p).view(np.uint32) == CANARY_F32))
        return bool(np.all(p == CANARY_16))


def make_matrix(rows: int, cols: int, *, kind: str, seed: int, matrix_id: int,
                dtype: int = DTYPE_F32, ld: int | None = None, scale: float = 1.0) -> Matrix:
    """Generate a stored rows x cols matrix (column-major, leading dimension ld >= max(1, rows)).

    kind: 'uniform' U[-1,1) on a 2^-23 grid | 'normal' N(0, scale^2) | 'absnormal' |N(0,1)|*scale |
          'int' integers in [-4,4] | 'ones' | 'zeros' | 'identity' | 'index' (its own linear index).
    Values are produced in fp64 and rounded once to `dtype`.
    """
    ld = max(1, rows) if ld is None else ld
    if ld < max(1, rows):
        raise ValueError("ld < rows")
    np_dt = np.float32 if dtype == DTYPE_F32 else np.uint16
    buf = np.empty(ld * cols, dtype=np_dt)
    view = buf.reshape(cols, ld)
    if dtype == DTYPE_F32:
        view.view(np.uint32)[:, rows:] = CANARY_F32
    else:
        view[:, rows:] = CANARY_16
    n = rows * cols
    if n == 0:
        return Matrix(buf, rows, cols, ld, dtype)
    dense = np.empty(n, dtype=np_dt)

    def fill(s):      # chunks are independent (counter-based generator): any order, any number of threads
        c = min(_CHUNK, n - s)
        v = _values(kind, seed, matrix_id, s, c, rows, scale)
        if dtype == DTYPE_F32:
            dense[s:s + c] = v.astype(np.float32)
        elif dtype == DTYPE_F16:
            dense[s:s + c] = encode_f16(v)
        else:
            dense[s:s + c] = encode_bf16(v)

    starts = range(0, n, _CHUNK)
    workers = min(len(starts), _gen_threads())
    if workers <= 1:
        for s in starts:
            fill(s)
    else:             # numpy releases the interpreter lock inside its array loops
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(fill, starts))
    view[:, :rows] = dense.reshape(cols, rows)
    return Matrix(buf, rows, cols, ld, dtype)
