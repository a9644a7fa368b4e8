"""Python face of the CPU oracle (plain C, see gemm_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the CPU-baseline leg of the
benchmark.  The CUDA library and its binding never import this package, and this package never
imports them.

The C source is compiled on first use (gcc, OpenMP, no fast-math, no FMA contraction) into
oracle/liboracle.so.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SO = _HERE / "liboracle.so"
_SRC = [_HERE / "gemm_oracle.c", _HERE / "gemm_l1_body.inc", _HERE / "conv_oracle.c"]

OR_F32, OR_F16, OR_BF16 = 0, 1, 2
ACC_F32, ACC_F32FMA, ACC_F64, ACC_F16 = 0, 1, 2, 3

# default blocking of the L1 layer: the 8 x 12 micro-kernel of Section III and kc = 512 (Section IV-A);
# mc and nc are free parameters (the paper takes them from a cache model it only cites)
DEFAULT_BLOCKING = dict(mr=8, nr=12, mc=120, kc=512, nc=3072)


def build(force: bool = False) -> Path:
    """Compile the oracle's C source into liboracle.so (idempotent)."""
    if not force and _SO.exists() and all(_SO.stat().st_mtime >= s.stat().st_mtime for s in _SRC):
        return _SO
    cmd = ["gcc", "-O3", "-march=x86-64-v3", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
           "-shared", "-fPIC", "-o", str(_SO), str(_SRC[0]), str(_SRC[2]), "-lm"]
    subprocess.run(cmd, check=True, cwd=str(_HERE))
    return _SO


class ConvGeom(ctypes.Structure):
    """Geometry of a convolution layer (conv_oracle.c): NHWC activations, kh x kw filters, strides, zero padding."""
    _fields_ = [("batch", ctypes.c_int64), ("h", ctypes.c_int64), ("w", ctypes.c_int64), ("c_in", ctypes.c_int64),
                ("c_out", ctypes.c_int64), ("kh", ctypes.c_int32), ("kw", ctypes.c_int32),
                ("stride_h", ctypes.c_int32), ("stride_w", ctypes.c_int32), ("pad_h", ctypes.c_int32),
                ("pad_w", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(str(_SO))
        i64, dbl, vp, ci = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int
        L.oracle_decode_f16.restype = dbl
        L.oracle_decode_f16.argtypes = [ctypes.c_uint16]
        L.oracle_decode_bf16.restype = dbl
        L.oracle_decode_bf16.argtypes = [ctypes.c_uint16]
        L.oracle_round_f16.restype = dbl
        L.oracle_round_f16.argtypes = [dbl]
        L.oracle_gemm_l0.restype = ci
        L.oracle_gemm_l0.argtypes = [ci, ci, ci, ci, i64, i64, i64, dbl, vp, i64, vp, i64,
                                     dbl, vp, i64, vp, vp, i64]
        L.oracle_gemm_samples_f64.restype = ci
        L.oracle_gemm_samples_f64.argtypes = [ci, ci, ci, i64, dbl, vp, i64, vp, i64, dbl, vp, i64,
                                              i64, vp, vp, vp]
        L.oracle_freivalds.restype = ci
        L.oracle_freivalds.argtypes = [ci, ci, ci, i64, i64, i64, dbl, vp, i64, vp, i64, dbl,
                                       vp, i64, vp, i64, vp, vp, vp]
        L.oracle_gemm_l1.restype = ci
        L.oracle_gemm_l1.argtypes = [ci, ci, ci, ci, i64, i64, i64, dbl, vp, i64, vp, i64, dbl,
                                     vp, i64, ci, ci, ci, ci, ci, ci]
        L.oracle_pack_A_f32.restype = ci
        L.oracle_pack_A_f32.argtypes = [ci, ci, vp, i64, i64, i64, i64, i64, ci, vp]
        L.oracle_pack_B_f32.restype = ci
        L.oracle_pack_B_f32.argtypes = [ci, ci, vp, i64, i64, i64, i64, i64, ci, vp]
        L.oracle_ukernel_f32.restype = ci
        L.oracle_ukernel_f32.argtypes = [ci, ci, i64, ctypes.c_float, vp, vp, ctypes.c_float, vp, ci]
        L.oracle_num_threads.restype = ci
        gp = ctypes.POINTER(ConvGeom)
        L.oracle_conv_out_h.restype = i64
        L.oracle_conv_out_h.argtypes = [gp]
        L.oracle_conv_out_w.restype = i64
        L.oracle_conv_out_w.argtypes = [gp]
        L.oracle_conv2d_direct.restype = ci
        L.oracle_conv2d_direct.argtypes = [ci, gp, dbl, vp, vp, i64, dbl, vp, i64, vp, i64]
        L.oracle_conv2d_samples_f64.restype = ci
        L.oracle_conv2d_samples_f64.argtypes = [ci, gp, dbl, vp, vp, i64, dbl, vp, i64, i64, vp, vp, vp]
        L.oracle_im2row.restype = ci
        L.oracle_im2row.argtypes = [ci, gp, vp, vp, i64]
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _ptr(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _t(flag: str) -> int:
    f = flag.upper()
    if f == "N":
        return 0
    if f in ("T", "C"):
        return 1
    raise ValueError(f"bad trans flag {flag!r}")


def _check_buf(buf: np.ndarray, dtype: int):
    want = np.float32 if dtype == OR_F32 else np.uint16
    if buf.dtype != want or not buf.flags.c_contiguous:
        raise TypeError("operand buffer has the wrong element type or is not contiguous")


def decode_f16(bits: int) -> float:
    return float(lib().oracle_decode_f16(int(bits)))


def decode_bf16(bits: int) -> float:
    return float(lib().oracle_decode_bf16(int(bits)))


def gemm_l0(dtype, transA, transB, m, n, k, alpha, A, lda, B, ldb, beta, C0, ldc0, acc=ACC_F64):
    """Definition of the operation, one dot product per entry.  Returns an m x n array
    (float64 for ACC_F64 and ACC_F16, float32 otherwise), F-ordered with leading dimension max(1, m).
    ACC_F16: the dot products are accumulated in binary16 (one fused multiply-add and one rounding per k: the
    paper's f16 arithmetic), then alpha*sum + beta*C0 is formed in double."""
    _check_buf(A, dtype), _check_buf(B, dtype)
    ldc = max(1, m)
    if acc in (ACC_F64, ACC_F16):
        out = np.zeros(ldc * n, dtype=np.float64)
        c64, c32 = out, None
    else:
        out = np.zeros(ldc * n, dtype=np.float32)
        c64, c32 = None, out
    if C0 is not None and C0.dtype != np.float32:
        raise TypeError("C0 must be float32")
    rc = lib().oracle_gemm_l0(dtype, acc, _t(transA), _t(transB), m, n, k, float(alpha), _ptr(A), lda,
                              _ptr(B), ldb, float(beta), _ptr(C0), ldc0, _ptr(c64), _ptr(c32), ldc)
    if rc != 0:
        raise RuntimeError(f"oracle_gemm_l0 failed: {rc}")
    return out.reshape(n, ldc).T[:m, :]


def round_f16(x: float) -> float:
    """Nearest binary16 number to x (ties to even), as a float; the rounding step of the ACC_F16 accumulation."""
    return float(lib().oracle_round_f16(float(x)))


def gemm_l1(dtype, transA, transB, m, n, k, alpha, A, lda, B, ldb, beta, C0, ldc0, acc=ACC_F32,
            paper_scaling=False, **blocking):
    """The blocked, packed algorithm (loops L1-L5 + packing + micro-kernel).  Returns m x n
    (float32 for ACC_F32, float64 for ACC_F64)."""
    _check_buf(A, dtype), _check_buf(B, dtype)
    blk = dict(DEFAULT_BLOCKING)
    blk.update(blocking)
    ldc = max(1, m)
    np_t = np.float32 if acc == ACC_F32 else np.float64
    C = np.zeros(ldc * n, dtype=np_t)
    if beta != 0.0:
        c0 = C0.reshape(n, ldc0).T[:m, :]
        C.reshape(n, ldc).T[:m, :] = c0.astype(np_t)
    else:
        C[:] = np.nan    # must never be read when beta == 0
    rc = lib().oracle_gemm_l1(dtype, acc, _t(transA), _t(transB), m, n, k, float(alpha), _ptr(A), lda,
                              _ptr(B), ldb, float(beta), _ptr(C), ldc,
                              blk["mr"], blk["nr"], blk["mc"], blk["kc"], blk["nc"], int(bool(paper_scaling)))
    if rc != 0:
        raise RuntimeError(f"oracle_gemm_l1 failed: {rc}")
    return C.reshape(n, ldc).T[:m, :]


def gemm_samples_f64(dtype, transA, transB, k, alpha, A, lda, B, ldb, beta, C0, ldc0, rows, cols):
    """fp64 values of the entries (rows[t], cols[t])."""
    _check_buf(A, dtype), _check_buf(B, dtype)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    out = np.zeros(rows.size, dtype=np.float64)
    rc = lib().oracle_gemm_samples_f64(dtype, _t(transA), _t(transB), k, float(alpha), _ptr(A), lda,
                                       _ptr(B), ldb, float(beta), _ptr(C0), ldc0, rows.size,
                                       _ptr(rows), _ptr(cols), _ptr(out))
    if rc != 0:
        raise RuntimeError(f"oracle_gemm_samples_f64 failed: {rc}")
    return out


def freivalds(dtype, transA, transB, m, n, k, alpha, A, lda, B, ldb, beta, C0, ldc0, C, ldc, x):
    """(resid, scale) of the randomised whole-matrix check for probe vector x (length n, fp64)."""
    _check_buf(A, dtype), _check_buf(B, dtype)
    x = np.ascontiguousarray(x, dtype=np.float64)
    resid = np.zeros(max(1, m), dtype=np.float64)
    scale = np.zeros(max(1, m), dtype=np.float64)
    rc = lib().oracle_freivalds(dtype, _t(transA), _t(transB), m, n, k, float(alpha), _ptr(A), lda,
                                _ptr(B), ldb, float(beta), _ptr(C0), ldc0, _ptr(C), ldc,
                                _ptr(x), _ptr(resid), _ptr(scale))
    if rc != 0:
        raise RuntimeError(f"oracle_freivalds failed: {rc}")
    return resid[:m], scale[:m]


def pack_A_f32(dtype, transA, A, lda, ic, pc, mcb, kcb, mr):
    npan = (mcb + mr - 1) // mr
    out = np.full(npan * kcb * mr, np.nan, dtype=np.float32)
    lib().oracle_pack_A_f32(dtype, _t(transA), _ptr(A), lda, ic, pc, mcb, kcb, mr, _ptr(out))
    return out.reshape(npan, kcb, mr)


def pack_B_f32(dtype, transB, B, ldb, pc, jc, kcb, ncb, nr):
    npan = (ncb + nr - 1) // nr
    out = np.full(npan * kcb * nr, np.nan, dtype=np.float32)
    lib().oracle_pack_B_f32(dtype, _t(transB), _ptr(B), ldb, pc, jc, kcb, ncb, nr, _ptr(out))
    return out.reshape(npan, kcb, nr)


def ukernel_f32(mr, nr, kc, alpha, Ac, Bc, beta, C, paper_scaling=False):
    """Micro-kernel with the signature of Fig. 3.  Ac: [kc, mr], Bc: [kc, nr], C: [nr, mr] float32;
    returns the updated C."""
    Ac = np.ascontiguousarray(Ac, dtype=np.float32)
    Bc = np.ascontiguousarray(Bc, dtype=np.float32)
    C = np.array(C, dtype=np.float32, order="C", copy=True)
    assert Ac.shape == (kc, mr) and Bc.shape == (kc, nr) and C.shape == (nr, mr)
    rc = lib().oracle_ukernel_f32(mr, nr, kc, float(alpha), _ptr(Ac), _ptr(Bc), float(beta), _ptr(C),
                                  int(bool(paper_scaling)))
    if rc != 0:
        raise RuntimeError("oracle_ukernel_f32 failed")
    return C


def fp32_tolerance(k, alpha, beta, max_a, max_b, max_c0):
    """Absolute bound for fp32 GEMM results: 4 * 2^-24 * (k |alpha| max|A| max|B| + |beta| max|C0|).
    At alpha = 1, beta = 0 this is the bound 4 k 2^-24 max|A| max|B|."""
    return 4.0 * 2.0 ** -24 * (k * abs(alpha) * max_a * max_b + abs(beta) * max_c0)


# ---------------------------------------------------------------- convolution layers lowered with im2row (conv_oracle.c)

def conv_geom(batch, h, w, c_in, c_out, kh, kw, stride_h=1, stride_w=1, pad_h=0, pad_w=0) -> ConvGeom:
    return ConvGeom(batch, h, w, c_in, c_out, kh, kw, stride_h, stride_w, pad_h, pad_w)


def conv_out_hw(g: ConvGeom):
    return int(lib().oracle_conv_out_h(ctypes.byref(g))), int(lib().oracle_conv_out_w(ctypes.byref(g)))


def conv2d_direct(dtype, g: ConvGeom, alpha, X, Wt, ldw, beta=0.0, Y0=None, ldy0=0):
    """Definition of the layer in fp64.  Returns a C_out x pixels float64 array (pixels in (b, ho, wo) order)."""
    _check_buf(X, dtype), _check_buf(Wt, dtype)
    ho, wo = conv_out_hw(g)
    npix = g.batch * ho * wo
    ldo = max(1, g.c_out)
    out = np.zeros(ldo * npix, dtype=np.float64)
    rc = lib().oracle_conv2d_direct(dtype, ctypes.byref(g), float(alpha), _ptr(X), _ptr(Wt), ldw, float(beta),
                                    _ptr(Y0), ldy0, _ptr(out), ldo)
    if rc != 0:
        raise RuntimeError(f"oracle_conv2d_direct failed: {rc}")
    return out.reshape(npix, ldo).T[:g.c_out, :]


def conv2d_samples_f64(dtype, g: ConvGeom, alpha, X, Wt, ldw, beta, Y0, ldy0, rows, cols):
    """fp64 values of the output entries (channel rows[t], pixel cols[t])."""
    _check_buf(X, dtype), _check_buf(Wt, dtype)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    out = np.zeros(rows.size, dtype=np.float64)
    rc = lib().oracle_conv2d_samples_f64(dtype, ctypes.byref(g), float(alpha), _ptr(X), _ptr(Wt), ldw, float(beta),
                                         _ptr(Y0), ldy0, rows.size, _ptr(rows), _ptr(cols), _ptr(out))
    if rc != 0:
        raise RuntimeError(f"oracle_conv2d_samples_f64 failed: {rc}")
    return out


def im2row(dtype, g: ConvGeom, X, ld=None):
    """The lowered activation matrix: buffer of the k x pixels column-major matrix (leading dimension ld >= k) in
    the element type of X; column j is the patch of output pixel j in (r, s, c) order."""
    _check_buf(X, dtype)
    ho, wo = conv_out_hw(g)
    k = g.kh * g.kw * g.c_in
    ld = k if ld is None else ld
    out = np.zeros(ld * g.batch * ho * wo, dtype=X.dtype)
    rc = lib().oracle_im2row(dtype, ctypes.byref(g), _ptr(X), _ptr(out), ld)
    if rc != 0:
        raise RuntimeError(f"oracle_im2row failed: {rc}")
    return out
