"""CPU oracle for the dual-sparse decode product (Celty, Sections 3.1-3.3).

TEST INFRASTRUCTURE ONLY: used by the tests, by the smoke check and by the benchmark's
cpu_baseline leg.  The CUDA library and its binding never import this module, and this
module imports nothing from them.  All arithmetic is fp64 (products of two FP16 numbers
are exact in fp64); decisions that produce integers (which activations survive the
threshold) are taken in fp32, the precision the method itself uses.

Functions and the passage each follows:

  keep_flags, compact     magnitude thresholding of the activation vector (Sections 1, 2.1)
                          and the column skip on zero activations (Section 3.1).
  masked_gemv             plain definition of y = W.x over kept weights and surviving
                          activations (Section 3.1); the method is exact, so this is the result.
  rlc_encode              n-bit run-length coded CSC, Section 3.2 (worked example there).
  rlc_decode_rows         Algorithm 1 as what it computes, plus the ordinal (Section 3.3).
  spmspv_rlc              decode + scatter-accumulate from the encoded arrays (Section 3.3).
  rlc_encode_column_py    the same encoding rule as a literal Python loop over one column,
                          for tiny cases and for replaying the printed example.
  silu, swiglu, to_half,  the element-wise step between the gate/up projections and the down
  swiglu_epilogue         projection of a decode layer (Section 6.2 runs the seven products of a LLaMA-2
                          layer; the MLP's activation is SiLU(gate) * up): plain definition in fp64, one
                          rounding to FP16 (nearest, ties to even), then the thresholded list.

Every function here is pinned by tests that do not call it to produce their expectation
(printed example, hand-derived vectors, closed forms, invariants, brute force).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "celty_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C half of the oracle with gcc (OpenMP for the timed dense product)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        P, I64, I32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        lib.orc_half_to_double.restype = ctypes.c_double
        lib.orc_half_to_double.argtypes = [ctypes.c_uint16]
        lib.orc_max_threads.restype = I32
        lib.orc_masked_gemv.restype = None
        lib.orc_masked_gemv.argtypes = [P, I64, P, I64, I64, I64, P, P, P, P, I32]
        lib.orc_rlc_count.restype = I64
        lib.orc_rlc_count.argtypes = [P, I64, I64, I64, I32, I64, P]
        lib.orc_rlc_fill.restype = None
        lib.orc_rlc_fill.argtypes = [P, I64, P, I64, I64, I64, I32, I64, P, P, P, P]
        lib.orc_rlc_decode_rows.restype = None
        lib.orc_rlc_decode_rows.argtypes = [P, P, I64, I64, I64, P]
        lib.orc_spmspv_rlc.restype = None
        lib.orc_spmspv_rlc.argtypes = [P, P, P, I64, I64, I64, P, P, P, P]
        _lib = lib
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _bits(a) -> np.ndarray:
    """FP16 array (or its uint16 bit patterns) -> contiguous uint16 bit patterns."""
    a = np.asarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("expected float16 values or uint16 bit patterns")
    return np.ascontiguousarray(a)


def max_threads() -> int:
    return int(_load().orc_max_threads())


def half_to_double(bits: int) -> float:
    return float(_load().orc_half_to_double(int(bits)))


# ----------------------------------------------------------------------------- thresholding
def keep_flags(x, tau: float) -> np.ndarray:
    """Activation j survives iff not(|x_j| <= tau), compared in fp32 (FP16 widens exactly).

    Magnitude thresholding, Sections 1 and 2.1.  The strict comparison makes tau = 0 drop
    exactly the zeros, which is the test the kernel of Section 3.1 applies; NaN survives.
    """
    xf = _bits(x).view(np.float16).astype(np.float32)
    with np.errstate(invalid="ignore"):
        return np.logical_not(np.abs(xf) <= np.float32(tau)).astype(np.uint8)


def compact(x, tau: float):
    """Surviving column list in ascending order: (idx int32, val uint16 bit patterns, n)."""
    xb = _bits(x)
    idx = np.flatnonzero(keep_flags(xb, tau)).astype(np.int32)
    return idx, xb[idx].copy(), int(idx.size)


# ----------------------------------------------------------------------------- plain product
def masked_gemv(W, mask, x, tau: float, threads: int = 1):
    """y_ref and a_ref = sum |W_ij x_j| in fp64 by the plain definition (Section 3.1)."""
    Wb = _bits(W)
    M, K = Wb.shape
    mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    assert mask.shape == (M, K)
    xb = _bits(x)
    assert xb.shape == (K,)
    keep = keep_flags(xb, tau)
    y = np.empty(M, np.float64)
    a = np.empty(M, np.float64)
    _load().orc_masked_gemv(_p(Wb), K, _p(mask), K, M, K, _p(xb), _p(keep), _p(y), _p(a),
                            int(threads))
    return y, a


# ----------------------------------------------------------------------------- format
def rlc_encode(W, mask, run_bits: int = 4, tile_rows: int = 0):
    """Encode a masked matrix into RLC-CSC (Section 3.2).

    Returns a namespace with
      block_ptr  int64[K*T+1]  entries before block b = j*T + t (row tile t of column j)
      vals       uint16[n]     FP16 bit patterns (+0 for pads)
      runs       uint8[n]      one run per stored entry, each in [0, 2^run_bits - 1]
      is_pad     uint8[n]
      rows       int32[n]      decoded absolute row of every entry (rlc_decode_rows)
    """
    Wb = _bits(W)
    M, K = Wb.shape
    mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    assert mask.shape == (M, K)
    T = (M + tile_rows - 1) // tile_rows if tile_rows > 0 else 1
    lib = _load()
    block_ptr = np.zeros(K * T + 1, np.int64)
    n = lib.orc_rlc_count(_p(mask), K, M, K, run_bits, tile_rows, _p(block_ptr))
    vals = np.zeros(n, np.uint16)
    runs = np.zeros(n, np.uint8)
    is_pad = np.zeros(n, np.uint8)
    lib.orc_rlc_fill(_p(Wb), K, _p(mask), K, M, K, run_bits, tile_rows, _p(block_ptr),
                     _p(vals), _p(runs), _p(is_pad))
    enc = SimpleNamespace(M=M, K=K, T=T, run_bits=run_bits, tile_rows=tile_rows,
                          block_ptr=block_ptr, vals=vals, runs=runs, is_pad=is_pad)
    enc.rows = rlc_decode_rows(enc)
    return enc


def rlc_count(mask, run_bits: int = 4, tile_rows: int = 0) -> np.ndarray:
    """block_ptr alone (stored entries before each block, Section 3.2's rule), without building the arrays:
    the counting pass of rlc_encode, for byte accounting on large masks."""
    mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    M, K = mask.shape
    T = (M + tile_rows - 1) // tile_rows if tile_rows > 0 else 1
    block_ptr = np.zeros(K * T + 1, np.int64)
    _load().orc_rlc_count(_p(mask), K, M, K, run_bits, tile_rows, _p(block_ptr))
    return block_ptr


def rlc_decode_rows(enc) -> np.ndarray:
    rows = np.zeros(enc.vals.size, np.int32)
    _load().orc_rlc_decode_rows(_p(enc.runs), _p(enc.block_ptr), enc.K, enc.M, enc.tile_rows,
                                _p(rows))
    return rows


def rlc_to_dense(enc) -> np.ndarray:
    """Dense M x K uint16 matrix rebuilt from the non-pad entries (+0 elsewhere)."""
    out = np.zeros((enc.M, enc.K), np.uint16)
    col_of_block = np.repeat(np.arange(enc.K * enc.T) // enc.T, np.diff(enc.block_ptr))
    real = enc.is_pad == 0
    out[enc.rows[real], col_of_block[real]] = enc.vals[real]
    return out


def column_entries(enc, j: int):
    """(rows, vals, is_pad, runs) of column j, all its row tiles concatenated."""
    b0, b1 = enc.block_ptr[j * enc.T], enc.block_ptr[(j + 1) * enc.T]
    return enc.rows[b0:b1], enc.vals[b0:b1], enc.is_pad[b0:b1], enc.runs[b0:b1]


def spmspv_rlc(enc, x, tau: float):
    """y and sum-of-magnitudes from the encoded arrays (decode, scatter; Section 3.3)."""
    xb = _bits(x)
    keep = keep_flags(xb, tau)
    y = np.empty(enc.M, np.float64)
    a = np.empty(enc.M, np.float64)
    _load().orc_spmspv_rlc(_p(enc.vals), _p(enc.rows), _p(enc.block_ptr), enc.K, enc.M,
                           enc.tile_rows, _p(xb), _p(keep), _p(y), _p(a))
    return y, a


# ----------------------------------------------------------------------------- MLP element-wise step
def silu(v) -> np.ndarray:
    """SiLU(v) = v / (1 + exp(-v)) in fp64 (the activation of the LLaMA MLP whose products Section 6.2 times)."""
    v = np.asarray(v, dtype=np.float64)
    with np.errstate(over="ignore"):
        return v / (1.0 + np.exp(-v))


def swiglu(gate, up) -> np.ndarray:
    """SiLU(gate) * up, element by element, fp64."""
    return silu(gate) * np.asarray(up, dtype=np.float64)


def to_half(v) -> np.ndarray:
    """fp64 -> FP16 bit patterns, one rounding, to nearest with ties to even; beyond the largest finite
    value (65520 and up) the result is infinity."""
    with np.errstate(over="ignore"):
        return np.asarray(v, dtype=np.float64).astype(np.float16).view(np.uint16)


def swiglu_epilogue(y, tau: float):
    """The step between the stacked [gate; up] product and the down projection.

    y holds the 2I results of the stacked product, gate rows first: h_i = SiLU(y_i) * y_{I+i} in fp64,
    rounded once to FP16; the list keeps i iff not(|h_i| <= tau) on the rounded value (compared in fp32,
    like every thresholding decision here).  Returns (h FP16 bit patterns, idx int32 ascending, val, n).
    """
    y = np.asarray(y, dtype=np.float64)
    assert y.ndim == 1 and y.size % 2 == 0
    half = y.size // 2
    h = to_half(swiglu(y[:half], y[half:]))
    idx, val, n = compact(h, tau)
    return h, idx, val, n


def rlc_encode_column_py(column, kept, run_bits: int):
    """Section 3.2's rule as a literal loop over one column.

    column: sequence of values, kept: sequence of booleans.  Returns (values, runs, is_pad).
    """
    max_run = (1 << run_bits) - 1
    values, runs, pads = [], [], []
    gap = 0
    for v, k in zip(column, kept):
        if not k:
            gap += 1
            continue
        while gap > max_run:          # a pad stands for max_run zeros and occupies a row itself
            values.append(0)
            runs.append(max_run)
            pads.append(True)
            gap -= max_run + 1
        values.append(v)
        runs.append(gap)
        pads.append(False)
        gap = 0
    return values, runs, pads


def rlc_decode_column_py(runs, first_row: int = 0):
    """Rows from runs for one block: inclusive prefix sum plus ordinal (Algorithm 1)."""
    rows, s = [], 0
    for e, r in enumerate(runs):
        s += r
        rows.append(first_row + s + e)
    return rows
