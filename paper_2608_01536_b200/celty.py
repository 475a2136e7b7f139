"""Thin ctypes binding over the C-ABI library declared in include/celty.h.

Argument marshalling only: every step of the path (packing, thresholding/compaction, run-length
decode, accumulation, reduction) runs inside the library.  PyTorch provides device memory and
streams.  There is no fallback: if the library is missing or a call fails, this raises.
"""
from __future__ import annotations

import ctypes
import os
from types import SimpleNamespace

import numpy as np

LAYOUT_COLUMN = 0
LAYOUT_LANE_TILE = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcelty.so")
_lib = None

_vp, _i64, _i32, _f32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_float
_sz = ctypes.c_size_t

# name -> (restype, argtypes); mirrors include/celty.h one to one
SIGNATURES = {
    "celty_encode": (ctypes.c_int, [_vp, _i64, _vp, _i64, _i64, _vp, ctypes.POINTER(_vp)]),
    "celty_destroy": (None, [_vp]),
    "celty_clone": (ctypes.c_int, [_vp, ctypes.POINTER(_vp)]),
    "celty_info": (ctypes.c_int, [_vp] + [ctypes.POINTER(_i64)] * 5 + [ctypes.POINTER(_i32)] * 2),
    "celty_row_map": (ctypes.c_int, [_vp] + [ctypes.POINTER(_i32)] * 3),
    "celty_decode_host": (ctypes.c_int, [_vp, _i64, _vp, _vp, _vp, _vp, _i64, ctypes.POINTER(_i64)]),
    "celty_host_image": (ctypes.c_int, [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "celty_device_bytes": (ctypes.c_int, [_vp, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "celty_bind_device": (ctypes.c_int, [_vp, _vp, _sz, _vp, _sz, _vp]),
    "celty_compact": (ctypes.c_int, [_vp, _i64, _f32, _vp, _vp, _vp, _vp]),
    "celty_spmspv": (ctypes.c_int, [_vp, _vp, _f32, _vp, _vp]),
    "celty_spmspv_ex": (ctypes.c_int, [_vp, _vp, _f32, _vp, _vp, _vp]),
    "celty_spmspv_swiglu": (ctypes.c_int, [_vp, _vp, _f32, _vp, _vp, _vp, _vp]),
    "celty_spmspv_list": (ctypes.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "celty_spmspv_batch": (ctypes.c_int, [_vp, _vp, _i64, _i32, _f32, _vp, _i64, _vp, _sz, _vp]),
    "celty_shard_columns": (ctypes.c_int, [_i64, _i32, _i32, ctypes.POINTER(_i64), ctypes.POINTER(_i64)]),
    "celty_spmspv_static": (ctypes.c_int, [_vp, _vp, _vp, _f32, _vp, _vp]),
    "celty_spmspv_host": (ctypes.c_int, [_vp, _vp, _f32, _vp, _vp, _vp, _vp]),
    "celty_last_compaction": (ctypes.c_int, [_vp, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp)]),
    "celty_decode_device": (ctypes.c_int, [_vp, _i64, _vp, _vp, _i64, _vp, _vp]),
    "celty_fetched_bytes": (ctypes.c_int, [_vp, _vp, _i64, ctypes.POINTER(_i64), ctypes.POINTER(_i64)]),
    "celty_stored_entries": (ctypes.c_int, [_vp, _vp, _i64, ctypes.POINTER(_i64)]),
    "celty_layout_stats": (ctypes.c_int, [_vp] + [ctypes.POINTER(_i64)] * 3),
    "celty_count_entries": (ctypes.c_int, [_vp, _i64, _i64, _i64, ctypes.c_int, ctypes.POINTER(_i64),
                                           ctypes.POINTER(_i64)]),
    "celty_last_status": (ctypes.c_int, [_vp, _vp]),
    "celty_set_launch": (ctypes.c_int, [_vp, _i32, _i32, _i32, _i32, _i32]),
    "celty_launch_plan": (ctypes.c_int, [_vp, ctypes.POINTER(_i32), _i32]),
    "celty_set_register_rows": (ctypes.c_int, [_vp, _i32]),
    "celty_set_wait_limit": (ctypes.c_int, [_vp, ctypes.c_uint32]),
    "celty_last_cuda_error": (ctypes.c_int, []),
    "celty_strerror": (ctypes.c_char_p, [ctypes.c_int]),
}


class CeltyError(RuntimeError):
    def __init__(self, status: int, where: str):
        lib = load()
        msg = lib.celty_strerror(status).decode()
        if status == -3:
            msg += f" (cudaError {lib.celty_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")
        self.status = status


def load():
    """Load libcelty.so (built by paper_2608_01536_b200.build).  Raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: run `python -m paper_2608_01536_b200.build` (needs nvcc). "
                "There is no CPU or PyTorch fallback for this path.")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _check(status: int, where: str):
    if status != 0:
        raise CeltyError(status, where)


def _np_ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _stream_ptr(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


class _Opts(ctypes.Structure):
    _fields_ = [("run_bits", _i32), ("layout", _i32), ("tile_rows", _i32), ("slabs_per_block", _i32)]


class _Epilogue(ctypes.Structure):
    _fields_ = [("kind", _i32), ("out_fp16", _vp), ("tau", _f32), ("list_idx", _vp), ("list_val", _vp),
                ("list_count", _vp)]


class SwigluOut:
    """Device buffers the SiLU(gate) * up epilogue of a stacked [gate; up] product fills: h (FP16, I values) and the
    thresholded list (idx, val, count) that `Matrix.spmspv_list` of the down projection consumes."""

    def __init__(self, I: int, tau: float, device):
        import torch
        self.tau = float(tau)
        self.h = torch.empty(I, dtype=torch.float16, device=device)
        self.idx = torch.empty(I, dtype=torch.int32, device=device)
        self.val = torch.empty(I, dtype=torch.int16, device=device)
        self.count = torch.zeros(1, dtype=torch.int32, device=device)

    def _struct(self):
        return _Epilogue(2, self.h.data_ptr(), self.tau, self.idx.data_ptr(), self.val.data_ptr(),
                         self.count.data_ptr())


class Matrix:
    """An RLC-CSC encoded weight matrix (host handle), optionally bound to device memory."""

    def __init__(self, W, mask=None, layout: int = LAYOUT_LANE_TILE, tile_rows: int = 0, device=None,
                 slabs_per_block: int = 0):
        lib = load()
        W = np.asarray(W)
        if W.dtype == np.float16:
            W = W.view(np.uint16)
        if W.dtype != np.uint16 or W.ndim != 2:
            raise TypeError("W must be a 2-D float16 array (or its uint16 bit patterns)")
        W = np.ascontiguousarray(W)
        M, K = W.shape
        mptr = None
        if mask is not None:
            mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
            if mask.shape != (M, K):
                raise ValueError("mask shape")
            mptr = _np_ptr(mask)
        opts = _Opts(4, layout, tile_rows, slabs_per_block)
        h = _vp()
        _check(lib.celty_encode(_np_ptr(W), K, mptr, M, K, ctypes.byref(opts), ctypes.byref(h)), "celty_encode")
        self._h = h
        self.M, self.K = M, K
        self._image = self._ws = None
        if device is not None:
            self.to(device)

    def clone(self, device=None):
        """A second handle on a copy of the encoded matrix (not packed again), optionally bound to `device`."""
        h = _vp()
        _check(load().celty_clone(self._h, ctypes.byref(h)), "celty_clone")
        other = object.__new__(Matrix)
        other._h, other.M, other.K = h, self.M, self.K
        other._image = other._ws = None
        if device is not None:
            other.to(device)
        return other

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h and _lib is not None:
            _lib.celty_destroy(h)

    # ---------------------------------------------------------------- host side
    def info(self):
        v = [_i64() for _ in range(5)]
        w = [_i32() for _ in range(2)]
        _check(load().celty_info(self._h, *[ctypes.byref(a) for a in v + w]), "celty_info")
        return SimpleNamespace(M=v[0].value, K=v[1].value, nnz=v[2].value, n_pad=v[3].value,
                               compressed_bytes=v[4].value, layout=w[0].value, tile_rows=w[1].value)

    def row_map(self):
        """(slabs S, local rows per tile R, chunk C) of the LANE_TILE row map."""
        w = [_i32() for _ in range(3)]
        _check(load().celty_row_map(self._h, *[ctypes.byref(a) for a in w]), "celty_row_map")
        return w[0].value, w[1].value, w[2].value

    def host_image(self):
        """(uint8 copy of the packed image, offset of the entry stream in it)."""
        p, n, o = _vp(), _sz(), _sz()
        _check(load().celty_host_image(self._h, ctypes.byref(p), ctypes.byref(n), ctypes.byref(o)), "celty_host_image")
        buf = (ctypes.c_uint8 * n.value).from_address(p.value)
        return np.frombuffer(buf, dtype=np.uint8).copy(), o.value

    def device_bytes(self):
        a, b = _sz(), _sz()
        _check(load().celty_device_bytes(self._h, ctypes.byref(a), ctypes.byref(b)), "celty_device_bytes")
        return a.value, b.value

    def decode_host(self, col: int):
        lib = load()
        n = _i64()
        rc = lib.celty_decode_host(self._h, col, None, None, None, None, 0, ctypes.byref(n))
        if rc not in (0, -2):
            _check(rc, "celty_decode_host")
        rows = np.zeros(n.value, np.int32)
        vals = np.zeros(n.value, np.uint16)
        runs = np.zeros(n.value, np.uint8)
        pad = np.zeros(n.value, np.uint8)
        _check(lib.celty_decode_host(self._h, col, _np_ptr(rows), _np_ptr(vals), _np_ptr(runs), _np_ptr(pad),
                                     n.value, ctypes.byref(n)), "celty_decode_host")
        return rows, vals, runs, pad

    def fetched_bytes(self, idx):
        idx = np.ascontiguousarray(np.asarray(idx, dtype=np.int32))
        s, t = _i64(), _i64()
        _check(load().celty_fetched_bytes(self._h, _np_ptr(idx), idx.size, ctypes.byref(s), ctypes.byref(t)),
               "celty_fetched_bytes")
        return s.value, t.value

    def layout_stats(self):
        """(sub-blocks, steps in total, groups of 8 entries in total) of the LANE_TILE image."""
        v = [_i64() for _ in range(3)]
        _check(load().celty_layout_stats(self._h, *[ctypes.byref(a) for a in v]), "celty_layout_stats")
        return tuple(a.value for a in v)

    def stored_entries(self, idx) -> int:
        """Stored entries (kept weights + padding entries) of the listed columns."""
        idx = np.ascontiguousarray(np.asarray(idx, dtype=np.int32))
        e = _i64()
        _check(load().celty_stored_entries(self._h, _np_ptr(idx), idx.size, ctypes.byref(e)), "celty_stored_entries")
        return e.value

    def set_launch(self, grid: int = 0, variant: int = 0, groups: int = 0, depth: int = 0, cluster: int = 0):
        _check(load().celty_set_launch(self._h, grid, variant, groups, depth, cluster), "celty_set_launch")

    def launch_plan(self) -> dict:
        """Shape of the fused kernel's launch for this handle on the current device."""
        out = (_i32 * 10)()
        _check(load().celty_launch_plan(self._h, out, 10), "celty_launch_plan")
        keys = ("grid", "threads", "smem_bytes", "teams_per_slab", "ring_depth", "cluster", "row_parts",
                "slabs_per_block", "slot_bytes", "merge")
        plan = dict(zip(keys, [int(v) for v in out]))
        plan["parts_per_spare_block"] = plan["merge"] >> 8
        plan["warp_pairs"], plan["merge"] = (plan["merge"] >> 4) & 1, plan["merge"] & 15
        return plan

    def set_register_rows(self, rows: int = 0):
        """Local rows per lane summed in registers instead of shared memory (0, 32, 64, 96 or 128)."""
        _check(load().celty_set_register_rows(self._h, rows), "celty_set_register_rows")

    def set_wait_limit(self, polls: int = 0):
        """Polls a bounded wait inside the kernels makes before it gives up (0 = the library's limit)."""
        _check(load().celty_set_wait_limit(self._h, polls), "celty_set_wait_limit")

    # ---------------------------------------------------------------- device side
    def to(self, device="cuda", stream=None):
        import torch
        ib, wb = self.device_bytes()
        dev = torch.device(device)
        with torch.cuda.device(dev):
            self._image = torch.empty(ib, dtype=torch.uint8, device=dev)
            self._ws = torch.empty(wb, dtype=torch.uint8, device=dev)
            _check(load().celty_bind_device(self._h, self._image.data_ptr(), ib, self._ws.data_ptr(), wb,
                                            _stream_ptr(stream)), "celty_bind_device")
        self.device = dev
        return self

    def spmspv(self, x, tau: float, y=None, stream=None):
        """y = W . threshold(x, tau); x: K float16 CUDA tensor, y: M float32 CUDA tensor (overwritten)."""
        import torch
        if y is None:
            y = torch.empty(self.M, dtype=torch.float32, device=x.device)
        assert x.dtype == torch.float16 and x.numel() == self.K and x.is_contiguous()
        assert y.dtype == torch.float32 and y.numel() == self.M and y.is_contiguous()
        _check(load().celty_spmspv(self._h, x.data_ptr(), tau, y.data_ptr(), _stream_ptr(stream)), "celty_spmspv")
        return y

    def spmspv_ex(self, x, tau: float, y=None, fp16_out=None, swiglu: "SwigluOut | None" = None, stream=None):
        """spmspv followed in the same launch by an FP16 copy of y (fp16_out: M float16) or by the SiLU(gate) * up
        step of a stacked [gate; up] matrix (swiglu: a SwigluOut)."""
        import torch
        if y is None:
            y = torch.empty(self.M, dtype=torch.float32, device=x.device)
        assert x.dtype == torch.float16 and x.numel() == self.K and x.is_contiguous()
        assert y.dtype == torch.float32 and y.numel() == self.M and y.is_contiguous()
        ep = None
        if swiglu is not None:
            ep = swiglu._struct()
        elif fp16_out is not None:
            assert fp16_out.dtype == torch.float16 and fp16_out.numel() == self.M
            ep = _Epilogue(1, fp16_out.data_ptr(), 0.0, None, None, None)
        _check(load().celty_spmspv_ex(self._h, x.data_ptr(), tau, y.data_ptr(), ctypes.byref(ep) if ep else None,
                                      _stream_ptr(stream)), "celty_spmspv_ex")
        return y

    def spmspv_swiglu(self, gate_up, tau: float, y=None, h_out=None, fp16_out=None, stream=None):
        """Down projection whose activations SiLU(gate) * up are made inside the call from the FP32 result of the
        stacked [gate; up] product (gate_up: 2K float32); h_out (K float16, optional) receives them."""
        import torch
        if y is None:
            y = torch.empty(self.M, dtype=torch.float32, device=gate_up.device)
        assert gate_up.dtype == torch.float32 and gate_up.numel() == 2 * self.K and gate_up.is_contiguous()
        ep = None
        if fp16_out is not None:
            ep = _Epilogue(1, fp16_out.data_ptr(), 0.0, None, None, None)
        _check(load().celty_spmspv_swiglu(self._h, gate_up.data_ptr(), tau, y.data_ptr(),
                                          h_out.data_ptr() if h_out is not None else None,
                                          ctypes.byref(ep) if ep else None, _stream_ptr(stream)), "celty_spmspv_swiglu")
        return y

    def spmspv_list(self, idx, val, count, y=None, fp16_out=None, stream=None):
        """The product from a ready-made survivor list (device tensors: int32 columns, FP16 bit patterns, int32[1]
        count), e.g. the one a SwigluOut holds."""
        import torch
        if y is None:
            y = torch.empty(self.M, dtype=torch.float32, device=idx.device)
        assert idx.dtype == torch.int32 and val.dtype in (torch.int16, torch.float16) and count.dtype == torch.int32
        ep = None
        if fp16_out is not None:
            assert fp16_out.dtype == torch.float16 and fp16_out.numel() == self.M
            ep = _Epilogue(1, fp16_out.data_ptr(), 0.0, None, None, None)
        _check(load().celty_spmspv_list(self._h, idx.data_ptr(), val.data_ptr(), count.data_ptr(), y.data_ptr(),
                                        ctypes.byref(ep) if ep else None, _stream_ptr(stream)), "celty_spmspv_list")
        return y

    def spmspv_batch(self, x, tau: float, y=None, stream=None):
        """y[n] = W . threshold(x[n], tau) for a batch x of shape (N, K), N <= 8; y: (N, M) float32."""
        import torch
        assert x.dtype == torch.float16 and x.dim() == 2 and x.shape[1] == self.K and x.stride(1) == 1
        N = x.shape[0]
        if y is None:
            y = torch.empty(N, self.M, dtype=torch.float32, device=x.device)
        assert y.dtype == torch.float32 and y.shape == (N, self.M) and y.stride(1) == 1
        need = 256 + (4 * self.K + 255) // 256 * 256 + 16 * self.K
        if getattr(self, "_batch_scratch", None) is None or self._batch_scratch.numel() < need:
            self._batch_scratch = torch.empty(need, dtype=torch.uint8, device=x.device)
        _check(load().celty_spmspv_batch(self._h, x.data_ptr(), x.stride(0), N, tau, y.data_ptr(), y.stride(0),
                                         self._batch_scratch.data_ptr(), self._batch_scratch.numel(),
                                         _stream_ptr(stream)), "celty_spmspv_batch")
        return y

    def spmspv_static(self, x, tau: float, y=None, stream=None):
        """Same product through the entry point that needs no workspace: its scratch is a fixed array inside
        the library, for callers that cannot allocate device memory.  K <= 32768; calls that overlap on the
        GPU race on that array.  The matrix's packed image must be on the device (`to()`)."""
        import torch
        if y is None:
            y = torch.empty(self.M, dtype=torch.float32, device=x.device)
        assert x.dtype == torch.float16 and x.numel() == self.K and x.is_contiguous()
        assert y.dtype == torch.float32 and y.numel() == self.M and y.is_contiguous()
        _check(load().celty_spmspv_static(self._h, self._image.data_ptr(), x.data_ptr(), tau, y.data_ptr(),
                                          _stream_ptr(stream)), "celty_spmspv_static")
        return y

    def spmspv_host(self, x_host, tau: float, y_host, x_stage, y_stage, stream=None):
        """Same product for host tensors (pinned for speed); copies run inside the library call."""
        _check(load().celty_spmspv_host(self._h, x_host.data_ptr(), tau, y_host.data_ptr(), x_stage.data_ptr(),
                                        y_stage.data_ptr(), _stream_ptr(stream)), "celty_spmspv_host")
        return y_host

    def last_compaction(self):
        """(idx int32 tensor, val int16-bit-pattern tensor) of the last spmspv call; synchronises."""
        import torch
        c, i, v = _vp(), _vp(), _vp()
        _check(load().celty_last_compaction(self._h, ctypes.byref(c), ctypes.byref(i), ctypes.byref(v)),
               "celty_last_compaction")
        torch.cuda.synchronize()
        ws0 = self._ws.data_ptr()
        n = int(self._ws[c.value - ws0:c.value - ws0 + 4].view(torch.int32).item())
        idx = self._ws[i.value - ws0:i.value - ws0 + 4 * n].view(torch.int32).clone()
        val = self._ws[v.value - ws0:v.value - ws0 + 2 * n].view(torch.int16).clone()
        return idx, val

    def decode_device(self, col: int, stream=None):
        import torch
        n = self.decode_host(col)[0].size
        rows = torch.full((max(n, 1),), -1, dtype=torch.int32, device=self.device)
        vals = torch.zeros(max(n, 1), dtype=torch.int16, device=self.device)
        cnt = torch.zeros(1, dtype=torch.int32, device=self.device)
        _check(load().celty_decode_device(self._h, col, rows.data_ptr(), vals.data_ptr(), n, cnt.data_ptr(),
                                          _stream_ptr(stream)), "celty_decode_device")
        torch.cuda.synchronize()
        k = int(cnt.item())
        return rows[:k].cpu().numpy(), vals[:k].cpu().numpy().view(np.uint16)

    def last_status(self, stream=None) -> int:
        return load().celty_last_status(self._h, _stream_ptr(stream))


def compact(x, tau: float, stream=None):
    """Activation compaction alone: returns (idx int32[n], val uint16-pattern int16[n]) CUDA tensors."""
    import torch
    assert x.dtype == torch.float16 and x.is_contiguous()
    K = x.numel()
    idx = torch.empty(K, dtype=torch.int32, device=x.device)
    val = torch.empty(K, dtype=torch.int16, device=x.device)
    cnt = torch.zeros(1, dtype=torch.int32, device=x.device)
    _check(load().celty_compact(x.data_ptr(), K, tau, idx.data_ptr(), val.data_ptr(), cnt.data_ptr(),
                                _stream_ptr(stream)), "celty_compact")
    n = int(cnt.item())
    return idx[:n], val[:n]


def shard_columns(K: int, world: int, rank: int):
    """Column range [k0, k1) of `rank` when a layer is sharded by columns over `world` GPUs."""
    a, b = _i64(), _i64()
    _check(load().celty_shard_columns(K, world, rank, ctypes.byref(a), ctypes.byref(b)), "celty_shard_columns")
    return a.value, b.value


class ColumnShard:
    """One rank's share of a layer sharded by columns (K-sharding): it packs columns [k0, k1) of W, thresholds its
    own slice of x, and the partial results of all ranks are summed by one all-reduce of M floats over the default
    torch.distributed process group (NCCL between GPUs).  With a world of one it is the plain product."""

    def __init__(self, W, mask=None, rank: int = 0, world: int = 1, device=None, **kw):
        W = np.asarray(W)
        self.K_full = W.shape[1]
        self.rank, self.world = rank, world
        self.k0, self.k1 = shard_columns(self.K_full, world, rank)
        self.empty = self.k1 <= self.k0
        if not self.empty:
            Ws = np.ascontiguousarray(W[:, self.k0:self.k1])
            ms = None if mask is None else np.ascontiguousarray(np.asarray(mask)[:, self.k0:self.k1])
            self.local = Matrix(Ws, ms, device=device, **kw)
        self.M = W.shape[0]

    def spmspv(self, x, tau: float, y=None, stream=None):
        """x: the FULL activation vector (K float16, on this rank's device); returns y = W . threshold(x, tau),
        identical on every rank after the all-reduce."""
        import torch
        import torch.distributed as dist
        if y is None:
            y = torch.empty(self.M, dtype=torch.float32, device=x.device)
        if self.empty:
            y.zero_()
        else:
            self.local.spmspv(x[self.k0:self.k1], tau, y, stream=stream)
        if self.world > 1:
            dist.all_reduce(y, op=dist.ReduceOp.SUM)
        return y


def count_entries(mask, run_bits: int = 4):
    """(kept positions, padding entries) the whole-column format would store for `mask` (M x K, nonzero =
    kept) with runs of `run_bits` bits; an entry then takes 2 + run_bits / 8 bytes.  Host only."""
    mask = np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))
    M, K = mask.shape
    nnz, pad = _i64(), _i64()
    _check(load().celty_count_entries(_np_ptr(mask), K, M, K, int(run_bits), ctypes.byref(nnz), ctypes.byref(pad)),
           "celty_count_entries")
    return nnz.value, pad.value
