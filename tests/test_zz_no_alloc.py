"""celty_spmspv_static: the entry point for callers that cannot allocate device memory (a stream capture
in progress, a pool that owns the whole device, a host application that forbids allocations on its
inference path).  Its scratch is a fixed array inside the library, so the call takes only the packed image,
x and y.  This file is collected last on purpose: the array is shared by every call in the process.

The check: two calls in a row must each reproduce what the existing entry point (celty_spmspv, with its
caller-provided workspace) returns, within the bound the parity tests use.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import celty_oracle as orc
from paper_2608_01536_b200 import build, celty, synth

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_the_workspace_entry_point_twice():
    build.build()
    assert torch.cuda.is_available(), "needs a CUDA device"
    M, K = 4096, 1536
    W = synth.weights(77, M, K)
    mask = synth.mask_bernoulli(77, M, K, 0.5)
    m = celty.Matrix(W, mask, device="cuda")
    # bound of the parity tests: 2e-3 * sum_j |W_ij x_j| + 1e-6 per element
    for call, seed in enumerate((1, 2)):                      # second call: other survivors, same scratch
        x = synth.activations(seed, K, "laplace")
        tau = synth.threshold_for_density(x, 0.5 if call == 0 else 0.3)
        xd = torch.from_numpy(x).cuda()
        y_ws = m.spmspv(xd, tau)                              # existing entry point
        y_st = m.spmspv_static(xd, tau, y=torch.full((M,), 3.0, device="cuda"))
        torch.cuda.synchronize()
        _, a_ref = orc.masked_gemv(W, mask, x, tau, threads=8)
        err = np.abs(y_st.cpu().numpy().astype(np.float64) - y_ws.cpu().numpy().astype(np.float64))
        assert np.all(err <= 2e-3 * a_ref + 1e-6), (call, float(err.max()))
        assert torch.count_nonzero(y_st).item() > 0


def test_static_scratch_entry_point_rejects_what_it_cannot_hold():
    build.build()
    lib = celty.load()
    wide = celty.Matrix(np.ones((4, 32769), np.float16))       # K beyond the fixed array
    p16 = ctypes.c_void_p(16)
    assert lib.celty_spmspv_static(wide._h, p16, p16, 0.0, p16, None) == -7
    assert lib.celty_strerror(-7) == b"size exceeds the fixed scratch of the no-allocation entry point"
    col = celty.Matrix(np.ones((4, 4), np.float16), layout=celty.LAYOUT_COLUMN)
    assert lib.celty_spmspv_static(col._h, p16, p16, 0.0, p16, None) == -1
    ok = celty.Matrix(np.ones((4, 4), np.float16))
    assert lib.celty_spmspv_static(ok._h, p16, p16, -1.0, p16, None) == -1
    assert lib.celty_spmspv_static(ok._h, None, p16, 0.0, p16, None) == -1
