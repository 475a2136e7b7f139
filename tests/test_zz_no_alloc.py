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
        y_ref, a_ref = orc.masked_gemv(W, mask, x, tau, threads=8)
        bound = 2e-3 * a_ref + 1e-6
        got = y_st.cpu().numpy().astype(np.float64)
        # against the existing entry point ...
        assert np.all(np.abs(got - y_ws.cpu().numpy().astype(np.float64)) <= bound), call
        # ... and against the definition itself
        assert np.all(np.abs(got - y_ref) <= bound), call
        assert torch.count_nonzero(y_st).item() > 0


def test_static_scratch_entry_point_leaves_device_memory_alone():
    """The point of the entry point: a call takes no device memory.  The free-memory figure of the
    driver must be the same before and after a call (the first call on the device has already looked
    up the array's address; outputs are allocated beforehand)."""
    build.build()
    M, K = 2048, 1024
    W = synth.weights(78, M, K)
    mask = synth.mask_bernoulli(78, M, K, 0.5)
    m = celty.Matrix(W, mask, device="cuda")
    x = synth.activations(3, K, "laplace")
    tau = synth.threshold_for_density(x, 0.5)
    xd = torch.from_numpy(x).cuda()
    y = torch.empty(M, dtype=torch.float32, device="cuda")
    m.spmspv_static(xd, tau, y=y)                             # set-up call
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    m.spmspv_static(xd, tau, y=y)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    y_ref, a_ref = orc.masked_gemv(W, mask, x, tau, threads=8)
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= 2e-3 * a_ref + 1e-6)


def test_static_and_two_launch_entry_points_share_one_kernel_attribute():
    """Both entry points launch the same lane-tile kernel with different amounts of dynamic shared memory
    (a 4096-row handle asks for more than a 12288-row one).  Interleaving them must not leave either with
    a stale idea of what the runtime currently allows."""
    build.build()
    K = 256
    mats = []
    for M in (4096, 12288):
        W = synth.weights(80 + M, M, K)
        mask = synth.mask_bernoulli(80 + M, M, K, 0.5)
        m = celty.Matrix(W, mask, device="cuda")
        m.set_launch(variant=1)
        mats.append((m, W, mask))
    x = synth.activations(5, K, "laplace")
    tau = synth.threshold_for_density(x, 0.5)
    xd = torch.from_numpy(x).cuda()
    small, big = 0, 1
    for which, static in ((small, False), (big, True), (small, False), (small, True), (big, False)):
        m, W, mask = mats[which]
        y = m.spmspv_static(xd, tau) if static else m.spmspv(xd, tau)
        torch.cuda.synchronize()
        y_ref, a_ref = orc.masked_gemv(W, mask, x, tau, threads=8)
        assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= 2e-3 * a_ref + 1e-6), (W.shape, static)


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
