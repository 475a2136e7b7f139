"""GPU parity for the decode-layer pieces around the product (Section 6.2 times the seven products of a layer):
FP16 output, the SiLU(gate) * up step fused behind the stacked [gate; up] product with its thresholded list, the
down projection that consumes that list, and the stacked four-call chain as a whole -- all against the oracle.

Tolerances are derived, not tuned.  An FP32 sum of n fused multiply-adds (exact products) in any order is within
gamma_n * sum|terms| of the exact sum, gamma_n = n u / (1 - n u), u = 2^-24.  SiLU has |slope| <= 1.1, its FP32
evaluation (exp, add, divide) and the product cost a few more roundings (16 u is generous), and the one rounding
to FP16 can move a value that was off by eps onto the next FP16 value: |h_gpu - h_ref| <= eps + ulp16(h_ref).
A value whose magnitude is within that distance of the threshold may legitimately fall on either side.
"""
import numpy as np
import pytest
import torch

from oracle import celty_oracle as orc
from paper_2608_01536_b200 import build, celty, synth

pytestmark = pytest.mark.gpu
U = 2.0 ** -24


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    celty.load()


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _ulp16(v):
    e = np.floor(np.log2(np.maximum(np.abs(v), 2.0 ** -14)))
    return 2.0 ** (e - 10)


def _fp32_sum_bound(a_ref, n_terms):
    g = (n_terms + 64) * U                      # the merge adds a few dozen partial sums on top of the n terms
    return g / (1 - g) * a_ref + 1e-30


def _layer(seed, I, K, d_w=0.5):
    """Stacked [gate; up] (2I x K) and down (K x I) weights with Bernoulli masks."""
    Wgu = synth.weights(seed, 2 * I, K)
    mgu = synth.mask_bernoulli(seed, 2 * I, K, d_w)
    Wd = synth.weights(seed + 1, K, I)
    md = synth.mask_bernoulli(seed + 1, K, I, d_w)
    return Wgu, mgu, Wd, md


def _reference_chain(Wgu, mgu, Wd, md, x, tau, d_h):
    """The oracle's own chain: stacked product, element-wise step with one FP16 rounding, list, down product.
    Returns what the GPU is compared with plus the error bounds that follow from the arithmetic."""
    I, K = Wgu.shape[0] // 2, Wgu.shape[1]
    y_ref, a_ref = orc.masked_gemv(Wgu, mgu, x, tau, threads=orc.max_threads())
    n_surv = orc.compact(x, tau)[2]
    By = _fp32_sum_bound(a_ref, n_surv)
    g, u = y_ref[:I], y_ref[I:]
    h64 = orc.swiglu(g, u)
    h16 = orc.to_half(h64)
    hv = h16.view(np.float16).astype(np.float64)
    tau2 = synth.threshold_for_density(h16.view(np.float16), d_h)
    eps = 1.1 * By[:I] * np.abs(u) + np.abs(orc.silu(g)) * By[I:] + 1.1 * By[:I] * By[I:] + 16 * U * np.abs(h64)
    tol_h = eps + _ulp16(hv)
    near = np.abs(np.abs(hv) - np.float64(np.float32(tau2))) <= tol_h
    idx_ref, val_ref, n_ref = orc.compact(h16, tau2)
    yd_ref, ad_ref = orc.masked_gemv(Wd, md, h16, tau2, threads=orc.max_threads())
    kept = np.zeros(I, bool)
    kept[idx_ref] = True
    E = np.where(near, np.abs(hv) + tol_h, np.where(kept, tol_h, 0.0))
    extra = (np.abs(Wd.astype(np.float32)) * md).astype(np.float64) @ E
    tol_yd = 2e-3 * ad_ref + 1e-6 + extra
    return dict(y=y_ref, a=a_ref, h16=h16, hv=hv, tol_h=tol_h, tau2=tau2, near=near, idx=idx_ref, yd=yd_ref,
                tol_yd=tol_yd)


@pytest.mark.parametrize("M,K,d_a", [(1000, 520, 0.5), (4096, 1024, 0.3), (11008, 256, 0.7)])
def test_fp16_output(M, K, d_a):
    W = synth.weights(M + K, M, K)
    mask = synth.mask_bernoulli(M + K, M, K, 0.5)
    x = synth.activations(M + K, K, "laplace")
    tau = synth.threshold_for_density(x, d_a)
    m = celty.Matrix(W, mask, device="cuda")
    y16 = torch.full((M,), 9.0, dtype=torch.float16, device="cuda")
    y = m.spmspv_ex(_dev(x), tau, fp16_out=y16)
    torch.cuda.synchronize()
    assert m.last_status() == 0
    y_ref, a_ref = orc.masked_gemv(W, mask, x, tau, threads=8)
    got32, got16 = y.cpu().numpy().astype(np.float64), y16.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got32 - y_ref) <= 2e-3 * a_ref + 1e-6)
    # the FP16 copy is the FP32 result rounded once
    assert np.all(np.abs(got16 - y_ref) <= 2e-3 * a_ref + 1e-6 + 0.5 * _ulp16(y_ref) * 1.0001)
    assert np.array_equal(y16.cpu().numpy(), y.cpu().numpy().astype(np.float16))


@pytest.mark.parametrize("I,K,d_a,d_h", [(1536, 1024, 0.4, 0.4), (700, 333, 0.9, 0.1), (4000, 512, 0.5, 1.0),
                                         (13824, 5120, 0.4, 0.4)])
def test_swiglu_step_list_and_down_projection(I, K, d_a, d_h):
    """[gate; up] product -> SiLU(gate) * up -> FP16 -> list, in one launch; then the down projection from that
    list.  (13824, 5120) is the Llama-2-13B layer of the bench's chain, at full size.)"""
    Wgu, mgu, Wd, md = _layer(I + K, I, K)
    x = synth.activations(I + K, K, "laplace")
    tau = synth.threshold_for_density(x, d_a)
    ref = _reference_chain(Wgu, mgu, Wd, md, x, tau, d_h)
    mg = celty.Matrix(Wgu, mgu, device="cuda")
    mdn = celty.Matrix(Wd, md, device="cuda")
    out = celty.SwigluOut(I, ref["tau2"], "cuda")
    for call in range(2):                                        # twice: the second ticket wraps around too
        out.count.fill_(12345)
        y = mg.spmspv_ex(_dev(x), tau, swiglu=out)
        yd = mdn.spmspv_list(out.idx, out.val, out.count)
        torch.cuda.synchronize()
        assert mg.last_status() == 0 and mdn.last_status() == 0
        # the stacked product itself
        assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - ref["y"]) <= 2e-3 * ref["a"] + 1e-6)
        # h against the oracle's, within the derived bound
        h_gpu = out.h.cpu().numpy()
        assert np.all(np.abs(h_gpu.astype(np.float64) - ref["hv"]) <= ref["tol_h"]), call
        # the list holds exactly the entries of the kernel's own h that pass the threshold, each once
        n = int(out.count.item())
        li = out.idx[:n].cpu().numpy()
        lv = out.val[:n].cpu().numpy().view(np.uint16)
        with np.errstate(invalid="ignore"):
            own = np.flatnonzero(~(np.abs(h_gpu.astype(np.float32)) <= np.float32(ref["tau2"])))
        assert np.array_equal(np.sort(li), own)
        assert np.array_equal(lv, h_gpu.view(np.uint16)[li])
        # ... and as a set it is the oracle's list, up to the entries that sit on the threshold
        sym = np.setxor1d(li, ref["idx"])
        assert np.all(ref["near"][sym]), (call, sym[:10])
        assert sym.size <= max(2, I // 200)
        # the down projection from the list
        err = np.abs(yd.cpu().numpy().astype(np.float64) - ref["yd"])
        worst = int(np.argmax(err - ref["tol_yd"]))
        assert np.all(err <= ref["tol_yd"]), (call, worst, err[worst], ref["tol_yd"][worst])


@pytest.mark.parametrize("I,K,d_a,d_h", [(1536, 1024, 0.4, 0.4), (701, 333, 0.9, 0.1), (13824, 5120, 0.4, 0.4)])
def test_swiglu_made_inside_the_down_projection(I, K, d_a, d_h):
    """The other way to fuse the step: the gate/up product is a plain call, and the down projection makes
    SiLU(gate) * up itself while it thresholds (no launch, no pass over memory in between)."""
    Wgu, mgu, Wd, md = _layer(I + K + 1, I, K)
    x = synth.activations(I + K + 1, K, "laplace")
    tau = synth.threshold_for_density(x, d_a)
    ref = _reference_chain(Wgu, mgu, Wd, md, x, tau, d_h)
    mg = celty.Matrix(Wgu, mgu, device="cuda")
    mdn = celty.Matrix(Wd, md, device="cuda")
    h = torch.zeros(I, dtype=torch.float16, device="cuda")
    for call in range(2):
        y = mg.spmspv(_dev(x), tau)
        yd = mdn.spmspv_swiglu(y, ref["tau2"], h_out=h)
        torch.cuda.synchronize()
        assert mg.last_status() == 0 and mdn.last_status() == 0
        h_gpu = h.cpu().numpy()
        assert np.all(np.abs(h_gpu.astype(np.float64) - ref["hv"]) <= ref["tol_h"]), call
        li, lv = mdn.last_compaction()
        li, lv = li.cpu().numpy(), lv.cpu().numpy().view(np.uint16)
        with np.errstate(invalid="ignore"):
            own = np.flatnonzero(~(np.abs(h_gpu.astype(np.float32)) <= np.float32(ref["tau2"])))
        assert np.array_equal(li, own)                               # ascending, exactly the kernel's own h thresholded
        assert np.array_equal(lv, h_gpu.view(np.uint16)[li])
        sym = np.setxor1d(li, ref["idx"])
        assert np.all(ref["near"][sym]) and sym.size <= max(2, I // 200)
        err = np.abs(yd.cpu().numpy().astype(np.float64) - ref["yd"])
        assert np.all(err <= ref["tol_yd"]), (call, float((err - ref["tol_yd"]).max()))


def test_list_input_matches_thresholded_input():
    """A list made by the oracle's compaction (shuffled: any order is allowed) gives the product that thresholding x
    inside the call gives."""
    M, K = 3000, 777
    W = synth.weights(5, M, K)
    mask = synth.mask_bernoulli(5, M, K, 0.5)
    x = synth.activations(5, K, "laplace")
    tau = synth.threshold_for_density(x, 0.5)
    idx, val, n = orc.compact(x, tau)
    perm = np.random.default_rng(1).permutation(n)
    m = celty.Matrix(W, mask, device="cuda")
    y = m.spmspv_list(_dev(idx[perm]), _dev(val[perm].view(np.int16)), _dev(np.array([n], np.int32)))
    torch.cuda.synchronize()
    assert m.last_status() == 0
    y_ref, a_ref = orc.masked_gemv(W, mask, x, tau, threads=8)
    assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= 2e-3 * a_ref + 1e-6)
    # an empty list
    y0 = m.spmspv_list(_dev(idx), _dev(val.view(np.int16)), _dev(np.zeros(1, np.int32)), y=torch.full((M,), 3.0, device="cuda"))
    assert torch.count_nonzero(y0).item() == 0


def test_stacked_decode_layer_chain():
    """The four calls of a decode layer with the products that share an input stacked: [q; k; v], o, [gate; up] with
    the SiLU(gate) * up step and its list, down from the list -- enqueued back to back on one stream, every output
    compared with the oracle.  (Attention and the normalisations between the products are outside the path, so the
    inputs of the first three calls are independent synthetic vectors; the down projection really consumes what the
    gate/up call produced.)  Shapes: the Llama-2-13B layer scaled by 1/4 in every dimension."""
    H, I = 1280, 3456
    seed = 400
    Wqkv, mqkv = synth.weights(seed, 3 * H, H), synth.mask_bernoulli(seed, 3 * H, H, 0.5)
    Wo, mo = synth.weights(seed + 1, H, H), synth.mask_bernoulli(seed + 1, H, H, 0.5)
    Wgu, mgu, Wd, md = _layer(seed + 2, I, H)
    xs = [synth.activations(seed + 10 + k, H, "laplace") for k in range(3)]
    taus = [synth.threshold_for_density(x, 0.4) for x in xs]
    ref = _reference_chain(Wgu, mgu, Wd, md, xs[2], taus[2], 0.4)
    mats = [celty.Matrix(Wqkv, mqkv, device="cuda"), celty.Matrix(Wo, mo, device="cuda"),
            celty.Matrix(Wgu, mgu, device="cuda"), celty.Matrix(Wd, md, device="cuda")]
    xd = [_dev(x) for x in xs]
    out = celty.SwigluOut(I, ref["tau2"], "cuda")
    qkv16 = torch.empty(3 * H, dtype=torch.float16, device="cuda")
    o16 = torch.empty(H, dtype=torch.float16, device="cuda")
    d16 = torch.empty(H, dtype=torch.float16, device="cuda")
    for rep in range(3):
        yq = mats[0].spmspv_ex(xd[0], taus[0], fp16_out=qkv16)
        yo = mats[1].spmspv_ex(xd[1], taus[1], fp16_out=o16)
        yg = mats[2].spmspv_ex(xd[2], taus[2], swiglu=out)
        yd = mats[3].spmspv_list(out.idx, out.val, out.count, fp16_out=d16)
    torch.cuda.synchronize()
    assert all(m.last_status() == 0 for m in mats)
    for y, y16, (W, mask, x, tau) in ((yq, qkv16, (Wqkv, mqkv, xs[0], taus[0])), (yo, o16, (Wo, mo, xs[1], taus[1]))):
        y_ref, a_ref = orc.masked_gemv(W, mask, x, tau, threads=8)
        assert np.all(np.abs(y.cpu().numpy().astype(np.float64) - y_ref) <= 2e-3 * a_ref + 1e-6)
        assert np.array_equal(y16.cpu().numpy(), y.cpu().numpy().astype(np.float16))
    assert np.all(np.abs(yg.cpu().numpy().astype(np.float64) - ref["y"]) <= 2e-3 * ref["a"] + 1e-6)
    assert np.all(np.abs(out.h.cpu().numpy().astype(np.float64) - ref["hv"]) <= ref["tol_h"])
    assert np.all(np.abs(yd.cpu().numpy().astype(np.float64) - ref["yd"]) <= ref["tol_yd"])
    assert np.array_equal(d16.cpu().numpy(), yd.cpu().numpy().astype(np.float16))


def test_epilogue_argument_errors():
    m = celty.Matrix(synth.weights(1, 65, 40), None, device="cuda")           # odd number of rows
    x = _dev(synth.activations(1, 40, "laplace"))
    with pytest.raises(celty.CeltyError):
        m.spmspv_ex(x, 0.1, swiglu=celty.SwigluOut(32, 0.1, "cuda"))
    m.set_launch(variant=2)                                                    # ordered merge: no work after it
    with pytest.raises(celty.CeltyError):
        m.spmspv_ex(x, 0.1, fp16_out=torch.empty(65, dtype=torch.float16, device="cuda"))
    col = celty.Matrix(synth.weights(1, 64, 40), None, layout=celty.LAYOUT_COLUMN, device="cuda")
    with pytest.raises(celty.CeltyError):
        col.spmspv_ex(x, 0.1, fp16_out=torch.empty(64, dtype=torch.float16, device="cuda"))
