"""Pins for the oracle's product, thresholding and compaction (Sections 1, 2.1, 3.1, 3.3)."""
import numpy as np
import pytest
import torch

from oracle import celty_oracle as orc
from paper_2608_01536_b200 import synth


def test_half_to_double_all_patterns_match_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float64)
    got = np.array([orc.half_to_double(int(b)) for b in bits])
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(ref[~nan]))


def _brute(W, mask, x, tau):
    """Triple-nested definition with Python floats (fp64), threshold decided in fp32."""
    M, K = W.shape
    y, a = [0.0] * M, [0.0] * M
    t32 = np.float32(tau)
    for i in range(M):
        for j in range(K):
            xj = np.float32(x[j])
            if abs(xj) <= t32:
                continue
            if not mask[i, j]:
                continue
            p = float(W[i, j]) * float(x[j])
            y[i] += p
            a[i] += abs(p)
    return np.array(y), np.array(a)


@pytest.mark.parametrize("M,K", [(1, 1), (7, 5), (33, 64), (64, 17)])
@pytest.mark.parametrize("d_w,d_a", [(0.0, 0.5), (0.1, 1.0), (0.5, 0.5), (1.0, 0.1), (1.0, 1.0), (0.5, 0.0)])
def test_masked_gemv_equals_brute_force(M, K, d_w, d_a):
    seed = 100 + M + K
    W = synth.weights(seed, M, K, std=1.0)
    mask = synth.mask_bernoulli(seed, M, K, d_w)
    x = synth.activations(seed, K, "laplace")
    tau = synth.threshold_for_density(x, d_a) if d_a > 0 else float(np.abs(x.astype(np.float32)).max())
    y, a = orc.masked_gemv(W, mask, x, tau)
    yb, ab = _brute(W, mask, x, tau)
    assert np.array_equal(y, yb) and np.array_equal(a, ab)
    # the product evaluated from the encoded arrays adds the same terms in the same order
    for tile_rows in (0, 16):
        y2, a2 = orc.spmspv_rlc(orc.rlc_encode(W, mask, 4, tile_rows), x, tau)
        assert np.array_equal(y2, y) and np.array_equal(a2, a)


def test_dense_special_case_is_textbook_gemv():
    M, K = 300, 257
    W = synth.weights(3, M, K, std=1.0)
    x = synth.activations(3, K, "normal")
    x[x == 0] = np.float16(1.0)
    y, a = orc.masked_gemv(W, np.ones((M, K), np.uint8), x, 0.0)
    ref = W.astype(np.float64) @ x.astype(np.float64)
    assert np.allclose(y, ref, rtol=0, atol=1e-11 * np.abs(ref).max())
    tref = torch.mv(torch.from_numpy(W.astype(np.float64)), torch.from_numpy(x.astype(np.float64))).numpy()
    assert np.allclose(y, tref, rtol=0, atol=1e-11 * np.abs(ref).max())
    aref = np.abs(W.astype(np.float64)) @ np.abs(x.astype(np.float64))
    assert np.allclose(a, aref, rtol=1e-12)


def test_unit_vector_selects_a_column_exactly():
    M, K = 129, 40
    W = synth.weights(5, M, K)
    mask = synth.mask_bernoulli(5, M, K, 0.4)
    for j in (0, 17, K - 1):
        x = np.zeros(K, np.float16)
        x[j] = 1.0
        y, _ = orc.masked_gemv(W, mask, x, 0.0)
        assert np.array_equal(y, np.where(mask[:, j] != 0, W[:, j].astype(np.float64), 0.0))


def test_identity_matrix_returns_thresholded_x():
    K = 50
    W = np.eye(K, dtype=np.float16)
    x = synth.activations(8, K, "laplace")
    tau = 0.7
    y, _ = orc.masked_gemv(W, W != 0, x, tau)
    xf = x.astype(np.float64)
    assert np.array_equal(y, np.where(np.abs(xf) > tau, xf, 0.0))


def test_masked_terms_are_skipped_not_multiplied():
    # an infinite weight that the mask drops must not poison the sum
    W = np.array([[np.inf, 2.0]], np.float16)
    mask = np.array([[0, 1]], np.uint8)
    x = np.array([1.0, 3.0], np.float16)
    y, a = orc.masked_gemv(W, mask, x, 0.0)
    assert y[0] == 6.0 and a[0] == 6.0
    # and a dropped activation likewise
    W = np.array([[1.0, 2.0]], np.float16)
    x = np.array([np.float16(0.25), 3.0], np.float16)
    y, _ = orc.masked_gemv(W, np.ones((1, 2), np.uint8), x, 0.25)
    assert y[0] == 6.0


def test_linearity_on_integer_data():
    M, K = 64, 48
    W = synth.integer_weights(1, M, K)
    mask = synth.mask_bernoulli(1, M, K, 0.5)
    x1 = synth.integer_activations(1, K)
    x2 = synth.integer_activations(2, K)
    x1[x1 == 0] = 1
    x2[x2 == 0] = 1
    s = (x1.astype(np.float32) + x2.astype(np.float32)).astype(np.float16)
    s_nonzero = s != 0
    y1, _ = orc.masked_gemv(W, mask, x1, 0.0)
    y2, _ = orc.masked_gemv(W, mask, x2, 0.0)
    ys, _ = orc.masked_gemv(W, mask, s, 0.0)
    assert s_nonzero.any()
    assert np.array_equal(ys, y1 + y2)


def test_threads_do_not_change_the_result():
    M, K = 200, 300
    W = synth.weights(4, M, K)
    mask = synth.mask_bernoulli(4, M, K, 0.5)
    x = synth.activations(4, K)
    y1, a1 = orc.masked_gemv(W, mask, x, 0.3, threads=1)
    y4, a4 = orc.masked_gemv(W, mask, x, 0.3, threads=4)
    assert np.array_equal(y1, y4) and np.array_equal(a1, a4)


# ----------------------------------------------------------------------------- thresholding
def test_keep_flags_special_values():
    x = np.array([0.0, -0.0, 1.0, -1.0, 0.5, -0.5, np.nan, np.inf, 6e-8], np.float16)
    assert orc.keep_flags(x, 0.0).tolist() == [0, 0, 1, 1, 1, 1, 1, 1, 1]      # tau = 0 drops exactly +-0
    assert orc.keep_flags(x, 0.5).tolist() == [0, 0, 1, 1, 0, 0, 1, 1, 0]      # ties at tau are dropped
    assert orc.keep_flags(x, 1.0).tolist() == [0, 0, 0, 0, 0, 0, 1, 1, 0]      # NaN survives


@pytest.mark.parametrize("K", [1, 7, 8, 9, 31, 33, 1023, 1025, 4099])
def test_compact_by_definition(K):
    x = synth.activations(K, K, "laplace")
    for d_a in (0.0, 0.3, 1.0):
        tau = synth.threshold_for_density(x, d_a) if d_a > 0 else 1e4
        idx, val, n = orc.compact(x, tau)
        expect = [j for j in range(K) if not (abs(np.float32(x[j])) <= np.float32(tau))]
        assert idx.tolist() == expect and n == len(expect)
        assert np.array_equal(val, x.view(np.uint16)[expect])
        assert n <= int(np.ceil(d_a * K)) + (0 if d_a < 1.0 else 0)


def test_compact_all_equal_magnitudes_are_all_dropped_at_tau():
    x = np.array([0.5, -0.5, 0.5, -0.5], np.float16)
    assert orc.compact(x, 0.5)[2] == 0
    assert orc.compact(x, 0.49)[2] == 4


# ----------------------------------------------------------------------------- input recipes
def test_synth_is_reproducible_and_has_the_requested_shape():
    a = synth.uniform(1536, 3, 1000)
    b = synth.uniform(1536, 3, 10, start=500)
    assert np.array_equal(a[500:510], b)
    assert 0.0 <= a.min() and a.max() < 1.0 and abs(a.mean() - 0.5) < 0.05
    W = synth.weights(1, 512, 64)
    assert abs(float(W.astype(np.float64).std()) - 0.02) < 0.002
    m = synth.mask_magnitude(W, 0.5)
    assert np.all(m.sum(axis=0) == 256)
    # pruned elements are the smaller ones
    aw = np.abs(W.astype(np.float32))
    assert np.all(np.where(m == 0, aw, 0).max(axis=0) <= np.where(m == 1, aw, np.inf).min(axis=0))
    p = synth.powerlaw_row_probability(8192, 0.5)
    assert abs(p.mean() - 0.5) < 1e-6 and p[0] == 1.0 and abs(p[-1] - 0.187) < 0.002
    x = synth.activations(2, 4096, "laplace")
    tau = synth.threshold_for_density(x, 0.5)
    kept = int((np.abs(x.astype(np.float32)) > np.float32(tau)).sum())
    assert 2040 <= kept <= 2048
