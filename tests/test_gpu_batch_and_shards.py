"""GPU parity for small batches (N = 1 .. 8 activation vectors against one matrix) and for a layer sharded by
columns: the oracle is N independent plain products, and the plain product of the whole layer."""
import numpy as np
import pytest
import torch

from oracle import celty_oracle as orc
from paper_2608_01536_b200 import build, celty, synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    celty.load()


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


@pytest.mark.parametrize("variant", [0, 1])          # N launches of the single-vector kernel / the widened kernels
@pytest.mark.parametrize("N", [1, 2, 3, 4, 5, 8])
@pytest.mark.parametrize("M,K,d_w,d_a", [(1000, 520, 0.5, 0.5), (4096, 1024, 0.3, 0.2), (11008, 300, 0.5, 0.9),
                                         (28672, 96, 0.5, 0.5)])
def test_batch_matches_independent_products(N, M, K, d_w, d_a, variant):
    W = synth.weights(M + K, M, K)
    mask = synth.mask_bernoulli(M + K, M, K, d_w)
    X = np.stack([synth.activations(100 * n + K, K, "laplace") for n in range(N)])
    tau = synth.threshold_for_density(X[0], d_a)
    m = celty.Matrix(W, mask, device="cuda")
    m.set_launch(variant=variant)
    Y = m.spmspv_batch(_dev(X), tau, y=torch.full((N, M), 4.0, device="cuda"))
    torch.cuda.synchronize()
    got = Y.cpu().numpy().astype(np.float64)
    for n in range(N):
        y_ref, a_ref = orc.masked_gemv(W, mask, X[n], tau, threads=8)
        err = np.abs(got[n] - y_ref)
        assert np.all(err <= 2e-3 * a_ref + 1e-6), (n, float(err.max()))


def test_batch_integer_data_is_bit_exact_and_strided():
    """Small integers make every FP32 sum exact in any order; the batch rows sit in wider buffers (ldx > K, ldy > M);
    one vector has no survivor at all and one keeps everything."""
    M, K, N = 3000, 257, 6
    W = synth.integer_weights(9, M, K)
    mask = synth.mask_bernoulli(9, M, K, 0.6)
    X = np.stack([synth.integer_activations(20 + n, K) for n in range(N)])
    X[2] = 0
    X[4][X[4] == 0] = 1
    tau = 1.0
    xb = torch.zeros(N, K + 7 + 8 - (K + 7) % 8, dtype=torch.float16, device="cuda")
    xb[:, :K] = _dev(X)
    yb = torch.full((N, M + 5), -1.0, device="cuda")
    m = celty.Matrix(W, mask, device="cuda")
    m.spmspv_batch(xb[:, :K], tau, y=yb[:, :M])
    torch.cuda.synchronize()
    for n in range(N):
        y_ref, _ = orc.masked_gemv(W, mask, X[n], tau, threads=4)
        assert np.array_equal(yb[n, :M].cpu().numpy().astype(np.float64), y_ref), n
    assert torch.all(yb[:, M:] == -1.0)                           # nothing written past a row
    assert torch.count_nonzero(yb[2, :M]).item() == 0


def test_batch_argument_errors():
    m = celty.Matrix(synth.weights(1, 64, 40), None, device="cuda")
    x = torch.zeros(9, 40, dtype=torch.float16, device="cuda")
    with pytest.raises(celty.CeltyError):
        m.spmspv_batch(x, 0.1)                                    # more than 8 vectors
    col = celty.Matrix(synth.weights(1, 64, 40), None, layout=celty.LAYOUT_COLUMN, device="cuda")
    with pytest.raises(celty.CeltyError):
        col.spmspv_batch(x[:2], 0.1)


@pytest.mark.parametrize("world", [1, 2, 3, 5])
def test_column_shards_add_up_to_the_layer(world):
    """Every rank's share of a column-sharded layer, run one after the other on this GPU (no process group: the
    all-reduce is replaced by adding the partial results here), against the plain product of the whole layer."""
    M, K = 2049, 1003
    W = synth.weights(31, M, K)
    mask = synth.mask_bernoulli(31, M, K, 0.5)
    x = synth.activations(31, K, "laplace")
    tau = synth.threshold_for_density(x, 0.5)
    xd = _dev(x)
    total = torch.zeros(M, dtype=torch.float32, device="cuda")
    covered = []
    for rank in range(world):
        shard = celty.ColumnShard(W, mask, rank=rank, world=1 if world == 1 else world, device="cuda")
        covered.append((shard.k0, shard.k1))
        shard.world = 1                                           # no collective in this test
        total += shard.spmspv(xd, tau)
    assert covered[0][0] == 0 and covered[-1][1] == K
    assert all(a[1] == b[0] for a, b in zip(covered, covered[1:]))
    y_ref, a_ref = orc.masked_gemv(W, mask, x, tau, threads=8)
    assert np.all(np.abs(total.cpu().numpy().astype(np.float64) - y_ref) <= 2e-3 * a_ref + 1e-6)
