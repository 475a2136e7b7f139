"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element.

Bit-exact for the compacted list and the decoded indices; |y_gpu - y_ref| <= 2e-3 * sum_j |W_ij x_j|
+ 1e-6 per element for FP16-in / FP32-accumulate values; bit-exact too where the data make the FP32
sum order-independent (small integers).
"""
import os

import numpy as np
import pytest
import torch

from conftest import permute_for_lane_tiles
from oracle import celty_oracle as orc
from paper_2608_01536_b200 import build, celty, synth

pytestmark = pytest.mark.gpu

# (layout, variant): the published column formulation, the fused lane-tile kernel, and the
# two-launch lane-tile path
LAYOUTS = [(celty.LAYOUT_COLUMN, 0), (celty.LAYOUT_LANE_TILE, 0), (celty.LAYOUT_LANE_TILE, 1)]
DECODE_LAYOUTS = [celty.LAYOUT_COLUMN, celty.LAYOUT_LANE_TILE]


def _matrix(W, mask, lv, tile_rows=0, slabs_per_block=0):
    layout, variant = lv
    lane = layout == celty.LAYOUT_LANE_TILE
    m = celty.Matrix(W, mask, layout=layout, tile_rows=tile_rows if lane else 0,
                     slabs_per_block=slabs_per_block if lane else 0, device="cuda")
    m.set_launch(variant=variant)
    m.variant = variant
    return m


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    celty.load()


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _run(m, x, tau):
    y = m.spmspv(_dev(x), tau)
    torch.cuda.synchronize()
    assert m.last_status() == 0
    return y.cpu().numpy()


def _check_y(y, W, mask, x, tau, exact=False):
    y_ref, a_ref = orc.masked_gemv(W, mask, x, tau, threads=8)
    if exact:
        assert np.array_equal(y.astype(np.float64), y_ref)
    else:
        err = np.abs(y.astype(np.float64) - y_ref)
        bound = 2e-3 * a_ref + 1e-6
        worst = int(np.argmax(err - bound))
        assert np.all(err <= bound), (worst, y[worst], y_ref[worst], a_ref[worst])


# ----------------------------------------------------------------------------- compaction
@pytest.mark.parametrize("K", [1, 7, 8, 9, 31, 33, 1000, 1024, 4096, 8191, 8193, 28672, 40000])
def test_compaction_bit_exact(K):
    x = synth.activations(K, K, "laplace")
    if K > 40:
        x[5] = np.float16(0.0)
        x[6] = np.float16(-0.0)
        x[17] = np.float16(np.nan)
    xd = _dev(x)
    amax = float(np.nanmax(np.abs(x.astype(np.float32))))
    for tau in (0.0, synth.threshold_for_density(x, 0.5), synth.threshold_for_density(x, 0.1), amax, 1e4):
        if not np.isfinite(tau):
            continue
        idx, val = celty.compact(xd, tau)
        oi, ov, n = orc.compact(x, tau)
        assert idx.numel() == n
        assert np.array_equal(idx.cpu().numpy(), oi)
        assert np.array_equal(val.cpu().numpy().view(np.uint16), ov)


SPECIAL_X = np.array([0x0000, 0x8000, 0x7E00, 0xFE00, 0x7C00, 0xFC00, 0x0001, 0x8001, 0x03FF, 0x83FF, 0x0400, 0x8400,
                      0x7BFF, 0xFBFF, 0x3C00, 0xBC00, 0x3C01, 0x3BFF, 0x3800, 0xB800], np.uint16)


@pytest.mark.parametrize("K", [20, 64, 1000, 4099])
@pytest.mark.parametrize("tau", [0.0, 1e-8, 5.9604645e-08, 0.99975586, 1.0, 1.0004883, 0.7, 65504.0, 65519.9, 1e5])
def test_fused_kernel_thresholding_bit_exact_on_special_values(K, tau):
    """The fused kernel has its own thresholding code (it compares in FP16 against tau rounded down to FP16, which
    is the same decision as |x| > tau in FP32): +-0, NaNs, +-infinity, the smallest and largest subnormals, the
    smallest normal, the largest finite value and the neighbours of 1, against thresholds that are 0, below the
    smallest subnormal, exactly on FP16 values, strictly between two FP16 neighbours, the largest finite FP16
    value and beyond it.  The list the call leaves behind must be the oracle's, bit for bit."""
    x = synth.activations(K + 3, K, "laplace").view(np.uint16).copy()
    pos = (np.arange(SPECIAL_X.size) * 37) % K if K > SPECIAL_X.size else np.arange(SPECIAL_X.size)
    x[pos[:K]] = SPECIAL_X[:K]
    x = x.view(np.float16)
    M = 64
    W = synth.weights(K, M, K)
    m = celty.Matrix(W, None, device="cuda")
    m.spmspv(_dev(x), tau)
    torch.cuda.synchronize()
    assert m.last_status() == 0
    idx, val = m.last_compaction()
    oi, ov, n = orc.compact(x, tau)
    assert idx.numel() == n
    assert np.array_equal(idx.cpu().numpy(), oi)
    assert np.array_equal(val.cpu().numpy().view(np.uint16), ov)
    # the stand-alone compaction kernel takes the same decisions
    i2, v2 = celty.compact(_dev(x), tau)
    assert np.array_equal(i2.cpu().numpy(), oi) and np.array_equal(v2.cpu().numpy().view(np.uint16), ov)


def test_compaction_ties_are_dropped():
    x = np.array([0.5, -0.5] * 20, np.float16)
    assert celty.compact(_dev(x), 0.5)[0].numel() == 0
    assert celty.compact(_dev(x), 0.499)[0].numel() == 40


# ----------------------------------------------------------------------------- decode
@pytest.mark.parametrize("layout", DECODE_LAYOUTS)
@pytest.mark.parametrize("M,K,d_w,tile_rows", [(257, 9, 0.5, 0), (4097, 6, 0.03, 0), (1000, 5, 1.0, 0),
                                               (3000, 7, 0.3, 40), (28672, 3, 0.5, 0), (2100, 4, 0.9, 7)])
def test_device_decode_bit_exact(layout, M, K, d_w, tile_rows):
    if layout == celty.LAYOUT_COLUMN:
        tile_rows = 0
    W = synth.weights(M, M, K)
    mask = synth.mask_bernoulli(M, M, K, d_w)
    mask[:, 0] = 0                      # empty column
    mask[:, 1] = 0
    mask[-1, 1] = 1                     # only the last row: maximum number of pads
    mask[:, 2] = 1                      # dense column
    m = celty.Matrix(W, mask, layout=layout, tile_rows=tile_rows, device="cuda")
    rowmap = None
    if layout == celty.LAYOUT_LANE_TILE:
        S, R, C = m.row_map()
        Wp, mp, rowmap = permute_for_lane_tiles(W, mask, S, R, C)
        enc = orc.rlc_encode(Wp, mp, 4, tile_rows=R)
    else:
        enc = orc.rlc_encode(W, mask, 4, tile_rows=0)
    for j in range(K):
        rows, vals = m.decode_device(j)
        orows, ovals, _, _ = orc.column_entries(enc, j)
        if rowmap is not None:
            orows = rowmap[orows]
        assert np.array_equal(rows, orows), j
        assert np.array_equal(vals, ovals), j


@pytest.mark.parametrize("case", range(24))
def test_device_decode_random_draws(case):
    rng = np.random.default_rng(9000 + case)
    M = int(rng.choice([1, 31, 33, 100, 777, 3001, 9001]))
    K = int(rng.choice([1, 3, 6]))
    d_w = float(rng.choice([0.03, 0.3, 0.7, 1.0]))
    tile_rows = int(rng.choice([0, 0, 1, 5, 16, 96, 240]))
    if tile_rows and (M + 31) // 32 > 32 * tile_rows:
        tile_rows = 0
    W = synth.weights(9500 + case, M, K)
    mask = synth.mask_bernoulli(9500 + case, M, K, d_w)
    m = celty.Matrix(W, mask, tile_rows=tile_rows, device="cuda")
    S, R, C = m.row_map()
    Wp, mp, rowmap = permute_for_lane_tiles(W, mask, S, R, C)
    enc = orc.rlc_encode(Wp, mp, 4, tile_rows=R)
    for j in range(K):
        rows, vals = m.decode_device(j)
        orows, ovals, _, _ = orc.column_entries(enc, j)
        assert np.array_equal(rows, rowmap[orows]) and np.array_equal(vals, ovals)


# ----------------------------------------------------------------------------- product
SHAPES = [
    # M, K, d_w, d_a
    (1, 1, 1.0, 1.0),
    (8, 8, 1.0, 1.0),
    (64, 64, 0.5, 0.5),
    (1000, 1003, 0.5, 0.5),
    (4097, 33, 0.3, 0.7),
    (257, 2050, 0.7, 0.3),
    (1024, 1024, 0.5, 0.5),
    (5120, 640, 0.5, 0.4),
    (11008, 300, 0.5, 0.5),
]


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("M,K,d_w,d_a", SHAPES)
def test_spmspv_random_within_bound(layout, M, K, d_w, d_a):
    seed = M * 7 + K
    W = synth.weights(seed, M, K)
    mask = synth.mask_bernoulli(seed, M, K, d_w)
    x = synth.activations(seed, K, "laplace")
    tau = synth.threshold_for_density(x, d_a)
    m = _matrix(W, mask, layout)
    y = _run(m, x, tau)
    _check_y(y, W, mask, x, tau)
    idx, val = m.last_compaction()
    oi, ov, _ = orc.compact(x, tau)
    assert np.array_equal(idx.cpu().numpy(), oi)
    assert np.array_equal(val.cpu().numpy().view(np.uint16), ov)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("M,K,d_w,d_a,tile_rows,spb", [(1000, 1003, 0.5, 0.5, 0, 0), (4096, 512, 0.5, 0.5, 0, 0),
                                                        (777, 129, 0.2, 0.9, 5, 0), (3000, 200, 0.6, 0.5, 24, 0),
                                                        (777, 129, 0.2, 0.9, 5, 2), (3000, 200, 0.6, 0.5, 24, 4),
                                                        (11008, 96, 0.5, 0.5, 0, 2), (28672, 64, 0.4, 0.6, 0, 3)])
def test_spmspv_integer_data_is_bit_exact(layout, M, K, d_w, d_a, tile_rows, spb):
    """Small-integer W and x keep every partial sum below 2^24: FP32 addition is then exact in any
    order, so the result must equal the fp64 definition bit for bit."""
    W = synth.integer_weights(M + K, M, K)
    mask = synth.mask_bernoulli(M + K, M, K, d_w)
    x = synth.integer_activations(M + K, K)
    tau = synth.threshold_for_density(x, d_a)
    m = _matrix(W, mask, layout, tile_rows, spb)
    for grid, groups, depth, cluster in ((0, 0, 0, 0), (1, 0, 0, 1), (3, 1, 1, 4), (36, 3, 2, 2), (148, 2, 4, 1),
                                        (148, 0, 0, 4), (7, 16, 0, 2)):
        # warp pairs: auto, always, never; 256: the build with every option compiled in instead of the lean ones
        for pairs in ((0, 16, 32, 256, 256 + 16) if layout == (celty.LAYOUT_LANE_TILE, 0) else (0,)):
            m.set_launch(grid=grid, variant=m.variant + pairs, groups=groups, depth=depth, cluster=cluster)
            y = _run(m, x, tau)
            _check_y(y, W, mask, x, tau, exact=True)


@pytest.mark.parametrize("M,K,tile_rows,grid,expect", [(28672, 300, 0, 0, 2), (28672, 300, 0, 20, 2), (28672, 300, 0, 9, 8),
                                                      (28672, 300, 0, 10, 4), (28672, 300, 0, 11, 1),
                                                      (14336, 257, 56, 148, 2), (11008, 96, 0, 0, 1)])
def test_spare_blocks_shared_between_row_parts(M, K, tile_rows, grid, expect):
    """Where the blocks do not divide by the row parts, the blocks left over serve several parts each (with fewer
    teams per part) when that can be done evenly (variant bit 128: wherever it can, 64: never, neither: where it
    pays).  Integer data: every setting must equal the fp64 definition bit for bit, list included."""
    W = synth.integer_weights(M + K, M, K)
    mask = synth.mask_bernoulli(M + K, M, K, 0.5)
    x = synth.integer_activations(M + K, K)
    tau = synth.threshold_for_density(x, 0.6)
    m = _matrix(W, mask, (celty.LAYOUT_LANE_TILE, 0), tile_rows, 0)
    oi, ov, _ = orc.compact(x, tau)
    for variant in (0, 128, 64, 16 + 128, 32 + 128):
        m.set_launch(grid=grid, variant=variant)
        plan = m.launch_plan()
        if variant & 128 and plan["teams_per_slab"] % max(1, expect) == 0 and plan["cluster"] == 1:
            assert plan["parts_per_spare_block"] == expect, plan
        if variant == 64:
            assert plan["parts_per_spare_block"] == 1, plan
        y = _run(m, x, tau)
        _check_y(y, W, mask, x, tau, exact=True)
        idx, val = m.last_compaction()
        assert np.array_equal(idx.cpu().numpy(), oi)
        assert np.array_equal(val.cpu().numpy().view(np.uint16), ov)


@pytest.mark.parametrize("case", range(int(os.environ.get("CELTY_RANDOM_CASES", "40"))))
def test_random_shapes_and_options(case):
    """Seeded draws (forty unless CELTY_RANDOM_CASES says otherwise) of shape, densities, tile rows, slabs per
    block and launch knobs on the fused path."""
    rng = np.random.default_rng(5000 + case)
    M = int(rng.choice([1, 7, 31, 32, 33, 100, 255, 777, 2048, 5000, 9001, 14000, 28672]))
    K = int(rng.choice([1, 5, 8, 31, 32, 33, 64, 200, 513, 1500]))
    d_w = float(rng.choice([0.02, 0.2, 0.5, 0.8, 1.0]))
    d_a = float(rng.choice([0.05, 0.3, 0.5, 0.9, 1.0]))
    tile_rows = int(rng.choice([0, 0, 0, 1, 3, 8, 17, 48, 100, 240]))
    spb = int(rng.choice([0, 0, 1, 2, 5]))
    W = synth.weights(6000 + case, M, K)
    mask = synth.mask_bernoulli(6000 + case, M, K, d_w)
    x = synth.activations(6000 + case, K, "laplace")
    tau = synth.threshold_for_density(x, d_a)
    try:
        m = celty.Matrix(W, mask, tile_rows=tile_rows, slabs_per_block=spb, device="cuda")
    except celty.CeltyError as e:                       # more than 32 slabs: a refused option, not a failure
        assert e.status == -1 and tile_rows > 0 and (M + 31) // 32 > 32 * tile_rows
        return
    grid, groups, depth, cluster = (int(rng.choice([0, 0, 1, 5, 40, 148])), int(rng.choice([0, 0, 1, 3])),
                                    int(rng.choice([0, 0, 1, 3])), int(rng.choice([0, 1, 2, 4])))
    variant = int(rng.choice([0, 0, 2, 8, 16, 24, 32, 64, 128, 144, 256, 272, 288]))
    m.set_launch(grid=grid, variant=variant, groups=groups, depth=depth, cluster=cluster)
    _check_y(_run(m, x, tau), W, mask, x, tau)
    idx, val = m.last_compaction()
    oi, ov, _ = orc.compact(x, tau)
    assert np.array_equal(idx.cpu().numpy(), oi)
    assert np.array_equal(val.cpu().numpy().view(np.uint16), ov)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_degenerate_cases(layout):
    M, K = 600, 96
    W = synth.weights(11, M, K)
    mask = synth.mask_bernoulli(11, M, K, 0.5)
    mask[:, :8] = 0                                   # empty columns
    mask[:, 8] = 0
    mask[-1, 8] = 1                                   # only the last row
    mask[:, 9] = 1                                    # dense column
    x = synth.activations(11, K, "laplace")
    m = _matrix(W, mask, layout)
    amax = float(np.abs(x.astype(np.float32)).max())
    # no survivor: y must be overwritten with zeros
    y = m.spmspv(_dev(x), amax, y=torch.full((M,), 7.0, device="cuda"))
    assert torch.count_nonzero(y).item() == 0
    # every activation survives
    xs = x.copy()
    xs[xs == 0] = np.float16(1.0)
    _check_y(_run(m, xs, 0.0), W, mask, xs, 0.0)
    # only empty columns survive
    xe = np.zeros(K, np.float16)
    xe[:8] = 1.0
    assert np.count_nonzero(_run(m, xe, 0.0)) == 0
    # unit vector selects a column exactly
    for j in (8, 9, 50):
        xu = np.zeros(K, np.float16)
        xu[j] = 1.0
        y = _run(m, xu, 0.0)
        assert np.array_equal(y, np.where(mask[:, j] != 0, W[:, j].astype(np.float32), np.float32(0)))
    # repeated calls on the same handle give the same answer
    tau = synth.threshold_for_density(x, 0.5)
    y1 = _run(m, x, tau)
    y2 = _run(m, x, tau)
    _check_y(y1, W, mask, x, tau)
    assert np.allclose(y1, y2, rtol=0, atol=1e-5)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_identity_returns_thresholded_x(layout):
    K = 300
    W = np.eye(K, dtype=np.float16)
    x = synth.activations(2, K, "laplace")
    m = _matrix(W, None, layout)
    y = _run(m, x, 0.6)
    xf = x.astype(np.float32)
    assert np.array_equal(y, np.where(np.abs(xf) > np.float32(0.6), xf, np.float32(0)))


@pytest.mark.parametrize("layout", LAYOUTS)
def test_longest_column_and_power_law_rows(layout):
    """M = 28672 (the tallest configured layer): a fully dense column (112 chunks of 256 entries),
    a column with only its last row, and row-clustered power-law masks."""
    M, K = 28672, 96
    W = synth.weights(5, M, K)
    mask = synth.mask_powerlaw(5, M, K, 0.3)
    mask[:, 0] = 1
    mask[:, 1] = 0
    mask[-1, 1] = 1
    x = synth.activations(5, K, "laplace")
    tau = synth.threshold_for_density(x, 0.7)
    x[0] = np.float16(2.0)
    x[1] = np.float16(-3.0)
    m = _matrix(W, mask, layout)
    _check_y(_run(m, x, tau), W, mask, x, tau)


def _full_size_case(W, mask, x, tau):
    """Every row within the bound, the list bit for bit, and a second call on the same handle (the tickets wrap
    around), in the launch configuration the library picks by default -- the one bench.py times."""
    m = celty.Matrix(W, mask, device="cuda")
    y_ref, a_ref = orc.masked_gemv(W, mask, x, tau, threads=orc.max_threads())
    oi, ov, _ = orc.compact(x, tau)
    xd = _dev(x)
    for call in range(2):
        y = m.spmspv(xd, tau, y=torch.full((W.shape[0],), float(call + 5), device="cuda"))
        torch.cuda.synchronize()
        assert m.last_status() == 0
        err = np.abs(y.cpu().numpy().astype(np.float64) - y_ref)
        bound = 2e-3 * a_ref + 1e-6
        worst = int(np.argmax(err - bound))
        assert np.all(err <= bound), (call, worst, err[worst], bound[worst])
        idx, val = m.last_compaction()
        assert np.array_equal(idx.cpu().numpy(), oi)
        assert np.array_equal(val.cpu().numpy().view(np.uint16), ov)


def _bench_module():
    import importlib
    return importlib.import_module("bench")


BENCH_WORKLOADS = ["llama7b_attn_4096x4096_s50_a50", "llama7b_gateup_11008x4096_s50_a50",
                   "llama7b_down_4096x11008_s50_a50", "llama13b_attn_5120x5120_s50_a40",
                   "llama13b_gateup_13824x5120_s50_a40", "llama13b_down_5120x13824_s50_a40",
                   "llama70b_mlp_28672x8192_s50_a50", "llama70b_down_8192x28672_s50_a50",
                   "llama70b_mlp_28672x8192_s30_a50", "llama70b_mlp_28672x8192_s70_a50", "small_1024x1024_s50_a50"]


@pytest.mark.parametrize("name", BENCH_WORKLOADS)
def test_every_bench_workload_at_full_size(name):
    """Each workload bench.py can time, at its full size, drawn by bench.py's own recipe (same seeds)."""
    bench = _bench_module()
    assert sorted(bench.WORKLOADS) == sorted(BENCH_WORKLOADS)          # none is left out of this test
    W, mask = bench.make_layer(name, 0)
    x, tau = bench.make_x(name, 0)
    _full_size_case(W, mask, x, tau)


@pytest.mark.parametrize("M,K,s,d_a", [(28672, 8192, 0.7, 0.3), (8192, 28672, 0.3, 0.7)])
def test_power_law_masks_of_the_large_sweep_at_full_size(M, K, s, d_a):
    """Row-clustered power-law masks of the 28672 x 8192 / 8192 x 28672 sweep (dense top rows, a long sparse tail
    with many gaps beyond 15 rows), at full size."""
    seed = synth.point_seed(5, 0)
    W = synth.weights_tiled(seed, M, K, K // 8)
    mask = synth.mask_powerlaw(seed, M, K, 1.0 - s)
    x = synth.activations(synth.point_seed(5, 50), K, "laplace")
    tau = synth.threshold_for_density(x, d_a)
    _full_size_case(W, mask, x, tau)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_tallest_layer_the_library_takes(layout):
    """M = 49152 rows (the documented limit): 12 slabs of 128 local rows."""
    M, K = 49152, 40
    W = synth.weights(77, M, K)
    mask = synth.mask_bernoulli(77, M, K, 0.3)
    x = synth.activations(77, K, "laplace")
    tau = synth.threshold_for_density(x, 0.7)
    m = _matrix(W, mask, layout)
    if layout[0] == celty.LAYOUT_LANE_TILE:
        assert m.row_map() == (12, 128, 16)
    _check_y(_run(m, x, tau), W, mask, x, tau)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("M,K,d_a", [(300, 70001, 0.05), (96, 131072, 0.5), (2049, 40000, 0.9)])
def test_very_wide_layers(layout, M, K, d_a):
    """Tens of thousands of columns: several passes of the thresholding loop and several chunks of the rank scan."""
    W = synth.weights(K + M, M, K)
    mask = synth.mask_bernoulli(K + M, M, K, 0.5)
    x = synth.activations(K + M, K, "laplace")
    tau = synth.threshold_for_density(x, d_a)
    m = _matrix(W, mask, layout)
    _check_y(_run(m, x, tau), W, mask, x, tau)
    idx, val = m.last_compaction()
    oi, ov, _ = orc.compact(x, tau)
    assert np.array_equal(idx.cpu().numpy(), oi)
    assert np.array_equal(val.cpu().numpy().view(np.uint16), ov)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_nan_activation_is_kept_and_propagates(layout):
    """NaN fails the comparison |x| <= tau, so it survives thresholding and every row with a kept weight in that
    column becomes NaN, as in the dense definition.  Zero-valued stored slots (padding entries, the slots that
    fill a lane's last group) multiply the NaN too, so a few more rows may turn NaN: the method needs finite
    activations for exact parity, and what is checked here is that nothing else is disturbed."""
    M, K = 2000, 160
    W = synth.weights(21, M, K)
    mask = synth.mask_bernoulli(21, M, K, 0.5)
    x = synth.activations(21, K, "laplace")
    x[77] = np.float16(np.nan)
    tau = synth.threshold_for_density(np.nan_to_num(x), 0.5)
    m = _matrix(W, mask, layout)
    y = _run(m, x, tau)
    y_ref, a_ref = orc.masked_gemv(W, mask, x, tau, threads=4)
    assert np.all(np.isnan(y)[np.isnan(y_ref)])
    ok = ~np.isnan(y)
    assert ok.sum() > M // 3
    assert np.all(np.abs(y[ok].astype(np.float64) - y_ref[ok]) <= 2e-3 * a_ref[ok] + 1e-6)
    idx, val = m.last_compaction()
    oi, ov, _ = orc.compact(x, tau)
    assert 77 in oi and np.array_equal(idx.cpu().numpy(), oi)
    assert np.array_equal(val.cpu().numpy().view(np.uint16), ov)


def test_back_to_back_calls_do_not_interfere():
    """Consecutive calls on one stream overlap at the seams (the next kernel is scheduled while the previous one
    drains): alternate two handles and several activation vectors, reuse one output buffer for every
    other call, and compare every result afterwards."""
    M, K = 4096, 1536
    mats, refs = [], []
    for v in range(2):
        W = synth.weights(40 + v, M, K)
        mask = synth.mask_bernoulli(40 + v, M, K, 0.5)
        mats.append((celty.Matrix(W, mask, device="cuda"), W, mask))
    xs = [synth.activations(60 + i, K, "laplace") for i in range(6)]
    taus = [synth.threshold_for_density(x, d) for x, d in zip(xs, (0.5, 0.1, 0.9, 0.3, 0.7, 0.5))]
    xd = [_dev(x) for x in xs]
    shared = torch.empty(M, dtype=torch.float32, device="cuda")
    outs = []
    for rep in range(4):
        for i in range(6):
            m = mats[i % 2][0]
            if i % 2 == 0:
                y = m.spmspv(xd[i], taus[i], y=shared)
                outs.append((i, y.clone()))                 # the clone is ordered after the call on the stream
            else:
                outs.append((i, m.spmspv(xd[i], taus[i])))
    torch.cuda.synchronize()
    for m, _, _ in mats:
        assert m.last_status() == 0
    for i, y in outs:
        _, W, mask = mats[i % 2]
        _check_y(y.cpu().numpy(), W, mask, xs[i], taus[i])


@pytest.mark.parametrize("rows", [32, 64, 96, 128])
@pytest.mark.parametrize("M,K,d_w,tile_rows", [(4096, 512, 0.5, 0), (11008, 160, 0.3, 0), (3000, 200, 0.7, 40),
                                               (28672, 64, 0.5, 0), (777, 129, 0.2, 5)])
def test_register_accumulation_variants(rows, M, K, d_w, tile_rows):
    """The software analogue of register-file accumulation (Section 4.1; the split of Section 6.4): the first
    `rows` local rows of every lane summed in registers.  Bit-exact on integer data, within the bound on random
    data, the list unchanged -- for every split, including splits beyond the tile's own rows."""
    Wi = synth.integer_weights(M + K + rows, M, K)
    mask = synth.mask_bernoulli(M + K + rows, M, K, d_w)
    xi = synth.integer_activations(M + K, K)
    m = celty.Matrix(Wi, mask, tile_rows=tile_rows, device="cuda")
    m.set_register_rows(rows)
    assert m.launch_plan()["threads"] == 256
    for grid, groups in ((0, 0), (5, 3), (148, 8)):
        m.set_launch(grid=grid, groups=groups)
        _check_y(_run(m, xi, 1.0), Wi, mask, xi, 1.0, exact=True)
    W = synth.weights(M + K, M, K)
    x = synth.activations(M + K, K, "laplace")
    tau = synth.threshold_for_density(x, 0.5)
    m2 = celty.Matrix(W, mask, tile_rows=tile_rows, device="cuda")
    m2.set_register_rows(rows)
    for _ in range(2):
        _check_y(_run(m2, x, tau), W, mask, x, tau)
    idx, val = m2.last_compaction()
    oi, ov, _ = orc.compact(x, tau)
    assert np.array_equal(idx.cpu().numpy(), oi) and np.array_equal(val.cpu().numpy().view(np.uint16), ov)
    m2.set_register_rows(0)
    assert m2.launch_plan()["threads"] == 512
    _check_y(_run(m2, x, tau), W, mask, x, tau)


def test_a_bounded_wait_that_runs_out_is_reported_and_the_handle_recovers():
    """Every wait inside the fused kernel has a poll limit.  Here one is made to run out without faulting or
    hanging anything: the limit is set low and the ticket counter that tells a block when every other block has
    cleared its share of y is moved ahead by hand, so that five blocks wait for a count that never comes.  The
    kernel must return by itself, celty_last_status must say CELTY_ETIMEOUT (and repair the counter), and the
    next call on the handle must be right again."""
    M, K = 4096, 1024
    W = synth.weights(91, M, K)
    mask = synth.mask_bernoulli(91, M, K, 0.5)
    x = synth.activations(91, K, "laplace")
    tau = synth.threshold_for_density(x, 0.5)
    m = celty.Matrix(W, mask, device="cuda")
    grid = m.launch_plan()["grid"]
    _check_y(_run(m, x, tau), W, mask, x, tau)                   # a normal call: the counter now stands at `grid`
    tickets = m._ws[8:16].view(torch.int32)
    assert int(tickets[0].item()) == grid % (2 * grid)
    m.set_wait_limit(2000)
    tickets[0] = grid + 5                                        # five blocks will land in the other half
    m.spmspv(_dev(x), tau)
    torch.cuda.synchronize()                                     # the kernel came back by itself
    assert m.last_status() == -5                                 # CELTY_ETIMEOUT
    assert celty.load().celty_strerror(-5) == b"a bounded wait inside a kernel ran out"
    m.set_wait_limit(0)
    assert m.last_status() == 0                                  # the status word was cleared
    for _ in range(2):
        _check_y(_run(m, x, tau), W, mask, x, tau)


def test_host_buffer_entry_point():
    M, K = 1024, 1024
    W = synth.weights(1, M, K)
    mask = synth.mask_bernoulli(1, M, K, 0.5)
    x = synth.activations(1, K, "normal")
    tau = synth.threshold_for_density(x, 0.5)
    m = celty.Matrix(W, mask, device="cuda")
    xh = torch.from_numpy(x.copy()).pin_memory()
    yh = torch.empty(M, dtype=torch.float32).pin_memory()
    xs = torch.empty(K, dtype=torch.float16, device="cuda")
    ys = torch.empty(M, dtype=torch.float32, device="cuda")
    m.spmspv_host(xh, tau, yh, xs, ys)
    _check_y(yh.numpy(), W, mask, x, tau)
    # ordinary (pageable) host memory
    xp, yp = torch.from_numpy(x.copy()), torch.zeros(M, dtype=torch.float32)
    m.spmspv_host(xp, tau, yp, xs, ys)
    _check_y(yp.numpy(), W, mask, x, tau)
    # an odd number of activations
    Wo, mo, xo = W[:, :K - 1].copy(), mask[:, :K - 1].copy(), x[:K - 1].copy()
    m2 = celty.Matrix(Wo, mo, device="cuda")
    xh2 = torch.from_numpy(xo).pin_memory()
    m2.spmspv_host(xh2, tau, yh, xs, ys)
    _check_y(yh.numpy(), Wo, mo, xo, tau)
