"""The library's host encoder against the oracle's, on the logical arrays (two independent programs)."""
import numpy as np
import pytest

from conftest import permute_for_lane_tiles, read_golden
from oracle import celty_oracle as orc
from paper_2608_01536_b200 import build, celty, synth

build.build()

CASES = [
    # M, K, d_w, layout, tile_rows
    (257, 19, 0.5, celty.LAYOUT_COLUMN, 0),
    (1000, 37, 0.3, celty.LAYOUT_COLUMN, 0),
    (4097, 5, 0.02, celty.LAYOUT_COLUMN, 0),
    (64, 7, 1.0, celty.LAYOUT_COLUMN, 0),
    (300, 9, 0.0, celty.LAYOUT_COLUMN, 0),
    (257, 19, 0.5, celty.LAYOUT_LANE_TILE, 0),
    (1000, 37, 0.3, celty.LAYOUT_LANE_TILE, 16),
    (4097, 5, 0.02, celty.LAYOUT_LANE_TILE, 100),
    (4097, 5, 0.6, celty.LAYOUT_LANE_TILE, 0),
    (64, 7, 1.0, celty.LAYOUT_LANE_TILE, 8),
    (300, 9, 0.0, celty.LAYOUT_LANE_TILE, 0),
    (33, 3, 0.5, celty.LAYOUT_LANE_TILE, 1),
]


@pytest.mark.parametrize("M,K,d_w,layout,tile_rows", CASES)
def test_encoder_matches_oracle(M, K, d_w, layout, tile_rows):
    W = synth.weights(M + K, M, K)
    mask = synth.mask_bernoulli(M + K, M, K, d_w)
    m = celty.Matrix(W, mask, layout=layout, tile_rows=tile_rows)
    info = m.info()
    R = info.tile_rows
    assert (R == 0) == (layout == celty.LAYOUT_COLUMN)
    rowmap = None
    if layout == celty.LAYOUT_LANE_TILE:
        S, R2, C = m.row_map()
        assert R2 == R and (tile_rows == 0 or R == tile_rows) and 32 * S * R >= M
        Wp, mp, rowmap = permute_for_lane_tiles(W, mask, S, R, C)
        enc = orc.rlc_encode(Wp, mp, 4, tile_rows=R)
    else:
        assert m.row_map() == (1, M, 1)
        enc = orc.rlc_encode(W, mask, 4, tile_rows=R)
    assert info.nnz == int(mask.sum())
    assert info.n_pad == int(enc.is_pad.sum())
    assert info.compressed_bytes == enc.vals.size * 5 // 2 + 4 * (K + 1)
    for j in range(K):
        rows, vals, runs, pad = m.decode_host(j)
        orows, ovals, opad, oruns = orc.column_entries(enc, j)
        if rowmap is not None:
            orows = rowmap[orows]
            assert orows.min(initial=0) >= 0
        assert np.array_equal(rows, orows)
        assert np.array_equal(vals, ovals)
        assert np.array_equal(runs, oruns)
        assert np.array_equal(pad, opad)


@pytest.mark.parametrize("case", range(60))
def test_encoder_matches_oracle_on_random_draws(case):
    """Seeded draws of shape, density and tile rows: the packed image decodes to exactly what the oracle's
    encoder produces for the row-permuted matrix."""
    rng = np.random.default_rng(7000 + case)
    M = int(rng.choice([1, 5, 31, 32, 33, 63, 100, 257, 1000, 3001]))
    K = int(rng.choice([1, 2, 7, 16]))
    d_w = float(rng.choice([0.0, 0.03, 0.3, 0.7, 1.0]))
    tile_rows = int(rng.choice([0, 1, 2, 5, 16, 33, 96, 240]))
    spb = int(rng.choice([0, 1, 3]))
    if tile_rows and (M + 31) // 32 > 32 * tile_rows:
        tile_rows = 0
    W = synth.weights(8000 + case, M, K)
    mask = synth.mask_bernoulli(8000 + case, M, K, d_w)
    m = celty.Matrix(W, mask, tile_rows=tile_rows, slabs_per_block=spb)
    S, R, C = m.row_map()
    assert 32 * S * R >= M and R % C == 0 and (tile_rows == 0 or R == tile_rows)
    Wp, mp, rowmap = permute_for_lane_tiles(W, mask, S, R, C)
    enc = orc.rlc_encode(Wp, mp, 4, tile_rows=R)
    info = m.info()
    assert info.nnz == int(mask.sum()) and info.n_pad == int(enc.is_pad.sum())
    for j in range(K):
        rows, vals, runs, pad = m.decode_host(j)
        orows, ovals, opad, oruns = orc.column_entries(enc, j)
        assert np.array_equal(rows, rowmap[orows])
        assert np.array_equal(vals, ovals) and np.array_equal(runs, oruns) and np.array_equal(pad, opad)


def test_null_mask_keeps_nonzero_weights():
    W = synth.weights(3, 100, 11)
    W[::3] = 0
    W[1, 1] = np.float16(-0.0)
    m = celty.Matrix(W, None, layout=celty.LAYOUT_COLUMN)
    enc = orc.rlc_encode(W, (W.view(np.uint16) & 0x7FFF) != 0, 4)
    assert m.info().nnz == int(((W.view(np.uint16) & 0x7FFF) != 0).sum())
    for j in range(11):
        assert np.array_equal(m.decode_host(j)[0], orc.column_entries(enc, j)[0])


@pytest.mark.parametrize("name", sorted(read_golden("rlc_hand_vectors_4bit.txt")))
@pytest.mark.parametrize("layout", [celty.LAYOUT_COLUMN, celty.LAYOUT_LANE_TILE])
def test_library_encoder_on_hand_vectors(name, layout):
    c = read_golden("rlc_hand_vectors_4bit.txt")[name]
    M = c["M"][0]
    # LANE_TILE with one slab deals row r to lane r mod 32: rows 32*i are lane 0's tile, local row i, so
    # the hand vector stretched by 32 must come back as lane 0's encoding
    stretch = 1 if layout == celty.LAYOUT_COLUMN else 32
    W = np.zeros((M * stretch, 1), np.float16)
    mask = np.zeros((M * stretch, 1), np.uint8)
    for r in c["kept_rows"]:
        W[r * stretch, 0] = r + 1
        mask[r * stretch, 0] = 1
    m = celty.Matrix(W, mask, layout=layout, tile_rows=0 if layout == celty.LAYOUT_COLUMN else max(4, M))
    if layout == celty.LAYOUT_LANE_TILE:
        assert m.row_map()[0] == 1
    rows, vals, runs, pad = m.decode_host(0)
    assert rows.tolist() == [r * stretch for r in c["rows"]]
    assert runs.tolist() == c["runs"] and pad.tolist() == c["is_pad"]


def test_packed_run_nibbles_are_little_endian():
    # 8 runs [0,15,0,15,5,1,2,3] must pack to the word 0x3215F0F0 (entry e in bits 4e..4e+3)
    rows = np.cumsum([0, 16, 1, 16, 6, 2, 3, 4])
    M = int(rows[-1]) + 1
    W = np.zeros((M, 1), np.float16)
    W[rows, 0] = np.arange(1, 9)
    m = celty.Matrix(W, None, layout=celty.LAYOUT_COLUMN)
    assert m.decode_host(0)[2].tolist() == [0, 15, 0, 15, 5, 1, 2, 3]
    image, off = m.host_image()
    # the column's single group: 16 bytes of values, then its run word
    assert image[off:off + 16].view(np.float16).tolist() == [1, 2, 3, 4, 5, 6, 7, 8]
    assert int(image[off + 16:off + 20].view(np.uint32)[0]) == 0x3215F0F0


def test_fetched_bytes_accounting():
    M, K = 512, 40
    W = synth.weights(1, M, K)
    mask = synth.mask_bernoulli(1, M, K, 0.5)
    enc = orc.rlc_encode(W, mask, 4)
    m = celty.Matrix(W, mask, layout=celty.LAYOUT_COLUMN)
    idx = np.array([0, 3, 17, 39], np.int32)
    sb, tb = m.fetched_bytes(idx)
    n_j = np.diff(enc.block_ptr)[idx]
    expect = sum(((int(n) + 7) // 8 * 20 + 15) // 16 * 16 for n in n_j)
    assert sb == expect
    assert abs(sb - 2.5 * n_j.sum()) <= 2.5 * 8 * idx.size + 16 * idx.size
    assert tb == sb + 8 * idx.size + 2 * K + 6 * idx.size + 4 * M
    assert m.fetched_bytes(np.zeros(0, np.int32)) == (0, 2 * K + 4 * M)


@pytest.mark.parametrize("run_bits", [1, 2, 3, 4, 5, 6, 8])
def test_entry_count_per_run_width_matches_oracle_encoder(run_bits):
    """celty_count_entries against the number of entries the oracle's encoder really emits at that run width,
    on Bernoulli and row-clustered masks, an empty matrix, a dense one and single-entry columns."""
    masks = []
    for M, K, d in ((257, 19, 0.5), (1000, 37, 0.1), (4097, 5, 0.02), (64, 7, 1.0), (300, 9, 0.0)):
        masks.append(synth.mask_bernoulli(M * 3 + K, M, K, d))
    masks.append(synth.mask_powerlaw(11, 2000, 13, 0.3))
    last = np.zeros((777, 3), dtype=np.uint8)
    last[776, 0] = last[255, 1] = last[256, 2] = 1                 # gaps of 776, 255 and 256 rows
    masks.append(last)
    for mask in masks:
        M, K = mask.shape
        enc = orc.rlc_encode(np.ones((M, K), dtype=np.float16), mask, run_bits=run_bits)
        nnz = int(np.count_nonzero(mask))
        assert celty.count_entries(mask, run_bits) == (nnz, len(enc.runs) - nnz)
    # by hand: a column whose only kept row is 776 needs floor(776 / 2^n) padding entries
    assert celty.count_entries(last[:, :1], run_bits) == (1, 776 >> run_bits)


def test_entry_count_rejects_bad_arguments():
    import ctypes
    lib = celty.load()
    mask = np.ones((4, 4), dtype=np.uint8)
    p = mask.ctypes.data_as(ctypes.c_void_p)
    n = ctypes.c_int64()
    assert lib.celty_count_entries(None, 4, 4, 4, 4, ctypes.byref(n), None) == -1
    assert lib.celty_count_entries(p, 4, 4, 4, 0, ctypes.byref(n), None) == -1
    assert lib.celty_count_entries(p, 4, 4, 4, 9, ctypes.byref(n), None) == -1
    assert lib.celty_count_entries(p, 3, 4, 4, 4, ctypes.byref(n), None) == -1
    assert lib.celty_count_entries(p, 4, 0, 4, 4, ctypes.byref(n), None) == -1
    assert lib.celty_count_entries(p, 4, 4, 4, 4, ctypes.byref(n), None) == 0 and n.value == 16


def test_clone_is_an_independent_copy():
    M, K = 300, 40
    W = synth.weights(3, M, K)
    mask = synth.mask_bernoulli(3, M, K, 0.4)
    a = celty.Matrix(W, mask)
    b = a.clone()
    ia, ib = a.info(), b.info()
    assert (ia.nnz, ia.n_pad, ia.tile_rows, ia.layout) == (ib.nnz, ib.n_pad, ib.tile_rows, ib.layout)
    ha, hb = a.host_image(), b.host_image()
    assert ha[1] == hb[1] and np.array_equal(ha[0], hb[0])
    del a                                                   # the copy owns its memory
    for j in (0, 7, K - 1):
        rows, vals, runs, pad = b.decode_host(j)
        kept = np.flatnonzero(mask[:, j])
        assert np.array_equal(np.sort(rows[pad == 0]), kept)


def test_stored_entries_and_layout_statistics_against_the_oracle():
    """Stored entries of a set of columns and the step / group totals of the lane-tile image, from the oracle's
    encoder on the row-permuted matrix: a sub-block (column, slab) takes as many steps as its fullest lane has groups
    of 8 entries."""
    M, K = 2100, 37
    W = synth.weights(8, M, K)
    mask = synth.mask_bernoulli(8, M, K, 0.45)
    m = celty.Matrix(W, mask)
    S, R, C = m.row_map()
    Wp, mp, _ = permute_for_lane_tiles(W, mask, S, R, C)
    ptr = orc.rlc_count(mp, 4, R)                               # entries before (column, tile); 32 * S tiles per column
    n = np.diff(ptr).reshape(K, 32 * S)
    cols = np.array([0, 5, 6, 36], np.int32)
    assert m.stored_entries(cols) == int(n[cols].sum())
    groups = (n + 7) // 8
    per_sub = groups.reshape(K, S, 32)
    nb, steps, total_groups = m.layout_stats()
    assert nb == K * S
    assert steps == int(per_sub.max(axis=2).sum())
    assert total_groups == int(groups.sum())
    col = celty.Matrix(W, mask, layout=celty.LAYOUT_COLUMN)
    with pytest.raises(celty.CeltyError):
        col.layout_stats()


@pytest.mark.parametrize("M,K,slabs,rows", [(4096, 4096, 2, 64), (4096, 6144, 2, 64), (4096, 6145, 1, 128), (4096, 11008, 1, 128),
                                            (1024, 1024, 2, 16), (512, 512, 1, 16), (5120, 5120, 2, 80), (11008, 4096, 3, 128),
                                            (28672, 64, 8, 120)])
def test_default_tile_shape(M, K, slabs, rows):
    """The library's own choice of slabs and rows per tile: one slab per 4096 rows, two for a layer of one slab and
    few columns (it streams for so short a time that halving what a block adds into y at the end is worth more than
    large sub-blocks), fewer rows per tile on very tall layers so that eight teams fit shared memory.  Every row has
    exactly one place whatever the shape."""
    W = synth.weights(77, M, K) if M * K <= 1 << 22 else np.zeros((M, K), np.float16)
    mask = synth.mask_bernoulli(78, M, K, 0.5)
    m = celty.Matrix(W, mask)
    S, R, C = m.row_map()
    assert (S, R) == (slabs, rows)
    assert 32 * S * R >= M and R % C == 0
