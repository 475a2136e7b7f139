"""Pins for the oracle's RLC-CSC encoder/decoder (Section 3.2, Algorithm 1).

Expected values come from the paper's printed example, hand-derived vectors, closed forms
and invariants computed here with plain numpy from the mask -- never from the encoder.
"""
import numpy as np
import pytest

from conftest import read_golden
from oracle import celty_oracle as orc
from paper_2608_01536_b200 import synth


def _encode_single_column(values, kept, run_bits, tile_rows=0):
    W = np.asarray(values, dtype=np.float16).reshape(-1, 1)
    mask = np.asarray(kept, dtype=np.uint8).reshape(-1, 1)
    return orc.rlc_encode(W, mask, run_bits=run_bits, tile_rows=tile_rows)


def test_paper_example_2bit():
    c = read_golden("rlc_example_section_3_2.txt")["paper_2bit"]
    col = c["column"]
    kept = [v != 0 for v in col]
    # literal-loop version
    v, r, p = orc.rlc_encode_column_py(col, kept, c["run_bits"][0])
    assert v == c["values"] and r == c["runs"] and [int(b) for b in p] == c["is_pad"]
    assert orc.rlc_decode_column_py(r) == c["rows"]
    # C version
    enc = _encode_single_column(col, kept, c["run_bits"][0])
    assert enc.vals.view(np.float16).astype(int).tolist() == c["values"]
    assert enc.runs.tolist() == c["runs"]
    assert enc.is_pad.tolist() == c["is_pad"]
    assert enc.rows.tolist() == c["rows"]


@pytest.mark.parametrize("name", sorted(read_golden("rlc_hand_vectors_4bit.txt")))
def test_hand_vectors_4bit(name):
    c = read_golden("rlc_hand_vectors_4bit.txt")[name]
    M = c["M"][0]
    col = np.zeros(M, np.float16)
    kept = np.zeros(M, bool)
    for r in c["kept_rows"]:
        col[r] = r + 1
        kept[r] = True
    expect_vals = [0 if p else row + 1 for row, p in zip(c["rows"], c["is_pad"])]
    for enc_vals, runs, pads, rows in (
        (lambda e: (e.vals.view(np.float16).astype(int).tolist(), e.runs.tolist(),
                    e.is_pad.tolist(), e.rows.tolist()))(_encode_single_column(col, kept, 4)),
        (lambda t: ([int(v) for v in t[0]], t[1], [int(b) for b in t[2]],
                    orc.rlc_decode_column_py(t[1])))(orc.rlc_encode_column_py(col, kept, 4)),
    ):
        assert runs == c["runs"]
        assert pads == c["is_pad"]
        assert rows == c["rows"]
        assert enc_vals == expect_vals


def _gaps_per_column(mask):
    """Lengths of the zero runs that precede each kept element, per column (numpy only)."""
    out = []
    for j in range(mask.shape[1]):
        rows = np.flatnonzero(mask[:, j])
        prev = np.concatenate(([-1], rows[:-1]))
        out.append(rows - prev - 1)
    return out


@pytest.mark.parametrize("M,K,d_w,seed", [(257, 19, 0.5, 1), (1000, 37, 0.3, 2), (513, 8, 0.08, 3),
                                           (64, 5, 1.0, 4), (300, 7, 0.0, 5), (4097, 3, 0.02, 6)])
def test_invariants_random(M, K, d_w, seed):
    W = synth.weights(seed, M, K)
    mask = synth.mask_bernoulli(seed, M, K, d_w)
    enc = orc.rlc_encode(W, mask, 4)
    # every run fits 4 bits; pads carry the maximum run and value +0
    assert enc.runs.max(initial=0) <= 15
    assert np.all(enc.runs[enc.is_pad == 1] == 15)
    assert np.all(enc.vals[enc.is_pad == 1] == 0)
    gaps = _gaps_per_column(mask)
    for j in range(K):
        rows, vals, pad, runs = orc.column_entries(enc, j)
        assert np.all(np.diff(rows) > 0) and (rows.size == 0 or (rows[0] >= 0 and rows[-1] < M))
        # non-pad entries are exactly the kept elements, in order, with their bit patterns
        kept_rows = np.flatnonzero(mask[:, j])
        assert np.array_equal(rows[pad == 0], kept_rows)
        assert np.array_equal(vals[pad == 0], W.view(np.uint16)[kept_rows, j])
        # minimal padding: floor(gap / 16) pads per gap, none after the last kept row
        assert int(pad.sum()) == int((gaps[j] // 16).sum())
        # run of a real entry = gap mod 16
        assert np.array_equal(runs[pad == 0], gaps[j] % 16)
    # round trip as a dense matrix, bitwise
    dense = orc.rlc_to_dense(enc)
    assert np.array_equal(dense, np.where(mask.astype(bool), W.view(np.uint16), 0))


@pytest.mark.parametrize("tile_rows", [16, 100, 128, 333])
def test_tiled_encoding_is_the_rule_per_tile(tile_rows):
    M, K = 700, 11
    W = synth.weights(9, M, K)
    mask = synth.mask_bernoulli(9, M, K, 0.2)
    enc = orc.rlc_encode(W, mask, 4, tile_rows=tile_rows)
    T = -(-M // tile_rows)
    assert enc.T == T
    for j in range(K):
        for t in range(T):
            r0, r1 = t * tile_rows, min(M, (t + 1) * tile_rows)
            v, r, p = orc.rlc_encode_column_py(W.view(np.uint16)[r0:r1, j], mask[r0:r1, j], 4)
            b0, b1 = enc.block_ptr[j * T + t], enc.block_ptr[j * T + t + 1]
            assert enc.vals[b0:b1].tolist() == [int(x) for x in v]
            assert enc.runs[b0:b1].tolist() == r
            assert enc.rows[b0:b1].tolist() == orc.rlc_decode_column_py(r, r0)
            assert np.all(enc.rows[b0:b1] < r1)
    assert np.array_equal(orc.rlc_to_dense(enc), np.where(mask.astype(bool), W.view(np.uint16), 0))


def test_kept_zero_and_negative_zero_are_stored():
    col = np.array([0.0, -0.0, 1.0, 0.0], np.float16)
    kept = [True, True, False, True]
    enc = _encode_single_column(col, kept, 4)
    assert enc.vals.tolist() == [0x0000, 0x8000, 0x0000]
    assert enc.runs.tolist() == [0, 0, 1]
    assert enc.is_pad.tolist() == [0, 0, 0]


def test_last_row_only_has_maximum_pads():
    M = 1000
    kept = np.zeros(M, bool)
    kept[-1] = True
    enc = _encode_single_column(np.ones(M), kept, 4)
    assert int(enc.is_pad.sum()) == (M - 1) // 16
    assert enc.rows[-1] == M - 1
    assert enc.runs[-1] == (M - 1) % 16


@pytest.mark.parametrize("s,expected", [(0.3, 0.8750), (0.5, 0.6250), (0.7, 0.3763)])
def test_compression_efficiency_closed_form(s, expected):
    """Section 3.2: 4-bit RLC-CSC takes ~63% of dense FP16 at 50% sparsity on 4096x4096.

    Closed form on a Bernoulli mask with density d = 1 - s: stored entries per element are
    d * (1 + rho), rho = s^16 / (1 - s^16) pads per non-zero; each entry costs 20 bits."""
    d = 1.0 - s
    rho = s ** 16 / (1.0 - s ** 16)
    closed = d * (1.0 + rho) * 20.0 / 16.0
    assert abs(closed - expected) < 5e-4
    M, K = 2048, 96
    mask = synth.mask_bernoulli(int(s * 100), M, K, d)
    enc = orc.rlc_encode(synth.weights(1, M, K), mask, 4)
    measured = enc.vals.size * 2.5 / (2.0 * M * K)
    assert abs(measured - closed) < 0.01
    if s == 0.5:
        assert round(measured, 2) in (0.62, 0.63)   # "approximately 63%"


def test_c_encoder_matches_literal_loop_random():
    rng = np.random.default_rng(0)
    for _ in range(50):
        M = int(rng.integers(1, 200))
        d = rng.choice([0.02, 0.1, 0.5, 0.9])
        kept = rng.random(M) < d
        col = rng.integers(1, 100, M).astype(np.float16)
        for bits in (2, 4):
            v, r, p = orc.rlc_encode_column_py(col.view(np.uint16), kept, bits)
            enc = _encode_single_column(col, kept, bits)
            assert enc.vals.tolist() == [int(x) for x in v]
            assert enc.runs.tolist() == r
            assert enc.is_pad.tolist() == [int(b) for b in p]
            assert enc.rows.tolist() == orc.rlc_decode_column_py(r)
