"""Host logic of the dense backward contractions' unit list (ngc_dense_schedule), no GPU needed.

The CTA-pair kernels compute D^T = A^T B per partition with A's columns in M blocks of 256 and B's columns in
passes of 512, some passes cut into halves; whatever the cut, every (partition, M block, column of B) must be
produced by exactly one unit, every pair must get its units in rounds, and cutting must never make the longest
pair longer than not cutting at all.
"""
import numpy as np
import pytest

import paper_2212_08580_b200 as ngc

SHAPES = [
    # batch, m_blocks, n_cols, k_chunks, max_pairs
    (50, 1, 1024, 64, 74),      # softmax50: G_j = X_j^T R_j
    (30, 2, 785, 32, 74),       # mlp30: [dW1; db1]
    (1, 1, 8, 1, 74),
    (1, 1, 256, 1, 74),
    (3, 1, 520, 5, 74),
    (7, 2, 96, 3, 74),
    (4, 1, 1024, 8, 74),
    (100, 1, 2048, 10, 74),
    (9, 3, 1536, 4, 5),
    (2, 1, 512, 2, 1),
    (33, 1, 1000, 7, 66),
]


@pytest.mark.parametrize("batch,m_blocks,n_cols,k_chunks,max_pairs", SHAPES)
def test_units_cover_every_column_once(batch, m_blocks, n_cols, k_chunks, max_pairs):
    units, pairs = ngc.dense_schedule(batch, m_blocks, n_cols, k_chunks, max_pairs)
    assert 1 <= pairs <= max_pairs and pairs <= len(units)
    seen = np.zeros((batch, m_blocks, n_cols), dtype=np.int32)
    for pair, rnd, j, mt, c0, w0, c1, w1 in units:
        assert 0 <= pair < pairs and 0 <= j < batch and 0 <= mt < m_blocks
        assert w0 > 0 and w0 % 32 == 0 and w0 <= 256 and w1 % 32 == 0 and 0 <= w1 <= 256
        assert c0 % 256 == 0 and c0 < n_cols
        seen[j, mt, c0:min(c0 + w0, n_cols)] += 1
        if w1:
            assert c1 == c0 + 256 and w0 == 256 and c1 < n_cols     # a second range only behind a full first one
            seen[j, mt, c1:min(c1 + w1, n_cols)] += 1
        # nothing a unit covers lies wholly past the matrix, and a range overshoots by less than 32 columns
        assert c0 + w0 - n_cols < 32 and (w1 == 0 or c1 + w1 - n_cols < 32)
    assert (seen == 1).all()


@pytest.mark.parametrize("batch,m_blocks,n_cols,k_chunks,max_pairs", SHAPES)
def test_units_are_dealt_in_rounds(batch, m_blocks, n_cols, k_chunks, max_pairs):
    units, pairs = ngc.dense_schedule(batch, m_blocks, n_cols, k_chunks, max_pairs)
    rounds = -(-len(units) // pairs)
    per_pair = {}
    for pair, rnd, *_ in units:
        per_pair.setdefault(int(pair), []).append(int(rnd))
    for pair, r in per_pair.items():
        assert r == sorted(set(r)) and r[-1] < rounds       # at most one unit per round, in order
    # every round but the last is full
    counts = np.bincount(units[:, 1], minlength=rounds)
    assert (counts[:-1] == pairs).all() and 1 <= counts[-1] <= pairs


def _bytes_moved(units, k_chunks):
    """Operand bytes a pair's units bring into shared memory (per CTA): 16 KB of A plus 8 KB per 64-column box of B
    per chunk: the quantity the cut is meant to balance."""
    load = {}
    for pair, rnd, j, mt, c0, w0, c1, w1 in units:
        boxes = -(-(w0 // 2) // 64) + -(-(w1 // 2) // 64)
        load[int(pair)] = load.get(int(pair), 0) + k_chunks * (16384 + 8192 * boxes)
    return load


def test_cut_passes_even_out_the_two_benchmark_shapes():
    # softmax50: 100 whole passes on 74 pairs would give 26 pairs two passes (192 KB per chunk) and 48 pairs one;
    # with 26 passes cut the longest pair carries one pass and one half (160 KB per chunk)
    units, pairs = ngc.dense_schedule(50, 1, 1024, 64, 74)
    assert pairs == 74 and len(units) == 74 + 52
    assert sum(1 for u in units if u[7]) == 74 and sum(1 for u in units if not u[7]) == 52
    load = _bytes_moved(units, 64)
    assert max(load.values()) == 64 * (49152 + 32768)
    # mlp30: never worse than the uncut list (one whole pass and one ragged pass on the longest pair)
    units, pairs = ngc.dense_schedule(30, 2, 785, 32, 74)
    load = _bytes_moved(units, 32)
    assert max(load.values()) <= 32 * (49152 + 40960)


def test_argument_errors():
    lib = ngc.load_library()
    import ctypes as C
    n, p = C.c_int32(0), C.c_int32(0)
    assert lib.ngc_dense_schedule(0, 1, 8, 1, 1, None, 0, C.byref(n), C.byref(p)) != 0
    assert lib.ngc_dense_schedule(1, 1, 8, 1, 1, None, 4, C.byref(n), C.byref(p)) != 0     # cap > 0 without a buffer
    assert lib.ngc_dense_schedule(1, 1, 8, 1, 1, None, 0, None, C.byref(p)) != 0
