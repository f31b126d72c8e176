"""Pins of the oracle's chunk-overlap statistic (Sec. "Chunk Overlap", Eq. Overlap) against what the equation
fixes: its two end points, a hand-worked block, the M = 2 closed form, a library routine for the union, and the
inter-block reuse count on constructed neighbours."""
import numpy as np

import oracle


def test_end_points_of_the_equation():
    """Overlap = 1 when every query retrieves the same chunks, 0 when no chunk is shared (the text under the Eq.)."""
    K, M = 4, 8
    same = np.tile(np.array([1, 5, 6, 9]), (M, 1))
    r = oracle.chunk_overlap(same, M)
    assert r["union"].tolist() == [K] and r["total"].tolist() == [M * K] and r["overlap"].tolist() == [1.0]
    disjoint = np.arange(M * K).reshape(M, K)
    r = oracle.chunk_overlap(disjoint, M)
    assert r["union"].tolist() == [M * K] and r["overlap"].tolist() == [0.0]


def test_hand_worked_block():
    """M = 3, K = 3: I = {0,1,2}, {1,2,3}, {2,3,7}: union {0,1,2,3,7} = 5, so (9 - 5) / (2 * 3) = 2/3."""
    sel = np.array([[0, 1, 2], [1, 2, 3], [2, 3, 7]])
    r = oracle.chunk_overlap(sel, 3)
    assert r["union"].tolist() == [5] and r["total"].tolist() == [9]
    assert abs(r["overlap"][0] - 2.0 / 3.0) < 1e-15


def test_two_queries_reduce_to_the_shared_fraction():
    """M = 2: 2K - |A u B| = |A n B|, so the ratio is the fraction of chunks the two queries share."""
    rng = np.random.default_rng(3)
    K = 8
    sel = np.stack([np.sort(rng.choice(20, K, replace=False)) for _ in range(64)])
    r = oracle.chunk_overlap(sel, 2)
    for b in range(32):
        shared = len(np.intersect1d(sel[2 * b], sel[2 * b + 1]))
        assert abs(r["overlap"][b] - shared / K) < 1e-15


def test_union_and_totals_against_numpy_with_padding_and_a_short_tail():
    rng = np.random.default_rng(4)
    L, K, M = 37, 6, 8
    sel = np.full((2, 3, L, K), -1, np.int64)
    for idx in np.ndindex(2, 3, L):
        n = min(K, idx[2] // 3)                                   # early queries have fewer candidates than K
        sel[idx][:n] = np.sort(rng.choice(max(n, 12), n, replace=False))
    r = oracle.chunk_overlap(sel, M)
    assert r["union"].shape == (2, 3, 5)
    for b in range(2):
        for h in range(3):
            for blk in range(5):
                rows = sel[b, h, blk * M:(blk + 1) * M]
                ids = rows[rows >= 0]
                assert r["union"][b, h, blk] == len(np.unique(ids)) and r["total"][b, h, blk] == len(ids)
                full = rows.shape[0] == M and (rows >= 0).all()
                assert np.isnan(r["overlap"][b, h, blk]) == (not full)
                if full:
                    assert abs(r["overlap"][b, h, blk] - (M * K - len(np.unique(ids))) / ((M - 1) * K)) < 1e-15
    assert np.isnan(r["overlap"][..., 4]).all()                   # 37 = 4 * 8 + 5: the last block is short


def test_inter_block_reuse():
    """Block 1 repeats block 0's chunks (all reused), block 2 keeps half of them, block 3 shares none."""
    K, M = 4, 2
    b0 = np.array([[0, 1, 2, 3], [2, 3, 4, 5]])                   # union {0..5}
    b1 = np.array([[0, 1, 4, 5], [1, 2, 3, 4]])                   # union {0..5}: 6 reused
    b2 = np.array([[0, 1, 2, 10], [0, 1, 2, 11]])                 # union {0,1,2,10,11}: 3 reused
    b3 = np.array([[20, 21, 22, 23], [20, 21, 22, 23]])           # nothing reused
    r = oracle.chunk_overlap(np.concatenate([b0, b1, b2, b3]), M)
    assert r["union"].tolist() == [6, 6, 5, 4]
    assert r["reused"].tolist() == [0, 6, 3, 0]


def test_single_query_blocks_have_no_ratio():
    sel = np.arange(12).reshape(3, 4)
    r = oracle.chunk_overlap(sel, 1)
    assert r["union"].tolist() == [4, 4, 4] and np.isnan(r["overlap"]).all()


def test_loaded_fraction_and_overlap_against_the_numbers_the_paper_prints():
    """Fig. chunk_overlap (left) as described in the text: pool 57 -> union 43.6 is 76.4 %, pool 1032 -> union 102.1
    is 9.9 %; and by Eq. Overlap a union of 102.1 of M K = 512 slots is an overlap of (512 - 102.1) / 480 = 0.854,
    inside the 80-93 % the section reports."""
    import os
    rows, consts = [], {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "chunk_overlap_loaded_fraction.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            kv = dict(t.split("=") for t in line.split())
            if "pool" in kv:
                rows.append(kv)
            else:
                consts.update(kv)
    assert len(rows) == 2 and consts == {"M": "16", "K": "32"}
    for r in rows:
        frac = oracle.loaded_fraction(float(r["union"]), float(r["pool"]))
        assert abs(100.0 * frac - float(r["fraction_pct"])) <= 0.15          # printed to one decimal
    # a block whose 16 queries (K = 32) cover exactly 102 distinct chunks: the oracle's Eq. Overlap
    M, K = int(consts["M"]), int(consts["K"])
    sel = np.zeros((M, K), np.int64)
    ids = iter(range(32, 102))
    for m in range(M):
        sel[m] = np.arange(K)                                    # 32 chunks shared by all
    for m in range(M):                                           # 70 more distinct chunks spread over the queries
        for s in range(K - 1, K - 1 - 5, -1):
            nxt = next(ids, None)
            if nxt is not None:
                sel[m, s] = nxt
    sel.sort(axis=1)
    r = oracle.chunk_overlap(sel, M)
    assert r["union"].tolist() == [102] and abs(r["overlap"][0] - (M * K - 102) / ((M - 1) * K)) < 1e-15
    assert 0.80 <= r["overlap"][0] <= 0.93
