"""The GEMM tile queue (Section 4: tile queues in chunk-pipeline DAG order), decoded on the host by
the routine the device runs.  The in-order schedulers cannot deadlock only if every gemm0 tile
that a gemm1 tile waits for comes earlier in the queue; every tile must appear exactly once."""
import numpy as np
import pytest

import paper_2609_21483_b200 as pk


def replay(rows, nt0, nt1):
    rows = np.atleast_2d(np.asarray(rows, dtype=np.int32))
    q = pk.gemm_queue(rows, nt0, nt1)
    mbs = (rows + 127) // 128
    nmb = int(mbs.sum())
    assert len(q) == int(((mbs + 1) // 2).sum()) * (nt0 + nt1)
    done0 = np.zeros(nmb, np.int64)
    seen = set()
    chunk_of_mb = np.repeat(np.arange(rows.shape[0]), mbs.sum(axis=1))
    last_chunk = 0
    for ty, mb, pmb, n, chunk, nrows in q.tolist():
        gemm = ty % 3 if ty < 3 else ty - 3
        swapped = ty >= 3
        assert gemm in (0, 1) and 0 <= n < (nt0 if gemm == 0 else nt1)
        assert chunk >= last_chunk                                # chunk by chunk
        last_chunk = chunk
        blocks = [mb] if swapped else [mb, pmb]
        assert 0 < nrows <= 128
        for m in blocks:
            assert 0 <= m < nmb and chunk_of_mb[m] == chunk
            assert (gemm, m, n) not in seen
            seen.add((gemm, m, n))
            if gemm == 0:
                done0[m] += 1
            else:
                assert done0[m] == nt0, f"gemm1 tile of m-block {m} queued before its gemm0 tiles"
    # every (m-block, n-tile) of both GEMMs exactly once: a regular pair tile may cover a missing
    # second half only when the segment's m-block count is even, so the sets match exactly
    assert len(seen) == nmb * (nt0 + nt1)
    return q


SHAPES = {
    "tiny experts": lambda r, E: r.integers(0, 129, E),
    "mixed": lambda r, E: r.integers(0, 5000, E),
    "heavy tail": lambda r, E: (r.pareto(1.0, E) * 200).astype(np.int64),
    "edges": lambda r, E: r.choice([0, 1, 127, 128, 129, 255, 256, 257, 384, 2061], E),
    "mostly tiny, few huge": lambda r, E: np.where(r.random(E) < 0.9, r.integers(0, 129, E), r.integers(1000, 9000, E)),
}


@pytest.mark.parametrize("kind", list(SHAPES))
def test_dependencies_precede_and_every_tile_once(kind):
    rng = np.random.default_rng(abs(hash(kind)) % (1 << 31))
    for trial in range(40):
        E = int(rng.integers(1, 70))
        K = int(rng.choice([1, 1, 2, 4, 8]))
        rows = np.stack([SHAPES[kind](rng, E) for _ in range(K)])
        replay(rows, int(rng.integers(1, 12)), int(rng.integers(1, 9)))


def test_empty_layer_and_single_block():
    assert len(pk.gemm_queue(np.zeros((1, 5), np.int32), 3, 2)) == 0
    q = replay([[0, 7, 0]], 3, 2)
    assert (q[:, 0] >= 3).all() and len(q) == 5                   # one swapped unit: 3 gemm0 then 2 gemm1 tiles


def test_an_unpaired_block_reads_each_weight_panel_beside_its_expert():
    """One expert with five m-blocks: its last, unpaired m-block is a member of the group, so the tile
    of n-tile j comes right after the two regular pair tiles of n-tile j (same weight panel)."""
    q = replay([[128 * 5]], 3, 2)
    g0 = q[:9]
    assert list(g0[:, 0]) == [0, 0, 3] * 3 and list(g0[:, 3]) == [0, 0, 0, 1, 1, 1, 2, 2, 2]
    assert list(g0[:, 1]) == [0, 2, 4] * 3


def test_bad_arguments():
    with pytest.raises(pk.WeaveError):
        pk.gemm_queue(np.ones((3, 4), np.int32), 2, 2)            # 3 chunks
    with pytest.raises(pk.WeaveError):
        pk.gemm_queue(np.ones((8, 200), np.int32), 2, 2)          # more than 1024 segments
