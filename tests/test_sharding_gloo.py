"""The N > 1 path on CPU: two gloo ranks split the independent groups of one problem, each rank
works on its share only (the CPU oracle stands in for the device here), and the union equals the
single-rank result; the timing aggregation used by bench.py (barrier, max / sum over ranks) is
exercised as well."""
import os
import socket
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, tmpdir):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2607_23844_b200 import inputs, sharding
    import oracle
    r, lr, w = sharding.init("gloo")
    assert (r, w) == (rank, world)
    wl = inputs.sd3_token_cache(seed=17, B=3, H=16, W=16, C=32, groups=(2, 2))      # 12 groups
    L = oracle.Layout(0, wl.dtype, *wl.shape, gy=2, gx=2)
    G, U = L.n_groups, L.units_per_group
    lo, hi = sharding.group_range(G, rank, world)
    # this rank's tokens only
    rows = np.array([L.unit_index(g, u) for g in range(lo, hi) for u in range(U)], dtype=np.int32)
    m = oracle.match_token(L, wl.x, rows=rows)
    np.save(os.path.join(tmpdir, f"sim{rank}.npy"), m["best_sim"])
    np.save(os.path.join(tmpdir, f"idx{rank}.npy"), m["best_idx"])
    np.save(os.path.join(tmpdir, f"rows{rank}.npy"), rows)
    sharding.barrier()
    t = sharding.max_over_ranks(1.0 + rank)
    s = sharding.sum_over_ranks(float(hi - lo))
    assert t == float(world) and s == float(G)
    sharding.finalize()


def test_group_range_partitions_every_group_once():
    sys.path.insert(0, ROOT)
    from paper_2607_23844_b200 import sharding
    for n in (0, 1, 7, 50, 148):
        for world in (1, 2, 3, 8):
            spans = [sharding.group_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.group_range(4, 2, 2)


def test_two_gloo_ranks_cover_the_problem_without_exchange(tmp_path, oracle):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    from paper_2607_23844_b200 import inputs
    wl = inputs.sd3_token_cache(seed=17, B=3, H=16, W=16, C=32, groups=(2, 2))
    L = oracle.Layout(0, wl.dtype, *wl.shape, gy=2, gx=2)
    full = oracle.match_token(L, wl.x)
    seen = np.zeros(L.n_units, bool)
    for r in range(2):
        rows = np.load(tmp_path / f"rows{r}.npy")
        sim, idx = np.load(tmp_path / f"sim{r}.npy"), np.load(tmp_path / f"idx{r}.npy")
        assert not seen[rows].any()
        seen[rows] = True
        assert np.array_equal(sim[rows], full["best_sim"][rows])
        assert np.array_equal(idx[rows], full["best_idx"][rows])
    assert seen.all()
