"""The multi-GPU host logic on CPU: two gloo ranks shard the rows, all-reduce the per-channel statistics and
agree with the single-process fit; timing is combined with a max over ranks."""
import os
import socket

import numpy as np
import pytest

from paper_2505_20932_b200 import sharding


def test_shard_rows_partition():
    for total, world, align in [(403456, 8, 128), (788, 2, 128), (5, 4, 1), (0, 3, 8), (12608, 3, 197), (100, 7, 16)]:
        spans = [sharding.shard_rows(total, world, r, align) for r in range(world)]
        pos = 0
        for (s, n) in spans:
            assert s == pos and n >= 0
            pos += n
        assert pos == total
        full = [n for (_, n) in spans if n > 0]
        assert all(n % align == 0 for n in full[:-1])
        if full:
            assert max(full) - min(full[:-1] or full) <= align
    with pytest.raises(ValueError):
        sharding.shard_rows(10, 2, 2)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, rows, C, out):
    import torch
    import torch.distributed as dist
    from oracle import qwt_oracle as O
    from paper_2505_20932_b200 import workload as WL
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        fp, q, _ = WL.host_calib_pair(rows, C, 4, seed=21)       # every rank draws the same bytes, keeps its shard
        s, n = sharding.shard_rows(rows, world, rank, align=8)
        local = O.cwac_stats(fp[s:s + n], q[s:s + n]) if n > 0 else np.zeros((5, C))
        if n == 0:
            local[0] = 0
        t = torch.from_numpy(local.reshape(-1).copy())
        sharding.allreduce_stats_(t)
        slowest = sharding.max_over_ranks(0.25 * (rank + 1))
        if rank == 0:
            np.save(out, np.concatenate([t.numpy(), [slowest]]))
    finally:
        dist.destroy_process_group()


def test_two_rank_statistics_allreduce_matches_single_process(tmp_path):
    import torch.multiprocessing as mp
    from oracle import qwt_oracle as O
    from paper_2505_20932_b200 import workload as WL
    rows, C, world = 1001, 24, 2
    out = str(tmp_path / "stats.npy")
    mp.spawn(_worker, args=(world, _free_port(), rows, C, out), nprocs=world, join=True)
    got = np.load(out)
    stats, slowest = got[:-1].reshape(5, C), got[-1]
    assert slowest == 0.5                                   # max over ranks of (0.25, 0.5)
    fp, q, _ = WL.host_calib_pair(rows, C, 4, seed=21)
    ref = O.cwac_stats(fp, q)
    assert np.allclose(stats, ref, rtol=1e-12, atol=1e-9)
    n, sq, sf, sqf, sqq = stats
    var = sqq / n - (sq / n) ** 2
    a = (sqf / n - (sq / n) * (sf / n)) / var
    b = sf / n - a * sq / n
    a_ref, b_ref, _ = O.cwac_fit(fp, q)
    assert np.allclose(a, a_ref, rtol=1e-9) and np.allclose(b, b_ref, rtol=1e-7, atol=1e-12)


class _CpuBinding:
    """Stands in for the ctypes binding on CPU tensors so that calibrate_sharded itself runs under gloo: the two calls
    it makes are answered with the oracle's sums and with Eq. 4-5 written out."""

    def qwt_cwac_stats_accumulate(self, fp, q, rows, C, ld, stats, ws, wsb, stream=None):
        import torch
        from oracle import qwt_oracle as O
        stats += torch.from_numpy(O.cwac_stats(fp.numpy()[:rows, :C], q.numpy()[:rows, :C]).reshape(-1))

    def qwt_cwac_solve(self, stats, C, a, b, nd, stream=None):
        import torch
        n, sq, sf, sqf, sqq = stats.reshape(5, C)
        alpha = (sqf / n - (sq / n) * (sf / n)) / (sqq / n - (sq / n) ** 2)
        a.copy_(alpha.float())
        b.copy_((sf / n - alpha * sq / n).float())


def _worker_sharded(rank, world, port, rows, C, out):
    import torch
    import torch.distributed as dist
    from paper_2505_20932_b200 import workload as WL
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        fp, q, _ = WL.host_calib_pair(rows, C, 4, seed=22)
        s, n = sharding.shard_rows(rows, world, rank, align=8)
        a, b = torch.empty(C), torch.empty(C)
        stats = torch.zeros(5 * C, dtype=torch.float64)
        sharding.calibrate_sharded(_CpuBinding(), torch.from_numpy(fp[s:s + n]), torch.from_numpy(q[s:s + n]), n, C, C,
                                   a, b, stats, None, 0)
        np.save(out + f".{rank}.npy", np.stack([a.numpy(), b.numpy()]))
    finally:
        dist.destroy_process_group()


def test_calibrate_sharded_over_two_ranks(tmp_path):
    import torch.multiprocessing as mp
    from oracle import qwt_oracle as O
    from paper_2505_20932_b200 import workload as WL
    rows, C, world = 1203, 16, 2
    out = str(tmp_path / "ab")
    mp.spawn(_worker_sharded, args=(world, _free_port(), rows, C, out), nprocs=world, join=True)
    fp, q, _ = WL.host_calib_pair(rows, C, 4, seed=22)
    a_ref, b_ref, _ = O.cwac_fit(fp, q)
    r0, r1 = np.load(out + ".0.npy"), np.load(out + ".1.npy")
    assert np.array_equal(r0, r1)                            # every rank solves the same summed statistics
    assert np.allclose(r0[0], a_ref, rtol=1e-6) and np.allclose(r0[1], b_ref, rtol=1e-6, atol=1e-7)
