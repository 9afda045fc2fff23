"""Host-side logic of bench.py: work accounting, cell sampling, and the multi-rank reduction (gloo, 2 ranks)."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
import synth  # noqa: E402


def brute_force_tiles(wl, lists):
    """Tiles the attention kernels issue: per 128-row tile, the listed blocks not entirely above its last row."""
    n = 0
    for (h, i), lst in lists.items():
        for qt in range(wl.L_S // 128):
            last = i * wl.L_S + qt * 128 + 127
            n += sum(1 for j in lst if j * wl.L_B <= last)
    return n


def test_executed_tiles_matches_brute_force():
    rng = np.random.default_rng(0)
    for (L_S, L_B) in [(128, 64), (256, 128), (512, 128), (1024, 128), (256, 64)]:
        wl = synth.Workload("t", 3, 1, 128, 4 * L_S, L_S, L_B, 0.5, 0.5, 1, 1)
        lists, k = {}, np.zeros((wl.H, wl.C_S), np.int32)
        for h in range(wl.H):
            for i in range(wl.C_S):
                cand = np.arange(wl.r * i)
                keep = cand[rng.random(cand.size) < 0.5]
                lst = list(keep) + list(range(wl.r * i, wl.r * (i + 1)))
                lists[(h, i)] = lst
                k[h, i] = len(lst)
        assert bench.executed_tiles(wl, k) == brute_force_tiles(wl, lists)


def test_sample_cells_is_stratified_and_seeded():
    wl = synth.WORKLOADS["llama3_8b_32k"]
    rigid = np.array([1, 0] * (wl.H // 2), np.uint8)
    a = bench.sample_cells(wl, rigid, 24, seed=1)
    b = bench.sample_cells(wl, rigid, 24, seed=1)
    assert a == b and len(a) == 24
    assert {rigid[h] for h, _ in a} == {0, 1}
    assert min(i for _, i in a) == 0 and max(i for _, i in a) == wl.C_S - 1


def test_job_value_counts_all_replicas():
    assert bench.job_value(8.0, 1) == 8.0 and bench.job_value(8.0, 4) == 2.0


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        v = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")   # the slower rank decides
        dist.barrier()
        out[rank] = v
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_two_gloo_ranks():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = mp.get_context("spawn").Manager().dict()
    mp.spawn(_rank_main, args=(2, port, out), nprocs=2, join=True)
    assert out[0] == out[1] == 15.0
    assert bench.max_over_ranks(3.0) == 3.0


# ---------------------------------------------------------------- a layer sharded by KV group: the host-side logic
def test_shard_heads_partitions_whole_kv_groups():
    H, Hkv = 32, 8
    for world in (1, 2, 4, 8):
        parts = [bench.shard_heads(H, Hkv, r, world) for r in range(world)]
        assert [p[0] for p in parts] == [r * H // world for r in range(world)]
        assert parts[-1][1] == H and parts[-1][3] == Hkv
        for h0, h1, g0, g1 in parts:
            assert (h1 - h0) == (g1 - g0) * (H // Hkv) and h0 == g0 * (H // Hkv)
    try:
        bench.shard_heads(28, 4, 0, 8)
        assert False
    except ValueError:
        pass
    wl = synth.WORKLOADS["llama3_8b_32k"]
    import oracle
    assert bench.total_blocks_all(wl) == oracle.total_blocks(wl.fraction, wl.H, wl.C_S, wl.r)


def _shard_rank_main(rank, world, port, out):
    """What one rank of `bench.py --shard kv` does with the tables, on the CPU with the oracle in place of the
    kernels: multipliers of its heads, all-gather, apportionment of the layer's total over the gathered table."""
    import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        H, Hkv, C_S, r = 8, 4, 12, 2
        rng = np.random.default_rng(5)                       # every rank draws the same table, keeps its rows
        e32 = (rng.random((H, C_S)) * np.where(rng.random((H, 1)) < 0.4, 1e-7, 1.0)).astype(np.float32)
        h0, h1, _, _ = bench.shard_heads(H, Hkv, rank, world)
        _, m_loc = oracle.multipliers(e32[h0:h1])
        M_loc = torch.from_numpy(np.floor(m_loc * 4096.0 + 0.5).astype(np.int32))
        M_all = torch.empty((H, C_S), dtype=torch.int32)
        dist.all_gather_into_tensor(M_all.view(-1), M_loc.view(-1))
        T = oracle.total_blocks(0.4, H, C_S, r)
        k_all, b_star = oracle.budgets_total(M_all.numpy().astype(np.float64) / 4096.0, r, T)
        out[rank] = (k_all[h0:h1].tolist(), b_star, M_all.numpy().tolist())
    finally:
        dist.destroy_process_group()


def test_gathered_multiplier_tables_give_the_global_apportionment_two_gloo_ranks():
    import oracle
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    out = mp.get_context("spawn").Manager().dict()
    mp.spawn(_shard_rank_main, args=(2, port, out), nprocs=2, join=True)
    H, C_S, r = 8, 12, 2
    rng = np.random.default_rng(5)
    e32 = (rng.random((H, C_S)) * np.where(rng.random((H, 1)) < 0.4, 1e-7, 1.0)).astype(np.float32)
    _, m = oracle.multipliers(e32)                           # the whole layer at once
    k, b_star = oracle.budgets_total(m, r, oracle.total_blocks(0.4, H, C_S, r))
    assert out[0][2] == out[1][2] == np.floor(m * 4096.0 + 0.5).astype(np.int32).tolist()   # rows in head order
    assert out[0][1] == out[1][1] == b_star
    assert out[0][0] + out[1][0] == k.tolist()
    assert int(k.sum()) == oracle.total_blocks(0.4, H, C_S, r)
