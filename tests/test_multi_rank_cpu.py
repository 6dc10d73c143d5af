"""The N > 1 paths on CPU with two gloo ranks: bench.py's independent replicas (ranks only agree on the slowest
rank's time), and the host side of the n-sharded step (column slices, one all-reduce of m*m + m doubles)."""
import os
import socket
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import torch.distributed as dist

    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, world, rank)
    my_ms = 2.0 if rank == 0 else 3.5  # rank 1 is the slow replica
    slowest = bench.max_over_ranks(my_ms, world, torch.device("cpu"))
    dist.barrier()
    out[rank] = (slowest, bench.whole_job_value(slowest, world))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_whole_job():
    world, port = 2, _free_port()
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 3.5
    assert abs(res[0][1] - 2 * 1000.0 / 3.5) < 1e-9


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(1.25, 1, torch.device("cpu")) == 1.25
    assert bench.whole_job_value(2.0, 1) == 500.0


# --------------------------------------------------------------------------- n-sharded step, host side
def test_shard_columns_partitions_the_range_on_aligned_boundaries():
    sys.path.insert(0, ROOT)
    from paper_1709_05069_b200 import qn

    for n in (0, 1, 7, 8, 9, 1000, 25_600_000, (1 << 28) + 8):
        for world in (1, 2, 3, 8):
            ranges = [qn.shard_columns(n, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            for (a0, a1), (b0, b1) in zip(ranges, ranges[1:]):
                assert a1 == b0 and a0 <= a1
            assert all(b % 8 == 0 for b, _ in ranges)
            sizes = [e - b for b, e in ranges]
            assert max(sizes) - min(sizes) <= 8 + 7  # balanced up to one aligned block and the ragged end


def _shard_rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import numpy as np
    import torch.distributed as dist

    import oracle
    import workloads as W
    from paper_1709_05069_b200 import qn

    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = W.Config(21, 6003, 5, "f32", -1, 1, 0, 0.1, 1e-3, 1.0, 0.01)
    theta, g = W.generate(cfg, "cpu")  # every rank generates the same bits and keeps its slice
    gb = W.to_bits(g)
    b, e = qn.shard_columns(cfg.n, world, rank)
    mine = np.ascontiguousarray(gb[:, b:e])
    m = cfg.m
    # what qn_gram writes for this slice, from the oracle: centred Gram, then G^T gbar
    C = oracle.gram(mine)
    g64 = oracle.storage_to_f64(mine)
    gbar = g64.mean(0)
    w = (g64 - gbar) @ gbar
    buf = torch.from_numpy(np.concatenate([C.reshape(-1), w]))
    dist.all_reduce(buf, op=dist.ReduceOp.SUM)
    out[rank] = buf.numpy().copy()
    dist.destroy_process_group()


def test_sharded_gram_buffers_add_up_to_the_whole_problem():
    """Every sum over the parameter index in the method is a sum over column slices and the centring is linear:
    the all-reduced per-slice buffers equal the whole problem's centred Gram and G^T gbar (the fact that
    qn_update_sharded rests on)."""
    import numpy as np

    sys.path.insert(0, ROOT)
    import oracle
    import workloads as W

    world, port = 2, _free_port()
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_shard_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    cfg = W.Config(21, 6003, 5, "f32", -1, 1, 0, 0.1, 1e-3, 1.0, 0.01)
    theta, g = W.generate(cfg, "cpu")
    gb = W.to_bits(g)
    C = oracle.gram(gb)
    g64 = oracle.storage_to_f64(gb)
    gbar = g64.mean(0)
    w = (g64 - gbar) @ gbar
    whole = np.concatenate([C.reshape(-1), w])
    assert np.array_equal(res[0], res[1])
    scale = np.abs(C).max()
    assert np.max(np.abs(res[0][: cfg.m ** 2] - whole[: cfg.m ** 2])) <= 1e-12 * scale
    assert np.max(np.abs(res[0][cfg.m ** 2:] - whole[cfg.m ** 2:])) <= 1e-12 * max(np.abs(w).max(), scale)


def test_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` needs no GPU: it times the oracle and prints one JSON line with the keys of the
    benchmark contract (checked on the smallest configuration)."""
    import json
    import subprocess

    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "qn_update/s" and line["unit"] == "updates/s"
    assert line["steps"] == 2 and line["warmup"] == 1 and line["higher_is_better"] is True and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["cpu_baseline"]["min"] <= line["cpu_baseline"]["median"] <= line["cpu_baseline"]["max"]
    assert line["e2e"] == {"value": line["value"], "unit": "updates/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["config"]["n"] == 4096 and line["config"]["m"] == 8 and line["gpu_launches"] == 0


def _slice_rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import torch.distributed as dist

    import workloads as W
    from paper_1709_05069_b200 import qn

    dist.init_process_group("gloo", rank=rank, world_size=world)
    # what bench.py --shard n does before its first step, on the CPU: every rank forms its share of the low-rank
    # products, the shares are added over the ranks, and every rank generates only its own column slice
    cfg = W.CONFIGS[4].with_shape(n=3 * W.CHUNK + 4104, m=6)
    nchunks = (cfg.n + W.CHUNK - 1) // W.CHUNK
    c0, c1 = nchunks * rank // world, nchunks * (rank + 1) // world
    wt = W.low_rank_products(cfg, "cpu", min(c0 * W.CHUNK, cfg.n), min(c1 * W.CHUNK, cfg.n))
    dist.all_reduce(wt)
    b, e = qn.shard_columns(cfg.n, world, rank)
    theta, g = W.generate_slice(cfg, "cpu", b, e, wt)
    out[rank] = (b, e, W.to_bits(theta), W.to_bits(g))
    dist.destroy_process_group()


def test_sharded_input_generation_matches_the_whole_problem():
    """Two ranks that each generate only their column slice (the low-rank part of A couples the columns, so its
    r x m products are added over the ranks first) hold exactly the bits of the whole problem's generator."""
    import numpy as np

    sys.path.insert(0, ROOT)
    import workloads as W

    world, port = 2, _free_port()
    with mp.get_context("spawn").Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_slice_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    cfg = W.CONFIGS[4].with_shape(n=3 * W.CHUNK + 4104, m=6)
    theta, g = W.generate(cfg, "cpu")
    tb, gb = W.to_bits(theta), W.to_bits(g)
    assert res[0][0] == 0 and res[0][1] == res[1][0] and res[1][1] == cfg.n
    for r in range(world):
        b, e, ts, gs = res[r]
        assert np.array_equal(ts, tb[:, b:e])
        # the products are added in another order than in the one-process generator: the gradient may differ by one
        # rounding of the fp32 sum, i.e. by at most one unit of the storage type in a few places
        diff = np.abs(gs.astype(np.int64) - gb[:, b:e].astype(np.int64))
        assert diff.max() <= 1 and (diff > 0).mean() < 1e-3
