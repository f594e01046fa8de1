"""World-size-2 checks of the multi-GPU plumbing on CPU (gloo): the path shards by
query stream with no data-path collective, so what is covered is the partition of
the stream and the barrier / max-over-ranks timing protocol of the benchmark."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2502_15572_b200 import dist_util


def test_query_slices_partition_the_stream():
    for n in (0, 1, 7, 1000, 1001):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                sl = dist_util.query_slice(n, r, world)
                seen.extend(sl)
                assert abs(len(sl) - n / world) < 1
            assert seen == list(range(n))
    with pytest.raises(ValueError):
        dist_util.query_slice(10, 2, 2)


def test_aggregate_throughput():
    assert dist_util.aggregate_throughput(1, 1000, 1, 800.0) == pytest.approx(1250.0)
    assert dist_util.aggregate_throughput(64, 100, 8, 100.0) == pytest.approx(512000.0)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert dist_util.rank_info() == (rank, rank, world)
        sl = dist_util.query_slice(1001, rank, world)
        dist.barrier()
        mine = [10.0 + rank, 5.0 - rank, float(len(sl))]
        got = dist_util.max_over_ranks(mine)
        dist.barrier()
        out.put((rank, got, (sl.start, sl.stop)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo_max_and_partition():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1] == [11.0, 5.0, 501.0]          # element-wise max over both ranks
    assert res[0][2] == (0, 501) and res[1][2] == (501, 1001)    # disjoint, covering


def _gather_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, n, L = 3, 4, 2
        rows = dist_util.shard_rows(1001, rank, world)
        ids = torch.arange(B * n, dtype=torch.int32).reshape(B, n) + 100 * rank
        scores = torch.full((B, n), float(rank), dtype=torch.float32)
        tokens = torch.full((B, n, L), 7 + rank, dtype=torch.int32)
        g = dist_util.gather_shard_results(ids, scores, tokens, rows.start)
        out.put((rank, [t.tolist() for t in g]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo_gather_of_shard_results():
    """The exchange step of the row-sharded mode: every rank ends up with all shards'
    results stacked by rank, and with the shards' row offsets."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_gather_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1]                                  # both ranks hold the same gathered view
    ids, scores, tokens, offsets = res[0][1]
    assert offsets == [0, 501]
    assert ids[0][0] == [0, 1, 2, 3] and ids[1][0] == [100, 101, 102, 103]
    assert scores[0][0][0] == 0.0 and scores[1][0][0] == 1.0
    assert tokens[0][0][0] == [7, 7] and tokens[1][0][0] == [8, 8]


def _packed_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        B, n, L = 3, 4, 2
        rows = dist_util.shard_rows(1001, rank, world)
        ex = dist_util.PackedExchange(B, n, L, rows.start, "cpu")
        ex.ids.copy_(torch.arange(B * n, dtype=torch.int32).reshape(B, n) + 100 * rank)
        ex.scores.fill_(0.5 + rank)
        ex.tokens.fill_(7 + rank)
        first = ex.exchange().clone()
        ex.scores.fill_(2.5 + rank)                    # the buffers are reused by the next call
        second = ex.exchange().clone()
        out.put((rank, ex.words, ex.offsets.tolist(), first.tolist(), second.view(torch.float32).tolist()))
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo_packed_exchange_is_one_block_per_rank():
    """The single-collective form of the exchange step: the three result arrays of a rank travel
    as one block ids | scores | tokens, the layout the packed merge kernel reads."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_packed_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    B, n, L = 3, 4, 2
    bn = B * n
    assert res[0][1:] == res[1][1:]                                # both ranks hold the same view
    _, words, offsets, first, second = res[0]
    assert words == bn * (2 + L) and offsets == [0, 501] and len(first) == 2 * words
    for r in range(2):
        blk = first[r * words:(r + 1) * words]
        assert blk[:bn] == [i + 100 * r for i in range(bn)]        # ids
        assert torch.tensor(blk[bn:2 * bn], dtype=torch.int32).view(torch.float32).tolist() == [0.5 + r] * bn
        assert blk[2 * bn:] == [7 + r] * (bn * L)                  # tokens
        assert second[r * words + bn:r * words + 2 * bn] == [2.5 + r] * bn


def test_sharded_row_count_must_fit_int32():
    """Merged ids are int32 row indices: shards whose rows pass 2^31 - 1 in all are refused."""
    dist_util.check_global_rows([0, 2 ** 30], [2 ** 30, 2 ** 30 - 1])
    with pytest.raises(ValueError):
        dist_util.check_global_rows([0, 2 ** 30], [2 ** 30, 2 ** 30])
    with pytest.raises(ValueError):
        dist_util.PackedExchange(1, 4, 2, 2 ** 31 - 10, "cpu", n_rows=100)
    ex = dist_util.PackedExchange(1, 4, 2, 2 ** 31 - 200, "cpu", n_rows=100)
    assert ex.offsets.tolist() == [2 ** 31 - 200]


def _inputs_worker(rank, world, port, out, shard_rows):
    import sys
    import numpy as np
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        argv = ["--workload", "c2_decode_b1_f16", "--rows", "150001", "--gpus", str(world)]
        sys.argv = ["bench.py"] + argv + (["--shard-rows"] if shard_rows else [])
        args = bench.parse_args()
        cfg, keys, toks, q, shard, host = bench.device_inputs(args, rank, world, device="cpu")
        out.put((rank, keys.view(torch.int16).numpy().copy(), toks.numpy().copy(), q.view(torch.int16).numpy().copy(),
                 None if shard is None else (shard.start, shard.stop), host is not None,
                 np.asarray(cfg.get("first_tokens", []))))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("shard_rows", [False, True])
def test_two_ranks_gloo_bench_inputs(shard_rows):
    """How bench.py hands the workload to N ranks.  Replicas: rank 0 generates, every rank ends
    up with the same datastore and queries.  Sharded rows: every rank generates only its rows,
    the shards tile the one datastore, and all ranks hold the queries of the 1-rank run."""
    import numpy as np
    from paper_2502_15572_b200 import synth
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_inputs_worker, args=(r, 2, port, out, shard_rows)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((out.get(timeout=300) for _ in procs), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = synth.WORKLOADS["c2_decode_b1_f16"]
    N = 150001
    keys, toks = synth.make_store(w["seed"], N, w["d"], w["C"], w["dtype"], w["stored_len"])
    q, src = synth.make_queries(w["seed"] + 100, keys, w["dtype"], 1000, w["sigma"])
    for r in res:
        assert np.array_equal(r[3], q.view(np.int16))              # the same queries on every rank
    if shard_rows:
        assert res[0][4] == (0, 75001) and res[1][4] == (75001, N)
        assert np.array_equal(np.concatenate([res[0][1], res[1][1]]), keys.view(np.int16))
        assert np.array_equal(np.concatenate([res[0][2], res[1][2]]), toks)
        assert not res[0][5] and not res[1][5]
    else:
        for r in res:
            assert r[4] is None
            assert np.array_equal(r[1], keys.view(np.int16)) and np.array_equal(r[2], toks)
            assert np.array_equal(r[6], toks[src, 0])
        assert res[0][5] and not res[1][5]                          # only rank 0 generated on the host


def test_bench_starts_its_own_ranks():
    """`python bench.py --gpus 2 ...` started plainly launches two ranks and prints ONE JSON line
    that says n_gpus 2 (shown with the CPU arm, which needs no device: rank 0 times the oracle,
    the other rank exits without work)."""
    import json
    import subprocess
    import sys
    import bench
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    cmd = bench.relaunch_command(["--gpus", "2", "--steps", "1"], 2, 29999)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=2" in cmd and "127.0.0.1" in cmd
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--rows", "20000", "--steps", "1", "--warmup", "0"], capture_output=True, text=True,
                       env=env, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["n_gpus"] == 2 and j["config"]["N"] == 20000
