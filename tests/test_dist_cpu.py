"""World-size-2 gloo run of the multi-rank plumbing bench.py uses: independent
replica sets per rank, barrier, max-over-ranks timing, whole-job aggregation.
The data path itself has no collective (each rank votes over its own replicas),
so every rank also runs the oracle pipeline on its own shard."""
import os
import socket

import torch.multiprocessing as mp

import helpers  # noqa: F401  (puts the repository root on sys.path for the children)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from oracle import scout_oracle as orc
    from paper_2608_11034_b200 import dist_util, inputs
    import helpers as h

    assert dist_util.rank_info() == (rank, world, rank)
    dist_util.init("gloo")
    w = inputs.workload(1, "default", 1 / 16)
    w.seed = dist_util.rank_seed(w.seed, rank)
    _, views = inputs.generate(w)
    sigs, chunks = h.oracle_sign_all(w, views, nthreads=1)
    got = orc.vote(sigs)
    assert got["outliers"] == h.expected_from_patches(w, chunks)[0]
    dist_util.barrier()
    ms_local = 10.0 + 5.0 * rank                     # rank 1 is the slow one
    ms = dist_util.max_over_ranks(ms_local)
    value = dist_util.aggregate_gbs(w.R * w.bytes_per_replica, world, 4, ms)
    out.put((rank, ms, value, int(sigs["hash"][0, 0])))
    dist_util.barrier()
    dist.destroy_process_group()


def test_two_ranks_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ms0, v0, h0), (r1, ms1, v1, h1) = res
    assert (r0, r1) == (0, 1)
    assert ms0 == ms1 == 15.0                         # the max over ranks, on every rank
    assert v0 == v1
    bytes_per_rank = 3 * 4 * 65536
    assert abs(v0 - 2 * bytes_per_rank * 4 / 15e-3 / 1e9) < 1e-12
    assert h0 != h1                                   # different replica sets per rank


def _gather_worker(rank, world, port, out):
    """One replica per rank: sign locally (oracle), all-gather the records, vote
    locally; every rank must reach the same result without a coordinator."""
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import numpy as np
    import torch
    import torch.distributed as dist
    from oracle import scout_oracle as orc
    from paper_2608_11034_b200 import dist_util, inputs
    import helpers as h

    dist_util.init("gloo")
    w = inputs.workload(1, "default", 1 / 16)
    w.R = world
    w.patches = [inputs.Patch(1, 0, 777, "xor", 1 << 4)]
    _, views = inputs.generate(w)                       # same seed everywhere: equivalent replicas
    tt = h.oracle_tensor_table(w)
    chunks = orc.chunk_table(tt, w.chunk_bytes)
    mine = np.zeros((len(chunks), 1), dtype=orc.SIG_DTYPE)
    orc.sign_replica(tt, [inputs.to_numpy_bytes(v) for v in views[rank]], w.chunk_bytes, mine, 0, 1)
    local = torch.from_numpy(mine.view(np.uint8).reshape(-1).copy())
    gathered = [torch.empty_like(local) for _ in range(world)]
    dist.all_gather(gathered, local)                    # Algorithm 1 line 2
    table = torch.stack(gathered).numpy().view(orc.SIG_DTYPE).reshape(world, len(chunks))
    res = orc.vote_wide(table, world, len(chunks), 1, len(chunks))     # rank-major strides
    out.put((rank, res["outliers"], res["undecided"], res["counts"]))
    dist_util.barrier()
    dist.destroy_process_group()


def test_three_ranks_gather_and_vote_identically():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gather_worker, args=(r, 3, port, out)) for r in range(3)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1:] for r in res] == [res[0][1:]] * 3
    chunk = (777 * 4) // 65536
    assert res[0][1] == [(chunk, 1)] and res[0][2] == []


def _records_worker(rank, world, port, out):
    """The product's gather step (gloo path: records in host memory) on oracle-signed records."""
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import numpy as np
    import torch
    import torch.distributed as dist
    from oracle import scout_oracle as orc
    from paper_2608_11034_b200 import dist_c3, dist_util, inputs
    import helpers as h

    dist_util.init("gloo")
    w = inputs.workload(2, "clean", 1 / 64)
    w.R = world
    _, views = inputs.generate(w)
    tt = h.oracle_tensor_table(w)
    n_ch = len(orc.chunk_table(tt, w.chunk_bytes))
    mine = np.zeros((n_ch, 1), dtype=orc.SIG_DTYPE)
    orc.sign_replica(tt, [inputs.to_numpy_bytes(v) for v in views[rank]], w.chunk_bytes, mine, 0, 1)
    mine["hash"][0, 0] ^= rank                      # make the ranks' rows distinguishable
    local = torch.from_numpy(mine.view(np.uint8).reshape(-1).copy())
    table = dist_c3.gather_records(local).numpy().view(orc.SIG_DTYPE).reshape(world, n_ch)
    out.put((rank, [int(x) for x in table["hash"][:, 0]], table[:, 1:].tobytes() == np.tile(mine[1:, 0], (world, 1)).tobytes()))
    dist_util.barrier()
    dist.destroy_process_group()


def test_gather_records_is_rank_major_on_every_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_records_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0][1] == res[1][1] and res[0][1][0] ^ res[0][1][1] == 1     # row r is rank r's, everywhere
    assert res[0][2] and res[1][2]
