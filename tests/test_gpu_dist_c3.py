"""The deployed form of C3 (one replica per rank: sign locally, all-gather the
records, vote locally) through the product module, as three processes.  One GPU
is enough: every process signs and votes on cuda:0 and the records travel over
gloo.  The result of every rank must equal the fused single-process path and
the oracle."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

import helpers
from oracle import scout_oracle as orc
from paper_2608_11034_b200 import inputs

pytestmark = pytest.mark.gpu


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _workload(world):
    w = inputs.workload(5, "default", 1 / 300)          # mixed dtypes, ragged tensors
    w.R = world
    w.patches = [inputs.Patch(1, 3, 11, "xor", 1 << 2), inputs.Patch(world - 1, 7, 0, "xor", 1)]
    return w


def _rank(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK="0",
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from paper_2608_11034_b200 import binding, dist_c3, dist_util
    import helpers as h

    torch.cuda.set_device(0)
    dist_util.init("gloo")
    w = _workload(world)
    _, views = inputs.generate(w, "cuda")               # same seed everywhere: equivalent replicas
    c3 = dist_c3.DistributedC3(binding.make_tensor_table(w.specs, h.shape_tags(w)), w.chunk_bytes)
    c3.bind(views[rank])                                 # this rank holds replica `rank` only
    first = c3.check()
    again = c3.check()                                   # a second round on the same buffers
    assert first["table"].tobytes() == again["table"].tobytes()
    out.put((rank, first["outliers"], first["undecided"], first["counts"],
             first["status"].tobytes(), first["bitmap"].tobytes(), first["table"].tobytes()))
    dist_util.barrier()
    c3.close()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [3])
def test_three_ranks_agree_with_the_fused_path_and_the_oracle(world):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert all(r[1:] == res[0][1:] for r in res)        # no coordinator, same answer everywhere

    w = _workload(world)
    _, views = inputs.generate(w, "cuda")
    fused = helpers.gpu_sign_vote(w, views)
    C = len(fused["status"])
    _, outliers, undecided, counts, status, bitmap, table = res[0]
    from paper_2608_11034_b200 import binding
    table = np.frombuffer(table, dtype=binding.SIG_DTYPE).reshape(world, C)
    assert table.T.tobytes() == np.ascontiguousarray(fused["sigs"]).tobytes()
    assert outliers == fused["outliers"] and undecided == fused["undecided"] and counts == fused["counts"]
    assert status == fused["status"].tobytes()
    assert np.frombuffer(bitmap, dtype=np.uint64).tolist() == fused["bitmap"].tolist()

    host = [[v.cpu() for v in rep] for rep in views]
    osigs, chunks = helpers.oracle_sign_all(w, host)
    helpers.assert_sigs_match(table.T, osigs, helpers.chunk_abs_sums(w, host, chunks))
    want = orc.vote(osigs)
    assert outliers == want["outliers"] == helpers.expected_from_patches(w, chunks)[0] and len(outliers) == 2
    assert undecided == want["undecided"] == []


def test_bench_multi_rank_path_runs_on_one_gpu():
    """`bench.py --gpus 2` through the launcher, with both ranks on cuda:0 and gloo between them
    (a test hook of bench.py): the barrier, the max over ranks and the distributed-C3 leg run and
    rank 0 prints one JSON line.  The numbers mean nothing; the code path is what is checked."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, SCOUT_BENCH_ALL_RANKS_ON_GPU0="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.join(root, "bench.py"),
           "--gpus", "2", "--steps", "2", "--warmup", "1", "--scale", "0.002", "--no-e2e", "--no-cpu-baseline"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["verified"] and line["scaling"] == "weak"
    d = line["distributed_c3"]
    assert d["R"] == 2 and d["value"] > 0 and len(d["chunks_named"]) >= 1
