"""The benchmark's multi-GPU protocol (independent replicas; barrier, max time over ranks, aggregate
throughput) exercised with two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r)
    from paper_2609_39223_b200 import replicas
    n, rank, local = replicas.world()
    replicas.init("gloo")
    replicas.barrier()
    # rank r pretends its timed region took 10 + 5 r ms for 3 units of work
    rate, ms = replicas.aggregate_rate(3.0, 10.0 + 5.0 * rank)
    assert ms == 15.0, ms                                  # the slowest of the two ranks
    assert abs(rate - 2 * 3.0 / 15e-3) < 1e-9, rate        # both ranks' work over the slowest rank's time
    assert replicas.max_over_ranks(float(rank)) == 1.0
    replicas.barrier()
    replicas.finish()
    print("rank", rank, "ok")
""" % str(ROOT))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_max_time_and_aggregate_rate(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


SHARD_WORKER = textwrap.dedent("""
    import sys
    sys.path.insert(0, %r); sys.path.insert(0, %r)
    import numpy as np, torch
    import oracle
    from paper_2609_39223_b200 import replicas, synth
    from util import torch_to_bits
    n, rank, local = replicas.world()
    replicas.init("gloo")
    W = synth.weight_with_outliers(64, 512, seed=3)              # the same full weight on both ranks (seeded)
    W[40, 7] = 1.75                                              # the tensor maximum lives in rank 1's half
    full = oracle.qdq(oracle.FMT_NVFP4, torch_to_bits(W))
    shard = W[rank * 32:(rank + 1) * 32]
    state = torch.tensor([float(shard.float().abs().max())], dtype=torch.float32)
    replicas.allreduce_max_(state)
    assert state.item() == 1.75
    scale = np.float32(state.item()) / np.float32(2688.0)
    assert scale == np.float32(full["tensor_scale"])
    mine = oracle.qdq(oracle.FMT_NVFP4, torch_to_bits(shard), float(scale))
    for k in ("out", "codes", "scales"):
        np.testing.assert_array_equal(mine[k], full[k][rank * 32:(rank + 1) * 32])
    if rank == 0:                                                # without the exchange rank 0 would pick a different scale
        alone = oracle.qdq(oracle.FMT_NVFP4, torch_to_bits(shard))
        assert np.float32(alone["tensor_scale"]) != scale
    replicas.finish()
    print("rank", rank, "ok")
""" % (str(ROOT), str(ROOT / "tests")))


def test_row_sharded_nvfp4_weight_shares_one_tensor_scale(tmp_path):
    """A weight split by rows over two ranks: one 4-byte MAX all-reduce of the shard maxima gives every rank the
    tensor scale of the whole weight, and each shard then quantizes to exactly its rows of the unsharded result."""
    script = tmp_path / "shard_worker.py"
    script.write_text(SHARD_WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_single_process_is_the_identity():
    from paper_2609_39223_b200 import replicas
    assert replicas.world()[0] >= 1
    rate, ms = replicas.aggregate_rate(4.0, 2.0)
    assert ms == 2.0 and rate == 4.0 / 2e-3


def test_reference_arm_other_ranks_exit_quietly():
    env = dict(os.environ, WORLD_SIZE="2", RANK="1", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
