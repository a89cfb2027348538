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
