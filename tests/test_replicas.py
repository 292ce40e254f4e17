"""The multi-GPU path is N independent replicas; its host logic runs here as two gloo ranks on CPU."""
import json
import os
import socket
import subprocess
import sys

from paper_2507_23777_b200 import replicas

HERE = os.path.dirname(os.path.abspath(__file__))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(script_args, nproc=2, timeout=300):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + script_args
    env = dict(os.environ, OMP_NUM_THREADS="1")
    return subprocess.run(cmd, capture_output=True, text=True, timeout=timeout, env=env, cwd=os.path.dirname(HERE))


def test_single_process_is_identity():
    job = replicas.reduce_totals(50, 2, 4.0, 5.0)
    assert (job.world, job.tokens, job.meshes, job.ms, job.ms_e2e) == (1, 50, 2, 4.0, 5.0)
    assert abs(job.tokens_per_s_per_mesh() - 50 / 4e-3 / 2) < 1e-9
    assert replicas.replica_seed(7, 0, 1) == 7 and replicas.replica_seed(7, 3, 1) == 7


def test_two_replicas_sum_tokens_take_slowest_rank_and_decode_different_meshes():
    r = _torchrun([os.path.join(HERE, "replica_worker.py")])
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads([ln for ln in r.stdout.splitlines() if ln.startswith("{")][-1])
    assert line["world"] == 2 and line["tokens"] == 201 and line["meshes"] == 2
    assert line["ms"] == 20.0 and line["ms_e2e"] == 40.0
    # 201 tokens in 20 ms, one mesh at a time per replica
    assert abs(line["value"] - 201 / 20e-3) < 1e-6
    (s0, d0), (s1, d1) = line["ranks"]
    assert s0 != s1 and d0 != d1


def test_reference_arm_runs_on_rank_zero_only():
    """Under a two-rank launch the oracle arm of bench.py prints one line, from rank 0; rank 1 exits 0 idle."""
    r = _torchrun([os.path.join(os.path.dirname(HERE), "bench.py"), "--impl", "reference", "--gpus", "2", "--config", "0",
                   "--steps", "1", "--warmup", "0", "--reference-seconds", "2"], timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(ln) for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    ln = lines[0]
    assert ln["impl"] == "reference" and ln["n_gpus"] == 2 and ln["value"] > 0 and ln["cpu_baseline"]["kind"] == "oracle"
    assert ln["e2e"]["h2d_bytes_per_step"] == 0 and ln["e2e"]["value"] == ln["value"]
