"""Host-side logic of bench.py for N > 1, on CPU with 2 gloo ranks (the data path itself has no
collective: ranks are independent replicas)."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(script_args, n=2, timeout=300):
    for attempt in range(2):                             # the probed port can be taken before the ranks bind it
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr",
               "127.0.0.1", "--master-port", str(_free_port())] + script_args
        r = subprocess.run(cmd, capture_output=True, text=True, timeout=timeout, cwd=ROOT)
        if r.returncode == 0:
            break
    return r


def _json_lines(out):
    return [json.loads(l) for l in out.splitlines() if l.startswith("{")]


def test_two_rank_timing_is_max_and_value_is_whole_job():
    r = _torchrun([os.path.join(ROOT, "tests", "_gloo_worker.py")])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_lines(r.stdout)
    assert len(lines) == 1
    assert lines[0]["world"] == 2 and lines[0]["slowest_ms"] == 20.0
    assert abs(lines[0]["value"] - 2 * 1000.0 / 0.020) < 1e-6


def test_reference_arm_prints_once_under_two_ranks():
    r = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup",
                   "0", "--sample-cols", "4096"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = _json_lines(r.stdout)
    assert len(lines) == 1
    l = lines[0]
    assert l["impl"] == "reference" and l["n_gpus"] == 2 and l["cpu_baseline"]["kind"] == "oracle"
    assert l["e2e"]["h2d_bytes_per_step"] == 0 and l["value"] > 0


def test_single_process_defaults():
    import bench
    assert bench.dist_env() == (0, 1, 0) or "RANK" in os.environ
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.aggregate(100.0, 50.0, 4) == 100.0 * 4 / 0.05


def test_mlp_step_bytes_and_flops_count_each_operand_once():
    """The fused MLP step's algorithmic figures: weights dominate, and the flops are five GEMMs plus the head."""
    sys.path.insert(0, ROOT)
    import bench
    by, fl = bench.mlp_step_bytes_flops((784, 1024, 1024, 10), 128)
    n_w = 784 * 1024 + 1024 * 1024
    # every big weight: two bf16 reads (forward, and W2 once more for dH1) plus the 10-byte stepped rewrite
    assert by > n_w * 12 + 1024 * 1024 * 2
    assert by < n_w * 12 + 1024 * 1024 * 2 + 6e6           # activations and the head add a few MB at most
    assert fl == 2.0 * 128 * (2 * 784 * 1024 + 3 * 1024 * 1024 + 2 * 1024 * 10)


def test_mlp_algorithmic_bytes_are_the_unavoidable_weight_traffic():
    import bench
    n_w = 784 * 1024 + 1024 + 1024 * 1024 + 1024 + 1024 * 10 + 10
    ab = bench.mlp_algorithmic_bytes((784, 1024, 1024, 10))
    assert ab == 12 * n_w + 2 * (1024 * 1024 + 1024 * 10)
    assert abs(ab / 1e6 - 24.5) < 0.1                      # the per-worker figure the roofline fraction is quoted on
    assert ab < bench.mlp_step_bytes_flops((784, 1024, 1024, 10), 128)[0]


def test_all_cores_oracle_leg_adds_up_independent_column_samples():
    """Two spawned processes, each timing the unchanged oracle on its own column sample; the record carries both
    the single-process and the all-cores figure with their core counts."""
    import bench

    class Args:
        workload, d, tau, momentum, weight_decay, mlp_unfused_step = "c4", 0, 0, None, 0.0, False
    spec = bench.workload_spec(Args)
    v, dt, n = bench.oracle_all_cores(spec, 2, 4096, n_proc=2)
    assert n == 2 and v > 0 and dt > 0
    rec = bench.cpu_baseline_record(spec, 1.0e7, 1, "2 steps x 16 workers x 4096 of 67108864 columns, 0.1 s", (v, dt, n))
    assert rec["cores"] == 2 and rec["single_core"]["cores"] == 1 and rec["kind"] == "oracle"
    assert rec["value"] == v and rec["single_core"]["value"] == 1.0e7
    Args.workload = "c2"
    assert bench.oracle_all_cores(bench.workload_spec(Args), 1, 4096) is None     # not a column-separable workload
