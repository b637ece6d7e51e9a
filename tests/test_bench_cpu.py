"""CPU-side checks of bench.py: the reference arm prints one well-formed JSON line, and under a
2-rank launch (replicas only: no data-path collective) rank 0 alone reports while the other rank
exits 0 without work."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _check_line(out):
    lines = [l for l in out.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1, out
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["config"]["workload"] == "layer7b"
    return d


def test_reference_arm_single_process():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "layer7b",
                        "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr
    _check_line(r.stdout)


def test_reference_arm_two_ranks():
    env = dict(os.environ, OMP_NUM_THREADS="2")
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                        "--master-addr", "127.0.0.1", "--master-port", "29533", os.path.join(ROOT, "bench.py"),
                        "--impl", "reference", "--gpus", "2", "--workload", "layer7b", "--steps", "2", "--warmup", "1"],
                       capture_output=True, text=True, timeout=900, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    d = _check_line(r.stdout)
    assert d["n_gpus"] == 2


def test_replica_timing_reduction_with_gloo():
    """The only cross-rank step of the benchmark is max-over-ranks of the step time: exercise it on gloo."""
    code = r'''
import os, torch, torch.distributed as dist
dist.init_process_group("gloo")
r = dist.get_rank()
t = torch.tensor([1.0 + r])
dist.barrier()
dist.all_reduce(t, op=dist.ReduceOp.MAX)
assert t.item() == float(dist.get_world_size()), t
if r == 0: print("max-ok")
dist.destroy_process_group()
'''
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                        "--master-addr", "127.0.0.1", "--master-port", "29534", "-c", code],
                       capture_output=True, text=True, timeout=300)
    if r.returncode != 0 and "-c" in r.stderr:   # older launchers cannot run -c: write a file instead
        import tempfile
        with tempfile.NamedTemporaryFile("w", suffix=".py", delete=False) as f:
            f.write(code)
        r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                            "--master-addr", "127.0.0.1", "--master-port", "29534", f.name],
                           capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and "max-ok" in r.stdout, r.stderr[-2000:]
