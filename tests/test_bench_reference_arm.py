"""The benchmark's reference arm (the oracle on the host cores) and its multi-rank launch, on CPU.

There is no exchange step in this path (replicas only), so the N > 1 launch has one rule to keep: rank 0
alone runs and prints the reference line, the other ranks exit 0 without work."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _line(out):
    lines = [l for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out
    return json.loads(lines[0])


def test_reference_arm_single_process():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "single",
                          "--steps", "1", "--warmup", "1"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    line = _line(out.stdout)
    assert line["impl"] == "reference" and line["unit"] == "us/image" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["gpu_launches"] == 0
    assert line["extrapolated"] is True and line["measured_s"] > 0


def test_input_generators_import_without_the_cuda_library():
    """The reference arm and the oracle's own tests use the seeded input generators; importing them must not
    load the product's shared library (the binding is loaded on first use only)."""
    code = ("import sys; from paper_2511_16047_b200 import synth; import paper_2511_16047_b200 as P; "
            "assert 'paper_2511_16047_b200.binding' not in sys.modules; "
            "assert not any('libamskv.so' in l for l in open('/proc/self/maps')); "
            "P.binding; assert 'paper_2511_16047_b200.binding' in sys.modules")
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr


def test_reference_arm_two_ranks_print_one_line():
    env = dict(os.environ, OMP_NUM_THREADS="2")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
                          "--master-addr", "127.0.0.1", "--master-port", "29541", os.path.join(ROOT, "bench.py"),
                          "--impl", "reference", "--gpus", "2", "--workload", "single", "--steps", "1", "--warmup", "1"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    line = _line(out.stdout)
    assert line["impl"] == "reference" and line["n_gpus"] == 2
