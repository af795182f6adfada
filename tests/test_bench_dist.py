"""Multi-rank plumbing of bench.py on CPU: two gloo ranks, barrier + max-over-ranks timing,
whole-job aggregation; and the reference arm under torchrun (rank 0 alone prints)."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def torchrun(script_args, nproc=2, timeout=600):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(nproc),
           "--master-addr", "127.0.0.1", "--master-port", str(free_port())] + script_args
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="1")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def json_lines(text):
    return [json.loads(l) for l in text.splitlines() if l.startswith("{")]


def test_two_rank_timing_is_max_over_ranks_and_value_is_whole_job():
    r = torchrun([os.path.join("tests", "dist_worker.py"), "--gpus", "2", "--steps", "4"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = json_lines(r.stdout)
    assert len(lines) == 1                                  # rank 0 alone prints
    out = lines[0]
    assert out["world"] == 2 and out["ms"] == 15.0          # slowest rank
    assert abs(out["value"] - 16 * 2 / (15e-3 / 32)) < 1e-6  # both replicas' tokens over that time


def test_reference_arm_under_torchrun_prints_once():
    r = torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "1",
                  "--context", "4096"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = json_lines(r.stdout)
    assert len(lines) == 1 and lines[0]["impl"] == "reference"
    assert lines[0]["cpu_baseline"]["kind"] == "oracle" and lines[0]["e2e"]["h2d_bytes_per_step"] == 0
    assert lines[0]["value"] > 0


def test_gather_grouping_follows_the_measured_regimes():
    """Layers per gather launch as a function of the link / compute ratio of a layer, the layer count and the layer's
    compute time: the five configurations' operating points and the edges of the rule."""
    sys.path.insert(0, ROOT)
    import bench
    pick = bench.pick_transfer_group
    assert pick(3.0, 32, 41.0) == 8          # configs[1] at fetch ratio 0.05: strongly link-bound, many layers
    assert pick(2.4, 8, 51.0) == 4           # configs[3]: half of its 8 layers
    assert pick(1.3, 4, 196.0) == 1          # configs[2]: mildly link-bound, 4 layers: one launch per layer
    assert pick(3.0, 4, 60.0) == 1           # few layers never share one launch, however link-bound
    assert pick(0.85, 32, 44.0) == 2         # configs[1] at fetch ratio 0.02: near the break-even
    assert pick(0.43, 32, 44.0) == 1         # far below it
    assert pick(0.8, 32, 10.0) == 1          # configs[0]: layers too short to wait for a second plan
    for r in (0.0, 0.4, 0.6, 1.0, 1.5, 2.5, 10.0):
        for layers in (1, 2, 4, 8, 32, 64):
            g = pick(r, layers, 50.0)
            assert 1 <= g <= max(1, min(8, layers))


def test_graph_upload_is_skipped_without_a_graph_handle():
    """DecodeEngine.upload is an optimisation of the first replay: where the graph object has no handle to give (or
    the driver library is not there) it reports False and does nothing."""
    from paper_2608_08097_b200 import pipeline

    class NoHandle:
        pass

    class Engine:
        main = None

    assert pipeline.DecodeEngine.upload(Engine(), NoHandle()) is False
