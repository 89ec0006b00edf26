"""The N > 1 path of bench.py has no data-path collective (replicas only); what
it does across ranks is a barrier, a MAX over the ranks' times and a SUM over
their work units.  Checked here with two gloo ranks on CPU."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch.distributed as dist
    import bench
    dist.init_process_group(backend="gloo")
    rank = dist.get_rank()
    bench.barrier()
    # rank r took (10 + 5 r) ms for 64*(r+1) images
    t, u = bench.aggregate(10.0 + 5.0 * rank, 64.0 * (rank + 1))
    print(json.dumps({"rank": rank, "t": t, "u": u}))
    bench.barrier()
    dist.destroy_process_group()
""") % ROOT


def test_aggregate_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
    import json
    for o, _ in outs:
        rec = json.loads(o.strip().splitlines()[-1])
        assert rec["t"] == 15.0          # slowest rank
        assert rec["u"] == 192.0         # 64 + 128 images


def test_single_process_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(3.5, 64) == (3.5, 64.0)


def test_reference_arm_runs_on_cpu_and_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "3", "--warmup", "3"], capture_output=True, text=True,
                         timeout=600, env=dict(os.environ, CUDA_VISIBLE_DEVICES=""))
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
