"""Host logic of the multi-GPU benchmark mode (independent replicas, no data-path collective):
world-size-2 gloo ranks on CPU check the max-over-ranks timing and the whole-job aggregation."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, {root!r})
    import torch.distributed as dist
    import bench
    rank, world, local = bench.dist_env()
    dist.init_process_group(backend="gloo", rank=rank, world_size=world)
    # rank r pretends its timed region took 10 + 5 r ms, its end-to-end loop 40 - 3 r ms
    ms, e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 40.0 - 3.0 * rank])
    value = bench.whole_job_tflops(2.0e12, world, ms)
    print(json.dumps({{"rank": rank, "world": world, "ms": ms, "e2e": e2e, "value": value}}), flush=True)
    dist.barrier()
    dist.destroy_process_group()
""")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_slowest_time_and_sum_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(out)
    import json
    for out in outs:
        rec = json.loads(out.strip().splitlines()[-1])
        assert rec["world"] == 2
        assert rec["ms"] == 15.0          # the slowest rank
        assert rec["e2e"] == 40.0
        # two replicas of 2 TFLOP each in 15 ms
        assert abs(rec["value"] - 2 * 2.0e12 / 15e-3 / 1e12) < 1e-9


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.5, 7.25]) == [3.5, 7.25]
    assert bench.whole_job_tflops(4.0e12, 1, 4.0) == 1000.0


def test_reference_arm_skips_nonzero_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
