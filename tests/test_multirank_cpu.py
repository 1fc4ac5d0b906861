"""World-size-2 checks of the multi-rank host logic of bench.py on CPU (gloo).

The (batch, head) units of the layer are independent, so N GPUs run N independent batches with
no collective on the data path; what ranks share is the barrier around the timed region, the
max-over-ranks of the step time and the aggregation of the throughput.  These tests run that
logic as two gloo ranks, with a stub in place of the CUDA step."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_RANK_PROGRAM = textwrap.dedent(
    """
    import json, os, sys
    sys.path.insert(0, {root!r})
    import torch, torch.distributed as dist
    import bench
    from paper_2602_02180_b200 import synth

    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    dev = torch.device("cpu")
    # every rank draws its own batch: different seeds, same shapes
    w = synth.WORKLOADS["c1"]
    wl = w.with_(seed=w.seed + 100 * rank)
    Q, _, _ = synth.make_qkv(wl, "cpu")
    digest = float(Q.double().sum())
    all_digests = [None] * world
    dist.all_gather_object(all_digests, digest)
    # the slowest rank sets the step time
    ms = bench._max_over_ranks(torch, dist, 10.0 * (rank + 1), dev)
    value = world * w.B * w.N / (ms * 1e-3)
    if rank == 0:
        print(json.dumps({{"ms": ms, "value": value, "digests": all_digests, "world": world}}))
    dist.barrier()
    dist.destroy_process_group()
    """
)


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_work(tmp_path):
    prog = tmp_path / "rank_program.py"
    prog.write_text(_RANK_PROGRAM.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    out = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr",
         "127.0.0.1", "--master-port", "29653", str(prog)],
        capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    r = json.loads(line)
    assert r["world"] == 2
    assert r["ms"] == 20.0                      # max over ranks, not rank 0's own 10 ms
    assert abs(r["value"] - 2 * 512 / 0.020) < 1e-6   # both ranks' tokens over the slowest time
    assert r["digests"][0] != r["digests"][1]   # ranks work on different batches


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""
