"""The multi-GPU arm of bench.py runs independent replicas; the only cross-rank steps are the barrier around the
timed region and the max-over-ranks of the step time.  Those host-side steps are covered here with two gloo ranks
on CPU (the replicas themselves need one GPU each)."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent('''
    import os, sys
    sys.path.insert(0, os.environ["SPECTRA_ROOT"])
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    # each rank reports its own step time; every rank must end with the slowest one
    mine = 1.0 + 0.5 * rank
    got = bench._max_over_ranks(mine, world, device="cpu")
    assert abs(got - (1.0 + 0.5 * (world - 1))) < 1e-12, got
    # whole-job value = units of all replicas / slowest time (weak scaling, replicas only)
    per_rank_tokens = 1000
    value = world * per_rank_tokens / got
    assert abs(value - 2000 / 1.5) < 1e-9
    dist.barrier()
    dist.destroy_process_group()
    print("rank", rank, "ok")
''')


def test_max_over_ranks_and_barrier_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, SPECTRA_ROOT=ROOT, MASTER_ADDR="127.0.0.1", MASTER_PORT="29617", WORLD_SIZE="2")
    procs = []
    for rank in range(2):
        e = dict(env, RANK=str(rank), LOCAL_RANK=str(rank))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=e, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT))
    outs = [p.communicate(timeout=240)[0].decode() for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert f"rank {rank} ok" in out


def test_reference_arm_only_rank_zero_prints(tmp_path):
    """Under torchrun the reference arm runs on rank 0 alone; other ranks exit 0 without work."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0"], env=env, capture_output=True, timeout=120)
    assert out.returncode == 0 and out.stdout.decode().strip() == ""
