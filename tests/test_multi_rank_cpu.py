"""The N > 1 path of bench.py on CPU: two gloo ranks, each an independent
replica with its own batch (the path shards by request, no data-path
collective); only the timing / token aggregation crosses ranks."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_two_rank_aggregation_and_per_rank_batches(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import numpy as np, torch, torch.distributed as dist
        import bench
        from dscale_inputs import CONFIGS, make_requests, small_variant
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        cfg = bench.replica_config(CONFIGS["tiny"], rank)
        req = make_requests(cfg)
        # every replica draws its own batch
        sig = torch.tensor([float(req["ctx_len"].sum())], dtype=torch.float64)
        sigs = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sigs, sig)
        assert len({{float(s) for s in sigs}}) == world
        # aggregation: max of times, sum of tokens
        t = torch.tensor([1.0 + rank, 2.0 - rank, 3.0, 10.0 + rank, 20.0], dtype=torch.float64)
        ms_step, attn_ms, e2e_s, tokens, e2e_tokens = bench.aggregate(dist, t)
        assert ms_step == float(world) and attn_ms == 2.0 and e2e_s == 3.0
        assert tokens == sum(10.0 + r for r in range(world)) and e2e_tokens == 20.0 * world
        if rank == 0:
            print("OK", tokens / ms_step)
        dist.destroy_process_group()
    """))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533")
    res = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                          "--nproc-per-node=2", "--master-addr", "127.0.0.1", "--master-port",
                          "29533", str(script)], capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "OK" in res.stdout


def test_reference_arm_runs_only_on_rank_zero(tmp_path):
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--gpus", "2", "--steps", "1", "--warmup", "0"], capture_output=True,
                         text=True, env=env, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""
