"""The N > 1 path of bench.py (independent replicas, no data-path collective) on CPU: two gloo ranks."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 0: 10 ms for 30 tokens; rank 1: 14 ms for 50 tokens
    dev_ms, wall, tokens, nbytes = bench.aggregate_replicas(10.0 + 4 * rank, 0.011 + 0.004 * rank, 30 + 20 * rank,
                                                            1e9 * (1 + rank), world, "cpu")
    out[rank] = (dev_ms, wall, tokens, nbytes)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_max_time_sum_tokens():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        out = m.dict()
        procs = [ctx.Process(target=_worker, args=(r, 2, 29731, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        for r in range(2):
            dev_ms, wall, tokens, nbytes = out[r]
            assert dev_ms == 14.0 and abs(wall - 0.015) < 1e-12      # slowest rank
            assert tokens == 80.0 and nbytes == 3e9                   # whole job
        # the job's value: all tokens over the slowest rank's time
        assert abs(out[0][2] / (out[0][0] / 1e3) - 80 / 0.014) < 1e-6


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_replicas(3.0, 0.004, 7, 5e8, 1, "cpu") == (3.0, 0.004, 7.0, 5e8)


def test_round_bytes_formula():
    """Algorithmic bytes of a round: gamma * (E * W_layer + W_lm) + L * W_layer + W_lm + KV terms."""
    sys.path.insert(0, ROOT)
    import bench
    import synth
    cfg = synth.CONFIGS["llama2_7b"]
    Wl, Wlm, kv = cfg.layer_bytes(), cfg.lm_head_bytes(), cfg.kv_bytes_per_pos_layer()
    assert abs(Wl / 1e6 - 404.8) < 0.1 and abs(Wlm / 1e6 - 262.1) < 0.1 and kv == 16384
    E, g, T = 9, 6, 640
    want = g * (E * Wl + Wlm) + cfg.n_layers * Wl + Wlm
    want += sum(E * kv * (T + i + 1) for i in range(g)) + cfg.n_layers * kv * (T + g + 1)
    assert bench.round_bytes(cfg, [(E, g, T)]) == want
    assert abs(want / 1e9 - 37.5) < 0.3                                # the worked figure for (9, 6)
    # vanilla step: one pass over the model
    assert abs(bench.round_bytes(cfg, [(1, 0, T)]) / 1e9 - 13.55) < 0.05


def test_reference_arm_other_ranks_exit_without_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "1"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_runs_the_named_workload():
    """The oracle arm prefills the configuration's whole prompt and prints the same `config` object as the GPU arm."""
    sys.path.insert(0, ROOT)
    import bench
    import synth
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny", "--steps", "3",
                        "--warmup", "1"], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-500:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    cfg = synth.CONFIGS["tiny"]
    assert line["impl"] == "reference" and line["config"] == bench.bench_config(cfg, 1)
    assert f"the {cfg.prompt_len}-token prompt" in line["cpu_baseline"]["sample"]
    assert line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
