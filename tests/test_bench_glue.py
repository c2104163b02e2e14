"""Host-side pieces of bench.py that need no GPU: the algorithmic-byte model of the roofline, the
max-over-ranks reduction used when N replicas run under torchrun (two gloo ranks on the CPU), the
clock-sample parser, and the reference arm's JSON contract."""
import json
import os
import subprocess
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2511_11373_b200 import workloads as wl  # noqa: E402


def test_algorithmic_bytes_match_the_hand_count():
    m = wl.MODEL_FULL
    b = bench.algorithmic_bytes(m, kv_tokens=557_000, active_per_layer=[126] * 48)
    w_attn = (2048 * 5120 + 4096 * 2048) * 2
    assert b["attn_router"] == 48 * (w_attn + 128 * 2048 * 2)
    assert b["experts"] == 48 * 126 * 3 * 2048 * 768 * 2
    assert b["kv"] == 557_000 * 2048 * 48            # 2 KB per cached token per layer
    assert b["lm_head"] == 151936 * 2048 * 2
    assert b["total"] == b["attn_router"] + b["experts"] + b["kv"] + b["lm_head"]
    assert 113e9 < b["total"] < 116e9                # the 114 GB step of the 48-layer model


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    dist.init_process_group("gloo", rank=rank, world_size=world)
    v = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
    bench.barrier(world)
    out.put((rank, v))
    dist.destroy_process_group()


def test_max_over_ranks_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    ps = [ctx.Process(target=_rank, args=(r, 2, 29511, q)) for r in range(2)]
    for p in ps:
        p.start()
    got = sorted(q.get(timeout=120) for _ in ps)
    for p in ps:
        p.join(60)
    assert got == [(0, 15.0), (1, 15.0)]
    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5


def test_reference_arm_prints_the_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "2",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-500:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "tokens/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["gpu_launches"] == 0 and line["vs_baseline"] is None
