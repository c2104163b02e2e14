"""Seeded synthetic inputs shared by the CUDA path's tests/benchmark and by the CPU oracle's tests.

This module holds NO arithmetic of the method: only model shapes, random tensors, context-length
draws and page assignments.  Every tensor is drawn from its own ``torch.Generator`` whose seed is
derived from (base seed, tensor name), so a tensor's bytes do not depend on which other tensors
were generated.  A tensor generated on a CUDA device differs from the one generated on the CPU for
the same seed; whoever needs the same bytes on both sides copies them.

Workload shapes follow the rollout settings of the paper's Section 4.1 (responses up to 64k
tokens in segments of 16k, inputs up to 32k, Solver/Verifier/Corrector stages sharing one model)
and the five evaluation configurations of this repository (see ``CONFIGS``).
"""
from __future__ import annotations

import hashlib
import math

import torch

# ------------------------------------------------------------------------------------ model shapes

MODEL_TINY = dict(n_layers=1, hidden=256, n_q_heads=4, n_kv_heads=1, head_dim=64, n_experts=8, top_k=2,
                  expert_inter=128, vocab=1024, qk_norm=0, rope_theta=1e6, rms_eps=1e-6)

# One Qwen3-30B-A3B-shaped layer.  The small vocabulary only exists so that the step has an
# lm_head to run; single-layer checks compare hidden states and routing.
MODEL_LAYER = dict(n_layers=1, hidden=2048, n_q_heads=32, n_kv_heads=4, head_dim=128, n_experts=128, top_k=8,
                   expert_inter=768, vocab=2048, qk_norm=1, rope_theta=1e6, rms_eps=1e-6)

MODEL_FULL = dict(MODEL_LAYER, n_layers=48, vocab=151936)

LAYER_SHAPES = {
    "attn_norm": lambda m: (m["hidden"],),
    "wqkv": lambda m: ((m["n_q_heads"] + 2 * m["n_kv_heads"]) * m["head_dim"], m["hidden"]),
    "q_norm": lambda m: (m["head_dim"],),
    "k_norm": lambda m: (m["head_dim"],),
    "wo": lambda m: (m["hidden"], m["n_q_heads"] * m["head_dim"]),
    "mlp_norm": lambda m: (m["hidden"],),
    "router": lambda m: (m["n_experts"], m["hidden"]),
    "w_gate_up": lambda m: (m["n_experts"], 2 * m["expert_inter"], m["hidden"]),
    "w_down": lambda m: (m["n_experts"], m["hidden"], m["expert_inter"]),
}
GAIN_NAMES = ("attn_norm", "q_norm", "k_norm", "mlp_norm", "final_norm")

CONFIGS = {
    1: dict(name="tiny-1layer-greedy", model=MODEL_TINY, page_size=16, ctx=[17, 64, 129, 200], steps=1,
            sampling=dict(greedy=1, temperature=1.0, top_p=1.0)),
    2: dict(name="qwen3-30b-a3b-1layer-decode", model=MODEL_LAYER, page_size=64, batch=64, ctx_range=(1024, 16384),
            steps=1, sampling=dict(greedy=1, temperature=1.0, top_p=1.0)),
    3: dict(name="qwen3-30b-a3b-48layer-decode-b64", model=MODEL_FULL, page_size=64, batch=64,
            ctx_range=(1024, 16384), steps=128, sampling=dict(greedy=0, temperature=1.0, top_p=0.95)),
    4: dict(name="qwen3-30b-a3b-48layer-mixed-b192+8x2048", model=MODEL_FULL, page_size=64, batch=192,
            ctx_lognormal=dict(sigma=0.6, medians=dict(solver=2896, verifier=4096, corrector=5793), clip=(512, 32768)),
            prefill=dict(requests=8, chunk=2048), steps=1, sampling=dict(greedy=0, temperature=1.0, top_p=0.95)),
    # profiling-sized stand-in for config 4: one layer, 64 decode sequences + 4 prompts of 1024 tokens
    6: dict(name="qwen3-30b-a3b-1layer-mixed-b64+4x1024", model=MODEL_LAYER, page_size=64, batch=64,
            ctx_range=(1024, 16384), prefill=dict(requests=4, chunk=1024), steps=1,
            sampling=dict(greedy=0, temperature=1.0, top_p=0.95)),
    5: dict(name="qwen3-30b-a3b-48layer-decode-b16-64k", model=MODEL_FULL, page_size=64, batch=16,
            ctx=[65536] * 16, steps=64, sampling=dict(greedy=1, temperature=1.0, top_p=1.0)),
    # grouped agentic rollouts: 8 groups of 8 responses, each group continuing one shared prompt
    # (whole pages, held once in the cache); every member has its own response so far
    7: dict(name="qwen3-30b-a3b-48layer-decode-8groups-of-8", model=MODEL_FULL, page_size=64, groups=8, members=8,
            prompt=8192, own_range=(256, 4096), steps=32, sampling=dict(greedy=0, temperature=1.0, top_p=0.95)),
    # one-layer stand-in of the same for quick checks
    8: dict(name="qwen3-30b-a3b-1layer-decode-8groups-of-8", model=MODEL_LAYER, page_size=64, groups=8, members=8,
            prompt=8192, own_range=(256, 4096), steps=8, sampling=dict(greedy=0, temperature=1.0, top_p=0.95)),
}

STAGES = ("solver", "verifier", "corrector")

# Context draw of configuration 3 (64 x U[1024, 16384], expected total 557 k tokens): the seed whose
# total is closest to the expectation among seeds 0..15, so that the timed step is a typical one.
CONFIG3_CONTEXT_SEED = 6


def tensor_seed(base_seed: int, name: str) -> int:
    h = hashlib.sha256(f"{base_seed}:{name}".encode()).digest()
    return int.from_bytes(h[:8], "little") & 0x7FFFFFFFFFFFFFFF


def _gen(device, base_seed: int, name: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(tensor_seed(base_seed, name))
    return g


def _normal_bf16(shape, mean, std, device, g) -> torch.Tensor:
    dev = torch.device(device)
    if dev.type == "cuda":
        t = torch.empty(shape, dtype=torch.bfloat16, device=dev)
        t.normal_(mean, std, generator=g)
        return t
    return torch.empty(shape, dtype=torch.float32).normal_(mean, std, generator=g).to(torch.bfloat16)


def make_weights(model: dict, seed: int = 0, device="cpu", gains: str = "ones") -> dict:
    """Random-init weights: every matrix ~ N(0, 0.02^2) in bf16; norm gains are 1 (``gains="ones"``)
    or 1 + 0.1 N(0,1) (``gains="perturbed"``, so that a dropped gain shows up in a comparison)."""
    def gain(name, n):
        if gains == "ones":
            return torch.ones(n, dtype=torch.bfloat16, device=device)
        return _normal_bf16((n,), 1.0, 0.1, device, _gen(device, seed, name))

    def mat(name, shape):
        return _normal_bf16(shape, 0.0, 0.02, device, _gen(device, seed, name))

    V, H = model["vocab"], model["hidden"]
    w = {"embed": mat("embed", (V, H)), "final_norm": gain("final_norm", H), "lm_head": mat("lm_head", (V, H)),
         "layers": []}
    for l in range(model["n_layers"]):
        layer = {}
        for f, shp in LAYER_SHAPES.items():
            shape = shp(model)
            layer[f] = gain(f"layer{l}.{f}", shape[0]) if f in GAIN_NAMES else mat(f"layer{l}.{f}", shape)
        w["layers"].append(layer)
    return w


def weights_to_cpu(weights: dict) -> dict:
    return {"embed": weights["embed"].cpu(), "final_norm": weights["final_norm"].cpu(),
            "lm_head": weights["lm_head"].cpu(),
            "layers": [{f: t.cpu() for f, t in layer.items()} for layer in weights["layers"]]}


def make_context_lengths(cfg: dict, seed: int = 0):
    """Context length of every decode sequence (tokens already cached) and its stage tag."""
    g = _gen("cpu", seed, cfg["name"] + ".ctx")
    if "ctx" in cfg:
        ctx = list(cfg["ctx"])
        return ctx, [STAGES[i % 3] for i in range(len(ctx))]
    B = cfg["batch"]
    if "ctx_range" in cfg:
        lo, hi = cfg["ctx_range"]
        ctx = torch.randint(lo, hi + 1, (B,), generator=g).tolist()
        return ctx, [STAGES[i % 3] for i in range(B)]
    spec = cfg["ctx_lognormal"]
    tags = torch.randint(0, 3, (B,), generator=g).tolist()
    z = torch.randn(B, generator=g).tolist()
    lo, hi = spec["clip"]
    ctx = []
    for t, zi in zip(tags, z):
        c = int(round(spec["medians"][STAGES[t]] * math.exp(spec["sigma"] * zi)))
        ctx.append(max(lo, min(hi, c)))
    return ctx, [STAGES[t] for t in tags]


def make_group_lengths(cfg: dict, seed: int = 0):
    """Tokens of its own response that every member of every group has cached: [groups][members]."""
    g = _gen("cpu", seed, cfg["name"] + ".own")
    lo, hi = cfg["own_range"]
    return torch.randint(lo, hi + 1, (cfg["groups"], cfg["members"]), generator=g).tolist()


def pages_needed(n_tokens: int, page_size: int) -> int:
    return (n_tokens + page_size - 1) // page_size


def make_page_assignment(token_capacity, page_size: int, n_pages: int, seed: int = 0, shuffle: bool = True):
    """Physical page ids for every sequence: sequence b gets enough pages for token_capacity[b]
    tokens, taken from a seeded permutation of the pool so that pages are scattered."""
    need = [pages_needed(c, page_size) for c in token_capacity]
    assert sum(need) <= n_pages, (sum(need), n_pages)
    if shuffle:
        perm = torch.randperm(n_pages, generator=_gen("cpu", seed, "pages")).tolist()
    else:
        perm = list(range(n_pages))
    out, at = [], 0
    for n in need:
        out.append(perm[at:at + n])
        at += n
    return out


def make_kv_pools(model: dict, n_pages: int, page_size: int, seed: int = 0, device="cpu", fill: bool = True):
    """K and V pools, bf16 [n_layers, n_pages, n_kv_heads, page_size, head_dim], filled with N(0,1)
    (standing for keys that are already normalised and rotated)."""
    shape = (model["n_layers"], n_pages, model["n_kv_heads"], page_size, model["head_dim"])
    pools = []
    for name in ("k_pool", "v_pool"):
        if not fill:
            pools.append(torch.zeros(shape, dtype=torch.bfloat16, device=device))
            continue
        if torch.device(device).type == "cuda":
            t = torch.empty(shape, dtype=torch.bfloat16, device=device)
            for l in range(shape[0]):   # layer by layer: bounded temporaries on large pools
                t[l].normal_(0.0, 1.0, generator=_gen(device, seed, f"{name}.{l}"))
        else:
            t = torch.stack([_normal_bf16(shape[1:], 0.0, 1.0, device, _gen(device, seed, f"{name}.{l}"))
                             for l in range(shape[0])])
        pools.append(t)
    return pools[0], pools[1]


def make_tokens(n: int, vocab: int, seed: int = 0, name: str = "tokens") -> torch.Tensor:
    """Token ids uniform over the vocabulary (int32, CPU)."""
    return torch.randint(0, vocab, (n,), generator=_gen("cpu", seed, name), dtype=torch.int32)


def block_table_tensor(pages, max_pages_per_seq: int) -> torch.Tensor:
    bt = torch.zeros(len(pages), max_pages_per_seq, dtype=torch.int32)
    for b, p in enumerate(pages):
        bt[b, :len(p)] = torch.tensor(p, dtype=torch.int32)
    return bt
