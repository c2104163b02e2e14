"""Shared test helpers: small model shapes and an oracle-side runner (CPU only)."""
import torch

import oracle
from paper_2511_11373_b200 import workloads as wl

SMALL = dict(n_layers=2, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, n_experts=4, top_k=2,
             expert_inter=32, vocab=50, qk_norm=1, rope_theta=1e4, rms_eps=1e-6)


def ocfg(model: dict) -> oracle.Config:
    return oracle.Config(**model)


def bf16_bits(t: torch.Tensor) -> torch.Tensor:
    return t.contiguous().view(torch.int16)


def fresh_cache(model, n_pages, page_size, seed=0, fill=True):
    return wl.make_kv_pools(model, n_pages, page_size, seed=seed, device="cpu", fill=fill)


def rel_l2(a: torch.Tensor, b: torch.Tensor) -> float:
    a, b = a.double(), b.double()
    return float((a - b).norm() / b.norm().clamp_min(1e-30))
