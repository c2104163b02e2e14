"""CPU oracle of the rollout step (TEST INFRASTRUCTURE -- not part of the product path).

Thin ctypes wrapper over ``mars_oracle.c`` (plain C, fp64 arithmetic).  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg may import this package; the CUDA library and
its Python binding never do, and nothing here touches the CUDA library.

All tensors are CPU ``torch`` tensors used purely as typed memory (bf16 weights and caches are
passed as raw 16-bit patterns, the residual stream and logits as fp32).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mars_oracle.c")
_LIB = os.path.join(_HERE, "libmars_oracle.so")
_lib = None

LAYER_FIELDS = ("attn_norm", "wqkv", "q_norm", "k_norm", "wo", "mlp_norm", "router", "w_gate_up", "w_down")


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP on outer loops only, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim",
                                              "n_experts", "top_k", "expert_inter", "vocab", "qk_norm")] + \
               [("rope_theta", ctypes.c_double), ("rms_eps", ctypes.c_double)]


class _Layer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in LAYER_FIELDS]


@dataclass
class Config:
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_experts: int
    top_k: int
    expert_inter: int
    vocab: int
    qk_norm: int = 0
    rope_theta: float = 1e6
    rms_eps: float = 1e-6

    def c(self) -> _Cfg:
        return _Cfg(self.n_layers, self.hidden, self.n_q_heads, self.n_kv_heads, self.head_dim, self.n_experts,
                    self.top_k, self.expert_inter, self.vocab, self.qk_norm, self.rope_theta, self.rms_eps)


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.orc_bf16_to_f32.restype = ctypes.c_float
        _lib.orc_bf16_to_f32.argtypes = [ctypes.c_uint16]
        _lib.orc_f32_to_bf16.restype = ctypes.c_uint16
        _lib.orc_f32_to_bf16.argtypes = [ctypes.c_float]
        _lib.orc_uniform.restype = ctypes.c_double
        _lib.orc_uniform.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint32]
        _lib.orc_logprob_of.restype = ctypes.c_float
        _lib.orc_logprob_of.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_int32]
        _lib.orc_rope.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_double]
        _lib.orc_rmsnorm.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_void_p]
        _lib.orc_softmax.argtypes = [ctypes.c_void_p, ctypes.c_int]
        _lib.orc_router.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                    ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _lib.orc_embed.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
        _lib.orc_lm_head.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                     ctypes.c_void_p, ctypes.c_void_p]
        _lib.orc_philox4x32_10.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _lib.orc_sample.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_int,
                                    ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                    ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        _lib.orc_layer_forward.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    return _lib


def _cpu(t: torch.Tensor, dtype) -> torch.Tensor:
    assert t.device.type == "cpu" and t.dtype == dtype and t.is_contiguous(), (t.device, t.dtype, t.is_contiguous())
    return t


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def bf16_to_f32(bits: int) -> float:
    return float(lib().orc_bf16_to_f32(bits))


def f32_to_bf16(value: float) -> int:
    return int(lib().orc_f32_to_bf16(value))


def rmsnorm(x: torch.Tensor, gain: torch.Tensor, eps: float = 1e-6) -> torch.Tensor:
    x = _cpu(x, torch.float64)
    out = torch.empty_like(x)
    lib().orc_rmsnorm(_ptr(x), _ptr(_cpu(gain, torch.bfloat16)), x.numel(), eps, _ptr(out))
    return out


def rope(u: torch.Tensor, pos: int, theta: float) -> torch.Tensor:
    out = _cpu(u, torch.float64).clone()
    lib().orc_rope(_ptr(out), out.numel(), pos, theta)
    return out


def softmax(z: torch.Tensor) -> torch.Tensor:
    out = _cpu(z, torch.float64).clone()
    lib().orc_softmax(_ptr(out), out.numel())
    return out


def router(w_router: torch.Tensor, h: torch.Tensor, k: int):
    E, H = w_router.shape
    idx = torch.empty(k, dtype=torch.int32)
    w = torch.empty(k, dtype=torch.float32)
    probs = torch.empty(E, dtype=torch.float32)
    lib().orc_router(_ptr(_cpu(w_router, torch.bfloat16)), E, H, k, _ptr(_cpu(h, torch.float64)),
                     _ptr(idx), _ptr(w), _ptr(probs))
    return idx, w, probs


def embed(table: torch.Tensor, tokens: torch.Tensor) -> torch.Tensor:
    V, H = table.shape
    tokens = _cpu(tokens, torch.int32)
    x = torch.empty(tokens.numel(), H, dtype=torch.float32)
    lib().orc_embed(_ptr(_cpu(table, torch.bfloat16)), H, tokens.numel(), _ptr(tokens), _ptr(x))
    return x


def lm_head(cfg: Config, final_norm: torch.Tensor, w_lm: torch.Tensor, x: torch.Tensor) -> torch.Tensor:
    x = _cpu(x, torch.float32)
    n = x.shape[0]
    logits = torch.empty(n, cfg.vocab, dtype=torch.float32)
    c = cfg.c()
    lib().orc_lm_head(ctypes.byref(c), _ptr(_cpu(final_norm, torch.bfloat16)), _ptr(_cpu(w_lm, torch.bfloat16)),
                      n, _ptr(x), _ptr(logits))
    return logits


def philox4x32_10(ctr, key):
    c = (ctypes.c_uint32 * 4)(*ctr)
    k = (ctypes.c_uint32 * 2)(*key)
    o = (ctypes.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, o)
    return tuple(int(v) for v in o)


def uniform(seed: int, step: int, seq_id: int) -> float:
    return float(lib().orc_uniform(seed, step, seq_id))


def sample(logits: torch.Tensor, temperature: float, top_p: float, greedy: bool, u: float, want_set: bool = False):
    """Returns dict(token, logp, nucleus_mass, cdf_lo, cdf_hi[, in_nucleus])."""
    logits = _cpu(logits, torch.float32)
    V = logits.numel()
    tok = ctypes.c_int32()
    lp = ctypes.c_float()
    mass, lo, hi = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    ins = torch.empty(V, dtype=torch.uint8) if want_set else None
    lib().orc_sample(_ptr(logits), V, temperature, top_p, int(bool(greedy)), u, ctypes.byref(tok), ctypes.byref(lp),
                     ctypes.byref(mass), _ptr(ins), ctypes.byref(lo), ctypes.byref(hi))
    out = dict(token=tok.value, logp=lp.value, nucleus_mass=mass.value, cdf_lo=lo.value, cdf_hi=hi.value)
    if want_set:
        out["in_nucleus"] = ins
    return out


def logprob_of(logits: torch.Tensor, temperature: float, token: int) -> float:
    logits = _cpu(logits, torch.float32)
    return float(lib().orc_logprob_of(_ptr(logits), logits.numel(), temperature, token))


def layer_forward(cfg: Config, layer: dict, x: torch.Tensor, seq: torch.Tensor, pos: torch.Tensor,
                  k_pool: torch.Tensor, v_pool: torch.Tensor, block_table: torch.Tensor, page_size: int,
                  forced_idx: torch.Tensor | None = None, want_attn: bool = False) -> dict:
    """One decoder layer over ``n`` new tokens; ``x`` [n, H] fp32 and the pools are updated in place.

    k_pool / v_pool: this layer's cache, bf16 [n_pages, n_kv_heads, page_size, head_dim].
    block_table: int32 [n_seqs, max_pages_per_seq]; seq / pos: int32 [n].
    """
    x = _cpu(x, torch.float32)
    n = x.shape[0]
    seq, pos = _cpu(seq, torch.int32), _cpu(pos, torch.int32)
    block_table = _cpu(block_table, torch.int32)
    assert k_pool.shape[1:] == (cfg.n_kv_heads, page_size, cfg.head_dim), k_pool.shape
    ws = _Layer(*[layer[f].data_ptr() if layer.get(f) is not None else None for f in LAYER_FIELDS])
    for f in LAYER_FIELDS:
        if layer.get(f) is not None:
            _cpu(layer[f], torch.bfloat16)
    k = cfg.top_k
    ridx = torch.empty(n, k, dtype=torch.int32)
    rw = torch.empty(n, k, dtype=torch.float32)
    rp = torch.empty(n, cfg.n_experts, dtype=torch.float32)
    ao = torch.empty(n, cfg.n_q_heads * cfg.head_dim, dtype=torch.float32) if want_attn else None
    if forced_idx is not None:
        forced_idx = _cpu(forced_idx, torch.int32)
        assert forced_idx.shape == (n, k)
    c = cfg.c()
    lib().orc_layer_forward(ctypes.byref(c), ctypes.byref(ws), n, _ptr(x), _ptr(seq), _ptr(pos),
                            _ptr(_cpu(k_pool, torch.bfloat16)), _ptr(_cpu(v_pool, torch.bfloat16)),
                            _ptr(block_table), block_table.shape[1], page_size, _ptr(forced_idx),
                            _ptr(ridx), _ptr(rw), _ptr(rp), _ptr(ao))
    out = dict(router_idx=ridx, router_w=rw, router_probs=rp)
    if want_attn:
        out["attn_out"] = ao
    return out


def forward(cfg: Config, weights: dict, tokens: torch.Tensor, seq: torch.Tensor, pos: torch.Tensor,
            k_pools, v_pools, block_table: torch.Tensor, page_size: int, forced_idx=None, want_logits=True) -> dict:
    """Whole model over ``n`` new tokens.  k_pools / v_pools: per-layer caches (sequence or a
    [L, ...] tensor), updated in place.  forced_idx: optional [L, n, k] routing override.
    Returns hidden [L+1, n, H] (residual stream before layer 0 and after every layer), the
    router's taps per layer and the logits [n, V]."""
    x = embed(weights["embed"], tokens)
    hidden = [x.clone()]
    ridx, rw, rp = [], [], []
    for l, layer in enumerate(weights["layers"]):
        out = layer_forward(cfg, layer, x, seq, pos, k_pools[l], v_pools[l], block_table, page_size,
                            None if forced_idx is None else forced_idx[l].contiguous())
        hidden.append(x.clone())
        ridx.append(out["router_idx"]); rw.append(out["router_w"]); rp.append(out["router_probs"])
    res = dict(hidden=torch.stack(hidden), router_idx=torch.stack(ridx), router_w=torch.stack(rw),
               router_probs=torch.stack(rp))
    if want_logits:
        res["logits"] = lm_head(cfg, weights["final_norm"], weights["lm_head"], x)
    return res
