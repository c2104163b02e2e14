"""Pins for the CPU oracle: closed forms, invariants, special cases that reduce to library
routines, brute force on tiny inputs.  None of these tests touches the CUDA library."""
import math
import os

import pytest
import torch

import oracle
from paper_2511_11373_b200 import workloads as wl
from helpers import SMALL, bf16_bits, fresh_cache, ocfg

torch.manual_seed(0)


def run_layer(model, layer, x, seq, pos, kp, vp, bt, ps, **kw):
    x = x.clone()
    out = oracle.layer_forward(ocfg(model), layer, x, torch.tensor(seq, dtype=torch.int32),
                               torch.tensor(pos, dtype=torch.int32), kp, vp, bt, ps, **kw)
    out["x"] = x
    return out


# ------------------------------------------------------------------ bf16 rounding = library cast
def test_bf16_rounding_matches_library_cast():
    vals = torch.randn(20000, dtype=torch.float32) * torch.logspace(-20, 20, 20000)
    # exact ties between two bf16 neighbours, both parities
    ties = torch.tensor([1.00390625, 1.01171875, -1.00390625, 3.0e38, 1e-40, 0.0, -0.0], dtype=torch.float32)
    vals = torch.cat([vals, ties])
    want = bf16_bits(vals.to(torch.bfloat16))
    for v, w in zip(vals.tolist(), want.tolist()):
        assert oracle.f32_to_bf16(v) == (w & 0xFFFF), v
    for b in (0x3F80, 0xBF80, 0x0001, 0x7F7F, 0x4049):
        t = torch.tensor([b - 65536 if b >= 32768 else b], dtype=torch.int16).view(torch.bfloat16).float().item()
        assert oracle.bf16_to_f32(b) == t


# ------------------------------------------------------------------ I-1 softmax, I-16 greedy log-prob
def test_softmax_sums_to_one_and_matches_library():
    z = torch.randn(333, dtype=torch.float64) * 5
    p = oracle.softmax(z)
    assert (p >= 0).all() and abs(p.sum().item() - 1) < 1e-14
    assert torch.allclose(p, torch.softmax(z, 0), rtol=1e-13, atol=0)
    big = torch.tensor([1e4, 1e4 - 1, -1e4], dtype=torch.float64)      # must not overflow
    assert torch.allclose(oracle.softmax(big), torch.softmax(big, 0), rtol=1e-13)


def test_logprobs_exponentiate_to_one_and_greedy_closed_form():
    V = 97
    logits = (torch.randn(V) * 3).float()
    for T in (1.0, 0.6, 0.85):
        tot = sum(math.exp(oracle.logprob_of(logits, T, v)) for v in range(V))
        assert abs(tot - 1) < 1e-5
    # the temperature divides the logits (R-10): library log-softmax of logits / T, entry by entry.
    # A function that ignored T, or multiplied by it, still sums to one above but fails here.
    for T in (0.6, 0.85, 1.0, 1.7):
        want = torch.log_softmax(logits.double() / T, 0)
        for v in (0, 1, 17, 50, V - 1, int(torch.argmax(logits)), int(torch.argmin(logits))):
            assert abs(oracle.logprob_of(logits, T, v) - want[v].item()) < 2e-6, (T, v)
    sharp, flat = oracle.logprob_of(logits, 0.6, int(torch.argmax(logits))), oracle.logprob_of(logits, 1.7, int(torch.argmax(logits)))
    assert sharp > flat                                                  # a lower temperature sharpens the mode
    g = oracle.sample(logits, 0.7, 0.9, True, 0.3)
    assert g["token"] == int(torch.argmax(logits))
    lse = torch.logsumexp(logits.double(), 0).item()
    assert abs(g["logp"] - (logits.max().item() - lse)) < 1e-6           # I-16: max - lse, temperature 1
    tie = torch.tensor([0.5, 2.0, 2.0, 1.0])
    assert oracle.sample(tie, 1.0, 1.0, True, 0.5)["token"] == 1         # lowest id on ties


# ------------------------------------------------------------------ I-7 RMSNorm
def test_rmsnorm_unit_rms_scale_invariance_and_gain():
    n = 128
    x = torch.randn(n, dtype=torch.float64) * 7
    ones = torch.ones(n, dtype=torch.bfloat16)
    y = oracle.rmsnorm(x, ones, 1e-6)
    assert abs(y.pow(2).mean().sqrt().item() - 1) < 1e-6
    assert torch.allclose(oracle.rmsnorm(3.7 * x, ones, 0.0), oracle.rmsnorm(x, ones, 0.0), rtol=1e-13)
    g = (1 + 0.1 * torch.randn(n)).to(torch.bfloat16)
    ref = torch.nn.functional.rms_norm(x, (n,), g.double(), 1e-6)          # library routine
    assert torch.allclose(oracle.rmsnorm(x, g, 1e-6), ref, rtol=1e-12)
    # eps sits inside the square root: an all-zero input maps to zero, a tiny input is damped
    tiny = torch.full((n,), 1e-4, dtype=torch.float64)
    assert torch.allclose(oracle.rmsnorm(tiny, ones, 1e-6), tiny / math.sqrt(1e-8 + 1e-6), rtol=1e-12)


# ------------------------------------------------------------------ I-4 RoPE
def test_rope_closed_forms():
    d, theta = 64, 1e6
    q, k = torch.randn(d, dtype=torch.float64), torch.randn(d, dtype=torch.float64)
    assert torch.equal(oracle.rope(q, 0, theta), q)                       # position 0 is the identity
    for p in (1, 17, 4095, 65535, 300000):
        assert abs(oracle.rope(q, p, theta).norm().item() - q.norm().item()) < 1e-12
    # the score depends on the offset only
    a = torch.dot(oracle.rope(q, 1000, theta), oracle.rope(k, 1007, theta))
    b = torch.dot(oracle.rope(q, 52000, theta), oracle.rope(k, 52007, theta))
    assert abs(a.item() - b.item()) < 1e-8
    # same rotation written with complex numbers: pairs (i, i + d/2), angle pos * theta^(-2i/d)
    p = 12345
    i = torch.arange(d // 2, dtype=torch.float64)
    rot = torch.polar(torch.ones(d // 2, dtype=torch.float64), p * theta ** (-2 * i / d))
    z = torch.complex(q[: d // 2], q[d // 2:]) * rot
    assert torch.allclose(oracle.rope(q, p, theta), torch.cat([z.real, z.imag]), rtol=1e-11, atol=1e-12)
    # first pair rotates at exactly `pos` radians, so pi/2 swaps it with a sign
    e = torch.zeros(4, dtype=torch.float64); e[0] = 1.0
    r = oracle.rope(e, 1, 1e4)
    assert abs(r[0].item() - math.cos(1.0)) < 1e-15 and abs(r[2].item() - math.sin(1.0)) < 1e-15


# ------------------------------------------------------------------ I-2 router
def test_router_weights_sum_to_one_topk_order_and_full_k():
    E, H, k = 16, 64, 4
    W = (torch.randn(E, H) * 0.3).to(torch.bfloat16)
    h = torch.randn(H, dtype=torch.float64)
    idx, w, probs = oracle.router(W, h, k)
    assert abs(w.double().sum().item() - 1) < 1e-6 and abs(probs.double().sum().item() - 1) < 1e-6
    ref = torch.softmax((W.double() @ h).float().double(), 0)
    assert torch.allclose(probs.double(), ref, rtol=1e-6)
    top = torch.topk(ref, k).indices.tolist()
    assert idx.tolist() == top                                            # larger first
    assert torch.allclose(w.double(), ref[top] / ref[top].sum(), rtol=1e-6)
    idx_all, w_all, probs_all = oracle.router(W, h, E)                    # k = E  =>  w = pi
    assert torch.allclose(w_all, probs_all[idx_all.long()], rtol=1e-6)
    # exact ties: identical router rows -> lower index first
    Wt = W.clone(); Wt[5] = Wt[2]; Wt[9] = Wt[2]
    idx_t, _, p_t = oracle.router(Wt, h, E)
    order = idx_t.tolist()
    assert order.index(2) < order.index(5) < order.index(9)
    assert p_t[2] == p_t[5] == p_t[9]


# ------------------------------------------------------------------ helpers for layer-level pins
def setup_small(model=SMALL, gains="perturbed", seed=1, n_pages=24, ps=4):
    w = wl.make_weights(model, seed=seed, device="cpu", gains=gains)
    kp, vp = fresh_cache(model, n_pages, ps, seed=seed)
    return w, kp, vp


# ------------------------------------------------------------------ I-3 attention over one token = its V row
def test_single_token_attention_returns_its_value_row():
    m = dict(SMALL, n_layers=1)
    w, kp, vp = setup_small(m)
    bt = torch.tensor([[7, 0, 0]], dtype=torch.int32)
    x = torch.randn(1, m["hidden"])
    out = run_layer(m, w["layers"][0], x, [0], [0], kp[0], vp[0], bt, 4, want_attn=True)
    d, g = m["head_dim"], m["n_q_heads"] // m["n_kv_heads"]
    for j in range(m["n_q_heads"]):
        assert torch.equal(out["attn_out"][0, j * d:(j + 1) * d], vp[0][7, j // g, 0].float())


# ------------------------------------------------------------------ I-11 / I-6: a dense layer against library ops
def torch_dense_layer(m, L, x, pos, K_hist, V_hist):
    """Pre-norm decoder layer written with torch fp64 library ops for ONE token; K_hist / V_hist are
    [n_kv, t, d] histories (already in the cache).  Score matrix is materialised (brute force)."""
    F = torch.nn.functional
    H, nq, nkv, d = m["hidden"], m["n_q_heads"], m["n_kv_heads"], m["head_dim"]
    W = {k: v.double() for k, v in L.items()}
    h = F.rms_norm(x, (H,), W["attn_norm"], m["rms_eps"])
    qkv = W["wqkv"] @ h
    q, k, v = qkv[: nq * d].view(nq, d), qkv[nq * d:(nq + nkv) * d].view(nkv, d), qkv[(nq + nkv) * d:].view(nkv, d)
    if m["qk_norm"]:
        q = F.rms_norm(q, (d,), W["q_norm"], m["rms_eps"])
        k = F.rms_norm(k, (d,), W["k_norm"], m["rms_eps"])
    i = torch.arange(d // 2, dtype=torch.float64)
    rot = torch.polar(torch.ones(d // 2, dtype=torch.float64), pos * m["rope_theta"] ** (-2 * i / d))
    def rope(u):
        z = torch.complex(u[..., : d // 2], u[..., d // 2:]) * rot
        return torch.cat([z.real, z.imag], -1)
    q, k = rope(q), rope(k)
    k16, v16 = k.float().to(torch.bfloat16), v.float().to(torch.bfloat16)
    Kall = torch.cat([K_hist.double(), k16.double()[:, None]], 1)      # [nkv, t+1, d]
    Vall = torch.cat([V_hist.double(), v16.double()[:, None]], 1)
    g = nq // nkv
    Kq, Vq = Kall.repeat_interleave(g, 0), Vall.repeat_interleave(g, 0)  # [nq, t+1, d]
    S = torch.einsum("jd,jtd->jt", q, Kq) / math.sqrt(d)
    o = torch.einsum("jt,jtd->jd", torch.softmax(S, -1), Vq).reshape(-1)
    x1 = x + W["wo"] @ o
    h2 = F.rms_norm(x1, (H,), W["mlp_norm"], m["rms_eps"])
    pi = torch.softmax((W["router"] @ h2).float().double(), 0).float().double()
    sel = torch.topk(pi, m["top_k"]).indices
    wsel = pi[sel] / pi[sel].sum()
    I = m["expert_inter"]
    y = torch.zeros(H, dtype=torch.float64)
    for e, we in zip(sel.tolist(), wsel.tolist()):
        gu = W["w_gate_up"][e] @ h2
        y += float(torch.tensor(we).float()) * (W["w_down"][e] @ (F.silu(gu[:I]) * gu[I:]))
    return x1 + y, o, k16, v16


@pytest.mark.parametrize("model", [
    dict(SMALL, n_layers=1, n_experts=1, top_k=1, n_kv_heads=4),          # I-11: plain dense transformer layer
    dict(SMALL, n_layers=1),                                             # GQA + MoE, QK-norm on
    dict(SMALL, n_layers=1, qk_norm=0, hidden=48, expert_inter=40),      # non-square everything, QK-norm off
])
def test_layer_matches_library_ops_with_materialised_scores(model):
    m = model
    w, kp, vp = setup_small(m, seed=3)
    L = w["layers"][0]
    ps, ctx = 4, 9
    bt = torch.tensor([[5, 2, 11, 0]], dtype=torch.int32)
    x = torch.randn(1, m["hidden"])
    K_hist = torch.stack([torch.stack([kp[0][bt[0, t // ps], h, t % ps] for t in range(ctx)]) for h in range(m["n_kv_heads"])])
    V_hist = torch.stack([torch.stack([vp[0][bt[0, t // ps], h, t % ps] for t in range(ctx)]) for h in range(m["n_kv_heads"])])
    want_x, want_o, k16, v16 = torch_dense_layer(m, L, x[0].double(), ctx, K_hist, V_hist)
    out = run_layer(m, L, x, [0], [ctx], kp[0], vp[0], bt, ps, want_attn=True)
    assert torch.allclose(out["attn_out"][0].double(), want_o, rtol=1e-5, atol=1e-6)
    assert torch.allclose(out["x"][0].double(), want_x, rtol=1e-5, atol=1e-6)
    page, slot = int(bt[0, ctx // ps]), ctx % ps
    assert torch.equal(kp[0][page, :, slot], k16) and torch.equal(vp[0][page, :, slot], v16)   # cache write


# ------------------------------------------------------------------ I-5 paged = contiguous, page permutation
def test_paged_equals_contiguous_and_page_permutation_is_invisible():
    m = SMALL
    w, _, _ = setup_small(m)
    ps, n_pages = 4, 16
    ctxs = [5, 12, 7]
    kp, vp = fresh_cache(m, n_pages, ps, seed=9)
    toks = wl.make_tokens(3, m["vocab"], seed=2)
    seq = torch.arange(3, dtype=torch.int32)
    pos = torch.tensor(ctxs, dtype=torch.int32)
    bt_a = torch.tensor([[0, 1, 0, 0], [2, 3, 4, 5], [6, 7, 0, 0]], dtype=torch.int32)   # contiguous
    perm = torch.randperm(n_pages, generator=torch.Generator().manual_seed(4))
    inv = torch.argsort(perm)
    bt_b = inv[bt_a.long()].to(torch.int32)                                            # scattered
    kp_b, vp_b = kp[:, perm].contiguous(), vp[:, perm].contiguous()
    ra = oracle.forward(ocfg(m), w, toks, seq, pos, kp, vp, bt_a, ps)
    rb = oracle.forward(ocfg(m), w, toks, seq, pos, kp_b, vp_b, bt_b, ps)
    assert torch.equal(ra["logits"], rb["logits"]) and torch.equal(ra["hidden"], rb["hidden"])
    assert torch.equal(kp, kp_b[:, inv]) and torch.equal(vp, vp_b[:, inv])
    # one big page per sequence (a contiguous cache) gives the same result
    big = 16
    kp_c = torch.zeros(m["n_layers"], 3, m["n_kv_heads"], big, m["head_dim"], dtype=torch.bfloat16)
    vp_c = torch.zeros_like(kp_c)
    kp0, vp0 = fresh_cache(m, n_pages, ps, seed=9)
    for b, c in enumerate(ctxs):
        for t in range(c):
            kp_c[:, b, :, t] = kp0[:, bt_a[b, t // ps], :, t % ps]
            vp_c[:, b, :, t] = vp0[:, bt_a[b, t // ps], :, t % ps]
    rc = oracle.forward(ocfg(m), w, toks, seq, pos, kp_c, vp_c, torch.tensor([[0], [1], [2]], dtype=torch.int32), big)
    assert torch.equal(ra["logits"], rc["logits"])


# ------------------------------------------------------------------ I-9 chunked prefill = token-by-token decode
def test_prefill_chunks_equal_single_token_steps():
    m = SMALL
    w, _, _ = setup_small(m)
    ps, n = 4, 11
    toks = wl.make_tokens(n, m["vocab"], seed=5)
    bt = torch.tensor([[3, 9, 1, 6]], dtype=torch.int32)

    def run(chunks):
        kp, vp = fresh_cache(m, 12, ps, fill=False)
        at, last = 0, None
        for c in chunks:
            pos = torch.arange(at, at + c, dtype=torch.int32)
            last = oracle.forward(ocfg(m), w, toks[at:at + c].contiguous(), torch.zeros(c, dtype=torch.int32), pos,
                                  kp, vp, bt, ps)
            at += c
        return last["logits"][-1], kp, vp

    l1, k1, v1 = run([n])
    l2, k2, v2 = run([4, 5, 2])
    l3, k3, v3 = run([1] * n)
    assert torch.allclose(l1, l2, atol=1e-5) and torch.allclose(l1, l3, atol=1e-5)
    assert torch.equal(k1, k2) and torch.equal(k1, k3) and torch.equal(v1, v3)


# ------------------------------------------------------------------ I-10 batch independence and order
def test_sequence_output_is_independent_of_the_batch():
    m = SMALL
    w, _, _ = setup_small(m)
    ps = 4
    bt = torch.tensor([[0, 1, 2, 0], [3, 4, 0, 0], [5, 6, 7, 8]], dtype=torch.int32)
    ctx = torch.tensor([9, 6, 13], dtype=torch.int32)
    toks = wl.make_tokens(3, m["vocab"], seed=6)
    kp, vp = fresh_cache(m, 12, ps, seed=2)
    full = oracle.forward(ocfg(m), w, toks, torch.arange(3, dtype=torch.int32), ctx, kp, vp, bt, ps)
    kp, vp = fresh_cache(m, 12, ps, seed=2)
    order = [2, 0, 1]
    shuf = oracle.forward(ocfg(m), w, toks[order].contiguous(), torch.tensor(order, dtype=torch.int32),
                          ctx[order].contiguous(), kp, vp, bt, ps)
    assert torch.equal(full["logits"][order], shuf["logits"])
    kp, vp = fresh_cache(m, 12, ps, seed=2)
    alone = oracle.forward(ocfg(m), w, toks[1:2].contiguous(), torch.tensor([1], dtype=torch.int32),
                           ctx[1:2].contiguous(), kp, vp, bt, ps)
    assert torch.equal(full["logits"][1], alone["logits"][0])


# ------------------------------------------------------------------ I-8 identical experts = one dense MLP
def test_identical_experts_reduce_to_a_dense_mlp():
    m = dict(SMALL, n_layers=1)
    w, kp, vp = setup_small(m)
    L = dict(w["layers"][0])
    L["w_gate_up"] = L["w_gate_up"][:1].repeat(m["n_experts"], 1, 1).contiguous()
    L["w_down"] = L["w_down"][:1].repeat(m["n_experts"], 1, 1).contiguous()
    bt = torch.tensor([[2, 5, 0]], dtype=torch.int32)
    x = torch.randn(1, m["hidden"])
    moe = run_layer(m, L, x, [0], [6], kp[0].clone(), vp[0].clone(), bt, 4)
    m1 = dict(m, n_experts=1, top_k=1)
    L1 = dict(L, w_gate_up=L["w_gate_up"][:1].contiguous(), w_down=L["w_down"][:1].contiguous(),
              router=L["router"][:1].contiguous())
    dense = run_layer(m1, L1, x, [0], [6], kp[0].clone(), vp[0].clone(), bt, 4)
    assert torch.allclose(moe["x"], dense["x"], rtol=1e-6, atol=1e-7)
    # forced routing changes nothing either
    forced = run_layer(m, L, x, [0], [6], kp[0].clone(), vp[0].clone(), bt, 4,
                       forced_idx=torch.tensor([[3, 1]], dtype=torch.int32))
    assert torch.allclose(moe["x"], forced["x"], rtol=1e-6, atol=1e-7)


def test_forced_routing_uses_renormalised_probabilities():
    m = dict(SMALL, n_layers=1)
    w, kp, vp = setup_small(m)
    L = w["layers"][0]
    bt = torch.tensor([[2, 5, 0]], dtype=torch.int32)
    x = torch.randn(1, m["hidden"])
    free = run_layer(m, L, x, [0], [6], kp[0].clone(), vp[0].clone(), bt, 4)
    same = run_layer(m, L, x, [0], [6], kp[0].clone(), vp[0].clone(), bt, 4, forced_idx=free["router_idx"])
    assert torch.equal(free["x"], same["x"]) and torch.equal(free["router_w"], same["router_w"])
    other = [e for e in range(m["n_experts"]) if e not in free["router_idx"][0].tolist()][:2]
    forced = run_layer(m, L, x, [0], [6], kp[0].clone(), vp[0].clone(), bt, 4,
                       forced_idx=torch.tensor([other], dtype=torch.int32))
    p = forced["router_probs"][0, other].double()
    assert torch.allclose(forced["router_w"][0].double(), p / p.sum(), rtol=1e-6)
    assert not torch.equal(forced["x"], free["x"])


# ------------------------------------------------------------------ I-12 GQA = MHA with replicated KV heads
def test_gqa_equals_mha_with_replicated_kv_heads():
    m = dict(SMALL, n_layers=1)
    nq, nkv, d = m["n_q_heads"], m["n_kv_heads"], m["head_dim"]
    g = nq // nkv
    w, kp, vp = setup_small(m)
    L = w["layers"][0]
    bt = torch.tensor([[1, 4, 6]], dtype=torch.int32)
    x = torch.randn(1, m["hidden"])
    a = run_layer(m, L, x, [0], [10], kp[0].clone(), vp[0].clone(), bt, 4)
    Wq, Wk, Wv = L["wqkv"][: nq * d], L["wqkv"][nq * d:(nq + nkv) * d], L["wqkv"][(nq + nkv) * d:]
    rep = lambda W: W.view(nkv, d, -1).repeat_interleave(g, 0).reshape(nq * d, -1)
    L2 = dict(L, wqkv=torch.cat([Wq, rep(Wk), rep(Wv)]).contiguous())
    m2 = dict(m, n_kv_heads=nq)
    kp2, vp2 = kp[0].repeat_interleave(g, 1).contiguous(), vp[0].repeat_interleave(g, 1).contiguous()
    b = run_layer(m2, L2, x, [0], [10], kp2, vp2, bt, 4)
    assert torch.equal(a["x"], b["x"])


# ------------------------------------------------------------------ I-13 zeroed projections
def test_zero_down_and_zero_out_projection():
    m = dict(SMALL, n_layers=1)
    w, kp, vp = setup_small(m)
    L = dict(w["layers"][0])
    bt = torch.tensor([[1, 4, 6]], dtype=torch.int32)
    x = torch.randn(2, m["hidden"])
    L["w_down"] = torch.zeros_like(L["w_down"])
    a = run_layer(m, L, x, [0, 0], [8, 9], kp[0].clone(), vp[0].clone(), bt, 4, want_attn=True)
    want = x.double() + a["attn_out"].double() @ L["wo"].double().T
    assert torch.allclose(a["x"].double(), want, rtol=1e-5, atol=1e-6)
    L["wo"] = torch.zeros_like(L["wo"])
    b = run_layer(m, L, x, [0, 0], [8, 9], kp[0].clone(), vp[0].clone(), bt, 4)
    assert torch.equal(b["x"], x)


def test_causal_prefill_token_ignores_later_tokens():
    m = dict(SMALL, n_layers=1)
    w, _, _ = setup_small(m)
    L = w["layers"][0]
    bt = torch.tensor([[1, 4, 6]], dtype=torch.int32)
    x = torch.randn(5, m["hidden"])
    kp, vp = fresh_cache(m, 8, 4, fill=False)
    full = run_layer(m, L, x, [0] * 5, list(range(5)), kp[0], vp[0], bt, 4)
    kp, vp = fresh_cache(m, 8, 4, fill=False)
    part = run_layer(m, L, x[:3].contiguous(), [0] * 3, list(range(3)), kp[0], vp[0], bt, 4)
    assert torch.equal(full["x"][:3], part["x"])


# ------------------------------------------------------------------ embedding and lm_head against library ops
def test_embed_and_lm_head_match_library_matmul():
    m = SMALL
    w = wl.make_weights(m, seed=2, gains="perturbed")
    toks = torch.tensor([3, 49, 0, 3], dtype=torch.int32)
    x = oracle.embed(w["embed"], toks)
    assert torch.equal(x, w["embed"][toks.long()].float())
    x = torch.randn(3, m["hidden"])
    logits = oracle.lm_head(ocfg(m), w["final_norm"], w["lm_head"], x)
    h = torch.nn.functional.rms_norm(x.double(), (m["hidden"],), w["final_norm"].double(), m["rms_eps"])
    assert torch.allclose(logits.double(), h @ w["lm_head"].double().T, rtol=1e-5, atol=1e-6)


# ------------------------------------------------------------------ I-15 Philox
def _philox_py(ctr, key):
    """Independent big-integer restatement of Philox4x32-10 (Salmon et al., SC'11)."""
    c, k = list(ctr), list(key)
    for _ in range(10):
        p0, p1 = 0xD2511F53 * c[0], 0xCD9E8D57 * c[2]
        c = [((p1 >> 32) ^ c[1] ^ k[0]) & 0xFFFFFFFF, p1 & 0xFFFFFFFF,
             ((p0 >> 32) ^ c[3] ^ k[1]) & 0xFFFFFFFF, p0 & 0xFFFFFFFF]
        k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
    return tuple(c)


def test_philox_known_answers_and_independent_restatement():
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        assert oracle.philox4x32_10(v[:4], v[4:6]) == tuple(v[6:])
        assert _philox_py(v[:4], v[4:6]) == tuple(v[6:])
    g = torch.Generator().manual_seed(1)
    words = torch.randint(0, 2 ** 32, (2000, 6), generator=g, dtype=torch.int64).tolist()
    for wd in words:
        assert oracle.philox4x32_10(wd[:4], wd[4:]) == _philox_py(wd[:4], wd[4:])


def test_uniform_mapping_and_uniformity():
    seed, step, sid = 0x1234567890ABCDEF, (1 << 40) + 17, 9
    x0 = _philox_py([step & 0xFFFFFFFF, step >> 32, sid, 0], [seed & 0xFFFFFFFF, seed >> 32])[0]
    assert oracle.uniform(seed, step, sid) == ((x0 >> 8) + 0.5) / 2 ** 24
    us = sorted(oracle.uniform(7, s, b) for s in range(200) for b in range(50))
    n = len(us)
    assert 0 < us[0] and us[-1] < 1
    ks = max(max((i + 1) / n - u, u - i / n) for i, u in enumerate(us))
    assert ks < 1.63 / math.sqrt(n)                                      # Kolmogorov-Smirnov, 1% level


# ------------------------------------------------------------------ I-14 nucleus sampling
def test_top_p_nucleus_invariants():
    V = 40
    logits = (torch.randn(V, generator=torch.Generator().manual_seed(3)) * 2).float()
    for T, p in ((1.0, 0.95), (0.6, 0.95), (0.85, 0.5), (1.0, 0.05)):
        pi = torch.softmax(logits.double() / T, 0)
        r = oracle.sample(logits, T, p, False, 0.37, want_set=True)
        S = r["in_nucleus"].bool()
        mass = pi[S].sum().item()
        assert abs(mass - r["nucleus_mass"]) < 1e-12 and mass >= p - 1e-12
        assert mass - pi[S].min().item() < p                              # minimal: dropping the least member falls short
        assert pi[S].min() >= pi[~S].max() if (~S).any() else True        # S is a top set
        assert S[r["token"]] and r["cdf_lo"] <= 0.37 < r["cdf_hi"]
        assert abs(r["logp"] - math.log(pi[r["token"]].item())) < 1e-6    # full-vocabulary log-prob at temperature T
    r = oracle.sample(logits, 1.0, 1.0, False, 0.5, want_set=True)        # p = 1  =>  S = vocabulary
    assert r["in_nucleus"].all()
    r = oracle.sample(logits, 1.0, 1e-9, False, 0.99)                     # p -> 0  =>  greedy
    assert r["token"] == int(torch.argmax(logits))
    # walk in ascending token id: u just below / above a boundary of the index-order CDF
    pi = torch.softmax(logits.double(), 0)
    cdf = torch.cumsum(pi, 0)
    for v in (0, 7, 25):
        assert oracle.sample(logits, 1.0, 1.0, False, cdf[v].item() - 1e-9)["token"] == v
        assert oracle.sample(logits, 1.0, 1.0, False, cdf[v].item() + 1e-9)["token"] == v + 1


def test_top_p_sampling_distribution_chi_square():
    V, T, p, n = 16, 0.8, 0.9, 40000
    logits = (torch.randn(V, generator=torch.Generator().manual_seed(5)) * 1.5).float()
    pi = torch.softmax(logits.double() / T, 0)
    S = oracle.sample(logits, T, p, False, 0.5, want_set=True)["in_nucleus"].bool()
    target = torch.where(S, pi, torch.zeros_like(pi)) / pi[S].sum()
    counts = torch.zeros(V, dtype=torch.float64)
    for s in range(n):
        counts[oracle.sample(logits, T, p, False, oracle.uniform(11, s, 3))["token"]] += 1
    assert counts[~S].sum() == 0
    exp = target[S] * n
    chi2 = ((counts[S] - exp) ** 2 / exp).sum().item()
    dof = int(S.sum()) - 1
    assert chi2 < dof + 4.5 * math.sqrt(2 * dof) + 5, (chi2, dof)
