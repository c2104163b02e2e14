"""Parity at the full sizes of the benchmark configurations (48 layers, vocabulary 151936), in the
launch configuration that bench.py times.  Sequences are independent inside a step, so the CPU
oracle checks a SUBSET of the batch: it is streamed one layer at a time (that layer's weights and
the subset's cache pages are copied from the device tensors the generator filled), with the GPU's
routing forced as the cascade rule prescribes.
"""
import pytest
import torch

import oracle
from harness import check_cache_rows, check_permutation, compare_sampled, compare_step
from paper_2511_11373_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def full_weights():
    need = 175 << 30
    if torch.cuda.get_device_properties(0).total_memory < need:
        pytest.skip("needs a 180 GB device")
    w = wl.make_weights(wl.MODEL_FULL, seed=0, device=DEV, gains="ones")
    yield w
    del w
    torch.cuda.empty_cache()


class FullCase:
    def __init__(self, cfg, weights, steps, seed=0, page_edge=None):
        self.cfg, self.model, self.ps = cfg, cfg["model"], cfg["page_size"]
        self.weights = weights
        self.ctx, _ = wl.make_context_lengths(cfg, seed=seed)
        self.B = len(self.ctx)
        if page_edge is not None:       # this sequence's context ends one token short of a page boundary:
            b = page_edge               # the first step fills the page, the second must take a new one
            self.ctx[b] = self.ctx[b] - self.ctx[b] % self.ps + self.ps - 1
        cap = [c + steps + 1 for c in self.ctx]
        self.n_pages = sum(wl.pages_needed(c, self.ps) for c in cap) + 4
        self.max_pages = max(wl.pages_needed(c, self.ps) for c in cap) + 1
        self.pages = wl.make_page_assignment(cap, self.ps, self.n_pages, seed=seed)
        self.k_pool, self.v_pool = wl.make_kv_pools(self.model, self.n_pages, self.ps, seed=seed, device=DEV)
        self.m = binding.Model(self.model, weights, max_decode_seqs=self.B, max_pos=max(cap) + 8)
        self.kv = binding.KvCache(self.m, self.k_pool, self.v_pool, self.ps, self.B, self.max_pages)
        for b in range(self.B):
            if b == page_edge:          # only the pages its context touches: the library must find the next one itself
                self.pages[b] = self.pages[b][: wl.pages_needed(self.ctx[b] + 1, self.ps)]
            self.kv.seq_adopt(b, self.pages[b], self.ctx[b])
        self.cur = list(self.ctx)
        self.page_edge = page_edge

    def gpu_step(self, tokens, sampling, step, seed):
        L, H, k, V, n = self.model["n_layers"], self.model["hidden"], self.model["top_k"], self.model["vocab"], self.B
        out = dict(tokens=torch.empty(n, dtype=torch.int32, device=DEV), logp=torch.empty(n, device=DEV),
                   logits=torch.empty(n, V, device=DEV), hidden=torch.empty(L + 1, n, H, device=DEV),
                   router_w=torch.empty(L, n, k, device=DEV),
                   router_idx=torch.empty(L, n, k, dtype=torch.int32, device=DEV),
                   nucleus_mass=torch.empty(n, device=DEV),
                   expert_off=torch.empty(L, self.model["n_experts"] + 1, dtype=torch.int32, device=DEV),
                   slot_token=torch.empty(L, n * k, dtype=torch.int32, device=DEV))
        dbg = binding.make_debug(out["logits"], out["hidden"], out["router_w"], out["router_idx"], None,
                                 out["nucleus_mass"], out["expert_off"], out["slot_token"])
        smp = binding.make_sampling(seed=seed, step=step, **sampling)
        st = binding.mars_decode_step(self.m, self.kv, list(range(n)), tokens.to(DEV), smp, out["tokens"], out["logp"], dbg)
        assert st == 0 and self.m.poll_status() == 0
        # the permutation of the WHOLE batch is consistent with the routing taps, whose subset rows the
        # oracle checks (offsets, tokens per expert, distinct experts: integer work, bit for bit)
        whole = dict(expert_off=out["expert_off"].cpu(), slot_token=out["slot_token"].cpu(),
                     active_experts=self.m.active_experts())
        check_permutation(whole, dict(router_idx=out["router_idx"].cpu()), label="whole batch")
        if self.page_edge is not None:  # a page taken from the free list inside the step shows up in the block table
            self.pages[self.page_edge] = self.kv.block_table(self.page_edge)
        return out

    def oracle_subset(self, subset, tokens, gpu_router_idx):
        """Oracle forward of the chosen sequences at their current positions, layer by layer."""
        model, ps = self.model, self.ps
        ocfg = oracle.Config(**dict(model, n_layers=1))
        n = len(subset)
        pages = [self.pages[b][: wl.pages_needed(self.cur[b] + 1, ps)] for b in subset]
        flat = torch.tensor([p for pg in pages for p in pg], dtype=torch.long, device=DEV)
        bt = torch.zeros(n, max(len(p) for p in pages), dtype=torch.int32)
        at = 0
        for i, pg in enumerate(pages):
            bt[i, : len(pg)] = torch.arange(at, at + len(pg), dtype=torch.int32)
            at += len(pg)
        seq = torch.arange(n, dtype=torch.int32)
        pos = torch.tensor([self.cur[b] for b in subset], dtype=torch.int32)
        x = oracle.embed(self.weights["embed"][tokens[subset].long().to(DEV)].cpu().contiguous(),
                         torch.arange(n, dtype=torch.int32))
        hidden, ridx, rw, rp = [x.clone()], [], [], []
        for l in range(model["n_layers"]):
            layer = {f: t.cpu() for f, t in self.weights["layers"][l].items()}
            kp, vp = self.k_pool[l, flat].cpu(), self.v_pool[l, flat].cpu()
            forced = gpu_router_idx[l, subset].contiguous()
            o = oracle.layer_forward(ocfg, layer, x, seq, pos, kp, vp, bt, ps, forced_idx=forced)
            hidden.append(x.clone()); ridx.append(o["router_idx"]); rw.append(o["router_w"]); rp.append(o["router_probs"])
            # the key / value rows appended at this step: kp / vp were copied from the device after the CUDA step and
            # the oracle has just overwritten its own rows in them; a fresh copy still holds what the CUDA path stored
            if l in (0, model["n_layers"] // 2, model["n_layers"] - 1):
                rows = [(int(bt[i, self.cur[b] // ps]), self.cur[b] % ps) for i, b in enumerate(subset)]
                okp, ovp = self.k_pool[l, flat].cpu(), self.v_pool[l, flat].cpu()
                check_cache_rows(okp[None], ovp[None], kp[None], vp[None], rows, label=f"layer {l} appended rows", first_layer=l)
        logits = oracle.lm_head(ocfg.__class__(**model), self.weights["final_norm"].cpu(), self.weights["lm_head"].cpu(), x)
        return dict(hidden=torch.stack(hidden), router_idx=torch.stack(ridx), router_w=torch.stack(rw),
                    router_probs=torch.stack(rp), logits=logits)


def take(gpu, subset):
    idx = torch.tensor(subset)
    return dict(tokens=gpu["tokens"].cpu()[idx], logp=gpu["logp"].cpu()[idx], logits=gpu["logits"][idx.to(DEV)].cpu(),
                hidden=gpu["hidden"][:, idx.to(DEV)].cpu(), router_w=gpu["router_w"][:, idx.to(DEV)].cpu(),
                router_idx=gpu["router_idx"][:, idx.to(DEV)].cpu(), nucleus_mass=gpu["nucleus_mass"].cpu()[idx])


def test_config3_full_model_decode_top_p(full_weights):
    """Step 0 is checked on 8 of the 64 sequences (spread over the sorted context lengths), step 1 on 3.
    One checked sequence ends one token short of a 64-token page and owns no page beyond it: step 0
    fills the page, step 1 makes the library take a new page from the free list inside the step."""
    cfg = wl.CONFIGS[3]
    ctx0, _ = wl.make_context_lengths(cfg, seed=wl.CONFIG3_CONTEXT_SEED)
    order = sorted(range(len(ctx0)), key=lambda b: ctx0[b])
    edge = order[len(order) // 2]
    case = FullCase(cfg, full_weights, steps=2, seed=wl.CONFIG3_CONTEXT_SEED, page_edge=edge)
    assert case.ctx[edge] % 64 == 63
    tokens = wl.make_tokens(case.B, cfg["model"]["vocab"], seed=0)
    smp = dict(greedy=0, temperature=1.0, top_p=0.95)
    eight = [order[i] for i in (0, 9, 18, 27, 32, 45, 54, 63)]      # includes the shortest, the edge one and the longest
    assert edge in eight
    for step, subset in enumerate((eight, [order[0], edge, order[-1]])):
        free_before = case.kv.free_pages
        gpu = case.gpu_step(tokens, smp, step=step, seed=7)
        if step == 1:
            assert case.kv.free_pages == free_before - 1 and case.cur[edge] % 64 == 0    # the in-step page grab
        orc = case.oracle_subset(subset, tokens, gpu["router_idx"].cpu())
        g = take(gpu, subset)
        stats = compare_step(g, orc, cfg["model"]["top_k"], greedy=False, label=f"config3 step {step}")
        stats.update(compare_sampled(g, orc, 1.0, 0.95, 7, step, subset, label=f"config3 step {step}"))
        print("config3", step, stats)
        assert torch.isfinite(gpu["hidden"]).all() and torch.isfinite(gpu["logp"]).all()
        assert (gpu["nucleus_mass"] >= 0.95 - 1e-3).all()
        act = case.m.active_experts()
        assert int(act.min()) >= 100
        tokens = gpu["tokens"].cpu()                                  # teacher-force the sampled tokens
        for b in range(case.B):
            case.cur[b] += 1
    del case
    torch.cuda.empty_cache()


def test_config5_long_context_decode_greedy(full_weights):
    cfg = wl.CONFIGS[5]
    free, _ = torch.cuda.mem_get_info(0)
    model = cfg["model"]
    kv_bytes = 2 * model["n_layers"] * 16 * (65536 + 64) * model["n_kv_heads"] * model["head_dim"] * 2
    if free < kv_bytes + (3 << 30):
        pytest.skip(f"not enough free device memory for the 16 x 64k cache ({free >> 30} GiB free)")
    case = FullCase(cfg, full_weights, steps=2)
    tokens = wl.make_tokens(case.B, model["vocab"], seed=5)
    for step in range(2):
        subset = [3, 12] if step == 0 else [3]
        gpu = case.gpu_step(tokens, dict(greedy=1, temperature=1.0, top_p=1.0), step=step, seed=0)
        orc = case.oracle_subset(subset, tokens, gpu["router_idx"].cpu())
        stats = compare_step(take(gpu, subset), orc, model["top_k"], greedy=True, label=f"config5 step {step}")
        print("config5", step, stats)
        assert torch.isfinite(gpu["hidden"]).all()
        tokens = gpu["tokens"].cpu()
        for b in range(case.B):
            case.cur[b] += 1
    del case
    torch.cuda.empty_cache()


def test_config4_mixed_batch_decode_and_prefill(full_weights):
    """192 decode sequences (lognormal contexts by stage) plus chunked prefill on the 48-layer model.
    The decode step is checked against the oracle on three sequences.  Prefill: a 264-token chunk
    that continues a cached context -- more than 256 rows, so it runs on the dense tensor-core
    contractions and the tensor-core causal attention like the benchmark's call -- is checked against
    the oracle token by token through all 48 layers (a 2048-token chunk would cost the CPU oracle
    tens of minutes); the full 8 x 2048 call of the benchmark is
    checked by a property that holds at any size: one call of 2048 tokens and two calls of 1024
    give the same last-position logits and the same sampled token."""
    cfg = wl.CONFIGS[4]
    model, ps = cfg["model"], cfg["page_size"]
    free, _ = torch.cuda.mem_get_info(0)
    ctx, _ = wl.make_context_lengths(cfg, seed=0)
    kv_bytes = 2 * model["n_layers"] * (sum(ctx) + 8 * 2200) * model["n_kv_heads"] * model["head_dim"] * 2
    if free < kv_bytes + (8 << 30):
        pytest.skip(f"not enough free device memory for the config-4 cache ({free >> 30} GiB free)")
    B, R, CH = len(ctx), 8, 2048
    cap = [c + 3 for c in ctx] + [CH + 100] * R
    n_pages = sum(wl.pages_needed(c, ps) for c in cap) + 4
    max_pages = max(wl.pages_needed(c, ps) for c in cap) + 1
    pages = wl.make_page_assignment(cap, ps, n_pages, seed=0)
    k_pool, v_pool = wl.make_kv_pools(model, n_pages, ps, seed=0, device=DEV)
    m = binding.Model(model, full_weights, max_decode_seqs=B, max_prefill_tokens=R * CH, max_pos=max(cap) + 8)
    kv = binding.KvCache(m, k_pool, v_pool, ps, B + R, max_pages)
    for b in range(B):
        kv.seq_adopt(b, pages[b], ctx[b])
    case = FullCase.__new__(FullCase)
    case.cfg, case.model, case.ps, case.weights = cfg, model, ps, full_weights
    case.ctx, case.B, case.pages, case.k_pool, case.v_pool, case.m, case.kv = ctx, B, pages, k_pool, v_pool, m, kv
    case.cur = list(ctx)
    case.page_edge = None

    # --- decode part
    tokens = wl.make_tokens(B, model["vocab"], seed=4)
    order = sorted(range(B), key=lambda b: ctx[b])
    subset = [order[0], order[B // 2], order[-1]]
    smp = dict(greedy=0, temperature=1.0, top_p=0.95)
    gpu = case.gpu_step(tokens, smp, step=0, seed=11)
    orc = case.oracle_subset(subset, tokens, gpu["router_idx"].cpu())
    g = take(gpu, subset)
    stats = compare_step(g, orc, model["top_k"], greedy=False, label="config4 decode")
    stats.update(compare_sampled(g, orc, 1.0, 0.95, 11, 0, subset, label="config4 decode"))
    print("config4 decode", stats)
    assert torch.isfinite(gpu["hidden"]).all()
    del gpu

    # --- prefill, oracle-checked: 264 tokens (> 256: the dense tcgen05 path) continuing 40 cached tokens of a fresh slot
    L, H, k, V = model["n_layers"], model["hidden"], model["top_k"], model["vocab"]
    slot, prior, n = B, 40, 264
    kv.seq_adopt(slot, pages[slot], prior)
    ptoks = wl.make_tokens(n, V, seed=9, name="prompt")
    out_t = torch.empty(1, dtype=torch.int32, device=DEV)
    out_l = torch.empty(1, device=DEV)
    logits = torch.empty(1, V, device=DEV)
    hidden = torch.empty(L + 1, n, H, device=DEV)
    ridx = torch.empty(L, n, k, dtype=torch.int32, device=DEV)
    rw = torch.empty(L, n, k, device=DEV)
    st = binding.mars_prefill_chunk(m, kv, [slot], [n], ptoks.to(DEV), [1], binding.make_sampling(greedy=1), out_t, out_l,
                                    binding.make_debug(logits, hidden, rw, ridx))
    assert st == 0 and m.poll_status() == 0
    ocfg1 = oracle.Config(**dict(model, n_layers=1))
    pg = pages[slot][: wl.pages_needed(prior + n, ps)]
    flat = torch.tensor(pg, dtype=torch.long, device=DEV)
    bt = torch.arange(len(pg), dtype=torch.int32)[None, :].contiguous()
    seq = torch.zeros(n, dtype=torch.int32)
    pos = torch.arange(prior, prior + n, dtype=torch.int32)
    x = oracle.embed(full_weights["embed"][ptoks.long().to(DEV)].cpu().contiguous(), torch.arange(n, dtype=torch.int32))
    hid, oi, ow, op = [x.clone()], [], [], []
    ridx_c = ridx.cpu()
    for l in range(L):
        layer = {f: t.cpu() for f, t in full_weights["layers"][l].items()}
        kp, vp = k_pool[l, flat].cpu(), v_pool[l, flat].cpu()
        # the oracle recomputes the chunk's own keys/values; positions < prior come from the generator
        o = oracle.layer_forward(ocfg1, layer, x, seq, pos, kp, vp, bt, ps, forced_idx=ridx_c[l].contiguous())
        hid.append(x.clone()); oi.append(o["router_idx"]); ow.append(o["router_w"]); op.append(o["router_probs"])
    ologits = oracle.lm_head(oracle.Config(**model), full_weights["final_norm"].cpu(), full_weights["lm_head"].cpu(), x[-1:].contiguous())
    gp = dict(router_idx=ridx_c, router_w=rw.cpu(), hidden=hidden.cpu(), logits=logits.cpu(), tokens=out_t.cpu(), logp=out_l.cpu())
    op_ = dict(hidden=torch.stack(hid), router_idx=torch.stack(oi), router_w=torch.stack(ow), router_probs=torch.stack(op),
               logits=ologits)
    stats = compare_step(gp, op_, k, greedy=True, label="config4 prefill chunk")
    print("config4 prefill", stats)
    kv.seq_release(slot)
    del hidden, ridx, rw

    # --- the same chunk through the scoring pass: log-probs of sampled rows against the oracle (T = 0.85)
    kv.seq_adopt(slot, pages[slot], prior)
    tgt = torch.cat([ptoks[1:], ptoks[:1]]).to(torch.int32)
    slp = torch.empty(n, device=DEV)
    st = binding.mars_score_chunk(m, kv, [slot], [n], ptoks.to(DEV), tgt.to(DEV), 0.85, slp)
    assert st == 0 and m.poll_status() == 0
    rows = [0, 17, 150, n - 1]
    olog = oracle.lm_head(oracle.Config(**model), full_weights["final_norm"].cpu(), full_weights["lm_head"].cpu(),
                          x[torch.tensor(rows)].contiguous())
    werr = max(abs(float(slp[r]) - oracle.logprob_of(olog[i].contiguous(), 0.85, int(tgt[r]))) for i, r in enumerate(rows))
    print("config4 score chunk: max log-prob error on sampled rows", werr)
    assert werr <= 2e-2
    kv.seq_release(slot)

    # --- the benchmark's 8 x 2048 call: one call equals two half calls (same logits, same token)
    big = wl.make_tokens(R * CH, V, seed=1, name="prompts").to(DEV)
    ids = list(range(B, B + R))
    lg = [torch.empty(R, V, device=DEV) for _ in range(2)]
    tk = [torch.empty(R, dtype=torch.int32, device=DEV) for _ in range(2)]
    lp = torch.empty(R, device=DEV)
    for s_ in ids:
        kv.seq_reserve(s_, 0)
    st = binding.mars_prefill_chunk(m, kv, ids, [CH] * R, big, [1] * R, binding.make_sampling(greedy=1), tk[0], lp,
                                    binding.make_debug(lg[0]))
    assert st == 0 and m.poll_status() == 0
    for s_ in ids:
        kv.seq_release(s_)
        kv.seq_reserve(s_, 0)
    half = CH // 2
    first = torch.cat([big[r * CH: r * CH + half] for r in range(R)])
    second = torch.cat([big[r * CH + half: (r + 1) * CH] for r in range(R)])
    for part in (first, second):
        st = binding.mars_prefill_chunk(m, kv, ids, [half] * R, part.contiguous(), [1] * R, binding.make_sampling(greedy=1),
                                        tk[1], lp, binding.make_debug(lg[1]))
        assert st == 0 and m.poll_status() == 0
    torch.cuda.synchronize()
    assert torch.isfinite(lg[0]).all()
    assert (lg[0] - lg[1]).abs().max() < 2e-3, float((lg[0] - lg[1]).abs().max())
    top2 = torch.topk(lg[0], 2, dim=-1).values
    sure = (top2[:, 0] - top2[:, 1]) >= 1e-2
    assert torch.equal(tk[0][sure], tk[1][sure])
    for s_ in ids:
        assert kv.seq_len(s_) == CH

    # --- scoring the same 8 x 2048 tokens: the last row of every request must reproduce the log-prob that
    # the prefill call's logits give to the token it sampled (vocabulary of 151936 = 593.5 column tiles)
    for s_ in ids:
        kv.seq_release(s_)
        kv.seq_reserve(s_, 0)
    tg = torch.cat([big[1:], big[:1]]).clone()
    last = torch.arange(R, device=DEV) * CH + CH - 1
    tg[last] = tk[0]
    slp = torch.empty(R * CH, device=DEV)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    st = binding.mars_score_chunk(m, kv, ids, [CH] * R, big, tg, 1.0, slp)
    e1.record()
    assert st == 0 and m.poll_status() == 0
    want = torch.log_softmax(lg[0].double(), -1).gather(-1, tk[0].long()[:, None])[:, 0]
    diff = float((slp[last].double() - want).abs().max())
    print(f"config4 score 8 x 2048: {e0.elapsed_time(e1):.1f} ms, last-row log-prob diff {diff:.2e}, "
          f"mean log-prob {float(slp.mean()):.3f}")
    assert diff <= 2e-3
    assert torch.isfinite(slp).all() and float(slp.max()) <= 0.0
