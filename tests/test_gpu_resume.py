"""Carrying sequences across rollout segments and forking group members (Section 2.3, segment
rollouts; Section 3.3, grouped agentic rollouts).

A trajectory that is cut at a segment boundary resumes later.  Whether its pages were kept, packed
into a host image and restored into other pages, or thrown away and the prefix prefilled again, the
next-token distribution must be the same: bit for bit for the first two (same kernels, same
arithmetic, only the page ids differ), within the logit tolerance for the re-prefill (the prefix
rows go through the prefill kernels).  A forked sequence must behave like one that was never
shared.
"""
import pytest
import torch

from harness import TOL_LOGIT_ABS, Case
from paper_2511_11373_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

GREEDY = dict(greedy=1, temperature=1.0, top_p=1.0)


def prefill(case, slots, tokens, emit=True):
    """Feeds `tokens` (same chunk for every listed slot) and returns (next tokens, logits)."""
    dev, V, n = case.device, case.model_shape["vocab"], len(slots)
    out_t = torch.empty(n, dtype=torch.int32, device=dev)
    out_l = torch.empty(n, dtype=torch.float32, device=dev)
    logits = torch.empty(n, V, dtype=torch.float32, device=dev)
    toks = tokens.repeat(n).to(dev)
    st = binding.mars_prefill_chunk(case.model, case.kv, slots, [len(tokens)] * n, toks, [1 if emit else 0] * n,
                                    binding.make_sampling(greedy=1), out_t, out_l, binding.make_debug(logits))
    assert st == 0 and case.model.poll_status() == 0
    return out_t.cpu(), logits.cpu()


def test_kept_pages_host_image_and_reprefill_give_the_same_continuation():
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    ps, P, N1, N2 = 16, 45, 7, 6
    case = Case(model, ps, [0, 0, 0], seed=41, headroom=P + N1 + N2 + 2, spare_pages=12, poison=False,
                max_prefill_tokens=3 * (P + N1), extra_seqs=1)
    kv = case.kv
    prompt = wl.make_tokens(P, model["vocab"], seed=90)
    nxt, _ = prefill(case, [0, 1], prompt)
    assert int(nxt[0]) == int(nxt[1])
    generated = [int(nxt[0])]
    for step in range(N1):                                   # first segment: slots 0 and 1 decode together
        tok = torch.tensor([generated[-1]] * 2, dtype=torch.int32)
        g = case.gpu_decode(tok, GREEDY, seq_ids=[0, 1], step=step)
        assert torch.equal(g["logits"][0], g["logits"][1])
        generated.append(int(g["tokens"][0]))
    n_cached = P + N1
    assert kv.seq_len(0) == n_cached and kv.seq_len(1) == n_cached

    # slot 1: park in pinned host memory, give its pages away, come back somewhere else
    nbytes = kv.seq_image_bytes(n_cached)
    page_bytes = model["n_kv_heads"] * ps * model["head_dim"] * 2
    assert nbytes == 2 * model["n_layers"] * wl.pages_needed(n_cached, ps) * page_bytes
    image = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    assert kv.seq_export(1, image) == 0
    old_pages = kv.block_table(1)
    free_before = kv.free_pages
    kv.seq_release(1)
    torch.cuda.synchronize()
    assert kv.free_pages == free_before + len(old_pages)
    kv.seq_reserve(3, len(old_pages) * ps)                   # another trajectory takes exactly those pages
    assert sorted(kv.block_table(3)) == sorted(old_pages)
    idx = torch.tensor(old_pages, device=case.device)
    case.k_pool[:, idx] = float("nan")
    case.v_pool[:, idx] = float("nan")
    assert kv.seq_import(1, image, n_cached) == 0
    assert kv.seq_len(1) == n_cached and not set(kv.block_table(1)) & set(old_pages)
    # the image holds the same rows as the kept pages of slot 0
    new_pages = kv.block_table(1)
    for i, (a, b) in enumerate(zip(kv.block_table(0), new_pages)):
        used = min(ps, n_cached - i * ps)
        assert torch.equal(case.k_pool[:, a, :, :used], case.k_pool[:, b, :, :used])
        assert torch.equal(case.v_pool[:, a, :, :used], case.v_pool[:, b, :, :used])

    # slot 2: nothing was kept; the prefix (prompt + generated tokens that are cached) is prefilled again
    prefix = torch.cat([prompt, torch.tensor(generated[:N1], dtype=torch.int32)])
    nxt2, logits2 = prefill(case, [2], prefix)
    assert kv.seq_len(2) == n_cached

    # second segment: all three continue with the same inputs
    worst = 0.0
    for step in range(N2):
        tok = torch.tensor([generated[-1]] * 3, dtype=torch.int32)
        g = case.gpu_decode(tok, GREEDY, seq_ids=[0, 1, 2], step=N1 + step)
        assert torch.equal(g["logits"][0], g["logits"][1]), "restored pages changed the result"
        assert torch.equal(g["logp"][0], g["logp"][1]) and int(g["tokens"][0]) == int(g["tokens"][1])
        d = float((g["logits"][0] - g["logits"][2]).abs().max())
        worst = max(worst, d)
        assert d <= TOL_LOGIT_ABS, (step, d)
        top2 = torch.topk(g["logits"][0], 2).values
        if float(top2[0] - top2[1]) >= 2 * TOL_LOGIT_ABS:
            assert int(g["tokens"][2]) == int(g["tokens"][0])
        generated.append(int(g["tokens"][0]))
    print("resume: max |logit(kept) - logit(re-prefilled)| =", worst)
    # the token the re-prefill emitted is the one the first segment's last step produced
    assert int(nxt2[0]) == generated[N1]


def test_export_import_argument_checks():
    model = dict(wl.MODEL_TINY, n_layers=1)
    case = Case(model, 16, [20], seed=3, extra_seqs=1, spare_pages=0, headroom=1)
    kv = case.kv
    n = kv.seq_image_bytes(20)
    pageable = torch.empty(n, dtype=torch.uint8)
    assert kv.seq_export(0, pageable) == 1                    # a kernel cannot address pageable host memory
    small = torch.empty(n - 16, dtype=torch.uint8, device=case.device)
    assert kv.seq_export(0, small) == 1
    assert kv.seq_export(1, small) == 6                       # empty slot
    image = torch.empty(n, dtype=torch.uint8, device=case.device)
    assert kv.seq_export(0, image) == 0                       # a device image works too
    assert kv.seq_import(0, image, 20) == 6                   # slot in use
    assert kv.seq_import(1, image, 20) == 4 and kv.seq_len(1) == -1      # no free page: slot stays empty
    kv.seq_release(0)
    assert kv.seq_import(1, image, 20) == 0 and kv.seq_len(1) == 20
    assert kv.seq_image_bytes(0) == 0 and kv.seq_image_bytes(-1) == 0
    torch.cuda.synchronize()


def test_fork_shares_full_pages_and_copies_the_partial_page():
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    ps, ctx = 16, 40                                          # two full pages and 8 tokens in the third
    case = Case(model, ps, [ctx], seed=51, headroom=30, spare_pages=10, extra_seqs=3, max_decode=4)
    kv = case.kv
    total_free = kv.free_pages
    src_pages = kv.block_table(0)
    assert kv.seq_fork(0, 1) == 0 and kv.seq_fork(0, 2) == 0
    assert kv.seq_fork(0, 1) == 6 and kv.seq_fork(3, 1) == 6 and kv.seq_fork(0, 0) == 6
    assert kv.free_pages == total_free - 2                    # one copied page per fork
    for s in (1, 2):
        bt = kv.block_table(s)
        assert bt[:2] == src_pages[:2] and bt[2] != src_pages[2] and len(bt) == 3 and kv.seq_len(s) == ctx
    assert [kv.page_refs(p) for p in src_pages[:3]] == [3, 3, 1]
    with pytest.raises(binding.MarsError):
        kv.seq_set_len(1, 20)                                 # the next append would land in a shared page
    kv.seq_set_len(1, ctx)

    # an unshared twin: the same case, where the members are plain copies in pages of their own
    twin = Case(model, ps, [ctx], seed=51, headroom=30, spare_pages=10, extra_seqs=3, max_decode=4)
    for s in (1, 2):
        twin.kv.seq_reserve(s, ctx)
        for a, b in zip(twin.kv.block_table(0), twin.kv.block_table(s)):
            twin.k_pool[:, b] = twin.k_pool[:, a]
            twin.v_pool[:, b] = twin.v_pool[:, a]
        twin.kv.seq_set_len(s, ctx)
    V = model["vocab"]
    smp = dict(greedy=0, temperature=0.85, top_p=1.0)
    ids = [0, 1, 2]
    for step in range(14):                                    # members diverge; position 48 opens a new page each
        toks = wl.make_tokens(3, V, seed=100 + step)[torch.tensor(ids)]
        if step == 0:
            toks = toks[:1].repeat(len(ids))                  # same input: the members must still agree exactly
        g = case.gpu_decode(toks, smp, seq_ids=ids, step=step, seed=4)
        t = twin.gpu_decode(toks, smp, seq_ids=ids, step=step, seed=4)
        assert torch.equal(g["logits"], t["logits"]) and torch.equal(g["tokens"], t["tokens"]), step
        if step == 0:
            assert torch.equal(g["logits"][0], g["logits"][1]) and torch.equal(g["logits"][0], g["logits"][2])
        if step == 5:
            kv.seq_release(0)                                 # the source leaves; its shared pages must survive
            assert [kv.page_refs(p) for p in src_pages[:3]] == [2, 2, 0]
            assert kv.seq_fork(1, 0) == 0                     # its slot is reused by a fork of a member ...
            assert [kv.page_refs(p) for p in src_pages[:2]] == [3, 3]
            kv.seq_release(0)                                 # ... which leaves again
            twin.kv.seq_release(0)
            ids = [1, 2]
    for s in (1, 2):
        kv.seq_release(s)
    torch.cuda.synchronize()
    assert kv.free_pages == kv.num_pages and all(kv.page_refs(p) == 0 for p in range(kv.num_pages))


def test_fork_at_a_page_boundary_and_without_free_pages():
    model = dict(wl.MODEL_TINY, n_layers=1)
    case = Case(model, 16, [32, 5], seed=52, headroom=0, spare_pages=0, extra_seqs=2, max_decode=4)
    kv = case.kv
    assert kv.free_pages == 0
    assert kv.seq_fork(0, 2) == 0                             # nothing to copy: both pages are full
    assert kv.block_table(2) == kv.block_table(0) and kv.seq_len(2) == 32
    assert kv.seq_fork(1, 3) == 4 and kv.seq_len(3) == -1     # the partial page needs a free page
    tok = wl.make_tokens(2, model["vocab"], seed=2).to(case.device)
    out_t = torch.empty(2, dtype=torch.int32, device=case.device)
    out_l = torch.empty(2, dtype=torch.float32, device=case.device)
    assert binding.mars_decode_step(case.model, kv, [0, 2], tok, binding.make_sampling(greedy=1), out_t, out_l) == 4
    kv.seq_release(1)                                         # one page comes back: enough for one of the two
    assert binding.mars_decode_step(case.model, kv, [0], tok, binding.make_sampling(greedy=1), out_t, out_l) == 0
    assert case.model.poll_status() == 0 and kv.seq_len(0) == 33 and kv.seq_len(2) == 32


def _slice_rows(d, rows, per_row=("tokens", "logp", "logits", "nucleus_mass")):
    """Rows `rows` of a result dict (taps are [L, n, ...], outputs [n, ...])."""
    idx = torch.tensor(rows)
    out = {}
    for key, v in d.items():
        if key in ("expert_off", "slot_token", "active_experts"):
            continue
        out[key] = v[idx] if key in per_row else v[:, idx]
    return out


def test_resumed_sequences_match_the_oracle():
    """Section 2.3 (segment rollouts): the first decode step of the next segment is compared with the
    CPU oracle run over the whole prefix, for a slot that kept its pages, a slot restored from a host
    image into other pages, and a slot whose prefix was prefilled again.  The oracle is teacher-forced
    with the tokens of the first segment and, by the cascade rule, with the routing the CUDA path took
    at every position of the prefix (the prefill call's and the decode steps' taps for the kept slots;
    the re-prefill's own taps for the third)."""
    import oracle
    from harness import compare_step
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    ps, P, N1 = 16, 45, 7
    L, H, k, V, E = model["n_layers"], model["hidden"], model["top_k"], model["vocab"], model["n_experts"]
    case = Case(model, ps, [0, 0, 0], seed=43, headroom=P + N1 + 4, spare_pages=12, poison=False,
                max_prefill_tokens=3 * (P + N1), extra_seqs=1)
    kv, dev = case.kv, case.device

    def prefill_taps(slots, tokens):
        n, R = len(tokens) * len(slots), len(slots)
        out = dict(tokens=torch.empty(R, dtype=torch.int32, device=dev), logp=torch.empty(R, device=dev),
                   logits=torch.empty(R, V, device=dev), hidden=torch.empty(L + 1, n, H, device=dev),
                   router_w=torch.empty(L, n, k, device=dev), router_idx=torch.empty(L, n, k, dtype=torch.int32, device=dev))
        dbg = binding.make_debug(out["logits"], out["hidden"], out["router_w"], out["router_idx"])
        st = binding.mars_prefill_chunk(case.model, kv, slots, [len(tokens)] * R, tokens.repeat(R).to(dev), [1] * R,
                                        binding.make_sampling(greedy=1), out["tokens"], out["logp"], dbg)
        assert st == 0 and case.model.poll_status() == 0
        return {key: v.cpu() for key, v in out.items()}

    # ---- first segment on slots 0 and 1: prompt, then N1 greedy steps; the taps of slot 0 are kept
    prompt = wl.make_tokens(P, V, seed=91)
    pf = prefill_taps([0, 1], prompt)
    generated = [int(pf["tokens"][0])]
    ridx_a, hid_a = [pf["router_idx"][:, :P]], [pf["hidden"][:, :P]]
    for step in range(N1):
        g = case.gpu_decode(torch.tensor([generated[-1]] * 2, dtype=torch.int32), GREEDY, seq_ids=[0, 1], step=step)
        ridx_a.append(g["router_idx"][:, :1]); hid_a.append(g["hidden"][:, :1])
        generated.append(int(g["tokens"][0]))
    n_cached = P + N1
    prefix = torch.cat([prompt, torch.tensor(generated[:N1], dtype=torch.int32)])

    # ---- slot 1 goes through a host image into other pages; slot 2 prefills the prefix again
    image = torch.empty(kv.seq_image_bytes(n_cached), dtype=torch.uint8).pin_memory()
    assert kv.seq_export(1, image) == 0
    old_pages = kv.block_table(1)
    kv.seq_release(1)
    torch.cuda.synchronize()
    kv.seq_reserve(3, len(old_pages) * ps)
    idx = torch.tensor(old_pages, device=dev)
    case.k_pool[:, idx] = float("nan"); case.v_pool[:, idx] = float("nan")
    assert kv.seq_import(1, image, n_cached) == 0
    pf2 = prefill_taps([2], prefix)

    # ---- oracle over the prefix, once per routing history
    seq0, pos = torch.zeros(n_cached, dtype=torch.int32), torch.arange(n_cached, dtype=torch.int32)
    bt = case.bt[:1].contiguous()
    def oracle_prefix(forced):
        kc, vc = case.k_cpu.clone(), case.v_cpu.clone()
        res = oracle.forward(case.ocfg, case.w_cpu, prefix, seq0, pos, kc, vc, bt, ps, forced_idx=forced.contiguous())
        return res, kc, vc
    forced_a = torch.cat(ridx_a, dim=1)
    orc_a, k_a, v_a = oracle_prefix(forced_a)
    orc_b, k_b, v_b = oracle_prefix(pf2["router_idx"])
    # the prefix itself: hidden states of every position on both histories, and the re-prefill's output
    for name, got, orc in (("kept", torch.cat(hid_a, dim=1), orc_a), ("re-prefilled", pf2["hidden"], orc_b)):
        rel = (got.double() - orc["hidden"].double()).norm(dim=-1) / orc["hidden"].double().norm(dim=-1).clamp_min(1e-30)
        assert float(rel.max()) <= 1e-2, (name, float(rel.max()))
    stats = compare_step(pf2, dict(orc_b, logits=orc_b["logits"][-1:]), k, greedy=True, label="re-prefill of the prefix")
    print("resume: re-prefill vs oracle", stats)

    # ---- the first step of the next segment, row by row against the oracle
    tok = torch.tensor([generated[N1]] * 3, dtype=torch.int32)
    g = case.gpu_decode(tok, GREEDY, seq_ids=[0, 1, 2], step=N1)
    assert torch.equal(g["logits"][0], g["logits"][1]), "restored pages changed the result"
    one = torch.tensor([n_cached], dtype=torch.int32)
    for row, (kc, vc) in ((0, (k_a, v_a)), (1, (k_a, v_a)), (2, (k_b, v_b))):
        gr = _slice_rows(g, [row])
        o = oracle.forward(case.ocfg, case.w_cpu, tok[:1].contiguous(), seq0[:1].contiguous(), one, kc.clone(), vc.clone(), bt, ps,
                           forced_idx=gr["router_idx"].contiguous())
        stats = compare_step(gr, o, k, greedy=True, label=f"resumed row {row}")
        print("resume: row", row, stats)
