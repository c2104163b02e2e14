"""Mixed step: decode rows and prompt chunks in one pass per layer (the pipeline's steady state,
Section 3.3), against the CPU oracle and against the two separate calls."""
import pytest
import torch

import oracle
from harness import TOL_LOGIT_ABS, Case, compare_sampled, compare_step
from paper_2511_11373_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


def mixed(case, dec_ids, dec_tokens, req_ids, lens, chunk_tokens, emit, sampling, step=0, seed=0):
    dev, m = case.device, case.model_shape
    L, H, k, V = m["n_layers"], m["hidden"], m["top_k"], m["vocab"]
    n = len(dec_ids) + sum(lens)
    n_emit = len(dec_ids) + sum(1 for e in emit if e)
    out = dict(tokens=torch.empty(n_emit, dtype=torch.int32, device=dev), logp=torch.empty(n_emit, device=dev),
               logits=torch.empty(n_emit, V, device=dev), hidden=torch.empty(L + 1, n, H, device=dev),
               router_w=torch.empty(L, n, k, device=dev), router_idx=torch.empty(L, n, k, dtype=torch.int32, device=dev),
               nucleus_mass=torch.empty(n_emit, device=dev))
    dbg = binding.make_debug(out["logits"], out["hidden"], out["router_w"], out["router_idx"], None, out["nucleus_mass"])
    st = binding.mars_mixed_step(case.model, case.kv, dec_ids, dec_tokens.to(dev), req_ids, lens, chunk_tokens.to(dev), emit,
                                 binding.make_sampling(seed=seed, step=step, **sampling), out["tokens"], out["logp"], dbg)
    assert st == 0, binding.STATUS_NAMES.get(st, st)
    assert case.model.poll_status() == 0
    return {k_: v.cpu() for k_, v in out.items()}


@pytest.mark.parametrize("ctx,n_dec,lens,emit", [([33, 80, 0, 21], 2, [50, 40], [1, 0]),      # 92 rows: tensor-core tiles
                                                 ([17, 5, 130, 16, 0], 3, [4, 7], [1, 1])])   # 14 rows: streaming path
def test_mixed_step_matches_the_oracle(ctx, n_dec, lens, emit):
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    V, ps = model["vocab"], 16
    B = len(ctx)
    case = Case(model, ps, ctx, seed=71, headroom=max(lens) + 3, max_prefill_tokens=n_dec + sum(lens), max_decode=B)
    dec_ids, req_ids = list(range(n_dec)), list(range(n_dec, B))
    dec_tok = wl.make_tokens(n_dec, V, seed=2)
    chunk_tok = wl.make_tokens(sum(lens), V, seed=3)
    smp = dict(greedy=0, temperature=0.85, top_p=0.95)
    g = mixed(case, dec_ids, dec_tok, req_ids, lens, chunk_tok, emit, smp, step=4, seed=6)
    seq = torch.tensor(dec_ids + [req_ids[r] for r in range(len(lens)) for _ in range(lens[r])], dtype=torch.int32)
    pos = torch.tensor([ctx[b] for b in dec_ids] + [ctx[req_ids[r]] + i for r in range(len(lens)) for i in range(lens[r])],
                       dtype=torch.int32)
    orc = oracle.forward(case.ocfg, case.w_cpu, torch.cat([dec_tok, chunk_tok]), seq, pos, case.k_cpu, case.v_cpu, case.bt, ps,
                         forced_idx=g["router_idx"].contiguous())
    emit_rows, slots, at = list(range(n_dec)), list(dec_ids), n_dec
    for r, n in enumerate(lens):
        at += n
        if emit[r]:
            emit_rows.append(at - 1)
            slots.append(req_ids[r])
    orc_e = dict(orc, logits=orc["logits"][torch.tensor(emit_rows)])
    stats = compare_step(g, orc_e, model["top_k"], greedy=False, label="mixed")
    stats.update(compare_sampled(g, orc_e, 0.85, 0.95, 6, 4, slots, label="mixed"))
    print("mixed", len(seq), stats)
    for b in dec_ids:
        assert case.kv.seq_len(b) == ctx[b] + 1
    for r, b in enumerate(req_ids):
        assert case.kv.seq_len(b) == ctx[b] + lens[r]
    # every sequence continues with a decode step on top of what the mixed step cached
    case.cur = [case.kv.seq_len(b) for b in range(B)]
    tok = wl.make_tokens(B, V, seed=9)
    g2 = case.gpu_decode(tok, dict(greedy=1, temperature=1.0, top_p=1.0))
    o2 = case.oracle_decode(tok, forced_idx=g2["router_idx"].contiguous())
    print("decode after mixed", compare_step(g2, o2, model["top_k"], greedy=True, label="decode after mixed"))


def test_mixed_step_equals_the_two_separate_calls():
    model = dict(wl.MODEL_TINY, n_layers=2)
    V, ps, ctx, lens = model["vocab"], 32, [40, 100, 7, 0], [60, 45]
    dec_tok = wl.make_tokens(2, V, seed=4)
    chunk_tok = wl.make_tokens(sum(lens), V, seed=5)
    greedy = dict(greedy=1, temperature=1.0, top_p=1.0)
    a = Case(model, ps, ctx, seed=72, headroom=70, max_prefill_tokens=2 + sum(lens), max_decode=4, poison=False)
    ga = mixed(a, [0, 1], dec_tok, [2, 3], lens, chunk_tok, [1, 1], greedy)
    b = Case(model, ps, ctx, seed=72, headroom=70, max_prefill_tokens=2 + sum(lens), max_decode=4, poison=False)
    gd = b.gpu_decode(dec_tok, greedy, seq_ids=[0, 1])
    dev = b.device
    out_t = torch.empty(2, dtype=torch.int32, device=dev)
    out_l = torch.empty(2, device=dev)
    logits = torch.empty(2, V, device=dev)
    st = binding.mars_prefill_chunk(b.model, b.kv, [2, 3], lens, chunk_tok.to(dev), [1, 1], binding.make_sampling(greedy=1),
                                    out_t, out_l, binding.make_debug(logits))
    assert st == 0 and b.model.poll_status() == 0
    sep = torch.cat([gd["logits"], logits.cpu()])
    d = float((ga["logits"] - sep).abs().max())
    print("mixed vs separate: max logit diff", d)
    assert d <= 2e-3
    assert torch.equal(ga["tokens"], torch.cat([gd["tokens"], out_t.cpu()]))
    for s in range(4):
        assert a.kv.seq_len(s) == b.kv.seq_len(s)


def test_mixed_step_argument_checks():
    model = dict(wl.MODEL_TINY, n_layers=1)
    case = Case(model, 16, [10, 3, 0], seed=73, headroom=12, max_prefill_tokens=12, max_decode=3)
    dev = case.device
    tok = wl.make_tokens(16, model["vocab"], seed=1).to(dev)
    out_t = torch.empty(3, dtype=torch.int32, device=dev)
    out_l = torch.empty(3, device=dev)
    smp = binding.make_sampling(greedy=1)
    call = lambda d, r, lens, emit=None: binding.mars_mixed_step(case.model, case.kv, d, tok, r, lens, tok, emit, smp, out_t, out_l)
    assert call([0, 1], [1], [4]) == 6                         # a slot in both lists
    assert call([0], [2], [12]) == 1                           # 13 rows > 12
    assert call([], [2], [4]) == 1                             # no decode rows: that is mars_prefill_chunk
    assert call([0, 1], [2], [4], [1]) == 0                    # 3 emitting rows = max_decode_seqs
    assert case.model.poll_status() == 0
    assert [case.kv.seq_len(s) for s in range(3)] == [11, 4, 4]
