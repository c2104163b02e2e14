"""Teacher-forced scoring pass: log pi(o_t | q, o_<t) for every position of known tokens (the
numerator of the importance ratio, Eq. 3) against the CPU oracle, and against the log-prob that the
decode step reports for the same token at the same position."""
import pytest
import torch

import oracle
from harness import TOL_LOGIT_ABS, Case, compare_step
from paper_2511_11373_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


def score(case, slots, lens, tokens, targets, temperature, want_logits=True):
    dev, m = case.device, case.model_shape
    n = sum(lens)
    L, H, k, V = m["n_layers"], m["hidden"], m["top_k"], m["vocab"]
    out = dict(logp=torch.full((n,), 99.0, dtype=torch.float32, device=dev),
               logits=torch.empty(n, V, dtype=torch.float32, device=dev) if want_logits else None,
               hidden=torch.empty(L + 1, n, H, dtype=torch.float32, device=dev),
               router_w=torch.empty(L, n, k, dtype=torch.float32, device=dev),
               router_idx=torch.empty(L, n, k, dtype=torch.int32, device=dev))
    dbg = binding.make_debug(out["logits"], out["hidden"], out["router_w"], out["router_idx"])
    st = binding.mars_score_chunk(case.model, case.kv, slots, lens, tokens.to(dev), targets.to(dev), temperature,
                                  out["logp"], dbg)
    assert st == 0, binding.STATUS_NAMES.get(st, st)
    assert case.model.poll_status() == 0
    return {k_: (v.cpu() if v is not None else None) for k_, v in out.items()}


def next_token_targets(tokens, lens):
    """targets[i] = the token that follows row i inside its request; -1 on each request's last row."""
    t = torch.full_like(tokens, -1)
    at = 0
    for n in lens:
        t[at:at + n - 1] = tokens[at + 1:at + n]
        at += n
    return t


def oracle_rows(case, ctx, lens, tokens, forced):
    seq = torch.tensor([r for r in range(len(lens)) for _ in range(lens[r])], dtype=torch.int32)
    pos = torch.tensor([ctx[r] + i for r in range(len(lens)) for i in range(lens[r])], dtype=torch.int32)
    return oracle.forward(case.ocfg, case.w_cpu, tokens, seq, pos, case.k_cpu, case.v_cpu, case.bt, case.ps,
                          forced_idx=forced.contiguous())


@pytest.mark.parametrize("lens,vocab,temperature", [([70, 30, 1], 1000, 0.85), ([9, 20], 1024, 1.0), ([130, 200], 1024, 0.6)])
def test_scores_match_the_oracle(lens, vocab, temperature):
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1, vocab=vocab)
    ctx = [0, 21, 48][: len(lens)]
    n = sum(lens)
    case = Case(model, 16, ctx, seed=61, headroom=max(lens) + 2, max_prefill_tokens=n)
    tokens = wl.make_tokens(n, vocab, seed=13)
    targets = next_token_targets(tokens, lens)
    targets[3] = -1                                            # a masked row in the middle
    g = score(case, list(range(len(lens))), lens, tokens, targets, temperature)
    orc = oracle_rows(case, ctx, lens, tokens, g["router_idx"])
    stats = compare_step(dict(g, tokens=None), orc, model["top_k"], greedy=False, label="score")
    worst = 0.0
    for i in range(n):
        if int(targets[i]) < 0:
            assert float(g["logp"][i]) == 0.0
            continue
        want = oracle.logprob_of(orc["logits"][i].contiguous(), temperature, int(targets[i]))
        worst = max(worst, abs(float(g["logp"][i]) - want))
    stats["logp_maxerr"] = worst
    print("score", lens, stats)
    assert worst <= TOL_LOGIT_ABS
    for r in range(len(lens)):
        assert case.kv.seq_len(r) == ctx[r] + lens[r]


def test_scoring_in_two_chunks_and_without_logit_tap():
    model = dict(wl.MODEL_TINY, n_layers=2)
    tokens = wl.make_tokens(150, model["vocab"], seed=5)
    targets = next_token_targets(tokens, [150])
    res = []
    for split in ((150,), (100, 50)):
        case = Case(model, 32, [7], seed=62, headroom=160, max_prefill_tokens=150, poison=False)
        parts, at = [], 0
        for n in split:
            g = score(case, [0], [n], tokens[at:at + n], targets[at:at + n], 0.85, want_logits=False)
            parts.append(g["logp"])
            at += n
        res.append(torch.cat(parts))
    assert float(res[0][-1]) == 0.0
    assert (res[0] - res[1]).abs().max() < 1e-3


def test_decode_logprob_equals_the_score_of_the_sampled_token():
    """Roll a short response out with the decode step (T 0.85, top_p 1: the behaviour-policy log-prob
    of Eq. 3), then score prompt + response in one pass: same positions, same tokens, same numbers."""
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    V, P, N, T = model["vocab"], 40, 12, 0.85
    case = Case(model, 16, [0, 0], seed=63, headroom=P + N + 2, max_prefill_tokens=P + N, poison=False)
    dev = case.device
    prompt = wl.make_tokens(P, V, seed=21)
    smp = dict(greedy=0, temperature=T, top_p=1.0)
    out_t = torch.empty(1, dtype=torch.int32, device=dev)
    out_l = torch.empty(1, dtype=torch.float32, device=dev)
    st = binding.mars_prefill_chunk(case.model, case.kv, [0], [P], prompt.to(dev), [1],
                                    binding.make_sampling(seed=9, step=0, **smp), out_t, out_l)
    assert st == 0 and case.model.poll_status() == 0
    response, behaviour = [int(out_t[0])], [float(out_l[0])]
    for step in range(1, N):
        g = case.gpu_decode(torch.tensor([response[-1]], dtype=torch.int32), smp, seq_ids=[0], step=step, seed=9)
        response.append(int(g["tokens"][0]))
        behaviour.append(float(g["logp"][0]))
    full = torch.cat([prompt, torch.tensor(response, dtype=torch.int32)])
    targets = next_token_targets(full, [P + N])
    targets[: P - 1] = -1                                      # only response tokens are scored
    g = score(case, [1], [P + N], full, targets, T, want_logits=False)
    got = g["logp"][P - 1: P + N - 1]                          # row P-1 predicts the first response token
    err = (got - torch.tensor(behaviour)).abs().max()
    print("decode vs score log-prob max diff", float(err))
    assert err <= TOL_LOGIT_ABS
    assert (g["logp"][: P - 1] == 0).all() and float(g["logp"][-1]) == 0.0
    ratio = torch.exp(got.double() - torch.tensor(behaviour, dtype=torch.float64))     # importance ratio, same weights
    assert (ratio - 1).abs().max() < 1e-2


def test_score_argument_and_target_checks():
    model = dict(wl.MODEL_TINY, n_layers=1)
    case = Case(model, 16, [5], seed=64, headroom=20, max_prefill_tokens=16)
    dev = case.device
    tok = wl.make_tokens(8, model["vocab"], seed=1).to(dev)
    tgt = torch.full((8,), -1, dtype=torch.int32, device=dev)
    out = torch.empty(8, dtype=torch.float32, device=dev)
    assert binding.mars_score_chunk(case.model, case.kv, [0], [8], tok, tgt, 0.0, out) == 1
    assert binding.mars_score_chunk(case.model, case.kv, [0], [8], tok, None, 1.0, out) == 1
    assert binding.mars_score_chunk(case.model, case.kv, [3], [8], tok, tgt, 1.0, out) == 6
    assert binding.mars_score_chunk(case.model, case.kv, [0], [17], tok, tgt, 1.0, out) == 1     # above max_prefill_tokens
    assert case.kv.seq_len(0) == 5
    tgt[2] = model["vocab"]                                    # reported through the status word, not by a fault
    assert binding.mars_score_chunk(case.model, case.kv, [0], [8], tok, tgt, 1.0, out) == 0
    assert case.model.poll_status() == 7 and case.model.poll_status() == 0
    assert (out.cpu() == 0).all() and case.kv.seq_len(0) == 13
