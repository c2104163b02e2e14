"""Parity of the CUDA path (through the C ABI) against the CPU oracle on seeded inputs."""
import pytest
import torch

import oracle
from harness import Case, check_cache_append, compare_sampled, compare_step, prefill_and_compare
from paper_2511_11373_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

GREEDY = dict(greedy=1, temperature=1.0, top_p=1.0)


def run_and_compare(case: Case, tokens, sampling=GREEDY, label="", step=0, seed=0):
    gpu = case.gpu_decode(tokens, sampling, step=step, seed=seed)
    forced = gpu["router_idx"].contiguous()
    orc = case.oracle_decode(tokens, forced_idx=forced)
    k = case.model_shape["top_k"]
    stats = compare_step(gpu, orc, k, greedy=bool(sampling["greedy"]), label=label)
    if not sampling["greedy"]:
        stats.update(compare_sampled(gpu, orc, sampling["temperature"], sampling["top_p"], seed, step,
                                     list(range(case.B)), label))
    return gpu, orc, stats


# ------------------------------------------------------------------ config 1: tiny single layer
@pytest.mark.parametrize("qk_norm", [0, 1])
def test_config1_tiny_layer_greedy(qk_norm):
    cfg = wl.CONFIGS[1]
    model = dict(cfg["model"], qk_norm=qk_norm)
    case = Case(model, cfg["page_size"], cfg["ctx"], seed=0, gains="perturbed")
    tokens = wl.make_tokens(len(cfg["ctx"]), model["vocab"], seed=0)
    _, _, stats = run_and_compare(case, tokens, label=f"config1 qk_norm={qk_norm}")
    check_cache_append(case, cfg["ctx"])
    assert stats["routing_checked"] >= 1
    print("config1", qk_norm, stats)


def test_config1_literal_weights_unit_gains():
    cfg = wl.CONFIGS[1]
    case = Case(cfg["model"], cfg["page_size"], cfg["ctx"], seed=0, gains="ones")
    tokens = wl.make_tokens(len(cfg["ctx"]), cfg["model"]["vocab"], seed=0)
    run_and_compare(case, tokens, label="config1 literal")


# ------------------------------------------------------------------ ragged / edge contexts
def test_edge_context_lengths_and_page_sizes():
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    for ps, ctx in ((16, [0, 1, 15, 16, 63, 64, 65, 511, 512, 513, 1100]), (32, [31, 32, 700]), (64, [63, 64, 1029]),
                    (128, [127, 128, 640])):
        case = Case(model, ps, ctx, seed=3)
        tokens = wl.make_tokens(len(ctx), model["vocab"], seed=ps)
        run_and_compare(case, tokens, label=f"edge ps={ps}")
        check_cache_append(case, ctx)


def test_multi_step_decode_teacher_forced_top_p():
    model = dict(wl.MODEL_TINY, n_layers=3, qk_norm=1)
    ctx = [14, 30, 47, 200]
    steps = 6                                  # crosses page boundaries at 16 / 32 / 48
    case = Case(model, 16, ctx, seed=5, headroom=steps)
    tokens = wl.make_tokens(len(ctx), model["vocab"], seed=11)
    smp = dict(greedy=0, temperature=0.85, top_p=0.95)
    for s in range(steps):
        gpu, _, stats = run_and_compare(case, tokens, sampling=smp, label=f"step {s}", step=s, seed=1234)
        tokens = gpu["tokens"]                 # the oracle is teacher-forced with the sampled tokens
        assert (gpu["nucleus_mass"] >= 0.95 - 1e-3).all() and (gpu["nucleus_mass"] <= 1.0 + 1e-6).all()
    for b, c in enumerate(ctx):
        assert case.kv.seq_len(b) == c + steps


def test_top_p_one_and_training_temperature():
    model = dict(wl.MODEL_TINY, n_layers=1)
    case = Case(model, 16, [40, 90], seed=8)
    tokens = wl.make_tokens(2, model["vocab"], seed=2)
    gpu, _, _ = run_and_compare(case, tokens, sampling=dict(greedy=0, temperature=0.85, top_p=1.0), step=77, seed=9)
    assert torch.allclose(gpu["nucleus_mass"], torch.ones(2), atol=1e-6)


@pytest.mark.parametrize("vocab", [1021, 1022, 130])
def test_vocabulary_sizes_off_every_tile_and_vector_width(vocab):
    """Odd and tiny vocabularies: the lm_head's last weight tile is ragged, a row of logits does not
    start on a 16-byte boundary, and the sampler takes its element-wise loads."""
    model = dict(wl.MODEL_TINY, n_layers=1, vocab=vocab)
    ctx = [9, 40, 17]
    case = Case(model, 16, ctx, seed=21, headroom=3)
    tokens = wl.make_tokens(len(ctx), vocab, seed=4)
    run_and_compare(case, tokens, label=f"vocab {vocab} greedy")
    for step, smp in enumerate((dict(greedy=0, temperature=0.85, top_p=0.95), dict(greedy=0, temperature=1.7, top_p=1.0)), 1):
        gpu, _, _ = run_and_compare(case, tokens, sampling=smp, label=f"vocab {vocab} {smp}", step=step, seed=77)
        tokens = gpu["tokens"]
        assert ((gpu["tokens"] >= 0) & (gpu["tokens"] < vocab)).all()


def test_nucleus_of_one_token_and_very_low_temperature():
    """top_p so small that the nucleus is the most probable token alone, and a temperature that makes
    the distribution nearly one-hot (most weights underflow): both must return the argmax."""
    model = dict(wl.MODEL_TINY, n_layers=1)
    ctx = [33, 70]
    case = Case(model, 16, ctx, seed=22, headroom=3)
    tokens = wl.make_tokens(len(ctx), model["vocab"], seed=6)
    greedy, orc, _ = run_and_compare(case, tokens, label="reference greedy")

    def rewind():                              # the same state again, on both sides
        for b, c in enumerate(ctx):
            case.kv.seq_set_len(b, c)
            case.cur[b] = c

    rewind()
    for step, smp in enumerate((dict(greedy=0, temperature=1.0, top_p=1e-6), dict(greedy=0, temperature=0.01, top_p=0.9)), 1):
        gpu, _, _ = run_and_compare(case, tokens, sampling=smp, label=f"{smp}", step=step, seed=5)
        gap = torch.topk(orc["logits"].double(), 2, dim=-1).values
        sure = (gap[:, 0] - gap[:, 1]) >= 1e-2
        assert (gpu["tokens"][sure] == greedy["tokens"][sure]).all()
        rewind()


def test_sampling_distribution_matches_oracle_probabilities():
    """Many draws from one fixed state (the context length is reset between steps): token-id bins
    are hit in proportion to the oracle's nucleus probabilities."""
    model = dict(wl.MODEL_TINY, n_layers=1)
    case = Case(model, 16, [33], seed=4)
    tok = wl.make_tokens(1, model["vocab"], seed=3)
    T, p, n_draw, bins = 0.7, 0.9, 3000, 16
    orc = case.oracle_decode(tok)
    pi = torch.softmax(orc["logits"][0].double() / T, 0)
    S = oracle.sample(orc["logits"][0].contiguous(), T, p, False, 0.5, want_set=True)["in_nucleus"].bool()
    target = torch.where(S, pi, torch.zeros_like(pi))
    target = (target / target.sum()).view(bins, -1).sum(1)
    dev = case.device
    out_t = torch.empty(1, dtype=torch.int32, device=dev)
    out_l = torch.empty(1, dtype=torch.float32, device=dev)
    tok_d = tok.to(dev)
    draws = torch.empty(n_draw, dtype=torch.int32, device=dev)
    for s in range(n_draw):
        case.kv.seq_set_len(0, 33)
        smp = binding.make_sampling(greedy=0, temperature=T, top_p=p, seed=21, step=s)
        assert binding.mars_decode_step(case.model, case.kv, [0], tok_d, smp, out_t, out_l) == 0
        draws[s] = out_t[0]
    torch.cuda.synchronize()
    d = draws.cpu().long()
    counts = torch.bincount(d // (model["vocab"] // bins), minlength=bins).double()
    chi2 = float(((counts - target * n_draw) ** 2 / (target * n_draw)).sum())
    assert chi2 < (bins - 1) + 5 * (2 * (bins - 1)) ** 0.5 + 5, chi2


# ------------------------------------------------------------------ invariances on the GPU
def test_page_permutation_and_batch_order_do_not_change_results():
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    ctx = [70, 19, 300]
    tokens = wl.make_tokens(3, model["vocab"], seed=1)
    a = Case(model, 16, ctx, seed=7)
    ga = a.gpu_decode(tokens, GREEDY)
    b = Case(model, 16, ctx, seed=7)
    order = [2, 0, 1]
    gb = b.gpu_decode(tokens[order], GREEDY, seq_ids=order)
    assert torch.equal(ga["logits"][order], gb["logits"]) and torch.equal(ga["tokens"][order], gb["tokens"])
    # same cache content under a different physical page assignment
    c = Case(model, 16, ctx, seed=7)
    perm = torch.randperm(c.n_pages, generator=torch.Generator().manual_seed(1))
    inv = torch.argsort(perm)
    for s in range(3):
        c.kv.seq_release(s)
    c.k_pool.copy_(c.k_pool[:, perm.to(c.device)].clone())
    c.v_pool.copy_(c.v_pool[:, perm.to(c.device)].clone())
    for s in range(3):
        c.kv.seq_adopt(s, [int(inv[p]) for p in c.pages[s]], ctx[s])
    gc = c.gpu_decode(tokens, GREEDY)
    assert torch.equal(ga["logits"], gc["logits"])


# ------------------------------------------------------------------ config 2: one full-size layer
def test_config2_one_qwen3_layer_decode():
    cfg = wl.CONFIGS[2]
    ctx, _ = wl.make_context_lengths(cfg, seed=0)
    case = Case(cfg["model"], cfg["page_size"], ctx, seed=0, gains="perturbed", poison=False)
    tokens = wl.make_tokens(len(ctx), cfg["model"]["vocab"], seed=0)
    _, _, stats = run_and_compare(case, tokens, label="config2")
    print("config2", stats)
    assert stats["routing_checked"] >= 16 and stats["routing_equal"] >= 0.9 * stats["routing_total"]
    act = case.model.active_experts()
    assert 100 <= int(act[0]) <= 128


# ------------------------------------------------------------------ chunked prefill
def test_prefill_chunks_then_decode_match_oracle():
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    ps = 16
    case = Case(model, ps, [0, 37], seed=9, headroom=80, max_prefill_tokens=128, poison=False)
    dev = case.device
    L, H, k, V = model["n_layers"], model["hidden"], model["top_k"], model["vocab"]
    lens = [50, 23]
    toks = wl.make_tokens(sum(lens), V, seed=12)
    n = sum(lens)
    out_t = torch.empty(2, dtype=torch.int32, device=dev)
    out_l = torch.empty(2, dtype=torch.float32, device=dev)
    logits = torch.empty(2, V, dtype=torch.float32, device=dev)
    hidden = torch.empty(L + 1, n, H, dtype=torch.float32, device=dev)
    ridx = torch.empty(L, n, k, dtype=torch.int32, device=dev)
    rw = torch.empty(L, n, k, dtype=torch.float32, device=dev)
    dbg = binding.make_debug(logits, hidden, rw, ridx)
    smp = binding.make_sampling(greedy=1)
    st = binding.mars_prefill_chunk(case.model, case.kv, [0, 1], lens, toks.to(dev), [1, 1], smp, out_t, out_l, dbg)
    assert st == 0 and case.model.poll_status() == 0
    seq = torch.tensor([0] * lens[0] + [1] * lens[1], dtype=torch.int32)
    pos = torch.tensor(list(range(0, lens[0])) + list(range(37, 37 + lens[1])), dtype=torch.int32)
    orc = oracle.forward(case.ocfg, case.w_cpu, toks, seq, pos, case.k_cpu, case.v_cpu, case.bt, ps,
                         forced_idx=ridx.cpu().contiguous())
    last = torch.tensor([lens[0] - 1, n - 1])
    gpu = dict(router_idx=ridx.cpu(), router_w=rw.cpu(), hidden=hidden.cpu(), logits=logits.cpu(), tokens=out_t.cpu(),
               logp=out_l.cpu())
    orc_cmp = dict(orc, logits=orc["logits"][last])
    stats = compare_step(gpu, orc_cmp, k, greedy=True, label="prefill")
    print("prefill", stats)
    assert case.kv.seq_len(0) == 50 and case.kv.seq_len(1) == 60
    # continue with a decode step on top of the prefilled cache
    case.cur = [50, 60]
    run_and_compare(case, out_t.cpu(), label="decode after prefill")


# ------------------------------------------------------------------ host-side failure paths (no GPU fault)
def test_error_paths_leave_state_unchanged():
    model = dict(wl.MODEL_TINY, n_layers=1)
    case = Case(model, 16, [16, 5], seed=2, headroom=0, spare_pages=0, extra_seqs=1)   # seq 0 needs a new page
    dev = case.device
    tok = wl.make_tokens(2, model["vocab"], seed=1).to(dev)
    out_t = torch.empty(2, dtype=torch.int32, device=dev)
    out_l = torch.empty(2, dtype=torch.float32, device=dev)
    smp = binding.make_sampling(greedy=1)
    assert case.kv.free_pages == 0
    assert binding.mars_decode_step(case.model, case.kv, [0, 1], tok, smp, out_t, out_l) == 4      # KV_FULL
    assert case.kv.seq_len(0) == 16 and case.kv.seq_len(1) == 5
    assert binding.mars_decode_step(case.model, case.kv, [1, 1], tok, smp, out_t, out_l) == 6      # duplicate slot
    assert binding.mars_decode_step(case.model, case.kv, [1, 2], tok, smp, out_t, out_l) == 6      # unused slot
    assert binding.mars_decode_step(case.model, case.kv, [0, 1, 1], tok, smp, out_t, out_l) == 1   # too many
    bad = binding.make_sampling(greedy=0, temperature=0.0, top_p=0.9)
    assert binding.mars_decode_step(case.model, case.kv, [1], tok, bad, out_t, out_l) == 1
    with pytest.raises(binding.MarsError):
        case.kv.seq_adopt(2, [case.pages[0][0]], 1)                                                # page owned
    with pytest.raises(binding.MarsError):
        case.kv.seq_release(2)                                                                     # never used
    # an out-of-range token id is reported through the status word, not by a fault
    big = torch.tensor([model["vocab"] + 5], dtype=torch.int32, device=dev)
    assert binding.mars_decode_step(case.model, case.kv, [1], big, smp, out_t, out_l) == 0
    assert case.model.poll_status() == 7
    assert case.model.poll_status() == 0
    # releasing makes room again
    case.kv.seq_release(1)
    assert binding.mars_decode_step(case.model, case.kv, [0], tok, smp, out_t, out_l) == 0
    assert case.model.poll_status() == 0 and case.kv.seq_len(0) == 17


def test_bounded_wait_gives_up_and_the_handle_stays_usable():
    """Every TMA / tensor-core wait is bounded; when its limit is reached the kernel sets the timeout
    bit, frees its tensor memory and returns.  The library's self-test block takes that path with an
    arrival that never comes: the status is MARS_ERR_TIMEOUT once, then clear, and a decode step on the
    same handle still matches the oracle.  Nothing hangs, traps or faults."""
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    case = Case(model, 16, [20, 77], seed=12)
    assert case.model.bounded_wait_selftest(arrive=True) == 0
    assert case.model.poll_status() == 0                     # the arrival came: nothing to report
    assert case.model.bounded_wait_selftest(arrive=False) == 0
    assert case.model.poll_status() == 5                     # the wait ran out
    assert case.model.poll_status() == 0                     # reading clears the word
    tokens = wl.make_tokens(2, model["vocab"], seed=6)
    run_and_compare(case, tokens, label="decode after a timed-out wait")
    check_cache_append(case, [20, 77])


def test_library_allocator_path_matches_adopted_pages():
    """Pages handed out by the library's own free list give the same results as caller-chosen ones."""
    model = dict(wl.MODEL_TINY, n_layers=1)
    ctx = [45, 16]
    a = Case(model, 16, ctx, seed=6, poison=False)
    tokens = wl.make_tokens(2, model["vocab"], seed=4)
    ga = a.gpu_decode(tokens, GREEDY)
    b = Case(model, 16, ctx, seed=6, poison=False)
    saved_k, saved_v = b.k_pool.clone(), b.v_pool.clone()
    old = [list(p) for p in b.pages]
    for s in range(2):
        b.kv.seq_release(s)
    for s in range(2):
        b.kv.seq_reserve(s, ctx[s])            # the decode step itself must grab the page for position 16
        new = b.kv.block_table(s)
        for i, p in enumerate(new):
            b.k_pool[:, p] = saved_k[:, old[s][i]]
            b.v_pool[:, p] = saved_v[:, old[s][i]]
        b.kv.seq_set_len(s, ctx[s])
    gb = b.gpu_decode(tokens, GREEDY)
    assert torch.equal(ga["logits"], gb["logits"])
    assert len(b.kv.block_table(1)) == 2


def test_prefill_small_chunks_use_the_causal_kernel():
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    case, toks = prefill_and_compare(model, 16, [0, 21, 64], [10, 5, 33], seed=21, label="prefill-small")
    run_and_compare(case, toks, label="decode after small prefill")


def test_prefill_many_tokens_tensor_core_path():
    """More than 64 token rows: QKV, output projection and the experts run on tcgen05 (several
    128-row tiles, several groups per expert), attention on the causal block kernel; chunks continue
    contexts that end inside a page, at a page boundary and at zero."""
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    case, toks = prefill_and_compare(model, 16, [0, 37, 512, 129], [300, 150, 70, 1], seed=22, label="prefill-large")
    run_and_compare(case, toks, label="decode after large prefill")


def test_prefill_with_thousands_of_tokens_uses_the_multi_block_permutation():
    """From 4096 (token, expert) pairs on, the expert slots are counted and handed out by many blocks
    (which slot a pair gets then depends on scheduling; the results must not)."""
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    prefill_and_compare(model, 32, [0, 10, 40], [1300, 640, 310], seed=27, label="prefill-2250")


MODEL_GQA8 = dict(n_layers=2, hidden=512, n_q_heads=16, n_kv_heads=2, head_dim=128, n_experts=8, top_k=2, expert_inter=128,
                  vocab=1024, qk_norm=1, rope_theta=1e6, rms_eps=1e-6)


@pytest.mark.parametrize("ps", [16, 64, 128])
def test_prefill_attention_on_tensor_cores(ps):
    """head_dim 128 with 8 query heads per KV head: the causal attention of a prefill-sized call runs
    on tcgen05 (blocks of 16 prompt tokens x 8 heads = 128 accumulator rows, 64-token key tiles).
    Chunks start at position 0, inside a page and on a page boundary; lengths leave ragged last
    blocks (70 = 4 x 16 + 6) and ragged last key tiles; one chunk is a single token."""
    case, toks = prefill_and_compare(MODEL_GQA8, ps, [0, 21, 128, 300, 64], [70, 33, 150, 1, 64], seed=24 + ps,
                                     label=f"prefill-tcgen05-attention ps={ps}")
    run_and_compare(case, toks, label="decode after tcgen05 prefill attention")


def test_prefill_tensor_core_path_at_the_full_layer_shape():
    """The dense tcgen05 path at the shape it runs in the mixed benchmark (hidden 2048, 32 / 4 heads of
    128, 128 experts top-8, expert_inter 768, per-head norm on, perturbed gains) with more than 256
    token rows in one call: the QKV contraction with norm, RoPE and cache append in its epilogue over
    20 column tiles, the output projection (8 tiles), the router logits as a contraction, the grouped
    gate/up (6 tiles) and down (8 tiles) contractions with groups of every expert id, the causal
    attention on tcgen05 and, from 4096 (token, expert) pairs on, the multi-block permutation.
    Chunks continue contexts that start at 0, inside a page, on a page boundary and at a single
    token; every tap and every appended cache row is compared with the oracle."""
    case, toks = prefill_and_compare(wl.MODEL_LAYER, 64, [0, 37, 512, 129], [300, 150, 70, 1], seed=61,
                                     label="prefill-full-shape-521")
    assert len(set(case.last_gpu["router_idx"].flatten().tolist())) == wl.MODEL_LAYER["n_experts"]
    run_and_compare(case, toks, label="decode after the full-shape prefill")
    # 4096 pairs and more: the expert slots are counted and handed out by many blocks
    prefill_and_compare(wl.MODEL_LAYER, 64, [0, 64], [400, 240], seed=62, label="prefill-full-shape-640")


def test_activation_planes_of_large_calls_can_be_switched():
    """mars_set_prefill_lo_planes: the default and the all-planes setting (and one in between) stay inside
    the tolerances on a tensor-core-sized call, all planes give a smaller hidden-state error than the
    default (experts on the hi plane), and a mask outside the defined bits is refused.  (With no lo
    plane at all the router weights leave their tolerance, which is why the default keeps three.)"""
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=64)
    err = {}
    for mask in (binding.MARS_LO_ALL, binding.MARS_LO_DEFAULT | binding.MARS_LO_DOWN, binding.MARS_LO_DEFAULT):
        case, _ = prefill_and_compare(model, 16, [0, 21], [200, 130], seed=41, label=f"lo planes {mask}", check_rows="ends",
                                      lo_planes=mask)
        err[mask] = case.stats["hidden_rel_max"]
    assert err[binding.MARS_LO_ALL] < err[binding.MARS_LO_DEFAULT]
    lib = binding.lib()
    assert lib.mars_set_prefill_lo_planes(case.model.handle, 32) == binding.MARS_ERR_INVALID_ARG
    assert lib.mars_set_prefill_lo_planes(case.model.handle, -1) == binding.MARS_ERR_INVALID_ARG


def test_prefill_in_two_calls_equals_one_call():
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=0)
    V = model["vocab"]
    toks = wl.make_tokens(200, V, seed=77)
    res = []
    for split in ((200,), (90, 110)):
        case = Case(model, 32, [11], seed=23, headroom=210, max_prefill_tokens=200, poison=False)
        dev = case.device
        out_t = torch.empty(1, dtype=torch.int32, device=dev)
        out_l = torch.empty(1, dtype=torch.float32, device=dev)
        logits = torch.empty(1, V, dtype=torch.float32, device=dev)
        at = 0
        for n in split:
            st = binding.mars_prefill_chunk(case.model, case.kv, [0], [n], toks[at:at + n].to(dev), [1],
                                            binding.make_sampling(greedy=1), out_t, out_l, binding.make_debug(logits))
            assert st == 0 and case.model.poll_status() == 0
            at += n
        res.append((logits.cpu(), int(out_t[0])))
    assert (res[0][0] - res[1][0]).abs().max() < 1e-3 and res[0][1] == res[1][1]


@pytest.mark.parametrize("n_seq", [70, 150, 256, 260])
def test_decode_with_more_than_64_sequences(n_seq):
    """65 to 256 decode rows keep the weight-streaming kernels (swap-AB projections with 128 or 256 token
    columns, streaming experts with up to 16 tokens per group); beyond 256 rows the dense projections,
    the lm_head and the experts move to the 128-row tensor-core tiles.  Results must not change."""
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    ctx = [5 + (7 * i) % 300 for i in range(n_seq)]
    case = Case(model, 16, ctx, seed=31)
    tokens = wl.make_tokens(len(ctx), model["vocab"], seed=8)
    _, _, stats = run_and_compare(case, tokens, sampling=dict(greedy=0, temperature=0.85, top_p=0.95), step=3, seed=5,
                                  label=f"decode-{n_seq}")
    print(f"decode-{n_seq}", stats)
    check_cache_append(case, ctx)
