"""Decode rows that share a cached prefix (members of a rollout group forked from one prompt, Section
3.3: a group of outputs continues one common input) read that prefix once per block of rows.  Checked
against the CPU oracle, which knows nothing of sharing (it just follows every row's block table), and
against the same step with the grouping switched off."""
import pytest
import torch

from harness import Case, compare_sampled, compare_step
from paper_2511_11373_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

MODEL_D128 = dict(n_layers=1, hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, n_experts=8, top_k=2, expert_inter=128,
                  vocab=1024, qk_norm=1, rope_theta=1e6, rms_eps=1e-6)


class ForkedCase(Case):
    """A Case whose extra sequence slots are filled by forks; keeps the oracle's block table, context
    lengths and CPU pools in step with what the library does on the device."""

    def fork(self, src: int, dst: int):
        assert self.kv.seq_fork(src, dst) == 0
        torch.cuda.synchronize()
        while len(self.cur) <= dst:
            self.cur.append(0)
        self.cur[dst] = self.cur[src]
        if self.cur[src] % self.ps:                       # the partly filled page was copied into a fresh page
            a, b = self.kv.block_table(src)[self.cur[src] // self.ps], self.kv.block_table(dst)[-1]
            assert a != b
            self.k_cpu[:, b] = self.k_cpu[:, a]
            self.v_cpu[:, b] = self.v_cpu[:, a]

    def sync_block_table(self, slots):
        """Pages that the last step took from the free list enter the oracle's block table."""
        rows = max(max(slots) + 1, self.bt.shape[0])
        bt = torch.zeros(rows, self.max_pages, dtype=torch.int32)
        bt[: self.bt.shape[0]] = self.bt
        for s in slots:
            pg = self.kv.block_table(s)
            bt[s, : len(pg)] = torch.tensor(pg, dtype=torch.int32)
        self.bt = bt


def build(model, ps, ctx, forks, share, seed, headroom, spare, later_forks=0):
    case = ForkedCase(model, ps, ctx, seed=seed, headroom=headroom, spare_pages=spare,
                      extra_seqs=len(forks) + later_forks, max_decode=len(ctx) + len(forks) + later_forks)
    case.kv.share_reads(share)
    for src, dst in forks:
        case.fork(src, dst)
    return case


def step_both(shared, plain, ids, tokens, smp, step, seed, label):
    """One decode step on the grouped and on the per-row cache; oracle parity of the grouped one."""
    g = shared.gpu_decode(tokens, smp, seq_ids=ids, step=step, seed=seed)
    u = plain.gpu_decode(tokens, smp, seq_ids=ids, step=step, seed=seed)
    shared.sync_block_table(ids)
    for b in ids:
        plain.cur[b] += 1
    orc = shared.oracle_decode(tokens, forced_idx=g["router_idx"].contiguous(), seq_ids=ids)
    stats = compare_step(g, orc, shared.model_shape["top_k"], greedy=bool(smp["greedy"]), label=label)
    if not smp["greedy"]:
        stats.update(compare_sampled(g, orc, smp["temperature"], smp["top_p"], seed, step, ids, label))
    # grouped against per-row reading: same function, other summation order
    assert torch.equal(g["router_idx"], u["router_idx"]), label
    stats["vs_per_row_logits"] = float((g["logits"] - u["logits"]).abs().max())
    stats["vs_per_row_hidden"] = float(((g["hidden"] - u["hidden"]).norm(dim=-1) / u["hidden"].norm(dim=-1)).max())
    assert stats["vs_per_row_logits"] <= 1e-3 and stats["vs_per_row_hidden"] <= 1e-4, (label, stats)
    return g, stats


def test_group_members_read_the_prompt_once_and_match_the_oracle():
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    ps, ctx = 16, [300, 77, 150]                            # 300 = 18 full pages + 12 tokens
    forks = [(0, s) for s in range(3, 9)] + [(2, 9)]        # a group of 7 (blocks of 4 + 3 rows) and a pair
    shared = build(model, ps, ctx, forks, True, seed=61, headroom=8, spare=40, later_forks=1)
    plain = build(model, ps, ctx, forks, False, seed=61, headroom=8, spare=40, later_forks=1)
    ids = [3, 1, 0, 9, 5, 2, 4, 8, 6, 7]                    # members scattered over the batch, one loner (slot 1)
    smp = dict(greedy=0, temperature=0.85, top_p=0.95)
    V = model["vocab"]
    tokens = wl.make_tokens(len(ids), V, seed=5)
    for step in range(5):
        g, stats = step_both(shared, plain, ids, tokens, smp, step, 77, f"group step {step}")
        info_s, info_p = shared.model.last_step_info(), plain.model.last_step_info()
        assert info_p["kv_tokens_streamed"] == info_p["kv_tokens_read"] == info_s["kv_tokens_read"]
        # 288 shared tokens: 7 (later 8) rows read them in 2 blocks; 144 shared tokens: 2 rows in 1 block
        members = 7 if step <= 2 else 8
        assert info_s["kv_tokens_streamed"] == info_s["kv_tokens_read"] - (members - 2) * 288 - (2 - 1) * 144
        print("shared-prefix", step, stats, info_s)
        tokens = g["tokens"]                                # members diverge from the first step on
        if step == 2:                                       # a member forks again: fork of a fork joins the group
            for c in (shared, plain):
                c.fork(3, 10)
            ids = ids + [10]
            tokens = torch.cat([tokens, tokens[:1]])
    assert shared.model.last_step_info()["kv_tokens_streamed"] < shared.model.last_step_info()["kv_tokens_read"]
    for s in ids:
        shared.kv.seq_release(s)
    assert shared.kv.free_pages == shared.kv.num_pages


def test_head_dim_128_pages_of_64_and_two_shared_spans():
    ps, ctx = 64, [1500, 70]                                # 23 full pages = 1472 shared tokens: spans of 1024 + 448
    forks = [(0, s) for s in range(2, 7)]                   # group of 6: blocks of 4 + 2 rows
    shared = build(MODEL_D128, ps, ctx, forks, True, seed=62, headroom=4, spare=12)
    plain = build(MODEL_D128, ps, ctx, forks, False, seed=62, headroom=4, spare=12)
    ids = [0, 2, 3, 1, 4, 5, 6]
    tokens = wl.make_tokens(len(ids), MODEL_D128["vocab"], seed=6)
    for step in range(2):
        g, stats = step_both(shared, plain, ids, tokens, dict(greedy=1, temperature=1.0, top_p=1.0), step, 0,
                             f"d128 step {step}")
        info = shared.model.last_step_info()
        assert info["kv_tokens_streamed"] == info["kv_tokens_read"] - (6 - 2) * 1472
        print("shared-prefix d128", step, stats, info)
        tokens = g["tokens"]


MODEL_GQA8 = dict(n_layers=2, hidden=512, n_q_heads=16, n_kv_heads=2, head_dim=128, n_experts=8, top_k=2, expert_inter=128,
                  vocab=1024, qk_norm=1, rope_theta=1e6, rms_eps=1e-6)


@pytest.mark.parametrize("ps", [16, 64])
def test_groups_on_the_tensor_core_kernel(ps):
    """head_dim 128 with 8 query heads per KV head: the shared spans run on tcgen05, up to 16 member rows x
    8 heads as the 128 accumulator rows of one pass over the keys.  A group of 18 members (blocks of
    16 + 2 rows) whose prompt spans two spans (1024 + 256 tokens, plus a partly filled page that is
    copied per member), a pair with a short prompt, and a loner."""
    ctx = [1290, 200, 77]
    forks = [(0, s) for s in range(3, 20)] + [(1, 20)]
    shared = build(MODEL_GQA8, ps, ctx, forks, True, seed=65 + ps, headroom=4, spare=40)
    plain = build(MODEL_GQA8, ps, ctx, forks, False, seed=65 + ps, headroom=4, spare=40)
    ids = [7, 2, 0, 20] + [s for s in range(3, 20) if s != 7] + [1]
    tokens = wl.make_tokens(len(ids), MODEL_GQA8["vocab"], seed=9)
    big = (1290 // ps) * ps                                  # whole pages of the long prompt
    small = (200 // ps) * ps
    smp = dict(greedy=0, temperature=0.85, top_p=0.95)
    for step in range(3):
        g, stats = step_both(shared, plain, ids, tokens, smp, step, 11, f"tcgen05 groups ps={ps} step {step}")
        info = shared.model.last_step_info()
        assert info["kv_tokens_streamed"] == info["kv_tokens_read"] - (18 - 2) * big - (2 - 1) * small
        print("shared-prefix tcgen05", ps, step, stats, info)
        tokens = g["tokens"]


def test_short_common_prefix_and_single_rows_take_the_per_row_path():
    model = dict(wl.MODEL_TINY, n_layers=1)
    shared = build(model, 16, [100, 200], [(0, 2)], True, seed=63, headroom=4, spare=8)   # 96 shared tokens < 128
    tokens = wl.make_tokens(3, model["vocab"], seed=1)
    shared.gpu_decode(tokens, dict(greedy=1, temperature=1.0, top_p=1.0), seq_ids=[0, 1, 2])
    info = shared.model.last_step_info()
    assert info["kv_tokens_streamed"] == info["kv_tokens_read"]
    # a group member decoded alone has nobody to share with
    big = build(model, 16, [200], [(0, 1)], True, seed=64, headroom=4, spare=8)
    big.gpu_decode(tokens[:1], dict(greedy=1, temperature=1.0, top_p=1.0), seq_ids=[1])
    info = big.model.last_step_info()
    assert info["kv_tokens_streamed"] == info["kv_tokens_read"] == 201
    assert binding.lib().mars_kv_share_reads(None, 1) == 6
