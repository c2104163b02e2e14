"""Parity at the full sizes of the benchmark configurations (48 layers, vocabulary 151936), in the
launch configuration that bench.py times.  Sequences are independent inside a step, so the CPU
oracle checks a SUBSET of the batch: it is streamed one layer at a time (that layer's weights and
the subset's cache pages are copied from the device tensors the generator filled), with the GPU's
routing forced as the cascade rule prescribes.
"""
import pytest
import torch

import oracle
from harness import compare_sampled, compare_step
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
    def __init__(self, cfg, weights, steps, seed=0):
        self.cfg, self.model, self.ps = cfg, cfg["model"], cfg["page_size"]
        self.weights = weights
        self.ctx, _ = wl.make_context_lengths(cfg, seed=seed)
        self.B = len(self.ctx)
        cap = [c + steps + 1 for c in self.ctx]
        self.n_pages = sum(wl.pages_needed(c, self.ps) for c in cap) + 4
        self.max_pages = max(wl.pages_needed(c, self.ps) for c in cap) + 1
        self.pages = wl.make_page_assignment(cap, self.ps, self.n_pages, seed=seed)
        self.k_pool, self.v_pool = wl.make_kv_pools(self.model, self.n_pages, self.ps, seed=seed, device=DEV)
        self.m = binding.Model(self.model, weights, max_decode_seqs=self.B, max_pos=max(cap) + 8)
        self.kv = binding.KvCache(self.m, self.k_pool, self.v_pool, self.ps, self.B, self.max_pages)
        for b in range(self.B):
            self.kv.seq_adopt(b, self.pages[b], self.ctx[b])
        self.cur = list(self.ctx)

    def gpu_step(self, tokens, sampling, step, seed):
        L, H, k, V, n = self.model["n_layers"], self.model["hidden"], self.model["top_k"], self.model["vocab"], self.B
        out = dict(tokens=torch.empty(n, dtype=torch.int32, device=DEV), logp=torch.empty(n, device=DEV),
                   logits=torch.empty(n, V, device=DEV), hidden=torch.empty(L + 1, n, H, device=DEV),
                   router_w=torch.empty(L, n, k, device=DEV),
                   router_idx=torch.empty(L, n, k, dtype=torch.int32, device=DEV),
                   nucleus_mass=torch.empty(n, device=DEV))
        dbg = binding.make_debug(out["logits"], out["hidden"], out["router_w"], out["router_idx"], None,
                                 out["nucleus_mass"])
        smp = binding.make_sampling(seed=seed, step=step, **sampling)
        st = binding.mars_decode_step(self.m, self.kv, list(range(n)), tokens.to(DEV), smp, out["tokens"], out["logp"], dbg)
        assert st == 0 and self.m.poll_status() == 0
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
        logits = oracle.lm_head(ocfg.__class__(**model), self.weights["final_norm"].cpu(), self.weights["lm_head"].cpu(), x)
        return dict(hidden=torch.stack(hidden), router_idx=torch.stack(ridx), router_w=torch.stack(rw),
                    router_probs=torch.stack(rp), logits=logits)


def take(gpu, subset):
    idx = torch.tensor(subset)
    return dict(tokens=gpu["tokens"].cpu()[idx], logp=gpu["logp"].cpu()[idx], logits=gpu["logits"][idx.to(DEV)].cpu(),
                hidden=gpu["hidden"][:, idx.to(DEV)].cpu(), router_w=gpu["router_w"][:, idx.to(DEV)].cpu(),
                router_idx=gpu["router_idx"][:, idx.to(DEV)].cpu(), nucleus_mass=gpu["nucleus_mass"].cpu()[idx])


def test_config3_full_model_decode_top_p(full_weights):
    cfg = wl.CONFIGS[3]
    case = FullCase(cfg, full_weights, steps=2)
    tokens = wl.make_tokens(case.B, cfg["model"]["vocab"], seed=0)
    smp = dict(greedy=0, temperature=1.0, top_p=0.95)
    order = sorted(range(case.B), key=lambda b: case.ctx[b])
    subset = [order[0], order[len(order) // 2], order[-1]]          # shortest, median, longest context
    for step in range(2):
        gpu = case.gpu_step(tokens, smp, step=step, seed=7)
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
    subset = [3]
    for step in range(2):
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
