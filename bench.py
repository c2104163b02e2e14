"""Benchmark of the rollout step: decode tokens/s on a Qwen3-30B-A3B-shaped MoE and the fraction of
the HBM roofline it reaches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 2|3|4|5|6|7|8] [--impl reference]

One "step" is one pass of the whole hot path (embedding, 48 x {QKV+RoPE+append, paged attention,
output projection, router, experts, combine}, lm_head, sampling) over the batch.  Inputs are
synthetic and seeded (random-init bf16 weights, N(0,1) cache, uniform tokens); every step streams far
more than the L2 holds (tens of GB), so no L2 flush is needed between timed steps.

With N > 1 (torchrun) every rank runs an independent replica of the same workload on its own GPU:
sequences are independent, there is no collective on the data path, and the reported value is the
sum over replicas divided by the slowest rank's time ("replicas only", weak scaling).

`--impl reference` times the CPU oracle (test infrastructure, plain C, as it stands) on a bounded
sample of the same workload on the host cores; it is a deliberately slow baseline.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2511_11373_b200 import workloads as wl  # noqa: E402

METRIC = "decode_tokens_per_sec"
UNIT = "tokens/s"
PEAKS_FALLBACK = dict(hbm_gbs=6650.0, source="fallback")
# (dram__bytes_read.sum + dram__bytes_write.sum) / algorithmic bytes of the captured launch, per kernel class.
# Set an entry to None (or delete it) when that kernel changes after the capture.
NCU_TRAFFIC_RATIO = {"attn": (1206.248e6 + 7.596e6) / 1201.844e6,     # attn_decode_kernel<128>, 586 166 cached tokens
                     "gate_up": (795.297e6 + 5.104e6) / 786.432e6,      # expert_gate_up_kernel, 125 experts
                     "down": (397.981e6 + 5.244e6) / 393.216e6}         # expert_down_kernel


def load_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), source="measured")
    return dict(PEAKS_FALLBACK)


# ----------------------------------------------------------------------------------- clocks sampler
CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


class ClockSampler:
    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={CLOCK_QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "200"], stdout=self.tmp,
                                         stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self) -> dict:
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        rows = [l.strip().split(", ") for l in open(self.tmp.name) if l.strip()]
        os.unlink(self.tmp.name)
        clocks, reasons, smax = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                clocks.append(float(r[1])); smax = float(r[2])
            except ValueError:
                continue
            for name, val in zip(names, r[5:9]):
                if val.strip().lower() == "active":
                    reasons.add(name)
        if clocks:
            out.update(sm_mhz=statistics.median(clocks), sm_max_mhz=smax, reasons=sorted(reasons), samples=len(clocks))
        return out


# ----------------------------------------------------------------------------------- workload set-up
def algorithmic_bytes(model: dict, kv_tokens: int, active_per_layer, n_lm_rows: int = 1) -> dict:
    """Bytes one decode step must move: attention + router weights, the weights of the experts that
    were actually selected, the cached keys/values read, and the lm_head (all bf16)."""
    H, nq, nkv, D = model["hidden"], model["n_q_heads"], model["n_kv_heads"], model["head_dim"]
    E, I, V, L = model["n_experts"], model["expert_inter"], model["vocab"], model["n_layers"]
    w_attn = (H * (nq + 2 * nkv) * D + nq * D * H) * 2
    w_router = E * H * 2
    w_expert = 3 * H * I * 2
    kv = 2 * nkv * D * 2 * kv_tokens * L
    experts = sum(int(a) for a in active_per_layer) * w_expert
    lm = V * H * 2
    return dict(attn_router=L * (w_attn + w_router), experts=experts, kv=kv, lm_head=lm,
                total=L * (w_attn + w_router) + experts + kv + lm, w_expert=w_expert)


class DecodeWorkload:
    """Builds a config (weights, cache, page tables) on one GPU and steps it through the C ABI."""

    def __init__(self, cfg: dict, total_steps: int, device: torch.device, seed: int = 0, prefill_reqs: int = 0,
                 prefill_chunk: int = 0, weights: dict | None = None):
        from paper_2511_11373_b200 import binding
        self.binding = binding
        self.cfg, self.device = cfg, device
        model, ps = cfg["model"], cfg["page_size"]
        self.model_shape = model
        # the uniform context draw of configs 2 / 3 uses the seed whose total is closest to its expectation
        ctx_seed = wl.CONFIG3_CONTEXT_SEED if "ctx_range" in cfg else seed
        self.ctx, self.stages = wl.make_context_lengths(cfg, seed=ctx_seed)
        B = len(self.ctx)
        self.B = B
        cap = [c + total_steps + 1 for c in self.ctx]
        n_pages = sum(wl.pages_needed(c, ps) for c in cap) + 8 + prefill_reqs * (wl.pages_needed(prefill_chunk, ps) + 1)
        max_pages = max(wl.pages_needed(c, ps) for c in cap + [prefill_chunk]) + 1
        free, _ = torch.cuda.mem_get_info(device)
        t0 = time.time()
        self.weights = weights if weights is not None else wl.make_weights(model, seed=seed, device=device, gains="ones")
        self.k_pool, self.v_pool = wl.make_kv_pools(model, n_pages, ps, seed=seed, device=device)
        torch.cuda.synchronize(device)
        self.setup_s = time.time() - t0
        self.pages = wl.make_page_assignment(cap, ps, n_pages, seed=seed)
        # a fused mixed step carries the decode rows and the prompt rows in one call
        self.model = binding.Model(model, self.weights, max_decode_seqs=B + prefill_reqs,
                                   max_prefill_tokens=prefill_reqs * prefill_chunk + (B if prefill_reqs else 0),
                                   max_pos=max(cap + [prefill_chunk]) + 8)
        self.kv = binding.KvCache(self.model, self.k_pool, self.v_pool, ps, B + prefill_reqs, max_pages)
        for b in range(B):
            self.kv.seq_adopt(b, self.pages[b], self.ctx[b])
        self.tok_a = wl.make_tokens(B, model["vocab"], seed=seed).to(device)
        self.tok_b = torch.empty_like(self.tok_a)
        self.logp = torch.empty(B, dtype=torch.float32, device=device)
        self.step_no = 0
        s = cfg["sampling"]
        self.sampling = dict(greedy=s["greedy"], temperature=s["temperature"], top_p=s["top_p"])
        self.ids = list(range(B))
        self.mem_free_before = free

    def step(self):
        b = self.binding
        smp = b.make_sampling(seed=2025, step=self.step_no, **self.sampling)
        st = b.mars_decode_step(self.model, self.kv, self.ids, self.tok_a, smp, self.tok_b, self.logp)
        if st != 0:
            raise b.MarsError(st, "mars_decode_step")
        self.tok_a, self.tok_b = self.tok_b, self.tok_a      # the sampled tokens feed the next step
        self.step_no += 1

    def step_host(self, in_host, out_tok_host, out_lp_host):
        b = self.binding
        smp = b.make_sampling(seed=2025, step=self.step_no, **self.sampling)
        st = b.mars_decode_step_host(self.model, self.kv, self.ids, in_host, smp, out_tok_host, out_lp_host)
        if st != 0:
            raise b.MarsError(st, "mars_decode_step_host")
        self.step_no += 1

    def kv_tokens_now(self) -> int:
        return sum(self.kv.seq_len(b) for b in range(self.B))

    def release_cache(self):
        """Frees the cache pools and the library handles (the weights stay, for the next configuration)."""
        torch.cuda.synchronize(self.device)
        self.kv.close()
        self.model.close()
        del self.k_pool, self.v_pool, self.kv, self.model
        torch.cuda.empty_cache()


# ----------------------------------------------------------------------------------- CPU baseline
ORACLE_SAMPLE_SEQS = 8     # sequences of the workload that both arms' CPU-oracle figures are taken on


class OracleSample:
    """The CPU oracle, as it stands, on a bounded sample of the workload: ONE decoder layer plus the
    lm_head and sampling over the first n_seq sequences (own CPU-generated weights and cache of the
    same shapes and distributions); a full step is the layer time scaled by the number of layers."""

    def __init__(self, cfg: dict, n_seq: int, seed: int = 0):
        import oracle
        self.oracle, self.cfg = oracle, cfg
        self.model = dict(cfg["model"])
        one = dict(self.model, n_layers=1)
        ctx_all, _ = wl.make_context_lengths(cfg, seed=wl.CONFIG3_CONTEXT_SEED if "ctx_range" in cfg else seed)
        self.n_all = len(ctx_all)
        self.n_seq = min(n_seq, self.n_all)
        ctx = ctx_all[: self.n_seq]
        self.ps = cfg["page_size"]
        cap = [c + 1 for c in ctx]
        n_pages = sum(wl.pages_needed(c, self.ps) for c in cap)
        pages = wl.make_page_assignment(cap, self.ps, n_pages, seed=seed, shuffle=False)
        self.w = wl.make_weights(one, seed=seed, device="cpu", gains="ones")
        self.kp, self.vp = wl.make_kv_pools(one, n_pages, self.ps, seed=seed, device="cpu")
        self.bt = wl.block_table_tensor(pages, max(len(p) for p in pages))
        self.ocfg = oracle.Config(**one)
        self.toks = wl.make_tokens(self.n_seq, self.model["vocab"], seed=seed)
        self.seq = torch.arange(self.n_seq, dtype=torch.int32)
        self.pos = torch.tensor(ctx, dtype=torch.int32)

    def run(self) -> dict:
        o = self.oracle
        x = o.embed(self.w["embed"], self.toks)
        t0 = time.perf_counter()
        o.layer_forward(self.ocfg, self.w["layers"][0], x, self.seq, self.pos, self.kp[0], self.vp[0], self.bt, self.ps)
        t_layer = time.perf_counter() - t0
        t0 = time.perf_counter()
        logits = o.lm_head(self.ocfg, self.w["final_norm"], self.w["lm_head"], x)
        s = self.cfg["sampling"]
        for i in range(self.n_seq):
            o.sample(logits[i].contiguous(), s["temperature"], s["top_p"], bool(s["greedy"]), o.uniform(1, 0, i))
        t_head = time.perf_counter() - t0
        total = t_layer * self.model["n_layers"] + t_head
        return dict(value=self.n_seq / total, unit=UNIT, cores=os.cpu_count(), kind="oracle",
                    sample=f"{self.n_seq} of {self.n_all} sequences; one decoder layer timed ({t_layer:.2f} s) and "
                           f"scaled by {self.model['n_layers']} layers, plus lm_head+sampling ({t_head:.2f} s)",
                    seconds=t_layer + t_head)


# ----------------------------------------------------------------------------------- distributed glue
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value: float, world: int, device) -> float:
    """Max of a scalar over ranks (NCCL on GPUs, gloo on CPU); identity for one rank."""
    if world == 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


# ----------------------------------------------------------------------------------- main arms
def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    cfg = wl.CONFIGS[args.workload]
    sample = OracleSample(cfg, ORACLE_SAMPLE_SEQS)
    for _ in range(args.warmup):
        sample.run()
    t0 = time.perf_counter()
    rates = [sample.run() for _ in range(args.steps)]
    wall = time.perf_counter() - t0
    value = statistics.mean(r["value"] for r in rates)
    base = rates[-1]
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1000.0 * wall / max(args.steps, 1), higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=cfg["name"], note="CPU oracle on a bounded sample per step, extrapolated to a full step"),
                cpu_baseline=dict(value=value, unit=UNIT, cores=base["cores"], kind="oracle", sample=base["sample"]),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line))


def measure_mixed(cfg: dict, args, device, weights=None) -> dict:
    """Config 4: one chunked-prefill call (8 fresh prompts of 2048 tokens) followed by one decode step
    over 192 sequences = one mixed step.  Returns decode-only against the HBM roofline, prefill-only
    against the bf16 tensor peak, the pair, and the same work as one fused call (mars_mixed_step)."""
    from paper_2511_11373_b200 import binding
    pf = cfg["prefill"]
    w = DecodeWorkload(cfg, 3 * (args.warmup + args.steps) + 16, device, prefill_reqs=pf["requests"], prefill_chunk=pf["chunk"],
                       weights=weights)
    model = cfg["model"]
    n_pf = pf["requests"] * pf["chunk"]
    toks = wl.make_tokens(n_pf, model["vocab"], seed=1, name="prompts").to(device)
    out_t = torch.empty(pf["requests"], dtype=torch.int32, device=device)
    out_l = torch.empty(pf["requests"], dtype=torch.float32, device=device)
    ids = list(range(w.B, w.B + pf["requests"]))
    smp = binding.make_sampling(seed=3, step=0, **w.sampling)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    stream = torch.cuda.current_stream()
    # decode steps back to back (steady state of a decode-only phase)
    for _ in range(max(args.warmup, 3)):
        w.step()
    n_steady = max(args.steps, 6)
    torch.cuda.synchronize()
    clk = ClockSampler(device.index or 0)
    ev[0].record(stream)
    for _ in range(n_steady):
        w.step()
    ev[1].record(stream)
    torch.cuda.synchronize()
    clocks_decode = clk.stop()
    steady_ms = ev[0].elapsed_time(ev[1]) / n_steady
    steady_bytes = algorithmic_bytes(model, w.kv_tokens_now() - w.B * n_steady // 2, w.model.active_experts().tolist())
    t_pf, t_dec = [], []
    clk = ClockSampler(device.index or 0)
    for it in range(args.warmup + args.steps):
        for s_ in ids:
            w.kv.seq_reserve(s_, 0)
        ev[0].record(stream)
        st = binding.mars_prefill_chunk(w.model, w.kv, ids, [pf["chunk"]] * pf["requests"], toks, [1] * pf["requests"],
                                        smp, out_t, out_l)
        assert st == 0, binding.STATUS_NAMES.get(st, st)
        ev[1].record(stream)
        w.step()
        ev[2].record(stream)
        torch.cuda.synchronize()
        assert w.model.poll_status() == 0
        for s_ in ids:
            w.kv.seq_release(s_)
        if it >= args.warmup:
            t_pf.append(ev[0].elapsed_time(ev[1])); t_dec.append(ev[1].elapsed_time(ev[2]))
    clocks_alternating = clk.stop()
    # the same work as ONE call: decode rows and prompt chunks share every projection and every expert pass
    mix_t = torch.empty(w.B + pf["requests"], dtype=torch.int32, device=device)
    mix_l = torch.empty(w.B + pf["requests"], dtype=torch.float32, device=device)
    t_fused = []
    for it in range(args.warmup + args.steps):
        for s_ in ids:
            w.kv.seq_reserve(s_, 0)
        ev[0].record(stream)
        st = binding.mars_mixed_step(w.model, w.kv, w.ids, w.tok_a, ids, [pf["chunk"]] * pf["requests"], toks,
                                     [1] * pf["requests"], smp, mix_t, mix_l)
        assert st == 0, binding.STATUS_NAMES.get(st, st)
        ev[1].record(stream)
        torch.cuda.synchronize()
        assert w.model.poll_status() == 0
        for s_ in ids:
            w.kv.seq_release(s_)
        if it >= args.warmup:
            t_fused.append(ev[0].elapsed_time(ev[1]))
    fused_ms = statistics.median(t_fused)
    # per-kernel-class device time of one more prefill call
    for s_ in ids:
        w.kv.seq_reserve(s_, 0)
    w.model.profile_enable(True)
    st = binding.mars_prefill_chunk(w.model, w.kv, ids, [pf["chunk"]] * pf["requests"], toks, [1] * pf["requests"], smp,
                                    out_t, out_l)
    assert st == 0
    pf_classes = {k: round(v[0], 3) for k, v in w.model.profile_read().items() if v[1]}
    w.model.profile_enable(False)
    for s_ in ids:
        w.kv.seq_release(s_)
    active = w.model.active_experts().tolist()
    peaks = load_peaks()
    if peaks["source"] == "measured":
        mp = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        tflops_peak, tflops_sustained = mp["bf16_tflops"], mp.get("bf16_tflops_sustained")
    else:
        tflops_peak, tflops_sustained = 1590.0, 1400.0
    H, nq, nkv, D, I, L = model["hidden"], model["n_q_heads"], model["n_kv_heads"], model["head_dim"], model["expert_inter"], model["n_layers"]
    per_tok = 2 * L * (H * (nq + 2 * nkv) * D + nq * D * H + model["top_k"] * 3 * H * I + model["n_experts"] * H)
    attn = L * pf["requests"] * 4 * nq * D * pf["chunk"] * (pf["chunk"] + 1) // 2
    flops = per_tok * n_pf + attn
    pf_ms, dec_ms = statistics.median(t_pf), statistics.median(t_dec)
    dec_bytes = algorithmic_bytes(model, w.kv_tokens_now(), active)
    w.release_cache()
    return dict(metric=METRIC, value=w.B / (dec_ms / 1e3), unit=UNIT, n_gpus=1, steps=args.steps, warmup=args.warmup,
                ms_per_step=pf_ms + dec_ms, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic",
                config=dict(workload=cfg["name"], decode_seqs=w.B, prefill_requests=pf["requests"], prefill_chunk=pf["chunk"],
                            l2="inputs larger than L2"),
                decode=dict(ms=dec_ms, bytes=dec_bytes["total"], frac_of_measured_hbm=dec_bytes["total"] / (dec_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                            note="one decode step right after each prefill call", clocks=clocks_alternating),
                decode_back_to_back=dict(ms=steady_ms, tokens_per_s=w.B / (steady_ms / 1e3), bytes=steady_bytes["total"], clocks=clocks_decode,
                                         frac_of_measured_hbm=steady_bytes["total"] / (steady_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]),
                prefill=dict(ms=pf_ms, tokens_per_s=n_pf / (pf_ms / 1e3), algorithmic_tflop=flops / 1e12,
                             achieved_tflops=flops / (pf_ms * 1e-3) / 1e12, frac_of_measured_bf16=flops / (pf_ms * 1e-3) / 1e12 / tflops_peak,
                             frac_of_sustained_bf16=(flops / (pf_ms * 1e-3) / 1e12 / tflops_sustained) if tflops_sustained else None,
                             note="algorithmic flops; the QKV / output / router projections and attention run on (hi, lo) bf16 "
                                  "activation pairs and execute twice that on the tensor cores, the experts use the hi plane only; "
                                  "the call is long enough to run under the power cap, so the sustained peak is the closer bound"),
                mixed_ms=pf_ms + dec_ms, fused_mixed_step_ms=fused_ms, prefill_ms_by_class=pf_classes)


def run_mixed(args):
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    print(json.dumps(measure_mixed(wl.CONFIGS[args.workload], args, device)))


def measure_decode(cfg: dict, steps: int, warmup: int, device, weights) -> dict:
    """Decode-only timing of another configuration on the same weights (device-resident inputs, CUDA events on
    the launching stream, clocks sampled during the timed steps)."""
    w = DecodeWorkload(cfg, warmup + steps + 2, device, weights=weights)
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        w.step()
    torch.cuda.synchronize()
    kv0 = w.kv_tokens_now()
    sampler = ClockSampler(device.index or 0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        w.step()
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    assert w.model.poll_status() == 0
    ms = e0.elapsed_time(e1) / steps
    active = w.model.active_experts().tolist()
    by = algorithmic_bytes(cfg["model"], kv0 + w.B * (steps + 1) // 2, active)
    peaks = load_peaks()
    out = dict(workload=cfg["name"], batch=w.B, steps=steps, warmup=warmup, ms_per_step=ms, tokens_per_s=w.B / (ms / 1e3),
               context_tokens=kv0, bytes_per_step=by["total"], achieved_gbs=by["total"] / (ms * 1e-3) / 1e9,
               frac_of_measured_hbm=by["total"] / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
               active_experts_mean=sum(active) / len(active), clocks=clocks, setup_s=round(w.setup_s, 1))
    w.release_cache()
    return out


def run_grouped(args):
    """Grouped rollouts: G groups of M sequences, every group forked from one cached prompt (its pages
    are held once).  Times the decode step with the shared prompt read once per block of rows and,
    on the same state, with every row reading its whole context."""
    from paper_2511_11373_b200 import binding
    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    cfg = wl.CONFIGS[args.workload]
    model, ps = cfg["model"], cfg["page_size"]
    G, M, P = cfg["groups"], cfg["members"], cfg["prompt"]
    own = wl.make_group_lengths(cfg)
    total_steps = 2 * (args.warmup + args.steps) + 2
    B = G * M
    n_pages = G * wl.pages_needed(P, ps) + sum(wl.pages_needed(o + total_steps + 1, ps) + 1 for g in own for o in g) + 8
    max_pages = wl.pages_needed(P + cfg["own_range"][1] + total_steps + 1, ps) + 2
    weights = wl.make_weights(model, seed=0, device=device, gains="ones")
    k_pool, v_pool = wl.make_kv_pools(model, n_pages, ps, seed=0, device=device)
    m = binding.Model(model, weights, max_decode_seqs=B, max_prefill_tokens=0, max_pos=P + cfg["own_range"][1] + total_steps + 8)
    kv = binding.KvCache(m, k_pool, v_pool, ps, B, max_pages)
    for g in range(G):                                   # the prompt, then M - 1 forks, then everyone's own tokens
        kv.seq_reserve(g * M, P)
        kv.seq_set_len(g * M, P)
        for j in range(1, M):
            assert kv.seq_fork(g * M, g * M + j) == 0
        for j in range(M):
            kv.seq_reserve(g * M + j, P + own[g][j])
            kv.seq_set_len(g * M + j, P + own[g][j])
    ids = list(range(B))
    tok_a = wl.make_tokens(B, model["vocab"], seed=0).to(device)
    tok_b = torch.empty_like(tok_a)
    logp = torch.empty(B, dtype=torch.float32, device=device)
    stream = torch.cuda.current_stream()
    step_no = 0
    out = {}
    peaks = load_peaks()
    for label, share in (("shared", True), ("per_row", False)):
        kv.share_reads(share)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler = None
        for it in range(args.warmup + args.steps):
            if it == args.warmup:
                torch.cuda.synchronize()
                sampler = ClockSampler(0)
                e0.record(stream)
            smp = binding.make_sampling(seed=2025, step=step_no, **cfg["sampling"])
            st = binding.mars_decode_step(m, kv, ids, tok_a, smp, tok_b, logp)
            assert st == 0, binding.STATUS_NAMES.get(st, st)
            tok_a, tok_b = tok_b, tok_a
            step_no += 1
        e1.record(stream)
        torch.cuda.synchronize()
        clocks = sampler.stop()
        assert m.poll_status() == 0
        info = m.last_step_info()
        ms = e0.elapsed_time(e1) / args.steps
        active = m.active_experts().tolist()
        logical = algorithmic_bytes(model, info["kv_tokens_read"], active)
        streamed = algorithmic_bytes(model, info["kv_tokens_streamed"], active)
        out[label] = dict(ms_per_step=ms, tokens_per_s=B / (ms / 1e3), kv_tokens_read=info["kv_tokens_read"],
                          kv_tokens_streamed=info["kv_tokens_streamed"], bytes_streamed=streamed["total"],
                          frac_of_measured_hbm_streamed=streamed["total"] / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                          frac_of_measured_hbm_logical=logical["total"] / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                          launches=info["kernel_launches"], clocks=clocks)
    line = dict(metric=METRIC, value=out["shared"]["tokens_per_s"], unit=UNIT, n_gpus=1, steps=args.steps, warmup=args.warmup,
                ms_per_step=out["shared"]["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="bf16", data="synthetic",
                config=dict(workload=cfg["name"], groups=G, members=M, prompt_tokens=P, own_range=cfg["own_range"],
                            l2="inputs larger than L2"),
                clocks=out["shared"]["clocks"], gpu_launches=int(out["shared"]["launches"]) * args.steps,
                shared_prefix_read_once=out["shared"], every_row_reads_its_context=out["per_row"],
                speedup=out["per_row"]["ms_per_step"] / out["shared"]["ms_per_step"])
    print(json.dumps(line))


def run_cuda(args):
    rank, local_rank, world = dist_env()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    cfg = wl.CONFIGS[args.workload]
    e2e_steps = min(args.steps, 16)
    prof_steps = min(args.steps, 8)
    total = args.warmup + args.steps + e2e_steps + prof_steps + 4
    w = DecodeWorkload(cfg, total, device)
    model = cfg["model"]
    stream = torch.cuda.current_stream()

    for _ in range(args.warmup):
        w.step()
    torch.cuda.synchronize()
    barrier(world)
    kv_tokens_start = w.kv_tokens_now()
    sampler = ClockSampler(local_rank)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(args.steps):
        w.step()
    e1.record(stream)
    torch.cuda.synchronize()
    barrier(world)
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1), world, device)
    assert w.model.poll_status() == 0
    info = w.model.last_step_info()
    ms_per_step = ms / args.steps
    value = world * w.B * args.steps / (ms / 1000.0)

    # end to end through the host-buffer entry point (pinned host tokens in, tokens + log-probs out)
    in_host = w.tok_a.cpu().pin_memory()
    out_tok = torch.empty(w.B, dtype=torch.int32).pin_memory()
    out_lp = torch.empty(w.B, dtype=torch.float32).pin_memory()
    torch.cuda.synchronize()
    barrier(world)
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        w.step_host(in_host, out_tok, out_lp)
        in_host.copy_(out_tok)
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1000.0, world, device)
    e2e = dict(value=world * w.B * e2e_steps / (e2e_ms / 1000.0), unit=UNIT, h2d_bytes_per_step=w.B * 4,
               d2h_bytes_per_step=w.B * 8, steps=e2e_steps)

    # per-kernel-class device time over a few more steps (event pairs around every launch)
    w.tok_a.copy_(out_tok.to(device))
    w.model.profile_enable(True)
    kv_tokens_prof = w.kv_tokens_now()
    for _ in range(prof_steps):
        w.step()
    prof = w.model.profile_read()
    w.model.profile_enable(False)
    active = w.model.active_experts().tolist()

    peaks = load_peaks()
    kv_mid = kv_tokens_start + w.B * (args.steps + 1) // 2          # cached tokens read by the average timed step
    bytes_step = algorithmic_bytes(model, kv_mid, active)
    step_gbs = bytes_step["total"] / (ms_per_step * 1e-3) / 1e9
    # dominant kernel: algorithmic bytes per launch / mean launch time
    kv_prof = kv_tokens_prof + w.B * (prof_steps + 1) // 2
    per_launch = {
        "attn": 2 * model["n_kv_heads"] * model["head_dim"] * 2 * kv_prof,
        "gate_up": (sum(active) / len(active)) * 2 * model["hidden"] * model["expert_inter"] * 2,
        "down": (sum(active) / len(active)) * model["hidden"] * model["expert_inter"] * 2,
    }
    kernels = {}
    for name, (kms, n) in prof.items():
        if n:
            kernels[name] = dict(ms_per_step=kms / prof_steps, launches_per_step=n / prof_steps,
                                 us_per_launch=1000.0 * kms / n)
            if name in per_launch:
                kernels[name]["achieved_gbs"] = per_launch[name] / (kms / n * 1e-3) / 1e9
    top = max(per_launch, key=lambda k: kernels.get(k, {}).get("ms_per_step", 0.0))
    # DRAM traffic per launch: dram read + write bytes of this kernel in an ncu capture of the one-layer workload
    # (64 sequences, contexts U[1k, 16k]), as a ratio to that launch's algorithmic bytes, scaled to this launch by
    # the units processed (traffic grows in proportion to the bytes streamed)
    traffic = per_launch[top] * NCU_TRAFFIC_RATIO[top] if top in NCU_TRAFFIC_RATIO else None
    roofline = dict(bound="hbm", kernel=top, achieved=kernels[top]["achieved_gbs"], peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=kernels[top]["achieved_gbs"] / peaks["hbm_gbs"], traffic=traffic, peak_source=peaks["source"],
                    bytes_per_launch=per_launch[top], us_per_launch=kernels[top]["us_per_launch"])

    if rank != 0:
        return
    # the other full-model configurations on the same weights (one GPU, default workload only): config 5 (16 x 64k,
    # greedy) decode-only, config 4 (192 sequences + 8 x 2048 prompt tokens) decode / prefill / both / fused
    extra = {}
    if world == 1 and args.workload == 3 and not args.no_extra_configs:
        weights = w.weights
        w.release_cache()
        free, _ = torch.cuda.mem_get_info(device)
        m5 = wl.CONFIGS[5]["model"]
        need5 = 2 * m5["n_layers"] * 16 * (65536 + 128) * m5["n_kv_heads"] * m5["head_dim"] * 2 + (4 << 30)
        if free >= need5:
            extra["5"] = measure_decode(wl.CONFIGS[5], 8, 3, device, weights)
        else:
            extra["5"] = dict(skipped=f"{free >> 30} GiB free, {need5 >> 30} GiB needed")
        sub = argparse.Namespace(steps=3, warmup=2, workload=4)
        extra["4"] = measure_mixed(wl.CONFIGS[4], sub, device, weights=weights)
        for k in ("metric", "unit", "n_gpus", "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "value", "steps", "warmup"):
            extra["4"].pop(k, None)
    cpu = OracleSample(cfg, ORACLE_SAMPLE_SEQS).run()
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                data="synthetic",
                config=dict(workload=cfg["name"], batch=w.B, n_layers=model["n_layers"], page_size=cfg["page_size"],
                            context_tokens=kv_tokens_start, context_tokens_expected=len(w.ctx) * sum(cfg.get("ctx_range", (0, 0))) // 2,
                            sampling=cfg["sampling"], l2="inputs larger than L2",
                            replicas=world, setup_s=round(w.setup_s, 1)),
                clocks=clocks, e2e=e2e, gpu_launches=int(info["kernel_launches"]) * args.steps,
                roofline=roofline,
                step_roofline=dict(bytes_per_step=bytes_step["total"], experts=bytes_step["experts"], kv=bytes_step["kv"],
                                   attn_router=bytes_step["attn_router"], lm_head=bytes_step["lm_head"],
                                   achieved_gbs=step_gbs, frac_of_measured_hbm=step_gbs / peaks["hbm_gbs"],
                                   frac_of_nominal_8tbs=step_gbs / 8000.0,
                                   active_experts_mean=sum(active) / len(active)),
                kernels=kernels, cpu_baseline={k: v for k, v in cpu.items() if k != "seconds"})
    if extra:
        line["configs"] = extra
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", type=int, default=3, choices=[2, 3, 4, 5, 6, 7, 8])
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-extra-configs", action="store_true",
                    help="time configuration 3 only (by default one GPU also times configurations 5 and 4 on the same weights)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
        if args.workload in (4, 6):
            run_mixed(args)
        elif args.workload in (7, 8):
            run_grouped(args)
        else:
            run_cuda(args)


if __name__ == "__main__":
    main()
