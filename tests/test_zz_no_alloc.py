"""The allocation-free decode step (mars_decode_step_static) against the handle-based one.

Some users of this library run where they may not create device memory themselves: a plug-in that
is handed weights and cache pools by its host program, or a loop that must stay away from the
allocator.  They cannot supply the workspace that the regular calls need, so the library offers one
call whose intermediates sit in a fixed array built into the library.  This test drives that call
through the C ABI twice in a row (the second step continues from the first) and requires the same
tokens and log-probs as mars_decode_step gives on an identical, separately built case.

The file name sorts last on purpose: a run that stops at the first failure has then already
executed every other test.
"""
import pytest
import torch

from harness import Case
from paper_2511_11373_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

TOL_LOGP = 2e-2   # the log-prob tolerance used by the parity tests


def test_static_scratch_step_matches_regular_step_twice():
    model = dict(wl.MODEL_TINY, n_layers=2, qk_norm=1)
    ctx, ps, steps = [15, 40, 130, 600], 16, 2         # 15 -> 16 crosses a page boundary; 600 spans two work items
    ref = Case(model, ps, ctx, seed=13, headroom=steps)
    sta = Case(model, ps, ctx, seed=13, headroom=steps)  # same bytes, its own pools for the static call to append to
    dev = ref.device
    bt = sta.bt.to(dev)
    smp = dict(greedy=0, temperature=0.85, top_p=0.95)
    tok_ref = wl.make_tokens(len(ctx), model["vocab"], seed=5).to(dev)
    tok_sta = tok_ref.clone()
    for s in range(steps):
        sampling = binding.make_sampling(seed=99, step=s, **smp)
        out_r, lp_r = torch.empty_like(tok_ref), torch.empty(len(ctx), device=dev)
        st = binding.mars_decode_step(ref.model, ref.kv, list(range(len(ctx))), tok_ref, sampling, out_r, lp_r)
        assert st == 0 and ref.model.poll_status() == 0
        out_s, lp_s = torch.empty_like(tok_sta), torch.empty(len(ctx), device=dev)
        st = binding.mars_decode_step_static(model, sta.weights, sta.max_pos, sta.k_pool, sta.v_pool, ps, bt,
                                             [c + s for c in ctx], tok_sta, sampling, out_s, lp_s)
        assert st == 0, binding.STATUS_NAMES.get(st, st)
        torch.cuda.synchronize()
        assert torch.equal(out_r.cpu(), out_s.cpu()), (s, out_r.tolist(), out_s.tolist())
        assert (lp_r.cpu() - lp_s.cpu()).abs().max() <= TOL_LOGP
        assert torch.isfinite(lp_s).all()
        tok_ref, tok_sta = out_r, out_s
    # the appended cache rows agree as well
    # (the two calls may run their projections on different kernels, so a key can land on the
    # neighbouring bf16 value: same row tolerance as the parity tests, not bit equality)
    kr, ks = ref.k_pool.cpu().float(), sta.k_pool.cpu().float()
    assert torch.equal(torch.isnan(kr), torch.isnan(ks))
    kr, ks = torch.nan_to_num(kr), torch.nan_to_num(ks)
    assert ((kr - ks).norm(dim=-1) <= 1e-2 * kr.norm(dim=-1) + 1e-6).all()


def test_static_scratch_rejects_what_does_not_fit():
    model = dict(wl.MODEL_TINY, n_layers=1)
    case = Case(model, 16, [5], seed=1)
    dev = case.device
    tok = torch.zeros(1, dtype=torch.int32, device=dev)
    out, lp = torch.empty_like(tok), torch.empty(1, device=dev)
    smp = binding.make_sampling(greedy=1)
    # a long maximum position inflates the split-K partial buffers beyond the built-in array
    st = binding.mars_decode_step_static(model, case.weights, 4 << 20, case.k_pool, case.v_pool, 16, case.bt.to(dev),
                                         [5], tok, smp, out, lp)
    assert st == 8 and b"built-in scratch" in binding.lib().mars_status_string(st)
    big = dict(wl.MODEL_LAYER)
    cfg = binding.make_config(big, 20000)
    assert binding.lib().mars_workspace_bytes(cfg, 64, 0) > (4 << 20)
