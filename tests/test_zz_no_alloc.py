"""dcut_accept_static, the acceptance call for callers that may not allocate (no context; its
scratch is a fixed array inside the library), must give exactly what dcut_accept gives.

Collected last on purpose: the array is shared by everything in the process, so this also runs
after every other test has used the GPU; it passes alone in a fresh process as well."""
import numpy as np
import pytest
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _inputs(cfg, depths, seed_shift):
    sel = wl.select_inputs(cfg)
    logits = wl.logits_rows(cfg, sel, depths)
    if seed_shift:                                   # a second, different batch for the second call
        logits = torch.roll(logits, shifts=seed_shift, dims=1)
    return sel, logits


def test_static_scratch_matches_context_scratch_on_two_calls_in_a_row():
    from paper_2607_14647_b200 import binding
    cfg = wl.config(0)
    ctx = binding.Context(max_B=cfg.B, max_gamma=cfg.gamma, vocab=cfg.vocab)
    i32 = dict(dtype=torch.int32, device="cuda")
    # first call: deep batch (68 rows); second call: shallower batch, so rows the first call used stay
    # behind in the shared array and must not leak into the result
    for depths, shift in ((np.full(cfg.B, cfg.gamma, np.int32), 0), (np.array([2, 0, 5, 1], np.int32), 7)):
        sel, logits = _inputs(cfg, depths, shift)
        cu = torch.from_numpy(wl.cu_q_from_depths(depths)).cuda()
        d_logits, d_draft = logits.cuda(), torch.from_numpy(sel.draft_ids).cuda()
        want = ctx.accept(d_logits, d_draft, cu, cfg.t_cap)
        got = (torch.full((cfg.B,), -7, **i32), torch.full((cfg.B,), -7, **i32),
               torch.full((cfg.B, cfg.gamma + 1), -7, **i32), torch.full((1,), -7, **i32))
        binding.accept_static(d_logits, d_draft, cu, cfg.t_cap, *got)
        torch.cuda.synchronize()
        for g, w in zip(got, want):
            assert torch.equal(g, w)
        ref = orc.accept(logits, sel.draft_ids, wl.cu_q_from_depths(depths), cfg.gamma)   # and both equal the oracle
        assert np.array_equal(got[0].cpu().numpy(), ref.accept_len) and np.array_equal(got[1].cpu().numpy(), ref.bonus)
        assert np.array_equal(got[2].cpu().numpy(), ref.out_tokens) and int(got[3].item()) == ref.n_accepted_total
    ctx.close()


def test_rows_past_T_cap_are_left_alone():
    """A cu_q that runs past T_cap breaks the caller's contract; the call must still stay inside the first T_cap
    words of the shared array.  T_cap = 8 with cu_q[B] = 12: rows 8..11 are left out, the outputs are defined,
    and a valid call right after (which would see any stray write to words 8..11) still matches the oracle."""
    from paper_2607_14647_b200 import binding
    from tests.test_gpu_accept import _past_cap_case
    x, draft, cu, g, want_len, want_bonus = _past_cap_case()
    i32 = dict(dtype=torch.int32, device="cuda")
    d_x, d_draft, d_cu = x.cuda(), torch.from_numpy(draft).cuda(), torch.from_numpy(cu).cuda()
    out = (torch.full((4,), -7, **i32), torch.full((4,), -7, **i32), torch.full((4, g + 1), -7, **i32), torch.full((1,), -7, **i32))
    binding.accept_static(d_x, d_draft, d_cu, 8, *out)
    torch.cuda.synchronize()
    assert np.array_equal(out[0].cpu().numpy(), want_len) and np.array_equal(out[1].cpu().numpy(), want_bonus)
    binding.accept_static(d_x, d_draft, d_cu, 12, *out)
    torch.cuda.synchronize()
    ref = orc.accept(x, draft, cu, g)
    assert np.array_equal(out[0].cpu().numpy(), ref.accept_len) and np.array_equal(out[1].cpu().numpy(), ref.bonus)


def test_rows_beyond_the_fixed_scratch_are_refused():
    from paper_2607_14647_b200 import binding
    i32 = dict(dtype=torch.int32, device="cuda")
    B, g, V = 4, 2, 64
    logits = torch.zeros((B * (g + 1), V), dtype=torch.bfloat16, device="cuda")
    cu = torch.arange(0, B * (g + 1) + 1, g + 1, **i32)
    out = (torch.zeros(B, **i32), torch.zeros(B, **i32), torch.zeros((B, g + 1), **i32), torch.zeros(1, **i32))
    with pytest.raises(binding.DcutError) as e:
        binding.accept_static(logits, torch.zeros((B, g), **i32), cu, binding.ACCEPT_STATIC_MAX_ROWS + 1, *out)
    assert e.value.status == binding.ECAPACITY and "exceed the fixed scratch" in str(e.value)
