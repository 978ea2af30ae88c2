"""Pins for the acceptance oracle: planted rows, constructed ties and NaNs, numpy argmax."""
import numpy as np
import pytest
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl


@pytest.mark.parametrize("depths", [None, [0, 0, 0, 0], [16, 16, 16, 16], [1, 9, 0, 16]])
def test_planted_reject_index(depths):
    """Rows before the planted reject index carry the draft token as their unique maximum, so
    the accepted prefix is min(R_i, d_i): A_i = 1 + min(L_i, n_i) of Section 3.2."""
    cfg = wl.config(0)
    sel = wl.select_inputs(cfg)
    if depths is None:
        depths = np.minimum(sel.reject_index + 1, cfg.gamma)
    depths = np.array(depths, np.int32)
    cu = wl.cu_q_from_depths(depths)
    logits = wl.logits_rows(cfg, sel, depths)
    r = orc.accept(logits, sel.draft_ids, cu, cfg.gamma)
    want = np.minimum(sel.reject_index, depths)
    assert np.array_equal(r.accept_len, want)
    assert r.n_accepted_total == int((want + 1).sum())
    am = logits.float().numpy().argmax(1)
    assert np.array_equal(r.argmax, am)                       # numpy: first maximum
    for i in range(cfg.B):
        m = want[i]
        assert r.bonus[i] == am[cu[i] + m]
        row = r.out_tokens[i]
        assert row[:m].tolist() == sel.draft_ids[i, :m].tolist()
        assert row[m] == r.bonus[i] and np.all(row[m + 1:] == -1)
        if m < depths[i]:
            assert r.bonus[i] != sel.draft_ids[i, m]          # a real rejection: the bonus corrects it


def test_full_accept_takes_bonus_from_last_row():
    B, g, V = 2, 3, 50
    draft = np.array([[4, 5, 6], [7, 8, 9]], np.int32)
    depths = np.array([3, 2], np.int32)
    cu = wl.cu_q_from_depths(depths)
    logits = torch.zeros((int(cu[-1]), V), dtype=torch.bfloat16)
    for i in range(B):
        for t in range(depths[i]):
            logits[cu[i] + t, draft[i, t]] = 1.0
    logits[cu[0] + 3, 33] = 2.0
    logits[cu[1] + 2, 44] = 2.0
    r = orc.accept(logits, draft, cu, g)
    assert r.accept_len.tolist() == [3, 2] and r.bonus.tolist() == [33, 44]
    assert r.out_tokens.tolist() == [[4, 5, 6, 33], [7, 8, 44, -1]]
    assert r.n_accepted_total == 7


def test_sequential_acceptance_stops_at_first_mismatch():
    g, V = 4, 20
    draft = np.array([[1, 2, 3, 4]], np.int32)
    cu = np.array([0, 5], np.int32)
    logits = torch.zeros((5, V), dtype=torch.bfloat16)
    for t, tok in enumerate([1, 9, 3, 4, 5]):       # row 1 disagrees; rows 2, 3 would agree again
        logits[t, tok] = 1.0
    r = orc.accept(logits, draft, cu, g)
    assert r.accept_len.tolist() == [1] and r.bonus.tolist() == [9]
    assert r.out_tokens.tolist() == [[1, 9, -1, -1, -1]]


def test_ties_nan_and_signed_zero():
    V = 16
    cu = np.array([0, 1, 2, 3, 4, 5, 6], np.int32)
    draft = np.zeros((6, 1), np.int32)
    logits = torch.full((6, V), -1.0, dtype=torch.bfloat16)
    logits[0, 5] = 3.0
    logits[0, 11] = 3.0                     # tie: lowest index
    logits[1, 2] = float("nan")
    logits[1, 7] = 0.5                      # NaN never wins
    logits[2, :] = float("nan")             # all NaN: 0
    logits[3, :] = float("-inf")
    logits[3, 9] = -1.0e30                  # a finite value beats -inf
    logits[4, :] = float("-inf")            # all -inf: first index
    logits[5, :] = -1.0
    logits[5, 3] = -0.0
    logits[5, 6] = 0.0                      # -0 == +0: the earlier one stays
    r = orc.accept(logits, draft, cu, 1)
    assert r.argmax.tolist() == [5, 7, 0, 9, 0, 3]
    assert r.accept_len.tolist() == [0] * 6 and r.bonus.tolist() == [5, 7, 0, 9, 0, 3]


def test_random_rows_match_numpy_argmax():
    rng = np.random.default_rng(11)
    T, V = 64, 3001
    x = torch.from_numpy(rng.standard_normal((T, V), dtype=np.float32)).to(torch.bfloat16)
    cu = np.arange(T + 1, dtype=np.int32)
    r = orc.accept(x, np.zeros((T, 1), np.int32), cu, 1)
    xf = x.float().numpy()
    assert np.array_equal(r.argmax, xf.argmax(1))
    assert ((xf == xf.max(1, keepdims=True)).sum(1) > 1).any()     # bf16 rows do tie: the rule matters
