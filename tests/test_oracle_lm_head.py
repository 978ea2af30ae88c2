"""Pins for the oracle of the LM head followed by acceptance (logits = x . W^T rounded to bf16, then greedy accept):
a hand example, numpy's float64 matmul, and the planted-row construction whose result is known in closed form."""
import numpy as np
import torch

from oracle import dcut_oracle as orc
from paper_2607_14647_b200 import workloads as wl


def _bf(a):
    return torch.tensor(a, dtype=torch.float32).to(torch.bfloat16)


def test_hand_example():
    # two requests: depths 1 and 0 -> rows (0,0), (0,1), (1,0)
    x = _bf([[1, 0], [0, 1], [1, 1]])
    w = _bf([[1, 0], [0, 2], [1, 0], [3, -3]])          # V = 4
    # logits: [1,0,1,3], [0,2,0,-3], [1,2,1,0]  -> argmax 3, 1, 1
    draft = np.array([[3, 9], [7, 7]], np.int32)        # request 0 drafts token 3 (accepted); request 1 has no draft kept
    cu = np.array([0, 2, 3], np.int32)
    res, logits = orc.lm_head_accept(x, w, draft, cu, 2)
    assert np.array_equal(logits, np.array([[1, 0, 1, 3], [0, 2, 0, -3], [1, 2, 1, 0]], np.float64))
    assert list(res.argmax) == [3, 1, 1]
    assert list(res.accept_len) == [1, 0] and list(res.bonus) == [1, 1]
    assert res.n_accepted_total == 3
    # a tie goes to the lowest index: swap request 0's draft to token 0 on a row [1,0,1,*]
    res2, _ = orc.lm_head_accept(_bf([[1, 0], [0, 1], [1, 1]]), _bf([[1, 0], [0, 2], [1, 0], [0.5, -3]]), draft, cu, 2)
    assert res2.argmax[0] == 0 and res2.accept_len[0] == 0 and res2.bonus[0] == 0


def test_logits_match_numpy_float64_and_are_not_transposed():
    rng = np.random.default_rng(3)
    x = torch.from_numpy(rng.standard_normal((7, 48), dtype=np.float32)).to(torch.bfloat16)
    w = torch.from_numpy(rng.standard_normal((29, 48), dtype=np.float32)).to(torch.bfloat16)
    cu = np.array([0, 3, 7], np.int32)
    draft = rng.integers(0, 29, (2, 4)).astype(np.int32)
    res, logits = orc.lm_head_accept(x, w, draft, cu, 4)
    want = x.double().numpy() @ w.double().numpy().T
    assert logits.shape == (7, 29) and np.allclose(logits, want, rtol=1e-13, atol=1e-13)
    want_bf = torch.from_numpy(want).to(torch.bfloat16).double().numpy()   # round-to-nearest-even
    assert np.array_equal(res.argmax, want_bf.argmax(axis=1))               # numpy: first index of the maximum


def test_planted_rows_accept_exactly_the_planted_prefix():
    cfg = wl.custom_config(B=6, gamma=8, n_q_heads=4, n_kv_heads=2, head_dim=64, vocab=300)
    sel = wl.select_inputs(cfg)
    depths = np.array([8, 0, 3, 5, 1, 8], np.int32)
    w = wl.lm_head_weight(cfg, vocab=300, hidden=128)
    x = wl.lm_head_x_rows(cfg, sel, depths, w)
    cu = wl.cu_q_from_depths(depths)
    res, logits = orc.lm_head_accept(x, w, sel.draft_ids, cu, cfg.gamma)
    for i, d in enumerate(depths):
        planted = min(int(sel.reject_index[i]), int(d))
        for t in range(planted):
            assert res.argmax[cu[i] + t] == sel.draft_ids[i, t] % 300
        assert res.accept_len[i] >= planted                    # a random row may match by chance, never fewer
        assert res.bonus[i] == res.argmax[cu[i] + res.accept_len[i]]
    assert res.n_accepted_total == int((res.accept_len + 1).sum())
