"""The input generator: determinism, shapes, recipe statistics, and the
entropy guard (rows too close to the gate threshold are redrawn)."""
import math

import numpy as np
import torch

from oracle import fly_oracle as O
from paper_2511_22972_b200 import synthetic as S


def oracle_entropy(rows):
    return O.row_stats(rows.double().cpu().numpy())[0]


def test_five_workloads_match_the_published_shapes():
    assert (S.TINY.rows, S.TINY.V, S.TINY.dtype) == (9, 32000, "f32")
    assert (S.LLAMA3.rows, S.LLAMA3.V, S.LLAMA3.dtype) == (144, 128256, "bf16")
    assert (S.LONG_DRAFT.rows, S.LONG_DRAFT.V) == (1088, 128256)
    assert (S.SERVING.rows, S.SERVING.V, S.SERVING.boundary) == (2304, 152064, "carry")
    assert (S.FUSED.rows, S.FUSED.hidden, S.FUSED.V) == (288, 8192, 128256)
    assert len(S.LONG_DRAFT_SETTINGS) == 9


def test_deterministic_and_step_dependent():
    w = S.shrink(S.LLAMA3, B=2, K=3, V=1000)
    a = S.make_logits(w, 5)
    b = S.make_logits(w, 5)
    c = S.make_logits(w, 6)
    assert a.dtype == torch.bfloat16 and a.shape == (2, 4, 1000)
    assert torch.equal(a, b) and not torch.equal(a, c)
    t5 = S.rank5(a.view(-1, w.V))
    assert torch.equal(S.make_draft(w, 5, t5), S.make_draft(w, 5, t5))
    assert S.make_draft(w, 5, t5).dtype == torch.int32


def test_recipe_statistics():
    w = S.shrink(S.LLAMA3, B=50, K=7, V=4096)
    x = S.make_logits(w, 0).view(-1, w.V).float()
    std = x.std(dim=1)
    assert 0.45 < std.min() and std.max() < 4.6          # s ~ U(0.5, 4) (+ spike)
    # with a narrow scale every spike (>= 8) stands > 7 sigma out; noise alone never does
    wn = S.shrink(w, scale=(0.5, 1.0))
    xn = S.make_logits(wn, 0).view(-1, w.V).float()
    frac_spiked = (xn.max(dim=1).values > 7.0).float().mean().item()
    assert 0.3 < frac_spiked < 0.5                       # 40% of rows
    t5 = S.rank5(x)
    assert torch.equal(t5[:, 0], torch.argmax(x, dim=1))
    d = S.make_draft(w, 0, t5)
    hit = (d.view(-1) == t5.view(w.B, w.K + 1, 5)[:, : w.K, 0].reshape(-1)).float().mean().item()
    assert 0.5 < hit < 0.7                               # P(argmax) = 0.6
    assert int(d.min()) >= 0 and int(d.max()) < w.V


def test_rank5_orders_ties_by_index():
    x = torch.tensor([[1.0, 3.0, 3.0, 0.0, 3.0, 2.0, 2.0]])
    assert S.rank5(x).tolist() == [[1, 2, 4, 5, 6]]


def test_entropy_guard_moves_rows_off_the_threshold():
    w = S.shrink(S.LLAMA3, B=8, K=3, V=512)
    x0 = S.make_logits(w, 1)
    H0 = oracle_entropy(x0.view(-1, w.V))
    # put the threshold exactly on one row's entropy: that row must be redrawn
    th = float(H0[5])
    x1 = S.make_logits(w, 1, entropy_fn=oracle_entropy, theta_nats=th)
    H1 = oracle_entropy(x1.view(-1, w.V))
    assert (np.abs(H1 - th) >= 1e-3).all()
    same = [torch.equal(x0.view(-1, w.V)[r], x1.view(-1, w.V)[r]) for r in range(w.rows)]
    assert not same[5] and sum(same) >= w.rows - 2


def test_tiny_workload_recipe():
    x = S.make_logits(S.TINY, 0)
    assert x.dtype == torch.float32 and x.shape == (1, 9, 32000)
    h = S.make_hidden(S.shrink(S.FUSED, B=1, K=1, hidden=64), 0)
    wt = S.make_weight(S.shrink(S.FUSED, V=100, hidden=64))
    assert h.shape == (2, 64) and wt.shape == (64, 100) and wt.dtype == torch.bfloat16
    assert abs(wt.float().std().item() - 0.02) < 0.002
