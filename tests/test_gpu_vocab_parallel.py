"""Vocabulary-parallel verification on ONE GPU: the ranks of a tensor-parallel LM head are played one after
the other (no kernel waits on another), each reducing its slice of the vocabulary to one partial state per
row; the gathered states are merged and verified.  The result must equal the oracle on the whole rows."""
import math

import numpy as np
import pytest
import torch

from paper_2511_22972_b200 import FlyVerify, VerifyBuffers, dist as D, synthetic as S
from tests._parity import assert_parity, draw, oracle_step

pytestmark = pytest.mark.gpu
DEV = "cuda"


def sharded_step(w, logits, draft, world, theta, W, theta_unit="nats", boundary="reject", state=None, temperature=0.0):
    B, K1, V = logits.shape
    rows = B * K1
    flat = logits.view(rows, V)
    gathered = torch.empty(world, rows, 4, dtype=torch.float32, device=DEV)
    st = torch.cuda.current_stream().cuda_stream
    merger = None
    for rank in range(world):
        off, width = D.shard_vocab(V, D.Ranks(rank, world, 0, ""))
        fv = FlyVerify(B, K1 - 1, max(width, 1), w.dtype)
        if width > 0:
            fv.reduce_shard(flat[:, off:off + width], off, gathered[rank], st, temperature=temperature)
        else:                                                     # an empty slice contributes the empty state
            gathered[rank] = torch.tensor([-999424.0, 0.0, 0.0, 0.0])
            gathered[rank].view(torch.int32)[:, 3] = 0x7fffffff
        torch.cuda.synchronize()
        merger = fv
    out = VerifyBuffers(B, K1 - 1, DEV)
    if state is not None:
        out.state.copy_(torch.as_tensor(state, dtype=torch.int32))
    a = merger.make_args(B, K1 - 1, draft, out.accept_len, out.out_tokens, theta=theta, theta_unit=theta_unit, W=W,
                         boundary=boundary, state_in=out.state if boundary == "carry" else None, state_out=out.state,
                         rollback=out.rollback, target_argmax=out.target_argmax, entropy=out.entropy,
                         row_flags=out.row_flags, temperature=temperature)
    merger.run_partials(a, gathered, world, V, st)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("world", [1, 2, 4, 7])
@pytest.mark.parametrize("dtype,V", [("bf16", 128256), ("f32", 32000), ("bf16", 50257)])
def test_sharded_vocabulary_equals_whole_rows(world, dtype, V):
    w = S.shrink(S.LLAMA3 if dtype == "bf16" else S.TINY, B=4, K=8, V=V)
    logits, draft = draw(w, step=world)
    out = sharded_step(w, logits, draft, world, 1.0, 3)
    assert_parity(out, oracle_step(logits, draft, 1.0, 3), f"world={world} {dtype} V={V}")


def test_paper_405b_setting_on_four_ranks_with_normalised_threshold():
    # K = 25, W = 6, threshold 0.3 on h = H / log|V| with |V| the WHOLE vocabulary, four vocabulary slices
    w = S.shrink(S.PAPER_405B, B=2)
    logits, draft = draw(w, step=3)
    out = sharded_step(w, logits, draft, 4, 0.3, w.W, theta_unit="normalized")
    assert_parity(out, oracle_step(logits, draft, 0.3, w.W, theta_unit="normalized"), "405b tp4")
    assert abs(w.theta - 0.3 * math.log(w.V)) < 1e-12


def test_ties_across_ranks_and_masked_slices():
    V = 4096
    w = S.shrink(S.LLAMA3, B=2, K=3, V=V)
    logits, draft = draw(w, step=9, guard=False)
    rows = logits.view(-1, V)
    top = rows.float().max().item() + 2.0
    rows[0, [3000, 1030, 2050]] = top                 # the same maximum in three different slices: lowest id wins
    rows[1, 1024:2048] = -math.inf                    # one rank's slice fully masked
    rows[2, :] = -math.inf
    rows[2, 4095] = 1.0                               # one-hot in the last slice
    out = sharded_step(w, logits, draft, 4, 0.5, 1)
    ref = oracle_step(logits, draft, 0.5, 1)
    assert_parity(out, ref, "ties and masks")
    assert out.target_argmax.view(-1)[0].item() == 1030 and out.target_argmax.view(-1)[2].item() == 4095


def test_carry_state_with_sharded_vocabulary():
    w = S.shrink(S.SERVING, B=8, K=8, V=32064)
    logits, draft = draw(w, step=4)
    state = [[b % 3, 4, 11] for b in range(w.B)]
    out = sharded_step(w, logits, draft, 2, w.theta, w.W, boundary="carry", state=state)
    assert_parity(out, oracle_step(logits, draft, w.theta, w.W, "carry", state), "carry tp2")


@pytest.mark.parametrize("T", [0.7, 1.5])
def test_sharded_vocabulary_at_a_temperature(T):
    # every rank and the merging call pass the same temperature: the merged entropy is that of softmax(l / T)
    w = S.shrink(S.LLAMA3, B=3, K=5, V=50264)
    logits, draft = draw(w, step=5, temperature=T)
    out = sharded_step(w, logits, draft, 4, 1.0, 2, temperature=T)
    assert_parity(out, oracle_step(logits, draft, 1.0, 2, temperature=T), f"tp4 T={T}")
