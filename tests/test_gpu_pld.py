"""Prompt-lookup drafting on the GPU (through the C ABI) against the CPU oracle: bit-exact."""
import random

import pytest
import torch

from oracle.pld_oracle import pld_draft as oracle_pld
from paper_2511_22972_b200 import binding as Bd

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run(seqs, K, mx, mn, pad_to=None):
    B = len(seqs)
    Lmax = pad_to or max(len(s) for s in seqs)
    tok = torch.full((B, Lmax), -7, dtype=torch.int32)
    for b, s in enumerate(seqs):
        tok[b, :len(s)] = torch.tensor(s, dtype=torch.int32)
    lengths = torch.tensor([len(s) for s in seqs], dtype=torch.int32)
    draft, count, pos, ng = Bd.pld_draft(tok.to(DEV), lengths.to(DEV), K, mx, mn,
                                         stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for b, s in enumerate(seqs):
        prop, p, n = oracle_pld(s, K, mx, mn)
        assert count[b].item() == len(prop) and pos[b].item() == p and ng[b].item() == n, (b, s[:20])
        assert draft[b, :len(prop)].tolist() == prop and (draft[b, len(prop):] == -1).all()


def test_golden_cases_on_the_gpu():
    from tests.test_oracle_pld import golden_cases
    for toks, K, mx, mn, prop, pos, n in golden_cases():
        run([toks], K, mx, mn)


@pytest.mark.parametrize("alphabet", [2, 5, 1000, 128256])
def test_random_sequences(alphabet):
    rng = random.Random(alphabet)
    seqs = [[rng.randrange(alphabet) for _ in range(rng.choice([1, 2, 3, 17, 255, 256, 257, 1000, 4099]))] for _ in range(64)]
    for K, mx, mn in [(8, 3, 1), (25, 8, 1), (1, 1, 1), (15, 4, 2)]:
        run(seqs, K, mx, mn, pad_to=4100)


def test_long_context_with_a_planted_repeat():
    # a prompt-like sequence: 60k mostly unique tokens, the last 5 tokens copied from two earlier places
    rng = random.Random(9)
    base = [rng.randrange(10 ** 6) + 10 for _ in range(60000)]
    tail = base[40000:40005]
    base[1234:1239] = tail                       # an earlier copy: it must win over the one at 40000
    seq = base + tail
    run([seq, seq[:50000], base], 15, 5, 1)
    prop, p, n = oracle_pld(seq, 15, 5, 1)
    assert (p, n) == (1234, 5) and prop == seq[1239:1254]


def test_argument_errors():
    t = torch.zeros(1, 4, dtype=torch.int32, device=DEV)
    l = torch.ones(1, dtype=torch.int32, device=DEV)
    for K, mx, mn in [(0, 3, 1), (4, 9, 1), (4, 2, 3), (4, 3, 0)]:
        with pytest.raises(Bd.FlyError) as e:
            Bd.pld_draft(t, l, K, mx, mn)
        assert e.value.status == Bd.FLY_ERR_INVALID_ARG


def test_lengths_outside_the_row_propose_nothing_and_read_nothing_outside_it():
    # lengths is device data: a length larger than the row stride, or negative, must not steer a load past the row
    B, stride, K = 6, 64, 8
    rng = random.Random(3)
    tok = torch.tensor([[rng.randrange(4) for _ in range(stride)] for _ in range(B)], dtype=torch.int32)
    lengths = torch.tensor([stride, stride + 1, 10 ** 9, -1, -(10 ** 9), 40], dtype=torch.int32)
    draft, count, pos, ng = Bd.pld_draft(tok.to(DEV), lengths.to(DEV), K, 3, 1, stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    for b in (1, 2, 3, 4):
        assert count[b].item() == 0 and pos[b].item() == -1 and ng[b].item() == 0 and (draft[b] == -1).all()
    for b in (0, 5):
        prop, p, n = oracle_pld(tok[b, :lengths[b]].tolist(), K, 3, 1)
        assert count[b].item() == len(prop) and pos[b].item() == p and draft[b, :len(prop)].tolist() == prop
