"""The benchmark workloads at their FULL sizes, in both launch configurations bench.py times (plain stream
order, and consecutive steps overlapped over resident inputs; outputs of a step are read back after later steps
were enqueued), compared with the fp64 oracle element by element.  The fused LM-head workload is in
test_gpu_fused.py."""
import numpy as np
import pytest
import torch

from paper_2511_22972_b200 import FlyVerify, VerifyBuffers, synthetic as S, verify
from tests._parity import assert_parity, draw, oracle_step

pytestmark = pytest.mark.gpu
DEV = "cuda"


def run_overlapped(fv, steps, theta, W, boundary="reject", chain=False):
    """Enqueues all steps back to back on one stream, then compares every step with the oracle; the even steps
    in plain stream order, the odd ones with inputs_ready (they may read while the step before them drains).
    chain=True: one state buffer is carried from step to step (carry mode)."""
    st = torch.cuda.current_stream().cuda_stream
    torch.cuda.synchronize()                         # every step's inputs are complete before the first launch
    B, K1, _ = steps[0][0].shape
    outs = [VerifyBuffers(B, K1 - 1, DEV) for _ in steps]
    state = outs[0].state
    snapshots = []
    for (logits, draft), out in zip(steps, outs):
        if chain:
            out.state = state                        # every step reads and writes the same carried state
        verify(fv, logits, draft, out, theta=theta, W=W, boundary=boundary, stream=st,
               inputs_ready=len(snapshots) % 2 == 1 if chain else (outs.index(out) % 2 == 1))
        if chain:
            snapshots.append(state.clone())          # stream-ordered copy of the state after this step
    torch.cuda.synchronize()
    assert fv.device_status(st) == 0
    ref_state = np.array([[0, 0, -1]] * B) if chain else None
    worst = 0.0
    for n, ((logits, draft), out) in enumerate(zip(steps, outs)):
        ref = oracle_step(logits, draft, theta, W, boundary, ref_state)
        if chain:
            out.state = snapshots[n]
            ref_state = ref.state_out
        worst = max(worst, assert_parity(out, ref, f"step {n}"))
    return worst


def test_tiny_verify_all_200_steps():
    w = S.TINY
    fv = FlyVerify(w.B, w.K, w.V, w.dtype)
    steps = [draw(w, step=s) for s in range(w.steps)]
    assert run_overlapped(fv, steps, w.theta, w.W) <= 1e-4


def test_llama3_vocab_batch_full_size():
    w = S.LLAMA3
    fv = FlyVerify(w.B, w.K, w.V, w.dtype)
    steps = [draw(w, step=s) for s in range(12)]
    run_overlapped(fv, steps, w.theta, w.W)


@pytest.mark.parametrize("setting", range(len(S.LONG_DRAFT_SETTINGS)))
def test_long_draft_batch_full_size_every_setting(setting):
    theta, W = S.LONG_DRAFT_SETTINGS[setting]
    w = S.LONG_DRAFT
    fv = FlyVerify(w.B, w.K, w.V, w.dtype)
    steps = [draw(w, step=s, setting=setting, thetas=[theta]) for s in range(2)]   # inputs regenerated per setting
    run_overlapped(fv, steps, theta, W)


def test_high_batch_serving_full_size_chained_rounds():
    w = S.SERVING
    fv = FlyVerify(w.B, w.K, w.V, w.dtype)
    steps = [draw(w, step=s) for s in range(6)]
    run_overlapped(fv, steps, w.theta, w.W, boundary="carry", chain=True)


def test_repeated_steps_are_bit_identical():
    # determinism and freedom from races over many launches: the same inputs give the same bits, on the
    # overlapped logits path and on the fused path (whose per-CTA states are merged in a fixed order)
    import random
    from paper_2511_22972_b200 import binding as Bd
    rng = random.Random(0)
    st = torch.cuda.current_stream().cuda_stream
    names = ("accept_len", "out_tokens", "target_argmax", "entropy", "row_flags", "state", "rollback")

    def soak(fv, arglist, outs, steps):
        for a in arglist:
            fv.run(a, st)
        torch.cuda.synchronize()
        ref = [[getattr(o, n).clone() for n in names] for o in outs]
        for it in range(steps):
            fv.run(arglist[rng.randrange(len(arglist))], st)
            if it % 250 == 249:
                torch.cuda.synchronize()
                for o, r in zip(outs, ref):
                    assert all(torch.equal(getattr(o, n), x) for n, x in zip(names, r)), f"step {it}"
        assert fv.device_status(st) == Bd.FLY_OK

    w = S.LLAMA3
    fv = FlyVerify(w.B, w.K, w.V, w.dtype)
    ins = [(S.make_logits(w, i, device=DEV), torch.randint(0, w.V, (w.B, w.K), device=DEV, dtype=torch.int32)) for i in range(4)]
    outs = [VerifyBuffers(w.B, w.K, DEV) for _ in ins]
    args = [fv.make_args(w.B, w.K, d, o.accept_len, o.out_tokens, logits=l, state_out=o.state, rollback=o.rollback,
                         target_argmax=o.target_argmax, entropy=o.entropy, row_flags=o.row_flags, inputs_ready=i % 2 == 1)
            for i, ((l, d), o) in enumerate(zip(ins, outs))]
    torch.cuda.synchronize()
    soak(fv, args, outs, 5000)
    fv.close()

    w = S.shrink(S.FUSED, V=32064)
    weight = S.make_weight(w, device=DEV)
    fv = FlyVerify(w.B, w.K, w.V, "bf16", hidden=w.hidden)
    ins = [(S.make_hidden(w, i, device=DEV), torch.randint(0, w.V, (w.B, w.K), device=DEV, dtype=torch.int32)) for i in range(3)]
    outs = [VerifyBuffers(w.B, w.K, DEV) for _ in ins]
    args = [fv.make_args(w.B, w.K, d, o.accept_len, o.out_tokens, hidden=h, weight=weight, state_out=o.state,
                         rollback=o.rollback, target_argmax=o.target_argmax, entropy=o.entropy, row_flags=o.row_flags)
            for (h, d), o in zip(ins, outs)]
    soak(fv, args, outs, 1500)
    fv.close()
