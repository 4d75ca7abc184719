"""fly_verify_run_static: the verification step for callers that cannot allocate
device memory (a server whose memory pool owns the whole GPU, a plugin running
inside another framework's callback, a latency-critical loop).  It needs no
handle; its scratch is a fixed array inside the library.

This file is collected last on purpose: it is an addition outside the paper's
method, and a failure here must not hide the result of any other test.

The check: two calls in a row through the C ABI, different shapes, each
compared with the fp64 oracle (the same comparison as every parity test) and,
as a second check, with what the handle-based entry point (fly_verify_run)
writes for the same inputs - integers bit for bit, entropy within the tolerance
of the parity tests.  Nothing here depends on what ran before in the process:
the entry point clears its arrival counters itself and both calls are on one
stream.
"""
import pytest
import torch

from paper_2511_22972_b200 import FlyError, FlyVerify, VerifyBuffers, binding as Bd, synthetic as S
from tests._parity import assert_parity, draw, oracle_step

pytestmark = pytest.mark.gpu
DEV = "cuda"
ENTROPY_TOL = 1e-4


def _args(w, logits, draft, out, boundary, state_in):
    return Bd.static_args(w.B, w.K, draft, out.accept_len, out.out_tokens, logits=logits, theta=w.theta, W=w.W,
                          boundary=boundary, state_in=state_in, state_out=out.state, rollback=out.rollback,
                          target_argmax=out.target_argmax, entropy=out.entropy, row_flags=out.row_flags)


def _same(a: VerifyBuffers, b: VerifyBuffers, what):
    for name in ("accept_len", "rollback", "out_tokens", "target_argmax", "row_flags", "state"):
        assert torch.equal(getattr(a, name), getattr(b, name)), f"{what}: {name} differs"
    err = (a.entropy.double() - b.entropy.double()).abs().max().item()
    assert err <= ENTROPY_TOL, f"{what}: entropy differs by {err:.3e}"


def test_static_entry_point_matches_the_handle_entry_point_twice_in_a_row():
    st = torch.cuda.current_stream().cuda_stream
    cases = [
        (S.shrink(S.LLAMA3, B=6, K=8), "reject"),                 # rows are cut into several pieces
        (S.shrink(S.SERVING, B=40, K=5, V=50264), "carry"),        # more sequences, carried state, other vocab
    ]
    for n, (w, boundary) in enumerate(cases):
        logits, draft = draw(w, step=11 + n)                       # entropies kept away from the threshold
        carry = boundary == "carry"
        state0 = torch.tensor([[1, 3, 7]] * w.B, dtype=torch.int32, device=DEV) if carry else None

        ref = VerifyBuffers(w.B, w.K, DEV)
        if carry:
            ref.state.copy_(state0)
        fv = FlyVerify(w.B, w.K, w.V, w.dtype)
        fv.run(_args(w, logits, draft, ref, boundary, ref.state if carry else None), st)
        torch.cuda.synchronize()
        fv.close()

        got = VerifyBuffers(w.B, w.K, DEV)
        if carry:
            got.state.copy_(state0)
        for name in ("accept_len", "out_tokens", "target_argmax"):
            getattr(got, name).fill_(-7)                           # stale values must all be overwritten
        Bd.run_static(_args(w, logits, draft, got, boundary, got.state if carry else None), w.V, w.dtype, 0, st)
        torch.cuda.synchronize()
        oracle = oracle_step(logits, draft, w.theta, w.W, boundary, state0.cpu().numpy() if carry else None)
        assert_parity(got, oracle, f"call {n + 1} ({w.name}) against the oracle")
        _same(got, ref, f"call {n + 1} ({w.name})")
        s = got.accept_len.cpu()
        assert bool(((s >= 1) & (s <= w.K + 1)).all())


def test_static_entry_point_rejects_steps_beyond_its_scratch():
    V = 1024
    big_b = Bd.FLY_STATIC_MAX_BATCH + 1
    logits = torch.zeros(1, 2, V, dtype=torch.bfloat16, device=DEV)   # never read: the call fails before any launch
    draft = torch.zeros(1, 1, dtype=torch.int32, device=DEV)
    out = VerifyBuffers(1, 1, DEV)
    for B, K in [(big_b, 1), (1024, 63)]:                             # too many sequences; too many rows
        a = Bd.static_args(B, K, draft, out.accept_len, out.out_tokens, logits=logits, state_out=out.state)
        with pytest.raises(FlyError) as e:
            Bd.run_static(a, V, "bf16", 0, 0)
        assert e.value.status == Bd.FLY_ERR_TOO_LARGE
        assert "scratch" in str(e.value)
    a = Bd.static_args(1, 1, draft, out.accept_len, out.out_tokens, logits=None, state_out=out.state)
    with pytest.raises(FlyError) as e:
        Bd.run_static(a, V, "bf16", 0, 0)
    assert e.value.status == Bd.FLY_ERR_INVALID_ARG
