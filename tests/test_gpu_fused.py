"""Parity of the fused LM-head path (tcgen05 GEMM with the entropy / argmax
epilogue, called through the C ABI) with the fp64 oracle: the oracle forms the
logits as the exact fp64 product of the bf16 inputs and verifies them as usual."""
import numpy as np
import pytest
import torch

from oracle import fly_oracle as O
from paper_2511_22972_b200 import FlyVerify, VerifyBuffers, binding as Bd, synthetic as S, verify_fused
from tests._parity import assert_parity

pytestmark = pytest.mark.gpu
DEV = "cuda"


def fused_case(B, K, D, V, step=0, weight_std=None, theta=1.0, min_gap=1e-3, guard=1e-3, temperature=1.0):
    """hidden, weight (bf16, device), draft and the oracle's logits for one step.  A hidden row is redrawn
    while its two largest fp64 logits are closer than min_gap (fp32 accumulation could then pick the other
    one) or its entropy is within `guard` of theta."""
    w = S.shrink(S.FUSED, B=B, K=K, V=V, hidden=D, weight_std=weight_std or 2.0 / np.sqrt(D))
    weight = S.make_weight(w, device="cpu")
    hidden = S.make_hidden(w, step, device="cpu")
    wd = weight.double().numpy()
    for attempt in range(1, 8):
        logits = O.lm_head_logits(hidden.double().numpy(), wd)
        top2 = np.partition(logits, V - 2, axis=1)[:, V - 2:]
        H = O.row_stats(logits / temperature)[0]
        bad = np.nonzero((np.abs(top2[:, 1] - top2[:, 0]) < min_gap) | (np.abs(H - theta) < guard))[0]
        if bad.size == 0:
            break
        fresh = S.make_hidden(w, step, device="cpu", attempt=attempt)
        hidden[torch.as_tensor(bad)] = fresh[torch.as_tensor(bad)]
    else:
        raise RuntimeError("could not separate the top two logits of every row")
    y = torch.as_tensor(logits.argmax(axis=1)).view(-1, 1)
    draft = S.make_draft(w, step, y)
    return w, hidden.to(DEV), weight.to(DEV), draft.to(DEV), logits


def run_and_check(B, K, D, V, theta=1.0, W=3, boundary="reject", state=None, temperature=0.0, **kw):
    w, hidden, weight, draft, logits = fused_case(B, K, D, V, theta=theta, temperature=temperature or 1.0, **kw)
    fv = FlyVerify(B, K, V, "bf16", hidden=D)
    out = VerifyBuffers(B, K, DEV)
    if state is not None:
        out.state.copy_(torch.as_tensor(state, dtype=torch.int32))
    verify_fused(fv, hidden, weight, draft, out, theta=theta, W=W, boundary=boundary,
                 stream=torch.cuda.current_stream().cuda_stream, temperature=temperature)
    assert fv.device_status(torch.cuda.current_stream().cuda_stream) == Bd.FLY_OK
    ref = O.verify_batch(logits.reshape(B, K + 1, V), draft.cpu().numpy(), theta, W, boundary=boundary,
                         state_in=None if state is None else np.asarray(state), temperature=temperature or 1.0)
    err = assert_parity(out, ref, f"fused B={B} K={K} D={D} V={V}")
    fv.close()
    return err, out, ref


@pytest.mark.parametrize("B,K", [(1, 1), (2, 7), (4, 8), (16, 8), (17, 8), (32, 8)])
def test_position_counts_up_to_one_block(B, K):
    # 2 .. 288 positions: one accumulator, both, a ragged second one
    run_and_check(B, K, D=256, V=1024)


@pytest.mark.parametrize("D,V", [(64, 128), (128, 256), (512, 4096), (200, 1000), (1024, 19000)])
def test_hidden_and_vocabulary_sizes(D, V):
    # one k-block, several, a ragged last k-block (200), a ragged last vocabulary tile (1000, 19000),
    # more tiles than SMs (19000 -> 149 tiles)
    run_and_check(4, 8, D=D, V=V)


def test_more_positions_than_one_block_and_carry_state():
    # 360 positions: two launches over the weight; carried state in and out
    B, K = 40, 8
    state = [[(b % 3), 4, 11] for b in range(B)]
    run_and_check(B, K, D=256, V=2048, boundary="carry", state=state)


@pytest.mark.parametrize("T", [0.7, 1.5])
def test_temperature_on_the_fused_path(T):
    # entropy of softmax(hidden x weight / T) out of tensor memory: 1/T rides in the epilogue's exponent constant
    run_and_check(8, 8, D=512, V=8192, theta=2.0, temperature=T, step=3)
    run_and_check(32, 8, D=256, V=1000, theta=1.0, W=2, temperature=T, step=4)


def test_theta_and_window_settings():
    for theta, W in [(0.5, 1), (2.0, 5), (float("inf"), 3), (0.0, 0)]:
        run_and_check(8, 8, D=256, V=2048, theta=theta, W=W)


def test_fused_matches_logits_path_on_materialised_logits():
    # same step through both paths: integers must agree, entropy within tolerance (the logits path reads the
    # product rounded to bf16, so only a loose entropy bound holds there; integers are compared where the
    # rounded logits keep the same argmax)
    B, K, D, V = 8, 8, 512, 8192
    w, hidden, weight, draft, logits = fused_case(B, K, D, V, step=3)
    fv = FlyVerify(B, K, V, "f32", hidden=D)
    out_f = VerifyBuffers(B, K, DEV)
    st = torch.cuda.current_stream().cuda_stream
    verify_fused(fv, hidden, weight, draft, out_f, stream=st)
    lg = torch.as_tensor(logits, dtype=torch.float32).view(B, K + 1, V).to(DEV)
    out_l = VerifyBuffers(B, K, DEV)
    from paper_2511_22972_b200 import verify
    verify(fv, lg, draft, out_l, stream=st)
    torch.cuda.synchronize()
    assert torch.equal(out_f.target_argmax, out_l.target_argmax)
    assert torch.equal(out_f.accept_len, out_l.accept_len)
    assert torch.equal(out_f.out_tokens, out_l.out_tokens)
    assert (out_f.entropy - out_l.entropy).abs().max().item() <= 1e-4


def test_host_buffer_entry_point_on_the_fused_path():
    B, K, D, V = 4, 8, 256, 2048
    w, hidden, weight, draft, logits = fused_case(B, K, D, V, step=5)
    fv = FlyVerify(B, K, V, "bf16", hidden=D)
    out = VerifyBuffers(B, K, "cpu", pinned=True)
    verify_fused(fv, hidden.cpu().pin_memory(), weight, draft.cpu().pin_memory(), out, host=True,
                 stream=torch.cuda.current_stream().cuda_stream)
    ref = O.verify_batch(logits.reshape(B, K + 1, V), draft.cpu().numpy(), 1.0, 3)
    assert_parity(out, ref, "fused host")


def test_fused_misuse():
    fv = FlyVerify(2, 4, 1024, "bf16")                       # no hidden size: the fused path is not available
    out = VerifyBuffers(2, 4, DEV)
    hidden = torch.zeros(10, 64, dtype=torch.bfloat16, device=DEV)
    weight = torch.zeros(64, 1024, dtype=torch.bfloat16, device=DEV)
    draft = torch.zeros(2, 4, dtype=torch.int32, device=DEV)
    with pytest.raises(Bd.FlyError) as e:
        verify_fused(fv, hidden, weight, draft, out)
    assert e.value.status == Bd.FLY_ERR_INVALID_ARG
    with pytest.raises(Bd.FlyError) as e:
        FlyVerify(2, 4, 1001, "bf16", hidden=64)             # row pitch of the weight not a multiple of 16 bytes
    assert e.value.status == Bd.FLY_ERR_UNSUPPORTED


def full_size_logits(hidden_cpu, weight_cpu, V):
    """Exact fp64 logits of some hidden rows against the whole weight, the product taken in vocabulary slices so
    that the fp64 copy of the weight never exists as a whole."""
    hs = hidden_cpu.double().numpy()
    parts = [O.lm_head_logits(hs, weight_cpu[:, v0:v0 + 16032].double().numpy()) for v0 in range(0, V, 16032)]
    return np.concatenate(parts, axis=1)


@pytest.mark.parametrize("vocab_major", [False, True])
def test_full_size_head_every_position(vocab_major):
    """The Llama-3.1-70B head shape of the benchmark (288 positions x 8192 x 128256), in the launch configuration
    the benchmark times, with ALL 288 rows compared with the oracle (bit-exact argmax / accept lengths / tokens,
    entropy within 1e-4), once per weight layout.  The oracle's side is one fp64 matrix product per vocabulary
    slice; a hidden row whose two largest fp64 logits are closer than 1e-3 (fp32 accumulation could pick the other)
    or whose entropy is within 1e-3 of the threshold is redrawn, as for the reduced shapes."""
    w = S.FUSED
    B, K, V, D = w.B, w.K, w.V, w.hidden
    weight = S.make_weight(w, device="cpu")
    hidden = S.make_hidden(w, 1 if vocab_major else 0, device="cpu")
    logits = full_size_logits(hidden, weight, V)                                   # [288, V] fp64
    for attempt in range(1, 6):
        top2 = np.partition(logits, V - 2, axis=1)[:, V - 2:]
        H = O.row_stats(logits)[0]
        bad = np.nonzero((np.abs(top2[:, 1] - top2[:, 0]) < 1e-3) | (np.abs(H - w.theta) < 1e-3))[0]
        if bad.size == 0:
            break
        fresh = S.make_hidden(w, 0, device="cpu", attempt=attempt)
        hidden[torch.as_tensor(bad)] = fresh[torch.as_tensor(bad)]
        logits[bad] = full_size_logits(hidden[torch.as_tensor(bad)], weight, V)
    else:
        raise RuntimeError("could not separate the top two logits of every row")
    y = torch.as_tensor(logits.argmax(axis=1)).view(-1, 1)
    draft = S.make_draft(w, 0, y).to(DEV)                                         # the oracle's token with p = 0.7, else uniform
    fv = FlyVerify(B, K, V, "bf16", hidden=D)
    fv.set_weight_layout(vocab_major)
    wdev = weight.to(DEV)
    if vocab_major:
        wdev = wdev.t().contiguous()                                              # [V, D], the usual layout of a linear layer
    out = VerifyBuffers(B, K, DEV)
    st = torch.cuda.current_stream().cuda_stream
    verify_fused(fv, hidden.to(DEV), wdev, draft, out, theta=w.theta, W=w.W, stream=st)
    assert fv.device_status(st) == Bd.FLY_OK
    assert fv.last_launch_count == 3
    ref = O.verify_batch(logits.reshape(B, K + 1, V), draft.cpu().numpy(), w.theta, w.W)
    err = assert_parity(out, ref, f"full-size head, weight {'[V, D]' if vocab_major else '[D, V]'}")
    assert err <= 1e-4 and (out.row_flags == 0).all()
    assert sorted(set(ref.accept_len.tolist())) != [K + 1]                        # the case exercises rejections too
    fv.close()


def test_a_wait_that_runs_out_is_reported_and_the_handle_stays_usable():
    # no fault, no hang: a one-thread kernel waits 2 ms on a barrier that nothing completes, gives up and
    # records it; the host reads FLY_ERR_TIMEOUT once, and the next fused step is correct again
    st = torch.cuda.current_stream().cuda_stream
    fv = FlyVerify(4, 8, 2048, "bf16", hidden=256)
    assert fv.device_status(st) == Bd.FLY_OK
    assert fv.selftest_wait(st) == Bd.FLY_OK
    assert fv.device_status(st) == Bd.FLY_ERR_TIMEOUT
    assert fv.device_status(st) == Bd.FLY_OK                      # the record was cleared
    # While a record is pending a fused step gives up early (every wait returns at once) and marks all of its rows:
    # the failure shows in the step's own outputs, in stream order, before anybody asks for the status.
    w, hidden, weight, draft, logits = fused_case(4, 8, 256, 2048)
    out = VerifyBuffers(4, 8, DEV)
    assert fv.selftest_wait(st) == Bd.FLY_OK
    verify_fused(fv, hidden, weight, draft, out, stream=st)
    torch.cuda.synchronize()
    assert (out.row_flags & 16).all() and (out.accept_len == 1).all()
    assert fv.device_status(st) == Bd.FLY_ERR_TIMEOUT and fv.device_status(st) == Bd.FLY_OK
    verify_fused(fv, hidden, weight, draft, out, stream=st)       # and the handle is as good as new
    assert fv.device_status(st) == Bd.FLY_OK
    assert_parity(out, O.verify_batch(logits.reshape(4, 9, 2048), draft.cpu().numpy(), 1.0, 3), "after a reported timeout")
    fv.close()
    run_and_check(4, 8, D=256, V=2048)


def test_seeded_fuzz_over_fused_shapes():
    import random
    rng = random.Random(22972)
    for case in range(24):
        B, K = rng.randint(1, 24), rng.randint(1, 15)
        D = 8 * rng.randint(8, 160)                      # 64 .. 1280, any multiple of 8 (ragged last k-block)
        V = 8 * rng.randint(16, 3000)                    # 128 .. 24000 (ragged last vocabulary tile, few or many tiles)
        theta, W = rng.choice([0.5, 1.0, 3.0]), rng.randint(0, K)
        boundary = rng.choice(["reject", "carry"])
        state = [[rng.randint(0, min(W, K)), 2, 5] for _ in range(B)] if boundary == "carry" else None
        run_and_check(B, K, D, V, theta=theta, W=W, boundary=boundary, state=state, step=case)


@pytest.mark.parametrize("D,V", [(64, 128), (512, 4096), (200, 1000), (1024, 19000)])
def test_weight_stored_vocabulary_major(D, V):
    # the same step with the weight stored [V, hidden] (the usual layout of a linear layer's parameter)
    B, K = 4, 8
    w, hidden, weight, draft, logits = fused_case(B, K, D, V, step=7)
    fv = FlyVerify(B, K, V, "bf16", hidden=D)
    fv.set_weight_layout(True)
    out = VerifyBuffers(B, K, DEV)
    st = torch.cuda.current_stream().cuda_stream
    verify_fused(fv, hidden, weight.t().contiguous(), draft, out, stream=st)
    assert fv.device_status(st) == Bd.FLY_OK
    ref = O.verify_batch(logits.reshape(B, K + 1, V), draft.cpu().numpy(), 1.0, 3)
    assert_parity(out, ref, f"[V, D] weight D={D} V={V}")
    fv.set_weight_layout(False)                                   # and back, on the same handle
    verify_fused(fv, hidden, weight, draft, out, stream=st)
    torch.cuda.synchronize()
    assert_parity(out, ref, f"[D, V] weight D={D} V={V}")
