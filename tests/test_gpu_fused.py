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


def fused_case(B, K, D, V, step=0, weight_std=None, theta=1.0, min_gap=1e-3, guard=1e-3):
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
        H = O.row_stats(logits)[0]
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


def run_and_check(B, K, D, V, theta=1.0, W=3, boundary="reject", state=None, **kw):
    w, hidden, weight, draft, logits = fused_case(B, K, D, V, theta=theta, **kw)
    fv = FlyVerify(B, K, V, "bf16", hidden=D)
    out = VerifyBuffers(B, K, DEV)
    if state is not None:
        out.state.copy_(torch.as_tensor(state, dtype=torch.int32))
    verify_fused(fv, hidden, weight, draft, out, theta=theta, W=W, boundary=boundary,
                 stream=torch.cuda.current_stream().cuda_stream)
    assert fv.device_status(torch.cuda.current_stream().cuda_stream) == Bd.FLY_OK
    ref = O.verify_batch(logits.reshape(B, K + 1, V), draft.cpu().numpy(), theta, W, boundary=boundary,
                         state_in=None if state is None else np.asarray(state))
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


def test_full_size_head_on_sampled_sequences():
    """The Llama-3.1-70B head shape of the benchmark (288 positions x 8192 x 128256), in the launch
    configuration the benchmark times.  The oracle cannot form all 288 x 128256 fp64 logits in seconds, so
    two whole sequences (18 rows) are verified exactly and the rest is checked through properties."""
    w = S.FUSED
    B, K, V, D = w.B, w.K, w.V, w.hidden
    weight = S.make_weight(w, device=DEV)
    hidden = S.make_hidden(w, 0, device=DEV)
    sample = [3, 20]
    hs = hidden.view(B, K + 1, D)[sample].reshape(-1, D).double().cpu().numpy()
    wc = weight.cpu()
    parts = [O.lm_head_logits(hs, wc[:, v0:v0 + 16032].double().numpy()) for v0 in range(0, V, 16032)]
    logits = np.concatenate(parts, axis=1)                       # [18, V] fp64
    top2 = np.partition(logits, V - 2, axis=1)[:, V - 2:]
    assert (top2[:, 1] - top2[:, 0]).min() >= 1e-3, "redraw: two logits of a sampled row are too close"
    y = logits.argmax(axis=1).reshape(len(sample), K + 1)
    g = torch.Generator().manual_seed(7)
    draft = torch.randint(0, V, (B, K), generator=g, dtype=torch.int32)
    for n, b in enumerate(sample):                               # the oracle's token with p = 0.7, else uniform
        keep = torch.rand(K, generator=g) < 0.7
        draft[b, keep] = torch.as_tensor(y[n, :K], dtype=torch.int32)[keep]
    draft = draft.to(DEV)
    fv = FlyVerify(B, K, V, "bf16", hidden=D)
    out = VerifyBuffers(B, K, DEV)
    st = torch.cuda.current_stream().cuda_stream
    verify_fused(fv, hidden, weight, draft, out, theta=w.theta, W=w.W, stream=st)
    assert fv.device_status(st) == Bd.FLY_OK
    assert fv.last_launch_count == 3
    ref = O.verify_batch(logits.reshape(len(sample), K + 1, V), draft[sample].cpu().numpy(), w.theta, w.W)
    assert np.array_equal(out.target_argmax[sample].cpu().numpy(), ref.target_argmax)
    assert np.abs(out.entropy[sample].double().cpu().numpy() - ref.entropy).max() <= 1e-4
    assert np.array_equal(out.accept_len[sample].cpu().numpy(), ref.accept_len)
    assert np.array_equal(out.out_tokens[sample].cpu().numpy(), ref.out_tokens)
    # every sequence: properties that hold whatever the logits are
    s = out.accept_len.cpu().numpy()
    toks = out.out_tokens.cpu().numpy()
    am = out.target_argmax.cpu().numpy()
    dr = draft.cpu().numpy()
    H = out.entropy.cpu().numpy()
    assert ((s >= 1) & (s <= K + 1)).all() and (out.row_flags == 0).all()
    assert ((H > 0) & (H <= np.log(V) + 1e-4)).all() and ((am >= 0) & (am < V)).all()
    for b in range(B):
        assert (toks[b, :s[b] - 1] == dr[b, :s[b] - 1]).all() and toks[b, s[b] - 1] == am[b, s[b] - 1]
        assert (toks[b, s[b]:] == -1).all()
        first_mismatch = next((i + 1 for i in range(K) if dr[b, i] != am[b, i]), K + 1)
        assert s[b] >= first_mismatch                              # s_FLy >= s_standard (Eq. 3 vs Eq. 11)


def test_a_wait_that_runs_out_is_reported_and_the_handle_stays_usable():
    # no fault, no hang: a one-thread kernel waits 2 ms on a barrier that nothing completes, gives up and
    # records it; the host reads FLY_ERR_TIMEOUT once, and the next fused step is correct again
    st = torch.cuda.current_stream().cuda_stream
    fv = FlyVerify(4, 8, 2048, "bf16", hidden=256)
    assert fv.device_status(st) == Bd.FLY_OK
    assert fv.selftest_wait(st) == Bd.FLY_OK
    assert fv.device_status(st) == Bd.FLY_ERR_TIMEOUT
    assert fv.device_status(st) == Bd.FLY_OK                      # the record was cleared
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
