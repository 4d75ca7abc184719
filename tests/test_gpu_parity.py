"""Parity of the CUDA path (called through the C ABI) with the fp64 oracle:
bit-exact argmax / accept lengths / tokens / state, entropy within 1e-4 nats."""
import math

import numpy as np
import pytest
import torch

from oracle import fly_oracle as O
from paper_2511_22972_b200 import FlyVerify, synthetic as S
from tests._parity import assert_parity, check, draw, gpu_step, oracle_step

pytestmark = pytest.mark.gpu
DEV = "cuda"


def small(dtype, B, K, V, **kw):
    base = S.TINY if dtype == "f32" else S.LLAMA3
    return S.shrink(base, B=B, K=K, V=V, **kw)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 2, 7, 33, 257, 1000, 4097, 8200])
def test_small_and_odd_vocabularies(dtype, V):
    # below one warp slice, odd lengths (element-wise path), and just past a vector slice
    for K in (1, 2, 4):
        w = small(dtype, B=3, K=K, V=V)
        fv = FlyVerify(w.B, K, V, dtype)
        logits, draft = draw(w, step=K, guard=V > 1)
        check(fv, logits, draft, theta=1.0 if V > 4 else 0.3, W=1, what=f"{dtype} V={V} K={K}")
        fv.close()


@pytest.mark.parametrize("dtype,V", [("bf16", 128256), ("bf16", 152064), ("f32", 32000), ("bf16", 50257), ("f32", 50257)])
@pytest.mark.parametrize("splits", [0, 1, 3, 8, 31])
def test_row_splitting_does_not_change_results(dtype, V, splits):
    # several slices per warp, a ragged last slice, every split count incl. ones that do not divide V
    w = small(dtype, B=2, K=3, V=V)
    fv = FlyVerify(w.B, w.K, V, dtype)
    fv.set_splits(splits)
    logits, draft = draw(w, step=1)
    check(fv, logits, draft, theta=1.0, W=2, what=f"{dtype} V={V} splits={splits}")
    fv.close()


def test_ties_pick_the_lowest_index_across_lanes_warps_and_blocks():
    V = 128256
    w = small("bf16", B=1, K=7, V=V)
    fv = FlyVerify(1, 7, V, "bf16")
    logits, draft = draw(w, step=3, guard=False)
    g = torch.Generator().manual_seed(5)
    rows = logits.view(-1, V)
    for r in range(rows.shape[0]):
        top = rows[r].float().max().item() + 1.0
        n = int(torch.randint(2, 9, (1,), generator=g))
        where = torch.randint(0, V, (n,), generator=g)
        if r == 0:
            where = torch.tensor([V - 1, 7, 8])            # same 16-byte segment and the very last element
        if r == 1:
            where = torch.tensor([1024 * 8 + 3, 1024 * 8 * 5 + 3])   # different slices of one warp
        rows[r, where.to(DEV)] = top
    for splits in (0, 1, 5):
        fv.set_splits(splits)
        out = gpu_step(fv, logits, draft, 1.0, 3)
        ref = oracle_step(logits, draft, 1.0, 3)
        assert np.array_equal(out.target_argmax.cpu().numpy(), ref.target_argmax)
    # bf16 rows of Gaussians tie at the top on their own
    x = (torch.randn(64, V, generator=torch.Generator().manual_seed(1)) * 2).to(torch.bfloat16)
    tied = (x.float() == x.float().max(dim=1, keepdim=True).values).sum(dim=1)
    assert (tied > 1).any()
    fv2 = FlyVerify(8, 7, V, "bf16")
    lg = x.view(8, 8, V).to(DEV)
    dr = torch.zeros(8, 7, dtype=torch.int32, device=DEV)
    out = gpu_step(fv2, lg, dr, 1.0, 3)
    ref = oracle_step(lg, dr, 1.0, 3)
    assert np.array_equal(out.target_argmax.cpu().numpy(), ref.target_argmax)


def test_masked_and_nonfinite_logits_and_bad_drafts():
    V = 4096 + 24
    w = small("bf16", B=6, K=3, V=V)
    for dtype in ("bf16", "f32"):
        w = small(dtype, B=6, K=3, V=V)
        fv = FlyVerify(w.B, w.K, V, dtype)
        logits, draft = draw(w, step=2, guard=False)
        logits[0, 1, 100:3000] = -math.inf          # masked vocabulary range: allowed
        logits[1, 0, 17] = math.nan
        logits[2, 2, V - 1] = math.inf
        logits[3, 3, :] = -math.inf                 # nothing finite
        logits[4, 1, :] = -math.inf
        logits[4, 1, 2000] = 0.5                    # one-hot: entropy exactly 0
        draft[5, 0] = V                             # out of vocabulary
        draft[5, 2] = -1
        # redraw drafts of the masked rows against the edited logits
        out = gpu_step(fv, logits, draft, 0.5, 1)
        ref = oracle_step(logits, draft, 0.5, 1)
        assert ref.row_flags[1, 0] == 1 and ref.row_flags[2, 2] == 1 and ref.row_flags[3, 3] == 1
        assert ref.row_flags[5, 0] == 2 and ref.row_flags[5, 2] == 2 and ref.row_flags[0].sum() == 0
        assert_parity(out, ref, dtype)
        assert out.entropy[4, 1].item() == 0.0 and out.target_argmax[4, 1].item() == 2000
        toks = out.out_tokens.cpu().numpy()
        assert ((toks >= -1) & (toks < V)).all()     # nothing out of range is ever emitted
        fv.close()


def test_strided_rows_and_unaligned_base():
    V = 5000
    w = small("bf16", B=2, K=2, V=V)
    logits, draft = draw(w, step=4)
    fv = FlyVerify(2, 2, V, "bf16")
    # rows 5008 elements apart (16-byte multiple): vector path with a stride
    wide = torch.full((2, 3, 5008), 99.0, dtype=torch.bfloat16, device=DEV)
    wide[:, :, :V] = logits
    check(fv, wide[:, :, :V], draft, 1.0, 1, what="strided")
    # base pointer off by one element: element-wise path
    flat = torch.zeros(2 * 3 * V + 1, dtype=torch.bfloat16, device=DEV)
    off = flat[1:].view(2, 3, V)
    off.copy_(logits)
    assert off.data_ptr() % 16 != 0
    check(fv, off, draft, 1.0, 1, what="unaligned")


def test_theta_units_and_limits():
    V = 32000
    w = small("f32", B=4, K=8, V=V)
    fv = FlyVerify(4, 8, V, "f32")
    th_norm = 0.3
    logits, draft = draw(w, step=9, thetas=[th_norm * math.log(V), 1.0])
    check(fv, logits, draft, th_norm, 3, theta_unit="normalized", what="normalized theta")
    # theta = +inf: exact-match acceptance (Eq. 3)
    _, out, ref = check(fv, logits, draft, math.inf, 3, what="theta=inf")
    for b in range(4):
        delta = O.match_indicator(draft[b].tolist(), ref.target_argmax[b, :8])
        assert out.accept_len[b].item() == O.s_standard(delta)
    # theta = 0, W = 0: everything accepted
    _, out, _ = check(fv, logits, draft, 0.0, 0, what="theta=0 W=0")
    assert (out.accept_len == 9).all()
    # very long windows behave like W = K+1
    check(fv, logits, draft, 1.0, 1000, what="W=1000")


@pytest.mark.parametrize("K", [1, 15, 25, 31, 32, 47, 63])
def test_draft_lengths_up_to_63(K):
    V = 2048
    w = small("bf16", B=5, K=K, V=V, draft_mix=(0.85, 0.1, 0.05))
    fv = FlyVerify(5, K, V, "bf16")
    logits, draft = draw(w, step=K, thetas=[0.5])
    for W in (0, 1, 6, K):
        check(fv, logits, draft, 0.5, W, what=f"K={K} W={W}")
        if W <= K:      # the carry extension needs the window to fit in one round
            check(fv, logits, draft, 0.5, W, boundary="carry", state=[[0, 0, -1]] * 5, what=f"carry K={K} W={W}")


def test_carry_chain_many_rounds_reduced_vocab():
    # the serving recipe at reduced V, state chained over 512 rounds
    w = S.shrink(S.SERVING, B=32, K=8, V=4096)
    fv = FlyVerify(w.B, w.K, w.V, "bf16")
    state_gpu = [[0, 0, -1]] * w.B
    state_ref = np.array(state_gpu)
    seen = {"pending": 0, "revoke": 0}
    for rnd in range(512):
        logits, draft = draw(w, step=rnd)
        out = gpu_step(fv, logits, draft, w.theta, w.W, "carry", state_gpu)
        ref = oracle_step(logits, draft, w.theta, w.W, "carry", state_ref)
        assert_parity(out, ref, f"round {rnd}")
        state_gpu = out.state.cpu().numpy()
        state_ref = ref.state_out
        seen["pending"] += int((ref.state_out[:, 0] > 0).sum())
        seen["revoke"] += int((ref.rollback > 0).sum())
    assert seen["pending"] > 50 and seen["revoke"] > 10      # the extension's branches were exercised


def test_host_buffer_entry_point_matches_device_entry_point():
    w = small("bf16", B=4, K=8, V=128256)
    fv = FlyVerify(4, 8, w.V, "bf16")
    logits, draft = draw(w, step=0)
    _, out_d, ref = check(fv, logits, draft, 1.0, 3, what="device")
    lh = logits.cpu().pin_memory()
    dh = draft.cpu().pin_memory()
    out_h = gpu_step(fv, lh, dh, 1.0, 3, host=True)
    assert_parity(out_h, ref, "host")
    assert torch.equal(out_h.entropy, out_d.entropy.cpu())


def test_api_misuse_returns_error_codes():
    from paper_2511_22972_b200 import FlyError, VerifyBuffers, binding as Bd
    V = 1024
    fv = FlyVerify(2, 4, V, "bf16")
    logits = torch.zeros(2, 5, V, dtype=torch.bfloat16, device=DEV)
    draft = torch.zeros(2, 4, dtype=torch.int32, device=DEV)
    out = VerifyBuffers(2, 4, DEV)

    def run(**kw):
        base = dict(B=2, K=4, draft=draft, accept_len=out.accept_len, out_tokens=out.out_tokens, logits=logits,
                    state_out=out.state)
        base.update(kw)
        fv.run(fv.make_args(**base))

    run()
    for bad, code in [(dict(B=3), Bd.FLY_ERR_INVALID_ARG), (dict(K=5), Bd.FLY_ERR_INVALID_ARG),
                      (dict(B=0), Bd.FLY_ERR_INVALID_ARG), (dict(W=-1), Bd.FLY_ERR_INVALID_ARG),
                      (dict(draft=None), Bd.FLY_ERR_INVALID_ARG), (dict(logits=None), Bd.FLY_ERR_INVALID_ARG),
                      (dict(theta=math.nan), Bd.FLY_ERR_INVALID_ARG), (dict(row_stride=V - 8), Bd.FLY_ERR_INVALID_ARG),
                      (dict(boundary="carry", W=5), Bd.FLY_ERR_UNSUPPORTED),
                      (dict(boundary="carry", state_out=None), Bd.FLY_ERR_INVALID_ARG),
                      (dict(state_in=out.state), Bd.FLY_ERR_INVALID_ARG)]:
        with pytest.raises(FlyError) as e:
            run(**bad)
        assert e.value.status == code, bad
    torch.cuda.synchronize()
    run()                                                    # the handle is still usable
    torch.cuda.synchronize()
    assert fv.last_launch_count == 1                         # scan fused into the reduction's tail
    fv.set_scan_mode(True)
    run()
    assert fv.last_launch_count == 2                         # reduction + stand-alone scan
    for opt, val in [(0, 33), (0, -1), (1, 2), (2, 2), (2, -1), (3, 2), (9, 0)]:
        with pytest.raises(FlyError):
            fv.set_option(opt, val)


@pytest.mark.parametrize("separate", [False, True])
def test_both_scan_modes_agree_with_the_oracle(separate):
    w = small("bf16", B=24, K=8, V=128256)
    fv = FlyVerify(w.B, w.K, w.V, "bf16")
    fv.set_scan_mode(separate)
    for step in range(3):
        logits, draft = draw(w, step=step)
        for splits in (0, 1, 7):
            fv.set_splits(splits)
            check(fv, logits, draft, 1.0, 3, what=f"separate={separate} step={step} splits={splits}")
    # the per-sequence arrival counters must be back at zero: run a different batch size
    w2 = small("bf16", B=5, K=3, V=128256)
    logits, draft = draw(w2, step=7)
    fv.set_splits(0)
    check(fv, logits, draft, 1.0, 3, what="smaller batch after larger")


def test_back_to_back_steps_with_stream_overlap():
    # consecutive steps over resident inputs, the reduction of step n+1 allowed to start
    # reading while step n drains; every step keeps its own outputs
    from paper_2511_22972_b200 import VerifyBuffers, verify
    w = small("bf16", B=16, K=8, V=128256)
    fv = FlyVerify(w.B, w.K, w.V, "bf16")
    steps = [draw(w, step=s) for s in range(6)]
    outs = [VerifyBuffers(w.B, w.K, DEV) for _ in steps]
    st = torch.cuda.current_stream().cuda_stream
    torch.cuda.synchronize()                          # the inputs are complete before the first launch
    for rep in range(3):
        for (logits, draft), out in zip(steps, outs):
            verify(fv, logits, draft, out, theta=1.0, W=3, stream=st, inputs_ready=True)
    torch.cuda.synchronize()
    for (logits, draft), out in zip(steps, outs):
        assert_parity(out, oracle_step(logits, draft, 1.0, 3), "overlap")


@pytest.mark.parametrize("name", ["paper_default_70b", "paper_default_405b"])
@pytest.mark.parametrize("B", [1, 4, 16])
def test_paper_default_operating_point(name, B):
    # K = 15 / 25, W = 6, threshold 0.3 on the normalised entropy, small batches (few rows, many pieces per row)
    w = S.shrink(S.WORKLOADS[name], B=B)
    fv = FlyVerify(w.B, w.K, w.V, "bf16")
    logits, draft = draw(w, step=B)
    check(fv, logits, draft, w.theta, w.W, what=f"{name} B={B} nats")
    check(fv, logits, draft, 0.3, w.W, theta_unit="normalized", what=f"{name} B={B} normalized")
    torch.cuda.synchronize()
    check(fv, logits, draft, w.theta, w.W, what=f"{name} B={B} overlap", inputs_ready=True)


def test_caller_supplied_target_tokens():
    # the hook for sampled (temperature-1) target tokens: they replace the argmax in Eq. 2 and in the output
    from paper_2511_22972_b200 import VerifyBuffers
    w = small("bf16", B=12, K=8, V=32064)
    fv = FlyVerify(w.B, w.K, w.V, "bf16")
    logits, draft = draw(w, step=21)
    g = torch.Generator().manual_seed(3)
    y = logits.float().argmax(dim=2).to(torch.int32).cpu()
    tt = y.clone()
    resample = torch.rand(tt.shape, generator=g) < 0.3
    tt[resample] = torch.randint(0, w.V, (int(resample.sum()),), generator=g, dtype=torch.int32)
    agree = torch.rand(w.B, w.K, generator=g) < 0.3           # the sample sometimes agrees with the draft
    tt[:, :w.K][agree] = draft.cpu()[agree]
    tt[3, 2] = w.V                                            # out of range: flagged, never accepted
    tt[5, w.K] = -2
    tt = tt.to(DEV)
    st = torch.cuda.current_stream().cuda_stream
    for boundary, state in (("reject", None), ("carry", [[1, 2, 5]] * w.B)):
        out = VerifyBuffers(w.B, w.K, DEV)
        if state is not None:
            out.state.copy_(torch.as_tensor(state, dtype=torch.int32))
        a = fv.make_args(w.B, w.K, draft, out.accept_len, out.out_tokens, logits=logits, theta=1.0, W=3,
                         boundary=boundary, state_in=out.state if state is not None else None, state_out=out.state,
                         rollback=out.rollback, target_argmax=out.target_argmax, entropy=out.entropy,
                         row_flags=out.row_flags, target_tokens=tt)
        fv.run(a, st)
        torch.cuda.synchronize()
        ref = O.verify_batch(logits.double().cpu().numpy(), draft.cpu().numpy(), 1.0, 3, boundary=boundary,
                             state_in=None if state is None else np.asarray(state), target_tokens=tt.cpu().numpy())
        assert ref.row_flags[3, 2] == 4 and ref.row_flags[5, w.K] == 4
        assert_parity(out, ref, f"target tokens {boundary}")


def _guarded(shape, dtype, fill):
    """A tensor with 64 canary elements on either side of the part handed to the library."""
    n = int(np.prod(shape))
    raw = torch.full((n + 128,), fill, dtype=dtype, device=DEV)
    return raw, raw[64:64 + n].view(*shape)


def test_nothing_is_written_outside_the_output_buffers():
    from paper_2511_22972_b200 import VerifyBuffers, verify, verify_fused
    B, K = 5, 7
    for fused in (False, True):
        V = 32064 if not fused else 2048
        out = VerifyBuffers(B, K, DEV)
        raws = {}
        for name, dtype, fill in [("accept_len", torch.int32, 12345), ("rollback", torch.int32, 12345),
                                  ("out_tokens", torch.int32, 12345), ("target_argmax", torch.int32, 12345),
                                  ("entropy", torch.float32, 777.0), ("row_flags", torch.int32, 12345),
                                  ("state", torch.int32, 12345)]:
            raw, view = _guarded(tuple(getattr(out, name).shape), dtype, fill)
            raws[name] = (raw, fill)
            setattr(out, name, view)
        st = torch.cuda.current_stream().cuda_stream
        if not fused:
            w = small("bf16", B=B, K=K, V=V)
            fv = FlyVerify(B, K, V, "bf16")
            logits, draft = draw(w, step=31)
            for splits in (0, 1, 5):
                fv.set_splits(splits)
                verify(fv, logits, draft, out, stream=st)
        else:
            w = S.shrink(S.FUSED, B=B, K=K, V=V, hidden=256, weight_std=0.1)
            fv = FlyVerify(B, K, V, "bf16", hidden=256)
            verify_fused(fv, S.make_hidden(w, 0, device=DEV), S.make_weight(w, device=DEV),
                         torch.zeros(B, K, dtype=torch.int32, device=DEV), out, stream=st)
        torch.cuda.synchronize()
        for name, (raw, fill) in raws.items():
            assert (raw[:64] == fill).all() and (raw[-64:] == fill).all(), f"{name}: canary overwritten (fused={fused})"
        s = out.accept_len
        assert ((s >= 1) & (s <= K + 1)).all()


def test_a_captured_step_replays_correctly():
    # fly_verify_run enqueues work only (no allocation, no synchronisation): it can be captured in a CUDA graph
    from paper_2511_22972_b200 import VerifyBuffers, verify
    w = small("bf16", B=8, K=8, V=128256)
    fv = FlyVerify(w.B, w.K, w.V, "bf16")
    logits, draft = draw(w, step=41)
    out = VerifyBuffers(w.B, w.K, DEV)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        verify(fv, logits, draft, out, stream=stream.cuda_stream)      # warm-up outside capture
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            verify(fv, logits, draft, out, stream=stream.cuda_stream)
        logits2, draft2 = draw(w, step=42)
        logits.copy_(logits2)                                          # new inputs in the captured buffers
        draft.copy_(draft2)
        out.accept_len.fill_(-1)
        g.replay()
        stream.synchronize()
    torch.cuda.synchronize()
    assert_parity(out, oracle_step(logits, draft, 1.0, 3), "graph replay")


def test_seeded_fuzz_over_shapes_options_and_boundary_modes():
    # 80 random small steps: shapes, dtypes, strides, thresholds, windows, split counts, scan modes, carried state
    import random
    rng = random.Random(2511)
    for case in range(80):
        dtype = rng.choice(["bf16", "f32"])
        B, K = rng.randint(1, 9), rng.randint(1, 20)
        V = rng.choice([3, 17, 64, 255, 1024, 4099, 9000, 33000])
        w = small(dtype, B=B, K=K, V=V, draft_mix=(0.7, 0.2, 0.1))
        theta = rng.choice([0.05, 0.5, 1.0, 2.5])
        W = rng.randint(0, K)
        boundary = rng.choice(["reject", "carry"])
        logits, draft = draw(w, step=1000 + case, thetas=[theta], guard=V > 4)
        pad = rng.choice([0, 0, 8, 24])
        if pad:                                        # rows further apart than V elements
            wide = torch.zeros(B, K + 1, V + pad, dtype=logits.dtype, device=DEV)
            wide[:, :, :V] = logits
            logits = wide[:, :, :V]
        state = None
        if boundary == "carry":
            state = [[rng.randint(0, min(W, K)), rng.randint(1, K + 1), rng.randrange(V)] if rng.random() < 0.5
                     else [0, 0, -1] for _ in range(B)]
        fv = FlyVerify(B, K, V, dtype)
        fv.set_splits(rng.choice([0, 0, 1, 2, 5]))
        fv.set_scan_mode(rng.random() < 0.3)
        what = f"fuzz {case}: {dtype} B={B} K={K} V={V} theta={theta} W={W} {boundary} pad={pad}"
        if V <= 4:                                     # entropies may sit on the threshold: compare the row statistics only
            out = gpu_step(fv, logits, draft, theta, W, boundary, state)
            ref = oracle_step(logits, draft, theta, W, boundary, state)
            assert np.array_equal(out.target_argmax.cpu().numpy(), ref.target_argmax), what
            assert np.abs(out.entropy.cpu().numpy() - ref.entropy).max() <= 1e-4, what
        else:
            check(fv, logits, draft, theta, W, boundary=boundary, state=state, what=what)
        fv.close()


def test_many_sequences_and_a_very_long_vocabulary():
    # sizes at the far ends: 4096 sequences (16384 rows, one arrival counter each), and a 1M-entry vocabulary
    w = small("bf16", B=4096, K=3, V=1000)
    fv = FlyVerify(w.B, w.K, w.V, "bf16")
    logits, draft = draw(w, step=51)
    check(fv, logits, draft, 1.0, 2, what="B=4096")
    check(fv, logits, draft, 1.0, 2, boundary="carry", state=[[b % 3, 2, 7] for b in range(w.B)], what="B=4096 carry")
    fv.close()
    V = (1 << 20) + 8
    w = small("bf16", B=2, K=1, V=V)
    fv = FlyVerify(w.B, w.K, V, "bf16")
    logits, draft = draw(w, step=52)
    for splits in (0, 1, 31):
        fv.set_splits(splits)
        check(fv, logits, draft, 1.0, 1, what=f"V=2^20+8 splits={splits}")
    rows = logits.view(-1, V)
    rows[1, :] = rows[1, 0]                      # a constant row: entropy = ln V exactly, argmax = 0 (first of all ties)
    out = gpu_step(fv, logits, draft, 1.0, 1)
    assert out.target_argmax.view(-1)[1].item() == 0
    assert abs(out.entropy.view(-1)[1].item() - math.log(V)) < 1e-4


@pytest.mark.parametrize("dtype,V", [("bf16", 128256), ("f32", 32000), ("bf16", 1001)])
@pytest.mark.parametrize("T", [0.7, 1.0, 1.5, 4.0])
def test_temperature_scaled_entropy(dtype, V, T):
    # the entropy of softmax(l / T): 1/T is folded into the exponent constant of every kernel and merge
    w = small(dtype, B=5, K=6, V=V)
    fv = FlyVerify(w.B, w.K, V, dtype)
    logits, draft = draw(w, step=int(T * 10), temperature=T)
    for splits in (0, 3):
        fv.set_splits(splits)
        err, out, ref = check(fv, logits, draft, w.theta, 2, temperature=T, what=f"{dtype} V={V} T={T} splits={splits}")
    plain = oracle_step(logits, draft, w.theta, 2)
    assert np.array_equal(ref.target_argmax, plain.target_argmax)          # the greedy token does not depend on T
    if T != 1.0:
        assert np.abs(ref.entropy - plain.entropy).max() > 1e-2           # ... the entropy does
    check(fv, logits.cpu().pin_memory(), draft.cpu().pin_memory(), w.theta, 2, temperature=T, host=True, what="host buffers")
    check(fv, logits, draft, 0.3, 2, theta_unit="normalized", temperature=T, what="normalised threshold")
    fv.close()


def test_temperature_argument_range():
    from paper_2511_22972_b200 import VerifyBuffers, binding as Bd
    w = small("bf16", B=1, K=2, V=1024)
    fv = FlyVerify(1, 2, 1024, "bf16")
    logits, draft = draw(w, guard=False)
    out = VerifyBuffers(1, 2, DEV)
    for T in (-1.0, 1e-9, 1e9, float("nan"), float("inf")):
        a = fv.make_args(1, 2, draft, out.accept_len, out.out_tokens, logits=logits, state_out=out.state, temperature=T)
        with pytest.raises(Bd.FlyError) as e:
            fv.run(a)
        assert e.value.status == Bd.FLY_ERR_INVALID_ARG
    a = fv.make_args(1, 2, draft, out.accept_len, out.out_tokens, logits=logits, state_out=out.state)
    a.inputs_ready = 2
    with pytest.raises(Bd.FlyError):
        fv.run(a)


def test_carried_state_that_the_library_never_writes_is_flagged_and_ignored():
    w = small("bf16", B=8, K=4, V=4096, boundary="carry")
    fv = FlyVerify(w.B, w.K, w.V, "bf16")
    logits, draft = draw(w, step=2)
    state = [[0, 0, -1], [5, 2, 1], [-1, 2, 1], [1, -3, 1], [2, 2, 4096], [1, 2, -1], [2, 3, 17], [4, 9, 4095]]
    err, out, ref = check(fv, logits, draft, 1.0, 3, boundary="carry", state=state, what="bad carried state")
    flags = out.row_flags.cpu().numpy()
    assert (flags[[1, 2, 3, 4, 5], 0] & 8).all() and not (flags[[0, 6, 7], 0] & 8).any()
    toks = out.out_tokens.cpu().numpy()
    assert toks.max() < w.V and toks.min() >= -1 and (out.rollback.cpu().numpy() >= 0).all()


@pytest.mark.parametrize("dtype,B,K,V", [("bf16", 50, 7, 128256), ("bf16", 100, 6, 128256), ("f32", 100, 3, 32000),
                                         ("bf16", 64, 9, 50264)])
def test_rows_packed_end_to_end(dtype, B, K, V):
    # row counts for which whole rows would leave most of a wave of blocks empty: the rows are laid end to end and cut
    # into equal block ranges, so blocks start and end in the middle of rows and cover several pieces
    from paper_2511_22972_b200 import binding as Bd
    w = small(dtype, B=B, K=K, V=V)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    p = Bd.plan(sms, w.rows, V, dtype)
    assert p.row_span == p.units_per_row and p.units_per_row % p.units_per_block != 0, "this shape is meant to be packed"
    fv = FlyVerify(B, K, V, dtype)
    logits, draft = draw(w, step=B)
    check(fv, logits, draft, 1.0, 2, what=f"packed rows {dtype} rows={w.rows} V={V}")
    check(fv, logits, draft, 1.0, 2, what="packed rows, scan as a kernel of its own") if fv.set_scan_mode(True) is None else None
    fv.close()


def test_two_handles_on_two_streams_at_once():
    # a handle owns its scratch: two handles may run concurrently on two streams without disturbing each other
    from paper_2511_22972_b200 import VerifyBuffers, verify
    wa = small("bf16", B=16, K=8, V=128256)
    wb = small("f32", B=7, K=5, V=32000)
    fa, fb = FlyVerify(wa.B, wa.K, wa.V, "bf16"), FlyVerify(wb.B, wb.K, wb.V, "f32")
    ins_a = [draw(wa, step=s) for s in range(4)]
    ins_b = [draw(wb, step=s) for s in range(4)]
    outs_a = [VerifyBuffers(wa.B, wa.K, DEV) for _ in ins_a]
    outs_b = [VerifyBuffers(wb.B, wb.K, DEV) for _ in ins_b]
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for rep in range(20):
        for (la, da), oa, (lb, db), ob in zip(ins_a, outs_a, ins_b, outs_b):
            verify(fa, la, da, oa, theta=1.0, W=3, stream=sa.cuda_stream, inputs_ready=rep % 2 == 1)
            verify(fb, lb, db, ob, theta=1.0, W=2, stream=sb.cuda_stream)
    torch.cuda.synchronize()
    for (la, da), oa in zip(ins_a, outs_a):
        assert_parity(oa, oracle_step(la, da, 1.0, 3), "stream a")
    for (lb, db), ob in zip(ins_b, outs_b):
        assert_parity(ob, oracle_step(lb, db, 1.0, 2), "stream b")
    fa.close()
    fb.close()
