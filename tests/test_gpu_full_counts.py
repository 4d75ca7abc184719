"""The bench workloads at FULL size over as many of their configured steps as a time budget allows (all of them on a
16-core host): 1000 independent steps of the Llama-3 vocab batch, 500 steps of one long-draft setting, 512 chained rounds
of the serving workload with the deferred state carried from round to round.

The fp64 oracle does ~1.2 k rows/s per core, so its side runs in worker processes (sequences are independent: every
worker verifies its own sequences with the single-threaded oracle) while the GPU works ahead.  Nothing the oracle
reads comes from the CUDA path: inputs are the generator's, and in the chained workload every worker carries the
ORACLE's own state of its sequences from round to round.

Timing inputs are drawn without the entropy guard (a redraw would need the oracle's entropies first); a sequence one of
whose drafted rows has an oracle entropy within 1e-3 nats of the threshold is compared on its row statistics only
(argmax, entropy, flags) - the gate decision there is a coin flip between fp32 and fp64 - and from then on, in the
chained workload, that sequence's later rounds are left out (its two states may differ legitimately).
"""
import multiprocessing as mp
import os
import time

import numpy as np
import pytest
import torch

from paper_2511_22972_b200 import FlyVerify, VerifyBuffers, synthetic as S, verify

pytestmark = pytest.mark.gpu
DEV = "cuda"
BUDGET_S = float(os.environ.get("FLY_FULL_COUNT_SECONDS", "60"))
GUARD = 1e-3
ENTROPY_TOL = 1e-4


def _oracle_job(job):
    """Worker: bf16 / fp32 bits -> exactly widened fp64 -> the oracle."""
    from oracle import fly_oracle as O
    bits, is_bf16, draft, theta, W, boundary, state = job
    if is_bf16:
        x = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    else:
        x = bits.astype(np.float64)
    r = O.verify_batch(x, draft, theta, W, boundary=boundary, state_in=state)
    return r.accept_len, r.rollback, r.out_tokens, r.target_argmax, r.entropy, r.row_flags, r.state_out


def _host_bits(logits):
    t = logits.cpu()
    return t.view(torch.int16).numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.numpy()


def _compare(out, ref, seqs, theta, K, alive, what):
    """out: dict of numpy arrays for all sequences of a step; ref: oracle tuple for the sequences `seqs`."""
    acc, rb, toks, am, H, flags, st = ref
    assert np.array_equal(out["row_flags"][seqs], flags), f"{what}: flags"
    assert np.array_equal(out["target_argmax"][seqs], am), f"{what}: argmax"
    err = np.abs(out["entropy"][seqs].astype(np.float64) - H).max()
    assert err <= ENTROPY_TOL, f"{what}: entropy off by {err:.2e}"
    near = (np.abs(H[:, :K] - theta) < GUARD).any(axis=1)
    ok = alive[seqs] & ~near
    for name, want in (("accept_len", acc), ("rollback", rb), ("out_tokens", toks), ("state", st)):
        assert np.array_equal(out[name][seqs][ok], want[ok]), f"{what}: {name}"
    return near, err


def run_full(w, steps, theta, W, setting=0, chained=False, min_steps=20):
    cores = len(os.sched_getaffinity(0))
    groups = min(cores, w.B)
    cuts = [round(i * w.B / groups) for i in range(groups + 1)]
    fv = FlyVerify(w.B, w.K, w.V, w.dtype)
    st = torch.cuda.current_stream().cuda_stream
    is_bf16 = w.dtype == "bf16"
    state_dev = torch.tensor([[0, 0, -1]] * w.B, dtype=torch.int32, device=DEV)
    oracle_state = [np.array([[0, 0, -1]] * (b - a), dtype=np.int32) for a, b in zip(cuts, cuts[1:])]
    alive = np.ones(w.B, dtype=bool)
    names = ("accept_len", "rollback", "out_tokens", "target_argmax", "entropy", "row_flags", "state")
    pending = []            # (step, outputs, [async results per group])
    worst, unguarded, done = 0.0, 0, 0
    t_start = time.time()

    def settle(item):
        nonlocal worst, unguarded, done
        step, out, futs = item
        for g, fut in enumerate(futs):
            ref = fut.get()
            seqs = slice(cuts[g], cuts[g + 1])
            near, err = _compare(out, ref, seqs, theta, w.K, alive, f"{w.name} step {step} sequences {cuts[g]}..{cuts[g + 1] - 1}")
            worst = max(worst, err)
            unguarded += int(near.sum())
            if chained:
                oracle_state[g] = ref[6]
                alive[seqs] &= ~near
        done += 1

    with mp.get_context("forkserver").Pool(groups) as pool:   # a clean server process forks the workers, not this CUDA process
        for step in range(steps):
            logits = S.make_logits(w, step, device=DEV, setting=setting)
            draft = S.make_draft(w, step, S.rank5(logits.view(-1, w.V)), setting=setting)
            out = VerifyBuffers(w.B, w.K, DEV)
            if chained:
                out.state = state_dev                    # read and written in place: carried to the next round
            verify(fv, logits, draft, out, theta=theta, W=W, boundary=w.boundary, stream=st)
            torch.cuda.synchronize()
            host = {n: getattr(out, n).cpu().numpy().copy() for n in names}
            host["row_flags"] = host["row_flags"].astype(np.uint32)
            bits, dr = _host_bits(logits), draft.cpu().numpy()
            if chained and pending:                      # the oracle's state of round r - 1 feeds its round r
                settle(pending.pop(0))
            futs = [pool.apply_async(_oracle_job, ((bits[a:b], is_bf16, dr[a:b], theta, W, w.boundary,
                                                    oracle_state[g] if chained else None),))
                    for g, (a, b) in enumerate(zip(cuts, cuts[1:]))]
            pending.append((step, host, futs))
            while len(pending) > (1 if chained else 3):
                settle(pending.pop(0))
            if time.time() - t_start > BUDGET_S and step + 1 >= min_steps:
                break
        while pending:
            settle(pending.pop(0))
    fv.close()
    print(f"{w.name}: {done} of {steps} steps compared at full size in {time.time() - t_start:.0f} s on {groups} cores; "
          f"max |dH| {worst:.2e}; {unguarded} sequence-steps within {GUARD} nats of the threshold (statistics only); "
          f"{int(alive.sum())} of {w.B} sequences compared to the end")
    assert done >= min(min_steps, steps)
    return done


def test_llama3_vocab_batch_as_many_of_its_1000_steps_as_the_budget_allows():
    w = S.LLAMA3
    run_full(w, w.steps, w.theta, w.W)


def test_long_draft_batch_as_many_of_its_500_steps_as_the_budget_allows():
    w = S.LONG_DRAFT
    theta, W = S.LONG_DRAFT_SETTINGS[4]
    run_full(w, w.steps, theta, W, setting=4, min_steps=5)


def test_high_batch_serving_as_many_of_its_512_chained_rounds_as_the_budget_allows():
    w = S.SERVING
    run_full(w, w.steps, w.theta, w.W, chained=True, min_steps=5)
