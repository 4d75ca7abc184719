"""Helpers of the GPU parity tests: run the CUDA path (through the C ABI) and
the fp64 oracle on the same seeded inputs and compare element by element."""
import numpy as np
import torch

from oracle import fly_oracle as O
from paper_2511_22972_b200 import FlyVerify, VerifyBuffers, synthetic as S, verify

ENTROPY_TOL = 1e-4      # nats, absolute (fp32 accumulation against fp64)


def oracle_entropy(rows: torch.Tensor):
    return O.row_stats(rows.double().cpu().numpy())[0]


def draw(w, step=0, setting=0, device="cuda", thetas=None, guard=True, temperature=1.0):
    """Logits (entropies - at the given temperature - kept >= 1e-3 away from every threshold) and drafts."""
    ent = oracle_entropy if temperature == 1.0 else (lambda rows: O.row_stats(rows.double().cpu().numpy() / temperature)[0])
    logits = S.make_logits(w, step, device=device, setting=setting,
                           entropy_fn=ent if guard else None,
                           theta_nats=thetas if thetas is not None else w.theta)
    top5 = S.rank5(logits.view(-1, w.V))
    draft = S.make_draft(w, step, top5, setting=setting)
    return logits, draft


def gpu_step(fv, logits, draft, theta, W, boundary="reject", state=None, theta_unit="nats", host=False,
             temperature=0.0, inputs_ready=False):
    B, K1, V = logits.shape
    out = VerifyBuffers(B, K1 - 1, logits.device if not host else "cpu", pinned=host)
    if state is not None:
        out.state.copy_(torch.as_tensor(state, dtype=torch.int32))
    verify(fv, logits, draft, out, theta=theta, W=W, theta_unit=theta_unit, boundary=boundary,
           stream=torch.cuda.current_stream().cuda_stream, host=host, temperature=temperature,
           inputs_ready=inputs_ready)
    torch.cuda.synchronize()
    return out


def oracle_step(logits, draft, theta, W, boundary="reject", state=None, theta_unit="nats", temperature=1.0):
    B, K1, V = logits.shape
    x = logits.double().cpu().numpy()
    return O.verify_batch(x, draft.cpu().numpy(), theta, W, theta_unit=theta_unit, boundary=boundary,
                          state_in=None if state is None else np.asarray(state), temperature=temperature)


def assert_parity(out, ref, what=""):
    """Bit-exact integers; entropy within ENTROPY_TOL.  Sequences holding a
    flagged row only have to agree on the flags."""
    flags = out.row_flags.cpu().numpy().astype(np.uint32)
    assert np.array_equal(flags, ref.row_flags), \
        f"{what}: row_flags differ at {np.argwhere(flags != ref.row_flags).tolist()[:8]}: got {flags[flags != ref.row_flags][:8]}"
    ok = ~(ref.row_flags & O.FLAG_NONFINITE).any(axis=1)
    am = out.target_argmax.cpu().numpy()
    assert np.array_equal(am[ok], ref.target_argmax[ok]), f"{what}: argmax differs"
    H = out.entropy.cpu().numpy().astype(np.float64)
    err = np.abs(H[ok] - ref.entropy[ok])
    assert err.size == 0 or err.max() <= ENTROPY_TOL, f"{what}: entropy off by {err.max():.3e}"
    assert np.array_equal(out.accept_len.cpu().numpy()[ok], ref.accept_len[ok]), f"{what}: accept_len differs"
    assert np.array_equal(out.out_tokens.cpu().numpy()[ok], ref.out_tokens[ok]), f"{what}: out_tokens differ"
    assert np.array_equal(out.rollback.cpu().numpy()[ok], ref.rollback[ok]), f"{what}: rollback differs"
    assert np.array_equal(out.state.cpu().numpy()[ok], ref.state_out[ok]), f"{what}: state differs"
    return float(err.max()) if err.size else 0.0


def check(fv, logits, draft, theta, W, boundary="reject", state=None, theta_unit="nats", what="", host=False,
          temperature=0.0, inputs_ready=False):
    out = gpu_step(fv, logits, draft, theta, W, boundary, state, theta_unit, host=host, temperature=temperature,
                   inputs_ready=inputs_ready)
    ref = oracle_step(logits, draft, theta, W, boundary, state, theta_unit, temperature=temperature or 1.0)
    return assert_parity(out, ref, what), out, ref
