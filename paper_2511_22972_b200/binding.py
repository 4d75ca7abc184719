"""ctypes binding of the C ABI in include/fly_verify.h.

Argument marshalling only: every step of the verification runs in the CUDA
kernels of libfly_verify.so.  There is no CPU fallback; a missing library that
cannot be built raises ImportError.
"""
from __future__ import annotations

import ctypes as C
import math
from typing import Optional

from . import build as _build

FLY_OK, FLY_ERR_INVALID_ARG, FLY_ERR_UNSUPPORTED, FLY_ERR_CUDA, FLY_ERR_TIMEOUT, FLY_ERR_TOO_LARGE = range(6)
FLY_STATIC_MAX_BATCH, FLY_STATIC_MAX_PIECES = 1024, 16384
FLY_F32, FLY_BF16 = 0, 1
FLY_THETA_NATS, FLY_THETA_NORMALIZED = 0, 1
FLY_BOUNDARY_REJECT, FLY_BOUNDARY_CARRY = 0, 1
FLY_OPT_SPLITS, FLY_OPT_SCAN_MODE, FLY_OPT_WEIGHT_LAYOUT = 0, 1, 3

EXPORTS = (
    "fly_verify_create", "fly_verify_destroy", "fly_verify_run", "fly_verify_run_host", "fly_verify_run_static",
    "fly_verify_device_status", "fly_verify_selftest_wait", "fly_verify_reduce_shard", "fly_verify_run_partials",
    "fly_pld_draft", "fly_verify_plan",
    "fly_verify_set_option", "fly_verify_last_launch_count", "fly_verify_last_cuda_error",
    "fly_status_string",
)


class fly_verify_config_t(C.Structure):
    _fields_ = [("device", C.c_int32), ("max_batch", C.c_int32), ("max_k", C.c_int32),
                ("vocab", C.c_int32), ("logits_dtype", C.c_int), ("hidden", C.c_int32)]


class fly_verify_args_t(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("K", C.c_int32),
        ("logits", C.c_void_p), ("row_stride", C.c_int64),
        ("hidden", C.c_void_p), ("weight", C.c_void_p),
        ("draft", C.c_void_p),
        ("theta", C.c_double), ("theta_unit", C.c_int), ("W", C.c_int32), ("boundary", C.c_int),
        ("state_in", C.c_void_p), ("state_out", C.c_void_p),
        ("accept_len", C.c_void_p), ("rollback", C.c_void_p), ("out_tokens", C.c_void_p),
        ("target_argmax", C.c_void_p), ("entropy", C.c_void_p), ("row_flags", C.c_void_p),
        ("target_tokens", C.c_void_p),
        ("temperature", C.c_double), ("inputs_ready", C.c_int32),
    ]


class fly_plan_t(C.Structure):
    _fields_ = [("grid", C.c_int32), ("slots", C.c_int32), ("units_per_block", C.c_int64), ("units_per_row", C.c_int64),
                ("row_span", C.c_int64)]


class FlyError(RuntimeError):
    def __init__(self, status: int, what: str, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        super().__init__(f"{what}: {status_string(status)} (status {status}, cuda error {cuda_error})")


_lib = None


def lib() -> C.CDLL:
    """Loads (building first if a source is newer) libfly_verify.so."""
    global _lib
    if _lib is not None:
        return _lib
    try:
        path = _build.ensure_built()
        L = C.CDLL(path)
    except Exception as e:  # no silent fallback: the CUDA library is the product
        raise ImportError(f"libfly_verify.so is missing and could not be built: {e}") from e
    L.fly_verify_create.argtypes = [C.POINTER(fly_verify_config_t), C.POINTER(C.c_void_p)]
    L.fly_verify_create.restype = C.c_int
    L.fly_verify_destroy.argtypes = [C.c_void_p]
    L.fly_verify_destroy.restype = C.c_int
    L.fly_verify_run.argtypes = [C.c_void_p, C.POINTER(fly_verify_args_t), C.c_void_p]
    L.fly_verify_run.restype = C.c_int
    L.fly_verify_run_host.argtypes = [C.c_void_p, C.POINTER(fly_verify_args_t), C.c_void_p]
    L.fly_verify_run_host.restype = C.c_int
    L.fly_verify_run_static.argtypes = [C.c_int32, C.c_int32, C.c_int, C.POINTER(fly_verify_args_t), C.c_void_p]
    L.fly_verify_run_static.restype = C.c_int
    L.fly_verify_device_status.argtypes = [C.c_void_p, C.c_void_p]
    L.fly_verify_device_status.restype = C.c_int
    L.fly_verify_selftest_wait.argtypes = [C.c_void_p, C.c_void_p]
    L.fly_verify_selftest_wait.restype = C.c_int
    L.fly_verify_reduce_shard.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int64, C.c_int32, C.c_double, C.c_void_p,
                                          C.c_void_p]
    L.fly_verify_reduce_shard.restype = C.c_int
    L.fly_verify_run_partials.argtypes = [C.c_void_p, C.POINTER(fly_verify_args_t), C.c_void_p, C.c_int32, C.c_int32,
                                          C.c_void_p]
    L.fly_verify_run_partials.restype = C.c_int
    L.fly_pld_draft.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    L.fly_pld_draft.restype = C.c_int
    L.fly_verify_plan.argtypes = [C.c_int32, C.c_int64, C.c_int32, C.c_int, C.c_int32, C.c_int32, C.c_int32,
                                  C.POINTER(fly_plan_t)]
    L.fly_verify_plan.restype = C.c_int
    L.fly_verify_set_option.argtypes = [C.c_void_p, C.c_int, C.c_int32]
    L.fly_verify_set_option.restype = C.c_int
    L.fly_verify_last_launch_count.argtypes = [C.c_void_p]
    L.fly_verify_last_launch_count.restype = C.c_int32
    L.fly_verify_last_cuda_error.argtypes = [C.c_void_p]
    L.fly_verify_last_cuda_error.restype = C.c_int32
    L.fly_status_string.argtypes = [C.c_int]
    L.fly_status_string.restype = C.c_char_p
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().fly_status_string(int(status)).decode()


def _ptr(t) -> Optional[int]:
    """Address of a torch tensor's storage (device or host), None for None."""
    if t is None:
        return None
    return int(t.data_ptr())


class FlyVerify:
    """Handle of one verifier (fly_verify_create / fly_verify_destroy).

    Tensors are torch tensors used purely as typed device (or, for run_host,
    pinned host) buffers; the caller owns them.
    """

    def __init__(self, max_batch: int, max_k: int, vocab: int, dtype: str = "bf16", device: int = 0,
                 hidden: int = 0):
        self._h = C.c_void_p()
        self.vocab = int(vocab)
        self.dtype = dtype
        cfg = fly_verify_config_t(int(device), int(max_batch), int(max_k), int(vocab),
                                  FLY_BF16 if dtype == "bf16" else FLY_F32, int(hidden))
        st = lib().fly_verify_create(C.byref(cfg), C.byref(self._h))
        if st != FLY_OK:
            self._h = C.c_void_p()
            raise FlyError(st, "fly_verify_create")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().fly_verify_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_option(self, option: int, value: int):
        st = lib().fly_verify_set_option(self._h, int(option), int(value))
        if st != FLY_OK:
            raise FlyError(st, "fly_verify_set_option")

    def set_splits(self, splits: int):
        self.set_option(FLY_OPT_SPLITS, splits)

    def set_scan_mode(self, separate_kernel: bool):
        self.set_option(FLY_OPT_SCAN_MODE, 1 if separate_kernel else 0)

    def set_weight_layout(self, vocab_major: bool):
        """Fused path: True if the weight is stored [V, hidden] (hidden contiguous), False for [hidden, V]."""
        self.set_option(FLY_OPT_WEIGHT_LAYOUT, 1 if vocab_major else 0)
        self.weight_vd = bool(vocab_major)

    def device_status(self, stream: int = 0) -> int:
        """fly_verify_device_status: synchronises the stream; FLY_OK or FLY_ERR_TIMEOUT."""
        return int(lib().fly_verify_device_status(self._h, C.c_void_p(stream)))

    def reduce_shard(self, logits, vocab_offset: int, partial_out, stream: int = 0, temperature: float = 0.0):
        """fly_verify_reduce_shard: logits [rows, vocab_slice] (a strided view is fine) -> partial_out
        [rows, 4] (any 16-byte element type, e.g. float32 x 4)."""
        rows = logits.shape[0]
        assert logits.shape[1] == self.vocab and logits.stride(1) == 1
        st = lib().fly_verify_reduce_shard(self._h, int(rows), _ptr(logits), int(logits.stride(0)), int(vocab_offset),
                                           float(temperature), _ptr(partial_out), C.c_void_p(stream))
        if st != FLY_OK:
            raise FlyError(st, "fly_verify_reduce_shard", lib().fly_verify_last_cuda_error(self._h))

    def run_partials(self, args: fly_verify_args_t, partials, world: int, total_vocab: int, stream: int = 0):
        """fly_verify_run_partials: partials [world, rows, 4] gathered from the ranks."""
        st = lib().fly_verify_run_partials(self._h, C.byref(args), _ptr(partials), int(world), int(total_vocab),
                                           C.c_void_p(stream))
        if st != FLY_OK:
            raise FlyError(st, "fly_verify_run_partials", lib().fly_verify_last_cuda_error(self._h))

    def selftest_wait(self, stream: int = 0) -> int:
        """fly_verify_selftest_wait: makes one bounded device-side wait run out on purpose (no fault)."""
        return int(lib().fly_verify_selftest_wait(self._h, C.c_void_p(stream)))

    @property
    def last_launch_count(self) -> int:
        return int(lib().fly_verify_last_launch_count(self._h))

    def make_args(self, B, K, draft, accept_len, out_tokens, logits=None, row_stride=0, hidden=None,
                  weight=None, theta=1.0, theta_unit="nats", W=3, boundary="reject", state_in=None,
                  state_out=None, rollback=None, target_argmax=None, entropy=None, row_flags=None,
                  target_tokens=None, temperature=0.0, inputs_ready=False):
        a = fly_verify_args_t()
        a.B, a.K = int(B), int(K)
        a.logits, a.row_stride = _ptr(logits), int(row_stride)
        a.hidden, a.weight = _ptr(hidden), _ptr(weight)
        a.draft = _ptr(draft)
        a.theta = float(theta)
        a.theta_unit = FLY_THETA_NATS if theta_unit == "nats" else FLY_THETA_NORMALIZED
        a.W = int(W)
        a.boundary = FLY_BOUNDARY_CARRY if boundary == "carry" else FLY_BOUNDARY_REJECT
        a.state_in, a.state_out = _ptr(state_in), _ptr(state_out)
        a.accept_len, a.rollback, a.out_tokens = _ptr(accept_len), _ptr(rollback), _ptr(out_tokens)
        a.target_argmax, a.entropy, a.row_flags = _ptr(target_argmax), _ptr(entropy), _ptr(row_flags)
        a.target_tokens = _ptr(target_tokens)
        a.temperature = float(temperature)
        a.inputs_ready = 1 if inputs_ready else 0
        return a

    def run(self, args: fly_verify_args_t, stream: int = 0):
        """fly_verify_run: device buffers, asynchronous on `stream` (a raw cudaStream_t value)."""
        st = lib().fly_verify_run(self._h, C.byref(args), C.c_void_p(stream))
        if st != FLY_OK:
            raise FlyError(st, "fly_verify_run", lib().fly_verify_last_cuda_error(self._h))

    def run_host(self, args: fly_verify_args_t, stream: int = 0):
        """fly_verify_run_host: host buffers, copies in and out, synchronises."""
        st = lib().fly_verify_run_host(self._h, C.byref(args), C.c_void_p(stream))
        if st != FLY_OK:
            raise FlyError(st, "fly_verify_run_host", lib().fly_verify_last_cuda_error(self._h))


def run_static(args: fly_verify_args_t, vocab: int, dtype: str = "bf16", device: int = 0, stream: int = 0):
    """fly_verify_run_static: the logits-path step without a handle, for callers that must not allocate
    device memory (its scratch is a fixed array inside the library).  `args` is the same struct that
    FlyVerify.run takes; `static_args` fills one without needing a handle.  Calls on one device must not
    overlap on the GPU."""
    st = lib().fly_verify_run_static(int(device), int(vocab), FLY_BF16 if dtype == "bf16" else FLY_F32,
                                     C.byref(args), C.c_void_p(stream))
    if st != FLY_OK:
        raise FlyError(st, "fly_verify_run_static")


def pld_draft(tokens, lengths, K: int, max_ngram: int = 3, min_ngram: int = 1, device: int = 0, stream: int = 0):
    """fly_pld_draft on tokens [B, Lmax] int32 and lengths [B] int32 (device tensors).  Returns
    (draft [B, K], count [B], match_pos [B], match_ngram [B]) as new device tensors."""
    import torch
    B = tokens.shape[0]
    assert tokens.dtype == torch.int32 and lengths.dtype == torch.int32 and tokens.stride(1) == 1
    draft = torch.empty(B, K, dtype=torch.int32, device=tokens.device)
    count, pos, ng = (torch.empty(B, dtype=torch.int32, device=tokens.device) for _ in range(3))
    st = lib().fly_pld_draft(int(device), int(B), _ptr(tokens), int(tokens.stride(0)), _ptr(lengths), int(max_ngram),
                             int(min_ngram), int(K), _ptr(draft), _ptr(count), _ptr(pos), _ptr(ng), C.c_void_p(stream))
    if st != FLY_OK:
        raise FlyError(st, "fly_pld_draft")
    return draft, count, pos, ng


def static_args(*a, **kw) -> fly_verify_args_t:
    """Fills a fly_verify_args_t (same parameters as FlyVerify.make_args) without creating a handle."""
    return FlyVerify.make_args(None, *a, **kw)


class VerifyBuffers:
    """Output buffers of one step, allocated once with torch and reused."""

    def __init__(self, B: int, K: int, device, pinned: bool = False):
        import torch
        kw = dict(device=device)
        if pinned:
            kw = dict(device="cpu", pin_memory=True)
        self.accept_len = torch.empty(B, dtype=torch.int32, **kw)
        self.rollback = torch.empty(B, dtype=torch.int32, **kw)
        self.out_tokens = torch.empty(B, K + 1, dtype=torch.int32, **kw)
        self.target_argmax = torch.empty(B, K + 1, dtype=torch.int32, **kw)
        self.entropy = torch.empty(B, K + 1, dtype=torch.float32, **kw)
        self.row_flags = torch.empty(B, K + 1, dtype=torch.int32, **kw)
        zero = torch.tensor([[0, 0, -1]] * B, dtype=torch.int32)   # the zero state of every sequence
        self.state = zero.pin_memory() if pinned else zero.to(device)


def plan(sm_count: int, rows: int, vocab: int, dtype: str = "bf16", vector_path: bool = True, inputs_ready: bool = False,
         forced_pieces: int = 0) -> fly_plan_t:
    """fly_verify_plan: the launch geometry of the row reduction (host arithmetic only, no CUDA call)."""
    out = fly_plan_t()
    st = lib().fly_verify_plan(int(sm_count), int(rows), int(vocab), FLY_BF16 if dtype == "bf16" else FLY_F32,
                               1 if vector_path else 0, 1 if inputs_ready else 0, int(forced_pieces), C.byref(out))
    if st != FLY_OK:
        raise FlyError(st, "fly_verify_plan")
    return out


def verify(fv: FlyVerify, logits, draft, out: VerifyBuffers, theta=1.0, W=3, theta_unit="nats",
           boundary="reject", stream: int = 0, host: bool = False, temperature=0.0, inputs_ready=False):
    """One verification step on logits [B, K+1, V] and draft [B, K] (int32).
    In carry mode out.state is both the carried-in and the carried-out state."""
    B, K1, V = logits.shape
    assert V == fv.vocab and logits.stride(2) == 1 and logits.stride(0) == K1 * logits.stride(1)
    carry = boundary == "carry"
    a = fv.make_args(B, K1 - 1, draft, out.accept_len, out.out_tokens, logits=logits,
                     row_stride=logits.stride(1), theta=theta, theta_unit=theta_unit, W=W, boundary=boundary,
                     state_in=out.state if carry else None, state_out=out.state, rollback=out.rollback,
                     target_argmax=out.target_argmax, entropy=out.entropy, row_flags=out.row_flags,
                     temperature=temperature, inputs_ready=inputs_ready)
    (fv.run_host if host else fv.run)(a, stream)
    return out


def verify_fused(fv: FlyVerify, hidden, weight, draft, out: VerifyBuffers, theta=1.0, W=3, theta_unit="nats",
                 boundary="reject", stream: int = 0, host: bool = False, temperature=0.0):
    """One verification step on the fused LM-head path: hidden [B*(K+1), D] bf16 and weight [D, V] bf16
    (device; with host=True hidden, draft and the outputs are host buffers, the weight stays on the device).
    The logits hidden @ weight are formed and reduced inside the kernel and never stored."""
    B, K = draft.shape
    rows, D = hidden.shape
    assert rows == B * (K + 1)
    assert tuple(weight.shape) == ((fv.vocab, D) if getattr(fv, "weight_vd", False) else (D, fv.vocab))
    assert hidden.is_contiguous() and weight.is_contiguous()
    carry = boundary == "carry"
    a = fv.make_args(B, K, draft, out.accept_len, out.out_tokens, hidden=hidden, weight=weight, theta=theta,
                     theta_unit=theta_unit, W=W, boundary=boundary, state_in=out.state if carry else None,
                     state_out=out.state, rollback=out.rollback, target_argmax=out.target_argmax,
                     entropy=out.entropy, row_flags=out.row_flags, temperature=temperature)
    (fv.run_host if host else fv.run)(a, stream)
    return out
