"""Host-side checks that need no GPU: the C-ABI library builds, loads and
exports every symbol the header declares; argument errors are caught before
any CUDA call."""
import ctypes as C
import os
import re

import pytest

from paper_2511_22972_b200 import binding as Bd, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "fly_verify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fly_[a-z_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    L = Bd.lib()
    names = declared_symbols()
    assert len(names) >= 8
    for n in names:
        assert hasattr(L, n), f"{n} is declared in the header but not exported"
    assert sorted(Bd.EXPORTS) == names
    assert os.path.exists(build.LIB_PATH) and not build.is_stale()


def test_status_strings():
    assert Bd.status_string(Bd.FLY_OK) == "ok"
    assert "invalid" in Bd.status_string(Bd.FLY_ERR_INVALID_ARG)
    assert "timed out" in Bd.status_string(Bd.FLY_ERR_TIMEOUT)
    assert Bd.status_string(99) == "unknown status"


def test_struct_layout_matches_the_header():
    # x86-64 SysV: the args struct has 2 int32, then 8-byte members
    assert C.sizeof(Bd.fly_verify_config_t) == 24
    a = Bd.fly_verify_args_t
    assert a.logits.offset == 8 and a.row_stride.offset == 16 and a.draft.offset == 40
    assert a.theta.offset == 48 and a.theta_unit.offset == 56 and a.W.offset == 60 and a.boundary.offset == 64
    assert a.state_in.offset == 72 and a.row_flags.offset == 128 and a.target_tokens.offset == 136
    assert a.temperature.offset == 144 and a.inputs_ready.offset == 152 and C.sizeof(a) == 160
    assert C.sizeof(Bd.fly_plan_t) == 32


@pytest.mark.parametrize("cfg", [
    dict(max_batch=0), dict(max_k=0), dict(max_k=64), dict(vocab=0), dict(dtype=7), dict(device=-1), dict(hidden=-1),
])
def test_create_rejects_bad_configs_without_touching_cuda(cfg):
    base = dict(device=0, max_batch=4, max_k=8, vocab=1000, dtype=Bd.FLY_BF16, hidden=0)
    base.update(cfg)
    c = Bd.fly_verify_config_t(base["device"], base["max_batch"], base["max_k"], base["vocab"], base["dtype"],
                               base["hidden"])
    h = C.c_void_p(123)
    st = Bd.lib().fly_verify_create(C.byref(c), C.byref(h))
    assert st == Bd.FLY_ERR_INVALID_ARG and not h.value


def test_null_arguments():
    L = Bd.lib()
    assert L.fly_verify_create(None, None) == Bd.FLY_ERR_INVALID_ARG
    assert L.fly_verify_destroy(None) == Bd.FLY_OK
    assert L.fly_verify_run(None, None, None) == Bd.FLY_ERR_INVALID_ARG
    assert L.fly_verify_run_host(None, None, None) == Bd.FLY_ERR_INVALID_ARG
    assert L.fly_verify_set_option(None, 0, 1) == Bd.FLY_ERR_INVALID_ARG
    assert L.fly_verify_last_launch_count(None) == 0


def test_header_is_plain_c_and_cxx(tmp_path):
    # the boundary has to be usable from C: the header compiles as strict C99 and as C++17
    import shutil
    import subprocess
    src = tmp_path / "h.c"
    src.write_text('#include "fly_verify.h"\nint main(void) { fly_verify_args_t a; (void)a; '
                   'return sizeof(fly_partial_t) == 16 && sizeof(fly_state_t) == 12 ? 0 : 1; }\n')
    inc = os.path.join(ROOT, "include")
    if shutil.which("gcc"):
        subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-I", inc, "-fsyntax-only", str(src)],
                       check=True)
    if shutil.which("g++"):
        subprocess.run(["g++", "-std=c++17", "-Wall", "-Wextra", "-Werror", "-I", inc, "-fsyntax-only", "-x", "c++", str(src)],
                       check=True)


def test_launch_geometry_rule():
    # host logic of the logits path (no GPU needed): how the rows of a step are cut into thread-block ranges
    row_units = 128256 // 8                                   # 16-byte segments in one bf16 row of the Llama-3 vocabulary
    p = Bd.plan(148, 144, 128256)
    assert p.units_per_row == row_units
    assert p.grid == 144 * 2 and p.slots == 2                 # whole pieces, all resident; 1, 2 and 4 pieces cost the busiest SM
    assert p.row_span == 2 * p.units_per_block and p.units_per_block * 2 >= row_units   # the same, 2 is nearest two blocks per SM
    assert Bd.plan(148, 144, 128256, forced_pieces=3).grid == 144 * 3
    p2 = Bd.plan(148, 144, 128256, inputs_ready=True)
    assert p2.grid == 144                                     # overlapping steps: about one block per SM, several steps deep
    assert Bd.plan(148, 16, 128256, inputs_ready=True).grid == 16 * 2
    assert Bd.plan(148, 16, 128256).grid == 16 * 9            # 9 pieces of 1.74 strides: two slices per warp, one block per SM
    big = Bd.plan(148, 1088, 128256)
    assert big.grid == 1088 and big.slots == 1                # more rows than resident slots: whole rows, two well-filled waves
    odd = Bd.plan(148, 700, 128256)                           # 700 whole rows would leave 82 % of the second wave empty:
    assert odd.row_span == row_units and 148 * 4 - 4 <= odd.grid <= 148 * 4   # rows packed end to end, cut evenly
    assert Bd.plan(148, 1, 128256).units_per_block >= 1024    # never less than 16 KB per block
    assert Bd.plan(148, 9, 32000, dtype="f32").grid == 9 * 7
    L = Bd.lib()
    out = Bd.fly_plan_t()
    assert L.fly_verify_plan(0, 1, 128256, Bd.FLY_BF16, 1, 0, 0, out) == Bd.FLY_ERR_INVALID_ARG
    assert L.fly_verify_plan(148, 0, 128256, Bd.FLY_BF16, 1, 0, 0, out) == Bd.FLY_ERR_INVALID_ARG
    assert L.fly_verify_plan(148, 1, 128256, Bd.FLY_BF16, 1, 0, 0, None) == Bd.FLY_ERR_INVALID_ARG
    assert L.fly_verify_plan(148, 1, 100, Bd.FLY_BF16, 1, 0, 0, out) == Bd.FLY_ERR_INVALID_ARG   # too short for 16-byte loads
    for rows in (1, 2, 3, 9, 17, 144, 500, 1088, 2304, 5000, 36864):
        for vocab, dtype, vec in ((128256, "bf16", True), (152064, "bf16", True), (32000, "f32", True), (257, "bf16", True),
                                  (1, "f32", False), (7, "bf16", False), (1001, "bf16", False), (1 << 20, "f32", True)):
            for ready in (False, True):
                for forced in (0, 1, 2, 5, 32):
                    p = Bd.plan(148, rows, vocab, dtype, vec, ready, forced)
                    n, Q, span = p.units_per_row, p.units_per_block, p.row_span
                    assert Q >= 1 and span >= n and p.grid == -(-(rows * span) // Q) and 1 <= p.slots <= 32
                    # every row's pieces fit its slots and cover exactly its n units
                    for r in {0, 1 % rows, rows // 2, rows - 1}:
                        first, last = (r * span) // Q, (r * span + span - 1) // Q
                        assert last - first + 1 <= p.slots, (rows, vocab, forced, first, last, p.slots)
                        covered = 0
                        for b in range(first, last + 1):
                            lo = max(b * Q, r * span) - r * span
                            hi = min((b + 1) * Q, (r + 1) * span) - r * span
                            covered += max(0, min(hi, n) - min(lo, n))
                        assert covered == n
                    if forced:
                        assert span == min(forced, n, -(-n // Q)) * Q or span % Q == 0
                        assert span % Q == 0 and span // Q <= forced
                    elif not ready:
                        assert p.grid <= max(148 * 4, rows)
                    else:
                        assert p.grid <= max(2 * 148, rows)
