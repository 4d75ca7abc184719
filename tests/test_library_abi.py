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
    assert a.state_in.offset == 72 and a.row_flags.offset == 128 and a.target_tokens.offset == 136 and C.sizeof(a) == 144


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


def test_split_planning_rule():
    # host logic of the logits path: how many pieces a row is cut into (no GPU needed)
    plan = Bd.lib().fly_verify_plan_splits
    row = 128256 * 2                                   # one bf16 row of the Llama-3 vocabulary
    assert plan(148, 144, row, 1) == 1                 # overlapped steps: whole rows
    assert plan(148, 144, row, 0) == 4                 # a lone grid wants >= 3.5 blocks per SM, evenly
    assert plan(148, 1088, row, 0) in (1, 2) and plan(148, 2304, 152064 * 2, 0) == 1
    assert plan(148, 16, row, 0) == 7                  # few rows: as many 32 KB pieces as the row has
    assert plan(148, 9, 32000 * 4, 0) == 7             # tiny step: down to 16 KB pieces
    assert plan(148, 16, row, 1) == 3                  # overlapped, few rows: a quarter of the SMs is enough
    assert plan(0, 1, 1, 0) == 0 and plan(148, 0, row, 0) == 0
    for rows in (1, 3, 17, 144, 500, 5000):
        for rb in (64, 4096, 40000, row, 10 * row):
            for ov in (0, 1):
                s = plan(148, rows, rb, ov)
                assert 1 <= s <= 32
                assert s == 1 or rb // s >= 16384      # pieces never shrink below 16 KB
