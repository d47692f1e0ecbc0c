"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, its structs match the Python mirror, and argument validation rejects bad calls before
touching the device."""
import ctypes as C
import re
import subprocess
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
HEADER = ROOT / "include" / "specattn.h"


@pytest.fixture(scope="module")
def sa():
    from paper_2510_27641_b200 import build
    build.build()
    import paper_2510_27641_b200 as sa
    return sa


def _declared_functions():
    text = re.sub(r"/\*.*?\*/", "", HEADER.read_text(), flags=re.S)
    return sorted(set(re.findall(r"\b(specattn_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(sa):
    names = _declared_functions()
    assert {"specattn_select_topp", "specattn_sparse_verify", "specattn_verify_workspace_bytes",
            "specattn_verify_workspace_init", "specattn_verify_step_host", "specattn_status_string",
            "specattn_kernel_launch_count", "specattn_verify_plan", "specattn_verify_plan_bytes",
            "specattn_select_workspace_bytes", "specattn_verify_plan_many"} <= set(names)
    L = sa.lib()
    for n in names:
        assert hasattr(L, n), f"{n} is declared in specattn.h but not exported"


def test_struct_layouts_match_the_header(sa, tmp_path):
    src = tmp_path / "sz.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "specattn.h"\nint main(){printf("%zu %zu %zu %zu %zu %zu\\n",'
                   'sizeof(specattn_select_args), sizeof(specattn_verify_args), sizeof(specattn_step_host_args),'
                   'offsetof(specattn_select_args, idx_stride), offsetof(specattn_verify_args, sm_scale),'
                   'offsetof(specattn_verify_args, workspace_bytes));return 0;}\n')
    exe = tmp_path / "sz"
    subprocess.run(["gcc", "-I", str(ROOT / "include"), str(src), "-o", str(exe)], check=True)
    got = [int(x) for x in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
    assert got == [C.sizeof(sa.SelectArgs), C.sizeof(sa.VerifyArgs), C.sizeof(sa.StepHostArgs),
                   sa.SelectArgs.idx_stride.offset, sa.VerifyArgs.sm_scale.offset,
                   sa.VerifyArgs.workspace_bytes.offset]


def test_status_strings_and_launch_counter(sa):
    assert sa.status_string(0) == "ok"
    for code in range(-8, 0):
        assert sa.status_string(code) not in ("ok", "unknown status code")
    assert sa.status_string(-99) == "unknown status code"
    assert sa.kernel_launch_count() >= 0


def test_validation_rejects_bad_arguments_without_a_device(sa):
    L = sa.lib()
    assert L.specattn_select_topp(None, None) == -1
    assert L.specattn_sparse_verify(None, None) == -1
    a = sa.SelectArgs()
    assert L.specattn_select_topp(C.byref(a), None) == -2          # struct_size
    a.struct_size = C.sizeof(sa.SelectArgs)
    assert L.specattn_select_topp(C.byref(a), None) == -1          # null pointers
    v = sa.VerifyArgs()
    assert L.specattn_sparse_verify(C.byref(v), None) == -2
    v.struct_size = C.sizeof(sa.VerifyArgs)
    v.batch, v.n_q, v.n_q_heads, v.n_kv_heads, v.head_dim, v.page_size, v.n_groups = 1, 5, 32, 8, 64, 16, 1
    assert L.specattn_sparse_verify(C.byref(v), None) == -6        # head_dim != 128
    v.head_dim, v.n_q_heads = 128, 30
    assert L.specattn_sparse_verify(C.byref(v), None) == -3        # heads not divisible
    v.n_q_heads, v.n_groups = 32, 3
    assert L.specattn_sparse_verify(C.byref(v), None) == -3        # groups must be 1 or H_kv
    assert L.specattn_verify_workspace_bytes(C.byref(v)) == 0
    assert L.specattn_verify_workspace_init(None, 0, None) == -1
    s = sa.StepHostArgs()
    assert L.specattn_verify_step_host(C.byref(s), None) == -2


def test_product_path_never_imports_the_oracle():
    for f in list((ROOT / "paper_2510_27641_b200").rglob("*.py")) + list((ROOT / "paper_2510_27641_b200").rglob("*.cu")):
        assert "oracle" not in f.read_text(), f
    for f in (ROOT / "oracle").rglob("*"):
        if f.suffix in (".py", ".cpp"):
            assert "paper_2510_27641_b200" not in f.read_text(), f


def test_select_workspace_query_follows_the_documented_rule(sa):
    """specattn_select_workspace_bytes reads host fields only: a workspace is asked for exactly
    when the default selection runs over multi-row lists of >= 2048 positions that are too few to
    give every SM a CTA with one cluster each."""
    L = sa.lib()

    def need(n_target, batch, heads, gamma, Ls, **kw):
        a = sa.SelectArgs()
        a.struct_size = C.sizeof(sa.SelectArgs)
        lm = (C.c_int32 * n_target)(*[j % 4 for j in range(n_target)])
        a.n_draft_layers, a.n_target_layers, a.batch = 4, n_target, batch
        a.n_draft_heads, a.gamma, a.n_groups, a.L_stride = heads, gamma, 1, Ls
        a.layer_map = lm
        for k, v in kw.items():
            setattr(a, k, v)
        return int(L.specattn_select_workspace_bytes(C.byref(a)))

    assert need(1, 4, 16, 4, 131072) == 4 * 131072 * 4            # 4 lists x 8 CTAs: underfilled
    assert need(8, 4, 16, 4, 131072) == 16 * 131072 * 4           # 16 lists x 8 = 128 < 148
    assert need(32, 8, 12, 5, 32768) == 0                          # 32 lists x 8 CTAs fill the GPU
    assert need(1, 4, 1, 1, 131072) == 0                           # single-row lists are read in place
    assert need(1, 4, 16, 4, 1024) == 0                            # short rows
    assert need(1, 4, 16, 4, 131072, per_step=1) == 0              # variants keep the cluster form
    # the caller's choice of form: two launches whatever the number of lists, or never
    assert need(32, 8, 12, 5, 32768, form=2) == 32 * 32768 * 4
    assert need(1, 4, 16, 4, 131072, form=1) == 0
    assert need(1, 4, 1, 1, 131072, form=2) == 0                   # single-row lists have nothing to sum
    assert need(1, 4, 16, 4, 131072, chunk=16) == 0
    assert need(1, 4, 16, 4, 131072, bisect_iters=10) == 0
    assert L.specattn_select_workspace_bytes(None) == 0
    bad = sa.SelectArgs()
    assert L.specattn_select_workspace_bytes(C.byref(bad)) == 0   # struct_size not set
