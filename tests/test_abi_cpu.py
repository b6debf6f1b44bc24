"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, and rejects
invalid arguments before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2604_23108_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "mohge.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mohge_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2604_23108_b200.build import build
    build()
    lib = B.lib()
    names = _declared_symbols()
    assert "mohge_route" in names and "mohge_expert_bwd" in names and len(names) >= 13
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(B.exported_symbols())


def test_sizes_and_validation_without_a_device():
    cfg = B.Config(1024, 3, 8, 2, 4, [1408, 704, 352])
    assert B.mohge_perm_rows(cfg, 8192) == 8192 * 4 + 24 * 127 + (128 - (8192 * 4 + 24 * 127) % 128) % 128
    assert B.mohge_workspace_bytes(cfg, 8192) > 0
    lib = B.lib()
    bad = [
        dict(k_experts=17),                 # K_e > K_g * N: Eq. 5 could not fill its slots
        dict(k_groups=4),
        dict(n_groups=9, group_width=[64] * 9),
        dict(experts_per_group=33),
        dict(d_model=1001),
        dict(group_width=[1408, 700, 352]),
        dict(row_align=64),
    ]
    for kw in bad:
        args = dict(d_model=1024, n_groups=3, experts_per_group=8, k_groups=2, k_experts=4,
                    group_width=[1408, 704, 352])
        args.update(kw)
        c = B.Config(**args).c() if len(args["group_width"]) <= 8 else None
        if c is None:
            c = B.Config(**dict(args, group_width=args["group_width"][:8])).c()
            c.n_groups = 9
        assert lib.mohge_workspace_bytes(C.byref(c), 128) == 0, kw
        rc = lib.mohge_combine(C.byref(c), 128, None, None, None, None, None, None)
        assert rc == -1, kw
        assert len(lib.mohge_last_error()) > 0
    # NULL and misaligned pointers are refused before any launch
    good = cfg.c()
    assert lib.mohge_combine(C.byref(good), 128, None, None, None, None, None, None) == -1
    assert lib.mohge_combine(C.byref(good), 128, C.c_void_p(8), C.c_void_p(16), C.c_void_p(16),
                             None, C.c_void_p(16), None) == -1
    assert b"16-byte" in lib.mohge_last_error()
    assert lib.mohge_route(C.byref(good), -5, *([None] * 12)) == -1


def test_combine_bwd_takes_y_perm_and_dgate_together_or_not_at_all():
    """mohge_combine_bwd computes the gate gradient from y_perm, or neither reads the one nor
    writes the other (the gradient then comes from mohge_expert_bwd_dgate); a call that gives only
    one of the two is refused before any launch."""
    lib = B.lib()
    good = B.Config(1024, 3, 8, 2, 4, [1408, 704, 352]).c()
    p = C.c_void_p(256)                    # never dereferenced: the call is refused first
    args = lambda y_perm, dgate: (C.byref(good), 128, p, y_perm, p, p, p, p, p, dgate, None)
    assert lib.mohge_combine_bwd(*args(p, None)) == -1
    assert b"both" in lib.mohge_last_error()
    assert lib.mohge_combine_bwd(*args(None, p)) == -1
    # the fused backward wants every pointer of its gate-gradient part
    rc = lib.mohge_expert_bwd_dgate(C.byref(good), 128, *([p] * 6), None, None, p, p, None, None, 0,
                                    p, None, p, p, p, p, None)
    assert rc == -1 and b"y_perm" in lib.mohge_last_error()


def test_switches_are_read_from_the_environment_once():
    """The debugging switches come from the environment the first time one is consulted; later
    changes of the environment are not seen, mohge_set_switch is the only way to change one.
    Runs in a child process so that the first consultation is under the test's control."""
    import subprocess
    import sys
    code = r'''
import os, sys
sys.path.insert(0, %r)
os.environ["MOHGE_TC_CG"] = "1"
os.environ.pop("MOHGE_TC_WIDE", None)
from paper_2604_23108_b200 import binding as B
assert B.mohge_get_switch("tc_cg") == 1              # first consultation reads the environment
assert B.mohge_get_switch("tc_wide") == -1           # not set: the library's rule decides
os.environ["MOHGE_TC_CG"] = "2"
os.environ["MOHGE_TC_WIDE"] = "63"
assert B.mohge_get_switch("tc_cg") == 1              # the environment is not read again
assert B.mohge_get_switch("tc_wide") == -1
B.mohge_set_switch("tc_cg", 2)
assert B.mohge_get_switch("tc_cg") == 2
B.mohge_set_switch("tc_cg", -1)
assert B.mohge_get_switch("tc_cg") == -1
assert B.lib().mohge_get_switch(b"no_such_switch") == -2**31
assert B.lib().mohge_set_switch(b"no_such_switch", 1) == -1
assert B.lib().mohge_set_switch(b"pdl", -7) == -1
print("ok")
''' % ROOT
    out = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True)
    assert out.returncode == 0 and out.stdout.strip() == "ok", out.stderr


def test_workspace_init_refuses_a_workspace_that_is_too_small():
    lib = B.lib()
    cfg = B.Config(1024, 3, 8, 2, 4, [1408, 704, 352])
    need = B.mohge_workspace_bytes(cfg, 8192)
    rc = lib.mohge_workspace_init(C.byref(cfg.c()), 8192, C.c_void_p(256), need - 1, None)
    assert rc == -3                                    # MOHGE_ERR_WORKSPACE, nothing touched
    assert str(need).encode() in lib.mohge_last_error()


def test_header_and_library_are_usable_from_plain_c(tmp_path):
    """A C99 program includes mohge.h, links libmohge.so and asks for sizes (no device needed)."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    from paper_2604_23108_b200.build import build
    build()
    pkg = os.path.join(ROOT, "paper_2604_23108_b200")
    src = tmp_path / "sizes.c"
    src.write_text(r'''
#include <stdio.h>
#include <string.h>
#include "mohge.h"
int main(void) {
  mohge_config c;
  memset(&c, 0, sizeof c);
  c.d_model = 1024; c.n_groups = 3; c.experts_per_group = 8; c.k_groups = 2; c.k_experts = 4;
  c.group_width[0] = 1408; c.group_width[1] = 704; c.group_width[2] = 352;
  c.dtype = MOHGE_BF16; c.alpha_g = 1e-4f; c.alpha_e = 2.5e-3f; c.eps = 1e-20f;
  c.f_norm_by_T = 1; c.fe_mode = 0; c.row_align = 128;
  printf("%lld %lld\n", (long long)mohge_workspace_bytes(&c, 8192), (long long)mohge_perm_rows(&c, 8192));
  c.k_experts = 17;                      /* more than K_g * N: refused */
  printf("%lld %s\n", (long long)mohge_workspace_bytes(&c, 8192), mohge_last_error());
  return 0;
}
''')
    exe = tmp_path / "sizes"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", str(src), "-I", os.path.join(ROOT, "include"),
                    "-L", pkg, "-lmohge", "-Wl,-rpath," + pkg, "-o", str(exe)], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True, check=True).stdout.split("\n")
    cfg = B.Config(1024, 3, 8, 2, 4, [1408, 704, 352])
    assert out[0].split() == [str(B.mohge_workspace_bytes(cfg, 8192)), str(B.mohge_perm_rows(cfg, 8192))]
    assert out[1].startswith("0 ") and "k_experts" in out[1]
