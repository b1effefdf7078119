"""The C-ABI library loads without a GPU and exports every function the header declares."""
import ctypes
import os
import re

from paper_1202_3173_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "strassen_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(strassen_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_three_named_calls():
    names = _declared()
    for must in ("strassen_plan_create", "strassen_dgemm", "strassen_plan_destroy"):
        assert must in names


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = _declared()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name


def test_binding_covers_the_header_one_to_one():
    assert sorted(n for n, _, _ in binding.SYMBOLS) == _declared()
    for n, _, _ in binding.SYMBOLS:
        assert callable(getattr(binding, n)), n


def test_no_torch_types_in_the_boundary():
    text = open(os.path.join(ROOT, "include", "strassen_b200.h")).read()
    assert "torch" not in text and "at::" not in text and "#include <cuda" not in text


def test_product_does_not_reach_into_the_oracle():
    pkg = os.path.join(ROOT, "paper_1202_3173_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cpp", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), os.path.join(dirpath, f)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            assert "paper_1202_3173_b200" not in open(os.path.join(ROOT, "oracle", f)).read()


def test_header_is_valid_c99_and_cxx():
    import subprocess
    import tempfile
    inc = os.path.join(ROOT, "include")
    prog = '#include "strassen_b200.h"\nint main(void) { strassen_options o = {0}; (void)o; return STRASSEN_OK; }\n'
    with tempfile.TemporaryDirectory() as d:
        for name, cc, std in (("t.c", "gcc", "-std=c99"), ("t.cpp", "g++", "-std=c++11")):
            path = os.path.join(d, name)
            open(path, "w").write(prog)
            subprocess.check_call([cc, std, "-Wall", "-Werror", "-pedantic", "-fsyntax-only", "-I", inc, path])


def test_c_program_links_against_the_library_and_plans_without_a_gpu():
    import subprocess
    import tempfile
    src = r'''
#include <stdio.h>
#include <string.h>
#include "strassen_b200.h"
int main(void) {
    strassen_plan *p = strassen_plan_create(4096, 512, "BBB");
    if (!p) { printf("create failed: %s\n", strassen_last_error()); return 1; }
    printf("%d %lld %s %zu\n", strassen_plan_levels(p), (long long)strassen_plan_base_size(p), strassen_plan_schedule(p),
           strassen_plan_workspace_bytes(p));
    strassen_plan_destroy(p);
    p = strassen_plan_create(4096, 512, "BXB");
    if (p || !strlen(strassen_last_error())) return 2;
    return 0;
}
'''
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "plan.c")
        exe = os.path.join(d, "plan")
        open(c, "w").write(src)
        subprocess.check_call(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), c, "-o", exe, binding.LIB_PATH,
                               "-Wl,-rpath," + os.path.dirname(binding.LIB_PATH)])
        out = subprocess.check_output([exe], text=True).split()
    assert out == ["3", "512", "BBB", str(8 * 15 * (2048 ** 2 + 7 * 1024 ** 2 + 49 * 512 ** 2))]
