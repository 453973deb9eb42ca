"""The C-ABI library builds, loads and exports every function the public
header declares (no compute calls: there is no GPU here)."""
import ctypes as C
import os
import re

from paper_1909_04823_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "des.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(des_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert {"des_table_create", "des_find_or_insert", "des_forward_partials", "des_aggregate",
            "des_backward_update"} <= set(names)
    lib = C.CDLL(build.build())
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_symbols():
    from paper_1909_04823_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()


def test_struct_layouts_match_header_sizes():
    # sizes the C compiler gives the public structs (compiled here with gcc)
    import subprocess, tempfile
    from paper_1909_04823_b200 import binding
    prog = r'''
#include <stdio.h>
#include "des.h"
int main(void) { printf("%zu %zu %zu %zu %zu\n", sizeof(des_config_t), sizeof(des_batch_t),
  sizeof(des_partials_t), sizeof(des_outputs_t), sizeof(des_grads_t)); return 0; }
'''
    with tempfile.TemporaryDirectory() as d:
        open(os.path.join(d, "a.c"), "w").write(prog)
        subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), "-o", os.path.join(d, "a"), os.path.join(d, "a.c")])
        out = subprocess.check_output([os.path.join(d, "a")]).split()
    want = [C.sizeof(binding.des_config_t), C.sizeof(binding.des_batch_t), C.sizeof(binding.des_partials_t),
            C.sizeof(binding.des_outputs_t), C.sizeof(binding.des_grads_t)]
    assert [int(v) for v in out] == want
