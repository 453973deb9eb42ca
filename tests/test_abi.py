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
int main(void) { printf("%zu %zu %zu %zu %zu %zu %zu %zu %zu\n", sizeof(des_config_t), sizeof(des_batch_t),
  sizeof(des_partials_t), sizeof(des_outputs_t), sizeof(des_grads_t), sizeof(des_comm_model_t),
  sizeof(des_comm_volume_t), sizeof(des_head_t), sizeof(des_head_grads_t)); return 0; }
'''
    with tempfile.TemporaryDirectory() as d:
        open(os.path.join(d, "a.c"), "w").write(prog)
        subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), "-o", os.path.join(d, "a"), os.path.join(d, "a.c")])
        out = subprocess.check_output([os.path.join(d, "a")]).split()
    want = [C.sizeof(binding.des_config_t), C.sizeof(binding.des_batch_t), C.sizeof(binding.des_partials_t),
            C.sizeof(binding.des_outputs_t), C.sizeof(binding.des_grads_t), C.sizeof(binding.des_comm_model_t),
            C.sizeof(binding.des_comm_volume_t), C.sizeof(binding.des_head_t), C.sizeof(binding.des_head_grads_t)]
    assert [int(v) for v in out] == want


def test_comm_volume_reproduces_the_papers_table_2():
    # Table 2 (Section 4.3): unique features per batch and saving ratios on a 4-node cluster; the
    # product's calculator (host code of the CUDA library, no GPU needed) against the printed values.
    from paper_1909_04823_b200 import binding
    rows = [l.split() for l in open(os.path.join(ROOT, "tests", "golden", "paper_table2_comm_saving.txt"))
            if l.strip() and l[0] != "#"]
    assert len(rows) == 5
    for r in rows:
        v = binding.comm_volume(4, int(r[0]), int(r[1]), 8, 256, 4800 * 256 * 4)
        for got, want in zip(v["saving"], r[2:5]):
            assert f"{100.0 * got:.3f}" == want
        # the volumes themselves: 3/4 of keys + weights against twice 3/4 of the partials
        assert v["q_mesh"][0] == 0.75 * (8 + 4) * int(r[1]) and v["q_des"][0] == 2 * 0.75 * 4 * int(r[0])
    import pytest
    with pytest.raises(binding.DesError):
        binding.comm_volume(1, 512, 1000, 8, 256, 0)          # one worker exchanges nothing
