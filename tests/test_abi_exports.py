"""The shared library loads without a GPU and exports every entry point the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "rmsnorm_tuner.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+)?(?:int|void|int32_t|int64_t|char\s*\*)\s*\*?\s*(\w+)\s*\(", text, flags=re.M)
    return [n for n in names if not n.startswith("rt_evaluate_fn")]


def test_library_exports_every_declared_symbol():
    from paper_2601_12698_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    declared = _declared_functions()
    assert len(declared) >= 20 and "rmsnorm_template_launch" in declared and "tuner_search" in declared
    assert "tuner_derive_feasible" in declared and "tuner_compare_static" in declared
    missing = [n for n in declared if not hasattr(lib, n)]
    assert not missing, missing


def test_binding_covers_the_header():
    from paper_2601_12698_b200 import binding
    assert sorted(binding.EXPORTED) == sorted(_declared_functions())
    # 677 norm (69 of them the ragged-row stage, 54 the persistent pipeline) + 64 silu_and_mul + 64 merge_attn_states
    # + 54 fp8-output + 165 all-reduce-fused
    assert binding.lib.rt_num_kernel_instances() == 1024
    assert binding.lib.rt_status_string(binding.RT_ERR_INFEASIBLE).decode().startswith("configuration outside")
    inst = binding.kernel_instances()
    assert {i["dtype"] for i in inst} == {0, 1, 2} and {i["stage"] for i in inst} == {0, 1, 2, 3, 4}
    assert sum(1 for i in inst if i["stage"] == 4) == 54 and {i["op"] for i in inst if i["stage"] == 4} == {0}
    assert sum(1 for i in inst if i["op"] == 2) == 64 and sum(1 for i in inst if i["op"] == 3) == 54
    assert sum(1 for i in inst if i["op"] == 1) == 64 and {i["stage"] for i in inst if i["op"] == 1} == {0, 2}
    fused = [i for i in inst if i["op"] == 4]
    assert len(fused) == 165 and {i["parts"] for i in fused} == {2, 4, 8} and {i["stage"] for i in fused} == {0}
    assert all(i["unroll"] * i["parts"] * i["vec_bytes"] <= 256 for i in fused) and all(i["parts"] == 0 for i in inst if i["op"] != 4)
    assert all(i["reg_vectors"] * (i["vec_bytes"] // (4 if i["dtype"] == 2 else 2)) <= 128 for i in inst)


def test_struct_layouts_match_the_header_sizes():
    """sizeof of each ctypes mirror equals what a C compiler gives for the header."""
    import subprocess
    import tempfile
    from paper_2601_12698_b200 import binding as B
    src = ('#include <stdio.h>\n#include "rmsnorm_tuner.h"\nint main(void){printf("%zu %zu %zu %zu %zu %zu %zu %zu\\n",'
           "sizeof(rt_params),sizeof(rt_shape),sizeof(rt_limits),sizeof(rt_budget),sizeof(rt_workspace),"
           "sizeof(rt_eval_record),sizeof(rt_result),sizeof(rt_block_record));return 0;}\n")
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "s.c")
        open(c, "w").write(src)
        exe = os.path.join(d, "s")
        subprocess.run(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), c, "-o", exe], check=True)
        sizes = [int(v) for v in subprocess.run([exe], capture_output=True, text=True, check=True).stdout.split()]
    mirrors = [B.rt_params, B.rt_shape, B.rt_limits, B.rt_budget, B.rt_workspace, B.rt_eval_record, B.rt_result, B.rt_block_record]
    assert sizes == [ctypes.sizeof(m) for m in mirrors]


def test_no_device_is_reported_not_crashed():
    import torch
    if torch.cuda.is_available():
        return
    from paper_2601_12698_b200 import binding as B
    L = B.rt_limits()
    assert B.lib.rt_query_limits(ctypes.byref(L)) == B.RT_ERR_NO_DEVICE
    n = ctypes.c_int32(0)
    s = B.shape_of(4, 64, "bf16")
    assert B.lib.tuner_derive_feasible(ctypes.byref(s), None, 0, ctypes.byref(n)) == B.RT_ERR_NO_DEVICE
    th = B.make_params()
    assert B.lib.rmsnorm_template_launch(ctypes.byref(th), 8, 8, 8, 8, 8, 4, 64, 1e-6, 0, None) == B.RT_ERR_NO_DEVICE


def test_launch_option_is_validated_and_remembered():
    from paper_2601_12698_b200 import binding as B
    opt = B.RT_OPTION_PROGRAMMATIC_LAUNCH
    assert B.lib.rt_get_option(opt) == 1                       # the default
    try:
        assert B.lib.rt_set_option(opt, 0) == B.RT_OK and B.lib.rt_get_option(opt) == 0
        assert B.lib.rt_set_option(opt, 2) == B.RT_ERR_SHAPE and B.lib.rt_get_option(opt) == 0
        assert B.lib.rt_set_option(7, 1) == B.RT_ERR_SHAPE and B.lib.rt_get_option(7) == -1
    finally:
        assert B.lib.rt_set_option(opt, 1) == B.RT_OK
