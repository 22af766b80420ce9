"""The C boundary without a GPU: the library loads and exports every declared symbol; host-side checks."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2504_03662_b200 import build, binding
    build.build_library()
    return binding.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "galv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(galv_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2504_03662_b200 import binding
    names = declared_functions()
    assert len(names) >= 11 and {"galv_eval_costs", "galv_dp_search", "galv_backtrack"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_host_side_answers_without_a_device(lib):
    from paper_2504_03662_b200 import binding as gb
    assert lib.galv_strerror(0) == b"ok"
    assert b"workspace" in lib.galv_strerror(gb.ERR_WORKSPACE)
    assert lib.galv_last_error(None) == b"no context"
    # size queries are pure host arithmetic and need no context
    sh = gb.make_shape(16, 24, 24, 2880, gb.STORE_C_FULL)
    assert sh.m_pitch == 2912
    small = lib.galv_dp_workspace_bytes(None, C.byref(sh))
    assert 0 < small < 1 << 20
    roll = lib.galv_dp_workspace_bytes(None, C.byref(gb.make_shape(16, 24, 24, 2880, 0)))
    assert roll >= small + 2 * 16 * 24 * 2912 * 4                # two rolling layers on top
    # flags that rule the packed 16-bit loop out drop its packed transition rows from the workspace
    lean = lib.galv_dp_workspace_bytes(None, C.byref(gb.make_shape(16, 24, 24, 2880, gb.STORE_C_FULL | gb.KERNEL_NO_PACKED)))
    assert small - lean >= 16 * 12 * 24 * 4
    assert lib.galv_dp_workspace_bytes(None, C.byref(gb.make_shape(16, 24, 0, 2880))) == 0
    assert lib.galv_search_host_arena_bytes(None, C.byref(sh), 1) > 16 * 24 * 24 * 2912 * 4
    # entry points refuse a missing context before touching the device
    assert lib.galv_dp_search(None, C.byref(sh), *([None] * 8), 0, None, None) == gb.ERR_INVALID_ARG
    assert lib.galv_create(None, 0) == gb.ERR_INVALID_ARG


def test_struct_sizes_match_the_header():
    from paper_2504_03662_b200 import inputs, binding as gb
    assert C.sizeof(gb.galv_shape) == 24
    assert (inputs.LAYER_DESC.itemsize, inputs.STRATEGY_DESC.itemsize, inputs.INST_PARAMS.itemsize) == (80, 32, 64)
    assert inputs.STRATEGY_DESC.fields["batch_div"][1] == 24
