"""Host-only checks of the C-ABI library: it loads, exports every symbol the header
declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2602_02864_b200 import build
    build.build()
    from paper_2602_02864_b200 import fdc
    return fdc


def test_exports_match_header(lib):
    hdr = open(os.path.join(ROOT, "include", "fdc.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(fdc_[a-z_0-9]+)\s*\(", hdr))
    assert {"fdc_plan_graph", "fdc_frontier", "fdc_build_masks", "fdc_kv_append", "fdc_decode_attn"} <= names
    dll = ctypes.CDLL(lib.LIB_PATH)
    for n in sorted(names):
        assert hasattr(dll, n), f"{n} declared in fdc.h but not exported"


def test_struct_layouts(lib, tmp_path):
    """The ctypes mirrors have the layout a C compiler gives the header's structs."""
    import subprocess
    src = tmp_path / "sz.c"
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "fdc.h"\nint main(void){printf("%zu %zu %zu %zu %zu\\n",'
                   'sizeof(fdc_graph_desc),sizeof(fdc_kv_desc),sizeof(fdc_sizes),'
                   'offsetof(fdc_kv_desc,stride_scene),offsetof(fdc_sizes,state_bytes));return 0;}\n')
    exe = tmp_path / "sz"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    got = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    assert got == [ctypes.sizeof(lib.fdc_graph_desc), ctypes.sizeof(lib.fdc_kv_desc), ctypes.sizeof(lib.fdc_sizes),
                   lib.fdc_kv_desc.stride_scene.offset, lib.fdc_sizes.state_bytes.offset]


def test_plan_rejects_bad_templates_on_host(lib):
    def code(*a):
        with pytest.raises(lib.FdcError) as e:
            lib.fdc_plan_graph(*a)
        return e.value.code
    assert code(3, [(0, 1), (1, 2), (2, 0)], [4, 4, 4], None, 8, 2) == lib.FDC_ERR_CYCLE
    assert code(2, [(1, 1)], [4, 4], None, 8, 2) == lib.FDC_ERR_CYCLE
    assert code(2, [(0, 5)], [4, 4], None, 8, 2) == lib.FDC_ERR_RANGE
    assert code(0, [], [], None, 8, 2) == lib.FDC_ERR_RANGE
    assert code(65, [], [1] * 65, None, 8, 2) == lib.FDC_ERR_RANGE
    assert code(2, [], [4, 0], None, 8, 2) == lib.FDC_ERR_RANGE
    assert code(2, [], [4, 4], [0, 4], 8, 2) == lib.FDC_ERR_RANGE
    assert code(2, [], [4, 4], None, -1, 2) == lib.FDC_ERR_RANGE
    assert code(2, [], [4, 4], None, 8, 0) == lib.FDC_ERR_RANGE
    assert "cycle" in lib.fdc_strerror(lib.FDC_ERR_CYCLE)
    assert lib.fdc_kernel_name(1) == "ref_cuda_core"
    assert lib.fdc_launch_count() >= 0
