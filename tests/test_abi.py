"""The C-ABI library loads without a GPU and exports every symbol that include/oz.h declares."""
import ctypes
import os
import re

import paper_2609_09095_b200 as oz
from paper_2609_09095_b200 import build as ozbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "oz.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(oz_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_the_header():
    ozbuild.build_library()
    lib = ctypes.CDLL(oz.LIB_PATH)
    names = declared_functions()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(names) == sorted(oz.EXPORTS)


def test_host_only_queries():
    r, p, mods = oz.oz_set_info(oz.OZ_SET_S)
    assert (r, p) == (12, 30) and mods[0] == 1089 and mods[-1] == 487
    r, p, mods = oz.oz_set_info(oz.OZ_SET_E)
    assert (r, p) == (13, 33) and mods[-1] == 227
    r, p, mods = oz.oz_set_info(oz.OZ_SET_A)
    assert (r, p) == (15, 44) and mods[0] == 256 and mods[-1] == 197
    assert oz.oz_plane_count(oz.OZ_SET_A, oz.OZ_SUB_INT8_NATIVE) == 15
    assert oz.oz_plane_count(oz.OZ_SET_S, oz.OZ_SUB_INT8_NATIVE) == 0      # native INT8 needs byte moduli
    assert oz.oz_plane_count(oz.OZ_SET_S, 0) == 30 and oz.oz_plane_count(oz.OZ_SET_E, oz.OZ_SUB_INT8) == 33
    assert oz.oz_row_pitch(1) == 16 and oz.oz_row_pitch(5003) == 5008 and oz.oz_row_pitch(4096) == 4096
    # residues of the all-byte set are stored as bytes
    assert [oz.oz_residue_elem_bytes(s) for s in (oz.OZ_SET_S, oz.OZ_SET_E, oz.OZ_SET_A, 7)] == [2, 2, 1, 0]
    assert oz.oz_workspace_bytes(4096, 4096, 512, oz.OZ_SET_A, oz.OZ_SUB_INT8_NATIVE) < 15 * (8192 * 512 + 4096 * 4096) + (1 << 22)
    # planes of A and B + residues dominate the workspace
    m, n, k = 16384, 16384, 1024
    need = oz.oz_workspace_bytes(m, n, k, oz.OZ_SET_S, oz.OZ_ACC_SEPARATE)
    assert need >= 30 * (m + n) * k + 24 * m * n
    assert need < 30 * (m + n) * k + 24 * m * n + (1 << 22)
    # default route: merged accumulators; the pre-scaled plane takes the place of d1, same workspace
    assert oz.oz_workspace_bytes(m, n, k, oz.OZ_SET_S, 0) == need
    assert oz.oz_workspace_bytes(m, n, k, 7, 0) == 0
    assert "workspace" in oz.oz_status_string(oz.OZ_ERR_WORKSPACE)


def test_header_is_plain_c(tmp_path):
    """include/oz.h is a C header: it compiles as C99 with no C++ or CUDA types, and a C program can
    name every entry point."""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    import paper_2609_09095_b200 as oz
    src = tmp_path / "use_oz.c"
    calls = "\n".join(f"    p[{i}] = (fn_t)&{name};" for i, name in enumerate(oz.EXPORTS))
    src.write_text('#include "oz.h"\ntypedef void (*fn_t)(void);\nint main(void)\n{\n    fn_t p[%d];\n%s\n'
                   '    return p[0] == 0;\n}\n' % (len(oz.EXPORTS), calls))
    inc = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include")
    subprocess.run([gcc, "-std=c99", "-Wall", "-Werror", "-pedantic", "-fsyntax-only", "-I", inc, str(src)], check=True)
