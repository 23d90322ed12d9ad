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


def test_misaligned_pointers_are_rejected_on_the_host():
    """Pointers that are not aligned to their element type are a host-detectable error of the stage
    entry points: OZ_ERR_INVALID_ARG comes back before any CUDA call (so this runs without a GPU;
    the addresses are never dereferenced)."""
    base = 0x7F0000000000                     # any 256-byte aligned number
    m, n, k, pitch = 8, 8, 16, 16
    ok_args = dict(PA=base, PB=base + 4096, R=base + 8192)
    for set_id, elem in ((oz.OZ_SET_S, 2), (oz.OZ_SET_E, 2)):
        assert oz.oz_residue_gemm(m, n, k, ok_args["PA"], m * pitch, pitch, ok_args["PB"], n * pitch, pitch, set_id,
                                  0, ok_args["R"] + 1, m, m * n, 0) == oz.OZ_ERR_INVALID_ARG      # odd address, uint16 residues
        assert oz.oz_reconstruct(m, n, base + 1, m, m * n, base + 4096, base + 8192, set_id, 1.0, 0.0,
                                 base + 16384, m, 0) == oz.OZ_ERR_INVALID_ARG
    # shifts are int32, matrices are double
    assert oz.oz_reconstruct(m, n, base, m, m * n, base + 4098, base + 8192, oz.OZ_SET_S, 1.0, 0.0, base + 16384, m, 0) \
        == oz.OZ_ERR_INVALID_ARG
    assert oz.oz_reconstruct(m, n, base, m, m * n, base + 4096, base + 8194, oz.OZ_SET_A, 1.0, 0.0, base + 16384, m, 0) \
        == oz.OZ_ERR_INVALID_ARG
    assert oz.oz_reconstruct(m, n, base, m, m * n, base + 4096, base + 8192, oz.OZ_SET_A, 1.0, 0.0, base + 16388, m, 0) \
        == oz.OZ_ERR_INVALID_ARG
    assert oz.oz_deconstruct(0, m, k, base + 4, m, oz.OZ_SET_S, 0, base + 4096, m * pitch, pitch, base + 8192,
                             base + 16384, 0) == oz.OZ_ERR_INVALID_ARG                        # X not 8-byte aligned
    assert oz.oz_deconstruct(0, m, k, base, m, oz.OZ_SET_S, 0, base + 4096, m * pitch, pitch, base + 8194,
                             base + 16384, 0) == oz.OZ_ERR_INVALID_ARG                        # shift not 4-byte aligned
    assert oz.oz_deconstruct_static(1, n, k, base + 2, k, oz.OZ_SET_S, 0, base + 4096, n * pitch, pitch,
                                    base + 8192, 0) == oz.OZ_ERR_INVALID_ARG


def test_prepared_operand_sizes():
    """Host-only queries of the planes-kept-across-calls interface."""
    m, n, k = 16384, 16384, 1024
    a = oz.oz_operand_bytes(0, m, k, oz.OZ_SET_S, 0)
    b = oz.oz_operand_bytes(1, n, k, oz.OZ_SET_S, 0)
    assert 30 * m * k <= a < 30 * m * k + 21 * m + 4096 and a == b
    assert oz.oz_operand_bytes(0, m, k, oz.OZ_SET_A, oz.OZ_SUB_INT8_NATIVE) < 15 * m * k + 21 * m + 4096
    assert oz.oz_operand_bytes(2, m, k, oz.OZ_SET_S, 0) == 0
    assert oz.oz_operand_bytes(0, m, oz.OZ_K_MAX + 1, oz.OZ_SET_S, 0) == 0
    # inner dimension padded to whole 128-byte lines
    assert oz.oz_operand_bytes(0, 1000, 5003, oz.OZ_SET_S, 0) >= 30 * 1000 * 5120
    r = oz.oz_product_workspace_bytes(m, n, oz.OZ_SET_S)
    assert r == 24 * m * n
    assert oz.oz_product_workspace_bytes(m, n, oz.OZ_SET_A) == 15 * m * n
    # planes of both operands + residues = the workspace of the whole-method call
    assert oz.oz_workspace_bytes(m, n, k, oz.OZ_SET_S, 0) == a + b + r
    # ragged shapes are stored as whole tiles
    assert oz.oz_product_workspace_bytes(10007, 9973, oz.OZ_SET_S) == 24 * 10240 * 9984
