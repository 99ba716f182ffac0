"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared symbol,
and rejects bad arguments with a status before anything is enqueued."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2603_13180_b200 import build
    build.build_library()
    from paper_2603_13180_b200 import binding as b
    return b


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mxnorm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mx\w+|rmsnorm\w+)\s*\(", text)) - {"mxn_status", "mxn_round", "mxn_scale_layout"})


def test_library_exports_every_declared_symbol(binding):
    names = declared_functions()
    assert {"mx_cast", "rmsnorm_mxfp8_fwd", "mxnorm_fwd", "mxnorm_nvfp4_fwd", "mxnorm_bwd",
            "mxnorm_bwd_workspace_bytes", "mxn_scale_bytes", "mxn_status_string"} <= set(names)
    for n in names:
        assert hasattr(binding.lib, n), n
    assert set(binding.EXPORTS) <= set(names)


def test_status_strings(binding):
    seen = {binding.status_string(i) for i in range(8)}
    assert len(seen) == 8 and binding.status_string(0) == "ok" and binding.status_string(99) == "unknown status"


def test_scale_bytes(binding):
    assert binding.scale_bytes(16384, 128, 0) == 16384 * 128
    assert binding.scale_bytes(16384, 128, 1) == 16384 * 128
    assert binding.scale_bytes(200, 6, 1) == 2 * 2 * 512
    assert binding.scale_bytes(1, 1, 1) == 512
    assert binding.scale_bytes(5, 5, 7) == 0


FAKE = 0x7F0000000000   # never dereferenced: every call below must fail (or return) before a launch


def test_argument_errors_are_statuses(binding):
    L = binding.lib
    ok = dict(T=4, D=128, block=32)
    call = lambda **kw: L.mxnorm_fwd(kw.get("x", FAKE), None, kw.get("T", 4), kw.get("D", 128), kw.get("block", 32),
                                     kw.get("p", 2), 0.0, 0.0, kw.get("codes", FAKE), kw.get("scales", FAKE), None,
                                     kw.get("round", 0), kw.get("layout", 0), None)
    assert call(T=0) == 0                         # empty input: ok, nothing launched
    assert call(T=-1) == 2 and call(D=0) == 2 and call(D=100) == 2 and call(block=8) == 2 and call(block=48) == 2
    assert call(D=32 * 32768 + 32) == 2           # wider than 8 warps x 128 elements per lane
    assert call(p=3) == 2
    assert call(round=3) == 4 and call(layout=2) == 4
    assert call(x=None) == 1 and call(codes=None) == 1 and call(scales=None) == 1
    assert call(x=FAKE + 16) == 3 and call(codes=FAKE + 8) == 3
    assert L.mx_cast(None, 4, 128, 32, FAKE, FAKE, 0, 0, None) == 1
    assert L.rmsnorm_mxfp8_fwd(FAKE, FAKE + 2, 4, 128, 32, 0.0, FAKE, FAKE, None, 0, 0, None) == 3
    assert L.mxnorm_nvfp4_fwd(FAKE, 4, 100, 2, 0.0, 0.0, 1.0, FAKE, FAKE, None, 0, None) == 2
    assert L.mxnorm_nvfp4_fwd(FAKE, 0, 128, 2, 0.0, 0.0, 1.0, FAKE, FAKE, None, 0, None) == 0
    assert L.mxnorm_mxfp4_fwd(FAKE, 4, 100, 32, 2, 0.0, 0.0, FAKE, FAKE, None, 0, None) == 2
    assert L.mxnorm_mxfp4_fwd(FAKE, 4, 128, 32, 5, 0.0, 0.0, FAKE, FAKE, None, 0, None) == 2
    assert L.mx_cast_fp4(FAKE, 4, 128, 32, None, FAKE, 0, None) == 1
    assert L.rmsnorm_mxfp4_fwd(FAKE, 4, 128, 32, 0.0, FAKE, FAKE, None, 3, None) == 4
    # backward
    ws = binding.mxnorm_bwd_workspace_bytes(64, 4096)
    assert ws > 0 and ws % (4096 * 4) == 0
    assert binding.mxnorm_bwd_workspace_bytes(64, 4100) == 0
    assert binding.mxnorm_bwd_workspace_bytes(64, 32768) == 0      # wider than the backward supports
    bwd = lambda **kw: L.mxnorm_bwd(kw.get("x", FAKE), FAKE, None, kw.get("rms", FAKE), kw.get("T", 64), kw.get("D", 4096),
                                    kw.get("dx", FAKE), 0, kw.get("dgain", FAKE), kw.get("ws", FAKE), kw.get("wsb", ws), None)
    assert bwd(D=4100) == 2 and bwd(T=-2) == 2
    assert bwd(x=None) == 1 and bwd(rms=None) == 1 and bwd(dx=None) == 1
    assert bwd(ws=None) == 5 and bwd(wsb=ws - 1) == 5
    assert bwd(x=FAKE + 2) == 3 and bwd(ws=FAKE + 4) == 3


def test_every_accepted_shape_has_a_kernel(binding):
    # host-only walk of the launchers: every row length the argument checks admit, with every option an entry point can
    # ask for, must select a compiled forward kernel, and every backward plan must fit the kernel it launches
    missing, first_d, first_case = binding.selftest_dispatch(1 << 17)
    assert missing == 0, (missing, first_d, first_case)
    n = ctypes.c_longlong(7)
    assert binding.lib.mxn_selftest_dispatch(8, ctypes.byref(n), None, None) == 2
    assert binding.lib.mxn_selftest_dispatch(4096, None, None, None) == 1


def test_backward_workspace_size_does_not_decrease_with_rows(binding):
    # the launch plan depends on the row count; the workspace a caller sized for T rows must serve fewer rows too
    for D in (1024, 1536, 2048, 3072, 4096, 5120, 8192, 16384):
        sizes = [binding.mxnorm_bwd_workspace_bytes(T, D) for T in (1, 7, 300, 2000, 16384, 32768, 65536, 1 << 20)]
        assert all(a <= b for a, b in zip(sizes, sizes[1:])) and sizes[0] > 0, (D, sizes)


def test_binding_module_has_no_fallback():
    src = open(os.path.join(ROOT, "paper_2603_13180_b200", "binding.py")).read()
    assert "oracle" not in src.replace("CPU oracle", "")
    assert "raise ImportError" in src


def test_header_is_plain_c(tmp_path):
    """The boundary is a C ABI: the header must compile as C99 on its own, with no CUDA or C++ headers."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    src = tmp_path / "use_header.c"
    src.write_text('#include "mxnorm.h"\n'
                   "int main(void) { return mxn_scale_bytes(0, 0, MXN_SCALES_ROWMAJOR) == 0 && MXN_OK == 0 ? 0 : 1; }\n")
    r = subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-Werror", "-pedantic", "-fsyntax-only",
                        "-I", os.path.join(ROOT, "include"), str(src)], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr


def test_library_links_and_runs_from_c(binding, tmp_path):
    """A C program linked against libmxnorm.so calls the host-only entry points (no GPU needed)."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no C compiler")
    libdir = os.path.join(ROOT, "paper_2603_13180_b200")
    src = tmp_path / "link_test.c"
    src.write_text('#include <stdio.h>\n#include <string.h>\n#include "mxnorm.h"\n'
                   "int main(void) {\n"
                   "    if (mxn_scale_bytes(16384, 128, MXN_SCALES_SWIZZLE_128x4) != 16384u * 128u) return 1;\n"
                   "    if (mxn_scale_bytes(130, 5, MXN_SCALES_SWIZZLE_128x4) != 2u * 2u * 512u) return 2;\n"
                   "    if (strlen(mxn_status_string(MXN_ERR_ALIGN)) == 0) return 3;\n"
                   "    if (mx_cast(0, -1, 4096, 32, 0, 0, MXN_ROUND_RCEIL_POW2, MXN_SCALES_ROWMAJOR, 0) != MXN_ERR_SHAPE) return 4;\n"
                   "    if (mxnorm_fwd(0, 0, 0, 4096, 32, 2, 0.0f, 0.0f, 0, 0, 0, MXN_ROUND_RCEIL_POW2, MXN_SCALES_ROWMAJOR, 0) != MXN_OK) return 5;\n"
                   '    puts("ok");\n    return 0;\n}\n')
    exe = tmp_path / "link_test"
    r = subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src),
                        "-L", libdir, "-lmxnorm", "-Wl,-rpath," + libdir, "-o", str(exe)], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    r = subprocess.run([str(exe)], capture_output=True, text=True)
    assert r.returncode == 0 and r.stdout.strip() == "ok", (r.returncode, r.stdout, r.stderr)
