"""The C-ABI library builds, loads and exports every symbol include/tt.h declares (no GPU needed)."""
import ctypes as C
import os
import re

from paper_2402_04466_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "tt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tt_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound():
    lib = binding.load_library()
    declared = _declared_symbols()
    assert "tt_create" in declared and "tt_submit_frames" in declared and "tt_sync" in declared and "tt_destroy" in declared
    for name in declared:
        assert hasattr(lib, name), f"libtt.so does not export {name}"
    assert set(binding.EXPORTED_SYMBOLS) == set(declared)
    assert lib.tt_abi_version() == binding.TT_ABI_VERSION


def test_struct_layouts_match_the_header():
    # sizes of the C structs as compiled by gcc from the header itself
    import subprocess, tempfile
    src = '#include "tt.h"\n#include <stdio.h>\nint main(){printf("%zu %zu %zu %zu\\n", sizeof(tt_config), sizeof(tt_weights), sizeof(tt_frame), sizeof(tt_result));return 0;}\n'
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "s.c"); exe = os.path.join(d, "s")
        open(c, "w").write(src)
        subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), c, "-o", exe], check=True)
        sizes = [int(x) for x in subprocess.run([exe], capture_output=True, text=True, check=True).stdout.split()]
    assert sizes == [C.sizeof(binding.tt_config), C.sizeof(binding.tt_weights), C.sizeof(binding.tt_frame), C.sizeof(binding.tt_result)]


def test_argument_errors_need_no_gpu():
    lib = binding.load_library()
    out = C.c_void_p()
    assert lib.tt_create(None, None, C.byref(out)) == 1 and not out.value
    cfg = binding.tt_config()
    w = binding.tt_weights()
    assert lib.tt_create(C.byref(cfg), C.byref(w), C.byref(out)) == 1      # struct_size == 0
    assert b"struct_size" in lib.tt_last_error(None)
    assert lib.tt_destroy(None) == 0
    assert lib.tt_postprocess_scratch_bytes(0, 1, 1, 4, 1) == 0
    assert lib.tt_postprocess_scratch_bytes(2, 60, 80, 128, 7) > 0
    assert lib.tt_preprocess(None, 1, 0, 8, 8, 24, None, 4, 4, 255.0, 0.5, 0.25, None) == 1
