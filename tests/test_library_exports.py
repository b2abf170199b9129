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


def test_stage_level_calls_refuse_misaligned_or_oversized_arguments_on_the_host():
    """Every pointer the kernels read with wide or 64-bit accesses is checked before any launch: a bad
    argument is a status, never a device fault.  (Fake addresses: nothing is dereferenced, nothing launches.)"""
    lib = binding.load_library()
    A = 0x7F0000000000            # a 256-byte aligned, never dereferenced address
    good = dict(h=A, hw=A + 0x10000, hb=A + 0x20000, cw=A + 0x30000, cb=A + 0x40000, lo=A + 0x50000, pr=A + 0x60000,
                ma=A + 0x70000, re=A + 0x80000, sc=A + 0x90000)

    def post(channels_last=1, hm=8, wm=8, hidden=16, **over):
        a = dict(good, **over)
        return lib.tt_postprocess(a["h"], channels_last, 1, hm, wm, hidden, 4, a["hw"], a["hb"], a["cw"], a["cb"], 1, 0.5,
                                  a["lo"], a["pr"], a["ma"], a["re"], a["sc"], None)

    def post_static(**over):
        a = dict(good, **over)
        return lib.tt_postprocess_static(a["h"], 1, 1, 8, 8, 16, 4, a["hw"], a["hb"], a["cw"], a["cb"], 1, 0.5,
                                         a["lo"], a["pr"], a["ma"], a["re"], None)

    assert post(h=A + 4) == 1 and b"misaligned" in lib.tt_last_error(None)       # channels-last rows are read 16 bytes at a time
    assert post(channels_last=0, h=A + 2) == 1                                   # planar input: 4-byte alignment
    assert post(sc=A + 0x90004) == 1 and b"scratch_dev" in lib.tt_last_error(None)   # 64-bit atomics on the scratch
    assert post(re=A + 0x80004) == 1                                             # result records hold 64-bit members
    assert post(lo=A + 0x50002) == 1 and post(pr=A + 0x60001) == 1 and post(hw=A + 0x10002) == 1 and post(cb=A + 0x40001) == 1
    assert post(hm=16385) == 1 and post(wm=20000) == 1                           # map extents are bounded
    assert post(hidden=514) == 2
    assert post_static(h=A + 8) == 1 and post_static(re=A + 0x80004) == 1
    # preprocess: fp32 destination; overlay: RGBA8 destination written as words; extents bounded
    assert lib.tt_preprocess(A, 1, 0, 8, 8, 24, A + 0x10002, 4, 4, 255.0, 0.5, 0.25, None) == 1
    assert b"dst_dev" in lib.tt_last_error(None)
    pal = (C.c_uint8 * 24)()
    assert lib.tt_overlay(A, 1, 0, 8, 8, 24, A + 0x10000, 4, 4, 4, pal, A + 0x20002, None) == 1
    assert b"dst_dev" in lib.tt_last_error(None)
    assert lib.tt_overlay(A, 1, 0, 8, 8, 24, A + 0x10000, 4, 20000, 4, pal, A + 0x20000, None) == 1
    assert lib.tt_debug_expire_wait(None, 1000) == 1
    assert lib.tt_render_layers(A, 1, 0, 8, 8, 24, A + 0x10000, 4, 4, 4, pal, 0, 0, A + 0x20000, None) == 1      # layers < 1
    assert lib.tt_render_layers(A, 1, 0, 8, 8, 24, A + 0x10000, 4, 4, 4, pal, 2, 0, A + 0x20001, None) == 1      # misaligned output


def test_option_indices_in_the_binding_match_the_header():
    text = open(os.path.join(ROOT, "include", "tt.h")).read()
    declared = {name: int(val) for name, val in re.findall(r"\b(TT_OPT_[A-Z_0-9]+)\s*=\s*(\d+)", text)}
    assert declared and len(set(declared.values())) == len(declared) and max(declared.values()) < 8
    for name, val in declared.items():
        assert getattr(binding, name) == val, name
    for name in dir(binding):
        if name.startswith("TT_OPT_"):
            assert name in declared, f"{name} is not in tt.h"


def test_limits_in_the_binding_match_the_header():
    text = open(os.path.join(ROOT, "include", "tt.h")).read()
    for name in ("TT_MAX_STREAMS", "TT_MAX_TOOLS", "TT_MAX_ENC", "TT_MAX_IN_FLIGHT"):
        (val,) = re.findall(r"#define\s+%s\s+(\d+)" % name, text)
        assert getattr(binding, name) == int(val), name
