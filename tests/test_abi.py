"""CPU-only checks of the boundary: the library builds, loads and exports every symbol that
include/spiral.h declares; argument validation that needs no device."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "spiral.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spiral_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2506_24119_b200 import build
    build.build()
    import paper_2506_24119_b200 as sp
    lib = ctypes.CDLL(sp.LIB_PATH)
    names = _declared()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(sp.EXPORTS) == names


def test_host_only_entry_points_validate_arguments():
    import paper_2506_24119_b200 as sp
    import synth
    assert sp.spiral_strerror(0) == "ok"
    assert "KV pages" in sp.spiral_strerror(sp.SPIRAL_ERR_OOM)
    assert sp.spiral_kv_page_bytes(synth.shape("qwen3_4b"), 16) == 16 * synth.kv_bytes_per_token(synth.shape("qwen3_4b"))
    lib = ctypes.CDLL(sp.LIB_PATH)
    lib.spiral_kv_seq_len.restype = ctypes.c_int
    assert lib.spiral_kv_seq_len(None, 0, None) == sp.SPIRAL_ERR_INVALID
    assert lib.spiral_kv_release(None, 0, None) == sp.SPIRAL_ERR_INVALID
    assert lib.spiral_init(None, None, None, 0, 1, 1) == sp.SPIRAL_ERR_INVALID
    assert lib.spiral_decode_step(None, None, 1, None, None, None, ctypes.c_float(1.0), None, None, None) == sp.SPIRAL_ERR_INVALID
