"""The C-ABI library builds, loads and exports every symbol include/tempo.h declares (no GPU, no compute)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "tempo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tempo_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_four_hot_path_calls():
    names = _declared()
    for n in ("tempo_count_dispatch", "tempo_permute_pad", "tempo_grouped_ffn", "tempo_unpermute_combine"):
        assert n in names


def test_library_exports_every_declared_symbol():
    from paper_2608_13057_b200 import build
    lib = ctypes.CDLL(build.build())
    for n in _declared():
        assert hasattr(lib, n), n
    from paper_2608_13057_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    assert binding.tempo_version() >= 1


def test_host_only_entry_points_and_argument_errors():
    from paper_2608_13057_b200 import binding as B
    s = B.make_shape(256, 8, 128, 20, 2, 4096, 1536, 128)
    assert B.tempo_m_cap_bound(s) == 2048 + 20 * 128
    assert B.tempo_sf_bytes(256, 4096) == 2 * 8 * 512
    assert B.tempo_sf_bytes(128, 256) == 512            # 2 column blocks still take one atom
    assert B.tempo_workspace_bytes(B.make_shape(256, 8, 128, 20, 2, 4096, 1536, 4608)) == 512
    s = B.make_shape(256, 8, 128, 20, 2, 4096, 1536, 4608)
    n = B.tempo_packed_weight_bytes(s)
    assert n >= 20 * 3 * 4096 * 1536 and n % 1024 == 0
    bad = B.make_shape(256, 8, 128, 20, 2, 4000, 1536, 4608)
    out = ctypes.c_size_t(0)
    assert B._lib.tempo_packed_weight_bytes(ctypes.byref(bad), ctypes.byref(out)) == -2
    big = B.make_shape(256, 64, 128, 20, 2, 4096, 1536, 4608)
    assert B._lib.tempo_packed_weight_bytes(ctypes.byref(big), ctypes.byref(out)) == -3
    assert B._lib.tempo_packed_weight_bytes(None, ctypes.byref(out)) == -1
    # a hot-path call with a NULL pointer launches nothing and reports it (no device needed)
    null = ctypes.c_void_p(0)
    rc = B._lib.tempo_unpermute_combine(ctypes.byref(s), null, null, null, null, null, null, null)
    assert rc == -1 and b"NULL" in B._lib.tempo_status_string(rc)
