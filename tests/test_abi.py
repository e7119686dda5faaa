"""The C-ABI library loads and exports every symbol include/fastmtp.h declares (no compute calls)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "fastmtp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(fmtp_[a-z_0-9]+|fastmtp_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2509_18362_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = _declared()
    assert {"fastmtp_draft", "fastmtp_verify_accept", "fastmtp_target_step", "fmtp_create"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in fastmtp.h but not exported"


def test_binding_export_list_matches_header():
    import importlib
    if not os.path.exists(os.path.join(ROOT, "paper_2509_18362_b200", "libfastmtp.so")):
        from paper_2509_18362_b200 import build
        build.build()
    B = importlib.import_module("paper_2509_18362_b200.binding")
    assert sorted(B.EXPORTS) == _declared()
    assert B.lib.fmtp_strerror(0) == b"ok" and B.lib.fmtp_strerror(-6).startswith(b"a bounded")


def test_host_argument_validation_needs_no_gpu():
    """Null / out-of-range arguments are rejected before any CUDA call."""
    import importlib
    B = importlib.import_module("paper_2509_18362_b200.binding")
    assert B.lib.fmtp_create(None, None) == -1
    assert B.lib.fmtp_workspace_bytes(None) == 0
    assert B.lib.fmtp_destroy(None) == -1
