"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and sizes workspaces."""
import os
import re

import paper_2511_02647_b200 as fa

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "fedattn.h")).read()
    declared = set(re.findall(r"\b(fedattn_[a-z_]+)\s*\(", hdr))
    assert declared, "no declarations found"
    import ctypes
    lib = ctypes.CDLL(fa.library_path())
    for name in sorted(declared):
        assert hasattr(lib, name), "library does not export %s" % name
    assert set(fa.exported_symbols()) == declared


def test_workspace_bytes_and_status_strings():
    s = fa.Shape(4, 32, 8, 128, fa.BF16)
    assert fa.fedattn_workspace_bytes(s, 8192, 8192) >= 256
    assert fa.fedattn_workspace_bytes(fa.Shape(4, 32, 7, 128, fa.BF16), 10, 10) == 0      # Hq % Hkv
    assert fa.fedattn_workspace_bytes(fa.Shape(4, 32, 8, 100, fa.BF16), 10, 10) == 0      # head_dim % 8
    assert fa.fedattn_workspace_bytes(fa.Shape(65, 32, 8, 128, fa.BF16), 10, 10) == 0     # too many participants
    assert fa.status_string(0) == "ok" and "invalid" in fa.status_string(1)
