"""The C-ABI library loads and exports every function that include/hisparse.h declares (no compute calls:
this runs without a GPU), and the argument checks that need no device work."""
import ctypes
import os
import re

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "hisparse.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hisparse_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2608_07009_b200 import build, hisparse
    build.build_cuda()
    lib = ctypes.CDLL(build.SO)
    names = declared_functions()
    assert len(names) >= 20
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, missing
    assert sorted(hisparse.EXPORTS) == names     # the binding knows every entry point, and no other


def test_error_strings_and_device_bytes_need_no_gpu():
    from paper_2608_07009_b200 import hisparse as hs
    lib = hs.lib()
    for code in (hs.OK, hs.EINVAL, hs.ENOTPINNED, hs.ENOMEM, hs.ECUDA, hs.ESTATE, hs.ETOOBIG):
        assert lib.hisparse_strerror(code)
    kv, meta = hs.device_bytes(32, 16, 1, 4096, 2048, 1152, [33000] * 32)
    assert kv == 32 * 16 * 4097 * 1152           # N * L * (B + 1) * E
    assert meta < kv // 10
    # the footprint bound of the paper's admission step: proportional to B, independent of the context length
    kv_long, _ = hs.device_bytes(32, 16, 1, 4096, 2048, 1152, [1 << 20] * 32)
    assert kv_long == kv


def test_create_validates_before_touching_a_device():
    from paper_2608_07009_b200 import hisparse as hs
    cap = np.array([64], dtype=np.int64)
    il = np.array([10], dtype=np.int64)
    cfg = hs.Config(1, 1, 1, 4, 8, 32, cap.ctypes.data, il.ctypes.data, None, 0, 0, 0, 0, 0)    # k > B
    h = ctypes.c_void_p()
    assert hs.lib().hisparse_create(ctypes.byref(cfg), ctypes.byref(h)) == hs.EINVAL
    assert not h.value
    st = hs.ExternalState()
    assert hs.lib().hisparse_resolve_noalloc(ctypes.byref(st), None, None, None, None, None, None) == hs.EINVAL
