"""The C-ABI library loads and exports every function include/klpm.h declares (no compute, no GPU)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "klpm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:rt|klpm)_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2502_04677_b200 import build
    path = build.build()
    lib = ctypes.CDLL(path)
    names = declared_functions()
    assert {"rt_build", "rt_insert", "rt_match_batch", "klpm_select", "klpm_replay"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    lib.klpm_abi_version.restype = ctypes.c_int32
    assert lib.klpm_abi_version() >= 1


def test_binding_has_the_same_names():
    from paper_2502_04677_b200 import build
    build.build()
    from paper_2502_04677_b200 import binding
    for name in declared_functions():
        assert hasattr(binding, name) or name in binding.EXPORTS, name
    assert set(binding.EXPORTS) == set(declared_functions())


def test_host_side_argument_checks_need_no_gpu():
    from paper_2502_04677_b200 import build
    build.build()
    from paper_2502_04677_b200 import binding as K
    lib = K.lib()
    assert lib.rt_create(None, None) == K.RT_ERR_INVALID
    assert lib.rt_destroy(None) == K.RT_ERR_INVALID
    assert lib.rt_match_batch(None, None, None, 0, None, None, None, None) == K.RT_ERR_INVALID
    bad = K.make_params(K.POLICY_KLPM, k=0)
    assert lib.klpm_select(None, None, None, 0, 0, ctypes.byref(bad), None, None) == K.RT_ERR_INVALID
