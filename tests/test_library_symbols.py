"""The C-ABI library loads and exports every symbol that include/psb.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_entry_point_is_exported():
    import __graft_entry__

    __graft_entry__.build()
    import paper_1904_02205_b200 as psb

    header = open(os.path.join(ROOT, "include", "psb.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(psb_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    lib = ctypes.CDLL(psb.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), "%s is declared in psb.h but not exported" % name
    assert declared == set(psb.EXPORTS)


def test_status_strings_and_host_side_validation_need_no_gpu():
    import paper_1904_02205_b200 as psb

    lib = psb.load_library()
    assert lib.psb_status_string(0) == b"PSB_OK"
    assert lib.psb_status_string(-6) == b"PSB_ERR_TIMEOUT"
    assert lib.psb_create(None, 0) == psb.PSB_ERR_INVALID_ARG
    assert lib.psb_destroy(None) == psb.PSB_ERR_INVALID_ARG
    assert lib.psb_set_sample_map(None, None, 0, 0, 0, 0) == psb.PSB_ERR_INVALID_ARG
