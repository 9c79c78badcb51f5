"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol that
include/plc.h declares, and its frequency tables are the oracle's."""
import os
import re

import numpy as np

import paper_2604_15356_b200 as plc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "plc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(plc_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    plc.build()
    lib = plc.lib()
    names = _declared()
    assert len(names) >= 15 and set(plc.EXPORTS) <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_table_constants_and_tables_equal_the_oracles(orc):
    plc.build()
    for qp in range(-24, 16):
        assert plc.table_constants(qp) == orc.table_constants(qp)
        f, c = plc.build_table(qp)
        fo, co = orc.build_table(qp)
        assert np.array_equal(f, fo) and np.array_equal(c, co)


def test_host_side_argument_checks():
    """Bad arguments are refused on the host before anything touches a device."""
    import ctypes as C
    plc.build()
    lib = plc.lib()
    h = C.c_void_p()
    cfg = plc.Config(1, 1, 48, 256, 16, 0.02, 0.0, 256, 0, 0)            # d = 48 unsupported
    assert lib.plc_create(C.byref(h), C.byref(cfg), C.c_void_p(4096)) == plc.E_SHAPE
    cfg = plc.Config(1, 1, 64, 256, 300, 0.02, 0.0, 256, 0, 0)           # K > V
    assert lib.plc_create(C.byref(h), C.byref(cfg), C.c_void_p(4096)) == plc.E_SHAPE
    cfg = plc.Config(1, 1, 64, 256, 16, 0.0, 0.0, 256, 0, 0)             # delta too small
    assert lib.plc_create(C.byref(h), C.byref(cfg), C.c_void_p(4096)) == plc.E_INVALID
    cfg = plc.Config(1, 1, 64, 256, 16, 0.02, 0.0, 256, 0, 0)
    assert lib.plc_create(C.byref(h), C.byref(cfg), C.c_void_p(4100)) == plc.E_ALIGN
    assert lib.plc_create(C.byref(h), C.byref(cfg), None) == plc.E_INVALID
    assert lib.plc_destroy(None) == plc.E_INVALID
    th, rh = C.c_uint32(), C.c_uint32()
    assert lib.plc_table_constants(16, C.byref(th), C.byref(rh)) == plc.E_INVALID
