"""The C-ABI library loads without a GPU and exports every function include/hap.h declares."""
import ctypes
import os
import re

import paper_2609_39350_b200 as hap
from paper_2609_39350_b200.build import build_library, LIB

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "hap.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hap_[a-z0-9_]+)\s*\(", text)))


def test_header_functions_are_exported_and_bound():
    build_library()
    lib = ctypes.CDLL(LIB)
    names = _declared_functions()
    assert "hap_problem_create" in names and "hap_search_best" in names and "hap_pipeline_dp" in names
    for n in names:
        assert getattr(lib, n) is not None, n
    assert sorted(hap.EXPORTS) == names
    for n in names:
        if n not in ("hap_status_str", "hap_last_error"):
            assert hasattr(hap, n), f"python binding lacks {n}"


def test_status_strings_and_null_arguments():
    lib = hap.load_library()
    assert lib.hap_status_str(0) == b"HAP_OK" and lib.hap_status_str(6) == b"HAP_E_INFEASIBLE"
    out = ctypes.c_void_p(0)
    assert lib.hap_problem_create(None, None, None, None, ctypes.byref(out)) == 1 and not out.value
    assert lib.hap_enumerate(None, None, None) == 1
    lib.hap_problem_destroy(None)
    # blobs are validated before any device work: garbage is refused without a GPU
    for blob in (b"", b"not a blob at all....", b"HAPBLOB1" + (24).to_bytes(8, "little") + b"\0" * 8):
        out = ctypes.c_void_p(0)
        assert lib.hap_problem_load(blob, ctypes.c_uint64(len(blob)), ctypes.byref(out)) == 1 and not out.value
    sites = ctypes.c_uint64(7)
    assert lib.hap_self_check(ctypes.byref(sites)) == 5 and sites.value == 0      # HAP_E_STATE: not the self-checking build


def test_layouts_match_the_header_sizes():
    from paper_2609_39350_b200 import binding as b
    assert b.PCONF_DTYPE.itemsize == 80 and b.CANDIDATE_DTYPE.itemsize == 96
    assert ctypes.sizeof(b._Plan) == 8 + 8 * 4 + 8 + 3 * 32 + 5 * 8


def test_binding_remembers_array_addresses_per_problem_object_only():
    """The binding keeps the address of a problem's arrays per object and field: a field that is reassigned, a copy of
    the problem and an array that needs converting each get their own, current address."""
    import copy
    import gc
    import numpy as np
    from gen import problems
    from paper_2609_39350_b200 import binding as b
    pb = problems.tiny()
    keep = []
    memo = b._address_memo(pb)
    assert b._address_memo(pb) is memo
    a1 = b._field_address(memo, pb, "tdf", np.float64, keep)
    assert a1 == pb.tdf.ctypes.data and b._field_address(memo, pb, "tdf", np.float64, keep) == a1 and keep[-1] is pb.tdf
    pb.tdf = pb.tdf.copy()                                           # a new array in the same field
    a2 = b._field_address(memo, pb, "tdf", np.float64, keep)
    assert a2 == pb.tdf.ctypes.data and a2 != a1
    pb.tp_list = [int(x) for x in pb.tp_list]                         # a list: converted, the converted array is kept alive
    a3 = b._field_address(memo, pb, "tp_list", np.int32, keep)
    assert a3 == keep[-1].ctypes.data and keep[-1].dtype == np.int32 and keep[-1].tolist() == pb.tp_list
    assert b._field_address(memo, pb, "tp_list", np.int32, keep) == a3
    other = copy.deepcopy(pb)                                         # copies start without addresses
    m2 = b._address_memo(other)
    assert m2 is not memo and not m2
    assert b._field_address(m2, other, "tdf", np.float64, keep) == other.tdf.ctypes.data != a2
    key = id(other)
    del other, m2
    gc.collect()
    assert key not in b._ADDRESSES
