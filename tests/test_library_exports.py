"""The C-ABI library loads without a GPU and exports every symbol include/sat_b200.h declares (no compute calls here)."""
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "sat_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sat_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2308_13466_b200.binding as B
    declared = _declared()
    assert len(declared) >= 30
    for name in declared:
        assert hasattr(B._lib, name), f"{name} is declared in the header but not exported by the library"
    assert sorted(B.EXPORTS) == declared, "binding.EXPORTS and the header disagree"
    for name in declared:
        assert hasattr(B, name), f"binding has no function named {name}"


def test_no_device_gives_an_error_status_not_a_crash():
    import torch
    import paper_2308_13466_b200.binding as B
    if torch.cuda.is_available():
        return
    try:
        B.sat_create(0, 0)
    except B.SatError as e:
        assert e.status in (B.SAT_EINVAL, B.SAT_ECUDA)
    else:
        raise AssertionError("sat_create succeeded without a CUDA device")
