"""The C-ABI library loads without a GPU and exports every symbol include/betty.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libpath():
    from paper_2207_02849_b200 import build
    return build.build()


def test_library_exports_every_declared_symbol(libpath):
    header = open(os.path.join(ROOT, "include", "betty.h")).read()
    code = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(betty_[a-z_0-9]+)\s*\(", code))
    assert {"betty_lower_step", "betty_hvp", "betty_mixed_vjp", "betty_hypergrad_neumann",
            "betty_hypergrad_cg", "betty_hypergrad_fd", "betty_chain_levels"} <= declared
    lib = ctypes.CDLL(libpath)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in betty.h but not exported"


def test_status_strings_and_host_side_argument_checks(libpath):
    import paper_2207_02849_b200 as bt
    assert bt.betty_status_string(0) == "ok"
    assert "breakdown" in bt.betty_status_string(bt.BETTY_ERR_BREAKDOWN)
    lib = bt.lib()
    # null descriptors are rejected before anything touches a device
    assert lib.betty_lower_step(None, 1, None, 0, None) == bt.BETTY_ERR_INVALID_ARG
    assert lib.betty_workspace_size(None, 0, None) == bt.BETTY_ERR_INVALID_ARG
    assert lib.betty_reset_status(None, 0, None) == bt.BETTY_ERR_WORKSPACE


def test_binding_struct_layout_matches_header():
    """Field order/types of the ctypes mirror follow the header's struct declaration."""
    from paper_2207_02849_b200 import binding
    header = open(os.path.join(ROOT, "include", "betty.h")).read()
    body = re.search(r"typedef struct betty_level \{(.*?)\} betty_level;", header, re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        for part in decl.split(","):
            names.append(re.findall(r"[A-Za-z_][A-Za-z_0-9]*", part)[-1])
    assert names == [f[0] for f in binding._Level._fields_]


def test_shared_memory_limits_are_remembered_per_device(libpath):
    """A kernel's raised shared-memory limit belongs to one device: what device 0 has set says nothing
    about device 1, a smaller request on the same device needs no new setting, a larger one does."""
    import paper_2207_02849_b200 as bt
    f = bt.betty_selftest_smem_limit
    assert f(True, 0, 98_000) is True
    assert f(False, 0, 98_000) is False
    assert f(False, 0, 64_000) is False
    assert f(False, 1, 64_000) is True          # another device starts from nothing
    assert f(False, 1, 98_000) is True
    assert f(False, 0, 200_000) is True         # grows on device 0
    assert f(False, 0, 98_000) is False
    assert f(False, -1, 1) is True and f(False, -1, 1) is True      # unknown ordinal: never cached
    assert f(False, 64, 1) is True
    assert f(True, 0, 10) is True               # reset forgets
