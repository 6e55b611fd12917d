"""CPU-only checks of the boundary: the built library loads and exports every symbol that
include/graft.h declares, and the ctypes structures match the header's field lists."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "graft.h")


def declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(graft_[a-z_0-9]+)\s*\(", text)))


def struct_fields(name):
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    end = text.index("} %s;" % name)
    body = text[text.rindex("typedef struct {", 0, end) + len("typedef struct {"):end]
    fields = []
    for decl in body.split(";"):
        decl = decl.strip()
        if not decl:
            continue
        # "int B, N_max" / "const int32_t* draft_token" / "int64_t a, b"
        names = re.sub(r"^(const\s+)?[A-Za-z_0-9]+\s*\*?\s*", "", decl)
        fields += [n.strip().lstrip("*").strip() for n in names.split(",")]
    return fields


@pytest.fixture(scope="module")
def lib():
    from paper_2605_20104_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_four_steps():
    fns = declared_functions()
    for need in ("graft_build_tree", "graft_tree_verify_attn", "graft_accept", "graft_compact_kv"):
        assert need in fns


def test_library_exports_every_declared_symbol(lib):
    for fn in declared_functions():
        assert hasattr(lib, fn), fn


def test_binding_lists_the_same_entry_points(lib):
    from paper_2605_20104_b200 import binding
    assert sorted(binding.EXPORTS) == [f for f in declared_functions()]
    for fn in binding.EXPORTS:
        assert callable(getattr(binding, fn, None)) or fn in ("graft_create", "graft_destroy", "graft_status_string",
                                                              "graft_device_status")


@pytest.mark.parametrize("cname,pyname", [("graft_build_params", "BuildParams"), ("graft_attn_params", "AttnParams"),
                                          ("graft_accept_params", "AcceptParams"),
                                          ("graft_compact_params", "CompactParams"),
                                          ("graft_update_params", "UpdateParams"),
                                          ("graft_envelope_params", "EnvelopeParams"),
                                          ("graft_paths_params", "PathsParams"),
                                          ("graft_accept_stochastic_params", "AcceptStochasticParams")])
def test_struct_layouts_follow_the_header(cname, pyname):
    from paper_2605_20104_b200 import binding
    assert [f[0] for f in getattr(binding, pyname)._fields_] == struct_fields(cname)


def test_status_strings(lib):
    lib.graft_status_string.restype = ctypes.c_char_p
    assert lib.graft_status_string(0) == b"ok"
    assert b"workspace" in lib.graft_status_string(-3)


def test_host_side_argument_checks_need_no_gpu(lib):
    """Null handles are rejected before anything touches a device."""
    for fn in ("graft_build_tree", "graft_tree_verify_attn", "graft_accept", "graft_compact_kv", "graft_update_adjacency",
               "graft_retrieve_envelope", "graft_path_indices", "graft_accept_stochastic"):
        f = getattr(lib, fn)
        f.restype = ctypes.c_int
        assert f(None, None, None) == -1
