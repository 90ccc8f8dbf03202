"""Host-side checks of the C-ABI library: it loads, exports every declared
symbol, validates arguments, and its budget helpers match the paper's tables.
No kernel is launched here (CPU only)."""
import ctypes as C
import os
import re

import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def pb():
    entry.build()
    from paper_2607_27591_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(pb):
    header = open(os.path.join(ROOT, "include", "prox.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(prox_[a-z0-9_]+)\s*\(", header))
    assert len(declared) >= 20
    lib = C.CDLL(os.path.join(ROOT, "paper_2607_27591_b200", "libprox.so"))
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(pb.EXPORTED)


def test_no_torch_types_in_signatures():
    header = open(os.path.join(ROOT, "include", "prox.h")).read()
    assert "torch" not in header.lower() and "at::" not in header and "Tensor" not in header


def test_status_strings(pb):
    assert pb.prox_status_string(0) == "ok"
    for s in range(1, 8):
        assert pb.prox_status_string(s) not in ("ok", "unknown status")
    assert pb.prox_status_string(99) == "unknown status"
    assert "sm_100a" in pb.prox_version()


def _rows():
    for line in open(os.path.join(GOLDEN, "stagewise_allocation.txt")):
        line = line.split("#")[0].strip()
        if line:
            src, e, cap, s1, s2 = line.split()
            yield float(e) / 100, float(cap) / 100, (None if s1 == "-" else float(s1) / 100), float(s2)


def test_budget_helper_matches_printed_tables(pb):
    """Sec. 4.2 allocation rule against the two tables the paper prints."""
    for e, cap, s1_want, s2_want in _rows():
        s1, s2 = pb.prox_allocate_budget(e, 1 / 3, 0.7, 0.0, cap)
        assert f"{100 * s2:.1f}" == f"{s2_want:.1f}"
        if s1_want is not None:
            assert abs(s1 - s1_want) < 1e-9


def test_budget_helper_matches_workload_table(pb):
    from paper_2607_27591_b200 import inputs
    for wl in inputs.WORKLOADS.values():
        for e, (k1, k2) in wl.points.items():
            s1, s2 = pb.prox_allocate_budget(e / 100)
            assert (pb.prox_sparsity_to_k(s1, wl.d_model), pb.prox_sparsity_to_k(s2, wl.d_ff)) == (k1, k2)
    assert pb.prox_sparsity_to_k(1.0, 100) == 1
    assert pb.prox_sparsity_to_k(0.0, 100) == 100
    assert pb.prox_sparsity_to_k(0.995, 100) == 1
    assert pb.prox_sparsity_to_k(0.985, 100) == 2


def test_host_argument_validation(pb):
    out = C.c_void_p()
    cfg = pb.ProxFFNConfig(512, 1536, 1, 0)
    create = pb.raw("prox_ffn_create")
    assert create(None, 16, 16, 16, None, C.byref(out)) == 1          # null config
    assert create(C.byref(cfg), None, 16, 16, None, C.byref(out)) == 1  # null weights
    assert create(C.byref(cfg), 16, 16, 16, None, None) == 1          # null out
    assert create(C.byref(cfg), 8, 16, 16, None, C.byref(out)) == 1   # misaligned
    for bad, want in ((pb.ProxFFNConfig(500, 1536, 1, 0), 2), (pb.ProxFFNConfig(512, 1000, 1, 0), 2),
                      (pb.ProxFFNConfig(512, 1536, 9, 0), 1), (pb.ProxFFNConfig(512, 1536, 0, 0), 1),
                      (pb.ProxFFNConfig(512, 1536, 1, 7), 1), (pb.ProxFFNConfig(0, 1536, 1, 0), 1),
                      (pb.ProxFFNConfig(32768, 1536, 1, 0), 2)):
        assert create(C.byref(bad), 16, 16, 16, None, C.byref(out)) == want
        assert out.value is None
    # null handle everywhere
    assert pb.raw("prox_quantize_proxy")(None, 4, 0, None) == 1
    assert pb.raw("prox_stage1_mask")(None, 16, 1, 1, 1, 16, None, None) == 1
    assert pb.raw("prox_stage2_ffn")(None, 16, 1, 16, 1, 16, None) == 1
    assert pb.raw("prox_ffn_forward")(None, 16, 1, 1, 1, 16, None) == 1
    assert pb.raw("prox_ffn_forward_host")(None, 16, 1, 1, 1, 16, None) == 1
    assert pb.raw("prox_pack_save")(None, b"/tmp/x") == 1
    assert pb.raw("prox_allocate_budget")(0.5, 0.0, 0.7, 0.0, 0.7, C.byref(C.c_double()), C.byref(C.c_double())) == 1
    assert pb.raw("prox_allocate_budget")(0.5, 1 / 3, 0.7, 0.8, 0.7, C.byref(C.c_double()), C.byref(C.c_double())) == 1
    assert pb.raw("prox_sparsity_to_k")(0.5, 0, C.byref(C.c_int())) == 1
    pb.prox_ffn_destroy(None)                                          # no-op
    with pytest.raises(pb.ProxError):
        pb.prox_quantize_proxy(None, 4, 0)


def test_create_without_device_reports_cuda_error(pb):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    out = C.c_void_p()
    cfg = pb.ProxFFNConfig(512, 1536, 1, 0)
    assert pb.raw("prox_ffn_create")(C.byref(cfg), 16, 16, 16, None, C.byref(out)) in (4, 5)
    assert out.value is None


def test_product_has_no_oracle_import():
    """The product path must not reach into oracle/ (nor the oracle into the product)."""
    pkg = os.path.join(ROOT, "paper_2607_27591_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                assert "oracle" not in open(os.path.join(dirpath, f)).read(), f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2607_27591_b200" not in src and "ctypes" not in src
