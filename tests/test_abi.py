"""The C-ABI library builds, loads and exports every entry point the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "isd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(isd_[a-z_]+)\s*\(", text)))


def test_header_declares_the_step_entry_points():
    names = declared_functions()
    for must in ("isd_attn", "isd_verify", "isd_commit", "isd_step", "isd_create", "isd_destroy"):
        assert must in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2604_11035_b200 import build
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    for name in declared_functions():
        assert hasattr(lib, name), name
    lib.isd_strerror.restype = ctypes.c_char_p
    assert lib.isd_strerror(0) == b"ok"
    assert b"head_dim" in lib.isd_strerror(-2)


def test_binding_mirrors_the_header():
    import paper_2604_11035_b200 as pkg
    assert sorted(pkg.EXPORTS) == declared_functions()
    for n in ("isd_attn", "isd_verify", "isd_commit", "isd_step", "isd_release", "isd_read_status"):
        assert hasattr(pkg.Isd, n)


def test_struct_layouts_match_the_header_field_order():
    import paper_2604_11035_b200 as pkg
    text = open(os.path.join(ROOT, "include", "isd.h")).read()

    def fields(struct):
        body = re.search(r"typedef struct %s \{(.*?)\} %s;" % (struct, struct), text, flags=re.S).group(1)
        body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
        return [re.findall(r"([A-Za-z_0-9]+)\s*;", line)[0] for line in body.split("\n") if ";" in line]

    assert fields("isd_config") == [n for n, _ in pkg.IsdConfig._fields_]
    assert fields("isd_batch_state") == [n for n, _ in pkg.IsdBatchState._fields_]
    assert fields("isd_verify_out") == [n for n, _ in pkg.IsdVerifyOut._fields_]
    assert fields("isd_step_args") == [n for n, _ in pkg.IsdStepArgs._fields_]


def test_no_cpu_fallback_without_a_gpu():
    import torch
    import paper_2604_11035_b200 as pkg
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(pkg.IsdError):
        pkg.Isd(batch=1, stride=2, n_q_heads=8, n_kv_heads=2, vocab=64, max_pages_per_slot=4, num_pages=8,
                logits_dtype="f32")


def test_product_package_does_not_import_the_oracle():
    pkg_dir = os.path.join(ROOT, "paper_2604_11035_b200")
    for dirpath, _, files in os.walk(pkg_dir):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "isd_oracle" not in src, f
    bench = open(os.path.join(ROOT, "bench.py")).read() if os.path.exists(os.path.join(ROOT, "bench.py")) else ""
    assert "_work/" not in bench
