"""CPU-side checks of the boundary: the built library loads and exports every symbol the
header declares (no compute calls: there is no GPU here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "dip.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dip_[a-z0-9_]+)\s*\(", text)))


def _lib_path():
    import importlib.util
    spec = importlib.util.spec_from_file_location("dip_build", os.path.join(ROOT, "paper_2412_01380_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod.build()


def test_header_declares_the_five_hot_path_calls():
    syms = _declared_symbols()
    for name in ("dip_mask_topk", "dip_ca_mask", "dip_sparse_gemv_gate_up", "dip_sparse_gemv_down", "dip_mlp_step"):
        assert name in syms


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(_lib_path())
    for name in _declared_symbols():
        assert hasattr(lib, name), name


def test_binding_names_match_header():
    _lib_path()
    import paper_2412_01380_b200 as dip
    assert sorted(dip.EXPORTED) == _declared_symbols()
    for name in ("dip_mask_topk", "dip_ca_mask", "dip_sparse_gemv_gate_up", "dip_sparse_gemv_down",
                 "dip_mlp_step", "dip_pack_weights", "dip_stack_step", "dip_residual_rmsnorm"):
        assert callable(getattr(dip, name))


def test_pure_host_calls():
    lib = ctypes.CDLL(_lib_path())
    lib.dip_status_string.restype = ctypes.c_char_p
    assert lib.dip_status_string(0) == b"ok"
    assert lib.dip_status_string(1) == b"invalid argument"
    lib.dip_packed_bytes.restype = ctypes.c_size_t
    # bf16 Phi-3-Medium block: gate/up bundle and down
    assert lib.dip_packed_bytes(1, 5120, 17920, 0) == 5120 * 2 * 17920 * 2
    assert lib.dip_packed_bytes(1, 5120, 17920, 1) == 5120 * 17920 * 2
    assert lib.dip_packed_bytes(1, 5120, 17920, 2) == 0
    # int4: half a byte per weight, one binary16 scale per 128 inputs and output
    assert lib.dip_packed_bytes(2, 4096, 14336, 0) == 4096 * 14336
    assert lib.dip_packed_bytes(2, 4096, 14336, 2) == (4096 // 128) * 2 * 14336 * 2
    assert lib.dip_packed_bytes(2, 4096, 14336, 3) == (14336 // 128) * 4096 * 2
    assert lib.dip_packed_bytes(1, 5121, 17920, 0) == 0       # bad shape
    assert lib.dip_packed_bytes(7, 5120, 17920, 0) == 0       # bad type


def test_product_path_does_not_reach_the_oracle():
    """The CUDA package and its sources never import, link or name the CPU oracle."""
    pkg = os.path.join(ROOT, "paper_2412_01380_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.replace("no CPU oracle", ""), f
