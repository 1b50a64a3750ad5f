"""CPU-side checks of the C boundary: the library builds, loads, exports every symbol that
include/spa.h declares, and rejects bad arguments on the host before touching a GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2410_23608_b200 import build, binding
    build.build()
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "spa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spa_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert "spa_gate" in names and "spa_packed_attention_bwd" in names and len(names) >= 14
    cdll = ctypes.CDLL(lib.LIB_PATH)
    for n in names:
        assert hasattr(cdll, n), n
    assert set(lib.EXPORTS) == set(names)


def test_status_strings(lib):
    L = lib.lib()
    assert L.spa_status_string(0) == b"ok"
    for code in (-1, -2, -3, -4, -5):
        assert L.spa_status_string(code) not in (b"ok", b"unknown status")
    assert L.spa_status_string(-99) == b"unknown status"


def test_host_side_validation_needs_no_gpu(lib):
    L = lib.lib()
    p = lib.make_params(2, 16, 64, 2, "f32")
    assert L.spa_gate(ctypes.byref(p), None, None, 0.0, None, None, None, None) == lib.SPA_ERR_INVALID_ARG
    assert L.spa_gate(None, None, None, 0.0, None, None, None, None) == lib.SPA_ERR_INVALID_ARG
    bad = lib.make_params(2, 16, 60, 2, "bf16")     # 120-byte rows: not a multiple of 16
    assert L.spa_gate(ctypes.byref(bad), None, None, 0.0, None, None, None, None) == lib.SPA_ERR_UNSUPPORTED
    big = lib.make_params(4096, 4096, 64, 2, "bf16")
    assert L.spa_workspace_bytes(ctypes.byref(big)) == 0     # B*N beyond the supported 2^20
    assert L.spa_launch_count() >= 0


def test_params_struct_layout_matches_header(lib):
    assert ctypes.sizeof(lib.SpaParams) == 36


def test_binding_constants_match_header(lib):
    text = open(os.path.join(ROOT, "include", "spa.h")).read()
    m = re.search(r"#define\s+SPA_STATIC_SCRATCH_BYTES\s+\((\d+)u\s*<<\s*(\d+)\)", text)
    assert m and lib.SPA_STATIC_SCRATCH_BYTES == int(m.group(1)) << int(m.group(2))
    for name, val in re.findall(r"\b(SPA_(?:ERR_[A-Z_]+|OK|FLAG_[A-Z_]+|F32|BF16))\s*=\s*(-?\d+)", text):
        assert getattr(lib, name) == int(val), name


def test_later_entry_points_validate_on_the_host(lib):
    """Fused, trainable-selection, ordered-packing and block calls: bad arguments come back as a status before
    anything touches a device."""
    L = lib.lib()
    p = lib.make_params(2, 16, 64, 2, "bf16")
    pp = ctypes.byref(p)
    inv, uns = lib.SPA_ERR_INVALID_ARG, lib.SPA_ERR_UNSUPPORTED
    assert L.spa_gate_prefill(pp, None, None, 0.0, None, None, None, None, None) == inv
    assert L.spa_unpack_prefill(pp, None, None, None) == inv
    assert L.spa_packed_proj_scatter(pp, None, None, None, None, None, None, None, None) == inv
    assert L.spa_packed_linear_bwd_scatter(pp, None, None, None, 64, 192, None, None, None, None, None, None, None, None) == inv
    assert L.spa_select_pack_ordered(pp, None, None, None, None, None, None, None, None, None, None) == inv
    assert L.spa_score_pool(None, 1, 2, 2, None, None) == inv
    assert L.spa_select_loss(pp, None, None, 1.0, None, None, None, None) == inv
    assert L.spa_select_pack_bwd_gated(pp, None, None, None, None, None, None, None, None, None) == inv
    assert L.spa_gate_bwd(pp, None, None, None, None, None, None, None, None, None, None, None) == inv
    assert L.spa_packed_linear(pp, None, None, None, 64, 256, None, None, 0, None, None) == inv
    assert L.spa_layer_norm(pp, None, None, None, 1e-5, None, None, None, None) == inv
    assert L.spa_layer_norm_bwd(pp, None, None, None, None, None, None, None, None, None, None, None) == inv
    assert L.spa_gelu(pp, None, 256, None, None) == inv
    assert L.spa_gelu_bwd(pp, None, None, 256, None, None) == inv
    assert L.spa_gate_select_pack(pp, None, None, 0.0, None, None, None, None, None, None, None, None, None, None, None) == inv
    assert L.spa_probe_mma_issue(0, 0, None, None, None) == inv and L.spa_probe_mma_issue(7, 0, None, None, None) == inv
    assert L.spa_pack_state_bytes(pp) >= 16 + 4 and L.spa_pack_state_bytes(None) == 0
    assert L.spa_gate_select_pack_supported(pp) == 1
    wide = lib.make_params(2, 16, 2048, 32, "bf16")                 # 256 chunks per row: two-kernel path only
    assert L.spa_gate_select_pack_supported(ctypes.byref(wide)) == 0
    empty = lib.SpaBlockBuffers()
    assert L.spa_block_fwd(pp, None, None) == inv and L.spa_block_bwd(pp, None, None) == inv
    assert L.spa_block_fwd(pp, ctypes.byref(empty), None) == inv      # no inputs: refused by the first call
    assert L.spa_block_bwd(pp, ctypes.byref(empty), None) == inv
    assert L.spa_block_fwd(None, ctypes.byref(empty), None) == inv
    assert L.spa_overlap_create(None) == inv and L.spa_overlap_destroy(None) == 0
    f32 = lib.make_params(2, 16, 64, 2, "f32")
    assert L.spa_fused_scatter_supported(ctypes.byref(f32)) == 0          # tensor-core problems only
    assert L.spa_packed_proj_scatter(ctypes.byref(f32), None, None, None, None, None, None, None, None) in (inv, uns)
    assert L.spa_train_workspace_bytes(pp) > 0 and L.spa_train_workspace_bytes(None) == 0
