"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "nsd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nsd_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_three_steps():
    names = _declared()
    for required in ("nsd_kv_prepare", "nsd_verify_attn", "nsd_spec_accept", "nsd_verify_plan", "nsd_verify_round",
                     "nsd_verify_round_host", "nsd_create", "nsd_destroy", "nsd_get_status"):
        assert required in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    from paper_2609_29364_b200 import build as nsd_build

    path = nsd_build.build()
    lib = ctypes.CDLL(path)
    for name in _declared():
        assert hasattr(lib, name), f"{name} declared in nsd.h but not exported"


def test_pure_host_entry_points_answer_without_a_gpu():
    import paper_2609_29364_b200 as nsd

    lib = nsd.load_library()
    assert lib.nsd_status_string(0) == b"ok"
    cfg = nsd.NsdConfig(num_layers=2, num_slabs=2, num_q_heads=8, num_kv_heads=2, head_dim=64, block_size=16,
                        num_blocks=10, region_b_begin=2, max_batch=4, max_gamma=4, vocab_size=100, reserved=0,
                        max_table_entries=64)
    assert lib.nsd_kv_pool_bytes(ctypes.byref(cfg)) == 2 * 10 * 2 * 2 * 16 * 64 * 2
    assert lib.nsd_workspace_bytes(ctypes.byref(cfg)) > 0
    cfg.head_dim = 96                                   # no kernel for this shape
    assert lib.nsd_workspace_bytes(ctypes.byref(cfg)) == 0
    out = ctypes.c_void_p()
    assert lib.nsd_create(ctypes.byref(cfg), 256, 1 << 20, ctypes.byref(out)) == 4   # NSD_ERR_UNSUPPORTED, nothing touched
    assert lib.nsd_launch_count(None) == 0


def test_binding_refuses_to_run_without_the_library(monkeypatch):
    import paper_2609_29364_b200.api as api

    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "_LIB_PATH", os.path.join(ROOT, "no_such_dir", "libnsd.so"))
    with pytest.raises(ImportError):
        api.load_library()


def test_binding_flag_constants_match_the_header():
    """`nsd_config.flags` bits are spelled twice, in the header and in the binding: they must agree, name by name."""
    import paper_2609_29364_b200.api as api

    text = open(os.path.join(ROOT, "include", "nsd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    header = {name: 1 << int(shift) for name, shift in re.findall(r"\b(NSD_FLAG_[A-Z0-9_]+)\s*=\s*1\s*<<\s*(\d+)", text)}
    assert len(header) >= 8
    binding = {name: getattr(api, name) for name in dir(api) if name.startswith("NSD_FLAG_")}
    assert binding == header
