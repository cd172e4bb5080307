"""The C-ABI library builds, loads and exports every symbol include/dc.h declares (no compute)."""
import ctypes
import os
import re

import paper_2609_35115_b200 as dc
from paper_2609_35115_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dc_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    lib = ctypes.CDLL(path)
    syms = declared_symbols()
    assert "dc_create" in syms and "dc_decode_chunk" in syms and "dc_stream_open" in syms and "dc_stream_close" in syms
    for s in syms:
        assert hasattr(lib, s), f"{s} declared in dc.h but not exported"
    assert sorted(binding.EXPORTS) == syms


def test_config_struct_matches_header_and_weight_counts():
    import dc_workloads as wl
    lib = dc.load_library()
    for name, cfg in wl.CONFIGS.items():
        c = dc.make_config(cfg, max_batch=max(cfg.n_streams, 1))
        assert lib.dc_weights_count(ctypes.byref(c)) == wl.blob_size(cfg), name
    bad = dc.make_config(wl.CONFIGS["cfg1"])
    bad.size = 7
    assert lib.dc_weights_count(ctypes.byref(bad)) == 0
    assert lib.dc_status_str(3) == b"DC_ERR_FRAMES"
