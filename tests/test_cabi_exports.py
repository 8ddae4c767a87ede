"""The C-ABI library loads without a GPU and exports every symbol include/sttm.h declares."""
import os
import re

import torch

from paper_2507_07990_b200 import binding, build


def declared_symbols():
    header = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "sttm.h")
    text = open(header).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sttm_[a-z_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_the_header():
    build.build()
    lib = binding.load_library()
    names = declared_symbols()
    assert "sttm_merge" in names and "sttm_spatial" in names and "sttm_temporal" in names
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == names


def test_host_only_entry_points():
    prob = binding.make_params((1, 1024, 13, 13, 3584), torch.bfloat16, 0.9, 0.9)
    assert binding.sttm_workspace_bytes(prob) > 0
    assert binding.sttm_sims_per_frame(13, 13, 4) == 169 + 49
    assert binding.sttm_sims_per_frame(16, 16, 4) == 256 + 64
    assert binding.sttm_sims_per_frame(8, 8, 2) == 64 + 16
    assert binding.sttm_sims_per_frame(4, 4, 4) == 0
    bad = binding.make_params((1, 4, 13, 13, 6), torch.bfloat16, 0.9, 0.9)
    assert binding.sttm_workspace_bytes(bad) == 0
    lib = binding.load_library()
    assert lib.sttm_status_string(2) == b"unsupported shape"
