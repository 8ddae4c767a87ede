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
    import ctypes as C
    lib.sttm_budget_workspace_bytes.restype = C.c_size_t
    three = binding.make_params((1, 8, 16, 16, 64), torch.bfloat16, 0.9, 0.9)
    deep = binding.make_params((1, 8, 24, 24, 64), torch.bfloat16, 0.9, 0.9)        # 24 -> 12 -> 6 -> 3: four levels
    too_deep = binding.make_params((1, 1, 600, 4, 64), torch.bfloat16, 0.9, 0.9)    # nine levels
    assert binding.sttm_workspace_bytes(deep) > 8 * (576 // 3) * 64 * 4             # holds the pooled fp32 maps
    assert lib.sttm_budget_workspace_bytes(C.byref(three.params)) > 0
    assert lib.sttm_budget_workspace_bytes(C.byref(deep.params)) == 0               # budget mode: three levels
    assert binding.sttm_workspace_bytes(too_deep) == 0


def test_merged_positions_argument_checks_need_no_gpu():
    import ctypes as C
    lib = binding.load_library()
    assert lib.sttm_merged_positions_workspace(0) == 0
    need = lib.sttm_merged_positions_workspace(1000)
    assert need >= 1000 * 12 and need % 4 == 0
    # null pointers, bad sizes, a workspace that is too small: refused on the host, nothing launched
    assert lib.sttm_merged_positions(None, None, 1, 10, None, 0, None, 10, None, None) == 1       # STTM_ERR_ARG
    buf = (C.c_char * 4096)()
    addr = (C.addressof(buf) + 255) // 256 * 256
    assert lib.sttm_merged_positions(addr, addr, 0, 10, addr, 2048, addr, 10, None, None) == 1
    assert lib.sttm_merged_positions(addr, addr, 1, 10, addr + 4, 2048, addr, 10, None, None) == 1   # misaligned ws
    assert lib.sttm_merged_positions(addr, addr, 1, 10, addr, 16, addr, 10, None, None) == 3        # STTM_ERR_WORKSPACE


def test_device_status_word_decoding_needs_no_gpu():
    """Host handling of the status word kernels OR their conditions into: every condition has a
    bit of its own (the wait that ran out does not share one with a CUDA error), the lowest set
    bit names the status, and every status has a message."""
    lib = binding.load_library()
    lib.sttm_status_string.restype = __import__("ctypes").c_char_p
    names = {"capacity": 4, "not_converged": 5, "cuda": 6, "timeout": 7}
    assert lib.sttm_status_from_bits(0) == 0
    for code in names.values():
        assert lib.sttm_status_from_bits(1 << code) == code
    assert lib.sttm_status_from_bits((1 << names["timeout"]) | (1 << names["capacity"])) == names["capacity"]
    assert lib.sttm_status_from_bits(1 << names["timeout"]) != lib.sttm_status_from_bits(1 << names["cuda"])
    assert lib.sttm_status_string(names["timeout"]) == b"a wait inside a kernel ran out"
    assert binding.STATUS_NAMES[names["timeout"]] == "a wait inside a kernel ran out"
    assert len(binding.STATUS_NAMES) == 8
