"""The C-ABI library loads without a GPU and exports every function include/sps.h declares."""
import ctypes
import os
import re

import paper_2302_01318_b200 as sps

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sps.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sps_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert {"sps_create", "sps_destroy", "sps_generate", "sps_generate_batch", "sps_verify", "sps_accept", "sps_reset",
            "sps_prefill", "sps_step", "sps_last_error"} <= set(names)
    lib = ctypes.CDLL(sps.lib_path()) if os.path.exists(sps.lib_path()) else sps.lib()
    for n in names:
        assert hasattr(lib, n), n


def test_struct_sizes_match_header():
    # int32 x7 + float x2 + int32 ; two of them + 4 int32 + pointer + uint32 (padded)
    assert ctypes.sizeof(sps.sps_model_cfg) == 40
    assert ctypes.sizeof(sps.sps_cfg) == 40 * 2 + 16 + 8 + 8
    assert ctypes.sizeof(sps.sps_weights) == (11 + 7) * 8      # 11 weight members + 7 row-scale members (int8 weights)
    assert ctypes.sizeof(sps.sps_stats) == 4 * (8 + 17 + 5 + 1)


def test_argument_errors_need_no_gpu():
    L = sps.lib()
    assert L.sps_create(None, None, None, None) == sps.SPS_EINVAL
    assert b"null" in L.sps_last_error(None)
    assert L.sps_accept(None, None, None, 1, 1, 8, 1.0, 0, 0, None, None, None, None) == sps.SPS_EINVAL
    assert L.sps_linear_workspace_bytes(1, 0, 10, 128) == -1
