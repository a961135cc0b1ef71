"""The C-ABI library builds, loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2607_19539_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "moe_ovl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moe_ovl_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported_and_bound():
    lib = B.load()
    names = declared_symbols()
    assert "moe_ovl_create" in names and "moe_ovl_expert_return" in names and "moe_ovl_destroy" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == names


def test_struct_sizes_match_header_layout():
    # field-by-field mirror of the header; sizes are what the library checks in struct_size
    assert ctypes.sizeof(B.Config) == 16 * 4
    assert ctypes.sizeof(B.Args) == 8 + 7 * 8 + 8 + 8 + 8 + 8 + 3 * 8 + 8
    assert ctypes.sizeof(B.Report) == 11 * 4 + 11 * 4
    assert ctypes.sizeof(B.TraceRecord) == 6 * 4 + 9 * 8 == B.TRACE_DTYPE.itemsize


def _cfg(**kw):
    base = dict(device=0, num_src_ranks=4, self_rank=0, tokens_per_rank=256, num_local_experts=2, top_k=2,
                d_model=256, d_ffn=512, max_rows=600)
    base.update(kw)
    return B.make_config(**base)


def test_workspace_and_limits_are_host_arithmetic():
    cfg = _cfg()
    bands, items = B.moe_ovl_limits(cfg)
    assert bands == -(-600 // 128) + 2 * 4            # ceil(M/128) + one partial band per (expert, rank) group
    assert items == bands * (512 // 128 + 256 // 256)
    n = B.moe_ovl_workspace_bytes(cfg)
    P = bands * 128
    assert n >= P * (256 + 512 + 256) * 2
    assert B.moe_ovl_workspace_bytes(_cfg(flags=B.FLAG_HOST_STAGING)) > n


@pytest.mark.parametrize("kw,code", [
    (dict(d_model=300), B.ERR_UNSUPPORTED), (dict(d_ffn=100), B.ERR_UNSUPPORTED),
    (dict(self_rank=4), B.ERR_INVALID_ARG), (dict(num_local_experts=0), B.ERR_INVALID_ARG),
    (dict(num_local_experts=300), B.ERR_UNSUPPORTED), (dict(max_rows=-1), B.ERR_INVALID_ARG),
    (dict(single_gemm_out=100), B.ERR_UNSUPPORTED), (dict(single_gemm_out=512, d_model=100), B.ERR_UNSUPPORTED),
])
def test_config_errors(kw, code):
    with pytest.raises(B.MoeOvlError) as e:
        B.moe_ovl_workspace_bytes(_cfg(**kw))
    assert e.value.code == code


def test_strerror_and_null_handling():
    lib = B.load()
    assert B.strerror(0) == "ok" and "timed out" in B.strerror(B.ERR_TIMEOUT)
    assert lib.moe_ovl_destroy(None) == 0
    assert lib.moe_ovl_expert_return(None, None) == B.ERR_INVALID_ARG
    ctx = ctypes.c_void_p(None)
    cfg = _cfg()
    assert lib.moe_ovl_create(ctypes.byref(ctx), ctypes.byref(cfg), None, 0) == B.ERR_WORKSPACE
