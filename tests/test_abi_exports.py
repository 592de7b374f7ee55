"""The shared library builds, loads without a GPU and exports what the header declares."""
import os
import re

from paper_2412_12094_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "sepllm.h")).read()
    return sorted(set(re.findall(r"\b(sepllm_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    build.build()
    lib = api.lib()
    names = _declared()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(api.EXPORTS) == names


def test_host_side_size_queries_need_no_gpu():
    d = api.IndexDesc(2, 1000, 4, 64, 9, 128, 128, 1000)
    ib, sb = api.sepllm_index_bytes(d)
    assert ib % 256 == 0 and sb % 256 == 0 and ib > 4 * 2 * (1001 + 1000 + 1000)
    a = api.AttnDesc(2, 4, 2, 128, 1000, 0.0, 0)
    fb, bb = api.sepllm_attn_workspace_bytes(a, d)
    assert fb >= 2 * 2 * 2 * 1024 * 128 * 2 and bb > fb
    sbytes, kv = api.sepllm_cache_bytes(api.CacheDesc(32, 8, 32, 128, 4, 1024, 256, 3332))
    assert kv == 32 * 8 * (3332 + 1024) * 128 * 2
    assert api.status_string(6) == "device wait timed out"
