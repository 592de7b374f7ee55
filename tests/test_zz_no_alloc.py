"""sepllm_build_index_static: the index build for callers that cannot allocate device memory
(it keeps its scratch in a fixed array inside the library).  Collected last on purpose.

Its output must equal sepllm_build_index's byte for byte, also on a second call right after the
first with different inputs (all calls share the one array, which keeps the previous contents).
"""
import numpy as np
import pytest
import torch

from paper_2412_12094_b200 import api, inputs

pytestmark = pytest.mark.gpu


def _both(ids, a, n, side_cap):
    B, L = ids.shape
    desc = api.IndexDesc(B, L, a, n, len(inputs.SEP_IDS), 128, 128, side_cap)
    ib, sb = api.sepllm_index_bytes(desc)
    ids_d = torch.from_numpy(np.ascontiguousarray(ids)).cuda()
    ref = api.alloc_bytes(ib)
    ref.zero_()
    api.sepllm_build_index(desc, ids_d, inputs.SEP_IDS, ref, api.alloc_bytes(sb))
    got = api.alloc_bytes(ib)
    got.zero_()
    api.sepllm_build_index_static(desc, ids_d, inputs.SEP_IDS, got)
    torch.cuda.synchronize()
    return got, ref


def test_static_scratch_index_equals_regular_index_twice_in_a_row():
    # first call: many chunks with many separators, so the shared array is left full of records
    ids1 = inputs.token_ids(21, 6, 50_000, 0.4, "iid")
    got, ref = _both(ids1, 4, 300, 50_000)
    assert torch.equal(got, ref)
    assert api.read_index(got)["header"].status == 0
    # second call straight after, other shape and far fewer separators
    ids2 = inputs.token_ids(22, 3, 9_001, 0.02, "geometric")
    got, ref = _both(ids2, 0, 17, 9_001)
    assert torch.equal(got, ref)
    idx = api.read_index(got)
    assert int(idx["n_side"].sum()) == int(np.isin(ids2, inputs.SEP_IDS).sum())


def test_static_scratch_rejects_sizes_beyond_its_limit():
    # 32 sequences of 2^24 ids need 32 * (2 * 4096 + 1) words > 65536: refused on the host,
    # nothing launched
    desc = api.IndexDesc(32, 1 << 24, 4, 256, len(inputs.SEP_IDS), 128, 128, 1024)
    dummy = api.alloc_bytes(256)
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_build_index_static(desc, dummy, inputs.SEP_IDS, dummy)
    assert e.value.code == api.BUFFER_TOO_SMALL
