"""sepllm_build_index_static: the index build for callers that cannot allocate device memory
(it keeps its scratch in a fixed array inside the library).  Collected last on purpose.

Its output must equal sepllm_build_index's byte for byte, also on a second call right after the
first with different inputs (all calls share the one array, which keeps the previous contents),
and the call must leave the amount of free device memory where it was.
"""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
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
    # and against the oracle's index, not only against the other entry point
    want = orc.build_index_fast(ids2, inputs.SEP_IDS, 0, 17, 128, 128, 9_001)
    for k in ("cnt", "lim", "side_pos", "n_side", "tile_meta"):
        assert np.array_equal(idx[k], want[k]), k


def test_static_scratch_call_leaves_free_device_memory_unchanged():
    ids = inputs.token_ids(23, 4, 20_000, 0.1, "iid")
    B, L = ids.shape
    desc = api.IndexDesc(B, L, 4, 64, len(inputs.SEP_IDS), 128, 128, L)
    ib, _ = api.sepllm_index_bytes(desc)
    ids_d = torch.from_numpy(np.ascontiguousarray(ids)).cuda()
    out = api.alloc_bytes(ib)
    api.sepllm_build_index_static(desc, ids_d, inputs.SEP_IDS, out)   # the kernel is loaded by now
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        api.sepllm_build_index_static(desc, ids_d, inputs.SEP_IDS, out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


def test_static_scratch_limit_is_exact():
    """21845 sequences of one 4096-id chunk need 21845 * 3 = 65535 of the 65536 words: accepted and
    equal to the regular build; one sequence more needs 65538: refused on the host, nothing
    launched (the pointers of the refused call are never used)."""
    ids = inputs.token_ids(24, 21845, 4096, 0.05, "iid")
    got, ref = _both(ids, 2, 32, 64)
    assert torch.equal(got, ref)
    desc = api.IndexDesc(21846, 4096, 2, 32, len(inputs.SEP_IDS), 128, 128, 64)
    dummy = api.alloc_bytes(256)
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_build_index_static(desc, dummy, inputs.SEP_IDS, dummy)
    assert e.value.code == api.BUFFER_TOO_SMALL
    # far beyond the limit: 32 sequences of 2^24 ids would need 32 * (2 * 4096 + 1) words
    desc = api.IndexDesc(32, 1 << 24, 4, 256, len(inputs.SEP_IDS), 128, 128, 1024)
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_build_index_static(desc, dummy, inputs.SEP_IDS, dummy)
    assert e.value.code == api.BUFFER_TOO_SMALL
