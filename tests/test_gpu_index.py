"""sepllm_build_index against the oracle's index, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import build_index

pytestmark = pytest.mark.gpu
KEYS = ("cnt", "lim", "side_pos", "n_side", "tile_meta")


def _compare(ids, sep_ids, a, n, BM=128, BN=128, side_cap=None, slow=False):
    desc, index = build_index(ids, sep_ids, a, n, side_cap, BM, BN)
    torch.cuda.synchronize()
    got = api.read_index(index)
    cap = desc.side_cap
    ref = (orc.build_index if slow else orc.build_index_fast)(ids, sep_ids, a, n, BM, BN, cap)
    for k in KEYS:
        assert got[k].dtype == ref[k].dtype and got[k].shape == ref[k].shape, k
        assert np.array_equal(got[k], ref[k]), k
    h = got["header"]
    assert h.magic == 0x58444953 and h.n_tiles == (ids.shape[1] + BM - 1) // BM
    return got


@pytest.mark.parametrize("name", ["tiny", "pythia160m", "llama8b_prefill", "llama8b_long_r05", "llama8b_long_r10",
                                  "llama8b_long_r20"])
def test_index_matches_oracle_on_workloads(name):
    c = inputs.CONFIGS[name]
    ids = inputs.token_ids(c["seed"], c["B"], c["L"], c["rho"], c["structure"])
    got = _compare(ids, inputs.SEP_IDS, c["n_init"], c["n_neighbor"], slow=(name == "tiny"))
    assert got["header"].status == 0


@pytest.mark.parametrize("L,a,n,BM,BN", [
    (1, 0, 1, 128, 128), (1, 4, 64, 128, 128), (127, 4, 64, 128, 128), (129, 0, 1, 128, 128),
    (4095, 3, 5000, 128, 128), (4096, 3, 4096, 128, 128), (4097, 300, 17, 64, 32), (10000, 4, 256, 128, 128),
])
def test_index_edge_shapes(L, a, n, BM, BN):
    ids = inputs.token_ids(7 + L, 3, L, 0.2, "iid")
    _compare(ids, inputs.SEP_IDS, a, n, BM, BN, slow=(L <= 4097))


def test_index_no_separators_and_all_separators():
    L = 3000
    ids = inputs.token_ids(5, 2, L, 0.0)
    _compare(ids, inputs.SEP_IDS, 0, 64)               # empty side list
    _compare(ids, np.zeros(0, np.int32), 4, 64)        # n_sep = 0
    ids[:] = inputs.SEP_IDS[3]
    _compare(ids, inputs.SEP_IDS, 4, 64)               # every token is a side member


def test_index_capacity_exceeded_is_reported_and_clamped():
    L = 2048
    ids = inputs.token_ids(9, 2, L, 0.5)
    desc, index = build_index(ids, inputs.SEP_IDS, 4, 64, side_cap=100)
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(index) == api.CAPACITY_EXCEEDED
    got = api.read_index(index)
    ref = orc.build_index_fast(ids, inputs.SEP_IDS, 4, 64, 128, 128, 100)
    assert np.array_equal(got["side_pos"], ref["side_pos"]) and np.array_equal(got["n_side"], ref["n_side"])
    assert (got["n_side"] > 100).all()


def test_index_decode_stream_full_size():
    """32 sequences of 2^20 token ids (the streaming workload's ids), bit-exact."""
    c = inputs.DECODE_CONFIG
    ids = inputs.decode_stream_ids(c["seed"], c["B"], c["stream_len"], c["rho"])
    _compare(ids, inputs.SEP_IDS, 4, 256, side_cap=1 << 18)


def test_index_bad_arguments_are_rejected_on_the_host():
    d = api.IndexDesc(1, 128, 4, 0, 9, 128, 128, 128)     # n_neighbor = 0
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_index_bytes(d)
    assert e.value.code == api.INVALID_ARG
    d = api.IndexDesc(1, 128, 4, 8, 65, 128, 128, 128)    # too many separator ids
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_index_bytes(d)
    assert e.value.code == api.UNSUPPORTED
