"""The fixed-interval variant (appendix "Fixed-Interval Variant") through the same index and
attention kernels."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import TOL_GRAD, TOL_LSE, TOL_O, assert_close, attn_bwd, attn_fwd
from tests.test_gpu_cache import GpuCache

pytestmark = pytest.mark.gpu
KEYS = ("cnt", "lim", "side_pos", "n_side", "tile_meta")


def _index(B, L, a, n, interval, BM=128, BN=128, side_cap=None):
    desc = api.IndexDesc(B, L, a, n, 0, BM, BN, L if side_cap is None else side_cap)
    ib, sb = api.sepllm_index_bytes(desc)
    index, scratch = api.alloc_bytes(ib), api.alloc_bytes(sb)
    api.sepllm_build_index_fixed_interval(desc, interval, index, scratch)
    torch.cuda.synchronize()
    return desc, index


def _oracle_index(B, L, a, n, interval, BM, BN, cap):
    # the oracle's builder takes token ids: id 1 where the variant keeps a token, 0 elsewhere
    ids = np.tile(orc.fixed_interval_flags(L, interval).astype(np.int32), (B, 1))
    return orc.build_index_fast(ids, np.array([1], np.int32), a, n, BM, BN, cap)


@pytest.mark.parametrize("L,a,n,interval,BM,BN", [
    (1, 0, 1, 1, 128, 128), (127, 3, 64, 5, 128, 128), (4096, 3, 256, 4, 128, 128),
    (4097, 3, 256, 8, 128, 128), (10000, 4, 300, 16, 128, 128), (9000, 0, 17, 7, 64, 32),
    (70000, 3, 256, 5, 128, 128), (5000, 2, 9, 6000, 128, 128), (300000, 4, 4096, 3, 128, 128),
])
def test_fixed_interval_index_matches_oracle(L, a, n, interval, BM, BN):
    B = 2
    desc, index = _index(B, L, a, n, interval, BM, BN)
    got = api.read_index(index)
    ref = _oracle_index(B, L, a, n, interval, BM, BN, L)
    for k in KEYS:
        assert np.array_equal(got[k], ref[k]), k
    assert got["header"].status == 0
    members = sorted(set(range(min(a, L))) | set(range(0, L, interval)))
    assert got["side_pos"][0][:len(members)].tolist() == members


@pytest.mark.parametrize("d,Hq,Hkv,L,a,n,interval", [(128, 4, 2, 1500, 3, 256, 5), (64, 2, 2, 700, 3, 64, 4),
                                                       (128, 2, 1, 900, 0, 32, 16)])
def test_fixed_interval_forward_and_backward(d, Hq, Hkv, L, a, n, interval):
    B = 1
    Q, K, V, dO = inputs.qkv_do(300 + interval, B, Hq, Hkv, L, d)
    idesc, index = _index(B, L, a, n, interval)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    f = np.tile(orc.fixed_interval_flags(L, interval), (B, 1))
    Oref, LSEref = orc.attn_fwd(Q.double().numpy(), K.double().numpy(), V.double().numpy(), f, a, n)
    assert_close(O.float().cpu().numpy(), Oref, TOL_O, "O")
    assert np.abs(LSE.cpu().numpy() - LSEref).max() <= TOL_LSE
    dQ, dK, dV = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, grad_dtype=1)
    rQ, rK, rV = orc.attn_bwd(Q.double().numpy(), K.double().numpy(), V.double().numpy(),
                              dO.double().numpy(), f, a, n)
    for got, ref, what in ((dQ, rQ, "dQ"), (dK, rK, "dK"), (dV, rV, "dV")):
        assert_close(got.cpu().numpy(), ref, TOL_GRAD, what)


def test_fixed_interval_prompt_hand_off():
    """The hand-off reads only the index, so the variant's cache comes out of the same call."""
    B, Hkv, Hq, d, a, s, w, c, interval = 2, 2, 4, 128, 3, 40, 16, 100, 5
    L = 1000
    K = inputs.normal_bf16(41, 31, (B, Hkv, L, d))
    V = inputs.normal_bf16(41, 32, (B, Hkv, L, d))
    idesc, index = _index(B, L, a, 64, interval)
    gc = GpuCache(B, Hkv, Hq, d, a, s, w, c)
    lens = torch.tensor([L, 333], dtype=torch.int32, device="cuda")
    api.sepllm_cache_from_prompt(gc.desc, idesc, index, lens, K.cuda(), V.cuda(), gc.state, gc.Kc, gc.Vc)
    torch.cuda.synchronize()
    st = api.read_cache_state(gc.state)
    f = orc.fixed_interval_flags(L, interval)
    Kc = gc.Kc.view(B, Hkv, gc.slots, d).cpu()
    for b, T in enumerate([L, 333]):
        oc = orc.cache_after_prompt(f[:T], a, s, w, c)
        assert gc.regions(st, b) == (oc.init, oc.sep, oc.window)
        assert st["compactions"][b] == oc.compactions
        assert torch.equal(Kc[b, 1][gc.slot_of_virtual(st, b)], K[b, 1][oc.retained()])


def test_fixed_interval_rejects_bad_arguments():
    desc = api.IndexDesc(1, 256, 3, 16, 0, 128, 128, 256)
    ib, sb = api.sepllm_index_bytes(desc)
    index, scratch = api.alloc_bytes(ib), api.alloc_bytes(sb)
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_build_index_fixed_interval(desc, 0, index, scratch)
    assert e.value.code == api.INVALID_ARG
    desc2 = api.IndexDesc(1, 256, 3, 16, 2, 128, 128, 256)      # a separator list makes no sense here
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_build_index_fixed_interval(desc2, 4, index, scratch)
    assert e.value.code == api.INVALID_ARG
