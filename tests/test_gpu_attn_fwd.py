"""sepllm_attn_fwd against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import TOL_LSE, TOL_O, assert_close, attn_fwd, build_index, flags_of

pytestmark = pytest.mark.gpu


def _run(B, Hq, Hkv, L, d, a, n, rho, seed, sep_ids=inputs.SEP_IDS, structure="iid", ids=None):
    if ids is None:
        ids = inputs.token_ids(seed, B, L, rho, structure)
    Q, K, V, _ = inputs.qkv_do(seed, B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, sep_ids, a, n)
    O, LSE = attn_fwd(Q.cuda(), K.cuda(), V.cuda(), idesc, index)
    Oref, LSEref = orc.attn_fwd(Q.double().numpy(), K.double().numpy(), V.double().numpy(),
                                flags_of(ids, sep_ids), a, n)
    # n = 1 or 2: rows that keep one or two keys copy V rows, whose entries reach 4 and more, where
    # a bf16 output is 0.016 off by rounding alone; only there is the bound taken relative
    assert_close(O.float().cpu().numpy(), Oref, TOL_O, "O", scaled=(n <= 2))
    assert np.abs(LSE.cpu().numpy() - LSEref).max() <= TOL_LSE
    return O, LSE


def test_fwd_tiny_config():
    c = inputs.CONFIGS["tiny"]
    _run(c["B"], c["Hq"], c["Hkv"], c["L"], c["d"], c["n_init"], c["n_neighbor"], c["rho"], c["seed"])


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 2, 2), (128, 4, 1), (128, 2, 2), (64, 4, 2)])
@pytest.mark.parametrize("L,a,n", [(512, 4, 64), (300, 4, 64), (777, 3, 200), (128, 0, 1), (129, 2, 128), (1000, 4, 1000)])
def test_fwd_shapes(d, Hq, Hkv, L, a, n):
    _run(2, Hq, Hkv, L, d, a, n, 0.15, 100 + L + d)


def test_fwd_dense_causal_and_sliding_window_and_all_separators():
    L = 640
    _run(1, 2, 1, L, 128, 0, L, 0.1, 31)                      # n >= L: dense causal
    _run(1, 2, 1, L, 64, 0, 100, 0.0, 32)                     # no separators, a = 0: sliding window
    ids = np.full((1, L), inputs.SEP_IDS[0], dtype=np.int32)
    _run(1, 2, 2, L, 64, 0, 1, 0.0, 33, ids=ids)              # every token a separator: dense causal
    _run(1, 1, 1, L, 128, 4, 64, 0.0, 34)                     # StreamingLLM mask


def test_fwd_many_side_tiles():
    """More than a few side tiles per query tile and a window that is not tile-aligned."""
    _run(1, 4, 2, 3000, 128, 4, 300, 0.3, 41)
    _run(1, 2, 2, 2500, 64, 4, 77, 0.4, 42)


def test_fwd_pythia_shape_sampled_heads():
    c = inputs.CONFIGS["pythia160m"]
    B, Hq, Hkv, L, d = c["B"], c["Hq"], c["Hkv"], c["L"], c["d"]
    ids = inputs.token_ids(c["seed"], B, L, c["rho"], c["structure"])
    Q, K, V, _ = inputs.qkv_do(c["seed"], B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, inputs.SEP_IDS, c["n_init"], c["n_neighbor"])
    O, LSE = attn_fwd(Q.cuda(), K.cuda(), V.cuda(), idesc, index)
    O = O.float().cpu().numpy()
    LSE = LSE.cpu().numpy()
    f = flags_of(ids, inputs.SEP_IDS)
    for b, h in [(0, 0), (3, 7), (7, 11)]:
        M = orc.mask_matrix(f[b], c["n_init"], c["n_neighbor"])
        o, lse, _ = orc.attn_fwd_rows(Q[b, h].double().numpy(), K[b, h].double().numpy(),
                                      V[b, h].double().numpy(), M)
        assert_close(O[b, h], o, TOL_O, f"O[{b},{h}]")
        assert np.abs(LSE[b, h] - lse).max() <= TOL_LSE


def test_fwd_rejects_unsupported():
    idesc = api.IndexDesc(1, 256, 4, 64, 9, 128, 128, 256)
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_attn_workspace_bytes(api.AttnDesc(1, 2, 2, 72, 256, 0.0, 0), idesc)
    assert e.value.code == api.UNSUPPORTED
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_attn_workspace_bytes(api.AttnDesc(1, 3, 2, 64, 256, 0.0, 0), idesc)
    assert e.value.code == api.INVALID_ARG


def test_fwd_scores_that_outgrow_the_first_tiles_reference():
    """Unmasked tiles after the first keep the row's old reference exponent; here the later keys
    score 2^100 above the first tile's, which must be caught and the tile redone with its own
    maximum (and a jump of 2^40, which must go through without that)."""
    B, Hq, Hkv, L, d = 1, 2, 1, 640, 64
    ids = inputs.token_ids(5, B, L, 0.0)
    _, _, V, _ = inputs.qkv_do(321, B, Hq, Hkv, L, d)
    for c in (3.0, 1.875):                      # sqrt(d) c^2 log2(e) = 104 and 40.6
        Q = torch.full((B, Hq, L, d), c, dtype=torch.bfloat16)
        K = torch.full((B, Hkv, L, d), c, dtype=torch.bfloat16)
        K[:, :, :128] = 0                        # the first key tile scores 0
        K[:, :, 300:] *= -1                      # and the last keys fall far below again
        idesc, index = build_index(ids, inputs.SEP_IDS, 0, L)     # dense causal
        O, LSE = attn_fwd(Q.cuda(), K.cuda(), V.cuda(), idesc, index)
        Oref, LSEref = orc.attn_fwd(Q.double().numpy(), K.double().numpy(), V.double().numpy(),
                                    flags_of(ids, inputs.SEP_IDS), 0, L)
        assert_close(O.float().cpu().numpy(), Oref, TOL_O, f"O c={c}")
        # LSE reaches 72 here: the fp32 product score * (scale * log2 e) carries 2^-24 of that per
        # rounding, so the bound scales with the magnitude beyond the workloads' |LSE| < 8
        assert np.abs(LSE.cpu().numpy() - LSEref).max() <= TOL_LSE * max(1.0, np.abs(LSEref).max() / 8)
