"""Ragged batches through the same kernels: sequences shorter than L are padded at the end.

The mask is causal, so a valid row never sees a padded key, and with dO = 0 on the padded rows the
padded queries add nothing to dK / dV: the valid part of every output equals the result for the
truncated sequence.  (Separator ids in the padding only lengthen the side list behind the rows
that matter.)"""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import inputs
from tests._gpu_util import TOL_GRAD, TOL_LSE, TOL_O, assert_close, attn_bwd, attn_fwd, build_index, flags_of

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 4, 2), (64, 2, 2)])
def test_padded_sequences_match_the_truncated_ones(d, Hq, Hkv):
    B, L, a, n = 3, 900, 3, 100
    lens = [900, 517, 128]
    ids = inputs.token_ids(400 + d, B, L, 0.2)
    Q, K, V, dO = inputs.qkv_do(400 + d, B, Hq, Hkv, L, d)
    for b, T in enumerate(lens):
        dO[b, :, T:] = 0
    idesc, index = build_index(ids, inputs.SEP_IDS, a, n)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    dQ, dK, dV = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, grad_dtype=1)
    f = flags_of(ids, inputs.SEP_IDS)
    for b, T in enumerate(lens):
        sl = lambda t: t[b:b + 1, :, :T].double().numpy()
        Oref, LSEref = orc.attn_fwd(sl(Q), sl(K), sl(V), f[b:b + 1, :T], a, n)
        assert_close(O[b:b + 1, :, :T].float().cpu().numpy(), Oref, TOL_O, f"O b={b}")
        assert np.abs(LSE[b:b + 1, :, :T].cpu().numpy() - LSEref).max() <= TOL_LSE
        rQ, rK, rV = orc.attn_bwd(sl(Q), sl(K), sl(V), sl(dO), f[b:b + 1, :T], a, n)
        assert_close(dQ[b:b + 1, :, :T].cpu().numpy(), rQ, TOL_GRAD, f"dQ b={b}")
        assert_close(dK[b:b + 1, :, :T].cpu().numpy(), rK, TOL_GRAD, f"dK b={b}")
        assert_close(dV[b:b + 1, :, :T].cpu().numpy(), rV, TOL_GRAD, f"dV b={b}")
        # padded keys get no gradient at all: only padded queries reach them, and their dO is 0
        assert float(dK[b, :, T:].abs().max() if T < L else 0.0) == 0.0
        assert float(dV[b, :, T:].abs().max() if T < L else 0.0) == 0.0
