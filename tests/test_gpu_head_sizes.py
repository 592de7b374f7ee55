"""Head sizes between the kernel widths (80, 96, 112): the kernels run 128 wide over rows of d
elements, so these cases check the row stride of every load and store, that the zero columns
change nothing, and that nothing is written outside a row (the tensors are dense, a store past a
row's end would land in the next row and break its parity)."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import (TOL_GRAD, TOL_LSE, TOL_O, assert_close, assert_grad_close, attn_bwd, attn_fwd,
                             build_index, errors, flags_of)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("grad_dtype", [0, 1])
@pytest.mark.parametrize("Hq,Hkv", [(4, 1), (2, 2), (3, 1)])
@pytest.mark.parametrize("d", [80, 96, 112])
def test_forward_and_backward_at_head_size(d, Hq, Hkv, grad_dtype):
    B, L, a, n, rho, seed = 2, 700, 3, 96, 0.15, 900 + d + Hq
    ids = inputs.token_ids(seed, B, L, rho, "iid")
    Q, K, V, dO = inputs.qkv_do(seed, B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, inputs.SEP_IDS, a, n)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    f = flags_of(ids, inputs.SEP_IDS)
    Qn, Kn, Vn, dOn = (t.double().numpy() for t in (Q, K, V, dO))
    Oref, LSEref = orc.attn_fwd(Qn, Kn, Vn, f, a, n)
    assert_close(O.float().cpu().numpy(), Oref, TOL_O, f"O d={d}")
    assert np.abs(LSE.cpu().numpy() - LSEref).max() <= TOL_LSE
    dQ, dK, dV = attn_bwd(dOd, Qd, Kd, Vd, O, LSE, idesc, index, grad_dtype)
    refs = orc.attn_bwd(Qn, Kn, Vn, dOn, f, a, n)
    scales = orc.attn_bwd_term_scale(Qn, Kn, Vn, dOn, f, a, n)
    for got, ref, rss, what in zip((dQ, dK, dV), refs, scales, ("dQ", "dK", "dV")):
        got = got.float().cpu().numpy()
        assert_grad_close(got, ref, rss, f"{what} d={d}", bf16_out=(grad_dtype == 0))
        assert errors(got, ref)[1] <= TOL_GRAD["rel_fro"], (what, errors(got, ref))


def test_outputs_inside_a_larger_buffer_leave_their_surroundings_alone():
    """O, dQ, dK and dV of d = 80 placed in the middle of sentinel-filled buffers: the bytes before
    and after each tensor are unchanged."""
    B, Hq, Hkv, L, d, a, n = 1, 4, 1, 300, 80, 2, 64
    ids = inputs.token_ids(77, B, L, 0.2, "iid")
    Q, K, V, dO = inputs.qkv_do(77, B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, inputs.SEP_IDS, a, n)
    Qd, Kd, Vd, dOd = Q.cuda(), K.cuda(), V.cuda(), dO.cuda()
    desc = api.AttnDesc(B, Hq, Hkv, d, L, 0.0, 0)
    fb, bb = api.sepllm_attn_workspace_bytes(desc, idesc)
    ws = api.alloc_bytes(bb)
    pad = 4096
    nq, nkv = B * Hq * L * d, B * Hkv * L * d
    bufs = {k: torch.full((pad + m + pad,), -7.0, dtype=torch.bfloat16, device="cuda")
            for k, m in (("O", nq), ("dQ", nq), ("dK", nkv), ("dV", nkv))}
    view = lambda k, shape: bufs[k][pad:pad + int(np.prod(shape))].view(shape)
    O, dQ = view("O", Q.shape), view("dQ", Q.shape)
    dK, dV = view("dK", K.shape), view("dV", K.shape)
    LSE = torch.empty((B, Hq, L), dtype=torch.float32, device="cuda")
    api.sepllm_attn_fwd(desc, idesc, Qd, Kd, Vd, index, O, LSE, ws)
    api.sepllm_attn_bwd(desc, idesc, dOd, Qd, Kd, Vd, O, LSE, index, dQ, dK, dV, ws)
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(ws) == 0
    for k, m in (("O", nq), ("dQ", nq), ("dK", nkv), ("dV", nkv)):
        assert bool((bufs[k][:pad] == -7.0).all()) and bool((bufs[k][pad + m:] == -7.0).all()), k
    f = flags_of(ids, inputs.SEP_IDS)
    Oref, _ = orc.attn_fwd(Q.double().numpy(), K.double().numpy(), V.double().numpy(), f, a, n)
    assert_close(O.float().cpu().numpy(), Oref, TOL_O, "O")


def test_head_sizes_outside_the_supported_set_are_refused():
    idesc = api.IndexDesc(1, 256, 4, 64, 9, 128, 128, 256)
    for d in (32, 72, 136, 256):
        with pytest.raises(api.SepllmError) as e:
            api.sepllm_attn_workspace_bytes(api.AttnDesc(1, 2, 2, d, 256, 0.0, 0), idesc)
        assert e.value.code == api.UNSUPPORTED
