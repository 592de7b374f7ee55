"""Seeded random cache shapes: hand-off at ragged prompt lengths, further updates, then plain or
rotary decode, against the oracle's state machine and decode."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import TOL_LSE, TOL_O, assert_close, build_index
from tests.test_gpu_cache import GpuCache
from tests.test_gpu_decode_rope import TOL_LSE_ROPE, TOL_O_ROPE

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(16))
def test_random_cache_shape(seed):
    g = np.random.default_rng(8000 + seed)
    d = int(g.choice([64, 128]))
    Hkv = int(g.choice([1, 2, 3]))
    G = int(g.choice([1, 2, 3, 4, 7, 8, 11, 16]))
    Hq, B = Hkv * G, int(g.choice([1, 2, 3]))
    a, s, w = int(g.choice([0, 1, 4])), int(g.choice([0, 1, 3, 8, 40])), int(g.choice([1, 2, 5, 16]))
    c = a + s + w + int(g.choice([1, 2, 5, 30, 100]))
    rho = float(g.choice([0.0, 0.1, 0.3, 0.9]))
    L, more = int(g.integers(1, 6 * c + 20)), int(g.integers(1, 3 * c))
    rope = bool(g.integers(0, 2))
    T = L + more
    ids = inputs.token_ids(8000 + seed, B, T, rho)
    f = np.isin(ids, inputs.SEP_IDS)
    K = inputs.normal_bf16(8000 + seed, 31, (B, Hkv, T, d))
    V = inputs.normal_bf16(8000 + seed, 32, (B, Hkv, T, d))
    q = inputs.normal_bf16(8000 + seed, 33, (B, Hq, d))
    gc = GpuCache(B, Hkv, Hq, d, a, s, w, c)
    table = api.alloc_bytes(api.sepllm_rope_table_bytes(gc.desc))
    api.sepllm_rope_table_build(gc.desc, 10000.0, table)
    Kr = torch.zeros_like(gc.Kc)
    Kd, Vd = K.cuda(), V.cuda()
    lens = [L] + [int(g.integers(0, L + 1)) for _ in range(B - 1)]
    idesc, index = build_index(np.ascontiguousarray(ids[:, :L]), inputs.SEP_IDS, a, 7)
    api.sepllm_cache_from_prompt(gc.desc, idesc, index, torch.tensor(lens, dtype=torch.int32, device="cuda"),
                                 Kd[:, :, :L].contiguous(), Vd[:, :, :L].contiguous(), gc.state, gc.Kc, gc.Vc,
                                 Kr if rope else None, table if rope else None)
    oc = [orc.cache_after_prompt(f[b, :lens[b]], a, s, w, c) for b in range(B)]
    for t in range(more):      # sequence b goes on with tokens lens[b], lens[b] + 1, ... of its own row
        at = [lens[b] + t for b in range(B)]
        kn = torch.stack([Kd[b, :, at[b]] for b in range(B)]).contiguous()
        vn = torch.stack([Vd[b, :, at[b]] for b in range(B)]).contiguous()
        tok = torch.from_numpy(np.array([ids[b, at[b]] for b in range(B)], dtype=np.int32)).cuda()
        if rope:
            api.sepllm_cache_update_rope(gc.desc, gc.state, gc.Kc, gc.Vc, Kr, table, tok, inputs.SEP_IDS, kn, vn)
        else:
            api.sepllm_cache_update(gc.desc, gc.state, gc.Kc, gc.Vc, tok, inputs.SEP_IDS, kn, vn)
        for b in range(B):
            oc[b].update(bool(f[b, at[b]]))
    o = torch.empty((B, Hq, d), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
    if rope:
        api.sepllm_decode_rope(gc.desc, 0.0, q.cuda(), gc.state, Kr, gc.Vc, table, o, lse, gc.ws)
    else:
        api.sepllm_decode(gc.desc, 0.0, q.cuda(), gc.state, gc.Kc, gc.Vc, o, lse, gc.ws)
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(gc.state) == 0
    st = api.read_cache_state(gc.state)
    tol_o, tol_l = (TOL_O_ROPE, TOL_LSE_ROPE) if rope else (TOL_O, TOL_LSE)
    for b in range(B):
        assert gc.regions(st, b) == (oc[b].init, oc[b].sep, oc[b].window), (seed, b)
        assert st["compactions"][b] == oc[b].compactions
        kept = oc[b].retained()
        for h in range(Hq):
            kk, vv = K[b, h // G][kept].double().numpy(), V[b, h // G][kept].double().numpy()
            if rope:
                oref, lref = orc.decode_attention_rope(q[b, h].double().numpy(), kk, vv, 10000.0)
            else:
                oref, lref = orc.decode_attention(q[b, h].double().numpy(), kk, vv)
            assert_close(o[b, h].float().cpu().numpy(), oref, tol_o, f"seed {seed} b{b} h{h}")
            assert abs(float(lse[b, h]) - lref) <= tol_l
