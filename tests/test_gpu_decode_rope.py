"""sepllm_decode_rope (positions inside the cache) against the oracle's rotary decode."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import TOL_O, assert_close
from tests.test_gpu_cache import GpuCache

pytestmark = pytest.mark.gpu

# The kernel rounds the rotated K rows and the rotated q to bf16 before the tensor-core products
# (the oracle rotates in fp64), so every score carries two relative roundings of 2^-9 per term:
# about 2^-9 * sqrt(2) * |q||k| / d ~ 3e-3 rms for N(0,1) inputs.  LSE is a weighted mean of the
# scores' errors, hence the looser bound than for the plain decode; O keeps the common tolerance.
TOL_LSE_ROPE = 1e-2


def _drive(B, Hkv, Hq, d, a, s, w, c, steps, rho, seed, base, check_at):
    ids = inputs.decode_stream_ids(seed, B, steps, rho)
    kp, vp, qp = inputs.decode_kv_pool(seed, steps, B, Hkv, Hq, d)
    kd, vd, qd = kp.cuda(), vp.cuda(), qp.cuda()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids.T)).cuda()
    gc = GpuCache(B, Hkv, Hq, d, a, s, w, c)
    table = api.alloc_bytes(api.sepllm_rope_table_bytes(gc.desc))
    api.sepllm_rope_table_build(gc.desc, base, table)
    G = Hq // Hkv
    o = torch.empty((B, Hq, d), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
    for t in range(steps):
        gc.update(ids_d[t], kd[t], vd[t])
        if t not in check_at:
            continue
        api.sepllm_decode_rope(gc.desc, 0.0, qd[t], gc.state, gc.Kc, gc.Vc, table, o, lse, gc.ws)
        torch.cuda.synchronize()
        st = api.read_cache_state(gc.state)
        Kc = gc.Kc.view(B, Hkv, gc.slots, d).float().cpu().numpy()
        Vc = gc.Vc.view(B, Hkv, gc.slots, d).float().cpu().numpy()
        on, ln = o.float().cpu().numpy(), lse.cpu().numpy()
        for b in range(B):
            slots = gc.slot_of_virtual(st, b)          # cache order: initial, separator, neighbour
            for hk in range(Hkv):
                for g in range(G):
                    h = hk * G + g
                    oref, lref = orc.decode_attention_rope(qp[t, b, h].double().numpy(), Kc[b, hk][slots],
                                                           Vc[b, hk][slots], base)
                    assert_close(on[b, h], oref, TOL_O, f"rope decode o t={t} b={b} h={h}")
                    assert abs(ln[b, h] - lref) <= TOL_LSE_ROPE


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 2, 2), (128, 8, 2), (128, 4, 1)])
def test_rope_decode_small(d, Hq, Hkv):
    _drive(2, Hkv, Hq, d, a=2, s=5, w=4, c=20, steps=90, rho=0.3, seed=70 + d + Hq, base=10000.0,
           check_at={0, 1, 5, 19, 20, 21, 47, 89})


def test_rope_decode_medium_llama_base():
    _drive(3, 2, 8, 128, a=4, s=64, w=256, c=800, steps=1700, rho=0.12, seed=77, base=500000.0,
           check_at={300, 799, 800, 1250, 1699})
