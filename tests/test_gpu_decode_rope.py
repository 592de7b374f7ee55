"""sepllm_cache_update_rope / sepllm_decode_rope (positions inside the cache) against the oracle's
rotary decode."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import TOL_O, assert_close
from tests.test_gpu_cache import GpuCache

pytestmark = pytest.mark.gpu

# The library rounds the rotated K rows and the rotated q to bf16 before the tensor-core products
# (the oracle rotates in fp64), so every score carries two relative roundings of 2^-9 per term:
# about 2^-9 * sqrt(2) * |q||k| / d ~ 3e-3 rms for N(0,1) inputs.  LSE is a weighted mean of the
# scores' errors, hence the looser bound than for the plain decode.  Each weight P_j then carries
# that score error as a relative error of its own (about 2e-3 rms, independent from key to key),
# which adds to the rounding of P and of the output that the plain decode already has: about 3e-3
# relative on O as a whole, up to 5e-3 on single heads with few cache entries, so the relative
# Frobenius bound on O is twice the common one here; the max-abs bound is the common one.
TOL_LSE_ROPE = 1e-2
TOL_O_ROPE = dict(max_abs=TOL_O["max_abs"], rel_fro=2 * TOL_O["rel_fro"])


def _check_rotated_keys(gc, Kr, st, base):
    """Every retained row of Kr is the row of Kc turned to its position inside the cache: half a
    bf16 ulp from the rounding plus the fp32 angle (position * theta carries 2^-24 relative error,
    under 3e-4 rad at position 4000)."""
    d = gc.desc
    Kc = gc.Kc.view(d.B, d.Hkv, gc.slots, d.d).double().cpu().numpy()
    Kr = Kr.view(d.B, d.Hkv, gc.slots, d.d).double().cpu().numpy()
    for b in range(d.B):
        slots = gc.slot_of_virtual(st, b)
        for hk in range(d.Hkv):
            ref = orc.rope_rotate(Kc[b, hk][slots], np.arange(len(slots)), base)
            err = np.abs(Kr[b, hk][slots] - ref)
            assert (err <= 2.0 ** -8 * np.maximum(1.0, np.abs(ref)) + 1e-3).all(), (b, hk, err.max())


def _drive(B, Hkv, Hq, d, a, s, w, c, steps, rho, seed, base, check_at, keys_every=0):
    ids = inputs.decode_stream_ids(seed, B, steps, rho)
    kp, vp, qp = inputs.decode_kv_pool(seed, steps, B, Hkv, Hq, d)
    kd, vd, qd = kp.cuda(), vp.cuda(), qp.cuda()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids.T)).cuda()
    gc = GpuCache(B, Hkv, Hq, d, a, s, w, c)
    table = api.alloc_bytes(api.sepllm_rope_table_bytes(gc.desc))
    api.sepllm_rope_table_build(gc.desc, base, table)
    Kr = torch.full_like(gc.Kc, float("nan"))      # a row the update failed to write would show
    G = Hq // Hkv
    o = torch.empty((B, Hq, d), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
    for t in range(steps):
        api.sepllm_cache_update_rope(gc.desc, gc.state, gc.Kc, gc.Vc, Kr, table, ids_d[t], inputs.SEP_IDS,
                                     kd[t], vd[t])
        if keys_every and t % keys_every == 0:
            torch.cuda.synchronize()
            _check_rotated_keys(gc, Kr, api.read_cache_state(gc.state), base)
        if t not in check_at:
            continue
        api.sepllm_decode_rope(gc.desc, 0.0, qd[t], gc.state, Kr, gc.Vc, table, o, lse, gc.ws)
        torch.cuda.synchronize()
        st = api.read_cache_state(gc.state)
        _check_rotated_keys(gc, Kr, st, base)
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
                    assert_close(on[b, h], oref, TOL_O_ROPE, f"rope decode o t={t} b={b} h={h}")
                    assert abs(ln[b, h] - lref) <= TOL_LSE_ROPE


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 2, 2), (128, 8, 2), (128, 4, 1), (64, 16, 1), (128, 12, 1)])
def test_rope_decode_small(d, Hq, Hkv):
    _drive(2, Hkv, Hq, d, a=2, s=5, w=4, c=20, steps=90, rho=0.3, seed=70 + d + Hq, base=10000.0,
           check_at={0, 1, 5, 19, 20, 21, 47, 89}, keys_every=1)


def test_rope_decode_medium_llama_base():
    _drive(3, 2, 8, 128, a=4, s=64, w=256, c=800, steps=1700, rho=0.12, seed=77, base=500000.0,
           check_at={300, 799, 800, 1250, 1699})


def test_rope_no_separator_cache_and_no_initial_tokens():
    _drive(1, 1, 2, 64, a=3, s=0, w=5, c=12, steps=60, rho=0.5, seed=78, base=10000.0,
           check_at={0, 11, 12, 59}, keys_every=1)
    _drive(1, 1, 1, 64, a=0, s=3, w=2, c=9, steps=60, rho=0.5, seed=79, base=10000.0,
           check_at={0, 8, 9, 59}, keys_every=1)


def test_rope_state_machine_is_the_plain_one():
    """The rotary update changes Kr only: state, Kc and Vc end up as with sepllm_cache_update."""
    B, Hkv, Hq, d, a, s, w, c, steps = 2, 2, 4, 128, 2, 6, 4, 24, 150
    ids = inputs.decode_stream_ids(81, B, steps, 0.3)
    kp, vp, _ = inputs.decode_kv_pool(81, steps, B, Hkv, Hq, d)
    kd, vd = kp.cuda(), vp.cuda()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids.T)).cuda()
    plain, rot = GpuCache(B, Hkv, Hq, d, a, s, w, c), GpuCache(B, Hkv, Hq, d, a, s, w, c)
    table = api.alloc_bytes(api.sepllm_rope_table_bytes(rot.desc))
    api.sepllm_rope_table_build(rot.desc, 10000.0, table)
    Kr = torch.zeros_like(rot.Kc)
    for t in range(steps):
        plain.update(ids_d[t], kd[t], vd[t])
        api.sepllm_cache_update_rope(rot.desc, rot.state, rot.Kc, rot.Vc, Kr, table, ids_d[t],
                                     inputs.SEP_IDS, kd[t], vd[t])
    torch.cuda.synchronize()
    assert torch.equal(plain.state, rot.state) and torch.equal(plain.Kc, rot.Kc) and torch.equal(plain.Vc, rot.Vc)
