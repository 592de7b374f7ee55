"""Generation in the fundamental design (Section 3.2 "Generation"; all separator KV kept, Section
4.2): the cache calls with SEPLLM_CACHE_FIXED_WINDOW against the oracle's FundamentalCache, and the
equivalence the design rests on: decoding token t over the retained set is row t of the
pre-filling attention."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import TOL_LSE, TOL_O, assert_close, attn_fwd, build_index, flags_of
from tests.test_gpu_cache import GpuCache

pytestmark = pytest.mark.gpu
FIXED = api.CACHE_FIXED_WINDOW


def _check_state(gc, oc, f, kp, vp, pool, t=None):
    d = gc.desc
    st = api.read_cache_state(gc.state)
    Kc = gc.Kc.view(d.B, d.Hkv, gc.slots, d.d).float().cpu().numpy()
    Vc = gc.Vc.view(d.B, d.Hkv, gc.slots, d.d).float().cpu().numpy()
    for b in range(d.B):
        assert gc.regions(st, b) == (oc[b].init, oc[b].sep, oc[b].window), (t, b)
        assert st["next_pos"][b] == oc[b].next_pos and st["compactions"][b] == oc[b].compactions
        slots = gc.slot_of_virtual(st, b)
        kept = oc[b].retained()
        assert st["slot_is_sep"][b][slots][len(oc[b].init):].astype(bool).tolist() == \
            [bool(f[b, p]) for p in kept[len(oc[b].init):]]
        for hk in range(d.Hkv):
            assert np.array_equal(Kc[b, hk][slots], kp[[p % pool for p in kept], b, hk].float().numpy())
            assert np.array_equal(Vc[b, hk][slots], vp[[p % pool for p in kept], b, hk].float().numpy())
    return st


@pytest.mark.parametrize("d,Hq,Hkv,a,n", [(64, 2, 2, 2, 5), (128, 8, 2, 4, 16), (128, 4, 1, 0, 1)])
def test_fixed_window_streaming_matches_oracle(d, Hq, Hkv, a, n):
    """Token by token: blocks, order, flags, cached rows bit for bit; decode against the oracle's
    attention over the retained set."""
    B, steps, rho = 2, 150, 0.3
    s_cap = 80
    ids = inputs.decode_stream_ids(300 + d + n, B, steps, rho)
    f = np.isin(ids, inputs.SEP_IDS)
    kp, vp, qp = inputs.decode_kv_pool(300 + d + n, steps, B, Hkv, Hq, d)
    kd, vd, qd = kp.cuda(), vp.cuda(), qp.cuda()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids.T)).cuda()
    gc = GpuCache(B, Hkv, Hq, d, a, s_cap, n, a + s_cap + n + 3, FIXED)
    oc = [orc.FundamentalCache(a, n) for _ in range(B)]
    G = Hq // Hkv
    for t in range(steps):
        gc.update(ids_d[t], kd[t], vd[t])
        for b in range(B):
            oc[b].update(bool(f[b, t]))
        if t % 7 and t != steps - 1:
            continue
        o, lse = gc.decode(qd[t])
        torch.cuda.synchronize()
        assert api.sepllm_last_device_status(gc.state) == 0
        _check_state(gc, oc, f, kp, vp, steps, t)
        o, lse = o.float().cpu().numpy(), lse.cpu().numpy()
        for b in range(B):
            kept = oc[b].retained()
            for h in range(Hq):
                oref, lref = orc.decode_attention(qp[t, b, h].double().numpy(), kp[kept, b, h // G].double().numpy(),
                                                  vp[kept, b, h // G].double().numpy())
                assert_close(o[b, h], oref, TOL_O, f"decode t={t} b={b} h={h}")
                assert abs(lse[b, h] - lref) <= TOL_LSE
    assert all(len(c.sep) > 10 for c in oc)


def test_fixed_window_separator_capacity_is_reported():
    B, Hkv, Hq, d, a, n, s_cap, steps = 1, 1, 1, 64, 1, 3, 4, 60
    ids = inputs.decode_stream_ids(310, B, steps, 0.5)
    kp, vp, _ = inputs.decode_kv_pool(310, steps, B, Hkv, Hq, d)
    ids_d = torch.from_numpy(np.ascontiguousarray(ids.T)).cuda()
    gc = GpuCache(B, Hkv, Hq, d, a, s_cap, n, a + s_cap + n + 2, FIXED)
    for t in range(steps):
        gc.update(ids_d[t], kp[t].cuda(), vp[t].cuda())
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(gc.state) == api.CAPACITY_EXCEEDED
    st = api.read_cache_state(gc.state)
    oc = orc.FundamentalCache(a, n)
    for t in range(steps):
        oc.update(bool(np.isin(ids[0, t], inputs.SEP_IDS)))
    init, sep, win = gc.regions(st, 0)
    assert sep == oc.sep[-s_cap:] and win == oc.window and len(oc.sep) > s_cap   # the newest s are kept


@pytest.mark.parametrize("d,Hq,Hkv", [(128, 8, 2), (64, 4, 4)])
def test_decode_over_the_retained_set_is_the_prefill_row(d, Hq, Hkv):
    """After the hand-off of a prompt of t + 1 tokens the fixed-window cache holds what row t of
    Eq. 2's mask keeps, so sepllm_decode(q_t) must return row t of sepllm_attn_fwd on the same
    Q, K, V: both against the oracle's row (the parity bar) and against each other."""
    B, L, a, n = 2, 700, 4, 64
    seed = 320 + d
    ids = inputs.token_ids(seed, B, L, 0.15)
    f = flags_of(ids, inputs.SEP_IDS)
    Q, K, V, _ = inputs.qkv_do(seed, B, Hq, Hkv, L, d)
    idesc, index = build_index(ids, inputs.SEP_IDS, a, n)
    Qd, Kd, Vd = Q.cuda(), K.cuda(), V.cuda()
    O, LSE = attn_fwd(Qd, Kd, Vd, idesc, index)
    O, LSE = O.float().cpu().numpy(), LSE.cpu().numpy()
    G = Hq // Hkv
    s_cap = int(f.sum(axis=1).max()) + 1
    first_sep = int(np.flatnonzero(f[0])[np.flatnonzero(f[0]) > n][0])
    ts = sorted({0, 2, a - 1, a, n - 1, n, n + 1, first_sep, first_sep + 1, first_sep + n, first_sep + n + 1,
                 L // 2, L - 1})
    gc = GpuCache(B, Hkv, Hq, d, a, s_cap, n, a + s_cap + n + 1, FIXED)
    for t in ts:
        lens = torch.full((B,), t + 1, dtype=torch.int32, device="cuda")
        api.sepllm_cache_from_prompt(gc.desc, idesc, index, lens, Kd, Vd, gc.state, gc.Kc, gc.Vc)
        o, lse = gc.decode(Qd[:, :, t].contiguous())
        torch.cuda.synchronize()
        assert api.sepllm_last_device_status(gc.state) == 0
        st = api.read_cache_state(gc.state)
        o, lse = o.float().cpu().numpy(), lse.cpu().numpy()
        for b in range(B):
            init, sep, win = gc.regions(st, b)
            M = orc.mask_rows(f[b], a, n, np.array([t]))[0]
            assert sorted(init + sep + win) == np.flatnonzero(M).tolist(), (t, b)
            for h in range(Hq):
                oref, lref, _ = orc.attn_fwd_rows(Q[b, h, t:t + 1].double().numpy(), K[b, h // G].double().numpy(),
                                                  V[b, h // G].double().numpy(), M[None, :])
                assert_close(o[b, h], oref[0], TOL_O, f"decode t={t} b={b} h={h}")
                assert abs(lse[b, h] - lref[0]) <= TOL_LSE
                # the two GPU paths against each other: each is within the bar of the oracle
                assert np.abs(o[b, h] - O[b, h, t]).max() <= 2 * TOL_O["max_abs"]
                assert abs(lse[b, h] - LSE[b, h, t]) <= 2 * TOL_LSE


def test_fixed_window_hand_off_equals_streaming_state():
    """Every prompt length: the hand-off leaves the blocks the token-by-token updates reach."""
    B, Hkv, Hq, d, a, n, L = 4, 2, 4, 64, 3, 6, 60
    ids = inputs.token_ids(330, B, L, 0.3)
    f = np.isin(ids, inputs.SEP_IDS)
    K = inputs.normal_bf16(330, 31, (B, Hkv, L, d))
    V = inputs.normal_bf16(330, 32, (B, Hkv, L, d))
    idesc, index = build_index(ids, inputs.SEP_IDS, a, n)
    s_cap = L
    for first in range(0, L + 1, B):
        lens = [min(L, first + b) for b in range(B)]
        gc = GpuCache(B, Hkv, Hq, d, a, s_cap, n, a + s_cap + n + 1, FIXED)
        api.sepllm_cache_from_prompt(gc.desc, idesc, index, torch.tensor(lens, dtype=torch.int32, device="cuda"),
                                     K.cuda(), V.cuda(), gc.state, gc.Kc, gc.Vc)
        torch.cuda.synchronize()
        assert api.sepllm_last_device_status(gc.state) == 0
        st = api.read_cache_state(gc.state)
        for b in range(B):
            oc = orc.FundamentalCache(a, n)
            for t in range(lens[b]):
                oc.update(bool(f[b, t]))
            assert gc.regions(st, b) == (oc.init, oc.sep, oc.window), (lens[b], b)
            assert st["compactions"][b] == oc.compactions and st["next_pos"][b] == lens[b]
            slots = gc.slot_of_virtual(st, b)
            kept = oc.retained()
            Kc = gc.Kc.view(B, Hkv, gc.slots, d).cpu()
            assert torch.equal(Kc[b, 1][slots], K[b, 1][kept])
