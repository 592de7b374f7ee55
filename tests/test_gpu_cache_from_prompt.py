"""sepllm_cache_from_prompt against the oracle's cache after a prompt, and against streaming."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import TOL_LSE, TOL_O, assert_close, build_index
from tests.test_gpu_cache import GpuCache

pytestmark = pytest.mark.gpu


def _prompt(seed, B, Hkv, L, d, rho):
    ids = inputs.token_ids(seed, B, L, rho)
    K = inputs.normal_bf16(seed, 31, (B, Hkv, L, d))
    V = inputs.normal_bf16(seed, 32, (B, Hkv, L, d))
    return ids, K, V


def _hand_off(gc, ids, K, V, a, lens=None, n=64):
    idesc, index = build_index(ids, inputs.SEP_IDS, a, n)
    lens_d = None if lens is None else torch.tensor(lens, dtype=torch.int32, device="cuda")
    api.sepllm_cache_from_prompt(gc.desc, idesc, index, lens_d, K.cuda(), V.cuda(), gc.state, gc.Kc, gc.Vc)
    torch.cuda.synchronize()


def _check_against_oracle(gc, oc, f, K, V, heads=None):
    """Sizes, retained positions in order, flags, counters and the cached rows, bit for bit."""
    d = gc.desc
    st = api.read_cache_state(gc.state)
    Kc = gc.Kc.view(d.B, d.Hkv, gc.slots, d.d).cpu()
    Vc = gc.Vc.view(d.B, d.Hkv, gc.slots, d.d).cpu()
    for b in range(d.B):
        init, sep, win = gc.regions(st, b)
        assert (init, sep, win) == (oc[b].init, oc[b].sep, oc[b].window), b
        assert st["next_pos"][b] == oc[b].next_pos and st["compactions"][b] == oc[b].compactions
        slots = gc.slot_of_virtual(st, b)
        flags = st["slot_is_sep"][b][slots].astype(bool).tolist()
        assert flags[len(init):] == [bool(f[b, p]) for p in sep + win]
        retained = oc[b].retained()
        for hk in (range(d.Hkv) if heads is None else heads):
            assert torch.equal(Kc[b, hk][slots], K[b, hk][retained])
            assert torch.equal(Vc[b, hk][slots], V[b, hk][retained])
    return st


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 2, 2), (128, 8, 2)])
def test_hand_off_every_prompt_length(d, Hq, Hkv):
    """Every prompt length from 0 to past several compactions, eight sequences per call."""
    a, s, w, c = 2, 5, 4, 20
    B, L = 8, 96
    ids, K, V = _prompt(70 + d, B, Hkv, L, d, 0.3)
    f = np.isin(ids, inputs.SEP_IDS)
    for first in range(0, L + 1, B):
        lens = [min(L, first + b) for b in range(B)]
        gc = GpuCache(B, Hkv, Hq, d, a, s, w, c)
        _hand_off(gc, ids, K, V, a, lens)
        assert api.sepllm_last_device_status(gc.state) == 0
        oc = [orc.cache_after_prompt(f[b, :lens[b]], a, s, w, c) for b in range(B)]
        _check_against_oracle(gc, oc, f, K, V)
    assert oc[-1].compactions >= 5


@pytest.mark.parametrize("a,s,w,c,rho", [(0, 3, 2, 9, 0.5), (3, 0, 5, 12, 0.5), (1, 4, 3, 30, 0.9),
                                          (4, 64, 256, 800, 0.12), (4, 16, 8, 30, 0.0)])
def test_hand_off_then_streaming_continues(a, s, w, c, rho):
    """No initial tokens, no separator cache, separator bursts, the paper-like sizes, no separators
    at all: hand-off at L, then 2(c - a) more tokens through sepllm_cache_update, compared with the
    oracle that streamed everything; decode after each stage."""
    B, Hkv, Hq, d = 2, 2, 4, 128
    L = 5 * c + 7
    more = 2 * (c - a)
    ids, K, V = _prompt(80 + c, B, Hkv, L + more, d, rho)
    f = np.isin(ids, inputs.SEP_IDS)
    gc = GpuCache(B, Hkv, Hq, d, a, s, w, c)
    _hand_off(gc, np.ascontiguousarray(ids[:, :L]), K[:, :, :L].contiguous(), V[:, :, :L].contiguous(), a)
    oc = [orc.cache_after_prompt(f[b, :L], a, s, w, c) for b in range(B)]
    _check_against_oracle(gc, oc, f, K, V)
    Kd, Vd = K.cuda(), V.cuda()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids.T)).cuda()
    q = inputs.normal_bf16(80 + c, 33, (B, Hq, d))
    G = Hq // Hkv
    for t in range(L, L + more):
        gc.update(ids_d[t], Kd[:, :, t].contiguous(), Vd[:, :, t].contiguous())
        for b in range(B):
            oc[b].update(bool(f[b, t]))
        if t % 97 and t != L + more - 1:
            continue
        o, lse = gc.decode(q.cuda())
        torch.cuda.synchronize()
        assert api.sepllm_last_device_status(gc.state) == 0
        st = api.read_cache_state(gc.state)
        for b in range(B):
            assert gc.regions(st, b) == (oc[b].init, oc[b].sep, oc[b].window), (t, b)
            kept = oc[b].retained()
            for h in range(Hq):
                oref, lref = orc.decode_attention(q[b, h].double().numpy(),
                                                  K[b, h // G][kept].double().numpy(),
                                                  V[b, h // G][kept].double().numpy())
                assert_close(o[b, h].float().cpu().numpy(), oref, TOL_O, f"decode t={t} b={b} h={h}")
                assert abs(float(lse[b, h]) - lref) <= TOL_LSE
    _check_against_oracle(gc, oc, f, K, V)
    assert all(x.compactions >= 6 for x in oc)


def test_hand_off_equals_streaming_on_the_device():
    """The same prompt through sepllm_cache_update token by token: decode reads the same entries in
    the same order, so the outputs agree exactly although the rings start elsewhere."""
    B, Hkv, Hq, d, a, s, w, c = 3, 2, 8, 128, 4, 16, 32, 100
    L = 777
    ids, K, V = _prompt(91, B, Hkv, L, d, 0.15)
    fast = GpuCache(B, Hkv, Hq, d, a, s, w, c)
    _hand_off(fast, ids, K, V, a)
    slow = GpuCache(B, Hkv, Hq, d, a, s, w, c)
    Kd, Vd = K.cuda(), V.cuda()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids.T)).cuda()
    for t in range(L):
        slow.update(ids_d[t], Kd[:, :, t].contiguous(), Vd[:, :, t].contiguous())
    q = inputs.normal_bf16(91, 33, (B, Hq, d)).cuda()
    o1, l1 = fast.decode(q)
    o2, l2 = slow.decode(q)
    torch.cuda.synchronize()
    sf, ss = api.read_cache_state(fast.state), api.read_cache_state(slow.state)
    for b in range(B):
        assert fast.regions(sf, b) == slow.regions(ss, b)
    assert (ss["win_start"] != 0).any() and (sf["win_start"] == 0).all()
    assert torch.equal(o1, o2) and torch.equal(l1, l2)


def test_hand_off_streaming_workload_shapes():
    """The streaming-decode workload's cache (32 sequences, 8 kv heads, c = 3332) from 8192-token
    prompts of mixed lengths."""
    c = inputs.DECODE_CONFIG
    B, Hkv, Hq, d, L = c["B"], c["Hkv"], c["Hq"], c["d"], 8192
    ids, K, V = _prompt(c["seed"], B, Hkv, L, d, c["rho"])
    f = np.isin(ids, inputs.SEP_IDS)
    lens = [L - 61 * b for b in range(B)]
    gc = GpuCache(B, Hkv, Hq, d, c["a"], c["s"], c["w"], c["c"])
    _hand_off(gc, ids, K, V, c["a"], lens, n=256)
    assert api.sepllm_last_device_status(gc.state) == 0
    oc = [orc.cache_after_prompt(f[b, :lens[b]], c["a"], c["s"], c["w"], c["c"]) for b in range(B)]
    _check_against_oracle(gc, oc, f, K, V, heads=(0, Hkv - 1))
    assert min(x.compactions for x in oc) >= 2


def test_hand_off_rejects_what_it_cannot_use():
    B, Hkv, Hq, d, a, s, w, c = 2, 1, 1, 64, 2, 3, 4, 16
    L = 50
    ids, K, V = _prompt(93, B, Hkv, L, d, 0.3)
    gc = GpuCache(B, Hkv, Hq, d, a, s, w, c)
    idesc, index = build_index(ids, inputs.SEP_IDS, a + 1, 8)            # other n_init
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_cache_from_prompt(gc.desc, idesc, index, None, K.cuda(), V.cuda(), gc.state, gc.Kc, gc.Vc)
    assert e.value.code == api.INVALID_ARG
    # a length beyond L: that sequence stays empty, the other is filled, the status says so
    _hand_off(gc, ids, K, V, a, [L + 1, 20])
    assert api.sepllm_last_device_status(gc.state) == api.INVALID_ARG
    st = api.read_cache_state(gc.state)
    assert st["next_pos"].tolist() == [0, 20] and st["size_win"][0] == 0 and st["size_init"][0] == 0
    # an index built for other ids of the same shape is accepted (the call cannot tell), but one
    # whose header says another length is not
    other = inputs.token_ids(94, B, L + 3, 0.3)
    idesc2, index2 = build_index(other, inputs.SEP_IDS, a, 8)
    idesc_l = api.IndexDesc(B, L, a, 8, len(inputs.SEP_IDS), 128, 128, L)
    api.sepllm_cache_from_prompt(gc.desc, idesc_l, index2, None, K.cuda(), V.cuda(), gc.state, gc.Kc, gc.Vc)
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(gc.state) == api.INVALID_ARG
    assert api.read_cache_state(gc.state)["next_pos"].tolist() == [0, 0]


def test_hand_off_fills_the_rotated_key_buffer():
    """Hand-off with Kr, then rotary updates: the rotary decode agrees exactly with a cache that took
    every token through sepllm_cache_update_rope (same rotated rows, same order)."""
    B, Hkv, Hq, d, a, s, w, c = 2, 2, 8, 128, 4, 16, 32, 100
    L, more = 500, 130
    ids, K, V = _prompt(95, B, Hkv, L + more, d, 0.15)
    Kd, Vd = K.cuda(), V.cuda()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids.T)).cuda()
    fast, slow = GpuCache(B, Hkv, Hq, d, a, s, w, c), GpuCache(B, Hkv, Hq, d, a, s, w, c)
    table = api.alloc_bytes(api.sepllm_rope_table_bytes(fast.desc))
    api.sepllm_rope_table_build(fast.desc, 10000.0, table)
    Kr_f, Kr_s = torch.zeros_like(fast.Kc), torch.zeros_like(slow.Kc)
    idesc, index = build_index(np.ascontiguousarray(ids[:, :L]), inputs.SEP_IDS, a, 64)
    api.sepllm_cache_from_prompt(fast.desc, idesc, index, None, Kd[:, :, :L].contiguous(),
                                 Vd[:, :, :L].contiguous(), fast.state, fast.Kc, fast.Vc, Kr_f, table)
    q = inputs.normal_bf16(95, 33, (B, Hq, d)).cuda()

    def decode(gc, Kr):
        o = torch.empty((B, Hq, d), dtype=torch.bfloat16, device="cuda")
        lse = torch.empty((B, Hq), dtype=torch.float32, device="cuda")
        api.sepllm_decode_rope(gc.desc, 0.0, q, gc.state, Kr, gc.Vc, table, o, lse, gc.ws)
        return o, lse

    for t in range(L + more):
        api.sepllm_cache_update_rope(slow.desc, slow.state, slow.Kc, slow.Vc, Kr_s, table, ids_d[t],
                                     inputs.SEP_IDS, Kd[:, :, t].contiguous(), Vd[:, :, t].contiguous())
        if t >= L:
            api.sepllm_cache_update_rope(fast.desc, fast.state, fast.Kc, fast.Vc, Kr_f, table, ids_d[t],
                                         inputs.SEP_IDS, Kd[:, :, t].contiguous(), Vd[:, :, t].contiguous())
        if t in (L - 1, L + 40, L + more - 1):
            (o1, l1), (o2, l2) = decode(fast, Kr_f), decode(slow, Kr_s)
            torch.cuda.synchronize()
            assert torch.equal(o1, o2) and torch.equal(l1, l2), t
    sf, ss = api.read_cache_state(fast.state), api.read_cache_state(slow.state)
    for b in range(B):
        assert fast.regions(sf, b) == slow.regions(ss, b)
        rows_f = Kr_f.view(B, Hkv, fast.slots, d)[b][:, fast.slot_of_virtual(sf, b)]
        rows_s = Kr_s.view(B, Hkv, slow.slots, d)[b][:, slow.slot_of_virtual(ss, b)]
        assert torch.equal(rows_f, rows_s)
    assert ss["compactions"].min() >= 5


def test_hand_off_with_a_side_list_cut_short():
    """side_cap below the number of side members: the index reports it, its prefix counts are still
    complete, and the hand-off finds the separators the list lacks from the counts."""
    B, Hkv, Hq, d, a, s, w, c = 2, 1, 2, 64, 2, 12, 4, 40
    L = 600
    ids, K, V = _prompt(97, B, Hkv, L, d, 0.3)
    f = np.isin(ids, inputs.SEP_IDS)
    gc = GpuCache(B, Hkv, Hq, d, a, s, w, c)
    idesc, index = build_index(ids, inputs.SEP_IDS, a, 16, side_cap=20)
    api.sepllm_cache_from_prompt(gc.desc, idesc, index, None, K.cuda(), V.cuda(), gc.state, gc.Kc, gc.Vc)
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(index) == api.CAPACITY_EXCEEDED
    assert api.sepllm_last_device_status(gc.state) == 0
    oc = [orc.cache_after_prompt(f[b], a, s, w, c) for b in range(B)]
    _check_against_oracle(gc, oc, f, K, V)
    assert all(len(x.sep) == s for x in oc)
