"""sepllm_cache_update / sepllm_decode against the oracle's cache state machine and decode."""
import numpy as np
import pytest
import torch

from oracle import sepllm_oracle as orc
from paper_2412_12094_b200 import api, inputs
from tests._gpu_util import TOL_LSE, TOL_O, assert_close

pytestmark = pytest.mark.gpu


class GpuCache:
    def __init__(self, B, Hkv, Hq, d, a, s, w, c, flags=0):
        self.desc = api.CacheDesc(B, Hkv, Hq, d, a, s, w, c, flags)
        sb, kb = api.sepllm_cache_bytes(self.desc)
        self.state = api.alloc_bytes(sb)
        self.Kc = torch.zeros(kb // 2, dtype=torch.bfloat16, device="cuda")
        self.Vc = torch.zeros(kb // 2, dtype=torch.bfloat16, device="cuda")
        self.ws = api.alloc_bytes(api.sepllm_decode_workspace_bytes(self.desc))
        api.sepllm_cache_init(self.desc, self.state)
        self.slots = c + s

    def update(self, ids, k, v):
        api.sepllm_cache_update(self.desc, self.state, self.Kc, self.Vc, ids, inputs.SEP_IDS, k, v)

    def decode(self, q):
        d = self.desc
        o = torch.empty((d.B, d.Hq, d.d), dtype=torch.bfloat16, device="cuda")
        lse = torch.empty((d.B, d.Hq), dtype=torch.float32, device="cuda")
        api.sepllm_decode(d, 0.0, q, self.state, self.Kc, self.Vc, o, lse, self.ws)
        return o, lse

    def regions(self, st, b):
        """Token positions per region in ascending order, read from the device state."""
        d = self.desc
        pos = st["slot_pos"][b]
        init = [int(pos[i]) for i in range(st["size_init"][b])]
        sep = [int(pos[d.a + (st["sep_start"][b] + i) % max(d.s, 1)]) for i in range(st["size_sep"][b])]
        ring = d.c - d.a
        win = [int(pos[d.a + d.s + (st["win_start"][b] + i) % ring]) for i in range(st["size_win"][b])]
        return init, sep, win

    def slot_of_virtual(self, st, b):
        d = self.desc
        ring = d.c - d.a
        return ([i for i in range(st["size_init"][b])]
                + [d.a + (st["sep_start"][b] + i) % max(d.s, 1) for i in range(st["size_sep"][b])]
                + [d.a + d.s + (st["win_start"][b] + i) % ring for i in range(st["size_win"][b])])


def _drive(B, Hkv, Hq, d, a, s, w, c, steps, rho, seed, check_every=1, pool=None):
    pool = steps if pool is None else pool
    ids = inputs.decode_stream_ids(seed, B, steps, rho)
    kp, vp, qp = inputs.decode_kv_pool(seed, pool, B, Hkv, Hq, d)
    kd, vd, qd = kp.cuda(), vp.cuda(), qp.cuda()
    ids_d = torch.from_numpy(np.ascontiguousarray(ids.T)).cuda()   # [steps][B]
    gc = GpuCache(B, Hkv, Hq, d, a, s, w, c)
    oc = [orc.StreamingCache(a, s, w, c) for _ in range(B)]
    f = np.isin(ids, inputs.SEP_IDS)
    G = Hq // Hkv
    checked = 0
    for t in range(steps):
        gc.update(ids_d[t], kd[t % pool], vd[t % pool])
        for b in range(B):
            oc[b].update(bool(f[b, t]))
        if (t + 1) % check_every and t != steps - 1:
            continue
        o, lse = gc.decode(qd[t % pool])
        torch.cuda.synchronize()
        assert api.sepllm_last_device_status(gc.state) == 0
        st = api.read_cache_state(gc.state)
        Kc = gc.Kc.view(B, Hkv, gc.slots, d).float().cpu().numpy()
        Vc = gc.Vc.view(B, Hkv, gc.slots, d).float().cpu().numpy()
        o = o.float().cpu().numpy()
        lse = lse.cpu().numpy()
        for b in range(B):
            init, sep, win = gc.regions(st, b)
            assert (init, sep, win) == (oc[b].init, oc[b].sep, oc[b].window), (t, b)
            assert st["next_pos"][b] == t + 1 and st["compactions"][b] == oc[b].compactions
            slots = gc.slot_of_virtual(st, b)
            retained = oc[b].retained()
            assert st["slot_is_sep"][b][slots].astype(bool).tolist() == [bool(f[b, p]) for p in retained]
            for hk in range(Hkv if checked % 4 == 0 else 1):
                # cached rows are the stream's rows at the retained positions, bit for bit
                kref = kp[[p % pool for p in retained], b, hk].float().numpy()
                vref = vp[[p % pool for p in retained], b, hk].float().numpy()
                assert np.array_equal(Kc[b, hk][slots], kref) and np.array_equal(Vc[b, hk][slots], vref)
                for g in range(G):
                    h = hk * G + g
                    oref, lref = orc.decode_attention(qp[t % pool, b, h].double().numpy(), kref, vref)
                    assert_close(o[b, h], oref, TOL_O, f"decode o t={t} b={b} h={h}")
                    assert abs(lse[b, h] - lref) <= TOL_LSE
        checked += 1
    return gc, oc


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 2, 2), (128, 8, 2), (128, 4, 1)])
def test_cache_small_every_step(d, Hq, Hkv):
    gc, oc = _drive(2, Hkv, Hq, d, a=2, s=5, w=4, c=20, steps=260, rho=0.3, seed=50 + d + Hq)
    assert min(c.compactions for c in oc) > 10


@pytest.mark.parametrize("d,Hq,Hkv", [(64, 16, 1), (128, 32, 2), (128, 9, 1), (64, 24, 2)])
def test_cache_wide_query_groups(d, Hq, Hkv):
    """9 to 16 query heads per kv head (Falcon-40B has 16 at d = 64): both halves of the decode
    kernel's 16-row tile are in use."""
    _drive(2, Hkv, Hq, d, a=2, s=6, w=5, c=40, steps=150, rho=0.3, seed=57 + d + Hq, check_every=7)


def test_cache_no_initial_tokens_and_no_separator_cache():
    _drive(1, 1, 1, 64, a=0, s=3, w=2, c=9, steps=80, rho=0.5, seed=61)
    _drive(1, 1, 2, 64, a=3, s=0, w=5, c=12, steps=80, rho=0.5, seed=62)     # StreamingLLM-like


def test_cache_separator_burst_overflows_the_separator_cache():
    # rho = 0.9: one compaction moves more separators than s holds
    _drive(2, 1, 1, 64, a=1, s=4, w=3, c=30, steps=200, rho=0.9, seed=63)


def test_cache_medium_periodic():
    gc, oc = _drive(3, 2, 8, 128, a=4, s=64, w=256, c=800, steps=3000, rho=0.12, seed=64,
                    check_every=331, pool=512)
    assert all(c.compactions >= 4 for c in oc)


def test_cache_full_size_streaming_workload():
    """The streaming-decode workload's shapes: 32 sequences, 8 kv heads, c = 3332."""
    c = inputs.DECODE_CONFIG
    gc, oc = _drive(c["B"], c["Hkv"], c["Hq"], c["d"], c["a"], c["s"], c["w"], c["c"], steps=6200,
                    rho=c["rho"], seed=c["seed"], check_every=3100, pool=256)
    assert all(x.compactions >= 2 for x in oc)


def test_cache_rejects_bad_capacities():
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_cache_bytes(api.CacheDesc(1, 1, 1, 64, 4, 10, 10, 24))      # a + s + w == c
    assert e.value.code == api.INVALID_ARG
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_cache_bytes(api.CacheDesc(1, 1, 1, 80, 4, 10, 10, 100))
    assert e.value.code == api.UNSUPPORTED
    with pytest.raises(api.SepllmError) as e:
        api.sepllm_cache_bytes(api.CacheDesc(1, 1, 17, 64, 4, 10, 10, 100))     # 17 query heads per kv head
    assert e.value.code == api.UNSUPPORTED
