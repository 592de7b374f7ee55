#!/usr/bin/env python
"""Benchmark of the SepLLM attention hot path on B200.

One step = the whole training-side hot path on one batch of synthetic input:
sepllm_build_index -> sepllm_attn_fwd -> sepllm_attn_bwd.  The headline value is
effective TFLOP/s on kept (query, key) pairs, 14*d flops per pair and query head
(4*d forward, 10*d backward).  The streaming path (cache update + decode), the
index builder on a long id stream and the prompt hand-off into the cache are
measured in the same run and reported under "decode", "decode_rope", "index" and
"hand_off" with their own HBM rooflines.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
    python bench.py --impl reference ...      # the CPU oracle on a bounded sample

With N > 1 (torchrun) every rank runs its own copy of the workload (independent
sequences; the path has no exchange step) and rank 0 reports the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2412_12094_b200 import inputs  # noqa: E402

METRIC = "SepAttn fwd+bwd effective TFLOP/s (kept pairs)"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


# ---------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(device_index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "25"],
                stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        rows = [r.strip().split(", ") for r in open(self.tmp.name) if r.strip()]
        os.unlink(self.tmp.name)
        sm, reasons = [], set()
        for r in rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0]))
                out["sm_max_mhz"] = float(r[1])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8]):
                if v.strip().lower() == "active":
                    reasons.add(name)
        if sm:
            out["sm_mhz"] = statistics.median(sm)
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ---------------------------------------------------------------------------- CPU oracle arm
def oracle_sample(cfg, heads: int, prefix: int, keep: dict | None = None):
    """Times the fp64 oracle (forward + backward) on the first `prefix` tokens of `heads`
    query heads of the workload; returns (effective TFLOP/s, seconds, cores, description).
    keep: if given, receives the oracle's dQ of head 0 on those tokens (rows of dQ depend on
    their own row only, and the mask is causal, so they are also rows of the full problem)."""
    from threadpoolctl import threadpool_info
    from oracle import sepllm_oracle as orc
    L = min(prefix, cfg["L"])
    ids = inputs.token_ids(cfg["seed"], 1, cfg["L"], cfg["rho"], cfg["structure"])[:, :L]
    f = np.isin(ids[0], inputs.SEP_IDS)
    d = cfg["d"]
    G = cfg["Hq"] // cfg["Hkv"]
    Q = inputs.normal_bf16(cfg["seed"], 1, (heads, L, d)).double().numpy()
    K = inputs.normal_bf16(cfg["seed"], 2, (heads, L, d)).double().numpy()
    V = inputs.normal_bf16(cfg["seed"], 3, (heads, L, d)).double().numpy()
    dO = inputs.normal_bf16(cfg["seed"], 4, (heads, L, d)).double().numpy()
    pairs = orc.kept_pairs(f, cfg["n_init"], cfg["n_neighbor"])
    t0 = time.perf_counter()
    M = orc.mask_matrix(f, cfg["n_init"], cfg["n_neighbor"])
    for h in range(heads):
        dq, _, _ = orc.attn_bwd_head(Q[h], K[h // G], V[h // G], dO[h], M)
        if keep is not None and h == 0:
            keep["dQ"] = dq
    dt = time.perf_counter() - t0
    if keep is not None:
        keep["O"], keep["LSE"], _ = orc.attn_fwd_rows(Q[0], K[0], V[0], M)    # untimed
    cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    tflops = 14.0 * d * pairs * heads / dt / 1e12
    return tflops, dt, cores, f"fwd+bwd of {heads} query head(s) on the first {L} tokens of the workload"


# ---------------------------------------------------------------------------- GPU arm
class Workload:
    def __init__(self, name: str, rank: int, device: torch.device, fwd_only: bool = False):
        from paper_2412_12094_b200 import api
        self.api = api
        self.fwd_only = fwd_only
        cfg = dict(inputs.CONFIGS[name])
        cfg["seed"] = cfg["seed"] + 1000 * rank
        self.cfg, self.name, self.device = cfg, name, device
        B, Hq, Hkv, L, d = cfg["B"], cfg["Hq"], cfg["Hkv"], cfg["L"], cfg["d"]
        self.ids_h = torch.from_numpy(inputs.token_ids(cfg["seed"], B, L, cfg["rho"], cfg["structure"])).pin_memory()
        Q, K, V, dO = inputs.qkv_do(cfg["seed"], B, Hq, Hkv, L, d)
        self.host = [t.pin_memory() for t in (Q, K, V, dO)]
        self.ids = self.ids_h.to(device)
        self.Q, self.K, self.V, self.dO = (t.to(device) for t in self.host)
        # capacity of the side list: initial tokens plus separators at 1.25x the expected rate and a
        # margin (the index reports CAPACITY_EXCEEDED if a sequence has more, and the run stops)
        side_cap = min(L, (int(1.25 * cfg["rho"] * L) + cfg["n_init"] + 2048 + 127) // 128 * 128)
        self.idesc = api.IndexDesc(B, L, cfg["n_init"], cfg["n_neighbor"], len(inputs.SEP_IDS), 128, 128, side_cap)
        ib, sb = api.sepllm_index_bytes(self.idesc)
        self.index = api.alloc_bytes(ib)
        self.scratch = api.alloc_bytes(sb)
        self.fdesc = api.AttnDesc(B, Hq, Hkv, d, L, 0.0, 0)
        self.bdesc = api.AttnDesc(B, Hq, Hkv, d, L, 0.0, 0)
        self.bdesc.flags = api.SIDE_READY          # backward reuses the forward's side K/V
        _, bb = api.sepllm_attn_workspace_bytes(self.fdesc, self.idesc)
        self.ws = api.alloc_bytes(bb)
        self.O = torch.empty_like(self.Q)
        self.LSE = torch.empty((B, Hq, L), dtype=torch.float32, device=device)
        self.dQ = torch.empty_like(self.Q)
        self.dK = torch.empty_like(self.K)
        self.dV = torch.empty_like(self.V)
        self.out_h = [torch.empty_like(t, device="cpu").pin_memory() for t in (self.O, self.dQ, self.dK, self.dV)]
        # index scan | side gather, forward | Delta, dQ, dK/dV side, dK/dV window
        # index (clear + scan); gather + forward; delta + dQ (two instances, the one that does not match the index
        # returns at once) + dK/dV side + dK/dV window
        self.launches_per_step = 2 + 2 + (0 if fwd_only else 5)

    def step(self, bufs=None):
        api = self.api
        ids, Q, K, V, dO, O, dQ, dK, dV = bufs if bufs is not None else (
            self.ids, self.Q, self.K, self.V, self.dO, self.O, self.dQ, self.dK, self.dV)
        api.sepllm_build_index(self.idesc, ids, inputs.SEP_IDS, self.index, self.scratch)
        api.sepllm_attn_fwd(self.fdesc, self.idesc, Q, K, V, self.index, O, self.LSE, self.ws)
        if not self.fwd_only:
            api.sepllm_attn_bwd(self.bdesc, self.idesc, dO, Q, K, V, O, self.LSE, self.index, dQ, dK, dV, self.ws)

    # End to end: every step copies its inputs from pinned host memory and its results back.  The
    # copies run on streams of their own over two sets of device buffers, so the copy-in of step
    # i+1 and the copy-out of step i-1 overlap the kernels of step i (both PCIe directions busy).
    def e2e_begin(self):
        if not hasattr(self, "sets"):
            first = (self.ids, self.Q, self.K, self.V, self.dO, self.O, self.dQ, self.dK, self.dV)
            self.sets = [first, tuple(torch.empty_like(t) for t in first)]
            self.s_in, self.s_out = torch.cuda.Stream(), torch.cuda.Stream()
        cur = torch.cuda.current_stream()
        self.s_in.wait_stream(cur)
        self.s_out.wait_stream(cur)
        self.ev_in = [None, None]      # inputs of the set have landed
        self.ev_comp = [None, None]    # kernels on the set are done (its inputs may be overwritten)
        self.ev_out = [None, None]     # results of the set are on the host (its outputs may be overwritten)
        self.e2e_i = 0

    def step_e2e(self):
        k = self.e2e_i % 2
        self.e2e_i += 1
        bufs = self.sets[k]
        cur = torch.cuda.current_stream()
        with torch.cuda.stream(self.s_in):
            if self.ev_comp[k] is not None:
                self.s_in.wait_event(self.ev_comp[k])
            for dst, src in zip(bufs[:5], [self.ids_h] + self.host):
                dst.copy_(src, non_blocking=True)
            self.ev_in[k] = self.s_in.record_event()
        cur.wait_event(self.ev_in[k])
        if self.ev_out[k] is not None:
            cur.wait_event(self.ev_out[k])
        self.step(bufs)
        self.ev_comp[k] = cur.record_event()
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_comp[k])
            for dst, src in zip(self.out_h, bufs[5:]):
                dst.copy_(src, non_blocking=True)
            self.ev_out[k] = self.s_out.record_event()

    def e2e_end(self):
        cur = torch.cuda.current_stream()
        cur.wait_stream(self.s_in)
        cur.wait_stream(self.s_out)

    def e2e_bytes(self):
        h2d = self.ids_h.numel() * 4 + sum(t.numel() * 2 for t in self.host)
        d2h = sum(t.numel() * 2 for t in self.out_h)
        return h2d, d2h

    def kept_pairs(self):
        torch.cuda.synchronize()
        idx = self.api.read_index(self.index)
        assert idx["header"].status == 0
        assert self.api.sepllm_last_device_status(self.ws) == 0
        total = idx["tile_meta"][:, :, 6].astype(np.int64).sum()
        side = idx["lim"].astype(np.int64).sum()
        # iterations of the key-stationary side pass per query head: every side tile meets the
        # query tiles from the first one that keeps its first entry to the last
        T, n = idx["header"].n_tiles, self.cfg["n_neighbor"]
        self.side_iters = 0
        for b in range(self.cfg["B"]):
            ns = int(min(idx["n_side"][b], idx["side_pos"].shape[1]))
            first = (idx["side_pos"][b, 0:ns:128].astype(np.int64) + n) // 128
            self.side_iters += int(np.maximum(T - first, 0).sum())
        return int(total), int(side)


def aggregate(sec: float, work: float, device, dist=None):
    """Whole-job figures from per-rank ones: time = max over ranks, work = sum over ranks."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return sec, work
    t = torch.tensor([sec], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    w = torch.tensor([work], device=device, dtype=torch.float64)
    dist.all_reduce(w, op=dist.ReduceOp.SUM)
    return float(t.item()), float(w.item())


def timed(fn, steps, warmup, dist_barrier, begin=None, end=None):
    """begin / end: hooks after the start event and before the stop event (work on other streams
    is tied to the timed stream there)."""
    if begin is not None:
        begin()
    for _ in range(warmup):
        fn()
    if end is not None:
        end()
    torch.cuda.synchronize()
    dist_barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    if begin is not None:
        begin()
    for _ in range(steps):
        fn()
    if end is not None:
        end()
    e1.record()
    torch.cuda.synchronize()
    dist_barrier()
    return e0.elapsed_time(e1) / 1e3


def kernel_times(wl: Workload, steps: int):
    """Per-kernel average durations (seconds) from events the library records between its launches."""
    def mk(n):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        for e in evs:
            e.record()           # creates the handle
        return evs
    fsets = [mk(3) for _ in range(steps)]
    bsets = [mk(6) for _ in range(steps)]
    isets = [mk(2) for _ in range(steps)]
    torch.cuda.synchronize()
    api = wl.api
    for s in range(steps):
        isets[s][0].record()
        api.sepllm_build_index(wl.idesc, wl.ids, inputs.SEP_IDS, wl.index, wl.scratch)
        isets[s][1].record()
        wl.fdesc.set_events(fsets[s])
        api.sepllm_attn_fwd(wl.fdesc, wl.idesc, wl.Q, wl.K, wl.V, wl.index, wl.O, wl.LSE, wl.ws)
        wl.bdesc.set_events(bsets[s])
        api.sepllm_attn_bwd(wl.bdesc, wl.idesc, wl.dO, wl.Q, wl.K, wl.V, wl.O, wl.LSE, wl.index,
                            wl.dQ, wl.dK, wl.dV, wl.ws)
    torch.cuda.synchronize()
    wl.fdesc.set_events(None)
    wl.bdesc.set_events(None)

    def avg(sets, i):
        return sum(s[i].elapsed_time(s[i + 1]) for s in sets) / len(sets) / 1e3
    return {
        "build_index": avg(isets, 0),
        "gather_side_kv": avg(fsets, 0),
        "attn_fwd_kernel": avg(fsets, 1),
        "bwd_delta": avg(bsets, 1),
        "bwd_dq_kernel": avg(bsets, 2),
        "bwd_dkv_kernel<side>": avg(bsets, 3),
        "bwd_dkv_kernel<window>": avg(bsets, 4),
    }


def bench_other_workloads(main_name, device, peaks, steps=10, warmup=3):
    """The remaining training / prefill workloads, each timed like the main one (device-resident
    inputs, index build inside the step).  The prefill-shaped workload is forward only."""
    out = {}
    for name in ("tiny", "pythia160m", "llama8b_prefill", "llama8b_long_r05", "llama8b_long_r10", "llama8b_long_r20"):
        if name == main_name:
            continue
        cfg = inputs.CONFIGS[name]
        fwd_only = name == "llama8b_prefill"
        wl = Workload(name, 0, device, fwd_only=fwd_only)
        wl.step()
        pairs, _ = wl.kept_pairs()
        sec = timed(wl.step, steps, warmup, lambda: None)
        flops = (4.0 if fwd_only else 14.0) * cfg["d"] * pairs * cfg["Hq"]
        tf = flops * steps / sec / 1e12
        out[name] = {"pass": "fwd" if fwd_only else "fwd+bwd", "ms_per_step": sec / steps * 1e3,
                     "tflops": tf, "frac_of_bf16_peak": tf / peaks["bf16_tflops_sustained"],
                     "kept_pairs": pairs, "steps": steps, "gpu_launches": wl.launches_per_step * steps}
        del wl
        torch.cuda.empty_cache()
    return out


def bench_decode(device, peaks, steps=4096, rope=False):
    """Streaming workload: cache update + decode per step at the full cache shape.  rope: positions
    inside the cache (the update keeps a rotated copy of the keys, the decode reads that)."""
    from paper_2412_12094_b200 import api
    c = inputs.DECODE_CONFIG
    B, Hq, Hkv, d = c["B"], c["Hq"], c["Hkv"], c["d"]
    desc = api.CacheDesc(B, Hkv, Hq, d, c["a"], c["s"], c["w"], c["c"])
    sb, kb = api.sepllm_cache_bytes(desc)
    state = api.alloc_bytes(sb)
    Kc = torch.zeros(kb // 2, dtype=torch.bfloat16, device=device)
    Vc = torch.zeros(kb // 2, dtype=torch.bfloat16, device=device)
    ws = api.alloc_bytes(api.sepllm_decode_workspace_bytes(desc))
    api.sepllm_cache_init(desc, state)
    if rope:
        table = api.alloc_bytes(api.sepllm_rope_table_bytes(desc))
        api.sepllm_rope_table_build(desc, 500000.0, table)
        Kr = torch.zeros_like(Kc)
    pool = 256
    warm = 12032                      # enough tokens to fill the separator cache (s / rho plus slack)
    T = warm + steps
    ids = inputs.decode_stream_ids(c["seed"], B, T, c["rho"])
    ids_d = torch.from_numpy(np.ascontiguousarray(ids.T)).to(device)
    kp, vp, qp = (t.to(device) for t in inputs.decode_kv_pool(c["seed"], pool, B, Hkv, Hq, d))
    o = torch.empty((B, Hq, d), dtype=torch.bfloat16, device=device)
    lse = torch.empty((B, Hq), dtype=torch.float32, device=device)

    def step(t, ids_row):
        if rope:
            api.sepllm_cache_update_rope(desc, state, Kc, Vc, Kr, table, ids_row, inputs.SEP_IDS,
                                         kp[t % pool], vp[t % pool])
            api.sepllm_decode_rope(desc, 0.0, qp[t % pool], state, Kr, Vc, table, o, lse, ws)
        else:
            api.sepllm_cache_update(desc, state, Kc, Vc, ids_row, inputs.SEP_IDS, kp[t % pool], vp[t % pool])
            api.sepllm_decode(desc, 0.0, qp[t % pool], state, Kc, Vc, o, lse, ws)

    for t in range(warm):
        step(t, ids_d[t])
    torch.cuda.synchronize()
    st0 = api.read_cache_state(state)
    # bookkeeping of Size_run per step (sizes only) for the byte count
    f = np.isin(ids, inputs.SEP_IDS)
    size_sep = st0["size_sep"].astype(np.int64).copy()
    size_win = st0["size_win"].astype(np.int64).copy()
    size_init = st0["size_init"].astype(np.int64)
    rows = 0
    # the window's separator flags are needed to know how many move at a compaction
    win_flags = [list(f[b, warm - size_win[b]:warm]) for b in range(B)]
    for t in range(warm, T):
        for b in range(B):
            win_flags[b].append(bool(f[b, t]))
            if size_init[b] + size_sep[b] + len(win_flags[b]) == c["c"]:
                n_past = len(win_flags[b]) - c["w"]
                size_sep[b] = min(c["s"], size_sep[b] + sum(win_flags[b][:n_past]))
                win_flags[b] = win_flags[b][n_past:]
            rows += size_init[b] + size_sep[b] + len(win_flags[b])
    # One CUDA graph holds `pool` consecutive steps (3 kernels each); the token ids of a chunk are
    # copied into the graph's fixed input buffer inside the timed region.
    assert warm % pool == 0 and steps % pool == 0
    ids_buf = torch.empty((pool, B), dtype=torch.int32, device=device)
    ids_buf.copy_(ids_d[warm:warm + pool])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(pool):
                step(warm + i, ids_buf[i])
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t0 in range(warm, T, pool):
        ids_buf.copy_(ids_d[t0:t0 + pool], non_blocking=True)
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(state) == 0
    st1 = api.read_cache_state(state)
    assert (st1["size_sep"] == size_sep).all() and (st1["size_win"] == [len(w) for w in win_flags]).all()
    sec = e0.elapsed_time(e1) / 1e3
    bytes_total = rows * Hkv * d * 2 * 2          # K and V rows of every retained entry, every kv head
    gbs = bytes_total / sec / 1e9
    return {"workload": "B32 Hq32 Hkv8 d128 a4 s1024 w256 c3332, update+decode per step"
                        + (", rotary positions inside the cache (base 500000)" if rope else ""),
            "steps": steps, "us_per_step": sec / steps * 1e6, "avg_size_run": rows / steps / B,
            "bytes_per_step": bytes_total / steps, "achieved_gbs": gbs,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "traffic": None},
            "tokens_per_s": B * steps / sec, "gpu_launches": 3 * steps}


def bench_index_stream(device, peaks, reps=20):
    from paper_2412_12094_b200 import api
    c = inputs.DECODE_CONFIG
    B, L = c["B"], c["stream_len"]
    ids = torch.from_numpy(inputs.decode_stream_ids(c["seed"], B, L, c["rho"])).to(device)
    desc = api.IndexDesc(B, L, 4, 256, len(inputs.SEP_IDS), 128, 128, L // 4)
    ib, sb = api.sepllm_index_bytes(desc)
    index, scratch = api.alloc_bytes(ib), api.alloc_bytes(sb)
    for _ in range(3):
        api.sepllm_build_index(desc, ids, inputs.SEP_IDS, index, scratch)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        api.sepllm_build_index(desc, ids, inputs.SEP_IDS, index, scratch)
    e1.record()
    torch.cuda.synchronize()
    sec = e0.elapsed_time(e1) / 1e3 / reps
    n_side = int(api.read_index(index)["n_side"].astype(np.int64).sum())
    T = (L + 127) // 128
    algo = 4 * B * L + 4 * B * (L + 1) + 4 * B * L + 4 * n_side + 32 * B * T
    gbs = algo / sec / 1e9
    return {"workload": "32 x 2^20 token ids", "us": sec * 1e6, "bytes": algo,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "traffic": None}}


def bench_hand_off(device, peaks, reps=20, L=16384):
    """Prompt hand-off: the streaming workload's cache filled from 16384-token prompts."""
    from paper_2412_12094_b200 import api
    c = inputs.DECODE_CONFIG
    B, Hq, Hkv, d = c["B"], c["Hq"], c["Hkv"], c["d"]
    desc = api.CacheDesc(B, Hkv, Hq, d, c["a"], c["s"], c["w"], c["c"])
    sb, kb = api.sepllm_cache_bytes(desc)
    state = api.alloc_bytes(sb)
    Kc = torch.zeros(kb // 2, dtype=torch.bfloat16, device=device)
    Vc = torch.zeros(kb // 2, dtype=torch.bfloat16, device=device)
    ids = torch.from_numpy(inputs.decode_stream_ids(c["seed"], B, L, c["rho"])).to(device)
    idesc = api.IndexDesc(B, L, c["a"], c["w"], len(inputs.SEP_IDS), 128, 128, L)
    ib, scb = api.sepllm_index_bytes(idesc)
    index, scratch = api.alloc_bytes(ib), api.alloc_bytes(scb)
    api.sepllm_build_index(idesc, ids, inputs.SEP_IDS, index, scratch)
    g = torch.Generator(device=device).manual_seed(c["seed"])
    K = torch.randn((B, Hkv, L, d), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    V = torch.randn((B, Hkv, L, d), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)

    def call():
        api.sepllm_cache_from_prompt(desc, idesc, index, None, K, V, state, Kc, Vc)

    for _ in range(3):
        call()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        call()
    e1.record()
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(state) == 0
    sec = e0.elapsed_time(e1) / 1e3 / reps
    st = api.read_cache_state(state)
    rows = int((st["size_init"] + st["size_sep"] + st["size_win"]).astype(np.int64).sum())
    algo = rows * Hkv * d * 2 * 2 * 2 + 9 * B * (c["c"] + c["s"])   # K and V rows read and written; slot metadata
    gbs = algo / sec / 1e9
    return {"workload": f"B32 Hkv8 d128 a4 s1024 w256 c3332 from {L}-token prompts", "us": sec * 1e6,
            "bytes": algo, "avg_size_run": rows / B, "gpu_launches": 2 * reps,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "traffic": None}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_long_r10", choices=sorted(inputs.CONFIGS))
    ap.add_argument("--no-extras", action="store_true", help="skip the decode / index-stream / e2e / CPU legs")
    ap.add_argument("--leg", default="all", choices=["all", "decode", "decode_rope", "index", "hand_off"],
                    help="run only that secondary leg and print its JSON")
    ap.add_argument("--cpu-prefix", type=int, default=8192)
    ap.add_argument("--cpu-heads", type=int, default=4)
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    cfg = inputs.CONFIGS[args.workload]
    config = {"workload": f"{args.workload}: B{cfg['B']} Hq{cfg['Hq']} Hkv{cfg['Hkv']} d{cfg['d']} L{cfg['L']} "
                          f"n_init{cfg['n_init']} n_neighbor{cfg['n_neighbor']} sep_rate{cfg['rho']} "
                          f"({cfg['structure']}), fwd+bwd incl. index build",
              "l2": "inputs larger than L2 (no flush)", "replicas": world}

    if args.impl == "reference":
        # the CPU oracle, as it stands, on a bounded sample; rank 0 only
        if rank != 0:
            return
        vals, secs = [], []
        for _ in range(args.warmup):
            oracle_sample(cfg, 1, min(args.cpu_prefix, 2048))
        for _ in range(args.steps):
            v, dt, cores, what = oracle_sample(cfg, 1, min(args.cpu_prefix, 4096))
            vals.append(v)
            secs.append(dt)
        val = sum(v * s for v, s in zip(vals, secs)) / sum(secs)   # time-weighted mean
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs) / len(secs),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config,
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

        def barrier():
            dist.barrier()
    else:
        dist = None

        def barrier():
            pass

    peaks = load_peaks()
    if args.leg != "all":
        print(json.dumps(bench_index_stream(device, peaks) if args.leg == "index"
                         else bench_hand_off(device, peaks) if args.leg == "hand_off"
                         else bench_decode(device, peaks, rope=(args.leg == "decode_rope"))))
        return
    wl = Workload(args.workload, rank, device)
    wl.step()
    pairs, side_pairs = wl.kept_pairs()
    d, Hq = cfg["d"], cfg["Hq"]
    flops_step = 14.0 * d * pairs * Hq            # pairs is summed over the batch already

    sampler = ClockSampler(local) if rank == 0 else None
    sec = timed(wl.step, args.steps, args.warmup, barrier)
    clocks = sampler.stop() if sampler else None
    sec, flops_total_step = aggregate(sec, flops_step, device, dist)
    value = flops_total_step * args.steps / sec / 1e12

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": sec / args.steps * 1e3, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
           "config": config, "gpu_launches": wl.launches_per_step * args.steps,
           "kept_pairs": pairs, "frac_of_bf16_peak": value / world / peaks["bf16_tflops_sustained"],
           "peaks": {k: peaks[k] for k in ("hbm_gbs", "bf16_tflops", "bf16_tflops_sustained", "source")}}
    if clocks is not None:
        out["clocks"] = clocks

    # per-kernel durations and the roofline of the dominant kernel (rank 0's replica)
    kt = kernel_times(wl, min(args.steps, 10))
    # (wl.side_iters was set by kept_pairs above)
    win_pairs = pairs - side_pairs
    kflops = {
        "attn_fwd_kernel": 4.0 * d * pairs * Hq,
        "bwd_dq_kernel": 6.0 * d * pairs * Hq,
        "bwd_dkv_kernel<side>": 8.0 * d * side_pairs * Hq,
        "bwd_dkv_kernel<window>": 8.0 * d * win_pairs * Hq,
    }
    tot = sum(kt.values())
    out["kernels"] = {k: {"ms": v * 1e3, "share": v / tot,
                          **({"tflops": kflops[k] / v / 1e12} if k in kflops and v > 0 else {})}
                      for k, v in kt.items()}
    side_iters = wl.side_iters
    dom = max(kflops, key=lambda k: kt[k])
    ach = kflops[dom] / kt[dom] / 1e12
    # DRAM bytes of the dominant kernel: from one ncu capture of the 16 384-token copy of this
    # workload (bytes read + written over 836 side-pass iterations per query head), scaled by the
    # iteration count, which is what the kernel's Q / dO stream grows with.  Valid for
    # bwd_dkv_kernel<side> as captured; None for anything else.
    traffic = None
    if dom == "bwd_dkv_kernel<side>" and cfg["d"] == 128 and cfg["Hq"] == 32 and cfg["B"] == 1:
        traffic = (686.49e6 + 39.55e6) * side_iters / 836.0
    out["roofline"] = {"kernel": dom, "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"],
                       "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops_sustained"], "traffic": traffic,
                       "peak_kind": f"bf16 sustained, {peaks['source']}",
                       "flops_per_launch": kflops[dom]}

    if not args.no_extras:
        # end to end: host buffers in, results back, copies inside the timed region
        n_e = max(2, args.steps)   # as many steps as the device-resident timing: the pipeline's fill and drain are inside
        sec_e = timed(wl.step_e2e, n_e, 2, barrier, wl.e2e_begin, wl.e2e_end)
        sec_e, _ = aggregate(sec_e, 0.0, device, dist)
        h2d, d2h = wl.e2e_bytes()
        out["e2e"] = {"value": flops_total_step * n_e / sec_e / 1e12, "unit": UNIT,
                      "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                      "ms_per_step": sec_e / n_e * 1e3, "steps": n_e,
                      "copies": "on their own streams over two sets of device buffers, overlapping the kernels"}
        if rank == 0:
            # rows of the last step's results that the CPU leg below recomputes (head 0, first tokens)
            P = min(args.cpu_prefix, cfg["L"])
            torch.cuda.synchronize()
            got = {"O": wl.O[0, 0, :P].float().cpu().numpy(), "LSE": wl.LSE[0, 0, :P].cpu().numpy(),
                   "dQ": wl.dQ[0, 0, :P].float().cpu().numpy()}
            del wl
            torch.cuda.empty_cache()
            out["workloads"] = bench_other_workloads(args.workload, device, peaks)
            out["decode"] = bench_decode(device, peaks)
            out["decode_rope"] = bench_decode(device, peaks, rope=True)
            out["index"] = bench_index_stream(device, peaks)
            out["hand_off"] = bench_hand_off(device, peaks)
            if world == 1:
                keep = {}
                v, dt, cores, what = oracle_sample(cfg, args.cpu_heads, args.cpu_prefix, keep)
                out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                       "sample": what, "seconds": dt}
                # the same rows from the timed GPU run against the oracle's (query head 0)
                out["parity"] = {"sample": f"O, LSE, dQ of query head 0, first {P} rows, against the fp64 oracle"}
                for k in ("O", "dQ"):
                    diff = got[k].astype(np.float64) - keep[k]
                    out["parity"][k] = {"max_abs": float(np.abs(diff).max()),
                                        "rel_fro": float(np.linalg.norm(diff) / np.linalg.norm(keep[k]))}
                out["parity"]["LSE"] = {"max_abs": float(np.abs(got["LSE"] - keep["LSE"]).max())}
    if world > 1:
        barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


if __name__ == "__main__":
    main()
