"""Helpers shared by the GPU parity tests: run the C-ABI calls on seeded inputs."""
import numpy as np
import torch

from paper_2412_12094_b200 import api, inputs

# Tolerances of the parity bar: bf16 outputs against the fp64 oracle.
TOL_O = dict(max_abs=1e-2, rel_fro=5e-3)
TOL_GRAD = dict(max_abs=2e-2, rel_fro=1e-2)
TOL_LSE = 1e-3


def errors(got: np.ndarray, ref: np.ndarray):
    """(max-abs, relative Frobenius).  The max-abs figure divides each element's error by
    max(1, |ref|): a bf16 result of magnitude 4 is 0.016 away from the exact value by rounding
    alone, so above 1 the bound has to scale with the value; on the paper-shaped workloads
    (|O| < 1) it is the plain max-abs error."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    diff = got - ref
    scaled = np.abs(diff) / np.maximum(1.0, np.abs(ref))
    return float(scaled.max()), float(np.linalg.norm(diff) / max(np.linalg.norm(ref), 1e-300))


def assert_close(got, ref, tol, what=""):
    ma, rf = errors(got, ref)
    assert np.isfinite(np.asarray(got, dtype=np.float64)).all(), f"{what}: non-finite output"
    assert ma <= tol["max_abs"] and rf <= tol["rel_fro"], f"{what}: max_abs={ma:.3e} rel_fro={rf:.3e}"
    return ma, rf


def build_index(token_ids_np, sep_ids, a, n, side_cap=None, BM=128, BN=128):
    B, L = token_ids_np.shape
    side_cap = L if side_cap is None else side_cap
    desc = api.IndexDesc(B, L, a, n, len(sep_ids), BM, BN, side_cap)
    ib, sb = api.sepllm_index_bytes(desc)
    index = api.alloc_bytes(ib)
    scratch = api.alloc_bytes(sb)
    ids = torch.from_numpy(np.ascontiguousarray(token_ids_np)).cuda()
    api.sepllm_build_index(desc, ids, sep_ids, index, scratch)
    return desc, index


def attn_fwd(Q, K, V, idesc, index, scale=0.0):
    """Q [B][Hq][L][d], K/V [B][Hkv][L][d] bf16 CUDA tensors -> O (bf16), LSE (fp32)."""
    B, Hq, L, d = Q.shape
    desc = api.AttnDesc(B, Hq, K.shape[1], d, L, scale, 0)
    fb, _ = api.sepllm_attn_workspace_bytes(desc, idesc)
    ws = api.alloc_bytes(fb)
    O = torch.empty_like(Q)
    LSE = torch.empty((B, Hq, L), dtype=torch.float32, device=Q.device)
    api.sepllm_attn_fwd(desc, idesc, Q, K, V, index, O, LSE, ws)
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(ws) == 0
    return O, LSE


def attn_bwd(dO, Q, K, V, O, LSE, idesc, index, grad_dtype=0, scale=0.0):
    B, Hq, L, d = Q.shape
    desc = api.AttnDesc(B, Hq, K.shape[1], d, L, scale, grad_dtype)
    _, bb = api.sepllm_attn_workspace_bytes(desc, idesc)
    ws = api.alloc_bytes(bb)
    dt = torch.bfloat16 if grad_dtype == 0 else torch.float32
    dQ = torch.empty(Q.shape, dtype=dt, device=Q.device)
    dK = torch.empty(K.shape, dtype=dt, device=Q.device)
    dV = torch.empty(V.shape, dtype=dt, device=Q.device)
    api.sepllm_attn_bwd(desc, idesc, dO, Q, K, V, O, LSE, index, dQ, dK, dV, ws)
    torch.cuda.synchronize()
    assert api.sepllm_last_device_status(ws) == 0
    return dQ, dK, dV


def flags_of(ids_np, sep_ids):
    return np.isin(ids_np, np.asarray(sep_ids))
