"""Helpers shared by the GPU parity tests: run the C-ABI calls on seeded inputs."""
import numpy as np
import torch

from paper_2412_12094_b200 import api, inputs

# Tolerances of the parity bar: bf16 outputs against the fp64 oracle.
TOL_O = dict(max_abs=1e-2, rel_fro=5e-3)
TOL_GRAD = dict(max_abs=2e-2, rel_fro=1e-2)
TOL_LSE = 1e-3


def errors(got: np.ndarray, ref: np.ndarray, scaled: bool = False):
    """(max-abs, relative Frobenius) of got against ref.  scaled=True divides each element's
    error by max(1, |ref|); only the named degenerate cases use it (rows that keep one or two
    keys copy V rows of magnitude 4 and more, where bf16 rounding alone is 0.016)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    diff = np.abs(got - ref)
    if scaled:
        diff = diff / np.maximum(1.0, np.abs(ref))
    return float(diff.max()) if diff.size else 0.0, \
        float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-300))


def assert_close(got, ref, tol, what="", scaled=False):
    ma, rf = errors(got, ref, scaled)
    assert np.isfinite(np.asarray(got, dtype=np.float64)).all(), f"{what}: non-finite output"
    assert ma <= tol["max_abs"] and rf <= tol["rel_fro"], f"{what}: max_abs={ma:.3e} rel_fro={rf:.3e}"
    return ma, rf


# Rounding floor of a gradient entry: the kernels feed P and dS to the tensor cores as bf16, so
# every term of the sum behind an entry is off by up to 2^-9 of its size (uniform, independent):
# standard deviation 2^-9 / sqrt(3) of the terms' root-sum-square `rss`.  Delta is computed from
# the bf16 output O, which perturbs dS by about as much again, and a bf16 result adds its own
# half ulp.  K_ROUND standard deviations of the two together: 6 * sqrt(2) / sqrt(3) ~ 5.
K_ROUND = 5.0


def assert_grad_close(got, ref, rss, what="", bf16_out=True):
    """Gradient entries against the oracle: the absolute bound of the parity bar, raised only for
    entries whose own terms are so large that bf16 operand rounding alone exceeds it (rss from
    oracle.attn_bwd_term_scale); relative Frobenius error as everywhere else."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    floor = K_ROUND * 2.0 ** -9 * np.asarray(rss) + (2.0 ** -9 * np.abs(ref) if bf16_out else 0.0)
    tol = np.maximum(TOL_GRAD["max_abs"], floor)
    diff = np.abs(got - ref)
    worst = float((diff / tol).max()) if diff.size else 0.0
    assert worst <= 1.0, f"{what}: an entry is off by {worst:.2f} x its bound (max_abs={diff.max():.3e})"
    return float(diff.max()), float((diff / np.maximum(floor, 1e-300)).max())


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


def assert_o_close(got, ref, rss, what=""):
    """Entries of O against the oracle: the absolute bound of the parity bar, raised only for
    entries whose own terms are so large that the bf16 rounding of the weights (rss from
    oracle.attn_fwd_term_scale) and of the bf16 output exceeds it -- rows that keep one or two
    keys return (nearly) a V row itself, entries of 3 and 4 among them, and inputs made of many
    short documents hold hundreds of such rows.  Relative Frobenius error as everywhere else."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    tol = np.maximum(TOL_O["max_abs"], K_ROUND * 2.0 ** -9 * np.asarray(rss) + 2.0 ** -9 * np.abs(ref))
    worst = float((np.abs(got - ref) / tol).max()) if got.size else 0.0
    assert worst <= 1.0, f"{what}: an entry is off by {worst:.2f} x its bound"
    assert errors(got, ref)[1] <= TOL_O["rel_fro"], (what, errors(got, ref))
