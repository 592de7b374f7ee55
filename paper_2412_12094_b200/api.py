"""Python binding of libsepllm: argument marshalling only.

Every function has the name of the C entry point it calls (see include/sepllm.h)
and passes torch tensors' device pointers and the current CUDA stream through.
Nothing here computes: if the shared library is missing the import fails.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsepllm.so")

OK, INVALID_ARG, UNSUPPORTED, BUFFER_TOO_SMALL, CUDA_ERROR, CAPACITY_EXCEEDED, TIMEOUT, NOT_BUILT = range(8)


class IndexDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("B", "L", "n_init", "n_neighbor", "n_sep", "BM", "BN", "side_cap")]


SIDE_READY = 1


class AttnDesc(C.Structure):
    _fields_ = [("B", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("d", C.c_int32),
                ("L", C.c_int32), ("scale", C.c_float), ("grad_dtype", C.c_int32),
                ("flags", C.c_int32), ("events", C.POINTER(C.c_void_p)), ("n_events", C.c_int32)]

    def set_events(self, events):
        """events: torch.cuda.Event objects (timing enabled, recorded once so their handles
        exist), or None to switch per-kernel timing off."""
        if not events:
            self.events, self.n_events, self._keep = None, 0, None
            return
        arr = (C.c_void_p * len(events))(*[e.cuda_event for e in events])
        self._keep = arr
        self.events = C.cast(arr, C.POINTER(C.c_void_p))
        self.n_events = len(events)


CACHE_FIXED_WINDOW = 1


class CacheDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("B", "Hkv", "Hq", "d", "a", "s", "w", "c", "flags")]


class IndexHeader(C.Structure):
    _fields_ = [("status", C.c_int32), ("magic", C.c_uint32), ("version", C.c_uint32),
                ("desc", IndexDesc), ("n_tiles", C.c_int32),
                ("off_cnt", C.c_int64), ("off_lim", C.c_int64), ("off_side_pos", C.c_int64),
                ("off_n_side", C.c_int64), ("off_tile_meta", C.c_int64), ("total_bytes", C.c_int64),
                ("off_seq_len", C.c_int64), ("off_doc_start", C.c_int64), ("off_doc_end", C.c_int64),
                ("packed", C.c_int64), ("reserved", C.c_int64 * 16)]


class CacheHeader(C.Structure):
    _fields_ = [("status", C.c_int32), ("magic", C.c_uint32), ("version", C.c_uint32),
                ("slots", C.c_int32), ("desc", CacheDesc),
                ("off_seq", C.c_int64), ("off_slot_pos", C.c_int64), ("off_slot_is_sep", C.c_int64),
                ("total_bytes", C.c_int64), ("reserved", C.c_int64 * 21)]


EXPORTS = [
    "sepllm_index_bytes", "sepllm_build_index", "sepllm_build_index_varlen", "sepllm_build_index_packed",
    "sepllm_build_index_static",
    "sepllm_build_index_fixed_interval",
    "sepllm_attn_workspace_bytes", "sepllm_attn_fwd",
    "sepllm_attn_bwd", "sepllm_cache_bytes", "sepllm_cache_init", "sepllm_cache_update",
    "sepllm_cache_from_prompt", "sepllm_cache_update_rope",
    "sepllm_decode_workspace_bytes", "sepllm_decode", "sepllm_rope_table_bytes",
    "sepllm_rope_table_build", "sepllm_decode_rope", "sepllm_last_device_status",
    "sepllm_status_string",
]

_lib = None


def lib() -> C.CDLL:
    """Loads libsepllm.so; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run paper_2412_12094_b200/build.py "
                               "(there is no fallback path)")
        _lib = C.CDLL(LIB_PATH)
        _lib.sepllm_status_string.restype = C.c_char_p
        _lib.sepllm_status_string.argtypes = [C.c_int]
        for name in EXPORTS:
            if name != "sepllm_status_string":
                getattr(_lib, name).restype = C.c_int
    return _lib


class SepllmError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib().sepllm_status_string(code).decode()} ({code})")


def _check(code: int, where: str):
    if code != OK:
        raise SepllmError(code, where)


def _ptr(t):
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, torch.Tensor):
        assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
        return C.c_void_p(t.data_ptr())
    return C.c_void_p(int(t))


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _sep_array(sep_ids):
    arr = np.ascontiguousarray(np.asarray(sep_ids, dtype=np.int32))
    return arr, arr.ctypes.data_as(C.c_void_p), int(arr.size)


def status_string(code: int) -> str:
    return lib().sepllm_status_string(code).decode()


# ---------------------------------------------------------------- index
def sepllm_index_bytes(desc: IndexDesc):
    ib, sb = C.c_size_t(0), C.c_size_t(0)
    _check(lib().sepllm_index_bytes(C.byref(desc), C.byref(ib), C.byref(sb)), "sepllm_index_bytes")
    return ib.value, sb.value


def sepllm_build_index(desc: IndexDesc, token_ids: torch.Tensor, sep_ids, index: torch.Tensor,
                       scratch: torch.Tensor):
    arr, p, n = _sep_array(sep_ids)
    assert n == desc.n_sep
    _check(lib().sepllm_build_index(C.byref(desc), _ptr(token_ids), p, _ptr(index), _ptr(scratch),
                                    _stream()), "sepllm_build_index")


def sepllm_build_index_varlen(desc: IndexDesc, token_ids: torch.Tensor, seq_len: torch.Tensor, sep_ids,
                              index: torch.Tensor, scratch: torch.Tensor):
    arr, p, n = _sep_array(sep_ids)
    assert n == desc.n_sep
    _check(lib().sepllm_build_index_varlen(C.byref(desc), _ptr(token_ids), _ptr(seq_len), p, _ptr(index),
                                           _ptr(scratch), _stream()), "sepllm_build_index_varlen")


def sepllm_build_index_packed(desc: IndexDesc, token_ids: torch.Tensor, doc_first: torch.Tensor, seq_len,
                              sep_ids, index: torch.Tensor):
    """Index of rows that pack several documents (doc_first [B][L] int32, non-zero where a document
    begins; seq_len [B] int32 or None)."""
    arr, p, n = _sep_array(sep_ids)
    assert n == desc.n_sep
    _check(lib().sepllm_build_index_packed(C.byref(desc), _ptr(token_ids), _ptr(doc_first), _ptr(seq_len), p,
                                           _ptr(index), _ptr(None), _stream()), "sepllm_build_index_packed")


def sepllm_build_index_static(desc: IndexDesc, token_ids: torch.Tensor, sep_ids, index: torch.Tensor):
    """Index build for callers that cannot allocate a scratch buffer: the library's own fixed
    array is used instead (B * (2 * ceil(L/4096) + 1) <= 65536).  Calls that may overlap on the GPU must be
    serialised by the caller; make the first call on a device outside any stream capture."""
    arr, p, n = _sep_array(sep_ids)
    assert n == desc.n_sep
    _check(lib().sepllm_build_index_static(C.byref(desc), _ptr(token_ids), p, _ptr(index), _stream()),
           "sepllm_build_index_static")


def sepllm_build_index_fixed_interval(desc: IndexDesc, interval: int, index: torch.Tensor,
                                      scratch: torch.Tensor):
    _check(lib().sepllm_build_index_fixed_interval(C.byref(desc), C.c_int32(interval), _ptr(index),
                                                   _ptr(scratch), _stream()),
           "sepllm_build_index_fixed_interval")


def read_index(index: torch.Tensor) -> dict:
    """Copies an index blob to the host and splits it into its arrays (for tests)."""
    raw = index.cpu().numpy().tobytes()
    h = IndexHeader.from_buffer_copy(raw[:256])
    d = h.desc
    T = h.n_tiles

    def arr(off, count):
        return np.frombuffer(raw, dtype=np.int32, count=count, offset=off).copy()

    return dict(
        header=h,
        cnt=arr(h.off_cnt, d.B * (d.L + 1)).reshape(d.B, d.L + 1),
        lim=arr(h.off_lim, d.B * d.L).reshape(d.B, d.L),
        side_pos=arr(h.off_side_pos, d.B * d.side_cap).reshape(d.B, d.side_cap),
        n_side=arr(h.off_n_side, d.B),
        tile_meta=arr(h.off_tile_meta, d.B * T * 8).reshape(d.B, T, 8),
        seq_len=arr(h.off_seq_len, d.B),
        doc_start=arr(h.off_doc_start, d.B * d.L).reshape(d.B, d.L),
        doc_end=arr(h.off_doc_end, d.B * d.L).reshape(d.B, d.L),
    )


# ---------------------------------------------------------------- attention
def sepllm_attn_workspace_bytes(desc: AttnDesc, idesc: IndexDesc):
    f, b = C.c_size_t(0), C.c_size_t(0)
    _check(lib().sepllm_attn_workspace_bytes(C.byref(desc), C.byref(idesc), C.byref(f), C.byref(b)),
           "sepllm_attn_workspace_bytes")
    return f.value, b.value


def sepllm_attn_fwd(desc, idesc, Q, K, V, index, O, LSE, workspace):
    _check(lib().sepllm_attn_fwd(C.byref(desc), C.byref(idesc), _ptr(Q), _ptr(K), _ptr(V), _ptr(index),
                                 _ptr(O), _ptr(LSE), _ptr(workspace), _stream()), "sepllm_attn_fwd")


def sepllm_attn_bwd(desc, idesc, dO, Q, K, V, O, LSE, index, dQ, dK, dV, workspace):
    _check(lib().sepllm_attn_bwd(C.byref(desc), C.byref(idesc), _ptr(dO), _ptr(Q), _ptr(K), _ptr(V),
                                 _ptr(O), _ptr(LSE), _ptr(index), _ptr(dQ), _ptr(dK), _ptr(dV),
                                 _ptr(workspace), _stream()), "sepllm_attn_bwd")


# ---------------------------------------------------------------- cache
def sepllm_cache_bytes(desc: CacheDesc):
    s, k = C.c_size_t(0), C.c_size_t(0)
    _check(lib().sepllm_cache_bytes(C.byref(desc), C.byref(s), C.byref(k)), "sepllm_cache_bytes")
    return s.value, k.value


def sepllm_cache_init(desc, state):
    _check(lib().sepllm_cache_init(C.byref(desc), _ptr(state), _stream()), "sepllm_cache_init")


def sepllm_cache_update(desc, state, Kc, Vc, new_token_ids, sep_ids, k_new, v_new):
    arr, p, n = _sep_array(sep_ids)
    _check(lib().sepllm_cache_update(C.byref(desc), _ptr(state), _ptr(Kc), _ptr(Vc),
                                     _ptr(new_token_ids), p, C.c_int32(n), _ptr(k_new), _ptr(v_new),
                                     _stream()), "sepllm_cache_update")


def sepllm_cache_from_prompt(desc, idesc, index, prompt_len, K, V, state, Kc, Vc, Kr=None, rope_table=None):
    _check(lib().sepllm_cache_from_prompt(C.byref(desc), C.byref(idesc), _ptr(index), _ptr(prompt_len),
                                          _ptr(K), _ptr(V), _ptr(state), _ptr(Kc), _ptr(Vc), _ptr(Kr),
                                          _ptr(rope_table), _stream()),
           "sepllm_cache_from_prompt")


def sepllm_decode_workspace_bytes(desc):
    b = C.c_size_t(0)
    _check(lib().sepllm_decode_workspace_bytes(C.byref(desc), C.byref(b)), "sepllm_decode_workspace_bytes")
    return b.value


def sepllm_decode(desc, scale, q, state, Kc, Vc, o, lse, workspace):
    _check(lib().sepllm_decode(C.byref(desc), C.c_float(scale), _ptr(q), _ptr(state), _ptr(Kc), _ptr(Vc),
                               _ptr(o), _ptr(lse), _ptr(workspace), _stream()), "sepllm_decode")


def sepllm_rope_table_bytes(desc):
    b = C.c_size_t(0)
    _check(lib().sepllm_rope_table_bytes(C.byref(desc), C.byref(b)), "sepllm_rope_table_bytes")
    return b.value


def sepllm_rope_table_build(desc, rope_base, table):
    _check(lib().sepllm_rope_table_build(C.byref(desc), C.c_float(rope_base), _ptr(table), _stream()),
           "sepllm_rope_table_build")


def sepllm_cache_update_rope(desc, state, Kc, Vc, Kr, rope_table, new_token_ids, sep_ids, k_new, v_new):
    arr, p, n = _sep_array(sep_ids)
    _check(lib().sepllm_cache_update_rope(C.byref(desc), _ptr(state), _ptr(Kc), _ptr(Vc), _ptr(Kr),
                                          _ptr(rope_table), _ptr(new_token_ids), p, C.c_int32(n),
                                          _ptr(k_new), _ptr(v_new), _stream()), "sepllm_cache_update_rope")


def sepllm_decode_rope(desc, scale, q, state, Kr, Vc, rope_table, o, lse, workspace):
    _check(lib().sepllm_decode_rope(C.byref(desc), C.c_float(scale), _ptr(q), _ptr(state), _ptr(Kr),
                                    _ptr(Vc), _ptr(rope_table), _ptr(o), _ptr(lse), _ptr(workspace),
                                    _stream()), "sepllm_decode_rope")


def read_cache_state(state: torch.Tensor) -> dict:
    """Copies a cache state to the host: per-sequence records and slot metadata (for tests)."""
    raw = state.cpu().numpy().tobytes()
    h = CacheHeader.from_buffer_copy(raw[:256])
    B, slots = h.desc.B, h.slots
    seq = np.frombuffer(raw, dtype=np.int32, count=B * 16, offset=h.off_seq).reshape(B, 16).copy()
    next_pos = np.frombuffer(raw, dtype=np.int64, count=B * 8, offset=h.off_seq).reshape(B, 8)[:, 3].copy()
    pos = np.frombuffer(raw, dtype=np.int64, count=B * slots, offset=h.off_slot_pos).reshape(B, slots).copy()
    flag = np.frombuffer(raw, dtype=np.uint8, count=B * slots, offset=h.off_slot_is_sep).reshape(B, slots).copy()
    return dict(header=h, size_init=seq[:, 0], sep_start=seq[:, 1], size_sep=seq[:, 2],
                win_start=seq[:, 3], size_win=seq[:, 4], compactions=seq[:, 5], next_pos=next_pos,
                slot_pos=pos, slot_is_sep=flag)


def sepllm_last_device_status(buffer) -> int:
    out = C.c_int32(0)
    _check(lib().sepllm_last_device_status(_ptr(buffer), C.byref(out), _stream()),
           "sepllm_last_device_status")
    return out.value


# ---------------------------------------------------------------- allocation helpers (torch = memory only)
def alloc_bytes(n: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned uint8 device buffer of at least n bytes."""
    t = torch.empty(n + 256, dtype=torch.uint8, device=device)
    off = (-t.data_ptr()) % 256
    return t[off:off + n]
