"""Thin ctypes binding of the MASW C ABI (include/masw.h): argument marshalling only.

PyTorch is used for device memory and streams; every step of the path runs in the library's CUDA
kernels.  There is no fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmasw.so")

MASW_OK, MASW_EINVAL, MASW_EALIGN, MASW_ECAPACITY, MASW_ESTATE, MASW_ECUDA = 0, -1, -2, -3, -4, -5
STATUS_SLOT_OVERFLOW, STATUS_WAIT_TIMEOUT, STATUS_BAD_LOGIT, STATUS_BAD_TOKEN = 1, 2, 4, 8
REGION_SINK, REGION_SLOT, REGION_LOCAL = 0, 1, 2
KV_DETERMINISTIC = 1
KV_STABLE = 2

EXPORTED_SYMBOLS = [
    "masw_sizes", "mem_init", "mem_free", "mem_load", "mem_set_state", "mem_get_state", "mem_update",
    "mem_advance", "mem_advance_deferred", "mem_flush", "mem_rollback", "draft_attend", "draft_append_attend", "draft_boundary_attend", "draft_prefill_slots",
    "draft_prefill_attend", "verify_workspace_bytes", "verify_attend", "verify_paged_workspace_bytes", "verify_attend_paged",
    "verify_fp8_workspace_bytes", "verify_attend_fp8",
    "accept_workspace_bytes", "accept_reject", "accept_reject_static", "masw_last_error", "masw_launch_count", "masw_version",
]


class MaswError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"masw error {code}: {text}")
        self.code = code


class masw_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "batch", "n_q_heads", "n_kv_heads", "head_dim", "d_model", "sink", "window",
        "slot_interval", "rollback", "max_slots", "gamma_max")] + [("softmax_scale", C.c_float), ("rope_base", C.c_float)]


class masw_kv_desc(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("stride_b", C.c_int64), ("stride_h", C.c_int64),
                ("stride_n", C.c_int64), ("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("capacity", C.c_int32), ("kv_len", C.c_void_p), ("softmax_scale", C.c_float),
                ("flags", C.c_int32), ("status", C.c_void_p), ("next_k", C.c_void_p), ("next_v", C.c_void_p)]


_lib = None


def load() -> C.CDLL:
    """Load libmasw.so (built in-tree by paper_2608_30252_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        _lib = _open(LIB_PATH)
    return _lib


def _open(path) -> C.CDLL:
    if not os.path.exists(path):
        raise FileNotFoundError(
            f"{path} not found: build it with `python -m paper_2608_30252_b200.build` "
            "(there is no CPU fallback)")
    lib = C.CDLL(path)
    vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
    lib.masw_sizes.argtypes = [C.POINTER(masw_config), C.POINTER(sz), C.POINTER(sz)]
    lib.mem_init.argtypes = [C.POINTER(masw_config), vp, sz, vp, sz, vp, C.POINTER(vp)]
    lib.mem_free.argtypes = [vp]
    lib.mem_free.restype = None
    lib.mem_load.argtypes = [vp, i32, i32, vp, vp, i32, i32, C.POINTER(C.c_int64), vp]
    lib.mem_set_state.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32), vp]
    lib.mem_get_state.argtypes = [vp, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32), vp]
    lib.mem_update.argtypes = [vp, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp]
    lib.mem_advance.argtypes = [vp, i32, i32, vp, vp]
    lib.mem_advance_deferred.argtypes = [vp, i32, i32]
    lib.mem_flush.argtypes = [vp, vp]
    lib.mem_rollback.argtypes = [vp, vp, vp, i32, vp]
    lib.draft_attend.argtypes = [vp, i32, vp, i32, i32, vp, vp, vp, vp]
    lib.draft_append_attend.argtypes = [vp, i32, vp, vp, vp, i32, i32, vp, vp, vp, vp]
    lib.draft_boundary_attend.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp]
    lib.draft_prefill_slots.argtypes = [C.POINTER(masw_config), i32]
    lib.verify_workspace_bytes.argtypes = [C.POINTER(masw_kv_desc), i32]
    lib.verify_workspace_bytes.restype = sz
    lib.verify_attend.argtypes = [C.POINTER(masw_kv_desc), vp, i32, vp, vp, vp, vp, sz, vp]
    lib.accept_workspace_bytes.argtypes = [i32, i32, i32]
    lib.accept_workspace_bytes.restype = sz
    lib.accept_reject.argtypes = [vp, vp, vp, vp, i32, i32, i32, C.c_float, vp, vp, vp, vp, sz, vp]
    lib.accept_reject_static.argtypes = [vp, vp, vp, vp, i32, i32, i32, C.c_float, vp, vp, vp, vp]
    lib.accept_reject_static.restype = C.c_int
    lib.masw_last_error.restype = C.c_char_p
    lib.masw_launch_count.restype = C.c_uint64
    lib.masw_version.restype = C.c_char_p
    for name in ("masw_sizes", "mem_init", "mem_load", "mem_set_state", "mem_get_state", "mem_update", "mem_advance",
                 "mem_advance_deferred", "mem_flush",
                 "mem_rollback", "draft_attend", "draft_append_attend", "draft_boundary_attend", "verify_attend", "accept_reject"):
        getattr(lib, name).restype = C.c_int
    return lib


def _check(rc: int) -> None:
    if rc != MASW_OK:
        raise MaswError(rc, load().masw_last_error().decode())


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def launch_count() -> int:
    return int(load().masw_launch_count())


def version() -> str:
    return load().masw_version().decode()


@dataclasses.dataclass
class MaswConfig:
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_model: int
    sink: int
    window: int
    slot_interval: int
    rollback: int = 16
    max_slots: int = 0
    gamma_max: int = 8
    softmax_scale: float = 0.0
    rope_base: float = 0.0

    def to_c(self) -> masw_config:
        return masw_config(*[getattr(self, f.name) for f in dataclasses.fields(self)])


def masw_sizes(cfg: MaswConfig):
    """(kv_arena_bytes, workspace_bytes); host only."""
    a, w = C.c_size_t(0), C.c_size_t(0)
    c = cfg.to_c()
    _check(load().masw_sizes(C.byref(c), C.byref(a), C.byref(w)))
    return a.value, w.value


class DraftMemory:
    """Owns the device buffers (torch) and the library handle of one draft memory."""

    def __init__(self, cfg: MaswConfig, device="cuda", lib=None):
        self.cfg = cfg
        self.lib = lib or load()
        self.device = torch.device(device)
        arena_bytes, ws_bytes = masw_sizes(cfg)
        self.arena = torch.empty(arena_bytes, dtype=torch.uint8, device=self.device)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)
        handle = C.c_void_p()
        c = cfg.to_c()
        _check(self.lib.mem_init(C.byref(c), _ptr(self.arena), arena_bytes, _ptr(self.workspace), ws_bytes,
                                 _stream(), C.byref(handle)))
        self.handle = handle

    def close(self):
        if getattr(self, "handle", None):
            self.lib.mem_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def kv_view(self, layer):
        """(K, V) views of one layer of the arena: bf16 [B, Hkv, entries, D]; entries are laid out
        [0, S) sink | [S, S + max_slots) slots | ring."""
        c = self.cfg
        ring = (c.window + c.rollback + c.gamma_max + 63) // 64 * 64
        n_cap = c.sink + c.max_slots + ring
        per = c.batch * c.n_kv_heads * n_cap * c.head_dim
        flat = self.arena.view(torch.bfloat16)
        shape = (c.batch, c.n_kv_heads, n_cap, c.head_dim)
        return flat[2 * layer * per:(2 * layer + 1) * per].view(shape), flat[(2 * layer + 1) * per:(2 * layer + 2) * per].view(shape)

    # ---- entry points, same names as the C ABI
    def mem_load(self, layer, region, k, v, first=0):
        """k, v: bf16 [B, n, Hkv, D] (any strides over the first three dims, D contiguous)."""
        assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.stride(-1) == 1 and v.stride() == k.stride()
        strides = (C.c_int64 * 3)(k.stride(0), k.stride(1), k.stride(2))
        _check(self.lib.mem_load(self.handle, layer, region, _ptr(k), _ptr(v), first, k.shape[1], strides, _stream()))

    def mem_set_state(self, t=None, n_slots=None):
        B = self.cfg.batch
        ta = (C.c_int32 * B)(*[int(x) for x in t]) if t is not None else None
        sa = (C.c_int32 * B)(*[int(x) for x in n_slots]) if n_slots is not None else None
        _check(self.lib.mem_set_state(self.handle, ta, sa, _stream()))

    def mem_get_state(self):
        B = self.cfg.batch
        ta, sa, st = (C.c_int32 * B)(), (C.c_int32 * B)(), C.c_int32(0)
        _check(self.lib.mem_get_state(self.handle, ta, sa, C.byref(st), _stream()))
        return list(ta), list(sa), st.value

    def mem_update(self, layer, k_raw=None, v_raw=None, h_g=None, Wk_g=None, Wv_g=None, slot_pos=None, active=None):
        n_raw = 0 if k_raw is None else k_raw.shape[1]
        for x in (k_raw, v_raw, h_g, Wk_g, Wv_g):
            assert x is None or (x.dtype == torch.bfloat16 and x.is_contiguous())
        assert slot_pos is None or slot_pos.dtype == torch.int32
        assert active is None or active.dtype == torch.uint8
        _check(self.lib.mem_update(self.handle, layer, _ptr(k_raw), _ptr(v_raw), n_raw, _ptr(h_g), _ptr(Wk_g),
                                   _ptr(Wv_g), _ptr(slot_pos), _ptr(active), _stream()))

    def mem_advance(self, n_tokens, add_slot=False, active=None, deferred=False):
        if deferred:
            assert active is None, "a deferred counter update applies to all sequences"
            _check(self.lib.mem_advance_deferred(self.handle, n_tokens, 1 if add_slot else 0))
        else:
            _check(self.lib.mem_advance(self.handle, n_tokens, 1 if add_slot else 0, _ptr(active), _stream()))

    def mem_flush(self):
        _check(self.lib.mem_flush(self.handle, _stream()))

    def mem_rollback(self, t_keep, slots_keep, slots_keep_max=-1):
        assert t_keep.dtype == torch.int32 and slots_keep.dtype == torch.int32
        _check(self.lib.mem_rollback(self.handle, _ptr(t_keep), _ptr(slots_keep), slots_keep_max, _stream()))

    def draft_attend(self, layer, q, last_row_is_slot=False, out=None, lse=None, out_bf16=None):
        """q: bf16 [B, n_q, Hq, D] -> (o fp32 [B, n_q, Hq, D], lse fp32 [B, n_q, Hq])."""
        assert q.dtype == torch.bfloat16 and q.is_contiguous()
        B, n_q, Hq, D = q.shape
        if out is None:
            out = torch.empty((B, n_q, Hq, D), dtype=torch.float32, device=q.device)
        if lse is None:
            lse = torch.empty((B, n_q, Hq), dtype=torch.float32, device=q.device)
        _check(self.lib.draft_attend(self.handle, layer, _ptr(q), n_q, 1 if last_row_is_slot else 0, _ptr(out),
                                     _ptr(lse), _ptr(out_bf16), _stream()))
        return out, lse


def _draft_append_attend(self, layer, k_raw, v_raw, q, last_row_is_slot=False, out=None, lse=None, out_bf16=None):
    """Raw-token append fused with the attention: k_raw, v_raw bf16 [B, n_raw, Hkv, D]; q as in draft_attend."""
    assert q.dtype == torch.bfloat16 and q.is_contiguous()
    assert k_raw.dtype == torch.bfloat16 and k_raw.is_contiguous() and v_raw.dtype == torch.bfloat16 and v_raw.is_contiguous()
    B, n_q, Hq, D = q.shape
    assert k_raw.shape[1] == n_q - (1 if last_row_is_slot else 0)
    if out is None:
        out = torch.empty((B, n_q, Hq, D), dtype=torch.float32, device=q.device)
    if lse is None:
        lse = torch.empty((B, n_q, Hq), dtype=torch.float32, device=q.device)
    _check(self.lib.draft_append_attend(self.handle, layer, _ptr(k_raw), _ptr(v_raw), _ptr(q), n_q,
                                        1 if last_row_is_slot else 0, _ptr(out), _ptr(lse), _ptr(out_bf16), _stream()))
    return out, lse


DraftMemory.draft_append_attend = _draft_append_attend


def _draft_boundary_attend(self, layer, k_raw, v_raw, h_g, Wk_g, Wv_g, slot_pos, q, active=None, out=None, lse=None,
                           out_bf16=None):
    """Boundary step in one launch: raw append + slot materialisation + attention (last row of q = slot row)."""
    for x in (k_raw, v_raw, h_g, Wk_g, Wv_g, q):
        assert x.dtype == torch.bfloat16 and x.is_contiguous()
    assert slot_pos.dtype == torch.int32 and (active is None or active.dtype == torch.uint8)
    B, n_q, Hq, D = q.shape
    assert k_raw.shape[1] == n_q - 1
    if out is None:
        out = torch.empty((B, n_q, Hq, D), dtype=torch.float32, device=q.device)
    if lse is None:
        lse = torch.empty((B, n_q, Hq), dtype=torch.float32, device=q.device)
    _check(self.lib.draft_boundary_attend(self.handle, layer, _ptr(k_raw), _ptr(v_raw), _ptr(h_g), _ptr(Wk_g), _ptr(Wv_g),
                                          _ptr(slot_pos), _ptr(active), _ptr(q), n_q, _ptr(out), _ptr(lse),
                                          _ptr(out_bf16), _stream()))
    return out, lse


DraftMemory.draft_boundary_attend = _draft_boundary_attend


def _draft_prefill_slots(self, P) -> int:
    """Slots created while P prefix tokens are processed."""
    c = self.cfg.to_c()
    return int(self.lib.draft_prefill_slots(C.byref(c), P))


def _draft_prefill_attend(self, layer, k, v, q, P, out=None, lse=None, out_bf16=None, import_memory=False,
                          want_fp32=True):
    """Masked prefill pass of one layer.  k, v: bf16 [B, Hkv, P + M, D] views (raw tokens, then the M slot
    tokens); q bf16 [B, P + M, Hq, D].  Returns (o fp32 or None, lse fp32, o_bf16 or None)."""
    assert q.dtype == torch.bfloat16 and q.is_contiguous()
    B, R, Hq, D = q.shape
    M = self.draft_prefill_slots(P)
    assert R == P + M and k.shape[2] >= R
    kv_len = torch.zeros(B, dtype=torch.int32, device=q.device)   # not read by the prefill pass
    desc = _kv_desc(k, v, kv_len, Hq)
    if out is None and want_fp32:
        out = torch.empty((B, R, Hq, D), dtype=torch.float32, device=q.device)
    if lse is None:
        lse = torch.empty((B, R, Hq), dtype=torch.float32, device=q.device)
    self.lib.draft_prefill_attend.argtypes = [C.c_void_p, C.c_int, C.POINTER(masw_kv_desc), C.c_void_p, C.c_int,
                                              C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
    _check(self.lib.draft_prefill_attend(self.handle, layer, C.byref(desc), _ptr(q), P, _ptr(out), _ptr(lse),
                                         _ptr(out_bf16), 1 if import_memory else 0, _stream()))
    return out, lse, out_bf16


DraftMemory.draft_prefill_slots = _draft_prefill_slots
DraftMemory.draft_prefill_attend = _draft_prefill_attend


def _kv_desc(k, v, kv_len, n_q_heads, softmax_scale=0.0, flags=0, status=None, next_kv=None) -> masw_kv_desc:
    assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.stride() == v.stride() and k.stride(-1) == 1
    assert kv_len.dtype == torch.int32 and (status is None or status.dtype == torch.int32)
    B, Hkv, cap, D = k.shape
    return masw_kv_desc(k.data_ptr(), v.data_ptr(), k.stride(0), k.stride(1), k.stride(2), B, n_q_heads, Hkv, D, cap,
                        kv_len.data_ptr(), softmax_scale, flags, None if status is None else status.data_ptr(),
                        None if next_kv is None else next_kv[0].data_ptr(), None if next_kv is None else next_kv[1].data_ptr())


def verify_workspace(k, kv_len, n_q_heads, T) -> torch.Tensor:
    """Zero-filled scratch for verify_attend on this cache geometry."""
    desc = _kv_desc(k, k, kv_len, n_q_heads)
    n = load().verify_workspace_bytes(C.byref(desc), T)
    return torch.zeros(n, dtype=torch.uint8, device=k.device)


def verify_attend(k, v, kv_len, q, workspace=None, out=None, lse=None, out_bf16=None, softmax_scale=0.0,
                  deterministic=False, stable_cache=False, status=None, next_kv=None, lib=None):
    """k, v: bf16 [B, Hkv, cap, D] views; kv_len int32 [B] (including the T rows); q bf16 [B, T, Hq, D].
    deterministic: static tile schedule (bitwise repeatable); stable_cache: the preceding kernel in the stream writes
    nothing of k and v (first tiles requested ahead of the wait); status: int32 [1] device tensor for MASW_STATUS_* bits;
    next_kv: (k, v) of the cache the next call will read (same geometry), an L2 hint for that call's first tiles."""
    assert q.dtype == torch.bfloat16 and q.is_contiguous()
    B, T, Hq, D = q.shape
    desc = _kv_desc(k, v, kv_len, Hq, softmax_scale,
                    (KV_DETERMINISTIC if deterministic else 0) | (KV_STABLE if stable_cache else 0), status, next_kv)
    if workspace is None:
        workspace = verify_workspace(k, kv_len, Hq, T)
    if out is None:
        out = torch.empty((B, T, Hq, D), dtype=torch.float32, device=q.device)
    if lse is None:
        lse = torch.empty((B, T, Hq), dtype=torch.float32, device=q.device)
    _check((lib or load()).verify_attend(C.byref(desc), _ptr(q), T, _ptr(out), _ptr(lse), _ptr(out_bf16), _ptr(workspace),
                                         workspace.numel(), _stream()))
    return out, lse


class masw_paged_kv_desc(C.Structure):
    _fields_ = [("k_pages", C.c_void_p), ("v_pages", C.c_void_p), ("page_table", C.c_void_p), ("n_pages", C.c_int32),
                ("max_pages", C.c_int32), ("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("kv_len", C.c_void_p), ("softmax_scale", C.c_float), ("flags", C.c_int32),
                ("status", C.c_void_p)]


def verify_attend_paged(k_pages, v_pages, page_table, kv_len, q, workspace=None, out=None, lse=None, out_bf16=None,
                        softmax_scale=0.0, deterministic=False, status=None):
    """k_pages, v_pages: bf16 [n_pages, Hkv, 128, D] contiguous; page_table int32 [B, max_pages]; kv_len int32 [B]
    (including the T rows); q bf16 [B, T, Hq, D].  Returns (o fp32, lse fp32, workspace)."""
    assert k_pages.dtype == torch.bfloat16 and k_pages.is_contiguous() and v_pages.is_contiguous() and k_pages.shape == v_pages.shape
    assert page_table.dtype == torch.int32 and page_table.is_contiguous() and kv_len.dtype == torch.int32
    assert q.dtype == torch.bfloat16 and q.is_contiguous()
    n_pages, Hkv, page, D = k_pages.shape
    assert page == 128
    B, T, Hq, _ = q.shape
    desc = masw_paged_kv_desc(k_pages.data_ptr(), v_pages.data_ptr(), page_table.data_ptr(), n_pages, page_table.shape[1], B, Hq,
                              Hkv, D, kv_len.data_ptr(), softmax_scale, KV_DETERMINISTIC if deterministic else 0,
                              None if status is None else status.data_ptr())
    lib = load()
    lib.verify_paged_workspace_bytes.argtypes = [C.POINTER(masw_paged_kv_desc), C.c_int]
    lib.verify_paged_workspace_bytes.restype = C.c_size_t
    lib.verify_attend_paged.argtypes = [C.POINTER(masw_paged_kv_desc), C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_size_t, C.c_void_p]
    if workspace is None:
        workspace = torch.zeros(lib.verify_paged_workspace_bytes(C.byref(desc), T), dtype=torch.uint8, device=q.device)
    if out is None:
        out = torch.empty((B, T, Hq, D), dtype=torch.float32, device=q.device)
    if lse is None:
        lse = torch.empty((B, T, Hq), dtype=torch.float32, device=q.device)
    _check(lib.verify_attend_paged(C.byref(desc), _ptr(q), T, _ptr(out), _ptr(lse), _ptr(out_bf16), _ptr(workspace),
                                   workspace.numel(), _stream()))
    return out, lse, workspace


class masw_fp8_kv_desc(C.Structure):
    _fields_ = [("k_pages", C.c_void_p), ("v_pages", C.c_void_p), ("k_scale", C.c_void_p), ("v_scale", C.c_void_p),
                ("page_table", C.c_void_p), ("n_pages", C.c_int32), ("max_pages", C.c_int32), ("batch", C.c_int32),
                ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("kv_len", C.c_void_p),
                ("softmax_scale", C.c_float), ("flags", C.c_int32), ("status", C.c_void_p)]


def verify_attend_fp8(k_pages, v_pages, k_scale, v_scale, page_table, kv_len, q, workspace=None, out=None, lse=None,
                      out_bf16=None, softmax_scale=0.0, deterministic=False, status=None):
    """k_pages, v_pages: uint8 (e4m3 bytes) [n_pages, Hkv, 128, 128] contiguous; k_scale, v_scale fp32 [n_pages, Hkv];
    page_table int32 [B, max_pages]; kv_len int32 [B] (including the T rows); q bf16 [B, T, Hq, 128].
    Returns (o fp32, lse fp32, workspace)."""
    assert k_pages.dtype == torch.uint8 and v_pages.dtype == torch.uint8 and k_pages.is_contiguous() and v_pages.is_contiguous()
    assert k_pages.shape == v_pages.shape and k_scale.dtype == torch.float32 and v_scale.dtype == torch.float32
    assert k_scale.is_contiguous() and v_scale.is_contiguous()
    assert page_table.dtype == torch.int32 and page_table.is_contiguous() and kv_len.dtype == torch.int32
    assert q.dtype == torch.bfloat16 and q.is_contiguous()
    n_pages, Hkv, page, D = k_pages.shape
    assert page == 128 and D == 128 and tuple(k_scale.shape) == (n_pages, Hkv) == tuple(v_scale.shape)
    B, T, Hq, _ = q.shape
    desc = masw_fp8_kv_desc(k_pages.data_ptr(), v_pages.data_ptr(), k_scale.data_ptr(), v_scale.data_ptr(),
                            page_table.data_ptr(), n_pages, page_table.shape[1], B, Hq, Hkv, D, kv_len.data_ptr(),
                            softmax_scale, KV_DETERMINISTIC if deterministic else 0,
                            None if status is None else status.data_ptr())
    lib = load()
    lib.verify_fp8_workspace_bytes.argtypes = [C.POINTER(masw_fp8_kv_desc), C.c_int]
    lib.verify_fp8_workspace_bytes.restype = C.c_size_t
    lib.verify_attend_fp8.argtypes = [C.POINTER(masw_fp8_kv_desc), C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_size_t, C.c_void_p]
    lib.verify_attend_fp8.restype = C.c_int
    if workspace is None:
        workspace = torch.zeros(lib.verify_fp8_workspace_bytes(C.byref(desc), T), dtype=torch.uint8, device=q.device)
    if out is None:
        out = torch.empty((B, T, Hq, D), dtype=torch.float32, device=q.device)
    if lse is None:
        lse = torch.empty((B, T, Hq), dtype=torch.float32, device=q.device)
    _check(lib.verify_attend_fp8(C.byref(desc), _ptr(q), T, _ptr(out), _ptr(lse), _ptr(out_bf16), _ptr(workspace),
                                 workspace.numel(), _stream()))
    return out, lse, workspace


def accept_workspace(batch, gamma, vocab, device="cuda") -> torch.Tensor:
    n = load().accept_workspace_bytes(batch, gamma, vocab)
    return torch.zeros(n, dtype=torch.uint8, device=device)


def accept_reject(target_logits, draft_logits, draft_tokens, uniforms, temperature=0.0, workspace=None,
                  n_accepted=None, out_tokens=None, status=None):
    """target_logits bf16 [B, gamma+1, V]; draft_logits bf16 [B, gamma, V] or None; draft_tokens int32
    [B, gamma]; uniforms fp32 [B, gamma+1] or None.  Returns (n_accepted int32 [B], out_tokens int32 [B, gamma+1])."""
    assert target_logits.dtype == torch.bfloat16 and target_logits.is_contiguous()
    assert draft_logits is None or (draft_logits.dtype == torch.bfloat16 and draft_logits.is_contiguous())
    assert draft_tokens.dtype == torch.int32 and draft_tokens.is_contiguous()
    assert uniforms is None or (uniforms.dtype == torch.float32 and uniforms.is_contiguous())
    B, g1, V = target_logits.shape
    gamma = g1 - 1
    dev = target_logits.device
    if workspace is None:
        workspace = accept_workspace(B, gamma, V, dev)
    if n_accepted is None:
        n_accepted = torch.empty(B, dtype=torch.int32, device=dev)
    if out_tokens is None:
        out_tokens = torch.empty((B, gamma + 1), dtype=torch.int32, device=dev)
    _check(load().accept_reject(_ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens), _ptr(uniforms), B, gamma,
                                V, float(temperature), _ptr(n_accepted), _ptr(out_tokens), _ptr(status),
                                _ptr(workspace), workspace.numel(), _stream()))
    return n_accepted, out_tokens


def accept_reject_static(target_logits, draft_logits, draft_tokens, uniforms, temperature=0.0, n_accepted=None,
                         out_tokens=None, status=None):
    """accept_reject without a workspace argument: the library keeps the scratch in a fixed device
    array of its own (batch <= 64, gamma <= 16), so nothing is allocated by the call itself when the
    output tensors are passed in.  Calls on one device share that array and must not overlap."""
    assert target_logits.dtype == torch.bfloat16 and target_logits.is_contiguous()
    assert draft_logits is None or (draft_logits.dtype == torch.bfloat16 and draft_logits.is_contiguous())
    assert draft_tokens.dtype == torch.int32 and draft_tokens.is_contiguous()
    assert uniforms is None or (uniforms.dtype == torch.float32 and uniforms.is_contiguous())
    B, g1, V = target_logits.shape
    gamma = g1 - 1
    dev = target_logits.device
    if n_accepted is None:
        n_accepted = torch.empty(B, dtype=torch.int32, device=dev)
    if out_tokens is None:
        out_tokens = torch.empty((B, gamma + 1), dtype=torch.int32, device=dev)
    _check(load().accept_reject_static(_ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens), _ptr(uniforms), B,
                                       gamma, V, float(temperature), _ptr(n_accepted), _ptr(out_tokens), _ptr(status),
                                       _stream()))
    return n_accepted, out_tokens


# ---- developer build (libmasw_trace.so, compiled with -DMASW_TRACE; never loaded by the product path) ----
TRACE_LIB_PATH = os.path.join(_HERE, "libmasw_trace.so")
_trace_lib = None


def load_trace() -> C.CDLL:
    """The developer build of the same sources: phase stamps in the attention kernels, a settable limit for
    their bounded waits and a switch that leaves one tile copy out.  Used by `bench.py --timeline` and by the
    test of the give-up path; it is a separate library, so the product library carries none of this."""
    global _trace_lib
    if _trace_lib is None:
        lib = _open(TRACE_LIB_PATH)
        lib.masw_debug_set_trace.argtypes = [C.c_void_p, C.c_longlong]
        lib.masw_debug_set_trace.restype = None
        lib.masw_debug_set_wait.argtypes = [C.c_int, C.c_int]
        lib.masw_debug_set_wait.restype = None
        lib.masw_debug_set_flags.argtypes = [C.c_int]
        lib.masw_debug_set_flags.restype = None
        _trace_lib = lib
    return _trace_lib


def select_trace_build() -> None:
    """Route every call of this module to the developer build (for `bench.py --timeline`; call it first)."""
    global _lib
    _lib = load_trace()


def debug_set_trace(buffer, stride_words=0) -> None:
    """Developer build: while `buffer` (an int64 CUDA tensor of at least 16 words per CTA of the next launches)
    is set, the attention kernels of libmasw_trace.so write a few %globaltimer stamps per CTA into it.  With
    stride_words > 0 every later launch writes `stride_words` further into the buffer (a chain of launches, also
    when captured into a CUDA graph, then keeps one record area per launch).  Pass None to switch the stamps off."""
    load_trace().masw_debug_set_trace(C.c_void_p(buffer.data_ptr()) if buffer is not None else None, int(stride_words))


def debug_set_wait(wait_limit=0, drop_tile=-1) -> None:
    """Developer build: polls after which the kernels' bounded waits give up (0 = the normal limit) and the
    CTA-local index of one tile whose copy is armed but never issued (-1 = none)."""
    load_trace().masw_debug_set_wait(int(wait_limit), int(drop_tile))


def debug_set_flags(flags=0) -> None:
    """Developer build, timing experiments on the draft kernel (results are then meaningless): 1 = no cross-split
    reduction, 2 = no tile arithmetic, 4 = never ahead of the predecessor."""
    load_trace().masw_debug_set_flags(int(flags))
