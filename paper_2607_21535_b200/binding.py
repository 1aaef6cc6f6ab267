"""ctypes binding of libwmtp.so: same names as the C ABI, argument marshalling only.

torch is used for device memory and streams; every step of the path runs in the
library's kernels. There is no fallback: a missing or unloadable library raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_float, c_int, c_int32, c_int64, c_size_t, c_void_p

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libwmtp.so")

WMTP_OK = 0
STATUS_NAMES = {
    0: "WMTP_OK", 1: "WMTP_ERR_INVALID_ARG", 2: "WMTP_ERR_UNSUPPORTED", 3: "WMTP_ERR_CAPACITY",
    4: "WMTP_ERR_WORKSPACE", 5: "WMTP_ERR_CUDA", 6: "WMTP_ERR_DEVICE_TIMEOUT", 7: "WMTP_ERR_DEVICE_BOUNDS",
}


class wmtp_ring(ctypes.Structure):
    _fields_ = [("k", c_void_p), ("v", c_void_p), ("slot_pos", c_void_p), ("len", c_void_p),
                ("batch", c_int32), ("Hkv", c_int32), ("D", c_int32), ("n_sink", c_int32), ("W", c_int32),
                ("cap", c_int32), ("kv_dtype", c_int32), ("k_scale", c_void_p), ("v_scale", c_void_p)]


class wmtp_kv(ctypes.Structure):
    _fields_ = [("k", c_void_p), ("v", c_void_p), ("page_table", c_void_p), ("len", c_void_p),
                ("S_cap", c_int64), ("batch", c_int32), ("Hkv", c_int32), ("D", c_int32), ("page_size", c_int32),
                ("max_pages", c_int32), ("num_pages", c_int32), ("kv_dtype", c_int32), ("k_scale", c_void_p),
                ("v_scale", c_void_p)]


WMTP_KV_BF16, WMTP_KV_FP8_E4M3 = 0, 1


class WmtpError(RuntimeError):
    def __init__(self, status: int, detail: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {detail}")
        self.status = status


# Every symbol include/wmtp.h declares, with its ctypes signature.
_SIGNATURES = {
    "wmtp_status_string": (c_char_p, [c_int]),
    "wmtp_last_error": (c_char_p, []),
    "wmtp_kv_elem_bytes": (c_size_t, [c_int]),
    "wmtp_ring_bytes": (c_size_t, [c_int, c_int, c_int, c_int, c_int, POINTER(c_size_t)]),
    "wmtp_workspace_bytes": (c_size_t, [c_int, c_int, c_int, c_int]),
    "wmtp_workspace_init": (c_int, [c_void_p, c_size_t, c_void_p]),
    "wmtp_device_status": (c_int, [c_void_p, c_void_p]),
    "wmtp_ring_reset": (c_int, [POINTER(wmtp_ring), c_void_p]),
    "wmtp_ring_init_from_kv": (c_int, [POINTER(wmtp_ring), POINTER(wmtp_kv), c_void_p]),
    "wmtp_ring_state_bytes": (c_size_t, [POINTER(wmtp_ring)]),
    "wmtp_ring_export": (c_int, [POINTER(wmtp_ring), c_void_p, c_size_t, c_void_p]),
    "wmtp_ring_import": (c_int, [POINTER(wmtp_ring), c_void_p, c_size_t, c_void_p]),
    "wmtp_ring_append": (c_int, [POINTER(wmtp_ring), c_void_p, c_void_p, c_void_p]),
    "wmtp_kv_append": (c_int, [POINTER(wmtp_kv), c_void_p, c_void_p, c_void_p, c_void_p]),
    "wmtp_draft_attn_windowed": (c_int, [c_void_p, c_int, POINTER(wmtp_ring), c_float, c_void_p, c_void_p, c_void_p,
                                         c_size_t, c_void_p]),
    "wmtp_draft_attn_full": (c_int, [c_void_p, c_int, POINTER(wmtp_kv), c_float, c_void_p, c_void_p, c_void_p, c_size_t,
                                     c_void_p]),
    "wmtp_draft_loop_windowed": (c_int, [POINTER(wmtp_ring), c_int, c_void_p, c_int, c_void_p, c_void_p, c_float,
                                         c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "wmtp_draft_loop_full": (c_int, [POINTER(wmtp_kv), c_int, c_void_p, c_int, c_void_p, c_void_p, c_float, c_void_p,
                                     c_void_p, c_void_p, c_size_t, c_void_p]),
    "wmtp_stage_bytes": (c_size_t, [c_int, c_int, c_int, c_int, c_int]),
    "wmtp_draft_loop_windowed_host": (c_int, [POINTER(wmtp_ring), c_int, c_void_p, c_int, c_void_p, c_void_p, c_float,
                                              c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "wmtp_draft_loop_full_host": (c_int, [POINTER(wmtp_kv), c_int, c_void_p, c_int, c_void_p, c_void_p, c_float,
                                          c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "wmtp_draft_attn_windowed_noalloc": (c_int, [c_void_p, c_int, POINTER(wmtp_ring), c_float, c_void_p, c_void_p, c_void_p]),
    "wmtp_draft_attn_windowed_kv": (c_int, [c_void_p, c_int, POINTER(wmtp_kv), c_int, c_int, c_float, c_void_p, c_void_p,
                                            c_void_p, c_size_t, c_void_p]),
    "wmtp_draft_loop_windowed_kv": (c_int, [POINTER(wmtp_kv), c_int, c_int, c_int, c_void_p, c_int, c_void_p, c_void_p,
                                            c_float, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "wmtp_reduced_block_table_width": (c_int, [c_int, c_int, c_int]),
    "wmtp_reduced_block_table": (c_int, [POINTER(wmtp_kv), c_int, c_int, c_void_p, c_int, c_void_p, c_void_p, c_void_p]),
    "wmtp_full_token_index": (c_int, [POINTER(wmtp_kv), c_void_p, c_int64, c_void_p, c_void_p]),
    "wmtp_ring_rewind": (c_int, [POINTER(wmtp_ring), c_void_p, c_void_p, c_void_p]),
    "wmtp_ring_append_many": (c_int, [POINTER(wmtp_ring), c_int, c_void_p, c_void_p, c_void_p]),
    "wmtp_ring_replace_tail": (c_int, [POINTER(wmtp_ring), c_void_p, c_int, c_void_p, c_void_p, c_void_p, c_void_p]),
    "wmtp_kv_append_many": (c_int, [POINTER(wmtp_kv), c_int, c_void_p, c_void_p, c_void_p, c_void_p]),
    "wmtp_draft_extend_windowed": (c_int, [c_void_p, c_int, c_int, POINTER(wmtp_ring), c_float, c_void_p, c_void_p, c_void_p,
                                           c_size_t, c_void_p]),
    "wmtp_draft_extend_full": (c_int, [c_void_p, c_int, c_int, POINTER(wmtp_kv), c_float, c_void_p, c_void_p, c_void_p,
                                       c_size_t, c_void_p]),
    "wmtp_attn_mass_diagnostics": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_int, c_int, c_void_p, c_void_p, c_void_p,
                                           c_void_p]),
    "wmtp_set_max_ctas": (None, [c_int]),
    "wmtp_set_work_stealing": (None, [c_int]),
    "wmtp_set_wait_limit": (None, [c_int]),
    "wmtp_launch_count": (c_int64, []),
}

_lib = None


def lib() -> ctypes.CDLL:
    """Loads libwmtp.so (built in-tree by ``build.py``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2607_21535_b200.build` "
                              "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(status: int) -> None:
    if status != WMTP_OK:
        raise WmtpError(status, lib().wmtp_last_error().decode())


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


# ------------------------------------------------------------------------------------------------
# Device-memory holders (torch allocations + the C descriptor)
# ------------------------------------------------------------------------------------------------
class Ring:
    """Device ring-buffer KV store for ``batch`` sequences: n_sink sink slots + ``cap`` window slots.

    ``k_scale`` / ``v_scale`` (device fp32 [Hkv]) select an fp8 (e4m3) store: uint8 codes, value = code * scale.
    ``alloc(shape, dtype, device)`` returns the (uninitialised) device tensor for each of the four arrays; the default is
    ``torch.empty``. A caller with its own memory pool, or a test that wants guard bands around the arrays, passes one."""

    def __init__(self, batch, Hkv, D, n_sink, W, cap=None, device="cuda", k_scale=None, v_scale=None, alloc=None):
        cap = W if cap is None else cap
        self.batch, self.Hkv, self.D, self.n_sink, self.W, self.cap = batch, Hkv, D, n_sink, W, cap
        slots = n_sink + cap
        assert (k_scale is None) == (v_scale is None)
        f8 = k_scale is not None
        dt = torch.uint8 if f8 else torch.bfloat16
        self.k_scale, self.v_scale = k_scale, v_scale
        alloc = alloc or (lambda shape, dtype, device: torch.empty(shape, dtype=dtype, device=device))
        self.k = alloc((batch, Hkv, slots, D), dt, device).zero_()
        self.v = alloc((batch, Hkv, slots, D), dt, device).zero_()
        self.slot_pos = alloc((batch, slots), torch.int32, device).fill_(-1)
        self.len = alloc((batch,), torch.int64, device).zero_()
        self.desc = wmtp_ring(self.k.data_ptr(), self.v.data_ptr(), self.slot_pos.data_ptr(), self.len.data_ptr(),
                              batch, Hkv, D, n_sink, W, cap, WMTP_KV_FP8_E4M3 if f8 else WMTP_KV_BF16, _ptr(k_scale),
                              _ptr(v_scale))


class KV:
    """Full-context KV descriptor over caller-provided device tensors.

    Contiguous: k, v bf16 [batch][Hkv][S_cap][D]. Paged: k, v bf16 [num_pages][Hkv][page_size][D]
    with ``page_table`` int32 [batch][max_pages]. uint8 tensors are an fp8 (e4m3) store and need
    ``k_scale`` / ``v_scale`` (device fp32 [Hkv]).
    """

    def __init__(self, k, v, lens, page_table=None, S_cap=None, k_scale=None, v_scale=None):
        self.k, self.v, self.len, self.page_table = k, v, lens, page_table
        f8 = k.dtype == torch.uint8
        assert v.dtype == k.dtype and f8 == (k_scale is not None) == (v_scale is not None)
        self.k_scale, self.v_scale = k_scale, v_scale
        if page_table is None:
            batch, Hkv, rows, D = k.shape
            self.S_cap = rows if S_cap is None else S_cap
            page_size = max_pages = num_pages = 0
        else:
            num_pages, Hkv, page_size, D = k.shape
            batch, max_pages = page_table.shape
            self.S_cap = max_pages * page_size if S_cap is None else S_cap
        self.batch, self.Hkv, self.D = batch, Hkv, D
        self.desc = wmtp_kv(k.data_ptr(), v.data_ptr(), _ptr(page_table), lens.data_ptr(), self.S_cap, batch, Hkv, D,
                            page_size, max_pages, num_pages, WMTP_KV_FP8_E4M3 if f8 else WMTP_KV_BF16, _ptr(k_scale),
                            _ptr(v_scale))


class Workspace:
    def __init__(self, batch, Hq, Hkv, D, device="cuda", stream=None, alloc=None):
        self.nbytes = int(lib().wmtp_workspace_bytes(batch, Hq, Hkv, D))
        alloc = alloc or (lambda shape, dtype, device: torch.empty(shape, dtype=dtype, device=device))
        # 0xFF bytes are NaN as floats: a partial result read before it is written cannot go unnoticed
        self.buf = alloc((self.nbytes,), torch.uint8, device).fill_(0xFF)
        assert self.buf.data_ptr() % 256 == 0
        wmtp_workspace_init(self, stream=stream)

    @property
    def ptr(self) -> int:
        return self.buf.data_ptr()


# ------------------------------------------------------------------------------------------------
# The C ABI, same names
# ------------------------------------------------------------------------------------------------
def wmtp_status_string(status: int) -> str:
    return lib().wmtp_status_string(status).decode()


def wmtp_last_error() -> str:
    return lib().wmtp_last_error().decode()


def wmtp_kv_elem_bytes(kv_dtype: int) -> int:
    return int(lib().wmtp_kv_elem_bytes(kv_dtype))


def wmtp_ring_bytes(batch, Hkv, D, n_sink, cap):
    pos = c_size_t(0)
    kb = lib().wmtp_ring_bytes(batch, Hkv, D, n_sink, cap, byref(pos))
    return int(kb), int(pos.value)


def wmtp_workspace_bytes(batch, Hq, Hkv, D) -> int:
    return int(lib().wmtp_workspace_bytes(batch, Hq, Hkv, D))


def wmtp_workspace_init(ws: Workspace, stream=None) -> None:
    _check(lib().wmtp_workspace_init(ws.ptr, ws.nbytes, _stream(stream)))


def wmtp_device_status(ws: Workspace, stream=None) -> None:
    _check(lib().wmtp_device_status(ws.ptr, _stream(stream)))


def wmtp_ring_reset(ring: Ring, stream=None) -> None:
    _check(lib().wmtp_ring_reset(byref(ring.desc), _stream(stream)))


def wmtp_ring_state_bytes(ring: Ring) -> int:
    return int(lib().wmtp_ring_state_bytes(byref(ring.desc)))


def wmtp_ring_export(ring: Ring, blob, stream=None) -> None:
    """blob: uint8 tensor (device or pinned host) of at least wmtp_ring_state_bytes(ring) bytes."""
    _check(lib().wmtp_ring_export(byref(ring.desc), _ptr(blob), blob.numel() * blob.element_size(), _stream(stream)))


def wmtp_ring_import(ring: Ring, blob, stream=None) -> None:
    _check(lib().wmtp_ring_import(byref(ring.desc), _ptr(blob), blob.numel() * blob.element_size(), _stream(stream)))


def wmtp_ring_init_from_kv(ring: Ring, kv: KV, stream=None) -> None:
    _check(lib().wmtp_ring_init_from_kv(byref(ring.desc), byref(kv.desc), _stream(stream)))


def wmtp_ring_append(ring: Ring, k_new, v_new, stream=None) -> None:
    _check(lib().wmtp_ring_append(byref(ring.desc), _ptr(k_new), _ptr(v_new), _stream(stream)))


def wmtp_kv_append(kv: KV, k_new, v_new, ws: Workspace | None = None, stream=None) -> None:
    _check(lib().wmtp_kv_append(byref(kv.desc), _ptr(k_new), _ptr(v_new), ws.ptr if ws is not None else None,
                                _stream(stream)))


def wmtp_draft_attn_windowed(q, ring: Ring, out, ws: Workspace, lse=None, sm_scale: float = 0.0, stream=None) -> None:
    Hq = q.shape[-2]
    _check(lib().wmtp_draft_attn_windowed(_ptr(q), Hq, byref(ring.desc), sm_scale, _ptr(out), _ptr(lse), ws.ptr,
                                          ws.nbytes, _stream(stream)))


def wmtp_draft_attn_full(q, kv: KV, out, ws: Workspace, lse=None, sm_scale: float = 0.0, stream=None) -> None:
    Hq = q.shape[-2]
    _check(lib().wmtp_draft_attn_full(_ptr(q), Hq, byref(kv.desc), sm_scale, _ptr(out), _ptr(lse), ws.ptr, ws.nbytes,
                                      _stream(stream)))


def wmtp_draft_loop_windowed(ring: Ring, q, k_new, v_new, out, ws: Workspace, lse=None, sm_scale: float = 0.0,
                             stream=None) -> None:
    gamma, Hq = q.shape[0], q.shape[-2]
    _check(lib().wmtp_draft_loop_windowed(byref(ring.desc), gamma, _ptr(q), Hq, _ptr(k_new), _ptr(v_new), sm_scale,
                                          _ptr(out), _ptr(lse), ws.ptr, ws.nbytes, _stream(stream)))


def wmtp_draft_loop_full(kv: KV, q, k_new, v_new, out, ws: Workspace, lse=None, sm_scale: float = 0.0,
                         stream=None) -> None:
    gamma, Hq = q.shape[0], q.shape[-2]
    _check(lib().wmtp_draft_loop_full(byref(kv.desc), gamma, _ptr(q), Hq, _ptr(k_new), _ptr(v_new), sm_scale, _ptr(out),
                                      _ptr(lse), ws.ptr, ws.nbytes, _stream(stream)))


def wmtp_stage_bytes(gamma, batch, Hq, Hkv, D) -> int:
    return int(lib().wmtp_stage_bytes(gamma, batch, Hq, Hkv, D))


def wmtp_draft_loop_windowed_host(ring: Ring, q_host, k_new_host, v_new_host, out_host, stage, ws: Workspace,
                                  lse_host=None, sm_scale: float = 0.0, stream=None) -> None:
    """Host tensors in, host tensors out (CPU torch tensors, ideally pinned); ``stage`` is a device byte buffer."""
    gamma, Hq = q_host.shape[0], q_host.shape[-2]
    _check(lib().wmtp_draft_loop_windowed_host(byref(ring.desc), gamma, _ptr(q_host), Hq, _ptr(k_new_host),
                                               _ptr(v_new_host), sm_scale, _ptr(out_host), _ptr(lse_host), _ptr(stage),
                                               ws.ptr, ws.nbytes, _stream(stream)))


def wmtp_draft_loop_full_host(kv: KV, q_host, k_new_host, v_new_host, out_host, stage, ws: Workspace, lse_host=None,
                              sm_scale: float = 0.0, stream=None) -> None:
    gamma, Hq = q_host.shape[0], q_host.shape[-2]
    _check(lib().wmtp_draft_loop_full_host(byref(kv.desc), gamma, _ptr(q_host), Hq, _ptr(k_new_host), _ptr(v_new_host),
                                           sm_scale, _ptr(out_host), _ptr(lse_host), _ptr(stage), ws.ptr, ws.nbytes,
                                           _stream(stream)))


def wmtp_draft_attn_windowed_noalloc(q, ring: Ring, out, lse=None, sm_scale: float = 0.0, stream=None) -> None:
    """Windowed attention on the library's built-in scratch, for callers that cannot allocate a workspace
    (they do not own the device allocator, or may not allocate once running). Calls sharing a device must
    not overlap on the GPU; the first call on a device should be made outside stream capture."""
    Hq = q.shape[-2]
    _check(lib().wmtp_draft_attn_windowed_noalloc(_ptr(q), Hq, byref(ring.desc), sm_scale, _ptr(out), _ptr(lse),
                                                  _stream(stream)))


def wmtp_draft_attn_windowed_kv(q, kv: KV, n_sink: int, W: int, out, ws: Workspace, lse=None, sm_scale: float = 0.0,
                                stream=None) -> None:
    Hq = q.shape[-2]
    _check(lib().wmtp_draft_attn_windowed_kv(_ptr(q), Hq, byref(kv.desc), n_sink, W, sm_scale, _ptr(out), _ptr(lse), ws.ptr,
                                             ws.nbytes, _stream(stream)))


def wmtp_draft_loop_windowed_kv(kv: KV, n_sink: int, W: int, q, k_new, v_new, out, ws: Workspace, lse=None,
                                sm_scale: float = 0.0, stream=None) -> None:
    gamma, Hq = q.shape[0], q.shape[-2]
    _check(lib().wmtp_draft_loop_windowed_kv(byref(kv.desc), n_sink, W, gamma, _ptr(q), Hq, _ptr(k_new), _ptr(v_new),
                                             sm_scale, _ptr(out), _ptr(lse), ws.ptr, ws.nbytes, _stream(stream)))


def wmtp_ring_rewind(ring: Ring, n_drop, ws: Workspace | None = None, stream=None) -> None:
    _check(lib().wmtp_ring_rewind(byref(ring.desc), _ptr(n_drop), ws.ptr if ws is not None else None, _stream(stream)))


def wmtp_ring_append_many(ring: Ring, k_new, v_new, stream=None) -> None:
    """k_new, v_new: [batch][n_tok][Hkv][D]."""
    _check(lib().wmtp_ring_append_many(byref(ring.desc), k_new.shape[1], _ptr(k_new), _ptr(v_new), _stream(stream)))


def wmtp_ring_replace_tail(ring: Ring, n_drop, k_new, v_new, ws: Workspace | None = None, stream=None) -> None:
    """Drop the last n_drop[r] tokens (device int32 [batch] or None), then append k_new / v_new [batch][n_tok][Hkv][D]."""
    _check(lib().wmtp_ring_replace_tail(byref(ring.desc), _ptr(n_drop), k_new.shape[1], _ptr(k_new), _ptr(v_new),
                                        ws.ptr if ws is not None else None, _stream(stream)))


def wmtp_kv_append_many(kv: KV, k_new, v_new, ws: Workspace | None = None, stream=None) -> None:
    _check(lib().wmtp_kv_append_many(byref(kv.desc), k_new.shape[1], _ptr(k_new), _ptr(v_new),
                                     ws.ptr if ws is not None else None, _stream(stream)))


def wmtp_draft_extend_windowed(q, ring: Ring, out, ws: Workspace, lse=None, sm_scale: float = 0.0, stream=None) -> None:
    """q, out: [batch][q_len][Hq][D]; the workspace must be sized for batch * q_len sequences."""
    q_len, Hq = q.shape[1], q.shape[2]
    _check(lib().wmtp_draft_extend_windowed(_ptr(q), q_len, Hq, byref(ring.desc), sm_scale, _ptr(out), _ptr(lse), ws.ptr,
                                            ws.nbytes, _stream(stream)))


def wmtp_draft_extend_full(q, kv: KV, out, ws: Workspace, lse=None, sm_scale: float = 0.0, stream=None) -> None:
    q_len, Hq = q.shape[1], q.shape[2]
    _check(lib().wmtp_draft_extend_full(_ptr(q), q_len, Hq, byref(kv.desc), sm_scale, _ptr(out), _ptr(lse), ws.ptr,
                                        ws.nbytes, _stream(stream)))


def wmtp_attn_mass_diagnostics(out_win, lse_win, out_full, lse_full, mass=None, perturb=None, tail=None, stream=None) -> None:
    D = out_win.shape[-1]
    rows = out_win.numel() // D
    _check(lib().wmtp_attn_mass_diagnostics(_ptr(out_win), _ptr(lse_win), _ptr(out_full), _ptr(lse_full), rows, D, _ptr(mass),
                                            _ptr(perturb), _ptr(tail), _stream(stream)))


def wmtp_full_token_index(kv: KV, index, ws: Workspace | None = None, stream=None) -> None:
    """index: device int32 [batch][stride]; entry s of a row is the pool row of token s, -1 beyond the length."""
    _check(lib().wmtp_full_token_index(byref(kv.desc), _ptr(index), index.shape[1], ws.ptr if ws is not None else None,
                                       _stream(stream)))


def wmtp_reduced_block_table_width(n_sink: int, W: int, page_size: int) -> int:
    return int(lib().wmtp_reduced_block_table_width(n_sink, W, page_size))


def wmtp_reduced_block_table(kv: KV, n_sink: int, W: int, table, meta, ws: Workspace | None = None, stream=None) -> None:
    """table: device int32 [batch][stride]; meta: device int32 [batch][5]."""
    _check(lib().wmtp_reduced_block_table(byref(kv.desc), n_sink, W, _ptr(table), table.shape[1], _ptr(meta),
                                          ws.ptr if ws is not None else None, _stream(stream)))


def wmtp_set_max_ctas(n: int) -> None:
    lib().wmtp_set_max_ctas(int(n))


def wmtp_set_work_stealing(enabled: bool) -> None:
    lib().wmtp_set_work_stealing(1 if enabled else 0)


def wmtp_set_wait_limit(polls: int) -> None:
    lib().wmtp_set_wait_limit(int(polls))


def wmtp_launch_count() -> int:
    return int(lib().wmtp_launch_count())
