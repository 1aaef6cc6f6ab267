"""CPU oracle for Windowed-MTP draft attention -- TEST INFRASTRUCTURE, not the product.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and never calls it.

What is here, and the passage each part restates:

* ``keep_set``      -- the two-branch key-set rule of the windowing pseudocode (Appendix A):
                       sink positions plus the last W positions when S > n_sink + W, else all.
* ``WindowStore``   -- an explicit list-based sink + window store (Section 4, "Mechanism":
                       the first n_sink tokens plus the most recent W tokens).
* ``RingSim``       -- a slot-level simulation of the compact ring buffer (Section 4,
                       "Memory"; Appendix A "RING" comment) with a wrapping write cursor.
* ``attention``     -- fp64 two-pass softmax attention over a key set (Appendix D:
                       o = sum_j p_j v_j; in-window mass = Z_win / Z), in C.
* ``DraftOracle``   -- gamma sequential draft steps: append the step's K/V, then attend,
                       in the windowed and in the full-context form (Section 3, Eq. 1:
                       gamma draft forwards per decode step).

Readings of points the paper leaves open are listed in the repository's design notes;
the ones that matter here: the window includes the token appended in the same step; sink
and window never double-count a position; the sink slots are fixed and only the window
region of the ring is circular; query head h reads KV head h // (Hq // Hkv); the softmax
scale defaults to 1/sqrt(D).

Pins (tests/test_oracle_*.py): closed forms of softmax attention, brute force against a
pure-Python twin on tiny inputs, torch's scaled_dot_product_attention in fp64, the
windowed == full identity for S <= n_sink + W, the mass identity, hand-written key sets
under tests/golden/.  No function here is "parity unpinned".
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wmtp_oracle.c")
_LIB = os.path.join(_HERE, "libwmtp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP over query heads)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.wmtp_oracle_attention.restype = ctypes.c_int
        L.wmtp_oracle_attention.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
            ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
        L.wmtp_oracle_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def threads() -> int:
    return int(lib().wmtp_oracle_threads())


def attention(q, K, V, keys=None, sm_scale=None, heads=None):
    """Softmax attention of one decode query per head over a key set, in fp64.

    q: uint16 [Hq][D] (bf16 bits); K, V: uint16 [Hkv][rows][D] (the two inner dimensions
    contiguous; heads may be strided).  ``keys`` selects rows (default: all rows).
    Returns (out float64 [Hq][D], lse float64 [Hq]).  ``heads=(lo, hi)`` computes only
    that range of query heads (other rows of the result are NaN).
    """
    q = np.ascontiguousarray(q, dtype=np.uint16)
    Hq, D = q.shape
    Hkv, rows, D2 = K.shape
    assert D2 == D and V.shape == K.shape and K.dtype == np.uint16 and V.dtype == np.uint16
    if rows > 0:
        assert K.strides[2] == 2 and K.strides[1] == 2 * D and V.strides == K.strides
    head_stride = K.strides[0] // 2 if (Hkv > 1 and rows > 0) else rows * D
    if keys is None:
        n, kptr, kref = rows, None, None
    else:
        kref = np.ascontiguousarray(keys, dtype=np.int64)
        n = kref.size
        assert n == 0 or (kref.min() >= 0 and kref.max() < rows)
        kptr = kref.ctypes.data
    if sm_scale is None:
        sm_scale = 1.0 / math.sqrt(D)
    out = np.full((Hq, D), np.nan, dtype=np.float64)
    lse = np.full((Hq,), np.nan, dtype=np.float64)
    lo, hi = (0, Hq) if heads is None else heads
    rc = lib().wmtp_oracle_attention(q.ctypes.data, K.ctypes.data, V.ctypes.data, head_stride, kptr, n,
                                     Hq, Hkv, D, float(sm_scale), out.ctypes.data, lse.ctypes.data, lo, hi)
    if rc != 0:
        raise RuntimeError("wmtp_oracle_attention failed")
    return out, lse


def keep_set(S: int, n_sink: int, W: int) -> list:
    """Positions the windowed draft attends at sequence length S (Appendix A pseudocode)."""
    if S > n_sink + W:
        return list(range(0, n_sink)) + list(range(S - W, S))
    return list(range(0, S))


class WindowStore:
    """Explicit sink list + window list; the key set is their concatenation."""

    def __init__(self, n_sink: int, W: int):
        assert n_sink >= 0 and W >= 1
        self.n_sink, self.W = n_sink, W
        self.sink = []      # entries (pos, k_row [Hkv][D], v_row [Hkv][D])
        self.window = []
        self.length = 0

    def append(self, k_row, v_row):
        entry = (self.length, k_row, v_row)
        if len(self.sink) < self.n_sink:
            self.sink.append(entry)
        else:
            self.window.append(entry)
            if len(self.window) > self.W:
                self.window.pop(0)
        self.length += 1

    def entries(self):
        return self.sink + self.window

    def positions(self):
        return [e[0] for e in self.entries()]

    def stacked(self):
        """(K [Hkv][n][D], V [Hkv][n][D]) of the stored rows in logical order."""
        ent = self.entries()
        K = np.ascontiguousarray(np.stack([e[1] for e in ent], axis=1))
        V = np.ascontiguousarray(np.stack([e[2] for e in ent], axis=1))
        return K, V


class RingSim:
    """Slot-level ring: n_sink fixed slots, then `cap` window slots written by a wrapping cursor."""

    def __init__(self, n_sink: int, cap: int, Hkv: int, D: int):
        self.n_sink, self.cap = n_sink, cap
        self.slot_pos = np.full(n_sink + cap, -1, dtype=np.int32)
        self.K = np.zeros((Hkv, n_sink + cap, D), dtype=np.uint16)
        self.V = np.zeros((Hkv, n_sink + cap, D), dtype=np.uint16)
        self.written = np.zeros(n_sink + cap, dtype=bool)
        self.cursor = n_sink
        self.length = 0

    def append(self, k_row, v_row):
        p = self.length
        if p < self.n_sink:
            slot = p
        else:
            slot = self.cursor
            self.cursor += 1
            if self.cursor == self.n_sink + self.cap:
                self.cursor = self.n_sink
        self.K[:, slot, :] = k_row
        self.V[:, slot, :] = v_row
        self.slot_pos[slot] = p
        self.written[slot] = True
        self.length = p + 1
        return slot


    def rewind(self, n_drop: int):
        """Discard the last n_drop tokens (rejected speculative tokens): their slots become empty."""
        assert 0 <= n_drop <= self.length
        for _ in range(n_drop):
            p = self.length - 1
            slot = p if p < self.n_sink else (self.cursor - 1 if self.cursor > self.n_sink else self.n_sink + self.cap - 1)
            assert self.slot_pos[slot] == p
            self.slot_pos[slot] = -1
            self.written[slot] = False
            if p >= self.n_sink:
                self.cursor = slot
            self.length = p


class DraftOracle:
    """One sequence's draft state: full KV, list store and ring simulation, stepped together."""

    def __init__(self, K0, V0, Hq: int, n_sink: int, W: int, cap: int | None = None,
                 sm_scale=None, reserve: int = 16, with_ring: bool = True):
        Hkv, S0, D = K0.shape
        self.Hq, self.Hkv, self.D = Hq, Hkv, D
        self.n_sink, self.W = n_sink, W
        self.sm_scale = sm_scale
        self.Kfull = np.zeros((Hkv, S0 + reserve, D), dtype=np.uint16)
        self.Vfull = np.zeros((Hkv, S0 + reserve, D), dtype=np.uint16)
        self.Kfull[:, :S0] = K0
        self.Vfull[:, :S0] = V0
        self.S = S0
        self.store = WindowStore(n_sink, W)
        self.ring = RingSim(n_sink, W if cap is None else cap, Hkv, D) if with_ring else None
        for p in range(S0):
            k, v = self.Kfull[:, p, :], self.Vfull[:, p, :]
            self.store.append(k, v)
            if self.ring is not None:
                self.ring.append(k, v)

    def append(self, k_row, v_row):
        assert self.S < self.Kfull.shape[1]
        self.Kfull[:, self.S, :] = k_row
        self.Vfull[:, self.S, :] = v_row
        k, v = self.Kfull[:, self.S, :], self.Vfull[:, self.S, :]
        self.store.append(k, v)
        if self.ring is not None:
            self.ring.append(k, v)
        self.S += 1

    def attend_windowed(self, q, heads=None):
        Kw, Vw = self.store.stacked()
        return attention(q, Kw, Vw, sm_scale=self.sm_scale, heads=heads)

    def attend_full(self, q, heads=None):
        return attention(q, self.Kfull[:, : self.S], self.Vfull[:, : self.S], sm_scale=self.sm_scale, heads=heads)

    def step(self, q, k_row, v_row, full: bool = True, windowed: bool = True):
        """Append this step's K/V, then attend with q.  Returns {'win': (out, lse), 'full': (out, lse)}."""
        self.append(k_row, v_row)
        res = {}
        if windowed:
            res["win"] = self.attend_windowed(q)
        if full:
            res["full"] = self.attend_full(q)
        return res


def in_window_mass(lse_win, lse_full):
    """Fraction of the full softmax mass that falls on the windowed key set (Appendix D)."""
    return np.exp(np.asarray(lse_win) - np.asarray(lse_full))


def tail_out_frac(o_full, o_win, lse_win, lse_full):
    """Share of the read-out norm contributed by the far keys (Appendix D): ||(1 - mu) o_far|| / ||o_full||,
    with (1 - mu) o_far = o_full - mu o_win."""
    o_full, o_win = np.asarray(o_full), np.asarray(o_win)
    mu = in_window_mass(lse_win, lse_full)[..., None]
    return np.linalg.norm(o_full - mu * o_win, axis=-1) / np.linalg.norm(o_full, axis=-1)


def win_perturb(o_full, o_win):
    """Relative L2 change of the read-out when the far keys are dropped (Appendix D)."""
    o_full, o_win = np.asarray(o_full), np.asarray(o_win)
    return np.linalg.norm(o_full - o_win, axis=-1) / np.linalg.norm(o_full, axis=-1)
