"""CPU oracle for Windowed-MTP draft attention -- TEST INFRASTRUCTURE, not the product.

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and never calls it.

What is here, and the passage each part restates:

* ``keep_set``      -- the two-branch key-set rule of the windowing pseudocode (Appendix A):
                       sink positions plus the last W positions when S > n_sink + W, else all.
* ``reduced_block_table`` -- the block table the windowed draft attends through (Section 4,
                       "Mechanism": [sink blocks] || [recent-W blocks]), with token-granular ends.
* ``WindowStore``   -- an explicit list-based sink + window store (Section 4, "Mechanism":
                       the first n_sink tokens plus the most recent W tokens).
* ``RingSim``       -- a slot-level simulation of the compact ring buffer (Section 4,
                       "Memory"; Appendix A "RING" comment) with a wrapping write cursor.
* ``attention``     -- fp64 two-pass softmax attention over a key set (Appendix D:
                       o = sum_j p_j v_j; in-window mass = Z_win / Z), in C.
* ``DraftOracle``   -- gamma sequential draft steps: append the step's K/V, then attend,
                       in the windowed and in the full-context form (Section 3, Eq. 1:
                       gamma draft forwards per decode step).
* ``e4m3_decode`` / ``e4m3_encode`` / ``quantize_rows`` and the uint8 branch of ``attention``
                    -- the fp8-KV variant (Section 6, "Robustness to KV-cache quantization":
                       the KV dtype only sets the bytes per entry): e4m3 codes with one fp32
                       scale per KV head, value = code value * scale; new rows are quantised
                       on append with round-to-nearest-even and saturation at 448.

Readings of points the paper leaves open, as far as they matter here: the window includes the token appended in the same step; sink
and window never double-count a position; the sink slots are fixed and only the window
region of the ring is circular; query head h reads KV head h // (Hq // Hkv); the softmax
scale defaults to 1/sqrt(D).

Pins (tests/test_oracle_*.py): closed forms of softmax attention, brute force against a
pure-Python twin on tiny inputs, torch's scaled_dot_product_attention in fp64, the
windowed == full identity for S <= n_sink + W, the mass identity, hand-written key sets
under tests/golden/; for fp8: hand-worked codes of the format, torch's float8_e4m3fn cast,
brute-force nearest-code search, equality with the bf16 read-out on exactly representable
values; ``win_perturb`` by hand vectors that fix its numerator and denominator separately.
No function here is "parity unpinned".
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
        L.wmtp_oracle_attention_f8.restype = ctypes.c_int
        L.wmtp_oracle_attention_f8.argtypes = [
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
            ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_double,
            ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
        L.wmtp_oracle_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def threads() -> int:
    return int(lib().wmtp_oracle_threads())


def attention(q, K, V, keys=None, sm_scale=None, heads=None, k_scale=None, v_scale=None):
    """Softmax attention of one decode query per head over a key set, in fp64.

    q: uint16 [Hq][D] (bf16 bits); K, V: [Hkv][rows][D] (the two inner dimensions contiguous; heads
    may be strided), either uint16 (bf16 bits) or uint8 (e4m3 codes; the value of an entry of KV head
    g is the code's value times k_scale[g] / v_scale[g], fp32 [Hkv]).  ``keys`` selects rows
    (default: all rows).  Returns (out float64 [Hq][D], lse float64 [Hq]).  ``heads=(lo, hi)``
    computes only that range of query heads (other rows of the result are NaN).
    """
    q = np.ascontiguousarray(q, dtype=np.uint16)
    Hq, D = q.shape
    Hkv, rows, D2 = K.shape
    f8 = K.dtype == np.uint8
    esz = 1 if f8 else 2
    assert D2 == D and V.shape == K.shape and K.dtype in (np.uint16, np.uint8) and V.dtype == K.dtype
    if rows > 0:
        assert K.strides[2] == esz and K.strides[1] == esz * D and V.strides == K.strides
    head_stride = K.strides[0] // esz if (Hkv > 1 and rows > 0) else rows * D
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
    if f8:
        ks = np.ascontiguousarray(k_scale, dtype=np.float32)
        vs = np.ascontiguousarray(v_scale, dtype=np.float32)
        assert ks.shape == (Hkv,) and vs.shape == (Hkv,)
        rc = lib().wmtp_oracle_attention_f8(q.ctypes.data, K.ctypes.data, V.ctypes.data, head_stride, kptr, n,
                                            Hq, Hkv, D, float(sm_scale), ks.ctypes.data, vs.ctypes.data,
                                            out.ctypes.data, lse.ctypes.data, lo, hi)
    else:
        assert k_scale is None and v_scale is None
        rc = lib().wmtp_oracle_attention(q.ctypes.data, K.ctypes.data, V.ctypes.data, head_stride, kptr, n,
                                         Hq, Hkv, D, float(sm_scale), out.ctypes.data, lse.ctypes.data, lo, hi)
    if rc != 0:
        raise RuntimeError("wmtp_oracle_attention failed")
    return out, lse


# ---- fp8 (e4m3) KV entries (Section 6, "Robustness to KV-cache quantization") ----------------------
def e4m3_decode(codes):
    """Value of e4m3 codes as float64: 1 sign, 4 exponent (bias 7), 3 mantissa bits; exponent 0 is
    subnormal; 0x7f / 0xff are NaN; no infinities; largest finite value 448."""
    b = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    s, e, m = b >> 7, (b >> 3) & 15, b & 7
    mag = np.where(e == 0, (m / 8.0) * 2.0 ** -6, (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64)))
    mag = np.where((e == 15) & (m == 7), np.nan, mag)
    return np.where(s == 1, -mag, mag)


def e4m3_encode(x):
    """Nearest e4m3 code of fp32 values: round to nearest, ties to the even mantissa, magnitudes that
    would round beyond 448 saturate to 448 (no infinities in the format), NaN stays NaN."""
    x = np.asarray(x, dtype=np.float32)
    a = np.abs(x.astype(np.float64))
    sign = np.signbit(x).astype(np.int64) << 7
    with np.errstate(invalid="ignore", divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0))).astype(np.int64)     # exact: a is an fp32 value
        e = np.clip(e, -6, 8)                                                  # below 2^-6 the spacing stays 2^-9
        steps = np.rint(a / np.exp2((e - 3).astype(np.float64))).astype(np.int64)   # multiples of the spacing, ties to even
    # steps in [0, 16]: 16 means the next binade (mantissa 0 there); subnormals (e = -6, steps < 8) have exponent field 0
    code = np.where(steps < 8, steps, ((e + 7) << 3) + (steps - 8))            # carries propagate into the exponent field
    code = np.where((a >= 448.0) | (code > 0x7e), 0x7e, code)
    code = np.where(np.isnan(a), 0x7f, code)
    return (code | sign).astype(np.uint8)


def bf16_bits_to_f32(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def quantize_rows(rows_bf16, scale):
    """Store-side quantisation of new K or V rows [Hkv][D] (bf16 bits): code = e4m3(x / scale[g]), the
    division in fp32 (so that value ~ code * scale[g], the dequantisation the attention applies)."""
    x = bf16_bits_to_f32(rows_bf16)
    sc = np.asarray(scale, dtype=np.float32).reshape(-1, 1)
    return e4m3_encode((x / sc).astype(np.float32))


def keep_set(S: int, n_sink: int, W: int) -> list:
    """Positions the windowed draft attends at sequence length S (Appendix A pseudocode)."""
    if S > n_sink + W:
        return list(range(0, n_sink)) + list(range(S - W, S))
    return list(range(0, S))


def reduced_block_table(S: int, n_sink: int, W: int, page_row, page_size: int):
    """The windowed draft's block table (Section 4 "Mechanism": the per-request table reduced to
    [sink blocks] || [recent-W blocks]) for one sequence of length S whose full table is ``page_row``.

    Returns (pages, meta): ``pages`` lists the pages holding the sink positions, then the pages holding the last-W
    positions (a page that holds both kinds appears in both parts); ``meta`` = [sink pages, window pages, sink rows
    used in the last sink page, first row used in the first window page, rows used in the last window page] -- what
    a reader needs to keep the ends token-granular.  Built in O((n_sink + W) / page_size) from S alone."""
    keep = keep_set(S, n_sink, W)
    ns = min(S, n_sink)
    sink_pos = [p for p in keep if p < ns]
    win_pos = [p for p in keep if p >= ns]
    sink_pages = sorted({p // page_size for p in sink_pos})
    win_pages = sorted({p // page_size for p in win_pos})
    pages = [int(page_row[i]) for i in sink_pages] + [int(page_row[i]) for i in win_pages]
    meta = [len(sink_pages), len(win_pages),
            (sink_pos[-1] % page_size + 1) if sink_pos else 0,
            (win_pos[0] % page_size) if win_pos else 0,
            (win_pos[-1] % page_size + 1) if win_pos else 0]
    return pages, meta


def full_token_index(S: int, page_row, page_size: int, stride: int):
    """The O(S) structure a full-context draft over a paged store rebuilds every step (Section 3, t_ctx; Appendix B,
    per-kernel table: the draft's KV index build): for each token position s < S the pool row that holds it,
    page_row[s // page_size] * page_size + s % page_size; -1 from S up to ``stride``.  One entry per token."""
    out = [-1] * stride
    for s in range(min(S, stride)):
        out[s] = int(page_row[s // page_size]) * page_size + s % page_size
    return out


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

    def __init__(self, n_sink: int, cap: int, Hkv: int, D: int, dtype=np.uint16):
        self.n_sink, self.cap = n_sink, cap
        self.slot_pos = np.full(n_sink + cap, -1, dtype=np.int32)
        self.K = np.zeros((Hkv, n_sink + cap, D), dtype=dtype)
        self.V = np.zeros((Hkv, n_sink + cap, D), dtype=dtype)
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
                 sm_scale=None, reserve: int = 16, with_ring: bool = True, k_scale=None, v_scale=None):
        """K0, V0: [Hkv][S0][D] bf16 bits (uint16), or e4m3 codes (uint8) with per-KV-head scales: the
        stores then hold codes, and the K/V rows of a step (always bf16) are quantised on append."""
        Hkv, S0, D = K0.shape
        self.Hq, self.Hkv, self.D = Hq, Hkv, D
        self.n_sink, self.W = n_sink, W
        self.sm_scale = sm_scale
        self.f8 = K0.dtype == np.uint8
        assert self.f8 == (k_scale is not None) == (v_scale is not None) and V0.dtype == K0.dtype
        self.k_scale = None if k_scale is None else np.asarray(k_scale, dtype=np.float32)
        self.v_scale = None if v_scale is None else np.asarray(v_scale, dtype=np.float32)
        self.Kfull = np.zeros((Hkv, S0 + reserve, D), dtype=K0.dtype)
        self.Vfull = np.zeros((Hkv, S0 + reserve, D), dtype=K0.dtype)
        self.Kfull[:, :S0] = K0
        self.Vfull[:, :S0] = V0
        self.S = S0
        self.store = WindowStore(n_sink, W)
        self.ring = RingSim(n_sink, W if cap is None else cap, Hkv, D, dtype=K0.dtype) if with_ring else None
        for p in range(S0):
            k, v = self.Kfull[:, p, :], self.Vfull[:, p, :]
            self.store.append(k, v)
            if self.ring is not None:
                self.ring.append(k, v)

    def append(self, k_row, v_row):
        assert self.S < self.Kfull.shape[1]
        if self.f8:
            k_row, v_row = quantize_rows(k_row, self.k_scale), quantize_rows(v_row, self.v_scale)
        self.Kfull[:, self.S, :] = k_row
        self.Vfull[:, self.S, :] = v_row
        k, v = self.Kfull[:, self.S, :], self.Vfull[:, self.S, :]
        self.store.append(k, v)
        if self.ring is not None:
            self.ring.append(k, v)
        self.S += 1

    def attend_windowed(self, q, heads=None):
        Kw, Vw = self.store.stacked()
        return attention(q, Kw, Vw, sm_scale=self.sm_scale, heads=heads, k_scale=self.k_scale, v_scale=self.v_scale)

    def attend_full(self, q, heads=None):
        return attention(q, self.Kfull[:, : self.S], self.Vfull[:, : self.S], sm_scale=self.sm_scale, heads=heads,
                         k_scale=self.k_scale, v_scale=self.v_scale)

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
