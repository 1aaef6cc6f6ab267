"""Helpers for the GPU parity tests: upload a synthetic workload, run the CUDA path through the
C-ABI binding, run the CPU oracle on the same bits, compare."""
from __future__ import annotations

import numpy as np
import torch

import paper_2607_21535_b200 as wm
import wmtp_inputs as wi
from oracle import reference as R

# Contract tolerances for bf16 outputs (differences taken in fp32/fp64 on the bf16 result) ...
MAX_ABS, MEAN_ABS = 2e-2, 2e-3
# ... and the stricter per-head checks that stay meaningful when outputs are small (large S).
REL_L2, LSE_ABS = 1e-2, 1e-3


class GuardedAlloc:
    """Device allocations with sentinel-filled bands before and after them: a kernel that writes outside one of the
    arrays it was given changes a band, which `check()` notices (the stand-in for a memory checker on this path)."""

    BAND, SENTINEL = 4096, 0xA5

    def __init__(self):
        self.blocks = []                                   # (name, padded uint8 buffer, payload offset, payload bytes)

    def __call__(self, shape, dtype, device="cuda", name=""):
        nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        padded = (nbytes + 255) // 256 * 256
        buf = torch.full((2 * self.BAND + padded + 256,), self.SENTINEL, dtype=torch.uint8, device=device)
        off = self.BAND + (-(buf.data_ptr() + self.BAND)) % 256        # the array itself starts on a 256-byte boundary
        self.blocks.append((name or f"array {len(self.blocks)}", buf, off, nbytes))
        return buf[off:off + nbytes].view(dtype).view(shape)

    def like(self, t: torch.Tensor, name=""):
        """A guarded copy of t (same shape, dtype, contents)."""
        g = self(tuple(t.shape), t.dtype, t.device, name)
        g.copy_(t)
        return g

    def check(self, what=""):
        if torch.cuda.is_available():
            torch.cuda.synchronize()
        for name, buf, off, nbytes in self.blocks:
            lo, hi = buf[:off], buf[off + nbytes:]
            ok = bool((lo == self.SENTINEL).all()) and bool((hi == self.SENTINEL).all())
            assert ok, f"{what}: bytes outside {name} were written"


def to_dev_bf16(a: np.ndarray, dev="cuda"):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(dev).view(torch.bfloat16)


def bits(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.uint8:                       # fp8 store: the codes themselves
        return t.contiguous().cpu().numpy()
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def to_dev_store(a: np.ndarray, dev="cuda"):
    """KV store contents: bf16 bit patterns (uint16) or e4m3 codes (uint8)."""
    if a.dtype == np.uint8:
        return torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    return to_dev_bf16(a, dev)


class DeviceWorkload:
    """Device copies of a Workload plus ring / KV descriptors / workspace."""

    def __init__(self, wl: wi.Workload, dev="cuda", cap=None):
        cfg = wl.cfg
        self.wl, self.cfg, self.dev = wl, cfg, dev
        # every array a kernel writes lives between guard bands (stores of more than 1 GiB are left as they are)
        self.guard = g = GuardedAlloc()
        self.K, self.V = to_dev_store(wl.K_dev, dev), to_dev_store(wl.V_dev, dev)
        if self.K.numel() * self.K.element_size() <= (1 << 30):
            self.K, self.V = g.like(self.K, "KV store K"), g.like(self.V, "KV store V")
        self.lens = g.like(torch.from_numpy(wl.seq_lens.copy()).to(dev), "the KV lengths")
        pt = torch.from_numpy(wl.page_table).to(dev) if cfg.paged else None
        self.k_scale = torch.from_numpy(wl.k_scale).to(dev) if wl.k_scale is not None else None
        self.v_scale = torch.from_numpy(wl.v_scale).to(dev) if wl.v_scale is not None else None
        self.kv = wm.KV(self.K, self.V, self.lens, page_table=pt, S_cap=None if cfg.paged else wl.S_cap,
                        k_scale=self.k_scale, v_scale=self.v_scale)
        self.ring = wm.Ring(cfg.batch, cfg.Hkv, cfg.D, cfg.n_sink, cfg.W, cap=cap if cap is not None else cfg.W + cfg.cap_slack,
                            device=dev, k_scale=self.k_scale, v_scale=self.v_scale,
                            alloc=lambda shape, dtype, device: g(shape, dtype, device, "a ring array"))
        self.ws = wm.Workspace(cfg.batch, cfg.Hq, cfg.Hkv, cfg.D, device=dev,
                               alloc=lambda shape, dtype, device: g(shape, dtype, device, "the workspace"))
        self.q, self.k_new, self.v_new = to_dev_bf16(wl.q, dev), to_dev_bf16(wl.k_new, dev), to_dev_bf16(wl.v_new, dev)
        self.out_w = g(tuple(self.q.shape), torch.bfloat16, dev, "out (windowed)").fill_(float("nan"))
        self.out_f = g(tuple(self.q.shape), torch.bfloat16, dev, "out (full)").fill_(float("nan"))
        self.lse_w = g(tuple(self.q.shape[:-1]), torch.float32, dev, "lse (windowed)").fill_(float("nan"))
        self.lse_f = g(tuple(self.q.shape[:-1]), torch.float32, dev, "lse (full)").fill_(float("nan"))

    def run_loops(self, windowed=True, full=True):
        if windowed:
            wm.wmtp_ring_init_from_kv(self.ring, self.kv)
            wm.wmtp_draft_loop_windowed(self.ring, self.q, self.k_new, self.v_new, self.out_w, self.ws, lse=self.lse_w)
        if full:
            wm.wmtp_draft_loop_full(self.kv, self.q, self.k_new, self.v_new, self.out_f, self.ws, lse=self.lse_f)
        wm.wmtp_device_status(self.ws)
        self.guard.check(self.cfg.name)


def compare(got_bf16: torch.Tensor, got_lse: torch.Tensor | None, ref_out: np.ndarray, ref_lse: np.ndarray, what=""):
    """got: bf16 [Hq][D] (+ fp32 lse [Hq]) from the GPU; ref: fp64 from the oracle."""
    got = got_bf16.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - ref_out)
    assert err.max() <= MAX_ABS, f"{what}: max-abs {err.max():.3e}"
    assert err.mean() <= MEAN_ABS, f"{what}: mean-abs {err.mean():.3e}"
    num = np.linalg.norm(got - ref_out, axis=-1)
    den = np.linalg.norm(ref_out, axis=-1)
    rel = num / np.maximum(den, 1e-30)
    assert (rel <= REL_L2).all(), f"{what}: per-head relative L2 {rel.max():.3e}"
    if got_lse is not None:
        dl = np.abs(got_lse.cpu().numpy().astype(np.float64) - ref_lse)
        assert (dl <= LSE_ABS).all(), f"{what}: lse error {dl.max():.3e}"
    return float(err.max()), float(rel.max())


def check_ring_against_sim(ring: wm.Ring, b: int, sim: R.RingSim, what=""):
    """Slot positions, length and the bf16 bit patterns of every written slot must be identical."""
    pos = ring.slot_pos[b].cpu().numpy()
    assert (pos == sim.slot_pos).all(), f"{what}: slot_pos differs"
    assert int(ring.len[b]) == sim.length, f"{what}: len differs"
    Kb, Vb = bits(ring.k[b]), bits(ring.v[b])
    w = sim.written
    assert (Kb[:, w] == sim.K[:, w]).all(), f"{what}: ring K bits differ"
    assert (Vb[:, w] == sim.V[:, w]).all(), f"{what}: ring V bits differ"


def oracle_for(wl: wi.Workload, b: int, cap=None, with_ring=True) -> R.DraftOracle:
    cfg = wl.cfg
    return R.DraftOracle(wl.K[b], wl.V[b], cfg.Hq, cfg.n_sink, cfg.W, cap=cap if cap is not None else cfg.W + cfg.cap_slack,
                         reserve=4 * cfg.gamma + 4, with_ring=with_ring, k_scale=wl.k_scale, v_scale=wl.v_scale)
