"""The synthetic draft-attention workloads (shapes, lengths, layouts) and their tensors.

Every workload is a batch of sequences with a bf16 (or fp8 e4m3) KV cache for one draft layer
(Hkv KV heads of head_dim D, Hq = G*Hkv query heads), an attention sink of n_sink
tokens, a window of W tokens and gamma sequential draft steps; each step brings one
new (q, k, v) per sequence.  Tensors are generated in *logical* form
(``K[b][g][pos][d]``) and, for the paged layout, scattered into a page pool through a
seeded random page table.  Only generation and layout live here -- no attention, softmax
or ring arithmetic.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace

import numpy as np

from . import gen

T_K, T_V, T_Q, T_KNEW, T_VNEW, T_LENS, T_PAGES = 1, 2, 3, 4, 5, 6, 7
BF16_NAN = np.uint16(0x7FC0)
E4M3_NAN = np.uint8(0x7F)
E4M3_RANGE_SIGMAS = 4.5          # an fp8 store maps +-4.5 standard deviations of its head onto +-448


@dataclass(frozen=True)
class DraftConfig:
    name: str
    batch: int
    S0: int                      # context length before the first draft step (batch 1)
    Hq: int
    Hkv: int
    D: int
    W: int
    n_sink: int
    gamma: int
    seed: int
    S0_range: tuple | None = None    # (lo, hi): per-sequence lengths log-uniform in [lo, hi]
    paged: bool = False
    page_size: int = 64
    key_scale: tuple | None = None   # (lo, hi): per-KV-head multiplier on K, log-spaced
    cap_slack: int = 0               # ring capacity = W + cap_slack window slots
    kv_dtype: str = "bf16"           # "bf16", or "fp8": e4m3 codes with one fp32 scale per KV head for K and for V
    logit_profile: tuple | None = None   # (delta, tau): recency-peaked logits, see recency_column (bf16 stores only)

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def kv_bytes_per_token(self) -> int:
        return self.Hkv * self.D * 2 * (1 if self.kv_dtype == "fp8" else 2)


# The five workloads named by the benchmark description; index = position in that list.
CONFIGS = [
    DraftConfig("tiny", 1, 4096, 16, 2, 128, 512, 4, 3, seed=1234),
    DraftConfig("s128k", 1, 131072, 16, 2, 256, 2048, 4, 3, seed=1235),
    DraftConfig("million", 1, 1048576, 16, 2, 256, 4096, 4, 7, seed=1236, key_scale=(0.5, 2.0)),
    DraftConfig("batched", 32, 0, 16, 2, 128, 2048, 4, 7, seed=1237, S0_range=(32768, 1048576),
                paged=True, page_size=64),
    DraftConfig("sweep", 1, 1048576, 32, 4, 128, 4096, 4, 7, seed=1238),
]


def sweep_configs():
    """Context/depth sweep: S x gamma x W for the Hq=32, Hkv=4, D=128 shape."""
    out = []
    for S in (65536, 262144, 524288, 1048576):
        for gamma in (3, 7, 9):
            for W in (1024, 4096):
                out.append(replace(CONFIGS[4], name=f"sweep_S{S}_g{gamma}_W{W}", S0=S, gamma=gamma, W=W))
    return out


@dataclass
class Workload:
    cfg: DraftConfig
    seq_lens: np.ndarray                 # int64 [B], lengths before the first draft step
    K: list = field(default_factory=list)    # per sequence: uint16 [Hkv][S0_b][D] logical keys
    V: list = field(default_factory=list)
    q: np.ndarray = None                 # uint16 [gamma][B][Hq][D]
    k_new: np.ndarray = None             # uint16 [gamma][B][Hkv][D]
    v_new: np.ndarray = None
    # device-layout copies (what the CUDA path is given)
    S_cap: int = 0
    K_dev: np.ndarray = None             # contiguous: [B][Hkv][S_cap][D]; paged: [num_pages][Hkv][ps][D]
    V_dev: np.ndarray = None
    page_table: np.ndarray = None        # int32 [B][max_pages] (paged only)
    num_pages: int = 0
    max_pages: int = 0
    k_scale: np.ndarray = None           # fp8 stores: float32 [Hkv], value = code * scale (None for bf16)
    v_scale: np.ndarray = None


def head_scales(cfg: DraftConfig) -> np.ndarray:
    if cfg.key_scale is None:
        return np.ones(cfg.Hkv)
    lo, hi = cfg.key_scale
    if cfg.Hkv == 1:
        return np.array([lo])
    return lo * (hi / lo) ** (np.arange(cfg.Hkv) / (cfg.Hkv - 1))


Q_ALONG = 4.0     # component of every query along the profile direction (dimension 0)


def recency_column(S: int, D: int, delta: float, tau: float, S_ref: int | None = None) -> np.ndarray:
    """Dimension-0 entries of the keys at positions [0, S) for a recency-peaked logit profile: with every query's
    dimension 0 set to Q_ALONG, the key at distance dist = S_ref - 1 - pos from the newest token gets
    delta * exp(-dist / tau) added to its scaled logit (softmax scale 1/sqrt(D)), on top of the i.i.d. noise of the
    other dimensions.  Large delta with a short tau imitates a locally peaked (RoPE-like) head, small delta a diffuse
    (NoPE-like) one."""
    S_ref = S if S_ref is None else S_ref
    dist = (S_ref - 1 - np.arange(S, dtype=np.float64))
    return (delta * np.sqrt(D) / Q_ALONG * np.exp(-np.maximum(dist, 0.0) / tau)).astype(np.float32)


def profile_window_mass(S: int, n_sink: int, W: int, delta: float, tau: float) -> float:
    """Share of the softmax mass that the profile alone (noise averaged out) puts on sink + last W at length S."""
    dist = S - 1 - np.arange(S, dtype=np.float64)
    w = np.exp(delta * np.exp(-dist / tau))
    inside = (np.arange(S) < n_sink) | (np.arange(S) >= S - W)
    return float(w[inside].sum() / w.sum())


def calibrate_delta(S: int, n_sink: int, W: int, tau: float, target_mass: float) -> float:
    """delta for which profile_window_mass equals target_mass (bisection; the mass grows with delta)."""
    lo, hi = 0.0, 40.0
    for _ in range(60):
        mid = (lo + hi) / 2
        if profile_window_mass(S, n_sink, W, mid, tau) < target_mass:
            lo = mid
        else:
            hi = mid
    return (lo + hi) / 2


def seq_lens(cfg: DraftConfig) -> np.ndarray:
    if cfg.S0_range is None:
        return np.full(cfg.batch, cfg.S0, dtype=np.int64)
    lo, hi = cfg.S0_range
    u = gen.rng(cfg.seed, T_LENS).random(cfg.batch)
    return np.rint(np.exp(np.log(lo) + u * (np.log(hi) - np.log(lo)))).astype(np.int64)


def make_workload(cfg: DraftConfig, poison_unused: bool = True, extra_cap: int = 0,
                  threads: int | None = None) -> Workload:
    """Generate all tensors of ``cfg``.

    Rows of the device-layout KV that hold no token yet (positions >= the sequence's
    length) are filled with a bf16 NaN pattern when ``poison_unused`` is set, so a
    kernel that lets a stale row leak into its result fails loudly.

    With ``kv_dtype == "fp8"`` the store holds e4m3 codes: the same N(0, head scale) draws, expressed in
    units of ``k_scale[g] = 4.5 * head scale / 448`` (``v_scale = 4.5 / 448``) and cut to the code grid by
    ``gen.e4m3_codes_trunc``; the per-step q / k_new / v_new stay bf16.
    """
    B, Hkv, Hq, D, gam = cfg.batch, cfg.Hkv, cfg.Hq, cfg.D, cfg.gamma
    lens = seq_lens(cfg)
    sc = head_scales(cfg)
    wl = Workload(cfg=cfg, seq_lens=lens)
    f8 = cfg.kv_dtype == "fp8"
    assert cfg.kv_dtype in ("bf16", "fp8")
    dt = np.uint8 if f8 else np.uint16
    if f8:
        wl.k_scale = (E4M3_RANGE_SIGMAS * sc / 448.0).astype(np.float32)
        wl.v_scale = np.full(Hkv, E4M3_RANGE_SIGMAS / 448.0, dtype=np.float32)
        fill = E4M3_NAN if poison_unused else np.uint8(0)
    else:
        fill = BF16_NAN if poison_unused else np.uint16(0)

    if cfg.paged:
        ps = cfg.page_size
        need = (lens + gam + extra_cap + ps - 1) // ps
        wl.num_pages = int(need.sum()) + 3          # a few pages no sequence owns
        wl.max_pages = int(need.max())
        perm = gen.rng(cfg.seed, T_PAGES).permutation(wl.num_pages).astype(np.int32)
        wl.page_table = np.full((B, wl.max_pages), -1, dtype=np.int32)
        off = 0
        for b in range(B):
            wl.page_table[b, : need[b]] = perm[off: off + need[b]]
            off += int(need[b])
        wl.K_dev = np.full((wl.num_pages, Hkv, ps, D), fill, dtype=dt)
        wl.V_dev = np.full((wl.num_pages, Hkv, ps, D), fill, dtype=dt)
        wl.S_cap = wl.max_pages * ps
    else:
        wl.S_cap = int(lens.max()) + gam + extra_cap
        wl.K_dev = np.empty((B, Hkv, wl.S_cap, D), dtype=dt)
        wl.V_dev = np.empty((B, Hkv, wl.S_cap, D), dtype=dt)

    for b in range(B):
        S = int(lens[b])
        if cfg.paged:
            Kb = np.empty((Hkv, S, D), dtype=dt)
            Vb = np.empty((Hkv, S, D), dtype=dt)
        else:
            # logical tensors are views of the device-layout buffer (no second copy in host memory)
            Kb = wl.K_dev[b, :, :S, :]
            Vb = wl.V_dev[b, :, :S, :]
            wl.K_dev[b, :, S:, :] = fill
            wl.V_dev[b, :, S:, :] = fill
        for g in range(Hkv):
            kb = gen.normal_bf16(cfg.seed, (T_K, b, g), (S, D), scale=float(sc[g]), threads=threads)
            vb = gen.normal_bf16(cfg.seed, (T_V, b, g), (S, D), threads=threads)
            if f8:
                kb = gen.e4m3_codes_trunc(kb, float(wl.k_scale[g]))
                vb = gen.e4m3_codes_trunc(vb, float(wl.v_scale[g]))
            Kb[g] = kb
            Vb[g] = vb
        if cfg.logit_profile is not None:
            assert not f8, "logit profiles are defined for bf16 stores"
            delta, tau = cfg.logit_profile
            col = gen.f32_to_bf16_bits(recency_column(S, D, delta, tau))
            for g in range(Hkv):
                Kb[g][:, 0] = col
        wl.K.append(Kb)
        wl.V.append(Vb)
        if cfg.paged:
            ps = cfg.page_size
            nfull = S // ps
            pages = wl.page_table[b]
            if nfull:
                # [Hkv][nfull*ps][D] -> [nfull][Hkv][ps][D]
                wl.K_dev[pages[:nfull]] = Kb[:, : nfull * ps].reshape(Hkv, nfull, ps, D).transpose(1, 0, 2, 3)
                wl.V_dev[pages[:nfull]] = Vb[:, : nfull * ps].reshape(Hkv, nfull, ps, D).transpose(1, 0, 2, 3)
            rem = S - nfull * ps
            if rem:
                wl.K_dev[pages[nfull], :, :rem] = Kb[:, nfull * ps:]
                wl.V_dev[pages[nfull], :, :rem] = Vb[:, nfull * ps:]

    wl.q = gen.normal_bf16(cfg.seed, T_Q, (gam, B, Hq, D), threads=threads)
    kn = gen.normal_bf16(cfg.seed, T_KNEW, (gam, B, Hkv, D), threads=threads)
    if cfg.key_scale is not None:
        kf = gen.bf16_bits_to_f32(kn) * sc.astype(np.float32)[None, None, :, None]
        kn = gen.f32_to_bf16_bits(kf)
    if cfg.logit_profile is not None:
        delta, tau = cfg.logit_profile
        wl.q[..., 0] = gen.f32_to_bf16_bits(np.float32([Q_ALONG]))[0]
        kn[..., 0] = gen.f32_to_bf16_bits(np.float32([delta * np.sqrt(D) / Q_ALONG]))[0]       # the newest token: distance 0
    wl.k_new = kn
    wl.v_new = gen.normal_bf16(cfg.seed, T_VNEW, (gam, B, Hkv, D), threads=threads)
    return wl


def scaled(cfg: DraftConfig, **kw) -> DraftConfig:
    """A copy of ``cfg`` with some fields replaced (smaller test-size variants)."""
    return replace(cfg, **kw)
