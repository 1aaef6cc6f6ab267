"""Pure-Python twin of the oracle for tiny inputs -- TEST INFRASTRUCTURE, not the product.

Lists, ``math.exp`` and ``struct`` only: no numpy, no C.  It restates softmax attention
over a key set (Appendix D: o = sum_j p_j v_j) and the windowed key set (Appendix A
pseudocode) as directly as Python allows, and exists to brute-force-check the C oracle.
"""
import math
import struct


def bf16_to_float(bits: int) -> float:
    return struct.unpack("<f", struct.pack("<I", (int(bits) & 0xFFFF) << 16))[0]


def attention_py(q, K, V, G, sm_scale):
    """q[h][d], K[g][j][d], V[g][j][d] as nested lists of bf16 bit patterns; returns (out, lse)."""
    out, lse = [], []
    for h in range(len(q)):
        g = h // G
        qf = [bf16_to_float(x) for x in q[h]]
        z = []
        for krow in K[g]:
            z.append(sm_scale * math.fsum(a * bf16_to_float(b) for a, b in zip(qf, krow)))
        if not z:
            out.append([0.0] * len(qf))
            lse.append(-math.inf)
            continue
        m = max(z)
        p = [math.exp(zj - m) for zj in z]
        Z = math.fsum(p)
        D = len(V[g][0])
        out.append([math.fsum(p[j] * bf16_to_float(V[g][j][d]) for j in range(len(p))) / Z for d in range(D)])
        lse.append(m + math.log(Z))
    return out, lse


def window_positions(S, n_sink, W):
    """Positions p in [0, S) that are a sink token or among the last W tokens."""
    return [p for p in range(S) if p < n_sink or p >= S - W]
