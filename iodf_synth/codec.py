"""Parameters of the entropy coder's prior tables (inputs of both the CPU oracle and the CUDA path,
like the weights: data, no coding arithmetic).

The prior is the discrete logistic of Sec. 3. Its integer form needs two tables:
  G[u + umax]  a sigmoid over u = 64 x, u in [-umax, umax], scaled to [0, M - (2 window + 1)] with
               M = 2^16 (the rest of the mass is the one extra count per symbol of the window)
  R[ls]        2^21 / s for the scales s = 2^(ls/4 - 2), ls = 0 .. n_scales-1 (0.25 .. ~13800), so that
               floor((2r - 1) R / 2^16) = floor(64 (r - 1/2) / s)
"""
import numpy as np

M_BITS = 16
WINDOW = 2048


def logistic_codec(n_scales=64, umax=1024, final_ls=40, elems_per_stream=128):
    M = 1 << M_BITS
    u = np.arange(-umax, umax + 1, dtype=np.float64)
    top = M - (2 * WINDOW + 1)
    G = np.floor(top / (1.0 + np.exp(-u / 64.0)) + 0.5)
    G = np.minimum(np.maximum.accumulate(G), top).astype(np.uint16)
    s = 2.0 ** (np.arange(n_scales, dtype=np.float64) / 4.0 - 2.0)
    R = np.floor(2.0 ** 21 / s + 0.5).astype(np.uint32)
    return {"G": G, "umax": int(umax), "R": R, "scales": s, "final_ls": int(final_ls),
            "elems_per_stream": int(elems_per_stream), "window": WINDOW, "M": M}
