"""Workload descriptions for the FreqFormer heterogeneous attention forward.

Pure data: grid sizes, band cut-offs and operator parameters in the paper's
notation (Method, "Setup and notation" .. "Cross-band residual exchange").
No arithmetic of the method lives here; both the CUDA path and the test
oracle read these records.

Notation
  T, H, W     token grid (temporal, height, width); N = T*H*W
  heads, d    number of heads n_h and per-head width d_k
  low_cut     per-axis cut-off L_a: coefficient k is LOW iff k_a < L_a on all axes
  mid_cut     per-axis cut-off M_a: MID iff not LOW and k_a < M_a on all axes
  r           low-band compression ratio (N_low -> ceil(N_low / r))
  b, s        mid-band block size and block stride
  R           high-band window radius (w = 2R+1 keys before clipping)
  m           summary tokens per band
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Tuple


@dataclass(frozen=True)
class FFConfig:
    name: str
    batch: int
    T: int
    H: int
    W: int
    heads: int
    head_dim: int
    dtype: str                      # "bf16" or "fp32": storage type of Q, K, V and out
    low_cut: Tuple[int, int, int]
    mid_cut: Tuple[int, int, int]
    r: int
    b: int
    s: int
    R: int
    m: int
    router_hidden: int = 64
    t_embed_dim: int = 64
    seed: int = 0
    timesteps: Tuple[float, ...] = (500.0,)
    smooth_cosines: int = 0         # number of separable cosines added to every tensor
    smooth_amplitude: float = 0.0
    transform: str = "dct"          # 1-D transform of every axis: "dct" (DCT-II, the reference design) or "haar"
    mid_pattern: str = "strided"    # mid-band sparse pattern: "strided" (own block + blocks at distance 0 mod s)
                                    # or "anchor" (own block + the anchor blocks J = s-1 mod s)

    @property
    def N(self) -> int:
        return self.T * self.H * self.W

    @property
    def grid(self) -> Tuple[int, int, int]:
        return (self.T, self.H, self.W)

    def scaled(self, name: str, **kw) -> "FFConfig":
        return replace(self, name=name, **kw)


def _cuts(grid, c_low_num, c_low_den):
    """L_a = n_a * c_low, M_a = n_a * (c_low + 1/2), both exact integers here."""
    low = tuple(n * c_low_num // c_low_den for n in grid)
    mid = tuple(n * c_low_num // c_low_den + n // 2 for n in grid)
    return low, mid


def _make(name, batch, grid, heads, d, dtype, c_low, r, b, s, R, m, seed, timesteps, **kw):
    low, mid = _cuts(grid, *c_low)
    return FFConfig(name=name, batch=batch, T=grid[0], H=grid[1], W=grid[2], heads=heads,
                    head_dim=d, dtype=dtype, low_cut=low, mid_cut=mid, r=r, b=b, s=s, R=R, m=m,
                    seed=seed, timesteps=tuple(float(t) for t in timesteps), **kw)


# The five workloads of the benchmark definition, in its order.
TINY = _make("tiny_fp32", 1, (4, 8, 8), 2, 32, "fp32", (1, 4), 4, 16, 4, 8, 4, 0, (500,))
G64K = _make("64k", 1, (16, 64, 64), 24, 128, "bf16", (1, 8), 8, 64, 8, 256, 16, 1, (800,))
G256K = _make("256k", 1, (64, 64, 64), 24, 128, "bf16", (1, 8), 8, 64, 8, 256, 16, 2, (200,),
              smooth_cosines=8, smooth_amplitude=3.0)
G1M = _make("1m", 1, (64, 128, 128), 16, 128, "bf16", (1, 16), 16, 128, 16, 512, 32, 3, (500,))
G128K = _make("128k_sweep", 2, (32, 64, 64), 24, 128, "bf16", (1, 8), 8, 64, 8, 256, 16, 4,
              (999, 750, 500, 250, 1))

CONFIGS = (TINY, G64K, G256K, G1M, G128K)
BY_NAME = {c.name: c for c in CONFIGS}

# Scaled-down replicas (same operator parameters, grids of 8K-16K tokens, axis lengths the tensor-core transform covers, fewer heads) on which
# the fp64 oracle can run every stage in full within seconds.
R64K = _make("64k_replica", 1, (16, 32, 32), 6, 128, "bf16", (1, 8), 8, 64, 8, 256, 16, 11, (800,))
R256K = _make("256k_replica", 1, (16, 32, 32), 6, 128, "bf16", (1, 8), 8, 64, 8, 256, 16, 12, (200,),
              smooth_cosines=8, smooth_amplitude=3.0)
R1M = _make("1m_replica", 1, (16, 32, 32), 4, 128, "bf16", (1, 16), 16, 128, 16, 512, 32, 13, (500,))
R128K = _make("128k_replica", 2, (16, 32, 16), 6, 128, "bf16", (1, 8), 8, 64, 8, 256, 16, 14,
              (999, 750, 500, 250, 1))

REPLICAS = (R64K, R256K, R1M, R128K)
BY_NAME.update({c.name: c for c in REPLICAS})

# The paper's own reference parameterisation ("Reference complexity instantiation", "Synthetic
# experiments"): d_k = 64, band fractions 0.125 / 0.375 / 0.5 (low box = half of every axis, mid box
# = the box of about 0.794 of every axis), r = 4 so that N_low_bar = N / 32, window w = 64 (R = 32),
# m = 8, and a mid pattern of constant degree k_mid = 256: blocks of 32 ranks with stride
# s = N_mid / 256 rounded, so that a residue class holds 8 blocks.  head_dim 64 is outside the
# tensor-core exchange kernel (head_dim 128 only), which the generic kernel replaces here.
PAPER_REF_64K = FFConfig(name="paper_ref_64k", batch=1, T=16, H=64, W=64, heads=16, head_dim=64, dtype="bf16",
                         low_cut=(8, 32, 32), mid_cut=(13, 51, 51), r=4, b=32, s=100, R=32, m=8, seed=5,
                         timesteps=(500.0,))
# ... and its replica on a grid the oracle covers in full (axis lengths the tensor-core transform
# covers): 16384 tokens, N_low_bar = N / 32 = 512 (four tiles of the dense low branch), eight or
# nine blocks per residue class.
R_PAPER_REF = FFConfig(name="paper_ref_replica", batch=1, T=16, H=32, W=32, heads=4, head_dim=64, dtype="bf16",
                       low_cut=(8, 16, 16), mid_cut=(13, 26, 26), r=4, b=32, s=26, R=32, m=8, seed=15,
                       timesteps=(500.0,))
# The same parameterisation at the paper's longest sequence: N = 1,048,576, N_low_bar = 32,768 (the
# dense low branch is no longer negligible), 1561 residue classes of 7 or 8 blocks.
PAPER_REF_1M = FFConfig(name="paper_ref_1m", batch=1, T=64, H=128, W=128, heads=16, head_dim=64, dtype="bf16",
                        low_cut=(32, 64, 64), mid_cut=(51, 102, 102), r=4, b=32, s=1561, R=32, m=8, seed=6,
                        timesteps=(500.0,))
BY_NAME.update({c.name: c for c in (PAPER_REF_64K, PAPER_REF_1M, R_PAPER_REF)})
