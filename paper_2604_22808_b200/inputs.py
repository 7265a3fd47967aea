"""Seeded synthetic inputs for the FreqFormer attention forward.

Everything here is input generation: random Q/K/V grids, random router weights,
random summary projections, sampled row indices.  None of the method's own
arithmetic (transform, bands, attention, routing) is implemented in this module,
so the CUDA path and the test oracle can both draw their inputs from it without
sharing any code of the method.

Streams are counter-based (Philox keyed by (seed, stream id)), so any
(tensor, batch, head) slice can be produced on its own and in any order.
Values for bf16 workloads are rounded to bf16 (round to nearest even) on the
host; the rounded values are what both sides consume.
"""
from __future__ import annotations

import numpy as np

from .configs import FFConfig

TENSOR_Q, TENSOR_K, TENSOR_V = 0, 1, 2
_STREAM_QKV, _STREAM_ROUTER, _STREAM_U, _STREAM_COS, _STREAM_ROWS, _STREAM_PROJ = 0, 1, 2, 3, 4, 5


def _rng(seed: int, kind: int, index: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64((kind << 48) | index)]))


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """float32 -> nearest bf16 (ties to even), returned as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) & np.uint32(0xFFFF0000)).view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 values that are exactly representable in bf16 -> their 16-bit patterns."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_float(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def smooth_frequencies(cfg: FFConfig) -> np.ndarray:
    """The integer frequency triples (a_j, b_j, c_j) of the smooth component: uniform in the
    low box, never all zero, shared by every tensor and head of the workload."""
    g = _rng(cfg.seed, _STREAM_COS, 0)
    out = np.zeros((cfg.smooth_cosines, 3), dtype=np.int64)
    for j in range(cfg.smooth_cosines):
        while True:
            f = np.array([g.integers(0, max(1, c)) for c in cfg.low_cut])
            if f.any() or all(c <= 1 for c in cfg.low_cut):
                break
        out[j] = f
    return out


def smooth_signs(cfg: FFConfig, tensor: int, batch: int, head: int) -> np.ndarray:
    """+-1 per (channel, cosine) for one tensor-head."""
    idx = 1 + ((tensor * cfg.batch + batch) * cfg.heads + head)
    g = _rng(cfg.seed, _STREAM_COS, idx)
    return g.integers(0, 2, size=(cfg.head_dim, cfg.smooth_cosines)).astype(np.float32) * 2.0 - 1.0


def _smooth_component(cfg: FFConfig, tensor: int, batch: int, head: int) -> np.ndarray:
    freqs = smooth_frequencies(cfg)
    sig = smooth_signs(cfg, tensor, batch, head)                      # [d, J]
    axes = []
    for n, col in zip(cfg.grid, range(3)):
        i = np.arange(n, dtype=np.float64)
        axes.append(np.cos(np.pi * (2.0 * i[:, None] + 1.0) * freqs[None, :, col] / (2.0 * n)))  # [n, J]
    wave = np.einsum("tj,hj,wj->thwj", axes[0], axes[1], axes[2]).reshape(cfg.N, -1)          # [N, J]
    comp = cfg.smooth_amplitude * (wave @ sig.T.astype(np.float64))                            # [N, d]
    return comp.reshape(cfg.T, cfg.H, cfg.W, cfg.head_dim).astype(np.float32)


def qkv_head(cfg: FFConfig, tensor: int, batch: int, head: int) -> np.ndarray:
    """One tensor-head X[T, H, W, d] as float32: i.i.d. N(0,1) (+ the smooth component when the
    workload has one), already rounded to the workload's storage type."""
    idx = (tensor * cfg.batch + batch) * cfg.heads + head
    x = _rng(cfg.seed, _STREAM_QKV, idx).standard_normal((cfg.T, cfg.H, cfg.W, cfg.head_dim), dtype=np.float32)
    if cfg.smooth_cosines:
        x = x + _smooth_component(cfg, tensor, batch, head)
    return round_to_bf16(x) if cfg.dtype == "bf16" else x


def qkv_full(cfg: FFConfig, tensor: int) -> np.ndarray:
    """[B, heads, T, H, W, d] float32 for one of Q, K, V."""
    out = np.empty((cfg.batch, cfg.heads, cfg.T, cfg.H, cfg.W, cfg.head_dim), dtype=np.float32)
    for bi in range(cfg.batch):
        for h in range(cfg.heads):
            out[bi, h] = qkv_head(cfg, tensor, bi, h)
    return out


def qkv_full_device(cfg: FFConfig, tensor: int, device):
    """[B, heads, T, H, W, d] for one of Q, K, V, drawn on the GPU: the same distribution as
    qkv_full (i.i.d. N(0,1) plus the workload's smooth component, rounded to the storage type)
    from torch's counter-based CUDA generator, seeded by (workload seed, tensor).  For benchmark
    runs at sizes where drawing on the host would take minutes; the values differ from qkv_full's,
    so parity tests keep to the host generator."""
    import torch
    dt = torch.float32 if cfg.dtype == "fp32" else torch.bfloat16
    out = torch.empty((cfg.batch, cfg.heads, cfg.T, cfg.H, cfg.W, cfg.head_dim), dtype=dt, device=device)
    gen = torch.Generator(device=device)
    gen.manual_seed(1000003 * cfg.seed + 101 * tensor + 7)
    axes = None
    if cfg.smooth_cosines:
        freqs = smooth_frequencies(cfg)
        axes = []
        for n, col in zip(cfg.grid, range(3)):
            i = np.arange(n, dtype=np.float64)
            a = np.cos(np.pi * (2.0 * i[:, None] + 1.0) * freqs[None, :, col] / (2.0 * n))
            axes.append(torch.from_numpy(a.astype(np.float32)).to(device))
        wave = torch.einsum("tj,hj,wj->thwj", axes[0], axes[1], axes[2]).reshape(cfg.N, -1)      # [N, J]
    for bi in range(cfg.batch):
        for h in range(cfg.heads):
            x = torch.randn((cfg.N, cfg.head_dim), generator=gen, device=device, dtype=torch.float32)
            if cfg.smooth_cosines:
                sig = torch.from_numpy(smooth_signs(cfg, tensor, bi, h)).to(device)                 # [d, J]
                x += cfg.smooth_amplitude * (wave @ sig.T)
            out[bi, h].copy_(x.view(cfg.T, cfg.H, cfg.W, cfg.head_dim))
    return out


def router_weights(cfg: FFConfig):
    """Random-init router MLP: W1 ~ N(0, 1/in), W2 ~ N(0, 16/hidden), zero biases.
    Drawn in a fixed order (W1 row-major, then W2) from the workload's seed."""
    g = _rng(cfg.seed, _STREAM_ROUTER, 0)
    n_in = 3 * cfg.head_dim + cfg.t_embed_dim
    hid = cfg.router_hidden
    W1 = (g.standard_normal((hid, n_in)) / np.sqrt(n_in)).astype(np.float32)
    W2 = (g.standard_normal((3, hid)) * (4.0 / np.sqrt(hid))).astype(np.float32)
    return {"W1": W1, "b1": np.zeros(hid, np.float32), "W2": W2, "b2": np.zeros(3, np.float32)}


def summary_projection(cfg: FFConfig, identity: bool = True, scale: float = 1.0) -> np.ndarray:
    """U[3, d, d]: identity (the benchmark workloads) or a seeded random matrix whose rows have
    norm `scale` on average (a small scale keeps the summary logits of a workload with large
    low-frequency coefficients of order one)."""
    d = cfg.head_dim
    if identity:
        return np.broadcast_to(np.eye(d, dtype=np.float32), (3, d, d)).copy()
    g = _rng(cfg.seed, _STREAM_U, 0)
    return (g.standard_normal((3, d, d)) * (scale / np.sqrt(d))).astype(np.float32)


def layer_input(cfg: FFConfig) -> np.ndarray:
    """X[B, N, D], D = heads * head_dim: the layer input of the projected entry point, i.i.d. N(0,1),
    rounded to bf16."""
    D = cfg.heads * cfg.head_dim
    x = _rng(cfg.seed, _STREAM_PROJ, 0).standard_normal((cfg.batch, cfg.N, D), dtype=np.float32)
    return round_to_bf16(x)


def projection_weights(cfg: FFConfig):
    """(Wqkv[3, D, D], Wo[D, D]) with y = x W, entries N(0, 1/D) rounded to bf16, so that projected
    channels of an N(0,1) input are N(0,1) again."""
    D = cfg.heads * cfg.head_dim
    g = _rng(cfg.seed, _STREAM_PROJ, 1)
    Wqkv = round_to_bf16((g.standard_normal((3, D, D)) / np.sqrt(D)).astype(np.float32))
    Wo = round_to_bf16((g.standard_normal((D, D)) / np.sqrt(D)).astype(np.float32))
    return Wqkv, Wo


def sample_rows(cfg: FFConfig, tag: int, length: int, count: int) -> np.ndarray:
    """`count` distinct row indices in [0, length), sorted; all rows when length <= count."""
    if length <= count:
        return np.arange(length, dtype=np.int64)
    g = _rng(cfg.seed, _STREAM_ROWS, tag)
    return np.sort(g.choice(length, size=count, replace=False)).astype(np.int64)
