"""fp64 CPU oracle for the FreqFormer heterogeneous attention forward.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
hot path computes, written from the paper's definitions.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import it; the product
(the CUDA library and its Python binding) never does, and the two share no
code.  Everything is numpy float64; library matmuls appear only where the
definition itself is a matrix product (a 1-D transform along one axis, QK^T,
PV, the router MLP).

Each function names the passage of the paper it follows.  Where the paper is
silent or its display equations are missing, the reading taken is stated in
the docstring and marked "reading".

Parity status of the free readings (low-band pooling operator, the strided
block pattern, pass-through for bands a head is not allocated to, router
statistics / activation / quota rule, summary segments): the paper fixes no
number for them, so they are pinned by invariants and special cases only
(dense-attention reductions, identities, brute force), not by paper values.

`cfg` arguments are duck-typed records with fields
T, H, W, heads, head_dim, low_cut, mid_cut, r, b, s, R, m, t_embed_dim and, optionally,
transform ("dct" or "haar") and mid_pattern ("strided" or "anchor").
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence

import numpy as np

BAND_LOW, BAND_MID, BAND_HIGH = 1, 2, 4          # per-head band-mask bits
_BITS = (BAND_LOW, BAND_MID, BAND_HIGH)


# ----------------------------------------------------------------------------------------------
# Separable spectral decomposition (Method, "Separable spectral decomposition")
# ----------------------------------------------------------------------------------------------
def dct_matrix(n: int) -> np.ndarray:
    """Orthonormal DCT-II matrix C[k, i] = alpha_k cos(pi (2i+1) k / (2n)),
    alpha_0 = sqrt(1/n), alpha_k = sqrt(2/n) for k > 0: the fixed 1-D transform
    F_t, F_h, F_w of the reference design."""
    k = np.arange(n, dtype=np.float64)[:, None]
    i = np.arange(n, dtype=np.float64)[None, :]
    C = np.sqrt(2.0 / n) * np.cos(np.pi * (2.0 * i + 1.0) * k / (2.0 * n))
    C[0, :] = np.sqrt(1.0 / n)
    return C


def haar_matrix(n: int) -> np.ndarray:
    """Orthonormal Haar wavelet matrix for n a power of two ("wavelets are also possible";
    "Transform choice").  Row 0 is the constant 1/sqrt(n); row 2^j + k (level j, shift k) is
    +sqrt(2^j / n) on the first half and -sqrt(2^j / n) on the second half of the k-th block of
    n / 2^j positions, zero elsewhere.  Rows run from the coarsest scale to the finest, so a low
    row index is a coarse scale, as a low DCT index is a low frequency."""
    if n < 1 or n & (n - 1):
        raise ValueError("the Haar transform needs a power-of-two axis length")
    Hm = np.zeros((n, n), dtype=np.float64)
    Hm[0, :] = 1.0 / math.sqrt(n)
    row, j = 1, 0
    while row < n:
        block = n >> j                       # support of a level-j wavelet
        amp = math.sqrt((1 << j) / n)
        for k in range(1 << j):
            Hm[row, k * block:k * block + block // 2] = amp
            Hm[row, k * block + block // 2:(k + 1) * block] = -amp
            row += 1
        j += 1
    return Hm


def transform_matrix(n: int, kind: str = "dct") -> np.ndarray:
    """The fixed orthonormal 1-D transform of one axis: DCT-II (the reference design) or Haar."""
    if kind == "dct":
        return dct_matrix(n)
    if kind == "haar":
        return haar_matrix(n)
    raise ValueError(f"unknown transform {kind!r}")


def forward_transform(X: np.ndarray, kind: str = "dct") -> np.ndarray:
    """X~ = (F_t (x) F_h (x) F_w) X for X[T, H, W, d]: each token axis is multiplied by its
    1-D matrix; the channel axis is untouched (the Kronecker product has no channel factor)."""
    T, H, W, d = X.shape
    Y = (transform_matrix(T, kind) @ X.reshape(T, H * W * d)).reshape(T, H, W, d)
    Y = (transform_matrix(H, kind)[None] @ Y.reshape(T, H, W * d)).reshape(T, H, W, d)
    Y = transform_matrix(W, kind)[None, None] @ Y
    return Y


def inverse_transform(Y: np.ndarray, kind: str = "dct") -> np.ndarray:
    """F^{-1}: the transposes of the orthonormal 1-D matrices along each token axis
    ("Reconstruction": mapped back into token space via the inverse transform)."""
    T, H, W, d = Y.shape
    X = transform_matrix(W, kind).T[None, None] @ Y
    X = (transform_matrix(H, kind).T[None] @ X.reshape(T, H, W * d)).reshape(T, H, W, d)
    X = (transform_matrix(T, kind).T @ X.reshape(T, H * W * d)).reshape(T, H, W, d)
    return X


# ----------------------------------------------------------------------------------------------
# Frequency band partitioning ("Frequency band partitioning")
# ----------------------------------------------------------------------------------------------
def band_labels(grid, low_cut, mid_cut) -> np.ndarray:
    """Label every coefficient k = (k_t, k_h, k_w) with 0 (low), 1 (mid) or 2 (high).
    Reading: nested boxes.  LOW iff k_a < L_a on all three axes; else MID iff k_a < M_a on
    all three; else HIGH.  The three regions are disjoint and cover the coefficient domain."""
    T, H, W = grid
    kt, kh, kw = np.meshgrid(np.arange(T), np.arange(H), np.arange(W), indexing="ij")
    in_low = (kt < low_cut[0]) & (kh < low_cut[1]) & (kw < low_cut[2])
    in_mid = (kt < mid_cut[0]) & (kh < mid_cut[1]) & (kw < mid_cut[2])
    lab = np.full((T, H, W), 2, dtype=np.int8)
    lab[in_mid] = 1
    lab[in_low] = 0
    return lab


def band_members(grid, low_cut, mid_cut) -> List[np.ndarray]:
    """Per band, the flat coefficient indices f(k) = (k_t H + k_h) W + k_w of its members in
    increasing order.  Reading: this is the band-local token order ("flattened spectral-token
    order induced by the separable layout"); the position in the list is the band rank p."""
    lab = band_labels(grid, low_cut, mid_cut).reshape(-1)
    return [np.nonzero(lab == l)[0] for l in range(3)]


def split_bands(Xs: np.ndarray, members: Sequence[np.ndarray]) -> List[np.ndarray]:
    """P_Omega applied to X~[T,H,W,d]: the rows of each band as a band-major list [N_l, d]."""
    flat = Xs.reshape(-1, Xs.shape[-1])
    return [flat[idx] for idx in members]


# ----------------------------------------------------------------------------------------------
# Low-band compression ("we apply explicit compression to obtain ...", operator unspecified)
# ----------------------------------------------------------------------------------------------
def compress_low(x: np.ndarray, r: int) -> np.ndarray:
    """Reading: D_Q = D_K = D_V = mean over groups of r consecutive low-band ranks;
    ceil(N_low / r) groups, the last one may be short."""
    n = x.shape[0]
    groups = -(-n // r)
    return np.stack([x[g * r:min(n, (g + 1) * r)].mean(axis=0) for g in range(groups)])


def decompress_low(y: np.ndarray, r: int, n_low: int) -> np.ndarray:
    """Reading: each compressed output refills the r coefficient slots it was pooled from."""
    return y[np.arange(n_low) // r]


# ----------------------------------------------------------------------------------------------
# Band operators ("Hierarchical frequency-domain attention")
# ----------------------------------------------------------------------------------------------
def softmax_rows(scores: np.ndarray) -> np.ndarray:
    e = np.exp(scores - scores.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def dense_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """softmax(Q K^T / sqrt(d)) V over all keys: the low-band operator on compressed tokens."""
    d = Q.shape[-1]
    return softmax_rows(Q @ K.T / math.sqrt(d)) @ V


def mid_allowed(p, pk, b: int, s: int, pattern: str = "strided"):
    """The mid-band sparse pattern S ("block-local plus strided").  Reading: blocks of b
    consecutive mid ranks.  "strided": query p sees key pk iff their block indices differ by a
    multiple of the stride s (the own block included).  "anchor" (the alternative of the
    "Mid-band sparse degree" ablation): the own block plus every anchor block, the blocks whose
    index is s-1 mod s ("strided connectors" shared by all queries).  This is the single place
    the pattern is defined."""
    Jk, Jq = np.asarray(pk) // b, np.asarray(p) // b
    if pattern == "strided":
        return ((Jk - Jq) % s) == 0
    if pattern == "anchor":
        return (Jk == Jq) | ((Jk % s) == s - 1)
    raise ValueError(f"unknown mid pattern {pattern!r}")


def mid_keys(p: int, n: int, b: int, s: int, pattern: str = "strided") -> np.ndarray:
    """Key set of mid-band query p among n tokens, increasing."""
    pk = np.arange(n)
    return pk[mid_allowed(p, pk, b, s, pattern)]


def high_keys(p: int, n: int, R: int) -> np.ndarray:
    """High-band sliding window.  Reading: symmetric and non-causal, |p - p'| <= R in band
    order, clipped to the band; w = 2R+1 keys before clipping."""
    return np.arange(max(0, p - R), min(n - 1, p + R) + 1)


def sparse_attention_rows(Q: np.ndarray, K: np.ndarray, V: np.ndarray, rows: np.ndarray, key_fn):
    """softmax over each query row's own key set.  Rows whose key sets are identical are
    evaluated together (one score matrix per distinct key set).  Returns (Y[rows], pairs)."""
    d = Q.shape[-1]
    out = np.empty((len(rows), d), dtype=np.float64)
    groups: Dict[bytes, List[int]] = {}
    keysets: Dict[bytes, np.ndarray] = {}
    for i, p in enumerate(rows):
        ks = key_fn(int(p))
        h = ks.tobytes()
        groups.setdefault(h, []).append(i)
        keysets[h] = ks
    pairs = 0
    for h, members in groups.items():
        ks = keysets[h]
        q = Q[rows[members]]
        out[members] = softmax_rows(q @ K[ks].T / math.sqrt(d)) @ V[ks]
        pairs += len(members) * len(ks)
    return out, pairs


def mid_operator(Q, K, V, b: int, s: int, rows: Optional[np.ndarray] = None, pattern: str = "strided"):
    n = Q.shape[0]
    rows = np.arange(n) if rows is None else rows
    return sparse_attention_rows(Q, K, V, rows, lambda p: mid_keys(p, n, b, s, pattern))


def high_operator(Q, K, V, R: int, rows: Optional[np.ndarray] = None):
    n = Q.shape[0]
    rows = np.arange(n) if rows is None else rows
    return sparse_attention_rows(Q, K, V, rows, lambda p: high_keys(p, n, R))


# ----------------------------------------------------------------------------------------------
# Spectral routing network ("Spectral routing network")
# ----------------------------------------------------------------------------------------------
def band_energy_sums(bands: Sequence[np.ndarray]) -> np.ndarray:
    """Per band, per channel sum of squared coefficients of one tensor-head: [3, d]."""
    return np.stack([(x * x).sum(axis=0) for x in bands])


def pooled_statistics(energy_sums: np.ndarray, counts: Sequence[float]) -> np.ndarray:
    """g in R^{3 d}.  Reading: E_l[c] = mean of x~^2 over heads, band-l ranks and {Q~,K~,V~};
    g_l[c] = ln(1 + E_l[c]); g = [g_low; g_mid; g_high] (so d_r = d).
    `energy_sums`[3, d] is the sum over everything pooled, `counts`[l] the number of terms."""
    E = energy_sums / np.asarray(counts, dtype=np.float64)[:, None]
    return np.log1p(E).reshape(-1)


def timestep_embedding(t: float, d_t: int) -> np.ndarray:
    """e(t).  Reading: sinusoidal, half = d_t/2, omega_i = 10000^(-i/half),
    e[i] = sin(t omega_i), e[half+i] = cos(t omega_i); t is the raw step index."""
    half = d_t // 2
    om = 10000.0 ** (-np.arange(half, dtype=np.float64) / half)
    return np.concatenate([np.sin(t * om), np.cos(t * om)])


def router_probabilities(g: np.ndarray, e: np.ndarray, W1, b1, W2, b2):
    """z = R([g; e(t)]) with R a two-layer MLP (reading: ReLU hidden layer), pi = softmax(z)."""
    x = np.concatenate([g, e])
    h = np.maximum(np.asarray(W1, np.float64) @ x + np.asarray(b1, np.float64), 0.0)
    z = np.asarray(W2, np.float64) @ h + np.asarray(b2, np.float64)
    return softmax_rows(z[None])[0], z


def head_quota(pi: np.ndarray, n_heads: int):
    """Heads per band from pi.  Reading: largest-remainder rounding of q_l = pi_l n_h (leftover
    heads to the largest fractional parts, ties to the lower band), in float64 like every other
    step here.  Returns (counts[3], margin) where margin is the smallest distance of the decision
    from flipping (a caller comparing with lower-precision arithmetic checks it first)."""
    q = np.asarray(pi, np.float64) * float(n_heads)
    base = np.floor(q).astype(np.int64)
    frac = q - np.floor(q)
    left = int(n_heads - base.sum())
    order = sorted(range(3), key=lambda l: (-frac[l], l))
    counts = base.copy()
    for l in order[:left]:
        counts[l] += 1
    margin = float(np.min(np.minimum(frac, 1.0 - frac)))
    if 0 < left < 3:
        fs = sorted(frac, reverse=True)
        margin = min(margin, float(fs[left - 1] - fs[left]))
    return counts, margin


def head_allocation(counts: Sequence[int]) -> np.ndarray:
    """Reading: heads [0, n_low) -> LOW, the next n_mid -> MID, the rest -> HIGH (one-hot masks)."""
    return np.concatenate([np.full(int(c), bit, dtype=np.uint8) for c, bit in zip(counts, _BITS)])


def router_parameter_count(n_in: int, hidden: int, n_out: int = 3) -> int:
    return n_in * hidden + hidden + hidden * n_out + n_out


def router_flops(n_in: int, hidden: int, n_out: int = 3) -> int:
    return 2 * (n_in * hidden) + 2 * (hidden * n_out)


# ----------------------------------------------------------------------------------------------
# Cross-band residual exchange ("Cross-band residual exchange")
# ----------------------------------------------------------------------------------------------
def summary_segments(n: int, m: int):
    """Reading: Pool = mean over m contiguous segments [a_j, e_j) of the band's working token
    list, a_j = floor(j n / m), e_j = max(a_j + 1, floor((j+1) n / m)) (so m > n repeats
    tokens instead of leaving a segment empty)."""
    return [((j * n) // m, max((j * n) // m + 1, ((j + 1) * n) // m)) for j in range(m)]


def summary_tokens(Y: np.ndarray, U: np.ndarray, m: int) -> np.ndarray:
    """S = U Pool(Y): m summary tokens [m, d] of one band of one head."""
    pooled = np.stack([Y[a:e].mean(axis=0) for a, e in summary_segments(Y.shape[0], m)])
    return pooled @ np.asarray(U, np.float64).T


def exchange(Y: np.ndarray, Z: np.ndarray) -> np.ndarray:
    """Y^ = Y + Attn_summary(Y, Z): every band token attends the 2m summary tokens of the other
    two bands.  Reading: plain softmax(Y Z^T / sqrt(d)) Z, no extra projections."""
    return Y + dense_attention(Y, Z, Z)


# ----------------------------------------------------------------------------------------------
# Whole layer for one sample
# ----------------------------------------------------------------------------------------------
def forward_sample(cfg, Q, K, V, weights, U, timestep: float, alloc=None, want_taps: bool = False):
    """The attention forward of one sample: Q, K, V [heads, T, H, W, d] -> out, same shape.

    Steps, in the paper's order: transform; band split; low compression; router (unless
    `alloc`, a uint8 band mask per head, is given); band operators on the bands in each head's
    mask and pass-through Y = V~ on the others (reading: a band a head is not allocated to
    keeps its value coefficients); summary tokens; exchange; recombination; inverse transform.
    Returns a dict with out, alloc, pi, z, margin, counters and (optionally) taps."""
    Q = np.asarray(Q, np.float64); K = np.asarray(K, np.float64); V = np.asarray(V, np.float64)
    n_h, T, H, W, d = Q.shape
    grid = (T, H, W)
    N = T * H * W
    members = band_members(grid, cfg.low_cut, cfg.mid_cut)
    sizes = [len(ix) for ix in members]
    kind = getattr(cfg, "transform", "dct")
    counters = {"pairs_low": 0, "pairs_mid": 0, "pairs_high": 0, "pairs_exchange": 0,
                "transform_macs": 0}

    Qb, Kb, Vb = [], [], []
    esum = np.zeros((3, d))
    for h in range(n_h):
        for X, dst in ((Q[h], Qb), (K[h], Kb), (V[h], Vb)):
            bands = split_bands(forward_transform(X, kind), members)
            dst.append(bands)
            esum += band_energy_sums(bands)
            counters["transform_macs"] += N * (T + H + W) * d

    g = pooled_statistics(esum, [3.0 * n_h * max(1, n) for n in sizes])
    pi = z = None
    margin = None
    if alloc is None:
        e = timestep_embedding(timestep, cfg.t_embed_dim)
        pi, z = router_probabilities(g, e, weights["W1"], weights["b1"], weights["W2"], weights["b2"])
        counts, margin = head_quota(pi, n_h)
        alloc = head_allocation(counts)
    alloc = np.asarray(alloc, dtype=np.uint8)

    out = np.empty_like(Q)
    taps = {"Qb": Qb, "Kb": Kb, "Vb": Vb, "Y": [], "S": [], "Yhat": [], "g": g}
    for h in range(n_h):
        mask = int(alloc[h])
        Y: List[np.ndarray] = [None, None, None]
        if mask & BAND_LOW and sizes[0]:
            q, k, v = (compress_low(x[h][0], cfg.r) for x in (Qb, Kb, Vb))
            Y[0] = dense_attention(q, k, v)
            counters["pairs_low"] += q.shape[0] * k.shape[0]
        else:
            Y[0] = Vb[h][0]
        if mask & BAND_MID and sizes[1]:
            Y[1], pairs = mid_operator(Qb[h][1], Kb[h][1], Vb[h][1], cfg.b, cfg.s,
                                       pattern=getattr(cfg, "mid_pattern", "strided"))
            counters["pairs_mid"] += pairs
        else:
            Y[1] = Vb[h][1]
        if mask & BAND_HIGH and sizes[2]:
            Y[2], pairs = high_operator(Qb[h][2], Kb[h][2], Vb[h][2], cfg.R)
            counters["pairs_high"] += pairs
        else:
            Y[2] = Vb[h][2]

        if cfg.m > 0:
            S = [summary_tokens(Y[l], U[l], cfg.m) if Y[l].shape[0] else np.zeros((0, d)) for l in range(3)]
            Yhat = []
            for l in range(3):
                Z = np.concatenate([S[o] for o in range(3) if o != l])
                if Y[l].shape[0] and Z.shape[0]:
                    Yhat.append(exchange(Y[l], Z))
                    counters["pairs_exchange"] += Y[l].shape[0] * Z.shape[0]
                else:
                    Yhat.append(Y[l])
        else:
            S = [np.zeros((0, d))] * 3
            Yhat = list(Y)

        spec = np.zeros((N, d))
        low = Yhat[0]
        if low.shape[0] != sizes[0]:
            low = decompress_low(low, cfg.r, sizes[0])
        for l, rows in enumerate((low, Yhat[1], Yhat[2])):
            spec[members[l]] = rows
        out[h] = inverse_transform(spec.reshape(T, H, W, d), kind)
        counters["transform_macs"] += N * (T + H + W) * d
        if want_taps:
            taps["Y"].append(Y); taps["S"].append(S); taps["Yhat"].append(Yhat)

    res = {"out": out, "alloc": alloc, "pi": pi, "z": z, "margin": margin, "g": g,
           "counters": counters, "sizes": sizes}
    if want_taps:
        res["taps"] = taps
    return res


# ----------------------------------------------------------------------------------------------
# The layer with its projections ("Setup and notation", "Reconstruction")
# ----------------------------------------------------------------------------------------------
def round_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bf16 (ties to even) of float64 values, as float64: the storage type of Q, K, V."""
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    u = x32.view(np.uint32)
    u = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return u.view(np.float32).astype(np.float64)


def project_qkv(X: np.ndarray, Wqkv: np.ndarray, heads: int, grid, bf16_storage: bool = True):
    """"Linear projections produce Q_h, K_h, V_h": X[N, D] (token-major, D = heads d) times
    W_q, W_k, W_v [D, D] (y = x W); output column h d + c is channel c of head h.  Returns Q, K, V as
    [heads, T, H, W, d].  With bf16_storage the results are rounded to bf16, the type in which the
    attention path receives them (reading: the benchmark fixes bf16 Q/K/V)."""
    X = np.asarray(X, np.float64)
    N, D = X.shape
    d = D // heads
    T, H, W = grid
    out = []
    for l in range(3):
        Y = X @ np.asarray(Wqkv[l], np.float64)                       # [N, D]
        if bf16_storage:
            Y = round_bf16(Y)
        out.append(Y.reshape(N, heads, d).transpose(1, 0, 2).reshape(heads, T, H, W, d))
    return out


def project_out(A: np.ndarray, Wo: np.ndarray) -> np.ndarray:
    """"Head outputs are concatenated and projected": A[heads, T, H, W, d] -> [N, D] (column h d + c
    = channel c of head h) times W_o [D, D]."""
    heads, T, H, W, d = A.shape
    cat = np.asarray(A, np.float64).reshape(heads, T * H * W, d).transpose(1, 0, 2).reshape(T * H * W, heads * d)
    return cat @ np.asarray(Wo, np.float64)


def forward_projected_sample(cfg, X, Wqkv, Wo, weights, U, timestep: float, alloc=None, bf16_storage: bool = True):
    """The attention layer of one sample from its input X[N, D]: projections, forward_sample, output
    projection.  The attention output is rounded to bf16 before the output projection when the path
    stores it in bf16."""
    Q, K, V = project_qkv(X, Wqkv, cfg.heads, (cfg.T, cfg.H, cfg.W), bf16_storage)
    res = forward_sample(cfg, Q, K, V, weights, U, timestep, alloc=alloc)
    A = round_bf16(res["out"]) if bf16_storage else res["out"]
    res["attention_out"] = res["out"]
    res["out"] = project_out(A, Wo)
    return res


# ----------------------------------------------------------------------------------------------
# Cost model ("Complexity Analysis")
# ----------------------------------------------------------------------------------------------
def paper_interactions(n_low_bar: float, n_mid: float, k_mid: float, n_high: float, w: float) -> float:
    """I_FreqFormer = N_low_bar^2 + N_mid k_mid + N_high w."""
    return n_low_bar ** 2 + n_mid * k_mid + n_high * w


def paper_attention_cost_reference(N: float, d_k: float) -> float:
    """C_attn with the reference configuration (N_low_bar = N/32, N_mid = 0.375 N, N_high = 0.5 N,
    k_mid = 256, w = 64)."""
    return paper_interactions(0.03125 * N, 0.375 * N, 256, 0.5 * N, 64) * d_k


def dense_attention_flops(N: int, d_k: int) -> int:
    """Interactions N^2 times 2 d_k ("Exact computed FLOPs")."""
    return 2 * d_k * N * N


def mid_interactions(n_mid: int, b: int, s: int, pattern: str = "strided") -> int:
    """Scored pairs of the mid band.  Strided: sum over residue classes of (tokens in the
    class)^2.  Anchor: every token sees the anchor blocks, and its own block if that is none."""
    nb = -(-n_mid // b)
    size = lambda J: min(b, n_mid - J * b)
    if pattern == "anchor":
        anchors = sum(size(J) for J in range(nb) if J % s == s - 1)
        return sum(size(J) * (anchors + (0 if J % s == s - 1 else size(J))) for J in range(nb))
    total = 0
    for c in range(min(s, nb)):
        n_c = sum(min(b, n_mid - J * b) for J in range(c, nb, s))
        total += n_c * n_c
    return total


def high_interactions(n_high: int, R: int) -> int:
    """Sum over p of the clipped window size."""
    return sum(min(n_high - 1, p + R) - max(0, p - R) + 1 for p in range(n_high))
