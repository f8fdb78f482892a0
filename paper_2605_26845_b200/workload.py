"""Seeded synthetic demand matrices (inputs only; none of the method's arithmetic).

The paper evaluates on routing traces of Mixtral 8x7B, Mixtral 8x22B and
DeepSeek-MoE-16B over two prompt datasets (Sec. 4); neither the traces nor the
datasets are available here, so token-routing matrices with the same
character (few heavy pairs, many light or empty ones, unequal row and column
sums: Sec. 2.2) are drawn from
a stated recipe instead. D[b, i, j] is the number of (token, expert) selections
that rank i sends to rank j in all-to-all b; the diagonal (tokens that stay on
their own rank) is kept.

Recipe, per matrix b and source rank i:
  1. expert popularity p over E experts (Zipf with exponent s over a popularity
     order that is fixed or reshuffled per matrix; or a Dirichlet draw per
     source rank with a few "hot" experts boosted);
  2. inclusion probabilities q_e = min(1, c * p_e) with c chosen so that
     sum_e q_e = top_k (an expert is picked at most once per token);
  3. every one of `tokens` tokens picks top_k DISTINCT experts by systematic
     sampling: one uniform offset u per token, expert e is picked when one of
     u, u+1, ..., u+top_k-1 falls into [Q_{e-1}, Q_e), Q = cumsum(q). The
     per-expert counts over all tokens are drawn exactly from that process
     through the multinomial law of the offsets over the arcs between the
     fractional parts of Q (a chain of binomials), without a per-token loop;
  4. D[b, i, owner(e)] += count_e, owner = the rank hosting expert e.
Hence every row sums to tokens * top_k exactly and no expert receives more
than `tokens` selections from one rank.

All randomness comes from numpy's Philox generator keyed by (seed, config,
chunk); the same array is handed to the CUDA library and to its CPU checker.
"""
from __future__ import annotations

import numpy as np

SEED = 260526845

# Link / compute model used with every configuration: 14336 B per token (bf16
# hidden size 7168), 400 Gb/s ports, 10 us reconfiguration, expert batch cost
# 20 us + 0.5 ns per token.
DEFAULT_MODEL = dict(bytes_per_token=14336, link_gbps=400, reconfig_ns=10_000,
                     expert_fixed_ns=20_000, expert_ps_per_token=500, expert_knee_tokens=0)
# The two constants the paper gives for its profiled expert-compute curve (Fig. 1, Sec. 3.1): about
# 250 us up to about 256 tokens, linear beyond (the slope is not stated; the affine model's is kept),
# with the 10 ns reconfiguration delay of its evaluation (Sec. 4.1).
PROFILED_MODEL = dict(DEFAULT_MODEL, reconfig_ns=10, expert_fixed_ns=250_000, expert_knee_tokens=256)

CONFIGS = {
    1: dict(N=8, B=64, tokens=4096, experts=8, top_k=2, kind="zipf", s=1.2, owner="block",
            reshuffle=False, k_max=(8,)),
    2: dict(N=16, B=1024, tokens=8192, experts=64, top_k=6, kind="zipf", s=1.0, owner="random",
            reshuffle=False, k_max=(4, 16)),
    3: dict(N=64, B=4096, tokens=16384, experts=256, top_k=8, kind="zipf", s=1.2, owner="block",
            reshuffle=True, k_max=(8, 16, 64)),
    4: dict(N=128, B=1024, tokens=8192, experts=512, top_k=8, kind="dirichlet", alpha=0.3,
            hot_prob=0.05, hot_factor=10.0, owner="block", k_max=(16, 32, 128)),
    5: dict(N=256, B=256, tokens=4096, experts=1024, top_k=8, kind="zipf", s=1.4, owner="block",
            reshuffle=True, allowed_prob=0.4, k_max=(4, 8, 16, 32, 256),
            expert_fixed_ns=(5_000, 20_000, 80_000)),
}


def bvn_capacity(N: int) -> int:
    """Output capacity that always holds a complete Birkhoff decomposition."""
    return N * N - 2 * N + 2


def _rng(seed, *key):
    return np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, *key])))


def _inclusion(p, top_k):
    """q = min(1, c p) with sum q = top_k, row-wise. p: [..., E], rows sum to 1."""
    capped = np.zeros(p.shape, bool)
    for _ in range(top_k + 1):
        free_mass = np.where(capped, 0.0, p).sum(-1, keepdims=True)
        c = (top_k - capped.sum(-1, keepdims=True)) / np.maximum(free_mass, 1e-300)
        new = (~capped) & (c * p >= 1.0)
        if not new.any():
            break
        capped |= new
    return np.where(capped, 1.0, np.minimum(c * p, 1.0))


def _systematic_counts(q, tokens, top_k, rng):
    """Per-expert selection counts of `tokens` tokens, each taking top_k distinct experts by
    systematic sampling with inclusion probabilities q. q: [R, E] -> int64 [R, E]."""
    R, E = q.shape
    Q = np.cumsum(q, axis=-1)
    Q[:, -1] = top_k
    whole = np.floor(Q)
    frac = Q - whole
    frac[:, -1] = 0.0
    order = np.argsort(frac, axis=-1, kind="stable")
    fs = np.take_along_axis(frac, order, axis=-1)            # sorted break points in [0, 1)
    arc = np.diff(fs, axis=-1, append=1.0)                   # arc a = [fs_a, fs_{a+1}); before fs_0: length fs_0
    # offsets falling below each sorted break point: chain of binomials over the arcs
    below = np.zeros((R, E), np.int64)
    rem = np.full(R, tokens, np.int64)
    mass = np.ones(R)
    n0 = rng.binomial(rem, np.clip(fs[:, 0], 0.0, 1.0))      # arc before the first break point
    rem = rem - n0
    mass = mass - fs[:, 0]
    run = n0.copy()
    for a in range(E):
        below[:, a] = run
        if a == E - 1:
            break
        pa = np.clip(arc[:, a] / np.maximum(mass, 1e-300), 0.0, 1.0)
        n = rng.binomial(rem, pa)
        rem = rem - n
        mass = mass - arc[:, a]
        run = run + n
    G = np.empty((R, E), np.int64)
    np.put_along_axis(G, order, below, axis=-1)              # G[e] = #offsets < frac(Q_e)
    F = tokens * whole.astype(np.int64) + G                  # selections landing below Q_e
    F[:, -1] = tokens * top_k
    return np.diff(F, axis=-1, prepend=0)


def _popularity(cfg, nb, rng):
    """Expert probabilities per (matrix, source rank): [nb, N or 1, E]."""
    N, E = cfg["N"], cfg["experts"]
    if cfg["kind"] == "zipf":
        base = np.arange(1, E + 1, dtype=np.float64) ** (-cfg["s"])
        if cfg.get("reshuffle"):
            ranks = rng.permuted(np.tile(np.arange(E), (nb, 1)), axis=1)
            p = base[ranks][:, None, :]
        else:
            p = np.broadcast_to(base, (nb, 1, E)).copy()
    else:
        p = rng.standard_gamma(cfg["alpha"], size=(nb, N, E))
        p = np.maximum(p, 1e-300)
        hot = rng.random((nb, 1, E)) < cfg["hot_prob"]
        p = p / p.sum(-1, keepdims=True)
        p = np.where(hot, p * cfg["hot_factor"], p)
    if "allowed_prob" in cfg:
        per_rank = E // N
        allow = rng.random((nb, N, N)) < cfg["allowed_prob"]
        idx = np.arange(N)
        allow[:, idx, idx] = True
        need = -(-cfg["top_k"] // per_rank)                  # ranks needed to host top_k experts
        for extra in range(1, need + 1):                     # guard: enough allowed destinations
            short = allow.sum(-1) < need
            allow[:, idx, (idx + extra) % N] |= short
        p = np.where(np.repeat(allow, per_rank, axis=-1), np.broadcast_to(p, (nb, N, E)), 0.0)
    return p / p.sum(-1, keepdims=True)


def make_demand(config: int, B: int | None = None, seed: int = SEED, chunk: int = 256) -> np.ndarray:
    """int32 [B, N, N] demand matrices of one of the five configurations."""
    cfg = CONFIGS[config]
    N, E, tokens, top_k = cfg["N"], cfg["experts"], cfg["tokens"], cfg["top_k"]
    B = cfg["B"] if B is None else B
    out = np.zeros((B, N, N), np.int32)
    per_rank = E // N
    for c0 in range(0, B, chunk):
        nb = min(chunk, B - c0)
        rng = _rng(seed, config, c0 // chunk)
        p = _popularity(cfg, nb, rng)
        q = _inclusion(p, top_k)
        q = np.broadcast_to(q, (nb, N, E)).reshape(nb * N, E)
        cnt = _systematic_counts(q, tokens, top_k, rng).reshape(nb, N, E)
        if cfg["owner"] == "block":
            out[c0:c0 + nb] = cnt.reshape(nb, N, N, per_rank).sum(-1)
        else:
            owner = rng.permuted(np.tile(np.arange(E) // per_rank, (nb, 1)), axis=1)   # [nb, E]
            d = np.zeros((nb, N, N), np.int64)
            bi = np.arange(nb)[:, None, None]
            ii = np.arange(N)[None, :, None]
            np.add.at(d, (bi, ii, owner[:, None, :]), cnt)
            out[c0:c0 + nb] = d
    return out


def random_matrices(B, N, seed, kind="uniform", high=1000, zero_frac=0.0):
    """Small seeded test matrices. kinds: uniform, ties ({0,1,2}-valued), sparse."""
    rng = _rng(seed, N, B)
    if kind == "ties":
        d = rng.integers(0, 3, size=(B, N, N))
    else:
        d = rng.integers(0, high + 1, size=(B, N, N))
    if zero_frac > 0:
        d = np.where(rng.random((B, N, N)) < zero_frac, 0, d)
    return d.astype(np.int32)


def structured_cases(N, m=7):
    """Named special matrices with closed-form decompositions: dict name -> int32 [N, N]."""
    idx = np.arange(N)
    shift = np.zeros((N, N), np.int32)
    shift[idx, (idx + 1) % N] = m                            # scaled permutation
    hot = np.zeros((N, N), np.int32)
    hot[:, 0] = m                                            # incast on rank 0
    diag = np.zeros((N, N), np.int32)
    diag[idx, idx] = idx + 1
    return {
        "zero": np.zeros((N, N), np.int32),
        "scaled_permutation": shift,
        "uniform": np.full((N, N), m, np.int32),
        "hot_column": hot,
        "diagonal": diag,
    }
