"""Seeded synthetic inputs shaped like the paper's workloads (Section 5.1, Table 2).

This module only makes data: key streams, integer sampling weights, training
pairs / triples / matrix cells and start values.  It holds none of the store's
arithmetic and is the one module that both the CPU oracle's tests and the CUDA
path's callers use, so that both sides always see the very same arrays.

Everything is generated with torch on the device asked for (CPU by default) from
an explicit seed.  The CPU and CUDA generators give different streams; what
matters is that one array is generated once and handed to both sides.

Zipf(s) over n ranks: rank r (1-based) has weight r^-s.  Rank r maps to key
``(A * (r-1) + B) mod n`` with A coprime to n, so hot keys are spread over the
table instead of sitting in adjacent rows.
"""
from __future__ import annotations

import math

import numpy as np
import torch


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def affine_bijection(n: int, seed: int = 0):
    """(A, B) with gcd(A, n) = 1: r -> (A*r + B) mod n permutes [0, n)."""
    a = (0x9E3779B97F4A7C15 ^ (seed * 0xD1342543DE82EF95)) % max(n, 1)
    a |= 1
    while math.gcd(a, n) != 1:
        a += 2
    b = (0xC2B2AE3D27D4EB4F * (seed + 1)) % max(n, 1)
    return a % max(n, 1) if n > 1 else 0, b


def rank_to_key(ranks0: torch.Tensor, n: int, seed: int = 0, spread: bool = True) -> torch.Tensor:
    """Map 0-based ranks to keys in [0, n)."""
    if not spread or n <= 2:
        return ranks0
    a, b = affine_bijection(n, seed)
    assert n < (1 << 31), "the affine map is computed in int64"
    return ((ranks0.to(torch.int64) * a) % n + b) % n


def zipf_cdf(n: int, s: float, device="cpu") -> torch.Tensor:
    w = torch.arange(1, n + 1, device=device, dtype=torch.float64).pow_(-s)
    cdf = torch.cumsum(w, 0)
    return cdf / cdf[-1]


def zipf_ranks(num: int, n: int, s: float, seed: int, device="cpu", cdf=None) -> torch.Tensor:
    """`num` iid 0-based ranks from Zipf(s) over n ranks (s = 0 is uniform)."""
    g = _gen(seed, device)
    if s == 0.0:
        return torch.randint(0, n, (num,), generator=g, device=device, dtype=torch.int64)
    if cdf is None:
        cdf = zipf_cdf(n, s, device)
    u = torch.rand(num, generator=g, device=device, dtype=torch.float64)
    return torch.searchsorted(cdf, u).clamp_(max=n - 1)


def zipf_keys(num: int, n: int, s: float, seed: int, device="cpu", spread=True, cdf=None, key_base=0) -> torch.Tensor:
    """`num` keys in [key_base, key_base + n), frequency ~ Zipf(s), as int64 (cast to uint32 by the caller)."""
    return rank_to_key(zipf_ranks(num, n, s, seed, device, cdf), n, seed=1, spread=spread) + key_base


def zipf_key_of_rank(n: int, device="cpu", spread=True) -> torch.Tensor:
    """key_of_rank[r] for every rank: the true-frequency order of a zipf_keys stream."""
    return rank_to_key(torch.arange(n, device=device, dtype=torch.int64), n, seed=1, spread=spread)


def integer_weights(counts: torch.Tensor, power: float = 0.75, scale_bits: int = 8) -> torch.Tensor:
    """Integer sampling weights w = max(1, floor(count^power * 2^scale_bits)) (word2vec's smoothed unigram)."""
    w = torch.floor(counts.to(torch.float64).pow(power) * float(1 << scale_bits)).clamp_(min=1, max=2 ** 32 - 1)
    return w.to(torch.int64)


def zipf_integer_weights(n: int, s: float, device="cpu", spread=True, top: int = 1 << 20) -> torch.Tensor:
    """Integer weights, indexed by key, of a Zipf(s) target: weight of rank r is max(1, floor(top * r^-s))."""
    r = torch.arange(1, n + 1, device=device, dtype=torch.float64)
    w = torch.floor(r.pow(-s) * float(top)).clamp_(min=1).to(torch.int64)
    out = torch.empty_like(w)
    out[zipf_key_of_rank(n, device, spread)] = w
    return out


def normal_init(num_keys: int, value_len: int, std: float, seed: int) -> np.ndarray:
    """N(0, std) start values, generated once on the host and given to both sides."""
    rng = np.random.default_rng(seed)
    return rng.normal(0.0, std, size=(num_keys, value_len)).astype(np.float32)


def skipgram_pairs(tokens: torch.Tensor, window: int = 5):
    """(centre, context) word pairs of a token stream: every position paired with the `window`
    positions on each side, clipped at the ends, in stream order."""
    n = tokens.numel()
    offs = torch.tensor([d for d in range(-window, window + 1) if d != 0], device=tokens.device)
    pos = torch.arange(n, device=tokens.device).unsqueeze(1) + offs.unsqueeze(0)
    ok = (pos >= 0) & (pos < n)
    centre = tokens.unsqueeze(1).expand(-1, offs.numel())[ok]
    context = tokens[pos.clamp(0, n - 1)][ok]
    return centre, context


def sgns_batch_stream(vocab: int, num_tokens: int, s: float, seed: int, device="cpu", window: int = 5):
    """Tokens ~ Zipf(s) over `vocab` words; returns (centre keys, context keys, word counts).
    Input-table key of word v is v, output-table key is vocab + v."""
    tokens = zipf_keys(num_tokens, vocab, s, seed, device)
    counts = torch.bincount(tokens, minlength=vocab)
    c, o = skipgram_pairs(tokens, window)
    return c, o + vocab, counts


def kge_triples(num: int, entities: int, relations: int, s_ent: float, s_rel: float, seed: int, device="cpu"):
    """(head, relation, tail) keys: entities in [0, E), relation keys in [E, E + relations)."""
    h = zipf_keys(num, entities, s_ent, seed * 3 + 0, device)
    t = zipf_keys(num, entities, s_ent, seed * 3 + 1, device)
    r = zipf_keys(num, relations, s_rel, seed * 3 + 2, device, key_base=entities)
    return h, r, t


def columns_in_visiting_order(num: int, cols: int, s: float, total_cells: int, seed: int, device="cpu") -> torch.Tensor:
    """Column ranks (0-based) of the first `num` cells of a data set of `total_cells` cells that is visited column by
    column (Section 5.1, matrix factorization): the columns come in random order, each with all of its cells, and a
    column of rank r holds max(1, round(total_cells * r^-s / sum_r r^-s)) cells."""
    g = _gen(seed, device)
    order = torch.randperm(cols, generator=g, device=device)
    w = torch.arange(1, cols + 1, device=device, dtype=torch.float64).pow_(-s)
    cells = torch.round(w / w.sum() * float(total_cells)).clamp_(min=1).to(torch.int64)[order]
    upto = int(torch.searchsorted(torch.cumsum(cells, 0), torch.tensor([num], device=device)).item()) + 1
    return torch.repeat_interleave(order[:upto], cells[:upto])[:num]


def mf_cells(num: int, rows: int, cols: int, s: float, rank: int, noise: float, seed: int, device="cpu",
             factor_seed: int = 1234, by_column_of: int = 0):
    """Revealed cells of a rows x cols matrix: indices ~ Zipf(s), value = <true row factor, true column
    factor> + N(0, noise).  True factor entries are N(0, rank^-1/4), made on the fly from a hash of
    (index, component) so that no full factor table is needed.  Row keys [0, rows), column keys
    [rows, rows + cols).  by_column_of = T > 0: the cells are the first `num` of a T-cell data set in
    column-by-column visiting order (see columns_in_visiting_order) instead of independent draws."""
    i = zipf_keys(num, rows, s, seed * 2 + 0, device)
    if by_column_of:
        j = rank_to_key(columns_in_visiting_order(num, cols, s, by_column_of, seed * 2 + 1, device), cols, seed=1)
    else:
        j = zipf_keys(num, cols, s, seed * 2 + 1, device)
    g = _gen(seed + 77, device)
    sigma = float(rank) ** -0.25

    def mix(z):
        # 64-bit finaliser (multiply / xor-shift rounds, wrapping int64 arithmetic): neighbouring inputs give
        # unrelated outputs, so the components of a factor row are independent
        for mul in (-4658895280553007687, -7723592293110705685):     # 0xBF58476D1CE4E5B9, 0x94D049BB133111EB as int64
            z = (z ^ ((z >> 30) & 0x3FFFFFFFF)) * mul
        return z ^ ((z >> 31) & 0x1FFFFFFFF)

    def factor(idx, salt):
        comp = torch.arange(rank, device=device, dtype=torch.int64).unsqueeze(0)
        z = mix(idx.unsqueeze(1) * 1000003 + comp * 7919 + (salt * 104729 + factor_seed))
        z2 = mix(z + 0x632BE5AB)
        u1 = ((z >> 11) & ((1 << 52) - 1)).to(torch.float64) / float(1 << 52) + 2.0 ** -53
        u2 = ((z2 >> 11) & ((1 << 52) - 1)).to(torch.float64) / float(1 << 52)
        return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos(2.0 * math.pi * u2) * sigma

    x = torch.empty(num, device=device, dtype=torch.float64)
    step = 1 << 18
    for a in range(0, num, step):
        b = min(num, a + step)
        x[a:b] = (factor(i[a:b], 0) * factor(j[a:b], 1)).sum(1)
    x = x + torch.randn(num, generator=g, device=device, dtype=torch.float64) * noise
    return i, j + rows, x.to(torch.float32)


def u32(t: torch.Tensor) -> np.ndarray:
    """Host uint32 copy of an integer tensor of keys."""
    return t.detach().cpu().numpy().astype(np.uint32)
