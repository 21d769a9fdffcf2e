"""Seeded synthetic input generators shared by the tests, the benchmark and the smoke check.

This module only *draws data* (token-id streams, bf16 matrices, uniforms, temperatures).
It contains none of the method's arithmetic (no histogram, selection, projection, softmax or
sampling), so the CPU oracle and the CUDA library can both be fed from it without sharing code.

All generators are torch based so the same function serves small CPU cases and corpus-scale
cases drawn directly in device memory.  A (seed, device-type) pair fixes the stream; CPU and
CUDA streams differ, which is fine because an array is drawn once and then handed, as data,
to both sides of a comparison.

Shapes and distributions follow the workloads the paper evaluates on (Llama-3 vocabulary of
128256 ids, hidden sizes 3072 / 4096, a heavy-tailed token-frequency profile as in the paper's
Figure 1 and introduction), stood in for by Zipf draws over a seeded permutation of the ids.
"""
from __future__ import annotations

import torch

LLAMA3_VOCAB = 128256


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def zipf_ids(n: int, V: int, s: float, seed: int, noise_frac: float = 0.0,
             device="cpu", chunk: int = 1 << 24) -> torch.Tensor:
    """n int32 token ids: rank r ~ Zipf(s) on {1..V} by inverse CDF, id = perm[r-1] with perm a
    seeded shuffle of [0,V); each element is independently replaced, with probability
    `noise_frac`, by a uniform id on [0,V).  Drawn in chunks to bound temporary memory."""
    device = torch.device(device)
    g = _gen(seed, device)
    perm = torch.randperm(V, generator=g, device=device).to(torch.int32)
    ranks = torch.arange(1, V + 1, dtype=torch.float64, device=device)
    cdf = torch.cumsum(ranks.pow(-float(s)), 0)
    cdf = cdf / cdf[-1]
    out = torch.empty(n, dtype=torch.int32, device=device)
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        u = torch.rand(m, generator=g, device=device, dtype=torch.float64)
        r = torch.searchsorted(cdf, u).clamp_(max=V - 1)
        ids = perm[r]
        if noise_frac > 0.0:
            coin = torch.rand(m, generator=g, device=device)
            noise = torch.randint(0, V, (m,), generator=g, device=device, dtype=torch.int32)
            ids = torch.where(coin < noise_frac, noise, ids)
        out[lo:lo + m] = ids
    return out


def gaussian_bf16(shape, std: float, seed: int, device="cpu") -> torch.Tensor:
    """N(0, std^2) drawn in fp32 and rounded to bf16 (round-to-nearest-even)."""
    device = torch.device(device)
    g = _gen(seed, device)
    x = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    return (x * float(std)).to(torch.bfloat16)


def uniforms(shape, seed: int, device="cpu") -> torch.Tensor:
    """fp32 uniforms of the form (2*x+1) * 2^-24 with x a 23-bit integer: exactly representable
    and strictly inside (0,1), so no clamping rule is ever exercised by accident."""
    device = torch.device(device)
    g = _gen(seed, device)
    x = torch.randint(0, 1 << 23, shape, generator=g, device=device, dtype=torch.int32)
    return (2.0 * x.to(torch.float32) + 1.0) * float(2.0 ** -24)


def temperatures(B: int, lo: float, hi: float, seed: int, device="cpu") -> torch.Tensor:
    """B per-row fp32 temperatures uniform on [lo, hi]; lo == hi gives a constant vector."""
    device = torch.device(device)
    if lo == hi:
        return torch.full((B,), float(lo), dtype=torch.float32, device=device)
    g = _gen(seed, device)
    return lo + (hi - lo) * torch.rand(B, generator=g, device=device, dtype=torch.float32)


def bf16_bits(t: torch.Tensor) -> torch.Tensor:
    """View a bf16 tensor as its raw 16-bit patterns (int16 storage, same memory)."""
    assert t.dtype == torch.bfloat16
    return t.view(torch.int16)


def draft_trees(S: int, N: int, width: int, vocab: int, p_match: float, seed: int):
    """S random draft trees of N nodes each, as CPU int32 tensors, plus a stand-in for the target's
    greedy tokens: (token [S,N], parent [S,N], target [S,N+1]).

    Node i hangs off a uniformly drawn earlier node (or off the committed prefix, parent -1) that
    still has fewer than `width` children; siblings carry distinct ids, as a top-k expansion
    gives.  target[s, j] is, with probability p_match, the id of a uniformly drawn child of node
    j-1 (so that walks of some depth occur) and a fresh id otherwise.  Data only: no acceptance
    logic lives here."""
    assert width <= vocab
    g = _gen(seed, "cpu")
    token = torch.empty(S, N, dtype=torch.int32)
    parent = torch.empty(S, N, dtype=torch.int32)
    target = torch.randint(0, vocab, (S, N + 1), generator=g, dtype=torch.int32)
    for s in range(S):
        kids = [[] for _ in range(N + 1)]                 # kids[j] = children of node j-1
        for i in range(N):
            open_ = [j for j in range(i + 1) if len(kids[j]) < width]
            j = open_[int(torch.randint(0, len(open_), (1,), generator=g))]
            kids[j].append(i)
            parent[s, i] = j - 1
        for j in range(N + 1):
            if kids[j]:
                ids = torch.randperm(vocab, generator=g)[:len(kids[j])].to(torch.int32)
                token[s, kids[j]] = ids
                if float(torch.rand((), generator=g)) < p_match:
                    target[s, j] = ids[int(torch.randint(0, len(ids), (1,), generator=g))]
    return token, parent, target


def head_candidates(B: int, topk: int, vocab: int, seed: int, tie_frac: float = 0.0):
    """Stand-in for the head's per-row top-k output, as CPU tensors: ids int32 [B,topk] (distinct per
    row) and log-probs fp32 [B,topk], descending per row and <= 0 (log of sorted Dirichlet-like
    masses).  tie_frac > 0 rounds log-probs to a coarse grid so that equal scores occur."""
    g = _gen(seed, "cpu")
    ids = torch.stack([torch.randperm(vocab, generator=g)[:topk] for _ in range(B)]).to(torch.int32)
    mass = torch.rand(B, topk + 1, generator=g, dtype=torch.float64) ** 3 + 1e-6
    mass = mass / mass.sum(dim=1, keepdim=True)
    lp = torch.log(mass[:, :topk]).sort(dim=1, descending=True).values.to(torch.float32)
    if tie_frac > 0:
        coarse = torch.round(lp * 2) / 2
        pick = torch.rand(B, topk, generator=g) < tie_frac
        lp = torch.where(pick, coarse, lp).sort(dim=1, descending=True).values
    return ids, lp.clamp(max=0.0)
