"""Python face of the CPU oracle (oracle/vt_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
product package never does.  It compiles the C file with gcc on first use and calls it through
ctypes on numpy arrays.  Nothing here touches CUDA.

Parity pins: see the header of vt_oracle.c -- pinned to definitions, invariants, library special
cases and brute force by the CPU tests; parity with paper-printed values is unpinned for the head
and the vocabulary build because the paper prints no numeric example for them; `mbsu` is pinned to
the (block efficiency, speed-up) pairs of the paper's Table 1.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from ctypes import POINTER, c_double, c_float, c_int, c_int32, c_int64, c_uint16, c_uint64, c_void_p

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vt_oracle.c")
_LIB = os.path.join(_HERE, "libvt_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP only parallelises independent vocabulary rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_softmax_row.restype = c_double
        _lib.orc_gumbel_row.restype = c_int32
        _lib.orc_max_threads.restype = c_int
    return _lib


def _p(a, ty):
    return a.ctypes.data_as(POINTER(ty)) if a is not None else None


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _bits(a) -> np.ndarray:
    """Accept raw bf16 bit patterns as uint16/int16 numpy arrays."""
    a = np.ascontiguousarray(a)
    if a.dtype == np.int16:
        a = a.view(np.uint16)
    assert a.dtype == np.uint16, "bf16 data must be passed as 16-bit patterns"
    return a


def max_threads() -> int:
    return int(_load().orc_max_threads())


def set_threads(t: int) -> None:
    _load().orc_set_threads(c_int(int(t)))


def decode_bf16(x) -> np.ndarray:
    x = _bits(x)
    out = np.empty(x.shape, dtype=np.float64)
    _load().orc_decode_bf16(_p(x, c_uint16), c_int64(x.size), _p(out, c_double))
    return out


def histogram(ids, V: int, counts=None):
    """Algorithm 1.  Returns (counts uint64 [V], n_bad).  Passing `counts` accumulates into it."""
    ids = _c(ids, np.int32)
    acc = counts is not None
    if not acc:
        counts = np.empty(V, dtype=np.uint64)
    assert counts.dtype == np.uint64 and counts.size == V and counts.flags.c_contiguous
    bad = c_uint64(0)
    _load().orc_histogram(_p(ids, c_int32), c_int64(ids.size), c_int32(V), _p(counts, c_uint64),
                          c_int(1 if acc else 0), ctypes.byref(bad))
    return counts, int(bad.value)


def select_topk(counts, K: int):
    """Eq. 1 (token selection).  Returns (map int32 [K] in rank order, inv_map int32 [V])."""
    counts = _c(counts, np.uint64)
    V = counts.size
    m = np.empty(K, dtype=np.int32)
    inv = np.empty(V, dtype=np.int32)
    rc = _load().orc_select_topk(_p(counts, c_uint64), c_int32(V), c_int32(K), _p(m, c_int32),
                                 _p(inv, c_int32))
    if rc:
        raise ValueError("select_topk: invalid V/K")
    return m, inv


def select_topp(counts, p: float):
    """Top-P variant of the selection (Method section).  Returns (K, map int32 [V] full ranking, inv_map [V])."""
    counts = _c(counts, np.uint64)
    V = counts.size
    m = np.empty(V, dtype=np.int32)
    inv = np.empty(V, dtype=np.int32)
    _load().orc_select_topp.restype = c_int32
    K = _load().orc_select_topp(_p(counts, c_uint64), c_int32(V), c_double(float(p)), _p(m, c_int32), _p(inv, c_int32))
    if K < 0:
        raise ValueError("select_topp: invalid arguments")
    return int(K), m, inv


def select_minfreq(counts, min_count: int):
    """Minimum-frequency variant of the selection (Method section).  Returns (K, map [V], inv_map [V])."""
    counts = _c(counts, np.uint64)
    V = counts.size
    m = np.empty(V, dtype=np.int32)
    inv = np.empty(V, dtype=np.int32)
    _load().orc_select_minfreq.restype = c_int32
    K = _load().orc_select_minfreq(_p(counts, c_uint64), c_int32(V), c_uint64(int(min_count)), _p(m, c_int32),
                                   _p(inv, c_int32))
    if K < 0:
        raise ValueError("select_minfreq: invalid arguments")
    return int(K), m, inv


def build_vocab(ids, V: int, K: int):
    counts, bad = histogram(ids, V)
    m, inv = select_topk(counts, K)
    return m, inv, counts, bad


def trim_head(W_full, map_):
    """Eq. 1 (head restriction).  W_full: bf16 bit patterns [V,d]; returns bit patterns [K,d]."""
    W_full = _bits(W_full)
    map_ = _c(map_, np.int32)
    K, d = map_.size, W_full.shape[1]
    out = np.empty((K, d), dtype=np.uint16)
    _load().orc_trim_head(_p(W_full, c_uint16), _p(map_, c_int32), c_int32(K), c_int32(d),
                          _p(out, c_uint16))
    return out


def logits(h, W) -> np.ndarray:
    """fp64 projection of bf16 rows h [B,d] onto bf16 head W [K,d]; returns [B,K]."""
    h, W = _bits(h), _bits(W)
    B, d = h.shape
    K = W.shape[0]
    assert W.shape[1] == d
    out = np.empty((B, K), dtype=np.float64)
    _load().orc_logits(_p(h, c_uint16), _p(W, c_uint16), c_int32(B), c_int32(K), c_int32(d),
                       _p(out, c_double))
    return out


def softmax_row(logit, T: float):
    """Returns (z = logit/T, lse) for one row."""
    logit = _c(logit, np.float64)
    z = np.empty_like(logit)
    lse = _load().orc_softmax_row(_p(logit, c_double), c_int32(logit.size), c_double(float(T)),
                                  _p(z, c_double))
    return z, float(lse)


def topk_row(z, topk: int) -> np.ndarray:
    z = _c(z, np.float64)
    idx = np.empty(topk, dtype=np.int32)
    _load().orc_topk_row(_p(z, c_double), c_int32(z.size), c_int32(topk), _p(idx, c_int32))
    return idx


def gumbel_row(z, u):
    """Returns (argmax index, score = z + g) for one row."""
    z = _c(z, np.float64)
    u = _c(u, np.float32)
    score = np.empty_like(z)
    j = _load().orc_gumbel_row(_p(z, c_double), _p(u, c_float), c_int32(z.size),
                               _p(score, c_double))
    return int(j), score


class DraftHeadResult:
    __slots__ = ("ids", "logprobs", "trim", "logits", "z", "lse", "score")


def draft_head(h, W_trim, map_, temp, topk: int, uniforms=None, want_full: bool = True):
    """Algorithm 2 (drafter forward over the trimmed head, then the index mapping), head part.  h [B,d], W_trim [K,d] as bf16 bit patterns; map_ int32
    [K] or None (identity); temp fp32 [B]; uniforms fp32 [B,K] or None.  Returns ids/logprobs of
    shape [B,1+topk] plus (when want_full) logits, z, lse and Gumbel scores for margin checks."""
    h, W_trim = _bits(h), _bits(W_trim)
    B, d = h.shape
    K = W_trim.shape[0]
    temp = _c(temp, np.float32)
    assert temp.size == B
    if map_ is not None:
        map_ = _c(map_, np.int32)
        assert map_.size == K
    if uniforms is not None:
        uniforms = _c(uniforms, np.float32)
        assert uniforms.shape == (B, K)
    r = DraftHeadResult()
    r.ids = np.empty((B, 1 + topk), dtype=np.int32)
    r.logprobs = np.empty((B, 1 + topk), dtype=np.float64)
    r.trim = np.empty((B, 1 + topk), dtype=np.int32)
    r.logits = np.empty((B, K), dtype=np.float64) if want_full else None
    r.z = np.empty((B, K), dtype=np.float64) if want_full else None
    r.lse = np.empty(B, dtype=np.float64)
    r.score = np.empty((B, K), dtype=np.float64) if (want_full and uniforms is not None) else None
    rc = _load().orc_draft_head(_p(h, c_uint16), _p(W_trim, c_uint16), _p(map_, c_int32),
                                c_int32(B), c_int32(K), c_int32(d), _p(temp, c_float),
                                c_int32(topk), _p(uniforms, c_float), _p(r.ids, c_int32),
                                _p(r.logprobs, c_double), _p(r.trim, c_int32),
                                _p(r.logits, c_double), _p(r.z, c_double), _p(r.lse, c_double),
                                _p(r.score, c_double))
    if rc:
        raise ValueError("draft_head: invalid shape arguments")
    return r


def verify_greedy(token, parent, target):
    """Greedy verification of S drafted blocks (Experiments section; Algorithm 2's accept loop).

    token [S,N], parent [S,N] or None (chains), target [S,N+1].  Returns (n_accept int32 [S],
    path int32 [S,N] padded with -1, emitted int32 [S,N+1] padded with -1)."""
    token = _c(token, np.int32)
    target = _c(target, np.int32)
    S, N = token.shape
    assert target.shape == (S, N + 1)
    if parent is not None:
        parent = _c(parent, np.int32)
        assert parent.shape == (S, N)
    n_acc = np.zeros(S, dtype=np.int32)
    path = np.full((S, N), -1, dtype=np.int32)
    emitted = np.full((S, N + 1), -1, dtype=np.int32)
    fn = _load().orc_verify_greedy
    fn.restype = c_int32
    for s in range(S):
        n_acc[s] = fn(_p(token[s], c_int32), _p(parent[s], c_int32) if parent is not None else None,
                      _p(target[s], c_int32), c_int32(N), _p(path[s], c_int32), _p(emitted[s], c_int32))
    return n_acc, path, emitted


def block_efficiency(n_accept) -> float:
    """tau: mean number of tokens a block yields = accepted drafts + the target's own token
    (Performance Metrics paragraph)."""
    n_accept = np.asarray(n_accept, dtype=np.float64)
    return float(np.mean(n_accept + 1.0))


def mbsu(tau: float, c: float, gamma: int) -> float:
    """Memory-bound speed-up tau / (c * gamma + 1), c = draft / target parameter ratio
    (Performance Metrics paragraph)."""
    return float(tau) / (float(c) * float(gamma) + 1.0)


# ---- draft-tree construction.  Section 4.1 (Settings) adopts the EAGLE-2 tree procedure with depth 3,
# top-K = 8 and at most 32 draft tokens (Table 4: 60 in the depth ablation); the steps below restate
# that published procedure.  Scores are cumulative log-probabilities kept in fp32, the
# precision the GPU path keeps them in, because they decide integers (which nodes are taken).

def _score_order(score, index):
    """Order of preference: higher score first, lower node index on equal scores; NaN ranks last."""
    s = np.where(np.isnan(score), -np.inf, score).astype(np.float32)
    return np.lexsort((index, -s.astype(np.float64)))


def tree_expand(cand_ids, cand_logprobs, frontier_nodes, pool_token, pool_parent, pool_score,
                pool_base: int, n_front: int):
    """One depth of the expansion.  Row b of cand_* holds the top-k ids / log-probs the head gave for
    the node frontier_nodes[b] (None: the single row is the committed prefix, parent -1, score 0).
    Every candidate becomes a pool node at pool_base + b*topk + j with
    score = score(parent) + min(logprob, 0); the n_front best new nodes are the next frontier.
    Mutates the pool arrays; returns the frontier's pool indices in order of preference."""
    cand_ids = np.asarray(cand_ids, dtype=np.int32)
    lp = np.asarray(cand_logprobs, dtype=np.float32)
    B, topk = cand_ids.shape
    for b in range(B):
        par = -1 if frontier_nodes is None else int(frontier_nodes[b])
        base_score = np.float32(0.0) if par < 0 else pool_score[par]
        for j in range(topk):
            node = pool_base + b * topk + j
            pool_token[node] = cand_ids[b, j]
            pool_parent[node] = par
            step = lp[b, j] if np.isnan(lp[b, j]) else min(lp[b, j], np.float32(0.0))
            pool_score[node] = np.float32(base_score + step)
    new = np.arange(pool_base, pool_base + B * topk, dtype=np.int32)
    order = _score_order(pool_score[new], new)
    return new[order[:n_front]].copy()


def tree_rerank(pool_token, pool_parent, pool_score, n: int, budget: int):
    """Final selection: the `budget` best of the n pool nodes by cumulative score, listed in pool
    order (parents precede children), parents renumbered into that list (-1 = committed prefix).
    Returns (nodes, token, parent), each of length min(budget, n)."""
    idx = np.arange(n, dtype=np.int32)
    keep = np.sort(idx[_score_order(np.asarray(pool_score[:n], dtype=np.float32), idx)[:budget]])
    pos = {int(node): k for k, node in enumerate(keep)}
    token = np.array([pool_token[i] for i in keep], dtype=np.int32)
    parent = np.array([-1 if pool_parent[i] < 0 else pos.get(int(pool_parent[i]), -2) for i in keep],
                      dtype=np.int32)
    return keep.astype(np.int32), token, parent
