"""Pins for the CPU oracle: every oracle function is checked against something other than
itself -- a closed form, an invariant, a library routine on a special case, or brute force on
tiny inputs -- chosen so that a dropped term, a wrong sign or index, or a transposed operand
fails at least one of them.  No GPU is involved."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
import vt_inputs


def _bits(t: torch.Tensor) -> np.ndarray:
    return vt_inputs.bf16_bits(t.contiguous()).numpy().view(np.uint16)


# ----------------------------------------------------------------------------- bf16 decode
def test_bf16_decode_all_patterns_match_torch():
    pats = torch.arange(0, 65536, dtype=torch.int32).to(torch.int16)
    ref = pats.view(torch.bfloat16).to(torch.float64).numpy()
    got = oracle.decode_bf16(pats.numpy())
    finite = np.isfinite(ref)
    assert np.array_equal(got[finite], ref[finite])
    assert np.array_equal(np.isnan(got), np.isnan(ref))
    assert np.array_equal(np.isinf(got), np.isinf(ref))
    # two hand values: 0x3F80 = 1.0, 0xC048 = -3.125
    assert oracle.decode_bf16(np.array([0x3F80, 0xC048], dtype=np.uint16)).tolist() == [1.0, -3.125]


# ----------------------------------------------------------------------------- histogram (Algorithm 1)
def test_histogram_hand_example():
    ids = np.array([3, 1, 3, 3, 0, 7, 1, -1, 8, 5], dtype=np.int32)  # V = 8: -1 and 8 are invalid
    counts, bad = oracle.histogram(ids, 8)
    assert counts.tolist() == [1, 2, 0, 3, 0, 1, 0, 1]
    assert bad == 2


def test_histogram_matches_bincount_and_sums_to_n():
    ids = vt_inputs.zipf_ids(200_000, 4096, 1.1, seed=11, noise_frac=0.05).numpy()
    counts, bad = oracle.histogram(ids, 4096)
    assert bad == 0
    assert int(counts.sum()) == ids.size
    assert np.array_equal(counts, np.bincount(ids, minlength=4096).astype(np.uint64))
    assert np.array_equal(counts.astype(np.int64),
                          torch.bincount(torch.from_numpy(ids).long(), minlength=4096).numpy())


def test_histogram_accumulates_over_chunks():
    ids = vt_inputs.zipf_ids(50_000, 1000, 1.07, seed=5).numpy()
    whole, _ = oracle.histogram(ids, 1000)
    part, _ = oracle.histogram(ids[:20_000], 1000)
    part, _ = oracle.histogram(ids[20_000:], 1000, counts=part)
    assert np.array_equal(whole, part)


# ----------------------------------------------------------------------------- top-K (Eq. 1 (token selection))
def _rank_by_definition(counts):
    """rank(v) = #{u : c_u > c_v or (c_u == c_v and u < v)} -- no sort involved."""
    V = len(counts)
    return [sum(1 for u in range(V) if counts[u] > counts[v] or (counts[u] == counts[v] and u < v))
            for v in range(V)]


def test_topk_exhaustive_tiny_against_rank_definition():
    for V in range(1, 7):
        for cv in itertools.product((0, 1, 2), repeat=V):
            rank = _rank_by_definition(cv)
            for K in range(1, V + 1):
                m, inv = oracle.select_topk(np.array(cv, dtype=np.uint64), K)
                for v in range(V):
                    if rank[v] < K:
                        assert m[rank[v]] == v and inv[v] == rank[v]
                    else:
                        assert inv[v] == -1


def test_topk_brute_force_best_subset():
    """The kept set must maximise the total count over all K-subsets (exhaustive enumeration)."""
    rng = np.random.default_rng(3)
    for _ in range(20):
        V, K = 9, int(rng.integers(1, 9))
        c = rng.integers(0, 5, size=V).astype(np.uint64)
        m, _ = oracle.select_topk(c, K)
        best = max(int(sum(c[list(s)])) for s in itertools.combinations(range(V), K))
        assert int(c[m].sum()) == best


def test_topk_invariants_with_massive_ties():
    ids = vt_inputs.zipf_ids(100_000, 4096, 1.1, seed=1001).numpy()
    counts, _ = oracle.histogram(ids, 4096)
    K = 1024
    m, inv = oracle.select_topk(counts, K)
    assert len(set(m.tolist())) == K
    kept = counts[m].astype(np.int64)
    assert np.all(np.diff(kept) <= 0)                        # counts non-increasing along the map
    same = np.diff(kept) == 0
    assert np.all(np.diff(m.astype(np.int64))[same] > 0)     # equal counts => ascending ids
    pruned = np.setdiff1d(np.arange(4096), m)
    assert kept.min() >= counts[pruned].max()
    cut = kept.min()                                          # ties at the cut: lower ids are kept
    tied_kept = m[kept == cut]
    tied_pruned = pruned[counts[pruned] == cut]
    if tied_pruned.size:
        assert tied_kept.max() < tied_pruned.min()
    assert np.array_equal(inv[m], np.arange(K))
    assert int((inv >= 0).sum()) == K


def test_topk_tie_free_matches_stable_argsort():
    rng = np.random.default_rng(7)
    c = rng.permutation(5000).astype(np.uint64)               # all counts distinct
    m, _ = oracle.select_topk(c, 777)
    assert np.array_equal(m, np.argsort(-c.astype(np.int64), kind="stable")[:777].astype(np.int32))


def test_topk_fewer_seen_ids_than_K_fills_tail_in_id_order():
    c = np.zeros(16, dtype=np.uint64)
    c[[9, 2, 13]] = [5, 7, 5]
    m, inv = oracle.select_topk(c, 8)
    assert m.tolist() == [2, 9, 13, 0, 1, 3, 4, 5]
    assert inv[6] == -1 and inv[0] == 3


def test_topk_K_equals_V_is_a_permutation():
    c = np.array([1, 1, 1, 1], dtype=np.uint64)
    m, inv = oracle.select_topk(c, 4)
    assert m.tolist() == [0, 1, 2, 3] and inv.tolist() == [0, 1, 2, 3]


# ----------------------------------------------------------------------------- gather (Eq. 1 (head restriction))
def test_trim_head_is_a_bit_copy_of_the_mapped_rows():
    W = _bits(vt_inputs.gaussian_bf16((50, 24), 0.02, seed=2))
    m = np.array([7, 0, 49, 7, 13], dtype=np.int32)
    Wt = oracle.trim_head(W, m)
    assert Wt.shape == (5, 24)
    for j, v in enumerate(m):
        assert np.array_equal(Wt[j], W[v])
    ident = np.arange(50, dtype=np.int32)
    assert np.array_equal(oracle.trim_head(W, ident), W)


# ----------------------------------------------------------------------------- logits (Algorithm 2, drafter forward)
def test_logits_match_numpy_fp64_matmul_nonsquare():
    h = _bits(vt_inputs.gaussian_bf16((3, 40), 1.0, seed=4))
    W = _bits(vt_inputs.gaussian_bf16((17, 40), 0.02, seed=5))
    got = oracle.logits(h, W)
    ref = oracle.decode_bf16(h) @ oracle.decode_bf16(W).T      # [B,d] x [d,K]: a transposed operand cannot pass
    ref_t = (vt_inputs.gaussian_bf16((3, 40), 1.0, seed=4).double()
             @ vt_inputs.gaussian_bf16((17, 40), 0.02, seed=5).double().T).numpy()
    assert got.shape == (3, 17)
    assert np.allclose(got, ref, rtol=0, atol=1e-12)
    assert np.allclose(got, ref_t, rtol=0, atol=1e-12)


def test_logits_exact_on_small_integers():
    rng = np.random.default_rng(9)
    hi = rng.integers(-4, 5, size=(2, 16))
    Wi = rng.integers(-4, 5, size=(11, 16))
    h = _bits(torch.from_numpy(hi).to(torch.bfloat16))
    W = _bits(torch.from_numpy(Wi).to(torch.bfloat16))
    assert np.array_equal(oracle.logits(h, W), (hi @ Wi.T).astype(np.float64))


def test_trimmed_logits_equal_full_logits_at_mapped_rows_exactly():
    V, d, K = 300, 64, 77
    W = _bits(vt_inputs.gaussian_bf16((V, d), 0.02, seed=6))
    h = _bits(vt_inputs.gaussian_bf16((4, d), 1.0, seed=7))
    ids = vt_inputs.zipf_ids(5000, V, 1.1, seed=8).numpy()
    m, inv, _, _ = oracle.build_vocab(ids, V, K)
    full = oracle.logits(h, W)
    trim = oracle.logits(h, oracle.trim_head(W, m))
    assert np.array_equal(trim, full[:, m])                    # same fp64 operation order: bit equal


def test_identity_map_reproduces_the_full_head():
    V, d = 200, 32
    W = _bits(vt_inputs.gaussian_bf16((V, d), 0.02, seed=16))
    h = _bits(vt_inputs.gaussian_bf16((2, d), 1.0, seed=17))
    T = np.array([1.0, 0.7], dtype=np.float32)
    u = vt_inputs.uniforms((2, V), seed=18).numpy()
    ident = np.arange(V, dtype=np.int32)
    a = oracle.draft_head(h, W, None, T, 5, u)
    b = oracle.draft_head(h, oracle.trim_head(W, ident), ident, T, 5, u)
    assert np.array_equal(a.ids, b.ids) and np.array_equal(a.logprobs, b.logprobs)
    assert np.array_equal(a.ids, a.trim)


# ----------------------------------------------------------------------------- softmax
def test_softmax_sums_to_one_and_is_shift_invariant():
    rng = np.random.default_rng(12)
    logit = rng.normal(0, 3, size=5000)
    for T in (1.0, 0.7, 1.5):
        z, lse = oracle.softmax_row(logit, T)
        assert np.array_equal(z, logit / T)
        p = np.exp(z - lse)
        assert abs(p.sum() - 1.0) < 1e-12
        z2, lse2 = oracle.softmax_row(logit + 5.0 * T, T)
        assert np.allclose(z2 - lse2, z - lse, rtol=0, atol=1e-12)


def test_softmax_matches_torch_log_softmax_fp64():
    rng = np.random.default_rng(13)
    logit = rng.normal(0, 2, size=3000)
    for T in (1.0, 0.5, 2.0):
        z, lse = oracle.softmax_row(logit, T)
        ref = torch.log_softmax(torch.from_numpy(logit) / T, dim=0).numpy()
        assert np.allclose(z - lse, ref, rtol=0, atol=1e-12)


def test_softmax_closed_form_two_classes():
    z, lse = oracle.softmax_row(np.array([0.0, math.log(3.0)]), 1.0)
    assert abs(math.exp(z[1] - lse) - 0.75) < 1e-15 and abs(lse - math.log(4.0)) < 1e-15
    # temperature 2 halves the logits: p = sqrt(3) / (1 + sqrt(3))
    z, lse = oracle.softmax_row(np.array([0.0, math.log(3.0)]), 2.0)
    assert abs(math.exp(z[1] - lse) - math.sqrt(3) / (1 + math.sqrt(3))) < 1e-15


# ----------------------------------------------------------------------------- top-k candidates
def test_topk_row_brute_force_and_ties_to_lower_index():
    rng = np.random.default_rng(14)
    for _ in range(50):
        K = int(rng.integers(1, 9))
        z = rng.integers(0, 4, size=K).astype(np.float64)     # many ties
        k = int(rng.integers(1, K + 1))
        ref = sorted(range(K), key=lambda j: (-z[j], j))[:k]
        assert oracle.topk_row(z, k).tolist() == ref
    z = rng.normal(size=1000)
    idx = oracle.topk_row(z, 10)
    assert idx[0] == int(np.argmax(z))
    assert np.array_equal(idx, torch.topk(torch.from_numpy(z), 10).indices.numpy())
    assert set(idx.tolist()) == set(np.nonzero(z >= z[idx[-1]])[0].tolist())


# ----------------------------------------------------------------------------- Gumbel-max
def test_gumbel_equal_uniforms_is_greedy_and_dominant_logit_always_wins():
    rng = np.random.default_rng(15)
    z = rng.normal(size=500)
    for uval in (0.01, 0.5, 0.99):
        j, _ = oracle.gumbel_row(z, np.full(500, uval, dtype=np.float32))
        assert j == int(np.argmax(z))
    z2 = z.copy()
    z2[123] = 1e4
    j, _ = oracle.gumbel_row(z2, vt_inputs.uniforms((500,), seed=3).numpy())
    assert j == 123


def test_gumbel_score_closed_form_and_clamp():
    # u = 1/e gives g = -log(1) = 0;  u = exp(-exp(-2)) gives g = 2
    u = np.array([math.exp(-1.0), math.exp(-math.exp(-2.0))], dtype=np.float32)
    _, score = oracle.gumbel_row(np.array([0.25, -1.0]), u)
    assert abs(score[0] - 0.25) < 1e-6 and abs(score[1] - 1.0) < 1e-6
    # u = 0 and u = 1 are clamped to 2^-24 and 1 - 2^-24: finite scores with the right signs
    _, score = oracle.gumbel_row(np.zeros(2), np.array([0.0, 1.0], dtype=np.float32))
    assert np.all(np.isfinite(score))
    assert abs(score[0] + math.log(24 * math.log(2.0))) < 1e-12
    assert abs(score[1] + math.log(-math.log1p(-2.0 ** -24))) < 1e-9
    # ties resolve to the first maximal index
    j, _ = oracle.gumbel_row(np.zeros(4), np.full(4, 0.3, dtype=np.float32))
    assert j == 0


def test_gumbel_draws_follow_softmax_chi_square():
    z = np.array([0.0, 0.5, 1.0, -1.0, 2.0, 0.3, -0.7, 1.4])
    p = np.exp(z - np.log(np.exp(z).sum()))
    n = 100_000
    u = vt_inputs.uniforms((n, 8), seed=77).numpy()
    hits = np.zeros(8)
    for i in range(n):
        j, _ = oracle.gumbel_row(z, u[i])
        hits[j] += 1
    chi2 = float((((hits - n * p) ** 2) / (n * p)).sum())
    assert chi2 < 24.3                                           # 7 dof, p = 0.001


def test_gumbel_restriction_property():
    """Sampling over the kept set with the kept uniforms equals the full-vocabulary Gumbel
    argmax restricted to the kept set."""
    V, K = 400, 90
    rng = np.random.default_rng(21)
    zfull = rng.normal(size=V)
    u = vt_inputs.uniforms((V,), seed=22).numpy()
    kept = np.sort(rng.choice(V, K, replace=False))
    _, score_full = oracle.gumbel_row(zfull, u)
    j, _ = oracle.gumbel_row(zfull[kept], u[kept])
    assert kept[j] == kept[int(np.argmax(score_full[kept]))]


# ----------------------------------------------------------------------------- full head + remap
def test_draft_head_outputs_are_consistent_with_its_parts():
    V, d, K, B, topk = 512, 64, 128, 3, 4
    W = _bits(vt_inputs.gaussian_bf16((V, d), 0.02, seed=31))
    h = _bits(vt_inputs.gaussian_bf16((B, d), 1.0, seed=32))
    ids = vt_inputs.zipf_ids(20_000, V, 1.1, seed=33).numpy()
    m, inv, _, _ = oracle.build_vocab(ids, V, K)
    Wt = oracle.trim_head(W, m)
    T = np.array([1.0, 0.7, 1.3], dtype=np.float32)
    u = vt_inputs.uniforms((B, K), seed=34).numpy()
    r = oracle.draft_head(h, Wt, m, T, topk, u)
    lg = oracle.logits(h, Wt)
    assert np.array_equal(r.logits, lg)
    for b in range(B):
        z, lse = oracle.softmax_row(lg[b], float(T[b]))
        assert np.array_equal(r.trim[b, 1:], oracle.topk_row(z, topk))
        assert r.trim[b, 1] == int(np.argmax(z))
        g, _ = oracle.gumbel_row(z, u[b])
        assert r.trim[b, 0] == g
        assert np.allclose(r.logprobs[b], z[r.trim[b]] - lse, rtol=0, atol=0)
        ref = torch.log_softmax(torch.from_numpy(lg[b]) / float(T[b]), 0).numpy()
        assert np.allclose(r.logprobs[b], ref[r.trim[b]], rtol=0, atol=1e-12)
    assert np.array_equal(r.ids, m[r.trim])                     # remap T_{d->t}
    assert np.array_equal(inv[r.ids], r.trim)                   # inverse map recovers the trimmed index
    greedy = oracle.draft_head(h, Wt, m, T, topk, None)
    assert np.array_equal(greedy.ids[:, 0], greedy.ids[:, 1])   # no uniforms: column 0 is the greedy id


def test_draft_head_rejects_bad_shapes():
    W = np.zeros((4, 8), dtype=np.uint16)
    h = np.zeros((1, 8), dtype=np.uint16)
    with pytest.raises(ValueError):
        oracle.draft_head(h, W, None, np.ones(1, dtype=np.float32), 5, None)


# ---- selection variants named in the Method section: Top-P and minimum frequency -----------------------
def _brute_topp(counts, p):
    """Definition written out: rank ids by (count desc, id asc); smallest K whose prefix holds >= ceil(p*total)."""
    order = sorted(range(len(counts)), key=lambda v: (-int(counts[v]), v))
    total = int(sum(int(c) for c in counts))
    target = int(np.ceil(p * total))
    cum = 0
    for j, v in enumerate(order):
        cum += int(counts[v])
        if cum >= target:
            return max(1, j + 1), order
    return len(counts), order


def test_select_topp_hand_example_and_definition_on_random_counts():
    c = np.array([5, 0, 3, 3, 9, 0, 1], dtype=np.uint64)          # total 21; ranking 4,0,2,3,6,1,5
    K, m, inv = oracle.select_topp(c, 0.5)                           # ceil(10.5) = 11 -> 9 + 5
    assert K == 2 and m.tolist() == [4, 0, 2, 3, 6, 1, 5] and inv.tolist() == [1, -1, -1, -1, 0, -1, -1]
    assert oracle.select_topp(c, 9 / 21)[0] == 1                     # exactly the top id's share
    assert oracle.select_topp(c, 1.0)[0] == 5                        # all ids that were ever seen
    rng = np.random.default_rng(7)
    for _ in range(200):
        V = int(rng.integers(1, 40))
        counts = rng.integers(0, 6, V).astype(np.uint64)
        p = float(rng.uniform(0.01, 1.0))
        K, m, inv = oracle.select_topp(counts, p)
        Kb, order = _brute_topp(counts, p)
        assert K == Kb and m.tolist() == order
        assert [int(inv[v]) for v in order] == [j if j < K else -1 for j in range(V)]


def test_select_topp_is_minimal_and_monotone_in_p():
    rng = np.random.default_rng(8)
    counts = np.sort(rng.zipf(1.3, 5000).astype(np.uint64))[::-1].copy()
    rng.shuffle(counts)
    total = int(counts.sum())
    last = 0
    for p in (0.1, 0.5, 0.9, 0.99, 1.0):
        K, m, _ = oracle.select_topp(counts, p)
        cum = np.cumsum(counts[m].astype(np.int64))
        target = int(np.ceil(p * total))
        assert cum[K - 1] >= target and (K == 1 or cum[K - 2] < target)
        assert K >= last
        last = K


def test_select_minfreq_counts_ids_at_or_above_the_threshold():
    c = np.array([5, 0, 3, 3, 9, 0, 1], dtype=np.uint64)
    assert oracle.select_minfreq(c, 3)[0] == 4 and oracle.select_minfreq(c, 0)[0] == 7
    assert oracle.select_minfreq(c, 10)[0] == 1                      # never an empty vocabulary
    rng = np.random.default_rng(9)
    counts = rng.integers(0, 50, 3000).astype(np.uint64)
    for f in (1, 7, 25, 49):
        K, m, inv = oracle.select_minfreq(counts, f)
        assert K == int((counts >= f).sum())
        assert np.all(counts[m[:K]] >= f) and np.all(counts[m[K:]] < f)
        ref_m, ref_inv = oracle.select_topk(counts, K)                # the same cut of the same ranking
        assert np.array_equal(m[:K], ref_m) and np.array_equal(inv, ref_inv)


# ---- greedy verification, block efficiency, MBSU (Experiments section; Algorithm 2's accept loop)

def _consistent_nodes(token, parent, target):
    """Set formulation: a node is accepted iff its token is the target's token at its parent and the
    parent is accepted (the committed prefix is).  With distinct sibling tokens this set is a path."""
    N = len(token)
    ok = np.zeros(N, dtype=bool)
    for i in range(N):                                   # parents precede children
        par = parent[i]
        ok[i] = (par == -1 or ok[par]) and token[i] == target[par + 1]
    return np.flatnonzero(ok)


def test_verify_chain_is_the_first_mismatch():
    rng = np.random.default_rng(5)
    S, N = 200, 7
    token = rng.integers(0, 4, size=(S, N)).astype(np.int32)
    target = rng.integers(0, 4, size=(S, N + 1)).astype(np.int32)
    target[:, :N] = np.where(rng.random((S, N)) < 0.7, token, target[:, :N])
    n_acc, path, emitted = oracle.verify_greedy(token, None, target)
    match = token == target[:, :N]
    first_miss = np.where(match.all(1), N, np.argmin(match, axis=1))
    assert np.array_equal(n_acc, first_miss)
    for s in range(S):
        n = n_acc[s]
        assert np.array_equal(path[s, :n], np.arange(n)) and np.all(path[s, n:] == -1)
        assert np.array_equal(emitted[s, :n], token[s, :n]) and emitted[s, n] == target[s, n]
        assert np.all(emitted[s, n + 1:] == -1)
    # the chain is the tree whose parent of node i is node i-1
    chain = np.tile(np.arange(-1, N - 1, dtype=np.int32), (S, 1))
    n2, p2, e2 = oracle.verify_greedy(token, chain, target)
    assert np.array_equal(n2, n_acc) and np.array_equal(p2, path) and np.array_equal(e2, emitted)


def test_verify_tree_against_the_set_formulation():
    for N, width, vocab, pm, seed in ((1, 1, 3, 0.5, 1), (12, 3, 5, 0.8, 2), (40, 8, 50, 0.7, 3), (63, 4, 4, 0.9, 4)):
        token, parent, target = (t.numpy() for t in vt_inputs.draft_trees(60, N, width, vocab, pm, seed))
        n_acc, path, emitted = oracle.verify_greedy(token, parent, target)
        assert n_acc.max() >= min(N, 2) - 1                  # the inputs do produce walks
        for s in range(token.shape[0]):
            want = _consistent_nodes(token[s], parent[s], target[s])
            n = int(n_acc[s])
            assert np.array_equal(path[s, :n], want)
            last = want[-1] if n else -1
            assert emitted[s, n] == target[s, last + 1]
            assert np.array_equal(emitted[s, :n], token[s][want])
            # every accepted node hangs off the previous one
            assert all(parent[s, path[s, k]] == (path[s, k - 1] if k else -1) for k in range(n))


def test_verify_hand_example_bounds_and_duplicate_siblings():
    # root children: node0 (tok 5), node1 (tok 4); node0's children: node2 (6), node3 (7); node3's child: node4 (8)
    token = np.array([[5, 4, 6, 7, 8]], dtype=np.int32)
    parent = np.array([[-1, -1, 0, 0, 3]], dtype=np.int32)
    target = np.array([[5, 7, 0, 0, 8, 3]], dtype=np.int32)
    n_acc, path, emitted = oracle.verify_greedy(token, parent, target)
    assert n_acc[0] == 3 and path[0, :3].tolist() == [0, 3, 4] and emitted[0, :4].tolist() == [5, 7, 8, 3]
    # nothing matches: the block still yields the target's own token (tau >= 1)
    n_acc, _, emitted = oracle.verify_greedy(token, parent, np.full((1, 6), 9, dtype=np.int32))
    assert n_acc[0] == 0 and emitted[0, 0] == 9 and oracle.block_efficiency(n_acc) == 1.0
    # a full match of a depth-gamma chain yields gamma + 1 tokens, the stated maximum of tau
    chain = np.arange(4, dtype=np.int32)[None]
    n_acc, _, _ = oracle.verify_greedy(chain, None, np.arange(5, dtype=np.int32)[None])
    assert oracle.block_efficiency(n_acc) == 5.0
    # two siblings with the same token: the lower index is taken; unreachable parents are ignored
    token = np.array([[3, 3, 1, 2]], dtype=np.int32)
    parent = np.array([[-1, -1, 1, 0]], dtype=np.int32)
    n_acc, path, _ = oracle.verify_greedy(token, parent, np.array([[3, 2, 1, 0, 0]], dtype=np.int32))
    assert n_acc[0] == 2 and path[0, :2].tolist() == [0, 3]
    bad_parent = np.array([[-1, 5, -7, 3]], dtype=np.int32)            # not in [-1, i)
    n_acc, path, _ = oracle.verify_greedy(token, bad_parent, np.array([[3, 3, 3, 3, 3]], dtype=np.int32))
    assert n_acc[0] == 1 and path[0, 0] == 0


def _mbsu_rows():
    here = os.path.join(os.path.dirname(__file__), "golden", "paper_mbsu_rows.txt")
    rows = {}
    for line in open(here):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        v = list(map(float, f[3:]))
        rows[f[0]] = (f[1], float(f[2]), np.array(v[0::2]), np.array(v[1::2]))
    return rows


def test_mbsu_reproduces_the_table_rows_of_the_paper():
    """Table 1 prints (BE, MBSU) per task.  MBSU = tau / (c*gamma + 1) with c the parameter ratio, so
    (i) within a row MBSU is BE over ONE constant; (ii) that constant moves with the draft
    parameter count only: fixing gamma / P_target from the untrimmed independent drafter (314M
    parameters) predicts the denominators of the three other drafters from the printed head sizes."""
    rows = _mbsu_rows()
    assert len(rows) == 6
    name, head, be, mb = rows["independent_full"]
    per_m = float(np.mean(be / mb) - 1.0) / 314.0                 # gamma / P_target per 1e6 draft parameters
    gamma = 4
    p_target = gamma / per_m
    assert abs(p_target - 3212.7) < 12.0                          # Llama-3.2-3B has 3.21e9 parameters at gamma = 4
    ind_trim = 314.0 - 131.3 + 33.8
    for key in ("independent_full", "independent_raw", "independent_target"):
        _, head, be, mb = rows[key]
        p_draft = 314.0 if head == 131.3 else ind_trim
        for tau, want in zip(be, mb):
            assert abs(oracle.mbsu(tau, p_draft / p_target, gamma) - want) < 2.5e-3
    # EAGLE drafter: its total size is not printed; one row fixes it, the trimmed rows follow from
    # the printed head sizes alone.
    _, head, be, mb = rows["eagle_full"]
    p_eagle = float(np.mean(be / mb) - 1.0) / per_m
    for key in ("eagle_full", "eagle_raw", "eagle_target"):
        _, head, be, mb = rows[key]
        p_draft = p_eagle - 394.0 + head
        for tau, want in zip(be, mb):
            assert abs(oracle.mbsu(tau, p_draft / p_target, gamma) - want) < 2.5e-3
    # a wrong form (tau * denominator, or gamma + c instead of c * gamma + 1) misses by far more
    assert abs(3.846 / (1 + 4 * 314.0 / p_target) - 2.765) < 2.5e-3
    assert abs(3.846 / (4 + 314.0 / p_target) - 2.765) > 1.0


# ---- draft-tree expansion and rerank (Settings: tree construction following EAGLE-2)

def _grow(depth, topk, n_front, vocab, seed, tie_frac=0.0):
    cap = topk + (depth - 1) * n_front * topk
    tok = np.full(cap, -9, dtype=np.int32)
    par = np.full(cap, -9, dtype=np.int32)
    sc = np.full(cap, np.nan, dtype=np.float32)
    steps = []
    ids, lp = (t.numpy() for t in vt_inputs.head_candidates(1, topk, vocab, seed, tie_frac))
    front = oracle.tree_expand(ids, lp, None, tok, par, sc, 0, n_front)
    steps.append((ids, lp, None, 0, front))
    base = topk
    for dep in range(1, depth):
        ids, lp = (t.numpy() for t in vt_inputs.head_candidates(len(front), topk, vocab, seed + dep, tie_frac))
        nxt = oracle.tree_expand(ids, lp, front, tok, par, sc, base, n_front)
        steps.append((ids, lp, front, base, nxt))
        base += len(front) * topk
        front = nxt
    return tok, par, sc, base, steps


def test_tree_scores_are_path_sums_and_frontier_is_the_brute_force_best():
    for depth, topk, seed in ((3, 8, 1), (5, 10, 2), (2, 3, 3), (7, 4, 4)):
        tok, par, sc, n, steps = _grow(depth, topk, topk, 1000, seed)
        assert n == topk + (depth - 1) * topk * topk and not np.isnan(sc[:n]).any()
        lp_of = {}
        for ids, lp, front, base, nxt in steps:
            B = ids.shape[0]
            for b in range(B):
                for j in range(topk):
                    node = base + b * topk + j
                    lp_of[node] = lp[b, j]
                    assert tok[node] == ids[b, j] and par[node] == (-1 if front is None else front[b])
            new = list(range(base, base + B * topk))
            best = sorted(new, key=lambda i: (-float(sc[i]), i))[:len(nxt)]
            assert best == nxt.tolist()
        for i in range(n):                                   # cumulative score = sum over the path, root first
            chain = []
            j = i
            while j >= 0:
                chain.append(j)
                j = par[j]
            acc = np.float32(0.0)
            for j in reversed(chain):
                acc = np.float32(acc + lp_of[j])
            assert acc == sc[i]
            assert par[i] < i and (par[i] < 0 or sc[par[i]] >= sc[i])


def test_tree_rerank_keeps_the_best_nodes_closed_under_parents():
    for depth, topk, budget, seed, ties in ((3, 8, 32, 1, 0.0), (6, 10, 60, 2, 0.0), (4, 5, 17, 3, 0.8),
                                            (2, 2, 100, 4, 0.5), (3, 4, 1, 5, 0.0)):
        tok, par, sc, n, _ = _grow(depth, topk, topk, 500, seed, ties)
        nodes, token, parent = oracle.tree_rerank(tok, par, sc, n, budget)
        m = min(budget, n)
        assert len(nodes) == m and np.all(np.diff(nodes) > 0)
        brute = sorted(sorted(range(n), key=lambda i: (-float(sc[i]), i))[:m])
        assert nodes.tolist() == brute
        worst_kept = min(float(sc[i]) for i in nodes)
        assert all(float(sc[i]) <= worst_kept for i in range(n) if i not in set(nodes.tolist()))
        for k in range(m):                                   # parents are kept, precede their children, renumbered
            assert token[k] == tok[nodes[k]]
            if par[nodes[k]] < 0:
                assert parent[k] == -1
            else:
                assert 0 <= parent[k] < k and nodes[parent[k]] == par[nodes[k]]


def test_tree_hand_example_ties_positive_logprob_and_nan():
    tok = np.zeros(6, dtype=np.int32); par = np.zeros(6, dtype=np.int32); sc = np.zeros(6, dtype=np.float32)
    ids = np.array([[7, 9]], dtype=np.int32)
    front = oracle.tree_expand(ids, np.array([[-0.5, -1.0]], dtype=np.float32), None, tok, par, sc, 0, 2)
    assert front.tolist() == [0, 1] and sc[:2].tolist() == [-0.5, -1.0]
    # children: of node 0: (-0.25, -2.0) -> -0.75, -2.5 ; of node 1: (+1e-7 clamps to 0, NaN) -> -1.0, NaN
    lp = np.array([[-0.25, -2.0], [1e-7, np.nan]], dtype=np.float32)
    front = oracle.tree_expand(np.array([[1, 2], [3, 4]], dtype=np.int32), lp, front, tok, par, sc, 2, 3)
    assert sc[2] == np.float32(-0.75) and sc[3] == np.float32(-2.5) and sc[4] == np.float32(-1.0) and np.isnan(sc[5])
    assert front.tolist() == [2, 4, 3]                        # NaN ranks last
    assert par[2:6].tolist() == [0, 0, 1, 1] and tok[2:6].tolist() == [1, 2, 3, 4]
    nodes, token, parent = oracle.tree_rerank(tok, par, sc, 6, 4)
    # scores: -0.5, -1.0, -0.75, -2.5, -1.0, NaN : best four = 0, 2, then 1 before 4 on the tie
    assert nodes.tolist() == [0, 1, 2, 4] and token.tolist() == [7, 9, 1, 3] and parent.tolist() == [-1, -1, 0, 1]
