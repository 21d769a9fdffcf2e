"""GPU parity of the draft-tree construction (Settings: tree construction following EAGLE-2) against
the CPU oracle.  Node ids, parents, frontier and the reranked draft are integers: bit-exact.  Scores
are fp32 sums taken in the same order on both sides: compared by bit pattern."""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_22694_b200 as vt
import vt_inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _bits(x):
    """fp32 bit patterns, with every NaN (payloads differ between host and device) as one pattern."""
    x = np.asarray(x, dtype=np.float32)
    return np.where(np.isnan(x), np.uint32(0x7fc00000), x.view(np.uint32))


def _grow_both(depth, topk, n_front, budget, vocab, seed, ties=0.0, nan_at=None, pad_cols=0):
    cap = topk + (depth - 1) * n_front * topk
    tok = np.full(cap, -9, dtype=np.int32)
    par = np.full(cap, -9, dtype=np.int32)
    sc = np.full(cap, np.nan, dtype=np.float32)
    pool = vt.tree_pool(cap)
    front_ref, front_gpu, base, B = None, None, 0, 1
    for dep in range(depth):
        ids, lp = vt_inputs.head_candidates(B, topk, vocab, seed + dep, ties)
        if nan_at is not None and dep == nan_at:
            lp[0, -1] = float("nan")
            lp[-1, 0] = 1e-6                                   # a rounding-positive log-prob clamps to 0
        nf = min(n_front, B * topk)
        front_ref = oracle.tree_expand(ids.numpy(), lp.numpy(), front_ref, tok, par, sc, base, nf)
        if pad_cols:                                           # the head's layout: candidates start at column 1
            ids = torch.cat([torch.full((B, pad_cols), -3, dtype=torch.int32), ids], dim=1)
            lp = torch.cat([torch.full((B, pad_cols), 5.0), lp], dim=1)
        front_gpu = vt.vt_tree_expand(ids.to(DEV), lp.to(DEV), front_gpu, pool, base, nf, col0=pad_cols)
        assert np.array_equal(front_gpu.cpu().numpy(), front_ref)
        base += B * topk
        B = nf
    assert np.array_equal(pool[0][:base].cpu().numpy(), tok[:base])
    assert np.array_equal(pool[1][:base].cpu().numpy(), par[:base])
    assert np.array_equal(_bits(pool[2][:base].cpu().numpy()), _bits(sc[:base]))
    nodes, token, parent = vt.vt_tree_rerank(pool, base, budget)
    rn, rt, rp = oracle.tree_rerank(tok, par, sc, base, budget)
    m = len(rn)
    assert np.array_equal(nodes.cpu().numpy()[:m], rn) and np.all(nodes.cpu().numpy()[m:] == -1)
    assert np.array_equal(token.cpu().numpy()[:m], rt) and np.all(token.cpu().numpy()[m:] == -1)
    assert np.array_equal(parent.cpu().numpy()[:m], rp) and np.all(parent.cpu().numpy()[m:] == -1)
    return nodes, token, parent, m


# (3, 8, 32) and depths 5-7 with 60 tokens are the paper's tree settings; B = 10 nodes per depth is the
# tree-drafter workload; the rest are ragged and degenerate sizes
@pytest.mark.parametrize("depth,topk,n_front,budget", [(3, 8, 8, 32), (5, 8, 8, 60), (6, 8, 8, 60), (7, 8, 8, 60),
                                                        (4, 10, 10, 60), (1, 1, 1, 1), (2, 3, 2, 100), (3, 16, 16, 17),
                                                        (9, 5, 7, 33)])
def test_tree_matches_oracle(depth, topk, n_front, budget):
    _grow_both(depth, topk, n_front, budget, vocab=128256, seed=depth * 100 + topk)


def test_tree_with_ties_nan_and_head_column_layout():
    _grow_both(4, 6, 6, 20, vocab=50, seed=7, ties=0.9)
    _grow_both(3, 8, 8, 32, vocab=1000, seed=8, ties=0.5, nan_at=1, pad_cols=1)
    _grow_both(3, 4, 4, 50, vocab=1000, seed=9, nan_at=2, pad_cols=1)


def test_tree_maximum_sizes_and_argument_checks():
    B, topk = 256, 16                                          # B*topk = VT_TREE_MAX_NODES new nodes in one depth
    ids, lp = vt_inputs.head_candidates(B, topk, 128256, seed=3, tie_frac=0.3)
    cap = 64 + B * topk
    tok = np.zeros(cap, dtype=np.int32); par = np.full(cap, -1, dtype=np.int32)
    sc = (-np.arange(cap, dtype=np.float32) / 7).astype(np.float32)
    pool = tuple(torch.from_numpy(a.copy()).to(DEV) for a in (tok, par, sc))
    front = torch.arange(0, 64, dtype=torch.int32).repeat(4)[:B].contiguous()
    ref = oracle.tree_expand(ids.numpy(), lp.numpy(), front.numpy(), tok, par, sc, 64, 300)
    got = vt.vt_tree_expand(ids.to(DEV), lp.to(DEV), front.to(DEV), pool, 64, 300)
    assert np.array_equal(got.cpu().numpy(), ref)
    assert np.array_equal(_bits(pool[2].cpu().numpy()), _bits(sc))
    n = 4096
    nodes, token, parent = vt.vt_tree_rerank(pool, n, 1000)
    rn, rt, rp = oracle.tree_rerank(tok, par, sc, n, 1000)
    assert np.array_equal(nodes.cpu().numpy(), rn) and np.array_equal(parent.cpu().numpy(), rp)
    assert np.array_equal(token.cpu().numpy(), rt)
    with pytest.raises(vt.VocabTrimError):                     # more new nodes than one call ranks
        vt.vt_tree_expand(torch.zeros(257, 16, dtype=torch.int32, device=DEV),
                          torch.zeros(257, 16, device=DEV), torch.zeros(257, dtype=torch.int32, device=DEV),
                          vt.tree_pool(8192), 0, 8)
    with pytest.raises(vt.VocabTrimError):                     # pool too small
        vt.vt_tree_expand(ids[:4].to(DEV), lp[:4].to(DEV), front[:4].to(DEV), vt.tree_pool(70), 64, 8)
    with pytest.raises(vt.VocabTrimError):                     # frontier larger than the new nodes
        vt.vt_tree_expand(ids[:1].to(DEV), lp[:1].to(DEV), None, vt.tree_pool(64), 0, 17)
    with pytest.raises(vt.VocabTrimError):
        vt.vt_tree_rerank(vt.tree_pool(5000), 4097, 10)


def test_head_to_tree_to_verification_on_the_trimmed_vocabulary():
    """The whole drafting block of Algorithm 2 on synthetic weights: trimmed head -> expansion per depth
    -> rerank -> greedy verification.  There is no drafter body, so hidden rows are re-drawn per depth;
    what is checked is structure: a valid tree over kept ids, scores that are path sums of the head's
    log-probs, and a verification result equal to the oracle's on the same tree."""
    V, K, d, topk, depth, budget = 8192, 2048, 512, 8, 3, 32
    ids = vt_inputs.zipf_ids(300_000, V, 1.1, seed=5, device=DEV)
    map_, _ = vt.vt_build_vocab(ids, V, K)
    Wt = vt.vt_trim_head(vt_inputs.gaussian_bf16((V, d), 0.05, seed=6, device=DEV), map_)
    cap = topk + (depth - 1) * topk * topk
    pool = vt.tree_pool(cap)
    front, base, B = None, 0, 1
    lps = []
    for dep in range(depth):
        h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=20 + dep, device=DEV)
        temp = torch.ones(B, dtype=torch.float32, device=DEV)
        out_ids, out_lp = vt.vt_draft_head(h, Wt, map_, temp, topk=topk)
        lps.append(out_lp[:, 1:].cpu().numpy())
        front = vt.vt_tree_expand(out_ids, out_lp, front, pool, base, topk, col0=1)
        base += B * topk
        B = topk
    tok, par, sc = (t.cpu().numpy() for t in pool)
    kept = set(map_.cpu().tolist())
    assert all(int(t) in kept for t in tok[:base])
    flat = np.concatenate([x.reshape(-1) for x in lps])
    for i in range(base):
        want = np.float32((sc[par[i]] if par[i] >= 0 else np.float32(0)) + min(flat[i], np.float32(0)))
        assert sc[i] == want and par[i] < i
    nodes, token, parent = vt.vt_tree_rerank(pool, base, budget)
    rn, rt, rp = oracle.tree_rerank(tok, par, sc, base, budget)
    assert np.array_equal(nodes.cpu().numpy(), rn) and np.array_equal(parent.cpu().numpy(), rp)
    target = torch.randint(0, V, (1, budget + 1), dtype=torch.int32, generator=torch.Generator().manual_seed(1))
    p = parent.cpu().numpy()
    kids = np.flatnonzero(p == -1)
    target[0, 0] = int(token[kids[0]])                          # the target agrees with one root child ...
    grand = np.flatnonzero(p == kids[0])
    if len(grand):
        target[0, kids[0] + 1] = int(token[grand[-1]])          # ... and with one of its children
    n_acc, path, emitted = vt.vt_verify_greedy(token[None].contiguous(), parent[None].contiguous(), target.to(DEV))
    r_acc, r_path, r_emit = oracle.verify_greedy(token.cpu().numpy()[None], p[None], target.numpy())
    assert np.array_equal(n_acc.cpu().numpy(), r_acc) and np.array_equal(path.cpu().numpy(), r_path)
    assert np.array_equal(emitted.cpu().numpy(), r_emit) and int(n_acc.item()) >= 1


@pytest.mark.parametrize("K,d,topk,n_front,depth,sample", [(4096, 512, 8, 8, 3, False), (3000, 1024, 10, 10, 4, True),
                                                            (700, 72, 4, 6, 3, True), (2048, 256, 16, 16, 2, False)])
def test_head_with_fused_expansion_equals_head_then_expansion(K, d, topk, n_front, depth, sample):
    """vt_draft_head_expand (one launch per tree depth on the streaming kernel) against vt_draft_head
    followed by vt_tree_expand: same ids, log-probs, pool and frontier, bit for bit; the pool is also what
    the oracle's expansion makes of those candidates."""
    W = vt_inputs.gaussian_bf16((K, d), 0.05, seed=K + 1, device=DEV)
    m = torch.randperm(K * 2, device=DEV)[:K].to(torch.int32)
    cap = topk + (depth - 1) * n_front * topk
    pool_a, pool_b = vt.tree_pool(cap), vt.tree_pool(cap)
    tok = np.full(cap, -9, dtype=np.int32); par = np.full(cap, -9, dtype=np.int32)
    sc = np.full(cap, np.nan, dtype=np.float32)
    fa = fb = fr = None
    base, B = 0, 1
    for dep in range(depth):
        h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=50 + dep, device=DEV)
        T = vt_inputs.temperatures(B, 0.7, 1.3, seed=60 + dep, device=DEV)
        u = vt_inputs.uniforms((B, K), seed=70 + dep, device=DEV) if sample else None
        nf = min(n_front, B * topk)
        ids_a, lp_a = vt.vt_draft_head(h, W, m, T, topk, u)
        fa = vt.vt_tree_expand(ids_a, lp_a, fa, pool_a, base, nf, col0=1)
        ids_b, lp_b, fb = vt.vt_draft_head_expand(h, W, m, T, topk, u, fb, pool_b, base, nf)
        assert torch.equal(ids_a, ids_b) and torch.equal(lp_a.view(torch.int32), lp_b.view(torch.int32))
        assert torch.equal(fa, fb)
        fr = oracle.tree_expand(ids_a[:, 1:].cpu().numpy(), lp_a[:, 1:].cpu().numpy(), fr, tok, par, sc, base, nf)
        assert np.array_equal(fb.cpu().numpy(), fr)
        base += B * topk
        B = nf
    for x, y in zip(pool_a, pool_b):
        assert torch.equal(x[:base].view(torch.int32), y[:base].view(torch.int32))
    assert np.array_equal(pool_b[0][:base].cpu().numpy(), tok[:base])
    assert np.array_equal(pool_b[1][:base].cpu().numpy(), par[:base])
    assert np.array_equal(_bits(pool_b[2][:base].cpu().numpy()), _bits(sc[:base]))


def test_fused_expansion_on_the_dense_path_and_argument_checks():
    K, d, topk, B = 1500, 128, 8, 40                         # more than 16 rows: tensor-core kernel + chained expansion
    W = vt_inputs.gaussian_bf16((K, d), 0.05, seed=3, device=DEV)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=4, device=DEV)
    T = torch.ones(B, device=DEV)
    cap = 64 + B * topk
    prev = (-torch.arange(cap, dtype=torch.float32, device=DEV) / 5)
    pool_a = (torch.zeros(cap, dtype=torch.int32, device=DEV), torch.full((cap,), -1, dtype=torch.int32, device=DEV), prev.clone())
    pool_b = tuple(t.clone() for t in pool_a)
    front = torch.arange(B, dtype=torch.int32, device=DEV)
    ids_a, lp_a = vt.vt_draft_head(h, W, None, T, topk, None)
    fa = vt.vt_tree_expand(ids_a, lp_a, front, pool_a, 64, 24, col0=1)
    ids_b, lp_b, fb = vt.vt_draft_head_expand(h, W, None, T, topk, None, front, pool_b, 64, 24)
    assert torch.equal(ids_a, ids_b) and torch.equal(fa, fb)
    for x, y in zip(pool_a, pool_b):
        assert torch.equal(x.view(torch.int32), y.view(torch.int32))
    with pytest.raises(vt.VocabTrimError):                     # pool too small for B*topk new nodes
        vt.vt_draft_head_expand(h, W, None, T, topk, None, front, vt.tree_pool(100), 64, 24)
    with pytest.raises(vt.VocabTrimError):                     # several rows need their frontier nodes
        vt.vt_draft_head_expand(h, W, None, T, topk, None, None, vt.tree_pool(cap), 0, 8)
