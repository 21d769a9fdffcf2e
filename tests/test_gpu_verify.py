"""GPU parity of greedy verification (Experiments section; Algorithm 2's accept loop) against the
CPU oracle: accepted counts, paths and emitted tokens are integers and compared bit-exactly."""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_22694_b200 as vt
import vt_inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _compare(token, parent, target):
    total = torch.zeros(1, dtype=torch.int64, device=DEV)
    n_acc, path, emitted = vt.vt_verify_greedy(token.to(DEV), parent.to(DEV) if parent is not None else None,
                                               target.to(DEV), tokens_total=total)
    rn, rp, re = oracle.verify_greedy(token.numpy(), parent.numpy() if parent is not None else None,
                                      target.numpy())
    assert np.array_equal(n_acc.cpu().numpy(), rn)
    assert np.array_equal(path.cpu().numpy(), rp)
    assert np.array_equal(emitted.cpu().numpy(), re)
    assert int(total.item()) == int(rn.astype(np.int64).sum()) + len(rn)
    return rn


# depth-3 / top-8 / 32-token and 60-token trees are the paper's draft-tree settings; the rest are
# ragged sizes around the warp width
@pytest.mark.parametrize("S,N,width,vocab,pm", [(1, 1, 1, 4, 0.5), (7, 31, 8, 100, 0.8), (64, 32, 8, 128256, 0.7),
                                                (33, 60, 8, 128256, 0.8), (5, 33, 2, 3, 0.9), (3, 200, 4, 50, 0.95),
                                                (1000, 32, 8, 1000, 0.6)])
def test_verify_trees_match_oracle(S, N, width, vocab, pm):
    token, parent, target = vt_inputs.draft_trees(S, N, width, vocab, pm, seed=S + N)
    rn = _compare(token, parent, target)
    if S >= 30:
        assert rn.max() >= 2 and rn.min() == 0


def test_verify_chains_and_extremes():
    g = torch.Generator().manual_seed(3)
    S, N = 257, 5
    token = torch.randint(0, 3, (S, N), generator=g, dtype=torch.int32)
    target = torch.randint(0, 3, (S, N + 1), generator=g, dtype=torch.int32)
    _compare(token, None, target)
    target[:, :N] = token                                     # every draft accepted: gamma + 1 tokens per block
    rn = _compare(token, None, target)
    assert (rn == N).all()
    target[:, 0] = 7                                          # first token rejected everywhere
    rn = _compare(token, None, target)
    assert (rn == 0).all()
    # a long chain crosses many 32-node scans
    N = 300
    token = torch.arange(N, dtype=torch.int32).repeat(2, 1)
    target = torch.arange(N + 1, dtype=torch.int32).repeat(2, 1)
    target[1, 170] = -5
    rn = _compare(token, None, target)
    assert rn.tolist() == [300, 170]


def test_verify_duplicate_siblings_unreachable_parents_and_accumulation():
    token = torch.tensor([[3, 3, 1, 2], [3, 3, 1, 2]], dtype=torch.int32)
    parent = torch.tensor([[-1, -1, 1, 0], [-1, 5, -7, 3]], dtype=torch.int32)
    target = torch.tensor([[3, 2, 1, 0, 0], [3, 3, 3, 3, 3]], dtype=torch.int32)
    rn = _compare(token, parent, target)
    assert rn.tolist() == [2, 1]
    total = torch.full((1,), 10, dtype=torch.int64, device=DEV)
    for _ in range(3):
        vt.vt_verify_greedy(token.to(DEV), parent.to(DEV), target.to(DEV), tokens_total=total)
    assert int(total.item()) == 10 + 3 * (2 + 1 + 2)
    empty = torch.empty(0, 4, dtype=torch.int32, device=DEV)
    n_acc, _, _ = vt.vt_verify_greedy(empty, None, torch.empty(0, 5, dtype=torch.int32, device=DEV))
    assert n_acc.numel() == 0


def test_draft_then_verify_only_accepts_ids_of_the_trimmed_vocabulary():
    """Algorithm 2 end to end on synthetic weights: drafted ids come out of the trimmed head through
    the index mapper, so a target token outside the kept set can never be accepted."""
    V, K, d, B = 4096, 512, 256, 16
    ids = vt_inputs.zipf_ids(200_000, V, 1.1, seed=2, device=DEV)
    map_, inv = vt.vt_build_vocab(ids, V, K)
    W = vt_inputs.gaussian_bf16((V, d), 0.05, seed=3, device=DEV)
    Wt = vt.vt_trim_head(W, map_)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=4, device=DEV)
    temp = torch.ones(B, dtype=torch.float32, device=DEV)
    out_ids, _ = vt.vt_draft_head(h, Wt, map_, temp, topk=1)
    draft = out_ids[:, 1:2].contiguous()                       # the top-1 id per sequence: chains of length 1
    kept = set(map_.cpu().tolist())
    assert all(int(t) in kept for t in draft.flatten().cpu())
    target = torch.empty(B, 2, dtype=torch.int32, device=DEV)
    target[:, 1] = 0
    target[:8, 0] = draft[:8, 0]                               # target agrees on the first half
    outside = [t for t in range(V) if t not in kept][:8]
    target[8:, 0] = torch.tensor(outside, dtype=torch.int32, device=DEV)
    n_acc, _, emitted = vt.vt_verify_greedy(draft, None, target)
    assert n_acc.cpu().tolist() == [1] * 8 + [0] * 8
    rn, _, re = oracle.verify_greedy(draft.cpu().numpy(), None, target.cpu().numpy())
    assert np.array_equal(n_acc.cpu().numpy(), rn) and np.array_equal(emitted.cpu().numpy(), re)
