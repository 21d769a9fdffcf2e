"""GPU parity of the trimmed drafter head (Algorithm 2, the drafter-forward and index-mapping steps) against the fp64 CPU oracle on
seeded synthetic inputs: logits, log-probabilities, greedy / top-k / Gumbel ids and the remap."""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_22694_b200 as vt
import vt_inputs
from parity_util import check_head, oracle_head

pytestmark = pytest.mark.gpu
DEV = "cuda"
V3 = vt_inputs.LLAMA3_VOCAB


def _vocab_map(V, K, seed):
    """A map built by the real path from 1e7 synthetic ids of the corpus distribution."""
    ids = vt_inputs.zipf_ids(10_000_000, V, 1.07, seed=seed, noise_frac=0.05, device=DEV)
    m, inv = vt.vt_build_vocab(ids, V, K)
    return m, inv


def _run(h, W, m, temp, topk, u, debug=True, ws=None):
    out = vt.vt_draft_head(h, W, m, temp, topk, u, ws=ws, debug=debug)
    torch.cuda.synchronize()
    return out


def test_config1_tiny_end_to_end():
    V, d, K, topk = 4096, 256, 1024, 4
    ids = vt_inputs.zipf_ids(100_000, V, 1.1, seed=1001, device=DEV)
    m, inv = vt.vt_build_vocab(ids, V, K)
    W = vt_inputs.gaussian_bf16((V, d), 0.02, seed=1002, device=DEV)
    Wt = vt.vt_trim_head(W, m)
    h = vt_inputs.gaussian_bf16((1, d), 1.0, seed=1003, device=DEV)
    T = vt_inputs.temperatures(1, 1.0, 1.0, 0, device=DEV)
    u = vt_inputs.uniforms((1, K), seed=1004, device=DEV)
    gi, gl, lg, lse = _run(h, Wt, m, T, topk, u)
    ref = oracle_head(h, Wt, m, T, topk, u)
    check_head(ref, gi, gl, T, m, lg, lse)
    trim = inv.cpu().numpy()[gi.cpu().numpy()]                   # inverse map recovers the trimmed index
    assert np.all(trim >= 0) and np.array_equal(m.cpu().numpy()[trim], gi.cpu().numpy())


@pytest.mark.parametrize("B,K,d,topk,sample", [
    (1, 8, 8, 1, True), (1, 9, 16, 9, True), (2, 100, 40, 7, True), (3, 1000, 264, 64, True),
    (4, 5003, 1024, 8, False), (7, 2048, 3072, 8, True), (8, 777, 4096, 10, True),
    (9, 4099, 4096, 10, True), (16, 3000, 2048, 16, True), (13, 12345, 1000, 5, True),
    (16, 1031, 4096, 64, True), (5, 64, 8192, 4, True),
])
def test_small_shapes_and_ragged_tails(B, K, d, topk, sample):
    W = vt_inputs.gaussian_bf16((K, d), 0.02, seed=K + d, device=DEV)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=B + 17, device=DEV)
    T = vt_inputs.temperatures(B, 0.5, 1.5, seed=K, device=DEV)
    u = vt_inputs.uniforms((B, K), seed=d + 1, device=DEV) if sample else None
    m = torch.randperm(K * 3, device=DEV)[:K].to(torch.int32)        # any injective map works for the remap
    gi, gl, lg, lse = _run(h, W, m, T, topk, u)
    ref = oracle_head(h, W, m, T, topk, u)
    check_head(ref, gi, gl, T, m, lg, lse, sampled=sample)
    if not sample:
        assert torch.equal(gi[:, 0], gi[:, 1]) and torch.equal(gl[:, 0], gl[:, 1])


def test_identity_map_equals_null_map_and_is_deterministic():
    B, K, d, topk = 10, 20_000, 4096, 10
    W = vt_inputs.gaussian_bf16((K, d), 0.02, seed=1, device=DEV)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=2, device=DEV)
    T = vt_inputs.temperatures(B, 0.7, 0.7, 0, device=DEV)
    u = vt_inputs.uniforms((B, K), seed=3, device=DEV)
    ident = torch.arange(K, dtype=torch.int32, device=DEV)
    a = _run(h, W, None, T, topk, u, debug=False)
    b = _run(h, W, ident, T, topk, u, debug=False)
    c = _run(h, W, None, T, topk, u, debug=False)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    assert torch.equal(a[0], c[0]) and torch.equal(a[1], c[1])            # bitwise run-to-run


def test_ties_go_to_the_lower_index():
    B, K, d = 2, 512, 64
    W = torch.zeros((K, d), dtype=torch.bfloat16, device=DEV)
    W[:, 0] = 1.0
    W[100:104, 0] = 2.0                                  # four tied maxima, everything else tied below
    h = torch.zeros((B, d), dtype=torch.bfloat16, device=DEV)
    h[:, 0] = 1.0
    T = vt_inputs.temperatures(B, 1.0, 1.0, 0, device=DEV)
    u = torch.full((B, K), 0.5, dtype=torch.float32, device=DEV)       # equal uniforms: sample == greedy
    gi, gl = _run(h, W, None, T, 8, u, debug=False)
    assert gi[0].tolist() == [100, 100, 101, 102, 103, 0, 1, 2, 3]
    ref = oracle_head(h, W, None, T, 8, u)
    assert np.array_equal(gi.cpu().numpy(), ref.ids)


def test_uniform_edge_values_are_clamped():
    B, K, d = 1, 256, 64
    W = vt_inputs.gaussian_bf16((K, d), 0.02, seed=5, device=DEV)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=6, device=DEV)
    T = vt_inputs.temperatures(B, 1.0, 1.0, 0, device=DEV)
    u = vt_inputs.uniforms((B, K), seed=7, device=DEV)
    u[0, 10] = 0.0
    u[0, 20] = 1.0                                       # clamps to 1 - 2^-24: a huge Gumbel, must win
    u[0, 30] = -3.0
    u[0, 40] = 7.0
    gi, gl = _run(h, W, None, T, 4, u, debug=False)
    ref = oracle_head(h, W, None, T, 4, u)
    check_head(ref, gi, gl, T, None)
    assert int(gi[0, 0]) in (20, 40)


def test_bad_temperature_is_flagged_not_fatal():
    B, K, d = 3, 300, 128
    W = vt_inputs.gaussian_bf16((K, d), 0.02, seed=8, device=DEV)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=9, device=DEV)
    T = torch.tensor([1.0, 0.0, 0.8], dtype=torch.float32, device=DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, K, d, B, 4))
    gi, gl = _run(h, W, None, T, 4, None, debug=False, ws=ws)
    st, flags, _ = ws.read_status()
    assert st == 7 and flags & vt.VT_FLAG_BAD_TEMP
    assert gi[1].tolist() == [-1] * 5 and bool(torch.isnan(gl[1]).all())
    ref = oracle_head(h[[0, 2]], W, None, T[[0, 2]], 4, None)
    check_head(ref, gi[[0, 2]], gl[[0, 2]], T[[0, 2]], None, sampled=False)
    gi2, _ = _run(h, W, None, torch.ones(B, device=DEV), 4, None, debug=False, ws=ws)   # workspace still usable
    assert ws.read_status()[0] == 0 and int(gi2.min()) >= 0


def test_an_expired_wait_is_reported_and_the_workspace_stays_usable():
    """Every device-side wait is bounded.  With the bound set to 1 ns the first wait that is not
    satisfied at once (the first stage of weights is still on its way) gives up: the kernel lets its
    copies land, reports VT_ERR_TIMEOUT and marks every row missing; nothing hangs, nothing is broken
    on purpose.  With the default bound back, the same workspace serves a clean call."""
    B, K, d, topk = 2, 20_000, 3072, 8
    W = vt_inputs.gaussian_bf16((K, d), 0.02, seed=21, device=DEV)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=22, device=DEV)
    T = vt_inputs.temperatures(B, 1.0, 1.0, 0, device=DEV)
    u = vt_inputs.uniforms((B, K), seed=23, device=DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, K, d, B, topk))
    good = tuple(t.clone() for t in _run(h, W, None, T, topk, u, debug=False, ws=ws))
    assert ws.read_status() == (0, 0, 0)
    ws.set_wait_limit(1)
    gi, gl = _run(h, W, None, T, topk, u, debug=False, ws=ws)
    st, flags, _ = ws.read_status()
    assert st == 5 and flags & vt.VT_FLAG_TIMEOUT                    # VT_ERR_TIMEOUT
    assert bool((gi == -1).all()) and bool(torch.isnan(gl).all())
    ws.set_wait_limit(0)
    for _ in range(2):
        gi, gl = _run(h, W, None, T, topk, u, debug=False, ws=ws)
        assert torch.equal(gi, good[0]) and torch.equal(gl, good[1])
    assert ws.read_status() == (0, 0, 0)


SLACK = {}            # workload -> [positions accepted through the margin rule, positions compared]


def _tally(name, slack, positions):
    acc = SLACK.setdefault(name, [0, 0])
    acc[0] += slack
    acc[1] += positions
    print("parity_slack %s: %d of %d positions accepted through the 1e-3 logit margin" % (name, slack, positions))


def test_config2_chain_drafting_trimmed_vs_full_head():
    """V=128256, d=3072, K=32768, B=1, 7 sequential steps, greedy + top-8, against the full head."""
    d, K, topk, steps = 3072, 32768, 8, 7
    m, inv = _vocab_map(V3, K, seed=1102)
    W = vt_inputs.gaussian_bf16((V3, d), 0.02, seed=1002, device=DEV)
    Wt = vt.vt_trim_head(W, m)
    T = vt_inputs.temperatures(1, 1.0, 1.0, 0, device=DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, V3, d, 1, topk))
    Wb = vt_inputs.bf16_bits(W).cpu().numpy().view(np.uint16)
    mh = m.cpu().numpy()
    slack = 0
    for step in range(steps):
        h = vt_inputs.gaussian_bf16((1, d), 1.0, seed=2000 + step, device=DEV)
        gi, gl, lg, lse = _run(h, Wt, m, T, topk, None, ws=ws)
        ref = oracle_head(h, Wt, m, T, topk, None)
        slack += check_head(ref, gi, gl, T, m, lg, lse, sampled=False)
        fi, fl, flg, flse = _run(h, W, None, T, topk, None, ws=ws)            # full K = V head, identity map
        if step < 2:
            full = oracle_head(h, W, None, T, topk, None)
            slack += check_head(full, fi, fl, T, None, flg, flse, sampled=False)
            # trimmed logits are the full head's logits at the mapped rows (oracle: exactly)
            assert np.array_equal(ref.logits[0], full.logits[0, mh])
        assert torch.allclose(lg[0], flg[0, m.long()], rtol=0, atol=2e-5)
    _tally("config2 K=32768 and K=V", slack, (steps + 2) * (1 + topk))
    assert slack <= 1
    assert ws.read_status() == (0, 0, 0)


@pytest.mark.parametrize("K", [8192, 16384, 32768, 65536, V3])
def test_config3_tree_drafting_sweep(K):
    """V=128256, d=4096, B=10 nodes, top-10, T=0.7, Gumbel sampling, 6 tree depths at every K of the
    sweep; K = V uses the identity map.  Every logit, log-probability and id meets the oracle."""
    d, B, topk, depths = 4096, 10, 10, 6
    W = vt_inputs.gaussian_bf16((V3, d), 0.02, seed=1003, device=DEV)
    if K == V3:
        m, Wt = None, W
    else:
        m, _ = _vocab_map(V3, K, seed=1103)
        Wt = vt.vt_trim_head(W, m)
        del W
    T = vt_inputs.temperatures(B, 0.7, 0.7, 0, device=DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, K, d, B, topk))
    slack = 0
    for depth in range(depths):
        h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=3000 + depth, device=DEV)
        u = vt_inputs.uniforms((B, K), seed=4000 + depth, device=DEV)
        gi, gl, lg, lse = _run(h, Wt, m, T, topk, u, ws=ws)
        ref = oracle_head(h, Wt, m, T, topk, u)
        slack += check_head(ref, gi, gl, T, m, lg, lse)
        # the timed entry point (no logits written) returns the same bits
        gi2, gl2 = _run(h, Wt, m, T, topk, u, debug=False, ws=ws)
        assert torch.equal(gi, gi2) and torch.equal(gl, gl2)
    positions = depths * B * (1 + topk)
    _tally("config3 K=%d" % K, slack, positions)
    assert slack <= 0.005 * positions + 1
    assert ws.read_status() == (0, 0, 0)


# ---- dense tensor-core path (more than 16 hidden rows, or shapes the streaming kernel does not take) ----
@pytest.mark.parametrize("B,K,d,topk,sample", [
    (17, 300, 72, 5, True), (40, 1000, 256, 8, True), (64, 128, 64, 1, False), (130, 515, 200, 16, True),
    (256, 2048, 512, 8, True), (128, 4099, 1024, 4, True), (12, 700, 4104, 6, True), (200, 9, 8, 9, True),
    (129, 300, 64, 3, True),
    # four tiles per CTA (pair): both accumulator stages are reused, the ring wraps many times
    (256, 60000, 64, 8, True), (100, 150001, 72, 4, False),
])
def test_dense_path_small_shapes_and_ragged_tails(B, K, d, topk, sample):
    W = vt_inputs.gaussian_bf16((K, d), 0.02, seed=K + d, device=DEV)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=B + 17, device=DEV)
    T = vt_inputs.temperatures(B, 0.5, 1.5, seed=K, device=DEV)
    u = vt_inputs.uniforms((B, K), seed=d + 1, device=DEV) if sample else None
    m = torch.randperm(K * 3, device=DEV)[:K].to(torch.int32)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, K, d, B, topk))
    gi, gl, lg, lse = _run(h, W, m, T, topk, u, ws=ws)
    ref = oracle_head(h, W, m, T, topk, u)
    check_head(ref, gi, gl, T, m, lg, lse, sampled=sample)
    assert ws.read_status() == (0, 0, 0)
    # the timed entry point (no logits written) must give the same ids, twice in a row
    a = _run(h, W, m, T, topk, u, debug=False, ws=ws)
    b = _run(h, W, m, T, topk, u, debug=False, ws=ws)
    assert torch.equal(a[0], gi) and torch.equal(b[0], gi) and torch.equal(a[1], b[1])


def test_dense_path_uniforms_need_no_16_byte_alignment():
    """The header asks 16-byte alignment of the bf16 tensors only: a [B,K] fp32 view that starts 4 bytes
    into an allocation must give the result of an aligned copy."""
    B, K, d, topk = 40, 1000, 256, 8
    W = vt_inputs.gaussian_bf16((K, d), 0.02, seed=11, device=DEV)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=12, device=DEV)
    T = vt_inputs.temperatures(B, 0.5, 1.5, seed=13, device=DEV)
    u = vt_inputs.uniforms((B, K), seed=14, device=DEV)
    flat = torch.empty(B * K + 1, dtype=torch.float32, device=DEV)
    shifted = flat[1:].view(B, K)
    shifted.copy_(u)
    assert shifted.data_ptr() % 16 == 4
    a = _run(h, W, None, T, topk, u, debug=False)
    b = _run(h, W, None, T, topk, shifted, debug=False)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_dense_path_rejects_long_candidate_lists():
    W = vt_inputs.gaussian_bf16((256, 64), 0.02, seed=1, device=DEV)
    h = vt_inputs.gaussian_bf16((32, 64), 1.0, seed=2, device=DEV)
    assert vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, 256, 64, 32, 17) == 0
    with pytest.raises((vt.VocabTrimError, ValueError)):
        vt.vt_draft_head(h, W, None, torch.ones(32, device=DEV), 17, None)


def test_config4_batched_serving_dense_head():
    """64 sequences x 4 tree nodes = 256 rows, d=4096, V=128256, K=32768, per-row T in [0.5,1.5],
    top-8, Gumbel sampling.  All 256 rows meet the oracle at the full K in the launch configuration the
    benchmark times (ids, log-probabilities); the logits themselves are compared on a 4096-row slice
    of the trimmed head (a full dump would be 33 MB of fp32 per call for no extra coverage)."""
    d, K, B, topk = 4096, 32768, 256, 8
    m, _ = _vocab_map(V3, K, seed=1104)
    W = vt_inputs.gaussian_bf16((V3, d), 0.02, seed=1004, device=DEV)
    Wt = vt.vt_trim_head(W, m)
    del W
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=5000, device=DEV)
    T = vt_inputs.temperatures(B, 0.5, 1.5, seed=5001, device=DEV)
    u = vt_inputs.uniforms((B, K), seed=5002, device=DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, K, d, B, topk))
    # slice: all 256 rows against the first 4096 vocabulary rows, logits included
    Ks = 4096
    us = u[:, :Ks].contiguous()
    gi, gl, lg, lse = _run(h, Wt[:Ks], m[:Ks], T, topk, us, ws=ws)
    ref = oracle_head(h, Wt[:Ks], m[:Ks], T, topk, us)
    slack = check_head(ref, gi, gl, T, m[:Ks], lg, lse)
    _tally("config4 slice K=4096", slack, B * (1 + topk))
    assert slack <= 0.005 * B * (1 + topk) + 1
    # full size, launch configuration of the benchmark: every row against the oracle
    gi, gl = _run(h, Wt, m, T, topk, u, debug=False, ws=ws)
    ref = oracle_head(h, Wt, m, T, topk, u)
    slack = check_head(ref, gi, gl, T, m)
    _tally("config4 K=32768", slack, B * (1 + topk))
    assert slack <= 0.005 * B * (1 + topk) + 1
    gi2, gl2 = _run(h, Wt, m, T, topk, u, debug=False, ws=ws)
    assert torch.equal(gi, gi2) and torch.equal(gl, gl2)                  # bitwise run-to-run
    assert ws.read_status() == (0, 0, 0)


def test_overlapped_launch_matches_plain_launch_over_a_chain_of_steps():
    """vt_draft_head_overlapped lets a step fetch weights while the previous step is finishing; the
    results must be those of plain calls, step after step, with the workspace shared."""
    K, d, topk = 20_000, 3072, 8
    Ws = [vt_inputs.gaussian_bf16((K, d), 0.02, seed=50 + i, device=DEV) for i in range(3)]
    T = vt_inputs.temperatures(1, 1.0, 1.0, 0, device=DEV)
    hs = [vt_inputs.gaussian_bf16((1, d), 1.0, seed=60 + i, device=DEV) for i in range(12)]
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, K, d, 1, topk))
    plain = []
    for i, h in enumerate(hs):
        ids, lps = vt.vt_draft_head(h, Ws[i % 3], None, T, topk, None, ws=ws)
        plain.append((ids.clone(), lps.clone()))
    torch.cuda.synchronize()                                   # weights are final from here on
    outs = [(torch.empty_like(plain[0][0]), torch.empty_like(plain[0][1])) for _ in hs]
    for i, h in enumerate(hs):                                 # back to back, nothing in between
        vt.vt_draft_head(h, Ws[i % 3], None, T, topk, None, ws=ws, out=outs[i], overlapped=True)
    torch.cuda.synchronize()
    for (pi, pl), (oi, ol) in zip(plain, outs):
        assert torch.equal(pi, oi) and torch.equal(pl, ol)
    # tree-drafting shape with sampling and a map
    B, topk = 10, 10
    W = vt_inputs.gaussian_bf16((K, 4096), 0.02, seed=70, device=DEV)
    m = torch.randperm(K * 2, device=DEV)[:K].to(torch.int32)
    T = vt_inputs.temperatures(B, 0.7, 0.7, 0, device=DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD, 0, 0, K, 4096, B, topk))
    hs = [vt_inputs.gaussian_bf16((B, 4096), 1.0, seed=80 + i, device=DEV) for i in range(6)]
    us = [vt_inputs.uniforms((B, K), seed=90 + i, device=DEV) for i in range(6)]
    plain = [tuple(t.clone() for t in vt.vt_draft_head(h, W, m, T, topk, u, ws=ws)) for h, u in zip(hs, us)]
    torch.cuda.synchronize()
    outs = [(torch.empty_like(plain[0][0]), torch.empty_like(plain[0][1])) for _ in hs]
    for i in range(6):
        vt.vt_draft_head(hs[i], W, m, T, topk, us[i], ws=ws, out=outs[i], overlapped=True)
    torch.cuda.synchronize()
    for (pi, pl), (oi, ol) in zip(plain, outs):
        assert torch.equal(pi, oi) and torch.equal(pl, ol)
    assert ws.read_status() == (0, 0, 0)


def test_all_candidates_in_one_slab_of_the_vocabulary():
    """The cross-CTA merge first tries a direct selection over the few best entries of every CTA's
    list; when one CTA holds most of the global candidates that shortcut must notice and fall back."""
    B, K, d, topk = 3, 8192, 128, 10
    W = vt_inputs.gaussian_bf16((K, d), 0.02, seed=77, device=DEV)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=78, device=DEV)
    W[3:19] = (h[0].float() * 0.05).to(torch.bfloat16)         # 16 neighbouring rows aligned with h[0]: huge logits
    W[5] = (h[0].float() * 0.06).to(torch.bfloat16)
    T = vt_inputs.temperatures(B, 1.0, 1.0, 0, device=DEV)
    u = vt_inputs.uniforms((B, K), seed=79, device=DEV)
    gi, gl, lg, lse = _run(h, W, None, T, topk, u)
    ref = oracle_head(h, W, None, T, topk, u)
    check_head(ref, gi, gl, T, None, lg, lse)
    assert set(gi[0, 1:].tolist()) <= set(range(3, 19))


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("B,K,d,topk,sample", [(1, 4099, 1024, 8, False), (10, 3000, 512, 10, True), (40, 700, 128, 4, True)])
def test_host_entry_point_matches_device_entry_point(B, K, d, topk, sample, pinned):
    """vt_draft_head_host with page-locked buffers (used in place by the kernels) and with pageable ones
    (staged through the workspace) returns what vt_draft_head returns on device copies of the same data."""
    W = vt_inputs.gaussian_bf16((K, d), 0.02, seed=K, device=DEV)
    m = torch.randperm(K * 2, device=DEV)[:K].to(torch.int32)
    h = vt_inputs.gaussian_bf16((B, d), 1.0, seed=B)
    T = vt_inputs.temperatures(B, 0.5, 1.5, seed=d)
    u = vt_inputs.uniforms((B, K), seed=3) if sample else None
    out = (torch.full((B, 1 + topk), -7, dtype=torch.int32), torch.zeros((B, 1 + topk), dtype=torch.float32))
    if pinned:
        h, T = h.pin_memory(), T.pin_memory()
        u = u.pin_memory() if u is not None else None
        out = tuple(t.pin_memory() for t in out)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_DRAFT_HEAD_HOST, 0, 0, K, d, B, topk))
    for _ in range(2):
        ids, lps = vt.vt_draft_head_host(h, W, m, T, topk, u, ws, out)
        torch.cuda.synchronize()
        ref_ids, ref_lps = vt.vt_draft_head(h.to(DEV), W, m, T.to(DEV), topk, u.to(DEV) if u is not None else None)
        assert torch.equal(ids, ref_ids.cpu())
        assert torch.equal(lps.view(torch.int32), ref_lps.cpu().view(torch.int32))
    assert ws.read_status() == (0, 0, 0)


def test_zz_parity_slack_report():
    """Totals of the margin-rule acceptances over the full-size configurations run above (printed with
    -s or -rP); the expectation is a handful at most, since a GPU id differs from the oracle's only
    where fp32 rounding flips two candidates whose fp64 scores are within ~1e-5."""
    for name in sorted(SLACK):
        print("parity_slack total %s: %d of %d" % (name, SLACK[name][0], SLACK[name][1]))
    tot = sum(v[0] for v in SLACK.values())
    pos = sum(v[1] for v in SLACK.values())
    assert tot <= 0.005 * pos + 1
