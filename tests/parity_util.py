"""Comparison rules between the CUDA path and the CPU oracle (test helpers).

Tolerances (stated by the benchmark spec, written out here):
  * histograms, map, inv_map, gathered rows: bit-exact;
  * logits: |err| <= 1e-3 + 1e-3 * |ref|;
  * probabilities exp(logprob): within 1e-5 absolute of the oracle's value for the same index;
  * log-probabilities themselves: |logp - ref| <= 2e-3, which is what the logit tolerance (1e-3 in z at
    T = 1, the lse being an average of the same errors) already implies; the probability test alone
    is blind at p ~ 1e-5, where a sampled id of a 32768-row head lives;
  * greedy / top-k / Gumbel ids: equal to the oracle's, except where the oracle's own margin
    between the two competing candidates is below 1e-3 in logit units, i.e.
    T_b * |score_ref[oracle choice] - score_ref[gpu choice]| < 1e-3 with score = z for candidates
    and z + g for the sample.  Ids inside one row's candidate list must be distinct.
"""
from __future__ import annotations

import numpy as np

import oracle

LOGIT_ATOL = 1e-3
LOGIT_RTOL = 1e-3
PROB_ATOL = 1e-5
LOGP_ATOL = 2e-3
MARGIN = 1e-3


def bits_of(t) -> np.ndarray:
    """bf16 torch tensor (any device) -> uint16 numpy bit patterns."""
    import torch

    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def oracle_head(h, W, map_, temp, topk, uniforms):
    return oracle.draft_head(bits_of(h), bits_of(W), None if map_ is None else map_.cpu().numpy(),
                             temp.cpu().numpy(), topk, None if uniforms is None else uniforms.cpu().numpy())


def check_head(ref, gpu_ids, gpu_lps, temp, map_, gpu_logits=None, gpu_lse=None, sampled=True):
    """Applies the rules above; returns the number of positions accepted through the margin rule."""
    ids = gpu_ids.cpu().numpy()
    lps = gpu_lps.cpu().numpy().astype(np.float64)
    T = temp.cpu().numpy().astype(np.float64)
    B, row = ids.shape
    K = ref.z.shape[1]
    if map_ is None:
        trim = ids.copy()
    else:
        m = map_.cpu().numpy()
        inv = {int(v): j for j, v in enumerate(m)}
        trim = np.array([[inv.get(int(x), -1) for x in r] for r in ids], dtype=np.int64)
    assert np.all((trim >= 0) & (trim < K)), "an emitted id is not in the trimmed vocabulary"
    slack = 0
    for b in range(B):
        assert len(set(trim[b, 1:].tolist())) == row - 1, "duplicate candidate ids in row %d" % b
        for c in range(row):
            jg, jo = int(trim[b, c]), int(ref.trim[b, c])
            score = ref.score[b] if (c == 0 and sampled and ref.score is not None) else ref.z[b]
            if jg != jo:
                gap = T[b] * abs(score[jo] - score[jg])
                assert gap < MARGIN, "row %d col %d: gpu %d vs oracle %d, logit margin %.3e" % (b, c, jg, jo, gap)
                slack += 1
            lp_ref = ref.z[b, jg] - ref.lse[b]
            assert abs(np.exp(lps[b, c]) - np.exp(lp_ref)) <= PROB_ATOL, "row %d col %d: probability off" % (b, c)
            assert abs(lps[b, c] - lp_ref) <= LOGP_ATOL, \
                "row %d col %d: log-prob %.6f vs %.6f" % (b, c, lps[b, c], lp_ref)
    if gpu_logits is not None:
        lg = gpu_logits.cpu().numpy().astype(np.float64)
        err = np.abs(lg - ref.logits)
        assert np.all(err <= LOGIT_ATOL + LOGIT_RTOL * np.abs(ref.logits)), "logit error %.3e" % err.max()
    if gpu_lse is not None:
        assert np.allclose(gpu_lse.cpu().numpy().astype(np.float64), ref.lse, rtol=0, atol=1e-4)
    return slack
