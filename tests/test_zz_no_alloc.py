"""vt_select_topk_static: the workspace-free selection for callers that cannot allocate.

Runs last on purpose (file name): if it fails under `-x`, every other test has already run.
The entry point is driven through the C ABI directly, twice in a row with different inputs --
its scratch is one array shared by all calls, so a second call sees the first call's leftovers --
and must reproduce vt_select_topk bit for bit (integer work: the tolerance is zero).
"""
import ctypes

import numpy as np
import pytest
import torch

import paper_2506_22694_b200 as vt
import vt_inputs

pytestmark = pytest.mark.gpu


def _call_static(counts, K):
    V = counts.numel()
    map_ = torch.full((K,), -7, dtype=torch.int32, device=counts.device)
    inv = torch.full((V,), -7, dtype=torch.int32, device=counts.device)
    st = vt.lib().vt_select_topk_static(ctypes.c_void_p(counts.data_ptr()), V, K,
                                        ctypes.c_void_p(map_.data_ptr()), ctypes.c_void_p(inv.data_ptr()),
                                        ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert st == vt.VT_OK, vt.status_str(st)
    return map_, inv


def test_static_selection_matches_workspace_selection_twice_in_a_row():
    dev = torch.device("cuda", 0)
    cases = [(vt_inputs.LLAMA3_VOCAB, 32768, 1.07, 11), (50_000, 777, 1.3, 12)]   # second call: smaller V, stale tail
    for V, K, s, seed in cases:
        ids = vt_inputs.zipf_ids(300_000, V, s, seed=seed, device=dev)
        counts = vt.vt_histogram(ids, V)
        ref_map, ref_inv = vt.vt_select_topk(counts, K)
        got_map, got_inv = _call_static(counts, K)
        torch.cuda.synchronize()
        assert torch.equal(got_map, ref_map)
        assert torch.equal(got_inv, ref_inv)
        # massive ties: the result is still unique (count descending, id ascending)
        flat = torch.full((V,), 3, dtype=torch.int32, device=dev)
        ref_map, ref_inv = vt.vt_select_topk(flat, K)
        got_map, got_inv = _call_static(flat, K)
        torch.cuda.synchronize()
        assert torch.equal(got_map, ref_map) and torch.equal(got_inv, ref_inv)
        assert np.array_equal(got_map.cpu().numpy(), np.arange(K, dtype=np.int32))


def test_static_selection_rejects_what_it_cannot_hold():
    dev = torch.device("cuda", 0)
    L = vt.lib()
    null = ctypes.c_void_p(0)
    big = torch.zeros(131073, dtype=torch.int32, device=dev)
    out = torch.zeros(131073, dtype=torch.int32, device=dev)
    p = lambda t: ctypes.c_void_p(t.data_ptr())
    assert L.vt_select_topk_static(p(big), 131073, 8, p(out), p(out), null) == 6      # VT_ERR_UNSUPPORTED
    assert L.vt_select_topk_static(null, 100, 8, p(out), p(out), null) == 1           # VT_ERR_INVALID_ARG
    assert L.vt_select_topk_static(p(big), 100, 101, p(out), p(out), null) == 1
