"""GPU parity of the vocabulary build (Algorithm 1, Eq. 1) against the CPU oracle: bit-exact
histograms, maps, inverse maps and gathered heads, on seeded synthetic id streams."""
import numpy as np
import pytest
import torch

import oracle
import paper_2506_22694_b200 as vt
import vt_inputs

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _u32(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint32).astype(np.uint64)


def _assert_clean(ws):
    st, flags, bad = ws.read_status()
    assert (st, flags, bad) == (0, 0, 0)


@pytest.mark.parametrize("n,V", [(0, 4096), (1, 4096), (7, 100), (100_000, 4096), (250_003, 50_000),
                                 (1_000_003, 128256), (3_000_000, 57_345), (777, 128256),
                                 (2_000_000, 655_360), (500_000, 300_001)])
def test_histogram_matches_oracle(n, V):
    ids = vt_inputs.zipf_ids(n, V, 1.1, seed=100 + n % 97, noise_frac=0.05, device=DEV) if n else \
        torch.empty(0, dtype=torch.int32, device=DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_HISTOGRAM, n, V))
    counts = vt.vt_histogram(ids, V, ws=ws)
    ref, bad = oracle.histogram(ids.cpu().numpy(), V)
    assert bad == 0
    assert np.array_equal(_u32(counts), ref)
    _assert_clean(ws)


def test_histogram_unaligned_start_and_accumulate():
    V = 128256
    base = vt_inputs.zipf_ids(2_000_011, V, 1.07, seed=7, noise_frac=0.05, device=DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_HISTOGRAM, base.numel(), V))
    for off in (1, 2, 3):
        ids = base[off:]                                   # 4-byte aligned only
        counts = vt.vt_histogram(ids, V, ws=ws)
        ref, _ = oracle.histogram(ids.cpu().numpy(), V)
        assert np.array_equal(_u32(counts), ref)
    counts = vt.vt_histogram(base[:900_000], V, ws=ws)
    vt.vt_histogram(base[900_000:], V, counts=counts, accumulate=True, ws=ws)
    ref, _ = oracle.histogram(base.cpu().numpy(), V)
    assert np.array_equal(_u32(counts), ref)
    _assert_clean(ws)


@pytest.mark.parametrize("V", [4096, 128256])
def test_histogram_skips_and_reports_out_of_range_ids(V):
    ids = vt_inputs.zipf_ids(300_000, V, 1.1, seed=9, device=DEV)
    ids[::1000] = V                 # just past the end
    ids[1::1000] = -1
    ids[2::5000] = 2**31 - 1
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_HISTOGRAM, ids.numel(), V))
    counts = vt.vt_histogram(ids, V, ws=ws)
    ref, bad = oracle.histogram(ids.cpu().numpy(), V)
    assert bad > 0 and np.array_equal(_u32(counts), ref)
    st, flags, n_bad = ws.read_status()
    assert st == 2 and flags & vt.VT_FLAG_BAD_ID and n_bad == bad
    assert ws.read_status() == (0, 0, 0)                   # flags are cleared by the read


@pytest.mark.parametrize("V,bins,n", [(128256, 57344, 1_000_003), (128256, 1000, 50_000), (300_000, 7, 100_001), (64, 64, 1000)])
def test_folded_histogram_counts_ids_modulo_the_bins(V, bins, n):
    ids = vt_inputs.zipf_ids(n, V, 1.07, seed=5, noise_frac=0.05, device=DEV)
    ids[::997] = V + 3                                            # skipped
    got = _u32(vt.vt_histogram_folded(ids, V, bins))
    full, _ = oracle.histogram(ids.cpu().numpy(), V)              # the oracle's histogram, folded on the host
    ref = np.zeros(bins, dtype=np.uint64)
    np.add.at(ref, np.arange(V) % bins, full)
    assert np.array_equal(got, ref)


def test_histogram_degenerate_streams():
    V = 128256
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_HISTOGRAM, 1 << 20, V))
    one = torch.full((1 << 20,), 77_777, dtype=torch.int32, device=DEV)       # a single hot bin
    c = _u32(vt.vt_histogram(one, V, ws=ws))
    assert c[77_777] == 1 << 20 and c.sum() == 1 << 20
    ramp = (torch.arange(1 << 20, device=DEV, dtype=torch.int32) % V).contiguous()  # every bin cold and equal
    ref, _ = oracle.histogram(ramp.cpu().numpy(), V)
    assert np.array_equal(_u32(vt.vt_histogram(ramp, V, ws=ws)), ref)


@pytest.mark.parametrize("V", [57_345, 100_003, 128256, 151_936, 172_032, 172_033])
def test_histogram_every_vocabulary_size_around_the_packed_layout(V):
    """Sizes on both sides of what three bins per shared-memory word can hold, with ids on the field borders."""
    n = 3_000_017
    ids = vt_inputs.zipf_ids(n, V, 1.07, seed=V % 1000, noise_frac=0.05, device=DEV)
    W = (V + 2) // 3
    edge = torch.tensor([0, W - 1, W, W + 1, 2 * W - 1, 2 * W, 2 * W + 1, V - 1], dtype=torch.int32, device=DEV).clamp_(0, V - 1)
    ids[:: 1013] = edge[torch.arange(ids[::1013].numel(), device=DEV) % edge.numel()]
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_HISTOGRAM, n, V))
    ref, bad = oracle.histogram(ids.cpu().numpy(), V)
    assert bad == 0
    assert np.array_equal(_u32(vt.vt_histogram(ids, V, ws=ws)), ref)
    _assert_clean(ws)


def test_histogram_hot_tokens_that_arrive_late_and_skipped_ids_are_counted_once():
    """A stream whose first part is flat and whose second part is mostly two tokens, with ids outside
    [0, V) sprinkled in: whichever kernels end up counting it, every id is counted once and every skipped id
    is reported once."""
    V = 128256
    n = 24_000_000
    g = torch.Generator(device=DEV).manual_seed(5)
    ids = torch.randint(0, V, (n,), device=DEV, dtype=torch.int32, generator=g)
    late = ids[n // 2:]
    u = torch.rand(late.numel(), device=DEV, generator=g)
    late[u < 0.45] = 31_337
    late[(u >= 0.45) & (u < 0.85)] = 90_001
    ids[5::100_003] = V
    ids[7::200_003] = -3
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_HISTOGRAM, n, V))
    ref, bad = oracle.histogram(ids.cpu().numpy(), V)
    assert bad > 0
    for _ in range(2):                                          # the second call starts from a used workspace
        got = _u32(vt.vt_histogram(ids, V, ws=ws))
        assert np.array_equal(got, ref)
        st, flags, n_bad = ws.read_status()
        assert flags == vt.VT_FLAG_BAD_ID and n_bad == bad


@pytest.mark.parametrize("shares", [(0.05,), (0.125, 0.125), (0.2,), (0.35, 0.1), (0.6,), (0.3, 0.3, 0.3), (1.0,)])
def test_histogram_skewed_streams_whichever_kernels_count_them(shares):
    """Streams in which one to three tokens hold the given shares, plus a run of 700 000 repeats of one token
    in the middle: some stay with the packed kernel, some make a field wrap and are counted again."""
    V, n = 128256, 8_000_000
    g = torch.Generator(device=DEV).manual_seed(int(sum(shares) * 1000) + len(shares))
    ids = torch.randint(0, V, (n,), device=DEV, dtype=torch.int32, generator=g)
    u = torch.rand(n, device=DEV, generator=g)
    lo = 0.0
    for k, sh in enumerate(shares):
        ids[(u >= lo) & (u < lo + sh)] = (k * 40_009 + 17) % V
        lo += sh
    ids[n // 3: n // 3 + 700_000] = 99_991
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_HISTOGRAM, n, V))
    ref, bad = oracle.histogram(ids.cpu().numpy(), V)
    assert bad == 0
    assert np.array_equal(_u32(vt.vt_histogram(ids, V, ws=ws)), ref)
    _assert_clean(ws)


def test_histogram_three_ids_carry_the_whole_stream():
    """Streams that drive single bins to 1e7 and more: neighbouring ids, ids around the middle and the
    end of the vocabulary, with a sprinkle of a fourth id."""
    V = 128256
    n = 40_000_000
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_HISTOGRAM, n, V))
    for a, b, c in ((4, 5, 6), (114_687, 114_688, 0), (128_255, 128_254, 57_345)):
        i = torch.arange(n, device=DEV, dtype=torch.int32)
        ids = torch.where(i % 3 == 0, a, torch.where(i % 3 == 1, b, c)).to(torch.int32)
        ids[::1_000_003] = 99_999                                   # a sprinkle of something else
        got = _u32(vt.vt_histogram(ids, V, ws=ws))
        ref = torch.bincount(ids.long(), minlength=V).cpu().numpy().astype(np.uint64)   # integers: torch counts as the oracle does
        small, _ = oracle.histogram(ids[:300_000].cpu().numpy(), V)
        assert np.array_equal(torch.bincount(ids[:300_000].long(), minlength=V).cpu().numpy().astype(np.uint64), small)
        assert np.array_equal(got, ref)
        _assert_clean(ws)
    acc = vt.vt_histogram(ids, V, ws=ws)                            # accumulate on top: counts double
    vt.vt_histogram(ids, V, counts=acc, accumulate=True, ws=ws)
    assert np.array_equal(_u32(acc), 2 * ref)


@pytest.mark.parametrize("V,K", [(1, 1), (6, 3), (4096, 1024), (4096, 4096), (128256, 8192), (128256, 32768),
                                 (128256, 128256), (131072, 1), (200_001, 70_000)])
def test_select_topk_matches_oracle(V, K):
    n = min(20 * V, 3_000_000)
    ids = vt_inputs.zipf_ids(n, V, 1.07, seed=V + K, noise_frac=0.05, device=DEV)
    counts = vt.vt_histogram(ids, V)
    m, inv = vt.vt_select_topk(counts, K)
    rm, rinv = oracle.select_topk(_u32(counts), K)
    assert np.array_equal(m.cpu().numpy(), rm)
    assert np.array_equal(inv.cpu().numpy(), rinv)


def test_select_topk_extreme_count_patterns():
    V, K = 70_000, 1234
    pats = {
        "all_equal": torch.full((V,), 5, dtype=torch.int32),
        "all_zero": torch.zeros(V, dtype=torch.int32),
        "two_levels": (torch.arange(V) % 2).to(torch.int32),
        "wide": torch.from_numpy(np.random.default_rng(1).integers(0, 2**32, V, dtype=np.uint64)
                                 .astype(np.uint32).view(np.int32)),
        "descending": torch.arange(V, 0, -1, dtype=torch.int32),
        "high_byte_only": (torch.from_numpy(np.random.default_rng(2).integers(0, 200, V).astype(np.int32)) << 24),
    }
    for name, c in pats.items():
        m, inv = vt.vt_select_topk(c.to(DEV), K)
        rm, rinv = oracle.select_topk(c.numpy().view(np.uint32).astype(np.uint64), K)
        assert np.array_equal(m.cpu().numpy(), rm), name
        assert np.array_equal(inv.cpu().numpy(), rinv), name


def test_config1_build_vocab_and_gather():
    """Tiny end-to-end case: V=4096, K=1024, 100k Zipf(1.1) ids, d=256."""
    V, K, d = 4096, 1024, 256
    ids = vt_inputs.zipf_ids(100_000, V, 1.1, seed=1001, device=DEV)
    m, inv = vt.vt_build_vocab(ids, V, K)
    rm, rinv, _, _ = oracle.build_vocab(ids.cpu().numpy(), V, K)
    assert np.array_equal(m.cpu().numpy(), rm) and np.array_equal(inv.cpu().numpy(), rinv)
    W = vt_inputs.gaussian_bf16((V, d), 0.02, seed=1002, device=DEV)
    Wt = vt.vt_trim_head(W, m)
    ref = oracle.trim_head(vt_inputs.bf16_bits(W).cpu().numpy(), rm)
    assert np.array_equal(vt_inputs.bf16_bits(Wt).cpu().numpy().view(np.uint16), ref)


def test_build_vocab_from_host_memory_matches_device_path():
    V, K = 128256, 8192
    ids = vt_inputs.zipf_ids(40_000_000, V, 1.07, seed=55, noise_frac=0.05, device=DEV)
    m, inv = vt.vt_build_vocab(ids, V, K)
    host = ids.cpu().pin_memory()
    m2, inv2 = vt.vt_build_vocab(host, V, K)
    torch.cuda.synchronize()
    assert torch.equal(m, m2) and torch.equal(inv, inv2)
    rm, rinv, _, _ = oracle.build_vocab(host.numpy(), V, K)
    assert np.array_equal(m.cpu().numpy(), rm) and np.array_equal(inv.cpu().numpy(), rinv)


def test_trim_head_identity_and_bad_map_entries():
    V, d = 1000, 64
    W = vt_inputs.gaussian_bf16((V, d), 0.02, seed=3, device=DEV)
    ident = torch.arange(V, dtype=torch.int32, device=DEV)
    assert torch.equal(vt_inputs.bf16_bits(vt.vt_trim_head(W, ident)), vt_inputs.bf16_bits(W))
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_TRIM_HEAD))
    bad = torch.tensor([5, -1, V, 7], dtype=torch.int32, device=DEV)
    Wt = vt.vt_trim_head(W, bad, ws=ws)
    st, flags, _ = ws.read_status()
    assert st == 2 and flags & vt.VT_FLAG_BAD_MAP
    assert torch.equal(vt_inputs.bf16_bits(Wt[0]), vt_inputs.bf16_bits(W[5]))
    assert torch.equal(vt_inputs.bf16_bits(Wt[3]), vt_inputs.bf16_bits(W[7]))
    assert int(vt_inputs.bf16_bits(Wt[1:3]).abs().sum()) == 0


def test_config5_corpus_scale_build_and_gather():
    """1e9 ids over V=128256 (95% Zipf(1.07) over a seeded permutation, 5% uniform noise), top-K
    for K in {8192, 32768}, then the gather of W_trim[K,4096]: all outputs bit-exact."""
    V, d, n = 128256, 4096, 1_000_000_000
    ids = vt_inputs.zipf_ids(n, V, 1.07, seed=1005, noise_frac=0.05, device=DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_BUILD_VOCAB, n, V, 32768))
    counts = vt.vt_histogram(ids, V, ws=ws)
    host_ids = ids.cpu().numpy()
    ref_counts, bad = oracle.histogram(host_ids, V)
    assert bad == 0 and int(ref_counts.sum()) == n
    assert np.array_equal(_u32(counts), ref_counts)
    W = vt_inputs.gaussian_bf16((V, d), 0.02, seed=1006, device=DEV)
    Wbits = vt_inputs.bf16_bits(W).cpu().numpy().view(np.uint16)
    for K in (8192, 32768):
        m, inv = vt.vt_build_vocab(ids, V, K, ws=ws)
        rm, rinv = oracle.select_topk(ref_counts, K)
        assert np.array_equal(m.cpu().numpy(), rm) and np.array_equal(inv.cpu().numpy(), rinv)
        Wt = vt.vt_trim_head(W, m)
        assert np.array_equal(vt_inputs.bf16_bits(Wt).cpu().numpy().view(np.uint16), oracle.trim_head(Wbits, rm))
    _assert_clean(ws)


def _counts_for_cut(V, n, seed):
    ids = vt_inputs.zipf_ids(n, V, 1.1, seed=seed, noise_frac=0.05)
    ref, _ = oracle.histogram(ids.numpy(), V)
    return ref


@pytest.mark.parametrize("V,n", [(128256, 3_000_000), (50_000, 200_003), (1000, 5000), (33, 10)])
@pytest.mark.parametrize("p", [1e-9, 0.25, 0.5, 0.9, 0.99, 0.999999, 1.0])
def test_select_topp_matches_oracle(V, n, p):
    ref = _counts_for_cut(V, n, seed=V % 101 + 3)
    counts = torch.from_numpy(ref.astype(np.uint32).view(np.int32)).to(DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_SELECT_TOPK, 0, V, V))
    k_out, map_, inv = vt.vt_select_topp(counts, p, ws=ws)
    K, rmap, rinv = oracle.select_topp(ref, p)
    assert int(k_out.item()) == K
    assert np.array_equal(map_.cpu().numpy()[:K], rmap[:K])       # the trimmed vocabulary; the rest of map is not defined
    assert np.array_equal(inv.cpu().numpy(), rinv)
    _assert_clean(ws)


@pytest.mark.parametrize("V,n", [(128256, 3_000_000), (4096, 100_000), (33, 10)])
@pytest.mark.parametrize("f", [0, 1, 2, 5, 100, 10_000, 2**31])
def test_select_minfreq_matches_oracle(V, n, f):
    ref = _counts_for_cut(V, n, seed=V % 89 + 5)
    counts = torch.from_numpy(ref.astype(np.uint32).view(np.int32)).to(DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_SELECT_TOPK, 0, V, V))
    k_out, map_, inv = vt.vt_select_minfreq(counts, f, ws=ws)
    K, rmap, rinv = oracle.select_minfreq(ref, f)
    assert int(k_out.item()) == K
    assert np.array_equal(map_.cpu().numpy()[:K], rmap[:K])
    assert np.array_equal(inv.cpu().numpy(), rinv)
    _assert_clean(ws)


@pytest.mark.parametrize("shape", ["tiny_values", "few_wide_buckets", "spikes_over_noise", "around_256", "one_value",
                                   "huge_counts_few_per_bucket", "huge_counts_full_buckets", "around_1024"])
def test_select_cuts_over_count_shapes_that_stress_the_buckets(shape):
    """Count vectors chosen against the bucket scheme of the selection kernel: huge buckets of equal counts, all
    counts in a handful of wide buckets, a few enormous counts over noise, counts on both sides of the value from
    which a bucket holds more than one count, a single value, and counts from 2^30.  Top-P, minimum frequency
    and Top-K."""
    V = 50_000
    rng = np.random.default_rng(len(shape))
    c = {"tiny_values": rng.integers(0, 4, V), "few_wide_buckets": rng.integers(1 << 20, 1 << 21, V),
         "spikes_over_noise": np.where(rng.random(V) < 0.01, rng.integers(1 << 28, 1 << 31, V), rng.integers(0, 3, V)),
         "around_256": rng.integers(250, 262, V), "one_value": np.full(V, 12345),
         # counts so large that what orders a bucket's keys (the count's low bits, then the id) passes 32 bits:
         # a dozen ids per such bucket, and hundreds
         "huge_counts_few_per_bucket": np.where(rng.random(V) < 0.02, (1 << 30) + rng.integers(0, 1 << 30, V), rng.integers(0, 3, V)),
         "huge_counts_full_buckets": (1 << 30) + rng.integers(0, 1 << 24, V),
         "around_1024": rng.integers(1000, 1050, V)}[shape].astype(np.uint64)
    counts = torch.from_numpy(c.astype(np.uint32).view(np.int32)).to(DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_SELECT_TOPK, 0, V, V))
    for p in (1e-12, 0.3, 0.9, 1.0):
        k_out, map_, inv = vt.vt_select_topp(counts, p, ws=ws)
        K, rmap, rinv = oracle.select_topp(c, p)
        assert int(k_out.item()) == K
        assert np.array_equal(map_.cpu().numpy()[:K], rmap[:K]) and np.array_equal(inv.cpu().numpy(), rinv)
    for f in (0, 1, 255, 256, 257, 1023, 1024, 1025, int(np.median(c)), int(c.max()), int(c.max()) + 1):
        k_out, map_, inv = vt.vt_select_minfreq(counts, f, ws=ws)
        K, rmap, rinv = oracle.select_minfreq(c, f)
        assert int(k_out.item()) == K
        assert np.array_equal(map_.cpu().numpy()[:K], rmap[:K]) and np.array_equal(inv.cpu().numpy(), rinv)
    for K in (1, V // 3, V // 2 + 1, V):
        map_, inv = vt.vt_select_topk(counts, K, ws=ws)
        rmap, rinv = oracle.select_topk(c, K)
        assert np.array_equal(map_.cpu().numpy(), rmap) and np.array_equal(inv.cpu().numpy(), rinv)
    _assert_clean(ws)


@pytest.mark.parametrize("V", [8 * 65535, 8 * 65535 + 1, 600_001])
def test_select_vocabulary_whose_slices_pass_the_sixteen_bit_counters(V):
    """A CTA ranks rare ids where it places them only while its slice of the vocabulary has at most 65535 ids
    (the first V is the last to which that applies); beyond that every count goes through the key buffer.
    Small counts in large numbers, Top-K, Top-P and minimum frequency."""
    rng = np.random.default_rng(11)
    c = np.where(rng.random(V) < 0.9, rng.integers(0, 6, V), (rng.pareto(1.1, V) * 800).astype(np.int64)).astype(np.uint64)
    counts = torch.from_numpy(c.astype(np.uint32).view(np.int32)).to(DEV)
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_SELECT_TOPK, 0, V, V))
    for K in (1, 5000, 70_000, V):
        map_, inv = vt.vt_select_topk(counts, K, ws=ws)
        rmap, rinv = oracle.select_topk(c, K)
        assert np.array_equal(map_.cpu().numpy(), rmap) and np.array_equal(inv.cpu().numpy(), rinv)
    for p in (0.5, 0.97):
        k_out, map_, inv = vt.vt_select_topp(counts, p, ws=ws)
        K, rmap, rinv = oracle.select_topp(c, p)
        assert int(k_out.item()) == K
        assert np.array_equal(map_.cpu().numpy()[:K], rmap[:K]) and np.array_equal(inv.cpu().numpy(), rinv)
    for f in (3, 1024):
        k_out, map_, inv = vt.vt_select_minfreq(counts, f, ws=ws)
        K, rmap, rinv = oracle.select_minfreq(c, f)
        assert int(k_out.item()) == K
        assert np.array_equal(map_.cpu().numpy()[:K], rmap[:K]) and np.array_equal(inv.cpu().numpy(), rinv)
    _assert_clean(ws)


def test_select_cut_degenerate_counts_and_bad_arguments():
    V = 4096
    ws = vt.Workspace(vt.workspace_bytes(vt.VT_OP_SELECT_TOPK, 0, V, V))
    zero = torch.zeros(V, dtype=torch.int32, device=DEV)
    for call, arg in ((vt.vt_select_topp, 0.5), (vt.vt_select_minfreq, 1)):
        k_out, map_, inv = call(zero, arg, ws=ws)
        K, rmap, rinv = (oracle.select_topp if call is vt.vt_select_topp else oracle.select_minfreq)(
            np.zeros(V, dtype=np.uint64), arg)
        assert int(k_out.item()) == K
        assert np.array_equal(map_.cpu().numpy()[:K], rmap[:K]) and np.array_equal(inv.cpu().numpy(), rinv)
    big = np.full(V, 2**32 - 1, dtype=np.uint64)            # prefix sums need 64 bits
    counts = torch.from_numpy(big.astype(np.uint32).view(np.int32)).to(DEV)
    k_out, map_, inv = vt.vt_select_topp(counts, 0.75, ws=ws)
    K, rmap, rinv = oracle.select_topp(big, 0.75)
    assert int(k_out.item()) == K == 3072
    assert np.array_equal(map_.cpu().numpy()[:K], rmap[:K])
    assert np.array_equal(inv.cpu().numpy(), rinv)
    for p in (0.0, -0.1, 1.5, float("nan")):
        with pytest.raises(vt.VocabTrimError):
            vt.vt_select_topp(zero, p, ws=ws)
