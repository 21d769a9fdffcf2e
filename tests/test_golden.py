"""Shape facts the paper prints, against the constants the synthetic workloads use.

The paper prints no numeric example of the head computation itself, so these fixtures pin what it
does print about this path: the sizes of the full and trimmed LM heads (Tables 1-3, 5)."""
import os

import vt_inputs

HERE = os.path.dirname(os.path.abspath(__file__))


def _rows():
    for line in open(os.path.join(HERE, "golden", "paper_head_sizes.txt")):
        if line.strip() and not line.startswith("#"):
            d, full, trim = line.split()[:3]
            yield int(d), float(full), float(trim)


def test_full_head_sizes_match_the_llama3_vocabulary():
    for d, full, _ in _rows():
        assert abs(vt_inputs.LLAMA3_VOCAB * d / 1e6 - full) <= 0.05        # printed to one decimal


def test_trimmed_head_sizes_are_one_k_for_all_drafters_and_close_to_the_benchmarked_k():
    ks = [trim * 1e6 / d for d, _, trim in _rows()]
    assert max(ks) - min(ks) < 60                                           # the same K (about 33.0K) in every table
    assert abs(sum(ks) / len(ks) - 32768) / 32768 < 0.01                    # the configs round it to 2^15


def test_bench_workloads_use_the_papers_shapes():
    import bench

    assert bench.V == 128256 and bench.HEAD["d"] == 3072 and bench.HEAD["K"] == 32768
    assert bench.TREE["d"] == 4096 and bench.DENSE["d"] == 4096
