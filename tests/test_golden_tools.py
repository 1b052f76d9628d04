"""CPU-only: the golden-score writer's bookkeeping (candidate selection, part files, joining) and the stored files'
shape.  The scores themselves come from the oracle; nothing here touches the CUDA path."""
import os
import subprocess
import sys

import numpy as np

import synth

GOLD = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
sys.path.insert(0, GOLD)
import make_scores  # noqa: E402


def test_stratified_ids_span_the_length_range():
    lens = np.array([50, 10, 30, 20, 40, 60, 70, 15])
    ids = make_scores.stratified_ids(lens, 3)
    assert ids == sorted(ids) and len(ids) == 3
    assert 1 in ids and 6 in ids                      # the shortest and the longest candidate
    assert make_scores.stratified_ids(lens, 8) == list(range(8))


def test_part_files_join_into_the_file_of_the_whole(tmp_path):
    """Two part files of the tiny workload, joined, equal the file written in one go (same oracle, same columns)."""
    run = lambda *a: subprocess.run([sys.executable, os.path.join(GOLD, "make_scores.py"), "0", "0", *a], check=True,
                                    capture_output=True)
    whole, p0, p1, joined = (str(tmp_path / n) for n in ("whole.txt", "p0.txt", "p1.txt", "joined.txt"))
    run("--out", whole)
    run("--part", "0/2", "--out", p0)
    run("--part", "1/2", "--out", p1)
    run("--merge", p1, p0, "--out", joined)
    Sw, iw, _ = make_scores.read_scores(whole)
    Sj, ij, _ = make_scores.read_scores(joined)
    assert iw == ij == list(range(synth.workload(0).n_candidates))
    for l in Sw:
        assert np.array_equal(Sw[l], Sj[l])


def test_stored_score_files_cover_what_the_parity_tests_expect():
    """Every full-size file names its candidates and holds one score per candidate and scored layer."""
    expect = {"cfg1_qwen3_0p6b_scores_r0.txt": (1, 100), "cfg1_qwen3_0p6b_scores_r1.txt": (1, 100),
              "cfg1_qwen3_0p6b_scores_r2.txt": (1, 100), "cfg2_qwen3_4b_scores_r0.txt": (2, 200),
              "cfg2_qwen3_4b_scores_r1.txt": (2, 200), "cfg3_qwen3_8b_streamed_scores_r0.txt": (3, 100),
              "cfg3_qwen3_8b_streamed_scores_r1.txt": (3, 100),
              "cfg4_stress_0p6b_scores_r0.txt": (4, 1000), "cfg4_stress_0p6b_scores_r1.txt": (4, 1000)}
    for name, (index, n) in expect.items():
        S, ids, head = make_scores.read_scores(os.path.join(GOLD, name))
        wl = synth.workload(index)
        if ids is None:                                # the oldest file carries no id line: all candidates in order
            ids = list(range(n))
        assert ids == list(range(n)), name
        assert sorted(S) == sorted(set(list(wl.schedule.probe_layers) + [wl.model.n_layers])), name
        assert all(len(v) == n and np.all(np.isfinite(v)) for v in S.values()), name
