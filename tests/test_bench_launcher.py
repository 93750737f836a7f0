"""bench.py on CPU: `--gpus N` without a launcher starts N ranks itself, and the strong-scaling split covers the
batch.  (The GPU arm needs a GPU; the oracle arm runs the same launcher path on the host.)"""
import json
import os
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2504_00030_b200 import synth  # noqa: E402


def test_gpus_2_without_a_launcher_starts_two_ranks():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    env["OMP_NUM_THREADS"] = "2"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--workload", "c1", "--oracle-seqs", "1"],
                         env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                  # rank 0 alone prints
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2 and lines[0]["value"] > 0


def test_strong_shares_cover_the_batch_and_balance_the_cached_tokens():
    base = synth.CONFIGS["c5"]
    cfg, seq_len, gamma, cu_q, cu_d = bench.workload_inputs(base, 0)
    for world in (2, 4, 8):
        counts, tokens, lens = [], [], []
        for rank in range(world):
            local, sl, g, cq, cd, global_batch = bench.strong_share(base, rank, world)
            assert global_batch == cfg.batch and local.batch == len(sl) == len(g)
            assert cq[0] == 0 and cq[-1] == local.batch * (local.gamma_max + 1)      # rebased, still padded slabs
            counts.append(local.batch)
            tokens.append(int(sl.sum()))
            lens.append(sl)
        assert sum(counts) == cfg.batch
        np.testing.assert_array_equal(np.concatenate(lens), seq_len)      # contiguous runs, in order
        assert max(tokens) - min(tokens) <= 2 * int(seq_len.max())         # equal up to a sequence at each cut
