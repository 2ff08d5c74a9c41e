"""The timeline build of the library (same sources, -DDA_TIMELINE): same results as the normal build, and
stamps that are ordered the way the three kernels run.  Runs in a child process, because a process loads
one build of the library."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r)
import numpy as np, torch
from paper_2512_10977_b200 import binding, build
binding.use_library(build.build_diag())
import oracle, workloads
case = workloads.build_case("tl", [2500, 3, 900, 0, 64, 4097, 130, 9000], 16, 5, "cpu")
ref, ref_lse = oracle.decode_attn_oracle(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, 0, case.scale)
dev = workloads.to_device(case, "cuda")
binding.timeline(clear=True)
out, lse = binding.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 0, dev.scale)
tl = binding.timeline()
assert np.allclose(out.cpu().numpy(), ref, atol=1e-3, rtol=1e-3)
got_lse = lse.cpu().numpy()
fin = np.isfinite(ref_lse)
assert np.allclose(got_lse[fin], ref_lse[fin], atol=1e-3, rtol=1e-3) and np.isneginf(got_lse[~fin]).all()
part = tl[:1024]; part = part[part[:, 4] > 0]
assert len(part) > 0
tiles = sum(8 * ((int(L) + 63) // 64) for L in case.seq_lens)
assert int(part[:, 5].sum()) == tiles, (int(part[:, 5].sum()), tiles)
plan0, plan1 = tl[1036:1044, 0], tl[1036:1044, 1]
assert (plan0 > 0).all() and (plan1 >= plan0).all()
assert (part[:, 1] >= plan1.max()).all()          # no block passes its wait before the plan is complete
assert (part[:, 0] <= part[:, 1]).all() and (part[:, 1] <= part[:, 2]).all()
assert (part[:, 2] <= part[:, 3]).all() and (part[:, 3] <= part[:, 4]).all()
m = tl[1024:1032]
assert (m[:, 1] >= part[:, 4].max()).all()        # the merge kernel is released after the last block left
assert tl[1032, 2] >= m[:, 2].max() >= m[:, 1].max()
print("timeline ok", len(part), "blocks", tiles, "tiles")
"""


@pytest.mark.gpu
def test_timeline_build_matches_the_oracle_and_orders_its_stamps():
    r = subprocess.run([sys.executable, "-c", CHILD % ROOT], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "timeline ok" in r.stdout
