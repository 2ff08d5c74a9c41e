"""The diagnostic build of the library (same sources with -DDA_TIMELINE -DDA_DIAG -DDA_BOUNDS_CHECK).

Two things are checked with it, both without faulting or hanging the device:

* The give-up paths of the kernels.  Every wait inside the kernels is bounded; the diagnostic build lets a
  test shorten the bound to a few milliseconds and make the loader of thread block 0 leave one tile out
  altogether (no copies issued, no barrier arrival), so that the warps waiting for that tile run out of time
  by themselves.  The call must come back with DA_DEV_TIMEOUT in the status record, and the next, normal
  call must be clean and match the oracle.
* The kernels' own indexing.  With -DDA_BOUNDS_CHECK every index into the plan arrays, merge lists, partial
  slots, block table and result tensors is compared with its extent and a violation lands in the status
  record; the small-shape, split-schedule and random suites are run again on this build (their own
  assertions require a clean status record after every call).

Each part runs in a child process, because a process loads one build of the library."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

PRELUDE = r"""
import sys, time
sys.path.insert(0, %r)
import numpy as np, torch
from paper_2512_10977_b200 import binding as da, build
da.use_library(build.build_diag())
import oracle, workloads

def close(got, ref):
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    both = np.isneginf(got) & np.isneginf(ref)
    err = np.where(both, 0.0, np.abs(got - np.where(both, 0.0, ref)))
    return bool((err <= 1e-3 + 1e-3 * np.abs(np.where(both, 0.0, ref))).all())
"""

PARTITION_CHILD = PRELUDE + r"""
case = workloads.build_case("to", [2500, 3, 900, 64, 4097, 130], 16, 11, "cpu")
ref, ref_lse = oracle.decode_attn_oracle(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, 0, case.scale)
dev = workloads.to_device(case, "cuda")
da.set_option("grid_blocks", 4)          # block 0 then holds a few hundred tiles

def call():
    out, lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 0, dev.scale)
    torch.cuda.synchronize()
    return out.cpu().numpy(), lse.cpu().numpy()

out, lse = call()
assert da.read_device_status() == (0, 0, 0, 0) and close(out, ref) and close(lse, ref_lse)
da.set_option("diag_wait_limit_us", 3000)
for tile in (0, 1, 7, 200):              # the very first wait, inside the ring's first lap, later laps
    da.set_option("diag_withhold_partition_tile", tile)
    t0 = time.perf_counter()
    call()                               # must return: every wait gives up after 3 ms
    dt = time.perf_counter() - t0
    st = da.read_device_status()
    assert st[0] == 3, (tile, st)        # DA_DEV_TIMEOUT
    assert st[2] == 0, (tile, st)        # reported by thread block 0
    assert dt < 5.0, dt
    da.set_option("diag_withhold_partition_tile", -1)
    out, lse = call()                    # the device, the workspace and the library are still usable
    assert da.read_device_status() == (0, 0, 0, 0), tile
    assert close(out, ref) and close(lse, ref_lse), tile
print("partition timeout ok")
"""

PREFIX_CHILD = PRELUDE + r"""
lens = 1024 + np.array([0, 5, 300, 77])
case = workloads.build_case("toc", lens, 16, 21, "cpu", shared_prefix_tokens=1024)
ref, ref_lse = oracle.decode_attn_oracle(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, 0, case.scale)
dev = workloads.to_device(case, "cuda")

def cascade():
    out, lse = da.decode_attn_cascade(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 1024, dev.scale)
    torch.cuda.synchronize()
    return out.cpu().numpy(), lse.cpu().numpy()

# the same kernel in extend mode: 200 new tokens of one sequence (1200 query rows per KV head)
ecase = workloads.build_case("toe", [1500], 16, 22, "cpu")
q = torch.randn((1, 200, 48, 128), generator=torch.Generator().manual_seed(3)).to(torch.bfloat16)
eref, eref_lse = oracle.extend_attn_oracle(q, ecase.k_pages, ecase.v_pages, ecase.block_table, ecase.seq_lens, ecase.scale)
edev = workloads.to_device(ecase, "cuda")
qd = q.cuda()

def extend():
    out, lse = da.decode_attn_extend(qd, edev.k_pages, edev.v_pages, edev.block_table, edev.seq_lens, edev.scale)
    torch.cuda.synchronize()
    return out.cpu().numpy(), lse.cpu().numpy()

for name, fn, want, want_lse, tiles in (("cascade", cascade, ref, ref_lse, (0, 1)), ("extend", extend, eref, eref_lse, (0, 2, 5))):
    out, lse = fn()
    assert da.read_device_status() == (0, 0, 0, 0) and close(out, want) and close(lse, want_lse), name
    da.set_option("diag_wait_limit_us", 3000)
    for tile in tiles:
        da.set_option("diag_withhold_prefix_tile", tile)
        t0 = time.perf_counter()
        fn()
        dt = time.perf_counter() - t0
        st = da.read_device_status()
        assert st[0] == 3 and st[2] == 0, (name, tile, st)
        assert dt < 5.0, dt
        da.set_option("diag_withhold_prefix_tile", -1)
        out, lse = fn()                  # tensor memory was freed on the way out: the next launch gets it
        assert da.read_device_status() == (0, 0, 0, 0), (name, tile)
        assert close(out, want) and close(lse, want_lse), (name, tile)
    da.set_option("diag_wait_limit_us", 2000000)
print("prefix timeout ok")
"""


def _run_child(code):
    r = subprocess.run([sys.executable, "-c", code % ROOT], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    return r.stdout


@pytest.mark.gpu
def test_a_wait_that_runs_out_in_the_partition_kernel_sets_timeout_and_the_next_call_is_clean():
    assert "partition timeout ok" in _run_child(PARTITION_CHILD)


@pytest.mark.gpu
def test_a_wait_that_runs_out_in_the_prefix_kernel_sets_timeout_frees_tensor_memory_and_the_next_call_is_clean():
    assert "prefix timeout ok" in _run_child(PREFIX_CHILD)


@pytest.mark.gpu
def test_bounds_checked_build_runs_the_small_shape_and_random_suites_with_a_clean_status_record():
    from paper_2512_10977_b200 import build
    env = dict(os.environ, DECODE_ATTN_LIBRARY=build.build_diag())
    picks = ["tests/test_gpu_parity.py", "tests/test_gpu_random.py", "tests/test_gpu_extend.py", "tests/test_gpu_cascade.py",
             "-k", "edges or sliding or group or split_schedule or ticketed or empty or many_sequences or random or "
                   "few_new_tokens or cascade_matches or cascade_group"]
    r = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider"] + picks,
                       capture_output=True, text=True, timeout=3000, cwd=ROOT, env=env)
    assert r.returncode == 0, r.stdout[-4000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
