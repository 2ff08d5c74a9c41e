"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU oracle on the same
seeded inputs.  Tolerances: fp32 out and lse |d| <= 1e-3 + 1e-3*|ref|; bf16 out |d| <= 8e-3 (one
bf16 ulp of the correctly rounded oracle value where |ref| >= 4); indexing checks are bit-exact."""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu


def same(host, dev):
    """A host-buffer call against the device-resident call on the same inputs: the same sums, but possibly
    folded in another order (two-piece pairs are folded by the partition kernel in the host-buffer calls)."""
    a, b = host.float(), dev.float().cpu()
    both_ninf = torch.isneginf(a) & torch.isneginf(b)
    return bool(torch.allclose(torch.where(both_ninf, torch.zeros_like(a), a), torch.where(both_ninf, torch.zeros_like(b), b),
                               atol=2e-5 if host.dtype == torch.float32 else 8e-3, rtol=1e-4))

ATOL, RTOL = 1e-3, 1e-3


@pytest.fixture(scope="module")
def da():
    import paper_2512_10977_b200 as pkg
    pkg.lib()
    yield pkg
    pkg.set_option("grid_blocks", 0)
    pkg.set_option("tail_units", 4)
    pkg.set_option("static_frac", 224)


def oracle_of(case):
    return oracle.decode_attn_oracle(case.q, case.k_pages, case.v_pages, case.block_table,
                                     case.seq_lens, case.window, case.scale)


def gpu_of(da, case, out_dtype=torch.float32):
    dev = workloads.to_device(case, "cuda")
    out, lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens,
                              dev.window, dev.scale, out_dtype=out_dtype)
    st = da.read_device_status()
    assert st == (0, 0, 0, 0), f"device status {st}"
    return out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)


def assert_close(got, ref, what, atol=ATOL, rtol=RTOL):
    got, ref = np.asarray(got), np.asarray(ref)
    both_ninf = np.isneginf(got) & np.isneginf(ref)
    with np.errstate(invalid="ignore"):
        err = np.where(both_ninf, 0.0, np.abs(got - ref))
    lim = atol + rtol * np.abs(np.where(both_ninf, 0.0, ref))
    bad = ~(err <= lim)
    if bad.any():
        i = np.unravel_index(np.argmax(np.where(bad, err, -1)), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outside tolerance; worst at {i}: "
                             f"got {got[i]!r} want {ref[i]!r}")


def assert_bf16_close(got, ref, what):
    """|d| <= 8e-3, or within one bf16 ulp of the correctly rounded reference where |ref| >= 4."""
    rounded = torch.from_numpy(ref).float().to(torch.bfloat16).double().numpy()
    err = np.abs(got - ref)
    ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(ref), 1e-30))) - 7)
    ok = (err <= 8e-3) | ((np.abs(ref) >= 4) & (np.abs(got - rounded) <= ulp))
    assert ok.all(), f"{what}: {np.count_nonzero(~ok)} elements outside the bf16 bar, worst {err.max()}"


def check(da, case, what, grid=0, out_dtype=torch.float32):
    da.set_option("grid_blocks", grid)
    ref, ref_lse = oracle_of(case)
    got, got_lse = gpu_of(da, case, out_dtype)
    if out_dtype == torch.float32:
        assert_close(got, ref, what + " out")
    else:
        assert_bf16_close(got, ref, what + " out(bf16)")
    assert_close(got_lse, ref_lse, what + " lse")
    return got, got_lse


# ------------------------------------------------------------------ small shapes, every path

LENS = [1, 2, 15, 16, 17, 31, 33, 63, 64, 65, 127, 129, 255, 257, 1000]


@pytest.mark.parametrize("P", [16, 32, 64, 128])
def test_lengths_around_tile_and_page_edges(da, P):
    case = workloads.build_case("edges", LENS, P, 100 + P, "cpu", pool_pages=None, pad_table_to=40)
    for grid in (0, 1, 5):
        check(da, case, f"P={P} grid={grid}", grid)


@pytest.mark.parametrize("window", [1, 5, 16, 17, 63, 64, 65, 200, 256, 257, 100000])
def test_sliding_window(da, window):
    lens = [1, 17, 64, 65, 200, 257, 258, 700]
    case = workloads.build_case("win", lens, 16, 7, "cpu", window=window)
    check(da, case, f"W={window}")
    check(da, case, f"W={window} one block", 1)


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (32, 8), (48, 8), (64, 8), (24, 2), (16, 1), (40, 4)])
def test_group_sizes(da, Hq, Hkv):
    case = workloads.build_case("gqa", [300, 77, 1, 129], 16, Hq, "cpu", Hq=Hq, Hkv=Hkv)
    check(da, case, f"Hq={Hq} Hkv={Hkv}")
    check(da, case, f"Hq={Hq} Hkv={Hkv} grid 3", 3)


@pytest.mark.parametrize("grid", [1, 2, 3, 7, 64, 148, 296, 1000, 4096])
def test_any_split_schedule_gives_the_same_answer(da, grid):
    case = workloads.build_case("splits", [2500, 3, 900, 64, 4097, 130], 16, 11, "cpu")
    got, got_lse = check(da, case, f"grid={grid}", grid)
    da.set_option("grid_blocks", 1)
    base, base_lse = gpu_of(da, case)
    np.testing.assert_allclose(got, base, atol=2e-5, rtol=1e-5)
    np.testing.assert_allclose(got_lse, base_lse, atol=2e-5, rtol=1e-5)


@pytest.mark.parametrize("tail,frac", [(0, 192), (1, 128), (6, 0), (6, 256), (20, 64), (64, 200)])
def test_any_mix_of_static_and_ticketed_units_gives_the_same_answer(da, tail, frac):
    case = workloads.build_case("units", [2500, 3, 900, 0, 64, 4097, 130, 9000], 16, 13, "cpu", window=0)
    try:
        da.set_option("tail_units", tail)
        da.set_option("static_frac", frac)
        for grid in (0, 5, 64):
            check(da, case, f"tail={tail} frac={frac} grid={grid}", grid)
        case.window = 700
        check(da, case, f"tail={tail} frac={frac} window", 0)
    finally:
        da.set_option("tail_units", 4)
        da.set_option("static_frac", 224)


@pytest.mark.parametrize("policy", [0, 1, 2])
def test_l2_priority_of_the_page_loads_does_not_change_the_answer(da, policy):
    """The K/V loads' L2 policy (normal, evict first, chosen on the device from how many sequences
    start on the same page) is a cache hint only: same result with and without a shared prefix."""
    unique = workloads.build_case("pol_u", [2500, 3, 900, 0, 64, 4097], 16, 31, "cpu")
    shared = workloads.build_case("pol_s", [2500, 640, 900, 1300, 4097], 16, 32, "cpu", shared_prefix_tokens=640)
    try:
        da.set_option("kv_evict_first", policy)
        assert da.get_option("kv_evict_first") == policy
        for case, what in ((unique, "unique pages"), (shared, "shared prefix")):
            check(da, case, f"{what}, policy {policy}")
    finally:
        da.set_option("kv_evict_first", 2)
    with pytest.raises(Exception):
        da.set_option("kv_evict_first", 3)


@pytest.mark.parametrize("B", [1, 2, 3, 7])
@pytest.mark.parametrize("P", [16, 64])
def test_batches_with_empty_sequences(da, B, P):
    lens = [0, 130, 0, 0, 5, 2049, 0][:B]
    case = workloads.build_case("empty", lens, P, 3 * B + P, "cpu")
    got, got_lse = check(da, case, f"B={B} P={P}")
    for b, L in enumerate(lens):
        if L == 0:
            assert (got[b] == 0).all() and np.isneginf(got_lse[b]).all()


def test_all_sequences_empty(da):
    case = workloads.build_case("allempty", [0, 0, 0], 16, 5, "cpu")
    got, got_lse = check(da, case, "all empty")
    assert (got == 0).all() and np.isneginf(got_lse).all()


@pytest.mark.parametrize("B", [512, 513, 1025, 1500, 4096, 4097, 6000])
def test_many_sequences(da, B):
    """Batches beyond one pass of the plan kernel's scan (512 sequences) and beyond what its shared
    memory holds (4096: the work units are then cut from the global copy of the prefix)."""
    rng = np.random.default_rng(B)
    lens = rng.integers(0, 150, size=B)
    lens[rng.integers(0, B, size=5)] = 700
    case = workloads.build_case("many", lens, 16, B, "cpu")
    for grid in (0, 3):
        got, got_lse = check(da, case, f"B={B} grid={grid}", grid)
    for b in np.nonzero(lens == 0)[0][:20]:
        assert (got[b] == 0).all() and np.isneginf(got_lse[b]).all()


def test_token_major_layout(da):
    case = workloads.build_case("tm", [513, 40, 1300], 16, 21, "cpu", layout="token_major")
    assert case.k_pages.stride(1) < case.k_pages.stride(2)
    check(da, case, "token-major")


def test_bf16_output(da):
    case = workloads.build_case("bf16", [700, 33, 2100, 1], 16, 23, "cpu")
    check(da, case, "bf16", 0, torch.bfloat16)
    check(da, case, "bf16 grid 2", 2, torch.bfloat16)


def test_stability_config_c1(da):
    """1 x 512 tokens, three keys x20: the weights collapse onto single tokens."""
    case = workloads.c1()
    check(da, case, "c1")
    check(da, case, "c1 one block", 1)
    check(da, case, "c1 bf16", 0, torch.bfloat16)


def test_huge_score_offsets(da):
    case = workloads.build_case("shift", [300, 90], 16, 29, "cpu")
    case.q[..., 127] = 1.0
    for cshift in (3.0e3, -3.0e3):
        case.k_pages[..., 127] = cshift
        got, got_lse = check(da, case, f"shift {cshift}")
        assert np.isfinite(got).all() and np.isfinite(got_lse).all()


def test_noncontiguous_q_and_out(da):
    case = workloads.build_case("strided", [400, 65, 31], 16, 31, "cpu")
    dev = workloads.to_device(case, "cuda")
    B, Hq, Dh = dev.q.shape
    q_big = torch.zeros((B, Hq + 3, 2 * Dh), dtype=torch.bfloat16, device="cuda")
    q_view = q_big[:, 1:Hq + 1, :Dh]
    q_view.copy_(dev.q)
    out_big = torch.full((B, Hq, 3 * Dh), 7.0, device="cuda")
    out_view = out_big[:, :, Dh:2 * Dh]
    lse_big = torch.full((Hq, B), 7.0, device="cuda")
    lse_view = lse_big.t()
    da.decode_attn(q_view, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 0, dev.scale,
                   out=out_view, lse=lse_view)
    ref, ref_lse = oracle_of(case)
    assert_close(out_view.cpu().numpy(), ref, "strided out")
    assert_close(lse_view.cpu().numpy(), ref_lse, "strided lse")
    assert (out_big[:, :, :Dh] == 7).all() and (out_big[:, :, 2 * Dh:] == 7).all()


def test_host_io_matches_device_call(da):
    case = workloads.build_case("hostio", [700, 33, 2100, 1, 0], 16, 37, "cpu")
    dev = workloads.to_device(case, "cuda")
    want, want_lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 9, dev.scale)
    q_h, bt_h, sl_h = (t.pin_memory() for t in (case.q, case.block_table, case.seq_lens))
    out_h = torch.empty(case.q.shape, dtype=torch.float32).pin_memory()
    lse_h = torch.empty(case.q.shape[:2], dtype=torch.float32).pin_memory()
    for _ in range(2):
        out_h.fill_(5)
        da.decode_attn_host_io(q_h, dev.k_pages, dev.v_pages, bt_h, sl_h, 9, dev.scale, out_h, lse_h)
        torch.cuda.synchronize()
        assert same(out_h, want) and same(lse_h, want_lse)


def test_host_io_with_pageable_buffers_takes_the_staged_path(da):
    case = workloads.build_case("hostio2", [700, 33, 2100, 1, 0], 16, 38, "cpu")
    dev = workloads.to_device(case, "cuda")
    want, want_lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 0, dev.scale)
    out_h = torch.full(case.q.shape, 5.0, dtype=torch.float32)            # pageable
    lse_h = torch.full(case.q.shape[:2], 5.0, dtype=torch.float32)
    da.decode_attn_host_io(case.q, dev.k_pages, dev.v_pages, case.block_table, case.seq_lens, 0, dev.scale, out_h, lse_h)
    torch.cuda.synchronize()
    assert same(out_h, want) and same(lse_h, want_lse)
    # pinned out, pageable lse: still staged (both must be mapped for direct writes)
    out_p = torch.full(case.q.shape, 5.0, dtype=torch.float32).pin_memory()
    lse_h.fill_(5)
    da.decode_attn_host_io(case.q, dev.k_pages, dev.v_pages, case.block_table, case.seq_lens, 0, dev.scale, out_p, lse_h)
    torch.cuda.synchronize()
    assert same(out_p, want) and same(lse_h, want_lse)
    # bf16 results written directly into pinned memory
    out_b = torch.zeros(case.q.shape, dtype=torch.bfloat16).pin_memory()
    lse_p = torch.zeros(case.q.shape[:2], dtype=torch.float32).pin_memory()
    da.decode_attn_host_io(case.q.pin_memory(), dev.k_pages, dev.v_pages, case.block_table.pin_memory(),
                           case.seq_lens.pin_memory(), 0, dev.scale, out_b, lse_p)
    torch.cuda.synchronize()
    want_b, _ = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 0, dev.scale,
                               out_dtype=torch.bfloat16)
    assert same(out_b, want_b) and same(lse_p, want_lse)
    assert da.read_device_status() == (0, 0, 0, 0)


# ------------------------------------------------------------------ indexing, bit-exact

def _probe_case(P, lens, window, seed):
    """K = 0 everywhere; V rows carry (token, physical page, kv head) as small integers."""
    case = workloads.build_case("probe", lens, P, seed, "cpu", window=window, poison=True, pool_pages=None)
    case.k_pages[torch.isfinite(case.k_pages)] = 0
    bt = case.block_table.numpy()
    for b, L in enumerate(lens):
        for t in range(L):
            pg = int(bt[b, t // P])
            for g in range(case.k_pages.shape[1]):
                v = torch.zeros(128)
                v[0], v[1], v[2], v[3], v[4], v[5] = t % 128, t // 128, pg % 128, pg // 128, g, b
                case.v_pages[pg, g, t % P] = v.to(torch.bfloat16)
    return case


@pytest.mark.parametrize("P", [16, 64])
def test_probe_token_is_returned_bit_for_bit(da, P):
    lens, W = [300, 77, 1025], 100
    base = _probe_case(P, lens, W, 41)
    dev = workloads.to_device(base, "cuda")
    bt = base.block_table.numpy()
    qn = base.q.float()
    for grid in (0, 1):
        da.set_option("grid_blocks", grid)
        for b, L in enumerate(lens):
            lo = max(L - W, 0)
            # first / last token of the window, of a page, of a 64-token tile
            cand = [lo, lo + 1, L - 1, (lo // P + 1) * P - 1, (lo // P + 1) * P,
                    (lo // 64 + 1) * 64 - 1, (lo // 64 + 1) * 64, (L - 1) // 64 * 64 - 1, (L - 1) // 64 * 64]
            inside = sorted({t for t in cand if lo <= t < L})
            for t_star in inside:
                pg = int(bt[b, t_star // P])
                saved = dev.k_pages[pg, :, t_star % P].clone()
                # k* = 40 q / |q|^2 * sqrt(128) ... simply a large multiple of q of the group's first head
                for g in range(8):
                    dev.k_pages[pg, g, t_star % P] = (qn[b, 6 * g] * 64).to(torch.bfloat16).cuda()
                q_same = dev.q.clone()
                for g in range(8):
                    q_same[b, 6 * g:6 * g + 6] = dev.q[b, 6 * g]
                out, _ = da.decode_attn(q_same, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, W, 1.0)
                want = dev.v_pages[pg, :, t_star % P].float()          # [8, 128]
                got = out[b].view(8, 6, 128)
                assert torch.equal(got, want[:, None, :].expand(8, 6, 128)), (P, grid, b, t_star)
                assert got[0, 0, 0].item() == t_star % 128 and got[0, 0, 1].item() == t_star // 128
                assert got[3, 2, 4].item() == 3 and got[0, 0, 5].item() == b
                dev.k_pages[pg, :, t_star % P] = saved
    assert da.read_device_status() == (0, 0, 0, 0)


@pytest.mark.parametrize("P", [16, 64])
def test_probe_token_outside_the_range_is_ignored(da, P):
    """A dominant key at lo-1 (just before the window) or in the page tail (>= L) must not count."""
    lens, W = [300, 70], 100
    base = _probe_case(P, lens, W, 43)
    ref, ref_lse = oracle_of(base)
    dev = workloads.to_device(base, "cuda")
    bt = base.block_table.numpy()
    for b, L in enumerate(lens):
        lo = max(L - W, 0)
        for t_bad in ([lo - 1] if lo > 0 else []) + ([L] if L % P else []):
            pg = int(bt[b, t_bad // P])
            saved = dev.k_pages[pg, :, t_bad % P].clone()
            dev.k_pages[pg, :, t_bad % P] = 1.0e4
            out, lse = da.decode_attn(dev.q.abs(), dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, W, 1.0)
            assert_close(out[b].cpu().numpy(), ref[b], f"probe outside b={b} t={t_bad}")
            assert_close(lse[b].cpu().numpy(), np.full(48, math.log(L - lo)), "lse of uniform weights")
            dev.k_pages[pg, :, t_bad % P] = saved


def test_integer_mean_is_exact(da):
    """K = 0 and V small integers over a power-of-two number of tokens: the mean is exact in fp32."""
    lens = [256, 1024, 64]
    case = workloads.build_case("int", lens, 16, 47, "cpu")
    case.k_pages[torch.isfinite(case.k_pages)] = 0
    vi = torch.randint(-8, 9, case.v_pages.shape, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    case.v_pages = torch.where(torch.isfinite(case.v_pages), vi, case.v_pages)
    ref, ref_lse = oracle_of(case)
    try:
        # one thread block, one unit: no split, so every sum is a sum of small integers
        da.set_option("grid_blocks", 1)
        da.set_option("tail_units", 0)
        got, got_lse = gpu_of(da, case)
        assert np.array_equal(got, ref)
        np.testing.assert_allclose(got_lse, ref_lse, atol=1e-6)
    finally:
        da.set_option("grid_blocks", 0)
        da.set_option("tail_units", 4)
    got, _ = gpu_of(da, case)
    np.testing.assert_allclose(got, ref, atol=1e-6)


def test_nan_canaries(da):
    """Unreferenced pages, page tails and block-table padding are poisoned; the output is finite and
    equals the run on a clean, exact-size pool."""
    lens = [5, 17, 300, 1029, 64]
    dirty = workloads.build_case("dirty", lens, 16, 53, "cpu", poison=True, pool_pages=400, pad_table_to=90)
    assert torch.isnan(dirty.k_pages).sum() > 1000 and (dirty.block_table == -1).any()
    for grid in (0, 1, 9):
        got, got_lse = check(da, dirty, f"canary grid={grid}", grid)
        assert np.isfinite(got).all() and np.isfinite(got_lse).all()
    check(da, workloads.build_case("dirtyw", lens, 16, 53, "cpu", poison=True, pool_pages=400, window=20), "canary window")


# ------------------------------------------------------------------ plan

@pytest.mark.parametrize("window", [0, 100, 8192])
def test_plan_covers_every_attended_token_exactly_once(da, window):
    lens = np.concatenate([workloads.lengths_c2(1, 20), [0, 1, 64, 65]])
    sl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    try:
        for grid, tail in ((0, 4), (1, 0), (7, 3), (1000, 1), (0, 0)):
            da.set_option("grid_blocks", grid)
            da.set_option("tail_units", tail)
            seq_info, unit_work, n_static, T = da.plan(sl, window, 8, 16, 2048)
            si = seq_info.numpy()
            for b, L in enumerate(lens):
                lo = L - window if 0 < window < L else 0
                assert si[b, 0] == lo and si[b, 1] == L
                if L > 0:
                    assert si[b, 2] == lo // T and si[b, 3] == (L - 1) // T - lo // T + 1
                else:
                    assert si[b, 3] == 0
            covered = np.zeros((len(lens), 8, int(si[:, 3].max()) + 1), dtype=np.int32)
            sizes = []
            for b0, g0, rel0, n in unit_work.numpy():
                sizes.append(int(n))
                b, g, rel = int(b0), int(g0), int(rel0)
                while n > 0:
                    while si[b, 3] == 0:
                        b += 1
                    take = min(si[b, 3] - rel, n)
                    covered[b, g, rel:rel + take] += 1
                    n -= take
                    rel = 0
                    g += 1
                    if g == 8:
                        g, b = 0, b + 1
            for b in range(len(lens)):
                assert (covered[b, :, :si[b, 3]] == 1).all() and (covered[b, :, si[b, 3]:] == 0).all()
            assert n_static == (grid if grid else 2 * torch.cuda.get_device_properties(0).multi_processor_count)
            assert len(sizes) <= n_static * (1 + tail)
            # equal work within the static ranges and within the ticketed units
            assert max(sizes[:n_static]) - min(sizes[:n_static]) <= 1
            if len(sizes) > n_static:
                assert max(sizes[n_static:]) - min(sizes[n_static:]) <= 1 and min(sizes[n_static:]) >= 4
            else:
                assert tail == 0 or sum(sizes) < 4 * 256 // 64 + 64
    finally:
        da.set_option("grid_blocks", 0)
        da.set_option("tail_units", 4)


# ------------------------------------------------------------------ two-piece pairs folded by the partition kernel

@pytest.mark.parametrize("grid", [2, 3, 7, 64, 148, 296, 1000])
def test_pairs_cut_in_two_are_folded_by_the_partition_kernel(da, grid):
    """Option fold_pairs = 1 (the default folds only in the host-buffer calls): a pair that the own ranges of
    two neighbouring thread blocks cut in two is folded by the block that finishes second, not by the merge
    kernel.  Same answer as the oracle, for every split schedule, output type and twice in a row (the
    counters are left at zero)."""
    case = workloads.build_case("fold", [2500, 3, 900, 0, 64, 4097, 130, 9000, 700], 16, 17, "cpu")
    try:
        da.set_option("fold_pairs", 1)
        da.set_option("tail_units", 1)
        for _ in range(2):
            check(da, case, f"fold grid={grid}", grid)
        check(da, case, f"fold grid={grid} bf16", grid, torch.bfloat16)
        da.set_option("tail_units", 0)
        check(da, case, f"fold grid={grid}, no ticketed units", grid)
    finally:
        da.set_option("fold_pairs", 2)
        da.set_option("tail_units", 4)
        da.set_option("grid_blocks", 0)


def test_c2_full_size_with_folded_pairs(da):
    try:
        da.set_option("fold_pairs", 1)
        da.set_option("grid_blocks", 0)
        case = workloads.c2("cuda")
        _full_size(da, case, list(range(0, case.B, 4)), "c2 folded pairs")
    finally:
        da.set_option("fold_pairs", 2)


# ------------------------------------------------------------------ small calls: one kernel instead of three

@pytest.mark.parametrize("lens,P,window", [([512], 16, 0), ([1, 2, 63, 64, 65, 300], 16, 0), ([700, 0, 33, 129], 64, 0),
                                           ([900, 250, 3], 16, 100), ([2048] * 4, 128, 0), ([0, 0], 16, 0)])
def test_direct_and_planned_paths_agree_with_the_oracle(da, lens, P, window):
    """A call whose pairs fit one wave of thread blocks runs as one kernel (every block finds its piece from
    seq_lens, the last block of a pair folds the pieces); option direct_path = 0 sends the same call through
    plan + partition + merge.  Both must match the oracle, twice in a row (the pair counters are left at zero)."""
    case = workloads.build_case("direct", lens, P, 300 + P + len(lens), "cpu", window=window)
    ref, ref_lse = oracle_of(case)
    dev = workloads.to_device(case, "cuda")
    da.set_option("grid_blocks", 0)
    try:
        for direct, launches in ((1, 1), (1, 1), (0, 3)):
            da.set_option("direct_path", direct)
            for dtype in (torch.float32, torch.bfloat16):
                n0 = da.launch_count()
                out, lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, dev.window,
                                          dev.scale, out_dtype=dtype)
                assert da.launch_count() - n0 == launches
                assert da.read_device_status() == (0, 0, 0, 0)
                got = out.float().cpu().numpy().astype(np.float64)
                if dtype == torch.float32:
                    assert_close(got, ref, f"direct={direct} out")
                else:
                    assert_bf16_close(got, ref, f"direct={direct} out(bf16)")
                assert_close(lse.cpu().numpy(), ref_lse, f"direct={direct} lse")
    finally:
        da.set_option("direct_path", 1)


# ------------------------------------------------------------------ errors, on the host and on the device

def test_host_side_argument_errors(da):
    case = workloads.to_device(workloads.build_case("err", [100], 16, 59, "cpu"), "cuda")
    def args(**kw):
        d = dict(q=case.q, k=case.k_pages, v=case.v_pages, bt=case.block_table, sl=case.seq_lens)
        d.update(kw)
        return d

    def call(q, k, v, bt, sl, out=None):
        return da.decode_attn(q, k, v, bt, sl, 0, 1.0, out=out)

    with pytest.raises(da.DecodeAttnError) as e:
        call(**args(q=case.q[:, :47]))                       # Hq not a multiple of Hkv
    assert e.value.status == 2
    with pytest.raises(da.DecodeAttnError) as e:
        call(**args(k=case.k_pages[..., :64].contiguous(), v=case.v_pages[..., :64].contiguous(), q=case.q[..., :64].contiguous()))
    assert e.value.status == 5                               # head_dim 64
    with pytest.raises(da.DecodeAttnError) as e:
        call(**args(k=case.k_pages[:, :, :8], v=case.v_pages[:, :, :8]))
    assert e.value.status == 5                               # page size 8
    with pytest.raises(da.DecodeAttnError) as e:
        call(**args(k=case.k_pages.view(-1)[4:4 + 8 * 16 * 128].view(1, 8, 16, 128)))
    assert e.value.status in (2, 4)                          # misaligned base / mismatched pools
    with pytest.raises(da.DecodeAttnError) as e:
        call(**args(sl=case.seq_lens.repeat(2)))
    assert e.value.status == 2
    with pytest.raises(da.DecodeAttnError) as e:
        call(**args(out=torch.empty((1, 48, 128), dtype=torch.float32, device="cuda")[..., ::2]))
    assert e.value.status in (2, 4)
    with pytest.raises(TypeError):
        call(**args(bt=case.block_table.long()))
    # pools without KV heads or without pages: refused with a status (never a division fault on the host),
    # by the single-token call and by the multi-token one (torch hands an empty tensor over as a NULL pointer)
    q4 = case.q[:, None].contiguous()
    for k, v in ((case.k_pages[:, :0], case.v_pages[:, :0]), (case.k_pages[:0], case.v_pages[:0])):
        with pytest.raises(da.DecodeAttnError) as e:
            call(**args(k=k, v=v))
        assert e.value.status in (1, 2)
        with pytest.raises(da.DecodeAttnError) as e:
            da.decode_attn_extend(q4, k, v, case.block_table, case.seq_lens, 1.0)
        assert e.value.status in (1, 2)
    assert da.read_device_status() == (0, 0, 0, 0)


def test_device_side_errors_set_the_status_word_without_faulting(da):
    good = workloads.build_case("bad", [100, 200, 40], 16, 61, "cpu")
    ref, ref_lse = oracle_of(good)
    dev = workloads.to_device(good, "cuda")
    # a corrupted block-table entry (corrupted on the host copy, then uploaded)
    bt = good.block_table.clone()
    bt[1, 3] = 10 ** 6
    out, lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, bt.cuda(), dev.seq_lens, 0, dev.scale)
    st = da.read_device_status()
    assert st[0] == 1 and st[1] == 1 and st[2] == 3 and st[3] == 10 ** 6
    assert_close(out[0].cpu().numpy(), ref[0], "other sequences are unaffected")
    assert_close(out[2].cpu().numpy(), ref[2], "other sequences are unaffected")
    # the sequence that lost a page is marked, not silently wrong: every head reads that page
    assert torch.isnan(out[1]).all() and torch.isnan(lse[1]).all()
    bt[1, 3] = -5
    for grid in (0, 1, 3, 50):   # whole pairs and pairs split between units (the mark passes through the merge)
        da.set_option("grid_blocks", grid)
        out, lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, bt.cuda(), dev.seq_lens, 0, dev.scale,
                                  out_dtype=torch.bfloat16 if grid == 3 else torch.float32)
        assert da.read_device_status()[0] == 1
        assert torch.isnan(out[1]).all() and torch.isnan(lse[1]).all(), grid
        assert_close(lse[0].cpu().numpy(), ref_lse[0], "other sequences are unaffected")
        assert_close(lse[2].cpu().numpy(), ref_lse[2], "other sequences are unaffected")
    da.set_option("grid_blocks", 0)
    # a window that leaves the bad page out: nothing is wrong with that call
    out, lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, bt.cuda(), dev.seq_lens, 100, dev.scale)
    assert da.read_device_status() == (0, 0, 0, 0) and torch.isfinite(out).all()
    # a sequence longer than its block-table row, and a negative length
    sl = good.seq_lens.clone()
    sl[0] = good.block_table.shape[1] * 16 + 1
    sl[2] = -4
    out, lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, sl.cuda(), 0, dev.scale)
    st = da.read_device_status()
    assert st[0] == 2 and st[1] in (0, 2)
    assert (out[0] == 0).all() and torch.isneginf(lse[0]).all() and (out[2] == 0).all()
    assert_close(out[1].cpu().numpy(), ref[1], "the valid sequence")
    # and the library still works afterwards
    check(da, good, "after errors")


# ------------------------------------------------------------------ the workloads at full size

def _full_size(da, case, ids, what, out_dtype=torch.float32):
    """The workload at full size in the default launch configuration, sequences `ids` against the oracle
    (the others: finite, clean status)."""
    out, lse = da.decode_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens,
                              case.window, case.scale, out_dtype=out_dtype)
    assert da.read_device_status() == (0, 0, 0, 0)
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
    sub = workloads.host_subcase(case, ids)
    ref, ref_lse = oracle_of(sub)
    got = out[ids].float().cpu().numpy().astype(np.float64)
    if out_dtype == torch.float32:
        assert_close(got, ref, what + " out")
    else:
        assert_bf16_close(got, ref, what + " out(bf16)")
    assert_close(lse[ids].cpu().numpy(), ref_lse, what + " lse")


def test_c2_full_size_every_sequence(da):
    da.set_option("grid_blocks", 0)
    case = workloads.c2("cuda")
    _full_size(da, case, list(range(case.B)), "c2")
    _full_size(da, case, list(range(0, case.B, 2)), "c2 bf16", torch.bfloat16)


def test_c4_long_context_page64_every_sequence(da):
    da.set_option("grid_blocks", 0)
    case = workloads.c4("cuda")
    _full_size(da, case, list(range(case.B)), "c4")


def test_c5_shared_prefix_full_and_window_every_fourth_sequence(da):
    da.set_option("grid_blocks", 0)
    full = workloads.c5("cuda", 0)
    ids = sorted(set(range(0, full.B, 4)) | {int(np.argmin(full.lens)), int(np.argmax(full.lens))})
    _full_size(da, full, ids, "c5a")
    full.window = 8192
    _full_size(da, full, ids, "c5b")


def test_c3_scattered_in_large_pool_every_fourth_sequence(da):
    da.set_option("grid_blocks", 0)
    case = workloads.c3("cuda")
    lens = case.lens
    ids = sorted(set(range(0, case.B, 4)) | {int(np.argmin(lens)), int(np.argmax(lens))})
    _full_size(da, case, ids, "c3")
