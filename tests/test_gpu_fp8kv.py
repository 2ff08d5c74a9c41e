"""GPU parity of decode_attn_fp8kv (8-bit E4M3 cache with per-KV-head factors), through the C ABI,
against the fp64 oracle of the same operation on the same seeded codes.  Tolerance as for the bf16
cache: fp32 out and lse |d| <= 1e-3 + 1e-3*|ref|; bf16 out |d| <= 8e-3; indexing checks bit-exact."""
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
    return oracle.decode_attn_fp8kv_oracle(case.q, case.k_pages, case.v_pages, case.k_scale, case.v_scale,
                                           case.block_table, case.seq_lens, case.window, case.scale)


def gpu_of(da, case, out_dtype=torch.float32):
    dev = workloads.to_device(case, "cuda")
    out, lse = da.decode_attn_fp8kv(dev.q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, dev.block_table,
                                    dev.seq_lens, dev.window, dev.scale, out_dtype=out_dtype)
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


def check(da, case, what, grid=0, out_dtype=torch.float32):
    da.set_option("grid_blocks", grid)
    ref, ref_lse = oracle_of(case)
    got, got_lse = gpu_of(da, case, out_dtype)
    if out_dtype == torch.float32:
        assert_close(got, ref, what + " out")
    else:
        assert (np.abs(got - ref) <= 8e-3).all(), what + " out(bf16)"
    assert_close(got_lse, ref_lse, what + " lse")
    return got, got_lse, ref, ref_lse


def fp8_case(name, lens, P, seed, **kw):
    return workloads.build_case(name, lens, P, seed, "cpu", kv_dtype="fp8", **kw)


LENS = [1, 2, 15, 16, 17, 31, 33, 63, 64, 65, 127, 128, 129, 255, 257, 1000]


@pytest.mark.parametrize("P", [16, 32, 64, 128])
def test_lengths_around_tile_and_page_edges(da, P):
    case = fp8_case("edges8", LENS, P, 200 + P, pad_table_to=40)
    for grid in (0, 1, 5):
        got, _, ref, _ = check(da, case, f"P={P} grid={grid}", grid)
    # how close the path really is on N(0,1)-like data (the bar above is much wider)
    assert np.abs(got - ref).max() < 2e-4


@pytest.mark.parametrize("window", [1, 5, 16, 17, 63, 64, 65, 127, 128, 129, 200, 257, 100000])
def test_sliding_window(da, window):
    lens = [1, 17, 64, 65, 200, 257, 258, 700]
    case = fp8_case("win8", lens, 16, 7, window=window)
    check(da, case, f"W={window}")
    check(da, case, f"W={window} one block", 1)


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (32, 8), (48, 8), (64, 8), (24, 2), (16, 1), (40, 4)])
def test_group_sizes(da, Hq, Hkv):
    case = fp8_case("gqa8", [300, 77, 1, 129], 16, Hq, Hq=Hq, Hkv=Hkv)
    check(da, case, f"Hq={Hq} Hkv={Hkv}")
    check(da, case, f"Hq={Hq} Hkv={Hkv} grid 3", 3)


@pytest.mark.parametrize("grid", [1, 2, 3, 7, 64, 148, 296, 1000, 4096])
def test_any_split_schedule_gives_the_same_answer(da, grid):
    case = fp8_case("splits8", [2500, 3, 900, 64, 4097, 130], 16, 11)
    check(da, case, f"grid={grid}", grid)


@pytest.mark.parametrize("tail,frac", [(0, 192), (1, 128), (6, 0), (6, 256), (64, 200)])
def test_any_mix_of_static_and_ticketed_units_gives_the_same_answer(da, tail, frac):
    case = fp8_case("units8", [2500, 3, 900, 0, 64, 4097, 130, 9000], 16, 13)
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


def test_empty_sequences(da):
    case = fp8_case("empty8", [0, 130, 0, 0, 5, 2049, 0], 16, 3)
    got, got_lse, _, _ = check(da, case, "empties")
    for b in (0, 2, 3, 6):
        assert (got[b] == 0).all() and np.isneginf(got_lse[b]).all()
    case = fp8_case("allempty8", [0, 0], 16, 5)
    got, got_lse, _, _ = check(da, case, "all empty")
    assert (got == 0).all() and np.isneginf(got_lse).all()


def test_token_major_layout(da):
    case = fp8_case("tm8", [513, 40, 1300], 16, 21, layout="token_major")
    assert case.k_pages.stride(1) < case.k_pages.stride(2)
    check(da, case, "token-major")


def test_bf16_output_and_unit_factors(da):
    case = fp8_case("bf16o8", [700, 33, 2100, 1], 16, 23)
    check(da, case, "bf16 out", 0, torch.bfloat16)
    case.k_scale = None
    case.scale = 0.002          # raw K codes reach ~200: keep the scores O(1)
    check(da, case, "no K factors")


def test_float8_dtype_pools_are_accepted(da):
    case = fp8_case("f8dtype", [300, 64], 16, 25)
    ref, ref_lse = oracle_of(case)
    dev = workloads.to_device(case, "cuda")
    out, lse = da.decode_attn_fp8kv(dev.q, dev.k_pages.view(torch.float8_e4m3fn), dev.v_pages.view(torch.float8_e4m3fn),
                                    dev.k_scale, dev.v_scale, dev.block_table, dev.seq_lens, 0, dev.scale)
    assert_close(out.cpu().numpy(), ref, "float8 view")


def test_wide_range_of_query_magnitudes(da):
    """Heads whose queries are tiny, huge or span many binades: the power-of-two rescaling and the
    two-term split of q must not lose them."""
    case = fp8_case("qrange8", [600, 90], 16, 27)
    q = case.q.float()
    q[:, 0] *= 2.0 ** -20
    q[:, 1] *= 2.0 ** 12
    q[:, 2, ::2] *= 2.0 ** -9          # elements far below the head's largest
    q[:, 3] = 0
    case.q = q.to(torch.bfloat16)
    case.scale = 1.0 / 64
    check(da, case, "q magnitudes")


def test_sharp_and_flat_softmax(da):
    """One dominant key (weights collapse) and scale 0 (all weights equal)."""
    case = fp8_case("sharp8", [900, 130], 16, 29)
    check(da, case, "flat", 0)
    case.scale = 0.0
    got, got_lse, ref, _ = check(da, case, "scale 0")
    case.scale = 4.0
    check(da, case, "sharp")


# ------------------------------------------------------------------ indexing, bit-exact

def _probe_case(P, lens, window, seed):
    """K codes 0 everywhere; V rows carry (token, physical page, kv head) as small integers (exact in
    E4M3 up to 16); factors 1."""
    case = fp8_case("probe8", lens, P, seed, window=window, poison=True)
    case.k_scale = case.v_scale = None
    nan = workloads.E4M3_NAN
    case.k_pages[case.k_pages != nan] = 0
    bt = case.block_table.numpy()
    for b, L in enumerate(lens):
        for t in range(L):
            pg = int(bt[b, t // P])
            for g in range(case.k_pages.shape[1]):
                v = torch.zeros(128)
                v[0], v[1], v[2], v[3] = t % 16, (t // 16) % 16, t // 256, pg % 16
                v[4], v[5], v[6] = (pg // 16) % 16, g, b
                case.v_pages[pg, g, t % P] = v.to(torch.float8_e4m3fn).view(torch.uint8)
    return case


@pytest.mark.parametrize("P", [16, 64])
def test_probe_token_is_returned_bit_for_bit(da, P):
    lens, W = [300, 77, 1025], 100
    base = _probe_case(P, lens, W, 41)
    dev = workloads.to_device(base, "cuda")
    bt = base.block_table.numpy()
    # queries: +-2 patterns (exact in two E4M3 terms); the probe key is 4 * q, others 0: gap = 16 * 128 * scale
    sign = torch.where(torch.rand((len(lens), 8, 128), generator=torch.Generator().manual_seed(3)) < 0.5, -1.0, 1.0)
    q = (2 * sign).repeat_interleave(6, dim=1).to(torch.bfloat16).cuda()
    for grid in (0, 1):
        da.set_option("grid_blocks", grid)
        for b, L in enumerate(lens):
            lo = max(L - W, 0)
            cand = [lo, lo + 1, L - 1, (lo // P + 1) * P - 1, (lo // P + 1) * P,
                    (lo // 128 + 1) * 128 - 1, (lo // 128 + 1) * 128, (L - 1) // 128 * 128 - 1, (L - 1) // 128 * 128,
                    (lo // 32 + 1) * 32 - 1, (lo // 32 + 1) * 32]
            for t_star in sorted({t for t in cand if lo <= t < L}):
                pg = int(bt[b, t_star // P])
                saved = dev.k_pages[pg, :, t_star % P].clone()
                kstar = (4 * sign[b]).to(torch.float8_e4m3fn).view(torch.uint8).cuda()      # [8, 128]
                dev.k_pages[pg, :, t_star % P] = kstar
                out, _ = da.decode_attn_fp8kv(q, dev.k_pages, dev.v_pages, None, None, dev.block_table, dev.seq_lens, W, 1.0)
                want = dev.v_pages[pg, :, t_star % P].view(torch.float8_e4m3fn).float()     # [8, 128]
                got = out[b].view(8, 6, 128)
                assert torch.equal(got, want[:, None, :].expand(8, 6, 128)), (P, grid, b, t_star)
                assert got[0, 0, 0].item() == t_star % 16 and got[0, 0, 2].item() == t_star // 256
                assert got[3, 2, 5].item() == 3 and got[0, 0, 6].item() == b
                dev.k_pages[pg, :, t_star % P] = saved
    assert da.read_device_status() == (0, 0, 0, 0)


def test_integer_mean_is_exact(da):
    """K = 0 and V small integers over a power-of-two number of tokens: the mean is exact in fp32."""
    lens = [256, 1024, 128]
    case = fp8_case("int8", lens, 16, 47)
    case.k_scale = case.v_scale = None
    nan = workloads.E4M3_NAN
    case.k_pages[case.k_pages != nan] = 0
    vi = torch.randint(-8, 9, case.v_pages.shape, generator=torch.Generator().manual_seed(1)).float()
    vi = vi.to(torch.float8_e4m3fn).view(torch.uint8)
    case.v_pages = torch.where(case.v_pages != nan, vi, case.v_pages)
    ref, ref_lse = oracle_of(case)
    try:
        da.set_option("grid_blocks", 1)
        da.set_option("tail_units", 0)
        got, got_lse = gpu_of(da, case)
        assert np.array_equal(got, ref)
        np.testing.assert_allclose(got_lse, ref_lse, atol=1e-6)
    finally:
        da.set_option("grid_blocks", 0)
        da.set_option("tail_units", 4)


def test_nan_canaries(da):
    lens = [5, 17, 300, 1029, 64, 128]
    dirty = fp8_case("dirty8", lens, 16, 53, poison=True, pool_pages=400, pad_table_to=90)
    assert (dirty.k_pages == workloads.E4M3_NAN).sum() > 1000 and (dirty.block_table == -1).any()
    for grid in (0, 1, 9):
        got, got_lse, _, _ = check(da, dirty, f"canary grid={grid}", grid)
        assert np.isfinite(got).all() and np.isfinite(got_lse).all()
    check(da, fp8_case("dirtyw8", lens, 16, 53, poison=True, pool_pages=400, window=20), "canary window")


def test_host_side_argument_errors(da):
    case = workloads.to_device(fp8_case("err8", [100], 16, 59), "cuda")
    bf = workloads.to_device(workloads.build_case("errbf", [100], 16, 59, "cpu"), "cuda")
    with pytest.raises(da.DecodeAttnError) as e:      # a bf16 pool handed to the 8-bit entry point
        da.decode_attn_fp8kv(case.q, bf.k_pages, bf.v_pages, None, None, case.block_table, case.seq_lens, 0, 1.0)
    assert e.value.status == 3
    with pytest.raises(da.DecodeAttnError) as e:      # and the reverse
        da.decode_attn(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, 0, 1.0)
    assert e.value.status == 3
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_fp8kv(case.q, case.k_pages[:, :, :8], case.v_pages[:, :, :8], None, None, case.block_table,
                             case.seq_lens, 0, 1.0)
    assert e.value.status == 5
    with pytest.raises(ValueError):
        da.decode_attn_fp8kv(case.q, case.k_pages, case.v_pages, case.k_scale[:4], None, case.block_table,
                             case.seq_lens, 0, 1.0)
    assert da.read_device_status() == (0, 0, 0, 0)


def test_device_side_errors_set_the_status_word_without_faulting(da):
    good = fp8_case("bad8", [100, 200, 40], 16, 61)
    ref, _ = oracle_of(good)
    dev = workloads.to_device(good, "cuda")
    bt = good.block_table.clone()
    bt[1, 3] = 10 ** 6
    out, lse = da.decode_attn_fp8kv(dev.q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, bt.cuda(), dev.seq_lens,
                                    0, dev.scale)
    st = da.read_device_status()
    assert st[0] == 1 and st[1] == 1 and st[3] == 10 ** 6
    assert_close(out[0].cpu().numpy(), ref[0], "other sequences are unaffected")
    check(da, good, "after errors")


# ------------------------------------------------------------------ the workloads at full size

def _full_size(da, case, ids, what):
    out, lse = da.decode_attn_fp8kv(case.q, case.k_pages, case.v_pages, case.k_scale, case.v_scale, case.block_table,
                                    case.seq_lens, case.window, case.scale)
    assert da.read_device_status() == (0, 0, 0, 0)
    assert torch.isfinite(out).all() and torch.isfinite(lse).all()
    sub = workloads.host_subcase(case, ids)
    ref, ref_lse = oracle_of(sub)
    assert_close(out[ids].cpu().numpy(), ref, what + " out")
    assert_close(lse[ids].cpu().numpy(), ref_lse, what + " lse")


def test_c2_full_size_every_sequence(da):
    da.set_option("grid_blocks", 0)
    case = workloads.c2("cuda", kv_dtype="fp8")
    _full_size(da, case, list(range(case.B)), "c2 fp8")


def test_c4_long_context_page64_every_sequence(da):
    da.set_option("grid_blocks", 0)
    case = workloads.c4("cuda", kv_dtype="fp8")
    _full_size(da, case, list(range(case.B)), "c4 fp8")


def test_c5b_window_every_eighth_sequence(da):
    da.set_option("grid_blocks", 0)
    case = workloads.c5("cuda", 8192, kv_dtype="fp8")
    _full_size(da, case, sorted(set(range(0, case.B, 8)) | {int(np.argmax(case.lens))}), "c5b fp8")


# ------------------------------------------------------------------ quantising append, bit-exact

@pytest.mark.parametrize("P", [16, 64])
@pytest.mark.parametrize("layout", ["head_major", "token_major"])
def test_append_quantises_bit_exactly(da, P, layout):
    lens = [1, 16, 17, 0, 64, 65, 300, 128, 129]
    case = fp8_case("app8", lens, P, 5 + P, layout=layout, poison=False)
    gen = torch.Generator().manual_seed(P)
    # values spread over the whole E4M3 range after division by the factors: ties, subnormals, saturation
    k_new = (torch.randn((len(lens), 8, 128), generator=gen) * torch.exp2(torch.randint(-12, 6, (len(lens), 8, 128), generator=gen).float()))
    v_new = torch.randn((len(lens), 8, 128), generator=gen)
    k_new[0, 0, :4] = torch.tensor([float("nan"), float("inf"), -float("inf"), 0.0])
    k_new, v_new = k_new.to(torch.bfloat16), v_new.to(torch.bfloat16)
    dev = workloads.to_device(case, "cuda")
    da.decode_attn_append_fp8kv(k_new.cuda(), v_new.cuda(), dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale,
                                dev.block_table, dev.seq_lens)
    assert da.read_device_status() == (0, 0, 0, 0)
    oracle.kv_append_fp8_oracle(k_new, v_new, case.k_pages, case.v_pages, case.k_scale, case.v_scale,
                                case.block_table, case.seq_lens)
    assert torch.equal(dev.k_pages.cpu(), case.k_pages) and torch.equal(dev.v_pages.cpu(), case.v_pages)


def test_every_bf16_value_quantises_as_the_oracle_says(da):
    """All 65536 bf16 bit patterns through the kernel's quantiser, for a factor that is not a power of two."""
    allbits = torch.arange(65536, dtype=torch.int32).to(torch.int16).view(torch.bfloat16)     # [65536]
    B = 65536 // (8 * 128)
    k_new = allbits.view(B, 8, 128)
    case = fp8_case("allbf16", [1] * B, 16, 3, poison=False, shuffle=False)
    dev = workloads.to_device(case, "cuda")
    da.decode_attn_append_fp8kv(k_new.cuda(), k_new.cuda(), dev.k_pages, dev.v_pages, dev.k_scale, None,
                                dev.block_table, dev.seq_lens)
    assert da.read_device_status() == (0, 0, 0, 0)
    got_k = dev.k_pages.cpu()[case.block_table[:, 0].long(), :, 0]     # [B, 8, 128]
    got_v = dev.v_pages.cpu()[case.block_table[:, 0].long(), :, 0]
    for g in range(8):
        want = oracle.e4m3_quantize(k_new[:, g].contiguous(), float(case.k_scale[g]))
        assert np.array_equal(got_k[:, g].numpy(), want), g
    want = oracle.e4m3_quantize(k_new.contiguous(), 1.0)
    assert np.array_equal(got_v.numpy(), want)


def test_decode_loop_append_then_attend(da):
    lens = np.array([15, 63, 200, 1])
    case = fp8_case("loop8", lens + 4, 16, 81, poison=False)
    case.seq_lens[:] = torch.from_numpy(lens.astype(np.int32))
    dev = workloads.to_device(case, "cuda")
    gen = torch.Generator().manual_seed(9)
    for step in range(4):
        k_new = torch.randn((4, 8, 128), generator=gen).to(torch.bfloat16)
        v_new = torch.randn((4, 8, 128), generator=gen).to(torch.bfloat16)
        q = torch.randn((4, 48, 128), generator=gen).to(torch.bfloat16)
        case.seq_lens += 1
        dev.seq_lens += 1
        da.decode_attn_append_fp8kv(k_new.cuda(), v_new.cuda(), dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale,
                                    dev.block_table, dev.seq_lens)
        out, lse = da.decode_attn_fp8kv(q.cuda(), dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, dev.block_table,
                                        dev.seq_lens, 0, case.scale)
        oracle.kv_append_fp8_oracle(k_new, v_new, case.k_pages, case.v_pages, case.k_scale, case.v_scale,
                                    case.block_table, case.seq_lens)
        ref, ref_lse = oracle.decode_attn_fp8kv_oracle(q, case.k_pages, case.v_pages, case.k_scale, case.v_scale,
                                                       case.block_table, case.seq_lens, 0, case.scale)
        assert_close(out.cpu().numpy(), ref, f"loop step {step} out")
        assert_close(lse.cpu().numpy(), ref_lse, f"loop step {step} lse")
    assert da.read_device_status() == (0, 0, 0, 0)
    assert torch.equal(dev.k_pages.cpu(), case.k_pages) and torch.equal(dev.v_pages.cpu(), case.v_pages)


def test_c3_scattered_in_large_pool_every_fourth_sequence(da):
    da.set_option("grid_blocks", 0)
    case = workloads.c3("cuda", kv_dtype="fp8")
    ids = sorted(set(range(0, case.B, 4)) | {int(np.argmin(case.lens)), int(np.argmax(case.lens))})
    _full_size(da, case, ids, "c3 fp8")


def test_host_io_matches_device_call(da):
    case = fp8_case("hostio8", [700, 33, 2100, 1, 0], 16, 37)
    dev = workloads.to_device(case, "cuda")
    want, want_lse = da.decode_attn_fp8kv(dev.q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, dev.block_table,
                                          dev.seq_lens, 9, dev.scale)
    q_h, bt_h, sl_h = (t.pin_memory() for t in (case.q, case.block_table, case.seq_lens))
    out_h = torch.empty(case.q.shape, dtype=torch.float32).pin_memory()
    lse_h = torch.empty(case.q.shape[:2], dtype=torch.float32).pin_memory()
    for _ in range(2):
        out_h.fill_(5)
        da.decode_attn_fp8kv_host_io(q_h, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, bt_h, sl_h, 9, dev.scale,
                                     out_h, lse_h)
        torch.cuda.synchronize()
        assert same(out_h, want) and same(lse_h, want_lse)
    out_p = torch.full(case.q.shape, 5.0, dtype=torch.float32)     # pageable: the staged path
    da.decode_attn_fp8kv_host_io(case.q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, case.block_table,
                                 case.seq_lens, 9, dev.scale, out_p, None)
    torch.cuda.synchronize()
    assert same(out_p, want)


# ------------------------------------------------------------------ a few new tokens over the 8-bit cache

@pytest.mark.parametrize("Hq,Hkv,Lq", [(48, 8, 2), (8, 8, 16), (16, 8, 8), (32, 8, 3), (24, 8, 5), (48, 8, 1),
                                       # 17 .. 48 query rows per KV head: two column sets per thread block
                                       (48, 8, 3), (48, 8, 4), (48, 8, 5), (48, 8, 8), (8, 8, 17), (8, 8, 33)])
@pytest.mark.parametrize("P", [16, 64])
def test_few_new_tokens_over_the_fp8_cache(da, Hq, Hkv, Lq, P):
    lens = [Lq, Lq + 1, 31 + Lq, 32 + Lq, 127 + Lq, 128 + Lq, 129 + Lq, 1000, 0, 2500]
    lens = [L if L == 0 else max(L, Lq) for L in lens]
    case = fp8_case("ext8", lens, P, 7 * Lq + P + Hq, Hq=Hq, Hkv=Hkv, poison=True,
                    pool_pages=400 if P == 16 else 120, pad_table_to=170 if P == 16 else 50)
    q = torch.randn((len(lens), Lq, Hq, 128), generator=torch.Generator().manual_seed(Lq)).to(torch.bfloat16)
    ref, ref_lse = oracle.extend_attn_fp8kv_oracle(q, case.k_pages, case.v_pages, case.k_scale, case.v_scale,
                                                   case.block_table, case.seq_lens, case.scale)
    dev = workloads.to_device(case, "cuda")
    try:
        for grid in (0, 1, 7):
            da.set_option("grid_blocks", grid)
            out, lse = da.decode_attn_fp8kv_extend(q.cuda(), dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale,
                                                   dev.block_table, dev.seq_lens, dev.scale)
            assert da.read_device_status() == (0, 0, 0, 0)
            assert_close(out.cpu().numpy(), ref, f"fp8 extend grid={grid} out")
            assert_close(lse.cpu().numpy(), ref_lse, f"fp8 extend grid={grid} lse")
    finally:
        da.set_option("grid_blocks", 0)
    with pytest.raises(da.DecodeAttnError) as e:     # more than 48 query rows per KV head
        big = torch.zeros((len(lens), 49, Hq, 128), dtype=torch.bfloat16, device="cuda")
        da.decode_attn_fp8kv_extend(big, dev.k_pages, dev.v_pages, None, None, dev.block_table, dev.seq_lens, 1.0)
    assert e.value.status == 5


# ------------------------------------------------------------------ long query blocks over the 8-bit cache

@pytest.mark.parametrize("Hq,Hkv,Lq", [(48, 8, 9), (48, 8, 64), (8, 8, 130), (32, 8, 100), (16, 1, 300)])
@pytest.mark.parametrize("P", [16, 64, 128])
def test_long_query_blocks_over_the_fp8_cache(da, Hq, Hkv, Lq, P):
    """decode_attn_fp8kv_extend_wide: the attended pages widened exactly to bf16 in scratch, then the
    tensor-core kernel with the per-head factors folded into the score scale and the result; the oracle is
    causal extend attention over the dequantised cache."""
    lens = [Lq, Lq + 1, 127 + Lq, 128 + Lq, 129 + Lq, 1000 + Lq, 0, 2500]
    lens = [L if L == 0 else max(L, Lq) for L in lens]
    case = fp8_case("wide8", lens, P, 5 * Lq + P + Hq, Hq=Hq, Hkv=Hkv, poison=True)
    q = torch.randn((len(lens), Lq, Hq, 128), generator=torch.Generator().manual_seed(Lq + P)).to(torch.bfloat16)
    ref, ref_lse = oracle.extend_attn_fp8kv_oracle(q, case.k_pages, case.v_pages, case.k_scale, case.v_scale,
                                                   case.block_table, case.seq_lens, case.scale)
    dev = workloads.to_device(case, "cuda")
    out, lse = da.decode_attn_fp8kv_extend_wide(q.cuda(), dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale,
                                                dev.block_table, dev.seq_lens, dev.scale)
    assert da.read_device_status() == (0, 0, 0, 0)
    assert_close(out.cpu().numpy(), ref, f"fp8 wide extend Lq={Lq} P={P} out")
    assert_close(lse.cpu().numpy(), ref_lse, f"fp8 wide extend Lq={Lq} P={P} lse")


def test_long_query_blocks_fp8_scratch_errors_and_marking(da):
    Lq = 40
    lens = [500, 41, 900, 0]
    case = fp8_case("wide8err", lens, 16, 77, poison=True)
    dev = workloads.to_device(case, "cuda")
    q = torch.randn((len(lens), Lq, 48, 128), generator=torch.Generator().manual_seed(3)).to(torch.bfloat16).cuda()
    args = (q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, dev.block_table, dev.seq_lens, dev.scale)
    need = da.lib().decode_attn_fp8kv_extend_wide_scratch_bytes(len(lens), dev.block_table.shape[1], 8, 16)
    assert need == 2 * len(lens) * dev.block_table.shape[1] * 8 * 16 * 256
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_fp8kv_extend_wide(*args, scratch=torch.empty(need + 512, dtype=torch.uint8, device="cuda")[16:])
    assert e.value.status == 4
    want, want_lse = da.decode_attn_fp8kv_extend_wide(*args)
    assert da.read_device_status() == (0, 0, 0, 0)
    # scratch for two of the four sequences, and for one: served in groups, same result
    one = need // len(lens)
    for room in (2 * one, one + 256):
        got, got_lse = da.decode_attn_fp8kv_extend_wide(*args, scratch=torch.empty(room, dtype=torch.uint8, device="cuda"))
        assert da.read_device_status() == (0, 0, 0, 0)
        assert torch.equal(got, want) and torch.equal(got_lse, want_lse)
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_fp8kv_extend_wide(*args, scratch=torch.empty(one - 256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 6
    # (the status record names the sequence by its place in the whole batch, whichever group it was served in)
    bt = dev.block_table.clone()
    bt[2, 10] = dev.k_pages.shape[0] + 5
    out, lse = da.decode_attn_fp8kv_extend_wide(q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, bt, dev.seq_lens,
                                                dev.scale, scratch=torch.empty(one, dtype=torch.uint8, device="cuda"))
    st = da.read_device_status()
    assert st[0] == 1 and st[1] == 2
    assert torch.isnan(out[2]).all() and torch.equal(out[[0, 1, 3]], want[[0, 1, 3]])
    # a page id outside the pool, in the middle of sequence 2: its rows are NaN, the others as before
    bt = dev.block_table.clone()
    bt[2, 10] = dev.k_pages.shape[0] + 5
    out, lse = da.decode_attn_fp8kv_extend_wide(q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, bt, dev.seq_lens,
                                                dev.scale)
    st = da.read_device_status()
    assert st[0] == 1 and st[1] == 2
    assert torch.isnan(out[2]).all() and torch.isnan(lse[2]).all()
    keep = [0, 1, 3]
    assert torch.equal(out[keep], want[keep]) and torch.equal(lse[keep], want_lse[keep])
    # a sequence shorter than its new tokens: refused, empty
    sl = dev.seq_lens.clone()
    sl[1] = Lq - 1
    out, lse = da.decode_attn_fp8kv_extend_wide(q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, dev.block_table, sl,
                                                dev.scale)
    assert da.read_device_status()[0] == 2
    assert (out[1] == 0).all() and torch.isneginf(lse[1]).all()
    assert torch.equal(out[[0, 2, 3]], want[[0, 2, 3]])


# ------------------------------------------------------------------ shared prefix over the 8-bit cache

@pytest.fixture(params=[0, 2], ids=["one-after-the-other", "side-by-side"])
def overlap(request, da):
    da.set_option("cascade_overlap", request.param)
    yield request.param
    da.set_option("cascade_overlap", 1)


@pytest.mark.parametrize("P", [16, 64, 128])
@pytest.mark.parametrize("prefix,B", [(128, 1), (256, 5), (1024, 22), (2048, 43)])
def test_fp8_cascade_matches_the_oracle(da, overlap, P, prefix, B):
    """decode_attn_fp8kv_cascade: the prefix's codes widened exactly to bf16 and attended once for the batch on
    the tensor cores (per-head factors folded into the score scale and the result), the rest through the 8-bit
    streaming kernels; the result is plain decode attention over the dequantised cache."""
    rng = np.random.default_rng(prefix + B + P)
    lens = prefix + rng.integers(0, 700, size=B)
    lens[0] = prefix                      # a sequence that is nothing but the prefix
    case = fp8_case("casc8", lens, P, 11 * B + P, shared_prefix_tokens=prefix)
    ref, ref_lse = oracle_of(case)
    dev = workloads.to_device(case, "cuda")
    out, lse = da.decode_attn_fp8kv_cascade(dev.q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, dev.block_table,
                                            dev.seq_lens, prefix, dev.scale)
    assert da.read_device_status() == (0, 0, 0, 0)
    assert_close(out.cpu().numpy(), ref, f"fp8 cascade P={P} prefix={prefix} B={B} out")
    assert_close(lse.cpu().numpy(), ref_lse, f"fp8 cascade P={P} prefix={prefix} B={B} lse")
    plain, plain_lse = da.decode_attn_fp8kv(dev.q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, dev.block_table,
                                            dev.seq_lens, 0, dev.scale)
    np.testing.assert_allclose(out.cpu().numpy(), plain.cpu().numpy(), atol=3e-5, rtol=1e-4)


def test_fp8_cascade_scratch_errors_and_marking(da):
    case = workloads.to_device(fp8_case("casc8e", [300, 400, 256], 16, 97, shared_prefix_tokens=256), "cuda")
    args = (case.q, case.k_pages, case.v_pages, case.k_scale, case.v_scale, case.block_table, case.seq_lens, 256, case.scale)
    need = da.lib().decode_attn_fp8kv_cascade_scratch_bytes(256, 8, 16)
    assert need == 2 * 256 * 8 * 128 * 2
    with pytest.raises(da.DecodeAttnError) as e:          # scratch too small
        da.decode_attn_fp8kv_cascade(*args, prefix_scratch=torch.empty(need - 256, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 6
    with pytest.raises(da.DecodeAttnError) as e:          # not 256-byte aligned
        da.decode_attn_fp8kv_cascade(*args, prefix_scratch=torch.empty(need + 512, dtype=torch.uint8, device="cuda")[16:])
    assert e.value.status == 4
    want, want_lse = da.decode_attn_fp8kv_cascade(*args)
    assert da.read_device_status() == (0, 0, 0, 0)
    # a page id outside the pool inside the shared prefix: every row attends it, so every row is NaN
    bt = case.block_table.clone()
    bt[:, 5] = 10 ** 6
    out, lse = da.decode_attn_fp8kv_cascade(case.q, case.k_pages, case.v_pages, case.k_scale, case.v_scale, bt,
                                            case.seq_lens, 256, case.scale)
    st = da.read_device_status()
    assert st[0] == 1 and st[3] == 10 ** 6
    assert torch.isnan(out).all() and torch.isnan(lse).all()
    # a sequence shorter than the prefix is refused and comes out empty
    sl = case.seq_lens.clone()
    sl[1] = 100
    out, lse = da.decode_attn_fp8kv_cascade(case.q, case.k_pages, case.v_pages, case.k_scale, case.v_scale, case.block_table,
                                            sl, 256, case.scale)
    assert da.read_device_status()[0] == 2
    assert (out[1] == 0).all() and torch.isneginf(lse[1]).all()
    assert torch.allclose(out[[0, 2]], want[[0, 2]], atol=2e-5, rtol=1e-4)


def test_c5a_full_size_fp8_cascade_every_eighth_sequence(da, overlap):
    case = workloads.c5("cuda", 0, kv_dtype="fp8")
    out, lse = da.decode_attn_fp8kv_cascade(case.q, case.k_pages, case.v_pages, case.k_scale, case.v_scale, case.block_table,
                                            case.seq_lens, 16384, case.scale)
    assert da.read_device_status() == (0, 0, 0, 0)
    assert torch.isfinite(out).all() and torch.isfinite(lse).all()
    ids = sorted(set(range(0, case.B, 8)) | {int(np.argmin(case.lens)), int(np.argmax(case.lens))})
    sub = workloads.host_subcase(case, ids)
    ref, ref_lse = oracle_of(sub)
    assert_close(out[ids].cpu().numpy(), ref, "c5a fp8 cascade out")
    assert_close(lse[ids].cpu().numpy(), ref_lse, "c5a fp8 cascade lse")


def test_c2_full_size_long_query_block_over_the_fp8_cache_sampled(da):
    """c2's 8-bit cache with 512 new tokens per sequence, as `bench.py --kv fp8 --extend 512` times it; sampled
    sequences and query tokens against the single-token oracle on a cache cut at each query's position."""
    Lq = 512
    case = workloads.c2("cuda", kv_dtype="fp8")
    q = torch.randn((case.B, Lq, 48, 128), device="cuda", generator=torch.Generator(device="cuda").manual_seed(7)).to(torch.bfloat16)
    out, lse = da.decode_attn_fp8kv_extend_wide(q, case.k_pages, case.v_pages, case.k_scale, case.v_scale, case.block_table,
                                                case.seq_lens, case.scale)
    assert da.read_device_status() == (0, 0, 0, 0)
    assert torch.isfinite(out).all() and torch.isfinite(lse).all()
    ids = sorted({int(np.argmin(case.lens)), int(np.argmax(case.lens)), 17})
    sub = workloads.host_subcase(case, ids)
    for qi in (0, Lq // 2, Lq - 1):
        cut = torch.from_numpy((sub.lens - Lq + qi + 1).astype(np.int32))
        ref, ref_lse = oracle.decode_attn_fp8kv_oracle(q[ids, qi].cpu().contiguous(), sub.k_pages, sub.v_pages, sub.k_scale,
                                                       sub.v_scale, sub.block_table, cut, 0, sub.scale)
        assert_close(out[ids, qi].cpu().numpy(), ref, f"c2 fp8 extend qi={qi} out")
        assert_close(lse[ids, qi].cpu().numpy(), ref_lse, f"c2 fp8 extend qi={qi} lse")
