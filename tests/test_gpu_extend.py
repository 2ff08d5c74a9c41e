"""GPU parity of decode_attn_extend (causal attention of Lq new tokens per sequence over the paged
cache, on the tcgen05 tensor cores) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import assert_bf16_close, assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def da():
    import paper_2512_10977_b200 as pkg
    pkg.lib()
    pkg.set_option("grid_blocks", 0)
    return pkg


def run_case(da, lens, Lq, P, seed, Hq=48, Hkv=8, out_dtype=torch.float32, **kw):
    case = workloads.build_case("ext", lens, P, seed, "cpu", Hq=Hq, Hkv=Hkv, **kw)
    q = torch.randn((len(lens), Lq, Hq, 128), generator=torch.Generator().manual_seed(seed)).to(torch.bfloat16)
    ref, ref_lse = oracle.extend_attn_oracle(q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, case.scale)
    dev = workloads.to_device(case, "cuda")
    out, lse = da.decode_attn_extend(q.cuda(), dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, dev.scale,
                                     out_dtype=out_dtype)
    assert da.read_device_status() == (0, 0, 0, 0)
    return out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), ref, ref_lse


@pytest.mark.parametrize("P", [16, 64, 128])
@pytest.mark.parametrize("Lq", [1, 2, 5, 22, 43, 130])
def test_extend_matches_oracle(da, P, Lq):
    lens = [Lq, Lq + 1, 127 + Lq, 128 + Lq, 129 + Lq, 1000, 257 + Lq]
    lens = [max(L, Lq) for L in lens]
    got, got_lse, ref, ref_lse = run_case(da, lens, Lq, P, 3 * Lq + P, pool_pages=None, pad_table_to=80)
    assert_close(got, ref, f"extend P={P} Lq={Lq} out")
    assert_close(got_lse, ref_lse, f"extend P={P} Lq={Lq} lse")


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (64, 8), (32, 2), (16, 1)])
def test_extend_group_sizes(da, Hq, Hkv):
    got, got_lse, ref, ref_lse = run_case(da, [300, 77, 513], 9, 16, Hq + Hkv, Hq=Hq, Hkv=Hkv)
    assert_close(got, ref, f"extend Hq={Hq} Hkv={Hkv} out")
    assert_close(got_lse, ref_lse, f"extend Hq={Hq} Hkv={Hkv} lse")


def test_extend_long_context_few_sequences_uses_kv_splits(da):
    got, got_lse, ref, ref_lse = run_case(da, [9000, 4100], 2, 16, 71)
    assert_close(got, ref, "extend splits out")
    assert_close(got_lse, ref_lse, "extend splits lse")


def test_extend_chunk_of_a_feedback_prompt(da):
    """A 1536-token chunk appended to contexts of a few thousand tokens (several row tiles per block row)."""
    got, got_lse, ref, ref_lse = run_case(da, [1536, 4000, 2500], 1536, 16, 73)
    assert_close(got, ref, "extend chunk out")
    assert_close(got_lse, ref_lse, "extend chunk lse")


def test_extend_bf16_out_empty_and_poisoned_tails(da):
    lens = [0, 37, 300, 0, 130]
    got, got_lse, ref, ref_lse = run_case(da, lens, 4, 16, 75, out_dtype=torch.bfloat16, poison=True, pool_pages=120, pad_table_to=40)
    # the oracle's convention for an empty sequence: zeros and -inf
    assert (got[0] == 0).all() and np.isneginf(got_lse[0]).all() and (got[3] == 0).all()
    assert np.isfinite(got).all()
    assert_bf16_close(got, ref, "extend bf16 out")
    assert_close(got_lse, ref_lse, "extend lse")


def test_extend_with_one_token_equals_decode_attn(da):
    case = workloads.build_case("ext1", [700, 33, 2100, 1], 16, 77, "cpu")
    dev = workloads.to_device(case, "cuda")
    want, want_lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 0, dev.scale)
    got, got_lse = da.decode_attn_extend(dev.q[:, None].contiguous(), dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, dev.scale)
    np.testing.assert_allclose(got[:, 0].cpu().numpy(), want.cpu().numpy(), atol=2e-5, rtol=1e-4)
    np.testing.assert_allclose(got_lse[:, 0].cpu().numpy(), want_lse.cpu().numpy(), atol=2e-5, rtol=1e-5)


def test_extend_errors(da):
    case = workloads.to_device(workloads.build_case("exterr", [300, 400], 16, 79, "cpu"), "cuda")
    q = torch.zeros((2, 8, 48, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_extend(q[:, :, :47], case.k_pages, case.v_pages, case.block_table, case.seq_lens, 1.0)
    assert e.value.status == 2
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_extend(q[..., :64], case.k_pages, case.v_pages, case.block_table, case.seq_lens, 1.0)
    assert e.value.status == 5
    sl = case.seq_lens.clone()
    sl[0] = 5                                # fewer tokens than the query block
    out, lse = da.decode_attn_extend(q, case.k_pages, case.v_pages, case.block_table, sl, 1.0)
    assert da.read_device_status()[0] == 2
    assert (out[0] == 0).all()


# ------------------------------------------------------------------ a few new tokens: the streaming path

@pytest.mark.parametrize("Hq,Hkv,Lq", [(48, 8, 2), (8, 8, 16), (16, 8, 8), (32, 8, 4), (32, 8, 3), (24, 8, 5), (48, 8, 1),
                                       # 17 .. 48 query rows per KV head: two column sets per thread block
                                       (48, 8, 3), (48, 8, 4), (48, 8, 5), (48, 8, 8), (8, 8, 17), (8, 8, 33), (64, 8, 6),
                                       (128, 8, 3), (32, 2, 2)])
@pytest.mark.parametrize("P", [16, 64])
def test_few_new_tokens_stream_and_tensor_core_paths_agree_with_the_oracle(da, Hq, Hkv, Lq, P):
    """Lq * (Hq / Hkv) <= 48 query rows per KV head go through the plan / partition / merge kernels as one
    wider group (per-column causal limits; beyond 16 rows as two column sets of warps over the same K and V
    tiles); option extend_stream_rows = 0 forces the tcgen05 kernel."""
    lens = [Lq, Lq + 1, 15 + Lq, 16 + Lq, 63 + Lq, 64 + Lq, 65 + Lq, 1000, 0, 2500]
    lens = [L if L == 0 else max(L, Lq) for L in lens]
    try:
        for rows, grid in ((48, 0), (48, 1), (48, 7), (48, 300), (0, 0)):
            da.set_option("extend_stream_rows", rows)
            da.set_option("grid_blocks", grid)
            got, got_lse, ref, ref_lse = run_case(da, lens, Lq, P, 5 * Lq + P + Hq, Hq=Hq, Hkv=Hkv, poison=True,
                                                  pool_pages=400 if P == 16 else 120, pad_table_to=170 if P == 16 else 50)
            assert np.isfinite(got[[i for i, L in enumerate(lens) if L]]).all()
            assert_close(got, ref, f"few tokens rows={rows} grid={grid} out")
            assert_close(got_lse, ref_lse, f"few tokens rows={rows} grid={grid} lse")
            assert (got[8] == 0).all() and np.isneginf(got_lse[8]).all()
    finally:
        da.set_option("extend_stream_rows", 16)
        da.set_option("grid_blocks", 0)


def test_few_new_tokens_bf16_out_strided_views_and_errors(da):
    lens, Lq = [300, 70, 2, 1030], 2
    case = workloads.build_case("extv", lens, 16, 91, "cpu")
    q = torch.randn((4, Lq, 48, 128), generator=torch.Generator().manual_seed(2)).to(torch.bfloat16)
    ref, ref_lse = oracle.extend_attn_oracle(q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, case.scale)
    dev = workloads.to_device(case, "cuda")
    q_big = torch.zeros((4, Lq + 1, 50, 256), dtype=torch.bfloat16, device="cuda")
    q_view = q_big[:, 1:, 1:49, :128]
    q_view.copy_(q)
    out_big = torch.full((4, Lq, 48, 384), 7.0, device="cuda")
    out_view = out_big[..., 128:256]
    lse_big = torch.full((Lq, 4, 48), 7.0, device="cuda")
    lse_view = lse_big.permute(1, 0, 2)
    da.decode_attn_extend(q_view, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, dev.scale, out=out_view, lse=lse_view)
    assert da.read_device_status() == (0, 0, 0, 0)
    assert_close(out_view.cpu().numpy(), ref, "strided out")
    assert_close(lse_view.cpu().numpy(), ref_lse, "strided lse")
    assert (out_big[..., :128] == 7).all() and (out_big[..., 256:] == 7).all()
    out16, _ = da.decode_attn_extend(q.cuda(), dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, dev.scale,
                                     out_dtype=torch.bfloat16)
    assert_bf16_close(out16.float().cpu().numpy().astype(np.float64), ref, "bf16 out")
    sl = dev.seq_lens.clone()
    sl[1] = 1                                # fewer tokens than the query block
    out, lse = da.decode_attn_extend(q.cuda(), dev.k_pages, dev.v_pages, dev.block_table, sl, dev.scale)
    st = da.read_device_status()
    assert st[0] == 2 and st[1] == 1
    assert (out[1] == 0).all() and torch.isneginf(lse[1]).all()
    assert_close(out[0].cpu().numpy(), ref[0], "other sequences are unaffected")


# ------------------------------------------------------------------ the benchmark's configurations at full size

@pytest.mark.parametrize("Lq", [2, 512])
def test_c2_full_size_extend_sampled(da, Lq):
    """c2's cache with Lq new tokens per sequence, as `bench.py --extend` times it; sampled sequences and
    query tokens against the single-token oracle on a cache cut at each query's position."""
    da.set_option("grid_blocks", 0)
    case = workloads.c2("cuda")
    B = case.B
    q = torch.randn((B, Lq, 48, 128), device="cuda", generator=torch.Generator(device="cuda").manual_seed(7)).to(torch.bfloat16)
    out, lse = da.decode_attn_extend(q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, case.scale)
    assert da.read_device_status() == (0, 0, 0, 0)
    assert torch.isfinite(out).all() and torch.isfinite(lse).all()
    ids = sorted({int(np.argmin(case.lens)), int(np.argmax(case.lens)), 17})
    sub = workloads.host_subcase(case, ids)
    for qi in sorted({0, Lq // 2, Lq - 1}):
        cut = (sub.lens - Lq + qi + 1).astype(np.int32)
        ref, ref_lse = oracle.decode_attn_oracle(q[ids, qi].cpu().contiguous(), sub.k_pages, sub.v_pages, sub.block_table,
                                                 cut, 0, sub.scale)
        assert_close(out[ids, qi].cpu().numpy(), ref, f"c2 extend Lq={Lq} qi={qi} out")
        assert_close(lse[ids, qi].cpu().numpy(), ref_lse, f"c2 extend Lq={Lq} qi={qi} lse")


@pytest.mark.parametrize("Lq,Hq", [(4, 48), (22, 48), (130, 8), (40, 16)])
def test_repeated_tensor_core_calls_give_identical_results(da, Lq, Hq):
    """The tensor-core kernel adds in a fixed order, so identical calls must agree bit for bit; a hand-over
    race between its warps would show up here as an occasional difference (partly filled row tiles included)."""
    lens = [Lq + 700, Lq, 2600, 1300 + Lq]
    case = workloads.build_case("rep", lens, 16, 90 + Lq, "cpu", Hq=Hq, Hkv=8)
    q = torch.randn((len(lens), Lq, Hq, 128), generator=torch.Generator().manual_seed(Lq)).to(torch.bfloat16).cuda()
    dev = workloads.to_device(case, "cuda")
    da.set_option("extend_stream_rows", 0)      # always the tensor-core kernel
    try:
        first, first_lse = da.decode_attn_extend(q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, dev.scale)
        first, first_lse = first.clone(), first_lse.clone()
        for _ in range(40):
            out, lse = da.decode_attn_extend(q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, dev.scale)
            assert torch.equal(out, first) and torch.equal(lse, first_lse)
    finally:
        da.set_option("extend_stream_rows", 16)
    assert da.read_device_status() == (0, 0, 0, 0)
