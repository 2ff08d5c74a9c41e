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
