"""GPU parity of decode_attn_append (the KV-cache write before each decode-attention call): the
pools after the CUDA kernel must equal, bit for bit, the pools after the CPU oracle's append, and a
decode loop of append + decode_attn must match the oracle's loop."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from test_gpu_parity import assert_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def da():
    import paper_2512_10977_b200 as pkg
    pkg.lib()
    pkg.set_option("grid_blocks", 0)
    return pkg


@pytest.mark.parametrize("P", [16, 64, 128])
@pytest.mark.parametrize("layout", ["head_major", "token_major"])
def test_append_is_bit_exact(da, P, layout):
    lens = [1, 16, 17, 0, 64, 65, 300, 128, 129]
    case = workloads.build_case("app", lens, P, 5 + P, "cpu", layout=layout, pool_pages=None, poison=False)
    gen = torch.Generator().manual_seed(P)
    k_new = torch.randn((len(lens), 8, 128), generator=gen).to(torch.bfloat16)
    v_new = torch.randn((len(lens), 8, 128), generator=gen).to(torch.bfloat16)
    dev = workloads.to_device(case, "cuda")
    da.decode_attn_append(k_new.cuda(), v_new.cuda(), dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens)
    assert da.read_device_status() == (0, 0, 0, 0)
    oracle.kv_append_oracle(k_new, v_new, case.k_pages, case.v_pages, case.block_table, case.seq_lens)
    assert torch.equal(dev.k_pages.cpu().view(torch.int16), case.k_pages.view(torch.int16))
    assert torch.equal(dev.v_pages.cpu().view(torch.int16), case.v_pages.view(torch.int16))


def test_append_with_strided_new_rows(da):
    lens = [33, 2, 100]
    case = workloads.build_case("apps", lens, 16, 77, "cpu", poison=False)
    big = torch.randn((3, 8, 2, 128), generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    k_new, v_new = big[:, :, 0], big[:, :, 1]          # interleaved K and V rows
    dev = workloads.to_device(case, "cuda")
    bigd = big.cuda()
    da.decode_attn_append(bigd[:, :, 0], bigd[:, :, 1], dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens)
    oracle.kv_append_oracle(k_new.contiguous(), v_new.contiguous(), case.k_pages, case.v_pages, case.block_table, case.seq_lens)
    assert torch.equal(dev.k_pages.cpu().view(torch.int16), case.k_pages.view(torch.int16))
    assert torch.equal(dev.v_pages.cpu().view(torch.int16), case.v_pages.view(torch.int16))


def test_decode_loop_append_then_attend(da):
    """Four decode steps: every step grows each sequence by one token (appending its K/V), then
    attends.  Outputs and the final pools must follow the oracle's loop."""
    lens = np.array([15, 63, 200, 1])
    case = workloads.build_case("loop", lens + 4, 16, 81, "cpu", poison=False)   # room for 4 more tokens
    case.seq_lens[:] = torch.from_numpy(lens.astype(np.int32))
    dev = workloads.to_device(case, "cuda")
    gen = torch.Generator().manual_seed(9)
    for step in range(4):
        k_new = torch.randn((4, 8, 128), generator=gen).to(torch.bfloat16)
        v_new = torch.randn((4, 8, 128), generator=gen).to(torch.bfloat16)
        q = torch.randn((4, 48, 128), generator=gen).to(torch.bfloat16)
        case.seq_lens += 1
        dev.seq_lens += 1
        da.decode_attn_append(k_new.cuda(), v_new.cuda(), dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens)
        out, lse = da.decode_attn(q.cuda(), dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 0, case.scale)
        oracle.kv_append_oracle(k_new, v_new, case.k_pages, case.v_pages, case.block_table, case.seq_lens)
        ref, ref_lse = oracle.decode_attn_oracle(q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, 0, case.scale)
        assert_close(out.cpu().numpy(), ref, f"loop step {step} out")
        assert_close(lse.cpu().numpy(), ref_lse, f"loop step {step} lse")
    assert da.read_device_status() == (0, 0, 0, 0)
    assert torch.equal(dev.k_pages.cpu().view(torch.int16), case.k_pages.view(torch.int16))


def test_append_errors(da):
    case = workloads.to_device(workloads.build_case("apperr", [40, 50], 16, 83, "cpu", poison=False), "cuda")
    k_new = torch.zeros((2, 8, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_append(k_new[:, :7], k_new[:, :7], case.k_pages, case.v_pages, case.block_table, case.seq_lens)
    assert e.value.status == 2
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_append(k_new.float().bfloat16()[..., :64], k_new[..., :64], case.k_pages, case.v_pages, case.block_table, case.seq_lens)
    assert e.value.status == 2
    before = case.k_pages.clone()
    bt = case.block_table.clone()
    bt[0, (40 - 1) // 16] = 10 ** 6
    sl = case.seq_lens.clone()
    da.decode_attn_append(k_new + 1, k_new + 1, case.k_pages, case.v_pages, bt, sl)
    st = da.read_device_status()
    assert st[0] == 1 and st[1] == 0 and st[3] == 10 ** 6
    # the bad sequence wrote nothing; the other one wrote its row
    pg1 = int(case.block_table[1, (50 - 1) // 16])
    assert (case.k_pages[pg1, :, (50 - 1) % 16] == 1).all()
    changed = (case.k_pages != before).flatten(1).any(1).nonzero().flatten().tolist()
    assert changed == [pg1]
    sl[1] = case.block_table.shape[1] * 16 + 1
    da.decode_attn_append(k_new, k_new, case.k_pages, case.v_pages, case.block_table, sl)
    assert da.read_device_status()[0] == 2
