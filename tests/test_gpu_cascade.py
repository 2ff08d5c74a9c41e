"""GPU parity of the shared-prefix (cascade) path: decode_attn_cascade must give what the fp64 oracle
gives for plain decode attention on the same inputs -- the shared prefix only changes the schedule
(prefix attended once for the whole batch on the tensor cores, suffixes per sequence, LSE fold)."""
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


@pytest.fixture(params=[0, 2], ids=["one-after-the-other", "side-by-side"], autouse=True)
def overlap(request, da):
    """Every test of this file runs with the two passes one after the other and (wherever the shapes allow it)
    side by side on the library's own streams."""
    da.set_option("cascade_overlap", request.param)
    yield request.param
    da.set_option("cascade_overlap", 1)


def run_both(da, case, prefix, out_dtype=torch.float32):
    ref, ref_lse = oracle.decode_attn_oracle(case.q, case.k_pages, case.v_pages, case.block_table,
                                             case.seq_lens, 0, case.scale)
    dev = workloads.to_device(case, "cuda")
    out, lse = da.decode_attn_cascade(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens,
                                      prefix, dev.scale, out_dtype=out_dtype)
    assert da.read_device_status() == (0, 0, 0, 0)
    return out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64), ref, ref_lse


@pytest.mark.parametrize("P", [16, 64, 128])
@pytest.mark.parametrize("prefix,B", [(128, 1), (256, 5), (1024, 22), (2048, 43)])
def test_cascade_matches_oracle(da, P, prefix, B):
    rng = np.random.default_rng(prefix + B + P)
    lens = prefix + rng.integers(0, 700, size=B)
    lens[0] = prefix                      # a sequence that is nothing but the prefix
    case = workloads.build_case("casc", lens, P, 7 * B + P, "cpu", shared_prefix_tokens=prefix)
    got, got_lse, ref, ref_lse = run_both(da, case, prefix)
    assert_close(got, ref, f"cascade P={P} prefix={prefix} B={B} out")
    assert_close(got_lse, ref_lse, f"cascade P={P} prefix={prefix} B={B} lse")


@pytest.mark.parametrize("Hq,Hkv", [(8, 8), (48, 8), (64, 8), (32, 2), (16, 1)])
def test_cascade_group_sizes(da, Hq, Hkv):
    lens = 512 + np.arange(9) * 37
    case = workloads.build_case("cascg", lens, 16, Hq + Hkv, "cpu", Hq=Hq, Hkv=Hkv, shared_prefix_tokens=512)
    got, got_lse, ref, ref_lse = run_both(da, case, 512)
    assert_close(got, ref, f"cascade Hq={Hq} Hkv={Hkv} out")
    assert_close(got_lse, ref_lse, f"cascade Hq={Hq} Hkv={Hkv} lse")


def test_cascade_equals_plain_decode_and_bf16_out(da):
    lens = [384, 385, 700, 2000, 384 + 64]
    case = workloads.build_case("casceq", lens, 16, 91, "cpu", shared_prefix_tokens=384)
    dev = workloads.to_device(case, "cuda")
    plain, plain_lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 0, dev.scale)
    casc, casc_lse = da.decode_attn_cascade(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 384, dev.scale)
    np.testing.assert_allclose(casc.cpu().numpy(), plain.cpu().numpy(), atol=2e-5, rtol=1e-4)
    np.testing.assert_allclose(casc_lse.cpu().numpy(), plain_lse.cpu().numpy(), atol=2e-5, rtol=1e-5)
    got, got_lse, ref, ref_lse = run_both(da, case, 384, torch.bfloat16)
    assert_bf16_close(got, ref, "cascade bf16 out")
    # prefix 0 falls back to the plain path
    z, zl = da.decode_attn_cascade(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 0, dev.scale)
    assert torch.equal(z, plain) and torch.equal(zl, plain_lse)


def test_cascade_dominant_keys_in_prefix_and_suffix(da):
    """Three keys x20 inside the prefix and one inside a suffix: the weights collapse onto single
    tokens, which is where rounding P to one bf16 would show."""
    lens = [1024 + 300, 1024 + 10, 1024]
    case = workloads.build_case("cascdom", lens, 16, 93, "cpu", shared_prefix_tokens=1024)
    bt = case.block_table.numpy()
    for t in (3, 517, 1000):
        pg = int(bt[0, t // 16])
        case.k_pages[pg, :, t % 16] = (case.k_pages[pg, :, t % 16].float() * 20).to(torch.bfloat16)
    pg = int(bt[0, (1024 + 150) // 16])
    case.k_pages[pg, :, (1024 + 150) % 16] = (case.k_pages[pg, :, (1024 + 150) % 16].float() * 20).to(torch.bfloat16)
    got, got_lse, ref, ref_lse = run_both(da, case, 1024)
    assert_close(got, ref, "cascade dominant out")
    assert_close(got_lse, ref_lse, "cascade dominant lse")


def test_cascade_argument_and_device_errors(da):
    case = workloads.to_device(workloads.build_case("cascerr", [300, 400], 16, 95, "cpu", shared_prefix_tokens=256), "cuda")
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_cascade(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, 200, case.scale)
    assert e.value.status == 2                                   # not a multiple of 128
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_cascade(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, 128 * 64, case.scale)
    assert e.value.status == 2                                   # longer than a block-table row
    sl = case.seq_lens.clone()
    sl[1] = 100                                                  # shorter than the prefix
    out, lse = da.decode_attn_cascade(case.q, case.k_pages, case.v_pages, case.block_table, sl, 256, case.scale)
    assert da.read_device_status()[0] == 2
    # ... and that sequence is treated as empty, the others are unaffected
    assert (out[1] == 0).all() and torch.isneginf(lse[1]).all()
    want, want_lse = da.decode_attn_cascade(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, 256, case.scale)
    assert da.read_device_status() == (0, 0, 0, 0)
    keep = [b for b in range(case.q.shape[0]) if b != 1]
    assert torch.allclose(out[keep], want[keep], atol=2e-5, rtol=1e-4) and torch.allclose(lse[keep], want_lse[keep], atol=2e-5, rtol=1e-4)
    # a page id outside the pool inside the shared prefix: every row attends it, so every row is NaN
    bt = case.block_table.clone()
    bt[:, 3] = 10 ** 6
    out, lse = da.decode_attn_cascade(case.q, case.k_pages, case.v_pages, bt, case.seq_lens, 256, case.scale)
    st = da.read_device_status()
    assert st[0] == 1 and st[3] == 10 ** 6
    assert torch.isnan(out).all() and torch.isnan(lse).all()
    # ... and one in a single sequence's own tokens marks that sequence only
    bt = case.block_table.clone()
    own = 256 // case.k_pages.shape[2]                           # first page after the prefix
    b_long = int(torch.argmax(case.seq_lens))
    bt[b_long, own] = -7
    out, lse = da.decode_attn_cascade(case.q, case.k_pages, case.v_pages, bt, case.seq_lens, 256, case.scale)
    assert da.read_device_status()[0] == 1
    assert torch.isnan(out[b_long]).all() and torch.isnan(lse[b_long]).all()
    keep = [b for b in range(case.q.shape[0]) if b != b_long]
    assert torch.allclose(out[keep], want[keep], atol=2e-5, rtol=1e-4) and torch.allclose(lse[keep], want_lse[keep], atol=2e-5, rtol=1e-4)


def test_c5a_full_size_cascade_every_fourth_sequence(da):
    case = workloads.c5("cuda", 0)
    out, lse = da.decode_attn_cascade(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens,
                                      16384, case.scale)
    assert da.read_device_status() == (0, 0, 0, 0)
    ids = sorted(set(range(0, case.B, 4)) | {int(np.argmin(case.lens)), int(np.argmax(case.lens)), 77})
    sub = workloads.host_subcase(case, ids)
    ref, ref_lse = oracle.decode_attn_oracle(sub.q, sub.k_pages, sub.v_pages, sub.block_table, sub.seq_lens, 0, sub.scale)
    assert_close(out[ids].cpu().numpy(), ref, "c5a cascade out")
    assert_close(lse[ids].cpu().numpy(), ref_lse, "c5a cascade lse")
    # the library's own choice (option 1) on this workload: own parts of up to 8192 tokens beside a 16384-token
    # prefix -> side by side, which shows as two launches of the prefix kernel (six launches instead of five)
    da.set_option("cascade_overlap", 1)
    before = da.launch_count()
    out1, lse1 = da.decode_attn_cascade(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens,
                                        16384, case.scale)
    assert da.launch_count() - before == 6
    assert torch.allclose(out1, out, atol=2e-5, rtol=1e-4) and torch.allclose(lse1, lse, atol=2e-5, rtol=1e-4)
    # ... and with block-table rows that can hold no more than the prefix and a page, one after the other
    narrow = case.block_table[:, :1025].contiguous()
    short = torch.clamp(case.seq_lens, max=16384 + 16)
    before = da.launch_count()
    da.decode_attn_cascade(case.q, case.k_pages, case.v_pages, narrow, short, 16384, case.scale)
    assert da.launch_count() - before == 5
    assert da.read_device_status() == (0, 0, 0, 0)


def test_cascade_side_by_side_replayed_from_a_cuda_graph(da, overlap):
    """The fork onto the library's own streams and the join are part of what is captured: a replay runs the two
    passes again (side by side if that is the mode) and reads seq_lens and q as they are then."""
    prefix = 1024
    lens = prefix + np.array([0, 5, 300, 2000, 64, 1500, 17, 900])
    case = workloads.build_case("cascgraph", lens + 2, 16, 29, "cpu", shared_prefix_tokens=prefix, poison=False)
    case.seq_lens[:] = torch.from_numpy(lens.astype(np.int32))
    dev = workloads.to_device(case, "cuda")
    out = torch.empty(dev.q.shape, dtype=torch.float32, device="cuda")
    lse = torch.empty(dev.q.shape[:2], dtype=torch.float32, device="cuda")

    def call(stream=None):
        da.decode_attn_cascade(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, prefix, dev.scale,
                               out=out, lse=lse, stream=stream)

    call()   # one-time set-up (kernel attributes, the library's streams) outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            call(side)
    for step in range(3):
        case.seq_lens += 1 if step else 0
        dev.seq_lens.copy_(case.seq_lens)
        qn = torch.randn(case.q.shape, generator=torch.Generator().manual_seed(step)).to(torch.bfloat16)
        case.q.copy_(qn)
        dev.q.copy_(qn)
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        ref, ref_lse = oracle.decode_attn_oracle(case.q, case.k_pages, case.v_pages, case.block_table, case.seq_lens,
                                                 0, case.scale)
        assert_close(out.cpu().numpy(), ref, f"cascade replay {step} out")
        assert_close(lse.cpu().numpy(), ref_lse, f"cascade replay {step} lse")
    assert da.read_device_status() == (0, 0, 0, 0)
