"""A decode step (KV append, then decode attention) captured once in a CUDA graph and replayed: the
launch-bound inner loop of a decoding service.  The library enqueues only kernels on the caller's
stream (the dependent kernels with programmatic stream serialization), so the calls can be captured;
the first, uncaptured call does the one-time work (kernel attributes, workspace, tensor maps)."""
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


@pytest.mark.parametrize("direct", [1, 0])
def test_append_and_decode_replayed_from_a_cuda_graph(da, direct):
    """direct = 1: this small batch runs as one kernel per call; 0: as plan + partition + merge."""
    da.set_option("direct_path", direct)
    try:
        _append_and_decode_replayed(da, 2 if direct else 4)
    finally:
        da.set_option("direct_path", 1)


def _append_and_decode_replayed(da, launches_per_step):
    lens = np.array([15, 63, 200, 1, 1000])
    steps = 5
    case = workloads.build_case("graph", lens + steps + 1, 16, 91, "cpu", poison=False)
    case.seq_lens[:] = torch.from_numpy(lens.astype(np.int32))
    dev = workloads.to_device(case, "cuda")
    B = len(lens)
    # static buffers the graph reads and writes
    k_new = torch.zeros((B, 8, 128), dtype=torch.bfloat16, device="cuda")
    v_new = torch.zeros_like(k_new)
    q = torch.zeros((B, 48, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((B, 48, 128), dtype=torch.float32, device="cuda")
    lse = torch.empty((B, 48), dtype=torch.float32, device="cuda")
    gen = torch.Generator().manual_seed(17)

    def host_inputs():
        return (torch.randn((B, 8, 128), generator=gen).to(torch.bfloat16),
                torch.randn((B, 8, 128), generator=gen).to(torch.bfloat16),
                torch.randn((B, 48, 128), generator=gen).to(torch.bfloat16))

    def step_on(stream):
        da.decode_attn_append(k_new, v_new, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, stream=stream)
        da.decode_attn(q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, 0, case.scale,
                       out=out, lse=lse, stream=stream)

    def reference(kn, vn, qn):
        oracle.kv_append_oracle(kn, vn, case.k_pages, case.v_pages, case.block_table, case.seq_lens)
        return oracle.decode_attn_oracle(qn, case.k_pages, case.v_pages, case.block_table, case.seq_lens, 0, case.scale)

    # one plain step first: one-time set-up happens outside the capture
    kn, vn, qn = host_inputs()
    case.seq_lens += 1
    dev.seq_lens += 1
    k_new.copy_(kn); v_new.copy_(vn); q.copy_(qn)
    step_on(torch.cuda.current_stream())
    ref, ref_lse = reference(kn, vn, qn)
    assert_close(out.cpu().numpy(), ref, "plain step out")

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    launches_before = da.launch_count()
    with torch.cuda.stream(side):
        # what is captured reads seq_lens at replay time, so the graph serves every later step
        dev.seq_lens += 1
        case.seq_lens += 1
        kn, vn, qn = host_inputs()
        k_new.copy_(kn); v_new.copy_(vn); q.copy_(qn)
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            step_on(side)
    # append + (partition | plan, partition, merge): recorded, not run
    assert da.launch_count() - launches_before == launches_per_step
    graph.replay()
    torch.cuda.synchronize()
    ref, ref_lse = reference(kn, vn, qn)
    assert_close(out.cpu().numpy(), ref, "first replay out")
    assert_close(lse.cpu().numpy(), ref_lse, "first replay lse")

    for s in range(steps - 2):
        kn, vn, qn = host_inputs()
        case.seq_lens += 1
        dev.seq_lens += 1
        k_new.copy_(kn); v_new.copy_(vn); q.copy_(qn)
        graph.replay()
        torch.cuda.synchronize()
        ref, ref_lse = reference(kn, vn, qn)
        assert_close(out.cpu().numpy(), ref, f"replay {s} out")
        assert_close(lse.cpu().numpy(), ref_lse, f"replay {s} lse")
    assert da.read_device_status() == (0, 0, 0, 0)
    assert torch.equal(dev.k_pages.cpu().view(torch.int16), case.k_pages.view(torch.int16))
