"""decode_attn_static_scratch: the entry point for callers that cannot allocate device memory
(a server whose KV-cache pool owns all of HBM, or a step that cannot take cudaMalloc's
device-wide synchronisation).  Its scratch is a fixed array inside the library, shared by every
call, so the check runs it twice in a row on different batches and compares each result with
what decode_attn() gives for the same inputs through its caller-provided workspace -- and with the
fp64 CPU oracle, so that a slip the two entry points share would not pass either.

Collected last on purpose: a run that stops at the first failure has then already run every
other test."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_decode_attn_on_two_calls_in_a_row():
    import paper_2512_10977_b200 as da
    da.set_option("grid_blocks", 0)
    # two different batches: the second must not see anything the first left in the array
    # (the first splits its long sequences over many thread blocks, the second hardly at all)
    cases = [workloads.build_case("na1", [9000, 3, 700, 0, 4097], 16, 71, "cuda", window=0),
             workloads.build_case("na2", [130, 2500, 64], 64, 72, "cuda", window=100)]
    want = [da.decode_attn(c.q, c.k_pages, c.v_pages, c.block_table, c.seq_lens, c.window, c.scale) for c in cases]
    assert da.read_device_status() == (0, 0, 0, 0)
    torch.cuda.synchronize()

    outs = [torch.full(c.q.shape, 3.0, dtype=torch.float32, device="cuda") for c in cases]
    lses = [torch.full(c.q.shape[:2], 3.0, dtype=torch.float32, device="cuda") for c in cases]
    status = [torch.full((4,), -1, dtype=torch.int32, device="cuda") for _ in cases]
    for c, o, l, s in zip(cases, outs, lses, status):      # back to back on one stream
        da.decode_attn_static_scratch(c.q, c.k_pages, c.v_pages, c.block_table, c.seq_lens, c.window, c.scale,
                                      o, l, s)
    torch.cuda.synchronize()
    for c, (w_out, w_lse), o, l, s in zip(cases, want, outs, lses, status):
        assert s.tolist() == [0, 0, 0, 0]
        host = workloads.to_device(c, "cpu")
        o_ref, l_ref = oracle.decode_attn_oracle(host.q, host.k_pages, host.v_pages, host.block_table,
                                                 host.seq_lens, host.window, host.scale)
        for ref, rl in ((w_out.cpu().numpy().astype(np.float64), w_lse.cpu().numpy().astype(np.float64)),
                        (np.asarray(o_ref, dtype=np.float64), np.asarray(l_ref, dtype=np.float64))):
            got = o.cpu().numpy().astype(np.float64)
            assert (np.abs(got - ref) <= 1e-3 + 1e-3 * np.abs(ref)).all()
            gl = l.cpu().numpy().astype(np.float64)
            both_ninf = np.isneginf(gl) & np.isneginf(rl)      # empty sequences: -inf on both sides
            gl, rl = np.where(both_ninf, 0.0, gl), np.where(both_ninf, 0.0, rl)
            assert (np.abs(gl - rl) <= 1e-3 + 1e-3 * np.abs(rl)).all()


def test_static_scratch_reports_device_errors_and_refuses_oversize_batches():
    import paper_2512_10977_b200 as da
    da.set_option("grid_blocks", 0)
    c = workloads.build_case("na3", [100, 200], 16, 73, "cuda")
    out = torch.empty(c.q.shape, dtype=torch.float32, device="cuda")
    st = torch.zeros(4, dtype=torch.int32, device="cuda")
    bt = c.block_table.clone()
    bt[1, 2] = 123456                      # corrupted on purpose; the kernel skips that load
    da.decode_attn_static_scratch(c.q, c.k_pages, c.v_pages, bt, c.seq_lens, 0, c.scale, out, None, st)
    torch.cuda.synchronize()
    assert st.tolist() == [1, 1, 2, 123456]
    da.decode_attn_static_scratch(c.q, c.k_pages, c.v_pages, c.block_table, c.seq_lens, 0, c.scale, out, None, st)
    torch.cuda.synchronize()
    assert st.tolist() == [0, 0, 0, 0]      # the record is per call

    B = 4097                                # one past the documented limit
    q = torch.zeros((B, 48, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_static_scratch(q, c.k_pages, c.v_pages, torch.zeros((B, 4), dtype=torch.int32, device="cuda"),
                                      torch.zeros(B, dtype=torch.int32, device="cuda"), 0, 1.0,
                                      torch.empty((B, 48, 128), device="cuda"))
    assert e.value.status == 6
    da.set_option("grid_blocks", 321)
    with pytest.raises(da.DecodeAttnError) as e:
        da.decode_attn_static_scratch(c.q, c.k_pages, c.v_pages, c.block_table, c.seq_lens, 0, c.scale, out)
    assert e.value.status == 6
    da.set_option("grid_blocks", 0)
