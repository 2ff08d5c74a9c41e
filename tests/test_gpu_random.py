"""Seeded random sweep over the entry points: shapes, lengths, page sizes, group sizes, windows, layouts
and split schedules drawn at random, every result compared with the fp64 oracle (fp32 bar:
|d| <= 1e-3 + 1e-3 |ref|).  The fixed tests pick their edge cases by hand; this one looks where nobody
thought to."""
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
    yield pkg
    pkg.set_option("grid_blocks", 0)
    pkg.set_option("tail_units", 4)
    pkg.set_option("static_frac", 224)


def _draw(rng):
    B = int(rng.integers(1, 9))
    P = int(rng.choice([16, 32, 64, 128]))
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 6, 8, 12, 16]))
    maxL = int(rng.choice([40, 300, 1500, 6000]))
    lens = rng.integers(0, maxL, size=B)
    lens[rng.integers(0, B)] = maxL
    return dict(B=B, P=P, Hkv=Hkv, Hq=Hkv * G, lens=lens, maxL=maxL,
                window=int(rng.choice([0, 0, 1, 17, 64, 200, 5000])),
                grid=int(rng.choice([0, 0, 1, 3, 50, 296, 2000])), tail=int(rng.choice([0, 1, 4, 9])),
                frac=int(rng.choice([0, 128, 224, 256])), layout=str(rng.choice(["head_major", "token_major"])),
                seed=int(rng.integers(1 << 30)))


@pytest.mark.parametrize("kind,chunk", [(k, c) for k in ("bf16", "fp8", "extend", "cascade") for c in range(3)])
def test_random_cases_match_the_oracle(da, kind, chunk):
    rng = np.random.default_rng(1000 * chunk + {"bf16": 1, "fp8": 2, "extend": 3, "cascade": 4}[kind])
    for _ in range(12):
        c = _draw(rng)
        da.set_option("grid_blocks", c["grid"])
        da.set_option("tail_units", c["tail"])
        da.set_option("static_frac", c["frac"])
        what = f"{kind} {c}"
        kw = dict(Hq=c["Hq"], Hkv=c["Hkv"], layout=c["layout"], poison=True)
        if kind in ("bf16", "fp8"):
            case = workloads.build_case("rnd", c["lens"], c["P"], c["seed"], "cpu", window=c["window"], kv_dtype=kind, **kw)
            dev = workloads.to_device(case, "cuda")
            if kind == "bf16":
                ref, ref_lse = oracle.decode_attn_oracle(case.q, case.k_pages, case.v_pages, case.block_table,
                                                         case.seq_lens, case.window, case.scale)
                out, lse = da.decode_attn(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, dev.window, dev.scale)
            else:
                ref, ref_lse = oracle.decode_attn_fp8kv_oracle(case.q, case.k_pages, case.v_pages, case.k_scale, case.v_scale,
                                                               case.block_table, case.seq_lens, case.window, case.scale)
                out, lse = da.decode_attn_fp8kv(dev.q, dev.k_pages, dev.v_pages, dev.k_scale, dev.v_scale, dev.block_table,
                                                dev.seq_lens, dev.window, dev.scale)
        elif kind == "extend":
            Lq = int(rng.choice([1, 2, 3, 7, 40, 150]))
            lens = np.where(c["lens"] > 0, np.maximum(c["lens"], Lq), 0)
            case = workloads.build_case("rnd", lens, c["P"], c["seed"], "cpu", **kw)
            q = torch.randn((c["B"], Lq, c["Hq"], 128), generator=torch.Generator().manual_seed(c["seed"])).to(torch.bfloat16)
            ref, ref_lse = oracle.extend_attn_oracle(q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, case.scale)
            dev = workloads.to_device(case, "cuda")
            out, lse = da.decode_attn_extend(q.cuda(), dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, dev.scale)
            what += f" Lq={Lq}"
        else:
            prefix = int(rng.choice([128, 256, 1024]))
            lens = prefix + rng.integers(0, c["maxL"], size=c["B"])
            case = workloads.build_case("rnd", lens, c["P"], c["seed"], "cpu", Hq=c["Hq"], Hkv=c["Hkv"],
                                        shared_prefix_tokens=prefix, poison=True)
            ref, ref_lse = oracle.decode_attn_oracle(case.q, case.k_pages, case.v_pages, case.block_table,
                                                     case.seq_lens, 0, case.scale)
            dev = workloads.to_device(case, "cuda")
            out, lse = da.decode_attn_cascade(dev.q, dev.k_pages, dev.v_pages, dev.block_table, dev.seq_lens, prefix, dev.scale)
            what += f" prefix={prefix}"
        assert da.read_device_status() == (0, 0, 0, 0), what
        assert_close(out.cpu().numpy(), ref, what + " out")
        assert_close(lse.cpu().numpy(), ref_lse, what + " lse")
