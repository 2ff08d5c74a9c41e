"""Pins for the oracle's 8-bit (E4M3) cache functions.

What fixes them, other than themselves:
  * the E4M3 format definition (FP8 Formats for Deep Learning, Sec. 3 / OCP 8-bit floating point
    specification): values written out by hand in golden/e4m3_values.txt, and torch's own
    float8_e4m3fn decoder as an independent library routine;
  * rounding: hand-worked ties and saturation cases, and torch's float32 -> float8_e4m3fn cast on
    random values inside the finite range;
  * the attention itself: on a cache whose codes are widened exactly to bf16 (every E4M3 value is a
    bf16 value) the 8-bit oracle must reproduce the pinned bf16 oracle bit for bit, power-of-two
    factors included; general factors are checked against a dense numpy/scipy brute force.
"""
import math
import os

import numpy as np
import pytest
import torch
from scipy.special import logsumexp, softmax

import oracle
import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def codes_to_f32(codes: np.ndarray) -> np.ndarray:
    """torch's decoder (library routine)."""
    return torch.from_numpy(np.ascontiguousarray(codes)).view(torch.float8_e4m3fn).to(torch.float32).numpy()


def tiny8(lens, P=4, seed=0, Hq=6, Hkv=2, Dh=8, **kw):
    return workloads.build_case("tiny8", lens, P, seed, "cpu", Hq=Hq, Hkv=Hkv, Dh=Dh, kv_dtype="fp8", **kw)


def run8(case, **kw):
    return oracle.decode_attn_fp8kv_oracle(case.q, case.k_pages, case.v_pages,
                                           kw.get("k_scale", case.k_scale), kw.get("v_scale", case.v_scale),
                                           case.block_table, case.seq_lens, kw.get("window", case.window),
                                           kw.get("scale", case.scale), kw.get("threads", 0))


# --------------------------------------------------------------------- the format

def test_e4m3_values_from_the_format_definition():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "e4m3_values.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) >= 16
    for code, value in rows:
        got = oracle.e4m3_value(int(code, 16))
        if value == "nan":
            assert math.isnan(got)
        else:
            want = float(eval(value, {"__builtins__": {}}))   # entries like 7*2**-9
            assert got == want and math.copysign(1.0, got) == math.copysign(1.0, want), (code, got, want)


def test_e4m3_table_equals_torch_decoder():
    codes = np.arange(256, dtype=np.uint8)
    mine = np.array([oracle.e4m3_value(int(c)) for c in codes])
    lib = codes_to_f32(codes).astype(np.float64)
    assert np.array_equal(np.isnan(mine), np.isnan(lib))
    ok = ~np.isnan(lib)
    assert np.array_equal(mine[ok], lib[ok])
    assert np.array_equal(np.signbit(mine[ok]), np.signbit(lib[ok]))
    # monotone in the code on the finite non-negative half (what the nearest-code search relies on)
    assert (np.diff(mine[:0x7F]) > 0).all()


def test_every_e4m3_value_is_a_bf16_value():
    codes = np.arange(256, dtype=np.uint8)
    v = torch.from_numpy(codes_to_f32(codes))
    ok = ~torch.isnan(v)
    assert torch.equal(v[ok].to(torch.bfloat16).to(torch.float32), v[ok])


# --------------------------------------------------------------------- rounding

def test_nearest_code_round_trip_ties_and_saturation():
    for code in range(256):
        if code & 0x7F == 0x7F:
            continue
        assert oracle.e4m3_nearest_code(oracle.e4m3_value(code)) == code
    # ties go to the even mantissa: 1.0625 lies midway between 1.0 (0x38) and 1.125 (0x39)
    assert oracle.e4m3_nearest_code(1.0625) == 0x38
    assert oracle.e4m3_nearest_code(1.1875) == 0x3A          # midway 1.125 (0x39) / 1.25 (0x3A)
    assert oracle.e4m3_nearest_code(-1.5 * 2 ** -9) == 0x82  # midway between -1 and -2 subnormal steps
    assert oracle.e4m3_nearest_code(0.5 * 2 ** -9) == 0x00   # midway 0 / smallest subnormal
    assert oracle.e4m3_nearest_code(np.nextafter(0.5 * 2 ** -9, 1.0)) == 0x01
    assert oracle.e4m3_nearest_code(1.0624) == 0x38 and oracle.e4m3_nearest_code(1.0626) == 0x39
    # saturation at the largest finite value, either sign; NaN
    assert oracle.e4m3_nearest_code(448.0) == 0x7E
    assert oracle.e4m3_nearest_code(1e9) == 0x7E and oracle.e4m3_nearest_code(-1e9) == 0xFE
    assert oracle.e4m3_nearest_code(float("inf")) == 0x7E
    assert oracle.e4m3_nearest_code(float("nan")) == 0x7F
    assert oracle.e4m3_nearest_code(-0.0) == 0x80


def test_quantiser_equals_torch_cast_inside_the_finite_range():
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 60, 4000), rng.uniform(-2 ** -5, 2 ** -5, 2000)])
    xb = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16)
    for scale in (1.0, 0.5, 0.0233, 3.7):
        y = xb.to(torch.float32) / np.float32(scale)                  # fp32 quotient, as the oracle states
        keep = (y.abs() <= 448.0)
        want = y.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
        got = oracle.e4m3_quantize(xb, scale)
        assert keep.sum() > 5000
        assert np.array_equal(got[keep.numpy()], want[keep.numpy()])
        big = ~keep.numpy()
        if big.any():   # beyond the range the oracle saturates, sign kept
            assert set(np.unique(got[big] & 0x7F)) == {0x7E}


def test_append_writes_quantised_rows_at_the_last_position():
    case = tiny8([9, 4, 1], P=4, seed=21)
    rng = torch.Generator().manual_seed(5)
    k_new = torch.randn((3, 2, 8), generator=rng).to(torch.bfloat16)
    v_new = torch.randn((3, 2, 8), generator=rng).to(torch.bfloat16)
    k0, v0 = case.k_pages.clone(), case.v_pages.clone()
    oracle.kv_append_fp8_oracle(k_new, v_new, case.k_pages, case.v_pages, case.k_scale, case.v_scale,
                                case.block_table, case.seq_lens)
    touched = torch.zeros_like(k0, dtype=torch.bool)
    for b, L in enumerate([9, 4, 1]):
        page, row = int(case.block_table[b, (L - 1) // 4]), (L - 1) % 4
        for g in range(2):
            # plain indexing plus torch's cast (library) on the fp32 quotient
            wk = (k_new[b, g].float() / case.k_scale[g]).to(torch.float8_e4m3fn).view(torch.uint8)
            wv = (v_new[b, g].float() / case.v_scale[g]).to(torch.float8_e4m3fn).view(torch.uint8)
            assert torch.equal(case.k_pages[page, g, row], wk)
            assert torch.equal(case.v_pages[page, g, row], wv)
        touched[page, :, row] = True
    assert torch.equal(case.k_pages[~touched], k0[~touched]) and torch.equal(case.v_pages[~touched], v0[~touched])


# --------------------------------------------------------------------- attention over the codes

def widened(case, k_mul=1.0, v_mul=1.0):
    """The same cache as bf16 tensors: code values times a power of two, exactly."""
    k = (torch.from_numpy(codes_to_f32(case.k_pages.numpy())) * k_mul).to(torch.bfloat16)
    v = (torch.from_numpy(codes_to_f32(case.v_pages.numpy())) * v_mul).to(torch.bfloat16)
    return k, v


@pytest.mark.parametrize("window", [0, 5])
def test_unit_factors_reproduce_the_bf16_oracle_bit_for_bit(window):
    case = tiny8([13, 1, 0, 22, 8], P=4, seed=31, poison=False)
    k, v = widened(case)
    want = oracle.decode_attn_oracle(case.q, k, v, case.block_table, case.seq_lens, window, case.scale)
    got = run8(case, k_scale=None, v_scale=None, window=window)
    ones = np.ones(2, np.float32)
    got1 = run8(case, k_scale=ones, v_scale=ones, window=window)
    for a, b_, c in zip(want, got, got1):
        assert np.array_equal(a, b_) and np.array_equal(a, c)


def test_power_of_two_factors_reproduce_the_bf16_oracle():
    case = tiny8([17, 6], P=4, seed=32, poison=False)
    ks, vs = np.array([0.25, 2.0], np.float32), np.array([0.5, 0.125], np.float32)
    # per-head exact scaling of the widened cache
    k = torch.from_numpy(codes_to_f32(case.k_pages.numpy())) * torch.from_numpy(ks).reshape(1, 2, 1, 1)
    v = torch.from_numpy(codes_to_f32(case.v_pages.numpy())) * torch.from_numpy(vs).reshape(1, 2, 1, 1)
    want = oracle.decode_attn_oracle(case.q, k.to(torch.bfloat16), v.to(torch.bfloat16), case.block_table,
                                     case.seq_lens, 0, case.scale)
    got = run8(case, k_scale=ks, v_scale=vs)
    np.testing.assert_allclose(got[0], want[0], rtol=1e-14, atol=0)
    np.testing.assert_allclose(got[1], want[1], rtol=1e-14, atol=1e-14)


@pytest.mark.parametrize("layout", ["head_major", "token_major"])
@pytest.mark.parametrize("P,window", [(4, 0), (16, 0), (4, 7)])
def test_general_factors_against_dense_bruteforce(layout, P, window):
    case = tiny8([33, 1, 70, 0, 16], P=P, seed=40 + P, layout=layout)
    got, got_lse = run8(case, window=window)
    scale = float(np.float32(case.scale))
    q = case.q.to(torch.float64).numpy()
    K = codes_to_f32(np.ascontiguousarray(case.k_pages.numpy())).astype(np.float64)
    V = codes_to_f32(np.ascontiguousarray(case.v_pages.numpy())).astype(np.float64)
    K = K * case.k_scale.numpy().astype(np.float64).reshape(1, 2, 1, 1)
    V = V * case.v_scale.numpy().astype(np.float64).reshape(1, 2, 1, 1)
    bt = case.block_table.numpy()
    for b, L in enumerate([33, 1, 70, 0, 16]):
        if L == 0:
            assert (got[b] == 0).all() and np.isneginf(got_lse[b]).all()
            continue
        lo = L - window if 0 < window < L else 0
        t = np.arange(lo, L)
        for h in range(6):
            Kd, Vd = K[bt[b, t // P], h // 3, t % P], V[bt[b, t // P], h // 3, t % P]
            s = scale * (Kd @ q[b, h])
            np.testing.assert_allclose(got[b, h], softmax(s) @ Vd, rtol=1e-12, atol=1e-13)
            assert got_lse[b, h] == pytest.approx(logsumexp(s), abs=1e-12)


def test_single_token_returns_dequantised_v():
    case = tiny8([1, 1], P=4, seed=50)
    out, lse = run8(case)
    for b in range(2):
        page = int(case.block_table[b, 0])
        for h in range(6):
            g = h // 3
            v = codes_to_f32(case.v_pages[page, g, 0].numpy()).astype(np.float64) * float(case.v_scale[g])
            assert np.array_equal(out[b, h], v)


def test_nan_codes_outside_the_attended_range_do_not_matter():
    case = tiny8([10, 7], P=4, seed=51, pool_pages=12, poison=True)
    clean = tiny8([10, 7], P=4, seed=51, pool_pages=12, poison=False)
    assert (case.k_pages == workloads.E4M3_NAN).any()
    a, b_ = run8(case), run8(clean)
    assert np.isfinite(a[0]).all() and np.array_equal(a[0], b_[0]) and np.array_equal(a[1], b_[1])


def test_planted_slips_are_seen():
    """A wrong bias, a dropped factor and K/V factors swapped each change the result measurably."""
    case = tiny8([19], P=4, seed=60)
    base, base_lse = run8(case)
    swapped = run8(case, k_scale=case.v_scale, v_scale=case.k_scale)
    no_v = run8(case, v_scale=None)
    assert np.abs(swapped[0] - base).max() > 1e-3
    assert np.abs(no_v[0] - base).max() > 1e-2
    # bias 8 instead of 7 would halve every K: emulate by halving k_scale
    half = run8(case, k_scale=case.k_scale * 0.5)
    assert np.abs(half[1] - base_lse).max() > 1e-2


def test_extend_over_codes_reproduces_the_bf16_extend_oracle():
    """Unit factors and a cache widened exactly to bf16: the causal multi-token oracle over codes must equal the
    (separately pinned) bf16 one bit for bit."""
    case = tiny8([13, 4, 0, 22], P=4, seed=71, poison=False)
    q = torch.randn((4, 3, 6, 8), generator=torch.Generator().manual_seed(3)).to(torch.bfloat16)
    lens = np.where(case.seq_lens.numpy() > 0, np.maximum(case.seq_lens.numpy(), 3), 0)
    assert (lens == case.seq_lens.numpy()).all()
    k, v = widened(case)
    want = oracle.extend_attn_oracle(q, k, v, case.block_table, case.seq_lens, case.scale)
    got = oracle.extend_attn_fp8kv_oracle(q, case.k_pages, case.v_pages, None, None, case.block_table, case.seq_lens,
                                          case.scale)
    assert np.array_equal(want[0], got[0]) and np.array_equal(want[1], got[1])
