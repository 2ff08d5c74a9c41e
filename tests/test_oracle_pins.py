"""Pins for the fp64 CPU oracle: closed forms, invariants and an independent dense
brute force.  Nothing here asks the oracle about itself only: each test compares
it with a value fixed by the mathematics of softmax attention (the operation the
FlashAttention papers cited in the paper's related work compute exactly), by a
library routine (scipy softmax / logsumexp on dense gathered K, V) or by
exact-rational arithmetic."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
from scipy.special import logsumexp, softmax

import oracle
import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf(x):
    """float array -> torch bf16 CPU tensor (round to nearest even)."""
    return torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)


def f64(t):
    return t.to(torch.float64).numpy()


def run(case, **kw):
    return oracle.decode_attn_oracle(case.q, case.k_pages, case.v_pages, case.block_table,
                                     case.seq_lens, kw.get("window", case.window),
                                     kw.get("scale", case.scale), kw.get("threads", 0))


def tiny(lens, P=4, seed=0, Hq=6, Hkv=2, Dh=8, **kw):
    return workloads.build_case("tiny", lens, P, seed, "cpu", Hq=Hq, Hkv=Hkv, Dh=Dh, **kw)


def dense_bruteforce(case, window=None, scale=None):
    """Independent restatement: gather each sequence's tokens into dense K, V
    with fancy indexing, then softmax / logsumexp from scipy."""
    window = case.window if window is None else window
    scale = float(np.float32(case.scale if scale is None else scale))
    q, K, V = f64(case.q), f64(case.k_pages), f64(case.v_pages)
    bt = case.block_table.numpy()
    B, Hq, Dh = q.shape
    Hkv, P = K.shape[1], K.shape[2]
    G = Hq // Hkv
    out = np.zeros((B, Hq, Dh))
    lse = np.full((B, Hq), -np.inf)
    for b in range(B):
        L = int(case.seq_lens[b])
        if L <= 0:
            continue
        lo = L - window if 0 < window < L else 0
        t = np.arange(lo, L)
        pages, rows = bt[b, t // P], t % P
        for h in range(Hq):
            Kd = K[pages, h // G, rows, :]          # [n, D]
            Vd = V[pages, h // G, rows, :]
            s = scale * (Kd @ q[b, h])
            out[b, h] = softmax(s) @ Vd
            lse[b, h] = logsumexp(s)
    return out, lse


# --------------------------------------------------------------------- closed forms

def test_single_token_returns_v_and_exact_lse():
    case = tiny([1, 1, 1], P=4, seed=3)
    out, lse = run(case)
    for b in range(3):
        page = int(case.block_table[b, 0])
        for h in range(6):
            g = h // 3
            assert np.array_equal(out[b, h], f64(case.v_pages[page, g, 0]))
            # exact rational q.k, then one rounding
            qk = sum(Fraction(float(a)) * Fraction(float(c))
                     for a, c in zip(case.q[b, h].tolist(), case.k_pages[page, g, 0].tolist()))
            want = float(Fraction(float(np.float32(case.scale))) * qk)
            assert lse[b, h] == pytest.approx(want, rel=1e-14, abs=1e-300)


def test_identical_keys_give_mean_of_v():
    case = tiny([13, 7], P=4, seed=5)
    krow = case.k_pages[int(case.block_table[0, 0]), :, 0:1, :].clone()
    case.k_pages[:] = krow.expand(-1, 4, -1)[None]
    out, lse = run(case)
    V, bt = f64(case.v_pages), case.block_table.numpy()
    for b, L in enumerate([13, 7]):
        t = np.arange(L)
        for h in range(6):
            mean = V[bt[b, t // 4], h // 3, t % 4].mean(0)
            np.testing.assert_allclose(out[b, h], mean, rtol=0, atol=1e-14)
            s = float(np.float32(case.scale)) * float(f64(case.q[b, h]) @ f64(krow[h // 3, 0]))
            assert lse[b, h] == pytest.approx(s + math.log(L), abs=1e-12)


def test_scale_zero_gives_mean_and_log_n():
    case = tiny([9, 16, 3], P=4, seed=6)
    out, lse = run(case, scale=0.0)
    V, bt = f64(case.v_pages), case.block_table.numpy()
    for b, L in enumerate([9, 16, 3]):
        t = np.arange(L)
        for h in range(6):
            np.testing.assert_allclose(out[b, h], V[bt[b, t // 4], h // 3, t % 4].mean(0), atol=1e-14)
            assert lse[b, h] == pytest.approx(math.log(L), abs=1e-14)


def test_two_token_closed_form_from_golden():
    """scores ln1, ln3 -> weights 1/4, 3/4; lse = ln 4 (golden/two_token_ln3.txt)."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "two_token_ln3.txt")) if l.strip() and l[0] != "#"]
    vals = {r[0]: [float(x) for x in r[1:]] for r in rows}
    Dh = 8
    q = np.zeros((1, 1, Dh)); q[0, 0, 0] = 1.0
    K = np.zeros((1, 1, 2, Dh)); K[0, 0, 1, 0] = 1.0
    V = np.zeros((1, 1, 2, Dh)); V[0, 0, 0] = vals["v0"]; V[0, 0, 1] = vals["v1"]
    # the score ln 3 enters through the scale, which the interface takes in fp32 (error < 3e-8)
    out, lse = oracle.decode_attn_oracle(bf(q), bf(K), bf(V), np.array([[0]], np.int32),
                                         np.array([2], np.int32), 0, vals["scale"][0])
    np.testing.assert_allclose(out[0, 0], vals["out_ideal"], atol=1e-6)
    assert lse[0, 0] == pytest.approx(vals["lse_ideal"][0], abs=1e-7)


def test_dominant_score_returns_that_tokens_v():
    case = tiny([37], P=4, seed=7, Hq=4, Hkv=2, Dh=8)
    t_star = 22
    page = int(case.block_table[0, t_star // 4])
    # k* = 64 * q for each group's first head; gap in score >= 200 against N(0,1) keys
    for g in range(2):
        case.k_pages[page, g, t_star % 4] = (case.q[0, 2 * g].float() * 64).to(torch.bfloat16)
        case.q[0, 2 * g + 1] = case.q[0, 2 * g]
    out, lse = run(case, scale=1.0)
    q64 = f64(case.q)
    assert (q64[0] ** 2).sum(-1).min() * 64 > 250
    for h in range(4):
        v = f64(case.v_pages[page, h // 2, t_star % 4])
        assert np.array_equal(out[0, h].astype(np.float32), v.astype(np.float32))
        s = float(q64[0, h] @ f64(case.k_pages[page, h // 2, t_star % 4]))
        assert lse[0, h] == pytest.approx(s, abs=1e-9)


def test_huge_score_offsets_stay_finite():
    case = tiny([20], P=4, seed=8, Hq=2, Hkv=1, Dh=8)
    base_out, base_lse = run(case, scale=1.0)
    # add a constant c to every score through an extra coordinate: q_7 = 1, k_7 = c
    for c in (1.0e4, -1.0e4):
        shifted = tiny([20], P=4, seed=8, Hq=2, Hkv=1, Dh=8)
        q0 = shifted.q.clone(); q0[..., 7] = 0; q0[..., 6] = 0
        shifted.q[:] = q0
        ref_out, ref_lse = run(shifted, scale=1.0)
        shifted.q[..., 7] = 1.0
        shifted.k_pages[..., 7] = c        # bf16(1e4) = 9984, exactly representable steps
        out, lse = run(shifted, scale=1.0)
        cc = float(shifted.k_pages[0, 0, 0, 7])
        assert np.isfinite(out).all() and np.isfinite(lse).all()
        np.testing.assert_allclose(out, ref_out, atol=1e-9)
        np.testing.assert_allclose(lse, ref_lse + cc, atol=1e-8)
    assert np.isfinite(base_out).all() and np.isfinite(base_lse).all()


def test_empty_sequence_is_zero_and_minus_inf():
    case = tiny([0, 5, 0], P=4, seed=9)
    out, lse = run(case)
    assert np.all(out[0] == 0) and np.all(out[2] == 0)
    assert np.all(np.isneginf(lse[0])) and np.all(np.isneginf(lse[2]))
    assert np.isfinite(out[1]).all() and np.isfinite(lse[1]).all()


# --------------------------------------------------------------------- invariants

def test_page_permutation_is_bit_identical():
    lens = [33, 1, 18, 64]
    a = tiny(lens, P=8, seed=11, shuffle=False, poison=False)
    out_a, lse_a = run(a)
    perm = np.random.default_rng(1).permutation(a.k_pages.shape[0])
    inv = np.argsort(perm)
    b_k = a.k_pages[torch.from_numpy(perm)]      # new page i holds old page perm[i]
    b_v = a.v_pages[torch.from_numpy(perm)]
    bt = a.block_table.numpy().copy()
    bt[bt >= 0] = inv[bt[bt >= 0]]
    out_b, lse_b = oracle.decode_attn_oracle(a.q, b_k, b_v, bt, a.seq_lens, 0, a.scale)
    assert np.array_equal(out_a, out_b) and np.array_equal(lse_a, lse_b)
    # and a shuffled build of the same recipe agrees with brute force on its own table
    c = tiny(lens, P=8, seed=11, shuffle=True)
    np.testing.assert_allclose(run(c)[0], dense_bruteforce(c)[0], atol=1e-12)


def test_token_major_layout_equals_head_major():
    a = tiny([29, 12], P=4, seed=12, layout="head_major", poison=False)
    k2 = a.k_pages.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    v2 = a.v_pages.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert k2.stride() != a.k_pages.stride()
    out_a, lse_a = run(a)
    out_b, lse_b = oracle.decode_attn_oracle(a.q, k2, v2, a.block_table, a.seq_lens, 0, a.scale)
    assert np.array_equal(out_a, out_b) and np.array_equal(lse_a, lse_b)


def test_gqa_head_mapping():
    case = tiny([21], P=4, seed=13, Hq=12, Hkv=3, Dh=8)   # G = 4
    # V of KV head g is the constant g+1, K = 0  ->  out[h] = h//4 + 1 exactly
    case.k_pages[:] = 0
    for g in range(3):
        case.v_pages[:, g] = g + 1
    out, _ = run(case)
    for h in range(12):
        np.testing.assert_allclose(out[0, h], h // 4 + 1, atol=1e-15)
    # NaN in the other KV heads never reaches head h
    case2 = tiny([21], P=4, seed=13, Hq=12, Hkv=3, Dh=8, poison=False)
    ref, ref_lse = run(case2)
    for g in range(3):
        k, v = case2.k_pages.clone(), case2.v_pages.clone()
        others = [x for x in range(3) if x != g]
        k[:, others] = float("nan"); v[:, others] = float("nan")
        o, l = oracle.decode_attn_oracle(case2.q, k, v, case2.block_table, case2.seq_lens, 0, case2.scale)
        hs = slice(4 * g, 4 * g + 4)
        assert np.array_equal(o[0, hs], ref[0, hs]) and np.array_equal(l[0, hs], ref_lse[0, hs])
    # heads of one group with the same q give the same row
    case2.q[0, 5] = case2.q[0, 4]
    o, l = run(case2)
    assert np.array_equal(o[0, 4], o[0, 5]) and l[0, 4] == l[0, 5]


def test_nan_canaries_never_reach_the_output():
    lens = [5, 17, 30]
    clean = tiny(lens, P=8, seed=14, poison=False)
    dirty = tiny(lens, P=8, seed=14, poison=True, pool_pages=20, pad_table_to=9)
    assert torch.isnan(dirty.k_pages).any()
    out_c, lse_c = run(clean)
    out_d, lse_d = run(dirty)
    assert np.isfinite(out_d).all() and np.isfinite(lse_d).all()
    # same seed and order of draws -> same values on referenced tokens
    np.testing.assert_allclose(out_d, dense_bruteforce(dirty)[0], atol=1e-12)
    assert out_c.shape == out_d.shape and np.isfinite(out_c).all() and np.isfinite(lse_c).all()


# --------------------------------------------------------------------- window

@pytest.mark.parametrize("P", [4, 16])
def test_window_identities(P):
    lens = [23, 40, 8, 1]
    case = tiny(lens, P=P, seed=15)
    full, full_lse = run(case, window=0)
    for W in (max(lens), max(lens) + 1, 10 ** 6, -3):
        o, l = run(case, window=W)
        assert np.array_equal(o, full) and np.array_equal(l, full_lse)
    # W = 1: the current token alone
    o1, l1 = run(case, window=1)
    V, K, q, bt = f64(case.v_pages), f64(case.k_pages), f64(case.q), case.block_table.numpy()
    for b, L in enumerate(lens):
        pg, r = bt[b, (L - 1) // P], (L - 1) % P
        for h in range(6):
            assert np.array_equal(o1[b, h], V[pg, h // 3, r])
            assert l1[b, h] == pytest.approx(float(np.float32(case.scale)) * float(q[b, h] @ K[pg, h // 3, r]), abs=1e-13)


@pytest.mark.parametrize("W", [1, 3, 4, 5, 7, 16, 17, 22])
def test_window_equals_full_attention_on_truncated_cache(W):
    P, lens = 4, [23, 9, 17]
    case = tiny(lens, P=P, seed=16, shuffle=False, poison=False)
    out_w, lse_w = run(case, window=W)
    K, V, bt = case.k_pages, case.v_pages, case.block_table.numpy()
    # rebuild each sequence as a fresh cache holding only its last min(W, L) tokens
    n = [min(W, L) for L in lens]
    npg = [(x + P - 1) // P for x in n]
    k2 = torch.zeros((sum(npg), 2, P, 8), dtype=torch.bfloat16)
    v2 = torch.zeros_like(k2)
    bt2 = np.full((3, max(npg)), -1, np.int32)
    cur = 0
    for b, L in enumerate(lens):
        for i in range(n[b]):
            t = L - n[b] + i
            src = (int(bt[b, t // P]), slice(None), t % P)
            k2[cur + i // P, :, i % P] = K[src]
            v2[cur + i // P, :, i % P] = V[src]
        bt2[b, :npg[b]] = np.arange(cur, cur + npg[b])
        cur += npg[b]
    out_t, lse_t = oracle.decode_attn_oracle(case.q, k2, v2, bt2, np.array(n, np.int32), 0, case.scale)
    assert np.array_equal(out_w, out_t) and np.array_equal(lse_w, lse_t)


# --------------------------------------------------------------------- split / merge algebra

@pytest.mark.parametrize("mid", [1, 8, 13, 31, 49])
def test_split_and_lse_merge_reproduces_the_whole(mid):
    """The log-sum-exp merge of two disjoint token ranges equals attention over their union."""
    L, P = 50, 8
    case = tiny([L], P=P, seed=17)
    whole, whole_lse = run(case)
    # [0, mid): a cache cut at mid;   [mid, L): the last L-mid tokens
    cut = tiny([L], P=P, seed=17)
    o1, l1 = oracle.decode_attn_oracle(cut.q, cut.k_pages, cut.v_pages, cut.block_table,
                                       np.array([mid], np.int32), 0, cut.scale)
    o2, l2 = run(case, window=L - mid)
    M = np.maximum(l1, l2)
    w1, w2 = np.exp(l1 - M), np.exp(l2 - M)
    merged = (w1[..., None] * o1 + w2[..., None] * o2) / (w1 + w2)[..., None]
    np.testing.assert_allclose(merged, whole, atol=1e-12)
    np.testing.assert_allclose(M + np.log(w1 + w2), whole_lse, atol=1e-12)


# --------------------------------------------------------------------- brute force

@pytest.mark.parametrize("P", [4, 16])
@pytest.mark.parametrize("window", [0, 5, 33])
@pytest.mark.parametrize("layout", ["head_major", "token_major"])
def test_dense_bruteforce_agrees(P, window, layout):
    case = workloads.build_case("bf", [70, 1, 37], P, 21 + P + window, "cpu", Hq=12, Hkv=3, Dh=16,
                                window=window, layout=layout, pool_pages=40, pad_table_to=20)
    out, lse = run(case)
    ref, ref_lse = dense_bruteforce(case)
    np.testing.assert_allclose(out, ref, atol=1e-12, rtol=0)
    np.testing.assert_allclose(lse, ref_lse, atol=1e-12, rtol=0)


def test_bruteforce_on_the_stability_config():
    case = workloads.c1()
    out, lse = run(case)
    ref, ref_lse = dense_bruteforce(case)
    np.testing.assert_allclose(out, ref, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, atol=1e-11)
    assert np.abs(lse).max() > 30          # the x20 keys really dominate


def test_thread_count_does_not_change_bits():
    case = tiny([45, 3, 60, 17], P=8, seed=23)
    a = run(case, threads=1)
    b = run(case, threads=5)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


# --------------------------------------------------------------------- planted mistakes

def test_pins_catch_planted_mistakes():
    """Each plausible slip, planted in a *copy* of the brute force, is seen by a pin's comparison."""
    case = workloads.build_case("m", [23, 9], 4, 31, "cpu", Hq=6, Hkv=2, Dh=8, window=5)
    good, good_lse = run(case)

    def variant(lo_shift=0, head_map=None, drop_scale=False, drop_max=False):
        q, K, V = f64(case.q), f64(case.k_pages), f64(case.v_pages)
        bt = case.block_table.numpy()
        out = np.zeros_like(good); lse = np.zeros_like(good_lse)
        for b, L in enumerate([23, 9]):
            lo = max(L - 5 + lo_shift, 0)
            t = np.arange(lo, L)
            for h in range(6):
                g = head_map(h) if head_map else h // 3
                Kd, Vd = K[bt[b, t // 4], g, t % 4], V[bt[b, t // 4], g, t % 4]
                s = (1.0 if drop_scale else float(np.float32(case.scale))) * (Kd @ q[b, h])
                out[b, h] = softmax(s) @ Vd
                lse[b, h] = np.log(np.exp(s).sum()) if drop_max else logsumexp(s)
        return out, lse

    assert np.allclose(variant()[0], good, atol=1e-12)
    assert not np.allclose(variant(lo_shift=1)[0], good, atol=1e-6)       # window off by one
    assert not np.allclose(variant(lo_shift=-1)[0], good, atol=1e-6)
    assert not np.allclose(variant(head_map=lambda h: h % 2)[0], good, atol=1e-6)  # interleaved GQA
    assert not np.allclose(variant(drop_scale=True)[1], good_lse, atol=1e-6)


# --------------------------------------------------------------------- KV append

@pytest.mark.parametrize("layout", ["head_major", "token_major"])
def test_kv_append_writes_exactly_the_new_rows(layout):
    """Pinned by plain indexing: after the call the row (page of token L-1, L-1 mod P) of every KV
    head holds the new vectors and every other element of the pools is untouched."""
    lens = [5, 8, 0, 13, 1]
    case = tiny(lens, P=4, seed=41, Hq=6, Hkv=2, Dh=8, layout=layout, pool_pages=12, poison=False)
    k0, v0 = case.k_pages.clone(), case.v_pages.clone()
    gen = torch.Generator().manual_seed(3)
    k_new = torch.randn((5, 2, 8), generator=gen).to(torch.bfloat16)
    v_new = torch.randn((5, 2, 8), generator=gen).to(torch.bfloat16)
    oracle.kv_append_oracle(k_new, v_new, case.k_pages, case.v_pages, case.block_table, case.seq_lens)
    want_k, want_v = k0.clone(), v0.clone()
    bt = case.block_table.numpy()
    for b, L in enumerate(lens):
        if L > 0:
            pg, r = int(bt[b, (L - 1) // 4]), (L - 1) % 4
            want_k[pg, :, r] = k_new[b]
            want_v[pg, :, r] = v_new[b]
    assert torch.equal(case.k_pages.view(torch.int16), want_k.view(torch.int16))
    assert torch.equal(case.v_pages.view(torch.int16), want_v.view(torch.int16))
    # and decode attention over the updated cache sees the new token: with window 1 it returns v_new
    out, _ = run(case, window=1)
    for b, L in enumerate(lens):
        if L > 0:
            for h in range(6):
                assert np.array_equal(out[b, h], f64(v_new[b, h // 3]))


# --------------------------------------------------------------------- multi-token (extend) attention

@pytest.mark.parametrize("P,Lq", [(4, 1), (4, 3), (16, 7)])
def test_extend_oracle_agrees_with_dense_causal_bruteforce(P, Lq):
    """Independent restatement: gather dense K, V per sequence, build the causal mask explicitly
    (query qi sees tokens <= L - Lq + qi), scipy softmax."""
    lens = [Lq, Lq + 5, 40, 23]
    case = workloads.build_case("ext", lens, P, 50 + P + Lq, "cpu", Hq=6, Hkv=2, Dh=8)
    gen = torch.Generator().manual_seed(Lq)
    q = torch.randn((4, Lq, 6, 8), generator=gen).to(torch.bfloat16)
    out, lse = oracle.extend_attn_oracle(q, case.k_pages, case.v_pages, case.block_table, case.seq_lens, case.scale)
    K, V, bt = f64(case.k_pages), f64(case.v_pages), case.block_table.numpy()
    qd = f64(q)
    sc = float(np.float32(case.scale))
    for b, L in enumerate(lens):
        t = np.arange(L)
        for h in range(6):
            Kd, Vd = K[bt[b, t // P], h // 3, t % P], V[bt[b, t // P], h // 3, t % P]
            s = sc * (qd[b, :, h] @ Kd.T)                                  # [Lq, L]
            mask = t[None, :] <= (L - Lq + np.arange(Lq))[:, None]
            s = np.where(mask, s, -np.inf)
            np.testing.assert_allclose(out[b, :, h], softmax(s, axis=1) @ Vd, atol=1e-12)
            np.testing.assert_allclose(lse[b, :, h], logsumexp(s, axis=1), atol=1e-12)
    # Lq = 1 is plain decode attention
    if Lq == 1:
        o1, l1 = run(case)
        o2, l2 = oracle.extend_attn_oracle(case.q[:, None], case.k_pages, case.v_pages, case.block_table, case.seq_lens, case.scale)
        assert np.array_equal(o1, o2[:, 0]) and np.array_equal(l1, l2[:, 0])
