"""Pins for the CPU oracle: it is checked against things other than itself --
an integer reference, exact rational arithmetic, numpy's dense matmul, the
textbook rotary embedding, invariants and closed forms.  CPU only."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2512_03383_b200 import synth


def _small_q(rng, N, K, symmetric=False):
    qw = synth.draw_qweight(rng, N, K, symmetric=symmetric)
    return qw, oracle.pack_u4(qw.codes)


# 1 ---------------------------------------------------------------- unpack / dequant, integer exact
def test_low_nibble_first_literal():
    # byte 0xA3 holds input channel 2b in its low nibble (3) and 2b+1 in its high nibble (10)
    packed = np.array([[0xA3, 0x0F]], dtype=np.uint8)
    assert oracle.unpack_u4(packed).tolist() == [[3, 10, 15, 0]]
    assert oracle.pack_u4(np.array([[3, 10, 15, 0]], dtype=np.uint8)).tolist() == [[0xA3, 0x0F]]


def test_unpack_all_bytes_against_divmod():
    packed = np.arange(256, dtype=np.uint8).reshape(2, 128)
    codes = oracle.unpack_u4(packed)
    ref = np.empty((2, 256), dtype=np.uint8)
    for n in range(2):
        for b in range(128):
            hi, lo = divmod(int(packed[n, b]), 16)
            ref[n, 2 * b], ref[n, 2 * b + 1] = lo, hi
    assert np.array_equal(codes, ref)
    assert np.array_equal(oracle.pack_u4(codes), packed)


def test_pack_rejects_bad_codes():
    with pytest.raises(ValueError):
        oracle.pack_u4(np.array([[16, 0]], dtype=np.uint8))


def test_dequant_exact_rational():
    rng = np.random.default_rng(11)
    qw, packed = _small_q(rng, 3, 256)
    w = oracle.dequant(packed, qw.scales, qw.zeros)
    for n in range(3):
        for k in range(256):
            s = Fraction(float(qw.scales[n, k // 128]))
            z = int(qw.zeros[n, k // 128])
            assert float(qw.zeros[n, k // 128]) == z
            exact = s * (int(qw.codes[n, k]) - z)       # integer subtraction, then scale
            assert Fraction(w[n, k]) == exact           # s*(small int) is exact in fp64


def test_dequant_noninteger_zero_and_group_boundary():
    codes = np.zeros((1, 256), dtype=np.uint8)
    codes[0, 127], codes[0, 128] = 5, 5
    s = np.array([[0.5, 2.0]], dtype=np.float16)
    z = np.array([[1.25, 7.5]], dtype=np.float16)
    w = oracle.dequant(oracle.pack_u4(codes), s, z)
    assert w[0, 127] == 0.5 * (5 - 1.25) and w[0, 128] == 2.0 * (5 - 7.5)
    assert w[0, 0] == 0.5 * (0 - 1.25) and w[0, 255] == 2.0 * (0 - 7.5)


def test_symmetric_case_is_the_papers_equation():
    # Section 3.4: Wbar = clamp(round(W/s), -8, 7), s = max|W|/7  ->  dequant = s*Wbar
    rng = np.random.default_rng(5)
    W = synth.draw_weight(rng, 4, 256)
    codes, s16, z16 = synth.quantize_sym_u4(W)
    w = oracle.dequant(oracle.pack_u4(codes), s16, z16)
    sd = s16.astype(np.float64)
    for n in range(4):
        for g in range(2):
            blk = W[n, g * 128:(g + 1) * 128].astype(np.float64)
            wbar = np.clip(np.rint(blk / sd[n, g]), -8, 7)
            assert np.array_equal(w[n, g * 128:(g + 1) * 128], sd[n, g] * wbar)
    assert np.abs(w - W).max() <= 0.5 * sd.max() + 1e-12    # within half a quantisation step


# 2, 3 ------------------------------------------------------------- dense matmul / slicing
def test_keep_rate_one_equals_dense_matmul():
    rng = np.random.default_rng(0)
    qw, packed = _small_q(rng, 96, 384)
    x = synth.draw_x(rng, 5, 384, "f16", outlier_frac=0.02)
    W = oracle.dequant(packed, qw.scales, qw.zeros)
    acc = oracle.qlinear(x, packed, qw.scales, qw.zeros, oracle.leading(96), oracle.leading(384))
    ref = x.astype(np.float64) @ W.T
    assert np.allclose(acc, ref, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("k_out,k_in", [(96, 384), (80, 324), (4, 4), (52, 128), (96, 132)])
def test_truncation_equals_slicing(k_out, k_in):
    rng = np.random.default_rng(1)
    qw, packed = _small_q(rng, 96, 384)
    x = synth.draw_x(rng, 3, k_in, "f16")
    W = oracle.dequant(packed, qw.scales, qw.zeros)
    acc = oracle.qlinear(x, packed, qw.scales, qw.zeros, oracle.leading(k_out), oracle.leading(k_in))
    ref = x.astype(np.float64) @ W[:k_out, :k_in].T
    assert acc.shape == (3, k_out)
    assert np.allclose(acc, ref, rtol=1e-12, atol=1e-12)


def test_expand_map_literal():
    assert oracle.expand_map([(0, 8, 3, 2)]).tolist() == [0, 1, 2, 8, 9, 10]
    assert oracle.expand_map([(4, 4, 2, 2), (20, 1, 1, 1)]).tolist() == [4, 5, 8, 9, 20]
    # symmetric-sorted head of dim 8 truncated to 4: rows {0,1} of the low half, {4,5} of the high half
    assert oracle.expand_map(oracle.qk_halfhead_map(2, 8, 4)).tolist() == [0, 1, 4, 5, 8, 9, 12, 13]


def test_segmented_maps_equal_fancy_slicing():
    rng = np.random.default_rng(2)
    qw, packed = _small_q(rng, 128, 512)
    O = oracle.expand_map([(0, 32, 20, 2), (64, 64, 64, 1)])        # two pruned heads + a dense block
    I = oracle.expand_map([(0, 64, 44, 8)])                         # per-head input pruning
    x = synth.draw_x(rng, 4, len(I), "f16")
    bias = rng.standard_normal(128)
    W = oracle.dequant(packed, qw.scales, qw.zeros)
    acc = oracle.qlinear(x, packed, qw.scales, qw.zeros, O, I, bias=bias)
    ref = x.astype(np.float64) @ W[np.ix_(O, I)].T + bias[O][None, :]
    assert np.allclose(acc, ref, rtol=1e-12, atol=1e-12)
    # row selection and a padded leading dimension
    xp = np.zeros((4, len(I) + 7), dtype=np.float32)
    xp[:, :len(I)] = x
    xp[:, len(I):] = 99.0                                           # must be ignored
    sub = oracle.qlinear(xp, packed, qw.scales, qw.zeros, O, I, bias=bias, rows=[3, 1])
    assert np.array_equal(sub, acc[[3, 1]])


# 7, 9 ------------------------------------------------------------- closed forms, exact brute force
def test_closed_form_constant_codes():
    N, K, c = 2, 384, 11
    codes = np.full((N, K), c, dtype=np.uint8)
    s = np.array([[0.5, 0.25, 2.0], [1.0, 1.0, 1.0]], dtype=np.float16)
    z = np.array([[8, 3, 15], [0, 11, 12]], dtype=np.float16)
    k_in = 300      # groups hold 128, 128 and 44 retained channels
    x = np.ones((1, k_in), dtype=np.float32)
    acc = oracle.qlinear(x, oracle.pack_u4(codes), s, z, oracle.leading(N), oracle.leading(k_in))
    cnt = [128, 128, 44]
    for n in range(N):
        want = sum(float(s[n, g]) * (c - float(z[n, g])) * cnt[g] for g in range(3))
        assert acc[0, n] == want


def test_one_hot_selects_a_column():
    rng = np.random.default_rng(3)
    qw, packed = _small_q(rng, 16, 256)
    W = oracle.dequant(packed, qw.scales, qw.zeros)
    for t in (0, 1, 127, 128, 255):
        x = np.zeros((1, 256), dtype=np.float32)
        x[0, t] = 1.0
        acc = oracle.qlinear(x, packed, qw.scales, qw.zeros, oracle.leading(16), oracle.leading(256))
        assert np.array_equal(acc[0], W[:, t])


def test_brute_force_exact_rational():
    rng = np.random.default_rng(4)
    qw, packed = _small_q(rng, 8, 256)
    O = oracle.expand_map([(0, 4, 3, 2)])
    I = oracle.expand_map([(0, 128, 100, 2)])
    x = synth.draw_x(rng, 2, len(I), "f16")
    acc = oracle.qlinear(x, packed, qw.scales, qw.zeros, O, I)
    for m in range(2):
        for j, n in enumerate(O):
            tot = Fraction(0)
            for t, k in enumerate(I):
                byte = int(packed[n, k // 2])
                code = byte % 16 if k % 2 == 0 else byte // 16
                tot += Fraction(float(x[m, t])) * Fraction(float(qw.scales[n, k // 128])) * \
                    (code - Fraction(float(qw.zeros[n, k // 128])))
            assert abs(Fraction(acc[m, j]) - tot) <= abs(tot) * Fraction(1, 10**12) + Fraction(1, 10**13)


# 4, 5, 6 ---------------------------------------------------------- rotary embedding
def _textbook_rope(v, pos, theta):
    """Half-split rotary embedding on [R, H, D]: v*cos + rotate_half(v)*sin."""
    R, H, D = v.shape
    inv = theta ** (-np.arange(0, D, 2, dtype=np.float64) / D)
    ang = np.outer(pos.astype(np.float64), inv)                 # [R, D/2]
    cos = np.concatenate([np.cos(ang), np.cos(ang)], axis=1)[:, None, :]
    sin = np.concatenate([np.sin(ang), np.sin(ang)], axis=1)[:, None, :]
    rot = np.concatenate([-v[..., D // 2:], v[..., :D // 2]], axis=-1)
    return v * cos + rot * sin


def test_full_rank_identity_index_is_textbook_rope():
    rng = np.random.default_rng(6)
    R, H, Hkv, D, theta = 5, 4, 2, 16, 500000.0
    v = rng.standard_normal((R, H, D))
    pos = synth.draw_pos(rng, R)
    idx = synth.draw_idx(rng, Hkv, D, D, kind="identity")
    out = oracle.rope(v.reshape(R, H * D), H, Hkv, D, D, idx, pos, theta)
    assert np.allclose(out.reshape(R, H, D), _textbook_rope(v, pos, theta), rtol=1e-12, atol=1e-12)


def test_rope_literal_quarter_turn():
    # one head of dim 4 truncated to 2: the surviving pair is ORIGINAL pair 1 whose
    # frequency is theta^(-2*1/4); with theta = (2/pi)^2 that frequency is pi/2, so
    # position 1 is a quarter turn: (a, b) -> (-b, a).
    theta = (2.0 / np.pi) ** 2
    idx = np.array([[1]], dtype=np.int32)
    out = oracle.rope(np.array([[3.0, 5.0]]), 1, 1, 4, 2, idx, [1], theta)
    assert np.allclose(out, [[-5.0, 3.0]], atol=1e-12)
    out = oracle.rope(np.array([[3.0, 5.0]]), 1, 1, 4, 2, idx, [2], theta)
    assert np.allclose(out, [[-3.0, -5.0]], atol=1e-12)
    # an explicit frequency table overrides theta
    out = oracle.rope(np.array([[3.0, 5.0]]), 1, 1, 4, 2, idx, [1], 123.0,
                      inv_freq=np.array([0.0, np.pi]))
    assert np.allclose(out, [[-3.0, -5.0]], atol=1e-12)


def test_rope_preserves_pair_norms_and_relative_position():
    rng = np.random.default_rng(7)
    H, Hkv, D, d, theta = 4, 2, 32, 20, 10000.0
    idx = synth.draw_idx(rng, Hkv, D, d)
    q = rng.standard_normal((1, H * d))
    k = rng.standard_normal((1, Hkv * d))
    half = d // 2

    def rot(v, nh, p):
        return oracle.rope(v, nh, Hkv, D, d, idx, [p], theta)

    q0 = rot(q, H, 1234).reshape(H, d)
    qq = q.reshape(H, d)
    assert np.allclose(q0[:, :half] ** 2 + q0[:, half:] ** 2, qq[:, :half] ** 2 + qq[:, half:] ** 2,
                       rtol=1e-12)
    dots = []
    for delta in (0, 1, 17, 4000):
        qr = rot(q, H, 100 + delta).reshape(H, d)
        kr = rot(k, Hkv, 37 + delta).reshape(Hkv, d)
        dots.append([float(qr[h] @ kr[h // (H // Hkv)]) for h in range(H)])
    dots = np.array(dots)
    assert np.allclose(dots, dots[0], rtol=1e-9, atol=1e-9)
    # ... and the score does change with the relative distance (the rotation is not a no-op)
    qr = rot(q, H, 101).reshape(H, d)
    kr = rot(k, Hkv, 37).reshape(Hkv, d)
    assert not np.allclose([float(qr[h] @ kr[h // 2]) for h in range(H)], dots[0])


def test_sorted_truncated_projection_matches_rope_on_original_then_gather():
    """Sort-consistency: permute the rotation pairs of an un-sorted quantised matrix per
    KV head (Algorithm 6), truncate, project + pruned rotation == textbook rotation of
    the un-sorted projection followed by gathering the retained original dims."""
    rng = np.random.default_rng(8)
    H, Hkv, D, d, K, theta = 4, 2, 16, 12, 128, 500000.0
    qw = synth.draw_qweight(rng, H * D, K)
    x = synth.draw_x(rng, 3, K, "f16")
    pos = synth.draw_pos(rng, 3)
    perm = np.stack([rng.permutation(D // 2) for _ in range(Hkv)])         # full pair permutation
    rows = []
    for h in range(H):
        p = perm[h // (H // Hkv)]
        rows += [h * D + int(i) for i in p] + [h * D + D // 2 + int(i) for i in p]
    sorted_codes = qw.codes[rows]
    sorted_s, sorted_z = qw.scales[rows], qw.zeros[rows]
    O = oracle.expand_map(oracle.qk_halfhead_map(H, D, d))
    acc = oracle.qlinear(x, oracle.pack_u4(sorted_codes), sorted_s, sorted_z, O, oracle.leading(K))
    fused = oracle.rope(acc, H, Hkv, D, d, perm[:, :d // 2], pos, theta).reshape(3, H, d)
    W = oracle.dequant(oracle.pack_u4(qw.codes), qw.scales, qw.zeros)
    full = _textbook_rope((x.astype(np.float64) @ W.T).reshape(3, H, D), pos, theta)
    for h in range(H):
        p = perm[h // (H // Hkv)][:d // 2]
        want = np.concatenate([full[:, h, p], full[:, h, D // 2 + p]], axis=1)
        assert np.allclose(fused[:, h], want, rtol=1e-10, atol=1e-12)


def test_rope_rejects_bad_arguments():
    with pytest.raises(ValueError):
        oracle.rope(np.zeros((1, 2)), 1, 1, 4, 2, np.array([[2]], dtype=np.int32), [0], 10.0)


# ------------------------------------------------------------------ gated MLP block (Section 3.2, MLP paragraph)
def test_swiglu_closed_forms_and_library_logistic():
    from scipy.special import expit                       # the library's logistic function
    # literal values: silu(0) = 0, silu(ln 3) = ln 3 * 3/4, silu(-ln 3) = -ln 3 / 4
    ln3 = math.log(3.0)
    g = np.array([0.0, ln3, -ln3, 1.0])
    u = np.array([5.0, 2.0, -4.0, 1.0])
    h = oracle.swiglu(g, u)
    assert h[0] == 0.0
    assert abs(h[1] - 2.0 * ln3 * 0.75) < 1e-15
    assert abs(h[2] - ln3) < 1e-15                        # (-ln3/4) * (-4)
    assert abs(h[3] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    rng = np.random.default_rng(11)
    g = rng.normal(0, 4, 4096)
    u = rng.normal(0, 2, 4096)
    h = oracle.swiglu(g, u)
    assert np.allclose(h, g * expit(g) * u, rtol=1e-13, atol=1e-300)
    # silu(t) - silu(-t) = t (logistic(t) + logistic(-t) = 1): fails for any other gate such as sigmoid or gelu
    one = np.ones_like(g)
    assert np.allclose(oracle.swiglu(g, one) - oracle.swiglu(-g, one), g, rtol=0, atol=1e-14)
    # linear in u, the gate acts on g only (a swapped operand order fails here)
    assert np.allclose(oracle.swiglu(g, 3.0 * u), 3.0 * h, rtol=1e-15)
    assert not np.allclose(oracle.swiglu(u, g), h)
    # saturation: silu(t) -> t for large t, -> 0 for very negative t, without overflow
    big = oracle.swiglu(np.array([800.0, -800.0]), np.array([1.0, 1.0]))
    assert big[0] == 800.0 and big[1] == 0.0 and np.isfinite(big).all()


def test_mlp_swiglu_equals_dense_definition():
    from scipy.special import expit
    rng = np.random.default_rng(12)
    hidden, inter, k_int, M = 256, 384, 200, 3
    qg, pg = _small_q(rng, inter, hidden)
    qu, pu = _small_q(rng, inter, hidden)
    qd, pd = _small_q(rng, hidden, inter)
    x = synth.draw_x(rng, M, hidden, "f16", outlier_frac=0.02)
    Wg = oracle.dequant(pg, qg.scales, qg.zeros)
    Wu = oracle.dequant(pu, qu.scales, qu.zeros)
    Wd = oracle.dequant(pd, qd.scales, qd.zeros)
    xd = x.astype(np.float64)
    gd = xd @ Wg[:k_int].T
    hd = gd * expit(gd) * (xd @ Wu[:k_int].T)
    h, y = oracle.mlp_swiglu(x, pg, qg.scales, qg.zeros, pu, qu.scales, qu.zeros, pd, qd.scales, qd.zeros, k_int)
    assert h.shape == (M, k_int) and y.shape == (M, hidden)
    assert np.allclose(h, hd, rtol=1e-11, atol=1e-13)
    # the down projection sees the fp16-rounded activations and only the kept columns of Wd
    yd = hd.astype(np.float16).astype(np.float64) @ Wd[:, :k_int].T
    assert np.allclose(y, yd, rtol=1e-11, atol=1e-12)
    # pruning the intermediate channels is not a no-op here
    assert not np.allclose(yd, hd.astype(np.float16).astype(np.float64)[:, :k_int - 8] @ Wd[:, :k_int - 8].T)
    ys = oracle.mlp_swiglu(x, pg, qg.scales, qg.zeros, pu, qu.scales, qu.zeros, pd, qd.scales, qd.zeros, k_int,
                           out_rows=[5, 77, 255])[1]
    assert np.array_equal(ys, y[:, [5, 77, 255]])
    # a bfloat16 model: the stored activations are the library's bfloat16 conversion of h
    import torch
    hb = torch.from_numpy(hd.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    yb = oracle.mlp_swiglu(x, pg, qg.scales, qg.zeros, pu, qu.scales, qu.zeros, pd, qd.scales, qd.zeros, k_int,
                           h_dtype="bf16")[1]
    assert np.allclose(yb, hb @ Wd[:, :k_int].T, rtol=1e-11, atol=1e-12) and not np.allclose(yb, y, rtol=1e-6)


def test_round_bf16_against_the_library_conversion_and_ties():
    import torch
    rng = np.random.default_rng(13)
    a = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000), [0.0, -0.0, 1.0, -1.0]])
    want = torch.from_numpy(a.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(oracle.round_bf16(a), want)
    # ties go to the even pattern: 1 + 2^-8 lies half-way between 1 and 1 + 2^-7; 1 + 3 * 2^-8 between 1 + 2^-7 and 1 + 2^-6
    assert np.array_equal(oracle.round_bf16(np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20])),
                          np.array([1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7]))
