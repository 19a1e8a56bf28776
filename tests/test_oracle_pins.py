"""Pins for the CPU oracle: facts fixed by the paper's definition of attention
(Section 2.2, "Attention computation") and by mathematics, none of which re-use the
oracle's own code.  A dropped term, wrong sign, wrong index, transposed operand or
wrong mask alignment in the oracle fails at least one of these."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import attn_oracle as orc
from workloads import bf16_bits, bits_to_float64, make_qkv

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def to_bits(x):
    """float array -> BF16 bits (round to nearest even), via torch."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return bf16_bits(t).copy()


def rand_bits(shape, seed, gain=1.0):
    rng = np.random.default_rng(seed)
    return to_bits(rng.standard_normal(shape) * gain)


def brute_force(q, k, v, causal, scale):
    """Independent pure-Python statement: naive exponentials, no max subtraction,
    explicit visibility test per (i, j).  Small magnitudes only."""
    qf, kf, vf = bits_to_float64(q), bits_to_float64(k), bits_to_float64(v)
    B, Sq, Hq, D = qf.shape
    _, Sk, Hkv, _ = kf.shape
    g = Hq // Hkv
    O = np.zeros((B, Sq, Hq, D))
    L = np.zeros((B, Hq, Sq))
    for b in range(B):
        for h in range(Hq):
            hk = h // g
            for i in range(Sq):
                num = [0.0] * D
                den = 0.0
                for j in range(Sk):
                    if causal and j > i + Sk - Sq:
                        continue
                    s = sum(qf[b, i, h, d] * kf[b, j, hk, d] for d in range(D)) * scale
                    e = math.exp(s)
                    den += e
                    for d in range(D):
                        num[d] += e * vf[b, j, hk, d]
                for d in range(D):
                    O[b, i, h, d] = num[d] / den if den > 0 else 0.0
                L[b, h, i] = math.log(den) if den > 0 else -math.inf
    return O, L


def test_golden_sigmoid_two_keys():
    vals = {}
    with open(os.path.join(GOLDEN, "sigmoid_two_keys.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *nums = line.split()
            vals[key] = [float(x) for x in nums]
    q = to_bits(np.array(vals["q"]).reshape(1, 1, 1, 2))
    k = to_bits(np.array([vals["k0"], vals["k1"]]).reshape(1, 2, 1, 2))
    v = to_bits(np.array([vals["v0"], vals["v1"]]).reshape(1, 2, 1, 2))
    # the file's constants are sigmoid(2) and softplus(2)
    assert vals["O"][0] == pytest.approx(1 / (1 + math.exp(-2)), abs=1e-15)
    assert vals["LSE"][0] == pytest.approx(math.log1p(math.exp(2)), abs=1e-15)
    for causal in (False, True):  # Sq=1, Sk=2: bottom-right aligned mask hides nothing
        o, lse = orc.attention_full(q, k, v, causal, vals["scale"][0])
        np.testing.assert_allclose(o.ravel(), vals["O"], atol=1e-15)
        np.testing.assert_allclose(lse.ravel(), vals["LSE"], atol=1e-15)
    # Sq=Sk=2 causal: the first row sees only k0
    q2 = np.concatenate([q, q], axis=1)
    o, lse = orc.attention_full(q2, k, v, True, vals["scale"][0])
    np.testing.assert_allclose(o[0, 0, 0], vals["v0"], atol=0)
    assert lse[0, 0, 0] == 2.0
    np.testing.assert_allclose(o[0, 1, 0], vals["O"], atol=1e-15)


def test_single_key_returns_v_and_scaled_dot():
    q = rand_bits((2, 5, 3, 8), 1)
    k = rand_bits((2, 1, 3, 8), 2)
    v = rand_bits((2, 1, 3, 8), 3)
    scale = 0.37
    o, lse = orc.attention_full(q, k, v, False, scale)
    vf = bits_to_float64(v)
    np.testing.assert_array_equal(o, np.broadcast_to(vf, o.shape))
    dots = np.einsum("bihd,bjhd->bhi", bits_to_float64(q), bits_to_float64(k))
    np.testing.assert_allclose(lse, np.float64(np.float32(scale)) * dots, rtol=1e-14)


@pytest.mark.parametrize("B,Hq,Hkv,Sq,Sk,D,causal", [
    (1, 1, 1, 2, 2, 1, False),
    (1, 1, 1, 2, 2, 2, True),
    (2, 4, 2, 5, 7, 3, False),
    (2, 4, 2, 5, 7, 3, True),     # Sq < Sk: bottom-right aligned mask
    (1, 6, 2, 7, 4, 4, True),     # Sq > Sk: leading rows see no key
    (1, 3, 1, 9, 9, 16, True),
])
def test_brute_force_tiny(B, Hq, Hkv, Sq, Sk, D, causal):
    q = rand_bits((B, Sq, Hq, D), 10)
    k = rand_bits((B, Sk, Hkv, D), 11)
    v = rand_bits((B, Sk, Hkv, D), 12)
    scale = 1.0 / math.sqrt(D)
    o, lse = orc.attention_full(q, k, v, causal, scale)
    o_ref, lse_ref = brute_force(q, k, v, causal, float(np.float32(scale)))
    np.testing.assert_allclose(o, o_ref, atol=1e-13)
    finite = np.isfinite(lse_ref)
    np.testing.assert_allclose(lse[finite], lse_ref[finite], atol=1e-13)
    assert np.all(lse[~finite] == -np.inf)
    assert np.all(o[np.broadcast_to(~finite.transpose(0, 2, 1)[..., None], o.shape)] == 0)


def test_weights_are_a_probability_vector():
    q = rand_bits((1, 6, 2, 16), 20, gain=3.0)
    k = rand_bits((1, 33, 2, 16), 21, gain=3.0)
    v = rand_bits((1, 33, 2, 16), 22)
    for causal in (False, True):
        for i in range(6):
            p = orc.softmax_weights(q, k, v, causal, 0.25, 0, 1, i)
            assert np.all(p >= 0)
            assert abs(p.sum() - 1.0) < 1e-14
            nvis = 33 if not causal else i + 33 - 6 + 1
            assert np.all(p[nvis:] == 0) and np.all(p[:nvis] > 0)


def test_constant_v_gives_constant_o():
    q = rand_bits((1, 9, 2, 8), 30, gain=2.0)
    k = rand_bits((1, 17, 1, 8), 31, gain=2.0)
    v = to_bits(np.full((1, 17, 1, 8), 1.75))
    for causal in (False, True):
        o, _ = orc.attention_full(q, k, v, causal, 0.5)
        np.testing.assert_allclose(o, 1.75, atol=1e-15)


def test_causal_row0_is_v_row0():
    q, k, v = (bf16_bits(t) for t in make_qkv(2, 4, 2, 12, 12, 8, seed=40))
    scale = 0.3
    o, lse = orc.attention_full(q, k, v, True, scale)
    vf, qf, kf = bits_to_float64(v), bits_to_float64(q), bits_to_float64(k)
    for h in range(4):
        np.testing.assert_array_equal(o[:, 0, h], vf[:, 0, h // 2])
        want = np.float64(np.float32(scale)) * np.einsum("bd,bd->b", qf[:, 0, h], kf[:, 0, h // 2])
        np.testing.assert_allclose(lse[:, h, 0], want, rtol=1e-14)


def test_key_permutation_invariance_noncausal():
    q, k, v = (bf16_bits(t) for t in make_qkv(1, 2, 2, 7, 19, 16, seed=50))
    perm = np.random.default_rng(5).permutation(19)
    o1, l1 = orc.attention_full(q, k, v, False, 0.25)
    o2, l2 = orc.attention_full(q, k[:, perm], v[:, perm], False, 0.25)
    np.testing.assert_allclose(o1, o2, atol=1e-13)
    np.testing.assert_allclose(l1, l2, atol=1e-13)


def test_lse_is_log_of_summed_exponentials():
    q, k, v = (bf16_bits(t) for t in make_qkv(1, 2, 1, 5, 11, 8, seed=60))
    scale = float(np.float32(0.2))
    _, lse = orc.attention_full(q, k, v, False, scale)
    s = scale * np.einsum("bihd,bjd->bhij", bits_to_float64(q), bits_to_float64(k)[:, :, 0])
    np.testing.assert_allclose(lse, np.log(np.exp(s).sum(-1)), atol=1e-13)


@pytest.mark.parametrize("causal", [False, True])
def test_zero_q_gives_mean_of_visible_v(causal):
    B, Hq, Hkv, Sq, Sk, D = 1, 2, 1, 6, 10, 4
    q = np.zeros((B, Sq, Hq, D), dtype=np.uint16)
    _, k, v = (bf16_bits(t) for t in make_qkv(B, Hq, Hkv, Sq, Sk, D, seed=70))
    o, lse = orc.attention_full(q, k, v, causal, 1.0)
    vf = bits_to_float64(v)[0, :, 0]
    for i in range(Sq):
        n = Sk if not causal else i + Sk - Sq + 1
        np.testing.assert_allclose(o[0, i, 0], vf[:n].mean(0), atol=1e-14)
        np.testing.assert_allclose(o[0, i, 1], vf[:n].mean(0), atol=1e-14)
        assert lse[0, 0, i] == pytest.approx(math.log(n), abs=1e-14)


def test_gqa_equals_mha_with_repeated_kv_heads():
    q, k, v = (bf16_bits(t) for t in make_qkv(2, 8, 2, 6, 9, 8, seed=80))
    k_rep, v_rep = np.repeat(k, 4, axis=2), np.repeat(v, 4, axis=2)
    for causal in (False, True):
        o1, l1 = orc.attention_full(q, k, v, causal, 0.4)
        o2, l2 = orc.attention_full(q, k_rep, v_rep, causal, 0.4)
        np.testing.assert_array_equal(o1, o2)
        np.testing.assert_array_equal(l1, l2)
    # the mapping is hq // group, not hq % Hkv: heads 0..3 share kv head 0
    o_all, _ = orc.attention_full(q, k, v, False, 0.4)
    o_h0, _ = orc.attention_full(q[:, :, :4], k[:, :, :1], v[:, :, :1], False, 0.4)
    np.testing.assert_array_equal(o_all[:, :, :4], o_h0)


def test_causal_equals_noncausal_on_truncated_keys():
    q, k, v = (bf16_bits(t) for t in make_qkv(1, 2, 2, 5, 8, 8, seed=90))
    o_c, l_c = orc.attention_full(q, k, v, True, 0.35)
    for i in range(5):
        n = i + 8 - 5 + 1
        o_n, l_n = orc.attention_full(q[:, i:i + 1], k[:, :n], v[:, :n], False, 0.35)
        np.testing.assert_allclose(o_c[:, i], o_n[:, 0], atol=1e-14)
        np.testing.assert_allclose(l_c[:, :, i], l_n[:, :, 0], atol=1e-14)


def test_key_shift_moves_lse_only():
    B, Hq, Hkv, Sq, Sk, D = 1, 2, 2, 4, 9, 8
    rng = np.random.default_rng(100)
    # small integers: k + c is exact in BF16
    q = to_bits(rng.integers(-2, 3, (B, Sq, Hq, D)))
    kf = rng.integers(-3, 4, (B, Sk, Hkv, D)).astype(np.float64)
    v = rand_bits((B, Sk, Hkv, D), 101)
    c = rng.integers(-2, 3, (D,)).astype(np.float64)
    scale = 0.125
    o1, l1 = orc.attention_full(q, to_bits(kf), v, False, scale)
    o2, l2 = orc.attention_full(q, to_bits(kf + c), v, False, scale)
    np.testing.assert_allclose(o1, o2, atol=1e-13)
    shift = scale * np.einsum("bihd,d->bhi", bits_to_float64(q), c)
    np.testing.assert_allclose(l2 - l1, shift, atol=1e-13)


def test_split_merge_identity():
    q, k, v = (bf16_bits(t) for t in make_qkv(1, 2, 1, 6, 20, 8, seed=110))
    o, l = orc.attention_full(q, k, v, False, 0.3)
    o1, l1 = orc.attention_full(q, k[:, :7], v[:, :7], False, 0.3)
    o2, l2 = orc.attention_full(q, k[:, 7:], v[:, 7:], False, 0.3)
    l12 = np.log(np.exp(l1) + np.exp(l2))
    np.testing.assert_allclose(l, l12, atol=1e-13)
    w1 = np.exp(l1 - l12).transpose(0, 2, 1)[..., None]
    w2 = np.exp(l2 - l12).transpose(0, 2, 1)[..., None]
    np.testing.assert_allclose(o, w1 * o1 + w2 * o2, atol=1e-13)


@pytest.mark.parametrize("causal", [False, True])
def test_matches_library_sdpa_float64(causal):
    B, Hq, Hkv, Sq, Sk, D = 2, 4, 4, 33, 33, 32
    qt, kt, vt = make_qkv(B, Hq, Hkv, Sq, Sk, D, seed=120)
    scale = float(np.float32(1 / math.sqrt(D)))
    o, _ = orc.attention_full(bf16_bits(qt), bf16_bits(kt), bf16_bits(vt), causal, scale)
    ref = torch.nn.functional.scaled_dot_product_attention(
        qt.double().transpose(1, 2), kt.double().transpose(1, 2), vt.double().transpose(1, 2),
        is_causal=causal, scale=scale).transpose(1, 2)
    np.testing.assert_allclose(o, ref.numpy(), atol=1e-12)


def test_rows_mode_equals_full_mode_and_is_thread_independent():
    q, k, v = (bf16_bits(t) for t in make_qkv(2, 4, 2, 40, 48, 16, seed=130))
    o, l = orc.attention_full(q, k, v, True, 0.25, threads=3)
    rows = np.array([(b, h, i) for b in range(2) for h in range(4) for i in (0, 7, 39)], dtype=np.int32)
    o_r, l_r = orc.attention_rows(q, k, v, True, 0.25, rows, threads=1)
    for n, (b, h, i) in enumerate(rows):
        np.testing.assert_array_equal(o_r[n], o[b, i, h])
        assert l_r[n] == l[b, h, i]


def test_bad_arguments_are_rejected():
    q, k, v = (bf16_bits(t) for t in make_qkv(1, 3, 2, 4, 4, 8, seed=140))  # 3 % 2 != 0
    with pytest.raises(ValueError):
        orc.attention_full(q, k, v, False, 1.0)
    q, k, v = (bf16_bits(t) for t in make_qkv(1, 2, 2, 4, 4, 8, seed=141))
    with pytest.raises(ValueError):
        orc.attention_rows(q, k, v, False, 1.0, np.array([[0, 0, 4]], dtype=np.int32))


def _f32_to_bits(x):
    return to_bits(x)


def test_merge_of_exact_halves_reproduces_the_whole():
    """Pins attn_oracle_merge: feed it partial results that are exactly representable (BF16 O parts
    from one-hot softmaxes) and compare with the attention over all keys."""
    # one query, D = 2; part 1 = key A only, part 2 = key B only: O_i = v_i exactly, LSE_i = s_i
    va, vb = np.array([1.0, -2.0]), np.array([0.5, 4.0])
    sa, sb = 1.25, -0.75          # exactly representable in fp32
    o, lse = orc.merge(to_bits(va.reshape(1, 2)), np.array([sa], np.float32),
                       to_bits(vb.reshape(1, 2)), np.array([sb], np.float32))
    wa = 1.0 / (1.0 + math.exp(sb - sa))
    np.testing.assert_allclose(o[0], wa * va + (1 - wa) * vb, atol=1e-15)
    assert lse[0] == pytest.approx(math.log(math.exp(sa) + math.exp(sb)), abs=1e-15)


def test_merge_special_cases():
    o1 = rand_bits((5, 8), 200)
    o2 = rand_bits((5, 8), 201)
    l1 = np.linspace(-3, 3, 5).astype(np.float32)
    # an empty second part changes nothing
    o, lse = orc.merge(o1, l1, o2, np.full(5, -np.inf, np.float32))
    np.testing.assert_array_equal(o, bits_to_float64(o1))
    np.testing.assert_array_equal(lse, l1.astype(np.float64))
    # equal LSEs: plain average, LSE + log 2
    o, lse = orc.merge(o1, l1, o2, l1)
    np.testing.assert_allclose(o, 0.5 * (bits_to_float64(o1) + bits_to_float64(o2)), atol=1e-15)
    np.testing.assert_allclose(lse, l1.astype(np.float64) + math.log(2.0), atol=1e-15)
    # symmetric in its two parts
    l2 = l1[::-1].copy()
    oa, la = orc.merge(o1, l1, o2, l2)
    ob, lb = orc.merge(o2, l2, o1, l1)
    np.testing.assert_allclose(oa, ob, atol=1e-15)
    np.testing.assert_allclose(la, lb, atol=1e-15)
    # both empty
    o, lse = orc.merge(o1, np.full(5, -np.inf, np.float32), o2, np.full(5, -np.inf, np.float32))
    assert np.all(o == 0) and np.all(lse == -np.inf)


def test_merge_n_of_single_key_parts_is_the_softmax_itself():
    """Pins attn_oracle_merge_n against the definition: n parts of one key each have O_i = v_i and
    LSE_i = s_i exactly, so their merge is the softmax-weighted mean of the v_i (closed form
    evaluated here with math.exp)."""
    vs = [np.array([1.0, -2.0]), np.array([0.5, 4.0]), np.array([-3.0, 0.25]), np.array([8.0, 1.0])]
    ss = [1.25, -0.75, 0.5, 2.0]  # exactly representable in fp32
    o, lse = orc.merge_n(np.stack([to_bits(v.reshape(1, 2)) for v in vs]),
                         np.array([[s] for s in ss], np.float32))
    z = sum(math.exp(s) for s in ss)
    want = sum(math.exp(s) / z * v for s, v in zip(ss, vs))
    np.testing.assert_allclose(o[0], want, atol=1e-14)
    assert lse[0] == pytest.approx(math.log(z), abs=1e-14)


def test_merge_n_special_cases_and_consistency_with_pairwise_merge():
    parts = np.stack([rand_bits((6, 8), 300 + i) for i in range(4)])
    lses = np.stack([np.linspace(-2, 2, 6), np.linspace(3, -3, 6), np.full(6, 0.5), np.linspace(0, 1, 6)]).astype(np.float32)
    o, lse = orc.merge_n(parts, lses)
    # weights are a probability vector: merging n copies of the same part returns it, LSE + log n
    same_o, same_l = orc.merge_n(np.stack([parts[0]] * 3), np.stack([lses[0]] * 3))
    np.testing.assert_allclose(same_o, bits_to_float64(parts[0]), atol=1e-15)
    np.testing.assert_allclose(same_l, lses[0].astype(np.float64) + math.log(3.0), atol=1e-15)
    # order of the parts does not matter
    perm = [2, 0, 3, 1]
    o_p, lse_p = orc.merge_n(parts[perm], lses[perm])
    np.testing.assert_allclose(o_p, o, atol=1e-14)
    np.testing.assert_allclose(lse_p, lse, atol=1e-14)
    # empty parts (LSE = -inf) have no say; all empty gives O = 0, LSE = -inf
    lses_e = lses.copy()
    lses_e[1] = -np.inf
    o_e, lse_e = orc.merge_n(parts, lses_e)
    o_3, lse_3 = orc.merge_n(parts[[0, 2, 3]], lses[[0, 2, 3]])
    np.testing.assert_allclose(o_e, o_3, atol=1e-15)
    np.testing.assert_allclose(lse_e, lse_3, atol=1e-15)
    o_0, lse_0 = orc.merge_n(parts, np.full_like(lses, -np.inf))
    assert np.all(o_0 == 0) and np.all(lse_0 == -np.inf)
    # n = 2 is the two-part merge
    o_2, lse_2 = orc.merge_n(parts[:2], lses[:2])
    o_pair, lse_pair = orc.merge(parts[0], lses[0], parts[1], lses[1])
    np.testing.assert_allclose(o_2, o_pair, atol=1e-15)
    np.testing.assert_allclose(lse_2, lse_pair, atol=1e-15)


@pytest.mark.parametrize("causal", [False, True])
def test_split_keys_n_ways_and_merge_equals_the_whole(causal):
    """The route attn_fwd_splitkv takes, in the oracle alone: attention over key ranges (under the
    causal mask each range with the offset that keeps global key indices), merged n ways, equals
    attention over all keys.  The parts are kept in float64 here, so the identity is exact."""
    B, Hq, Hkv, Sq, Sk, D = 1, 2, 1, 5, 23, 8
    q, k, v = (bf16_bits(t) for t in make_qkv(B, Hq, Hkv, Sq, Sk, D, seed=310))
    o, l = orc.attention_full(q, k, v, causal, 0.3)
    cuts = [0, 6, 7, 16, 23]
    num = np.zeros_like(o)
    parts_l = []
    parts_o = []
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        if causal:
            # rows see keys j <= i + Sk - Sq; inside the range that is j - lo <= i + (Sk - Sq - lo):
            # emulate the shifted mask by giving the sub-problem only the keys each row may see
            o_p = np.zeros_like(o)
            l_p = np.full(l.shape, -np.inf)
            for i in range(Sq):
                last = min(hi, i + Sk - Sq + 1)
                if last > lo:
                    oi, li = orc.attention_full(q[:, i:i + 1], k[:, lo:last], v[:, lo:last], False, 0.3)
                    o_p[:, i] = oi[:, 0]
                    l_p[:, :, i] = li[:, :, 0]
        else:
            o_p, l_p = orc.attention_full(q, k[:, lo:hi], v[:, lo:hi], False, 0.3)
        parts_o.append(o_p)
        parts_l.append(l_p)
    tot = np.log(sum(np.exp(lp) for lp in parts_l))
    np.testing.assert_allclose(tot, l, atol=1e-13)
    for o_p, l_p in zip(parts_o, parts_l):
        num += np.exp(l_p - tot).transpose(0, 2, 1)[..., None] * o_p
    np.testing.assert_allclose(num, o, atol=1e-13)
