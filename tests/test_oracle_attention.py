"""Pins for the oracle's decode attention (Eq. 2 with the appendix's 1/sqrt(d); Eq. 3)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import bf16_bits_to_f64, f32_to_bf16_bits


def _rand_bf16(rng, shape, scale=1.0):
    return f32_to_bf16_bits((rng.standard_normal(shape) * scale).astype(np.float32))


def _torch_attention(q, K, V, sm_scale):
    q, K, V = (torch.from_numpy(np.asarray(a, np.float64)) for a in (q, K, V))
    return (torch.softmax((K @ q) * sm_scale, dim=0) @ V).numpy()


def test_no_quantised_tokens_is_textbook_attention():
    # N <= 3W: nothing has been filtered out; the result is plain softmax attention on the bf16 inputs.
    B, Hq, Hkv, D, W, G = 2, 8, 2, 128, 32, 32
    rng = np.random.default_rng(0)
    N = 3 * W
    k, v = _rand_bf16(rng, (B, Hkv, N, D)), _rand_bf16(rng, (B, Hkv, N, D))
    q = _rand_bf16(rng, (B, Hq, D))
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    oc.append(k, v)
    assert oc.n_quant == 0
    out = oc.attention(q, 1 / np.sqrt(D))
    r = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            ref = _torch_attention(bf16_bits_to_f64(q[b, h]), bf16_bits_to_f64(k[b, h // r]),
                                   bf16_bits_to_f64(v[b, h // r]), 1 / np.sqrt(D))
            np.testing.assert_allclose(out[b, h], ref, rtol=0, atol=1e-13)


def test_mixed_cache_equals_library_attention_on_dequantised_rows_and_gqa_mapping():
    B, Hq, Hkv, D, W, G = 2, 6, 2, 128, 32, 32
    rng = np.random.default_rng(1)
    N = 7 * W + 5
    k, v = _rand_bf16(rng, (B, Hkv, N, D)), _rand_bf16(rng, (B, Hkv, N, D))
    q = _rand_bf16(rng, (B, Hq, D))
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    oc.append(k, v)
    img = oc.export()
    nf, nq = oc.n_fp, oc.n_quant
    assert nq > 0 and nf + nq == N
    out = oc.attention(q, 0.07, n_threads=3)
    out1 = oc.attention(q, 0.07, n_threads=1)
    assert np.array_equal(out, out1)
    kc = oracle.unpack2(img["k_codes"]).reshape(B, Hkv, nq, D).astype(np.float64)
    vc = oracle.unpack2(img["v_codes"]).reshape(B, Hkv, nq, D).astype(np.float64)
    # dequantise with numpy broadcasting: key scale/zero indexed by (token // G, channel),
    # value scale/zero by (token, channel // G)
    Kq = bf16_bits_to_f64(img["k_zero"]).repeat(G, axis=2) + kc * bf16_bits_to_f64(img["k_scale"]).repeat(G, axis=2)
    Vq = bf16_bits_to_f64(img["v_zero"]).repeat(G, axis=3) + vc * bf16_bits_to_f64(img["v_scale"]).repeat(G, axis=3)
    r = Hq // Hkv
    for b in range(B):
        for h in range(Hq):
            kv = h // r  # consecutive query heads share a KV head
            K = np.concatenate([bf16_bits_to_f64(img["fp_k"][b, kv]), Kq[b, kv]])
            V = np.concatenate([bf16_bits_to_f64(img["fp_v"][b, kv]), Vq[b, kv]])
            ref = _torch_attention(bf16_bits_to_f64(q[b, h]), K, V, 0.07)
            np.testing.assert_allclose(out[b, h], ref, rtol=0, atol=1e-13)
        Kd, Vd = oc.dense_rows(b, 1)
        assert np.array_equal(Kd, np.concatenate([bf16_bits_to_f64(img["fp_k"][b, 1]), Kq[b, 1]]))
        assert np.array_equal(Vd, np.concatenate([bf16_bits_to_f64(img["fp_v"][b, 1]), Vq[b, 1]]))
    # dequantised rows stay within scale/2 (+ bf16 slack on the scale) of the original tokens
    Q = img["quant_ids"]
    err = np.abs(Kq - bf16_bits_to_f64(k[:, :, Q, :]))
    assert np.all(err <= bf16_bits_to_f64(img["k_scale"]).repeat(G, axis=2) * (0.5 + 3 * 2.0 ** -8))


def test_permutation_invariance():
    # Eq. 3: A.V = A_P.V_P -- any order of the (already dequantised) cache rows gives the same output.
    rng = np.random.default_rng(2)
    n, D = 300, 128
    K, V, q = rng.standard_normal((n, D)), rng.standard_normal((n, D)), rng.standard_normal(D)
    ref = oracle.attention_dense(q, K, V, 0.09)
    for _ in range(5):
        P = rng.permutation(n)
        np.testing.assert_allclose(oracle.attention_dense(q, K[P], V[P], 0.09), ref, rtol=0, atol=1e-12)


def test_closed_form_special_cases():
    rng = np.random.default_rng(3)
    n, D = 77, 128
    K, q = rng.standard_normal((n, D)), rng.standard_normal(D)
    v = rng.standard_normal(D)
    # all value rows equal -> output is that row
    np.testing.assert_allclose(oracle.attention_dense(q, K, np.tile(v, (n, 1)), 0.1), v, rtol=0, atol=1e-13)
    # q = 0 -> uniform weights -> mean of the value rows
    V = rng.standard_normal((n, D))
    np.testing.assert_allclose(oracle.attention_dense(np.zeros(D), K, V, 0.1), V.mean(0), rtol=0, atol=1e-13)
    # one token -> its value row
    np.testing.assert_allclose(oracle.attention_dense(q, K[:1], V[:1], 0.1), V[0], rtol=0, atol=0)
    # a dominant score -> (almost) that token's value row; sign and scale of sm_scale matter
    Kb = K.copy()
    Kb[5] = q * 50
    np.testing.assert_allclose(oracle.attention_dense(q, Kb, V, 1.0), V[5], rtol=0, atol=1e-9)
    Kb[5] = -q * 50
    assert np.abs(oracle.attention_dense(q, Kb, V, 1.0) - V[5]).max() > 0.1
    # two tokens, hand formula: weights e^{s0}/(e^{s0}+e^{s1})
    s = (K[:2] @ q) * 0.05
    w0 = 1 / (1 + np.exp(s[1] - s[0]))
    np.testing.assert_allclose(oracle.attention_dense(q, K[:2], V[:2], 0.05), w0 * V[0] + (1 - w0) * V[1],
                               rtol=0, atol=1e-13)


@pytest.mark.parametrize("cuts", [[0, 300], [0, 257, 300], [0, 1, 2, 150, 150, 299, 300]])
def test_partial_merge_equals_one_pass(cuts):
    # (m, l) online-softmax merge of segment partials equals the one-pass softmax; empty segments allowed.
    rng = np.random.default_rng(4)
    n, D = 300, 128
    K, V, q = rng.standard_normal((n, D)) * 3, rng.standard_normal((n, D)), rng.standard_normal(D)
    ref = oracle.attention_dense(q, K, V, 0.3)
    ms, ls, os_ = [], [], []
    for a, b in zip(cuts[:-1], cuts[1:]):
        m, l, o = oracle.attention_partial(q, K[a:b], V[a:b], 0.3)
        ms.append(m), ls.append(l), os_.append(o)
    out = oracle.attention_merge(np.array(ms), np.array(ls), np.stack(os_))
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-13)


def test_quantisation_error_of_attention_is_small_but_nonzero():
    # sanity: the mixed cache is an approximation of exact attention, and a good one at N(0,1) inputs
    B, Hq, Hkv, D, W, G = 1, 4, 1, 128, 32, 32
    rng = np.random.default_rng(6)
    N = 12 * W + 1
    k, v = _rand_bf16(rng, (B, Hkv, N, D)), _rand_bf16(rng, (B, Hkv, N, D))
    q = _rand_bf16(rng, (B, Hq, D))
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    oc.append(k, v)
    out = oc.attention(q, 1 / np.sqrt(D))
    exact = np.stack([_torch_attention(bf16_bits_to_f64(q[0, h]), bf16_bits_to_f64(k[0, 0]),
                                       bf16_bits_to_f64(v[0, 0]), 1 / np.sqrt(D)) for h in range(Hq)])
    err = np.abs(out[0] - exact).max()
    assert 1e-6 < err < 0.2


def _subset_case(W=32, G=32, N=7 * 32 + 5, B=3, Hq=4, Hkv=2, seed=11):
    rng = np.random.default_rng(seed)
    k, v = _rand_bf16(rng, (B, Hkv, N, 128)), _rand_bf16(rng, (B, Hkv, N, 128))
    q = _rand_bf16(rng, (B, Hq, 128))
    oc = oracle.OracleCache(B, Hq, Hkv, 128, W, G)
    oc.append(k, v)
    return oc, q, k, v


def test_subset_attention_full_precision_only_is_attention_over_the_kept_tokens():
    # the eviction variants of Sec. 2.3: tokens the filter removes are dropped.  Expected value from torch
    # on the ORIGINAL bf16 rows of the ids Algorithm 1 keeps (hand simulation in helpers.alg1_python).
    from helpers import alg1_python
    oc, q, k, v = _subset_case()
    B, Hq, Hkv, N = 3, 4, 2, k.shape[2]
    kept, _ = alg1_python(32, N)
    out = oc.attention_subset(q, 0.09, fp_only=True)
    for b in range(B):
        for h in range(Hq):
            ref = _torch_attention(bf16_bits_to_f64(q[b, h]), bf16_bits_to_f64(k[b, h // 2][kept]),
                                   bf16_bits_to_f64(v[b, h // 2][kept]), 0.09)
            np.testing.assert_allclose(out[b, h], ref, rtol=0, atol=1e-13)
    # nothing selected away: the plain attention
    assert np.array_equal(oc.attention_subset(q, 0.09), oc.attention(q, 0.09))
    assert np.array_equal(oc.attention_subset(q, 0.09, pad=np.zeros(B, np.int32)), oc.attention(q, 0.09))


def test_subset_attention_left_padding_drops_exactly_the_padded_ids():
    oc, q, k, v = _subset_case()
    B, Hq, Hkv, G = 3, 4, 2, 32
    img = oc.export()
    nq = oc.n_quant
    pad = np.array([0, 37, 150], np.int32)  # none; inside the first removed groups; beyond several groups
    out = oc.attention_subset(q, 0.11, pad=pad)
    kc = oracle.unpack2(img["k_codes"]).reshape(B, Hkv, nq, 128).astype(np.float64)
    vc = oracle.unpack2(img["v_codes"]).reshape(B, Hkv, nq, 128).astype(np.float64)
    Kq = bf16_bits_to_f64(img["k_zero"]).repeat(G, axis=2) + kc * bf16_bits_to_f64(img["k_scale"]).repeat(G, axis=2)
    Vq = bf16_bits_to_f64(img["v_zero"]).repeat(G, axis=3) + vc * bf16_bits_to_f64(img["v_scale"]).repeat(G, axis=3)
    ids = np.concatenate([img["kept_ids"], img["quant_ids"]])
    for b in range(B):
        sel = ids >= pad[b]
        assert sel.sum() == k.shape[2] - pad[b]
        for h in range(Hq):
            K = np.concatenate([bf16_bits_to_f64(img["fp_k"][b, h // 2]), Kq[b, h // 2]])[sel]
            V = np.concatenate([bf16_bits_to_f64(img["fp_v"][b, h // 2]), Vq[b, h // 2]])[sel]
            ref = _torch_attention(bf16_bits_to_f64(q[b, h]), K, V, 0.11)
            np.testing.assert_allclose(out[b, h], ref, rtol=0, atol=1e-13)
    # padded VALUES never reach the output: rewriting the value rows of sequence 2's padding inside whole
    # removed groups (a value group lies inside one token) changes nothing for that sequence
    k2, v2 = k.copy(), v.copy()
    v2[2, :, :150] = _rand_bf16(np.random.default_rng(5), (Hkv, 150, 128), 3.0)
    oc2 = oracle.OracleCache(B, Hq, Hkv, 128, 32, G)
    oc2.append(k2, v2)
    out2 = oc2.attention_subset(q, 0.11, pad=pad)
    np.testing.assert_allclose(out2[2], out[2], rtol=0, atol=1e-13)
    # both selections together
    both = oc.attention_subset(q, 0.11, fp_only=True, pad=pad)
    for b in range(B):
        keep = img["kept_ids"][img["kept_ids"] >= pad[b]]
        ref = _torch_attention(bf16_bits_to_f64(q[b, 0]), bf16_bits_to_f64(k[b, 0][keep]),
                               bf16_bits_to_f64(v[b, 0][keep]), 0.11)
        np.testing.assert_allclose(both[b, 0], ref, rtol=0, atol=1e-13)
