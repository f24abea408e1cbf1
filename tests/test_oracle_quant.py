"""Pins for the oracle's 2-bit and 4-bit quantisers and packers."""
import os

import numpy as np
import pytest

import oracle
from helpers import bf16_bits_to_f64, f32_to_bf16_bits

GOLD = os.path.join(os.path.dirname(__file__), "golden", "quant_worked_example.txt")


def _gold():
    out = []
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        vals, sz, codes, bts = [s.split() for s in line.split("|")]
        out.append(([float(v) for v in vals], float(sz[0]), float(sz[1]), [int(c) for c in codes],
                    [int(b, 16) for b in bts]))
    return out


@pytest.mark.parametrize("vals,scale,zero,codes,packed", _gold())
def test_worked_examples(vals, scale, zero, codes, packed):
    x = f32_to_bf16_bits(np.array(vals, np.float32))
    assert np.array_equal(bf16_bits_to_f64(x), np.array(vals))  # the fixture is bf16-exact
    s, z, c = oracle.quantize_group(x)
    assert oracle.bf16_to_f32(s) == scale and oracle.bf16_to_f32(z) == zero
    assert c.tolist() == codes
    assert oracle.pack2(c).tolist() == packed


def test_pack_unpack_all_bytes():
    allb = np.arange(256, dtype=np.uint8)
    codes = oracle.unpack2(allb)
    assert codes.max() == 3
    assert np.array_equal(oracle.pack2(codes), allb)
    # bit layout: element 4j+i in bits [2i+1:2i] of byte j
    for i in range(4):
        c = np.zeros(8, np.uint8)
        c[4 + i] = 3
        assert oracle.pack2(c).tolist() == [0, 3 << (2 * i)]


@pytest.mark.parametrize("n", [32, 64])
@pytest.mark.parametrize("spread", [1.0, 10.0, 1e-3, 300.0])
def test_round_trip_bound_and_order(n, spread):
    rng = np.random.default_rng(1234 + n)
    for trial in range(200):
        x = f32_to_bf16_bits((rng.standard_normal(n) * spread + rng.standard_normal() * spread).astype(np.float32))
        s, z, c = oracle.quantize_group(x)
        xv = bf16_bits_to_f64(x)
        sv, zv = oracle.bf16_to_f32(s), oracle.bf16_to_f32(z)
        assert zv == xv.min()
        assert abs(sv - (xv.max() - xv.min()) / 3) <= 2.0 ** -8 * sv  # scale is (max-min)/3 to bf16 precision
        xh = np.array([oracle.dequant(s, z, int(ci)) for ci in c])
        assert np.all(np.abs(xv - xh) <= sv / 2 * (1 + 1e-6) + 3 * sv * 2.0 ** -8)
        assert np.array_equal(xh, zv + c.astype(np.float64) * sv)
        assert c[np.argmin(xv)] == 0 and c[np.argmax(xv)] == 3
        order = np.argsort(xv, kind="stable")
        assert np.all(np.diff(c[order].astype(int)) >= 0)  # codes are monotone in x


def test_half_scale_bound_when_scale_is_exact():
    # When (max-min)/3 is exactly a bf16 value the bound |x - x^| <= scale/2 holds with no slack.
    rng = np.random.default_rng(7)
    worst = 0.0
    for trial in range(300):
        s = 2.0 ** rng.integers(-6, 4)
        a = float(rng.integers(-8, 8)) * s
        x = a + rng.uniform(0, 3 * s, 32)
        x[0], x[1] = a, a + 3 * s
        xb = f32_to_bf16_bits(x.astype(np.float32))
        xv = bf16_bits_to_f64(xb)
        sb, zb, c = oracle.quantize_group(xb)
        assert oracle.bf16_to_f32(sb) == s and oracle.bf16_to_f32(zb) == a
        err = np.abs(xv - (a + c * s))
        worst = max(worst, float(err.max() / s))
        assert np.all(err <= s / 2)
    assert worst > 0.4  # the bound is tight


def test_lattice_groups_round_trip_exactly():
    rng = np.random.default_rng(3)
    for trial in range(100):
        s = 2.0 ** rng.integers(-5, 5)
        a = float(rng.integers(-16, 16)) * s
        k = rng.integers(0, 4, 32)
        k[:2] = [0, 3]
        x = f32_to_bf16_bits((a + k * s).astype(np.float32))
        sb, zb, c = oracle.quantize_group(x)
        assert np.array_equal(c, k.astype(np.uint8))
        assert oracle.bf16_to_f32(sb) == s and oracle.bf16_to_f32(zb) == a


def test_constant_group():
    x = f32_to_bf16_bits(np.full(64, 1.2345, np.float32))
    s, z, c = oracle.quantize_group(x)
    assert s == 0 and not c.any() and oracle.dequant(s, z, 0) == bf16_bits_to_f64(x)[0]


def test_cache_grouping_matches_vectorised_numpy():
    """Keys: groups run down G evicted tokens per channel; values: across G channels per token.
    The groups are re-formed here with numpy reshapes from the literal Algorithm 1 eviction order."""
    from helpers import alg1_python, bf16_bits_to_f32
    B, Hq, Hkv, D, W, G = 2, 4, 2, 128, 32, 32
    N = 3 * W + W + 1  # two events
    rng = np.random.default_rng(11)
    k = f32_to_bf16_bits(rng.standard_normal((B, Hkv, N, D)).astype(np.float32))
    v = f32_to_bf16_bits(rng.standard_normal((B, Hkv, N, D)).astype(np.float32))
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    oc.append(k, v)
    img = oc.export()
    A, Q = alg1_python(W, N)
    assert img["kept_ids"].tolist() == A and img["quant_ids"].tolist() == Q
    assert np.array_equal(img["fp_k"], k[:, :, A, :]) and np.array_equal(img["fp_v"], v[:, :, A, :])

    def quant(x, axis):  # x fp32, group along `axis`; fp32 arithmetic like the quantiser's reading
        mn, mx = x.min(axis, keepdims=True), x.max(axis, keepdims=True)
        sc = bf16_bits_to_f32(f32_to_bf16_bits(((mx - mn) / np.float32(3.0)).astype(np.float32)))
        with np.errstate(divide="ignore", invalid="ignore"):
            c = np.clip(np.rint((x - mn) / sc), 0, 3)
        c = np.where(sc == 0, 0, c).astype(np.uint8)
        return c, f32_to_bf16_bits(sc), f32_to_bf16_bits(mn)

    kq = bf16_bits_to_f32(k[:, :, Q, :]).reshape(B, Hkv, len(Q) // G, G, D)
    c, s, z = quant(kq, 3)
    assert np.array_equal(oracle.unpack2(img["k_codes"]).reshape(kq.shape), c)
    assert np.array_equal(img["k_scale"], s[:, :, :, 0, :]) and np.array_equal(img["k_zero"], z[:, :, :, 0, :])
    vq = bf16_bits_to_f32(v[:, :, Q, :]).reshape(B, Hkv, len(Q), D // G, G)
    c, s, z = quant(vq, 4)
    assert np.array_equal(oracle.unpack2(img["v_codes"]).reshape(vq.shape), c)
    assert np.array_equal(img["v_scale"], s[..., 0]) and np.array_equal(img["v_zero"], z[..., 0])


def test_export_sizes_match_byte_formulas():
    B, Hq, Hkv, D, W, G = 1, 8, 2, 128, 128, 32
    rng = np.random.default_rng(5)
    N = 1024
    k = f32_to_bf16_bits(rng.standard_normal((B, Hkv, N, D)).astype(np.float32))
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    oc.append(k, k)
    assert (oc.n_quant, oc.n_fp, oc.n_events) == (640, 384, 5)
    oc.append(k[:, :, :1], k[:, :, :1])
    assert (oc.n_quant, oc.n_fp, oc.n_events) == (768, 257, 6)
    img = oc.export()
    per_tok = sum(img[n].nbytes for n in ("k_codes", "v_codes", "k_scale", "k_zero", "v_scale", "v_zero"))
    assert per_tok == B * Hkv * oc.n_quant * 96  # 96 B per quantised token per KV head at G = 32
    assert img["fp_k"].nbytes + img["fp_v"].nbytes == B * Hkv * oc.n_fp * 512


def test_signed_zero_is_canonical():
    # min (or max) equal to zero is stored as +0 whatever the sign bit of the inputs
    neg0, pos0, one = 0x8000, 0x0000, 0x3F80
    for grp in ([neg0, pos0, one, one], [pos0, neg0, one, one], [neg0, neg0, one, one]):
        s, z, c = oracle.quantize_group(np.array(grp, np.uint16))
        assert z == 0x0000 and c.tolist() == [0, 0, 3, 3]
    s, z, c = oracle.quantize_group(np.array([neg0, pos0, neg0, neg0], np.uint16))
    assert (s, z) == (0, 0) and not c.any()
    minus1 = 0xBF80
    s, z, c = oracle.quantize_group(np.array([minus1, neg0, minus1, pos0], np.uint16))
    assert z == minus1 and c.tolist() == [0, 3, 0, 3]


# ---- 4-bit variant (the paper's second precision) ------------------------------------------
GOLD4 = os.path.join(os.path.dirname(__file__), "golden", "quant4_worked_example.txt")


def _gold4():
    out = []
    for line in open(GOLD4):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        vals, sz, codes, bts = [s.split() for s in line.split("|")]
        out.append(([float(v) for v in vals], float(sz[0]), float(sz[1]), [int(c) for c in codes],
                    [int(b, 16) for b in bts]))
    return out


@pytest.mark.parametrize("vals,scale,zero,codes,packed", _gold4())
def test_worked_examples_4bit(vals, scale, zero, codes, packed):
    x = f32_to_bf16_bits(np.array(vals, np.float32))
    assert np.array_equal(bf16_bits_to_f64(x), np.array(vals))  # the fixture is bf16-exact
    s, z, c = oracle.quantize_group(x, bits=4)
    assert oracle.bf16_to_f32(s) == scale and oracle.bf16_to_f32(z) == zero
    assert c.tolist() == codes
    assert oracle.pack4(c).tolist() == packed


def test_pack4_unpack4_all_bytes():
    allb = np.arange(256, dtype=np.uint8)
    codes = oracle.unpack4(allb)
    assert codes.max() == 15 and codes.size == 512
    assert np.array_equal(oracle.pack4(codes), allb)
    assert np.array_equal(codes[0::2], allb & 15) and np.array_equal(codes[1::2], allb >> 4)


@pytest.mark.parametrize("n", [32, 64])
@pytest.mark.parametrize("spread", [1.0, 10.0, 1e-3, 300.0])
def test_round_trip_bound_and_order_4bit(n, spread):
    rng = np.random.default_rng(4321 + n)
    for trial in range(200):
        x = f32_to_bf16_bits((rng.standard_normal(n) * spread + rng.standard_normal() * spread).astype(np.float32))
        s, z, c = oracle.quantize_group(x, bits=4)
        xv = bf16_bits_to_f64(x)
        sv, zv = oracle.bf16_to_f32(s), oracle.bf16_to_f32(z)
        assert zv == xv.min()
        assert abs(sv - (xv.max() - xv.min()) / 15) <= 2.0 ** -8 * sv
        xh = zv + c.astype(np.float64) * sv
        # half a step, plus what the bf16 rounding of the step can move the top of the grid (15 steps)
        assert np.all(np.abs(xv - xh) <= sv / 2 * (1 + 1e-6) + 15 * sv * 2.0 ** -8)
        assert c[np.argmin(xv)] == 0 and c[np.argmax(xv)] == 15
        order = np.argsort(xv, kind="stable")
        assert np.all(np.diff(c[order].astype(int)) >= 0)
        # the finer grid is never worse than the 2-bit one by more than its own half step
        s2, z2, c2 = oracle.quantize_group(x)
        e2 = np.abs(xv - (oracle.bf16_to_f32(z2) + c2.astype(np.float64) * oracle.bf16_to_f32(s2))).max()
        assert np.abs(xv - xh).max() <= e2 + sv


def test_lattice_groups_round_trip_exactly_4bit():
    # x = zero + k * step with a power-of-two step: scale is exact and every value is a grid point
    rng = np.random.default_rng(7)
    for step in (0.5, 2.0 ** -6, 4.0):
        for trial in range(50):
            k = rng.integers(0, 16, 32)
            k[0], k[1] = 0, 15
            zero = float(rng.integers(-8, 8)) * step
            vals = (zero + k * step).astype(np.float32)
            x = f32_to_bf16_bits(vals)
            if not np.array_equal(bf16_bits_to_f64(x), vals.astype(np.float64)):
                continue
            s, z, c = oracle.quantize_group(x, bits=4)
            assert oracle.bf16_to_f32(s) == step and oracle.bf16_to_f32(z) == zero
            assert np.array_equal(c, k.astype(np.uint8))


def test_cache_4bit_grouping_and_image_sizes():
    B, Hq, Hkv, D, W, G = 1, 2, 1, 128, 32, 32
    rng = np.random.default_rng(9)
    n = 3 * W + 1
    k = f32_to_bf16_bits(rng.standard_normal((B, Hkv, n, D)).astype(np.float32))
    v = f32_to_bf16_bits(rng.standard_normal((B, Hkv, n, D)).astype(np.float32))
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G, bits=4)
    oc.append(k, v)
    img = oc.export()
    assert img["k_codes"].shape == (B, Hkv, W, D // 2) and img["v_codes"].shape == (B, Hkv, W, D // 2)
    ev = img["quant_ids"]
    assert ev.tolist() == list(range(1, 2 * W, 2))
    # keys: one group = G removed tokens of one channel; values: G channels of one token
    kc = oracle.unpack4(img["k_codes"].reshape(-1)).reshape(W, D)
    vc = oracle.unpack4(img["v_codes"].reshape(-1)).reshape(W, D)
    for d in (0, 17, 127):
        s, z, c = oracle.quantize_group(k[0, 0, ev[:G], d], bits=4)
        assert (s, z) == (img["k_scale"][0, 0, 0, d], img["k_zero"][0, 0, 0, d])
        assert np.array_equal(c, kc[:G, d])
    for e in (0, 5, W - 1):
        for g in range(D // G):
            s, z, c = oracle.quantize_group(v[0, 0, ev[e], g * G:(g + 1) * G], bits=4)
            assert (s, z) == (img["v_scale"][0, 0, e, g], img["v_zero"][0, 0, e, g])
            assert np.array_equal(c, vc[e, g * G:(g + 1) * G])
    # attention over the dequantised rows agrees with the dense definition on those rows
    q = f32_to_bf16_bits(rng.standard_normal((B, Hq, D)).astype(np.float32))
    out = oc.attention(q, 1 / np.sqrt(D))
    K, V = oc.dense_rows(0, 0)
    ref = oracle.attention_dense(bf16_bits_to_f64(q[0, 1]), K, V, 1 / np.sqrt(D))
    assert np.allclose(out[0, 1], ref, rtol=0, atol=1e-12)
    # 4-bit rows are closer to the originals than 2-bit rows
    oc2 = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    oc2.append(k, v)
    K2, _ = oc2.dense_rows(0, 0)
    orig = bf16_bits_to_f64(k[0, 0, ev])
    nf = oc.n_fp
    assert np.abs(K[nf:] - orig).max() < np.abs(K2[nf:] - orig).max() / 3


# ---- W not a multiple of G: key groups span overflow steps -------------------------------------
@pytest.mark.parametrize("W,G", [(42, 64), (85, 64), (48, 32), (21, 32)])
def test_key_groups_across_overflow_steps(W, G):
    """The paper's own settings (G = 64, W = 42 or 85) give no whole key groups per overflow step.  Reading:
    removed tokens wait at original precision, in removal order, until G of them form a key group.  Pins: the
    id sets follow from the (separately pinned) filter in closed form, a group that spans two steps has the
    codes of the stand-alone quantiser on the original rows, and attention is the dense definition."""
    B, Hq, Hkv, D = 1, 2, 1, 128
    rng = np.random.default_rng(W * 100 + G)
    oc = oracle.OracleCache(B, Hq, Hkv, D, W, G)
    n_total = 0
    ks, vs = [], []
    for step in (3 * W, 1, W, 2 * W + 7, 5, 3 * W):
        k = f32_to_bf16_bits(rng.standard_normal((B, Hkv, step, D)).astype(np.float32))
        v = f32_to_bf16_bits(rng.standard_normal((B, Hkv, step, D)).astype(np.float32))
        oc.append(k, v)
        ks.append(k); vs.append(v)
        n_total += step
        kept, removed, n_ev = oracle.filter_ids(W, n_total)
        nq = len(removed) // G * G
        img = oc.export()
        assert oc.n_events == n_ev and oc.n_quant == nq and oc.n_fp == n_total - nq
        assert img["quant_ids"].tolist() == removed[:nq].tolist()
        assert img["kept_ids"].tolist() == sorted(kept.tolist() + removed[nq:].tolist())
    K_all = np.concatenate(ks, axis=2)[0, 0]
    V_all = np.concatenate(vs, axis=2)[0, 0]
    # full-precision rows are the original rows of their ids
    assert np.array_equal(img["fp_k"][0, 0], K_all[img["kept_ids"]])
    assert np.array_equal(img["fp_v"][0, 0], V_all[img["kept_ids"]])
    # every key group (several span two overflow steps) against the stand-alone quantiser
    kc = oracle.unpack2(img["k_codes"].reshape(-1)).reshape(nq, D)
    vc = oracle.unpack2(img["v_codes"].reshape(-1)).reshape(nq, D)
    qids = img["quant_ids"]
    for grp in range(nq // G):
        ids = qids[grp * G:(grp + 1) * G]
        for d in (0, 63, 127):
            s, z, c = oracle.quantize_group(K_all[ids, d])
            assert (s, z) == (img["k_scale"][0, 0, grp, d], img["k_zero"][0, 0, grp, d])
            assert np.array_equal(c, kc[grp * G:(grp + 1) * G, d])
    for e in (0, nq // 2, nq - 1):
        for g in range(D // G):
            s, z, c = oracle.quantize_group(V_all[qids[e], g * G:(g + 1) * G])
            assert (s, z) == (img["v_scale"][0, 0, e, g], img["v_zero"][0, 0, e, g])
            assert np.array_equal(c, vc[e, g * G:(g + 1) * G])
    q = f32_to_bf16_bits(rng.standard_normal((B, Hq, D)).astype(np.float32))
    out = oc.attention(q, 1 / np.sqrt(D))
    K, V = oc.dense_rows(0, 0)
    assert K.shape[0] == n_total
    ref = oracle.attention_dense(bf16_bits_to_f64(q[0, 0]), K, V, 1 / np.sqrt(D))
    assert np.allclose(out[0, 0], ref, rtol=0, atol=1e-12)
