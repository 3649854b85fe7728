"""Pins for the arithmetic oracle: exact special cases, closed forms and brute
force in plain Python on tiny shapes."""
import math
from fractions import Fraction

import numpy as np

from oracle import decode as od
from oracle import linalg as ol
from paper_2609_13592_b200 import synth


def bits(values):
    return synth.f32_to_bf16_bits(np.asarray(values, dtype=np.float32))


def bf16_value(b):
    """Decode one bf16 bit pattern by hand: sign, 8-bit exponent, 7-bit mantissa."""
    b = int(b)
    sign = -1 if b >> 15 else 1
    exp = (b >> 7) & 0xFF
    man = b & 0x7F
    if exp == 0:
        return sign * Fraction(man, 128) * Fraction(2) ** (-126)
    return sign * (1 + Fraction(man, 128)) * Fraction(2) ** (exp - 127)


def test_bf16_widening_matches_hand_decoding():
    pats = np.array([0x3F80, 0xC000, 0x3DCD, 0x0000, 0x8000, 0x4049, 0x3F81, 0x0080, 0x7F7F], dtype=np.uint16)
    got = ol.bf16_bits_to_f64(pats)
    for g, p in zip(got, pats):
        assert Fraction(float(g)) == bf16_value(p)
    assert got[0] == 1.0 and got[1] == -2.0


def test_bf16_rounding_ties_to_even_and_roundtrip():
    one = 1.0
    ulp = 2.0 ** -7
    cases = {
        one + ulp / 2: 0x3F80,            # midpoint between 1 and 1+ulp -> even mantissa (0)
        one + 3 * ulp / 2: 0x3F82,        # midpoint between 0x3F81 and 0x3F82 -> even
        one + ulp / 2 + 2.0 ** -30: 0x3F81,   # just above the midpoint
        one + ulp / 2 - 2.0 ** -30: 0x3F80,   # just below
        -(one + ulp / 2): 0xBF80,
        0.0: 0x0000,
        3.140625: 0x4049,
    }
    for x, want in cases.items():
        assert int(ol.f64_to_bf16_bits(np.array([x]))[0]) == want, x
    allbits = np.arange(0x0080, 0x7F80, 7, dtype=np.uint16)      # positive normals
    assert np.array_equal(ol.f64_to_bf16_bits(ol.bf16_bits_to_f64(allbits)), allbits)
    # direct rounding agrees with the generator's float32 path on float32 inputs
    x = np.random.default_rng(0).standard_normal(5000).astype(np.float32)
    assert np.array_equal(ol.f64_to_bf16_bits(x.astype(np.float64)), synth.f32_to_bf16_bits(x))


def test_gemm_brute_force_exact_rationals():
    x = synth.normal_bf16((3, 16), 1.0, 11)
    w = synth.normal_bf16((8, 16), 0.02, 12)
    y = ol.gemm(x, w)
    for m in range(3):
        for n in range(8):
            exact = sum(bf16_value(x[m, k]) * bf16_value(w[n, k]) for k in range(16))
            assert abs(y[m, n] - float(exact)) <= 1e-15 * max(1.0, abs(float(exact)))
    # vector form
    assert np.allclose(ol.gemm(x[0], w), y[0], rtol=0, atol=0)


def test_gemm_identity_onehot_and_transpose_sensitivity():
    n = 32
    eye = bits(np.eye(n))
    x = synth.normal_bf16((2, n), 1.0, 5)
    assert np.array_equal(ol.gemm(x, eye), ol.bf16_bits_to_f64(x))
    w = synth.normal_bf16((7, n), 1.0, 6)
    e3 = bits(np.eye(n)[3])
    assert np.array_equal(ol.gemm(e3, w), ol.bf16_bits_to_f64(w[:, 3]))   # picks column 3 of W
    # integer-valued inputs give exact integers
    xi = bits(np.arange(-8, 8).reshape(1, 16))
    wi = bits(np.arange(16 * 4).reshape(4, 16) % 5 - 2)
    want = (np.arange(-8, 8).reshape(1, 16) @ (np.arange(64).reshape(4, 16) % 5 - 2).T).astype(np.float64)
    assert np.array_equal(ol.gemm(xi, wi), want)


def test_stream_sum_against_integer_arithmetic():
    page_elems = 4096
    n = 5 * page_elems + 100
    vals = synth.small_int_values(0, n)
    per_page, total = ol.stream_sum(synth.small_int_bf16(0, n), page_elems)
    assert len(per_page) == 6
    for p in range(6):
        assert per_page[p] == float(vals[p * page_elems:(p + 1) * page_elems].sum())
    assert total == float(vals.sum())
    assert vals.min() == -4 and vals.max() == 4


def make_cache(n_heads, n_blocks, d, seed):
    k = synth.normal_bf16((n_heads, n_blocks, ol.BLOCK_TOKENS, d), 1.0, seed)
    v = synth.normal_bf16((n_heads, n_blocks, ol.BLOCK_TOKENS, d), 1.0, seed + 1)
    return k, v


def test_attention_brute_force_tiny():
    d, hq, hkv = 8, 2, 1
    k, v = make_cache(hkv, 5, d, 21)
    q = synth.normal_bf16((1, hq, d), 1.0, 23)
    table = [[4, 0, 2]]
    for ctx in (1, 15, 16, 17, 40):
        scale = 0.37
        out = ol.paged_attention_decode(q, k, v, table, [ctx], scale)
        for j in range(hq):
            s = []
            rows = []
            for t in range(ctx):
                blk, slot = table[0][t // 16], t % 16
                kr = [float(bf16_value(k[0, blk, slot, i])) for i in range(d)]
                rows.append([float(bf16_value(v[0, blk, slot, i])) for i in range(d)])
                s.append(scale * sum(float(bf16_value(q[0, j, i])) * kr[i] for i in range(d)))
            mx = max(s)
            e = [math.exp(si - mx) for si in s]
            z = sum(e)
            for i in range(d):
                want = sum(e[t] / z * rows[t][i] for t in range(ctx))
                assert abs(out[0, j, i] - want) < 1e-12


def test_attention_special_cases():
    d, hq, hkv = 128, 8, 2
    k, v = make_cache(hkv, 8, d, 31)
    q = synth.normal_bf16((2, hq, d), 1.0, 33)
    table = np.array([[3, 1, 7, 0], [2, 5, 6, 4]])
    scale = 1 / math.sqrt(d)
    # ctx = 1 -> the single V row of the right KV head (consecutive query heads share a KV head)
    out = ol.paged_attention_decode(q, k, v, table, [1, 1], scale)
    for b in range(2):
        for j in range(hq):
            assert np.array_equal(out[b, j], ol.bf16_bits_to_f64(v[j // 4, table[b, 0], 0]))
    # all keys equal -> uniform weights -> mean of V
    k_same = k.copy()
    k_same[:] = k[0, 0, 0]
    out = ol.paged_attention_decode(q, k_same, v, table, [40, 23], scale)
    vv = ol.bf16_bits_to_f64(v[1, table[1, :2]]).reshape(-1, d)[:23]
    assert np.allclose(out[1, 5], vv.mean(axis=0), rtol=0, atol=1e-14)
    # one dominant key -> its V row
    k_dom = np.zeros_like(k)
    big = bits(np.full(d, 30.0))
    k_dom[0, table[0, 1], 3] = big
    q_pos = np.broadcast_to(bits(np.ones(d)), (2, hq, d)).copy()
    out = ol.paged_attention_decode(q_pos, k_dom, v, table, [40, 40], 1.0)
    assert np.allclose(out[0, 0], ol.bf16_bits_to_f64(v[0, table[0, 1], 3]), rtol=0, atol=1e-12)
    # ctx = 0 gives zeros
    out = ol.paged_attention_decode(q, k, v, table, [0, 5], scale)
    assert not out[0].any() and out[1].any()


def test_attention_invariant_under_block_renaming():
    d, hq, hkv = 16, 4, 2
    k, v = make_cache(hkv, 6, d, 41)
    q = synth.normal_bf16((1, hq, d), 1.0, 43)
    table = np.array([[0, 1, 2]])
    out = ol.paged_attention_decode(q, k, v, table, [37], 0.25)
    perm = np.array([5, 3, 4, 0, 2, 1])                      # block i moves to perm[i]
    k2, v2 = np.zeros_like(k), np.zeros_like(v)
    k2[:, perm], v2[:, perm] = k, v
    out2 = ol.paged_attention_decode(q, k2, v2, perm[table], [37], 0.25)
    assert np.array_equal(out, out2)
    # tokens beyond ctx do not matter
    k3 = k.copy()
    k3[:, 2, 5:] = bits(np.full(d, 99.0))
    assert np.array_equal(out, ol.paged_attention_decode(q, k3, v, table, [37], 0.25))


def test_rmsnorm_rope_silu_special_cases():
    ones_w = bits(np.ones(64))
    x = np.full((2, 64), 3.0)
    y = od.rmsnorm(x, ones_w, eps=0.0)
    assert np.allclose(y, 1.0, rtol=0, atol=1e-15)            # constant row -> all ones
    xr = np.random.default_rng(1).standard_normal((3, 64))
    y = od.rmsnorm(xr, ones_w, eps=0.0)
    assert np.allclose((y * y).mean(axis=-1), 1.0)            # unit mean square
    assert np.allclose(od.rmsnorm(2 * xr, ones_w, eps=0.0), y)  # scale invariant
    w2 = bits(np.full(64, 2.0))
    assert np.allclose(od.rmsnorm(xr, w2, eps=0.0), 2 * y)
    # RoPE: identity at position 0, a rotation (norm preserved), relative-position property
    h = np.random.default_rng(2).standard_normal((1, 2, 128))
    assert np.array_equal(od.rope(h, [0]), h)
    r = od.rope(h, [1234])
    assert np.allclose((r * r).sum(-1), (h * h).sum(-1))
    g = np.random.default_rng(3).standard_normal((1, 2, 128))
    d1 = (od.rope(h, [100]) * od.rope(g, [60])).sum(-1)
    d2 = (od.rope(h, [1040]) * od.rope(g, [1000])).sum(-1)
    assert np.allclose(d1, d2, rtol=1e-9)
    # lowest-frequency pair (i = D/2 - 1 with i + D/2): angle = pos * base^(-(D-2)/D)
    e = np.zeros((1, 1, 128))
    e[0, 0, 63] = 1.0
    ang = 7 * od.ROPE_BASE ** (-126 / 128)
    r = od.rope(e, [7])
    assert abs(r[0, 0, 63] - math.cos(ang)) < 1e-15 and abs(r[0, 0, 127] - math.sin(ang)) < 1e-15
    # pair 0 rotates by pos radians
    e = np.zeros((1, 1, 128))
    e[0, 0, 0] = 1.0
    r = od.rope(e, [2])
    assert abs(r[0, 0, 0] - math.cos(2)) < 1e-15 and abs(r[0, 0, 64] - math.sin(2)) < 1e-15
    assert od.silu(np.array([0.0]))[0] == 0.0
    assert abs(od.silu(np.array([1.0]))[0] - 1 / (1 + math.exp(-1))) < 1e-15
    assert abs(od.silu(np.array([-40.0]))[0]) < 1e-15 and abs(od.silu(np.array([40.0]))[0] - 40) < 1e-12


def test_decode_step_reduces_to_known_cases():
    cfg = dict(synth.TINY_LLAMA)
    w = synth.llama_weights(cfg, 3)
    n_seq, n_blocks = 3, 8
    hkv, d = cfg["n_kv_heads"], cfg["head_dim"]
    kc = [np.zeros((hkv, n_blocks, 16, d), np.uint16) for _ in range(cfg["n_layers"])]
    vc = [np.zeros((hkv, n_blocks, 16, d), np.uint16) for _ in range(cfg["n_layers"])]
    table = np.array([[0, 1], [2, 3], [4, 5]])
    tokens = np.array([5, 77, 300])
    # with zero output and down projections every layer is the identity on the residual
    # stream: logits = rmsnorm(embed[token]) @ lm_head^T
    wz = dict(w, layers=[dict(l, wo=np.zeros_like(l["wo"]), wd=np.zeros_like(l["wd"])) for l in w["layers"]])
    out = od.decode_step(cfg, wz, tokens, kc, vc, table, [1, 1, 1])
    h0 = ol.bf16_bits_to_f64(w["embed"][tokens])
    # textbook RMSNorm then the product, nothing rounded: the step's factored form (norm weight
    # folded into the matrix with one bf16 rounding) must agree to that rounding
    want = od.rmsnorm(h0, w["norm_f"]) @ ol.bf16_bits_to_f64(w["lm_head"]).T
    # Derived bound.  The two forms differ only in the one rounding of W[n,k] * gamma[k] to bf16,
    # which moves each product by at most half a bf16 ulp, i.e. by 2^-9 of its size (round to
    # nearest, 8 significant bits).  The logit is rs * sum_k h[k] * (W * gamma)[n,k], so element
    # (m, n) can move by at most 2^-9 * rs[m] * sum_k |h[m,k]| * |W[n,k] * gamma[k]|.
    wg = np.abs(ol.bf16_bits_to_f64(w["lm_head"]) * ol.bf16_bits_to_f64(w["norm_f"])[None, :])
    rs0 = 1.0 / np.sqrt((h0 * h0).mean(-1, keepdims=True) + od.RMS_EPS)
    bound = 2.0 ** -9 * rs0 * (np.abs(h0) @ wg.T)
    assert (np.abs(out["logits"] - want) <= bound * (1 + 1e-9) + 1e-15).all()
    # That is the worst case (all roundings pushing the same way).  The roundings are independent
    # and uniform within half an ulp, so the deviation of element (m, n) has standard deviation
    # rs[m] * sqrt(sum_k h[m,k]^2 * ulp(W[n,k] gamma[k])^2 / 12), ulp(v) = 2^(floor(log2 |v|) - 7):
    # about 2^-9 of rms(logits) here.  Over the 1920 outputs the measured spread must match it;
    # a second rounding anywhere in the step would double the variance.
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(wg, 1e-300))) - 7)
    sigma = rs0 * np.sqrt((h0 * h0) @ (ulp * ulp).T / 12.0)
    z = (out["logits"] - want) / sigma
    assert 0.9 < np.sqrt((z * z).mean()) < 1.1 and np.abs(z).max() < 5.0
    assert sigma.max() < 2.0 ** -8 * np.sqrt((want ** 2).mean())
    assert np.array_equal(out["next_tokens"], out["logits"].astype(np.float32).argmax(-1))
    # the step wrote the new token's K/V at position ctx-1 of the right block and nowhere else
    assert kc[0][:, 0, 0].any() and not kc[0][:, 0, 1:].any() and not kc[0][:, 1].any()
    assert kc[0][:, 2, 0].any() and vc[1][:, 4, 0].any()
    # first step (ctx = 1): attention output equals V of the token itself
    kc2 = [np.zeros_like(a) for a in kc]
    vc2 = [np.zeros_like(a) for a in vc]
    out = od.decode_step(cfg, w, tokens, kc2, vc2, table, [1, 1, 1], keep=True)
    v_new = out["qkv"][:, (cfg["n_q_heads"] + hkv) * d:].reshape(n_seq, hkv, d)
    attn = out["attn"].reshape(n_seq, cfg["n_q_heads"], d)
    group = cfg["n_q_heads"] // hkv
    for j in range(cfg["n_q_heads"]):
        assert np.array_equal(attn[:, j], v_new[:, j // group])
    # a second step at ctx = 2 reads what the first wrote: changing the cached token changes the logits
    out2 = od.decode_step(cfg, w, tokens, kc2, vc2, table, [2, 2, 2])
    vc3 = [a.copy() for a in vc2]
    vc3[0][:, 0, 0] = bits(np.full(d, 50.0))
    out3 = od.decode_step(cfg, w, tokens, kc2, vc3, table, [2, 2, 2])
    assert not np.array_equal(out2["logits"][0], out3["logits"][0])
    assert np.array_equal(out2["logits"][1], out3["logits"][1])
