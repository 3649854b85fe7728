"""Pin of oracle.decode.decode_step from the outside: one whole decode step of a tiny
Llama-shaped model recomputed with plain Python loops over scalars.

Nothing here imports the oracle's helpers for the arithmetic: bf16 values are decoded and
rounded with integer operations on IEEE bit patterns, sums are `for` loops, the only library
calls are math.sqrt / exp / cos / sin.  The structure written out below is the public
Llama-3 layer (the paper fixes none of it: it treats decode as weight products plus
attention, Sec. 2.1):

    rs1 = 1/sqrt(mean(h^2) + eps);  qkv = bf16(rs1 * (h W'qkv^T)),  W' = bf16(W * gamma1)
    rows of wqkv: q heads, then k heads, then v heads;  rotate-half RoPE on q and k at
    position ctx - 1 (element i pairs with i + D/2, angle pos * base^(-2i/D)), -> bf16
    k, v appended to block table[b][pos // 16], slot pos % 16
    attention of q head j over KV head j // (Hq / Hkv), all ctx tokens, -> bf16
    h = bf16(h + attn Wo^T)
    gu = bf16(rs2 * (h W'gu^T)); rows of wgu: gate rows, then up rows
    act = bf16(silu(gate) * up);  h = bf16(h + act Wd^T)
    logits = rsf * (h W'head^T);  next token = argmax of the fp32 logits, lowest index on ties

Which slip trips what: every `slip` below is one plausible mistake put into the scalar
restatement; test_each_slip_is_caught shows that each one moves the logits far outside the
agreement that test_decode_step_matches_scalar_restatement demands, so the same mistake
in the oracle would fail that test:
    gate_up_swapped     silu taken of the up rows instead of the gate rows
    q_k_swapped         q read from the k row range and k from the q row range
    no_residual_attn    h = attn Wo^T without the residual add
    no_residual_mlp     h = act Wd^T without the residual add
    no_second_rms       gate/up product without its row scale
    no_final_rms        logits without the final row scale
    rope_interleaved    RoPE pairing (2i, 2i+1) instead of (i, i + D/2)
    rope_sign           rotation by the negative angle
    append_off_by_one   new K/V written at position ctx instead of ctx - 1
    gqa_modulo          q head j reads KV head j % Hkv instead of j // (Hq / Hkv)
    no_softmax_scale    scores without the 1/sqrt(D) factor
    norm_not_folded     gamma left out of the weight product
    v_not_appended      attention reads the cache without the new token's V
"""
import math
import struct

import numpy as np
import pytest

from oracle import decode as od

EPS = 1e-5
BASE = 500000.0


def bf16_to_float(bits):
    """bf16 bit pattern -> Python float, by widening the pattern to an IEEE float32."""
    return struct.unpack("<f", struct.pack("<I", (int(bits) & 0xFFFF) << 16))[0]


def round_to_bf16(x):
    """Nearest bf16 value of a Python float (ties to even) in ONE rounding, on the IEEE
    double's bit pattern: keep sign, exponent and the top 7 fraction bits, round on the 45
    bits below.  Values here are normal and far from overflow."""
    if x == 0.0:
        return 0.0
    u = struct.unpack("<Q", struct.pack("<d", x))[0]
    low = u & ((1 << 45) - 1)
    u >>= 45
    half = 1 << 44
    if low > half or (low == half and (u & 1)):
        u += 1                       # a carry out of the fraction moves into the exponent: still right
    return struct.unpack("<d", struct.pack("<Q", u << 45))[0]


def scalar_decode_step(cfg, w, tokens, k_cache, v_cache, table, ctx_lens, slip=None):
    """One decode step with loops over scalars.  w: nested lists of Python floats (bf16 values);
    k_cache / v_cache: per layer [Hkv][n_blocks][16][D] nested lists, updated in place.
    Returns (logits [B][V], next tokens [B])."""
    hq, hkv, d = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    hid, ffn, vocab = cfg["hidden"], cfg["ffn"], cfg["vocab"]
    half = d // 2
    group = hq // hkv
    all_logits, nxt = [], []
    for b, tok in enumerate(tokens):
        ctx = ctx_lens[b]
        pos = ctx - 1
        h = list(w["embed"][tok])
        for li in range(cfg["n_layers"]):
            lw = w["layers"][li]
            ms = sum(v * v for v in h) / hid
            rs = 1.0 / math.sqrt(ms + EPS)
            qkv = []
            for n in range((hq + 2 * hkv) * d):
                s = 0.0
                for k in range(hid):
                    g = 1.0 if slip == "norm_not_folded" else lw["norm1"][k]
                    s += h[k] * round_to_bf16(lw["wqkv"][n][k] * g)
                qkv.append(round_to_bf16(rs * s))
            q_lo, k_lo, v_lo = 0, hq * d, (hq + hkv) * d
            if slip == "q_k_swapped":          # only meaningful when hq == hkv; else shift the ranges
                q_lo, k_lo = hkv * d, 0
            q = [[qkv[q_lo + j * d + i] for i in range(d)] for j in range(hq)]
            kn = [[qkv[k_lo + j * d + i] for i in range(d)] for j in range(hkv)]
            vn = [[qkv[v_lo + j * d + i] for i in range(d)] for j in range(hkv)]

            def rotate(vec):
                out = [0.0] * d
                for i in range(half):
                    ang = pos * BASE ** (-2.0 * i / d)
                    if slip == "rope_sign":
                        ang = -ang
                    c, s_ = math.cos(ang), math.sin(ang)
                    i1, i2 = (2 * i, 2 * i + 1) if slip == "rope_interleaved" else (i, i + half)
                    out[i1] = round_to_bf16(vec[i1] * c - vec[i2] * s_)
                    out[i2] = round_to_bf16(vec[i2] * c + vec[i1] * s_)
                return out

            q = [rotate(v) for v in q]
            kn = [rotate(v) for v in kn]
            wpos = pos + 1 if slip == "append_off_by_one" else pos
            blk, slot = table[b][wpos // 16], wpos % 16
            for g in range(hkv):
                k_cache[li][g][blk][slot] = list(kn[g])
                if slip != "v_not_appended":
                    v_cache[li][g][blk][slot] = list(vn[g])
            scale = 1.0 if slip == "no_softmax_scale" else 1.0 / math.sqrt(d)
            attn = []
            for j in range(hq):
                g = j % hkv if slip == "gqa_modulo" else j // group
                scores = []
                for t in range(ctx):
                    krow = k_cache[li][g][table[b][t // 16]][t % 16]
                    scores.append(scale * sum(q[j][i] * krow[i] for i in range(d)))
                mx = max(scores)
                p = [math.exp(s - mx) for s in scores]
                z = sum(p)
                for i in range(d):
                    o = 0.0
                    for t in range(ctx):
                        o += p[t] / z * v_cache[li][g][table[b][t // 16]][t % 16][i]
                    attn.append(round_to_bf16(o))
            h_new = []
            for n in range(hid):
                s = sum(attn[k] * lw["wo"][n][k] for k in range(hq * d))
                h_new.append(round_to_bf16(s if slip == "no_residual_attn" else h[n] + s))
            h = h_new
            ms = sum(v * v for v in h) / hid
            rs = 1.0 if slip == "no_second_rms" else 1.0 / math.sqrt(ms + EPS)
            gu = []
            for n in range(2 * ffn):
                s = 0.0
                for k in range(hid):
                    s += h[k] * round_to_bf16(lw["wgu"][n][k] * lw["norm2"][k])
                gu.append(round_to_bf16(rs * s))
            gate, up = gu[:ffn], gu[ffn:]
            if slip == "gate_up_swapped":
                gate, up = up, gate
            act = [round_to_bf16(gate[i] / (1.0 + math.exp(-gate[i])) * up[i]) for i in range(ffn)]
            h_new = []
            for n in range(hid):
                s = sum(act[k] * lw["wd"][n][k] for k in range(ffn))
                h_new.append(round_to_bf16(s if slip == "no_residual_mlp" else h[n] + s))
            h = h_new
        ms = sum(v * v for v in h) / hid
        rs = 1.0 if slip == "no_final_rms" else 1.0 / math.sqrt(ms + EPS)
        logits = []
        for n in range(vocab):
            s = 0.0
            for k in range(hid):
                s += h[k] * round_to_bf16(w["lm_head"][n][k] * w["norm_f"][k])
            logits.append(rs * s)
        all_logits.append(logits)
        f32 = [struct.unpack("<f", struct.pack("<f", v))[0] for v in logits]
        best = 0
        for n in range(1, vocab):
            if f32[n] > f32[best]:           # strict: the lowest index wins a tie
                best = n
        nxt.append(best)
    return all_logits, nxt


CFG = dict(n_layers=2, hidden=16, ffn=24, n_q_heads=4, n_kv_heads=2, head_dim=8, vocab=20)
N_BLOCKS = 6


def make_case(seed=4):
    """Random bf16 bit patterns for a tiny model, two sequences (one inside its first block,
    one whose new token opens a second block) and a cache with a random prefix."""
    rng = np.random.default_rng(seed)
    hq, hkv, d, hid, ffn, vocab = (CFG[k] for k in ("n_q_heads", "n_kv_heads", "head_dim", "hidden", "ffn", "vocab"))

    def bits(shape, std, mean=0.0):
        x = (mean + std * rng.standard_normal(shape)).astype(np.float32)
        return (x.view(np.uint32) >> 16).astype(np.uint16)        # truncation: any bf16 pattern will do

    w = {"embed": bits((vocab, hid), 1.0), "norm_f": bits(hid, 0.2, 1.0), "lm_head": bits((vocab, hid), 0.3),
         "layers": [{"norm1": bits(hid, 0.2, 1.0), "wqkv": bits(((hq + 2 * hkv) * d, hid), 0.3),
                     "wo": bits((hid, hq * d), 0.3), "norm2": bits(hid, 0.2, 1.0),
                     "wgu": bits((2 * ffn, hid), 0.3), "wd": bits((hid, ffn), 0.3)} for _ in range(CFG["n_layers"])]}
    kc = [bits((hkv, N_BLOCKS, 16, d), 1.0) for _ in range(CFG["n_layers"])]
    vc = [bits((hkv, N_BLOCKS, 16, d), 1.0) for _ in range(CFG["n_layers"])]
    table = [[4, 1], [2, 5]]
    ctx = [3, 17]
    tokens = [7, 19]
    return w, kc, vc, table, ctx, tokens


def to_floats(a):
    a = np.asarray(a)
    if a.ndim == 0:
        return bf16_to_float(a)
    return [to_floats(x) for x in a]


def run_scalar(case, slip=None):
    w, kc, vc, table, ctx, tokens = case
    wf = {k: to_floats(v) for k, v in w.items() if k != "layers"}
    wf["layers"] = [{k: to_floats(v) for k, v in lw.items()} for lw in w["layers"]]
    kf, vf = [to_floats(a) for a in kc], [to_floats(a) for a in vc]
    logits, nxt = scalar_decode_step(CFG, wf, tokens, kf, vf, table, ctx, slip)
    return np.array(logits), nxt, kf, vf


def test_bf16_helpers_against_known_patterns():
    assert bf16_to_float(0x3F80) == 1.0 and bf16_to_float(0xC000) == -2.0 and bf16_to_float(0x3DCD) == 0.10009765625
    assert round_to_bf16(1.0) == 1.0
    assert round_to_bf16(1.0 + 2.0 ** -8) == 1.0                 # tie -> even (1.0 has an even last bit)
    assert round_to_bf16(1.0 + 2.0 ** -7 + 2.0 ** -8) == 1.0 + 2.0 ** -6   # tie -> even, upwards
    assert round_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -30) == 1.0 + 2.0 ** -7
    assert round_to_bf16(-(2.0 - 2.0 ** -9)) == -2.0             # carry into the exponent
    assert round_to_bf16(0.1) == bf16_to_float(0x3DCD)


def test_decode_step_matches_scalar_restatement():
    case = make_case()
    w, kc, vc, table, ctx, tokens = case
    want, want_next, kf, vf = run_scalar(case)
    kc2, vc2 = [a.copy() for a in kc], [a.copy() for a in vc]
    out = od.decode_step(CFG, w, np.array(tokens), kc2, vc2, np.array(table), np.array(ctx))
    # same roundings at the same places: what is left is the order of fp64 sums
    assert np.allclose(out["logits"], want, rtol=1e-9, atol=1e-9)
    assert out["next_tokens"].tolist() == want_next
    for li in range(CFG["n_layers"]):
        assert np.array_equal(np.array(to_floats(kc2[li])), np.array(kf[li]))
        assert np.array_equal(np.array(to_floats(vc2[li])), np.array(vf[li]))
    # the step wrote exactly one K row and one V row per sequence, layer and KV head
    changed = sum(int((a != b).any(axis=-1).sum()) for a, b in zip(kc + vc, kc2 + vc2))
    assert changed == 2 * CFG["n_layers"] * CFG["n_kv_heads"] * len(tokens)


def test_argmax_tie_takes_lowest_index():
    case = make_case()
    w = dict(case[0])
    head = w["lm_head"].copy()
    head[13] = head[5]                                           # two identical rows: identical logits
    head[5 + 1:13] = 0
    head[:5] = 0
    head[14:] = 0
    w["lm_head"] = head
    case = (w,) + case[1:]
    want, want_next, _, _ = run_scalar(case)
    out = od.decode_step(CFG, w, np.array(case[5]), [a.copy() for a in case[1]], [a.copy() for a in case[2]],
                         np.array(case[3]), np.array(case[4]))
    for b in range(2):
        if want[b][5] > 0:                                       # otherwise a zero row wins, also the lowest
            assert want_next[b] == 5
    assert out["next_tokens"].tolist() == want_next


SLIPS = ["gate_up_swapped", "q_k_swapped", "no_residual_attn", "no_residual_mlp", "no_second_rms", "no_final_rms",
         "rope_interleaved", "rope_sign", "append_off_by_one", "gqa_modulo", "no_softmax_scale", "norm_not_folded",
         "v_not_appended"]


@pytest.mark.parametrize("slip", SLIPS)
def test_each_slip_is_caught(slip):
    case = make_case()
    good, _, _, _ = run_scalar(case)
    bad, _, _, _ = run_scalar(case, slip)
    rms = float(np.sqrt((good ** 2).mean()))
    # every sequence's logits move by far more than the agreement demanded above
    for b in range(good.shape[0]):
        assert np.abs(bad[b] - good[b]).max() > 1e-3 * rms, slip
