"""Oracle: one decode step of a Llama-shaped model over a paged KV cache.

Test infrastructure only (see the package docstring).

The paper treats decode as a chain of weight-streaming matrix products and
attention kernels (Sec. 2.1; weights about 70 % and attention about 30 % of the
time, Sec. 5.4) and says nothing about the small operators between them.  The
layer structure below is the public Llama-3 architecture; its constants -
RMSNorm epsilon 1e-5, RoPE base 500000 with the "rotate-half" pairing
(element i pairs with i + D/2) - are choices of this repository: the three
constants are parity unpinned by the paper.  The structure of the step itself
(row ranges, pairing, append position, head mapping, residual adds, both row
scales, gate/up order, argmax ties) is pinned from outside by a restatement
with plain loops over scalars on a tiny model, and by textbook special cases.

All arithmetic is fp64.  Tensors that the device path stores as bf16 between
kernels are rounded to bf16 here at the same places (marked "-> bf16"), so that
32 layers of rounding do not separate the two; logits stay unrounded.

RMSNorm in the step is evaluated in its factored form, the way an inference
engine prepares a model for decoding: the norm weight is folded into the matrix
it feeds when the model is loaded, W' = bf16(W * gamma) (one rounding, at load
time), and the step computes rs * (h W'^T) with rs = 1/sqrt(mean(h^2) + eps)
taken from the bf16 residual stream h.  This is x*rsqrt(mean(x^2)+eps)*gamma
followed by the product, with the normalised activations never stored; the
paper is silent on all of this (it treats decode as weight products plus
attention), so the choice is this repository's and is stated in its design notes.
"""
import numpy as np

from .linalg import (BLOCK_TOKENS, bf16_bits_to_f64, f64_to_bf16_bits,
                     paged_attention_decode)

RMS_EPS = 1e-5
ROPE_BASE = 500000.0


def _round_bf16(x):
    bits = f64_to_bf16_bits(x)
    return bits, bf16_bits_to_f64(bits)


def rmsnorm(x, weight_bits, eps=RMS_EPS):
    """x * rsqrt(mean(x^2) + eps) * w, row-wise.  x: fp64 [B, H]."""
    w = bf16_bits_to_f64(weight_bits)
    ms = (x * x).mean(axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * w


def rope(x, positions, base=ROPE_BASE):
    """Rotary embedding, rotate-half pairing.  x: fp64 [B, n_heads, D]."""
    d = x.shape[-1]
    half = d // 2
    inv_freq = base ** (-np.arange(half, dtype=np.float64) * 2.0 / d)
    ang = np.asarray(positions, dtype=np.float64)[:, None, None] * inv_freq[None, None, :]
    c, s = np.cos(ang), np.sin(ang)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def fold_norm_weight(w_bits, gamma_bits):
    """W' = bf16(W * gamma): the RMSNorm weight folded into the matrix it feeds (load time)."""
    return f64_to_bf16_bits(bf16_bits_to_f64(w_bits) * bf16_bits_to_f64(gamma_bits)[None, :])


def rms_scale(x, eps=RMS_EPS):
    """1 / sqrt(mean(x^2) + eps), row-wise.  x: fp64 [B, H] -> [B, 1]."""
    return 1.0 / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)


def silu(x):
    return x / (1.0 + np.exp(-x))


def decode_step(cfg, weights, tokens, k_caches, v_caches, block_table, ctx_lens,
                n_layers=None, keep=False):
    """Run one decode step for B sequences.

    cfg: dict(hidden, ffn, n_q_heads, n_kv_heads, head_dim, vocab, n_layers).
    weights: dict with 'embed' [V, hidden], 'norm_f' [hidden], 'lm_head'
    [V, hidden] and 'layers' = list of dicts with 'norm1', 'wqkv'
    [(Hq + 2 Hkv) D, hidden] (q rows, then k rows, then v rows), 'wo'
    [hidden, Hq D], 'norm2', 'wgu' [2 F, hidden] (gate rows then up rows),
    'wd' [hidden, F]; all uint16 bf16 bit patterns.
    k_caches / v_caches: per layer uint16 [Hkv, N_blocks, 16, D]; the new
    token's K and V are written into them (position ctx_lens[b] - 1).
    ctx_lens counts the new token.  Returns dict(logits fp64 [B, V],
    next_tokens int64 [B]) plus intermediates when keep=True.
    """
    hq, hkv, d = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    n_layers = cfg["n_layers"] if n_layers is None else n_layers
    tokens = np.asarray(tokens, dtype=np.int64)
    ctx_lens = np.asarray(ctx_lens, dtype=np.int64)
    n_seq = tokens.shape[0]
    pos = ctx_lens - 1
    scale = 1.0 / np.sqrt(float(d))
    trace = {}

    h = bf16_bits_to_f64(weights["embed"][tokens])              # [B, hidden], bf16 values
    for li in range(n_layers):
        lw = weights["layers"][li]
        wqkv = bf16_bits_to_f64(fold_norm_weight(lw["wqkv"], lw["norm1"]))     # load-time fold -> bf16
        _, qkv = _round_bf16(rms_scale(h) * (h @ wqkv.T))        # rmsnorm + product -> bf16
        q = qkv[:, :hq * d].reshape(n_seq, hq, d)
        k = qkv[:, hq * d:(hq + hkv) * d].reshape(n_seq, hkv, d)
        v = qkv[:, (hq + hkv) * d:].reshape(n_seq, hkv, d)
        q_bits, _ = _round_bf16(rope(q, pos))                    # -> bf16
        k_bits, _ = _round_bf16(rope(k, pos))                    # -> bf16
        v_bits = f64_to_bf16_bits(v)                             # already bf16 values
        for b in range(n_seq):                                   # append to the paged cache
            blk = int(block_table[b][pos[b] // BLOCK_TOKENS])
            slot = int(pos[b] % BLOCK_TOKENS)
            k_caches[li][:, blk, slot, :] = k_bits[b]
            v_caches[li][:, blk, slot, :] = v_bits[b]
        attn = paged_attention_decode(q_bits, k_caches[li], v_caches[li],
                                      block_table, ctx_lens, scale)
        _, attn = _round_bf16(attn.reshape(n_seq, hq * d))       # -> bf16
        _, h = _round_bf16(h + attn @ bf16_bits_to_f64(lw["wo"]).T)   # residual -> bf16
        wgu = bf16_bits_to_f64(fold_norm_weight(lw["wgu"], lw["norm2"]))       # load-time fold -> bf16
        _, gu = _round_bf16(rms_scale(h) * (h @ wgu.T))          # rmsnorm + product -> bf16
        f = gu.shape[1] // 2
        _, act = _round_bf16(silu(gu[:, :f]) * gu[:, f:])        # -> bf16
        _, h = _round_bf16(h + act @ bf16_bits_to_f64(lw["wd"]).T)    # residual -> bf16
        if keep:
            trace[f"h{li}"] = h.copy()
            if li == 0:
                trace.update(qkv=qkv, q_rope=bf16_bits_to_f64(q_bits),
                             k_rope=bf16_bits_to_f64(k_bits), attn=attn, act=act)
    w_head = bf16_bits_to_f64(fold_norm_weight(weights["lm_head"], weights["norm_f"]))   # load-time fold -> bf16
    logits = rms_scale(h) * (h @ w_head.T)                       # fp64, not rounded
    # The device takes the argmax of fp32 logits: decide in that precision, lowest index on ties.
    next_tokens = np.argmax(logits.astype(np.float32), axis=-1).astype(np.int64)
    out = {"logits": logits, "next_tokens": next_tokens, "h_final": h}
    out.update(trace)
    return out
