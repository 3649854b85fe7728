"""Oracle: the arithmetic of the decode kernels, in fp64 on the given bf16 bits.

Test infrastructure only (see the package docstring).  bf16 tensors travel as
numpy uint16 arrays holding the raw bit patterns; every function widens them
to fp64 exactly and computes in fp64.  numpy's matmul is the only library step.

The paper does not define new arithmetic: decode is made of weight-streaming
matrix products and attention over paged KV (Sec. 2.1, Sec. 3.1, Sec. 3.3), and
its micro-benchmark streams a buffer with trivial compute (Sec. 2.6).  The
functions below are therefore the textbook definitions written out.
"""
import numpy as np

BLOCK_TOKENS = 16  # tokens per KV block (Sec. 4.3)


def bf16_bits_to_f64(bits):
    """Exact widening: a bf16 is the upper half of an IEEE float32."""
    b = np.asarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x):
    """Round fp64 to the nearest bf16 (ties to even), in one rounding step.

    For a normal value with binary exponent e (x = m * 2**e, 0.5 <= |m| < 1) the
    bf16 grid spacing is 2**(e-8); x is scaled by an exact power of two, rounded
    to the nearest integer (ties to even) and scaled back.  Values here are O(1),
    far from bf16's overflow and subnormal ranges."""
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)
    q = np.ldexp(1.0, e - 8)
    r = np.rint(x / q) * q
    return (r.astype(np.float32).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def gemm(x_bits, w_bits):
    """y[m, n] = sum_k x[m, k] * W[n, k]  (weights row-major [N, K], Sec. 3.1).

    x_bits: uint16 [M_b, K] (or [K]); w_bits: uint16 [N, K]; returns fp64 [M_b, N]
    (or [N])."""
    x = bf16_bits_to_f64(x_bits)
    w = bf16_bits_to_f64(w_bits)
    return x @ w.T


def stream_sum(buf_bits, page_elems):
    """Per-page sum of a bf16 buffer (the add micro-benchmark of Sec. 2.6 with
    its trivial compute replaced by a sum).  Returns (per-page fp64, total)."""
    v = bf16_bits_to_f64(np.asarray(buf_bits).reshape(-1))
    n_pages = (v.size + page_elems - 1) // page_elems
    per_page = np.zeros(n_pages, dtype=np.float64)
    for p in range(n_pages):
        per_page[p] = v[p * page_elems:(p + 1) * page_elems].sum()
    return per_page, float(per_page.sum())


def paged_attention_decode(q_bits, k_cache_bits, v_cache_bits, block_table, ctx_lens, scale):
    """One decode step of softmax attention over a paged KV cache.

    q_bits: uint16 [B, Hq, D].  k_cache_bits / v_cache_bits: uint16
    [Hkv, N_blocks, 16, D] - heads outermost, one 16-token chunk per (head,
    block) (Sec. 4.5).  block_table: int [B, max_blocks] of block ids;
    ctx_lens: int [B].  Query head j reads KV head j // (Hq // Hkv).  The query
    attends to all ctx_lens[b] cached tokens (its own K/V are already in the
    cache).  Returns fp64 [B, Hq, D].
    """
    q = bf16_bits_to_f64(q_bits)
    n_seq, n_q_heads, d = q.shape
    n_kv_heads = k_cache_bits.shape[0]
    group = n_q_heads // n_kv_heads
    out = np.zeros((n_seq, n_q_heads, d), dtype=np.float64)
    for b in range(n_seq):
        ctx = int(ctx_lens[b])
        if ctx == 0:
            continue
        n_blk = (ctx + BLOCK_TOKENS - 1) // BLOCK_TOKENS
        blocks = np.asarray(block_table[b][:n_blk], dtype=np.int64)
        for g in range(n_kv_heads):
            k = bf16_bits_to_f64(k_cache_bits[g, blocks]).reshape(-1, d)[:ctx]
            v = bf16_bits_to_f64(v_cache_bits[g, blocks]).reshape(-1, d)[:ctx]
            for j in range(g * group, (g + 1) * group):
                s = scale * (k @ q[b, j])
                p = np.exp(s - s.max())
                p = p / p.sum()
                out[b, j] = p @ v
    return out
