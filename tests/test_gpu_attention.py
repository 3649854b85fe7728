"""GPU parity: tiered paged decode attention over a wave-aware KV pool against the oracle."""
import math

import numpy as np
import pytest

from oracle import kv_pool as okp
from oracle import linalg as ol
from paper_2609_13592_b200 import binding as B
from paper_2609_13592_b200 import synth
from tests.helpers import assert_close_to_oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2609_13592_b200 import build
    build.build_library()
    B.lib()
    return torch.device("cuda:0")


def bf16_tensor(bits, dev):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)


def bits_of(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def build_tables(pool, ref_pool, ctx_lens, churn):
    """Block tables through the wave-aware pool, the library and the oracle side by side:
    round-robin growth one block at a time, optionally after a churn phase (16 requests,
    every other one freed)."""
    n_seq = len(ctx_lens)
    need = [(int(c) + 15) // 16 for c in ctx_lens]
    if churn:
        for r in range(16):
            a = pool.alloc(1000 + r, 20 + 3 * r).tolist()
            assert a == ref_pool.alloc(1000 + r, 20 + 3 * r)
        for r in range(0, 16, 2):
            pool.free(1000 + r)
            ref_pool.free_request(1000 + r)
    tables = [[] for _ in range(n_seq)]
    for step in range(max(need) if need else 0):
        for b in range(n_seq):
            if step < need[b]:
                got = pool.alloc(b, 1).tolist()
                assert got == ref_pool.alloc(b, 1)      # allocations are bit-exact
                tables[b] += got
    max_blocks = max(1, max(need) if need else 1)
    table = np.zeros((n_seq, max_blocks), dtype=np.int32)
    for b in range(n_seq):
        table[b, :need[b]] = tables[b]
    flat = [x for t in tables for x in t]
    assert len(flat) == len(set(flat))                   # no block handed out twice
    return table


def run_attention(dev, n_seq, hq, hkv, ctx_lens, n_blocks, modulus, seed, churn=False):
    from paper_2609_13592_b200.tiers import TieredKVCache, aligned_workspace
    d = 128
    pool, ref_pool = B.KVPool(n_blocks, hkv, modulus), okp.KVPool(n_blocks, hkv, modulus)
    table = build_tables(pool, ref_pool, ctx_lens, churn)
    k_bits = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, seed)
    v_bits = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, seed + 1)
    q_bits = synth.normal_bf16((n_seq, hq, d), 1.0, seed + 2)
    cache = TieredKVCache(pool, hkv, n_blocks, d, dev)
    assert cache.tier.tolist() == ref_pool.page_tiers()
    assert (int((cache.tier == 1).sum()) > 0) == (modulus > 0)     # a tiered case really has host pages
    cache.load(bf16_tensor(k_bits, dev), bf16_tensor(v_bits, dev))
    back_k, back_v = cache.dump()
    assert np.array_equal(bits_of(back_k), k_bits) and np.array_equal(bits_of(back_v), v_bits)
    q = bf16_tensor(q_bits, dev)
    max_blocks = table.shape[1]
    ws_bytes = B.boost_paged_attn_workspace_bytes(n_seq, hq, d, max_blocks)
    ws_t, ws = aligned_workspace(ws_bytes, dev)
    out = torch.full((n_seq, hq, d), float("nan"), dtype=torch.bfloat16, device=dev)
    table_d = torch.from_numpy(table).to(dev)
    ctx_d = torch.tensor(list(ctx_lens), dtype=torch.int32, device=dev)
    scale = 1.0 / math.sqrt(d)
    outs = []
    for _ in range(2):   # second call reuses the workspace as the first left it
        out.fill_(float("nan"))
        B.boost_paged_attn_decode_tiered(q, cache.k.page_ptr, cache.v.page_ptr, cache.tier, cache.n_pages,
                                         n_blocks, table_d, max_blocks, ctx_d, n_seq, hq, hkv, d, scale,
                                         ws, ws_bytes, out)
        torch.cuda.synchronize()
        outs.append(out.float().cpu().numpy().copy())
    off = ws - ws_t.data_ptr()
    assert int(ws_t[off:off + 4].cpu().numpy().view(np.uint32)[0]) == 0     # status word
    assert not ws_t[off:off + (16 + n_seq * hkv) * 4].cpu().numpy().any()    # counters back at zero
    assert np.array_equal(outs[0], outs[1])
    ref = ol.paged_attention_decode(q_bits, k_bits, v_bits, table, ctx_lens, scale)
    pool.close()
    return outs[0], ref, cache


def test_attention_config2(dev):
    # batch 8, 32 query heads, 8 KV heads, head_dim 128, context uniform in [512, 4096],
    # pool of 2048 blocks with 1/8 of its pages on the host, blocks through the pool
    ctx = synth.ctx_lens_uniform(8, 512, 4096, seed=2).tolist()
    n_blocks = 2560
    assert sum((c + 15) // 16 for c in ctx) <= n_blocks
    out, ref, cache = run_attention(dev, 8, 32, 8, ctx, n_blocks, 8, seed=20)
    assert int((cache.tier == 1).sum()) * 8 == cache.tier.size
    assert_close_to_oracle(out, ref, "config 2 attention")


def test_attention_config2_after_churn(dev):
    ctx = synth.ctx_lens_uniform(8, 512, 2048, seed=3).tolist()
    out, ref, _ = run_attention(dev, 8, 32, 8, ctx, 2048, 8, seed=30, churn=True)
    assert_close_to_oracle(out, ref, "attention after churn")


@pytest.mark.parametrize("ctx", [[1], [15], [16], [17], [127, 128, 129], [0, 5], [300, 1, 0, 2049]])
def test_attention_edge_lengths(dev, ctx):
    # 2048 blocks x 2 KV heads = 8 pages per tensor, modulus 4: the last two in host memory
    out, ref, _ = run_attention(dev, len(ctx), 8, 2, ctx, 2048, 4, seed=40 + len(ctx) + ctx[0])
    assert_close_to_oracle(out, ref, f"attention ctx={ctx}")
    for b, c in enumerate(ctx):
        if c == 0:
            assert not out[b].any()


@pytest.mark.parametrize("hq,hkv,modulus", [(8, 8, 0), (16, 1, 2), (4, 4, 12), (8, 8, 5), (32, 2, 3)])
def test_attention_head_layouts(dev, hq, hkv, modulus):
    # pool sizes that give every tiered case at least one host page (pages = heads * blocks / 512)
    n_blocks = {(8, 0): 512, (1, 2): 1024, (4, 12): 1536, (8, 5): 2560, (2, 3): 1536}[(hkv, modulus)]
    ctx = [700, 33, 260]
    out, ref, _ = run_attention(dev, 3, hq, hkv, ctx, n_blocks, modulus, seed=hq * 100 + hkv)
    assert_close_to_oracle(out, ref, f"attention hq={hq} hkv={hkv} M={modulus}")


def test_attention_special_cases(dev):
    # ctx = 1: output is the V row itself (bf16 in, bf16 out: exact)
    # (2048 blocks x 2 heads = 8 pages, the last two in host memory)
    out, ref, _ = run_attention(dev, 4, 8, 2, [1, 1, 1, 1], 2048, 4, seed=77)
    assert np.array_equal(out, ref)


def test_attention_argument_errors(dev):
    from paper_2609_13592_b200.tiers import aligned_workspace
    q = torch.zeros(1, 8, 128, dtype=torch.bfloat16, device=dev)
    pp = torch.zeros(8, dtype=torch.int64, device=dev)
    tbl = torch.zeros(1, 4, dtype=torch.int32, device=dev)
    ctx = torch.zeros(1, dtype=torch.int32, device=dev)
    ws_t, ws = aligned_workspace(1 << 16, dev)
    args = dict(q=q, k=pp, v=pp, tier=None, n_pages=2, n_blocks=512, tbl=tbl, mb=4, ctx=ctx)

    def call(hq=8, hkv=2, d=128, n_pages=2, ws_bytes=1 << 16, tier=None):
        B.boost_paged_attn_decode_tiered(q, pp, pp, tier, n_pages, 512, tbl, 4, ctx, 1, hq, hkv, d, 1.0,
                                         ws, ws_bytes, q)
    for kwargs, code in ((dict(d=64), B.ERR_UNSUPPORTED), (dict(hq=7), B.ERR_INVALID),
                         (dict(n_pages=3), B.ERR_INVALID), (dict(ws_bytes=64), B.ERR_CAPACITY),
                         (dict(tier=np.array([1, 0], np.uint8)), B.ERR_UNSUPPORTED)):
        with pytest.raises(B.BoostError) as e:
            call(**kwargs)
        assert e.value.code == code, kwargs
    del args


def test_attention_config5_shape_on_sampled_sequences(dev):
    """Configuration 5's attention launch: batch 128, context lengths uniform in [2048, 4096]
    (seed 5), 32 / 8 heads, a pool of 25088 blocks with host modulus 5 (one page in five of the
    K and V tensors in host memory), blocks through the wave-aware pool.  The device computes
    all 128 sequences; the oracle computes every head of 6 sampled sequences (the longest, the
    shortest and four drawn with seed 7)."""
    from paper_2609_13592_b200.tiers import TieredKVCache, aligned_workspace
    n_seq, hq, hkv, d, n_blocks, modulus = 128, 32, 8, 128, 25088, 5
    ctx = synth.ctx_lens_uniform(n_seq, 2048, 4096, seed=5)
    assert int(((ctx + 15) // 16).sum()) <= n_blocks
    pool, ref_pool = B.KVPool(n_blocks, hkv, modulus), okp.KVPool(n_blocks, hkv, modulus)
    table = build_tables(pool, ref_pool, ctx.tolist(), churn=False)
    k_bits = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 50)
    v_bits = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 51)
    q_bits = synth.normal_bf16((n_seq, hq, d), 1.0, 52)
    cache = TieredKVCache(pool, hkv, n_blocks, d, dev)
    assert cache.tier.tolist() == ref_pool.page_tiers()
    assert int((cache.tier == 1).sum()) == cache.tier.size // 5
    cache.load(bf16_tensor(k_bits, dev), bf16_tensor(v_bits, dev))
    max_blocks = table.shape[1]
    ws_bytes = B.boost_paged_attn_workspace_bytes(n_seq, hq, d, max_blocks)
    ws_t, ws = aligned_workspace(ws_bytes, dev)
    out = torch.full((n_seq, hq, d), float("nan"), dtype=torch.bfloat16, device=dev)
    scale = 1.0 / math.sqrt(d)
    B.boost_paged_attn_decode_tiered(bf16_tensor(q_bits, dev), cache.k.page_ptr, cache.v.page_ptr, cache.tier,
                                     cache.n_pages, n_blocks, torch.from_numpy(table).to(dev), max_blocks,
                                     torch.from_numpy(ctx.astype(np.int32)).to(dev), n_seq, hq, hkv, d, scale,
                                     ws, ws_bytes, out)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy()
    assert np.isfinite(got).all()
    off = ws - ws_t.data_ptr()
    assert int(ws_t[off:off + 4].cpu().numpy().view(np.uint32)[0]) == 0     # status word
    sel = sorted({int(np.argmax(ctx)), int(np.argmin(ctx)),
                  *np.random.default_rng(7).choice(n_seq, size=4, replace=False).tolist()})
    ref = ol.paged_attention_decode(q_bits[sel], k_bits, v_bits, table[sel], ctx[sel].tolist(), scale)
    assert_close_to_oracle(got[sel], ref, "config 5 attention, sampled sequences")
    pool.close()


def test_attention_on_a_pool_under_serving_churn(dev):
    """Four KV heads (eight query heads each), one KV page in twelve on the host, the batch as a
    pool leaves it after 7000 decode steps of Poisson arrivals with a long-generation length
    mix at about 80 % utilisation (Sec. 5.11): about 95 sequences of up to 6000 tokens whose
    blocks are scattered over the pool, so a sequence takes several work items and its
    partial results meet in global memory.  The library and the oracle pool replay the trace
    side by side; the oracle computes the longest, the shortest and three more sequences."""
    from paper_2609_13592_b200 import serving
    from paper_2609_13592_b200.tiers import TieredKVCache, aligned_workspace
    hq, hkv, d, n_blocks, modulus = 32, 4, 128, 12 * 1024, 12
    pool, ref_pool = B.KVPool(n_blocks, hkv, modulus), okp.KVPool(n_blocks, hkv, modulus)

    class Both:
        def alloc(self, r, n):
            got = pool.alloc(r, n)
            assert got.tolist() == ref_pool.alloc(r, n)
            return got

        def free(self, r):
            pool.free(r)
            ref_pool.free_request(r)

        def query(self):
            return pool.query()

    trace = synth.serving_churn_trace(n_blocks, 7000, 0.045, 96, seed=7)
    _, _, _, snapshots, _ = serving.replay_churn(Both(), trace, [6999])
    ctx, table = snapshots[0]["ctx_lens"], snapshots[0]["table"]
    n_seq, max_blocks = table.shape
    assert n_seq >= 40 and ctx.max() > 4096 + 64
    k_bits = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 60)
    v_bits = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 61)
    q_bits = synth.normal_bf16((n_seq, hq, d), 1.0, 62)
    cache = TieredKVCache(pool, hkv, n_blocks, d, dev)
    assert cache.tier.tolist() == ref_pool.page_tiers() and int((cache.tier == 1).sum()) * 12 == cache.tier.size
    cache.load(bf16_tensor(k_bits, dev), bf16_tensor(v_bits, dev))
    ws_bytes = B.boost_paged_attn_workspace_bytes(n_seq, hq, d, max_blocks)
    ws_t, ws = aligned_workspace(ws_bytes, dev)
    out = torch.full((n_seq, hq, d), float("nan"), dtype=torch.bfloat16, device=dev)
    scale = 1.0 / math.sqrt(d)
    B.boost_paged_attn_decode_tiered(bf16_tensor(q_bits, dev), cache.k.page_ptr, cache.v.page_ptr, cache.tier,
                                     cache.n_pages, n_blocks, torch.from_numpy(table).to(dev), max_blocks,
                                     torch.from_numpy(ctx).to(dev), n_seq, hq, hkv, d, scale, ws, ws_bytes, out)
    torch.cuda.synchronize()
    got = out.float().cpu().numpy()
    assert np.isfinite(got).all()
    off = ws - ws_t.data_ptr()
    assert int(ws_t[off:off + 4].cpu().numpy().view(np.uint32)[0]) == 0     # status word
    sel = sorted({int(np.argmax(ctx)), int(np.argmin(ctx)),
                  *np.random.default_rng(9).choice(n_seq, size=3, replace=False).tolist()})
    ref = ol.paged_attention_decode(q_bits[sel], k_bits, v_bits, table[sel], ctx[sel].tolist(), scale)
    assert_close_to_oracle(got[sel], ref, "attention on a churned pool, sampled sequences")
    pool.close()


def test_attention_repeated_launches_are_identical(dev):
    """100 launches of configuration 2's attention give the same bits (ring stages are refilled
    by bulk copies right after they are read)."""
    from paper_2609_13592_b200.tiers import TieredKVCache, aligned_workspace
    n_seq, hq, hkv, d, n_blocks = 8, 32, 8, 128, 2560
    ctx = synth.ctx_lens_uniform(n_seq, 512, 4096, seed=2).tolist()
    for modulus in (0, 8):
        pool, ref_pool = B.KVPool(n_blocks, hkv, modulus), okp.KVPool(n_blocks, hkv, modulus)
        table = build_tables(pool, ref_pool, ctx, churn=False)
        cache = TieredKVCache(pool, hkv, n_blocks, d, dev)
        cache.load(bf16_tensor(synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 80), dev),
                   bf16_tensor(synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 81), dev))
        q = bf16_tensor(synth.normal_bf16((n_seq, hq, d), 1.0, 82), dev)
        max_blocks = table.shape[1]
        ws_bytes = B.boost_paged_attn_workspace_bytes(n_seq, hq, d, max_blocks)
        ws_t, ws = aligned_workspace(ws_bytes, dev)
        table_d = torch.from_numpy(table).to(dev)
        ctx_d = torch.tensor(ctx, dtype=torch.int32, device=dev)
        outs = []
        for _ in range(101):
            out = torch.empty((n_seq, hq, d), dtype=torch.bfloat16, device=dev)
            B.boost_paged_attn_decode_tiered(q, cache.k.page_ptr, cache.v.page_ptr, cache.tier, cache.n_pages, n_blocks,
                                             table_d, max_blocks, ctx_d, n_seq, hq, hkv, d, 1.0 / math.sqrt(d), ws, ws_bytes, out)
            torch.cuda.synchronize()
            outs.append(out)
        assert all(torch.equal(o, outs[0]) for o in outs[1:])
        pool.close()


def test_attention_context_length_outside_the_table_is_clamped_and_flagged(dev):
    """A context length beyond what the block table's row describes does not read past the row:
    the sequence is processed up to 16 * max_blocks tokens and bit 2 of the status word is set."""
    from paper_2609_13592_b200.tiers import TieredKVCache, aligned_workspace
    n_seq, hq, hkv, d, n_blocks, max_blocks = 2, 8, 2, 128, 512, 8
    pool = B.KVPool(n_blocks, hkv, 0)
    table = np.stack([pool.alloc(b, max_blocks) for b in range(n_seq)]).astype(np.int32)
    k_bits = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 90)
    v_bits = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 91)
    q_bits = synth.normal_bf16((n_seq, hq, d), 1.0, 92)
    cache = TieredKVCache(pool, hkv, n_blocks, d, dev)
    cache.load(bf16_tensor(k_bits, dev), bf16_tensor(v_bits, dev))
    ws_bytes = B.boost_paged_attn_workspace_bytes(n_seq, hq, d, max_blocks)
    ws_t, ws = aligned_workspace(ws_bytes, dev)
    out = torch.empty((n_seq, hq, d), dtype=torch.bfloat16, device=dev)
    ctx = np.array([100, 5000], dtype=np.int32)          # the second one is far beyond 8 blocks
    scale = 1.0 / math.sqrt(d)
    B.boost_paged_attn_decode_tiered(bf16_tensor(q_bits, dev), cache.k.page_ptr, cache.v.page_ptr, cache.tier, cache.n_pages,
                                     n_blocks, torch.from_numpy(table).to(dev), max_blocks, torch.from_numpy(ctx).to(dev),
                                     n_seq, hq, hkv, d, scale, ws, ws_bytes, out)
    torch.cuda.synchronize()
    off = ws - ws_t.data_ptr()
    assert int(ws_t[off:off + 4].cpu().numpy().view(np.uint32)[0]) == 2
    ref = ol.paged_attention_decode(q_bits, k_bits, v_bits, table, [100, 16 * max_blocks], scale)
    assert_close_to_oracle(out.float().cpu().numpy(), ref, "attention with a clamped context length")
    pool.close()
