"""GPU parity: the small operators of a decode step and the whole step against the oracle."""
import numpy as np
import pytest

from oracle import decode as od
from oracle import kv_pool as okp
from oracle import linalg as ol
from paper_2609_13592_b200 import binding as B
from paper_2609_13592_b200 import synth
from tests.helpers import assert_bulk_close, assert_chain_close, assert_close_to_oracle

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


def test_embed_rmsnorm_swiglu_argmax(dev):
    rng = np.random.default_rng(0)
    vocab, hid, n_seq, ffn = 300, 512, 5, 384
    table = synth.normal_bf16((vocab, hid), 0.02, 1)
    tokens = np.array([0, 299, 17, 17, 123], np.int32)
    out = torch.zeros(n_seq, hid, dtype=torch.bfloat16, device=dev)
    B.boost_embed_gather(bf16_tensor(table, dev), vocab, hid, torch.from_numpy(tokens).to(dev), n_seq, out)
    assert np.array_equal(bits_of(out), table[tokens])

    x = synth.normal_bf16((n_seq, hid), 1.0, 2)
    w = synth.f32_to_bf16_bits(1.0 + 0.1 * rng.standard_normal(hid).astype(np.float32))
    y = torch.zeros(n_seq, hid, dtype=torch.bfloat16, device=dev)
    B.boost_rmsnorm(bf16_tensor(x, dev), bf16_tensor(w, dev), n_seq, hid, od.RMS_EPS, y)
    assert_close_to_oracle(y.float().cpu().numpy(), od.rmsnorm(ol.bf16_bits_to_f64(x), w), "rmsnorm")

    gu = synth.normal_bf16((n_seq, 2 * ffn), 0.4, 3)   # outputs stay below 4: half a bf16 ulp < 2e-2
    act = torch.zeros(n_seq, ffn, dtype=torch.bfloat16, device=dev)
    B.boost_swiglu(bf16_tensor(gu, dev), n_seq, ffn, act)
    g64 = ol.bf16_bits_to_f64(gu)
    assert_close_to_oracle(act.float().cpu().numpy(), od.silu(g64[:, :ffn]) * g64[:, ffn:], "swiglu")

    v = 128256
    logits = rng.standard_normal((4, v)).astype(np.float32)
    logits[1, 5000] = logits[1, 70000] = 9.0           # tie: lowest index wins
    logits[2, v - 1] = 10.0
    logits[3, 0] = 11.0
    got = torch.zeros(4, dtype=torch.int32, device=dev)
    B.boost_argmax(torch.from_numpy(logits).to(dev), 4, v, got)
    torch.cuda.synchronize()
    assert got.cpu().numpy().tolist() == np.argmax(logits, axis=-1).tolist() == [int(np.argmax(logits[0])), 5000, v - 1, 0]


def test_rope_kv_append(dev):
    from paper_2609_13592_b200.tiers import TieredKVCache
    hq, hkv, d, n_blocks = 8, 2, 128, 2048     # 8 pages per tensor, the last two in host memory
    pool = B.KVPool(n_blocks, hkv, 4)
    cache = TieredKVCache(pool, hkv, n_blocks, d, dev)
    assert int((cache.tier == 1).sum()) == 2
    k0 = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 5)
    v0 = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 6)
    cache.load(bf16_tensor(k0, dev), bf16_tensor(v0, dev))
    ctx = np.array([1, 16, 17, 4000, 0], np.int32)
    n_seq = len(ctx)
    table = np.zeros((n_seq, 256), np.int32)
    used = iter(np.random.default_rng(1).permutation(n_blocks))
    for b in range(n_seq):
        for j in range((ctx[b] + 15) // 16):
            table[b, j] = next(used)
    qkv = synth.normal_bf16((n_seq, (hq + 2 * hkv) * d), 1.0, 7)
    q_out = torch.zeros(n_seq, hq, d, dtype=torch.bfloat16, device=dev)
    status = torch.zeros(4, dtype=torch.int32, device=dev)
    B.boost_rope_kv_append(bf16_tensor(qkv, dev), q_out, cache.k.page_ptr, cache.v.page_ptr, n_blocks,
                           torch.from_numpy(table).to(dev), 256, torch.from_numpy(ctx).to(dev), n_seq, hq, hkv,
                           d, od.ROPE_BASE, status)
    torch.cuda.synchronize()
    assert int(status[0]) == 0
    x = ol.bf16_bits_to_f64(qkv)
    pos = np.maximum(ctx - 1, 0)
    q_ref = od.rope(x[:, :hq * d].reshape(n_seq, hq, d), pos)
    k_ref = od.rope(x[:, hq * d:(hq + hkv) * d].reshape(n_seq, hkv, d), pos)
    v_ref = x[:, (hq + hkv) * d:].reshape(n_seq, hkv, d)
    live = ctx > 0
    assert_close_to_oracle(q_out.float().cpu().numpy()[live], q_ref[live], "rope q")
    k_now, v_now = (bits_of(t) for t in cache.dump())
    k_want, v_want = k0.copy(), v0.copy()
    for b in range(n_seq):
        if ctx[b] == 0:
            continue
        blk, slot = table[b, pos[b] // 16], pos[b] % 16
        assert_close_to_oracle(ol.bf16_bits_to_f64(k_now[:, blk, slot]), k_ref[b], "rope k")
        assert np.array_equal(ol.bf16_bits_to_f64(v_now[:, blk, slot]), v_ref[b])
        k_want[:, blk, slot] = k_now[:, blk, slot]
        v_want[:, blk, slot] = v_now[:, blk, slot]
    # nothing else in the cache was touched
    assert np.array_equal(k_now, k_want) and np.array_equal(v_now, v_want)
    pool.close()


def build_decoder(dev, cfg, w, n_pool_blocks, kv_modulus, weight_ratio, max_batch, max_blocks, weight_tier=None):
    from paper_2609_13592_b200.llama import LlamaDecoder

    def get_weight(name, layer):
        src = w[name] if layer is None else w["layers"][layer][name]
        return bf16_tensor(src, dev)

    return LlamaDecoder(cfg, get_weight, weight_ratio, n_pool_blocks, kv_modulus, max_batch, max_blocks, dev,
                        weight_tier=weight_tier)


def first_page_on_host(name, layer, n_pages):
    """Explicit tier table: the first page of every matrix in host memory.  The matrices of the
    tiny test model are one page each - shorter than any placement period - so this is how a
    multi-step decode gets host-tier weights (all of them, here)."""
    tier = np.zeros(n_pages, np.uint8)
    tier[0] = 1
    return tier


def all_weights(dec):
    return [dec.lm_head] + [ly[k] for ly in dec.layers for k in ("wqkv", "wo", "wgu", "wd")]


def load_caches(dev, dec, k_host, v_host):
    hkv, d = dec.cfg["n_kv_heads"], dec.cfg["head_dim"]
    for li, ly in enumerate(dec.layers):
        B.boost_kv_scatter(bf16_tensor(k_host[li], dev), hkv, dec.n_pool_blocks, d, ly["k"].page_ptr, ly["k"].n_pages)
        B.boost_kv_scatter(bf16_tensor(v_host[li], dev), hkv, dec.n_pool_blocks, d, ly["v"].page_ptr, ly["v"].n_pages)


def dump_cache(dev, dec, li, name):
    hkv, d = dec.cfg["n_kv_heads"], dec.cfg["head_dim"]
    t = torch.empty(hkv, dec.n_pool_blocks, 16, d, dtype=torch.bfloat16, device=dev)
    B.boost_kv_gather(t, hkv, dec.n_pool_blocks, d, dec.layers[li][name].page_ptr, dec.layers[li][name].n_pages)
    return bits_of(t)


@pytest.mark.parametrize("n_seq,kv_modulus,host_weights,recycle", [
    (3, 4, True, False), (1, 0, False, False), (20, 2, True, False), (40, 4, True, False), (6, 4, False, True),
    (2, 4, True, True), (70, 2, True, False), (150, 2, False, False), (256, 4, True, False),
    (3, 4, "two_queues", False), (24, 2, "two_queues", False), (70, 2, "two_queues", False)])
def test_decode_steps_match_oracle(dev, n_seq, kv_modulus, host_weights, recycle):
    """16 consecutive decode steps of the tiny model against the oracle.  host_weights: every weight
    matrix has its (only) page in host memory, so all products of the chain take the host-tier
    path (read in place under the even partition; "two_queues": the two-queue schedule, host pages
    first); otherwise all weights are in HBM (even partition).  kv_modulus > 0 puts KV pages on
    the host as the pool places them.  Batch 1 - 2 is the CUDA-core kernel, 3 - 32 mma.sync, 40 and
    70 the tcgen05 kernel, 150 and 256 (the largest batch a step takes) its 256-column form."""
    from tests.helpers import chain_error
    B.boost_gemv_set_tier_schedule(host_weights == "two_queues")   # (reset at the end of the test)
    host_weights = bool(host_weights)
    cfg = dict(synth.TINY_LLAMA)
    w = synth.llama_weights(cfg, seed=n_seq, std=0.02)
    hkv, d, nl = cfg["n_kv_heads"], cfg["head_dim"], cfg["n_layers"]
    n_pool_blocks, max_blocks = 2048, 8      # a K or V tensor is 8 pages: modulus 4 puts 2 on the host, modulus 2 four
    dec = build_decoder(dev, cfg, w, n_pool_blocks, kv_modulus, 0.0, max(n_seq, 4), max_blocks,
                        weight_tier=first_page_on_host if host_weights else None)
    assert all((tw.buf.n_host > 0) == host_weights for tw in all_weights(dec))
    assert (dec.layers[0]["k"].n_host > 0) == (kv_modulus > 0)
    ref_pool = okp.KVPool(n_pool_blocks, hkv, kv_modulus, 16 * d * 2)
    assert dec.kv_tier.tolist() == ref_pool.page_tiers()
    # every sequence starts with a random prefix already in the cache (prefill stand-in)
    rng = np.random.default_rng(10 + n_seq)
    prefix = rng.integers(0, 40, size=n_seq)
    k_host = [synth.normal_bf16((hkv, n_pool_blocks, 16, d), 1.0, 100 + li) for li in range(nl)]
    v_host = [synth.normal_bf16((hkv, n_pool_blocks, 16, d), 1.0, 200 + li) for li in range(nl)]
    table = np.zeros((n_seq, max_blocks), np.int32)
    n_have = np.zeros(n_seq, np.int64)
    ctx = prefix.astype(np.int64).copy()
    tokens = rng.integers(0, cfg["vocab"], size=n_seq).astype(np.int32)
    tok_pin = torch.zeros(n_seq, dtype=torch.int32).pin_memory()
    ctx_pin = torch.zeros(n_seq, dtype=torch.int32).pin_memory()
    tab_pin = torch.zeros(n_seq, max_blocks, dtype=torch.int32).pin_memory()
    nxt_pin = torch.zeros(n_seq, dtype=torch.int32).pin_memory()
    exact_rows = total_rows = 0
    for step in range(16):
        # both sides start every step from the same cache, so that a bf16 rounding that fell
        # differently in an earlier step does not carry over
        load_caches(dev, dec, k_host, v_host)
        if recycle and step in (5, 9, 12):
            # a sequence ends and a new one takes its place in the batch: its blocks go back to the
            # pool (both sides) and the newcomer starts from an empty context on whatever the pool
            # hands out next
            gone = step % n_seq
            dec.pool.free(gone)
            ref_pool.free_request(gone)
            ctx[gone], n_have[gone] = 0, 0
            table[gone, :] = 0
            tokens[gone] = (37 * step) % cfg["vocab"]
        ctx += 1                                           # the new token joins the context
        for b in range(n_seq):                             # blocks through the pool, both sides
            while n_have[b] * 16 < ctx[b]:
                got = dec.pool.alloc(b, 1).tolist()
                assert got == ref_pool.alloc(b, 1)
                table[b, n_have[b]] = got[0]
                n_have[b] += 1
        tok_pin.numpy()[:] = tokens
        ctx_pin.numpy()[:] = ctx
        tab_pin.numpy()[:] = table
        n_launch = dec.step_host(tok_pin.numpy(), tab_pin.numpy(), ctx_pin.numpy(), nxt_pin.numpy())
        # attention plan, rope table, embedding, first qkv product, per layer attention + chain, argmax;
        # + a combine kernel after a chain whose last product has many partial sums
        assert 5 + 2 * nl <= n_launch <= 5 + 3 * nl + 1
        ref = od.decode_step(cfg, w, tokens, k_host, v_host, table, ctx)
        logits = dec.buf["logits"][:n_seq].cpu().numpy()
        assert_chain_close(logits, ref["logits"], f"logits step {step}")
        for b in range(n_seq):
            total_rows += 1
            exact_rows += chain_error(logits[b], ref["logits"][b])[0] < 1e-4
        got_next = nxt_pin.numpy().copy()
        # the device's own argmax of its own logits (integer work: exact) ...
        assert np.array_equal(got_next, np.argmax(logits, axis=-1))
        # ... and against the oracle wherever its top two logits are clearly separated
        top2 = np.sort(ref["logits"], axis=-1)[:, -2:]
        clear = (top2[:, 1] - top2[:, 0]) > 4e-2
        assert np.array_equal(got_next[clear], ref["next_tokens"][clear])
        # the K/V rows written by this step
        pos = ctx - 1
        for li in range(nl):
            for name, host in (("k", k_host), ("v", v_host)):
                now = dump_cache(dev, dec, li, name)
                for b in range(n_seq):
                    blk, slot = table[b, pos[b] // 16], pos[b] % 16
                    assert_chain_close(ol.bf16_bits_to_f64(now[:, blk, slot]),
                                       ol.bf16_bits_to_f64(host[li][:, blk, slot]), f"new {name} row")
                    now[:, blk, slot] = host[li][:, blk, slot]
                assert np.array_equal(now, host[li])       # nothing else was written
        tokens = ref["next_tokens"].astype(np.int32)       # both sides continue from the oracle's choice
    B.boost_gemv_set_tier_schedule(False)
    assert dec.status_words() == [0, 0]
    assert exact_rows >= 0.6 * total_rows, (exact_rows, total_rows)
    if kv_modulus:
        # the sequences really read host-tier KV: some of their blocks have a head in host memory
        info = dec.pool.query()
        assert info["live_host_chunks"] > 0, info


@pytest.mark.parametrize("n_seq", [2, 12, 48, 150])
def test_step_bits_do_not_depend_on_weight_placement(dev, n_seq):
    """With host pages read in place the work partition of a product is the same wherever its
    pages live, so a decode step whose weights all sit in host memory gives the same logits, bit
    for bit, as the step with all weights in HBM (CUDA-core, mma.sync and both tcgen05 forms)."""
    cfg = dict(synth.TINY_LLAMA)
    w = synth.llama_weights(cfg, seed=77, std=0.02)
    hkv, d, nl = cfg["n_kv_heads"], cfg["head_dim"], cfg["n_layers"]
    n_pool_blocks, max_blocks = 2048, 8
    rng = np.random.default_rng(5)
    ctx = rng.integers(1, 60, size=n_seq).astype(np.int32)
    table = np.zeros((n_seq, max_blocks), np.int32)
    perm = rng.permutation(n_pool_blocks)[:n_seq * 4].reshape(n_seq, 4)
    table[:, :4] = perm
    tokens = rng.integers(0, cfg["vocab"], size=n_seq).astype(np.int32)
    k_host = [synth.normal_bf16((hkv, n_pool_blocks, 16, d), 1.0, 300 + li) for li in range(nl)]
    v_host = [synth.normal_bf16((hkv, n_pool_blocks, 16, d), 1.0, 400 + li) for li in range(nl)]
    logits = []
    for tier_fn in (None, first_page_on_host):
        dec = build_decoder(dev, cfg, w, n_pool_blocks, 0, 0.0, max(n_seq, 4), max_blocks, weight_tier=tier_fn)
        assert all((tw.buf.n_host > 0) == (tier_fn is not None) for tw in all_weights(dec))
        load_caches(dev, dec, k_host, v_host)
        nxt = np.zeros(n_seq, np.int32)
        per_step = []
        tok, c = tokens.copy(), ctx.copy()
        for step in range(3):
            dec.step_host(tok, table, c, nxt)
            per_step.append(dec.buf["logits"][:n_seq].cpu().numpy().copy())
            tok, c = nxt.copy(), c + 1
        assert dec.status_words() == [0, 0]
        logits.append(per_step)
        del dec
    for a_, b_ in zip(*logits):
        assert np.isfinite(a_).all() and np.array_equal(a_, b_)


def test_fused_product_epilogues_match_oracle(dev):
    """boost_gemv_tiered_fused: RMS row scale with folded norm weight + row statistics, SwiGLU,
    RoPE + KV append - each against the oracle's operators applied one after the other."""
    from paper_2609_13592_b200.tiers import TieredKVCache, TieredWeight
    m_b, hid, ffn, hq, hkv, d = 20, 512, 384, 4, 2, 128
    x_bits = synth.normal_bf16((m_b, hid), 1.0, 1)
    gamma = synth.f32_to_bf16_bits(1.0 + 0.1 * np.random.default_rng(2).standard_normal(hid).astype(np.float32))
    x = bf16_tensor(x_bits, dev)
    x64 = ol.bf16_bits_to_f64(x_bits)
    rs = od.rms_scale(x64)
    stride = 32
    # row statistics of x as the embedding kernel produces them (gather rows 0..m_b-1 of x itself)
    ssq = torch.zeros(hid // 128, stride, dtype=torch.float32, device=dev)
    xcopy = torch.zeros_like(x)
    B.boost_embed_gather_ssq(x, m_b, hid, torch.arange(m_b, dtype=torch.int32, device=dev), m_b, xcopy, ssq, stride)
    torch.cuda.synchronize()
    assert torch.equal(xcopy, x)
    want_ssq = (x64.reshape(m_b, hid // 128, 128) ** 2).sum(-1).T
    assert np.allclose(ssq.cpu().numpy()[:, :m_b], want_ssq, rtol=1e-5)

    def epilogue(mode, **kw):
        e = B.GemvEpilogue()
        e.mode, e.ssq_in, e.ssq_in_tiles, e.ssq_stride, e.rms_eps = mode, ssq.data_ptr(), hid // 128, stride, od.RMS_EPS
        for k, v in kw.items():
            setattr(e, k, v)
        return e

    # 1. plain: y = rs * (x W'^T) + residual, bf16, with the row statistics of y
    w_bits = synth.normal_bf16((640, hid), 0.05, 3)
    res_bits = synth.normal_bf16((m_b, 640), 1.0, 4)
    on_host = np.array([1], np.uint8)       # the matrices here are one page each: that page in host memory
    w = TieredWeight(bf16_tensor(w_bits, dev), device=dev, tier=on_host, col_scale=bf16_tensor(gamma, dev))
    assert w.buf.n_host == 1
    ssq_out = torch.zeros(5, stride, dtype=torch.float32, device=dev)
    y = w.gemv(x, y_dtype=torch.bfloat16, residual=bf16_tensor(res_bits, dev),
               epilogue=epilogue(B.EPI_PLAIN, ssq_out=ssq_out.data_ptr()))
    torch.cuda.synchronize()
    wf = ol.bf16_bits_to_f64(od.fold_norm_weight(w_bits, gamma))
    ref = rs * (x64 @ wf.T) + ol.bf16_bits_to_f64(res_bits)
    assert_close_to_oracle(y.float().cpu().numpy(), ref, "scaled product + residual")
    y64 = y.float().cpu().numpy().astype(np.float64)
    assert np.allclose(ssq_out.cpu().numpy()[:, :m_b], (y64.reshape(m_b, 5, 128) ** 2).sum(-1).T, rtol=1e-5)

    # 2. SwiGLU: [gate; up] packed with interleaved rows
    wgu_bits = synth.normal_bf16((2 * ffn, hid), 0.05, 5)
    wgu = TieredWeight(bf16_tensor(wgu_bits, dev), device=dev, row_mode=1, col_scale=bf16_tensor(gamma, dev))   # all in HBM
    act = wgu.gemv(x, y_dtype=torch.bfloat16, epilogue=epilogue(B.EPI_SWIGLU))
    torch.cuda.synchronize()
    assert tuple(act.shape) == (m_b, ffn)
    gu = ol.bf16_bits_to_f64(ol.f64_to_bf16_bits(rs * (x64 @ ol.bf16_bits_to_f64(od.fold_norm_weight(wgu_bits, gamma)).T)))
    assert_chain_close(act.float().cpu().numpy(), od.silu(gu[:, :ffn]) * gu[:, ffn:], "fused swiglu")

    # 3. RoPE + KV append after the QKV product
    n_blocks = 2048                            # 8 pages per tensor, the last two in host memory
    pool = B.KVPool(n_blocks, hkv, 4)
    cache = TieredKVCache(pool, hkv, n_blocks, d, dev)
    assert int((cache.tier == 1).sum()) == 2
    k0 = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 6)
    v0 = synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 7)
    cache.load(bf16_tensor(k0, dev), bf16_tensor(v0, dev))
    ctx = np.array([1, 16, 17, 100, 0] * 4, np.int32)
    table = np.zeros((m_b, 8), np.int32)
    used = iter(np.random.default_rng(8).permutation(n_blocks))
    for b in range(m_b):
        for j in range((ctx[b] + 15) // 16):
            table[b, j] = next(used)
    wqkv_bits = synth.normal_bf16(((hq + 2 * hkv) * d, hid), 0.05, 9)
    wqkv = TieredWeight(bf16_tensor(wqkv_bits, dev), device=dev, tier=on_host, col_scale=bf16_tensor(gamma, dev))
    q_out = torch.zeros(m_b, hq, d, dtype=torch.bfloat16, device=dev)
    table_d, ctx_d = torch.from_numpy(table).to(dev), torch.from_numpy(ctx).to(dev)
    rope_table = torch.zeros(m_b, d // 2, 2, dtype=torch.float32, device=dev)
    B.boost_rope_table(ctx_d, m_b, d, od.ROPE_BASE, rope_table)
    wqkv.gemv(x, epilogue=epilogue(B.EPI_ROPE_APPEND, q_out=q_out.data_ptr(), k_page_ptr=cache.k.page_ptr.data_ptr(),
                                   v_page_ptr=cache.v.page_ptr.data_ptr(), n_pool_blocks=n_blocks,
                                   block_table=table_d.data_ptr(), max_blocks=8, ctx_lens=ctx_d.data_ptr(),
                                   n_q_heads=hq, n_kv_heads=hkv, rope_table=rope_table.data_ptr()))
    torch.cuda.synchronize()
    assert wqkv.status_words() == [0]
    qkv = ol.bf16_bits_to_f64(ol.f64_to_bf16_bits(rs * (x64 @ ol.bf16_bits_to_f64(od.fold_norm_weight(wqkv_bits, gamma)).T)))
    pos = np.maximum(ctx - 1, 0)
    q_ref = od.rope(qkv[:, :hq * d].reshape(m_b, hq, d), pos)
    k_ref = od.rope(qkv[:, hq * d:(hq + hkv) * d].reshape(m_b, hkv, d), pos)
    v_ref = qkv[:, (hq + hkv) * d:].reshape(m_b, hkv, d)
    live = ctx > 0
    assert_chain_close(q_out.float().cpu().numpy()[live], q_ref[live], "fused rope q")
    k_now, v_now = (bits_of(t) for t in cache.dump())
    k_want, v_want = k0.copy(), v0.copy()
    for b in range(m_b):
        if ctx[b] == 0:
            continue
        blk, slot = table[b, pos[b] // 16], pos[b] % 16
        assert_chain_close(ol.bf16_bits_to_f64(k_now[:, blk, slot]), k_ref[b], "fused rope k")
        assert_chain_close(ol.bf16_bits_to_f64(v_now[:, blk, slot]), v_ref[b], "fused v")
        k_want[:, blk, slot] = k_now[:, blk, slot]
        v_want[:, blk, slot] = v_now[:, blk, slot]
    assert np.array_equal(k_now, k_want) and np.array_equal(v_now, v_want)   # nothing else was touched
    # block-table entries that point outside the pool: recorded in the status word (bit 1), the row
    # is not written anywhere, every other sequence's row is
    bad = table.copy()
    bad[2, pos[2] // 16] = n_blocks + 5
    bad[3, pos[3] // 16] = -1
    cache.load(bf16_tensor(k0, dev), bf16_tensor(v0, dev))
    bad_d = torch.from_numpy(bad).to(dev)
    wqkv.gemv(x, epilogue=epilogue(B.EPI_ROPE_APPEND, q_out=q_out.data_ptr(), k_page_ptr=cache.k.page_ptr.data_ptr(),
                                   v_page_ptr=cache.v.page_ptr.data_ptr(), n_pool_blocks=n_blocks,
                                   block_table=bad_d.data_ptr(), max_blocks=8, ctx_lens=ctx_d.data_ptr(),
                                   n_q_heads=hq, n_kv_heads=hkv, rope_table=rope_table.data_ptr()))
    torch.cuda.synchronize()
    assert wqkv.status_words() == [2]
    k_bad, v_bad = (bits_of(t) for t in cache.dump())
    k_want2, v_want2 = k0.copy(), v0.copy()
    for b in range(m_b):
        if ctx[b] == 0 or b in (2, 3):
            continue
        blk, slot = table[b, pos[b] // 16], pos[b] % 16
        k_want2[:, blk, slot] = k_now[:, blk, slot]
        v_want2[:, blk, slot] = v_now[:, blk, slot]
    assert np.array_equal(k_bad, k_want2) and np.array_equal(v_bad, v_want2)
    pool.close()


@pytest.mark.parametrize("m_b", [48, 128, 200])
def test_tile_finish_from_tensor_memory(dev, m_b):
    """tcgen05 kernel, tile-by-tile mode: products wide enough that every threadblock holds several
    row tiles (so their partial sums are not combined at the end of the phase), cut so that most
    tiles have two or three partial sums.  The threadblock that delivers a tile's last one keeps
    its accumulator in tensor memory and finishes the tile from there: SwiGLU with row scales
    (gate / up partners exchanged through shared memory) and a plain product with a residual,
    every output against the oracle."""
    from paper_2609_13592_b200.tiers import TieredWeight
    hid, ffn, n_plain = 192, 39040, 77952          # 3 k-blocks; 610 and 609 row tiles on 148 threadblocks
    x_bits = synth.normal_bf16((m_b, hid), 1.0, 31)
    gamma = synth.f32_to_bf16_bits(1.0 + 0.1 * np.random.default_rng(32).standard_normal(hid).astype(np.float32))
    x = bf16_tensor(x_bits, dev)
    x64 = ol.bf16_bits_to_f64(x_bits)
    rs = od.rms_scale(x64)
    stride = 256
    ssq = torch.zeros(2, stride, dtype=torch.float32, device=dev)       # row statistics of x, two tiles of columns
    ssq[0, :m_b] = torch.from_numpy((x64[:, :128] ** 2).sum(-1).astype(np.float32)).to(dev)
    ssq[1, :m_b] = torch.from_numpy((x64[:, 128:] ** 2).sum(-1).astype(np.float32)).to(dev)
    e = B.GemvEpilogue()
    e.mode, e.ssq_in, e.ssq_in_tiles, e.ssq_stride, e.rms_eps = B.EPI_SWIGLU, ssq.data_ptr(), 2, stride, od.RMS_EPS
    wgu_bits = synth.normal_bf16((2 * ffn, hid), 0.05, 33)
    wgu = TieredWeight(bf16_tensor(wgu_bits, dev), device=dev, row_mode=1, col_scale=bf16_tensor(gamma, dev))
    act = wgu.gemv(x, y_dtype=torch.bfloat16, epilogue=e)
    torch.cuda.synchronize()
    assert wgu.status_words() == [0]
    gu = ol.bf16_bits_to_f64(ol.f64_to_bf16_bits(rs * (x64 @ ol.bf16_bits_to_f64(od.fold_norm_weight(wgu_bits, gamma)).T)))
    assert_chain_close(act.float().cpu().numpy(), od.silu(gu[:, :ffn]) * gu[:, ffn:], f"swiglu finished from tensor memory, M_b={m_b}")
    # plain, fp32 output with a residual, ragged last row tile (77952 = 609 x 128)
    w_bits = synth.normal_bf16((n_plain - 40, hid), 0.05, 34)
    res_bits = synth.normal_bf16((m_b, n_plain - 40), 1.0, 35)
    w = TieredWeight(bf16_tensor(w_bits, dev), device=dev)
    y = w.gemv(x, y_dtype=torch.float32, residual=bf16_tensor(res_bits, dev))
    torch.cuda.synchronize()
    assert w.status_words() == [0]
    ref = x64 @ ol.bf16_bits_to_f64(w_bits).T + ol.bf16_bits_to_f64(res_bits)
    assert_close_to_oracle(y.cpu().numpy(), ref, f"plain product finished from tensor memory, M_b={m_b}")
    # the same launch again: the tile counters were left at zero, the result is the same bits
    y2 = w.gemv(x, y_dtype=torch.float32, residual=bf16_tensor(res_bits, dev))
    torch.cuda.synchronize()
    assert torch.equal(y, y2)


def test_full_size_step_matches_oracle_on_samples(dev):
    """One layer + LM head at the bench's shapes (hidden 4096, FFN 14336, 32 / 8 heads, vocab
    128256, batch 32, context about 2048, weight host share 1/131, block tables 133 wide): the
    launch configuration that bench.py times.  The oracle computes the layer in full and the
    logits of every 61st vocabulary row (so every 128-row tile of the LM head is sampled)."""
    cfg = dict(synth.LLAMA3_8B)
    cfg["n_layers"] = 1
    hq, hkv, d, hid, ffn, vocab = (cfg[k] for k in ("n_q_heads", "n_kv_heads", "head_dim", "hidden", "ffn", "vocab"))
    n_seq, max_blocks, n_pool_blocks = 32, 133, 4608
    head = synth.normal_bf16((vocab, hid), 0.02, 11)
    gam = lambda s: synth.f32_to_bf16_bits(1.0 + 0.02 * np.random.default_rng(s).standard_normal(hid).astype(np.float32))
    w = {"embed": head, "lm_head": head, "norm_f": gam(1), "layers": [{
        "norm1": gam(2), "wqkv": synth.normal_bf16(((hq + 2 * hkv) * d, hid), 0.02, 12),
        "wo": synth.normal_bf16((hid, hq * d), 0.02, 13), "norm2": gam(3),
        "wgu": synth.normal_bf16((2 * ffn, hid), 0.02, 14), "wd": synth.normal_bf16((hid, ffn), 0.02, 15)}]}
    dec = build_decoder(dev, cfg, w, n_pool_blocks, 0, 1.0 / 131, n_seq, max_blocks)
    assert dec.host_weight_pages() > 0
    k_host = [synth.normal_bf16((hkv, n_pool_blocks, 16, d), 1.0, 21)]
    v_host = [synth.normal_bf16((hkv, n_pool_blocks, 16, d), 1.0, 22)]
    load_caches(dev, dec, k_host, v_host)
    rng = np.random.default_rng(5)
    ctx = rng.integers(1900, 2101, size=n_seq).astype(np.int32)
    table = np.zeros((n_seq, max_blocks), np.int32)
    for j in range(max_blocks):                      # round-robin growth through the pool
        for b in range(n_seq):
            if j * 16 < ctx[b]:
                table[b, j] = dec.pool.alloc(b, 1)[0]
    tokens = rng.integers(0, vocab, size=n_seq).astype(np.int32)
    nxt = np.zeros(n_seq, np.int32)
    n_launch = dec.step_host(tokens, table, ctx, nxt)
    assert 5 + 2 <= n_launch <= 5 + 2 + 2
    assert dec.status_words() == [0, 0]

    rows = np.arange(0, vocab, 61)
    w_ref = dict(w)
    w_ref["lm_head"] = head[rows]
    ref = od.decode_step(cfg, w_ref, tokens, k_host, v_host, table, ctx, n_layers=1, keep=True)
    assert_chain_close(dec.buf["act"].float().cpu().numpy(), ref["act"], "SwiGLU output, full width", wide=True)
    assert_chain_close(dec.buf["h"].float().cpu().numpy(), ref["h_final"], "residual stream, full width", wide=True)
    logits = dec.buf["logits"].cpu().numpy()
    assert_chain_close(logits[:, rows], ref["logits"], "sampled logits", wide=True)
    # the bound above is for the few outputs behind a bf16 rounding that fell the other way; the
    # bulk must sit far inside it
    assert_bulk_close(dec.buf["h"].float().cpu().numpy(), ref["h_final"], "residual stream")
    assert_bulk_close(logits[:, rows], ref["logits"], "sampled logits")
    # integer work: the device's argmax of its own logits, lowest index on ties
    assert np.array_equal(nxt, np.argmax(logits, axis=-1))
    # every logit was written by this step: the buffer starts at zero, and an fp32 sum that
    # cancels exactly is a once-in-10^7 event per element
    assert logits.size - np.count_nonzero(logits) <= 4
    # the same step again and again (it rewrites the same cache rows): the same bits every time
    first = dec.buf["logits"].clone()
    differing = 0
    for _ in range(40):
        dec.step_host(tokens, table, ctx, nxt)
        differing += int(not torch.equal(dec.buf["logits"], first))
    assert differing == 0
    assert dec.status_words() == [0, 0]


def test_config5_launch_shape_matches_oracle_on_samples(dev):
    """Configuration 5's launch shape: one Llama-3-8B-shaped layer + LM head at batch 128 (tcgen05
    chain), context lengths uniform in [2048, 4096], KV blocks handed out by the wave-aware pool
    with host modulus 5 (20 % of the KV pages in host memory), weight host share 1/131.  The
    oracle runs the step for six sampled sequences (sequences do not interact) and every 61st
    vocabulary row; the device runs the whole batch."""
    cfg = dict(synth.LLAMA3_8B)
    cfg["n_layers"] = 1
    hq, hkv, d, hid, ffn, vocab = (cfg[k] for k in ("n_q_heads", "n_kv_heads", "head_dim", "hidden", "ffn", "vocab"))
    n_seq, max_blocks, n_pool_blocks = 128, 256, 2560 * 13
    head = synth.normal_bf16((vocab, hid), 0.02, 31)
    gam = lambda s: synth.f32_to_bf16_bits(1.0 + 0.02 * np.random.default_rng(s).standard_normal(hid).astype(np.float32))
    w = {"embed": head, "lm_head": head, "norm_f": gam(1), "layers": [{
        "norm1": gam(2), "wqkv": synth.normal_bf16(((hq + 2 * hkv) * d, hid), 0.02, 32),
        "wo": synth.normal_bf16((hid, hq * d), 0.02, 33), "norm2": gam(3),
        "wgu": synth.normal_bf16((2 * ffn, hid), 0.02, 34), "wd": synth.normal_bf16((hid, ffn), 0.02, 35)}]}
    dec = build_decoder(dev, cfg, w, n_pool_blocks, 5, 1.0 / 131, n_seq, max_blocks)
    assert dec.host_weight_pages() > 0
    n_kv_pages = dec.layers[0]["k"].n_pages
    assert dec.layers[0]["k"].n_host == n_kv_pages // 5          # linear placement: the last fifth
    ref_pool = okp.KVPool(n_pool_blocks, hkv, 5, 16 * d * 2)
    assert dec.kv_tier.tolist() == ref_pool.page_tiers()
    k_host = [synth.normal_bf16((hkv, n_pool_blocks, 16, d), 1.0, 41)]
    v_host = [synth.normal_bf16((hkv, n_pool_blocks, 16, d), 1.0, 42)]
    load_caches(dev, dec, k_host, v_host)
    ctx = synth.ctx_lens_uniform(n_seq, 2048, 4096, 5).astype(np.int32)
    table = np.zeros((n_seq, max_blocks), np.int32)
    sample = [0, 17, 45, 77, 101, 127]
    for j in range(max_blocks):                      # round-robin growth through the pool
        for b in range(n_seq):
            if j * 16 < ctx[b]:
                table[b, j] = dec.pool.alloc(b, 1)[0]
                got_ref = ref_pool.alloc(b, 1)[0]
                if b in sample:
                    assert table[b, j] == got_ref
    tokens = np.random.default_rng(6).integers(0, vocab, size=n_seq).astype(np.int32)
    nxt = np.zeros(n_seq, np.int32)
    n_launch = dec.step_host(tokens, table, ctx, nxt)
    assert 5 + 2 <= n_launch <= 5 + 2 + 2
    assert dec.status_words() == [0, 0]

    rows = np.arange(0, vocab, 61)
    w_ref = dict(w)
    w_ref["lm_head"] = head[rows]
    ref = od.decode_step(cfg, w_ref, tokens[sample], k_host, v_host, table[sample], ctx[sample], n_layers=1, keep=True)
    # the sampled sequences read host-tier KV: the second-to-last head's blocks above the pool's
    # threshold and every block of the last head
    assert dec.pool.query()["n_pages"] == n_kv_pages
    assert_chain_close(dec.buf["act"].float().cpu().numpy()[sample], ref["act"], "SwiGLU output", wide=True)
    assert_chain_close(dec.buf["h"].float().cpu().numpy()[sample], ref["h_final"], "residual stream", wide=True)
    logits = dec.buf["logits"].cpu().numpy()
    assert_chain_close(logits[sample][:, rows], ref["logits"], "sampled logits", wide=True)
    assert_bulk_close(dec.buf["h"].float().cpu().numpy()[sample], ref["h_final"], "residual stream")
    assert_bulk_close(logits[sample][:, rows], ref["logits"], "sampled logits")
    assert np.array_equal(nxt, np.argmax(logits, axis=-1))
    # the new K / V rows of the sampled sequences (the oracle appended them to k_host / v_host)
    k_now, v_now = dump_cache(dev, dec, 0, "k"), dump_cache(dev, dec, 0, "v")
    for b in sample:
        pos = int(ctx[b]) - 1
        blk, slot = table[b, pos // 16], pos % 16
        assert_chain_close(ol.bf16_bits_to_f64(k_now[:, blk, slot]), ol.bf16_bits_to_f64(k_host[0][:, blk, slot]), "new k row", wide=True)
        assert_chain_close(ol.bf16_bits_to_f64(v_now[:, blk, slot]), ol.bf16_bits_to_f64(v_host[0][:, blk, slot]), "new v row", wide=True)
    # a second launch of the same step gives the same bits
    first = dec.buf["logits"].clone()
    dec.step_host(tokens, table, ctx, nxt)
    assert torch.equal(dec.buf["logits"], first)
    assert dec.status_words() == [0, 0]


@pytest.fixture
def two_queue_schedule(request):
    """The weight products of the test run under the schedule the parameter names (True: two queues,
    host pages first; False: host pages read in place); the default comes back afterwards."""
    B.boost_gemv_set_tier_schedule(bool(request.param))
    yield bool(request.param)
    B.boost_gemv_set_tier_schedule(False)


@pytest.mark.parametrize("two_queue_schedule", [False, True], indirect=True)
@pytest.mark.parametrize("m_b", [1, 24, 70])
def test_gemv_chain_matches_separate_launches_and_oracle(dev, m_b, two_queue_schedule):
    """boost_gemv_tiered_chain: four dependent products in one launch (output product with
    residual and row statistics -> gate/up with row scale and SwiGLU -> down product with
    residual and statistics -> a scaled product with fp32 output and a ragged row count) give
    bit for bit what the same calls of boost_gemv_tiered_fused give one after the other, and
    agree with the oracle's operators; repeated launches reuse the workspace."""
    from paper_2609_13592_b200.tiers import TieredWeight, aligned_workspace
    kin, hid, ffn, n_out, stride = 768, 1024, 1536, 2000, 128
    x_bits = synth.normal_bf16((m_b, kin), 1.0, 1)
    h0_bits = synth.normal_bf16((m_b, hid), 1.0, 2)
    g1 = synth.f32_to_bf16_bits(1.0 + 0.1 * np.random.default_rng(3).standard_normal(hid).astype(np.float32))
    g2 = synth.f32_to_bf16_bits(1.0 + 0.1 * np.random.default_rng(4).standard_normal(hid).astype(np.float32))
    wb = [synth.normal_bf16((hid, kin), 0.03, 5), synth.normal_bf16((2 * ffn, hid), 0.03, 6),
          synth.normal_bf16((hid, ffn), 0.03, 7), synth.normal_bf16((n_out, hid), 0.03, 8)]
    # explicit tier tables (the matrices are 1, 3, 2 and 2 pages: shorter than a placement period):
    # an all-host matrix, a host page in the middle, at the end, at the start
    t8 = lambda *t: np.array(t, np.uint8)
    w = [TieredWeight(bf16_tensor(wb[0], dev), device=dev, tier=t8(1)),
         TieredWeight(bf16_tensor(wb[1], dev), device=dev, tier=t8(0, 1, 0), row_mode=1, col_scale=bf16_tensor(g1, dev)),
         TieredWeight(bf16_tensor(wb[2], dev), device=dev, tier=t8(0, 1)),
         TieredWeight(bf16_tensor(wb[3], dev), device=dev, tier=t8(1, 0), col_scale=bf16_tensor(g2, dev))]
    assert [tw.buf.n_pages for tw in w] == [1, 3, 2, 2]
    x = bf16_tensor(x_bits, dev)

    def buffers():
        return {"h": bf16_tensor(h0_bits, dev).clone(), "act": torch.zeros(m_b, ffn, dtype=torch.bfloat16, device=dev),
                "logits": torch.zeros(m_b, n_out, dtype=torch.float32, device=dev),
                "ssq_b": torch.zeros(hid // 128, stride, dtype=torch.float32, device=dev),
                "ssq_a": torch.zeros(hid // 128, stride, dtype=torch.float32, device=dev)}

    def epi(mode=B.EPI_PLAIN, ssq_in=None, ssq_out=None):
        e = B.GemvEpilogue()
        e.mode, e.ssq_stride, e.rms_eps, e.ssq_in_tiles = mode, stride, od.RMS_EPS, hid // 128
        e.ssq_in = None if ssq_in is None else ssq_in.data_ptr()
        e.ssq_out = None if ssq_out is None else ssq_out.data_ptr()
        return e

    def calls_for(b):
        return [dict(w=w[0].struct(), x=x, y=b["h"], y_dtype=1, residual=b["h"], epilogue=epi(ssq_out=b["ssq_b"])),
                dict(w=w[1].struct(), x=b["h"], y=b["act"], y_dtype=1, epilogue=epi(B.EPI_SWIGLU, ssq_in=b["ssq_b"])),
                dict(w=w[2].struct(), x=b["act"], y=b["h"], y_dtype=1, residual=b["h"], epilogue=epi(ssq_out=b["ssq_a"])),
                dict(w=w[3].struct(), x=b["h"], y=b["logits"], y_dtype=0, epilogue=epi(ssq_in=b["ssq_a"]))]

    # the same four calls, one launch each
    sep = buffers()
    for c, tw in zip(calls_for(sep), w):
        tw.gemv(c["x"], y=c["y"], residual=c.get("residual"), epilogue=c["epilogue"])
    torch.cuda.synchronize()
    assert all(tw.status_words() == [0] for tw in w)

    # one launch for the chain, several times over the same workspace
    probe = B.gemv_calls(calls_for(sep))
    ws_bytes = B.boost_gemv_chain_workspace_bytes(probe, m_b)
    assert ws_bytes > 0
    ws_t, ws_ptr = aligned_workspace(ws_bytes, dev)
    for rep in range(6):
        got = buffers()
        arr = B.gemv_calls(calls_for(got))
        B.boost_gemv_tiered_chain(arr, m_b, ws_ptr, ws_bytes)
        torch.cuda.synchronize()
        for name in ("h", "act", "logits", "ssq_a", "ssq_b"):
            assert torch.equal(got[name], sep[name]), (name, rep)
    off = ws_ptr - ws_t.data_ptr()
    assert int(ws_t[off:off + 4].cpu().numpy().view(np.uint32)[0]) == 0          # status word
    tail = ws_t[off + ws_bytes - 64 * 5:off + ws_bytes]
    assert int(tail.count_nonzero()) == 0                                         # queue words and phase counters reset

    # The same workspace reused by launches that follow each other on the stream with nothing in
    # between (no synchronise, no other kernel): a launch's threadblocks become resident while the
    # one before drains, and must not touch the queue words (all four weights have host pages: under
    # the two-queue schedule every product runs off the queues) before it has finished.  Chains of
    # four and of one.
    assert all(tw.buf.n_host > 0 for tw in w)
    sets = [buffers() for _ in range(8)]
    arrs = [B.gemv_calls(calls_for(b)) for b in sets]
    torch.cuda.synchronize()
    for arr in arrs:
        B.boost_gemv_tiered_chain(arr, m_b, ws_ptr, ws_bytes)
    torch.cuda.synchronize()
    for i, b in enumerate(sets):
        for name in ("h", "act", "logits", "ssq_a", "ssq_b"):
            assert torch.equal(b[name], sep[name]), (name, i)
    singles = [torch.zeros(m_b, n_out, dtype=torch.float32, device=dev) for _ in range(8)]
    one = [B.gemv_calls([dict(w=w[3].struct(), x=sep["h"], y=y1, y_dtype=0, epilogue=epi(ssq_in=sep["ssq_a"]))]) for y1 in singles]
    torch.cuda.synchronize()
    for arr in one:
        B.boost_gemv_tiered_chain(arr, m_b, ws_ptr, ws_bytes)
    torch.cuda.synchronize()
    for i, y1 in enumerate(singles):
        assert torch.equal(y1, sep["logits"]), i
    assert int(ws_t[off:off + 4].cpu().numpy().view(np.uint32)[0]) == 0

    # the oracle's operators one after the other, bf16 where the device stores bf16
    rnd = lambda a: ol.bf16_bits_to_f64(ol.f64_to_bf16_bits(a))
    x64, h64 = ol.bf16_bits_to_f64(x_bits), ol.bf16_bits_to_f64(h0_bits)
    h1 = rnd(h64 + x64 @ ol.bf16_bits_to_f64(wb[0]).T)
    gu = rnd(od.rms_scale(h1) * (h1 @ ol.bf16_bits_to_f64(od.fold_norm_weight(wb[1], g1)).T))
    act = rnd(od.silu(gu[:, :ffn]) * gu[:, ffn:])
    h2 = rnd(h1 + act @ ol.bf16_bits_to_f64(wb[2]).T)
    logits = od.rms_scale(h2) * (h2 @ ol.bf16_bits_to_f64(od.fold_norm_weight(wb[3], g2)).T)
    assert_chain_close(got["act"].float().cpu().numpy(), act, "chain: SwiGLU output", wide=True)
    assert_chain_close(got["h"].float().cpu().numpy(), h2, "chain: residual stream", wide=True)
    assert_chain_close(got["logits"].cpu().numpy(), logits, "chain: scaled product", wide=True)
    assert_bulk_close(got["h"].float().cpu().numpy(), h2, "chain: residual stream")
    assert_bulk_close(got["logits"].cpu().numpy(), logits, "chain: scaled product")


def test_prefetch_variant_matches_tiered_step(dev):
    """boost_llama_decode_step_prefetch (host KV pages staged into HBM by the copy engine, two
    layers ahead) gives bit for bit the logits, tokens and cache contents of the step that
    reads the host pages in place: the same bytes reach the same arithmetic."""
    from paper_2609_13592_b200.llama import LlamaDecoder
    cfg = dict(synth.TINY_LLAMA)
    cfg["n_layers"] = 5                                   # staging buffers are reused: 0, 1, 0, 1, 0
    w = synth.llama_weights(cfg, seed=9, std=0.02)
    hkv, d, nl = cfg["n_kv_heads"], cfg["head_dim"], cfg["n_layers"]
    n_seq, n_pool_blocks, max_blocks = 6, 512, 8

    def get_weight(name, layer):
        return bf16_tensor(w[name] if layer is None else w["layers"][layer][name], dev)

    decs = [LlamaDecoder(cfg, get_weight, 0.25, n_pool_blocks, 2, n_seq, max_blocks, dev, kv_prefetch=pf)
            for pf in (False, True)]
    assert decs[1].layers[0]["k"].n_host > 0
    k_host = [synth.normal_bf16((hkv, n_pool_blocks, 16, d), 1.0, 300 + li) for li in range(nl)]
    v_host = [synth.normal_bf16((hkv, n_pool_blocks, 16, d), 1.0, 400 + li) for li in range(nl)]
    for dec in decs:
        load_caches(dev, dec, k_host, v_host)
    rng = np.random.default_rng(3)
    ctx = rng.integers(5, 60, size=n_seq).astype(np.int32)
    table = np.zeros((n_seq, max_blocks), np.int32)
    for b in range(n_seq):
        for j in range(max_blocks):
            got = [dec.pool.alloc(b, 1)[0] for dec in decs]
            assert got[0] == got[1]
            table[b, j] = got[0]
    table_dev = torch.from_numpy(table).to(dev)
    tok0 = torch.from_numpy(rng.integers(0, cfg["vocab"], size=n_seq).astype(np.int32)).to(dev)
    tok = [tok0, tok0.clone()]
    nxt = [torch.zeros(n_seq, dtype=torch.int32, device=dev) for _ in decs]
    for step in range(6):
        ctx += 1
        ctx_dev = torch.from_numpy(ctx).to(dev)
        n0 = decs[0].step(tok[0], table_dev, ctx_dev, nxt[0])
        n1 = decs[1].step_prefetch(tok[1], table_dev, ctx_dev, nxt[1])
        torch.cuda.synchronize()
        assert n0 == n1 and 5 + 2 * nl <= n0 <= 5 + 3 * nl + 1
        assert torch.equal(decs[0].buf["logits"][:n_seq], decs[1].buf["logits"][:n_seq]), step
        assert torch.equal(nxt[0], nxt[1])
        tok = [nxt[0].clone(), nxt[1].clone()]
    for li in range(nl):
        for name in ("k", "v"):
            assert np.array_equal(dump_cache(dev, decs[0], li, name), dump_cache(dev, decs[1], li, name))
    assert decs[0].status_words() == [0, 0] and decs[1].status_words() == [0, 0]
