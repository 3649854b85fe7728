"""GPU: the schedule the tier-aware kernels realise (which tier every work item streamed, from
when to when), logged by the kernels on request and turned into host-share statistics per wave
of work and per stretch of time - by the library and, from the same log, by the oracle."""
import numpy as np
import pytest

from oracle import kv_pool as okp
from oracle import placement as op
from paper_2609_13592_b200 import binding as B
from paper_2609_13592_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu
PAGE = B.PAGE_BYTES


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


def make_log(dev, capacity):
    log = torch.zeros(B.boost_schedule_log_bytes(capacity), dtype=torch.uint8, device=dev)
    log[:32].view(torch.int64)[1] = capacity
    return log


def attach(ws_tensor, ws_ptr, log):
    """Put the log's address into words 6 and 7 of the workspace header (None: take it out)."""
    off = ws_ptr - ws_tensor.data_ptr()
    ws_tensor[off:off + 64].view(torch.int64)[B.WS_LOG_WORD // 2] = 0 if log is None else log.data_ptr()
    torch.cuda.synchronize()


def check_against_oracle(log, kind, per_wave, window_ns, ratio):
    host = log.cpu().numpy()
    recs, claimed = B.schedule_records(host)
    assert claimed == len(recs) > 0                                  # nothing dropped
    tuples = [tuple(int(v) for v in r) for r in recs]
    got = B.boost_schedule_stats(host, kind, per_wave, window_ns, ratio)
    ref = op.schedule_stats(tuples, per_wave, window_ns, ratio, kind)
    assert got[2] == ref[2]
    for g, r in zip(got[:2], ref[:2]):
        for key in ("n_waves", "n_host_pages", "n_zero_waves"):
            assert g[key] == r[key], key
        for key in ("mean", "var", "min", "max"):
            assert abs(g[key] - r[key]) <= 1e-12 * max(1.0, abs(r[key])), key
    return recs, got


def test_stream_reduce_schedule(dev):
    """Configuration 3's kernel on 256 pages with one page in 16 on the host: every tile is logged
    once, the tiers' bytes add up, and the host tier streams from the first window on (host tiles
    are handed out first) instead of all at the end of the address range."""
    from paper_2609_13592_b200.tiers import TieredBuffer
    n_pages = 256
    buf = TieredBuffer(n_pages * PAGE, 1 / 16, B.POLICY_CONTIGUOUS, device=dev)   # host pages at the END of the buffer
    assert buf.n_host == 16 and buf.tier[-16:].all()
    buf.scatter_from(synth.small_int_bf16_torch(0, n_pages * PAGE // 2, dev))
    ws_bytes = B.boost_stream_reduce_workspace_bytes(n_pages)
    ws = torch.zeros(ws_bytes + 256, dtype=torch.uint8, device=dev)
    ws_ptr = ws.data_ptr() + (-ws.data_ptr()) % 256
    sums = torch.zeros(n_pages, dtype=torch.float32, device=dev)
    B.boost_stream_reduce_tiered(buf.page_ptr, buf.order, n_pages, buf.n_host, sums, ws_ptr, ws_bytes)   # warm-up, no log
    torch.cuda.synchronize()
    want = sums.clone()
    log = make_log(dev, 16 * n_pages + 8)
    attach(ws, ws_ptr, log)
    B.boost_stream_reduce_tiered(buf.page_ptr, buf.order, n_pages, buf.n_host, sums, ws_ptr, ws_bytes)
    torch.cuda.synchronize()
    assert torch.equal(sums, want)                                   # logging changes no result
    recs, (waves, windows, n) = check_against_oracle(log, B.SCHED_KIND_STREAM, 148 * 4, 2000, 1 / 16)
    assert n == 16 * n_pages and (recs["kind_phase"] == B.SCHED_KIND_STREAM).all()
    assert int(recs["bytes"].sum()) == n_pages * PAGE and int(recs["host_bytes"].sum()) == buf.n_host * PAGE
    assert (recs["t_consumed"] > recs["t_request"]).all()
    # address order would give waves of share 0, 0, ..., 1 (contiguous placement); the queues put a
    # host tile into the very first wave of starts and keep the link busy from the first window
    first_wave = np.sort(recs, order=["t_request", "cta_warp"])[:148 * 4]
    assert first_wave["host_bytes"].sum() > 0
    addr = op.wave_stats(buf.tier.tolist(), 128 * 1024, 148 * 4, 1 / 16)
    assert addr["n_zero_waves"] >= addr["n_waves"] - 1 > 1
    assert windows["n_zero_waves"] <= windows["n_waves"] // 4        # most of the run reads both tiers at once
    attach(ws, ws_ptr, None)


@pytest.mark.parametrize("two_queues", [False, True])
def test_gemv_chain_and_attention_schedule(dev, two_queues):
    from paper_2609_13592_b200.tiers import TieredKVCache, TieredWeight, aligned_workspace
    # a two-product chain: the first weight has a host page (read in place under the even
    # partition, or cut into queue items handed out host first), the second is all HBM (even
    # partition: one record per threadblock and row tile it touches)
    B.boost_gemv_set_tier_schedule(two_queues)
    m_b, kin, hid, ffn, stride = 32, 2048, 2048, 2048, 128
    t8 = lambda *t: np.array(t, np.uint8)
    w0 = TieredWeight(bf16_tensor(synth.normal_bf16((hid, kin), 0.03, 5), dev), device=dev, tier=t8(0, 1, 0, 0))
    gamma = bf16_tensor(synth.f32_to_bf16_bits(np.ones(hid, np.float32)), dev)
    w1 = TieredWeight(bf16_tensor(synth.normal_bf16((2 * ffn, hid), 0.03, 6), dev), device=dev, row_mode=1, col_scale=gamma)
    x = bf16_tensor(synth.normal_bf16((m_b, kin), 1.0, 1), dev)
    h = bf16_tensor(synth.normal_bf16((m_b, hid), 1.0, 2), dev)
    act = torch.zeros(m_b, ffn, dtype=torch.bfloat16, device=dev)
    ssq = torch.zeros(hid // 128, stride, dtype=torch.float32, device=dev)

    def epi(mode, ssq_in=None, ssq_out=None):
        e = B.GemvEpilogue()
        e.mode, e.ssq_stride, e.rms_eps, e.ssq_in_tiles = mode, stride, 1e-5, hid // 128
        e.ssq_in = None if ssq_in is None else ssq_in.data_ptr()
        e.ssq_out = None if ssq_out is None else ssq_out.data_ptr()
        return e

    calls = B.gemv_calls([dict(w=w0.struct(), x=x, y=h, y_dtype=1, epilogue=epi(B.EPI_PLAIN, ssq_out=ssq)),
                          dict(w=w1.struct(), x=h, y=act, y_dtype=1, epilogue=epi(B.EPI_SWIGLU, ssq_in=ssq))])
    ws_bytes = B.boost_gemv_chain_workspace_bytes(calls, m_b)
    ws_t, ws_ptr = aligned_workspace(ws_bytes, dev)
    B.boost_gemv_tiered_chain(calls, m_b, ws_ptr, ws_bytes)
    torch.cuda.synchronize()
    want = act.clone()
    log = make_log(dev, 4096)
    attach(ws_t, ws_ptr, log)
    B.boost_gemv_tiered_chain(calls, m_b, ws_ptr, ws_bytes)
    torch.cuda.synchronize()
    assert torch.equal(act, want)
    recs, (waves, windows, n) = check_against_oracle(log, B.SCHED_KIND_GEMV, 64, 1000, 0.25)
    phase = recs["kind_phase"] >> 8
    assert set(phase.tolist()) == {0, 1}
    for ph, tw in ((0, w0), (1, w1)):
        mine = recs[phase == ph]
        assert int(mine["bytes"].sum()) == tw.layout["n_row_tiles"] * tw.layout["k_blocks"] * 16384   # every block once
        assert int(mine["host_bytes"].sum()) == tw.buf.n_host * PAGE
    assert (recs["t_consumed"] > recs["t_request"]).all()
    # the second product's weights start streaming before the first product's last item is consumed
    assert recs[phase == 1]["t_request"].min() < recs[phase == 0]["t_consumed"].max()
    attach(ws_t, ws_ptr, None)
    B.boost_gemv_set_tier_schedule(False)

    # attention over a pool with a quarter of its pages on the host: records per warp and item
    n_seq, hq, hkv, d, n_blocks, modulus = 6, 8, 2, 128, 2048, 4
    ctx = [700, 33, 260, 1500, 16, 901]
    pool = B.KVPool(n_blocks, hkv, modulus)
    table = np.zeros((n_seq, 128), np.int32)
    for b, c in enumerate(ctx):
        nb = (c + 15) // 16
        table[b, :nb] = pool.alloc(b, nb)
    cache = TieredKVCache(pool, hkv, n_blocks, d, dev)
    assert int((cache.tier == 1).sum()) == 2
    cache.load(bf16_tensor(synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 8), dev),
               bf16_tensor(synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, 9), dev))
    q = bf16_tensor(synth.normal_bf16((n_seq, hq, d), 1.0, 10), dev)
    out = torch.zeros(n_seq, hq, d, dtype=torch.bfloat16, device=dev)
    aws_bytes = B.boost_paged_attn_workspace_bytes(n_seq, hq, d, 128)
    aws_t, aws = aligned_workspace(aws_bytes, dev)
    args = (q, cache.k.page_ptr, cache.v.page_ptr, cache.tier, cache.n_pages, n_blocks, torch.from_numpy(table).to(dev), 128,
            torch.from_numpy(np.array(ctx, np.int32)).to(dev), n_seq, hq, hkv, d, 1.0 / np.sqrt(d), aws, aws_bytes, out)
    B.boost_paged_attn_decode_tiered(*args)
    torch.cuda.synchronize()
    want = out.clone()
    log = make_log(dev, 4096)
    attach(aws_t, aws, log)
    B.boost_paged_attn_decode_tiered(*args)
    torch.cuda.synchronize()
    assert torch.equal(out, want)
    recs, _ = check_against_oracle(log, B.SCHED_KIND_ATTN, 32, 500, 0.25)
    blocks = sum((c + 15) // 16 for c in ctx)
    assert int(recs["bytes"].sum()) == blocks * hkv * 8192            # every (block, KV head) once: 4 KiB of K + 4 KiB of V
    # host bytes: the blocks whose chunk of a head lies in a host page, from the pool's own tier table
    tier = cache.tier
    host_chunks = sum(int(tier[(g * n_blocks + int(blk)) // 512]) for b, c in enumerate(ctx)
                      for blk in table[b, :(c + 15) // 16] for g in range(hkv))
    assert int(recs["host_bytes"].sum()) == host_chunks * 8192 and host_chunks > 0
    pool.close()
