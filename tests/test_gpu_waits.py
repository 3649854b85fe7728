"""GPU: the bounded waits of the weight-product kernels really run out and wind the kernel down.

Every wait inside the kernels (on a shared-memory barrier, on a grid-wide counter) gives up after
a limit, records bit 0 in the workspace's status word and makes every role of the threadblock
leave.  In normal operation no wait ever gets near the limit (about a second), so this file makes
one run out on purpose, the gentle way: two words of the workspace header shorten the limit to
about a millisecond and tell threadblock 0 to leave out one phase-boundary arrival, so the warps
that wait for that count give up.  Nothing faults, traps or spins without bound; the kernel returns,
the status word says what happened, and after the workspace is zero-filled again the next launch is
bit for bit what it was before."""
import numpy as np
import pytest

from paper_2609_13592_b200 import binding as B
from paper_2609_13592_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

WS_WAIT_LIMIT_WORD, WS_SKIP_ARRIVALS_WORD = 4, 5


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


@pytest.mark.parametrize("m_b", [24, 70])       # the mma.sync kernel, the tcgen05 kernel
def test_missing_arrival_times_out_and_kernel_returns(dev, m_b):
    from paper_2609_13592_b200.tiers import TieredWeight, aligned_workspace
    kin, hid, ffn, stride = 768, 1024, 1536, 128
    x = bf16_tensor(synth.normal_bf16((m_b, kin), 1.0, 1), dev)
    h0 = bf16_tensor(synth.normal_bf16((m_b, hid), 1.0, 2), dev)
    gamma = bf16_tensor(synth.f32_to_bf16_bits(np.ones(hid, np.float32)), dev)
    w0 = TieredWeight(bf16_tensor(synth.normal_bf16((hid, kin), 0.03, 5), dev), device=dev)
    w1 = TieredWeight(bf16_tensor(synth.normal_bf16((2 * ffn, hid), 0.03, 6), dev), device=dev, row_mode=1, col_scale=gamma)

    def epi(mode, ssq_in=None, ssq_out=None):
        e = B.GemvEpilogue()
        e.mode, e.ssq_stride, e.rms_eps, e.ssq_in_tiles = mode, stride, 1e-5, hid // 128
        e.ssq_in = None if ssq_in is None else ssq_in.data_ptr()
        e.ssq_out = None if ssq_out is None else ssq_out.data_ptr()
        return e

    def run(ws_ptr, ws_bytes):
        h = h0.clone()
        act = torch.zeros(m_b, ffn, dtype=torch.bfloat16, device=dev)
        ssq = torch.zeros(hid // 128, stride, dtype=torch.float32, device=dev)
        calls = B.gemv_calls([
            dict(w=w0.struct(), x=x, y=h, y_dtype=1, residual=h, epilogue=epi(B.EPI_PLAIN, ssq_out=ssq)),
            dict(w=w1.struct(), x=h, y=act, y_dtype=1, epilogue=epi(B.EPI_SWIGLU, ssq_in=ssq))])
        B.boost_gemv_tiered_chain(calls, m_b, ws_ptr, ws_bytes)
        torch.cuda.synchronize()          # the launch has come back: nothing hangs
        return h, act

    probe = B.gemv_calls([dict(w=w0.struct(), x=x, y=h0, y_dtype=1), dict(w=w1.struct(), x=h0, y=h0, y_dtype=1)])
    ws_bytes = B.boost_gemv_chain_workspace_bytes(probe, m_b)
    ws_t, ws_ptr = aligned_workspace(ws_bytes, dev)
    off = ws_ptr - ws_t.data_ptr()
    header = ws_t[off:off + 64].view(torch.int32)

    good_h, good_act = run(ws_ptr, ws_bytes)
    assert int(header[0]) == 0
    assert float(good_act.float().abs().sum()) > 0

    # about a millisecond instead of a second, and threadblock 0 keeps its arrival at the end of
    # the first product to itself: the activation warps of the second product wait in vain
    header[WS_WAIT_LIMIT_WORD] = 2_000_000
    header[WS_SKIP_ARRIVALS_WORD] = 1
    torch.cuda.synchronize()
    run(ws_ptr, ws_bytes)                 # outputs of this launch mean nothing
    assert int(header[0]) & 1 == 1        # kErrWaitTimeout is on record

    # a status word that is not zero means: zero-fill the workspace before the next launch
    ws_t.zero_()
    torch.cuda.synchronize()
    again_h, again_act = run(ws_ptr, ws_bytes)
    assert int(header[0]) == 0
    assert torch.equal(again_h, good_h) and torch.equal(again_act, good_act)


def test_missing_partial_sum_times_out_in_tile_finish(dev):
    """tcgen05 kernel, tile-by-tile mode: the threadblock that holds a row tile's last partial sum
    waits until the others' are in memory before it finishes the tile from tensor memory.  Every
    threadblock here keeps that announcement to itself, the waits give up after the shortened limit,
    the kernel returns with the time-out on record, and after a zero-fill the next launch is bit
    for bit what it was."""
    from paper_2609_13592_b200.tiers import TieredWeight, aligned_workspace
    m_b, hid, n = 96, 192, 77824                    # 608 row tiles on 148 threadblocks: most tiles in two or three pieces
    x = bf16_tensor(synth.normal_bf16((m_b, hid), 1.0, 1), dev)
    w = TieredWeight(bf16_tensor(synth.normal_bf16((n, hid), 0.05, 2), dev), device=dev)
    ws_bytes = B.boost_gemv_workspace_bytes(n, hid, m_b)
    ws_t, ws_ptr = aligned_workspace(ws_bytes, dev)
    off = ws_ptr - ws_t.data_ptr()
    header = ws_t[off:off + 64].view(torch.int32)

    def run():
        y = w.gemv(x, y_dtype=torch.float32, workspace=(ws_ptr, ws_bytes))
        torch.cuda.synchronize()
        return y

    good = run()
    assert int(header[0]) == 0 and float(good.abs().sum()) > 0
    header[WS_WAIT_LIMIT_WORD] = 2_000_000
    header[WS_SKIP_ARRIVALS_WORD] = 1 << 20         # every threadblock
    torch.cuda.synchronize()
    run()
    assert int(header[0]) & 1 == 1
    ws_t.zero_()
    torch.cuda.synchronize()
    again = run()
    assert int(header[0]) == 0 and torch.equal(again, good)
