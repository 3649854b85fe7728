"""A peer GPU's HBM as the second tier ("Bandwidth Ratio Ablation with NVLinks"): the set-up calls
on any GPU machine, and - where a second GPU with peer access is present - the stream reduce and the
weight product over pages that live in the peer's memory, against the oracle."""
import numpy as np
import pytest

from oracle import linalg as ol
from oracle import placement as op
from paper_2609_13592_b200 import binding as B
from paper_2609_13592_b200 import synth
from tests.helpers import assert_close_to_oracle

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

PAGE = B.PAGE_BYTES
PAGE_ELEMS = PAGE // 2


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2609_13592_b200 import build
    build.build_library()
    B.lib()
    torch.cuda.set_device(0)
    torch.zeros(1, device="cuda:0")   # a context on device 0
    return torch.device("cuda:0")


@pytest.fixture(scope="module")
def peer(dev):
    if torch.cuda.device_count() < 2:
        pytest.skip("needs a second GPU")
    try:
        B.boost_peer_tier_open(1)
    except B.BoostError as e:
        if e.code == B.ERR_UNSUPPORTED:
            pytest.skip("no peer access between GPU 0 and GPU 1")
        raise
    return 1


def test_peer_tier_argument_errors(dev):
    n = torch.cuda.device_count()
    for bad in (0, -1, n, n + 7):   # the current device itself, and ordinals that do not exist
        with pytest.raises(B.BoostError) as e:
            B.boost_peer_tier_open(bad)
        assert e.value.code == B.ERR_INVALID
        with pytest.raises(B.BoostError) as e:
            B.boost_peer_tier_alloc(bad, PAGE)
        assert e.value.code == B.ERR_INVALID
    B.boost_peer_tier_free(0, None)   # nothing to free: accepted
    assert torch.cuda.current_device() == 0


def test_stream_reduce_over_peer_pages(dev, peer):
    from paper_2609_13592_b200.tiers import TieredBuffer
    n_pages, ratio = 40, 1 / 8
    n_elems = n_pages * PAGE_ELEMS
    buf = TieredBuffer(n_elems * 2, ratio, B.POLICY_MODULO, device=dev, peer_device=peer)
    assert buf.tier.tolist() == op.place_pages(n_elems * 2, ratio) and buf.n_host == 5
    # the second-tier pages really are in the peer's memory
    rt = pytest.importorskip("cuda.bindings.runtime")
    for address in buf.page_table_host[buf.tier == B.TIER_HOST]:
        err, attr = rt.cudaPointerGetAttributes(int(address))
        assert int(err) == 0 and attr.device == peer
    for address in buf.page_table_host[buf.tier == B.TIER_HBM][:3]:
        err, attr = rt.cudaPointerGetAttributes(int(address))
        assert int(err) == 0 and attr.device == 0
    buf.scatter_from(synth.small_int_bf16_torch(3, n_elems, dev))
    ws_bytes = B.boost_stream_reduce_workspace_bytes(n_pages)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    sums = torch.zeros(n_pages, dtype=torch.float32, device=dev)
    B.boost_stream_reduce_tiered(buf.page_ptr, buf.order, n_pages, buf.n_host, sums, ws, ws_bytes)
    torch.cuda.synchronize()
    want, _ = ol.stream_sum(synth.small_int_bf16(3, n_elems), PAGE_ELEMS)
    assert np.array_equal(sums.cpu().numpy().astype(np.float64), want)
    assert int(ws[:4].cpu().numpy().view(np.uint32)[0]) == 0
    assert torch.cuda.current_device() == 0


@pytest.mark.parametrize("m_b", [1, 8, 32, 64])
def test_weight_product_over_peer_pages(dev, peer, m_b):
    from paper_2609_13592_b200.tiers import TieredWeight
    n, k = 4096, 4096
    w_bits = synth.normal_bf16((n, k), 0.02, 11)
    x_bits = synth.normal_bf16((m_b, k), 1.0, 12)
    as_dev = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)
    w = TieredWeight(as_dev(w_bits), 1 / 8, device=dev, peer_device=peer)
    assert w.buf.n_host == 2
    y = w.gemv(as_dev(x_bits))
    torch.cuda.synchronize()
    ref = ol.gemm(x_bits, w_bits)
    got = y.float().cpu().numpy()
    for r in range(m_b):
        assert_close_to_oracle(got[r], ref[r], f"row {r}")
    assert w.status_words() == [0]
