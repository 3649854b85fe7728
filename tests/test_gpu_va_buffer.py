"""GPU: one virtual address range over both tiers (CUDA virtual-memory API).  The range is a flat
buffer for a plain copy, its pages are where the tier table says, and the library's kernels read
it through the trivial page table base + i * 2 MiB with the same bits as a slab-backed buffer."""
import numpy as np
import pytest

from oracle import linalg as ol
from oracle import placement as op
from paper_2609_13592_b200 import binding as B
from paper_2609_13592_b200 import synth

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
    return torch.device("cuda:0")


def make(tier):
    try:
        return B.VABuffer(tier)
    except B.BoostError as e:
        if e.code == B.ERR_UNSUPPORTED:
            pytest.skip("this driver / platform maps no host-NUMA memory into a device address range")
        raise


def memcpy(dst, src, n_bytes):
    """One plain cudaMemcpy between two device addresses (the CUDA runtime through its Python binding)."""
    runtime = pytest.importorskip("cuda.bindings.runtime")
    err, = runtime.cudaMemcpy(dst, src, n_bytes, runtime.cudaMemcpyKind.cudaMemcpyDefault)
    assert int(err) == 0, err


@pytest.mark.parametrize("n_pages,ratio,policy", [(37, 1 / 8, B.POLICY_MODULO), (16, 1 / 4, B.POLICY_CONTIGUOUS),
                                                   (5, 0.0, B.POLICY_MODULO)])
def test_va_buffer_is_flat_and_tiered(dev, n_pages, ratio, policy):
    tier, _ = B.boost_place_pages_ex(None, n_pages * PAGE, ratio, 0, policy, 0, 1)
    assert tier.tolist() == op.place_pages(n_pages * PAGE, ratio, policy)
    buf = make(tier)
    table = buf.page_table()
    assert table.tolist() == [buf.base + i * PAGE for i in range(n_pages)]
    # one flat copy in, one flat copy out: the range is contiguous for the copy engine
    n_elems = n_pages * PAGE_ELEMS
    src = synth.small_int_bf16_torch(3, n_elems, dev)
    memcpy(buf.base, src.data_ptr(), n_pages * PAGE)
    back = torch.zeros_like(src)
    memcpy(back.data_ptr(), buf.base, n_pages * PAGE)
    torch.cuda.synchronize()
    assert torch.equal(src, back)
    # every page is where the tier table says: the runtime reports the memory type per address
    runtime = pytest.importorskip("cuda.bindings.runtime")
    for i in range(n_pages):
        err, attr = runtime.cudaPointerGetAttributes(buf.base + i * PAGE)
        assert int(err) == 0
        want_type = runtime.cudaMemoryType.cudaMemoryTypeHost if tier[i] else runtime.cudaMemoryType.cudaMemoryTypeDevice
        assert attr.type == want_type, (i, int(tier[i]), attr.type)
    # the stream-reduce kernel over the range's page table, host pages first: page sums bit for bit
    page_ptr = torch.from_numpy(table.view(np.int64).copy()).to(dev)
    order, n_host = B.boost_tier_order(tier)
    assert n_host == int(tier.sum())
    order_d = torch.from_numpy(order.view(np.int32).copy()).to(dev)
    ws_bytes = B.boost_stream_reduce_workspace_bytes(n_pages)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    sums = torch.zeros(n_pages, dtype=torch.float32, device=dev)
    B.boost_stream_reduce_tiered(page_ptr, order_d, n_pages, n_host, sums, ws, ws_bytes)
    torch.cuda.synchronize()
    want, _ = ol.stream_sum(synth.small_int_bf16(3, n_elems), PAGE_ELEMS)
    assert np.array_equal(sums.cpu().numpy().astype(np.float64), want)
    assert int(ws[:4].view(torch.int32)[0]) == 0
    buf.close()


def test_weight_product_over_a_va_buffer(dev):
    """A packed weight whose pages are a VA buffer's: the same product, the same bits as with slabs."""
    from paper_2609_13592_b200.tiers import TieredWeight
    n, k, m_b = 2048, 4096, 8                      # 16 row tiles x 64 k-blocks = 8 pages
    w_bits = synth.normal_bf16((n, k), 0.02, 1)
    x_bits = synth.normal_bf16((m_b, k), 1.0, 2)
    w_dev = torch.from_numpy(w_bits.view(np.int16)).to(dev).view(torch.bfloat16)
    x = torch.from_numpy(x_bits.view(np.int16)).to(dev).view(torch.bfloat16)
    tier = np.array([0, 0, 0, 1, 0, 0, 0, 1], np.uint8)
    ref_w = TieredWeight(w_dev, device=dev, tier=tier)
    y_ref = ref_w.gemv(x).clone()
    buf = make(tier)
    page_ptr = torch.from_numpy(buf.page_table().view(np.int64).copy()).to(dev)
    B.boost_pack_weights_ex(w_dev, n, k, page_ptr, 8, 0, None)
    y = torch.zeros(m_b, n, dtype=torch.float32, device=dev)
    ws_ptr, ws_bytes = ref_w.workspace(m_b)
    B.boost_gemv_tiered(page_ptr, ref_w.buf.order, 8, 2, n, k, x, m_b, y, 0, None, ws_ptr, ws_bytes)
    torch.cuda.synchronize()
    assert torch.equal(y, y_ref)
    from tests.helpers import assert_close_to_oracle
    assert_close_to_oracle(y.cpu().numpy(), ol.gemm(x_bits, w_bits), "product over a VA buffer")
    assert ref_w.status_words() == [0]
    buf.close()
