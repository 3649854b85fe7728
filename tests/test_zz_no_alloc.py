"""The allocation-free stream reduce (scratch inside the library) against the ordinary
entry point.  Collected last on purpose: if it fails, every other test has already run.

Some callers cannot allocate scratch at call time - an engine that reserved all GPU memory
up front, a plug-in confined to its host's allocator - so this entry point takes none; the
test checks that it gives exactly the sums of boost_stream_reduce_tiered, twice in a row
(the second call finds the shared scratch as the first one left it), and that it refuses
buffers beyond its stated limit."""
import numpy as np
import pytest

from paper_2609_13592_b200 import binding as B
from paper_2609_13592_b200 import synth

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

PAGE_ELEMS = B.PAGE_BYTES // 2


def test_static_scratch_stream_reduce_matches_workspace_version():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2609_13592_b200 import build
    from paper_2609_13592_b200.tiers import TieredBuffer
    build.build_library()
    dev = torch.device("cuda:0")
    assert B.boost_stream_reduce_static_max_pages() == 4096
    for n_pages, ratio, start in ((21, 1 / 4, 0), (9, 1 / 2, 777)):
        buf = TieredBuffer(n_pages * B.PAGE_BYTES, ratio, device=dev)
        buf.scatter_from(synth.small_int_bf16_torch(start, n_pages * PAGE_ELEMS, dev))
        ws_bytes = B.boost_stream_reduce_workspace_bytes(n_pages)
        ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
        want = torch.zeros(n_pages, dtype=torch.float32, device=dev)
        B.boost_stream_reduce_tiered(buf.page_ptr, buf.order, n_pages, buf.n_host, want, ws, ws_bytes)
        torch.cuda.synchronize()
        for call in range(2):
            got = torch.full((n_pages,), float("nan"), dtype=torch.float32, device=dev)
            B.boost_stream_reduce_tiered_static(buf.page_ptr, buf.order, n_pages, buf.n_host, got)
            torch.cuda.synchronize()
            # integer-valued data: the sums are exact, so the two entry points agree bit for bit
            assert torch.equal(got, want), (n_pages, call)
    # beyond the built-in limit the call refuses instead of overrunning its scratch
    with pytest.raises(B.BoostError) as e:
        B.boost_stream_reduce_tiered_static(buf.page_ptr, buf.order, 4097, 0, got)
    assert e.value.code == B.ERR_CAPACITY
