"""Device-memory plumbing for tiered buffers: slabs, page tables, visit order.

PyTorch allocates the HBM slab and the pinned host slab; the library decides
the placement (boost_place_pages*), assigns page addresses (boost_page_table)
and orders the pages for the kernels (boost_tier_order).  No arithmetic of the
method lives here.
"""
import numpy as np
import torch

from . import binding as B

PAGE = B.PAGE_BYTES


def _aligned(t, align=PAGE):
    """Address inside the uint8 tensor t aligned up to `align`."""
    p = t.data_ptr()
    return (p + align - 1) // align * align


class Slabs:
    """An HBM slab and a pinned host slab that several TieredBuffers may map their pages onto
    (for placement sweeps, where only the page table changes between runs)."""

    def __init__(self, hbm_pages, host_pages, device="cuda", peer_device=None):
        self.device = torch.device(device)
        self.hbm_pages, self.host_pages = hbm_pages, host_pages
        self._hbm = torch.empty(hbm_pages * PAGE + PAGE, dtype=torch.uint8, device=self.device)
        self.hbm_base = _aligned(self._hbm)
        if peer_device is None:
            self._host = torch.empty(max(host_pages, 1) * PAGE + PAGE, dtype=torch.uint8, pin_memory=True)
            self.host_base_cpu = _aligned(self._host)
            self.host_base = B.boost_host_device_pointer(self.host_base_cpu)
        else:
            self._host = PeerSlab(peer_device, max(host_pages, 1) * PAGE + PAGE)
            self.host_base_cpu, self.host_base = 0, self._host.base


class PeerSlab:
    """Second-tier pages in a peer GPU's HBM (read over NVLink): a slab on peer_device that the
    kernels of the current device may read.  Freed with the object."""

    def __init__(self, peer_device, n_bytes):
        self.peer_device = int(peer_device)
        B.boost_peer_tier_open(self.peer_device)
        self.ptr = B.boost_peer_tier_alloc(self.peer_device, n_bytes)
        self.base = (self.ptr + PAGE - 1) // PAGE * PAGE

    def __del__(self):
        ptr, self.ptr = getattr(self, "ptr", 0), 0
        if ptr:
            try:
                B.boost_peer_tier_free(self.peer_device, ptr)
            except Exception:
                pass


class TieredBuffer:
    """A buffer of n_bytes cut into 2 MiB pages placed over HBM and pinned host memory."""

    def __init__(self, n_bytes, host_ratio=0.0, policy=B.POLICY_MODULO, seed=0, superpage_pages=1,
                 device="cuda", tier=None, wave_size=0, slabs=None, peer_device=None):
        """peer_device: ordinal of a second GPU whose HBM holds the second-tier pages instead of
        pinned host memory (scatter_from / gather_to and the kernels work unchanged)."""
        self.n_bytes = int(n_bytes)
        self.device = torch.device(device)
        if tier is None:
            tier, self.flags = B.boost_place_pages_ex(None, self.n_bytes, host_ratio, wave_size, policy,
                                                      seed, superpage_pages)
        else:
            tier, self.flags = np.ascontiguousarray(tier, dtype=np.uint8), 0
        self.tier = tier
        self.n_pages = int(tier.size)
        self.n_host = int((tier == B.TIER_HOST).sum())
        self.n_hbm = self.n_pages - self.n_host
        if slabs is not None:
            assert self.n_hbm <= slabs.hbm_pages and self.n_host <= slabs.host_pages
            self._hbm, self.hbm_base = slabs._hbm, slabs.hbm_base
            self._host, self.host_base_cpu, self.host_base = slabs._host, slabs.host_base_cpu, slabs.host_base
        else:
            self._hbm = torch.empty(self.n_hbm * PAGE + PAGE, dtype=torch.uint8, device=self.device)
            self.hbm_base = _aligned(self._hbm)
        if slabs is not None:
            pass
        elif self.n_host and peer_device is not None:
            self._host = PeerSlab(peer_device, self.n_host * PAGE + PAGE)
            self.host_base_cpu, self.host_base = 0, self._host.base
        elif self.n_host:
            self._host = torch.empty(self.n_host * PAGE + PAGE, dtype=torch.uint8, pin_memory=True)
            self.host_base_cpu = _aligned(self._host)
            self.host_base = B.boost_host_device_pointer(self.host_base_cpu)
        else:
            self._host, self.host_base_cpu, self.host_base = None, 0, 0
        table = B.boost_page_table(tier, self.hbm_base, self.n_hbm * PAGE,
                                   self.host_base or None, self.n_host * PAGE)
        self.page_table_host = table
        self.page_ptr = torch.from_numpy(table.view(np.int64).copy()).to(self.device)
        order, n_host = B.boost_tier_order(tier)
        assert n_host == self.n_host
        self.order_host = order
        self.order = torch.from_numpy(order.view(np.int32).copy()).to(self.device)

    def staged_page_ptr(self, stage_base):
        """Page table in which every host page points at its slot of a staging buffer in HBM
        (device address stage_base, n_host pages long) instead of the pinned slab."""
        table = B.boost_page_table(self.tier, self.hbm_base, self.n_hbm * PAGE, stage_base or None,
                                   self.n_host * PAGE)
        return torch.from_numpy(table.view(np.int64).copy()).to(self.device)

    def scatter_from(self, flat, stream=None):
        """Copy a contiguous device tensor (any dtype) of n_bytes into the pages."""
        assert flat.is_cuda and flat.is_contiguous() and flat.numel() * flat.element_size() == self.n_bytes
        B.boost_scatter_pages(flat, self.n_bytes, self.page_ptr, self.n_pages, stream)

    def gather_to(self, flat, stream=None):
        assert flat.is_cuda and flat.is_contiguous() and flat.numel() * flat.element_size() == self.n_bytes
        B.boost_gather_pages(flat, self.n_bytes, self.page_ptr, self.n_pages, stream)


class TieredWeight:
    """A row-major bf16 weight [N, K] packed into tiered pages for boost_gemv_tiered."""

    def __init__(self, w, host_ratio=0.0, policy=B.POLICY_MODULO, seed=0, device="cuda", tier=None,
                 superpage_pages=1, row_mode=0, col_scale=None, peer_device=None):
        """row_mode 1 interleaves the two halves of the rows (gate / up) per 64 rows; col_scale
        (bf16 [K]) is an RMSNorm weight folded into the matrix (see boost_pack_weights_ex)."""
        assert w.dtype == torch.bfloat16 and w.dim() == 2 and w.is_cuda and w.is_contiguous()
        self.N, self.K = int(w.shape[0]), int(w.shape[1])
        self.layout = B.boost_weight_layout(self.N, self.K)
        self.buf = TieredBuffer(self.layout["bytes"], host_ratio, policy, seed, superpage_pages, device, tier,
                                peer_device=peer_device)
        B.boost_pack_weights_ex(w, self.N, self.K, self.buf.page_ptr, self.buf.n_pages, row_mode, col_scale)
        torch.cuda.current_stream().synchronize()
        self._ws = {}

    def struct(self):
        """The weight as the binding.Weight structure that chains and the decode step take."""
        return B.Weight(self.buf.page_ptr.data_ptr(), self.buf.order.data_ptr(), self.buf.n_pages, self.buf.n_host,
                        self.N, self.K)

    def workspace(self, m_b):
        n = B.boost_gemv_workspace_bytes(self.N, self.K, m_b)
        ws = self._ws.get(n)
        if ws is None:
            ws = torch.zeros(n + 256, dtype=torch.uint8, device=self.buf.device)
            self._ws[n] = ws
        off = (-ws.data_ptr()) % 256
        return ws.data_ptr() + off, n

    def status_words(self):
        """Status word (sticky error bits) of every workspace this weight has used."""
        out = []
        for ws in self._ws.values():
            off = (-ws.data_ptr()) % 256
            out.append(int(ws[off:off + 4].cpu().numpy().view(np.uint32)[0]))
        return out

    def gemv(self, x, y=None, y_dtype=torch.float32, residual=None, workspace=None, stream=None,
             epilogue=None):
        """y = x @ W^T (+ residual); x bf16 [M_b, K] (or [K]).  epilogue: a binding.GemvEpilogue
        (then y may be None for the RoPE-append mode)."""
        x2 = x.reshape(-1, self.K)
        m_b = x2.shape[0]
        if y is None and (epilogue is None or epilogue.mode != B.EPI_ROPE_APPEND):
            n_out = self.N // 2 if (epilogue is not None and epilogue.mode == B.EPI_SWIGLU) else self.N
            y = torch.empty(m_b, n_out, dtype=y_dtype, device=x.device)
        ws_ptr, ws_bytes = workspace if workspace is not None else self.workspace(m_b)
        y_code = 1 if (y is None or y.dtype != torch.float32) else 0
        if epilogue is None:
            B.boost_gemv_tiered(self.buf.page_ptr, self.buf.order, self.buf.n_pages, self.buf.n_host,
                                self.N, self.K, x2, m_b, y, y_code, residual, ws_ptr, ws_bytes, stream)
        else:
            B.boost_gemv_tiered_fused(self.buf.page_ptr, self.buf.order, self.buf.n_pages, self.buf.n_host,
                                      self.N, self.K, x2, m_b, y, y_code, residual, epilogue, ws_ptr, ws_bytes,
                                      stream)
        return y


class TieredKVCache:
    """K and V tensors of one layer, [Hkv][n_blocks][16][128] bf16, placed linearly by a KV pool."""

    def __init__(self, pool, n_kv_heads, n_blocks, head_dim=128, device="cuda"):
        self.pool = pool
        self.n_kv_heads, self.n_blocks, self.head_dim = n_kv_heads, n_blocks, head_dim
        self.tier = pool.page_tiers()
        n_bytes = n_kv_heads * n_blocks * 16 * head_dim * 2
        assert n_bytes == self.tier.size * PAGE
        self.k = TieredBuffer(n_bytes, device=device, tier=self.tier)
        self.v = TieredBuffer(n_bytes, device=device, tier=self.tier)
        self.n_pages = self.k.n_pages

    def load(self, k_logical, v_logical):
        """Fill from logical [Hkv, n_blocks, 16, D] bf16 device tensors."""
        for buf, t in ((self.k, k_logical), (self.v, v_logical)):
            assert t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16
            B.boost_kv_scatter(t, self.n_kv_heads, self.n_blocks, self.head_dim, buf.page_ptr, buf.n_pages)

    def dump(self):
        out = []
        for buf in (self.k, self.v):
            t = torch.empty(self.n_kv_heads, self.n_blocks, 16, self.head_dim, dtype=torch.bfloat16,
                            device=buf.device)
            B.boost_kv_gather(t, self.n_kv_heads, self.n_blocks, self.head_dim, buf.page_ptr, buf.n_pages)
            out.append(t)
        return out


def aligned_workspace(n_bytes, device):
    """Zero-filled device scratch of n_bytes whose address is 256-byte aligned -> (tensor, ptr)."""
    t = torch.zeros(n_bytes + 256, dtype=torch.uint8, device=device)
    return t, t.data_ptr() + (-t.data_ptr()) % 256
