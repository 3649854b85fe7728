"""Assembly of a Llama-shaped decoder over tiered weights and a pooled, tiered KV cache.

Plumbing only: allocates device / pinned memory through PyTorch, asks the library for
placements, packs weights into pages and fills the C structures that
boost_llama_decode_step consumes.  Every step of the decode path runs in the library.
"""
import ctypes as C

import numpy as np
import torch

from . import binding as B
from .tiers import TieredBuffer, TieredWeight, aligned_workspace

RMS_EPS = 1e-5
ROPE_BASE = 500000.0


def _weight_struct(tw):
    return B.Weight(tw.buf.page_ptr.data_ptr(), tw.buf.order.data_ptr(), tw.buf.n_pages, tw.buf.n_host,
                    tw.N, tw.K)


class LlamaDecoder:
    """cfg: dict(n_layers, hidden, ffn, n_q_heads, n_kv_heads, head_dim, vocab).

    get_weight(name, layer) returns a bf16 device tensor: 'embed' [V, hidden], 'norm_f' [hidden],
    'lm_head' [V, hidden] (layer None) and per layer 'norm1', 'wqkv', 'wo', 'norm2', 'wgu', 'wd'.
    Weight matrices are placed per tensor with `weight_host_ratio` (modulo placement restarts
    for every tensor); the KV cache of every layer is placed linearly by a pool with
    `kv_host_modulus`.  weight_tier, if given, is a callable (name, layer, n_pages) -> uint8 tier
    array (or None for the placement function): an explicit page-to-tier table per matrix, for
    models whose matrices are shorter than one placement period.
    """

    def __init__(self, cfg, get_weight, weight_host_ratio=0.0, n_pool_blocks=512, kv_host_modulus=0,
                 max_batch=32, max_blocks=8, device="cuda", weight_policy=B.POLICY_MODULO, kv_prefetch=False,
                 weight_tier=None):
        self.cfg = dict(cfg)
        self.device = torch.device(device)
        self.max_batch, self.max_blocks = max_batch, max_blocks
        hq, hkv, d = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
        hid, ffn, vocab, nl = cfg["hidden"], cfg["ffn"], cfg["vocab"], cfg["n_layers"]
        self.pool = B.KVPool(n_pool_blocks, hkv, kv_host_modulus, 16 * d * 2)
        self.kv_tier = self.pool.page_tiers()
        self.n_pool_blocks = n_pool_blocks
        kv_bytes = hkv * n_pool_blocks * 16 * d * 2

        def tiered(name, layer, norm=None, row_mode=0):
            # norm: name of the RMSNorm weight folded into this matrix at load time
            w = get_weight(name, layer).contiguous()
            g = get_weight(norm, layer).contiguous() if norm else None
            tier = None
            if weight_tier is not None:
                tier = weight_tier(name, layer, B.boost_weight_layout(int(w.shape[0]), int(w.shape[1]))["n_pages"])
            tw = TieredWeight(w, weight_host_ratio, weight_policy, device=self.device, row_mode=row_mode,
                              col_scale=g, tier=tier)
            del w, g
            return tw

        self.embed = get_weight("embed", None).contiguous()
        self.lm_head = tiered("lm_head", None, norm="norm_f")
        self.layers = []
        self._layer_structs = (B.LlamaLayer * nl)()
        for li in range(nl):
            ly = {"wqkv": tiered("wqkv", li, norm="norm1"), "wo": tiered("wo", li),
                  "wgu": tiered("wgu", li, norm="norm2", row_mode=1), "wd": tiered("wd", li)}
            ly["k"] = TieredBuffer(kv_bytes, device=self.device, tier=self.kv_tier)
            ly["v"] = TieredBuffer(kv_bytes, device=self.device, tier=self.kv_tier)
            self.layers.append(ly)
            st = self._layer_structs[li]
            st.wqkv, st.wo = _weight_struct(ly["wqkv"]), _weight_struct(ly["wo"])
            st.wgu, st.wd = _weight_struct(ly["wgu"]), _weight_struct(ly["wd"])
            st.k_page_ptr, st.v_page_ptr = ly["k"].page_ptr.data_ptr(), ly["v"].page_ptr.data_ptr()
        self._kv_tier_c = np.ascontiguousarray(self.kv_tier, dtype=np.uint8)
        m = B.LlamaModel()
        m.n_layers, m.hidden, m.ffn, m.n_q_heads, m.n_kv_heads = nl, hid, ffn, hq, hkv
        m.head_dim, m.vocab, m.rms_eps, m.rope_base = d, vocab, RMS_EPS, ROPE_BASE
        m.embed, m.lm_head = self.embed.data_ptr(), _weight_struct(self.lm_head)
        m.layers = C.cast(self._layer_structs, C.POINTER(B.LlamaLayer))
        m.kv_tier = self._kv_tier_c.ctypes.data
        m.n_kv_pages, m.n_pool_blocks = int(self.kv_tier.size), n_pool_blocks
        self.model = m

        bm = max_batch
        bf = dict(dtype=torch.bfloat16, device=self.device)
        self.buf = {
            "h": torch.zeros(bm, hid, **bf), "q_rot": torch.zeros(bm, hq * d, **bf),
            "attn": torch.zeros(bm, hq * d, **bf), "act": torch.zeros(bm, ffn, **bf),
            "logits": torch.zeros(bm, vocab, dtype=torch.float32, device=self.device),
            "ssq_a": torch.zeros(hid // 128, bm, dtype=torch.float32, device=self.device),
            "ssq_b": torch.zeros(hid // 128, bm, dtype=torch.float32, device=self.device),
            "rope_table": torch.zeros(bm, d // 2, 2, dtype=torch.float32, device=self.device),
            "tokens_dev": torch.zeros(bm, dtype=torch.int32, device=self.device),
            "ctx_dev": torch.zeros(bm, dtype=torch.int32, device=self.device),
            "table_dev": torch.zeros(bm, max_blocks, dtype=torch.int32, device=self.device),
            "next_dev": torch.zeros(bm, dtype=torch.int32, device=self.device),
        }
        gemv_bytes = B.boost_llama_gemv_workspace_bytes(m, bm)
        assert gemv_bytes > 0
        attn_bytes = B.boost_paged_attn_workspace_bytes(bm, hq, d, max_blocks)
        self._gemv_ws_t, gemv_ws = aligned_workspace(gemv_bytes, self.device)
        self._attn_ws_t, attn_ws = aligned_workspace(attn_bytes, self.device)
        s = B.LlamaScratch()
        for k in ("h", "q_rot", "attn", "act", "logits", "ssq_a", "ssq_b", "rope_table",
                  "tokens_dev", "ctx_dev", "table_dev", "next_dev"):
            setattr(s, k, self.buf[k].data_ptr())
        s.ssq_stride = bm
        s.gemv_ws, s.gemv_ws_bytes, s.attn_ws, s.attn_ws_bytes = gemv_ws, gemv_bytes, attn_ws, attn_bytes
        self.scratch = s
        self._gemv_ws_ptr, self._attn_ws_ptr = gemv_ws, attn_ws
        self._prefetch = None
        if kv_prefetch:
            self._make_prefetch()
        torch.cuda.synchronize(self.device)

    def _make_prefetch(self):
        """Structures of the prefetch-to-HBM variant: two staging buffers per tensor kind, and
        per layer a page table whose host pages point into staging buffer (layer % 2)."""
        n_host = self.layers[0]["k"].n_host
        host_bytes = n_host * B.PAGE_BYTES
        self._stage_t = [torch.empty(host_bytes + B.PAGE_BYTES, dtype=torch.uint8, device=self.device) for _ in range(4)]
        stage = [(t.data_ptr() + B.PAGE_BYTES - 1) // B.PAGE_BYTES * B.PAGE_BYTES for t in self._stage_t]
        self._pf_layers = (B.KVPrefetchLayer * len(self.layers))()
        self._pf_tables = []
        for li, ly in enumerate(self.layers):
            kt = ly["k"].staged_page_ptr(stage[li % 2])
            vt = ly["v"].staged_page_ptr(stage[2 + li % 2])
            self._pf_tables += [kt, vt]
            e = self._pf_layers[li]
            e.k_host_src, e.v_host_src = ly["k"].host_base_cpu or None, ly["v"].host_base_cpu or None
            e.k_page_ptr_staged, e.v_page_ptr_staged = kt.data_ptr(), vt.data_ptr()
        pf = B.KVPrefetch()
        pf.host_bytes = host_bytes
        pf.k_stage[0], pf.k_stage[1], pf.v_stage[0], pf.v_stage[1] = stage
        pf.layers = C.cast(self._pf_layers, C.POINTER(B.KVPrefetchLayer))
        self._prefetch = pf
        self._prefetch_ctx = B.boost_prefetch_ctx_create(len(self.layers))

    def step_prefetch(self, tokens, block_table, ctx_lens, next_tokens, stream=None):
        """Device-buffer step of the prefetch-to-HBM variant (the decoder was built with kv_prefetch=True)."""
        assert self._prefetch is not None
        return B.boost_llama_decode_step_prefetch(self.model, self.scratch, self._prefetch, self._prefetch_ctx,
                                                  tokens, block_table, block_table.shape[1], ctx_lens,
                                                  tokens.shape[0], next_tokens, stream)

    # bytes the kernels must read per step (algorithmic): all weight pages plus live KV
    def weight_bytes(self):
        total = self.lm_head.layout["bytes"]
        for ly in self.layers:
            total += sum(ly[k].layout["bytes"] for k in ("wqkv", "wo", "wgu", "wd"))
        return total

    def kv_bytes_per_token(self):
        c = self.cfg
        return c["n_layers"] * 2 * c["n_kv_heads"] * c["head_dim"] * 2

    def host_weight_pages(self):
        n = self.lm_head.buf.n_host
        for ly in self.layers:
            n += sum(ly[k].buf.n_host for k in ("wqkv", "wo", "wgu", "wd"))
        return n

    def step(self, tokens, block_table, ctx_lens, next_tokens, stream=None):
        """Device-buffer step; returns the number of kernels launched."""
        b = tokens.shape[0]
        return B.boost_llama_decode_step(self.model, self.scratch, tokens, block_table, block_table.shape[1],
                                         ctx_lens, b, next_tokens, stream)

    def step_host(self, tokens, block_table, ctx_lens, next_tokens, stream=None):
        """Host-buffer step (numpy int32 arrays, ideally views of pinned tensors)."""
        b = tokens.shape[0]
        assert block_table.shape[1] <= self.max_blocks
        return B.boost_llama_decode_step_host(self.model, self.scratch, tokens, block_table,
                                              block_table.shape[1], ctx_lens, b, next_tokens, stream)

    def status_words(self):
        out = []
        for t, ptr in ((self._gemv_ws_t, self._gemv_ws_ptr), (self._attn_ws_t, self._attn_ws_ptr)):
            off = ptr - t.data_ptr()
            out.append(int(t[off:off + 4].cpu().numpy().view(np.uint32)[0]))
        return out
