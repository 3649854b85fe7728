"""Thin ctypes layer over libboost_b200.so: argument marshalling only.

Function names and argument order follow include/boost.h.  Device buffers are
passed as torch tensors (their data_ptr) or raw integer addresses; host arrays
are numpy arrays.  Nothing is computed here, and there is no fallback: if the
shared library is missing, `lib()` raises.
"""
import ctypes as C
import os

import numpy as np

PAGE_BYTES = 2 * 1024 * 1024
TIER_HBM, TIER_HOST = 0, 1
POLICY_MODULO, POLICY_CONTIGUOUS, POLICY_RANDOM = 0, 1, 2
OK, ERR_INVALID, ERR_NOMEM, ERR_ALIGN, ERR_CUDA, ERR_CAPACITY, ERR_UNSUPPORTED = 0, -1, -2, -3, -4, -5, -6

_ERR_NAMES = {-1: "BOOST_ERR_INVALID", -2: "BOOST_ERR_NOMEM", -3: "BOOST_ERR_ALIGN",
              -4: "BOOST_ERR_CUDA", -5: "BOOST_ERR_CAPACITY", -6: "BOOST_ERR_UNSUPPORTED"}

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libboost_b200.so")


class BoostError(RuntimeError):
    def __init__(self, code, where):
        extra = ""
        if code == ERR_CUDA:
            extra = f" (cudaError {lib().boost_last_cuda_error()})"
        super().__init__(f"{where}: {_ERR_NAMES.get(code, code)}{extra}")
        self.code = code


class WaveStats(C.Structure):
    _fields_ = [("n_waves", C.c_uint64), ("n_host_pages", C.c_uint64),
                ("n_zero_waves", C.c_uint64), ("n_over_waves", C.c_uint64),
                ("mean", C.c_double), ("var", C.c_double), ("min", C.c_double), ("max", C.c_double)]


class PoolInfo(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in
                ("n_blocks", "n_kv_heads", "host_modulus", "chunk_bytes", "n_pages", "n_host_pages",
                 "host_heads_lo", "first_hi_block", "free_lo", "free_hi", "live_blocks", "n_requests")] + \
               [("live_host_chunks", C.c_uint64), ("live_chunks", C.c_uint64)]


class WeightLayout(C.Structure):
    _fields_ = [("n_row_tiles", C.c_uint32), ("k_blocks", C.c_uint32), ("blocks_per_item", C.c_uint32),
                ("splits", C.c_uint32), ("bytes", C.c_uint64), ("n_pages", C.c_uint64)]


class Weight(C.Structure):
    _fields_ = [("page_ptr", C.c_void_p), ("order", C.c_void_p), ("n_pages", C.c_uint64),
                ("n_host_pages", C.c_uint64), ("N", C.c_uint32), ("K", C.c_uint32)]


class GemvEpilogue(C.Structure):
    _fields_ = [("mode", C.c_int), ("ssq_in", C.c_void_p), ("ssq_in_tiles", C.c_uint32),
                ("ssq_stride", C.c_uint32), ("rms_eps", C.c_float), ("ssq_out", C.c_void_p),
                ("q_out", C.c_void_p), ("k_page_ptr", C.c_void_p), ("v_page_ptr", C.c_void_p),
                ("n_pool_blocks", C.c_uint32), ("block_table", C.c_void_p), ("max_blocks", C.c_uint32),
                ("ctx_lens", C.c_void_p), ("n_q_heads", C.c_uint32), ("n_kv_heads", C.c_uint32),
                ("rope_table", C.c_void_p), ("k_page_ptr2", C.c_void_p), ("v_page_ptr2", C.c_void_p)]


class GemvCall(C.Structure):
    _fields_ = [("w", Weight), ("x", C.c_void_p), ("y", C.c_void_p), ("y_dtype", C.c_int),
                ("residual", C.c_void_p), ("has_epilogue", C.c_int), ("epilogue", GemvEpilogue)]


class LlamaLayer(C.Structure):
    _fields_ = [("wqkv", Weight), ("wo", Weight), ("wgu", Weight), ("wd", Weight),
                ("k_page_ptr", C.c_void_p), ("v_page_ptr", C.c_void_p)]


class LlamaModel(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in
                ("n_layers", "hidden", "ffn", "n_q_heads", "n_kv_heads", "head_dim", "vocab")] + \
               [("rms_eps", C.c_float), ("rope_base", C.c_float),
                ("embed", C.c_void_p), ("lm_head", Weight),
                ("layers", C.POINTER(LlamaLayer)), ("kv_tier", C.c_void_p),
                ("n_kv_pages", C.c_uint64), ("n_pool_blocks", C.c_uint32)]


class KVPrefetchLayer(C.Structure):
    _fields_ = [("k_host_src", C.c_void_p), ("v_host_src", C.c_void_p),
                ("k_page_ptr_staged", C.c_void_p), ("v_page_ptr_staged", C.c_void_p)]


class KVPrefetch(C.Structure):
    _fields_ = [("host_bytes", C.c_uint64), ("k_stage", C.c_void_p * 2), ("v_stage", C.c_void_p * 2),
                ("layers", C.POINTER(KVPrefetchLayer))]


class LlamaScratch(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("h", "q_rot", "attn", "act", "logits", "ssq_a", "ssq_b")] + \
               [("ssq_stride", C.c_uint32), ("rope_table", C.c_void_p),
                ("gemv_ws", C.c_void_p), ("gemv_ws_bytes", C.c_size_t),
                ("attn_ws", C.c_void_p), ("attn_ws_bytes", C.c_size_t)] + \
               [(n, C.c_void_p) for n in ("tokens_dev", "ctx_dev", "table_dev", "next_dev")]


EPI_PLAIN, EPI_SWIGLU, EPI_ROPE_APPEND = 0, 1, 2

_vp, _sz, _u32, _u64, _i32, _dbl, _int, _flt = (C.c_void_p, C.c_size_t, C.c_uint32, C.c_uint64,
                                                 C.c_int32, C.c_double, C.c_int, C.c_float)

# name -> (restype, argtypes); mirrors include/boost.h
SIGNATURES = {
    "boost_last_cuda_error": (_int, []),
    "boost_modulus_from_ratio": (_int, [_dbl, _vp]),
    "boost_modulus_from_bandwidths": (_int, [_dbl, _dbl, _vp]),
    "boost_place_pages": (_int, [_vp, _sz, _dbl, _u32, _vp, _sz, _vp]),
    "boost_place_pages_ex": (_int, [_vp, _sz, _dbl, _u32, _int, _u64, _u32, _vp, _sz, _vp, _vp]),
    "boost_wave_stats": (_int, [_vp, _sz, _sz, _u32, _dbl, _vp]),
    "boost_tier_order": (_int, [_vp, _sz, _vp, _vp]),
    "boost_host_device_pointer": (_int, [_vp, _vp]),
    "boost_peer_tier_open": (_int, [C.c_int]),
    "boost_peer_tier_alloc": (_int, [C.c_int, C.c_size_t, _vp]),
    "boost_peer_tier_free": (_int, [C.c_int, _vp]),
    "boost_page_table": (_int, [_vp, _sz, _vp, _sz, _vp, _sz, _vp]),
    "boost_scatter_pages": (_int, [_vp, _sz, _vp, _sz, _vp]),
    "boost_gather_pages": (_int, [_vp, _sz, _vp, _sz, _vp]),
    "boost_kv_pool_create": (_int, [_u32, _u32, _u32, _u32, _vp]),
    "boost_kv_pool_alloc": (_int, [_vp, _u64, _u32, _vp]),
    "boost_kv_pool_free": (_int, [_vp, _u64]),
    "boost_kv_pool_query": (_int, [_vp, _vp]),
    "boost_kv_pool_request_kind": (_int, [_vp, _u64, _vp]),
    "boost_kv_pool_page_tiers": (_int, [_vp, _vp, _sz, _vp]),
    "boost_kv_pool_destroy": (_int, [_vp]),
    "boost_stream_reduce_workspace_bytes": (_sz, [_sz]),
    "boost_stream_reduce_tiered": (_int, [_vp, _vp, _sz, _sz, _vp, _vp, _sz, _vp]),
    "boost_stream_reduce_static_max_pages": (_sz, []),
    "boost_stream_reduce_tiered_static": (_int, [_vp, _vp, _sz, _sz, _vp, _vp]),
    "boost_weight_layout": (_int, [_u32, _u32, _vp]),
    "boost_pack_weights": (_int, [_vp, _u32, _u32, _vp, _sz, _vp]),
    "boost_pack_weights_ex": (_int, [_vp, _u32, _u32, _vp, _sz, _int, _vp, _vp]),
    "boost_gemv_tiered_fused": (_int, [_vp, _vp, _sz, _sz, _u32, _u32, _vp, _u32, _vp, _int, _vp, _vp, _vp, _sz, _vp]),
    "boost_embed_gather_ssq": (_int, [_vp, _u32, _u32, _vp, _u32, _vp, _vp, _u32, _vp]),
    "boost_gemv_workspace_bytes": (_sz, [_u32, _u32, _u32]),
    "boost_gemv_tiered": (_int, [_vp, _vp, _sz, _sz, _u32, _u32, _vp, _u32, _vp, _int, _vp, _vp, _sz, _vp]),
    "boost_kv_scatter": (_int, [_vp, _u32, _u32, _u32, _vp, _sz, _vp]),
    "boost_kv_gather": (_int, [_vp, _u32, _u32, _u32, _vp, _sz, _vp]),
    "boost_paged_attn_workspace_bytes": (_sz, [_u32, _u32, _u32, _u32]),
    "boost_paged_attn_decode_tiered": (_int, [_vp, _vp, _vp, _vp, _sz, _u32, _vp, _u32, _vp,
                                              _u32, _u32, _u32, _u32, _flt, _vp, _sz, _vp, _vp]),
    "boost_embed_gather": (_int, [_vp, _u32, _u32, _vp, _u32, _vp, _vp]),
    "boost_rmsnorm": (_int, [_vp, _vp, _u32, _u32, _flt, _vp, _vp]),
    "boost_rope_kv_append": (_int, [_vp, _vp, _vp, _vp, _u32, _vp, _u32, _vp, _u32, _u32, _u32, _u32,
                                    _flt, _vp, _vp]),
    "boost_rope_table": (_int, [_vp, _u32, _u32, _flt, _vp, _vp]),
    "boost_swiglu": (_int, [_vp, _u32, _u32, _vp, _vp]),
    "boost_argmax": (_int, [_vp, _u32, _u32, _vp, _vp]),
    "boost_va_buffer_create": (_int, [_vp, C.c_size_t, _int, _vp]),
    "boost_va_buffer_base": (C.c_void_p, [_vp]),
    "boost_va_buffer_page_table": (_int, [_vp, _vp, C.c_size_t]),
    "boost_va_buffer_destroy": (_int, [_vp]),
    "boost_schedule_log_bytes": (C.c_size_t, [C.c_size_t]),
    "boost_schedule_stats": (_int, [_vp, C.c_size_t, _u32, _u32, C.c_uint64, C.c_double, _vp, _vp, _vp]),
    "boost_gemv_set_tc_min_batch": (_int, [_u32]),
    "boost_gemv_set_tier_schedule": (_int, [_u32]),
    "boost_gemv_set_end_combine": (_int, [_u32]),
    "boost_gemv_chain_workspace_bytes": (C.c_size_t, [_vp, _u32, _u32]),
    "boost_gemv_tiered_chain": (_int, [_vp, _u32, _u32, _vp, _sz, _vp]),
    "boost_llama_gemv_workspace_bytes": (C.c_size_t, [_vp, _u32]),
    "boost_llama_decode_step": (_int, [_vp, _vp, _vp, _vp, _u32, _vp, _u32, _vp, _vp, _vp]),
    "boost_prefetch_ctx_create": (_int, [_u32, _vp]),
    "boost_prefetch_ctx_destroy": (None, [_vp]),
    "boost_llama_decode_step_prefetch": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _u32, _vp, _u32, _vp, _vp, _vp]),
    "boost_llama_decode_step_profile": (_int, [_vp, _vp, _vp, _vp, _u32, _vp, _u32, _vp, _vp, _vp, _vp]),
    "boost_llama_decode_step_host": (_int, [_vp, _vp, _vp, _vp, _u32, _vp, _u32, _vp, _vp, _vp]),
}

_lib = None


def lib():
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2609_13592_b200.build` "
                               "(or __graft_entry__.build()); there is no CPU fallback")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            if not hasattr(handle, name):
                continue  # reported by the export test; calling it raises AttributeError
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _check(code, where):
    if code != OK:
        raise BoostError(code, where)


def _ptr(obj):
    """Address of a torch tensor, numpy array, ctypes object or plain int (None -> NULL)."""
    if obj is None:
        return None
    if isinstance(obj, int):
        return obj
    if hasattr(obj, "data_ptr"):
        return obj.data_ptr()
    if isinstance(obj, np.ndarray):
        return obj.ctypes.data
    return C.addressof(obj)


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


# ------------------------------------------------------------------ placement

def boost_modulus_from_ratio(host_ratio):
    out = C.c_uint32(0)
    _check(lib().boost_modulus_from_ratio(host_ratio, C.addressof(out)), "boost_modulus_from_ratio")
    return out.value


def boost_modulus_from_bandwidths(hbm_bw, link_bw):
    out = C.c_uint32(0)
    _check(lib().boost_modulus_from_bandwidths(hbm_bw, link_bw, C.addressof(out)),
           "boost_modulus_from_bandwidths")
    return out.value


def boost_place_pages(buffer, n_bytes, host_ratio, wave_size=0):
    """-> numpy uint8 tier table (modulo placement)."""
    cap = (n_bytes + PAGE_BYTES - 1) // PAGE_BYTES
    tier = np.zeros(max(cap, 1), dtype=np.uint8)
    n = C.c_size_t(0)
    _check(lib().boost_place_pages(_ptr(buffer), n_bytes, host_ratio, wave_size, tier.ctypes.data,
                                   cap, C.addressof(n)), "boost_place_pages")
    return tier[:n.value]


def boost_place_pages_ex(buffer, n_bytes, host_ratio, wave_size=0, policy=POLICY_MODULO, seed=0,
                         superpage_pages=1):
    """-> (tier table, flags)."""
    cap = (n_bytes + PAGE_BYTES - 1) // PAGE_BYTES
    tier = np.zeros(max(cap, 1), dtype=np.uint8)
    n = C.c_size_t(0)
    flags = C.c_uint32(0)
    _check(lib().boost_place_pages_ex(_ptr(buffer), n_bytes, host_ratio, wave_size, policy, seed,
                                      superpage_pages, tier.ctypes.data, cap, C.addressof(n),
                                      C.addressof(flags)), "boost_place_pages_ex")
    return tier[:n.value], flags.value


def boost_wave_stats(tier, tile_bytes, ctas_per_wave, host_ratio):
    tier = np.ascontiguousarray(tier, dtype=np.uint8)
    st = WaveStats()
    _check(lib().boost_wave_stats(tier.ctypes.data, tier.size, tile_bytes, ctas_per_wave, host_ratio,
                                  C.addressof(st)), "boost_wave_stats")
    return {k: getattr(st, k) for k, _ in WaveStats._fields_}


def boost_tier_order(tier):
    """-> (order uint32 array, n_host)."""
    tier = np.ascontiguousarray(tier, dtype=np.uint8)
    order = np.zeros(max(tier.size, 1), dtype=np.uint32)
    n_host = C.c_size_t(0)
    _check(lib().boost_tier_order(tier.ctypes.data, tier.size, order.ctypes.data, C.addressof(n_host)),
           "boost_tier_order")
    return order[:tier.size], n_host.value


# ------------------------------------------------------------ materialisation

def boost_host_device_pointer(pinned):
    out = C.c_void_p(0)
    _check(lib().boost_host_device_pointer(_ptr(pinned), C.addressof(out)), "boost_host_device_pointer")
    return out.value or 0


def boost_peer_tier_open(peer_device):
    _check(lib().boost_peer_tier_open(int(peer_device)), "boost_peer_tier_open")


def boost_peer_tier_alloc(peer_device, n_bytes):
    """-> address of a slab of n_bytes in peer_device's memory."""
    out = C.c_void_p(0)
    _check(lib().boost_peer_tier_alloc(int(peer_device), int(n_bytes), C.addressof(out)), "boost_peer_tier_alloc")
    return out.value or 0


def boost_peer_tier_free(peer_device, slab):
    _check(lib().boost_peer_tier_free(int(peer_device), slab or None), "boost_peer_tier_free")


def boost_page_table(tier, hbm_slab, hbm_slab_bytes, host_slab, host_slab_bytes):
    """-> numpy uint64 array of page addresses."""
    tier = np.ascontiguousarray(tier, dtype=np.uint8)
    table = np.zeros(max(tier.size, 1), dtype=np.uint64)
    _check(lib().boost_page_table(tier.ctypes.data, tier.size, _ptr(hbm_slab), hbm_slab_bytes,
                                  _ptr(host_slab), host_slab_bytes, table.ctypes.data), "boost_page_table")
    return table[:tier.size]


def boost_scatter_pages(src, n_bytes, page_ptr, n_pages, stream=None):
    _check(lib().boost_scatter_pages(_ptr(src), n_bytes, _ptr(page_ptr), n_pages, _stream(stream)),
           "boost_scatter_pages")


def boost_gather_pages(dst, n_bytes, page_ptr, n_pages, stream=None):
    _check(lib().boost_gather_pages(_ptr(dst), n_bytes, _ptr(page_ptr), n_pages, _stream(stream)),
           "boost_gather_pages")


# -------------------------------------------------------------------- KV pool

class KVPool:
    """Owner of a boost_kv_pool_t handle."""

    def __init__(self, n_blocks, n_kv_heads, host_modulus, chunk_bytes=4096):
        self._h = C.c_void_p(0)
        _check(lib().boost_kv_pool_create(n_blocks, n_kv_heads, host_modulus, chunk_bytes,
                                          C.addressof(self._h)), "boost_kv_pool_create")

    def alloc(self, request_id, n):
        out = np.zeros(max(n, 1), dtype=np.int32)
        _check(lib().boost_kv_pool_alloc(self._h, request_id, n, out.ctypes.data), "boost_kv_pool_alloc")
        return out[:n]

    def free(self, request_id):
        _check(lib().boost_kv_pool_free(self._h, request_id), "boost_kv_pool_free")

    def query(self):
        info = PoolInfo()
        _check(lib().boost_kv_pool_query(self._h, C.addressof(info)), "boost_kv_pool_query")
        return {k: getattr(info, k) for k, _ in PoolInfo._fields_}

    def request_kind(self, request_id):
        out = C.c_int(0)
        _check(lib().boost_kv_pool_request_kind(self._h, request_id, C.addressof(out)),
               "boost_kv_pool_request_kind")
        return out.value

    def page_tiers(self):
        n = self.query()["n_pages"]
        tier = np.zeros(n, dtype=np.uint8)
        got = C.c_size_t(0)
        _check(lib().boost_kv_pool_page_tiers(self._h, tier.ctypes.data, n, C.addressof(got)),
               "boost_kv_pool_page_tiers")
        return tier

    def close(self):
        if self._h:
            lib().boost_kv_pool_destroy(self._h)
            self._h = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# -------------------------------------------------------------------- kernels

def boost_stream_reduce_workspace_bytes(n_pages):
    return lib().boost_stream_reduce_workspace_bytes(n_pages)


def boost_stream_reduce_tiered(page_ptr, order, n_pages, n_host_pages, per_page_sum, workspace,
                               workspace_bytes, stream=None):
    _check(lib().boost_stream_reduce_tiered(_ptr(page_ptr), _ptr(order), n_pages, n_host_pages,
                                            _ptr(per_page_sum), _ptr(workspace), workspace_bytes,
                                            _stream(stream)), "boost_stream_reduce_tiered")


def boost_stream_reduce_static_max_pages():
    return lib().boost_stream_reduce_static_max_pages()


def boost_stream_reduce_tiered_static(page_ptr, order, n_pages, n_host_pages, per_page_sum, stream=None):
    """Stream reduce with the library's built-in scratch: for callers that cannot allocate a
    workspace (see include/boost.h).  At most boost_stream_reduce_static_max_pages() pages."""
    _check(lib().boost_stream_reduce_tiered_static(_ptr(page_ptr), _ptr(order), n_pages, n_host_pages,
                                                   _ptr(per_page_sum), _stream(stream)),
           "boost_stream_reduce_tiered_static")


def boost_weight_layout(n, k):
    lay = WeightLayout()
    _check(lib().boost_weight_layout(n, k, C.addressof(lay)), "boost_weight_layout")
    return {f: getattr(lay, f) for f, _ in WeightLayout._fields_}


def boost_pack_weights(w_row_major, n, k, w_page_ptr, n_pages, stream=None):
    _check(lib().boost_pack_weights(_ptr(w_row_major), n, k, _ptr(w_page_ptr), n_pages, _stream(stream)),
           "boost_pack_weights")


def boost_pack_weights_ex(w_row_major, n, k, w_page_ptr, n_pages, row_mode=0, col_scale=None, stream=None):
    _check(lib().boost_pack_weights_ex(_ptr(w_row_major), n, k, _ptr(w_page_ptr), n_pages, row_mode,
                                       _ptr(col_scale), _stream(stream)), "boost_pack_weights_ex")


def boost_gemv_tiered_fused(w_page_ptr, w_order, n_pages, n_host_pages, n, k, x, m_b, y, y_dtype, residual,
                            epilogue, workspace, workspace_bytes, stream=None):
    """epilogue: a GemvEpilogue structure or None (plain)."""
    _check(lib().boost_gemv_tiered_fused(_ptr(w_page_ptr), _ptr(w_order), n_pages, n_host_pages, n, k,
                                         _ptr(x), m_b, _ptr(y), y_dtype, _ptr(residual),
                                         None if epilogue is None else C.addressof(epilogue),
                                         _ptr(workspace), workspace_bytes, _stream(stream)),
           "boost_gemv_tiered_fused")


def gemv_calls(calls):
    """calls: list of dict(w=Weight, x, y, y_dtype (0 fp32 / 1 bf16), residual=None, epilogue=None)
    -> ctypes array of GemvCall."""
    arr = (GemvCall * len(calls))()
    for c, d in zip(arr, calls):
        c.w, c.x, c.y, c.y_dtype = d["w"], _ptr(d["x"]), _ptr(d.get("y")), d["y_dtype"]
        c.residual = _ptr(d.get("residual"))
        epi = d.get("epilogue")
        c.has_epilogue = 0 if epi is None else 1
        if epi is not None:
            c.epilogue = epi
    return arr


def boost_gemv_set_tc_min_batch(m_b):
    _check(lib().boost_gemv_set_tc_min_batch(m_b), "boost_gemv_set_tc_min_batch")


def boost_gemv_set_tier_schedule(two_queues):
    _check(lib().boost_gemv_set_tier_schedule(1 if two_queues else 0), "boost_gemv_set_tier_schedule")


class VABuffer:
    """Owner of a boost_va_buffer_t: one virtual range whose pages live on the tiers of `tier`."""

    def __init__(self, tier, host_numa_node=0):
        tier = np.ascontiguousarray(tier, dtype=np.uint8)
        self.tier, self.n_pages = tier, int(tier.size)
        self._h = C.c_void_p(0)
        _check(lib().boost_va_buffer_create(tier.ctypes.data, tier.size, host_numa_node, C.addressof(self._h)),
               "boost_va_buffer_create")
        self.base = int(lib().boost_va_buffer_base(self._h))

    def page_table(self):
        out = np.zeros(self.n_pages, dtype=np.uint64)
        _check(lib().boost_va_buffer_page_table(self._h, out.ctypes.data, out.size), "boost_va_buffer_page_table")
        return out

    def close(self):
        if self._h:
            lib().boost_va_buffer_destroy(self._h)
            self._h = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


SCHED_KIND_STREAM, SCHED_KIND_GEMV, SCHED_KIND_ATTN = 1, 2, 3
WS_WAIT_LIMIT_WORD, WS_SKIP_ARRIVALS_WORD, WS_LOG_WORD = 4, 5, 6
SCHED_RECORD_DTYPE = np.dtype([("kind_phase", "<u4"), ("cta_warp", "<u4"), ("bytes", "<u4"), ("host_bytes", "<u4"),
                               ("t_request", "<u8"), ("t_consumed", "<u8")])


def boost_schedule_log_bytes(capacity):
    return int(lib().boost_schedule_log_bytes(capacity))


def schedule_records(log_host):
    """Records of a schedule log copied to the host (numpy uint8 array of the whole buffer) as a
    structured array, and the number of records the kernels tried to write."""
    head = log_host[:32].view("<u8")
    claimed, capacity = int(head[0]), int(head[1])
    n = min(claimed, capacity)
    return log_host[32:32 + n * SCHED_RECORD_DTYPE.itemsize].view(SCHED_RECORD_DTYPE), claimed


def boost_schedule_stats(log_host, kind, items_per_wave, window_ns, host_ratio):
    """log_host: numpy uint8 array holding the whole log buffer -> (waves, windows, n_records)."""
    log_host = np.ascontiguousarray(log_host, dtype=np.uint8)
    waves, windows, n = WaveStats(), WaveStats(), C.c_uint64(0)
    _check(lib().boost_schedule_stats(log_host.ctypes.data, log_host.size, kind, items_per_wave, window_ns, host_ratio,
                                      C.addressof(waves), C.addressof(windows), C.addressof(n)), "boost_schedule_stats")
    as_dict = lambda st: {f: getattr(st, f) for f, _ in WaveStats._fields_}
    return as_dict(waves), as_dict(windows), int(n.value)


def boost_gemv_set_end_combine(on):
    _check(lib().boost_gemv_set_end_combine(1 if on else 0), "boost_gemv_set_end_combine")


def boost_gemv_chain_workspace_bytes(calls, m_b):
    return int(lib().boost_gemv_chain_workspace_bytes(C.addressof(calls), len(calls), m_b))


def boost_gemv_tiered_chain(calls, m_b, workspace, workspace_bytes, stream=None):
    """calls: the array made by gemv_calls; one launch for the whole chain."""
    _check(lib().boost_gemv_tiered_chain(C.addressof(calls), len(calls), m_b, _ptr(workspace), workspace_bytes,
                                         _stream(stream)), "boost_gemv_tiered_chain")


def boost_embed_gather_ssq(table, vocab, hidden, tokens, b, out, ssq_out, ssq_stride, stream=None):
    _check(lib().boost_embed_gather_ssq(_ptr(table), vocab, hidden, _ptr(tokens), b, _ptr(out),
                                        _ptr(ssq_out), ssq_stride, _stream(stream)), "boost_embed_gather_ssq")


def boost_gemv_workspace_bytes(n, k, m_b):
    return lib().boost_gemv_workspace_bytes(n, k, m_b)


def boost_gemv_tiered(w_page_ptr, w_order, n_pages, n_host_pages, n, k, x, m_b, y, y_dtype, residual,
                      workspace, workspace_bytes, stream=None):
    _check(lib().boost_gemv_tiered(_ptr(w_page_ptr), _ptr(w_order), n_pages, n_host_pages, n, k, _ptr(x),
                                   m_b, _ptr(y), y_dtype, _ptr(residual), _ptr(workspace),
                                   workspace_bytes, _stream(stream)), "boost_gemv_tiered")


def boost_kv_scatter(src, n_kv_heads, n_pool_blocks, d, page_ptr, n_pages, stream=None):
    _check(lib().boost_kv_scatter(_ptr(src), n_kv_heads, n_pool_blocks, d, _ptr(page_ptr), n_pages,
                                  _stream(stream)), "boost_kv_scatter")


def boost_kv_gather(dst, n_kv_heads, n_pool_blocks, d, page_ptr, n_pages, stream=None):
    _check(lib().boost_kv_gather(_ptr(dst), n_kv_heads, n_pool_blocks, d, _ptr(page_ptr), n_pages,
                                 _stream(stream)), "boost_kv_gather")


def boost_paged_attn_workspace_bytes(b, hq, d, max_blocks):
    return lib().boost_paged_attn_workspace_bytes(b, hq, d, max_blocks)


def boost_paged_attn_decode_tiered(q, k_page_ptr, v_page_ptr, kv_tier, n_kv_pages, n_pool_blocks,
                                   block_table, max_blocks, ctx_lens, b, hq, hkv, d, scale, workspace,
                                   workspace_bytes, out, stream=None):
    tier = None if kv_tier is None else np.ascontiguousarray(kv_tier, dtype=np.uint8)
    _check(lib().boost_paged_attn_decode_tiered(
        _ptr(q), _ptr(k_page_ptr), _ptr(v_page_ptr), _ptr(tier), n_kv_pages, n_pool_blocks,
        _ptr(block_table), max_blocks, _ptr(ctx_lens), b, hq, hkv, d, scale, _ptr(workspace),
        workspace_bytes, _ptr(out), _stream(stream)), "boost_paged_attn_decode_tiered")


# ----------------------------------------------------------------------- glue

def boost_embed_gather(table, vocab, hidden, tokens, b, out, stream=None):
    _check(lib().boost_embed_gather(_ptr(table), vocab, hidden, _ptr(tokens), b, _ptr(out), _stream(stream)),
           "boost_embed_gather")


def boost_rmsnorm(x, weight, b, hidden, eps, out, stream=None):
    _check(lib().boost_rmsnorm(_ptr(x), _ptr(weight), b, hidden, eps, _ptr(out), _stream(stream)),
           "boost_rmsnorm")


def boost_rope_kv_append(qkv, q_out, k_page_ptr, v_page_ptr, n_pool_blocks, block_table, max_blocks,
                         ctx_lens, b, hq, hkv, d, rope_base, status_word, stream=None):
    _check(lib().boost_rope_kv_append(_ptr(qkv), _ptr(q_out), _ptr(k_page_ptr), _ptr(v_page_ptr),
                                      n_pool_blocks, _ptr(block_table), max_blocks, _ptr(ctx_lens), b, hq,
                                      hkv, d, rope_base, _ptr(status_word), _stream(stream)),
           "boost_rope_kv_append")


def boost_rope_table(ctx_lens, b, d, rope_base, table, stream=None):
    _check(lib().boost_rope_table(_ptr(ctx_lens), b, d, rope_base, _ptr(table), _stream(stream)), "boost_rope_table")


def boost_swiglu(gate_up, b, f, out, stream=None):
    _check(lib().boost_swiglu(_ptr(gate_up), b, f, _ptr(out), _stream(stream)), "boost_swiglu")


def boost_argmax(logits, b, v, out, stream=None):
    _check(lib().boost_argmax(_ptr(logits), b, v, _ptr(out), _stream(stream)), "boost_argmax")


def boost_llama_gemv_workspace_bytes(model, b):
    return int(lib().boost_llama_gemv_workspace_bytes(C.addressof(model), b))


def boost_llama_decode_step(model, scratch, tokens, block_table, max_blocks, ctx_lens, b, next_tokens,
                            stream=None):
    """model / scratch: LlamaModel / LlamaScratch structures; returns the number of launches."""
    n = C.c_uint32(0)
    _check(lib().boost_llama_decode_step(C.addressof(model), C.addressof(scratch), _ptr(tokens),
                                         _ptr(block_table), max_blocks, _ptr(ctx_lens), b,
                                         _ptr(next_tokens), C.addressof(n), _stream(stream)),
           "boost_llama_decode_step")
    return n.value


def boost_prefetch_ctx_create(n_layers):
    h = C.c_void_p()
    _check(lib().boost_prefetch_ctx_create(n_layers, C.addressof(h)), "boost_prefetch_ctx_create")
    return h


def boost_prefetch_ctx_destroy(handle):
    lib().boost_prefetch_ctx_destroy(handle)


def boost_llama_decode_step_prefetch(model, scratch, prefetch, ctx, tokens, block_table, max_blocks, ctx_lens, b,
                                     next_tokens, stream=None):
    """Prefetch-to-HBM variant of boost_llama_decode_step; prefetch: a KVPrefetch structure."""
    n = C.c_uint32(0)
    _check(lib().boost_llama_decode_step_prefetch(C.addressof(model), C.addressof(scratch), C.addressof(prefetch),
                                                  ctx, _ptr(tokens), _ptr(block_table), max_blocks,
                                                  _ptr(ctx_lens), b, _ptr(next_tokens), C.addressof(n),
                                                  _stream(stream)), "boost_llama_decode_step_prefetch")
    return n.value


def boost_llama_decode_step_host(model, scratch, tokens, block_table, max_blocks, ctx_lens, b, next_tokens,
                                 stream=None):
    """Host-buffer variant: tokens / block_table / ctx_lens / next_tokens are host arrays."""
    n = C.c_uint32(0)
    _check(lib().boost_llama_decode_step_host(C.addressof(model), C.addressof(scratch), _ptr(tokens),
                                              _ptr(block_table), max_blocks, _ptr(ctx_lens), b,
                                              _ptr(next_tokens), C.addressof(n), _stream(stream)),
           "boost_llama_decode_step_host")
    return n.value


def boost_llama_decode_step_profile(model, scratch, tokens, block_table, max_blocks, ctx_lens, b, next_tokens,
                                    stream=None):
    """-> (ms per kind [gemv, attn, glue], launches per kind)."""
    ms = (C.c_float * 3)()
    n = (C.c_uint32 * 3)()
    _check(lib().boost_llama_decode_step_profile(C.addressof(model), C.addressof(scratch), _ptr(tokens),
                                                 _ptr(block_table), max_blocks, _ptr(ctx_lens), b,
                                                 _ptr(next_tokens), C.addressof(ms), C.addressof(n),
                                                 _stream(stream)), "boost_llama_decode_step_profile")
    return list(ms), list(n)
