// One decode step of a Llama-shaped model as a fixed sequence of launches on one stream.
// Host code only: every step of the path runs in the kernels of the other files.
#include <cuda_runtime.h>

#include <new>

#include "host_common.h"

namespace {

enum Kind { kKindGemv = 0, kKindAttn = 1, kKindGlue = 2, kNumKinds = 3 };

// Issues the launches of a step in order; optionally brackets each with a pair of events so
// that the time of every kind of kernel can be read back afterwards.
struct Launcher {
  void* stream;
  bool timed = false;
  uint32_t count = 0;   // launches issued through run()
  uint32_t extra = 0;   // kernels those launches added on their own
  int rc = BOOST_OK;
  cudaEvent_t ev[2 * 512];
  int kind_of[512];
  bool ok() const { return rc == BOOST_OK; }
  template <typename F>
  void run(int kind, F&& f) {
    if (rc != BOOST_OK) return;
    if (timed && count < 512) {
      rc = boosth::check(cudaEventRecord(ev[2 * count], (cudaStream_t)stream));
      if (rc != BOOST_OK) return;
    }
    rc = f();
    if (rc != BOOST_OK) return;
    if (timed && count < 512) {
      rc = boosth::check(cudaEventRecord(ev[2 * count + 1], (cudaStream_t)stream));
      kind_of[count] = kind;
    }
    ++count;
  }
};

// The tail of the GEMV workspace holds one set of queue words per launch of a step, so that a
// weight product can take work and stream weights while the kernel before it is still running.
constexpr size_t kQueueSlots = 512;
constexpr size_t kQueueSlotBytes = 64;
constexpr size_t kQueueRegionBytes = kQueueSlots * kQueueSlotBytes;

// All products of a step share one workspace: the counter area is sized for the product with
// the most row tiles, so that no product's partial sums lie where another keeps its counters.
uint32_t max_row_tiles(const boost_llama_model_t* m) {
  uint32_t n = m->lm_head.N;
  for (uint32_t li = 0; li < m->n_layers; ++li) {
    const boost_llama_layer_t& ly = m->layers[li];
    const uint32_t ns[4] = {ly.wqkv.N, ly.wo.N, ly.wgu.N, ly.wd.N};
    for (uint32_t v : ns) n = v > n ? v : n;
  }
  return (n + 127) / 128;
}

// Sync words of a launch: `n_calls + 1` slots from the region at the tail of the workspace.
struct SyncSlots {
  uint32_t next = 0;
  uint32_t* take(const boost_llama_scratch_t* s, size_t usable, uint32_t n) {
    if (next + n > kQueueSlots) next = 0;
    uint8_t* slots = static_cast<uint8_t*>(s->gemv_ws) + usable;
    uint32_t* r = reinterpret_cast<uint32_t*>(slots + (size_t)next * kQueueSlotBytes);
    next += n;
    return r;
  }
};

boost_gemv_call_t call_of(const boost_weight_t& w, const void* x, void* y, int y_dtype, const void* residual,
                          const boost_gemv_epilogue_t& epi) {
  boost_gemv_call_t c = {};
  c.w = w; c.x = x; c.y = y; c.y_dtype = y_dtype; c.residual = residual;
  c.has_epilogue = 1;
  c.epilogue = epi;
  return c;
}

}  // namespace

// Copy stream and events of the prefetch-to-HBM variant.
struct boost_prefetch_ctx {
  cudaStream_t copy_stream = nullptr;
  uint32_t n_layers = 0;
  cudaEvent_t* copy_done = nullptr;   // [n_layers]: layer's host pages are in its staging buffer
  cudaEvent_t* attn_done = nullptr;   // [n_layers]: the attention kernel of the layer has been issued and finished
  cudaEvent_t step_begin = nullptr;   // everything issued to the compute stream before this step
};

namespace {

int run_step(Launcher& L, const boost_llama_model_t* m, const boost_llama_scratch_t* s, const int32_t* tokens,
             const int32_t* block_table, uint32_t max_blocks, const int32_t* ctx_lens, uint32_t B,
             int32_t* next_tokens, const boost_kv_prefetch_t* pf = nullptr, boost_prefetch_ctx* pc = nullptr) {
  if (!m || !s || !tokens || !block_table || !ctx_lens || !next_tokens) return BOOST_ERR_INVALID;
  if (B == 0 || B > 256 || !m->layers || m->n_layers == 0) return BOOST_ERR_INVALID;
  if (!s->h || !s->q_rot || !s->attn || !s->act || !s->logits || !s->ssq_a || !s->ssq_b || !s->rope_table || !s->gemv_ws ||
      !s->attn_ws || s->ssq_stride < B)
    return BOOST_ERR_INVALID;
  if (m->hidden % 128 != 0 || m->head_dim != 128) return BOOST_ERR_UNSUPPORTED;
  if (s->gemv_ws_bytes <= kQueueRegionBytes + 256) return BOOST_ERR_CAPACITY;
  const size_t usable = (s->gemv_ws_bytes - kQueueRegionBytes) & ~(size_t)255;
  void* stream = L.stream;
  const uint32_t hq = m->n_q_heads, hkv = m->n_kv_heads, d = m->head_dim;
  const float scale = 1.0f / sqrtf((float)d);
  const uint32_t h_tiles = m->hidden / 128;
  const uint32_t tiles = max_row_tiles(m);
  SyncSlots slots;

  // epilogue descriptors: x = residual stream h with row statistics in ssq_a / ssq_b
  boost_gemv_epilogue_t scaled = {};
  scaled.mode = BOOST_EPI_PLAIN;
  scaled.ssq_in_tiles = h_tiles;
  scaled.ssq_stride = s->ssq_stride;
  scaled.rms_eps = m->rms_eps;
  boost_gemv_epilogue_t stats = {};
  stats.mode = BOOST_EPI_PLAIN;
  stats.ssq_stride = s->ssq_stride;

  // q, k, v = rope(rmsnorm(h) Wqkv^T): row scale from ssq_a, RoPE + KV append in the epilogue
  auto qkv_call = [&](const boost_llama_layer_t& ly) {
    boost_gemv_epilogue_t qkv = scaled;
    qkv.mode = BOOST_EPI_ROPE_APPEND;
    qkv.ssq_in = s->ssq_a;
    qkv.q_out = s->q_rot;
    qkv.k_page_ptr = ly.k_page_ptr;
    qkv.v_page_ptr = ly.v_page_ptr;
    qkv.n_pool_blocks = m->n_pool_blocks;
    qkv.block_table = block_table;
    qkv.max_blocks = max_blocks;
    qkv.ctx_lens = ctx_lens;
    qkv.n_q_heads = hq;
    qkv.n_kv_heads = hkv;
    qkv.rope_table = s->rope_table;
    if (pf) {
      const uint32_t li = (uint32_t)(&ly - m->layers);
      qkv.k_page_ptr2 = pf->layers[li].k_page_ptr_staged;
      qkv.v_page_ptr2 = pf->layers[li].v_page_ptr_staged;
    }
    return call_of(ly.wqkv, s->h, nullptr, 1, nullptr, qkv);
  };
  // Prefetch variant: the copy engine stages layer l's host pages into buffer l % 2.  A buffer
  // is free again once the attention kernel two layers back has finished; the staged copy must
  // be complete before the product that appends the new rows of layer l is launched.
  cudaStream_t cs = pc ? pc->copy_stream : nullptr;
  auto stage_layer = [&](uint32_t li) -> int {
    if (pf->host_bytes == 0) return BOOST_OK;
    int rc = BOOST_OK;
    if (li >= 2) rc = boosth::check(cudaStreamWaitEvent(cs, pc->attn_done[li - 2], 0));
    if (rc == BOOST_OK)
      rc = boosth::check(cudaMemcpyAsync(pf->k_stage[li & 1], pf->layers[li].k_host_src, pf->host_bytes,
                                         cudaMemcpyHostToDevice, cs));
    if (rc == BOOST_OK)
      rc = boosth::check(cudaMemcpyAsync(pf->v_stage[li & 1], pf->layers[li].v_host_src, pf->host_bytes,
                                         cudaMemcpyHostToDevice, cs));
    if (rc == BOOST_OK) rc = boosth::check(cudaEventRecord(pc->copy_done[li], cs));
    return rc;
  };
  auto wait_staged = [&](uint32_t li) -> int {
    if (pf->host_bytes == 0) return BOOST_OK;
    return boosth::check(cudaStreamWaitEvent((cudaStream_t)stream, pc->copy_done[li], 0));
  };
  if (pf) {
    if (!pc || pc->n_layers < m->n_layers || !pf->layers) return BOOST_ERR_INVALID;
    // the copies of this step come after everything already on the compute stream: the previous
    // step (which read the staging buffers and wrote new rows into the host pages), cache loads
    L.rc = boosth::check(cudaEventRecord(pc->step_begin, (cudaStream_t)stream));
    if (L.ok()) L.rc = boosth::check(cudaStreamWaitEvent(cs, pc->step_begin, 0));
    for (uint32_t li = 0; li < 2 && li < m->n_layers && L.ok(); ++li) L.rc = stage_layer(li);
    if (L.ok()) L.rc = wait_staged(0);
    if (!L.ok()) return L.rc;
  }
  auto chain = [&](const boost_gemv_call_t* calls, uint32_t n) {
    uint32_t extra = 0;
    const int rc = boosth::gemv_chain_launch(calls, n, B, s->gemv_ws, usable, slots.take(s, usable, n + 1), true, tiles,
                                             stream, &extra);
    L.extra += extra;   // (a product's combine may be a kernel of its own)
    return rc;
  };

  // The run length of the attention kernels' work items is a function of the context lengths:
  // decided once, by a one-threadblock kernel, for all the layers' launches of this step.
  L.run(kKindGlue, [&] {
    const boost_llama_layer_t& l0 = m->layers[0];
    return boosth::paged_attn_launch(s->q_rot, l0.k_page_ptr, l0.v_page_ptr, pf ? nullptr : m->kv_tier, (size_t)m->n_kv_pages,
                                     m->n_pool_blocks, block_table, max_blocks, ctx_lens, B, hq, hkv, d, scale, s->attn_ws,
                                     s->attn_ws_bytes, s->attn, stream, boosth::kAttnPlanOnly);
  });
  L.run(kKindGlue, [&] { return boost_rope_table(ctx_lens, B, d, m->rope_base, s->rope_table, stream); });
  L.run(kKindGlue, [&] {
    return boost_embed_gather_ssq(m->embed, m->vocab, m->hidden, tokens, B, s->h, s->ssq_a, s->ssq_stride, stream);
  });
  {
    const boost_gemv_call_t first = qkv_call(m->layers[0]);
    L.run(kKindGemv, [&] { return chain(&first, 1); });
  }
  for (uint32_t li = 0; li < m->n_layers && L.ok(); ++li) {
    const boost_llama_layer_t& ly = m->layers[li];
    L.run(kKindAttn, [&] {
      // prefetch variant: every page is read from HBM (host pages from their staged copy)
      // (with the plan of the step's attention launches - see the top of the step)
      return boosth::paged_attn_launch(s->q_rot, pf ? pf->layers[li].k_page_ptr_staged : ly.k_page_ptr,
                                       pf ? pf->layers[li].v_page_ptr_staged : ly.v_page_ptr,
                                       pf ? nullptr : m->kv_tier, (size_t)m->n_kv_pages, m->n_pool_blocks, block_table,
                                       max_blocks, ctx_lens, B, hq, hkv, d, scale, s->attn_ws, s->attn_ws_bytes, s->attn,
                                       stream, boosth::kAttnPlanReuse);
    });
    if (pf && L.ok()) {
      L.rc = boosth::check(cudaEventRecord(pc->attn_done[li], (cudaStream_t)stream));
      if (L.ok() && li + 2 < m->n_layers) L.rc = stage_layer(li + 2);
      if (L.ok() && li + 1 < m->n_layers) L.rc = wait_staged(li + 1);
    }
    // One launch for the four products between two attention kernels:
    //   h += attn Wo^T                       (row statistics of the new h into ssq_b)
    //   act = swiglu(rmsnorm(h) Wgu^T)       (row scale from ssq_b)
    //   h += act Wd^T                        (row statistics of the new h into ssq_a)
    //   next layer's q, k, v - or the logits = rmsnorm(h) Whead^T after the last layer
    boost_gemv_epilogue_t wo = stats;
    wo.ssq_out = s->ssq_b;
    boost_gemv_epilogue_t gu = scaled;
    gu.mode = BOOST_EPI_SWIGLU;
    gu.ssq_in = s->ssq_b;
    boost_gemv_epilogue_t wd = stats;
    wd.ssq_out = s->ssq_a;
    boost_gemv_epilogue_t head = scaled;
    head.ssq_in = s->ssq_a;
    boost_gemv_call_t calls[4] = {
        call_of(ly.wo, s->attn, s->h, 1, s->h, wo), call_of(ly.wgu, s->h, s->act, 1, nullptr, gu),
        call_of(ly.wd, s->act, s->h, 1, s->h, wd),
        li + 1 < m->n_layers ? qkv_call(m->layers[li + 1]) : call_of(m->lm_head, s->h, s->logits, 0, nullptr, head)};
    L.run(kKindGemv, [&] { return chain(calls, 4); });
  }
  L.run(kKindGlue, [&] { return boost_argmax(s->logits, B, m->vocab, next_tokens, stream); });
  return L.rc;
}

}  // namespace

extern "C" size_t boost_llama_gemv_workspace_bytes(const boost_llama_model_t* m, uint32_t B) {
  if (!m || !m->layers || B == 0 || B > 256) return 0;
  size_t partial = boosth::gemv_partial_bytes(m->lm_head.N, m->lm_head.K, B);
  for (uint32_t li = 0; li < m->n_layers; ++li) {
    const boost_llama_layer_t& ly = m->layers[li];
    const boost_weight_t* ws[4] = {&ly.wqkv, &ly.wo, &ly.wgu, &ly.wd};
    for (const boost_weight_t* w : ws) {
      const size_t b = boosth::gemv_partial_bytes(w->N, w->K, B);
      partial = b > partial ? b : partial;
    }
  }
  return boosth::gemv_header_bytes(max_row_tiles(m)) + partial + kQueueRegionBytes + 256;
}

extern "C" int boost_llama_decode_step(const boost_llama_model_t* m, const boost_llama_scratch_t* s,
                                       const int32_t* tokens, const int32_t* block_table,
                                       uint32_t max_blocks, const int32_t* ctx_lens, uint32_t B,
                                       int32_t* next_tokens, uint32_t* n_launches_out, void* stream) {
  static thread_local Launcher L;
  L.stream = stream; L.timed = false; L.count = 0; L.extra = 0; L.rc = BOOST_OK;
  const int rc = run_step(L, m, s, tokens, block_table, max_blocks, ctx_lens, B, next_tokens);
  if (n_launches_out) *n_launches_out = L.count + L.extra;
  return rc;
}

extern "C" int boost_prefetch_ctx_create(uint32_t n_layers, boost_prefetch_ctx** out) {
  if (!out || n_layers == 0) return BOOST_ERR_INVALID;
  boost_prefetch_ctx* c = new (std::nothrow) boost_prefetch_ctx;
  if (!c) return BOOST_ERR_INVALID;
  c->n_layers = n_layers;
  c->copy_done = new (std::nothrow) cudaEvent_t[n_layers]();
  c->attn_done = new (std::nothrow) cudaEvent_t[n_layers]();
  int rc = (c->copy_done && c->attn_done) ? BOOST_OK : BOOST_ERR_INVALID;
  if (rc == BOOST_OK) rc = boosth::check(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
  for (uint32_t i = 0; i < n_layers && rc == BOOST_OK; ++i) {
    rc = boosth::check(cudaEventCreateWithFlags(&c->copy_done[i], cudaEventDisableTiming));
    if (rc == BOOST_OK) rc = boosth::check(cudaEventCreateWithFlags(&c->attn_done[i], cudaEventDisableTiming));
  }
  if (rc == BOOST_OK) rc = boosth::check(cudaEventCreateWithFlags(&c->step_begin, cudaEventDisableTiming));
  if (rc != BOOST_OK) {
    boost_prefetch_ctx_destroy(c);
    return rc;
  }
  *out = c;
  return BOOST_OK;
}

extern "C" void boost_prefetch_ctx_destroy(boost_prefetch_ctx* c) {
  if (!c) return;
  for (uint32_t i = 0; i < c->n_layers; ++i) {
    if (c->copy_done && c->copy_done[i]) cudaEventDestroy(c->copy_done[i]);
    if (c->attn_done && c->attn_done[i]) cudaEventDestroy(c->attn_done[i]);
  }
  if (c->step_begin) cudaEventDestroy(c->step_begin);
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  delete[] c->copy_done;
  delete[] c->attn_done;
  delete c;
}

extern "C" int boost_llama_decode_step_prefetch(const boost_llama_model_t* m, const boost_llama_scratch_t* s,
                                                const boost_kv_prefetch_t* prefetch, boost_prefetch_ctx* ctx,
                                                const int32_t* tokens, const int32_t* block_table,
                                                uint32_t max_blocks, const int32_t* ctx_lens, uint32_t B,
                                                int32_t* next_tokens, uint32_t* n_launches_out, void* stream) {
  if (!prefetch || !ctx) return BOOST_ERR_INVALID;
  if (prefetch->host_bytes % BOOST_PAGE_BYTES != 0) return BOOST_ERR_INVALID;
  if (prefetch->host_bytes && (!prefetch->k_stage[0] || !prefetch->k_stage[1] || !prefetch->v_stage[0] || !prefetch->v_stage[1]))
    return BOOST_ERR_INVALID;
  static thread_local Launcher L;
  L.stream = stream; L.timed = false; L.count = 0; L.extra = 0; L.rc = BOOST_OK;
  const int rc = run_step(L, m, s, tokens, block_table, max_blocks, ctx_lens, B, next_tokens, prefetch, ctx);
  if (n_launches_out) *n_launches_out = L.count + L.extra;
  return rc;
}

extern "C" int boost_llama_decode_step_profile(const boost_llama_model_t* m, const boost_llama_scratch_t* s,
                                               const int32_t* tokens, const int32_t* block_table,
                                               uint32_t max_blocks, const int32_t* ctx_lens, uint32_t B,
                                               int32_t* next_tokens, float* kind_ms_out,
                                               uint32_t* kind_launches_out, void* stream) {
  if (!kind_ms_out || !kind_launches_out || !m) return BOOST_ERR_INVALID;
  if (5 + 2 * (uint64_t)m->n_layers > 512) return BOOST_ERR_UNSUPPORTED;
  static thread_local Launcher L;
  L.stream = stream; L.timed = true; L.count = 0; L.extra = 0; L.rc = BOOST_OK;
  const uint32_t n_events = 2 * (5 + 2 * m->n_layers);   // attention plan, rope table, embedding, first qkv, attention + chain per layer, argmax
  uint32_t made = 0;
  int rc = BOOST_OK;
  for (; made < n_events && rc == BOOST_OK; ++made) rc = boosth::check(cudaEventCreate(&L.ev[made]));
  if (rc == BOOST_OK) rc = run_step(L, m, s, tokens, block_table, max_blocks, ctx_lens, B, next_tokens);
  if (rc == BOOST_OK) rc = boosth::check(cudaStreamSynchronize((cudaStream_t)stream));
  for (int k = 0; k < kNumKinds; ++k) { kind_ms_out[k] = 0.f; kind_launches_out[k] = 0; }
  for (uint32_t i = 0; i < L.count && rc == BOOST_OK; ++i) {
    float ms = 0.f;
    rc = boosth::check(cudaEventElapsedTime(&ms, L.ev[2 * i], L.ev[2 * i + 1]));
    kind_ms_out[L.kind_of[i]] += ms;
    kind_launches_out[L.kind_of[i]] += 1;
  }
  for (uint32_t i = 0; i < made; ++i) cudaEventDestroy(L.ev[i]);
  return rc;
}

extern "C" int boost_llama_decode_step_host(const boost_llama_model_t* m, const boost_llama_scratch_t* s,
                                            const int32_t* tokens, const int32_t* block_table,
                                            uint32_t max_blocks, const int32_t* ctx_lens, uint32_t B,
                                            int32_t* next_tokens, uint32_t* n_launches_out, void* stream) {
  if (!m || !s || !tokens || !block_table || !ctx_lens || !next_tokens) return BOOST_ERR_INVALID;
  if (!s->tokens_dev || !s->ctx_dev || !s->table_dev || !s->next_dev) return BOOST_ERR_INVALID;
  cudaStream_t st = (cudaStream_t)stream;
  int rc = boosth::check(cudaMemcpyAsync(s->tokens_dev, tokens, (size_t)B * 4, cudaMemcpyHostToDevice, st));
  if (rc == BOOST_OK)
    rc = boosth::check(cudaMemcpyAsync(s->ctx_dev, ctx_lens, (size_t)B * 4, cudaMemcpyHostToDevice, st));
  if (rc == BOOST_OK)
    rc = boosth::check(cudaMemcpyAsync(s->table_dev, block_table, (size_t)B * max_blocks * 4,
                                       cudaMemcpyHostToDevice, st));
  if (rc != BOOST_OK) return rc;
  rc = boost_llama_decode_step(m, s, s->tokens_dev, s->table_dev, max_blocks, s->ctx_dev, B, s->next_dev,
                               n_launches_out, stream);
  if (rc != BOOST_OK) return rc;
  rc = boosth::check(cudaMemcpyAsync(next_tokens, s->next_dev, (size_t)B * 4, cudaMemcpyDeviceToHost, st));
  if (rc != BOOST_OK) return rc;
  return boosth::check(cudaStreamSynchronize(st));
}
