#!/usr/bin/env python
"""Benchmark of the tiered decode hot path on B200.

Default workload (N = 1): one Llama-3-8B-shaped decode step - 32 layers, hidden 4096, FFN
14336, 32 query / 8 KV heads, vocab 128256, bf16 random-init weights N(0, 0.02^2), batch
32, context 2048 - with weight pages placed by modulo placement at the host share that the
measured host-link / HBM bandwidth ratio gives, KV cache in HBM.  A step runs every kernel
of the path through the C ABI: RoPE table, embedding gather, the first layer's QKV product
(RMSNorm scale, RoPE and KV append in its epilogue), then 32 x [paged attention; ONE launch
for the output product + residual, the gate/up product with RMSNorm scale and SwiGLU, the
down product + residual and the next layer's QKV product - the LM head after the last
layer], argmax - 68 launches.

  python bench.py --gpus N --steps K --warmup W            # this repository's kernels
  python bench.py --impl reference ...                      # the CPU oracle on the host cores

Prints ONE JSON line on rank 0.  With N > 1 every rank runs an independent replica (the
path does not shard across GPUs; no collective on the data path) and the value is the sum
over ranks divided by the slowest rank's time.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

WORKLOAD = "llama3_8b_shaped_decode_step_b32_ctx2048_tiered_weights"
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + write) per algorithmic byte of the weight-product kernel, from one ncu
# capture of two full-size chain launches of this workload (profiles/
# gemv_tiered_kernel_chain_llama8b_m32.md): 1955.5 MB moved for 1872.8 MB of packed weights.
GEMV_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.046
GEMV_TRAFFIC_PROFILE = "profiles/gemv_tiered_kernel_chain_llama8b_m32.md (captured at commit 9e981ac)"
# the tcgen05 kernel (batches above 32), same kind of capture at batch 128: (511.7 + 1610.7) MB moved for
# (436.2 + 1436.6) MB of packed weights
GEMV_TC_TRAFFIC_PER_ALGORITHMIC_BYTE = 1.133
GEMV_TC_TRAFFIC_PROFILE = "profiles/gemv_tc_kernel_llama8b_m128.md"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.tmp = None

    def start(self):
        try:
            self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        clocks, reasons, mx = [], set(), None
        for line in self.tmp.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                clocks.append(float(f[1]))
                mx = float(f[2])
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.tmp.name)
        except OSError:
            pass
        if clocks:
            out.update(sm_mhz=float(np.median(clocks)), sm_max_mhz=mx, reasons=sorted(reasons),
                       samples=len(clocks))
        return out


# --------------------------------------------------------------------------- CPU oracle leg

_ORACLE_SAMPLE_INPUTS = {}   # (batch, ctx, seed) -> generated inputs, already passed through one untimed step


def cpu_oracle_sample(batch, ctx, seed=0):
    """Times the CPU oracle (as it stands) on a bounded sample of the default workload: one of
    the 32 layers plus the LM head at full batch and context; the layer time is scaled by 32.
    The inputs are generated, and the untimed first pass is run, once per process: repeated
    samples (the reference arm's steps) time the oracle only.
    Returns (tokens_per_s, description, threads, seconds of oracle time in this sample)."""
    from oracle import decode as od
    from paper_2609_13592_b200 import synth
    key = (batch, ctx, seed)
    if key not in _ORACLE_SAMPLE_INPUTS:
        _ORACLE_SAMPLE_INPUTS[key] = _oracle_sample_inputs(batch, ctx, seed)
    cfg, w, tokens, kc, vc, table, ctx_lens = _ORACLE_SAMPLE_INPUTS[key]
    t0 = time.perf_counter()
    od.decode_step(cfg, w, tokens, kc, vc, table, ctx_lens, n_layers=0)
    t_head = time.perf_counter() - t0
    t0 = time.perf_counter()
    od.decode_step(cfg, w, tokens, kc, vc, table, ctx_lens, n_layers=1)
    t_one = time.perf_counter() - t0
    t_layer = max(t_one - t_head, 1e-9)
    t_step = 32 * t_layer + t_head
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    desc = (f"1 of 32 layers + LM head at batch {batch}, context {ctx} "
            f"(layer {t_layer:.2f} s x 32 + head {t_head:.2f} s)")
    return batch / t_step, desc, threads, t_one + t_head


def _oracle_sample_inputs(batch, ctx, seed):
    from oracle import decode as od
    from paper_2609_13592_b200 import synth
    cfg = dict(synth.LLAMA3_8B, n_layers=1)
    hq, hkv, d, hid, ffn, vocab = (cfg[k] for k in ("n_q_heads", "n_kv_heads", "head_dim", "hidden", "ffn", "vocab"))
    head = synth.normal_bf16((vocab, hid), 0.02, seed + 1)
    layer = {"norm1": synth.f32_to_bf16_bits(np.ones(hid, np.float32)),
             "norm2": synth.f32_to_bf16_bits(np.ones(hid, np.float32)),
             "wqkv": synth.normal_bf16(((hq + 2 * hkv) * d, hid), 0.02, seed + 2),
             "wo": synth.normal_bf16((hid, hq * d), 0.02, seed + 3),
             "wgu": synth.normal_bf16((2 * ffn, hid), 0.02, seed + 4),
             "wd": synth.normal_bf16((hid, ffn), 0.02, seed + 5)}
    w = {"embed": head, "lm_head": head, "norm_f": layer["norm1"], "layers": [layer]}
    n_blk_seq = (ctx + 15) // 16
    n_blocks = batch * n_blk_seq
    kc = [synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, seed + 6)]
    vc = [synth.normal_bf16((hkv, n_blocks, 16, d), 1.0, seed + 7)]
    table = np.arange(n_blocks, dtype=np.int64).reshape(batch, n_blk_seq)
    tokens = np.arange(batch) * 97 % vocab
    ctx_lens = np.full(batch, ctx)
    # (one untimed pass of the head-only step first: the first touch of the multi-GB fp64 temporaries
    # would otherwise land in whichever of the two timed passes comes first)
    od.decode_step(cfg, w, tokens, kc, vc, table, ctx_lens, n_layers=0)
    return cfg, w, tokens, kc, vc, table, ctx_lens


def run_reference(args, rank, world):
    if rank != 0:
        return
    steps, vals = max(1, min(args.steps, 3)), []
    for _ in range(max(0, min(args.warmup, 1))):
        cpu_oracle_sample(32, 2048)
    desc, threads = "", 1
    t_total = 0.0
    for _ in range(steps):
        v, desc, threads, t = cpu_oracle_sample(32, 2048)
        vals.append(v)
        t_total += t
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": "decode_tokens_per_s", "value": value, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": steps, "warmup": min(args.warmup, 1),
            "ms_per_step": 1000.0 * 32 / value, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "note": "CPU oracle on the host cores, bounded sample per step"},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_reference_configs(args):
    """The CPU oracle, as it stands, timed on configurations 1 - 3 and on a sample of configuration 5
    (one layer's attention for 8 of its 128 sequences) on this machine's host cores: with
    one thread and with all of them (the BLAS calls inside numpy are what threads).  One JSON
    document; the decode-step sample of configuration 4 is the default `--impl reference` line."""
    from oracle import kv_pool as okp
    from oracle import linalg as ol
    from oracle import placement as op
    from paper_2609_13592_b200 import synth
    try:
        from threadpoolctl import threadpool_limits
    except Exception:
        threadpool_limits = None
    # inputs (not timed)
    w1, x1 = synth.normal_bf16((4096, 4096), 0.02, 1), synth.normal_bf16((1, 4096), 1.0, 2)
    ctx2 = synth.ctx_lens_uniform(8, 512, 4096, seed=2).tolist()
    pool = okp.KVPool(2560, 8, 8, 16 * 128 * 2)
    table = np.zeros((8, 256), np.int64)
    for b, c in enumerate(ctx2):
        blocks = pool.alloc(b, (c + 15) // 16)
        table[b, :len(blocks)] = blocks
    k2, v2 = synth.normal_bf16((8, 2560, 16, 128), 1.0, 20), synth.normal_bf16((8, 2560, 16, 128), 1.0, 21)
    q2 = synth.normal_bf16((8, 32, 128), 1.0, 22)
    page_elems = (2 << 20) // 2
    buf3 = synth.small_int_bf16(0, 512 * page_elems) if hasattr(synth, "small_int_bf16") else \
        synth.f32_to_bf16_bits(synth.small_int_values(0, 512 * page_elems).astype(np.float32))

    def timed(fn):
        t0 = time.perf_counter()
        fn()
        return time.perf_counter() - t0

    # configuration 5, sampled: the attention of one layer for 8 of the 128 sequences (context lengths
    # uniform in [2048, 4096], seed 5) through a pool with one page in five on the host
    ctx5 = synth.ctx_lens_uniform(128, 2048, 4096, seed=5)[:8].tolist()
    pool5 = okp.KVPool(2560, 8, 5, 16 * 128 * 2)
    table5 = np.zeros((8, 256), np.int64)
    for j in range(256):
        for b, c in enumerate(ctx5):
            if j < (c + 15) // 16:
                table5[b, j] = pool5.alloc(b, 1)[0]
    k5, v5 = synth.normal_bf16((8, 2560, 16, 128), 1.0, 50), synth.normal_bf16((8, 2560, 16, 128), 1.0, 51)
    q5 = synth.normal_bf16((8, 32, 128), 1.0, 52)
    cases = {
        "c5_sample_attention_of_one_layer_8_of_128_sequences_ctx2048_4096": lambda: ol.paged_attention_decode(
            q5, k5, v5, table5, ctx5, 1.0 / np.sqrt(128.0)),
        "c1_place_pages_and_gemv_4096x4096_batch1": lambda: (op.place_pages(4096 * 4096 * 2, 1 / 16), ol.gemm(x1, w1)),
        "c2_attention_batch8_ctx512_4096": lambda: ol.paged_attention_decode(q2, k2, v2, table, ctx2, 1.0 / np.sqrt(128.0)),
        "c3_stream_sum_1gib": lambda: ol.stream_sum(buf3, page_elems),
    }
    out = {}
    for name, fn in cases.items():
        row = {"all_cores_s": timed(fn)}
        if threadpool_limits is not None:
            with threadpool_limits(limits=1):
                row["one_thread_s"] = timed(fn)
        out[name] = row
    print(json.dumps({"impl": "reference", "workload": "oracle_on_configs_1_to_3_and_a_sample_of_5", "cores": os.cpu_count(),
                      "seconds": out}), flush=True)


# ------------------------------------------------------------------------------ device leg

def measure_stream(dev, n_pages, tier_value, reps=5, peer_device=None):
    """GB/s of the tiered stream-reduce kernel over n_pages pages all in one tier (the second
    tier: pinned host memory, or a peer GPU's memory when peer_device is given)."""
    import torch
    from paper_2609_13592_b200 import binding as B
    from paper_2609_13592_b200.tiers import TieredBuffer
    tier = np.full(n_pages, tier_value, np.uint8)
    buf = TieredBuffer(n_pages * B.PAGE_BYTES, device=dev, tier=tier, peer_device=peer_device)
    ws_bytes = B.boost_stream_reduce_workspace_bytes(n_pages)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
    sums = torch.zeros(n_pages, dtype=torch.float32, device=dev)
    best = float("inf")
    for i in range(reps + 2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.boost_stream_reduce_tiered(buf.page_ptr, buf.order, n_pages, buf.n_host, sums, ws, ws_bytes)
        e1.record()
        torch.cuda.synchronize(dev)
        if i >= 2:
            best = min(best, e0.elapsed_time(e1))
    del buf
    return n_pages * B.PAGE_BYTES / best / 1e6


def build_decoder(dev, cfg, host_ratio, batch, n_pool_blocks, max_blocks, seed, kv_host_modulus=0, kv_prefetch=False):
    import torch
    from paper_2609_13592_b200.llama import LlamaDecoder
    hq, hkv, d, hid, ffn, vocab = (cfg[k] for k in ("n_q_heads", "n_kv_heads", "head_dim", "hidden", "ffn", "vocab"))
    shapes = {"embed": (vocab, hid), "lm_head": (vocab, hid), "wqkv": ((hq + 2 * hkv) * d, hid),
              "wo": (hid, hq * d), "wgu": (2 * ffn, hid), "wd": (hid, ffn)}
    names = ["embed", "norm_f", "lm_head", "norm1", "wqkv", "wo", "norm2", "wgu", "wd"]

    def get_weight(name, layer):
        g = torch.Generator(device=dev)
        g.manual_seed(seed * 100003 + (0 if layer is None else layer + 1) * 101 + names.index(name))
        if name.startswith("norm"):
            return (1.0 + 0.02 * torch.randn(hid, generator=g, device=dev)).to(torch.bfloat16)
        return (0.02 * torch.randn(shapes[name], generator=g, device=dev)).to(torch.bfloat16)

    dec = LlamaDecoder(cfg, get_weight, host_ratio, n_pool_blocks, kv_host_modulus, batch, max_blocks, dev,
                       kv_prefetch=kv_prefetch)
    g = torch.Generator(device=dev)
    g.manual_seed(seed + 7)
    for ly in dec.layers:                      # synthetic context: KV ~ N(0, 1)
        for name in ("k", "v"):
            hbm = ly[name]._hbm.view(torch.bfloat16)
            hbm.normal_(0.0, 1.0, generator=g)
            if ly[name]._host is not None:     # host pages: a copy of device-generated values
                host = ly[name]._host.view(torch.bfloat16)
                n = min(host.numel(), hbm.numel())
                host[:n].copy_(hbm[:n])
    torch.cuda.synchronize(dev)
    return dec


class StepDriver:
    """Holds the per-step inputs of a run of consecutive decode steps of one decoder."""

    def __init__(self, dec, dev, batch, ctx0, n_steps, max_blocks):
        import torch
        self.dec, self.dev, self.batch, self.ctx0, self.max_blocks = dec, dev, batch, ctx0, max_blocks
        ctx0 = np.broadcast_to(np.asarray(ctx0, np.int64), (batch,))   # one length, or one per sequence
        need0 = (ctx0 + 15) // 16
        self.table = np.zeros((batch, max_blocks), np.int32)
        self.n_have = np.zeros(batch, np.int64)
        for j in range(int(need0.max())):      # round-robin growth through the wave-aware pool
            for b in range(batch):
                if j < need0[b]:
                    self.table[b, j] = dec.pool.alloc(b, 1)[0]
        self.n_have[:] = need0
        self.ctx = ctx0 - 1                             # the first step brings it to ctx0
        self.torch = torch

    def advance(self):
        """Next step's context lengths; new blocks come from the pool when a sequence crosses
        a block boundary."""
        self.ctx += 1
        for b in range(self.batch):
            while self.n_have[b] * 16 < self.ctx[b]:
                self.table[b, self.n_have[b]] = self.dec.pool.alloc(b, 1)[0]
                self.n_have[b] += 1
        return self.ctx

    def release(self):
        for b in range(self.batch):
            self.dec.pool.free(b)


def timed_device_steps(dec, dev, batch, ctx0, warmup, steps, max_blocks, dist_ctx, prefetch=False, profile=True):
    """Device-resident loop: inputs already in HBM; K steps between two events."""
    import torch
    step_fn = dec.step_prefetch if prefetch else dec.step
    drv = StepDriver(dec, dev, batch, ctx0, warmup + steps, max_blocks)
    ctx_all = np.zeros((warmup + steps, batch), np.int32)
    for i in range(warmup + steps):
        ctx_all[i] = drv.advance()
    ctx_dev = torch.from_numpy(ctx_all).to(dev)
    table_dev = torch.from_numpy(drv.table).to(dev)
    tok = [torch.arange(batch, dtype=torch.int32, device=dev) * 97 % dec.cfg["vocab"],
           torch.zeros(batch, dtype=torch.int32, device=dev)]
    stream = torch.cuda.current_stream(dev)
    launches = 0
    for i in range(warmup):
        step_fn(tok[i % 2], table_dev, ctx_dev[i], tok[(i + 1) % 2], stream)
    dist_ctx.barrier()
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(warmup, warmup + steps):
        launches += step_fn(tok[i % 2], table_dev, ctx_dev[i], tok[(i + 1) % 2], stream)
    e1.record(stream)
    torch.cuda.synchronize(dev)
    dist_ctx.barrier()
    ms = e0.elapsed_time(e1)
    kv_tokens = int(ctx_all[warmup:].sum())
    dec.last_tokens = tok[(warmup + steps) % 2].cpu().numpy().copy()   # what the last timed step produced
    if not profile:
        drv.release()
        return ms, launches, kv_tokens, None, None
    # per-kind device time of one more step (events around every launch)
    i = warmup + steps - 1
    from paper_2609_13592_b200 import binding as B
    kind_ms, kind_n = B.boost_llama_decode_step_profile(dec.model, dec.scratch, tok[i % 2], table_dev,
                                                        max_blocks, ctx_dev[i], batch, tok[(i + 1) % 2], stream)
    drv.release()
    return ms, launches, kv_tokens, kind_ms, kind_n


def timed_host_steps(dec, dev, batch, ctx0, warmup, steps, max_blocks, dist_ctx):
    """End-to-end loop through the host-buffer entry point: per step the tokens, context
    lengths and block table go host -> device and the next tokens come back."""
    import torch
    drv = StepDriver(dec, dev, batch, ctx0, warmup + steps, max_blocks)
    tok_pin = torch.zeros(batch, dtype=torch.int32).pin_memory()
    ctx_pin = torch.zeros(batch, dtype=torch.int32).pin_memory()
    tab_pin = torch.zeros(batch, max_blocks, dtype=torch.int32).pin_memory()
    nxt_pin = torch.zeros(batch, dtype=torch.int32).pin_memory()
    tok_pin.numpy()[:] = np.arange(batch) * 97 % dec.cfg["vocab"]
    stream = torch.cuda.current_stream(dev)

    def one_step():
        ctx_pin.numpy()[:] = drv.advance()
        tab_pin.numpy()[:] = drv.table
        dec.step_host(tok_pin.numpy(), tab_pin.numpy(), ctx_pin.numpy(), nxt_pin.numpy(), stream)
        tok_pin.numpy()[:] = nxt_pin.numpy()         # the generated token is the next input

    for _ in range(warmup):
        one_step()
    dist_ctx.barrier()
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        one_step()
    e1.record(stream)
    torch.cuda.synchronize(dev)
    dist_ctx.barrier()
    ms = e0.elapsed_time(e1)
    drv.release()
    h2d = batch * 4 * 2 + batch * max_blocks * 4
    d2h = batch * 4
    return ms, h2d, d2h


def aggregate_replicas(ms, dist, device):
    """Slowest rank's time: MAX all-reduce over the ranks (each rank ran its own replica)."""
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_job_value(batch, world, ms_per_step):
    """Whole-job decode tokens/s of `world` independent replicas of `batch` sequences."""
    return world * batch / (ms_per_step / 1e3)


class DistCtx:
    def __init__(self, rank, world, dev):
        self.rank, self.world, self.dev = rank, world, dev
        self.dist = None
        if world > 1:
            import torch.distributed as dist
            dist.init_process_group(backend="nccl", device_id=dev)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def max(self, x):
        if self.dist is None:
            return x
        return aggregate_replicas(x, self.dist, self.dev)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def run_ours(args, rank, world, local_rank):
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    from paper_2609_13592_b200 import binding as B
    from paper_2609_13592_b200 import build as libbuild
    from paper_2609_13592_b200 import synth
    libbuild.build_library()
    B.lib()
    dev = torch.device(f"cuda:{local_rank}")
    torch.cuda.set_device(dev)
    dist_ctx = DistCtx(rank, world, dev)
    hbm_peak, peak_src = load_peaks()

    # host-link and HBM read bandwidth of this machine, measured in this run with the same kernel
    link_gbs = measure_stream(dev, 64, 1)            # 128 MiB of host-mapped pinned pages
    hbm_read_gbs = measure_stream(dev, 1024, 0)      # 2 GiB in HBM
    # K = HBM read bandwidth / link bandwidth, both measured with the same kernel in this run
    modulus = B.boost_modulus_from_bandwidths(max(hbm_read_gbs, hbm_peak), link_gbs)
    host_ratio = 1.0 / modulus

    cfg = dict(synth.LLAMA3_8B)
    if args.layers:
        cfg["n_layers"] = args.layers
    batch, ctx0 = args.batch, args.ctx
    total_steps = args.warmup + args.steps
    blocks_per_seq = (ctx0 + total_steps + 15) // 16 + 1
    max_blocks = blocks_per_seq
    n_pool_blocks = -(-batch * blocks_per_seq // 512) * 512

    results = {}
    clocks = None
    for label, ratio in (("hbm_only", 0.0), ("tiered", host_ratio)):
        dec = build_decoder(dev, cfg, ratio, batch, n_pool_blocks, max_blocks, seed=1)
        sampler = ClockSampler(local_rank)
        if label == "tiered":
            sampler.start()
        ms, launches, kv_tokens, kind_ms, kind_n = timed_device_steps(dec, dev, batch, ctx0, args.warmup,
                                                                     args.steps, max_blocks, dist_ctx)
        if label == "tiered":
            clocks = sampler.stop()
        r = {"ms": dist_ctx.max(ms), "launches": launches, "kv_tokens": kv_tokens, "kind_ms": kind_ms,
             "kind_n": kind_n, "weight_bytes": dec.weight_bytes(), "kv_bytes_per_token": dec.kv_bytes_per_token(),
             "host_pages": dec.host_weight_pages(), "status": dec.status_words(),
             "last_tokens": dec.last_tokens}
        if label == "tiered":
            e_ms, h2d, d2h = timed_host_steps(dec, dev, batch, ctx0, args.warmup, args.steps, max_blocks, dist_ctx)
            r.update(e2e_ms=dist_ctx.max(e_ms), h2d=h2d, d2h=d2h)
            # comparison variant: the same model and placement under the paper's schedule for weights
            # with host pages (two queues of work items, host pages first, Sec. 3.1 / 3.2)
            B.boost_gemv_set_tier_schedule(True)
            try:
                q_ms = timed_device_steps(dec, dev, batch, ctx0, args.warmup, args.steps, max_blocks, dist_ctx)[0]
            finally:
                B.boost_gemv_set_tier_schedule(False)
            r.update(two_queue_ms=dist_ctx.max(q_ms))
        results[label] = r
        del dec
        torch.cuda.empty_cache()

    if rank == 0:
        t = results["tiered"]
        ms_step = t["ms"] / args.steps
        value = replica_job_value(batch, world, ms_step)
        bytes_step = t["weight_bytes"] + t["kv_tokens"] / args.steps * t["kv_bytes_per_token"]
        combined = bytes_step / (ms_step / 1e3) / 1e9
        roof = hbm_peak + link_gbs
        gemv_ms, gemv_n = t["kind_ms"][0], t["kind_n"][0]
        gemv_gbs = t["weight_bytes"] / (gemv_ms / 1e3) / 1e9
        gemv_bytes_per_launch = t["weight_bytes"] / max(gemv_n, 1)
        gemv_step_bytes = t["weight_bytes"]
        # tier-wise bound: the slower of the two tiers if each streamed its own bytes at its own peak
        host_bytes = t["host_pages"] * (2 << 20)
        t_min_ms = 1e3 * max((bytes_step - host_bytes) / (hbm_peak * 1e9), host_bytes / (link_gbs * 1e9))
        attn_ms, attn_n = t["kind_ms"][1], t["kind_n"][1]
        attn_bytes = t["kv_tokens"] / args.steps * t["kv_bytes_per_token"]
        attn_gbs = attn_bytes / (attn_ms / 1e3) / 1e9
        hb = results["hbm_only"]
        hb_ms = hb["ms"] / args.steps
        line = {
            "metric": "decode_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "batch": batch, "context": ctx0, "layers": cfg["n_layers"],
                       "weight_placement": f"modulo, host share 1/{modulus} per tensor",
                       "kv_placement": "HBM", "l2": "inputs larger than L2 (weights 15 GB per step)",
                       "multi_gpu": "replicas only" if world > 1 else "single GPU"},
            "tpot_ms": ms_step,
            "combined_read_gbs": combined,
            "combined_roofline_gbs": roof,
            "combined_roofline_frac": combined / roof,
            "tier_bound": {"t_min_ms": t_min_ms, "frac_of_t_min": t_min_ms / ms_step,
                           "host_bytes_per_step": host_bytes},
            "hbm_peak_gbs": hbm_peak, "hbm_peak_source": peak_src,
            "host_link": {"type": "PCIe (zero-copy SM loads of pinned host memory)", "read_gbs": link_gbs,
                          "alpha": link_gbs / hbm_peak, "modulus": modulus},
            "hbm_read_gbs_stream_kernel": hbm_read_gbs,
            "algorithmic_bytes_per_step": bytes_step,
            "host_weight_pages": t["host_pages"],
            "hbm_only": {"ms_per_step": hb_ms, "value": world * batch / (hb_ms / 1e3),
                         "tiered_over_hbm_only_time": ms_step / hb_ms},
            "tiered_over_hbm_only_time": ms_step / hb_ms,
            # same model, inputs and steps: with host pages read in place the work partition does not
            # depend on the placement, so the tiered run must reproduce the HBM-only run's tokens
            "tiered_tokens_equal_hbm_only": bool(np.array_equal(t["last_tokens"], results["hbm_only"]["last_tokens"])),
            "weight_tier_schedule": {"this_line": "host pages read in place under the even partition",
                                     "two_queues_host_first_ms_per_step": t["two_queue_ms"] / args.steps},
            "roofline": {"bound": "hbm", "kernel": (f"gemv_tiered_kernel (weight products, M_b = {batch})" if batch <= 32 else
                                                    f"gemv_tc_kernel (weight products on tcgen05, M_b = {batch})"),
                         "achieved": gemv_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gemv_gbs / hbm_peak,
                         "algorithmic_bytes_per_launch": gemv_bytes_per_launch,
                         "traffic": (GEMV_TRAFFIC_PER_ALGORITHMIC_BYTE if batch <= 32 else GEMV_TC_TRAFFIC_PER_ALGORITHMIC_BYTE) * gemv_bytes_per_launch,
                         "traffic_source": ("ncu dram bytes of this workload's launches, ratio 1.046 to algorithmic" if batch <= 32 else
                                            "ncu dram bytes of the same chains at batch 128, ratio 1.133 to algorithmic"),
                         "launches_per_step": gemv_n, "avg_launch_us": 1e3 * gemv_ms / max(gemv_n, 1),
                         "peak_source": peak_src,
                         # events around every launch serialise the step: no launch overlaps its neighbours
                         "serialised": True,
                         # the same bytes over the weight products' share of the overlapped step
                         # (step time minus the serialised time of the other kinds): an upper estimate
                         "achieved_in_step": gemv_step_bytes / (max(ms_step - t["kind_ms"][1] - t["kind_ms"][2], 1e-6) / 1e3) / 1e9,
                         "traffic_profile": GEMV_TRAFFIC_PROFILE if batch <= 32 else GEMV_TC_TRAFFIC_PROFILE},
            "roofline_attention": {"bound": "hbm", "kernel": "paged_attn_kernel", "achieved": attn_gbs,
                                   "peak": hbm_peak, "unit": "GB/s", "frac": attn_gbs / hbm_peak,
                                   "launches_per_step": attn_n, "avg_launch_us": 1e3 * attn_ms / max(attn_n, 1)},
            "kernel_time_share": {"gemv": t["kind_ms"][0], "attention": t["kind_ms"][1], "glue": t["kind_ms"][2],
                                  "unit": "ms of one step, events around every launch"},
            "e2e": {"value": world * batch / (t["e2e_ms"] / args.steps / 1e3), "unit": "tokens/s",
                    "h2d_bytes_per_step": t["h2d"], "d2h_bytes_per_step": t["d2h"],
                    "ms_per_step": t["e2e_ms"] / args.steps},
            "gpu_launches": t["launches"],
            "clocks": clocks,
            "device_status_words": t["status"],
        }
        if not args.no_cpu_baseline and world == 1:
            v, desc, threads, _ = cpu_oracle_sample(batch, ctx0)
            line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                                    "sample": desc}
        elif world > 1:
            line["cpu_baseline"] = None
        print(json.dumps(line), flush=True)
    dist_ctx.close()


def run_kv_spill(args):
    """Configuration 5: Llama-3-8B-shaped decode, batch 128, context lengths uniform in
    [2048, 4096]; the pool keeps one page in five of every KV tensor in host memory (an HBM
    budget of 80 % of the pages).  Three runs of the same kernels: host pages read in place by
    the SMs (the tiered path), the prefetch-to-HBM variant (copy engine, two layers ahead), and
    HBM-only at the largest batch whose blocks fit the 80 % budget.  One JSON line."""
    import torch
    from paper_2609_13592_b200 import binding as B
    from paper_2609_13592_b200 import build as libbuild
    from paper_2609_13592_b200 import synth
    libbuild.build_library()
    B.lib()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    hbm_peak, peak_src = load_peaks()
    link_gbs = measure_stream(dev, 64, 1)
    cfg = dict(synth.LLAMA3_8B)
    if args.layers:
        cfg["n_layers"] = args.layers
    batch = args.batch if args.batch != 32 else 128
    steps, warmup = min(args.steps, 5), 3
    total_steps = warmup + steps
    ctx0 = synth.ctx_lens_uniform(batch, 2048, 4096, seed=5).astype(np.int64)
    blocks = (ctx0 + total_steps + 15) // 16 + 1
    max_blocks = int(blocks.max())
    n_pool_blocks = -(-int(blocks.sum()) // 512) * 512
    # HBM-only comparison: the longest prefix of the batch whose blocks fit 80 % of the pool
    budget = int(0.8 * n_pool_blocks) // 512 * 512
    small = int(np.searchsorted(np.cumsum(blocks), budget, side="right"))
    null = DistCtx(0, 1, dev)
    out = {}
    last_tokens = {}
    for label, b_run, pool_blocks, modulus, prefetch in (("tiered", batch, n_pool_blocks, 5, False),
                                                         ("prefetch", batch, n_pool_blocks, 5, True),
                                                         ("hbm_only", small, budget, 0, False)):
        dec = build_decoder(dev, cfg, 0.0, b_run, pool_blocks, max_blocks, seed=1, kv_host_modulus=modulus,
                            kv_prefetch=prefetch)
        ms, launches, kv_tokens, _, _ = timed_device_steps(dec, dev, b_run, ctx0[:b_run], warmup, steps, max_blocks,
                                                           null, prefetch=prefetch, profile=False)
        host_pages = dec.layers[0]["k"].n_host
        kv_bytes = kv_tokens / steps * dec.kv_bytes_per_token()
        host_share = host_pages / dec.layers[0]["k"].n_pages
        out[label] = {"batch": b_run, "ms_per_step": ms / steps, "tokens_per_s": b_run / (ms / steps / 1e3),
                      "kv_bytes_per_step": kv_bytes, "host_kv_bytes_per_step": kv_bytes * host_share,
                      "weight_bytes": dec.weight_bytes(), "launches_per_step": launches // steps,
                      "pool_blocks": pool_blocks, "kv_host_pages_per_tensor": host_pages,
                      "status": dec.status_words()}
        last_tokens[label] = dec.last_tokens
        del dec
        torch.cuda.empty_cache()
    t = out["tiered"]
    bytes_step = t["weight_bytes"] + t["kv_bytes_per_step"]
    t_min_ms = 1e3 * max((bytes_step - t["host_kv_bytes_per_step"]) / (hbm_peak * 1e9),
                         t["host_kv_bytes_per_step"] / (link_gbs * 1e9))
    line = {"metric": "decode_tokens_per_s", "value": t["tokens_per_s"], "unit": "tokens/s", "n_gpus": 1,
            "steps": steps, "warmup": warmup, "ms_per_step": t["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "llama3_8b_shaped_decode_b128_ctx2048_4096_kv_spill_one_page_in_five",
                       "batch": batch, "layers": cfg["n_layers"], "kv_placement": "pool, host modulus 5",
                       "weight_placement": "HBM"},
            "host_link_gbs": link_gbs, "hbm_peak_gbs": hbm_peak, "hbm_peak_source": peak_src,
            "combined_read_gbs": bytes_step / (t["ms_per_step"] / 1e3) / 1e9,
            "combined_roofline_gbs": hbm_peak + link_gbs,
            "tier_bound": {"t_min_ms": t_min_ms, "frac_of_t_min": t_min_ms / t["ms_per_step"],
                           "note": "the host share (20 %) is far above the link share of this box, so the step is link-bound"},
            "runs": out,
            # the same seeded model, cache and inputs: reading host pages in place and reading their
            # staged copies must produce the same tokens after the same steps, sequence by sequence
            "verified": {"tiered_vs_prefetch_next_tokens_equal": bool(np.array_equal(last_tokens["tiered"], last_tokens["prefetch"])),
                         "sequences_compared": int(last_tokens["tiered"].size),
                         "all_status_words_zero": all(v == 0 for r in out.values() for v in r["status"])}}
    print(json.dumps(line), flush=True)
    if not (line["verified"]["tiered_vs_prefetch_next_tokens_equal"] and line["verified"]["all_status_words_zero"]):
        raise SystemExit("kv_spill: the tiered and the prefetch run disagree, or a kernel recorded an error")


def run_pool_churn(args):
    """KV pool under serving-like churn (Sec. 5.8, Sec. 5.11): Poisson arrivals with a
    long-generation length mix are replayed on the wave-aware pool at about 80 % utilisation for
    12 000 decode steps; the host share of the live KV chunks is recorded after every step
    (rolling median and min - max band over 500 steps, against the configured 1/M and the 1/H
    granularity bound), and at five steps the attention kernel is timed on the batch as the
    churned pool laid it out, on the same batch laid out by an unused pool, and with every KV
    page in HBM.  Three pools: four KV heads with one page in twelve on the host, eight KV
    heads with one page in eight, and eight KV heads at the measured link share.  Prints one
    JSON document."""
    import math
    import torch
    from paper_2609_13592_b200 import binding as B
    from paper_2609_13592_b200 import build as libbuild
    from paper_2609_13592_b200 import serving, synth
    from paper_2609_13592_b200.tiers import TieredKVCache, aligned_workspace
    libbuild.build_library()
    B.lib()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    hbm_peak, peak_src = load_peaks()
    link = measure_stream(dev, 64, 1)
    link_modulus = B.boost_modulus_from_bandwidths(hbm_peak, link)
    d, n_steps, window = 128, args.churn_steps, 500
    snaps = [int(n_steps * f) - 1 for f in (1 / 3, 1 / 2, 2 / 3, 5 / 6, 1.0)]
    pools = [dict(name="4_kv_heads_one_page_in_12", n_blocks=12 * 1024, hkv=4, hq=32, modulus=12, rate=0.045, max_batch=96),
             dict(name="8_kv_heads_one_page_in_8", n_blocks=8 * 1024, hkv=8, hq=32, modulus=8, rate=0.028, max_batch=64),
             dict(name=f"8_kv_heads_link_share_one_page_in_{link_modulus}", n_blocks=64 * 1024, hkv=8, hq=32,
                  modulus=link_modulus, rate=0.22, max_batch=384)]
    g = torch.Generator(device=dev)
    g.manual_seed(11)
    scale = 1.0 / math.sqrt(d)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    flush_read = torch.zeros(256 << 18, dtype=torch.float32, device=dev)

    def time_attention(cache, table, ctx, hq, hkv, n_blocks, reps=20):
        n_seq, max_blocks = table.shape
        ws_bytes = B.boost_paged_attn_workspace_bytes(n_seq, hq, d, max_blocks)
        ws_t, ws = aligned_workspace(ws_bytes, dev)
        q = torch.randn(n_seq, hq, d, generator=g, device=dev).to(torch.bfloat16)
        out = torch.empty(n_seq, hq, d, dtype=torch.bfloat16, device=dev)
        table_d, ctx_d = torch.from_numpy(table).to(dev), torch.from_numpy(ctx).to(dev)
        # every launch starts with a cold and clean L2: a 256 MB buffer (twice the L2) is written,
        # then another one is read, which pushes the written lines out - left dirty they would be
        # written back during the timed launch and add up to an L2's worth of HBM writes to it
        # (measured: 10 - 15 % on these launches).  The launch is queued while the flush still
        # runs, so the events see the kernel and not the host's launch path
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps + 3)]
        for e0, e1 in ev:
            flush.zero_()
            flush_read.sum()
            e0.record()
            B.boost_paged_attn_decode_tiered(q, cache.k.page_ptr, cache.v.page_ptr, cache.tier, cache.n_pages, n_blocks,
                                             table_d, max_blocks, ctx_d, n_seq, hq, hkv, d, scale, ws, ws_bytes, out)
            e1.record()
        torch.cuda.synchronize(dev)
        times = [e0.elapsed_time(e1) * 1e3 for e0, e1 in ev[3:]]
        off = ws - ws_t.data_ptr()
        status = int(ws_t[off:off + 4].cpu().numpy().view(np.uint32)[0])
        assert bool(torch.isfinite(out.float()).all())
        return float(np.median(times)), status

    results = []
    for pc in pools:
        n_blocks, hkv, hq, m = pc["n_blocks"], pc["hkv"], pc["hq"], pc["modulus"]
        pool = B.KVPool(n_blocks, hkv, m)
        trace = synth.serving_churn_trace(n_blocks, n_steps, pc["rate"], pc["max_batch"], seed=7)
        shares, batch_sizes, live_blocks, snapshots, stats = serving.replay_churn(pool, trace, snaps)
        warm = n_steps // 4
        s = shares[warm:]
        medians = [float(np.median(s[i:i + window])) for i in range(0, len(s) - window, 50)]
        lows = [float(s[i:i + window].min()) for i in range(0, len(s) - window, 50)]
        highs = [float(s[i:i + window].max()) for i in range(0, len(s) - window, 50)]
        info = pool.query()
        cache = TieredKVCache(pool, hkv, n_blocks, d, dev)
        hbm_pool = B.KVPool(n_blocks, hkv, 0)
        hbm_cache = TieredKVCache(hbm_pool, hkv, n_blocks, d, dev)
        for c in (cache, hbm_cache):
            for buf in (c.k, c.v):
                t = torch.randn(hkv, n_blocks, 16, d, generator=g, device=dev, dtype=torch.bfloat16)
                B.boost_kv_scatter(t, hkv, n_blocks, d, buf.page_ptr, buf.n_pages)
                torch.cuda.synchronize(dev)
                del t
        points = []
        for sn in snapshots:
            ctx, table = sn["ctx_lens"], sn["table"]
            host_b, all_b = serving.host_kv_bytes(table, ctx, dict(info, n_kv_heads=hkv), d)
            fresh_pool = B.KVPool(n_blocks, hkv, m)
            fresh = serving.fresh_tables(fresh_pool, ctx)
            fresh_host_b, _ = serving.host_kv_bytes(fresh, ctx, dict(info, n_kv_heads=hkv), d)
            fresh_pool.close()
            us_churn, st1 = time_attention(cache, table, ctx, hq, hkv, n_blocks)
            us_fresh, st2 = time_attention(cache, fresh, ctx, hq, hkv, n_blocks)
            us_hbm, st3 = time_attention(hbm_cache, table, ctx, hq, hkv, n_blocks)

            def bound_us(host_bytes):
                return 1e6 * max((all_b - host_bytes) / (hbm_peak * 1e9), host_bytes / (link * 1e9))
            points.append({"step": sn["step"], "batch": int(len(ctx)), "tokens": int(ctx.sum()), "max_ctx": int(ctx.max()),
                           "kv_bytes": all_b, "host_share_churned": host_b / all_b, "host_share_fresh": fresh_host_b / all_b,
                           "us_churned": us_churn, "us_fresh": us_fresh, "us_hbm_only": us_hbm,
                           "tier_bound_us_churned": bound_us(host_b), "tier_bound_us_fresh": bound_us(fresh_host_b),
                           "frac_of_tier_bound_churned": bound_us(host_b) / us_churn,
                           "frac_of_tier_bound_fresh": bound_us(fresh_host_b) / us_fresh,
                           "hbm_only_gbs": all_b / us_hbm / 1e3, "status": [st1, st2, st3]})
        results.append({"pool": pc["name"], "n_blocks": n_blocks, "n_kv_heads": hkv, "n_q_heads": hq, "host_modulus": m,
                        "target_share": info["n_host_pages"] / info["n_pages"], "granularity_bound": 1.0 / hkv,
                        "arrivals_per_step": pc["rate"], "max_batch": pc["max_batch"], "steps": n_steps,
                        "trace": stats, "mean_batch": float(batch_sizes[warm:].mean()),
                        "mean_utilisation": float(live_blocks[warm:].mean() / n_blocks),
                        "peak_utilisation": float(live_blocks.max() / n_blocks),
                        "share_after_warm_in": {"min": float(s.min()), "median": float(np.median(s)), "max": float(s.max())},
                        "rolling_median_band": [min(medians), max(medians)],
                        "rolling_min_max_band": [min(lows), max(highs)],
                        "attention": points})
        pool.close()
        hbm_pool.close()
        del cache, hbm_cache
        torch.cuda.empty_cache()
    print(json.dumps({"workload": "kv_pool_under_serving_churn", "hbm_peak_gbs": hbm_peak, "hbm_peak_source": peak_src,
                      "host_link_gbs": link, "pools": results}))


def run_gemv_sweep(args):
    """Weight-product sweep over the Llama-3-8B matrix shapes, batch 1 .. 128 and three host
    shares (0, the measured link share, 1/16): where tiering is free, where the link binds, and
    where each of the three product kernels (CUDA cores, mma.sync, tcgen05) takes over.  Every
    point: a CUDA graph of back-to-back launches over rotating copies of the weight that
    together exceed twice the L2.  Prints one JSON document."""
    import torch
    from paper_2609_13592_b200 import binding as B
    from paper_2609_13592_b200 import build as libbuild
    from paper_2609_13592_b200.tiers import TieredWeight
    libbuild.build_library()
    B.lib()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    hbm_peak, peak_src = load_peaks()
    link = measure_stream(dev, 64, 1)
    modulus = B.boost_modulus_from_bandwidths(hbm_peak, link)
    shapes = {"qkv": (6144, 4096), "o": (4096, 4096), "gate_up": (28672, 4096), "down": (4096, 14336),
              "lm_head": (128256, 4096)}
    ratios = [("hbm_only", 0.0), (f"link_share_1/{modulus}", 1.0 / modulus), ("1/16", 1.0 / 16)]
    batches = [1, 2, 4, 8, 16, 32, 64, 128, 256]
    points = []
    g = torch.Generator(device=dev)
    g.manual_seed(3)
    for name, (n, k) in shapes.items():
        n_copies = max(2, int(np.ceil(2 * 126e6 / (n * k * 2))))
        for label, ratio in ratios:
            ws = [TieredWeight((0.02 * torch.randn(n, k, generator=g, device=dev)).to(torch.bfloat16), ratio, device=dev)
                  for _ in range(n_copies)]
            host_pages, pages = ws[0].buf.n_host, ws[0].buf.n_pages
            for mb in batches:
                x = torch.randn(mb, k, generator=g, device=dev).to(torch.bfloat16)
                y = torch.empty(mb, n, dtype=torch.bfloat16, device=dev)
                for w in ws:
                    w.gemv(x, y=y)
                torch.cuda.synchronize(dev)
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    for w in ws:
                        w.gemv(x, y=y)
                graph.replay()
                torch.cuda.synchronize(dev)
                reps = 5 if host_pages > 8 else 10
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(reps):
                    graph.replay()
                e1.record()
                torch.cuda.synchronize(dev)
                us = e0.elapsed_time(e1) * 1e3 / (reps * n_copies)
                nbytes = ws[0].layout["bytes"]
                host_bytes = host_pages * B.PAGE_BYTES
                t_min_us = 1e6 * max((nbytes - host_bytes) / (hbm_peak * 1e9), host_bytes / (link * 1e9))
                points.append({"matrix": name, "N": n, "K": k, "batch": mb, "placement": label, "pages": pages,
                               "host_pages": host_pages, "us": us, "gbs": nbytes / us / 1e3,
                               "tier_bound_us": t_min_us, "frac_of_tier_bound": t_min_us / us,
                               "status": ws[0].status_words()})
                del graph
            del ws
            torch.cuda.empty_cache()
    print(json.dumps({"workload": "weight_product_shape_batch_sweep", "hbm_peak_gbs": hbm_peak, "hbm_peak_source": peak_src,
                      "host_link_gbs": link, "points": points}))


def run_peer_tier(args):
    """The second tier in a peer GPU's HBM, read over NVLink (the paper's bandwidth-ratio
    ablation): one process, GPU 0 computes, GPU 1 only holds pages.  Measures the peer-read
    bandwidth with the stream-reduce kernel, derives the modulus from it, and compares tiered
    with HBM-only runs of the stream reduce and of two weight products.  Needs two GPUs with peer
    access; prints an `unavailable` line otherwise.  Prints one JSON document."""
    import torch
    from paper_2609_13592_b200 import binding as B
    from paper_2609_13592_b200 import build as libbuild
    from paper_2609_13592_b200.tiers import TieredBuffer, TieredWeight
    if torch.cuda.device_count() < 2:
        print(json.dumps({"workload": "peer_gpu_second_tier", "unavailable": "needs two GPUs in one process; this box shows %d" % torch.cuda.device_count()}))
        return
    libbuild.build_library()
    B.lib()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    torch.zeros(1, device=dev)
    try:
        B.boost_peer_tier_open(1)
    except B.BoostError as e:
        print(json.dumps({"workload": "peer_gpu_second_tier", "unavailable": "no peer access from GPU 0 to GPU 1: %s" % e}))
        return
    hbm_peak, peak_src = load_peaks()
    link = measure_stream(dev, 512, 1, peer_device=1)
    modulus = B.boost_modulus_from_bandwidths(hbm_peak, link)
    out = {"workload": "peer_gpu_second_tier", "hbm_peak_gbs": hbm_peak, "hbm_peak_source": peak_src, "peer_read_gbs": link,
           "alpha": link / (hbm_peak + link), "modulus": modulus, "stream": [], "weight_products": []}

    def time_us(fn, reps):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) * 1e3 / reps

    n_pages = 2048   # 4 GiB: larger than L2 many times over
    for label, ratio in (("hbm_only", 0.0), ("1/%d" % modulus, 1.0 / modulus), ("1/%d" % max(2, modulus // 2), 1.0 / max(2, modulus // 2))):
        buf = TieredBuffer(n_pages * B.PAGE_BYTES, ratio, B.POLICY_MODULO, device=dev, peer_device=1)
        ws_bytes = B.boost_stream_reduce_workspace_bytes(n_pages)
        ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
        sums = torch.zeros(n_pages, dtype=torch.float32, device=dev)
        us = time_us(lambda: B.boost_stream_reduce_tiered(buf.page_ptr, buf.order, n_pages, buf.n_host, sums, ws, ws_bytes), 5)
        out["stream"].append({"placement": label, "peer_pages": buf.n_host, "us": us, "gbs": n_pages * B.PAGE_BYTES / us / 1e3,
                              "status": int(ws[:4].cpu().numpy().view(np.uint32)[0])})
        del buf
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    for name, (n, k) in {"gate_up": (28672, 4096), "lm_head": (128256, 4096)}.items():
        n_copies = max(2, int(np.ceil(2 * 126e6 / (n * k * 2))))
        for label, ratio in (("hbm_only", 0.0), ("1/%d" % modulus, 1.0 / modulus)):
            ws_ = [TieredWeight((0.02 * torch.randn(n, k, generator=g, device=dev)).to(torch.bfloat16), ratio, device=dev, peer_device=1)
                   for _ in range(n_copies)]
            for mb in (1, 32, 128):
                x = torch.randn(mb, k, generator=g, device=dev).to(torch.bfloat16)
                y = torch.empty(mb, n, dtype=torch.bfloat16, device=dev)
                for sched in ((0, 1) if ratio else (0,)):
                    B.boost_gemv_set_tier_schedule(sched)

                    def all_copies():
                        for w in ws_:
                            w.gemv(x, y=y)
                    us = time_us(all_copies, 5) / n_copies
                    out["weight_products"].append({"matrix": name, "batch": mb, "placement": label, "peer_pages": ws_[0].buf.n_host,
                                                   "schedule": "two queues" if sched else "in place", "us": us,
                                                   "gbs": ws_[0].layout["bytes"] / us / 1e3, "status": ws_[0].status_words()})
                B.boost_gemv_set_tier_schedule(0)
            del ws_
            torch.cuda.empty_cache()
    print(json.dumps(out))


def run_stream_sweep(args):
    """Configuration 3: tiered streaming-read sweep.  A bf16 buffer of 1 / 4 / 16 (/ 64) GiB is
    reduced by the stream-reduce kernel (full waves of 4 threadblocks per SM) with the host
    share in {0, 1/256, ..., 1/8} under modulo, contiguous and random placement.  Prints one
    JSON document with combined GB/s and the per-wave host-share statistics of each point."""
    import torch
    from paper_2609_13592_b200 import binding as B
    from paper_2609_13592_b200 import build as libbuild
    from paper_2609_13592_b200.tiers import Slabs, TieredBuffer
    libbuild.build_library()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    hbm_peak, peak_src = load_peaks()
    link = measure_stream(dev, 64, 1)
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    ratios = [0.0, 1 / 256, 1 / 128, 1 / 64, 1 / 32, 1 / 16, 1 / 8]
    policies = [("modulo", B.POLICY_MODULO), ("contiguous", B.POLICY_CONTIGUOUS), ("random", B.POLICY_RANDOM)]
    if args.sweep_ratios:     # a subset, for a profiler capture of single points
        ratios = [float(x) for x in args.sweep_ratios.split(",")]
    if args.sweep_policies:
        policies = [pp for pp in policies if pp[0] in args.sweep_policies.split(",")]
    sizes = [int(x) for x in args.sweep_gib.split(",")]
    points = []
    checked_points = 0
    from paper_2609_13592_b200 import synth
    page_elems = B.PAGE_BYTES // 2
    for gib in sizes:
        n_pages = gib * 512
        slabs = Slabs(n_pages, n_pages // 8 + n_pages // 32 + 8, dev)
        ws_bytes = B.boost_stream_reduce_workspace_bytes(n_pages)
        ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=dev)
        sums = torch.zeros(n_pages, dtype=torch.float32, device=dev)
        # The 1 GiB points are checked: the buffer holds the integer fill of the synthetic generator
        # (values in [-4, 4], so fp32 page sums are exact) and every page sum must equal the integer
        # sum of the generator's values for that page, bit for bit, under every placement.
        check = gib == 1
        if check:
            flat = synth.small_int_bf16_torch(0, n_pages * page_elems, dev)
            want = torch.from_numpy(synth.small_int_values(0, n_pages * page_elems).reshape(n_pages, page_elems)
                                    .sum(axis=1).astype(np.float32)).to(dev)
        log = torch.zeros(B.boost_schedule_log_bytes(16 * n_pages), dtype=torch.uint8, device=dev) if gib <= 16 else None
        for ratio in ratios:
            for name, pol in policies:
                seeds = range(args.sweep_seeds) if (pol == B.POLICY_RANDOM and ratio > 0) else [0]
                gbs, var = [], []
                n_host = 0
                realised = None
                for seed in seeds:
                    buf = TieredBuffer(n_pages * B.PAGE_BYTES, ratio, pol, seed=seed, device=dev, slabs=slabs)
                    n_host = buf.n_host
                    st = B.boost_wave_stats(buf.tier, 128 * 1024, sms * 4, ratio)
                    best = float("inf")
                    for i in range(5):
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record()
                        B.boost_stream_reduce_tiered(buf.page_ptr, buf.order, n_pages, buf.n_host, sums, ws, ws_bytes)
                        e1.record()
                        torch.cuda.synchronize(dev)
                        if i >= 1:
                            best = min(best, e0.elapsed_time(e1))
                    gbs.append(n_pages * B.PAGE_BYTES / best / 1e6)
                    var.append(st["var"])
                    if check and seed == 0:
                        buf.scatter_from(flat)
                        B.boost_stream_reduce_tiered(buf.page_ptr, buf.order, n_pages, buf.n_host, sums, ws, ws_bytes)
                        torch.cuda.synchronize(dev)
                        if not torch.equal(sums, want):
                            raise SystemExit(f"stream_sweep: page sums differ at ratio {ratio}, placement {name}")
                        checked_points += 1
                    if log is not None and seed == 0 and ratio > 0:
                        # one more launch with the schedule log attached: the host share the queues realise,
                        # per wave of tile starts and per 10 us of the run (address order: st above)
                        log.zero_()
                        log[:32].view(torch.int64)[1] = 16 * n_pages
                        ws[:64].view(torch.int64)[B.WS_LOG_WORD // 2] = log.data_ptr()
                        B.boost_stream_reduce_tiered(buf.page_ptr, buf.order, n_pages, buf.n_host, sums, ws, ws_bytes)
                        torch.cuda.synchronize(dev)
                        ws[:64].view(torch.int64)[B.WS_LOG_WORD // 2] = 0
                        w_st, t_st, n_rec = B.boost_schedule_stats(log.cpu().numpy(), B.SCHED_KIND_STREAM, sms * 4, 10_000, ratio)
                        realised = {"records": n_rec, "per_wave_of_starts": w_st, "per_10us_window": t_st}
                    del buf
                bound = min(hbm_peak + link, link / ratio * 1.0) if ratio > 0 else hbm_peak
                points.append({"gib": gib, "host_ratio": ratio, "placement": name, "host_pages": n_host,
                               "combined_gbs": float(np.mean(gbs)), "gbs_min": float(min(gbs)),
                               "gbs_max": float(max(gbs)), "wave_host_share_var": float(np.mean(var)),
                               "tier_bound_gbs": bound, "seeds": len(list(seeds)), "realised_schedule": realised})
        del slabs, ws, sums
        torch.cuda.empty_cache()
    print(json.dumps({"workload": "c3_tiered_stream_sweep", "hbm_peak_gbs": hbm_peak, "hbm_peak_source": peak_src,
                      "host_link_gbs": link, "combined_roofline_gbs": hbm_peak + link,
                      "points_with_page_sums_verified": checked_points, "points": points}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--ctx", type=int, default=2048)
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (0 = 32)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="decode", choices=["decode", "stream_sweep", "kv_spill", "gemv_sweep", "pool_churn", "peer_tier", "oracle_configs"],
                    help="decode: the benchmark line; stream_sweep: the placement sweep of configuration 3; "
                         "kv_spill: configuration 5 (batch 128, one KV page in five on the host) with its "
                         "HBM-only and prefetch-to-HBM comparison runs; gemv_sweep: weight products over shapes, "
                         "batch sizes and host shares; pool_churn: the KV pool under serving-like arrivals, realised host "
                         "share over time and attention timed on churned against fresh layouts; peer_tier: the second tier in a peer GPU's HBM "
                         "over NVLink (needs two GPUs in one process); oracle_configs (with --impl reference): the CPU oracle timed on "
                         "configurations 1 - 3")
    ap.add_argument("--churn-steps", type=int, default=12000, help="pool_churn: decode steps replayed")
    ap.add_argument("--sweep-gib", default="1,4,16")
    ap.add_argument("--sweep-seeds", type=int, default=20)
    ap.add_argument("--sweep-ratios", default="", help="stream_sweep: comma-separated host shares (default: the full list)")
    ap.add_argument("--sweep-policies", default="", help="stream_sweep: subset of modulo,contiguous,random")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.workload == "kv_spill":
        if rank == 0:
            run_kv_spill(args)
    elif args.workload == "gemv_sweep":
        if rank == 0:
            run_gemv_sweep(args)
    elif args.workload == "pool_churn":
        if rank == 0:
            run_pool_churn(args)
    elif args.workload == "stream_sweep":
        if rank == 0:
            run_stream_sweep(args)
    elif args.workload == "peer_tier":
        if rank == 0:
            run_peer_tier(args)
    elif args.impl == "reference" and args.workload == "oracle_configs":
        if rank == 0:
            run_reference_configs(args)
    elif args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
