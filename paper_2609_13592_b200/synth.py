"""Seeded synthetic inputs shaped like the paper's workloads.

Only generators live here: nothing of the method (placement, pool, kernels'
arithmetic) is computed in this module, so both the CPU oracle's tests and the
CUDA path can take their inputs from it.  bf16 tensors are numpy uint16 arrays
of raw bit patterns on the host and torch.bfloat16 tensors on the device.

The paper evaluates on FP8 70-80B checkpoints with synthetic input/output
lengths (Sec. 5.1) and on dataset traces; neither is available here, so the
generators reproduce shapes, value distributions and length mixes only:
weights N(0, 0.02^2), activations and KV N(0, 1), context lengths uniform in a
range, all from explicit seeds.
"""
import numpy as np

PAGE_BYTES = 2 * 1024 * 1024


def f32_to_bf16_bits(x):
    """float32 -> bf16 bit patterns, round to nearest even (input preparation)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(shape, std, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    return f32_to_bf16_bits(rng.standard_normal(shape, dtype=np.float32) * np.float32(std))


def ctx_lens_uniform(batch, lo, hi, seed):
    """Context lengths uniform in [lo, hi] (inclusive)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(lo, hi + 1, size=batch, dtype=np.int64)


def small_int_values(start, count):
    """Integer fill in [-4, 4] from a hash of the element index; sums of up to a
    page of these stay exact in fp32.  Returns int64 values."""
    i = np.arange(start, start + count, dtype=np.uint64)
    h = (i * np.uint64(2654435761)) & np.uint64(0xFFFFFFFF)
    return ((h >> np.uint64(13)) % np.uint64(9)).astype(np.int64) - 4


def small_int_bf16(start, count):
    return f32_to_bf16_bits(small_int_values(start, count).astype(np.float32))


def small_int_bf16_torch(start, count, device):
    """Same fill as small_int_bf16, produced on `device` as a torch.bfloat16 tensor."""
    import torch
    i = torch.arange(start, start + count, dtype=torch.int64, device=device)
    h = (i * 2654435761) & 0xFFFFFFFF
    return (((h >> 13) % 9) - 4).to(torch.bfloat16)


LLAMA3_8B = dict(n_layers=32, hidden=4096, ffn=14336, n_q_heads=32, n_kv_heads=8,
                 head_dim=128, vocab=128256)

TINY_LLAMA = dict(n_layers=2, hidden=256, ffn=512, n_q_heads=4, n_kv_heads=2,
                  head_dim=128, vocab=640)


def llama_weights(cfg, seed, std=0.02):
    """Random-init weights of a Llama-shaped model as bf16 bit patterns (numpy).
    Norm weights are 1 + N(0, 0.02^2) so that they matter in parity checks."""
    hq, hkv, d = cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    hid, ffn, vocab = cfg["hidden"], cfg["ffn"], cfg["vocab"]
    s = seed * 1000

    def norm_w(k):
        rng = np.random.Generator(np.random.PCG64(s + k))
        return f32_to_bf16_bits(1.0 + rng.standard_normal(hid, dtype=np.float32) * np.float32(std))

    w = {"embed": normal_bf16((vocab, hid), std, s + 1),
         "norm_f": norm_w(2),
         "lm_head": normal_bf16((vocab, hid), std, s + 3),
         "layers": []}
    for li in range(cfg["n_layers"]):
        b = s + 10 * (li + 1)
        w["layers"].append({
            "norm1": norm_w(b),
            "wqkv": normal_bf16(((hq + 2 * hkv) * d, hid), std, b + 1),
            "wo": normal_bf16((hid, hq * d), std, b + 2),
            "norm2": norm_w(b + 3),
            "wgu": normal_bf16((2 * ffn, hid), std, b + 4),
            "wd": normal_bf16((hid, ffn), std, b + 5),
        })
    return w


def serving_churn_trace(n_blocks, n_steps, arrivals_per_step, max_batch, seed, prompt_lo=64, prompt_hi=1024,
                        out_median=1500.0, out_sigma=0.8, out_cap=8192, block_tokens=16):
    """Allocation trace of a continuously batched decode server, one decode step at a time
    (a stand-in for the paper's serving runs with Poisson arrivals and a long-generation
    length mix, Sec. 5.8 and Sec. 5.11; shapes only, no dataset items).

    Arrivals per step are Poisson; a request has a prompt of U[prompt_lo, prompt_hi] tokens
    and generates a log-normal number of tokens (median out_median, log-sigma out_sigma,
    capped).  Waiting requests are admitted first come first served while fewer than
    max_batch are running and the pool has room for the prompt plus one block per running
    request; every running request grows by one token per step and needs a new block every
    block_tokens tokens; a request that cannot grow is dropped (counted).  Admission counts
    free blocks only, so the trace does not depend on which blocks a pool hands out.

    Yields, per step, (ops, live, stats): ops is the list of ("alloc", request, n_blocks) and
    ("free", request) calls of the step in order, live maps each running request to its
    context length after the step (the generator's own dict: read, do not change), stats
    counts arrivals, admissions, completions and drops so far."""
    rng = np.random.Generator(np.random.PCG64(seed))
    free = int(n_blocks)
    live, left, held = {}, {}, {}
    waiting = []
    next_id = 0
    stats = {"arrived": 0, "admitted": 0, "finished": 0, "dropped": 0}

    def blocks_of(tokens):
        return -(-tokens // block_tokens)

    for _ in range(n_steps):
        ops = []
        for _ in range(int(rng.poisson(arrivals_per_step))):
            prompt = int(rng.integers(prompt_lo, prompt_hi + 1))
            out = int(min(out_cap, max(1, round(float(rng.lognormal(np.log(out_median), out_sigma))))))
            waiting.append((prompt, out))
            stats["arrived"] += 1
        # completions of the previous step give their blocks back before anything is handed out
        for r in [r for r, n in left.items() if n <= 0]:
            ops.append(("free", r))
            free += held.pop(r)
            del live[r], left[r]
            stats["finished"] += 1
        # running requests take their next token
        for r in list(live):
            if live[r] % block_tokens == 0:
                if free == 0:
                    ops.append(("free", r))
                    free += held.pop(r)
                    del live[r], left[r]
                    stats["dropped"] += 1
                    continue
                ops.append(("alloc", r, 1))
                free -= 1
                held[r] += 1
            live[r] += 1
            left[r] -= 1
        # admissions: the prompt is cached and the first token generated in this step
        while waiting and len(live) < max_batch:
            prompt, out = waiting[0]
            need = blocks_of(prompt + 1)
            if free < need + len(live):
                break
            waiting.pop(0)
            r, next_id = next_id, next_id + 1
            ops.append(("alloc", r, need))
            free -= need
            held[r], live[r], left[r] = need, prompt + 1, out - 1
            stats["admitted"] += 1
        yield ops, live, dict(stats, waiting=len(waiting), free_blocks=free)
