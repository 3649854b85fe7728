"""Replay of a serving-like allocation trace on a KV pool (plumbing for the churn workload).

The trace (synth.serving_churn_trace) says which request asks for how many blocks and which
request finishes at every decode step; the pool decides which blocks are handed out.  This
module applies the calls, remembers each request's blocks and, at chosen steps, returns the
batch as the attention kernel takes it (block table and context lengths).  The pool object
needs alloc(request, n) -> block ids, free(request) and query(); nothing of the pool's policy
is computed here.
"""
import numpy as np


def replay_churn(pool, trace, snapshot_steps=()):
    """Apply `trace` to `pool`.  Returns (shares, batch_sizes, live_blocks, snapshots, stats): the
    host share of the live KV chunks, the number of running requests and the number of blocks
    in use after every step, and for each step in snapshot_steps a dict(step, requests,
    ctx_lens int32 [B], table int32 [B, max_blocks], info = pool.query())."""
    snapshot_steps = set(int(s) for s in snapshot_steps)
    blocks = {}
    shares, batch_sizes, live_blocks, snapshots = [], [], [], []
    stats = {}
    for step, (ops, live, stats) in enumerate(trace):
        for op in ops:
            if op[0] == "alloc":
                got = pool.alloc(op[1], op[2])
                blocks.setdefault(op[1], []).extend(int(b) for b in got)
            else:
                pool.free(op[1])
                del blocks[op[1]]
        q = pool.query()
        shares.append(q["live_host_chunks"] / q["live_chunks"] if q["live_chunks"] else 0.0)
        batch_sizes.append(len(live))
        live_blocks.append(q["live_blocks"])
        if step in snapshot_steps and live:
            reqs = sorted(live)
            ctx = np.array([live[r] for r in reqs], dtype=np.int32)
            need = (ctx.astype(np.int64) + 15) // 16
            table = np.zeros((len(reqs), int(need.max())), dtype=np.int32)
            for i, r in enumerate(reqs):
                assert len(blocks[r]) == need[i]
                table[i, :need[i]] = blocks[r]
            snapshots.append({"step": step, "requests": reqs, "ctx_lens": ctx, "table": table, "info": q})
    return np.array(shares), np.array(batch_sizes), np.array(live_blocks), snapshots, stats


def fresh_tables(pool, ctx_lens):
    """Block table of the same batch on an unused pool: the requests grow one block at a time in
    turn (the allocation pattern of a batch that starts together)."""
    need = (np.asarray(ctx_lens, dtype=np.int64) + 15) // 16
    table = np.zeros((len(need), int(need.max())), dtype=np.int32)
    for j in range(int(need.max())):
        for i in range(len(need)):
            if j < need[i]:
                table[i, j] = int(pool.alloc(i, 1)[0])
    return table


def host_kv_bytes(table, ctx_lens, info, head_dim=128):
    """(bytes read from host pages, bytes read in total) by one attention launch over the batch:
    every cached token of every KV head is read once from K and once from V (2 bytes per
    element); a block below info["first_hi_block"] has info["host_heads_lo"] heads on the host,
    a block from there on one more."""
    ctx = np.asarray(ctx_lens, dtype=np.int64)
    need = (ctx + 15) // 16
    cols = np.arange(table.shape[1], dtype=np.int64)[None, :]
    tokens = np.clip(ctx[:, None] - 16 * cols, 0, 16) * (cols < need[:, None])
    host_heads = info["host_heads_lo"] + (table >= info["first_hi_block"]).astype(np.int64)
    per_token_head = 2 * head_dim * 2
    return int((tokens * host_heads).sum()) * per_token_head, int(tokens.sum()) * info["n_kv_heads"] * per_token_head
