"""Pins for the KV-pool oracle: the paper's ratios and bounds, invariants over
random and exhaustive traces, and the boundary conditions of Sec. 4.3."""
import itertools
import random
from fractions import Fraction

import pytest

from oracle import kv_pool as kp
from tests.helpers import load_paper_values

PAPER = load_paper_values()


def static_host_share(pool):
    host = sum(pool.host_heads(b) for b in range(pool.n_blocks))
    return Fraction(host, pool.n_blocks * pool.n_kv_heads)


def check_invariants(pool):
    q = pool.query()
    assert q["free_lo"] + q["free_hi"] + q["live_blocks"] == pool.n_blocks     # conserved count
    live = [b for blocks in pool.requests.values() for b in blocks]
    assert len(live) == len(set(live))                                        # no double allocation
    free = list(pool.free[kp.KIND_LO]) + list(pool.free[kp.KIND_HI])
    assert len(free) == len(set(free)) and not (set(free) & set(live))
    assert all(0 <= b < pool.n_blocks for b in live + free)
    assert all(pool.kind[b] == kp.KIND_LO for b in pool.free[kp.KIND_LO])
    assert all(pool.kind[b] == kp.KIND_HI for b in pool.free[kp.KIND_HI])


def test_few_heads_example_from_paper():
    # Sec. 4.3: four KV heads, one head on the host tier -> 25 % of KV accesses
    pool = kp.KVPool(512, 4, 4)
    assert 100 * static_host_share(pool) == PAPER["few_heads_host_share_percent"]
    assert all(pool.host_heads(b) == 1 for b in range(512))
    assert all(pool.chunk_tier(3, b) == 1 and pool.chunk_tier(0, b) == 0 for b in range(512))


def test_block_kind_ratio_H_to_M_minus_H():
    # Sec. 4.3: single-head-host : all-local = H : M - H, host share 1/M
    for h, m, n in ((4, 12, 1536), (8, 16, 1024), (8, 8, 512), (2, 10, 2560), (8, 12, 1536)):
        pool = kp.KVPool(n, h, m)
        n_hi = sum(1 for k in pool.kind if k == kp.KIND_HI)
        if m == h:
            assert pool.k_lo == 1 and n_hi == 0
        else:
            assert pool.k_lo == 0
            assert Fraction(n_hi, n - n_hi) == Fraction(h, m - h)
        assert static_host_share(pool) == Fraction(1, m)
        # hi blocks are exactly those whose address falls in the linear tail (Sec. 4.2)
        assert pool.kind == sorted(pool.kind)


def test_more_heads_than_modulus_mixes_floor_and_ceil():
    # Sec. 4.5: H > M -> blocks with floor(H/M) and ceil(H/M) host heads
    pool = kp.KVPool(2560, 8, 5)
    counts = {pool.host_heads(b) for b in range(2560)}
    assert counts == {8 // 5, -(-8 // 5)}
    assert static_host_share(pool) == Fraction(1, 5)
    assert pool.kind.index(kp.KIND_HI) == 1024      # head 6 is on the host from 0.4 N on
    pool = kp.KVPool(512, 8, 2)
    assert {pool.host_heads(b) for b in range(512)} == {4}
    assert static_host_share(pool) == Fraction(1, 2)


def test_no_host_and_bad_geometry():
    pool = kp.KVPool(512, 8, 0)
    assert static_host_share(pool) == 0 and pool.query()["free_hi"] == 0
    for args in ((500, 8, 8), (0, 8, 8), (512, 0, 8), (512, 8, 1), (512, 8, -2)):
        with pytest.raises(kp.PoolError):
            kp.KVPool(*args)


def test_request_share_bounded_by_one_over_H():
    # Sec. 4.5: the host access ratio is at most 1/H even under maximum imbalance (M >= H)
    pool = kp.KVPool(1536, 4, 12)
    rng = random.Random(1)
    rid = 0
    for _ in range(300):
        if pool.requests and rng.random() < 0.4:
            pool.free_request(rng.choice(list(pool.requests)))
        else:
            try:
                pool.alloc(rid, rng.randint(1, 200))
                rid += 1
            except kp.PoolError as e:
                assert e.code == kp.ERR_NOMEM
        for blocks in pool.requests.values():
            host = sum(pool.host_heads(b) for b in blocks)
            assert Fraction(host, len(blocks) * 4) <= Fraction(1, 4)
        check_invariants(pool)


def test_greedy_rule_and_shared_kind():
    # Sec. 4.3: a new request gets the host-heavy kind iff its free share exceeds the target share
    pool = kp.KVPool(1536, 4, 12)        # 512 hi, 1024 lo; target hi share 1/3
    a = pool.alloc("a", 10)              # free hi share is exactly 1/3: not above -> lo
    assert pool.request_kind["a"] == kp.KIND_LO and a == list(range(10))
    b = pool.alloc("b", 10)              # now hi share 512/1526 > 1/3 -> hi
    assert pool.request_kind["b"] == kp.KIND_HI and b == list(range(1024, 1034))
    # all blocks of a request share one kind, later calls included
    assert pool.alloc("a", 5) == list(range(10, 15))
    assert pool.alloc("b", 5) == list(range(1034, 1039))
    check_invariants(pool)


def test_fifo_and_free_order():
    pool = kp.KVPool(512, 8, 8)
    a = pool.alloc(1, 3)
    b = pool.alloc(2, 2)
    assert a == [0, 1, 2] and b == [3, 4]
    pool.free_request(1)
    assert list(pool.free[kp.KIND_LO])[-3:] == [0, 1, 2]
    assert pool.alloc(3, 2) == [5, 6]
    with pytest.raises(kp.PoolError) as e:
        pool.free_request(1)                      # second free
    assert e.value.code == kp.ERR_INVALID
    with pytest.raises(kp.PoolError):
        pool.alloc(4, 0)


def test_boundary_hi_list_empty_falls_back_to_local():
    # Sec. 4.3: when the single-head-host list empties, requests get all-local blocks
    pool = kp.KVPool(1536, 4, 12)
    pool.alloc("warm", 1)                          # lo (tie)
    got = pool.alloc("big", 512)                   # hi, drains the hi list
    assert all(pool.kind[b] == kp.KIND_HI for b in got) and pool.query()["free_hi"] == 0
    pool.alloc("next", 4)
    assert pool.request_kind["next"] == kp.KIND_LO
    more = pool.alloc("big", 3)                    # its list is empty: borrows lo and stays lo
    assert all(pool.kind[b] == kp.KIND_LO for b in more)
    assert pool.request_kind["big"] == kp.KIND_LO
    check_invariants(pool)


def test_boundary_lo_list_empty_borrow_is_sticky():
    # Sec. 4.3: when the all-local list empties, host-heavy blocks are appended to an
    # all-local request, which then keeps receiving that kind even after all-local
    # blocks become free again.
    pool = kp.KVPool(1536, 4, 12)                  # 1024 lo (0..1023), 512 hi (1024..1535)
    assert pool.alloc("y", 10) == list(range(10))  # tie -> lo
    pool.alloc("h", 6)                             # hi share 512/1526 > 1/3 -> hi
    assert pool.request_kind["h"] == kp.KIND_HI
    pool.alloc("a", 1000)                          # hi share 506/1520 < 1/3 -> lo
    assert pool.request_kind["a"] == kp.KIND_LO and pool.query()["free_lo"] == 14
    got = pool.alloc("a", 20)                      # 14 lo left, then borrows 6 hi
    assert [pool.kind[b] for b in got] == [kp.KIND_LO] * 14 + [kp.KIND_HI] * 6
    assert pool.request_kind["a"] == kp.KIND_HI
    pool.alloc("c", 5)                             # lo list empty: served from hi
    assert all(pool.kind[b] == kp.KIND_HI for b in pool.requests["c"])
    pool.free_request("y")                         # lo blocks 0..9 are free again
    assert pool.query()["free_lo"] == 10
    nxt = pool.alloc("a", 3)                       # sticky: still hi
    assert all(pool.kind[b] == kp.KIND_HI for b in nxt)
    check_invariants(pool)


def test_nomem_changes_nothing():
    pool = kp.KVPool(512, 8, 8)
    pool.alloc(1, 500)
    before = (list(pool.free[0]), list(pool.free[1]), dict(pool.request_kind),
              {k: list(v) for k, v in pool.requests.items()})
    with pytest.raises(kp.PoolError) as e:
        pool.alloc(2, 13)
    assert e.value.code == kp.ERR_NOMEM
    with pytest.raises(kp.PoolError):
        pool.alloc(1, 13)
    after = (list(pool.free[0]), list(pool.free[1]), dict(pool.request_kind),
             {k: list(v) for k, v in pool.requests.items()})
    assert before == after
    assert pool.alloc(2, 12) == list(range(500, 512))
    check_invariants(pool)


def test_exhaustive_short_traces_keep_invariants():
    # every trace of up to 3 operations over 3 request ids on a 1024-block pool
    # with large requests, so that both lists empty and borrow paths are taken
    ops = [("alloc", r, n) for r in range(3) for n in (200, 600)] + [("free", r, 0) for r in range(3)]
    n_traces = 0
    for length in range(1, 4):
        for trace in itertools.product(ops, repeat=length):
            pool = kp.KVPool(1024, 4, 8)
            for op, r, n in trace:
                try:
                    if op == "alloc":
                        got = pool.alloc(r, n)
                        assert len(got) == n
                    else:
                        pool.free_request(r)
                except kp.PoolError as e:
                    assert e.code in (kp.ERR_NOMEM, kp.ERR_INVALID)
            check_invariants(pool)
            n_traces += 1
    assert n_traces > 700


def test_churn_keeps_live_host_share_near_target():
    # Sec. 5.11: four KV heads, target one page in twelve (8.3 %): the realised share of
    # live KV chunks on the host stays within about a point of the target and far below 1/H.
    pool = kp.KVPool(12 * 1024, 4, 12)
    rng = random.Random(2024)
    live = {}
    shares = []
    rid = 0
    for step in range(4000):
        # arrivals: long generations, lengths spread over an order of magnitude
        if rng.random() < 0.5:                     # about 160 requests in flight
            want = rng.randint(8, 64)
            try:
                pool.alloc(rid, want)
                live[rid] = rng.randint(50, 600)   # remaining decode steps (x16 tokens/block/16)
                rid += 1
            except kp.PoolError:
                pass
        for r in list(live):
            live[r] -= 1
            if live[r] <= 0:
                pool.free_request(r)
                del live[r]
            elif rng.random() < 1 / 16:            # one new block every 16 tokens
                try:
                    pool.alloc(r, 1)
                except kp.PoolError:
                    pass
        q = pool.query()
        if step > 1500 and q["live_chunks"] > 0:
            shares.append(q["live_host_chunks"] / q["live_chunks"])
    check_invariants(pool)
    shares.sort()
    median = shares[len(shares) // 2]
    assert abs(100 * median - PAPER["eval_host_share_percent"]) < 1.0
    assert 100 * shares[0] > PAPER["dsr_realised_share_low_percent"] - 0.7
    assert 100 * shares[-1] < PAPER["dsr_realised_share_high_percent"] + 0.7
    assert shares[-1] < 1 / 4                      # the 1/H bound of Sec. 4.5
