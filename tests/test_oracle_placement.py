"""Pins for the placement oracle: values the paper prints, closed forms, brute force."""
import math
import random
from fractions import Fraction

import pytest

from oracle import placement as op
from tests.helpers import load_paper_values

PAPER = load_paper_values()
MIB = 1 << 20


def test_paper_worked_example_alpha_10_percent():
    # Sec. 3.1: K = 1/alpha = 10 HBM pages then one host page: period 11.
    period = op.modulus_from_bandwidths(10, 1)
    assert period == PAPER["mpp_period_pages_at_alpha_10pct"]
    tier = op.place_pages(period * op.PAGE_BYTES, 1.0 / period)
    assert tier == [0] * 10 + [1]
    share = Fraction(sum(tier), len(tier))
    # the host share of such a period is the proportional share alpha/(1+alpha) = 9.1 %
    assert share == Fraction(1, 10) / (1 + Fraction(1, 10))
    assert round(100 * float(share), 1) == PAPER["proportional_share_percent_at_alpha_10pct"]
    # Sec. 2.5: (1+alpha)/(1-alpha) advantage over a perfect prefetcher
    assert round(100 * (1.1 / 0.9 - 1)) == PAPER["prefetch_advantage_percent_at_alpha_10pct"]


def test_paper_evaluation_modulus_12():
    m = int(PAPER["eval_placement_modulus"])
    assert op.modulus_from_ratio(1.0 / m) == m
    tier = op.place_pages(10 * m * op.PAGE_BYTES, 1.0 / m)
    assert round(100.0 * sum(tier) / len(tier), 1) == PAPER["eval_host_share_percent"]
    # measured GH200 bandwidths (Sec. 5.1) give the ideal gain and K
    assert abs(100 * 350 / 3330 - PAPER["ideal_gain_percent_gh200"]) < 0.2
    assert op.modulus_from_bandwidths(3330, 350) == 11  # ceil(9.51) + 1


def test_config1_table():
    # 4096 x 4096 bf16 = 32 MiB = 16 pages, host_ratio 1/16 -> only the last page on the host
    tier = op.place_pages(4096 * 4096 * 2, 1.0 / 16)
    assert len(tier) == 16 and tier == [0] * 15 + [1]


def test_modulus_roundtrip_all_small_moduli():
    for m in range(2, 4097):
        assert op.modulus_from_ratio(1.0 / m) == m, m


def test_modulus_rounding_rule_never_exceeds_request():
    # Sec. 4.4: rounding up keeps the host fraction at or below the target
    rng = random.Random(7)
    for _ in range(2000):
        r = rng.uniform(1e-4, 0.5)
        m = op.modulus_from_ratio(r)
        assert Fraction(1, m) <= Fraction(r) * (1 + Fraction(1, 2 ** 40))
        assert m == 1 or Fraction(1, m - 1) > Fraction(r) * (1 + Fraction(1, 2 ** 40))
    assert op.modulus_from_ratio(0.0) == 0
    for bad in (-0.1, 0.6, 1e-12):
        with pytest.raises(ValueError):
            op.modulus_from_ratio(bad)


def test_modulo_brute_force_small():
    # independent statement: page i (1-based count) is host iff its group count is a multiple of M
    for p in range(0, 65):
        for m in range(2, 20):
            for s in (1, 2, 3, 7):
                tier = op.place_pages(p * op.PAGE_BYTES, 1.0 / m, op.POLICY_MODULO, 0, s)
                want = [1 if ((i // s) + 1) % m == 0 else 0 for i in range(p)]
                assert tier == want
                if s == 1:
                    assert sum(tier) == p // m


def test_partial_last_page_counts():
    assert op.n_pages(1) == 1
    assert op.n_pages(op.PAGE_BYTES) == 1
    assert op.n_pages(op.PAGE_BYTES + 1) == 2
    assert len(op.place_pages(5 * op.PAGE_BYTES + 17, 0.25)) == 6
    assert op.place_pages(0, 0.25) == []


def test_exact_ratio_in_every_window():
    # Insight 1 (Sec. 3.1): every wave sees the exact ratio.  Any window of W groups
    # holds floor(W/M) or ceil(W/M) host groups, exactly W/M when M divides W.
    for m in (2, 5, 11, 12, 16):
        tier = op.place_pages(40 * m * op.PAGE_BYTES, 1.0 / m)
        for w in (1, m - 1, m, m + 1, 2 * m, 3 * m + 2):
            for start in range(0, len(tier) - w):
                c = sum(tier[start:start + w])
                assert c in (w // m, -(-w // m))
                if w % m == 0:
                    assert c == w // m


def test_zero_ratio_and_restart_per_tensor():
    assert sum(op.place_pages(100 * op.PAGE_BYTES, 0.0)) == 0
    # stateless: two tensors get the same table, the pattern restarts (Sec. 3.1)
    a = op.place_pages(30 * op.PAGE_BYTES, 1 / 12)
    b = op.place_pages(30 * op.PAGE_BYTES, 1 / 12)
    assert a == b and a[:12] == [0] * 11 + [1]
    # a tensor shorter than one period gets no host page: its share stays <= target
    assert sum(op.place_pages(11 * op.PAGE_BYTES, 1 / 12)) == 0


def test_contiguous_is_tail_and_iso_bytes():
    for p in (1, 12, 37, 512):
        for m in (2, 8, 12):
            lin = op.place_pages(p * op.PAGE_BYTES, 1.0 / m, op.POLICY_CONTIGUOUS)
            mod = op.place_pages(p * op.PAGE_BYTES, 1.0 / m, op.POLICY_MODULO)
            assert sum(lin) == sum(mod) == p // m
            assert lin == sorted(lin)  # HBM head, host tail (Sec. 4.2)


def test_contiguous_waves_go_from_all_hbm_to_all_host():
    # Sec. 5.7: early waves hit HBM only, late waves the host only
    tier = op.place_pages(512 * op.PAGE_BYTES, 1 / 8, op.POLICY_CONTIGUOUS)
    st = op.wave_stats(tier, op.PAGE_BYTES // 8, 8 * 16, 1 / 8)  # a wave = 16 pages
    assert st["n_waves"] == 32 and st["n_zero_waves"] == 28 and st["n_over_waves"] == 4
    assert st["min"] == 0.0 and st["max"] == 1.0
    assert abs(st["mean"] - 1 / 8) < 1e-15


def test_modulo_waves_have_zero_variance():
    for m in (8, 12, 16):
        tier = op.place_pages(20 * m * op.PAGE_BYTES, 1.0 / m)
        st = op.wave_stats(tier, op.PAGE_BYTES // 4, 4 * 2 * m, 1.0 / m)  # a wave = 2 periods
        assert st["var"] == 0.0 and st["n_zero_waves"] == 0 and st["n_over_waves"] == 0
        assert abs(st["mean"] - 1.0 / m) < 1e-15 and st["min"] == st["max"]


def test_wave_stats_last_wave_short_and_errors():
    tier = [0, 1, 0, 1, 1]
    st = op.wave_stats(tier, op.PAGE_BYTES, 2, 0.5)
    # waves: [0,1] -> 1/2, [0,1] -> 1/2, [1] -> 1
    assert st["n_waves"] == 3 and st["n_over_waves"] == 1 and st["n_zero_waves"] == 0
    assert abs(st["mean"] - (0.5 + 0.5 + 1.0) / 3) < 1e-15
    mean = (0.5 + 0.5 + 1.0) / 3
    assert abs(st["var"] - ((0.5 - mean) ** 2 * 2 + (1 - mean) ** 2) / 3) < 1e-15
    with pytest.raises(ValueError):
        op.wave_stats(tier, 3000, 2, 0.5)


def test_mix64_matches_published_splitmix64_vectors():
    # first outputs of SplitMix64 seeded with 0 (public-domain reference generator)
    assert op.mix64(0, 0) == 0xE220A8397B1DCDAF
    assert op.mix64(0, 1) == 0x6E789E6AA1B965F4
    assert op.mix64(0, 2) == 0x06C45D188009454F


def test_random_placement_statistics_match_paper_spread():
    # Sec. 2.6: 10 % +- 1.5 % over whole kernels of hundreds of pages, and
    # 10 % +- 3.6 % within a wave; both are what an i.i.d. draw gives.
    m = 10
    p = 512
    shares = []
    for seed in range(100):
        tier = op.place_pages(p * op.PAGE_BYTES, 1.0 / m, op.POLICY_RANDOM, seed)
        shares.append(sum(tier) / p)
    mean = sum(shares) / len(shares)
    sd = math.sqrt(sum((s - mean) ** 2 for s in shares) / len(shares))
    assert abs(mean - 0.1) < 0.005
    assert 0.7 * PAPER["bappr_kernel_spread_percent"] < 100 * sd < 1.2 * PAPER["bappr_kernel_spread_percent"]
    # a wave that spans about 70 pages shows the per-wave spread the paper prints
    pages_per_wave = 70
    tier = op.place_pages(2000 * pages_per_wave * op.PAGE_BYTES, 1.0 / m, op.POLICY_RANDOM, 3)
    st = op.wave_stats(tier, op.PAGE_BYTES, pages_per_wave, 1.0 / m)
    assert st["n_waves"] == 2000
    assert abs(100 * math.sqrt(st["var"]) - PAPER["bappr_wave_spread_percent"]) < 0.3
    assert abs(st["var"] - 0.1 * 0.9 / pages_per_wave) < 2e-4  # binomial closed form
    # different seeds give different tables, same seed the same table
    assert op.place_pages(64 * op.PAGE_BYTES, 0.1, op.POLICY_RANDOM, 1) != \
        op.place_pages(64 * op.PAGE_BYTES, 0.1, op.POLICY_RANDOM, 2)


def test_superpage_example_from_paper():
    # Sec. 4.4: a CTA footprint of 3.5 MB against 2 MB pages -> superpage LCM = 14 MB = 7 pages;
    # Sec. 2.6: a page holds 73 of the 28 KB columns, the footprint spans 1.75 pages.
    foot_kib = int(PAPER["superpage_cta_footprint_mb"] * 1024)
    page_kib = 2048
    assert math.lcm(foot_kib, page_kib) == PAPER["superpage_lcm_mb"] * 1024
    s = math.lcm(foot_kib, page_kib) // page_kib
    assert s == 7
    assert (2 * MIB) // (28 * 1024) == PAPER["columns_per_page_down_proj"]
    assert foot_kib / page_kib == PAPER["cta_footprint_pages_down_proj"]
    tier = op.place_pages(7 * 24 * op.PAGE_BYTES, 1 / 12, op.POLICY_MODULO, 0, s)
    n_foot = len(tier) * page_kib // foot_kib
    for f in range(n_foot):  # no CTA footprint is split across tiers (Sec. 3.2)
        first = f * foot_kib // page_kib
        last = ((f + 1) * foot_kib - 1) // page_kib
        assert len({tier[i] for i in range(first, last + 1)}) == 1
    # without superpages some footprint is split
    plain = op.place_pages(7 * 24 * op.PAGE_BYTES, 1 / 12)
    split = 0
    for f in range(n_foot):
        first = f * foot_kib // page_kib
        last = ((f + 1) * foot_kib - 1) // page_kib
        split += len({plain[i] for i in range(first, last + 1)}) > 1
    assert split > 0
    # host share across superpages still bounded by the target
    assert Fraction(sum(tier), len(tier)) <= Fraction(1, 12)


def test_tier_order():
    tier = op.place_pages(50 * op.PAGE_BYTES, 1 / 8, op.POLICY_RANDOM, 5)
    order, n_host = op.tier_order(tier)
    assert sorted(order) == list(range(50)) and n_host == sum(tier)
    assert all(tier[i] == 1 for i in order[:n_host]) and all(tier[i] == 0 for i in order[n_host:])
    assert order[:n_host] == sorted(order[:n_host]) and order[n_host:] == sorted(order[n_host:])


def test_schedule_stats_closed_forms():
    """The realised-schedule statistics on logs whose answer is known by construction."""
    K = 2          # kind
    # 12 items of 100 bytes, one after the other on one warp, every 4th from the host tier
    recs = [(K, 0, 100, 100 if i % 4 == 3 else 0, 1000 * i, 1000 * (i + 1)) for i in range(12)]
    waves, windows, n = op.schedule_stats(recs, 4, 1000, 0.25)
    assert n == 12 and waves["n_waves"] == 3 and waves["n_host_pages"] == 3
    assert waves["mean"] == 0.25 and waves["var"] == 0.0 and waves["min"] == waves["max"] == 0.25
    assert waves["n_zero_waves"] == 0 and waves["n_over_waves"] == 0
    # windows of one item each: share 1 in the host items' windows, 0 elsewhere
    assert windows["n_waves"] == 12 and windows["n_zero_waves"] == 9 and windows["max"] == 1.0 and windows["mean"] == 0.25
    # windows of four items: exactly the target everywhere ("exact ratio at every wave", Sec. 3.1)
    _, windows, _ = op.schedule_stats(recs, 4, 4000, 0.25)
    assert windows["n_waves"] == 3 and windows["min"] == windows["max"] == 0.25 and windows["var"] == 0.0
    # contiguous hand-out (host items last): waves 0, 0, 3/4 -> one over the target, two without host work
    recs_c = [(K, 0, 100, 100 if i >= 9 else 0, 1000 * i, 1000 * (i + 1)) for i in range(12)]
    waves, _, _ = op.schedule_stats(recs_c, 4, 1000, 0.25)
    assert (waves["n_zero_waves"], waves["n_over_waves"], waves["max"]) == (2, 1, 0.75)
    assert abs(waves["var"] - (2 * 0.25 ** 2 + 0.5 ** 2) / 3) < 1e-15
    # a host item that streams for the whole kernel beside eight HBM items: every window sees both tiers
    recs_p = [(K, 0, 800, 800, 0, 8000)] + [(K, 1, 100, 0, 1000 * i, 1000 * (i + 1)) for i in range(8)]
    _, windows, _ = op.schedule_stats(recs_p, 3, 1000, 0.5)
    assert windows["n_waves"] == 8 and windows["min"] == windows["max"] == 0.5
    # an item across a window boundary is split by time: 300 bytes over [500, 2000) -> 100 | 200
    _, windows, _ = op.schedule_stats([(K, 0, 300, 300, 500, 2000), (K, 1, 100, 0, 500, 1500)], 1, 1000, 1.0)
    # window 0 = [500, 1500): host 200, hbm 100; window 1 = [1500, 2500): host 100, hbm 0
    assert windows["n_waves"] == 2 and abs(windows["min"] - 2 / 3) < 1e-15 and windows["max"] == 1.0
    # filters: other kinds, unfinished and empty records do not count; ties ordered by cta_warp
    noisy = recs + [(3, 0, 100, 100, 0, 10), (K, 5, 100, 100, 50, 0), (K, 6, 0, 0, 60, 70)]
    assert op.schedule_stats(noisy, 4, 1000, 0.25, kind=K)[2] == 12
    a = op.schedule_stats([(K, 2, 10, 10, 7, 9), (K, 1, 10, 0, 7, 9), (K, 3, 10, 0, 8, 9), (K, 0, 10, 0, 8, 9)], 2, 10, 0.5)[0]
    assert (a["n_waves"], a["min"], a["max"]) == (2, 0.0, 0.5)
    with pytest.raises(ValueError):
        op.schedule_stats(recs, 0, 1000, 0.25)
