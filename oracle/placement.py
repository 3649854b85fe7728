"""Oracle: page placement across the two tiers and per-wave host share.

Test infrastructure only (see the package docstring).  Pure Python integers and
fractions; no floating point decides an integer here.

What the paper fixes
  * a buffer is cut into 2 MiB pages (Sec. 1, Sec. 2.6);
  * modulo placement: with period M = K + 1 the first K pages of every period
    go to HBM and the (K+1)-th to the host tier (Sec. 1 "First, page
    placement", Sec. 3.1); alpha = 10 % gives K = 10 and a period of 11 pages
    (Sec. 3.1); the evaluation uses modulus 12, one page of twelve on the host,
    a share of 8.3 % (Sec. 5.1);
  * a non-integer 1/alpha is rounded up so that the host share never exceeds
    the request (Sec. 4.4);
  * superpages: contiguous groups of pages share one tier and the modulo rule
    runs across groups (Sec. 3.2, Sec. 4.4);
  * linear placement: the head of the range is HBM, the tail is host (Sec. 4.2);
  * random placement: every page is host-resident with the target probability,
    independently (Sec. 2.6; the i.i.d. reading matches the printed spread of
    10 % +- 1.5 % over kernels of hundreds of pages);
  * the pattern restarts for every tensor: the function keeps no state
    (Sec. 3.1, last paragraph).

Readings taken where the paper is silent are listed in the repository's design
notes; the ones that matter here: `host_ratio` is the share of ALL pages that
live on the host (1/M), the host residue is M-1, a trailing partial page counts
as a page, and linear placement uses the same host count as modulo placement so
the two compare at equal bytes.
"""
from fractions import Fraction

PAGE_BYTES = 2 * 1024 * 1024

TIER_HBM = 0
TIER_HOST = 1

POLICY_MODULO = 0
POLICY_CONTIGUOUS = 1
POLICY_RANDOM = 2

_MASK64 = (1 << 64) - 1
_RATIO_SLACK = Fraction(1, 2 ** 40)


def modulus_from_ratio(host_ratio):
    """Smallest period M whose host share 1/M does not exceed `host_ratio`.

    Sec. 4.4: K = ceil(1/alpha) keeps the host fraction at or below the target.
    Here the target is the share of all pages, so M = ceil(1/host_ratio).  A
    binary double cannot hold 1/12 exactly, so the comparison allows a relative
    slack of 2**-40; it is carried out in exact rational arithmetic.
    Returns 0 for host_ratio == 0 (no host pages).
    """
    r = Fraction(host_ratio)  # exact value of the double
    if r == 0:
        return 0
    if r < Fraction(1, 2 ** 30) or r > Fraction(1, 2):
        raise ValueError("host_ratio must be 0 or lie in [2**-30, 1/2]")
    bound = r * (1 + _RATIO_SLACK)
    # 1/M <= bound  <=>  M >= 1/bound, so M is the exact ceiling of 1/bound.
    inv = 1 / bound
    m = inv.numerator // inv.denominator
    if Fraction(m) < inv:
        m += 1
    return m


def modulus_from_bandwidths(hbm_bw, link_bw):
    """Period K + 1 with K = ceil(HBM bandwidth / link bandwidth).

    Sec. 3.1 defines K = 1/alpha as the HBM-to-host bandwidth ratio and Sec. 4.4
    rounds it up; K pages of HBM are followed by one host page.
    """
    ratio = Fraction(hbm_bw) / Fraction(link_bw)
    k = int(ratio)
    if Fraction(k) < ratio:
        k += 1
    return k + 1


def n_pages(n_bytes):
    """Pages covering n_bytes; a trailing partial page is a page."""
    return (int(n_bytes) + PAGE_BYTES - 1) // PAGE_BYTES


def mix64(seed, index):
    """Counter-based 64-bit hash (the SplitMix64 output function applied to
    seed + (index + 1) * golden-gamma).  Random placement draws from it so that
    any implementation can reproduce the same table from (seed, page index)."""
    z = (seed + (index + 1) * 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def place_pages(n_bytes, host_ratio, policy=POLICY_MODULO, seed=0, superpage_pages=1):
    """Tier of every 2 MiB page of a buffer of n_bytes -> list of 0 (HBM) / 1 (host)."""
    p = n_pages(n_bytes)
    m = modulus_from_ratio(host_ratio)
    s = int(superpage_pages)
    if s < 1:
        raise ValueError("superpage_pages must be >= 1")
    tier = [TIER_HBM] * p
    if m == 0:
        return tier
    if policy == POLICY_MODULO:
        # Sec. 3.1 / Sec. 4.4: K = M-1 groups to HBM, then one group to host.
        for i in range(p):
            group = i // s
            if group % m == m - 1:
                tier[i] = TIER_HOST
    elif policy == POLICY_CONTIGUOUS:
        # Sec. 4.2: the last part of the range is host; count as under MODULO
        # at page granularity so the comparison is at equal host bytes.
        n_host = p // m
        for i in range(p - n_host, p):
            tier[i] = TIER_HOST
    elif policy == POLICY_RANDOM:
        # Sec. 2.6: each page host with probability 1/M, independently.
        threshold = (1 << 64) // m
        for i in range(p):
            if mix64(seed, i) < threshold:
                tier[i] = TIER_HOST
    else:
        raise ValueError("unknown policy")
    return tier


def tier_order(tier):
    """Visit order used by tier-specialised kernels: host pages first (ascending),
    then HBM pages (ascending).  Sec. 3.2 keeps every CTA on one tier; starting
    the slow tier's pages first lets both tiers stream for the whole kernel.
    Returns (order, n_host)."""
    host = [i for i, t in enumerate(tier) if t == TIER_HOST]
    hbm = [i for i, t in enumerate(tier) if t != TIER_HOST]
    return host + hbm, len(host)


def wave_stats(tier, tile_bytes, ctas_per_wave, host_ratio):
    """Host share of every wave when tiles are handed out in address order.

    Sec. 2.2 defines a wave as the CTAs resident at once; Sec. 2.6 measures the
    spread of the host share across waves.  Tiles of `tile_bytes` (a divisor of
    the page size) are numbered in address order and wave w holds tiles
    [w*G, (w+1)*G); the last wave may be short (Sec. 4.4, last paragraph).
    """
    if tile_bytes <= 0 or PAGE_BYTES % tile_bytes != 0 or ctas_per_wave <= 0:
        raise ValueError("tile_bytes must divide the page size; ctas_per_wave > 0")
    tiles_per_page = PAGE_BYTES // tile_bytes
    n_tiles = len(tier) * tiles_per_page
    fractions = []
    for start in range(0, n_tiles, ctas_per_wave):
        stop = min(n_tiles, start + ctas_per_wave)
        host = sum(1 for t in range(start, stop) if tier[t // tiles_per_page] == TIER_HOST)
        fractions.append(Fraction(host, stop - start))
    target = Fraction(host_ratio)
    n = len(fractions)
    out = {
        "n_waves": n,
        "n_host_pages": sum(1 for t in tier if t == TIER_HOST),
        "n_zero_waves": sum(1 for f in fractions if f == 0),
        "n_over_waves": sum(1 for f in fractions if f > target * (1 + _RATIO_SLACK)),
        "mean": 0.0, "var": 0.0, "min": 0.0, "max": 0.0,
    }
    if n:
        mean = sum(fractions, Fraction(0)) / n
        var = sum(((f - mean) ** 2 for f in fractions), Fraction(0)) / n
        out.update(mean=float(mean), var=float(var),
                   min=float(min(fractions)), max=float(max(fractions)))
    return out


def schedule_stats(records, items_per_wave, window_ns, host_ratio, kind=0):
    """Host share per wave of work and per stretch of time, of a schedule a kernel realised.

    Sec. 2.6 and Sec. 3.1 judge a placement by the host share of every wave; with threadblocks
    specialised by tier (Sec. 3.2) the order in which work is handed out, not the address order,
    decides that share, so it is computed from a log of the run: `records` is a sequence of
    (kind_phase, cta_warp, bytes, host_bytes, t_request, t_consumed) tuples of integers.

    Waves: records ordered by (t_request, cta_warp, kind_phase) and cut into groups of
    items_per_wave consecutive starts; share = host bytes / bytes of the group.
    Windows: the time from the first request to the last consumption in windows of window_ns; a
    record's bytes are spread evenly over [t_request, max(t_consumed, t_request + 1)); share =
    host bytes / bytes that fall into the window; windows without traffic are left out.
    Unfinished (t_consumed == 0) and empty records are skipped; kind != 0 keeps only records
    whose kind_phase & 0xFF equals it.  Exact rational arithmetic.  Returns (waves, windows,
    n_records), the first two shaped like wave_stats()."""
    if items_per_wave <= 0 or window_ns <= 0:
        raise ValueError("items_per_wave and window_ns must be positive")
    recs = [r for r in records if (not kind or (r[0] & 0xFF) == kind) and r[5] != 0 and r[2] != 0]
    recs.sort(key=lambda r: (r[4], r[1], r[0]))
    n_host_items = sum(1 for r in recs if r[3] > 0)
    target = Fraction(host_ratio) * (1 + _RATIO_SLACK)

    def summary(shares):
        n = len(shares)
        out = {"n_waves": n, "n_host_pages": n_host_items,
               "n_zero_waves": sum(1 for f in shares if f == 0),
               "n_over_waves": sum(1 for f in shares if f > target),
               "mean": 0.0, "var": 0.0, "min": 0.0, "max": 0.0}
        if n:
            mean = sum(shares, Fraction(0)) / n
            var = sum(((f - mean) ** 2 for f in shares), Fraction(0)) / n
            out.update(mean=float(mean), var=float(var), min=float(min(shares)), max=float(max(shares)))
        return out

    waves = []
    for i in range(0, len(recs), items_per_wave):
        group = recs[i:i + items_per_wave]
        waves.append(Fraction(sum(r[3] for r in group), sum(r[2] for r in group)))
    windows = []
    if recs:
        t0 = recs[0][4]
        ends = [max(r[5], r[4] + 1) for r in recs]
        n_win = -(-(max(ends) - t0) // window_ns)
        host = [Fraction(0)] * n_win
        total = [Fraction(0)] * n_win
        for r, end in zip(recs, ends):
            a, e = r[4] - t0, end - t0
            w = a // window_ns
            while w * window_ns < e:
                lo, hi = max(w * window_ns, a), min((w + 1) * window_ns, e)
                part = Fraction(hi - lo, e - a)
                host[w] += part * r[3]
                total[w] += part * r[2]
                w += 1
        windows = [h / t for h, t in zip(host, total) if t > 0]
    return summary(waves), summary(windows), len(recs)

