"""Oracle: wave-aware pool of free KV blocks over a linearly placed KV range.

Test infrastructure only (see the package docstring).  Integer logic throughout.

What the paper fixes (Sec. 4.2, Sec. 4.3, Sec. 4.5)
  * the KV range is placed linearly: its head in HBM, its tail on the host
    tier, so the tier of a byte is a function of its address (Sec. 4.2);
  * a block holds 16 tokens of every KV head; the tensor is stored with heads
    outermost so each head's data is contiguous and page aligned (Sec. 4.5);
  * two kinds of block exist - one more head on the host than the other kind
    (for a host share 1/M with H >= ... heads: "single-head-host" against
    "all-local", kept in the ratio H : M - H; for H > M blocks carry
    floor(H/M) or ceil(H/M) host heads) (Sec. 4.3, Sec. 4.5);
  * one free list per kind (Sec. 4.5); a new request gets the host-heavier
    kind when the free share of that kind exceeds its target share, else the
    other kind; all blocks of a request share the kind (Sec. 4.3);
  * when the request's list is empty it borrows from the other list and keeps
    that kind from then on ("sticky"); when too few blocks remain in total the
    pool refuses and leaves the decision to the scheduler (Sec. 4.3).

Readings where the paper is silent (canonical choices; any order of equal
blocks would be valid, one is fixed so results can be compared bit for bit):
free lists are FIFO and start in ascending block order; the share in the
greedy rule is taken over all free blocks and a tie goes to the lighter kind;
the borrow rule is applied in both directions; a refused call changes nothing;
freed blocks return in the order they were handed out.
"""
from collections import deque

from .placement import PAGE_BYTES, TIER_HBM, TIER_HOST

OK = 0
ERR_INVALID = -1
ERR_NOMEM = -2

KIND_LO = 0  # fewer host heads per block
KIND_HI = 1  # one more host head per block


class PoolError(Exception):
    def __init__(self, code, msg):
        super().__init__(msg)
        self.code = code


class KVPool:
    def __init__(self, n_blocks, n_kv_heads, host_modulus, chunk_bytes=4096):
        if n_blocks <= 0 or n_kv_heads <= 0 or chunk_bytes <= 0 or host_modulus < 0:
            raise PoolError(ERR_INVALID, "bad pool geometry")
        if host_modulus == 1:
            raise PoolError(ERR_INVALID, "host_modulus 1 would put everything on the host")
        if PAGE_BYTES % chunk_bytes != 0 or (n_blocks * chunk_bytes) % PAGE_BYTES != 0:
            raise PoolError(ERR_INVALID, "a head's range must be a whole number of pages")
        self.n_blocks = n_blocks
        self.n_kv_heads = n_kv_heads
        self.host_modulus = host_modulus
        self.chunk_bytes = chunk_bytes
        # Sec. 4.5: [head][block][16 tokens][D]; chunk (h, b) starts at (h*N + b)*chunk_bytes.
        self.pages_per_head = n_blocks * chunk_bytes // PAGE_BYTES
        self.n_pages = n_kv_heads * self.pages_per_head
        # Sec. 4.2: the last floor(P/M) pages of the range are host pages.
        self.n_host_pages = self.n_pages // host_modulus if host_modulus else 0
        self.first_host_page = self.n_pages - self.n_host_pages
        # kind of every block, by counting its host heads from the definition
        counts = [self.host_heads(b) for b in range(n_blocks)]
        self.k_lo = min(counts)
        if any(c not in (self.k_lo, self.k_lo + 1) for c in counts):
            raise PoolError(ERR_INVALID, "blocks differ by more than one host head")
        self.kind = [KIND_HI if c > self.k_lo else KIND_LO for c in counts]
        self.free = {KIND_LO: deque(b for b in range(n_blocks) if self.kind[b] == KIND_LO),
                     KIND_HI: deque(b for b in range(n_blocks) if self.kind[b] == KIND_HI)}
        self.requests = {}      # id -> list of blocks in allocation order
        self.request_kind = {}  # id -> current kind

    # ---- geometry -------------------------------------------------------
    def chunk_page(self, head, block):
        return (head * self.n_blocks + block) * self.chunk_bytes // PAGE_BYTES

    def chunk_tier(self, head, block):
        return TIER_HOST if self.chunk_page(head, block) >= self.first_host_page else TIER_HBM

    def host_heads(self, block):
        return sum(1 for h in range(self.n_kv_heads) if self.chunk_tier(h, block) == TIER_HOST)

    def page_tiers(self):
        return [TIER_HOST if p >= self.first_host_page else TIER_HBM for p in range(self.n_pages)]

    # ---- allocation -----------------------------------------------------
    def _greedy_kind(self):
        """Sec. 4.3: host-heavier kind iff its share of the free blocks exceeds
        its target share.  The target share of that kind is H/M - floor(H/M)
        (H/M when M >= H).  Written with integers: free_hi / free > (H - k_lo*M) / M."""
        free_hi = len(self.free[KIND_HI])
        free_all = free_hi + len(self.free[KIND_LO])
        if self.host_modulus == 0:
            return KIND_LO
        target_num = self.n_kv_heads - self.k_lo * self.host_modulus
        if free_hi * self.host_modulus > target_num * free_all:
            return KIND_HI
        return KIND_LO

    def alloc(self, request_id, n):
        if n <= 0:
            raise PoolError(ERR_INVALID, "n must be positive")
        if len(self.free[KIND_LO]) + len(self.free[KIND_HI]) < n:
            raise PoolError(ERR_NOMEM, "not enough free blocks; defer to the scheduler")
        if request_id not in self.requests:
            self.requests[request_id] = []
            self.request_kind[request_id] = self._greedy_kind()
        out = []
        for _ in range(n):
            kind = self.request_kind[request_id]
            if not self.free[kind]:
                kind = 1 - kind                      # borrow from the other list ...
                self.request_kind[request_id] = kind  # ... and stay there (sticky)
            b = self.free[kind].popleft()
            self.requests[request_id].append(b)
            out.append(b)
        return out

    def free_request(self, request_id):
        if request_id not in self.requests:
            raise PoolError(ERR_INVALID, "unknown request")
        for b in self.requests.pop(request_id):
            self.free[self.kind[b]].append(b)
        del self.request_kind[request_id]

    # ---- inspection -----------------------------------------------------
    def query(self):
        live = [b for blocks in self.requests.values() for b in blocks]
        host_chunks = sum(self.k_lo + (1 if self.kind[b] == KIND_HI else 0) for b in live)
        return {
            "free_lo": len(self.free[KIND_LO]),
            "free_hi": len(self.free[KIND_HI]),
            "live_blocks": len(live),
            "live_host_chunks": host_chunks,
            "live_chunks": len(live) * self.n_kv_heads,
            "n_requests": len(self.requests),
        }
