"""Oracle for the chained block hash and the hint index probe of Section 4.3 (Eq. design-hash and the paragraph on
galloping and bisecting, and the paragraph on the backward scan for recurrent snapshots).

TEST INFRASTRUCTURE ONLY: plain Python integers and a dict; shares no code with the library's implementation
(`wpp_hash_blocks`, `wpp_hint_*`); only tests import it.

The paper fixes the structure: H_{-1} = 0, H_i = hash(B_i, extraKeys_i, salt, H_{i-1}) over FULL token blocks; an
index keyed by (cache window, H_i) with a counter per key (incremented when a block joins the tree, decremented when
it leaves, entry dropped at zero); for dense attention prefixes, probes at depths 1, 2, 4, ... until the first
miss, then bisection between the last match and that miss.  It does not fix the hash function.
READING (parity unpinned for this choice): 64-bit arithmetic throughout; mix64 is the splitmix64 finaliser;
  term_k   = mix64(((token_k mod 2^32) << 32 | k) xor 0xD6E8FEB86659FD93)      k = position inside the block
  digest_i = sum_k term_k                                         (mod 2^64; order-sensitive through k)
  H_i      = mix64(H_{i-1} xor mix64(digest_i + extraKeys_i) xor (salt * 0x9E3779B97F4A7C15))
"""
MASK = (1 << 64) - 1


def mix64(x):
    x &= MASK
    x ^= x >> 30
    x = (x * 0xBF58476D1CE4E5B9) & MASK
    x ^= x >> 27
    x = (x * 0x94D049BB133111EB) & MASK
    x ^= x >> 31
    return x


def block_digest(tokens):
    d = 0
    for k, t in enumerate(tokens):
        d = (d + mix64((((int(t) & 0xFFFFFFFF) << 32) | k) ^ 0xD6E8FEB86659FD93)) & MASK
    return d


def chained_hashes(tokens, B, salt=0, extra_keys=None):
    """H_0 .. H_{n-1} for the n = len(tokens) // B full blocks of one request (Eq. design-hash)."""
    n = len(tokens) // B
    out, h = [], 0
    s = (salt * 0x9E3779B97F4A7C15) & MASK
    for i in range(n):
        e = 0 if extra_keys is None else int(extra_keys[i]) & MASK
        d = block_digest(tokens[i * B:(i + 1) * B])
        h = mix64(h ^ mix64((d + e) & MASK) ^ s)
        out.append(h)
    return out


class HintIndex:
    """Counted set of (window, hash) keys."""

    def __init__(self):
        self.count = {}

    def add(self, window, hashes):
        for h in hashes:
            self.count[(window, h)] = self.count.get((window, h), 0) + 1

    def remove(self, window, hashes):
        for h in hashes:
            c = self.count.get((window, h), 0)
            if c <= 1:
                self.count.pop((window, h), None)
            else:
                self.count[(window, h)] = c - 1

    def has(self, window, h):
        return (window, h) in self.count

    def __len__(self):
        return len(self.count)


def longest_prefix_linear(index, window, hashes):
    """The definition: number of leading blocks whose keys are all in the index, found block by block."""
    n = 0
    for h in hashes:
        if not index.has(window, h):
            break
        n += 1
    return n


def probe_reverse_scan(index, window, hashes, limit):
    """Recurrent snapshots are sparse: walk backward from the attention-limited endpoint `limit` to the first depth
    whose key is present.  Returns (depth, list of probed depths); depth 0 when nothing at or below `limit` is."""
    probed = []
    d = min(limit, len(hashes))
    while d >= 1:
        probed.append(d)
        if index.has(window, hashes[d - 1]):
            break
        d -= 1
    return d, probed


def reuse_candidate(endpoints):
    """The minimum of the local caches' endpoints (Section 4.3); the all-rank minimum is taken over these."""
    return min(endpoints)


def probe_gallop_bisect(index, window, hashes):
    """Depths 1, 2, 4, ... until the first miss, then bisect between the last match and the miss.  Returns
    (matched depth, list of probed depths).  Exact when presence is monotone in depth, which holds for an index
    whose blocks were added as whole prefixes (a chained key can only be present if its prefix was hashed)."""
    N = len(hashes)
    probed = []

    def present(depth):
        probed.append(depth)
        return index.has(window, hashes[depth - 1])

    lo, hi, d = 0, N + 1, 1          # depth lo is known to match (0: nothing), depth hi is known or assumed to miss
    while d <= N:
        if present(d):
            lo = d
            d *= 2
        else:
            hi = d
            break
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if present(mid):
            lo = mid
        else:
            hi = mid
    return lo, probed
