"""Which declined writes could the tier afford to decline?  (Section 5.5 and Appendix D,
"Reuse distance of declined chunks": a declined chunk meets the condition of Proposition 1
if the chunk's next reference has D >= K_H, or if there is no next reference.)

Also the threshold sensitivity of Appendix D: for a write threshold kappa under fixed
admission (every request under pressure), which requests are filtered and what share of
the new-chunk writes they carry.
"""
import math

from . import stackdist
from .tier import FILTER_FIXED, HostTier


def declined_audit(stream, declined_positions, capacity):
    """stream: chunk keys in reference order; declined_positions: indices of declined misses.
    Returns dict(declined, meets, never_again, ratios) where ratios holds D / K_H of the
    declined chunks that are referenced again."""
    D = stackdist.reuse_distances(stream)
    nxt = {}
    last = {}
    for i, k in enumerate(stream):
        if k in last:
            nxt[last[k]] = i
        last[k] = i
    meets = never = 0
    ratios = []
    for i in declined_positions:
        j = nxt.get(i)
        if j is None:
            never += 1
            meets += 1
            continue
        d = D[j]
        ratios.append(d / capacity)
        if d >= capacity:
            meets += 1
    return dict(declined=len(declined_positions), meets=meets, never_again=never, ratios=ratios)


def kappa_sensitivity(requests, capacity, chunk_tokens, kappas):
    """requests: list of (keys, n_tokens, agent, now_ms).  For each kappa, run fixed admission
    and report (filtered requests, declined new chunks, all new chunks of a write-all run)."""
    out = {}
    for kappa in kappas:
        tier = HostTier(capacity, chunk_tokens, FILTER_FIXED, kappa)
        filtered = declined = 0
        for keys, n, agent, now in requests:
            r = tier.step(keys, n, agent, now)
            if not r.save:
                filtered += 1
                declined += sum(1 for h, a in zip(r.hit, r.admit) if not h and not a)
        out[kappa] = dict(filtered_requests=filtered, declined_chunks=declined,
                          admitted_chunks=tier.stats["admitted"])
    return out


def median(xs):
    xs = sorted(xs)
    if not xs:
        return math.nan
    m = len(xs) // 2
    return xs[m] if len(xs) % 2 else 0.5 * (xs[m - 1] + xs[m])
