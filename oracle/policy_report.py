"""Hit rates of the cache policies of Sec. 5.1 on a synthetic, temporally correlated activation
trace, with the CPU oracle only: DIP masks under LRU, LFU and offline Belady, and DIP-CA
(gamma 0.2) under LRU and LFU.  Mirrors the structure of the paper's policy comparison; the
numbers depend on the synthetic trace and say nothing about real models.

    python -m oracle.policy_report [d] [keep_ratio] [cache_budget] [tokens] [correlation]
"""
import sys

import numpy as np

import oracle


def trace(d, tokens, corr, seed=0):
    rng = np.random.default_rng(seed)
    scale = np.exp(rng.standard_normal(d))          # some columns are habitually larger
    x = rng.standard_t(3.0, d)
    out = []
    for _ in range(tokens):
        x = corr * x + np.sqrt(1.0 - corr * corr) * rng.standard_t(3.0, d)
        out.append((x * scale).astype(np.float32))
    return np.stack(out)


def main():
    a = sys.argv[1:]
    d = int(a[0]) if len(a) > 0 else 1024
    rho = float(a[1]) if len(a) > 1 else 0.25
    beta = float(a[2]) if len(a) > 2 else 0.5
    tokens = int(a[3]) if len(a) > 3 else 300
    corr = float(a[4]) if len(a) > 4 else 0.8
    k, cap = max(1, int(rho * d + 0.5)), int(beta * d)
    xs = trace(d, tokens, corr)
    rows = []
    masks = np.stack([oracle.dip_ca_mask(x, k)[0] for x in xs])
    for pol in ("lru", "lfu"):
        c = oracle.Cache(d, cap, pol)
        for m in masks:
            oracle.cache_update(c, m)
        rows.append(("DIP + " + pol.upper(), c.counters[0] / (tokens * k)))
    hb, mb = oracle.belady_hits(masks, cap)
    rows.append(("DIP + Belady (offline)", hb / (tokens * k)))
    for pol in ("lru", "lfu"):
        c = oracle.Cache(d, cap, pol)
        for x in xs:
            oracle.dip_ca_mask(x, k, 0.2, c)
        rows.append(("DIP-CA (gamma 0.2) + " + pol.upper(), c.counters[0] / (tokens * k)))
    print("d %d, k %d, capacity %d, %d tokens, correlation %.2f" % (d, k, cap, tokens, corr))
    for name, hr in rows:
        print("  %-28s hit rate %.3f" % (name, hr))


if __name__ == "__main__":
    main()
