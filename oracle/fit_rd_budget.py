"""Fit the RD allocator's bit budget of a benchmark recipe so that the plan it realises lands on the
rate the recipe names (test infrastructure, like the rest of oracle/: it calls only the oracle's
allocator on seeded workload data and prints the constant that workloads.config() records).

The allocator (Sec. 3.3) snaps every block up to a ladder rung and then applies the monotone
projections, so the realised rate sits below the budget it is given, by an amount that depends on
the data.  The recipes name realised averages ("5 bits/value average", "4-bit average"), so the
budget is chosen by bisection on sampled streams of the recipe's own data.

    python -m oracle.fit_rd_budget CONFIG TARGET_BPV [n_layers] [streams_per_layer]
"""
import sys

import numpy as np

from oracle import gkv_oracle as O
from paper_2608_23599_b200 import workloads as W

P = 64


def block_stats(k, mass):
    """Per-block mass (sequential fp32 sum) and key range proxy of one stream: k fp32 [T][d], mass fp32 [T]."""
    n = k.shape[0] // P
    mb = np.zeros(n, dtype=np.float32)
    rb = np.zeros(n, dtype=np.float32)
    for i in range(n):
        acc = np.float32(0.0)
        for t in range(P):
            acc = np.float32(acc + mass[i * P + t])
        mb[i] = acc
        blk = k[i * P:(i + 1) * P]
        rb[i] = np.max(blk.max(axis=0) - blk.min(axis=0))
    return mb, rb


def realised_bpv(w, stats, budget):
    bits = vals = 0
    for mb, rb, n_tail in stats:
        lv, _tau, _flag = O.rd_allocate(mb, rb, w.d_k, w.d_v, bool(w.v_aliases_k), n_tail, budget, w.n_sink_blocks, w.retire_after)
        nval = w.d_k + w.d_v
        bits += sum(O.block_bits(int(L), w.d_k, w.d_v, False) for L in lv) + n_tail * 16 * nval
        vals += (len(lv) * P + n_tail) * nval
    return bits / vals


def main():
    cid, target = int(sys.argv[1]), float(sys.argv[2])
    n_layers = int(sys.argv[3]) if len(sys.argv) > 3 else 2
    per_layer = int(sys.argv[4]) if len(sys.argv) > 4 else 2
    w = W.config(cid)
    stats = []
    for layer in range(n_layers):
        data = W.make_layer(w, layer, "cpu")
        k = data["k"].float().numpy()
        mass = data["mass"].numpy()
        picks = [(b, h) for b in range(w.batch) for h in range(w.n_kv_heads)]
        step = max(1, len(picks) // per_layer)
        for b, h in picks[::step][:per_layer]:
            mb, rb = block_stats(k[b, :, h], mass[b, h])
            stats.append((mb, rb, w.ctx % P))
    lo, hi = 0.25, 16.0
    for _ in range(30):
        mid = 0.5 * (lo + hi)
        if realised_bpv(w, stats, mid) < target:
            lo = mid
        else:
            hi = mid
    # the allocator's rate is a step function of the budget: report the step closest to the target
    best = min((abs(realised_bpv(w, stats, b) - target), b) for b in (lo, hi))[1]
    print("config %d: rd_budget_bpv = %.4f realises %.4f bits/value on %d sampled streams (target %.3f)"
          % (cid, best, realised_bpv(w, stats, best), len(stats), target))


if __name__ == "__main__":
    main()
