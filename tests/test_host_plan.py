"""Host-side policy code of the library against the oracle, without a GPU: the staircase plan
(Sec. 3.2, Fig. 1) and the monotone rate-distortion allocator (Sec. 3.3) through the host-only
entry point gkv_debug_plan_levels, plus the arena sizing / configuration checks."""
import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import gkv_oracle as O  # noqa: E402
from paper_2608_23599_b200 import binding as B  # noqa: E402


@pytest.mark.parametrize("stair,sinks", [((512, 1024, 1536, 1024), 0), ((128, 0, 0, 0), 0), ((-1, 0, 0, 0), 0),
                                         ((64, 128, -1, 0), 2), ((0, 0, 0, 0), 1), ((1024, 4096, 16384, 8192), 4)])
def test_staircase_plan_matches_oracle(stair, sinks):
    for n_closed in (0, 1, 7, 64, 300, 777):
        cfg = B.make_config(1, 1, 8, 2, 128, 128, 65536, stair_tokens=stair, n_sink_blocks=sinks)
        got, _ = B.gkv_debug_plan_levels(cfg, n_closed)
        want = O.staircase_levels(n_closed, stair, sinks)
        assert np.array_equal(got.astype(np.int32), np.asarray(want, dtype=np.int32)), (stair, sinks, n_closed)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("mono", [1, 0])
def test_rd_allocator_matches_oracle(seed, mono):
    rng = np.random.default_rng(1000 + seed)
    n = int(rng.integers(5, 400))
    n_tail = int(rng.integers(0, 64))
    budget = float(rng.choice([1.5, 2.5, 4.0, 4.84, 7.0, 12.0]))
    retire = int(rng.choice([0, 64, 128, 512]))
    sinks = int(rng.integers(0, 3))
    # masses decay with age and carry a few heavy blocks; ranges are log-normal
    mass = (rng.random(n) ** 3 / n).astype(np.float32)
    mass[rng.integers(0, n, size=3)] += np.float32(0.2)
    rge = np.exp(rng.normal(1.0, 0.5, size=n)).astype(np.float32)
    cfg = B.make_config(1, 1, 8, 2, 128, 128, 65536, policy=B.POLICY_RD, rd_budget_bpv=budget, retire_after=retire,
                        n_sink_blocks=sinks, monotone_in_age=mono)
    got, miss = B.gkv_debug_plan_levels(cfg, n, n_tail, mass, rge)
    want, _tau, flag = O.rd_allocate(mass, rge, 128, 128, 0, n_tail, budget, sinks, retire, monotone_in_age=mono)
    assert np.array_equal(got.astype(np.int32), np.asarray(want, dtype=np.int32))
    assert miss == bool(flag)
    # the plan never spends more than the budget unless it says so, and pins stay exact
    bits = sum(O.block_bits(int(L), 128, 128, 0) for L in got) + n_tail * 16 * 256
    if not miss:
        assert bits <= np.floor(budget * (n * 64 + n_tail) * 256)
    assert all(got[i] == 16 for i in range(min(sinks, n)))


def test_plan_rejects_bad_arguments():
    cfg = B.make_config(1, 1, 8, 2, 128, 128, 4096, policy=B.POLICY_RD, rd_budget_bpv=4.0)
    with pytest.raises(B.GkvError):
        B.gkv_debug_plan_levels(cfg, 10, 0, None, None)          # the allocator needs mass and range
    with pytest.raises(B.GkvError):
        B.gkv_debug_plan_levels(cfg, 10, 64, np.ones(10), np.ones(10))   # a tail holds fewer than 64 tokens
    ext = B.make_config(1, 1, 8, 2, 128, 128, 4096, policy=B.POLICY_EXTERNAL)
    with pytest.raises(B.GkvError):
        B.gkv_debug_plan_levels(ext, 10)


def test_arena_size_covers_the_worst_case_and_grows_with_context():
    sizes = []
    for ctx in (4096, 16384, 65536):
        cfg = B.make_config(2, 2, 8, 2, 128, 128, ctx, stair_tokens=(-1, 0, 0, 0))
        need = B.gkv_query_arena_bytes(cfg)
        # an all-exact cache: every token of every stream holds 512 bytes
        assert need >= 2 * 2 * 2 * ctx * 512
        sizes.append(need)
    assert sizes[0] < sizes[1] < sizes[2]
    graded = B.gkv_query_arena_bytes(B.make_config(2, 2, 8, 2, 128, 128, 65536, stair_tokens=(1024, 4096, 16384, 8192)))
    assert graded < sizes[2] // 2                              # the ladder is what makes the arena small
    with pytest.raises(B.GkvError):
        B.gkv_query_arena_bytes(B.make_config(1, 1, 7, 2, 128, 128, 4096))     # heads must divide
    with pytest.raises(B.GkvError):
        B.gkv_query_arena_bytes(B.make_config(1, 1, 8, 2, 96, 96, 4096))       # head dim 128 only


@pytest.mark.parametrize("seed", range(8))
def test_decode_time_replan_matches_oracle_and_never_promotes(seed):
    """The plan of gkv_rd_reallocate (host part) against the oracle's allocator run with the current
    levels as upper bounds (Sec. 3.2: demotion only), on the plan of an earlier, shorter context."""
    rng = np.random.default_rng(7000 + seed)
    n0 = int(rng.integers(8, 200))
    grow = int(rng.integers(1, 6))
    n = n0 + grow
    n_tail = int(rng.integers(0, 64))
    budget = float(rng.choice([2.5, 4.0, 4.84, 7.0]))
    retire = int(rng.choice([64, 128, 512]))
    sinks = int(rng.integers(0, 3))
    mono = int(seed % 2)
    mass0 = (rng.random(n0) ** 3 / n0).astype(np.float32)
    rge = np.exp(rng.normal(1.0, 0.5, size=n)).astype(np.float32)
    cfg = B.make_config(1, 1, 8, 2, 128, 128, 65536, policy=B.POLICY_RD, rd_budget_bpv=budget, retire_after=retire,
                        n_sink_blocks=sinks, monotone_in_age=mono)
    first, _ = B.gkv_debug_plan_levels(cfg, n0, 0, mass0, rge[:n0])
    # the context grew by `grow` exact blocks and the running masses moved
    prev = np.concatenate([first, np.full(grow, 16, dtype=np.int8)])
    mass = np.concatenate([0.6 * mass0 + 0.4 * (rng.random(n0) / n0), rng.random(grow) / n]).astype(np.float32)
    got, miss = B.gkv_debug_replan_levels(cfg, n_tail, mass, rge, prev)
    want, _tau, flag = O.rd_allocate(mass, rge, 128, 128, 0, n_tail, budget, sinks, retire, prev.astype(np.int32), mono)
    assert np.array_equal(got.astype(np.int32), np.asarray(want, dtype=np.int32))
    assert miss == bool(flag)
    assert np.all(got <= prev)                                       # no promotion
    recent = retire // 64
    assert all(got[i] == 16 for i in range(n) if (i < sinks or n - 1 - i < recent) and prev[i] == 16)
    if not miss:
        bits = sum(O.block_bits(int(L), 128, 128, 0) for L in got) + n_tail * 16 * 256
        assert bits <= np.floor(np.float32(budget) * (n * 64 + n_tail) * 256)
