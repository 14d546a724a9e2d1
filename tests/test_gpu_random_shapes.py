"""GPU parity on randomly drawn shapes and call sequences (fixed seeds): KV heads 1-4, 1-8 query
heads per KV head, batch 1-3, contexts from 1 to 3100 tokens, staircase plans with random rung
widths / random external plans / the RD policy, exact residual rows, page sizes 0 / 16 / 32 / 64, up
to 200 single-token appends with their demotions, page selection with a sparse read.

What is held: the discrete state (levels, codes, scale / zero, centroids, exact rows, residual indices,
selected pages, resident bits) bit for bit and the attention outputs within the stated bounds
(max-abs 2e-3, relative L2 1e-2), in every case.
"""
import random

import numpy as np
import pytest
import torch

from oracle import gkv_oracle as O
from paper_2608_23599_b200 import workloads as W
import parity_util as U

pytestmark = pytest.mark.gpu

N_CASES = 36


def _draw(case):
    rnd = random.Random(20_000 + case)
    hkv = rnd.choice([1, 2, 3, 4])
    grp = rnd.choice([1, 2, 3, 4, 5, 6, 7, 8])
    batch = rnd.choice([1, 2, 3])
    T = rnd.choice([1, 30, 63, 64, 65, 127, 128, 200, 333, 512, 700, 1000, 1999, 2048, 3100])
    pol = rnd.choice(["stair", "stair", "ext", "rd"])
    page = rnd.choice([0, 0, 16, 32, 64])
    resf = rnd.choice([0.0, 0.0, 0.02, 0.1]) if pol != "ext" else 0.0
    n_app = rnd.choice([0, 1, 5, 70, 130, 200])
    kw = dict(name="random_shape", config_id=50 + case % 40, n_layers=1, batch=batch, n_q_heads=hkv * grp, n_kv_heads=hkv,
              d_k=128, d_v=128, ctx=T, max_ctx=T + 256, page_tokens=page, residual_fraction=resf)
    if pol == "stair":
        kw.update(policy=W.POLICY_STAIRCASE, stair_tokens=tuple(64 * rnd.choice([0, 1, 2, 3]) for _ in range(4)))
    elif pol == "ext":
        kw.update(policy=W.POLICY_EXTERNAL)
    else:
        kw.update(policy=W.POLICY_RD, rd_budget_bpv=rnd.choice([2.5, 4.0, 5.0, 7.0]), retire_after=rnd.choice([64, 128]))
    return W.Workload(**kw), pol, n_app


def _run_case(case, B):
    """Returns the largest max-abs output error of the case."""
    w, pol, n_app = _draw(case)
    tag = (f"case {case}: {w.n_kv_heads} KV heads x {w.n_q_heads // w.n_kv_heads}, batch {w.batch}, T {w.ctx}, {pol}, "
           f"page {w.page_tokens}, residual {w.residual_fraction}, {n_app} appends, rungs {tuple(w.stair_tokens)}")
    ocache = O.GradedCache(U.oracle_config(w))
    gcache = B.Cache(B.config_from_workload(w))
    dev = gcache.device
    worst = 0.0

    def check(out, o_out, what):
        nonlocal worst
        err, _ = U.assert_outputs_close(out, o_out, what)
        worst = max(worst, float(err))

    try:
        data = W.make_layer(w, 0, "cpu", with_mass=(pol == "rd" or w.residual_fraction > 0))
        plan = None
        if pol == "ext":
            prs = np.random.RandomState(case)
            plan = prs.choice(np.array([16, 8, 4, 2, 1], dtype=np.int8), size=(w.batch, w.n_kv_heads, w.ctx // 64)).astype(np.int8)
        U.ingest_both(w, 0, data, ocache, gcache, level_plan=plan)
        U.assert_state_equal(ocache, gcache, 0)
        out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
        check(out, o_out, tag)
        for step in range(n_app):
            tok = W.make_decode_tokens(w, 0, step, "cpu")
            ocache.append_demote(0, U.f32(tok["k"]), U.f32(tok["v"]))
            gcache.gkv_append_demote(0, tok["k"].to(dev), tok["v"].to(dev))
            if step in (0, n_app - 1) or (w.ctx + step + 1) % 64 in (0, 1):
                out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, tok["q"])
                check(out, o_out, tag + f", step {step}")
        if n_app:
            U.assert_state_equal(ocache, gcache, 0)
        assert gcache.gkv_bits_report(0).resident_bits == ocache.bits_report(0)["resident_bits"], tag
        ctx = w.ctx + n_app
        page = w.page_tokens
        if page > 0 and w.residual_fraction == 0.0 and ctx // page > 2:
            budget = page * max(1, (ctx // page) // 3)
            pages = torch.zeros((w.batch, w.n_kv_heads, budget // page), dtype=torch.int32, device=dev)
            n_sel = gcache.gkv_quest_select(0, data["q"].to(dev), budget, pages)
            sel_o = ocache.quest_select(0, U.f32(data["q"]), budget)
            torch.cuda.synchronize()
            pg = pages.cpu().numpy()
            for b in range(w.batch):
                for h in range(w.n_kv_heads):
                    assert np.array_equal(pg[b, h, :n_sel], sel_o[b][h]), f"{tag}: selected pages differ for stream {(b, h)}"
            out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"], page_idx_gpu=pages, n_sel=n_sel,
                                                   page_idx_oracle=sel_o)
            check(out, o_out, tag + ", page-list read")
    finally:
        gcache.close()
    return worst


@pytest.mark.parametrize("case", range(N_CASES))
def test_random_shape_state_bit_exact_and_outputs_within_bounds(case):
    from paper_2608_23599_b200 import binding as B
    B.build()
    _run_case(case, B)
