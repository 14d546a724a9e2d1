"""Pins for the CPU oracle: it is checked against what the paper and the mathematics fix
(closed forms, brute force on tiny inputs, printed accounting identities, invariants), never
against itself.  Each test names the passage it pins."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import gkv_oracle as O

RNG = np.random.default_rng(1234)


def bf(x):
    return O.bf16_round(np.asarray(x, dtype=np.float32))


def small_cfg(**kw):
    base = dict(n_layers=1, batch=1, n_q_heads=4, n_kv_heads=2, d_k=32, d_v=32)
    base.update(kw)
    return O.Config(**base)


def rand_kv(cfg, T, rng=RNG, scale=1.0):
    k = bf(scale * rng.standard_normal((cfg.batch, T, cfg.n_kv_heads, cfg.d_k)))
    v = bf(rng.standard_normal((cfg.batch, T, cfg.n_kv_heads, cfg.d_v)))
    q = bf(rng.standard_normal((cfg.batch, cfg.n_q_heads, cfg.d_k)))
    return k, v, q


def dense_attention_torch(k, v, q, n_kv, scale):
    """Independent textbook softmax attention (Eq. 1) in float64 via torch."""
    B, T, _, dk = k.shape
    Hq = q.shape[1]
    g = Hq // n_kv
    out = np.zeros((B, Hq, v.shape[3]))
    for b in range(B):
        for h in range(Hq):
            kk = torch.from_numpy(k[b, :, h // g].astype(np.float64))
            vv = torch.from_numpy(v[b, :, h // g].astype(np.float64))
            qq = torch.from_numpy(q[b, h].astype(np.float64))
            w = torch.softmax(kk @ qq * scale, dim=0)
            out[b, h] = (w @ vv).numpy()
    return out


# ---- N0 conversions -------------------------------------------------------------------------
def test_bf16_round_matches_torch():
    x = RNG.standard_normal(10000).astype(np.float32) * np.float32(37.0)
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 3.0e-39]      # exact ties and a subnormal
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.bf16_round(x), ref)
    assert np.array_equal(O.bf16_bits(ref), torch.from_numpy(ref).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


def test_fp16_sat():
    x = np.array([1e6, -1e6, 65504.0, 65520.0, 0.1], dtype=np.float32)
    y = O.fp16_sat(x)
    assert y[0] == np.float16(65504) and y[1] == np.float16(-65504) and y[3] == np.float16(65504)
    assert y[4] == np.float16(0.1)


# ---- P1: exact tier equals dense attention (Sec. 3.2 level 16; Eq. 1) ------------------------
def test_exact_tier_equals_dense_attention():
    cfg = small_cfg(stair_tokens=(-1, 0, 0, 0))
    k, v, q = rand_kv(cfg, 200)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v)
    out, lse = c.decode_attn(0, q)
    ref = dense_attention_torch(k, v, q, cfg.n_kv_heads, c.scale)
    assert np.max(np.abs(out - ref)) < 1e-12
    assert set(c.levels(0, 0, 0)) == {16}


# ---- P2: brute force on a tiny context + permutation invariance ------------------------------
def test_bruteforce_tiny_and_permutation():
    cfg = small_cfg(n_q_heads=2, n_kv_heads=1, d_k=8, d_v=8, stair_tokens=(-1, 0, 0, 0))
    k, v, q = rand_kv(cfg, 40)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v)
    out, lse = c.decode_attn(0, q)
    sc = 1.0 / math.sqrt(8)
    sc = float(np.float32(sc))
    for h in range(2):
        logits = [sc * math.fsum(float(q[0, h, c_]) * float(k[0, t, 0, c_]) for c_ in range(8)) for t in range(40)]
        m = max(logits)
        e = [math.exp(l - m) for l in logits]
        s = math.fsum(e)
        for c_ in range(8):
            o = math.fsum(e[t] / s * float(v[0, t, 0, c_]) for t in range(40))
            assert abs(o - out[0, h, c_]) < 1e-13
        assert abs(m + math.log(s) - lse[0, h]) < 1e-12
    # permuting the tokens of an all-exact cache leaves the output unchanged
    perm = RNG.permutation(40)
    c2 = O.GradedCache(cfg)
    c2.append_demote(0, k[:, perm], v[:, perm])
    out2, _ = c2.decode_attn(0, q)
    assert np.max(np.abs(out - out2)) < 1e-13


# ---- P3: the paper's printed accounting identities (Tables 1-2, Sec. 3.4-3.5, Eq. 7-8) --------
def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "accounting_identities.txt")
    vals = []
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        vals.append(float(line.split("|")[0]))
    return vals


def test_accounting_identities_from_paper():
    g_stream, g_snap, g_quest_res, g_quest_read, g_box, g_five = _golden()
    D = 32
    # Quest: exact resident K/V + boxes at 64-token pages; read = boxes + 12.5 % pages + current page
    cfg = small_cfg(n_q_heads=1, n_kv_heads=1, d_k=D, d_v=D, page_tokens=64, stair_tokens=(-1, 0, 0, 0))
    k, v, q = rand_kv(cfg, 16384)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v)
    rep = c.bits_report(0)
    assert rep["bpv_resident"] == g_quest_res
    assert rep["box_bits"] / rep["values"] == g_box
    sel = c.quest_select(0, q, 33 * 64)               # 12.5 % of 256 pages + one current 64-token page
    assert len(sel[0][0]) == 33
    c.decode_attn(0, q, sel)
    assert c.bits_report(0)["bpv_read"] == g_quest_read
    # the summaries count for the read that scored them: the same list read again, without a new
    # scoring pass, costs the pages alone (12.5 % of the pages + the current page = 33 / 256 of 16 bits)
    c.decode_attn(0, q, sel)
    assert c.bits_report(0)["bpv_read"] == g_quest_read - g_box == 33 / 256 * 16
    # exact tokens cost 16 bits per value each, tail included: StreamingLLM / SnapKV rows
    for kept, want in ((4 + 2048, g_stream), (2304, g_snap)):
        c2 = O.GradedCache(cfg)
        c2.append_demote(0, k[:, :kept], v[:, :kept])
        assert c2.bits_report(0)["resident_bits"] - c2.bits_report(0)["box_bits"] == int(want * 16384 * 2 * D)
    # five-bit budgets: base rate B plus 16 bits on the exact fraction (Sec. 3.4)
    assert 4.875 + 16 * 0.0078125 == g_five and 4.5 + 16 * 0.03125 == g_five
    cfg3 = small_cfg(n_q_heads=1, n_kv_heads=1, d_k=D, d_v=D, policy=O.POLICY_EXTERNAL, residual_fraction=0.03125)
    T = 8192
    k, v, q = rand_kv(cfg3, T)
    plan = np.array([[[4] * 96 + [2] * 32]], dtype=np.int8)      # 0.75*5 + 0.25*3 = 4.5 bits/value
    mass = RNG.random((1, 1, T)).astype(np.float32)
    c3 = O.GradedCache(cfg3)
    c3.append_demote(0, k, v, token_mass=mass, level_plan=plan)
    rep = c3.bits_report(0)
    assert len(c3.streams[(0, 0, 0)].res_idx) == 256
    assert rep["bpv_paper"] == g_five


# ---- P4: beta(L) including scales; config-0 ladder = 6.875 bits/value --------------------------
def test_beta_and_cfg0_rate():
    assert [O.beta_bits(L) for L in (16, 8, 4, 2, 1)] == [16.0, 9.0, 5.0, 3.0, 0.25]
    cfg = small_cfg(n_q_heads=2, n_kv_heads=1, stair_tokens=(512, 1024, 1536, 1024))
    k, v, q = rand_kv(cfg, 4096)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v)
    rep = c.bits_report(0)
    assert rep["blocks_by_level"] == {16: 8, 8: 16, 4: 24, 2: 16, 1: 0}
    assert rep["bpv_resident"] == 6.875
    c.decode_attn(0, q)
    assert c.bits_report(0)["bpv_read"] == 6.875          # dense graded read: read = resident
    for L in (16, 8, 4, 2, 1):
        assert O.block_bits(L, 32, 32, False) == int(O.beta_bits(L) * 64 * 64)


# ---- P5: quantiser properties (Sec. 3.2 'packed scalar quantizers') ----------------------------
@pytest.mark.parametrize("bits", [8, 4, 2])
def test_quantizer_properties(bits):
    qmax = 2 ** bits - 1
    x = bf(RNG.standard_normal((50, 4, 32)) * 3.0)
    code, s, z, flag = O.quantize_groups(x, bits)
    assert not flag and code.min() >= 0 and code.max() <= qmax
    xh = O.dequantize_groups(code, s, z)
    s32, z32 = s.astype(np.float32), z.astype(np.float32)
    # the group minimum maps to code 0
    amin = x.argmin(axis=-1)
    assert np.all(np.take_along_axis(code, amin[..., None], -1) == 0)
    # error bound: half a step inside the grid + the slack of rounding s and z to fp16
    slack = qmax * s32 * 2.0 ** -11 + np.abs(x.min(-1)) * 2.0 ** -11 + 1e-6
    assert np.all(np.abs(x - xh) <= (s32 / 2 + slack)[..., None])
    # brute-force nearest code agrees (up to ties in the last fp32 bit)
    grid = np.arange(qmax + 1, dtype=np.float64)
    for idx in [(0, 0), (7, 3), (49, 1)]:
        cand = grid[None, :] * float(s32[idx]) + float(z32[idx])
        err = np.abs(x[idx][:, None].astype(np.float64) - cand)
        best = err.min(axis=1)
        mine = np.abs(x[idx].astype(np.float64) - xh[idx].astype(np.float64))
        assert np.all(mine <= best + 1e-6 * (1 + np.abs(x[idx])))
    # data already on the grid with fp16-exact end points is reproduced exactly
    grid_x = (RNG.integers(0, qmax + 1, (6, 32)).astype(np.float32)) * np.float32(0.25) - np.float32(2.0)
    grid_x[:, 0] = -2.0
    grid_x[:, 1] = -2.0 + 0.25 * qmax
    code, s, z, _ = O.quantize_groups(grid_x, bits)
    assert np.array_equal(O.dequantize_groups(code, s, z), grid_x)
    # constant group: s = 0, all codes 0, exact reconstruction of the (fp16-representable) constant
    const = np.full((2, 32), 1.5, dtype=np.float32)
    code, s, z, _ = O.quantize_groups(const, bits)
    assert np.all(code == 0) and np.all(s == 0) and np.array_equal(O.dequantize_groups(code, s, z), const)


def test_group_axes_keys_time_values_channels():
    """Keys are grouped along time, values along channels (Sec. 3.2): an outlier CHANNEL in K
    must not inflate the step of other channels; an outlier TOKEN in V must not inflate other tokens."""
    xk = bf(RNG.standard_normal((64, 32)))
    xk[:, 5] *= 100.0
    kc, ks, kz, _ = O.quantize_k_block(xk, 4)
    assert ks.shape == (2, 32) and float(ks[0, 5]) > 20 * float(np.median(ks[0].astype(np.float32)))
    rec = O.dequantize_k_block(kc, ks, kz)
    other = np.delete(np.arange(32), 5)
    assert np.max(np.abs(rec[:, other] - xk[:, other])) < 0.5
    xv = bf(RNG.standard_normal((64, 64)))
    xv[9] *= 100.0
    vc, vs, vz, _ = O.quantize_v_block(xv, 4)
    assert vs.shape == (64, 2)
    rec = O.dequantize_v_block(vc, vs, vz)
    assert np.max(np.abs(np.delete(rec, 9, 0) - np.delete(xv, 9, 0))) < 0.5
    # a block equals a direct per-group call (layout bookkeeping only)
    c0, s0, z0, _ = O.quantize_groups(xk[:32, 7][None, :], 4)
    assert np.array_equal(c0[0], kc[:32, 7]) and s0[0] == ks[0, 7] and z0[0] == kz[0, 7]
    c1, s1, z1, _ = O.quantize_groups(xv[3, 32:64][None, :], 4)
    assert np.array_equal(c1[0], vc[3, 32:64]) and s1[0] == vs[3, 1] and z1[0] == vz[3, 1]


# ---- P6: requantisation chain (Sec. 3.2: no dense copy survives) --------------------------------
def test_requant_chain_uses_current_reconstruction():
    cfg = small_cfg(n_q_heads=1, n_kv_heads=1)
    k, v, q = rand_kv(cfg, 64)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v)
    st = c.streams[(0, 0, 0)]
    c.demote_to(0, 0, 0, 0, 8)
    rec8_k = st.blocks[0].recon_k().copy()
    rec8_v = st.blocks[0].recon_v().copy()
    c.demote_to(0, 0, 0, 0, 4)
    kc, ks, kz, _ = O.quantize_k_block(rec8_k, 4)
    vc, vs, vz, _ = O.quantize_v_block(rec8_v, 4)
    b = st.blocks[0]
    assert np.array_equal(b.k_codes, kc) and np.array_equal(b.k_scale, ks) and np.array_equal(b.v_codes, vc)
    assert b.history == [16, 8, 4]
    with pytest.raises(AssertionError):
        c.demote_to(0, 0, 0, 0, 8)                       # promotion is forbidden
    # requantising a reconstruction at its own level moves codes by at most one step
    kc2, _, _, _ = O.quantize_k_block(b.recon_k(), 4)
    assert np.max(np.abs(kc2.astype(int) - b.k_codes.astype(int))) <= 1
    c.demote_to(0, 0, 0, 0, 1)
    assert np.array_equal(st.blocks[0].k_cent, O.centroid_of(b.recon_k()))


# ---- P7: centroid tier (Sec. 3.2 level 1: logically repeated centroid pair) ---------------------
def test_centroid_of_identical_tokens_equals_exact():
    cfg_c = small_cfg(n_q_heads=2, n_kv_heads=1, stair_tokens=(64, 0, 0, 0))
    cfg_e = small_cfg(n_q_heads=2, n_kv_heads=1, stair_tokens=(-1, 0, 0, 0))
    k, v, q = rand_kv(cfg_c, 192)
    k[:, :64] = k[:, :1]
    v[:, :64] = v[:, :1]
    outs = []
    for cfg in (cfg_c, cfg_e):
        c = O.GradedCache(cfg)
        c.append_demote(0, k, v)
        outs.append(c.decode_attn(0, q)[0])
    c = O.GradedCache(cfg_c)
    c.append_demote(0, k, v)
    assert list(c.levels(0, 0, 0)) == [1, 1, 16]
    # block 0 is 64 identical tokens -> identical contribution; block 1 differs, so compare a cache
    # whose block 1 is also constant
    k[:, 64:128] = k[:, 64:65]
    v[:, 64:128] = v[:, 64:65]
    outs = []
    for cfg in (cfg_c, cfg_e):
        c = O.GradedCache(cfg)
        c.append_demote(0, k, v)
        outs.append(c.decode_attn(0, q)[0])
    assert np.max(np.abs(outs[0] - outs[1])) < 1e-12
    x = np.concatenate([np.full((32, 4), 3.0), np.full((32, 4), -3.0)]).astype(np.float32)
    assert np.all(O.centroid_of(x) == 0)
    # sequential fp32 sum, then bf16 rounding
    y = bf(RNG.standard_normal((64, 3)))
    acc = np.float32(0)
    for t in range(64):
        acc = np.float32(acc + y[t, 1])
    assert O.centroid_of(y)[1] == O.bf16_round(np.float32(acc / np.float32(64)))[()]


# ---- P8 / P11: monotone demotion and causality under appends (Sec. 3.1, 3.2) --------------------
def test_monotone_levels_and_causality_under_appends():
    cfg = small_cfg(n_q_heads=2, n_kv_heads=1, stair_tokens=(64, 64, 64, 64))
    T0, n_app = 300, 200
    k, v, q = rand_kv(cfg, T0 + n_app)
    c = O.GradedCache(cfg)
    c.append_demote(0, k[:, :T0], v[:, :T0])
    snapshots = {}
    for t in range(T0, T0 + n_app):
        c.append_demote(0, k[:, t:t + 1], v[:, t:t + 1])
        st = c.streams[(0, 0, 0)]
        lv = c.levels(0, 0, 0)
        assert np.all(np.diff(lv) >= 0)                   # precision never decreases toward recent
        snapshots[t] = [b.level for b in st.blocks]
    st = c.streams[(0, 0, 0)]
    for b in st.blocks:
        assert all(x >= y for x, y in zip(b.history, b.history[1:]))      # levels only fall over time
    assert list(c.levels(0, 0, 0)) == [1, 1, 1, 2, 4, 8, 16]
    assert st.blocks[0].history[0] >= 2 and st.blocks[-1].history == [16]
    # causality: changing FUTURE tokens never changes what was stored before them
    k2, v2 = k.copy(), v.copy()
    k2[:, T0 + 100:] += 1.0
    v2[:, T0 + 100:] -= 1.0
    k2, v2 = bf(k2), bf(v2)
    ca, cb = O.GradedCache(cfg), O.GradedCache(cfg)
    for cc, (kk, vv) in ((ca, (k, v)), (cb, (k2, v2))):
        cc.append_demote(0, kk[:, :T0], vv[:, :T0])
        for t in range(T0, T0 + 100):
            cc.append_demote(0, kk[:, t:t + 1], vv[:, t:t + 1])
    oa, _ = ca.decode_attn(0, q)
    ob, _ = cb.decode_attn(0, q)
    assert np.array_equal(oa, ob)
    # block content depends on its demotion history: one-shot int4 differs from 16->8->4
    one = O.GradedCache(small_cfg(n_q_heads=2, n_kv_heads=1, stair_tokens=(0, 0, 6400, 0)))
    one.append_demote(0, k[:, :64], v[:, :64])
    hist_blk = [b for b in st.blocks if b.history == [16, 8, 4]]
    assert hist_blk, "expected a block that walked 16->8->4"


# ---- P9: allocator (Sec. 3.3, Eq. 4-5) -----------------------------------------------------------
def test_rd_allocator_bruteforce():
    kmap = {1: 1.0, 2: 3.0, 4: 15.0, 8: 255.0}
    rng = np.random.default_rng(7)
    for trial in range(12):
        n = 6
        mass = rng.random(n).astype(np.float32) ** 3
        rng_b = (1 + 5 * rng.random(n)).astype(np.float32)
        budget = float(rng.uniform(1.0, 9.0))
        mono = trial % 2
        lv, tau, flag = O.rd_allocate(mass, rng_b, 32, 32, False, 10, budget, 0, 64, None, mono)
        y = mass.astype(np.float64) * rng_b.astype(np.float64)
        T = n * 64 + 10
        budget_bits = math.floor(float(np.float32(budget)) * T * 64)

        def bits(assign):
            return sum(O.block_bits(L, 32, 32, False) for L in assign) + 10 * 16 * 64

        def plan_for(t):
            """rule (snap up to the ladder) followed by the projections, re-derived here"""
            out = []
            for b in range(n):
                L = 16
                for cand in (1, 2, 4, 8):
                    if y[b] <= t * kmap[cand]:
                        L = cand
                        break
                out.append(L)
            out[-1] = 16                                          # retire_after pins the newest block
            if mono:
                for b in range(n - 3, -1, -1):
                    out[b] = min(out[b], out[b + 1])
            return out

        if not mono:
            # without the age projection every block obeys its own tolerance, so the smallest
            # feasible multiplier can be found by brute force over all 5^n assignments
            best_tau = None
            for assign in itertools.product((1, 2, 4, 8, 16), repeat=n):
                if assign[-1] != 16 or bits(assign) > budget_bits:
                    continue
                req = max([float(y[b]) / kmap[L] for b, L in enumerate(assign) if L != 16] + [0.0])
                best_tau = req if best_tau is None else min(best_tau, req)
            if flag:
                assert best_tau is None
                continue
            assert best_tau is not None and abs(best_tau - tau) <= 1e-12 * max(1.0, tau)
            for b in range(n - 1):
                if lv[b] != 16:
                    assert y[b] <= tau * kmap[int(lv[b])] * (1 + 1e-12)
                    lower = {2: 1, 4: 2, 8: 4}.get(int(lv[b]))
                    if lower:
                        assert y[b] > tau * kmap[lower] * (1 - 1e-12)     # the next lower rung does not suffice
        cands = sorted({0.0} | {float(y[b]) / kk for b in range(n) for kk in kmap.values()})
        if flag:
            assert all(bits(plan_for(t)) > budget_bits for t in cands)
            continue
        assert bits(lv) <= budget_bits and lv[-1] == 16
        assert list(lv) == plan_for(tau)
        assert all(bits(plan_for(t)) > budget_bits for t in cands if t < tau)    # tau is the smallest
        if mono:
            assert all(lv[b] <= lv[b + 1] for b in range(n - 2))


def test_rd_allocator_prefers_bits_for_heavy_wide_blocks():
    n = 32
    mass = np.full(n, 1e-4, np.float32)
    rng_b = np.full(n, 2.0, np.float32)
    mass[5] = 0.5
    lv, tau, flag = O.rd_allocate(mass, rng_b, 32, 32, False, 0, 3.0, 0, 0, None, 0)
    assert not flag and lv[5] == max(lv) and lv[5] > np.median(lv)
    prev = np.full(n, 2, np.int32)
    lv2, _, _ = O.rd_allocate(mass, rng_b, 32, 32, False, 0, 8.0, 0, 0, prev, 0)
    assert np.all(lv2 <= 2)                                       # never above the previous level


# ---- P10: GQA sharing (Sec. 3.1) ----------------------------------------------------------------
def test_gqa_sharing_equals_expanded_mha():
    cfg = small_cfg(n_q_heads=4, n_kv_heads=2, stair_tokens=(64, 64, 64, 64))
    k, v, q = rand_kv(cfg, 400)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v)
    out, _ = c.decode_attn(0, q)
    cfg_m = small_cfg(n_q_heads=4, n_kv_heads=4, stair_tokens=(64, 64, 64, 64))
    km = np.repeat(k, 2, axis=2)
    vm = np.repeat(v, 2, axis=2)
    cm = O.GradedCache(cfg_m)
    cm.append_demote(0, km, vm)
    outm, _ = cm.decode_attn(0, q)
    assert np.array_equal(out, outm)
    assert np.array_equal(c.streams[(0, 0, 1)].blocks[2].k_codes, cm.streams[(0, 0, 3)].blocks[2].k_codes)


# ---- P12 / P15: page scorer and top-k (Sec. 3.5) -------------------------------------------------
def test_quest_bound_and_selection():
    cfg = small_cfg(n_q_heads=4, n_kv_heads=2, page_tokens=16, stair_tokens=(128, 128, 128, 128))
    T = 1000
    k, v, q = rand_kv(cfg, T)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v)
    scores = c.quest_scores(0, q)
    n_pages = (T // 64) * 4
    for (b, h), sc in scores.items():
        assert len(sc) == n_pages            # only pages of closed blocks carry boxes
        for p in range(n_pages):
            blk = k[b, p * 16:(p + 1) * 16, h].astype(np.float64)
            best = max(float(np.max(blk @ q[b, h * 2 + j].astype(np.float64))) for j in range(2))
            assert sc[p] >= best - 1e-4 * (1 + abs(best))          # box score upper-bounds q.k
    # selecting every closed page = full graded attention over closed pages + tail
    sel_all = c.quest_select(0, q, 10 ** 9)
    full, _ = c.decode_attn(0, q)
    sparse, _ = c.decode_attn(0, q, sel_all)
    assert np.array_equal(full, sparse)
    # hard mask: a 2-page budget reads exactly those pages plus the tail
    sel = c.quest_select(0, q, 32)
    st = c.streams[(0, 0, 0)]
    m = c.token_mask(st, sel[0][0])
    assert m.sum() == 32 + (T - (T // 64) * 64) and m[(T // 64) * 64:].all()
    assert list(sel[0][0]) == sorted(sel[0][0])


def test_topk_ties_prefer_lower_index_and_emit_ascending():
    s = np.array([1.0, 5.0, 5.0, 0.0, 5.0, -0.0, 2.0], dtype=np.float32)
    assert list(O.topk_ascending(s, 2)) == [1, 2]
    assert list(O.topk_ascending(s, 4)) == [1, 2, 4, 6]
    assert list(O.topk_ascending(s, 6)) == [0, 1, 2, 3, 4, 6]      # +0 at 3 beats -0 at 5 only by index
    assert list(O.topk_ascending(s, 100)) == list(range(7))


# ---- P13: exact residual (Sec. 3.4, Eq. 6) -------------------------------------------------------
def test_rd_residual_selection():
    cfg = small_cfg(n_q_heads=2, n_kv_heads=1, policy=O.POLICY_EXTERNAL, residual_fraction=0.01)
    T = 640
    k, v, q = rand_kv(cfg, T)
    mass = (RNG.random((1, 1, T)) * 1e-3).astype(np.float32)
    mass[0, 0, 100] = 0.5
    v[0, 100, 0] = bf(v[0, 100, 0] + 6.0)                          # highly attended and far from its centroid
    mass[0, 0, 200:264] = 0.0                                      # zero-mass tokens never outrank positives
    plan = np.full((1, 1, 10), 4, dtype=np.int8)
    plan[0, 0, 9] = 16                                             # exact blocks are not eligible
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v, token_mass=mass, level_plan=plan)
    st = c.streams[(0, 0, 0)]
    assert len(st.res_idx) == 6 and 100 in st.res_idx
    assert not any(200 <= j < 264 for j in st.res_idx) and not any(j >= 576 for j in st.res_idx)
    # a brute-force ranking by a_j * ||v_j - centroid||^2 agrees
    sc = []
    for j in range(576):
        blk = v[0, (j // 64) * 64:(j // 64 + 1) * 64, 0]
        cen = O.centroid_of(blk).astype(np.float64)
        sc.append(float(mass[0, 0, j]) * float(np.sum((v[0, j, 0].astype(np.float64) - cen) ** 2)))
    want = sorted(sorted(range(576), key=lambda j: (-sc[j], j))[:6])
    assert list(st.res_idx) == want
    # residual rows are served exactly: with every eligible token exact the output equals all-exact
    cfg_all = small_cfg(n_q_heads=2, n_kv_heads=1, policy=O.POLICY_EXTERNAL, residual_fraction=1.0)
    ca = O.GradedCache(cfg_all)
    ca.append_demote(0, k, v, token_mass=mass + np.float32(1e-6), level_plan=plan)
    ce = O.GradedCache(small_cfg(n_q_heads=2, n_kv_heads=1, stair_tokens=(-1, 0, 0, 0)))
    ce.append_demote(0, k, v)
    assert np.max(np.abs(ca.decode_attn(0, q)[0] - ce.decode_attn(0, q)[0])) < 1e-12


# ---- P14: the attention error certificate holds (Sec. 3.6, Eq. 9) ---------------------------------
def test_error_certificate_holds():
    cfg = small_cfg(n_q_heads=2, n_kv_heads=1, stair_tokens=(64, 128, 128, 128))
    T = 640
    k, v, q = rand_kv(cfg, T)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v)
    ce = O.GradedCache(small_cfg(n_q_heads=2, n_kv_heads=1, stair_tokens=(-1, 0, 0, 0)))
    ce.append_demote(0, k, v)
    o_hat, _, w_hat = c.decode_attn(0, q, return_weights=True)
    o, _ = ce.decode_attn(0, q)
    st = c.streams[(0, 0, 0)]
    Kh, Vh = c.reconstruct(st)
    for h in range(2):
        qq = q[0, h].astype(np.float64)
        dl = np.abs((Kh - k[0, :, 0]) @ qq) * c.scale
        dvn = np.linalg.norm(Vh - v[0, :, 0], axis=1)
        nb = T // 64
        a_b = [w_hat[(0, h)][i * 64:(i + 1) * 64].sum() for i in range(nb)]
        eps_b = [dl[i * 64:(i + 1) * 64].max() for i in range(nb)]
        dv_b = [dvn[i * 64:(i + 1) * 64].max() for i in range(nb)]
        bound = O.certificate_bound(a_b, eps_b, dv_b, float(np.linalg.norm(v[0, :, 0], axis=1).max()))
        err = float(np.linalg.norm(o[0, h] - o_hat[0, h]))
        assert err <= bound
        assert err > 0


# ---- staircase policy widths (Sec. 3.2 retire_after reading; Fig. 1 sinks) -------------------------
def test_staircase_levels():
    lv = O.staircase_levels(10, (128, 128, 64, 128), 0)
    assert list(lv) == [1, 1, 1, 2, 2, 4, 8, 8, 16, 16]
    lv = O.staircase_levels(10, (128, 128, 64, 128), 2)
    assert list(lv[:2]) == [16, 16]
    assert list(O.staircase_levels(3, (-1, 0, 0, 0), 0)) == [16, 16, 16]


# ---- block attention mass and its running average (Sec. 3.1, Eq. 2) ---------------------------
def test_block_mass_bruteforce_and_partition_of_unity():
    """a_b against softmax written out with scalar loops; masses of a stream sum to one; with
    identical keys a block's mass is its share of the tokens (closed form)."""
    cfg = small_cfg(n_q_heads=4, n_kv_heads=2, d_k=32, d_v=32, stair_tokens=(64, 64, 0, 0))
    T = 3 * 64 + 17                                   # exact, 8-bit, centroid blocks and a partial block
    k, v, q = rand_kv(cfg, T)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v)
    assert list(c.levels(0, 0, 0)) == [1, 8, 16]
    _, _, obs = c.decode_attn_observe(0, q)
    sc = float(np.float32(1.0 / math.sqrt(32)))
    for h_kv in range(2):
        a = obs[(0, h_kv)]
        assert a.shape == (4,)
        assert abs(a.sum() - 1.0) < 1e-12
        K, _ = c.reconstruct(c.streams[(0, 0, h_kv)])
        want = [0.0] * 4
        for j in range(2):                            # the two query heads of this KV head
            hq = 2 * h_kv + j
            logits = [sc * math.fsum(float(q[0, hq, d]) * float(K[t, d]) for d in range(32)) for t in range(T)]
            m = max(logits)
            e = [math.exp(x - m) for x in logits]
            z = math.fsum(e)
            for t in range(T):
                want[t // 64] += e[t] / z / 2
        assert np.max(np.abs(a - np.array(want))) < 1e-13
    # identical keys -> uniform weights -> mass = tokens of the block / T
    k2 = np.repeat(k[:, :1], T, axis=1)
    c2 = O.GradedCache(small_cfg(n_q_heads=4, n_kv_heads=2, d_k=32, d_v=32, stair_tokens=(-1, 0, 0, 0)))
    c2.append_demote(0, k2, v)
    _, _, obs2 = c2.decode_attn_observe(0, q)
    assert np.max(np.abs(obs2[(0, 1)] - np.array([64, 64, 64, 17]) / T)) < 1e-13


def test_block_mass_counts_residual_tokens_for_their_block_and_ema_closed_form():
    cfg = small_cfg(n_q_heads=2, n_kv_heads=1, d_k=32, d_v=32, policy=O.POLICY_RD, rd_budget_bpv=4.0,
                    residual_fraction=0.05, retire_after=64)
    T = 4 * 64
    k, v, q = rand_kv(cfg, T)
    mass = np.abs(RNG.standard_normal((1, 1, T))).astype(np.float32)
    mass /= mass.sum()
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v, token_mass=mass)
    st = c.streams[(0, 0, 0)]
    assert len(st.res_idx) == int(0.05 * T)
    # the running mass starts from the prefill observer's block masses
    m0 = st.ema_mass.copy()
    assert np.allclose(m0, mass[0, 0].reshape(4, 64).sum(axis=1), rtol=1e-6)
    out, lse, w = c.decode_attn(0, q, None, return_weights=True)
    _, _, obs = c.decode_attn_observe(0, q)
    a = obs[(0, 0)]
    # residual tokens are part of the dense weights, so the block sums need no special case ...
    want = sum(w[(0, j)].reshape(4, 64).sum(axis=1) for j in range(2)) / 2
    assert np.max(np.abs(a - want)) < 1e-14
    # ... and a block's mass includes the weight of its exact residual tokens
    blk = int(st.res_idx[0]) // 64
    in_blk = [int(t) for t in st.res_idx if int(t) // 64 == blk]
    assert a[blk] >= sum(w[(0, 0)][t] + w[(0, 1)][t] for t in in_blk) / 2
    # n identical observations: m = 0.9^n m0 + (1 - 0.9^n) a
    for _ in range(4):
        c.decode_attn_observe(0, q)
    n = 5
    assert np.max(np.abs(st.ema_mass - (0.9 ** n * m0 + (1 - 0.9 ** n) * a))) < 1e-13


def test_block_mass_of_new_blocks_starts_from_zero():
    cfg = small_cfg(n_q_heads=2, n_kv_heads=1, d_k=8, d_v=8, stair_tokens=(-1, 0, 0, 0))
    k, v, q = rand_kv(cfg, 64 + 3)
    c = O.GradedCache(cfg)
    c.append_demote(0, k[:, :60], v[:, :60])
    st = c.streams[(0, 0, 0)]
    _, _, obs = c.decode_attn_observe(0, q)
    assert obs[(0, 0)].shape == (1,) and abs(obs[(0, 0)][0] - 1.0) < 1e-13
    assert abs(st.ema_mass[0] - 0.1) < 1e-15
    for t in range(60, 67):
        c.append_demote(0, k[:, t:t + 1], v[:, t:t + 1])
    _, _, obs = c.decode_attn_observe(0, q)
    a = obs[(0, 0)]
    assert a.shape == (2,)
    assert abs(st.ema_mass[0] - (0.9 * 0.1 + 0.1 * a[0])) < 1e-15 and abs(st.ema_mass[1] - 0.1 * a[1]) < 1e-15


def test_decode_time_reallocation_keeps_the_temporal_constraint():
    """Re-running the allocator on running masses (Sec. 3.1-3.3): no level rises, the recent window
    and new blocks inside it stay exact, a block leaving the window gets a level, the budget of the
    grown context holds, and requantisation starts from the block's current representation."""
    cfg = small_cfg(n_q_heads=2, n_kv_heads=1, d_k=32, d_v=32, policy=O.POLICY_RD, rd_budget_bpv=5.0, retire_after=128,
                    max_ctx=4096)
    T = 8 * 64
    k, v, q = rand_kv(cfg, T + 130)
    mass = np.abs(RNG.standard_normal((1, 1, T))).astype(np.float32)
    mass /= mass.sum()
    c = O.GradedCache(cfg)
    c.append_demote(0, k[:, :T], v[:, :T], token_mass=mass)
    st = c.streams[(0, 0, 0)]
    before = c.levels(0, 0, 0).copy()
    assert list(before[-2:]) == [16, 16] and len(st.range_b) == 8
    for t in range(T, T + 130):
        c.decode_attn_observe(0, q)
        c.append_demote(0, k[:, t:t + 1], v[:, t:t + 1])
    assert st.n_closed == 10 and len(st.range_b) == 10
    mid = c.levels(0, 0, 0).copy()
    assert np.array_equal(mid[:8], before) and list(mid[8:]) == [16, 16]      # appends alone change nothing under RD
    recon_before = st.blocks[7].recon_k().copy()
    plans = c.rd_reallocate(0)
    after = c.levels(0, 0, 0)
    assert np.array_equal(after, plans[(0, 0)])
    assert np.all(after <= mid)
    assert list(after[-2:]) == [16, 16]                                        # the new recent window
    assert after[6] < 16 or after[7] < 16 or st.budget_flag                    # blocks that left it were allocated
    bits = sum(O.block_bits(int(L), 32, 32, False) for L in after) + st.n_tail * 16 * 64
    assert st.budget_flag or bits <= math.floor(float(np.float32(5.0)) * st.ctx * 64)
    if after[7] < 16:
        # block 7 was exact: its new codes quantise those exact rows
        blk, _ = O.make_block(int(after[7]), k[0, 7 * 64:8 * 64, 0], v[0, 7 * 64:8 * 64, 0])
        assert np.array_equal(blk.recon_k(), st.blocks[7].recon_k()) and not np.array_equal(recon_before, st.blocks[7].recon_k())
    # a second run on the same masses changes nothing (the plan is a fixed point)
    c.rd_reallocate(0)
    assert np.array_equal(c.levels(0, 0, 0), after)


def test_carried_error_bounds_and_runtime_certificate():
    """The per-block bounds carried through requantisation (Sec. 3.6) really bound the distance to
    the ORIGINAL rows, equal it for a block encoded once, and the certificate built from them
    (a) agrees with Eq. 9 evaluated by the stand-alone helper and (b) bounds the true output error
    against dense attention on the original cache, with demotions and residual rows in play."""
    cfg = small_cfg(n_q_heads=4, n_kv_heads=2, stair_tokens=(64, 64, 64, 64))
    T = 5 * 64 + 9
    k, v, q = rand_kv(cfg, T + 70)
    c = O.GradedCache(cfg)
    c.append_demote(0, k[:, :T], v[:, :T])
    for t in range(T, T + 70):                              # one more block closes: every block moves a rung
        c.append_demote(0, k[:, t:t + 1], v[:, t:t + 1])
    dense = O.GradedCache(small_cfg(n_q_heads=4, n_kv_heads=2, stair_tokens=(-1, 0, 0, 0)))
    dense.append_demote(0, k, v)
    o_true, _ = dense.decode_attn(0, q)
    o_hat, _, w_hat = c.decode_attn(0, q, return_weights=True)
    cert = c.certificate(0, q)
    for h_kv in range(2):
        st = c.streams[(0, 0, h_kv)]
        assert [b.level for b in st.blocks] == [1, 1, 2, 4, 8, 16]
        for i, blk in enumerate(st.blocks):
            k0, v0 = k[0, i * 64:(i + 1) * 64, h_kv].astype(np.float64), v[0, i * 64:(i + 1) * 64, h_kv].astype(np.float64)
            true_k = np.linalg.norm(k0 - blk.recon_k(), axis=1).max()
            true_v = np.linalg.norm(v0 - blk.recon_v(), axis=1).max()
            assert true_k <= blk.kappa * (1 + 1e-12) and true_v <= blk.delta * (1 + 1e-12)
            assert abs(blk.vnorm - np.linalg.norm(v0, axis=1).max()) < 1e-12
            if len(blk.history) == 1:                     # encoded once from the original rows: the bound is the distance
                assert abs(true_k - blk.kappa) < 1e-12 and abs(true_v - blk.delta) < 1e-12
        assert st.blocks[-1].kappa == 0.0 and st.blocks[-1].delta == 0.0
        assert st.blocks[1].history == [2, 1] and st.blocks[2].history == [4, 2] and st.blocks[1].kappa > 0
        for j in range(2):
            hq = 2 * h_kv + j
            w = w_hat[(0, hq)]
            n = st.n_closed
            qn = np.linalg.norm(q[0, hq].astype(np.float64))
            a_b = [w[i * 64:(i + 1) * 64].sum() for i in range(n)] + [w[n * 64:].sum()]
            eps_b = [c.scale * qn * blk.kappa for blk in st.blocks] + [0.0]
            dv_b = [blk.delta for blk in st.blocks] + [0.0]
            vmax = float(np.linalg.norm(v[0, :, h_kv].astype(np.float64), axis=1).max())
            want = O.certificate_bound(a_b, eps_b, dv_b, vmax)
            assert abs(cert[0, hq] - want) < 1e-12 * max(1.0, want)
            err = float(np.linalg.norm(o_true[0, hq] - o_hat[0, hq]))
            assert 0 < err <= cert[0, hq]


def test_certificate_is_zero_for_an_exact_cache_and_ignores_exact_residual_rows():
    cfg = small_cfg(n_q_heads=2, n_kv_heads=1, stair_tokens=(-1, 0, 0, 0))
    k, v, q = rand_kv(cfg, 200)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v)
    assert np.all(c.certificate(0, q) == 0.0)
    # residual rows are exact: their weight enters M+ and M- with eps = 0 and adds nothing to the first term
    cfg2 = small_cfg(n_q_heads=2, n_kv_heads=1, policy=O.POLICY_RD, rd_budget_bpv=3.0, residual_fraction=0.25, retire_after=0)
    mass = np.abs(RNG.standard_normal((1, 1, 256))).astype(np.float32)
    k3, v3, q3 = rand_kv(cfg2, 256)
    c3 = O.GradedCache(cfg2)
    c3.append_demote(0, k3, v3, token_mass=mass)
    st = c3.streams[(0, 0, 0)]
    assert len(st.res_idx) == 64
    c_with = c3.certificate(0, q3)
    no_res = O.GradedCache(small_cfg(n_q_heads=2, n_kv_heads=1, policy=O.POLICY_EXTERNAL))
    no_res.append_demote(0, k3, v3, level_plan=c3.levels(0, 0, 0)[None, None])
    c_without = no_res.certificate(0, q3)
    dense = O.GradedCache(small_cfg(n_q_heads=2, n_kv_heads=1, stair_tokens=(-1, 0, 0, 0)))
    dense.append_demote(0, k3, v3)
    o_true, _ = dense.decode_attn(0, q3)
    o_hat, _ = c3.decode_attn(0, q3)
    for h in range(2):
        assert np.linalg.norm(o_true[0, h] - o_hat[0, h]) <= c_with[0, h]
    assert np.all(c_with > 0) and np.all(c_without > 0)


# ---- Sec. 3.5 Eq. 8: bits a page-list read touches, written out by hand -------------------------
def test_page_list_read_bits_by_hand():
    """d_k = d_v = 32, 16-token pages, 64-token blocks, groups of 32: every term of the read cost of
    a page list, counted by hand for one stream whose six closed blocks sit on known rungs."""
    D = 32
    cfg = small_cfg(n_q_heads=1, n_kv_heads=1, d_k=D, d_v=D, page_tokens=16, policy=O.POLICY_EXTERNAL)
    T = 6 * 64 + 5                                    # six closed blocks and a partial block of 5 tokens
    k, v, q = rand_kv(cfg, T)
    plan = np.array([[[4, 1, 16, 8, 2, 1]]], dtype=np.int8)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v, level_plan=plan)
    nval = 2 * D                                      # values per token
    tail = 5 * 16 * nval                              # the partial block is always read, exact

    def read(pages):
        c.decode_attn(0, q, [[np.array(pages, dtype=np.int32)]])
        return c.bits_report(0)["last_read_bits"]

    codes4 = 16 * nval * 4                            # one page of 4-bit codes (keys and values)
    vpar = 16 * (D // 32) * 32                        # value params: one group of 32 channels per token
    kgrp = D * 32                                     # key params of one 32-token group: D channels x (scale + zero)
    # one page of the int4 block 0
    assert read([0]) == codes4 + vpar + kgrp + tail == 4096 + 512 + 1024 + tail
    # pages 0 and 1 share one 32-token key group: its params are read once
    assert read([0, 1]) == 2 * (codes4 + vpar) + kgrp + tail
    # pages 0 and 2 lie in different halves of the block: two key groups
    assert read([0, 2]) == 2 * (codes4 + vpar) + 2 * kgrp + tail
    # a centroid block (block 1 = pages 4..7) costs its two centroid rows once, however many pages
    cent = 16 * nval
    assert read([4]) == cent + tail
    assert read([4, 5, 7]) == cent + tail
    # an exact block (block 2 = pages 8..11): 16 bits per value of the page, no params
    assert read([9]) == 16 * nval * 16 + tail
    # int8 block 3 (pages 12..15) and int2 block 4 (pages 16..19)
    assert read([12]) == 16 * nval * 8 + vpar + kgrp + tail
    assert read([16, 17, 18, 19]) == 4 * (16 * nval * 2 + vpar) + 2 * kgrp + tail
    # everything mixed: the sum of the parts (block 5 is a second centroid block: pages 20..23)
    assert read([0, 1, 5, 9, 12, 19, 22]) == (2 * (codes4 + vpar) + kgrp) + cent + 16 * nval * 16 + (16 * nval * 8 + vpar + kgrp) \
        + (16 * nval * 2 + vpar + kgrp) + cent + tail
    # selecting every page of a quantised block reads the whole block: codes + all params
    whole4 = 64 * nval * 4 + (64 * nval // 32) * 32
    assert read([0, 1, 2, 3]) == whole4 + tail
    # an empty list reads the partial block only
    assert read([]) == tail


# ---- Sec. 3.5 page score with the sum over the KV head's query heads -----------------------------
def test_quest_scores_sum_reduction():
    """The flag variant of the page score (sum instead of max over the g query heads): scalar fp32
    loops in the stated order (channels ascending, then heads ascending), the upper-bound property
    head by head, and g = 1 where sum and max coincide."""
    cfg_sum = small_cfg(n_q_heads=6, n_kv_heads=2, page_tokens=16, stair_tokens=(-1, 0, 0, 0), quest_reduce=O.REDUCE_SUM)
    T = 330
    k, v, q = rand_kv(cfg_sum, T)
    c = O.GradedCache(cfg_sum)
    c.append_demote(0, k, v)
    scores = c.quest_scores(0, q)
    g = 3
    n_pages = (T // 64) * 4
    f32 = np.float32
    for (b, h), sc in scores.items():
        assert len(sc) == n_pages and sc.dtype == np.float32
        for p in range(n_pages):
            page = k[b, 16 * p:16 * p + 16, h]                        # bf16 values
            lo, hi = page.min(axis=0), page.max(axis=0)
            total = None
            bound = 0.0
            for j in range(g):
                qh = q[b, h * g + j]
                acc = f32(0.0)
                for d in range(cfg_sum.d_k):
                    acc = f32(acc + f32(qh[d]) * f32(hi[d] if qh[d] >= 0 else lo[d]))     # the product is exact in fp32
                total = acc if total is None else f32(total + acc)
                bound += float(np.max(page.astype(np.float64) @ qh.astype(np.float64)))
            assert sc[p] == total, (b, h, p)
            assert sc[p] >= bound - 1e-4 * (1 + abs(bound))           # sum of per-head upper bounds
    # one query head per KV head: nothing to reduce, sum == max
    for red in (O.REDUCE_SUM, O.REDUCE_MAX):
        cfg1 = small_cfg(n_q_heads=2, n_kv_heads=2, page_tokens=16, stair_tokens=(-1, 0, 0, 0), quest_reduce=red)
        c1 = O.GradedCache(cfg1)
        c1.append_demote(0, k, v)
        s1 = c1.quest_scores(0, q[:, :2])
        if red == O.REDUCE_SUM:
            keep = s1
        else:
            for key in s1:
                assert np.array_equal(s1[key], keep[key])
    # the selection follows the summed score
    sel = c.quest_select(0, q, 64)
    for (b, h), sc in scores.items():
        assert list(sel[b][h]) == sorted(np.argsort(-sc.astype(np.float64), kind="stable")[:4].tolist())


def test_page_list_with_residual_tokens_masks_cold_pages_and_counts_listed_rows():
    """Sec. 3.4 + 3.5 together: exact residual tokens of pages that are not listed are masked like
    the rest of their page; those of listed pages are read exact.  Checked against dense attention
    over hand-built rows, and the read bits against a count by hand."""
    D = 32
    cfg = small_cfg(n_q_heads=2, n_kv_heads=1, d_k=D, d_v=D, page_tokens=16, policy=O.POLICY_EXTERNAL, residual_fraction=0.05)
    T = 4 * 64 + 3
    k, v, q = rand_kv(cfg, T)
    mass = RNG.random((1, 1, T)).astype(np.float32)
    plan = np.array([[[4, 1, 2, 8]]], dtype=np.int8)
    c = O.GradedCache(cfg)
    c.append_demote(0, k, v, token_mass=mass, level_plan=plan)
    st = c.streams[(0, 0, 0)]
    res = [int(t) for t in st.res_idx]
    assert len(res) == int(0.05 * T) and len(res) >= 8
    pages = sorted(set([res[0] // 16, res[3] // 16, 5]))            # two pages holding residual tokens and page 5
    out, _ = c.decode_attn(0, q, [[np.array(pages, dtype=np.int32)]])
    # dense attention over exactly the readable rows: listed pages (residual tokens exact, the others
    # reconstructed) and the partial block
    K, V = c.reconstruct(st)
    rows = [t for pg in pages for t in range(16 * pg, 16 * pg + 16)] + list(range(256, T))
    for t in rows:
        if t in res:
            assert np.array_equal(K[t], k[0, t, 0].astype(np.float64)) and np.array_equal(V[t], v[0, t, 0].astype(np.float64))
    for h in range(2):
        w = np.exp(K[rows] @ q[0, h].astype(np.float64) * c.scale)      # the oracle's softmax scale (fp32 1/sqrt(d))
        ref = (w[:, None] * V[rows]).sum(0) / w.sum()
        assert np.abs(out[0, h] - ref).max() < 1e-12, np.abs(out[0, h] - ref).max()
    # read bits: the pages' own cost plus 16 bits per value for every residual row on a listed page
    n_listed = sum(1 for t in res if t // 16 in pages)
    assert n_listed >= 2
    with_res = c.bits_report(0)["last_read_bits"]
    c2 = O.GradedCache(small_cfg(n_q_heads=2, n_kv_heads=1, d_k=D, d_v=D, page_tokens=16, policy=O.POLICY_EXTERNAL))
    c2.append_demote(0, k, v, level_plan=plan)
    c2.decode_attn(0, q, [[np.array(pages, dtype=np.int32)]])
    assert with_res == c2.bits_report(0)["last_read_bits"] + n_listed * 16 * 2 * D
