"""Full-size parity: the configurations of the benchmark spec at their real shapes, in the launch
configuration bench.py times (all sequences and KV heads of a layer in one call), checked against
the oracle on a sample of streams (the oracle is run on those streams only) plus properties that
hold at any size.  Inputs are drawn on the GPU with the same recipe and copied to the host for the
oracle."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import gkv_oracle as O
from paper_2608_23599_b200 import workloads as W
import parity_util as U

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2608_23599_b200 import binding as B
    B.build()
    return B


def _sample_oracle(w, data, streams, n_layers=1):
    """Oracle cache holding only the sampled (b, kv head) streams of one layer: they become KV heads
    0..n-1 of a batch-1 cache with the matching query heads."""
    g = w.group_size
    cfg = U.oracle_config(dataclasses.replace(w, batch=1, n_kv_heads=len(streams), n_q_heads=g * len(streams)), n_layers)
    k = torch.stack([data["k"][b, :, h] for b, h in streams], dim=1)[None]
    v = torch.stack([data["v"][b, :, h] for b, h in streams], dim=1)[None]
    q = torch.cat([data["q"][b, h * g:(h + 1) * g] for b, h in streams], dim=0)[None]
    mass = None
    if data.get("mass") is not None:
        mass = torch.stack([data["mass"][b, h] for b, h in streams], dim=0)[None].cpu().numpy()
    return O.GradedCache(cfg), U.f32(k), U.f32(v), U.f32(q), mass


def _compare_blocks(B, gcache, ocache, layer, streams, blocks):
    for j, (b, h) in enumerate(streams):
        st = ocache.streams[(layer, 0, j)]
        assert np.array_equal(gcache.gkv_debug_export_levels(layer, b, h), ocache.levels(layer, 0, j))
        assert np.array_equal(gcache.gkv_debug_export_residual(layer, b, h), st.res_idx)
        for i in blocks:
            if i >= st.n_closed:
                continue
            blk = st.blocks[i]
            for which, name in ((B.TENSOR_K, "k"), (B.TENSOR_V, "v")):
                ex = gcache.gkv_debug_export_block(layer, b, h, i, which)
                tag = f"stream {(b, h)} block {i} {name} level {blk.level}"
                assert ex["level"] == blk.level, tag
                if blk.level == 16:
                    assert np.array_equal(ex["rows"], O.bf16_bits(getattr(blk, f"{name}_exact"))), tag
                elif blk.level == 1:
                    assert np.array_equal(ex["rows"][0], O.bf16_bits(getattr(blk, f"{name}_cent"))), tag
                else:
                    assert np.array_equal(ex["scale"], getattr(blk, f"{name}_scale").view(np.uint16)), tag
                    assert np.array_equal(ex["zero"], getattr(blk, f"{name}_zero").view(np.uint16)), tag
                    assert np.array_equal(ex["codes"], getattr(blk, f"{name}_codes")), tag


def _heads_of(streams, g, n_kv):
    return [(b, h * g + j) for b, h in streams for j in range(g)]


def _assert_sampled_outputs(out_gpu, o_out, streams, g, what):
    got = torch.stack([out_gpu[b, hq] for b, hq in _heads_of(streams, g, None)], dim=0)[None]
    return U.assert_outputs_close(got, o_out, what)


def test_cfg2_full_size_sampled_streams_with_appends():
    """Config 2 at full size (B=8, 32/8 heads, T=32768, one layer): bulk ingest, then 65 decode
    steps (one block fill with the four staircase demotions)."""
    B = _binding()
    w = dataclasses.replace(W.config(2), n_layers=1)
    gcache = B.Cache(B.config_from_workload(w, 1))
    dev = gcache.device
    data = W.make_layer(w, 0, dev)
    gcache.gkv_append_demote(0, data["k"], data["v"])
    streams = [(0, 0), (3, 5), (7, 7)]
    ocache, k, v, q, _ = _sample_oracle(w, data, streams)
    ocache.append_demote(0, k, v)
    blocks = [0, 1, 47, 48, 49, 175, 176, 300, 431, 432, 433, 495, 496, 511]      # every rung and its borders
    _compare_blocks(B, gcache, ocache, 0, streams, blocks)
    out = torch.empty((w.batch, w.n_q_heads, 128), dtype=torch.float32, device=dev)
    gcache.gkv_decode_attn(0, data["q"], out)
    torch.cuda.synchronize()
    o_out, _ = ocache.decode_attn(0, q)
    err, rel = _assert_sampled_outputs(out, o_out, streams, w.group_size, "cfg2 full step 0")
    print(f"cfg2 full: max-abs error {err:.2e}, relative L2 {rel:.2e}")
    # no NaN anywhere and every head's output is a convex combination of bounded values
    assert torch.isfinite(out).all() and float(out.abs().max()) < 50
    rep = gcache.gkv_bits_report(0)
    assert abs(rep.bpv_resident - 4.8984375) < 1e-9 and rep.last_read_bits == rep.resident_bits
    g = torch.Generator(device=dev)
    g.manual_seed(99)
    for step in range(65):
        kn = torch.randn((w.batch, 1, w.n_kv_heads, 128), generator=g, device=dev).to(torch.bfloat16)
        vn = torch.randn((w.batch, 1, w.n_kv_heads, 128), generator=g, device=dev).to(torch.bfloat16)
        qn = torch.randn((w.batch, w.n_q_heads, 128), generator=g, device=dev).to(torch.bfloat16)
        gcache.gkv_append_demote(0, kn, vn)
        sub = {"k": kn, "v": vn, "q": qn}
        ks = torch.stack([kn[b, :, h] for b, h in streams], dim=1)[None]
        vs = torch.stack([vn[b, :, h] for b, h in streams], dim=1)[None]
        ocache.append_demote(0, U.f32(ks), U.f32(vs))
        if step in (0, 62, 63, 64):
            gcache.gkv_decode_attn(0, qn, out)
            torch.cuda.synchronize()
            qs = torch.cat([qn[b, h * 4:(h + 1) * 4] for b, h in streams], dim=0)[None]
            o_out, _ = ocache.decode_attn(0, U.f32(qs))
            _assert_sampled_outputs(out, o_out, streams, w.group_size, f"cfg2 full step {step + 1}")
    # after the block fill: the demoted blocks (one per rung border) are bit-exact
    _compare_blocks(B, gcache, ocache, 0, streams, [48, 176, 432, 496, 497, 512])
    assert gcache.gkv_ctx_len(0) == 32768 + 65
    for j in range(len(streams)):
        for blk in ocache.streams[(0, 0, j)].blocks:
            assert all(a >= b for a, b in zip(blk.history, blk.history[1:]))      # monotone demotion
    # the observing call at full size: same output bits, block masses and certificate of the sampled streams
    n_items = (gcache.gkv_ctx_len(0) + 63) // 64
    mass = torch.full((w.batch, w.n_kv_heads, n_items), -1.0, dtype=torch.float32, device=dev)
    cert = torch.full((w.batch, w.n_q_heads), -1.0, dtype=torch.float32, device=dev)
    out2 = torch.empty_like(out)
    gcache.gkv_decode_attn_observe(0, qn, out2, None, mass, cert)
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    mass_h, cert_h = mass.cpu().numpy().astype(np.float64), cert.cpu().numpy().astype(np.float64)
    assert np.all(mass_h >= 0) and np.allclose(mass_h.sum(-1), 1.0, atol=2e-3)
    assert np.all(np.isfinite(cert_h)) and np.all(cert_h > 0)
    _, _, o_obs = ocache.decode_attn_observe(0, U.f32(qs))
    o_cert = ocache.certificate(0, U.f32(qs))
    for j, (b, h) in enumerate(streams):
        want = o_obs[(0, j)]
        assert np.allclose(mass_h[b, h], want, rtol=1e-2, atol=2e-6), (b, h, float(np.abs(mass_h[b, h] - want).max()))
        assert np.allclose(cert_h[b, h * 4:(h + 1) * 4], o_cert[0, j * 4:(j + 1) * 4], rtol=1e-2, atol=1e-5)
    gcache.close()


def test_cfg1_full_size_rd_and_residual_sampled():
    """Config 1 at full size (16/2 heads, T=16384, RD allocator + 1 % residual; the budget is fitted so that the
    36 layers realise 4.84 + 0.16 = 5.0 bits/value on average), two layers:
    every stream is checked (there are only two per layer)."""
    B = _binding()
    w = dataclasses.replace(W.config(1), n_layers=2)
    gcache = B.Cache(B.config_from_workload(w, 2))
    dev = gcache.device
    for layer in range(2):
        data = W.make_layer(w, layer, dev)
        gcache.gkv_append_demote(layer, data["k"], data["v"], token_mass=data["mass"])
        streams = [(0, 0), (0, 1)]
        ocache, k, v, q, mass = _sample_oracle(w, data, streams)
        ocache.append_demote(0, k, v, token_mass=mass)
        # the oracle cache is layer 0 of its own; compare against `layer` of the GPU cache
        for j, (b, h) in enumerate(streams):
            st = ocache.streams[(0, 0, j)]
            assert np.array_equal(gcache.gkv_debug_export_levels(layer, b, h), ocache.levels(0, 0, j))
            res = gcache.gkv_debug_export_residual(layer, b, h)
            assert len(res) == 163 and np.array_equal(res, st.res_idx)
        lv = ocache.levels(0, 0, 0)
        assert len(set(lv.tolist())) >= 3
        nb = len(lv)
        picks = sorted(set([0, 1, nb // 4, nb // 2, nb - 9, nb - 8, nb - 1]))
        for j, (b, h) in enumerate(streams):
            for i in picks:
                blk = ocache.streams[(0, 0, j)].blocks[i]
                ex = gcache.gkv_debug_export_block(layer, b, h, i, B.TENSOR_V)
                assert ex["level"] == blk.level
                if blk.level in (8, 4, 2):
                    assert np.array_equal(ex["codes"], blk.v_codes)
                    assert np.array_equal(ex["scale"], blk.v_scale.view(np.uint16))
        out = torch.empty((w.batch, w.n_q_heads, 128), dtype=torch.float32, device=dev)
        gcache.gkv_decode_attn(layer, data["q"], out)
        torch.cuda.synchronize()
        o_out, _ = ocache.decode_attn(0, q)
        err, rel = U.assert_outputs_close(out, o_out, f"cfg1 full layer {layer}")
        print(f"cfg1 full layer {layer}: max-abs error {err:.2e}, relative L2 {rel:.2e}")
        rep_g, rep_o = gcache.gkv_bits_report(layer), ocache.bits_report(0)
        assert rep_g.resident_bits == rep_o["resident_bits"]
        assert rep_g.bpv_paper <= w.rd_budget_bpv + 16 * 163 / 16384 + 1e-9
    gcache.close()


def test_cfg3_full_size_quest_sampled():
    """Config 3 at full size (B=4, 32/8 heads, T=32768, 16-token pages, budget 2048 tokens):
    selected pages bit-exact and sparse attention outputs on sampled streams."""
    B = _binding()
    w = dataclasses.replace(W.config(3), n_layers=1)
    gcache = B.Cache(B.config_from_workload(w, 1))
    dev = gcache.device
    data = W.make_layer(w, 0, dev)
    gcache.gkv_append_demote(0, data["k"], data["v"], token_mass=data["mass"])
    streams = [(0, 0), (2, 3), (3, 7)]
    ocache, k, v, q, mass = _sample_oracle(w, data, streams)
    ocache.append_demote(0, k, v, token_mass=mass)
    for j, (b, h) in enumerate(streams):
        assert np.array_equal(gcache.gkv_debug_export_levels(0, b, h), ocache.levels(0, 0, j))
    # boxes and page scores of the sampled streams, bit for bit (the oracle holds them as streams 0..2 of sequence 0)
    scores_g = gcache.gkv_debug_export_scores(0, data["q"])
    scores_o = ocache.quest_scores(0, q)
    for j, (b, h) in enumerate(streams):
        lo, hi = gcache.gkv_debug_export_boxes(0, b, h)
        st = ocache.streams[(0, 0, j)]
        assert np.array_equal(lo, O.bf16_bits(np.stack(st.box_lo))) and np.array_equal(hi, O.bf16_bits(np.stack(st.box_hi)))
        assert np.array_equal(scores_g[b, h].view(np.uint32), scores_o[(0, j)].view(np.uint32)), f"page scores of stream {(b, h)}"
    k_sel = w.quest_budget_tokens // w.page_tokens
    pages = torch.full((w.batch, w.n_kv_heads, k_sel), -1, dtype=torch.int32, device=dev)
    n_sel = gcache.gkv_quest_select(0, data["q"], w.quest_budget_tokens, pages)
    torch.cuda.synchronize()
    assert n_sel == k_sel == 128
    sel_o = ocache.quest_select(0, q, w.quest_budget_tokens)
    pg = pages.cpu().numpy()
    for j, (b, h) in enumerate(streams):
        assert np.array_equal(pg[b, h], sel_o[0][j]), f"pages differ for stream {(b, h)}"
    # properties for every stream: ascending, unique, in range
    assert (np.diff(pg, axis=-1) > 0).all() and pg.min() >= 0 and pg.max() < 2048
    out = torch.empty((w.batch, w.n_q_heads, 128), dtype=torch.float32, device=dev)
    gcache.gkv_decode_attn(0, data["q"], out, page_idx=pages, n_sel=n_sel)
    torch.cuda.synchronize()
    o_out, _ = ocache.decode_attn(0, q, sel_o)
    err, rel = _assert_sampled_outputs(out, o_out, streams, w.group_size, "cfg3 full sparse")
    print(f"cfg3 full: max-abs error {err:.2e}, relative L2 {rel:.2e}")
    assert torch.isfinite(out).all()
    gcache.close()


def test_cfg0_repeated_through_bench_sized_launches():
    """Config 0 is small enough to be checked in full in test_gpu_parity; here its launch is
    repeated with changing tail lengths (every value of ctx mod 64 after the ingest)."""
    B = _binding()
    w = dataclasses.replace(W.config(0), max_ctx=4096 + 192)
    ocache = O.GradedCache(U.oracle_config(w))
    gcache = B.Cache(B.config_from_workload(w))
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    worst = 0.0
    for step in range(70):
        tok = W.make_decode_tokens(w, 0, step, "cpu")
        ocache.append_demote(0, U.f32(tok["k"]), U.f32(tok["v"]))
        gcache.gkv_append_demote(0, tok["k"].to(dev), tok["v"].to(dev))
        if step % 7 == 0 or step in (62, 63, 64):
            out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, tok["q"])
            err, rel = U.assert_outputs_close(out, o_out, f"cfg0 step {step}")
            worst = max(worst, err)
    U.assert_state_equal(ocache, gcache, 0)
    print(f"cfg0 worst max-abs error over 70 steps: {worst:.2e}")
    gcache.close()


def test_cfg4_full_size_mla_one_million_tokens():
    """Config 4 at full size: MLA 576/512, 16 heads, 1,048,576 tokens, 5.0 bits/value ladder
    (newest 4096 exact, int8, int4, oldest quarter centroid).
    (a) sampled blocks of every rung are bit-exact against the oracle's per-block encoder;
    (b) property that holds at any size: the million-token result equals the log-sum-exp merge of
        four quarter caches that hold the same blocks at the same levels;
    (c) the newest quarter (exact + int8 rungs, 262,144 tokens, 4096 blocks) matches the oracle;
    (d) the two rungs that hold three quarters of the context: a 65,536-token window of the int4 rung, one
        of the centroid rung and one across the centroid / int4 border, read from caches that hold these
        windows at the exported levels, match the oracle on the same rows (outputs and log-sum-exp), and the
        merge of (b) ties the windows' quarters to the million-token result."""
    B = _binding()
    w = dataclasses.replace(W.config(4), n_layers=1)
    gcache = B.Cache(B.config_from_workload(w, 1))
    dev = gcache.device
    data = W.make_layer(w, 0, dev)
    k = data["k"]                                                    # [1][T][1][576]
    gcache.gkv_append_demote(0, k, None)
    T = w.ctx
    levels = gcache.gkv_debug_export_levels(0, 0, 0)
    assert len(levels) == T // 64
    rep = gcache.gkv_bits_report(0)
    assert abs(rep.bpv_resident - 5.0) < 1e-3
    assert list(rep.blocks_by_level) == [64, int((levels == 8).sum()), int((levels == 4).sum()), 0, 4096]
    out_full = torch.empty((1, 16, 512), dtype=torch.float32, device=dev)
    lse_full = torch.empty((1, 16), dtype=torch.float32, device=dev)
    gcache.gkv_decode_attn(0, data["q"], out_full, lse_full)
    torch.cuda.synchronize()
    assert torch.isfinite(out_full).all()
    # (a) sampled blocks, every rung and its borders
    nb = len(levels)
    b8 = int(np.argmax(levels == 8)); b4 = int(np.argmax(levels == 4))
    picks = sorted(set([0, 1, 4095, 4096, b4, b4 + 1, b8 - 1, b8, b8 + 1, nb - 65, nb - 64, nb - 1] +
                       list(range(37, nb, nb // 97))))
    kh = k[0, :, 0].cpu()
    for i in picks:
        blk, _ = O.make_block(int(levels[i]), U.f32(kh[i * 64:(i + 1) * 64]), None)
        ex = gcache.gkv_debug_export_block(0, 0, 0, i, B.TENSOR_K)
        assert ex["level"] == levels[i]
        if blk.level == 16:
            assert np.array_equal(ex["rows"], O.bf16_bits(blk.k_exact)), f"block {i}"
        elif blk.level == 1:
            assert np.array_equal(ex["rows"][0], O.bf16_bits(blk.k_cent)), f"block {i}"
        else:
            assert np.array_equal(ex["codes"], blk.k_codes), f"block {i} codes"
            assert np.array_equal(ex["scale"], blk.k_scale.view(np.uint16)) and np.array_equal(ex["zero"], blk.k_zero.view(np.uint16))
    # (b) four quarter caches with the same per-block levels, merged by their log-sum-exp
    Tq = T // 4
    wq = dataclasses.replace(w, ctx=Tq, max_ctx=Tq + 64, policy=W.POLICY_EXTERNAL)
    outs, lses = [], []
    newest = None
    for qi in range(4):
        qc = B.Cache(B.config_from_workload(wq, 1))
        plan = levels[qi * (Tq // 64):(qi + 1) * (Tq // 64)].astype(np.int8).reshape(1, 1, -1)
        qc.gkv_append_demote(0, k[:, qi * Tq:(qi + 1) * Tq].contiguous(), None, level_plan=plan)
        o = torch.empty_like(out_full); l = torch.empty_like(lse_full)
        qc.gkv_decode_attn(0, data["q"], o, l)
        torch.cuda.synchronize()
        outs.append(o.double()); lses.append(l.double())
        if qi == 3:
            newest = (o.clone(), l.clone())
        qc.close()
    L = torch.stack(lses); Mx = L.max(dim=0).values
    wts = torch.exp(L - Mx)
    merged = (torch.stack(outs) * wts[..., None]).sum(0) / wts.sum(0)[..., None]
    gap = float((merged - out_full.double()).abs().max())
    assert gap < 2e-4, f"million-token result differs from the merge of its quarters by {gap:.2e}"
    lse_merged = Mx + torch.log(wts.sum(0))
    assert float((lse_merged - lse_full.double()).abs().max()) < 1e-3
    # (c) oracle on the newest quarter (exact + int8 rungs)
    ocfg = U.oracle_config(wq, 1)
    oc = O.GradedCache(ocfg)
    plan = levels[3 * (Tq // 64):].astype(np.int8).reshape(1, 1, -1)
    oc.append_demote(0, U.f32(k[:, 3 * Tq:].cpu()), None, level_plan=plan)
    o_out, o_lse = oc.decode_attn(0, U.f32(data["q"]))
    err, rel = U.assert_outputs_close(newest[0], o_out, "cfg4 newest quarter")
    assert np.max(np.abs(newest[1].cpu().numpy() - o_lse)) < 5e-3
    print(f"cfg4 full: quarter-merge gap {gap:.2e}, newest-quarter max-abs error {err:.2e}, relative L2 {rel:.2e}")
    # (d) windows of the int4 and centroid rungs against the oracle
    first4 = int(np.argmax(levels == 4)) * 64                        # first token of the int4 rung (the centroid rung ends here)
    Wn = 65536
    wwin = dataclasses.replace(w, ctx=Wn, max_ctx=Wn + 64, policy=W.POLICY_EXTERNAL)
    for name, start in (("centroid rung", 1024 * 64), ("centroid / int4 border", first4 - Wn // 2), ("int4 rung", first4 + 2048 * 64)):
        lv = levels[start // 64:(start + Wn) // 64].astype(np.int8)
        assert set(np.unique(lv)) <= {1, 4}
        plan = lv.reshape(1, 1, -1)
        kw = k[:, start:start + Wn].contiguous()
        wc = B.Cache(B.config_from_workload(wwin, 1))
        wc.gkv_append_demote(0, kw, None, level_plan=plan)
        o = torch.empty_like(out_full); l = torch.empty_like(lse_full)
        wc.gkv_decode_attn(0, data["q"], o, l)
        torch.cuda.synchronize()
        oc = O.GradedCache(U.oracle_config(wwin, 1))
        oc.append_demote(0, U.f32(kw.cpu()), None, level_plan=plan)
        o_out, o_lse = oc.decode_attn(0, U.f32(data["q"]))
        err, rel = U.assert_outputs_close(o, o_out, f"cfg4 window in the {name}")
        assert np.max(np.abs(l.cpu().numpy() - o_lse)) < 5e-3
        # a few blocks of the window, bit for bit
        st = oc.streams[(0, 0, 0)]
        for i in (0, 511, 1023):
            ex = wc.gkv_debug_export_block(0, 0, 0, i, B.TENSOR_K)
            blk = st.blocks[i]
            assert ex["level"] == blk.level
            if blk.level == 1:
                assert np.array_equal(ex["rows"][0], O.bf16_bits(blk.k_cent))
            else:
                assert np.array_equal(ex["codes"], blk.k_codes) and np.array_equal(ex["scale"], blk.k_scale.view(np.uint16))
        print(f"cfg4 full: window in the {name}: max-abs error {err:.2e}, relative L2 {rel:.2e}")
        wc.close()
    gcache.close()
