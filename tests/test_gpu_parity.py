"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.
Discrete state (levels, codes, scale/zero, centroids, exact rows, residual indices, selected
pages, bit counts) must match bit for bit; fp32 attention outputs within max-abs 2e-3 and
relative L2 1e-2."""
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


def _pair(w, n_layers=None):
    B = _binding()
    ocache = O.GradedCache(U.oracle_config(w, n_layers))
    gcache = B.Cache(B.config_from_workload(w, n_layers))
    return ocache, gcache


def _tiny(T, **kw):
    base = dict(name="tiny", config_id=9, n_layers=1, batch=1, n_q_heads=8, n_kv_heads=2, d_k=128, d_v=128,
                ctx=T, max_ctx=T + 256)
    base.update(kw)
    return W.Workload(**base)


@pytest.mark.parametrize("level", [16, 8, 4, 2, 1])
@pytest.mark.parametrize("T", [64, 200, 1000])
def test_single_tier(level, T):
    """Every rung on its own: external plan puts all closed blocks on one level; ragged tail."""
    w = _tiny(T, policy=W.POLICY_EXTERNAL)
    ocache, gcache = _pair(w)
    data = W.make_layer(w, 0, "cpu")
    plan = np.full((w.batch, w.n_kv_heads, T // 64), level, dtype=np.int8)
    U.ingest_both(w, 0, data, ocache, gcache, level_plan=plan)
    U.assert_state_equal(ocache, gcache, 0)
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
    U.assert_outputs_close(out, o_out, f"level {level} T {T}")
    assert np.max(np.abs(lse.cpu().numpy() - o_lse)) < 5e-3
    rep_g, rep_o = gcache.gkv_bits_report(0), ocache.bits_report(0)
    assert rep_g.resident_bits == rep_o["resident_bits"] and rep_g.last_read_bits == rep_o["last_read_bits"]
    gcache.close()


def test_ingest_of_rows_that_are_not_16_byte_aligned():
    """The bulk encoder wants 16-byte aligned rows; other inputs go through the general block encoder.
    Same prompt, key / value tensors placed 4 bytes off a 16-byte boundary: same bits as the oracle."""
    w = _tiny(456)
    ocache, gcache = _pair(w)
    data = W.make_layer(w, 0, "cpu")
    ocache.append_demote(0, U.f32(data["k"]), U.f32(data["v"]))
    dev = gcache.device

    def shifted(t):
        flat = torch.empty(t.numel() + 8, dtype=t.dtype, device=dev)
        view = flat[2:2 + t.numel()].view(t.shape)
        view.copy_(t.to(dev))
        assert view.data_ptr() % 16 == 4
        return view

    k, v = shifted(data["k"]), shifted(data["v"])
    gcache.gkv_append_demote(0, k, v)
    U.assert_state_equal(ocache, gcache, 0)
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
    U.assert_outputs_close(out, o_out, "unaligned ingest")
    gcache.close()


def test_tail_only_and_single_token():
    """Contexts shorter than one block: only the exact tail exists."""
    for T in (1, 17, 63):
        w = _tiny(T)
        ocache, gcache = _pair(w)
        data = W.make_layer(w, 0, "cpu")
        U.ingest_both(w, 0, data, ocache, gcache)
        U.assert_state_equal(ocache, gcache, 0)
        out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
        U.assert_outputs_close(out, o_out, f"tail only T {T}")
        gcache.close()


def test_cfg0_full_parity():
    """Config 0: 8 query / 2 KV heads, context 4096, ladder 512 exact / 1024 int8 / 1536 int4 / 1024 int2,
    outlier key channels, planted heavy tokens.  Everything, all blocks."""
    w = W.config(0)
    ocache, gcache = _pair(w)
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    U.assert_state_equal(ocache, gcache, 0)
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
    err, rel = U.assert_outputs_close(out, o_out, "cfg0")
    rep_g, rep_o = gcache.gkv_bits_report(0), ocache.bits_report(0)
    assert rep_g.bpv_resident == rep_o["bpv_resident"] == 6.875
    assert rep_g.last_read_bits == rep_o["last_read_bits"]
    assert list(rep_g.blocks_by_level) == [16, 32, 48, 32, 0]
    # run to run determinism: bitwise identical outputs
    out2 = torch.empty_like(out)
    gcache.gkv_decode_attn(0, data["q"].to(gcache.device), out2)
    torch.cuda.synchronize()
    assert torch.equal(out, out2)
    gcache.close()


def test_cfg2_small_append_and_demotion():
    """Config 2 structure at small size: bulk ingest, then one token per step with staircase
    demotion (16 -> 8 -> 4 -> 2 -> centroid) at every block fill; state bit-exact at checkpoints."""
    w = W.config(2, "small")
    ocache, gcache = _pair(w)
    dev = gcache.device
    for layer in range(w.n_layers):
        data = W.make_layer(w, layer, "cpu")
        U.ingest_both(w, layer, data, ocache, gcache)
    U.assert_state_equal(ocache, gcache, 0)
    check_out = {0, 1, 63, 64, 65, 127, 128, 129}
    check_state = {64, 128}
    for step in range(w.decode_steps):
        for layer in range(w.n_layers):
            tok = W.make_decode_tokens(w, layer, step, "cpu")
            ocache.append_demote(layer, U.f32(tok["k"]), U.f32(tok["v"]))
            gcache.gkv_append_demote(layer, tok["k"].to(dev), tok["v"].to(dev))
            if step in check_out:
                out, lse, o_out, o_lse = U.decode_both(ocache, gcache, layer, tok["q"])
                U.assert_outputs_close(out, o_out, f"cfg2-small step {step} layer {layer}")
        if step + 1 in check_state:
            for layer in range(w.n_layers):
                U.assert_state_equal(ocache, gcache, layer)
                rep_g, rep_o = gcache.gkv_bits_report(layer), ocache.bits_report(layer)
                assert rep_g.resident_bits == rep_o["resident_bits"]
    # monotonicity: no block ever rose (oracle history) and the GPU agrees with the final levels
    for key, st in ocache.streams.items():
        for blk in st.blocks:
            assert all(a >= b for a, b in zip(blk.history, blk.history[1:]))
    gcache.close()


def test_cfg1_small_rd_allocator_and_residual():
    """Config 1 structure: RD allocator at 4.84 bits/value + 1 % exact residual, drifted K/V."""
    w = W.config(1, "small")
    ocache, gcache = _pair(w)
    for layer in range(w.n_layers):
        data = W.make_layer(w, layer, "cpu")
        U.ingest_both(w, layer, data, ocache, gcache)
        U.assert_state_equal(ocache, gcache, layer)
        lv = ocache.levels(layer, 0, 0)
        assert len(set(lv.tolist())) >= 3, f"allocator produced a flat plan: {lv}"
        out, lse, o_out, o_lse = U.decode_both(ocache, gcache, layer, data["q"])
        U.assert_outputs_close(out, o_out, f"cfg1-small layer {layer}")
        rep_g, rep_o = gcache.gkv_bits_report(layer), ocache.bits_report(layer)
        assert rep_g.resident_bits == rep_o["resident_bits"]
        assert rep_g.last_read_bits == rep_o["last_read_bits"]
        assert rep_g.bpv_paper <= 4.84 + 16 * 0.01 + 1e-9
    gcache.close()


def test_rdv2_operating_point_small():
    """The paper's RD-V2 operating point (Table 2): every closed block outside a short exact window
    is a centroid, 10 % of the tokens stay exact as residual rows; then decode steps with appends."""
    w = W.config(5, "small")
    ocache, gcache = _pair(w)
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    U.assert_state_equal(ocache, gcache, 0)
    lv = ocache.levels(0, 0, 0)
    assert set(lv.tolist()) <= {16, 1} and (lv == 1).sum() >= len(lv) - 3
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
    U.assert_outputs_close(out, o_out, "rdv2-small")
    rep_g, rep_o = gcache.gkv_bits_report(0), ocache.bits_report(0)
    assert rep_g.resident_bits == rep_o["resident_bits"] and rep_g.last_read_bits == rep_o["last_read_bits"]
    assert 1.5 < rep_g.bpv_paper < 3.5
    for step in range(30):
        tok = W.make_decode_tokens(w, 0, step, "cpu")
        ocache.append_demote(0, U.f32(tok["k"]), U.f32(tok["v"]))
        gcache.gkv_append_demote(0, tok["k"].to(dev), tok["v"].to(dev))
        if step in (0, 23, 24, 29):
            out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, tok["q"])
            U.assert_outputs_close(out, o_out, f"rdv2-small step {step}")
    U.assert_state_equal(ocache, gcache, 0)
    gcache.close()


def test_cfg3_small_quest_select_and_sparse_attention():
    """Config 3 structure: exact page boxes, box upper-bound scores, top-k pages, attention over
    the selected graded pages plus the partial tail block."""
    w = W.config(3, "small")
    ocache, gcache = _pair(w)
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    U.assert_state_equal(ocache, gcache, 0)
    U.assert_boxes_and_scores_equal(ocache, gcache, 0, data["q"])
    k = w.quest_budget_tokens // w.page_tokens
    pages = torch.full((w.batch, w.n_kv_heads, k), -1, dtype=torch.int32, device=dev)
    n_sel = gcache.gkv_quest_select(0, data["q"].to(dev), w.quest_budget_tokens, pages)
    torch.cuda.synchronize()
    sel_o = ocache.quest_select(0, U.f32(data["q"]), w.quest_budget_tokens)
    assert n_sel == k
    pg = pages.cpu().numpy()
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            assert np.array_equal(pg[b, h], sel_o[b][h]), f"selected pages differ for stream {(b, h)}"
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"], page_idx_gpu=pages, n_sel=n_sel,
                                           page_idx_oracle=sel_o)
    U.assert_outputs_close(out, o_out, "cfg3-small sparse")
    rep_g, rep_o = gcache.gkv_bits_report(0), ocache.bits_report(0)
    assert rep_g.resident_bits == rep_o["resident_bits"]
    assert rep_g.last_read_bits == rep_o["last_read_bits"]
    # a full read on the same cache still matches
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
    U.assert_outputs_close(out, o_out, "cfg3-small full")
    gcache.close()


@pytest.mark.parametrize("page", [32, 64])
def test_quest_larger_pages(page):
    """Page sizes 32 and 64 (the paper's own Quest setting is page = block = 64 tokens with a
    12.5 % page budget): boxes, scores, selection and the page-sparse read."""
    w = dataclasses.replace(W.config(3, "small"), page_tokens=page, quest_budget_tokens=256)
    ocache, gcache = _pair(w)
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    U.assert_state_equal(ocache, gcache, 0)
    U.assert_boxes_and_scores_equal(ocache, gcache, 0, data["q"])
    k = w.quest_budget_tokens // page
    pages = torch.full((w.batch, w.n_kv_heads, k), -1, dtype=torch.int32, device=dev)
    n_sel = gcache.gkv_quest_select(0, data["q"].to(dev), w.quest_budget_tokens, pages)
    torch.cuda.synchronize()
    sel_o = ocache.quest_select(0, U.f32(data["q"]), w.quest_budget_tokens)
    assert n_sel == k
    pg = pages.cpu().numpy()
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            assert np.array_equal(pg[b, h], sel_o[b][h]), f"selected pages differ for stream {(b, h)}"
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"], page_idx_gpu=pages, n_sel=n_sel,
                                           page_idx_oracle=sel_o)
    U.assert_outputs_close(out, o_out, f"page {page} sparse")
    rep_g, rep_o = gcache.gkv_bits_report(0), ocache.bits_report(0)
    assert rep_g.resident_bits == rep_o["resident_bits"] and rep_g.last_read_bits == rep_o["last_read_bits"]
    gcache.close()


@pytest.mark.parametrize("group", [1, 3, 4, 8])
def test_quest_sum_reduction_and_boxes_after_appends(group):
    """The page score summed (instead of maximised) over the KV head's query heads, for several group
    sizes; boxes and scores bit for bit, also after appends have closed further blocks."""
    w = dataclasses.replace(W.config(3, "small"), n_q_heads=2 * group, quest_reduce=1, ctx=1000, max_ctx=1000 + 256)
    ocache, gcache = _pair(w)
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    U.assert_boxes_and_scores_equal(ocache, gcache, 0, data["q"])
    for step in range(70):
        tok = W.make_decode_tokens(w, 0, step, "cpu")
        ocache.append_demote(0, U.f32(tok["k"]), U.f32(tok["v"]))
        gcache.gkv_append_demote(0, tok["k"].to(dev), tok["v"].to(dev))
    U.assert_boxes_and_scores_equal(ocache, gcache, 0, data["q"])
    k = 8
    pages = torch.full((w.batch, w.n_kv_heads, k), -1, dtype=torch.int32, device=dev)
    n_sel = gcache.gkv_quest_select(0, data["q"].to(dev), k * w.page_tokens, pages)
    torch.cuda.synchronize()
    sel_o = ocache.quest_select(0, U.f32(data["q"]), k * w.page_tokens)
    assert n_sel == k
    pg = pages.cpu().numpy()
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            assert np.array_equal(pg[b, h], sel_o[b][h])
    gcache.close()


def test_quest_selecting_every_page_equals_full_read():
    w = dataclasses.replace(W.config(3, "small"), quest_budget_tokens=1 << 20)
    ocache, gcache = _pair(w)
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    n_pages = (w.ctx // 64) * 4
    pages = torch.zeros((w.batch, w.n_kv_heads, n_pages), dtype=torch.int32, device=dev)
    n_sel = gcache.gkv_quest_select(0, data["q"].to(dev), w.quest_budget_tokens, pages)
    assert n_sel == n_pages
    out_s = torch.empty((w.batch, w.n_q_heads, w.d_v), dtype=torch.float32, device=dev)
    out_f = torch.empty_like(out_s)
    gcache.gkv_decode_attn(0, data["q"].to(dev), out_s, page_idx=pages, n_sel=n_sel)
    gcache.gkv_decode_attn(0, data["q"].to(dev), out_f)
    torch.cuda.synchronize()
    assert torch.allclose(out_s, out_f, atol=2e-4, rtol=0)
    assert torch.equal(pages.cpu(), torch.arange(n_pages, dtype=torch.int32).expand(w.batch, w.n_kv_heads, n_pages))
    gcache.close()


def test_host_side_errors():
    B = _binding()
    w = _tiny(200)
    gcache = B.Cache(B.config_from_workload(w))
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    out = torch.empty((1, 8, 128), dtype=torch.float32, device=dev)
    with pytest.raises(B.GkvError) as e:
        gcache.gkv_decode_attn(0, data["q"].to(dev), out)            # empty layer
    assert e.value.status == -4
    gcache.gkv_append_demote(0, data["k"].to(dev), data["v"].to(dev))
    with pytest.raises(B.GkvError) as e:
        gcache.gkv_append_demote(0, data["k"].to(dev), data["v"].to(dev))   # bulk ingest on a non-empty layer
    assert e.value.status == -4
    with pytest.raises(B.GkvError) as e:
        gcache.gkv_append_demote(3, data["k"].to(dev), data["v"].to(dev))   # bad layer
    assert e.value.status == -1
    pages = torch.zeros((1, 2, 4), dtype=torch.int32, device=dev)
    with pytest.raises(B.GkvError) as e:
        gcache.gkv_quest_select(0, data["q"].to(dev), 64, pages)            # no page scorer configured
    assert e.value.status == -4
    gcache.close()
    # an arena that holds the metadata but not the blocks reports ARENA_TOO_SMALL at append time
    cfg = B.config_from_workload(_tiny(4096))
    small = B.Cache(cfg, arena_bytes=B.gkv_query_arena_bytes(cfg) - 3 * 1024 * 1024)
    big = W.make_layer(_tiny(4096), 0, "cpu")
    with pytest.raises(B.GkvError) as e:
        small.gkv_append_demote(0, big["k"].to(dev), big["v"].to(dev))
    assert e.value.status == -2
    small.close()
    # context capacity
    w2 = _tiny(200)
    w2 = dataclasses.replace(w2, max_ctx=200)
    full = B.Cache(B.config_from_workload(w2))
    d2 = W.make_layer(w2, 0, "cpu")
    full.gkv_append_demote(0, d2["k"].to(dev), d2["v"].to(dev))
    tok = W.make_decode_tokens(w2, 0, 0, "cpu")
    with pytest.raises(B.GkvError) as e:
        full.gkv_append_demote(0, tok["k"].to(dev), tok["v"].to(dev))
    assert e.value.status == -3
    # pointers off their natural boundary are refused before anything is launched
    def off_by(t, n_elem):
        flat = torch.empty(t.numel() + 16, dtype=t.dtype, device=dev)
        view = flat[n_elem:n_elem + t.numel()].view(t.shape)
        view.copy_(t.to(dev))
        return view
    qd = d2["q"].to(dev).to(torch.bfloat16)
    out = torch.empty((w2.batch, w2.n_q_heads, w2.d_v), dtype=torch.float32, device=dev)
    with pytest.raises(B.GkvError) as e:
        full.gkv_decode_attn(0, off_by(qd, 1), out)            # query 2 bytes off
    assert e.value.status == -1
    with pytest.raises(B.GkvError) as e:
        full.gkv_decode_attn(0, qd, off_by(out, 1))            # output 4 bytes off a 16-byte boundary
    assert e.value.status == -1
    fresh = B.Cache(B.config_from_workload(w2))
    with pytest.raises(B.GkvError) as e:
        fresh.gkv_append_demote(0, off_by(d2["k"], 1), d2["v"].to(dev))   # rows 2 bytes off
    assert e.value.status == -1
    fresh.close()
    full.close()


# ---- latent attention (MLA): 576-wide stream, 16 heads, values = key channels [0, 512) --------------
def _mla(T, **kw):
    base = dict(name="mla_tiny", config_id=14, n_layers=1, batch=2, n_q_heads=16, n_kv_heads=1, d_k=576, d_v=512,
                ctx=T, max_ctx=T + 256, v_aliases_k=1, softmax_scale=1.0 / 192 ** 0.5, n_outlier=8, outlier_gain=6.0,
                n_heavy=0)
    base.update(kw)
    return W.Workload(**base)


@pytest.mark.parametrize("level", [16, 8, 4, 1])
@pytest.mark.parametrize("T", [64, 200, 1100])
def test_mla_single_tier(level, T):
    w = _mla(T, policy=W.POLICY_EXTERNAL)
    ocache, gcache = _pair(w)
    data = W.make_layer(w, 0, "cpu")
    plan = np.full((w.batch, 1, T // 64), level, dtype=np.int8)
    U.ingest_both(w, 0, data, ocache, gcache, level_plan=plan)
    U.assert_state_equal(ocache, gcache, 0)
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
    U.assert_outputs_close(out, o_out, f"mla level {level} T {T}")
    assert np.max(np.abs(lse.cpu().numpy() - o_lse)) < 5e-3
    rep_g, rep_o = gcache.gkv_bits_report(0), ocache.bits_report(0)
    assert rep_g.resident_bits == rep_o["resident_bits"] and rep_g.last_read_bits == rep_o["last_read_bits"]
    gcache.close()


def test_mla_ingest_of_rows_that_are_not_16_byte_aligned():
    """Latent rows 4 bytes off a 16-byte boundary go through the general block encoder: same bits."""
    T = 328
    w = _mla(T, policy=W.POLICY_EXTERNAL)
    ocache, gcache = _pair(w)
    data = W.make_layer(w, 0, "cpu")
    plan = np.tile(np.array([1, 4, 8, 4, 16], dtype=np.int8), (w.batch, 1, 1))
    ocache.append_demote(0, U.f32(data["k"]), None, level_plan=plan)
    dev = gcache.device
    flat = torch.empty(data["k"].numel() + 8, dtype=data["k"].dtype, device=dev)
    k = flat[2:2 + data["k"].numel()].view(data["k"].shape)
    k.copy_(data["k"].to(dev))
    assert k.data_ptr() % 16 == 4
    gcache.gkv_append_demote(0, k, None, level_plan=plan)
    U.assert_state_equal(ocache, gcache, 0)
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
    U.assert_outputs_close(out, o_out, "mla unaligned ingest")
    gcache.close()


def test_mla_runs_of_mixed_levels_inside_one_warp_group_range():
    """65,541 tokens per sequence under an external plan of short runs (1-8 blocks) of random levels: every
    CTA of the read kernel gets several blocks, so the block ranges of its warp groups mix exact, 8-bit, 4-bit
    and centroid units, cut centroid runs at range ends and switch between the unit kinds while the running
    output stays in place."""
    T = 65536 + 5
    w = _mla(T, policy=W.POLICY_EXTERNAL)
    ocache, gcache = _pair(w)
    data = W.make_layer(w, 0, "cpu")
    rs = np.random.RandomState(4242)
    plan = np.empty((w.batch, 1, T // 64), dtype=np.int8)
    for b in range(w.batch):
        i = 0
        while i < T // 64:
            n = int(rs.randint(1, 9))
            plan[b, 0, i:i + n] = rs.choice(np.array([16, 8, 4, 1], dtype=np.int8))
            i += n
    U.ingest_both(w, 0, data, ocache, gcache, level_plan=plan)
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
    U.assert_outputs_close(out, o_out, "mla mixed runs")
    assert np.max(np.abs(lse.cpu().numpy() - o_lse)) < 5e-3
    rep_g, rep_o = gcache.gkv_bits_report(0), ocache.bits_report(0)
    assert rep_g.resident_bits == rep_o["resident_bits"] and rep_g.last_read_bits == rep_o["last_read_bits"]
    gcache.close()


def test_cfg4_small_mla_ladder_with_appends():
    """Config 4 structure at small size: exact newest rung, int8, int4, centroid for the oldest
    quarter (5.0 bits/value), then appends with staircase demotion."""
    w = W.config(4, "small")
    ocache, gcache = _pair(w)
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    U.assert_state_equal(ocache, gcache, 0)
    rep = gcache.gkv_bits_report(0)
    assert abs(rep.bpv_resident - 5.0) < 0.01 and rep.blocks_by_level[3] == 0 and rep.blocks_by_level[4] == 32
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
    err, rel = U.assert_outputs_close(out, o_out, "cfg4-small")
    for step in range(66):
        tok = W.make_decode_tokens(w, 0, step, "cpu")
        ocache.append_demote(0, U.f32(tok["k"]), None)
        gcache.gkv_append_demote(0, tok["k"].to(dev), None)
        if step in (0, 31, 62, 63, 64, 65):
            out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, tok["q"])
            U.assert_outputs_close(out, o_out, f"cfg4-small step {step}")
    U.assert_state_equal(ocache, gcache, 0)
    assert gcache.gkv_bits_report(0).resident_bits == ocache.bits_report(0)["resident_bits"]
    gcache.close()


@pytest.mark.gpu
@pytest.mark.parametrize("hq,hkv", [(2, 2), (4, 2), (16, 2), (8, 1)])
def test_query_group_sizes(hq, hkv):
    """1, 2, 8 query heads per KV head (the tensor-core tile holds up to 8) on a full ladder."""
    w = _tiny(1000, n_q_heads=hq, n_kv_heads=hkv, stair_tokens=(192, 192, 256, 192))
    ocache, gcache = _pair(w)
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    U.assert_state_equal(ocache, gcache, 0)
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"])
    U.assert_outputs_close(out, o_out, f"group {hq // hkv}")
    assert np.max(np.abs(lse.cpu().numpy() - o_lse)) < 5e-3
    gcache.close()


@pytest.mark.gpu
def test_decode_is_bitwise_reproducible():
    """The split-K merge runs in a fixed order whichever CTA finishes last: the same call twice,
    and the same cache read through a second handle, give identical bits."""
    w = W.config(2, "small")
    outs = []
    for _ in range(2):
        _, gcache = _pair(w)
        dev = gcache.device
        data = W.make_layer(w, 0, "cpu")
        gcache.gkv_append_demote(0, data["k"].to(dev), data["v"].to(dev))
        q = data["q"].to(dev)
        for _rep in range(3):
            out = torch.empty((w.batch, w.n_q_heads, w.d_v), dtype=torch.float32, device=dev)
            lse = torch.empty((w.batch, w.n_q_heads), dtype=torch.float32, device=dev)
            gcache.gkv_decode_attn(0, q, out, lse=lse)
            torch.cuda.synchronize()
            outs.append((out.cpu().numpy().copy(), lse.cpu().numpy().copy()))
        gcache.close()
    for o, l in outs[1:]:
        assert np.array_equal(o, outs[0][0]) and np.array_equal(l, outs[0][1])


@pytest.mark.gpu
def test_mla_decode_is_bitwise_reproducible():
    """Latent streams: the partial logits of a warp group are added in warp order, its warps' results and
    the CTAs' rows are merged in a fixed order, so the same call twice and a second handle on the same rows
    give identical bits.  The context is long enough for every warp group of every CTA to have blocks."""
    w = _mla(148 * 4 * 3 * 64 + 17, batch=1, policy=W.POLICY_STAIRCASE, stair_tokens=(4096, 32768, 49152, 0))
    outs = []
    for _ in range(2):
        _, gcache = _pair(w)
        dev = gcache.device
        data = W.make_layer(w, 0, "cpu")
        gcache.gkv_append_demote(0, data["k"].to(dev), None)
        q = data["q"].to(dev)
        for _rep in range(3):
            out = torch.empty((w.batch, w.n_q_heads, w.d_v), dtype=torch.float32, device=dev)
            lse = torch.empty((w.batch, w.n_q_heads), dtype=torch.float32, device=dev)
            gcache.gkv_decode_attn(0, q, out, lse=lse)
            torch.cuda.synchronize()
            outs.append((out.cpu().numpy().copy(), lse.cpu().numpy().copy()))
        gcache.close()
    for o, l in outs[1:]:
        assert np.array_equal(o, outs[0][0]) and np.array_equal(l, outs[0][1])


# ---- block attention mass observed by the decode pass (Sec. 3.1) -------------------------------
MASS_RTOL, MASS_ATOL = 1e-2, 2e-6     # weights carry the logit error of fp16 operands (about 1e-3 relative)


def _observe_both(ocache, gcache, layer, q_bf16):
    cfg = ocache.cfg
    dev = gcache.device
    n_items = (gcache.gkv_ctx_len(layer) + 63) // 64
    out = torch.empty((cfg.batch, cfg.n_q_heads, cfg.d_v), dtype=torch.float32, device=dev)
    lse = torch.empty((cfg.batch, cfg.n_q_heads), dtype=torch.float32, device=dev)
    mass = torch.full((cfg.batch, cfg.n_kv_heads, n_items), -1.0, dtype=torch.float32, device=dev)
    gcache.gkv_decode_attn_observe(layer, q_bf16.to(dev), out, lse, mass)
    torch.cuda.synchronize()
    o_out, o_lse, o_obs = ocache.decode_attn_observe(layer, U.f32(q_bf16))
    return out, o_out, mass.cpu().numpy().astype(np.float64), o_obs


def _assert_mass_close(got, want_by_stream, tag, unit_sum=True):
    for (b, h), want in want_by_stream.items():
        g = got[b, h]
        assert g.shape == want.shape, (tag, g.shape, want.shape)
        err = np.abs(g - want)
        bad = err > MASS_RTOL * np.abs(want) + MASS_ATOL
        assert not bad.any(), (tag, b, h, int(np.argmax(err)), float(err.max()), float(want[np.argmax(err)]))
        if unit_sum:
            assert abs(g.sum() - 1.0) < 2e-3, (tag, b, h, float(g.sum()))


def _ema_of(ocache, layer):
    cfg = ocache.cfg
    return {(b, h): ocache.streams[(layer, b, h)].ema_mass for b in range(cfg.batch) for h in range(cfg.n_kv_heads)}


def test_block_mass_all_levels_with_appends():
    """Config 0 (every rung of the ladder, query groups of 4): the observed block masses and the
    running masses against the oracle, across appends that grow the partial block, close it and
    demote blocks; the attention output of the observing call equals the plain call's."""
    w = W.config(0)
    ocache, gcache = _pair(w)
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    out, o_out, mass, o_obs = _observe_both(ocache, gcache, 0, data["q"])
    U.assert_outputs_close(out, o_out, "observe cfg0")
    _assert_mass_close(mass, o_obs, "cfg0 step -1")
    plain = torch.empty_like(out)
    gcache.gkv_decode_attn(0, data["q"].to(dev), plain)
    torch.cuda.synchronize()
    assert torch.equal(plain, out)                 # observing does not change the arithmetic of the output
    for step in range(70):
        tok = W.make_decode_tokens(w, 0, step, "cpu")
        ocache.append_demote(0, U.f32(tok["k"]), U.f32(tok["v"]))
        gcache.gkv_append_demote(0, tok["k"].to(dev), tok["v"].to(dev))
        if step in (0, 1, 62, 63, 64, 69):
            out, o_out, mass, o_obs = _observe_both(ocache, gcache, 0, tok["q"])
            U.assert_outputs_close(out, o_out, f"observe cfg0 step {step}")
            _assert_mass_close(mass, o_obs, f"cfg0 step {step}")
    _assert_mass_close(gcache.gkv_debug_export_mass(0).astype(np.float64), _ema_of(ocache, 0), "cfg0 running mass", unit_sum=False)
    gcache.close()


def test_block_mass_centroid_runs_and_residual_rows():
    """RD-V2 shape: almost every block a centroid (read as runs of 16 blocks), 10 % of the tokens in
    the exact residual whose weight counts for their block."""
    w = W.config(5, "small")
    ocache, gcache = _pair(w)
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    for step in range(3):
        q = data["q"] if step == 0 else W.make_decode_tokens(w, 0, step, "cpu")["q"]
        out, o_out, mass, o_obs = _observe_both(ocache, gcache, 0, q)
        U.assert_outputs_close(out, o_out, f"observe rdv2 {step}")
        _assert_mass_close(mass, o_obs, f"rdv2 {step}")
        tok = W.make_decode_tokens(w, 0, step, "cpu")
        ocache.append_demote(0, U.f32(tok["k"]), U.f32(tok["v"]))
        gcache.gkv_append_demote(0, tok["k"].to(dev), tok["v"].to(dev))
    _assert_mass_close(gcache.gkv_debug_export_mass(0).astype(np.float64), _ema_of(ocache, 0), "rdv2 running mass", unit_sum=False)
    gcache.close()


def test_block_mass_query_group_of_8_and_single_block():
    w = _tiny(40, n_q_heads=16, n_kv_heads=2)
    ocache, gcache = _pair(w)
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    out, o_out, mass, o_obs = _observe_both(ocache, gcache, 0, data["q"])
    assert mass.shape[-1] == 1 and np.allclose(mass, 1.0, atol=1e-5)
    _assert_mass_close(mass, o_obs, "tiny")
    gcache.close()


def test_block_mass_running_average_starts_from_prompt_masses():
    """RD policy (config 1 structure): the running mass is seeded with the block sums of the prompt
    masses given at ingest, then follows m <- 0.9 m + 0.1 a."""
    w = W.config(1, "small")
    ocache, gcache = _pair(w, n_layers=1)
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    seed = _ema_of(ocache, 0)
    got0 = gcache.gkv_debug_export_mass(0).astype(np.float64)
    for (b, h), want in seed.items():
        assert len(want) == w.ctx // 64 and want.sum() > 0.5
        assert np.allclose(got0[b, h, :len(want)], want, rtol=1e-6, atol=1e-9)     # the same fp32 block sums
    for step in range(2):
        out, o_out, mass, o_obs = _observe_both(ocache, gcache, 0, data["q"])
        U.assert_outputs_close(out, o_out, f"observe cfg1 {step}")
        _assert_mass_close(mass, o_obs, f"cfg1 {step}")
    _assert_mass_close(gcache.gkv_debug_export_mass(0).astype(np.float64), _ema_of(ocache, 0), "cfg1 running mass",
                       unit_sum=False)
    gcache.close()


def test_decode_time_reallocation_from_running_masses():
    """RD policy, config 1 structure: observe every decode query, append, and after each block close
    re-run the allocator on the running masses (gkv_rd_reallocate).

    The level decisions compare masses with thresholds, and the library's masses (fp32, weights at
    fp16 operand precision) differ from the oracle's (fp64) in the third digit, so a block that sits
    on a threshold may legitimately land on either side.  What is unique is checked exactly: the
    decision rule on identical inputs (CPU test of gkv_debug_replan_levels against the oracle), the
    temporal constraint, the budget, and - with the library's plan replayed as the oracle's demotion
    plan - every code, scale, zero and centroid plus the attention outputs.  The two plans are also
    compared directly and may differ in a few blocks only."""
    import dataclasses
    w = W.config(1, "small")
    w = dataclasses.replace(w, max_ctx=w.ctx + 256)
    ocache, gcache = _pair(w, n_layers=1)
    ofree = O.GradedCache(U.oracle_config(w, 1))          # the oracle left to its own decisions
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    ofree.append_demote(0, U.f32(data["k"]), U.f32(data["v"]), token_mass=data["mass"].numpy())
    cfg = ocache.cfg
    n_changed = 0
    differ = total = 0
    for step in range(130):
        tok = W.make_decode_tokens(w, 0, step, "cpu")
        out, o_out, mass, o_obs = _observe_both(ocache, gcache, 0, tok["q"])
        ofree.decode_attn_observe(0, U.f32(tok["q"]))
        if step % 40 == 0:
            _assert_mass_close(mass, o_obs, f"realloc step {step}")
        ocache.append_demote(0, U.f32(tok["k"]), U.f32(tok["v"]))
        ofree.append_demote(0, U.f32(tok["k"]), U.f32(tok["v"]))
        gcache.gkv_append_demote(0, tok["k"].to(dev), tok["v"].to(dev))
        if gcache.gkv_ctx_len(0) % 64 != 0:
            continue
        before = {(b, h): gcache.gkv_debug_export_levels(0, b, h).copy() for b in range(cfg.batch) for h in range(cfg.n_kv_heads)}
        # the plan is made on the device: bit for bit the host allocator's plan on the same masses and ranges
        B = _binding()
        lv_dev, ms, rg, _ = gcache.gkv_debug_device_plan(0)
        for (b, h), old in before.items():
            lv_host, _ = B.gkv_debug_replan_levels(gcache.cfg, gcache.gkv_ctx_len(0) % 64, ms[b, h], rg[b, h], old)
            assert np.array_equal(lv_dev[b, h], lv_host), f"device and host plans differ for stream {(b, h)} at step {step}"
        gcache.gkv_rd_reallocate(0)
        for (b, h) in before:
            assert np.array_equal(gcache.gkv_debug_export_levels(0, b, h), lv_dev[b, h])
        free_plan = ofree.rd_reallocate(0)
        recent = w.retire_after // 64
        for (b, h), old in before.items():
            new = gcache.gkv_debug_export_levels(0, b, h)
            n = len(new)
            assert np.all(new <= old)                                          # no promotion
            assert all(new[i] == 16 for i in range(n) if n - 1 - i < recent)   # the recent window stays exact
            differ += int(np.sum(new != free_plan[(b, h)]))
            total += n
            for i in np.nonzero(new < old)[0]:
                ocache.demote_to(0, b, h, int(i), int(new[i]))
                n_changed += 1
        U.assert_state_equal(ocache, gcache, 0)
        rep = gcache.gkv_bits_report(0)
        assert rep.bpv_paper <= w.rd_budget_bpv + 16 * w.residual_fraction + 1e-6
        out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, tok["q"])
        U.assert_outputs_close(out, o_out, f"after reallocation at step {step}")
    assert n_changed > 0                       # blocks that left the recent window were given a level
    assert differ <= max(2, total // 50), (differ, total)
    gcache.close()


# ---- attention error certificate as a runtime output (Sec. 3.6, Eq. 9) ---------------------------
def _bounds_of(ocache, layer):
    cfg = ocache.cfg
    out = {}
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            blocks = ocache.streams[(layer, b, h)].blocks
            out[(b, h)] = np.array([[blk.kappa, blk.delta, blk.vnorm] for blk in blocks], dtype=np.float64).reshape(-1, 3)
    return out


def _check_bounds_and_certificate(w, ocache, gcache, dense, q_bf16, tag, scale=None):
    cfg = ocache.cfg
    dev = gcache.device
    got = gcache.gkv_debug_export_bounds(0).astype(np.float64)
    for (b, h), want in _bounds_of(ocache, 0).items():
        g = got[b, h, :, :3]
        assert g.shape == want.shape, (tag, g.shape, want.shape)
        assert np.allclose(g, want, rtol=3e-5, atol=1e-6), (tag, b, h, float(np.abs(g - want).max()))
        assert np.all(got[b, h, :, 3] == 0)
    out = torch.empty((cfg.batch, cfg.n_q_heads, cfg.d_v), dtype=torch.float32, device=dev)
    cert = torch.full((cfg.batch, cfg.n_q_heads), -1.0, dtype=torch.float32, device=dev)
    gcache.gkv_decode_attn_observe(0, q_bf16.to(dev), out, None, None, cert)
    torch.cuda.synchronize()
    cert = cert.cpu().numpy().astype(np.float64)
    want = ocache.certificate(0, U.f32(q_bf16))
    # the weights behind the certificate carry the kernel's logit error (about 1e-3 relative)
    assert np.allclose(cert, want, rtol=1e-2, atol=1e-5), (tag, float(np.abs(cert - want).max()), float(want.max()))
    o_true, _ = dense.decode_attn(0, U.f32(q_bf16))
    err = np.linalg.norm(o_true - out.cpu().numpy().astype(np.float64), axis=-1)
    assert np.all(err <= cert * (1 + 1e-3) + 1e-4), (tag, float((err - cert).max()))
    return cert, err


def test_certificate_all_levels_with_demotions():
    """Config 0: bounds of blocks encoded at ingest, then carried through a chain of demotions at
    decode time; the certificate against the oracle's and against the true error of the library's
    output with respect to attention over the original rows."""
    import dataclasses
    w = W.config(0)
    ocache, gcache = _pair(w)
    dense = O.GradedCache(U.oracle_config(dataclasses.replace(w, stair_tokens=(-1, 0, 0, 0))))
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    dense.append_demote(0, U.f32(data["k"]), U.f32(data["v"]))
    cert, err = _check_bounds_and_certificate(w, ocache, gcache, dense, data["q"], "cfg0 ingest")
    assert np.all(cert > 0) and np.all(err > 0)
    for step in range(66):
        tok = W.make_decode_tokens(w, 0, step, "cpu")
        ocache.append_demote(0, U.f32(tok["k"]), U.f32(tok["v"]))
        dense.append_demote(0, U.f32(tok["k"]), U.f32(tok["v"]))
        gcache.gkv_append_demote(0, tok["k"].to(dev), tok["v"].to(dev))
        if step in (5, 63, 65):
            _check_bounds_and_certificate(w, ocache, gcache, dense, tok["q"], f"cfg0 step {step}")
    hist = [len(b.history) for b in ocache.streams[(0, 0, 0)].blocks]
    assert max(hist) >= 2                                   # some bounds were carried through a requantisation
    gcache.close()


def test_certificate_with_centroids_and_residual_rows():
    import dataclasses
    w = W.config(5, "small")
    ocache, gcache = _pair(w)
    dense = O.GradedCache(U.oracle_config(dataclasses.replace(w, stair_tokens=(-1, 0, 0, 0), residual_fraction=0.0)))
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    dense.append_demote(0, U.f32(data["k"]), U.f32(data["v"]))
    _check_bounds_and_certificate(w, ocache, gcache, dense, data["q"], "rdv2")
    gcache.close()


def test_certificate_of_an_exact_cache_is_zero():
    w = _tiny(300)
    ocache, gcache = _pair(w)
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    dev = gcache.device
    out = torch.empty((1, 8, 128), dtype=torch.float32, device=dev)
    cert = torch.full((1, 8), -1.0, dtype=torch.float32, device=dev)
    gcache.gkv_decode_attn_observe(0, data["q"].to(dev), out, None, None, cert)
    torch.cuda.synchronize()
    assert torch.all(cert == 0)
    gcache.close()


@pytest.mark.parametrize("hq,hkv", [(2, 2), (4, 2), (16, 2)])
def test_observe_query_group_sizes(hq, hkv):
    """Block masses, running masses and the certificate with 1, 2 and 8 query heads per KV head."""
    import dataclasses
    w = _tiny(1000, n_q_heads=hq, n_kv_heads=hkv, stair_tokens=(192, 192, 256, 192))
    ocache, gcache = _pair(w)
    dense = O.GradedCache(U.oracle_config(dataclasses.replace(w, stair_tokens=(-1, 0, 0, 0))))
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    dense.append_demote(0, U.f32(data["k"]), U.f32(data["v"]))
    out, o_out, mass, o_obs = _observe_both(ocache, gcache, 0, data["q"])
    U.assert_outputs_close(out, o_out, f"observe group {hq // hkv}")
    _assert_mass_close(mass, o_obs, f"group {hq // hkv}")
    _check_bounds_and_certificate(w, ocache, gcache, dense, data["q"], f"group {hq // hkv}")
    gcache.close()


def test_observe_and_reallocate_reject_what_they_do_not_cover():
    B = _binding()
    # latent-attention streams: no block-mass observation
    wm = W.config(4, "small")
    _, gm = _pair(wm)
    dev = gm.device
    dm = W.make_layer(wm, 0, "cpu")
    gm.gkv_append_demote(0, dm["k"].to(dev), None)
    out = torch.empty((wm.batch, wm.n_q_heads, wm.d_v), dtype=torch.float32, device=dev)
    with pytest.raises(B.GkvError) as e:
        gm.gkv_decode_attn_observe(0, dm["q"].to(dev), out)
    assert e.value.status == B.ERR_UNSUPPORTED
    gm.close()
    # re-allocation is the RD policy's
    w = W.config(0)
    _, g = _pair(w)
    with pytest.raises(B.GkvError) as e:
        g.gkv_rd_reallocate(0)
    assert e.value.status == B.ERR_BAD_STATE
    g.close()


# ---- page lists on layers that hold exact residual tokens (Sec. 3.4 + 3.5) ----------------------
@pytest.mark.parametrize("group", [4, 8])
def test_page_list_read_with_residual_tokens(group):
    """RD-graded store with exact residual rows, read through a page list: residual tokens of pages
    that are not listed are masked with their page, those of listed pages are served exact, centroid
    pages count only their readable tokens.  Selected pages, outputs and read bits against the oracle."""
    w = dataclasses.replace(W.config(1, "small"), n_q_heads=2 * group, page_tokens=16, residual_fraction=0.05, ctx=2048 + 40,
                            max_ctx=2048 + 256, quest_budget_tokens=384)
    ocache, gcache = _pair(w, 1)
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu", with_mass=True)
    U.ingest_both(w, 0, data, ocache, gcache)
    U.assert_state_equal(ocache, gcache, 0)
    assert all(len(ocache.streams[(0, b, h)].res_idx) > 50 for b in range(w.batch) for h in range(w.n_kv_heads))
    k = w.quest_budget_tokens // w.page_tokens
    pages = torch.full((w.batch, w.n_kv_heads, k), -1, dtype=torch.int32, device=dev)
    n_sel = gcache.gkv_quest_select(0, data["q"].to(dev), w.quest_budget_tokens, pages)
    torch.cuda.synchronize()
    sel_o = ocache.quest_select(0, U.f32(data["q"]), w.quest_budget_tokens)
    pg = pages.cpu().numpy()
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            assert np.array_equal(pg[b, h, :n_sel], sel_o[b][h])
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"], page_idx_gpu=pages, n_sel=n_sel, page_idx_oracle=sel_o)
    U.assert_outputs_close(out, o_out, "page list + residual rows")
    assert np.max(np.abs(lse.cpu().numpy() - o_lse)) < 5e-3
    rep_g, rep_o = gcache.gkv_bits_report(0), ocache.bits_report(0)
    assert rep_g.resident_bits == rep_o["resident_bits"] and rep_g.last_read_bits == rep_o["last_read_bits"]
    # a list of the caller's own choosing that covers pages with and without residual tokens, centroid blocks included
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            st = ocache.streams[(0, b, h)]
            with_res = sorted(set(int(t) // 16 for t in st.res_idx))[:5]
            own = sorted(set(with_res + [0, 1, 2, 3, 17, 40, 77, 101]))[:12]
            own += [p for p in range(120, 128) if p not in own][: 12 - len(own)]
            pg[b, h, :12] = sorted(own)
    pages2 = torch.from_numpy(np.ascontiguousarray(pg[:, :, :12])).to(dev)
    sel2 = [[pg[b, h, :12] for h in range(w.n_kv_heads)] for b in range(w.batch)]
    out, lse, o_out, o_lse = U.decode_both(ocache, gcache, 0, data["q"], page_idx_gpu=pages2, n_sel=12, page_idx_oracle=sel2)
    U.assert_outputs_close(out, o_out, "own page list + residual rows")
    rep_g, rep_o = gcache.gkv_bits_report(0), ocache.bits_report(0)
    assert rep_g.last_read_bits == rep_o["last_read_bits"]
    # listing every page equals the full read
    n_pages = (w.ctx // 64) * 4
    all_pages = torch.arange(n_pages, dtype=torch.int32, device=dev).repeat(w.batch, w.n_kv_heads, 1).contiguous()
    full = torch.empty((w.batch, w.n_q_heads, 128), dtype=torch.float32, device=dev)
    gcache.gkv_decode_attn(0, data["q"].to(dev), full)
    sparse = torch.empty_like(full)
    gcache.gkv_decode_attn(0, data["q"].to(dev), sparse, page_idx=all_pages, n_sel=n_pages)
    torch.cuda.synchronize()
    assert float((full - sparse).abs().max()) < 1e-5
    gcache.close()


def test_page_list_entries_out_of_range_are_skipped_and_reported():
    """A page list is the caller's memory: entries outside [0, closed pages) are skipped by the kernel
    (no table entry and no byte is read through them), the output stays finite and equals the read of the
    valid entries, and the next bits report returns GKV_ERR_BAD_STATE."""
    B = _binding()
    w = W.config(3, "small")
    ocache, gcache = _pair(w)
    dev = gcache.device
    data = W.make_layer(w, 0, "cpu")
    U.ingest_both(w, 0, data, ocache, gcache)
    n_pages = (w.ctx // 64) * 4
    good = np.array([3, 9, 10, 57, 100], dtype=np.int32)
    bad = np.array([-5, 3, 9, 10, 57, 100, n_pages, 1 << 30], dtype=np.int32)      # ascending, three entries invalid
    lists = torch.from_numpy(np.tile(bad, (w.batch, w.n_kv_heads, 1))).to(dev)
    out = torch.empty((w.batch, w.n_q_heads, 128), dtype=torch.float32, device=dev)
    gcache.gkv_decode_attn(0, data["q"].to(dev), out, page_idx=lists, n_sel=len(bad))
    torch.cuda.synchronize()
    assert torch.isfinite(out).all()
    sel = [[good for _ in range(w.n_kv_heads)] for _ in range(w.batch)]
    o_out, _ = ocache.decode_attn(0, U.f32(data["q"]), sel)
    U.assert_outputs_close(out, o_out, "list with invalid entries")
    with pytest.raises(B.GkvError) as e:
        gcache.gkv_bits_report(0)
    assert e.value.status == B.ERR_BAD_STATE
    gcache.close()


def test_arena_exhausted_by_a_demotion_step_leaves_the_cache_consistent():
    """An arena that holds the ingested cache but not the slots of the next block-close demotions: the
    append that closes the block reports GKV_ERR_ARENA_TOO_SMALL, and the cache stays what the host
    mirror says it is (levels unchanged, attention still equal to the oracle with the same levels)."""
    B = _binding()
    w = dataclasses.replace(_tiny(1024 + 63, stair_tokens=(128, 256, 256, 256)), max_ctx=2048)
    cfg = B.config_from_workload(w)
    data = W.make_layer(w, 0, "cpu")
    full_bytes = B.gkv_query_arena_bytes(cfg)

    def try_ingest(nbytes):
        try:
            g = B.Cache(cfg, arena_bytes=nbytes)
        except B.GkvError:
            return None
        try:
            g.gkv_append_demote(0, data["k"].to(g.device), data["v"].to(g.device))
        except B.GkvError:
            g.close()
            return None
        return g

    # the smallest arena (in steps of 4 KiB) that still holds the ingested cache
    lo, hi = 0, full_bytes                                   # lo fails, hi succeeds
    g = try_ingest(hi)
    assert g is not None
    g.close()
    while hi - lo > 4096:
        mid = (lo + hi) // 2 // 256 * 256
        g = try_ingest(mid)
        if g is None:
            lo = mid
        else:
            g.close()
            hi = mid
    tok = W.make_decode_tokens(w, 0, 0, "cpu")
    failed = None
    for extra in range(0, 16):                               # the close needs ~35 KB of new slots before it frees the old ones
        gcache = try_ingest(hi + extra * 2048)
        assert gcache is not None
        try:
            gcache.gkv_append_demote(0, tok["k"].to(gcache.device), tok["v"].to(gcache.device))
        except B.GkvError as e:
            assert e.status == B.ERR_ARENA_TOO_SMALL
            failed = gcache
            break
        gcache.close()
    assert failed is not None, "no arena size found where only the demotion step runs out of slots"
    gcache = failed
    # the block closed (17 closed blocks, all levels as before the failed demotions, the new one exact)
    lv = gcache.gkv_debug_export_levels(0, 0, 0)
    assert len(lv) == 17 and lv[-1] == 16
    ocfg = U.oracle_config(dataclasses.replace(w, policy=W.POLICY_EXTERNAL))
    oc = O.GradedCache(ocfg)
    kk = torch.cat([data["k"], tok["k"]], dim=1)
    vv = torch.cat([data["v"], tok["v"]], dim=1)
    plan = np.tile(lv.astype(np.int8), (w.batch, w.n_kv_heads, 1))
    oc.append_demote(0, U.f32(kk), U.f32(vv), level_plan=plan)
    out = torch.empty((w.batch, w.n_q_heads, 128), dtype=torch.float32, device=gcache.device)
    gcache.gkv_decode_attn(0, tok["q"].to(gcache.device), out)
    torch.cuda.synchronize()
    o_out, _ = oc.decode_attn(0, U.f32(tok["q"]))
    U.assert_outputs_close(out, o_out, "after a failed demotion step")
    assert gcache.gkv_bits_report(0).resident_bits == oc.bits_report(0)["resident_bits"]
    gcache.close()


@pytest.mark.parametrize("budget", [2.5, 4.84, 9.0, 0.05])
def test_device_allocator_equals_host_allocator(budget):
    """The threshold search on the device (gkv_rd_reallocate's planner) against the host allocator on
    the same masses, ranges and present levels: 127 closed blocks per stream, several budgets (the last one
    cannot be met: both report it and agree on the plan), after observed queries have moved the masses."""
    w = dataclasses.replace(W.config(1, "small"), ctx=8192 - 37, max_ctx=8192 + 256, rd_budget_bpv=budget)
    B = _binding()
    g = B.Cache(B.config_from_workload(w, 1))
    dev = g.device
    data = W.make_layer(w, 0, "cpu")
    g.gkv_append_demote(0, data["k"].to(dev), data["v"].to(dev), token_mass=data["mass"].to(dev).contiguous())
    out = torch.empty((w.batch, w.n_q_heads, w.d_v), dtype=torch.float32, device=dev)
    for step in range(5):
        tok = W.make_decode_tokens(w, 0, step, "cpu")
        g.gkv_decode_attn_observe(0, tok["q"].to(dev), out)
    torch.cuda.synchronize()
    lv_dev, ms, rg, miss_dev = g.gkv_debug_device_plan(0)
    assert lv_dev.shape[2] == 127 and np.all(ms >= 0) and np.all(rg >= 0)
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            prev = g.gkv_debug_export_levels(0, b, h)
            lv_host, miss_host = B.gkv_debug_replan_levels(g.cfg, g.gkv_ctx_len(0) % 64, ms[b, h], rg[b, h], prev)
            assert np.array_equal(lv_dev[b, h], lv_host), (budget, b, h)
            assert np.all(lv_dev[b, h] <= prev)
            if miss_host:
                assert miss_dev
            # and the oracle's allocator (Sec. 3.3) on the same fp32 numbers
            want, _tau, flag = O.rd_allocate(ms[b, h], rg[b, h], w.d_k, w.d_v, 0, g.gkv_ctx_len(0) % 64, budget, w.n_sink_blocks,
                                             w.retire_after, prev.astype(np.int32), 1)
            assert np.array_equal(lv_dev[b, h].astype(np.int32), np.asarray(want, dtype=np.int32))
            assert bool(flag) == miss_host
    g.close()


@pytest.mark.parametrize("level,ok_span,bad_span", [(8, 1.0e6, 1.1e6), (4, 5.0e4, 7.0e4), (2, 1.2e4, 1.3e4)])
@pytest.mark.parametrize("aligned", [True, False])
def test_value_scale_beyond_the_read_path_is_reported(level, ok_span, bad_span, aligned):
    """A 32-channel value group whose span makes the fp16 scale larger than the read path takes
    (4094) is stored as the quantiser defines it and reported as
    GKV_ERR_RANGE by the next bits report, by the bulk encoder (16-byte aligned rows) and by the general
    one alike; a span just below the limit is not."""
    B = _binding()
    w = _tiny(128, policy=W.POLICY_EXTERNAL)
    plan = np.full((w.batch, w.n_kv_heads, 2), level, dtype=np.int8)
    for span, want in ((ok_span, B.OK), (bad_span, B.ERR_RANGE)):
        g = B.Cache(B.config_from_workload(w))
        dev = g.device
        data = W.make_layer(w, 0, "cpu")
        v = data["v"].clone()
        v[0, 5, 0, 1] = span              # the group's minimum stays near zero: the zero point does not saturate

        def place(t):
            if aligned:
                return t.to(dev).contiguous()
            flat = torch.empty(t.numel() + 8, dtype=t.dtype, device=dev)
            view = flat[2:2 + t.numel()].view(t.shape)
            view.copy_(t.to(dev))
            return view

        g.gkv_append_demote(0, place(data["k"]), place(v), level_plan=plan)
        g.gkv_bits_report(0)
        assert g.last_report_status == want, (level, span, g.last_report_status)
        g.close()
