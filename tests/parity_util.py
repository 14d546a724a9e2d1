"""Shared helpers for the parity tests: build the oracle cache and the CUDA cache from the same
seeded inputs and compare them (bit-exact discrete state; fp32 outputs within the stated bounds)."""
import numpy as np
import torch

from oracle import gkv_oracle as O
from paper_2608_23599_b200 import workloads as W

ABS_TOL = 2e-3      # max-abs error on fp32-accumulated attention outputs
REL_TOL = 1e-2      # relative L2 error per (sequence, head)


def oracle_config(w: W.Workload, n_layers=None) -> O.Config:
    return O.Config(n_layers=n_layers or w.n_layers, batch=w.batch, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                    d_k=w.d_k, d_v=w.d_v, v_aliases_k=w.v_aliases_k, max_ctx=w.max_ctx, page_tokens=w.page_tokens,
                    policy=w.policy, stair_tokens=tuple(w.stair_tokens), n_sink_blocks=w.n_sink_blocks,
                    retire_after=w.retire_after, rd_budget_bpv=w.rd_budget_bpv,
                    residual_fraction=w.residual_fraction, quest_reduce=w.quest_reduce, softmax_scale=w.softmax_scale)


def f32(t):
    return None if t is None else t.detach().to("cpu").to(torch.float32).numpy()


def ingest_both(w, layer, data, ocache, gcache, level_plan=None):
    """data: dict from workloads.make_layer on CPU."""
    mass = data.get("mass")
    ocache.append_demote(layer, f32(data["k"]), f32(data.get("v")),
                         token_mass=None if mass is None else mass.numpy(), level_plan=level_plan)
    dev = gcache.device
    gcache.gkv_append_demote(layer, data["k"].to(dev), None if data.get("v") is None else data["v"].to(dev),
                             token_mass=None if mass is None else mass.to(dev).contiguous(),
                             level_plan=level_plan)


def assert_state_equal(ocache, gcache, layer, streams=None, blocks=None):
    """Levels, codes, scale/zero, exact rows, centroids and residual indices, bit for bit."""
    from paper_2608_23599_b200 import binding as B
    cfg = ocache.cfg
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            if streams is not None and (b, h) not in streams:
                continue
            st = ocache.streams[(layer, b, h)]
            lv_g = gcache.gkv_debug_export_levels(layer, b, h)
            lv_o = ocache.levels(layer, b, h)
            assert np.array_equal(lv_g, lv_o), f"levels differ stream {(b, h)}: {lv_g} vs {lv_o}"
            assert np.array_equal(gcache.gkv_debug_export_residual(layer, b, h), st.res_idx), "residual indices"
            todo = range(st.n_closed) if blocks is None else [i for i in blocks if i < st.n_closed]
            for i in todo:
                blk = st.blocks[i]
                tensors = ((B.TENSOR_K, "k"),) if cfg.v_aliases_k else ((B.TENSOR_K, "k"), (B.TENSOR_V, "v"))
                for which, name in tensors:
                    ex = gcache.gkv_debug_export_block(layer, b, h, i, which)
                    assert ex["level"] == blk.level
                    tag = f"layer {layer} stream {(b, h)} block {i} {name} level {blk.level}"
                    if blk.level == 16:
                        want = O.bf16_bits(getattr(blk, f"{name}_exact"))
                        assert np.array_equal(ex["rows"], want), tag
                    elif blk.level == 1:
                        want = O.bf16_bits(getattr(blk, f"{name}_cent"))
                        assert np.array_equal(ex["rows"][0], want), tag
                    else:
                        assert np.array_equal(ex["scale"], getattr(blk, f"{name}_scale").view(np.uint16)), tag + " scale"
                        assert np.array_equal(ex["zero"], getattr(blk, f"{name}_zero").view(np.uint16)), tag + " zero"
                        assert np.array_equal(ex["codes"], getattr(blk, f"{name}_codes")), tag + " codes"
            if st.n_tail and blocks is None:
                ex = gcache.gkv_debug_export_block(layer, b, h, st.n_closed, B.TENSOR_K)
                assert ex["n_rows"] == st.n_tail
                assert np.array_equal(ex["rows"][: st.n_tail], O.bf16_bits(st.tail_k))
                if not cfg.v_aliases_k:
                    ex = gcache.gkv_debug_export_block(layer, b, h, st.n_closed, B.TENSOR_V)
                    assert np.array_equal(ex["rows"][: st.n_tail], O.bf16_bits(st.tail_v))


def assert_boxes_and_scores_equal(ocache, gcache, layer, q_bf16, streams=None):
    """Page boxes (exact per-page per-channel key minima / maxima) and page scores of every stream,
    bit for bit against the oracle's."""
    cfg = ocache.cfg
    scores_g = gcache.gkv_debug_export_scores(layer, q_bf16.to(gcache.device))
    scores_o = ocache.quest_scores(layer, f32(q_bf16))
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            if streams is not None and (b, h) not in streams:
                continue
            st = ocache.streams[(layer, b, h)]
            n_pages = st.n_closed * (64 // cfg.page_tokens)
            lo, hi = gcache.gkv_debug_export_boxes(layer, b, h)
            assert lo.shape == (n_pages, cfg.d_k)
            if n_pages:
                assert np.array_equal(lo, O.bf16_bits(np.stack(st.box_lo[:n_pages]))), f"box minima of stream {(b, h)}"
                assert np.array_equal(hi, O.bf16_bits(np.stack(st.box_hi[:n_pages]))), f"box maxima of stream {(b, h)}"
            want = scores_o[(b, h)]
            assert np.array_equal(scores_g[b, h].view(np.uint32), want.view(np.uint32)), f"page scores of stream {(b, h)}"


def assert_outputs_close(out_gpu, out_oracle, what=""):
    """Plain max-abs error <= ABS_TOL over all outputs and relative L2 error <= REL_TOL per
    (sequence, head).  Returns (max-abs error, largest relative error)."""
    g = out_gpu.detach().to("cpu").to(torch.float64).numpy()
    o = np.asarray(out_oracle, dtype=np.float64)
    assert g.shape == o.shape
    assert np.all(np.isfinite(g)), f"{what}: non-finite output"
    err = np.abs(g - o).max()
    assert err <= ABS_TOL, f"{what}: max-abs error {err:.3e} > {ABS_TOL}"
    num = np.linalg.norm(g - o, axis=-1)
    den = np.linalg.norm(o, axis=-1) + 1e-30
    rel = (num / den).max()
    assert rel <= REL_TOL, f"{what}: relative error {rel:.3e} > {REL_TOL}"
    return err, rel


def decode_both(ocache, gcache, layer, q_bf16, page_idx_gpu=None, n_sel=0, page_idx_oracle=None):
    cfg = ocache.cfg
    dev = gcache.device
    out = torch.empty((cfg.batch, cfg.n_q_heads, cfg.d_v), dtype=torch.float32, device=dev)
    lse = torch.empty((cfg.batch, cfg.n_q_heads), dtype=torch.float32, device=dev)
    gcache.gkv_decode_attn(layer, q_bf16.to(dev), out, lse, page_idx=page_idx_gpu, n_sel=n_sel)
    torch.cuda.synchronize()
    o_out, o_lse = ocache.decode_attn(layer, f32(q_bf16), page_idx_oracle)
    return out, lse, o_out, o_lse
