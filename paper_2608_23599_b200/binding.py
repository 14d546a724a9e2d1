"""ctypes binding of libgkv.so: the same names as include/gkv.h, argument marshalling only.

Every step of the path runs in the CUDA kernels behind the C ABI.  PyTorch is used for device
memory (the arena, inputs, outputs) and for the current CUDA stream.  If the library is missing
or a CUDA device is needed and absent, calls fail loudly; there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from . import build as _build

GKV_ABI_VERSION = 1
POLICY_STAIRCASE, POLICY_RD, POLICY_EXTERNAL = 0, 1, 2
REDUCE_MAX, REDUCE_SUM = 0, 1
TENSOR_K, TENSOR_V = 0, 1
OK = 0
ERR_INVALID_ARG, ERR_ARENA_TOO_SMALL, ERR_CTX_FULL, ERR_BAD_STATE, ERR_UNSUPPORTED = -1, -2, -3, -4, -5
ERR_RANGE, ERR_BUDGET, ERR_CUDA = -6, -7, -8

EXPORTS = [
    "gkv_query_arena_bytes", "gkv_create", "gkv_destroy", "gkv_append_demote", "gkv_decode_attn",
    "gkv_decode_attn_observe", "gkv_debug_export_mass", "gkv_debug_export_bounds", "gkv_rd_reallocate", "gkv_debug_device_plan",
    "gkv_debug_replan_levels",
    "gkv_quest_select", "gkv_quest_select_static", "gkv_debug_export_boxes", "gkv_debug_export_scores", "gkv_bits_report",
    "gkv_debug_export_block", "gkv_debug_export_residual",
    "gkv_debug_export_levels", "gkv_debug_plan_levels", "gkv_ctx_len", "gkv_strerror", "gkv_last_cuda_error",
]


class GkvConfig(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("abi_version", C.c_uint32),
        ("n_layers", C.c_int32), ("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("d_k", C.c_int32), ("d_v", C.c_int32), ("v_aliases_k", C.c_int32), ("max_ctx", C.c_int32),
        ("block_tokens", C.c_int32), ("group", C.c_int32), ("page_tokens", C.c_int32), ("policy", C.c_int32),
        ("stair_tokens", C.c_int32 * 4), ("n_sink_blocks", C.c_int32), ("retire_after", C.c_int32),
        ("rd_budget_bpv", C.c_float), ("residual_fraction", C.c_float), ("quest_reduce", C.c_int32),
        ("monotone_in_age", C.c_int32), ("softmax_scale", C.c_float),
    ]


class GkvBits(C.Structure):
    _fields_ = [
        ("values", C.c_uint64), ("code_bits", C.c_uint64), ("param_bits", C.c_uint64), ("exact_bits", C.c_uint64),
        ("centroid_bits", C.c_uint64), ("tail_bits", C.c_uint64), ("residual_bits", C.c_uint64),
        ("residual_index_bits", C.c_uint64), ("box_bits", C.c_uint64), ("resident_bits", C.c_uint64),
        ("meta_bits", C.c_uint64), ("last_read_bits", C.c_uint64), ("blocks_by_level", C.c_uint64 * 5),
        ("bpv_resident", C.c_double), ("bpv_paper", C.c_double), ("bpv_read", C.c_double),
    ]


class GkvError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {status} ({strerror(status)})")
        self.status = status


_lib = None


def lib_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libgkv.so")


def load():
    """Load libgkv.so (building it is the job of ``build()`` / ``__graft_entry__.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise FileNotFoundError(f"{path} is missing: run `python -m paper_2608_23599_b200.build` first")
    lib = C.CDLL(path)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    lib.gkv_query_arena_bytes.argtypes = [C.POINTER(GkvConfig), C.POINTER(sz)]
    lib.gkv_create.argtypes = [C.POINTER(GkvConfig), vp, sz, C.POINTER(vp)]
    lib.gkv_destroy.argtypes = [vp]
    lib.gkv_append_demote.argtypes = [vp, i32, vp, vp, i32, vp, vp, vp]
    lib.gkv_decode_attn.argtypes = [vp, i32, vp, vp, i32, vp, vp, vp]
    lib.gkv_decode_attn_observe.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
    lib.gkv_debug_export_bounds.argtypes = [vp, i32, vp]
    lib.gkv_debug_export_mass.argtypes = [vp, i32, vp]
    lib.gkv_rd_reallocate.argtypes = [vp, i32, vp]
    lib.gkv_debug_device_plan.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.gkv_debug_replan_levels.argtypes = [C.POINTER(GkvConfig), i32, i32, C.POINTER(C.c_float), C.POINTER(C.c_float),
                                            C.POINTER(C.c_int8), C.POINTER(C.c_int8), C.POINTER(i32)]
    lib.gkv_quest_select.argtypes = [vp, i32, vp, i32, vp, C.POINTER(i32), vp]
    lib.gkv_debug_export_boxes.argtypes = [vp, i32, i32, i32, vp, vp, i32, C.POINTER(i32)]
    lib.gkv_debug_export_scores.argtypes = [vp, i32, vp, vp, vp]
    lib.gkv_quest_select_static.argtypes = [vp, i32, vp, i32, vp, C.POINTER(i32), vp]
    lib.gkv_bits_report.argtypes = [vp, i32, C.POINTER(GkvBits)]
    lib.gkv_debug_export_block.argtypes = [vp, i32, i32, i32, i32, i32, C.POINTER(i32), vp, vp, vp, vp, C.POINTER(i32)]
    lib.gkv_debug_export_residual.argtypes = [vp, i32, i32, i32, vp, i32, C.POINTER(i32)]
    lib.gkv_debug_export_levels.argtypes = [vp, i32, i32, i32, vp, i32, C.POINTER(i32)]
    lib.gkv_debug_plan_levels.argtypes = [C.POINTER(GkvConfig), i32, i32, C.POINTER(C.c_float), C.POINTER(C.c_float),
                                          C.POINTER(C.c_int8), C.POINTER(i32)]
    lib.gkv_ctx_len.argtypes = [vp, i32, C.POINTER(i32)]
    lib.gkv_strerror.argtypes = [C.c_int]
    lib.gkv_strerror.restype = C.c_char_p
    lib.gkv_last_cuda_error.argtypes = [vp]
    for name in EXPORTS:
        if name != "gkv_strerror":
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load().gkv_strerror(status).decode()


def make_config(n_layers, batch, n_q_heads, n_kv_heads, d_k, d_v, max_ctx, *, v_aliases_k=0, page_tokens=0,
                policy=POLICY_STAIRCASE, stair_tokens=(-1, 0, 0, 0), n_sink_blocks=0, retire_after=0,
                rd_budget_bpv=0.0, residual_fraction=0.0, quest_reduce=REDUCE_MAX, monotone_in_age=1,
                softmax_scale=0.0) -> GkvConfig:
    cfg = GkvConfig()
    cfg.struct_size = C.sizeof(GkvConfig)
    cfg.abi_version = GKV_ABI_VERSION
    cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads = n_layers, batch, n_q_heads, n_kv_heads
    cfg.d_k, cfg.d_v, cfg.v_aliases_k, cfg.max_ctx = d_k, d_v, v_aliases_k, max_ctx
    cfg.block_tokens, cfg.group, cfg.page_tokens, cfg.policy = 64, 32, page_tokens, policy
    cfg.stair_tokens = (C.c_int32 * 4)(*stair_tokens)
    cfg.n_sink_blocks, cfg.retire_after = n_sink_blocks, retire_after
    cfg.rd_budget_bpv, cfg.residual_fraction = rd_budget_bpv, residual_fraction
    cfg.quest_reduce, cfg.monotone_in_age, cfg.softmax_scale = quest_reduce, monotone_in_age, softmax_scale
    return cfg


def config_from_workload(w, n_layers: Optional[int] = None) -> GkvConfig:
    return make_config(n_layers or w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.d_k, w.d_v, w.max_ctx,
                       v_aliases_k=w.v_aliases_k, page_tokens=w.page_tokens, policy=w.policy,
                       stair_tokens=tuple(w.stair_tokens), n_sink_blocks=w.n_sink_blocks,
                       retire_after=w.retire_after, rd_budget_bpv=w.rd_budget_bpv,
                       residual_fraction=w.residual_fraction, quest_reduce=getattr(w, "quest_reduce", REDUCE_MAX),
                       softmax_scale=w.softmax_scale)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    return t if isinstance(t, int) else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(rc: int, what: str, allow=()):
    if rc != OK and rc not in allow:
        raise GkvError(rc, what)
    return rc


def gkv_query_arena_bytes(cfg: GkvConfig) -> int:
    out = C.c_size_t(0)
    _check(load().gkv_query_arena_bytes(C.byref(cfg), C.byref(out)), "gkv_query_arena_bytes")
    return out.value


def gkv_debug_plan_levels(cfg: GkvConfig, n_closed: int, n_tail: int = 0, mass=None, rng=None):
    """Host-only level plan of one stream (no device needed): (levels int8 [n_closed], budget_miss)."""
    levels = np.zeros(max(n_closed, 1), dtype=np.int8)
    miss = C.c_int32(0)
    fp = C.POINTER(C.c_float)
    m = None if mass is None else np.ascontiguousarray(mass, dtype=np.float32)
    r = None if rng is None else np.ascontiguousarray(rng, dtype=np.float32)
    _check(load().gkv_debug_plan_levels(C.byref(cfg), n_closed, n_tail,
                                        None if m is None else m.ctypes.data_as(fp),
                                        None if r is None else r.ctypes.data_as(fp),
                                        levels.ctypes.data_as(C.POINTER(C.c_int8)), C.byref(miss)),
           "gkv_debug_plan_levels")
    return levels[:n_closed], bool(miss.value)


def gkv_debug_replan_levels(cfg: GkvConfig, n_tail: int, mass, rng, prev):
    """Host-only plan of a decode-time re-allocation of one stream: (levels int8 [n_closed], budget_miss)."""
    m = np.ascontiguousarray(mass, dtype=np.float32)
    r = np.ascontiguousarray(rng, dtype=np.float32)
    pv = np.ascontiguousarray(prev, dtype=np.int8)
    n = len(pv)
    levels = np.zeros(n, dtype=np.int8)
    miss = C.c_int32(0)
    fp, bp = C.POINTER(C.c_float), C.POINTER(C.c_int8)
    _check(load().gkv_debug_replan_levels(C.byref(cfg), n, n_tail, m.ctypes.data_as(fp), r.ctypes.data_as(fp),
                                          pv.ctypes.data_as(bp), levels.ctypes.data_as(bp), C.byref(miss)),
           "gkv_debug_replan_levels")
    return levels, bool(miss.value)


class Cache:
    """Owner of a gkv_cache handle and of the torch arena behind it."""

    def __init__(self, cfg: GkvConfig, arena_bytes: Optional[int] = None, device="cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("gkv needs a CUDA device: there is no CPU fallback")
        self.cfg = cfg
        self.device = torch.device(device)
        nbytes = gkv_query_arena_bytes(cfg) if arena_bytes is None else arena_bytes
        self.arena = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = self.arena.data_ptr()
        self._arena_ptr = (base + 255) // 256 * 256
        h = C.c_void_p()
        _check(load().gkv_create(C.byref(cfg), self._arena_ptr, nbytes, C.byref(h)), "gkv_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            load().gkv_destroy(self.handle)
            self.handle = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    stream_handle = None   # set to a cudaStream_t (int) to skip the per-call look-up of torch's current stream

    def _st(self) -> int:
        return self.stream_handle if self.stream_handle is not None else _stream()

    def gkv_append_demote(self, layer, k_new, v_new, token_mass=None, level_plan=None, n_new=None):
        """k_new/v_new: cuda bf16 [B][n_new][Hkv][d]; token_mass cuda fp32 [B][Hkv][n_new];
        level_plan: host int8 numpy [B][Hkv][n_new // 64].  Device buffers may be given as tensors or as
        plain integer device addresses (then pass n_new): a serving loop that calls once per layer and step
        keeps its addresses instead of building tensor views."""
        if n_new is None:
            n_new = k_new.shape[1]
        plan_ptr = None
        if level_plan is not None:
            self._plan_keep = level_plan = level_plan.astype("int8", copy=False)
            plan_ptr = level_plan.ctypes.data
        return _check(load().gkv_append_demote(self.handle, layer, _ptr(k_new), _ptr(v_new), n_new,
                                               _ptr(token_mass), plan_ptr, self._st()),
                      "gkv_append_demote", allow=(ERR_RANGE, ERR_BUDGET))

    def gkv_decode_attn(self, layer, q, out, lse=None, page_idx=None, n_sel=0):
        return _check(load().gkv_decode_attn(self.handle, layer, _ptr(q), _ptr(page_idx), n_sel, _ptr(out),
                                             _ptr(lse), self._st()), "gkv_decode_attn")

    def gkv_decode_attn_observe(self, layer, q, out, lse=None, block_mass=None, certificate=None):
        """Full-context decode that also observes the attention mass of every block and updates the
        cache's running masses (block_mass: device fp32 [batch][n_kv_heads][ceil(ctx / 64)] or None;
        certificate: device fp32 [batch][n_q_heads] or None, the error certificate of this query)."""
        return _check(load().gkv_decode_attn_observe(self.handle, layer, _ptr(q), _ptr(out), _ptr(lse), _ptr(block_mass),
                                                     _ptr(certificate), self._st()), "gkv_decode_attn_observe")

    def gkv_debug_export_bounds(self, layer):
        """Per-block certificate bounds as numpy [batch][n_kv_heads][n_closed][4] (kappa, delta, max |v|, 0)."""
        n = self.gkv_ctx_len(layer) // 64
        out = np.zeros((self.cfg.batch, self.cfg.n_kv_heads, n, 4), dtype=np.float32)
        _check(load().gkv_debug_export_bounds(self.handle, layer, out.ctypes.data_as(C.c_void_p)), "gkv_debug_export_bounds")
        return out

    def gkv_debug_device_plan(self, layer):
        """(levels int8, mass fp32, range fp32) as numpy [batch][n_kv_heads][n_closed]: the plan the device
        allocator makes now and the numbers it was made from; flag: a stream missed the budget."""
        n = self.gkv_ctx_len(layer) // 64
        shp = (self.cfg.batch, self.cfg.n_kv_heads, n)
        lv, ms, rg = np.zeros(shp, np.int8), np.zeros(shp, np.float32), np.zeros(shp, np.float32)
        rc = load().gkv_debug_device_plan(self.handle, layer, lv.ctypes.data_as(C.c_void_p), ms.ctypes.data_as(C.c_void_p),
                                          rg.ctypes.data_as(C.c_void_p), self._st())
        _check(rc, "gkv_debug_device_plan", allow=(ERR_BUDGET,))
        return lv, ms, rg, rc == ERR_BUDGET

    def gkv_rd_reallocate(self, layer):
        """Decode-time re-allocation of an RD-policy layer from the running block masses."""
        return _check(load().gkv_rd_reallocate(self.handle, layer, self._st()), "gkv_rd_reallocate",
                      allow=(ERR_RANGE, ERR_BUDGET))

    def gkv_debug_export_mass(self, layer):
        """Running block masses of a layer as a numpy array [batch][n_kv_heads][ceil(ctx / 64)]."""
        n_items = (self.gkv_ctx_len(layer) + 63) // 64
        out = np.zeros((self.cfg.batch, self.cfg.n_kv_heads, n_items), dtype=np.float32)
        _check(load().gkv_debug_export_mass(self.handle, layer, out.ctypes.data_as(C.c_void_p)), "gkv_debug_export_mass")
        return out

    def gkv_debug_export_boxes(self, layer, b, kv_head):
        """Page boxes of one stream: (lo, hi) uint16 arrays [n_pages][d_k] of bf16 bits."""
        page = self.cfg.page_tokens
        cap = (self.gkv_ctx_len(layer) // 64) * (64 // page) if page > 0 else 0
        lo = np.zeros((max(cap, 1), self.cfg.d_k), dtype=np.uint16)
        hi = np.zeros((max(cap, 1), self.cfg.d_k), dtype=np.uint16)
        n = C.c_int32(0)
        _check(load().gkv_debug_export_boxes(self.handle, layer, b, kv_head, lo.ctypes.data_as(C.c_void_p),
                                             hi.ctypes.data_as(C.c_void_p), cap, C.byref(n)), "gkv_debug_export_boxes")
        return lo[: n.value], hi[: n.value]

    def gkv_debug_export_scores(self, layer, q):
        """Page scores of every stream for query q: float32 [batch][n_kv_heads][n_pages]."""
        page = self.cfg.page_tokens
        n_pages = (self.gkv_ctx_len(layer) // 64) * (64 // page) if page > 0 else 0
        out = np.zeros((self.cfg.batch, self.cfg.n_kv_heads, n_pages), dtype=np.float32)
        _check(load().gkv_debug_export_scores(self.handle, layer, _ptr(q), out.ctypes.data_as(C.c_void_p), self._st()),
               "gkv_debug_export_scores")
        return out

    def gkv_quest_select(self, layer, q, budget_tokens, page_idx_out) -> int:
        n = C.c_int32(0)
        _check(load().gkv_quest_select(self.handle, layer, _ptr(q), budget_tokens, _ptr(page_idx_out), C.byref(n),
                                       self._st()), "gkv_quest_select")
        return n.value

    def gkv_quest_select_static(self, layer, q, budget_tokens, page_idx_out) -> int:
        """gkv_quest_select with its score scratch in the library's fixed device array: for callers
        that must not trigger any device allocation.  Same arguments and results."""
        n = C.c_int32(0)
        _check(load().gkv_quest_select_static(self.handle, layer, _ptr(q), budget_tokens, _ptr(page_idx_out),
                                              C.byref(n), self._st()), "gkv_quest_select_static")
        return n.value

    def gkv_bits_report(self, layer=-1) -> GkvBits:
        out = GkvBits()
        # the warnings (a saturated or oversized scale, a missed budget) do not fail the call; the last one is kept
        self.last_report_status = _check(load().gkv_bits_report(self.handle, layer, C.byref(out)), "gkv_bits_report",
                                         allow=(ERR_RANGE, ERR_BUDGET))
        return out

    def gkv_ctx_len(self, layer) -> int:
        n = C.c_int32(0)
        _check(load().gkv_ctx_len(self.handle, layer, C.byref(n)), "gkv_ctx_len")
        return n.value

    def gkv_debug_export_levels(self, layer, b, kv_head):
        import numpy as np
        cap = (self.cfg.max_ctx + 63) // 64
        lv = np.zeros(cap, dtype=np.int8)
        n = C.c_int32(0)
        _check(load().gkv_debug_export_levels(self.handle, layer, b, kv_head, lv.ctypes.data, cap, C.byref(n)),
               "gkv_debug_export_levels")
        return lv[: n.value].astype(np.int32)

    def gkv_debug_export_residual(self, layer, b, kv_head):
        import numpy as np
        cap = self.cfg.max_ctx
        idx = np.zeros(cap, dtype=np.int32)
        n = C.c_int32(0)
        _check(load().gkv_debug_export_residual(self.handle, layer, b, kv_head, idx.ctypes.data, cap, C.byref(n)),
               "gkv_debug_export_residual")
        return idx[: n.value]

    def gkv_debug_export_block(self, layer, b, kv_head, block, which):
        """Returns dict(level, codes u8 [64][d], scale/zero uint16 fp16 bits, rows uint16 bf16 bits, n_rows)."""
        import numpy as np
        d = self.cfg.d_k if which == TENSOR_K else self.cfg.d_v
        codes = np.zeros((64, d), dtype=np.uint8)
        npar = 2 * d if which == TENSOR_K else 64 * (d // 32)
        scale = np.zeros(npar, dtype=np.uint16)
        zero = np.zeros(npar, dtype=np.uint16)
        rows = np.zeros((64, d), dtype=np.uint16)
        level = C.c_int32(0)
        n_rows = C.c_int32(0)
        _check(load().gkv_debug_export_block(self.handle, layer, b, kv_head, block, which, C.byref(level),
                                             codes.ctypes.data, scale.ctypes.data, zero.ctypes.data,
                                             rows.ctypes.data, C.byref(n_rows)), "gkv_debug_export_block")
        shape = (2, d) if which == TENSOR_K else (64, d // 32)
        return dict(level=level.value, codes=codes, scale=scale.reshape(shape), zero=zero.reshape(shape),
                    rows=rows, n_rows=n_rows.value)


def build(force: bool = False, verbose: bool = False) -> str:
    return _build.build(force=force, verbose=verbose)
