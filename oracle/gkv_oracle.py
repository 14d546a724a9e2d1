"""CPU oracle for graded KV-cache decode attention (Geodesia-KV hot path).

TEST INFRASTRUCTURE ONLY.  This is a plain, slow, obviously-correct numpy
implementation of what the path computes.  It shares no code with the CUDA
library, is never imported by it, and may only be used by ``tests/``, the
smoke check and the benchmark's ``cpu_baseline`` / reference leg.

What it follows (paper sections / equations):

* Precision ladder, 64-token blocks, keys grouped along time and values along
  channels, centroid tier, monotone demotion (Sec. 3.2).
* Lagrangian allocator: tolerance eps_t = tau / (N_b m_b), bit depth
  b* = ceil(log2(c |q| e_b / (2 eps_t) + 1)), snapped to the ladder (Sec. 3.3,
  Eq. 4-5).
* Exact residual ranked by s_j = a_j |v_j - vbar_b(j)|^2 (Sec. 3.4, Eq. 6).
* Compressed-Quest: exact per-page key min/max boxes taken before
  quantisation, box upper bound ranks closed pages, current partial page always
  readable, cold pages hard-masked; resident / read accounting (Sec. 3.5,
  Eq. 7-8).
* Attention error certificate (Sec. 3.6, Eq. 9) - used as a pin in the tests.
* Block attention mass m_b (Sec. 3.1, Eq. 2): the summed softmax weight of a
  block's tokens, averaged over the KV head's query heads, and its running
  update m_b <- 0.9 m_b + 0.1 m_b_new at every observed decode query.
* Dense softmax attention over the reconstructed cache (Sec. 3.1, Eq. 1;
  Sec. 3.7) evaluated in float64.

Pinned by tests/test_oracle_pins.py (closed forms, brute force, the paper's
printed accounting identities, invariants).  The paper prints no numeric
example of a code, score or output, so *values* are pinned only through those
properties ("parity unpinned by the paper" for raw tensor values).

Numeric rules (needed because discrete outputs must be reproducible bit for
bit by an independent implementation; the paper is silent on all of them):

N0  bf16<->fp32 and fp16<->fp32 are round-to-nearest-even; inputs finite.
N1  Arithmetic feeding a discrete decision is IEEE fp32 (fp64 where stated),
    one rounding per written operation; every sum is sequential in ascending
    index.
N2  Dequant: x^ = fp32(code * s) + z  (code*s is exact in fp32, so this equals
    a fused multiply-add).
N3  Quantise a group to L bits, qmax = 2^L - 1: mn = min, mx = max,
    s = fp16((mx - mn) / qmax), z = fp16(mn) (both saturating at +-65504),
    inv = 1/s if s > 0 else 0, code = clamp(rint((x - z) * inv), 0, qmax),
    ties to even.
N4  Centroid: sequential fp32 sum over the 64 tokens of the block's current
    reconstruction, times 1/64, rounded to bf16.
N5  Box: exact per-page per-channel min / max of the original bf16 keys.
N6  Page score per head: acc <- acc + q_d * (hi_d if q_d >= 0 else lo_d),
    sequential in d, fp32 (each product of two bf16 is exact in fp32); reduce
    over the KV head's query heads with max (or sequential sum).
N7  Residual score: err = sum_c (v_c - vbar_c)^2 sequential in fp64,
    score = fp32(a_j * err).
N8  Top-k: order by (score descending, index ascending), take k, emit
    ascending by index; -0 == +0.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

P = 64            # tokens per block (Sec. 3.2)
G = 32            # quantisation group (keys: 32 tokens x 1 channel; values: 1 token x 32 channels)
LADDER = (16, 8, 4, 2, 1)          # 1 = centroid tier
POLICY_STAIRCASE, POLICY_RD, POLICY_EXTERNAL = 0, 1, 2
REDUCE_MAX, REDUCE_SUM = 0, 1
FP16_MAX = np.float32(65504.0)
F32 = np.float32


# --------------------------------------------------------------------------------------
# N0: conversions
# --------------------------------------------------------------------------------------
def bf16_round(x) -> np.ndarray:
    """fp32 -> nearest bf16 (ties to even), returned as fp32 holding that value."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    u = (u + 0x7FFF + lsb) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x) -> np.ndarray:
    """fp32 array holding bf16-representable values -> uint16 bit patterns."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


def fp16_sat(x) -> np.ndarray:
    """fp32 -> fp16 RNE, saturating at +-65504 (N3)."""
    x = np.clip(np.asarray(x, dtype=np.float32), -FP16_MAX, FP16_MAX)
    return x.astype(np.float16)


def beta_bits(level: int) -> float:
    """Bits per value of a ladder level incl. fp16 scale + zero per group of 32
    (Sec. 1 contribution 2: 'including the exact scale overhead')."""
    if level == 16:
        return 16.0
    if level == 1:
        return 16.0 / P
    return level + 32.0 / G


# --------------------------------------------------------------------------------------
# N2 / N3: scalar quantiser.  Groups lie along the LAST axis of x.
# --------------------------------------------------------------------------------------
def quantize_groups(x, bits: int):
    """x: fp32 [..., n_groups, G].  Returns (codes uint8 same shape, scale fp16 [..., n_groups],
    zero fp16 [..., n_groups], range_flag)."""
    x = np.asarray(x, dtype=np.float32)
    qmax = F32(2 ** bits - 1)
    mn = x.min(axis=-1)
    mx = x.max(axis=-1)
    s_raw = (mx - mn) / qmax                      # fp32 subtract, fp32 divide
    flag = bool(np.any(np.abs(s_raw) > FP16_MAX) or np.any(np.abs(mn) > FP16_MAX))
    s = fp16_sat(s_raw)
    z = fp16_sat(mn)
    s32 = s.astype(np.float32)
    z32 = z.astype(np.float32)
    with np.errstate(divide="ignore"):
        inv = np.where(s32 > 0, F32(1.0) / s32, F32(0.0)).astype(np.float32)
    t = (x - z32[..., None]) * inv[..., None]     # fp32 subtract, then fp32 multiply
    code = np.clip(np.rint(t), F32(0.0), qmax)    # rint = ties to even
    return code.astype(np.uint8), s, z, flag


def dequantize_groups(codes, scale, zero):
    """N2.  codes [..., n_groups, G] uint8, scale/zero fp16 [..., n_groups] -> fp32."""
    c = codes.astype(np.float32)
    prod = c * scale.astype(np.float32)[..., None]          # exact (<= 19 significant bits)
    return (prod + zero.astype(np.float32)[..., None]).astype(np.float32)


def quantize_k_block(xk, bits):
    """Keys: groups run along TIME - 32 tokens x 1 channel (Sec. 3.2).
    xk fp32 [64][d].  Returns codes [64][d], scale/zero fp16 [2][d]."""
    d = xk.shape[1]
    g = xk.reshape(P // G, G, d).transpose(0, 2, 1)          # [half][channel][32 tokens]
    code, s, z, flag = quantize_groups(g, bits)
    return code.transpose(0, 2, 1).reshape(P, d), s, z, flag


def dequantize_k_block(codes, s, z):
    d = codes.shape[1]
    g = codes.reshape(P // G, G, d).transpose(0, 2, 1)
    return dequantize_groups(g, s, z).transpose(0, 2, 1).reshape(P, d)


def quantize_v_block(xv, bits):
    """Values: groups run along CHANNELS - 1 token x 32 channels (Sec. 3.2).
    xv fp32 [64][d].  Returns codes [64][d], scale/zero fp16 [64][d/32]."""
    d = xv.shape[1]
    g = xv.reshape(P, d // G, G)
    code, s, z, flag = quantize_groups(g, bits)
    return code.reshape(P, d), s, z, flag


def dequantize_v_block(codes, s, z):
    d = codes.shape[1]
    return dequantize_groups(codes.reshape(P, d // G, G), s, z).reshape(P, d)


def centroid_of(x):
    """N4.  x fp32 [64][d] -> bf16-rounded mean (fp32 holding bf16 values)."""
    acc = np.zeros(x.shape[1], dtype=np.float32)
    for t in range(x.shape[0]):
        acc = (acc + x[t].astype(np.float32)).astype(np.float32)
    return bf16_round(acc * F32(1.0 / P))


# --------------------------------------------------------------------------------------
# N8: top-k
# --------------------------------------------------------------------------------------
def topk_ascending(scores, k: int) -> np.ndarray:
    """Indices of the k largest scores, ties to the lower index, emitted ascending."""
    scores = np.asarray(scores, dtype=np.float32) + F32(0.0)      # -0 -> +0
    n = scores.shape[0]
    k = min(k, n)
    order = sorted(range(n), key=lambda i: (-float(scores[i]), i))
    return np.array(sorted(order[:k]), dtype=np.int32)


# --------------------------------------------------------------------------------------
# cache state
# --------------------------------------------------------------------------------------
@dataclass
class Block:
    level: int
    # level 16
    k_exact: Optional[np.ndarray] = None     # fp32 [64][dk] (bf16 values)
    v_exact: Optional[np.ndarray] = None
    # levels 8/4/2
    k_codes: Optional[np.ndarray] = None     # uint8 [64][dk]
    k_scale: Optional[np.ndarray] = None     # fp16 [2][dk]
    k_zero: Optional[np.ndarray] = None
    v_codes: Optional[np.ndarray] = None     # uint8 [64][dv]
    v_scale: Optional[np.ndarray] = None     # fp16 [64][dv/32]
    v_zero: Optional[np.ndarray] = None
    # level 1
    k_cent: Optional[np.ndarray] = None      # fp32 [dk] (bf16 values)
    v_cent: Optional[np.ndarray] = None
    history: List[int] = field(default_factory=list)
    # error bounds carried for the certificate (Sec. 3.6): kappa >= max_j |k_j - k^_j|_2 and
    # delta >= max_j |v_j - v^_j|_2 against the ORIGINAL rows, vnorm = max_j |v_j|_2 of the originals
    kappa: float = 0.0
    delta: float = 0.0
    vnorm: float = 0.0

    def recon_k(self) -> np.ndarray:
        if self.level == 16:
            return self.k_exact
        if self.level == 1:
            return np.broadcast_to(self.k_cent, (P, self.k_cent.shape[0]))
        return dequantize_k_block(self.k_codes, self.k_scale, self.k_zero)

    def recon_v(self) -> np.ndarray:
        if self.level == 16:
            return self.v_exact
        if self.level == 1:
            return np.broadcast_to(self.v_cent, (P, self.v_cent.shape[0]))
        return dequantize_v_block(self.v_codes, self.v_scale, self.v_zero)


def _max_row_norm(x) -> float:
    x = np.asarray(x, dtype=np.float64)
    return float(np.sqrt((x * x).sum(axis=1)).max())


def make_block(level: int, xk: np.ndarray, xv: Optional[np.ndarray], history=None, parent: Optional["Block"] = None
               ) -> Tuple[Block, bool]:
    """Encode current (fp32) block contents at ``level``.  xv None = values alias keys (MLA).

    parent = the block these contents were reconstructed from (None: xk / xv are the original
    rows).  The error bounds of Sec. 3.6 follow the requantisation chain by the triangle
    inequality: bound(new) = bound(parent) + max_j |x^_parent,j - x^_new,j|_2."""
    hist = list(history or []) + [level]
    flag = False
    if level == 16:
        b = Block(16, k_exact=xk.astype(np.float32), v_exact=None if xv is None else xv.astype(np.float32), history=hist)
    elif level == 1:
        b = Block(1, k_cent=centroid_of(xk), v_cent=None if xv is None else centroid_of(xv), history=hist)
    else:
        kc, ks, kz, f1 = quantize_k_block(xk, level)
        b = Block(level, k_codes=kc, k_scale=ks, k_zero=kz, history=hist)
        flag = f1
        if xv is not None:
            b.v_codes, b.v_scale, b.v_zero, f2 = quantize_v_block(xv, level)
            flag = flag or f2
    b.kappa = (parent.kappa if parent else 0.0) + _max_row_norm(np.asarray(xk, np.float64) - b.recon_k())
    if xv is not None:
        b.delta = (parent.delta if parent else 0.0) + _max_row_norm(np.asarray(xv, np.float64) - b.recon_v())
        b.vnorm = parent.vnorm if parent else _max_row_norm(xv)
    return b, flag


@dataclass
class Stream:
    """One (sequence, KV head) of one layer."""
    d_k: int
    d_v: int
    alias: bool
    blocks: List[Block] = field(default_factory=list)
    tail_k: Optional[np.ndarray] = None          # fp32 [n_tail][dk]
    tail_v: Optional[np.ndarray] = None
    box_lo: List[np.ndarray] = field(default_factory=list)   # per closed page, fp32 [dk]
    box_hi: List[np.ndarray] = field(default_factory=list)
    res_idx: np.ndarray = field(default_factory=lambda: np.zeros(0, np.int32))
    res_k: Optional[np.ndarray] = None           # fp32 [n_res][dk]
    res_v: Optional[np.ndarray] = None
    range_flag: bool = False
    budget_flag: bool = False
    ema_mass: np.ndarray = field(default_factory=lambda: np.zeros(0, np.float64))   # running m_b, one per block (+ partial block)
    range_b: List[float] = field(default_factory=list)       # fp32 range proxy e_b of every closed block (Sec. 3.3)

    @property
    def n_closed(self) -> int:
        return len(self.blocks)

    @property
    def n_tail(self) -> int:
        return 0 if self.tail_k is None else self.tail_k.shape[0]

    @property
    def ctx(self) -> int:
        return self.n_closed * P + self.n_tail


@dataclass
class Config:
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    d_k: int
    d_v: int
    v_aliases_k: int = 0
    max_ctx: int = 1 << 30
    page_tokens: int = 0
    policy: int = POLICY_STAIRCASE
    stair_tokens: Tuple[int, int, int, int] = (-1, 0, 0, 0)
    n_sink_blocks: int = 0
    retire_after: int = 0
    rd_budget_bpv: float = 0.0
    residual_fraction: float = 0.0
    quest_reduce: int = REDUCE_MAX
    softmax_scale: float = 0.0
    monotone_in_age: int = 1


# --------------------------------------------------------------------------------------
# policies
# --------------------------------------------------------------------------------------
def staircase_levels(n_closed: int, stair_tokens, n_sink_blocks: int) -> np.ndarray:
    """Level per closed block (index 0 = oldest) from rung widths given newest-first in
    tokens (-1 = unbounded); whatever is older than all four rungs is centroid; sink
    blocks stay exact (Fig. 1: sinks and recent window at 16 bits)."""
    lv = np.ones(n_closed, dtype=np.int32)
    edges = []
    acc = 0
    for wtok in stair_tokens:
        if wtok < 0:
            acc = None
        elif acc is not None:
            acc += wtok // P
        edges.append(acc)
    for i in range(n_closed):
        age = n_closed - 1 - i
        level = 1
        for e, L in zip(edges, (16, 8, 4, 2)):
            if e is None or age < e:
                level = L
                break
        if i < n_sink_blocks:
            level = 16
        lv[i] = level
    return lv


def block_bits(level: int, d_k: int, d_v: int, alias: bool) -> int:
    """Resident bits of one closed block at ``level`` (codes + fp16 scale/zero, or centroid)."""
    nval = P * (d_k if alias else d_k + d_v)
    if level == 16:
        return 16 * nval
    if level == 1:
        return 16 * (d_k if alias else d_k + d_v)
    return level * nval + (nval // G) * 32


def _levels_for_tau(y, tau, pinned, prev, monotone_in_age):
    """Per-block ladder level for multiplier tau (Sec. 3.3), then the projections:
    pinned blocks exact, never above the previous level, non-decreasing toward recent."""
    n = len(y)
    # b bits suffice iff y_b <= tau * (2^b - 1); snap UP to the ladder; b* <= 1 -> centroid
    lv = np.where(y <= tau, 1,
         np.where(y <= tau * 3.0, 2,
         np.where(y <= tau * 15.0, 4,
         np.where(y <= tau * 255.0, 8, 16)))).astype(np.int32)
    for b in range(n):
        if pinned[b]:
            lv[b] = 16
        if prev is not None:
            lv[b] = min(lv[b], prev[b])
    if monotone_in_age:
        nxt = None
        for b in range(n - 1, -1, -1):
            if pinned[b]:
                continue
            if nxt is not None:
                lv[b] = min(lv[b], nxt)
            nxt = lv[b]
    return lv


def rd_allocate(mass_b, range_b, d_k, d_v, alias, n_tail, budget_bpv, n_sink_blocks, retire_after,
                prev=None, monotone_in_age=1):
    """Monotone rate-distortion allocator (Sec. 3.3).

    mass_b fp32 [n], range_b fp32 [n].  The paper's b* = ceil(log2(c|q| e_b / (2 eps_t) + 1))
    with eps_t = tau/(N_b m_b) says 'b bits suffice iff  c|q| N_b m_b e_b / 2 <= tau (2^b - 1)';
    the constants are absorbed by tau, so the test is y_b = m_b e_b <= tau (2^b - 1) in fp64.
    tau is the smallest breakpoint {y_b / k, k in 1,3,15,255} U {0} whose plan fits the
    budget.  Returns (levels, tau, budget_flag)."""
    n = len(mass_b)
    y = np.asarray(mass_b, dtype=np.float64) * np.asarray(range_b, dtype=np.float64)
    pinned = np.zeros(n, dtype=bool)
    recent_blocks = retire_after // P
    for b in range(n):
        age = n - 1 - b
        if b < n_sink_blocks or age < recent_blocks:
            pinned[b] = True
    nval_tok = d_k if alias else d_k + d_v
    T = n * P + n_tail
    budget_bits = int(math.floor(float(np.float32(budget_bpv)) * float(T * nval_tok)))
    tail_bits = n_tail * 16 * nval_tok

    def total_bits(lv):
        return sum(block_bits(int(L), d_k, d_v, alias) for L in lv) + tail_bits

    cands = {0.0}
    for b in range(n):
        for k in (1.0, 3.0, 15.0, 255.0):
            cands.add(float(y[b] / k))
    cands = sorted(cands)
    for tau in cands:                      # ascending: first feasible = smallest feasible
        lv = _levels_for_tau(y, tau, pinned, prev, monotone_in_age)
        if total_bits(lv) <= budget_bits:
            return lv, tau, False
    return lv, cands[-1], True             # even the largest tau misses the budget: flagged


def rd_residual_select(token_mass, v_tokens, levels, n_sink_blocks, fraction, ctx):
    """Exact-residual selection (Sec. 3.4, Eq. 6).  token_mass fp32 [ctx]; v_tokens fp32
    [n_closed*64][dv] original values; levels per closed block.  Eligible: tokens of closed,
    non-sink blocks whose planned level is below 16.  Returns ascending token indices."""
    n_closed = len(levels)
    n_res = int(math.floor(float(np.float32(fraction)) * float(ctx)))
    scores = np.full(n_closed * P, -1.0, dtype=np.float32)
    eligible = np.zeros(n_closed * P, dtype=bool)
    for b in range(n_closed):
        if b < n_sink_blocks or levels[b] == 16:
            continue
        blk = v_tokens[b * P:(b + 1) * P].astype(np.float32)
        cen = centroid_of(blk).astype(np.float64)              # value centroid of the block (N4)
        rows = blk.astype(np.float64)
        err = np.zeros(P, dtype=np.float64)
        for c in range(blk.shape[1]):                          # sequential in c, fp64 (N7)
            dlt = rows[:, c] - cen[c]
            err = err + dlt * dlt
        mass = np.asarray(token_mass[b * P:(b + 1) * P], dtype=np.float64)
        scores[b * P:(b + 1) * P] = (mass * err).astype(np.float32)
        eligible[b * P:(b + 1) * P] = True
    idx_e = np.nonzero(eligible)[0]
    n_res = min(n_res, len(idx_e))
    if n_res == 0:
        return np.zeros(0, np.int32)
    sel = topk_ascending(scores[idx_e], n_res)
    return idx_e[sel].astype(np.int32)


# --------------------------------------------------------------------------------------
# the cache object
# --------------------------------------------------------------------------------------
class GradedCache:
    """Logical graded KV cache: a dict of Streams keyed by (layer, b, kv_head)."""

    def __init__(self, cfg: Config):
        self.cfg = cfg
        self.alias = bool(cfg.v_aliases_k)
        self.streams: Dict[Tuple[int, int, int], Stream] = {}
        for l in range(cfg.n_layers):
            for b in range(cfg.batch):
                for h in range(cfg.n_kv_heads):
                    self.streams[(l, b, h)] = Stream(cfg.d_k, cfg.d_v, self.alias)
        self.last_read_bits: Dict[int, int] = {}
        self.last_box_bits: Dict[int, int] = {}        # boxes scored by a quest_select that no read has used yet
        self.last_read_box_bits: Dict[int, int] = {}   # boxes that count for the last read

    @property
    def scale(self) -> float:
        c = self.cfg
        return float(np.float32(c.softmax_scale)) if c.softmax_scale > 0 else float(np.float32(1.0 / math.sqrt(c.d_k)))

    # -- append + demote ---------------------------------------------------------------
    def append_demote(self, layer: int, k_new, v_new, token_mass=None, level_plan=None):
        """k_new fp32 [B][n_new][Hkv][dk] (bf16 values); v_new likewise or None (alias).
        n_new == 1 is a decode step; larger n_new on an empty stream is bulk ingest."""
        cfg = self.cfg
        n_new = k_new.shape[1]
        for b in range(cfg.batch):
            for h in range(cfg.n_kv_heads):
                st = self.streams[(layer, b, h)]
                kk = np.asarray(k_new[b, :, h], dtype=np.float32)
                vv = None if self.alias else np.asarray(v_new[b, :, h], dtype=np.float32)
                tm = None if token_mass is None else np.asarray(token_mass[b, h], dtype=np.float32)
                lp = None if level_plan is None else np.asarray(level_plan[b, h])
                if st.ctx == 0 and n_new > 1:
                    self._bulk_ingest(st, kk, vv, tm, lp)
                else:
                    for t in range(n_new):
                        self._append_one(st, kk[t], None if vv is None else vv[t])

    def _close_boxes(self, st: Stream, xk: np.ndarray):
        """N5: exact per-page min/max of the unquantised keys, recorded at block close."""
        page = self.cfg.page_tokens
        if page <= 0:
            return
        for p0 in range(0, P, page):
            st.box_lo.append(xk[p0:p0 + page].min(axis=0).astype(np.float32))
            st.box_hi.append(xk[p0:p0 + page].max(axis=0).astype(np.float32))

    def _bulk_ingest(self, st: Stream, kk, vv, token_mass, level_plan):
        cfg = self.cfg
        T = kk.shape[0]
        n_closed = T // P
        n_tail = T - n_closed * P
        for i in range(n_closed):
            self._close_boxes(st, kk[i * P:(i + 1) * P])
        if cfg.policy == POLICY_STAIRCASE:
            levels = staircase_levels(n_closed, cfg.stair_tokens, cfg.n_sink_blocks)
        elif cfg.policy == POLICY_EXTERNAL:
            levels = np.asarray(level_plan[:n_closed], dtype=np.int32)
        else:
            mass_b = np.zeros(n_closed, dtype=np.float32)
            range_b = np.zeros(n_closed, dtype=np.float32)
            for i in range(n_closed):
                acc = F32(0.0)
                for t in range(P):
                    acc = F32(acc + token_mass[i * P + t])
                mass_b[i] = acc
                blk = kk[i * P:(i + 1) * P]
                range_b[i] = np.max(blk.max(axis=0) - blk.min(axis=0))     # fp32 subtract, exact max
            levels, _tau, bflag = rd_allocate(mass_b, range_b, cfg.d_k, cfg.d_v, self.alias, n_tail,
                                              cfg.rd_budget_bpv, cfg.n_sink_blocks, cfg.retire_after,
                                              None, cfg.monotone_in_age)
            st.budget_flag = bflag
            st.range_b = [np.float32(x) for x in range_b]
            st.ema_mass = mass_b.astype(np.float64)        # the prefill observer's masses start the running average
        if cfg.residual_fraction > 0 and token_mass is not None:
            vsrc = kk[:, :cfg.d_v] if self.alias else vv
            st.res_idx = rd_residual_select(token_mass, vsrc[:n_closed * P], levels, cfg.n_sink_blocks,
                                            cfg.residual_fraction, T)
            st.res_k = kk[st.res_idx].copy()
            st.res_v = None if self.alias else vv[st.res_idx].copy()
        for i in range(n_closed):
            blk, flag = make_block(int(levels[i]), kk[i * P:(i + 1) * P],
                                   None if self.alias else vv[i * P:(i + 1) * P])
            st.range_flag |= flag
            st.blocks.append(blk)
        st.tail_k = kk[n_closed * P:].copy()
        st.tail_v = None if self.alias else vv[n_closed * P:].copy()

    def _append_one(self, st: Stream, k_row, v_row):
        cfg = self.cfg
        if st.tail_k is None:
            st.tail_k = np.zeros((0, cfg.d_k), np.float32)
            st.tail_v = None if self.alias else np.zeros((0, cfg.d_v), np.float32)
        st.tail_k = np.concatenate([st.tail_k, k_row[None]], axis=0)
        if not self.alias:
            st.tail_v = np.concatenate([st.tail_v, v_row[None]], axis=0)
        if st.tail_k.shape[0] < P:
            return
        # the tail block closes: boxes from unquantised keys, block enters at level 16
        self._close_boxes(st, st.tail_k)
        if cfg.policy == POLICY_RD:
            st.range_b.append(np.float32(np.max(st.tail_k.max(axis=0) - st.tail_k.min(axis=0))))
        blk, _ = make_block(16, st.tail_k, st.tail_v)
        st.blocks.append(blk)
        st.tail_k = np.zeros((0, cfg.d_k), np.float32)
        st.tail_v = None if self.alias else np.zeros((0, cfg.d_v), np.float32)
        if cfg.policy == POLICY_STAIRCASE:
            target = staircase_levels(st.n_closed, cfg.stair_tokens, cfg.n_sink_blocks)
            for i, blk in enumerate(st.blocks):
                if target[i] < blk.level:              # monotone: levels only fall (Sec. 3.2)
                    self._demote(st, i, int(target[i]))

    def rd_reallocate(self, layer: int):
        """Decode-time re-allocation (Sec. 3.1-3.3): the allocator of Eq. 4 run again on the running
        block masses (rounded to fp32, the precision they are kept in) and the range proxies taken
        when the blocks closed, at the budget of the current context, under the temporal constraint
        of Sec. 3.2 - no level rises, sinks and the recent window stay exact.  Blocks whose level
        falls are requantised from their current reconstruction.  Returns {(b, h): levels}."""
        cfg = self.cfg
        plans = {}
        for b in range(cfg.batch):
            for h in range(cfg.n_kv_heads):
                st = self.streams[(layer, b, h)]
                n = st.n_closed
                if n == 0:
                    continue
                mass = np.zeros(n, dtype=np.float32)
                mass[:min(n, len(st.ema_mass))] = np.asarray(st.ema_mass[:n], dtype=np.float32)
                prev = np.array([blk.level for blk in st.blocks], dtype=np.int32)
                levels, _tau, flag = rd_allocate(mass, np.asarray(st.range_b[:n], dtype=np.float32), cfg.d_k, cfg.d_v,
                                                 self.alias, st.n_tail, cfg.rd_budget_bpv, cfg.n_sink_blocks,
                                                 cfg.retire_after, prev, cfg.monotone_in_age)
                st.budget_flag |= flag
                for i in range(n):
                    if levels[i] < st.blocks[i].level:
                        self._demote(st, i, int(levels[i]))
                plans[(b, h)] = np.asarray(levels, dtype=np.int32)
        return plans

    def _demote(self, st: Stream, i: int, new_level: int):
        """Requantise block i from its CURRENT reconstruction (the dense data no longer
        exists, Sec. 3.2); never upward."""
        old = st.blocks[i]
        assert new_level < old.level, "promotion is forbidden"
        xk = np.asarray(old.recon_k(), dtype=np.float32)
        xv = None if self.alias else np.asarray(old.recon_v(), dtype=np.float32)
        st.blocks[i], flag = make_block(new_level, xk, xv, old.history, parent=old)
        st.range_flag |= flag

    def demote_to(self, layer: int, b: int, h: int, block: int, new_level: int):
        self._demote(self.streams[(layer, b, h)], block, new_level)

    # -- reconstruction + attention ----------------------------------------------------
    def reconstruct(self, st: Stream):
        """Logical cache the attention sees: (K~ [T][dk], V~ [T][dv], ) in float64 with
        residual tokens replaced by their exact rows."""
        ks = [np.asarray(b.recon_k(), dtype=np.float64) for b in st.blocks]
        if st.n_tail:
            ks.append(st.tail_k.astype(np.float64))
        K = np.concatenate(ks, axis=0) if ks else np.zeros((0, st.d_k))
        if self.alias:
            V = K[:, :st.d_v]
        else:
            vs = [np.asarray(b.recon_v(), dtype=np.float64) for b in st.blocks]
            if st.n_tail:
                vs.append(st.tail_v.astype(np.float64))
            V = np.concatenate(vs, axis=0)
        if len(st.res_idx):
            K = K.copy()
            K[st.res_idx] = st.res_k.astype(np.float64)
            if self.alias:
                V = K[:, :st.d_v]
            else:
                V = V.copy()
                V[st.res_idx] = st.res_v.astype(np.float64)
        return K, V

    def token_mask(self, st: Stream, page_idx) -> np.ndarray:
        """True for readable tokens.  With a page list: selected closed pages plus the
        current partial page; everything else is hard-masked (Sec. 3.5)."""
        T = st.ctx
        if page_idx is None:
            return np.ones(T, dtype=bool)
        page = self.cfg.page_tokens
        mask = np.zeros(T, dtype=bool)
        for p in page_idx:
            mask[int(p) * page:(int(p) + 1) * page] = True
        # boxes exist only for closed blocks, so everything after the last closed block (the
        # partial block being filled) plays the role of the always-readable current page
        mask[st.n_closed * P:] = True
        return mask

    def decode_attn(self, layer: int, q, page_idx=None, return_weights=False):
        """q fp32 [B][Hq][dk] (bf16 values); page_idx None or int [B][Hkv][n_sel] ascending.
        Returns out float64 [B][Hq][dv] and lse float64 [B][Hq] (natural log)."""
        cfg = self.cfg
        g = cfg.n_q_heads // cfg.n_kv_heads
        out = np.zeros((cfg.batch, cfg.n_q_heads, cfg.d_v), dtype=np.float64)
        lse = np.zeros((cfg.batch, cfg.n_q_heads), dtype=np.float64)
        weights = {}
        read_bits = 0
        for b in range(cfg.batch):
            for h in range(cfg.n_kv_heads):
                st = self.streams[(layer, b, h)]
                K, V = self.reconstruct(st)
                sel = None if page_idx is None else page_idx[b][h]
                mask = self.token_mask(st, sel)
                read_bits += self._read_bits(st, sel)
                for j in range(g):
                    hq = h * g + j
                    logits = (K @ np.asarray(q[b, hq], dtype=np.float64)) * self.scale
                    logits = np.where(mask, logits, -np.inf)
                    m = logits.max()
                    e = np.exp(logits - m)
                    s = e.sum()
                    w = e / s
                    out[b, hq] = w @ V
                    lse[b, hq] = m + math.log(s)
                    if return_weights:
                        weights[(b, hq)] = w
        self.last_read_bits[layer] = read_bits
        # Sec. 3.5: the read cost of a scored query is "all summaries + selected pages".  The boxes
        # count for the page-list read that follows a quest_select; a later read with a list that
        # was not scored (or a full read) did not look at them.
        self.last_read_box_bits[layer] = self.last_box_bits.pop(layer, 0) if page_idx is not None else 0
        self.last_box_bits.pop(layer, None)
        if return_weights:
            return out, lse, weights
        return out, lse

    def decode_attn_observe(self, layer: int, q):
        """decode_attn over the full context that also observes block attention mass (Sec. 3.1).

        For every stream: a_b = (1/g) sum over the KV head's g query heads of sum_{j in b} w_{h,j}
        (Eq. 2 with the current query as the observed one; the heads that share the KV head are
        aggregated, Sec. 3.1 last paragraph), b = 0 .. n_closed with the last entry the partial
        block (absent when it is empty).  Tokens served from the exact residual count for the
        block they sit in.  Then the running mass: m_b <- 0.9 m_b + 0.1 a_b (a block seen for the
        first time starts from 0).  Returns out, lse, {(b, kv head): a}."""
        cfg = self.cfg
        g = cfg.n_q_heads // cfg.n_kv_heads
        out, lse, weights = self.decode_attn(layer, q, None, return_weights=True)
        observed = {}
        for b in range(cfg.batch):
            for h in range(cfg.n_kv_heads):
                st = self.streams[(layer, b, h)]
                nb = st.n_closed + (1 if st.n_tail else 0)
                a = np.zeros(nb, dtype=np.float64)
                for j in range(g):
                    w = weights[(b, h * g + j)]
                    for blk in range(nb):
                        a[blk] += w[blk * P:(blk + 1) * P].sum()
                a /= g
                old = np.zeros(nb, dtype=np.float64)
                old[:min(nb, len(st.ema_mass))] = st.ema_mass[:nb]
                st.ema_mass = 0.9 * old + 0.1 * a
                observed[(b, h)] = a
        return out, lse, observed

    def certificate(self, layer: int, q):
        """Attention error certificate of a full-context decode query, per query head (Sec. 3.6,
        Eq. 9): sum_b a^_b delta_b^v + min(2, M+/M- - M-/M+) max_j |v_j| with
        M+- = sum_b a^_b exp(+-eps_b).  a^_b is the compressed-cache attention weight of block b's
        tokens; eps_b = scale |q| kappa_b bounds the logit error of the block's tokens
        (Cauchy-Schwarz); tokens that are exact (exact blocks, the partial block, residual rows)
        enter with eps = delta = 0; max_j |v_j| is taken over the original value rows.
        Returns float64 [B][Hq]."""
        cfg = self.cfg
        g = cfg.n_q_heads // cfg.n_kv_heads
        _, _, weights = self.decode_attn(layer, q, None, return_weights=True)
        cert = np.zeros((cfg.batch, cfg.n_q_heads), dtype=np.float64)
        for b in range(cfg.batch):
            for h in range(cfg.n_kv_heads):
                st = self.streams[(layer, b, h)]
                n = st.n_closed
                exact_tok = np.zeros(st.ctx, dtype=bool)
                exact_tok[n * P:] = True
                if len(st.res_idx):
                    exact_tok[st.res_idx] = True
                vmax = max([blk.vnorm for blk in st.blocks] + ([_max_row_norm(st.tail_v)] if st.n_tail else [0.0]))
                for j in range(g):
                    hq = h * g + j
                    w = weights[(b, hq)]
                    qn = float(np.sqrt((np.asarray(q[b, hq], dtype=np.float64) ** 2).sum()))
                    first = 0.0
                    m_plus = m_minus = float(w[exact_tok].sum())
                    for i, blk in enumerate(st.blocks):
                        sel = ~exact_tok[i * P:(i + 1) * P]
                        a = float(w[i * P:(i + 1) * P][sel].sum())
                        eps = self.scale * qn * blk.kappa
                        first += a * blk.delta
                        m_plus += a * math.exp(eps)
                        m_minus += a * math.exp(-eps)
                    cert[b, hq] = first + min(2.0, m_plus / m_minus - m_minus / m_plus) * vmax
        return cert

    # -- page scorer -------------------------------------------------------------------
    def quest_scores(self, layer: int, q):
        """N6 per (b, kv head): fp32 score per closed page."""
        cfg = self.cfg
        g = cfg.n_q_heads // cfg.n_kv_heads
        res = {}
        for b in range(cfg.batch):
            for h in range(cfg.n_kv_heads):
                st = self.streams[(layer, b, h)]
                n_pages = st.n_closed * (P // cfg.page_tokens)      # pages of closed blocks
                lo = np.stack(st.box_lo[:n_pages]).astype(np.float32) if n_pages else np.zeros((0, cfg.d_k), np.float32)
                hi = np.stack(st.box_hi[:n_pages]).astype(np.float32) if n_pages else np.zeros((0, cfg.d_k), np.float32)
                per_head = []
                for j in range(g):
                    qh = np.asarray(q[b, h * g + j], dtype=np.float32)
                    acc = np.zeros(n_pages, dtype=np.float32)
                    for d in range(cfg.d_k):
                        pick = hi[:, d] if qh[d] >= 0 else lo[:, d]
                        acc = (acc + qh[d] * pick).astype(np.float32)       # product exact, one rounding
                    per_head.append(acc)
                if cfg.quest_reduce == REDUCE_MAX:
                    score = per_head[0]
                    for a in per_head[1:]:
                        score = np.maximum(score, a)
                else:
                    score = per_head[0]
                    for a in per_head[1:]:
                        score = (score + a).astype(np.float32)
                res[(b, h)] = score
        return res

    def quest_select(self, layer: int, q, budget_tokens: int):
        """Top-k closed pages per (b, kv head), k = min(budget/page, closed pages); ascending."""
        cfg = self.cfg
        scores = self.quest_scores(layer, q)
        k_nom = budget_tokens // cfg.page_tokens
        sel = [[None] * cfg.n_kv_heads for _ in range(cfg.batch)]
        box_bits = 0
        for (b, h), sc in scores.items():
            sel[b][h] = topk_ascending(sc, min(k_nom, len(sc)))
            box_bits += len(sc) * 2 * cfg.d_k * 16
        self.last_box_bits[layer] = box_bits
        return sel

    # -- accounting (Sec. 3.5 Eq. 7-8, Sec. 4.4) -----------------------------------------
    def _read_bits(self, st: Stream, page_idx) -> int:
        """Bits of graded K/V a query touches: whole blocks for a full read; for a page list,
        per selected page its share of codes, its V params, and each touched 32-token K group's
        params once.  Centroid and exact blocks: centroid rows once / exact rows per token.
        Residual rows: all of them in a full read, those of listed pages with a page list."""
        alias = self.alias
        dk, dv = st.d_k, st.d_v
        nval_tok = dk if alias else dk + dv
        bits = 0
        if page_idx is None:
            for blk in st.blocks:
                bits += block_bits(blk.level, dk, dv, alias)
            bits += st.n_tail * 16 * nval_tok
            bits += len(st.res_idx) * 16 * nval_tok
            return bits
        page = self.cfg.page_tokens
        touched_groups = set()
        touched_cent = set()
        for p in page_idx:
            p = int(p)
            blk_i = (p * page) // P
            blk = st.blocks[blk_i]
            if blk.level == 16:
                bits += page * 16 * nval_tok
            elif blk.level == 1:
                touched_cent.add(blk_i)
            else:
                bits += page * nval_tok * blk.level                        # codes
                if not alias:
                    bits += page * (dv // G) * 32                          # V params of its tokens
                for t0 in range(p * page, (p + 1) * page, G):
                    touched_groups.add(t0 // G)
        bits += len(touched_groups) * dk * 32                              # K params per touched group
        bits += len(touched_cent) * 16 * nval_tok
        # exact residual rows of listed pages are read too (those of other pages are masked, Sec. 3.5)
        listed = set(int(p) for p in page_idx)
        bits += sum(1 for t in st.res_idx if int(t) // page in listed) * 16 * nval_tok
        # the current partial block is always read, exact
        bits += st.n_tail * 16 * nval_tok
        return bits

    def bits_report(self, layer: int) -> dict:
        """Exact integer resident bits by category for one layer (all its streams)."""
        cfg = self.cfg
        alias = self.alias
        rep = dict(values=0, code_bits=0, param_bits=0, exact_bits=0, centroid_bits=0, tail_bits=0,
                   residual_bits=0, residual_index_bits=0, box_bits=0,
                   blocks_by_level={16: 0, 8: 0, 4: 0, 2: 0, 1: 0})
        for b in range(cfg.batch):
            for h in range(cfg.n_kv_heads):
                st = self.streams[(layer, b, h)]
                nval_tok = st.d_k if alias else st.d_k + st.d_v
                rep["values"] += st.ctx * nval_tok
                for blk in st.blocks:
                    rep["blocks_by_level"][blk.level] += 1
                    if blk.level == 16:
                        rep["exact_bits"] += 16 * P * nval_tok
                    elif blk.level == 1:
                        rep["centroid_bits"] += 16 * nval_tok
                    else:
                        rep["code_bits"] += blk.level * P * nval_tok
                        rep["param_bits"] += (P * nval_tok // G) * 32
                rep["tail_bits"] += st.n_tail * 16 * nval_tok
                rep["residual_bits"] += len(st.res_idx) * 16 * nval_tok
                rep["residual_index_bits"] += len(st.res_idx) * 32
                if cfg.page_tokens > 0:
                    rep["box_bits"] += len(st.box_lo) * 2 * st.d_k * 16
        rep["resident_bits"] = (rep["code_bits"] + rep["param_bits"] + rep["exact_bits"] + rep["centroid_bits"]
                                + rep["tail_bits"] + rep["residual_bits"] + rep["residual_index_bits"]
                                + rep["box_bits"])
        rep["bpv_resident"] = rep["resident_bits"] / max(1, rep["values"])
        rep["bpv_paper"] = (rep["resident_bits"] - rep["residual_index_bits"]) / max(1, rep["values"])
        rep["last_read_bits"] = self.last_read_bits.get(layer, 0) + self.last_read_box_bits.get(layer, 0)
        rep["bpv_read"] = rep["last_read_bits"] / max(1, rep["values"])
        return rep

    # -- parity helpers ----------------------------------------------------------------
    def levels(self, layer: int, b: int, h: int) -> np.ndarray:
        return np.array([blk.level for blk in self.streams[(layer, b, h)].blocks], dtype=np.int32)


# --------------------------------------------------------------------------------------
# Attention error certificate (Sec. 3.6, Eq. 9) - diagnostic used by the pins
# --------------------------------------------------------------------------------------
def certificate_bound(a_hat_blocks, eps_blocks, delta_v_blocks, vmax: float) -> float:
    """sum_b a^_b delta_b^v + min(2, M+/M- - M-/M+) max|v_j| with M+- = sum_b a^_b e^{+-eps_b}."""
    a = np.asarray(a_hat_blocks, dtype=np.float64)
    eps = np.asarray(eps_blocks, dtype=np.float64)
    dv = np.asarray(delta_v_blocks, dtype=np.float64)
    m_plus = float(np.sum(a * np.exp(eps)))
    m_minus = float(np.sum(a * np.exp(-eps)))
    second = min(2.0, m_plus / m_minus - m_minus / m_plus)
    return float(np.sum(a * dv)) + second * vmax
