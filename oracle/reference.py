"""CPU oracle for composed-cache query prefill - Python front end.

TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and the benchmark's CPU-baseline
leg.  It shares no code with the CUDA path and never imports it.

What it computes, in the paper's order (Section 3.1, Eq. 2; Section 2.1, Eq. 1; Section 3.2 step 4):

1. ``compose``     - lay the request's packets end to end, each as  header | document | trailer
                     (Eq. 2 order), positions dense from 0; for every composed position record
                     where the token was cached and the offset Delta = new - old position.
2. ``composed_kv`` - gather those rows and re-align every key by Eq. 1 (values untouched).
3. ``query_prefill`` - append the query chunk's own K/V and let query token i attend to all
                     prefix tokens and to query tokens <= i (softmax attention, GQA).

All arithmetic is fp64 on the exactly-widened stored bytes; the rotation and the attention
loops are in ``kvp_oracle.c``.  A second, differently written routine lives in ``bruteforce.py``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libkvp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``kvp_oracle.c`` with gcc (OpenMP) next to this file."""
    src = os.path.join(_HERE, "kvp_oracle.c")
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(src):
        tmp = _LIB_PATH + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, src, "-lm"])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB_PATH)
        dp = ctypes.POINTER(ctypes.c_double)
        lib.kvp_oracle_threads.restype = ctypes.c_int
        lib.kvp_oracle_rope_rows.argtypes = [dp, dp, ctypes.c_longlong, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                             dp, ctypes.POINTER(ctypes.c_longlong)]
        lib.kvp_oracle_rope_rows.restype = None
        ip = ctypes.POINTER(ctypes.c_int)
        lib.kvp_oracle_attention_rows.argtypes = [dp, dp, dp, ctypes.c_longlong, ctypes.c_int, ctypes.c_int,
                                                  ctypes.c_int, ctypes.c_int, ctypes.c_double, ip, ip,
                                                  ctypes.c_longlong, dp, dp, dp]
        lib.kvp_oracle_attention_rows.restype = None
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().kvp_oracle_threads())


def _dptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def widen(x: np.ndarray, dtype: str) -> np.ndarray:
    """Stored bytes -> float64, exactly.  bf16 arrives as uint16 bit patterns."""
    if dtype == "bf16":
        u = np.ascontiguousarray(x, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
        return u.view(np.float32).astype(np.float64)
    if dtype == "f32":
        return np.asarray(x, dtype=np.float32).astype(np.float64)
    if dtype == "f64":
        return np.asarray(x, dtype=np.float64)
    raise ValueError(dtype)


def inv_freq(theta: float, head_dim: int) -> np.ndarray:
    """theta_i = theta^(-2i/d), i = 0 .. d/2-1 (no frequency scaling)."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    return np.float64(theta) ** (-(2.0 * i) / np.float64(head_dim))


def rope(x: np.ndarray, delta, inv_f: np.ndarray, pairing: int = 0) -> np.ndarray:
    """Eq. 1 on rows: x [n_rows][n_heads][d] fp64, delta int per row (scalar broadcasts)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    assert x.ndim == 3
    n, h, d = x.shape
    dl = np.ascontiguousarray(np.broadcast_to(np.asarray(delta, dtype=np.int64), (n,)), dtype=np.int64)
    y = np.empty_like(x)
    inv_f = np.ascontiguousarray(inv_f, dtype=np.float64)
    assert inv_f.shape == (d // 2,)
    _load().kvp_oracle_rope_rows(_dptr(x), _dptr(y), n, h, d, int(pairing), _dptr(inv_f),
                                 dl.ctypes.data_as(ctypes.POINTER(ctypes.c_longlong)))
    return y


# --------------------------------------------------------------------------------------
# the store: what was cached offline, in registration order
# --------------------------------------------------------------------------------------

@dataclass
class _Segment:
    row0: int          # first row in the store (rows are dense in registration order)
    n: int
    pos0: int          # position the first token had when it was cached


class Store:
    """Registered packets and adapters.  Store rows are assigned densely in registration order;
    an adapter takes its header rows first, then its trailer rows.  ``loader(layer)`` returns the
    stored-dtype arrays ``[n_tokens][n_kv_heads][head_dim]`` for that layer."""

    def __init__(self, dtype: str):
        self.dtype = dtype
        self.rows = 0
        self.packets: List[Tuple[_Segment, Callable]] = []
        self.adapters: List[Tuple[_Segment, _Segment, Callable]] = []
        self.kept: dict = {}       # packet id -> kept[layer][kv_head] token indices (compressed packets only)

    def register_packet(self, n_tokens: int, cache_pos0: int, loader: Callable, kept=None) -> int:
        """``kept`` marks a compressed packet (Section 4.3): after unstructured pruning, layer l / kv head h
        of its cache holds only the tokens ``kept[l][h]``; the loader still returns the full document and
        the packet still spans n_tokens positions (pruned tokens leave their positions unoccupied)."""
        seg = _Segment(self.rows, int(n_tokens), int(cache_pos0))
        self.rows += int(n_tokens)
        self.packets.append((seg, loader))
        if kept is not None:
            self.kept[len(self.packets) - 1] = kept
        return len(self.packets) - 1

    def register_adapter(self, n_header: int, header_pos0: int, n_trailer: int, trailer_pos0: int,
                         loader: Callable) -> int:
        hs = _Segment(self.rows, int(n_header), int(header_pos0))
        self.rows += int(n_header)
        ts = _Segment(self.rows, int(n_trailer), int(trailer_pos0))
        self.rows += int(n_trailer)
        self.adapters.append((hs, ts, loader))
        return len(self.adapters) - 1


@dataclass
class Plan:
    """The composed sequence of one request, token by token."""
    src_row: np.ndarray      # int32 [P]  store row each composed position is read from
    cache_pos: np.ndarray    # int32 [P]  position that token had when cached
    delta: np.ndarray        # int32 [P]  rotation offset applied to its key (0 when rebase is off)
    segments: np.ndarray     # int32 [n_seg][4]: src_row0, length, dst_pos0, delta (zero-length segments omitted)
    refs: list               # per segment: ("packet"|"header"|"trailer", id)

    @property
    def prefix_len(self) -> int:
        return int(self.src_row.shape[0])


def compose(store: Store, slots: Sequence[Tuple[int, int]], rebase: bool = True) -> Plan:
    """Section 3.1: header | document | trailer for each slot in order; positions dense from 0
    (Section 3.2 step 4: the caches are re-aligned by Eq. 1 and concatenated).  ``adapter_id`` -1
    means the slot has no adapter tokens (the paper's "No Recompute" layout)."""
    src, cpos, dl, segs, refs = [], [], [], [], []
    t = 0
    for pid, aid in slots:
        parts = []
        if aid >= 0:
            parts.append(("header", aid, store.adapters[aid][0]))
        parts.append(("packet", pid, store.packets[pid][0]))
        if aid >= 0:
            parts.append(("trailer", aid, store.adapters[aid][1]))
        for kind, ident, seg in parts:
            if seg.n == 0:
                continue
            d = (t - seg.pos0) if rebase else 0
            segs.append((seg.row0, seg.n, t, d))
            refs.append((kind, ident))
            for o in range(seg.n):
                src.append(seg.row0 + o)
                cpos.append(seg.pos0 + o)
                dl.append((t + o - (seg.pos0 + o)) if rebase else 0)
            t += seg.n
    return Plan(np.asarray(src, dtype=np.int32).reshape(-1), np.asarray(cpos, dtype=np.int32).reshape(-1),
                np.asarray(dl, dtype=np.int32).reshape(-1),
                np.asarray(segs, dtype=np.int32).reshape(-1, 4), refs)


def composed_kv(store: Store, plan: Plan, layer: int, inv_f: np.ndarray, pairing: int = 0):
    """Gather the plan's rows for one layer and re-align the keys (Eq. 1).  Returns fp64
    ``K' [P][Hkv][d]``, ``V' [P][Hkv][d]`` and the un-rotated gathered keys (for byte checks)."""
    ks, vs = [], []
    for (kind, ident), (row0, n, dst, d) in zip(plan.refs, plan.segments):
        if kind == "packet":
            k, v = store.packets[ident][1](layer)
        else:
            hk, hv, tk, tv = store.adapters[ident][2](layer)
            k, v = (hk, hv) if kind == "header" else (tk, tv)
        assert k.shape[0] == n and v.shape[0] == n
        ks.append(widen(k, store.dtype))
        vs.append(widen(v, store.dtype))
    if not ks:
        # a request without packets: the concatenation of Eq. 2 over zero slots is the empty sequence
        like = store.packets[0][1](layer)[0] if store.packets else store.adapters[0][2](layer)[0]
        empty = np.zeros((0,) + tuple(like.shape[1:]), dtype=np.float64)
        return empty, empty.copy(), empty.copy()
    k_raw = np.concatenate(ks, axis=0)
    v_cat = np.concatenate(vs, axis=0)
    k_reb = rope(k_raw, plan.delta.astype(np.int64), inv_f, pairing)
    return k_reb, v_cat, k_raw


def attention_rows(K: np.ndarray, V: np.ndarray, Q: np.ndarray, prefix_len: int, scale: float,
                   rows: Optional[Sequence[Tuple[int, int]]] = None, want_prob_sum: bool = False):
    """K, V: fp64 [prefix_len + q_len][Hkv][d] (query K/V already appended); Q: fp64 [q_len][Hq][d].
    rows: list of (head, query token); default every row in (token, head) order.
    Returns out [n_rows][d], lse [n_rows] (and the per-row probability sum if asked)."""
    K = np.ascontiguousarray(K, dtype=np.float64)
    V = np.ascontiguousarray(V, dtype=np.float64)
    Q = np.ascontiguousarray(Q, dtype=np.float64)
    q_len, Hq, d = Q.shape
    n_tot, Hkv, d2 = K.shape
    assert d2 == d and V.shape == K.shape and n_tot == prefix_len + q_len and Hq % Hkv == 0
    if rows is None:
        rows = [(h, i) for i in range(q_len) for h in range(Hq)]
    rh = np.ascontiguousarray([r[0] for r in rows], dtype=np.int32)
    ri = np.ascontiguousarray([r[1] for r in rows], dtype=np.int32)
    assert rh.size == 0 or (rh.min() >= 0 and rh.max() < Hq and ri.min() >= 0 and ri.max() < q_len)
    n = len(rows)
    out = np.empty((n, d), dtype=np.float64)
    lse = np.empty((n,), dtype=np.float64)
    ps = np.empty((n,), dtype=np.float64)
    ip = ctypes.POINTER(ctypes.c_int)
    _load().kvp_oracle_attention_rows(_dptr(K), _dptr(V), _dptr(Q), int(prefix_len), int(q_len), int(Hq), int(Hkv),
                                      int(d), float(scale), rh.ctypes.data_as(ip), ri.ctypes.data_as(ip), n,
                                      _dptr(out), _dptr(lse), _dptr(ps))
    if want_prob_sum:
        return out, lse, ps
    return out, lse


def query_prefill(store: Store, plan: Plan, layer: int, q, k_new, v_new, inv_f: np.ndarray,
                  pairing: int = 0, scale: Optional[float] = None, rope_query: bool = False,
                  rows: Optional[Sequence[Tuple[int, int]]] = None, want_prob_sum: bool = False):
    """One request, one layer.  q [q_len][Hq][d], k_new/v_new [q_len][Hkv][d] in the stored dtype.
    By default q and k_new are already rotated for positions prefix_len + i; with ``rope_query``
    they are raw and rotated here at those positions (Eq. 1 with Delta = absolute position).
    Returns (out [n_rows][d], lse [n_rows], K_full, V_full) with the appended cache."""
    Kp, Vp, _ = composed_kv(store, plan, layer, inv_f, pairing)
    P = plan.prefix_len
    Q = widen(q, store.dtype)
    Kn = widen(k_new, store.dtype)
    Vn = widen(v_new, store.dtype)
    q_len, Hq, d = Q.shape
    if rope_query:
        pos = np.arange(P, P + q_len, dtype=np.int64)
        Q = rope(Q, pos, inv_f, pairing)
        Kn = rope(Kn, pos, inv_f, pairing)
    K = np.concatenate([Kp, Kn], axis=0)
    V = np.concatenate([Vp, Vn], axis=0)
    if scale is None:
        scale = 1.0 / np.sqrt(np.float64(d))
    present = kept_mask(store, plan, layer, Kp.shape[1])
    if present is None:
        res = attention_rows(K, V, Q, P, float(scale), rows, want_prob_sum)
        return res + (K, V)
    # Compressed packets: kv head h simply does not have the pruned keys, so its q heads attend over the
    # surviving prefix keys (in order) followed by the query block - one plain attention per kv head.
    Hkv = Kp.shape[1]
    g = Hq // Hkv
    if rows is None:
        rows = [(h, i) for i in range(q_len) for h in range(Hq)]
    out = np.empty((len(rows), d), dtype=np.float64)
    lse = np.empty((len(rows),), dtype=np.float64)
    ps = np.empty((len(rows),), dtype=np.float64)
    for hk in range(Hkv):
        sel = [n for n, (h, i) in enumerate(rows) if h // g == hk]
        if not sel:
            continue
        idx = np.nonzero(present[:, hk])[0]
        Kh = np.concatenate([Kp[idx, hk:hk + 1], Kn[:, hk:hk + 1]], axis=0)
        Vh = np.concatenate([Vp[idx, hk:hk + 1], Vn[:, hk:hk + 1]], axis=0)
        sub = [(rows[n][0] - hk * g, rows[n][1]) for n in sel]
        o, l, s_ = attention_rows(Kh, Vh, Q[:, hk * g:(hk + 1) * g], len(idx), float(scale), sub, True)
        out[sel], lse[sel], ps[sel] = o, l, s_
    if want_prob_sum:
        return out, lse, ps, K, V
    return out, lse, K, V


def segment_mass(store: Store, plan: Plan, layer: int, q, k_new, inv_f: np.ndarray, pairing: int = 0,
                 scale: Optional[float] = None, rope_query: bool = False,
                 rows: Optional[Sequence[Tuple[int, int]]] = None) -> np.ndarray:
    """Attention mass per segment (Section 4.4, Fig. 5: what the attention maps show).  For each row
    (head, query token i): softmax over the keys the token sees - the composed prefix (re-aligned by Eq. 1)
    and query tokens <= i - then the probabilities are added up per segment of ``plan.segments`` and,
    last column, over the query block.  Returns [n_rows][n_segments + 1]; every row sums to 1."""
    Kp, _, _ = composed_kv(store, plan, layer, inv_f, pairing)
    P = plan.prefix_len
    Q = widen(q, store.dtype)
    Kn = widen(k_new, store.dtype)
    q_len, Hq, d = Q.shape
    Hkv = Kp.shape[1]
    g = Hq // Hkv
    if rope_query:
        pos = np.arange(P, P + q_len, dtype=np.int64)
        Q = rope(Q, pos, inv_f, pairing)
        Kn = rope(Kn, pos, inv_f, pairing)
    if scale is None:
        scale = 1.0 / np.sqrt(np.float64(d))
    present = kept_mask(store, plan, layer, Hkv)
    if rows is None:
        rows = [(h, i) for i in range(q_len) for h in range(Hq)]
    n_seg = plan.segments.shape[0]
    out = np.zeros((len(rows), n_seg + 1), dtype=np.float64)
    for n, (h, i) in enumerate(rows):
        hk = h // g
        sc = np.concatenate([Kp[:, hk] @ Q[i, h], Kn[:i + 1, hk] @ Q[i, h]]) * scale
        if present is not None:
            sc[:P][~present[:, hk]] = -np.inf
        p = np.exp(sc - sc.max())
        p /= p.sum()
        for s_, (_, length, t0, _) in enumerate(plan.segments):
            out[n, s_] = p[t0:t0 + length].sum()
        out[n, n_seg] = p[P:].sum()
    return out


def kept_mask(store: Store, plan: Plan, layer: int, n_kv_heads: int):
    """present[t][h]: does kv head h of this layer still hold the key at composed position t?  None when
    the request has no compressed packet (everything is present)."""
    if not any(kind == "packet" and ident in store.kept for kind, ident in plan.refs):
        return None
    present = np.ones((plan.prefix_len, n_kv_heads), dtype=bool)
    for (row0, n, t0, _), (kind, ident) in zip(plan.segments, plan.refs):
        if kind == "packet" and ident in store.kept:
            present[t0:t0 + n] = False
            for h in range(n_kv_heads):
                present[t0 + np.asarray(store.kept[ident][layer][h], dtype=np.int64), h] = True
    return present
