"""Seeded synthetic inputs for composed-cache query prefill.

This module only *draws numbers and arranges them in arrays*.  It holds none of the
method's arithmetic (no rotation, no softmax, no composition): both the CUDA path
and the CPU oracle are fed from here and share nothing else.

A workload imitates the *shape* of the paper's RAG requests (Section 4.1: N retrieved
documents, each wrapped in N_h header and N_t trailer soft tokens, then a query):

* ``packets[p]``  - per-layer K/V of one document, ``[n_layers][n_tokens][n_kv_heads][head_dim]``
* ``adapters[a]`` - per-layer K/V of header and trailer soft tokens (same layout)
* ``items[b]``    - the request: an ordered list of ``(packet_id, adapter_id)`` slots
* ``q, k_new, v_new`` - the query chunk's projections for every layer

Stored dtype is either float32 or bfloat16.  bfloat16 arrays are carried as
``numpy.uint16`` bit patterns (numpy has no bf16); ``to_stored`` does the
round-to-nearest-even narrowing that "N(0,1) rounded to bf16" asks for.

Small workloads are drawn with ``numpy.random.default_rng(seed)`` in the fixed order
documented in ``make_workload`` so that any machine reproduces the bytes.  Large
ones (gigabytes) are drawn on the GPU by ``DeviceWorkload`` with one
``torch.Generator`` seed per tensor and can re-draw any tensor on demand.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------------------
# dtype plumbing (no method arithmetic)
# --------------------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float32 exactly."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_stored(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "bf16":
        return f32_to_bf16_bits(x)
    raise ValueError(dtype)


def stored_to_f64(x: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of the stored bytes to float64 (what the oracle computes on)."""
    if dtype == "f32":
        return np.asarray(x, dtype=np.float32).astype(np.float64)
    return bf16_bits_to_f32(x).astype(np.float64)


# --------------------------------------------------------------------------------------
# containers
# --------------------------------------------------------------------------------------

@dataclass
class ModelShape:
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str = "bf16"            # "bf16" | "f32"
    rope_theta: float = 10000.0
    rope_pairing: int = 0          # 0: pairs (i, i+d/2); 1: pairs (2i, 2i+1)

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


@dataclass
class Packet:
    k: np.ndarray                  # [n_layers][n_tokens][n_kv_heads][head_dim], stored dtype
    v: np.ndarray
    cache_pos0: int = 0
    kept: Optional[list] = None    # compressed packet: kept[layer][kv_head] = sorted token indices that survive pruning

    @property
    def n_tokens(self) -> int:
        return int(self.k.shape[1])


@dataclass
class Adapter:
    hk: np.ndarray                 # [n_layers][n_header][n_kv_heads][head_dim]
    hv: np.ndarray
    tk: np.ndarray                 # [n_layers][n_trailer][n_kv_heads][head_dim]
    tv: np.ndarray
    header_pos0: int = 0
    trailer_pos0: int = 0

    @property
    def n_header(self) -> int:
        return int(self.hk.shape[1])

    @property
    def n_trailer(self) -> int:
        return int(self.tk.shape[1])


@dataclass
class Workload:
    """A fully host-resident workload (small enough for numpy)."""
    shape: ModelShape
    packets: List[Packet]
    adapters: List[Adapter]
    items: List[List[Tuple[int, int]]]      # per batch item: [(packet_id, adapter_id or -1), ...]
    q: np.ndarray                           # [n_layers][batch][q_len][n_q_heads][head_dim]
    k_new: np.ndarray                       # [n_layers][batch][q_len][n_kv_heads][head_dim]
    v_new: np.ndarray
    rebase: bool = True
    name: str = ""
    seed: int = 0
    notes: dict = field(default_factory=dict)

    @property
    def batch(self) -> int:
        return len(self.items)

    @property
    def q_len(self) -> int:
        return int(self.q.shape[2])

    def prefix_len(self, b: int) -> int:
        n = 0
        for pid, aid in self.items[b]:
            n += self.packets[pid].n_tokens
            if aid >= 0:
                n += self.adapters[aid].n_header + self.adapters[aid].n_trailer
        return n

    # uniform accessors shared with DeviceWorkload
    def packet_layer(self, pid: int, layer: int):
        p = self.packets[pid]
        return p.k[layer], p.v[layer]

    def query_layer(self, layer: int):
        return self.q[layer], self.k_new[layer], self.v_new[layer]


def draw_kept(packets, keep_rate, seed: int, n_layers: int, n_kv_heads: int, per_head: bool = True) -> None:
    """Stand-in for an unstructured KV compressor (Section 4.3): packet i keeps about keep_rate[i] of its tokens
    (None: not pruned), a different seeded random subset per layer and - with per_head - per kv head."""
    krng = np.random.default_rng(seed + 104729)
    for i, rate in enumerate(keep_rate):
        if rate is None:
            continue
        n = packets[i].n_tokens
        kept = []
        for l in range(n_layers):
            n_layer = max(1, min(n, int(round(n * rate * krng.uniform(0.7, 1.3)))))
            row = []
            for h in range(n_kv_heads):
                n_h = max(1, min(n, int(round(n_layer * krng.uniform(0.6, 1.0))))) if per_head else n_layer
                row.append(np.sort(krng.choice(n, size=n_h, replace=False)).astype(np.int64))
            kept.append(row)
        packets[i].kept = kept


def wrap_workload(wl: Workload, keep_rate=None, seed: int = 0) -> Workload:
    """The same requests with every slot's cache stored as ONE wrapped unit  header | document | trailer  (Eq. 2:
    the form in which the paper computes a packet offline), registered as a packet of its own with no separate
    adapter.  The fillers must have been cached where the wrapped layout puts them (header right before the
    document, trailer right behind).  With keep_rate (one rate per slot, in slot order) the wrapped units are
    pruned as a whole, fillers included - Section 4.3's "KVPacket Normal" setting."""
    packets, items = [], []
    for it in wl.items:
        part = []
        for pid, aid in it:
            p = wl.packets[pid]
            if aid < 0:
                packets.append(Packet(p.k, p.v, p.cache_pos0))
            else:
                a = wl.adapters[aid]
                assert a.header_pos0 + a.n_header == p.cache_pos0 and a.trailer_pos0 == p.cache_pos0 + p.n_tokens, \
                    "fillers not cached at the wrapped layout's positions"
                packets.append(Packet(np.concatenate([a.hk, p.k, a.tk], axis=1), np.concatenate([a.hv, p.v, a.tv], axis=1),
                                      a.header_pos0))
            part.append((len(packets) - 1, -1))
        items.append(part)
    out = Workload(wl.shape, packets, [], items, wl.q, wl.k_new, wl.v_new, wl.rebase, wl.name + "_wrapped", wl.seed, dict(wl.notes))
    if keep_rate is not None:
        draw_kept(packets, keep_rate, seed, wl.shape.n_layers, wl.shape.n_kv_heads, True)
    return out


def shard_workload(wl: Workload, rank: int, world: int):
    """Rank ``rank``'s part of a workload whose requests are sharded by prefix over ``world`` ranks: every
    request's slot list is cut into ``world`` contiguous parts (slot counts as equal as possible, some possibly
    empty); the rank keeps only the packets its parts name (local ids in order of first use), all adapters and
    the whole query.  Returns (sub-workload, pos_base) with pos_base[b] = composed position at which the rank's
    part of request b starts (the lengths of the slots before it, adapters included)."""
    local = {}
    items, pos_base = [], []
    for it in wl.items:
        n = len(it)
        lo, hi = (n * rank) // world, (n * (rank + 1)) // world
        pos = 0
        for pid, aid in it[:lo]:
            pos += wl.packets[pid].n_tokens + (wl.adapters[aid].n_header + wl.adapters[aid].n_trailer if aid >= 0 else 0)
        pos_base.append(pos)
        part = []
        for pid, aid in it[lo:hi]:
            if pid not in local:
                local[pid] = len(local)
            part.append((local[pid], aid))
        items.append(part)
    packets = [wl.packets[pid] for pid, _ in sorted(local.items(), key=lambda kv: kv[1])]
    sub = Workload(wl.shape, packets, wl.adapters, items, wl.q, wl.k_new, wl.v_new, wl.rebase, f"{wl.name}_rank{rank}of{world}",
                   wl.seed, dict(wl.notes))
    return sub, pos_base


def digest64(*arrays) -> str:
    """64-bit BLAKE2b digest (hex) of the raw bytes of the given arrays, in order: what a report carries so that two
    runs (or the two sides of one run) can tell whether they worked on the same input bytes."""
    import hashlib
    h = hashlib.blake2b(digest_size=8)
    for a in arrays:
        h.update(np.ascontiguousarray(a).view(np.uint8).reshape(-1).data)
    return h.hexdigest()


def shard_heads(wl: Workload, rank: int, world: int) -> Workload:
    """Rank ``rank``'s part of a workload sharded by kv head over ``world`` ranks: kv heads
    [rank * Hkv / world, (rank + 1) * Hkv / world) of every packet, adapter and query tensor, with the query heads
    that read them.  Plain slicing: attention is independent per kv head, so the ranks' outputs put side by side
    along the head axis are the whole workload's output."""
    s = wl.shape
    assert s.n_kv_heads % world == 0, "kv heads do not divide over the ranks"
    n_kv = s.n_kv_heads // world
    h0, h1 = rank * n_kv, (rank + 1) * n_kv
    g = s.group
    shape = ModelShape(s.n_layers, n_kv * g, n_kv, s.head_dim, s.dtype, s.rope_theta, s.rope_pairing)
    cut = lambda a: np.ascontiguousarray(a[..., h0:h1, :])
    packets = []
    for pk in wl.packets:
        kept = None if pk.kept is None else [list(layer[h0:h1]) for layer in pk.kept]
        packets.append(Packet(cut(pk.k), cut(pk.v), pk.cache_pos0, kept))
    adapters = [Adapter(cut(a.hk), cut(a.hv), cut(a.tk), cut(a.tv), a.header_pos0, a.trailer_pos0) for a in wl.adapters]
    q = np.ascontiguousarray(wl.q[..., h0 * g:h1 * g, :])
    return Workload(shape, packets, adapters, [list(it) for it in wl.items], q, cut(wl.k_new), cut(wl.v_new), wl.rebase,
                    f"{wl.name}_heads{rank}of{world}", wl.seed, dict(wl.notes))


# --------------------------------------------------------------------------------------
# small, numpy-drawn workloads
# --------------------------------------------------------------------------------------

def make_workload(shape: ModelShape,
                  packet_lens: Sequence[int],
                  items: Sequence[Sequence[Tuple[int, int]]],
                  q_len: int,
                  n_header: int = 16,
                  n_trailer: int = 16,
                  n_adapters: int = 1,
                  adapter_std: float = 1.0,
                  seed: int = 0,
                  rebase: bool = True,
                  packet_pos0: Optional[Sequence[int]] = None,
                  adapter_pos0: Optional[Sequence[Tuple[int, int]]] = None,
                  outlier_channels: int = 0,
                  outlier_scale: float = 8.0,
                  keep_rate: Optional[Sequence[Optional[float]]] = None,
                  keep_per_head: bool = True,
                  name: str = "") -> Workload:
    """Draw a workload with ``numpy.random.default_rng(seed)``.

    Draw order (fixed, so the bytes are reproducible): for each packet in id order K then V;
    for each adapter in id order header-K, header-V, trailer-K, trailer-V; then Q, K_new,
    V_new (all layers at once, layer-major).  Everything is N(0,1) in float32 scaled by the
    stated std, then narrowed to the stored dtype.  ``outlier_channels`` > 0 multiplies that
    many seeded channels per (layer, kv head) of every packet's K and V by ``outlier_scale``
    before narrowing (same channels for all packets).
    ``keep_rate[p]`` (None = not compressed) marks packet p as pruned: a stand-in for an unstructured
    KV compressor, every (layer, kv head) keeps a seeded random subset of the tokens, about that
    fraction of them - a different count per head with ``keep_per_head``, else one count per layer.
    These draws come from their own generator, after everything else.
    """
    rng = np.random.default_rng(seed)
    L, Hq, Hkv, d = shape.n_layers, shape.n_q_heads, shape.n_kv_heads, shape.head_dim

    chan_scale = None
    if outlier_channels > 0:
        crng = np.random.default_rng(seed + 7919)
        chan_scale = np.ones((L, 1, Hkv, d), dtype=np.float32)
        for l in range(L):
            for h in range(Hkv):
                idx = crng.choice(d, size=outlier_channels, replace=False)
                chan_scale[l, 0, h, idx] = outlier_scale

    def draw(n, heads, std=1.0, scale=None):
        x = rng.standard_normal((L, n, heads, d), dtype=np.float32) * np.float32(std)
        if scale is not None:
            x = x * scale
        return to_stored(x, shape.dtype)

    packets = []
    for i, n in enumerate(packet_lens):
        k = draw(n, Hkv, 1.0, chan_scale)
        v = draw(n, Hkv, 1.0, chan_scale)
        packets.append(Packet(k, v, int(packet_pos0[i]) if packet_pos0 is not None else 0))

    adapters = []
    for a in range(n_adapters):
        hk = draw(n_header, Hkv, adapter_std)
        hv = draw(n_header, Hkv, adapter_std)
        tk = draw(n_trailer, Hkv, adapter_std)
        tv = draw(n_trailer, Hkv, adapter_std)
        hp, tp = adapter_pos0[a] if adapter_pos0 is not None else (0, 0)
        adapters.append(Adapter(hk, hv, tk, tv, int(hp), int(tp)))

    B = len(items)
    q = to_stored(rng.standard_normal((L, B, q_len, Hq, d), dtype=np.float32), shape.dtype)
    k_new = to_stored(rng.standard_normal((L, B, q_len, Hkv, d), dtype=np.float32), shape.dtype)
    v_new = to_stored(rng.standard_normal((L, B, q_len, Hkv, d), dtype=np.float32), shape.dtype)
    wl = Workload(shape, packets, adapters, [list(map(tuple, it)) for it in items], q, k_new, v_new,
                  rebase=rebase, name=name, seed=seed)
    wl.notes["chan_scale"] = chan_scale        # [L][1][Hkv][d] multipliers applied to packet K/V, or None
    if keep_rate is not None:
        draw_kept(packets, keep_rate, seed, L, Hkv, keep_per_head)
    return wl


def config1(seed: int = 0) -> Workload:
    """Tiny correctness case: 1 layer, 4/2 heads, d 64, fp32, 3 x 128-token packets, 8+8 adapter
    tokens with std 0.02, 32 query tokens, theta 1e4, everything cached at position 0."""
    shape = ModelShape(1, 4, 2, 64, "f32", 10000.0, 0)
    return make_workload(shape, [128, 128, 128], [[(0, 0), (1, 0), (2, 0)]], q_len=32,
                         n_header=8, n_trailer=8, adapter_std=0.02, seed=seed, name="config1")


def config2(seed: int = 0) -> Workload:
    """Llama-3.1-8B attention shape, one layer: 32/8 heads, d 128, bf16, 5 x 512-token packets,
    one shared 16+16 adapter, 64 query tokens, theta 5e5."""
    shape = ModelShape(1, 32, 8, 128, "bf16", 500000.0, 0)
    return make_workload(shape, [512] * 5, [[(p, 0) for p in range(5)]], q_len=64,
                         n_header=16, n_trailer=16, seed=seed, name="config2")


# --------------------------------------------------------------------------------------
# large, GPU-drawn workloads (configs 3-5 and their scaled-down test versions)
# --------------------------------------------------------------------------------------

@dataclass
class LargeSpec:
    name: str
    shape: ModelShape
    packet_lens: List[int]                  # pool of packets
    items: List[List[Tuple[int, int]]]
    q_len: int
    n_header: int = 16
    n_trailer: int = 16
    seed: int = 0
    outlier_channels: int = 0
    outlier_scale: float = 8.0
    rebase: bool = True
    packet_seed_offset: int = 0             # packet p is drawn with the seeds of packet p + offset (a rank's part of a sharded spec)

    @property
    def batch(self) -> int:
        return len(self.items)

    def prefix_len(self, b: int) -> int:
        n = 0
        for pid, aid in self.items[b]:
            n += self.packet_lens[pid] + (self.n_header + self.n_trailer if aid >= 0 else 0)
        return n


def spec_config3(seed: int = 0, n_layers: int = 32, batch: int = 4, pool: int = 64,
                 per_item: int = 10, doc_len: int = 1024, q_len: int = 128) -> LargeSpec:
    """Llama-3.1-8B full attention stack: every item draws ``per_item`` distinct packets from a
    ``pool``-packet pool (order as drawn); one shared 16+16 adapter."""
    rng = np.random.default_rng(seed + 3000)
    items = [[(int(p), 0) for p in rng.choice(pool, size=per_item, replace=False)] for _ in range(batch)]
    shape = ModelShape(n_layers, 32, 8, 128, "bf16", 500000.0, 0)
    return LargeSpec("config3", shape, [doc_len] * pool, items, q_len, seed=seed)


def spec_config4(seed: int = 0, n_layers: int = 28, batch: int = 8, per_item: int = 20,
                 lo: int = 256, hi: int = 1024, q_len: int = 256) -> LargeSpec:
    """Qwen2.5-7B attention stack: 28/4 heads, ragged packets (lengths uniform in [lo, hi]),
    distinct packets per item, two outlier channels (x8) per (layer, kv head)."""
    rng = np.random.default_rng(seed + 4000)
    lens = [int(x) for x in rng.integers(lo, hi + 1, size=batch * per_item)]
    items = [[(b * per_item + s, 0) for s in range(per_item)] for b in range(batch)]
    shape = ModelShape(n_layers, 28, 4, 128, "bf16", 1000000.0, 0)
    return LargeSpec("config4", shape, lens, items, q_len, seed=seed, outlier_channels=2)


def spec_config5(n_packets: int, q_len: int, batch: int, seed: int = 0, doc_len: int = 2048) -> LargeSpec:
    """Long-context sweep point, Llama-3.1-8B single-layer shape; distinct packets per item."""
    items = [[(b * n_packets + s, 0) for s in range(n_packets)] for b in range(batch)]
    shape = ModelShape(1, 32, 8, 128, "bf16", 500000.0, 0)
    return LargeSpec(f"config5_n{n_packets}_q{q_len}_b{batch}", shape, [doc_len] * (batch * n_packets),
                     items, q_len, seed=seed)


def shard_spec(spec: LargeSpec, rank: int, world: int):
    """Rank ``rank``'s part of a spec whose requests use consecutive, distinct packets (config 5): every request's
    slot list is cut into ``world`` equal contiguous parts; the rank's packets keep the seeds they have in the whole
    spec, so the ranks together hold exactly the whole workload's bytes.  Returns (sub-spec, pos_base)."""
    per = [len(it) for it in spec.items]
    assert all(n % world == 0 for n in per), "slots do not divide over the ranks"
    flat = [pid for it in spec.items for pid, _ in it]
    assert flat == list(range(len(flat))), "requests must use consecutive distinct packets"
    # a rank's packets are not one contiguous range of the whole spec unless there is a single request, so the
    # sub-spec keeps one seed offset per request by laying its packets out request by request
    assert len(spec.items) == 1 or world == 1, "shard_spec handles one request per spec (use one spec per request)"
    n = per[0] // world
    lo = rank * n
    items = [[(s, aid) for s, (_, aid) in enumerate(spec.items[0][lo:lo + n])]]
    lens = [spec.packet_lens[pid] for pid, _ in spec.items[0][lo:lo + n]]
    pos = sum(spec.packet_lens[pid] + (spec.n_header + spec.n_trailer if aid >= 0 else 0) for pid, aid in spec.items[0][:lo])
    sub = LargeSpec(f"{spec.name}_rank{rank}of{world}", spec.shape, lens, items, spec.q_len, spec.n_header, spec.n_trailer,
                    spec.seed, spec.outlier_channels, spec.outlier_scale, spec.rebase, spec.packet_seed_offset + lo)
    return sub, [pos]


def shard_heads_spec(spec: LargeSpec, rank: int, world: int) -> LargeSpec:
    """Rank ``rank``'s part of a spec sharded by kv head: the same requests and packet lengths with Hkv / world kv
    heads (and their query heads), drawn with the rank's own seed - every rank holds different heads' values."""
    s = spec.shape
    assert s.n_kv_heads % world == 0, "kv heads do not divide over the ranks"
    n_kv = s.n_kv_heads // world
    shape = ModelShape(s.n_layers, n_kv * s.group, n_kv, s.head_dim, s.dtype, s.rope_theta, s.rope_pairing)
    return LargeSpec(spec.name, shape, list(spec.packet_lens), [list(it) for it in spec.items], spec.q_len, spec.n_header,
                     spec.n_trailer, spec.seed + 17 * rank, spec.outlier_channels, spec.outlier_scale, spec.rebase,
                     spec.packet_seed_offset)


class DeviceWorkload:
    """Draws a ``LargeSpec`` on the GPU, one tensor per ``torch.Generator`` seed, and re-draws any
    tensor on demand (same seed, same device, same bytes), so that the gigabytes never have to
    live on the host.  Seeds: ``base = seed*1_000_003``; packet p: K ``base+4p``, V ``base+4p+1``;
    adapter: ``base+10_000_000 + {0,1,2,3}``; query of layer l: ``base+20_000_000 + 4l + {0,1,2}``.
    """

    def __init__(self, spec: LargeSpec, device: str = "cuda:0"):
        import torch
        self.torch = torch
        self.spec = spec
        self.shape = spec.shape
        self.device = torch.device(device)
        self.items = spec.items
        self.rebase = spec.rebase
        self.name = spec.name
        self._base = spec.seed * 1_000_003
        self._chan = None
        self.notes = {"chan_scale": None}
        if spec.outlier_channels > 0:
            s = spec.shape
            crng = np.random.default_rng(spec.seed + 7919)
            cs = np.ones((s.n_layers, 1, s.n_kv_heads, s.head_dim), dtype=np.float32)
            for l in range(s.n_layers):
                for h in range(s.n_kv_heads):
                    cs[l, 0, h, crng.choice(s.head_dim, size=spec.outlier_channels, replace=False)] = spec.outlier_scale
            self._chan = torch.from_numpy(cs).to(self.device)
            self.notes["chan_scale"] = cs

    @property
    def batch(self) -> int:
        return len(self.items)

    @property
    def q_len(self) -> int:
        return self.spec.q_len

    def prefix_len(self, b: int) -> int:
        return self.spec.prefix_len(b)

    def _randn(self, seed: int, dims, scale=None):
        torch = self.torch
        g = torch.Generator(device=self.device)
        g.manual_seed(int(seed))
        x = torch.randn(dims, generator=g, device=self.device, dtype=torch.float32)
        if scale is not None:
            x = x * scale
        return x.to(torch.bfloat16 if self.shape.dtype == "bf16" else torch.float32)

    # device tensors -------------------------------------------------------------------
    def packet_device(self, pid: int):
        s = self.shape
        dims = (s.n_layers, self.spec.packet_lens[pid], s.n_kv_heads, s.head_dim)
        gp = pid + self.spec.packet_seed_offset
        return (self._randn(self._base + 4 * gp, dims, self._chan),
                self._randn(self._base + 4 * gp + 1, dims, self._chan))

    def adapter_device(self):
        s = self.shape
        hd = (s.n_layers, self.spec.n_header, s.n_kv_heads, s.head_dim)
        td = (s.n_layers, self.spec.n_trailer, s.n_kv_heads, s.head_dim)
        b = self._base + 10_000_000
        return (self._randn(b, hd), self._randn(b + 1, hd), self._randn(b + 2, td), self._randn(b + 3, td))

    def query_device(self, layer: int):
        s = self.shape
        B, Lq = self.batch, self.q_len
        b = self._base + 20_000_000 + 4 * layer
        return (self._randn(b, (B, Lq, s.n_q_heads, s.head_dim)),
                self._randn(b + 1, (B, Lq, s.n_kv_heads, s.head_dim)),
                self._randn(b + 2, (B, Lq, s.n_kv_heads, s.head_dim)))

    # host copies of the same bytes (for the oracle) ------------------------------------
    def _host(self, t):
        torch = self.torch
        if t.dtype == torch.bfloat16:
            return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
        return t.contiguous().cpu().numpy()

    def packet_layer(self, pid: int, layer: int):
        k, v = self.packet_device(pid)
        return self._host(k[layer]), self._host(v[layer])

    def adapter_host(self) -> Adapter:
        hk, hv, tk, tv = self.adapter_device()
        return Adapter(self._host(hk), self._host(hv), self._host(tk), self._host(tv), 0, 0)

    def query_layer(self, layer: int):
        q, k, v = self.query_device(layer)
        return self._host(q), self._host(k), self._host(v)
