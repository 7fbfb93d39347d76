"""CPU-side checks of the product library: it loads, exports what the header declares, validates
arguments on the host, and its planner's index map equals the oracle's composition bit for bit."""
import os
import re

import numpy as np
import pytest

from oracle import reference as orc
from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from helpers import make_store

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "kvp.h")).read()
    declared = sorted(set(re.findall(r"KVP_API[^;(]*?\b(kvp_\w+)\s*\(", header)))
    assert len(declared) >= 12 and "kvp_query_prefill" in declared and "kvp_assemble" in declared
    L = kvp.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert sorted(kvp.EXPORTED) == declared
    assert L.kvp_version() >= 100


def host_ctx(shape, wl, **kw):
    n_slots = sum(len(it) for it in wl.items)
    args = dict(max_packets=max(1, len(wl.packets)), max_adapters=max(1, len(wl.adapters)), max_batch=wl.batch,
                max_slots=max(1, n_slots), max_prefix_tokens=max(wl.prefix_len(b) for b in range(wl.batch)),
                max_query_tokens=wl.q_len, max_ws_rows=sum(wl.prefix_len(b) for b in range(wl.batch)) + wl.batch * wl.q_len,
                device=-1)
    args.update(kw)
    ctx = kvp.Context(shape.n_layers, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.dtype,
                      rope_theta=shape.rope_theta, **args)
    for p in wl.packets:
        ctx.register_packet(None, None, p.n_tokens, p.cache_pos0)
    for a in wl.adapters:
        ctx.register_adapter(None, None, a.n_header, a.header_pos0, None, None, a.n_trailer, a.trailer_pos0)
    return ctx


def ragged_workload(seed=0):
    shape = gen.ModelShape(2, 4, 2, 64, "bf16", 10000.0)
    lens = [37, 128, 300, 1, 129, 64]
    items = [[(0, 0), (2, 1), (5, -1)], [(3, 1)], [(4, 0), (1, 0), (0, 1), (2, -1)]]
    return gen.make_workload(shape, lens, items, q_len=5, n_header=3, n_trailer=2, n_adapters=2, seed=seed,
                             packet_pos0=[0, 5, 0, 7, 100, 0], adapter_pos0=[(0, 0), (2, 40)])


@pytest.mark.parametrize("flags", [kvp.REBASE, 0, kvp.REBASE | kvp.MATERIALIZE])
def test_planner_index_map_equals_oracle(flags):
    wl = ragged_workload()
    ctx = host_ctx(wl.shape, wl)
    aid, plen = ctx.assemble(wl.items, flags)
    st = make_store(wl)
    for b, slots in enumerate(wl.items):
        plan = orc.compose(st, slots, rebase=bool(flags & kvp.REBASE))
        assert plen[b] == plan.prefix_len == wl.prefix_len(b)
        src, dl, segs = ctx.export_plan(aid, b)
        assert np.array_equal(src, plan.src_row)
        assert np.array_equal(dl, plan.delta)
        assert np.array_equal(segs, plan.segments)
    ctx.close()


def test_planner_config1_and_config2_layouts():
    for wl in (gen.config1(), gen.config2()):
        ctx = host_ctx(wl.shape, wl)
        aid, plen = ctx.assemble(wl.items, kvp.REBASE)
        plan = orc.compose(make_store(wl), wl.items[0])
        src, dl, segs = ctx.export_plan(aid, 0)
        assert plen[0] == plan.prefix_len
        assert np.array_equal(src, plan.src_row) and np.array_equal(dl, plan.delta) and np.array_equal(segs, plan.segments)
        ctx.close()


def test_argument_errors_are_status_codes():
    wl = ragged_workload()
    ctx = host_ctx(wl.shape, wl, max_slots=8)
    with pytest.raises(kvp.KvpError) as e:
        ctx.assemble([[(99, 0)]])
    assert e.value.code == 3
    with pytest.raises(kvp.KvpError) as e:
        ctx.assemble([[(0, 7)]])
    assert e.value.code == 3
    with pytest.raises(kvp.KvpError) as e:
        ctx.assemble([[(0, 0)] * 9])
    assert e.value.code == 2                       # more slots than max_slots
    with pytest.raises(kvp.KvpError) as e:
        ctx.assemble([[(2, 0)] * 8])
    assert e.value.code == 2                       # prefix longer than max_prefix_tokens
    with pytest.raises(kvp.KvpError) as e:
        ctx.assemble(wl.items, 64)
    assert e.value.code == 1                       # unknown flag
    with pytest.raises(kvp.KvpError) as e:
        ctx.register_packet(None, None, 0, 0)
    assert e.value.code == 1
    aid, plen = ctx.assemble(wl.items)
    with pytest.raises(kvp.KvpError) as e:
        ctx.export_plan(aid + 5, 0)
    assert e.value.code == 3
    # a host-only context cannot launch anything: the call fails loudly instead of computing on the CPU
    with pytest.raises(kvp.KvpError) as e:
        ctx.query_prefill(aid, 0, 1, 1, 1, 1, 1)
    assert e.value.code == 4
    ctx.close()


def test_misaligned_pointers_are_refused_on_the_host():
    # 16-byte vector accesses need 16-byte aligned pointers; the check comes before any CUDA call, so it can be
    # exercised without a device (the addresses are never dereferenced)
    wl = ragged_workload()
    ctx = host_ctx(wl.shape, wl, max_slots=8)
    for k, v in ((4096 + 8, 4096), (4096, 4096 + 2)):
        with pytest.raises(kvp.KvpError) as e:
            ctx.register_packet(k, v, 4, 0)
        assert e.value.code == 1 and "aligned" in str(e.value)
    with pytest.raises(kvp.KvpError) as e:
        ctx.register_adapter(4096, 4096, 2, 0, 4096, 4096 + 4, 2, 0)
    assert e.value.code == 1 and "aligned" in str(e.value)
    ctx.close()
    ok = 1 << 20
    for bad in range(4):
        ptrs = [ok, ok, ok, ok]
        ptrs[bad] += 8
        with pytest.raises(kvp.KvpError) as e:
            kvp.compose_noalloc(ptrs[0], ptrs[1], 64, 4, 128, "bf16", 0, 10000.0, [(0, 8, 0)], ptrs[2], ptrs[3], 128)
        assert e.value.code == 1 and "aligned" in str(e.value)
    # the running row count is checked before it is narrowed to 32 bits
    big = [(0, 2 ** 31 - 8, 0), (0, 2 ** 31 - 8, 0)]
    with pytest.raises(kvp.KvpError) as e:
        kvp.compose_noalloc(ok, ok, 2 ** 31 - 1, 1, 128, "bf16", 0, 10000.0, big, ok, ok, 2 ** 33)
    assert e.value.code == 2
    with pytest.raises(kvp.KvpError) as e:
        kvp.compose_noalloc(ok, ok, 64, 4, 128, "bf16", 0, 10000.0, [(0, 1, 0)] * 97, ok, ok, 128)
    assert e.value.code == 2 and "96" in str(e.value)
    with pytest.raises(kvp.KvpError) as e:
        kvp.compose_noalloc(ok, ok, 64, 4, 128, "bf16", 0, 10000.0, [(60, 10, 0)], ok, ok, 128)
    assert e.value.code == 1


def test_bad_configurations_rejected():
    for kw in (dict(n_q_heads=5, n_kv_heads=2), dict(head_dim=96), dict(n_layers=0)):
        args = dict(n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64)
        args.update(kw)
        with pytest.raises(kvp.KvpError):
            kvp.Context(args["n_layers"], args["n_q_heads"], args["n_kv_heads"], args["head_dim"], "bf16", device=-1)


def test_assembly_ring_drops_old_ids():
    wl = ragged_workload()
    ctx = host_ctx(wl.shape, wl, max_assemblies=2)
    a0, plen = ctx.assemble(wl.items)
    a1, _ = ctx.assemble(wl.items)
    a2, _ = ctx.assemble(wl.items)
    assert (a0, a1, a2) == (0, 1, 2)
    ctx.export_plan(a1, 0)
    ctx.export_plan(a2, 0)
    with pytest.raises(kvp.KvpError):
        ctx.export_plan(a0, 0)
    ctx.close()


# ------------------------------------------------------------------------------------------------
# work list of the persistent attention kernel: every key tile of every unit exactly once
# ------------------------------------------------------------------------------------------------

def _schedule_case(n_q, n_kv, lens, items, q_len):
    shape = gen.ModelShape(1, n_q, n_kv, 128, "bf16", 500000.0)
    wl = gen.make_workload(shape, lens, items, q_len=q_len, n_header=16, n_trailer=16, seed=1)
    ctx = host_ctx(shape, wl)
    aid, plen = ctx.assemble(wl.items, kvp.REBASE)
    return ctx, aid, plen, shape


@pytest.mark.parametrize("case", [
    (32, 8, [1024] * 10, [[(i, 0) for i in range(10)]] * 4, 128),        # config-3 shape: two-tile units, split
    (32, 8, [2048] * 8, [[(i, 0) for i in range(8)]], 16),                # 64 rows per kv head: mode 1 units
    (28, 4, [300, 1000, 257, 640], [[(0, 0), (1, 0)], [(2, 0), (3, 0), (0, -1)]], 50),   # g = 7, ragged
    (8, 8, [100], [[(0, 0)]], 1),                                          # decode-like: one row per head
    (32, 8, [512] * 5, [[(i, 0) for i in range(5)]], 64),                 # config-2 shape: little work
    (4, 4, [200, 3000], [[(0, 0)], [(1, 0), (0, 0)]], 700),               # g = 1, many query tiles
])
def test_schedule_covers_every_tile_once(case):
    n_q, n_kv, lens, items, q_len = case
    ctx, aid, plen, shape = _schedule_case(n_q, n_kv, lens, items, q_len)
    cb, works, merges, n_slots = ctx.export_schedule(aid, q_len)
    g = n_q // n_kv
    n_rows = g * q_len
    assert cb[0] == 0 and cb[-1] == len(works) and np.all(np.diff(cb) > 0) and len(cb) - 1 <= 148
    # expected units and their tile counts, from the assembly's own description
    covered = {}
    for w in works:
        b, hk, row_base, mode, lo, n, s0, s1 = (int(x) for x in w)
        assert 0 <= b < len(items) and 0 <= hk < n_kv and row_base % 256 == 0 and 0 <= row_base < n_rows
        assert mode == (1 if n_rows - row_base <= 128 else 0) and n >= 1 and lo >= 0
        covered.setdefault((b, hk, row_base), []).append((lo, n, s0, s1, mode))
    slots_seen = []
    for b in range(len(items)):
        _, _, segs = ctx.export_plan(aid, b)
        # prefix tiles: staged adapter rows form one run, each document its own run of <=128-key tiles
        adapters = sum(int(s[1]) for s in segs if int(s[1]) in (16,) )
        docs = [int(s[1]) for s in segs if int(s[1]) != 16]
        n_prefix = -(-adapters // 128) + sum(-(-d // 128) for d in docs)
        for hk in range(n_kv):
            for row_base in range(0, n_rows, 256):
                mode = 1 if n_rows - row_base <= 128 else 0
                last = min(n_rows - 1, row_base + (128 if mode else 256) - 1)
                n_all = (last // g) // 128 + 1 + n_prefix
                pieces = sorted(covered.pop((b, hk, row_base)))
                pos = 0
                for lo, n, s0, s1, m in pieces:
                    assert lo == pos
                    pos += n
                    if len(pieces) == 1:
                        assert s0 == -1 and s1 == -1
                    else:
                        assert s0 >= 0 and (s1 >= 0) == (m == 0)
                        slots_seen += [s0] + ([s1] if m == 0 else [])
                assert pos == n_all
    assert not covered
    assert sorted(slots_seen) == list(range(n_slots))
    # merge items name every slot exactly once, grouped per 128-row query tile
    named = []
    for m in merges:
        b, hk, row_base, s0, n = (int(x) for x in m[:5])
        assert n >= 2 and row_base % 128 == 0 and row_base < n_rows
        named += list(range(s0, s0 + n))
    assert sorted(named) == list(range(n_slots))
    # balance: no CTA carries more than its share plus a few tiles (a piece's fixed cost counts as 4)
    cost = [sum(int(works[i][5]) * (1 if works[i][3] else 2) + 4 for i in range(cb[c], cb[c + 1])) for c in range(len(cb) - 1)]
    assert max(cost) <= sum(cost) / len(cost) + 16


def test_compressed_registration_and_per_layer_lists_host_only():
    shape = gen.ModelShape(3, 8, 2, 128, "bf16", 500000.0)
    wl = gen.make_workload(shape, [300, 700], [[(0, 0), (1, 0)]], q_len=8, seed=2, keep_rate=[0.5, None])
    ctx = kvp.Context(3, 8, 2, 128, "bf16", rope_theta=500000.0, max_packets=4, max_adapters=1, max_batch=1, max_slots=2,
                      max_prefix_tokens=1100, max_query_tokens=8, max_ws_rows=200, device=-1, max_compressed=1)
    counts = [len(wl.packets[0].kept[l][h]) for l in range(3) for h in range(2)]
    pid = ctx.register_packet_compressed(None, None, 300, 0, counts)
    ctx.register_packet(None, None, 700, 0)
    ctx.register_adapter(None, None, 16, 0, None, None, 16, 0)
    aid, plen = ctx.assemble(wl.items, kvp.REBASE)
    assert pid == 0 and plen == [16 + 300 + 16 + 16 + 700 + 16]
    src, dl, segs = ctx.export_plan(aid, 0)
    assert np.all(src[16:316] == -1) and np.all(dl[16:316] == 16)       # one offset for the compressed packet
    assert src[348] == max(counts)                                       # the next packet follows max(kept) pool rows
    with pytest.raises(kvp.KvpError) as e:
        ctx.register_packet_compressed(None, None, 300, 0, [0] * 6)
    assert e.value.code == 1
    with pytest.raises(kvp.KvpError) as e:
        ctx.register_packet_compressed(None, None, 300, 0, [301] * 6)
    assert e.value.code == 1
    plain = kvp.Context(3, 8, 2, 128, "bf16", max_packets=2, device=-1)
    with pytest.raises(kvp.KvpError) as e:
        plain.register_packet_compressed(None, None, 300, 0, counts)
    assert e.value.code == 4


def test_schedule_gives_units_that_share_keys_the_same_cuts_on_neighbouring_ctas():
    # Config-3 shape: every (request, kv head) has two 256-row units that stream the same K/V.  Each row block is
    # cut on its own run of CTAs, so the second unit's pieces repeat the first one's cuts, and the j-th CTAs of the
    # row blocks are emitted next to each other: the two CTAs reach the same key tiles at the same time.
    ctx, aid, plen, shape = _schedule_case(32, 8, [1024] * 10, [[(i, 0) for i in range(10)]] * 4, 128)
    cb, works, merges, n_slots = ctx.export_schedule(aid, 128)
    n_ctas = len(cb) - 1
    assert n_ctas == 148
    pieces = {}
    for c in range(n_ctas):
        for i in range(cb[c], cb[c + 1]):
            b, hk, row_base, mode, lo, n = (int(x) for x in works[i][:6])
            pieces.setdefault((b, hk, row_base), []).append((c, lo, n))
    for (b, hk, row_base), first in pieces.items():
        if row_base != 0:
            continue
        second = pieces[(b, hk, 256)]
        assert len(first) == len(second)
        for (c0, lo0, n0), (c1, lo1, n1) in zip(first, second):
            assert (c1, lo1, n1) == (c0 + 1, lo0, n0)
    ctx.close()


def test_row_blocks_with_different_causal_tiles_are_cut_at_the_same_prefix_tiles():
    # 256 query tokens, g = 4: four 256-row units per (request, kv head) with 1, 1, 2, 2 causal tiles in front of
    # the same 65 prefix tiles.  Counted from the first prefix tile the cuts of all row blocks coincide, and the j-th
    # CTAs of the row blocks sit next to each other: CTAs that stream the same K/V stay on the same tiles.
    ctx, aid, plen, shape = _schedule_case(32, 8, [2048] * 4, [[(i, 0) for i in range(4)]] * 2, 256)
    cb, works, merges, n_slots = ctx.export_schedule(aid, 256)
    n_ctas = len(cb) - 1
    starts = {}
    for c in range(n_ctas):
        for i in range(cb[c], cb[c + 1]):
            b, hk, row_base, mode, lo, n = (int(x) for x in works[i][:6])
            last = min(4 * 256, row_base + 256) - 1
            n_tail = (last // 4) // 128 + 1
            starts.setdefault(row_base, []).append((b, hk, 0 if lo == 0 else lo - n_tail, c))
    assert sorted(starts) == [0, 256, 512, 768]
    ref = [(b, hk, p) for b, hk, p, c in starts[0]]
    assert any(p > 0 for _, _, p in ref)                       # units are split
    for rb, lst in starts.items():
        assert [(b, hk, p) for b, hk, p, c in lst] == ref       # same cuts in prefix coordinates
    for j in range(len(ref)):                                   # and the CTAs that share a cut are neighbours
        ctas = [starts[rb][j][3] for rb in sorted(starts)]
        assert max(ctas) - min(ctas) <= 2 * len(starts)
    ctx.close()


def test_packets_registered_from_host_memory_plan_like_any_other():
    # host-only context: nothing is copied, but rows are reserved in the same order and the plan is the same;
    # only packets that came from host memory can be evicted
    shape = gen.ModelShape(2, 8, 2, 128, "bf16", 500000.0)
    wl = gen.make_workload(shape, [200, 37, 300], [[(0, 0), (2, 0)], [(1, 0), (0, -1)]], q_len=8, n_header=16, n_trailer=16, seed=2)
    a = host_ctx(shape, wl)
    aid_a, plen_a = a.assemble(wl.items, kvp.REBASE)
    b = kvp.Context(shape.n_layers, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.dtype, rope_theta=shape.rope_theta,
                    pool_tokens=1000, max_packets=3, max_adapters=1, max_batch=2, max_slots=4, max_prefix_tokens=1000,
                    max_query_tokens=8, max_ws_rows=1200, device=-1)
    for p_ in wl.packets:
        b.register_packet_host(None, None, p_.n_tokens, p_.cache_pos0)
    ad = wl.adapters[0]
    b.register_adapter(None, None, ad.n_header, ad.header_pos0, None, None, ad.n_trailer, ad.trailer_pos0)
    aid_b, plen_b = b.assemble(wl.items, kvp.REBASE)
    assert plen_a == plen_b
    for i in range(2):
        pa, pb = a.export_plan(aid_a, i), b.export_plan(aid_b, i)
        assert all(np.array_equal(x, y) for x, y in zip(pa, pb))
    b.evict_packet(1)
    with pytest.raises(kvp.KvpError):
        a.evict_packet(1)
    a.close()
    b.close()

