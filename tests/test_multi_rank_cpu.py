"""The N > 1 path of the benchmark on CPU: two `gloo` ranks.  The path shards requests across ranks with no
data-path collective (requests are independent, Section 3.2), so what there is to check is that every rank
plans a different batch of the same shape, that the timing exchange takes the maximum over ranks, and that
the whole-job rate counts every rank's tokens."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import json, os, sys
sys.path.insert(0, os.environ["KVP_ROOT"])
import torch.distributed as dist
import bench
from paper_2604_13226_b200 import binding as kvp
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
spec = bench.rank_spec("config5:3:16:2", 5, rank)
s = spec.shape
# host-only planning of this rank's batch through the C ABI: prefix lengths and the kernel's work list
ctx = kvp.Context(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, s.dtype, rope_theta=s.rope_theta,
                  max_packets=len(spec.packet_lens), max_adapters=1, max_batch=spec.batch,
                  max_slots=sum(len(it) for it in spec.items), max_prefix_tokens=max(spec.prefix_len(b) for b in range(spec.batch)),
                  max_query_tokens=spec.q_len, max_ws_rows=4096, device=-1)
for n in spec.packet_lens:
    ctx.register_packet(None, None, n, 0)
ctx.register_adapter(None, None, spec.n_header, 0, None, None, spec.n_trailer, 0)
aid, plen = ctx.assemble(spec.items, kvp.REBASE)
cb, works, merges, n_slots = ctx.export_schedule(aid, spec.q_len)
ms = bench.max_over_ranks([10.0 + rank, 7.0 - rank], world)
dist.barrier()
print(json.dumps({"rank": rank, "seed": spec.seed, "prefix": plen, "batch": spec.batch, "q_len": spec.q_len,
                  "pieces": int(len(works)), "ms": ms, "value": bench.job_tokens_per_s(spec, world, ms[0])}))
dist.destroy_process_group()
'''


def test_two_gloo_ranks_shard_requests_and_reduce_timings(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = 29500 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   KVP_ROOT=ROOT, CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    a, b = outs
    assert a["seed"] != b["seed"]                                   # every rank draws its own batch
    assert a["batch"] == b["batch"] == 2 and a["q_len"] == b["q_len"] == 16
    assert a["prefix"] == b["prefix"] == [3 * (2048 + 32)] * 2      # same shape on every rank
    assert a["pieces"] >= 1 and b["pieces"] >= 1
    assert a["ms"] == b["ms"] == [11.0, 7.0]                        # maximum over ranks, element-wise
    assert abs(a["value"] - 2 * 2 * 16 / 11.0e-3) < 1e-6 and a["value"] == b["value"]


# Prefix sharding (the packets of one request spread over the ranks): every rank plans its part with
# kvp_assemble_at; the parts must tile the whole request - same segment lengths, the rotation offsets the oracle's
# composition of the whole request gives, positions shifted by the rank's base - and the ranks agree on the total.
SHARD_WORKER = r'''
import json, os, sys
sys.path.insert(0, os.environ["KVP_ROOT"]); sys.path.insert(0, os.path.join(os.environ["KVP_ROOT"], "tests"))
import numpy as np
import torch.distributed as dist
from oracle import reference as orc
from paper_2604_13226_b200 import binding as kvp, inputs as gen
from helpers import make_store
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
shape = gen.ModelShape(1, 4, 2, 64, "f32", 10000.0, 0)
lens = [40, 130, 7, 64, 90]
items = [[(0, 0), (1, 0), (2, -1), (3, 0), (4, 0)], [(4, 0), (0, 0), (1, -1)], [(2, 0)]]
wl = gen.make_workload(shape, lens, items, q_len=4, n_header=3, n_trailer=5, seed=9, packet_pos0=[0, 11, 0, 500, 2])
sub, pos_base = gen.shard_workload(wl, rank, world)
ctx = kvp.Context(1, 4, 2, 64, "f32", rope_theta=10000.0, max_packets=8, max_adapters=1, max_batch=3, max_slots=16,
                  max_prefix_tokens=1024, max_query_tokens=4, max_ws_rows=4096, device=-1)
for p in sub.packets:
    ctx.register_packet(None, None, p.n_tokens, p.cache_pos0)
a = sub.adapters[0]
ctx.register_adapter(None, None, a.n_header, a.header_pos0, None, None, a.n_trailer, a.trailer_pos0)
aid, plen = ctx.assemble(sub.items, kvp.REBASE, pos_base=pos_base)
st = make_store(wl)
ok = True
for b in range(wl.batch):
    whole = orc.compose(st, wl.items[b])
    segs = whole.segments                                          # [src_row0, len, dst_pos0, delta] of the whole request
    mine = [s for s in segs if pos_base[b] <= s[2] < pos_base[b] + plen[b]]
    _, dl, got = ctx.export_plan(aid, b)
    ok = ok and len(got) == len(mine)
    for g, m in zip(got, mine):
        ok = ok and int(g[1]) == int(m[1]) and int(g[3]) == int(m[3]) and int(g[2]) + pos_base[b] == int(m[2])
    ok = ok and np.array_equal(dl, whole.delta[pos_base[b]:pos_base[b] + plen[b]])
gathered = [None] * world
dist.all_gather_object(gathered, (pos_base, plen))
total = [sum(g[1][b] for g in gathered) for b in range(wl.batch)]
tiles = all(gathered[r][0][b] + gathered[r][1][b] == gathered[r + 1][0][b] for r in range(world - 1) for b in range(wl.batch))
print(json.dumps({"rank": rank, "ok": bool(ok), "total": total, "whole": [wl.prefix_len(b) for b in range(wl.batch)],
                  "tiles": bool(tiles), "partial_bytes": ctx.partial_bytes(3, 4)}))
dist.destroy_process_group()
'''


def test_two_gloo_ranks_plan_the_parts_of_prefix_sharded_requests(tmp_path):
    script = tmp_path / "shard_worker.py"
    script.write_text(SHARD_WORKER)
    port = 31500 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   KVP_ROOT=ROOT, CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    for p in procs:
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-2000:]
        d = json.loads(out.strip().splitlines()[-1])
        assert d["ok"] and d["tiles"] and d["total"] == d["whole"]
        # 3 requests x 2 kv heads x 1 row tile of 128 packed rows, 64 fp32 columns + (m, l) per row
        assert d["partial_bytes"] == 3 * 2 * 1 * 128 * (64 * 4 + 8)


# Kv-head sharding: every rank plans the SAME requests for its own heads; the head ranges tile [0, Hkv), the ranks'
# slices put side by side are the whole tensors, the composition (which rows, which offsets) does not depend on the
# heads, and the whole-job rate counts the batch once.
HEAD_WORKER = r'''
import json, os, sys
sys.path.insert(0, os.environ["KVP_ROOT"]); sys.path.insert(0, os.path.join(os.environ["KVP_ROOT"], "tests"))
import numpy as np
import torch.distributed as dist
from oracle import reference as orc
import bench
from paper_2604_13226_b200 import binding as kvp, inputs as gen
from helpers import make_store
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
shape = gen.ModelShape(2, 12, 4, 64, "f32", 10000.0, 0)
items = [[(0, 0), (1, 0), (2, -1)], [(2, 0), (0, 0)]]
wl = gen.make_workload(shape, [40, 130, 7], items, q_len=5, n_header=3, n_trailer=5, seed=11, packet_pos0=[0, 11, 2])
sub = gen.shard_heads(wl, rank, world)
s = sub.shape
ctx = kvp.Context(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, s.dtype, rope_theta=s.rope_theta, max_packets=4,
                  max_adapters=1, max_batch=2, max_slots=8, max_prefix_tokens=512, max_query_tokens=5, max_ws_rows=1024, device=-1)
for p in sub.packets:
    ctx.register_packet(None, None, p.n_tokens, p.cache_pos0)
a = sub.adapters[0]
ctx.register_adapter(None, None, a.n_header, a.header_pos0, None, None, a.n_trailer, a.trailer_pos0)
aid, plen = ctx.assemble(sub.items, kvp.REBASE)
st = make_store(wl)                                              # the whole workload's store: the plan must not depend on the heads
ok = plen == [wl.prefix_len(b) for b in range(wl.batch)]
for b in range(wl.batch):
    whole = orc.compose(st, wl.items[b])
    src, dl, segs = ctx.export_plan(aid, b)
    ok = ok and np.array_equal(dl, whole.delta) and len(segs) == len(whole.segments)
    ok = ok and all(int(g[1]) == int(m[1]) and int(g[2]) == int(m[2]) and int(g[3]) == int(m[3]) for g, m in zip(segs, whole.segments))
gathered = [None] * world
dist.all_gather_object(gathered, (sub.q, sub.k_new, sub.packets[1].k, sub.adapters[0].tv))
whole_again = [np.concatenate([g[i] for g in gathered], axis=-2) for i in range(4)]
tiles = all(np.array_equal(x, y) for x, y in zip(whole_again, (wl.q, wl.k_new, wl.packets[1].k, wl.adapters[0].tv)))
spec = bench.head_spec("config3", 0, rank, world)
ms = bench.max_over_ranks([4.0 + rank], world)
print(json.dumps({"rank": rank, "ok": bool(ok), "tiles": bool(tiles), "heads": [s.n_q_heads, s.n_kv_heads],
                  "spec_heads": [spec.shape.n_q_heads, spec.shape.n_kv_heads], "spec_seed": spec.seed, "items": spec.items,
                  "value": bench.job_tokens_per_s(spec, world, ms[0], "heads")}))
dist.destroy_process_group()
'''


def test_two_gloo_ranks_shard_kv_heads_of_the_same_requests(tmp_path):
    script = tmp_path / "head_worker.py"
    script.write_text(HEAD_WORKER)
    port = 33500 + os.getpid() % 2000
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port),
                   KVP_ROOT=ROOT, CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=240)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    a, b = outs
    assert a["ok"] and b["ok"] and a["tiles"] and b["tiles"]
    assert a["heads"] == b["heads"] == [6, 2]                       # 12 / 4 heads over two ranks, g = 3 kept
    assert a["spec_heads"] == b["spec_heads"] == [16, 4]            # config 3: 32 / 8 heads over two ranks
    assert a["items"] == b["items"] and a["spec_seed"] != b["spec_seed"]      # the same requests, each rank its heads' values
    assert abs(a["value"] - 4 * 128 / 5.0e-3) < 1e-6 and a["value"] == b["value"]   # the batch counted once, slowest rank


def test_oracle_over_head_slices_equals_slices_of_the_oracle_over_all_heads():
    # What kv-head sharding rests on, checked on the oracle alone: the definition's result for query head h depends on
    # kv head h // g only, so the oracle run on rank r's slice of a workload (inputs.shard_heads) gives, bit for bit,
    # rank r's slice of the oracle's result for the whole workload - plain and with a pruned packet.
    import numpy as np
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from paper_2604_13226_b200 import inputs as gen
    from helpers import oracle_outputs
    shape = gen.ModelShape(2, 12, 4, 64, "f32", 10000.0, 1)
    items = [[(0, 0), (1, 0), (2, -1)], [(2, 0), (0, 0)]]
    for keep in (None, [0.5, None, 0.8]):
        wl = gen.make_workload(shape, [40, 130, 7], items, q_len=5, n_header=3, n_trailer=5, seed=12, packet_pos0=[0, 11, 2],
                               keep_rate=keep)
        whole = oracle_outputs(wl, layer=1)
        for world in (2, 4):
            g, per = shape.group, shape.n_q_heads // world
            for r in range(world):
                part = oracle_outputs(gen.shard_heads(wl, r, world), layer=1)
                for b in range(wl.batch):
                    wo = whole[b][0].reshape(wl.q_len, shape.n_q_heads, shape.head_dim)[:, r * per:(r + 1) * per]
                    wlse = whole[b][1].reshape(wl.q_len, shape.n_q_heads)[:, r * per:(r + 1) * per]
                    assert np.array_equal(part[b][0].reshape(wl.q_len, per, shape.head_dim), wo)
                    assert np.array_equal(part[b][1].reshape(wl.q_len, per), wlse)
