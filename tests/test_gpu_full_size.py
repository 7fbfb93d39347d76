"""GPU parity at the full sizes of the workloads the benchmark times (configs 3, 4 and points of the
config-5 sweep), in the launch configuration `bench.py` uses (default tuning, documents read in place).
The fp64 oracle cannot run gigabytes in seconds, so it computes sampled output rows one by one - fixed
tokens {0, 1, 63, 64, 127, 128, last} plus seeded random (head, token) pairs - and every output row is
additionally cross-checked between the tcgen05 kernel and the fp32 CUDA-core kernel.  The assembly's index
map is compared bit for bit with the oracle's composition."""
import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from paper_2604_13226_b200.session import Session, torch_to_np
from helpers import attention_error_stats, make_store, oracle_outputs

pytestmark = pytest.mark.gpu

def sample_rows(spec, seed, n_random=24):
    s = spec.shape
    rng = np.random.default_rng(seed)
    toks = sorted(set([0, 1, 63, 64, 127, 128, spec.q_len - 1]) & set(range(spec.q_len)))
    rows = {(int(rng.integers(s.n_q_heads)), t) for t in toks}
    rows |= {(h, spec.q_len - 1) for h in range(0, s.n_q_heads, max(1, s.n_q_heads // 4))}
    while len(rows) < len(toks) + 4 + n_random:
        rows.add((int(rng.integers(s.n_q_heads)), int(rng.integers(spec.q_len))))
    return sorted(rows)


def check_sampled(wl, sess, layer, requests, seed, flags=0):
    spec, s = wl.spec, wl.shape
    qkv = sess.query_tensors(layer)
    out, lse = sess.prefill(layer, flags, qkv=qkv)
    assert sess.ctx.status_word() == 0 and sess.ctx.last_launch()["kind"] == 1
    o = orc.widen(torch_to_np(out, s.dtype), s.dtype)
    lse = lse.cpu().numpy().astype(np.float64)
    rows = sample_rows(spec, seed)
    st = make_store(wl)
    f = orc.inv_freq(s.rope_theta, s.head_dim)
    q, kn, vn = wl.query_layer(layer)
    got, want = [], []
    for b in requests:
        plan = orc.compose(st, wl.items[b], wl.rebase)
        ro, rl, _, _ = orc.query_prefill(st, plan, layer, q[b], kn[b], vn[b], f, s.rope_pairing, rows=rows)
        for n, (h, i) in enumerate(rows):
            got.append(o[b, i, h])
            want.append(ro[n])
            assert abs(lse[b, h, i] - rl[n]) <= 2e-2, (b, h, i)
    stats = attention_error_stats(np.stack(got), np.stack(want))       # raw 2e-2 / 2e-3, no per-channel scaling
    print("raw attention error vs oracle:", spec.name, "layer", layer, "requests", list(requests), stats)
    return out, qkv


def cross_check_all_rows(sess, layer, out, qkv):
    # two bf16-rounded outputs: each may sit half an ulp (2^-8 |O| at worst) from the exact value
    ref, _ = sess.prefill(layer, kvp.FORCE_SIMPLE, qkv=qkv)
    d = (out.float() - ref.float()).abs()
    over = d - (3e-2 + 2.0 ** -7 * ref.float().abs())
    assert float(over.max()) <= 0 and float(d.mean()) <= 2e-3, (float(d.max()), float(d.mean()))


def check_index_map(wl, sess, requests):
    st = make_store(wl)
    for b in requests:
        plan = orc.compose(st, wl.items[b], wl.rebase)
        src, dl, segs = sess.ctx.export_plan(sess.assembly_id, b)
        assert np.array_equal(src, plan.src_row) and np.array_equal(dl, plan.delta) and np.array_equal(segs, plan.segments)


def test_config3_full_size():
    spec = gen.spec_config3(seed=0)
    assert spec.shape.n_layers == 32 and spec.batch == 4 and spec.q_len == 128 and spec.prefix_len(0) == 10560
    wl = gen.DeviceWorkload(spec, "cuda:0")
    sess = Session(wl)
    sess.assemble()
    check_index_map(wl, sess, range(4))
    for layer, reqs in ((0, [0, 3]), (17, [1]), (31, [2])):
        out, qkv = check_sampled(wl, sess, layer, reqs, seed=100 + layer)
    cross_check_all_rows(sess, 31, out, qkv)
    sess.close()


def test_config4_full_size_ragged_group7_outlier_channels():
    spec = gen.spec_config4(seed=0)
    s = spec.shape
    assert (s.n_layers, s.n_q_heads, s.n_kv_heads) == (28, 28, 4) and spec.batch == 8 and spec.q_len == 256
    assert len(set(spec.prefix_len(b) for b in range(8))) > 1                      # ragged prefixes
    wl = gen.DeviceWorkload(spec, "cuda:0")
    sess = Session(wl)
    sess.assemble()
    check_index_map(wl, sess, [0, 7])
    shortest = min(range(8), key=spec.prefix_len)
    longest = max(range(8), key=spec.prefix_len)
    # x8 outlier channels in K and V: the workload the library's KVP_PRECISE_QK is for (bench.py times it the same way)
    out, qkv = check_sampled(wl, sess, 0, [shortest], seed=200, flags=kvp.PRECISE_QK)
    out, qkv = check_sampled(wl, sess, 27, [longest], seed=201, flags=kvp.PRECISE_QK)
    cross_check_all_rows(sess, 27, out, qkv)
    sess.close()


@pytest.mark.parametrize("n_packets,q_len,batch,requests", [
    (64, 16, 1, [0]),            # 133,120-token prefix, memory-bound
    (2, 16, 16, [0, 15]),        # shortest prefix, widest batch
    (16, 256, 4, [1]),           # compute-bound middle of the sweep
    (64, 1024, 1, [0]),          # longest prefix x longest query
    (64, 16, 16, [5]),           # the sweep's largest footprint: 1024 distinct packets, 8.6 GB of K/V
    (8, 1, 4, [2]),              # a decode-sized query
])
def test_config5_sweep_points(n_packets, q_len, batch, requests):
    spec = gen.spec_config5(n_packets, q_len, batch, seed=0)
    assert spec.prefix_len(0) == n_packets * 2080
    wl = gen.DeviceWorkload(spec, "cuda:0")
    sess = Session(wl)
    sess.assemble()
    check_index_map(wl, sess, requests[:1])
    out, qkv = check_sampled(wl, sess, 0, requests, seed=300 + n_packets + q_len)
    if n_packets * q_len * batch <= 16 * 256 * 4:
        cross_check_all_rows(sess, 0, out, qkv)
    sess.close()
    del sess, wl
    torch.cuda.empty_cache()


def test_config5_longest_prefix_sharded_over_two_ranks():
    # the 133,120-token request of the memory-bound sweep point with its 64 packets on two ranks (32 each, the same
    # bytes as the whole workload): partial prefill per rank, the gathered buffers merged, sampled rows against the
    # oracle over the WHOLE request - the launch configuration `bench.py --shard prefix` times
    whole = gen.spec_config5(64, 16, 1, seed=0)
    wl = gen.DeviceWorkload(whole, "cuda:0")
    s = whole.shape
    parts, sessions = [], []
    for r in range(2):
        sub, pos_base = gen.shard_spec(whole, r, 2)
        assert sub.prefix_len(0) == 32 * 2080 and pos_base == [r * 32 * 2080]
        sess = Session(gen.DeviceWorkload(sub, "cuda:0"))
        aid, plen = sess.assemble(pos_base=pos_base)
        q, kn, vn = wl.query_device(0)
        buf = torch.empty(sess.ctx.partial_bytes(1, 16), dtype=torch.uint8, device=q.device)
        sess.ctx.query_prefill(aid, 0, q, kn, vn, 16, buf, None, kvp.PARTIAL | (kvp.SKIP_QUERY_BLOCK if r == 0 else 0))
        assert sess.ctx.status_word() == 0
        parts.append(buf)
        sessions.append(sess)
    out = torch.zeros(1, 16, s.n_q_heads, s.head_dim, dtype=torch.bfloat16, device="cuda:0")
    lse = torch.zeros(1, s.n_q_heads, 16, dtype=torch.float32, device="cuda:0")
    sessions[0].ctx.merge_partials(torch.cat(parts), 2, 1, 16, out, lse)
    torch.cuda.synchronize()
    o = orc.widen(torch_to_np(out, "bf16"), "bf16")
    rows = sample_rows(whole, 400)
    st = make_store(wl)
    q, kn, vn = wl.query_layer(0)
    plan = orc.compose(st, wl.items[0], True)
    ro, rl, _, _ = orc.query_prefill(st, plan, 0, q[0], kn[0], vn[0], orc.inv_freq(s.rope_theta, s.head_dim), s.rope_pairing, rows=rows)
    stats = attention_error_stats(np.stack([o[0, i, h] for h, i in rows]), ro)
    print("raw attention error vs oracle, prefix sharded over 2 ranks:", stats)
    l = lse.cpu().numpy()
    assert max(abs(l[0, h, i] - rl[n]) for n, (h, i) in enumerate(rows)) <= 2e-2
    for sess in sessions:
        sess.close()
    del sessions, parts, wl
    torch.cuda.empty_cache()


def test_device_workload_redraws_the_same_bytes_and_a_second_instance_too():
    # The large workloads are never stored: every tensor is re-drawn from its seed when it is needed - by the session
    # that registers it, by the oracle that checks it, by the CPU baseline.  The digests a bench report carries are
    # only worth something if a re-draw gives the same bytes: same object twice, a second object, device against host.
    spec = gen.spec_config3(seed=5, n_layers=2, batch=2, pool=6, per_item=3, doc_len=300, q_len=16)
    a, b = gen.DeviceWorkload(spec, "cuda:0"), gen.DeviceWorkload(spec, "cuda:0")
    for pid in (0, 5):
        k0, v0 = a.packet_layer(pid, 1)
        k1, v1 = a.packet_layer(pid, 1)
        k2, v2 = b.packet_layer(pid, 1)
        kd, vd = a.packet_device(pid)
        assert gen.digest64(k0, v0) == gen.digest64(k1, v1) == gen.digest64(k2, v2)
        assert gen.digest64(k0) == gen.digest64(torch_to_np(kd[1], "bf16")) and gen.digest64(v0) == gen.digest64(torch_to_np(vd[1], "bf16"))
    assert gen.digest64(*a.query_layer(1)) == gen.digest64(*b.query_layer(1)) != gen.digest64(*a.query_layer(0))
    other = gen.DeviceWorkload(gen.spec_config3(seed=6, n_layers=2, batch=2, pool=6, per_item=3, doc_len=300, q_len=16), "cuda:0")
    assert gen.digest64(*other.packet_layer(0, 1)) != gen.digest64(*a.packet_layer(0, 1))
