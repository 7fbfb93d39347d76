"""Seeded random workloads (head counts, document lengths, batch composition, query length, adapters or none,
CTA count of the work list): the tcgen05 kernel against the CUDA-core kernel on every row, and against the oracle
on the first request, plus one chunked continuation.  Sizes stay small: the point is the odd corners of the tile
numbering, the work-list cuts and the per-request masks, not throughput."""
import numpy as np
import pytest
import torch

from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from paper_2604_13226_b200.session import Session
from test_gpu_parity import check_attention

pytestmark = pytest.mark.gpu


def random_workload(seed):
    rng = np.random.default_rng(1000 + seed)
    n_kv = int(rng.choice([1, 2, 4]))
    group = int(rng.choice([1, 2, 4, 7, 8]))
    shape = gen.ModelShape(1, n_kv * group, n_kv, 128, "bf16", 500000.0, int(rng.integers(0, 2)))
    n_packets = int(rng.integers(1, 6))
    lens = [int(rng.choice([1, 17, 127, 128, 129, 300, 511, 1024])) for _ in range(n_packets)]
    batch = int(rng.integers(1, 4))
    items = []
    for _ in range(batch):
        n = int(rng.integers(0, 4))
        items.append([(int(rng.integers(0, n_packets)), int(rng.choice([0, 0, -1]))) for _ in range(n)])
    if all(len(it) == 0 for it in items):
        items[0] = [(0, 0)]
    q_len = int(rng.choice([1, 2, 15, 16, 33, 64, 100, 129, 260]))
    n_h, n_t = (16, 16) if rng.integers(0, 3) else (int(rng.integers(0, 5)), int(rng.integers(0, 40)))
    wl = gen.make_workload(shape, lens, items, q_len=q_len, n_header=n_h, n_trailer=n_t, seed=seed)
    return wl, int(rng.choice([0, 0, 1, 3, 17, 148]))


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_tensor_kernel_against_cuda_core_kernel_and_oracle(seed):
    wl, ctas = random_workload(seed)
    sess = Session(wl)
    sess.assemble()
    if ctas:
        sess.ctx.tune(kvp.TUNE_SPLIT_TARGET_CTAS, ctas)
    qkv = sess.query_tensors(0)
    out, lse = sess.prefill(0, qkv=qkv)
    assert sess.ctx.status_word() == 0 and sess.ctx.last_launch()["kind"] == 1
    ref, ref_lse = sess.prefill(0, kvp.FORCE_SIMPLE, qkv=qkv)
    d = (out.float() - ref.float()).abs()
    assert float(d.max()) <= 3e-2 and float(d.mean()) <= 2e-3, (seed, float(d.max()), float(d.mean()))
    assert float((lse - ref_lse).abs().max()) <= 2e-2
    check_attention(wl, sess)                                   # and the oracle, all requests
    sess.close()


@pytest.mark.parametrize("seed", [3, 8, 13, 21])
def test_random_shapes_chunked_continuation(seed):
    # the same query block in two calls (KVP_CONTINUE): the rows of both calls together equal the one-call result
    wl, ctas = random_workload(seed)
    if wl.q_len < 2:
        pytest.skip("one token cannot be split")
    sess = Session(wl)
    sess.assemble()
    q, kn, vn = sess.query_tensors(0)
    whole, _ = sess.prefill(0, qkv=(q, kn, vn))
    cut = wl.q_len // 2
    sess.assemble()
    outs = []
    for lo, hi, fl in ((0, cut, 0), (cut, wl.q_len, kvp.CONTINUE)):
        qq, kk, vv = (t[:, lo:hi].contiguous() for t in (q, kn, vn))
        o = torch.empty_like(qq)
        sess.ctx.query_prefill(sess.assembly_id, 0, qq, kk, vv, hi - lo, o, None, fl)
        outs.append(o)
    torch.cuda.synchronize()
    assert sess.ctx.status_word() == 0
    both = torch.cat(outs, dim=1)
    d = (both.float() - whole.float()).abs()
    assert float(d.max()) <= 3e-2 and float(d.mean()) <= 2e-3
    sess.close()


def random_large_workload(seed):
    rng = np.random.default_rng(5000 + seed)
    n_kv = int(rng.choice([1, 2, 4, 8]))
    group = int(rng.choice([1, 4, 7, 8]))
    shape = gen.ModelShape(1, n_kv * group, n_kv, 128, "bf16", 500000.0, int(rng.integers(0, 2)))
    n_packets = int(rng.integers(1, 9))
    lens = [int(rng.choice([1, 64, 129, 700, 1024, 2048, 3000])) for _ in range(n_packets)]
    batch = int(rng.integers(1, 5))
    items = [[(int(rng.integers(0, n_packets)), int(rng.choice([0, 0, -1]))) for _ in range(int(rng.integers(0, 7)))]
             for _ in range(batch)]
    if all(len(it) == 0 for it in items):
        items[0] = [(0, 0)]
    q_len = int(rng.choice([5, 128, 300, 512, 777, 1024]))
    keep = None
    if rng.integers(0, 4) == 0:                                 # a quarter of the cases with pruned packets
        keep = [float(rng.choice([0.1, 0.5, 0.9])) if rng.integers(0, 2) else None for _ in range(n_packets)]
    wl = gen.make_workload(shape, lens, items, q_len=q_len, seed=seed, keep_rate=keep)
    cuts = sorted(set([0, q_len] + [int(x) for x in rng.integers(1, q_len, size=2)]))
    return wl, int(rng.choice([0, 0, 5, 60, 148])), keep is not None, cuts


@pytest.mark.parametrize("seed", range(16))
def test_random_large_shapes_long_queries_pruned_packets_and_three_chunk_continuation(seed):
    # Longer queries (many query tiles per kv head, several causal tiles), longer and pruned documents, up to 8 kv
    # heads: the tcgen05 kernel against the CUDA-core kernel on every row (the oracle would take minutes here; the
    # CUDA-core kernel is checked against it on the small cases above), then the same query in three calls.
    wl, ctas, pruned, cuts = random_large_workload(seed)
    sess = Session(wl)
    if ctas:
        sess.ctx.tune(kvp.TUNE_SPLIT_TARGET_CTAS, ctas)
    sess.assemble()
    q, kn, vn = sess.query_tensors(0)
    out, lse = sess.prefill(0, qkv=(q, kn, vn))
    assert sess.ctx.status_word() == 0 and sess.ctx.last_launch()["kind"] == 1
    ref, ref_lse = sess.prefill(0, kvp.FORCE_SIMPLE, qkv=(q, kn, vn))
    d = (out.float() - ref.float()).abs()
    assert float(d.max()) <= 3e-2 and float(d.mean()) <= 2e-3, (seed, float(d.max()), float(d.mean()))
    assert float((lse - ref_lse).abs().max()) <= 2e-2
    if not pruned:
        sess.assemble()
        outs = []
        for i in range(len(cuts) - 1):
            a, b = cuts[i], cuts[i + 1]
            qq, kk, vv = (t[:, a:b].contiguous() for t in (q, kn, vn))
            o = torch.empty_like(qq)
            sess.ctx.query_prefill(sess.assembly_id, 0, qq, kk, vv, b - a, o, None, kvp.CONTINUE if i else 0)
            outs.append(o)
        torch.cuda.synchronize()
        assert sess.ctx.status_word() == 0
        d = (torch.cat(outs, dim=1).float() - ref.float()).abs()
        assert float(d.max()) <= 3e-2 and float(d.mean()) <= 2e-3, (seed, cuts, float(d.max()), float(d.mean()))
    sess.close()
