"""GPU parity for compressed packets (Section 4.3): document caches pruned to a different token subset
per layer and kv head are composed as opaque units - one offset per packet, positions retained - and the
query attends over what each head still holds.  Compared with the fp64 oracle, which drops the pruned keys
from a plain attention per kv head."""
import numpy as np
import pytest

from oracle import reference as orc
from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from paper_2604_13226_b200.session import Session, torch_to_np
from helpers import oracle_outputs
from test_gpu_decode import check, run_chunks

pytestmark = pytest.mark.gpu


def compressed_small(dtype="bf16", d=128, keep=(0.5, None, 0.3, 0.02), q_len=40, per_head=True, seed=41, pairing=0):
    shape = gen.ModelShape(2, 8, 2, d, dtype, 500000.0, pairing)
    return gen.make_workload(shape, [300, 700, 129, 260], [[(0, 0), (1, 0), (2, -1)], [(3, 0), (0, 0)]], q_len=q_len,
                             n_header=16, n_trailer=16, seed=seed, packet_pos0=[0, 3, 0, 50], keep_rate=list(keep),
                             keep_per_head=per_head)


@pytest.mark.parametrize("per_head", [True, False])
@pytest.mark.parametrize("flags", [0, kvp.ROPE_QUERY, kvp.FORCE_SIMPLE])
def test_compressed_attention_bf16(per_head, flags):
    wl = compressed_small(per_head=per_head)
    # packet 3 keeps ~2 %: some heads hold a handful of keys, whole tiles of the layer's list are empty for them
    assert min(len(x) for row in wl.packets[3].kept for x in row) < 16
    sess = Session(wl)
    sess.assemble()
    for layer in range(wl.shape.n_layers):
        out, lse = sess.prefill(layer, flags)
        assert sess.ctx.status_word() == 0
        check(wl, out, lse, layer, rope_query=bool(flags & kvp.ROPE_QUERY))
    assert sess.ctx.last_launch()["kind"] == (0 if flags & kvp.FORCE_SIMPLE else 1)
    sess.close()


def test_compressed_fp32_and_interleaved_pairs():
    wl = compressed_small("f32", 64, pairing=1)
    sess = Session(wl)
    sess.assemble()
    out, lse = sess.prefill(1)
    check(wl, out, lse, 1, tol=(2e-5, 2e-6, 1e-4))
    sess.close()


def test_compressed_llama_shape_split_units_and_decode():
    # 32/8 heads, 4 x 1024-token documents pruned to ~50 % / ~25 %, 128 query tokens: two-tile units cut
    # into pieces whose tile lists differ per layer; then two decode steps over the same cache
    shape = gen.ModelShape(2, 32, 8, 128, "bf16", 500000.0, 0)
    wl = gen.make_workload(shape, [1024] * 4, [[(0, 0), (1, 0), (2, 0), (3, 0)]], q_len=130, seed=43,
                           keep_rate=[0.5, 0.25, None, 0.5])
    sess = Session(wl)
    sess.assemble()
    for layer in (1, 0):
        out, lse = run_chunks(wl, sess, [(0, 128), (128, 129), (129, 130)], layer)
        check(wl, out, lse, layer)
    ll = sess.ctx.last_launch()
    assert ll["kind"] == 1
    sess.close()


def test_compressed_unsupported_paths_and_validation():
    wl = compressed_small()
    sess = Session(wl)
    aid, plen = sess.assemble()
    assert plen == [wl.prefix_len(b) for b in range(wl.batch)]          # positions are retained
    q, kn, vn = sess.query_tensors(0)
    with pytest.raises(kvp.KvpError) as e:
        sess.ctx.export_cache(aid, 0, 0, plen[0], 0)
    assert e.value.code == 5
    with pytest.raises(kvp.KvpError) as e:
        sess.ctx.assemble(wl.items, kvp.REBASE | kvp.MATERIALIZE)
    assert e.value.code == 5
    sess.close()


def test_normal_mode_wrapped_packets_pruned_with_their_fillers():
    # Section 4.3, "KVPacket Normal": the compressor runs over the whole wrapped cache  header | document | trailer,
    # so filler tokens are pruned like any other.  A wrapped cache is registered as one packet (no separate
    # adapter): it is still an opaque unit with one offset.
    shape = gen.ModelShape(2, 8, 2, 128, "bf16", 500000.0, 0)
    L, nh, nt = 200, 16, 16
    base = gen.make_workload(shape, [L, L, L], [[(0, 0), (1, 0)], [(2, 0), (0, 0), (1, 0)]], q_len=24, n_header=nh, n_trailer=nt,
                             seed=47, packet_pos0=[nh, nh, nh], adapter_pos0=[(0, nh + L)])
    # (a) unpruned: the wrapped registration composes to the same sequence as packets + shared fillers
    wrapped = gen.wrap_workload(base)
    assert [p.n_tokens for p in wrapped.packets] == [nh + L + nt] * 5 and wrapped.adapters == []
    sess = Session(wrapped)
    _, plen = sess.assemble()
    assert plen == [base.prefix_len(b) for b in range(base.batch)]
    for layer in range(2):
        out, lse = sess.prefill(layer)
        check(base, out, lse, layer)                    # the oracle over the ORIGINAL registration
    sess.close()
    # (b) pruned as a whole, a different subset per layer and kv head; some units lose most of their fillers
    pruned = gen.wrap_workload(base, keep_rate=[0.5, 0.3, 0.6, None, 0.1], seed=48)
    filler = np.r_[0:nh, nh + L:nh + L + nt]
    assert any(len(np.intersect1d(k, filler)) < (nh + nt) // 2 for p in pruned.packets if p.kept for row in p.kept for k in row)
    sess = Session(pruned)
    sess.assemble()
    for layer in range(2):
        for flags in (0, kvp.FORCE_SIMPLE):
            out, lse = sess.prefill(layer, flags)
            assert sess.ctx.status_word() == 0
            check(pruned, out, lse, layer)
    sess.close()
