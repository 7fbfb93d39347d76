"""GPU parity of kvp_segment_mass: the probability mass a query row puts on each segment of the composed
request (header / document / trailer per slot, then the query block), against the fp64 oracle's plain
softmax summed per segment.  Tolerance: the kernel re-forms scores in fp32 against the bf16 kernel's LSE
(itself within 2e-2 of the oracle), so a mass can be off by a factor exp(2e-2): 2e-2 relative + 1e-5."""
import numpy as np
import pytest

from oracle import reference as orc
from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from paper_2604_13226_b200.session import Session
from helpers import make_store
from test_gpu_compressed import compressed_small

pytestmark = pytest.mark.gpu


def check_mass(wl, sess, layer, flags=0, rtol=2e-2):
    s = wl.shape
    q, kn, vn = sess.query_tensors(layer)
    out, lse = sess.prefill(layer, flags, qkv=(q, kn, vn))
    n_cols = max(len(it) for it in wl.items) * 3 + 2
    mass = sess.ctx.segment_mass(sess.assembly_id, layer, q, lse, wl.q_len, n_cols, flags).cpu().numpy().astype(np.float64)
    assert sess.ctx.status_word() == 0
    st = make_store(wl)
    f = orc.inv_freq(s.rope_theta, s.head_dim)
    hq, hk, _ = wl.query_layer(layer)
    for b in range(wl.batch):
        plan = orc.compose(st, wl.items[b], wl.rebase)
        ref = orc.segment_mass(st, plan, layer, hq[b], hk[b], f, s.rope_pairing, rope_query=bool(flags & kvp.ROPE_QUERY))
        ref = ref.reshape(wl.q_len, s.n_q_heads, -1)
        n_seg = plan.segments.shape[0]
        got = mass[b, :, :, :n_seg + 1]
        assert np.all(mass[b, :, :, n_seg + 1:] == 0.0)
        assert np.max(np.abs(got.sum(-1) - 1.0)) <= rtol
        assert np.all(np.abs(got - ref) <= rtol * ref + 1e-5), float(np.max(np.abs(got - ref)))


def ragged(dtype="bf16", d=128, pairing=0):
    shape = gen.ModelShape(2, 8, 2, d, dtype, 500000.0, pairing)
    return gen.make_workload(shape, [200, 37, 300, 129], [[(0, 0), (2, 0), (1, -1)], [(3, 0), (0, 0)]], q_len=24,
                             n_header=16, n_trailer=16, seed=51, packet_pos0=[0, 3, 0, 1000])


@pytest.mark.parametrize("flags", [0, kvp.ROPE_QUERY])
def test_segment_mass_bf16(flags):
    wl = ragged()
    sess = Session(wl)
    sess.assemble()
    for layer in range(2):
        check_mass(wl, sess, layer, flags)
    sess.close()


def test_segment_mass_fp32_interleaved_and_config1():
    for wl in (ragged("f32", 64, 1), gen.config1()):
        sess = Session(wl)
        sess.assemble()
        check_mass(wl, sess, 0, rtol=1e-3)
        sess.close()


def test_segment_mass_compressed_packets():
    wl = compressed_small(q_len=16)
    sess = Session(wl)
    sess.assemble()
    check_mass(wl, sess, 1)
    sess.close()


def test_segment_mass_argument_checks():
    wl = ragged()
    sess = Session(wl)
    sess.assemble()
    q, kn, vn = sess.query_tensors(0)
    import torch
    lse = torch.zeros((2, 8, 24), dtype=torch.float32, device=q.device)
    with pytest.raises(kvp.KvpError) as e:                      # no prefill yet for this layer
        sess.ctx.segment_mass(sess.assembly_id, 0, q, lse, 24, 12)
    assert e.value.code == 4
    sess.prefill(0, qkv=(q, kn, vn))
    with pytest.raises(kvp.KvpError) as e:                      # 7 segments + the query block do not fit 7 columns
        sess.ctx.segment_mass(sess.assembly_id, 0, q, lse, 24, 7)
    assert e.value.code == 2
    sess.close()
