"""Packets that wait in host memory (Section 4.3 counts the CPU-to-GPU cache transfer inside time-to-first-token):
registered with kvp_register_packet_host they reach the pool at the first assemble that names them, layer by layer
on the context's own stream, and each layer's attention waits for its own layer only.  The arithmetic is the same
path as for device-registered packets: outputs must be bit-identical to it, and within tolerance of the oracle."""
import numpy as np
import pytest
import torch

from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from paper_2604_13226_b200.session import Session, torch_to_np
from test_gpu_parity import check_attention, ragged_small

pytestmark = pytest.mark.gpu


def all_layers(sess, wl):
    outs = []
    for layer in range(wl.shape.n_layers):
        out, lse = sess.prefill(layer)
        outs.append((out.clone(), lse.clone()))
    torch.cuda.synchronize()
    assert sess.ctx.status_word() == 0
    return outs


@pytest.mark.parametrize("maker", [ragged_small, gen.config2])
def test_host_packets_give_the_device_path_results(maker):
    wl = maker()
    dev = Session(wl)
    dev.assemble()
    want = all_layers(dev, wl)
    dev.close()
    host = Session(wl, host_packets=True)
    aid, plen = host.assemble()
    got = all_layers(host, wl)
    for (o0, l0), (o1, l1) in zip(want, got):
        assert torch.equal(o0, o1) and torch.equal(l0, l1)
    for layer in range(wl.shape.n_layers):                    # and against the oracle
        check_attention(wl, host, layer=layer)
    # a second assembly of the now resident packets, and one after eviction, give the same again
    host.assemble()
    again = all_layers(host, wl)
    for pid in range(len(wl.packets)):
        host.ctx.evict_packet(pid)
    host.assemble()
    back = all_layers(host, wl)
    for (o0, l0), (o1, l1), (o2, l2) in zip(want, again, back):
        assert torch.equal(o0, o1) and torch.equal(o0, o2) and torch.equal(l0, l2)
    host.close()


def test_host_packets_materialised_cache_bytes():
    # the gather of a materialised assembly reads every layer of the documents: it waits for the last layer's load
    wl = ragged_small()
    dev = Session(wl, materialize=True)
    aid, plen = dev.assemble()
    want = [dev.ctx.export_cache(aid, l, b, plen[b], 0) for l in range(wl.shape.n_layers) for b in range(wl.batch)]
    host = Session(wl, materialize=True, host_packets=True)
    aid2, plen2 = host.assemble()
    assert plen2 == plen
    got = [host.ctx.export_cache(aid2, l, b, plen[b], 0) for l in range(wl.shape.n_layers) for b in range(wl.batch)]
    for (k0, v0), (k1, v1) in zip(want, got):
        assert torch.equal(k0, k1) and torch.equal(v0, v1)
    dev.close()
    host.close()


def test_evict_needs_a_host_copy():
    wl = ragged_small()
    sess = Session(wl)
    with pytest.raises(kvp.KvpError):
        sess.ctx.evict_packet(0)                               # registered from device memory: nothing to come back from
    with pytest.raises(kvp.KvpError):
        sess.ctx.evict_packet(99)
    sess.close()
