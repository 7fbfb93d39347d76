"""Requests of one batch with query chunks of different lengths (kvp_query_prefill_ragged): every request's rows
against the oracle run on that request's own tokens; rows beyond a request's length stay untouched."""
import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from paper_2604_13226_b200.session import Session, torch_to_np
from helpers import make_store

pytestmark = pytest.mark.gpu

BF16_MAX_ABS, BF16_MEAN_ABS = 2e-2, 2e-3


def run_ragged(wl, q_lens, layer=0, split_ctas=0):
    sess = Session(wl)
    sess.assemble()
    if split_ctas:
        sess.ctx.tune(kvp.TUNE_SPLIT_TARGET_CTAS, split_ctas)
    q, kn, vn = sess.query_tensors(layer)
    out = torch.full_like(q, 7.0)                                # sentinel: padded rows must keep it
    lse = torch.full((q.shape[0], wl.shape.n_q_heads, q.shape[1]), -5.0, dtype=torch.float32, device=q.device)
    sess.ctx.query_prefill_ragged(sess.assembly_id, layer, q, kn, vn, wl.q_len, q_lens, out, lse)
    torch.cuda.synchronize()
    assert sess.ctx.status_word() == 0
    s = wl.shape
    o = orc.widen(torch_to_np(out, s.dtype), s.dtype)           # [B][Lq][Hq][d]
    l = lse.cpu().numpy().astype(np.float64)                     # [B][Hq][Lq]
    st = make_store(wl)
    f = orc.inv_freq(s.rope_theta, s.head_dim)
    hq, hk, hv = wl.query_layer(layer)
    for b, slots in enumerate(wl.items):
        n = q_lens[b]
        plan = orc.compose(st, slots, wl.rebase)
        ro, rl, K, V = orc.query_prefill(st, plan, layer, hq[b][:n], hk[b][:n], hv[b][:n], f, s.rope_pairing)
        ro = ro.reshape(n, s.n_q_heads, s.head_dim)
        rl = rl.reshape(n, s.n_q_heads).T
        err = np.abs(o[b, :n] - ro)
        assert err.max() <= BF16_MAX_ABS and err.mean() <= BF16_MEAN_ABS, (b, err.max(), err.mean())
        assert np.max(np.abs(l[b][:, :n] - rl)) <= 2e-2
        assert np.all(o[b, n:] == 7.0) and np.all(l[b][:, n:] == -5.0)          # nothing written past the request's length
    # the rows behind the prefixes now differ in number per request: exporting them is refused
    for b in range(wl.batch):
        with pytest.raises(kvp.KvpError):
            sess.ctx.export_cache(sess.assembly_id, layer, b, sess.prefix_len[b], 1)
    sess.close()


def ragged_wl(q_len, seed=11, n_layers=1):
    shape = gen.ModelShape(n_layers, 8, 2, 128, "bf16", 500000.0, 0)
    lens = [200, 37, 300, 129, 512]
    items = [[(0, 0), (2, 0)], [(3, 0), (0, 0), (1, -1)], [(4, 0)], [(1, 0), (2, 0)]]
    return gen.make_workload(shape, lens, items, q_len=q_len, n_header=16, n_trailer=16, seed=seed)


@pytest.mark.parametrize("q_lens", [[150, 37, 1, 200], [200, 200, 200, 200], [1, 1, 2, 3], [129, 64, 65, 33]])
def test_ragged_query_lengths_against_the_oracle(q_lens):
    run_ragged(ragged_wl(200), q_lens)


def test_ragged_query_lengths_with_split_units():
    run_ragged(ragged_wl(200), [150, 37, 1, 200], split_ctas=148)
    run_ragged(ragged_wl(200), [150, 37, 1, 200], split_ctas=3)


def test_ragged_rejects_bad_lengths_and_other_paths():
    wl = ragged_wl(64)
    sess = Session(wl)
    sess.assemble()
    q, kn, vn = sess.query_tensors(0)
    out = torch.empty_like(q)
    for bad in ([0, 1, 1, 1], [65, 1, 1, 1]):
        with pytest.raises(kvp.KvpError):
            sess.ctx.query_prefill_ragged(sess.assembly_id, 0, q, kn, vn, 64, bad, out)
    sess.ctx.tune(kvp.TUNE_FUSED_APPEND, 0)
    with pytest.raises(kvp.KvpError):
        sess.ctx.query_prefill_ragged(sess.assembly_id, 0, q, kn, vn, 64, [64, 3, 2, 1], out)
    sess.close()
