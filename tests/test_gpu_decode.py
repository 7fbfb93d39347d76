"""GPU parity of KVP_CONTINUE: the step after the prefill (decoding, one token at a time) and a prefill
fed in chunks.  The oracle is the plain definition - causal attention of the whole query block over
[prefix | query] (Section 3.2 step 4) - so feeding the same tokens in several calls must reproduce its
rows: token i of a later call sees the prefix, every row appended before, and its own call's tokens <= i."""
import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from paper_2604_13226_b200.session import Session, torch_to_np
from helpers import attention_error_stats, oracle_outputs

pytestmark = pytest.mark.gpu


def run_chunks(wl, sess, chunks, layer=0, flags=0):
    """Feed query tokens [a, b) per chunk; returns out [B][Lq][Hq][d] and lse [B][Hq][Lq] assembled from the calls."""
    q, kn, vn = sess.query_tensors(layer)
    outs, lses = [], []
    for n, (a, b) in enumerate(chunks):
        o, l = sess.prefill(layer, flags | (kvp.CONTINUE if n > 0 else 0),
                            qkv=(q[:, a:b].contiguous(), kn[:, a:b].contiguous(), vn[:, a:b].contiguous()))
        outs.append(o)
        lses.append(l)
    assert sess.ctx.status_word() == 0
    return torch.cat(outs, dim=1), torch.cat(lses, dim=2)


def check(wl, out, lse, layer=0, rope_query=False, tol=(2e-2, 2e-3, 2e-2)):
    s = wl.shape
    o = orc.widen(torch_to_np(out, s.dtype), s.dtype)
    lse = lse.cpu().numpy().astype(np.float64)
    ref = oracle_outputs(wl, layer, rope_query=rope_query)
    for b in range(wl.batch):
        ro = ref[b][0].reshape(wl.q_len, s.n_q_heads, s.head_dim)
        rl = ref[b][1].reshape(wl.q_len, s.n_q_heads).T
        err = np.abs(o[b] - ro)
        if s.dtype == "bf16":
            attention_error_stats(o[b], ro)                  # raw 2e-2 / 2e-3
        else:
            assert err.max() <= tol[0] and err.mean() <= tol[1], (b, err.max(), err.mean())
        assert np.max(np.abs(lse[b] - rl)) <= tol[2]


def small(dtype="bf16", q_len=40, seed=31):
    shape = gen.ModelShape(2, 8, 2, 128, dtype, 500000.0, 0)
    return gen.make_workload(shape, [200, 37, 300, 129], [[(0, 0), (2, 0), (1, -1)], [(3, 0), (0, 0)]], q_len=q_len,
                             n_header=16, n_trailer=16, seed=seed, packet_pos0=[0, 3, 0, 1000])


@pytest.mark.parametrize("chunks", [[(0, 17), (17, 40)], [(0, 37), (37, 38), (38, 39), (39, 40)], [(0, 1), (1, 2), (2, 40)]])
@pytest.mark.parametrize("rope_query", [False, True])
def test_chunked_prefill_and_decode_steps_bf16(chunks, rope_query):
    wl = small()
    sess = Session(wl)
    sess.assemble()
    for layer in range(wl.shape.n_layers):
        out, lse = run_chunks(wl, sess, chunks, layer, kvp.ROPE_QUERY if rope_query else 0)
        check(wl, out, lse, layer, rope_query)
    # the cache holds every appended row, in order
    k, v = sess.ctx.export_cache(sess.assembly_id, 1, 0, sess.prefix_len[0], wl.q_len)
    if not rope_query:
        assert np.array_equal(torch_to_np(k, "bf16")[sess.prefix_len[0]:], wl.k_new[1][0])
    assert np.array_equal(torch_to_np(v, "bf16")[sess.prefix_len[0]:], wl.v_new[1][0])
    sess.close()


def test_continue_across_tail_tiles_group7():
    # g = 7, 300 query tokens in three calls: the appended rows span three 128-key tiles, and the later
    # calls' causal limits fall inside tiles written by earlier calls
    shape = gen.ModelShape(1, 28, 4, 128, "bf16", 1000000.0, 0)
    wl = gen.make_workload(shape, [256, 700, 333], [[(0, 0), (1, 0)], [(2, 0), (0, 0)]], q_len=300, seed=33)
    sess = Session(wl)
    sess.assemble()
    for flags in (0, kvp.PRECISE_QK):              # the second: value + remainder query tiles behind the append kernel
        out, lse = run_chunks(wl, sess, [(0, 130), (130, 257), (257, 300)], flags=flags)
        check(wl, out, lse)
    sess.close()


def test_decode_steps_fp32_kernel_and_forced_simple():
    wl = gen.config1()
    sess = Session(wl)
    sess.assemble()
    out, lse = run_chunks(wl, sess, [(0, 29), (29, 30), (30, 31), (31, 32)])
    check(wl, out, lse, tol=(2e-5, 2e-6, 1e-4))
    sess.close()
    wl = small()
    sess = Session(wl)
    sess.assemble()
    out, lse = run_chunks(wl, sess, [(0, 39), (39, 40)], flags=kvp.FORCE_SIMPLE)
    check(wl, out, lse)
    sess.close()


def test_continue_capacity_and_restart():
    wl = small()
    sess = Session(wl)
    sess.assemble()
    q, kn, vn = sess.query_tensors(0)
    sess.prefill(0, qkv=(q, kn, vn))
    with pytest.raises(kvp.KvpError) as e:                 # 40 rows are there; one more does not fit
        sess.prefill(0, kvp.CONTINUE, qkv=(q[:, :1].contiguous(), kn[:, :1].contiguous(), vn[:, :1].contiguous()))
    assert e.value.code == 2
    out, lse = sess.prefill(0, qkv=(q, kn, vn))            # without the flag the layer starts again at the prefix
    check(wl, out, lse)
    sess.close()
