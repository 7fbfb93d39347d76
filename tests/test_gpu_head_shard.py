"""GPU parity of kv-head sharding: rank r holds kv heads [r Hkv / N, (r + 1) Hkv / N) of every packet and adapter
and the query heads that read them; there is no exchange inside the path, a rank's output is its heads' slice of the
output.  One GPU plays the ranks one after the other, a context per rank holding only that rank's heads.  The oracle
is the plain definition over the WHOLE workload (Section 3.2 step 4): attention is computed per query head over the
keys of its kv head (grouped-query mapping: kv head = query head // g), so the slices put side by side along the head
axis must be the whole result."""
import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from paper_2604_13226_b200.session import Session, torch_to_np
from helpers import attention_error_stats, oracle_outputs

pytestmark = pytest.mark.gpu


def run_head_sharded(wl, world, layer=0, flags=0):
    outs, lses = [], []
    for r in range(world):
        sub = gen.shard_heads(wl, r, world)
        sess = Session(sub)
        sess.assemble()
        out, lse = sess.prefill(layer, flags)
        assert sess.ctx.status_word() == 0
        outs.append(out.clone())
        lses.append(lse.clone())
        sess.close()
    return torch.cat(outs, dim=2), torch.cat(lses, dim=1)          # [b][q_len][Hq][d], [b][Hq][q_len]


def check_against_whole_workload(wl, out, lse, layer=0):
    s = wl.shape
    o = orc.widen(torch_to_np(out, s.dtype), s.dtype)
    l = lse.cpu().numpy().astype(np.float64)
    ref = oracle_outputs(wl, layer)
    for b in range(wl.batch):
        ro = ref[b][0].reshape(wl.q_len, s.n_q_heads, s.head_dim)
        rl = ref[b][1].reshape(wl.q_len, s.n_q_heads).T
        attention_error_stats(o[b], ro)
        assert np.max(np.abs(l[b] - rl)) <= 2e-2


@pytest.mark.parametrize("world,n_q,n_kv,q_len", [(2, 8, 2, 40), (4, 32, 8, 16), (2, 28, 4, 70), (8, 32, 8, 1)])
def test_head_sharded_ranks_match_the_oracle_over_all_heads(world, n_q, n_kv, q_len):
    shape = gen.ModelShape(2, n_q, n_kv, 128, "bf16", 500000.0, 0)
    items = [[(0, 0), (1, 0), (2, -1), (3, 0)], [(3, 0), (0, 0)]]
    wl = gen.make_workload(shape, [300, 1024, 129, 640], items, q_len=q_len, seed=70 + world, packet_pos0=[0, 3, 0, 1000])
    for layer in (0, 1):
        out, lse = run_head_sharded(wl, world, layer)
        check_against_whole_workload(wl, out, lse, layer)


def test_head_sharded_compressed_packets_keep_each_heads_own_tokens():
    # pruned packets hold a different token subset per (layer, kv head): a rank takes its heads' subsets with it
    shape = gen.ModelShape(1, 8, 4, 128, "bf16", 500000.0, 0)
    wl = gen.make_workload(shape, [700, 300, 512], [[(0, 0), (1, 0), (2, 0)]], q_len=24, seed=77, keep_rate=[0.4, None, 0.7])
    out, lse = run_head_sharded(wl, 2)
    check_against_whole_workload(wl, out, lse)


def test_one_rank_is_the_unsharded_call_bit_for_bit():
    shape = gen.ModelShape(1, 8, 2, 128, "bf16", 500000.0, 0)
    wl = gen.make_workload(shape, [300, 640], [[(0, 0), (1, 0)]], q_len=32, seed=79)
    out, lse = run_head_sharded(wl, 1)
    sess = Session(wl)
    sess.assemble()
    ref_out, ref_lse = sess.prefill(0)
    assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)
    sess.close()
