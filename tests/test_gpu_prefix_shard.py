"""GPU parity of prefix sharding: the packets of a request spread over several ranks, every rank attending
to the keys it holds (`kvp_assemble_at`, `KVP_PARTIAL`), one exchange of the partial results, one merge
(`kvp_merge_partials`).  One GPU plays the ranks one after the other - a context per rank, holding only that
rank's packets - and the exchange is a concatenation of the ranks' buffers, which is what an all-gather delivers.
The oracle is the plain definition over the WHOLE request (Section 3.2 step 4): softmax attention over a union
of key sets equals the log-sum-exp merge of the attention over each set."""
import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from paper_2604_13226_b200.session import Session, torch_to_np
from helpers import attention_error_stats, make_store, oracle_outputs

pytestmark = pytest.mark.gpu


def run_sharded(wl, world, query_rank=None, flags=0):
    """Returns (out, lse) merged over `world` ranks; the query's own keys are attended to on `query_rank`."""
    query_rank = world - 1 if query_rank is None else query_rank
    parts, sessions = [], []
    for r in range(world):
        sub, pos_base = gen.shard_workload(wl, r, world)
        sess = Session(sub)
        aid, plen = sess.assemble(pos_base=pos_base)
        assert plen == [sub.prefix_len(b) for b in range(sub.batch)]
        q, kn, vn = sess.query_tensors(0)
        buf = torch.full((sess.ctx.partial_bytes(wl.batch, wl.q_len),), 0x7f, dtype=torch.uint8, device=q.device)
        f = flags | kvp.PARTIAL | (0 if r == query_rank else kvp.SKIP_QUERY_BLOCK)
        sess.ctx.query_prefill(aid, 0, q, kn, vn, wl.q_len, buf, None, f)
        assert sess.ctx.status_word() == 0
        parts.append(buf)
        sessions.append(sess)
    gathered = torch.cat(parts)                                   # [world][partial_bytes]: the all-gather's result
    s = wl.shape
    out = torch.zeros(wl.batch, wl.q_len, s.n_q_heads, s.head_dim, dtype=torch.bfloat16, device=gathered.device)
    lse = torch.zeros(wl.batch, s.n_q_heads, wl.q_len, dtype=torch.float32, device=gathered.device)
    sessions[0].ctx.merge_partials(gathered, world, wl.batch, wl.q_len, out, lse)
    torch.cuda.synchronize()
    for sess in sessions:
        sess.close()
    return out, lse


def check_against_whole_request(wl, out, lse):
    s = wl.shape
    o = orc.widen(torch_to_np(out, "bf16"), "bf16")
    l = lse.cpu().numpy().astype(np.float64)
    ref = oracle_outputs(wl, 0)
    for b in range(wl.batch):
        ro = ref[b][0].reshape(wl.q_len, s.n_q_heads, s.head_dim)
        rl = ref[b][1].reshape(wl.q_len, s.n_q_heads).T
        attention_error_stats(o[b], ro)
        assert np.max(np.abs(l[b] - rl)) <= 2e-2


def workload(q_len, seed, lens=(300, 1024, 129, 640, 77, 512), items=None, n_q=8, n_kv=2):
    shape = gen.ModelShape(1, n_q, n_kv, 128, "bf16", 500000.0, 0)
    items = items or [[(0, 0), (1, 0), (2, -1), (3, 0), (4, 0), (5, 0)], [(5, 0), (3, 0), (0, 0)]]
    return gen.make_workload(shape, list(lens), items, q_len=q_len, seed=seed, packet_pos0=[0, 3, 0, 1000, 5, 0][:len(lens)])


@pytest.mark.parametrize("world,q_len", [(2, 40), (2, 1), (3, 70), (4, 16)])
def test_two_to_four_ranks_match_the_oracle_over_the_whole_request(world, q_len):
    wl = workload(q_len, seed=40 + world)
    out, lse = run_sharded(wl, world)
    check_against_whole_request(wl, out, lse)


def test_query_block_on_the_first_rank_and_a_rank_without_keys():
    # request 1 has three slots over four ranks: one rank holds nothing of it and hands in an empty partial;
    # which rank takes the query's own keys does not matter
    wl = workload(33, seed=51)
    for query_rank in (0, 2):
        out, lse = run_sharded(wl, 4, query_rank=query_rank)
        check_against_whole_request(wl, out, lse)


def test_one_rank_partial_plus_merge_equals_the_plain_prefill_and_precise_mode():
    wl = workload(48, seed=52, n_q=28, n_kv=4)                   # g = 7
    out, lse = run_sharded(wl, 1)
    check_against_whole_request(wl, out, lse)
    sess = Session(wl)
    sess.assemble()
    ref, ref_lse = sess.prefill(0)
    assert float((out.float() - ref.float()).abs().max()) <= 2.0 ** -7 and float((lse - ref_lse).abs().max()) <= 1e-4
    sess.close()
    out, lse = run_sharded(wl, 2, flags=kvp.PRECISE_QK)
    check_against_whole_request(wl, out, lse)


def test_partial_flag_misuse_is_refused():
    wl = workload(8, seed=53)
    sub, pos_base = gen.shard_workload(wl, 1, 2)
    sess = Session(sub)
    aid, _ = sess.assemble(pos_base=pos_base)
    q, kn, vn = sess.query_tensors(0)
    buf = torch.empty(sess.ctx.partial_bytes(wl.batch, wl.q_len), dtype=torch.uint8, device=q.device)
    for flags, code in ((kvp.SKIP_QUERY_BLOCK, 1), (kvp.PARTIAL | kvp.CONTINUE, 5), (kvp.PARTIAL | kvp.FORCE_SIMPLE, 5),
                        (kvp.ROPE_QUERY, 5)):
        with pytest.raises(kvp.KvpError) as e:
            sess.ctx.query_prefill(aid, 0, q, kn, vn, wl.q_len, buf, None, flags)
        assert e.value.code == code
    with pytest.raises(kvp.KvpError) as e:
        sess.ctx.assemble(sub.items, kvp.REBASE, pos_base=[-1] * sub.batch)
    assert e.value.code == 1
    sess.close()
