"""The allocation-free gather entry point against the regular one.

`kvp_compose_noalloc` serves callers that can neither hand the library a workspace nor tolerate an
allocation inside it (a frozen device heap, a plugin without an allocator): its scratch is a fixed
device array inside the library.  Here it is called through the C ABI twice in a row - two requests of
different size, so the second call finds the first call's records in the array - and each result is
compared with what `kvp_assemble(KVP_MATERIALIZE)` + `kvp_export_cache` give for the same request and
with the fp64 oracle's composed cache: values bit-exact, re-based keys within the stored-dtype
tolerance the other GPU tests use.  Both pair layouts and both head sizes run (they take different
branches and thread geometries in the kernel)."""
import numpy as np
import pytest

from oracle import reference as orc
from paper_2604_13226_b200 import binding as kvp
from paper_2604_13226_b200 import inputs as gen
from paper_2604_13226_b200.session import Session, torch_to_np
from helpers import make_store

pytestmark = pytest.mark.gpu


def pair_rel_err(k_gpu, k_ref, pairing=0):
    d = k_ref.shape[-1]
    if pairing == 0:
        a, b, ga, gb = k_ref[..., : d // 2], k_ref[..., d // 2:], k_gpu[..., : d // 2], k_gpu[..., d // 2:]
    else:
        a, b, ga, gb = k_ref[..., 0::2], k_ref[..., 1::2], k_gpu[..., 0::2], k_gpu[..., 1::2]
    nrm = np.sqrt(a * a + b * b)
    return float(np.max(np.maximum(np.abs(ga - a), np.abs(gb - b)) / np.maximum(nrm, 1e-30)))


@pytest.mark.parametrize("dtype,head_dim,pairing", [("bf16", 128, 0), ("f32", 128, 0), ("bf16", 64, 1), ("f32", 64, 0),
                                                    ("bf16", 128, 1), ("f32", 128, 1)])
def test_noalloc_gather_matches_assemble_twice_in_a_row(dtype, head_dim, pairing):
    import torch
    shape = gen.ModelShape(2, 8, 2, head_dim, dtype, 500000.0, pairing)
    lens = [200, 37, 300, 129]
    items = [[(0, 0), (2, 0), (1, -1)], [(3, 0), (0, 0)]]
    wl = gen.make_workload(shape, lens, items, q_len=8, n_header=16, n_trailer=16, seed=21, packet_pos0=[0, 3, 0, 1000])
    sess = Session(wl, materialize=True)
    aid, plen = sess.assemble()
    ctx = sess.ctx
    n_planes = shape.n_layers * shape.n_kv_heads
    pool_rows = ctx.cfg.pool_bytes // ctx.token_bytes
    pool_k = ctx.cfg.pool
    pool_v = pool_k + n_planes * pool_rows * shape.head_dim * shape.elem_bytes
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    store = make_store(wl)
    f = orc.inv_freq(shape.rope_theta, shape.head_dim)
    tol = 1e-4 if dtype == "f32" else 2.0 ** -8
    for b in range(wl.batch):                                   # two calls in a row sharing the scratch array
        _, _, segs = ctx.export_plan(aid, b)
        P = plen[b]
        ck = torch.full((n_planes, P, shape.head_dim), 7.0, dtype=tdt, device=sess.device)
        cv = torch.full((n_planes, P, shape.head_dim), 7.0, dtype=tdt, device=sess.device)
        kvp.compose_noalloc(pool_k, pool_v, pool_rows, n_planes, shape.head_dim, dtype, pairing, shape.rope_theta,
                            [(int(s[0]), int(s[1]), int(s[3])) for s in segs], ck, cv, P,
                            stream=torch.cuda.current_stream())
        torch.cuda.synchronize()
        for layer in range(shape.n_layers):
            k_ref, v_ref = ctx.export_cache(aid, layer, b, P, 0)          # [P][Hkv][d] from the regular entry point
            sl = slice(layer * shape.n_kv_heads, (layer + 1) * shape.n_kv_heads)
            k_new = ck[sl].permute(1, 0, 2).contiguous()
            v_new = cv[sl].permute(1, 0, 2).contiguous()
            assert torch.equal(v_new, v_ref)
            kn = orc.widen(torch_to_np(k_new, dtype), dtype)
            kr = orc.widen(torch_to_np(k_ref, dtype), dtype)
            assert pair_rel_err(kn, kr, pairing) <= tol
            # and against the oracle's composition itself (Eq. 1 on every key of the concatenated sequence)
            ko, vo, _ = orc.composed_kv(store, orc.compose(store, wl.items[b]), layer, f, pairing)
            assert np.array_equal(orc.widen(torch_to_np(v_new, dtype), dtype), vo)
            assert pair_rel_err(kn, ko, pairing) <= tol
    assert ctx.status_word() == 0
    sess.close()


def test_noalloc_rejects_too_many_segments_and_bad_arguments():
    import torch
    buf = torch.zeros(4 * 64 * 128, dtype=torch.bfloat16, device="cuda:0")
    segs = [(0, 1, 0)] * (97)
    with pytest.raises(kvp.KvpError) as e:
        kvp.compose_noalloc(buf.data_ptr(), buf.data_ptr(), 64, 4, 128, "bf16", 0, 10000.0, segs, buf, buf, 128)
    assert e.value.code == 2 and "96" in str(e.value)
    with pytest.raises(kvp.KvpError) as e:
        kvp.compose_noalloc(buf.data_ptr(), buf.data_ptr(), 64, 4, 128, "bf16", 0, 10000.0, [(60, 10, 0)], buf, buf, 128)
    assert e.value.code == 1
