"""Pins for the CPU oracle: each test ties a part of it to something other than itself -
a brute-force routine, a closed form, an identity the paper states, or a hand-worked fixture -
chosen so that a dropped term, a wrong sign or index, or a transposed operand fails one of them."""
import math
import os

import numpy as np
import pytest

from oracle import bruteforce as bf
from oracle import reference as orc
from paper_2604_13226_b200 import inputs as gen
from helpers import make_store, oracle_outputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def tiny(seed=1, dtype="f32", d=16, Hq=4, Hkv=2, lens=(5, 9, 3), nh=2, nt=3, q_len=4, pairing=0, **kw):
    shape = gen.ModelShape(1, Hq, Hkv, d, dtype, 10000.0, pairing)
    items = [[(p, 0) for p in range(len(lens))]]
    return gen.make_workload(shape, list(lens), items, q_len, n_header=nh, n_trailer=nt, seed=seed, **kw)


# ---------------------------------------------------------------------------- RoPE (Eq. 1)

def test_rope_hand_values():
    # one pair, angle pi/2 per position: (1,0) -> (0,1); a sign error gives (0,-1)
    y = orc.rope(np.array([[[1.0, 0.0]]]), 1, np.array([math.pi / 2]))
    assert np.allclose(y, [[[0.0, 1.0]]], atol=1e-15)
    y = orc.rope(np.array([[[1.0, 0.0]]]), -1, np.array([math.pi / 2]))
    assert np.allclose(y, [[[0.0, -1.0]]], atol=1e-15)
    # d=4: half-split pairs (0,2),(1,3); interleaved pairs (0,1),(2,3); second pair frequency 0 -> untouched
    x = np.array([[[1.0, 2.0, 3.0, 4.0]]])
    f = np.array([math.pi / 2, 0.0])
    assert np.allclose(orc.rope(x, 1, f, 0), [[[-3.0, 2.0, 1.0, 4.0]]], atol=1e-15)
    assert np.allclose(orc.rope(x, 1, f, 1), [[[-2.0, 1.0, 3.0, 4.0]]], atol=1e-15)


def test_inv_freq_closed_form():
    f = orc.inv_freq(10000.0, 8)
    assert np.allclose(f, [1.0, 0.1, 0.01, 0.001], rtol=1e-14)
    f = orc.inv_freq(500000.0, 128)
    assert f[0] == 1.0 and abs(f[63] - 500000.0 ** (-126 / 128)) < 1e-18


@pytest.mark.parametrize("pairing", [0, 1])
def test_rope_matches_complex_multiplication(pairing):
    rng = np.random.default_rng(3)
    d = 32
    x = rng.standard_normal((7, 3, d))
    delta = np.array([0, 1, -1, 17, -250, 131072, 99999])
    f = orc.inv_freq(500000.0, d)
    y = orc.rope(x, delta, f, pairing)
    if pairing == 0:
        z = x[..., : d // 2] + 1j * x[..., d // 2:]
    else:
        z = x[..., 0::2] + 1j * x[..., 1::2]
    w = z * np.exp(1j * delta[:, None, None] * f[None, None, :])
    if pairing == 0:
        ref = np.concatenate([w.real, w.imag], axis=-1)
    else:
        ref = np.empty_like(x)
        ref[..., 0::2], ref[..., 1::2] = w.real, w.imag
    assert np.max(np.abs(y - ref)) < 1e-12


@pytest.mark.parametrize("pairing", [0, 1])
def test_rope_identities(pairing):
    rng = np.random.default_rng(4)
    d = 64
    f = orc.inv_freq(10000.0, d)
    k = rng.standard_normal((5, 2, d))
    q = rng.standard_normal((5, 2, d))
    p, dl = 37, -12
    # composition: rotating a key cached at p by delta equals rotating the raw key at p+delta
    assert np.max(np.abs(orc.rope(orc.rope(k, p, f, pairing), dl, f, pairing) - orc.rope(k, p + dl, f, pairing))) < 1e-12
    assert np.array_equal(orc.rope(k, 0, f, pairing), k)                                   # R_0 = I
    assert np.max(np.abs(orc.rope(orc.rope(k, 9, f, pairing), -9, f, pairing) - k)) < 1e-12  # inverse
    # pair norms preserved
    y = orc.rope(k, 1234, f, pairing)
    if pairing == 0:
        n0, n1 = k[..., :32] ** 2 + k[..., 32:] ** 2, y[..., :32] ** 2 + y[..., 32:] ** 2
    else:
        n0, n1 = k[..., 0::2] ** 2 + k[..., 1::2] ** 2, y[..., 0::2] ** 2 + y[..., 1::2] ** 2
    assert np.max(np.abs(n0 - n1)) < 1e-12
    # scores depend on relative displacement only
    s0 = np.sum(orc.rope(q, 40, f, pairing) * orc.rope(k, 11, f, pairing), axis=-1)
    s1 = np.sum(orc.rope(q, 40 + 1000, f, pairing) * orc.rope(k, 11 + 1000, f, pairing), axis=-1)
    assert np.max(np.abs(s0 - s1)) < 1e-10
    # counter-rotating the query is the same score as rotating the key
    s2 = np.sum(orc.rope(q, -dl, f, pairing) * k, axis=-1)
    s3 = np.sum(q * orc.rope(k, dl, f, pairing), axis=-1)
    assert np.max(np.abs(s2 - s3)) < 1e-12


# ---------------------------------------------------------------------------- composition

def test_compose_matches_hand_worked_config1():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "config1_plan.txt")) if l.strip() and not l.startswith("#")]
    segs = np.array(rows[:-1], dtype=np.int32)
    P = int(rows[-1][0])
    wl = gen.config1()
    plan = orc.compose(make_store(wl), wl.items[0], rebase=True)
    assert plan.prefix_len == P == wl.prefix_len(0)
    assert np.array_equal(plan.segments, segs)
    # token-level map agrees with the segment table
    for r0, n, dst, dl in segs:
        assert np.array_equal(plan.src_row[dst:dst + n], np.arange(r0, r0 + n))
        assert np.all(plan.delta[dst:dst + n] == dl)
        assert np.array_equal(plan.cache_pos[dst:dst + n], np.arange(n))


def test_compose_paper_packet_positions_give_one_delta_per_packet():
    # the paper caches header|doc|trailer as one unit from position 0 (Section 3.1): header at 0,
    # document at N_h, trailer at N_h + L  ->  all three segments of a packet share one Delta
    shape = gen.ModelShape(1, 2, 1, 8, "f32")
    wl = gen.make_workload(shape, [6, 6], [[(0, 0), (1, 0)]], 2, n_header=2, n_trailer=3, seed=0,
                           packet_pos0=[2, 2], adapter_pos0=[(0, 8)])
    plan = orc.compose(make_store(wl), wl.items[0])
    assert list(plan.segments[:, 3]) == [0, 0, 0, 11, 11, 11]


def test_rebase_off_and_no_adapters_is_plain_concatenation():
    wl = tiny(lens=(4, 7, 2))
    st = make_store(wl)
    plan = orc.compose(st, [(p, -1) for p in range(3)], rebase=False)
    f = orc.inv_freq(wl.shape.rope_theta, wl.shape.head_dim)
    k_reb, v_cat, k_raw = orc.composed_kv(st, plan, 0, f)
    kc = np.concatenate([p.k[0] for p in wl.packets]).astype(np.float64)
    vc = np.concatenate([p.v[0] for p in wl.packets]).astype(np.float64)
    assert np.all(plan.delta == 0) and np.array_equal(plan.src_row, np.arange(13))
    assert np.array_equal(k_reb, kc) and np.array_equal(v_cat, vc) and np.array_equal(k_raw, kc)


def test_composed_keys_equal_raw_keys_rotated_at_slot_positions():
    # build "raw" (position-free) keys, cache each segment at its own cache positions, compose,
    # and compare with the raw keys rotated directly at their composed positions (Eq. 1 both ways)
    rng = np.random.default_rng(9)
    d, Hkv = 16, 2
    f = orc.inv_freq(10000.0, d)
    lens, pos0 = [5, 3, 8], [0, 4, 100]
    raw = [rng.standard_normal((n, Hkv, d)) for n in lens]
    st = orc.Store("f64")
    for r, p0 in zip(raw, pos0):
        cached = orc.rope(r, p0 + np.arange(len(r)), f)
        st.register_packet(len(r), p0, (lambda layer, c=cached: (c, c)))
    plan = orc.compose(st, [(2, -1), (0, -1), (1, -1)])
    k_reb, _, _ = orc.composed_kv(st, plan, 0, f)
    direct = orc.rope(np.concatenate([raw[2], raw[0], raw[1]]), np.arange(16), f)
    assert np.max(np.abs(k_reb - direct)) < 1e-12


# ---------------------------------------------------------------------------- attention

@pytest.mark.parametrize("pairing", [0, 1])
def test_attention_equals_dense_mask_bruteforce(pairing):
    wl = tiny(seed=5, pairing=pairing)
    st = make_store(wl)
    plan = orc.compose(st, wl.items[0])
    s = wl.shape
    f = orc.inv_freq(s.rope_theta, s.head_dim)
    q, kn, vn = wl.query_layer(0)
    out, lse, K, V = orc.query_prefill(st, plan, 0, q[0], kn[0], vn[0], f, pairing)
    P, Lq = plan.prefix_len, wl.q_len
    rng = np.random.default_rng(0)
    Q_all = np.concatenate([rng.standard_normal((P, s.n_q_heads, s.head_dim)), q[0].astype(np.float64)])
    seg_lens = [2 + n + 3 for n in (5, 9, 3)]
    ref = bf.dense_mask_attention(K, V, Q_all, bf.fig2d_mask(seg_lens, Lq), 1 / math.sqrt(s.head_dim), s.group)
    ref = ref[P:].reshape(Lq * s.n_q_heads, s.head_dim)
    assert np.max(np.abs(out - ref)) < 1e-12


def test_rows_sum_to_one_and_lse():
    wl = tiny(seed=6)
    st = make_store(wl)
    plan = orc.compose(st, wl.items[0])
    s = wl.shape
    f = orc.inv_freq(s.rope_theta, s.head_dim)
    q, kn, vn = wl.query_layer(0)
    out, lse, ps, K, V = orc.query_prefill(st, plan, 0, q[0], kn[0], vn[0], f, want_prob_sum=True)
    assert np.max(np.abs(ps - 1.0)) < 1e-13
    P = plan.prefix_len
    Q = q[0].astype(np.float64)
    r = 0
    for i in range(wl.q_len):
        for h in range(s.n_q_heads):
            sc = (K[: P + i + 1, h // s.group] @ Q[i, h]) / math.sqrt(s.head_dim)
            assert abs(lse[r] - np.log(np.sum(np.exp(sc)))) < 1e-12
            r += 1


def test_single_packet_no_adapter_is_ordinary_causal_prefill_bitwise():
    shape = gen.ModelShape(1, 4, 2, 8, "f32")
    wl = gen.make_workload(shape, [11], [[(0, -1)]], 5, n_header=0, n_trailer=0, seed=2)
    st = make_store(wl)
    plan = orc.compose(st, wl.items[0])
    assert np.all(plan.delta == 0)
    f = orc.inv_freq(shape.rope_theta, 8)
    q, kn, vn = wl.query_layer(0)
    out, lse, K, V = orc.query_prefill(st, plan, 0, q[0], kn[0], vn[0], f)
    seqK = np.concatenate([wl.packets[0].k[0], kn[0]]).astype(np.float64)
    seqV = np.concatenate([wl.packets[0].v[0], vn[0]]).astype(np.float64)
    ref = bf.ordinary_causal_prefill(seqK, seqV, q[0].astype(np.float64), 11, 1.0 / np.sqrt(np.float64(8)), 2)
    assert np.array_equal(out, ref.reshape(-1, 8))


def test_packet_permutation_with_positions_carried():
    wl = tiny(seed=7, lens=(6, 4, 7))
    st = make_store(wl)
    plan = orc.compose(st, wl.items[0])
    s = wl.shape
    f = orc.inv_freq(s.rope_theta, s.head_dim)
    q, kn, vn = wl.query_layer(0)
    out, lse, K, V = orc.query_prefill(st, plan, 0, q[0], kn[0], vn[0], f)
    P = plan.prefix_len
    # permute whole packets of already re-based keys (their positions travel inside the rotation)
    b = np.cumsum([0, 11, 9, 12])
    order = [2, 0, 1]
    idx = np.concatenate([np.arange(b[o], b[o + 1]) for o in order] + [np.arange(P, P + wl.q_len)])
    out2, lse2 = orc.attention_rows(K[idx], V[idx], q[0].astype(np.float64), P, 1 / math.sqrt(s.head_dim))
    assert np.max(np.abs(out - out2)) < 1e-12 and np.max(np.abs(lse - lse2)) < 1e-12
    # whereas composing in another order without carrying positions does change the result
    plan3 = orc.compose(st, [wl.items[0][o] for o in order])
    out3 = orc.query_prefill(st, plan3, 0, q[0], kn[0], vn[0], f)[0]
    assert np.max(np.abs(out - out3)) > 1e-6


def test_closed_forms():
    rng = np.random.default_rng(8)
    P, Lq, Hq, Hkv, d = 13, 3, 4, 2, 8
    Q = rng.standard_normal((Lq, Hq, d))
    V = rng.standard_normal((P + Lq, Hkv, d))
    # all keys equal -> uniform weights -> mean of the visible values
    K = np.broadcast_to(rng.standard_normal((1, Hkv, d)), (P + Lq, Hkv, d)).copy()
    out, lse = orc.attention_rows(K, V, Q, P, 0.3)
    r = 0
    for i in range(Lq):
        for h in range(Hq):
            assert np.max(np.abs(out[r] - V[: P + i + 1, h // 2].mean(axis=0))) < 1e-12
            r += 1
    # constant values -> constant output
    K = rng.standard_normal((P + Lq, Hkv, d))
    Vc = np.full((P + Lq, Hkv, d), 2.5)
    out, _ = orc.attention_rows(K, Vc, Q, P, 0.3)
    assert np.max(np.abs(out - 2.5)) < 1e-12
    # one key far above the rest -> that value row; a key beyond the causal limit is never seen
    K2 = K * 0.01
    K2[4, 0] = Q[0, 0] * 50.0
    K2[P + 2, 0] = Q[0, 0] * 500.0      # query token 2's own key: invisible to token 0
    out, _ = orc.attention_rows(K2, V, Q, P, 1.0, rows=[(0, 0)])
    assert np.max(np.abs(out[0] - V[4, 0])) < 1e-9
    # adding a constant to all scores changes nothing (scale the keys' projection on q uniformly)
    out_a, lse_a = orc.attention_rows(K, V, Q, P, 0.3, rows=[(1, 2)])
    Kshift = K + 3.0 * Q[2, 1][None, None, :] / np.dot(Q[2, 1], Q[2, 1])
    out_b, lse_b = orc.attention_rows(Kshift, V, Q, P, 0.3, rows=[(1, 2)])
    assert np.max(np.abs(out_a - out_b)) < 1e-12 and abs((lse_b - lse_a)[0] - 0.9) < 1e-12


def test_gqa_head_mapping_and_operand_order():
    # q head h must read kv head floor(h/g); make the kv heads wildly different
    rng = np.random.default_rng(10)
    P, Hq, Hkv, d = 6, 4, 2, 4
    Q = rng.standard_normal((1, Hq, d))
    K = rng.standard_normal((P + 1, Hkv, d))
    V = np.zeros((P + 1, Hkv, d))
    V[:, 0, :] = 1.0
    V[:, 1, :] = -1.0
    out, _ = orc.attention_rows(K, V, Q, P, 0.5)
    assert np.allclose(out[:2], 1.0) and np.allclose(out[2:], -1.0)
    # explicit two-key example: weights softmax([q.k0, q.k1]) applied to values, not transposed
    Q = np.array([[[1.0, 0.0]]])
    K = np.array([[[2.0, 7.0]], [[0.0, -3.0]]])
    V = np.array([[[10.0, 20.0]], [[30.0, 40.0]]])
    out, lse = orc.attention_rows(K, V, Q, 1, 1.0)
    w0 = math.exp(2.0) / (math.exp(2.0) + 1.0)
    assert np.allclose(out[0], [10 * w0 + 30 * (1 - w0), 20 * w0 + 40 * (1 - w0)], atol=1e-13)
    assert abs(lse[0] - math.log(math.exp(2.0) + 1.0)) < 1e-13


def test_split_and_merge_by_lse_equals_unsplit():
    rng = np.random.default_rng(11)
    P, Hq, Hkv, d = 21, 2, 1, 8
    Q = rng.standard_normal((1, Hq, d))
    K = rng.standard_normal((P + 1, Hkv, d))
    V = rng.standard_normal((P + 1, Hkv, d))
    full, lse = orc.attention_rows(K, V, Q, P, 0.4)
    P1 = 9
    # part A: keys [0,P1) and the query's own key; part B: keys [P1,P) (its last key plays "own key")
    ia = np.r_[np.arange(P1), P]
    oa, la = orc.attention_rows(K[ia], V[ia], Q, P1, 0.4)
    ob, lb = orc.attention_rows(K[P1:P], V[P1:P], Q, P - P1 - 1, 0.4)
    wa, wb = np.exp(la - lse), np.exp(lb - lse)
    assert np.max(np.abs(wa + wb - 1.0)) < 1e-12
    assert np.max(np.abs(full - (wa[:, None] * oa + wb[:, None] * ob))) < 1e-12


def test_rope_query_flag_equals_prerotated_inputs():
    wl = tiny(seed=12, dtype="f32")
    st = make_store(wl)
    plan = orc.compose(st, wl.items[0])
    s = wl.shape
    f = orc.inv_freq(s.rope_theta, s.head_dim)
    q, kn, vn = wl.query_layer(0)
    P = plan.prefix_len
    out_a = orc.query_prefill(st, plan, 0, q[0], kn[0], vn[0], f, rope_query=True)[0]
    pos = np.arange(P, P + wl.q_len)
    st64 = orc.Store("f64")
    for p in wl.packets:
        st64.register_packet(p.n_tokens, 0, (lambda l, p=p: (p.k[l].astype(np.float64), p.v[l].astype(np.float64))))
    a = wl.adapters[0]
    st64.register_adapter(a.n_header, 0, a.n_trailer, 0,
                          (lambda l: tuple(x[l].astype(np.float64) for x in (a.hk, a.hv, a.tk, a.tv))))
    out_b = orc.query_prefill(st64, plan, 0, orc.rope(q[0].astype(np.float64), pos, f),
                              orc.rope(kn[0].astype(np.float64), pos, f), vn[0].astype(np.float64), f)[0]
    assert np.max(np.abs(out_a - out_b)) < 1e-12


def test_widen_bf16_exact():
    bits = np.array([0x3F80, 0xBF80, 0x4049, 0x0000, 0x7F7F], dtype=np.uint16)
    assert list(orc.widen(bits, "bf16")) == [1.0, -1.0, 3.140625, 0.0, float(np.float32(3.3895314e38))]
    x = np.array([1.0, 1.00390625, 1.001953125, 1.005859375], dtype=np.float32)   # ties-to-even cases
    assert list(gen.f32_to_bf16_bits(x)) == [0x3F80, 0x3F80, 0x3F80, 0x3F81]


# ------------------------------------------------------------------------------------------------
# compressed packets (Section 4.3): a kv head attends over the keys its pruned cache still holds
# ------------------------------------------------------------------------------------------------

def _compressed_case(keep_rate, seed=11, q_len=6, dtype="f32"):
    shape = gen.ModelShape(2, 4, 2, 64, dtype, 10000.0, 0)
    return gen.make_workload(shape, [50, 33, 70], [[(0, 0), (1, 0), (2, -1)]], q_len=q_len, n_header=3, n_trailer=2,
                             seed=seed, keep_rate=keep_rate, packet_pos0=[0, 4, 0])


def test_compressed_keep_everything_equals_uncompressed():
    wl = _compressed_case([None, None, None])
    ref = oracle_outputs(wl, layer=1)[0]
    for p in wl.packets:
        p.kept = [[np.arange(p.n_tokens) for _ in range(2)] for _ in range(2)]
    got = oracle_outputs(wl, layer=1)[0]
    assert np.array_equal(got[0], ref[0]) and np.array_equal(got[1], ref[1])


def test_compressed_equals_masked_dense_attention():
    # independent route: dense scores over the whole composed sequence, pruned keys masked to -inf
    wl = _compressed_case([0.5, None, 0.3])
    s = wl.shape
    for layer in range(s.n_layers):
        out, lse, K, V, plan = oracle_outputs(wl, layer=layer)[0]
        P = plan.prefix_len
        present = np.ones((P + wl.q_len, s.n_kv_heads), dtype=bool)
        t = 0
        for pid, aid in wl.items[0]:
            if aid >= 0:
                t += wl.adapters[aid].n_header
            p = wl.packets[pid]
            if p.kept is not None:
                present[t:t + p.n_tokens] = False
                for h in range(s.n_kv_heads):
                    present[t + p.kept[layer][h], h] = True
            t += p.n_tokens
            if aid >= 0:
                t += wl.adapters[aid].n_trailer
        assert t == P and not present[:P].all()
        Q = orc.widen(wl.q[layer][0], s.dtype)
        n = 0
        for i in range(wl.q_len):
            for h in range(s.n_q_heads):
                hk = h // s.group
                sc = (K[:P + i + 1, hk] @ Q[i, h]) / np.sqrt(s.head_dim)
                sc = np.where(present[:P + i + 1, hk], sc, -np.inf)
                w = np.exp(sc - sc.max())
                o = (w[:, None] * V[:P + i + 1, hk]).sum(0) / w.sum()
                assert np.max(np.abs(o - out[n])) <= 1e-12
                assert abs(sc.max() + np.log(w.sum()) - lse[n]) <= 1e-12
                n += 1


def test_compressed_closed_forms():
    wl = _compressed_case([0.4, 0.6, None], dtype="f32")
    s = wl.shape
    # constant values: the output is that constant whatever is pruned
    for p in wl.packets:
        p.v[...] = np.float32(0.75)
    for a in wl.adapters:
        a.hv[...] = np.float32(0.75)
        a.tv[...] = np.float32(0.75)
    wl.v_new[...] = np.float32(0.75)
    out = oracle_outputs(wl, layer=0)[0][0]
    assert np.max(np.abs(out - 0.75)) <= 1e-14
    # a pruned key cannot matter: give it an enormous score and a wild value, nothing changes
    wl2 = _compressed_case([0.4, 0.6, None])
    ref = oracle_outputs(wl2, layer=0)[0][0]
    p = wl2.packets[0]
    dropped = sorted(set(range(p.n_tokens)) - set(int(x) for x in p.kept[0][0]))
    assert dropped
    p.k[0][dropped[0], 0, :] = np.float32(30.0)
    p.v[0][dropped[0], 0, :] = np.float32(1e6)
    got = oracle_outputs(wl2, layer=0)[0][0]
    assert np.array_equal(got, ref)


# ------------------------------------------------------------------------------------------------
# attention mass per segment
# ------------------------------------------------------------------------------------------------

def test_segment_mass_rows_sum_to_one_and_match_closed_forms():
    shape = gen.ModelShape(1, 4, 2, 64, "f32", 10000.0, 0)
    wl = gen.make_workload(shape, [50, 33], [[(0, 0), (1, -1)]], q_len=5, n_header=3, n_trailer=2, seed=3)
    st = make_store(wl)
    plan = orc.compose(st, wl.items[0])
    f = orc.inv_freq(shape.rope_theta, 64)
    m = orc.segment_mass(st, plan, 0, wl.q[0][0], wl.k_new[0][0], f)
    assert m.shape == (5 * 4, 4 + 1) and np.max(np.abs(m.sum(1) - 1.0)) <= 1e-14 and m.min() >= 0
    # consistency with the attention routine: exp(score - lse) summed over everything is the same 1,
    # and with V replaced by one-hot segment indicators the attention output IS the mass
    P = plan.prefix_len
    ind = np.zeros((P + 5, 2, 64))
    for s_, (_, length, t0, _) in enumerate(plan.segments):
        ind[t0:t0 + length, :, s_] = 1.0
    ind[P:, :, 4] = 1.0
    Kp, _, _ = orc.composed_kv(st, plan, 0, f)
    K = np.concatenate([Kp, orc.widen(wl.k_new[0][0], "f32")])
    o, _ = orc.attention_rows(K, ind, orc.widen(wl.q[0][0], "f32"), P, 1.0 / 8.0)
    assert np.max(np.abs(o[:, :5] - m)) <= 1e-14
    # all keys equal: every visible key gets the same probability, mass = segment length / keys seen
    for p in wl.packets:
        p.k[...] = np.float32(0.25)
    for a in wl.adapters:
        a.hk[...] = np.float32(0.25)
        a.tk[...] = np.float32(0.25)
    wl.k_new[...] = np.float32(0.25)
    plan0 = orc.compose(st, wl.items[0], rebase=False)
    m = orc.segment_mass(st, plan0, 0, wl.q[0][0], wl.k_new[0][0], f, rows=[(1, 2)])
    seen = P + 3
    assert np.allclose(m[0], [3 / seen, 50 / seen, 2 / seen, 33 / seen, 3 / seen], atol=1e-14)


def test_empty_prefix_is_plain_causal_attention_over_the_query_block():
    shape = gen.ModelShape(1, 4, 2, 64, "f32", 10000.0, 0)
    wl = gen.make_workload(shape, [20], [[]], q_len=6, seed=4)
    out, lse, K, V, plan = oracle_outputs(wl)[0]
    assert plan.prefix_len == 0 and K.shape[0] == 6
    Q = orc.widen(wl.q[0][0], "f32")
    n = 0
    for i in range(6):
        for h in range(4):
            sc = (K[:i + 1, h // 2] @ Q[i, h]) / 8.0
            w = np.exp(sc - sc.max())
            assert np.max(np.abs((w[:, None] * V[:i + 1, h // 2]).sum(0) / w.sum() - out[n])) <= 1e-14
            n += 1
