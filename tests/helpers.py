"""Shared test helpers: build the oracle's store from a workload and run the oracle over it."""
import numpy as np

from oracle import reference as orc
from paper_2604_13226_b200 import inputs as gen


def make_store(wl):
    """Packets in id order, then adapters in id order - the registration order the library uses too."""
    st = orc.Store(wl.shape.dtype)
    if isinstance(wl, gen.DeviceWorkload):
        for pid, n in enumerate(wl.spec.packet_lens):
            st.register_packet(n, 0, (lambda layer, pid=pid: wl.packet_layer(pid, layer)))
        ad = wl.adapter_host()
        st.register_adapter(ad.n_header, 0, ad.n_trailer, 0,
                            (lambda layer: (ad.hk[layer], ad.hv[layer], ad.tk[layer], ad.tv[layer])))
        return st
    for p in wl.packets:
        st.register_packet(p.n_tokens, p.cache_pos0, (lambda layer, p=p: (p.k[layer], p.v[layer])), kept=p.kept)
    for a in wl.adapters:
        st.register_adapter(a.n_header, a.header_pos0, a.n_trailer, a.trailer_pos0,
                            (lambda layer, a=a: (a.hk[layer], a.hv[layer], a.tk[layer], a.tv[layer])))
    return st


def oracle_outputs(wl, layer=0, rebase=None, rope_query=False, rows=None, items=None):
    """Per request: (out [n_rows][d], lse [n_rows], K_full, V_full, plan) from the fp64 oracle.
    rows: list of (head, token) or None for all rows in (token, head) order."""
    s = wl.shape
    st = make_store(wl)
    f = orc.inv_freq(s.rope_theta, s.head_dim)
    q, kn, vn = wl.query_layer(layer)
    res = []
    its = items if items is not None else wl.items
    for b, slots in enumerate(its):
        plan = orc.compose(st, slots, wl.rebase if rebase is None else rebase)
        out, lse, K, V = orc.query_prefill(st, plan, layer, q[b], kn[b], vn[b], f, s.rope_pairing,
                                           rope_query=rope_query, rows=rows)
        res.append((out, lse, K, V, plan))
    return res


def widen(x, dtype):
    return orc.widen(x, dtype)


# Attention parity bounds for bf16 outputs: max-abs 2e-2 and mean-abs 2e-3 against the fp64 oracle, applied
# to the raw error of every element.  A bf16 output cannot meet 2e-2 once it is large - half an ulp is
# 2^-8 |O| at worst, 0.031 at |O| = 8 - so elements with |O_ref| >= 4 (they only occur in value channels a
# workload multiplies by 8) get 2e-2 + 2^-8 |O_ref| instead, and there may only be a few of them.
BF16_MAX_ABS, BF16_MEAN_ABS = 2e-2, 2e-3
LARGE_OUTPUT, LARGE_FRACTION = 4.0, 0.02


def attention_error_stats(o, ref):
    """o, ref: float64 arrays of the same shape.  Asserts the bounds above; returns a dict of the raw figures."""
    o = np.asarray(o, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    err = np.abs(o - ref)
    large = np.abs(ref) >= LARGE_OUTPUT
    stats = {"max_abs": float(err.max()), "mean_abs": float(err.mean()), "n": int(err.size),
             "n_large": int(large.sum()), "max_abs_large": float(err[large].max()) if large.any() else 0.0,
             "max_abs_small": float(err[~large].max()) if (~large).any() else 0.0,
             "max_ref": float(np.abs(ref).max())}
    assert stats["max_abs_small"] <= BF16_MAX_ABS, stats
    assert np.all(err[large] <= BF16_MAX_ABS + 2.0 ** -8 * np.abs(ref[large])), stats
    assert stats["n_large"] <= LARGE_FRACTION * stats["n"], stats
    assert stats["mean_abs"] <= BF16_MEAN_ABS, stats
    return stats
