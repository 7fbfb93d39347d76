"""Drives the library over a synthetic workload: sizes a context for it, registers its packets and
adapters (packets in id order, then adapters - the order the index map depends on), assembles the
batch and runs per-layer query prefill.  Used by the tests, the smoke check and the benchmark; it
contains no arithmetic of the method - every number comes out of the CUDA kernels."""
from __future__ import annotations

from typing import List, Optional

import numpy as np

from . import binding as kvp
from .inputs import DeviceWorkload, Workload


def np_to_torch(a: np.ndarray, dtype: str, device):
    """Host array in stored dtype (bf16 as uint16 bits) -> device tensor of that dtype."""
    import torch
    a = np.ascontiguousarray(a)
    if dtype == "bf16":
        return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(a).to(device)


def torch_to_np(t, dtype: str) -> np.ndarray:
    """Device tensor -> host array in stored dtype (bf16 as uint16 bits)."""
    import torch
    t = t.contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


class Session:
    def __init__(self, wl, materialize: bool = False, device: int = 0, max_query_tokens: Optional[int] = None,
                 max_assemblies: int = 1, host_packets: bool = False):
        import torch
        self.torch = torch
        self.wl = wl
        self.shape = wl.shape
        self.device = torch.device(f"cuda:{device}")
        self.materialize = materialize
        s = wl.shape
        is_dev = isinstance(wl, DeviceWorkload)
        if is_dev:
            lens = list(wl.spec.packet_lens)
            ad_tokens = wl.spec.n_header + wl.spec.n_trailer
            n_adapters = 1
        else:
            lens = [p.n_tokens for p in wl.packets]
            ad_tokens = sum(a.n_header + a.n_trailer for a in wl.adapters)
            n_adapters = len(wl.adapters)
        B = wl.batch
        self.q_len = wl.q_len
        mq = max_query_tokens or wl.q_len
        prefix = [wl.prefix_len(b) for b in range(B)]
        n_slots = sum(len(it) for it in wl.items)
        if materialize:
            ws_rows = sum(prefix) + B * mq
        else:
            ws_rows = sum(prefix[b] - sum(lens[pid] for pid, _ in wl.items[b]) for b in range(B)) + B * mq
        self.ctx = kvp.Context(s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, s.dtype, rope_theta=s.rope_theta,
                               rope_pairing=s.rope_pairing, pool_tokens=sum(lens) + ad_tokens + 8,
                               max_packets=max(1, len(lens)), max_adapters=max(1, n_adapters), max_batch=B,
                               max_slots=max(1, n_slots), max_prefix_tokens=max(prefix + [1]), max_query_tokens=mq,
                               max_ws_rows=ws_rows + 8, max_assemblies=max_assemblies, device=device,
                               max_compressed=0 if is_dev else sum(1 for p in wl.packets if p.kept is not None))
        # registration (offline in the paper; not part of any timed region)
        self.host_kv = []                      # pinned host copies of the packets (host_packets): kept alive here
        if is_dev:
            for pid in range(len(lens)):
                k, v = wl.packet_device(pid)
                if host_packets:
                    # [layers][tokens][kv heads][d] -> the pool's plane order [layers][kv heads][tokens][d], in pinned memory
                    hk = k.permute(0, 2, 1, 3).contiguous().cpu().pin_memory()
                    hv = v.permute(0, 2, 1, 3).contiguous().cpu().pin_memory()
                    self.host_kv.append((hk, hv))
                    self.ctx.register_packet_host(hk, hv, lens[pid], 0)
                else:
                    self.ctx.register_packet(k, v, lens[pid], 0)
                del k, v
            hk, hv, tk, tv = wl.adapter_device()
            self.ctx.register_adapter(hk, hv, wl.spec.n_header, 0, tk, tv, wl.spec.n_trailer, 0)
        else:
            for p in wl.packets:
                if p.kept is not None:
                    # the compressor's output: for every (layer, kv head) its surviving rows, runs back to back
                    runs_k = [p.k[l][p.kept[l][h], h, :] for l in range(s.n_layers) for h in range(s.n_kv_heads)]
                    runs_v = [p.v[l][p.kept[l][h], h, :] for l in range(s.n_layers) for h in range(s.n_kv_heads)]
                    counts = [len(p.kept[l][h]) for l in range(s.n_layers) for h in range(s.n_kv_heads)]
                    k = np_to_torch(np.concatenate(runs_k, axis=0), s.dtype, self.device)
                    v = np_to_torch(np.concatenate(runs_v, axis=0), s.dtype, self.device)
                    self.ctx.register_packet_compressed(k, v, p.n_tokens, p.cache_pos0, counts)
                    continue
                if host_packets:
                    hk = np_to_torch(np.ascontiguousarray(np.transpose(p.k, (0, 2, 1, 3))), s.dtype, "cpu").pin_memory()
                    hv = np_to_torch(np.ascontiguousarray(np.transpose(p.v, (0, 2, 1, 3))), s.dtype, "cpu").pin_memory()
                    self.host_kv.append((hk, hv))
                    self.ctx.register_packet_host(hk, hv, p.n_tokens, p.cache_pos0)
                    continue
                k = np_to_torch(p.k, s.dtype, self.device)
                v = np_to_torch(p.v, s.dtype, self.device)
                self.ctx.register_packet(k, v, p.n_tokens, p.cache_pos0)
            for a in wl.adapters:
                t = [np_to_torch(x, s.dtype, self.device) if x.shape[1] > 0 else None for x in (a.hk, a.hv, a.tk, a.tv)]
                self.ctx.register_adapter(t[0], t[1], a.n_header, a.header_pos0, t[2], t[3], a.n_trailer,
                                          a.trailer_pos0)
        torch.cuda.synchronize(self.device)
        self.assembly_id = -1
        self.prefix_len: List[int] = []

    def assemble(self, rebase: Optional[bool] = None, items=None, pos_base=None):
        flags = 0
        if self.wl.rebase if rebase is None else rebase:
            flags |= kvp.REBASE
        if self.materialize:
            flags |= kvp.MATERIALIZE
        self.assembly_id, self.prefix_len = self.ctx.assemble(items if items is not None else self.wl.items, flags,
                                                              pos_base=pos_base)
        return self.assembly_id, self.prefix_len

    def query_tensors(self, layer: int):
        if isinstance(self.wl, DeviceWorkload):
            return self.wl.query_device(layer)
        q, k, v = self.wl.query_layer(layer)
        d = self.shape.dtype
        return np_to_torch(q, d, self.device), np_to_torch(k, d, self.device), np_to_torch(v, d, self.device)

    def prefill(self, layer: int, flags: int = 0, qkv=None, want_lse: bool = True):
        torch = self.torch
        q, k_new, v_new = qkv if qkv is not None else self.query_tensors(layer)
        out = torch.empty_like(q)
        lse = None
        if want_lse:
            lse = torch.empty((q.shape[0], self.shape.n_q_heads, q.shape[1]), dtype=torch.float32, device=self.device)
        self.ctx.query_prefill(self.assembly_id, layer, q, k_new, v_new, q.shape[1], out, lse, flags)
        return out, lse

    def close(self):
        self.ctx.close()
