"""ctypes binding of ``libkvp.so`` - argument marshalling only; every step of the path runs in the
library's CUDA kernels.  Function names mirror ``include/kvp.h``.

PyTorch is used here for device memory and streams only (``Context`` accepts torch tensors and
passes their ``data_ptr()``).  There is no CPU fallback: if the shared library is missing or cannot
be loaded, importing a symbol raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

from . import build as _build

KVP_OK = 0
STATUS_NAMES = {0: "KVP_OK", 1: "KVP_ERR_INVALID", 2: "KVP_ERR_CAPACITY", 3: "KVP_ERR_NOT_FOUND",
                4: "KVP_ERR_STATE", 5: "KVP_ERR_UNSUPPORTED", 6: "KVP_ERR_CUDA", 7: "KVP_ERR_TIMEOUT"}
DTYPE_F32, DTYPE_BF16 = 0, 1
REBASE, MATERIALIZE = 1, 2
ROPE_QUERY, FORCE_SIMPLE, CONTINUE, PRECISE_QK, PARTIAL, SKIP_QUERY_BLOCK = 1, 2, 4, 8, 16, 32
TUNE_SPLIT_TARGET_CTAS, TUNE_FORCE_SPLITS, TUNE_TIME_KERNELS, TUNE_FUSED_APPEND = 1, 2, 3, 5


class KvpError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"{STATUS_NAMES.get(code, code)}: {text}")
        self.code = code


class kvp_config(ctypes.Structure):
    _fields_ = [
        ("struct_bytes", ctypes.c_int32), ("device", ctypes.c_int32), ("n_layers", ctypes.c_int32),
        ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("rope_pairing", ctypes.c_int32), ("rope_theta", ctypes.c_double),
        ("inv_freq", ctypes.POINTER(ctypes.c_double)), ("softmax_scale", ctypes.c_double),
        ("pool", ctypes.c_void_p), ("pool_bytes", ctypes.c_uint64), ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_uint64), ("max_packets", ctypes.c_int32), ("max_adapters", ctypes.c_int32),
        ("max_batch", ctypes.c_int32), ("max_slots", ctypes.c_int32), ("max_prefix_tokens", ctypes.c_int32),
        ("max_query_tokens", ctypes.c_int32), ("max_ws_rows", ctypes.c_int32), ("max_assemblies", ctypes.c_int32),
        ("max_compressed", ctypes.c_int32),
    ]


_lib = None


def lib() -> ctypes.CDLL:
    """Load (building first if the sources are newer) ``libkvp.so``; raises if that fails."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if not os.path.exists(path) or os.environ.get("KVP_REBUILD"):
        path = _build.build()
    L = ctypes.CDLL(path)
    vp, i32, u32, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32, ctypes.c_uint64
    pi32 = ctypes.POINTER(ctypes.c_int32)
    pcfg = ctypes.POINTER(kvp_config)
    sig = {
        "kvp_version": (i32, []),
        "kvp_token_bytes": (u64, [pcfg]),
        "kvp_workspace_bytes": (u64, [pcfg]),
        "kvp_create": (i32, [pcfg, ctypes.POINTER(vp)]),
        "kvp_destroy": (i32, [vp]),
        "kvp_register_packet": (i32, [vp, vp, vp, i32, i32, vp, pi32]),
        "kvp_register_packet_compressed": (i32, [vp, vp, vp, i32, i32, pi32, vp, pi32]),
        "kvp_register_packet_host": (i32, [vp, vp, vp, i32, i32, pi32]),
        "kvp_evict_packet": (i32, [vp, i32]),
        "kvp_register_adapter": (i32, [vp, vp, vp, i32, i32, vp, vp, i32, i32, vp, pi32]),
        "kvp_assemble": (i32, [vp, i32, pi32, pi32, pi32, u32, vp, pi32, pi32]),
        "kvp_assemble_at": (i32, [vp, i32, pi32, pi32, pi32, pi32, u32, vp, pi32, pi32]),
        "kvp_partial_bytes": (u64, [vp, i32, i32]),
        "kvp_merge_partials": (i32, [vp, vp, i32, i32, i32, vp, vp, vp]),
        "kvp_query_prefill": (i32, [vp, i32, i32, vp, vp, vp, i32, u32, vp, vp, vp]),
        "kvp_query_prefill_ragged": (i32, [vp, i32, i32, vp, vp, vp, i32, pi32, vp, vp, vp]),
        "kvp_export_plan": (i32, [vp, i32, i32, pi32, pi32, pi32, pi32]),
        "kvp_export_cache": (i32, [vp, i32, i32, i32, i32, vp, vp, i32, vp]),
        "kvp_export_schedule": (i32, [vp, i32, i32, pi32, i32, pi32, i32, pi32, i32, pi32]),
        "kvp_segment_mass": (i32, [vp, i32, i32, vp, vp, i32, u32, vp, i32, vp]),
        "kvp_status_word": (i32, [vp, pi32]),
        "kvp_last_launch": (i32, [vp, pi32, pi32, pi32, pi32]),
        "kvp_tune": (i32, [vp, i32, i32]),
        "kvp_kernel_times": (i32, [vp, i32, ctypes.POINTER(ctypes.c_float), i32, pi32]),
        "kvp_last_error": (ctypes.c_char_p, [vp]),
        "kvp_compose_noalloc": (i32, [vp, vp, ctypes.c_int64, i32, i32, i32, i32, ctypes.c_double, i32, pi32, pi32, pi32,
                                      vp, vp, ctypes.c_int64, vp, ctypes.c_char_p, i32]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)          # AttributeError if the library lacks a declared symbol
        fn.restype = res
        fn.argtypes = args
    _lib = L
    return L


EXPORTED = ["kvp_version", "kvp_token_bytes", "kvp_workspace_bytes", "kvp_create", "kvp_destroy",
            "kvp_register_packet", "kvp_register_packet_compressed", "kvp_register_packet_host", "kvp_evict_packet",
            "kvp_register_adapter", "kvp_assemble", "kvp_assemble_at", "kvp_partial_bytes", "kvp_merge_partials", "kvp_query_prefill", "kvp_query_prefill_ragged",
            "kvp_export_plan", "kvp_export_cache", "kvp_export_schedule", "kvp_segment_mass", "kvp_status_word", "kvp_last_launch", "kvp_tune",
            "kvp_kernel_times", "kvp_last_error", "kvp_compose_noalloc"]


def _i32_array(xs: Sequence[int]):
    return (ctypes.c_int32 * max(1, len(xs)))(*[int(x) for x in xs])


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return int(t.data_ptr())


class Context:
    """Thin object wrapper over the C calls.  ``device=-1`` makes a host-only planning context
    (no GPU needed; nothing can be launched)."""

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: str,
                 rope_theta: float = 10000.0, rope_pairing: int = 0, softmax_scale: float = 0.0,
                 inv_freq: Optional[Sequence[float]] = None, pool_tokens: int = 0, max_packets: int = 64,
                 max_adapters: int = 4, max_batch: int = 1, max_slots: int = 64, max_prefix_tokens: int = 4096,
                 max_query_tokens: int = 128, max_ws_rows: int = 0, max_assemblies: int = 1, device: int = 0,
                 max_compressed: int = 0):
        self._L = lib()
        self._h = ctypes.c_void_p()
        cfg = kvp_config()
        cfg.struct_bytes = ctypes.sizeof(kvp_config)
        cfg.device = device
        cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim = n_layers, n_q_heads, n_kv_heads, head_dim
        cfg.dtype = DTYPE_BF16 if dtype == "bf16" else DTYPE_F32
        cfg.rope_pairing = rope_pairing
        cfg.rope_theta = rope_theta
        self._inv_freq = None
        if inv_freq is not None:
            self._inv_freq = (ctypes.c_double * (head_dim // 2))(*inv_freq)
            cfg.inv_freq = ctypes.cast(self._inv_freq, ctypes.POINTER(ctypes.c_double))
        cfg.softmax_scale = softmax_scale
        cfg.max_packets, cfg.max_adapters, cfg.max_batch, cfg.max_slots = max_packets, max_adapters, max_batch, max_slots
        cfg.max_prefix_tokens, cfg.max_query_tokens = max_prefix_tokens, max_query_tokens
        if max_ws_rows <= 0:
            max_ws_rows = max_batch * max_query_tokens + 64 * max_slots
        cfg.max_ws_rows, cfg.max_assemblies = max_ws_rows, max_assemblies
        cfg.max_compressed = max_compressed
        self.dtype, self.device = dtype, device
        self.n_layers, self.n_q_heads, self.n_kv_heads, self.head_dim = n_layers, n_q_heads, n_kv_heads, head_dim
        self.token_bytes = int(self._L.kvp_token_bytes(ctypes.byref(cfg)))
        if self.token_bytes == 0:
            raise KvpError(1, "invalid configuration")
        self.pool = self.workspace = None
        if device >= 0:
            import torch
            self._torch = torch
            dev = torch.device(f"cuda:{device}")
            ws_bytes = int(self._L.kvp_workspace_bytes(ctypes.byref(cfg)))
            self.pool = torch.empty(max(1, pool_tokens) * self.token_bytes + 1024, dtype=torch.uint8, device=dev)
            self.workspace = torch.empty(ws_bytes + 1024, dtype=torch.uint8, device=dev)
            pa = (self.pool.data_ptr() + 1023) // 1024 * 1024
            wa = (self.workspace.data_ptr() + 1023) // 1024 * 1024
            cfg.pool, cfg.pool_bytes = pa, max(1, pool_tokens) * self.token_bytes
            cfg.workspace, cfg.workspace_bytes = wa, ws_bytes
            self.workspace_bytes = ws_bytes
        self.cfg = cfg
        rc = self._L.kvp_create(ctypes.byref(cfg), ctypes.byref(self._h))
        if rc != KVP_OK:
            raise KvpError(rc, (self._L.kvp_last_error(None) or b"").decode())

    # -- plumbing ------------------------------------------------------------------------------
    def _check(self, rc: int):
        if rc != KVP_OK:
            raise KvpError(rc, (self._L.kvp_last_error(self._h) or b"").decode())

    def _stream(self, stream=None):
        if self.device < 0:
            return None
        if stream is None:
            stream = self._torch.cuda.current_stream(self.device)
        return ctypes.c_void_p(stream.cuda_stream)

    def close(self):
        if self._h:
            self._L.kvp_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the six calls ---------------------------------------------------------------------------
    def register_packet(self, k, v, n_tokens: int, cache_pos0: int = 0, stream=None) -> int:
        out = ctypes.c_int32(-1)
        self._check(self._L.kvp_register_packet(self._h, _ptr(k), _ptr(v), n_tokens, cache_pos0,
                                                self._stream(stream), ctypes.byref(out)))
        return out.value

    def register_packet_compressed(self, k, v, n_tokens: int, cache_pos0: int, kept: Sequence[int], stream=None) -> int:
        """kept: n_layers * n_kv_heads row counts; k, v: the kept rows of every (layer, kv head), runs back to back."""
        out = ctypes.c_int32(-1)
        self._check(self._L.kvp_register_packet_compressed(self._h, _ptr(k), _ptr(v), n_tokens, cache_pos0,
                                                           _i32_array(list(kept)), self._stream(stream), ctypes.byref(out)))
        return out.value

    def register_packet_host(self, k_host, v_host, n_tokens: int, cache_pos0: int = 0) -> int:
        """k_host, v_host: host tensors [n_layers][n_kv_heads][n_tokens][head_dim] (pinned for overlap), kept alive
        by the caller; they are copied into the pool by the first assemble that names the packet."""
        out = ctypes.c_int32(-1)
        self._check(self._L.kvp_register_packet_host(self._h, _ptr(k_host), _ptr(v_host), n_tokens, cache_pos0,
                                                     ctypes.byref(out)))
        return out.value

    def evict_packet(self, packet_id: int) -> None:
        self._check(self._L.kvp_evict_packet(self._h, packet_id))

    def register_adapter(self, hk, hv, n_header: int, header_pos0: int, tk, tv, n_trailer: int,
                         trailer_pos0: int, stream=None) -> int:
        out = ctypes.c_int32(-1)
        self._check(self._L.kvp_register_adapter(self._h, _ptr(hk), _ptr(hv), n_header, header_pos0, _ptr(tk),
                                                 _ptr(tv), n_trailer, trailer_pos0, self._stream(stream),
                                                 ctypes.byref(out)))
        return out.value

    def assemble(self, items: Sequence[Sequence[Tuple[int, int]]], flags: int = REBASE, stream=None, pos_base=None):
        """items[b] = [(packet_id, adapter_id), ...].  Returns (assembly_id, prefix_len list).
        pos_base (one position per request) -> ``kvp_assemble_at``: this rank's part of a sharded request."""
        offs, pids, aids = [0], [], []
        for it in items:
            for pid, aid in it:
                pids.append(pid)
                aids.append(aid)
            offs.append(len(pids))
        B = len(items)
        plen = (ctypes.c_int32 * max(1, B))()
        aid = ctypes.c_int32(-1)
        if pos_base is not None:
            self._check(self._L.kvp_assemble_at(self._h, B, _i32_array(offs), _i32_array(pids), _i32_array(aids),
                                                _i32_array(list(pos_base)), flags, self._stream(stream), plen, ctypes.byref(aid)))
        else:
            self._check(self._L.kvp_assemble(self._h, B, _i32_array(offs), _i32_array(pids), _i32_array(aids), flags,
                                             self._stream(stream), plen, ctypes.byref(aid)))
        return aid.value, [int(plen[b]) for b in range(B)]

    def partial_bytes(self, batch: int, q_len: int) -> int:
        return int(self._L.kvp_partial_bytes(self._h, batch, q_len))

    def merge_partials(self, parts, n_parts: int, batch: int, q_len: int, out, lse=None, stream=None):
        self._check(self._L.kvp_merge_partials(self._h, _ptr(parts), n_parts, batch, q_len, _ptr(out), _ptr(lse),
                                               self._stream(stream)))

    def query_prefill(self, assembly_id: int, layer: int, q, k_new, v_new, q_len: int, out, lse=None,
                      flags: int = 0, stream=None):
        self._check(self._L.kvp_query_prefill(self._h, assembly_id, layer, _ptr(q), _ptr(k_new), _ptr(v_new), q_len,
                                              flags, _ptr(out), _ptr(lse), self._stream(stream)))

    def query_prefill_ragged(self, assembly_id: int, layer: int, q, k_new, v_new, q_len_max: int, q_lens: Sequence[int],
                             out, lse=None, stream=None):
        """Per-request query lengths; the tensors are padded to q_len_max tokens per request."""
        self._check(self._L.kvp_query_prefill_ragged(self._h, assembly_id, layer, _ptr(q), _ptr(k_new), _ptr(v_new),
                                                     q_len_max, _i32_array(list(q_lens)), _ptr(out), _ptr(lse),
                                                     self._stream(stream)))

    # -- helpers ---------------------------------------------------------------------------------
    def export_plan(self, assembly_id: int, b: int):
        """(src_row [P], delta [P], seg_table [n_seg][4]) of request b as numpy int32 arrays."""
        import numpy as np
        nseg = ctypes.c_int32(0)
        pi = ctypes.POINTER(ctypes.c_int32)
        self._check(self._L.kvp_export_plan(self._h, assembly_id, b, None, None, None, ctypes.byref(nseg)))
        segs = np.zeros((max(1, nseg.value), 4), dtype=np.int32)
        self._check(self._L.kvp_export_plan(self._h, assembly_id, b, None, None, segs.ctypes.data_as(pi),
                                            ctypes.byref(nseg)))
        segs = segs[:nseg.value]
        prefix_len = int((segs[:, 1] + segs[:, 2]).max()) if nseg.value else 0
        src = np.zeros(max(1, prefix_len), dtype=np.int32)
        dl = np.zeros(max(1, prefix_len), dtype=np.int32)
        self._check(self._L.kvp_export_plan(self._h, assembly_id, b, src.ctypes.data_as(pi), dl.ctypes.data_as(pi),
                                            None, ctypes.byref(nseg)))
        return src[:prefix_len], dl[:prefix_len], segs

    def export_cache(self, assembly_id: int, layer: int, b: int, prefix_len: int, n_query_rows: int,
                     k_as_f32: bool = False, stream=None):
        torch = self._torch
        dt = torch.bfloat16 if self.dtype == "bf16" else torch.float32
        n = prefix_len + n_query_rows
        dev = torch.device(f"cuda:{self.device}")
        k = torch.empty((n, self.n_kv_heads, self.head_dim), dtype=torch.float32 if k_as_f32 else dt, device=dev)
        v = torch.empty((n, self.n_kv_heads, self.head_dim), dtype=dt, device=dev)
        self._check(self._L.kvp_export_cache(self._h, assembly_id, layer, b, n_query_rows, _ptr(k), _ptr(v),
                                             1 if k_as_f32 else 0, self._stream(stream)))
        return k, v

    def export_schedule(self, assembly_id: int, q_len: int):
        """(cta_begin [n_ctas+1], works [n][8], merges [m][8], n_slots) as numpy int32 arrays."""
        import numpy as np
        pi = ctypes.POINTER(ctypes.c_int32)
        counts = (ctypes.c_int32 * 4)()
        self._check(self._L.kvp_export_schedule(self._h, assembly_id, q_len, None, 0, None, 0, None, 0, counts))
        cb = np.zeros(counts[0] + 1, dtype=np.int32)
        works = np.zeros((max(1, counts[1]), 8), dtype=np.int32)
        merges = np.zeros((max(1, counts[2]), 8), dtype=np.int32)
        self._check(self._L.kvp_export_schedule(self._h, assembly_id, q_len, cb.ctypes.data_as(pi), cb.size,
                                                works.ctypes.data_as(pi), works.shape[0],
                                                merges.ctypes.data_as(pi), merges.shape[0], counts))
        return cb, works[:counts[1]], merges[:counts[2]], int(counts[3])

    def segment_mass(self, assembly_id: int, layer: int, q, lse, q_len: int, n_cols: int, flags: int = 0, stream=None):
        """float32 [batch][q_len][n_q_heads][n_cols] attention mass per segment (+ query block) of the last prefill."""
        torch = self._torch
        mass = torch.empty((q.shape[0], q_len, self.n_q_heads, n_cols), dtype=torch.float32, device=q.device)
        self._check(self._L.kvp_segment_mass(self._h, assembly_id, layer, _ptr(q), _ptr(lse), q_len, flags, _ptr(mass),
                                             n_cols, self._stream(stream)))
        return mass

    def status_word(self) -> int:
        w = ctypes.c_int32(0)
        rc = self._L.kvp_status_word(self._h, ctypes.byref(w))
        if rc not in (KVP_OK, 7):
            self._check(rc)
        return w.value

    def last_launch(self):
        a, b, c, d = (ctypes.c_int32() for _ in range(4))
        self._check(self._L.kvp_last_launch(self._h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c), ctypes.byref(d)))
        return {"kind": a.value, "ctas": b.value, "splits": c.value, "launches": d.value}

    def tune(self, key: int, value: int):
        self._check(self._L.kvp_tune(self._h, key, value))

    def kernel_times(self, which: int = 0, cap: int = 4096) -> List[float]:
        """Device durations (ms) of the attention (0) / gather (1) kernels since the last call."""
        buf = (ctypes.c_float * cap)()
        n = ctypes.c_int32(0)
        self._check(self._L.kvp_kernel_times(self._h, which, buf, cap, ctypes.byref(n)))
        return [float(buf[i]) for i in range(n.value)]


def compose_noalloc(pool_k: int, pool_v: int, pool_rows: int, n_planes: int, head_dim: int, dtype: str,
                    rope_pairing: int, rope_theta: float, segments, cache_k, cache_v, cache_rows: int, stream=None):
    """``kvp_compose_noalloc``: gather + re-base ``segments`` = [(src_row0, length, delta), ...] from the
    caller's pool planes into the caller's cache planes without any allocation in the library.
    ``pool_k``/``pool_v`` are device addresses, ``cache_k``/``cache_v`` torch tensors (or addresses)."""
    L = lib()
    n = len(segments)
    err = ctypes.create_string_buffer(256)
    st = ctypes.c_void_p(stream.cuda_stream) if stream is not None else None
    rc = L.kvp_compose_noalloc(pool_k, pool_v, pool_rows, n_planes, head_dim, DTYPE_BF16 if dtype == "bf16" else DTYPE_F32,
                               rope_pairing, rope_theta, n, _i32_array([s[0] for s in segments]),
                               _i32_array([s[1] for s in segments]), _i32_array([s[2] for s in segments]),
                               _ptr(cache_k), _ptr(cache_v), cache_rows, st, err, 256)
    if rc != KVP_OK:
        raise KvpError(rc, err.value.decode())
