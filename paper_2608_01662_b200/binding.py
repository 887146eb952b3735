"""ctypes binding of liblsa.so: same names as include/lsa.h, argument marshalling only.

Every function takes torch tensors (device memory, plumbing) or None, passes their data pointers to
the C ABI and raises LsaError on a negative status.  Nothing is computed here, and there is no
fallback: a missing or unloadable library raises at first use.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_float, c_int, c_int32, c_int64, c_size_t, c_uint32, c_void_p

import torch

from .configs import LsaConfig

_LIB = None
# LSA_LIBRARY selects another build of the same library (the checking build liblsa_check.so, see build.py)
LIB_PATH = os.environ.get("LSA_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblsa.so")

LSA_KEY_BF16, LSA_KEY_E4M3 = 0, 1
LSA_POOL_MEAN, LSA_POOL_MINMAX = 0, 1
KERNEL_CLASSES = ("block_means", "coarse_score", "fine_select", "select", "convert", "sparse_attn", "merge_splits")


class LsaError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: {code} ({lib().lsa_strerror(code).decode()}) {detail}")


class LsaParams(ctypes.Structure):
    _fields_ = [("struct_size", c_uint32), ("n_heads_idx", c_int32), ("d_idx", c_int32), ("key_dtype", c_int32),
                ("page", c_int32), ("sub_block", c_int32), ("keep_pages", c_int32), ("k_sparse", c_int32),
                ("k_sink", c_int32), ("k_swa", c_int32), ("n_heads", c_int32), ("d_qk", c_int32), ("d_v", c_int32),
                ("sm_scale", c_float), ("n_layers", c_int32), ("q_chunk", c_int32), ("hi_enable", c_int32),
                ("paged", c_int32), ("kv_page", c_int32), ("pooling", c_int32)]


EXPORTS = {
    "lsa_create": (c_int, [POINTER(c_void_p), c_int, c_void_p, c_void_p, c_size_t]),
    "lsa_destroy": (c_int, [c_void_p]),
    "lsa_workspace_bytes": (c_int, [POINTER(LsaParams), c_int64, c_int64, c_int, POINTER(c_size_t)]),
    "lsa_status": (c_int, [c_void_p, POINTER(c_int)]),
    "lsa_strerror": (c_char_p, [c_int]),
    "lsa_last_cuda_error": (c_char_p, [c_void_p]),
    "lsa_launch_count": (c_int64, [c_void_p]),
    "lsa_tune": (c_int, [c_void_p, c_int, c_int]),
    "lsa_selftest_wait": (c_int, [c_void_p, c_int64]),
    "lsa_profile_enable": (c_int, [c_void_p, c_int]),
    "lsa_profile_read": (c_int, [c_void_p, POINTER(ctypes.c_double), POINTER(c_int64)]),
    "lsa_block_means": (c_int, [c_void_p, POINTER(LsaParams), c_void_p, c_void_p, c_int64, c_void_p, c_int64,
                                c_void_p, c_int, c_void_p]),
    "lsa_index": (c_int, [c_void_p, POINTER(LsaParams), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64,
                          c_int64, c_int64, c_void_p, c_int64, c_void_p, c_int, c_void_p, c_void_p, c_void_p]),
    "lsa_index_static": (c_int, [c_int, c_void_p, POINTER(LsaParams), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                 c_int64, c_int64, c_int64, c_void_p, c_void_p]),
    "lsa_index_static_status": (c_int, [c_int, c_void_p, POINTER(c_int)]),
    "lsa_select": (c_int, [c_void_p, POINTER(LsaParams), c_void_p, c_int64, c_void_p, c_int64, c_int64, c_int64,
                           c_int32, c_int32, c_void_p, c_void_p]),
    "lsa_convert": (c_int, [c_void_p, POINTER(LsaParams), c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_int64,
                            c_void_p, c_int, c_void_p, c_void_p, c_void_p]),
    "lsa_sparse_attn": (c_int, [c_void_p, POINTER(LsaParams), c_void_p, c_void_p, c_void_p, c_int64, c_int64,
                                c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int64, c_int64, c_void_p, c_int,
                                c_void_p, c_void_p]),
    "lsa_append": (c_int, [c_void_p, POINTER(LsaParams), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64,
                           c_void_p, c_int, c_void_p, c_int, POINTER(c_void_p), POINTER(c_void_p), c_int64]),
    "lsa_merge": (c_int, [c_void_p, POINTER(LsaParams), c_int, POINTER(c_void_p), POINTER(c_void_p), c_int64, c_void_p,
                          c_void_p]),
    "lsa_layer_group": (c_int, [c_void_p, POINTER(LsaParams), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                c_int64, c_int64, c_int64, c_void_p, c_int64, c_void_p, c_int, POINTER(c_void_p),
                                POINTER(c_void_p), POINTER(c_void_p), c_int64, c_int64, POINTER(c_void_p),
                                POINTER(c_void_p), c_void_p, c_void_p]),
    "lsa_layer_group_host": (c_int, [c_void_p, POINTER(LsaParams), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                     c_int64, c_int64, c_int64, POINTER(c_void_p), POINTER(c_void_p), POINTER(c_void_p),
                                     c_int64, c_int64, POINTER(c_void_p), c_int64, POINTER(c_void_p), c_size_t]),
    "lsa_host_stage_bytes": (c_int, [POINTER(LsaParams), c_int64, POINTER(c_size_t)]),
}


def lib() -> ctypes.CDLL:
    """The loaded library.  Raises if it has not been built: there is no other implementation."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2608_01662_b200.build` "
                               "(the CUDA library is the only implementation of this path)")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _LIB = handle
    return _LIB


def make_params(cfg: LsaConfig) -> LsaParams:
    return LsaParams(ctypes.sizeof(LsaParams), cfg.H_I, cfg.d_I, LSA_KEY_E4M3 if cfg.key_dtype == "e4m3" else LSA_KEY_BF16,
                     cfg.P, cfg.B, cfg.M, cfg.Ksp, cfg.S, cfg.W, cfg.H, cfg.d_qk, cfg.d_v, cfg.sm_scale, cfg.R,
                     cfg.q_chunk, 1 if cfg.hi_enable else 0, 1 if cfg.mode == "decode" else 0, cfg.kv_page,
                     LSA_POOL_MINMAX if cfg.pooling == "minmax" else LSA_POOL_MEAN)


def _p(t):
    if t is None:
        return None
    if isinstance(t, int):
        return c_void_p(t)
    assert t.is_contiguous() or t.dim() == 2, "tensors are passed by base pointer"
    return c_void_p(t.data_ptr())


def _parr(ts):
    if ts is None:
        return None
    return (c_void_p * len(ts))(*[None if t is None else (t if isinstance(t, int) else t.data_ptr()) for t in ts])


def workspace_bytes(params: LsaParams, n_query: int, n_key_max: int, batch: int = 1) -> int:
    out = c_size_t(0)
    r = lib().lsa_workspace_bytes(ctypes.byref(params), n_query, n_key_max, batch, ctypes.byref(out))
    if r != 0:
        raise LsaError(r, "lsa_workspace_bytes")
    return out.value


def host_stage_bytes(params: LsaParams, stage_queries: int) -> int:
    out = c_size_t(0)
    r = lib().lsa_host_stage_bytes(ctypes.byref(params), stage_queries, ctypes.byref(out))
    if r != 0:
        raise LsaError(r, "lsa_host_stage_bytes")
    return out.value


STATIC_SCRATCH_BYTES = 8 << 20


def index_static(params: LsaParams, q_idx, w, k_idx, k_scale, kmean, q_pos0, n_query, n_key, sparse_idx, n_sparse,
                 stream=None):
    """lsa_index_static: the prefill indexer with its scratch inside the library (no context, no workspace)."""
    dev = q_idx.device
    stream = stream if stream is not None else torch.cuda.current_stream(dev)
    r = lib().lsa_index_static(dev.index or 0, c_void_p(stream.cuda_stream), ctypes.byref(params), _p(q_idx), _p(w),
                               _p(k_idx), _p(k_scale), _p(kmean), q_pos0, n_query, n_key, _p(sparse_idx), _p(n_sparse))
    if r != 0:
        raise LsaError(r, "lsa_index_static")


def index_static_status(device, stream=None) -> int:
    """lsa_index_static_status: waits for the stream, returns and clears the status word of lsa_index_static."""
    dev = torch.device(device)
    stream = stream if stream is not None else torch.cuda.current_stream(dev)
    st = c_int(0)
    r = lib().lsa_index_static_status(dev.index or 0, c_void_p(stream.cuda_stream), ctypes.byref(st))
    if r != 0:
        raise LsaError(r, "lsa_index_static_status")
    return st.value


class Context:
    """lsa_ctx bound to the current torch CUDA stream; owns its workspace tensor."""

    def __init__(self, params: LsaParams, n_query: int, n_key_max: int, batch: int = 1, device=None, stream=None):
        self.params = params
        self.device = torch.device(device if device is not None else "cuda:0")
        nbytes = workspace_bytes(params, n_query, n_key_max, batch)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        h = c_void_p()
        r = lib().lsa_create(ctypes.byref(h), self.device.index or 0, c_void_p(self.stream.cuda_stream),
                             c_void_p(self.workspace.data_ptr()), nbytes)
        if r != 0:
            raise LsaError(r, "lsa_create")
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            lib().lsa_destroy(self.h)
            self.h = None

    __del__ = close

    def _chk(self, r, where):
        if r != 0:
            raise LsaError(r, where, lib().lsa_last_cuda_error(self.h).decode())

    def status(self) -> int:
        out = c_int(0)
        self._chk(lib().lsa_status(self.h, ctypes.byref(out)), "lsa_status")
        return out.value

    def launch_count(self) -> int:
        return lib().lsa_launch_count(self.h)

    def selftest_wait(self, budget_cycles: int):
        """lsa_selftest_wait: a bounded device-side wait that runs out (status() then returns LSA_ERR_TIMEOUT)."""
        self._chk(lib().lsa_selftest_wait(self.h, budget_cycles), "lsa_selftest_wait")

    def tune(self, knob: int, value: int):
        self._chk(lib().lsa_tune(self.h, knob, value), "lsa_tune")

    def profile_enable(self, on: bool):
        self._chk(lib().lsa_profile_enable(self.h, 1 if on else 0), "lsa_profile_enable")

    def profile_read(self) -> dict:
        """{kernel class: (total ms, launches)} since the last read."""
        n = len(KERNEL_CLASSES)
        ms, cnt = (ctypes.c_double * n)(), (c_int64 * n)()
        self._chk(lib().lsa_profile_read(self.h, ms, cnt), "lsa_profile_read")
        return {KERNEL_CLASSES[i]: (ms[i], cnt[i]) for i in range(n)}

    def block_means(self, k_idx, k_scale, n_key, kmean, page_table=None, ctx_len=None):
        pt_stride = page_table.shape[1] if page_table is not None else 0
        batch = page_table.shape[0] if page_table is not None else 1
        self._chk(lib().lsa_block_means(self.h, ctypes.byref(self.params), _p(k_idx), _p(k_scale), n_key,
                                        _p(page_table), pt_stride, _p(ctx_len), batch, _p(kmean)), "lsa_block_means")

    def index(self, q_idx, w, k_idx, k_scale, kmean, q_pos0, n_query, n_key, sparse_idx, n_sparse, pages_out=None,
              page_table=None, ctx_len=None):
        pt_stride = page_table.shape[1] if page_table is not None else 0
        batch = page_table.shape[0] if page_table is not None else 1
        self._chk(lib().lsa_index(self.h, ctypes.byref(self.params), _p(q_idx), _p(w), _p(k_idx), _p(k_scale),
                                  _p(kmean), q_pos0, n_query, n_key, _p(page_table), pt_stride, _p(ctx_len), batch,
                                  _p(sparse_idx), _p(n_sparse), _p(pages_out)), "lsa_index")

    def select(self, scores, cand_pos, q_pos0, k, apply_range, idx_out, n_out):
        n_query, n_cand = scores.shape
        self._chk(lib().lsa_select(self.h, ctypes.byref(self.params), _p(scores), scores.stride(0), _p(cand_pos),
                                   q_pos0, n_query, n_cand, k, 1 if apply_range else 0, _p(idx_out), _p(n_out)),
                  "lsa_select")

    def convert(self, sparse_idx, n_sparse, q_pos0, n_query, rows_out, n_rows_out, runs_out=None, page_table=None,
                ctx_len=None):
        pt_stride = page_table.shape[1] if page_table is not None else 0
        batch = page_table.shape[0] if page_table is not None else 1
        self._chk(lib().lsa_convert(self.h, ctypes.byref(self.params), _p(sparse_idx), _p(n_sparse), q_pos0, n_query,
                                    _p(page_table), pt_stride, _p(ctx_len), batch, _p(rows_out), _p(n_rows_out),
                                    _p(runs_out)), "lsa_convert")

    def sparse_attn(self, q, k, v, sparse_idx, n_sparse, q_pos0, n_query, n_key, out, lse=None, rows=None,
                    n_rows=None, ctx_len=None, batch=1, params=None):
        prm = params if params is not None else self.params
        self._chk(lib().lsa_sparse_attn(self.h, ctypes.byref(prm), _p(q), _p(k), _p(v), k.stride(0),
                                        v.stride(0), _p(sparse_idx), _p(n_sparse), _p(rows), _p(n_rows), q_pos0,
                                        n_query, n_key, _p(ctx_len), batch, _p(out), _p(lse)), "lsa_sparse_attn")

    def append(self, k_new, k_idx, k_scale, kmean, page_table, ctx_len, ctx_len_out=None, kv_new=(), kv_pool=()):
        batch = page_table.shape[0]
        row_bytes = kv_pool[0].stride(0) * kv_pool[0].element_size() if len(kv_pool) else 0
        self._chk(lib().lsa_append(self.h, ctypes.byref(self.params), _p(k_new), _p(k_idx), _p(k_scale), _p(kmean),
                                   _p(page_table), page_table.shape[1], _p(ctx_len), batch, _p(ctx_len_out),
                                   len(kv_pool), _parr(list(kv_new)) if len(kv_pool) else None,
                                   _parr(list(kv_pool)) if len(kv_pool) else None, row_bytes), "lsa_append")

    def merge(self, outs, lses, n_query, out, lse=None, params=None):
        prm = params if params is not None else self.params
        self._chk(lib().lsa_merge(self.h, ctypes.byref(prm), len(outs), _parr(outs), _parr(lses), n_query, _p(out),
                                  _p(lse)), "lsa_merge")

    def layer_group(self, q_idx, w, k_idx, k_scale, kmean, q_pos0, n_query, n_key, q, k, v, out, lse, sparse_idx,
                    n_sparse, page_table=None, ctx_len=None):
        pt_stride = page_table.shape[1] if page_table is not None else 0
        batch = page_table.shape[0] if page_table is not None else 1
        self._chk(lib().lsa_layer_group(self.h, ctypes.byref(self.params), _p(q_idx), _p(w), _p(k_idx), _p(k_scale),
                                        _p(kmean), q_pos0, n_query, n_key, _p(page_table), pt_stride, _p(ctx_len),
                                        batch, _parr(q), _parr(k), _parr(v), k[0].stride(0), v[0].stride(0),
                                        _parr(out), _parr(lse), _p(sparse_idx), _p(n_sparse)), "lsa_layer_group")

    def layer_group_host(self, q_idx_host, w_host, k_idx, k_scale, kmean, q_pos0, n_query, n_key, q_host, k, v, out_host,
                         stage_queries, stage):
        self._chk(lib().lsa_layer_group_host(self.h, ctypes.byref(self.params), _p(q_idx_host), _p(w_host), _p(k_idx),
                                             _p(k_scale), _p(kmean), q_pos0, n_query, n_key, _parr(q_host), _parr(k),
                                             _parr(v), k[0].stride(0), v[0].stride(0), _parr(out_host), stage_queries,
                                             _parr(stage), stage[0].numel()), "lsa_layer_group_host")
