"""Thin ctypes binding of include/kvattn.h: same names, argument marshalling only.

Tensors are torch tensors used as device memory; every step of the path runs in the library's
kernels.  There is no CPU fallback: if the shared library is missing the import fails.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvattn.so")

KV_OK, KV_ERR_INVALID, KV_ERR_OOM, KV_ERR_NOT_ALLOCATED, KV_ERR_BOUNDS = 0, 1, 2, 3, 4
KV_ERR_UNSUPPORTED, KV_ERR_CUDA, KV_ERR_TIMEOUT, KV_ERR_WORKSPACE, KV_ERR_PINNED = 5, 6, 7, 8, 9


class KvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().kv_status_str(status).decode()} ({status})")


class ExtendArgs(C.Structure):
    _fields_ = [("q", C.c_void_p), ("cu_q", C.c_void_p), ("block_tables", C.c_void_p), ("max_pages", C.c_int),
                ("prefix_lens", C.c_void_p), ("extend_lens", C.c_void_p), ("batch", C.c_int), ("total_q", C.c_int),
                ("max_extend_len", C.c_int), ("max_total_len", C.c_int), ("out", C.c_void_p), ("lse", C.c_void_p)]


class DecodeArgs(C.Structure):
    _fields_ = [("q", C.c_void_p), ("block_tables", C.c_void_p), ("max_pages", C.c_int), ("ctx_lens", C.c_void_p),
                ("batch", C.c_int), ("max_ctx_len", C.c_int), ("out", C.c_void_p), ("lse", C.c_void_p)]


_lib = None
_I, _P, _F, _SZ, _I64 = C.c_int, C.c_void_p, C.c_float, C.c_size_t, C.c_int64

_SIGNATURES = {
    "kv_status_str": (C.c_char_p, [_I]),
    "kv_pool_create": (_I, [_I, _I, _I, _I, C.POINTER(_P)]),
    "kv_pool_create_ex": (_I, [_I, _I, _I, _I, _P, _P, C.POINTER(_P)]),
    "kv_pool_destroy": (_I, [_P]),
    "kv_pool_stats": (_I, [_P, C.POINTER(_I), C.POINTER(_I), C.POINTER(_I64)]),
    "kv_pool_raw": (_I, [_P, C.POINTER(_P), C.POINTER(_P), C.POINTER(_I64)]),
    "kv_pool_elem_offset": (_I64, [_P, _I, _I, _I, _I]),
    "kv_pool_set_poison": (_I, [_P, _I]),
    "kv_alloc": (_I, [_P, _I, C.POINTER(_I)]),
    "kv_free": (_I, [_P, C.POINTER(_I), _I]),
    "kv_evict": (_I, [_P, C.POINTER(_I), _I]),
    "kv_ref": (_I, [_P, C.POINTER(_I), _I]),
    "kv_pin": (_I, [_P, C.POINTER(_I), _I]),
    "kv_unpin": (_I, [_P, C.POINTER(_I), _I]),
    "kv_unpin_all": (_I, [_P, C.POINTER(_I)]),
    "kv_touch": (_I, [_P, C.POINTER(_I), _I]),
    "kv_evict_lru": (_I, [_P, _I, C.POINTER(_I), C.POINTER(_I)]),
    "kv_page_info": (_I, [_P, _I, C.POINTER(_I), C.POINTER(_I), C.POINTER(_I)]),
    "kv_append": (_I, [_P, _P, _P, _P, _P, _P, _P, _I, _I, _I, _P]),
    "kv_gather": (_I, [_P, _P, _I, _P, _P, _P]),
    "attn_workspace_bytes": (_SZ, [_P, _I, _I, _I, _I, _I, _I]),
    "attn_extend": (_I, [_P, _P, _I, _P, _P, _I, _P, _P, _I, _I, _I, _I, _F, _P, _P, _P, _SZ, _P]),
    "attn_extend_append": (_I, [_P, _P, _P, _P, _I, _P, _P, _I, _P, _P, _I, _I, _I, _I, _F, _P, _P, _P, _SZ, _P]),
    "attn_extend_plan": (_I, [_P, _I, _P, _P, _I, _P, _P, _I, _I, _I, _I, _P, _SZ, _P]),
    "attn_extend_planned": (_I, [_P, _P, _I, _P, _P, _I, _P, _P, _I, _I, _I, _I, _F, _P, _P, _P, _SZ, _P]),
    "attn_extend_host_staging_bytes": (_SZ, [_P, _I, _I, _I, _I, _I]),
    "attn_extend_host": (_I, [_P, _P, _P, _P, _I, _P, _P, _I, _P, _P, _I, _I, _I, _I, _F, _P, _P, _P, _SZ, _P]),
    "attn_extend_shared_workspace_bytes": (_SZ, [_P, _I, _I, _I, _I, _I]),
    "attn_extend_shared": (_I, [_P, _P, _I, _P, _P, _P, _I, _P, _P, _I, _P, _I, _I, _I, _I, _I, _I, _F, _P, _P, _P, _SZ,
                                _P]),
    "attn_decode": (_I, [_P, _P, _I, _P, _I, _P, _I, _I, _F, _P, _P, _P, _SZ, _P]),
    "attn_decode_static": (_I, [_P, _P, _I, _P, _I, _P, _I, _I, _F, _P, _P, _P]),
    "attn_decode_static_scratch_bytes": (_SZ, []),
    "attn_mixed": (_I, [_P, _I, _F, C.POINTER(ExtendArgs), C.POINTER(DecodeArgs), _P, _SZ, _P]),
    "kv_check_batch": (_I, [_P, _P, _I, _P, _I, _P]),
    "kv_last_async_status": (_I, [_P]),
    "kvattn_set_extend_impl": (_I, [_I]),
    "kvattn_set_shared_impl": (_I, [_I]),
    "kvattn_set_decode_impl": (_I, [_I]),
    "kvattn_set_mixed_extend_ctas": (_I, [_I]),
    "kvattn_selftest_bounded_wait": (_I, [_P, C.c_ulonglong, _P, _P]),
    "kvattn_launch_count": (_I64, []),
}


def lib():
    """Loads libkvattn.so once.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_23815_b200.build` "
                              "(needs nvcc); this package has no CPU or PyTorch fallback")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype, fn.argtypes = res, args
        _lib = l
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to the library must be contiguous"
    return C.c_void_p(t.data_ptr())


def _dev_ptr(t: Optional[torch.Tensor]):
    if t is not None:
        assert t.is_cuda, "expected a CUDA tensor"
    return _ptr(t)


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def _check(status: int, where: str):
    if status != KV_OK:
        raise KvError(status, where)


def _int_array(ids: Sequence[int]):
    return (C.c_int * len(ids))(*[int(i) for i in ids])


class Pool:
    """Handle to a kv_pool_t (kv_pool_create / kv_pool_destroy)."""

    def __init__(self, num_pages: int, page_size: int, n_kv_heads: int, head_dim: int,
                 k_base: Optional[torch.Tensor] = None, v_base: Optional[torch.Tensor] = None):
        self.handle = C.c_void_p()
        self.num_pages, self.page_size, self.n_kv_heads, self.head_dim = num_pages, page_size, n_kv_heads, head_dim
        self._keep = (k_base, v_base)
        if k_base is None:
            st = lib().kv_pool_create(num_pages, page_size, n_kv_heads, head_dim, C.byref(self.handle))
        else:
            st = lib().kv_pool_create_ex(num_pages, page_size, n_kv_heads, head_dim, _dev_ptr(k_base),
                                         _dev_ptr(v_base), C.byref(self.handle))
        _check(st, "kv_pool_create")

    def destroy(self):
        if self.handle:
            lib().kv_pool_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def kv_pool_create(num_pages, page_size, n_kv_heads, head_dim) -> Pool:
    return Pool(num_pages, page_size, n_kv_heads, head_dim)


def kv_pool_create_ex(num_pages, page_size, n_kv_heads, head_dim, k_base, v_base) -> Pool:
    return Pool(num_pages, page_size, n_kv_heads, head_dim, k_base, v_base)


def kv_pool_destroy(pool: Pool):
    pool.destroy()


def kv_pool_stats(pool: Pool):
    f, u, e = C.c_int(), C.c_int(), C.c_int64()
    _check(lib().kv_pool_stats(pool.handle, C.byref(f), C.byref(u), C.byref(e)), "kv_pool_stats")
    return f.value, u.value, e.value


def kv_pool_raw(pool: Pool):
    k, v, n = C.c_void_p(), C.c_void_p(), C.c_int64()
    _check(lib().kv_pool_raw(pool.handle, C.byref(k), C.byref(v), C.byref(n)), "kv_pool_raw")
    return k.value, v.value, n.value


def kv_pool_elem_offset(pool: Pool, page, kv_head, slot, d) -> int:
    return lib().kv_pool_elem_offset(pool.handle, page, kv_head, slot, d)


def kv_pool_set_poison(pool: Pool, on: bool):
    _check(lib().kv_pool_set_poison(pool.handle, int(on)), "kv_pool_set_poison")


def kv_alloc(pool: Pool, n: int):
    out = (C.c_int * max(n, 1))()
    _check(lib().kv_alloc(pool.handle, n, out), "kv_alloc")
    return list(out[:n])


def kv_free(pool: Pool, page_ids: Sequence[int]):
    _check(lib().kv_free(pool.handle, _int_array(page_ids), len(page_ids)), "kv_free")


def kv_evict(pool: Pool, page_ids: Sequence[int]):
    _check(lib().kv_evict(pool.handle, _int_array(page_ids), len(page_ids)), "kv_evict")


def kv_ref(pool: Pool, page_ids: Sequence[int]):
    _check(lib().kv_ref(pool.handle, _int_array(page_ids), len(page_ids)), "kv_ref")


def kv_pin(pool: Pool, page_ids: Sequence[int]):
    _check(lib().kv_pin(pool.handle, _int_array(page_ids), len(page_ids)), "kv_pin")


def kv_unpin(pool: Pool, page_ids: Sequence[int]):
    _check(lib().kv_unpin(pool.handle, _int_array(page_ids), len(page_ids)), "kv_unpin")


def kv_unpin_all(pool: Pool) -> int:
    n = C.c_int()
    _check(lib().kv_unpin_all(pool.handle, C.byref(n)), "kv_unpin_all")
    return n.value


def kv_touch(pool: Pool, page_ids: Sequence[int]):
    _check(lib().kv_touch(pool.handle, _int_array(page_ids), len(page_ids)), "kv_touch")


def kv_evict_lru(pool: Pool, n: int):
    out, cnt = (C.c_int * max(n, 1))(), C.c_int()
    _check(lib().kv_evict_lru(pool.handle, n, out, C.byref(cnt)), "kv_evict_lru")
    return list(out[:cnt.value])


def kv_page_info(pool: Pool, page: int):
    a, r, p = C.c_int(), C.c_int(), C.c_int()
    _check(lib().kv_page_info(pool.handle, page, C.byref(a), C.byref(r), C.byref(p)), "kv_page_info")
    return a.value, r.value, p.value


def kv_append(pool: Pool, k_new, v_new, cu_new, start_pos, seg_row, block_tables, stream=None):
    n_seg = start_pos.numel()
    _check(lib().kv_append(pool.handle, _dev_ptr(k_new), _dev_ptr(v_new), _dev_ptr(cu_new), _dev_ptr(start_pos),
                           _dev_ptr(seg_row), _dev_ptr(block_tables), block_tables.shape[1], n_seg,
                           k_new.shape[0], _stream(stream)), "kv_append")


def kv_gather(pool: Pool, block_table_row, length, k_out, v_out, stream=None):
    _check(lib().kv_gather(pool.handle, _dev_ptr(block_table_row), length, _dev_ptr(k_out), _dev_ptr(v_out),
                           _stream(stream)), "kv_gather")


def attn_workspace_bytes(pool: Pool, n_q_heads, batch_ext=0, total_q=0, max_total_len=0, batch_dec=0,
                         max_ctx_len=0) -> int:
    return lib().attn_workspace_bytes(pool.handle, n_q_heads, batch_ext, total_q, max_total_len, batch_dec,
                                      max_ctx_len)


def attn_extend(pool: Pool, q, cu_q, block_tables, prefix_lens, extend_lens, max_extend_len, max_total_len, scale,
                out, lse, workspace=None, stream=None):
    _check(lib().attn_extend(pool.handle, _dev_ptr(q), q.shape[1], _dev_ptr(cu_q), _dev_ptr(block_tables),
                             block_tables.shape[1], _dev_ptr(prefix_lens), _dev_ptr(extend_lens),
                             prefix_lens.numel(), q.shape[0], max_extend_len, max_total_len, float(scale),
                             _dev_ptr(out), _dev_ptr(lse), _dev_ptr(workspace),
                             0 if workspace is None else workspace.numel() * workspace.element_size(),
                             _stream(stream)), "attn_extend")


def attn_extend_append(pool: Pool, q, k_new, v_new, cu_q, block_tables, prefix_lens, extend_lens, max_extend_len,
                       max_total_len, scale, out, lse, workspace=None, stream=None):
    """kv_append of the suffix rows (k_new, v_new, ragged by cu_q) at positions prefix_lens[i].. and attn_extend, one call."""
    _check(lib().attn_extend_append(pool.handle, _dev_ptr(q), _dev_ptr(k_new), _dev_ptr(v_new), q.shape[1], _dev_ptr(cu_q),
                                    _dev_ptr(block_tables), block_tables.shape[1], _dev_ptr(prefix_lens),
                                    _dev_ptr(extend_lens), prefix_lens.numel(), q.shape[0], max_extend_len, max_total_len,
                                    float(scale), _dev_ptr(out), _dev_ptr(lse), _dev_ptr(workspace),
                                    0 if workspace is None else workspace.numel() * workspace.element_size(),
                                    _stream(stream)), "attn_extend_append")


def attn_extend_plan(pool: Pool, n_q_heads, cu_q, block_tables, prefix_lens, extend_lens, total_q, max_extend_len,
                     max_total_len, workspace, stream=None):
    """Builds attn_extend's work list for these lengths into the workspace (once per step, reused by every layer)."""
    _check(lib().attn_extend_plan(pool.handle, n_q_heads, _dev_ptr(cu_q), _dev_ptr(block_tables), block_tables.shape[1],
                                  _dev_ptr(prefix_lens), _dev_ptr(extend_lens), prefix_lens.numel(), total_q,
                                  max_extend_len, max_total_len, _dev_ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream(stream)), "attn_extend_plan")


def attn_extend_planned(pool: Pool, q, cu_q, block_tables, prefix_lens, extend_lens, max_extend_len, max_total_len, scale,
                        out, lse, workspace, stream=None):
    """attn_extend over the plan that attn_extend_plan left in the workspace (same arguments)."""
    _check(lib().attn_extend_planned(pool.handle, _dev_ptr(q), q.shape[1], _dev_ptr(cu_q), _dev_ptr(block_tables),
                                     block_tables.shape[1], _dev_ptr(prefix_lens), _dev_ptr(extend_lens),
                                     prefix_lens.numel(), q.shape[0], max_extend_len, max_total_len, float(scale),
                                     _dev_ptr(out), _dev_ptr(lse), _dev_ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream(stream)), "attn_extend_planned")


def attn_extend_host_staging_bytes(pool: Pool, n_q_heads, batch, total_q, max_pages, max_total_len) -> int:
    return lib().attn_extend_host_staging_bytes(pool.handle, n_q_heads, batch, total_q, max_pages, max_total_len)


def attn_extend_host(pool: Pool, q, k_new, v_new, cu_q, block_tables, prefix_lens, extend_lens, max_extend_len,
                     max_total_len, scale, out, lse, staging, stream=None):
    """One step from host tensors (pinned for asynchrony): copies in, kv_append of the suffix, attn_extend, copies out.
    `staging` is a device byte tensor of attn_extend_host_staging_bytes() bytes."""
    for t in (q, k_new, v_new, cu_q, block_tables, prefix_lens, extend_lens, out, lse):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("attn_extend_host takes contiguous host tensors")
    _check(lib().attn_extend_host(pool.handle, C.c_void_p(q.data_ptr()), C.c_void_p(k_new.data_ptr()),
                                  C.c_void_p(v_new.data_ptr()), q.shape[1], C.c_void_p(cu_q.data_ptr()),
                                  C.c_void_p(block_tables.data_ptr()), block_tables.shape[1],
                                  C.c_void_p(prefix_lens.data_ptr()), C.c_void_p(extend_lens.data_ptr()),
                                  prefix_lens.numel(), q.shape[0], max_extend_len, max_total_len, float(scale),
                                  C.c_void_p(out.data_ptr()), C.c_void_p(lse.data_ptr()), _dev_ptr(staging),
                                  staging.numel() * staging.element_size(), _stream(stream)), "attn_extend_host")


def kvattn_set_shared_impl(impl: int):
    _check(lib().kvattn_set_shared_impl(impl), "kvattn_set_shared_impl")


def attn_extend_shared_workspace_bytes(pool: Pool, n_q_heads, n_parents, n_children, total_q, max_parent_len) -> int:
    return lib().attn_extend_shared_workspace_bytes(pool.handle, n_q_heads, n_parents, n_children, total_q,
                                                    max_parent_len)


def attn_extend_shared(pool: Pool, q, cu_q, cu_children, parent_tables, parent_lens, child_tables, child_lens,
                       max_child_len, max_parent_rows, max_parent_len, scale, out, lse, workspace, stream=None):
    """Children that share their parent's prefix pages (see the header): the shared pages are read once per parent."""
    _check(lib().attn_extend_shared(pool.handle, _dev_ptr(q), q.shape[1], _dev_ptr(cu_q), _dev_ptr(cu_children),
                                    _dev_ptr(parent_tables), parent_tables.shape[1], _dev_ptr(parent_lens),
                                    _dev_ptr(child_tables), child_tables.shape[1], _dev_ptr(child_lens),
                                    parent_lens.numel(), child_lens.numel(), q.shape[0], max_child_len,
                                    max_parent_rows, max_parent_len, float(scale), _dev_ptr(out), _dev_ptr(lse),
                                    _dev_ptr(workspace),
                                    0 if workspace is None else workspace.numel() * workspace.element_size(),
                                    _stream(stream)), "attn_extend_shared")


def attn_decode(pool: Pool, q, block_tables, ctx_lens, max_ctx_len, scale, out, lse, workspace=None, stream=None):
    _check(lib().attn_decode(pool.handle, _dev_ptr(q), q.shape[1], _dev_ptr(block_tables), block_tables.shape[1],
                             _dev_ptr(ctx_lens), q.shape[0], max_ctx_len, float(scale), _dev_ptr(out),
                             _dev_ptr(lse), _dev_ptr(workspace),
                             0 if workspace is None else workspace.numel() * workspace.element_size(),
                             _stream(stream)), "attn_decode")


def attn_decode_static(pool: Pool, q, block_tables, ctx_lens, max_ctx_len, scale, out, lse, stream=None):
    """attn_decode for callers that cannot allocate: no workspace argument, the scratch is a fixed array inside
    the library (see the header for the limit and the sharing rules)."""
    _check(lib().attn_decode_static(pool.handle, _dev_ptr(q), q.shape[1], _dev_ptr(block_tables),
                                    block_tables.shape[1], _dev_ptr(ctx_lens), q.shape[0], max_ctx_len, float(scale),
                                    _dev_ptr(out), _dev_ptr(lse), _stream(stream)), "attn_decode_static")


def attn_decode_static_scratch_bytes() -> int:
    return lib().attn_decode_static_scratch_bytes()


def extend_args(q, cu_q, block_tables, prefix_lens, extend_lens, max_extend_len, max_total_len, out, lse) -> ExtendArgs:
    return ExtendArgs(q.data_ptr(), cu_q.data_ptr(), block_tables.data_ptr(), block_tables.shape[1],
                      prefix_lens.data_ptr(), extend_lens.data_ptr(), prefix_lens.numel(), q.shape[0],
                      max_extend_len, max_total_len, out.data_ptr(), lse.data_ptr())


def decode_args(q, block_tables, ctx_lens, max_ctx_len, out, lse) -> DecodeArgs:
    return DecodeArgs(q.data_ptr(), block_tables.data_ptr(), block_tables.shape[1], ctx_lens.data_ptr(),
                      q.shape[0], max_ctx_len, out.data_ptr(), lse.data_ptr())


def attn_mixed(pool: Pool, n_q_heads, scale, ext: Optional[ExtendArgs], dec: Optional[DecodeArgs], workspace,
               stream=None):
    _check(lib().attn_mixed(pool.handle, n_q_heads, float(scale), C.byref(ext) if ext is not None else None,
                            C.byref(dec) if dec is not None else None, _dev_ptr(workspace),
                            0 if workspace is None else workspace.numel() * workspace.element_size(),
                            _stream(stream)), "attn_mixed")


def kv_check_batch(pool: Pool, block_tables, lens, stream=None) -> int:
    return lib().kv_check_batch(pool.handle, _dev_ptr(block_tables), block_tables.shape[1], _dev_ptr(lens),
                                lens.numel(), _stream(stream))


def kv_last_async_status(pool: Pool) -> int:
    return lib().kv_last_async_status(pool.handle)


def kvattn_set_extend_impl(impl: int):
    _check(lib().kvattn_set_extend_impl(impl), "kvattn_set_extend_impl")


def kvattn_set_decode_impl(impl: int):
    _check(lib().kvattn_set_decode_impl(impl), "kvattn_set_decode_impl")


def kvattn_set_mixed_extend_ctas(n: int):
    _check(lib().kvattn_set_mixed_extend_ctas(n), "kvattn_set_mixed_extend_ctas")


def kvattn_selftest_bounded_wait(pool: Pool, limit_ns: int, trace, stream=None):
    """Test surface: lets a bounded device-side wait run out (see the header); trace is an int32 device tensor [4]."""
    _check(lib().kvattn_selftest_bounded_wait(pool.handle, int(limit_ns), _dev_ptr(trace), _stream(stream)),
           "kvattn_selftest_bounded_wait")


def kvattn_launch_count() -> int:
    return lib().kvattn_launch_count()
