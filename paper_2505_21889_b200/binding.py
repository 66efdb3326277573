"""ctypes binding of include/efim.h.  Argument marshalling only: every step of the
path runs inside libefim.so.  There is no fallback: if the library is missing or
cannot be loaded, load_library() raises."""
import ctypes
import os
from ctypes import c_int32, c_void_p, c_float, c_double, c_size_t, c_char_p, POINTER, Structure

import numpy as np

_LIB = None
_HERE = os.path.dirname(os.path.abspath(__file__))


class EfimError(RuntimeError):
    def __init__(self, code, where):
        self.code = int(code)
        detail = f" [{load_library().efim_last_cuda_error().decode()}]" if int(code) == 5 else ""
        super().__init__(f"{where}: {efim_strerror(code)} (status {int(code)}){detail}")


class _CacheDesc(Structure):
    _fields_ = [("d_k_pool", c_void_p), ("d_v_pool", c_void_p), ("num_pages", c_int32),
                ("page_size", c_int32), ("num_q_heads", c_int32), ("num_kv_heads", c_int32),
                ("head_dim", c_int32)]


class _BatchDesc(Structure):
    _fields_ = [("batch", c_int32), ("max_pages_per_seq", c_int32), ("total_new_tokens", c_int32),
                ("d_cached_len", c_void_p), ("d_new_len", c_void_p), ("d_q_indptr", c_void_p),
                ("d_block_table", c_void_p), ("h_cached_len", c_void_p), ("h_new_len", c_void_p)]


class _RopeDesc(Structure):
    _fields_ = [("d_cos_sin", c_void_p), ("max_position", c_int32), ("interleaved", c_int32)]


EXPORTS = ("efim_last_cuda_error", "efim_strerror", "efim_version", "efim_rope_table_build", "efim_kv_append",
           "efim_prefill_workspace_bytes", "efim_append_prefill_attn",
           "efim_decode_workspace_bytes", "efim_decode_attn",
           "efim_decode_static_scratch_bytes", "efim_decode_attn_static",
           "efim_prefill_launch_count", "efim_decode_launch_count",
           "efim_prefill_plan_bytes", "efim_prefill_plan", "efim_append_prefill_attn_planned", "efim_decode_step",
           "efim_append_prefill_step", "efim_selftest_bounded_wait",
           "efim_fragment_cuts", "efim_fim_split", "efim_fim_fragment_spans",
           "efim_frontend_create", "efim_frontend_destroy", "efim_frontend_transform", "efim_frontend_admit",
           "efim_frontend_finish", "efim_frontend_stats")


def library_path() -> str:
    return os.path.join(_HERE, "libefim.so")


def load_library():
    """dlopen libefim.so (built in-tree by paper_2505_21889_b200.build). Raises if absent."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} not found: build it first (python -m paper_2505_21889_b200.build); "
                           "there is no CPU fallback")
    lib = ctypes.CDLL(path)
    lib.efim_strerror.restype = c_char_p
    lib.efim_strerror.argtypes = [ctypes.c_int]
    lib.efim_last_cuda_error.restype = c_char_p
    lib.efim_version.restype = ctypes.c_int
    lib.efim_rope_table_build.restype = ctypes.c_int
    lib.efim_rope_table_build.argtypes = [c_double, c_int32, c_int32, c_void_p]
    lib.efim_kv_append.restype = ctypes.c_int
    lib.efim_kv_append.argtypes = [POINTER(_CacheDesc), POINTER(_BatchDesc), POINTER(_RopeDesc),
                                   c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.efim_prefill_workspace_bytes.restype = c_size_t
    lib.efim_prefill_workspace_bytes.argtypes = [POINTER(_CacheDesc), POINTER(_BatchDesc)]
    lib.efim_append_prefill_attn.restype = ctypes.c_int
    lib.efim_append_prefill_attn.argtypes = [POINTER(_CacheDesc), POINTER(_BatchDesc), c_void_p, c_void_p,
                                             c_void_p, c_float, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.efim_prefill_plan_bytes.restype = c_size_t
    lib.efim_prefill_plan_bytes.argtypes = [POINTER(_CacheDesc), POINTER(_BatchDesc)]
    lib.efim_prefill_plan.restype = ctypes.c_int
    lib.efim_prefill_plan.argtypes = [POINTER(_CacheDesc), POINTER(_BatchDesc), c_void_p, c_size_t]
    lib.efim_append_prefill_attn_planned.restype = ctypes.c_int
    lib.efim_append_prefill_attn_planned.argtypes = [POINTER(_CacheDesc), POINTER(_BatchDesc), c_void_p, c_size_t,
                                                     c_int32, c_void_p, c_void_p, c_void_p, c_float, c_void_p, c_size_t,
                                                     c_void_p, c_void_p]
    lib.efim_append_prefill_step.restype = ctypes.c_int
    lib.efim_append_prefill_step.argtypes = [POINTER(_CacheDesc), POINTER(_BatchDesc), POINTER(_RopeDesc), c_void_p,
                                             c_void_p, c_void_p, c_void_p, c_void_p, c_float, c_void_p, c_size_t,
                                             c_int32, c_void_p, c_size_t, c_void_p, c_void_p]
    lib.efim_selftest_bounded_wait.restype = ctypes.c_int
    lib.efim_selftest_bounded_wait.argtypes = [ctypes.c_uint64, c_void_p, c_void_p, c_void_p]
    lib.efim_decode_workspace_bytes.restype = c_size_t
    lib.efim_decode_workspace_bytes.argtypes = [POINTER(_CacheDesc), c_int32, c_int32]
    lib.efim_decode_attn.restype = ctypes.c_int
    lib.efim_decode_attn.argtypes = [POINTER(_CacheDesc), c_int32, c_void_p, c_int32, c_void_p, c_int32,
                                     c_void_p, c_void_p, c_void_p, c_float, c_void_p, c_size_t,
                                     c_void_p, c_void_p]
    lib.efim_decode_step.restype = ctypes.c_int
    lib.efim_decode_step.argtypes = [POINTER(_CacheDesc), c_int32, c_void_p, c_int32, c_void_p, c_int32,
                                     POINTER(_RopeDesc), c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_float,
                                     c_void_p, c_size_t, c_void_p, c_void_p]
    lib.efim_prefill_launch_count.restype = c_int32
    lib.efim_prefill_launch_count.argtypes = [POINTER(_CacheDesc), POINTER(_BatchDesc)]
    lib.efim_decode_launch_count.restype = c_int32
    lib.efim_decode_launch_count.argtypes = [POINTER(_CacheDesc), c_int32, c_int32]
    lib.efim_decode_static_scratch_bytes.restype = c_size_t
    lib.efim_decode_static_scratch_bytes.argtypes = []
    lib.efim_decode_attn_static.restype = ctypes.c_int
    lib.efim_decode_attn_static.argtypes = [POINTER(_CacheDesc), c_int32, c_void_p, c_int32, c_void_p, c_int32,
                                            c_void_p, c_void_p, c_void_p, c_float, c_void_p, c_void_p]
    lib.efim_frontend_create.restype = c_void_p
    lib.efim_frontend_create.argtypes = [c_int32, c_int32, c_int32, c_int32, c_int32, c_int32]
    lib.efim_frontend_destroy.restype = None
    lib.efim_frontend_destroy.argtypes = [c_void_p]
    lib.efim_frontend_transform.restype = ctypes.c_int
    lib.efim_frontend_transform.argtypes = [c_void_p, ctypes.c_int64, c_void_p, c_int32, c_void_p, c_int32, c_void_p,
                                            c_int32, c_void_p, c_void_p, c_void_p]
    lib.efim_frontend_admit.restype = ctypes.c_int
    lib.efim_frontend_admit.argtypes = [c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_int32, c_void_p, c_void_p,
                                        c_void_p]
    lib.efim_frontend_finish.restype = ctypes.c_int
    lib.efim_frontend_finish.argtypes = [c_void_p, ctypes.c_int64, c_void_p, c_int32]
    lib.efim_frontend_stats.restype = None
    lib.efim_frontend_stats.argtypes = [c_void_p, c_void_p]
    _LIB = lib
    return lib


def exported_symbols():
    """Names declared in include/efim.h that the loaded library exports."""
    lib = load_library()
    return [n for n in EXPORTS if hasattr(lib, n)]


def efim_strerror(code) -> str:
    return load_library().efim_strerror(int(code)).decode()


def efim_version() -> int:
    return load_library().efim_version()


def _ptr(t):
    """Device/host address of a torch tensor, numpy array, int or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream_ptr(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class Cache:
    """Paged KV cache of one layer: two torch.bfloat16 CUDA tensors
    [num_pages, num_kv_heads, page_size, head_dim] owned by the caller."""

    def __init__(self, k_pool, v_pool, num_q_heads):
        assert k_pool.shape == v_pool.shape and k_pool.is_contiguous() and v_pool.is_contiguous()
        self.k_pool, self.v_pool = k_pool, v_pool
        n, hkv, p, d = k_pool.shape
        self.desc = _CacheDesc(k_pool.data_ptr(), v_pool.data_ptr(), n, p, num_q_heads, hkv, d)


class Batch:
    """Ragged batch descriptor.  `cached_len`, `new_len` are host int32 arrays (kept
    as the host mirrors); the device copies and q_indptr are made here with torch."""

    def __init__(self, cached_len, new_len, block_table, device="cuda"):
        import torch
        self.h_cached_len = np.ascontiguousarray(cached_len, dtype=np.int32)
        self.h_new_len = np.ascontiguousarray(new_len, dtype=np.int32)
        indptr = np.zeros(len(self.h_new_len) + 1, dtype=np.int32)
        np.cumsum(self.h_new_len, out=indptr[1:])
        self.h_q_indptr = indptr
        self.d_cached_len = torch.from_numpy(self.h_cached_len).to(device)
        self.d_new_len = torch.from_numpy(self.h_new_len).to(device)
        self.d_q_indptr = torch.from_numpy(indptr).to(device)
        if isinstance(block_table, np.ndarray):
            block_table = torch.from_numpy(np.ascontiguousarray(block_table, dtype=np.int32)).to(device)
        self.d_block_table = block_table
        self.desc = _BatchDesc(len(self.h_new_len), self.d_block_table.shape[1], int(indptr[-1]),
                               self.d_cached_len.data_ptr(), self.d_new_len.data_ptr(),
                               self.d_q_indptr.data_ptr(), self.d_block_table.data_ptr(),
                               self.h_cached_len.ctypes.data, self.h_new_len.ctypes.data)


class Rope:
    """Rotary table on the device (built on the host by the library in double)."""

    def __init__(self, base, head_dim, max_position, interleaved=False, device="cuda"):
        import torch
        host = efim_rope_table_build(base, head_dim, max_position)
        self.table = torch.from_numpy(host).to(device)
        self.desc = _RopeDesc(self.table.data_ptr(), max_position, 1 if interleaved else 0)


def efim_rope_table_build(base, head_dim, max_position) -> np.ndarray:
    out = np.empty((max_position, head_dim), dtype=np.float32)
    st = load_library().efim_rope_table_build(float(base), head_dim, max_position, out.ctypes.data)
    if st != 0:
        raise EfimError(st, "efim_rope_table_build")
    return out


def efim_kv_append(cache: Cache, batch: Batch, rope, q, k_new, v_new, status=None, stream=None):
    st = load_library().efim_kv_append(ctypes.byref(cache.desc), ctypes.byref(batch.desc),
                                       ctypes.byref(rope.desc) if rope is not None else None,
                                       _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(status), _stream_ptr(stream))
    if st != 0:
        raise EfimError(st, "efim_kv_append")


def efim_prefill_workspace_bytes(cache: Cache, batch: Batch) -> int:
    return int(load_library().efim_prefill_workspace_bytes(ctypes.byref(cache.desc), ctypes.byref(batch.desc)))


def efim_prefill_plan(cache: Cache, batch: Batch) -> np.ndarray:
    """The work list of efim_append_prefill_attn for this batch as a host blob (uint8 array);
    pass it as `plan=` to run without planning, e.g. once per layer."""
    lib = load_library()
    n = int(lib.efim_prefill_plan_bytes(ctypes.byref(cache.desc), ctypes.byref(batch.desc)))
    if n == 0:
        raise EfimError(1, "efim_prefill_plan_bytes")
    blob = np.zeros(n, np.uint8)
    st = lib.efim_prefill_plan(ctypes.byref(cache.desc), ctypes.byref(batch.desc), blob.ctypes.data, n)
    if st != 0:
        raise EfimError(st, "efim_prefill_plan")
    return blob


def efim_append_prefill_attn(cache: Cache, batch: Batch, q, out, lse=None, sm_scale=0.0,
                             workspace=None, status=None, stream=None, plan=None, lists_resident=False):
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    lib = load_library()
    if plan is None:
        st = lib.efim_append_prefill_attn(ctypes.byref(cache.desc), ctypes.byref(batch.desc),
                                          _ptr(q), _ptr(out), _ptr(lse), float(sm_scale),
                                          _ptr(workspace), nbytes, _ptr(status), _stream_ptr(stream))
    else:
        st = lib.efim_append_prefill_attn_planned(ctypes.byref(cache.desc), ctypes.byref(batch.desc),
                                                  plan.ctypes.data, plan.nbytes, 1 if lists_resident else 0,
                                                  _ptr(q), _ptr(out), _ptr(lse),
                                                  float(sm_scale), _ptr(workspace), nbytes, _ptr(status),
                                                  _stream_ptr(stream))
    if st != 0:
        raise EfimError(st, "efim_append_prefill_attn")


def efim_append_prefill_step(cache: Cache, batch: Batch, rope, q, k_new, v_new, out, lse=None, sm_scale=0.0,
                             workspace=None, status=None, stream=None, plan=None, lists_resident=False):
    """kv_append of the new tokens' k/v and append-prefill attention with q rotated on load
    (q is not modified)."""
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    st = load_library().efim_append_prefill_step(
        ctypes.byref(cache.desc), ctypes.byref(batch.desc), ctypes.byref(rope.desc) if rope is not None else None,
        _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(lse), float(sm_scale),
        plan.ctypes.data if plan is not None else None, plan.nbytes if plan is not None else 0,
        1 if lists_resident else 0, _ptr(workspace), nbytes, _ptr(status), _stream_ptr(stream))
    if st != 0:
        raise EfimError(st, "efim_append_prefill_step")


def efim_selftest_bounded_wait(limit_ns: int, status, waited_ns=None, stream=None):
    st = load_library().efim_selftest_bounded_wait(int(limit_ns), _ptr(status), _ptr(waited_ns), _stream_ptr(stream))
    if st != 0:
        raise EfimError(st, "efim_selftest_bounded_wait")


def efim_decode_workspace_bytes(cache: Cache, batch: int, max_ctx_len: int) -> int:
    return int(load_library().efim_decode_workspace_bytes(ctypes.byref(cache.desc), batch, max_ctx_len))


def efim_decode_attn(cache: Cache, batch: int, d_ctx_len, max_ctx_len, d_block_table, q, out, lse=None,
                     sm_scale=0.0, workspace=None, status=None, stream=None):
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    st = load_library().efim_decode_attn(ctypes.byref(cache.desc), batch, _ptr(d_ctx_len), int(max_ctx_len),
                                         _ptr(d_block_table), int(d_block_table.shape[1]), _ptr(q), _ptr(out),
                                         _ptr(lse), float(sm_scale), _ptr(workspace), nbytes,
                                         _ptr(status), _stream_ptr(stream))
    if st != 0:
        raise EfimError(st, "efim_decode_attn")


def efim_decode_static_scratch_bytes() -> int:
    return int(load_library().efim_decode_static_scratch_bytes())


def efim_decode_attn_static(cache: Cache, batch: int, d_ctx_len, max_ctx_len, d_block_table, q, out, lse=None,
                            sm_scale=0.0, status=None, stream=None):
    """efim_decode_attn for callers that cannot allocate a workspace: the chunk
    partials use the library's fixed 8 MiB array (shared by all calls on the device)."""
    st = load_library().efim_decode_attn_static(ctypes.byref(cache.desc), batch, _ptr(d_ctx_len), int(max_ctx_len),
                                                _ptr(d_block_table), int(d_block_table.shape[1]), _ptr(q),
                                                _ptr(out), _ptr(lse), float(sm_scale), _ptr(status),
                                                _stream_ptr(stream))
    if st != 0:
        raise EfimError(st, "efim_decode_attn_static")


def efim_prefill_launch_count(cache: Cache, batch: Batch) -> int:
    return int(load_library().efim_prefill_launch_count(ctypes.byref(cache.desc), ctypes.byref(batch.desc)))


def efim_decode_launch_count(cache: Cache, batch: int, max_ctx_len: int) -> int:
    return int(load_library().efim_decode_launch_count(ctypes.byref(cache.desc), batch, max_ctx_len))


class Frontend:
    """The host-side front end of include/efim.h (prompt transformation of Sec. 3.1 and
    page-granular cross-request KV reuse); every method is one C call on numpy arrays."""

    def __init__(self, tok_p, tok_s, tok_m, num_pages, page_size=16, rebase_inc_tokens=0):
        self._lib = load_library()
        self._fe = self._lib.efim_frontend_create(tok_p, tok_s, tok_m, rebase_inc_tokens, num_pages, page_size)
        if not self._fe:
            raise EfimError(1, "efim_frontend_create")
        self.page_size = page_size

    def close(self):
        if self._fe:
            self._lib.efim_frontend_destroy(self._fe)
            self._fe = None

    def __del__(self):
        self.close()

    def transform(self, user, prefix, suffix):
        """-> (prompt int32 array, format, inc_len)."""
        prefix = np.ascontiguousarray(prefix, np.int32)
        suffix = np.ascontiguousarray(suffix, np.int32)
        out = np.empty(len(prefix) + len(suffix) + 3, np.int32)
        n, fmt, inc = c_int32(), c_int32(), c_int32()
        st = self._lib.efim_frontend_transform(self._fe, int(user), prefix.ctypes.data, len(prefix),
                                               suffix.ctypes.data, len(suffix), out.ctypes.data, len(out),
                                               ctypes.addressof(n), ctypes.addressof(fmt), ctypes.addressof(inc))
        if st != 0:
            raise EfimError(st, "efim_frontend_transform")
        return out[:n.value], fmt.value, inc.value

    def admit(self, prompt, reserve_tokens, block_table_row):
        """Fills `block_table_row` (int32 numpy row) -> (handle, cached_len, pages used)."""
        prompt = np.ascontiguousarray(prompt, np.int32)
        assert block_table_row.dtype == np.int32 and block_table_row.flags.c_contiguous
        cached, npages, handle = c_int32(), c_int32(), ctypes.c_int64()
        st = self._lib.efim_frontend_admit(self._fe, prompt.ctypes.data, len(prompt), int(reserve_tokens),
                                           block_table_row.ctypes.data, len(block_table_row),
                                           ctypes.addressof(cached), ctypes.addressof(npages),
                                           ctypes.addressof(handle))
        if st != 0:
            raise EfimError(st, "efim_frontend_admit")
        return handle.value, cached.value, npages.value

    def finish(self, handle, tokens):
        tokens = np.ascontiguousarray(tokens, np.int32)
        st = self._lib.efim_frontend_finish(self._fe, int(handle), tokens.ctypes.data, len(tokens))
        if st != 0:
            raise EfimError(st, "efim_frontend_finish")

    def stats(self):
        out = np.zeros(4, np.int64)
        self._lib.efim_frontend_stats(self._fe, out.ctypes.data)
        return dict(prompt_tokens=int(out[0]), hit_tokens=int(out[1]), evictions=int(out[2]), free_pages=int(out[3]))


def efim_decode_step(cache: Cache, batch: int, d_ctx_len, max_ctx_len, d_block_table, rope, q, k_new, v_new, out,
                     lse=None, sm_scale=0.0, workspace=None, status=None, stream=None):
    """kv_append of one token per row and decode attention in one launch (q is not modified)."""
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    st = load_library().efim_decode_step(ctypes.byref(cache.desc), batch, _ptr(d_ctx_len), int(max_ctx_len),
                                         _ptr(d_block_table), int(d_block_table.shape[1]),
                                         ctypes.byref(rope.desc) if rope is not None else None,
                                         _ptr(q), _ptr(k_new), _ptr(v_new), _ptr(out), _ptr(lse), float(sm_scale),
                                         _ptr(workspace), nbytes, _ptr(status), _stream_ptr(stream))
    if st != 0:
        raise EfimError(st, "efim_decode_step")
