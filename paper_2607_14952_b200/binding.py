"""ctypes binding over the C ABI declared in include/ls.h.

Argument marshalling only: every step of the path runs in the library's kernels.
Functions carry the C names.  Tensors are torch tensors (device memory and streams
come from torch); page tables and plan arrays are numpy.  The library must be built
(`build.build_library`); loading fails loudly when it is missing -- there is no
CPU fallback.
"""
import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

LS_OK = 0
LS_ERR_INVALID_ARG, LS_ERR_BAD_PAGE_TABLE, LS_ERR_UNSUPPORTED_SHAPE, LS_ERR_ALIGNMENT = -1, -2, -3, -4
LS_ERR_WORKSPACE, LS_ERR_STALE, LS_ERR_CUDA, LS_ERR_TIMEOUT, LS_ERR_NONFINITE = -5, -6, -7, -8, -9
LS_SHARD_CONTIGUOUS, LS_SHARD_CYCLIC, LS_SHARD_ZIGZAG = 0, 1, 2
LS_WORKSPACE_FWD, LS_WORKSPACE_BWD, LS_WORKSPACE_FWD_MERGED = 0, 1, 2
LS_FLAG_ADD_SUFFIX_GRAD = 1
LS_FLAG_NO_RESPONSE_BLOCK = 2
LS_KERNEL_FWD, LS_KERNEL_BWD_DQ, LS_KERNEL_BWD_DK, LS_KERNEL_BWD_DV = 0, 1, 2, 3


class ls_pages_desc_t(C.Structure):
    _fields_ = [("prefix_len", C.c_int64), ("page_size", C.c_int32), ("num_shards", C.c_int32),
                ("shard_policy", C.c_int32), ("num_kv_heads", C.c_int32), ("dim_k", C.c_int32),
                ("dim_v", C.c_int32), ("v_aliases_k", C.c_int32), ("stream_budget_kib", C.c_int32),
                ("num_phys_pages", C.c_int64), ("k_pool", C.c_void_p), ("v_pool", C.c_void_p),
                ("k_stride_page", C.c_int64), ("k_stride_tok", C.c_int64), ("k_stride_head", C.c_int64),
                ("v_stride_page", C.c_int64), ("v_stride_tok", C.c_int64), ("v_stride_head", C.c_int64)]


class ls_attn_params_t(C.Structure):
    _fields_ = [("R", C.c_int32), ("num_q_heads", C.c_int32), ("scale", C.c_float), ("flags", C.c_int32),
                ("generation", C.c_uint64)]


class ls_dsa_desc_t(C.Structure):
    _fields_ = [("R", C.c_int32), ("num_q_heads", C.c_int32), ("num_index_heads", C.c_int32),
                ("index_dim", C.c_int32), ("top_k", C.c_int32), ("reserved", C.c_int32), ("ki_pool", C.c_void_p),
                ("ki_stride_page", C.c_int64), ("ki_stride_tok", C.c_int64), ("gathered", C.c_void_p)]


class LsError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, lib().ls_status_string(status).decode(), status))


_LIB = None


def lib():
    """Loads (building first if the sources are newer) the shared library."""
    global _LIB
    if _LIB is None:
        path = _build.build_library() if os.environ.get("LS_NO_BUILD") != "1" else _build.LIB
        if not os.path.exists(path):
            raise RuntimeError("libls_replay.so is missing: run paper_2607_14952_b200/build.py")
        L = C.CDLL(path)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.ls_prefix_pages_build.argtypes = [C.POINTER(ls_pages_desc_t), vp, C.POINTER(vp)]
        L.ls_prefix_pages_export.argtypes = [vp, vp, vp, vp, vp, vp]
        L.ls_prefix_pages_checksum.argtypes = [vp, vp, C.POINTER(C.c_uint64), vp]
        L.ls_prefix_pages_destroy.argtypes = [vp]
        L.ls_replay_attn_workspace_bytes.argtypes = [vp, C.POINTER(ls_attn_params_t), C.c_int]
        L.ls_replay_attn_workspace_bytes.restype = C.c_size_t
        L.ls_replay_attn_fwd.argtypes = [vp, C.POINTER(ls_attn_params_t), vp, vp, vp, vp, vp, vp, C.c_size_t, vp, vp]
        L.ls_lse_merge.argtypes = [i32, i64, i32, vp, vp, vp, vp, vp, vp, vp]
        L.ls_lse_merge_bf16_numerator.argtypes = [i32, i64, i32, vp, vp, vp, vp, vp, vp, vp]
        L.ls_replay_attn_fwd_merged.argtypes = [vp, C.POINTER(ls_attn_params_t), vp, vp, vp, vp, vp, vp, vp, C.c_size_t,
                                                vp, vp]
        L.ls_suffix_pages_reserve.argtypes = [vp, i32, i32, vp, vp]
        L.ls_suffix_pages_append.argtypes = [vp, i32, vp, vp, vp, vp]
        L.ls_suffix_pages_pop.argtypes = [vp]
        L.ls_dsa_gathered_bytes.argtypes = [vp, C.POINTER(ls_dsa_desc_t)]
        L.ls_dsa_gathered_bytes.restype = C.c_size_t
        L.ls_dsa_plan_create.argtypes = [vp, C.POINTER(ls_dsa_desc_t), C.POINTER(vp)]
        L.ls_dsa_plan_destroy.argtypes = [vp]
        L.ls_dsa_selected_count.argtypes = [vp]
        L.ls_dsa_selected_count.restype = C.c_int32
        L.ls_dsa_workspace_bytes.argtypes = [vp, C.c_int]
        L.ls_dsa_workspace_bytes.restype = C.c_size_t
        L.ls_dsa_index_scores.argtypes = [vp, vp, vp, vp, vp, vp]
        L.ls_dsa_topk.argtypes = [vp, vp, vp, vp]
        L.ls_dsa_attn_fwd.argtypes = [vp, vp, C.c_float, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp, vp]
        L.ls_dsa_attn_bwd.argtypes = [vp, C.c_float, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, C.c_size_t, vp, vp]
        for f in ("ls_dsa_plan_create", "ls_dsa_plan_destroy", "ls_dsa_index_scores", "ls_dsa_topk", "ls_dsa_attn_fwd",
                  "ls_dsa_attn_bwd"):
            getattr(L, f).restype = C.c_int
        L.ls_pages_generation.argtypes = [vp]
        L.ls_pages_generation.restype = C.c_uint64
        L.ls_suffix_pages_tokens.argtypes = [vp]
        L.ls_suffix_pages_tokens.restype = C.c_int64
        L.ls_replay_attn_bwd.argtypes = [vp, C.POINTER(ls_attn_params_t), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                         C.c_size_t, vp, vp]
        L.ls_replay_attn_bwd_static.argtypes = [vp, C.POINTER(ls_attn_params_t), vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                                vp, vp]
        L.ls_replay_attn_bwd_static.restype = C.c_int
        L.ls_replay_attn_bwd_static_capacity.argtypes = []
        L.ls_replay_attn_bwd_static_capacity.restype = C.c_size_t
        L.ls_selftest_bounded_wait.argtypes = [vp, C.c_uint64, vp]
        L.ls_selftest_bounded_wait.restype = C.c_int
        L.ls_profile_arm_events.argtypes = [C.c_int, vp, vp]
        L.ls_profile_arm_events.restype = C.c_int
        L.ls_status_string.argtypes = [C.c_int]
        L.ls_status_string.restype = C.c_char_p
        for f in ("ls_prefix_pages_build", "ls_prefix_pages_export", "ls_prefix_pages_checksum",
                  "ls_prefix_pages_destroy", "ls_replay_attn_fwd", "ls_lse_merge", "ls_lse_merge_bf16_numerator",
                  "ls_replay_attn_bwd",
                  "ls_replay_attn_fwd_merged", "ls_suffix_pages_reserve", "ls_suffix_pages_append",
                  "ls_suffix_pages_pop"):
            getattr(L, f).restype = C.c_int
        _LIB = L
    return _LIB


def _check(status, where):
    if status != LS_OK:
        raise LsError(status, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


class Pages:
    """Owner of an ls_pages_t handle (and of references to the pool tensors)."""

    def __init__(self, handle, desc, k_pool, v_pool):
        self.handle, self.desc, self.k_pool, self.v_pool = handle, desc, k_pool, v_pool
        self.num_logical_pages = (desc.prefix_len + desc.page_size - 1) // desc.page_size

    def close(self):
        if self.handle:
            lib().ls_prefix_pages_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def ls_prefix_pages_build(prefix_len, page_size, num_shards, num_kv_heads, dim_k, dim_v, num_phys_pages,
                          page_table=None, k_pool=None, v_pool=None, shard_policy=LS_SHARD_CONTIGUOUS,
                          v_aliases_k=False, stream_budget_kib=0):
    """k_pool/v_pool: bf16 CUDA tensors [num_phys_pages, page_size, num_kv_heads, dim] (last dim dense) or
    None for a host-only plan.  page_table: int32 numpy array or None (identity)."""
    d = ls_pages_desc_t()
    d.prefix_len, d.page_size, d.num_shards, d.shard_policy = prefix_len, page_size, num_shards, shard_policy
    d.num_kv_heads, d.dim_k, d.dim_v, d.v_aliases_k = num_kv_heads, dim_k, dim_v, int(bool(v_aliases_k))
    d.num_phys_pages = num_phys_pages
    d.stream_budget_kib = stream_budget_kib
    if k_pool is not None:
        assert k_pool.dtype == torch.bfloat16 and k_pool.stride(-1) == 1
        d.k_pool = k_pool.data_ptr()
        d.k_stride_page, d.k_stride_tok, d.k_stride_head = k_pool.stride(0), k_pool.stride(1), k_pool.stride(2)
        if v_pool is not None and not v_aliases_k:
            assert v_pool.dtype == torch.bfloat16 and v_pool.stride(-1) == 1
            d.v_pool = v_pool.data_ptr()
            d.v_stride_page, d.v_stride_tok, d.v_stride_head = v_pool.stride(0), v_pool.stride(1), v_pool.stride(2)
    tbl = None
    if page_table is not None:
        tbl = np.ascontiguousarray(page_table, dtype=np.int32)
    out = C.c_void_p()
    st = lib().ls_prefix_pages_build(C.byref(d), None if tbl is None else tbl.ctypes.data_as(C.c_void_p), C.byref(out))
    _check(st, "ls_prefix_pages_build")
    return Pages(out, d, k_pool, v_pool)


def ls_prefix_pages_export(pages):
    Np, S = pages.num_logical_pages, pages.desc.num_shards
    table = np.zeros(Np, np.int32)
    owner = np.zeros(Np, np.int32)
    offs = np.zeros(S + 1, np.int64)
    order = np.zeros(Np, np.int32)
    toks = np.zeros(S, np.int64)
    p = lambda a: a.ctypes.data_as(C.c_void_p)
    _check(lib().ls_prefix_pages_export(pages.handle, p(table), p(owner), p(offs), p(order), p(toks)),
           "ls_prefix_pages_export")
    return dict(page_table=table, shard_of_page=owner, shard_page_offset=offs, shard_logical_pages=order,
                shard_tokens=toks)


def ls_prefix_pages_checksum(pages):
    scratch = torch.zeros(1, dtype=torch.int64, device=pages.k_pool.device)
    out = C.c_uint64(0)
    _check(lib().ls_prefix_pages_checksum(pages.handle, _ptr(scratch), C.byref(out), _stream()),
           "ls_prefix_pages_checksum")
    return int(out.value)


def _params(R, Hq, scale, flags=0, generation=0):
    return ls_attn_params_t(R, Hq, float(scale), flags, generation)


def ls_replay_attn_workspace_bytes(pages, R, Hq, scale, which):
    prm = _params(R, Hq, scale)
    return int(lib().ls_replay_attn_workspace_bytes(pages.handle, C.byref(prm), which))


def ls_replay_attn_fwd(pages, q, k_resp, v_resp, scale, o_part=None, lse_part=None, status=None, flags=0,
                       workspace=None, generation=0):
    """Returns (o_part [(S+1),R,Hq,Dv] fp32, lse_part [(S+1),R,Hq] fp32)."""
    R, Hq, _ = q.shape
    S, Dv = pages.desc.num_shards, pages.desc.dim_v
    if o_part is None:
        o_part = torch.empty((S + 1, R, Hq, Dv), dtype=torch.float32, device=q.device)
    if lse_part is None:
        lse_part = torch.empty((S + 1, R, Hq), dtype=torch.float32, device=q.device)
    prm = _params(R, Hq, scale, flags, generation)
    if workspace is None:
        nbytes = ls_replay_attn_workspace_bytes(pages, R, Hq, scale, LS_WORKSPACE_FWD)
        if nbytes:
            workspace = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    st = lib().ls_replay_attn_fwd(pages.handle, C.byref(prm), _ptr(q), _ptr(k_resp), _ptr(v_resp), _ptr(o_part),
                                  _ptr(lse_part), _ptr(workspace), 0 if workspace is None else workspace.numel(),
                                  _ptr(status), _stream())
    _check(st, "ls_replay_attn_fwd")
    return o_part, lse_part


def ls_lse_merge(o_part, lse_part, o_bf16=None, o_f32=None, lse=None, want_bf16=True, want_f32=True, status=None,
                 bf16_numerator=False):
    """o_part [parts, ..., Dv] fp32, lse_part [parts, ...] fp32 -> (o_bf16, o_f32, lse).
    bf16_numerator: ls_lse_merge_bf16_numerator (the numerator summed in bf16)."""
    parts, dv = o_part.shape[0], o_part.shape[-1]
    rows = lse_part[0].numel()
    shape = tuple(o_part.shape[1:])
    if o_bf16 is None and want_bf16:
        o_bf16 = torch.empty(shape, dtype=torch.bfloat16, device=o_part.device)
    if o_f32 is None and want_f32:
        o_f32 = torch.empty(shape, dtype=torch.float32, device=o_part.device)
    if lse is None:
        lse = torch.empty(shape[:-1], dtype=torch.float32, device=o_part.device)
    fn = lib().ls_lse_merge_bf16_numerator if bf16_numerator else lib().ls_lse_merge
    st = fn(parts, rows, dv, _ptr(o_part), _ptr(lse_part), _ptr(o_bf16), _ptr(o_f32), _ptr(lse), _ptr(status), _stream())
    _check(st, "ls_lse_merge")
    return o_bf16, o_f32, lse


def ls_replay_attn_fwd_merged(pages, q, k_resp, v_resp, scale, o_bf16=None, o_f32=None, lse=None, status=None,
                              workspace=None, want_bf16=True, generation=0):
    """Forward with the merge folded in: returns (o_bf16 [R,Hq,Dv] or None, o_f32, lse [R,Hq])."""
    R, Hq, _ = q.shape
    Dv = pages.desc.dim_v
    if o_bf16 is None and want_bf16:
        o_bf16 = torch.empty((R, Hq, Dv), dtype=torch.bfloat16, device=q.device)
    if o_f32 is None:
        o_f32 = torch.empty((R, Hq, Dv), dtype=torch.float32, device=q.device)
    if lse is None:
        lse = torch.empty((R, Hq), dtype=torch.float32, device=q.device)
    prm = _params(R, Hq, scale, 0, generation)
    if workspace is None:
        nbytes = ls_replay_attn_workspace_bytes(pages, R, Hq, scale, LS_WORKSPACE_FWD_MERGED)
        workspace = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=q.device)
    st = lib().ls_replay_attn_fwd_merged(pages.handle, C.byref(prm), _ptr(q), _ptr(k_resp), _ptr(v_resp),
                                         _ptr(o_bf16), _ptr(o_f32), _ptr(lse), _ptr(workspace), workspace.numel(),
                                         _ptr(status), _stream())
    _check(st, "ls_replay_attn_fwd_merged")
    return o_bf16, o_f32, lse


def ls_suffix_pages_reserve(pages, max_blocks, max_pages, dk_grad=None, dv_grad=None):
    """dk_grad / dv_grad: fp32 CUDA tensors [max_pages, page_size, Hkv, Dk|Dv] or None (forward only)."""
    _check(lib().ls_suffix_pages_reserve(pages.handle, max_blocks, max_pages, _ptr(dk_grad), _ptr(dv_grad)),
           "ls_suffix_pages_reserve")
    pages.grad_pages = (dk_grad, dv_grad)


def ls_suffix_pages_append(pages, phys_pages, k_block, v_block=None):
    """Appends one block of response K/V ([n,Hkv,D] bf16) into the given free pool pages."""
    ids = np.ascontiguousarray(phys_pages, dtype=np.int32)
    _check(lib().ls_suffix_pages_append(pages.handle, k_block.shape[0], ids.ctypes.data_as(C.c_void_p), _ptr(k_block),
                                        _ptr(v_block), _stream()), "ls_suffix_pages_append")


def ls_suffix_pages_pop(pages):
    _check(lib().ls_suffix_pages_pop(pages.handle), "ls_suffix_pages_pop")


def ls_pages_generation(pages):
    return int(lib().ls_pages_generation(pages.handle))


def ls_suffix_pages_tokens(pages):
    return int(lib().ls_suffix_pages_tokens(pages.handle))


def ls_replay_attn_bwd(pages, q, k_resp, v_resp, o_f32, lse, d_o, scale, workspace=None, dq=None, dk_resp=None,
                       dv_resp=None, status=None, flags=0, generation=0):
    """Returns (dq, dk_resp, dv_resp) in bf16."""
    R, Hq, _ = q.shape
    if workspace is None:
        nbytes = ls_replay_attn_workspace_bytes(pages, R, Hq, scale, LS_WORKSPACE_BWD)
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    if dq is None:
        dq = torch.empty_like(q)
    if dk_resp is None and k_resp is not None:       # (no response block: nothing to return for its keys)
        dk_resp = torch.empty_like(k_resp)
    if dv_resp is None and v_resp is not None:
        dv_resp = torch.empty_like(v_resp)
    prm = _params(R, Hq, scale, flags, generation)
    st = lib().ls_replay_attn_bwd(pages.handle, C.byref(prm), _ptr(q), _ptr(k_resp), _ptr(v_resp), _ptr(o_f32),
                                  _ptr(lse), _ptr(d_o), _ptr(dq), _ptr(dk_resp), _ptr(dv_resp), _ptr(workspace),
                                  workspace.numel(), _ptr(status), _stream())
    _check(st, "ls_replay_attn_bwd")
    return dq, dk_resp, dv_resp


def ls_replay_attn_bwd_static_capacity():
    return int(lib().ls_replay_attn_bwd_static_capacity())


def ls_replay_attn_bwd_static(pages, q, k_resp, v_resp, o_f32, lse, d_o, scale, dq, dk_resp, dv_resp, status=None):
    """Backward that takes no workspace: its scratch is a fixed array inside the library, for
    callers that have no device memory left to lend (page pool sized to the whole GPU, or an
    allocator that owns it all).  Outputs must be passed in; nothing is allocated here."""
    R, Hq, _ = q.shape
    prm = _params(R, Hq, scale)
    st = lib().ls_replay_attn_bwd_static(pages.handle, C.byref(prm), _ptr(q), _ptr(k_resp), _ptr(v_resp),
                                         _ptr(o_f32), _ptr(lse), _ptr(d_o), _ptr(dq), _ptr(dk_resp),
                                         _ptr(dv_resp), _ptr(status), _stream())
    _check(st, "ls_replay_attn_bwd_static")
    return dq, dk_resp, dv_resp


def ls_profile_arm_events(kernel, start_event, stop_event):
    """start/stop: torch.cuda.Event(enable_timing=True) that the next launch of `kernel` records."""
    for e in (start_event, stop_event):
        if e is not None and not e.cuda_event:
            e.record()          # torch creates the CUDA event lazily; force it into existence
    a = None if start_event is None else C.c_void_p(start_event.cuda_event)
    b = None if stop_event is None else C.c_void_p(stop_event.cuda_event)
    _check(lib().ls_profile_arm_events(kernel, a, b), "ls_profile_arm_events")


def ls_selftest_bounded_wait(status, budget_ns):
    """Runs the bounded-wait self test; `status` is a zeroed int32 CUDA tensor."""
    _check(lib().ls_selftest_bounded_wait(_ptr(status), int(budget_ns), _stream()), "ls_selftest_bounded_wait")


class DsaPlan:
    """Owner of an ls_dsa_plan_t handle, of its gathered buffer and of references to the pools."""

    def __init__(self, handle, pages, ki_pool, gathered, desc):
        self.handle, self.pages, self.ki_pool, self.gathered, self.desc = handle, pages, ki_pool, gathered, desc
        self.count = int(lib().ls_dsa_selected_count(handle))

    def close(self):
        if self.handle:
            lib().ls_dsa_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def ls_dsa_plan_create(pages, ki_pool, R, num_q_heads, num_index_heads, top_k):
    """ki_pool: bf16 CUDA tensor [num_phys_pages, page_size, index_dim] (indexer-key pages, same page
    ids as the latent pool).  Allocates the gathered buffer with torch (device memory only)."""
    d = ls_dsa_desc_t()
    d.R, d.num_q_heads, d.num_index_heads, d.index_dim, d.top_k = R, num_q_heads, num_index_heads, ki_pool.shape[-1], top_k
    assert ki_pool.dtype == torch.bfloat16 and ki_pool.stride(-1) == 1
    d.ki_pool = ki_pool.data_ptr()
    d.ki_stride_page, d.ki_stride_tok = ki_pool.stride(0), ki_pool.stride(1)
    nbytes = int(lib().ls_dsa_gathered_bytes(pages.handle, C.byref(d)))
    gathered = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=ki_pool.device)
    d.gathered = gathered.data_ptr()
    out = C.c_void_p()
    _check(lib().ls_dsa_plan_create(pages.handle, C.byref(d), C.byref(out)), "ls_dsa_plan_create")
    return DsaPlan(out, pages, ki_pool, gathered, d)


def ls_dsa_index_scores(plan, q_index, w_index, scores=None, status=None):
    """q_index [R, H_I, 128] bf16, w_index [R, H_I] fp32 -> scores [R, P] fp32."""
    P = plan.pages.desc.prefix_len
    if scores is None:
        scores = torch.empty((plan.desc.R, P), dtype=torch.float32, device=q_index.device)
    _check(lib().ls_dsa_index_scores(plan.handle, _ptr(q_index), _ptr(w_index), _ptr(scores), _ptr(status), _stream()),
           "ls_dsa_index_scores")
    return scores


def ls_dsa_topk(plan, scores, sel=None):
    """scores [R, P] fp32 -> sel [R, count] int32: the selected prefix positions, ascending."""
    if sel is None:
        sel = torch.empty((plan.desc.R, plan.count), dtype=torch.int32, device=scores.device)
    _check(lib().ls_dsa_topk(plan.handle, _ptr(scores), _ptr(sel), _stream()), "ls_dsa_topk")
    return sel


def ls_dsa_attn_fwd(plan, sel, q, k_resp, v_resp, scale, status=None, workspace=None):
    """Returns (o_bf16, o_f32, lse) of the sparse operator."""
    R, Hq, _ = q.shape
    dv = plan.pages.desc.dim_v
    o_bf16 = torch.empty((R, Hq, dv), dtype=torch.bfloat16, device=q.device)
    o_f32 = torch.empty((R, Hq, dv), dtype=torch.float32, device=q.device)
    lse = torch.empty((R, Hq), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = torch.empty(int(lib().ls_dsa_workspace_bytes(plan.handle, LS_WORKSPACE_FWD)), dtype=torch.uint8,
                                device=q.device)
    _check(lib().ls_dsa_attn_fwd(plan.handle, _ptr(sel), float(scale), _ptr(q), _ptr(k_resp), _ptr(v_resp), _ptr(o_bf16),
                                 _ptr(o_f32), _ptr(lse), _ptr(workspace), workspace.numel(), _ptr(status), _stream()),
           "ls_dsa_attn_fwd")
    return o_bf16, o_f32, lse


def ls_dsa_attn_bwd(plan, q, k_resp, v_resp, o_f32, lse, d_o, scale, status=None, workspace=None):
    """Returns (dq, dk_resp, dv_resp) with the selection of the plan's last forward held fixed."""
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k_resp), torch.empty_like(v_resp)
    if workspace is None:
        workspace = torch.empty(int(lib().ls_dsa_workspace_bytes(plan.handle, LS_WORKSPACE_BWD)), dtype=torch.uint8,
                                device=q.device)
    _check(lib().ls_dsa_attn_bwd(plan.handle, float(scale), _ptr(q), _ptr(k_resp), _ptr(v_resp), _ptr(o_f32), _ptr(lse),
                                 _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(workspace), workspace.numel(),
                                 _ptr(status), _stream()), "ls_dsa_attn_bwd")
    return dq, dk, dv
