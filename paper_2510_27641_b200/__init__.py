"""Python binding of libspecattn.so, the C-ABI CUDA library for the SpecAttn verification hot path.

Argument marshalling only: every function here fills the C structs of ``include/specattn.h``
from torch tensors (device memory, streams) and calls the entry point of the same name.  There
is no fallback: if the shared library has not been built the first call raises.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path
from typing import Sequence

import torch

__all__ = ["select_topp", "sparse_verify", "sparse_verify_static", "verify_workspace", "verify_workspace_bytes",
           "verify_step_host", "status_string", "kernel_launch_count", "library_path",
           "SelectArgs", "VerifyArgs", "StepHostArgs", "lib", "SpecAttnError",
           "ROW_OK", "ROW_INVALID_PROB", "ROW_OVERFLOW", "ROW_BAD_INDEX", "ROW_TIMEOUT",
           "VERIFY_LISTS_STABLE", "VERIFY_ENGINE_MMA_SYNC", "VERIFY_ENGINE_TCGEN05",
           "VERIFY_TEST_LOSE_ARRIVAL", "VERIFY_PAGE_LISTS", "SELECT_FORM_AUTO", "SELECT_FORM_CLUSTER",
           "SELECT_FORM_TWO_LAUNCH", "verify_plan",
           "verify_plan_buffer", "verify_plan_many"]

ROW_OK, ROW_INVALID_PROB, ROW_OVERFLOW, ROW_BAD_INDEX, ROW_TIMEOUT = 0, 1, 2, 4, 8
VERIFY_LISTS_STABLE = 1
VERIFY_ENGINE_MMA_SYNC = 2
VERIFY_ENGINE_TCGEN05 = 4
VERIFY_PAGE_LISTS = 8
SELECT_FORM_AUTO, SELECT_FORM_CLUSTER, SELECT_FORM_TWO_LAUNCH = 0, 1, 2
VERIFY_TEST_LOSE_ARRIVAL = 0x80000000   # test only: see include/specattn.h

_LIB_PATH = Path(__file__).resolve().parent / "libspecattn.so"
_lib = None


class SpecAttnError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


class SelectArgs(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_draft_layers", C.c_int32),
                ("n_target_layers", C.c_int32), ("batch", C.c_int32), ("n_draft_heads", C.c_int32),
                ("gamma", C.c_int32), ("n_groups", C.c_int32), ("L_stride", C.c_int64),
                ("draft_probs", C.POINTER(C.c_void_p)), ("kv_len", C.c_void_p),
                ("layer_map", C.POINTER(C.c_int32)), ("head_group", C.POINTER(C.c_int32)),
                ("p", C.c_float), ("idx", C.c_void_p), ("idx_stride", C.c_int64),
                ("counts", C.c_void_p), ("row_status", C.c_void_p), ("diag", C.c_void_p),
                ("per_step", C.c_int32), ("bisect_iters", C.c_int32), ("chunk", C.c_int32),
                ("form", C.c_int32), ("workspace", C.c_void_p), ("workspace_bytes", C.c_uint64)]


class VerifyArgs(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("batch", C.c_int32), ("n_q", C.c_int32),
                ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("page_size", C.c_int32), ("n_groups", C.c_int32), ("dense", C.c_int32),
                ("q", C.c_void_p), ("kv_pages", C.c_void_p), ("n_pages", C.c_int64),
                ("stride_page", C.c_int64), ("stride_kv", C.c_int64), ("stride_slot", C.c_int64),
                ("stride_head", C.c_int64), ("block_table", C.c_void_p),
                ("block_table_stride", C.c_int64), ("kv_len", C.c_void_p), ("idx", C.c_void_p),
                ("idx_stride", C.c_int64), ("counts", C.c_void_p), ("sm_scale", C.c_float),
                ("out", C.c_void_p), ("lse", C.c_void_p), ("status", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("flags", C.c_uint32),
                ("tail_len", C.c_int32), ("plan", C.c_void_p)]


class StepHostArgs(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_target_layers", C.c_int32),
                ("select", C.POINTER(SelectArgs)), ("draft_probs_host", C.POINTER(C.c_void_p)),
                ("verify", C.POINTER(VerifyArgs)), ("q_host", C.POINTER(C.c_void_p)),
                ("out_host", C.POINTER(C.c_void_p)), ("lse_host", C.POINTER(C.c_void_p))]


def library_path() -> Path:
    return _LIB_PATH


def lib() -> C.CDLL:
    """The loaded C-ABI library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with "
                               "`python -m paper_2510_27641_b200.build` (nvcc, sm_100a)")
        L = C.CDLL(str(_LIB_PATH))
        L.specattn_select_topp.argtypes = [C.POINTER(SelectArgs), C.c_void_p]
        L.specattn_select_topp.restype = C.c_int
        L.specattn_select_workspace_bytes.argtypes = [C.POINTER(SelectArgs)]
        L.specattn_select_workspace_bytes.restype = C.c_size_t
        L.specattn_sparse_verify.argtypes = [C.POINTER(VerifyArgs), C.c_void_p]
        L.specattn_sparse_verify.restype = C.c_int
        L.specattn_verify_workspace_bytes.argtypes = [C.POINTER(VerifyArgs)]
        L.specattn_verify_workspace_bytes.restype = C.c_size_t
        L.specattn_verify_workspace_init.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]
        L.specattn_verify_workspace_init.restype = C.c_int
        L.specattn_verify_plan_bytes.argtypes = [C.POINTER(VerifyArgs)]
        L.specattn_verify_plan_bytes.restype = C.c_size_t
        L.specattn_verify_plan.argtypes = [C.POINTER(VerifyArgs), C.c_void_p, C.c_size_t, C.c_void_p]
        L.specattn_verify_plan.restype = C.c_int
        L.specattn_verify_plan_many.argtypes = [C.POINTER(C.POINTER(VerifyArgs)), C.POINTER(C.c_void_p),
                                                C.POINTER(C.c_size_t), C.c_int32, C.c_void_p]
        L.specattn_verify_plan_many.restype = C.c_int
        L.specattn_sparse_verify_static.argtypes = [C.POINTER(VerifyArgs), C.c_void_p]
        L.specattn_sparse_verify_static.restype = C.c_int
        L.specattn_verify_step_host.argtypes = [C.POINTER(StepHostArgs), C.c_void_p]
        L.specattn_verify_step_host.restype = C.c_int
        L.specattn_status_string.argtypes = [C.c_int]
        L.specattn_status_string.restype = C.c_char_p
        L.specattn_kernel_launch_count.argtypes = []
        L.specattn_kernel_launch_count.restype = C.c_int64
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().specattn_status_string(int(code)).decode()


def kernel_launch_count() -> int:
    return int(lib().specattn_kernel_launch_count())


def _stream_ptr(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _ptr(t: torch.Tensor | None):
    return None if t is None else C.c_void_p(t.data_ptr())


def make_select_args(draft_probs: Sequence[torch.Tensor | None], kv_len: torch.Tensor,
                     layer_map: Sequence[int], p: float, *, n_groups: int = 1,
                     head_group: Sequence[int] | None = None, idx: torch.Tensor,
                     counts: torch.Tensor, row_status: torch.Tensor,
                     diag: torch.Tensor | None = None, per_step: bool = False, bisect_iters: int = 0,
                     chunk: int = 1, workspace: torch.Tensor | bool | None = True, form: int = 0):
    """Fills a SelectArgs.  Returns (args, keepalive) -- keepalive holds the host arrays the
    struct points at and must outlive the call.  workspace: a uint8 CUDA tensor, True (allocate
    what specattn_select_workspace_bytes asks for, if anything) or None / False (none: the
    one-launch cluster form)."""
    n_d = len(draft_probs)
    ref = next(t for t in draft_probs if t is not None)
    B, H, gamma, Ls = ref.shape
    for t in draft_probs:
        if t is not None:
            assert t.dtype == torch.float32 and t.is_contiguous() and tuple(t.shape) == (B, H, gamma, Ls)
    assert kv_len.dtype == torch.int32 and idx.dtype == torch.int32 and counts.dtype == torch.int32
    assert idx.is_contiguous() and idx.dim() == 4 and tuple(idx.shape[:3]) == (n_d, B, n_groups)
    ptrs = (C.c_void_p * n_d)(*[None if t is None else t.data_ptr() for t in draft_probs])
    lm = (C.c_int32 * len(layer_map))(*[int(x) for x in layer_map])
    hg = None if head_group is None else (C.c_int32 * len(head_group))(*[int(x) for x in head_group])
    a = SelectArgs()
    a.struct_size = C.sizeof(SelectArgs)
    a.n_draft_layers, a.n_target_layers, a.batch = n_d, len(layer_map), B
    a.n_draft_heads, a.gamma, a.n_groups, a.L_stride = H, gamma, n_groups, Ls
    a.draft_probs = ptrs
    a.kv_len = kv_len.data_ptr()
    a.layer_map = lm
    a.head_group = hg
    a.p = float(p)
    a.idx, a.idx_stride = idx.data_ptr(), idx.shape[3]
    a.counts, a.row_status = counts.data_ptr(), row_status.data_ptr()
    a.diag = None if diag is None else diag.data_ptr()
    a.per_step, a.bisect_iters, a.chunk = int(bool(per_step)), int(bisect_iters), int(chunk)
    a.form = int(form)
    if workspace is True:
        need = int(lib().specattn_select_workspace_bytes(C.byref(a)))
        workspace = torch.empty((need,), dtype=torch.uint8, device=ref.device) if need > 0 else None
    elif workspace is False:
        workspace = None
    if workspace is not None:
        assert workspace.dtype == torch.uint8 and workspace.is_contiguous()
        a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel()
    return a, (ptrs, lm, hg, draft_probs, kv_len, idx, counts, row_status, diag, workspace)


def select_topp(draft_probs: Sequence[torch.Tensor | None], kv_len: torch.Tensor,
                layer_map: Sequence[int], p: float, *, n_groups: int = 1,
                head_group: Sequence[int] | None = None, idx_stride: int | None = None,
                idx: torch.Tensor | None = None, counts: torch.Tensor | None = None,
                row_status: torch.Tensor | None = None, diag: torch.Tensor | None = None,
                want_diag: bool = False, per_step: bool = False, bisect_iters: int = 0, chunk: int = 1,
                workspace: torch.Tensor | bool | None = True, form: int = 0, stream=None):
    """specattn_select_topp.  draft_probs: per draft layer a float32 CUDA tensor
    [B, H_d, gamma, L_stride] (None for layers no target layer maps to).  Returns
    (idx [n_d,B,G,idx_stride] int32, counts [n_d,B,G], row_status [n_d,B,G], diag or None)."""
    n_d = len(draft_probs)
    ref = next(t for t in draft_probs if t is not None)
    B, _, _, Ls = ref.shape
    dev = ref.device
    stride = int(Ls if idx_stride is None else idx_stride)
    if idx is None:
        idx = torch.empty((n_d, B, n_groups, stride), dtype=torch.int32, device=dev)
    if counts is None:
        counts = torch.full((n_d, B, n_groups), -1, dtype=torch.int32, device=dev)
    if row_status is None:
        row_status = torch.full((n_d, B, n_groups), -1, dtype=torch.int32, device=dev)
    if diag is None and want_diag:
        diag = torch.zeros((n_d, B, n_groups, 4), dtype=torch.float64, device=dev)
    args, keep = make_select_args(draft_probs, kv_len, layer_map, p, n_groups=n_groups,
                                  head_group=head_group, idx=idx, counts=counts,
                                  row_status=row_status, diag=diag, per_step=per_step,
                                  bisect_iters=bisect_iters, chunk=chunk, workspace=workspace, form=form)
    rc = lib().specattn_select_topp(C.byref(args), _stream_ptr(stream))
    if rc != 0:
        raise SpecAttnError(rc, "specattn_select_topp")
    if keep[-1] is not None and stream is not None and workspace is True:
        keep[-1].record_stream(stream)   # allocated here, used on the caller's stream
    del keep
    return idx, counts, row_status, diag


def make_verify_args(q: torch.Tensor, kv_pages: torch.Tensor, kv_len: torch.Tensor, *,
                     block_table: torch.Tensor | None, pages_per_seq: int | None = None,
                     idx: torch.Tensor | None, counts: torch.Tensor | None, n_groups: int = 1,
                     dense: bool = False, sm_scale: float = 0.0, out: torch.Tensor,
                     lse: torch.Tensor, status: torch.Tensor | None = None,
                     workspace: torch.Tensor | None = None, flags: int = 0, tail_len: int = 0) -> VerifyArgs:
    """Fills a VerifyArgs from tensors.  kv_pages is [n_pages, 2, page_size, H_kv, d] bf16 (any
    strides with a unit innermost stride); idx [B, G, idx_stride] / counts [B, G] are the lists
    of ONE draft layer."""
    B, T, Hq, d = q.shape
    n_pages, two, page_size, Hkv, d2 = kv_pages.shape
    assert two == 2 and d2 == d and kv_pages.stride(4) == 1 and q.is_contiguous()
    assert q.dtype == torch.bfloat16 and kv_pages.dtype == torch.bfloat16
    a = VerifyArgs()
    a.struct_size = C.sizeof(VerifyArgs)
    a.batch, a.n_q, a.n_q_heads, a.n_kv_heads, a.head_dim = B, T, Hq, Hkv, d
    a.page_size, a.n_groups, a.dense = page_size, n_groups, int(bool(dense))
    a.q, a.kv_pages, a.n_pages = q.data_ptr(), kv_pages.data_ptr(), n_pages
    a.stride_page, a.stride_kv = kv_pages.stride(0), kv_pages.stride(1)
    a.stride_slot, a.stride_head = kv_pages.stride(2), kv_pages.stride(3)
    if block_table is not None:
        assert block_table.dtype == torch.int32 and block_table.stride(1) == 1
        a.block_table, a.block_table_stride = block_table.data_ptr(), block_table.stride(0)
    else:
        a.block_table, a.block_table_stride = None, int(pages_per_seq)
    a.kv_len = kv_len.data_ptr()
    if not dense:
        assert idx.dtype == torch.int32 and idx.dim() == 3 and idx.stride(2) == 1
        assert idx.stride(1) == idx.shape[2] and idx.stride(0) == idx.shape[1] * idx.shape[2]
        assert counts.dtype == torch.int32 and counts.is_contiguous()
        a.idx, a.idx_stride, a.counts = idx.data_ptr(), idx.shape[2], counts.data_ptr()
    a.sm_scale = float(sm_scale)
    a.flags = int(flags)
    a.tail_len = int(tail_len)
    a.out, a.lse = out.data_ptr(), lse.data_ptr()
    a.status = None if status is None else status.data_ptr()
    if workspace is not None:
        a.workspace, a.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    return a


def verify_workspace_bytes(args: VerifyArgs) -> int:
    return int(lib().specattn_verify_workspace_bytes(C.byref(args)))


def verify_workspace(args: VerifyArgs, device=None, stream=None) -> torch.Tensor:
    """Allocates (with torch) and initialises a workspace large enough for ``args``."""
    n = verify_workspace_bytes(args)
    if n == 0:
        raise SpecAttnError(-6, "specattn_verify_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device or torch.device("cuda"))
    rc = lib().specattn_verify_workspace_init(C.c_void_p(ws.data_ptr()), n, _stream_ptr(stream))
    if rc != 0:
        raise SpecAttnError(rc, "specattn_verify_workspace_init")
    return ws


def sparse_verify(q: torch.Tensor, kv_pages: torch.Tensor, kv_len: torch.Tensor, *,
                  block_table: torch.Tensor | None = None, pages_per_seq: int | None = None,
                  idx: torch.Tensor | None = None, counts: torch.Tensor | None = None,
                  n_groups: int = 1, dense: bool = False, sm_scale: float = 0.0,
                  out: torch.Tensor | None = None, lse: torch.Tensor | None = None,
                  status: torch.Tensor | None = None, workspace: torch.Tensor | None = None,
                  flags: int = 0, tail_len: int = 0, stream=None):
    """specattn_sparse_verify for one target layer.  Returns (out f32 [B,T,H_q,d], lse f32
    [B,T,H_q], status int32 [B])."""
    B, T, Hq, d = q.shape
    if out is None:
        out = torch.empty((B, T, Hq, d), dtype=torch.float32, device=q.device)
    if lse is None:
        lse = torch.empty((B, T, Hq), dtype=torch.float32, device=q.device)
    if status is None:
        status = torch.zeros((B,), dtype=torch.int32, device=q.device)
    args = make_verify_args(q, kv_pages, kv_len, block_table=block_table, pages_per_seq=pages_per_seq,
                            idx=idx, counts=counts, n_groups=n_groups, dense=dense, sm_scale=sm_scale,
                            out=out, lse=lse, status=status, workspace=workspace, flags=flags,
                            tail_len=tail_len)
    if workspace is None:
        workspace = verify_workspace(args, q.device, stream)
        args.workspace, args.workspace_bytes = workspace.data_ptr(), workspace.numel()
    rc = lib().specattn_sparse_verify(C.byref(args), _stream_ptr(stream))
    if rc != 0:
        raise SpecAttnError(rc, "specattn_sparse_verify")
    return out, lse, status


def verify_plan_buffer(args: VerifyArgs, device=None) -> torch.Tensor:
    """A device buffer large enough for the work partition of launches shaped like ``args``."""
    n = int(lib().specattn_verify_plan_bytes(C.byref(args)))
    if n == 0:
        raise SpecAttnError(-6, "specattn_verify_plan_bytes")
    dev = device if device is not None else torch.device("cuda", torch.cuda.current_device())
    return torch.zeros((n + 3) // 4, dtype=torch.int32, device=dev)


def verify_plan(args: VerifyArgs, plan: torch.Tensor, stream=None) -> None:
    """specattn_verify_plan: computes the work partition of launches shaped like ``args`` (same
    lists / kv_len, tail_len, shapes) into ``plan``; point ``args.plan`` at it afterwards."""
    rc = lib().specattn_verify_plan(C.byref(args), plan.data_ptr(), plan.numel() * plan.element_size(),
                                    _stream_ptr(stream))
    if rc != 0:
        raise SpecAttnError(rc, "specattn_verify_plan")


def verify_plan_many(args: Sequence[VerifyArgs], plans: Sequence[torch.Tensor], stream=None) -> None:
    """specattn_verify_plan_many: the plans of several launches in one kernel launch."""
    n = len(args)
    assert len(plans) == n
    a = (C.POINTER(VerifyArgs) * n)(*[C.pointer(x) for x in args])
    p = (C.c_void_p * n)(*[t.data_ptr() for t in plans])
    b = (C.c_size_t * n)(*[t.numel() * t.element_size() for t in plans])
    rc = lib().specattn_verify_plan_many(a, p, b, n, _stream_ptr(stream))
    if rc != 0:
        raise SpecAttnError(rc, "specattn_verify_plan_many")


def sparse_verify_static(args: VerifyArgs, stream=None) -> None:
    """specattn_sparse_verify_static: the same attention call for code that may not allocate
    device memory (plug-ins handed only their inputs and outputs, engines whose pool owns the
    whole GPU).  ``args`` is a filled VerifyArgs; its workspace fields are ignored because the
    scratch is a fixed array inside the library.  Calls on one device share that array, so
    they must not overlap on the GPU."""
    rc = lib().specattn_sparse_verify_static(C.byref(args), _stream_ptr(stream))
    if rc != 0:
        raise SpecAttnError(rc, "specattn_sparse_verify_static")


def verify_step_host(select_args: SelectArgs, draft_probs_host: Sequence[torch.Tensor | None],
                     verify_args: Sequence[VerifyArgs], q_host: Sequence[torch.Tensor],
                     out_host: Sequence[torch.Tensor], lse_host: Sequence[torch.Tensor], stream=None):
    """specattn_verify_step_host: one whole step from (pinned) host tensors; see the header."""
    n = len(verify_args)
    a = StepHostArgs()
    a.struct_size = C.sizeof(StepHostArgs)
    a.n_target_layers = n
    a.select = C.pointer(select_args)
    dp = (C.c_void_p * len(draft_probs_host))(*[None if t is None else t.data_ptr() for t in draft_probs_host])
    va = (VerifyArgs * max(n, 1))(*verify_args)
    qh = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in q_host])
    oh = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in out_host])
    lh = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in lse_host])
    a.draft_probs_host, a.verify, a.q_host, a.out_host, a.lse_host = dp, va, qh, oh, lh
    rc = lib().specattn_verify_step_host(C.byref(a), _stream_ptr(stream))
    if rc != 0:
        raise SpecAttnError(rc, "specattn_verify_step_host")
