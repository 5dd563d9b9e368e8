"""ctypes binding of libpivot.so: argument marshalling only.

Every function below has the name and argument order of the C entry point it forwards to
(include/pivot.h); tensors are torch tensors whose device pointers are passed through.  torch
is used for device memory and streams, nothing else: all arithmetic runs in the library's CUDA
kernels.  Importing this module fails loudly when the shared library has not been built.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# PIVOT_LIB selects another build of the same sources that sits next to the default one
# (libpivot_<name>.so from build.build_variant, e.g. the checked -DPIVOT_DEBUG build).
LIB_PATH = os.path.join(_HERE, os.path.basename(os.environ.get("PIVOT_LIB", "libpivot.so")))

BF16, FP8_E4M3 = 0, 1
REUSE, REFINE = 0, 1
POOL_MEAN, POOL_FIRST, POOL_LAST = 0, 1, 2
OK = 0

SYMBOLS = [
    "pivot_workspace_bytes", "pivot_decode_workspace_bytes", "pivot_set_workspace", "pivot_index_prefill", "pivot_index_prefill_ex",
    "pivot_index_prefill_varlen",
    "pivot_index_decode", "pivot_index_decode_ex", "pivot_index_decode_paged", "dense_index", "dense_index_ex", "dense_index_static",
    "pivot_prefill_host_arena_bytes", "pivot_index_prefill_host", "pivot_device_status",
    "pivot_stage_timing", "pivot_stage_times", "pivot_launch_count_reset", "pivot_status_str", "pivot_last_cuda_error",
    "dense_index_decode", "dense_index_decode_ex", "pivot_debug_wait_expiry", "pivot_debug_mma_model", "pivot_debug_key_stream", "pivot_debug_counters", "pivot_merge_topk",
]
DEV_OK, DEV_WAIT_EXPIRED, DEV_CAND_OVERFLOW, DEV_BAD_POS, DEV_BOUNDS = 0, 1, 2, 3, 4


class pivot_tensor(C.Structure):
    _fields_ = [("data", C.c_void_p), ("scale", C.c_void_p), ("dtype", C.c_int), ("stride_row", C.c_size_t)]


class pivot_opts(C.Structure):
    _fields_ = [("guard_len", C.c_int), ("pool", C.c_int), ("dbg_cand", C.c_void_p),
                ("dbg_scores", C.c_void_p), ("dbg_cand_scores", C.c_void_p),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("impl", C.c_int),
                ("row_begin", C.c_int), ("row_end", C.c_int), ("W", C.c_int), ("cand_in", C.c_void_p)]


class PivotError(RuntimeError):
    pass


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2607_24593_b200.build` "
            "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    T, O, I, P, S = C.POINTER(pivot_tensor), C.POINTER(pivot_opts), C.c_int, C.c_void_p, C.c_size_t
    lib.pivot_workspace_bytes.restype = S
    lib.pivot_workspace_bytes.argtypes = [I, I, I, I]
    lib.pivot_decode_workspace_bytes.restype = S
    lib.pivot_decode_workspace_bytes.argtypes = [I, I, I, I, I]
    lib.pivot_set_workspace.argtypes = [P, S]
    lib.pivot_index_prefill.argtypes = [T, P, T, I, I, I, I, I, I, I, P, P]
    lib.pivot_index_prefill_ex.argtypes = [T, P, T, I, I, I, I, I, I, I, P, P, O]
    lib.pivot_index_prefill_varlen.argtypes = [T, P, T, C.POINTER(C.c_int32), I, I, I, I, I, I, I, P, P, O]
    lib.pivot_index_decode.argtypes = [T, P, T, P, I, I, I, I, I, I, I, I, P, P]
    lib.pivot_index_decode_ex.argtypes = [T, P, T, P, I, I, I, I, I, I, I, I, P, P, O]
    lib.pivot_index_decode_paged.argtypes = [T, P, T, P, P, I, I, I, I, I, I, I, I, I, P, P, O]
    lib.dense_index.argtypes = [T, P, T, I, I, I, I, P, P]
    lib.dense_index_ex.argtypes = [T, P, T, I, I, I, I, P, P, O]
    lib.dense_index_static.argtypes = [T, P, T, I, I, I, I, P, P]
    lib.dense_index_decode.argtypes = [T, P, T, P, I, I, I, I, I, I, P, P]
    lib.dense_index_decode_ex.argtypes = [T, P, T, P, I, I, I, I, I, I, P, P, O]
    lib.pivot_debug_wait_expiry.argtypes = [C.c_ulonglong, P]
    lib.pivot_debug_mma_model.argtypes = [P, P]
    lib.pivot_debug_key_stream.argtypes = [P, I, I, I, I, I, P, P]
    lib.pivot_debug_counters.argtypes = [P, C.POINTER(C.c_ulonglong), I]
    lib.pivot_merge_topk.argtypes = [P, P, I, I, P, I, P, P, P]
    lib.pivot_prefill_host_arena_bytes.restype = S
    lib.pivot_prefill_host_arena_bytes.argtypes = [I, I, I, I, I, I, I]
    lib.pivot_index_prefill_host.argtypes = [T, P, T, I, I, I, I, I, I, I, P, P, S, P]
    lib.pivot_device_status.argtypes = [P, C.POINTER(C.c_int)]
    lib.pivot_stage_timing.argtypes = [I]
    lib.pivot_stage_times.argtypes = [C.POINTER(C.c_float), I]
    lib.pivot_launch_count_reset.restype = C.c_longlong
    lib.pivot_status_str.restype = C.c_char_p
    lib.pivot_status_str.argtypes = [I]
    return lib


lib = _load()
_workspaces: dict[int, torch.Tensor] = {}


def _check(rc: int):
    if rc != OK:
        extra = f" (cudaError {lib.pivot_last_cuda_error()})" if rc == 4 else ""
        raise PivotError(f"libpivot: {lib.pivot_status_str(rc).decode()}{extra}")


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float8_e4m3fn:
        return FP8_E4M3
    raise TypeError(f"unsupported operand dtype {t.dtype}")


def _tensor(data: torch.Tensor, scale) -> pivot_tensor:
    """Dense tensors, or key caches whose rows are padded: a view [..., rows, d] of a wider buffer with
    unit stride along d and every outer dimension dense over the padded rows (stride_row = bytes per row)."""
    assert scale is None or (scale.is_contiguous() and scale.dtype == torch.float32)
    stride_row = 0
    if not data.is_contiguous():
        assert data.stride(-1) == 1, "the last dimension must be contiguous"
        rs = data.stride(-2)
        for i in range(data.dim() - 2):            # outer dimensions must be dense over the padded rows
            assert data.stride(i) == rs * int(torch.tensor(data.shape[i + 1:-1]).prod()), "unsupported strides"
        stride_row = rs * data.element_size()
    return pivot_tensor(data.data_ptr(), None if scale is None else scale.data_ptr(), _dtype_code(data), stride_row)


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


IMPL_TENSOR_CORE, IMPL_CUDA_CORE, IMPL_TENSOR_CORE_FP32_HEAD_SUM = 0, 1, 2


def _opts(guard_len, pool, dbg_cand, dbg_scores, dbg_cand_scores, workspace, impl=0, rows=None, W=0, cand_in=None) -> pivot_opts:
    p = lambda t: None if t is None else t.data_ptr()
    r0, r1 = (0, 0) if rows is None else rows
    return pivot_opts(-1 if guard_len is None else guard_len, pool, p(dbg_cand), p(dbg_scores),
                      p(dbg_cand_scores), p(workspace), 0 if workspace is None else workspace.numel(), impl,
                      r0, r1, W, p(cand_in))


def pivot_workspace_bytes(rows: int, n_groups: int, c: int, k: int) -> int:
    return int(lib.pivot_workspace_bytes(rows, n_groups, c, k))


def pivot_set_workspace(workspace: torch.Tensor | None):
    """Registers a uint8 CUDA tensor as the scratch of the short entry points (kept alive here)."""
    if workspace is None:
        _check(lib.pivot_set_workspace(None, 0))
        _workspaces.pop(torch.cuda.current_device(), None)
        return
    assert workspace.dtype == torch.uint8 and workspace.is_cuda
    _check(lib.pivot_set_workspace(workspace.data_ptr(), workspace.numel()))
    _workspaces[workspace.device.index] = workspace


def pivot_decode_workspace_bytes(B: int, Lmax: int, g: int, c: int, k: int) -> int:
    return int(lib.pivot_decode_workspace_bytes(B, Lmax, g, c, k))


def ensure_workspace(rows: int, n_groups: int, c: int, k: int, device="cuda", need: int | None = None) -> torch.Tensor:
    """Allocates (or reuses) a registered workspace large enough for these sizes."""
    need = pivot_workspace_bytes(rows, n_groups, c, k) if need is None else need
    dev = torch.device(device)
    idx = dev.index if dev.index is not None else torch.cuda.current_device()
    cur = _workspaces.get(idx)
    if cur is None or cur.numel() < need:
        with torch.cuda.device(idx):
            cur = torch.empty(need, dtype=torch.uint8, device=f"cuda:{idx}")
            pivot_set_workspace(cur)
    return cur


def pivot_index_prefill(q, w, kcache, L, H_I, d, g, c, k, mode, out_idx, stream=None, *,
                        q_scale=None, k_scale=None, guard_len=None, pool=POOL_MEAN, dbg_cand=None,
                        dbg_scores=None, dbg_cand_scores=None, workspace=None, impl=0, rows=None, W=0):
    """rows=(row_begin, row_end) indexes just that chunk of query rows (chunked prefill); W is
    the local window of Appendix B (0 = off)."""
    tq, tk = _tensor(q, q_scale), _tensor(kcache, k_scale)
    assert w.dtype == torch.float32 and out_idx.dtype == torch.int32 and out_idx.numel() >= L * k
    if workspace is None:
        ensure_workspace(L, (L + g - 1) // g, c, k, q.device)
    o = _opts(guard_len, pool, dbg_cand, dbg_scores, dbg_cand_scores, workspace, impl, rows, W)
    _check(lib.pivot_index_prefill_ex(C.byref(tq), w.data_ptr(), C.byref(tk), L, H_I, d, g, c, k, mode,
                                      out_idx.data_ptr(), _stream(stream), C.byref(o)))
    return out_idx


def pivot_index_prefill_varlen(q, w, kcache, cu_seqlens, H_I, d, g, c, k, mode, out_idx, stream=None, *,
                               q_scale=None, k_scale=None, guard_len=None, pool=POOL_MEAN, workspace=None, impl=0, W=0):
    """Several requests packed back to back; cu_seqlens is a host sequence [n_req + 1] starting at 0.
    Positions in out_idx are relative to each row's own request."""
    cu = [int(v) for v in cu_seqlens]
    n_req = len(cu) - 1
    tq, tk = _tensor(q, q_scale), _tensor(kcache, k_scale)
    assert w.dtype == torch.float32 and out_idx.dtype == torch.int32 and out_idx.numel() >= cu[-1] * k
    if workspace is None:
        Lmax = max((b - a for a, b in zip(cu[:-1], cu[1:])), default=1)
        ensure_workspace(max(Lmax, 1), (max(Lmax, 1) + g - 1) // g, c, k, q.device)
    o = _opts(guard_len, pool, None, None, None, workspace, impl, None, W)
    arr = (C.c_int32 * (n_req + 1))(*cu)
    _check(lib.pivot_index_prefill_varlen(C.byref(tq), w.data_ptr(), C.byref(tk), arr, n_req, H_I, d, g, c, k, mode,
                                          out_idx.data_ptr(), _stream(stream), C.byref(o)))
    return out_idx


def dense_index(q, w, kcache, L, H_I, d, k, out_idx, stream=None, *, q_scale=None, k_scale=None,
                dbg_scores=None, workspace=None, impl=0):
    tq, tk = _tensor(q, q_scale), _tensor(kcache, k_scale)
    assert w.dtype == torch.float32 and out_idx.dtype == torch.int32 and out_idx.numel() >= L * k
    if workspace is None:
        ensure_workspace(L, L, k, k, q.device)
    o = _opts(None, POOL_MEAN, None, dbg_scores, None, workspace, impl)
    _check(lib.dense_index_ex(C.byref(tq), w.data_ptr(), C.byref(tk), L, H_I, d, k, out_idx.data_ptr(),
                              _stream(stream), C.byref(o)))
    return out_idx


def dense_index_static(q, w, kcache, L, H_I, d, k, out_idx, stream=None, *, q_scale=None, k_scale=None):
    """dense_index for callers that may not allocate device memory: no workspace argument, the
    scratch is an array built into the library (L <= 4096, k <= 512).  Nothing is allocated
    here either -- the tensors are the caller's."""
    tq, tk = _tensor(q, q_scale), _tensor(kcache, k_scale)
    assert w.dtype == torch.float32 and out_idx.dtype == torch.int32 and out_idx.numel() >= L * k
    _check(lib.dense_index_static(C.byref(tq), w.data_ptr(), C.byref(tk), L, H_I, d, k, out_idx.data_ptr(),
                                  _stream(stream)))
    return out_idx


def pivot_index_decode(q, w, kcache, pos0, B, Lmax, H_I, d, g, c, k, mode, out_idx, stream=None, *,
                       q_scale=None, k_scale=None, guard_len=None, pool=POOL_MEAN, dbg_cand=None,
                       dbg_scores=None, dbg_cand_scores=None, workspace=None, impl=0, W=0, cand_in=None):
    """cand_in ([B, c] int32, device): Refine on candidate sets supplied from outside (no scan)."""
    tq, tk = _tensor(q, q_scale), _tensor(kcache, k_scale)
    assert w.dtype == torch.float32 and out_idx.dtype == torch.int32 and pos0.dtype == torch.int32
    assert out_idx.numel() >= B * g * k
    assert cand_in is None or (cand_in.dtype == torch.int32 and cand_in.is_contiguous() and cand_in.numel() >= B * c)
    if workspace is None:
        ensure_workspace(B * g, B, c, k, q.device, need=pivot_decode_workspace_bytes(B, Lmax, g, c, k))
    o = _opts(guard_len, pool, dbg_cand, dbg_scores, dbg_cand_scores, workspace, impl, W=W, cand_in=cand_in)
    _check(lib.pivot_index_decode_ex(C.byref(tq), w.data_ptr(), C.byref(tk), pos0.data_ptr(), B, Lmax,
                                     H_I, d, g, c, k, mode, out_idx.data_ptr(), _stream(stream), C.byref(o)))
    return out_idx


def pivot_index_decode_paged(q, w, kpages, block_table, pos0, B, max_pages, n_pages, H_I, d, g, c, k, mode,
                             out_idx, stream=None, *, q_scale=None, k_scale=None, pool=POOL_MEAN, dbg_cand=None,
                             dbg_scores=None, dbg_cand_scores=None, workspace=None, impl=0, W=0):
    tq, tk = _tensor(q, q_scale), _tensor(kpages, k_scale)
    assert w.dtype == torch.float32 and out_idx.dtype == torch.int32 and pos0.dtype == torch.int32
    assert block_table.dtype == torch.int32 and block_table.is_contiguous() and block_table.numel() >= B * max_pages
    assert out_idx.numel() >= B * g * k
    if workspace is None:
        ensure_workspace(B * g, B, c, k, q.device, need=pivot_decode_workspace_bytes(B, max_pages * 128, g, c, k))
    o = _opts(None, pool, dbg_cand, dbg_scores, dbg_cand_scores, workspace, impl, W=W)
    _check(lib.pivot_index_decode_paged(C.byref(tq), w.data_ptr(), C.byref(tk), block_table.data_ptr(),
                                        pos0.data_ptr(), B, max_pages, n_pages, H_I, d, g, c, k, mode,
                                        out_idx.data_ptr(), _stream(stream), C.byref(o)))
    return out_idx


def dense_index_decode(q, w, kcache, pos0, B, Lmax, H_I, d, g, k, out_idx, stream=None, *, q_scale=None, k_scale=None,
                       dbg_scores=None, workspace=None, impl=0):
    """Dense control of a decode step: Eq. 1 + TopK for each of the g queries of every sequence."""
    tq, tk = _tensor(q, q_scale), _tensor(kcache, k_scale)
    assert w.dtype == torch.float32 and out_idx.dtype == torch.int32 and pos0.dtype == torch.int32
    assert out_idx.numel() >= B * g * k
    if workspace is None:
        ensure_workspace(B * g, B * g, k, k, q.device, need=pivot_decode_workspace_bytes(B * g, Lmax, 1, k, k))
    o = _opts(None, POOL_MEAN, None, dbg_scores, None, workspace, impl)
    _check(lib.dense_index_decode_ex(C.byref(tq), w.data_ptr(), C.byref(tk), pos0.data_ptr(), B, Lmax, H_I, d, g, k,
                                     out_idx.data_ptr(), _stream(stream), C.byref(o)))
    return out_idx


def pivot_merge_topk(scores, idx, K, out_idx, out_scores=None, seg_offset=None, stream=None):
    """Top-K of the union of candidate lists: scores / idx [n_seg, seg_len] (idx < 0 = empty slot), seg_offset [n_seg]
    int32 added to each list's positions.  Uses the registered workspace."""
    assert scores.dtype == torch.float32 and idx.dtype == torch.int32 and scores.shape == idx.shape and idx.dim() == 2
    assert scores.is_contiguous() and idx.is_contiguous() and out_idx.dtype == torch.int32 and out_idx.numel() >= K
    n_seg, seg_len = idx.shape
    need = 256 + 8 * n_seg * seg_len
    dev = idx.device.index if idx.device.index is not None else torch.cuda.current_device()
    cur = _workspaces.get(dev)
    if cur is None or cur.numel() < need:
        with torch.cuda.device(dev):
            pivot_set_workspace(torch.empty(need, dtype=torch.uint8, device=f"cuda:{dev}"))
    p = lambda t: None if t is None else t.data_ptr()
    _check(lib.pivot_merge_topk(scores.data_ptr(), idx.data_ptr(), n_seg, seg_len, p(seg_offset), K, out_idx.data_ptr(),
                                p(out_scores), _stream(stream)))
    return out_idx


def pivot_debug_wait_expiry(limit_ns: int, stream=None):
    """Diagnostic: lets the library's bounded device waits run out after limit_ns (see pivot.h)."""
    _check(lib.pivot_debug_wait_expiry(int(limit_ns), _stream(stream)))


MMA_MODEL_VARIANTS = ["M1 fp8 N=256 (4 K-steps)", "M1 fp8 N=192", "M1 fp8 2 x N=128", "M2 bf16 A in TMEM, 16 K-steps",
                      "M2 bf16 A in TMEM, 8 K-steps", "M2 fp8 A in TMEM, 8 K-steps", "M2 int8 A in TMEM, 8 K-steps",
                      "M1 + M2 bf16 x16", "M1 + M2 bf16 x8", "M1 + M2 int8 x8", "M1 N=192 + M2 int8 x6",
                      "linear block fp8 N=16 (4 K-steps)", "M1 + linear block"]
MMA_MODEL_PHASES = ["alone", "with ReLU-pass traffic (4 warps: load 32 cols, pack, store 16)",
                    "with load-only traffic (4 warps)", "with load-only traffic (8 warps)"]


def pivot_debug_mma_model(stream=None) -> dict:
    """Runs the one-SM timing probe (see pivot.h) and labels its numbers: clocks per tile."""
    out = torch.zeros(256, dtype=torch.int64, device="cuda")
    _check(lib.pivot_debug_mma_model(out.data_ptr(), _stream(stream)))
    torch.cuda.synchronize()
    v = out.cpu().tolist()
    res = {"abort_flag": v[254], "handover_clk": {"mbarrier try_wait, one way": v[128], "mbarrier test_wait, one way": v[129],
                                                  "tcgen05.commit -> waiter -> arrive -> issuer, round trip": v[130]}}
    for ph, pname in enumerate(MMA_MODEL_PHASES):
        d = {name: v[ph * 32 + i] for i, name in enumerate(MMA_MODEL_VARIANTS)}
        if ph:
            d["traffic warps: clk per 256-column pass"] = [x for x in v[ph * 32 + 16: ph * 32 + 24] if x]
        res[pname] = d
    return res


PROF_SLOTS = ("scan_wait_queries", "scan_wait_accumulator", "scan_wait_keys", "scan_wait_gates", "scan_wait_relu",
              "scan_total", "scan_tiles",
              "rescore_wait_queries", "rescore_wait_accumulator", "rescore_wait_keys", "rescore_wait_gates",
              "rescore_wait_relu", "rescore_total", "rescore_tiles",
              "rescore_select_wait", "rescore_select_work", "rescore_select_groups",
              "decode_select_boundary", "decode_select_collect", "decode_select_handover", "decode_select_topk",
              "decode_select_sequences",
              "decode_scan_producer_wait", "decode_scan_max_total", "decode_scan_wait_accumulator", "decode_scan_wait_keys",
              "decode_scan_total", "decode_scan_tiles")


def pivot_debug_counters(stream=None) -> dict:
    """Cycle counters of a -DPIVOT_PROF build since the last read (read and cleared); raises in an
    ordinary build."""
    out = (C.c_ulonglong * len(PROF_SLOTS))()
    _check(lib.pivot_debug_counters(_stream(stream), out, len(PROF_SLOTS)))
    return dict(zip(PROF_SLOTS, [int(v) for v in out]))


def pivot_debug_key_stream(n_keys=131072, ctas=148, tiles=2048, stages=4, mode=0, stream=None) -> dict:
    """Key-tile streaming probe (see pivot.h): clocks per 16 KB tile, mean over the CTAs, per stream."""
    keys = torch.zeros((n_keys, 128), dtype=torch.uint8, device="cuda")
    out = torch.zeros(2 * ctas, dtype=torch.int64, device="cuda")
    if n_keys * 128 > (64 << 20):          # an HBM-sized stream: nothing of it may still sit in L2
        torch.empty(512 << 20, dtype=torch.uint8, device="cuda").fill_(1)
    _check(lib.pivot_debug_key_stream(keys.data_ptr(), n_keys, ctas, tiles, stages, mode, out.data_ptr(), _stream(stream)))
    torch.cuda.synchronize()
    v = out.cpu().float().view(ctas, 2)
    return {"n_keys": n_keys, "ctas": ctas, "stages": stages, "tiles_per_cta": tiles,
            "mode": ["one TMA stream", "two TMA streams", "TMA stream + cp.async stream",
                     "one thread, four 32-key boxes per tile", "four lanes, one 32-key box each"][mode],
            "clk_per_tile_stream0": float(v[:, 0].mean()), "clk_per_tile_stream1": float(v[:, 1].mean()) if mode else None}


def pivot_prefill_host_arena_bytes(L, H_I, d, g, c, k, dtype) -> int:
    return int(lib.pivot_prefill_host_arena_bytes(L, H_I, d, g, c, k, dtype))


def pivot_index_prefill_host(q, w, kcache, L, H_I, d, g, c, k, mode, out_idx, arena, stream=None, *,
                             q_scale=None, k_scale=None):
    """Host-buffer form: q / w / kcache / scales / out_idx are CPU tensors (pin them), `arena` a
    uint8 CUDA tensor of at least pivot_prefill_host_arena_bytes(...) bytes.  Returns after the
    result has landed in out_idx."""
    for t in (q, w, kcache, out_idx):
        assert not t.is_cuda
    tq, tk = _tensor(q, q_scale), _tensor(kcache, k_scale)
    _check(lib.pivot_index_prefill_host(C.byref(tq), w.data_ptr(), C.byref(tk), L, H_I, d, g, c, k, mode,
                                        out_idx.data_ptr(), arena.data_ptr(), arena.numel(), _stream(stream)))
    return out_idx


def pivot_device_status(stream=None) -> int:
    st = C.c_int(0)
    _check(lib.pivot_device_status(_stream(stream), C.byref(st)))
    return st.value


def pivot_stage_timing(enable: bool):
    _check(lib.pivot_stage_timing(1 if enable else 0))


def pivot_stage_times() -> dict:
    """Elapsed ms of the last call's stages (needs pivot_stage_timing(True) before the call)."""
    ms = (C.c_float * 7)()
    _check(lib.pivot_stage_times(ms, 7))
    return dict(zip(("proxy_build", "plan", "scan_select", "refine", "total", "decode_scan", "decode_select"),
                    [float(v) for v in ms]))


def pivot_launch_count_reset() -> int:
    return int(lib.pivot_launch_count_reset())
