"""ctypes binding of the liblightkv C ABI (include/lightkv.h): same names, argument marshalling only.

PyTorch is used for device memory and streams: tensors are handed over as data pointers plus element
strides, the current CUDA stream as a raw handle.  No arithmetic of the method happens here.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

BF16, FP32 = 0, 1
XI_GIVEN, XI_ATTN_FULL, XI_ATTN_LSE, XI_UNIFORM = 0, 1, 2, 3
KV_MERGE, KV_GATHER = 0, 1
ENGINE_AUTO, ENGINE_SIMT = 0, 1
FD_COSINE, FD_L2SQ, FD_L2 = 0, 1, 2
DIR_A2B, DIR_B2A = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None


class LightKVError(RuntimeError):
    pass


class _Tile(C.Structure):
    _fields_ = [("rows", C.c_int32), ("cols", C.c_int32)]


class _Config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("batch", C.c_int32), ("hidden", C.c_int32),
                ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("n_layers", C.c_int32), ("n_tiles", C.c_int32), ("tiles", C.POINTER(_Tile)),
                ("n_stages", C.c_int32), ("layers", C.POINTER(C.c_int32)),
                ("windows", C.POINTER(C.c_int32)), ("keep", C.POINTER(C.c_double)),
                ("max_text", C.c_int32), ("dtype", C.c_int32), ("xi_mode", C.c_int32),
                ("engine", C.c_int32), ("ragged_input", C.c_int32), ("divergence", C.c_int32),
                ("direction", C.c_int32)]


class _StageInfo(C.Structure):
    _fields_ = [("layer", C.c_int32), ("window", C.c_int32), ("keep", C.c_double),
                ("cap_in", C.c_int32), ("cap_out", C.c_int32), ("n_windows", C.c_int32),
                ("counts_exact", C.c_int32), ("uses_tensor_cores", C.c_int32),
                ("workspace_bytes", C.c_size_t), ("cap_a", C.c_int32), ("cap_b", C.c_int32),
                ("fd_tiles", C.c_int32), ("reserved", C.c_int32)]


class _LayerArgs(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("stage", C.c_int32), ("vis_begin", C.c_int32),
                ("n_text_after", C.c_int32), ("text_begin", C.c_int32), ("text_end", C.c_int32),
                ("hidden", C.c_void_p), ("hidden_batch_stride", C.c_int64), ("hidden_row_stride", C.c_int64),
                ("hidden_out", C.c_void_p), ("hidden_out_batch_stride", C.c_int64),
                ("hidden_out_row_stride", C.c_int64),
                ("q", C.c_void_p), ("q_batch_stride", C.c_int64), ("q_head_stride", C.c_int64),
                ("q_row_stride", C.c_int64),
                ("k", C.c_void_p), ("k_batch_stride", C.c_int64), ("k_head_stride", C.c_int64),
                ("k_row_stride", C.c_int64),
                ("lse", C.c_void_p), ("lse_batch_stride", C.c_int64), ("lse_head_stride", C.c_int64),
                ("xi", C.c_void_p), ("n_vis", C.c_void_p), ("pos", C.c_void_p),
                ("n_vis_out", C.c_void_p), ("pos_out", C.c_void_p), ("dst", C.c_void_p),
                ("weight", C.c_void_p), ("grp_off", C.c_void_p), ("grp_src", C.c_void_p),
                ("xi_out", C.c_void_p), ("status", C.c_void_p), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t), ("stream", C.c_void_p),
                ("trace_events", C.POINTER(C.c_void_p)), ("seq_rows", C.c_int32), ("aux_stream", C.c_void_p),
                ("map_event", C.c_void_p), ("fork_event", C.c_void_p), ("join_event", C.c_void_p),
                ("n_text_ranges", C.c_int32), ("bidirectional", C.c_int32),
                ("text_ranges", C.POINTER(C.c_int32)),
                ("lse_out", C.c_void_p), ("lse_out_batch_stride", C.c_int64), ("lse_out_head_stride", C.c_int64),
                ("seq_start", C.c_void_p), ("seq_start_out", C.c_void_p)]


MAX_TEXT_RANGES = 8
TRACE_EVENTS = 6
TRACE_NAMES = ("window_build", "xi", "fd_best_partner", "select_map", "merge_hidden")


class _KvArgs(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("stage", C.c_int32), ("vis_begin", C.c_int32),
                ("n_text_after", C.c_int32), ("mode", C.c_int32),
                ("n_vis", C.c_void_p), ("n_vis_out", C.c_void_p), ("grp_off", C.c_void_p),
                ("grp_src", C.c_void_p), ("weight", C.c_void_p),
                ("k_src", C.c_void_p), ("v_src", C.c_void_p), ("k_dst", C.c_void_p), ("v_dst", C.c_void_p),
                ("src_batch_stride", C.c_int64), ("src_head_stride", C.c_int64), ("src_row_stride", C.c_int64),
                ("dst_batch_stride", C.c_int64), ("dst_head_stride", C.c_int64), ("dst_row_stride", C.c_int64),
                ("page_size", C.c_int32), ("max_blocks", C.c_int32),
                ("src_block_table", C.c_void_p), ("dst_block_table", C.c_void_p),
                ("src_page_stride", C.c_int64), ("dst_page_stride", C.c_int64),
                ("status", C.c_void_p), ("stream", C.c_void_p),
                ("src_seq_start", C.c_void_p), ("dst_seq_start", C.c_void_p)]


EXPORTS = ("lightkv_plan", "lightkv_plan_stage_info", "lightkv_plan_destroy", "lightkv_plan_retention",
           "lightkv_compress_layer", "lightkv_compress_layer_builtin_ws", "lightkv_compact_kv",
           "lightkv_status_string", "lightkv_version")
BUILTIN_WS_BYTES = 8 << 20


def library_path() -> str:
    return os.path.join(_HERE, "liblightkv.so")


def library() -> C.CDLL:
    """Load liblightkv.so (built in-tree).  There is no fallback: a missing library is an error."""
    global _LIB
    if _LIB is None:
        path = library_path()
        if not os.path.exists(path):
            raise LightKVError(f"{path} is missing: build it first (python -c 'import __graft_entry__ as g; g.build()')")
        lib = C.CDLL(path)
        lib.lightkv_plan.argtypes = [C.POINTER(_Config), C.POINTER(C.c_void_p)]
        lib.lightkv_plan.restype = C.c_int
        lib.lightkv_plan_stage_info.argtypes = [C.c_void_p, C.c_int32, C.POINTER(_StageInfo)]
        lib.lightkv_plan_stage_info.restype = C.c_int
        lib.lightkv_plan_destroy.argtypes = [C.c_void_p]
        lib.lightkv_plan_destroy.restype = None
        lib.lightkv_plan_retention.argtypes = [C.c_void_p]
        lib.lightkv_plan_retention.restype = C.c_double
        lib.lightkv_compress_layer.argtypes = [C.c_void_p, C.POINTER(_LayerArgs)]
        lib.lightkv_compress_layer.restype = C.c_int
        lib.lightkv_compress_layer_builtin_ws.argtypes = [C.c_void_p, C.POINTER(_LayerArgs)]
        lib.lightkv_compress_layer_builtin_ws.restype = C.c_int
        lib.lightkv_compact_kv.argtypes = [C.c_void_p, C.POINTER(_KvArgs)]
        lib.lightkv_compact_kv.restype = C.c_int
        lib.lightkv_status_string.argtypes = [C.c_int]
        lib.lightkv_status_string.restype = C.c_char_p
        lib.lightkv_version.argtypes = []
        lib.lightkv_version.restype = C.c_int
        _LIB = lib
    return _LIB


def version() -> int:
    return library().lightkv_version()


def status_string(code: int) -> str:
    return library().lightkv_status_string(code).decode()


def _check(code: int, what: str) -> None:
    if code != 0:
        raise LightKVError(f"{what}: {status_string(code)} ({code})")


class Plan:
    """lightkv_plan: schedule, capacities and workspace sizes (host only)."""

    def __init__(self, batch: int, hidden: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 n_layers: int, tiles: Sequence[Tuple[int, int]], layers: Sequence[int],
                 windows: Sequence[int], keep: Sequence[float], max_text: int,
                 dtype: int = BF16, xi_mode: int = XI_ATTN_FULL, engine: int = ENGINE_AUTO,
                 ragged_input: bool = False, divergence: int = FD_COSINE, direction: int = DIR_A2B):
        lib = library()
        n_stages = len(layers)
        self._tiles = (_Tile * len(tiles))(*[_Tile(int(r), int(c)) for r, c in tiles])
        self._layers = (C.c_int32 * n_stages)(*[int(v) for v in layers])
        self._windows = (C.c_int32 * n_stages)(*[int(v) for v in windows])
        self._keep = (C.c_double * n_stages)(*[float(v) for v in keep])
        cfg = _Config(C.sizeof(_Config), batch, hidden, n_q_heads, n_kv_heads, head_dim, n_layers,
                      len(tiles), self._tiles, n_stages, self._layers, self._windows, self._keep,
                      max_text, dtype, xi_mode, engine, int(ragged_input), divergence, direction)
        handle = C.c_void_p()
        _check(lib.lightkv_plan(C.byref(cfg), C.byref(handle)), "lightkv_plan")
        self.handle = handle
        self.batch, self.hidden, self.n_q_heads, self.n_kv_heads = batch, hidden, n_q_heads, n_kv_heads
        self.head_dim, self.n_layers, self.n_stages = head_dim, n_layers, n_stages
        self.dtype, self.xi_mode, self.engine, self.max_text = dtype, xi_mode, engine, max_text
        self.tiles = [tuple(t) for t in tiles]

    def stage_info(self, stage: int) -> _StageInfo:
        info = _StageInfo()
        _check(library().lightkv_plan_stage_info(self.handle, stage, C.byref(info)), "lightkv_plan_stage_info")
        return info

    def retention(self) -> float:
        return library().lightkv_plan_retention(self.handle)

    def close(self) -> None:
        if getattr(self, "handle", None):
            library().lightkv_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


class StageBuffers:
    """Device outputs + workspace of one stage, allocated with torch (plumbing only)."""

    def __init__(self, plan: Plan, stage: int, n_seq_out: int, device="cuda"):
        import torch
        info = plan.stage_info(stage)
        self.info = info
        b = plan.batch
        tdt = torch.bfloat16 if plan.dtype == BF16 else torch.float32
        i32 = dict(dtype=torch.int32, device=device)
        self.hidden_out = torch.empty((b, n_seq_out, plan.hidden), dtype=tdt, device=device)
        self.n_vis_out = torch.zeros((b,), **i32)
        self.pos_out = torch.full((b, info.cap_out), -1, **i32)
        self.dst = torch.full((b, info.cap_in), -1, **i32)
        self.weight = torch.zeros((b, info.cap_in), dtype=torch.float32, device=device)
        self.grp_off = torch.zeros((b, info.cap_out + 1), **i32)
        self.grp_src = torch.full((b, info.cap_in), -1, **i32)
        self.xi_out = torch.zeros((b, info.cap_in), dtype=torch.float32, device=device)
        self.status = torch.zeros((1,), **i32)
        self.workspace = torch.empty((info.workspace_bytes + 256,), dtype=torch.uint8, device=device)

    def workspace_ptr(self) -> int:
        p = self.workspace.data_ptr()
        return (p + 255) // 256 * 256


def _stream_handle(stream) -> int:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _layer_args(plan: Plan, stage: int, hidden, out: StageBuffers, *, vis_begin: int,
                n_text_after: int = 0, text_begin: int = 0, text_end: Optional[int] = None,
                q=None, k=None, lse=None, xi=None, n_vis=None, pos=None, stream=None,
                trace_events=None, aux_stream=None, map_event=None, fork_event=None, join_event=None,
                text_ranges=None, bidirectional: bool = False, lse_out=None, seq_start=None, seq_start_out=None,
                hidden_out=None) -> _LayerArgs:
    a = _LayerArgs()
    a.struct_size = C.sizeof(_LayerArgs)
    a.stage, a.vis_begin, a.n_text_after = stage, vis_begin, n_text_after
    a.text_begin, a.text_end = text_begin, vis_begin if text_end is None else text_end
    a.hidden, a.hidden_batch_stride, a.hidden_row_stride = hidden.data_ptr(), hidden.stride(0), hidden.stride(1)
    ho = out.hidden_out if hidden_out is None else hidden_out
    a.hidden_out, a.hidden_out_batch_stride, a.hidden_out_row_stride = ho.data_ptr(), ho.stride(0), ho.stride(1)
    if q is not None:
        a.seq_rows = q.shape[2]
        a.q, a.q_batch_stride, a.q_head_stride, a.q_row_stride = q.data_ptr(), q.stride(0), q.stride(1), q.stride(2)
    if k is not None:
        a.k, a.k_batch_stride, a.k_head_stride, a.k_row_stride = k.data_ptr(), k.stride(0), k.stride(1), k.stride(2)
    if lse is not None:
        a.lse, a.lse_batch_stride, a.lse_head_stride = lse.data_ptr(), lse.stride(0), lse.stride(1)
    a.xi, a.n_vis, a.pos = _ptr(xi), _ptr(n_vis), _ptr(pos)
    a.n_vis_out, a.pos_out, a.dst, a.weight = _ptr(out.n_vis_out), _ptr(out.pos_out), _ptr(out.dst), _ptr(out.weight)
    a.grp_off, a.grp_src, a.xi_out, a.status = _ptr(out.grp_off), _ptr(out.grp_src), _ptr(out.xi_out), _ptr(out.status)
    a.workspace, a.workspace_bytes = out.workspace_ptr(), out.info.workspace_bytes
    a.stream = _stream_handle(stream)
    if aux_stream is not None:
        # the library creates no events: the fork / join pair is the caller's (kept with the stage's buffers here)
        import torch
        a.aux_stream = aux_stream.cuda_stream
        if fork_event is None or join_event is None:
            if not hasattr(out, "fork_join"):
                out.fork_join = (torch.cuda.Event(), torch.cuda.Event())
                for e in out.fork_join:
                    e.record()            # torch creates the CUDA event lazily; the C ABI needs a live handle
            fork_event, join_event = out.fork_join
        a.fork_event, a.join_event = fork_event.cuda_event, join_event.cuda_event
    if text_ranges is not None:       # [(begin, end), ...] instead of the single range text_begin / text_end
        flat = [int(v) for r in text_ranges for v in r]
        a._ranges = (C.c_int32 * len(flat))(*flat)          # kept alive by the struct object
        a.text_ranges, a.n_text_ranges = a._ranges, len(flat) // 2
    a.bidirectional = int(bool(bidirectional))
    if lse_out is not None:
        a.lse_out, a.lse_out_batch_stride, a.lse_out_head_stride = lse_out.data_ptr(), lse_out.stride(0), lse_out.stride(1)
    if seq_start is not None:
        # packed batch: tensors of shape [1, rows, ...] hold the samples back to back; sample b starts at row
        # seq_start[b], so the batch strides are 0 and q / k span all rows
        a.seq_start, a.seq_start_out = seq_start.data_ptr(), _ptr(seq_start_out)
        a.hidden_batch_stride = a.q_batch_stride = a.k_batch_stride = a.lse_batch_stride = a.lse_out_batch_stride = 0
        if seq_start_out is not None:
            a.hidden_out_batch_stride = 0
    if map_event is not None:         # a torch.cuda.Event that has been recorded once (torch creates it lazily)
        a.map_event = map_event.cuda_event
    if trace_events is not None:      # TRACE_EVENTS torch.cuda.Event objects (enable_timing=True), already created
        assert len(trace_events) == TRACE_EVENTS
        a.trace_events = (C.c_void_p * TRACE_EVENTS)(*[e.cuda_event for e in trace_events])
    return a


def compress_layer(plan: Plan, stage: int, hidden, out: StageBuffers, **kw) -> None:
    """lightkv_compress_layer.  hidden [B,N,d]; keywords: vis_begin, n_text_after, text_begin, text_end,
    q [B,H,N,dh], k [B,H_kv,N,dh] (any strides with a contiguous last dimension), lse [B,H,N] fp32,
    xi [B,cap_in] fp32, n_vis [B] int32, pos [B,cap_in] int32, stream, trace_events, aux_stream, map_event,
    fork_event / join_event, text_ranges [(begin, end), ...], bidirectional, lse_out [B,H,N] fp32,
    seq_start / seq_start_out [B] int32 (packed batches), hidden_out (instead of out.hidden_out)."""
    a = _layer_args(plan, stage, hidden, out, **kw)
    _check(library().lightkv_compress_layer(plan.handle, C.byref(a)), "lightkv_compress_layer")


def compress_layer_builtin_ws(plan: Plan, stage: int, hidden, out: StageBuffers, **kw) -> None:
    """lightkv_compress_layer_builtin_ws: same call, but the stage's scratch is the fixed array inside
    the library (BUILTIN_WS_BYTES), so the workspace tensor of `out` is not used.  Meant for callers
    that may not allocate device memory; stages needing more scratch than that are refused."""
    a = _layer_args(plan, stage, hidden, out, **kw)
    a.workspace, a.workspace_bytes = None, 0
    _check(library().lightkv_compress_layer_builtin_ws(plan.handle, C.byref(a)),
           "lightkv_compress_layer_builtin_ws")


def compact_kv(plan: Plan, stage: int, out: StageBuffers, k_src, v_src, k_dst, v_dst, *, vis_begin: int,
               n_text_after: int = 0, mode: int = KV_MERGE, n_vis=None, page_size: int = 0,
               src_block_table=None, dst_block_table=None, stream=None, src_seq_start=None,
               dst_seq_start=None) -> None:
    """lightkv_compact_kv.  Contiguous: k/v [B,H_kv,N,dh] views (any batch/head/row strides).
    Paged: k/v page pools [n_pages, H_kv, page_size, dh] views and int32 block tables [B, max_blocks]."""
    a = _KvArgs()
    a.struct_size = C.sizeof(_KvArgs)
    a.stage, a.vis_begin, a.n_text_after, a.mode = stage, vis_begin, n_text_after, mode
    a.n_vis, a.n_vis_out = _ptr(n_vis), _ptr(out.n_vis_out)
    a.grp_off, a.grp_src, a.weight = _ptr(out.grp_off), _ptr(out.grp_src), _ptr(out.weight)
    a.k_src, a.v_src, a.k_dst, a.v_dst = k_src.data_ptr(), v_src.data_ptr(), k_dst.data_ptr(), v_dst.data_ptr()
    assert k_src.stride() == v_src.stride() and k_dst.stride() == v_dst.stride()
    if page_size > 0:
        a.src_page_stride, a.src_head_stride, a.src_row_stride = k_src.stride(0), k_src.stride(1), k_src.stride(2)
        a.dst_page_stride, a.dst_head_stride, a.dst_row_stride = k_dst.stride(0), k_dst.stride(1), k_dst.stride(2)
        a.page_size, a.max_blocks = page_size, src_block_table.shape[1]
        assert dst_block_table.shape[1] == src_block_table.shape[1]
        a.src_block_table, a.dst_block_table = src_block_table.data_ptr(), dst_block_table.data_ptr()
    else:
        a.src_batch_stride, a.src_head_stride, a.src_row_stride = k_src.stride(0), k_src.stride(1), k_src.stride(2)
        a.dst_batch_stride, a.dst_head_stride, a.dst_row_stride = k_dst.stride(0), k_dst.stride(1), k_dst.stride(2)
    a.status = _ptr(out.status)
    a.stream = _stream_handle(stream)
    if src_seq_start is not None:     # packed caches: sample b's first token; contiguous batch strides become 0
        a.src_seq_start, a.src_batch_stride = src_seq_start.data_ptr(), 0
    if dst_seq_start is not None:
        a.dst_seq_start, a.dst_batch_stride = dst_seq_start.data_ptr(), 0
    _check(library().lightkv_compact_kv(plan.handle, C.byref(a)), "lightkv_compact_kv")
