"""Thin ctypes binding over the C-ABI library (``include/moe.h``).

Argument marshalling only: every step of the layer runs in the library's CUDA kernels.  There is
no CPU path and no fallback -- if ``libmoe_b200.so`` is missing or a call fails, this raises.
PyTorch is used for device memory and streams.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libmoe_b200.so"

MOE_OK = 0
MOE_FLAG_NONE = 0
MOE_FLAG_VALIDATION_GEMM = 1
MOE_FLAG_SINGLE_CTA_GEMM = 2
MOE_FLAG_TWO_SLAB_GEMM = 4
MOE_FLAG_NARROW_TILES = 8
MOE_FLAG_GATHER_IN_LOAD = 16

EXPORTED = ["moe_workspace_bytes", "moe_workspace_layout", "moe_route_workspace_bytes", "moe_route", "moe_route_static",
            "moe_forward",
            "moe_forward_ex", "moe_forward_local", "moe_route_grouped", "moe_forward_grouped", "moe_forward_fp8w", "moe_mxfp8_workspace_bytes",
            "moe_mxfp8_workspace_layout", "moe_mxfp8_pack_scales", "moe_mxfp8_quantize_rows", "moe_forward_mxfp8", "moe_forward_mxfp8_host",
            "moe_forward_staged", "moe_forward_host", "moe_last_status", "moe_selftest_wait_timeout", "moe_forward_launch_count", "moe_token_tile_rows", "moe_status_string",
            "gqa_decode_workspace_bytes", "gqa_paged_decode", "gqa_decode_split_tokens", "gqa_selftest_wait_timeout"]


class MoeError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({moe_status_string(status)})")


class WorkspaceLayout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_size_t) for n in
                ("total_bytes", "status", "topk_ids", "topk_weights", "expert_offsets", "sorted_to_flat",
                 "flat_to_sorted", "route_scratch", "x_perm", "h", "y", "staging")]


class GroupedRouter(ctypes.Structure):
    _fields_ = [("n_group", ctypes.c_int), ("topk_group", ctypes.c_int), ("selection_bias", ctypes.c_void_p),
                ("route_scale", ctypes.c_float)]


def grouped_router(n_group: int, topk_group: int, selection_bias=None, route_scale: float = 1.0) -> GroupedRouter:
    """Description of the grouped sigmoid router; ``selection_bias`` is a device f32 tensor [E] or None (the
    caller keeps it alive)."""
    return GroupedRouter(n_group, topk_group, None if selection_bias is None else selection_bias.data_ptr(), route_scale)


class MxWorkspaceLayout(ctypes.Structure):
    _fields_ = [(n, ctypes.c_size_t) for n in
                ("total_bytes", "status", "topk_ids", "topk_weights", "expert_offsets", "sorted_to_flat",
                 "flat_to_sorted", "route_scratch", "x_q", "x_sf", "h_q", "h_sf", "y", "staging", "sf_atoms", "tile_rows")]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library.  Raises if it has not been built (python -m paper_2602_19128_b200.build)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise FileNotFoundError(f"{_LIB_PATH} is missing: build it with `python -m paper_2602_19128_b200.build`; "
                                    "there is no fallback path")
        L = ctypes.CDLL(str(_LIB_PATH))
        i, sz, vp = ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p
        L.moe_workspace_bytes.restype = sz
        L.moe_workspace_bytes.argtypes = [i] * 5
        L.moe_workspace_layout.restype = i
        L.moe_workspace_layout.argtypes = [i] * 5 + [ctypes.POINTER(WorkspaceLayout)]
        L.moe_route_workspace_bytes.restype = sz
        L.moe_route_workspace_bytes.argtypes = [i] * 3
        L.moe_route.restype = i
        L.moe_route.argtypes = [vp, i, i, i, vp, vp, vp, vp, vp, vp, sz, vp]
        L.moe_route_static.restype = i
        L.moe_route_static.argtypes = [vp, i, i, i, vp, vp, vp, vp, vp, vp]
        L.moe_forward.restype = i
        L.moe_forward.argtypes = [vp, vp, vp, vp, i, i, i, i, i, vp, vp, sz, vp]
        L.moe_forward_ex.restype = i
        L.moe_forward_ex.argtypes = [vp, vp, vp, vp, i, i, i, i, i, vp, vp, sz, vp, ctypes.c_uint]
        L.moe_forward_local.restype = i
        L.moe_forward_local.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, vp, vp, sz, vp, ctypes.c_uint]
        L.moe_route_grouped.restype = i
        L.moe_route_grouped.argtypes = [vp, i, i, i, ctypes.POINTER(GroupedRouter), vp, vp, vp, vp, vp, vp, sz, vp]
        L.moe_forward_grouped.restype = i
        L.moe_forward_grouped.argtypes = [vp, vp, vp, vp, i, i, i, i, i, ctypes.POINTER(GroupedRouter), i, i, vp, vp, sz, vp,
                                          ctypes.c_uint]
        L.moe_forward_fp8w.restype = i
        L.moe_forward_fp8w.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, vp, vp, sz, vp, ctypes.POINTER(vp)]
        L.moe_mxfp8_workspace_bytes.restype = sz
        L.moe_mxfp8_workspace_bytes.argtypes = [i] * 5
        L.moe_mxfp8_workspace_layout.restype = i
        L.moe_mxfp8_workspace_layout.argtypes = [i] * 5 + [ctypes.POINTER(MxWorkspaceLayout)]
        L.moe_mxfp8_pack_scales.restype = i
        L.moe_mxfp8_pack_scales.argtypes = [vp, i, i, i, i, vp, vp]
        L.moe_mxfp8_quantize_rows.restype = i
        L.moe_mxfp8_quantize_rows.argtypes = [vp, i, i, vp, vp, vp]
        L.moe_forward_mxfp8.restype = i
        L.moe_forward_mxfp8.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, ctypes.POINTER(GroupedRouter), i, i, vp, vp, sz,
                                        vp, ctypes.POINTER(vp)]
        L.moe_forward_mxfp8_host.restype = i
        L.moe_forward_mxfp8_host.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, ctypes.POINTER(GroupedRouter), i, i, vp, vp,
                                             sz, vp]
        L.moe_forward_staged.restype = i
        L.moe_forward_staged.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, vp, vp, sz, vp, ctypes.c_uint,
                                         ctypes.POINTER(vp)]
        L.moe_forward_host.restype = i
        L.moe_forward_host.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, vp, vp, sz, vp]
        L.moe_selftest_wait_timeout.restype = i
        L.moe_selftest_wait_timeout.argtypes = [vp, sz, vp]
        L.moe_last_status.restype = i
        L.moe_last_status.argtypes = [vp, vp]
        L.moe_forward_launch_count.restype = i
        L.moe_forward_launch_count.argtypes = [i, ctypes.c_uint]
        L.moe_token_tile_rows.restype = i
        L.moe_token_tile_rows.argtypes = [i] * 5 + [ctypes.c_uint]
        L.gqa_decode_workspace_bytes.restype = sz
        L.gqa_decode_workspace_bytes.argtypes = [i] * 5
        L.gqa_decode_split_tokens.restype = i
        L.gqa_decode_split_tokens.argtypes = [i] * 5
        L.gqa_selftest_wait_timeout.restype = i
        L.gqa_selftest_wait_timeout.argtypes = [vp, sz, vp]
        L.gqa_paged_decode.restype = i
        L.gqa_paged_decode.argtypes = [vp] * 6 + [i] * 7 + [ctypes.c_float, vp, vp, vp, sz, vp]
        L.moe_status_string.restype = ctypes.c_char_p
        L.moe_status_string.argtypes = [i]
        _lib = L
    return _lib


def _ptr(t):
    """The address of a contiguous tensor (an int: ctypes converts it for a void* parameter)."""
    if t is None:
        return None
    assert t.is_contiguous(), "tensors must be contiguous"
    return t.data_ptr()


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream):
    """The cudaStream_t to launch on: the given torch stream, else the current stream of the current device."""
    if stream is not None:
        return stream.cuda_stream
    if _raw_stream is not None:
        return _raw_stream(torch.cuda.current_device())
    return torch.cuda.current_stream().cuda_stream


def moe_status_string(status: int) -> str:
    return lib().moe_status_string(int(status)).decode()


def moe_workspace_bytes(T: int, H: int, I: int, E: int, top_k: int) -> int:
    return int(lib().moe_workspace_bytes(T, H, I, E, top_k))


def moe_route_workspace_bytes(T: int, E: int, top_k: int) -> int:
    return int(lib().moe_route_workspace_bytes(T, E, top_k))


def moe_workspace_layout(T: int, H: int, I: int, E: int, top_k: int) -> WorkspaceLayout:
    L = WorkspaceLayout()
    st = lib().moe_workspace_layout(T, H, I, E, top_k, ctypes.byref(L))
    if st != MOE_OK:
        raise MoeError(st, "moe_workspace_layout")
    return L


def moe_forward_launch_count(T: int, flags: int = 0) -> int:
    return int(lib().moe_forward_launch_count(T, flags))


def moe_token_tile_rows(T: int, H: int, I: int, E: int, top_k: int, flags: int = 0) -> int:
    return int(lib().moe_token_tile_rows(T, H, I, E, top_k, flags))


def alloc_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A 256-byte aligned device buffer of at least ``nbytes`` (torch's allocator aligns to 512)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def moe_route(router_logits, top_k: int, topk_ids, topk_weights, expert_offsets, sorted_to_flat, flat_to_sorted,
              workspace, stream=None, check: bool = True) -> int:
    T, E = router_logits.shape
    st = lib().moe_route(_ptr(router_logits), T, E, top_k, _ptr(topk_ids), _ptr(topk_weights), _ptr(expert_offsets),
                         _ptr(sorted_to_flat), _ptr(flat_to_sorted), _ptr(workspace), workspace.numel(),
                         _stream(stream))
    if check and st != MOE_OK:
        raise MoeError(st, "moe_route")
    return st


def moe_route_static(router_logits, top_k: int, topk_ids, topk_weights, expert_offsets, sorted_to_flat, flat_to_sorted,
                     stream=None, check: bool = True) -> int:
    """moe_route without a workspace: the scratch is a fixed array inside the library (no allocation
    anywhere in the call).  Problems beyond its 512 KiB return MOE_ERR_STATIC_LIMIT (-9)."""
    T, E = router_logits.shape
    st = lib().moe_route_static(_ptr(router_logits), T, E, top_k, _ptr(topk_ids), _ptr(topk_weights),
                                _ptr(expert_offsets), _ptr(sorted_to_flat), _ptr(flat_to_sorted), _stream(stream))
    if check and st != MOE_OK:
        raise MoeError(st, "moe_route_static")
    return st


def moe_forward(x, router_logits, w13, w2, top_k: int, out, workspace, stream=None, flags: int = 0,
                check: bool = True) -> int:
    T, H = x.shape
    E, I2, _ = w13.shape
    st = lib().moe_forward_ex(_ptr(x), _ptr(router_logits), _ptr(w13), _ptr(w2), T, H, I2 // 2, E, top_k, _ptr(out),
                              _ptr(workspace), workspace.numel(), _stream(stream), flags)
    if check and st != MOE_OK:
        raise MoeError(st, "moe_forward")
    return st


def moe_forward_local(x, router_logits, w13_local, w2_local, top_k: int, local_expert_offset: int, out, workspace,
                      stream=None, flags: int = 0, check: bool = True) -> int:
    """The layer restricted to the resident experts [local_expert_offset, + w13_local.shape[0])."""
    T, H = x.shape
    E = router_logits.shape[1]
    n_local, I2, _ = w13_local.shape
    st = lib().moe_forward_local(_ptr(x), _ptr(router_logits), _ptr(w13_local), _ptr(w2_local), T, H, I2 // 2, E, top_k,
                                 local_expert_offset, n_local, _ptr(out), _ptr(workspace), workspace.numel(),
                                 _stream(stream), flags)
    if check and st != MOE_OK:
        raise MoeError(st, "moe_forward_local")
    return st


def moe_route_grouped(router_logits, top_k: int, router: GroupedRouter, topk_ids, topk_weights, expert_offsets,
                      sorted_to_flat, flat_to_sorted, workspace, stream=None, check: bool = True) -> int:
    T, E = router_logits.shape
    st = lib().moe_route_grouped(_ptr(router_logits), T, E, top_k, ctypes.byref(router), _ptr(topk_ids), _ptr(topk_weights),
                                 _ptr(expert_offsets), _ptr(sorted_to_flat), _ptr(flat_to_sorted), _ptr(workspace),
                                 workspace.numel(), _stream(stream))
    if check and st != MOE_OK:
        raise MoeError(st, "moe_route_grouped")
    return st


def moe_forward_grouped(x, router_logits, w13, w2, top_k: int, router: GroupedRouter, out, workspace, stream=None,
                        flags: int = 0, local_expert_offset: int = 0, check: bool = True) -> int:
    """The layer with the grouped sigmoid router; w13 may hold a local subset of the experts."""
    T, H = x.shape
    E = router_logits.shape[1]
    n_local, I2, _ = w13.shape
    st = lib().moe_forward_grouped(_ptr(x), _ptr(router_logits), _ptr(w13), _ptr(w2), T, H, I2 // 2, E, top_k,
                                   ctypes.byref(router), local_expert_offset, n_local, _ptr(out), _ptr(workspace),
                                   workspace.numel(), _stream(stream), flags)
    if check and st != MOE_OK:
        raise MoeError(st, "moe_forward_grouped")
    return st


def moe_forward_fp8w(x, router_logits, w13_q, w13_scale, w2_q, w2_scale, top_k: int, out, workspace, stream=None,
                     stage_events=None, check: bool = True) -> int:
    """The layer with FP8 (E4M3, uint8 codes) weights and one fp32 scale per 128 x 128 block."""
    T, H = x.shape
    E, I2, _ = w13_q.shape
    handles = None
    if stage_events is not None:
        handles = (ctypes.c_void_p * (len(STAGE_NAMES) + 1))(*[e.cuda_event for e in stage_events])
    st = lib().moe_forward_fp8w(_ptr(x), _ptr(router_logits), _ptr(w13_q), _ptr(w13_scale), _ptr(w2_q), _ptr(w2_scale),
                                T, H, I2 // 2, E, top_k, _ptr(out), _ptr(workspace), workspace.numel(), _stream(stream),
                                handles)
    if check and st != MOE_OK:
        raise MoeError(st, "moe_forward_fp8w")
    return st


def moe_mxfp8_workspace_bytes(T: int, H: int, I: int, E: int, top_k: int) -> int:
    return int(lib().moe_mxfp8_workspace_bytes(T, H, I, E, top_k))


def moe_mxfp8_workspace_layout(T: int, H: int, I: int, E: int, top_k: int) -> MxWorkspaceLayout:
    L = MxWorkspaceLayout()
    st = lib().moe_mxfp8_workspace_layout(T, H, I, E, top_k, ctypes.byref(L))
    if st != MOE_OK:
        raise MoeError(st, "moe_mxfp8_workspace_layout")
    return L


def moe_mxfp8_pack_scales(scales, gate_up: bool, stream=None) -> torch.Tensor:
    """Repack plain MX scale bytes [E, rows, K/32] of a weight tensor into the atoms moe_forward_mxfp8 reads."""
    E, rows, kb = scales.shape
    packed = torch.empty(scales.numel(), dtype=torch.uint8, device=scales.device)
    st = lib().moe_mxfp8_pack_scales(_ptr(scales), E, rows, kb * 32, int(gate_up), _ptr(packed), _stream(stream))
    if st != MOE_OK:
        raise MoeError(st, "moe_mxfp8_pack_scales")
    return packed


def moe_mxfp8_quantize_rows(x, stream=None):
    """MX quantisation of bf16 rows [R,K]: (codes uint8 [R,K], scale bytes uint8 [R,K/32])."""
    R, K = x.shape
    codes = torch.empty((R, K), dtype=torch.uint8, device=x.device)
    scales = torch.empty((R, K // 32), dtype=torch.uint8, device=x.device)
    st = lib().moe_mxfp8_quantize_rows(_ptr(x), R, K, _ptr(codes), _ptr(scales), _stream(stream))
    if st != MOE_OK:
        raise MoeError(st, "moe_mxfp8_quantize_rows")
    return codes, scales


def moe_forward_mxfp8(x, router_logits, w13_q, w13_sf_packed, w2_q, w2_sf_packed, top_k: int, out, workspace,
                      stream=None, stage_events=None, local_expert_offset: int = 0, router: GroupedRouter = None,
                      check: bool = True) -> int:
    """The layer in MX FP8 (E4M3 codes, packed E8M0 scale bytes); w13_q may hold a local subset of the experts;
    ``router`` = None for the softmax router, else a grouped_router(...)."""
    T, H = x.shape
    E = router_logits.shape[1]
    n_local, I2, _ = w13_q.shape
    handles = None
    if stage_events is not None:
        handles = (ctypes.c_void_p * (len(STAGE_NAMES) + 1))(*[e.cuda_event for e in stage_events])
    st = lib().moe_forward_mxfp8(_ptr(x), _ptr(router_logits), _ptr(w13_q), _ptr(w13_sf_packed), _ptr(w2_q),
                                 _ptr(w2_sf_packed), T, H, I2 // 2, E, top_k, None if router is None else ctypes.byref(router),
                                 local_expert_offset, n_local, _ptr(out), _ptr(workspace), workspace.numel(),
                                 _stream(stream), handles)
    if check and st != MOE_OK:
        raise MoeError(st, "moe_forward_mxfp8")
    return st


def moe_forward_mxfp8_host(x_host, router_logits_host, w13_q, w13_sf_packed, w2_q, w2_sf_packed, top_k: int, out_host,
                           workspace, stream=None, local_expert_offset: int = 0, router: GroupedRouter = None,
                           check: bool = True) -> int:
    """moe_forward_mxfp8 with CPU tensors for x, the router logits and the result (pinned for asynchronous copies)."""
    T, H = x_host.shape
    E = router_logits_host.shape[1]
    n_local, I2, _ = w13_q.shape
    st = lib().moe_forward_mxfp8_host(_ptr(x_host), _ptr(router_logits_host), _ptr(w13_q), _ptr(w13_sf_packed), _ptr(w2_q),
                                      _ptr(w2_sf_packed), T, H, I2 // 2, E, top_k,
                                      None if router is None else ctypes.byref(router), local_expert_offset, n_local,
                                      _ptr(out_host), _ptr(workspace), workspace.numel(), _stream(stream))
    if check and st != MOE_OK:
        raise MoeError(st, "moe_forward_mxfp8_host")
    return st


def mx_workspace_views(workspace: torch.Tensor, T: int, H: int, I: int, E: int, top_k: int) -> dict:
    """Typed views of what a moe_forward_mxfp8 call left in ``workspace`` (scale atoms as [K/128, atoms, 512])."""
    L = moe_mxfp8_workspace_layout(T, H, I, E, top_k)
    A = T * top_k
    n = int(L.sf_atoms)

    def view(off, nbytes, dtype, shape):
        return workspace[off:off + nbytes].view(dtype).view(shape)

    return dict(
        status=view(L.status, 16, torch.int32, (4,)),
        topk_ids=view(L.topk_ids, A * 4, torch.int32, (T, top_k)),
        topk_weights=view(L.topk_weights, A * 4, torch.float32, (T, top_k)),
        expert_offsets=view(L.expert_offsets, (E + 1) * 4, torch.int32, (E + 1,)),
        sorted_to_flat=view(L.sorted_to_flat, A * 4, torch.int32, (A,)),
        flat_to_sorted=view(L.flat_to_sorted, A * 4, torch.int32, (A,)),
        x_q=view(L.x_q, A * H, torch.uint8, (A, H)),
        x_sf=view(L.x_sf, (H // 128) * n * 512, torch.uint8, (H // 128, n, 512)),
        h_q=view(L.h_q, A * I, torch.uint8, (A, I)),
        h_sf=view(L.h_sf, (I // 128) * n * 512, torch.uint8, (I // 128, n, 512)),
        y=view(L.y, A * H * 2, torch.bfloat16, (A, H)),
        sf_atoms=n,
        tile_rows=int(L.tile_rows),
    )


STAGE_NAMES = ("route", "gather", "gemm1_swiglu", "gemm2", "combine")
NUM_STAGE_EVENTS = len(STAGE_NAMES) + 1


def make_stage_events() -> list:
    """CUDA events for moe_forward_staged; each is recorded once so that its handle exists."""
    events = [torch.cuda.Event(enable_timing=True) for _ in range(NUM_STAGE_EVENTS)]
    for e in events:
        e.record()
    torch.cuda.synchronize()
    return events


def moe_forward_staged(x, router_logits, w13, w2, top_k: int, out, workspace, stage_events, stream=None,
                       flags: int = 0, local_expert_offset: int = 0, check: bool = True) -> int:
    """moe_forward (or moe_forward_local when w13 holds fewer experts than the router has columns) that
    records ``stage_events`` (from make_stage_events) around the five stages."""
    T, H = x.shape
    E = router_logits.shape[1]
    n_local, I2, _ = w13.shape
    handles = (ctypes.c_void_p * NUM_STAGE_EVENTS)(*[e.cuda_event for e in stage_events])
    st = lib().moe_forward_staged(_ptr(x), _ptr(router_logits), _ptr(w13), _ptr(w2), T, H, I2 // 2, E, top_k,
                                  local_expert_offset, n_local, _ptr(out), _ptr(workspace), workspace.numel(),
                                  _stream(stream), flags, handles)
    if check and st != MOE_OK:
        raise MoeError(st, "moe_forward_staged")
    return st


def moe_forward_host(x_host, router_logits_host, w13, w2, top_k: int, out_host, workspace, stream=None,
                     local_expert_offset: int = 0, check: bool = True) -> int:
    """x_host / router_logits_host / out_host are CPU tensors (pinned for asynchronous copies); w13 / w2 are
    the resident experts on the device (all E of them, or a local subset starting at local_expert_offset)."""
    T, H = x_host.shape
    E = router_logits_host.shape[1]
    n_local, I2, _ = w13.shape
    st = lib().moe_forward_host(_ptr(x_host), _ptr(router_logits_host), _ptr(w13), _ptr(w2), T, H, I2 // 2, E, top_k,
                                local_expert_offset, n_local, _ptr(out_host), _ptr(workspace), workspace.numel(),
                                _stream(stream))
    if check and st != MOE_OK:
        raise MoeError(st, "moe_forward_host")
    return st


def moe_selftest_wait_timeout(workspace, stream=None) -> int:
    """Enqueues the bounded-wait self-test; moe_last_status(workspace) must then report MOE_ERR_DEVICE_TIMEOUT (-7)."""
    st = lib().moe_selftest_wait_timeout(_ptr(workspace), workspace.numel(), _stream(stream))
    if st != MOE_OK:
        raise MoeError(st, "moe_selftest_wait_timeout")
    return st


def moe_last_status(workspace, stream=None) -> int:
    return int(lib().moe_last_status(_ptr(workspace), _stream(stream)))


def workspace_views(workspace: torch.Tensor, T: int, H: int, I: int, E: int, top_k: int) -> dict:
    """Typed views of the routing arrays and intermediates a moe_forward call left in ``workspace``."""
    L = moe_workspace_layout(T, H, I, E, top_k)
    A = T * top_k

    def view(off, nbytes, dtype, shape):
        return workspace[off:off + nbytes].view(dtype).view(shape)

    return dict(
        status=view(L.status, 16, torch.int32, (4,)),
        topk_ids=view(L.topk_ids, A * 4, torch.int32, (T, top_k)),
        topk_weights=view(L.topk_weights, A * 4, torch.float32, (T, top_k)),
        expert_offsets=view(L.expert_offsets, (E + 1) * 4, torch.int32, (E + 1,)),
        sorted_to_flat=view(L.sorted_to_flat, A * 4, torch.int32, (A,)),
        flat_to_sorted=view(L.flat_to_sorted, A * 4, torch.int32, (A,)),
        x_perm=view(L.x_perm, A * H * 2, torch.bfloat16, (A, H)),
        h=view(L.h, A * I * 2, torch.bfloat16, (A, I)),
        y=view(L.y, A * H * 2, torch.bfloat16, (A, H)),
    )


# ---- second workload: paged grouped-query decode attention (include/gqa_decode.h) -------------------------------
def gqa_decode_workspace_bytes(B: int, Hq: int, Hkv: int, D: int, max_kv_len: int) -> int:
    return int(lib().gqa_decode_workspace_bytes(B, Hq, Hkv, D, max_kv_len))


def gqa_selftest_wait_timeout(workspace, stream=None) -> int:
    """Enqueue the decode kernel's bounded-wait self-test; read the outcome with moe_last_status(workspace)."""
    st = lib().gqa_selftest_wait_timeout(_ptr(workspace), workspace.numel(), _stream(stream))
    if st != MOE_OK:
        raise MoeError(st, "gqa_selftest_wait_timeout")
    return st


def gqa_decode_split_tokens(B: int, Hq: int, Hkv: int, D: int, max_kv_len: int) -> int:
    return int(lib().gqa_decode_split_tokens(B, Hq, Hkv, D, max_kv_len))


def gqa_paged_decode(q, k_cache, v_cache, kv_indptr, kv_indices, kv_last_page_len, max_kv_len: int, sm_scale: float, out,
                     workspace, lse=None, stream=None, check: bool = True) -> int:
    """One decode step: q [B,Hq,D] bf16, caches [num_pages,page_size,Hkv,D] bf16, int32 page tables, out [B,Hq,D]
    bf16, lse [B,Hq] f32 or None.  Marshalling only."""
    B, Hq, D = q.shape
    num_pages, page_size, Hkv, _ = k_cache.shape
    st = lib().gqa_paged_decode(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(kv_indptr), _ptr(kv_indices),
                                _ptr(kv_last_page_len), B, Hq, Hkv, D, page_size, num_pages, int(max_kv_len),
                                float(sm_scale), _ptr(out), _ptr(lse), _ptr(workspace), workspace.numel(), _stream(stream))
    if check and st != MOE_OK:
        raise MoeError(st, "gqa_paged_decode")
    return st
