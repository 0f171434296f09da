"""Thin ctypes binding of libmoehub.so (the C ABI in include/moehub.h).

Argument marshalling only: every step of the path runs in the CUDA kernels behind the C ABI.
torch is used for device memory and streams.  There is no CPU fallback: if the library is
missing or no CUDA device is present, calls raise.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libmoehub.so")
_lib = None

MOE_OK = 0
DTYPE_FP32, DTYPE_BF16 = 0, 1
DISPATCH_SCAN, DISPATCH_ATOMIC_STATIC, DISPATCH_ATOMIC_PAGED, DISPATCH_ATOMIC_ORDERED = 0, 1, 2, 3
TILE_ROWS = 128
STAGES = ["route", "dispatch", "worklist", "gemm1", "gemm2", "combine"]

EXPORTS = ["moe_dispatch_noalloc", "moe_dispatch_ep", "moe_ep_tiles", "moe_combine_ep", "moe_pool_tiles", "moe_workspace_bytes", "moe_plan_create", "moe_plan_destroy", "moe_route",
           "moe_dispatch", "moe_expert_ffn", "moe_expert_ffn_push", "moe_combine", "moe_combine_staged", "moe_layer", "moe_layer_host", "moe_layer_host_submit", "moe_layer_host_wait", "moe_layer_timed",
           "moe_layer_buffer", "moe_availability_trace",
           "moe_ffn_clock_mhz", "moe_last_launch_count", "moe_last_status", "moe_last_cuda_error", "moe_strerror"]


class MoeConfig(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int32), ("H", ctypes.c_int32), ("E", ctypes.c_int32), ("R", ctypes.c_int32),
                ("K", ctypes.c_int32), ("F", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("renormalize", ctypes.c_int32), ("dispatch_mode", ctypes.c_int32),
                ("identity_experts", ctypes.c_int32), ("ffn_kernel", ctypes.c_int32), ("ffn_split", ctypes.c_int32),
                ("ffn_hot_min_tiles", ctypes.c_int32), ("ffn_thin_tiles", ctypes.c_int32),
                ("overlap", ctypes.c_int32), ("combine_mode", ctypes.c_int32),
                ("tp_shards", ctypes.c_int32), ("route_filter", ctypes.c_int32),
                ("capacity_rows", ctypes.c_int64), ("spin_limit", ctypes.c_uint64), ("wait_limit_ns", ctypes.c_uint64)]


class EpPeer(ctypes.Structure):
    """moe_ep_peer_t: one rank's receive buffers as device pointers valid on the calling GPU."""
    _fields_ = [("recv", ctypes.c_void_p), ("row_pointer", ctypes.c_void_p), ("tile_count", ctypes.c_void_p),
                ("src_info", ctypes.c_void_p), ("rows_done", ctypes.c_void_p)]


class MoeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


def lib() -> ctypes.CDLL:
    """Loads libmoehub.so (built in-tree by build.py). Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(_SO):
            raise RuntimeError(f"{_SO} not found: build it with paper_2605_05888_b200/build.py (needs nvcc)")
        L = ctypes.CDLL(_SO)
        vp, i32p, fp = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
        cfgp = ctypes.POINTER(MoeConfig)
        L.moe_pool_tiles.argtypes = [cfgp, ctypes.POINTER(ctypes.c_int64)]
        L.moe_workspace_bytes.argtypes = [cfgp, ctypes.POINTER(ctypes.c_size_t)]
        L.moe_plan_create.argtypes = [cfgp, vp, ctypes.c_size_t, ctypes.POINTER(vp)]
        L.moe_plan_destroy.argtypes = [vp]
        L.moe_route.argtypes = [vp, vp, vp, fp, i32p, fp, vp]
        L.moe_dispatch.argtypes = [vp, vp, i32p, vp, i32p, i32p, i32p, i32p, i32p, i32p, vp]
        L.moe_dispatch_noalloc.argtypes = [cfgp, vp, i32p, vp, i32p, i32p, i32p, i32p, i32p, vp]
        L.moe_dispatch_ep.argtypes = [cfgp, ctypes.c_int32, ctypes.POINTER(EpPeer), ctypes.c_int64, vp, i32p, i32p, i32p, vp]
        L.moe_ep_tiles.argtypes = [ctypes.c_int32, ctypes.c_int64, i32p, i32p, i32p, vp]
        L.moe_combine_ep.argtypes = [cfgp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.c_int64, vp, i32p, i32p, i32p, vp]
        L.moe_expert_ffn.argtypes = [vp, vp, i32p, vp, vp, vp, vp, i32p, i32p, vp]
        L.moe_combine.argtypes = [vp, vp, i32p, fp, vp, vp]
        L.moe_expert_ffn_push.argtypes = [vp, vp, i32p, i32p, vp, vp, vp, vp, i32p, i32p, vp]
        L.moe_combine_staged.argtypes = [vp, vp, i32p, fp, vp, vp]
        L.moe_layer.argtypes = [vp] * 9
        L.moe_layer_host.argtypes = [vp] * 9
        L.moe_layer_host_submit.argtypes = [vp] * 9 + [ctypes.POINTER(ctypes.c_int64)]
        L.moe_layer_host_wait.argtypes = [vp, ctypes.c_int64]
        L.moe_layer_timed.argtypes = [vp] * 9 + [ctypes.POINTER(ctypes.c_float)]
        L.moe_layer_buffer.argtypes = [vp, ctypes.c_int, ctypes.POINTER(vp)]
        L.moe_availability_trace.argtypes = [vp, ctypes.c_int]
        L.moe_ffn_clock_mhz.argtypes = [vp, vp, ctypes.c_int, ctypes.POINTER(ctypes.c_float)]
        L.moe_last_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
        L.moe_last_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
        L.moe_last_cuda_error.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_char_p)]
        L.moe_strerror.argtypes = [ctypes.c_int]
        L.moe_strerror.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name != "moe_strerror":
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().moe_strerror(code).decode()


def _check(rc: int, where: str) -> None:
    if rc != MOE_OK:
        raise MoeError(rc, where)


def _ptr(t) -> int | None:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous()
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def make_config(T, H, E, R, K, F, dtype, renormalize=0, dispatch_mode=DISPATCH_ATOMIC_PAGED, identity_experts=0,
                ffn_kernel=0, capacity_rows=0, spin_limit=0, ffn_split=0, wait_limit_ns=0,
                ffn_hot_min_tiles=0, ffn_thin_tiles=0, overlap=0, combine_mode=0, tp_shards=0, route_filter=0) -> MoeConfig:
    return MoeConfig(T, H, E, R, K, F, dtype, int(renormalize), dispatch_mode, int(identity_experts), ffn_kernel, int(ffn_split),
                     int(ffn_hot_min_tiles), int(ffn_thin_tiles), int(overlap), int(combine_mode), int(tp_shards), int(route_filter), capacity_rows, spin_limit, wait_limit_ns)


def moe_pool_tiles(cfg: MoeConfig) -> int:
    out = ctypes.c_int64()
    _check(lib().moe_pool_tiles(ctypes.byref(cfg), ctypes.byref(out)), "moe_pool_tiles")
    return out.value


def moe_workspace_bytes(cfg: MoeConfig) -> int:
    out = ctypes.c_size_t()
    _check(lib().moe_workspace_bytes(ctypes.byref(cfg), ctypes.byref(out)), "moe_workspace_bytes")
    return out.value


def moe_dispatch_noalloc(cfg: MoeConfig, x, topk_idx, recv, expert_count, tile_expert, src_info, slot_of, status,
                         stream=None) -> None:
    """Paged dispatch that needs no plan and no workspace: for callers that cannot allocate device
    memory.  Its scratch is a fixed array inside the library (T <= 16384, E <= 256).  `status` is a
    caller-owned int32[2] device tensor that receives (code, detail)."""
    _check(lib().moe_dispatch_noalloc(ctypes.byref(cfg), _ptr(x), _ptr(topk_idx), _ptr(recv), _ptr(expert_count),
                                      _ptr(tile_expert), _ptr(src_info), _ptr(slot_of), _ptr(status),
                                      _stream(stream)), "moe_dispatch_noalloc")


def moe_dispatch_ep(cfg: MoeConfig, rank: int, peers, cap_rows: int, x, topk_idx, slot_of, status, stream=None) -> None:
    """Dispatch of THIS rank's tokens into the owning ranks' receive regions (real expert parallelism).
    peers: one dict per rank with the tensors (or device pointers valid on this GPU) recv, row_pointer, tile_count,
    src_info, rows_done.  cfg.T is this rank's token count, cfg.E the experts of all ranks."""
    table = (EpPeer * len(peers))()
    for r, q in enumerate(peers):
        table[r] = EpPeer(*(_ptr(q[k]) for k in ("recv", "row_pointer", "tile_count", "src_info", "rows_done")))
    _check(lib().moe_dispatch_ep(ctypes.byref(cfg), rank, table, cap_rows, _ptr(x), _ptr(topk_idx), _ptr(slot_of),
                                 _ptr(status), _stream(stream)), "moe_dispatch_ep")


def moe_ep_tiles(experts_local: int, cap_rows: int, row_pointer, expert_count, tile_expert, stream=None) -> None:
    """The owner's tile table (static regions of cap_rows rows) from its allocation pointers."""
    _check(lib().moe_ep_tiles(experts_local, cap_rows, _ptr(row_pointer), _ptr(expert_count), _ptr(tile_expert),
                              _stream(stream)), "moe_ep_tiles")


def moe_combine_ep(cfg: MoeConfig, staging, rows_back, cap_rows: int, out_rows, src_info, expert_count, status,
                   stream=None) -> None:
    """The owner's result rows back to their source ranks' staging buffers.  staging, rows_back: one tensor (or
    device pointer valid on this GPU) per rank."""
    n = len(staging)
    st = (ctypes.c_void_p * n)(*(_ptr(t) for t in staging))
    rb = (ctypes.c_void_p * n)(*(_ptr(t) for t in rows_back))
    _check(lib().moe_combine_ep(ctypes.byref(cfg), st, rb, cap_rows, _ptr(out_rows), _ptr(src_info), _ptr(expert_count),
                                _ptr(status), _stream(stream)), "moe_combine_ep")


class Plan:
    """Owns a moe_plan_t and the torch-allocated workspace it points into."""

    def __init__(self, cfg: MoeConfig, device="cuda"):
        if not torch.cuda.is_available():
            raise RuntimeError("moehub needs a CUDA device; there is no CPU path")
        self.cfg = cfg
        self.device = torch.device(device)
        self.P = moe_pool_tiles(cfg)
        nbytes = moe_workspace_bytes(cfg)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            h = ctypes.c_void_p()
            _check(lib().moe_plan_create(ctypes.byref(cfg), base, nbytes, ctypes.byref(h)), "moe_plan_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.moe_plan_destroy(self.handle)
            self.handle = None

    __del__ = close

    # ---- the C ABI, same names -------------------------------------------------------------
    def moe_route(self, x, wr, bias, topk_idx, topk_w, stream=None):
        _check(lib().moe_route(self.handle, _ptr(x), _ptr(wr), _ptr(bias), _ptr(topk_idx), _ptr(topk_w),
                               _stream(stream)), "moe_route")

    def moe_dispatch(self, x, topk_idx, recv, expert_count, tile_expert, src_info, slot_of, tile_count=None,
                     rows_done=None, stream=None):
        _check(lib().moe_dispatch(self.handle, _ptr(x), _ptr(topk_idx), _ptr(recv), _ptr(expert_count),
                                  _ptr(tile_expert), _ptr(src_info), _ptr(slot_of), _ptr(tile_count), _ptr(rows_done),
                                  _stream(stream)), "moe_dispatch")

    def moe_expert_ffn(self, recv, tile_expert, wg, wu, wd, out_rows, tile_count=None, rows_done=None, stream=None):
        _check(lib().moe_expert_ffn(self.handle, _ptr(recv), _ptr(tile_expert), _ptr(wg), _ptr(wu), _ptr(wd),
                                    _ptr(out_rows), _ptr(tile_count), _ptr(rows_done), _stream(stream)),
               "moe_expert_ffn")

    def moe_expert_ffn_push(self, recv, tile_expert, src_info, wg, wu, wd, staged, tile_count=None, rows_done=None,
                            stream=None):
        _check(lib().moe_expert_ffn_push(self.handle, _ptr(recv), _ptr(tile_expert), _ptr(src_info), _ptr(wg), _ptr(wu),
                                         _ptr(wd), _ptr(staged), _ptr(tile_count), _ptr(rows_done), _stream(stream)),
               "moe_expert_ffn_push")

    def moe_combine_staged(self, staged, slot_of, topk_w, y, stream=None):
        _check(lib().moe_combine_staged(self.handle, _ptr(staged), _ptr(slot_of), _ptr(topk_w), _ptr(y), _stream(stream)),
               "moe_combine_staged")

    def moe_combine(self, rows, slot_of, topk_w, y, stream=None):
        _check(lib().moe_combine(self.handle, _ptr(rows), _ptr(slot_of), _ptr(topk_w), _ptr(y), _stream(stream)),
               "moe_combine")

    def moe_layer(self, x, wr, bias, wg, wu, wd, y, stream=None):
        _check(lib().moe_layer(self.handle, _ptr(x), _ptr(wr), _ptr(bias), _ptr(wg), _ptr(wu), _ptr(wd), _ptr(y),
                               _stream(stream)), "moe_layer")

    def moe_layer_host(self, h_x, wr, bias, wg, wu, wd, h_y, stream=None):
        """h_x, h_y: HOST tensors (pinned for asynchronous copies); weights: device tensors."""
        assert not h_x.is_cuda and not h_y.is_cuda
        _check(lib().moe_layer_host(self.handle, _ptr(h_x), _ptr(wr), _ptr(bias), _ptr(wg), _ptr(wu), _ptr(wd),
                                    _ptr(h_y), _stream(stream)), "moe_layer_host")

    def moe_layer_host_submit(self, h_x, wr, bias, wg, wu, wd, h_y, stream=None) -> int:
        """Pipelined host-buffer step: returns a ticket at once; moe_layer_host_wait(ticket) blocks until h_y is
        complete. At most two steps in flight; h_x, h_y pinned."""
        assert not h_x.is_cuda and not h_y.is_cuda
        t = ctypes.c_int64()
        _check(lib().moe_layer_host_submit(self.handle, _ptr(h_x), _ptr(wr), _ptr(bias), _ptr(wg), _ptr(wu), _ptr(wd),
                                           _ptr(h_y), _stream(stream), ctypes.byref(t)), "moe_layer_host_submit")
        return t.value

    def moe_layer_host_wait(self, ticket: int) -> None:
        _check(lib().moe_layer_host_wait(self.handle, ticket), "moe_layer_host_wait")

    def moe_layer_timed(self, x, wr, bias, wg, wu, wd, y, stream=None) -> list[float]:
        """Runs the layer once with an event after every kernel; returns ms per stage (see STAGES)."""
        ms = (ctypes.c_float * len(STAGES))()
        _check(lib().moe_layer_timed(self.handle, _ptr(x), _ptr(wr), _ptr(bias), _ptr(wg), _ptr(wu), _ptr(wd),
                                     _ptr(y), _stream(stream), ms), "moe_layer_timed")
        return list(ms)

    def moe_layer_buffer(self, which: int) -> int:
        out = ctypes.c_void_p()
        _check(lib().moe_layer_buffer(self.handle, which, ctypes.byref(out)), "moe_layer_buffer")
        return out.value

    def moe_availability_trace(self, enable: bool) -> None:
        _check(lib().moe_availability_trace(self.handle, int(enable)), "moe_availability_trace")

    def moe_ffn_clock_mhz(self, reset: bool = True, stream=None) -> float:
        out = ctypes.c_float()
        _check(lib().moe_ffn_clock_mhz(self.handle, _stream(stream), int(reset), ctypes.byref(out)), "moe_ffn_clock_mhz")
        return out.value

    def moe_last_launch_count(self) -> int:
        out = ctypes.c_int32()
        _check(lib().moe_last_launch_count(self.handle, ctypes.byref(out)), "moe_last_launch_count")
        return out.value

    def moe_last_cuda_error(self) -> tuple[int, str]:
        """(step of moe_layer that met a CUDA error, the error's name); step 0: none."""
        step, name = ctypes.c_int32(), ctypes.c_char_p()
        _check(lib().moe_last_cuda_error(self.handle, ctypes.byref(step), ctypes.byref(name)), "moe_last_cuda_error")
        return step.value, (name.value or b"").decode()

    def moe_last_status(self, stream=None) -> tuple[int, int]:
        code, detail = ctypes.c_int32(), ctypes.c_int32()
        _check(lib().moe_last_status(self.handle, _stream(stream), ctypes.byref(code), ctypes.byref(detail)),
               "moe_last_status")
        return code.value, detail.value

    # ---- convenience: read one of moe_layer's internal buffers back as a torch tensor ----------
    def layer_tensor(self, which: int) -> torch.Tensor:
        c = self.cfg
        rows = self.P * TILE_ROWS
        el = torch.bfloat16 if c.dtype == DTYPE_BF16 else torch.float32
        tp = max(1, c.tp_shards)                     # with TP shards the stages see E*tp experts, K*tp picks, width F/tp
        K, E, F = c.K * tp, c.E * tp, c.F // tp
        shapes = {0: ((c.T, K), torch.int32), 1: ((c.T, K), torch.float32), 2: ((rows, c.H), el),
                  3: ((E,), torch.int32), 4: ((self.P,), torch.int32), 5: ((rows,), torch.int32),
                  6: ((c.T, K), torch.int32), 7: ((rows, c.H), el), 8: ((self.P + 2,), torch.int64),
                  9: ((self.P * ((F + 127) // 128 + (c.H + 255) // 256), 4), torch.int64)}
        shape, dt = shapes[which]
        ptr = self.moe_layer_buffer(which)
        off = ptr - self.workspace.data_ptr()
        n = 1
        for s in shape:
            n *= s
        nbytes = n * torch.empty(0, dtype=dt).element_size()
        return self.workspace[off: off + nbytes].view(dt).view(shape)
