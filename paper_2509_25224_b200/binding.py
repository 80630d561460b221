"""ctypes binding of libamla.so -- argument marshalling only.

Every step of the decode path runs inside the library's CUDA kernels; torch is
used here for device memory and streams.  There is no fallback: if the library
is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libamla.so")

AMLA_OK = 0
RESCALE_ALG2 = 0
RESCALE_FOLD = 1
RESCALE_FMUL = 2
FLAG_UNGUARDED_ADD = 4
FLAG_KERNEL_SIMT = 8
FLAG_KERNEL_ROWS128 = 16
DEFAULT_TAU = 8


def lazy(tau: int) -> int:
    """Flag bits for a lazy-reference threshold of `tau` octaves (0 = Algorithm 2 to the letter)."""
    if not 0 <= int(tau) <= 15:
        raise ValueError("tau must be in 0..15")
    return int(tau) << 8


DEFAULT_FLAGS = RESCALE_ALG2 | lazy(DEFAULT_TAU)   # what amla_mla_decode (without _ex) uses

EXPORTS = [
    "amla_status_string", "amla_mla_decode_workspace_size", "amla_mla_decode", "amla_mla_decode_ex",
    "amla_check_status", "amla_last_launch_count", "amla_plan_host", "amla_profile_enable",
    "amla_profile_last_ms", "amla_mla_decode_static", "amla_static_check_status", "amla_wait_selftest",
    "amla_validate_paging_host", "amla_mla_decode_fp8", "amla_mla_decode_fp8_workspace_size",
]

_lib = None


class AmlaError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} ({code})")
        self.code = code


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2509_25224_b200.build` "
                "(there is no CPU or PyTorch fallback for the decode path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        L.amla_status_string.argtypes = [i32]
        L.amla_status_string.restype = ctypes.c_char_p
        L.amla_mla_decode_workspace_size.argtypes = [i32, i32, i32, i32, i32, ctypes.POINTER(sz)]
        L.amla_mla_decode_workspace_size.restype = i32
        dec = [vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, vp, vp, vp, sz, vp]
        L.amla_mla_decode.argtypes = dec
        L.amla_mla_decode.restype = i32
        L.amla_mla_decode_ex.argtypes = dec + [i32]
        L.amla_mla_decode_ex.restype = i32
        L.amla_mla_decode_fp8_workspace_size.argtypes = [i32, i32, i32, i32, i32, ctypes.POINTER(sz)]
        L.amla_mla_decode_fp8_workspace_size.restype = i32
        L.amla_mla_decode_fp8.argtypes = [vp, vp, f32, vp, vp, f32, i32, i32, i32, i32, i32, vp, vp, vp, sz, vp, i32]
        L.amla_mla_decode_fp8.restype = i32
        L.amla_mla_decode_static.argtypes = [vp, vp, vp, vp, f32, i32, i32, i32, i32, i32, vp, vp, vp]
        L.amla_mla_decode_static.restype = i32
        L.amla_static_check_status.argtypes = [vp]
        L.amla_static_check_status.restype = i32
        L.amla_wait_selftest.argtypes = [vp, ctypes.c_ulonglong, vp]
        L.amla_wait_selftest.restype = i32
        L.amla_validate_paging_host.argtypes = [vp, vp, i32, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
        L.amla_validate_paging_host.restype = i32
        L.amla_check_status.argtypes = [vp, vp]
        L.amla_check_status.restype = i32
        L.amla_last_launch_count.argtypes = []
        L.amla_last_launch_count.restype = i32
        L.amla_plan_host.argtypes = [vp, i32, i32, i32, i32, vp, i32]
        L.amla_plan_host.restype = i32
        L.amla_profile_enable.argtypes = [i32]
        L.amla_profile_enable.restype = i32
        L.amla_profile_last_ms.argtypes = [ctypes.POINTER(ctypes.c_float)]
        L.amla_profile_last_ms.restype = i32
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().amla_status_string(int(code)).decode()


def workspace_size(B: int, Sq: int, H: int, max_blocks_per_seq: int, device: int = 0) -> int:
    n = ctypes.c_size_t(0)
    rc = lib().amla_mla_decode_workspace_size(B, Sq, H, max_blocks_per_seq, device, ctypes.byref(n))
    if rc != AMLA_OK:
        raise AmlaError(rc, "amla_mla_decode_workspace_size")
    return int(n.value)


def plan_host(seqlens, Sq: int, H: int, num_parts: int) -> np.ndarray:
    """Host mirror of the split-KV schedule: int32 [n_units, 6] rows of
    (part, item, tile_begin, tile_end, slot, n_split).  Items are 128-row blocks with 64-key tiles for
    Sq*H <= 128, 256-row blocks with 128-key tiles above."""
    sl = np.ascontiguousarray(seqlens, dtype=np.int32)
    B = sl.shape[0]
    nrb = (Sq * H + 127) // 128
    cap = B * nrb + num_parts + 8
    units = np.zeros((cap, 6), dtype=np.int32)
    n = lib().amla_plan_host(sl.ctypes.data_as(ctypes.c_void_p), B, Sq, H, num_parts,
                             units.ctypes.data_as(ctypes.c_void_p), cap)
    if n < 0:
        raise AmlaError(n, "amla_plan_host")
    return units[:n].copy()


def mla_decode_raw(q_ptr: int, kv_ptr: int, bt_ptr: int, sl_ptr: int, scale: float, B: int, Sq: int, H: int,
                   num_blocks: int, max_blocks_per_seq: int, out_ptr: int, lse_ptr: int, ws_ptr: int,
                   ws_bytes: int, stream: int = 0, flags: int | None = None) -> None:
    """amla_mla_decode (flags None) or amla_mla_decode_ex on raw device addresses."""
    if flags is None:
        rc = lib().amla_mla_decode(q_ptr, kv_ptr, bt_ptr, sl_ptr, float(scale), B, Sq, H, num_blocks,
                                   max_blocks_per_seq, out_ptr, lse_ptr, ws_ptr, ws_bytes, stream)
    else:
        rc = lib().amla_mla_decode_ex(q_ptr, kv_ptr, bt_ptr, sl_ptr, float(scale), B, Sq, H, num_blocks,
                                      max_blocks_per_seq, out_ptr, lse_ptr, ws_ptr, ws_bytes, stream, int(flags))
    if rc != AMLA_OK:
        raise AmlaError(rc, "amla_mla_decode")


def mla_decode_static(q, kv_cache, block_table, seqlens, softmax_scale: float, out, lse) -> None:
    """amla_mla_decode_static on device tensors: the decode call that takes no workspace and allocates nothing
    (its scratch is a fixed array inside the library).  `out` and `lse` must be given -- this wrapper allocates
    nothing either.  Raises AmlaError(-6) when the problem exceeds the built-in scratch."""
    import torch

    B, Sq, H, _ = q.shape
    stream = torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        rc = lib().amla_mla_decode_static(q.data_ptr(), kv_cache.data_ptr(), block_table.data_ptr(), seqlens.data_ptr(),
                                          float(softmax_scale), B, Sq, H, kv_cache.shape[0], block_table.shape[1],
                                          out.data_ptr(), lse.data_ptr(), stream)
    if rc != AMLA_OK:
        raise AmlaError(rc, "amla_mla_decode_static")


def fp8_workspace_size(B: int, Sq: int, H: int, max_blocks_per_seq: int, device: int = 0) -> int:
    n = ctypes.c_size_t(0)
    rc = lib().amla_mla_decode_fp8_workspace_size(B, Sq, H, max_blocks_per_seq, device, ctypes.byref(n))
    if rc != AMLA_OK:
        raise AmlaError(rc, "amla_mla_decode_fp8_workspace_size")
    return int(n.value)


def mla_decode_fp8(q, kv_cache_e4m3, kv_scale: float, block_table, seqlens, softmax_scale: float, out=None, lse=None,
                   workspace=None, flags: int | None = None):
    """amla_mla_decode_fp8 on device tensors: q bf16 [B,Sq,H,576], kv_cache_e4m3 uint8 [num_blocks,64,576] (E4M3 bytes;
    element value = decode(byte) * kv_scale).  Returns (out bf16, lse fp32)."""
    import torch

    if kv_cache_e4m3.dtype != torch.uint8 or q.dtype != torch.bfloat16:
        raise ValueError("q must be bfloat16 and the cache uint8 (E4M3 bytes)")
    if block_table.dtype != torch.int32 or seqlens.dtype != torch.int32:
        raise ValueError("block_table and seqlens must be int32")
    if not (q.is_contiguous() and kv_cache_e4m3.is_contiguous() and block_table.is_contiguous() and seqlens.is_contiguous()):
        raise ValueError("inputs must be contiguous")
    B, Sq, H, d = q.shape
    if d != 576 or tuple(kv_cache_e4m3.shape[1:]) != (64, 576) or block_table.shape[0] != B or seqlens.shape[0] != B:
        raise ValueError("shape mismatch")
    dev = q.device
    if out is None:
        out = torch.empty((B, Sq, H, 512), dtype=torch.bfloat16, device=dev)
    if lse is None:
        lse = torch.empty((B, Sq, H), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = torch.empty(fp8_workspace_size(B, Sq, H, block_table.shape[1], dev.index or 0), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev).cuda_stream
    with torch.cuda.device(dev):
        rc = lib().amla_mla_decode_fp8(q.data_ptr(), kv_cache_e4m3.data_ptr(), float(kv_scale), block_table.data_ptr(),
                                       seqlens.data_ptr(), float(softmax_scale), B, Sq, H, kv_cache_e4m3.shape[0],
                                       block_table.shape[1], out.data_ptr(), lse.data_ptr(), workspace.data_ptr(),
                                       workspace.numel(), stream, DEFAULT_FLAGS if flags is None else int(flags))
    if rc != AMLA_OK:
        raise AmlaError(rc, "amla_mla_decode_fp8")
    return out, lse


def static_check_status(stream: int = 0) -> None:
    """Raises AmlaError(-5) if a bounded wait expired during the last amla_mla_decode_static call on this device."""
    rc = lib().amla_static_check_status(stream)
    if rc != AMLA_OK:
        raise AmlaError(rc, "amla_static_check_status")


def wait_selftest(workspace, limit_ns: int = 1_000_000, stream: int = 0) -> None:
    """Launches the bounded-wait self-test (a wait nothing satisfies, given up after limit_ns); afterwards
    check_status(workspace) raises AmlaError(-5)."""
    rc = lib().amla_wait_selftest(workspace.data_ptr(), int(limit_ns), stream)
    if rc != AMLA_OK:
        raise AmlaError(rc, "amla_wait_selftest")


def validate_paging_host(block_table, seqlens, num_blocks: int):
    """Host-side debug check of numpy copies of the paging inputs.  Returns None when they are consistent, else
    (bad_seq, bad_block) with bad_block = -1 for an out-of-range length."""
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    sl = np.ascontiguousarray(seqlens, dtype=np.int32)
    bs, bb = ctypes.c_int(-1), ctypes.c_int(-1)
    rc = lib().amla_validate_paging_host(bt.ctypes.data_as(ctypes.c_void_p), sl.ctypes.data_as(ctypes.c_void_p),
                                         bt.shape[0], int(num_blocks), bt.shape[1], ctypes.byref(bs), ctypes.byref(bb))
    if rc == AMLA_OK:
        return None
    if rc != -1:
        raise AmlaError(rc, "amla_validate_paging_host")
    return int(bs.value), int(bb.value)


def last_launch_count() -> int:
    return int(lib().amla_last_launch_count())


def profile_enable(on: bool) -> None:
    rc = lib().amla_profile_enable(1 if on else 0)
    if rc != AMLA_OK:
        raise AmlaError(rc, "amla_profile_enable")


def profile_last_ms():
    """(schedule_ms, decode_ms, combine_ms) of the last profiled call on this thread."""
    ms = (ctypes.c_float * 3)()
    rc = lib().amla_profile_last_ms(ms)
    if rc != AMLA_OK:
        raise AmlaError(rc, "amla_profile_last_ms")
    return float(ms[0]), float(ms[1]), float(ms[2])


def check_status(workspace, stream: int = 0) -> None:
    rc = lib().amla_check_status(workspace.data_ptr(), stream)
    if rc != AMLA_OK:
        raise AmlaError(rc, "amla_check_status")


def mla_decode(q, kv_cache, block_table, seqlens, softmax_scale: float, out=None, lse=None, workspace=None,
               flags: int | None = None):
    """Device tensors in, device tensors out (torch is the allocator and stream provider).

    q bf16 [B,Sq,H,576], kv_cache bf16 [num_blocks,64,576], block_table int32 [B,max_blocks],
    seqlens int32 [B].  Returns (out bf16 [B,Sq,H,512], lse fp32 [B,Sq,H]).
    """
    import torch

    if not (q.is_cuda and kv_cache.is_cuda and block_table.is_cuda and seqlens.is_cuda):
        raise ValueError("mla_decode needs CUDA tensors")
    if q.dtype != torch.bfloat16 or kv_cache.dtype != torch.bfloat16:
        raise ValueError("q and kv_cache must be bfloat16")
    if block_table.dtype != torch.int32 or seqlens.dtype != torch.int32:
        raise ValueError("block_table and seqlens must be int32")
    if not (q.is_contiguous() and kv_cache.is_contiguous() and block_table.is_contiguous() and seqlens.is_contiguous()):
        raise ValueError("inputs must be contiguous")
    B, Sq, H, d = q.shape
    if d != 576 or tuple(kv_cache.shape[1:]) != (64, 576) or block_table.shape[0] != B or seqlens.shape[0] != B:
        raise ValueError("shape mismatch")
    dev = q.device
    if out is None:
        out = torch.empty((B, Sq, H, 512), dtype=torch.bfloat16, device=dev)
    if lse is None:
        lse = torch.empty((B, Sq, H), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = torch.empty(workspace_size(B, Sq, H, block_table.shape[1], dev.index or 0),
                                dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev).cuda_stream
    with torch.cuda.device(dev):
        mla_decode_raw(q.data_ptr(), kv_cache.data_ptr(), block_table.data_ptr(), seqlens.data_ptr(),
                       softmax_scale, B, Sq, H, kv_cache.shape[0], block_table.shape[1], out.data_ptr(),
                       lse.data_ptr(), workspace.data_ptr(), workspace.numel(), stream, flags)
    return out, lse


class HostSession:
    """End-to-end path with HOST buffers: pinned staging, device buffers and workspace are created
    once; each ``run`` copies the inputs host->device, decodes, and copies out/lse device->host."""

    def __init__(self, B, Sq, H, num_blocks, max_blocks_per_seq, device=0):
        import torch

        self.torch = torch
        self.dev = torch.device("cuda", device)
        self.shape = (B, Sq, H, num_blocks, max_blocks_per_seq)
        mk = lambda shp, dt: torch.empty(shp, dtype=dt, device=self.dev)
        self.d_q = mk((B, Sq, H, 576), torch.bfloat16)
        self.d_kv = mk((num_blocks, 64, 576), torch.bfloat16)
        self.d_bt = mk((B, max_blocks_per_seq), torch.int32)
        self.d_sl = mk((B,), torch.int32)
        self.d_out = mk((B, Sq, H, 512), torch.bfloat16)
        self.d_lse = mk((B, Sq, H), torch.float32)
        self.ws = mk((workspace_size(B, Sq, H, max_blocks_per_seq, device),), torch.uint8)
        pin = lambda t: torch.empty(t.shape, dtype=t.dtype, pin_memory=True)
        self.h_q, self.h_kv, self.h_bt, self.h_sl = pin(self.d_q), pin(self.d_kv), pin(self.d_bt), pin(self.d_sl)
        self.h_out, self.h_lse = pin(self.d_out), pin(self.d_lse)

    def set_inputs(self, q_bits, kv_bits, block_table, seqlens):
        """Fill the pinned host buffers from numpy arrays (bf16 given as uint16 bit patterns)."""
        t = self.torch
        self.h_q.view(t.int16).copy_(t.from_numpy(np.ascontiguousarray(q_bits).view(np.int16)))
        self.h_kv.view(t.int16).copy_(t.from_numpy(np.ascontiguousarray(kv_bits).view(np.int16)))
        self.h_bt.copy_(t.from_numpy(np.ascontiguousarray(block_table, dtype=np.int32)))
        self.h_sl.copy_(t.from_numpy(np.ascontiguousarray(seqlens, dtype=np.int32)))

    @property
    def h2d_bytes(self):
        return sum(x.numel() * x.element_size() for x in (self.h_q, self.h_kv, self.h_bt, self.h_sl))

    @property
    def d2h_bytes(self):
        return sum(x.numel() * x.element_size() for x in (self.h_out, self.h_lse))

    def run(self, scale, flags=None, sync=True):
        self.d_q.copy_(self.h_q, non_blocking=True)
        self.d_kv.copy_(self.h_kv, non_blocking=True)
        self.d_bt.copy_(self.h_bt, non_blocking=True)
        self.d_sl.copy_(self.h_sl, non_blocking=True)
        mla_decode(self.d_q, self.d_kv, self.d_bt, self.d_sl, scale, self.d_out, self.d_lse, self.ws, flags)
        self.h_out.copy_(self.d_out, non_blocking=True)
        self.h_lse.copy_(self.d_lse, non_blocking=True)
        if sync:
            self.torch.cuda.current_stream(self.dev).synchronize()
        return self.h_out, self.h_lse
