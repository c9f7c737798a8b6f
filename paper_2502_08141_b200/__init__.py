"""Thin Python binding of the LowRA B200 hot-path library (``liblowra.so``).

Argument marshalling only: every step of the path (encode, decode, fused dequant + LoRA products)
runs in the CUDA kernels behind the C ABI declared in ``include/lowra.h``.  PyTorch is used for
device memory and streams, nothing else.  There is no CPU fallback: if the shared library has
not been built, or the device is not a B200, the calls raise.

Function names are those of the C ABI.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblowra.so")

LOWRA_OK = 0
(LOWRA_ERR_NULL, LOWRA_ERR_SHAPE, LOWRA_ERR_ALIGN, LOWRA_ERR_PREC, LOWRA_ERR_WORKSPACE,
 LOWRA_ERR_CUDA, LOWRA_ERR_TIMEOUT, LOWRA_ERR_ARCH, LOWRA_ERR_LIMIT) = range(1, 10)
LOWRA_STATIC_SCRATCH_BYTES = 8 << 20

EXPORTS = (
    "lowra_status_string", "lowra_plan", "lowra_encode", "lowra_decode", "lowra_workspace_bytes",
    "lowra_lora_forward", "lowra_lora_backward_input", "lowra_device_status", "lowra_dense_nt",
    "lowra_lora_forward_static", "lowra_learn_codebooks", "lowra_adapter_workspace_bytes",
    "lowra_lora_backward_adapters", "lowra_quant_error", "lowra_natural_offsets", "lowra_reorder_rows",
    "lowra_channel_errors", "lowra_deal_bytes", "lowra_deal_build", "lowra_workspace_init",
    "lowra_learn_codebooks_all", "lowra_lora_forward_adapters", "lowra_batch_workspace_bytes",
    "lowra_lora_forward_batch", "lowra_lora_backward_input_batch", "lowra_lora_backward_adapters_reuse",
    "lowra_workspace_projection", "lowra_set_wait_limit", "lowra_diag_wait_expiry", "lowra_diag_drop_t_flags",
    "lowra_encode_group", "lowra_decode_group",
)


class LowraError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


class _CLayout(ctypes.Structure):
    _fields_ = [
        ("N", ctypes.c_int32), ("K", ctypes.c_int32), ("block", ctypes.c_int32),
        ("counts", ctypes.c_int32 * 3),
        ("seg_off", ctypes.c_uint64 * 3),
        ("packed_bytes", ctypes.c_uint64),
        ("precs_dev", ctypes.c_void_p), ("perm_dev", ctypes.c_void_p), ("inv_perm_dev", ctypes.c_void_p),
        ("deal_dev", ctypes.c_void_p), ("natural_offsets_dev", ctypes.c_void_p),
    ]


class _CGroupMember(ctypes.Structure):
    _fields_ = [("layout", ctypes.POINTER(_CLayout)), ("W_dev", ctypes.c_void_p), ("tables_dev", ctypes.c_void_p),
                ("packed_dev", ctypes.c_void_p), ("absmax_dev", ctypes.c_void_p), ("W_bf16_dev", ctypes.c_void_p)]


class _CMember(ctypes.Structure):
    _fields_ = [("layout", ctypes.POINTER(_CLayout)), ("packed_dev", ctypes.c_void_p), ("absmax_dev", ctypes.c_void_p),
                ("maps_dev", ctypes.c_void_p), ("act_dev", ctypes.c_void_p), ("A_dev", ctypes.c_void_p),
                ("B_dev", ctypes.c_void_p), ("out_dev", ctypes.c_void_p)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2502_08141_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, u64p = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_uint64)
        lp = ctypes.POINTER(_CLayout)
        L.lowra_status_string.argtypes = [ctypes.c_int]
        L.lowra_status_string.restype = ctypes.c_char_p
        L.lowra_plan.argtypes = [i32, i32, vp, vp, vp, vp, vp, u64p]
        L.lowra_plan.restype = ctypes.c_int
        L.lowra_encode.argtypes = [lp, vp, vp, vp, vp, vp]
        L.lowra_encode.restype = ctypes.c_int
        L.lowra_decode.argtypes = [lp, vp, vp, vp, vp, vp]
        L.lowra_decode.restype = ctypes.c_int
        for fn in (L.lowra_encode_group, L.lowra_decode_group):
            fn.argtypes = [ctypes.POINTER(_CGroupMember), i32, vp]
            fn.restype = ctypes.c_int
        L.lowra_workspace_bytes.argtypes = [lp, i32, i32]
        L.lowra_workspace_bytes.restype = ctypes.c_size_t
        L.lowra_deal_bytes.argtypes = [lp]
        L.lowra_deal_bytes.restype = ctypes.c_size_t
        L.lowra_deal_build.argtypes = [lp, vp, ctypes.c_size_t, vp]
        L.lowra_deal_build.restype = ctypes.c_int
        L.lowra_workspace_init.argtypes = [vp, ctypes.c_size_t, vp]
        L.lowra_workspace_init.restype = ctypes.c_int
        gemm_args = [lp, vp, vp, vp, vp, i32, vp, vp, i32, ctypes.c_float, vp, vp, ctypes.c_size_t, vp]
        L.lowra_lora_forward.argtypes = gemm_args
        L.lowra_lora_forward.restype = ctypes.c_int
        L.lowra_lora_backward_input.argtypes = gemm_args
        L.lowra_lora_backward_input.restype = ctypes.c_int
        L.lowra_lora_forward_adapters.argtypes = [lp, vp, vp, vp, i32, vp, i32, vp, vp, vp, i32, ctypes.c_float, vp, vp,
                                                  ctypes.c_size_t, vp]
        L.lowra_lora_forward_adapters.restype = ctypes.c_int
        L.lowra_batch_workspace_bytes.argtypes = [lp, i32, i32, i32]
        L.lowra_batch_workspace_bytes.restype = ctypes.c_size_t
        batch_args = [ctypes.POINTER(_CMember), i32, i32, i32, ctypes.c_float, vp, ctypes.c_size_t, vp]
        L.lowra_lora_forward_batch.argtypes = batch_args
        L.lowra_lora_forward_batch.restype = ctypes.c_int
        L.lowra_lora_backward_input_batch.argtypes = batch_args
        L.lowra_lora_backward_input_batch.restype = ctypes.c_int
        L.lowra_lora_forward_static.argtypes = [lp, vp, vp, vp, vp, i32, vp, vp, i32, ctypes.c_float, vp, vp, vp]
        L.lowra_lora_forward_static.restype = ctypes.c_int
        L.lowra_learn_codebooks.argtypes = [lp, vp, vp, vp, i32, vp, vp, vp]
        L.lowra_learn_codebooks.restype = ctypes.c_int
        L.lowra_learn_codebooks_all.argtypes = [i32, i32, vp, vp, vp, i32, vp, vp, vp]
        L.lowra_learn_codebooks_all.restype = ctypes.c_int
        L.lowra_natural_offsets.argtypes = [i32, i32, vp, vp]
        L.lowra_natural_offsets.restype = ctypes.c_int
        L.lowra_reorder_rows.argtypes = [lp, i32, vp, vp, vp, vp, vp, vp]
        L.lowra_reorder_rows.restype = ctypes.c_int
        L.lowra_channel_errors.argtypes = [i32, i32, vp, vp, vp, vp, vp]
        L.lowra_channel_errors.restype = ctypes.c_int
        L.lowra_quant_error.argtypes = [lp, vp, vp, vp, vp, vp, vp]
        L.lowra_quant_error.restype = ctypes.c_int
        L.lowra_adapter_workspace_bytes.argtypes = [i32, i32]
        L.lowra_adapter_workspace_bytes.restype = ctypes.c_size_t
        L.lowra_lora_backward_adapters.argtypes = [vp, vp, i32, i32, i32, vp, vp, i32, ctypes.c_float, vp, vp, vp,
                                                   ctypes.c_size_t, vp]
        L.lowra_lora_backward_adapters.restype = ctypes.c_int
        L.lowra_lora_backward_adapters_reuse.argtypes = [vp, vp, i32, i32, i32, vp, vp, i32, vp, vp, vp, ctypes.c_size_t, vp]
        L.lowra_lora_backward_adapters_reuse.restype = ctypes.c_int
        L.lowra_workspace_projection.argtypes = [vp, i32, i32, i32]
        L.lowra_workspace_projection.restype = ctypes.c_void_p
        L.lowra_device_status.argtypes = [vp, vp]
        L.lowra_device_status.restype = ctypes.c_int
        L.lowra_dense_nt.argtypes = [vp, vp, i32, i32, i32, vp, vp, ctypes.c_size_t, vp]
        L.lowra_dense_nt.restype = ctypes.c_int
        L.lowra_set_wait_limit.argtypes = [ctypes.c_uint64]
        L.lowra_set_wait_limit.restype = ctypes.c_int
        L.lowra_diag_wait_expiry.argtypes = [vp, ctypes.c_size_t, ctypes.c_uint64, vp]
        L.lowra_diag_wait_expiry.restype = ctypes.c_int
        L.lowra_diag_drop_t_flags.argtypes = [i32]
        L.lowra_diag_drop_t_flags.restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().lowra_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != LOWRA_OK:
        raise LowraError(code, where)


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _ptr(t: Optional[torch.Tensor]) -> ctypes.c_void_p:
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t


# ---------------------------------------------------------------------------------------------
def lowra_plan(precs_host: np.ndarray, K: int) -> dict:
    """Host-side storage planner. -> dict(perm, inv_perm, counts, seg_off, packed_bytes)."""
    precs = np.ascontiguousarray(precs_host, dtype=np.uint8)
    N = int(precs.shape[0])
    perm = np.empty(max(N, 1), dtype=np.int32)
    inv = np.empty(max(N, 1), dtype=np.int32)
    counts = (ctypes.c_int32 * 3)()
    seg = (ctypes.c_uint64 * 3)()
    total = ctypes.c_uint64(0)
    code = lib().lowra_plan(N, int(K), precs.ctypes.data, perm.ctypes.data, inv.ctypes.data,
                            ctypes.addressof(counts), ctypes.addressof(seg), ctypes.byref(total))
    _check(code, "lowra_plan")
    return dict(perm=perm[:N], inv_perm=inv[:N], counts=[int(c) for c in counts],
                seg_off=[int(s) for s in seg], packed_bytes=int(total.value))


class Layout:
    """A ``lowra_layout`` plus the device arrays it points to (kept alive here)."""

    def __init__(self, precs_host: np.ndarray, K: int, device="cuda", natural: bool = False):
        """natural=True: packed codes and absmax rows are kept in the paper's own order (rows in original order at
        offsets that follow from their precisions); every call on this layout then reads / writes that buffer."""
        self.precs_host = np.ascontiguousarray(precs_host, dtype=np.uint8)
        self.N, self.K = int(self.precs_host.shape[0]), int(K)
        self.plan = lowra_plan(self.precs_host, K)
        self.device = torch.device(device)
        self.precs = torch.from_numpy(self.precs_host).to(self.device)
        self.perm = torch.from_numpy(self.plan["perm"]).to(self.device)
        self.inv_perm = torch.from_numpy(self.plan["inv_perm"]).to(self.device)
        self.packed_bytes = self.plan["packed_bytes"]
        c = _CLayout()
        c.N, c.K, c.block = self.N, self.K, 64
        for i in range(3):
            c.counts[i] = self.plan["counts"][i]
            c.seg_off[i] = self.plan["seg_off"][i]
        c.packed_bytes = self.packed_bytes
        c.precs_dev = self.precs.data_ptr()
        c.perm_dev = self.perm.data_ptr()
        c.inv_perm_dev = self.inv_perm.data_ptr()
        c.deal_dev = None
        c.natural_offsets_dev = None
        self.c = c
        self.deal = None
        self.natural_offsets = None
        if natural:
            off = lowra_natural_offsets(self.precs_host, K)
            self.natural_offsets = torch.from_numpy(off.view(np.int64)).to(self.device)
            c.natural_offsets_dev = self.natural_offsets.data_ptr()

    def build_deal(self, stream=None) -> "Layout":
        """Deal the rows to the dequantising warps once for this weight (lowra_deal_build): the fused calls on this
        layout then launch no prologue.  Their workspace must have been through lowra_workspace_init."""
        n = int(lib().lowra_deal_bytes(self.ref))
        if n == 0:
            raise LowraError(LOWRA_ERR_SHAPE, "lowra_deal_bytes")
        deal = torch.empty(n, dtype=torch.uint8, device=self.device)
        _check(lib().lowra_deal_build(self.ref, _ptr(deal), n, _stream(stream)), "lowra_deal_build")
        self.deal = deal
        self.c.deal_dev = deal.data_ptr()
        return self

    def drop_deal(self) -> "Layout":
        self.deal = None
        self.c.deal_dev = None
        return self

    @property
    def ref(self):
        return ctypes.byref(self.c)


def lowra_encode(layout: Layout, W: torch.Tensor, thresholds: torch.Tensor,
                 packed: Optional[torch.Tensor] = None, absmax: Optional[torch.Tensor] = None,
                 stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """W fp32 [N,K], thresholds fp32 [N,16] -> packed uint8 [packed_bytes], absmax fp32 [N,K/64]."""
    _dev(W, torch.float32, "W")
    _dev(thresholds, torch.float32, "thresholds")
    if tuple(W.shape) != (layout.N, layout.K) or tuple(thresholds.shape) != (layout.N, 16):
        raise ValueError("shape mismatch")
    if packed is None:
        packed = torch.empty(max(layout.packed_bytes, 16), dtype=torch.uint8, device=W.device)
    if absmax is None:
        absmax = torch.empty((layout.N, layout.K // 64), dtype=torch.float32, device=W.device)
    _dev(packed, torch.uint8, "packed")
    _dev(absmax, torch.float32, "absmax")
    code = lib().lowra_encode(layout.ref, _ptr(W), _ptr(thresholds), _ptr(packed), _ptr(absmax), _stream(stream))
    _check(code, "lowra_encode")
    return packed, absmax


def lowra_decode(layout: Layout, packed: torch.Tensor, absmax: torch.Tensor, maps: torch.Tensor,
                 out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """-> bf16 [N, K], original row order."""
    _dev(packed, torch.uint8, "packed")
    _dev(absmax, torch.float32, "absmax")
    _dev(maps, torch.float32, "maps")
    if out is None:
        out = torch.empty((layout.N, layout.K), dtype=torch.bfloat16, device=packed.device)
    _dev(out, torch.bfloat16, "out")
    code = lib().lowra_decode(layout.ref, _ptr(packed), _ptr(absmax), _ptr(maps), _ptr(out), _stream(stream))
    _check(code, "lowra_decode")
    return out


LOWRA_MAX_GROUP = 8


def lowra_encode_group(members, stream=None):
    """Several matrices in one launch.  `members`: up to LOWRA_MAX_GROUP dicts with layout, W (fp32 [N, K]), thresholds
    (fp32 [N, 16]) and, optionally, packed / absmax to write into.  Returns the list of (packed, absmax) pairs; every
    pair is bit for bit what lowra_encode gives."""
    n = len(members)
    arr = (_CGroupMember * max(n, 1))()
    outs = []
    for i, m in enumerate(members):
        layout, W, thr = m["layout"], m["W"], m["thresholds"]
        _dev(W, torch.float32, "W")
        _dev(thr, torch.float32, "thresholds")
        if tuple(W.shape) != (layout.N, layout.K) or tuple(thr.shape) != (layout.N, 16):
            raise ValueError("shape mismatch")
        packed = m.get("packed")
        absmax = m.get("absmax")
        if packed is None:
            packed = torch.empty(max(layout.packed_bytes, 16), dtype=torch.uint8, device=W.device)
        if absmax is None:
            absmax = torch.empty((layout.N, layout.K // 64), dtype=torch.float32, device=W.device)
        _dev(packed, torch.uint8, "packed")
        _dev(absmax, torch.float32, "absmax")
        arr[i].layout = ctypes.pointer(layout.c)
        arr[i].W_dev, arr[i].tables_dev = W.data_ptr(), thr.data_ptr()
        arr[i].packed_dev, arr[i].absmax_dev, arr[i].W_bf16_dev = packed.data_ptr(), absmax.data_ptr(), None
        outs.append((packed, absmax))
    _check(lib().lowra_encode_group(arr, n, _stream(stream)), "lowra_encode_group")
    return outs


def lowra_decode_group(members, stream=None):
    """Several matrices in one launch.  `members`: up to LOWRA_MAX_GROUP dicts with layout, packed, absmax, maps and,
    optionally, out (bf16 [N, K]).  Returns the list of outputs; every one is bit for bit what lowra_decode gives."""
    n = len(members)
    arr = (_CGroupMember * max(n, 1))()
    outs = []
    for i, m in enumerate(members):
        layout, packed, absmax, maps = m["layout"], m["packed"], m["absmax"], m["maps"]
        _dev(packed, torch.uint8, "packed")
        _dev(absmax, torch.float32, "absmax")
        _dev(maps, torch.float32, "maps")
        out = m.get("out")
        if out is None:
            out = torch.empty((layout.N, layout.K), dtype=torch.bfloat16, device=packed.device)
        _dev(out, torch.bfloat16, "out")
        arr[i].layout = ctypes.pointer(layout.c)
        arr[i].W_dev, arr[i].tables_dev = None, maps.data_ptr()
        arr[i].packed_dev, arr[i].absmax_dev, arr[i].W_bf16_dev = packed.data_ptr(), absmax.data_ptr(), out.data_ptr()
        outs.append(out)
    _check(lib().lowra_decode_group(arr, n, _stream(stream)), "lowra_decode_group")
    return outs


def lowra_learn_codebooks(layout: Layout, W: torch.Tensor, init_levels, init_thresholds, iterations: int,
                          maps: Optional[torch.Tensor] = None, thresholds: Optional[torch.Tensor] = None,
                          stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Weighted Lloyd-Max per row at the row's precision -> (maps fp32 [N,16], thresholds fp32 [N,16]).

    init_levels / init_thresholds: host arrays [3, 16] float64 (rows: 1-, 2-, 4-bit starting tables)."""
    _dev(W, torch.float32, "W")
    y0 = np.ascontiguousarray(init_levels, dtype=np.float64)
    t0 = np.ascontiguousarray(init_thresholds, dtype=np.float64)
    if y0.shape != (3, 16) or t0.shape != (3, 16):
        raise ValueError("init_levels and init_thresholds must be [3, 16]")
    if maps is None:
        maps = torch.empty((layout.N, 16), dtype=torch.float32, device=W.device)
    if thresholds is None:
        thresholds = torch.empty((layout.N, 16), dtype=torch.float32, device=W.device)
    _dev(maps, torch.float32, "maps")
    _dev(thresholds, torch.float32, "thresholds")
    code = lib().lowra_learn_codebooks(layout.ref, _ptr(W), y0.ctypes.data_as(ctypes.c_void_p),
                                       t0.ctypes.data_as(ctypes.c_void_p), int(iterations), _ptr(maps),
                                       _ptr(thresholds), _stream(stream))
    _check(code, "lowra_learn_codebooks")
    return maps, thresholds


def lowra_learn_codebooks_all(W: torch.Tensor, init_levels, init_thresholds, iterations: int,
                              maps3: Optional[torch.Tensor] = None, thresholds3: Optional[torch.Tensor] = None,
                              stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Every row of W learnt at 1, 2 and 4 bits in one pass -> (maps3, thresholds3) fp32 [3, N, 16], the input
    format of lowra_channel_errors."""
    _dev(W, torch.float32, "W")
    N, K = int(W.shape[0]), int(W.shape[1])
    y0 = np.ascontiguousarray(init_levels, dtype=np.float64)
    t0 = np.ascontiguousarray(init_thresholds, dtype=np.float64)
    if y0.shape != (3, 16) or t0.shape != (3, 16):
        raise ValueError("init_levels and init_thresholds must be [3, 16]")
    if maps3 is None:
        maps3 = torch.empty((3, N, 16), dtype=torch.float32, device=W.device)
    if thresholds3 is None:
        thresholds3 = torch.empty((3, N, 16), dtype=torch.float32, device=W.device)
    _dev(maps3, torch.float32, "maps3")
    _dev(thresholds3, torch.float32, "thresholds3")
    if tuple(maps3.shape) != (3, N, 16) or tuple(thresholds3.shape) != (3, N, 16):
        raise ValueError("maps3 and thresholds3 must be [3, N, 16]")
    code = lib().lowra_learn_codebooks_all(N, K, _ptr(W), y0.ctypes.data_as(ctypes.c_void_p),
                                           t0.ctypes.data_as(ctypes.c_void_p), int(iterations), _ptr(maps3),
                                           _ptr(thresholds3), _stream(stream))
    _check(code, "lowra_learn_codebooks_all")
    return maps3, thresholds3


def lowra_workspace_bytes(layout: Layout, M: int, r: int) -> int:
    return int(lib().lowra_workspace_bytes(layout.ref, int(M), int(r)))


def _workspace(layout: Layout, M: int, r: int, device) -> torch.Tensor:
    n = lowra_workspace_bytes(layout, M, r)
    if n == 0:
        raise LowraError(LOWRA_ERR_SHAPE, "lowra_workspace_bytes")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    if layout.deal is not None:   # no prologue launch will clear it
        lowra_workspace_init(ws)
    return ws


def lowra_workspace_init(workspace: torch.Tensor, stream=None) -> torch.Tensor:
    """Zero-fill a workspace: needed once before calls on a layout that carries a deal (Layout.build_deal)."""
    _dev(workspace, torch.uint8, "workspace")
    _check(lib().lowra_workspace_init(_ptr(workspace), workspace.numel(), _stream(stream)), "lowra_workspace_init")
    return workspace


def lowra_lora_forward(layout: Layout, packed, absmax, maps, X, A, B, s: float,
                       Y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                       stream=None) -> torch.Tensor:
    """Y = X . deq(Wq)^T + s (X . A) . B ; X bf16 [M,K], A bf16 [K,r], B bf16 [r,N] -> Y bf16 [M,N]."""
    for t, n in ((X, "X"), (A, "A"), (B, "B")):
        _dev(t, torch.bfloat16, n)
    M, r = int(X.shape[0]), int(A.shape[1])
    if tuple(X.shape) != (M, layout.K) or tuple(A.shape) != (layout.K, r) or tuple(B.shape) != (r, layout.N):
        raise ValueError("shape mismatch")
    if Y is None:
        Y = torch.empty((M, layout.N), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = _workspace(layout, M, r, X.device)
    code = lib().lowra_lora_forward(layout.ref, _ptr(packed), _ptr(absmax), _ptr(maps), _ptr(X), M, _ptr(A),
                                    _ptr(B), r, ctypes.c_float(s), _ptr(Y), _ptr(workspace),
                                    workspace.numel(), _stream(stream))
    _check(code, "lowra_lora_forward")
    return Y


def lowra_batch_workspace_bytes(layout: Layout, count: int, M: int, r: int) -> int:
    return int(lib().lowra_batch_workspace_bytes(layout.ref, int(count), int(M), int(r)))


def _batch(fn_name: str, members, s: float, workspace: torch.Tensor, backward: bool, stream=None):
    """members: sequence of dicts with layout, packed, absmax, maps, act, A, B, out (device tensors)."""
    n = len(members)
    arr = (_CMember * n)()
    M = int(members[0]["act"].shape[0])
    r = int(members[0]["A"].shape[1])
    for i, m in enumerate(members):
        lay = m["layout"]
        for key in ("act", "A", "B", "out"):
            _dev(m[key], torch.bfloat16, key)
        act_cols, out_cols = (lay.N, lay.K) if backward else (lay.K, lay.N)
        if (tuple(m["act"].shape) != (M, act_cols) or tuple(m["out"].shape) != (M, out_cols) or
                tuple(m["A"].shape) != (lay.K, r) or tuple(m["B"].shape) != (r, lay.N)):
            raise ValueError("shape mismatch in member %d" % i)
        arr[i].layout = ctypes.pointer(lay.c)
        arr[i].packed_dev, arr[i].absmax_dev, arr[i].maps_dev = m["packed"].data_ptr(), m["absmax"].data_ptr(), m["maps"].data_ptr()
        arr[i].act_dev, arr[i].A_dev, arr[i].B_dev, arr[i].out_dev = (m["act"].data_ptr(), m["A"].data_ptr(), m["B"].data_ptr(),
                                                                     m["out"].data_ptr())
    code = getattr(lib(), fn_name)(arr, n, M, r, ctypes.c_float(s), _ptr(workspace), workspace.numel(), _stream(stream))
    _check(code, fn_name)
    return [m["out"] for m in members]


def lowra_lora_forward_batch(members, s: float, workspace: torch.Tensor, stream=None):
    """Several weights of one shape in one launch: Y_i = X_i deq(Wq_i)^T + s (X_i A_i) B_i.  `members`: dicts with
    layout (carrying a deal), packed, absmax, maps, act (X_i), A, B, out (Y_i).  Returns the outputs."""
    return _batch("lowra_lora_forward_batch", members, s, workspace, False, stream)


def lowra_lora_backward_input_batch(members, s: float, workspace: torch.Tensor, stream=None):
    """The input gradients of several weights of one shape in one launch; act = dY_i, out = dX_i."""
    return _batch("lowra_lora_backward_input_batch", members, s, workspace, True, stream)


def lowra_lora_forward_adapters(layout: Layout, packed, absmax, maps, X, group_start, A, B, s: float,
                                Y: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                                stream=None) -> torch.Tensor:
    """Several adapters on one quantised base weight: maps fp32 [n, N, 16], A bf16 [n, K, r], B bf16 [n, r, N];
    adapter a owns the token rows group_start[a] .. group_start[a + 1] of X (host sequence of n + 1 ints)."""
    for t, nm in ((X, "X"), (A, "A"), (B, "B")):
        _dev(t, torch.bfloat16, nm)
    _dev(maps, torch.float32, "maps")
    n, M, r = int(maps.shape[0]), int(X.shape[0]), int(A.shape[2])
    if (tuple(maps.shape) != (n, layout.N, 16) or tuple(X.shape) != (M, layout.K) or tuple(A.shape) != (n, layout.K, r)
            or tuple(B.shape) != (n, r, layout.N)):
        raise ValueError("shape mismatch")
    gs = np.ascontiguousarray(group_start, dtype=np.int32)
    if gs.shape != (n + 1,):
        raise ValueError("group_start must have n_adapters + 1 entries")
    if Y is None:
        Y = torch.empty((M, layout.N), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = _workspace(layout, M, r, X.device)
    code = lib().lowra_lora_forward_adapters(layout.ref, _ptr(packed), _ptr(absmax), _ptr(maps), n, _ptr(X), M,
                                             gs.ctypes.data_as(ctypes.c_void_p), _ptr(A), _ptr(B), r, ctypes.c_float(s),
                                             _ptr(Y), _ptr(workspace), workspace.numel(), _stream(stream))
    _check(code, "lowra_lora_forward_adapters")
    return Y


def lowra_lora_forward_static(layout: Layout, packed, absmax, maps, X, A, B, s: float,
                              Y: Optional[torch.Tensor] = None, status_out: Optional[torch.Tensor] = None,
                              stream=None) -> torch.Tensor:
    """lowra_lora_forward for callers that may not allocate device memory (a plug-in inside a host
    application's CUDA context, a loop whose allocations were frozen at start-up): the scratch is a fixed
    array inside the library (LOWRA_STATIC_SCRATCH_BYTES), shared by every call on the device, so calls
    must not overlap on the GPU.  Raises LowraError(LOWRA_ERR_LIMIT) when the problem needs more scratch.
    `status_out`: optional int32/uint32 device tensor of one element that receives the device status word.
    This wrapper allocates Y only if the caller passes none; the library call itself allocates nothing."""
    for t, n in ((X, "X"), (A, "A"), (B, "B")):
        _dev(t, torch.bfloat16, n)
    M, r = int(X.shape[0]), int(A.shape[1])
    if tuple(X.shape) != (M, layout.K) or tuple(A.shape) != (layout.K, r) or tuple(B.shape) != (r, layout.N):
        raise ValueError("shape mismatch")
    if Y is None:
        Y = torch.empty((M, layout.N), dtype=torch.bfloat16, device=X.device)
    code = lib().lowra_lora_forward_static(layout.ref, _ptr(packed), _ptr(absmax), _ptr(maps), _ptr(X), M, _ptr(A),
                                           _ptr(B), r, ctypes.c_float(s), _ptr(Y), _ptr(status_out), _stream(stream))
    _check(code, "lowra_lora_forward_static")
    return Y


def lowra_lora_backward_input(layout: Layout, packed, absmax, maps, dY, A, B, s: float,
                              dX: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                              stream=None) -> torch.Tensor:
    """dX = dY . deq(Wq) + s (dY . B^T) . A^T ; dY bf16 [M,N] -> dX bf16 [M,K]."""
    for t, n in ((dY, "dY"), (A, "A"), (B, "B")):
        _dev(t, torch.bfloat16, n)
    M, r = int(dY.shape[0]), int(A.shape[1])
    if tuple(dY.shape) != (M, layout.N) or tuple(A.shape) != (layout.K, r) or tuple(B.shape) != (r, layout.N):
        raise ValueError("shape mismatch")
    if dX is None:
        dX = torch.empty((M, layout.K), dtype=torch.bfloat16, device=dY.device)
    if workspace is None:
        workspace = _workspace(layout, M, r, dY.device)
    code = lib().lowra_lora_backward_input(layout.ref, _ptr(packed), _ptr(absmax), _ptr(maps), _ptr(dY), M,
                                           _ptr(A), _ptr(B), r, ctypes.c_float(s), _ptr(dX), _ptr(workspace),
                                           workspace.numel(), _stream(stream))
    _check(code, "lowra_lora_backward_input")
    return dX


def lowra_natural_offsets(precs, K: int):
    """Byte offsets [N + 1] (numpy uint64) of the rows in the natural-order buffer."""
    import numpy as np
    precs = np.ascontiguousarray(precs, dtype=np.uint8)
    off = np.zeros(precs.size + 1, dtype=np.uint64)
    code = lib().lowra_natural_offsets(int(precs.size), int(K), ctypes.c_void_p(precs.ctypes.data),
                                       ctypes.c_void_p(off.ctypes.data))
    _check(code, "lowra_natural_offsets")
    return off


def lowra_reorder_rows(layout: Layout, to_natural: bool, offsets: torch.Tensor, packed: torch.Tensor,
                       absmax: torch.Tensor, packed_out: Optional[torch.Tensor] = None,
                       absmax_out: Optional[torch.Tensor] = None, stream=None):
    """Grouped <-> natural row order of the packed codes and the absmax rows.  `offsets`: the natural offsets
    as an int64 / uint64 device tensor [N + 1].  Returns (packed_out, absmax_out)."""
    _dev(packed, torch.uint8, "packed")
    _dev(absmax, torch.float32, "absmax")
    if not offsets.is_cuda or offsets.element_size() != 8 or offsets.numel() != layout.N + 1:
        raise ValueError("offsets must be a 64-bit device tensor of N + 1 entries")
    if packed_out is None:
        packed_out = torch.empty_like(packed)
    if absmax_out is None:
        absmax_out = torch.empty_like(absmax)
    code = lib().lowra_reorder_rows(layout.ref, 1 if to_natural else 0, _ptr(offsets), _ptr(packed), _ptr(absmax),
                                    _ptr(packed_out), _ptr(absmax_out), _stream(stream))
    _check(code, "lowra_reorder_rows")
    return packed_out, absmax_out


def lowra_quant_error(layout: Layout, W: torch.Tensor, maps: torch.Tensor, thresholds: torch.Tensor,
                      sse: Optional[torch.Tensor] = None, residual: Optional[torch.Tensor] = None,
                      want_residual: bool = False, stream=None):
    """Per-channel summed square error (fp64 [N]) of quantising W with these tables, and optionally the
    residual W - W_hat (fp32 [N,K]).  Returns (sse, residual or None)."""
    _dev(W, torch.float32, "W")
    _dev(maps, torch.float32, "maps")
    _dev(thresholds, torch.float32, "thresholds")
    if tuple(W.shape) != (layout.N, layout.K) or tuple(maps.shape) != (layout.N, 16) or tuple(thresholds.shape) != (layout.N, 16):
        raise ValueError("shape mismatch")
    if sse is None:
        sse = torch.empty(layout.N, dtype=torch.float64, device=W.device)
    if residual is None and want_residual:
        residual = torch.empty((layout.N, layout.K), dtype=torch.float32, device=W.device)
    code = lib().lowra_quant_error(layout.ref, _ptr(W), _ptr(maps), _ptr(thresholds), _ptr(sse),
                                   _ptr(residual) if residual is not None else None, _stream(stream))
    _check(code, "lowra_quant_error")
    return sse, residual


def lowra_channel_errors(W: torch.Tensor, maps3: torch.Tensor, thresholds3: torch.Tensor,
                         sse3: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Summed square error of every row of W under 1, 2 and 4 bits (fp64 [N,3]); tables fp32 [3,N,16]."""
    _dev(W, torch.float32, "W")
    _dev(maps3, torch.float32, "maps3")
    _dev(thresholds3, torch.float32, "thresholds3")
    N, K = int(W.shape[0]), int(W.shape[1])
    if tuple(maps3.shape) != (3, N, 16) or tuple(thresholds3.shape) != (3, N, 16):
        raise ValueError("shape mismatch")
    if sse3 is None:
        sse3 = torch.empty((N, 3), dtype=torch.float64, device=W.device)
    code = lib().lowra_channel_errors(N, K, _ptr(W), _ptr(maps3), _ptr(thresholds3), _ptr(sse3), _stream(stream))
    _check(code, "lowra_channel_errors")
    return sse3


def lowra_adapter_workspace_bytes(M: int, r: int) -> int:
    return int(lib().lowra_adapter_workspace_bytes(int(M), int(r)))


def lowra_lora_backward_adapters(X, dY, A, B, s: float, dA: Optional[torch.Tensor] = None,
                                 dB: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                                 stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """dA = s X^T (dY B^T) [K,r] and dB = s (X A)^T dY [r,N]; all operands bf16 on the device."""
    for t, n in ((X, "X"), (dY, "dY"), (A, "A"), (B, "B")):
        _dev(t, torch.bfloat16, n)
    M, K = int(X.shape[0]), int(X.shape[1])
    N, r = int(dY.shape[1]), int(A.shape[1])
    if tuple(dY.shape) != (M, N) or tuple(A.shape) != (K, r) or tuple(B.shape) != (r, N):
        raise ValueError("shape mismatch")
    if dA is None:
        dA = torch.empty((K, r), dtype=torch.bfloat16, device=X.device)
    if dB is None:
        dB = torch.empty((r, N), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        nbytes = lowra_adapter_workspace_bytes(M, r)
        if nbytes == 0:
            raise LowraError(LOWRA_ERR_SHAPE, "lowra_adapter_workspace_bytes")
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=X.device)
    code = lib().lowra_lora_backward_adapters(_ptr(X), _ptr(dY), M, K, N, _ptr(A), _ptr(B), r, ctypes.c_float(s),
                                              _ptr(dA), _ptr(dB), _ptr(workspace), workspace.numel(),
                                              _stream(stream))
    _check(code, "lowra_lora_backward_adapters")
    return dA, dB


def lowra_workspace_projection(workspace: torch.Tensor, M: int, r: int, member: int = 0) -> torch.Tensor:
    """The down-projection (s X A after a forward call, s dY B^T after a backward-input call) that the last fused call
    left in `workspace`: a bf16 [M, rp] view into the workspace, rp = r rounded up to 64."""
    _dev(workspace, torch.uint8, "workspace")
    p = lib().lowra_workspace_projection(_ptr(workspace), int(member), int(M), int(r))
    if not p:
        raise LowraError(LOWRA_ERR_SHAPE, "lowra_workspace_projection")
    rp = (int(r) + 63) // 64 * 64
    off = int(p) - workspace.data_ptr()
    return workspace[off:off + int(M) * rp * 2].view(torch.bfloat16).view(int(M), rp)


def lowra_lora_backward_adapters_reuse(X, dY, T, U, r: int, dA: Optional[torch.Tensor] = None,
                                       dB: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                                       stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """dA = X^T U [K, r] and dB = T^T dY [r, N] from the down-projections T, U (bf16 [M, rp]) that the forward and the
    backward-input call left in their workspaces (lowra_workspace_projection): X and dY are read once."""
    for t, n in ((X, "X"), (dY, "dY"), (T, "T"), (U, "U")):
        _dev(t, torch.bfloat16, n)
    M, K, N = int(X.shape[0]), int(X.shape[1]), int(dY.shape[1])
    rp = (int(r) + 63) // 64 * 64
    if tuple(dY.shape) != (M, N) or tuple(T.shape) != (M, rp) or tuple(U.shape) != (M, rp):
        raise ValueError("shape mismatch")
    if dA is None:
        dA = torch.empty((K, r), dtype=torch.bfloat16, device=X.device)
    if dB is None:
        dB = torch.empty((r, N), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = torch.empty(256, dtype=torch.uint8, device=X.device)
    code = lib().lowra_lora_backward_adapters_reuse(_ptr(X), _ptr(dY), M, K, N, _ptr(T), _ptr(U), int(r), _ptr(dA), _ptr(dB),
                                                    _ptr(workspace), workspace.numel(), _stream(stream))
    _check(code, "lowra_lora_backward_adapters_reuse")
    return dA, dB


def lowra_device_status(workspace: torch.Tensor, stream=None) -> int:
    """Synchronises the stream and returns the status word of the last fused call."""
    return int(lib().lowra_device_status(_ptr(workspace), _stream(stream)))


def lowra_set_wait_limit(nanoseconds: int) -> None:
    """Limit of every device-side wait of the tensor-core kernels (0: the default of one second)."""
    _check(lib().lowra_set_wait_limit(int(nanoseconds)), "lowra_set_wait_limit")


def lowra_diag_wait_expiry(workspace: torch.Tensor, limit_ns: int, stream=None) -> None:
    """Self test: a one-warp kernel whose two waits run out after `limit_ns` each; status word -> LOWRA_ERR_TIMEOUT."""
    _dev(workspace, torch.uint8, "workspace")
    _check(lib().lowra_diag_wait_expiry(_ptr(workspace), workspace.numel(), int(limit_ns), _stream(stream)),
           "lowra_diag_wait_expiry")


def lowra_diag_drop_t_flags(calls: int) -> None:
    """Self test: the next `calls` fused calls do not publish their "down-projection ready" flags and time out."""
    _check(lib().lowra_diag_drop_t_flags(int(calls)), "lowra_diag_drop_t_flags")


def lowra_dense_nt(P: torch.Tensor, Q: torch.Tensor, C: Optional[torch.Tensor] = None,
                   workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Diagnostic: C = P . Q^T through the same tensor-core pipeline (both operands plain bf16)."""
    _dev(P, torch.bfloat16, "P")
    _dev(Q, torch.bfloat16, "Q")
    M, K = P.shape
    N = Q.shape[0]
    if C is None:
        C = torch.empty((M, N), dtype=torch.bfloat16, device=P.device)
    if workspace is None:
        workspace = torch.empty(256, dtype=torch.uint8, device=P.device)
    code = lib().lowra_dense_nt(_ptr(P), _ptr(Q), int(M), int(N), int(K), _ptr(C), _ptr(workspace),
                                workspace.numel(), _stream(stream))
    _check(code, "lowra_dense_nt")
    return C
