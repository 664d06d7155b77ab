"""Thin ctypes binding of libbsa.so: argument marshalling only.

Every step of the request path (mask state, plan selection, launch preparation,
attention, Split-K merge) runs inside the C-ABI library; torch is used here only
to own device memory and streams.  Loading fails loudly if the library has not
been built -- there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbsa.so")

BSA_OK = 0
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "NO_ELIGIBLE_PLAN", 4: "OOM", 5: "CUDA",
                6: "DEVICE_TIMEOUT", 7: "LUT"}
MAP_NAMES = {0: "direct", 1: "coarsened", 2: "refined"}


class PlanDesc(ctypes.Structure):
    _fields_ = [("plan_id", ctypes.c_int32), ("T_Q", ctypes.c_int32), ("T_KV", ctypes.c_int32),
                ("stages", ctypes.c_int32), ("split_tau", ctypes.c_int32), ("split_pmax", ctypes.c_int32),
                ("order", ctypes.c_int32), ("kernel", ctypes.c_int32), ("name", ctypes.c_char * 48)]


DTYPES = {"bf16": 0, "fp16": 1}  # BSA_DTYPE_*
LAYOUTS = {"hnd": 0, "nhd": 1}   # BSA_LAYOUT_*: [heads, N, d] or [N, heads, d]


class Options(ctypes.Structure):
    _fields_ = [("force_plan_id", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("max_workspace_bytes", ctypes.c_int64), ("N_kv", ctypes.c_int64),
                ("layout", ctypes.c_int32), ("batch", ctypes.c_int32)]


class PlanInfo(ctypes.Structure):
    _fields_ = [("plan", PlanDesc), ("map_q", ctypes.c_int32), ("map_kv", ctypes.c_int32),
                ("heads", ctypes.c_int32), ("d", ctypes.c_int32), ("B_Q", ctypes.c_int32), ("B_KV", ctypes.c_int32),
                ("N", ctypes.c_int64),
                ("nQb", ctypes.c_int32), ("nKb", ctypes.c_int32), ("nQt", ctypes.c_int32), ("nKt", ctypes.c_int32),
                ("member_bits", ctypes.c_int32), ("lut_hit", ctypes.c_int32), ("regime_bucket", ctypes.c_int32 * 4),
                ("nnz_blocks", ctypes.c_int64), ("blocks_in_runs", ctypes.c_int64),
                ("max_row_nnz", ctypes.c_int32), ("member_words", ctypes.c_int32),
                ("density", ctypes.c_double), ("run_coverage", ctypes.c_double), ("skew", ctypes.c_double),
                ("ntiles", ctypes.c_int64), ("nitems", ctypes.c_int64), ("nsplit_rows", ctypes.c_int64),
                ("workspace_bytes", ctypes.c_int64), ("covered_pairs", ctypes.c_int64),
                ("us_mask_state", ctypes.c_float), ("us_stats_sync", ctypes.c_float), ("us_lookup", ctypes.c_float),
                ("us_launch_prep", ctypes.c_float), ("us_total", ctypes.c_float), ("device_status", ctypes.c_int32),
                ("N_kv", ctypes.c_int64), ("dtype", ctypes.c_int32), ("layout", ctypes.c_int32)]

    def as_dict(self) -> Dict:
        out = {}
        for name, _ in self._fields_:
            v = getattr(self, name)
            if name == "plan":
                v = {f: (getattr(v, f).decode() if f == "name" else getattr(v, f)) for f, _ in PlanDesc._fields_}
            elif name == "regime_bucket":
                v = list(v)
            out[name] = v
        return out


_lib = None


def lib() -> ctypes.CDLL:
    """Load libbsa.so (raises if it was not built: there is no other code path)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_25869_b200.build` "
                           "(nvcc, sm_100a). There is no CPU or PyTorch fallback.")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_double
    L.bsa_plan_create.argtypes = [vp, i32, i32, i64, i32, i32, ctypes.POINTER(vp)]
    L.bsa_plan_create_ex.argtypes = [vp, i32, i32, i64, i32, i32, ctypes.POINTER(Options), vp, ctypes.POINTER(vp)]
    L.bsa_plan_create_packed.argtypes = [vp, i64, i32, i32, i64, i32, i32, ctypes.POINTER(Options), vp, ctypes.POINTER(vp)]
    L.bsa_plan_cache_create.argtypes = [i32, ctypes.POINTER(vp)]
    L.bsa_plan_cache_get.argtypes = [vp, vp, i64, i32, i32, i64, i32, i32, ctypes.POINTER(Options), vp, ctypes.POINTER(vp),
                                     ctypes.POINTER(i32)]
    L.bsa_plan_cache_request.argtypes = [vp, vp, i64, i32, i32, i64, i32, i32, vp, vp, vp, vp, vp, ctypes.POINTER(Options),
                                         vp, ctypes.POINTER(vp), ctypes.POINTER(i32)]
    L.bsa_plan_cache_stats.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64), ctypes.POINTER(i64),
                                       ctypes.POINTER(ctypes.c_int32)]
    L.bsa_plan_cache_destroy.argtypes = [vp]
    L.bsa_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.bsa_request_device.argtypes = [vp, i64, i32, i32, i64, i32, i32, vp, vp, vp, vp, vp, ctypes.POINTER(Options), vp,
                                     ctypes.POINTER(vp)]
    L.bsa_plan_destroy.argtypes = [vp]
    L.bsa_request_host.argtypes = [vp, i32, i32, i64, i32, i32, vp, vp, vp, vp, vp, ctypes.POINTER(Options),
                                   ctypes.POINTER(PlanInfo)]
    L.bsa_mask_stats_noalloc.argtypes = [vp, i32, i32, i32, vp, vp]
    L.bsa_plan_get_info.argtypes = [vp, ctypes.POINTER(PlanInfo)]
    L.bsa_plan_export_csr.argtypes = [vp, vp, vp]
    L.bsa_plan_export_tiles.argtypes = [vp, i32, vp, vp, vp, i64, ctypes.POINTER(i64)]
    L.bsa_plan_export_items.argtypes = [vp, vp, i64, ctypes.POINTER(i64)]
    L.bsa_catalog_size.restype = i32
    L.bsa_catalog_get.argtypes = [i32, ctypes.POINTER(PlanDesc)]
    L.bsa_plan_eligible.argtypes = [i32, i32, i32, i64, i32, i32, i64]
    L.bsa_plan_eligible_ex.argtypes = [i32, i32, i32, i64, i64, i32, i32, i32, i64]
    L.bsa_debug_set_wait_limit.argtypes = [ctypes.c_longlong]
    L.bsa_debug_withhold_arrival.argtypes = [i32]
    L.bsa_debug_merge_only.argtypes = [vp, vp, vp, vp]
    L.bsa_base_plan.argtypes = [i32, i32, i32]
    L.bsa_catalog_hash.restype = ctypes.c_uint64
    L.bsa_lut_load.argtypes = [ctypes.c_char_p]
    L.bsa_lut_clear.restype = None
    L.bsa_lut_select.argtypes = [i32, i32, i64, i32, i32, f64, f64, f64, i64, ctypes.POINTER(i32)]
    L.bsa_lut_buckets.argtypes = [i64, f64, f64, f64, ctypes.POINTER(ctypes.c_int32)]
    L.bsa_lut_buckets.restype = None
    L.bsa_force_plan.argtypes = [i32]
    L.bsa_force_plan.restype = None
    L.bsa_status_string.argtypes = [i32]
    L.bsa_status_string.restype = ctypes.c_char_p
    L.bsa_last_cuda_error.restype = ctypes.c_char_p
    L.bsa_version.restype = ctypes.c_char_p
    L.bsa_kernel_launch_count.restype = i64
    _lib = L
    load_default_table()
    return L


DEFAULT_TABLE = os.path.join(_HERE, "plan_table_b200.lut")


def load_default_table() -> bool:
    """Load the plan table shipped with the package (written by ``lut_build.py`` on a B200).  A table built
    for another catalog is rejected by the library; base plans are used then.  Returns True if loaded."""
    if _lib is None or not os.path.exists(DEFAULT_TABLE):
        return False
    return _lib.bsa_lut_load(DEFAULT_TABLE.encode()) == BSA_OK


class BsaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = lib().bsa_last_cuda_error().decode() if status == 5 else ""
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} "
                         f"({lib().bsa_status_string(status).decode()}) {detail}")


def _check(status: int, where: str):
    if status != BSA_OK:
        raise BsaError(status, where)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    return getattr(stream, "cuda_stream", stream) or None


def _lse_shape(Q, layout: str):
    """[heads, N] for Q stored [heads, N, d], [N, heads, d] or, batched and token-major, [batch, N, heads/batch, d]."""
    if layout == "hnd":
        return (Q.shape[0], Q.shape[1]) if Q.dim() == 3 else (Q.shape[0] * Q.shape[1], Q.shape[2])
    if Q.dim() == 4:
        return (Q.shape[0] * Q.shape[2], Q.shape[1])
    return (Q.shape[1], Q.shape[0])


class Plan:
    """Handle of a prepared plan (``bsa_plan_create`` ... ``bsa_plan_destroy``)."""

    def __init__(self, handle: int, layout: str = "hnd"):
        self._h = ctypes.c_void_p(handle)
        self.layout = layout

    def forward(self, Q, K, V, O=None, LSE=None, stream=None):
        """``bsa_forward``: Q, K, V are bf16 CUDA tensors ``[heads, N, d]``; returns ``(O, LSE)``."""
        import torch
        assert Q.is_cuda and Q.dtype in (torch.bfloat16, torch.float16) and Q.is_contiguous()  # as the plan's dtype
        assert K.is_contiguous() and V.is_contiguous() and K.dtype == V.dtype == Q.dtype
        if O is None:
            O = torch.empty_like(Q)
        if LSE is None:  # [heads, N] whatever the layout of Q
            LSE = torch.empty(_lse_shape(Q, self.layout), dtype=torch.float32, device=Q.device)
        _check(lib().bsa_forward(self._h, Q.data_ptr(), K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(),
                                 _stream_ptr(stream)), "bsa_forward")
        return O, LSE

    def merge_only(self, O, LSE, stream=None):
        """``bsa_debug_merge_only`` (measurement hook): the Split-K reduction kernel alone, over the last forward's partials."""
        _check(lib().bsa_debug_merge_only(self._h, O.data_ptr(), LSE.data_ptr(), _stream_ptr(stream)), "bsa_debug_merge_only")

    def info(self) -> Dict:
        inf = PlanInfo()
        _check(lib().bsa_plan_get_info(self._h, ctypes.byref(inf)), "bsa_plan_get_info")
        return inf.as_dict()

    def export_csr(self) -> Tuple[np.ndarray, np.ndarray]:
        inf = self.info()
        rp = np.zeros(inf["heads"] * inf["nQb"] + 1, dtype=np.int32)
        ci = np.zeros(max(1, inf["nnz_blocks"]), dtype=np.int32)
        _check(lib().bsa_plan_export_csr(self._h, rp.ctypes.data, ci.ctypes.data), "bsa_plan_export_csr")
        return rp, ci[: inf["nnz_blocks"]]

    def export_tiles(self, head: int):
        """Tiles of one head: ``(tile_row_ptr [nQt+1], tile_col [n], tile_member [n, W] uint64)`` with
        ``W = T_Q / 128`` membership words per tile (one per 128-row slot)."""
        n = ctypes.c_int64(0)
        _check(lib().bsa_plan_export_tiles(self._h, head, None, None, None, 0, ctypes.byref(n)), "export_tiles(size)")
        inf = self.info()
        nQt, W = inf["nQt"], inf["member_words"]
        rp = np.zeros(nQt + 1, dtype=np.int32)
        tc = np.zeros(max(1, n.value), dtype=np.int32)
        tm = np.zeros((max(1, n.value), W), dtype=np.uint64)
        _check(lib().bsa_plan_export_tiles(self._h, head, rp.ctypes.data, tc.ctypes.data, tm.ctypes.data,
                                           max(1, n.value), ctypes.byref(n)), "export_tiles")
        return rp, tc[: n.value], tm[: n.value]

    def export_items(self) -> np.ndarray:
        n = ctypes.c_int64(0)
        _check(lib().bsa_plan_export_items(self._h, None, 0, ctypes.byref(n)), "export_items(size)")
        it = np.zeros((max(1, n.value), 8), dtype=np.int32)
        _check(lib().bsa_plan_export_items(self._h, it.ctypes.data, max(1, n.value), ctypes.byref(n)), "export_items")
        return it[: n.value]

    def destroy(self):
        if self._h:
            _check(lib().bsa_plan_destroy(self._h), "bsa_plan_destroy")
            self._h = None

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.destroy()


def plan_create(mask, B_Q: int, B_KV: int, N: int, heads: int, d: int, plan_id: int = -1,
                max_workspace_bytes: int = 0, stream=None, N_kv: int = 0, dtype: str = "bf16",
                layout: str = "hnd", batch: int = 0) -> Plan:
    """``bsa_plan_create_ex``: ``mask`` is a uint8/bool CUDA tensor ``[heads, nQb, nKb]``; ``N_kv`` > 0 gives K and V
    that many tokens per head (Q, O, LSE keep ``N``); ``dtype`` "fp16" prepares the plan for half tensors; ``batch`` > 1
    with ``layout="nhd"`` makes the tensors ``[batch, N, heads / batch, d]`` (``heads`` counts all problems)."""
    import torch
    assert mask.is_cuda and mask.is_contiguous() and mask.dtype in (torch.uint8, torch.bool)
    h = ctypes.c_void_p()
    opt = Options(plan_id, DTYPES[dtype], max_workspace_bytes, N_kv, LAYOUTS[layout], batch)
    _check(lib().bsa_plan_create_ex(mask.data_ptr(), B_Q, B_KV, N, heads, d, ctypes.byref(opt), _stream_ptr(stream),
                                    ctypes.byref(h)), "bsa_plan_create")
    return Plan(h.value, layout)


def request(mask, B_Q: int, B_KV: int, N: int, heads: int, d: int, Q, K, V, O=None, LSE=None, plan_id: int = -1,
            max_workspace_bytes: int = 0, stream=None, N_kv: int = 0, dtype: str = "bf16", layout: str = "hnd",
            row_stride: int = 0):
    """``bsa_request_device``: plan create + forward in one call (CUDA tensors).  Returns ``(plan, O, LSE)``; the plan
    can run further forwards and is given back with ``plan.destroy()``."""
    import torch
    if O is None:
        O = torch.empty_like(Q)
    if LSE is None:
        LSE = torch.empty(_lse_shape(Q, layout), dtype=torch.float32, device=Q.device)
    h = ctypes.c_void_p()
    opt = Options(plan_id, DTYPES[dtype], max_workspace_bytes, N_kv, LAYOUTS[layout], 0)
    _check(lib().bsa_request_device(mask.data_ptr(), row_stride, B_Q, B_KV, N, heads, d, Q.data_ptr(), K.data_ptr(),
                                    V.data_ptr(), O.data_ptr(), LSE.data_ptr(), ctypes.byref(opt), _stream_ptr(stream),
                                    ctypes.byref(h)), "bsa_request_device")
    return Plan(h.value, layout), O, LSE


def pack_mask(mask):
    """Bit-pack a uint8/bool mask tensor ``[heads, nQb, nKb]`` (CUDA or CPU) into the layout ``plan_create_packed``
    reads: little-endian bits, rows padded to a multiple of 4 bytes.  Returns ``(packed uint8 tensor, row stride)``.
    A convenience for callers and tests (plain torch ops, not part of the timed path)."""
    import torch
    h, nq, nk = mask.shape
    stride = ((nk + 31) // 32) * 4
    m = (mask != 0).to(torch.uint8)
    pad = stride * 8 - nk
    if pad:
        m = torch.nn.functional.pad(m, (0, pad))
    w = torch.tensor([1, 2, 4, 8, 16, 32, 64, 128], dtype=torch.uint8, device=m.device)
    packed = (m.view(h, nq, stride, 8) * w).sum(dim=-1, dtype=torch.int32).to(torch.uint8).contiguous()
    return packed, stride


def plan_create_packed(mask_bits, row_stride: int, B_Q: int, B_KV: int, N: int, heads: int, d: int, plan_id: int = -1,
                       max_workspace_bytes: int = 0, stream=None, N_kv: int = 0, dtype: str = "bf16",
                       layout: str = "hnd") -> Plan:
    """``bsa_plan_create_packed``: ``mask_bits`` is a uint8 CUDA tensor of bit-packed rows (see ``pack_mask``)."""
    import torch
    assert mask_bits.is_cuda and mask_bits.is_contiguous() and mask_bits.dtype == torch.uint8
    h = ctypes.c_void_p()
    opt = Options(plan_id, DTYPES[dtype], max_workspace_bytes, N_kv, LAYOUTS[layout], 0)
    _check(lib().bsa_plan_create_packed(mask_bits.data_ptr(), row_stride, B_Q, B_KV, N, heads, d, ctypes.byref(opt),
                                        _stream_ptr(stream), ctypes.byref(h)), "bsa_plan_create_packed")
    return Plan(h.value, layout)


class PlanCache:
    """``bsa_plan_cache_*``: prepared plans keyed by a fingerprint of the mask's activity pattern (warm path)."""

    def __init__(self, capacity: int = 64):
        h = ctypes.c_void_p()
        _check(lib().bsa_plan_cache_create(capacity, ctypes.byref(h)), "bsa_plan_cache_create")
        self._h = h.value

    def get(self, mask, B_Q: int, B_KV: int, N: int, heads: int, d: int, plan_id: int = -1, max_workspace_bytes: int = 0,
            stream=None, row_stride: int = 0, N_kv: int = 0, dtype: str = "bf16", layout: str = "hnd"):
        """``bsa_plan_cache_get``: returns ``(plan, hit)``.  ``row_stride`` > 0: ``mask`` is bit-packed (``pack_mask``).
        The plan is shared with the cache; ``plan.destroy()`` only gives it back."""
        import torch
        assert mask.is_cuda and mask.is_contiguous() and mask.dtype in (torch.uint8, torch.bool)
        h = ctypes.c_void_p()
        hit = ctypes.c_int(0)
        opt = Options(plan_id, DTYPES[dtype], max_workspace_bytes, N_kv, LAYOUTS[layout], 0)
        _check(lib().bsa_plan_cache_get(self._h, mask.data_ptr(), row_stride, B_Q, B_KV, N, heads, d, ctypes.byref(opt),
                                        _stream_ptr(stream), ctypes.byref(h), ctypes.byref(hit)), "bsa_plan_cache_get")
        return Plan(h.value, layout), bool(hit.value)

    def request(self, mask, B_Q: int, B_KV: int, N: int, heads: int, d: int, Q, K, V, O, LSE, plan_id: int = -1,
                max_workspace_bytes: int = 0, stream=None, row_stride: int = 0, N_kv: int = 0, dtype: str = "bf16",
                layout: str = "hnd"):
        """``bsa_plan_cache_request``: ``get`` + ``forward`` in one call; returns ``(plan, hit)``."""
        h = ctypes.c_void_p()
        hit = ctypes.c_int(0)
        opt = Options(plan_id, DTYPES[dtype], max_workspace_bytes, N_kv, LAYOUTS[layout], 0)
        _check(lib().bsa_plan_cache_request(self._h, mask.data_ptr(), row_stride, B_Q, B_KV, N, heads, d, Q.data_ptr(),
                                            K.data_ptr(), V.data_ptr(), O.data_ptr(), LSE.data_ptr(), ctypes.byref(opt),
                                            _stream_ptr(stream), ctypes.byref(h), ctypes.byref(hit)),
               "bsa_plan_cache_request")
        return Plan(h.value, layout), bool(hit.value)

    def stats(self) -> Dict:
        a, b, c = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
        n = ctypes.c_int32()
        _check(lib().bsa_plan_cache_stats(self._h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c), ctypes.byref(n)),
               "bsa_plan_cache_stats")
        return {"hits": a.value, "misses": b.value, "evictions": c.value, "entries": n.value}

    def destroy(self):
        if self._h:
            _check(lib().bsa_plan_cache_destroy(self._h), "bsa_plan_cache_destroy")
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def request_host(mask: np.ndarray, B_Q: int, B_KV: int, N: int, heads: int, d: int, Q, K, V, O, LSE,
                 plan_id: int = -1, N_kv: int = 0, dtype: str = "bf16", layout: str = "hnd", batch: int = 0) -> Dict:
    """``bsa_request_host``: all arguments are HOST buffers (torch CPU tensors or numpy arrays)."""
    def ptr(x):
        return x.data_ptr() if hasattr(x, "data_ptr") else x.ctypes.data
    inf = PlanInfo()
    opt = Options(plan_id, DTYPES[dtype], 0, N_kv, LAYOUTS[layout], batch)
    _check(lib().bsa_request_host(ptr(mask), B_Q, B_KV, N, heads, d, ptr(Q), ptr(K), ptr(V), ptr(O), ptr(LSE),
                                  ctypes.byref(opt), ctypes.byref(inf)), "bsa_request_host")
    return inf.as_dict()


NOALLOC_MAX_ROWS = 1 << 20


def mask_stats_noalloc(mask, out=None, stream=None):
    """``bsa_mask_stats_noalloc``: statistics of a uint8/bool CUDA mask ``[heads, nQb, nKb]`` into an int64
    CUDA tensor of 4 entries, using the library's built-in scratch (no allocation inside the call when
    ``out`` is given).  Returns ``out``; raises ``BsaError`` (UNSUPPORTED) beyond ``NOALLOC_MAX_ROWS`` rows."""
    import torch
    assert mask.is_cuda and mask.is_contiguous() and mask.dtype in (torch.uint8, torch.bool) and mask.dim() == 3
    if out is None:
        out = torch.empty(4, dtype=torch.int64, device=mask.device)
    assert out.is_cuda and out.dtype == torch.int64 and out.numel() >= 4 and out.is_contiguous()
    h, nq, nk = mask.shape
    _check(lib().bsa_mask_stats_noalloc(mask.data_ptr(), h, nq, nk, out.data_ptr(), _stream_ptr(stream)),
           "bsa_mask_stats_noalloc")
    return out


def catalog() -> List[Dict]:
    out = []
    for i in range(lib().bsa_catalog_size()):
        d = PlanDesc()
        _check(lib().bsa_catalog_get(i, ctypes.byref(d)), "bsa_catalog_get")
        out.append({f: (getattr(d, f).decode() if f == "name" else getattr(d, f)) for f, _ in PlanDesc._fields_})
    return out


def plan_eligible(plan_id, B_Q, B_KV, N, heads, d, max_workspace_bytes=0, N_kv=0, dtype="bf16") -> bool:
    """``bsa_plan_eligible_ex``: Eligible(P, R) for the request's geometry, token counts, head dim and element type."""
    return bool(lib().bsa_plan_eligible_ex(plan_id, B_Q, B_KV, N, N_kv, heads, d, DTYPES[dtype], max_workspace_bytes))


def debug_set_wait_limit(cycles: int):
    """``bsa_debug_set_wait_limit`` (test hook): limit of the kernels' bounded waits in SM cycles; <= 0 = default."""
    _check(lib().bsa_debug_set_wait_limit(cycles), "bsa_debug_set_wait_limit")


def debug_withhold_arrival(on: bool):
    """``bsa_debug_withhold_arrival`` (test hook): make the next forwards' first V tile never arrive."""
    _check(lib().bsa_debug_withhold_arrival(1 if on else 0), "bsa_debug_withhold_arrival")


def lut_load(path: str):
    _check(lib().bsa_lut_load(path.encode()), "bsa_lut_load")


def lut_clear():
    lib().bsa_lut_clear()


def lut_select(B_Q, B_KV, N, heads, d, density, run_coverage, skew, max_workspace_bytes=0) -> Tuple[int, bool]:
    hit = ctypes.c_int(0)
    pid = lib().bsa_lut_select(B_Q, B_KV, N, heads, d, density, run_coverage, skew, max_workspace_bytes,
                               ctypes.byref(hit))
    return pid, bool(hit.value)


def lut_buckets(N, density, skew, run_coverage) -> List[int]:
    out = (ctypes.c_int32 * 4)()
    lib().bsa_lut_buckets(N, density, skew, run_coverage, out)
    return list(out)


def force_plan(plan_id: int):
    lib().bsa_force_plan(plan_id)


def kernel_launch_count() -> int:
    return int(lib().bsa_kernel_launch_count())
