"""Thin ctypes binding of librago.so: same names as include/rago.h, argument marshalling only.

Tensors are torch CUDA tensors (device memory and streams are torch's); every computation runs in
the library's kernels.  A missing or unloadable library raises -- there is no fallback path.
"""

from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librago.so")
_lib = None

RAGO_OK = 0
STATUS_NAMES = {0: "RAGO_OK", 1: "RAGO_EINVAL", 2: "RAGO_EALIGN", 3: "RAGO_EUNSUPPORTED", 4: "RAGO_ENOMEM",
                5: "RAGO_ECUDA", 6: "RAGO_ETIMEOUT"}
RAGO_L2, RAGO_IP = 0, 1
RAGO_F32, RAGO_BF16 = 0, 1
NUM_STAGES = 5
STAGE_NAMES = ("coarse_scores", "probe_select", "plan", "table_scan", "merge")

EXPORTS = ("rago_index_load", "rago_index_load_pq4", "rago_index_set_coarse_tree", "rago_index_free", "rago_search_workspace_bytes", "rago_search",
           "rago_search_probes", "rago_search_probes_noalloc", "rago_search_host", "rago_host_staging_bytes", "rago_flat_search",
           "rago_flat_workspace_bytes", "rago_check", "rago_set_coarse_mode", "rago_profile_enable", "rago_profile_read",
           "rago_merge_results", "rago_selftest_wait_timeout", "rago_debug_set_gemm_pairing", "rago_kernel_launches", "rago_last_error")


class RagoError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__("%s: %s" % (STATUS_NAMES.get(status, status), message))
        self.status = status


def lib() -> ctypes.CDLL:
    """Open librago.so (built by paper_2503_14649_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("librago.so is not built: run `python -m paper_2503_14649_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        L.rago_index_load.argtypes = [ctypes.POINTER(vp), vp, ctypes.c_int, vp, vp, vp, vp, i64, i32, i32, i32,
                                      ctypes.c_int, vp]
        L.rago_index_load_pq4.argtypes = L.rago_index_load.argtypes
        L.rago_index_set_coarse_tree.argtypes = [vp, vp, vp, i32, i32, vp]
        L.rago_index_free.argtypes = [vp]
        L.rago_search_workspace_bytes.argtypes = [vp, i32, i32, i32, ctypes.POINTER(sz)]
        L.rago_host_staging_bytes.argtypes = [vp, i32, i32, ctypes.POINTER(sz)]
        L.rago_search.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, sz, vp]
        L.rago_search_probes.argtypes = [vp, vp, i32, i32, vp, vp, vp, sz, vp]
        L.rago_search_probes_noalloc.argtypes = [vp, vp, i32, i32, vp, vp, vp]
        L.rago_search_host.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, sz, vp]
        L.rago_flat_search.argtypes = [vp, i64, i32, vp, i32, i32, vp, vp, vp, sz, vp]
        L.rago_flat_workspace_bytes.argtypes = [i64, i32, i32, i32, ctypes.POINTER(sz)]
        L.rago_merge_results.argtypes = [vp, vp, i32, i64, i32, i32, i32, i32, vp, vp, vp]
        L.rago_check.argtypes = [vp, vp]
        L.rago_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint32, i32, vp]
        L.rago_debug_set_gemm_pairing.argtypes = [i32]
        L.rago_set_coarse_mode.argtypes = [vp, i32]
        L.rago_profile_enable.argtypes = [vp, i32]
        L.rago_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
        L.rago_kernel_launches.restype = i64
        L.rago_last_error.restype = ctypes.c_char_p
        for name in EXPORTS:
            if name not in ("rago_kernel_launches", "rago_last_error"):
                getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _check(status: int):
    if status != RAGO_OK:
        raise RagoError(status, lib().rago_last_error().decode())


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def rago_kernel_launches() -> int:
    return int(lib().rago_kernel_launches())


class Index:
    """Handle from rago_index_load.  Keeps references to the borrowed tensors so they outlive it."""

    def __init__(self, centroids: torch.Tensor, codebooks: torch.Tensor, codes: torch.Tensor,
                 list_offsets: torch.Tensor, ids: torch.Tensor, metric):
        metric = {"l2": RAGO_L2, "ip": RAGO_IP}.get(metric, metric)
        dtype = RAGO_BF16 if centroids.dtype == torch.bfloat16 else RAGO_F32
        nlist, d = centroids.shape
        N = codes.shape[0]
        self._keep = (centroids, codebooks, codes, list_offsets, ids)
        self._h = ctypes.c_void_p()
        if codebooks.shape[1] == 16:  # 4-bit codes, two per byte: rago_index_load_pq4
            M4 = codebooks.shape[0]
            M = M4 // 2
            _check(lib().rago_index_load_pq4(ctypes.byref(self._h), _ptr(centroids), dtype, _ptr(codebooks),
                                             _ptr(codes), _ptr(list_offsets), _ptr(ids), N, d, nlist, M4, metric,
                                             _stream()))
        else:
            M = codebooks.shape[0]
            _check(lib().rago_index_load(ctypes.byref(self._h), _ptr(centroids), dtype, _ptr(codebooks), _ptr(codes),
                                         _ptr(list_offsets), _ptr(ids), N, d, nlist, M, metric, _stream()))
        self.nlist, self.d, self.M, self.N, self.metric = nlist, d, M, N, metric
        self._ws = None

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value and _lib is not None:
            try:
                _lib.rago_index_free(self._h)
            except Exception:  # interpreter shutdown: the module globals may already be gone
                pass
            self._h = ctypes.c_void_p()

    __del__ = close

    # -- sizes ---------------------------------------------------------------------------------
    def search_workspace_bytes(self, nq: int, nprobe: int, k: int) -> int:
        out = ctypes.c_size_t()
        _check(lib().rago_search_workspace_bytes(self._h, nq, nprobe, k, ctypes.byref(out)))
        return out.value

    def host_staging_bytes(self, nq: int, k: int) -> int:
        out = ctypes.c_size_t()
        _check(lib().rago_host_staging_bytes(self._h, nq, k, ctypes.byref(out)))
        return out.value

    def workspace(self, nbytes: int, device) -> torch.Tensor:
        """A cached, 256-byte aligned scratch tensor of at least nbytes (torch allocations are)."""
        if self._ws is None or self._ws.numel() < nbytes or self._ws.device != torch.device(device):
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
        return self._ws

    # -- calls ---------------------------------------------------------------------------------
    def rago_search(self, queries: torch.Tensor, nprobe: int, k: int,
                    out_ids: Optional[torch.Tensor] = None, out_dists: Optional[torch.Tensor] = None,
                    workspace: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
        nq = queries.shape[0]
        dev = queries.device
        if out_ids is None:
            out_ids = torch.empty((nq, k), dtype=torch.int64, device=dev)
        if out_dists is None:
            out_dists = torch.empty((nq, k), dtype=torch.float32, device=dev)
        if workspace is None:
            workspace = self.workspace(self.search_workspace_bytes(nq, nprobe, k), dev)
        _check(lib().rago_search(self._h, _ptr(queries), nq, nprobe, k, _ptr(out_ids), _ptr(out_dists),
                                 _ptr(workspace), workspace.numel(), _stream()))
        return out_ids, out_dists

    def rago_search_probes(self, queries: torch.Tensor, nprobe: int,
                           workspace: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
        nq = queries.shape[0]
        dev = queries.device
        lists = torch.empty((nq, nprobe), dtype=torch.int32, device=dev)
        coarse = torch.empty((nq, nprobe), dtype=torch.float32, device=dev)
        if workspace is None:
            workspace = self.workspace(self.search_workspace_bytes(nq, nprobe, 1), dev)
        _check(lib().rago_search_probes(self._h, _ptr(queries), nq, nprobe, _ptr(lists), _ptr(coarse),
                                        _ptr(workspace), workspace.numel(), _stream()))
        return lists, coarse

    def rago_search_probes_noalloc(self, queries: torch.Tensor, nprobe: int, out_lists: torch.Tensor,
                                   out_coarse: torch.Tensor):
        """rago_search_probes without a workspace: scratch is the library's built-in array, so the
        call allocates nothing (the outputs are the caller's).  Calls must not overlap on the GPU."""
        _check(lib().rago_search_probes_noalloc(self._h, _ptr(queries), queries.shape[0], nprobe, _ptr(out_lists),
                                                _ptr(out_coarse), _stream()))

    def rago_search_host(self, host_queries: torch.Tensor, nprobe: int, k: int, host_out_ids: torch.Tensor,
                         host_out_dists: torch.Tensor, workspace: torch.Tensor):
        nq = host_queries.shape[0]
        _check(lib().rago_search_host(self._h, _ptr(host_queries), nq, nprobe, k, _ptr(host_out_ids),
                                      _ptr(host_out_dists), _ptr(workspace), workspace.numel(), _stream()))

    def rago_check(self, workspace: Optional[torch.Tensor] = None):
        ws = workspace if workspace is not None else self._ws
        _check(lib().rago_check(_ptr(ws), _stream()))

    def rago_set_coarse_mode(self, mode: int):
        _check(lib().rago_set_coarse_mode(self._h, int(mode)))
        self._ws = None  # workspace sizes depend on the mode

    def rago_index_set_coarse_tree(self, level1: Optional[torch.Tensor], child_offsets: Optional[torch.Tensor], b1: int = 0):
        """Set (or, with level1 = None, remove) the level above the coarse centroids; tensors are borrowed."""
        if level1 is None:
            _check(lib().rago_index_set_coarse_tree(self._h, None, None, 0, 0, _stream()))
            self._tree = None
        else:
            _check(lib().rago_index_set_coarse_tree(self._h, _ptr(level1), _ptr(child_offsets), level1.shape[0], int(b1),
                                                    _stream()))
            self._tree = (level1, child_offsets)
        self._ws = None  # workspace sizes depend on it

    def rago_profile_enable(self, enable: bool = True):
        _check(lib().rago_profile_enable(self._h, int(enable)))

    def rago_profile_read(self):
        out = (ctypes.c_float * NUM_STAGES)()
        _check(lib().rago_profile_read(self._h, out))
        return dict(zip(STAGE_NAMES, [float(v) for v in out]))


def rago_index_load(centroids, codebooks, codes, list_offsets, ids, metric) -> Index:
    return Index(centroids, codebooks, codes, list_offsets, ids, metric)


def rago_index_load_pq4(centroids, pq4_codebooks, packed_codes, list_offsets, ids, metric) -> Index:
    """pq4_codebooks [M4, 16, d / M4], packed_codes uint8 [N, M4 / 2] (low nibble = even sub-space)."""
    if pq4_codebooks.shape[1] != 16:
        raise ValueError("4-bit codebooks have 16 codewords per sub-space")
    return Index(centroids, pq4_codebooks, packed_codes, list_offsets, ids, metric)


def rago_debug_set_gemm_pairing(mode: int):
    """0: the library chooses the tensor-core main loop by operand size, 1: one row tile per CTA, 2: two row tiles
    per CTA, 3: two row tiles per CTA pair (cluster of two)."""
    _check(lib().rago_debug_set_gemm_pairing(int(mode)))


def rago_selftest_wait_timeout(workspace: torch.Tensor, max_polls: int, with_tmem: bool):
    """Launch the bounded-wait self-test on `workspace` (see rago.h); follow with rago_check(workspace)."""
    _check(lib().rago_selftest_wait_timeout(_ptr(workspace), int(max_polls), int(bool(with_tmem)), _stream()))


def rago_check(workspace: torch.Tensor):
    """rago_check on a bare workspace tensor (Index.rago_check does the same for an index's workspace)."""
    _check(lib().rago_check(_ptr(workspace), _stream()))


def rago_flat_workspace_bytes(N: int, d: int, nq: int, k: int) -> int:
    out = ctypes.c_size_t()
    _check(lib().rago_flat_workspace_bytes(N, d, nq, k, ctypes.byref(out)))
    return out.value


def rago_flat_search(db: torch.Tensor, queries: torch.Tensor, k: int, workspace: Optional[torch.Tensor] = None):
    N, d = db.shape
    nq = queries.shape[0]
    dev = queries.device
    out_ids = torch.empty((nq, k), dtype=torch.int64, device=dev)
    out_scores = torch.empty((nq, k), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = torch.empty(rago_flat_workspace_bytes(N, d, nq, k), dtype=torch.uint8, device=dev)
    _check(lib().rago_flat_search(_ptr(db), N, d, _ptr(queries), nq, k, _ptr(out_ids), _ptr(out_scores),
                                  _ptr(workspace), workspace.numel(), _stream()))
    return out_ids, out_scores


def rago_merge_results(part_ids: torch.Tensor, part_dists: torch.Tensor, k_out: int, metric,
                       out_ids: Optional[torch.Tensor] = None, out_dists: Optional[torch.Tensor] = None):
    """part_ids / part_dists: contiguous [nparts, nq, k_in] device tensors (the shards' answers side by side)."""
    metric = {"l2": RAGO_L2, "ip": RAGO_IP}.get(metric, metric)
    nparts, nq, k_in = part_ids.shape
    if part_dists.shape != part_ids.shape or not (part_ids.is_contiguous() and part_dists.is_contiguous()):
        raise ValueError("part_ids and part_dists must be contiguous tensors of one shape [nparts, nq, k_in]")
    dev = part_ids.device
    if out_ids is None:
        out_ids = torch.empty((nq, k_out), dtype=torch.int64, device=dev)
    if out_dists is None:
        out_dists = torch.empty((nq, k_out), dtype=torch.float32, device=dev)
    _check(lib().rago_merge_results(_ptr(part_ids), _ptr(part_dists), nparts, nq * k_in, nq, k_in, k_out, metric,
                                    _ptr(out_ids), _ptr(out_dists), _stream()))
    return out_ids, out_dists


def load_index_from(data, device="cuda") -> Index:
    """rago_index_load over a synth.IvfPqData (moves its tensors to `device` first)."""
    dev = torch.device(device)
    return Index(data.centroids.to(dev).contiguous(), data.codebooks.to(dev).contiguous(),
                 data.codes.to(dev).contiguous(), data.list_offsets.to(dev).contiguous(),
                 data.ids.to(dev).contiguous(), data.metric)
