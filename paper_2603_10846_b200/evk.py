"""Python binding of the C-ABI library ``libevk.so`` (see ``include/evk.h``).

Argument marshalling only: tensors are checked for device, dtype and contiguity
and handed to the library as raw pointers; every step of retrieval and of the
value update runs in the library's CUDA kernels.  PyTorch supplies device memory
and streams.  There is no CPU fallback: importing this module without the built
library raises, and calling into it without a CUDA device fails in the library.

Function names mirror the C ABI: ``evk_mem_create``, ``evk_mem_insert``,
``evk_retrieve``, ``evk_q_update`` and the helpers around them.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libevk.so")

EVK_OK = 0
EVK_ERR_INVALID = -1
EVK_ERR_CAPACITY = -2
EVK_ERR_WORKSPACE = -3
EVK_ERR_RANGE = -4
EVK_ERR_NONFINITE = -5
EVK_ERR_DEVICE_TIMEOUT = -6
EVK_ERR_CUDA = -7
EVK_ERR_UNSUPPORTED = -8
EVK_ERR_INCOMPLETE = -9

EVK_DTYPE_F32, EVK_DTYPE_BF16 = 0, 1
EVK_STAGE_DRAFT, EVK_STAGE_REFINE, EVK_STAGE_ALL = 0, 1, -1
EVK_SCORING_AUTO, EVK_SCORING_STREAM, EVK_SCORING_TENSOR = 0, 1, 2
EVK_NORM_NONE, EVK_NORM_POOL_ZSCORE = 0, 1
EVK_MAX_K1 = 1024

# Every symbol include/evk.h declares.
EXPORTS = (
    "evk_mem_bytes_required", "evk_mem_create", "evk_mem_destroy", "evk_mem_size",
    "evk_mem_set_scoring", "evk_mem_set_score_norm", "evk_mem_inject_stall", "evk_mem_insert", "evk_retrieve_workspace_bytes", "evk_retrieve",
    "evk_q_update_workspace_bytes", "evk_q_update", "evk_q_update_static", "evk_q_update_decay", "evk_visits_read", "evk_visits_write", "evk_q_read", "evk_q_write", "evk_bank_read",
    "evk_retrieve_host_workspace_bytes", "evk_retrieve_host", "evk_q_update_host_workspace_bytes",
    "evk_q_update_host", "evk_mem_set_host_staging", "evk_mem_insert_host_workspace_bytes", "evk_mem_insert_host",
    "evk_retrieve_plan", "evk_mem_profile_scoring", "evk_retrieve_explore_workspace_bytes",
    "evk_retrieve_explore", "evk_select_by_value", "evk_retrieve_local_workspace_bytes", "evk_retrieve_local",
    "evk_merge_shards", "evk_reward_draft",
    "evk_reward_refine", "evk_reward_norm_state_bytes", "evk_reward_norm_reset", "evk_reward_normalize", "evk_last_status",
    "evk_launch_count", "evk_strerror", "evk_mem_tombstone", "evk_mem_export", "evk_mem_import", "evk_mem_stats",
    "evk_mem_read_probe",
)


class EvkError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} ({status})")


class _Stats(ctypes.Structure):
    _fields_ = [(name, ctypes.c_int64) for name in (
        "entries", "live_entries", "dropped_entries", "retrieve_calls", "update_calls", "insert_calls",
        "kernel_launches", "candidates_filed", "list_cutbacks", "longest_update_run")]


class _Config(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("n_stages", ctypes.c_int32), ("capacity", ctypes.c_int64),
                ("q_default", ctypes.c_float), ("reserved", ctypes.c_int32),
                ("arena", ctypes.c_void_p), ("arena_bytes", ctypes.c_size_t)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2603_10846_b200.build` "
            "(nvcc, sm_100a). There is no fallback path.")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
    cint = ctypes.c_int
    cfgp = ctypes.POINTER(_Config)
    sig = {
        "evk_mem_bytes_required": (sz, [cfgp]),
        "evk_mem_create": (cint, [cfgp, ctypes.POINTER(vp)]),
        "evk_mem_destroy": (cint, [vp]),
        "evk_mem_size": (i64, [vp]),
        "evk_mem_set_scoring": (cint, [vp, cint]),
        "evk_mem_set_score_norm": (cint, [vp, cint]),
        "evk_mem_inject_stall": (cint, [vp]),
        "evk_mem_insert": (cint, [vp, vp, cint, i64, cint, vp, vp, vp]),
        "evk_retrieve_workspace_bytes": (sz, [vp, i32, i32]),
        "evk_retrieve": (cint, [vp, vp, cint, i32, cint, i32, i32, f32, vp, vp, vp, vp, vp, sz, vp]),
        "evk_q_update_workspace_bytes": (sz, [vp, i64]),
        "evk_q_update": (cint, [vp, vp, i64, cint, vp, f32, vp, sz, vp]),
        "evk_q_update_static": (cint, [vp, vp, i64, cint, vp, f32, vp]),
        "evk_q_update_decay": (cint, [vp, vp, i64, cint, vp, vp, sz, vp]),
        "evk_visits_read": (cint, [vp, cint, i64, i64, vp, vp]),
        "evk_visits_write": (cint, [vp, cint, i64, i64, vp, vp]),
        "evk_q_read": (cint, [vp, cint, i64, i64, vp, vp]),
        "evk_q_write": (cint, [vp, cint, i64, i64, vp, vp]),
        "evk_bank_read": (cint, [vp, i64, i64, vp, vp]),
        "evk_retrieve_host_workspace_bytes": (sz, [vp, i32, i32, i32]),
        "evk_retrieve_host": (cint, [vp, vp, cint, i32, cint, i32, i32, f32, vp, vp, vp, sz, vp]),
        "evk_q_update_host_workspace_bytes": (sz, [vp, i64]),
        "evk_q_update_host": (cint, [vp, vp, i64, cint, vp, f32, vp, sz, vp]),
        "evk_mem_set_host_staging": (cint, [vp, vp, sz]),
        "evk_mem_insert_host_workspace_bytes": (sz, [vp, i64]),
        "evk_mem_insert_host": (cint, [vp, vp, cint, i64, cint, vp, vp, sz, vp]),
        "evk_retrieve_plan": (cint, [vp, i32, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]),
        "evk_mem_profile_scoring": (cint, [vp, vp, vp]),
        "evk_retrieve_explore_workspace_bytes": (sz, [vp, i32, i32]),
        "evk_retrieve_explore": (cint, [vp, vp, cint, i32, cint, i32, i32, f32, f32, ctypes.c_uint64, ctypes.c_uint64,
                                        vp, vp, vp, vp, vp, vp, sz, vp]),
        "evk_select_by_value": (cint, [vp, vp, vp, i32, cint, i32, vp, vp, vp]),
        "evk_retrieve_local_workspace_bytes": (sz, [vp, i32, i32]),
        "evk_retrieve_local": (cint, [vp, vp, cint, i32, cint, i32, i32, vp, vp, vp, vp, sz, vp]),
        "evk_merge_shards": (cint, [vp, vp, vp, i32, i32, i32, i32, f32, vp, vp, vp, vp, vp]),
        "evk_reward_draft": (cint, [vp, i64, vp, vp]),
        "evk_reward_refine": (cint, [vp, vp, vp, i64, vp, vp]),
        "evk_reward_norm_state_bytes": (sz, []),
        "evk_reward_norm_reset": (cint, [vp, vp]),
        "evk_reward_normalize": (cint, [vp, vp, i64, f32, f32, vp, vp]),
        "evk_last_status": (cint, [vp, vp]),
        "evk_launch_count": (i64, [vp]),
        "evk_strerror": (ctypes.c_char_p, [cint]),
        "evk_mem_tombstone": (cint, [vp, vp, i64, vp]),
        "evk_mem_export": (cint, [vp, i64, i64, vp, vp, vp, vp, vp]),
        "evk_mem_import": (cint, [vp, i64, vp, vp, vp, vp, vp, vp]),
        "evk_mem_stats": (cint, [vp, ctypes.POINTER(_Stats), vp]),
        "evk_mem_read_probe": (cint, [vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


_lib = _load()


def strerror(status: int) -> str:
    return _lib.evk_strerror(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != EVK_OK:
        raise EvkError(status, where)


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    if stream is not None:
        return int(stream.cuda_stream)
    if _raw_stream is not None:      # the current stream's handle without building a Stream object
        return int(_raw_stream(torch.cuda.current_device()))
    return int(torch.cuda.current_stream().cuda_stream)


def _dev(t: Optional[torch.Tensor], dtype=None, name="tensor") -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _host(t: torch.Tensor, dtype=None, name="tensor") -> int:
    if t.is_cuda or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous host tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _emb_dtype(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return EVK_DTYPE_F32
    if t.dtype == torch.bfloat16:
        return EVK_DTYPE_BF16
    raise ValueError(f"embeddings must be float32 or bfloat16, got {t.dtype}")


class EvkMem:
    """Handle of one memory bank: the opaque pointer plus the arena tensor that
    backs it (kept alive here; the library does not own device memory)."""

    def __init__(self, handle: int, arena: torch.Tensor, d: int, capacity: int, n_stages: int):
        self.handle = handle
        self.arena = arena
        self.d, self.capacity, self.n_stages = d, capacity, n_stages
        self._ws = {}
        self._ws_bytes = {}
        self.staging = None      # the page-locked tensor given to evk_mem_set_host_staging, kept alive here

    def workspace_for(self, kind: str, key, size_fn) -> torch.Tensor:
        """The scratch tensor of one call shape; the library is asked for its size once per shape
        (sizes depend on the shape, the bank's capacity and the scoring mode only)."""
        nbytes = self._ws_bytes.get((kind, key))
        if nbytes is None:
            nbytes = self._ws_bytes[(kind, key)] = int(size_fn())
        return self.workspace(kind, nbytes)

    def workspace(self, kind: str, nbytes: int) -> torch.Tensor:
        """A cached scratch tensor of at least nbytes on the arena's device."""
        t = self._ws.get(kind)
        if t is None or t.numel() < nbytes:
            t = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=self.arena.device)
            self._ws[kind] = t
        return t

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h and _lib is not None:   # at interpreter exit the module may already be torn down
            _lib.evk_mem_destroy(h)


def evk_mem_bytes_required(d: int, capacity: int, n_stages: int = 2) -> int:
    cfg = _Config(d, n_stages, capacity, 0.0, 0, None, 0)
    n = _lib.evk_mem_bytes_required(ctypes.byref(cfg))
    if n == 0:
        raise EvkError(EVK_ERR_INVALID, "evk_mem_bytes_required")
    return int(n)


def evk_mem_create(d: int, capacity: int, n_stages: int = 2, q_default: float = 0.0,
                   device="cuda", arena: Optional[torch.Tensor] = None) -> EvkMem:
    nbytes = evk_mem_bytes_required(d, capacity, n_stages)
    if arena is None:
        arena = torch.empty(nbytes, dtype=torch.uint8, device=device)
    cfg = _Config(d, n_stages, capacity, q_default, 0, _dev(arena, torch.uint8, "arena"), arena.numel())
    out = ctypes.c_void_p()
    with torch.cuda.device(arena.device):
        _check(_lib.evk_mem_create(ctypes.byref(cfg), ctypes.byref(out)), "evk_mem_create")
    return EvkMem(out.value, arena, d, capacity, n_stages)


def evk_mem_destroy(mem: EvkMem) -> None:
    h, mem.handle = mem.handle, None
    if h:
        _check(_lib.evk_mem_destroy(h), "evk_mem_destroy")


def evk_mem_size(mem: EvkMem) -> int:
    return int(_lib.evk_mem_size(mem.handle))


def evk_launch_count(mem: EvkMem) -> int:
    return int(_lib.evk_launch_count(mem.handle))


def evk_mem_set_scoring(mem: EvkMem, mode: int) -> None:
    _check(_lib.evk_mem_set_scoring(mem.handle, mode), "evk_mem_set_scoring")
    mem._ws_bytes.clear()


def evk_mem_set_score_norm(mem: EvkMem, mode: int) -> None:
    _check(_lib.evk_mem_set_score_norm(mem.handle, mode), "evk_mem_set_score_norm")


def evk_mem_insert(mem: EvkMem, emb: torch.Tensor, stage: int = EVK_STAGE_ALL,
                   q_init: Optional[torch.Tensor] = None, return_ids: bool = False, stream=None):
    n = emb.shape[0]
    if emb.dim() != 2 or emb.shape[1] != mem.d:
        raise ValueError("emb must be [n][d]")
    ids = torch.empty(n, dtype=torch.int32, device=emb.device) if return_ids else None
    _check(_lib.evk_mem_insert(mem.handle, _dev(emb, None, "emb"), _emb_dtype(emb), n, stage,
                               _dev(q_init, torch.float32, "q_init"), _dev(ids), _stream_ptr(stream)),
           "evk_mem_insert")
    return ids


def evk_retrieve_workspace_bytes(mem: EvkMem, B: int, k1: int) -> int:
    return int(_lib.evk_retrieve_workspace_bytes(mem.handle, B, k1))


def evk_retrieve(mem: EvkMem, queries: torch.Tensor, stage: int, k1: int, k2: int, w: float,
                 return_pool: bool = False, workspace: Optional[torch.Tensor] = None, stream=None,
                 out=None):
    """Returns (ids [B][k2] int32, scores [B][k2] fp32[, pool_ids, pool_sims])."""
    if queries.dim() != 2 or queries.shape[1] != mem.d:
        raise ValueError("queries must be [B][d]")
    B = queries.shape[0]
    dev = queries.device
    if out is None:
        ids = torch.empty((B, k2), dtype=torch.int32, device=dev)
        scores = torch.empty((B, k2), dtype=torch.float32, device=dev)
    else:
        ids, scores = out
    pool_ids = torch.empty((B, k1), dtype=torch.int32, device=dev) if return_pool else None
    pool_sims = torch.empty((B, k1), dtype=torch.float32, device=dev) if return_pool else None
    if workspace is None:
        workspace = mem.workspace_for("retrieve", (B, k1), lambda: _lib.evk_retrieve_workspace_bytes(mem.handle, B, k1))
    _check(_lib.evk_retrieve(mem.handle, _dev(queries, None, "queries"), _emb_dtype(queries), B, stage,
                             k1, k2, float(w), _dev(ids, torch.int32), _dev(scores, torch.float32),
                             _dev(pool_ids), _dev(pool_sims),
                             _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream)),
           "evk_retrieve")
    if return_pool:
        return ids, scores, pool_ids, pool_sims
    return ids, scores


def evk_q_update_workspace_bytes(mem: EvkMem, M: int) -> int:
    return int(_lib.evk_q_update_workspace_bytes(mem.handle, M))


def evk_q_update(mem: EvkMem, ids: torch.Tensor, stage: int, rewards: torch.Tensor, alpha: float,
                 workspace: Optional[torch.Tensor] = None, stream=None) -> None:
    M = ids.numel()
    if rewards.numel() != M:
        raise ValueError("ids and rewards must have the same length")
    if workspace is None:
        workspace = mem.workspace_for("q_update", M, lambda: _lib.evk_q_update_workspace_bytes(mem.handle, M))
    _check(_lib.evk_q_update(mem.handle, _dev(ids, torch.int32, "ids"), M, stage,
                             _dev(rewards, torch.float32, "rewards"), float(alpha),
                             _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream)),
           "evk_q_update")


EVK_Q_UPDATE_STATIC_MAX = 65536


def evk_q_update_static(mem: EvkMem, ids: torch.Tensor, stage: int, rewards: torch.Tensor, alpha: float,
                        stream=None) -> None:
    """evk_q_update without a workspace: the sort's scratch is a fixed array inside the
    library, so nothing is allocated here or in the library.  For callers whose device memory
    is fully budgeted or who may not allocate while serving.  At most EVK_Q_UPDATE_STATIC_MAX
    updates per call; calls on one device share the scratch and must not overlap on the GPU."""
    M = ids.numel()
    if rewards.numel() != M:
        raise ValueError("ids and rewards must have the same length")
    _check(_lib.evk_q_update_static(mem.handle, _dev(ids, torch.int32, "ids"), M, stage,
                                    _dev(rewards, torch.float32, "rewards"), float(alpha), _stream_ptr(stream)),
           "evk_q_update_static")


def evk_q_read(mem: EvkMem, stage: int, first: int = 0, n: Optional[int] = None, stream=None) -> torch.Tensor:
    n = evk_mem_size(mem) - first if n is None else n
    out = torch.empty(n, dtype=torch.float32, device=mem.arena.device)
    _check(_lib.evk_q_read(mem.handle, stage, first, n, _dev(out), _stream_ptr(stream)), "evk_q_read")
    return out


def evk_q_write(mem: EvkMem, stage: int, values: torch.Tensor, first: int = 0, stream=None) -> None:
    _check(_lib.evk_q_write(mem.handle, stage, first, values.numel(), _dev(values, torch.float32, "values"),
                            _stream_ptr(stream)), "evk_q_write")


def evk_bank_read(mem: EvkMem, first: int = 0, n: Optional[int] = None, stream=None) -> torch.Tensor:
    n = evk_mem_size(mem) - first if n is None else n
    out = torch.empty((n, mem.d), dtype=torch.bfloat16, device=mem.arena.device)
    _check(_lib.evk_bank_read(mem.handle, first, n, _dev(out), _stream_ptr(stream)), "evk_bank_read")
    return out


def evk_mem_tombstone(mem: EvkMem, ids: torch.Tensor, stream=None) -> None:
    """Drop the entries `ids` (int32 CUDA tensor) from the memory; the others keep their ids."""
    _check(_lib.evk_mem_tombstone(mem.handle, _dev(ids, torch.int32, "ids"), ids.numel(), _stream_ptr(stream)),
           "evk_mem_tombstone")


def evk_mem_export(mem: EvkMem, first: int = 0, n: Optional[int] = None, stream=None):
    """Entries [first, first + n) as (rows bf16 [n][d], q fp32 [S][n], visits int32 [S][n], live uint8 [n])."""
    n = evk_mem_size(mem) - first if n is None else n
    dev = mem.arena.device
    rows = torch.empty((n, mem.d), dtype=torch.bfloat16, device=dev)
    q = torch.empty((mem.n_stages, n), dtype=torch.float32, device=dev)
    visits = torch.empty((mem.n_stages, n), dtype=torch.int32, device=dev)
    live = torch.empty(n, dtype=torch.uint8, device=dev)
    _check(_lib.evk_mem_export(mem.handle, first, n, _dev(rows), _dev(q), _dev(visits), _dev(live),
                               _stream_ptr(stream)), "evk_mem_export")
    return rows, q, visits, live


def evk_mem_import(mem: EvkMem, rows: torch.Tensor, q: Optional[torch.Tensor] = None,
                   visits: Optional[torch.Tensor] = None, live: Optional[torch.Tensor] = None,
                   return_ids: bool = False, stream=None):
    """Append entries with their per-stage values [S][n], update counts [S][n] and live marks [n]."""
    n = rows.shape[0]
    if rows.dim() != 2 or rows.shape[1] != mem.d:
        raise ValueError("rows must be [n][d]")
    for name, t in (("q", q), ("visits", visits)):
        if t is not None and tuple(t.shape) != (mem.n_stages, n):
            raise ValueError(f"{name} must be [n_stages][n]")
    if live is not None and live.numel() != n:
        raise ValueError("live must have n elements")
    ids = torch.empty(n, dtype=torch.int32, device=rows.device) if return_ids else None
    _check(_lib.evk_mem_import(mem.handle, n, _dev(rows, torch.bfloat16, "rows"), _dev(q, torch.float32, "q"),
                               _dev(visits, torch.int32, "visits"), _dev(live, torch.uint8, "live"), _dev(ids),
                               _stream_ptr(stream)), "evk_mem_import")
    return ids


def evk_mem_stats(mem: EvkMem, stream=None) -> dict:
    """Counters of the bank (synchronises the stream): see evk_stats in the header."""
    st = _Stats()
    _check(_lib.evk_mem_stats(mem.handle, ctypes.byref(st), _stream_ptr(stream)), "evk_mem_stats")
    return {name: int(getattr(st, name)) for name, _ in _Stats._fields_}


def evk_mem_read_probe(mem: EvkMem, stream=None) -> None:
    """Measurement aid: stream the stored rows once into shared memory (time it with CUDA events)."""
    _check(_lib.evk_mem_read_probe(mem.handle, _stream_ptr(stream)), "evk_mem_read_probe")


def evk_retrieve_host(mem: EvkMem, queries_host: torch.Tensor, stage: int, k1: int, k2: int, w: float,
                      ids_out_host: torch.Tensor, scores_out_host: torch.Tensor, stream=None) -> None:
    """Host-buffer form: copies queries in and results out inside the call, then synchronises."""
    B = queries_host.shape[0]
    ws = mem.workspace_for("retrieve_host", (B, k1, k2),
                           lambda: _lib.evk_retrieve_host_workspace_bytes(mem.handle, B, k1, k2))
    _check(_lib.evk_retrieve_host(mem.handle, _host(queries_host, None, "queries_host"),
                                  _emb_dtype(queries_host), B, stage, k1, k2, float(w),
                                  _host(ids_out_host, torch.int32), _host(scores_out_host, torch.float32),
                                  _dev(ws), ws.numel(), _stream_ptr(stream)), "evk_retrieve_host")


def evk_mem_set_host_staging(mem: EvkMem, nbytes: int = 4 << 20) -> None:
    """Give the bank a page-locked staging buffer of nbytes (0 withdraws it): evk_q_update_host and
    evk_mem_insert_host then return without waiting for the device, and evk_retrieve_host receives
    its result without a copy of its own."""
    if nbytes <= 0:
        _check(_lib.evk_mem_set_host_staging(mem.handle, None, 0), "evk_mem_set_host_staging")
        mem.staging = None
        return
    # a torch allocation may start anywhere: over-allocate and hand over the 256-byte aligned part
    buf = torch.empty(int(nbytes) + 256, dtype=torch.uint8).pin_memory()
    skip = (-buf.data_ptr()) % 256
    with torch.cuda.device(mem.arena.device):
        _check(_lib.evk_mem_set_host_staging(mem.handle, buf.data_ptr() + skip, int(nbytes)), "evk_mem_set_host_staging")
    mem.staging = buf


def evk_mem_insert_host(mem: EvkMem, emb_host: torch.Tensor, stage: int = EVK_STAGE_ALL,
                        q_init_host: Optional[torch.Tensor] = None, stream=None) -> None:
    """Host-buffer form of evk_mem_insert: the rows (and start values) are host tensors."""
    if emb_host.dim() != 2 or emb_host.shape[1] != mem.d:
        raise ValueError("emb_host must be [n][d]")
    n = emb_host.shape[0]
    ws = mem.workspace_for("insert_host", n, lambda: _lib.evk_mem_insert_host_workspace_bytes(mem.handle, n))
    _check(_lib.evk_mem_insert_host(mem.handle, _host(emb_host, None, "emb_host"), _emb_dtype(emb_host), n, stage,
                                    _host(q_init_host, torch.float32, "q_init_host") if q_init_host is not None else None,
                                    _dev(ws), ws.numel(), _stream_ptr(stream)), "evk_mem_insert_host")


def evk_q_update_host(mem: EvkMem, ids_host: torch.Tensor, stage: int, rewards_host: torch.Tensor,
                      alpha: float, stream=None) -> None:
    M = ids_host.numel()
    ws = mem.workspace_for("q_update_host", M, lambda: _lib.evk_q_update_host_workspace_bytes(mem.handle, M))
    _check(_lib.evk_q_update_host(mem.handle, _host(ids_host, torch.int32), M, stage,
                                  _host(rewards_host, torch.float32), float(alpha),
                                  _dev(ws), ws.numel(), _stream_ptr(stream)), "evk_q_update_host")


def evk_retrieve_plan(mem: EvkMem, B: int, k1: int):
    """(kernel kind, number of phase-1 launches) evk_retrieve would use at the current size."""
    kind, launches = ctypes.c_int32(), ctypes.c_int32()
    _check(_lib.evk_retrieve_plan(mem.handle, B, k1, ctypes.byref(kind), ctypes.byref(launches)),
           "evk_retrieve_plan")
    return kind.value, launches.value


def evk_mem_profile_scoring(mem: EvkMem, start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]) -> None:
    """Arm the next evk_retrieve to record these events around its phase-1 launches.
    The events must already exist on the device (record them once before first use)."""
    s = start.cuda_event if start is not None else None
    e = stop.cuda_event if stop is not None else None
    _check(_lib.evk_mem_profile_scoring(mem.handle, s, e), "evk_mem_profile_scoring")


def evk_last_status(mem: EvkMem, stream=None) -> int:
    return int(_lib.evk_last_status(mem.handle, _stream_ptr(stream)))


def evk_reward_draft(feasible: torch.Tensor, stream=None) -> torch.Tensor:
    """Eq. 5: +1 where feasible else -1.  feasible: uint8 CUDA tensor."""
    out = torch.empty(feasible.numel(), dtype=torch.float32, device=feasible.device)
    _check(_lib.evk_reward_draft(_dev(feasible, torch.uint8, "feasible"), feasible.numel(), _dev(out),
                                 _stream_ptr(stream)), "evk_reward_draft")
    return out


def evk_reward_refine(best_latency: torch.Tensor, latency: torch.Tensor, feasible: torch.Tensor,
                      stream=None) -> torch.Tensor:
    """Eq. 6: -1 where infeasible else tanh(log best - log latency)."""
    n = latency.numel()
    out = torch.empty(n, dtype=torch.float32, device=latency.device)
    _check(_lib.evk_reward_refine(_dev(best_latency, torch.float32, "best_latency"),
                                  _dev(latency, torch.float32, "latency"), _dev(feasible, torch.uint8, "feasible"),
                                  n, _dev(out), _stream_ptr(stream)), "evk_reward_refine")
    return out


def evk_reward_norm_state(device="cuda", stream=None) -> torch.Tensor:
    """A fresh (zeroed) running-statistics state for evk_reward_normalize."""
    state = torch.empty(int(_lib.evk_reward_norm_state_bytes()) // 8, dtype=torch.float64, device=device)
    _check(_lib.evk_reward_norm_reset(_dev(state), _stream_ptr(stream)), "evk_reward_norm_reset")
    return state


def evk_reward_normalize(state: torch.Tensor, raw: torch.Tensor, sigma_min: float, clip: float = 0.0,
                         stream=None) -> torch.Tensor:
    """Running z-score of raw rewards with the statistics seen before each one (Appendix A)."""
    out = torch.empty(raw.numel(), dtype=torch.float32, device=raw.device)
    _check(_lib.evk_reward_normalize(_dev(state, torch.float64, "state"), _dev(raw, torch.float32, "raw"),
                                     raw.numel(), float(sigma_min), float(clip), _dev(out), _stream_ptr(stream)),
           "evk_reward_normalize")
    return out


def evk_retrieve_explore(mem: EvkMem, queries: torch.Tensor, stage: int, k1: int, k2: int, w: float,
                         epsilon: float, seed: int, step: int, return_pool: bool = False, stream=None):
    """evk_retrieve with epsilon-greedy exploration; returns (ids, scores, explored[, pool_ids, pool_sims])."""
    if queries.dim() != 2 or queries.shape[1] != mem.d:
        raise ValueError("queries must be [B][d]")
    B, dev = queries.shape[0], queries.device
    ids = torch.empty((B, k2), dtype=torch.int32, device=dev)
    scores = torch.empty((B, k2), dtype=torch.float32, device=dev)
    explored = torch.empty(B, dtype=torch.uint8, device=dev)
    pool_ids = torch.empty((B, k1), dtype=torch.int32, device=dev) if return_pool else None
    pool_sims = torch.empty((B, k1), dtype=torch.float32, device=dev) if return_pool else None
    ws = mem.workspace("retrieve_explore", int(_lib.evk_retrieve_explore_workspace_bytes(mem.handle, B, k1)))
    _check(_lib.evk_retrieve_explore(mem.handle, _dev(queries, None, "queries"), _emb_dtype(queries), B, stage,
                                     k1, k2, float(w), float(epsilon), int(seed), int(step), _dev(ids), _dev(scores),
                                     _dev(explored), _dev(pool_ids), _dev(pool_sims), _dev(ws), ws.numel(),
                                     _stream_ptr(stream)), "evk_retrieve_explore")
    if return_pool:
        return ids, scores, explored, pool_ids, pool_sims
    return ids, scores, explored


def evk_select_by_value(mem: EvkMem, cand_ids: torch.Tensor, offsets: torch.Tensor, stage: int, k: int,
                        stream=None):
    """Per task, the k candidates of largest Q_stage: (ids [T][k], q [T][k])."""
    T = offsets.numel() - 1
    ids = torch.empty((T, k), dtype=torch.int32, device=cand_ids.device)
    q = torch.empty((T, k), dtype=torch.float32, device=cand_ids.device)
    _check(_lib.evk_select_by_value(mem.handle, _dev(cand_ids, torch.int32, "cand_ids"),
                                    _dev(offsets, torch.int32, "offsets"), T, stage, k, _dev(ids), _dev(q),
                                    _stream_ptr(stream)), "evk_select_by_value")
    return ids, q


def evk_q_update_decay(mem: EvkMem, ids: torch.Tensor, stage: int, rewards: torch.Tensor, stream=None) -> None:
    """Value update with alpha_t = 1 / visits (running mean of an entry's rewards)."""
    M = ids.numel()
    if rewards.numel() != M:
        raise ValueError("ids and rewards must have the same length")
    ws = mem.workspace("q_update", evk_q_update_workspace_bytes(mem, M))
    _check(_lib.evk_q_update_decay(mem.handle, _dev(ids, torch.int32, "ids"), M, stage,
                                   _dev(rewards, torch.float32, "rewards"), _dev(ws), ws.numel(),
                                   _stream_ptr(stream)), "evk_q_update_decay")


def evk_visits_read(mem: EvkMem, stage: int, first: int = 0, n: Optional[int] = None, stream=None) -> torch.Tensor:
    n = evk_mem_size(mem) - first if n is None else n
    out = torch.empty(n, dtype=torch.int32, device=mem.arena.device)
    _check(_lib.evk_visits_read(mem.handle, stage, first, n, _dev(out), _stream_ptr(stream)), "evk_visits_read")
    return out


def evk_visits_write(mem: EvkMem, visits, device=None, stream=None) -> None:
    """Restore per-stage update counts: visits is [n_stages][size] (numpy uint32 or int32 tensor)."""
    import numpy as _np
    dev = device or mem.arena.device
    for s in range(mem.n_stages):
        row = visits[s]
        t = row if isinstance(row, torch.Tensor) else torch.from_numpy(_np.ascontiguousarray(row).view(_np.int32))
        t = t.to(dev).contiguous()
        _check(_lib.evk_visits_write(mem.handle, s, 0, t.numel(), _dev(t, torch.int32, "visits"),
                                     _stream_ptr(stream)), "evk_visits_write")


def evk_mem_inject_stall(mem: EvkMem) -> None:
    """Test aid: the next tensor-path retrieve lets a bounded wait run out (EVK_ERR_DEVICE_TIMEOUT)."""
    _check(_lib.evk_mem_inject_stall(mem.handle), "evk_mem_inject_stall")


def evk_retrieve_local(mem: EvkMem, queries: torch.Tensor, stage: int, k1: int, id_offset: int, stream=None):
    """Phase 1 on one row shard: (global ids, sims, Q_stage) per candidate, each [B][k1]."""
    B, dev = queries.shape[0], queries.device
    gids = torch.empty((B, k1), dtype=torch.int32, device=dev)
    sims = torch.empty((B, k1), dtype=torch.float32, device=dev)
    qs = torch.empty((B, k1), dtype=torch.float32, device=dev)
    ws = mem.workspace("retrieve_local", int(_lib.evk_retrieve_local_workspace_bytes(mem.handle, B, k1)))
    _check(_lib.evk_retrieve_local(mem.handle, _dev(queries, None, "queries"), _emb_dtype(queries), B, stage, k1,
                                   int(id_offset), _dev(gids), _dev(sims), _dev(qs), _dev(ws), ws.numel(),
                                   _stream_ptr(stream)), "evk_retrieve_local")
    return gids, sims, qs


def evk_merge_shards(gids: torch.Tensor, sims: torch.Tensor, qs: torch.Tensor, k2: int, w: float,
                     return_pool: bool = False, stream=None):
    """Merge gathered shard pools [G][B][k1] (ascending id ranges) and run phase 2."""
    G, B, k1 = gids.shape
    dev = gids.device
    ids = torch.empty((B, k2), dtype=torch.int32, device=dev)
    scores = torch.empty((B, k2), dtype=torch.float32, device=dev)
    pool_g = torch.empty((B, k1), dtype=torch.int32, device=dev) if return_pool else None
    pool_s = torch.empty((B, k1), dtype=torch.float32, device=dev) if return_pool else None
    _check(_lib.evk_merge_shards(_dev(gids, torch.int32, "gids"), _dev(sims, torch.float32, "sims"),
                                 _dev(qs, torch.float32, "qs"), G, B, k1, k2, float(w), _dev(ids), _dev(scores),
                                 _dev(pool_g), _dev(pool_s), _stream_ptr(stream)), "evk_merge_shards")
    if return_pool:
        return ids, scores, pool_g, pool_s
    return ids, scores
