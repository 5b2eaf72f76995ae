"""Thin ctypes binding of the C ABI in include/ccr.h (same names, argument marshalling only).

Every step of the join runs in the CUDA library; torch is used here only for device memory, streams
and pointer/size bookkeeping.  There is no CPU fallback: if the shared object is missing or no CUDA
device is present, calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# CCR_LIB_OVERRIDE names another build of the same library (kernel A/B comparisons); unset = the in-tree build
LIB_PATH = os.environ.get("CCR_LIB_OVERRIDE") or os.path.join(_HERE, "libccr.so")

CCR_OK = 0
CCR_ERR_INVALID_ARG = 1
CCR_ERR_UNSUPPORTED = 2
CCR_ERR_OOM = 3
CCR_ERR_CUDA = 4
CCR_ERR_BAD_HANDLE = 5
CCR_ERR_VALIDATION = 6
CCR_ERR_DEVICE_WAIT = 7
CCR_ERR_BOUNDS = 8

CCR_F16 = 0
CCR_F32 = 1

CCR_FLAG_FORCE_SMEM = 1 << 0
CCR_FLAG_FORCE_GLOBAL = 1 << 1
CCR_FLAG_CANDS_SORTED = 1 << 2
CCR_FLAG_VALIDATE = 1 << 3
CCR_FLAG_FIRST_DEGREE_ONLY = 1 << 4
CCR_FLAG_FORCE_SAMPLED = 1 << 5
CCR_FLAG_STATIC_SPLIT = 1 << 6
CCR_FLAG_TWO_PHASE = 1 << 7
CCR_FLAG_COSINE = 1 << 8
CCR_FLAG_WARP_SPECIALISED = 1 << 9
CCR_FLAG_NO_REBALANCE = 1 << 10
CCR_FLAG_NO_OVERLAP = 1 << 11
CCR_FLAG_WARP_SEARCH = 1 << 12

EXPORTS = (
    "ccr_docstore_create", "ccr_docstore_upload", "ccr_docstore_upsert", "ccr_docstore_free", "ccr_out_row_bytes", "ccr_join_batch",
    "ccr_compact_valid", "ccr_join_batch_padded", "ccr_join_batch_ex", "ccr_docstore_set_cosine",
    "ccr_workspace_create", "ccr_workspace_free", "ccr_workspace_outputs", "ccr_join_batch_host", "ccr_docstore_device_status",
    "ccr_docstore_set_tuning", "ccr_docstore_launch_count", "ccr_status_str", "ccr_version",
    "ccr_static_payload_capacity", "ccr_join_payload_static", "ccr_docstore_selftest_wait",
    "ccr_sort_edges", "ccr_idindex_create", "ccr_idindex_free", "ccr_resolve_ids",
    "ccr_debug_bounds_enabled", "ccr_debug_shrink_outputs",
)


class ccr_cosine_spec(ctypes.Structure):
    _fields_ = [("item_first", ctypes.c_int32), ("dim", ctypes.c_int32), ("n_chunks", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


class ccr_join_io(ctypes.Structure):
    _fields_ = [("struct_bytes", ctypes.c_uint32), ("n_req", ctypes.c_int32), ("total_cands", ctypes.c_int64),
                ("max_edge_len", ctypes.c_int64), ("n_max", ctypes.c_int64), ("edge_keys", ctypes.c_void_p),
                ("edge_feats", ctypes.c_void_p), ("edge_offsets", ctypes.c_void_p), ("cand_idx", ctypes.c_void_p),
                ("cand_offsets", ctypes.c_void_p), ("req_feats", ctypes.c_void_p), ("member_emb", ctypes.c_void_p),
                ("out_rows", ctypes.c_void_p), ("out_mask", ctypes.c_void_p)]


class ccr_docstore_desc(ctypes.Structure):
    _fields_ = [
        ("n_docs", ctypes.c_int64),
        ("doc_dim", ctypes.c_int32), ("doc_dtype", ctypes.c_int32),
        ("edge_dim", ctypes.c_int32), ("edge_dtype", ctypes.c_int32),
        ("req_dim", ctypes.c_int32), ("req_dtype", ctypes.c_int32),
        ("max_actors", ctypes.c_int32), ("device", ctypes.c_int32),
        ("reduce_sum_mask", ctypes.c_uint64),
    ]


class ccr_tuning(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "tile_cands", "key_capacity", "ws_streamers", "ws_resolvers", "blocks_per_sm")]


class CcrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        msg = lib().ccr_status_str(self.status).decode() if _lib is not None else "?"
        super().__init__("%s: %s (status %d)" % (where, msg, self.status))


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built in-tree by `paper_2609_22441_b200.build`); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "CUDA library %s is not built; run `python -m paper_2609_22441_b200.build` "
            "(there is no CPU fallback)" % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u32, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32, ctypes.c_uint64
    L.ccr_docstore_create.restype = ctypes.c_int
    L.ccr_docstore_create.argtypes = [ctypes.POINTER(ccr_docstore_desc), ctypes.POINTER(vp)]
    L.ccr_docstore_upload.restype = ctypes.c_int
    L.ccr_docstore_upload.argtypes = [vp, i64, i64, vp, vp, vp, vp, ctypes.c_int, vp]
    L.ccr_docstore_free.restype = ctypes.c_int
    L.ccr_docstore_free.argtypes = [vp]
    L.ccr_out_row_bytes.restype = ctypes.c_size_t
    L.ccr_out_row_bytes.argtypes = [vp, u32]
    L.ccr_join_batch.restype = ctypes.c_int
    L.ccr_join_batch.argtypes = [vp, i32, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, u32, vp]
    L.ccr_workspace_create.restype = ctypes.c_int
    L.ccr_workspace_create.argtypes = [vp, i32, i64, i64, ctypes.POINTER(vp)]
    L.ccr_workspace_free.restype = ctypes.c_int
    L.ccr_workspace_free.argtypes = [vp]
    L.ccr_docstore_upsert.restype = ctypes.c_int
    L.ccr_docstore_upsert.argtypes = [vp, i64, vp, vp, vp, vp, vp, vp]
    L.ccr_join_batch_ex.restype = ctypes.c_int
    L.ccr_join_batch_ex.argtypes = [vp, ctypes.POINTER(ccr_join_io), u32, vp]
    L.ccr_docstore_set_cosine.restype = ctypes.c_int
    L.ccr_docstore_set_cosine.argtypes = [vp, ctypes.POINTER(ccr_cosine_spec)]
    L.ccr_compact_valid.restype = ctypes.c_int
    L.ccr_compact_valid.argtypes = [vp, i32, i64, vp, vp, vp, vp, vp, vp]
    L.ccr_join_batch_padded.restype = ctypes.c_int
    L.ccr_join_batch_padded.argtypes = [vp, i32, i64, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, u32, vp]
    L.ccr_workspace_outputs.restype = ctypes.c_int
    L.ccr_workspace_outputs.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    L.ccr_join_batch_host.restype = ctypes.c_int
    L.ccr_join_batch_host.argtypes = [vp, vp, i32, i64, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, u32, vp]
    L.ccr_static_payload_capacity.restype = ctypes.c_size_t
    L.ccr_static_payload_capacity.argtypes = []
    L.ccr_join_payload_static.restype = ctypes.c_int
    L.ccr_join_payload_static.argtypes = [vp, i32, i64, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, u32, vp]
    L.ccr_idindex_create.restype = ctypes.c_int
    L.ccr_idindex_create.argtypes = [i32, i64, vp, vp, ctypes.c_int, ctypes.POINTER(vp)]
    L.ccr_idindex_free.restype = ctypes.c_int
    L.ccr_idindex_free.argtypes = [vp]
    L.ccr_resolve_ids.restype = ctypes.c_int
    L.ccr_resolve_ids.argtypes = [vp, i64, vp, vp, vp]
    L.ccr_sort_edges.restype = ctypes.c_int
    L.ccr_sort_edges.argtypes = [vp, i32, i64, vp, vp, vp, vp, vp, vp, vp]
    L.ccr_docstore_selftest_wait.restype = ctypes.c_int
    L.ccr_docstore_selftest_wait.argtypes = [vp, vp]
    L.ccr_docstore_device_status.restype = ctypes.c_int
    L.ccr_docstore_device_status.argtypes = [vp, vp]
    L.ccr_docstore_set_tuning.restype = ctypes.c_int
    L.ccr_docstore_set_tuning.argtypes = [vp, ctypes.POINTER(ccr_tuning)]
    L.ccr_docstore_launch_count.restype = i64
    L.ccr_docstore_launch_count.argtypes = [vp]
    L.ccr_status_str.restype = ctypes.c_char_p
    L.ccr_status_str.argtypes = [ctypes.c_int]
    L.ccr_version.restype = ctypes.c_int
    L.ccr_version.argtypes = []
    L.ccr_debug_bounds_enabled.restype = ctypes.c_int
    L.ccr_debug_bounds_enabled.argtypes = []
    L.ccr_debug_shrink_outputs.restype = ctypes.c_int
    L.ccr_debug_shrink_outputs.argtypes = [vp, i64]
    _lib = L
    return L


def _check(status: int, where: str) -> None:
    if status != CCR_OK:
        raise CcrError(status, where)


def _dtype_code(dt) -> int:
    dt = np.dtype(dt)
    if dt == np.float16:
        return CCR_F16
    if dt == np.float32:
        return CCR_F32
    raise ValueError("feature dtype must be float16 or float32")


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor (device or host) or numpy array; None stays NULL."""
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        if not x.is_contiguous():
            raise ValueError("tensors passed to the library must be contiguous")
        return x.data_ptr()
    if isinstance(x, np.ndarray):
        if not x.flags["C_CONTIGUOUS"]:
            raise ValueError("arrays passed to the library must be contiguous")
        return x.ctypes.data
    raise TypeError(type(x))


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return int(stream) or None


class Docstore:
    """ccr_docstore handle: the GPU-resident document-feature store of one shard."""

    def __init__(self, n_docs: int, doc_dim: int, doc_dtype, edge_dim: int, edge_dtype=np.float16,
                 req_dim: int = 0, req_dtype=np.float32, max_actors: int = 0, reduce_sum_mask: int = 0,
                 device: int = 0):
        self._h = ctypes.c_void_p()
        self.desc = ccr_docstore_desc(
            int(n_docs), int(doc_dim), _dtype_code(doc_dtype), int(edge_dim), _dtype_code(edge_dtype),
            int(req_dim), _dtype_code(req_dtype), int(max_actors), int(device),
            int(reduce_sum_mask) & (2**64 - 1))
        self.device = int(device)
        _check(lib().ccr_docstore_create(ctypes.byref(self.desc), ctypes.byref(self._h)), "ccr_docstore_create")

    @property
    def handle(self) -> ctypes.c_void_p:
        return self._h

    def upload(self, first_doc: int, doc_feats=None, author_ids=None, actor_ids=None, actor_types=None,
               stream=None) -> None:
        """ccr_docstore_upload: rows [first_doc, first_doc + n); sources all on the host or all on the device."""
        given = [x for x in (doc_feats, author_ids, actor_ids, actor_types) if x is not None]
        if not given:
            return
        n = int(given[0].shape[0])
        on_dev = [isinstance(x, torch.Tensor) and x.is_cuda for x in given]
        if any(on_dev) != all(on_dev):
            raise ValueError("upload sources must be all on the host or all on the device")
        _check(lib().ccr_docstore_upload(self._h, int(first_doc), n, _ptr(doc_feats), _ptr(author_ids),
                                         _ptr(actor_ids), _ptr(actor_types), 1 if all(on_dev) else 0,
                                         _stream_ptr(stream)), "ccr_docstore_upload")

    def upsert(self, positions, doc_feats=None, author_ids=None, actor_ids=None, actor_types=None, stream=None) -> None:
        """ccr_docstore_upsert: batch row i replaces row positions[i]; every argument is a device tensor."""
        _check(lib().ccr_docstore_upsert(self._h, int(positions.shape[0]), _ptr(positions), _ptr(doc_feats),
                                         _ptr(author_ids), _ptr(actor_ids), _ptr(actor_types), _stream_ptr(stream)),
               "ccr_docstore_upsert")

    def set_cosine(self, item_first: int, dim: int, n_chunks: int) -> None:
        """ccr_docstore_set_cosine: where the item embedding sits in a document row (n_chunks == 0 switches off)."""
        if n_chunks == 0:
            _check(lib().ccr_docstore_set_cosine(self._h, None), "ccr_docstore_set_cosine")
            return
        spec = ccr_cosine_spec(int(item_first), int(dim), int(n_chunks), 0)
        _check(lib().ccr_docstore_set_cosine(self._h, ctypes.byref(spec)), "ccr_docstore_set_cosine")

    def out_row_bytes(self, flags: int = 0) -> int:
        return int(lib().ccr_out_row_bytes(self._h, int(flags)))

    def set_tuning(self, tile_cands: int = 0, key_capacity: int = 0, ws_streamers: int = 0, ws_resolvers: int = 0,
                   blocks_per_sm: int = 0) -> None:
        t = ccr_tuning(int(tile_cands), int(key_capacity), int(ws_streamers), int(ws_resolvers), int(blocks_per_sm))
        _check(lib().ccr_docstore_set_tuning(self._h, ctypes.byref(t)), "ccr_docstore_set_tuning")

    def launch_count(self) -> int:
        return int(lib().ccr_docstore_launch_count(self._h))

    def selftest_wait(self, stream=None) -> None:
        _check(lib().ccr_docstore_selftest_wait(self._h, _stream_ptr(stream)), "ccr_docstore_selftest_wait")

    def device_status(self, stream=None) -> int:
        return int(lib().ccr_docstore_device_status(self._h, _stream_ptr(stream)))

    def free(self) -> None:
        if self._h:
            _check(lib().ccr_docstore_free(self._h), "ccr_docstore_free")
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            if self._h:
                lib().ccr_docstore_free(self._h)
                self._h = ctypes.c_void_p()
        except Exception:
            pass


def ccr_join_batch(store: Docstore, n_req: int, total_cands: int, max_edge_len: int,
                   edge_keys, edge_feats, edge_offsets, cand_idx, cand_offsets, req_feats,
                   out_rows, out_mask, flags: int = 0, stream=None) -> int:
    """Raw call, device tensors in, status out (raises on error)."""
    st = lib().ccr_join_batch(store.handle, int(n_req), int(total_cands), int(max_edge_len), _ptr(edge_keys),
                              _ptr(edge_feats), _ptr(edge_offsets), _ptr(cand_idx), _ptr(cand_offsets),
                              _ptr(req_feats), _ptr(out_rows), _ptr(out_mask), int(flags), _stream_ptr(stream))
    _check(st, "ccr_join_batch")
    return st


def ccr_join_batch_ex(store: Docstore, n_req: int, total_cands: int, max_edge_len: int, edge_keys, edge_feats,
                      edge_offsets, cand_idx, cand_offsets, req_feats, out_rows, out_mask, flags: int = 0, stream=None,
                      n_max: int = 0, member_emb=None) -> int:
    """Raw call: the join with every optional input (padded layout, member embeddings for the cosine section)."""
    p = _ptr
    io = ccr_join_io(ctypes.sizeof(ccr_join_io), int(n_req), int(total_cands), int(max_edge_len), int(n_max),
                     p(edge_keys), p(edge_feats), p(edge_offsets), p(cand_idx), p(cand_offsets), p(req_feats),
                     p(member_emb), p(out_rows), p(out_mask))
    st = lib().ccr_join_batch_ex(store.handle, ctypes.byref(io), int(flags), _stream_ptr(stream))
    _check(st, "ccr_join_batch_ex")
    return st


def ccr_compact_valid(store: Docstore, n_req: int, total_cands: int, cand_idx, cand_offsets, idx_out, offsets_out,
                      src_out=None, stream=None) -> int:
    """Raw call: per-request stable compaction of the valid positions (device tensors in and out)."""
    st = lib().ccr_compact_valid(store.handle, int(n_req), int(total_cands), _ptr(cand_idx), _ptr(cand_offsets), _ptr(idx_out),
                                 _ptr(offsets_out), _ptr(src_out), _stream_ptr(stream))
    _check(st, "ccr_compact_valid")
    return st


def ccr_join_batch_padded(store: Docstore, n_req: int, total_cands: int, max_edge_len: int, n_max: int,
                          edge_keys, edge_feats, edge_offsets, cand_idx, cand_offsets, req_feats,
                          out_rows, out_mask, flags: int = 0, stream=None) -> int:
    """Raw call: the join written straight into the padded [n_req, n_max] layout."""
    st = lib().ccr_join_batch_padded(store.handle, int(n_req), int(total_cands), int(max_edge_len), int(n_max),
                                     _ptr(edge_keys), _ptr(edge_feats), _ptr(edge_offsets), _ptr(cand_idx),
                                     _ptr(cand_offsets), _ptr(req_feats), _ptr(out_rows), _ptr(out_mask), int(flags),
                                     _stream_ptr(stream))
    _check(st, "ccr_join_batch_padded")
    return st


class DeviceBatch:
    """A ragged batch resident on the device (torch tensors), plus the host scalars the call needs."""

    def __init__(self, batch, device: int = 0):
        dev = torch.device("cuda", device)
        self.n_req = int(batch.n_req)
        self.total_cands = int(batch.total_cands)
        self.max_edge_len = int(batch.max_edge_len)
        self.total_edges = int(len(batch.edge_keys))
        self.n_max_cands = int(np.diff(np.asarray(batch.cand_offsets)).max()) if self.n_req > 0 else 0

        def up(a):
            if a is None:
                return None
            t = torch.from_numpy(np.ascontiguousarray(a))
            return t.to(dev) if t.numel() else torch.empty(t.shape, dtype=t.dtype, device=dev)

        self.edge_keys = up(batch.edge_keys)
        self.edge_feats = up(batch.edge_feats)
        self.edge_offsets = up(batch.edge_offsets)
        self.cand_idx = up(batch.cand_idx)
        self.cand_offsets = up(batch.cand_offsets)
        self.req_feats = up(batch.req_feats)


def join_batch(store: Docstore, db: DeviceBatch, flags: int = 0, out_rows: Optional[torch.Tensor] = None,
               out_mask: Optional[torch.Tensor] = None, stream=None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Allocate outputs if needed (torch, outside the library) and call ccr_join_batch."""
    out_b = store.out_row_bytes(flags)
    dev = torch.device("cuda", store.device)
    if out_rows is None:
        out_rows = torch.empty((db.total_cands, out_b), dtype=torch.uint8, device=dev)
    if out_mask is None:
        out_mask = torch.empty((db.total_cands,), dtype=torch.uint8, device=dev)
    ccr_join_batch(store, db.n_req, db.total_cands, db.max_edge_len, db.edge_keys, db.edge_feats, db.edge_offsets,
                   db.cand_idx, db.cand_offsets, db.req_feats, out_rows, out_mask, flags, stream)
    return out_rows, out_mask


def join_batch_padded(store: Docstore, db: DeviceBatch, n_max: Optional[int] = None, flags: int = 0, stream=None):
    """Section 6.3.1 batching and padding in two calls: ccr_compact_valid, then ccr_join_batch_padded over the
    compacted candidates.  Returns (T uint8[n_req, n_max, out_b], mask uint8[n_req, n_max],
    offsets int64[n_req + 1] of the compacted batch, src int32[total_cands] flat input index per kept
    candidate; entries behind offsets[n_req] are unwritten).  n_max defaults to the longest request of the
    input, an upper bound of the longest compacted one, known on the host without a synchronisation."""
    dev = torch.device("cuda", store.device)
    if n_max is None:
        n_max = max(1, int(db.n_max_cands))
    out_b = store.out_row_bytes(flags)
    idx = torch.empty((db.total_cands,), dtype=torch.int32, device=dev)
    src = torch.empty((db.total_cands,), dtype=torch.int32, device=dev)
    offs = torch.empty((db.n_req + 1,), dtype=torch.int64, device=dev)
    T = torch.empty((db.n_req, n_max, out_b), dtype=torch.uint8, device=dev)
    M = torch.empty((db.n_req, n_max), dtype=torch.uint8, device=dev)
    ccr_compact_valid(store, db.n_req, db.total_cands, db.cand_idx, db.cand_offsets, idx, offs, src, stream)
    ccr_join_batch_padded(store, db.n_req, db.total_cands, db.max_edge_len, n_max, db.edge_keys, db.edge_feats,
                          db.edge_offsets, idx, offs, db.req_feats, T, M, flags, stream)
    return T, M, offs, src


class Workspace:
    """ccr_workspace handle: device staging for ccr_join_batch_host."""

    def __init__(self, store: Docstore, max_req: int, max_cands: int, max_edges: int):
        self._h = ctypes.c_void_p()
        self.store = store
        _check(lib().ccr_workspace_create(store.handle, int(max_req), int(max_cands), int(max_edges),
                                          ctypes.byref(self._h)), "ccr_workspace_create")

    @property
    def handle(self):
        return self._h

    def outputs(self):
        """ccr_workspace_outputs: device addresses (rows, mask) of the workspace's output buffers."""
        rows, mask = ctypes.c_void_p(), ctypes.c_void_p()
        _check(lib().ccr_workspace_outputs(self._h, ctypes.byref(rows), ctypes.byref(mask)), "ccr_workspace_outputs")
        return rows.value, mask.value

    def free(self) -> None:
        if self._h:
            _check(lib().ccr_workspace_free(self._h), "ccr_workspace_free")
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def ccr_join_batch_host(store: Docstore, ws: Workspace, n_req: int, total_cands: int, max_edge_len: int,
                        total_edges: int, edge_keys, edge_feats, edge_offsets, cand_idx, cand_offsets, req_feats,
                        out_rows, out_mask, flags: int = 0, stream=None) -> int:
    """Raw call with HOST buffers (numpy arrays or pinned CPU tensors); copies are inside the call."""
    st = lib().ccr_join_batch_host(store.handle, ws.handle, int(n_req), int(total_cands), int(max_edge_len),
                                   int(total_edges), _ptr(edge_keys), _ptr(edge_feats), _ptr(edge_offsets),
                                   _ptr(cand_idx), _ptr(cand_offsets), _ptr(req_feats), _ptr(out_rows),
                                   _ptr(out_mask), int(flags), _stream_ptr(stream))
    _check(st, "ccr_join_batch_host")
    return st


def ccr_join_payload_static(store: Docstore, n_req: int, total_cands: int, max_edge_len: int, total_edges: int,
                            edge_keys, edge_feats, edge_offsets, cand_idx, cand_offsets, req_feats,
                            out_rows, out_mask, flags: int = 0, stream=None) -> int:
    """Raw call of the entry for callers that must not allocate: HOST payload (numpy arrays or pinned CPU
    tensors), DEVICE outputs; the library stages the payload in its fixed device block."""
    st = lib().ccr_join_payload_static(store.handle, int(n_req), int(total_cands), int(max_edge_len),
                                       int(total_edges), _ptr(edge_keys), _ptr(edge_feats), _ptr(edge_offsets),
                                       _ptr(cand_idx), _ptr(cand_offsets), _ptr(req_feats), _ptr(out_rows),
                                       _ptr(out_mask), int(flags), _stream_ptr(stream))
    _check(st, "ccr_join_payload_static")
    return st


class IdIndex:
    """ccr_idindex handle: sorted document ids (+ optional positions) with sampled search levels on the device."""

    def __init__(self, sorted_ids, positions=None, device: int = 0):
        self._h = ctypes.c_void_p()
        on_dev = isinstance(sorted_ids, torch.Tensor) and sorted_ids.is_cuda
        if positions is not None and (isinstance(positions, torch.Tensor) and positions.is_cuda) != on_dev:
            raise ValueError("ids and positions must be on the same side")
        self.n_ids = int(sorted_ids.shape[0])
        self.device = int(device)
        _check(lib().ccr_idindex_create(int(device), self.n_ids, _ptr(sorted_ids), _ptr(positions), 1 if on_dev else 0,
                                        ctypes.byref(self._h)), "ccr_idindex_create")

    @property
    def handle(self):
        return self._h

    def resolve(self, query_ids: torch.Tensor, out_pos: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """ccr_resolve_ids on a device tensor of int64 queries; returns int32 positions (-1 = not indexed)."""
        if out_pos is None:
            out_pos = torch.empty(query_ids.shape, dtype=torch.int32, device=query_ids.device)
        _check(lib().ccr_resolve_ids(self._h, int(query_ids.numel()), _ptr(query_ids), _ptr(out_pos), _stream_ptr(stream)),
               "ccr_resolve_ids")
        return out_pos

    def free(self) -> None:
        if self._h:
            _check(lib().ccr_idindex_free(self._h), "ccr_idindex_free")
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def ccr_sort_edges(store: Docstore, n_req: int, max_edge_len: int, edge_keys_in, edge_feats_in, edge_offsets,
                   edge_keys_out, edge_feats_out, perm_out=None, stream=None) -> int:
    """Raw call: per-request sort of (key, row) records by key on the device (device tensors in and out)."""
    st = lib().ccr_sort_edges(store.handle, int(n_req), int(max_edge_len), _ptr(edge_keys_in), _ptr(edge_feats_in),
                              _ptr(edge_offsets), _ptr(edge_keys_out), _ptr(edge_feats_out), _ptr(perm_out),
                              _stream_ptr(stream))
    _check(st, "ccr_sort_edges")
    return st


def store_from_workload(wl, device: int = 0, upload_doc_feats: bool = True) -> Docstore:
    """Create a store with the workload's schema and upload its arrays (host sources)."""
    s, b = wl.store, wl.batch
    st = Docstore(s.n_docs, s.doc_dim, s.doc_dtype, b.edge_dim, b.edge_dtype, b.req_dim, b.req_dtype,
                  s.max_actors, s.reduce_sum_mask, device)
    st.upload(0, s.doc_feats if upload_doc_feats else None, s.author_ids, s.actor_ids, s.actor_types)
    torch.cuda.synchronize(device)
    return st


def store_from_generated(wl, device: int = 0, keep_rows_of=None, keep_all: bool = False):
    """Create the store of a workload whose doc features are generated on the device in chunks
    (`workloads.doc_feats_chunk_device`): ids are uploaded from the host, features chunk by chunk from device
    memory.  Returns (store, kept, full): `kept` = {"idx", "rows"} host copies of the rows of the doc
    positions in `keep_rows_of` (taken from the generator's output before the library sees it), `full` = the
    whole generated matrix as a device tensor when keep_all is set."""
    from . import workloads as W

    s, b = wl.store, wl.batch
    store = Docstore(s.n_docs, s.doc_dim, s.doc_dtype, b.edge_dim, b.edge_dtype, b.req_dim, b.req_dtype,
                     s.max_actors, s.reduce_sum_mask, device)
    store.upload(0, None, s.author_ids, s.actor_ids, s.actor_types)
    want = None if keep_rows_of is None else np.unique(np.asarray(keep_rows_of, dtype=np.int64))
    kept_idx, kept_rows, full = [], [], []
    step = W.DOC_DEVICE_CHUNK
    dev = torch.device("cuda", device)
    for first in range(0, s.n_docs, step):
        n = min(step, s.n_docs - first)
        chunk = W.doc_feats_chunk_device(wl.seed, first, n, s.doc_dim, dev)
        store.upload(first, chunk)
        if want is not None:
            lo, hi = np.searchsorted(want, [first, first + n])
            if hi > lo:
                local = torch.from_numpy(want[lo:hi] - first).to(dev)
                kept_idx.append(want[lo:hi])
                kept_rows.append(chunk.index_select(0, local).cpu().numpy())
        if keep_all:
            full.append(chunk)
        torch.cuda.synchronize(device)
    kept = {}
    if want is not None and kept_idx:
        kept = {"idx": np.concatenate(kept_idx), "rows": np.concatenate(kept_rows)}
    return store, kept, (torch.cat(full) if keep_all else None)
