"""ctypes binding of libbsr.so: the same calls as include/bsr.h, argument marshalling only.

No step of the restore path runs here; every function forwards to the CUDA library.  Importing
this module loads the library and raises if it has not been built (python -m
paper_2608_17826_b200.build): there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# BSR_LIBRARY selects another build of the same source (the tests' small-stage build of the install
# kernel, see build.py); it must exist, nothing is built or substituted for it.
LIB_PATH = os.environ.get("BSR_LIBRARY") or os.path.join(_HERE, "libbsr.so")

BSR_OK, BSR_ERR_INVALID, BSR_ERR_MISSING, BSR_ERR_CHECKSUM, BSR_ERR_TIMEOUT = 0, -1, -2, -3, -4
BSR_ERR_TRANSFER, BSR_ERR_NOMEM, BSR_ERR_ALIGN, BSR_ERR_STATE, BSR_ERR_CUDA = -5, -6, -7, -8, -9
BSR_LOC_HOST, BSR_LOC_DEVICE = 0, 1
BSR_INSTALL_AUTO, BSR_INSTALL_VECTOR, BSR_INSTALL_BULK = 0, 1, 2
BSR_SCRUB = 1
BSR_INJECT_NONE, BSR_INJECT_CORRUPT_SLOT, BSR_INJECT_FILL_ERROR, BSR_INJECT_FILL_STALL = 0, 1, 2, 3
BSR_INJECT_KERNEL_WAIT = 4
BSR_MAX_GROUPS, BSR_MAX_RANKS, BSR_CHUNK_TOKENS = 8, 8, 256

ERROR_NAMES = {0: "BSR_OK", -1: "BSR_ERR_INVALID", -2: "BSR_ERR_MISSING", -3: "BSR_ERR_CHECKSUM",
               -4: "BSR_ERR_TIMEOUT", -5: "BSR_ERR_TRANSFER", -6: "BSR_ERR_NOMEM",
               -7: "BSR_ERR_ALIGN", -8: "BSR_ERR_STATE", -9: "BSR_ERR_CUDA"}

EXPORTS = [
    "bsr_ctx_create", "bsr_ctx_destroy", "bsr_last_error", "bsr_register", "bsr_chunk_bytes",
    "bsr_tier_put", "bsr_tier_remove", "bsr_tier_checksums", "bsr_probe", "bsr_req_create",
    "bsr_req_release", "bsr_restore", "bsr_commit", "bsr_invalidate", "bsr_req_bitmap",
    "bsr_req_checksums", "bsr_get_stats", "bsr_reset_stats", "bsr_test_inject",
    "bsr_probe_keys_noalloc", "bsr_tier_put_at", "bsr_tier_remove_at", "bsr_tier_set_available",
    "bsr_probe_request", "bsr_req_bind", "bsr_request_done", "bsr_request_is_force_local",
    "bsr_get_trace", "bsr_tier_set_fetch", "bsr_restore_async", "bsr_restore_wait",
    "bsr_req_invalid_blocks", "bsr_install_kernel_in_use", "bsr_restore_calibrate", "bsr_numa_of_pci",
    "bsr_plan_spans", "bsr_plan_pieces",
]
# int fn(void *user, uint32 tier, uint32 rank, uint64 key, uint64 offset, uint64 len, void *dst)
BSR_FETCH_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint64, C.c_uint64,
                           C.c_uint64, C.c_void_p)
BSR_MAX_TIERS = 4
BSR_CAL_FILL, BSR_CAL_FILL_H2D = 1, 2
BSR_NUMA_AUTO, BSR_NUMA_OFF, BSR_NUMA_ALWAYS = 0, 1, 2
BSR_NOALLOC_MAX_CHUNKS = 8192


class bsr_config(C.Structure):
    _fields_ = [("window_chunks", C.c_uint32), ("n_ranks", C.c_uint32), ("chunk_tokens", C.c_uint32),
                ("load_concurrency", C.c_uint32), ("dev_staging_depth", C.c_uint32),
                ("timeout_ms", C.c_uint32), ("slot_align", C.c_uint32), ("device", C.c_int32),
                ("reg_id", C.c_uint64), ("install_variant", C.c_uint32), ("time_kernels", C.c_uint32),
                ("direct_install", C.c_uint32), ("budget_slots", C.c_uint32),
                ("install_batch", C.c_uint32), ("numa_bind", C.c_uint32)]


class bsr_group_desc(C.Structure):
    _fields_ = [("block_tokens", C.c_uint32), ("num_phys_blocks", C.c_uint32)]


class bsr_tensor_desc(C.Structure):
    _fields_ = [("group", C.c_uint32), ("bytes_per_token", C.c_uint32), ("dev_base", C.c_void_p)]


class bsr_stats(C.Structure):
    _fields_ = [("peak_staging_bytes", C.c_uint64 * BSR_MAX_RANKS),
                ("ring_bytes_allocated", C.c_uint64 * BSR_MAX_RANKS),
                ("bytes_filled", C.c_uint64 * BSR_MAX_RANKS),
                ("bytes_h2d", C.c_uint64 * BSR_MAX_RANKS),
                ("bytes_installed", C.c_uint64 * BSR_MAX_RANKS),
                ("slot_bytes", C.c_uint64), ("dev_aux_bytes", C.c_uint64), ("windows", C.c_uint64),
                ("tier_bytes_read_by_probe", C.c_uint64), ("kernel_launches", C.c_uint64),
                ("h2d_copies", C.c_uint64), ("install_launches", C.c_uint64),
                ("bytes_restored_by_tier", C.c_uint64 * 4),
                ("install_kernel_ms", C.c_double), ("last_restore_ms", C.c_double),
                ("install_descriptors", C.c_uint64), ("fill_numa_node", C.c_int64),
                ("install_span_ms", C.c_double)]


class bsr_trace_rec(C.Structure):
    _fields_ = [("chunk", C.c_uint32), ("rank", C.c_uint32), ("slot", C.c_uint32), ("reserved", C.c_uint32),
                ("t_admit_ns", C.c_uint64), ("t_filled_ns", C.c_uint64), ("t_submit_ns", C.c_uint64),
                ("t_done_ns", C.c_uint64)]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH) and not os.environ.get("BSR_LIBRARY"):
        try:  # a fresh checkout: compile once with nvcc, in-tree
            from . import build as _build
            _build.build()
        except Exception as exc:  # noqa: BLE001 - reported below, never hidden behind a fallback
            raise ImportError(f"{LIB_PATH} is missing and could not be built: {exc}") from exc
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2608_17826_b200.build` "
            "(needs nvcc). The BSR path has no CPU fallback.")
    lib = C.CDLL(LIB_PATH)
    vp, u32, u64, i32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int
    sig = {
        "bsr_ctx_create": [C.POINTER(bsr_config), C.POINTER(vp)],
        "bsr_ctx_destroy": [vp],
        "bsr_register": [vp, u32, C.POINTER(bsr_group_desc), u32, C.POINTER(bsr_tensor_desc), u32],
        "bsr_chunk_bytes": [vp, C.POINTER(u64), C.POINTER(u64)],
        "bsr_tier_put": [vp, u32, u64, vp, C.c_size_t, vp, i32],
        "bsr_tier_remove": [vp, u32, u64],
        "bsr_tier_checksums": [vp, u32, u64, vp],
        "bsr_probe": [vp, vp, C.c_size_t, i32, u64, vp, vp, C.POINTER(u32)],
        "bsr_req_create": [vp, vp, u32, C.POINTER(vp), C.POINTER(vp)],
        "bsr_req_release": [vp, vp],
        "bsr_restore": [vp, vp, vp],
        "bsr_commit": [vp, vp, C.POINTER(u32)],
        "bsr_invalidate": [vp, vp, C.c_uint],
        "bsr_req_bitmap": [vp, vp, vp, C.c_size_t],
        "bsr_req_checksums": [vp, vp, vp, C.c_size_t],
        "bsr_get_stats": [vp, C.POINTER(bsr_stats)],
        "bsr_reset_stats": [vp],
        "bsr_test_inject": [vp, i32, u32, u32, u32, u64],
        "bsr_probe_keys_noalloc": [i32, vp, C.c_size_t, u64, u64, vp, vp],
        "bsr_tier_put_at": [vp, u32, u32, u64, vp, C.c_size_t, vp, i32],
        "bsr_tier_remove_at": [vp, u32, u32, u64],
        "bsr_tier_set_available": [vp, u32, i32],
        "bsr_probe_request": [vp, u64, vp, C.c_size_t, i32, u64, vp, vp, C.POINTER(u32), C.POINTER(i32)],
        "bsr_req_bind": [vp, vp, u64, u32],
        "bsr_request_done": [vp, u64],
        "bsr_request_is_force_local": [vp, u64, C.POINTER(i32)],
        "bsr_get_trace": [vp, vp, C.c_size_t, C.POINTER(C.c_size_t)],
        "bsr_tier_set_fetch": [vp, u32, BSR_FETCH_FN, vp],
        "bsr_restore_async": [vp, vp, vp],
        "bsr_restore_wait": [vp, vp, C.POINTER(i32)],
        "bsr_req_invalid_blocks": [vp, vp, u32, u32, vp, C.c_size_t, C.POINTER(C.c_size_t)],
        "bsr_install_kernel_in_use": [vp, C.POINTER(i32)],
        "bsr_restore_calibrate": [vp, vp, i32, C.POINTER(C.c_double)],
        "bsr_plan_spans": [C.POINTER(bsr_group_desc), u32, C.POINTER(bsr_tensor_desc), u32, vp, C.c_size_t,
                           C.POINTER(C.c_size_t)],
        "bsr_numa_of_pci": [C.c_char_p, C.c_char_p, C.POINTER(i32), C.c_char_p, C.c_size_t, C.POINTER(i32)],
        "bsr_plan_pieces": [C.c_uint64, u32, u32, u32, vp, C.c_size_t, C.POINTER(C.c_size_t)],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.bsr_last_error.argtypes = [vp]
    lib.bsr_last_error.restype = C.c_char_p
    return lib


lib = _load()


def _ptr(a) -> int | None:
    """Address of a numpy array (host) or a raw integer address (device); None stays NULL."""
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        assert a.flags["C_CONTIGUOUS"]
        return a.ctypes.data
    return int(a)


# ---- the C calls, one thin function each ---------------------------------------------------------
def bsr_ctx_create(W: int, n_ranks: int, *, load_concurrency: int = 0, dev_staging_depth: int = 0,
                   timeout_ms: int = 0, slot_align: int = 0, device: int = 0, reg_id: int = 1,
                   install_variant: int = BSR_INSTALL_AUTO, time_kernels: bool = False,
                   direct_install: bool = False, budget_slots: int = 0, install_batch: int = 0,
                   numa_bind: int = BSR_NUMA_AUTO):
    cfg = bsr_config(W, n_ranks, BSR_CHUNK_TOKENS, load_concurrency, dev_staging_depth, timeout_ms,
                     slot_align, device, reg_id, install_variant, int(time_kernels),
                     int(direct_install), budget_slots, install_batch, numa_bind)
    ctx = C.c_void_p()
    rc = lib.bsr_ctx_create(C.byref(cfg), C.byref(ctx))
    return rc, (ctx if rc == BSR_OK else None)


def bsr_ctx_destroy(ctx) -> int:
    return lib.bsr_ctx_destroy(ctx)


def bsr_last_error(ctx) -> str:
    return lib.bsr_last_error(ctx).decode()


def bsr_register(ctx, rank: int, groups, tensors) -> int:
    """groups: [(block_tokens, num_phys_blocks)], tensors: [(group, bytes_per_token, dev_ptr)]."""
    g = (bsr_group_desc * len(groups))(*[bsr_group_desc(b, n) for b, n in groups])
    t = (bsr_tensor_desc * len(tensors))(*[bsr_tensor_desc(gg, e, p) for gg, e, p in tensors])
    return lib.bsr_register(ctx, rank, g, len(groups), t, len(tensors))


def bsr_install_kernel_in_use(ctx):
    """Returns (rc, BSR_INSTALL_VECTOR or BSR_INSTALL_BULK)."""
    v = C.c_int(0)
    rc = lib.bsr_install_kernel_in_use(ctx, C.byref(v))
    return rc, v.value


def bsr_chunk_bytes(ctx):
    a, b = C.c_uint64(), C.c_uint64()
    rc = lib.bsr_chunk_bytes(ctx, C.byref(a), C.byref(b))
    return rc, a.value, b.value


def bsr_tier_put(ctx, rank: int, key: int, data, nbytes: int, group_ck=None,
                 location: int = BSR_LOC_HOST) -> int:
    ck = None if group_ck is None else np.ascontiguousarray(group_ck, dtype=np.uint64)
    return lib.bsr_tier_put(ctx, rank, int(key), _ptr(data), nbytes, _ptr(ck), location)


def bsr_tier_remove(ctx, rank: int, key: int) -> int:
    return lib.bsr_tier_remove(ctx, rank, int(key))


def bsr_tier_checksums(ctx, rank: int, key: int, n_groups: int):
    out = np.zeros(n_groups, dtype=np.uint64)
    rc = lib.bsr_tier_checksums(ctx, rank, int(key), _ptr(out))
    return rc, out


def bsr_probe(ctx, tok, n_tok: int, salt: int, tok_on_device: bool = False):
    """Returns (rc, keys[N], hit_bitmap[ceil(N/64)], n_hit_chunks)."""
    n = n_tok // BSR_CHUNK_TOKENS
    keys = np.zeros(n, dtype=np.uint64)
    bitmap = np.zeros((n + 63) // 64, dtype=np.uint64)
    n_hit = C.c_uint32(0)
    rc = lib.bsr_probe(ctx, _ptr(tok), n_tok, int(tok_on_device), int(salt), _ptr(keys),
                       _ptr(bitmap), C.byref(n_hit))
    return rc, keys, bitmap, n_hit.value


def bsr_req_create(ctx, keys: np.ndarray, block_tables):
    """block_tables: list (rank-major, then group) of int32 numpy arrays."""
    keys = np.ascontiguousarray(keys, dtype=np.uint64)
    tabs = [np.ascontiguousarray(t, dtype=np.int32) for t in block_tables]
    arr = (C.c_void_p * len(tabs))(*[t.ctypes.data for t in tabs])
    req = C.c_void_p()
    rc = lib.bsr_req_create(ctx, _ptr(keys), len(keys), arr, C.byref(req))
    return rc, (req if rc == BSR_OK else None)


def bsr_req_release(ctx, req) -> int:
    return lib.bsr_req_release(ctx, req)


def bsr_restore(ctx, req, cuda_stream: int | None = None) -> int:
    return lib.bsr_restore(ctx, req, cuda_stream)


def bsr_restore_calibrate(ctx, req, stages: int):
    """Returns (rc, seconds) of a fill-only or fill + copy pass over the request's chunks."""
    sec = C.c_double(0.0)
    rc = lib.bsr_restore_calibrate(ctx, req, stages, C.byref(sec))
    return rc, sec.value


def bsr_plan_spans(block_tokens, tensors, capacity: int = 1 << 20):
    """block_tokens: per group; tensors: [(group, bytes_per_token)].  Returns (rc, numpy structured array)
    with one record per span of a chunk (host only, no CUDA call)."""
    g = (bsr_group_desc * len(block_tokens))(*[bsr_group_desc(b, 1) for b in block_tokens])
    t = (bsr_tensor_desc * len(tensors))(*[bsr_tensor_desc(gg, e, None) for gg, e in tensors])
    dt = np.dtype([(k, "<u4") for k in ("src_off", "bytes", "dst_off", "run_bytes", "tensor", "group", "block", "n_runs")])
    out = np.zeros(capacity, dtype=dt)
    n = C.c_size_t(0)
    rc = lib.bsr_plan_spans(g, len(block_tokens), t, len(tensors), out.ctypes.data, capacity, C.byref(n))
    return rc, out[: min(n.value, capacity)]


def bsr_plan_pieces(chunk_bytes: int, n_chunks: int, n_ranks: int, fill_threads: int, capacity: int = 1 << 20):
    """Returns (rc, numpy structured array) with one record (chunk, rank, offset, bytes) per fill piece of a
    restore, in the order the pieces are handed out (host only, no CUDA call)."""
    dt = np.dtype([(k, "<u4") for k in ("chunk", "rank", "offset", "bytes")])
    out = np.zeros(capacity, dtype=dt)
    n = C.c_size_t(0)
    rc = lib.bsr_plan_pieces(chunk_bytes, n_chunks, n_ranks, fill_threads, out.ctypes.data, capacity, C.byref(n))
    return rc, out[: min(n.value, capacity)]


def bsr_numa_of_pci(sysfs_root: str, pci_bus_id: str):
    """Returns (rc, node, cpulist, n_nodes) read from a sysfs tree (host only, no CUDA call)."""
    node, n_nodes = C.c_int(-1), C.c_int(0)
    buf = C.create_string_buffer(1024)
    rc = lib.bsr_numa_of_pci(sysfs_root.encode(), pci_bus_id.encode(), C.byref(node), buf, len(buf),
                             C.byref(n_nodes))
    return rc, node.value, buf.value.decode(), n_nodes.value


def bsr_restore_async(ctx, req, cuda_stream: int | None = None) -> int:
    return lib.bsr_restore_async(ctx, req, cuda_stream)


def bsr_restore_wait(ctx, req):
    """Returns (rc, status of the restore that was started with bsr_restore_async)."""
    st = C.c_int(0)
    rc = lib.bsr_restore_wait(ctx, req, C.byref(st))
    return rc, st.value


def bsr_commit(ctx, req):
    n = C.c_uint32(0)
    rc = lib.bsr_commit(ctx, req, C.byref(n))
    return rc, n.value


def bsr_invalidate(ctx, req, flags: int = 0) -> int:
    return lib.bsr_invalidate(ctx, req, flags)


def bsr_req_bitmap(ctx, req, n_ranks: int, n_groups: int, n_adv: int):
    out = np.zeros(n_ranks * n_groups * ((n_adv + 63) // 64), dtype=np.uint64)
    rc = lib.bsr_req_bitmap(ctx, req, _ptr(out), out.size)
    return rc, out


def bsr_req_invalid_blocks(ctx, req, rank: int, group: int, capacity: int):
    """Returns (rc, int32 array of the erroneous destination block ids of (rank, group))."""
    out = np.zeros(max(capacity, 1), dtype=np.int32)
    n = C.c_size_t(0)
    rc = lib.bsr_req_invalid_blocks(ctx, req, rank, group, _ptr(out), capacity, C.byref(n))
    return rc, out[: min(n.value, capacity)]


def bsr_req_checksums(ctx, req, n_ranks: int, n_groups: int, n_adv: int):
    out = np.zeros(n_ranks * n_groups * n_adv, dtype=np.uint64)
    rc = lib.bsr_req_checksums(ctx, req, _ptr(out), out.size)
    return rc, out.reshape(n_ranks, n_groups, n_adv)


def bsr_get_stats(ctx):
    st = bsr_stats()
    rc = lib.bsr_get_stats(ctx, C.byref(st))
    return rc, st


def bsr_reset_stats(ctx) -> int:
    return lib.bsr_reset_stats(ctx)


def bsr_test_inject(ctx, kind: int, rank: int = 0, group: int = 0, chunk: int = 0, seed: int = 0) -> int:
    return lib.bsr_test_inject(ctx, kind, rank, group, chunk, int(seed))


def bsr_probe_keys_noalloc(device: int, d_tok: int, n_tok: int, salt: int, reg_id: int,
                           d_keys_out: int, cuda_stream: int | None = None) -> int:
    """Prefix keys for callers that must not allocate: device pointers in, device pointer out,
    enqueued on `cuda_stream`; at most BSR_NOALLOC_MAX_CHUNKS chunks (see include/bsr.h)."""
    return lib.bsr_probe_keys_noalloc(device, d_tok, n_tok, int(salt), int(reg_id), d_keys_out, cuda_stream)


# ---- request-level recovery ----------------------------------------------------------------------
def bsr_tier_put_at(ctx, tier: int, rank: int, key: int, data, nbytes: int, group_ck=None,
                    location: int = BSR_LOC_HOST) -> int:
    ck = None if group_ck is None else np.ascontiguousarray(group_ck, dtype=np.uint64)
    return lib.bsr_tier_put_at(ctx, tier, rank, int(key), _ptr(data), nbytes, _ptr(ck), location)


def bsr_tier_remove_at(ctx, tier: int, rank: int, key: int) -> int:
    return lib.bsr_tier_remove_at(ctx, tier, rank, int(key))


def bsr_tier_set_available(ctx, tier: int, available: bool) -> int:
    return lib.bsr_tier_set_available(ctx, tier, int(available))


def bsr_probe_request(ctx, request_id: int, tok, n_tok: int, salt: int, tok_on_device: bool = False):
    """Returns (rc, keys[N], hit_bitmap[ceil(N/64)], n_hit_chunks, tier)."""
    n = n_tok // BSR_CHUNK_TOKENS
    keys = np.zeros(n, dtype=np.uint64)
    bitmap = np.zeros((n + 63) // 64, dtype=np.uint64)
    n_hit, tier = C.c_uint32(0), C.c_int(-1)
    rc = lib.bsr_probe_request(ctx, int(request_id), _ptr(tok), n_tok, int(tok_on_device), int(salt),
                               _ptr(keys), _ptr(bitmap), C.byref(n_hit), C.byref(tier))
    return rc, keys, bitmap, n_hit.value, tier.value


def bsr_req_bind(ctx, req, request_id: int, tier: int) -> int:
    return lib.bsr_req_bind(ctx, req, int(request_id), tier)


def bsr_request_done(ctx, request_id: int) -> int:
    return lib.bsr_request_done(ctx, int(request_id))


def bsr_request_is_force_local(ctx, request_id: int):
    out = C.c_int(0)
    rc = lib.bsr_request_is_force_local(ctx, int(request_id), C.byref(out))
    return rc, bool(out.value)


def bsr_tier_set_fetch(ctx, tier: int, fn, user=None) -> int:
    """fn: a BSR_FETCH_FN instance (keep a reference to it for as long as it is registered), or None."""
    return lib.bsr_tier_set_fetch(ctx, tier, fn if fn is not None else BSR_FETCH_FN(0), user)


def bsr_get_trace(ctx, capacity: int = 1 << 16):
    """Returns (rc, numpy structured array) with the timeline of the last restore through the slot pool."""
    dt = np.dtype([("chunk", "<u4"), ("rank", "<u4"), ("slot", "<u4"), ("reserved", "<u4"),
                   ("t_admit_ns", "<u8"), ("t_filled_ns", "<u8"), ("t_submit_ns", "<u8"), ("t_done_ns", "<u8")])
    out = np.zeros(capacity, dtype=dt)
    n = C.c_size_t(0)
    rc = lib.bsr_get_trace(ctx, out.ctypes.data, capacity, C.byref(n))
    return rc, out[: min(n.value, capacity)]
