"""ctypes binding of libcodedreduce.so: the same entry points as include/codedreduce.h,
with argument marshalling only.  Device buffers are torch CUDA tensors (torch supplies
device memory and streams); every step of the computation runs in the library's kernels.

The library is loaded on first use and a missing build raises: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
# the in-tree build, unless CODEDREDUCE_LIB names a library built elsewhere (e.g. with other compiler flags)
LIB_PATH = os.environ.get("CODEDREDUCE_LIB") or os.path.join(_PKG, "libcodedreduce.so")

# status codes / enums of codedreduce.h
CR_OK = 0
CR_ERR_INVALID_ARG, CR_ERR_BAD_PARTITION_COUNT, CR_ERR_CODE_UNAVAILABLE = 1, 2, 3
CR_ERR_ILL_CONDITIONED, CR_ERR_UNDECODABLE_MASK, CR_ERR_DTYPE = 4, 5, 6
CR_ERR_CUDA, CR_ERR_OOM, CR_ERR_TIMEOUT = 7, 8, 9
CR_CODE_CYCLIC_RANDOM, CR_CODE_FRACTIONAL_REPETITION, CR_CODE_PAPER_3_1, CR_CODE_EXPLICIT = 0, 1, 2, 3
CR_F32, CR_I32 = 0, 1
CR_AGG_FUSED, CR_AGG_FUSED_LDG, CR_AGG_UNFUSED, CR_AGG_UNCODED_SUM = 0, 1, 2, 3
CR_AGG_ALL_NODES = 0x100
CR_AGG_FROM_CODED = 0x200
CR_LOSS_SQUARED, CR_LOSS_LOGISTIC = 0, 1


class cr_plan_desc_t(C.Structure):
    _fields_ = [("n", C.c_int32), ("L", C.c_int32), ("s", C.c_int32), ("P", C.c_int32), ("d", C.c_int64),
                ("code", C.c_int32), ("dtype", C.c_int32), ("seed", C.c_uint64),
                ("B_explicit", C.POINTER(C.c_double)), ("max_kappa", C.c_double),
                ("device", C.c_int32), ("reserved", C.c_int32)]


class CodedReduceError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = ""
        if status == CR_ERR_CUDA:
            detail = " (" + lib().cr_last_cuda_error().decode() + ")"
        super().__init__(f"{where}: {lib().cr_status_string(status).decode()}{detail}")


_lib = None

_SIGNATURES = {
    "cr_plan_create": (C.c_int, [C.POINTER(cr_plan_desc_t), C.POINTER(C.c_void_p)]),
    "cr_plan_destroy": (C.c_int, [C.c_void_p]),
    "cr_status_string": (C.c_char_p, [C.c_int]),
    "cr_last_cuda_error": (C.c_char_p, []),
    "cr_plan_num_nodes": (C.c_int32, [C.c_void_p]),
    "cr_plan_num_groups": (C.c_int32, [C.c_void_p]),
    "cr_plan_load": (C.c_int32, [C.c_void_p]),
    "cr_plan_int_scale": (C.c_int64, [C.c_void_p]),
    "cr_plan_get_B": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_uint64)]),
    "cr_plan_get_slots": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]),
    "cr_plan_get_decode": (C.c_int, [C.c_void_p, C.c_int32, C.c_uint32, C.c_void_p]),
    "cr_plan_expand": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                 C.POINTER(C.c_int32)]),
    "cr_latency_masks": (C.c_int, [C.c_void_p, C.c_void_p, C.c_double, C.c_void_p, C.POINTER(C.c_double)]),
    "cr_plan_device_status": (C.c_int, [C.c_void_p]),
    "cr_plan_clear_status": (C.c_int, [C.c_void_p]),
    "cr_plan_set_wait_limit": (C.c_int, [C.c_void_p, C.c_uint64]),
    "cr_selftest_wait": (C.c_int, [C.c_void_p, C.c_uint64, C.c_void_p]),
    "cr_plan_tune_batch": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32]),
    "cr_plan_batch_stats": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]),
    "cr_schedule_create": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_uint32, C.POINTER(C.c_void_p)]),
    "cr_schedule_destroy": (C.c_int, [C.c_void_p]),
    "cr_schedule_bytes": (C.c_int, [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int32)]),
    "cr_aggregate_scheduled": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t,
                                         C.c_void_p]),
    "cr_partial_gradients_workspace_bytes": (C.c_size_t, [C.c_void_p, C.c_int32]),
    "cr_partial_gradients": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_size_t, C.c_void_p]),
    "cr_partial_gradients_loss": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "cr_coded_gradients": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                     C.c_void_p]),
    "cr_partial_gradients_multi_workspace_bytes": (C.c_size_t, [C.c_void_p, C.c_int32]),
    "cr_partial_gradients_multi": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p,
                                             C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "cr_partial_gradients_static_capacity": (C.c_size_t, []),
    "cr_partial_gradients_static": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                              C.c_void_p]),
    "cr_encode": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "cr_decode": (C.c_int, [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "cr_aggregate_workspace_bytes": (C.c_size_t, [C.c_void_p, C.c_int32, C.c_uint32]),
    "cr_aggregate": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_uint32, C.c_void_p,
                               C.c_size_t, C.c_void_p]),
    "cr_aggregate_host": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_uint32,
                                    C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "cr_aggregate_bytes": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int32)]),
    "cr_plan_tune": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32]),
    "cr_plan_tune_gradients": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_int32]),
    "cr_plan_tune_items": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32]),
    "cr_plan_launch_count": (C.c_int64, [C.c_void_p]),
    "cr_plan_last_kernel": (C.c_char_p, [C.c_void_p]),
}


def lib() -> C.CDLL:
    """The loaded library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_1902_01981_b200.build` "
                "(there is no CPU fallback)")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def _check(status: int, where: str) -> None:
    if status != CR_OK:
        raise CodedReduceError(status, where)


def _dev_ptr(t) -> int:
    """Address of a contiguous torch CUDA tensor (or None -> NULL)."""
    if t is None:
        return 0
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream_ptr(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _masks(masks, cols: int) -> np.ndarray:
    m = masks if (isinstance(masks, np.ndarray) and masks.dtype == np.uint32 and masks.flags.c_contiguous) \
        else np.ascontiguousarray(np.asarray(masks, dtype=np.uint32))
    if m.size % cols != 0:
        raise ValueError(f"mask array of {m.size} entries is not a multiple of {cols}")
    return m.reshape(-1, cols)


_groups_of_plan = {}


def _num_groups(plan: int) -> int:
    """cr_plan_num_groups, remembered per live plan (the hot calls need it to shape the masks)."""
    g = _groups_of_plan.get(plan)
    if g is None:
        g = _groups_of_plan[plan] = lib().cr_plan_num_groups(plan)
    return g


# ------------------------------------------------------------------ plan

def cr_plan_create(n: int, L: int, s: int, P: int, d: int, code: int = CR_CODE_CYCLIC_RANDOM,
                   dtype: int = CR_F32, seed: int = 0, B_explicit=None, max_kappa: float = 0.0,
                   device: int = -1) -> int:
    """Returns an opaque plan handle.  device = -1 builds a host-only plan (queries only)."""
    desc = cr_plan_desc_t()
    desc.n, desc.L, desc.s, desc.P, desc.d = n, L, s, P, d
    desc.code, desc.dtype, desc.seed = code, dtype, seed
    desc.max_kappa, desc.device, desc.reserved = max_kappa, device, 0
    keep = None
    if B_explicit is not None:
        keep = np.ascontiguousarray(np.asarray(B_explicit, dtype=np.float64))
        if keep.size != L * n * n:
            raise ValueError("B_explicit must hold L*n*n doubles")
        desc.B_explicit = keep.ctypes.data_as(C.POINTER(C.c_double))
    out = C.c_void_p()
    _check(lib().cr_plan_create(C.byref(desc), C.byref(out)), "cr_plan_create")
    return out.value


def cr_plan_destroy(plan: int) -> None:
    _groups_of_plan.pop(plan, None)      # the handle may be reused by a later plan
    _check(lib().cr_plan_destroy(plan), "cr_plan_destroy")


def cr_plan_num_nodes(plan: int) -> int:
    return lib().cr_plan_num_nodes(plan)


def cr_plan_num_groups(plan: int) -> int:
    return lib().cr_plan_num_groups(plan)


def cr_plan_load(plan: int) -> int:
    return lib().cr_plan_load(plan)


def cr_plan_int_scale(plan: int) -> int:
    return lib().cr_plan_int_scale(plan)


def cr_plan_launch_count(plan: int) -> int:
    return lib().cr_plan_launch_count(plan)


def cr_plan_last_kernel(plan: int) -> str:
    return lib().cr_plan_last_kernel(plan).decode()


def cr_plan_get_B(plan: int, level: int, n: int):
    """(B [n, n] float64, kappa, sub_seed) of the parents at `level`."""
    B = np.empty((n, n), dtype=np.float64)
    kappa, sub = C.c_double(), C.c_uint64()
    _check(lib().cr_plan_get_B(plan, level, B.ctypes.data, C.byref(kappa), C.byref(sub)), "cr_plan_get_B")
    return B, kappa.value, sub.value


def cr_plan_get_slots(plan: int, node: int):
    """(partition ids int32 [m], coefficients float64 [m]) of flat node `node`."""
    m = cr_plan_load(plan)
    part = np.empty(m, dtype=np.int32)
    coeff = np.empty(m, dtype=np.float64)
    _check(lib().cr_plan_get_slots(plan, node, part.ctypes.data, coeff.ctypes.data), "cr_plan_get_slots")
    return part, coeff


def cr_plan_get_decode(plan: int, level: int, straggler_mask: int, n: int) -> np.ndarray:
    a = np.empty(n, dtype=np.float64)
    _check(lib().cr_plan_get_decode(plan, level, straggler_mask, a.ctypes.data), "cr_plan_get_decode")
    return a


def cr_plan_expand(plan: int, masks):
    """(nodes, layers, weights) of the post-order schedule of one straggler pattern."""
    N = cr_plan_num_nodes(plan)
    mk = _masks(masks, cr_plan_num_groups(plan))
    nodes = np.empty(N, dtype=np.int32)
    layers = np.empty(N, dtype=np.int32)
    weights = np.empty(N, dtype=np.float64)
    count = C.c_int32()
    _check(lib().cr_plan_expand(plan, mk.ctypes.data, N, nodes.ctypes.data, layers.ctypes.data,
                                weights.ctypes.data, C.byref(count)), "cr_plan_expand")
    k = count.value
    return nodes[:k].copy(), layers[:k].copy(), weights[:k].copy()


def cr_latency_masks(plan: int, compute_time, t_c: float):
    """(masks uint32 [groups], T_CR) for one vector of per-node computation times."""
    ct = np.ascontiguousarray(np.asarray(compute_time, dtype=np.float64))
    if ct.size != cr_plan_num_nodes(plan):
        raise ValueError("one computation time per node is needed")
    masks = np.zeros(cr_plan_num_groups(plan), dtype=np.uint32)
    total = C.c_double()
    _check(lib().cr_latency_masks(plan, ct.ctypes.data, t_c, masks.ctypes.data, C.byref(total)), "cr_latency_masks")
    return masks, total.value


def cr_plan_device_status(plan: int) -> int:
    return lib().cr_plan_device_status(plan)


def cr_plan_clear_status(plan: int) -> None:
    _check(lib().cr_plan_clear_status(plan), "cr_plan_clear_status")


def cr_plan_set_wait_limit(plan: int, limit_ns: int) -> None:
    _check(lib().cr_plan_set_wait_limit(plan, limit_ns), "cr_plan_set_wait_limit")


def cr_selftest_wait(plan: int, limit_ns: int, stream=None) -> None:
    """Enqueues the kernel that lets one bounded wait run out (see codedreduce.h)."""
    _check(lib().cr_selftest_wait(plan, limit_ns, _stream_ptr(stream)), "cr_selftest_wait")


def cr_plan_tune_batch(plan: int, share_messages: int = 0, e_buffers: int = 0) -> None:
    _check(lib().cr_plan_tune_batch(plan, share_messages, e_buffers), "cr_plan_tune_batch")


def cr_plan_batch_stats(plan: int, masks, share_messages: int = 0) -> dict:
    """Host-side figures of the expansion of a batch (see codedreduce.h)."""
    mk = _masks(masks, cr_plan_num_groups(plan))
    st = np.zeros(6, dtype=np.int64)
    _check(lib().cr_plan_batch_stats(plan, mk.ctypes.data, mk.shape[0], share_messages, st.ctypes.data), "cr_plan_batch_stats")
    return dict(zip(("entries", "union", "shared_nodes", "variants", "reduced_entries", "rows"), (int(x) for x in st)))


def cr_plan_tune(plan: int, consumer_warps: int = 0, stages: int = 0, ctas_per_sm: int = 0,
                 rows_per_box: int = 0) -> None:
    _check(lib().cr_plan_tune(plan, consumer_warps, stages, ctas_per_sm, rows_per_box), "cr_plan_tune")


def cr_plan_tune_gradients(plan: int, block_kb: int = 0, stages: int = 0, cluster: int = 0) -> None:
    _check(lib().cr_plan_tune_gradients(plan, block_kb, stages, cluster), "cr_plan_tune_gradients")


def cr_plan_tune_items(plan: int, item_order: int = 0, multi_stages: int = 0) -> None:
    _check(lib().cr_plan_tune_items(plan, item_order, multi_stages), "cr_plan_tune_items")


# ------------------------------------------------------------------ device work

def cr_partial_gradients_workspace_bytes(plan: int, rows: int) -> int:
    return lib().cr_partial_gradients_workspace_bytes(plan, rows)


def cr_partial_gradients(plan: int, X, y, rows: int, w, G_slots, workspace, stream=None) -> None:
    _check(lib().cr_partial_gradients(plan, _dev_ptr(X), _dev_ptr(y), rows, _dev_ptr(w), _dev_ptr(G_slots),
                                      _dev_ptr(workspace),
                                      0 if workspace is None else workspace.numel() * workspace.element_size(),
                                      _stream_ptr(stream)), "cr_partial_gradients")


def cr_partial_gradients_loss(plan: int, loss: int, X, y, rows: int, w, G_slots, workspace, stream=None) -> None:
    _check(lib().cr_partial_gradients_loss(plan, loss, _dev_ptr(X), _dev_ptr(y), rows, _dev_ptr(w), _dev_ptr(G_slots),
                                           _dev_ptr(workspace),
                                           0 if workspace is None else workspace.numel() * workspace.element_size(),
                                           _stream_ptr(stream)), "cr_partial_gradients_loss")


def cr_coded_gradients(plan: int, loss: int, X, y, rows: int, w, E, stream=None) -> None:
    """E[v] = coded gradient of node v (its slots' gradients combined with their coefficients)."""
    _check(lib().cr_coded_gradients(plan, loss, _dev_ptr(X), _dev_ptr(y), rows, _dev_ptr(w), _dev_ptr(E),
                                    _stream_ptr(stream)), "cr_coded_gradients")


def cr_partial_gradients_multi_workspace_bytes(plan: int, rows: int) -> int:
    return lib().cr_partial_gradients_multi_workspace_bytes(plan, rows)


def cr_partial_gradients_multi(plan: int, loss: int, X, y, rows: int, W, K: int, G_multi, workspace, R_out=None,
                               stream=None) -> None:
    """G_multi[k][v][j] = partial gradient of slot j of node v at model W[k], K <= 32 models in one pass."""
    nbytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(lib().cr_partial_gradients_multi(plan, loss, _dev_ptr(X), _dev_ptr(y), rows, _dev_ptr(W), K,
                                            _dev_ptr(G_multi), _dev_ptr(R_out), _dev_ptr(workspace), nbytes,
                                            _stream_ptr(stream)), "cr_partial_gradients_multi")


def cr_partial_gradients_static_capacity() -> int:
    return lib().cr_partial_gradients_static_capacity()


def cr_partial_gradients_static(plan: int, X, y, rows: int, w, G_slots, stream=None) -> None:
    """cr_partial_gradients for callers that cannot allocate: the residual scratch is a fixed array
    inside the library (N * m * rows <= cr_partial_gradients_static_capacity()); calls that may
    overlap on one GPU race on it."""
    _check(lib().cr_partial_gradients_static(plan, _dev_ptr(X), _dev_ptr(y), rows, _dev_ptr(w), _dev_ptr(G_slots),
                                             _stream_ptr(stream)), "cr_partial_gradients_static")


def cr_encode(plan: int, G_slots, E, stream=None) -> None:
    _check(lib().cr_encode(plan, _dev_ptr(G_slots), _dev_ptr(E), _stream_ptr(stream)), "cr_encode")


def cr_decode(plan: int, parent_layer: int, M_child, E_parent, masks, M_parent, stream=None) -> None:
    mk = np.ascontiguousarray(np.asarray(masks, dtype=np.uint32))
    _check(lib().cr_decode(plan, parent_layer, _dev_ptr(M_child), _dev_ptr(E_parent), mk.ctypes.data,
                           _dev_ptr(M_parent), _stream_ptr(stream)), "cr_decode")


def cr_aggregate_workspace_bytes(plan: int, batch: int, flags: int) -> int:
    return lib().cr_aggregate_workspace_bytes(plan, batch, flags)


def cr_aggregate(plan: int, G_slots, masks, g_out, flags: int = CR_AGG_FUSED, workspace=None, stream=None) -> None:
    """masks: [batch, groups] (or [groups]) uint32 on the host; g_out: [batch, d] device tensor."""
    mk = _masks(masks, _num_groups(plan))
    _check(lib().cr_aggregate(plan, _dev_ptr(G_slots), mk.ctypes.data, mk.shape[0], _dev_ptr(g_out), flags,
                              _dev_ptr(workspace),
                              0 if workspace is None else workspace.numel() * workspace.element_size(),
                              _stream_ptr(stream)), "cr_aggregate")


def cr_schedule_create(plan: int, masks, flags: int = CR_AGG_FUSED) -> int:
    """Expands masks [batch, groups] (or [groups]) once; returns an opaque schedule handle."""
    mk = _masks(masks, _num_groups(plan))
    out = C.c_void_p()
    _check(lib().cr_schedule_create(plan, mk.ctypes.data, mk.shape[0], flags, C.byref(out)), "cr_schedule_create")
    return out.value


def cr_schedule_destroy(sched: int) -> None:
    _check(lib().cr_schedule_destroy(sched), "cr_schedule_destroy")


def cr_schedule_bytes(sched: int):
    """(algorithmic bytes, size of the union of used nodes) of one call with this schedule."""
    nbytes, used = C.c_int64(), C.c_int32()
    _check(lib().cr_schedule_bytes(sched, C.byref(nbytes), C.byref(used)), "cr_schedule_bytes")
    return nbytes.value, used.value


def _ptr_and_bytes(t):
    return (0, 0) if t is None else (_dev_ptr(t), t.numel() * t.element_size())


def cr_aggregate_scheduled(plan: int, G_slots, sched: int, g_out, workspace=None, stream=None) -> None:
    """cr_aggregate with a schedule made by cr_schedule_create.  G_slots / g_out / workspace are torch
    CUDA tensors, or plain integer device addresses (workspace then as (address, bytes)) for loops that
    do not want to pay for the tensor look-ups; stream likewise a torch stream, None or a raw handle."""
    g = G_slots if isinstance(G_slots, int) else _dev_ptr(G_slots)
    o = g_out if isinstance(g_out, int) else _dev_ptr(g_out)
    w, wb = workspace if isinstance(workspace, tuple) else _ptr_and_bytes(workspace)
    st = stream if isinstance(stream, int) else _stream_ptr(stream)
    rc = lib().cr_aggregate_scheduled(plan, g, sched, o, w, wb, st)
    if rc != CR_OK:
        raise CodedReduceError(rc, "cr_aggregate_scheduled")


def cr_aggregate_host(plan: int, G_slots_host, masks, g_out_host, dev_slots, dev_out, flags: int = CR_AGG_FUSED,
                      workspace=None, stream=None) -> None:
    """Host-buffer form: G_slots_host / g_out_host are CPU tensors (pinned for full copy speed)."""
    mk = _masks(masks, cr_plan_num_groups(plan))
    if G_slots_host.is_cuda or g_out_host.is_cuda or not G_slots_host.is_contiguous() or not g_out_host.is_contiguous():
        raise ValueError("host buffers must be contiguous CPU tensors")
    _check(lib().cr_aggregate_host(plan, G_slots_host.data_ptr(), mk.ctypes.data, mk.shape[0],
                                   g_out_host.data_ptr(), flags, _dev_ptr(dev_slots), _dev_ptr(dev_out),
                                   _dev_ptr(workspace),
                                   0 if workspace is None else workspace.numel() * workspace.element_size(),
                                   _stream_ptr(stream)), "cr_aggregate_host")


def cr_aggregate_bytes(plan: int, masks):
    """(algorithmic bytes, size of the union of used nodes) of one cr_aggregate call."""
    mk = _masks(masks, cr_plan_num_groups(plan))
    nbytes, used = C.c_int64(), C.c_int32()
    _check(lib().cr_aggregate_bytes(plan, mk.ctypes.data, mk.shape[0], C.byref(nbytes), C.byref(used)),
           "cr_aggregate_bytes")
    return nbytes.value, used.value


def slot_partitions(plan: int) -> np.ndarray:
    """[N, m] int32 table of the partition each slot holds (marshalling of cr_plan_get_slots)."""
    N = cr_plan_num_nodes(plan)
    return np.stack([cr_plan_get_slots(plan, v)[0] for v in range(N)])
