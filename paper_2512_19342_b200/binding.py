"""Thin ctypes binding of ``libbls.so``: argument marshalling only.

Every step of the path runs inside the CUDA library; torch is used here for
device memory (workspace, tables, inputs) and for the current stream.  There is
no CPU fallback: if the shared library is missing the first call raises.
"""
from __future__ import annotations

import collections
import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbls.so")

BLS_OK, BLS_EINVAL, BLS_ENOSPC, BLS_ECUDA, BLS_ERANGE, BLS_ETIMEOUT, BLS_ESTATE = range(7)
BLS_F32, BLS_BF16, BLS_F16 = 0, 1, 2
BLS_PART_TABLE_RR, BLS_PART_ROW_BLOCK = 0, 1
PART = {"table_rr": BLS_PART_TABLE_RR, "row_block": BLS_PART_ROW_BLOCK}
_DTYPE = {torch.float32: BLS_F32, torch.bfloat16: BLS_BF16, torch.float16: BLS_F16}

EXPORTS = ["bls_plan_bytes", "bls_plan", "bls_destroy", "bls_route", "bls_lookup", "bls_step",
           "bls_drain", "bls_step_host", "bls_drain_host", "bls_view", "bls_counters", "bls_status",
           "bls_set_stall", "bls_set_wait_limit", "bls_strerror", "bls_fill_hash_table",
           "bls_profile", "bls_profile_read", "bls_set_tuning", "bls_route_table_rr_static",
           "bls_set_random_stall", "bls_set_ring", "bls_timeline", "bls_set_poison", "bls_set_overlap", "bls_set_fused", "bls_a2a_bytes", "bls_a2a_create", "bls_a2a_destroy", "bls_a2a_post", "bls_a2a_wait",
           "bls_a2a_status", "bls_mlp_bytes", "bls_mlp_create", "bls_mlp_destroy", "bls_mlp_forward", "bls_interact",
           "bls_mlp_status", "bls_hot_bytes", "bls_hot_attach", "bls_hot_observe", "bls_hot_build", "bls_hot_view"]


class BlsError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib().bls_strerror(code).decode()} (status {code})")


class _Table(C.Structure):
    _fields_ = [("weight", C.c_void_p), ("rows", C.c_int64), ("dim", C.c_int32), ("dtype", C.c_int32)]


class _View(C.Structure):
    _fields_ = [("sendcounts", C.c_void_p), ("sdispls", C.c_void_p), ("recvcounts", C.c_void_p),
                ("rdispls", C.c_void_p), ("sendbuf", C.c_void_p), ("sendbuf_stride", C.c_int64),
                ("sub_start", C.c_void_p), ("sub_stride", C.c_int64), ("subbags_per_rank", C.c_int64),
                ("sub_entries", C.c_int64), ("sub_bag_major", C.c_int32), ("out", C.c_void_p)]


_lib = None


def lib():
    """Load the CUDA library; fails loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_19342_b200.build` "
                               "(there is no CPU fallback)")
        _lib = C.CDLL(LIB_PATH)
        _lib.bls_strerror.restype = C.c_char_p
        _lib.bls_strerror.argtypes = [C.c_int]
        # the call of the inner loop: with declared argument types plain Python integers can be passed
        _lib.bls_step.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
    return _lib


def _check(code: int, where: str):
    if code != BLS_OK:
        raise BlsError(code, where)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> C.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _table_array(tables: Sequence[torch.Tensor]):
    arr = (_Table * len(tables))()
    for i, w in enumerate(tables):
        if w.dim() != 2 or not w.is_contiguous():
            raise ValueError("tables must be contiguous 2-D tensors")
        arr[i] = _Table(w.data_ptr(), w.shape[0], w.shape[1], _DTYPE[w.dtype])
    return arr


class Plan:
    """Handle of a plan plus the tensors it borrows (kept alive here)."""

    def __init__(self, handle, tables, workspace, P, T, b, D, k_max, part, stream):
        self.handle, self.tables, self.workspace = handle, list(tables), workspace
        self.P, self.T, self.b, self.D, self.k_max, self.part = P, T, b, D, k_max, part
        self.stream = stream
        # inputs of the iterations still in the ring stay referenced here (the library borrows them)
        self._borrowed = collections.deque(maxlen=k_max + 2)
        self._keep = self._borrowed.append
        self._outs = {}                      # output slot address -> tensor view (a ring has k_max + 1 of them)
        self._ret = (C.c_void_p(), C.c_int64(-1))   # bls_step / bls_drain write their results here
        self._ret_refs = (C.byref(self._ret[0]), C.byref(self._ret[1]))

    def _wrap(self, ptr: int, n_elems: int, dtype: torch.dtype) -> torch.Tensor:
        off = ptr - self.workspace.data_ptr()
        nbytes = n_elems * torch.empty((), dtype=dtype).element_size()
        return self.workspace[off:off + nbytes].view(dtype)

    def out_tensor(self, ptr: int) -> torch.Tensor:
        t = self._outs.get(ptr)
        if t is None:
            t = self._wrap(ptr, self.P * self.b * self.T * self.D, torch.float32).view(self.P, self.b, self.T, self.D)
            self._outs[ptr] = t
        return t

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h:
            try:
                lib().bls_destroy(h)
            except Exception:          # interpreter shutting down: the process is about to free everything anyway
                pass


def bls_plan_bytes(tables: Sequence[torch.Tensor], part: str, P: int, local_batch: int, k_max: int,
                   max_ids_per_rank: int) -> int:
    n = C.c_size_t(0)
    arr = _table_array(tables)
    _check(lib().bls_plan_bytes(arr, len(tables), PART[part], P, local_batch, k_max,
                                C.c_int64(max_ids_per_rank), C.byref(n)), "bls_plan_bytes")
    return n.value


def bls_plan(tables: Sequence[torch.Tensor], part: str, P: int, local_batch: int, k_max: int,
             max_ids_per_rank: int, stream: Optional[torch.cuda.Stream] = None) -> Plan:
    nbytes = bls_plan_bytes(tables, part, P, local_batch, k_max, max_ids_per_rank)
    workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=tables[0].device)
    pad = (-workspace.data_ptr()) % 256
    workspace = workspace[pad:pad + nbytes]
    handle = C.c_void_p()
    arr = _table_array(tables)
    _check(lib().bls_plan(arr, len(tables), PART[part], P, local_batch, k_max, C.c_int64(max_ids_per_rank),
                          C.c_void_p(workspace.data_ptr()), C.c_size_t(nbytes), _stream_ptr(stream),
                          C.byref(handle)), "bls_plan")
    return Plan(handle, tables, workspace, P, len(tables), local_batch, tables[0].shape[1], k_max, part, stream)


def bls_route(plan: Plan, it: int, ids: torch.Tensor, offsets: torch.Tensor) -> None:
    plan._keep((ids, offsets))
    _check(lib().bls_route(plan.handle, C.c_int64(it), C.c_void_p(ids.data_ptr()),
                           C.c_void_p(offsets.data_ptr()), C.c_int64(ids.numel())), "bls_route")


def bls_lookup(plan: Plan, it: int) -> None:
    _check(lib().bls_lookup(plan.handle, C.c_int64(it)), "bls_lookup")


def bls_step(plan: Plan, k: int, ids: torch.Tensor, offsets: torch.Tensor):
    """Returns (out, out_iter): out is a [P][b][T][D] fp32 view into the ring or None."""
    plan._keep((ids, offsets))
    (out, it), (p_out, p_it) = plan._ret, plan._ret_refs
    code = lib().bls_step(plan.handle, k, ids.data_ptr(), offsets.data_ptr(), ids.numel(), p_out, p_it)
    if code != BLS_OK:
        raise BlsError(code, "bls_step")
    return (plan.out_tensor(out.value) if out.value else None), it.value


def bls_drain(plan: Plan):
    (out, it), (p_out, p_it) = plan._ret, plan._ret_refs
    _check(lib().bls_drain(plan.handle, p_out, p_it), "bls_drain")
    return (plan.out_tensor(out.value) if out.value else None), it.value


def bls_step_host(plan: Plan, k: int, ids: torch.Tensor, offsets: torch.Tensor,
                  host_out: Optional[torch.Tensor]) -> int:
    """ids/offsets/host_out are HOST tensors (pinned recommended); returns the iteration copied out or -1."""
    plan._keep((ids, offsets))
    it = C.c_int64(-1)
    _check(lib().bls_step_host(plan.handle, k, C.c_void_p(ids.data_ptr()), C.c_void_p(offsets.data_ptr()),
                               C.c_int64(ids.numel()),
                               C.c_void_p(host_out.data_ptr() if host_out is not None else None),
                               C.byref(it)), "bls_step_host")
    return it.value


def bls_drain_host(plan: Plan, host_out: Optional[torch.Tensor]) -> int:
    it = C.c_int64(-1)
    _check(lib().bls_drain_host(plan.handle, C.c_void_p(host_out.data_ptr() if host_out is not None else None),
                                C.byref(it)), "bls_drain_host")
    return it.value


def bls_view(plan: Plan, it: int) -> dict:
    """Tensors (views into the ring) of iteration ``it``'s routing artefacts and output."""
    v = _View()
    _check(lib().bls_view(plan.handle, C.c_int64(it), C.byref(v)), "bls_view")
    P = plan.P
    i32 = torch.int32
    d = {k: plan._wrap(getattr(v, k), P * P, i32).view(P, P)
         for k in ("sendcounts", "sdispls", "recvcounts", "rdispls")}
    d["sendbuf"] = plan._wrap(v.sendbuf, P * v.sendbuf_stride, i32).view(P, v.sendbuf_stride)
    d["sub_start"] = plan._wrap(v.sub_start, P * v.sub_stride, i32).view(P, v.sub_stride)[:, :v.sub_entries]
    d["sub_bag_major"] = bool(v.sub_bag_major)
    d["out"] = plan.out_tensor(v.out)
    return d


def bls_counters(plan: Plan):
    arrs = [(C.c_int64 * plan.P)() for _ in range(3)]
    _check(lib().bls_counters(plan.handle, *arrs), "bls_counters")
    return tuple(list(a) for a in arrs)


def bls_status(plan: Plan):
    """(status code, max lag seen); synchronises the plan's stream."""
    lag = C.c_int64(0)
    return lib().bls_status(plan.handle, C.byref(lag)), lag.value


def bls_set_stall(plan: Plan, rank: int, ns: int) -> None:
    _check(lib().bls_set_stall(plan.handle, rank, C.c_int64(ns)), "bls_set_stall")


def bls_set_random_stall(plan: Plan, rank: int, max_ns: int, seed: int = 0) -> None:
    _check(lib().bls_set_random_stall(plan.handle, rank, C.c_int64(max_ns), C.c_uint64(seed)), "bls_set_random_stall")


def bls_set_ring(plan: Plan, mode: int) -> None:
    """-1 persistent ring kernel only while delays are injected (default), 0 also for small iterations, 1 always."""
    _check(lib().bls_set_ring(plan.handle, int(mode)), "bls_set_ring")


def bls_timeline(plan: Plan, first_iter: int, n_iter: int):
    """(post_ns, serve_ns, done_ns): three numpy uint64 arrays [n_iter][P] of device time stamps."""
    import numpy as np
    arrs = [np.zeros((n_iter, plan.P), np.uint64) for _ in range(3)]
    _check(lib().bls_timeline(plan.handle, C.c_int64(first_iter), n_iter,
                              *[a.ctypes.data_as(C.c_void_p) for a in arrs]), "bls_timeline")
    return tuple(arrs)


def bls_set_poison(plan: Plan, enable: bool) -> None:
    _check(lib().bls_set_poison(plan.handle, int(enable)), "bls_set_poison")


def bls_set_overlap(plan: Plan, mode: int) -> None:
    """-1 never, 0 by iteration size (default), 1 whenever the overlapped mode applies."""
    _check(lib().bls_set_overlap(plan.handle, int(mode)), "bls_set_overlap")


def bls_set_fused(plan: Plan, mode: int) -> None:
    """One-launch kernel for small table-wise iterations: -1 never, 0 by iteration size (default), 1 whenever it applies."""
    _check(lib().bls_set_fused(plan.handle, int(mode)), "bls_set_fused")


def bls_set_wait_limit(plan: Plan, ns: int) -> None:
    _check(lib().bls_set_wait_limit(plan.handle, C.c_int64(ns)), "bls_set_wait_limit")


def bls_set_tuning(plan: Plan, bags_per_run: int = 0, rows_in_flight: int = 0) -> None:
    _check(lib().bls_set_tuning(plan.handle, bags_per_run, rows_in_flight), "bls_set_tuning")


def bls_profile(plan: Plan, enable: bool) -> None:
    _check(lib().bls_profile(plan.handle, int(enable)), "bls_profile")


def bls_profile_read(plan: Plan) -> dict:
    """Summed stage times (ms) of the calls recorded since the last read; synchronises."""
    r, g, c = C.c_double(0), C.c_double(0), C.c_double(0)
    n, kn = C.c_int64(0), C.c_int64(0)
    _check(lib().bls_profile_read(plan.handle, C.byref(r), C.byref(g), C.byref(c), C.byref(n), C.byref(kn)),
           "bls_profile_read")
    return {"ms_route": r.value, "ms_gather": g.value, "ms_ring": c.value, "calls": n.value,
            "kernels_total": kn.value}


def bls_fill_hash_table(weight: torch.Tensor, seed: int, t: int,
                        stream: Optional[torch.cuda.Stream] = None) -> None:
    _check(lib().bls_fill_hash_table(C.c_void_p(weight.data_ptr()), C.c_int64(weight.shape[0]),
                                     C.c_int32(weight.shape[1]), _DTYPE[weight.dtype],
                                     C.c_uint64(seed & ((1 << 64) - 1)), C.c_int32(t), _stream_ptr(stream)),
           "bls_fill_hash_table")


def bls_route_table_rr_static(table_rows: torch.Tensor, P: int, local_batch: int, ids: torch.Tensor,
                              offsets: torch.Tensor, sendcounts: torch.Tensor, sdispls: torch.Tensor,
                              sendbuf: torch.Tensor, sub_start: torch.Tensor, status: torch.Tensor,
                              stream: Optional[torch.cuda.Stream] = None) -> None:
    """Table-wise router without a plan or workspace, for callers that cannot allocate
    device memory (the scratch is a static array inside the library).  Every tensor is
    the caller's: table_rows int64 [T]; sendcounts/sdispls int32 [P][P]; sendbuf int32
    [P][cap]; sub_start int32 [P][T*local_batch+1]; status int32 [1].  This wrapper
    allocates nothing either."""
    T = table_rows.numel()
    _check(lib().bls_route_table_rr_static(
        C.c_void_p(table_rows.data_ptr()), T, P, local_batch, C.c_void_p(ids.data_ptr()),
        C.c_void_p(offsets.data_ptr()), C.c_int64(ids.numel()), C.c_void_p(sendcounts.data_ptr()),
        C.c_void_p(sdispls.data_ptr()), C.c_void_p(sendbuf.data_ptr()), C.c_int64(sendbuf.shape[1]),
        C.c_void_p(sub_start.data_ptr()), C.c_void_p(status.data_ptr()), _stream_ptr(stream)),
        "bls_route_table_rr_static")


def bls_hot_attach(plan: Plan, rows_per_table: int) -> None:
    """Allocate (with torch) and attach the buffer for hot-row staging with `rows_per_table` slots."""
    n = C.c_size_t(0)
    _check(lib().bls_hot_bytes(plan.handle, rows_per_table, C.byref(n)), "bls_hot_bytes")
    buf = torch.empty(n.value + 256, dtype=torch.uint8, device=plan.workspace.device)
    pad = (-buf.data_ptr()) % 256
    buf = buf[pad:pad + n.value]
    _check(lib().bls_hot_attach(plan.handle, rows_per_table, C.c_void_p(buf.data_ptr()), C.c_size_t(n.value)),
           "bls_hot_attach")
    plan.hot_buffer, plan.hot_rows_per_table = buf, rows_per_table


def bls_hot_observe(plan: Plan, ids: torch.Tensor, offsets: torch.Tensor) -> None:
    _check(lib().bls_hot_observe(plan.handle, C.c_void_p(ids.data_ptr()), C.c_void_p(offsets.data_ptr()),
                                 C.c_int64(ids.numel())), "bls_hot_observe")


def bls_hot_build(plan: Plan) -> None:
    _check(lib().bls_hot_build(plan.handle), "bls_hot_build")


def bls_hot_view(plan: Plan):
    """(rows [T][K] int32, count [T] int32) as views into the attached buffer."""
    rows, count, k = C.c_void_p(), C.c_void_p(), C.c_int(0)
    _check(lib().bls_hot_view(plan.handle, C.byref(rows), C.byref(count), C.byref(k)), "bls_hot_view")
    buf = plan.hot_buffer

    def wrap(ptr, n):
        off = ptr - buf.data_ptr()
        return buf[off:off + 4 * n].view(torch.int32)
    return wrap(rows.value, plan.T * k.value).view(plan.T, k.value), wrap(count.value, plan.T)


class A2a:
    """Handle of a stand-alone BLS alltoallv (raw bytes between the logical ranks)."""

    def __init__(self, P: int, k_max: int, max_bytes_per_rank: int, device="cuda",
                 stream: Optional[torch.cuda.Stream] = None):
        n = C.c_size_t(0)
        _check(lib().bls_a2a_bytes(P, k_max, C.c_int64(max_bytes_per_rank), C.byref(n)), "bls_a2a_bytes")
        ws = torch.empty(n.value + 256, dtype=torch.uint8, device=device)
        pad = (-ws.data_ptr()) % 256
        self.workspace = ws[pad:pad + n.value]
        self.P, self.k_max = P, k_max
        self.handle = C.c_void_p()
        _check(lib().bls_a2a_create(P, k_max, C.c_int64(max_bytes_per_rank), C.c_void_p(self.workspace.data_ptr()),
                                    C.c_size_t(n.value), _stream_ptr(stream), C.byref(self.handle)), "bls_a2a_create")
        self._borrowed = collections.deque(maxlen=k_max + 2)   # buffers of the requests still in flight
        self._views = {}                     # receive slot address -> the three tensor views of that slot
        self._ret = (C.c_void_p(), C.c_int64(0), C.c_void_p(), C.c_void_p(), C.c_int64(-1))
        self._ret_refs = tuple(C.byref(x) for x in self._ret)
        l = lib()
        l.bls_a2a_post.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64]
        l.bls_a2a_wait.argtypes = [C.c_void_p] * 6

    def post(self, sendbuf: torch.Tensor, sendcounts: torch.Tensor, sdispls: torch.Tensor, max_segment_bytes: int):
        """sendbuf uint8 [P][stride]; sendcounts/sdispls int64 [P][P] (bytes), all on the device."""
        self._borrowed.append((sendbuf, sendcounts, sdispls))
        _check(lib().bls_a2a_post(self.handle, sendbuf.data_ptr(), sendbuf.shape[1], sendcounts.data_ptr(),
                                  sdispls.data_ptr(), max_segment_bytes), "bls_a2a_post")

    def wait(self):
        """Completes the oldest request: (recv uint8 [P][stride], recvcounts, rdispls int64 [P][P], request number)."""
        recv, stride, rc, rd, req = self._ret
        _check(lib().bls_a2a_wait(self.handle, *self._ret_refs), "bls_a2a_wait")
        key = (recv.value, stride.value)
        views = self._views.get(key)
        if views is None:
            ws, P = self.workspace, self.P

            def view(ptr, nbytes):
                off = ptr - ws.data_ptr()
                return ws[off:off + nbytes]
            views = (view(recv.value, P * stride.value).view(P, stride.value),
                     view(rc.value, 8 * P * P).view(torch.int64).view(P, P),
                     view(rd.value, 8 * P * P).view(torch.int64).view(P, P))
            self._views[key] = views
        return views + (req.value,)

    def status(self) -> int:
        return lib().bls_a2a_status(self.handle)

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h:
            try:
                lib().bls_a2a_destroy(h)
            except Exception:
                pass


class Mlp:
    """Handle of a stand-in MLP stage (bottom or top MLP of Listing 1 / Listing 2).

    weights[i]: bf16 [dims[i+1]][dims[i]] device tensors, biases[i]: fp32 [dims[i+1]]; hidden layers
    use ReLU, the last one last_act (0 none, 1 ReLU, 2 logistic function)."""

    def __init__(self, weights: Sequence[torch.Tensor], biases: Sequence[torch.Tensor], last_act: int, max_rows: int,
                 stream: Optional[torch.cuda.Stream] = None):
        n = len(weights)
        self.dims = [weights[0].shape[1]] + [w.shape[0] for w in weights]
        for w, b in zip(weights, biases):
            if w.dtype != torch.bfloat16 or b.dtype != torch.float32 or not w.is_contiguous() or not b.is_contiguous():
                raise ValueError("weights must be contiguous bf16 [out][in], biases contiguous fp32")
        dims = (C.c_int * (n + 1))(*self.dims)
        nbytes = C.c_size_t(0)
        _check(lib().bls_mlp_bytes(n, dims, max_rows, C.byref(nbytes)), "bls_mlp_bytes")
        ws = torch.empty(nbytes.value + 256, dtype=torch.uint8, device=weights[0].device)
        pad = (-ws.data_ptr()) % 256
        self.workspace = ws[pad:pad + nbytes.value]
        self.weights, self.biases, self.max_rows = list(weights), list(biases), max_rows
        wp = (C.c_void_p * n)(*[w.data_ptr() for w in weights])
        bp = (C.c_void_p * n)(*[b.data_ptr() for b in biases])
        self.handle = C.c_void_p()
        _check(lib().bls_mlp_create(n, dims, wp, bp, last_act, max_rows, C.c_void_p(self.workspace.data_ptr()),
                                    C.c_size_t(nbytes.value), _stream_ptr(stream), C.byref(self.handle)), "bls_mlp_create")

    def forward(self, x: torch.Tensor, y: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
        """x bf16 [rows][ldx] -> y [rows][ldy] (bf16 or fp32); asynchronous on the stream."""
        _check(lib().bls_mlp_forward(self.handle, C.c_void_p(x.data_ptr()), x.stride(0), x.shape[0],
                                     C.c_void_p(y.data_ptr()), y.stride(0), int(y.dtype == torch.float32),
                                     _stream_ptr(stream)), "bls_mlp_forward")

    def status(self, stream: Optional[torch.cuda.Stream] = None) -> int:
        return lib().bls_mlp_status(self.handle, _stream_ptr(stream))

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h:
            try:
                lib().bls_mlp_destroy(h)
            except Exception:
                pass


def bls_interact(x: torch.Tensor, pooled: torch.Tensor, r: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> None:
    """x bf16 [rows][>=D], pooled fp32 [rows][T][D] (or any shape with rows*T*D elements in that order), r bf16 [rows][ldr]."""
    rows, D = x.shape[0], pooled.shape[-1]
    T = pooled.numel() // (rows * D)
    _check(lib().bls_interact(C.c_void_p(x.data_ptr()), x.stride(0), C.c_void_p(pooled.data_ptr()), rows, T, D,
                              C.c_void_p(r.data_ptr()), r.stride(0), _stream_ptr(stream)), "bls_interact")
