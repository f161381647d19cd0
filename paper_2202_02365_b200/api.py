"""Thin ctypes binding over libmgdense.so: argument marshalling only.

Every step of the path (sampling, relabelling, aggregation, GEMMs, scoring) runs in the
library's CUDA kernels; torch is used here for device memory and streams.  There is no
CPU fallback: a missing library or a failing call raises.
"""
from __future__ import annotations

import ctypes as C
import os
import weakref
from dataclasses import dataclass

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libmgdense.so")

MG_OK = 0
ERR_NAMES = {-1: "MG_ERR_ARG", -2: "MG_ERR_STATE", -3: "MG_ERR_NONRESIDENT", -4: "MG_ERR_DUPLICATE",
             -5: "MG_ERR_CAPACITY", -6: "MG_ERR_OOM", -7: "MG_ERR_TIMEOUT", -8: "MG_ERR_CUDA"}
DTYPE_F32, DTYPE_F16 = 0, 1
BACKING_HBM, BACKING_HOST = 0, 1
GEMM_TF32, GEMM_FP32 = 0, 1
CORRUPT_DST, CORRUPT_SRC, CORRUPT_BOTH = 1, 2, 3

# every symbol include/mgdense.h declares
EXPORTS = [
    "mg_create", "mg_destroy", "mg_last_error", "mg_load_graph", "mg_load_out_graph", "mg_set_sample_direction", "mg_set_partitioning",
    "mg_load_features", "mg_set_partition_source", "mg_set_resident", "mg_commit_resident", "mg_sample_many", "mg_sample_many_begin", "mg_sample_many_end", "mg_sample",
    "mg_dense_counts", "mg_dense_view", "mg_dense_export_many", "mg_dense_export_view", "mg_dense_free", "mg_model_create", "mg_model_set_aggregator", "mg_model_set_intermediates", "mg_model_free",
    "mg_forward", "mg_set_layer_window", "mg_keep_layer_outputs", "mg_forward_host_async", "mg_wait_output", "mg_forward_noalloc", "mg_gather_h0", "mg_layer_output", "mg_lp_prepare", "mg_lp_view", "mg_lp_free",
    "mg_distmult_score", "mg_kernel_launches", "mg_profile", "mg_profile_read", "mg_comet_plan", "mg_comet_bias", "mg_comet_autotune", "mg_gat_model_create", "mg_gat_model_set_heads", "mg_gat_model_free", "mg_gat_forward", "mg_backward", "mg_model_grads", "mg_model_sgd_step", "mg_model_adagrad_step", "mg_dense_packed_ids", "mg_apply_embedding_sgd",
]


class MgError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{ERR_NAMES.get(code, code)}: {msg}")
        self.code = code


class SampleCaps(C.Structure):
    _fields_ = [("max_nodes_total", C.c_int64), ("max_entries_total", C.c_int64),
                ("max_nodes_per_batch", C.c_int32), ("max_inner_nodes_per_batch", C.c_int32)]


class DenseArrays(C.Structure):
    _fields_ = [("k", C.c_int32), ("n_nodes", C.c_int32), ("n_sampled", C.c_int32), ("n_entries", C.c_int32),
                ("node_ids", C.c_void_p), ("node_id_offsets", C.c_void_p), ("nbrs", C.c_void_p),
                ("nbr_offsets", C.c_void_p), ("repr_map", C.c_void_p)]


_lib = None


def load_library(path: str = LIB_PATH) -> C.CDLL:
    """dlopen the library (works without a GPU; calls then fail with MG_ERR_CUDA)."""
    global _lib
    if _lib is None:
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run `python -m paper_2202_02365_b200.build` "
                               "(there is no fallback implementation)")
        _lib = C.CDLL(path)
        _lib.mg_last_error.restype = C.c_char_p
        _lib.mg_kernel_launches.restype = C.c_int64
    return _lib


def _ptr(t: torch.Tensor | None):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


def _host(x, dtype) -> torch.Tensor:
    t = torch.as_tensor(x, dtype=dtype)
    return t.cpu().contiguous()


def comet_plan(p: int, l: int, c_l: int, seed: int):
    """One epoch's COMET plan (host-side, no GPU needed): logical grouping, the sequence of resident sets of
    logical partitions, the set that trains each edge bucket, and the resident physical partitions of each set."""
    lib = load_library()
    cap = max(1, l * l)
    lop = np.zeros(p, dtype=np.int32)
    sets = np.zeros((cap, c_l), dtype=np.int32)
    buckets = np.zeros((p, p), dtype=np.int32)
    n = C.c_int32(0)
    rc = lib.mg_comet_plan(C.c_int32(p), C.c_int32(l), C.c_int32(c_l), C.c_uint64(int(seed) & 0xFFFFFFFFFFFFFFFF), C.c_int32(cap),
                           C.c_void_p(lop.ctypes.data), C.byref(n), C.c_void_p(sets.ctypes.data), C.c_void_p(buckets.ctypes.data))
    if rc != MG_OK:
        raise MgError(rc, "mg_comet_plan")
    sets = sets[:n.value].copy()
    physical = [sorted(int(q) for q in range(p) if lop[q] in set(s.tolist())) for s in sets]
    return {"logical_of_physical": lop, "sets": sets, "bucket_set": buckets, "physical_sets": physical}


def comet_bias(bucket_set: np.ndarray, n_sets: int) -> float:
    lib = load_library()
    b = np.ascontiguousarray(bucket_set, dtype=np.int32)
    out = C.c_double(0.0)
    rc = lib.mg_comet_bias(C.c_int32(b.shape[0]), C.c_int32(n_sets), C.c_void_p(b.ctypes.data), C.byref(out))
    if rc != MG_OK:
        raise MgError(rc, "mg_comet_bias")
    return out.value


def comet_autotune(n_nodes: int, dim: int, n_edges: int, bytes_per_edge: int, cpu_bytes: int, block_bytes: int,
                   fudge_bytes: int, max_parts: int):
    lib = load_library()
    p, l, c = C.c_int32(0), C.c_int32(0), C.c_int32(0)
    rc = lib.mg_comet_autotune(C.c_int64(n_nodes), C.c_int32(dim), C.c_int64(n_edges), C.c_int32(bytes_per_edge),
                               C.c_int64(cpu_bytes), C.c_int64(block_bytes), C.c_int64(fudge_bytes), C.c_int32(max_parts),
                               C.byref(p), C.byref(l), C.byref(c))
    if rc != MG_OK:
        raise MgError(rc, "mg_comet_autotune")
    return p.value, l.value, c.value


class _DeviceInts:
    """A library-owned device buffer of n int32 values, exposed through the CUDA array interface."""

    def __init__(self, ptr: int, n: int):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": "<i4", "data": (int(ptr), False), "version": 2}


def _from_dev(ptr, n: int, device) -> torch.Tensor:
    """Copy n int32 values out of a library-owned device buffer into a torch tensor."""
    if n == 0 or not ptr:
        return torch.empty(0, dtype=torch.int32, device=device)
    return torch.as_tensor(_DeviceInts(ptr, n), device=device).clone()


class _DeviceFloats:
    def __init__(self, ptr: int, n: int):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": "<f4", "data": (int(ptr), False), "version": 2}


def _from_dev_f32(ptr, n: int, device) -> torch.Tensor:
    """View n float32 values of a library-owned device buffer (the caller clones what it keeps)."""
    if n == 0 or not ptr:
        return torch.empty(0, dtype=torch.float32, device=device)
    return torch.as_tensor(_DeviceFloats(ptr, n), device=device)


@dataclass
class DenseView:
    """One batch's DENSE in the paper's layout (device int32 tensors)."""
    node_ids: torch.Tensor
    node_id_offsets: torch.Tensor
    nbrs: torch.Tensor
    nbr_offsets: torch.Tensor
    repr_map: torch.Tensor


class Dense:
    def __init__(self, ctx: "Context"):
        self.ctx = ctx
        self.handle = C.c_void_p(0)
        ctx._children.add(self)

    def counts(self):
        lib = self.ctx.lib
        nb, k = C.c_int32(0), C.c_int32(0)
        self.ctx._check(lib.mg_dense_counts(self.handle, C.byref(nb), C.byref(k), None, None))
        nodes = torch.zeros((nb.value, k.value + 1), dtype=torch.int64)
        ents = torch.zeros((nb.value, k.value), dtype=torch.int64)
        self.ctx._check(lib.mg_dense_counts(self.handle, None, None, _ptr(nodes), _ptr(ents)))
        return nodes, ents

    def view(self, batch: int = 0) -> DenseView:
        arr = DenseArrays()
        self.ctx._check(self.ctx.lib.mg_dense_view(self.ctx.handle, self.handle, C.c_int32(batch), C.byref(arr)))
        dev = self.ctx.device
        return DenseView(
            _from_dev(arr.node_ids, arr.n_nodes, dev), _from_dev(arr.node_id_offsets, arr.k + 2, dev),
            _from_dev(arr.nbrs, arr.n_entries, dev), _from_dev(arr.nbr_offsets, arr.n_sampled + 1, dev),
            _from_dev(arr.repr_map, arr.n_entries, dev))

    def export_many(self):
        """Queue the export of every mini-batch into the paper's arrays (asynchronous, on the sampling stream)."""
        self.ctx._check(self.ctx.lib.mg_dense_export_many(self.ctx.handle, self.handle))

    def export_view(self, batch: int = 0) -> DenseView:
        """Mini-batch `batch` of the last export_many (waits for it the first time)."""
        arr = DenseArrays()
        self.ctx._check(self.ctx.lib.mg_dense_export_view(self.ctx.handle, self.handle, C.c_int32(batch), C.byref(arr)))
        dev = self.ctx.device
        return DenseView(
            _from_dev(arr.node_ids, arr.n_nodes, dev), _from_dev(arr.node_id_offsets, arr.k + 2, dev),
            _from_dev(arr.nbrs, arr.n_entries, dev), _from_dev(arr.nbr_offsets, arr.n_sampled + 1, dev),
            _from_dev(arr.repr_map, arr.n_entries, dev))

    def free(self):
        if self.handle:
            self.ctx.lib.mg_dense_free(self.handle)
            self.handle = C.c_void_p(0)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class Model:
    def __init__(self, ctx: "Context", layers, precision: int = GEMM_TF32):
        self.ctx = ctx
        self.handle = C.c_void_p(0)
        ctx._children.add(self)
        k = len(layers)
        self.dims = [int(layers[0][0].shape[0])] + [int(l[0].shape[1]) for l in layers]
        keep = []
        arrs = []
        for idx in range(3):
            ptrs = (C.c_void_p * k)()
            for i, l in enumerate(layers):
                t = _host(l[idx], torch.float32)
                keep.append(t)
                ptrs[i] = t.data_ptr()
            arrs.append(ptrs)
        dims = (C.c_int32 * (k + 1))(*self.dims)
        ctx._check(ctx.lib.mg_model_create(ctx.handle, C.c_int32(k), dims, arrs[0], arrs[1], arrs[2],
                                           C.c_int(precision), C.byref(self.handle)))

    def set_intermediates(self, dtype):
        """torch.float16: keep H^1 .. H^{k-1} as fp16 inside forward (where the model allows it); torch.float32: default."""
        code = {torch.float32: DTYPE_F32, torch.float16: DTYPE_F16}[dtype]
        self.ctx._check(self.ctx.lib.mg_model_set_intermediates(self.handle, C.c_int(code)))

    def set_aggregator(self, aggregator: str):
        """"mean" (GraphSage's mean over the sampled neighbours, the default) or "sum"."""
        self.ctx._check(self.ctx.lib.mg_model_set_aggregator(self.handle, C.c_int({"mean": 0, "sum": 1}[aggregator])))

    def free(self):
        if self.handle:
            self.ctx.lib.mg_model_free(self.handle)
            self.handle = C.c_void_p(0)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class GatModel:
    """layers: list of (w [d_in, d_out], a_src [d_out], a_dst [d_out], bias [d_out]) host tensors."""

    def __init__(self, ctx: "Context", layers, precision: int = GEMM_TF32, negative_slope: float = 0.2):
        self.ctx = ctx
        self.handle = C.c_void_p(0)
        k = len(layers)
        self.dims = [int(layers[0][0].shape[0])] + [int(l[0].shape[1]) for l in layers]
        keep, arrs = [], []
        for idx in range(4):
            ptrs = (C.c_void_p * k)()
            for i, l in enumerate(layers):
                t = _host(l[idx], torch.float32)
                keep.append(t)
                ptrs[i] = t.data_ptr()
            arrs.append(ptrs)
        dims = (C.c_int32 * (k + 1))(*self.dims)
        ctx._check(ctx.lib.mg_gat_model_create(ctx.handle, C.c_int32(k), dims, arrs[0], arrs[1], arrs[2], arrs[3],
                                               C.c_float(negative_slope), C.c_int(precision), C.byref(self.handle)))

    def set_heads(self, heads: int):
        """Attention heads per layer: equal column blocks of every layer's width, concatenated."""
        self.ctx._check(self.ctx.lib.mg_gat_model_set_heads(self.handle, C.c_int32(heads)))

    def free(self):
        if self.handle:
            self.ctx.lib.mg_gat_model_free(self.handle)
            self.handle = C.c_void_p(0)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class LpBatch:
    def __init__(self, ctx: "Context"):
        self.ctx = ctx
        self.handle = C.c_void_p(0)
        ctx._children.add(self)
        self.n_edges = 0
        self.negs = 0

    def targets(self) -> torch.Tensor:
        """The batch's target union (distinct ids, ascending) alone: what the sampler is called with."""
        n = C.c_int32(0)
        p = C.c_void_p(0)
        self.ctx._check(self.ctx.lib.mg_lp_view(self.handle, C.byref(n), C.byref(p), None, None, None, None))
        return _from_dev(p.value, n.value, self.ctx.device)

    def view(self):
        n = C.c_int32(0)
        p = [C.c_void_p(0) for _ in range(5)]
        self.ctx._check(self.ctx.lib.mg_lp_view(self.handle, C.byref(n), *[C.byref(x) for x in p]))
        dev = self.ctx.device
        nt = n.value
        return {
            "targets": _from_dev(p[0].value, nt, dev), "src_idx": _from_dev(p[1].value, self.n_edges, dev),
            "dst_idx": _from_dev(p[2].value, self.n_edges, dev),
            "neg_ids": _from_dev(p[3].value, self.n_chunks * self.negs, dev).view(self.n_chunks, self.negs),
            "neg_idx": _from_dev(p[4].value, self.n_chunks * self.negs, dev).view(self.n_chunks, self.negs),
        }

    def free(self):
        if self.handle:
            self.ctx.lib.mg_lp_free(self.handle)
            self.handle = C.c_void_p(0)

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class Context:
    """One device, one stream.  Mirrors the C calls one to one."""

    def __init__(self, device: int = 0, stream: torch.cuda.Stream | None = None):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("mgdense needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", device)
        self.stream = stream
        self.handle = C.c_void_p(0)
        self._children = weakref.WeakSet()
        sptr = C.c_void_p(stream.cuda_stream if stream is not None else 0)
        rc = self.lib.mg_create(C.byref(self.handle), C.c_int(device), sptr)
        if rc != MG_OK:
            raise MgError(rc, "mg_create failed")
        self._keep = {}

    # -- plumbing
    def _check(self, rc: int):
        if rc != MG_OK:
            msg = self.lib.mg_last_error(self.handle)
            raise MgError(rc, msg.decode() if msg else "")

    def close(self):
        if self.handle:
            for child in list(self._children):
                child.free()
            self.lib.mg_destroy(self.handle)
            self.handle = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def kernel_launches(self) -> int:
        return int(self.lib.mg_kernel_launches(self.handle))

    def profile(self, on: bool):
        self._check(self.lib.mg_profile(self.handle, C.c_int(1 if on else 0)))

    def profile_read(self, reset: bool = True):
        n = C.c_int32(0)
        names = (C.c_char_p * 32)()
        ms = (C.c_double * 32)()
        launches = (C.c_int64 * 32)()
        self._check(self.lib.mg_profile_read(self.handle, C.byref(n), names, ms, launches, C.c_int(1 if reset else 0)))
        return {names[i].decode(): {"ms": ms[i], "launches": launches[i]} for i in range(n.value)}

    # -- graph store and buffer
    def load_graph(self, row_offsets: torch.Tensor, nbrs: torch.Tensor):
        assert row_offsets.dtype in (torch.int32, torch.int64) and nbrs.dtype == torch.int32
        assert row_offsets.is_cuda == nbrs.is_cuda
        row_offsets, nbrs = row_offsets.contiguous(), nbrs.contiguous()
        n_nodes, n_edges = row_offsets.numel() - 1, nbrs.numel()
        self._check(self.lib.mg_load_graph(self.handle, C.c_int64(n_nodes), C.c_int64(n_edges), _ptr(row_offsets),
                                           C.c_int(row_offsets.dtype == torch.int64), _ptr(nbrs),
                                           C.c_int(row_offsets.is_cuda)))
        self.n_nodes = n_nodes

    def load_out_graph(self, row_offsets: torch.Tensor, nbrs: torch.Tensor):
        """Second edge list (rows by source) for incoming + outgoing sampling."""
        assert row_offsets.dtype in (torch.int32, torch.int64) and nbrs.dtype == torch.int32
        assert row_offsets.is_cuda == nbrs.is_cuda
        row_offsets, nbrs = row_offsets.contiguous(), nbrs.contiguous()
        assert row_offsets.numel() - 1 == self.n_nodes
        self._check(self.lib.mg_load_out_graph(self.handle, C.c_int64(nbrs.numel()), _ptr(row_offsets),
                                               C.c_int(row_offsets.dtype == torch.int64), _ptr(nbrs),
                                               C.c_int(row_offsets.is_cuda)))

    def set_sample_direction(self, direction: str):
        self._check(self.lib.mg_set_sample_direction(self.handle, C.c_int({"in": 0, "inout": 1}[direction])))

    def set_partitioning(self, n_parts: int, part_of_node: torch.Tensor | None = None):
        """part_of_node: optional uint8 partition id per node (host); None = contiguous equal id ranges."""
        pn = None if part_of_node is None else part_of_node.to(torch.uint8).cpu().contiguous()
        self._check(self.lib.mg_set_partitioning(self.handle, C.c_int32(n_parts), _ptr(pn)))

    def load_features(self, table: torch.Tensor | None, capacity_parts: int = 1, backing: int = BACKING_HBM, dtype=None, dim=None):
        """table = None (host backing only): no whole table exists; give dtype and dim, and name every partition's
        host block with set_partition_source before asking for it."""
        if table is None:
            dt = {torch.float32: DTYPE_F32, torch.float16: DTYPE_F16}[dtype]
            self._check(self.lib.mg_load_features(self.handle, None, C.c_int(0), C.c_int(dt), C.c_int32(dim),
                                                  C.c_int32(capacity_parts), C.c_int(backing)))
            return
        assert table.dim() == 2 and table.is_contiguous()
        dt = {torch.float32: DTYPE_F32, torch.float16: DTYPE_F16}[table.dtype]
        self._keep["features"] = table          # device tables are borrowed, host tables stay the backing store
        self._check(self.lib.mg_load_features(self.handle, _ptr(table), C.c_int(table.is_cuda), C.c_int(dt),
                                              C.c_int32(table.shape[1]), C.c_int32(capacity_parts), C.c_int(backing)))

    def set_partition_source(self, part: int, block: torch.Tensor | None):
        """Partition `part`'s rows are in `block` (host tensor, preferably pinned; kept alive by this context)."""
        if block is not None:
            assert not block.is_cuda and block.is_contiguous()
            self._keep[("source", part)] = block
        self._check(self.lib.mg_set_partition_source(self.handle, C.c_int32(part), _ptr(block)))

    def set_resident(self, parts, async_: bool = False):
        p = _host(list(parts), torch.int32)
        self._check(self.lib.mg_set_resident(self.handle, _ptr(p), C.c_int32(p.numel()), C.c_int(1 if async_ else 0)))

    def commit_resident(self, timeout_ms: int = 60000):
        self._check(self.lib.mg_commit_resident(self.handle, C.c_int32(timeout_ms)))

    def backward(self, model: "Model", dense: "Dense", d_out: torch.Tensor, want_h0_grad: bool = False):
        """Gradients through the last forward(model, dense) (keep_layer_outputs(True) must be set).  Returns the list of
        (dW_self, dW_nbr, dbias) device tensors per layer and, on request, (dH0 rows, their node ids)."""
        assert d_out.is_cuda and d_out.dtype == torch.float32 and d_out.is_contiguous()
        nodes, _ = dense.counts()
        n_rows = int(nodes.sum())
        g_h0 = torch.empty((n_rows, model.dims[0]), dtype=torch.float32, device=d_out.device) if want_h0_grad else None
        self._check(self.lib.mg_backward(self.handle, model.handle, dense.handle, _ptr(d_out), _ptr(g_h0)))
        grads = []
        for l in range(1, len(model.dims)):
            ps, pn, pb = C.c_void_p(0), C.c_void_p(0), C.c_void_p(0)
            self._check(self.lib.mg_model_grads(model.handle, C.c_int32(l), C.byref(ps), C.byref(pn), C.byref(pb)))
            di, dn = model.dims[l - 1], model.dims[l]
            grads.append((_from_dev_f32(ps.value, di * dn, d_out.device).view(di, dn).clone(),
                          _from_dev_f32(pn.value, di * dn, d_out.device).view(di, dn).clone(),
                          _from_dev_f32(pb.value, dn, d_out.device).clone()))
        if not want_h0_grad:
            return grads
        ids = torch.empty(n_rows, dtype=torch.int32, device=d_out.device)
        self._check(self.lib.mg_dense_packed_ids(self.handle, dense.handle, _ptr(ids)))
        return grads, g_h0, ids

    def apply_embedding_sgd(self, dense: "Dense", g_h0: torch.Tensor, lr: float):
        assert g_h0.is_cuda and g_h0.dtype == torch.float32 and g_h0.is_contiguous()
        self._check(self.lib.mg_apply_embedding_sgd(self.handle, dense.handle, _ptr(g_h0), C.c_float(lr)))

    def adagrad_step(self, model: "Model", lr: float, eps: float = 1e-10):
        self._check(self.lib.mg_model_adagrad_step(self.handle, model.handle, C.c_float(lr), C.c_float(eps)))

    def sgd_step(self, model: "Model", lr: float):
        self._check(self.lib.mg_model_sgd_step(self.handle, model.handle, C.c_float(lr)))

    def gat_model(self, layers, precision: int = GEMM_TF32, negative_slope: float = 0.2) -> "GatModel":
        return GatModel(self, layers, precision, negative_slope)

    def gat_forward(self, model: "GatModel", dense: "Dense", out: torch.Tensor):
        assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous()
        self._check(self.lib.mg_gat_forward(self.handle, model.handle, dense.handle, _ptr(out)))

    # -- sampling
    def _sample_many_call(self, fn, targets, target_offsets, fanouts, seeds, caps, out):
        assert targets.dtype == torch.int32
        targets = targets.contiguous()
        offs = _host(target_offsets, torch.int64)
        fo = _host(list(fanouts), torch.int32)
        sd = np.ascontiguousarray(np.array([int(s) & 0xFFFFFFFFFFFFFFFF for s in seeds], dtype=np.uint64))
        d = out if out is not None else Dense(self)
        cp = None
        if caps is not None:
            cp = SampleCaps(int(caps.get("max_nodes_total", 0)), int(caps.get("max_entries_total", 0)),
                            int(caps.get("max_nodes_per_batch", 0)), int(caps.get("max_inner_nodes_per_batch", 0)))
        self._check(fn(self.handle, _ptr(targets), C.c_int(targets.is_cuda), _ptr(offs),
                       C.c_int32(offs.numel() - 1), _ptr(fo), C.c_int32(fo.numel()), C.c_void_p(sd.ctypes.data),
                       C.byref(cp) if cp is not None else None, C.byref(d.handle)))
        d._targets_keepalive = targets     # device targets must outlive the queued kernels
        return d

    def sample_many(self, targets: torch.Tensor, target_offsets, fanouts, seeds, caps=None, out: Dense | None = None) -> Dense:
        return self._sample_many_call(self.lib.mg_sample_many, targets, target_offsets, fanouts, seeds, caps, out)

    def sample_many_begin(self, targets: torch.Tensor, target_offsets, fanouts, seeds, caps=None, out: Dense | None = None) -> Dense:
        """Queue a sample on the sampling stream; finish it with sample_many_end(dense)."""
        return self._sample_many_call(self.lib.mg_sample_many_begin, targets, target_offsets, fanouts, seeds, caps, out)

    def sample_many_end(self, dense: Dense):
        self._check(self.lib.mg_sample_many_end(self.handle, dense.handle))

    def sample(self, targets: torch.Tensor, fanouts, seed: int, caps=None, out: Dense | None = None) -> Dense:
        assert targets.dtype == torch.int32
        targets = targets.contiguous()
        fo = _host(list(fanouts), torch.int32)
        d = out if out is not None else Dense(self)
        cp = None
        if caps is not None:
            cp = SampleCaps(int(caps.get("max_nodes_total", 0)), int(caps.get("max_entries_total", 0)),
                            int(caps.get("max_nodes_per_batch", 0)), int(caps.get("max_inner_nodes_per_batch", 0)))
        self._check(self.lib.mg_sample(self.handle, _ptr(targets), C.c_int(targets.is_cuda), C.c_int32(targets.numel()),
                                       _ptr(fo), C.c_int32(fo.numel()), C.c_uint64(int(seed) & 0xFFFFFFFFFFFFFFFF),
                                       C.byref(cp) if cp is not None else None, C.byref(d.handle)))
        return d

    # -- forward
    def model(self, layers, precision: int = GEMM_TF32) -> Model:
        return Model(self, layers, precision)

    def forward(self, model: Model, dense: Dense, out: torch.Tensor) -> torch.Tensor:
        assert out.dtype == torch.float32 and out.is_contiguous()
        self._check(self.lib.mg_forward(self.handle, model.handle, dense.handle, _ptr(out), C.c_int(out.is_cuda)))
        return out

    def set_layer_window(self, mini_batches: int):
        self._check(self.lib.mg_set_layer_window(self.handle, C.c_int32(mini_batches)))

    def keep_layer_outputs(self, on: bool = True):
        self._check(self.lib.mg_keep_layer_outputs(self.handle, C.c_int(1 if on else 0)))

    def forward_host_async(self, model: Model, dense: Dense, out: torch.Tensor) -> torch.Tensor:
        """mg_forward_host_async: `out` (pinned CPU tensor) is valid after wait_output()."""
        assert out.dtype == torch.float32 and out.is_contiguous() and not out.is_cuda
        self._check(self.lib.mg_forward_host_async(self.handle, model.handle, dense.handle, _ptr(out)))
        return out

    def wait_output(self):
        self._check(self.lib.mg_wait_output(self.handle))

    def forward_noalloc(self, model: Model, dense: Dense, out: torch.Tensor) -> torch.Tensor:
        """mg_forward_noalloc: same result as forward(), all temporaries in the library's built-in
        scratch array, no device allocation.  `out` must be a CUDA tensor."""
        assert out.dtype == torch.float32 and out.is_contiguous() and out.is_cuda
        self._check(self.lib.mg_forward_noalloc(self.handle, model.handle, dense.handle, _ptr(out)))
        return out

    def gather_h0(self, dense: Dense, batch: int, n_nodes: int, dim: int) -> torch.Tensor:
        out = torch.empty((n_nodes, dim), dtype=torch.float32, device=self.device)
        self._check(self.lib.mg_gather_h0(self.handle, dense.handle, C.c_int32(batch), _ptr(out)))
        return out

    def layer_output(self, model: Model, dense: Dense, layer: int, batch: int, n_rows: int) -> torch.Tensor:
        out = torch.empty((n_rows, model.dims[layer]), dtype=torch.float32, device=self.device)
        self._check(self.lib.mg_layer_output(self.handle, model.handle, dense.handle, C.c_int32(layer),
                                             C.c_int32(batch), _ptr(out)))
        return out

    # -- link prediction
    def lp_prepare(self, src, rel, dst, n_chunks: int, negs_per_chunk: int, seed: int) -> LpBatch:
        s, r, d = _host(src, torch.int32), _host(rel, torch.int32), _host(dst, torch.int32)
        lp = LpBatch(self)
        lp.n_edges, lp.negs, lp.n_chunks = s.numel(), negs_per_chunk, n_chunks
        self._check(self.lib.mg_lp_prepare(self.handle, _ptr(s), _ptr(r), _ptr(d), C.c_int64(s.numel()),
                                           C.c_int32(n_chunks), C.c_int32(negs_per_chunk),
                                           C.c_uint64(int(seed) & 0xFFFFFFFFFFFFFFFF), C.byref(lp.handle)))
        return lp

    def distmult_score(self, lp: LpBatch, h: torch.Tensor, rel_emb: torch.Tensor, corrupt: int = CORRUPT_BOTH,
                       precision: int = GEMM_TF32):
        assert h.is_cuda and rel_emb.is_cuda and h.dtype == torch.float32 and rel_emb.dtype == torch.float32
        h, rel_emb = h.contiguous(), rel_emb.contiguous()
        pos = torch.empty(lp.n_edges, dtype=torch.float32, device=self.device)
        nd = torch.empty((lp.n_edges, lp.negs), dtype=torch.float32, device=self.device) if corrupt & CORRUPT_DST else None
        ns = torch.empty((lp.n_edges, lp.negs), dtype=torch.float32, device=self.device) if corrupt & CORRUPT_SRC else None
        self._check(self.lib.mg_distmult_score(self.handle, lp.handle, _ptr(h), C.c_int32(h.shape[1]), _ptr(rel_emb),
                                               C.c_int32(rel_emb.shape[0]), C.c_int(corrupt), C.c_int(precision), _ptr(pos), _ptr(nd), _ptr(ns)))
        return pos, nd, ns
