"""Partitioned execution (Sec. 4 of the paper) over the C ABI of include/ripple_part.h.

Argument marshalling and sequencing only: routing runs in the library's router (host code), every step
of a hop in the library's kernels.  Two ways to run the workers:

  Cluster          all workers in this process (one context each, on the current device or on the
                   devices given): peers are registered by device address.  This is also how the
                   multi-worker path is exercised on a single GPU: the phases run one worker after the
                   other, nothing waits on the device.
  DistributedWorker  one worker per process (one process per GPU, torch.distributed for the barriers
                   and for handing out the CUDA IPC handles); every process runs its own replica of
                   the router on the same batches.
"""
from __future__ import annotations

import ctypes
from typing import List, Optional, Sequence, Tuple

import numpy as np

from . import ripple as R

ROUTE_LOCALITY, ROUTE_HASH = 0, 1


class Router:
    """Vertex-partition map, placement of new vertices (Alg. 1 or hashing), routing of updates and
    global-to-local id translation (Sec. 4.3, 4.4)."""

    def __init__(self, n_partitions: int, owner: np.ndarray, src: np.ndarray, dst: np.ndarray,
                 routing: int = ROUTE_LOCALITY, hd_refresh: int = 500_000, spare_local: int = 0,
                 halo_capacity: Optional[int] = None):
        self.lib = R.load_library()
        self.P = int(n_partitions)
        owner = np.ascontiguousarray(owner, dtype=np.int32)
        src = np.ascontiguousarray(src, dtype=np.int32)
        dst = np.ascontiguousarray(dst, dtype=np.int32)
        self.n = owner.size
        if halo_capacity is None:
            halo_capacity = self.n
        self.h = ctypes.c_void_p(None)
        st = self.lib.ripple_router_create(self.P, self.n, owner.ctypes.data, src.size, src.ctypes.data,
                                           dst.ctypes.data, int(routing), int(hd_refresh), int(spare_local),
                                           int(halo_capacity), ctypes.byref(self.h))
        if st != R.OK:
            raise R.RippleError(st, "router creation failed")

    def close(self):
        if getattr(self, "h", None) and self.h.value:
            self.lib.ripple_router_destroy(self.h)
            self.h = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def partition(self, rank: int):
        """(n_local, num_vertices, src_local, dst_local, global_of, halo_owner, halo_remote_id, edge_of):
        edge_of[i] = index, in the arrays the router was created from, of the edge behind local edge i."""
        a, b, c, d = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
        st = self.lib.ripple_router_partition_shape(self.h, rank, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c),
                                                    ctypes.byref(d))
        if st != R.OK:
            raise R.RippleError(st, "partition shape")
        src = np.zeros(max(c.value, 1), dtype=np.int32)
        dst = np.zeros(max(c.value, 1), dtype=np.int32)
        gof = np.zeros(b.value, dtype=np.int32)
        ho = np.zeros(max(d.value, 1), dtype=np.int32)
        hr = np.zeros(max(d.value, 1), dtype=np.int32)
        eof = np.zeros(max(c.value, 1), dtype=np.int64)
        st = self.lib.ripple_router_partition_fill(self.h, rank, src.ctypes.data, dst.ctypes.data, eof.ctypes.data,
                                                   gof.ctypes.data, ho.ctypes.data, hr.ctypes.data)
        if st != R.OK:
            raise R.RippleError(st, "partition fill")
        return a.value, b.value, src[: c.value], dst[: c.value], gof, ho[: d.value], hr[: d.value], eof[: c.value]

    def route(self, ups: np.ndarray) -> None:
        ups = np.ascontiguousarray(ups, dtype=R.UPDATE_DTYPE)
        st = self.lib.ripple_router_route(self.h, ups.ctypes.data, ups.size)
        if st != R.OK:
            raise R.RippleError(st, "routing failed")

    def batch(self, rank: int):
        """(ups_local, no_compute, row_of, first_halo, halo_owner, halo_remote_id, op_of) of the routed batch;
        op_of[i] = position in the batch of the operation that local operation i comes from."""
        a, b, c = ctypes.c_int64(), ctypes.c_int64(), ctypes.c_int64()
        st = self.lib.ripple_router_batch_shape(self.h, rank, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
        if st != R.OK:
            raise R.RippleError(st, "batch shape")
        ups = np.zeros(max(a.value, 1), dtype=R.UPDATE_DTYPE)
        nc = np.zeros(max(a.value, 1), dtype=np.uint8)
        row_of = np.zeros(max(b.value, 1), dtype=np.int32)
        ho = np.zeros(max(c.value, 1), dtype=np.int32)
        hr = np.zeros(max(c.value, 1), dtype=np.int32)
        first = ctypes.c_int32()
        op_of = np.zeros(max(a.value, 1), dtype=np.int32)
        st = self.lib.ripple_router_batch_fill(self.h, rank, ups.ctypes.data, nc.ctypes.data, op_of.ctypes.data,
                                               row_of.ctypes.data, ctypes.byref(first), ho.ctypes.data, hr.ctypes.data)
        if st != R.OK:
            raise R.RippleError(st, "batch fill")
        return (ups[: a.value], nc[: a.value], row_of[: b.value], first.value, ho[: c.value], hr[: c.value],
                op_of[: a.value])

    def global_ids(self, rank: int, num_vertices: int) -> np.ndarray:
        """The global id behind every local id of worker `rank` (locals, then halo slots; -1: unused)."""
        out = np.zeros(int(num_vertices), dtype=np.int32)
        st = self.lib.ripple_router_global_ids(self.h, int(rank), out.ctypes.data, out.size)
        if st != R.OK:
            raise R.RippleError(st, "global ids")
        return out

    def owner(self, v: int) -> int:
        return int(self.lib.ripple_router_owner(self.h, int(v)))

    def local_id(self, v: int) -> int:
        return int(self.lib.ripple_router_local_id(self.h, int(v)))

    def global_id(self, rank: int, local_id: int) -> int:
        return int(self.lib.ripple_router_global_id(self.h, int(rank), int(local_id)))

    def is_high_degree(self, v: int) -> bool:
        return bool(self.lib.ripple_router_is_high_degree(self.h, int(v)))

    def load(self, rank: int) -> int:
        return int(self.lib.ripple_router_load(self.h, int(rank)))


class Worker(R.Ripple):
    """One partition's context (ids are local ids) with the phase calls of a partitioned batch."""

    def exports(self) -> "R._PartExports":
        e = R._PartExports()
        self._check(self.lib.ripple_part_exports_get(self.h, ctypes.byref(e)))
        return e

    def set_peer(self, rank: int, e) -> None:
        self._check(self.lib.ripple_part_set_peer(self.h, int(rank), ctypes.byref(e)))

    def ipc_export(self) -> bytes:
        e = R._PartIpc()
        self._check(self.lib.ripple_part_ipc_export(self.h, ctypes.byref(e)))
        return bytes(e)

    def ipc_open(self, rank: int, blob: bytes) -> None:
        e = R._PartIpc.from_buffer_copy(blob)
        self._check(self.lib.ripple_part_ipc_open(self.h, int(rank), ctypes.byref(e)))

    def set_halos(self, first: int, owner: np.ndarray, remote_id: np.ndarray) -> None:
        owner = np.ascontiguousarray(owner, dtype=np.int32)
        remote_id = np.ascontiguousarray(remote_id, dtype=np.int32)
        self._check(self.lib.ripple_part_set_halos(self.h, int(first), owner.size, owner.ctypes.data, remote_id.ctypes.data))

    def bootstrap_layer(self, l: int) -> None:
        self._check(self.lib.ripple_part_bootstrap_layer(self.h, int(l)))

    def begin(self, ups: np.ndarray, rows: Optional[np.ndarray], no_compute: np.ndarray,
              op_weights: Optional[np.ndarray] = None) -> None:
        ups = np.ascontiguousarray(ups, dtype=R.UPDATE_DTYPE)
        no_compute = np.ascontiguousarray(no_compute, dtype=np.uint8)
        wptr = None
        if op_weights is not None and ups.size:
            op_weights = np.ascontiguousarray(op_weights, dtype=np.float32)
            wptr = op_weights.ctypes.data
        nr, fptr = 0, None
        if rows is not None and rows.shape[0]:
            rows = np.ascontiguousarray(rows, dtype=np.float32)
            nr, fptr = rows.shape[0], rows.ctypes.data
        self._check(self.lib.ripple_part_begin(self.h, ups.ctypes.data if ups.size else None, ups.size, fptr, nr,
                                               no_compute.ctypes.data if ups.size else None, wptr, R.MEM_HOST))

    def hop_send(self, l: int) -> None:
        self._check(self.lib.ripple_part_hop_send(self.h, int(l)))

    def hop_compute(self, l: int) -> None:
        self._check(self.lib.ripple_part_hop_compute(self.h, int(l)))

    def end(self) -> None:
        self._check(self.lib.ripple_part_end(self.h))

    def rows_sent(self) -> List[int]:
        out = np.zeros(R.MAX_LAYERS + 1, dtype=np.int64)
        self._check(self.lib.ripple_part_rows_sent(self.h, out.ctypes.data))
        return out[: self.L + 1].tolist()


def payload_rows(rows: Optional[np.ndarray], row_of: np.ndarray, d0: int) -> Optional[np.ndarray]:
    """A worker's payload rows: copies of the batch's rows, zeros where the router says -1 (the feature row
    of a deleted vertex)."""
    if not row_of.size:
        return None
    out = np.zeros((row_of.size, d0), dtype=np.float32)
    keep = row_of >= 0
    if keep.any():
        out[keep] = rows[row_of[keep]]
    return out


def _make_worker(router: Router, rank: int, X: np.ndarray, model, weights, edge_weights=None, **kw) -> Tuple[Worker, np.ndarray]:
    n_local, nv, src, dst, gof, ho, hr, edge_of = router.partition(rank)
    if edge_weights is not None:      # a cut edge is held, with its weight, by both of its workers
        kw["edge_weights"] = np.ascontiguousarray(edge_weights, dtype=np.float32)[edge_of]
    feats = np.zeros((nv, X.shape[1]), dtype=np.float32)
    own = gof[:n_local]
    feats[: n_local][own >= 0] = X[own[own >= 0]]
    w = Worker(nv, src, dst, feats, model, weights, n_local=n_local, **kw)
    if ho.size:
        w.set_halos(0, ho, hr)
    return w, gof


class Cluster:
    """All workers of a partitioned execution in one process.  `devices`: one CUDA device ordinal per
    worker (default: all on the current device)."""

    def __init__(self, n_partitions: int, owner: np.ndarray, src: np.ndarray, dst: np.ndarray, X: np.ndarray,
                 model, weights, routing: int = ROUTE_LOCALITY, hd_refresh: int = 500_000, spare_local: int = 0,
                 halo_capacity: Optional[int] = None, devices: Optional[Sequence[int]] = None, edge_weights=None, **kw):
        import torch
        self._torch = torch
        self.P = int(n_partitions)
        self.L = len(model.layers)
        self.model = model
        self.router = Router(self.P, owner, src, dst, routing, hd_refresh, spare_local, halo_capacity)
        self.devices = list(devices) if devices is not None else [torch.cuda.current_device()] * self.P
        self.workers: List[Worker] = []
        for r in range(self.P):
            with torch.cuda.device(self.devices[r]):
                w, _ = _make_worker(self.router, r, X, model, weights, edge_weights=edge_weights, **kw)
            self.workers.append(w)
        exports = [w.exports() for w in self.workers]
        for w in self.workers:
            for r, e in enumerate(exports):
                w.set_peer(r, e)
        for l in range(1, self.L + 1):      # every worker finishes a layer before any starts the next
            for w in self.workers:
                w.bootstrap_layer(l)

    def recompute_full(self) -> None:
        """Layer-wise inference on the current graph on every worker (between two batches): all cached rows anew."""
        for l in range(1, self.L + 1):
            for w in self.workers:
                w.bootstrap_layer(l)

    def close(self):
        for w in self.workers:
            w.close()
        self.router.close()

    def apply_batch(self, ups: np.ndarray, rows: Optional[np.ndarray], op_weights: Optional[np.ndarray] = None) -> None:
        """ups in global ids (op_weights: the weight of every added edge, graphs with stored edge weights).  Every
        phase runs on all workers before the next begins."""
        self.router.route(ups)
        for r, w in enumerate(self.workers):
            lu, nc, row_of, first, ho, hr, op_of = self.router.batch(r)
            if ho.size:
                w.set_halos(first, ho, hr)
            w.begin(lu, payload_rows(rows, row_of, w.dims[0]), nc,
                    np.asarray(op_weights, dtype=np.float32)[op_of] if op_weights is not None else None)
        for l in range(1, self.L + 1):
            for w in self.workers:
                w.hop_send(l)
            for w in self.workers:
                w.hop_compute(l)
        for w in self.workers:
            w.end()

    # ---- read-out in global ids ---------------------------------------------------------------
    def embeddings(self, l: int, n: int) -> np.ndarray:
        """H^l of every placed vertex (rows of unplaced ids are zero), gathered from the owners."""
        d = self.workers[0].dims[l]
        out = np.zeros((n, d), dtype=np.float32)
        for r, w in enumerate(self.workers):
            nl = w.n_local
            gof = self.router.global_ids(r, w.n)[:nl].astype(np.int64)
            h = w.embeddings(l)[:nl].cpu().numpy()
            out[gof[gof >= 0]] = h[gof >= 0]
        return out

    def affected(self, l: int) -> np.ndarray:
        ids = []
        for r, w in enumerate(self.workers):
            ids.append(self.router.global_ids(r, w.n)[w.affected(l).cpu().numpy()])
        return np.sort(np.concatenate(ids)).astype(np.int32)

    def rows_sent(self) -> List[int]:
        tot = np.zeros(self.L + 1, dtype=np.int64)
        for w in self.workers:
            tot += np.array(w.rows_sent())
        return tot.tolist()


class DistributedWorker:
    """One worker per process: `torch.distributed` must be initialised (one rank per GPU).  Every rank
    passes the same global graph description and the same batches; its router replica picks this
    rank's share.  Barriers separate the phases; peers are reached through CUDA IPC mappings."""

    def __init__(self, owner, src, dst, X, model, weights, routing: int = ROUTE_LOCALITY,
                 hd_refresh: int = 500_000, spare_local: int = 0, halo_capacity: Optional[int] = None,
                 edge_weights=None, **kw):
        import torch.distributed as dist
        self.dist = dist
        self.rank, self.P = dist.get_rank(), dist.get_world_size()
        self.L = len(model.layers)
        self.router = Router(self.P, owner, src, dst, routing, hd_refresh, spare_local, halo_capacity)
        self.worker, _ = _make_worker(self.router, self.rank, X, model, weights, edge_weights=edge_weights, **kw)
        blobs: List[Optional[bytes]] = [None] * self.P
        dist.all_gather_object(blobs, self.worker.ipc_export())
        for r, blob in enumerate(blobs):
            if r == self.rank:
                self.worker.set_peer(r, self.worker.exports())
            else:
                self.worker.ipc_open(r, blob)
        self.recompute_full()

    def recompute_full(self) -> None:
        """Layer-wise inference on the current graph, in step with the other ranks (the bootstrap; between two
        batches: every cached row anew).  Collective."""
        for l in range(1, self.L + 1):
            self.dist.barrier()
            self.worker.bootstrap_layer(l)
        self.dist.barrier()

    def apply_batch(self, ups: np.ndarray, rows: Optional[np.ndarray], op_weights: Optional[np.ndarray] = None) -> None:
        self.router.route(ups)
        lu, nc, row_of, first, ho, hr, op_of = self.router.batch(self.rank)
        if ho.size:
            self.worker.set_halos(first, ho, hr)
        self.worker.begin(lu, payload_rows(rows, row_of, self.worker.dims[0]), nc,
                          np.asarray(op_weights, dtype=np.float32)[op_of] if op_weights is not None else None)
        for l in range(1, self.L + 1):
            self.dist.barrier()
            self.worker.hop_send(l)
            self.dist.barrier()
            self.worker.hop_compute(l)
        self.dist.barrier()
        self.worker.end()

    def close(self):
        self.worker.close()
        self.router.close()
