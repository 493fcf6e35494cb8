"""CPU oracle of the distributed execution model (Sec. 4): a server that routes updates, workers that
each hold one partition, halo mailboxes with a combiner, one remote send per hop.

TEST INFRASTRUCTURE ONLY.  Plain NumPy in fp64, one Python object per worker, messages passed as
Python lists; it shares no code with the CUDA library and never imports it.  Written for graphs of
a few thousand vertices.

What it follows:
  Sec. 4.2  a worker holds the embeddings and inboxes of its local vertices; for halo vertices (remote
            sinks of local edges) it holds no embedding, only a mailbox in which the messages of the
            local partition are combined; after the local sends of a hop the combined messages go to
            the owners, which aggregate them once more; the next hop starts when all have arrived.
  Sec. 4.3  a vertex or feature update goes to the owner; an edge update whose endpoints live on one
            worker goes there; otherwise it goes to the source's worker and a no-compute copy goes to
            the sink's worker, which only updates its partition with it.
  Sec. 4.4, Alg. 1  placement of vertices that an edge addition creates: hash-based (id modulo the
            number of partitions) or locality-aware (a new source joins the partition of an existing
            high in-degree sink, else the least loaded partition; an edge with no existing endpoint
            goes to the least loaded partition).
  Sec. 4.5  per hop: aggregate inboxes, compute local embeddings, prepare messages, local send, remote
            send.

Readings where the paper is silent:
  - Alg. 1 has no branch for "source exists, sink is new": the new sink is placed by the final Else
    (least loaded partition), like any edge that does not fall under the earlier branches;
  - when neither endpoint exists both are placed on the same (least loaded) partition: the edge is
    assigned to one partition;
  - the high in-degree set holds the vertices whose in-degree exceeds twice the average degree
    (edges / placed vertices); it is rebuilt after every `hd_refresh` updates seen by the server;
  - load(P_i) counts the vertices placed on P_i; ties go to the lowest partition number;
  - the sink's worker learns that the sink is a hop-l vertex from the arrival of the (possibly zero)
    combined message that the source's worker sends for every changed edge at every hop;
  - vertex deletion (Sec. 4.3 routes it to the owner and says no more): the server, which keeps the edge
    lists for this purpose, replaces it at its position in the batch by one edge deletion per incident
    edge (out-edges in ascending sink order, then in-edges in ascending source order), each routed like
    any edge deletion, followed by a feature update of the vertex with a row of zeros (payload row -1);
The numerical rules (delta messages, coefficients, Update) are those of the single-machine method
(Sec. 3.3); the pin is that the workers' rows equal the single-machine oracle's full recomputation.
"""
from __future__ import annotations

from typing import Dict, List, Tuple

import numpy as np

OP_ADD_EDGE, OP_DEL_EDGE, OP_SET_FEATURE, OP_DEL_VERTEX = 0, 1, 2, 3
KIND_SAGE, KIND_GRAPHCONV, KIND_GIN = 0, 1, 2
AGG_SUM, AGG_MEAN, AGG_WSUM_GCN = 0, 1, 2
ACT_RELU = 1


# ------------------------------------------------------------------------------------------------
# server: vertex-partition map, high in-degree set, routing (Sec. 4.3, 4.4, Alg. 1)
# ------------------------------------------------------------------------------------------------
class Server:
    def __init__(self, n_partitions: int, owner: np.ndarray, src: np.ndarray, dst: np.ndarray,
                 routing: str = "locality", hd_refresh: int = 500_000):
        assert routing in ("locality", "hash")
        self.P = int(n_partitions)
        self.owner = np.array(owner, dtype=np.int64)          # V:P map, -1 = vertex not placed yet
        self.in_degree = np.bincount(dst, minlength=self.owner.size).astype(np.int64)
        self.n_edges = int(src.size)
        self.load = np.bincount(self.owner[self.owner >= 0], minlength=self.P).astype(np.int64)
        self.routing = routing
        self.hd_refresh = int(hd_refresh)
        self.seen = 0
        self.edges = set(zip(src.tolist(), dst.tolist()))     # to keep in-degrees right under no-op updates
        self.out_adj: Dict[int, set] = {}                     # edge lists, for the expansion of vertex deletions
        self.in_adj: Dict[int, set] = {}
        for u, v in self.edges:
            self.out_adj.setdefault(u, set()).add(v)
            self.in_adj.setdefault(v, set()).add(u)
        self.refresh_hd()

    def refresh_hd(self):
        placed = int((self.owner >= 0).sum())
        avg = self.n_edges / max(placed, 1)
        self.hd = set(np.nonzero(self.in_degree > 2.0 * avg)[0].tolist())

    def _place(self, v: int, p: int):
        self.owner[v] = p
        self.load[p] += 1

    def assign_edge(self, u: int, v: int):
        """Places whichever endpoint does not exist yet (Alg. 1, or the hash rule)."""
        eu, ev = self.owner[u] >= 0, self.owner[v] >= 0
        if eu and ev:
            return
        if self.routing == "hash":
            if not eu:
                self._place(u, u % self.P)
            if not ev:
                self._place(v, v % self.P)
            return
        if not eu and ev:                      # the source is new, the sink exists
            if v in self.hd:
                self._place(u, int(self.owner[v]))
            else:
                self._place(u, int(np.argmin(self.load)))
            return
        p = int(np.argmin(self.load))          # the final Else: every remaining case
        if not eu:
            self._place(u, p)
        if not ev:
            self._place(v, p)

    def _count(self):
        self.seen += 1
        if self.seen % self.hd_refresh == 0:
            self.refresh_hd()

    def route(self, ups: np.ndarray) -> List[List[Tuple[int, int, int, int, bool]]]:
        """Per worker: (position in the batch, op, u, v, compute?) in batch order.  A feature update's v is
        the payload row (-1: a row of zeros, from the expansion of a vertex deletion)."""
        out: List[List[Tuple[int, int, int, int, bool]]] = [[] for _ in range(self.P)]
        todo = [(i, int(r["op"]), int(r["u"]), int(r["v"])) for i, r in enumerate(ups)]
        k = 0
        while k < len(todo):
            i, op, u, v = todo[k]
            k += 1
            if op == OP_DEL_VERTEX:        # replaced, at its position, by the deletions of its edges and a zero row
                if self.owner[u] >= 0:
                    gen = [(i, OP_DEL_EDGE, u, x) for x in sorted(self.out_adj.get(u, ()))]
                    gen += [(i, OP_DEL_EDGE, x, u) for x in sorted(self.in_adj.get(u, ()))]
                    gen.append((i, OP_SET_FEATURE, u, -1))
                    todo[k:k] = gen
            elif op == OP_SET_FEATURE:
                assert self.owner[u] >= 0, "feature update of a vertex that is not in the graph"
                out[int(self.owner[u])].append((i, op, u, v, True))
            elif op in (OP_ADD_EDGE, OP_DEL_EDGE):
                if op == OP_ADD_EDGE:
                    self.assign_edge(u, v)
                pu, pv = int(self.owner[u]), int(self.owner[v])
                if pu >= 0 and pv >= 0:        # (deleting an edge of a vertex that was never placed: nothing exists)
                    out[pu].append((i, op, u, v, True))
                    if pv != pu:
                        out[pv].append((i, op, u, v, False))      # the no-compute copy
                    if op == OP_ADD_EDGE and (u, v) not in self.edges:
                        self.edges.add((u, v)); self.in_degree[v] += 1; self.n_edges += 1
                        self.out_adj.setdefault(u, set()).add(v); self.in_adj.setdefault(v, set()).add(u)
                    elif op == OP_DEL_EDGE and (u, v) in self.edges:
                        self.edges.discard((u, v)); self.in_degree[v] -= 1; self.n_edges -= 1
                        self.out_adj[u].discard(v); self.in_adj[v].discard(u)
            else:
                raise ValueError("unknown op code")
            self._count()
        return out


# ------------------------------------------------------------------------------------------------
# worker
# ------------------------------------------------------------------------------------------------
def _coef(agg: int, deg: int) -> float:
    if agg != AGG_WSUM_GCN:
        return 1.0
    return 1.0 / np.sqrt(deg) if deg > 0 else 0.0


def _norm(agg: int, deg_in: int) -> float:
    if agg == AGG_MEAN:
        return 1.0 / deg_in if deg_in > 0 else 0.0
    if agg == AGG_WSUM_GCN:
        return 1.0 / np.sqrt(deg_in) if deg_in > 0 else 0.0
    return 1.0


def _update(ly, w, h_self: np.ndarray, x: np.ndarray) -> np.ndarray:
    """Update function of one layer (Eq. 2) on one row; x = normalised aggregate."""
    Wa = w["Wa"].astype(np.float64)
    if ly.kind == KIND_SAGE:
        z = h_self @ Wa + x @ w["Wb"].astype(np.float64) + w["ba"]
    elif ly.kind == KIND_GRAPHCONV:
        z = x @ Wa + w["ba"]
    else:
        t = np.maximum(((1.0 + ly.eps) * h_self + x) @ Wa + w["ba"], 0.0)
        z = t @ w["Wb"].astype(np.float64) + w["bb"]
    return np.maximum(z, 0.0) if ly.act == ACT_RELU else z


class Worker:
    """One partition: out-lists, degrees, embeddings H^l and un-normalised aggregates S^l of its local
    vertices; a combiner mailbox per halo vertex while a hop runs."""

    def __init__(self, rank: int, model, weights):
        self.rank, self.model, self.weights = rank, model, weights
        self.L = len(model.layers)
        self.dims = [model.layers[0].d_in] + [l.d_out for l in model.layers]
        self.out: Dict[int, Dict[int, float]] = {}   # local source -> {sink (global id, local or halo): stored edge weight}
        self.deg_in: Dict[int, int] = {}    # local sink -> in-degree over ALL sources (local and remote)
        self.H: List[Dict[int, np.ndarray]] = [dict() for _ in range(self.L + 1)]
        self.S: List[Dict[int, np.ndarray]] = [dict() for _ in range(self.L + 1)]
        self.remote_in: Dict[int, set] = {}   # local sink -> its remote in-neighbours (kept up to date by no-compute copies)

    def is_local(self, v: int) -> bool:
        return v in self.H[0]

    def add_vertex(self, v: int, x: np.ndarray):
        """A placed vertex: feature row x, no edges yet; its rows are those of an isolated vertex."""
        self.out[v] = {}
        self.deg_in[v] = 0
        self.H[0][v] = np.array(x, dtype=np.float64)
        for l in range(1, self.L + 1):
            self.S[l][v] = np.zeros(self.dims[l - 1])
            self.H[l][v] = _update(self.model.layers[l - 1], self.weights[l - 1], self.H[l - 1][v], self.S[l][v])

    # -- apply (Sec. 4.5): topology and features; returns what the hops need -------------------------
    def apply(self, ops, feat_rows, op_w=None):
        """op_w: one weight per operation of the whole batch (stored edge weights; an added edge takes the
        weight given with its operation, an edge that exists keeps the one it has), or None: all ones."""
        self.added, self.deleted = [], []          # net edge changes this worker computes for: (u, v, weight)
        self.old_deg_out: Dict[int, int] = {}
        last_edge: Dict[Tuple[int, int], Tuple[int, bool, int]] = {}
        last_feat: Dict[int, int] = {}
        for (i, op, u, v, compute) in ops:         # the last operation on a pair / a vertex wins
            if op == OP_SET_FEATURE:
                last_feat[u] = v
            else:
                last_edge[(u, v)] = (op, compute, i)
        for (u, v), (op, compute, i) in sorted(last_edge.items()):
            src_local, dst_local = self.is_local(u), self.is_local(v)
            present = (v in self.out[u]) if src_local else None
            if src_local:
                if op == OP_ADD_EDGE and not present:
                    self.old_deg_out.setdefault(u, len(self.out[u]))
                    w = float(op_w[i]) if op_w is not None else 1.0
                    self.out[u][v] = w; self.added.append((u, v, w))
                    if dst_local:
                        self.deg_in[v] += 1
                elif op == OP_DEL_EDGE and present:
                    self.old_deg_out.setdefault(u, len(self.out[u]))
                    self.deleted.append((u, v, self.out[u].pop(v)))
                    if dst_local:
                        self.deg_in[v] -= 1
            else:
                # no-compute copy: the sink is local, the source is not; only the partition is updated.
                # Whether the edge existed is known to the source's worker alone; this worker keeps the
                # set of remote in-neighbours to apply the same rule.
                assert dst_local and not compute
                rin = self.remote_in.setdefault(v, set())
                if op == OP_ADD_EDGE and u not in rin:
                    rin.add(u); self.deg_in[v] += 1
                elif op == OP_DEL_EDGE and u in rin:
                    rin.discard(u); self.deg_in[v] -= 1
        # hop 0: feature replacements, old rows kept for the messages
        A, old = [], {}
        for u, row in sorted(last_feat.items()):
            old[u] = self.H[0][u].copy()
            self.H[0][u] = feat_rows[row].astype(np.float64) if row >= 0 else np.zeros_like(old[u])
            A.append(u)
        return A, old

    # -- one hop: prepare + local send + combine (returns the combined halo messages) ----------------
    def send(self, l: int, A_prev: List[int], old_prev: Dict[int, np.ndarray]):
        agg = self.model.agg
        K = self.dims[l - 1]
        self.inbox: Dict[int, np.ndarray] = {}
        halo: Dict[int, np.ndarray] = {}

        def deliver(v, m):
            box = self.inbox if self.is_local(v) else halo
            if v not in box:
                box[v] = np.zeros(K)
            box[v] += m

        senders = set(A_prev)
        if agg == AGG_WSUM_GCN:
            senders |= set(self.old_deg_out.keys())
        added = {(u, v) for (u, v, _) in self.added}
        for u in sorted(senders):
            hn = self.H[l - 1][u]
            ho = old_prev.get(u, hn)
            cn = _coef(agg, len(self.out[u]))
            co = _coef(agg, self.old_deg_out.get(u, len(self.out[u])))
            m = cn * hn - co * ho
            for v in sorted(self.out[u]):
                if (u, v) not in added:
                    deliver(v, self.out[u][v] * m)     # the edge's stored weight scales the message (Sec. 3.3.3)
        for (u, v, w) in self.added:      # the whole new term arrives
            deliver(v, w * _coef(agg, len(self.out[u])) * self.H[l - 1][u])
        for (u, v, w) in self.deleted:    # the whole old term leaves
            ho = old_prev.get(u, self.H[l - 1][u])
            deliver(v, -w * _coef(agg, self.old_deg_out[u]) * ho)
        return halo

    def receive(self, msgs: Dict[int, np.ndarray]):
        for v, m in msgs.items():
            if v not in self.inbox:
                self.inbox[v] = np.zeros_like(m)
            self.inbox[v] += m

    # -- aggregate inboxes, compute, keep old rows ---------------------------------------------------
    def compute(self, l: int, A_prev: List[int]):
        ly, w = self.model.layers[l - 1], self.weights[l - 1]
        A = set(self.inbox.keys())
        if ly.kind != KIND_GRAPHCONV:
            A |= set(A_prev)
        old = {}
        for v in sorted(A):
            if v in self.inbox:
                self.S[l][v] = self.S[l][v] + self.inbox[v]
            old[v] = self.H[l][v].copy()
            self.H[l][v] = _update(ly, w, self.H[l - 1][v], _norm(self.model.agg, self.deg_in[v]) * self.S[l][v])
        return sorted(A), old


class Cluster:
    """P workers and the server; apply_batch runs the hops with one remote send per hop."""

    def __init__(self, n_partitions, owner, n, src, dst, X, model, weights, full_H, full_S,
                 routing="locality", hd_refresh=500_000, edge_weights=None):
        """full_H / full_S: embeddings and aggregates of the initial graph (the state every worker
        starts from is given, as in Sec. 4.1: computed before the stream starts, then partitioned)."""
        self.P = n_partitions
        self.model, self.weights = model, weights
        self.server = Server(n_partitions, owner, src, dst, routing, hd_refresh)
        self.workers = [Worker(r, model, weights) for r in range(n_partitions)]
        self.X = X
        L = len(model.layers)
        for v in range(n):
            p = int(owner[v])
            if p < 0:
                continue
            w = self.workers[p]
            w.out[v] = {}
            w.deg_in[v] = 0
            for l in range(L + 1):
                w.H[l][v] = np.array(full_H[l][v], dtype=np.float64)
                if l:
                    w.S[l][v] = np.array(full_S[l][v], dtype=np.float64)
        ew = edge_weights.tolist() if edge_weights is not None else [1.0] * int(src.size)
        for u, v, a in zip(src.tolist(), dst.tolist(), ew):
            pu, pv = int(owner[u]), int(owner[v])
            self.workers[pu].out[u][v] = float(a)
            self.workers[pv].deg_in[v] += 1
            if pu != pv:
                self.workers[pv].remote_in.setdefault(v, set()).add(u)
        self.affected: List[List[int]] = []
        self.halo_rows_sent: List[int] = []

    def apply_batch(self, ups: np.ndarray, feat_rows: np.ndarray, op_w=None):
        L = len(self.model.layers)
        before = self.server.owner.copy()
        routed = self.server.route(ups)
        d0 = self.model.layers[0].d_in
        for v in np.nonzero((before < 0) & (self.server.owner >= 0))[0].tolist():   # vertices the batch created
            self.workers[int(self.server.owner[v])].add_vertex(v, np.zeros(d0))
        state = [w.apply(routed[r], feat_rows, op_w) for r, w in enumerate(self.workers)]
        A = [s[0] for s in state]
        old = [s[1] for s in state]
        self.affected = [sorted(sum(A, []))]
        self.halo_rows_sent = [0]
        for l in range(1, L + 1):
            outgoing = [w.send(l, A[r], old[r]) for r, w in enumerate(self.workers)]
            sent = 0
            for r, halo in enumerate(outgoing):        # remote send, receiver-side aggregation
                per_owner: Dict[int, Dict[int, np.ndarray]] = {}
                for v, m in halo.items():
                    per_owner.setdefault(int(self.server.owner[v]), {})[v] = m
                for p, msgs in per_owner.items():
                    assert p != r
                    self.workers[p].receive(msgs)
                    sent += len(msgs)
            res = [w.compute(l, A[r]) for r, w in enumerate(self.workers)]   # after all messages have arrived
            A = [x[0] for x in res]
            old = [x[1] for x in res]
            self.affected.append(sorted(sum(A, [])))
            self.halo_rows_sent.append(sent)

    def gather(self, l: int, n: int) -> np.ndarray:
        d = self.workers[0].dims[l]
        out = np.zeros((n, d))
        for w in self.workers:
            for v, row in w.H[l].items():
                out[v] = row
        return out
