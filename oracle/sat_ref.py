"""CPU oracle of the SAT partition-parallel GCN epoch.  TEST INFRASTRUCTURE ONLY.

The integer structures (partition lists, halo sets, cache slots) are written out from
their definitions with numpy; the floating-point steps call the plain C loops of
sat_oracle.c (double accumulation, formula order).  Nothing here is shared with, or
imported by, the CUDA library.

Paper passages followed (section / equation names of arXiv 2308.13466):
  partition, non-overlapping subgraphs            Preliminaries, "Distributed Training for GNNs"
  in- / out-of-subgraph neighbours                Eq. "mini-batch", Eq. "matrix form forward"
  1-hop extended subgraph G-bar_m                 Section "Embedding Predictor", temporal graphs
  halo set  U_{v in V_m} N(v) \\ V_m               Eq. "communication complexity"
  historical embeddings, sliding window tau       Section "Problem Formulation"; Eq. "problem formulation"
  predictor = LSTM + GCN, skip connection         Section "Embedding Predictor"
  pull / forward / push / loss / gradients        Algorithm 1
  layer forward / backward formulas               Appendix (forward and backward of SAT)
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass, field

import numpy as np

from .build import build_oracle

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build_oracle())
        _lib.orc_loss_ce.restype = C.c_double
        _lib.orc_loss_bce.restype = C.c_double
        _lib.orc_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _p(a, ctype=C.c_void_p):
    if a is None:
        return None
    return a.ctypes.data_as(ctype)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


# --------------------------------------------------------------------------------------
# O-1  degrees of A + I and D~^{-1/2}
# --------------------------------------------------------------------------------------
def degrees(rowptr: np.ndarray):
    n = rowptr.shape[0] - 1
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    dtil = np.empty(n, dtype=np.int32)
    dinv = np.empty(n, dtype=np.float32)
    lib().orc_degrees(C.c_int32(n), _p(rowptr), _p(dtil), _p(dinv))
    return dtil, dinv


# --------------------------------------------------------------------------------------
# O-2  partition structures
# --------------------------------------------------------------------------------------
def contig_blocks(n: int, M: int) -> np.ndarray:
    """Contiguous id blocks: part[v] = floor(v * M / n)."""
    return (np.arange(n, dtype=np.int64) * M // n).astype(np.int32)


def bfs_rank(rowptr: np.ndarray, col: np.ndarray) -> np.ndarray:
    """rank[v] = position of v in the breadth-first visit order (FIFO queue from node 0, neighbours ascending, restart at
    the smallest unvisited id)."""
    n = rowptr.shape[0] - 1
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int64)
    col = np.ascontiguousarray(col, dtype=np.int32)
    rank = np.empty(n, dtype=np.int32)
    lib().orc_bfs_rank(C.c_int32(n), _p(rowptr), _p(col), _p(rank))
    return rank


def bfs_blocks(rowptr: np.ndarray, col: np.ndarray, M: int) -> np.ndarray:
    """Breadth-first block partition: part[v] = floor(rank[v] * M / n); the graph is not relabelled."""
    n = rowptr.shape[0] - 1
    return (bfs_rank(rowptr, col).astype(np.int64) * M // n).astype(np.int32)


@dataclass
class Partitioning:
    n: int
    M: int
    part: np.ndarray
    slot: np.ndarray                       # int32 [n]: rank in C (sorted union of all halo sets) or -1
    n_slots: int
    inner_gid: list = field(default_factory=list)   # I_m, ascending global ids
    halo_gid: list = field(default_factory=list)    # B_m, ascending global ids
    loc_rowptr: list = field(default_factory=list)  # local CSR over rows I_m, int64
    loc_col: list = field(default_factory=list)     # local column ids (inner < n_m <= halo), ascending per row
    hrow_ptr: list = field(default_factory=list)    # halo-row CSR (rows B_m), int64
    hrow_col: list = field(default_factory=list)    # local inner ids of the neighbours inside m, ascending
    halo_slot: list = field(default_factory=list)   # slot[B_m]
    push_local: list = field(default_factory=list)  # local ids of inner nodes that are in C, ascending
    push_slot: list = field(default_factory=list)   # their slots


def build_partition(rowptr: np.ndarray, col: np.ndarray, part: np.ndarray, M: int, only_parts=None) -> Partitioning:
    """All per-partition lists, from their definitions.

    I_m = {v : part[v] = m};  B_m = sorted unique { u not in V_m : exists v in V_m, (v,u) in E };
    local CSR: rows I_m, entries N(v) + {v}, columns renamed to local ids (inner: rank in
    I_m; halo: n_m + rank in B_m) and sorted ascending; halo-row CSR: for u in B_m the
    neighbours of u inside V_m (the transpose of the halo block); C = sorted union of the
    B_m, slot = rank in C; push list = inner nodes of m that are in C.
    `only_parts` builds the per-partition lists of a subset only (the others stay None); C and
    slot[] are always global: u is in some B_m exactly when an edge (v, u) has part[v] != part[u].
    """
    n = rowptr.shape[0] - 1
    part = np.ascontiguousarray(part, dtype=np.int32)
    deg = np.diff(rowptr)
    P = Partitioning(n=n, M=M, part=part, slot=None, n_slots=0)
    in_any_halo = np.zeros(n, dtype=bool)
    step = 1 << 24                                    # union of all halo sets, edge chunk by edge chunk
    row_of = np.repeat(np.arange(n, dtype=np.int32), deg)
    for e0 in range(0, col.shape[0], step):
        c = col[e0:e0 + step]
        cut = part[row_of[e0:e0 + step]] != part[c]
        in_any_halo[c[cut]] = True
    del row_of
    per = []
    todo = list(range(M)) if only_parts is None else list(only_parts)
    for m in range(M):
        if m not in todo:
            per.append(None)
            continue
        inner = np.nonzero(part == m)[0].astype(np.int64)
        n_m = inner.shape[0]
        loc_of = np.full(n, -1, dtype=np.int64)
        loc_of[inner] = np.arange(n_m)
        d_m = deg[inner]
        src = np.repeat(np.arange(n_m, dtype=np.int64), d_m)
        # positions of the rows of I_m inside the global col array
        starts = np.repeat(rowptr[inner] - np.concatenate([[0], np.cumsum(d_m)[:-1]]), d_m)
        dst = col[starts + np.arange(src.shape[0], dtype=np.int64)].astype(np.int64)
        outside = part[dst] != m
        halo = np.unique(dst[outside])
        # add the self-loop of every inner row
        src2 = np.concatenate([src, np.arange(n_m, dtype=np.int64)])
        dst2 = np.concatenate([dst, inner])
        out2 = np.concatenate([outside, np.zeros(n_m, dtype=bool)])
        lid = np.where(out2, n_m + np.searchsorted(halo, dst2), loc_of[dst2])
        order = np.lexsort((lid, src2))
        loc_col = lid[order].astype(np.int32)
        loc_rowptr = np.zeros(n_m + 1, dtype=np.int64)
        np.cumsum(np.bincount(src2, minlength=n_m), out=loc_rowptr[1:])
        # halo-row CSR = cut edges regrouped by halo node
        hs = np.searchsorted(halo, dst[outside])
        hv = src[outside]
        o2 = np.lexsort((hv, hs))
        hrow_col = hv[o2].astype(np.int32)
        hrow_ptr = np.zeros(halo.shape[0] + 1, dtype=np.int64)
        np.cumsum(np.bincount(hs, minlength=halo.shape[0]), out=hrow_ptr[1:])
        per.append((inner.astype(np.int32), halo.astype(np.int32), loc_rowptr, loc_col, hrow_ptr, hrow_col))
    Cset = np.nonzero(in_any_halo)[0]
    slot = np.full(n, -1, dtype=np.int32)
    slot[Cset] = np.arange(Cset.shape[0], dtype=np.int32)
    P.slot, P.n_slots = slot, int(Cset.shape[0])
    for item in per:
        if item is None:
            for lst in (P.inner_gid, P.halo_gid, P.loc_rowptr, P.loc_col, P.hrow_ptr, P.hrow_col, P.halo_slot, P.push_local, P.push_slot):
                lst.append(None)
            continue
        inner, halo, lrp, lc, hp, hc = item
        P.inner_gid.append(inner)
        P.halo_gid.append(halo)
        P.loc_rowptr.append(lrp)
        P.loc_col.append(lc)
        P.hrow_ptr.append(hp)
        P.hrow_col.append(hc)
        P.halo_slot.append(slot[halo])
        pl = np.nonzero(slot[inner] >= 0)[0].astype(np.int32)
        P.push_local.append(pl)
        P.push_slot.append(slot[inner[pl]])
    return P


# --------------------------------------------------------------------------------------
# O-3  historical-embedding cache: ring of tau readable snapshots + 1 write buffer
# --------------------------------------------------------------------------------------
class CacheRing:
    """Per cached layer l (embeddings H^(l), l = 1..L-1) a ring of tau+1 buffers over the
    |C| boundary nodes.  Reads during an epoch see only committed snapshots (at most the
    tau newest); pushes of the running epoch go to the write buffer, which becomes the
    newest snapshot at commit.  Initially everything is zero and no snapshot is valid."""

    def __init__(self, n_slots: int, widths, tau: int):
        self.tau = tau
        self.n_slots = n_slots
        self.widths = list(widths)
        self.buf = [np.zeros((tau + 1, n_slots, w), dtype=np.float32) for w in widths]
        self.write_idx = 0
        self.n_valid = 0

    def snapshots(self, layer: int):
        """Valid snapshots of cached layer `layer` (1-based), oldest first."""
        k = min(self.n_valid, self.tau)
        idx = [(self.write_idx - 1 - a) % (self.tau + 1) for a in range(k - 1, -1, -1)]
        return [self.buf[layer - 1][i] for i in idx]

    def newest(self, layer: int):
        s = self.snapshots(layer)
        return s[-1] if s else None

    def push(self, layer: int, slots: np.ndarray, rows: np.ndarray):
        self.buf[layer - 1][self.write_idx][slots] = rows

    def commit(self):
        self.write_idx = (self.write_idx + 1) % (self.tau + 1)
        self.n_valid = min(self.n_valid + 1, self.tau)


# --------------------------------------------------------------------------------------
# O-4 / O-5  predictor
# --------------------------------------------------------------------------------------
def lstm_state(snaps, d: int, h: int, Wx, Uh, b, n_slots: int, slots_sel=None) -> np.ndarray:
    """Final LSTM hidden state S [n_slots, h] over the snapshots (oldest first)."""
    k = len(snaps)
    S = np.zeros((n_slots, h), dtype=np.float32)
    if k == 0:
        return S
    snaps = [_f32(s) for s in snaps]
    ld = snaps[0].shape[1]
    arr = (C.c_void_p * k)(*[s.ctypes.data for s in snaps])
    Wx, Uh, b = _f32(Wx), _f32(Uh), _f32(b)
    sel = None if slots_sel is None else np.ascontiguousarray(slots_sel, dtype=np.int32)
    lib().orc_lstm(C.c_int32(0 if sel is None else sel.shape[0]), _p(sel), C.c_int32(n_slots), C.c_int32(k),
                   arr, C.c_int64(ld), C.c_int32(d), C.c_int32(h), _p(Wx), _p(Uh), _p(b), _p(S))
    return S


def gru_state(snaps, d: int, h: int, Wx, Uh, b, n_slots: int, slots_sel=None) -> np.ndarray:
    """Final GRU hidden state S [n_slots, h] over the snapshots (oldest first): Wx [d, 3h] and Uh [h, 3h] in gate order
    (r, z, n), b [4h] = (b_r, b_z, b_n, b_hn)."""
    k = len(snaps)
    S = np.zeros((n_slots, h), dtype=np.float32)
    if k == 0:
        return S
    snaps = [_f32(s) for s in snaps]
    ld = snaps[0].shape[1]
    arr = (C.c_void_p * k)(*[s.ctypes.data for s in snaps])
    Wx, Uh, b = _f32(Wx), _f32(Uh), _f32(b)
    assert Wx.shape == (d, 3 * h) and Uh.shape == (h, 3 * h) and b.shape == (4 * h,)
    sel = None if slots_sel is None else np.ascontiguousarray(slots_sel, dtype=np.int32)
    lib().orc_gru(C.c_int32(0 if sel is None else sel.shape[0]), _p(sel), C.c_int32(n_slots), C.c_int32(k),
                  arr, C.c_int64(ld), C.c_int32(d), C.c_int32(h), _p(Wx), _p(Uh), _p(b), _p(S))
    return S


def predict_halo(P: Partitioning, m: int, dtil, S, newest, Wg, bg, rows_sel=None) -> np.ndarray:
    """Predicted halo embeddings of partition m: newest snapshot + GCN(S) (skip connection)."""
    h, d = Wg.shape
    nh = P.halo_gid[m].shape[0]
    out = np.zeros((nh, d), dtype=np.float32)
    sel = None if rows_sel is None else np.ascontiguousarray(rows_sel, dtype=np.int32)
    S = _f32(S)
    newest = None if newest is None else _f32(newest)
    Wg, bg = _f32(Wg), _f32(bg)
    lib().orc_predict_halo(C.c_int32(0 if sel is None else sel.shape[0]), _p(sel),
                           C.c_int32(nh), _p(P.hrow_ptr[m]), _p(P.hrow_col[m]),
                           _p(P.inner_gid[m]), _p(P.halo_gid[m]), _p(P.slot), _p(dtil),
                           C.c_int32(h), C.c_int32(d), _p(S), _p(newest),
                           C.c_int64(0 if newest is None else newest.shape[1]),
                           _p(Wg), _p(bg), _p(out), C.c_int64(d))
    return out


def historical_halo(P: Partitioning, m: int, newest, d: int) -> np.ndarray:
    """Identity predictor: the plain historical embedding (newest snapshot, zeros if none)."""
    nh = P.halo_gid[m].shape[0]
    if newest is None:
        return np.zeros((nh, d), dtype=np.float32)
    return np.ascontiguousarray(newest[P.halo_slot[m]], dtype=np.float32)


# --------------------------------------------------------------------------------------
# O-6  layer forward,  O-9  layer backward,  O-8  loss
# --------------------------------------------------------------------------------------
def layer_fwd(P: Partitioning, m: int, dtil, H_in, H_halo, W, bias, act: int, rows_sel=None):
    """Returns (AGG float64 [n_m, d_in], Z float64 [n_m, d_out], H fp32 [n_m, d_out])."""
    n_in = P.inner_gid[m].shape[0]
    d_in, d_out = W.shape
    H_in, H_halo, W = _f32(H_in), _f32(H_halo), _f32(W)
    bias = None if bias is None else _f32(bias)
    if H_halo.shape[0] == 0:
        H_halo = np.zeros((1, d_in), dtype=np.float32)
    AGG = np.zeros((n_in, d_in), dtype=np.float64)
    Z = np.zeros((n_in, d_out), dtype=np.float64)
    H = np.zeros((n_in, d_out), dtype=np.float32)
    sel = None if rows_sel is None else np.ascontiguousarray(rows_sel, dtype=np.int32)
    lib().orc_layer_fwd(C.c_int32(0 if sel is None else sel.shape[0]), _p(sel),
                        C.c_int32(n_in), _p(P.loc_rowptr[m]), _p(P.loc_col[m]),
                        _p(P.inner_gid[m]), _p(P.halo_gid[m]), _p(dtil),
                        C.c_int32(d_in), C.c_int32(d_out),
                        _p(H_in), C.c_int64(H_in.shape[1]), _p(H_halo), C.c_int64(H_halo.shape[1]),
                        _p(W), _p(bias), C.c_int32(act), _p(AGG), _p(Z), _p(H), C.c_int64(d_out))
    return AGG, Z, H


def layer_bwd(P: Partitioning, m: int, dtil, G_out, mask, AGG, W, G_W, G_b, want_in=True, want_halo=False):
    """Accumulates into G_W, G_b (float64); returns (G_in fp32 or None, G_halo fp32 or None)."""
    n_in = P.inner_gid[m].shape[0]
    n_halo = P.halo_gid[m].shape[0]
    d_in, d_out = W.shape
    G_out, W = _f32(G_out), _f32(W)
    AGG = np.ascontiguousarray(AGG, dtype=np.float64)
    mask = None if mask is None else np.ascontiguousarray(mask, dtype=np.uint8)
    G_in = np.zeros((n_in, d_in), dtype=np.float32) if want_in else None
    G_halo = np.zeros((n_halo, d_in), dtype=np.float32) if want_halo else None
    lib().orc_layer_bwd(C.c_int32(n_in), C.c_int32(n_halo), _p(P.loc_rowptr[m]), _p(P.loc_col[m]),
                        _p(P.inner_gid[m]), _p(P.halo_gid[m]), _p(dtil),
                        C.c_int32(d_in), C.c_int32(d_out), _p(G_out), C.c_int64(G_out.shape[1]), _p(mask),
                        _p(AGG), _p(W), _p(G_W), _p(G_b), _p(G_in), C.c_int64(d_in), _p(G_halo), C.c_int64(d_in))
    return G_in, G_halo


def loss_grad(kind: str, Z, labels, scale: float):
    """(scaled loss sum over the rows, G = scale * dLoss/dZ fp32)."""
    Z = _f32(Z)
    n, c = Z.shape
    G = np.zeros((n, c), dtype=np.float32)
    if kind == "ce":
        y = np.ascontiguousarray(labels, dtype=np.int32)
        val = lib().orc_loss_ce(C.c_int32(n), C.c_int32(c), _p(Z), C.c_int64(c), _p(y), C.c_double(scale), _p(G), C.c_int64(c))
    else:
        Y = np.ascontiguousarray(labels, dtype=np.uint8)
        val = lib().orc_loss_bce(C.c_int32(n), C.c_int32(c), _p(Z), C.c_int64(c), _p(Y), C.c_double(scale), _p(G), C.c_int64(c))
    return float(val), G


# --------------------------------------------------------------------------------------
# O-10  one SAT epoch over all partitions (Algorithm 1, lines of the epoch loop)
# --------------------------------------------------------------------------------------
@dataclass
class EpochResult:
    loss: float
    G_W: list
    G_b: list
    per_part: list      # per partition: dict(H=[H^(1..L)], halo=[Hhat inputs of layers 1..L], G_in=[...], Z=[...], AGG=[...])
    S: list             # per cached layer: LSTM state table or None (identity predictor)
    S_slots: object = None  # slots for which S was computed (None = all)


class GradHistory:
    """Gradient-side history (Appendix, back-propagation of SAT): for every layer j = 2..L the matrix
    Q^(j) = sum_m P_out^(m)T D^(m, j) over the |C| boundary nodes, D = G o sigma'(Z) being the layer's pre-activation
    gradient.  Row v holds what the partitions that use v as a halo node sent back for it.  `read[j-2]` is the snapshot
    of the previous epoch (None before the first commit), `write[j-2]` collects the running epoch."""

    def __init__(self, n_slots: int, widths):
        self.n_slots, self.widths = n_slots, list(widths)        # widths[j-2] = d_j
        self.read = [None] * len(self.widths)
        self.write = [np.zeros((n_slots, w), dtype=np.float64) for w in self.widths]

    def commit(self):
        self.read = [w.astype(np.float32) for w in self.write]
        self.write = [np.zeros((self.n_slots, w), dtype=np.float64) for w in self.widths]


def halo_pre_gradient(P: Partitioning, m: int, dtil, D) -> np.ndarray:
    """(P_out^T D)[u] = sum_{v in V_m, v ~ u} p_uv D[v] for the halo nodes u of partition m (float64)."""
    dt = np.asarray(dtil, dtype=np.float64)
    halo = P.halo_gid[m]
    counts = np.diff(P.hrow_ptr[m]).astype(np.int64)
    rows = np.repeat(np.arange(halo.shape[0], dtype=np.int64), counts)
    loc = P.hrow_col[m].astype(np.int64)
    p = 1.0 / np.sqrt(dt[halo[rows]] * dt[P.inner_gid[m][loc]])
    out = np.zeros((halo.shape[0], D.shape[1]))
    np.add.at(out, rows, p[:, None] * np.asarray(D, dtype=np.float64)[loc])
    return out


def run_epoch(P: Partitioning, dtil, cache: CacheRing, X, labels, W, b, pred, loss_kind: str,
              order=None, keep: bool = True, want_halo_grad: bool = False, parts=None, masks=None,
              grad_hist: GradHistory = None) -> EpochResult:
    """pull (predict) -> forward -> push, per layer; loss; backward; commit the ring.

    pred: list (one entry per cached layer) of dict(Wx, Uh, b, Wg, bg) or None for the
    identity predictor (plain historical embeddings).  `parts` restricts the epoch to a
    subset of partitions (then the ring is not committed).  `masks[m][l-1]`, when given,
    replaces [Z^(l) > 0] in the backward of partition m (the derivative of ReLU where Z is
    zero up to rounding is a tie: either sign decision is a correct result).
    grad_hist switches the stale-gradient term of the Appendix's back-propagation on:
    G_H^(t, l-1) = P_in^T D^(t, l) W^(l)T + [Q^(t-1, l) W^(l)T on the boundary rows], and this epoch's P_out^T D^(t, l) is
    collected for the next one."""
    L = len(W)
    n = P.n
    ms = list(range(P.M)) if parts is None else list(parts)
    if order is not None:
        ms = list(order)
    # LSTM state table: depends only on committed snapshots, one per cached layer
    S = []
    sel = None
    if parts is not None:
        # only the cached nodes these partitions read: their halo nodes and the halo nodes' neighbours inside them
        need = [P.halo_slot[m] for m in ms] + [P.slot[P.inner_gid[m][P.hrow_col[m]]] for m in ms]
        sel = np.unique(np.concatenate(need)) if need else np.empty(0, dtype=np.int32)
    for l in range(1, L):
        pr = pred[l - 1] if pred is not None else None
        if pr is None:
            S.append(None)
        else:
            h, d = pr["Wg"].shape
            state = gru_state if pr.get("cell", "lstm") == "gru" else lstm_state
            S.append(state(cache.snapshots(l), d, h, pr["Wx"], pr["Uh"], pr["b"], P.n_slots, slots_sel=sel))
    G_W = [np.zeros(w.shape, dtype=np.float64) for w in W]
    G_b = [np.zeros(w.shape[1], dtype=np.float64) for w in W]
    total_loss = 0.0
    per_part = [None] * P.M
    for m in ms:
        inner, halo = P.inner_gid[m], P.halo_gid[m]
        H_in = _f32(X[inner])
        rec = dict(H=[], halo=[], G_in=[], Z=[], AGG=[], G_halo=[])
        for l in range(1, L + 1):
            if l == 1:
                H_halo = _f32(X[halo])                      # raw features are exact
            else:
                pr = pred[l - 2] if pred is not None else None
                if pr is None:
                    H_halo = historical_halo(P, m, cache.newest(l - 1), W[l - 1].shape[0])
                else:
                    H_halo = predict_halo(P, m, dtil, S[l - 2], cache.newest(l - 1), pr["Wg"], pr["bg"])
            AGG, Z, H = layer_fwd(P, m, dtil, H_in, H_halo, W[l - 1], b[l - 1], 1 if l < L else 0)
            if l < L:
                cache.push(l, P.push_slot[m], H[P.push_local[m]])
            rec["halo"].append(H_halo)
            rec["AGG"].append(AGG)
            rec["Z"].append(Z)
            rec["H"].append(H)
            H_in = H
        lab = labels[inner]
        val, G = loss_grad(loss_kind, rec["H"][-1], lab, 1.0 / n)
        total_loss += val
        rec["G_L"] = G
        g_ins = [None] * L
        g_halos = [None] * L
        for l in range(L, 0, -1):
            mask = None if l == L else (rec["Z"][l - 1] > 0.0).astype(np.uint8)
            if mask is not None and masks is not None and masks[m] is not None and masks[m][l - 1] is not None:
                mask = np.ascontiguousarray(masks[m][l - 1], dtype=np.uint8)
            G_in, G_halo = layer_bwd(P, m, dtil, G, mask, rec["AGG"][l - 1], W[l - 1], G_W[l - 1], G_b[l - 1],
                                     want_in=(l > 1), want_halo=want_halo_grad)
            if grad_hist is not None and l >= 2:
                D = np.asarray(G, dtype=np.float64) * (1.0 if mask is None else mask)
                grad_hist.write[l - 2][P.halo_slot[m]] += halo_pre_gradient(P, m, dtil, D)
                if grad_hist.read[l - 2] is not None:
                    stale = grad_hist.read[l - 2][P.push_slot[m]].astype(np.float64) @ np.asarray(W[l - 1], dtype=np.float64).T
                    G_in = G_in.astype(np.float64)
                    G_in[P.push_local[m]] += stale
                    G_in = G_in.astype(np.float32)
            g_ins[l - 1] = G_in
            g_halos[l - 1] = G_halo
            G = G_in
        rec["G_in"] = g_ins
        rec["G_halo"] = g_halos
        if not keep:
            rec["AGG"] = rec["Z"] = None
        per_part[m] = rec
    if parts is None:
        cache.commit()
        if grad_hist is not None:
            grad_hist.commit()
    return EpochResult(loss=total_loss, G_W=G_W, G_b=G_b, per_part=per_part, S=S, S_slots=sel)


# ------------------------------------------------------------------------------------------
# Lossy storage of historical embeddings (Supplement, "Data Compression for Historical Embedding Storage")
# ------------------------------------------------------------------------------------------
def codec_encode(X: np.ndarray, precision: int):
    """Polyline-style encoding of every row of X (fp32 [rows, d]) at `precision` decimal places.
    Returns (bytes uint8 [total], offsets int64 [rows + 1])."""
    X = _f32(X)
    rows, d = X.shape
    sizes = np.zeros(rows, dtype=np.int32)
    lib().orc_codec_row_bytes(C.c_int64(rows), C.c_int32(d), _p(X), C.c_int64(X.strides[0] // 4), C.c_int32(precision), _p(sizes))
    offsets = np.zeros(rows + 1, dtype=np.int64)
    np.cumsum(sizes, out=offsets[1:])
    out = np.zeros(int(offsets[-1]), dtype=np.uint8)
    lib().orc_codec_encode(C.c_int64(rows), C.c_int32(d), _p(X), C.c_int64(X.strides[0] // 4), C.c_int32(precision), _p(offsets), _p(out))
    return out, offsets


def codec_decode(data: np.ndarray, offsets: np.ndarray, d: int, precision: int) -> np.ndarray:
    """Inverse of codec_encode: fp32 [rows, d]; raises on a malformed row."""
    data = np.ascontiguousarray(data, dtype=np.uint8)
    offsets = np.ascontiguousarray(offsets, dtype=np.int64)
    rows = offsets.shape[0] - 1
    X = np.zeros((rows, d), dtype=np.float32)
    lib().orc_codec_decode.restype = C.c_int64
    bad = lib().orc_codec_decode(C.c_int64(rows), C.c_int32(d), _p(data), _p(offsets), C.c_int32(precision), _p(X), C.c_int64(d))
    if bad:
        raise ValueError(f"codec_decode: malformed row {bad - 1}")
    return X


# ------------------------------------------------------------------------------------------
# Staleness of the out-of-subgraph embeddings (Eq. "staleness def"): || H_out - H~_out || over the halo of a partition
# ------------------------------------------------------------------------------------------
def staleness(P: Partitioning, m: int, H_fresh_by_gid: np.ndarray, H_used_halo: np.ndarray) -> float:
    """Frobenius norm of the difference between the fresh embeddings of the halo nodes of partition m
    (rows of H_fresh_by_gid [n, d], indexed by global node id) and the embeddings the partition used for them
    (H_used_halo [b_m, d], in halo order)."""
    fresh = np.asarray(H_fresh_by_gid)[P.halo_gid[m]].astype(np.float64)
    diff = fresh - np.asarray(H_used_halo).astype(np.float64)
    return float(np.sqrt(np.sum(diff * diff)))


# ------------------------------------------------------------------------------------------
# O-12  embedding-predictor objective and its gradient (Eq. "predictor loss", Eq. "mini-batch training",
#       Algorithm 1 "Embedding predictor update"); fp64 numpy, written out step by step
# ------------------------------------------------------------------------------------------
def _logistic(x):
    return 1.0 / (1.0 + np.exp(-x))


def pred_halo_weights(P: Partitioning, m: int, dtil):
    """Entries of the predictor's graph convolution for the halo rows of partition m as three arrays
    (halo row j, cache slot, weight p): the self term p_uu and p_uv for the neighbours v of u inside V_m."""
    dt = np.asarray(dtil, dtype=np.float64)
    halo = P.halo_gid[m]
    nh = halo.shape[0]
    counts = np.diff(P.hrow_ptr[m]).astype(np.int64)
    rows_nb = np.repeat(np.arange(nh, dtype=np.int64), counts)
    v = P.inner_gid[m][P.hrow_col[m]]
    p_nb = 1.0 / np.sqrt(dt[halo[rows_nb]] * dt[v])
    rows = np.concatenate([np.arange(nh, dtype=np.int64), rows_nb])
    slots = np.concatenate([P.slot[halo], P.slot[v]]).astype(np.int64)
    p = np.concatenate([1.0 / dt[halo], p_nb])
    return rows, slots, p


def pred_loss_grad(P: Partitioning, dtil, snaps, target, Wx, Uh, b, Wg, bg, row_weight=None):
    """Objective of the embedding predictor of one cached layer and its gradient.

    snaps: the valid snapshots [n_slots x d], oldest first (the temporal graph of the last tau epochs);
    target: [n_slots x d] the embeddings pushed in the running epoch (what the prediction should have been).
    Prediction for halo node u of partition m (Section "Embedding Predictor"): LSTM over the snapshots -> final
    hidden state S; a_u = p_uu S_u + sum_{v in N(u) cap V_m} p_uv S_v; Hhat_u = newest_u + a_u Wg + bg.
    Loss (Eq. "predictor loss" with the squared Euclidean norm, Eq. "mini-batch training" for the weights):
        L = (1/M) sum_m sum_{u in B_m} w_u^(m) * 1/2 |Hhat_u - target_u|^2,
    w_u^(m) = 1/b_m by default; row_weight[m] (length b_m) replaces it (1/|batch| on a sampled batch, 0 elsewhere).
    Returns (L, dict(Wx, Uh, b, Wg, bg)) in float64."""
    Wx, Uh, b, Wg, bg = (np.asarray(a, dtype=np.float64) for a in (Wx, Uh, b, Wg, bg))
    h, d = Wg.shape
    ns = P.n_slots
    k = len(snaps)
    X = [np.asarray(s, dtype=np.float64)[:, :d] for s in snaps]
    T = np.asarray(target, dtype=np.float64)[:, :d]
    # ---- LSTM over the snapshots, every cached node a sequence of length k, zero initial state ----
    hs = [np.zeros((ns, h))]
    cs = [np.zeros((ns, h))]
    gates = []
    for t in range(k):
        z = X[t] @ Wx + hs[-1] @ Uh + b
        gi, gf = _logistic(z[:, :h]), _logistic(z[:, h:2 * h])
        gg, go = np.tanh(z[:, 2 * h:3 * h]), _logistic(z[:, 3 * h:])
        c = gf * cs[-1] + gi * gg
        gates.append((gi, gf, gg, go))
        cs.append(c)
        hs.append(go * np.tanh(c))
    S = hs[-1]
    newest = X[-1] if k > 0 else np.zeros((ns, d))
    # ---- graph convolution on S, skip connection, loss ----
    loss = 0.0
    G = dict(Wx=np.zeros_like(Wx), Uh=np.zeros_like(Uh), b=np.zeros_like(b), Wg=np.zeros_like(Wg), bg=np.zeros_like(bg))
    G_S = np.zeros((ns, h))
    for m in range(P.M):
        nh = P.halo_gid[m].shape[0]
        if nh == 0:
            continue
        rows, slots, p = pred_halo_weights(P, m, dtil)
        a = np.zeros((nh, h))
        np.add.at(a, rows, p[:, None] * S[slots])
        hs_m = P.halo_slot[m].astype(np.int64)
        pred = newest[hs_m] + a @ Wg + bg
        w = np.full(nh, 1.0 / nh) if row_weight is None or row_weight[m] is None else np.asarray(row_weight[m], dtype=np.float64)
        diff = pred - T[hs_m]
        loss += float(np.sum(w * 0.5 * np.sum(diff * diff, axis=1))) / P.M
        E = diff * (w / P.M)[:, None]                  # dL / dHhat
        G["bg"] += E.sum(axis=0)
        G["Wg"] += a.T @ E
        G_a = E @ Wg.T
        np.add.at(G_S, slots, p[:, None] * G_a[rows])  # transpose of the graph convolution
    # ---- back-propagation through time ----
    dh = G_S
    dc = np.zeros((ns, h))
    for t in range(k - 1, -1, -1):
        gi, gf, gg, go = gates[t]
        tc = np.tanh(cs[t + 1])
        dc = dc + dh * go * (1.0 - tc * tc)
        dz = np.concatenate([dc * gg * gi * (1.0 - gi),            # input gate
                             dc * cs[t] * gf * (1.0 - gf),         # forget gate
                             dc * gi * (1.0 - gg * gg),            # candidate
                             dh * tc * go * (1.0 - go)], axis=1)   # output gate
        G["Wx"] += X[t].T @ dz
        G["Uh"] += hs[t].T @ dz
        G["b"] += dz.sum(axis=0)
        dh = dz @ Uh.T
        dc = dc * gf
    return loss, G


# ------------------------------------------------------------------------------------------
# O-13  Graph-attention layer as the local layer of a partition (the paper evaluates SAT with a GAT backbone as well and
#       gives no equations for it; this is the standard single-head graph attention layer on the 1-hop extended subgraph,
#       with the out-of-subgraph embeddings taken from the cache / predictor exactly as for the GCN layer).  float64 numpy.
# ------------------------------------------------------------------------------------------
GAT_SLOPE = 0.2


def _gat_rows(P: Partitioning, m: int):
    counts = np.diff(P.loc_rowptr[m]).astype(np.int64)
    rows = np.repeat(np.arange(counts.shape[0], dtype=np.int64), counts)
    return rows, P.loc_col[m].astype(np.int64)


def gat_fwd(P: Partitioning, m: int, H_in, H_halo, W, a_src, a_dst, bias, act: int):
    """For inner node v of partition m, over the entries u of its local row (its neighbours inside and outside the
    partition and v itself):
        z_u = h_u W;  e_vu = LeakyReLU_0.2(a_dst . z_v + a_src . z_u);  alpha_vu = softmax_u(e_vu);
        o_v = sum_u alpha_vu z_u + bias;  h'_v = ReLU(o_v) (act = 1) or o_v.
    Returns dict(Z=[n_m + b_m, d_out] (inner rows first), alpha=[entries], O, H (fp32))."""
    Hc = np.concatenate([np.asarray(H_in, dtype=np.float64), np.asarray(H_halo, dtype=np.float64).reshape(-1, np.asarray(H_in).shape[1])])
    W = np.asarray(W, dtype=np.float64)
    a_src, a_dst = np.asarray(a_src, dtype=np.float64), np.asarray(a_dst, dtype=np.float64)
    n_in = np.asarray(H_in).shape[0]
    Z = Hc @ W
    s_src, s_dst = Z @ a_src, Z[:n_in] @ a_dst
    rows, cols = _gat_rows(P, m)
    pre = s_dst[rows] + s_src[cols]
    e = np.where(pre > 0, pre, GAT_SLOPE * pre)
    mx = np.full(n_in, -np.inf)
    np.maximum.at(mx, rows, e)
    w = np.exp(e - mx[rows])
    den = np.zeros(n_in)
    np.add.at(den, rows, w)
    alpha = w / den[rows]
    O = np.zeros((n_in, W.shape[1]))
    np.add.at(O, rows, alpha[:, None] * Z[cols])
    if bias is not None:
        O = O + np.asarray(bias, dtype=np.float64)
    H = np.maximum(O, 0.0) if act else O
    return dict(Z=Z, alpha=alpha, pre=pre, O=O, H=H.astype(np.float32))


def gat_bwd(P: Partitioning, m: int, H_in, H_halo, W, a_src, a_dst, fwd, G_out, act: int, mask=None, positive=None):
    """Gradients of sum(G_out * h') for the layer above; the out-of-subgraph embeddings are constants of the epoch, the
    weights act on them as on the inner rows.  Returns dict(W, a_src, a_dst, b, H_in) in float64.
    `positive` (bool per entry of the local rows), when given, replaces [pre > 0] as the LeakyReLU's slope decision:
    where a logit is zero up to rounding either slope is a correct result (as `mask` does for the ReLU)."""
    Hc = np.concatenate([np.asarray(H_in, dtype=np.float64), np.asarray(H_halo, dtype=np.float64).reshape(-1, np.asarray(H_in).shape[1])])
    W = np.asarray(W, dtype=np.float64)
    a_src, a_dst = np.asarray(a_src, dtype=np.float64), np.asarray(a_dst, dtype=np.float64)
    n_in = np.asarray(H_in).shape[0]
    Z, alpha, pre = fwd["Z"], fwd["alpha"], fwd["pre"]
    rows, cols = _gat_rows(P, m)
    D = np.asarray(G_out, dtype=np.float64)
    if act:
        D = D * ((fwd["O"] > 0) if mask is None else np.asarray(mask, dtype=np.float64))
    d_alpha = np.sum(D[rows] * Z[cols], axis=1)                       # dL / d alpha_vu
    t = np.zeros(n_in)
    np.add.at(t, rows, alpha * d_alpha)
    pos = (pre > 0) if positive is None else np.asarray(positive, dtype=bool)
    d_pre = alpha * (d_alpha - t[rows]) * np.where(pos, 1.0, GAT_SLOPE)        # through softmax and LeakyReLU
    ds_dst = np.zeros(n_in)
    np.add.at(ds_dst, rows, d_pre)
    ds_src = np.zeros(Z.shape[0])
    np.add.at(ds_src, cols, d_pre)
    dZ = np.zeros_like(Z)
    np.add.at(dZ, cols, alpha[:, None] * D[rows])
    dZ += ds_src[:, None] * a_src
    dZ[:n_in] += ds_dst[:, None] * a_dst
    return dict(W=Hc.T @ dZ, a_src=Z.T @ ds_src, a_dst=Z[:n_in].T @ ds_dst, b=D.sum(axis=0), H_in=dZ[:n_in] @ W.T)


def run_epoch_gat(P: Partitioning, dtil, cache: CacheRing, X, labels, params, pred, loss_kind: str, masks=None, positive=None):
    """One SAT epoch with graph-attention layers in place of the GCN layers (Algorithm 1 unchanged around them): for every
    partition and layer pull (features for layer 1, predicted / historical embeddings of the cached layer otherwise),
    gat_fwd, push; loss; gat_bwd down the layers with the pulled embeddings held constant; commit.
    params: per layer dict(W, a_src, a_dst, b).  Returns dict(loss, grads=[per layer dict(W, a_src, a_dst, b)], H=[per
    partition [H^(1..L)]], O=[per partition [pre-activation outputs]], pre=[per partition [per layer: the attention logits
    before the LeakyReLU, one per entry of the local rows]], logit_margin=[per layer: the smallest |logit| relative to
    their rms: where it is at rounding level the slope of that logit is a tie]).  masks[m][l-1] / positive[m][l-1] replace
    the ReLU / LeakyReLU sign decisions of partition m, layer l in the backward pass."""
    L = len(params)
    n = P.n
    S = []
    for l in range(1, L):
        pr = pred[l - 1] if pred is not None else None
        if pr is None:
            S.append(None)
        else:
            h, d = pr["Wg"].shape
            state = gru_state if pr.get("cell", "lstm") == "gru" else lstm_state
            S.append(state(cache.snapshots(l), d, h, pr["Wx"], pr["Uh"], pr["b"], P.n_slots))
    grads = [dict(W=np.zeros(p["W"].shape), a_src=np.zeros(p["a_src"].shape), a_dst=np.zeros(p["a_dst"].shape), b=np.zeros(p["b"].shape))
             for p in params]
    total, Hs, Os, Pres = 0.0, [None] * P.M, [None] * P.M, [None] * P.M
    margin = [np.inf] * L        # per layer: smallest |pre-activation of an attention logit| relative to their rms
    for m in range(P.M):
        inner, halo = P.inner_gid[m], P.halo_gid[m]
        H_in = _f32(X[inner])
        ins, halos, fws = [], [], []
        for l in range(1, L + 1):
            if l == 1:
                H_halo = _f32(X[halo])
            else:
                pr = pred[l - 2] if pred is not None else None
                d_prev = params[l - 1]["W"].shape[0]
                if pr is None:
                    H_halo = historical_halo(P, m, cache.newest(l - 1), d_prev)
                else:
                    H_halo = predict_halo(P, m, dtil, S[l - 2], cache.newest(l - 1), pr["Wg"], pr["bg"])
            p = params[l - 1]
            f = gat_fwd(P, m, H_in, H_halo, _f32(p["W"]), _f32(p["a_src"]), _f32(p["a_dst"]), _f32(p["b"]), 1 if l < L else 0)
            if f["pre"].size:
                margin[l - 1] = min(margin[l - 1], float(np.min(np.abs(f["pre"])) / max(np.sqrt(np.mean(f["pre"] ** 2)), 1e-300)))
            if l < L:
                cache.push(l, P.push_slot[m], f["H"][P.push_local[m]])
            ins.append(H_in)
            halos.append(H_halo)
            fws.append(f)
            H_in = f["H"]
        val, G = loss_grad(loss_kind, fws[-1]["H"], labels[inner], 1.0 / n)
        total += val
        for l in range(L, 0, -1):
            p = params[l - 1]
            mk = None
            if masks is not None and masks[m] is not None and l < L and masks[m][l - 1] is not None:
                mk = masks[m][l - 1]
            ps = None
            if positive is not None and positive[m] is not None and positive[m][l - 1] is not None:
                ps = positive[m][l - 1]
            g = gat_bwd(P, m, ins[l - 1], halos[l - 1], _f32(p["W"]), _f32(p["a_src"]), _f32(p["a_dst"]), fws[l - 1], G, 1 if l < L else 0, mask=mk,
                        positive=ps)
            for k in ("W", "a_src", "a_dst", "b"):
                grads[l - 1][k] += g[k]
            G = g["H_in"].astype(np.float32)
        Hs[m] = [f["H"] for f in fws]
        Os[m] = [f["O"] for f in fws]
        Pres[m] = [f["pre"] for f in fws]
    cache.commit()
    return dict(loss=total, grads=grads, H=Hs, O=Os, pre=Pres, logit_margin=margin)
