"""One SAT epoch as a sequence of library calls (Algorithm 1 of the paper, epoch body).

This module only owns device buffers (torch tensors) and strings the C entry points
together in the order of Algorithm 1:  for every layer: pull (predict) -> forward ->
push;  then loss, backward, commit.  It contains no arithmetic of its own.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B


def _pad4(d: int) -> int:
    return (d + 3) & ~3


def _buf(rows: int, d: int, device) -> torch.Tensor:
    """[rows, d] view of a zero-initialised buffer whose row stride is a multiple of 4 floats."""
    full = torch.zeros((max(rows, 1), _pad4(d)), dtype=torch.float32, device=device)
    return full[:rows, :d]


class SatEpoch:
    """Holds a context, the partitioned graph, the cache ring and the activation / gradient buffers
    of a GCN with layer widths `dims`, and runs epochs either with one launch set for all
    partitions (`step`) or partition by partition (`step_per_partition`)."""

    def __init__(self, rowptr, col, M: int, dims, tau: int, loss: str, part_given=None, device: int = 0):
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.stream = torch.cuda.current_stream(self.device)
        self.ctx = B.sat_create(device, self.stream.cuda_stream)
        self.n = int(rowptr.shape[0] - 1)
        self.M, self.dims, self.tau, self.loss = M, list(dims), tau, loss
        self.L = len(dims) - 1
        B.sat_graph_load(self.ctx, rowptr, col)
        if part_given is None:
            B.sat_partition(self.ctx, M, B.SAT_PART_CONTIG_BLOCKS)
        else:
            B.sat_partition(self.ctx, M, B.SAT_PART_GIVEN, part_given)
        self.sizes = [B.sat_part_sizes(self.ctx, m) for m in range(M)]
        tot = B.sat_part_sizes(self.ctx, B.SAT_ALL_PARTS)
        self.nb, self.nnz, self.n_slots = tot[1], tot[2], tot[3]
        self.inner_off = np.concatenate([[0], np.cumsum([s[0] for s in self.sizes])]).astype(np.int64)
        self.halo_off = np.concatenate([[0], np.cumsum([s[1] for s in self.sizes])]).astype(np.int64)
        B.sat_cache_init(self.ctx, self.dims[1:-1], tau)
        dev = self.device
        self.H = [None] + [_buf(self.n, d, dev) for d in self.dims[1:]]          # H[l], l = 1..L (partition-major rows)
        self.G = [None] + [_buf(self.n, d, dev) for d in self.dims[1:]]          # gradient w.r.t. H[l]
        self.halo = _buf(self.nb, max(self.dims[1:-1] or [1]), dev)               # predicted halo input of the running layer (layers >= 2)
        self.X_in = None                                                          # partition-major copy of the features (made on demand)
        self.gW = [torch.zeros((self.dims[l], self.dims[l + 1]), dtype=torch.float32, device=dev) for l in range(self.L)]
        self.gb = [torch.zeros(self.dims[l + 1], dtype=torch.float32, device=dev) for l in range(self.L)]
        self.loss_sum = torch.zeros(1, dtype=torch.float64, device=dev)
        self.X = None
        self.labels = None

    def close(self):
        """Destroys the context and drops the activation / gradient buffers (sizes and offsets stay readable)."""
        if self.ctx is not None:
            B.sat_destroy(self.ctx)
            self.ctx = None
        self.H = self.G = self.halo = self.X_in = self.X = self.labels = None
        if hasattr(self, "gat_halo"):
            self.gat_halo = None

    # ---- inputs -------------------------------------------------------------------
    def set_inputs(self, X: torch.Tensor, labels_perm: torch.Tensor):
        """X: [n, d0] CUDA features in global id order (row stride multiple of 4);
        labels_perm: labels in partition-major row order (int32 [n] or uint8 [n, C])."""
        self.X = X
        self.labels = labels_perm
        self.X_in = None

    def inner_features(self) -> torch.Tensor:
        """The features of the inner nodes in partition-major row order (a gathered copy, made when first asked for: the
        GCN layer step reads the feature matrix itself)."""
        if self.X_in is None:
            self.X_in = _buf(self.n, self.dims[0], self.device)
            B.sat_gather_rows(self.ctx, B.SAT_ALL_PARTS, B.SAT_ROWS_INNER, self.X, self.X_in)
        return self.X_in

    def halo_view(self, l: int, m: int = B.SAT_ALL_PARTS):
        """Halo rows of the input of GNN layer l + 1 (predicted embeddings of cached layer l), all partitions or one."""
        d = self.dims[l]
        if m == B.SAT_ALL_PARTS:
            return self.halo[:, :d]
        return self.halo[self.halo_off[m]:self.halo_off[m + 1], :d]

    def rows(self, t: torch.Tensor, m: int):
        if m == B.SAT_ALL_PARTS:
            return t
        return t[self.inner_off[m]:self.inner_off[m + 1]]

    # ---- one epoch ----------------------------------------------------------------
    def _forward_backward(self, m: int, W, b, pred, accumulate: int, reuse_state: int, grad_history: bool = False):
        ctx, L = self.ctx, self.L
        h_in = None
        for l in range(1, L + 1):
            act = (B.SAT_ACT_RELU | B.SAT_FWD_PUSH) if l < L else B.SAT_ACT_NONE
            if l == 1:
                # layer 1: in- and out-of-subgraph rows are raw features, exact; the layer reads both from the feature matrix
                # itself (global id order) through the partition's inner and halo lists: no gathered copies, no pull
                h_in, hv = self.X, None
                act |= B.SAT_FWD_INPUT_GLOBAL
            else:
                hv = self.halo_view(l - 1, m)
                B.sat_predict(ctx, l - 1, m, pred[l - 2] if pred is not None else None, reuse_state, hv)  # pull predicted
            h_out = self.rows(self.H[l], m)
            # forward; for the cached layers the push of the boundary rows rides on the transform's epilogue
            B.sat_layer_fwd(ctx, m, l, h_in, hv, W[l - 1], b[l - 1], act, h_out)
            h_in = h_out
        kind = B.SAT_LOSS_SOFTMAX_CE if self.loss == "ce" else B.SAT_LOSS_SIGMOID_BCE
        g = self.rows(self.G[L], m)
        B.sat_loss_grad(ctx, m, kind, self.rows(self.H[L], m), self.rows(self.labels, m), self.loss_sum, g)
        for l in range(L, 0, -1):
            g_in = self.rows(self.G[l - 1], m) if l > 1 else None
            # the gradient handed down is written already multiplied by the ReLU mask of the layer below (no separate pass)
            flags = accumulate | (B.SAT_BWD_MASK_G_IN if l > 1 else 0) | (B.SAT_BWD_G_OUT_MASKED if l < L else 0)
            if grad_history and l > 1:
                flags |= B.SAT_BWD_GRAD_HISTORY      # stale-gradient term of the Appendix's back-propagation
            B.sat_layer_bwd(ctx, m, l, g, W[l - 1], self.gW[l - 1], self.gb[l - 1], flags, g_in, None)
            g = g_in

    def pred_update(self, pred, lr: float, max_steps: int = 1, min_gain: float | None = None, row_weight=None):
        """Algorithm 1 "Embedding predictor update", to be called after the pushes of an epoch and before the commit:
        up to max_steps gradient steps omega <- omega - lr grad L_Pred per cached layer, on the parameter tensors behind the
        sat_pred_params; the parameter version (when one is used) is bumped.  min_gain switches early stopping on: the
        steps of a layer end when a step lowered the loss by less than that fraction (this reads the loss back every
        step).  row_weight: per cached layer a CUDA fp32 [sum_m b_m] of mini-batch weights, or None.
        Returns the losses seen, per cached layer (empty lists without early stopping)."""
        seen = []
        for l in range(1, self.L):
            p = pred[l - 1]
            losses = []
            if p is None:
                seen.append(losses)
                continue
            if not hasattr(p, "_grads"):
                p._grads = tuple(torch.zeros_like(t) for t in p._keep)
            rw = None if row_weight is None else row_weight[l - 1]
            for _ in range(max_steps):
                loss = B.sat_pred_grad(self.ctx, l, p, rw, *p._grads, want_loss=min_gain is not None)
                if min_gain is not None:
                    losses.append(loss)
                    if len(losses) > 1 and losses[-1] > (1.0 - min_gain) * losses[-2]:
                        break
                B.sat_sgd_steps(self.ctx, list(p._keep), list(p._grads), lr)
                if p.version:
                    p.version += 1
            seen.append(losses)
        return seen

    def step(self, W, b, pred, lr: float | None = None, pred_lr: float | None = None, grad_history: bool = False):
        """All partitions per launch.  W, b: lists of CUDA tensors; pred: list of sat_pred_params or None.
        pred_lr: also run one predictor update (pred_update) before the ring is committed.
        grad_history: back-propagate with the stale-gradient term (gradient-side history of the previous epoch)."""
        self.loss_sum.zero_()
        self._forward_backward(B.SAT_ALL_PARTS, W, b, pred, 0, 0, grad_history)
        if pred_lr is not None and pred is not None:
            self.pred_update(pred, pred_lr)
        B.sat_cache_commit(self.ctx)
        if lr is not None:
            B.sat_sgd_steps(self.ctx, list(W) + list(b), list(self.gW) + list(self.gb), lr)

    def step_per_partition(self, W, b, pred, order=None, lr: float | None = None, grad_history: bool = False):
        """Same epoch, one partition at a time (the LSTM state table is computed by the first call of every layer)."""
        self.loss_sum.zero_()
        for i, m in enumerate(order if order is not None else range(self.M)):
            self._forward_backward(m, W, b, pred, 0 if i == 0 else 1, 0 if i == 0 else 1, grad_history)
        B.sat_cache_commit(self.ctx)
        if lr is not None:
            B.sat_sgd_steps(self.ctx, list(W) + list(b), list(self.gW) + list(self.gb), lr)

    # ---- graph-attention backbone ---------------------------------------------------
    def step_gat(self, params, pred, lr: float | None = None):
        """One SAT epoch with graph-attention layers in place of the GCN layers, all partitions per launch: the pull / predict,
        push, loss and commit calls are the same; sat_gat_fwd / sat_gat_bwd take the place of sat_layer_fwd / sat_layer_bwd.
        params: per layer dict(W, a_src, a_dst, b) of CUDA tensors.  The gradients land in self.gat_grads (same keys)."""
        ctx, L, m = self.ctx, self.L, B.SAT_ALL_PARTS
        dev = self.device
        if not hasattr(self, "gat_grads"):
            self.gat_grads = [{k: torch.zeros_like(v) for k, v in p.items()} for p in params]
            self.gat_halo = [_buf(self.nb, self.dims[l], dev) for l in range(L)]       # the pulled embeddings are needed again in the backward
        self.loss_sum.zero_()
        h_in = self.inner_features()
        ins = []
        for l in range(1, L + 1):
            hv = self.gat_halo[l - 1]
            if l == 1:
                B.sat_gather_rows(ctx, m, B.SAT_ROWS_HALO, self.X, hv)
            else:
                B.sat_predict(ctx, l - 1, m, pred[l - 2] if pred is not None else None, 0, hv)
            p = params[l - 1]
            B.sat_gat_fwd(ctx, m, l, h_in, hv, p["W"], p["a_src"], p["a_dst"], p["b"], B.SAT_ACT_RELU if l < L else B.SAT_ACT_NONE, self.H[l])
            if l < L:
                B.sat_cache_update(ctx, m, l, self.H[l])
            ins.append(h_in)
            h_in = self.H[l]
        kind = B.SAT_LOSS_SOFTMAX_CE if self.loss == "ce" else B.SAT_LOSS_SIGMOID_BCE
        g = self.G[L]
        B.sat_loss_grad(ctx, m, kind, self.H[L], self.labels, self.loss_sum, g)
        for l in range(L, 0, -1):
            p, gr = params[l - 1], self.gat_grads[l - 1]
            g_in = self.G[l - 1] if l > 1 else None
            B.sat_gat_bwd(ctx, m, l, g, self.H[l], ins[l - 1], self.gat_halo[l - 1], p["W"], p["a_src"], p["a_dst"], gr["W"], gr["a_src"], gr["a_dst"],
                          gr["b"], 0, g_in)
            g = g_in
        B.sat_cache_commit(ctx)
        if lr is not None:
            keys = [(l, k) for l, p in enumerate(params) for k in p]
            B.sat_sgd_steps(ctx, [params[l][k] for l, k in keys], [self.gat_grads[l][k] for l, k in keys], lr)
