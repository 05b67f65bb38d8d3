"""The five synthetic workloads (graph + features + labels + initial parameters).

Shapes follow the dataset table of the paper (Table I) and the benchmark
configurations this build is measured on; the files of those datasets are not used —
every value is drawn from the seeded generators of this package.

  tiny        2,048-node SBM, 4 blocks = 4 partitions, avg degree 8 (p_in : p_out = 9 : 1),
              32 -> 16 -> 4, predictor history 3
  medium      169,343 nodes, 1.2 M accepted directed R-MAT samples symmetrised,
              128 -> 256 -> 256 -> 40, 8 partitions, history 4
  dense       232,965 nodes, 57 M distinct undirected R-MAT edges (~114 M directed, avg
              degree ~490), 602 -> 256 -> 41, 16 partitions, history 4
  large       2,449,029 nodes, 62 M distinct undirected edges (~124 M directed),
              100 -> 256 -> 256 -> 47, 32 partitions, history 4
  multilabel  717,000 nodes, 7 M distinct undirected edges, 300 -> 512 -> 512 -> 512 -> 100,
              100 independent Bernoulli(0.1) labels, 16 partitions, history 8
  odd         (parity tests only) 6,000-node R-MAT graph, 50 -> 72 -> 40 -> 7, 3 partitions, history 3,
              predictor width 24, non-zero biases everywhere: widths that are no multiple of a tile, a k-block or 8

R-MAT graphs use (a, b, c, d) = (0.57, 0.19, 0.19, 0.05), get a seeded id permutation,
and are then relabelled in BFS order so that contiguous id blocks are the partitions.
`shrink=s` divides the node and edge counts by s (dimensions, partition count and
history depth stay), which gives parity-test sizes with the same structure.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from .graphs import bfs_relabel, rmat_graph, sbm_graph
from .tensors import bernoulli_labels, glorot_uniform, normal_features, uniform_labels

WORKLOADS = {
    "tiny": dict(kind="sbm", n=2048, blocks=4, avg_degree=8.0, ratio=9.0,
                 dims=[32, 16, 4], M=4, tau=3, h=16, loss="ce"),
    "medium": dict(kind="rmat", scale=18, n=169_343, n_samples=1_200_000,
                   dims=[128, 256, 256, 40], M=8, tau=4, h=64, loss="ce"),
    "dense": dict(kind="rmat", scale=18, n=232_965, n_unique=57_000_000,
                  dims=[602, 256, 41], M=16, tau=4, h=64, loss="ce"),
    "large": dict(kind="rmat", scale=22, n=2_449_029, n_unique=62_000_000,
                  dims=[100, 256, 256, 47], M=32, tau=4, h=64, loss="ce"),
    "multilabel": dict(kind="rmat", scale=20, n=717_000, n_unique=7_000_000,
                       dims=[300, 512, 512, 512, 100], M=16, tau=8, h=64, loss="bce"),
    "odd": dict(kind="rmat", scale=13, n=6_000, n_samples=40_000,
                dims=[50, 72, 40, 7], M=3, tau=3, h=24, loss="ce", bias=0.1),
}


@dataclass
class Workload:
    name: str
    seed: int
    n: int
    rowptr: np.ndarray            # int64 [n+1]
    col: np.ndarray               # int32 [nnz_offdiag]; symmetric, sorted rows, no self-loops
    M: int                        # number of partitions
    part_given: np.ndarray | None # int32 [n] when the workload prescribes the partition, else None
                                  # (None: partitions are contiguous id blocks, computed by the consumer)
    dims: list                    # d_0 .. d_L
    tau: int
    h: int
    loss: str                     # "ce" | "bce"
    X: np.ndarray                 # fp32 [n, d_0]
    labels: np.ndarray            # int32 [n] (ce) or uint8 [n, d_L] (bce)
    W: list = field(default_factory=list)     # per GNN layer fp32 [d_{l-1}, d_l]
    b: list = field(default_factory=list)     # per GNN layer fp32 [d_l] (zeros)
    pred: list = field(default_factory=list)  # per cached layer dict(Wx, Uh, b, Wg, bg)

    @property
    def L(self) -> int:
        return len(self.dims) - 1

    @property
    def nnz(self) -> int:
        """Non-zeros of A + I (both edge directions plus one self-loop per node)."""
        return int(self.col.shape[0]) + self.n


def _bias(seed: int, d: int, tag: str, scale: float) -> np.ndarray:
    """Zeros (the benchmark workloads) or seeded values in (-scale sqrt(6/(1+d)), +...) x sqrt(1+d): order `scale`."""
    if scale == 0.0:
        return np.zeros(d, dtype=np.float32)
    u = glorot_uniform(seed, 1, d, tag).reshape(d)          # uniform in +-sqrt(6 / (1 + d))
    return (u * (scale / np.sqrt(6.0 / (1 + d)))).astype(np.float32)


def make_workload(name: str, seed: int = 0, shrink: int = 1, with_dense: bool = True, **overrides) -> Workload:
    """`overrides` replace entries of the workload's configuration (e.g. h=20, bias=0.05)."""
    cfg = dict(WORKLOADS[name])
    cfg.update(overrides)
    part_given = None
    if cfg["kind"] == "sbm":
        n = cfg["n"] // shrink
        nb = cfg["blocks"]
        bs = n // nb
        # expected degree = (bs-1) p_in + (n-bs) p_out with p_in = ratio * p_out
        p_out = cfg["avg_degree"] / ((bs - 1) * cfg["ratio"] + (n - bs))
        rowptr, col, block = sbm_graph(seed, n, nb, cfg["ratio"] * p_out, p_out)
        part_given = block.astype(np.int32)
    else:
        n = cfg["n"] // shrink
        scale = cfg["scale"]
        s = shrink
        while s > 1:
            scale -= 1
            s //= 2
        while (1 << scale) < n:
            scale += 1
        kw = {}
        if "n_samples" in cfg:
            kw["n_samples"] = cfg["n_samples"] // shrink
        else:
            kw["n_unique_undirected"] = cfg["n_unique"] // shrink
        if "attach_isolated" in cfg:          # False keeps the nodes R-MAT leaves without an edge (degenerate-case tests)
            kw["attach_isolated"] = bool(cfg["attach_isolated"])
        rowptr, col = rmat_graph(seed, scale, n, **kw)
        rowptr, col, _ = bfs_relabel(rowptr, col)
    dims = list(cfg["dims"])
    L = len(dims) - 1
    wl = Workload(name=name, seed=seed, n=n, rowptr=rowptr, col=col, M=cfg["M"], part_given=part_given,
                  dims=dims, tau=cfg["tau"], h=cfg["h"], loss=cfg["loss"],
                  X=None, labels=None)
    if with_dense:
        wl.X = normal_features(seed, n, dims[0])
        if cfg["loss"] == "ce":
            wl.labels = uniform_labels(seed, n, dims[-1])
        else:
            wl.labels = bernoulli_labels(seed, n, dims[-1], 0.1)
    for l in range(1, L + 1):
        wl.W.append(glorot_uniform(seed, dims[l - 1], dims[l], f"W{l}"))
        wl.b.append(_bias(seed, dims[l], f"b{l}", cfg.get("bias", 0.0)))
    for l in range(1, L):  # cached layers store H^(l), width dims[l]
        d, h = dims[l], min(cfg["h"], dims[l])
        wl.pred.append(dict(
            Wx=glorot_uniform(seed, d, 4 * h, f"pred{l}.Wx"),
            Uh=glorot_uniform(seed, h, 4 * h, f"pred{l}.Uh"),
            b=_bias(seed, 4 * h, f"pred{l}.b", cfg.get("bias", 0.0)),
            Wg=glorot_uniform(seed, h, d, f"pred{l}.Wg"),
            bg=_bias(seed, d, f"pred{l}.bg", cfg.get("bias", 0.0)),
            h=h,
        ))
    return wl


def as_gru(pred):
    """GRU-shaped parameters cut out of LSTM-shaped ones (a generator of inputs, no arithmetic): the first 3h gate columns
    of Wx and Uh become (r, z, n); the 4h bias entries become (b_r, b_z, b_n, b_hn)."""
    out = []
    for p in pred:
        h = int(p["h"])
        q = dict(p)
        q["Wx"] = np.ascontiguousarray(p["Wx"][:, :3 * h])
        q["Uh"] = np.ascontiguousarray(p["Uh"][:, :3 * h])
        q["cell"] = "gru"
        out.append(q)
    return out
