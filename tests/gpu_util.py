"""Helpers of the GPU parity tests (test-only code)."""
from __future__ import annotations

import numpy as np

TOL = 1e-4  # max relative error for floating results (fp32 accumulate), see rel_err


def rel_err(got, want) -> float:
    """max_i |g_i - o_i| / max(|o_i|, rms(o)) — the per-tensor relative error the build is held to."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    if want.size == 0:
        return 0.0
    rms = float(np.sqrt(np.mean(want * want)))
    den = np.maximum(np.abs(want), rms)
    den = np.where(den == 0.0, 1.0, den)
    return float(np.max(np.abs(got - want) / den))


def assert_close(got, want, what: str, tol: float = TOL):
    e = rel_err(got, want)
    assert e <= tol, f"{what}: relative error {e:.3e} > {tol:.1e}"
    return e


def dev2d(a: np.ndarray, device="cuda"):
    """Upload a 2-D fp32 array into a buffer whose row stride is a multiple of 4 floats; returns the [r, d] view."""
    import torch
    a = np.ascontiguousarray(a, dtype=np.float32)
    r, d = a.shape
    full = torch.zeros((max(r, 1), (d + 3) & ~3), dtype=torch.float32, device=device)
    view = full[:r, :d]
    if r:
        view.copy_(torch.from_numpy(a))
    return view


def empty2d(r: int, d: int, device="cuda", fill=None):
    import torch
    full = torch.empty((max(r, 1), (d + 3) & ~3), dtype=torch.float32, device=device)
    full.fill_(float("nan") if fill is None else fill)
    return full[:r, :d]


def dev(a: np.ndarray, device="cuda"):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def pred_to_device(pred_list, B, version: int = 0):
    """Oracle-side predictor dicts -> list of sat_pred_params (device copies kept alive by the structs)."""
    out = []
    for p in pred_list:
        h = int(p["Wg"].shape[0])
        out.append(B.make_pred_params(dev(p["Wx"].astype(np.float32)), dev(p["Uh"].astype(np.float32)),
                                      dev(p["b"].astype(np.float32)), dev(p["Wg"].astype(np.float32)),
                                      dev(p["bg"].astype(np.float32)), h, version,
                                      B.SAT_CELL_GRU if p.get("cell", "lstm") == "gru" else B.SAT_CELL_LSTM))
    return out


TIE = 1e-4  # a hidden pre-activation with |Z| <= TIE * rms(Z) is below the tolerance of Z itself: its ReLU mask bit is a tie


def relu_tie_masks(res, P, H_gpu, inner_off, L):
    """Compares the oracle's ReLU masks [Z > 0] with the CUDA path's (H > 0) for every partition and hidden layer.

    Where |Z| is at rounding level the two sides may decide the sign differently and both are correct; anywhere else a
    disagreement is an error (asserted).  Returns (masks, differs): masks[m][l-1] = the CUDA path's decision (uint8) to hand
    to the oracle's backward, differs = whether any tie was decided differently."""
    masks, differs = [None] * P.M, False
    for m in range(P.M):
        if res.per_part[m] is None:
            continue
        masks[m] = []
        r0 = int(inner_off[m])
        for l in range(1, L):
            Z = res.per_part[m]["Z"][l - 1]
            theirs = H_gpu[l][r0:r0 + Z.shape[0]] > 0
            diff = (Z > 0) != theirs
            if diff.any():
                rms = float(np.sqrt(np.mean(Z * Z)))
                assert np.all(np.abs(Z[diff]) <= TIE * rms), f"ReLU mask disagreement away from zero (partition {m}, layer {l})"
                differs = True
            masks[m].append(theirs.astype(np.uint8))
        masks[m].append(None)
    return masks, differs
