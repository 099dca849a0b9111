"""Shared helpers of the GPU parity tests (comparison against the fp64 oracle)."""
import numpy as np
import torch

TOL = {torch.bfloat16: (2e-2, 1e-3), torch.float32: (1e-4, 1e-3)}   # (max-abs O, max-abs LSE)


def compare(o_gpu, lse_gpu, o_ref, lse_ref, tol_o, tol_lse, what=""):
    """Element-wise max-abs comparison; -inf LSE entries must match exactly and have O == 0."""
    o = o_gpu.detach().float().cpu().double().numpy()
    lse = lse_gpu.detach().float().cpu().double().numpy()
    assert o.shape == o_ref.shape and lse.shape == lse_ref.shape, (what, o.shape, o_ref.shape)
    assert not np.isnan(o).any() and not np.isnan(lse).any(), f"{what}: NaN in the GPU result"
    empty = np.isneginf(lse_ref)
    assert np.array_equal(np.isneginf(lse), empty), f"{what}: empty-row pattern differs"
    assert (o[empty] == 0).all(), f"{what}: empty rows must be zero"
    err_o = float(np.abs(o - o_ref).max()) if o.size else 0.0
    fin = ~empty
    err_l = float(np.abs(lse[fin] - lse_ref[fin]).max()) if fin.any() else 0.0
    print(f"[parity] {what}: max|dO| = {err_o:.3e} (tol {tol_o:g}), max|dLSE| = {err_l:.3e} (tol {tol_lse:g})")
    assert err_o <= tol_o, f"{what}: max |dO| = {err_o:.3e} > {tol_o}"
    assert err_l <= tol_lse, f"{what}: max |dLSE| = {err_l:.3e} > {tol_lse}"
    return err_o, err_l


def sample_rows(seq_len, boundaries, n_random, seed, lo=0, hi=None):
    """Rows next to every given boundary plus seeded random rows, inside [lo, hi)."""
    hi = seq_len if hi is None else hi
    rows = {lo, hi - 1}
    for b in boundaries:
        for d in (-1, 0, 1):
            if lo <= b + d < hi:
                rows.add(b + d)
    g = np.random.Generator(np.random.Philox(key=seed))
    rows.update(int(x) for x in g.integers(lo, hi, size=n_random))
    return sorted(rows)
