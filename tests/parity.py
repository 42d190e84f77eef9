"""Helpers shared by the GPU parity tests: moving tensors to the oracle's numpy
formats and the comparison rule."""
import numpy as np
import torch

REL_TOL = 1e-6     # max relative error on fp32 params and momentum (the stated bar)


def grad_to_numpy(t: torch.Tensor) -> np.ndarray:
    """fp32 -> float32 array; bf16 -> uint16 array of the raw bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16).copy()
    return t.numpy().copy()


def assert_matches(gpu: torch.Tensor, want: np.ndarray, what: str, exact: bool = True) -> None:
    """The stated bar is max |gpu - want| / |want| <= 1e-6 with exact zeros where
    the oracle has zeros; the design point is equality of every bit (both sides
    run the same correctly rounded sequence), asserted when ``exact``."""
    got = gpu.detach().cpu().numpy()
    assert got.shape == want.shape, what
    both_nan = np.isnan(got) & np.isnan(want)
    zero = want == 0
    assert np.all(got[zero] == 0), "%s: nonzero where the oracle has zero" % what
    with np.errstate(divide="ignore", invalid="ignore"):
        rel = np.abs(got.astype(np.float64) - want.astype(np.float64)) / np.abs(want.astype(np.float64))
    rel[zero | both_nan] = 0.0
    same_inf = np.isinf(got) & (got == want)
    rel[same_inf] = 0.0
    worst = float(np.nanmax(rel)) if rel.size else 0.0
    assert not np.any(np.isnan(rel)), "%s: NaN mismatch" % what
    assert worst <= REL_TOL, "%s: max relative error %.3e" % (what, worst)
    if exact:
        diff = (got.view(np.uint32) != want.view(np.uint32)) & ~both_nan & ~(zero & (got == 0))
        assert not diff.any(), "%s: %d elements differ in bits (first at %d)" % (
            what, int(diff.sum()), int(np.argmax(diff)))


def sample_indices(n: int, seed: int, chunk: int = 4096, n_chunks: int = 48) -> np.ndarray:
    """Sorted unique element indices: the head, the ragged tail, and randomly
    placed contiguous runs (unaligned starts, so they straddle tile edges)."""
    if n <= (n_chunks + 2) * chunk:
        return np.arange(n, dtype=np.int64)
    rng = np.random.default_rng(seed)
    starts = [0, n - chunk] + [int(s) for s in rng.integers(0, n - chunk, n_chunks)]
    idx = np.concatenate([np.arange(s, s + chunk, dtype=np.int64) for s in starts])
    return np.unique(idx)
