"""Shared helpers for the GPU-vs-oracle parity tests: tolerances, canaries, sampling."""
import numpy as np
import torch

# Tolerances of the build target:
#   bf16 results:  |x - ref| <= 1e-2 |ref| + 2e-3 elementwise, and two scale-free additions
#                  (the absolute term is larger than some gradients): relative Frobenius error
#                  <= 5e-3 and max |x - ref| <= 2^-7 max|ref|
#   fp32 dweight / dbias: relative Frobenius error <= 5e-3
BF16_RTOL, BF16_ATOL = 1e-2, 2e-3
FROB_TOL = 5e-3
MAXABS_FRAC = 2.0 ** -7


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def rel_frob(x, ref) -> float:
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    d = np.linalg.norm(ref)
    return float(np.linalg.norm(x - ref) / d) if d > 0 else float(np.linalg.norm(x))


def check_bf16(x, ref, name: str, extra=None):
    """``extra`` (array or None) widens the elementwise bound where the definition of the call
    itself rounds an intermediate: the caller derives it from that rounding."""
    x = f32(x).astype(np.float64) if torch.is_tensor(x) else np.asarray(x, np.float64)
    ref = np.asarray(ref, np.float64)
    assert x.shape == ref.shape, (name, x.shape, ref.shape)
    assert np.isfinite(x).all(), name
    err = np.abs(x - ref)
    bound = BF16_RTOL * np.abs(ref) + BF16_ATOL
    if extra is not None:
        bound = bound + np.asarray(extra, np.float64)
    bad = err > bound
    assert not bad.any(), f"{name}: {int(bad.sum())}/{bad.size} elements out of tolerance, worst {err.max():.3e}"
    if np.abs(ref).max() > 0:
        r = rel_frob(x, ref)
        assert r <= FROB_TOL, f"{name}: relative Frobenius error {r:.3e}"
        assert err.max() <= MAXABS_FRAC * np.abs(ref).max(), f"{name}: max abs error {err.max():.3e}"
    else:
        assert err.max() == 0.0, name


def check_f32(x, ref, name: str):
    x = f32(x).astype(np.float64) if torch.is_tensor(x) else np.asarray(x, np.float64)
    ref = np.asarray(ref, np.float64)
    assert x.shape == ref.shape, (name, x.shape, ref.shape)
    assert np.isfinite(x).all(), name
    r = rel_frob(x, ref)
    assert r <= FROB_TOL, f"{name}: relative Frobenius error {r:.3e}"


class Guarded:
    """A device tensor with canary rows before and after it, to catch out-of-bounds writes."""
    PAD = 4096  # elements

    def __init__(self, shape, dtype, device="cuda", fill=None):
        n = int(np.prod(shape))
        self.buf = torch.empty(n + 2 * self.PAD, dtype=dtype, device=device)
        self.canary = 12345.0 if dtype != torch.bfloat16 else 12352.0
        self.buf.fill_(self.canary)
        self.t = self.buf[self.PAD:self.PAD + n].view(*shape)
        assert self.t.data_ptr() % 16 == 0
        if fill is not None:
            self.t.fill_(fill)

    def check(self, name=""):
        assert torch.all(self.buf[:self.PAD] == self.canary), f"{name}: write before the buffer"
        assert torch.all(self.buf[-self.PAD:] == self.canary), f"{name}: write past the buffer"


def sample_indices(n: int, k: int, seed: int) -> np.ndarray:
    """k distinct indices of range(n), always including both ends."""
    k = min(k, n)
    rng = np.random.default_rng(seed)
    idx = set([0, n - 1]) if n > 1 else set([0])
    while len(idx) < k:
        idx.add(int(rng.integers(0, n)))
    return np.array(sorted(idx), dtype=np.int64)


def stratified_indices(n: int, box: int, seed: int) -> np.ndarray:
    """One index in every consecutive box of `box` indices of range(n), at a seeded offset inside
    the box: a grid of such rows and columns puts an element into every tile and every store box
    of a result, whatever the tiling."""
    rng = np.random.default_rng(seed)
    starts = np.arange(0, n, box, dtype=np.int64)
    idx = np.minimum(starts + rng.integers(0, box, size=starts.size), n - 1)
    return np.unique(idx)
